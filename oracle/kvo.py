"""ctypes loader for the oracle (oracle/kvo.c).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's cpu_baseline leg may import this module; the
product package never does.  Arrays are numpy, host memory, in the paper's plain layout:
K, V [S, n, d] and q [S, d] as bf16 bit patterns (uint16), S = batch * heads.
"""
import ctypes as C
import os

import numpy as np

from . import build as _build

AGG_MEAN, AGG_MLP, AGG_IDENTITY, AGG_MAX, AGG_TOKEN_MLP = 0, 1, 2, 3, 4
ATTEND_SUMMARY, ATTEND_RAW = 0, 1

_u16p = C.POINTER(C.c_uint16)
_f32p = C.POINTER(C.c_float)
_i32p = C.POINTER(C.c_int32)
_i64p = C.POINTER(C.c_int64)


def _ptr(a, typ):
    if a is None:
        return C.cast(None, typ)
    assert a.flags["C_CONTIGUOUS"], "oracle arrays must be C-contiguous"
    return a.ctypes.data_as(typ)


def set_threads(n: int) -> None:
    """Number of OpenMP threads the oracle's per-sequence loops use."""
    C.CDLL("libgomp.so.1").omp_set_num_threads(int(n))


class Oracle:
    """kind = 'f64' (mathematical reference) or 'f32' (decisions in the kernels' precision)."""

    def __init__(self, kind: str = "f64"):
        assert kind in ("f32", "f64")
        _build.build()
        self.kind = kind
        self.real = np.float32 if kind == "f32" else np.float64
        self._realp = C.POINTER(C.c_float if kind == "f32" else C.c_double)
        self.lib = C.CDLL(_build.lib_path(kind))
        assert self.lib.kvo_real_bytes() == np.dtype(self.real).itemsize
        self.lib.kvo_bf16_rne.restype = C.c_uint16
        self.lib.kvo_bf16_rne.argtypes = [C.c_double]
        self.lib.kvo_bf16_widen.restype = C.c_double
        self.lib.kvo_bf16_widen.argtypes = [C.c_uint16]

    # -- scalar helpers (for tests of the rounding routine) --
    def bf16_rne(self, x: float) -> int:
        return int(self.lib.kvo_bf16_rne(float(x)))

    def bf16_widen(self, b: int) -> float:
        return float(self.lib.kvo_bf16_widen(int(b)))

    # -- Eq. 2 --
    def summarize(self, K, V, Cs, t0, t1, agg=AGG_MEAN, mlp=None, stride=None, out=None):
        S, n, d = K.shape
        stride = int(stride if stride is not None else max(t1, 1))
        if out is None:
            out = dict(ksum=np.zeros((S, stride, d), self.real), vsum=np.zeros((S, stride, d), self.real),
                       ksum_b16=np.zeros((S, stride, d), np.uint16), vsum_b16=np.zeros((S, stride, d), np.uint16))
        w = {}
        d_sum = 0
        if agg in (AGG_MLP, AGG_TOKEN_MLP):
            d_sum = mlp["W1K"].shape[0]
            for k in ("W1K", "b1K", "W2K", "b2K", "W1V", "b1V", "W2V", "b2V"):
                w[k] = np.ascontiguousarray(mlp[k], np.float32)
        g = lambda k: _ptr(w.get(k), _f32p)
        rc = self.lib.kvo_summarize(
            _ptr(K, _u16p), _ptr(V, _u16p), C.c_int(S), C.c_int(n), C.c_int(d), C.c_int(Cs),
            C.c_int(t0), C.c_int(t1), C.c_int(agg), C.c_int(d_sum),
            g("W1K"), g("b1K"), g("W2K"), g("b2K"), g("W1V"), g("b1V"), g("W2V"), g("b2V"),
            C.c_int(stride), _ptr(out["ksum"], self._realp), _ptr(out["vsum"], self._realp),
            _ptr(out["ksum_b16"], _u16p), _ptr(out["vsum_b16"], _u16p))
        if rc != 0:
            raise ValueError(f"kvo_summarize rc={rc}")
        return out

    # -- Eq. 3 --
    def gate(self, ksum_b16, vsum_b16, t0, t1, lstm, h=None, c=None, scores=None):
        S, stride, d = ksum_b16.shape
        d_g = lstm["W_hh"].shape[1]
        if h is None:
            h = np.zeros((S, d_g), self.real)
        if c is None:
            c = np.zeros((S, d_g), self.real)
        if scores is None:
            scores = np.zeros((S, stride), self.real)
        W_ih = np.ascontiguousarray(lstm["W_ih"], np.float32)
        W_hh = np.ascontiguousarray(lstm["W_hh"], np.float32)
        b_ih = np.ascontiguousarray(lstm["b_ih"], np.float32)
        b_hh = np.ascontiguousarray(lstm["b_hh"], np.float32)
        w_s = np.ascontiguousarray(lstm["w_s"], np.float32)
        assert W_ih.shape == (4 * d_g, 2 * d) and W_hh.shape == (4 * d_g, d_g)
        rc = self.lib.kvo_gate(
            _ptr(ksum_b16, _u16p), _ptr(vsum_b16, _u16p), C.c_int(S), C.c_int(stride), C.c_int(d),
            C.c_int(t0), C.c_int(t1), C.c_int(d_g), _ptr(W_ih, _f32p), _ptr(W_hh, _f32p),
            _ptr(b_ih, _f32p), _ptr(b_hh, _f32p), _ptr(w_s, _f32p), C.c_float(float(lstm["b_s"])),
            _ptr(h, self._realp), _ptr(c, self._realp), _ptr(scores, self._realp))
        if rc != 0:
            raise ValueError(f"kvo_gate rc={rc}")
        return scores, h, c

    # -- retention rule --
    def compact(self, scores, n_chunks, tau):
        S, stride = scores.shape
        keep_idx = np.full((S, stride), -1, np.int32)
        keep_cnt = np.zeros((S,), np.int32)
        rc = self.lib.kvo_compact(_ptr(scores, self._realp), C.c_int(S), C.c_int(stride),
                                  C.c_int(n_chunks), C.c_double(float(tau)),
                                  _ptr(keep_idx, _i32p), _ptr(keep_cnt, _i32p))
        if rc != 0:
            raise ValueError(f"kvo_compact rc={rc}")
        return keep_idx, keep_cnt

    # -- gating variant: keep the k highest-scoring chunks (ties: older chunk first) --
    def compact_topk(self, scores, n_chunks, k):
        S, stride = scores.shape
        keep_idx = np.full((S, stride), -1, np.int32)
        keep_cnt = np.zeros((S,), np.int32)
        rc = self.lib.kvo_compact_topk(_ptr(scores, self._realp), C.c_int(S), C.c_int(stride), C.c_int(n_chunks),
                                       C.c_int(int(k)), _ptr(keep_idx, _i32p), _ptr(keep_cnt, _i32p))
        if rc != 0:
            raise ValueError(f"kvo_compact_topk rc={rc}")
        return keep_idx, keep_cnt

    # -- Sec. 3.3 memory reduction: pages of gated chunks handed back --
    def reclaim(self, page_table, scores, t0, t1, tau, mode):
        """page_table [S, stride] int32 is edited in place (-1 where a page was handed back);
        returns the free list (int32 array) in sequence-major, chunk-ascending order."""
        S, stride = scores.shape
        assert page_table.shape == (S, stride) and page_table.dtype == np.int32 and page_table.flags.c_contiguous
        free = np.empty((S * max(t1 - t0, 0) + 1,), np.int32)
        self.lib.kvo_reclaim.restype = C.c_long
        m = self.lib.kvo_reclaim(_ptr(page_table, _i32p), _ptr(scores, self._realp), C.c_int(S), C.c_int(stride),
                                 C.c_int(t0), C.c_int(t1), C.c_double(float(tau)), C.c_int(mode), _ptr(free, _i32p))
        if m < 0:
            raise ValueError(f"kvo_reclaim rc={m}")
        return free[:m].copy()

    # -- Sec. 3.3 attention over window + retained chunks --
    def attn(self, q, K, V, Cs, n_chunks, keep_idx, keep_cnt, ksum_b16, vsum_b16, attend, scale):
        S, n, d = K.shape
        stride = keep_idx.shape[1]
        if ksum_b16 is None:
            ksum_b16 = np.zeros((S, stride, d), np.uint16)
            vsum_b16 = np.zeros((S, stride, d), np.uint16)
        assert ksum_b16.shape == (S, stride, d)
        out = np.zeros((S, d), self.real)
        out_b16 = np.zeros((S, d), np.uint16)
        lse = np.zeros((S,), self.real)
        n_eff = np.zeros((S,), np.int64)
        rc = self.lib.kvo_attn(
            _ptr(q, _u16p), _ptr(K, _u16p), _ptr(V, _u16p), C.c_int(S), C.c_int(n), C.c_int(d),
            C.c_int(Cs), C.c_int(n_chunks), _ptr(keep_idx, _i32p), _ptr(keep_cnt, _i32p),
            _ptr(ksum_b16, _u16p), _ptr(vsum_b16, _u16p), C.c_int(stride), C.c_int(attend),
            C.c_double(float(scale)), _ptr(out, self._realp), _ptr(out_b16, _u16p),
            _ptr(lse, self._realp), _ptr(n_eff, _i64p))
        if rc != 0:
            raise ValueError(f"kvo_attn rc={rc}")
        return out, out_b16, lse, n_eff

    # -- Eq. 1 over the full cache --
    def attn_dense(self, q, K, V, scale):
        S, n, d = K.shape
        out = np.zeros((S, d), self.real)
        out_b16 = np.zeros((S, d), np.uint16)
        lse = np.zeros((S,), self.real)
        rc = self.lib.kvo_attn_dense(_ptr(q, _u16p), _ptr(K, _u16p), _ptr(V, _u16p), C.c_int(S),
                                     C.c_int(n), C.c_int(d), C.c_double(float(scale)),
                                     _ptr(out, self._realp), _ptr(out_b16, _u16p), _ptr(lse, self._realp))
        if rc != 0:
            raise ValueError(f"kvo_attn_dense rc={rc}")
        return out, out_b16, lse

    # -- Sec. 3.3 attention for a block of queries: T query tokens decoded together (the action
    #    tokens of Sec. 1 / Sec. 4.2) and Hq query heads on Hkv KV heads (grouped-query attention,
    #    Sec. 4.1: 32 heads on 8 KV heads).  Every (token, query head) pair is one independent
    #    query of Eq. 1 against the retained set of KV head hq // (Hq / Hkv); the tokens of a block
    #    do not see each other.  q [B, T, Hq, d] bf16 bits; results [B, T, Hq, d] / [B, T, Hq]. --
    def attn_block(self, q, Hkv, K, V, Cs, n_chunks, keep_idx, keep_cnt, ksum_b16, vsum_b16, attend, scale,
                   dense=False, causal=False):
        B, T, Hq, d = q.shape
        S = K.shape[0]
        assert S == B * Hkv and Hq % Hkv == 0
        G = Hq // Hkv
        out = np.zeros((B, T, Hq, d), self.real)
        out_b16 = np.zeros((B, T, Hq, d), np.uint16)
        lse = np.zeros((B, T, Hq), self.real)
        n = K.shape[1]
        for t in range(T):
            # causal: the block's tokens are the T newest tokens of the cache, and query token t attends (Eq. 1)
            # over the cache up to and including its own position, i.e. without the last T - 1 - t tokens
            n_t = n - (T - 1 - t) if causal else n
            assert n_t >= n_chunks * Cs, "the gated chunks lie before the block's tokens"
            Kt, Vt = (K, V) if n_t == n else (np.ascontiguousarray(K[:, :n_t]), np.ascontiguousarray(V[:, :n_t]))
            for g in range(G):
                # the g-th query head of every group: query head hkv * G + g reads KV head hkv
                qs = np.ascontiguousarray(q[:, t, g::G, :].reshape(S, d))
                if dense:
                    o, ob, l = self.attn_dense(qs, Kt, Vt, scale)
                else:
                    o, ob, l, _ = self.attn(qs, Kt, Vt, Cs, n_chunks, keep_idx, keep_cnt, ksum_b16, vsum_b16,
                                            attend, scale)
                out[:, t, g::G, :] = o.reshape(B, Hkv, d)
                out_b16[:, t, g::G, :] = ob.reshape(B, Hkv, d)
                lse[:, t, g::G] = l.reshape(B, Hkv)
        return out, out_b16, lse
