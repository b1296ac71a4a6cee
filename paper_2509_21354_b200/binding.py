"""Thin ctypes binding over libkve.so (C ABI in include/kve.h).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.  PyTorch is
used for device memory and streams.  There is no CPU fallback: if the library is missing or no
CUDA device is present, calls raise.

The module-level functions carry the C entry points' names (kvE_append, kvE_summarize_chunks,
kvE_gate, kvE_compact, kvE_decode_attn, ...) and take the same arguments with torch tensors in place
of device pointers; `Store` bundles the caller-owned buffers a handle needs.
"""
import ctypes as C
import os

import numpy as np
import torch

from . import build as _build

AGG = {"mean": 0, "mlp": 1, "identity": 2, "max": 3, "token_mlp": 4}
ATTEND = {"summary": 0, "raw": 1}
STATUS = {0: "KVE_OK", -1: "KVE_ERR_ARG", -2: "KVE_ERR_GEOMETRY", -3: "KVE_ERR_CAPACITY",
          -4: "KVE_ERR_STATE", -5: "KVE_ERR_CUDA", -6: "KVE_ERR_TIMEOUT"}

EXPORTS = ["kvE_workspace_bytes", "kvE_create", "kvE_destroy", "kvE_set_attend", "kvE_set_gate_planes", "kvE_append", "kvE_append_next", "kvE_set_len",
           "kvE_summarize_chunks", "kvE_gate", "kvE_gate_next", "kvE_refresh", "kvE_refresh_next", "kvE_adopt_device_state", "kvE_compact", "kvE_compact_topk", "kvE_decode_attn", "kvE_decode_step", "kvE_decode_attn_dense", "kvE_decode_attn_block",
           "kvE_decode_attn_static", "kvE_reclaim_pages", "kvE_decode_step_host", "kvE_decode_step_host_async", "kvE_poll_status", "kvE_layer_state", "kvE_last_cuda_error",
           "kvE_profile", "kvE_profile_read", "kvE_selftest_timeout"]
KERNEL_IDS = ["append", "chunk_mean", "chunk_mlp", "gate_proj", "gate_rnn", "compact", "attn", "attn_dense", "attn_block"]


class KveError(RuntimeError):
    def __init__(self, fn, rc, detail=""):
        self.rc = rc
        super().__init__(f"{fn} -> {STATUS.get(rc, rc)} {detail}".strip())


class kvE_config(C.Structure):
    _fields_ = [(k, C.c_int32) for k in ("B", "Hq", "Hkv", "d", "C", "W", "max_tokens", "n_layers", "agg",
                                         "d_sum", "d_g", "attend", "max_query_tokens")]


class kvE_buffers(C.Structure):
    _fields_ = [("k_pages", C.c_void_p), ("v_pages", C.c_void_p), ("n_pages", C.c_int64),
                ("page_table", C.c_void_p), ("seq_len", C.c_void_p),
                ("ksum_f32", C.c_void_p), ("vsum_f32", C.c_void_p), ("ksum_bf16", C.c_void_p), ("vsum_bf16", C.c_void_p),
                ("scores", C.c_void_p), ("keep_idx", C.c_void_p), ("keep_cnt", C.c_void_p),
                ("lstm_h", C.c_void_p), ("lstm_c", C.c_void_p),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t), ("status_word", C.c_void_p)]


class kvE_agg_weights(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in ("W1K", "W2K", "W1V", "W2V", "b1K", "b2K", "b1V", "b2V")]


class kvE_lstm_weights(C.Structure):
    _fields_ = [("W_ih", C.c_void_p), ("W_hh", C.c_void_p), ("b_ih", C.c_void_p), ("b_hh", C.c_void_p),
                ("w_s", C.c_void_p), ("b_s", C.c_float)]


_lib = None


def load_library(build_if_missing: bool = True) -> C.CDLL:
    """dlopen libkve.so (building it first if its sources are newer).  Raises if that fails."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB
    if build_if_missing:
        path = _build.build()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: run `python -m paper_2509_21354_b200.build`")
    lib = C.CDLL(path)
    lib.kvE_workspace_bytes.restype = C.c_size_t
    lib.kvE_workspace_bytes.argtypes = [C.POINTER(kvE_config)]
    lib.kvE_create.argtypes = [C.POINTER(kvE_config), C.POINTER(kvE_buffers), C.POINTER(C.c_void_p)]
    lib.kvE_destroy.argtypes = [C.c_void_p]
    lib.kvE_append.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int, C.POINTER(C.c_int), C.c_void_p]
    lib.kvE_set_len.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p]
    lib.kvE_set_attend.argtypes = [C.c_void_p, C.c_int]
    lib.kvE_set_gate_planes.argtypes = [C.c_void_p, C.c_int]
    lib.kvE_append_next.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p]
    lib.kvE_summarize_chunks.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.POINTER(kvE_agg_weights), C.c_void_p]
    lib.kvE_gate.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.POINTER(kvE_lstm_weights), C.c_void_p]
    lib.kvE_gate_next.argtypes = [C.c_void_p, C.c_int, C.POINTER(kvE_lstm_weights), C.c_float, C.c_void_p]
    lib.kvE_refresh_next.argtypes = [C.c_void_p, C.c_int, C.POINTER(kvE_agg_weights), C.POINTER(kvE_lstm_weights), C.c_float, C.c_void_p]
    lib.kvE_adopt_device_state.argtypes = [C.c_void_p, C.c_int, C.c_void_p]
    lib.kvE_compact.argtypes = [C.c_void_p, C.c_int, C.c_float, C.c_void_p]
    lib.kvE_refresh.argtypes = [C.c_void_p, C.c_int, C.POINTER(kvE_agg_weights), C.POINTER(kvE_lstm_weights), C.c_float, C.c_void_p]
    lib.kvE_compact_topk.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p]
    lib.kvE_decode_attn.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_float, C.c_void_p]
    lib.kvE_decode_attn_dense.argtypes = lib.kvE_decode_attn.argtypes
    lib.kvE_decode_step.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_float,
                                    C.c_int, C.c_void_p]
    lib.kvE_decode_attn_static.argtypes = lib.kvE_decode_attn.argtypes
    lib.kvE_decode_attn_block.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                          C.c_float, C.c_void_p]
    lib.kvE_reclaim_pages.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p]
    lib.kvE_decode_step_host.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                         C.POINTER(kvE_agg_weights), C.POINTER(kvE_lstm_weights), C.c_float,
                                         C.c_float, C.c_int, C.c_void_p]
    lib.kvE_decode_step_host_async.argtypes = lib.kvE_decode_step_host.argtypes
    lib.kvE_poll_status.argtypes = [C.c_void_p, C.POINTER(C.c_int)]
    lib.kvE_layer_state.argtypes = [C.c_void_p, C.c_int] + [C.POINTER(C.c_int)] * 4
    lib.kvE_profile.argtypes = [C.c_void_p, C.c_int]
    lib.kvE_profile_read.argtypes = [C.c_void_p, C.POINTER(C.c_float)]
    lib.kvE_selftest_timeout.argtypes = [C.c_void_p, C.c_int, C.c_void_p]
    lib.kvE_last_cuda_error.restype = C.c_char_p
    lib.kvE_last_cuda_error.argtypes = [C.c_void_p]
    for name in EXPORTS:
        fn = getattr(lib, name)
        if name not in ("kvE_workspace_bytes", "kvE_last_cuda_error"):
            fn.restype = C.c_int
    _lib = lib
    return lib


def _stream(stream=None) -> C.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _p(t) -> C.c_void_p:
    if t is None:
        return C.c_void_p(0)
    assert t.is_cuda and t.is_contiguous()
    return C.c_void_p(t.data_ptr())


def _check(fn, rc, handle=None):
    if rc != 0:
        detail = ""
        if rc == -5 and handle is not None:
            detail = load_library().kvE_last_cuda_error(handle).decode()
        raise KveError(fn, rc, detail)


def bits_to_bf16(a: np.ndarray, device="cuda") -> torch.Tensor:
    """numpy uint16 bf16 bit patterns -> torch.bfloat16 tensor on `device`."""
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(device).view(torch.bfloat16)


def bf16_to_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class AggWeights:
    """Device copies of the aggregator MLP weights (bf16 matrices, fp32 biases)."""

    def __init__(self, w: dict, device="cuda"):
        self.t = {}
        for k in ("W1K", "W2K", "W1V", "W2V"):
            self.t[k] = torch.from_numpy(np.ascontiguousarray(w[k], np.float32)).to(device).to(torch.bfloat16).contiguous()
        for k in ("b1K", "b2K", "b1V", "b2V"):
            self.t[k] = torch.from_numpy(np.ascontiguousarray(w[k], np.float32)).to(device).contiguous()
        self.c = kvE_agg_weights(**{k: self.t[k].data_ptr() for k in self.t})


class LstmWeights:
    """Device copies of the gate weights (bf16 W_ih, W_hh; fp32 biases and score head)."""

    def __init__(self, w: dict, device="cuda"):
        self.t = {}
        for k in ("W_ih", "W_hh"):
            self.t[k] = torch.from_numpy(np.ascontiguousarray(w[k], np.float32)).to(device).to(torch.bfloat16).contiguous()
        for k in ("b_ih", "b_hh", "w_s"):
            self.t[k] = torch.from_numpy(np.ascontiguousarray(w[k], np.float32)).to(device).contiguous()
        self.c = kvE_lstm_weights(**{k: self.t[k].data_ptr() for k in self.t}, b_s=float(w["b_s"]))

    def set_b_s(self, b_s: float):
        self.c.b_s = float(b_s)


class Store:
    """A kvE_store handle plus the device buffers it borrows (allocated here with torch).

    page_perm: None -> page id = flat (layer, s, chunk) index; "random" -> a seeded permutation of the
    page ids (exercises the page-table indirection); or an explicit int32 array [n_layers, S, max_chunks].
    """

    def __init__(self, B, H, C_, W, max_tokens, d_g, agg="mean", d_sum=0, attend="summary", n_layers=1,
                 page_perm=None, device="cuda", seed=0, Hq=None, max_query_tokens=0):
        """H = KV heads (S = B * H sequences); Hq = query heads (default H); max_query_tokens > 0 enables
        decode_attn_block."""
        if not torch.cuda.is_available():
            raise RuntimeError("libkve needs a CUDA device; there is no CPU path")
        self.lib = load_library()
        self.device = torch.device(device)
        self.Hq = H if Hq is None else Hq
        self.cfg = kvE_config(B=B, Hq=self.Hq, Hkv=H, d=128, C=C_, W=W, max_tokens=max_tokens, n_layers=n_layers,
                              agg=AGG[agg], d_sum=d_sum, d_g=d_g, attend=ATTEND[attend],
                              max_query_tokens=max_query_tokens)
        self.B, self.H, self.S, self.C, self.W, self.d_g = B, H, B * H, C_, W, d_g
        self.n_layers, self.max_tokens = n_layers, max_tokens
        self.max_chunks = -(-max_tokens // C_)
        S, mc, L, dev = self.S, self.max_chunks, n_layers, self.device
        n_pages = L * S * mc
        ws_bytes = int(self.lib.kvE_workspace_bytes(C.byref(self.cfg)))
        if ws_bytes == 0:
            raise KveError("kvE_workspace_bytes", -2, "unsupported geometry")
        z = lambda shape, dt: torch.zeros(shape, dtype=dt, device=dev)
        self.k_pages = z((n_pages, C_, 128), torch.bfloat16)
        self.v_pages = z((n_pages, C_, 128), torch.bfloat16)
        if page_perm is None:
            pt = np.arange(n_pages, dtype=np.int32)
        elif isinstance(page_perm, str) and page_perm == "random":
            pt = np.random.default_rng(seed).permutation(n_pages).astype(np.int32)
        else:
            pt = np.asarray(page_perm, np.int32)
        self.page_table = torch.from_numpy(pt.reshape(L, S, mc).copy()).to(dev)
        self.seq_len = z((L, B), torch.int32)
        self.ksum_f32 = z((L, S, mc, 128), torch.float32)
        self.vsum_f32 = z((L, S, mc, 128), torch.float32)
        self.ksum_bf16 = z((L, S, mc, 128), torch.bfloat16)
        self.vsum_bf16 = z((L, S, mc, 128), torch.bfloat16)
        self.scores = z((L, S, mc), torch.float32)
        self.keep_idx = torch.full((L, S, mc), -1, dtype=torch.int32, device=dev)
        self.keep_cnt = z((L, S), torch.int32)
        self.lstm_h = z((L, S, d_g), torch.float32)
        self.lstm_c = z((L, S, d_g), torch.float32)
        self.workspace = z((ws_bytes + 256,), torch.uint8)
        ws_ptr = (self.workspace.data_ptr() + 255) // 256 * 256
        self.status_word = z((1,), torch.int32)
        self.buf = kvE_buffers(
            k_pages=self.k_pages.data_ptr(), v_pages=self.v_pages.data_ptr(), n_pages=n_pages,
            page_table=self.page_table.data_ptr(), seq_len=self.seq_len.data_ptr(),
            ksum_f32=self.ksum_f32.data_ptr(), vsum_f32=self.vsum_f32.data_ptr(),
            ksum_bf16=self.ksum_bf16.data_ptr(), vsum_bf16=self.vsum_bf16.data_ptr(),
            scores=self.scores.data_ptr(), keep_idx=self.keep_idx.data_ptr(), keep_cnt=self.keep_cnt.data_ptr(),
            lstm_h=self.lstm_h.data_ptr(), lstm_c=self.lstm_c.data_ptr(),
            workspace=ws_ptr, workspace_bytes=ws_bytes, status_word=self.status_word.data_ptr())
        torch.cuda.synchronize()
        self.handle = C.c_void_p()
        _check("kvE_create", self.lib.kvE_create(C.byref(self.cfg), C.byref(self.buf), C.byref(self.handle)))

    def close(self):
        if getattr(self, "handle", None):
            self.lib.kvE_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the C entry points, same names without the prefix ----
    def append(self, layer, k_new, v_new, stream=None) -> int:
        return kvE_append(self, layer, k_new, v_new, stream)

    def set_len(self, layer, n, stream=None):
        kvE_set_len(self, layer, n, stream)

    def set_attend(self, attend: str):
        """"summary" | "raw": what a kept chunk contributes to attention from now on"""
        _check("kvE_set_attend", self.lib.kvE_set_attend(self.handle, ATTEND[attend]))

    def set_gate_planes(self, planes: int):
        """2 (default) or 3 (exact products) bf16 planes of the LSTM state in the recurrent product"""
        _check("kvE_set_gate_planes", self.lib.kvE_set_gate_planes(self.handle, int(planes)))

    def summarize_chunks(self, layer, chunk_begin, chunk_end, agg_weights=None, stream=None):
        kvE_summarize_chunks(self, layer, chunk_begin, chunk_end, agg_weights, stream)

    def gate(self, layer, chunk_begin, chunk_end, lstm_weights, stream=None):
        kvE_gate(self, layer, chunk_begin, chunk_end, lstm_weights, stream)

    def gate_next(self, layer, lstm_weights, tau, stream=None):
        kvE_gate_next(self, layer, lstm_weights, tau, stream)

    def refresh_next(self, layer, agg_weights, lstm_weights, tau, stream=None):
        """the trigger with its position taken from the device at execution time (replayable from a CUDA graph)"""
        aw = C.byref(agg_weights.c) if agg_weights is not None else None
        _check("kvE_refresh_next", self.lib.kvE_refresh_next(self.handle, layer, aw, C.byref(lstm_weights.c), C.c_float(tau),
                                                             _stream(stream)), self.handle)

    def adopt_device_state(self, layer, stream=None):
        _check("kvE_adopt_device_state", self.lib.kvE_adopt_device_state(self.handle, layer, _stream(stream)), self.handle)

    def compact(self, layer, tau, stream=None):
        kvE_compact(self, layer, tau, stream)

    def refresh(self, layer, agg_weights, lstm_weights, tau, stream=None):
        """summaries of all stale chunks, gate from scratch, keep list, in one call"""
        aw = C.byref(agg_weights.c) if agg_weights is not None else None
        _check("kvE_refresh", self.lib.kvE_refresh(self.handle, layer, aw, C.byref(lstm_weights.c), C.c_float(tau), _stream(stream)),
               self.handle)

    def compact_topk(self, layer, k, stream=None):
        kvE_compact_topk(self, layer, k, stream)

    def decode_attn(self, layer, q, out=None, lse=None, scale=None, stream=None):
        return kvE_decode_attn(self, layer, q, out, lse, scale, stream)

    def decode_step(self, layer, k_new, v_new, q, out=None, lse=None, scale=None, n_reserve=0, stream=None):
        """append one token per sequence (k_new, v_new: bf16 [S, 128]) at the device-held length and attend, one launch"""
        for t in (k_new, v_new, q):
            assert t.dtype == torch.bfloat16 and tuple(t.shape) == (self.S, 128)
        if out is None:
            out = torch.empty_like(q)
        scale = 1.0 / np.sqrt(128.0) if scale is None else scale
        _check("kvE_decode_step", self.lib.kvE_decode_step(self.handle, layer, _p(k_new), _p(v_new), _p(q), _p(out), _p(lse),
                                                           C.c_float(scale), int(n_reserve), _stream(stream)), self.handle)
        return out

    def decode_attn_dense(self, layer, q, out=None, lse=None, scale=None, stream=None):
        return kvE_decode_attn_dense(self, layer, q, out, lse, scale, stream)

    def append_next(self, layer, k_new, v_new, n_reserve=0, stream=None):
        """k_new, v_new: bf16 [S, n_new, 128] (or [S, 128] for one token); appended at the device-held length
        (graph-replayable); n_reserve: further tokens replays may add."""
        assert k_new.dtype == torch.bfloat16 and k_new.shape == v_new.shape and k_new.shape[0] == self.S
        n_new = k_new.numel() // (self.S * 128)
        assert n_new * self.S * 128 == k_new.numel()
        _check("kvE_append_next", self.lib.kvE_append_next(self.handle, layer, _p(k_new), _p(v_new), n_new, int(n_reserve),
                                                           _stream(stream)), self.handle)

    def decode_attn_block(self, layer, q, dense=False, out=None, lse=None, scale=None, stream=None, causal=False):
        return kvE_decode_attn_block(self, layer, q, dense, out, lse, scale, stream, causal)

    def reclaim_pages(self, layer, chunk_begin, chunk_end, mode="discarded", free_list=None, free_count=None, stream=None):
        return kvE_reclaim_pages(self, layer, chunk_begin, chunk_end, mode, free_list, free_count, stream)

    def decode_attn_static(self, layer, q, out=None, lse=None, scale=None, stream=None):
        return kvE_decode_attn_static(self, layer, q, out, lse, scale, stream)

    def decode_step_host(self, layer, k_new, v_new, q, out, agg_weights, lstm_weights, tau, scale=None,
                         from_scratch=False, stream=None, wait=True):
        kvE_decode_step_host(self, layer, k_new, v_new, q, out, agg_weights, lstm_weights, tau, scale, from_scratch, stream, wait)

    def poll_status(self) -> int:
        return kvE_poll_status(self)

    def selftest_timeout(self, which: int, stream=None):
        """launches the kernel whose bounded wait runs out (which: 0 = CTA-scope wait, 1 = cluster-scope wait)"""
        _check("kvE_selftest_timeout", self.lib.kvE_selftest_timeout(self.handle, int(which), _stream(stream)), self.handle)

    def layer_state(self, layer=0) -> dict:
        return kvE_layer_state(self, layer)

    def profile(self, enable: bool):
        kvE_profile(self, enable)

    def profile_read(self) -> dict:
        return kvE_profile_read(self)


def kvE_append(st: Store, layer, k_new, v_new, stream=None) -> int:
    """k_new, v_new: bf16 [S, n_new, 128] device tensors.  Returns the number of chunks ready to gate."""
    assert k_new.dtype == torch.bfloat16 and k_new.shape == v_new.shape and k_new.shape[0] == st.S and k_new.shape[2] == 128
    ready = C.c_int(0)
    _check("kvE_append", st.lib.kvE_append(st.handle, layer, _p(k_new), _p(v_new), int(k_new.shape[1]),
                                           C.byref(ready), _stream(stream)), st.handle)
    return ready.value


def kvE_set_len(st: Store, layer, n, stream=None):
    _check("kvE_set_len", st.lib.kvE_set_len(st.handle, layer, int(n), _stream(stream)), st.handle)


def kvE_summarize_chunks(st: Store, layer, chunk_begin, chunk_end, agg_weights=None, stream=None):
    w = C.byref(agg_weights.c) if agg_weights is not None else None
    _check("kvE_summarize_chunks", st.lib.kvE_summarize_chunks(st.handle, layer, int(chunk_begin), int(chunk_end), w,
                                                               _stream(stream)), st.handle)


def kvE_gate(st: Store, layer, chunk_begin, chunk_end, lstm_weights, stream=None):
    _check("kvE_gate", st.lib.kvE_gate(st.handle, layer, int(chunk_begin), int(chunk_end), C.byref(lstm_weights.c),
                                       _stream(stream)), st.handle)


def kvE_gate_next(st: Store, layer, lstm_weights, tau, stream=None):
    _check("kvE_gate_next", st.lib.kvE_gate_next(st.handle, layer, C.byref(lstm_weights.c), C.c_float(tau), _stream(stream)),
           st.handle)


def kvE_compact(st: Store, layer, tau, stream=None):
    _check("kvE_compact", st.lib.kvE_compact(st.handle, layer, C.c_float(tau), _stream(stream)), st.handle)


def kvE_compact_topk(st: Store, layer, k, stream=None):
    _check("kvE_compact_topk", st.lib.kvE_compact_topk(st.handle, layer, int(k), _stream(stream)), st.handle)


def _attn(fn_name, st, layer, q, out, lse, scale, stream):
    assert q.dtype == torch.bfloat16 and tuple(q.shape) == (st.S, 128)
    if out is None:
        out = torch.empty_like(q)
    scale = 1.0 / np.sqrt(128.0) if scale is None else scale
    _check(fn_name, getattr(st.lib, fn_name)(st.handle, layer, _p(q), _p(out), _p(lse), C.c_float(scale),
                                              _stream(stream)), st.handle)
    return out


def kvE_decode_attn(st: Store, layer, q, out=None, lse=None, scale=None, stream=None):
    return _attn("kvE_decode_attn", st, layer, q, out, lse, scale, stream)


def kvE_decode_attn_dense(st: Store, layer, q, out=None, lse=None, scale=None, stream=None):
    return _attn("kvE_decode_attn_dense", st, layer, q, out, lse, scale, stream)


def kvE_decode_attn_block(st: Store, layer, q, dense=False, out=None, lse=None, scale=None, stream=None, causal=False):
    """q: bf16 [B, T, Hq, 128] device tensor (T query tokens on all query heads).  Returns out (same shape);
    lse, if given, is an fp32 [B, T, Hq] device tensor."""
    assert q.dtype == torch.bfloat16 and q.dim() == 4 and q.shape[0] == st.B and q.shape[2] == st.Hq and q.shape[3] == 128
    if out is None:
        out = torch.empty_like(q)
    assert out.shape == q.shape and out.dtype == torch.bfloat16
    if lse is not None:
        assert lse.dtype == torch.float32 and tuple(lse.shape) == tuple(q.shape[:3])
    scale = (1.0 / 128.0 ** 0.5) if scale is None else scale
    _check("kvE_decode_attn_block", st.lib.kvE_decode_attn_block(st.handle, layer, _p(q), int(q.shape[1]), int(bool(dense)),
                                                                 int(bool(causal)), _p(out), _p(lse), C.c_float(scale), _stream(stream)), st.handle)
    return out


RECLAIM = {"discarded": 0, "gated": 1}


def kvE_reclaim_pages(st: Store, layer, chunk_begin, chunk_end, mode="discarded", free_list=None, free_count=None, stream=None):
    """Hands pages of gated chunks back (Sec. 3.3).  free_list: int32 device tensor (its length is the
    capacity; allocated here for the whole range if omitted), free_count: int32 device tensor [1].
    Returns (free_list, free_count); the first free_count entries are valid once the stream has run."""
    if free_list is None:
        free_list = torch.empty((max(1, st.S * max(chunk_end - chunk_begin, 0)),), dtype=torch.int32, device=st.device)
    if free_count is None:
        free_count = torch.zeros((1,), dtype=torch.int32, device=st.device)
    assert free_list.dtype == torch.int32 and free_count.dtype == torch.int32
    _check("kvE_reclaim_pages", st.lib.kvE_reclaim_pages(st.handle, layer, int(chunk_begin), int(chunk_end), RECLAIM[mode],
                                                        _p(free_list), C.c_int64(free_list.numel()), _p(free_count),
                                                        _stream(stream)), st.handle)
    return free_list, free_count


def kvE_decode_attn_static(st: Store, layer, q, out=None, lse=None, scale=None, stream=None):
    """kvE_decode_attn with the split-K scratch inside the library image (no caller scratch, no
    allocation inside the call).  `out` is allocated here with torch only when the caller passes none;
    a caller that must not allocate passes its own."""
    return _attn("kvE_decode_attn_static", st, layer, q, out, lse, scale, stream)


def kvE_decode_step_host(st: Store, layer, k_new, v_new, q, out, agg_weights, lstm_weights, tau, scale=None,
                         from_scratch=False, stream=None, wait=True):
    """k_new, v_new, q, out: HOST bf16 [S, 128] tensors (pinned for asynchronous copies).
    wait=False calls kvE_decode_step_host_async: the step is only enqueued (pinned buffers required)."""
    for t in (k_new, v_new, q, out):
        assert not t.is_cuda and t.dtype == torch.bfloat16 and tuple(t.shape) == (st.S, 128) and t.is_contiguous()
    scale = 1.0 / np.sqrt(128.0) if scale is None else scale
    aw = C.byref(agg_weights.c) if agg_weights is not None else None
    if not wait:
        assert all(t.is_pinned() for t in (k_new, v_new, q, out))
    fn = st.lib.kvE_decode_step_host if wait else st.lib.kvE_decode_step_host_async
    _check("kvE_decode_step_host",
           fn(st.handle, layer, C.c_void_p(k_new.data_ptr()), C.c_void_p(v_new.data_ptr()),
                                       C.c_void_p(q.data_ptr()), C.c_void_p(out.data_ptr()), aw,
                                       C.byref(lstm_weights.c), C.c_float(tau), C.c_float(scale),
                                       1 if from_scratch else 0, _stream(stream)), st.handle)


def kvE_poll_status(st: Store) -> int:
    word = C.c_int(0)
    _check("kvE_poll_status", st.lib.kvE_poll_status(st.handle, C.byref(word)), st.handle)
    return word.value


def kvE_layer_state(st: Store, layer=0) -> dict:
    v = [C.c_int(0) for _ in range(4)]
    _check("kvE_layer_state", st.lib.kvE_layer_state(st.handle, layer, *[C.byref(x) for x in v]))
    return dict(zip(("n_tokens", "n_summarised", "n_gated", "n_compacted"), (x.value for x in v)))


def kvE_profile(st: Store, enable: bool):
    _check("kvE_profile", st.lib.kvE_profile(st.handle, 1 if enable else 0), st.handle)


def kvE_profile_read(st: Store) -> dict:
    """microseconds of the most recent launch of each kernel (None if it has not run)"""
    us = (C.c_float * len(KERNEL_IDS))()
    _check("kvE_profile_read", st.lib.kvE_profile_read(st.handle, us), st.handle)
    return {k: (float(us[i]) if us[i] >= 0 else None) for i, k in enumerate(KERNEL_IDS)}
