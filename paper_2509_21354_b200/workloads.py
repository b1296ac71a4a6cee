"""Seeded synthetic inputs for the gated chunked KV cache (shared by the tests, the benchmark and
the oracle-side checks).  This module holds NO arithmetic of the method: it only draws numbers,
rounds them to bf16 and names the workload geometries.

The workloads stand in for the LLaMA-2-7B-backed VLA decoding traffic the paper measures
(Sec. 4.1-4.2: 32 heads x 128, bf16 KV, long image-token histories): same shapes, N(0,1)
keys/values, optional per-chunk key offsets so chunk utility varies.

Layout produced here is the plain one: K, V [S, n, d] and q [S, d] as bf16 bit patterns
(numpy uint16), S = B * H with s = b * H + h.
"""
from dataclasses import dataclass, replace

import numpy as np

D_HEAD = 128
BIAS_STD = 0.1


# ---- bf16 bit helpers (input quantisation only) ----------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit pattern, round to nearest even (finite inputs)."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """float32 array whose every value is exactly representable in bf16."""
    return bf16_bits_to_f32(f32_to_bf16_bits(x))


# ---- workload geometry -----------------------------------------------------------------------
@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    n: int                 # tokens in the cache when the step starts
    C: int                 # chunk size
    W: int                 # recent window kept raw
    d_g: int               # LSTM hidden size
    agg: str = "mean"      # "mean" | "mlp" | "identity" | "max" | "token_mlp"
    d_sum: int = 0         # MLP hidden size (agg == "mlp")
    n_layers: int = 1
    tau: float = 0.5
    key_offset_std: float = 0.0   # per-(sequence, chunk) offset vector added to all keys of the chunk
    n_append: int = 0      # tokens appended autoregressively after the gate (one decode each)
    d: int = D_HEAD
    seed: int = 0

    @property
    def S(self) -> int:
        return self.B * self.H

    def n_stale_chunks(self, n=None) -> int:
        n = self.n if n is None else n
        return max(0, (n - self.W) // self.C)

    @property
    def max_tokens(self) -> int:
        return self.n + self.n_append

    @property
    def max_chunks(self) -> int:
        return -(-self.max_tokens // self.C)

    def small(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five configurations the benchmark definition names (single layer shown where the
# definition has 32 identical, independent layers: each layer is its own seeded instance).
CFG1 = Workload("cfg1_b1_h8_n2048", B=1, H=8, n=2048, C=64, W=256, d_g=128, agg="mean")
CFG2 = Workload("cfg2_llama7b_layer_b8_h32_n4096", B=8, H=32, n=4096, C=64, W=512, d_g=256,
                agg="mlp", d_sum=256, key_offset_std=0.5)
CFG3 = Workload("cfg3_vla_history_b4_h32_n4160", B=4, H=32, n=64 + 16 * 256, C=64, W=256, d_g=256,
                agg="mlp", d_sum=256, key_offset_std=0.5, n_layers=32, n_append=7)
CFG4 = Workload("cfg4_long_horizon_b16_h32_n16512", B=16, H=32, n=128 + 64 * 256, C=128, W=1024,
                d_g=256, agg="mlp", d_sum=256, key_offset_std=0.5, n_layers=32)
CONFIGS = {"cfg1": CFG1, "cfg2": CFG2, "cfg3": CFG3, "cfg4": CFG4}


def sweep_points():
    """cfg5: the stress sweep grid (batch x context x chunk x keep ratio), 32 heads, W = 512."""
    for B in (1, 2, 4, 8, 16, 32, 64):
        for n in (2048, 4096, 8192, 16384, 32768):
            for Cs in (32, 64, 128, 256):
                for keep in (0.25, 0.5, 0.75, 1.0):
                    yield Workload(f"sweep_b{B}_n{n}_c{Cs}", B=B, H=32, n=n, C=Cs, W=512, d_g=256,
                                   agg="mean", key_offset_std=0.5), keep


# ---- generators ------------------------------------------------------------------------------
def _rng(*key) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=np.random.SeedSequence([int(k) & 0xFFFFFFFF for k in key]).generate_state(2, np.uint64)))


_TAG_KV, _TAG_CHUNK, _TAG_Q, _TAG_MLP, _TAG_LSTM, _TAG_NEW = 1, 2, 3, 4, 5, 6


def gen_kv_seq(wl: Workload, layer: int, s: int, n=None):
    """K, V [n, d] bf16 bits of sequence s alone (its own sub-seeded stream, so any subset of the
    sequences can be drawn without the others).  K rows get a per-chunk offset when the workload asks."""
    n = wl.n if n is None else n
    rng = _rng(wl.seed, _TAG_KV, layer, s)
    k = rng.standard_normal((n, wl.d), dtype=np.float32)
    v = rng.standard_normal((n, wl.d), dtype=np.float32)
    if wl.key_offset_std > 0:
        n_chunks = -(-n // wl.C)
        off = rng.standard_normal((n_chunks, wl.d), dtype=np.float32) * np.float32(wl.key_offset_std)
        k += np.repeat(off, wl.C, axis=0)[:n]
    return f32_to_bf16_bits(k), f32_to_bf16_bits(v)


def gen_kv(wl: Workload, layer: int = 0, n=None, seqs=None):
    """K, V [len(seqs), n, d] bf16 bits (all S sequences by default)."""
    n = wl.n if n is None else n
    seqs = range(wl.S) if seqs is None else seqs
    K = np.empty((len(seqs), n, wl.d), np.uint16)
    V = np.empty((len(seqs), n, wl.d), np.uint16)
    for i, s in enumerate(seqs):
        K[i], V[i] = gen_kv_seq(wl, layer, int(s), n)
    return K, V


def gen_chunk(wl: Workload, layer: int, s: int, t: int, attempt: int):
    """Replacement draw for chunk t of sequence s (attempt >= 1): K, V [C, d] bf16 bits."""
    rng = _rng(wl.seed, _TAG_CHUNK, layer, s, t, attempt)
    k = rng.standard_normal((wl.C, wl.d), dtype=np.float32)
    v = rng.standard_normal((wl.C, wl.d), dtype=np.float32)
    if wl.key_offset_std > 0:
        k += rng.standard_normal((1, wl.d), dtype=np.float32) * np.float32(wl.key_offset_std)
    return f32_to_bf16_bits(k), f32_to_bf16_bits(v)


def apply_redraws(wl: Workload, layer: int, K, V, redraws) -> None:
    """redraws: iterable of (s, t, attempt); overwrites those chunks in place."""
    for s, t, attempt in redraws:
        k, v = gen_chunk(wl, layer, int(s), int(t), int(attempt))
        K[s, t * wl.C:(t + 1) * wl.C] = k
        V[s, t * wl.C:(t + 1) * wl.C] = v


def gen_q(wl: Workload, layer: int = 0, step: int = 0) -> np.ndarray:
    return f32_to_bf16_bits(_rng(wl.seed, _TAG_Q, layer, step).standard_normal((wl.S, wl.d), dtype=np.float32))


def gen_q_block(wl: Workload, T: int, Hq: int, layer: int = 0, step: int = 0) -> np.ndarray:
    """queries of T tokens on Hq query heads, [B, T, Hq, d] bf16 bits (wl.H counts the KV heads)"""
    return f32_to_bf16_bits(_rng(wl.seed, _TAG_Q, layer, 7919 + step).standard_normal((wl.B, T, Hq, wl.d), dtype=np.float32))


def gen_new_tokens(wl: Workload, layer: int = 0, step: int = 0, n_new: int = 1):
    """k_new, v_new [S, n_new, d] bf16 bits for an autoregressive append."""
    rng = _rng(wl.seed, _TAG_NEW, layer, step)
    k = rng.standard_normal((wl.S, n_new, wl.d), dtype=np.float32)
    v = rng.standard_normal((wl.S, n_new, wl.d), dtype=np.float32)
    return f32_to_bf16_bits(k), f32_to_bf16_bits(v)


def gen_mlp_weights(wl: Workload, layer: int = 0):
    """Aggregator weights, N(0, 1/fan_in) entries rounded to bf16-representable float32; small N(0, BIAS_STD^2) biases
    so that a dropped bias term shows up in parity."""
    if wl.agg not in ("mlp", "token_mlp"):
        return None
    rng = _rng(wl.seed, _TAG_MLP, layer)
    d, ds = wl.d, wl.d_sum
    w = {}
    for side in ("K", "V"):
        w["W1" + side] = round_to_bf16(rng.standard_normal((ds, d), dtype=np.float32) / np.float32(np.sqrt(d)))
        w["b1" + side] = rng.standard_normal((ds,), dtype=np.float32) * np.float32(BIAS_STD)
        w["W2" + side] = round_to_bf16(rng.standard_normal((d, ds), dtype=np.float32) / np.float32(np.sqrt(ds)))
        w["b2" + side] = rng.standard_normal((d,), dtype=np.float32) * np.float32(BIAS_STD)
    return w


HEAD_GAIN = 4.0


def gen_lstm_weights(wl: Workload, layer: int = 0, b_s: float = 0.0):
    """Gate weights, N(0, 1/fan_in) entries; W_ih and W_hh rounded to bf16-representable float32.
    The score head w_s is drawn the same way and scaled by HEAD_GAIN so that scores spread over a
    useful part of [0, 1] instead of huddling at sigmoid(b_s)."""
    rng = _rng(wl.seed, _TAG_LSTM, layer)
    d_in, dg = 2 * wl.d, wl.d_g
    return dict(
        W_ih=round_to_bf16(rng.standard_normal((4 * dg, d_in), dtype=np.float32) / np.float32(np.sqrt(d_in))),
        W_hh=round_to_bf16(rng.standard_normal((4 * dg, dg), dtype=np.float32) / np.float32(np.sqrt(dg))),
        b_ih=rng.standard_normal((4 * dg,), dtype=np.float32) * np.float32(BIAS_STD),
        b_hh=rng.standard_normal((4 * dg,), dtype=np.float32) * np.float32(BIAS_STD),
        w_s=(rng.standard_normal((dg,), dtype=np.float32) * np.float32(HEAD_GAIN / np.sqrt(dg))).astype(np.float32),
        b_s=float(b_s),
    )
