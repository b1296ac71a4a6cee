"""The paper's FLOPs and memory cost model (Sec. 3.3, Eq. 4-7) as plain arithmetic.

Not on the GPU path: a calculator for printing the paper's own kind of ratio next to measured
numbers.  Symbols follow Sec. 3.3: B batch, n context tokens, H heads, d_k head dim,
d_model = H * d_k, d_ff FFN width, C chunk size, W window, M retained chunks, d_sum aggregator
hidden size, d_g LSTM hidden size.
"""
from dataclasses import dataclass


@dataclass(frozen=True)
class ModelDims:
    d_model: int = 4096      # LLaMA-2-7B, as in Sec. 4.1
    H: int = 32
    d_k: int = 128
    d_ff: int = 11008
    B: int = 1


def flops_base(n: float, m: ModelDims = ModelDims()) -> float:
    """Eq. 4: projections and attention of one layer over n tokens."""
    return 4 * m.B * n * m.d_model ** 2 + 2 * m.B * m.H * n ** 2 * m.d_k


def flops_ffn(n: float, m: ModelDims = ModelDims()) -> float:
    """Eq. 5: the feed-forward block."""
    return 3 * m.B * n * m.d_model * m.d_ff


def n_effective(W: float, M: float) -> float:
    """Sec. 3.3: attention runs over n' = W + M positions."""
    return W + M


def flops_kv_efficient(n: float, W: float, M: float, C: float, d_sum: int, d_g: int, m: ModelDims = ModelDims(),
                       gated_chunks=None) -> float:
    """Eq. 6: the same layer over n' = W + M positions plus the aggregator and LSTM work per gated chunk
    (4 d_sum d_model + 4 d_g d_model + 4 d_g^2 each).  gated_chunks defaults to (n - W) / C, the chunks that
    lie outside the window (the count that reproduces the number printed in Sec. 4.1)."""
    np_ = n_effective(W, M)
    chunks = (n - W) / C if gated_chunks is None else gated_chunks
    return (4 * m.B * np_ * m.d_model ** 2 + 2 * m.B * m.H * np_ ** 2 * m.d_k
            + chunks * m.B * m.H * (4 * d_sum * m.d_model + 4 * d_g * m.d_model + 4 * d_g ** 2))


def speedup(n: float, W: float, M: float, C: float, d_sum: int, d_g: int, m: ModelDims = ModelDims()) -> float:
    """Eq. 7: (base + FFN) / (KV-efficient + FFN)."""
    f = flops_ffn(n, m)
    return (flops_base(n, m) + f) / (flops_kv_efficient(n, W, M, C, d_sum, d_g, m) + f)


def memory_ratio(n: float, W: float, M: float) -> float:
    """Sec. 3.3: KV rows held, n / (W + M)."""
    return n / n_effective(W, M)
