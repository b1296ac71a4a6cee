"""The benchmark's algorithmic byte and FLOP counts, pinned to figures worked out by hand from the
geometry of the Llama-2-7B-shaped configuration (256 sequences, 56 stale chunks of 64 tokens,
4096 tokens, d = 128, d_g = 256, d_sum = 256).  A bf16 row is 256 bytes."""
import bench
from paper_2509_21354_b200 import workloads as wlm


def test_algorithmic_bytes_of_cfg2():
    wl = wlm.CFG2
    Nc, R = wl.n_stale_chunks(), wl.n - wl.n_stale_chunks() * wl.C
    assert (wl.S, Nc, R) == (256, 56, 512)
    by = bench.algorithmic_bytes(wl, Nc, keep_mean=28.0, R=R)
    units = 256 * 56
    assert by["chunk_mean"] == units * (2 * 64 * 256 + 2 * 128 * 4) == 484_442_112      # every stale K and V row once
    assert by["attn_dense"] == 256 * (2 * 4096 * 256 + 512) == 537_001_984
    assert by["attn_gated"] == 256 * (2 * (512 + 28) * 256 + 512)                          # window + one row per kept chunk
    raw = bench.algorithmic_bytes(wl, Nc, keep_mean=28.0, R=R, attend="raw")
    assert raw["attn_gated"] == 256 * (2 * (512 + 28 * 64) * 256 + 512)                    # kept chunks at full resolution
    assert by["gate_proj"] == units * (2 * 256 + 1024 * 4)
    assert by["compact"] == 256 * (56 * 8 + 4)


def test_algorithmic_flops_of_cfg2():
    wl = wlm.CFG2
    fl = bench.algorithmic_flops(wl, 56)
    units = 256 * 56
    assert fl["gate_proj"] == units * 2 * 256 * 1024 == 7_516_192_768
    assert fl["chunk_mlp"] == 2 * units * 2 * (128 * 256 + 256 * 128) == 3_758_096_384
    assert fl["gate_rnn"] == units * (2 * 256 * 1024 + 512)
    assert "chunk_mlp" not in bench.algorithmic_flops(wlm.CFG1, 28)                        # mean aggregator: no MLP
