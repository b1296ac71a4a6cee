"""No-GPU checks of the product side: the C-ABI library builds, loads and exports every entry point
the header declares; host-side argument checks that need no device; the input generators."""
import ctypes as C
import os
import re

import numpy as np

from paper_2509_21354_b200 import binding, workloads as wlm

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_entry_points():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in os.listdir(inc):
        if f.endswith(".h"):
            text = re.sub(r"/\*.*?\*/", "", open(os.path.join(inc, f)).read(), flags=re.S)
            names |= set(re.findall(r"\b(kvE_[A-Za-z0-9_]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol():
    lib = binding.load_library()
    names = declared_entry_points()
    assert {"kvE_append", "kvE_summarize_chunks", "kvE_gate", "kvE_compact", "kvE_decode_attn"} <= names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/ but not exported"
    assert set(binding.EXPORTS) <= names


def test_struct_layouts_match_header():
    assert C.sizeof(binding.kvE_config) == 13 * 4
    assert C.sizeof(binding.kvE_buffers) == 17 * 8
    assert C.sizeof(binding.kvE_agg_weights) == 8 * 8
    assert C.sizeof(binding.kvE_lstm_weights) == 5 * 8 + 8


def test_workspace_bytes_and_geometry_checks_need_no_device():
    lib = binding.load_library()
    cfg = binding.kvE_config(B=8, Hq=32, Hkv=32, d=128, C=64, W=512, max_tokens=4096, n_layers=1, agg=1, d_sum=256,
                             d_g=256, attend=0)
    ws = lib.kvE_workspace_bytes(C.byref(cfg))
    assert ws >= 256 * 64 * 1024 * 4          # at least the gate projection buffer [S * max_chunks][4 d_g] fp32
    for field, bad in (("d", 64), ("d_g", 100), ("Hq", 16), ("C", 4096), ("d_sum", 12)):
        c2 = binding.kvE_config.from_buffer_copy(cfg)
        setattr(c2, field, bad)
        assert lib.kvE_workspace_bytes(C.byref(c2)) == 0
    # grouped query heads: Hq a multiple of Hkv; a query block holds at most 128 rows per KV head and
    # enlarges the workspace by its split records
    gq = binding.kvE_config.from_buffer_copy(cfg)
    gq.Hkv, gq.max_query_tokens = 8, 7
    assert lib.kvE_workspace_bytes(C.byref(gq)) > 0
    gq.max_query_tokens = 33                                               # 33 tokens x 4 heads per KV head = 132 rows
    assert lib.kvE_workspace_bytes(C.byref(gq)) == 0
    gq.max_query_tokens, gq.C = 7, 12                                      # no box of 8 rows divides a 12-token chunk
    assert lib.kvE_workspace_bytes(C.byref(gq)) == 0
    with_block = binding.kvE_config.from_buffer_copy(cfg)
    with_block.max_query_tokens = 4
    assert lib.kvE_workspace_bytes(C.byref(with_block)) > ws
    out = C.c_void_p()
    assert lib.kvE_create(C.byref(cfg), None, C.byref(out)) == -1          # null buffers
    assert lib.kvE_append(None, 0, None, None, 1, None, None) == -1        # null handle
    assert lib.kvE_poll_status(None, None) == -1
    assert lib.kvE_append_next(None, 0, None, None, 1, 0, None) == -1
    assert lib.kvE_decode_attn_block(None, 0, None, 1, 0, 0, None, None, 0.1, None) == -1


def test_store_refuses_to_run_without_cuda():
    import pytest
    import torch
    if torch.cuda.is_available():
        pytest.skip("CUDA present")
    with pytest.raises(RuntimeError):
        binding.Store(B=1, H=1, C_=64, W=0, max_tokens=128, d_g=128)


def test_generators_are_seeded_and_bf16_exact():
    wl = wlm.CFG1.small(n=256)
    K1, V1 = wlm.gen_kv(wl)
    K2, V2 = wlm.gen_kv(wl, seqs=[3, 5])
    assert np.array_equal(K1[[3, 5]], K2) and np.array_equal(V1[[3, 5]], V2)
    assert not np.array_equal(K1[0], K1[1])
    w = wlm.gen_lstm_weights(wl)
    assert np.array_equal(wlm.round_to_bf16(w["W_ih"]), w["W_ih"]) and w["W_hh"].shape == (512, 128)
    m = wlm.gen_mlp_weights(wlm.CFG2)
    assert m["W1K"].shape == (256, 128) and m["W2V"].shape == (128, 256) and np.abs(m["b1K"]).max() > 0
    k, v = wlm.gen_chunk(wl, 0, 1, 2, 1)
    k2, _ = wlm.gen_chunk(wl, 0, 1, 2, 2)
    assert k.shape == (64, 128) and not np.array_equal(k, k2)
    assert [c.n_stale_chunks() for c in (wlm.CFG1, wlm.CFG2, wlm.CFG3, wlm.CFG4)] == [28, 56, 61, 121]
