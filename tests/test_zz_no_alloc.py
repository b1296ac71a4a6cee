"""kvE_decode_attn_static: gated attention for callers that may not allocate device memory while
they run (a control loop whose framework owns the whole GPU pool, a plug-in working on somebody
else's device).  Its split-K scratch is an array inside the library image, so the test drives it
through the C ABI next to kvE_decode_attn, which takes its scratch from the caller's workspace, and
asks for the same answer on two calls in a row -- the second call finds the array as the first
one left it.  Collected last on purpose: a failure here cannot hide another test's result.
"""
import numpy as np
import pytest
import torch

from paper_2509_21354_b200 import workloads as wlm
from tests import harness as hz

pytestmark = pytest.mark.gpu


def _prepared_store(wl, attend):
    from paper_2509_21354_b200 import binding as b
    pb = hz.Problem(wl)
    st = b.Store(B=wl.B, H=wl.H, C_=wl.C, W=wl.W, max_tokens=wl.max_tokens, d_g=wl.d_g, agg=wl.agg,
                 d_sum=wl.d_sum, attend=attend, page_perm="random", seed=11)
    st.append(0, b.bits_to_bf16(pb.K), b.bits_to_bf16(pb.V))
    st.summarize_chunks(0, 0, pb.Nc, b.AggWeights(pb.mlp) if pb.mlp is not None else None)
    st.gate(0, 0, pb.Nc, b.LstmWeights(pb.lstm))
    st.compact(0, pb.tau)
    torch.cuda.synchronize()
    assert st.poll_status() == 0
    return b, pb, st


@pytest.mark.parametrize("attend,n", [("summary", 4096), ("raw", 3000)])
def test_static_scratch_attention_matches_workspace_attention_twice(attend, n):
    # several splits per sequence (so partial records and tickets are really used) and a ragged tail
    wl = wlm.CFG1.small(B=2, H=8, n=n, seed=5)
    b, pb, st = _prepared_store(wl, attend)
    for call in range(2):
        q = b.bits_to_bf16(wlm.gen_q(wl, 0, 40 + call))
        lse_ws = torch.zeros(st.S, dtype=torch.float32, device="cuda")
        lse_static = torch.zeros_like(lse_ws)
        out_static = torch.full((st.S, 128), float("nan"), dtype=torch.bfloat16, device="cuda")   # caller-provided output
        want = st.decode_attn(0, q, lse=lse_ws)
        st.decode_attn_static(0, q, out=out_static, lse=lse_static)
        torch.cuda.synchronize()
        assert st.poll_status() == 0
        got_bits, want_bits = b.bf16_to_bits(out_static), b.bf16_to_bits(want)
        hz.check_output(got_bits, wlm.bf16_bits_to_f32(want_bits), f"static vs workspace, call {call}")
        assert hz.bf16_ulp_distance(got_bits, want_bits).max() <= 1
        assert np.abs(lse_static.cpu().numpy() - lse_ws.cpu().numpy()).max() <= 1e-3
        # and against the oracle, like every other attention test
        ref, _, _, _ = pb.oracle_attn(wlm.gen_q(wl, 0, 40 + call), attend)
        hz.check_output(got_bits, ref, f"static vs oracle, call {call}")


def test_static_scratch_attention_rejects_sizes_beyond_its_array():
    from paper_2509_21354_b200 import binding as b
    # 2080 sequences: more tickets than the built-in array holds -> refused on the host, nothing launched
    st = b.Store(B=65, H=32, C_=64, W=64, max_tokens=128, d_g=64, agg="mean", attend="summary")
    kv = torch.zeros((st.S, 128, 128), dtype=torch.bfloat16, device="cuda")
    st.append(0, kv, kv)
    q = torch.zeros((st.S, 128), dtype=torch.bfloat16, device="cuda")
    st.decode_attn(0, q)                                  # the workspace path takes this size
    with pytest.raises(b.KveError) as err:
        st.decode_attn_static(0, q)
    assert err.value.rc == -3                             # KVE_ERR_CAPACITY
    assert "built-in scratch" in st.lib.kvE_last_cuda_error(st.handle).decode()
    torch.cuda.synchronize()
    assert st.poll_status() == 0
