"""GPU parity: every step of the CUDA path, called through the C ABI, against the oracle on the same
seeded inputs.  Index sets bit-exact; floating point within the stated tolerances."""
import numpy as np
import pytest
import torch

from oracle import kvo
from paper_2509_21354_b200 import workloads as wlm
from tests import harness as hz

pytestmark = pytest.mark.gpu


def _binding():
    from paper_2509_21354_b200 import binding
    return binding


def make_store(wl, attend="summary", page_perm="random", n_layers=1, S=None):
    b = _binding()
    return b.Store(B=wl.B, H=wl.H, C_=wl.C, W=wl.W, max_tokens=wl.max_tokens, d_g=wl.d_g, agg=wl.agg,
                   d_sum=wl.d_sum, attend=attend, n_layers=n_layers, page_perm=page_perm, seed=wl.seed + 7)


def load_kv(st, layer, K, V, pieces=(1.0,)):
    """prefill through kvE_append, optionally in several ragged pieces"""
    b = _binding()
    n = K.shape[1]
    cuts = sorted({0, n} | {int(n * f) for f in pieces})
    for a, e in zip(cuts, cuts[1:]):
        st.append(layer, b.bits_to_bf16(K[:, a:e]), b.bits_to_bf16(V[:, a:e]))


def pages_to_plain(st, layer, n):
    """read the paged store back into the plain [S, n, d] layout (host), via the page table"""
    b = _binding()
    pt = st.page_table[layer].cpu().numpy()
    kp, vp = b.bf16_to_bits(st.k_pages), b.bf16_to_bits(st.v_pages)
    nch = -(-n // st.C)
    K = kp[pt[:, :nch]].reshape(st.S, nch * st.C, 128)[:, :n]
    V = vp[pt[:, :nch]].reshape(st.S, nch * st.C, 128)[:, :n]
    return K, V


def run_gpu_pipeline(st, pb, layer=0, agg_w=None, lstm_w=None):
    st.summarize_chunks(layer, 0, pb.Nc, agg_w)
    st.gate(layer, 0, pb.Nc, lstm_w)
    st.compact(layer, pb.tau)
    torch.cuda.synchronize()
    assert st.poll_status() == 0


def check_summaries(st, pb, layer=0):
    b = _binding()
    Nc = pb.Nc
    if Nc == 0:
        return
    kf = st.ksum_f32[layer, :, :Nc].cpu().numpy()
    vf = st.vsum_f32[layer, :, :Nc].cpu().numpy()
    kb = b.bf16_to_bits(st.ksum_bf16[layer, :, :Nc])
    vb = b.bf16_to_bits(st.vsum_bf16[layer, :, :Nc])
    if pb.wl.agg in ("mean", "identity", "max"):
        # same sequential fp32 sum and IEEE division as the f32 oracle: bit for bit
        assert np.array_equal(kf, pb.sm32["ksum"][:, :Nc]) and np.array_equal(vf, pb.sm32["vsum"][:, :Nc])
        assert np.array_equal(kb, pb.sm32["ksum_b16"][:, :Nc]) and np.array_equal(vb, pb.sm32["vsum_b16"][:, :Nc])
    else:
        # MLP: fp32 dot products in another order; erf from another library
        for got, want in ((kf, pb.sm64["ksum"][:, :Nc]), (vf, pb.sm64["vsum"][:, :Nc])):
            assert np.abs(got - want).max() <= 2e-5 * max(1.0, np.abs(want).max())
        for got, want in ((kb, pb.sm32["ksum_b16"][:, :Nc]), (vb, pb.sm32["vsum_b16"][:, :Nc])):
            # a rounding decision flips only next to a tie: at most one bf16 step (2^-7 relative; near
            # zero the fp32 noise itself spans several tiny steps), and rarely
            g, w = wlm.bf16_bits_to_f32(got).astype(np.float64), wlm.bf16_bits_to_f32(want).astype(np.float64)
            assert np.all(np.abs(g - w) <= 2.0 ** -7 * np.abs(w) + 1e-5)
            assert (got != want).mean() < 2e-3
    assert np.abs(kf - pb.sm64["ksum"][:, :Nc]).max() <= 2e-5 * max(1.0, np.abs(pb.sm64["ksum"]).max())


def check_gate_and_keep(st, pb, layer=0):
    Nc = pb.Nc
    if Nc == 0:                                    # nothing has left the window: no scores, empty keep lists
        assert int(st.keep_cnt[layer].abs().sum()) == 0
        return
    sc = st.scores[layer, :, :Nc].cpu().numpy()
    assert np.abs(sc - pb.sc32[:, :Nc]).max() <= 2e-4
    assert np.abs(sc - pb.sc64[:, :Nc]).max() <= 2e-4
    assert np.abs(sc - pb.tau).min() >= 1e-3 if Nc else True     # the margin survived on the GPU side too
    if Nc:
        assert np.abs(st.lstm_h[layer].cpu().numpy() - pb.h64).max() <= 2e-4
        assert np.abs(st.lstm_c[layer].cpu().numpy() - pb.c64).max() <= 4e-4
    idx, cnt = st.keep_idx[layer].cpu().numpy(), st.keep_cnt[layer].cpu().numpy()
    for want_idx, want_cnt in ((pb.idx32, pb.cnt32), (pb.idx64, pb.cnt64)):
        assert np.array_equal(cnt, want_cnt)
        assert np.array_equal(idx, want_idx)       # ascending kept ids, then -1 padding: bit-exact


def check_attention(st, pb, attend, layer=0, step=0, K=None, V=None, n_chunks=None):
    b = _binding()
    q = wlm.gen_q(pb.wl, layer, step)[pb.seq_ids]
    qd = b.bits_to_bf16(q)
    lse = torch.zeros(st.S, dtype=torch.float32, device="cuda")
    out = st.decode_attn(layer, qd, lse=lse)
    torch.cuda.synchronize()
    assert st.poll_status() == 0
    want, want_b, want_lse, n_eff = pb.oracle_attn(q, attend, "f64", K, V, n_chunks)
    err = hz.check_output(b.bf16_to_bits(out), want, f"attn/{attend}")
    assert np.abs(lse.cpu().numpy() - want_lse).max() <= 1e-3
    return err, n_eff


def check_dense(st, pb, layer=0, step=0, K=None, V=None):
    b = _binding()
    q = wlm.gen_q(pb.wl, layer, 100 + step)[pb.seq_ids]
    lse = torch.zeros(st.S, dtype=torch.float32, device="cuda")
    out = st.decode_attn_dense(layer, b.bits_to_bf16(q), lse=lse)
    torch.cuda.synchronize()
    assert st.poll_status() == 0
    want, _, want_lse = pb.oracle_dense(q, "f64", K, V)
    hz.check_output(b.bf16_to_bits(out), want, "dense")
    assert np.abs(lse.cpu().numpy() - want_lse).max() <= 1e-3


def full_check(wl, attend="summary", pieces=(1.0,), keep=0.5):
    b = _binding()
    pb = hz.Problem(wl, keep=keep)
    st = make_store(wl, attend)
    load_kv(st, 0, pb.K, pb.V, pieces)
    torch.cuda.synchronize()
    Kp, Vp = pages_to_plain(st, 0, wl.n)
    assert np.array_equal(Kp, pb.K) and np.array_equal(Vp, pb.V)          # append: byte-exact through the page table
    assert st.seq_len[0].cpu().tolist() == [wl.n] * wl.B
    agg_w = b.AggWeights(pb.mlp) if pb.mlp is not None else None
    lstm_w = b.LstmWeights(pb.lstm)
    run_gpu_pipeline(st, pb, 0, agg_w, lstm_w)
    check_summaries(st, pb)
    check_gate_and_keep(st, pb)
    check_attention(st, pb, attend)
    check_dense(st, pb)
    return st, pb, agg_w, lstm_w


# ------------------------------------------------------------------------------------------------
def test_config1_full(request):
    full_check(wlm.CFG1, "summary")
    full_check(wlm.CFG1, "raw", pieces=(0.37, 0.9))


@pytest.mark.parametrize("attend", ["summary", "raw"])
def test_small_mlp_ragged(attend):
    # S = 15 (not a multiple of the gate's 8 sequences per cluster), n ragged against C and the 64-row tiles
    wl = wlm.Workload("ragged", B=3, H=5, n=1000 + 37, C=32, W=100, d_g=256, agg="mlp", d_sum=64, key_offset_std=0.5, seed=3)
    full_check(wl, attend, pieces=(0.5,))


@pytest.mark.parametrize("d_g", [64, 128, 256])
@pytest.mark.parametrize("C", [32, 128, 256])
def test_gate_sizes_and_chunk_sizes(d_g, C):
    wl = wlm.Workload("sizes", B=2, H=9, n=6 * C + 150, C=C, W=128, d_g=d_g, agg="mean", key_offset_std=0.5, seed=d_g + C)
    full_check(wl, "summary")


@pytest.mark.parametrize("d_g,B,H", [(64, 37, 33), (256, 9, 35)])
def test_two_sequence_groups_per_cluster(d_g, B, H):
    # more sequences than one group of 8 per cluster places in one wave: every cluster walks two groups;
    # S is ragged against 16 (a cluster's last group is partly or wholly empty)
    wl = wlm.Workload("groups", B=B, H=H, n=9 * 16 + 40, C=16, W=32, d_g=d_g, agg="mean", key_offset_std=0.5, seed=d_g + B)
    assert wl.S > 8 * (148 if d_g == 64 else 37)
    st, pb, _, lstm_w = full_check(wl, "summary")
    # one chunk at a time with the carried state: the same scores as the whole range
    want = st.scores[0].clone()
    for t in range(pb.Nc):
        st.gate(0, t, t + 1, lstm_w)
    torch.cuda.synchronize()
    assert st.poll_status() == 0
    assert torch.equal(st.scores[0, :, :pb.Nc], want[:, :pb.Nc])


def test_chunk_of_one_identity_keep_all_is_dense():
    # C = 1 with identity aggregation and tau = 0: the summary path reproduces dense attention
    b = _binding()
    wl = wlm.Workload("ident", B=1, H=4, n=300, C=1, W=44, d_g=64, agg="identity", seed=11, tau=0.0)
    pb = hz.Problem(wl, keep=None, tau=0.0, margin_eps=0.0)
    st = make_store(wl, "summary")
    load_kv(st, 0, pb.K, pb.V)
    run_gpu_pipeline(st, pb, 0, None, b.LstmWeights(pb.lstm))
    assert np.array_equal(b.bf16_to_bits(st.ksum_bf16[0, :, :pb.Nc]), pb.K[:, :pb.Nc])
    assert st.keep_cnt[0].cpu().tolist() == [pb.Nc] * wl.S
    q = wlm.gen_q(wl)
    out = st.decode_attn(0, b.bits_to_bf16(q))
    dense = st.decode_attn_dense(0, b.bits_to_bf16(q))
    want, _, _ = pb.oracle_dense(q)
    hz.check_output(b.bf16_to_bits(out), want, "identity keep-all")
    hz.check_output(b.bf16_to_bits(dense), want, "dense")


def test_keep_everything_raw_equals_dense_and_keep_nothing_is_window_only():
    b = _binding()
    wl = wlm.CFG1.small(n=1500, seed=5)
    pb = hz.Problem(wl)
    st = make_store(wl, "raw")
    load_kv(st, 0, pb.K, pb.V)
    lw = b.LstmWeights(pb.lstm)
    st.summarize_chunks(0, 0, pb.Nc)
    st.gate(0, 0, pb.Nc, lw)
    q = wlm.gen_q(wl)
    qd = b.bits_to_bf16(q)
    st.compact(0, 0.0)                                   # tau = 0 keeps every chunk
    assert st.keep_cnt[0].cpu().tolist() == [pb.Nc] * wl.S
    want, _, _ = pb.oracle_dense(q)
    hz.check_output(b.bf16_to_bits(st.decode_attn(0, qd)), want, "raw keep-all == dense")
    st.compact(0, 1.5)                                   # tau > 1 keeps nothing
    assert st.keep_cnt[0].cpu().tolist() == [0] * wl.S
    R = wl.n - pb.Nc * wl.C
    want, _, _ = pb.o64.attn_dense(q, np.ascontiguousarray(pb.K[:, -R:]), np.ascontiguousarray(pb.V[:, -R:]), hz.SCALE)
    hz.check_output(b.bf16_to_bits(st.decode_attn(0, qd)), want, "keep-nothing == window only")
    assert st.poll_status() == 0


def test_no_stale_chunks_and_empty_cache():
    b = _binding()
    wl = wlm.Workload("short", B=2, H=3, n=100, C=64, W=256, d_g=128, seed=2)      # n < W: nothing to gate
    pb = hz.Problem(wl, keep=None)
    assert pb.Nc == 0
    st = make_store(wl)
    q = wlm.gen_q(wl)
    qd = b.bits_to_bf16(q)
    lse = torch.zeros(wl.S, device="cuda")
    out = st.decode_attn(0, qd, lse=lse)                 # empty cache: zeros, lse = -inf
    assert torch.all(out.float() == 0) and torch.all(torch.isneginf(lse))
    load_kv(st, 0, pb.K, pb.V)
    lw = b.LstmWeights(pb.lstm)
    st.summarize_chunks(0, 0, 0)
    st.gate(0, 0, 0, lw)
    st.compact(0, 0.5)
    check_attention(st, pb, "summary")
    check_dense(st, pb)


def test_incremental_gate_equals_from_scratch_and_append_decode_steps():
    """Gate the first chunks, append tokens until more chunks leave the window, gate only the new
    ones with the carried (h, c): scores and keep list equal the from-scratch oracle.  Then a few
    append + decode steps (the cache grows, no chunk completes) against the oracle."""
    b = _binding()
    wl = wlm.CFG3.small(B=2, H=4, n_layers=1, n=64 + 5 * 256, seed=9)
    pb = hz.Problem(wl)
    st = make_store(wl)
    aw, lw = b.AggWeights(pb.mlp), b.LstmWeights(pb.lstm)
    n1 = 64 + 3 * 256 + 17
    st.append(0, b.bits_to_bf16(pb.K[:, :n1]), b.bits_to_bf16(pb.V[:, :n1]))
    nc1 = wl.n_stale_chunks(n1)
    st.summarize_chunks(0, 0, nc1, aw)
    st.gate(0, 0, nc1, lw)
    ready = st.append(0, b.bits_to_bf16(pb.K[:, n1:]), b.bits_to_bf16(pb.V[:, n1:]))
    assert ready == pb.Nc - nc1 and ready > 0
    st.summarize_chunks(0, nc1, pb.Nc, aw)
    st.gate(0, nc1, pb.Nc, lw)
    st.compact(0, pb.tau)
    check_summaries(st, pb)
    check_gate_and_keep(st, pb)
    K, V = pb.K, pb.V
    for step in range(wl.n_append):
        kn, vn = wlm.gen_new_tokens(wl, 0, step)
        st.append(0, b.bits_to_bf16(kn), b.bits_to_bf16(vn))
        K, V = np.concatenate([K, kn], axis=1), np.concatenate([V, vn], axis=1)
        check_attention(st, pb, "summary", step=step, K=K, V=V)
    check_dense(st, pb, K=K, V=V)
    assert st.layer_state(0) == dict(n_tokens=wl.n + wl.n_append, n_summarised=pb.Nc, n_gated=pb.Nc, n_compacted=pb.Nc)


def test_set_len_below_the_compacted_range_drops_the_keep_list():
    """Roll a step back across a chunk boundary without compacting again: the keep list on the device still
    names the chunk that is raw tail again, so the handle must stop using it.  Attention then reads every
    stored row (exact: Eq. 1 over all n tokens) and the status word stays clean."""
    b = _binding()
    wl = wlm.CFG1.small(B=1, H=4, n=1024, C=64, W=256, seed=12)          # 1024 - 256 = 12 chunks exactly
    pb = hz.Problem(wl, keep=None, tau=0.0, margin_eps=0.0)             # tau = 0 keeps every chunk, the last one included
    st = make_store(wl)
    load_kv(st, 0, pb.K, pb.V)
    run_gpu_pipeline(st, pb, 0, None, b.LstmWeights(pb.lstm))
    assert int(st.keep_cnt[0].min()) == pb.Nc == 12
    st.set_len(0, wl.n - 1)                                              # 11 stale chunks now; chunk 11 is raw tail again
    assert st.layer_state(0) == dict(n_tokens=wl.n - 1, n_summarised=11, n_gated=0, n_compacted=0)
    q = wlm.gen_q(wl, 0, 5)
    for fn in (st.decode_attn, st.decode_attn_static):
        out = fn(0, b.bits_to_bf16(q))
        torch.cuda.synchronize()
        assert st.poll_status() == 0
        want, _, _ = pb.oracle_dense(q, "f64", np.ascontiguousarray(pb.K[:, :-1]), np.ascontiguousarray(pb.V[:, :-1]))
        hz.check_output(b.bf16_to_bits(out), want, "attention after roll-back")
    # gating and compacting again brings the gated path back
    st.append(0, b.bits_to_bf16(pb.K[:, -1:]), b.bits_to_bf16(pb.V[:, -1:]))
    run_gpu_pipeline(st, pb, 0, None, b.LstmWeights(pb.lstm))
    assert np.array_equal(st.keep_idx[0].cpu().numpy(), pb.idx64)
    check_attention(st, pb, "summary")


@pytest.mark.parametrize("agg", ["mlp", "mean", "token_mlp"])
def test_refresh_equals_the_stepwise_calls(agg):
    """kvE_refresh = summaries of all stale chunks + gate from scratch + keep list in one call: against the oracle, and
    bit for bit against the three calls issued one after the other; also replayed from a CUDA graph."""
    b = _binding()
    wl = wlm.CFG2.small(B=2, H=6, n=64 * 75 + 9, C=64, W=128, agg=agg, d_sum=256 if agg != "mean" else 0, seed=91)
    pb = hz.Problem(wl)
    assert pb.Nc == 73
    st = make_store(wl)
    load_kv(st, 0, pb.K, pb.V)
    aw = b.AggWeights(pb.mlp) if pb.mlp is not None else None
    lw = b.LstmWeights(pb.lstm)
    for rep in range(2):                                     # twice: the second run finds the first one's state
        st.refresh(0, aw, lw, pb.tau)
        torch.cuda.synchronize()
        assert st.poll_status() == 0
        assert st.layer_state(0) == dict(n_tokens=wl.n, n_summarised=pb.Nc, n_gated=pb.Nc, n_compacted=pb.Nc)
        check_summaries(st, pb)
        check_gate_and_keep(st, pb)
        check_attention(st, pb, "summary", step=rep)
    got = [x.clone() for x in (st.scores[0], st.keep_idx[0], st.lstm_h[0], st.lstm_c[0], st.ksum_bf16[0])]
    run_gpu_pipeline(st, pb, 0, aw, lw)
    for a_, b_ in zip(got, (st.scores[0], st.keep_idx[0], st.lstm_h[0], st.lstm_c[0], st.ksum_bf16[0])):
        assert torch.equal(a_, b_)
    # inside a CUDA graph
    graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            st.refresh(0, aw, lw, pb.tau)
    torch.cuda.current_stream().wait_stream(side)
    st.scores.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert st.poll_status() == 0 and torch.equal(st.scores[0], got[0])


@pytest.mark.parametrize("d_g,agg,planes,B,H", [(256, "mlp", 2, 3, 5), (256, "mean", 3, 3, 5), (128, "mean", 2, 3, 5), (64, "mean", 2, 3, 5),
                                                  (64, "max", 3, 3, 5),
                                                  # more groups of 8 sequences than clusters in a wave: 2 and 4 groups per cluster
                                                  (256, "mean", 2, 9, 35), (256, "mean", 2, 19, 32), (256, "mean", 3, 19, 32),
                                                  (128, "mean", 2, 37, 33), (64, "mean", 2, 75, 32)])
def test_gate_next_extends_scores_and_keep_list_one_chunk_at_a_time(d_g, agg, planes, B, H):
    """The trigger's gate step in one launch: from a keep list over the first chunks, kvE_gate_next takes the chunks one
    by one; scores, carried state, keep list and the compacted summary rows (through attention) must match the oracle
    exactly as kvE_gate + kvE_compact over the whole range do."""
    b = _binding()
    Nc = 21 if B * H < 100 else 7
    wl = wlm.Workload("next", B=B, H=H, n=32 * Nc + 64 + 5, C=32, W=64, d_g=d_g, agg=agg, d_sum=128 if agg == "mlp" else 0,
                      key_offset_std=0.5, seed=300 + d_g + planes + B)
    pb = hz.Problem(wl, keep=0.5)
    assert pb.Nc == Nc
    aw = b.AggWeights(pb.mlp) if pb.mlp is not None else None
    lw = b.LstmWeights(pb.lstm)
    ref = make_store(wl)
    load_kv(ref, 0, pb.K, pb.V)
    ref.set_gate_planes(planes)
    run_gpu_pipeline(ref, pb, 0, aw, lw)

    st = make_store(wl)
    load_kv(st, 0, pb.K, pb.V)
    st.set_gate_planes(planes)
    with pytest.raises(b.KveError) as e:                  # nothing summarised yet
        st.gate_next(0, lw, pb.tau)
    assert e.value.rc == -4
    st.summarize_chunks(0, 0, pb.Nc, aw)
    st.gate_next(0, lw, pb.tau)                           # chunk 0: no list yet, the general path
    assert st.layer_state(0)["n_gated"] == 1 and st.layer_state(0)["n_compacted"] == 1
    st.gate(0, 1, 4, lw)                                  # the list is stale now ...
    assert st.layer_state(0)["n_compacted"] <= 1
    st.gate_next(0, lw, pb.tau)                           # ... so this one re-lists as well
    assert st.layer_state(0) == dict(n_tokens=wl.n, n_summarised=pb.Nc, n_gated=5, n_compacted=5)
    for t in range(5, pb.Nc):
        st.gate_next(0, lw, pb.tau)                       # one launch each
    torch.cuda.synchronize()
    assert st.poll_status() == 0
    assert st.layer_state(0) == dict(n_tokens=wl.n, n_summarised=pb.Nc, n_gated=pb.Nc, n_compacted=pb.Nc)
    check_gate_and_keep(st, pb)
    check_attention(st, pb, "summary")
    # against the range kernels on the same device: another summation order, nothing more
    assert (st.scores[0, :, :pb.Nc] - ref.scores[0, :, :pb.Nc]).abs().max().item() <= 2e-6
    assert (st.lstm_h[0] - ref.lstm_h[0]).abs().max().item() <= 2e-6
    assert torch.equal(st.keep_idx[0], ref.keep_idx[0]) and torch.equal(st.keep_cnt[0], ref.keep_cnt[0])
    with pytest.raises(b.KveError) as e:                  # every summarised chunk is gated
        st.gate_next(0, lw, pb.tau)
    assert e.value.rc == -4


def test_layers_are_independent():
    b = _binding()
    wl = wlm.CFG1.small(n=1024, B=2, H=4, n_layers=3)
    st = make_store(wl, n_layers=3)
    pbs = [hz.Problem(wl.small(seed=wl.seed + L), layer=L) for L in range(3)]
    for L in (2, 0, 1):
        load_kv(st, L, pbs[L].K, pbs[L].V)
    for L in range(3):
        lw = b.LstmWeights(pbs[L].lstm)
        run_gpu_pipeline(st, pbs[L], L, None, lw)
    for L in range(3):
        check_summaries(st, pbs[L], L)
        check_gate_and_keep(st, pbs[L], L)
        check_attention(st, pbs[L], "summary", L)


def test_decode_step_host_matches_stepwise_calls():
    b = _binding()
    wl = wlm.CFG1.small(n=1024 - 1, seed=4)
    pb0 = hz.Problem(wl.small(n=1024), keep=0.5)          # oracle on the cache AFTER the step's append
    st = make_store(wl.small(n=1024))
    lw = b.LstmWeights(pb0.lstm)
    load_kv(st, 0, pb0.K[:, :-1], pb0.V[:, :-1])
    q = wlm.gen_q(wl)
    pin = lambda a: b.bits_to_bf16(a, "cpu").pin_memory()
    out = torch.zeros(wl.S, 128, dtype=torch.bfloat16).pin_memory()
    st.decode_step_host(0, pin(pb0.K[:, -1]), pin(pb0.V[:, -1]), pin(q), out, None, lw, pb0.tau, from_scratch=True)
    want, _, _, _ = pb0.oracle_attn(q, "summary")
    hz.check_output(b.bf16_to_bits(out), want, "step_host")
    check_gate_and_keep(st, pb0)
    # the asynchronous form: two steps enqueued back to back (the second rolls the first one's token back and
    # redoes it), nothing waited for until the stream is synchronised; same result
    out2 = torch.zeros(wl.S, 128, dtype=torch.bfloat16).pin_memory()
    hk, hv, hq = pin(pb0.K[:, -1]), pin(pb0.V[:, -1]), pin(q)
    for _ in range(2):
        st.set_len(0, 1024 - 1)
        st.decode_step_host(0, hk, hv, hq, out2, None, lw, pb0.tau, from_scratch=True, wait=False)
    torch.cuda.synchronize()
    assert st.poll_status() == 0
    assert torch.equal(out2, out)


@pytest.mark.parametrize("agg", ["mean", "mlp"])
def test_decode_step_host_streams_across_triggers(agg):
    """The host-buffer step without the from-scratch refresh: tokens arrive one by one, and whenever a chunk has left
    the window the step summarises it, gates it with the carried state (kvE_gate_next) and extends the keep list.
    After 2 C + 3 steps - two triggers - everything must match the oracle on the final cache."""
    b = _binding()
    C_, W, n0 = 16, 32, 16 * 6 + 32 + 3
    n1 = n0 + 2 * C_ + 3
    wl1 = wlm.Workload("hoststream", B=2, H=5, n=n1, C=C_, W=W, d_g=128, agg=agg, d_sum=64 if agg == "mlp" else 0,
                       key_offset_std=0.5, seed=77)
    pb = hz.Problem(wl1, keep=0.5)
    st = make_store(wl1)
    aw = b.AggWeights(pb.mlp) if pb.mlp is not None else None
    lw = b.LstmWeights(pb.lstm)
    load_kv(st, 0, np.ascontiguousarray(pb.K[:, :n0]), np.ascontiguousarray(pb.V[:, :n0]))
    st.refresh(0, aw, lw, pb.tau)
    pin = lambda a: b.bits_to_bf16(np.ascontiguousarray(a), "cpu").pin_memory()
    out = torch.zeros(wl1.S, 128, dtype=torch.bfloat16).pin_memory()
    q = wlm.gen_q(wl1)
    hq = pin(q)
    gated = [st.layer_state(0)["n_gated"]]
    for pos in range(n0, n1):
        st.decode_step_host(0, pin(pb.K[:, pos]), pin(pb.V[:, pos]), hq, out, aw, lw, pb.tau, from_scratch=False)
        gated.append(st.layer_state(0)["n_gated"])
    assert st.poll_status() == 0
    assert gated[0] == pb.Nc - 2 and gated[-1] == pb.Nc and sorted(set(gated)) == [pb.Nc - 2, pb.Nc - 1, pb.Nc]
    assert st.layer_state(0) == dict(n_tokens=n1, n_summarised=pb.Nc, n_gated=pb.Nc, n_compacted=pb.Nc)
    check_summaries(st, pb)
    check_gate_and_keep(st, pb)
    want, _, _, _ = pb.oracle_attn(q, "summary")
    hz.check_output(b.bf16_to_bits(out), want, "host stream")


def test_host_side_errors():
    b = _binding()
    wl = wlm.CFG1.small(n=512)
    st = make_store(wl)
    pb = hz.Problem(wl)
    lw = b.LstmWeights(pb.lstm)
    with pytest.raises(b.KveError) as e:                  # nothing stored yet: no chunk may be summarised
        st.summarize_chunks(0, 0, 1)
    assert e.value.rc == -4
    load_kv(st, 0, pb.K, pb.V)
    with pytest.raises(b.KveError) as e:                  # gate before summarize
        st.gate(0, 0, pb.Nc, lw)
    assert e.value.rc == -4
    with pytest.raises(b.KveError) as e:                  # capacity
        st.append(0, b.bits_to_bf16(pb.K[:, :1]), b.bits_to_bf16(pb.V[:, :1]))
    assert e.value.rc == -3
    with pytest.raises(b.KveError) as e:                  # bad layer
        st.compact(5, 0.5)
    assert e.value.rc == -1
    st.summarize_chunks(0, 0, pb.Nc)
    with pytest.raises(b.KveError) as e:                  # gate must continue where it stopped
        st.gate(0, 2, pb.Nc, lw)
    assert e.value.rc == -4
    with pytest.raises(b.KveError):                       # unsupported geometry is refused at create
        b.Store(B=1, H=1, C_=64, W=0, max_tokens=128, d_g=100)
    assert st.poll_status() == 0


def test_bad_page_id_sets_status_word_without_fault():
    b = _binding()
    wl = wlm.CFG1.small(n=512)
    pt = np.arange(wl.S * wl.max_chunks, dtype=np.int32).reshape(1, wl.S, wl.max_chunks)
    pt[0, 1, 2] = 10 ** 6                                 # beyond n_pages: the kernels must skip it
    st = make_store(wl, page_perm=pt)
    pb = hz.Problem(wl)
    load_kv(st, 0, pb.K, pb.V)
    torch.cuda.synchronize()
    assert st.poll_status() == -3
    assert st.poll_status() == 0                          # cleared by the poll


# ------------------------------------------------------------------------------------------------ full sizes
@pytest.mark.parametrize("which", [0, 1])
def test_a_bounded_wait_that_runs_out_reports_timeout_and_leaves_the_handle_usable(which):
    """The failure path of every kernel: a wait on a barrier nothing completes gives up after its limit, the kernel
    returns, the status word reads KVE_ERR_TIMEOUT (-6), and ordinary calls on the same handle keep working."""
    b = _binding()
    wl = wlm.CFG1.small(n=512, seed=3)
    pb = hz.Problem(wl)
    st = make_store(wl)
    load_kv(st, 0, pb.K, pb.V)
    run_gpu_pipeline(st, pb, 0, None, b.LstmWeights(pb.lstm))
    st.selftest_timeout(which)
    torch.cuda.synchronize()                       # the kernel came back by itself
    assert st.poll_status() == -6
    assert st.poll_status() == 0                   # reading clears the word
    check_attention(st, pb, "summary")             # same handle, same context: still correct
    check_gate_and_keep(st, pb)


def test_config2_full_size():
    """Llama-2-7B-shaped layer at the size bench.py times (B 8, H 32, n 4096, MLP aggregator, d_g 256)."""
    st, pb, aw, lw = full_check(wlm.CFG2, "summary")
    keep = st.keep_cnt[0].float().mean().item() / pb.Nc
    assert 0.4 < keep < 0.6
    # the RAW reading on the same store contents
    st2 = make_store(wlm.CFG2, "raw")
    load_kv(st2, 0, pb.K, pb.V)
    run_gpu_pipeline(st2, pb, 0, aw, lw)
    check_gate_and_keep(st2, pb)
    check_attention(st2, pb, "raw")


def _sampled_full_size(wl, n_sample, attend="summary", n_steps=0):
    """Full-size launch, oracle on a sample of the sequences: the sampled sequences carry seeded,
    margin-repaired inputs, the others carry device-generated filler of the same distribution."""
    b = _binding()
    rng = np.random.default_rng(wl.seed)
    seqs = sorted(rng.choice(wl.S, n_sample, replace=False).tolist())
    pb = hz.Problem(wl, seq_ids=seqs)
    st = make_store(wl, attend, page_perm=None)
    g = torch.Generator(device="cuda").manual_seed(wl.seed)
    for b0 in range(0, wl.S if n_sample < wl.S else 0, 64):  # filler, 64 sequences at a time
        shape = (min(64, wl.S - b0), wl.n, 128)
        kf = torch.randn(shape, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        vf = torch.randn(shape, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        pages = st.page_table[0, b0:b0 + shape[0]].long()   # [s, max_chunks]
        nch = wl.n // wl.C
        st.k_pages[pages[:, :nch].reshape(-1)] = kf[:, :nch * wl.C].reshape(-1, wl.C, 128)
        st.v_pages[pages[:, :nch].reshape(-1)] = vf[:, :nch * wl.C].reshape(-1, wl.C, 128)
        del kf, vf
    for i, s in enumerate(seqs):                            # the sampled sequences' real data
        pages = st.page_table[0, s].long()
        nch = -(-wl.n // wl.C)
        pad = nch * wl.C - wl.n
        kk = np.pad(pb.K[i], ((0, pad), (0, 0)))
        vv = np.pad(pb.V[i], ((0, pad), (0, 0)))
        st.k_pages[pages[:nch]] = b.bits_to_bf16(kk).reshape(nch, wl.C, 128)
        st.v_pages[pages[:nch]] = b.bits_to_bf16(vv).reshape(nch, wl.C, 128)
    st.set_len(0, wl.n)
    aw, lw = (b.AggWeights(pb.mlp) if pb.mlp else None), b.LstmWeights(pb.lstm)
    run_gpu_pipeline(st, pb, 0, aw, lw)
    sel = torch.tensor(seqs, device="cuda")
    Nc = pb.Nc
    sc = st.scores[0, sel, :Nc].cpu().numpy()
    assert np.abs(sc - pb.sc64[:, :Nc]).max() <= 2e-4
    assert np.array_equal(st.keep_cnt[0, sel].cpu().numpy(), pb.cnt64)
    assert np.array_equal(st.keep_idx[0, sel].cpu().numpy(), pb.idx64)
    kb = b.bf16_to_bits(st.ksum_bf16[0, sel, :Nc])
    kg, kw = (wlm.bf16_bits_to_f32(x).astype(np.float64) for x in (kb, pb.sm32["ksum_b16"][:, :Nc]))
    assert np.all(np.abs(kg - kw) <= 2.0 ** -7 * np.abs(kw) + 1e-5)
    # properties that hold for every sequence at any size
    cnt = st.keep_cnt[0].cpu().numpy()
    idx = st.keep_idx[0].cpu().numpy()
    scores = st.scores[0, :, :Nc].cpu().numpy()
    assert np.array_equal(cnt, (scores >= np.float32(pb.tau)).sum(axis=1))
    for s in range(0, wl.S, 7):
        assert np.array_equal(idx[s, :cnt[s]], np.nonzero(scores[s] >= np.float32(pb.tau))[0]) and np.all(idx[s, cnt[s]:] == -1)
    K, V = pb.K, pb.V
    for step in range(max(1, n_steps)):
        if n_steps:
            kn, vn = wlm.gen_new_tokens(wl, 0, step)
            st.append(0, b.bits_to_bf16(kn), b.bits_to_bf16(vn))
            K, V = np.concatenate([K, kn[seqs]], axis=1), np.concatenate([V, vn[seqs]], axis=1)
        q = wlm.gen_q(wl, 0, step)
        out = st.decode_attn(0, b.bits_to_bf16(q))
        want, _, _, _ = pb.oracle_attn(q[seqs], attend, "f64", K, V)
        hz.check_output(b.bf16_to_bits(out[sel]), want, f"sampled attn step {step}")
        assert torch.isfinite(out.float()).all()
    dense = st.decode_attn_dense(0, b.bits_to_bf16(q))
    want, _, _ = pb.oracle_dense(q[seqs], "f64", K, V)
    hz.check_output(b.bf16_to_bits(dense[sel]), want, "sampled dense")
    assert st.poll_status() == 0


def test_config3_one_layer_full_size_all_sequences():
    # every one of the 128 sequences against the oracle (the oracle needs a few seconds for the layer)
    _sampled_full_size(wlm.CFG3.small(n_layers=1), n_sample=wlm.CFG3.S, n_steps=wlm.CFG3.n_append)


def test_config4_one_layer_full_size_all_sequences():
    # all 512 sequences x 16512 tokens: the oracle with margin repair takes well under a minute on 16 cores
    _sampled_full_size(wlm.CFG4.small(n_layers=1), n_sample=wlm.CFG4.S)


@pytest.mark.parametrize("B,n,C,keep", [(1, 2048, 32, 0.25), (4, 8192, 64, 0.75), (2, 32768, 256, 1.0), (64, 2048, 128, 0.5),
                                        (64, 32768, 32, 0.5)])      # the last: the largest point of the sweep (about 46 GB)
def test_sweep_points_sampled(B, n, C, keep):
    wl = wlm.Workload(f"sweep_b{B}_n{n}_c{C}", B=B, H=32, n=n, C=C, W=512, d_g=256, agg="mean", key_offset_std=0.5, seed=B + n + C)
    b = _binding()
    rng = np.random.default_rng(1)
    seqs = sorted(rng.choice(wl.S, min(4, wl.S), replace=False).tolist())
    if keep >= 1.0:
        pb = hz.Problem(wl, seq_ids=seqs, keep=None, tau=0.0, margin_eps=0.0)
    else:
        pb = hz.Problem(wl, seq_ids=seqs, keep=keep)
    for attend in ("summary", "raw"):
        st = make_store(wl, attend, page_perm=None)
        for i, s in enumerate(seqs):
            pages = st.page_table[0, s].long()
            nch = wl.n // wl.C
            st.k_pages[pages[:nch]] = b.bits_to_bf16(pb.K[i]).reshape(nch, wl.C, 128)
            st.v_pages[pages[:nch]] = b.bits_to_bf16(pb.V[i]).reshape(nch, wl.C, 128)
        st.set_len(0, wl.n)
        run_gpu_pipeline(st, pb, 0, None, b.LstmWeights(pb.lstm))
        sel = torch.tensor(seqs, device="cuda")
        assert np.array_equal(st.keep_idx[0, sel].cpu().numpy(), pb.idx64)
        q = wlm.gen_q(wl)
        out = st.decode_attn(0, b.bits_to_bf16(q))
        want, _, _, _ = pb.oracle_attn(q[seqs], attend)
        hz.check_output(b.bf16_to_bits(out[sel]), want, f"sweep {attend}")
        del st
        torch.cuda.empty_cache()


def test_long_gate_chain_two_and_three_planes():
    """The longest recurrence of the stress sweep (n = 32768, C = 32: 1008 LSTM steps per sequence) on the cluster
    path: scores against the f64 oracle at the usual 2e-4 and keep lists bit-exact, with the default two bf16 planes of
    h in the recurrent product and with three (exact products); the drift of the two is printed side by side."""
    b = _binding()
    wl = wlm.Workload("long_chain", B=1, H=32, n=32768, C=32, W=512, d_g=256, agg="mean", key_offset_std=0.5, seed=77)
    pb = hz.Problem(wl)
    assert pb.Nc == 1008
    st = make_store(wl, page_perm=None)
    load_kv(st, 0, pb.K, pb.V)
    lw = b.LstmWeights(pb.lstm)
    st.summarize_chunks(0, 0, pb.Nc, None)
    drift = {}
    for planes in (3, 2):
        st.set_gate_planes(planes)
        st.gate(0, 0, pb.Nc, lw)
        st.compact(0, pb.tau)
        torch.cuda.synchronize()
        assert st.poll_status() == 0
        sc = st.scores[0, :, :pb.Nc].cpu().numpy().astype(np.float64)
        err = np.abs(sc - pb.sc64[:, :pb.Nc])
        drift[planes] = (float(err.max()), float(err[:, -64:].max()), float(np.abs(st.lstm_h[0].cpu().numpy() - pb.h64).max()))
        assert err.max() <= 2e-4
        assert np.array_equal(st.keep_idx[0].cpu().numpy(), pb.idx64) and np.array_equal(st.keep_cnt[0].cpu().numpy(), pb.cnt64)
    print(f"score error vs f64 over 1008 steps (max, max over the last 64 steps, final |h| error): "
          f"3 planes {drift[3]}, 2 planes {drift[2]}")
    # the error does not grow along the chain: the LSTM forgets, so the last steps are no worse than the whole
    assert drift[2][1] <= 2e-4 and drift[3][0] <= drift[2][0] + 5e-5
    check_attention(st, pb, "summary")


def test_streaming_soak_reuses_reclaimed_pages_over_several_triggers():
    """Sec. 3.3 as it runs: tokens arrive one by one (kvE_decode_step: append at the device-held length + attention in one
    launch, captured ONCE in a CUDA graph and replayed for the whole run); every C tokens a chunk leaves the window: true length to the host, that ONE chunk summarised and gated
    with the carried (h, c), keep list rebuilt, the pages of all gated chunks handed back, and the freed pages given to
    the chunks that fill next.  After every trigger: attention against the oracle on the grown cache, the raw tail
    read back through the page table, the pages really re-used, status word clean."""
    b = _binding()
    C_, W, n0, n_triggers = 32, 64, 64 + 3 * 32, 6
    wl_full = wlm.Workload("soak", B=1, H=4, n=n0 + n_triggers * C_, C=C_, W=W, d_g=64, agg="mean", key_offset_std=0.5, seed=88)
    pb = hz.Problem(wl_full)                       # repaired inputs and oracle results for the whole run
    K, V, S = pb.K, pb.V, wl_full.S
    st = make_store(wl_full.small(n_append=2 * C_), page_perm=None)
    mc = st.max_chunks
    lw = b.LstmWeights(pb.lstm)
    # pages: only the chunks in use and ONE spare chunk per sequence own a page; everything further is unassigned
    pt = st.page_table[0].clone()
    first_unassigned = n0 // C_ + 2
    pt[:, first_unassigned:] = -1
    st.page_table[0].copy_(pt)
    next_slot = first_unassigned                   # next chunk index that needs a page
    st.append(0, b.bits_to_bf16(K[:, :n0]), b.bits_to_bf16(V[:, :n0]))
    nc = wl_full.n_stale_chunks(n0)
    assert nc == 3
    st.summarize_chunks(0, 0, nc, None)
    st.gate(0, 0, nc, lw)
    st.compact(0, pb.tau)
    k_in = torch.zeros((S, 128), dtype=torch.bfloat16, device="cuda")
    v_in, q_in, out = torch.zeros_like(k_in), torch.zeros_like(k_in), torch.zeros_like(k_in)
    side = torch.cuda.Stream()
    reclaimed_ever, reused = set(), 0
    n = n0

    def oracle_out(q, n_now, nc_now):
        idx, cnt = pb.o64.compact(pb.sc64, nc_now, pb.tau)
        return pb.o64.attn(q, np.ascontiguousarray(K[:, :n_now]), np.ascontiguousarray(V[:, :n_now]), C_, nc_now, idx, cnt,
                           pb.sm64["ksum_b16"], pb.sm64["vsum_b16"], hz.ATT["summary"], hz.SCALE)[0]

    # ONE graph for the whole run: the step appends at the length the device holds and reads the number of chunks under the
    # keep list from the device too, so the triggers that happen between replays need no new capture
    graph = torch.cuda.CUDAGraph()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            st.decode_step(0, k_in, v_in, q_in, out, n_reserve=n_triggers * C_)
    torch.cuda.current_stream().wait_stream(side)
    for trig in range(n_triggers):
        # ---- hand back the pages of every gated chunk, give them to the chunks that fill next ----
        free_list, free_count = st.reclaim_pages(0, 0, nc, mode="gated")
        torch.cuda.synchronize()
        got = free_list[:int(free_count)].cpu().numpy()
        assert len(got) == S * (nc if trig == 0 else 1)            # all gated chunks the first time, the new one afterwards
        reclaimed_ever.update(int(p) for p in got)
        pt = st.page_table[0].clone()
        assert int((pt[:, :nc] >= 0).sum()) == 0                  # gated chunks own no page any more
        pt[:, next_slot] = torch.from_numpy(got[:S].astype(np.int32)).cuda()
        reused += S
        st.page_table[0].copy_(pt)
        next_slot += 1
        # ---- C decode steps between two triggers: replays of the one graph ----
        for step in range(C_):
            q = wlm.gen_q(wl_full, 0, 1000 * trig + step)
            k_in.copy_(b.bits_to_bf16(K[:, n])); v_in.copy_(b.bits_to_bf16(V[:, n])); q_in.copy_(b.bits_to_bf16(q))
            graph.replay()
            n += 1
            if step % 8 == 7 or step == C_ - 1:
                torch.cuda.synchronize()
                hz.check_output(b.bf16_to_bits(out), oracle_out(q, n, nc), f"trigger {trig}, step {step}")
        torch.cuda.synchronize()
        assert st.poll_status() == 0 and int(st.seq_len[0, 0]) == n
        # ---- the trigger: one chunk per sequence has left the window ----
        st.set_len(0, n)
        assert wl_full.n_stale_chunks(n) == nc + 1
        st.summarize_chunks(0, nc, nc + 1, None)
        st.gate(0, nc, nc + 1, lw)                                 # carried (h, c)
        st.compact(0, pb.tau)
        nc += 1
        torch.cuda.synchronize()
        assert st.poll_status() == 0
        sc = st.scores[0, :, :nc].cpu().numpy()
        assert np.abs(sc - pb.sc64[:, :nc]).max() <= 2e-4
        idx, cnt = pb.o64.compact(pb.sc64, nc, pb.tau)
        assert np.array_equal(st.keep_cnt[0].cpu().numpy(), cnt) and np.array_equal(st.keep_idx[0, :, :nc].cpu().numpy(), idx[:, :nc])
        q = wlm.gen_q(wl_full, 0, 5000 + trig)
        got_out = st.decode_attn(0, b.bits_to_bf16(q))
        torch.cuda.synchronize()
        hz.check_output(b.bf16_to_bits(got_out), oracle_out(q, n, nc), f"after trigger {trig}")
        # the raw tail, read back through the (partly re-used) pages
        ptab = st.page_table[0].cpu().numpy()
        kp = b.bf16_to_bits(st.k_pages)
        for t in range(nc, -(-n // C_)):
            rows = min(C_, n - t * C_)
            assert np.array_equal(kp[ptab[:, t]][:, :rows], K[:, t * C_:t * C_ + rows])
            if t >= first_unassigned:
                assert all(int(p) in reclaimed_ever for p in ptab[:, t])     # this chunk lives in pages that held gated chunks
    assert n == wl_full.n and nc == pb.Nc and reused == n_triggers * S


@pytest.mark.parametrize("agg,d_g,B,H", [("mean", 64, 1, 4), ("mlp", 256, 2, 5), ("max", 128, 3, 3), ("mean", 256, 9, 35)])
def test_one_graph_runs_decode_steps_and_triggers_without_the_host(agg, d_g, B, H):
    """Sec. 3.3 with the host out of the loop: ONE captured graph holds C decode steps (kvE_decode_step) followed by the
    trigger in its device-positioned form (kvE_refresh_next).  Every replay appends C tokens, attends after each, and
    takes the chunk that has left the window through summary, gate and keep list.  After each replay: scores, keep lists
    and the carried state against the oracle, attention outputs of the last step too; the handle then adopts the device's
    counters and a host-issued step continues from there."""
    b = _binding()
    C_, W, n_replays = 16, 32, 5
    n0 = W + 3 * C_                                  # three chunks gated before the graph takes over; (n0 - W) % C == 0
    wl_full = wlm.Workload("graphtrig", B=B, H=H, n=n0 + n_replays * C_ + 1, C=C_, W=W, d_g=d_g, agg=agg,
                           d_sum=64 if agg == "mlp" else 0, key_offset_std=0.5, seed=500 + d_g + B)
    pb = hz.Problem(wl_full)
    K, V, S = pb.K, pb.V, wl_full.S
    st = make_store(wl_full)
    aw = b.AggWeights(pb.mlp) if pb.mlp is not None else None
    lw = b.LstmWeights(pb.lstm)
    st.append(0, b.bits_to_bf16(np.ascontiguousarray(K[:, :n0])), b.bits_to_bf16(np.ascontiguousarray(V[:, :n0])))
    nc = wl_full.n_stale_chunks(n0)
    assert nc == 3
    with pytest.raises(b.KveError) as e:             # no keep list yet: nothing for the device to append to
        st.refresh_next(0, aw, lw, pb.tau)
    assert e.value.rc == -4
    st.refresh(0, aw, lw, pb.tau)
    # per-step inputs of one replay live in [C] slots that the graph's launches read
    k_in = torch.zeros((C_, S, 128), dtype=torch.bfloat16, device="cuda")
    v_in, q_in, out = torch.zeros_like(k_in), torch.zeros_like(k_in), torch.zeros_like(k_in)
    graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for i in range(C_):
                st.decode_step(0, k_in[i], v_in[i], q_in[i], out[i], n_reserve=n_replays * C_)
            st.refresh_next(0, aw, lw, pb.tau)
    torch.cuda.current_stream().wait_stream(side)
    st.adopt_device_state(0)                         # capture advanced the handle's counters, nothing ran
    assert st.layer_state(0) == dict(n_tokens=n0, n_summarised=3, n_gated=3, n_compacted=3)

    def oracle_out(q, n_now, nc_now):
        idx, cnt = pb.o64.compact(pb.sc64, nc_now, pb.tau)
        return pb.o64.attn(q, np.ascontiguousarray(K[:, :n_now]), np.ascontiguousarray(V[:, :n_now]), C_, nc_now, idx, cnt,
                           pb.sm64["ksum_b16"], pb.sm64["vsum_b16"], hz.ATT["summary"], hz.SCALE)[0]

    n = n0
    for rep in range(n_replays):
        qs = [wlm.gen_q(wl_full, 0, 100 * rep + i) for i in range(C_)]
        k_in.copy_(b.bits_to_bf16(np.ascontiguousarray(K[:, n:n + C_].transpose(1, 0, 2))))
        v_in.copy_(b.bits_to_bf16(np.ascontiguousarray(V[:, n:n + C_].transpose(1, 0, 2))))
        q_in.copy_(b.bits_to_bf16(np.stack(qs)))
        graph.replay()
        torch.cuda.synchronize()
        assert st.poll_status() == 0
        # step i of the replay saw n + i + 1 tokens and the keep list over nc chunks; the trigger came after the last step
        for i in (0, C_ // 2, C_ - 1):
            hz.check_output(b.bf16_to_bits(out[i]), oracle_out(qs[i], n + i + 1, nc), f"replay {rep}, step {i}")
        n += C_
        nc += 1
        assert int(st.seq_len[0, 0]) == n
        sc = st.scores[0, :, :nc].cpu().numpy()
        assert np.abs(sc - pb.sc64[:, :nc]).max() <= 2e-4
        idx, cnt = pb.o64.compact(pb.sc64, nc, pb.tau)
        assert np.array_equal(st.keep_cnt[0].cpu().numpy(), cnt) and np.array_equal(st.keep_idx[0, :, :nc].cpu().numpy(), idx[:, :nc])
    # the host takes over again: its counters come from the device, the next step is issued directly
    st.adopt_device_state(0)
    assert st.layer_state(0) == dict(n_tokens=n, n_summarised=nc, n_gated=nc, n_compacted=nc)
    q = wlm.gen_q(wl_full, 0, 9999)
    got = torch.zeros((S, 128), dtype=torch.bfloat16, device="cuda")
    st.decode_step(0, b.bits_to_bf16(np.ascontiguousarray(K[:, n])), b.bits_to_bf16(np.ascontiguousarray(V[:, n])), b.bits_to_bf16(q), got)
    torch.cuda.synchronize()
    assert st.poll_status() == 0
    hz.check_output(b.bf16_to_bits(got), oracle_out(q, n + 1, nc), "host step after the graph")
    assert n + 1 == wl_full.n and nc == pb.Nc
    # a trigger that is not due does nothing
    before = (st.scores[0].clone(), st.keep_cnt[0].clone(), st.lstm_h[0].clone())
    st.refresh_next(0, aw, lw, pb.tau)
    torch.cuda.synchronize()
    assert st.poll_status() == 0 and st.layer_state(0)["n_gated"] == nc
    assert all(torch.equal(a_, b_) for a_, b_ in zip(before, (st.scores[0], st.keep_cnt[0], st.lstm_h[0])))


def test_one_graph_serves_two_layers_with_their_own_triggers():
    """Two layers with different data and weights in ONE graph: per token the decode step of layer 0, then of layer 1; after
    C tokens the device-positioned trigger of each.  The layers' counters, tickets and keep lists must not mix."""
    b = _binding()
    C_, W, n_replays, n_layers = 16, 32, 3, 2
    n0 = W + 2 * C_
    wl = wlm.Workload("graph2", B=2, H=4, n=n0 + n_replays * C_, C=C_, W=W, d_g=256, agg="mean", key_offset_std=0.5, seed=640,
                      n_layers=n_layers)
    pbs = [hz.Problem(wl.small(seed=wl.seed + L), layer=L) for L in range(n_layers)]
    S = wl.S
    st = make_store(wl, n_layers=n_layers)
    lws = [b.LstmWeights(pb.lstm) for pb in pbs]
    for L, pb in enumerate(pbs):
        st.append(L, b.bits_to_bf16(np.ascontiguousarray(pb.K[:, :n0])), b.bits_to_bf16(np.ascontiguousarray(pb.V[:, :n0])))
        st.refresh(L, None, lws[L], pb.tau)
    k_in = torch.zeros((n_layers, C_, S, 128), dtype=torch.bfloat16, device="cuda")
    v_in, q_in, out = torch.zeros_like(k_in), torch.zeros_like(k_in), torch.zeros_like(k_in)
    graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for i in range(C_):
                for L in range(n_layers):
                    st.decode_step(L, k_in[L, i], v_in[L, i], q_in[L, i], out[L, i], n_reserve=n_replays * C_)
            for L in range(n_layers):
                st.refresh_next(L, None, lws[L], pbs[L].tau)
    torch.cuda.current_stream().wait_stream(side)
    for L in range(n_layers):
        st.adopt_device_state(L)
    n, nc = n0, 2
    for rep in range(n_replays):
        qs = [[wlm.gen_q(wl, L, 100 * rep + i) for i in range(C_)] for L in range(n_layers)]
        for L, pb in enumerate(pbs):
            k_in[L].copy_(b.bits_to_bf16(np.ascontiguousarray(pb.K[:, n:n + C_].transpose(1, 0, 2))))
            v_in[L].copy_(b.bits_to_bf16(np.ascontiguousarray(pb.V[:, n:n + C_].transpose(1, 0, 2))))
            q_in[L].copy_(b.bits_to_bf16(np.stack(qs[L])))
        graph.replay()
        torch.cuda.synchronize()
        assert st.poll_status() == 0
        for L, pb in enumerate(pbs):
            idx, cnt = pb.o64.compact(pb.sc64, nc, pb.tau)
            i = C_ - 1
            want = pb.o64.attn(qs[L][i], np.ascontiguousarray(pb.K[:, :n + i + 1]), np.ascontiguousarray(pb.V[:, :n + i + 1]), C_, nc,
                               idx, cnt, pb.sm64["ksum_b16"], pb.sm64["vsum_b16"], hz.ATT["summary"], hz.SCALE)[0]
            hz.check_output(b.bf16_to_bits(out[L, i]), want, f"layer {L}, replay {rep}")
            idx1, cnt1 = pb.o64.compact(pb.sc64, nc + 1, pb.tau)
            assert np.abs(st.scores[L, :, :nc + 1].cpu().numpy() - pb.sc64[:, :nc + 1]).max() <= 2e-4
            assert np.array_equal(st.keep_cnt[L].cpu().numpy(), cnt1)
            assert np.array_equal(st.keep_idx[L, :, :nc + 1].cpu().numpy(), idx1[:, :nc + 1])
        n += C_
        nc += 1
    for L in range(n_layers):
        st.adopt_device_state(L)
        assert st.layer_state(L) == dict(n_tokens=n, n_summarised=nc, n_gated=nc, n_compacted=nc)
    assert n == wl.n and nc == pbs[0].Nc


# ---- Sec. 3.3 memory reduction: pages of gated chunks handed back ---------------------------------
@pytest.mark.parametrize("attend,mode", [("summary", "discarded"), ("summary", "gated"), ("raw", "discarded")])
def test_reclaim_pages_matches_oracle_and_leaves_attention_unchanged(attend, mode):
    b = _binding()
    wl = wlm.CFG2.small(B=2, H=8, n=2048 + 37, W=256, seed=21)       # ragged tail, MLP aggregator, 16 sequences
    st, pb, agg_w, lstm_w = full_check(wl, attend)
    q = b.bits_to_bf16(wlm.gen_q(wl, 0, 7))
    before = b.bf16_to_bits(st.decode_attn(0, q))
    table0 = st.page_table[0].cpu().numpy().copy()
    want_table = table0.copy()
    want_free = pb.o32.reclaim(want_table, pb.sc32.astype(np.float32), 0, pb.Nc, pb.tau, 0 if mode == "discarded" else 1)
    # the f64 oracle takes the same decisions (scores keep their margin from tau)
    t64 = table0.copy()
    assert np.array_equal(pb.o64.reclaim(t64, pb.sc64, 0, pb.Nc, pb.tau, 0 if mode == "discarded" else 1), want_free)
    free, cnt = st.reclaim_pages(0, 0, pb.Nc, mode)
    torch.cuda.synchronize()
    assert st.poll_status() == 0
    n_free = int(cnt.item())
    assert n_free == len(want_free)
    assert np.array_equal(free[:n_free].cpu().numpy(), want_free)                  # bit-exact, same order
    assert np.array_equal(st.page_table[0].cpu().numpy(), want_table)
    if mode == "gated":
        assert n_free == st.S * pb.Nc                                               # n / (W + M): only summaries and the window remain
    # attention never needed those pages
    after = b.bf16_to_bits(st.decode_attn(0, q))
    torch.cuda.synchronize()
    assert st.poll_status() == 0 and np.array_equal(before, after)
    # a second call finds nothing; the dense baseline now runs into the holes and says so without faulting
    _, cnt2 = st.reclaim_pages(0, 0, pb.Nc, mode)
    torch.cuda.synchronize()
    assert int(cnt2.item()) == 0
    if n_free:
        st.decode_attn_dense(0, q)
        torch.cuda.synchronize()
        assert st.poll_status() == -3


def test_reclaim_pages_host_errors_and_overflow():
    b = _binding()
    wl = wlm.CFG1.small(B=1, H=4, n=1024, seed=3)
    st, pb, _, lstm_w = full_check(wl, "raw")
    with pytest.raises(b.KveError) as e:
        st.reclaim_pages(0, 0, pb.Nc, "gated")                  # RAW attention still reads kept pages
    assert e.value.rc == -4
    with pytest.raises(b.KveError) as e:
        st.reclaim_pages(0, 0, pb.Nc + 1, "discarded")          # beyond the keep list
    assert e.value.rc == -4
    table0 = st.page_table[0].clone()
    n_disc = int(st.S * pb.Nc - st.keep_cnt[0].sum().item())
    assert n_disc > 1
    small = torch.empty((n_disc - 1,), dtype=torch.int32, device="cuda")
    _, cnt = st.reclaim_pages(0, 0, pb.Nc, "discarded", free_list=small)
    torch.cuda.synchronize()
    assert int(cnt.item()) == 0 and torch.equal(st.page_table[0], table0)          # nothing handed back
    assert st.poll_status() == -3
    _, cnt = st.reclaim_pages(0, 0, 0, "discarded")             # empty range
    torch.cuda.synchronize()
    assert int(cnt.item()) == 0 and st.poll_status() == 0


def test_compact_topk_beyond_the_staged_range():
    """More gated chunks per sequence than the top-k kernel stages in shared memory (2048): the ranking then walks the
    scores in global memory.  Chunks of one token keep the case small; the list must equal the oracle's ranking of the
    same fp32 scores bit for bit, and attention over it the oracle's."""
    b = _binding()
    wl = wlm.Workload("topk_long", B=1, H=3, n=2300 + 40, C=1, W=40, d_g=64, agg="identity", seed=17, tau=0.0)
    pb = hz.Problem(wl, keep=None, tau=0.0, margin_eps=0.0)
    assert pb.Nc == 2300
    st = make_store(wl)
    load_kv(st, 0, pb.K, pb.V)
    lw = b.LstmWeights(pb.lstm)
    st.summarize_chunks(0, 0, pb.Nc)
    st.gate(0, 0, pb.Nc, lw)
    sc_gpu = st.scores[0].cpu().numpy()
    for k in (1, 700, 2299):
        st.compact_topk(0, k)
        torch.cuda.synchronize()
        assert st.poll_status() == 0
        want_idx, want_cnt = pb.o32.compact_topk(sc_gpu.astype(np.float32), pb.Nc, k)
        assert np.array_equal(st.keep_cnt[0].cpu().numpy(), want_cnt)
        assert np.array_equal(st.keep_idx[0].cpu().numpy(), want_idx)
    st.compact_topk(0, 700)
    q = wlm.gen_q(wl, 0, 1)
    out = st.decode_attn(0, b.bits_to_bf16(q))
    torch.cuda.synchronize()
    assert st.poll_status() == 0
    idx, cnt = st.keep_idx[0].cpu().numpy(), st.keep_cnt[0].cpu().numpy()
    want = pb.o64.attn(q, pb.K, pb.V, wl.C, pb.Nc, idx, cnt, pb.sm64["ksum_b16"], pb.sm64["vsum_b16"], hz.ATT["summary"], hz.SCALE)[0]
    hz.check_output(b.bf16_to_bits(out), want, "attn after a long top-k")


# ---- gating variant: top-k retention ---------------------------------------------------------------
@pytest.mark.parametrize("attend", ["summary", "raw"])
def test_compact_topk_matches_oracle_and_feeds_attention(attend):
    b = _binding()
    wl = wlm.CFG2.small(B=2, H=8, n=3000, W=256, seed=31)            # 42 gated chunks, ragged tail
    st, pb, _, _ = full_check(wl, attend)
    Nc = pb.Nc
    sc_gpu = st.scores[0].cpu().numpy()                               # the ranking is an integer function of these floats
    for k in (0, 1, 13, Nc - 1, Nc, Nc + 9):
        st.compact_topk(0, k)
        torch.cuda.synchronize()
        assert st.poll_status() == 0
        want_idx, want_cnt = pb.o32.compact_topk(sc_gpu.astype(np.float32), Nc, k)
        assert np.array_equal(st.keep_cnt[0].cpu().numpy(), want_cnt)
        assert np.array_equal(st.keep_idx[0].cpu().numpy(), want_idx)                # bit-exact
        # and, where the k-th and (k+1)-th oracle scores are clearly apart, the same list as the oracle's own scores give
        o_idx, o_cnt = pb.o64.compact_topk(pb.sc64, Nc, k)
        srt = -np.sort(-pb.sc64[:, :Nc], axis=1)
        clear = np.ones(st.S, bool) if (k <= 0 or k >= Nc) else (srt[:, k - 1] - srt[:, k] > 1e-3)
        assert clear.any()
        assert np.array_equal(st.keep_idx[0].cpu().numpy()[clear], o_idx[clear])
    # attention over a top-k list: the oracle's attention with that list
    k = 13
    st.compact_topk(0, k)
    q = wlm.gen_q(wl, 0, 3)
    out = st.decode_attn(0, b.bits_to_bf16(q))
    torch.cuda.synchronize()
    assert st.poll_status() == 0
    idx, cnt = st.keep_idx[0].cpu().numpy(), st.keep_cnt[0].cpu().numpy()
    want = pb.o64.attn(q, pb.K, pb.V, wl.C, Nc, idx, cnt, pb.sm64["ksum_b16"], pb.sm64["vsum_b16"], hz.ATT[attend], hz.SCALE)[0]
    hz.check_output(b.bf16_to_bits(out), want, f"attn after top-k/{attend}")
    # "discarded" has no meaning without a threshold
    with pytest.raises(b.KveError) as e:
        st.reclaim_pages(0, 0, Nc, "discarded")
    assert e.value.rc == -4


# ---- "pooling" aggregator: element-wise maximum ---------------------------------------------------------
@pytest.mark.parametrize("C", [32, 64])
def test_max_pool_aggregator_full_pipeline(C):
    wl = wlm.CFG1.small(B=2, H=4, n=1500, C=C, W=256, agg="max", seed=17)      # ragged tail; summaries must be bit-exact
    full_check(wl, "summary")


@pytest.mark.parametrize("C,d_sum", [(32, 128), (64, 256), (128, 256), (256, 128)])
def test_token_mlp_aggregator_full_pipeline(C, d_sum):
    """Eq. 2 taken literally (the MLP on every token, outputs mean-pooled): tiles of several chunks (C < 128), of one
    chunk, and chunks of two tiles (C = 256); ragged tail; the whole path behind it against the oracle."""
    wl = wlm.CFG2.small(B=2, H=3, n=C * 9 + 5, C=C, W=2 * C, agg="token_mlp", d_sum=d_sum, seed=60 + C)
    st, pb, aw, lw = full_check(wl, "summary")
    assert pb.Nc == 7


def test_token_mlp_aggregator_incremental_ranges_and_unsupported_geometry():
    b = _binding()
    wl = wlm.CFG2.small(B=1, H=5, n=64 * 11, C=64, W=128, agg="token_mlp", d_sum=256, seed=71)
    pb = hz.Problem(wl)
    st = make_store(wl)
    load_kv(st, 0, pb.K, pb.V)
    aw, lw = b.AggWeights(pb.mlp), b.LstmWeights(pb.lstm)
    for lo, hi in ((0, 3), (3, 4), (4, pb.Nc)):          # an odd number of chunks per call: half-filled tiles
        st.summarize_chunks(0, lo, hi, aw)
    st.gate(0, 0, pb.Nc, lw)
    st.compact(0, pb.tau)
    torch.cuda.synchronize()
    assert st.poll_status() == 0
    check_summaries(st, pb)
    check_gate_and_keep(st, pb)
    with pytest.raises(b.KveError) as e:                  # chunk sizes the tensor-core tiling does not cover are refused at create
        b.Store(B=1, H=1, C_=48, W=48, max_tokens=480, d_g=64, agg="token_mlp", d_sum=256)
    assert e.value.rc == -2
    with pytest.raises(b.KveError) as e:
        b.Store(B=1, H=1, C_=64, W=64, max_tokens=640, d_g=64, agg="token_mlp", d_sum=192)
    assert e.value.rc == -2


def test_decode_tick_replays_from_a_cuda_graph():
    """append + gated attention of two layers captured once and replayed: the calls neither synchronise nor
    allocate, so the replay must reproduce the eager outputs bit for bit (and the oracle's within tolerance)."""
    b = _binding()
    wl = wlm.CFG1.small(B=2, H=4, n=1500, seed=41)
    st = make_store(wl, n_layers=2)
    pbs = [hz.Problem(wl, layer=L) for L in range(2)]
    for L, pb in enumerate(pbs):
        load_kv(st, L, pb.K[:, :-1], pb.V[:, :-1])
        Nc = wl.n_stale_chunks(wl.n - 1)
        st.summarize_chunks(L, 0, Nc, None)
        st.gate(L, 0, Nc, b.LstmWeights(pb.lstm))
        st.compact(L, pb.tau)
    qs = [b.bits_to_bf16(wlm.gen_q(wl, L, 9)) for L in range(2)]
    kn = [b.bits_to_bf16(pb.K[:, -1:]) for pb in pbs]
    vn = [b.bits_to_bf16(pb.V[:, -1:]) for pb in pbs]
    out = torch.zeros((2, st.S, 128), dtype=torch.bfloat16, device="cuda")

    def tick():
        for L in range(2):
            st.set_len(L, wl.n - 1)
            st.append(L, kn[L], vn[L])
            st.decode_attn(L, qs[L], out[L])

    tick()
    torch.cuda.synchronize()
    eager = out.clone()
    side, graph = torch.cuda.Stream(), torch.cuda.CUDAGraph()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            tick()
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(2):
        out.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(out, eager)
    assert st.poll_status() == 0
    for L, pb in enumerate(pbs):
        Nc = wl.n_stale_chunks(wl.n - 1)
        want, _, _, _ = pb.o64.attn(wlm.gen_q(wl, L, 9), pb.K, pb.V, wl.C, Nc, pb.idx64, pb.cnt64, pb.sm64["ksum_b16"],
                                    pb.sm64["vsum_b16"], hz.ATT["summary"], hz.SCALE)
        hz.check_output(b.bf16_to_bits(out[L]), want, f"graph replay, layer {L}")


def test_decode_loop_advances_under_a_cuda_graph():
    """kvE_append_next + gated attention captured ONCE; every replay appends the next token at the
    device-held length and attends over the grown cache.  Each step against the oracle on the cache
    as it then stands; afterwards the host is told the length and gates the chunk that completed."""
    b = _binding()
    wl = wlm.CFG1.small(B=2, H=4, n=1530, C=64, W=256, seed=43, n_append=16)   # the loop crosses a chunk boundary
    st = make_store(wl)
    pb = hz.Problem(wl)
    load_kv(st, 0, pb.K, pb.V)
    aw, lw = None, b.LstmWeights(pb.lstm)
    run_gpu_pipeline(st, pb, 0, aw, lw)
    steps = 12
    k_in = torch.zeros((st.S, 128), dtype=torch.bfloat16, device="cuda")
    v_in, q_in = torch.zeros_like(k_in), torch.zeros_like(k_in)
    out = torch.zeros_like(k_in)
    side, graph = torch.cuda.Stream(), torch.cuda.CUDAGraph()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            st.append_next(0, k_in, v_in, n_reserve=steps)
            st.decode_attn(0, q_in, out)
    torch.cuda.current_stream().wait_stream(side)
    K, V = pb.K, pb.V
    for step in range(steps):
        kn, vn = wlm.gen_new_tokens(wl, 0, step)
        q = wlm.gen_q(wl, 0, 50 + step)
        k_in.copy_(b.bits_to_bf16(kn[:, 0])); v_in.copy_(b.bits_to_bf16(vn[:, 0])); q_in.copy_(b.bits_to_bf16(q))
        graph.replay()
        torch.cuda.synchronize()
        assert st.poll_status() == 0
        K, V = np.concatenate([K, kn], axis=1), np.concatenate([V, vn], axis=1)
        assert int(st.seq_len[0, 0]) == wl.n + step + 1
        want, _, _, n_eff = pb.oracle_attn(q, "summary", "f64", K, V, pb.Nc)
        hz.check_output(b.bf16_to_bits(out), want, f"graph loop, step {step}")
    Kd, Vd = pages_to_plain(st, 0, wl.n + steps)
    assert np.array_equal(Kd, K) and np.array_equal(Vd, V)          # every token landed at its own position
    # back on the host: the true length, then the chunk that has left the window meanwhile
    st.set_len(0, wl.n + steps)
    nc = (wl.n + steps - wl.W) // wl.C
    assert nc == pb.Nc + 1
    st.summarize_chunks(0, pb.Nc, nc, aw)
    st.gate(0, pb.Nc, nc, lw)
    torch.cuda.synchronize()
    assert st.poll_status() == 0
    # a single-query attention launch is cut into pieces on the device from the length it finds there, so a replay far
    # beyond the growth that was announced (n_reserve = 0) still attends to every row
    wl2 = wlm.CFG1.small(B=1, H=2, n=300, C=64, W=64, seed=44, n_append=400)
    st2 = make_store(wl2)
    pb2 = hz.Problem(wl2)
    load_kv(st2, 0, pb2.K, pb2.V)
    run_gpu_pipeline(st2, pb2, 0, None, b.LstmWeights(pb2.lstm))
    z = torch.zeros((st2.S, 128), dtype=torch.bfloat16, device="cuda")
    q2 = wlm.gen_q(wl2, 0, 9)
    q2d, out2 = b.bits_to_bf16(q2), torch.empty_like(z)
    g2 = torch.cuda.CUDAGraph()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(g2, stream=side):
            st2.append_next(0, z, z, n_reserve=0)
            st2.decode_attn(0, q2d, out2)
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(200):
        g2.replay()
    torch.cuda.synchronize()
    assert st2.poll_status() == 0 and int(st2.seq_len[0, 0]) == wl2.n + 200
    pad = np.zeros((st2.S, 200, 128), np.uint16)
    want, _, _, _ = pb2.oracle_attn(q2, "summary", "f64", np.concatenate([pb2.K, pad], axis=1), np.concatenate([pb2.V, pad], axis=1), pb2.Nc)
    hz.check_output(b.bf16_to_bits(out2), want, "replayed 200 tokens past the announced growth")
    # the cache is full after 400 appended tokens: further replays are refused on the device, nothing is overwritten
    for _ in range(201):
        g2.replay()
    torch.cuda.synchronize()
    assert st2.poll_status() == -3 and int(st2.seq_len[0, 0]) == wl2.n + 400


@pytest.mark.parametrize("attend", ["summary", "raw"])
def test_decode_step_appends_and_attends_in_one_launch(attend):
    """kvE_decode_step = append one token at the device-held length + gated attention over the cache with it, one launch:
    against the oracle on the growing cache, byte-exact pages, across a page boundary, and replayed from a CUDA graph."""
    b = _binding()
    steps = 40
    wl = wlm.CFG3.small(B=2, H=4, n_layers=1, n=64 + 2 * 256 + 50, n_append=steps + 2, seed=55)      # 50 rows into a page: crosses at step 14
    pb = hz.Problem(wl)
    st = make_store(wl, attend)
    aw, lw = b.AggWeights(pb.mlp), b.LstmWeights(pb.lstm)
    load_kv(st, 0, pb.K, pb.V)
    run_gpu_pipeline(st, pb, 0, aw, lw)
    S = st.S
    k_in = torch.zeros((S, 128), dtype=torch.bfloat16, device="cuda")
    v_in, q_in, out = torch.zeros_like(k_in), torch.zeros_like(k_in), torch.zeros_like(k_in)
    lse = torch.zeros(S, dtype=torch.float32, device="cuda")
    K, V = pb.K, pb.V
    graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    for step in range(steps):
        kn, vn = wlm.gen_new_tokens(wl, 0, step)
        q = wlm.gen_q(wl, 0, step)
        k_in.copy_(b.bits_to_bf16(kn[:, 0])); v_in.copy_(b.bits_to_bf16(vn[:, 0])); q_in.copy_(b.bits_to_bf16(q))
        if step < 3:                                   # issued directly
            st.decode_step(0, k_in, v_in, q_in, out, lse=lse, n_reserve=steps)
        else:
            if step == 3:                              # then captured once and replayed
                side.wait_stream(torch.cuda.current_stream())
                with torch.cuda.stream(side):
                    with torch.cuda.graph(graph, stream=side):
                        st.decode_step(0, k_in, v_in, q_in, out, lse=lse, n_reserve=steps)
                torch.cuda.current_stream().wait_stream(side)
            graph.replay()
        torch.cuda.synchronize()
        assert st.poll_status() == 0
        K, V = np.concatenate([K, kn], axis=1), np.concatenate([V, vn], axis=1)
        assert int(st.seq_len[0, 0]) == wl.n + step + 1
        want, _, want_lse, _ = pb.oracle_attn(q, attend, "f64", K, V, pb.Nc)
        hz.check_output(b.bf16_to_bits(out), want, f"decode_step {attend}, step {step}")
        assert np.abs(lse.cpu().numpy() - want_lse).max() <= 1e-3
    Kd, Vd = pages_to_plain(st, 0, wl.n + steps)
    assert np.array_equal(Kd, K) and np.array_equal(Vd, V)          # every token landed at its own position
    # the same tokens through kvE_append_next + kvE_decode_attn on a second handle: same outputs bit for bit
    st2 = make_store(wl, attend)
    load_kv(st2, 0, pb.K, pb.V)
    run_gpu_pipeline(st2, pb, 0, aw, lw)
    for step in range(steps):
        kn, vn = wlm.gen_new_tokens(wl, 0, step)
        st2.append_next(0, b.bits_to_bf16(kn[:, 0]), b.bits_to_bf16(vn[:, 0]), n_reserve=steps)
        out2 = st2.decode_attn(0, b.bits_to_bf16(wlm.gen_q(wl, 0, step)))
    torch.cuda.synchronize()
    assert torch.equal(out2, out)
    # a full cache: the call is refused on the host once the handle's own count is at the limit
    st.set_len(0, wl.max_tokens)
    with pytest.raises(b.KveError) as e:
        st.decode_step(0, k_in, v_in, q_in, out)
    assert e.value.rc == -3


@pytest.mark.parametrize("seed", list(range(12)) + [104])      # 104: nothing has left the window yet
def test_whole_path_random_geometries(seed):
    """Seeded random small geometries (chunk size, window, length, gate width, aggregator, keep ratio, append
    pattern) through append, summaries, gate, keep list and both attentions against the oracle."""
    rng = np.random.default_rng(2000 + seed)
    C = int(rng.choice([1, 3, 8, 16, 50, 64, 128]))
    agg = "identity" if C == 1 else str(rng.choice(["mean", "mlp", "max"]))
    W = int(rng.integers(0, 3 * C + 2))
    n = int(rng.integers(1, 1200 if C > 1 else 300))
    d_sum = int(rng.choice([8, 64, 200, 256])) if agg == "mlp" else 0
    wl = wlm.CFG1.small(B=int(rng.integers(1, 4)), H=int(rng.integers(1, 5)), n=n, C=C, W=W, d_g=int(rng.choice([64, 128, 256])),
                        agg=agg, d_sum=d_sum, seed=60 + seed)
    pieces = tuple(sorted(rng.random(int(rng.integers(0, 3))).tolist())) + (1.0,)
    full_check(wl, str(rng.choice(["summary", "raw"])), pieces=pieces, keep=float(rng.choice([0.25, 0.5, 0.75])))
