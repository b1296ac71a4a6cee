"""GPU parity of kvE_decode_attn_block (query blocks: several query tokens on grouped query heads)
against the oracle, which treats every (token, query head) pair as one independent query of Eq. 1."""
import numpy as np
import pytest
import torch

from paper_2509_21354_b200 import workloads as wlm
from tests import harness as hz

pytestmark = pytest.mark.gpu


def _prepared(wl, attend, G, T, n_layers=1, layer=0):
    from paper_2509_21354_b200 import binding as b
    pb = hz.Problem(wl, layer=layer)
    st = b.Store(B=wl.B, H=wl.H, Hq=wl.H * G, C_=wl.C, W=wl.W, max_tokens=wl.max_tokens, d_g=wl.d_g, agg=wl.agg,
                 d_sum=wl.d_sum, attend=attend, page_perm="random", seed=3, n_layers=n_layers, max_query_tokens=T)
    st.append(layer, b.bits_to_bf16(pb.K), b.bits_to_bf16(pb.V))
    if pb.Nc > 0:
        st.summarize_chunks(layer, 0, pb.Nc, b.AggWeights(pb.mlp) if pb.mlp is not None else None)
        st.gate(layer, 0, pb.Nc, b.LstmWeights(pb.lstm))
        st.compact(layer, pb.tau)
    torch.cuda.synchronize()
    assert st.poll_status() == 0
    return b, pb, st


def _check(b, pb, st, attend, G, T, layer=0, dense=False, step=0, causal=False):
    wl = pb.wl
    q = wlm.gen_q_block(wl, T, wl.H * G, layer, step)
    lse = torch.full((wl.B, T, wl.H * G), float("nan"), dtype=torch.float32, device="cuda")
    out = st.decode_attn_block(layer, b.bits_to_bf16(q), dense=dense, lse=lse, causal=causal)
    torch.cuda.synchronize()
    assert st.poll_status() == 0
    args = (wl.C, pb.Nc, pb.idx64, pb.cnt64, pb.sm64["ksum_b16"])
    want, _, want_lse = pb.o64.attn_block(q, wl.H, pb.K, pb.V, *args, pb.sm64["vsum_b16"], hz.ATT[attend], hz.SCALE, dense=dense,
                                          causal=causal)
    # the same attention over |V|: the scale of the rounding error of bf16 softmax numerators
    spread, _, _ = pb.o64.attn_block(q, wl.H, pb.K, pb.V & 0x7FFF, *args, pb.sm64["vsum_b16"] & 0x7FFF, hz.ATT[attend],
                                     hz.SCALE, dense=dense, causal=causal)
    hz.check_output_bf16_weights(b.bf16_to_bits(out), want, spread, f"block/{attend}/G{G}T{T}")
    assert np.abs(lse.cpu().numpy() - want_lse).max() <= 1e-3
    return out


# (G query heads per KV head, T query tokens): 1..128 query rows per KV head; up to 32, 64 and 128 rows the
# kernel lays the block out four times, twice and once over its 128 accumulator rows
@pytest.mark.parametrize("G,T", [(1, 1), (4, 3), (4, 7), (2, 20), (8, 8), (1, 33), (8, 12), (4, 32)])
@pytest.mark.parametrize("attend", ["summary", "raw"])
def test_block_attention_matches_oracle(attend, G, T):
    # two KV sequences: many splits per sequence; ragged tail (n not a multiple of 8)
    wl = wlm.CFG1.small(B=1, H=2, n=2443, W=300, seed=21)
    b, pb, st = _prepared(wl, attend, G, T)
    _check(b, pb, st, attend, G, T)
    _check(b, pb, st, attend, G, T, dense=True, step=1)


@pytest.mark.parametrize("C,n", [(32, 1500), (24, 1000), (128, 3001), (8, 700)])
def test_block_attention_chunk_sizes_and_page_boxes(C, n):
    # C = 32: boxes of 32 rows; 24 and 8: boxes of 8; 128: half pages
    wl = wlm.CFG1.small(B=2, H=3, n=n, C=C, W=3 * C + 5, seed=22)
    for attend in ("summary", "raw"):
        b, pb, st = _prepared(wl, attend, 4, 7)
        _check(b, pb, st, attend, 4, 7)
        _check(b, pb, st, attend, 4, 7, dense=True)


def test_block_attention_many_sequences_single_split_and_second_layer():
    # 160 KV sequences (more than one per SM: no splits), layer 1 of 2 (summary rows of another layer)
    wl = wlm.CFG1.small(B=20, H=8, n=900, W=128, seed=23)
    b, pb, st = _prepared(wl, "summary", 4, 7, n_layers=2, layer=1)
    _check(b, pb, st, "summary", 4, 7, layer=1)


def test_block_attention_short_and_empty_caches():
    from paper_2509_21354_b200 import binding as b
    wl = wlm.CFG1.small(B=2, H=2, n=50, W=256, seed=24)      # nothing has left the window: raw tail only
    bb, pb, st = _prepared(wl, "summary", 4, 7)
    assert pb.Nc == 0
    _check(bb, pb, st, "summary", 4, 7)
    st.set_len(0, 0)                                          # empty cache: zeros out, lse = -inf
    q = b.bits_to_bf16(wlm.gen_q_block(wl, 7, 8))
    lse = torch.zeros((2, 7, 8), dtype=torch.float32, device="cuda")
    out = st.decode_attn_block(0, q, lse=lse)
    torch.cuda.synchronize()
    assert st.poll_status() == 0
    assert torch.all(out == 0) and torch.all(torch.isinf(lse) & (lse < 0))


def test_block_of_one_row_agrees_with_the_single_query_kernel():
    wl = wlm.CFG1.small(B=2, H=4, n=3000, seed=25)
    b, pb, st = _prepared(wl, "summary", 1, 1)
    q = wlm.gen_q(wl, 0, 5)
    one = st.decode_attn(0, b.bits_to_bf16(q))
    blk = st.decode_attn_block(0, b.bits_to_bf16(q.reshape(wl.B, 1, wl.H, 128)))
    torch.cuda.synchronize()
    one_b, blk_b = b.bf16_to_bits(one).reshape(-1), b.bf16_to_bits(blk).reshape(-1)
    # the block kernel rounds the softmax numerators to bf16, the single-query kernel does not: the two agree
    # within that rounding (2^-8 of the typical |v| ~ 1, in practice far less) plus one bf16 step of the result
    x, y = wlm.bf16_bits_to_f32(one_b).astype(np.float64), wlm.bf16_bits_to_f32(blk_b).astype(np.float64)
    assert np.all(np.abs(x - y) <= 2.0 ** -7 * np.abs(x) + 2.0 ** -9)
    assert np.abs(x - y).mean() <= 2e-4


def test_block_attention_argument_checks():
    from paper_2509_21354_b200 import binding as b
    wl = wlm.CFG1.small(B=1, H=2, n=600, seed=26)
    with pytest.raises(b.KveError):                            # 17 tokens x 8 heads per KV head > 128 query rows
        b.Store(B=1, H=2, Hq=16, C_=64, W=256, max_tokens=1024, d_g=128, max_query_tokens=17)
    with pytest.raises(b.KveError):                            # chunk size without a box of at least 8 rows
        b.Store(B=1, H=2, Hq=8, C_=20, W=256, max_tokens=1024, d_g=128, max_query_tokens=4)
    st = b.Store(B=1, H=2, Hq=8, C_=64, W=256, max_tokens=1024, d_g=128, max_query_tokens=4)
    q = torch.zeros((1, 5, 8, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(b.KveError) as err:
        st.decode_attn_block(0, q)
    assert err.value.rc == -3
    with pytest.raises(b.KveError) as err:                     # grouped heads: the single-query entry points refuse
        st.decode_attn(0, torch.zeros((2, 128), dtype=torch.bfloat16, device="cuda"))
    assert err.value.rc == -2
    st0 = b.Store(B=1, H=2, C_=64, W=256, max_tokens=1024, d_g=128)
    with pytest.raises(b.KveError) as err:                     # not enabled at create
        st0.decode_attn_block(0, torch.zeros((1, 1, 2, 128), dtype=torch.bfloat16, device="cuda"))
    assert err.value.rc == -4


def test_block_attention_growing_maxima_force_rescales():
    """Keys grow in magnitude along the order the kernel walks the rows (raw tail oldest to newest, then
    the kept chunks), so the running row maximum keeps climbing by far more than the slack the
    kernel allows before it rescales its accumulator; peaked rows (one dominant key) ride along."""
    from paper_2509_21354_b200 import binding as b
    wl = wlm.CFG1.small(B=1, H=2, n=1500, W=700, C=64, seed=27)
    pb = hz.Problem(wl)
    K = pb.K.copy()
    kf = wlm.bf16_bits_to_f32(K)
    ramp = np.ones(wl.n, np.float32)
    tail0 = pb.Nc * wl.C
    ramp[tail0:] = np.linspace(0.5, 12.0, wl.n - tail0)      # logits of the newest rows ~ N(0, 12^2)
    ramp[:tail0] = 20.0                                      # kept chunks (walked last) larger still
    pb.K = wlm.f32_to_bf16_bits(kf * ramp[None, :, None])
    for attend in ("raw", "summary"):
        st = b.Store(B=wl.B, H=wl.H, Hq=wl.H * 4, C_=wl.C, W=wl.W, max_tokens=wl.max_tokens, d_g=wl.d_g, agg=wl.agg,
                     attend=attend, page_perm="random", seed=3, max_query_tokens=7)
        st.append(0, b.bits_to_bf16(pb.K), b.bits_to_bf16(pb.V))
        # summaries, scores and the keep list of the modified keys, through the oracle's own steps
        sm = pb.o64.summarize(pb.K, pb.V, wl.C, 0, pb.Nc, pb.agg, pb.mlp, stride=wl.max_chunks)
        rng = np.random.default_rng(4)
        idx, cnt = pb.o64.compact(rng.uniform(size=(wl.S, wl.max_chunks)), pb.Nc, 0.5)
        st.summarize_chunks(0, 0, pb.Nc, None)
        st.gate(0, 0, pb.Nc, b.LstmWeights(pb.lstm))
        st.compact(0, pb.tau)
        st.keep_idx[0].copy_(torch.from_numpy(idx).cuda())
        st.keep_cnt[0].copy_(torch.from_numpy(cnt).cuda())
        torch.cuda.synchronize()
        q = wlm.gen_q_block(wl, 7, wl.H * 4, 0, 3)
        lse = torch.zeros((wl.B, 7, wl.H * 4), dtype=torch.float32, device="cuda")
        out = st.decode_attn_block(0, b.bits_to_bf16(q), lse=lse)
        torch.cuda.synchronize()
        assert st.poll_status() == 0
        want, _, want_lse = pb.o64.attn_block(q, wl.H, pb.K, pb.V, wl.C, pb.Nc, idx, cnt, sm["ksum_b16"], sm["vsum_b16"],
                                              hz.ATT[attend], hz.SCALE)
        spread, _, _ = pb.o64.attn_block(q, wl.H, pb.K, pb.V & 0x7FFF, wl.C, pb.Nc, idx, cnt, sm["ksum_b16"],
                                         sm["vsum_b16"] & 0x7FFF, hz.ATT[attend], hz.SCALE)
        assert np.ptp(want_lse) > 20                          # the rows really are far apart / peaked
        hz.check_output_bf16_weights(b.bf16_to_bits(out), want, spread, f"block/{attend}/growing maxima")
        assert np.abs(lse.cpu().numpy() - want_lse).max() <= 1e-3 * np.abs(want_lse).max()


def test_block_attention_at_the_benchmarked_size():
    """The geometry bench.py times for query blocks: cfg2 with 8 KV heads (64 KV sequences, n = 4096,
    C = 64, W = 512), 4 query heads per KV head, 7 query tokens; every output against the oracle."""
    wl = wlm.CFG2.small(H=8)
    b, pb, st = _prepared(wl, "summary", 4, 7)
    assert 0.4 < pb.cnt64.mean() / pb.Nc < 0.6
    _check(b, pb, st, "summary", 4, 7)
    _check(b, pb, st, "summary", 4, 7, dense=True, step=1)


def test_action_token_loop_replays_from_a_cuda_graph():
    """One control step = append the 7 new tokens of every KV head, then attend with the 7 query tokens
    on all query heads: captured once, replayed three times, each step against the oracle on the cache
    as it then stands."""
    wl = wlm.CFG1.small(B=2, H=2, n=1200, C=64, W=256, seed=29, n_append=40)
    G, T, steps = 4, 7, 3
    b, pb, st = _prepared(wl, "summary", G, T)
    k_in = torch.zeros((st.S, T, 128), dtype=torch.bfloat16, device="cuda")
    v_in = torch.zeros_like(k_in)
    q_in = torch.zeros((wl.B, T, wl.H * G, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros_like(q_in)
    side, graph = torch.cuda.Stream(), torch.cuda.CUDAGraph()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            st.append_next(0, k_in, v_in, n_reserve=(steps - 1) * T)
            st.decode_attn_block(0, q_in, out=out)
    torch.cuda.current_stream().wait_stream(side)
    K, V = pb.K, pb.V
    for step in range(steps):
        kn, vn = wlm.gen_new_tokens(wl, 0, step, n_new=T)
        q = wlm.gen_q_block(wl, T, wl.H * G, 0, 10 + step)
        k_in.copy_(b.bits_to_bf16(kn)); v_in.copy_(b.bits_to_bf16(vn)); q_in.copy_(b.bits_to_bf16(q))
        graph.replay()
        torch.cuda.synchronize()
        assert st.poll_status() == 0
        K, V = np.concatenate([K, kn], axis=1), np.concatenate([V, vn], axis=1)
        args = (wl.C, pb.Nc, pb.idx64, pb.cnt64, pb.sm64["ksum_b16"])
        want, _, _ = pb.o64.attn_block(q, wl.H, K, V, *args, pb.sm64["vsum_b16"], hz.ATT["summary"], hz.SCALE)
        spread, _, _ = pb.o64.attn_block(q, wl.H, K, V & 0x7FFF, *args, pb.sm64["vsum_b16"] & 0x7FFF, hz.ATT["summary"], hz.SCALE)
        hz.check_output_bf16_weights(b.bf16_to_bits(out), want, spread, f"action-token loop, step {step}")
    assert int(st.seq_len[0, 0]) == wl.n + steps * T


# causal blocks: the block's tokens are the newest rows of the cache and token t sees the cache up to itself
@pytest.mark.parametrize("G,T,n", [(4, 7, 2443), (1, 33, 2200), (2, 40, 1989), (4, 32, 2048 + 31)])
def test_causal_block_attention_matches_oracle(G, T, n):
    # the last T rows sit in the last tile of the raw tail, or straddle two tiles (n - raw0 just above a multiple of 64)
    wl = wlm.CFG1.small(B=1, H=2, n=n, W=300, seed=31)
    for attend in ("summary", "raw"):
        b, pb, st = _prepared(wl, attend, G, T)
        _check(b, pb, st, attend, G, T, causal=True)
        _check(b, pb, st, attend, G, T, dense=True, step=1, causal=True)


def test_causal_block_with_a_tail_shorter_than_the_block_is_refused():
    # W = 4, C = 8: the raw tail holds 4..11 rows, fewer than the 12 query tokens, so the first tokens would
    # have no position inside the raw tail (the oracle refuses that case as well): KVE_ERR_STATE, nothing runs
    wl = wlm.CFG1.small(B=1, H=2, n=203, C=8, W=4, seed=32)
    b, pb, st = _prepared(wl, "summary", 2, 12)
    tail = wl.n - pb.Nc * wl.C
    assert tail < 12
    q = b.bits_to_bf16(wlm.gen_q_block(wl, 12, 4, 0, 0))
    with pytest.raises(b.KveError) as e:
        st.decode_attn_block(0, q, causal=True)
    assert e.value.rc == -4
    # as many query tokens as the tail has rows is the limit case and is served
    T = tail
    q = wlm.gen_q_block(wl, T, 4, 0, 0)
    out = st.decode_attn_block(0, b.bits_to_bf16(q), causal=True)
    torch.cuda.synchronize()
    assert st.poll_status() == 0
    got = wlm.bf16_bits_to_f32(b.bf16_to_bits(out)).astype(np.float64)
    for t in range(T):
        n_t = wl.n - (T - 1 - t)
        for g in range(2):
            qs = np.ascontiguousarray(q[:, t, g::2, :].reshape(wl.S, 128))
            want, _, _, _ = pb.o64.attn(qs, np.ascontiguousarray(pb.K[:, :n_t]), np.ascontiguousarray(pb.V[:, :n_t]), wl.C, pb.Nc,
                                        pb.idx64, pb.cnt64, pb.sm64["ksum_b16"], pb.sm64["vsum_b16"], hz.ATT["summary"], hz.SCALE)
            assert np.abs(got[0, t, g::2] - want).max() <= 2e-2
    # the full-cache form counts all stored tokens as the tail, so 12 tokens are fine there
    st.decode_attn_block(0, b.bits_to_bf16(wlm.gen_q_block(wl, 12, 4, 0, 0)), dense=True, causal=True)
    torch.cuda.synchronize()
    assert st.poll_status() == 0


@pytest.mark.parametrize("n", [2048, 2051])
def test_block_attention_without_window_and_with_large_chunks(n):
    # W = 0 and n a multiple of C = 512: no raw row at all, the retained set is the kept chunks only
    # (summary rows, or four tiles of raw rows per kept chunk); n = 2051: a three-row tail
    wl = wlm.CFG1.small(B=1, H=3, n=n, C=512, W=0, seed=33)
    for attend in ("summary", "raw"):
        b, pb, st = _prepared(wl, attend, 4, 7)
        assert pb.Nc == 4 and 0 < pb.cnt64.sum() < 12
        _check(b, pb, st, attend, 4, 7)
        _check(b, pb, st, attend, 4, 7, dense=True, step=2)


def test_block_attention_after_the_gated_pages_were_handed_back():
    """Sec. 3.3 memory reduction: once every gated chunk's page is back on the free list, the gated query-block
    attention (summary rows + raw tail) still answers as before; the full-cache variant cannot and says so
    through the status word instead of reading a page it no longer owns."""
    wl = wlm.CFG1.small(B=1, H=2, n=1800, seed=34)
    b, pb, st = _prepared(wl, "summary", 4, 7)
    before = _check(b, pb, st, "summary", 4, 7).clone()
    free_list, free_count = st.reclaim_pages(0, 0, pb.Nc, mode="gated")
    torch.cuda.synchronize()
    assert int(free_count) == wl.S * pb.Nc and st.poll_status() == 0
    after = _check(b, pb, st, "summary", 4, 7)
    assert torch.equal(before, after)
    q = b.bits_to_bf16(wlm.gen_q_block(wl, 7, 8))
    st.decode_attn_block(0, q, dense=True)
    torch.cuda.synchronize()
    assert st.poll_status() == -3


@pytest.mark.parametrize("seed", range(16))
def test_block_attention_random_geometries(seed):
    """Seeded random small geometries (chunk size, window, length, heads, block shape, mode, causal or not)
    against the oracle: the cases nobody thought of."""
    rng = np.random.default_rng(1000 + seed)
    C = int(rng.choice([8, 16, 24, 32, 64, 128]))
    W = int(rng.integers(0, 3 * C + 1))
    G = int(rng.choice([1, 2, 4, 8]))
    T = int(rng.integers(1, 128 // G + 1)) if rng.random() < 0.3 else int(rng.integers(1, max(2, 32 // G) + 1))
    n = int(rng.integers(max(T, 1), 1500))
    attend = str(rng.choice(["summary", "raw"]))
    causal = bool(rng.random() < 0.5)
    wl = wlm.CFG1.small(B=int(rng.integers(1, 3)), H=int(rng.integers(1, 4)), n=n, C=C, W=W, seed=40 + seed)
    b, pb, st = _prepared(wl, attend, G, T)
    if causal and n - pb.Nc * C < T:
        causal = False                      # the oracle's causal form wants the block's tokens inside the raw tail
    _check(b, pb, st, attend, G, T, causal=causal)
    _check(b, pb, st, attend, G, T, dense=True, step=1, causal=causal)
