"""Pins for the oracle: each part is checked against something that is not the oracle itself —
hand-worked values (tests/golden), closed forms, brute force on tiny inputs, invariants the paper's
definitions imply, and independent library routines (torch CPU LSTM / SDPA / bf16 cast).
Runs without a GPU.
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import kvo
from paper_2509_21354_b200 import workloads as wlm

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def bits(x):
    return wlm.f32_to_bf16_bits(np.asarray(x, np.float32))


def widen(b):
    return wlm.bf16_bits_to_f32(b).astype(np.float64)


def rand_bits(rng, *shape, scale=1.0):
    return bits(rng.standard_normal(shape).astype(np.float32) * scale)


def read_golden(name):
    out = {}
    for line in open(os.path.join(GOLD, name)):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, *v = line.split()
        out[k] = [float(x) for x in v]
    return out


# ---------------------------------------------------------------- bf16 rounding
def test_bf16_rne_known_values(o64):
    # 1 + 2^-8 is a tie between 1.0 (even mantissa) and 1 + 2^-7: goes to 1.0
    assert o64.bf16_rne(1.0 + 2.0 ** -8) == 0x3F80
    # 1 + 3*2^-8 is a tie between 1+2^-7 (odd) and 1+2^-6 (even): goes up
    assert o64.bf16_rne(1.0 + 3 * 2.0 ** -8) == 0x3F82
    assert o64.bf16_rne(1.0 + 2.0 ** -8 + 2.0 ** -30) == 0x3F81      # just above the tie
    assert o64.bf16_rne(-2.5) == 0xC020
    assert o64.bf16_rne(0.0) == 0x0000
    assert o64.bf16_rne(3.0e38 * 2) == 0x7F80                        # overflow -> inf
    assert o64.bf16_widen(0x3F81) == 1.0 + 2.0 ** -7


def test_bf16_rne_matches_torch_cast(o64, o32):
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.standard_normal(4000), rng.standard_normal(2000) * 1e-3,
                        rng.standard_normal(2000) * 1e4]).astype(np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    for o in (o64, o32):
        got = np.array([o.bf16_rne(float(v)) for v in x], np.uint16)
        assert np.array_equal(got, want)
    assert np.array_equal(wlm.f32_to_bf16_bits(x), want)             # the input generator's rounding too


def test_bf16_double_build_rounds_once(o64):
    # a double just below a bf16 tie that float32 rounding would push onto the tie
    x = 1.0 + 2.0 ** -8 - 2.0 ** -40
    assert o64.bf16_rne(x) == 0x3F80
    x = 1.0 + 3 * 2.0 ** -8 - 2.0 ** -40     # via float32 this would become the tie and round UP
    assert o64.bf16_rne(x) == 0x3F81


# ---------------------------------------------------------------- Eq. 1: dense attention
def brute_attention(q, K, V, scale):
    """two-pass softmax written with python floats (tiny inputs only)"""
    n, d = len(K), len(q)
    logit = [scale * sum(q[x] * K[r][x] for x in range(d)) for r in range(n)]
    m = max(logit)
    p = [math.exp(l - m) for l in logit]
    den = sum(p)
    return [sum(p[r] * V[r][x] for r in range(n)) / den for x in range(d)], m + math.log(den)


@pytest.mark.parametrize("n,d", [(1, 1), (3, 2), (8, 4), (5, 3)])
def test_dense_attention_brute_force(o64, o32, n, d):
    rng = np.random.default_rng(n * 10 + d)
    S = 2
    q, K, V = rand_bits(rng, S, d), rand_bits(rng, S, n, d), rand_bits(rng, S, n, d)
    scale = 1.0 / math.sqrt(d)
    for o, tol in ((o64, 1e-14), (o32, 2e-6)):
        out, out_b, lse = o.attn_dense(q, K, V, scale)
        for s in range(S):
            want, want_lse = brute_attention(widen(q[s]).tolist(), widen(K[s]).tolist(), widen(V[s]).tolist(), scale)
            assert np.allclose(out[s], want, rtol=0, atol=tol)
            assert abs(lse[s] - want_lse) <= tol * 10
        assert np.array_equal(out_b, np.array([[o.bf16_rne(float(v)) for v in row] for row in out], np.uint16))


def test_dense_attention_special_cases(o64):
    rng = np.random.default_rng(7)
    S, n, d = 3, 37, 16
    K, V = rand_bits(rng, S, n, d), rand_bits(rng, S, n, d)
    # q = 0: uniform weights, output = mean of the V rows, lse = log n
    out, _, lse = o64.attn_dense(np.zeros((S, d), np.uint16), K, V, 0.25)
    assert np.allclose(out, widen(V).mean(axis=1), atol=1e-14)
    assert np.allclose(lse, math.log(n), atol=1e-14)
    # one key with a huge logit: output = that V row
    q = bits(np.ones((S, d)))
    K2 = K.copy()
    K2[:, 11] = bits(np.full((S, d), 64.0))
    out, _, _ = o64.attn_dense(q, K2, V, 1.0)
    assert np.allclose(out, widen(V[:, 11]), atol=1e-12)
    # empty cache: zeros and lse = -inf
    out, _, lse = o64.attn_dense(q, K[:, :0].copy(), V[:, :0].copy(), 1.0)
    assert np.all(out == 0) and np.all(np.isneginf(lse))


def test_dense_attention_matches_torch_sdpa(o64, o32):
    rng = np.random.default_rng(3)
    S, n, d = 4, 200, 128
    q, K, V = rand_bits(rng, S, d), rand_bits(rng, S, n, d), rand_bits(rng, S, n, d)
    scale = 1.0 / math.sqrt(d)
    tq, tK, tV = (torch.from_numpy(widen(a)) for a in (q, K, V))
    want = torch.nn.functional.scaled_dot_product_attention(tq[:, None, None, :], tK[:, None], tV[:, None], scale=scale)
    want = want[:, 0, 0].numpy()
    out, _, _ = o64.attn_dense(q, K, V, scale)
    assert np.allclose(out, want, atol=1e-13)
    out32, _, _ = o32.attn_dense(q, K, V, scale)
    assert np.allclose(out32, want, atol=5e-6)


def test_dense_attention_is_not_symmetric_in_k_and_v(o64):
    # guards against a transposed / swapped operand: swapping K and V must change the result
    rng = np.random.default_rng(5)
    q, K, V = rand_bits(rng, 1, 8), rand_bits(rng, 1, 6, 8), rand_bits(rng, 1, 6, 8)
    a, _, _ = o64.attn_dense(q, K, V, 0.5)
    b, _, _ = o64.attn_dense(q, V, K, 0.5)
    assert not np.allclose(a, b)


# ---------------------------------------------------------------- Eq. 2: aggregator
def test_summary_identity_chunk_of_one_is_raw_kv(o64, o32):
    rng = np.random.default_rng(11)
    S, n, d = 3, 9, 8
    K, V = rand_bits(rng, S, n, d), rand_bits(rng, S, n, d)
    for o in (o64, o32):
        for agg in (kvo.AGG_IDENTITY, kvo.AGG_MEAN):
            r = o.summarize(K, V, 1, 0, n, agg)
            assert np.array_equal(r["ksum_b16"], K) and np.array_equal(r["vsum_b16"], V)
            assert np.array_equal(r["ksum"], widen(K).astype(o.real))


def test_summary_identity_needs_unit_chunks(o64):
    K = np.zeros((1, 4, 2), np.uint16)
    with pytest.raises(ValueError):
        o64.summarize(K, K, 2, 0, 2, kvo.AGG_IDENTITY)


def test_summary_mean_closed_forms(o64):
    rng = np.random.default_rng(12)
    S, C, d, Nc = 2, 5, 4, 3
    K, V = rand_bits(rng, S, C * Nc + 2, d), rand_bits(rng, S, C * Nc + 2, d)
    # constant chunk -> the constant
    K[:, C:2 * C] = bits(np.full((S, C, d), 0.75))
    r = o64.summarize(K, V, C, 0, Nc, kvo.AGG_MEAN)
    assert np.all(r["ksum"][:, 1] == 0.75)
    # definition: arithmetic mean per chunk, per head dim, keys and values separately
    want_k = widen(K)[:, :C * Nc].reshape(S, Nc, C, d).mean(axis=2)
    want_v = widen(V)[:, :C * Nc].reshape(S, Nc, C, d).mean(axis=2)
    assert np.allclose(r["ksum"], want_k, atol=1e-15) and np.allclose(r["vsum"], want_v, atol=1e-15)
    assert not np.allclose(r["ksum"], want_v)
    # order of tokens inside a chunk does not matter (up to reassociation)
    perm = rng.permutation(C)
    K2, V2 = K.copy(), V.copy()
    K2[:, :C] = K[:, :C][:, perm]
    V2[:, :C] = V[:, :C][:, perm]
    r2 = o64.summarize(K2, V2, C, 0, Nc, kvo.AGG_MEAN)
    assert np.allclose(r2["ksum"], r["ksum"], atol=1e-15)
    # a chunk range writes only its own rows
    r3 = o64.summarize(K, V, C, 1, 2, kvo.AGG_MEAN, stride=Nc)
    assert np.all(r3["ksum"][:, 0] == 0) and np.all(r3["ksum"][:, 2] == 0)
    assert np.array_equal(r3["ksum"][:, 1], r["ksum"][:, 1])


def test_summary_mlp_hand_worked(o64, o32):
    g = read_golden("mlp_2x2.txt")
    K = bits(np.array([[[1, 3], [1, -1]]], np.float32))
    V = np.zeros((1, 2, 2), np.uint16)
    mlp = dict(W1K=np.array([[1, 0], [0, -1]], np.float32), b1K=np.zeros(2, np.float32),
               W2K=np.array([[1, 1], [2, 0]], np.float32), b2K=np.array([0.5, 0], np.float32),
               W1V=np.array([[3, 1], [1, 2]], np.float32), b1V=np.zeros(2, np.float32),
               W2V=np.array([[5, 7], [1, 1]], np.float32), b2V=np.array([0.25, -0.75], np.float32))
    for o, tol in ((o64, 1e-15), (o32, 2e-7)):
        r = o.summarize(K, V, 2, 0, 1, kvo.AGG_MLP, mlp)
        assert np.allclose(r["ksum"][0, 0], g["kbar"], atol=tol)
        assert np.allclose(r["vsum"][0, 0], g["vbar"], atol=tol)


def test_summary_mlp_matches_torch_modules(o64):
    rng = np.random.default_rng(13)
    wl = wlm.Workload("t", B=1, H=2, n=24, C=4, W=8, d_g=8, agg="mlp", d_sum=6, d=8)
    K, V = wlm.gen_kv(wl)
    mlp = wlm.gen_mlp_weights(wl)
    r = o64.summarize(K, V, wl.C, 0, 4, kvo.AGG_MLP, mlp)
    gelu = torch.nn.GELU(approximate="none")
    for side, X, got in (("K", K, r["ksum"]), ("V", V, r["vsum"])):
        m = torch.from_numpy(widen(X))[:, :16].reshape(2, 4, 4, 8).mean(dim=2)
        W1, b1, W2, b2 = (torch.from_numpy(mlp[k + side]).double() for k in ("W1", "b1", "W2", "b2"))
        want = torch.nn.functional.linear(gelu(torch.nn.functional.linear(m, W1, b1)), W2, b2).numpy()
        assert np.allclose(got, want, atol=1e-14)
    assert np.array_equal(r["ksum_b16"], np.vectorize(o64.bf16_rne, otypes=[np.uint16])(r["ksum"]))


def test_summary_token_mlp_hand_worked(o64, o32):
    """Eq. 2 with the MLP on every token, then the mean: differs from mean-then-MLP on the same numbers."""
    g = read_golden("token_mlp_2x2.txt")
    K = bits(np.array([[[1, 3], [1, -1]]], np.float32))
    V = np.zeros((1, 2, 2), np.uint16)
    mlp = dict(W1K=np.array([[1, 0], [0, -1]], np.float32), b1K=np.zeros(2, np.float32),
               W2K=np.array([[1, 1], [2, 0]], np.float32), b2K=np.array([0.5, 0], np.float32),
               W1V=np.array([[3, 1], [1, 2]], np.float32), b1V=np.zeros(2, np.float32),
               W2V=np.array([[5, 7], [1, 1]], np.float32), b2V=np.array([0.25, -0.75], np.float32))
    for o, tol in ((o64, 1e-14), (o32, 3e-7)):
        r = o.summarize(K, V, 2, 0, 1, kvo.AGG_TOKEN_MLP, mlp)
        assert np.allclose(r["ksum"][0, 0], g["kbar"], atol=tol)
        assert np.allclose(r["vsum"][0, 0], g["vbar"], atol=tol)
    other = read_golden("mlp_2x2.txt")
    assert abs(g["kbar"][0] - other["kbar"][0]) > 0.5          # the two readings of Eq. 2 give different numbers here


def test_summary_token_mlp_matches_torch_modules_and_special_cases(o64):
    wl = wlm.Workload("t", B=1, H=2, n=24, C=4, W=8, d_g=8, agg="token_mlp", d_sum=6, d=8)
    K, V = wlm.gen_kv(wl)
    mlp = wlm.gen_mlp_weights(wl)
    r = o64.summarize(K, V, wl.C, 0, 4, kvo.AGG_TOKEN_MLP, mlp)
    gelu = torch.nn.GELU(approximate="none")
    for side, X, got in (("K", K, r["ksum"]), ("V", V, r["vsum"])):
        x = torch.from_numpy(widen(X))[:, :16].reshape(2, 4, 4, 8)                     # [S, chunk, token, d]
        W1, b1, W2, b2 = (torch.from_numpy(mlp[k + side]).double() for k in ("W1", "b1", "W2", "b2"))
        per_token = torch.nn.functional.linear(gelu(torch.nn.functional.linear(x, W1, b1)), W2, b2)
        assert np.allclose(got, per_token.mean(dim=2).numpy(), atol=1e-14)
        # the last layer is affine and the mean is linear: pooling the activations first gives the same vector
        pooled = gelu(torch.nn.functional.linear(x, W1, b1)).mean(dim=2)
        assert np.allclose(got, torch.nn.functional.linear(pooled, W2, b2).numpy(), atol=1e-13)
    # chunks of one token: nothing to pool, so both readings of Eq. 2 coincide
    a = o64.summarize(K, V, 1, 0, 24, kvo.AGG_TOKEN_MLP, mlp)
    b_ = o64.summarize(K, V, 1, 0, 24, kvo.AGG_MLP, mlp)
    assert np.allclose(a["ksum"], b_["ksum"], atol=1e-15) and np.allclose(a["vsum"], b_["vsum"], atol=1e-15)
    # a chunk of identical tokens: the mean of equal outputs is that output = the MLP of the (equal) mean
    Kc = np.repeat(K[:, :1], 4, axis=1)
    Vc = np.repeat(V[:, :1], 4, axis=1)
    a = o64.summarize(Kc, Vc, 4, 0, 1, kvo.AGG_TOKEN_MLP, mlp)
    b_ = o64.summarize(Kc, Vc, 4, 0, 1, kvo.AGG_MLP, mlp)
    assert np.allclose(a["ksum"], b_["ksum"], atol=1e-14) and np.allclose(a["vsum"], b_["vsum"], atol=1e-14)
    assert np.array_equal(r["ksum_b16"], np.vectorize(o64.bf16_rne, otypes=[np.uint16])(r["ksum"]))


# ---------------------------------------------------------------- Eq. 3: LSTM gate
def small_gate_problem(seed=21, S=3, Nc=6, d=4, d_g=5):
    rng = np.random.default_rng(seed)
    wl = wlm.Workload("g", B=1, H=S, n=Nc, C=1, W=0, d_g=d_g, d=d, seed=seed)
    lstm = wlm.gen_lstm_weights(wl, b_s=0.3)
    return rand_bits(rng, S, Nc, d), rand_bits(rng, S, Nc, d), lstm


def test_gate_zero_weights_gives_sigmoid_of_bias(o64):
    ks, vs, lstm = small_gate_problem()
    z = {k: (np.zeros_like(v) if isinstance(v, np.ndarray) else v) for k, v in lstm.items()}
    z["b_s"] = -1.25
    scores, h, c = o64.gate(ks, vs, 0, ks.shape[1], z)
    assert np.all(h == 0) and np.all(c == 0)
    assert np.allclose(scores, 1 / (1 + math.exp(1.25)), atol=1e-16)


def test_gate_saturated_cell_closed_form(o64, o32):
    """d = 1, d_g = 1; input and output gates pinned open (bias +40), forget gate open (+40):
    c_t = c_{t-1} + tanh(a*Kbar_t + b*Vbar_t + r*h_{t-1}),  h_t = tanh(c_t),  s_t = sigmoid(w*h_t + b_s)."""
    a, b, r, w, b_s = 1.0, 2.0, 0.5, 1.5, -0.25
    ks, vs = bits(np.array([[[0.5], [-1.0], [0.25]]])), bits(np.array([[[0.25], [0.5], [2.0]]]))
    lstm = dict(W_ih=np.array([[0, 0], [0, 0], [a, b], [0, 0]], np.float32),
                W_hh=np.array([[0], [0], [r], [0]], np.float32),
                b_ih=np.array([40, 15, 0, 25], np.float32), b_hh=np.array([0, 25, 0, 15], np.float32),
                w_s=np.array([w], np.float32), b_s=b_s)
    c = h = 0.0
    want = []
    for kt, vt in ((0.5, 0.25), (-1.0, 0.5), (0.25, 2.0)):
        c = c + math.tanh(a * kt + b * vt + r * h)
        h = math.tanh(c)
        want.append(1 / (1 + math.exp(-(w * h + b_s))))
    for o, tol in ((o64, 1e-15), (o32, 3e-7)):
        scores, hh, cc = o.gate(ks, vs, 0, 3, lstm)
        assert np.allclose(scores[0], want, atol=tol)
        assert abs(hh[0, 0] - h) <= tol and abs(cc[0, 0] - c) <= tol
    # forget gate shut instead (bias -40): the cell forgets, c_t = tanh(pre_g) alone
    lstm["b_ih"] = np.array([40, -40, 0, 25], np.float32)
    lstm["b_hh"] = np.array([0, 0, 0, 15], np.float32)
    scores, hh, cc = o64.gate(ks, vs, 0, 3, lstm)
    h = 0.0
    for kt, vt in ((0.5, 0.25), (-1.0, 0.5), (0.25, 2.0)):
        c = math.tanh(a * kt + b * vt + r * h)
        h = math.tanh(c)
    assert abs(cc[0, 0] - c) < 1e-15


@pytest.mark.parametrize("d,d_g", [(4, 5), (128, 32)])
def test_gate_matches_torch_lstm(o64, o32, d, d_g):
    ks, vs, lstm = small_gate_problem(seed=22, S=3, Nc=7, d=d, d_g=d_g)
    ref = torch.nn.LSTM(2 * d, d_g, num_layers=1, batch_first=True, bidirectional=False).double()
    with torch.no_grad():
        ref.weight_ih_l0.copy_(torch.from_numpy(lstm["W_ih"]))
        ref.weight_hh_l0.copy_(torch.from_numpy(lstm["W_hh"]))
        ref.bias_ih_l0.copy_(torch.from_numpy(lstm["b_ih"]))
        ref.bias_hh_l0.copy_(torch.from_numpy(lstm["b_hh"]))
        x = torch.from_numpy(np.concatenate([widen(ks), widen(vs)], axis=-1))      # [Kbar ; Vbar]
        hs, (hN, cN) = ref(x)
        want = torch.sigmoid(hs @ torch.from_numpy(lstm["w_s"]).double() + lstm["b_s"]).numpy()
    scores, h, c = o64.gate(ks, vs, 0, 7, lstm)
    assert np.allclose(scores, want, atol=1e-13)
    assert np.allclose(h, hN[0].numpy(), atol=1e-13) and np.allclose(c, cN[0].numpy(), atol=1e-13)
    s32, _, _ = o32.gate(ks, vs, 0, 7, lstm)
    assert np.allclose(s32, want, atol=5e-6)


def test_gate_prefix_causality_and_incremental(o64, o32):
    ks, vs, lstm = small_gate_problem(seed=23, S=4, Nc=9)
    for o in (o64, o32):
        full, hF, cF = o.gate(ks, vs, 0, 9, lstm)
        # changing chunks > t leaves s[0..t] untouched
        ks2, vs2 = ks.copy(), vs.copy()
        ks2[:, 5:] = ks[:, 5:][:, ::-1]
        vs2[:, 5:] ^= 0x0100
        part, _, _ = o.gate(ks2, vs2, 0, 9, lstm)
        assert np.array_equal(part[:, :5], full[:, :5]) and not np.array_equal(part[:, 5:], full[:, 5:])
        # two calls carrying (h, c) == one call, bit for bit
        sc, h, c = o.gate(ks, vs, 0, 4, lstm)
        sc, h, c = o.gate(ks, vs, 4, 9, lstm, h, c, sc)
        assert np.array_equal(sc, full) and np.array_equal(h, hF) and np.array_equal(c, cF)
        # order over chunks matters (the LSTM is recurrent)...
        rev, _, _ = o.gate(ks[:, ::-1].copy(), vs[:, ::-1].copy(), 0, 9, lstm)
        assert not np.allclose(rev[:, ::-1], full)
        # ...but sequences are independent: permuting them permutes the scores
        p = np.array([2, 0, 3, 1])
        perm, _, _ = o.gate(ks[p].copy(), vs[p].copy(), 0, 9, lstm)
        assert np.array_equal(perm, full[p])


def test_gate_input_order_is_k_then_v(o64):
    ks, vs, lstm = small_gate_problem(seed=24)
    a, _, _ = o64.gate(ks, vs, 0, 6, lstm)
    b, _, _ = o64.gate(vs, ks, 0, 6, lstm)
    assert not np.allclose(a, b)
    # swapping the halves of W_ih's columns undoes swapping the inputs
    d = ks.shape[2]
    sw = dict(lstm)
    sw["W_ih"] = np.concatenate([lstm["W_ih"][:, d:], lstm["W_ih"][:, :d]], axis=1)
    c, _, _ = o64.gate(vs, ks, 0, 6, sw)
    assert np.allclose(a, c, atol=1e-15)


def test_gate_f32_tracks_f64(o64, o32):
    wl = wlm.Workload("g", B=1, H=4, n=40, C=1, W=0, d_g=128, seed=5)
    lstm = wlm.gen_lstm_weights(wl)
    rng = np.random.default_rng(5)
    ks, vs = rand_bits(rng, 4, 40, 128), rand_bits(rng, 4, 40, 128)
    s64, _, _ = o64.gate(ks, vs, 0, 40, lstm)
    s32, _, _ = o32.gate(ks, vs, 0, 40, lstm)
    assert np.abs(s64 - s32).max() < 5e-6
    assert 0.0 <= s64.min() and s64.max() <= 1.0 and s64.std() > 1e-3


# ---------------------------------------------------------------- retention rule
def test_compact_threshold_is_inclusive(o64, o32):
    for o in (o64, o32):
        tau = 0.3
        t = np.float32(tau) if o.kind == "f32" else tau
        sc = np.array([[np.nextafter(t, 0, dtype=o.real) if o.kind == "f32" else np.nextafter(t, 0), t,
                        np.nextafter(t, 1, dtype=o.real) if o.kind == "f32" else np.nextafter(t, 1), 0.0, 1.0]], o.real)
        idx, cnt = o.compact(sc, 5, tau)
        assert cnt[0] == 3 and idx[0].tolist() == [1, 2, 4, -1, -1]


@pytest.mark.parametrize("Nc", [0, 1, 3, 10])
def test_compact_exhaustive_masks(o64, Nc):
    masks = list(itertools.product([0, 1], repeat=Nc))
    sc = np.array([[0.9 if b else 0.1 for b in m] + [0.9, 0.9] for m in masks], np.float64).reshape(len(masks), Nc + 2)
    idx, cnt = o64.compact(sc, Nc, 0.5)        # the two trailing entries lie beyond n_chunks: ignored
    for i, m in enumerate(masks):
        want = [t for t, b in enumerate(m) if b]
        assert cnt[i] == len(want) == sum(m)
        assert idx[i, :cnt[i]].tolist() == want and np.all(idx[i, cnt[i]:] == -1)
        assert all(x < y for x, y in zip(want, want[1:]))


# ---------------------------------------------------------------- Sec. 3.3: attention over window + retained chunks
def gated_problem(seed=31, S=3, n=45, C=4, W=10, d=8):
    rng = np.random.default_rng(seed)
    q, K, V = rand_bits(rng, S, d), rand_bits(rng, S, n, d), rand_bits(rng, S, n, d)
    Nc = (n - W) // C
    return q, K, V, Nc


def test_gated_keep_all_raw_equals_dense(o64, o32):
    q, K, V, Nc = gated_problem()
    for o in (o64, o32):
        sm = o.summarize(K, V, 4, 0, Nc, kvo.AGG_MEAN)
        idx, cnt = o.compact(np.ones((3, Nc), o.real), Nc, 0.0)        # tau = 0 keeps everything
        out, out_b, lse, n_eff = o.attn(q, K, V, 4, Nc, idx, cnt, sm["ksum_b16"], sm["vsum_b16"], kvo.ATTEND_RAW, 0.3)
        dn, dn_b, dlse = o.attn_dense(q, K, V, 0.3)
        assert np.array_equal(out, dn) and np.array_equal(out_b, dn_b) and np.array_equal(lse, dlse)
        assert np.all(n_eff == 45)


def test_gated_keep_nothing_equals_window_only(o64):
    q, K, V, Nc = gated_problem()
    sm = o64.summarize(K, V, 4, 0, Nc, kvo.AGG_MEAN)
    idx, cnt = o64.compact(np.full((3, Nc), 0.5), Nc, 1.5)               # tau > 1 keeps nothing
    assert np.all(cnt == 0)
    R = 45 - Nc * 4
    for mode in (kvo.ATTEND_SUMMARY, kvo.ATTEND_RAW):
        out, _, lse, n_eff = o64.attn(q, K, V, 4, Nc, idx, cnt, sm["ksum_b16"], sm["vsum_b16"], mode, 0.3)
        dn, _, dlse = o64.attn_dense(q, K[:, -R:].copy(), V[:, -R:].copy(), 0.3)
        assert np.array_equal(out, dn) and np.array_equal(lse, dlse) and np.all(n_eff == R)
    assert 10 <= R < 10 + 4                                              # W <= R < W + C


def test_gated_summary_equals_dense_over_explicit_list(o64):
    q, K, V, Nc = gated_problem(seed=32)
    S = 3
    sm = o64.summarize(K, V, 4, 0, Nc, kvo.AGG_MEAN)
    sc = np.random.default_rng(1).uniform(size=(S, Nc))
    idx, cnt = o64.compact(sc, Nc, 0.5)
    assert 0 < cnt.min() and cnt.max() < Nc and len(set(cnt.tolist())) > 1
    out, _, lse, n_eff = o64.attn(q, K, V, 4, Nc, idx, cnt, sm["ksum_b16"], sm["vsum_b16"], kvo.ATTEND_SUMMARY, 0.3)
    outr, _, _, n_effr = o64.attn(q, K, V, 4, Nc, idx, cnt, sm["ksum_b16"], sm["vsum_b16"], kvo.ATTEND_RAW, 0.3)
    R = 45 - Nc * 4
    for s in range(S):
        kept = idx[s, :cnt[s]]
        Ks = np.concatenate([sm["ksum_b16"][s, kept], K[s, Nc * 4:]])[None]
        Vs = np.concatenate([sm["vsum_b16"][s, kept], V[s, Nc * 4:]])[None]
        dn, _, dlse = o64.attn_dense(q[s:s + 1], Ks, Vs, 0.3)
        assert np.array_equal(out[s], dn[0]) and lse[s] == dlse[0]
        assert n_eff[s] == R + cnt[s]                                    # n' = W + M (with the ragged tail in R)
        rows = np.concatenate([np.arange(t * 4, t * 4 + 4) for t in kept] + [np.arange(Nc * 4, 45)])
        dn, _, _ = o64.attn_dense(q[s:s + 1], K[s:s + 1, rows], V[s:s + 1, rows], 0.3)
        assert np.array_equal(outr[s], dn[0]) and n_effr[s] == R + 4 * cnt[s]


def test_gated_chunk_of_one_identity_keep_all_equals_dense(o64):
    # C = 1, identity aggregation, everything kept: the summary path IS dense attention
    q, K, V, _ = gated_problem(seed=33, n=20, C=1, W=6)
    Nc = 14
    sm = o64.summarize(K, V, 1, 0, Nc, kvo.AGG_IDENTITY)
    idx, cnt = o64.compact(np.ones((3, Nc)), Nc, 0.0)
    out, out_b, _, _ = o64.attn(q, K, V, 1, Nc, idx, cnt, sm["ksum_b16"], sm["vsum_b16"], kvo.ATTEND_SUMMARY, 0.3)
    dn, dn_b, _ = o64.attn_dense(q, K, V, 0.3)
    assert np.array_equal(out, dn) and np.array_equal(out_b, dn_b)


def test_window_rows_are_never_transformed(o64):
    # changing stale chunks that are NOT kept cannot change the output; changing a window row does
    q, K, V, Nc = gated_problem(seed=34)
    sm = o64.summarize(K, V, 4, 0, Nc, kvo.AGG_MEAN)
    keep_idx = np.full((3, Nc), -1, np.int32)
    keep_idx[:, 0] = 2
    keep_cnt = np.ones(3, np.int32)
    base, _, _, _ = o64.attn(q, K, V, 4, Nc, keep_idx, keep_cnt, sm["ksum_b16"], sm["vsum_b16"], kvo.ATTEND_SUMMARY, 0.3)
    K2 = K.copy()
    K2[:, 0:8] ^= 0x0040                         # chunks 0, 1: discarded
    a, _, _, _ = o64.attn(q, K2, V, 4, Nc, keep_idx, keep_cnt, sm["ksum_b16"], sm["vsum_b16"], kvo.ATTEND_SUMMARY, 0.3)
    assert np.array_equal(a, base)
    K3 = K.copy()
    K3[:, -1] ^= 0x0040                          # newest token
    b, _, _, _ = o64.attn(q, K3, V, 4, Nc, keep_idx, keep_cnt, sm["ksum_b16"], sm["vsum_b16"], kvo.ATTEND_SUMMARY, 0.3)
    assert not np.array_equal(b, base)


def test_memory_ratio_closed_form():
    # Sec. 3.3: ratio n / (W + M); the paper's instance prints 2.44 for n = 10000, W = 4096, M = 2
    g = read_golden("cost_model.txt")
    assert round(10000 / (4096 + 2), 2) == g["memory_ratio"][0]
    assert 4 * 10000 * 4096 ** 2 + 2 * 32 * 10000 ** 2 * 128 == int(g["flops_base"][0])


# ---------------------------------------------------------------- whole pipeline sanity at config-1 scale
def test_pipeline_config1_shapes_and_counts(o32, o64):
    wl = wlm.CFG1.small(n=512, W=128)
    K, V = wlm.gen_kv(wl)
    q = wlm.gen_q(wl)
    lstm = wlm.gen_lstm_weights(wl)
    Nc = wl.n_stale_chunks()
    assert Nc == 6
    res = {}
    for o in (o32, o64):
        sm = o.summarize(K, V, wl.C, 0, Nc, kvo.AGG_MEAN)
        sc, _, _ = o.gate(sm["ksum_b16"], sm["vsum_b16"], 0, Nc, lstm)
        idx, cnt = o.compact(sc, Nc, wl.tau)
        out, out_b, lse, n_eff = o.attn(q, K, V, wl.C, Nc, idx, cnt, sm["ksum_b16"], sm["vsum_b16"],
                                        kvo.ATTEND_SUMMARY, 1 / math.sqrt(wl.d))
        assert np.all(n_eff == 128 + cnt)
        res[o.kind] = (sc, out)
    assert np.abs(res["f32"][0] - res["f64"][0]).max() < 1e-5
    assert np.abs(res["f32"][1] - res["f64"][1]).max() < 1e-5


# ---- Sec. 3.3 memory reduction: pages of gated chunks handed back ---------------------------------
def test_reclaim_is_the_complement_of_the_retention_rule_and_conserves_pages(o64, o32):
    rng = np.random.default_rng(3)
    S, stride, Nc, tau = 5, 12, 9, 0.5
    for o in (o64, o32):
        scores = rng.random((S, stride)).astype(o.real)
        scores[0, 0] = tau                      # equality is retained (Sec. 3.2), hence NOT handed back in mode 0
        pages = rng.permutation(S * stride).astype(np.int32).reshape(S, stride)
        idx, cnt = o.compact(scores, Nc, tau)
        pt = pages.copy()
        free = o.reclaim(pt, scores, 0, Nc, tau, 0)
        # brute force: every gated chunk not in the keep list, sequence-major, ascending
        want = [pages[s, t] for s in range(S) for t in range(Nc) if t not in set(idx[s, :cnt[s]].tolist())]
        assert free.tolist() == want and pages[0, 0] not in free
        assert len(free) == S * Nc - int(cnt.sum())
        for s in range(S):
            for t in range(stride):
                kept_or_ungated = t >= Nc or t in idx[s, :cnt[s]]
                assert pt[s, t] == (pages[s, t] if kept_or_ungated else -1)
        # nothing is lost or duplicated; a second call finds nothing left
        assert sorted(free.tolist() + pt[pt >= 0].tolist()) == sorted(pages.ravel().tolist())
        assert len(o.reclaim(pt, scores, 0, Nc, tau, 0)) == 0
        # mode 1 (retained chunks live on as summaries): the rest of the gated range follows, window chunks never
        rest = o.reclaim(pt, scores, 0, Nc, tau, 1)
        assert sorted(rest.tolist()) == sorted(pages[s, t] for s in range(S) for t in range(Nc) if pt[s, t] == -1 and pages[s, t] not in free)
        assert (pt[:, :Nc] == -1).all() and np.array_equal(pt[:, Nc:], pages[:, Nc:])
        # the memory ratio of Sec. 3.3: n / (W + M) rows remain addressable per sequence
        assert len(free) + len(rest) == S * Nc


def test_reclaim_ranges_and_bad_arguments(o64):
    scores = np.zeros((2, 6), np.float64)          # everything discarded at tau = 0.5
    pt = np.arange(12, dtype=np.int32).reshape(2, 6)
    assert o64.reclaim(pt, scores, 2, 4, 0.5, 0).tolist() == [2, 3, 8, 9]
    assert o64.reclaim(pt, scores, 0, 6, 0.5, 0).tolist() == [0, 1, 4, 5, 6, 7, 10, 11]
    with pytest.raises(ValueError):
        o64.reclaim(pt, scores, 0, 7, 0.5, 0)
    with pytest.raises(ValueError):
        o64.reclaim(pt, scores, 0, 6, 0.5, 2)


# ---- gating variant: top-k retention ---------------------------------------------------------------
def test_topk_matches_a_stable_sort_and_the_threshold_rule(o64, o32):
    rng = np.random.default_rng(11)
    S, stride, Nc = 6, 40, 33
    for o in (o64, o32):
        scores = rng.random((S, stride)).astype(o.real)
        scores[1, 5] = scores[1, 9] = scores[1, 20] = 0.77            # ties: the older chunk ranks first
        for k in (0, 1, 7, 16, Nc, Nc + 5):
            idx, cnt = o.compact_topk(scores, Nc, k)
            for s in range(S):
                order = np.argsort(-scores[s, :Nc].astype(np.float64), kind="stable")   # descending, ties keep index order
                want = np.sort(order[:max(0, min(k, Nc))])
                assert cnt[s] == len(want) and np.array_equal(idx[s, :cnt[s]], want)
                assert (idx[s, cnt[s]:] == -1).all()
        # thresholding at a value strictly between the k-th and (k+1)-th score keeps exactly the top k
        k = 12
        idx, cnt = o.compact_topk(scores, Nc, k)
        for s in range(S):
            srt = np.sort(scores[s, :Nc].astype(np.float64))[::-1]
            if srt[k - 1] > srt[k]:
                tau = 0.5 * (srt[k - 1] + srt[k])
                tidx, tcnt = o.compact(scores[s:s + 1].copy(), Nc, tau)
                assert tcnt[0] == k and np.array_equal(tidx[0, :k], idx[s, :k])


def test_topk_ties_at_the_boundary_prefer_older_chunks(o64):
    scores = np.array([[0.5, 0.9, 0.5, 0.5, 0.1, 0.5]], np.float64)
    idx, cnt = o64.compact_topk(scores, 6, 3)
    assert cnt[0] == 3 and idx[0, :3].tolist() == [0, 1, 2]           # 0.9, then the two oldest 0.5s
    idx, cnt = o64.compact_topk(scores, 6, 0)
    assert cnt[0] == 0 and (idx == -1).all()


# ---- the paper's cost model (Sec. 3.3, Eq. 4-7) against the numbers printed in Sec. 4.1 --------------
def test_cost_model_reproduces_the_printed_instance():
    from paper_2509_21354_b200 import cost_model as cm
    g = read_golden("cost_model.txt")
    n, W, C, d_sum, d_g, r = 10000, 4096, 3136, 128, 128, 0.687       # n = 10000 is what the printed FLOPs_base implies
    M = r * n / C                                                      # retained chunks at the stated retention ratio
    assert cm.flops_base(n) == g["flops_base"][0]                      # exact
    kv = cm.flops_kv_efficient(n, W, M, C, d_sum, d_g)
    assert abs(kv / g["flops_kv_eff"][0] - 1) < 2e-5                   # printed with "approximately"
    assert round(cm.speedup(n, W, M, C, d_sum, d_g), 2) == g["speedup"][0]
    assert round(cm.memory_ratio(n, W, 2), 2) == g["memory_ratio"][0]  # the paper rounds M to 2 chunks here
    # Eq. 5 evaluates to 1,352,663,040,000; the paper prints a figure 0.07 % lower (recorded, not reproduced)
    assert cm.flops_ffn(n) == 3 * 10000 * 4096 * 11008
    assert abs(cm.flops_ffn(n) / g["flops_ffn_printed"][0] - 1) < 1e-3
    # sanity of the closed forms: keeping everything in the window is the base model plus the gate's overhead
    assert cm.flops_kv_efficient(n, n, 0, C, d_sum, d_g) == cm.flops_base(n)
    assert cm.memory_ratio(n, n, 0) == 1.0


# ---- "pooling" aggregator (Sec. 3.1): element-wise maximum of the chunk ---------------------------------
def test_max_pool_aggregator_is_the_elementwise_maximum(o64, o32):
    wl = wlm.CFG1.small(B=1, H=2, n=512, W=128)
    K, V = wlm.gen_kv(wl)
    Nc = wl.n_stale_chunks()
    Kf, Vf = wlm.bf16_bits_to_f32(K), wlm.bf16_bits_to_f32(V)
    for o in (o64, o32):
        sm = o.summarize(K, V, wl.C, 0, Nc, kvo.AGG_MAX)
        want_k = Kf[:, :Nc * wl.C].reshape(wl.S, Nc, wl.C, 128).max(axis=2)
        want_v = Vf[:, :Nc * wl.C].reshape(wl.S, Nc, wl.C, 128).max(axis=2)
        assert np.array_equal(sm["ksum"][:, :Nc].astype(np.float32), want_k)
        assert np.array_equal(sm["vsum"][:, :Nc].astype(np.float32), want_v)
        # a maximum of bf16 values is a bf16 value: the rounded copy is the value itself, an entry of the chunk
        assert np.array_equal(wlm.bf16_bits_to_f32(sm["ksum_b16"][:, :Nc]), want_k)
        assert (sm["ksum"][:, :Nc] >= o.summarize(K, V, wl.C, 0, Nc, kvo.AGG_MEAN)["ksum"][:, :Nc]).all()   # max >= mean
    # C = 1: max-pool is the identity
    wl1 = wlm.CFG1.small(B=1, H=1, n=40, C=1, W=8)
    K1, V1 = wlm.gen_kv(wl1)
    a = o64.summarize(K1, V1, 1, 0, 32, kvo.AGG_MAX)
    assert np.array_equal(a["ksum_b16"][:, :32], K1[:, :32]) and np.array_equal(a["vsum_b16"][:, :32], V1[:, :32])


# ---------------------------------------------------------------- query blocks: grouped-query attention (Sec. 4.1) and several query tokens at once
def test_query_block_brute_force_grouped_heads(o64, o32):
    """Every (token, query head) of a block against python-float softmax over an explicitly built
    row list of ITS KV head (query head hq reads KV head hq // group), summary and raw modes."""
    rng = np.random.default_rng(77)
    B, Hkv, G, T, d, n, C, W = 2, 2, 3, 2, 4, 23, 4, 6
    Hq, S = Hkv * G, B * Hkv
    K, V = rand_bits(rng, S, n, d), rand_bits(rng, S, n, d)
    q = rand_bits(rng, B, T, Hq, d)
    Nc = (n - W) // C
    for o, tol in ((o64, 1e-13), (o32, 3e-6)):
        sm = o.summarize(K, V, C, 0, Nc, kvo.AGG_MEAN)
        idx, cnt = o.compact(np.random.default_rng(3).uniform(size=(S, Nc)).astype(o.real), Nc, 0.5)
        assert 0 < cnt.sum() < S * Nc
        for mode in (kvo.ATTEND_SUMMARY, kvo.ATTEND_RAW):
            out, out_b, lse = o.attn_block(q, Hkv, K, V, C, Nc, idx, cnt, sm["ksum_b16"], sm["vsum_b16"], mode, 0.4)
            for b, t, hq in itertools.product(range(B), range(T), range(Hq)):
                s = b * Hkv + hq // G
                kept = idx[s, :cnt[s]]
                if mode == kvo.ATTEND_SUMMARY:
                    Kr = [widen(sm["ksum_b16"][s, c]).tolist() for c in kept]
                    Vr = [widen(sm["vsum_b16"][s, c]).tolist() for c in kept]
                else:
                    Kr = [widen(K[s, r]).tolist() for c in kept for r in range(c * C, c * C + C)]
                    Vr = [widen(V[s, r]).tolist() for c in kept for r in range(c * C, c * C + C)]
                Kr += [widen(K[s, r]).tolist() for r in range(Nc * C, n)]
                Vr += [widen(V[s, r]).tolist() for r in range(Nc * C, n)]
                want, want_lse = brute_attention(widen(q[b, t, hq]).tolist(), Kr, Vr, 0.4)
                assert np.allclose(out[b, t, hq], want, rtol=0, atol=tol), (mode, b, t, hq)
                assert abs(lse[b, t, hq] - want_lse) <= 10 * tol
            assert np.array_equal(out_b, np.vectorize(lambda v: o.bf16_rne(float(v)), otypes=[np.uint16])(out))
        # full-cache baseline for the block
        out, _, lse = o.attn_block(q, Hkv, K, V, C, Nc, idx, cnt, None, None, kvo.ATTEND_RAW, 0.4, dense=True)
        for b, t, hq in itertools.product(range(B), range(T), range(Hq)):
            s = b * Hkv + hq // G
            want, _ = brute_attention(widen(q[b, t, hq]).tolist(), widen(K[s]).tolist(), widen(V[s]).tolist(), 0.4)
            assert np.allclose(out[b, t, hq], want, rtol=0, atol=tol)


def test_query_block_of_one_token_one_head_per_kv_head_is_the_single_query_path(o64):
    q, K, V, Nc = gated_problem(seed=35)
    sm = o64.summarize(K, V, 4, 0, Nc, kvo.AGG_MEAN)
    idx, cnt = o64.compact(np.random.default_rng(2).uniform(size=(3, Nc)), Nc, 0.4)
    want, want_b, want_lse, _ = o64.attn(q, K, V, 4, Nc, idx, cnt, sm["ksum_b16"], sm["vsum_b16"], kvo.ATTEND_SUMMARY, 0.3)
    got, got_b, got_lse = o64.attn_block(q.reshape(1, 1, 3, 8), 3, K, V, 4, Nc, idx, cnt, sm["ksum_b16"], sm["vsum_b16"],
                                         kvo.ATTEND_SUMMARY, 0.3)
    assert np.array_equal(got[0, 0], want) and np.array_equal(got_b[0, 0], want_b) and np.array_equal(got_lse[0, 0], want_lse)


def test_query_block_rows_are_independent_and_permutable(o64):
    """Swapping two tokens of a block swaps their outputs; two equal queries get equal outputs;
    heads of one group that carry the same query agree (they read the same KV head), heads of
    different groups do not."""
    rng = np.random.default_rng(5)
    B, Hkv, G, T, d, n, C, W = 1, 2, 2, 3, 8, 30, 4, 8
    S = B * Hkv
    K, V = rand_bits(rng, S, n, d), rand_bits(rng, S, n, d)
    q = rand_bits(rng, B, T, Hkv * G, d)
    q[0, 2] = q[0, 0]                       # token 2 repeats token 0
    q[0, 1, 1] = q[0, 1, 0]                 # heads 0, 1 (one group) carry one query
    q[0, 1, 2] = q[0, 1, 0]                 # head 2 (the other group) carries it too
    Nc = (n - W) // C
    sm = o64.summarize(K, V, C, 0, Nc, kvo.AGG_MEAN)
    idx, cnt = o64.compact(np.random.default_rng(9).uniform(size=(S, Nc)), Nc, 0.5)
    args = (Hkv, K, V, C, Nc, idx, cnt, sm["ksum_b16"], sm["vsum_b16"], kvo.ATTEND_SUMMARY, 0.35)
    out, _, lse = o64.attn_block(q, *args)
    assert np.array_equal(out[0, 2], out[0, 0]) and np.array_equal(lse[0, 2], lse[0, 0])
    assert np.array_equal(out[0, 1, 1], out[0, 1, 0])
    assert not np.array_equal(out[0, 1, 2], out[0, 1, 0])
    perm = [1, 0, 2]
    out_p, _, lse_p = o64.attn_block(np.ascontiguousarray(q[:, perm]), *args)
    assert np.array_equal(out_p, out[:, perm]) and np.array_equal(lse_p, lse[:, perm])


def test_causal_query_block_is_one_query_per_prefix(o64):
    """Causal blocks: query token t against a python-float softmax over the row list of the cache cut
    after its own position (the block's tokens are the newest rows); the last token sees everything, so it
    equals the non-causal result, the first one does not."""
    rng = np.random.default_rng(78)
    B, Hkv, G, T, d, n, C, W = 1, 2, 2, 3, 4, 21, 4, 5
    S = B * Hkv
    K, V = rand_bits(rng, S, n, d), rand_bits(rng, S, n, d)
    q = rand_bits(rng, B, T, Hkv * G, d)
    Nc = (n - T - W) // C                                   # gated before the block's tokens arrived
    sm = o64.summarize(K, V, C, 0, Nc, kvo.AGG_MEAN)
    idx, cnt = o64.compact(np.random.default_rng(4).uniform(size=(S, Nc)), Nc, 0.5)
    args = (Hkv, K, V, C, Nc, idx, cnt, sm["ksum_b16"], sm["vsum_b16"])
    for mode, dense in ((kvo.ATTEND_SUMMARY, False), (kvo.ATTEND_RAW, False), (kvo.ATTEND_RAW, True)):
        out, _, lse = o64.attn_block(q, *args, mode, 0.4, dense=dense, causal=True)
        full, _, _ = o64.attn_block(q, *args, mode, 0.4, dense=dense, causal=False)
        assert np.array_equal(out[:, T - 1], full[:, T - 1]) and not np.array_equal(out[:, 0], full[:, 0])
        for t, hq in itertools.product(range(T), range(Hkv * G)):
            s = hq // G
            n_t = n - (T - 1 - t)
            kept = idx[s, :cnt[s]]
            if dense:
                rows_k, rows_v = [widen(K[s, r]).tolist() for r in range(n_t)], [widen(V[s, r]).tolist() for r in range(n_t)]
            else:
                if mode == kvo.ATTEND_SUMMARY:
                    rows_k = [widen(sm["ksum_b16"][s, c]).tolist() for c in kept]
                    rows_v = [widen(sm["vsum_b16"][s, c]).tolist() for c in kept]
                else:
                    rows_k = [widen(K[s, r]).tolist() for c in kept for r in range(c * C, c * C + C)]
                    rows_v = [widen(V[s, r]).tolist() for c in kept for r in range(c * C, c * C + C)]
                rows_k += [widen(K[s, r]).tolist() for r in range(Nc * C, n_t)]
                rows_v += [widen(V[s, r]).tolist() for r in range(Nc * C, n_t)]
            want, want_lse = brute_attention(widen(q[0, t, hq]).tolist(), rows_k, rows_v, 0.4)
            assert np.allclose(out[0, t, hq], want, rtol=0, atol=1e-13) and abs(lse[0, t, hq] - want_lse) <= 1e-12
