"""Shared test plumbing: builds one seeded problem, runs the oracle on it (after margin repair) and
drives the CUDA library through the same steps.  Used by the GPU parity tests and the smoke check."""
import math

import numpy as np

from oracle import kvo, margin
from paper_2509_21354_b200 import workloads as wlm

SCALE = 1.0 / math.sqrt(128.0)
ATT = {"summary": kvo.ATTEND_SUMMARY, "raw": kvo.ATTEND_RAW}


class Problem:
    """Inputs of one layer of a workload (all or a subset of its sequences) plus oracle results."""

    def __init__(self, wl, layer=0, seq_ids=None, keep=0.5, margin_eps=2e-3, tau=None):
        self.wl, self.layer = wl, layer
        self.seq_ids = list(range(wl.S)) if seq_ids is None else list(seq_ids)
        self.o64, self.o32 = kvo.Oracle("f64"), kvo.Oracle("f32")
        self.K, self.V = wlm.gen_kv(wl, layer, seqs=self.seq_ids)
        self.mlp = wlm.gen_mlp_weights(wl, layer)
        self.lstm = wlm.gen_lstm_weights(wl, layer)
        self.tau = wl.tau if tau is None else tau
        self.Nc = wl.n_stale_chunks()
        self.agg = margin.AGG_CODE[wl.agg]
        if keep is not None and self.Nc > 0:
            self.lstm["b_s"] = margin.centred_b_s(self.o64, wl, self.K, self.V, self.mlp, self.lstm, keep=keep)
        # repair on the reference oracle, then both oracles see the same repaired inputs
        self.sm64, self.sc64, self.h64, self.c64, self.redraws = margin.repair_margin(
            self.o64, wl, layer, self.K, self.V, self.mlp, self.lstm, tau=self.tau, margin=margin_eps,
            seq_ids=self.seq_ids)
        stride = max(wl.max_chunks, 1)
        S = len(self.seq_ids)
        self.sm32 = dict(ksum=np.zeros((S, stride, wl.d), np.float32), vsum=np.zeros((S, stride, wl.d), np.float32),
                         ksum_b16=np.zeros((S, stride, wl.d), np.uint16), vsum_b16=np.zeros((S, stride, wl.d), np.uint16))
        if self.Nc > 0:
            self.o32.summarize(self.K, self.V, wl.C, 0, self.Nc, self.agg, self.mlp, stride=stride, out=self.sm32)
        self.sc32, self.h32, self.c32 = self.o32.gate(self.sm32["ksum_b16"], self.sm32["vsum_b16"], 0, self.Nc, self.lstm)
        self.idx64, self.cnt64 = self.o64.compact(self.sc64, self.Nc, self.tau)
        self.idx32, self.cnt32 = self.o32.compact(self.sc32, self.Nc, self.tau)

    def oracle_attn(self, q, attend, which="f64", K=None, V=None, n_chunks=None):
        o, sm, idx, cnt = ((self.o64, self.sm64, self.idx64, self.cnt64) if which == "f64"
                           else (self.o32, self.sm32, self.idx32, self.cnt32))
        K = self.K if K is None else K
        V = self.V if V is None else V
        n_chunks = self.Nc if n_chunks is None else n_chunks
        return o.attn(q, K, V, self.wl.C, n_chunks, idx, cnt, sm["ksum_b16"], sm["vsum_b16"], ATT[attend], SCALE)

    def oracle_dense(self, q, which="f64", K=None, V=None):
        o = self.o64 if which == "f64" else self.o32
        return o.attn_dense(q, self.K if K is None else K, self.V if V is None else V, SCALE)


def bf16_ulp_distance(a_bits, b_bits):
    """distance in bf16 steps between two bit-pattern arrays (sign-magnitude -> ordered integers)"""
    def key(x):
        x = x.astype(np.int32)
        return np.where(x & 0x8000, -(x & 0x7FFF), x & 0x7FFF)
    return np.abs(key(a_bits) - key(b_bits))


def check_output(out_bits, want_real, name=""):
    """The tolerance of the benchmark definition (max-abs 2e-2, mean-abs 2e-3) plus a tighter bound that
    follows from the arithmetic: fp32 accumulation then ONE bf16 rounding (half a bf16 step, 2^-8
    relative) on top of fp32 noise."""
    got = wlm.bf16_bits_to_f32(out_bits).astype(np.float64)
    want = np.asarray(want_real, np.float64)
    err = np.abs(got - want)
    assert err.max() <= 2e-2, f"{name}: max-abs {err.max()}"
    assert err.mean() <= 2e-3, f"{name}: mean-abs {err.mean()}"
    tight = 2.0 ** -8 * np.abs(want) + 2e-5
    bad = err > tight
    assert not bad.any(), f"{name}: {bad.sum()} entries beyond one bf16 step, worst {err[bad].max()}"
    return float(err.max()), float(err.mean())


def check_output_bf16_weights(out_bits, want_real, spread, name=""):
    """The same for a kernel that rounds the softmax numerators p_i to bf16 before the product with V
    (tensor-core operand): p_i (1 + e_i), |e_i| <= 2^-8 (bf16 has 8 significant bits, so half a step is
    2^-8 relative), shifts an output by at most 2^-8 * sum_i p_i |v_i| / sum_i p_i = 2^-8 * spread, where `spread` is the same attention
    evaluated on |V| (the oracle computes it).  On top: fp32 accumulation and the one bf16 rounding
    of the result, as in check_output."""
    got = wlm.bf16_bits_to_f32(out_bits).astype(np.float64)
    want = np.asarray(want_real, np.float64)
    err = np.abs(got - want)
    assert err.max() <= 2e-2, f"{name}: max-abs {err.max()}"
    assert err.mean() <= 2e-3, f"{name}: mean-abs {err.mean()}"
    bound = 2.0 ** -8 * np.abs(want) + 2.0 ** -8 * np.asarray(spread, np.float64) + 2e-5
    bad = err > bound
    assert not bad.any(), f"{name}: {bad.sum()} entries beyond the rounding bound, worst {(err / bound).max()} x"
    # the bound is a worst case; rounding errors of independent rows mostly cancel
    assert err.mean() <= 0.25 * bound.mean(), f"{name}: mean error {err.mean()} vs mean bound {bound.mean()}"
    return float(err.max()), float(err.mean())
