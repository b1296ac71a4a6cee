#!/usr/bin/env python
"""Benchmark of the gated chunked-KV decode path (one JSON line on stdout).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfg4] [--legs ...]

The headline workload is the largest single-GPU configuration (cfg4: batch 16, 32 heads, 16512 tokens,
chunk 128, window 1024), one layer.  A *step* is one pass of the whole hot path over that layer, from scratch:
append one token to every sequence, summarise every chunk that lies outside the window, run the
LSTM gate over all of them, compact the keep list, run the gated decode attention.  `value` is
whole-job steps per second with all inputs resident in HBM; `e2e` is the same step through
kvE_decode_step_host with pinned HOST buffers (H2D of k_new, v_new, q and D2H of the output inside
the timed region).  The K-step loop is repeated R times (R in the line) so that the timed device work
lasts at least --min-timed-s; the median loop gives `value`.  Under torchrun every rank runs the same
per-GPU workload on its own batch shard (weak scaling, no data-path collective: (layer, batch, head)
units are independent).

The single-GPU run adds, in the same JSON line: `per_config` (cfg1..cfg4: from-scratch step, steady
step, every kernel in-step and alone with L2 flushed, gated vs full-cache attention; cfg3 also as 7
action tokens x 32 layers replayed from a CUDA graph), `sweep` (the stress sweep, bounded), `trigger`
(the aggregation-and-gating step for one new chunk, and the step amortised over a chunk's tokens),
`cpu_baseline` and `cpu_oracle_per_config` (the oracle on the host cores, single-threaded and OpenMP).

`--impl reference` times the CPU oracle (oracle/, as it stands) on the host cores on a bounded
sample of the same workload.
"""
import argparse
import json
import math
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2509_21354_b200 import workloads as wlm  # noqa: E402

METRIC = "gated_decode_attention_steps_per_sec"
UNIT = "steps/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
SCALE = 1.0 / math.sqrt(128.0)
def kernels_per_step(wl, Nc):
    """kernel launches of one from-scratch step: set_len, append, chunk mean [+ chunk MLP], gate projection,
    recurrence, score head, keep list, kept-row gather, attention"""
    return 9 + (1 if wl.agg == "mlp" else 0)


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def shard_batch(B_per_gpu: int, rank: int, world: int):
    """Weak scaling: every rank owns B_per_gpu sequences-batches of its own; returns the global batch
    range [lo, hi) this rank stands for (used to derive its data seed).  No collective is needed:
    the gated cache of one (layer, batch, head) never reads another's."""
    lo = rank * B_per_gpu
    return lo, lo + B_per_gpu


def paper_cost_model(wl, keep_mean):
    """The paper's own FLOPs / memory model (Sec. 3.3, Eq. 4-7) at this workload's n, W, C and measured M, for a
    LLaMA-2-7B-sized layer: context for the measured ratios, not a measurement."""
    from paper_2509_21354_b200 import cost_model as cm
    d_sum = wl.d_sum if wl.agg == "mlp" else 0
    return {"n": wl.n, "W": wl.W, "C": wl.C, "M": keep_mean,
            "memory_ratio": cm.memory_ratio(wl.n, wl.W, keep_mean),
            "speedup_incl_ffn": cm.speedup(wl.n, wl.W, keep_mean, wl.C, d_sum, wl.d_g),
            "attention_flops_ratio": cm.flops_base(wl.n) / cm.flops_kv_efficient(wl.n, wl.W, keep_mean, wl.C, d_sum, wl.d_g)}


def max_over_ranks(values, world: int, device="cuda"):
    """Element-wise maximum of a list of floats over all ranks (the slowest rank sets the time of a
    multi-GPU step).  The only collective of the benchmark; identity when world == 1."""
    if world <= 1:
        return list(values)
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


# ---------------------------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU while the timed region runs (read-only NVML)."""

    def __init__(self, index: int, period_s: float = 0.01):
        self.index, self.period, self.samples, self.reasons = index, period_s, [], set()
        self.max_mhz, self._stop, self._thr = None, threading.Event(), None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4)}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thr = threading.Thread(target=self._run, daemon=True)
            self._thr.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thr is not None:
            self._thr.join()

    def summary(self):
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ---------------------------------------------------------------------------------------------- GPU arm
def fill_cache(st, wl, seed, layer=0):
    """Synthetic cache of the workload's shape, generated on the device: N(0,1) keys and values, keys
    shifted by a per-(sequence, chunk) offset ~ N(0, key_offset_std^2); stored through kvE_append."""
    import torch
    g = torch.Generator(device="cuda").manual_seed(seed)
    slab = max(wl.C, (512 // wl.C) * wl.C)
    n_fill = wl.n - 1                      # the step appends the last token itself
    for a in range(0, n_fill, slab):
        m = min(slab, n_fill - a)
        k = torch.randn((wl.S, m, 128), generator=g, device="cuda", dtype=torch.float32)
        v = torch.randn((wl.S, m, 128), generator=g, device="cuda", dtype=torch.float32)
        if wl.key_offset_std > 0:
            nch = -(-m // wl.C)
            off = torch.randn((wl.S, nch, 128), generator=g, device="cuda", dtype=torch.float32) * wl.key_offset_std
            k += off.repeat_interleave(wl.C, dim=1)[:, :m]
        st.append(layer, k.to(torch.bfloat16).contiguous(), v.to(torch.bfloat16).contiguous())
    return g


def algorithmic_bytes(wl, Nc, keep_mean, R, attend="summary"):
    """Bytes each kernel must move per launch (per-unit figures x units; bf16 rows are 256 bytes)."""
    S, d_g = wl.S, wl.d_g
    by = {}
    by["chunk_mean"] = S * Nc * (2 * wl.C * 256 + 2 * 128 * 4)            # every stale K and V row once; fp32 means out
    by["chunk_mlp"] = S * Nc * 2 * (128 * 4 + 128 * 4 + 128 * 2)          # means in, fp32 + bf16 summaries out
    by["gate_proj"] = S * Nc * (2 * 256 + 4 * d_g * 4)                    # bf16 summaries in, fp32 P out
    by["gate_rnn"] = S * Nc * (4 * d_g * 4 + 4)                           # P in, scores out
    by["compact"] = S * (Nc * 4 + Nc * 4 + 4)
    rows_per_kept = wl.C if attend == "raw" else 1                          # a kept chunk: its C raw rows, or its one summary row
    by["attn_gated"] = S * (2 * (R + keep_mean * rows_per_kept) * 256 + 2 * 256)   # retained rows of K and V once (+ q, out)
    by["attn_dense"] = S * (2 * wl.n * 256 + 2 * 256)
    return by


def algorithmic_flops(wl, Nc):
    """Floating-point operations of the contraction-shaped kernels as the method defines them (one
    multiply-add = 2; the exact-split planes the kernels use on top are not counted)."""
    S, d_g, d = wl.S, wl.d_g, 128
    fl = {"gate_proj": S * Nc * 2 * (2 * d) * (4 * d_g),
          "gate_rnn": S * Nc * (2 * d_g * 4 * d_g + 2 * d_g)}
    if wl.agg == "mlp":
        fl["chunk_mlp"] = 2 * S * Nc * 2 * (d * wl.d_sum + wl.d_sum * d)
    return fl


def query_block_leg(wl, hbm, tensor_peak, peak_kind, seed):
    """kvE_decode_attn_block on the workload's geometry with grouped query heads (the 32 query heads on
    8 KV heads of Sec. 4.1) and 7 query tokens decoded together: gated and full-cache attention, each
    launch timed alone with L2 flushed.  Mean aggregator (the summaries only feed the keep list here)."""
    import torch
    from paper_2509_21354_b200 import binding as b
    Hkv, G, T = 8, wl.H // 8, 7
    g = wl.small(H=Hkv, agg="mean", d_sum=0)
    st = b.Store(B=g.B, H=Hkv, Hq=Hkv * G, C_=g.C, W=g.W, max_tokens=g.n + g.C, d_g=g.d_g, agg="mean", attend="summary",
                 page_perm="random", seed=seed, max_query_tokens=T)
    gen = fill_cache(st, g, seed)
    lstm = wlm.gen_lstm_weights(g)
    lw = b.LstmWeights(lstm)
    n = g.n - 1
    Nc = g.n_stale_chunks(n)
    st.summarize_chunks(0, 0, Nc, None)
    st.gate(0, 0, Nc, lw)
    torch.cuda.synchronize()
    sc = st.scores[0, :, :Nc].double().clamp(1e-9, 1 - 1e-9)
    lw.set_b_s(float(-torch.median(torch.log(sc / (1 - sc))).item()) + lstm["b_s"])      # keep about half
    st.gate(0, 0, Nc, lw)
    st.compact(0, g.tau)
    torch.cuda.synchronize()
    keep = st.keep_cnt[0].float().mean().item()
    q = torch.randn((g.B, T, Hkv * G, 128), generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    out = torch.empty_like(q)
    flush = Flusher()
    st.profile(True)
    res = {"what": f"kvE_decode_attn_block: {T} query tokens x {Hkv * G} query heads on {Hkv} KV heads, B={g.B}, n={n}; "
                   "tcgen05 kernel, one launch timed alone, L2 flushed",
           "query_rows_per_kv_head": T * G, "kept_chunks_mean": keep}
    for name, dense, rows in (("gated", False, n - Nc * g.C + keep), ("dense", True, n)):
        ts = []
        for i in range(12):
            flush()
            st.decode_attn_block(0, q, dense=dense, out=out)
            torch.cuda.synchronize()
            if i >= 2:
                ts.append(st.profile_read()["attn_block"])
        us = float(np.median(ts))
        by = g.S * rows * 512                                  # every retained K and V row once per KV head
        fl = 4 * 128 * T * G * g.S * rows                      # Q K^T and P V
        res[name] = {"us": us, "kv_bytes": int(by), "GB/s": by / us / 1e3, "frac_of_hbm_peak": by / us / 1e3 / hbm,
                     "TFLOP/s": fl / us / 1e6, "frac_of_bf16_peak": fl / us / 1e6 / tensor_peak,
                     "peak_kind": f"of {peak_kind}"}
    assert st.poll_status() == 0
    res["gated_vs_dense"] = res["dense"]["us"] / res["gated"]["us"]
    return res


def host_free_loop_leg(wl, attend, seed, steady_ms, replays=6):
    """Sec. 3.3 with the host out of the loop: ONE captured graph = C decode steps (kvE_decode_step) + the trigger in its
    device-positioned form (kvE_refresh_next: the chunk that has just left the window is summarised, gated and appended
    to the keep list, its index found on the device).  Every replay moves one layer C tokens ahead, trigger included;
    the graph is replayed across several triggers without a new capture."""
    import torch
    rig = Rig(wl, attend, seed, extra_tokens=(replays + 3) * wl.C)
    st, S, C_ = rig.st, wl.S, wl.C
    # start on a chunk boundary of the stale range: C more tokens make exactly one chunk leave the window
    n_start = wl.W + (rig.Nc + 1) * C_
    fillk = torch.randn((S, n_start - wl.n, 128), generator=rig.gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    st.append(0, fillk, fillk)
    st.refresh(0, rig.aw, rig.lw, wl.tau)
    torch.cuda.synchronize()
    k_in = torch.randn((C_, S, 128), generator=rig.gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    q_in = torch.randn((C_, S, 128), generator=rig.gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    out = torch.empty_like(q_in)
    graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for i in range(C_):
                st.decode_step(0, k_in[i], k_in[i], q_in[i], out[i], n_reserve=(replays + 2) * C_)
            st.refresh_next(0, rig.aw, rig.lw, wl.tau)
    torch.cuda.current_stream().wait_stream(side)
    st.adopt_device_state(0)
    gated0 = st.layer_state(0)["n_gated"]
    graph.replay()                                         # warm-up: one replay = C tokens + one trigger
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(replays):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    assert st.poll_status() == 0
    st.adopt_device_state(0)
    state = st.layer_state(0)
    assert state["n_gated"] == gated0 + 1 + replays and state["n_tokens"] == n_start + (1 + replays) * C_
    ms_replay = e0.elapsed_time(e1) / replays
    st.close()
    return {"what": f"one CUDA graph of C = {C_} x kvE_decode_step + kvE_refresh_next (trigger positioned on the device), one layer, "
                    f"replayed {replays} times across as many triggers, no host work besides the replay",
            "ms_per_replay": ms_replay, "us_per_token_trigger_included": 1e3 * ms_replay / C_,
            "tokens_per_s": 1e3 * C_ / ms_replay, "steady_us_per_token_without_trigger": 1e3 * steady_ms,
            "triggers_crossed": replays, "launches_per_replay": C_ + kernels_per_trigger(wl)}


def kernels_per_trigger(wl):
    """launches of the device-positioned trigger: chunk mean (+ MLP) + the gate step"""
    return 3 if wl.agg == "mlp" else 2


def graph_tick_leg(wl, n_layers, seed, replays=20, mem_cap=40e9, fused=True):
    """The decode loop of a whole model between two gate triggers: per token, for each of n_layers layers
    append the new token at the device-held length (kvE_append_next) and run the gated attention; all
    layers captured once in a CUDA graph, every replay advancing by one token.  Compared with the
    same calls issued one by one.  fused: kvE_decode_step (append + attention in one launch) instead of the two calls."""
    import torch
    from paper_2509_21354_b200 import binding as b
    g = wl.small(agg="mean", d_sum=0)                      # the aggregator only feeds the keep list here
    per_layer = g.S * (g.n + g.C) * 512 * 1.1
    n_layers = max(1, min(n_layers, int(mem_cap // per_layer)))
    st = b.Store(B=g.B, H=g.H, C_=g.C, W=g.W, max_tokens=g.n + g.C, d_g=g.d_g, agg="mean", attend="summary",
                 n_layers=n_layers, page_perm="random", seed=seed)
    lstm = wlm.gen_lstm_weights(g)
    lw = b.LstmWeights(lstm)
    Nc = g.n_stale_chunks(g.n - 1)                         # the cache holds n - 1 tokens; the tick appends the n-th
    gen = None
    for L in range(n_layers):
        gen = fill_cache(st, g, seed + L, layer=L)
        st.summarize_chunks(L, 0, Nc, None)
        st.gate(L, 0, Nc, lw)
        if L == 0:
            torch.cuda.synchronize()
            sc = st.scores[0, :, :Nc].double().clamp(1e-9, 1 - 1e-9)
            lw.set_b_s(float(-torch.median(torch.log(sc / (1 - sc))).item()) + lstm["b_s"])
            st.gate(L, 0, Nc, lw)
        st.compact(L, g.tau)
    torch.cuda.synchronize()
    S = g.S
    rnd = lambda: torch.randn((n_layers, S, 128), generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    k_new, v_new, q = rnd(), rnd(), rnd()
    out = torch.empty_like(q)

    budget = 3 + replays                                   # tokens one timed phase appends per layer
    assert 2 * budget + 2 < g.C, "the loop must stay between two gate triggers"

    def rewind():
        for L in range(n_layers):
            st.set_len(L, g.n - 1)

    def tick():                                            # every call / replay appends the NEXT token of every layer
        for L in range(n_layers):
            if fused:
                st.decode_step(L, k_new[L], v_new[L], q[L], out[L], n_reserve=2 * budget)
            else:
                st.append_next(L, k_new[L], v_new[L], n_reserve=2 * budget)
                st.decode_attn(L, q[L], out[L])

    tick()
    torch.cuda.synchronize()
    eager_out = out.clone()
    rewind()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            tick()
    torch.cuda.current_stream().wait_stream(side)
    out.zero_()
    graph.replay()
    torch.cuda.synchronize()
    same = bool(torch.equal(out, eager_out))
    calls = "kvE_decode_step: append at the device-held length + gated attention in one launch" if fused else \
        "kvE_append_next at the device-held length, then kvE_decode_attn"
    res = {"what": f"decode loop over {n_layers} layers between two gate triggers (per layer and token: {calls}), captured once "
                   "in a CUDA graph and replayed - every replay appends the next token - vs the same calls issued one by one",
           "n_layers": n_layers, "launches_per_layer_and_token": 1 if fused else 2, "graph_first_tick_equals_eager": same}
    for name, fn in (("eager", tick), ("graph", graph.replay)):
        rewind()
        for _ in range(3):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(replays):
            fn()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / replays
        res[name] = {"ms_per_tick": ms, "us_per_layer": ms * 1e3 / n_layers, "ticks_per_s": 1e3 / ms}
        assert int(st.seq_len[0, 0]) == g.n - 1 + budget   # the loop really advanced
    assert st.poll_status() == 0
    res["kv_bytes_per_tick"] = int(n_layers * S * (g.n - Nc * g.C + st.keep_cnt.float().mean().item()) * 512)
    res["GB/s_graph"] = res["kv_bytes_per_tick"] / (res["graph"]["ms_per_tick"] * 1e-3) / 1e9
    return res


# ---------------------------------------------------------------------------------------------- one workload on the device
class Rig:
    """One layer of a workload resident on the device: the cache holds n - 1 tokens, the gate's head bias is
    tuned so that about `keep` of the stale chunks are retained (deterministic given the seed)."""

    def __init__(self, wl, attend, seed, extra_tokens=0, keep=0.5):
        import torch
        from paper_2509_21354_b200 import binding as b
        self.wl, self.attend, self.b = wl, attend, b
        self.st = st = b.Store(B=wl.B, H=wl.H, C_=wl.C, W=wl.W, max_tokens=wl.n + wl.C + extra_tokens, d_g=wl.d_g, agg=wl.agg,
                               d_sum=wl.d_sum, attend=attend, page_perm="random", seed=seed)
        self.gen = g = fill_cache(st, wl, seed)
        mlp, lstm = wlm.gen_mlp_weights(wl), wlm.gen_lstm_weights(wl)
        self.aw = b.AggWeights(mlp) if mlp is not None else None
        self.lw = b.LstmWeights(lstm)
        S = self.S = wl.S
        rnd = lambda: torch.randn((S, 128), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16).contiguous()
        self.k_new, self.v_new, self.q = rnd(), rnd(), rnd()
        self.k3, self.v3 = self.k_new.view(S, 1, 128), self.v_new.view(S, 1, 128)
        self.out = torch.empty_like(self.q)
        self.n0 = wl.n
        self.Nc = wl.n_stale_chunks(wl.n)
        self.R = wl.n - self.Nc * wl.C
        self.step_full()
        torch.cuda.synchronize()
        if self.Nc > 0:
            sc = st.scores[0, :, :self.Nc].double().clamp(1e-9, 1 - 1e-9)
            logit = torch.log(sc / (1 - sc))
            self.lw.set_b_s(float(-torch.quantile(logit.flatten()[:1 << 20], 1.0 - keep).item()) + lstm["b_s"])
        self.step_full()
        torch.cuda.synchronize()
        assert st.poll_status() == 0
        self.keep_mean = st.keep_cnt[0].float().mean().item()
        self.rows_per_kept = wl.C if attend == "raw" else 1
        self.n_eff = self.R + self.keep_mean * self.rows_per_kept

    def step_full(self):
        """the whole hot path from scratch: roll the last token back, append it, summarise every stale
        chunk, gate them all, compact, gated attention"""
        st, wl = self.st, self.wl
        st.set_len(0, self.n0 - 1)
        st.append(0, self.k3, self.v3)
        st.summarize_chunks(0, 0, self.Nc, self.aw)
        st.gate(0, 0, self.Nc, self.lw)
        st.compact(0, wl.tau)
        st.decode_attn(0, self.q, self.out)

    def step_steady(self):
        """the step between two gate triggers (token n0 + 1: no chunk leaves the window, the keep list stands):
        roll back, then append + gated attention in one launch (kvE_decode_step)"""
        st = self.st
        st.set_len(0, self.n0)
        st.decode_step(0, self.k_new, self.v_new, self.q, self.out)

    def step_steady_two_launches(self):
        st = self.st
        st.set_len(0, self.n0)
        st.append(0, self.k3, self.v3)
        st.decode_attn(0, self.q, self.out)


def time_loop(fn, iters, repeats=1, sync=None):
    """`repeats` loops of `iters` calls, each loop bracketed by CUDA events on the current stream (and by `sync`
    = barrier + device synchronise when given); list of milliseconds per loop"""
    import torch
    sync = sync or torch.cuda.synchronize
    out = []
    for _ in range(repeats):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sync()
        e0.record()
        for _ in range(iters):
            fn()
        e1.record()
        sync()
        out.append(e0.elapsed_time(e1))
    return out


def iters_for(fn, target_s=0.15, lo=10, hi=400):
    """how many calls of fn fill about target_s (pilot of 5 calls after 3 warm-up calls)"""
    for _ in range(3):
        fn()
    ms = time_loop(fn, 5)[0] / 5
    return int(min(hi, max(lo, target_s * 1e3 / max(ms, 1e-3))))


class Flusher:
    """Leaves L2 (126 MB) cold AND clean before the next launch: writes a 256 MB buffer (every line of the launch's
    data is gone), then reads another 256 MB buffer (the dirty lines of the write are written back now, not under the
    timed kernel's first reads, where they would be billed to it as extra DRAM traffic)."""

    def __init__(self):
        import torch
        self.wbuf = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
        self.rbuf = torch.zeros(256 << 20, dtype=torch.uint8, device="cuda")

    def __call__(self):
        self.wbuf.fill_(1)
        self.rbuf.max()

    def write_only(self):
        """the cruder flush: L2 cold but full of dirty lines, whose write-back the next launch's first reads pay for"""
        self.wbuf.fill_(1)


def copy_us(total_bytes, flush):
    """a plain device copy that moves total_bytes (read + write), timed like the kernels: L2 flushed, events"""
    import torch
    src = torch.empty(max(1, int(total_bytes) // 2), dtype=torch.uint8, device="cuda")
    dst = torch.empty_like(src)
    ts = []
    for i in range(8):
        flush()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        dst.copy_(src)
        e1.record()
        torch.cuda.synchronize()
        if i >= 2:
            ts.append(e0.elapsed_time(e1) * 1e3)
    return float(np.median(ts))


def kernel_times(rig, flush, n_in_step=20, n_cold=8):
    """microseconds per kernel from the library's own event pairs: inside the from-scratch step (caches as the
    step leaves them) and with L2 flushed before the call that launches the kernel"""
    st, b = rig.st, rig.b
    st.profile(True)
    in_step = {k: [] for k in b.KERNEL_IDS}
    for _ in range(n_in_step):
        rig.step_full()
        for k, v in st.profile_read().items():
            if v is not None and k not in ("attn_dense", "attn_block"):
                in_step[k].append(v)
    cold = {k: [] for k in ("chunk_mean", "chunk_mlp", "gate_proj", "gate_rnn", "compact", "attn", "attn_dense")}
    for _ in range(n_cold):
        # each call after a flush; the kernels a call launches back to back share what the first one left in L2
        flush(); st.summarize_chunks(0, 0, rig.Nc, rig.aw); r = st.profile_read()
        cold["chunk_mean"].append(r["chunk_mean"])
        if r["chunk_mlp"] is not None:
            cold["chunk_mlp"].append(r["chunk_mlp"])
        flush(); st.gate(0, 0, rig.Nc, rig.lw); r = st.profile_read()
        cold["gate_proj"].append(r["gate_proj"]); cold["gate_rnn"].append(r["gate_rnn"])
        flush(); st.compact(0, rig.wl.tau); cold["compact"].append(st.profile_read()["compact"])
        flush(); st.decode_attn(0, rig.q, rig.out); cold["attn"].append(st.profile_read()["attn"])
        flush(); st.decode_attn_dense(0, rig.q, rig.out); cold["attn_dense"].append(st.profile_read()["attn_dense"])
    cold["attn_dirty_l2"] = []
    for _ in range(n_cold):
        flush.write_only(); st.decode_attn(0, rig.q, rig.out); cold["attn_dirty_l2"].append(st.profile_read()["attn"])
    st.profile(False)
    rig.step_full()
    med = lambda v: float(np.median(v))
    return ({k: med(v) for k, v in in_step.items() if v}, {k: med(v) for k, v in cold.items() if v})


def measure_config(rig, peaks, peak_kind, flush, headline=False):
    """Everything the report gives per configuration: the from-scratch step, the steady step, every kernel in-step
    and L2-flushed with its algorithmic bytes / flops and fractions of the measured peaks, gated vs dense."""
    import torch
    wl, st = rig.wl, rig.st
    hbm = peaks["hbm_gbs"]
    tensor_peak = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
    res = {"workload": wl.name, "S": wl.S, "n": wl.n, "C": wl.C, "W": wl.W, "attend": rig.attend, "stale_chunks": rig.Nc,
           "kept_chunks_mean": rig.keep_mean, "n_eff": rig.n_eff, "memory_ratio_n_over_n_eff": wl.n / rig.n_eff}
    if not headline:
        it = iters_for(rig.step_full)
        ms = float(np.median(time_loop(rig.step_full, it, 3))) / it
        res["full_step"] = {"ms": ms, "steps_per_s": 1e3 / ms, "iters": it, "repeats": 3}
        it = iters_for(rig.step_steady)
        ms = float(np.median(time_loop(rig.step_steady, it, 3))) / it
        res["steady_step"] = {"ms": ms, "steps_per_s": 1e3 / ms, "iters": it, "repeats": 3}
        rig.step_full()
    us_in, us_cold = kernel_times(rig, flush)
    by = algorithmic_bytes(wl, rig.Nc, rig.keep_mean, rig.R, rig.attend)
    by_kernel = {"append": wl.S * 4 * 256, "chunk_mean": by["chunk_mean"], "chunk_mlp": by["chunk_mlp"],
                 "gate_proj": by["gate_proj"], "gate_rnn": by["gate_rnn"], "compact": by["compact"],
                 "attn": by["attn_gated"], "attn_dense": by["attn_dense"]}
    fl = algorithmic_flops(wl, rig.Nc)
    kern = {}
    us_attn_dirty = us_cold.pop("attn_dirty_l2")
    for k in sorted(set(us_in) | set(us_cold)):
        e = {"bytes": by_kernel[k]}
        if k in us_in:
            e["us"] = us_in[k]
            e["GB/s"] = by_kernel[k] / us_in[k] / 1e3
            e["frac_of_hbm_peak"] = e["GB/s"] / hbm
        if k in us_cold:
            e["us_l2_flushed"] = us_cold[k]
            e["GB/s_l2_flushed"] = by_kernel[k] / us_cold[k] / 1e3
            e["frac_of_hbm_peak_l2_flushed"] = e["GB/s_l2_flushed"] / hbm
        if k in fl:
            t = us_in.get(k, us_cold.get(k))
            e["flops"] = fl[k]
            e["TFLOP/s"] = fl[k] / t / 1e6
            e["frac_of_bf16_peak"] = e["TFLOP/s"] / tensor_peak
        kern[k] = e
    res["kernels"] = kern
    g_us, d_us = us_cold["attn"], us_cold["attn_dense"]
    cg, cd = copy_us(by["attn_gated"], flush), copy_us(by["attn_dense"], flush)
    res["attention_vs_dense"] = {
        "note": "attention kernels alone, L2 flushed (cold and clean: a written buffer, then a read one) before every launch; "
                "gated_us_after_write_only_flush = the same launch on an L2 full of dirty lines",
        "gated_us": g_us, "dense_us": d_us, "speedup": d_us / g_us, "gated_us_after_write_only_flush": us_attn_dirty,
        "gated_frac_of_measured_peak_after_write_only_flush": by["attn_gated"] / us_attn_dirty / 1e3 / hbm,
        "kv_bytes_gated": by["attn_gated"], "kv_bytes_dense": by["attn_dense"],
        "gated_GB/s": by["attn_gated"] / g_us / 1e3, "dense_GB/s": by["attn_dense"] / d_us / 1e3,
        "gated_frac_of_measured_peak": by["attn_gated"] / g_us / 1e3 / hbm,
        "dense_frac_of_measured_peak": by["attn_dense"] / d_us / 1e3 / hbm,
        "gated_frac_of_nominal_8TBps": by["attn_gated"] / g_us / 1e3 / 8000.0,
        "dense_frac_of_nominal_8TBps": by["attn_dense"] / d_us / 1e3 / 8000.0,
        "size_matched_copy": {"note": "a plain torch device copy moving the same number of bytes (read + write), same timing "
                                      "method: what this transfer size allows on this GPU",
                              "gated_bytes_copy_us": cg, "dense_bytes_copy_us": cd,
                              "gated_time_over_copy": g_us / cg, "dense_time_over_copy": d_us / cd},
        "peak_kind": f"of {peak_kind}"}
    assert st.poll_status() == 0
    return res


def trigger_leg(wl, attend, seed, steady_ms, n_triggers=24):
    """The aggregation-and-gating step of Sec. 3.3 as it happens while decoding: C more tokens have arrived, ONE chunk
    per sequence leaves the window; it is summarised, takes one LSTM step with the carried (h, c), and joins the keep
    list.  Timed per trigger (events around the calls), n_triggers triggers in a row on a growing cache, in two forms:
    kvE_summarize_chunks + kvE_gate_next (the LSTM step, the score and the keep-list append in one launch) and the
    general calls kvE_summarize_chunks + kvE_gate + kvE_compact (projection GEMM, recurrence, score head, compaction
    and kept-row gather as separate launches)."""
    import torch
    out = {}
    for form in ("gate_next", "general"):
        rig = Rig(wl, attend, seed, extra_tokens=(n_triggers + 1) * wl.C)
        st = rig.st
        kC = torch.randn((wl.S, wl.C, 128), generator=rig.gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        vC = torch.randn((wl.S, wl.C, 128), generator=rig.gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        ts = []
        for i in range(n_triggers):
            ready = st.append(0, kC, vC)
            assert ready == 1
            t = rig.Nc + i
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            st.summarize_chunks(0, t, t + 1, rig.aw)
            if form == "gate_next":
                st.gate_next(0, rig.lw, wl.tau)
            else:
                st.gate(0, t, t + 1, rig.lw)
                st.compact(0, wl.tau)
            e1.record()
            torch.cuda.synchronize()
            if i >= 4:
                ts.append(e0.elapsed_time(e1))
        assert st.poll_status() == 0
        out[form] = float(np.median(ts))
        n_timed = len(ts)
        st.close()
    trig = out["gate_next"]
    return {"what": "one chunk per sequence leaves the window: kvE_summarize_chunks(t, t+1) + kvE_gate_next (one LSTM step with "
                    "carried state, score, keep-list append: one launch), per layer; the amortised step spreads it over the C "
                    "tokens between two triggers",
            "trigger_ms": trig, "trigger_ms_with_gate_and_compact": out["general"], "triggers_timed": n_timed,
            "steady_ms": steady_ms, "C": wl.C,
            "amortised_ms_per_token": (wl.C * steady_ms + trig) / wl.C,
            "amortised_steps_per_s": 1e3 * wl.C / (wl.C * steady_ms + trig),
            "trigger_share_of_amortised_step": trig / (wl.C * steady_ms + trig)}


def token_mlp_leg(wl, peaks, peak_kind, flush, seed):
    """Eq. 2 taken literally (KVE_AGG_TOKEN_MLP): the aggregator MLP on EVERY stale token, outputs mean-pooled, on the
    workload's geometry.  The first layer is a tcgen05 contraction [tokens, 128] x [128, d_sum]; the kernel is bound by
    the activation arithmetic of its epilogue (erf GELU: about 21 FP32-pipe instructions and 2 special-function ops per
    activation, plus the pooling shuffles), so its roofline is the FP32 issue rate: SMs x 128 lanes x clock / 21."""
    import torch
    d_sum = 256
    g = wl.small(agg="token_mlp", d_sum=d_sum)
    rig = Rig(g, "summary", seed)
    st = rig.st
    st.profile(True)
    ts = []
    for _ in range(6):
        flush()
        st.summarize_chunks(0, 0, rig.Nc, rig.aw)
        ts.append(st.profile_read()["chunk_mlp"])
    st.profile(False)
    us = float(np.median(ts[1:]))
    assert st.poll_status() == 0
    tokens = g.S * rig.Nc * g.C
    flops = 2 * tokens * 2 * 128 * d_sum + 2 * g.S * rig.Nc * 2 * d_sum * 128
    acts = 2 * tokens * d_sum
    kv_bytes = tokens * 512
    sm_mhz = peaks.get("sm_max_mhz", 1965.0)
    alu_peak = 148 * 128 * sm_mhz * 1e6 / 21.0          # activations per second if the FP32 pipe did nothing else
    tensor_peak = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
    res = {"what": f"kvE_summarize_chunks with the per-token MLP aggregator (d_sum {d_sum}) over all {rig.Nc} stale chunks of "
                   f"{g.S} sequences ({tokens} tokens per side), both kernels, L2 flushed",
           "us": us, "stale_kv_bytes": kv_bytes, "GB/s": kv_bytes / us / 1e3, "frac_of_hbm_peak": kv_bytes / us / 1e3 / peaks["hbm_gbs"],
           "flops": flops, "TFLOP/s": flops / us / 1e6, "frac_of_bf16_peak": flops / us / 1e6 / tensor_peak,
           "activations": acts, "Gact/s": acts / us / 1e3,
           "roofline": {"bound": "alu", "achieved": acts / us / 1e3, "peak": alu_peak / 1e9, "unit": "Gact/s",
                        "frac": acts / us / 1e3 / (alu_peak / 1e9),
                        "peak_kind": "derived: 148 SMs x 128 FP32 lanes x max SM clock / 21 instructions per activation"},
           "peak_kind": f"of {peak_kind}"}
    st.close()
    return res


SWEEP_GEOMETRIES = [  # (B, n, C): every corner of the grid, then a diagonal through its middle
    (1, 2048, 32), (1, 2048, 256), (1, 32768, 32), (1, 32768, 256),
    (64, 2048, 32), (64, 2048, 256), (64, 32768, 32), (64, 32768, 256),
    (2, 4096, 64), (4, 8192, 128), (8, 16384, 64), (16, 8192, 128), (32, 4096, 64), (16, 32768, 128)]
SWEEP_KEEPS = {"corner": (0.25, 1.0), "diagonal": (0.5, 0.75)}


def sweep_leg(peaks, peak_kind, flush, seed, mem_cap=120e9):
    """cfg5: a bounded walk over workloads.sweep_points() - all 16 corners of (batch 1/64, context 2k/32k, chunk
    32/256, keep 0.25/1.0) plus a diagonal - 32 heads, W = 512, single layer.  Per point: dense attention, gated
    attention with kept chunks as summary rows and as raw rows, each launch alone with L2 flushed: microseconds,
    steps/s, KV bytes, GB/s, fraction of the measured HBM peak.  The keep ratio is set by thresholding the scores at
    the matching quantile."""
    import torch
    from paper_2509_21354_b200 import binding as b
    hbm = peaks["hbm_gbs"]
    grid = {(w.B, w.n, w.C, k) for w, k in wlm.sweep_points()}
    points, skipped = [], []
    for gi, (B, n, Cs) in enumerate(SWEEP_GEOMETRIES):
        keeps = SWEEP_KEEPS["corner" if gi < 8 else "diagonal"]
        wl = wlm.Workload(f"sweep_b{B}_n{n}_c{Cs}", B=B, H=32, n=n, C=Cs, W=512, d_g=256, agg="mean", key_offset_std=0.5)
        assert all((B, n, Cs, k) in grid for k in keeps)
        need = wl.S * (n + Cs) * 512 * 1.35 + wl.S * wl.max_chunks * 4096 * 1.1
        if need > mem_cap:
            skipped.append({"B": B, "n": n, "C": Cs, "why": f"needs {need / 1e9:.0f} GB on the device"})
            continue
        st = b.Store(B=B, H=32, C_=Cs, W=512, max_tokens=n + Cs, d_g=256, agg="mean", attend="summary", page_perm="random",
                     seed=seed + gi)
        gen = fill_cache(st, wl.small(n=n + 1), seed + gi)               # fill_cache leaves the last token out
        lw = b.LstmWeights(wlm.gen_lstm_weights(wl))
        Nc = wl.n_stale_chunks()
        st.summarize_chunks(0, 0, Nc, None)
        st.gate(0, 0, Nc, lw)
        torch.cuda.synchronize()
        sc = st.scores[0, :, :Nc].flatten()
        q = torch.randn((wl.S, 128), generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        out = torch.empty_like(q)
        st.profile(True)

        def timed(fn, key):
            ts = []
            for i in range(7):
                flush()
                fn(0, q, out)
                ts.append(st.profile_read()[key])
            return float(np.median(ts[2:]))

        d_us = timed(st.decode_attn_dense, "attn_dense")
        d_by = wl.S * (2 * n * 256 + 512)
        for keep in keeps:
            tau = 0.0 if keep >= 1.0 else float(torch.quantile(sc[:1 << 22].float(), 1.0 - keep).item())
            st.compact(0, tau)
            torch.cuda.synchronize()
            M = st.keep_cnt[0].float().mean().item()
            pt = {"B": B, "n": n, "C": Cs, "keep": keep, "kept_chunks_mean": M, "stale_chunks": Nc,
                  "dense": {"us": d_us, "steps_per_s": 1e6 / d_us, "kv_bytes": d_by, "GB/s": d_by / d_us / 1e3,
                            "frac_of_hbm_peak": d_by / d_us / 1e3 / hbm}}
            for attend, per in (("summary", 1), ("raw", Cs)):
                st.set_attend(attend)
                us = timed(st.decode_attn, "attn")
                by = wl.S * (2 * (n - Nc * Cs + M * per) * 256 + 512)
                pt["gated_" + attend] = {"us": us, "steps_per_s": 1e6 / us, "kv_bytes": int(by), "GB/s": by / us / 1e3,
                                         "frac_of_hbm_peak": by / us / 1e3 / hbm, "speedup_vs_dense": d_us / us}
            points.append(pt)
        assert st.poll_status() == 0
        st.close()
        del st, q, out, sc
        torch.cuda.empty_cache()
    big = [p for p in points if p["gated_summary"]["kv_bytes"] >= 256e6]
    return {"what": "stress sweep (cfg5), bounded: 16 corner points + a diagonal; attention launches alone, L2 flushed; "
                    f"fractions of the {peak_kind} HBM copy figure",
            "n_points": len(points), "points": points, "skipped": skipped,
            "gated_summary_min_frac_at_256MB_or_more": min((p["gated_summary"]["frac_of_hbm_peak"] for p in big), default=None)}


def action_step_leg(seed):
    """cfg3 in its stated form: one control step = 7 action tokens appended autoregressively, each through all 32
    layers (append at the device-held length + gated attention per layer and token), the 32-layer tick captured in a
    CUDA graph and replayed 7 times; with kvE_decode_step (one launch per layer and token) and, for comparison, with the two
    separate calls."""
    wl = wlm.CFG3
    two = graph_tick_leg(wl, wl.n_layers, seed, replays=wl.n_append, fused=False)
    r = graph_tick_leg(wl, wl.n_layers, seed, replays=wl.n_append)
    ms = r["graph"]["ms_per_tick"] * wl.n_append
    return {"what": f"{wl.n_append} action tokens x {r['n_layers']} layers, graph-replayed (B={wl.B}, H={wl.H}, n={wl.n})",
            "ms_per_action_step": ms, "action_steps_per_s": 1e3 / ms, "attention_calls_per_action_step": wl.n_append * r["n_layers"],
            "us_per_layer_and_token": r["graph"]["us_per_layer"], "eager_ms_per_action_step": r["eager"]["ms_per_tick"] * wl.n_append,
            "kv_bytes_per_token": r["kv_bytes_per_tick"], "GB/s": r["GB/s_graph"], "graph_first_tick_equals_eager": r["graph_first_tick_equals_eager"],
            "launches_per_layer_and_token": 1,
            "with_two_launches_per_layer_and_token": {"ms_per_action_step": two["graph"]["ms_per_tick"] * wl.n_append,
                                                      "us_per_layer_and_token": two["graph"]["us_per_layer"]}}


def run_ours(args, rank, world, local_rank):
    import torch
    import torch.distributed as dist

    torch.cuda.set_device(local_rank)
    wl = wlm.CONFIGS[args.workload].small(n_layers=1)
    lo, _ = shard_batch(wl.B, rank, world)
    seed = 1000 + lo
    rig = Rig(wl, args.attend, seed)
    st, S = rig.st, wl.S

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- the headline: K from-scratch steps, repeated so that the timed work lasts long enough -------------
    for _ in range(args.warmup):
        rig.step_full()
    pilot = time_loop(rig.step_full, 3, 1, barrier)[0] / 3                       # ms per step
    repeats = int(min(50, max(1, math.ceil(args.min_timed_s * 1e3 / max(pilot * args.steps, 1e-6)))))
    repeats = int(max_over_ranks([repeats], world)[0])
    with ClockSampler(local_rank) as clk:
        loops = time_loop(rig.step_full, args.steps, repeats, barrier)
    assert st.poll_status() == 0
    loops = [max_over_ranks([t], world)[0] for t in loops] if world > 1 else loops
    ms_total = float(np.median(loops))

    # ---- steady-state decode step (between two gate triggers): append one token, gated attention ----
    for _ in range(3):
        rig.step_steady()
    ms_steady = float(np.median(max_over_ranks(time_loop(rig.step_steady, args.steps, min(repeats, 5), barrier), world)))
    assert st.poll_status() == 0
    rig.step_full()                      # back to the state and output of a full step
    torch.cuda.synchronize()
    ms_two = float(np.median(max_over_ranks(time_loop(rig.step_steady_two_launches, args.steps, min(repeats, 3), barrier), world)))
    steady = {"what": "append + gated attention only (summaries, gate and keep list reused: the state between two triggers), "
                      "through kvE_decode_step (one launch)",
              "value": world * args.steps / (ms_steady * 1e-3), "unit": UNIT, "ms_per_step": ms_steady / args.steps,
              "ms_per_step_with_separate_append_and_attention": ms_two / args.steps}

    # ---- end to end: the same step through kvE_decode_step_host, host buffers, copies timed ----
    hk, hv, hq = (t.cpu().pin_memory() for t in (rig.k_new, rig.v_new, rig.q))
    hout = torch.zeros((S, 128), dtype=torch.bfloat16).pin_memory()

    # every step: H2D of its inputs and D2H of its result inside the timed region; steps are enqueued
    # back to back (kvE_decode_step_host_async) and the stream is waited for once, at the end
    def step_e2e():
        st.set_len(0, rig.n0 - 1)
        st.decode_step_host(0, hk, hv, hq, hout, rig.aw, rig.lw, wl.tau, from_scratch=True, wait=False)

    for _ in range(3):
        step_e2e()
    e2e_runs = []
    for _ in range(min(repeats, 5)):
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.steps):
            step_e2e()
        barrier()
        e2e_runs.append(time.perf_counter() - t0)
    e2e_s = float(np.median(max_over_ranks(e2e_runs, world)))
    # the same step through the separate device-side calls: the host-buffer path must give the same output
    rig.step_full()
    torch.cuda.synchronize()
    e2e_diff = float((hout.cuda().float() - rig.out.float()).abs().max().item())
    e2e_ref = float(rig.out.float().abs().max().item())
    if rank != 0:
        return None

    # ---- rank 0: per-kernel figures, rooflines, and (single GPU only) the other configurations and legs ----
    peaks, peak_kind = load_peaks()
    hbm = peaks["hbm_gbs"]
    tensor_peak = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])     # kernels timed inside a long step
    flush = Flusher()
    head = measure_config(rig, peaks, peak_kind, flush, headline=True)
    kern = head["kernels"]
    in_step = {k: v for k, v in kern.items() if "us" in v and k != "attn_dense"}
    dominant = max(in_step, key=lambda k: in_step[k]["us"])
    traffic = None
    tp = os.path.join(ROOT, "profiles", f"traffic_{args.workload}.txt")
    if os.path.exists(tp) and args.attend == "summary":
        with open(tp) as f:
            tab = dict(line.split()[:2] for line in f if line.strip() and not line.startswith("#"))
        traffic = int(tab[dominant]) if dominant in tab else None
    if "flops" in kern[dominant]:
        roofline = {"kernel": dominant, "bound": "tensor", "achieved": kern[dominant]["TFLOP/s"], "peak": tensor_peak,
                    "unit": "TFLOP/s", "frac": kern[dominant]["frac_of_bf16_peak"], "traffic": traffic,
                    "peak_kind": f"of {peak_kind} (sustained bf16)", "algorithmic_flops": kern[dominant]["flops"],
                    "us_per_launch": kern[dominant]["us"]}
        if dominant == "gate_rnn":
            roofline["note"] = (f"{rig.Nc} strictly sequential LSTM steps per sequence: bounded by per-step latency "
                                f"({kern[dominant]['us'] / rig.Nc:.2f} us per step), not by tensor throughput")
    else:
        roofline = {"kernel": dominant, "bound": "hbm", "achieved": kern[dominant]["GB/s"], "peak": hbm, "unit": "GB/s",
                    "frac": kern[dominant]["GB/s"] / hbm, "traffic": traffic, "peak_kind": f"of {peak_kind}",
                    "algorithmic_bytes": kern[dominant]["bytes"], "us_per_launch": kern[dominant]["us"]}
    hbm_kernel = max((k for k in ("chunk_mean", "attn") if k in in_step), key=lambda k: in_step[k]["us"])
    roofline_hbm = {"kernel": hbm_kernel, "bound": "hbm", "achieved": kern[hbm_kernel]["GB/s"], "peak": hbm, "unit": "GB/s",
                    "frac": kern[hbm_kernel]["GB/s"] / hbm, "algorithmic_bytes": kern[hbm_kernel]["bytes"],
                    "us_per_launch": kern[hbm_kernel]["us"], "peak_kind": f"of {peak_kind}"}
    avd = head["attention_vs_dense"]
    kv_stale_gb = S * rig.Nc * wl.C * 512 / 1e9
    ms_step = ms_total / args.steps
    res = {
        "metric": METRIC, "value": world * args.steps / (ms_total * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": wl.name, "B_per_gpu": wl.B, "H": wl.H, "d": 128, "n": wl.n, "C": wl.C, "W": wl.W,
                   "d_g": wl.d_g, "agg": wl.agg, "d_sum": wl.d_sum, "attend": args.attend, "n_layers_timed": 1,
                   "stale_chunks": rig.Nc, "kept_chunks_mean": rig.keep_mean, "n_eff": rig.n_eff,
                   "memory_ratio_n_over_n_eff": wl.n / rig.n_eff,
                   "l2": f"inputs larger than L2 (each step streams {kv_stale_gb:.2f} GB of stale KV + "
                         f"{S * rig.R * 512 / 1e9:.2f} GB of window); kernels are also timed alone with L2 flushed before the launch"},
        "timing": {"repeats": repeats, "statistic": "median over repeats of one K-step loop (events, max over ranks)",
                   "loops_ms": loops, "timed_s_total": sum(loops) / 1e3},
        "e2e": {"value": world * args.steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": 3 * S * 256,
                "d2h_bytes_per_step": S * 256,
                "max_abs_diff_vs_device_path": e2e_diff, "max_abs_output": e2e_ref},
        "gpu_launches": kernels_per_step(wl, rig.Nc) * args.steps * repeats,
        "clocks": clk.summary(),
        "roofline": roofline,
        "roofline_largest_hbm_kernel": roofline_hbm,
        "gated_attention": {"us_l2_flushed": avd["gated_us"], "GB/s": avd["gated_GB/s"], "frac_of_hbm_peak": avd["gated_frac_of_measured_peak"],
                            "target": 0.70, "dense_us_l2_flushed": avd["dense_us"], "dense_frac_of_hbm_peak": avd["dense_frac_of_measured_peak"],
                            "kv_bytes_gated": avd["kv_bytes_gated"], "kv_bytes_dense": avd["kv_bytes_dense"], "speedup_vs_dense": avd["speedup"]},
        "steady_state": steady,
        "paper_cost_model": paper_cost_model(wl, rig.keep_mean),
        "kernels": kern,
        "attention_vs_dense": avd,
    }
    legs = set(args.legs.split(",")) if args.legs else set()
    if world > 1:
        legs = set()                     # the other legs are single-GPU properties: reported by the N = 1 run
    short = args.workload
    per = {short: {k: head[k] for k in head if k != "kernels"}}
    per[short]["full_step"] = {"ms": ms_step, "steps_per_s": 1e3 / ms_step}
    per[short]["steady_step"] = {"ms": steady["ms_per_step"], "steps_per_s": 1e3 / steady["ms_per_step"]}
    per[short]["kernels_us"] = {k: {a: v[a] for a in ("us", "us_l2_flushed", "frac_of_hbm_peak_l2_flushed") if a in v} for k, v in kern.items()}
    if "trigger" in legs:
        res["trigger"] = trigger_leg(wl, args.attend, seed + 5, steady["ms_per_step"])
        if wl.agg != "token_mlp":
            res["host_free_loop"] = host_free_loop_leg(wl, args.attend, seed + 6, steady["ms_per_step"])
    rig.st.close()
    del rig, st
    torch.cuda.empty_cache()
    if "per_config" in legs:
        for name in ("cfg1", "cfg2", "cfg3", "cfg4"):
            if name == short:
                continue
            w2 = wlm.CONFIGS[name].small(n_layers=1)
            r2 = Rig(w2, args.attend, seed + 100)
            m = measure_config(r2, peaks, peak_kind, flush)
            m["kernels_us"] = {k: {a: v[a] for a in ("us", "us_l2_flushed", "frac_of_hbm_peak_l2_flushed") if a in v}
                               for k, v in m.pop("kernels").items()}
            per[name] = m
            r2.st.close()
            del r2
            torch.cuda.empty_cache()
        per["cfg3"]["action_step_32_layers"] = action_step_leg(seed + 41)
    res["per_config"] = per
    if "sweep" in legs:
        res["sweep"] = sweep_leg(peaks, peak_kind, flush, seed + 200)
    if "token_mlp" in legs:
        res["token_mlp_aggregator"] = token_mlp_leg(wlm.CFG2.small(n_layers=1), peaks, peak_kind, flush, seed + 300)
    if "query_block" in legs:
        res["query_block_attention"] = query_block_leg(wl, hbm, tensor_peak, peak_kind, seed + 17)
    if "tick_graph" in legs and args.tick_layers > 0:
        res["decode_tick_graph"] = graph_tick_leg(wl, args.tick_layers, seed + 31)
    if "cpu" in legs:
        res["cpu_baseline"] = cpu_baseline(wl, args.attend, budget_s=12.0)
        res["cpu_oracle_per_config"] = oracle_per_config(args.attend)
    return res


# ---------------------------------------------------------------------------------------------- CPU oracle arm
def oracle_times(wl, attend, n_seq, threads=None):
    """Seconds the oracle (f64 build, OpenMP over sequences, `threads` threads) needs on n_seq sequences of the
    workload: T1 = the whole path (summaries, gate, keep list, gated attention), T2 = its gated attention alone,
    T0 = full-cache attention (Eq. 1 over all n tokens)."""
    from oracle import kvo, margin
    cores = os.cpu_count() or 1
    kvo.set_threads(threads or cores)
    try:
        o = kvo.Oracle("f64")
        seqs = list(range(n_seq))
        K, V = wlm.gen_kv(wl, 0, seqs=seqs)
        mlp, lstm = wlm.gen_mlp_weights(wl), wlm.gen_lstm_weights(wl)
        q = wlm.gen_q(wl)[seqs]
        Nc = wl.n_stale_chunks()
        agg = margin.AGG_CODE[wl.agg]
        att = kvo.ATTEND_RAW if attend == "raw" else kvo.ATTEND_SUMMARY
        t0 = time.perf_counter()
        sm = o.summarize(K, V, wl.C, 0, Nc, agg, mlp, stride=max(wl.max_chunks, 1))
        sc, _, _ = o.gate(sm["ksum_b16"], sm["vsum_b16"], 0, Nc, lstm)
        idx, cnt = o.compact(sc, Nc, wl.tau)
        t1 = time.perf_counter()
        o.attn(q, K, V, wl.C, Nc, idx, cnt, sm["ksum_b16"], sm["vsum_b16"], att, SCALE)
        t2 = time.perf_counter()
        o.attn_dense(q, K, V, SCALE)
        t3 = time.perf_counter()
    finally:
        kvo.set_threads(cores)
    return {"T1": t2 - t0, "T2": t2 - t1, "T0": t3 - t2}


def oracle_step_time(wl, attend, n_seq, repeat=1):
    """Seconds the oracle needs for the whole path (T1) on n_seq sequences, all host cores."""
    return min(oracle_times(wl, attend, n_seq)["T1"] for _ in range(repeat))


def cpu_baseline(wl, attend, budget_s=15.0):
    cores = os.cpu_count() or 1
    n_probe = min(wl.S, max(cores, 8))
    t = oracle_step_time(wl, attend, n_probe)
    n_seq = int(min(wl.S, max(n_probe, n_probe * budget_s / max(t, 1e-6))))
    n_seq = max(cores, n_seq // cores * cores) if n_seq >= cores else n_seq
    n_seq = min(n_seq, wl.S)
    t = oracle_step_time(wl, attend, n_seq)
    step_s = t * wl.S / n_seq
    return {"value": 1.0 / step_s, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{n_seq} of {wl.S} sequences of {wl.name} (whole path, f64 oracle, OpenMP over sequences), "
                      f"{t:.2f} s measured, scaled to the full step"}


def oracle_per_config(attend):
    """The oracle on every fixed configuration (one layer), single-threaded and with OpenMP on all host cores, on a
    bounded sample of sequences scaled to the layer: ms per step for T0 (full-cache attention), T1 (whole path) and T2
    (gated attention only)."""
    cores = os.cpu_count() or 1
    out = {"cores": cores, "note": "f64 oracle as it stands; sample of sequences scaled to one full layer; ms"}
    for name in ("cfg1", "cfg2", "cfg3", "cfg4"):
        wl = wlm.CONFIGS[name].small(n_layers=1)
        n_seq = min(wl.S, max(cores, 8))
        scale = wl.S / n_seq * 1e3
        one = oracle_times(wl, attend, n_seq, threads=1)
        omp = oracle_times(wl, attend, n_seq, threads=cores)
        out[name] = {"sample_sequences": n_seq, "of": wl.S,
                     "single_thread_ms": {k: v * scale for k, v in one.items()},
                     "openmp_ms": {k: v * scale for k, v in omp.items()}}
    return out


def run_reference(args, rank):
    if rank != 0:
        return None
    wl = wlm.CONFIGS[args.workload].small(n_layers=1)
    cores = os.cpu_count() or 1
    n_seq = min(wl.S, max(8, cores))
    for _ in range(min(args.warmup, 1)):
        oracle_step_time(wl, args.attend, n_seq)
    t0 = time.perf_counter()
    ts = [oracle_step_time(wl, args.attend, n_seq) for _ in range(args.steps)]
    wall = time.perf_counter() - t0
    step_s = float(np.mean(ts)) * wl.S / n_seq
    val = 1.0 / step_s
    sample = f"each step = {n_seq} of {wl.S} sequences of {wl.name}, scaled to the full step (f64 oracle, OpenMP over sequences)"
    return {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": step_s * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "B_per_gpu": wl.B, "H": wl.H, "d": 128, "n": wl.n, "C": wl.C, "W": wl.W,
                       "d_g": wl.d_g, "agg": wl.agg, "d_sum": wl.d_sum, "attend": args.attend, "n_layers_timed": 1},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0, "wall_s": wall}


ALL_LEGS = "per_config,sweep,trigger,token_mlp,query_block,tick_graph,cpu"


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4", choices=sorted(wlm.CONFIGS),
                    help="the configuration the headline step is timed on (default: the largest single-GPU one)")
    ap.add_argument("--attend", default="summary", choices=["summary", "raw"])
    ap.add_argument("--legs", default=ALL_LEGS,
                    help="comma-separated extra legs of the single-GPU report (per_config, sweep, trigger, token_mlp, "
                         "query_block, tick_graph, cpu); empty string: the headline only")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--min-timed-s", type=float, default=0.25,
                    help="the K-step loop is repeated until at least this much device time has been timed")
    ap.add_argument("--tick-layers", type=int, default=32,
                    help="layers of the CUDA-graph decode-tick leg (0 = skip; reduced if the caches would not fit 40 GB)")
    args = ap.parse_args()
    if args.no_cpu_baseline:
        args.legs = ",".join(x for x in args.legs.split(",") if x != "cpu")
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if args.steps > 20:
            args.steps = 20          # a bounded sample per step; keep the whole run within minutes
        res = run_reference(args, rank)
    else:
        if args.warmup < 3:
            args.warmup = 3
        if world > 1:
            import torch
            import torch.distributed as dist
            torch.cuda.set_device(local_rank)
            dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        res = run_ours(args, rank, world, local_rank)
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
            dist.destroy_process_group()
    if res is not None:
        print(json.dumps(res))


if __name__ == "__main__":
    main()
