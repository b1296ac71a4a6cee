#!/usr/bin/env python
"""Benchmark of the gated chunked-KV decode path (one JSON line on stdout).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfg2]

A *step* is one pass of the whole hot path over one layer of the workload, from scratch:
append one token to every sequence, summarise every chunk that lies outside the window, run the
LSTM gate over all of them, compact the keep list, run the gated decode attention.  `value` is
whole-job steps per second with all inputs resident in HBM; `e2e` is the same step through
kvE_decode_step_host with pinned HOST buffers (H2D of k_new, v_new, q and D2H of the output inside
the timed region).  Under torchrun every rank runs the same per-GPU workload on its own batch
shard (weak scaling, no data-path collective: (layer, batch, head) units are independent).

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
KERNELS_PER_STEP = 9   # set_len, append, chunk mean, chunk MLP, gate projection, gate recurrence, score head, compact, attention


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
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    st.profile(True)
    res = {"what": f"kvE_decode_attn_block: {T} query tokens x {Hkv * G} query heads on {Hkv} KV heads, B={g.B}, n={n}; "
                   "tcgen05 kernel, one launch timed alone, L2 flushed",
           "query_rows_per_kv_head": T * G, "kept_chunks_mean": keep}
    for name, dense, rows in (("gated", False, n - Nc * g.C + keep), ("dense", True, n)):
        ts = []
        for i in range(12):
            flush.fill_(1)
            st.decode_attn_block(0, q, dense=dense, out=out)
            torch.cuda.synchronize()
            if i >= 2:
                ts.append(st.profile_read()["attn_block"])
        us = float(np.mean(ts))
        by = g.S * rows * 512                                  # every retained K and V row once per KV head
        fl = 4 * 128 * T * G * g.S * rows                      # Q K^T and P V
        res[name] = {"us": us, "kv_bytes": int(by), "GB/s": by / us / 1e3, "frac_of_hbm_peak": by / us / 1e3 / hbm,
                     "TFLOP/s": fl / us / 1e6, "frac_of_bf16_peak": fl / us / 1e6 / tensor_peak,
                     "peak_kind": f"of {peak_kind}"}
    assert st.poll_status() == 0
    res["gated_vs_dense"] = res["dense"]["us"] / res["gated"]["us"]
    return res


def graph_tick_leg(wl, n_layers, seed, replays=20):
    """The decode loop of a whole model between two gate triggers: per token, for each of n_layers layers
    append the new token at the device-held length (kvE_append_next) and run the gated attention; all
    layers captured once in a CUDA graph, every replay advancing by one token.  Compared with the
    same calls issued one by one."""
    import torch
    from paper_2509_21354_b200 import binding as b
    g = wl.small(agg="mean", d_sum=0)                      # the aggregator only feeds the keep list here
    per_layer = g.S * (g.n + g.C) * 512 * 1.1
    n_layers = max(1, min(n_layers, int(40e9 // per_layer)))
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
    res = {"what": f"decode loop over {n_layers} layers between two gate triggers (per layer and token: kvE_append_next at the "
                   "device-held length, gated attention), captured once in a CUDA graph and replayed - every replay "
                   "appends the next token - vs the same calls issued one by one",
           "n_layers": n_layers, "graph_first_tick_equals_eager": same}
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


def run_ours(args, rank, world, local_rank):
    import torch
    import torch.distributed as dist
    from paper_2509_21354_b200 import binding as b

    torch.cuda.set_device(local_rank)
    wl = wlm.CONFIGS[args.workload].small(n_layers=1)
    lo, _ = shard_batch(wl.B, rank, world)
    seed = 1000 + lo
    st = b.Store(B=wl.B, H=wl.H, C_=wl.C, W=wl.W, max_tokens=wl.n + wl.C, d_g=wl.d_g, agg=wl.agg, d_sum=wl.d_sum,
                 attend=args.attend, page_perm="random", seed=seed)
    g = fill_cache(st, wl, seed)
    mlp = wlm.gen_mlp_weights(wl)
    lstm = wlm.gen_lstm_weights(wl)
    aw = b.AggWeights(mlp) if mlp is not None else None
    lw = b.LstmWeights(lstm)
    S = wl.S
    rnd = lambda: torch.randn((S, 128), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16).contiguous()
    k_new, v_new, q = rnd(), rnd(), rnd()
    k3, v3 = k_new.view(S, 1, 128), v_new.view(S, 1, 128)
    out = torch.empty_like(q)
    n0 = wl.n
    Nc = wl.n_stale_chunks(n0)

    def step():
        st.set_len(0, n0 - 1)
        st.append(0, k3, v3)
        st.summarize_chunks(0, 0, Nc, aw)
        st.gate(0, 0, Nc, lw)
        st.compact(0, wl.tau)
        st.decode_attn(0, q, out)

    # head bias that retains about half of the chunks (deterministic given the seed)
    step()
    torch.cuda.synchronize()
    sc = st.scores[0, :, :Nc].double().clamp(1e-9, 1 - 1e-9)
    lw.set_b_s(float(-torch.median(torch.log(sc / (1 - sc))).item()) + lstm["b_s"])
    step()
    torch.cuda.synchronize()
    assert st.poll_status() == 0
    keep_mean = st.keep_cnt[0].float().mean().item()
    R = n0 - Nc * wl.C

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    with ClockSampler(local_rank) as clk:
        ev0.record()
        for _ in range(args.steps):
            step()
        ev1.record()
        barrier()
    ms_total = ev0.elapsed_time(ev1)
    assert st.poll_status() == 0

    # ---- steady-state decode step (between two gate triggers): append one token, gated attention ----
    # (token n0 + 1: no chunk leaves the window, so the keep list of the last full step stands)
    def step_steady():
        st.set_len(0, n0)
        st.append(0, k3, v3)
        st.decode_attn(0, q, out)

    for _ in range(3):
        step_steady()
    barrier()
    ev0.record()
    for _ in range(args.steps):
        step_steady()
    ev1.record()
    barrier()
    ms_steady = max_over_ranks([ev0.elapsed_time(ev1)], world)[0]
    assert st.poll_status() == 0
    step()                      # back to the state and output of a full step
    torch.cuda.synchronize()
    steady = {"what": "append + gated attention only (summaries, gate and keep list reused: the state between two triggers)",
              "value": world * args.steps / (ms_steady * 1e-3), "unit": UNIT, "ms_per_step": ms_steady / args.steps}

    # ---- end to end: the same step through kvE_decode_step_host, host buffers, copies timed ----
    hk, hv, hq = (t.cpu().pin_memory() for t in (k_new, v_new, q))
    hout = torch.zeros((S, 128), dtype=torch.bfloat16).pin_memory()

    # every step: H2D of its inputs and D2H of its result inside the timed region; steps are enqueued
    # back to back (kvE_decode_step_host_async) and the stream is waited for once, at the end
    def step_e2e():
        st.set_len(0, n0 - 1)
        st.decode_step_host(0, hk, hv, hq, hout, aw, lw, wl.tau, from_scratch=True, wait=False)

    for _ in range(min(args.warmup, 3)):
        step_e2e()
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step_e2e()
    barrier()
    e2e_s = time.perf_counter() - t0
    same = bool(torch.equal(hout.cuda(), out))

    ms_total, e2e_s = max_over_ranks([ms_total, e2e_s], world)
    if rank != 0:
        return None

    # ---- per-kernel timing (rank 0): the library brackets every launch with CUDA events on its stream ----
    peaks, peak_kind = load_peaks()
    hbm = peaks["hbm_gbs"]
    st.profile(True)
    in_step = {k: [] for k in b.KERNEL_IDS}
    for _ in range(min(args.steps, 30)):          # same step as the timed region
        step()
        for k, v in st.profile_read().items():
            if v is not None and k != "attn_dense":
                in_step[k].append(v)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    cold = {"attn": [], "attn_dense": []}
    for _ in range(10):                            # attention alone, L2 flushed before every launch
        for name, fn in (("attn", st.decode_attn), ("attn_dense", st.decode_attn_dense)):
            flush.fill_(1)
            fn(0, q, out)
            cold[name].append(st.profile_read()[name])
    st.profile(False)
    us = {k: float(np.mean(v)) for k, v in in_step.items() if v}
    us["attn_dense"] = float(np.mean(cold["attn_dense"]))
    us_attn_cold = float(np.mean(cold["attn"]))
    by = algorithmic_bytes(wl, Nc, keep_mean, R, args.attend)

    def copy_us(total_bytes):
        """a plain device copy that moves total_bytes (read + write), timed like the kernels: L2 flushed, events"""
        src = torch.empty(max(1, int(total_bytes) // 2), dtype=torch.uint8, device="cuda")
        dst = torch.empty_like(src)
        ts = []
        for i in range(8):
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            dst.copy_(src)
            e1.record()
            torch.cuda.synchronize()
            if i >= 2:
                ts.append(e0.elapsed_time(e1) * 1e3)
        return float(np.mean(ts))

    copy_gated_us, copy_dense_us = copy_us(by["attn_gated"]), copy_us(by["attn_dense"])
    by_kernel = {"append": S * 4 * 256, "chunk_mean": by["chunk_mean"], "chunk_mlp": by["chunk_mlp"],
                 "gate_proj": by["gate_proj"], "gate_rnn": by["gate_rnn"], "compact": by["compact"],
                 "attn": by["attn_gated"], "attn_dense": by["attn_dense"]}
    fl = algorithmic_flops(wl, Nc)
    tensor_peak = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])     # kernels timed inside a long step
    kern = {}
    for k, t in us.items():
        kern[k] = {"us": t, "bytes": by_kernel[k], "GB/s": by_kernel[k] / (t * 1e-6) / 1e9}
        kern[k]["frac_of_hbm_peak"] = kern[k]["GB/s"] / hbm
        if k in fl:
            kern[k]["flops"] = fl[k]
            kern[k]["TFLOP/s"] = fl[k] / (t * 1e-6) / 1e12
            kern[k]["frac_of_bf16_peak"] = kern[k]["TFLOP/s"] / tensor_peak
    kern["attn"]["us_l2_flushed"] = us_attn_cold
    kern["attn"]["GB/s_l2_flushed"] = by_kernel["attn"] / (us_attn_cold * 1e-6) / 1e9
    dominant = max((k for k in kern if k != "attn_dense"), key=lambda k: kern[k]["us"])
    traffic = None
    tp = os.path.join(ROOT, "profiles", f"traffic_{args.workload}.txt")
    if os.path.exists(tp) and args.attend == "summary":
        with open(tp) as f:
            tab = dict(line.split() for line in f if line.strip() and not line.startswith("#"))
        traffic = int(tab[dominant]) if dominant in tab else None
    if dominant in fl:
        roofline = {"kernel": dominant, "bound": "tensor", "achieved": kern[dominant]["TFLOP/s"], "peak": tensor_peak,
                    "unit": "TFLOP/s", "frac": kern[dominant]["frac_of_bf16_peak"], "traffic": traffic,
                    "peak_kind": f"of {peak_kind} (sustained bf16)", "algorithmic_flops": fl[dominant],
                    "us_per_launch": kern[dominant]["us"]}
        if dominant == "gate_rnn":
            roofline["note"] = (f"{Nc} strictly sequential LSTM steps per sequence: bounded by per-step latency "
                                f"({kern[dominant]['us'] / Nc:.2f} us per step), not by tensor throughput")
    else:
        roofline = {"kernel": dominant, "bound": "hbm", "achieved": kern[dominant]["GB/s"], "peak": hbm, "unit": "GB/s",
                    "frac": kern[dominant]["GB/s"] / hbm, "traffic": traffic, "peak_kind": f"of {peak_kind}",
                    "algorithmic_bytes": kern[dominant]["bytes"], "us_per_launch": kern[dominant]["us"]}
    hbm_kernel = max((k for k in ("chunk_mean", "attn")), key=lambda k: kern[k]["us"])
    roofline_hbm = {"kernel": hbm_kernel, "bound": "hbm", "achieved": kern[hbm_kernel]["GB/s"], "peak": hbm, "unit": "GB/s",
                    "frac": kern[hbm_kernel]["GB/s"] / hbm, "algorithmic_bytes": kern[hbm_kernel]["bytes"],
                    "us_per_launch": kern[hbm_kernel]["us"], "peak_kind": f"of {peak_kind}"}
    us["attn_gated"] = us_attn_cold

    ms_step = ms_total / args.steps
    res = {
        "metric": METRIC, "value": world * args.steps / (ms_total * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": wl.name, "B_per_gpu": wl.B, "H": wl.H, "d": 128, "n": wl.n, "C": wl.C, "W": wl.W,
                   "d_g": wl.d_g, "agg": wl.agg, "d_sum": wl.d_sum, "attend": args.attend, "n_layers_timed": 1,
                   "stale_chunks": Nc, "kept_chunks_mean": keep_mean, "n_eff": R + keep_mean * (wl.C if args.attend == "raw" else 1),
                   "memory_ratio_n_over_n_eff": n0 / (R + keep_mean * (wl.C if args.attend == "raw" else 1)),
                   "l2": "inputs larger than L2 (each step streams 0.45 GB of stale KV + 0.06 GB window); per-kernel timings flush L2 before every launch"},
        "e2e": {"value": world * args.steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": 3 * S * 256,
                "d2h_bytes_per_step": S * 256, "matches_device_path": same},
        "gpu_launches": KERNELS_PER_STEP * args.steps,
        "clocks": clk.summary(),
        "roofline": roofline,
        "roofline_largest_hbm_kernel": roofline_hbm,
        "steady_state": steady,
        "query_block_attention": query_block_leg(wl, hbm, tensor_peak, peak_kind, seed + 17),
        "decode_tick_graph": graph_tick_leg(wl, args.tick_layers, seed + 31) if args.tick_layers > 0 else None,
        "paper_cost_model": paper_cost_model(wl, keep_mean),
        "kernels": kern,
        "attention_vs_dense": {"note": "attention kernels alone, L2 flushed before every launch",
                               "gated_us": us["attn_gated"], "dense_us": us["attn_dense"],
                               "speedup": us["attn_dense"] / us["attn_gated"],
                               "kv_bytes_gated": by["attn_gated"], "kv_bytes_dense": by["attn_dense"],
                               "gated_GB/s": kern["attn"]["GB/s_l2_flushed"], "dense_GB/s": kern["attn_dense"]["GB/s"],
                               "gated_frac_of_measured_peak": kern["attn"]["GB/s_l2_flushed"] / hbm,
                               "dense_frac_of_measured_peak": kern["attn_dense"]["GB/s"] / hbm,
                               "size_matched_copy": {
                                   "note": "a plain torch device copy moving the same number of bytes (read + write), "
                                           "same timing method: what this transfer size allows on this GPU",
                                   "gated_bytes_copy_us": copy_gated_us, "dense_bytes_copy_us": copy_dense_us,
                                   "gated_frac_of_copy": copy_gated_us / us["attn_gated"],
                                   "dense_frac_of_copy": copy_dense_us / us["attn_dense"]},
                               "gated_frac_of_nominal_8TBps": kern["attn"]["GB/s_l2_flushed"] / 8000.0,
                               "dense_frac_of_nominal_8TBps": kern["attn_dense"]["GB/s"] / 8000.0},
    }
    if not args.no_cpu_baseline and world == 1:
        res["cpu_baseline"] = cpu_baseline(wl, args.attend, budget_s=15.0)
    return res


# ---------------------------------------------------------------------------------------------- CPU oracle arm
def oracle_step_time(wl, attend, n_seq, repeat=1):
    """Seconds the oracle (f64 build, OpenMP over sequences) needs for the whole path on n_seq sequences."""
    from oracle import kvo, margin
    o = kvo.Oracle("f64")
    seqs = list(range(n_seq))
    K, V = wlm.gen_kv(wl, 0, seqs=seqs)
    mlp, lstm = wlm.gen_mlp_weights(wl), wlm.gen_lstm_weights(wl)
    q = wlm.gen_q(wl)[seqs]
    Nc = wl.n_stale_chunks()
    agg = margin.AGG_CODE[wl.agg]
    att = kvo.ATTEND_RAW if attend == "raw" else kvo.ATTEND_SUMMARY
    best = float("inf")
    for _ in range(repeat):
        t0 = time.perf_counter()
        sm = o.summarize(K, V, wl.C, 0, Nc, agg, mlp, stride=max(wl.max_chunks, 1))
        sc, _, _ = o.gate(sm["ksum_b16"], sm["vsum_b16"], 0, Nc, lstm)
        idx, cnt = o.compact(sc, Nc, wl.tau)
        o.attn(q, K, V, wl.C, Nc, idx, cnt, sm["ksum_b16"], sm["vsum_b16"], att, SCALE)
        best = min(best, time.perf_counter() - t0)
    return best


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
                       "d_g": wl.d_g, "agg": wl.agg, "d_sum": wl.d_sum, "attend": args.attend},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0, "wall_s": wall}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=sorted(wlm.CONFIGS))
    ap.add_argument("--attend", default="summary", choices=["summary", "raw"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--tick-layers", type=int, default=32,
                    help="layers of the CUDA-graph decode-tick leg (0 = skip; reduced if the caches would not fit 40 GB)")
    args = ap.parse_args()
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
