"""Cycle budget of one step of the gate recurrence (kve_gate_rnn_kernel).

    python -m paper_2509_21354_b200.rnn_stamps [cfg2 cfg4 ...]

Builds an instrumented copy of the library (-DKVE_RNN_STAMPS; the product library carries no stamps), runs kvE_gate
over all stale chunks of each configuration and prints where warp 0 of CTA 0 spends a step, in clock cycles and in
microseconds at the SM clock nvidia-smi reports, averaged over all steps (and groups of 8 sequences).  CUDA device
required."""
import ctypes as C
import os
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2509_21354_b200 import build as kb  # noqa: E402

PHASES = ["wait for the peers' h (mbarrier)", "ldmatrix + MMA chain (W_hh h)", "prefetch of the next step's P",
          "cell update + plane split", "send h (staging, fence, bulk copies, arrive)",
          "round to round (P_{t+1} lands in place, expect_tx)"]
SLOTS = [6, 0, 1, 2, 3, 4]


def main(cfgs):
    lib_path = kb.build(defines=("KVE_RNN_STAMPS",), lib=os.path.join(kb.HERE, "libkve_rnn_stamps.so"),
                        obj_dir=os.path.join(kb.HERE, "_build_rnn_stamps"))
    kb.LIB, kb.build = lib_path, (lambda *a, **k: lib_path)          # the binding loads the instrumented copy
    import torch
    import bench
    from paper_2509_21354_b200 import binding as b, workloads as wlm
    lib = b.load_library()
    lib.kve_rnn_cycles_read.argtypes = [C.c_void_p]
    mhz = float(subprocess.run(["nvidia-smi", "--query-gpu=clocks.max.sm", "--format=csv,noheader,nounits", "-i", "0"],
                               capture_output=True, text=True).stdout.strip() or 1965)
    buf = np.zeros(8, np.uint64)
    for cfg in cfgs:
        rig = bench.Rig(wlm.CONFIGS[cfg].small(n_layers=1), "summary", 1000)
        for planes in (2, 3):
            rig.st.set_gate_planes(planes)
            for _ in range(3):
                rig.st.gate(0, 0, rig.Nc, rig.lw)
            torch.cuda.synchronize()
            lib.kve_rnn_cycles_read(buf.ctypes.data)              # clears
            rig.st.profile(True)
            rig.st.gate(0, 0, rig.Nc, rig.lw)
            us_kernel = rig.st.profile_read()["gate_rnn"]
            rig.st.profile(False)
            lib.kve_rnn_cycles_read(buf.ctypes.data)
            once = np.zeros(8, np.uint64)
            lib.kve_rnn_once_read(once.ctypes.data)
            rounds = int(buf[5])
            groups = max(1, rounds // rig.Nc)
            print(f"== {rig.wl.name}: {rig.Nc} steps, {rig.wl.S} sequences, {groups} group(s) of 8 sequences per cluster, "
                  f"{planes} planes of h; recurrence + score head {us_kernel:.1f} us = {us_kernel / rig.Nc:.2f} us per step")
            tot = 0
            for i, nm in zip(SLOTS, [PHASES[5]] + PHASES[:5]):
                cyc = float(buf[i]) / max(rounds, 1)
                tot += cyc
                print(f"  {nm:52s} {cyc:8.0f} cycles  {cyc / mhz:6.3f} us   (per step and group)")
            o = (once.astype(np.int64) - int(once[0])) / 1e3
            print(f"  CTA 0, us after its entry: W_hh fragments loaded {o[1]:.2f}, predecessor waited for {o[2]:.2f}, initial state and "
                  f"first P {o[3]:.2f}, cluster barrier {o[4]:.2f}, step loop done {o[5]:.2f}, state out + cluster barrier {o[6]:.2f}")
            loop_us = tot * rounds / mhz
            print(f"  {'sum':52s} {tot:8.0f} cycles  {tot / mhz:6.3f} us   x {groups} group(s) = {tot * groups / mhz:.3f} us per step; "
                  f"step loop {loop_us:.1f} us of the {us_kernel:.1f} us (rest: W_hh fragments into registers, first P, "
                  "cluster syncs, score head)")
        rig.st.close()


if __name__ == "__main__":
    main(sys.argv[1:] or ["cfg2", "cfg4"])
