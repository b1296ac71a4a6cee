"""Where the time of one attention launch goes: per-CTA time stamps of kve_decode_attn_kernel.

    python -m paper_2509_21354_b200.attn_stamps [cfg4 cfg2 cfg1 ...]

Builds an instrumented copy of the library (-DKVE_ATTN_STAMPS; the product library carries no stamps), runs the gated
and the full-cache attention of each configuration once per repetition with L2 cold and clean, and prints, for the
last repetition, the minimum / median / maximum over the CTAs of every stamp in microseconds after the first CTA's
entry.  CUDA device required."""
import ctypes as C
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2509_21354_b200 import build as kb  # noqa: E402

NAMES = ["kernel entry", "predecessor waited for", "first copy issued", "first tile landed", "last tile consumed",
         "merger warp done", "producer warp done"]


def main(cfgs):
    lib_path = kb.build(defines=("KVE_ATTN_STAMPS",), lib=os.path.join(kb.HERE, "libkve_stamps.so"),
                        obj_dir=os.path.join(kb.HERE, "_build_stamps"))
    kb.LIB, kb.build = lib_path, (lambda *a, **k: lib_path)          # the binding loads the instrumented copy
    import torch
    import bench
    from paper_2509_21354_b200 import binding as b, workloads as wlm
    lib = b.load_library()
    lib.kve_attn_stamps_read.argtypes = [C.c_void_p, C.c_int]
    flush = bench.Flusher()
    for cfg in cfgs:
        rig = bench.Rig(wlm.CONFIGS[cfg].small(n_layers=1), "summary", 1000)
        for dense in (False, True):
            fn = rig.st.decode_attn_dense if dense else rig.st.decode_attn
            for _ in range(5):
                flush()
                lib.kve_attn_stamps_clear()
                torch.cuda.synchronize()
                fn(0, rig.q, rig.out)
                torch.cuda.synchronize()
            buf = np.zeros(2048 * 8, np.uint64)
            lib.kve_attn_stamps_read(buf.ctypes.data, buf.size)
            st = buf.reshape(2048, 8).astype(np.int64)
            st = st[st[:, 0] > 0]
            rel = (st - st[:, 0].min()) / 1e3
            print(f"== {rig.wl.name}, {'full-cache' if dense else 'gated'} attention: {len(rel)} CTAs; "
                  "microseconds after the first CTA's entry (min / median / max over the CTAs)")
            for i, nm in enumerate(NAMES):
                col = rel[:, i]
                print(f"  {nm:26s} {col.min():8.2f} {np.median(col):8.2f} {col.max():8.2f}")
            stream, drain = rel[:, 4] - rel[:, 3], rel[:, 5] - rel[:, 4]
            print(f"  first tile landed -> last tile consumed, per CTA: median {np.median(stream):.2f}, max {stream.max():.2f}")
            print(f"  last tile consumed -> merger done, per CTA:       median {np.median(drain):.2f}, max {drain.max():.2f}")
        rig.st.close()


if __name__ == "__main__":
    main(sys.argv[1:] or ["cfg4", "cfg1"])
