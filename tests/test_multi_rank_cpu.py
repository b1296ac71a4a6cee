"""The multi-GPU path on CPU: two gloo ranks, each owning its own batch shard (replicas, no data-path
collective).  Checks what the benchmark's N > 1 mode relies on: shards are disjoint and cover the
global batch, a rank's inputs depend only on its shard, per-shard results equal the corresponding
slice of a single-process run, and the max-over-ranks reduction of the step time."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402
from oracle import kvo, margin  # noqa: E402
from paper_2509_21354_b200 import workloads as wlm  # noqa: E402

B_PER_RANK, H = 2, 2
SCALE = 1.0 / np.sqrt(128.0)


def _shard_result(lo, hi):
    """oracle output of the sequences of global batches [lo, hi) of one fixed global workload"""
    wl = wlm.CFG1.small(B=2 * B_PER_RANK, H=H, n=512, W=128, seed=9)
    seqs = [b * H + h for b in range(lo, hi) for h in range(H)]
    o = kvo.Oracle("f64")
    K, V = wlm.gen_kv(wl, 0, seqs=seqs)
    lstm = wlm.gen_lstm_weights(wl)
    Nc = wl.n_stale_chunks()
    sm = o.summarize(K, V, wl.C, 0, Nc, margin.AGG_CODE[wl.agg], None, stride=wl.max_chunks)
    sc, _, _ = o.gate(sm["ksum_b16"], sm["vsum_b16"], 0, Nc, lstm)
    idx, cnt = o.compact(sc, Nc, 0.5)
    q = wlm.gen_q(wl)[seqs]
    out = o.attn(q, K, V, wl.C, Nc, idx, cnt, sm["ksum_b16"], sm["vsum_b16"], kvo.ATTEND_SUMMARY, SCALE)[0]
    return np.asarray(out, np.float64), np.asarray(cnt)


def _worker(rank, world, port, ret):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        lo, hi = bench.shard_batch(B_PER_RANK, rank, world)
        out, cnt = _shard_result(lo, hi)
        # the benchmark's only collective: the slowest rank sets the step time
        times = bench.max_over_ranks([10.0 + rank, 5.0 - rank], world, device="cpu")
        gathered = [None] * world
        dist.all_gather_object(gathered, (lo, hi, out, cnt))
        dist.barrier()
        if rank == 0:
            ret["times"] = times
            ret["shards"] = gathered
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_the_batch_without_a_data_collective():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ret = mp.Manager().dict()
    mp.spawn(_worker, args=(2, port, ret), nprocs=2, join=True)
    assert ret["times"] == [11.0, 5.0]
    shards = sorted(ret["shards"], key=lambda t: t[0])
    assert [(lo, hi) for lo, hi, _, _ in shards] == [(0, B_PER_RANK), (B_PER_RANK, 2 * B_PER_RANK)]   # disjoint, covering
    full_out, full_cnt = _shard_result(0, 2 * B_PER_RANK)
    got_out = np.concatenate([o for _, _, o, _ in shards])
    got_cnt = np.concatenate([c for _, _, _, c in shards])
    assert np.array_equal(got_cnt, full_cnt)
    assert np.array_equal(got_out, full_out)        # a sequence's result does not depend on which rank holds it


def test_single_rank_reduction_is_identity():
    assert bench.max_over_ranks([1.5, 2.5], 1) == [1.5, 2.5]
    assert bench.shard_batch(8, 3, 4) == (24, 32)
