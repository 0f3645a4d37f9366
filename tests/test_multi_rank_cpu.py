"""The N > 1 path of bench.py on CPU: two gloo ranks.  The path has no exchange step
(every rank is an independent replica on its own draw of the workload), so what
is tested is the only thing the ranks share: the whole-job reduction (summed
audio, slowest rank's time) and that the replicas really differ."""
import os
import socket
import sys

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    from paper_1912_11040_b200 import synth
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = synth.make_workload(2, seed=rank, batch=4, dur_scale=0.05)
    ms, dt = 10.0 + 5.0 * rank, 0.5 - 0.1 * rank
    res = bench.combine_ranks(w.audio_seconds, ms, dt, world, "cpu")
    dist.barrier()
    out.put((rank, w.audio_seconds, int(w.lengths.sum()), res))
    dist.destroy_process_group()


def test_two_rank_reduction_over_gloo():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (_, a0, n0, r0), (_, a1, n1, r1) = got
    assert n0 != n1                                   # different draws per rank
    assert r0 == r1                                   # every rank holds the job-wide figures
    audio, ms, dt = r0
    assert audio == np.float64(a0) + np.float64(a1)   # work adds up (weak scaling)
    assert ms == 15.0 and dt == 0.5                   # the slowest rank sets the time


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.combine_ranks(3.0, 2.0, 1.0, 1, "cpu") == (3.0, 2.0, 1.0)
