"""The multi-GPU leg of the benchmark is N independent replicas: each rank runs its own shard, the job's step time is
the slowest rank's, the value is the sum of the work over that time. Checked on two CPU ranks (gloo)."""
import os
import socket
import sys
from pathlib import Path

import numpy as np

sys.path.insert(0, str(Path(__file__).resolve().parent.parent))


def _worker(rank, world, port, out_dir):
    import torch.distributed as dist

    import bench

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = bench.rank_workload(3, 0, rank)
        ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, "cpu")
        value = bench.whole_job_value(sum(w.flops()), world, ms)
        np.save(os.path.join(out_dir, f"r{rank}.npy"),
                np.array([ms, value, float(w.lengths.sum()), float(w.n_seg), float(sum(w.flops()))]))
    finally:
        dist.destroy_process_group()


def test_two_replicas_on_cpu_ranks(tmp_path):
    import torch.multiprocessing as mp

    import bench

    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    r0, r1 = np.load(tmp_path / "r0.npy"), np.load(tmp_path / "r1.npy")
    assert r0[0] == 15.0 and r1[0] == 15.0  # both ranks see the slowest rank's time
    assert r0[2] == r1[2] == 65536  # same configuration and token budget on every rank ...
    w0, w1 = bench.rank_workload(3, 0, 0), bench.rank_workload(3, 0, 1)
    assert not np.array_equal(w0.lengths, w1.lengths)  # ... but its own draw of the lengths
    assert r0[1] == bench.whole_job_value(r0[4], 2, 15.0)
    # one rank: no collective, the value is that rank's
    assert bench.max_over_ranks(7.0, 1, "cpu") == 7.0
