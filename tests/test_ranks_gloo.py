"""The multi-rank plumbing (one process per GPU, weak scaling, no data-path collective) on two
CPU ranks over gloo: rank-private inputs, the barrier, the maximum over ranks and the whole-job
throughput that the benchmark reports."""
import os
import socket

import numpy as np
import torch.multiprocessing as mp

from paper_2310_05869_b200 import ranks as RK
from paper_2310_05869_b200 import workloads as WL


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update({"RANK": str(rank), "LOCAL_RANK": str(rank), "WORLD_SIZE": str(world),
                       "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port)})
    info = RK.rank_env()
    assert (info.rank, info.world) == (rank, world)
    RK.init(info, "gloo")
    w = WL.CONFIGS[0]
    q = WL.make_inputs(RK.rank_workload(w, rank))[0]
    RK.barrier(info)
    ms = RK.max_over_ranks(info, 10.0 + 5.0 * rank)            # rank 1 is the slow one
    value = RK.job_throughput(info, w.B * w.n, 4, ms)
    RK.barrier(info)
    np.save(os.path.join(out_dir, f"r{rank}.npy"), np.array([ms, value, float(q.astype(np.float64).sum())]))
    RK.shutdown(info)


def test_two_ranks_weak_scaling(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r0, r1 = (np.load(tmp_path / f"r{r}.npy") for r in range(world))
    assert r0[0] == r1[0] == 15.0                              # every rank sees the slowest rank's time
    w = WL.CONFIGS[0]
    assert r0[1] == r1[1] == w.B * w.n * 4 * 2 / 15e-3          # units of all ranks / that time
    assert r0[2] != r1[2]                                       # the ranks work on different inputs
    q0 = WL.make_inputs(w)[0]
    assert r0[2] == float(q0.astype(np.float64).sum())          # rank 0 keeps the single-process workload


def test_single_process_is_a_no_op():
    info = RK.rank_env({})
    assert info == RK.RankInfo(0, 0, 1)
    RK.init(info, "gloo")
    RK.barrier(info)
    assert RK.max_over_ranks(info, 3.5) == 3.5
    assert RK.job_throughput(info, 1000, 2, 4.0) == 1000 * 2 / 4e-3
    RK.shutdown(info)
