"""The N > 1 host logic of the benchmark on CPU: two gloo ranks, each an independent replica,
agree on the slowest rank's time and on the whole-job rate; replicas draw different data."""
import os
import socket
import sys

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import torch.distributed as dist
    from paper_2109_15082_b200 import dist as D
    from paper_2109_15082_b200 import synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert D.env_rank() == (rank, world, rank)
    ms = 10.0 + 5.0 * rank                                 # rank 1 is the slow one
    dist.barrier()
    slowest = D.max_over_ranks(ms)
    rate = D.whole_job_rate(4096, 20, world, slowest)
    x = synth.normal(D.replica_seed(rank), "probe", (4,))
    out.put((rank, slowest, rate, x.tolist()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_max_time_and_rate():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [15.0, 15.0]
    assert np.isclose(res[0][2], 2 * 4096 * 20 / 15e-3) and res[0][2] == res[1][2]
    assert res[0][3] != res[1][3]                         # replicas are independent problems


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    from paper_2109_15082_b200 import dist as D
    assert D.max_over_ranks(3.5) == 3.5
    assert D.whole_job_rate(10, 2, 1, 1000.0) == 20.0
