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


# ----------------------------------------------------------------------------- data-parallel step (2 gloo ranks, oracle as the engine)

def _dp_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import torch
    import torch.distributed as dist
    from oracle import mrem_oracle as O
    from paper_2109_15082_b200 import dist as D
    from paper_2109_15082_b200 import synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = synth.Workload("dp", 2, 32, 2, 64, 8, 5, act_dtype="f64", outlier_channels=2, len_lo=3, len_hi=8)
    desc = O.ModuleDesc(2, 32, 2, 64, 4, 8, act_dtype="f64")
    teacher = synth.teacher_params(wl, 0, bias_std=0.1)            # every rank builds the same module (seed 0)
    student = [{k: (v + synth.normal(1, f"n{l}{k}", v.shape, 0.01)).astype(np.float32) for k, v in p.items()} for l, p in enumerate(teacher)]
    x = synth.hidden_states(wl, wl.batch, 0)
    vl = synth.valid_lengths(wl, wl.batch, 0)
    lo, hi = D.shard_bounds(wl.batch, rank, world)                  # 5 sequences on 2 ranks: 3 + 2
    # activation ranges: each rank from its own sequences, then combined
    ws = O.init_weight_steps(desc, student, 0)
    a_loc, off_loc = O.init_act_steps(desc, student, x[lo:hi], vl[lo:hi])
    a_t, off_t = torch.from_numpy(a_loc.copy()), torch.from_numpy(off_loc.copy())
    D.combine_act_ranges(a_t, off_t, 8, 3)
    a_all, off_all = O.init_act_steps(desc, student, x, vl)
    steps = O.make_steps(ws, (a_all * 0.8).astype(np.float32), off_all)
    # this rank's share of the whole batch's loss and gradients (Eq. 3 is a sum over sequences)
    share = (hi - lo) / wl.batch
    r = O.forward_loss_backward(desc, teacher, student, steps, x[lo:hi], x[lo:hi], vl[lo:hi])
    buckets = []
    for g in r["grads"]:
        flat = [np.asarray(g[k], np.float64).ravel() for k in O.PARAMS] + [np.asarray(g["w"][k]).ravel() for k in O.WEIGHTS] + [g["a"], g["a_off"]]
        buckets.append(torch.from_numpy(np.concatenate(flat) * share))
    loss = torch.tensor([r["loss"] * share], dtype=torch.float64)
    order = []
    works = D.allreduce_buckets(list(reversed(buckets)), async_op=True)
    works.append(dist.all_reduce(loss, async_op=True))
    for w in works:
        w.wait()
    out.put((rank, (lo, hi), a_t.numpy(), off_t.numpy(), a_all, off_all, [b.numpy() for b in buckets], float(loss[0])))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_sum_to_the_full_batch_gradient():
    """Data parallel on 2 ranks (3 + 2 sequences of a batch of 5): the all-reduced per-layer buckets and the loss equal the
    oracle's full-batch gradients and loss; the combined activation ranges equal those of the whole batch."""
    sys.path.insert(0, ROOT)
    from oracle import mrem_oracle as O
    from paper_2109_15082_b200 import dist as D
    from paper_2109_15082_b200 import synth
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_dp_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted((out.get(timeout=180) for _ in procs), key=lambda t: t[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [(0, 3), (3, 5)]
    assert [D.shard_bounds(7, r, 3) for r in range(3)] == [(0, 3), (3, 5), (5, 7)]
    # the full batch in this process
    wl = synth.Workload("dp", 2, 32, 2, 64, 8, 5, act_dtype="f64", outlier_channels=2, len_lo=3, len_hi=8)
    desc = O.ModuleDesc(2, 32, 2, 64, 4, 8, act_dtype="f64")
    teacher = synth.teacher_params(wl, 0, bias_std=0.1)
    student = [{k: (v + synth.normal(1, f"n{l}{k}", v.shape, 0.01)).astype(np.float32) for k, v in p.items()} for l, p in enumerate(teacher)]
    x, vl = synth.hidden_states(wl, wl.batch, 0), synth.valid_lengths(wl, wl.batch, 0)
    ws = O.init_weight_steps(desc, student, 0)
    a_all, off_all = O.init_act_steps(desc, student, x, vl)
    full = O.forward_loss_backward(desc, teacher, student, O.make_steps(ws, (a_all * 0.8).astype(np.float32), off_all), x, x, vl)
    for rank, _, a_comb, off_comb, a_ref, off_ref, buckets, loss in res:
        assert np.allclose(a_comb, a_ref, rtol=1e-6) and np.allclose(off_comb, off_ref, rtol=1e-6, atol=1e-7)
        assert np.isclose(loss, full["loss"], rtol=1e-12)
        for l, g in enumerate(full["grads"]):
            flat = np.concatenate([np.asarray(g[k], np.float64).ravel() for k in O.PARAMS] + [np.asarray(g["w"][k]).ravel() for k in O.WEIGHTS] + [g["a"], g["a_off"]])
            assert np.allclose(buckets[l], flat, rtol=1e-9, atol=1e-12 * np.abs(flat).max()), (rank, l)
    assert np.array_equal(res[0][6][0], res[1][6][0])                 # both ranks hold the same sums
