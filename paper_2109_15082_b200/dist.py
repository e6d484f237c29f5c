"""Host-side helpers for more than one GPU, one process per GPU (torch.distributed).

Two modes.  Replicas: one independent module (its own weights and calibration set) per rank, no collective on the
data path; torch.distributed serves the barrier and the max of the timings (bench.py --gpus N).  Data parallel:
every rank holds the same module and takes its share of each batch; the gradients of a layer are summed over the
ranks by one all-reduce per layer before the update (DataParallelModule, bench.py --gpus N --dp)."""
from __future__ import annotations

import os


def env_rank():
    """(rank, world_size, local_rank) from the torchrun environment; (0, 1, 0) when absent."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def replica_seed(rank: int, base: int = 0) -> int:
    """Each replica draws its own weights and calibration set."""
    return base + rank


def max_over_ranks(value: float, device=None) -> float:
    """The slowest rank's time (all ranks get it).  Works on any initialised backend."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0])


def whole_job_rate(units_per_step_per_rank: int, steps: int, world: int, ms: float) -> float:
    """Aggregate units/s of `world` replicas that all ran `steps` steps within `ms` (the max over ranks)."""
    return world * units_per_step_per_rank * steps / (ms * 1e-3)


# ----------------------------------------------------------------------------- data-parallel reconstruction step
#
# The loss of Eq. 3 is a sum over the sequences of the batch, so R ranks that hold identical parameters and steps and
# each take batch / R sequences get the whole batch's gradient by adding theirs (one all-reduce per layer), after
# which every rank applies the same update and the replicas stay identical.  The only other exchange is at
# initialisation: the activation steps come from the value ranges of the first batch, which are maxima / minima over
# all ranks' sequences.

def shard_bounds(n_items: int, rank: int, world: int):
    """[lo, hi) of this rank's contiguous share of n_items; the first n_items % world ranks get one more."""
    base, extra = divmod(int(n_items), int(world))
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def allreduce_buckets(buckets, group=None, async_op=True):
    """Sum every tensor of `buckets` over the ranks, in the given order (top layer first: the order in which the
    backward pass finishes them).  With async_op the collectives are only enqueued; returns the work handles, to be
    waited for before the update reads the sums."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return []
    works = []
    for t in buckets:
        w = dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group, async_op=async_op)
        if async_op:
            works.append(w)
    return works


def combine_act_ranges(a_steps, a_off, a_bits, asym_sites, group=None):
    """Activation steps / offsets [L, 8] that every rank initialised from ITS sequences -> those of all sequences.
    A symmetric site's step is max|x| / qmax and the softmax site's max / (2^b - 1): the maximum over ranks.  The GELU
    site (asymmetric, offset = min): offset = minimum over ranks, step = (max over ranks of offset + step * (2^b - 1)
    - that minimum) / (2^b - 1).  In place on torch tensors; returns them."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return a_steps, a_off
    qu = float(2 ** a_bits - 1)
    g_site = 7
    asym_g = bool(asym_sites & 2)
    hi = a_off[:, g_site] + a_steps[:, g_site] * qu if asym_g else None
    dist.all_reduce(a_steps, op=dist.ReduceOp.MAX, group=group)
    if asym_g:
        lo = a_off[:, g_site].clone()
        dist.all_reduce(lo, op=dist.ReduceOp.MIN, group=group)
        dist.all_reduce(hi, op=dist.ReduceOp.MAX, group=group)
        a_off[:, g_site] = lo
        a_steps[:, g_site] = torch.clamp((hi - lo) / qu, min=1e-8)
    return a_steps, a_off


class DataParallelModule:
    """One replica of a teacher / student module pair per rank (a `session.ReconModule`), stepped on its share of every
    batch.  All ranks must create their module from the same parameters.  The collectives are torch.distributed's
    (NCCL on GPUs) on ranges of this GPU's own workspace; nothing reads another GPU's memory."""

    def __init__(self, module, group=None):
        import torch.distributed as dist
        from . import binding as B
        self.m, self.group = module, group
        self.world = dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1
        self.rank = dist.get_rank(group) if self.world > 1 else 0
        import torch
        self.buckets = []
        for l in range(module.L):
            ptr, n = B.mrem_grad_bucket(module.ctx, l)
            self.buckets.append(module._ws_view(ptr, n, torch.float32))
        self._B = B

    def shard(self, batch):
        return shard_bounds(batch, self.rank, self.world)

    def init_act_steps(self, x_local, len_local, batch_local, seq):
        m = self.m
        m.init_act_steps(x_local, len_local, batch_local, seq)
        if self.world > 1:
            a, off = m.a_steps[:, :, 0].contiguous(), m.a_off[:, :, 0].contiguous()
            combine_act_ranges(a, off, self.a_bits(), self.asym_sites(), self.group)
            m.a_steps[:, :, 0].copy_(a)
            m.a_off[:, :, 0].copy_(off)
            self._B.mrem_invalidate_weight_codes(m.ctx)

    def a_bits(self):
        return int(self.m.desc.a_bits)

    def asym_sites(self):
        return int(self.m.desc.act_asym_sites)

    def step(self, x_teacher_local, x_student_local, len_local, batch_local, batch_global, seq, optim, lam=0.0):
        """One reconstruction step on this rank's `batch_local` of the step's `batch_global` sequences.  Returns the
        device tensor holding the WHOLE batch's loss (after the all-reduce)."""
        import torch.distributed as dist
        m, B = self.m, self._B
        B.mrem_set_loss_share(m.ctx, batch_local / float(batch_global))
        m.quantize_weights()
        m.forward_teacher(x_teacher_local, len_local, batch_local, seq)
        m.forward_student(x_student_local, len_local, batch_local, seq, x_teacher=x_teacher_local, lam=lam)
        loss, _ = m.recon_loss()
        m.backward()
        works = allreduce_buckets(list(reversed(self.buckets)), self.group, async_op=True)
        if self.world > 1:
            works.append(dist.all_reduce(loss, op=dist.ReduceOp.SUM, group=self.group, async_op=True))
        for w in works:
            w.wait()
        m.step(optim)
        return loss
