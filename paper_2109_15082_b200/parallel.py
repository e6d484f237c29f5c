"""Parallel module-wise training (Algorithm 1, Sec. 4.2) on one GPU: every module is a libmrem context on
its own CUDA stream, adjacent modules are connected by first-in-first-out input queues of the last t0
outputs (teacher-side and student-side), and the student's input is the annealed teacher-forcing mix of
Eq. 4.  A module reads only what its predecessor produced in earlier steps (in the same step while the
queues are being filled), so the modules of one step run concurrently; the streams are ordered by events.

Host orchestration only: gathers, forward passes, loss, backward and update are libmrem calls; the queues
are device tensors that the calls write into and read from."""
from __future__ import annotations

from typing import Callable, List, Optional, Sequence

import numpy as np
import torch

from . import binding as B
from .session import ReconModule


class ParallelModules:
    """modules:   ReconModules bottom to top, each created on its OWN stream, same batch / seq / hidden
    calib:     [N, seq, hidden] storage-type tensor; valid_len: [N] int32 tensor or None
    batch_ids: batch_ids(t) -> indices of the calibration batch module 0 takes at step t (int array)
    draws:     draws[t][n] in [0, t0): which of the t0 most recent queue entries module n >= 1 samples at
               step t >= t0 (0 = most recent); the same entry on the teacher and the student side
    t0:        staleness threshold = queue length; the first t0 steps fill the queues sequentially
    T0:        steps of teacher forcing: lambda_t = max(1 - t / T0, 0) for t < T0, none afterwards
    """

    def __init__(self, modules: Sequence[ReconModule], calib: torch.Tensor, valid_len: Optional[torch.Tensor], batch: int,
                 batch_ids: Callable[[int], np.ndarray], draws: np.ndarray, t0: int, T0: int):
        assert t0 >= 1
        self.mods = list(modules)
        self.N = len(self.mods)
        self.calib, self.valid_len, self.batch = calib, valid_len, batch
        self.batch_ids, self.draws, self.t0, self.T0 = batch_ids, np.asarray(draws), t0, T0
        m0 = self.mods[0]
        self.dev, self.seq, self.H = m0.device, calib.shape[1], m0.H
        assert len({m.stream.cuda_stream for m in self.mods}) == self.N, "each module needs its own stream"
        shape = (t0 + 1, batch, self.seq, self.H)          # one slot more than the queue holds: the slot being
        self.q_t = [torch.zeros(shape, dtype=calib.dtype, device=self.dev) for _ in range(self.N)]   # written is never sampled
        self.q_s = [torch.zeros(shape, dtype=calib.dtype, device=self.dev) for _ in range(self.N)]
        self.q_len = [torch.zeros(t0 + 1, max(batch, 64), dtype=torch.int32, device=self.dev) for _ in range(self.N)]
        self.x0 = torch.zeros(batch, self.seq, self.H, dtype=calib.dtype, device=self.dev)
        self.len0 = torch.zeros(max(batch, 64), dtype=torch.int32, device=self.dev)
        self.done = [[None, None] for _ in range(self.N)]  # events of the two most recent steps of each module
        self.loss_log: List[List[torch.Tensor]] = [[] for _ in range(self.N)]
        self.t = 0

    def _slot(self, t: int) -> int:
        return t % (self.t0 + 1)

    def init_steps(self, weight_step_rule: int = 0):
        """Initial step sizes of every module: module n sees the first calibration batch after it went through
        the full-precision modules below it."""
        idx = torch.from_numpy(self.batch_ids(0).astype(np.int32)).to(self.dev)
        x = self.calib.index_select(0, idx.long()).contiguous()
        ln = None
        if self.valid_len is not None:
            ln = torch.zeros(max(self.batch, 64), dtype=torch.int32, device=self.dev)
            ln[: self.batch] = self.valid_len.index_select(0, idx.long())
        torch.cuda.synchronize(self.dev)
        for m in self.mods:
            with torch.cuda.stream(m.stream):
                m.init_weight_steps(weight_step_rule)
                m.init_act_steps(x, ln, self.batch, self.seq)
                out = m.forward_teacher(x, ln, self.batch, self.seq)[m.L - 1].clone()
                m.stream.synchronize()
            x = out

    def step(self, optim_of: Callable[[int], "B.Optim"]):
        """One step t of every module (Algorithm 1's loop body, the modules side by side)."""
        t, t0 = self.t, self.t0
        lam = max(1.0 - t / self.T0, 0.0) if (self.T0 > 0 and t < self.T0) else 0.0
        filling = t < t0
        new_events = []
        for n, m in enumerate(self.mods):
            st = m.stream
            with torch.cuda.stream(st):
                if n == 0:
                    idx = torch.from_numpy(self.batch_ids(t).astype(np.int32)).to(self.dev, non_blocking=False)
                    row_bytes = self.seq * self.H * self.calib.element_size()
                    B.mrem_gather_rows(self.calib, idx, self.batch, row_bytes, self.x0, st.cuda_stream)
                    xt = xs = self.x0
                    ln = None
                    if self.valid_len is not None:
                        self.len0[: self.batch].copy_(self.valid_len.index_select(0, idx.long()))
                        ln = self.len0
                else:
                    if filling:
                        src_t, k = t, None                   # the predecessor's output of this very step
                        st.wait_event(new_events[n - 1])
                    else:
                        k = int(self.draws[t][n])
                        assert 0 <= k < t0
                        src_t = t - 1 - k
                        st.wait_event(self.done[n - 1][(t - 1) & 1])   # everything up to step t-1 of the predecessor
                    s = self._slot(src_t)
                    xt, xs = self.q_t[n - 1][s], self.q_s[n - 1][s]
                    ln = self.q_len[n - 1][s] if self.valid_len is not None else None
                # the slot this step writes was last readable by the successor in its step t-1
                if n + 1 < self.N and self.done[n + 1][(t - 1) & 1] is not None:
                    st.wait_event(self.done[n + 1][(t - 1) & 1])
                m.quantize_weights()
                f_t = m.forward_teacher(xt, ln, self.batch, self.seq)
                f_s = m.forward_student(xs, ln, self.batch, self.seq, x_teacher=xt, lam=lam)
                m.recon_loss()
                self.loss_log[n].append(m.loss[:1].clone())
                w = self._slot(t)
                self.q_t[n][w].copy_(f_t[m.L - 1])
                self.q_s[n][w].copy_(f_s[m.L - 1])
                if ln is not None:
                    self.q_len[n][w].copy_(ln)
                m.backward_and_step(optim_of(t))
                ev = torch.cuda.Event()
                ev.record(st)
                new_events.append(ev)
        for n in range(self.N):
            self.done[n][t & 1] = new_events[n]
        self.t += 1

    def run(self, T: int, optim_of) -> List[List[float]]:
        for _ in range(T):
            self.step(optim_of)
        torch.cuda.synchronize(self.dev)
        return [[float(v.item()) for v in log] for log in self.loss_log]
