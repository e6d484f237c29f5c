"""Sequential module-wise sweep (Algorithm 2 around its inner loop, Sec. 3.2): modules are
optimised one after the other; once module n has taken its T steps, the teacher's and the
student's outputs of module n over the whole calibration set are computed once and cached as
the inputs of module n+1 (the teacher path always sees full-precision activations, the student
path the output of the already-quantized modules below it).

Host orchestration only: batches are gathered, stepped and written back by libmrem calls
(mrem_gather_rows, the captured reconstruction step, mrem_module_forward); every tensor stays
on the device."""
from __future__ import annotations

from typing import Callable, List, Optional, Sequence

import numpy as np
import torch

from . import binding as B
from .session import ReconModule


class ModuleSweep:
    """Runs `steps` reconstruction steps on each module in turn over a device-resident calibration set.

    modules:    the ReconModules, bottom to top, all with the same hidden size, batch and sequence length
    calib:      [N, seq, hidden] storage-type tensor, the input of module 0 (teacher and student alike)
    valid_len:  [N] int32 tensor of valid lengths, or None
    order:      order(module_index, epoch) -> permutation of range(N) as an int array (the seeded sampler)
    weight_step_rule: 0 = max|w| / qmax per row, 1 = mean|w| per row (initial weight steps)
    """

    def __init__(self, modules: Sequence[ReconModule], calib: torch.Tensor, valid_len: Optional[torch.Tensor],
                 batch: int, order: Callable[[int, int], np.ndarray], weight_step_rule: int = 0):
        self.modules = list(modules)
        self.batch = batch
        self.order = order
        self.weight_step_rule = weight_step_rule
        m0 = self.modules[0]
        n, seq, hidden = calib.shape
        assert hidden == m0.H and n % batch == 0 and n >= batch
        self.n, self.seq = n, seq
        self.dev = m0.device
        self.x_teacher = calib                       # inputs of the current module: teacher path ...
        self.x_student = calib                       # ... and student path (identical below the first module)
        self.valid_len = valid_len
        self.losses: List[List[float]] = []
        self._xt = torch.empty(batch, seq, hidden, dtype=calib.dtype, device=self.dev)
        self._xs = torch.empty(batch, seq, hidden, dtype=calib.dtype, device=self.dev)
        self._len = torch.empty(max(batch, 64), dtype=torch.int32, device=self.dev) if valid_len is not None else None

    def _gather(self, idx: torch.Tensor, m: ReconModule, same: bool):
        st = m.stream.cuda_stream
        row_bytes = self.seq * m.H * self.x_teacher.element_size()
        B.mrem_gather_rows(self.x_teacher, idx, self.batch, row_bytes, self._xt, st)
        if not same:
            B.mrem_gather_rows(self.x_student, idx, self.batch, row_bytes, self._xs, st)
        if self._len is not None:       # 4-byte rows are below the gather kernel's 16-byte granule: plain indexing
            self._len[: self.batch].copy_(self.valid_len.index_select(0, idx.long()))

    def run_module(self, k: int, steps: int, optim, lam: float = 0.0, init_steps: bool = True,
                   record_every: int = 1) -> List[float]:
        """T steps on module k (weights are expected to be loaded).  Returns the recorded losses."""
        m = self.modules[k]
        same = self.x_student is self.x_teacher
        xs = self._xt if same else self._xs
        n_batches = self.n // self.batch
        with torch.cuda.stream(m.stream):
            if init_steps:
                first = torch.from_numpy(self.order(k, 0)[: self.batch].astype(np.int32)).to(self.dev)
                self._gather(first, m, same)
                m.init_weight_steps(self.weight_step_rule)
                m.init_act_steps(xs, self._len, self.batch, self.seq)
            if steps > 0:
                # one capture, replayed every step: the staging buffers are the graph's inputs
                B.mrem_graph_capture_step(m.ctx, self._xt, xs, lam, self._len, self.batch, self.seq, m.t_out, m.s_out,
                                          m.loss, optim)
            losses = []
            t = 0
            epoch = 0
            while t < steps:
                perm = torch.from_numpy(self.order(k, epoch).astype(np.int32)).to(self.dev)
                for b in range(n_batches):
                    if t >= steps:
                        break
                    self._gather(perm[b * self.batch:(b + 1) * self.batch], m, same)
                    B.mrem_graph_launch(m.ctx)
                    if record_every and t % record_every == 0:
                        losses.append(m.loss[:1].clone())
                    t += 1
                epoch += 1
            m.stream.synchronize()
        out = [float(v.item()) for v in losses]
        self.losses.append(out)
        return out

    def cache_outputs(self, k: int):
        """Teacher and student outputs of module k over the whole calibration set become the inputs of k+1."""
        m = self.modules[k]
        same = self.x_student is self.x_teacher
        nxt_t = torch.empty_like(self.x_teacher)
        nxt_s = torch.empty_like(self.x_teacher)
        with torch.cuda.stream(m.stream):
            m.quantize_weights()
            for b in range(self.n // self.batch):
                idx = torch.arange(b * self.batch, (b + 1) * self.batch, dtype=torch.int32, device=self.dev)
                self._gather(idx, m, same)
                xs = self._xt if same else self._xs
                t_all = m.forward_teacher(self._xt, self._len, self.batch, self.seq)
                s_all = m.forward_student(xs, self._len, self.batch, self.seq)
                nxt_t[b * self.batch:(b + 1) * self.batch].copy_(t_all[m.L - 1])
                nxt_s[b * self.batch:(b + 1) * self.batch].copy_(s_all[m.L - 1])
            m.stream.synchronize()
        self.x_teacher, self.x_student = nxt_t, nxt_s

    def run(self, steps: int, optim, lam: float = 0.0) -> List[List[float]]:
        for k in range(len(self.modules)):
            self.run_module(k, steps, optim, lam)
            if k + 1 < len(self.modules):
                self.cache_outputs(k)
        return self.losses
