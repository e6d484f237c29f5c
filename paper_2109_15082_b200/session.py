"""Device-memory plumbing around the C-ABI: a ReconModule owns the torch tensors (workspace,
parameters, step sizes, outputs) that one libmrem context borrows, and forwards each call
to the binding.  All arithmetic happens inside libmrem's kernels."""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B

MATRICES = (B.WQKV, B.WO, B.W1, B.W2)


def _align(t: torch.Tensor) -> torch.Tensor:
    assert t.data_ptr() % 256 == 0, "torch allocation not 256-byte aligned"
    return t


class ReconModule:
    """One teacher/student module pair on `device` (a CUDA device)."""

    def __init__(self, n_layers, hidden, n_heads, ffn, max_seq, max_batch, w_bits=4, a_bits=8, w_grid=0,
                 w_step_per_row=True, act_asym_sites=3, act_dtype="bf16", loss_mean=True, trainable_mask=B.TRAIN_ALL,
                 ln_eps=1e-12, device="cuda:0", stream=None):
        if not torch.cuda.is_available():
            raise RuntimeError("ReconModule needs a CUDA device; libmrem has no CPU path")
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.dt = B.BF16 if act_dtype == "bf16" else B.F32
        self.tdtype = torch.bfloat16 if act_dtype == "bf16" else torch.float32
        self.L, self.H, self.h, self.F = n_layers, hidden, n_heads, ffn
        self.max_seq, self.max_batch = max_seq, max_batch
        self.per_row = bool(w_step_per_row)
        self.desc = B.make_desc(n_layers, hidden, n_heads, ffn, max_seq, max_batch, w_bits, a_bits, w_grid,
                                int(self.per_row), act_asym_sites, self.dt, int(loss_mean), trainable_mask, ln_eps)
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        self.ws_bytes = B.mrem_workspace_bytes(self.desc)
        self.workspace = _align(torch.empty(self.ws_bytes, dtype=torch.uint8, device=self.device))
        self.ctx = B.mrem_create(self.desc, self.workspace, self.ws_bytes, self.stream.cuda_stream)
        self.shapes = {B.WQKV: (3 * hidden, hidden), B.BQKV: (3 * hidden,), B.WO: (hidden, hidden), B.BO: (hidden,),
                       B.LN1_G: (hidden,), B.LN1_B: (hidden,), B.W1: (ffn, hidden), B.B1: (ffn,),
                       B.W2: (hidden, ffn), B.B2: (hidden,), B.LN2_G: (hidden,), B.LN2_B: (hidden,)}
        self.teacher, self.student, self.w_steps = [], [], []
        self.a_steps = torch.zeros(n_layers, 8, 64, dtype=torch.float32, device=self.device)   # 256-byte slots
        self.a_off = torch.zeros(n_layers, 8, 64, dtype=torch.float32, device=self.device)
        for l in range(n_layers):
            t, s = {}, {}
            for pid, shp in self.shapes.items():
                tdt = self.tdtype if pid in MATRICES else torch.float32
                t[pid] = _align(torch.zeros(shp, dtype=tdt, device=self.device))
                s[pid] = _align(torch.zeros(shp, dtype=torch.float32, device=self.device))
                B.mrem_bind_param(self.ctx, B.TEACHER, l, pid, t[pid], self.dt if pid in MATRICES else B.F32)
                B.mrem_bind_param(self.ctx, B.STUDENT, l, pid, s[pid], B.F32)
            self.teacher.append(t)
            self.student.append(s)
            ws = []
            for k, pid in enumerate(MATRICES):
                n = self.shapes[pid][0] if self.per_row else 1
                ws.append(_align(torch.ones(n, dtype=torch.float32, device=self.device)))
                B.mrem_bind_steps(self.ctx, l, k, ws[-1], None)
            self.w_steps.append(ws)
            for site in range(8):
                B.mrem_bind_steps(self.ctx, l, 4 + site, self.a_steps[l, site], self.a_off[l, site])
        self.loss = torch.zeros(64, dtype=torch.float32, device=self.device)
        self.loss_per_layer = torch.zeros(max(64, n_layers), dtype=torch.float32, device=self.device)
        self._alloc_outputs(max_batch, max_seq)

    def _alloc_outputs(self, batch, seq):
        n = self.L * batch * seq * self.H
        self.t_out = _align(torch.zeros(n, dtype=self.tdtype, device=self.device))
        self.s_out = _align(torch.zeros(n, dtype=self.tdtype, device=self.device))

    def close(self):
        if self.ctx is not None:
            torch.cuda.synchronize(self.device)
            B.mrem_destroy(self.ctx)
            self.ctx = None

    # ---- parameters -------------------------------------------------------------------
    def load_teacher(self, params):
        """params: per layer a dict name -> float32 numpy array (names of binding.PARAM_NAMES)."""
        for l, p in enumerate(params):
            for pid, name in enumerate(B.PARAM_NAMES):
                self.teacher[l][pid].copy_(torch.from_numpy(np.ascontiguousarray(p[name])).to(self.teacher[l][pid].dtype))

    def load_student(self, params):
        for l, p in enumerate(params):
            for pid, name in enumerate(B.PARAM_NAMES):
                self.student[l][pid].copy_(torch.from_numpy(np.ascontiguousarray(p[name], dtype=np.float32)))
        B.mrem_invalidate_weight_codes(self.ctx)

    def student_numpy(self):
        return [{name: self.student[l][pid].float().cpu().numpy() for pid, name in enumerate(B.PARAM_NAMES)}
                for l in range(self.L)]

    def teacher_numpy(self):
        return [{name: self.teacher[l][pid].float().cpu().numpy() for pid, name in enumerate(B.PARAM_NAMES)}
                for l in range(self.L)]

    def set_steps(self, w_steps, a_steps, a_off):
        """w_steps: per layer dict name->array; a_steps, a_off: [L, 8]."""
        for l in range(self.L):
            for k, pid in enumerate(MATRICES):
                v = np.asarray(w_steps[l][B.PARAM_NAMES[pid]], np.float32).reshape(-1)
                self.w_steps[l][k].copy_(torch.from_numpy(v))
        self.a_steps[:, :, 0].copy_(torch.from_numpy(np.asarray(a_steps, np.float32)))
        self.a_off[:, :, 0].copy_(torch.from_numpy(np.asarray(a_off, np.float32)))
        B.mrem_invalidate_weight_codes(self.ctx)

    def get_steps(self):
        w = [{B.PARAM_NAMES[pid]: self.w_steps[l][k].cpu().numpy() for k, pid in enumerate(MATRICES)}
             for l in range(self.L)]
        return w, self.a_steps[:, :, 0].cpu().numpy(), self.a_off[:, :, 0].cpu().numpy()

    def init_student_from_teacher(self):
        B.mrem_init_student_from_teacher(self.ctx)

    def init_weight_steps(self, rule=0):
        B.mrem_init_weight_steps(self.ctx, rule)

    def init_act_steps(self, x, valid_len, batch, seq):
        B.mrem_init_act_steps(self.ctx, x, valid_len, batch, seq)

    # ---- the step ---------------------------------------------------------------------
    def to_device(self, x_np):
        return _align(torch.from_numpy(np.ascontiguousarray(x_np, dtype=np.float32)).to(self.device).to(self.tdtype).contiguous())

    def quantize_weights(self):
        B.mrem_quantize_weights(self.ctx)

    def forward_teacher(self, x, valid_len, batch, seq):
        B.mrem_module_forward(self.ctx, B.TEACHER, x, None, 0.0, valid_len, batch, seq, self.t_out)
        return self.t_out[: self.L * batch * seq * self.H].view(self.L, batch, seq, self.H)

    def forward_student(self, x, valid_len, batch, seq, x_teacher=None, lam=0.0):
        B.mrem_module_forward(self.ctx, B.STUDENT, x, x_teacher, lam, valid_len, batch, seq, self.s_out)
        return self.s_out[: self.L * batch * seq * self.H].view(self.L, batch, seq, self.H)

    def recon_loss(self):
        B.mrem_recon_loss(self.ctx, self.loss, self.loss_per_layer)
        return self.loss[:1], self.loss_per_layer[: self.L]

    def backward(self):
        B.mrem_module_backward(self.ctx)

    def set_fused_attention_backward(self, on):
        B.mrem_set_fused_attention_backward(self.ctx, on)

    def step(self, optim):
        B.mrem_step(self.ctx, optim)

    def input_grad(self, batch, seq):
        """d loss / d (student module input) of the last backward pass, [batch, seq, hidden] (a copy)."""
        return self._ws_view(B.mrem_get_input_grad(self.ctx), batch * seq * self.H, self.tdtype).view(batch, seq, self.H).clone()

    def activation(self, role, layer, which, shape):
        """A copy of a tensor the last forward pass of `role` stored inside `layer` (binding.ACT_*)."""
        ptr = B.mrem_get_activation(self.ctx, role, layer, which)
        return self._ws_view(ptr, int(np.prod(shape)), self.tdtype).view(*shape).clone()

    def bind_head(self, head):
        """head: dict Wp [H, H], bp [H], Wc [C, H], bc [C] (numpy) of the classification head, or None to unbind."""
        if head is None:
            B.mrem_bind_head(self.ctx, None, None, None, None, 0)
            self._head = None
            return
        t = {k: torch.from_numpy(np.ascontiguousarray(head[k], dtype=np.float32)).to(self.device) for k in ("Wp", "bp", "Wc", "bc")}
        C_ = int(t["Wc"].shape[0])
        self.logit_loss = torch.zeros(1, dtype=torch.float32, device=self.device)
        self.logits = torch.zeros(2, self.max_batch, C_, dtype=torch.float32, device=self.device)
        self._head = t                                       # keeps the device tensors alive while bound
        B.mrem_bind_head(self.ctx, t["Wp"], t["bp"], t["Wc"], t["bc"], C_, self.logit_loss, self.logits)

    def rem_step(self, layer, tensor_id, a, optim):
        """One step of Eq. 2 on one matrix product; `a` is a [rows, in] device tensor (optim None: loss and
        gradients only).  Returns the loss tensor."""
        B.mrem_rem_step(self.ctx, layer, tensor_id, a, a.shape[0], optim, self.loss)
        return self.loss[:1]

    def backward_and_step(self, optim):
        B.mrem_backward_and_step(self.ctx, optim)

    def grad(self, layer, grad_id, shape):
        ptr = B.mrem_get_grad(self.ctx, layer, grad_id)
        n = int(np.prod(shape))
        return self._ws_view(ptr, n, torch.float32).view(*shape).clone()

    def weight_codes(self, layer, pid):
        codes, rowsum = B.mrem_get_weight_codes(self.ctx, layer, pid)
        rows, cols = self.shapes[pid]
        return (self._ws_view(codes, rows * cols, torch.int8).view(rows, cols).clone(),
                self._ws_view(rowsum, rows, torch.int32).clone())

    def _ws_view(self, ptr, n, dtype):
        """A typed view of `n` elements at a borrowed address inside the workspace."""
        off = ptr - self.workspace.data_ptr()
        nbytes = n * torch.empty((), dtype=dtype).element_size()
        assert 0 <= off and off + nbytes <= self.ws_bytes
        return self.workspace[off: off + nbytes].view(dtype)

    def poll_status(self):
        return B.mrem_poll_status(self.ctx)
