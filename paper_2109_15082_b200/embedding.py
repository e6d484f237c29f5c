"""Owner of the tensors of the embedding step (first module of the model): torch allocates, libmrem computes."""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B

TABLES = ("word", "pos", "type", "ln_g", "ln_b")


class EmbeddingStep:
    """Teacher and student embedding tables on the device, gradients, AdamW moments and the workspace of
    `mrem_embed_step`.  `teacher`: dict word [V, H], pos [P, H], type [T, H], ln_g [H], ln_b [H] (numpy)."""

    def __init__(self, teacher, e_bits, max_tokens, act_dtype="bf16", loss_mean=True, ln_eps=1e-12, device="cuda:0", stream=None):
        if not torch.cuda.is_available():
            raise RuntimeError("EmbeddingStep needs a CUDA device (there is no CPU path)")
        self.device = torch.device(device)
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        V, H = teacher["word"].shape
        self.V, self.H, self.P, self.T = V, H, teacher["pos"].shape[0], teacher["type"].shape[0]
        self.tdtype = torch.bfloat16 if act_dtype == "bf16" else torch.float32
        self.desc = B.make_embed_desc(V, H, self.P, self.T, e_bits, B.BF16 if act_dtype == "bf16" else B.F32, int(loss_mean), ln_eps)
        f32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(self.device)
        self.t = {k: f32(teacher[k]) for k in TABLES}
        self.s = {k: self.t[k].clone() for k in TABLES}
        self.word_step = torch.ones(V, dtype=torch.float32, device=self.device)
        zeros = lambda ref: torch.zeros_like(ref)
        self.g = {k: zeros(self.s[k]) for k in TABLES}
        self.g["word_step"] = zeros(self.word_step)
        self.m = {k: zeros(v) for k, v in self.g.items()}
        self.v = {k: zeros(v) for k, v in self.g.items()}
        self.counter = torch.zeros(1, dtype=torch.int32, device=self.device)
        self.status = torch.zeros(1, dtype=torch.int32, device=self.device)
        self.loss = torch.zeros(1, dtype=torch.float32, device=self.device)
        self.max_tokens = max_tokens
        self.ws_bytes = B.mrem_embed_workspace_bytes(self.desc, max_tokens)
        self.workspace = torch.empty(self.ws_bytes + 256, dtype=torch.uint8, device=self.device)
        off = (-self.workspace.data_ptr()) % 256
        self.ws_ptr = self.workspace.data_ptr() + off
        self.e_teacher = torch.empty(max_tokens * H, dtype=self.tdtype, device=self.device)
        self.e_student = torch.empty(max_tokens * H, dtype=self.tdtype, device=self.device)
        self.dirty = True                                  # the codes in the workspace do not match word / word_step yet
        ptr = lambda t: t.data_ptr()
        vals = dict(t_word=ptr(self.t["word"]), t_pos=ptr(self.t["pos"]), t_type=ptr(self.t["type"]), t_ln_g=ptr(self.t["ln_g"]),
                    t_ln_b=ptr(self.t["ln_b"]), word_step=ptr(self.word_step), d_step_counter=ptr(self.counter))
        for k in TABLES:
            vals[k] = ptr(self.s[k])
        for k in self.g:
            vals["g_" + k], vals["m_" + k], vals["v_" + k] = ptr(self.g[k]), ptr(self.m[k]), ptr(self.v[k])
        self.tensors = B.EmbedTensors(**{n: vals[n] for n in B.EMBED_TENSOR_FIELDS})

    def set_student(self, tables=None, word_step=None):
        for k, a in (tables or {}).items():
            self.s[k].copy_(torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)))
        if word_step is not None:
            self.word_step.copy_(torch.from_numpy(np.ascontiguousarray(word_step, dtype=np.float32)))
        self.dirty = True

    def step(self, ids, type_ids, optim, extra_grad=None):
        """ids, type_ids: int32 device tensors [batch, seq].  optim None: loss and gradients only.  extra_grad: device
        tensor or address of a gradient at the student's embedding output (the first module's input gradient).
        Returns the loss tensor."""
        batch, seq = ids.shape
        B.mrem_embed_step(self.desc, self.tensors, self.ws_ptr, self.ws_bytes, ids, type_ids, batch, seq, int(self.dirty),
                          self.e_teacher, self.e_student, extra_grad, optim, self.loss, self.status, self.stream.cuda_stream)
        self.dirty = False
        return self.loss[:1]

    def outputs(self, batch, seq):
        n = batch * seq * self.H
        return self.e_teacher[:n].view(batch, seq, self.H), self.e_student[:n].view(batch, seq, self.H)
