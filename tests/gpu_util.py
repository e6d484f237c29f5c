"""Shared helpers of the GPU parity tests: run the same seeded problem through libmrem and
through the CPU oracle and report relative L2 errors."""
import numpy as np
import torch

from oracle import mrem_oracle as O
from paper_2109_15082_b200 import binding as B
from paper_2109_15082_b200 import synth
from paper_2109_15082_b200.session import ReconModule

SITE_NAMES = ("x", "q", "k", "v", "p", "c", "a", "g")


def rel(got, ref):
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    return float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300))


class Problem:
    """A module pair on the GPU and its twin in the oracle, from identical bytes."""

    def __init__(self, wl, seed=0, student_noise=0.0, step_shrink=1.0, w_per_row=True, asym=3, loss_mean=True,
                 bias_std=0.02, a_bits=None):
        self.wl = wl
        a_bits = a_bits or wl.a_bits
        self.m = ReconModule(wl.n_layers, wl.hidden, wl.n_heads, wl.ffn, wl.seq, wl.batch, wl.w_bits, a_bits,
                             wl.w_grid, w_per_row, asym, wl.act_dtype, loss_mean)
        self.twn = wl.w_grid in (2, 3)                               # closed-form weight scales: no weight steps
        self.desc = O.ModuleDesc(wl.n_layers, wl.hidden, wl.n_heads, wl.ffn, wl.w_bits, a_bits, 0 if self.twn else wl.w_grid,
                                 w_per_row, bool(asym & 1), bool(asym & 2), wl.act_dtype, loss_mean,
                                 w_twn=wl.w_grid == 2, w_laq=wl.w_grid == 3)
        m = self.m
        m.load_teacher(synth.teacher_params(wl, seed, bias_std=bias_std))
        m.init_student_from_teacher()
        if student_noise > 0:
            st = m.student_numpy()
            for l, p in enumerate(st):
                for k in p:
                    p[k] = (p[k] + synth.normal(seed + 1, f"noise{l}{k}", p[k].shape, student_noise)).astype(np.float32)
            m.load_student(st)
        self.teacher = m.teacher_numpy()
        self.student = m.student_numpy()
        x = synth.hidden_states(wl, wl.batch, seed)
        self.xd = m.to_device(x)
        self.x = self.xd.float().cpu().numpy()                       # the stored bytes, widened
        xt = x + synth.normal(seed + 2, "xt", x.shape, 0.05)
        self.xtd = m.to_device(xt)
        self.xt = self.xtd.float().cpu().numpy()
        self.vl = synth.valid_lengths(wl, wl.batch, seed)
        self.vld = torch.from_numpy(self.vl).to(m.device)
        rule = wl.w_step_rule
        ws = O.init_weight_steps(self.desc, self.student, rule)
        a, off = O.init_act_steps(self.desc, self.student, self.x, self.vl)
        a = (a * step_shrink).astype(np.float32)
        ws = [{k: (v * (step_shrink if rule == 0 else 1.0)).astype(np.float32) for k, v in d.items()} for d in ws]
        self.ws, self.a, self.off = ws, a, off
        m.set_steps(ws, a, off)

    def close(self):
        self.m.close()

    def oracle_steps(self):
        return O.make_steps(self.ws, self.a, self.off)

    def run_gpu(self, lam=0.0, same_input=True):
        """quantize, both forwards, loss, backward.  Returns dict of numpy results."""
        m, wl = self.m, self.wl
        xt = self.xd if same_input else self.xtd
        m.quantize_weights()
        ft = m.forward_teacher(xt, self.vld, wl.batch, wl.seq).float().cpu().numpy()
        fs = m.forward_student(self.xd, self.vld, wl.batch, wl.seq, x_teacher=xt, lam=lam).float().cpu().numpy()
        loss, per = m.recon_loss()
        m.backward()
        torch.cuda.synchronize()
        out = dict(f_t=ft, f_s=fs, loss=float(loss[0]), per=per.cpu().numpy(), grads=self.gpu_grads())
        assert m.poll_status() == 0
        return out

    def gpu_grads(self):
        m = self.m
        gs = []
        for l in range(m.L):
            g = {}
            for pid, name in enumerate(B.PARAM_NAMES):
                g[name] = m.grad(l, pid, m.shapes[pid]).cpu().numpy()
            g["w"] = {}
            for k, pid in enumerate((B.WQKV, B.WO, B.W1, B.W2)):
                n = m.shapes[pid][0] if m.per_row else 1
                g["w"][B.PARAM_NAMES[pid]] = None if self.twn else m.grad(l, B.GRAD_STEP + k, (n,)).cpu().numpy()
            g["a"] = np.array([m.grad(l, B.GRAD_STEP + 4 + s, (1,)).item() for s in range(8)])
            g["a_off"] = np.array([m.grad(l, B.GRAD_OFFSET + 4 + s, (1,)).item() for s in range(8)])
            gs.append(g)
        return gs

    def run_oracle(self, lam=0.0, same_input=True):
        xt = self.x if same_input else self.xt
        return O.forward_loss_backward(self.desc, self.teacher, self.student, self.oracle_steps(), xt, self.x,
                                       self.vl, lam)


def compare_grads(gpu, ora, tol, skip_small=1e-12, check_offset=True, scalar_tol=None, deep_scalar_floor=0.02, deep_group_tol=None):
    """Relative L2 error of every gradient group; returns the worst (name, value).

    The offset gradient of the GELU site is the sum of the incoming gradient over the CLIPPED
    elements only.  With freshly initialised steps the range is covered exactly and at most the
    extreme element or two sit on the boundary, on either side of it depending on the last bit
    of erf: that sum is then compared only when `check_offset` (cases that really clip).
    `scalar_tol`: another bound for the activation step gradients (scalars) than for the tensors.
    The eight activation step gradients of a layer are also compared as one group (relative L2 of the 8-vector)
    at `tol`.  `deep_scalar_floor`: the floor (as a share of the layer's largest step gradient) used for the
    scalars of layers above the first; `deep_group_tol`: the bound on their group (default: as for the first layer)."""
    worst = ("", 0.0)
    for l, (g, r) in enumerate(zip(gpu, ora)):
        items = [(k, g[k], r[k]) for k in O.PARAMS]
        items += [("s_" + k, g["w"][k], r["w"][k]) for k in O.WEIGHTS if r["w"][k] is not None]
        if check_offset:
            items += [("a_off", g["a_off"][7:8], r["a_off"][7:8])]
        # activation step gradients are scalars: compare each one on its own; a scalar that is a
        # heavily cancelling sum is measured against the largest of the layer's step gradients
        floor = (0.02 if l == 0 else deep_scalar_floor) * np.abs(r["a"]).max()
        group_tol = (deep_group_tol if (l > 0 and deep_group_tol) else None) or scalar_tol or tol
        assert rel(g["a"], r["a"]) < group_tol, (l, "a_steps as a group", rel(g["a"], r["a"]))
        for s, name in enumerate(SITE_NAMES):
            e = abs(g["a"][s] - r["a"][s]) / max(abs(r["a"][s]), floor, 1e-300)
            assert e < ((deep_group_tol if (l > 0 and deep_group_tol) else None) or scalar_tol or tol), (l, "a_step_" + name, e, g["a"][s], r["a"][s])
            if e > worst[1]:
                worst = (f"L{l}.a_step_{name}", e)
        for name, a, b in items:
            if np.linalg.norm(b) < skip_small:
                continue
            e = rel(a, b)
            bound = deep_group_tol if (name == "a_off" and l > 0 and deep_group_tol) else tol   # a scalar like the step gradients
            assert e < bound, (l, name, e)
            if e > worst[1]:
                worst = (f"L{l}.{name}", e)
    return worst


def code_flip_rate(codes_gpu, codes_ref):
    return float((np.asarray(codes_gpu) != np.asarray(codes_ref)).mean())


def bf16_step(x):
    """Spacing of bfloat16 numbers at the magnitude of x (8 significand bits): 2^(floor(log2|x|) - 7)."""
    a = np.maximum(np.abs(np.asarray(x, np.float64)), 2.0 ** -126)
    return np.exp2(np.floor(np.log2(a)) - 7.0)


def bf16_closeness(got, ref, floor_frac=0.125):
    """Element-wise distance of two bf16-stored tensors of shape [..., hidden], in bfloat16 spacings.

    The unit of element i is the bf16 spacing at max(|ref_i|, floor_frac * rms of its row): two correct
    implementations differ where a value sat within rounding noise of a bf16 rounding boundary (then by exactly
    one spacing of that element) and, for elements far below the row's scale, by the noise that a flipped
    rounding elsewhere in the row sends through the row's mean and variance, which is absolute, not relative.
    Returns dict(frac_differ, frac_over_1, max_units, rel_l2)."""
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    rms = np.sqrt((ref * ref).mean(-1, keepdims=True))
    unit = bf16_step(np.maximum(np.abs(ref), floor_frac * rms))
    d = np.abs(got - ref) / unit
    return dict(frac_differ=float((got != ref).mean()), frac_over_1=float((d > 1.0 + 1e-9).mean()),
                max_units=float(d.max()), rel_l2=rel(got, ref))
