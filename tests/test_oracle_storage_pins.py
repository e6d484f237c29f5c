"""Pins for the parts of the CPU oracle that the module-level autograd pins do not reach (they run in 'f64'
storage, which rounds nowhere): the initial activation steps, WHERE the storage-emulation mode rounds, and the
bookkeeping of a whole reconstruction step (weight decay on the four matrices only, the positivity clamp of
the step sizes).  Each is held against torch library layers / torch.optim.AdamW or against what Eq. 1 fixes,
never against the oracle's own formula.  No GPU needed."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import mrem_oracle as O
from paper_2109_15082_b200 import synth


def _case(act_dtype, n_layers=1, H=32, h=2, Fd=64, B=3, S=8, seed=0, **kw):
    wl = synth.Workload("pin2", n_layers, H, h, Fd, S, B, act_dtype=act_dtype, outlier_channels=2)
    params = synth.teacher_params(wl, seed, bias_std=0.1)
    for p in params:
        for k in O.WEIGHTS:
            p[k] = (p[k] * 8).astype(np.float32)
            if act_dtype == "bf16":
                p[k] = O.round_bf16(p[k]).astype(np.float32)
    x = synth.hidden_states(wl, B, seed)
    if act_dtype == "bf16":
        x = O.round_bf16(x).astype(np.float32)
    desc = O.ModuleDesc(n_layers, H, h, Fd, act_dtype=act_dtype, **kw)
    return desc, params, x


def _site_tensors_torch(p, x, vl, h):
    """The eight tensors that feed a quantizer inside one unquantized layer, from torch library layers."""
    t = {k: torch.tensor(np.asarray(v, np.float64)) for k, v in p.items()}
    xt = torch.tensor(np.asarray(x, np.float64))
    B, S, H = xt.shape
    d = H // h
    qkv = F.linear(xt, t["Wqkv"], t["bqkv"])
    Q, K, V = qkv.split(H, dim=-1)
    sp = lambda u: u.reshape(B, S, h, d).transpose(1, 2)
    pad = (torch.arange(S)[None, :] >= torch.as_tensor(vl)[:, None])[:, None, None, :]
    P = torch.softmax((sp(Q) @ sp(K).transpose(-1, -2) / math.sqrt(d)).masked_fill(pad, float("-inf")), dim=-1)
    ctx = (P @ sp(V)).transpose(1, 2).reshape(B, S, H)
    a = F.layer_norm(F.linear(ctx, t["Wo"], t["bo"]) + xt, (H,), t["ln1_g"], t["ln1_b"], 1e-12)
    g = F.gelu(F.linear(a, t["W1"], t["b1"]))
    return [u.numpy() for u in (xt, Q, K, V, P, ctx, a, g)]


@pytest.mark.parametrize("a_bits", [8, 4])
@pytest.mark.parametrize("asym", [True, False])
def test_initial_activation_steps_put_the_extremes_on_the_ends_of_the_code_range(a_bits, asym):
    """Initial activation steps: one unquantized pass over the first batch, then per site the step that maps the
    batch's extreme value onto the last code, so that Eq. 1 clips nothing at the start: symmetric sites
    max|x| -> +-qmax; the softmax site (offset 0) max -> 2^b - 1; the GELU site min -> 0 (offset = min) and
    max -> 2^b - 1."""
    desc, params, x = _case("f64", w_bits=4, a_bits=a_bits, asym_p=asym, asym_g=asym)
    vl = np.array([8, 5, 1], np.int32)
    a, off = O.init_act_steps(desc, params, x, vl)
    tens = _site_tensors_torch(params[0], x, vl, desc.n_heads)
    qs, qu = 2 ** (a_bits - 1) - 1, 2 ** a_bits - 1
    for site, t in enumerate(tens):
        t32 = t.astype(np.float32)
        s = np.float32(a[0, site])
        if asym and site in (O.SITE_P, O.SITE_G):
            beta = np.float32(off[0, site])
            if site == O.SITE_P:
                assert beta == 0.0
            else:
                assert beta == t32.min()                                    # the offset is the minimum itself
            q, z = O.quantize_asym(t32, s, beta, a_bits)
            assert q.min() == 0 and q.max() == qu
            assert z.min() >= 0.0 and z.max() <= qu * (1 + 2.0 ** -22)      # nothing beyond the range (one rounding of slack)
            assert np.all(np.abs(s * q.astype(np.float64) + beta - t32) <= 0.5 * s * (1 + 1e-6))
        else:
            assert off[0, site] == 0.0
            q, z = O.quantize_sym(t32, s, a_bits)
            assert np.abs(q).max() == qs
            assert np.abs(z).max() <= qs * (1 + 2.0 ** -22)
            assert np.all(np.abs(s * q.astype(np.float64) - t32) <= 0.5 * s * (1 + 1e-6))
            # the step is the smallest that clips nothing: a 1 % smaller one pushes the extreme out of range
            assert np.abs(O.quantize_sym(t32, np.float32(s * 0.99), a_bits)[1]).max() > qs


# ----------------------------------------------------------------------------- where the storage mode rounds

from tests.torch_storage_ref import round_bf16_t as _bf, teacher_layer_torch as _teacher_layer_torch, bf16_numbers_apart as _ulps_apart


def test_teacher_layer_rounds_where_the_storage_type_says():
    desc, params, x = _case("bf16", w_bits=0, a_bits=0)
    vl = np.array([8, 5, 2], np.int32)
    got = O.teacher_layer(desc, params[0], x, vl)
    want = _teacher_layer_torch(params[0], x, vl, desc.n_heads, _bf)
    assert np.array_equal(O.round_bf16(got), got)                         # the output itself is stored
    apart = _ulps_apart(got, want)
    # float64 sums in another order can tip a value that sits on a rounding boundary, nothing else
    assert apart.max() <= 1 and (apart > 0).mean() < 2e-3, (apart.max(), (apart > 0).mean())
    # and the roundings matter: without them the result is measurably different
    plain = _teacher_layer_torch(params[0], x, vl, desc.n_heads, lambda t: t)
    assert 1e-4 < np.linalg.norm(got - plain) / np.linalg.norm(plain) < 2e-2
    # leaving out any single rounding is visible: drop them one at a time in the torch model
    calls = {"n": 0}

    def counting(t):
        calls["n"] += 1
        return _bf(t)

    _teacher_layer_torch(params[0], x, vl, desc.n_heads, counting)
    n_roundings = calls["n"]
    assert n_roundings == 13          # 4 matrices, input, qkv, P, ctx, y1, a, g, y2, output (nothing pre-GELU)
    for skip in range(n_roundings):
        calls["n"] = 0

        def all_but_one(t):
            calls["n"] += 1
            return t if calls["n"] - 1 == skip else _bf(t)

        other = _teacher_layer_torch(params[0], x, vl, desc.n_heads, all_but_one)
        if skip < 5 or skip == n_roundings - 1:
            continue                   # inputs are representable already; the last one is checked above
        assert (_ulps_apart(O.round_bf16(other), got) > 0).mean() > 5e-3, skip


def test_student_layer_stores_and_decides_on_stored_values():
    """Storage mode in the quantized layer: every tensor the backward pass re-reads (qkv, softmax output, context,
    both pre-LayerNorm sums, the first LayerNorm's output, the pre-GELU tensor, the GELU output, the layer output)
    holds values of the storage type, and every quantizer takes its decision from those stored values in float32:
    the codes are Eq. 1 applied, in float32, to the cached tensor itself."""
    desc, params, x = _case("bf16", w_bits=4, a_bits=8)
    vl = np.array([8, 5, 2], np.int32)
    ws = O.init_weight_steps(desc, params, 0)
    a, off = O.init_act_steps(desc, params, x, vl)
    steps = O.make_steps(ws, (a * 0.8).astype(np.float32), off)
    f, c = O.student_layer(desc, params[0], steps[0], x, vl)
    for name in ("qkv", "P", "ctx", "y1", "a", "u", "g", "y2", "f"):
        assert np.array_equal(O.round_bf16(c[name]), c[name]), name
        assert not np.array_equal(c[name], np.zeros_like(c[name]))
    Q, K, V = np.split(c["qkv"], 3, axis=-1)
    for key, site, t in (("qx", O.SITE_X, x), ("qQ", O.SITE_Q, Q), ("qK", O.SITE_K, K), ("qV", O.SITE_V, V),
                         ("qC", O.SITE_C, c["ctx"]), ("qA", O.SITE_A, c["a"])):
        s = np.float32(steps[0]["a"][site])
        z32 = (t.astype(np.float32) / s).astype(np.float32)                # Eq. 1 in float32 on the stored value
        assert np.array_equal(c[key]["q"], np.rint(np.clip(z32, -127, 127)).astype(np.int64)), key
    for key, site, t, beta in (("qP", O.SITE_P, c["P"], 0.0), ("qG", O.SITE_G, c["g"], steps[0]["a_off"][O.SITE_G])):
        s = np.float32(steps[0]["a"][site])
        z32 = ((t.astype(np.float32) - np.float32(beta)).astype(np.float32) / s).astype(np.float32)
        assert np.array_equal(c[key]["q"], np.rint(np.clip(z32, 0, 255)).astype(np.int64)), key
    # the GELU output is rounded BEFORE its quantizer sees it (the quantizer reads a stored tensor)
    assert np.array_equal(c["g"], O.round_bf16(O.gelu(c["u"])))
    # 'f32' storage keeps float32 values, 'f64' rounds nowhere, and the three stay close to one another
    outs = {}
    for dt in ("bf16", "f32", "f64"):
        d2 = O.ModuleDesc(**{**desc.__dict__, "act_dtype": dt})
        outs[dt], c2 = O.student_layer(d2, params[0], steps[0], x, vl)
        if dt == "f32":
            assert np.array_equal(c2["u"].astype(np.float32).astype(np.float64), c2["u"])
    rel = lambda p, q: np.linalg.norm(p - q) / np.linalg.norm(q)
    assert 0 < rel(outs["f32"], outs["f64"]) < 2e-2 and 1e-4 < rel(outs["bf16"], outs["f64"]) < 5e-2


# ----------------------------------------------------------------------------- a whole step's bookkeeping

def test_recon_step_decays_only_the_matrices_and_keeps_steps_positive():
    """Two whole steps against torch.optim.AdamW fed with the oracle's own gradients (those are pinned against
    autograd elsewhere): the four matrices of a layer are decayed, nothing else is; the step count advances by one
    per call and is shared by all parameters; step sizes never fall below the smallest positive value allowed
    (Eq. 1 needs s > 0) and offsets are not clamped."""
    desc, params, x = _case("f64", n_layers=2, w_bits=4, a_bits=8)
    vl = np.array([8, 6, 3], np.int32)
    teacher = [{k: v.copy() for k, v in p.items()} for p in params]
    student = [{k: (v + synth.normal(3, f"n{l}{k}", v.shape, 0.01)).astype(np.float32) for k, v in p.items()}
               for l, p in enumerate(params)]
    ws = O.init_weight_steps(desc, student, 0)
    a, off = O.init_act_steps(desc, student, x, vl)
    a = (a * 0.8).astype(np.float32)
    # two step sizes that the first update would push below zero
    ws[0]["Wo"][3] = np.float32(3e-8)
    a[1, O.SITE_C] = np.float32(2e-8)
    steps = O.make_steps(ws, a, off)
    lr, wd = 1e-3, 0.1
    # torch side: float64 leaves, two parameter groups
    tp = [{k: torch.tensor(np.asarray(v, np.float64), requires_grad=True) for k, v in p.items()} for p in student]
    tsw = [{k: torch.tensor(np.asarray(s["w"][k], np.float64), requires_grad=True) for k in O.WEIGHTS} for s in steps]
    tsa = [torch.tensor(np.asarray(s["a"], np.float64), requires_grad=True) for s in steps]
    tso = [torch.tensor(np.asarray(s["a_off"], np.float64), requires_grad=True) for s in steps]
    decayed = [tp[l][k] for l in range(2) for k in O.WEIGHTS]
    plain = [tp[l][k] for l in range(2) for k in O.PARAMS if k not in O.WEIGHTS] + [t for d in tsw for t in d.values()] + tsa + tso
    opt = torch.optim.AdamW([dict(params=decayed, weight_decay=wd), dict(params=plain, weight_decay=0.0)], lr=lr,
                            betas=(0.9, 0.999), eps=1e-8)
    state = {}
    for t in range(1, 3):
        cur_student = [{k: v.copy() for k, v in p.items()} for p in student]
        cur_steps = [dict(w={k: v.copy() for k, v in s["w"].items()}, a=s["a"].copy(), a_off=s["a_off"].copy()) for s in steps]
        g = O.forward_loss_backward(desc, teacher, cur_student, cur_steps, x, x, vl)["grads"]
        O.recon_step(desc, teacher, student, steps, state, x, x, vl, lr=lr, weight_decay=wd)
        assert state["t"] == t
        for l in range(2):
            for k in O.PARAMS:
                tp[l][k].grad = torch.tensor(np.asarray(g[l][k], np.float64))
            for k in O.WEIGHTS:
                tsw[l][k].grad = torch.tensor(np.asarray(g[l]["w"][k], np.float64))
            tsa[l].grad = torch.tensor(np.asarray(g[l]["a"], np.float64))
            tso[l].grad = torch.tensor(np.asarray(g[l]["a_off"], np.float64))
        opt.step()
        with torch.no_grad():                                      # the clamp is part of the method's step, not of AdamW
            for l in range(2):
                for k in O.WEIGHTS:
                    tsw[l][k].clamp_(min=1e-8)
                tsa[l].clamp_(min=1e-8)
                # the oracle keeps parameters and steps in float32 between steps
                for k in O.PARAMS:
                    tp[l][k].copy_(tp[l][k].float().double())
                for k in O.WEIGHTS:
                    tsw[l][k].copy_(tsw[l][k].float().double())
                tsa[l].copy_(tsa[l].float().double())
                tso[l].copy_(tso[l].float().double())
        for l in range(2):
            for k in O.PARAMS:
                assert np.array_equal(student[l][k], tp[l][k].detach().numpy().astype(np.float32)), (t, l, k)
            for k in O.WEIGHTS:
                assert np.array_equal(steps[l]["w"][k], tsw[l][k].detach().numpy().astype(np.float32)), (t, l, "s", k)
            assert np.array_equal(steps[l]["a"], tsa[l].detach().numpy().astype(np.float32)), (t, l, "a")
            assert np.array_equal(steps[l]["a_off"], tso[l].detach().numpy().astype(np.float32)), (t, l, "off")
        if t == 1:
            # the two tiny steps had positive gradients large enough to cross zero: they sit on the floor now
            assert g[0]["w"]["Wo"][3] != 0 and g[1]["a"][O.SITE_C] != 0
    assert steps[0]["w"]["Wo"].min() >= np.float32(1e-8) and steps[1]["a"].min() >= np.float32(1e-8)
    # decay really differs between the groups: with the gradient's part removed, a matrix shrank by lr * wd, a bias did not
    assert wd > 0 and not np.array_equal(student[0]["Wqkv"], params[0]["Wqkv"])
