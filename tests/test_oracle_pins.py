"""Pins for the CPU oracle: each part is checked against something other than itself
(facts fixed by Eq. 1 / Eq. 2 / Eq. 3 / Eq. 4, brute force, closed forms, library
autograd).  These run without a GPU."""
import itertools

import numpy as np
import pytest
import torch

from oracle import mrem_oracle as O
from paper_2109_15082_b200 import synth
from tests import torch_ste_ref as R


# ----------------------------------------------------------------------------- Eq. 1 quantizer

@pytest.mark.parametrize("bits", [2, 4, 8])
def test_code_range_is_omega_b(bits):
    # Omega(b) = {-2^(b-1)+1 .. 2^(b-1)-1}: the most negative two's-complement code never appears
    x = synth.normal(1, "rng", (20000,), 3.0)
    q, _ = O.quantize_sym(x, np.float32(0.01), bits)
    qmax = 2 ** (bits - 1) - 1
    assert q.min() == -qmax and q.max() == qmax
    assert set(np.unique(q)).issubset(set(range(-qmax, qmax + 1)))


def test_omega_2_is_ternary_and_printed_ranges():
    assert O.sym_qmax(2) == 1 and O.sym_qmax(4) == 7 and O.sym_qmax(8) == 127


@pytest.mark.parametrize("bits", [4, 8])
def test_grid_points_ties_and_error_bound(bits):
    s = np.float32(0.125)                          # power of two: x = s*k is exact
    qmax = 2 ** (bits - 1) - 1
    k = np.arange(-qmax - 3, qmax + 4)
    q, _ = O.quantize_sym((s * k).astype(np.float32), s, bits)
    assert np.array_equal(q, np.clip(k, -qmax, qmax))            # grid points map to themselves, then clip
    halves = np.array([0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.5], np.float32) * s
    q, _ = O.quantize_sym(halves, s, bits)
    assert q.tolist() == [0, 2, 2, 0, -2, -2, 4]                 # closest integer, ties to even
    x = synth.normal(2, "err", (5000,), 0.3)
    q, z = O.quantize_sym(x, s, bits)
    inside = np.abs(x / s) <= qmax
    assert np.all(np.abs(s * q - x)[inside] <= s / 2 + 1e-7)     # closest integer => |x_hat - x| <= s/2


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_idempotence(bits):
    x = synth.normal(3, "idem", (4096,), 1.0)
    s = np.float32(0.037)
    q1, _ = O.quantize_sym(x, s, bits)
    q2, _ = O.quantize_sym((s * q1).astype(np.float32), s, bits)
    assert np.array_equal(q1, q2)
    qa, _ = O.quantize_asym(np.abs(x), s, np.float32(-0.17), 8)
    xa = (s * qa.astype(np.float32) + np.float32(-0.17)).astype(np.float32)
    qb, _ = O.quantize_asym(xa, s, np.float32(-0.17), 8)
    assert np.array_equal(qa, qb) and qa.min() >= 0 and qa.max() <= 255


def test_half_integer_2bit_grid_is_nearest_level():
    s = np.float32(0.25)
    x = synth.normal(4, "w2", (4000,), 0.4)
    c, scale, _ = O.quantize_weight(x.reshape(1, -1), np.array([[s]], np.float32), 2, 1)
    what = (scale * c).reshape(-1)
    levels = np.array([-1.5, -0.5, 0.5, 1.5]) * s
    nearest = levels[np.abs(x[:, None].astype(np.float64) - levels[None, :]).argmin(1)]
    assert set(np.unique(c)) == {-3, -1, 1, 3}
    assert np.allclose(what, nearest)


def test_initial_weight_steps_clip_nothing():
    wl = synth.workloads()["tiny"]
    params = synth.teacher_params(wl, 0)
    desc = O.ModuleDesc(1, wl.hidden, wl.n_heads, wl.ffn, 4, 8)
    s = O.init_weight_steps(desc, params, 0)[0]
    for k in O.WEIGHTS:
        q, _, z = O.quantize_weight(params[0][k], s[k].reshape(-1, 1), 4, 0)
        assert np.all(np.abs(q).max(-1) == 7)                    # each row's largest weight gets code +-7
        assert np.all(np.abs(z) <= 7 * (1 + 1e-6))               # and nothing is clipped


# ----------------------------------------------------------------------------- integer products, Eq. 2

def test_int_matmul_brute_force():
    rng = np.random.default_rng(0)
    qa = rng.integers(-127, 128, (5, 19))
    qw = rng.integers(-7, 8, (7, 19))
    ref = [[sum(int(qa[m, k]) * int(qw[n, k]) for k in range(19)) for n in range(7)] for m in range(5)]
    assert O.int_matmul(qa, qw).tolist() == ref


@pytest.mark.parametrize("asym", [False, True])
def test_student_linear_is_quantized_product_of_eq2(asym):
    # y = w_hat^T a_hat (+ bias): integer accumulate + scales must equal the float product
    x = np.abs(synth.normal(5, "a", (6, 24), 1.0)) if asym else synth.normal(5, "a", (6, 24), 1.0)
    w = synth.normal(5, "w", (10, 24), 0.02)
    b = synth.normal(5, "b", (10,), 0.1).astype(np.float64)
    desc = O.ModuleDesc(1, 24, 1, 10, 4, 8, act_dtype="f32", asym_g=asym)
    sw = O.init_weight_steps(desc, [dict(Wqkv=w, Wo=w, W1=w, W2=w)])[0]["W1"]
    steps = dict(a=np.full(8, 0.02, np.float32), a_off=np.full(8, 0.11, np.float32))
    qa = O._q_act(desc, x, steps, O.SITE_G if asym else O.SITE_A)
    qw = O._q_w(desc, w, sw)
    y = O.student_linear(qa, qw, b)
    assert np.allclose(y, qa["xhat"] @ qw["what"].T + b, rtol=1e-12, atol=1e-12)
    if asym:
        assert qa["beta"] != 0.0 and qa["q"].min() >= 0


# ----------------------------------------------------------------------------- module vs library autograd

def _tiny(n_layers=2, H=16, h=2, Fd=32, B=2, S=5, seed=0, **kw):
    wl = synth.Workload("pin", n_layers, H, h, Fd, S, B, act_dtype="f64", outlier_channels=0)
    params = synth.teacher_params(wl, seed, bias_std=0.1)
    for p in params:                                   # larger weights: every term matters
        for k in O.WEIGHTS:
            p[k] = (p[k] * 10).astype(np.float32)
    x = synth.hidden_states(wl, B, seed)
    desc = O.ModuleDesc(n_layers, H, h, Fd, act_dtype="f64", **kw)
    return wl, desc, params, x


def _to_torch(params, steps):
    tp = [{k: torch.tensor(np.asarray(v, np.float64), requires_grad=True) for k, v in p.items()} for p in params]
    ts = [dict(w={k: torch.tensor(np.asarray(s["w"][k], np.float64), requires_grad=True) for k in O.WEIGHTS},
               a=torch.tensor(np.asarray(s["a"], np.float64), requires_grad=True),
               a_off=torch.tensor(np.asarray(s["a_off"], np.float64), requires_grad=True)) for s in steps]
    return tp, ts


def _cfg(desc):
    return dict(n_heads=desc.n_heads, a_bits=desc.a_bits, w_bits=desc.w_bits, w_grid=desc.w_grid,
                asym_p=desc.asym_p, asym_g=desc.asym_g, ln_eps=desc.ln_eps)


def test_unquantized_module_matches_torch_layers():
    wl, desc, params, x = _tiny(w_bits=0, a_bits=0)
    vl = np.array([5, 3], np.int32)
    outs = O.teacher_forward(desc, params, x, vl)
    tp, _ = _to_torch(params, [])
    ref = R.module(torch.tensor(x, dtype=torch.float64), tp, [None] * len(tp), _cfg(desc), vl, quant=False)
    for a, b in zip(outs, ref):
        assert np.allclose(a, b.detach().numpy(), rtol=1e-10, atol=1e-12)


CASES = [dict(w_bits=4, a_bits=8), dict(w_bits=2, a_bits=8, w_grid=1), dict(w_bits=2, a_bits=8, w_grid=0),
         dict(w_bits=4, a_bits=8, w_per_row=False), dict(w_bits=4, a_bits=8, asym_p=False, asym_g=False),
         dict(w_bits=4, a_bits=4)]


@pytest.mark.parametrize("kw", CASES)
@pytest.mark.parametrize("loss_mean", [True, False])
def test_ste_forward_backward_matches_torch_autograd(kw, loss_mean):
    wl, desc, params, x = _tiny(loss_mean=loss_mean, **kw)
    vl = np.array([4, 5], np.int32)
    teacher = [{k: v.copy() for k, v in p.items()} for p in params]
    student = [{k: (v + synth.normal(7, k + str(i), v.shape, 0.01)).astype(np.float32) for k, v in p.items()}
               for i, p in enumerate(params)]
    rule = 1 if desc.w_bits == 2 else 0
    ws = O.init_weight_steps(desc, student, rule)
    if not desc.w_per_row:
        ws = [{k: v.reshape(1) for k, v in d.items()} for d in ws]
    a, off = O.init_act_steps(desc, student, x, vl)
    a = (a * 0.8).astype(np.float32)                    # shrink: some activations clip, masks matter
    steps = O.make_steps(ws, a, off)
    x_t = x + synth.normal(8, "xt", x.shape, 0.05)
    r = O.forward_loss_backward(desc, teacher, student, steps, x_t, x, vl, lam=0.3)

    tp, ts = _to_torch(student, steps)
    tt, _ = _to_torch(teacher, [])
    xs = torch.tensor(x, dtype=torch.float64)
    xt = torch.tensor(x_t, dtype=torch.float64)
    f_t = R.module(xt, tt, [None] * len(tt), _cfg(desc), vl, quant=False)
    f_s = R.module(0.3 * xt + 0.7 * xs, tp, ts, _cfg(desc), vl, quant=True)
    c = 1.0 / f_s[0].numel() if loss_mean else 1.0
    loss = sum(c * ((a_ - b_.detach()) ** 2).sum() for a_, b_ in zip(f_s, f_t))
    loss.backward()

    for a_, b_ in zip(r["f_s"], f_s):
        assert np.allclose(a_, b_.detach().numpy(), rtol=1e-9, atol=1e-11)
    assert np.isclose(r["loss"], loss.item(), rtol=1e-10)
    clipped = 0
    for l, g in enumerate(r["grads"]):
        for k in O.PARAMS:
            ref = tp[l][k].grad.numpy()
            assert np.allclose(g[k], ref, rtol=1e-7, atol=1e-9 * np.abs(ref).max()), (l, k)
        for k in O.WEIGHTS:
            ref = ts[l]["w"][k].grad.numpy()
            assert np.allclose(g["w"][k], ref, rtol=1e-7, atol=1e-9 * np.abs(ref).max()), (l, "s", k)
        ref = ts[l]["a"].grad.numpy()
        assert np.allclose(g["a"], ref, rtol=1e-7, atol=1e-9 * np.abs(ref).max()), (l, "a")
        if desc.asym_g:
            ref = ts[l]["a_off"].grad.numpy()
            assert np.allclose(g["a_off"][O.SITE_G], ref[O.SITE_G], rtol=1e-7, atol=1e-12), (l, "a_off")
        else:
            assert g["a_off"][O.SITE_G] == 0.0
        clipped += int((np.abs(r["caches"][l]["qx"]["z"]) > r["caches"][l]["qx"]["hi"]).sum())
    assert clipped > 0                                   # the case really exercises the clip masks


def test_bypass_gives_zero_loss_and_zero_grads():
    wl, desc, params, x = _tiny(w_bits=0, a_bits=0)
    steps = O.make_steps([{k: np.ones(1) for k in O.WEIGHTS}] * 2, np.ones((2, 8)), np.zeros((2, 8)))
    r = O.forward_loss_backward(desc, params, params, steps, x, x)
    assert r["loss"] == 0.0
    assert all(np.all(g[k] == 0) for g in r["grads"] for k in O.PARAMS)


def test_high_bit_width_gives_vanishing_error_and_4x_per_bit():
    wl, desc, params, x = _tiny(n_layers=1, H=32, Fd=64, B=4, S=8)
    losses = {}
    for bits in (4, 5, 6, 7, 8, 16):
        d = O.ModuleDesc(1, 32, 2, 64, bits, bits, act_dtype="f64")
        ws = O.init_weight_steps(d, params, 0)
        a, off = O.init_act_steps(d, params, x)
        r = O.forward_loss_backward(d, params, params, O.make_steps(ws, a, off), x, x)
        losses[bits] = r["loss"]
    norm = float((r["f_t"][0] ** 2).mean())
    assert losses[16] < 1e-6 * norm
    vals = [losses[b] for b in (4, 5, 6, 7, 8)]
    assert all(a > b for a, b in zip(vals, vals[1:]))            # monotone in the bit width
    ratios = [a / b for a, b in zip(vals, vals[1:])]
    assert all(2.0 < r_ < 8.0 for r_ in ratios), ratios          # ~4x per bit (uniform-noise model)


# ----------------------------------------------------------------------------- finite differences

def test_unquantized_backward_matches_central_differences():
    wl, desc, params, x = _tiny(n_layers=1, H=8, h=2, Fd=12, B=2, S=3, w_bits=0, a_bits=0)
    teacher = [{k: (v + synth.normal(9, k, v.shape, 0.05)).astype(np.float32) for k, v in params[0].items()}]
    steps = O.make_steps([{k: np.ones(1) for k in O.WEIGHTS}], np.ones((1, 8)), np.zeros((1, 8)))
    student = [{k: v.astype(np.float64) for k, v in params[0].items()}]
    g = O.forward_loss_backward(desc, teacher, student, steps, x, x)["grads"][0]
    for k in O.PARAMS:
        flat = student[0][k].reshape(-1)
        for i in range(0, flat.size, max(1, flat.size // 5)):
            old = flat[i]
            flat[i] = old + 1e-5
            lp = O.forward_loss_backward(desc, teacher, student, steps, x, x)["loss"]
            flat[i] = old - 1e-5
            lm = O.forward_loss_backward(desc, teacher, student, steps, x, x)["loss"]
            flat[i] = old
            fd = (lp - lm) / 2e-5
            assert np.isclose(g[k].reshape(-1)[i], fd, rtol=2e-5, atol=1e-9), (k, i)


def test_single_linear_ste_matches_surrogate_differences():
    # REM special case (Eq. 2): one product.  Hold the rounding residual r = q - z and the clip
    # masks fixed; the surrogate x_hat(x, s) = x + s*r (inside) | s*q (clipped) is smooth, and
    # the STE gradient is its exact gradient.
    x = synth.normal(10, "x", (7, 12), 1.0).astype(np.float64)
    w = synth.normal(10, "w", (5, 12), 0.3).astype(np.float64)
    tgt = synth.normal(10, "t", (7, 5), 1.0).astype(np.float64)
    sa, sw = 0.012, np.full((5, 1), 0.06)
    qa, za = O.quantize_sym(x, sa, 8, "f64")
    qw, _, zw = O.quantize_weight(w, sw, 4, 0, "f64")
    ia, iw = (np.abs(za) <= 127), (np.abs(zw) <= 7)
    ra, rw = qa - za, qw - zw
    assert (~ia).sum() > 0 and (~iw).sum() > 0

    def loss(x_, w_, sa_, sw_):
        xh = np.where(ia, x_ + sa_ * ra, sa_ * qa)
        wh = np.where(iw, w_ + sw_ * rw, sw_ * qw)
        return float(((xh @ wh.T - tgt) ** 2).sum())

    dy = 2 * ((sa * qa) @ (sw * qw).T - tgt)
    dwhat = dy.T @ (sa * qa)
    dxhat = dy @ (sw * qw)
    ins_w, dw_ds = O.weight_ste(zw, qw, 4, 0)
    ins_a, da_ds = O.act_ste(za, qa, -127, 127)
    e = 1e-6
    assert np.isclose((dxhat * da_ds).sum(), (loss(x, w, sa + e, sw) - loss(x, w, sa - e, sw)) / (2 * e), rtol=1e-6)
    for n in range(5):
        d = np.zeros((5, 1)); d[n] = e
        fd = (loss(x, w, sa, sw + d) - loss(x, w, sa, sw - d)) / (2 * e)
        assert np.isclose((dwhat * dw_ds).sum(-1)[n], fd, rtol=1e-6)
    for (i, j) in itertools.product(range(0, 5, 2), range(0, 12, 5)):
        d = np.zeros_like(w); d[i, j] = e
        fd = (loss(x, w + d, sa, sw) - loss(x, w - d, sa, sw)) / (2 * e)
        assert np.isclose((dwhat * ins_w)[i, j], fd, rtol=1e-6, atol=1e-9)


# ----------------------------------------------------------------------------- Eq. 4, AdamW, storage

def test_teacher_forcing_mix_endpoints():
    f = synth.normal(11, "f", (3, 4), 1.0)
    fh = synth.normal(11, "fh", (3, 4), 1.0)
    assert np.array_equal(O.teacher_forcing_mix(f, fh, 1.0), f.astype(np.float64))
    assert np.array_equal(O.teacher_forcing_mix(f, fh, 0.0), fh.astype(np.float64))
    assert O.teacher_forcing_lambda(0, 10) == 1.0 and O.teacher_forcing_lambda(5, 10) == 0.5
    assert O.teacher_forcing_lambda(12, 10) == 0.0


def test_adamw_first_step_closed_form_and_library():
    p0 = synth.normal(12, "p", (50,), 1.0).astype(np.float64)
    g = synth.normal(12, "g", (50,), 0.3).astype(np.float64)
    lr, wd, eps = 1e-2, 0.1, 1e-8
    p1, m, v = O.adamw_update(p0, g, 0 * p0, 0 * p0, 1, lr, 0.9, 0.999, eps, wd)
    assert np.allclose(p1, p0 * (1 - lr * wd) - lr * g / (np.abs(g) + eps), rtol=1e-12)
    tp = torch.tensor(p0.copy(), requires_grad=True)
    opt = torch.optim.AdamW([tp], lr=lr, betas=(0.9, 0.999), eps=eps, weight_decay=wd)
    p, m, v = p0, 0 * p0, 0 * p0
    for t in range(1, 4):
        gt = g * t
        tp.grad = torch.tensor(gt.copy())
        opt.step()
        p, m, v = O.adamw_update(p, gt, m, v, t, lr, 0.9, 0.999, eps, wd)
        assert np.allclose(p, tp.detach().numpy(), rtol=1e-10, atol=1e-12)


def test_bf16_rounding_matches_library_conversion():
    x = np.concatenate([synth.normal(13, "r", (20000,), 3.0),
                        np.array([1.00390625, 1.01171875, -1.00390625, 0.0], np.float32)])
    ref = torch.tensor(x).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(O.round_bf16(x), ref)


def test_recon_step_reduces_loss_on_repeated_batch():
    # qualitative fact of the paper's training-loss curves: the reconstruction loss goes down
    wl = synth.workloads()["tiny"]
    wl = synth.shrink(wl, hidden=32, ffn=64, seq=8, batch=4)
    params = synth.teacher_params(wl, 0)
    x = synth.hidden_states(wl, 4, 0)
    desc = O.ModuleDesc(1, 32, 2, 64, 4, 8, act_dtype="f32")
    student = [{k: v.copy() for k, v in params[0].items()}]
    ws = O.init_weight_steps(desc, student, 0)
    a, off = O.init_act_steps(desc, student, x)
    steps, state, losses = O.make_steps(ws, a, off), {}, []
    for t in range(40):
        losses.append(O.recon_step(desc, params, student, steps, state, x, x, lr=3e-5)["loss"])
    assert np.mean(losses[-5:]) < 0.7 * losses[0]


# ----------------------------------------------------------------------------- Algorithm 1 (modules in parallel from input queues)

def _mremp_setup(n_modules, seed=0):
    wl = synth.shrink(synth.workloads()["tiny"], hidden=32, ffn=64, seq=8, batch=2, n_heads=2)
    descs, teachers, students, steps = [], [], [], []
    x0 = synth.hidden_states(wl, 2, seed)
    for n in range(n_modules):
        desc = O.ModuleDesc(1, 32, 2, 64, 4, 8, act_dtype="f32")
        params = synth.teacher_params(wl, seed + 10 * n)
        student = [{k: v.copy() for k, v in params[0].items()}]
        ws = O.init_weight_steps(desc, student, 0)
        a, off = O.init_act_steps(desc, student, x0)
        descs.append(desc); teachers.append(params); students.append(student); steps.append(O.make_steps(ws, a, off))
    return wl, descs, teachers, students, steps


def test_mremp_single_module_is_the_plain_step_loop():
    wl, descs, teachers, students, steps = _mremp_setup(1)
    batches = [(synth.hidden_states(wl, 2, 100 + t), None) for t in range(4)]
    ref_student = [{k: v.copy() for k, v in students[0][0].items()}]
    ref_steps = O.make_steps([s["w"] for s in steps[0]], np.stack([s["a"] for s in steps[0]]), np.stack([s["a_off"] for s in steps[0]]))
    got = O.mremp_run(descs, teachers, students, steps, batches, draws=np.zeros((4, 1), int), t0=2, T=4, T0=0, lr0=1e-4)
    state, want = {}, []
    for t in range(4):
        want.append(O.recon_step(descs[0], teachers[0], ref_student, ref_steps, state, batches[t][0], batches[t][0], lr=1e-4)["loss"])
    assert got[0] == want
    assert all(np.array_equal(students[0][0][k], ref_student[0][k]) for k in O.PARAMS)


def test_mremp_queue_is_fifo_fill_phase_is_sequential_and_lambda_follows_the_schedule(monkeypatch):
    """Replace the step by a recorder: what each module is fed pins the schedule of Algorithm 1 on its own."""
    calls = []

    def fake_step(desc, teacher, student, steps, state, x_t, x_s, vl, lam, lr=None, **kw):
        n = desc                                    # the 'descs' passed below are just the module indices
        t = state["t"] = state.get("t", -1) + 1
        calls.append((t, n, float(x_t), float(x_s), lam, lr))
        # teacher output = 1000 * (n + 1) + t, student output = its negative: recognisable stamps
        return dict(loss=0.0, f_t=[np.float64(1000 * (n + 1) + t)], f_s=[-np.float64(1000 * (n + 1) + t)])

    monkeypatch.setattr(O, "recon_step", fake_step)
    T, t0, T0, N = 7, 3, 4, 3
    batches = [(np.float64(t), None) for t in range(T)]
    draws = np.array([[0, (t + n) % t0, (2 * t + n) % t0] for t in range(T) for n in (0,)]).reshape(T, 3)
    log = []
    O.mremp_run(list(range(N)), [None] * N, [None] * N, [None] * N, batches, draws, t0, T, T0, lr0=1.0, lr_total=10, log=log)
    for (t, n, x_t, x_s, lam, lr) in calls:
        assert lam == (max(1 - t / T0, 0.0) if t < T0 else 0.0)          # Alg. 2: lambda_t, none after T0
        assert lr == pytest.approx(1.0 - t / 10)                          # linear decay
        if n == 0:
            assert x_t == t and x_s == t                                  # calibration batch of step t
        elif t < t0:
            assert x_t == 1000 * n + t and x_s == -(1000 * n + t)         # filling: predecessor's output of the same step
        else:
            k = draws[t][n]
            assert x_t == 1000 * n + (t - 1 - k) and x_s == -x_t          # k-th most recent entry, same entry on both sides
            assert 0 <= k < t0                                            # never older than t0 steps (first in, first out)
    assert len(calls) == T * N and [c[:2] for c in calls] == [(t, n) for t in range(T) for n in range(N)]


# ----------------------------------------------------------------------------- closed-form ternary weights (TWN rule)

def test_twn_threshold_scale_and_least_squares_property():
    rng = np.random.default_rng(3)
    w = (rng.standard_normal((6, 40)) * 0.05).astype(np.float32)
    w[4] = 0.0                                                  # a dead row: nothing kept, scale 0
    t, alpha, delta = O.quantize_weight_twn(w, per_row=True)
    assert set(np.unique(t)) <= {-1, 0, 1} and not t[4].any() and alpha[4, 0] == 0.0
    for r in range(6):
        a = np.abs(w[r].astype(np.float64))
        d = 0.7 * a.mean()
        assert delta[r, 0] == np.float32(d)
        keep = np.abs(w[r]) > np.float32(d)
        assert np.array_equal(t[r], (np.sign(w[r]) * keep).astype(np.int64))
        if keep.any():
            assert alpha[r, 0] == pytest.approx(a[keep].mean(), rel=1e-6)
            # with the support fixed, the mean of the kept magnitudes is the least-squares scale
            err = lambda al: ((w[r] - al * t[r]) ** 2).sum()
            assert err(alpha[r, 0]) <= min(err(alpha[r, 0] * 1.01), err(alpha[r, 0] * 0.99))
    # one group for the whole matrix
    t1, a1, d1 = O.quantize_weight_twn(w, per_row=False)
    assert a1.shape == (1, 1) and d1[0, 0] == np.float32(0.7 * np.abs(w.astype(np.float64)).mean())


def test_twn_module_matches_torch_autograd_with_plain_straight_through():
    """The module with closed-form ternary weights: forward = the layers on alpha * t, backward = the gradient
    with respect to w_hat passed to w unchanged, no weight-step gradient."""
    wl, desc, params, x = _tiny(w_bits=2, w_twn=True)
    vl = np.array([4, 5], np.int32)
    teacher = [{k: v.copy() for k, v in p.items()} for p in params]
    student = [{k: (v + synth.normal(7, k + str(i), v.shape, 0.01)).astype(np.float32) for k, v in p.items()}
               for i, p in enumerate(params)]
    ws = O.init_weight_steps(desc, student, 1)                     # unused by this quantizer
    a, off = O.init_act_steps(desc, student, x, vl)
    steps = O.make_steps(ws, (a * 0.8).astype(np.float32), off)
    r = O.forward_loss_backward(desc, teacher, student, steps, x, x, vl, lam=0.0)
    tp, ts = _to_torch(student, steps)
    tt, _ = _to_torch(teacher, [])
    xs = torch.tensor(x, dtype=torch.float64)
    cfg = dict(_cfg(desc), w_twn=True, w_per_row=desc.w_per_row)
    f_t = R.module(xs, tt, [None] * len(tt), cfg, vl, quant=False)
    f_s = R.module(xs, tp, ts, cfg, vl, quant=True)
    c = 1.0 / f_s[0].numel()
    loss = sum(c * ((a_ - b_.detach()) ** 2).sum() for a_, b_ in zip(f_s, f_t))
    loss.backward()
    for a_, b_ in zip(r["f_s"], f_s):
        assert np.allclose(a_, b_.detach().numpy(), rtol=1e-9, atol=1e-11)
    assert np.isclose(r["loss"], loss.item(), rtol=1e-10)
    for l, g in enumerate(r["grads"]):
        for k in O.PARAMS:
            ref = tp[l][k].grad.numpy()
            assert np.allclose(g[k], ref, rtol=1e-7, atol=1e-9 * np.abs(ref).max()), (l, k)
        assert all(g["w"][k] is None for k in O.WEIGHTS)
        assert np.allclose(g["a"], ts[l]["a"].grad.numpy(), rtol=1e-7, atol=1e-9 * np.abs(ts[l]["a"].grad.numpy()).max())
    # every row keeps some weights and drops some: the threshold is exercised
    q = r["caches"][0]["qw"]["W1"]["q"]
    assert (q == 0).any() and (q != 0).any()


# ----------------------------------------------------------------------------- refitted scales (alternating rule)

def _sq_err(w, alpha, q):
    return float(((np.asarray(w, np.float64) - alpha * q) ** 2).sum())


def test_laq_keeps_a_grid_point_fixed_and_handles_dead_rows():
    rng = np.random.default_rng(11)
    for bits in (2, 4, 8):
        qmax = 2 ** (bits - 1) - 1
        b0 = rng.integers(-qmax, qmax + 1, (5, 48))
        a0 = np.float32(2.0 ** -5) * np.array([[1], [3], [5], [7], [9]], np.float32)     # scales exact in float32
        w = (a0 * b0).astype(np.float32)
        w[3] = 0.0
        q, alpha, _ = O.quantize_weight_laq(w, bits, alpha0=a0)      # started at the true scale, the rounds stay there
        keep = [0, 1, 2, 4]
        assert np.array_equal(q[keep], b0[keep]) and np.array_equal(alpha[keep, 0], a0[keep, 0].astype(np.float64))
        assert not q[3].any() and alpha[3, 0] == 0.0
        q, alpha, _ = O.quantize_weight_laq(w, bits)                  # default start: dead row all the same
        assert not q[3].any() and alpha[3, 0] == 0.0 and np.all(alpha[keep] > 0)
        # rows of +-c only: three mean|w| lies beyond every weight, the start falls back on max|w| and nothing collapses
        flat = np.where(rng.random((3, 32)) < 0.5, -0.25, 0.25).astype(np.float32)
        q, alpha, _ = O.quantize_weight_laq(flat, bits)
        assert np.allclose(alpha * q, flat.astype(np.float64), rtol=1e-6, atol=0)


def test_laq_half_steps_are_exact_and_the_error_never_rises():
    rng = np.random.default_rng(5)
    w = (rng.standard_normal((7, 200)) * 0.04).astype(np.float32)
    w[:, :3] *= 6.0                                               # a few outliers: the min-max start is far from the fit
    for bits in (2, 4):
        qmax = 2 ** (bits - 1) - 1
        levels = np.arange(-qmax, qmax + 1)
        q, alpha, trace = O.quantize_weight_laq(w, bits)
        assert len(trace) == O.LAQ_ROUNDS and np.array_equal(trace[-1][1], q)
        assert np.array_equal(trace[0][0][:, 0], (np.minimum(3 * np.abs(w.astype(np.float64)).mean(1), np.abs(w.astype(np.float64)).max(1)) / qmax).astype(np.float32))
        for r in range(7):
            prev = None
            for i, (a_r, q_r) in enumerate(trace):
                a_r = a_r[r, 0]
                # projection: every code is the nearest level of alpha_r * Omega(b), by brute force over the levels
                d = np.abs(w[r].astype(np.float64)[:, None] - a_r * levels[None, :])
                best = levels[d.argmin(1)]
                clear = np.sort(d, 1)[:, 1] - np.sort(d, 1)[:, 0] > 1e-9 * a_r      # not a tie
                assert np.array_equal(q_r[r][clear], best[clear])
                # scale: the least-squares solution of q * alpha = w from the library solver
                a_next = trace[i + 1][0][r, 0] if i + 1 < len(trace) else alpha[r, 0]
                ls = np.linalg.lstsq(q_r[r].astype(np.float64)[:, None], w[r].astype(np.float64), rcond=None)[0][0]
                assert a_next == pytest.approx(ls, rel=2e-7)
                e0, e1 = _sq_err(w[r], a_r, q_r[r]), _sq_err(w[r], a_next, q_r[r])
                assert e1 <= e0 * (1 + 1e-6)
                if prev is not None:
                    assert e0 <= prev * (1 + 1e-6)
                prev = e1
            # 15 levels: below the min-max scale, which follows the outliers (with 3 levels either local optimum,
            # the bulk or the outliers, can be the better one)
            mm = np.float32(np.abs(w[r]).max() / qmax)
            assert bits == 2 or _sq_err(w[r], alpha[r, 0], q[r]) < _sq_err(w[r], mm, O.quantize_weight(w[r:r + 1], mm.reshape(1, 1), bits, 0, "f32")[0][0])


def test_laq_against_exhaustive_search_on_tiny_rows():
    """2-bit rows of 5 weights: all 3^5 code vectors with their least-squares scale.  The alternating rule never
    beats the global optimum, never ends above its start, and finds the optimum on most rows."""
    import itertools
    rng = np.random.default_rng(2)
    w = rng.standard_normal((60, 5)).astype(np.float32)
    q, alpha, trace = O.quantize_weight_laq(w, 2)
    hits = 0
    for r in range(60):
        best = np.inf
        for c in itertools.product((-1, 0, 1), repeat=5):
            c = np.array(c, np.float64)
            if c.any():
                a = (c @ w[r].astype(np.float64)) / (c @ c)
                best = min(best, _sq_err(w[r], a, c))
        e = _sq_err(w[r], alpha[r, 0], q[r])
        assert e >= best * (1 - 1e-6) and e <= _sq_err(w[r], trace[0][0][r, 0], trace[0][1][r]) * (1 + 1e-6)
        hits += e <= best * (1 + 1e-5)
    assert hits >= 45, hits


def test_laq_step_on_gaussian_rows_is_the_uniform_quantizer_optimum():
    """The mean-square-optimal uniform quantizer of a unit Gaussian has a step of 0.335 sigma with 16 levels and of
    1.22 sigma with 3 (Max 1960, uniform-quantizer table); the 15-level fit must land just above the first (one level
    fewer), the 3-level fit on the second."""
    rng = np.random.default_rng(9)
    w = rng.standard_normal((4, 1 << 16)).astype(np.float32)
    _, a4, _ = O.quantize_weight_laq(w, 4)
    _, a2, _ = O.quantize_weight_laq(w, 2)
    assert np.all((a4 > 0.335) & (a4 < 0.365)), a4.ravel()
    assert np.all((a2 > 1.20) & (a2 < 1.25)), a2.ravel()
    one, a1, _ = O.quantize_weight_laq(w, 4, per_row=False)
    assert a1.shape == (1, 1) and one.shape == w.shape and 0.335 < a1[0, 0] < 0.365


def test_laq_module_matches_torch_autograd_with_plain_straight_through():
    wl, desc, params, x = _tiny(w_bits=4, w_laq=True)
    vl = np.array([4, 5], np.int32)
    teacher = [{k: v.copy() for k, v in p.items()} for p in params]
    student = [{k: (v + synth.normal(7, k + str(i), v.shape, 0.01)).astype(np.float32) for k, v in p.items()}
               for i, p in enumerate(params)]
    ws = O.init_weight_steps(desc, student, 0)                     # unused by this quantizer
    a, off = O.init_act_steps(desc, student, x, vl)
    steps = O.make_steps(ws, (a * 0.8).astype(np.float32), off)
    r = O.forward_loss_backward(desc, teacher, student, steps, x, x, vl, lam=0.0)
    tp, ts = _to_torch(student, steps)
    tt, _ = _to_torch(teacher, [])
    xs = torch.tensor(x, dtype=torch.float64)
    cfg = dict(_cfg(desc), w_laq=True, w_per_row=desc.w_per_row)
    f_t = R.module(xs, tt, [None] * len(tt), cfg, vl, quant=False)
    f_s = R.module(xs, tp, ts, cfg, vl, quant=True)
    c = 1.0 / f_s[0].numel()
    loss = sum(c * ((a_ - b_.detach()) ** 2).sum() for a_, b_ in zip(f_s, f_t))
    loss.backward()
    for a_, b_ in zip(r["f_s"], f_s):
        assert np.allclose(a_, b_.detach().numpy(), rtol=1e-9, atol=1e-11)
    assert np.isclose(r["loss"], loss.item(), rtol=1e-10)
    for l, g in enumerate(r["grads"]):
        for k in O.PARAMS:
            ref = tp[l][k].grad.numpy()
            assert np.allclose(g[k], ref, rtol=1e-7, atol=1e-9 * np.abs(ref).max()), (l, k)
        assert all(g["w"][k] is None for k in O.WEIGHTS)
    q = r["caches"][0]["qw"]["W1"]["q"]
    assert np.abs(q).max() == 7 and len(np.unique(q)) > 8


# ----------------------------------------------------------------------------- Eq. 2 (one product)

def _rem_case(name, asym_g=True, w_bits=4, w_grid=0, a_bits=8, rows=24, h=32, f=48, seed=3, shrink=0.8):
    rng = np.random.default_rng(seed)
    shape = {"Wqkv": (3 * h, h), "Wo": (h, h), "W1": (f, h), "W2": (h, f)}[name]
    desc = O.ModuleDesc(1, h, 2, f, w_bits, a_bits, w_grid, True, True, asym_g, "f64", True)
    w_t = rng.normal(0, 0.05, shape)
    w_s = w_t + rng.normal(0, 0.004, shape)
    a = rng.normal(0.3 if name == "W2" else 0.0, 1.0, (rows, shape[1]))
    qmax = O.sym_qmax(w_bits)
    ws = {k: np.ones(1, np.float32) for k in O.WEIGHTS}
    ws[name] = (shrink * np.abs(w_s).max(1) / qmax if w_grid == 0 else np.abs(w_s).mean(1)).astype(np.float32)
    a_st = np.ones(O.N_SITES, np.float32)
    a_off = np.zeros(O.N_SITES, np.float32)
    site = O.REM_SITE[name]
    if site == O.SITE_G and asym_g:
        a_off[site] = np.float32(a.min() + 0.2)                       # some values clip at the lower end
        a_st[site] = np.float32(shrink * (a.max() - a_off[site]) / (2 ** a_bits - 1))
    else:
        a_st[site] = np.float32(shrink * np.abs(a).max() / O.sym_qmax(a_bits))
    steps = O.make_steps([ws], [a_st], [a_off])[0]
    return desc, w_t, w_s, steps, a, site


@pytest.mark.parametrize("name,asym_g,w_bits,w_grid,a_bits", [("Wqkv", True, 4, 0, 8), ("Wo", True, 2, 1, 8), ("W1", True, 2, 0, 8),
                                                            ("W2", True, 4, 0, 8), ("W2", False, 4, 0, 4)])
def test_rem_objective_matches_definition_and_torch_autograd(name, asym_g, w_bits, w_grid, a_bits):
    """Eq. 2 for one product: the loss is || w_hat^T a_hat - w^T a ||^2 written out with the quantizers of
    Eq. 1, and every gradient equals library autograd over the detach form of the straight-through estimator."""
    desc, w_t, w_s, steps, a, site = _rem_case(name, asym_g, w_bits, w_grid, a_bits)
    r = O.rem_forward_loss_backward(desc, w_t, w_s, steps, name, a)
    # the definition, written out independently of the oracle's helpers
    s_w = steps["w"][name].astype(np.float64).reshape(-1, 1)
    if w_grid == 0:
        qm = 2 ** (w_bits - 1) - 1
        w_hat = s_w * np.rint(np.clip((w_s.astype(np.float32) / s_w.astype(np.float32)).astype(np.float64), -qm, qm))
    else:
        w_hat = s_w * (np.clip(np.floor((w_s.astype(np.float32) / s_w.astype(np.float32)).astype(np.float64)), -2, 1) + 0.5)
    s_a, beta = float(steps["a"][site]), float(steps["a_off"][site])
    if site == O.SITE_G and asym_g:
        z = ((a.astype(np.float32) - np.float32(beta)) / np.float32(s_a)).astype(np.float64)
        a_hat = s_a * np.rint(np.clip(z, 0, 2 ** a_bits - 1)) + beta
    else:
        qa = 2 ** (a_bits - 1) - 1
        a_hat = s_a * np.rint(np.clip((a.astype(np.float32) / np.float32(s_a)).astype(np.float64), -qa, qa))
    diff = a_hat @ w_hat.T - a @ w_t.T
    assert np.isclose(r["loss"], (diff ** 2).mean(), rtol=1e-10)
    assert np.allclose(r["target"], a @ w_t.T, rtol=1e-12, atol=0)
    # autograd
    tw = torch.tensor(w_s, dtype=torch.float64, requires_grad=True)
    tsw = torch.tensor(steps["w"][name].astype(np.float64), requires_grad=True)
    tsa = torch.tensor(float(steps["a"][site]), dtype=torch.float64, requires_grad=True)
    tb = torch.tensor(float(steps["a_off"][site]), dtype=torch.float64, requires_grad=True)
    ta = torch.tensor(a, dtype=torch.float64)
    ah = R.q_asym(ta, tsa, tb, a_bits) if (site == O.SITE_G and asym_g) else R.q_sym(ta, tsa, a_bits)
    wh = R.q_weight(tw, tsw, w_bits, w_grid)
    loss = ((ah @ wh.T - ta @ torch.tensor(w_t).T) ** 2).mean()
    loss.backward()
    assert np.isclose(r["loss"], loss.item(), rtol=1e-10)
    assert np.allclose(r["dW"], tw.grad.numpy(), rtol=1e-8, atol=1e-14)
    assert np.allclose(r["d_w_step"], tsw.grad.numpy(), rtol=1e-8, atol=1e-14)
    assert np.isclose(r["d_a_step"], tsa.grad.item(), rtol=1e-8, atol=1e-14)
    if site == O.SITE_G and asym_g:
        assert abs(tb.grad.item()) > 0                                # the case really clips
        assert np.isclose(r["d_a_off"], tb.grad.item(), rtol=1e-8, atol=1e-14)


def test_rem_bypass_and_high_bit_width():
    """Without quantizers the two products coincide when the student equals the teacher (loss 0, zero gradients);
    at 16 bits the reconstruction error of Eq. 2 all but vanishes, and it grows as bits are taken away."""
    desc, w_t, _, steps, a, site = _rem_case("W1")
    bypass = O.ModuleDesc(1, desc.hidden, 2, desc.ffn, 0, 0, act_dtype="f64")
    r = O.rem_forward_loss_backward(bypass, w_t, w_t, steps, "W1", a)
    assert r["loss"] == 0.0 and not np.any(r["dW"])
    losses = []
    for bits in (16, 8, 6, 4):
        d = O.ModuleDesc(1, desc.hidden, 2, desc.ffn, bits, bits, act_dtype="f64")
        st = {"w": dict(steps["w"]), "a": steps["a"].copy(), "a_off": steps["a_off"].copy()}
        st["w"]["W1"] = (np.abs(w_t).max(1) / O.sym_qmax(bits)).astype(np.float32)
        st["a"][site] = np.float32(np.abs(a).max() / O.sym_qmax(bits))
        losses.append(O.rem_forward_loss_backward(d, w_t, w_t, st, "W1", a)["loss"])
    assert losses[0] < 1e-8 * float(((a @ w_t.T) ** 2).mean())
    assert losses[0] < losses[1] < losses[2] < losses[3]


def test_rem_step_reduces_the_reconstruction_error():
    """Repeating the step of Eq. 2 on one batch lowers its loss (the objective is what the step descends), and the
    first step moves every weight with a non-zero gradient by lr (AdamW's first step, decay aside)."""
    desc, w_t, w_s, steps, a, site = _rem_case("Wqkv", shrink=0.6)
    state, w = {}, w_s.astype(np.float32)
    r0, w1 = O.rem_step(desc, w_t, w, steps, state, "Wqkv", a, lr=1e-3, weight_decay=0.0)
    moved = np.abs(w1.astype(np.float64) - w.astype(np.float64))
    nz = np.abs(r0["dW"]) > 1e-4                                    # lr / (1 + eps / |g|) with eps = 1e-8
    assert nz.sum() > 100 and np.allclose(moved[nz], 1e-3, rtol=1e-3)
    w = w1
    first = r0["loss"]
    for _ in range(30):
        r, w = O.rem_step(desc, w_t, w, steps, state, "Wqkv", a, lr=2e-4, weight_decay=0.0)
    assert r["loss"] < 0.7 * first


# ----------------------------------------------------------------------------- output logits of the last module

def _head(h, n_classes, seed=11):
    rng = np.random.default_rng(seed)
    return dict(Wp=rng.normal(0, 0.3, (h, h)), bp=rng.normal(0, 0.1, h), Wc=rng.normal(0, 0.3, (n_classes, h)),
                bc=rng.normal(0, 0.1, n_classes))


@pytest.mark.parametrize("loss_mean", [True, False])
def test_logit_loss_matches_torch_head_and_autograd(loss_mean):
    """Pooler (dense + tanh on the first token) and classifier as library layers; the gradient of the logit MSE
    with respect to the student's last layer output from library autograd; zero away from the first token."""
    rng = np.random.default_rng(2)
    B_, S_, H_, C_ = 3, 5, 16, 4
    head = _head(H_, C_)
    f_s, f_t = rng.normal(0, 1, (B_, S_, H_)), rng.normal(0, 1, (B_, S_, H_))
    desc = O.ModuleDesc(1, H_, 2, 32, loss_mean=loss_mean)
    loss, dF, z_s, z_t = O.logit_loss(desc, head, f_s, f_t)
    tp = {k: torch.tensor(v, dtype=torch.float64) for k, v in head.items()}
    ts = torch.tensor(f_s, dtype=torch.float64, requires_grad=True)

    def logits(f):
        return torch.nn.functional.linear(torch.tanh(torch.nn.functional.linear(f[:, 0], tp["Wp"], tp["bp"])), tp["Wc"], tp["bc"])

    zs, zt = logits(ts), logits(torch.tensor(f_t, dtype=torch.float64))
    ref = ((zs - zt) ** 2).mean() if loss_mean else ((zs - zt) ** 2).sum()
    ref.backward()
    assert np.allclose(z_s, zs.detach().numpy(), rtol=1e-12) and np.allclose(z_t, zt.numpy(), rtol=1e-12)
    assert np.isclose(loss, ref.item(), rtol=1e-12)
    assert np.allclose(dF, ts.grad.numpy(), rtol=1e-10, atol=1e-16)
    assert not np.any(dF[:, 1:, :]) and np.any(dF[:, 0, :])
    assert O.logit_loss(desc, head, f_t, f_t)[0] == 0.0             # equal outputs: no logit error


def test_module_with_head_adds_the_logit_term_at_the_last_layer_only():
    """Loss = Eq. 3 + logit term; the extra gradient enters at the last layer's output: against torch autograd of the
    whole quantized module with the head on top."""
    wl = synth.shrink(synth.workloads()["tiny"], n_layers=2, hidden=16, n_heads=2, ffn=32, seq=6, batch=3)
    desc = O.ModuleDesc(2, 16, 2, 32, 4, 8, act_dtype="f64")
    params = synth.teacher_params(wl, 0, bias_std=0.02)
    student = [{k: (v + synth.normal(1, f"n{l}{k}", v.shape, 0.003)).astype(np.float32) for k, v in p.items()} for l, p in enumerate(params)]
    x = synth.hidden_states(wl, wl.batch, 0).astype(np.float64)
    vl = np.array([6, 4, 5])
    ws = O.init_weight_steps(desc, student, 0)
    a, off = O.init_act_steps(desc, student, x, vl)
    steps = O.make_steps(ws, (a * 0.8).astype(np.float32), off)
    head = _head(16, 3)
    base = O.forward_loss_backward(desc, params, student, steps, x, x, vl)
    r = O.forward_loss_backward(desc, params, student, steps, x, x, vl, head=head)
    assert np.isclose(r["loss"], base["loss"] + r["logit_loss"], rtol=1e-12) and r["logit_loss"] > 0
    # autograd over the torch model of the module (detach form of the estimator) with the head on top
    cfg = dict(n_heads=2, a_bits=8, w_bits=4, w_grid=0, asym_p=True, asym_g=True, ln_eps=desc.ln_eps)
    tparams = [{k: torch.tensor(v.astype(np.float64), requires_grad=True) for k, v in p.items()} for p in student]
    tsteps = [dict(w={k: torch.tensor(st["w"][k].astype(np.float64), requires_grad=True) for k in O.WEIGHTS},
                   a=[torch.tensor(float(v), dtype=torch.float64, requires_grad=True) for v in st["a"]],
                   a_off=[torch.tensor(float(v), dtype=torch.float64, requires_grad=True) for v in st["a_off"]]) for st in steps]
    outs = R.module(torch.tensor(x), tparams, tsteps, cfg, vl)
    tp = {k: torch.tensor(v, dtype=torch.float64) for k, v in head.items()}
    logits = lambda f: torch.nn.functional.linear(torch.tanh(torch.nn.functional.linear(f[:, 0], tp["Wp"], tp["bp"])), tp["Wc"], tp["bc"])
    loss = sum(((o - torch.tensor(ft)) ** 2).mean() for o, ft in zip(outs, r["f_t"]))
    loss = loss + ((logits(outs[-1]) - logits(torch.tensor(r["f_t"][-1]))) ** 2).mean()
    loss.backward()
    assert np.isclose(r["loss"], loss.item(), rtol=1e-9)
    for l in range(2):
        for k in O.PARAMS:
            assert np.allclose(r["grads"][l][k], tparams[l][k].grad.numpy(), rtol=1e-6, atol=1e-12), (l, k)
        assert np.allclose(r["grads"][l]["a"], [t.grad.item() if t.grad is not None else 0.0 for t in tsteps[l]["a"]], rtol=1e-6, atol=1e-12)
    assert not np.allclose(r["grads"][0]["W1"], base["grads"][0]["W1"], rtol=1e-6, atol=0)   # the term reaches the layers below


# ----------------------------------------------------------------------------- embedding layers of the first module

def _embed_case(e_bits=4, V=40, H=16, P=12, B_=3, S_=7, seed=4, shrink=0.7):
    rng = np.random.default_rng(seed)
    teacher = dict(word=rng.normal(0, 0.05, (V, H)), pos=rng.normal(0, 0.02, (P, H)), type=rng.normal(0, 0.02, (2, H)),
                   ln_g=1 + rng.normal(0, 0.1, H), ln_b=rng.normal(0, 0.05, H))
    student = {k: (v + rng.normal(0, 0.004, v.shape)).astype(np.float32) for k, v in teacher.items()}
    ids = rng.integers(0, V, (B_, S_))
    ids[0, :3] = 5                                                  # one row gathered several times
    ids[2, 1] = 5
    tt = (np.arange(S_)[None, :] >= np.array([3, 7, 4])[:, None]).astype(np.int64)
    step = (shrink * np.abs(student["word"]).max(1) / O.sym_qmax(e_bits)).astype(np.float32)
    return teacher, student, step, ids, tt


@pytest.mark.parametrize("e_bits,loss_mean", [(4, True), (2, True), (8, False)])
def test_embedding_objective_matches_torch_embedding_layers_and_autograd(e_bits, loss_mean):
    """Gather, sum of the three embeddings, LayerNorm as library layers over the detach form of the quantized
    table; the scatter of repeated rows, the row-step gradients and the position / type / LayerNorm gradients
    from library autograd."""
    teacher, student, step, ids, tt = _embed_case(e_bits)
    desc = O.ModuleDesc(1, 16, 2, 32, loss_mean=loss_mean, act_dtype="f64")
    r = O.embed_loss_backward(desc, teacher, student, step, e_bits, ids, tt)
    F_ = torch.nn.functional
    tp = {k: torch.tensor(np.asarray(v, np.float64), requires_grad=True) for k, v in student.items()}
    ts = torch.tensor(step.astype(np.float64), requires_grad=True)
    tid, ttt = torch.tensor(ids), torch.tensor(tt)
    S_ = ids.shape[1]

    def emb(p, table):
        y = F_.embedding(tid, table) + p["pos"][:S_][None] + F_.embedding(ttt, p["type"])
        return F_.layer_norm(y, (16,), p["ln_g"], p["ln_b"], desc.ln_eps)

    e_s = emb(tp, R.q_weight(tp["word"], ts, e_bits, 0))
    tt_ = {k: torch.tensor(np.asarray(v, np.float64)) for k, v in teacher.items()}
    e_t = emb(tt_, tt_["word"])
    loss = ((e_s - e_t) ** 2).mean() if loss_mean else ((e_s - e_t) ** 2).sum()
    loss.backward()
    assert np.allclose(r["e_t"], e_t.numpy(), rtol=1e-10) and np.allclose(r["e_s"], e_s.detach().numpy(), rtol=1e-10)
    assert np.isclose(r["loss"], loss.item(), rtol=1e-10)
    for k in O.EMBED_PARAMS:
        assert np.allclose(r["grads"][k], tp[k].grad.numpy(), rtol=1e-7, atol=1e-14), k
    assert np.allclose(r["grads"]["word_step"], ts.grad.numpy(), rtol=1e-7, atol=1e-14)
    used = np.zeros(40, bool)
    used[ids.reshape(-1)] = True
    assert not np.any(r["grads"]["word"][~used]) and np.any(r["grads"]["word"][5])


def test_embedding_bypass_is_exact_and_step_reduces_the_loss():
    teacher, student, step, ids, tt = _embed_case(4)
    desc = O.ModuleDesc(1, 16, 2, 32, act_dtype="f64")
    same = {k: np.asarray(v, np.float64) for k, v in teacher.items()}
    assert O.embed_loss_backward(desc, teacher, same, step, 0, ids, tt)["loss"] == 0.0
    state = {}
    first = O.embed_step(desc, teacher, student, step, state, 4, ids, tt, lr=2e-4)["loss"]
    for _ in range(40):
        r = O.embed_step(desc, teacher, student, step, state, 4, ids, tt, lr=2e-4)
    assert r["loss"] < 0.8 * first


def test_embedding_extra_gradient_and_module_input_gradient_match_autograd():
    """First module of the model: the layers' gradient with respect to their input (the student's embedding output)
    is added to the embedding MSE's own gradient.  (i) The module's input gradient equals autograd's d loss / d x of
    the torch model of the module; (ii) an extra gradient g at the embedding output acts like the extra loss
    term <g, e_hat>."""
    wl = synth.shrink(synth.workloads()["tiny"], n_layers=1, hidden=16, n_heads=2, ffn=32, seq=7, batch=3)
    desc = O.ModuleDesc(1, 16, 2, 32, 4, 8, act_dtype="f64")
    params = synth.teacher_params(wl, 0, bias_std=0.02)
    student = [{k: (v + synth.normal(1, f"m{l}{k}", v.shape, 0.003)).astype(np.float32) for k, v in p.items()} for l, p in enumerate(params)]
    x = synth.hidden_states(wl, wl.batch, 0).astype(np.float64)
    ws = O.init_weight_steps(desc, student, 0)
    a, off = O.init_act_steps(desc, student, x, None)
    steps = O.make_steps(ws, (a * 0.8).astype(np.float32), off)
    r = O.forward_loss_backward(desc, params, student, steps, x, x)
    cfg = dict(n_heads=2, a_bits=8, w_bits=4, w_grid=0, asym_p=True, asym_g=True, ln_eps=desc.ln_eps)
    tx = torch.tensor(x, requires_grad=True)
    tparams = [{k: torch.tensor(v.astype(np.float64)) for k, v in p.items()} for p in student]
    tsteps = [dict(w={k: torch.tensor(st["w"][k].astype(np.float64)) for k in O.WEIGHTS},
                   a=[torch.tensor(float(v), dtype=torch.float64) for v in st["a"]],
                   a_off=[torch.tensor(float(v), dtype=torch.float64) for v in st["a_off"]]) for st in steps]
    outs = R.module(tx, tparams, tsteps, cfg, None)
    sum(((o - torch.tensor(ft)) ** 2).mean() for o, ft in zip(outs, r["f_t"])).backward()
    assert np.allclose(r["d_input"], tx.grad.numpy(), rtol=1e-7, atol=1e-13) and np.any(r["d_input"])
    # (ii)
    teacher, est, step, ids, tt = _embed_case(4, H=16, B_=3, S_=7)
    extra = r["d_input"] * 50
    re = O.embed_loss_backward(desc, teacher, est, step, 4, ids, tt, d_extra=extra)
    F_ = torch.nn.functional
    tp = {k: torch.tensor(np.asarray(v, np.float64), requires_grad=True) for k, v in est.items()}
    ts = torch.tensor(step.astype(np.float64), requires_grad=True)
    y = F_.embedding(torch.tensor(ids), R.q_weight(tp["word"], ts, 4, 0)) + tp["pos"][:7][None] + F_.embedding(torch.tensor(tt), tp["type"])
    e_s = F_.layer_norm(y, (16,), tp["ln_g"], tp["ln_b"], desc.ln_eps)
    (((e_s - torch.tensor(re["e_t"])) ** 2).mean() + (torch.tensor(extra) * e_s).sum()).backward()
    for k in O.EMBED_PARAMS:
        assert np.allclose(re["grads"][k], tp[k].grad.numpy(), rtol=1e-7, atol=1e-13), k
    assert np.allclose(re["grads"]["word_step"], ts.grad.numpy(), rtol=1e-7, atol=1e-13)
