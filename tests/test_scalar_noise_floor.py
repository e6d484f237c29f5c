"""How far apart are two CORRECT implementations on the gradients that the GPU tests hold to more than 2e-2?

The activation step gradients are scalars: sums over a whole tensor of terms of both signs, so the rounding of the
stored activations (bf16) can move them by far more than it moves a weight gradient.  The GPU tests bound some of
them at 3e-2 or 0.1 (of max(|reference|, 2 % of the layer's largest)).  Here the same cases run twice through the
CPU oracle: as it stands, and with every stored tensor computed to about tensor-core accumulation accuracy before
it is rounded (a relative perturbation of 3e-6 in front of each storage rounding: the bf16 products of the CUDA
path carry 1.3e-6 to 5.5e-6 relative error against float64).  The perturbed run is a second correct implementation;
its distance from the first is the noise floor.  A bound used on the GPU that is wider than the stated 2e-2 must not be
more than twice that floor (so that it admits no error a correct implementation could not show as well).  No GPU needed."""
import numpy as np
import pytest

from oracle import mrem_oracle as O
from paper_2109_15082_b200 import synth
from tests import test_gpu_module as G

EPS = 3e-6


def _problem(wl, seed=0, student_noise=0.0, step_shrink=1.0, a_bits=None):
    """The oracle half of tests.gpu_util.Problem, from the same generators."""
    twn = wl.w_grid in (2, 3)
    desc = O.ModuleDesc(wl.n_layers, wl.hidden, wl.n_heads, wl.ffn, wl.w_bits, a_bits or wl.a_bits, 0 if twn else wl.w_grid, True,
                        True, True, wl.act_dtype, True, w_twn=wl.w_grid == 2, w_laq=wl.w_grid == 3)
    narrow = (lambda v: O.round_bf16(v).astype(np.float32)) if wl.act_dtype == "bf16" else (lambda v: v)
    teacher = [{k: (narrow(v) if k in O.WEIGHTS else v) for k, v in p.items()} for p in synth.teacher_params(wl, seed, bias_std=0.02)]
    student = [{k: (v + (synth.normal(seed + 1, f"noise{l}{k}", v.shape, student_noise) if student_noise > 0 else 0)).astype(np.float32)
                for k, v in p.items()} for l, p in enumerate(teacher)]
    x = narrow(synth.hidden_states(wl, wl.batch, seed))
    vl = synth.valid_lengths(wl, wl.batch, seed)
    ws = O.init_weight_steps(desc, student, wl.w_step_rule)
    a, off = O.init_act_steps(desc, student, x, vl)
    a = (a * step_shrink).astype(np.float32)
    ws = [{k: (v * (step_shrink if wl.w_step_rule == 0 else 1.0)).astype(np.float32) for k, v in d.items()} for d in ws]
    return desc, teacher, student, O.make_steps(ws, a, off), x, vl


def _scalar_noise(wl, monkeypatch, **kw):
    desc, teacher, student, steps, x, vl = _problem(wl, **kw)
    base = O.forward_loss_backward(desc, teacher, student, steps, x, x, vl)
    plain_store = O.store
    worst = 0.0
    for trial in range(3):
        rng = np.random.default_rng(100 + trial)
        monkeypatch.setattr(O, "store", lambda v, dt: plain_store(np.asarray(v, np.float64) * (1.0 + EPS * rng.standard_normal(np.shape(v))), dt))
        other = O.forward_loss_backward(desc, teacher, student, steps, x, x, vl)
        monkeypatch.setattr(O, "store", plain_store)
        for g, r in zip(other["grads"], base["grads"]):
            floor = 0.02 * np.abs(r["a"]).max()
            for s in range(8):
                worst = max(worst, abs(g["a"][s] - r["a"][s]) / max(abs(r["a"][s]), floor))
    return worst


@pytest.mark.parametrize("case", [k for k, v in G.CLOSED_FORM.items() if v[5] is not None])
def test_bound_on_step_gradients_with_refitted_scales_is_within_the_noise_floor(case, monkeypatch):
    """Measured here (worst of 3 perturbation seeds x 2 layers x 8 sites): 0.29 to 2.5 for the closed-form cases, most
    of it in layer 1, whose input already differs.  The GPU tests bound these scalars at 0.1; the CUDA path is closer to
    the oracle than this second CPU implementation is, so that bound does not hide an error larger than the distance
    between two correct implementations."""
    base, kw, _, _, _, scalar_tol = G.CLOSED_FORM[case]
    noise = _scalar_noise(G._wl(base, **kw), monkeypatch, student_noise=0.002)
    print(case, "noise floor of the activation step gradients", round(noise, 4), "bound used on the GPU", scalar_tol)
    assert noise >= scalar_tol / 2


def test_step_gradients_of_the_plain_cases_have_a_floor_near_the_stated_tolerance(monkeypatch):
    """The cases held to 2e-2 scalar by scalar: the same experiment gives 0.03 to 0.04, i.e. the stated tolerance is
    already at the floor for these sums and the CUDA path meets it."""
    for name in ("bf16_small", "bf16_tiles"):
        wl, kw = G.CASES[name]
        noise = _scalar_noise(wl, monkeypatch, student_noise=kw.get("student_noise", 0.0), step_shrink=kw.get("step_shrink", 1.0))
        print(name, "noise floor", round(noise, 4))
        assert 5e-3 < noise < 0.2
