"""CPU oracle for the MREM reconstruction step (test infrastructure, not a product path).

A plain, slow numpy implementation of what one reconstruction step computes:
the quantizers of Eq. 1 (Sec. 3.1), a full-precision teacher module and its
fake-quantized student (Sec. 3.1, Sec. 4.1), the module-wise reconstruction loss
of Eq. 3, the teacher-forcing mix of Eq. 4, the straight-through backward
(Sec. 3.1.1) and the AdamW update named after Algorithm 2.  Float sums are
carried in float64; integer-code products are exact.  Only tests, the smoke
check and the benchmark's CPU-baseline leg may import this file; it shares no
code with the CUDA path and imports nothing from it.

Every function is pinned by tests/test_oracle_*.py against something other
than itself (library autograd, brute force, closed forms, invariants of Eq. 1;
the storage roundings, the initial activation steps and a whole step's
bookkeeping in tests/test_oracle_storage_pins.py against torch layers with the
roundings written out and torch.optim.AdamW).
The only part that stays "parity unpinned" by the paper is the multi-step loss
trajectory, for which the paper prints no numbers (only the qualitative trend
of its training-loss figure).

Storage emulation.  The CUDA path keeps activations in float32 or bfloat16.
`desc.act_dtype` ('f32' | 'bf16' | 'f64') makes the oracle round to that type at
exactly the tensors that path stores, and take every quantizer decision
(x / s, clip, round) in float32 arithmetic on the stored value, so that integer
codes are comparable bit for bit.  'f64' rounds nowhere (used by the pins).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
from scipy.special import erf as _erf

# quantizer sites inside one Transformer layer (activations), in forward order
SITE_X, SITE_Q, SITE_K, SITE_V, SITE_P, SITE_C, SITE_A, SITE_G = range(8)
N_SITES = 8
WEIGHTS = ("Wqkv", "Wo", "W1", "W2")
PARAMS = ("Wqkv", "bqkv", "Wo", "bo", "ln1_g", "ln1_b", "W1", "b1", "W2", "b2", "ln2_g", "ln2_b")


@dataclass
class ModuleDesc:
    n_layers: int
    hidden: int
    n_heads: int
    ffn: int
    w_bits: int = 4            # 0 = weights not quantized (bypass)
    a_bits: int = 8            # 0 = activations not quantized (bypass)
    w_grid: int = 0            # 0: Omega(b) of Eq. 1; 1: half-integer 2-bit grid {-1.5,-.5,.5,1.5}*s
    w_per_row: bool = True     # one step per output row, else one per matrix
    asym_p: bool = True        # softmax output quantized asymmetrically (unsigned codes, offset 0)
    asym_g: bool = True        # GELU output quantized asymmetrically (unsigned codes, learnable offset)
    act_dtype: str = "f64"
    loss_mean: bool = True     # True: mean over B*S*H per layer; False: the plain sum of Eq. 3
    ln_eps: float = 1e-12
    w_twn: bool = False        # 2-bit weights by the closed-form ternary rule (threshold 0.7 mean|w|, scale = mean
                               # of the kept |w|, per output row) instead of a learnable step
    w_laq: bool = False        # b-bit weights with the scale refitted by alternating least squares (quantize_weight_laq)


# ----------------------------------------------------------------------------- storage

def round_bf16(x):
    """Round float values to bfloat16 (nearest, ties to even) via float32; returns float64."""
    x32 = np.ascontiguousarray(np.asarray(x, dtype=np.float32))
    u = x32.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = ((u + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)).astype(np.uint32)
    return r.view(np.float32).astype(np.float64).reshape(np.shape(x))


def store(x, act_dtype):
    """Value of x after being written to a tensor of the given storage type."""
    if act_dtype == "f64":
        return np.asarray(x, dtype=np.float64)
    if act_dtype == "f32":
        return np.asarray(x, dtype=np.float64).astype(np.float32).astype(np.float64)
    if act_dtype == "bf16":
        return round_bf16(x)
    raise ValueError(act_dtype)


def _div(x, s, act_dtype):
    """x / s in the precision the quantizer decision is taken in (float32 unless 'f64')."""
    if act_dtype == "f64":
        return np.asarray(x, np.float64) / np.asarray(s, np.float64)
    return (np.asarray(x, np.float32) / np.asarray(s, np.float32)).astype(np.float32)


def _sub(x, b, act_dtype):
    if act_dtype == "f64":
        return np.asarray(x, np.float64) - np.asarray(b, np.float64)
    return (np.asarray(x, np.float32) - np.asarray(b, np.float32)).astype(np.float32)


# ----------------------------------------------------------------------------- quantizers (Eq. 1)

def sym_qmax(bits):
    """Largest code of Omega(b) = {-2^(b-1)+1, ..., 2^(b-1)-1} (Eq. 1)."""
    return 2 ** (bits - 1) - 1


def quantize_sym(x, s, bits, act_dtype="f32"):
    """Symmetric uniform quantizer of Eq. 1: q = Pi_Omega(b)(x / s), x_hat = s * q.

    The projection takes x / s to its closest integer (ties to even) inside
    Omega(b); clipping first and rounding second gives the same integer.
    Returns (q int64, z) with z = x / s as computed for the decision.
    """
    qmax = sym_qmax(bits)
    z = _div(x, s, act_dtype)
    q = np.rint(np.clip(z, -qmax, qmax)).astype(np.int64)
    return q, z


def quantize_asym(x, s, beta, bits, act_dtype="f32"):
    """Asymmetric quantizer for mostly-positive activations (Sec. 3.1): unsigned
    codes q = clip(rne((x - beta) / s), 0, 2^b - 1), x_hat = s * q + beta."""
    qmax = 2 ** bits - 1
    z = _div(_sub(x, beta, act_dtype), s, act_dtype)
    q = np.rint(np.clip(z, 0, qmax)).astype(np.int64)
    return q, z


def quantize_weight(w, s, bits, grid, act_dtype="f32"):
    """Weight quantizer.  s has one entry per output row ([N,1]) or one in all ([1,1]).

    grid 0: Eq. 1, codes in Omega(b), w_hat = s * q.
    grid 1: symmetric 2-bit levels {-1.5,-0.5,0.5,1.5} * s, carried as odd integer
            codes c = 2*clip(floor(w/s), -2, 1) + 1 in {-3,-1,1,3} with w_hat = (s/2) * c.
    Returns (codes int64, scale float64 with w_hat = scale * codes, z).
    """
    z = _div(w, s, act_dtype)
    s64 = np.asarray(s, np.float64)
    if grid == 0:
        qmax = sym_qmax(bits)
        q = np.rint(np.clip(z, -qmax, qmax)).astype(np.int64)
        return q, s64, z
    assert bits == 2
    c = 2 * np.clip(np.floor(z), -2, 1).astype(np.int64) + 1
    return c, s64 * 0.5, z


def quantize_weight_twn(w, per_row=True):
    """Ternary weights with closed-form threshold and scale (the TWN rule the paper names for 2-bit weights,
    Sec. 5.1): per group (output row or whole matrix) delta = 0.7 * mean|w|, t = sign(w) * 1[|w| > delta],
    alpha = mean of |w| over the kept entries (0 when none is kept); w_hat = alpha * t.  The means are taken in
    float64 and the comparison |w| > delta in float32 on float32(delta), the precision in which the kernel
    decides.  Returns (codes int64 in {-1, 0, 1}, alpha float64 [groups, 1], delta float32 [groups, 1])."""
    w32 = np.asarray(w, np.float32)
    a = np.abs(w32.astype(np.float64))
    g = a if per_row else a.reshape(1, -1)
    delta = (0.7 * g.mean(-1, keepdims=True)).astype(np.float32)
    keep = np.abs(w32 if per_row else w32.reshape(1, -1)) > delta
    cnt = keep.sum(-1, keepdims=True)
    alpha = (g * keep).sum(-1, keepdims=True) / np.maximum(cnt, 1)
    alpha = alpha.astype(np.float32).astype(np.float64)
    t = (np.sign(w32 if per_row else w32.reshape(1, -1)) * keep).astype(np.int64).reshape(w32.shape)
    return t, alpha, delta


LAQ_ROUNDS = 16


def quantize_weight_laq(w, bits, per_row=True, rounds=LAQ_ROUNDS, alpha0=None):
    """b-bit weights whose scale is refitted from the weights instead of learnt (the loss-aware quantizer the paper
    names for 4-bit weights, Sec. 5.1, read with unit curvature weights): per group (output row or whole matrix)
    minimise ||w - alpha q||^2 over alpha and q in Omega(b)^n by alternating the two exact half-steps,
        q     = Pi_Omega(b)(w / alpha)        (alpha fixed: Eq. 1, element by element)
        alpha = <q, w> / <q, q>               (q fixed: least squares)
    `rounds` times from alpha_0 = min(3 mean|w|, max|w|) / qmax (a clipping range of 3 mean|w|, about 2.4 standard
    deviations of a Gaussian row, which does not follow single outliers the way max|w| does; never beyond max|w|, so
    that the largest weight always gets a non-zero code and no later scale can exceed max|w|; `alpha0` overrides it);
    w_hat = alpha_rounds * q_rounds.
    A group of zeros keeps alpha = 0 and codes 0.  Every alpha is rounded to float32 (the type the scale is stored
    in) and the division w / alpha is the float32 one of Eq. 1; the mean and the two inner products are accumulated
    in float64.
    Returns (codes int64, alpha float64 [groups, 1], trace): trace[r] = (alpha_r, q_{r+1}) per round, for tests."""
    w32 = np.asarray(w, np.float32)
    g = w32 if per_row else w32.reshape(1, -1)
    g64 = g.astype(np.float64)
    qmax = sym_qmax(bits)
    if alpha0 is None:
        a = np.abs(g64)
        alpha = (np.minimum(3.0 * a.mean(-1, keepdims=True), a.max(-1, keepdims=True)) / qmax).astype(np.float32)
    else:
        alpha = np.asarray(alpha0, np.float32).reshape(-1, 1)
    q = np.zeros(g.shape, np.int64)
    trace = []
    for _ in range(rounds):
        live = alpha[:, 0] > 0
        q = np.zeros(g.shape, np.int64)
        if live.any():
            q[live] = quantize_weight(g[live], alpha[live], bits, 0, "f32")[0]
        trace.append((alpha.astype(np.float64), q.copy()))
        qq = (q * q).sum(-1, keepdims=True)
        qw = (q * g64).sum(-1, keepdims=True)
        alpha = np.where(qq > 0, qw / np.maximum(qq, 1), 0.0).astype(np.float32)
    return q.reshape(w32.shape), alpha.astype(np.float64), trace


def weight_ste(z, codes, bits, grid):
    """Straight-through factors of the weight quantizer at z = w / s.

    Returns (inside, dwhat_ds): inside = 1 where the gradient passes to w (z within
    the representable range, bounds inclusive for grid 0, [-2, 2) for grid 1) and
    d w_hat / d s = level - z inside, = the clipped level outside."""
    z = np.asarray(z, np.float64)
    if grid == 0:
        qmax = sym_qmax(bits)
        inside = ((z >= -qmax) & (z <= qmax)).astype(np.float64)
        level = codes.astype(np.float64)
    else:
        inside = ((z >= -2) & (z < 2)).astype(np.float64)
        level = codes.astype(np.float64) * 0.5
    return inside, level - z * inside


def act_ste(z, q, lo, hi):
    """Straight-through factors of an activation quantizer with code range [lo, hi]."""
    z = np.asarray(z, np.float64)
    inside = ((z >= lo) & (z <= hi)).astype(np.float64)
    return inside, q.astype(np.float64) - z * inside


def int_matmul(qa, qw):
    """acc[m, n] = sum_k qa[m, k] * qw[n, k], exact.

    The float64 matrix product of integer-valued operands is exact while every
    partial sum stays below 2^53 (asserted), so the library routine is the plain
    definition here."""
    qa = np.asarray(qa)
    qw = np.asarray(qw)
    k = qa.shape[-1]
    bound = float(np.abs(qa).max(initial=0)) * float(np.abs(qw).max(initial=0)) * k
    assert bound < 2.0 ** 53
    acc = qa.astype(np.float64) @ np.swapaxes(qw.astype(np.float64), -1, -2)
    return np.rint(acc).astype(np.int64)


# ----------------------------------------------------------------------------- layer ops

def gelu(u):
    """erf form of GELU."""
    u = np.asarray(u, np.float64)
    return 0.5 * u * (1.0 + _erf(u / np.sqrt(2.0)))


def gelu_grad(u):
    u = np.asarray(u, np.float64)
    return 0.5 * (1.0 + _erf(u / np.sqrt(2.0))) + u * np.exp(-0.5 * u * u) / np.sqrt(2.0 * np.pi)


def layernorm(y, g, b, eps):
    """Returns (out, xn, rstd) with xn the normalised input."""
    y = np.asarray(y, np.float64)
    mu = y.mean(-1, keepdims=True)
    var = ((y - mu) ** 2).mean(-1, keepdims=True)
    rstd = 1.0 / np.sqrt(var + eps)
    xn = (y - mu) * rstd
    return xn * g + b, xn, rstd


def layernorm_backward(dout, xn, rstd, g):
    dg = (dout * xn).reshape(-1, xn.shape[-1]).sum(0)
    db = dout.reshape(-1, xn.shape[-1]).sum(0)
    dxn = dout * g
    dy = rstd * (dxn - dxn.mean(-1, keepdims=True) - xn * (dxn * xn).mean(-1, keepdims=True))
    return dy, dg, db


def key_mask(valid_len, batch, seq):
    """[batch, 1, 1, seq] boolean, True where the key position is padding."""
    if valid_len is None:
        return np.zeros((batch, 1, 1, seq), bool)
    return (np.arange(seq)[None, :] >= np.asarray(valid_len)[:, None])[:, None, None, :]


def softmax_masked(scores, pad):
    """Softmax over the last axis; padded keys get probability exactly 0."""
    s = np.where(pad, -np.inf, scores)
    s = s - s.max(-1, keepdims=True)
    e = np.exp(s)
    return e / e.sum(-1, keepdims=True)


def _heads(x, h):
    b, s, hd = x.shape
    return x.reshape(b, s, h, hd // h).transpose(0, 2, 1, 3)      # [B,h,S,d]


def _merge(x):
    b, h, s, d = x.shape
    return x.transpose(0, 2, 1, 3).reshape(b, s, h * d)


# ----------------------------------------------------------------------------- teacher (Alg. 2: full-precision module output)

def teacher_layer(desc, p, x, valid_len):
    """One post-LayerNorm BERT encoder layer in full precision; x is [B,S,H] as stored."""
    st = lambda t: store(t, desc.act_dtype)
    B, S, H = x.shape
    h, d = desc.n_heads, H // desc.n_heads
    W = {k: st(p[k]) for k in WEIGHTS}                  # teacher matrices live in the storage type
    qkv = st(x @ W["Wqkv"].T + p["bqkv"])
    q, k, v = (_heads(t, h) for t in np.split(qkv, 3, axis=-1))
    P = st(softmax_masked(q @ k.transpose(0, 1, 3, 2) / np.sqrt(d), key_mask(valid_len, B, S)))
    ctx = st(_merge(P @ v))
    y1 = st(ctx @ W["Wo"].T + p["bo"] + x)
    a = st(layernorm(y1, p["ln1_g"], p["ln1_b"], desc.ln_eps)[0])
    g = st(gelu(a @ W["W1"].T + p["b1"]))            # the pre-GELU tensor is never stored here
    y2 = st(g @ W["W2"].T + p["b2"] + a)
    return st(layernorm(y2, p["ln2_g"], p["ln2_b"], desc.ln_eps)[0])


def teacher_forward(desc, params, x, valid_len=None):
    """Outputs f_l of every layer of the module, list of [B,S,H]."""
    outs, cur = [], store(x, desc.act_dtype)
    for p in params:
        cur = teacher_layer(desc, p, cur, valid_len)
        outs.append(cur)
    return outs


# ----------------------------------------------------------------------------- student (Alg. 2: quantized module output)

def _q_act(desc, x, steps, site):
    """Quantize activation `x` (stored values) at `site`.  Returns dict with
    x_hat, codes q, z, range (lo, hi), step s and offset beta."""
    if desc.a_bits == 0:
        return dict(xhat=np.asarray(x, np.float64), q=None)
    s = float(steps["a"][site])
    asym = (site == SITE_P and desc.asym_p) or (site == SITE_G and desc.asym_g)
    if asym:
        beta = float(steps["a_off"][site]) if site == SITE_G else 0.0
        q, z = quantize_asym(x, s, beta, desc.a_bits, desc.act_dtype)
        lo, hi = 0, 2 ** desc.a_bits - 1
    else:
        beta = 0.0
        q, z = quantize_sym(x, s, desc.a_bits, desc.act_dtype)
        hi = sym_qmax(desc.a_bits)
        lo = -hi
    return dict(xhat=s * q + beta, q=q, z=z, lo=lo, hi=hi, s=s, beta=beta, asym=asym)


def _q_w(desc, w, s_w):
    if desc.w_bits == 0:
        return dict(what=np.asarray(w, np.float64), q=None)
    if desc.w_twn:
        q, alpha, _ = quantize_weight_twn(w, desc.w_per_row)
        return dict(what=alpha * q, q=q, z=None, scale=alpha, closed=True)
    if desc.w_laq:
        q, alpha, _ = quantize_weight_laq(w, desc.w_bits, desc.w_per_row)
        alpha_e = alpha if desc.w_per_row else alpha.reshape(1, 1)
        return dict(what=alpha_e * q, q=q, z=None, scale=alpha, closed=True)
    s = np.asarray(s_w, np.float32).reshape(-1, 1)
    q, scale, z = quantize_weight(w, s, desc.w_bits, desc.w_grid, desc.act_dtype)
    return dict(what=scale * q, q=q, z=z, scale=scale)


def student_linear(qa, qw, bias):
    """y = w_hat^T a_hat + bias (the quantized product of Eq. 2).  With integer
    codes on both sides: acc = sum_k qa*qw exactly, then
    y = s_a * scale_w[n] * acc + beta_a * scale_w[n] * sum_k qw[n,k] + bias[n]."""
    if qa["q"] is None or qw["q"] is None:
        return qa["xhat"] @ qw["what"].T + bias
    lead = qa["q"].shape[:-1]
    acc = int_matmul(qa["q"].reshape(-1, qa["q"].shape[-1]), qw["q"]).reshape(*lead, -1)
    scale_n = qw["scale"].reshape(-1) * np.ones(qw["q"].shape[0])
    y = qa["s"] * scale_n * acc + bias
    if qa["beta"] != 0.0:
        y = y + qa["beta"] * scale_n * qw["q"].sum(-1)
    return y


def student_layer(desc, p, steps, x, valid_len):
    """Fake-quantized layer: a quantizer on both operands of every matrix product
    (Sec. 3.1); LayerNorm, skip connections and biases are not quantized.
    Returns (layer output f_hat_l, cache for the backward)."""
    st = lambda t: store(t, desc.act_dtype)
    B, S, H = x.shape
    h, d = desc.n_heads, H // desc.n_heads
    c = dict(x=x, B=B, S=S)
    c["pad"] = key_mask(valid_len, B, S)
    qw = {k: _q_w(desc, p[k], steps["w"][k]) for k in WEIGHTS}
    c["qw"] = qw

    c["qx"] = _q_act(desc, x, steps, SITE_X)
    c["qkv"] = st(student_linear(c["qx"], qw["Wqkv"], p["bqkv"]))
    Q, K, V = np.split(c["qkv"], 3, axis=-1)
    c["qQ"], c["qK"], c["qV"] = (_q_act(desc, t, steps, s) for t, s in
                                 ((Q, SITE_Q), (K, SITE_K), (V, SITE_V)))
    Qh, Kh, Vh = (_heads(c[n]["xhat"], h) for n in ("qQ", "qK", "qV"))
    c["P"] = st(softmax_masked(Qh @ Kh.transpose(0, 1, 3, 2) / np.sqrt(d), c["pad"]))
    c["qP"] = _q_act(desc, c["P"], steps, SITE_P)
    c["ctx"] = st(_merge(c["qP"]["xhat"] @ Vh))
    c["qC"] = _q_act(desc, c["ctx"], steps, SITE_C)
    c["y1"] = st(student_linear(c["qC"], qw["Wo"], p["bo"]) + x)
    a, c["xn1"], c["rstd1"] = layernorm(c["y1"], p["ln1_g"], p["ln1_b"], desc.ln_eps)
    c["a"] = st(a)
    c["qA"] = _q_act(desc, c["a"], steps, SITE_A)
    c["u"] = st(student_linear(c["qA"], qw["W1"], p["b1"]))
    c["g"] = st(gelu(c["u"]))
    c["qG"] = _q_act(desc, c["g"], steps, SITE_G)
    c["y2"] = st(student_linear(c["qG"], qw["W2"], p["b2"]) + c["a"])
    f, c["xn2"], c["rstd2"] = layernorm(c["y2"], p["ln2_g"], p["ln2_b"], desc.ln_eps)
    c["f"] = st(f)
    return c["f"], c


def teacher_forcing_mix(f_teacher, f_student, lam, act_dtype="f64"):
    """Eq. 4: lam * f + (1 - lam) * f_hat, the student module's input under teacher forcing."""
    return store(lam * np.asarray(f_teacher, np.float64) + (1.0 - lam) * np.asarray(f_student, np.float64),
                 act_dtype)


def teacher_forcing_lambda(t, t0):
    """lambda_t = max(1 - t / T0, 0) (Sec. 4.2.1)."""
    return max(1.0 - t / t0, 0.0) if t0 > 0 else 0.0


def student_forward(desc, params, steps, x, valid_len=None, x_teacher=None, lam=0.0):
    """Outputs f_hat_l of every layer plus the caches.  With lam > 0 the module input
    is the Eq. 4 mix of the teacher-side input `x_teacher` and the student-side `x`."""
    cur = store(x, desc.act_dtype)
    if lam != 0.0 and x_teacher is not None:
        cur = teacher_forcing_mix(store(x_teacher, desc.act_dtype), cur, lam, desc.act_dtype)
    outs, caches = [], []
    for p, s in zip(params, steps):
        cur, c = student_layer(desc, p, s, cur, valid_len)
        outs.append(cur)
        caches.append(c)
    return outs, caches


# ----------------------------------------------------------------------------- loss (Eq. 3)

def recon_loss(desc, f_student, f_teacher):
    """l = sum over the module's layers of c * ||f_hat_l - f_l||^2, c = 1/(B*S*H) when
    `loss_mean` (the MSE reading) or 1 (Eq. 3 as printed).  Returns (total, per layer,
    list of d l / d f_hat_l)."""
    per, grads = [], []
    for fs, ft in zip(f_student, f_teacher):
        diff = np.asarray(fs, np.float64) - np.asarray(ft, np.float64)
        c = 1.0 / diff.size if desc.loss_mean else 1.0
        per.append(c * float((diff * diff).sum()))
        grads.append(2.0 * c * diff)
    return float(sum(per)), per, grads


# ----------------------------------------------------------------------------- backward (straight-through estimator, Sec. 3.1.1)

def _act_back(desc, qa, dxhat, g, site):
    """Gradient through one activation quantizer: passes dxhat where x/s lies inside
    the code range, and accumulates d l / d s (and d l / d beta for asymmetric sites)."""
    if qa["q"] is None:
        return dxhat
    inside, dxhat_ds = act_ste(qa["z"], qa["q"], qa["lo"], qa["hi"])
    g["a"][site] += float((dxhat * dxhat_ds).sum())
    if qa["asym"] and site == SITE_G:
        g["a_off"][site] += float((dxhat * (1.0 - inside)).sum())
    return dxhat * inside


def _linear_back(desc, qa, qw, dy, name, g, site):
    """Backward of y = a_hat w_hat^T + bias: returns d l / d a (after the STE of the
    input quantizer) and fills the gradients of the latent weight, its step and the bias."""
    K = qa["xhat"].shape[-1]
    dy2 = dy.reshape(-1, dy.shape[-1])
    dwhat = dy2.T @ qa["xhat"].reshape(-1, K)
    g["b" + name[1:] if name != "Wqkv" else "bqkv"] = dy2.sum(0)
    if qw["q"] is None or qw.get("closed"):
        g[name] = dwhat                                   # closed-form scales: plain straight-through, nothing to learn
        g["w"][name] = None
    else:
        inside, dwhat_ds = weight_ste(qw["z"], qw["q"], desc.w_bits, desc.w_grid)
        g[name] = dwhat * inside
        ds = (dwhat * dwhat_ds).sum(-1)
        g["w"][name] = ds if desc.w_per_row else np.array([ds.sum()])
    dxhat = dy @ qw["what"]
    return _act_back(desc, qa, dxhat, g, site)


def student_layer_backward(desc, p, c, dF):
    """Gradients of one layer given d l / d f_hat_l (loss term of this layer plus what
    flows back from the next layer).  Returns (d l / d layer input, grads dict)."""
    B, S = c["B"], c["S"]
    H = c["x"].shape[-1]
    h, d = desc.n_heads, H // desc.n_heads
    g = {"a": np.zeros(N_SITES), "a_off": np.zeros(N_SITES), "w": {}}
    qw = c["qw"]

    dy2, g["ln2_g"], g["ln2_b"] = layernorm_backward(dF, c["xn2"], c["rstd2"], p["ln2_g"])
    dG = _linear_back(desc, c["qG"], qw["W2"], dy2, "W2", g, SITE_G)
    dU = dG * gelu_grad(c["u"])
    dA = _linear_back(desc, c["qA"], qw["W1"], dU, "W1", g, SITE_A) + dy2
    dy1, g["ln1_g"], g["ln1_b"] = layernorm_backward(dA, c["xn1"], c["rstd1"], p["ln1_g"])
    dctx = _linear_back(desc, c["qC"], qw["Wo"], dy1, "Wo", g, SITE_C)

    dctx_h = _heads(dctx, h)
    Qh, Kh, Vh = (_heads(c[n]["xhat"], h) for n in ("qQ", "qK", "qV"))
    dPhat = dctx_h @ Vh.transpose(0, 1, 3, 2)
    dVhat = c["qP"]["xhat"].transpose(0, 1, 3, 2) @ dctx_h
    dP = _act_back(desc, c["qP"], dPhat, g, SITE_P)
    P = c["P"]
    dS = P * (dP - (dP * P).sum(-1, keepdims=True))
    dQhat = dS @ Kh / np.sqrt(d)
    dKhat = dS.transpose(0, 1, 3, 2) @ Qh / np.sqrt(d)
    dQ = _act_back(desc, c["qQ"], _merge(dQhat), g, SITE_Q)
    dK = _act_back(desc, c["qK"], _merge(dKhat), g, SITE_K)
    dV = _act_back(desc, c["qV"], _merge(dVhat), g, SITE_V)
    dqkv = np.concatenate([dQ, dK, dV], axis=-1)
    dX = _linear_back(desc, c["qx"], qw["Wqkv"], dqkv, "Wqkv", g, SITE_X) + dy1
    return dX, g


def student_backward(desc, params, caches, dF_list):
    """Backward through the module.  The loss gradient of Eq. 3 enters at every layer
    output; the gradient stops at the module input (it stays local to the module,
    Sec. 4.2).  Returns the list of per-layer gradient dicts."""
    return student_backward_with_input_grad(desc, params, caches, dF_list)[0]


def student_backward_with_input_grad(desc, params, caches, dF_list):
    """The same, returning also the gradient with respect to the module's input (after the straight-through pass
    of the first layer's input quantizer and its skip connection): the model's first module hands it to the
    embedding layers, which belong to that module (Sec. 4.1)."""
    grads = [None] * len(params)
    carry = 0.0
    for l in reversed(range(len(params))):
        carry, grads[l] = student_layer_backward(desc, params[l], caches[l], dF_list[l] + carry)
    return grads, carry


# ----------------------------------------------------------------------------- update (Alg. 2, Update(.) = AdamW)

def adamw_update(p, g, m, v, t, lr, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0):
    """One AdamW step (decoupled weight decay, bias-corrected moments); t counts from 1.
    Returns (p, m, v) as new float64 arrays."""
    p, g, m, v = (np.asarray(a, np.float64) for a in (p, g, m, v))
    m = beta1 * m + (1.0 - beta1) * g
    v = beta2 * v + (1.0 - beta2) * g * g
    mhat = m / (1.0 - beta1 ** t)
    vhat = v / (1.0 - beta2 ** t)
    p = p * (1.0 - lr * weight_decay) - lr * mhat / (np.sqrt(vhat) + eps)
    return p, m, v


def linear_decay_lr(lr0, t, total):
    """Learning rate of step t (0-based) under linear decay to zero over `total` steps (Sec. 5.1)."""
    return lr0 * (1.0 - t / total)


MIN_STEP = 1e-8   # step sizes are positive (Eq. 1: s in R+); clamp after each update


# ----------------------------------------------------------------------------- initial step sizes

def init_weight_steps(desc, params, rule=0):
    """rule 0: s = max|w| / qmax per group (nothing is clipped at the start);
    rule 1: s = mean|w| per group (2-bit settings).  Group = output row or whole matrix."""
    out = []
    for p in params:
        d = {}
        for k in WEIGHTS:
            w = np.abs(np.asarray(p[k], np.float64))
            if not desc.w_per_row:
                w = w.reshape(1, -1)
            if rule == 0:
                qmax = sym_qmax(desc.w_bits) if desc.w_grid == 0 else 1.5
                d[k] = (w.max(-1) / qmax).astype(np.float32)
            else:
                d[k] = w.mean(-1).astype(np.float32)
            d[k] = np.maximum(d[k], np.float32(MIN_STEP))
        out.append(d)
    return out


def init_act_steps(desc, params, x, valid_len=None):
    """One pass of the unquantized student over a batch; each site gets
    s = max|x| / qmax (symmetric) or (max - min) / (2^b - 1) with offset min (GELU site;
    the softmax site keeps offset 0: s = max / (2^b - 1)).  Returns (a[L,8], a_off[L,8])."""
    byp = ModuleDesc(**{**desc.__dict__, "w_bits": 0, "a_bits": 0})
    L = len(params)
    a = np.zeros((L, N_SITES), np.float32)
    off = np.zeros((L, N_SITES), np.float32)
    dummy = [dict(w={k: None for k in WEIGHTS}, a=a[0], a_off=off[0])] * L
    _, caches = student_forward(byp, params, dummy, x, valid_len)
    qs = sym_qmax(desc.a_bits)
    qu = 2 ** desc.a_bits - 1
    for l, c in enumerate(caches):
        Q, K, V = np.split(c["qkv"], 3, axis=-1)
        tens = {SITE_X: c["x"], SITE_Q: Q, SITE_K: K, SITE_V: V, SITE_P: c["P"],
                SITE_C: c["ctx"], SITE_A: c["a"], SITE_G: c["g"]}
        for site, t in tens.items():
            if site == SITE_P and desc.asym_p:
                a[l, site] = np.float32(np.float32(t.max()) / np.float32(qu))
            elif site == SITE_G and desc.asym_g:
                lo, hi = np.float32(t.min()), np.float32(t.max())
                a[l, site] = np.float32(np.float32(hi - lo) / np.float32(qu))
                off[l, site] = lo
            else:
                a[l, site] = np.float32(np.float32(np.abs(t).max()) / np.float32(qs))
    return np.maximum(a, np.float32(MIN_STEP)), off


# ----------------------------------------------------------------------------- one reconstruction step (Alg. 2)

def make_steps(w_steps, a, a_off):
    return [dict(w={k: np.array(w_steps[l][k], np.float32) for k in WEIGHTS},
                 a=np.array(a[l], np.float32), a_off=np.array(a_off[l], np.float32))
            for l in range(len(w_steps))]


def forward_loss_backward(desc, teacher, student, steps, x_t, x_s, valid_len=None, lam=0.0, head=None):
    """Teacher output, student output, loss of Eq. 3 and all gradients (no update).  With `head` (the last
    module of the model) the output-logit term is added to the loss and its gradient enters at the last
    layer's output beside that layer's own term."""
    f_t = teacher_forward(desc, teacher, x_t, valid_len)
    f_s, caches = student_forward(desc, student, steps, x_s, valid_len, x_teacher=x_t, lam=lam)
    total, per, dF = recon_loss(desc, f_s, f_t)
    out = dict(f_t=f_t, f_s=f_s, loss_per_layer=per, caches=caches)
    if head is not None:
        lz, dFz, z_s, z_t = logit_loss(desc, head, f_s[-1], f_t[-1])
        total += lz
        dF[-1] = dF[-1] + dFz
        out.update(logit_loss=lz, logits_student=z_s, logits_teacher=z_t)
    out["loss"] = total
    out["grads"], out["d_input"] = student_backward_with_input_grad(desc, student, caches, dF)
    return out


def recon_step(desc, teacher, student, steps, state, x_t, x_s, valid_len=None, lam=0.0,
               lr=1e-4, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01):
    """One call of the MREM procedure (Alg. 2): forward both modules, loss, gradients,
    then Update(w) and Update(s).  `state` holds the step count 't' and the moments
    (created on first use).  Matrices get weight decay, everything else none.
    Updates `student` and `steps` in place; returns the forward/backward record."""
    r = forward_loss_backward(desc, teacher, student, steps, x_t, x_s, valid_len, lam)
    state["t"] = state.get("t", 0) + 1
    t = state["t"]

    def upd(key, p, g, wd):
        m, v = state.get(key, (np.zeros_like(p, np.float64), np.zeros_like(p, np.float64)))
        p2, m, v = adamw_update(p, g, m, v, t, lr, beta1, beta2, eps, wd)
        state[key] = (m, v)
        return p2

    for l, g in enumerate(r["grads"]):
        for k in PARAMS:
            wd = weight_decay if k in WEIGHTS else 0.0
            student[l][k] = upd((l, k), student[l][k], g[k], wd).astype(np.float32)
        for k in WEIGHTS:
            if g["w"][k] is not None:
                steps[l]["w"][k] = np.maximum(upd((l, "s", k), steps[l]["w"][k], g["w"][k], 0.0),
                                              MIN_STEP).astype(np.float32)
        if desc.a_bits:
            steps[l]["a"] = np.maximum(upd((l, "a"), steps[l]["a"], g["a"], 0.0), MIN_STEP).astype(np.float32)
            steps[l]["a_off"] = upd((l, "a_off"), steps[l]["a_off"], g["a_off"], 0.0).astype(np.float32)
    return r


# ----------------------------------------------------------------------------- embedding layers of the first module (Sec. 4.1)

EMBED_PARAMS = ("word", "pos", "type", "ln_g", "ln_b")


def embed_forward(desc, tables, ids, type_ids, word_step=None, e_bits=0):
    """BERT embedding layers: LayerNorm(word[ids] + pos[0..S) + type[type_ids]) -> [B, S, H].
    Student side (`e_bits` > 0): the word-embedding table is quantized by Eq. 1 with one learnable step per
    row (symmetric uniform, Sec. 3.1); position / token-type tables and the LayerNorm are not.  The sum
    before the LayerNorm and the output are rounded as stored.  Returns (output, cache)."""
    st = lambda t: store(t, desc.act_dtype)
    ids = np.asarray(ids)
    B, S = ids.shape
    word = np.asarray(tables["word"], np.float64)
    c = dict(ids=ids, type_ids=np.asarray(type_ids), B=B, S=S)
    if e_bits:
        s_rows = np.asarray(word_step, np.float32).reshape(-1, 1)
        q, scale, z = quantize_weight(tables["word"], s_rows, e_bits, 0, desc.act_dtype)
        c.update(q=q, z=z)
        rows = (scale * q)[ids]
    else:
        rows = word[ids]
    y = st(rows + np.asarray(tables["pos"], np.float64)[None, :S, :] + np.asarray(tables["type"], np.float64)[c["type_ids"]])
    out, xn, rstd = layernorm(y, tables["ln_g"], tables["ln_b"], desc.ln_eps)
    c.update(y=y, xn=xn, rstd=rstd)
    return st(out), c


def embed_loss_backward(desc, teacher, student, word_step, e_bits, ids, type_ids, d_extra=None):
    """MSE between the student's and the teacher's embedding output (Sec. 4.1) and its gradients w.r.t. the
    student's latent word table (straight-through, rows gathered several times add up), its row steps, the
    position and token-type tables and the LayerNorm parameters.  `d_extra` [B, S, H]: a gradient that arrives
    at the student's embedding output from the layers it feeds (the first module's input gradient), added to
    the gradient of the MSE."""
    e_t, _ = embed_forward(desc, teacher, ids, type_ids)
    e_s, c = embed_forward(desc, student, ids, type_ids, word_step, e_bits)
    diff = e_s - e_t
    cc = 1.0 / diff.size if desc.loss_mean else 1.0
    loss = cc * float((diff * diff).sum())
    dE = 2.0 * cc * diff
    if d_extra is not None:
        dE = store(dE, desc.act_dtype) + np.asarray(d_extra, np.float64)
    dy, g_ln_g, g_ln_b = layernorm_backward(dE, c["xn"], c["rstd"], student["ln_g"])
    B, S, H = dy.shape
    g = dict(ln_g=g_ln_g, ln_b=g_ln_b)
    g["pos"] = np.zeros(np.shape(student["pos"]), np.float64)
    g["pos"][:S] = dy.sum(0)
    g["type"] = np.zeros(np.shape(student["type"]), np.float64)
    np.add.at(g["type"], c["type_ids"].reshape(-1), dy.reshape(-1, H))
    dwhat = np.zeros(np.shape(student["word"]), np.float64)
    np.add.at(dwhat, c["ids"].reshape(-1), dy.reshape(-1, H))
    if e_bits:
        inside, dwhat_ds = weight_ste(c["z"], c["q"], e_bits, 0)
        g["word"] = dwhat * inside
        g["word_step"] = (dwhat * dwhat_ds).sum(-1)
    else:
        g["word"], g["word_step"] = dwhat, None
    return dict(e_t=e_t, e_s=e_s, loss=loss, grads=g, cache=c)


def embed_step(desc, teacher, student, word_step, state, e_bits, ids, type_ids, lr=1e-4, beta1=0.9, beta2=0.999,
               eps=1e-8, weight_decay=0.01, d_extra=None):
    """One optimisation step of the embedding objective: gradients as above, then AdamW on every student
    table (the three embedding tables decayed like weight matrices, LayerNorm parameters not) and on the word
    table's row steps (kept >= MIN_STEP).  Updates `student` and `word_step` in place; returns the record."""
    r = embed_loss_backward(desc, teacher, student, word_step, e_bits, ids, type_ids, d_extra)
    state["t"] = state.get("t", 0) + 1
    t = state["t"]

    def upd(key, p, g, wd):
        p = np.asarray(p, np.float64)
        m, v = state.get(key, (np.zeros_like(p), np.zeros_like(p)))
        p2, m, v = adamw_update(p, np.asarray(g, np.float64), m, v, t, lr, beta1, beta2, eps, wd)
        state[key] = (m, v)
        return p2

    for k in EMBED_PARAMS:
        wd = weight_decay if k in ("word", "pos", "type") else 0.0
        student[k] = upd(k, student[k], r["grads"][k], wd).astype(np.float32)
    if r["grads"]["word_step"] is not None:
        word_step[:] = np.maximum(upd("word_step", word_step, r["grads"]["word_step"], 0.0), MIN_STEP).astype(np.float32)
    return r


# ----------------------------------------------------------------------------- output logits of the last module (Sec. 4.1)

def head_logits(head, f_last):
    """Classification head on the last layer's output f_last [B, S, H] (as stored): the first token of every
    sequence through the pooler (dense + tanh) and the classifier (dense).  The head is not quantized
    (Sec. 3.1) and is the same on the teacher and the student side.  head: dict Wp [H, H], bp [H],
    Wc [C, H], bc [C].  Returns (logits [B, C], pooled [B, H])."""
    cls = np.asarray(f_last, np.float64)[:, 0, :]
    pooled = np.tanh(cls @ np.asarray(head["Wp"], np.float64).T + np.asarray(head["bp"], np.float64))
    return pooled @ np.asarray(head["Wc"], np.float64).T + np.asarray(head["bc"], np.float64), pooled


def logit_loss(desc, head, f_student_last, f_teacher_last):
    """The output-logit term of the last module: l_z = c * || z_hat - z ||^2, c = 1 / (B * C) when `loss_mean`
    (MSE) else 1.  Returns (loss, d l_z / d f_hat_last [B, S, H]: non-zero at the first token only, logits of
    the student, logits of the teacher)."""
    z_t, _ = head_logits(head, f_teacher_last)
    z_s, pooled = head_logits(head, f_student_last)
    diff = z_s - z_t
    c = 1.0 / diff.size if desc.loss_mean else 1.0
    loss = c * float((diff * diff).sum())
    dz = 2.0 * c * diff
    dpre = (dz @ np.asarray(head["Wc"], np.float64)) * (1.0 - pooled * pooled)
    dF = np.zeros(np.shape(f_student_last), np.float64)
    dF[:, 0, :] = dpre @ np.asarray(head["Wp"], np.float64)
    return loss, dF, z_s, z_t


# ----------------------------------------------------------------------------- Eq. 2: reconstruction error of ONE matrix product

# the activation quantizer that sits at the input of each of a layer's four products
REM_SITE = {"Wqkv": SITE_X, "Wo": SITE_C, "W1": SITE_A, "W2": SITE_G}


def rem_forward_loss_backward(desc, w_teacher, w_student, steps, name, a):
    """The per-product objective of Eq. 2 for the matrix `name` of one layer:
        l = c * || Q(w)^T Q(a) - w^T a ||^2   over the rows of a,
    w the full-precision (teacher) matrix, Q(w) the student's quantized one, Q(a) the
    input quantizer of that product; c = 1 / (rows * out) when `loss_mean`, else 1 as
    printed.  No bias on either side (Eq. 2 has none).  `steps` is the layer's step
    dict (make_steps).  Returns the target, the quantized product, the loss and the
    gradients w.r.t. the latent matrix, its step(s), the activation step and offset
    (straight-through estimator of Sec. 3.1.1)."""
    st = lambda t: store(t, desc.act_dtype)
    a = np.asarray(a, np.float64)
    site = REM_SITE[name]
    target = st(a @ st(w_teacher).T)
    qa = _q_act(desc, a, steps, site)
    qw = _q_w(desc, w_student, steps["w"][name])
    y = st(student_linear(qa, qw, 0.0))
    diff = y - target
    c = 1.0 / diff.size if desc.loss_mean else 1.0
    loss = c * float((diff * diff).sum())
    dy = 2.0 * c * diff
    dwhat = dy.T @ qa["xhat"]
    out = dict(target=target, y=y, loss=loss, qa=qa, qw=qw, d_a_step=0.0, d_a_off=0.0)
    if qw["q"] is None or qw.get("closed"):
        out["dW"], out["d_w_step"] = dwhat, None
    else:
        inside, dwhat_ds = weight_ste(qw["z"], qw["q"], desc.w_bits, desc.w_grid)
        out["dW"] = dwhat * inside
        ds = (dwhat * dwhat_ds).sum(-1)
        out["d_w_step"] = ds if desc.w_per_row else np.array([ds.sum()])
    if qa["q"] is not None:
        dxhat = dy @ qw["what"]
        inside, dxhat_ds = act_ste(qa["z"], qa["q"], qa["lo"], qa["hi"])
        out["d_a_step"] = float((dxhat * dxhat_ds).sum())
        if qa["asym"]:
            out["d_a_off"] = float((dxhat * (1.0 - inside)).sum())
    return out


def rem_step(desc, w_teacher, w_student, steps, state, name, a, lr=1e-4, beta1=0.9, beta2=0.999, eps=1e-8,
             weight_decay=0.01):
    """One optimisation step of Eq. 2 on one product: gradients as above, then AdamW on
    the latent matrix (with weight decay), its step(s), the input quantizer's step and
    offset.  `state`: step count 't' and moments per key.  Returns (record, new matrix);
    `steps` is updated in place."""
    r = rem_forward_loss_backward(desc, w_teacher, w_student, steps, name, a)
    site = REM_SITE[name]
    state["t"] = state.get("t", 0) + 1
    t = state["t"]

    def upd(key, p, g, wd):
        p = np.asarray(p, np.float64)
        m, v = state.get(key, (np.zeros_like(p), np.zeros_like(p)))
        p2, m, v = adamw_update(p, np.asarray(g, np.float64), m, v, t, lr, beta1, beta2, eps, wd)
        state[key] = (m, v)
        return p2

    w_new = upd(("W", name), w_student, r["dW"], weight_decay).astype(np.float32)
    if r["d_w_step"] is not None:
        steps["w"][name] = np.maximum(upd(("s", name), steps["w"][name], r["d_w_step"].reshape(np.shape(steps["w"][name])), 0.0),
                                      MIN_STEP).astype(np.float32)
    if desc.a_bits:
        steps["a"][site] = np.float32(max(float(upd(("a", site), np.array([steps["a"][site]]), np.array([r["d_a_step"]]), 0.0)[0]), MIN_STEP))
        if r["qa"]["asym"] and site == SITE_G:
            steps["a_off"][site] = np.float32(upd(("off", site), np.array([steps["a_off"][site]]), np.array([r["d_a_off"]]), 0.0)[0])
    return r, w_new


# ----------------------------------------------------------------------------- Algorithm 1: modules trained in parallel from input queues

def mremp_run(descs, teachers, students, steps, batches, draws, t0, T, T0, lr0, lr_total=0, log=None, **adam):
    """Algorithm 1 (Sec. 4.2) on N modules, one module after the other inside a step (the result does not
    depend on the order: a module only reads what its predecessor produced in EARLIER steps, except while the
    queues are being filled).

    descs, teachers, students, steps: per module n = 0 .. N-1 (students and steps are updated in place)
    batches: batches[t] = (x [B,S,H], valid_len or None), the calibration batch module 0 takes at step t
    draws:   draws[t][n] in [0, t0): which of the t0 most recent queue entries module n >= 1 samples at step
             t >= t0 (0 = the most recent); the same entry is taken from the teacher-side and the
             student-side queue, so both modules see the same sequences
    t0:      staleness threshold = queue length.  In the first t0 steps every module is computed one after
             another and module n takes what module n-1 produced in the SAME step (filling the queues)
    T, T0:   steps per module; teacher forcing lambda_t = max(1 - t/T0, 0) for t < T0, none afterwards (Alg. 2)
    lr0, lr_total: AdamW learning rate, linearly decayed over lr_total steps when lr_total > 0
    Queue entries are (f_t, f_hat_t, valid_len) of the forward pass of step t (before that step's update),
    kept first-in-first-out.  Returns losses[n][t]; `log`, if a list, receives (t, n, entry index or None).
    """
    N = len(descs)
    queues = [[] for _ in range(N)]                      # queues[n]: most recent first, at most t0 entries
    states = [dict() for _ in range(N)]
    losses = [[] for _ in range(N)]
    for t in range(T):
        lam = teacher_forcing_lambda(t, T0) if t < T0 else 0.0
        lr = linear_decay_lr(lr0, t, lr_total) if lr_total > 0 else lr0
        produced = []
        for n in range(N):
            if n == 0:
                x_t, vl = batches[t]
                x_s, k = x_t, None
            elif t < t0:
                x_t, x_s, vl = produced[n - 1]           # filling: the predecessor's output of this very step
                k = None
            else:
                k = int(draws[t][n])
                assert 0 <= k < len(queues[n - 1])
                x_t, x_s, vl = queues[n - 1][k]
            if log is not None:
                log.append((t, n, k))
            r = recon_step(descs[n], teachers[n], students[n], steps[n], states[n], x_t, x_s, vl, lam, lr=lr, **adam)
            losses[n].append(r["loss"])
            produced.append((r["f_t"][-1], r["f_s"][-1], vl))
        for n in range(N):                               # first in, first out
            queues[n].insert(0, produced[n])
            del queues[n][t0:]
    return losses
