"""A float64 torch model of the quantized module whose gradients come from library
autograd.  It is used only to pin the oracle's hand-written forward and backward.

The straight-through estimator is expressed with the detach idiom: with
z = x / s and zc = clamp(z), the quantized value is s * (zc + (round(zc) - zc).detach()),
so autograd yields d/dx = 1[inside] and d/ds = q - z inside, the clipped code outside.
"""
import math

import torch
import torch.nn.functional as F


def q_sym(x, s, bits):
    qmax = 2 ** (bits - 1) - 1
    zc = torch.clamp(x / s, -qmax, qmax)
    return s * (zc + (torch.round(zc) - zc).detach())


def q_asym(x, s, beta, bits):
    qmax = 2 ** bits - 1
    zc = torch.clamp((x - beta) / s, 0, qmax)
    return s * (zc + (torch.round(zc) - zc).detach()) + beta


def q_weight(w, s, bits, grid):
    s = s.reshape(-1, 1)
    if grid == 0:
        return q_sym(w, s, bits)
    # levels (k + 0.5) * s, k = floor(z) in [-2, 1]; gradient passes for -2 <= z < 2
    z = w / s
    inside = ((z >= -2) & (z < 2)).to(w.dtype)
    level = (torch.clamp(torch.floor(z), -2, 1) + 0.5).detach()
    # value: s * level ; d/dw = inside ; d/ds = level - z * inside
    return s * level + inside * (w - (s * z).detach()) + (s - s.detach()) * (-(z * inside)).detach()


def q_weight_twn(w, per_row=True):
    # closed-form ternary weights: value alpha * t, gradient passed to w unchanged
    a = w.detach().abs()
    g = a if per_row else a.reshape(1, -1)
    delta = (0.7 * g.mean(-1, keepdim=True)).float()                 # the comparison is made in float32
    w32 = (w.detach() if per_row else w.detach().reshape(1, -1)).float()
    keep = w32.abs() > delta
    alpha = (g * keep).sum(-1, keepdim=True) / keep.sum(-1, keepdim=True).clamp(min=1)
    alpha = alpha.float().double()
    what = (alpha * torch.sign(w32).double() * keep).reshape(w.shape)
    return w + (what - w).detach()


def q_weight_laq(w, bits, per_row=True, rounds=16):
    # scale refitted by alternating least squares from min(3 mean|w|, max|w|) / qmax: value alpha * q, gradient passed to w unchanged
    g = w.detach() if per_row else w.detach().reshape(1, -1)
    g32 = g.float()                                                   # codes are decided in float32
    qmax = 2 ** (bits - 1) - 1
    alpha = (torch.minimum(3.0 * g.abs().mean(-1, keepdim=True), g.abs().amax(-1, keepdim=True)) / qmax).float()
    q = torch.zeros_like(g)
    for _ in range(rounds):
        z = torch.where(alpha > 0, g32 / torch.where(alpha > 0, alpha, torch.ones_like(alpha)), torch.zeros_like(g32))
        q = torch.clamp(torch.round(z), -qmax, qmax).double()
        qq = (q * q).sum(-1, keepdim=True)
        alpha = torch.where(qq > 0, (q * g).sum(-1, keepdim=True) / qq.clamp(min=1), torch.zeros_like(qq)).float()
    what = (alpha.double() * q).reshape(w.shape)
    return w + (what - w).detach()


def layer(x, p, st, cfg, pad, quant=True):
    H = x.shape[-1]
    h = cfg["n_heads"]
    d = H // h
    ab, wb, grid = cfg["a_bits"], cfg["w_bits"], cfg["w_grid"]

    def qa(t, site):
        if not quant or ab == 0:
            return t
        if (site == 4 and cfg["asym_p"]):
            return q_asym(t, st["a"][site], torch.zeros((), dtype=t.dtype), ab)
        if (site == 7 and cfg["asym_g"]):
            return q_asym(t, st["a"][site], st["a_off"][site], ab)
        return q_sym(t, st["a"][site], ab)

    def qw(name):
        if not quant or wb == 0:
            return p[name]
        if cfg.get("w_twn"):
            return q_weight_twn(p[name], cfg.get("w_per_row", True))
        if cfg.get("w_laq"):
            return q_weight_laq(p[name], wb, cfg.get("w_per_row", True))
        return q_weight(p[name], st["w"][name], wb, grid)

    B, S, _ = x.shape
    qkv = F.linear(qa(x, 0), qw("Wqkv"), p["bqkv"])
    Q, K, V = qkv.split(H, dim=-1)
    sp = lambda t: t.reshape(B, S, h, d).transpose(1, 2)
    Qh, Kh, Vh = sp(qa(Q, 1)), sp(qa(K, 2)), sp(qa(V, 3))
    sc = Qh @ Kh.transpose(-1, -2) / math.sqrt(d)
    sc = sc.masked_fill(pad, float("-inf"))
    P = torch.softmax(sc, dim=-1)
    ctx = (qa(P, 4) @ Vh).transpose(1, 2).reshape(B, S, H)
    y1 = F.linear(qa(ctx, 5), qw("Wo"), p["bo"]) + x
    a = F.layer_norm(y1, (H,), p["ln1_g"], p["ln1_b"], cfg["ln_eps"])
    u = F.linear(qa(a, 6), qw("W1"), p["b1"])
    g = F.gelu(u)
    y2 = F.linear(qa(g, 7), qw("W2"), p["b2"]) + a
    return F.layer_norm(y2, (H,), p["ln2_g"], p["ln2_b"], cfg["ln_eps"])


def module(x, params, steps, cfg, valid_len, quant=True):
    B, S, _ = x.shape
    if valid_len is None:
        pad = torch.zeros(B, 1, 1, S, dtype=torch.bool)
    else:
        pad = (torch.arange(S)[None, :] >= torch.as_tensor(valid_len)[:, None])[:, None, None, :]
    outs, cur = [], x
    for p, st in zip(params, steps):
        cur = layer(cur, p, st, cfg, pad, quant)
        outs.append(cur)
    return outs
