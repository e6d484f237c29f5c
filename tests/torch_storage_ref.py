"""A second statement of the full-precision (teacher) layer with bfloat16 storage, from torch library layers.

Used two ways, never by the product and never by the oracle:
  * in float64 it pins WHERE the oracle's storage-emulation mode rounds (tests/test_oracle_storage_pins.py);
  * in float32 it is "another correct implementation" (float32 sums in the library's own order, same storage
    points), whose distance from the float64 oracle is the noise floor that the GPU comparison at full width
    is held against (tests/test_gpu_full_width.py, tests/test_gpu_module.py): with bf16 storage a difference in
    the last bits before a rounding flips that rounding, the flip (2^-8 relative) feeds the next sum, and the
    outlier channels of the workloads spread a single flipped element over its whole row through the
    LayerNorm statistics, so even two exact-to-float32 implementations differ in a sizeable share of the
    output elements."""
import math

import numpy as np
import torch
import torch.nn.functional as F

WEIGHTS = ("Wqkv", "Wo", "W1", "W2")


def round_bf16_t(t):
    return t.to(torch.bfloat16).to(t.dtype)


def teacher_layer_torch(p, x, vl, h, rnd=round_bf16_t, dtype=torch.float64, eps=1e-12):
    """Full-precision layer with the storage roundings written out: the layer input, the matrices, qkv, the
    softmax output, the context, both pre-LayerNorm sums, both LayerNorm outputs and the GELU output live in the
    storage type; the pre-GELU tensor does not (bias and GELU are applied to the accumulator before it is
    stored).  `rnd` is applied at each of those 13 points; sums run in `dtype`.  Returns float64 numpy."""
    t = {k: torch.tensor(np.asarray(v, np.float64)).to(dtype) for k, v in p.items()}
    W = {k: rnd(t[k]) for k in WEIGHTS}
    xt = rnd(torch.tensor(np.asarray(x, np.float64)).to(dtype))
    B, S, H = xt.shape
    d = H // h
    qkv = rnd(F.linear(xt, W["Wqkv"], t["bqkv"]))
    Q, K, V = qkv.split(H, dim=-1)
    sp = lambda u: u.reshape(B, S, h, d).transpose(1, 2)
    pad = (torch.arange(S)[None, :] >= torch.as_tensor(vl)[:, None])[:, None, None, :]
    P = rnd(torch.softmax((sp(Q) @ sp(K).transpose(-1, -2) / math.sqrt(d)).masked_fill(pad, float("-inf")), dim=-1))
    ctx = rnd((P @ sp(V)).transpose(1, 2).reshape(B, S, H))
    y1 = rnd(F.linear(ctx, W["Wo"], t["bo"]) + xt)
    a = rnd(F.layer_norm(y1, (H,), t["ln1_g"], t["ln1_b"], eps))
    g = rnd(F.gelu(F.linear(a, W["W1"], t["b1"])))
    y2 = rnd(F.linear(g, W["W2"], t["b2"]) + a)
    return rnd(F.layer_norm(y2, (H,), t["ln2_g"], t["ln2_b"], eps)).to(torch.float64).numpy()


def bf16_numbers_apart(a, b):
    """bf16-representable arrays -> distance counted in representable numbers."""
    def key(v):
        u = np.ascontiguousarray(np.asarray(v, np.float32)).view(np.uint32).astype(np.int64) >> 16
        return np.where(u & 0x8000, -(u & 0x7FFF), u)
    return np.abs(key(a) - key(b))
