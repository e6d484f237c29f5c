"""Seeded synthetic inputs for MREM reconstruction steps.

This module only draws numbers: it holds none of the method's arithmetic (no
quantizer, no Transformer op, no loss).  Both the CUDA tests and the CPU oracle's
tests take their tensors from here so that the two sides see identical bytes.

Generator: a counter-based stream.  Element ``i`` of the tensor called ``name``
under ``seed`` is produced from splitmix64(hash(seed, name) + i); two 53-bit
uniforms give one normal deviate by the Box-Muller transform.  Everything is
returned as float32 numpy arrays (or int32 for lengths / indices).

The workloads mimic the shape and structure of the paper's calibration data
(Sec. 5.1: a few thousand sequences of BERT-base / BERT-large hidden states at
sequence length 128 for classification and 384 for reading comprehension):
teacher weights ~ N(0, 0.02^2), LayerNorm gamma = 1 / beta = 0, biases 0,
hidden states ~ N(0, 1) with a few fixed channels scaled up as activation
outliers, and padded sequences with uniformly drawn valid lengths.
"""
from __future__ import annotations

import zlib
from dataclasses import dataclass, field

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _splitmix64(x: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        z = x + _GOLDEN
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        return z ^ (z >> np.uint64(31))


def _stream_base(seed: int, name: str) -> np.uint64:
    h = zlib.crc32(name.encode()) & 0xFFFFFFFF
    base = np.array([(int(seed) & 0xFFFFFFFF) << 32 | h], dtype=np.uint64)
    return _splitmix64(_splitmix64(base))[0]


def uniform(seed: int, name: str, n: int) -> np.ndarray:
    """n doubles in (0, 1), stream (seed, name)."""
    with np.errstate(over="ignore"):
        idx = np.arange(n, dtype=np.uint64) + _stream_base(seed, name)
    bits = _splitmix64(idx) >> np.uint64(11)
    return (bits.astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal(seed: int, name: str, shape, std: float = 1.0) -> np.ndarray:
    """float32 N(0, std^2) tensor of the given shape, stream (seed, name)."""
    n = int(np.prod(shape))
    u = uniform(seed, name, 2 * n)
    r = np.sqrt(-2.0 * np.log(u[:n]))
    v = r * np.cos(2.0 * np.pi * u[n:])
    return (v * std).astype(np.float32).reshape(shape)


def integers(seed: int, name: str, n: int, lo: int, hi: int) -> np.ndarray:
    """n int32 values uniform in [lo, hi] (inclusive)."""
    u = uniform(seed, name, n)
    return (lo + np.floor(u * (hi - lo + 1))).astype(np.int32).clip(lo, hi)


def permutation(seed: int, name: str, n: int) -> np.ndarray:
    """A seeded permutation of range(n) (argsort of a uniform stream)."""
    return np.argsort(uniform(seed, name, n), kind="stable").astype(np.int32)


PARAM_NAMES = ("Wqkv", "bqkv", "Wo", "bo", "ln1_g", "ln1_b",
               "W1", "b1", "W2", "b2", "ln2_g", "ln2_b")
WEIGHT_NAMES = ("Wqkv", "Wo", "W1", "W2")


@dataclass
class Workload:
    """Shape and structure of one reconstruction workload."""
    name: str
    n_layers: int
    hidden: int
    n_heads: int
    ffn: int
    seq: int
    batch: int
    w_bits: int = 4
    a_bits: int = 8
    w_grid: int = 0            # 0: integer grid Omega(b) of Eq. 1; 1: half-integer 2-bit grid; 2 / 3: closed-form scales
    act_dtype: str = "bf16"    # storage type of activations
    outlier_channels: int = 4  # channels of the input scaled by outlier_scale
    outlier_scale: float = 20.0
    len_lo: int = 0            # valid lengths uniform in [len_lo, len_hi]; 0 = no padding
    len_hi: int = 0
    input_layernorm: bool = False
    calib: int = 0             # sequences in the calibration set (0: a single batch)
    steps: int = 1
    lr: float = 1e-4
    w_step_rule: int = 0       # 0: max|w|/qmax per row; 1: mean|w| per row
    extra: dict = field(default_factory=dict)


def workloads() -> dict:
    """The five configurations the benchmark and the parity tests are stated on."""
    return {
        "tiny": Workload("tiny", 1, 128, 2, 512, 32, 4, act_dtype="f32",
                         outlier_channels=0, input_layernorm=True),
        "base3_w4a8": Workload("base3_w4a8", 3, 768, 12, 3072, 128, 32,
                               len_lo=32, len_hi=128, calib=1024, steps=100),
        "base3_w2a8": Workload("base3_w2a8", 3, 768, 12, 3072, 128, 32, w_bits=2, w_grid=1,
                               len_lo=32, len_hi=128, calib=1024, steps=100, w_step_rule=1),
        "large6_w4a8": Workload("large6_w4a8", 6, 1024, 16, 4096, 128, 32,
                                len_lo=32, len_hi=128, calib=1024, steps=200),
        "large6_w2a8_s384": Workload("large6_w2a8_s384", 6, 1024, 16, 4096, 384, 16,
                                     w_bits=2, w_grid=1, len_lo=128, len_hi=384,
                                     calib=1024, steps=200, w_step_rule=1),
    }


def param_shape(wl: Workload, name: str):
    H, F = wl.hidden, wl.ffn
    return {"Wqkv": (3 * H, H), "bqkv": (3 * H,), "Wo": (H, H), "bo": (H,),
            "ln1_g": (H,), "ln1_b": (H,), "W1": (F, H), "b1": (F,),
            "W2": (H, F), "b2": (H,), "ln2_g": (H,), "ln2_b": (H,)}[name]


def teacher_params(wl: Workload, seed: int = 0, bias_std: float = 0.0) -> list:
    """Per layer a dict name -> float32 array.  Weights N(0, 0.02^2); LayerNorm
    gamma 1, beta 0; biases 0 unless bias_std > 0 (tests use non-zero biases so
    that a dropped bias term cannot hide)."""
    layers = []
    for l in range(wl.n_layers):
        p = {}
        for name in PARAM_NAMES:
            shp = param_shape(wl, name)
            if name in WEIGHT_NAMES:
                p[name] = normal(seed, f"{wl.name}/L{l}/{name}", shp, 0.02)
            elif name.endswith("_g"):
                p[name] = np.ones(shp, np.float32)
                if bias_std > 0:
                    p[name] = p[name] + normal(seed, f"{wl.name}/L{l}/{name}", shp, bias_std)
            else:
                p[name] = np.zeros(shp, np.float32)
                if bias_std > 0:
                    p[name] = normal(seed, f"{wl.name}/L{l}/{name}", shp, bias_std)
        layers.append(p)
    return layers


def outlier_channel_ids(wl: Workload, seed: int = 0) -> np.ndarray:
    if wl.outlier_channels <= 0:
        return np.zeros((0,), np.int32)
    return np.sort(permutation(seed, f"{wl.name}/outliers", wl.hidden)[: wl.outlier_channels])


def hidden_states(wl: Workload, n_seq: int, seed: int = 0, tag: str = "x") -> np.ndarray:
    """[n_seq, seq, hidden] float32 module inputs."""
    x = normal(seed, f"{wl.name}/{tag}", (n_seq, wl.seq, wl.hidden))
    ch = outlier_channel_ids(wl, seed)
    if ch.size:
        x[:, :, ch] *= np.float32(wl.outlier_scale)
    if wl.input_layernorm:
        # plain standardisation of each token (a data-generation step, gamma=1, beta=0)
        x64 = x.astype(np.float64)
        mu = x64.mean(-1, keepdims=True)
        var = x64.var(-1, keepdims=True)
        x = ((x64 - mu) / np.sqrt(var + 1e-12)).astype(np.float32)
    return x


def valid_lengths(wl: Workload, n_seq: int, seed: int = 0) -> np.ndarray:
    """[n_seq] int32 valid lengths; positions >= length are padding keys."""
    if wl.len_lo <= 0:
        return np.full((n_seq,), wl.seq, np.int32)
    return integers(seed, f"{wl.name}/len", n_seq, wl.len_lo, wl.len_hi)


def shrink(wl: Workload, **kw) -> Workload:
    """A copy of a workload with some fields replaced (smaller batch, fewer layers ...)."""
    d = dict(wl.__dict__)
    d.update(kw)
    d["extra"] = dict(wl.extra)
    return Workload(**d)
