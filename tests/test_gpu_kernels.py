"""Parity of the single CUDA operations with the CPU oracle, through the C-ABI.
Integer codes and int32 accumulators must match bit for bit."""
import numpy as np
import pytest
import torch

from oracle import mrem_oracle as O
from paper_2109_15082_b200 import binding as B
from paper_2109_15082_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _stream():
    return torch.cuda.current_stream().cuda_stream


def _status():
    return torch.zeros(64, dtype=torch.int32, device=DEV)


def _bf16_from_bits(bits_u16: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits_u16.astype(np.int16)).view(torch.bfloat16)


# ----------------------------------------------------------------------------- activation quantizer

@pytest.mark.parametrize("step", [0.037, 1.0, 2.5e-3, 11.0])
@pytest.mark.parametrize("mode", ["sym8", "sym4", "asym8"])
def test_quantize_act_all_bf16_patterns(step, mode):
    bits = np.arange(65536, dtype=np.uint16)
    x = _bf16_from_bits(bits)
    xf = x.float().numpy()
    keep = np.isfinite(xf)
    x = x[torch.from_numpy(keep)].contiguous()
    xf = xf[keep]
    n = xf.size                                               # not a multiple of 8: ragged tail
    lo, hi, off = {"sym8": (-127, 127, None), "sym4": (-7, 7, None), "asym8": (0, 255, -0.17)}[mode]
    if off is None:
        q_ref, _ = O.quantize_sym(xf, np.float32(step), 8 if hi == 127 else 4, "f32")
    else:
        q_ref, _ = O.quantize_asym(xf, np.float32(step), np.float32(off), 8, "f32")
    xd = x.to(DEV)
    sd = torch.tensor([step], dtype=torch.float32, device=DEV)
    od = None if off is None else torch.tensor([off], dtype=torch.float32, device=DEV)
    q8 = torch.zeros(n, dtype=torch.int8, device=DEV)
    qt = torch.zeros(n, dtype=torch.bfloat16, device=DEV)
    B.mrem_quantize_act(xd, B.BF16, n, sd, od, lo, hi, q8, qt, _stream())
    torch.cuda.synchronize()
    got8 = q8.cpu().numpy()
    got8 = got8.astype(np.uint8).astype(np.int64) if lo == 0 else got8.astype(np.int64)
    assert np.array_equal(got8, q_ref)
    assert np.array_equal(qt.float().cpu().numpy().astype(np.int64), q_ref)


@pytest.mark.parametrize("n", [0, 1, 7, 4096, 100003])
def test_quantize_act_f32_sizes(n):
    x = synth.normal(3, f"qa{n}", (max(n, 1),), 2.0)[:n]
    step = np.float32(0.0131)
    q_ref, _ = O.quantize_sym(x, step, 8, "f32")
    xd = torch.from_numpy(x.copy()).to(DEV)
    sd = torch.tensor([step], dtype=torch.float32, device=DEV)
    q8 = torch.full((n + 8,), 99, dtype=torch.int8, device=DEV)
    B.mrem_quantize_act(xd if n else q8, B.F32, n, sd, None, -127, 127, q8, None, _stream())
    torch.cuda.synchronize()
    assert np.array_equal(q8[:n].cpu().numpy().astype(np.int64), q_ref)
    assert torch.all(q8[n:] == 99)                              # nothing written past the end


# ----------------------------------------------------------------------------- weight quantizer

@pytest.mark.parametrize("bits,grid,per_row", [(4, 0, 1), (4, 0, 0), (2, 0, 1), (2, 1, 1), (8, 0, 1), (2, 1, 0)])
@pytest.mark.parametrize("rows,cols", [(37, 130), (256, 1024)])
def test_quantize_weight_codes_rowsums(bits, grid, per_row, rows, cols):
    w = synth.normal(4, f"w{rows}", (rows, cols), 0.02)
    desc = O.ModuleDesc(1, cols, 1, rows, bits, 8, w_grid=grid, w_per_row=bool(per_row))
    steps = O.init_weight_steps(desc, [dict(Wqkv=w, Wo=w, W1=w, W2=w)], 1 if bits == 2 else 0)[0]["W1"]
    steps = (steps * 0.7).astype(np.float32)                    # some weights clip
    c_ref, scale_ref, _ = O.quantize_weight(w, steps.reshape(-1, 1), bits, grid, "f32")
    wd = torch.from_numpy(w).to(DEV)
    sd = torch.from_numpy(steps).to(DEV)
    codes = torch.zeros(rows, cols, dtype=torch.int8, device=DEV)
    rowsum = torch.zeros(rows, dtype=torch.int32, device=DEV)
    scale = torch.zeros(rows, dtype=torch.float32, device=DEV)
    what = torch.zeros(rows, cols, dtype=torch.bfloat16, device=DEV)
    B.mrem_quantize_weight(wd, rows, cols, sd, per_row, bits, grid, codes, rowsum, scale, what, B.BF16, _stream())
    torch.cuda.synchronize()
    assert np.array_equal(codes.cpu().numpy().astype(np.int64), c_ref)
    assert np.array_equal(rowsum.cpu().numpy().astype(np.int64), c_ref.sum(-1))
    assert np.array_equal(scale.cpu().numpy(), np.broadcast_to(scale_ref.astype(np.float32).reshape(-1, 1), (rows, 1)).reshape(-1)
                          if per_row else np.full(rows, scale_ref.astype(np.float32).reshape(-1)[0]))
    ref_hat = O.round_bf16((scale_ref.astype(np.float32) * c_ref.astype(np.float32)).astype(np.float32))
    assert np.array_equal(what.float().cpu().numpy().astype(np.float64), ref_hat)


# ----------------------------------------------------------------------------- int8 tensor-core product

I8_SHAPES = [(128, 128, 128), (300, 200, 144), (1000, 520, 1040), (77, 3072, 1024), (1, 16, 16), (513, 72, 4096)]


@pytest.mark.parametrize("M,N,K", I8_SHAPES)
@pytest.mark.parametrize("block_n", [0, 64, 128, 256])
@pytest.mark.parametrize("a_unsigned", [0, 1])
def test_gemm_i8_exact(M, N, K, block_n, a_unsigned):
    rng = np.random.default_rng(M * 7 + N * 3 + K + a_unsigned)
    a = rng.integers(0, 256, (M, K)) if a_unsigned else rng.integers(-127, 128, (M, K))
    b = rng.integers(-127, 128, (N, K))
    ref = O.int_matmul(a, b)
    ad = torch.from_numpy(a.astype(np.uint8).view(np.int8) if a_unsigned else a.astype(np.int8)).to(DEV)
    bd = torch.from_numpy(b.astype(np.int8)).to(DEV)
    acc = torch.full((M, N), -1, dtype=torch.int32, device=DEV)
    st = _status()
    B.mrem_gemm_i8(ad, a_unsigned, bd, M, N, K, acc, block_n, st, _stream())
    torch.cuda.synchronize()
    assert int(st[0]) == 0
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), ref)


def test_gemm_i8_worst_case_magnitude_and_errors():
    M, N, K = 130, 70, 4096                                    # |acc| = K*127*127 < 2^31: no overflow
    a = np.full((M, K), 127, np.int8)
    b = np.full((N, K), -127, np.int8)
    acc = torch.zeros(M, N, dtype=torch.int32, device=DEV)
    st = _status()
    B.mrem_gemm_i8(torch.from_numpy(a).to(DEV), 0, torch.from_numpy(b).to(DEV), M, N, K, acc, 0, st, _stream())
    torch.cuda.synchronize()
    assert torch.all(acc == -K * 127 * 127)
    with pytest.raises(B.MremError) as e:                      # K not a multiple of 16: rejected on the host
        B.mrem_gemm_i8(acc, 0, acc, 4, 4, 24, acc, 0, st, _stream())
    assert e.value.code == -2
    with pytest.raises(B.MremError):
        B.mrem_gemm_i8(None, 0, acc, 4, 4, 16, acc, 0, st, _stream())
    B.mrem_gemm_i8(acc, 0, acc, 0, 4, 16, acc, 0, st, _stream())   # empty problem: no-op


def test_gemm_i8_full_size_sampled():
    # the benchmark's largest linear shape; the oracle checks sampled rows/columns
    M, N, K = 4096, 4096, 1024
    rng = np.random.default_rng(5)
    a = rng.integers(-127, 128, (M, K)).astype(np.int8)
    b = rng.integers(-7, 8, (N, K)).astype(np.int8)
    acc = torch.zeros(M, N, dtype=torch.int32, device=DEV)
    st = _status()
    B.mrem_gemm_i8(torch.from_numpy(a).to(DEV), 0, torch.from_numpy(b).to(DEV), M, N, K, acc, 0, st, _stream())
    torch.cuda.synchronize()
    assert int(st[0]) == 0
    rows = rng.integers(0, M, 64)
    got = acc.cpu().numpy()
    assert np.array_equal(got[rows].astype(np.int64), O.int_matmul(a[rows], b))
    cols = rng.integers(0, N, 64)
    assert np.array_equal(got[:, cols].astype(np.int64), O.int_matmul(a, b[cols]))


# ----------------------------------------------------------------------------- bf16 / f32 products, every operand layout

def _layout(x, mn):
    """x: [batch, MN, K] logical.  mn=0: stored k-contiguous, mn=1: stored mn-contiguous."""
    return np.ascontiguousarray(x.transpose(0, 2, 1)) if mn else np.ascontiguousarray(x)


@pytest.mark.parametrize("dtype", [B.BF16, B.F32])
@pytest.mark.parametrize("a_mn,b_mn", [(0, 0), (0, 1), (1, 0), (1, 1)])
@pytest.mark.parametrize("M,N,K,nb", [(128, 128, 64, 1), (200, 136, 72, 3), (384, 64, 384, 4), (520, 264, 200, 1)])
def test_gemm_float_layouts(dtype, a_mn, b_mn, M, N, K, nb):
    a = synth.normal(6, f"A{M}{a_mn}", (nb, M, K), 1.0)
    b = synth.normal(6, f"B{N}{b_mn}", (nb, N, K), 1.0)
    tdt = torch.bfloat16 if dtype == B.BF16 else torch.float32
    ad = torch.from_numpy(_layout(a, a_mn)).to(DEV).to(tdt).contiguous()
    bd = torch.from_numpy(_layout(b, b_mn)).to(DEV).to(tdt).contiguous()
    a64 = ad.float().cpu().numpy().astype(np.float64)
    b64 = bd.float().cpu().numpy().astype(np.float64)
    a64 = a64.transpose(0, 2, 1) if a_mn else a64
    b64 = b64.transpose(0, 2, 1) if b_mn else b64
    ref = 0.5 * a64 @ b64.transpose(0, 2, 1)
    out = torch.zeros(nb, M, N, dtype=torch.float32, device=DEV)
    st = _status()
    B.mrem_gemm(dtype, ad, a_mn, M if a_mn else K, M * K, bd, b_mn, N if b_mn else K, N * K, M, N, K, nb, 0.5, out,
                N, M * N, 0, st, _stream())
    torch.cuda.synchronize()
    assert int(st[0]) == 0
    got = out.cpu().numpy().astype(np.float64)
    rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    assert rel < 2e-6, rel


@pytest.mark.parametrize("shape", [(128, 64, 384, 2), (320, 576, 208, 1), (4096, 1024, 128, 1)])
@pytest.mark.parametrize("a_mn,b_mn", [(0, 0), (0, 1), (1, 0), (1, 1)])
def test_gemm_bf16_on_integer_codes_is_exact(a_mn, b_mn, shape):
    # attention products run on codes held as bf16 numbers: sums stay below 2^24, so fp32 accumulation is exact.
    # Extents that are multiples of 64 take the one-load-per-stage form of the m- / n-contiguous operands (a ragged last
    # tile of 64 in the second shape, many tiles per CTA in the third); every element is checked bit for bit
    rng = np.random.default_rng(11)
    M, N, K, nb = shape
    a = rng.integers(0, 256, (nb, M, K)).astype(np.float32)
    b = rng.integers(-127, 128, (nb, N, K)).astype(np.float32)
    ad = torch.from_numpy(_layout(a, a_mn)).to(DEV).to(torch.bfloat16)
    bd = torch.from_numpy(_layout(b, b_mn)).to(DEV).to(torch.bfloat16)
    out = torch.zeros(nb, M, N, dtype=torch.float32, device=DEV)
    st = _status()
    B.mrem_gemm(B.BF16, ad, a_mn, M if a_mn else K, M * K, bd, b_mn, N if b_mn else K, N * K, M, N, K, nb, 1.0, out,
                N, M * N, 0, st, _stream())
    torch.cuda.synchronize()
    ref = np.stack([O.int_matmul(a[i].astype(np.int64), b[i].astype(np.int64)) for i in range(nb)])
    assert np.array_equal(out.cpu().numpy().astype(np.int64), ref)
