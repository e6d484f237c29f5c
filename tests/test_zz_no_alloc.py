"""The allocation-free loss entry point against the regular one.

mrem_recon_loss_noalloc serves callers that cannot allocate device memory (a plug-in living on
memory the host application hands out, a hook that runs under the application's allocator lock,
a loop in which cudaMalloc's device-wide synchronisation is not allowed).  It must give what
mrem_recon_loss gives for the same layer outputs; the only difference is where the partial sums
of the reduction live.  Two calls in a row check that nothing left in the built-in scratch by
one call disturbs the next.  This file sorts last on purpose: a run that stops at the first
failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

from paper_2109_15082_b200 import binding as B
from paper_2109_15082_b200 import synth
from tests.gpu_util import Problem

pytestmark = pytest.mark.gpu


def _workload(act_dtype):
    base = synth.workloads()["base3_w4a8"]
    return synth.shrink(base, n_layers=2, hidden=128, n_heads=2, ffn=256, seq=40, batch=3, len_lo=10, len_hi=40,
                        act_dtype=act_dtype)


@pytest.mark.parametrize("act_dtype,loss_mean", [("bf16", True), ("f32", False)])
def test_noalloc_loss_matches_context_loss_twice(act_dtype, loss_mean):
    wl = _workload(act_dtype)
    p = Problem(wl, step_shrink=0.8, student_noise=0.002, loss_mean=loss_mean)
    try:
        m = p.m
        n_per_layer = wl.batch * wl.seq * wl.hidden
        grad = torch.zeros(wl.n_layers * n_per_layer, dtype=m.tdtype, device=m.device)
        total = torch.zeros(64, dtype=torch.float32, device=m.device)
        per = torch.zeros(64, dtype=torch.float32, device=m.device)
        stream = torch.cuda.current_stream().cuda_stream
        for call in range(2):
            if call == 1:                                   # a different problem for the second call
                p.xd.mul_(0.5)
            m.quantize_weights()
            m.forward_teacher(p.xd, p.vld, wl.batch, wl.seq)
            m.forward_student(p.xd, p.vld, wl.batch, wl.seq)
            ref_total, ref_per = m.recon_loss()
            total.fill_(-1.0)
            per.fill_(-1.0)
            B.mrem_recon_loss_noalloc(m.s_out, m.t_out, m.dt, wl.n_layers, n_per_layer, loss_mean, grad, total, per,
                                      stream)
            torch.cuda.synchronize()
            # same kernels, same reduction order: the tolerance of the other loss tests (2e-2) is far from needed
            assert np.allclose(total[:1].cpu().numpy(), ref_total.cpu().numpy(), rtol=2e-2)
            assert np.allclose(per[: wl.n_layers].cpu().numpy(), ref_per.cpu().numpy(), rtol=2e-2)
            assert float(total[0]) == float(ref_total[0])
            # gradient 2c(f_hat - f) against the definition, on the stored outputs
            fs = m.s_out[: wl.n_layers * n_per_layer].float()
            ft = m.t_out[: wl.n_layers * n_per_layer].float()
            c = 1.0 / n_per_layer if loss_mean else 1.0
            want = 2.0 * c * (fs - ft)
            got = grad.float()
            assert torch.allclose(got, want, rtol=1e-2, atol=1e-2 * float(want.abs().max()))
        assert float(total[0]) > 0
    finally:
        p.close()


def test_noalloc_loss_rejects_what_it_cannot_hold():
    dev = "cuda:0"
    x = torch.zeros(1024, dtype=torch.float32, device=dev)
    out = torch.zeros(64, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream().cuda_stream
    with pytest.raises(B.MremError) as e:                    # more layers than the built-in scratch covers
        B.mrem_recon_loss_noalloc(x, x, B.F32, B.NOALLOC_MAX_LAYERS + 1, 16, 1, x, out, None, stream)
    assert e.value.code == -3
    with pytest.raises(B.MremError) as e:
        B.mrem_recon_loss_noalloc(None, x, B.F32, 1, 16, 1, x, out, None, stream)
    assert e.value.code == -1
    with pytest.raises(B.MremError) as e:
        B.mrem_recon_loss_noalloc(x, x, 7, 1, 16, 1, x, out, None, stream)
    assert e.value.code == -1
