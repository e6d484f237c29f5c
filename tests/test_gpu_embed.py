"""Embedding step of the first module (quantized word-embedding table, MSE on the embedding output) through the
C-ABI against the CPU oracle.  Tolerances as for the module: outputs 1e-3 relative L2 (bf16 storage emulated by the
oracle) / 1e-4 (float32), loss and gradients 2e-2 relative L2; the codes of the re-quantized table bit for bit."""
import numpy as np
import pytest
import torch

from oracle import mrem_oracle as O
from paper_2109_15082_b200 import binding as B
from paper_2109_15082_b200 import synth
from paper_2109_15082_b200.embedding import EmbeddingStep
from tests.gpu_util import rel

pytestmark = pytest.mark.gpu


def _problem(act_dtype, e_bits, V=500, H=128, P=48, batch=5, seq=40, seed=3):
    teacher = dict(word=synth.normal(seed, "emb_word", (V, H), 0.05), pos=synth.normal(seed, "emb_pos", (P, H), 0.02),
                   type=synth.normal(seed, "emb_type", (2, H), 0.02), ln_g=1 + synth.normal(seed, "emb_g", (H,), 0.1),
                   ln_b=synth.normal(seed, "emb_b", (H,), 0.05))
    teacher = {k: v.astype(np.float32) for k, v in teacher.items()}
    student = {k: (v + synth.normal(seed + 1, "emb_noise" + k, v.shape, 0.004)).astype(np.float32) for k, v in teacher.items()}
    rng = np.random.default_rng(seed)
    ids = rng.zipf(1.3, (batch, seq)) % V                               # a few very frequent rows, many rows unused
    ids[0, :4] = 7
    lens = rng.integers(seq // 2, seq + 1, batch)
    tt = (np.arange(seq)[None, :] >= (lens // 2)[:, None]).astype(np.int32)
    step = (0.7 * np.abs(student["word"]).max(1) / O.sym_qmax(e_bits)).astype(np.float32)   # the largest values clip
    e = EmbeddingStep(teacher, e_bits, batch * seq, act_dtype)
    e.set_student(student, step)
    desc = O.ModuleDesc(1, H, 2, 4 * H, act_dtype=act_dtype)
    return e, desc, teacher, student, step, ids.astype(np.int32), tt


# the last case has the sizes of BERT-large's embedding layers and of the benchmark batch (32 x 128 tokens)
@pytest.mark.parametrize("act_dtype,e_bits,sizes", [("bf16", 4, {}), ("bf16", 2, {}), ("f32", 8, {}),
                                                    ("bf16", 4, dict(V=30522, H=1024, P=512, batch=32, seq=128))])
def test_embedding_step_matches_the_oracle(act_dtype, e_bits, sizes):
    e, desc, teacher, student, step, ids, tt = _problem(act_dtype, e_bits, **sizes)
    dev = e.device
    d_ids, d_tt = torch.from_numpy(ids).to(dev), torch.from_numpy(tt).to(dev)
    batch, seq = ids.shape
    fwd_tol = 1e-3 if act_dtype == "bf16" else 1e-4
    r = O.embed_loss_backward(desc, teacher, student, step, e_bits, ids, tt)

    # loss, outputs and gradients (no update)
    loss = float(e.step(d_ids, d_tt, None)[0])
    torch.cuda.synchronize()
    assert int(e.status[0]) == 0
    e_t, e_s = (t.float().cpu().numpy() for t in e.outputs(batch, seq))
    assert rel(e_t, r["e_t"]) < fwd_tol and rel(e_s, r["e_s"]) < fwd_tol
    assert abs(loss - r["loss"]) / r["loss"] < 2e-2
    g = {k: v.cpu().numpy() for k, v in e.g.items()}
    for k in ("word", "pos", "type", "ln_g", "ln_b", "word_step"):
        assert rel(g[k], r["grads"][k]) < 2e-2, (k, rel(g[k], r["grads"][k]))
    used = np.zeros(e.V, bool)
    used[ids.reshape(-1)] = True
    assert not np.any(g["word"][~used]) and used.sum() < e.V            # rows nobody gathered: exactly zero
    assert np.array_equal(g["pos"][seq:], np.zeros_like(g["pos"][seq:]))

    # same call again: the same bits (token-order sums, no atomics)
    loss_b = float(e.step(d_ids, d_tt, None)[0])
    assert loss_b == loss and np.array_equal(e.g["word"].cpu().numpy(), g["word"])

    # one update: AdamW of the oracle fed with the gradients just read; then the loss on the same batch went down
    opt = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    assert float(e.step(d_ids, d_tt, B.make_optim(step=1, **opt))[0]) == loss
    torch.cuda.synchronize()

    def expect(p0, grad, wd, clamp=None):
        z = np.zeros_like(np.asarray(p0, np.float64))
        p1, _, _ = O.adamw_update(np.asarray(p0, np.float64), np.asarray(grad, np.float64), z, z, 1, opt["lr"], 0.9, 0.999, 1e-8, wd)
        return np.maximum(p1, clamp) if clamp is not None else p1

    tol = dict(rtol=1e-5, atol=2e-3 * opt["lr"])
    after = {k: v.cpu().numpy() for k, v in e.s.items()}
    for k in ("word", "pos", "type"):
        assert np.allclose(after[k], expect(student[k], g[k], 0.01), **tol), k
    for k in ("ln_g", "ln_b"):
        assert np.allclose(after[k], expect(student[k], g[k], 0.0), **tol), k
    step1 = e.word_step.cpu().numpy()
    assert np.allclose(step1, expect(step, g["word_step"], 0.0, O.MIN_STEP), **tol)
    loss_after = float(e.step(d_ids, d_tt, None)[0])
    assert loss_after < loss
    # the update re-quantized the table: the student output of the next call equals the oracle's on the updated tables
    r2 = O.embed_loss_backward(desc, teacher, after, step1, e_bits, ids, tt)
    assert rel(e.outputs(batch, seq)[1].float().cpu().numpy(), r2["e_s"]) < fwd_tol
    assert abs(loss_after - r2["loss"]) / r2["loss"] < 2e-2


def test_embedding_step_rejects_and_reports_bad_input():
    e, desc, teacher, student, step, ids, tt = _problem("bf16", 4, V=64, H=32, P=16, batch=2, seq=8)
    d_ids, d_tt = torch.from_numpy(ids).to(e.device), torch.from_numpy(tt).to(e.device)
    with pytest.raises(B.MremError):                                    # longer than the position table
        long_ids = torch.zeros(1, 17, dtype=torch.int32, device=e.device)
        B.mrem_embed_step(e.desc, e.tensors, e.ws_ptr, e.ws_bytes, long_ids, None, 1, 17, 1, e.e_teacher, e.e_student, None, None, e.loss,
                          e.status, e.stream.cuda_stream)
    with pytest.raises(B.MremError):                                    # workspace too small
        B.mrem_embed_step(e.desc, e.tensors, e.ws_ptr, 1024, d_ids, d_tt, 2, 8, 1, e.e_teacher, e.e_student, None, None, e.loss, e.status,
                          e.stream.cuda_stream)
    bad = d_ids.clone()
    bad[1, 3] = 64                                                      # one index past the table: clamped, reported
    e.step(bad, d_tt, None)
    torch.cuda.synchronize()
    assert int(e.status[0]) == 5


def test_first_module_hands_its_input_gradient_to_the_embedding_step():
    """The model's first module: the embedding output is the module's input, and the gradient the layers send back to it
    (mrem_get_input_grad) joins the gradient of the embedding MSE.  The module's input gradient against the oracle's;
    the embedding gradients with that extra gradient against the oracle's with the same one."""
    from tests.gpu_util import Problem
    wl = synth.shrink(synth.workloads()["base3_w4a8"], n_layers=2, hidden=128, n_heads=2, ffn=256, seq=40, batch=5, len_lo=10, len_hi=40)
    p = Problem(wl, step_shrink=0.8, student_noise=0.002)
    try:
        p.run_gpu()
        torch.cuda.synchronize()
        d_in = p.m.input_grad(wl.batch, wl.seq)
        r = O.forward_loss_backward(p.desc, p.teacher, p.student, p.oracle_steps(), p.x, p.x, p.vl)
        assert rel(d_in.float().cpu().numpy(), r["d_input"]) < 2e-2
        e, desc, teacher, student, step, ids, tt = _problem("bf16", 4, H=128, batch=wl.batch, seq=wl.seq)
        d_ids, d_tt = torch.from_numpy(ids).to(e.device), torch.from_numpy(tt).to(e.device)
        extra = (d_in.float() * 20).to(torch.bfloat16).contiguous()      # of the size of the MSE's own gradient
        e.step(d_ids, d_tt, None, extra_grad=extra)
        torch.cuda.synchronize()
        re = O.embed_loss_backward(desc, teacher, student, step, 4, ids, tt, d_extra=extra.float().cpu().numpy())
        plain = O.embed_loss_backward(desc, teacher, student, step, 4, ids, tt)
        for k in ("word", "pos", "type", "ln_g", "ln_b", "word_step"):
            got = e.g[k].cpu().numpy()
            assert rel(got, re["grads"][k]) < 2e-2, (k, rel(got, re["grads"][k]))
            assert rel(got, plain["grads"][k]) > 0.1, k                  # the extra gradient is not a rounding-level term
    finally:
        p.close()
