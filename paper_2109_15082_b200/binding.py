"""ctypes binding of libmrem.so: same names as include/mrem.h, argument marshalling only.

Pointers are passed as integers (torch `tensor.data_ptr()`, `stream.cuda_stream`) or
ctypes pointers.  Every wrapper raises MremError on a negative status.  There is no CPU
fallback: importing this module without the built library, or calling a compute entry
point without a CUDA device, fails loudly.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmrem.so")

# ids of include/mrem.h
TEACHER, STUDENT = 0, 1
F32, BF16 = 0, 1
WQKV, BQKV, WO, BO, LN1_G, LN1_B, W1, B1, W2, B2, LN2_G, LN2_B = range(12)
PARAM_NAMES = ("Wqkv", "bqkv", "Wo", "bo", "ln1_g", "ln1_b", "W1", "b1", "W2", "b2", "ln2_g", "ln2_b")
Q_WQKV, Q_WO, Q_W1, Q_W2, Q_X, Q_Q, Q_K, Q_V, Q_P, Q_C, Q_A, Q_G = range(12)
GRAD_STEP, GRAD_OFFSET = 100, 200
TRAIN_ALL = 31
ERRORS = {0: "OK", -1: "ARG", -2: "ALIGN", -3: "SHAPE", -4: "WORKSPACE", -5: "ORDER", -6: "CUDA",
          -7: "TIMEOUT", -8: "NONFINITE", -9: "UNSUPPORTED"}

EXPORTS = (
    "mrem_workspace_bytes", "mrem_create", "mrem_destroy", "mrem_last_error", "mrem_bind_param", "mrem_bind_steps",
    "mrem_init_student_from_teacher", "mrem_init_weight_steps", "mrem_init_act_steps", "mrem_quantize_weights",
    "mrem_get_weight_codes", "mrem_module_forward", "mrem_recon_loss", "mrem_module_backward", "mrem_get_grad",
    "mrem_step", "mrem_recon_step_host", "mrem_poll_status", "mrem_state_bytes", "mrem_export_state",
    "mrem_import_state", "mrem_graph_capture_step", "mrem_graph_launch", "mrem_gather_rows", "mrem_quantize_act",
    "mrem_quantize_weight", "mrem_gemm_i8", "mrem_gemm", "mrem_graph_num_kernels", "mrem_trace_enable",
    "mrem_trace_read", "mrem_invalidate_weight_codes", "mrem_recon_loss_noalloc", "mrem_set_programmatic_launch",
    "mrem_set_fused_attention_backward", "mrem_backward_and_step", "mrem_recon_step_host_submit",
    "mrem_recon_step_host_wait", "mrem_rem_step", "mrem_bind_head", "mrem_embed_workspace_bytes", "mrem_embed_step", "mrem_get_input_grad",
    "mrem_get_activation", "mrem_set_wait_limit_ns", "mrem_selftest_wait_limit",
    "mrem_set_loss_share", "mrem_grad_bucket", "mrem_set_two_streams",
)


class MremError(RuntimeError):
    def __init__(self, code, where, text=""):
        self.code = code
        super().__init__(f"{where}: MREM_ERR_{ERRORS.get(code, code)} {text}".strip())


class ModuleDesc(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("n_layers", C.c_int32), ("hidden", C.c_int32), ("n_heads", C.c_int32),
                ("ffn", C.c_int32), ("max_seq", C.c_int32), ("max_batch", C.c_int32), ("w_bits", C.c_int32),
                ("a_bits", C.c_int32), ("w_grid", C.c_int32), ("w_step_per_row", C.c_int32),
                ("act_asym_sites", C.c_int32), ("act_dtype", C.c_int32), ("loss_mean", C.c_int32),
                ("trainable_mask", C.c_int32), ("ln_eps", C.c_float)]


class Optim(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("weight_decay", C.c_float), ("step", C.c_int32), ("decay_total_steps", C.c_int32)]


def make_desc(n_layers, hidden, n_heads, ffn, max_seq, max_batch, w_bits=4, a_bits=8, w_grid=0, w_step_per_row=1,
              act_asym_sites=3, act_dtype=BF16, loss_mean=1, trainable_mask=TRAIN_ALL, ln_eps=1e-12):
    return ModuleDesc(C.sizeof(ModuleDesc), n_layers, hidden, n_heads, ffn, max_seq, max_batch, w_bits, a_bits, w_grid,
                      w_step_per_row, act_asym_sites, act_dtype, loss_mean, trainable_mask, ln_eps)


def make_optim(lr=1e-4, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01, step=0, decay_total_steps=0):
    return Optim(lr, beta1, beta2, eps, weight_decay, step, decay_total_steps)


_lib = None


def lib():
    """The loaded library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2109_15082_b200.build` "
                               "(or __graft_entry__.build()); there is no fallback path")
        _lib = C.CDLL(LIB_PATH)
        _lib.mrem_last_error.restype = C.c_char_p
        _lib.mrem_last_error.argtypes = [C.c_void_p]
        for name in EXPORTS:
            if name != "mrem_last_error":
                getattr(_lib, name).restype = C.c_int32
    return _lib


def _p(x):
    """A device/host address as c_void_p (None -> NULL)."""
    if x is None:
        return C.c_void_p(0)
    if isinstance(x, int):
        return C.c_void_p(x)
    if hasattr(x, "data_ptr"):
        return C.c_void_p(x.data_ptr())
    return x


def _check(rc, where, ctx=None):
    if rc < 0:
        text = lib().mrem_last_error(ctx).decode() if ctx is not None else lib().mrem_last_error(None).decode()
        raise MremError(rc, where, text)
    return rc


def mrem_workspace_bytes(desc) -> int:
    out = C.c_size_t(0)
    _check(lib().mrem_workspace_bytes(C.byref(desc), C.byref(out)), "mrem_workspace_bytes")
    return out.value


def mrem_create(desc, workspace, workspace_bytes, stream):
    ctx = C.c_void_p(0)
    _check(lib().mrem_create(C.byref(desc), _p(workspace), C.c_size_t(workspace_bytes), _p(stream), C.byref(ctx)),
           "mrem_create")
    return ctx


def mrem_destroy(ctx):
    _check(lib().mrem_destroy(ctx), "mrem_destroy")


def mrem_bind_param(ctx, role, layer, tensor_id, ptr, dtype):
    _check(lib().mrem_bind_param(ctx, role, layer, tensor_id, _p(ptr), dtype), "mrem_bind_param", ctx)


def mrem_bind_steps(ctx, layer, quantizer_id, steps, offset=None):
    _check(lib().mrem_bind_steps(ctx, layer, quantizer_id, _p(steps), _p(offset)), "mrem_bind_steps", ctx)


def mrem_init_student_from_teacher(ctx):
    _check(lib().mrem_init_student_from_teacher(ctx), "mrem_init_student_from_teacher", ctx)


def mrem_init_weight_steps(ctx, rule):
    _check(lib().mrem_init_weight_steps(ctx, rule), "mrem_init_weight_steps", ctx)


def mrem_init_act_steps(ctx, x, valid_len, batch, seq):
    _check(lib().mrem_init_act_steps(ctx, _p(x), _p(valid_len), batch, seq), "mrem_init_act_steps", ctx)


def mrem_set_programmatic_launch(on):
    _check(lib().mrem_set_programmatic_launch(int(on)), "mrem_set_programmatic_launch")


def mrem_set_fused_attention_backward(ctx, on):
    _check(lib().mrem_set_fused_attention_backward(ctx, int(on)), "mrem_set_fused_attention_backward", ctx)


def mrem_invalidate_weight_codes(ctx):
    _check(lib().mrem_invalidate_weight_codes(ctx), "mrem_invalidate_weight_codes", ctx)


def mrem_quantize_weights(ctx):
    _check(lib().mrem_quantize_weights(ctx), "mrem_quantize_weights", ctx)


def mrem_get_weight_codes(ctx, layer, tensor_id):
    codes, rowsum = C.c_void_p(0), C.c_void_p(0)
    _check(lib().mrem_get_weight_codes(ctx, layer, tensor_id, C.byref(codes), C.byref(rowsum)),
           "mrem_get_weight_codes", ctx)
    return codes.value, rowsum.value


def mrem_module_forward(ctx, role, x, x_other, lam, valid_len, batch, seq, layer_outputs):
    _check(lib().mrem_module_forward(ctx, role, _p(x), _p(x_other), C.c_float(lam), _p(valid_len), batch, seq,
                                     _p(layer_outputs)), "mrem_module_forward", ctx)


def mrem_recon_loss(ctx, loss_total, loss_per_layer=None):
    _check(lib().mrem_recon_loss(ctx, _p(loss_total), _p(loss_per_layer)), "mrem_recon_loss", ctx)


def mrem_module_backward(ctx):
    _check(lib().mrem_module_backward(ctx), "mrem_module_backward", ctx)


def mrem_get_grad(ctx, layer, grad_id) -> int:
    g = C.c_void_p(0)
    _check(lib().mrem_get_grad(ctx, layer, grad_id, C.byref(g)), "mrem_get_grad", ctx)
    return g.value


def mrem_step(ctx, optim):
    _check(lib().mrem_step(ctx, C.byref(optim)), "mrem_step", ctx)


def mrem_backward_and_step(ctx, optim):
    _check(lib().mrem_backward_and_step(ctx, C.byref(optim)), "mrem_backward_and_step", ctx)


class EmbedDesc(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("vocab", C.c_int32), ("hidden", C.c_int32), ("max_pos", C.c_int32),
                ("n_types", C.c_int32), ("e_bits", C.c_int32), ("act_dtype", C.c_int32), ("loss_mean", C.c_int32),
                ("ln_eps", C.c_float)]


EMBED_TENSOR_FIELDS = ("t_word", "t_pos", "t_type", "t_ln_g", "t_ln_b", "word", "pos", "type", "ln_g", "ln_b", "word_step",
                       "g_word", "g_pos", "g_type", "g_ln_g", "g_ln_b", "g_word_step", "m_word", "v_word", "m_pos", "v_pos",
                       "m_type", "v_type", "m_ln_g", "v_ln_g", "m_ln_b", "v_ln_b", "m_word_step", "v_word_step", "d_step_counter")


class EmbedTensors(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in EMBED_TENSOR_FIELDS]


def make_embed_desc(vocab, hidden, max_pos, n_types, e_bits, act_dtype=BF16, loss_mean=1, ln_eps=1e-12):
    return EmbedDesc(C.sizeof(EmbedDesc), vocab, hidden, max_pos, n_types, e_bits, act_dtype, loss_mean, ln_eps)


def mrem_embed_workspace_bytes(desc, max_tokens) -> int:
    out = C.c_size_t(0)
    _check(lib().mrem_embed_workspace_bytes(C.byref(desc), int(max_tokens), C.byref(out)), "mrem_embed_workspace_bytes")
    return out.value


def mrem_get_input_grad(ctx) -> int:
    out = C.c_void_p(0)
    _check(lib().mrem_get_input_grad(ctx, C.byref(out)), "mrem_get_input_grad", ctx)
    return out.value


def mrem_set_loss_share(ctx, share):
    _check(lib().mrem_set_loss_share(ctx, C.c_float(float(share))), "mrem_set_loss_share", ctx)


def mrem_grad_bucket(ctx, layer):
    """(device address, float32 count) of the range that holds every gradient of `layer`."""
    ptr, n = C.c_void_p(0), C.c_size_t(0)
    _check(lib().mrem_grad_bucket(ctx, int(layer), C.byref(ptr), C.byref(n)), "mrem_grad_bucket", ctx)
    return ptr.value, n.value


def mrem_set_two_streams(ctx, on):
    _check(lib().mrem_set_two_streams(ctx, int(bool(on))), "mrem_set_two_streams", ctx)


def mrem_set_wait_limit_ns(ns):
    _check(lib().mrem_set_wait_limit_ns(C.c_uint64(int(ns))), "mrem_set_wait_limit_ns")


def mrem_selftest_wait_limit(ctx):
    _check(lib().mrem_selftest_wait_limit(ctx), "mrem_selftest_wait_limit", ctx)


ACT_QKV, ACT_P, ACT_CTX, ACT_Y1, ACT_A, ACT_G, ACT_Y2 = range(7)


def mrem_get_activation(ctx, role, layer, which) -> int:
    out = C.c_void_p(0)
    _check(lib().mrem_get_activation(ctx, int(role), int(layer), int(which), C.byref(out)), "mrem_get_activation", ctx)
    return out.value


def mrem_embed_step(desc, tensors, workspace, workspace_bytes, d_ids, d_type_ids, batch, seq, requantize, d_e_teacher,
                    d_e_student, d_extra_grad, optim, d_loss, d_status, stream):
    _check(lib().mrem_embed_step(C.byref(desc), C.byref(tensors), _p(workspace), C.c_size_t(workspace_bytes), _p(d_ids),
                                 _p(d_type_ids), int(batch), int(seq), int(requantize), _p(d_e_teacher), _p(d_e_student),
                                 _p(d_extra_grad), C.byref(optim) if optim is not None else None, _p(d_loss), _p(d_status), _p(stream)),
           "mrem_embed_step")


def mrem_bind_head(ctx, d_wp, d_bp, d_wc, d_bc, n_classes, d_logit_loss=None, d_logits=None):
    _check(lib().mrem_bind_head(ctx, _p(d_wp), _p(d_bp), _p(d_wc), _p(d_bc), int(n_classes), _p(d_logit_loss), _p(d_logits)),
           "mrem_bind_head", ctx)


def mrem_rem_step(ctx, layer, tensor_id, d_a, rows, optim, d_loss):
    _check(lib().mrem_rem_step(ctx, int(layer), int(tensor_id), _p(d_a), int(rows), C.byref(optim) if optim is not None else None, _p(d_loss)),
           "mrem_rem_step", ctx)


def mrem_recon_step_host(ctx, h_x_teacher, h_x_student, h_valid_len, batch, seq, lam, optim) -> float:
    loss = C.c_float(0)
    _check(lib().mrem_recon_step_host(ctx, _p(h_x_teacher), _p(h_x_student), _p(h_valid_len), batch, seq,
                                      C.c_float(lam), C.byref(optim), C.byref(loss)), "mrem_recon_step_host", ctx)
    return loss.value


def mrem_recon_step_host_submit(ctx, h_x_teacher, h_x_student, h_valid_len, batch, seq, lam, optim):
    _check(lib().mrem_recon_step_host_submit(ctx, _p(h_x_teacher), _p(h_x_student), _p(h_valid_len), batch, seq,
                                             C.c_float(lam), C.byref(optim)), "mrem_recon_step_host_submit", ctx)


def mrem_recon_step_host_wait(ctx) -> float:
    loss = C.c_float(0)
    _check(lib().mrem_recon_step_host_wait(ctx, C.byref(loss)), "mrem_recon_step_host_wait", ctx)
    return loss.value


def mrem_poll_status(ctx) -> int:
    st = C.c_int32(0)
    _check(lib().mrem_poll_status(ctx, C.byref(st)), "mrem_poll_status", ctx)
    return st.value


def mrem_state_bytes(ctx) -> int:
    out = C.c_size_t(0)
    _check(lib().mrem_state_bytes(ctx, C.byref(out)), "mrem_state_bytes", ctx)
    return out.value


def mrem_export_state(ctx, blob, nbytes):
    _check(lib().mrem_export_state(ctx, _p(blob), C.c_size_t(nbytes)), "mrem_export_state", ctx)


def mrem_import_state(ctx, blob, nbytes):
    _check(lib().mrem_import_state(ctx, _p(blob), C.c_size_t(nbytes)), "mrem_import_state", ctx)


def mrem_graph_capture_step(ctx, x_teacher, x_student, lam, valid_len, batch, seq, teacher_outputs, student_outputs,
                            loss_total, optim):
    _check(lib().mrem_graph_capture_step(ctx, _p(x_teacher), _p(x_student), C.c_float(lam), _p(valid_len), batch, seq,
                                         _p(teacher_outputs), _p(student_outputs), _p(loss_total), C.byref(optim)),
           "mrem_graph_capture_step", ctx)


def mrem_graph_launch(ctx):
    _check(lib().mrem_graph_launch(ctx), "mrem_graph_launch", ctx)


def mrem_graph_num_kernels(ctx) -> int:
    n = C.c_int32(0)
    _check(lib().mrem_graph_num_kernels(ctx, C.byref(n)), "mrem_graph_num_kernels", ctx)
    return n.value


class TraceEntry(C.Structure):
    _fields_ = [("name", C.c_char * 40), ("ms", C.c_double), ("work", C.c_double), ("launches", C.c_int64),
                ("is_flops", C.c_int32), ("reserved", C.c_int32)]


def mrem_trace_enable(ctx, on):
    _check(lib().mrem_trace_enable(ctx, int(on)), "mrem_trace_enable", ctx)


def mrem_trace_read(ctx, max_entries=64):
    """-> list of dicts name, ms, work, launches, is_flops."""
    buf = (TraceEntry * max_entries)()
    n = C.c_int32(0)
    _check(lib().mrem_trace_read(ctx, buf, max_entries, C.byref(n)), "mrem_trace_read", ctx)
    return [dict(name=buf[i].name.decode(), ms=buf[i].ms, work=buf[i].work, launches=buf[i].launches,
                 is_flops=bool(buf[i].is_flops)) for i in range(n.value)]


def mrem_gather_rows(src, idx, n_rows, row_bytes, out, stream):
    _check(lib().mrem_gather_rows(_p(src), _p(idx), n_rows, C.c_size_t(row_bytes), _p(out), _p(stream)),
           "mrem_gather_rows")


def mrem_quantize_act(x, dtype, n, step, offset, lo, hi, codes8, codes_t, stream):
    _check(lib().mrem_quantize_act(_p(x), dtype, C.c_int64(n), _p(step), _p(offset), lo, hi, _p(codes8), _p(codes_t),
                                   _p(stream)), "mrem_quantize_act")


def mrem_quantize_weight(w, rows, cols, steps, per_row, bits, grid, codes, rowsum, scale, what, dtype, stream):
    _check(lib().mrem_quantize_weight(_p(w), rows, cols, _p(steps), per_row, bits, grid, _p(codes), _p(rowsum),
                                      _p(scale), _p(what), dtype, _p(stream)), "mrem_quantize_weight")


def mrem_gemm_i8(a, a_unsigned, b, M, N, K, acc, block_n, status, stream):
    _check(lib().mrem_gemm_i8(_p(a), a_unsigned, _p(b), M, N, K, _p(acc), block_n, _p(status), _p(stream)),
           "mrem_gemm_i8")


def mrem_gemm(dtype, a, a_mn, lda, a_bs, b, b_mn, ldb, b_bs, M, N, K, batches, alpha, out, ldc, c_bs, block_n, status,
              stream):
    _check(lib().mrem_gemm(dtype, _p(a), a_mn, C.c_int64(lda), C.c_int64(a_bs), _p(b), b_mn, C.c_int64(ldb),
                           C.c_int64(b_bs), M, N, K, batches, C.c_float(alpha), _p(out), C.c_int64(ldc),
                           C.c_int64(c_bs), block_n, _p(status), _p(stream)), "mrem_gemm")


NOALLOC_MAX_LAYERS = 32


def mrem_recon_loss_noalloc(f_student, f_teacher, dtype, n_layers, n_per_layer, loss_mean, grad, loss_total,
                            loss_per_layer, stream):
    """Loss of Eq. 3 and its gradient for callers that cannot allocate device memory: no context, no
    workspace; the reduction scratch is a fixed array inside the library (see include/mrem.h)."""
    _check(lib().mrem_recon_loss_noalloc(_p(f_student), _p(f_teacher), dtype, n_layers, C.c_int64(n_per_layer),
                                         int(loss_mean), _p(grad), _p(loss_total), _p(loss_per_layer), _p(stream)),
           "mrem_recon_loss_noalloc")
