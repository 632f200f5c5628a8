"""paper_2609_17380_b200: bit-exact, replayable transformer training-step arithmetic on B200.

Thin ctypes binding of libdet.so (see include/det.h).  Every function here has the name and the argument
order of its C-ABI entry point and only marshals arguments: torch tensors (CUDA, contiguous) are passed as
device pointers, the current torch CUDA stream as the stream.  Nothing is computed in Python and there is
no CPU fallback: importing the binding without the built library raises.
"""
import ctypes as C
import os

import torch

_DIR = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_DIR, "libdet.so")

DET_OK = 0
DET_F32, DET_BF16 = 0, 1
DET_DEV_TARGET, DET_DEV_TIMEOUT, DET_DEV_NONFINITE = 1, 2, 4   # bits of a device status word
DEV_TARGET, DEV_TIMEOUT, DEV_NONFINITE = 1, 2, 4
STATUS_NAMES = {0: "DET_OK", -1: "DET_ERR_ARG", -2: "DET_ERR_SHAPE", -3: "DET_ERR_ALIGN", -4: "DET_ERR_WORKSPACE",
                -5: "DET_ERR_RANGE", -6: "DET_ERR_CUDA"}


class DetError(RuntimeError):
    def __init__(self, fn, code):
        super().__init__("%s returned %s (%d)" % (fn, STATUS_NAMES.get(code, "?"), code))
        self.code = code


class det_accum(C.Structure):
    _fields_ = [("accum", C.c_int), ("dp_shard", C.c_int), ("dp_replicate", C.c_int), ("pushes", C.c_int),
                ("nstack", C.c_int), ("level", C.c_int * 34), ("slot", C.c_int * 34),
                ("free_mask", C.c_ulonglong), ("n", C.c_size_t), ("bufs", C.c_void_p), ("inner_slot", C.c_int),
                ("gr_slot", C.c_int)]


class det_adamw_desc(C.Structure):
    _fields_ = [("lr", C.c_double), ("beta1", C.c_double), ("beta2", C.c_double), ("eps", C.c_double),
                ("weight_decay", C.c_double), ("step", C.c_int)]


_lib = None


def load():
    """Load libdet.so; raises if it has not been built (python -m paper_2609_17380_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_SO):
            raise ImportError("libdet.so is missing: build it with `python paper_2609_17380_b200/build.py` "
                              "(there is no fallback path)")
        _lib = C.CDLL(_SO)
        for name in ("det_sum_ws_bytes", "det_grad_norm_ws_bytes", "det_lsq_weight_scale_ws_bytes",
                     "det_lsq_act_scale_init_ws_bytes", "det_lsq_quantize_weight_ws_bytes", "det_linear_bwd_ws_bytes",
                     "det_rmsnorm_bwd_ws_bytes", "det_xent_ws_bytes", "det_attn_bwd_ws_bytes", "det_attn_bwd_fixq_ws_bytes",
                     "det_tensor_hash_ws_bytes", "det_lmhead_fwd_v2_ws_bytes", "det_lmhead_bwd_v2_ws_bytes",
                     "det_attn_fwd_v2_ws_bytes"):
            getattr(_lib, name).restype = C.c_size_t
        _lib.det_launch_count.restype = C.c_ulonglong
    return _lib


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return C.c_void_p(t)
    assert t.is_cuda and t.is_contiguous(), "tensors must be contiguous CUDA tensors"
    return C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(fn, rc):
    if rc != DET_OK:
        raise DetError(fn, rc)


def _ws(ws):
    return (_ptr(ws), C.c_size_t(ws.numel() * ws.element_size())) if ws is not None else (None, C.c_size_t(0))


# ---- information / primitives ------------------------------------------------------------------------
def det_device_sm_count():
    return load().det_device_sm_count()


def det_launch_count():
    return load().det_launch_count()


def det_test_prim(op, a, b, out):
    _check("det_test_prim", load().det_test_prim(C.c_int(op), _ptr(a), _ptr(b), _ptr(out), C.c_size_t(a.numel()), _stream()))


# ---- sums, norm, clip -----------------------------------------------------------------------------------
def det_sum_ws_bytes(n):
    return load().det_sum_ws_bytes(C.c_size_t(n))


def det_sum(x, n, squares, out, ws):
    _check("det_sum", load().det_sum(_ptr(x), C.c_size_t(n), C.c_int(squares), _ptr(out), *_ws(ws), _stream()))


def det_sum_static_max_n():
    lib = load()
    lib.det_sum_static_max_n.restype = C.c_size_t
    return lib.det_sum_static_max_n()


def det_sum_static(x, n, squares, out):
    """det_sum without a workspace argument: scratch lives in a fixed array inside the library (see det.h)."""
    _check("det_sum_static", load().det_sum_static(_ptr(x), C.c_size_t(n), C.c_int(squares), _ptr(out), _stream()))


def _tensor_table(tensors):
    ptrs = (C.c_void_p * len(tensors))(*[t.data_ptr() for t in tensors])
    ns = (C.c_size_t * len(tensors))(*[t.numel() for t in tensors])
    return ptrs, ns


def det_grad_norm_ws_bytes(tensors):
    _, ns = _tensor_table(tensors)
    return load().det_grad_norm_ws_bytes(ns, C.c_int(len(tensors)))


def det_grad_norm(tensors, max_norm, norm_out, coef_out, ws, status_dev=None):
    ptrs, ns = _tensor_table(tensors)
    _check("det_grad_norm", load().det_grad_norm(ptrs, ns, C.c_int(len(tensors)), C.c_float(max_norm), _ptr(norm_out),
                                                 _ptr(coef_out), *_ws(ws), _stream(), _ptr(status_dev)))


def det_scale_inplace(g, n, coef_dev):
    _check("det_scale_inplace", load().det_scale_inplace(_ptr(g), C.c_size_t(n), _ptr(coef_dev), _stream()))


# ---- LSQ int8 linear -------------------------------------------------------------------------------------
def det_lsq_weight_scale_ws_bytes(N, K):
    return load().det_lsq_weight_scale_ws_bytes(C.c_int(N), C.c_int(K))


def det_lsq_weight_scale(W, N, K, per_tensor, s_w, ws):
    _check("det_lsq_weight_scale", load().det_lsq_weight_scale(_ptr(W), C.c_int(N), C.c_int(K), C.c_int(per_tensor),
                                                               _ptr(s_w), *_ws(ws), _stream()))


def det_lsq_act_scale_init_ws_bytes(n):
    return load().det_lsq_act_scale_init_ws_bytes(C.c_size_t(n))


def det_lsq_act_scale_init(X, n, s_x, ws):
    _check("det_lsq_act_scale_init", load().det_lsq_act_scale_init(_ptr(X), C.c_size_t(n), _ptr(s_x), *_ws(ws), _stream()))


def det_lsq_quantize_weight_ws_bytes(N, K):
    return load().det_lsq_quantize_weight_ws_bytes(C.c_int(N), C.c_int(K))


def det_lsq_quantize_weight(W, s_w, N, K, hadamard_block, qW, qWt_bwd, s_u, ws):
    _check("det_lsq_quantize_weight", load().det_lsq_quantize_weight(
        _ptr(W), _ptr(s_w), C.c_int(N), C.c_int(K), C.c_int(hadamard_block), _ptr(qW), _ptr(qWt_bwd), _ptr(s_u), *_ws(ws),
        _stream()))


def det_linear_fwd(X, qW, s_x, s_w, M, N, K, Y, qX_save, status_dev=None):
    _check("det_linear_fwd", load().det_linear_fwd(_ptr(X), _ptr(qW), _ptr(s_x), _ptr(s_w), C.c_int(M), C.c_int(N),
                                                   C.c_int(K), _ptr(Y), _ptr(qX_save), _stream(), _ptr(status_dev)))


def det_linear_fwd_q(qX, qW, s_x, s_w, M, N, K, Y, status_dev=None):
    _check("det_linear_fwd_q", load().det_linear_fwd_q(_ptr(qX), _ptr(qW), _ptr(s_x), _ptr(s_w), C.c_int(M), C.c_int(N),
                                                       C.c_int(K), _ptr(Y), _stream(), _ptr(status_dev)))


def det_linear_bwd_ws_bytes(M, N, K):
    return load().det_linear_bwd_ws_bytes(C.c_int(M), C.c_int(N), C.c_int(K))


def det_linear_bwd(dY, X, qX, W, qWt_bwd, s_x, s_w, s_u, M, N, K, hadamard_block, dX, dW, ds_x, ws, status_dev=None):
    _check("det_linear_bwd", load().det_linear_bwd(
        _ptr(dY), _ptr(X), _ptr(qX), _ptr(W), _ptr(qWt_bwd), _ptr(s_x), _ptr(s_w), _ptr(s_u), C.c_int(M), C.c_int(N),
        C.c_int(K), C.c_int(hadamard_block), _ptr(dX), _ptr(dW), _ptr(ds_x), *_ws(ws), _stream(), _ptr(status_dev)))


def det_test_wait_timeout(status_dev, limit_cycles):
    _check("det_test_wait_timeout", load().det_test_wait_timeout(_ptr(status_dev), C.c_longlong(limit_cycles), _stream()))


def det_test_igemm_tn(A, B, I, J, K, Cout, force_one_cta=0, status_dev=None):
    _check("det_test_igemm_tn", load().det_test_igemm_tn(_ptr(A), _ptr(B), C.c_int(I), C.c_int(J), C.c_int(K), _ptr(Cout),
                                                         C.c_int(force_one_cta), _stream(), _ptr(status_dev)))


# ---- RMSNorm, cross-entropy ---------------------------------------------------------------------------------
def det_rmsnorm_fwd(io, x, gamma, rows, D, eps, y, rstd):
    _check("det_rmsnorm_fwd", load().det_rmsnorm_fwd(C.c_int(io), _ptr(x), _ptr(gamma), C.c_int(rows), C.c_int(D),
                                                     C.c_float(eps), _ptr(y), _ptr(rstd), _stream()))


def det_rmsnorm_fwd_q(x, gamma, rows, D, eps, y, rstd, s_q, qy):
    _check("det_rmsnorm_fwd_q", load().det_rmsnorm_fwd_q(_ptr(x), _ptr(gamma), C.c_int(rows), C.c_int(D), C.c_float(eps),
                                                         _ptr(y), _ptr(rstd), _ptr(s_q), _ptr(qy), _stream()))


def det_headnorm_fwd(x, ld, T, nh, eps, y, ld_y, rstd):
    _check("det_headnorm_fwd", load().det_headnorm_fwd(_ptr(x), C.c_int(ld), C.c_int(T), C.c_int(nh), C.c_float(eps), _ptr(y),
                                                       C.c_int(ld_y), _ptr(rstd), _stream()))


def det_headnorm_bwd(dy, ld_dy, x, ld, rstd, T, nh, dx, ld_dx):
    _check("det_headnorm_bwd", load().det_headnorm_bwd(_ptr(dy), C.c_int(ld_dy), _ptr(x), C.c_int(ld), _ptr(rstd), C.c_int(T),
                                                       C.c_int(nh), _ptr(dx), C.c_int(ld_dx), _stream()))


def det_rope(x, ld, T, nh, S, cos_tab, sin_tab, inverse, y, ld_y):
    _check("det_rope", load().det_rope(_ptr(x), C.c_int(ld), C.c_int(T), C.c_int(nh), C.c_int(S), _ptr(cos_tab), _ptr(sin_tab),
                                       C.c_int(int(inverse)), _ptr(y), C.c_int(ld_y), _stream()))


def det_rmsnorm_bwd_ws_bytes(rows, D):
    return load().det_rmsnorm_bwd_ws_bytes(C.c_int(rows), C.c_int(D))


def det_rmsnorm_bwd(io, dy, x, gamma, rstd, rows, D, dx, dgamma, ws):
    _check("det_rmsnorm_bwd", load().det_rmsnorm_bwd(C.c_int(io), _ptr(dy), _ptr(x), _ptr(gamma), _ptr(rstd), C.c_int(rows),
                                                     C.c_int(D), _ptr(dx), _ptr(dgamma), *_ws(ws), _stream()))


def det_xent_ws_bytes(rows, V):
    return load().det_xent_ws_bytes(C.c_int(rows), C.c_int(V))


def det_xent_fwd(logits, target, rows, V, z_weight, loss_row, lse, loss_mean, z_mean, ws, status_dev=None):
    _check("det_xent_fwd", load().det_xent_fwd(_ptr(logits), _ptr(target), C.c_int(rows), C.c_int(V), C.c_float(z_weight),
                                               _ptr(loss_row), _ptr(lse), _ptr(loss_mean), _ptr(z_mean), *_ws(ws), _stream(),
                                               _ptr(status_dev)))


def det_xent_bwd(logits_inout, target, lse, rows, V, z_weight, scale):
    _check("det_xent_bwd", load().det_xent_bwd(_ptr(logits_inout), _ptr(target), _ptr(lse), C.c_int(rows), C.c_int(V),
                                               C.c_float(z_weight), C.c_float(scale), _stream()))


# ---- attention ------------------------------------------------------------------------------------------------
def det_attn_fwd(q, k, v, ld, B, H, S, out, ld_out, lse, Hkv=None, window=0):
    _check("det_attn_fwd", load().det_attn_fwd(_ptr(q), _ptr(k), _ptr(v), C.c_int(ld), C.c_int(B), C.c_int(H),
                                               C.c_int(H if Hkv is None else Hkv), C.c_int(S), C.c_int(window), _ptr(out),
                                               C.c_int(ld_out), _ptr(lse), _stream()))


def det_attn_fwd_q(q, k, v, ld, B, H, S, out, ld_out, lse, s_q, qout, Hkv=None, window=0):
    _check("det_attn_fwd_q", load().det_attn_fwd_q(_ptr(q), _ptr(k), _ptr(v), C.c_int(ld), C.c_int(B), C.c_int(H),
                                                   C.c_int(H if Hkv is None else Hkv), C.c_int(S), C.c_int(window), _ptr(out),
                                                   C.c_int(ld_out), _ptr(lse), _ptr(s_q), _ptr(qout), _stream()))


def det_attn_fwd_int8pv(q, k, v, ld, B, H, S, out, ld_out, lse, status_dev=None, Hkv=None, window=0):
    _check("det_attn_fwd_int8pv", load().det_attn_fwd_int8pv(_ptr(q), _ptr(k), _ptr(v), C.c_int(ld), C.c_int(B), C.c_int(H),
                                                             C.c_int(H if Hkv is None else Hkv), C.c_int(S), C.c_int(window),
                                                             _ptr(out), C.c_int(ld_out), _ptr(lse), _stream(), _ptr(status_dev)))


def det_attn_bwd_ws_bytes(B, H, S, Hkv=None):
    return load().det_attn_bwd_ws_bytes(C.c_int(B), C.c_int(H), C.c_int(H if Hkv is None else Hkv), C.c_int(S))


def det_attn_bwd(dout, q, k, v, out, lse, ld, ld_out, B, H, S, dq, dk, dv, ld_d, ws, Hkv=None, window=0):
    _check("det_attn_bwd", load().det_attn_bwd(_ptr(dout), _ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(lse), C.c_int(ld),
                                               C.c_int(ld_out), C.c_int(B), C.c_int(H), C.c_int(H if Hkv is None else Hkv),
                                               C.c_int(S), C.c_int(window), _ptr(dq), _ptr(dk), _ptr(dv), C.c_int(ld_d),
                                               *_ws(ws), _stream()))


def det_attn_bwd_fixq_ws_bytes(B, H, S, Hkv=None):
    return load().det_attn_bwd_fixq_ws_bytes(C.c_int(B), C.c_int(H), C.c_int(H if Hkv is None else Hkv), C.c_int(S))


def det_attn_bwd_fixq(dout, q, k, v, out, lse, ld, ld_out, B, H, S, dq, dk, dv, ld_d, ws, Hkv=None, window=0):
    _check("det_attn_bwd_fixq", load().det_attn_bwd_fixq(_ptr(dout), _ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(lse),
                                                         C.c_int(ld), C.c_int(ld_out), C.c_int(B), C.c_int(H),
                                                         C.c_int(H if Hkv is None else Hkv), C.c_int(S), C.c_int(window),
                                                         _ptr(dq), _ptr(dk), _ptr(dv), C.c_int(ld_d), *_ws(ws), _stream()))


# ---- glue --------------------------------------------------------------------------------------------------------
def det_swiglu_fwd(gu, rows, F, h):
    _check("det_swiglu_fwd", load().det_swiglu_fwd(_ptr(gu), C.c_int(rows), C.c_int(F), _ptr(h), _stream()))


def det_swiglu_fwd_q(gu, rows, F, h, s_q, qh):
    _check("det_swiglu_fwd_q", load().det_swiglu_fwd_q(_ptr(gu), C.c_int(rows), C.c_int(F), _ptr(h), _ptr(s_q), _ptr(qh), _stream()))


def det_swiglu_bwd(dh, gu, rows, F, dgu):
    _check("det_swiglu_bwd", load().det_swiglu_bwd(_ptr(dh), _ptr(gu), C.c_int(rows), C.c_int(F), _ptr(dgu), _stream()))


def det_residual_add(a, b, n, y):
    _check("det_residual_add", load().det_residual_add(_ptr(a), _ptr(b), C.c_size_t(n), _ptr(y), _stream()))


def det_embed_fwd(tok, T, E, V, D, y):
    _check("det_embed_fwd", load().det_embed_fwd(_ptr(tok), C.c_int(T), _ptr(E), C.c_int(V), C.c_int(D), _ptr(y), _stream()))


def det_embed_bwd(tok, T, dy, V, D, dE):
    _check("det_embed_bwd", load().det_embed_bwd(_ptr(tok), C.c_int(T), _ptr(dy), C.c_int(V), C.c_int(D), _ptr(dE), _stream()))


def det_lmhead_fwd(H, W, M, V, K, logits):
    _check("det_lmhead_fwd", load().det_lmhead_fwd(_ptr(H), _ptr(W), C.c_int(M), C.c_int(V), C.c_int(K), _ptr(logits), _stream()))


def det_lmhead_fwd_v2_ws_bytes(M, V, K):
    return load().det_lmhead_fwd_v2_ws_bytes(C.c_int(M), C.c_int(V), C.c_int(K))


def det_lmhead_fwd_v2(H, W, M, V, K, logits, ws, status_dev=None):
    _check("det_lmhead_fwd_v2", load().det_lmhead_fwd_v2(_ptr(H), _ptr(W), C.c_int(M), C.c_int(V), C.c_int(K), _ptr(logits),
                                                         *_ws(ws), _stream(), _ptr(status_dev)))


def det_lmhead_bwd_v2_ws_bytes(M, V, K):
    return load().det_lmhead_bwd_v2_ws_bytes(C.c_int(M), C.c_int(V), C.c_int(K))


def det_lmhead_bwd_v2(dlogits, H, W, M, V, K, dH, dW, ws, status_dev=None):
    _check("det_lmhead_bwd_v2", load().det_lmhead_bwd_v2(_ptr(dlogits), _ptr(H), _ptr(W), C.c_int(M), C.c_int(V), C.c_int(K),
                                                         _ptr(dH), _ptr(dW), *_ws(ws), _stream(), _ptr(status_dev)))


def det_attn_fwd_v2_ws_bytes(B, H, S):
    return load().det_attn_fwd_v2_ws_bytes(C.c_int(B), C.c_int(H), C.c_int(S))


def det_attn_fwd_v2(q, k, v, ld, B, H, S, out, ld_out, lse, ws, status_dev=None):
    _check("det_attn_fwd_v2", load().det_attn_fwd_v2(_ptr(q), _ptr(k), _ptr(v), C.c_int(ld), C.c_int(B), C.c_int(H), C.c_int(S),
                                                     _ptr(out), C.c_int(ld_out), _ptr(lse), *_ws(ws), _stream(), _ptr(status_dev)))


def det_lmhead_bwd(dlogits, H, W, M, V, K, dH, dW, first_chunk):
    _check("det_lmhead_bwd", load().det_lmhead_bwd(_ptr(dlogits), _ptr(H), _ptr(W), C.c_int(M), C.c_int(V), C.c_int(K),
                                                   _ptr(dH), _ptr(dW), C.c_int(first_chunk), _stream()))


# ---- gradient accumulation, AdamW, hash ---------------------------------------------------------------------------
def det_grad_accum_nbufs(dp_replicate):
    return load().det_grad_accum_nbufs(C.c_int(dp_replicate))


def det_grad_accum_init(st, accum, dp_shard, dp_replicate, n, bufs):
    _check("det_grad_accum_init", load().det_grad_accum_init(C.byref(st), C.c_int(accum), C.c_int(dp_shard),
                                                             C.c_int(dp_replicate), C.c_size_t(n), _ptr(bufs)))


def det_grad_accum_push(st, g_microbatch):
    _check("det_grad_accum_push", load().det_grad_accum_push(C.byref(st), _ptr(g_microbatch), _stream()))


def det_grad_accum_result(st, g_out):
    _check("det_grad_accum_result", load().det_grad_accum_result(C.byref(st), _ptr(g_out), _stream()))


def det_adamw_step(desc, pdtype, p, g, m, v, n):
    _check("det_adamw_step", load().det_adamw_step(C.byref(desc), C.c_int(pdtype), _ptr(p), _ptr(g), _ptr(m), _ptr(v),
                                                   C.c_size_t(n), _stream()))


def det_tensor_hash_ws_bytes(nbytes):
    return load().det_tensor_hash_ws_bytes(C.c_size_t(nbytes))


def det_tensor_hash_async(p, nbytes, out32_dev, ws):
    """Queues the hash; the 32-byte root lands in out32_dev (device) in stream order, nothing synchronises."""
    _check("det_tensor_hash_async", load().det_tensor_hash_async(_ptr(p), C.c_size_t(nbytes), _ptr(out32_dev), *_ws(ws),
                                                                 _stream()))


def det_tensor_hash(p, nbytes, ws):
    """Returns the 32-byte root as a hex string (synchronises the current stream)."""
    out = (C.c_uint8 * 32)()
    _check("det_tensor_hash", load().det_tensor_hash(_ptr(p), C.c_size_t(nbytes), out, *_ws(ws), _stream()))
    return bytes(out).hex()
