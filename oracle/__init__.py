"""CPU oracle bindings -- TEST INFRASTRUCTURE ONLY.

Loads ``liboracle.so`` (plain C, built by :func:`oracle.build`) and exposes numpy
wrappers.  Only tests, the smoke check and the timed cpu baseline may import this
package; the product path (``paper_2609_17380_b200``) never does.

bf16 tensors are numpy ``uint16`` arrays holding the raw bit patterns.
"""
import ctypes as C
import os
import subprocess

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_DIR, "liboracle.so")
_SRC = [os.path.join(_DIR, "oracle.c"), os.path.join(_DIR, "prim.h")]


def build(force=False):
    """Compile the oracle with contraction disabled and no FMA-capable -march."""
    if not force and os.path.exists(_SO) and all(os.path.getmtime(_SO) >= os.path.getmtime(s) for s in _SRC):
        return _SO
    cmd = ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-msse4.1", "-fopenmp", "-shared", "-fPIC",
           "-o", _SO, _SRC[0], "-lm"]
    subprocess.check_call(cmd)
    return _SO


_lib = None


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(_SO)
        _lib.orc_det_sum.restype = C.c_float
        _lib.orc_sumsq.restype = C.c_float
        _lib.orc_accum_new.restype = C.c_void_p
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


def _c(a, dt):
    a = np.ascontiguousarray(a, dtype=dt)
    return a


# ---- primitives -----------------------------------------------------------
OPS = dict(add=0, sub=1, mul=2, div=3, sqrt=4, exp=5, log=6, max=7, bf16=8, mul_add=9)


def prim(op, a, b=None):
    a = _c(a, np.float32)
    b = _c(b, np.float32) if b is not None else None
    out = np.empty_like(a)
    lib().orc_prim(C.c_int(OPS[op]), _p(a), _p(b), _p(out), C.c_size_t(a.size))
    return out


def det_sum(x):
    x = _c(x, np.float32)
    return np.float32(lib().orc_det_sum(_p(x), C.c_size_t(x.size)))


def sumsq(x):
    x = _c(x, np.float32)
    return np.float32(lib().orc_sumsq(_p(x), C.c_size_t(x.size)))


def f2bf(x):
    x = _c(x, np.float32)
    y = np.empty(x.shape, np.uint16)
    lib().orc_f2bf(_p(x), _p(y), C.c_size_t(x.size))
    return y


def bf2f(h):
    return (np.asarray(h, np.uint16).astype(np.uint32) << 16).view(np.float32)


# ---- LSQ int8 linear ------------------------------------------------------
def lsq_weight_scale(W, per_tensor=False):
    W = _c(W, np.uint16)
    N, K = W.shape
    s = np.empty(N, np.float32)
    lib().orc_lsq_weight_scale(_p(W), C.c_int(N), C.c_int(K), C.c_int(int(per_tensor)), _p(s))
    return s


def lsq_act_scale_init(X):
    X = _c(X, np.uint16)
    s = np.empty(1, np.float32)
    lib().orc_lsq_act_scale_init(_p(X), C.c_size_t(X.size), _p(s))
    return s


def lsq_quantize(X, s, per_row):
    X = _c(X, np.uint16)
    s = _c(s, np.float32)
    q = np.empty(X.shape, np.int8)
    lib().orc_lsq_quantize(_p(X), C.c_int(X.shape[0]), C.c_int(X.shape[1]), _p(s), C.c_int(int(per_row)), _p(q))
    return q


def igemm_tn(A, B):
    A = _c(A, np.int8)
    B = _c(B, np.int8)
    out = np.empty((A.shape[0], B.shape[0]), np.int32)
    lib().orc_igemm_tn(_p(A), _p(B), C.c_int(A.shape[0]), C.c_int(B.shape[0]), C.c_int(A.shape[1]), _p(out))
    return out


def linear_fwd(X, W, s_x, s_w):
    X = _c(X, np.uint16)
    W = _c(W, np.uint16)
    s_x = _c(s_x, np.float32).reshape(1)
    s_w = _c(s_w, np.float32)
    M, K = X.shape
    N = W.shape[0]
    Y = np.empty((M, N), np.uint16)
    qX = np.empty((M, K), np.int8)
    qW = np.empty((N, K), np.int8)
    lib().orc_linear_fwd(_p(X), _p(W), C.c_int(M), C.c_int(N), C.c_int(K), _p(s_x), _p(s_w), _p(Y), _p(qX), _p(qW))
    return Y, qX, qW


def linear_bwd(dY, X, W, s_x, s_w, hb=128, debug=False):
    dY = _c(dY, np.uint16)
    X = _c(X, np.uint16)
    W = _c(W, np.uint16)
    s_x = _c(s_x, np.float32).reshape(1)
    s_w = _c(s_w, np.float32)
    M, K = X.shape
    N = W.shape[0]
    if hb:
        assert hb == 128 and M % 128 == 0 and N % 128 == 0, "rotation blocks of 128 along both contraction dimensions"
    dX = np.empty((M, K), np.uint16)
    dW = np.empty((N, K), np.float32)
    ds = np.empty(1, np.float32)
    dbg = None
    if debug:
        dbg = dict(Aq=np.empty((M, N), np.int8), UqT=np.empty((K, N), np.int8), GqT=np.empty((N, M), np.int8),
                   ZqT=np.empty((K, M), np.int8), scales=np.empty(4, np.float32))
    lib().orc_linear_bwd(_p(dY), _p(X), _p(W), C.c_int(M), C.c_int(N), C.c_int(K), _p(s_x), _p(s_w), C.c_int(hb),
                         _p(dX), _p(dW), _p(ds), *(_p(dbg[k]) if dbg else None for k in
                                                     ("Aq", "UqT", "GqT", "ZqT", "scales")))
    return (dX, dW, ds, dbg) if debug else (dX, dW, ds)


def wht128_f(v):
    v = _c(v, np.float32).copy()
    lib().orc_wht128_f(_p(v))
    return v


def wht128_i(v):
    v = _c(v, np.int32).copy()
    lib().orc_wht128_i(_p(v))
    return v


# ---- norm / loss ----------------------------------------------------------
def _io(a, bf):
    return _c(a, np.uint16 if bf else np.float32) if a is not None else None


def rmsnorm_fwd(x, gamma, eps=1e-6, bf=False):
    x = _io(x, bf)
    gamma = _io(gamma, bf)
    rows, D = x.shape
    y = np.empty_like(x)
    rstd = np.empty(rows, np.float32)
    lib().orc_rmsnorm_fwd(C.c_int(int(bf)), _p(x), _p(gamma), C.c_int(rows), C.c_int(D), C.c_float(eps), _p(y), _p(rstd))
    return y, rstd


def rmsnorm_bwd(dy, x, gamma, rstd, bf=False):
    dy = _io(dy, bf)
    x = _io(x, bf)
    gamma = _io(gamma, bf)
    rstd = _c(rstd, np.float32)
    rows, D = x.shape
    dx = np.empty_like(x)
    dg = np.empty(D, np.float32)
    lib().orc_rmsnorm_bwd(C.c_int(int(bf)), _p(dy), _p(x), _p(gamma), _p(rstd), C.c_int(rows), C.c_int(D), _p(dx), _p(dg))
    return dx, dg


def rope(x, S, cos, sin, inverse=False):
    """x: bf16 bits [T, nh, 128]; cos, sin: f32 [S, 64]; position = t mod S."""
    x = _c(x, np.uint16)
    T, nh, d = x.shape
    assert d == 128
    cos = _c(cos, np.float32)
    sin = _c(sin, np.float32)
    assert cos.shape == (S, 64) and sin.shape == (S, 64)
    y = np.empty_like(x)
    lib().orc_rope(_p(x), C.c_int(T), C.c_int(nh), C.c_int(S), _p(cos), _p(sin), C.c_int(int(inverse)), _p(y))
    return y


def xent_fwd(logits, target, z_weight=0.0):
    logits = _c(logits, np.float32)
    target = _c(target, np.int32)
    rows, V = logits.shape
    loss_row = np.empty(rows, np.float32)
    lse = np.empty(rows, np.float32)
    lm = np.empty(1, np.float32)
    zm = np.empty(1, np.float32)
    lib().orc_xent_fwd.restype = C.c_int
    bad = lib().orc_xent_fwd(_p(logits), _p(target), C.c_int(rows), C.c_int(V), C.c_float(z_weight), _p(loss_row),
                             _p(lse), _p(lm), _p(zm))
    return loss_row, lse, lm, zm, bad


def xent_bwd(logits, target, lse, z_weight=0.0, scale=1.0):
    dz = _c(logits, np.float32).copy()
    target = _c(target, np.int32)
    lse = _c(lse, np.float32)
    rows, V = dz.shape
    lib().orc_xent_bwd(_p(dz), _p(target), _p(lse), C.c_int(rows), C.c_int(V), C.c_float(z_weight), C.c_float(scale))
    return dz


# ---- attention ------------------------------------------------------------
def attn_fwd(qkv, B, H, S, Hkv=None, window=0, int8_pv=False):
    """qkv: uint16 [B*S, (H + 2*Hkv)*128] (q | k | v column blocks).  Returns out [B*S, H*128], lse [B,H,S].
    Hkv < H: grouped-query attention; window > 0: sliding-window attention over the last `window` keys;
    int8_pv: the P.V product of every block of 128 keys in int8 with per-block scales."""
    qkv = _c(qkv, np.uint16)
    Hkv = H if Hkv is None else Hkv
    ld = qkv.shape[1]
    assert ld == (H + 2 * Hkv) * 128 and H % Hkv == 0
    HD, KD = H * 128, Hkv * 128
    out = np.empty((B * S, HD), np.uint16)
    lse = np.empty((B, H, S), np.float32)
    base = qkv.ctypes.data
    fn = lib().orc_attn_fwd_int8pv if int8_pv else lib().orc_attn_fwd
    fn(C.c_void_p(base), C.c_void_p(base + 2 * HD), C.c_void_p(base + 2 * (HD + KD)), C.c_int(ld), C.c_int(B),
       C.c_int(H), C.c_int(Hkv), C.c_int(S), C.c_int(window), _p(out), C.c_int(HD), _p(lse))
    return out, lse


def attn_bwd(dout, qkv, out, lse, B, H, S, Hkv=None, window=0, fixq=False):
    """fixq: the query gradient accumulated over the key blocks in 64-bit fixed point (48 fractional bits)."""
    dout = _c(dout, np.uint16)
    qkv = _c(qkv, np.uint16)
    out = _c(out, np.uint16)
    lse = _c(lse, np.float32)
    Hkv = H if Hkv is None else Hkv
    ld = qkv.shape[1]
    HD, KD = H * 128, Hkv * 128
    dqkv = np.empty_like(qkv)
    base = qkv.ctypes.data
    dbase = dqkv.ctypes.data
    fn = lib().orc_attn_bwd_fixq if fixq else lib().orc_attn_bwd
    fn(_p(dout), C.c_void_p(base), C.c_void_p(base + 2 * HD), C.c_void_p(base + 2 * (HD + KD)), _p(out), _p(lse),
                       C.c_int(ld), C.c_int(HD), C.c_int(B), C.c_int(H), C.c_int(Hkv), C.c_int(S), C.c_int(window),
                       C.c_void_p(dbase), C.c_void_p(dbase + 2 * HD), C.c_void_p(dbase + 2 * (HD + KD)), C.c_int(ld))
    return dqkv


def fix48(u):
    """float32 -> the 64-bit fixed-point contribution (48 fractional bits) of the query-gradient accumulator."""
    f = lib().orc_fix48
    f.restype, f.argtypes = C.c_int64, [C.c_float]
    return int(f(C.c_float(float(np.float32(u)))))


def unfix48(a):
    f = lib().orc_unfix48
    f.restype, f.argtypes = C.c_float, [C.c_int64]
    return np.float32(f(C.c_int64(int(a))))


# ---- glue -----------------------------------------------------------------
def swiglu_fwd(gu):
    gu = _c(gu, np.uint16)
    rows, F2 = gu.shape
    h = np.empty((rows, F2 // 2), np.uint16)
    lib().orc_swiglu_fwd(_p(gu), C.c_int(rows), C.c_int(F2 // 2), _p(h))
    return h


def swiglu_bwd(dh, gu):
    dh = _c(dh, np.uint16)
    gu = _c(gu, np.uint16)
    rows, F2 = gu.shape
    dgu = np.empty_like(gu)
    lib().orc_swiglu_bwd(_p(dh), _p(gu), C.c_int(rows), C.c_int(F2 // 2), _p(dgu))
    return dgu


def residual_add(a, b):
    a = _c(a, np.uint16)
    b = _c(b, np.uint16)
    y = np.empty_like(a)
    lib().orc_residual_add(_p(a), _p(b), C.c_size_t(a.size), _p(y))
    return y


def embed_fwd(tok, E):
    tok = _c(tok, np.int32).reshape(-1)
    E = _c(E, np.uint16)
    y = np.empty((tok.size, E.shape[1]), np.uint16)
    lib().orc_embed_fwd(_p(tok), C.c_int(tok.size), _p(E), C.c_int(E.shape[1]), _p(y))
    return y


def embed_bwd(tok, dy, V):
    tok = _c(tok, np.int32).reshape(-1)
    dy = _c(dy, np.uint16)
    dE = np.empty((V, dy.shape[1]), np.float32)
    lib().orc_embed_bwd(_p(tok), C.c_int(tok.size), _p(dy), C.c_int(V), C.c_int(dy.shape[1]), _p(dE))
    return dE


def linear_bwd_rows(dY, X, W, s_x, s_w, rows_m, rows_n, hb=128):
    """Rows rows_m of dX and rows rows_n of dW of linear_bwd (same bits), without the full contractions."""
    dY = _c(dY, np.uint16)
    X = _c(X, np.uint16)
    W = _c(W, np.uint16)
    s_x = _c(s_x, np.float32).reshape(1)
    s_w = _c(s_w, np.float32)
    rows_m = _c(rows_m, np.int32)
    rows_n = _c(rows_n, np.int32)
    M, K = X.shape
    N = W.shape[0]
    if hb:
        assert M % 128 == 0 and N % 128 == 0
    dX = np.empty((rows_m.size, K), np.uint16)
    dW = np.empty((rows_n.size, K), np.float32)
    lib().orc_linear_bwd_rows(_p(dY), _p(X), _p(W), C.c_int(M), C.c_int(N), C.c_int(K), _p(s_x), _p(s_w), C.c_int(hb),
                              _p(rows_m), C.c_int(rows_m.size), _p(rows_n), C.c_int(rows_n.size), _p(dX), _p(dW))
    return dX, dW


def lmhead_fwd(Hh, W):
    Hh = _c(Hh, np.uint16)
    W = _c(W, np.uint16)
    M, K = Hh.shape
    V = W.shape[0]
    out = np.empty((M, V), np.float32)
    lib().orc_lmhead_fwd(_p(Hh), _p(W), C.c_int(M), C.c_int(V), C.c_int(K), _p(out))
    return out


def lmhead_bwd(dlogits, Hh, W, dW=None):
    """dW=None starts the token-ordered weight-gradient sum from +0; else continues it in place."""
    dlogits = _c(dlogits, np.float32)
    Hh = _c(Hh, np.uint16)
    W = _c(W, np.uint16)
    M, K = Hh.shape
    V = W.shape[0]
    first = dW is None
    if first:
        dW = np.empty((V, K), np.float32)
    dH = np.empty((M, K), np.uint16)
    lib().orc_lmhead_bwd(_p(dlogits), _p(Hh), _p(W), C.c_int(M), C.c_int(V), C.c_int(K), _p(dH), _p(dW), C.c_int(int(first)))
    return dH, dW


# ---- gradient reduction replay, clip, optimizer, hash ---------------------
class Accum:
    """Algorithm 1 + Algorithm 2 as a push interface (mesh order)."""

    def __init__(self, accum, dp_shard, dp_replicate, n):
        self.h = C.c_void_p(lib().orc_accum_new(C.c_int(accum), C.c_int(dp_shard), C.c_int(dp_replicate), C.c_size_t(n)))
        self.n = n

    def push(self, g):
        g = _c(g, np.float32)
        assert g.size == self.n
        return lib().orc_accum_push(self.h, _p(g))

    def result(self):
        out = np.empty(self.n, np.float32)
        rc = lib().orc_accum_result(self.h, _p(out))
        if rc != 0:
            raise ValueError("push count does not match the mesh")
        return out

    @property
    def max_resident(self):
        return lib().orc_accum_max_resident(self.h)

    @property
    def stack_size(self):
        return lib().orc_accum_stack_size(self.h)

    def __del__(self):
        if getattr(self, "h", None):
            lib().orc_accum_free(self.h)
            self.h = None


def grad_norm(tensors, max_norm=1.0):
    ts = [_c(t, np.float32).reshape(-1) for t in tensors]
    ptrs = (C.c_void_p * len(ts))(*[t.ctypes.data for t in ts])
    ns = (C.c_size_t * len(ts))(*[t.size for t in ts])
    norm = np.empty(1, np.float32)
    coef = np.empty(1, np.float32)
    lib().orc_grad_norm(ptrs, ns, C.c_int(len(ts)), C.c_float(max_norm), _p(norm), _p(coef))
    return norm[0], coef[0]


def scale(g, coef):
    g = _c(g, np.float32).copy()
    lib().orc_scale(_p(g), C.c_size_t(g.size), C.c_float(coef))
    return g


def adamw(p, g, m, v, lr, beta1, beta2, eps, wd, step):
    """Returns updated copies (p keeps its dtype: uint16 = bf16 bits, float32 = f32)."""
    bf = p.dtype == np.uint16
    p = np.ascontiguousarray(p).copy()
    g = _c(g, np.float32)
    m = _c(m, np.float32).copy()
    v = _c(v, np.float32).copy()
    lib().orc_adamw(C.c_double(lr), C.c_double(beta1), C.c_double(beta2), C.c_double(eps), C.c_double(wd), C.c_int(step),
                    C.c_int(int(bf)), _p(p), _p(g), _p(m), _p(v), C.c_size_t(p.size))
    return p, m, v


def sha256(data):
    b = np.frombuffer(bytes(data), np.uint8) if not isinstance(data, np.ndarray) else data.view(np.uint8).reshape(-1)
    b = np.ascontiguousarray(b)
    out = np.empty(32, np.uint8)
    lib().orc_sha256(_p(b), C.c_size_t(b.size), _p(out))
    return out.tobytes().hex()


def tensor_hash(arr):
    b = np.ascontiguousarray(arr).view(np.uint8).reshape(-1)
    out = np.empty(32, np.uint8)
    lib().orc_tensor_hash(_p(b), C.c_size_t(b.size), _p(out))
    return out.tobytes().hex()
