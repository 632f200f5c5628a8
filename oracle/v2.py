"""CPU oracle, arithmetic version 2 -- TEST INFRASTRUCTURE ONLY.

Version 2 replaces one definition of version 1: the LM-head contraction becomes an order-free, exactly defined sum of
integer products of aligned bf16 significands with a single rounding (see v2.c).  It lives in files of its own so that
version 1 and everything keyed to its sources stay untouched.  bf16 tensors are numpy uint16 bit patterns.
"""
import ctypes as C
import os
import subprocess

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_DIR, "liboracle_v2.so")
_SRC = os.path.join(_DIR, "v2.c")
_HDR = os.path.join(_DIR, "prim.h")
_lib = None


def build(force=False):
    if not force and os.path.exists(_SO) and os.path.getmtime(_SO) >= max(os.path.getmtime(_SRC), os.path.getmtime(_HDR)):
        return _SO
    subprocess.check_call(["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-msse4.1", "-fopenmp", "-shared", "-fPIC", "-o", _SO,
                           _SRC, "-lm"])
    return _SO


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(_SO)
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def slice_rows(X):
    """X bf16 [R,K] -> (hi int8 [R,K], lo int8 [R,K], E int32 [R]); bit 30 of E marks a row with a non-finite value."""
    X = np.ascontiguousarray(X, dtype=np.uint16)
    R, K = X.shape
    hi, lo, E = np.empty((R, K), np.int8), np.empty((R, K), np.int8), np.empty(R, np.int32)
    lib().orc2_slice_rows(_p(X), C.c_int(R), C.c_int(K), _p(hi), _p(lo), _p(E))
    return hi, lo, E


def lmhead_fwd(Hh, W):
    """logits f32 [M,V]: version-2 contraction of the rows of Hh [M,K] with the rows of W [V,K]."""
    Hh = np.ascontiguousarray(Hh, dtype=np.uint16)
    W = np.ascontiguousarray(W, dtype=np.uint16)
    M, K = Hh.shape
    V = W.shape[0]
    assert W.shape[1] == K
    out = np.empty((M, V), np.float32)
    lib().orc2_lmhead_fwd(_p(Hh), _p(W), C.c_int(M), C.c_int(V), C.c_int(K), _p(out))
    return out


def attn_fwd(qkv, B, H, S):
    """Causal attention in arithmetic version 2 (see v2.c).  qkv: uint16 [B*S, 3*H*128] (q | k | v column blocks).
    Returns out bf16 [B*S, H*128] and lse f32 [B,H,S]."""
    qkv = np.ascontiguousarray(qkv, dtype=np.uint16)
    ld = qkv.shape[1]
    assert qkv.shape[0] == B * S and ld == 3 * H * 128
    out = np.empty((B * S, H * 128), np.uint16)
    lse = np.empty((B, H, S), np.float32)
    flat = qkv.reshape(-1)
    q, k, v = flat[0:], flat[H * 128:], flat[2 * H * 128:]
    lib().orc2_attn_fwd(_p(q), C.c_void_p(q.ctypes.data + 2 * H * 128), C.c_void_p(q.ctypes.data + 4 * H * 128), C.c_int(ld),
                        C.c_int(B), C.c_int(H), C.c_int(S), _p(out), C.c_int(H * 128), _p(lse))
    return out, lse


def _f2bf(x):
    """binary32 -> bf16 bit patterns: subnormal inputs flushed to signed zero, then round to nearest even on the upper 16 bits."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = np.where((u & 0x7F800000) == 0, u & 0x80000000, u)
    r = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    nan = ((u & 0x7F800000) == 0x7F800000) & ((u & 0x007FFFFF) != 0)
    r = np.where(nan, (u >> 16) | 0x0040, r)
    return r.astype(np.uint16)


def lmhead_bwd(dlogits, Hh, W):
    """Version-2 gradients of the LM head: the two contractions are the version-2 contraction itself on transposed
    operands (the definition is symmetric in its two rows and order-free, so a transpose is all it takes).
      g  = bf16(dlogits)                                    (rounded once, as in version 1)
      dH = bf16(contraction of row m of g with column k of W over the vocabulary)     [M,K] bf16
      dW = contraction of column v of g with column k of Hh over the tokens           [V,K] f32
    Row exponents are taken over the contracted index: per token for g and per input dimension for W in dH, per
    vocabulary entry for g and per input dimension for Hh in dW."""
    g = _f2bf(dlogits)
    Hh = np.ascontiguousarray(Hh, dtype=np.uint16)
    W = np.ascontiguousarray(W, dtype=np.uint16)
    dH = _f2bf(lmhead_fwd(g, np.ascontiguousarray(W.T)))
    dW = lmhead_fwd(np.ascontiguousarray(g.T), np.ascontiguousarray(Hh.T))
    return dH, dW
