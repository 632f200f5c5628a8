"""Pins for the oracle's operations against independent references: brute-force integer GEMMs,
float64 numpy evaluations, closed forms, hand-worked elements and invariants."""
import math

import numpy as np
import pytest

import oracle
import synth

F = np.float32
bf = synth.from_bf16


def rel_err(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


def hadamard(n):
    i = np.arange(n)
    pc = np.array([[bin(a & b).count("1") for b in i] for a in i])
    return np.where(pc % 2 == 0, 1, -1).astype(np.int64)


# ---------------------------------------------------------------- LSQ linear
def test_weight_step_closed_form():
    # rows of constant magnitude c give exactly 2c * c127 (two roundings); Sec. 3.1 / Sec. 4.4 formula
    c127 = F(1 / math.sqrt(127))
    W = np.empty((3, 256), F)
    for r, c in enumerate((0.5, 0.015625, 2.0)):
        W[r] = c * np.where(np.arange(256) % 3 == 0, -1, 1)
    s = oracle.lsq_weight_scale(synth.to_bf16(W))
    exp = np.array([F(F(2 * c) * c127) for c in (0.5, 0.015625, 2.0)], F)
    assert np.array_equal(s, exp)
    Wn = synth.normal_bf16((64, 2048), 0.02, seed=0, tid=1)
    s = oracle.lsq_weight_scale(Wn)
    ref = 2 * np.abs(bf(Wn).astype(np.float64)).mean(axis=1) / math.sqrt(127)
    assert np.allclose(s, ref, rtol=1e-5) and abs(s.mean() - 0.002832) < 1e-4
    st = oracle.lsq_weight_scale(Wn, per_tensor=True)
    assert np.all(st == st[0]) and abs(st[0] - ref.mean()) < 1e-6
    sx = oracle.lsq_act_scale_init(Wn)
    assert sx[0] == st[0]


def test_quantiser_hand_cases():
    # t = 0.5, 1.5, 2.5, -0.5, 127.5, -128.5, 300 -> 0, 2, 2, 0, 127, -128, 127 (ties to even, clip)
    t = np.array([[0.5, 1.5, 2.5, -0.5, 127.5, -128.5, 300.0, -1.5]], F)
    q = oracle.lsq_quantize(synth.to_bf16(t), np.array([1.0], F), per_row=False)
    assert q.tolist() == [[0, 2, 2, 0, 127, -128, 127, -2]]


def test_int_gemm_bruteforce_and_forward():
    M, N, K = 37, 29, 384
    X = synth.normal_bf16((M, K), 1.0, seed=0, tid=10)
    W = synth.normal_bf16((N, K), 0.02, seed=0, tid=11)
    s_w = oracle.lsq_weight_scale(W)
    s_x = oracle.lsq_act_scale_init(X)
    Y, qX, qW = oracle.linear_fwd(X, W, s_x, s_w)
    acc = qX.astype(np.int64) @ qW.astype(np.int64).T
    assert np.array_equal(oracle.igemm_tn(qX, qW).astype(np.int64), acc)
    # independent quantiser in float64: products x*(1/s) are exact in double, rint ties to even
    inv = F(1) / s_x[0]
    t = (bf(X).astype(np.float64) * np.float64(inv)).astype(F)
    assert np.array_equal(qX, np.clip(np.rint(t), -128, 127).astype(np.int8))
    # dequantise: one f32 product of the scales, one f32 product with the accumulator, one bf16 rounding
    sc = (np.float64(s_x[0]) * s_w.astype(np.float64)).astype(F)
    ref = synth.to_bf16((acc.astype(F).astype(np.float64) * sc[None, :].astype(np.float64)).astype(F))
    assert np.array_equal(Y, ref)
    # and it approximates the unquantised product
    assert rel_err(bf(Y), bf(X).astype(np.float64) @ bf(W).astype(np.float64).T) < 0.1


def test_hadamard_butterflies():
    H = hadamard(128)
    v = np.random.default_rng(0).integers(-128, 128, 128).astype(np.int32)
    assert np.array_equal(oracle.wht128_i(v).astype(np.int64), H @ v.astype(np.int64))
    assert np.array_equal(oracle.wht128_i(oracle.wht128_i(v)), 128 * v)       # H*H = 128 I
    x = np.random.default_rng(1).integers(-1000, 1000, 128).astype(F)          # small integers: exact in f32
    assert np.array_equal(oracle.wht128_f(x).astype(np.int64), H @ x.astype(np.int64))
    assert np.array_equal(oracle.wht128_f(oracle.wht128_f(x)), 128 * x)


def test_gradient_absmax_ignores_nan_wherever_it_sits():
    """The per-tensor absmax of the rotated gradient operands skips NaNs, so the steps do not depend on the order in which
    the tensor is scanned: with one NaN in dY the step of each operand is the absmax over the finite rotated values / 127,
    recomputed here with a Hadamard matrix product (small integers times powers of two: exact in float64)."""
    M = N = K = 256
    rng = np.random.default_rng(7)
    dY = synth.to_bf16((rng.integers(-64, 64, (M, N)) * 2.0 ** -10).astype(F))
    X = synth.normal_bf16((M, K), 1.0, seed=0, tid=80)
    W = synth.normal_bf16((N, K), 0.02, seed=0, tid=81)
    s_x, s_w = oracle.lsq_act_scale_init(X), np.full(N, 2.0 ** -6, F)
    H = hadamard(128).astype(np.float64)
    for (r, c) in ((3, 5), (200, 250)):                      # early and late in either scan order
        d = dY.copy(); d[r, c] = 0x7FC0
        _, _, _, dbg = oracle.linear_bwd(d, X, W, s_x, s_w, hb=128, debug=True)
        g = bf(d).astype(np.float64)
        a = (g * 2.0 ** -6).reshape(M, N // 128, 128) @ H                    # rotation along n, rows scaled by s_w
        gt = np.einsum("ij,bjn->bin", H, g.reshape(M // 128, 128, N))        # rotation along the token index
        assert dbg["scales"][0] == F(np.nanmax(np.abs(a))) / F(127.0)
        assert dbg["scales"][2] == F(np.nanmax(np.abs(gt))) / F(127.0)


def _ref_linear_bwd(dY, X, W, s_x, s_w):
    """float64 straight-through reference with exact (unquantised-gradient) contractions."""
    inv = F(1) / s_x[0]
    tx = (bf(X).astype(np.float64) * np.float64(inv)).astype(F)
    qX = np.clip(np.rint(tx), -128, 127)
    inv_w = (F(1) / s_w).astype(F)
    tw = (bf(W).astype(np.float64) * inv_w[:, None].astype(np.float64)).astype(F)
    qW = np.clip(np.rint(tw), -128, 127)
    g = bf(dY).astype(np.float64)
    gx = g @ (qW * s_w[:, None].astype(np.float64))
    dX = np.where((tx >= -128) & (tx <= 127), gx, 0)
    dW = np.where((tw >= -128) & (tw <= 127), g.T @ (qX * np.float64(s_x[0])), 0)
    phi = np.where(tx < -128, -128, np.where(tx > 127, 127, qX - tx.astype(np.float64)))
    ds = (gx * phi).sum() / math.sqrt(X.size * 127)
    return dX, dW, ds


@pytest.mark.parametrize("hb", [0, 128])
def test_linear_bwd_against_float64(hb):
    M, N, K = 256, 256, 384
    X = synth.normal_bf16((M, K), 1.0, seed=0, tid=20)
    X.reshape(-1)[:5] = synth.to_bf16(np.array([40, -40, 30, -35, 50], F))   # out-of-range activations (mask)
    W = synth.normal_bf16((N, K), 0.02, seed=0, tid=21)
    dY = synth.normal_bf16((M, N), 0.01, seed=0, tid=22)
    s_w = oracle.lsq_weight_scale(W)
    s_x = oracle.lsq_act_scale_init(X)
    dX, dW, ds = oracle.linear_bwd(dY, X, W, s_x, s_w, hb=hb)
    rX, rW, rs = _ref_linear_bwd(dY, X, W, s_x, s_w)
    assert rel_err(bf(dX), rX) < 0.03
    assert rel_err(dW, rW) < 0.03
    assert abs(ds[0] - rs) < 0.05 * abs(rs) + 1e-6
    assert np.all(bf(dX).reshape(-1)[:5] == 0)                               # STE range mask


def test_linear_bwd_rows_is_a_view_of_the_full_backward():
    """The row-sampled entry (used for checks at shapes too large for a CPU contraction) gives the bits of the full one."""
    M, N, K = 256, 384, 256
    X, W, dY = synth.normal_bf16((M, K), 1.0, seed=0, tid=90), synth.normal_bf16((N, K), 0.02, seed=0, tid=91), \
        synth.normal_bf16((M, N), 0.01, seed=0, tid=92)
    sw, sx = oracle.lsq_weight_scale(W), oracle.lsq_act_scale_init(X)
    for hb in (128, 0):
        full = oracle.linear_bwd(dY, X, W, sx, sw, hb)
        rm, rn = np.array([0, 5, 130, 255], np.int32), np.array([1, 100, 383], np.int32)
        dx, dw = oracle.linear_bwd_rows(dY, X, W, sx, sw, rm, rn, hb)
        assert np.array_equal(dx, full[0][rm]) and np.array_equal(dw.view(np.uint32), full[1][rn].view(np.uint32))


def test_hadamard_modes_agree_when_quantisation_is_exact():
    # one non-zero per 128-block, power-of-two magnitudes: rotated and unrotated operands both quantise exactly
    M = N = K = 128
    X = np.zeros((M, K), F); W = np.zeros((N, K), F); dY = np.zeros((M, N), F)
    X[5, 9] = 2.0
    W[17, 9] = 0.5
    dY[5, 17] = 0.25
    s_x = np.array([2.0 / 64], F); s_w = np.full(N, 0.5 / 64, F)
    a0 = oracle.linear_bwd(synth.to_bf16(dY), synth.to_bf16(X), synth.to_bf16(W), s_x, s_w, hb=0)
    a1 = oracle.linear_bwd(synth.to_bf16(dY), synth.to_bf16(X), synth.to_bf16(W), s_x, s_w, hb=128)
    for u, v in zip(a0, a1):
        assert np.array_equal(u, v)
    assert bf(a0[0])[5, 9] == F(0.25 * 0.5) and a0[1][17, 9] == F(0.25 * 2.0)


def test_step_size_gradient_by_hand():
    """ds_x = det_sum(gx * phi) / sqrt(M K 127) (the LSQ step-size gradient, Sec. 3.1) on two hand-made elements whose
    quantisation is exact.  Element (5, 9): x / s = 4.5 rounds to the code 4 (ties to even), phi = 4 - 4.5 = -0.5, the
    gradient reaching it is 0.25 * 0.5 = 0.125.  Element (6, 10): x / s = 200 lies above the range, so phi = 127, the
    gradient of x is masked to 0 and the same 0.125 enters the step-size gradient.  The sum of the two terms,
    0.125 * (127 - 0.5) = 15.8125, is exact; with or without the rotation."""
    M = N = K = 128
    X = np.zeros((M, K), F); W = np.zeros((N, K), F); dY = np.zeros((M, N), F)
    X[5, 9], X[6, 10] = 2.25, 100.0
    W[17, 9] = W[18, 10] = 0.5
    dY[5, 17] = dY[6, 18] = 0.25
    s_x = np.array([0.5], F); s_w = np.full(N, 0.5 / 64, F)
    gs = F(1.0 / math.sqrt(M * K * 127.0))
    for hb in (0, 128):
        dX, dW, ds = oracle.linear_bwd(synth.to_bf16(dY), synth.to_bf16(X), synth.to_bf16(W), s_x, s_w, hb=hb)
        assert bf(dX)[5, 9] == F(0.125) and bf(dX)[6, 10] == 0.0                  # in range: passed on; out of range: masked
        assert ds[0] == F(gs * F(15.8125))
        assert abs(float(ds[0]) - 15.8125 / math.sqrt(M * K * 127.0)) < 1e-9
        assert dW[17, 9] == F(0.25 * 4 * 0.5) and abs(dW[18, 10] - 0.25 * 127 * 0.5) < 2e-6   # x^ = code * s_x: 2.0 and 63.5


def test_hadamard_reduces_weight_gradient_error_on_heavy_tails():
    # Sec. 3.2: rotation flattens gradient outliers (paper: ~5% -> ~1% at its shapes; a sanity check)
    M, N, K = 1024, 128, 128
    X = synth.normal_bf16((M, K), 1.0, seed=0, tid=30)
    W = synth.normal_bf16((N, K), 0.02, seed=0, tid=31)
    g = synth.normal_f32((M, N), 0.01, seed=0, tid=32)
    g[::97, ::13] *= 60.0                                                      # sparse outliers
    dY = synth.to_bf16(g)
    s_w = oracle.lsq_weight_scale(W); s_x = oracle.lsq_act_scale_init(X)
    _, rW, _ = _ref_linear_bwd(dY, X, W, s_x, s_w)
    e0 = rel_err(oracle.linear_bwd(dY, X, W, s_x, s_w, hb=0)[1], rW)
    e1 = rel_err(oracle.linear_bwd(dY, X, W, s_x, s_w, hb=128)[1], rW)
    assert e1 < 0.5 * e0 and e1 < 0.03


# ---------------------------------------------------------------- RMSNorm
def test_rmsnorm_hand_row_and_float64():
    x = np.array([[1.0, 2.0, 2.0, 4.0]], F)        # mean square = 25/4 = 6.25, eps = 0 -> rstd = 0.4 (rounded)
    g = np.array([1.0, 0.5, 2.0, 1.0], F)
    y, rstd = oracle.rmsnorm_fwd(x, g, eps=0.0)
    r = F(1) / F(2.5)
    assert rstd[0] == r
    assert np.array_equal(y[0], np.array([F(F(1 * r) * 1), F(F(2 * r) * F(0.5)), F(F(2 * r) * 2), F(F(4 * r) * 1)], F))
    rows, D = 33, 2048
    x = synth.normal_f32((rows, D), seed=0, tid=40)
    g = 1 + synth.normal_f32(D, 0.02, seed=0, tid=41)
    dy = synth.normal_f32((rows, D), seed=0, tid=42)
    y, rstd = oracle.rmsnorm_fwd(x, g, eps=1e-6)
    x64, g64, dy64 = x.astype(np.float64), g.astype(np.float64), dy.astype(np.float64)
    rs64 = 1 / np.sqrt((x64 ** 2).mean(1) + 1e-6)
    assert np.allclose(rstd, rs64, rtol=3e-7) and np.allclose(y, x64 * rs64[:, None] * g64, rtol=1e-6, atol=1e-7)
    dx, dg = oracle.rmsnorm_bwd(dy, x, g, rstd)
    w = dy64 * g64; xh = x64 * rs64[:, None]
    dx64 = rs64[:, None] * (w - xh * (w * xh).mean(1, keepdims=True))
    assert np.allclose(dx, dx64, rtol=1e-4, atol=1e-6) and np.allclose(dg, (dy64 * xh).sum(0), rtol=1e-4, atol=1e-5)
    # constant row c: y = gamma * sign(c) (up to rounding), gain-free variant
    yc, _ = oracle.rmsnorm_fwd(np.full((1, 256), 3.0, F), None, eps=0.0)
    assert np.allclose(yc, 1.0, atol=2e-7)
    # bf16 I/O variant rounds once at the output
    xb = synth.to_bf16(x); gb = synth.to_bf16(g)
    yb, rb = oracle.rmsnorm_fwd(xb, gb, bf=True)
    yf, rf = oracle.rmsnorm_fwd(bf(xb), bf(gb))
    assert np.array_equal(yb, synth.to_bf16(yf)) and np.array_equal(rb, rf)


# ---------------------------------------------------------------- cross-entropy
def test_xent_closed_forms():
    V = 50304
    z = np.full((2, V), 3.25, F)
    loss, lse, lm, zm, bad = oracle.xent_fwd(z, np.array([7, V - 1], np.int32))
    logV = oracle.prim("log", [float(V)])[0]                 # S = V exactly, so loss = det_log(V) ~ log V
    assert bad == 0 and np.all(loss == F(F(3.25) + logV) - F(3.25)) and abs(loss[0] - math.log(V)) < 2e-6
    z = np.zeros((1, 1000), F); z[0, 5] = 100.0                # gap >= 88: every other term flushes to +0
    loss, lse, lm, _, _ = oracle.xent_fwd(z, np.array([5], np.int32))
    assert loss[0] == 0 and lse[0] == 100 and lm[0] == 0
    z = np.array([[0.0, 1.0]], F)                               # V = 2 by hand: log(1 + e^-1) for target 1
    loss, lse, _, _, _ = oracle.xent_fwd(z, np.array([1], np.int32))
    assert abs(loss[0] - math.log1p(math.exp(-1))) < 1e-6
    # out-of-range target: counted, row contributes zero
    loss, _, lm, _, bad = oracle.xent_fwd(z, np.array([2], np.int32))
    assert bad == 1 and loss[0] == 0


def test_xent_against_float64():
    rows, V = 16, 50304
    z = synth.normal_f32((rows, V), 2.0, seed=0, tid=50)
    t = synth.randint(rows, V, seed=0, tid=51)
    loss, lse, lm, zm, _ = oracle.xent_fwd(z, t, z_weight=1e-4)
    z64 = z.astype(np.float64)
    lse64 = np.log(np.exp(z64 - z64.max(1, keepdims=True)).sum(1)) + z64.max(1)
    assert np.allclose(lse, lse64, rtol=3e-7)
    assert np.allclose(loss, lse64 - z64[np.arange(rows), t], rtol=1e-5)
    assert abs(lm[0] - ((lse64 - z64[np.arange(rows), t]).mean() + 1e-4 * (lse64 ** 2).mean())) < 1e-5
    dz = oracle.xent_bwd(z, t, lse, scale=1.0 / rows)
    p = np.exp(z64 - lse64[:, None]); p[np.arange(rows), t] -= 1
    assert np.allclose(dz, p / rows, rtol=1e-4, atol=1e-9)
    assert np.abs(dz.astype(np.float64).sum(1)).max() < 1e-6   # softmax gradient sums to ~0 without z-loss
    dzz = oracle.xent_bwd(z, t, lse, z_weight=1e-4, scale=1.0)
    pz = np.exp(z64 - lse64[:, None])
    ref = pz * (1 + 2e-4 * lse64[:, None]); ref[np.arange(rows), t] -= 1
    assert np.allclose(dzz, ref, rtol=1e-4, atol=1e-9)


# ---------------------------------------------------------------- attention
def _attn_ref(qkv, B, H, S):
    x = bf(qkv).astype(np.float64).reshape(B, S, 3, H, 128)
    q, k, v = (x[:, :, i].transpose(0, 2, 1, 3) for i in range(3))
    s = q @ k.transpose(0, 1, 3, 2) / math.sqrt(128)
    s = np.where(np.tril(np.ones((S, S), bool)), s, -np.inf)
    lse = np.log(np.exp(s - s.max(-1, keepdims=True)).sum(-1)) + s.max(-1)
    p = np.exp(s - lse[..., None])
    return q, k, v, p, p @ v, lse


def test_attention_forward_pins():
    B, H, S = 1, 2, 257                       # 257 exercises a full tile, a second full tile and a 1-key tile
    qkv = synth.normal_bf16((B * S, 3 * H * 128), 1.0, seed=0, tid=60)
    out, lse = oracle.attn_fwd(qkv, B, H, S)
    q, k, v, p, o, l = _attn_ref(qkv, B, H, S)
    o = o.transpose(0, 2, 1, 3).reshape(B * S, H * 128)
    assert np.abs(bf(out) - o).max() < 0.02 and np.allclose(lse, l, rtol=1e-5, atol=1e-5)
    assert np.array_equal(out[0], qkv[0, 2 * H * 128:])                       # i = 0 -> out = v_0 exactly
    # causality: changing keys/values after position i leaves rows <= i bit-identical
    qkv2 = qkv.copy(); qkv2[200:, H * 128:] = synth.normal_bf16((S - 200, 2 * H * 128), 1.0, seed=1, tid=61)
    out2, lse2 = oracle.attn_fwd(qkv2, B, H, S)
    assert np.array_equal(out2[:200], out[:200]) and np.array_equal(lse2[:, :, :200], lse[:, :, :200])
    # q = 0 -> uniform weights, out_i ~ mean(v_0..v_i)
    qkv3 = qkv.copy(); qkv3[:, :H * 128] = 0
    out3, lse3 = oracle.attn_fwd(qkv3, B, H, S)
    vm = np.cumsum(bf(qkv3[:, 2 * H * 128:]).astype(np.float64), 0) / np.arange(1, S + 1)[:, None]
    assert np.abs(bf(out3) - vm).max() < 0.02
    assert np.allclose(lse3[0, 0], np.log(np.arange(1, S + 1)), atol=1e-5)


def _qkv_rows(S, H=1):
    return np.zeros((S, 3 * H * 128), np.uint16)


def _bfrow(vals):
    return synth.to_bf16(np.asarray(vals, F))


def test_attention_logit_is_a_sequential_ascending_dot():
    """One key, q = k = (4096, 1, 1, ..., 1): the products are 2^24, 1, ..., 1.  Added in ascending order every 1 is
    lost against 2^24 (ties to even), so the logit is 2^24/sqrt(128); a pairwise tree or a descending sum collects the
    127 ones first and gives (2^24 + 128)/sqrt(128).  With a single key the weight is 1, so lse is the logit itself."""
    qkv = _qkv_rows(1)
    r = _bfrow([4096.0] + [1.0] * 127)
    qkv[0, :128] = r; qkv[0, 128:256] = r; qkv[0, 256:] = _bfrow(np.arange(128) - 60.0)
    out, lse = oracle.attn_fwd(qkv, 1, 1, 1)
    scale = F(float.fromhex("0x1.6a09e6p-4"))
    assert lse[0, 0, 0] == F(F(2.0 ** 24) * scale) and lse[0, 0, 0] != F(F(2.0 ** 24 + 128) * scale)
    assert np.array_equal(out[0], qkv[0, 256:])
    # the same for the backward's recomputed logit: dV_0 = bf16(P) dO with P = exp(s - lse) = exp(0) = 1
    dout = _bfrow(np.linspace(-1, 1, 128)).reshape(1, 128)
    d = oracle.attn_bwd(dout, qkv, out, lse, 1, 1, 1)
    assert np.array_equal(d[0, 256:], dout[0])


def test_attention_rounds_the_weights_to_bf16_for_pv_but_not_for_the_row_sum():
    """Two keys seen by row 1, logits (s0, 0) through one-hot dimensions, v0 = 1, v1 = 0: the output is
    bf16(p0) / (p0 + 1) with p0 = exp(s0) (the oracle's exp, pinned on its own), the division being a reciprocal and a
    product in binary32, the result rounded to bf16.  Leaving out the rounding of p0, or summing the rounded weights,
    gives another bf16 value for most of the arguments below."""
    scale = F(float.fromhex("0x1.6a09e6p-4"))
    seen_unrounded = seen_roundsum = 0
    for x0 in (-1.0, -3.0, -5.0, -7.0, -9.0, -11.0, -13.0, -19.0, -23.0, -29.0):
        qkv = _qkv_rows(2)
        qkv[1, 0] = _bfrow([1.0])[0]                      # q_1 = e_0
        qkv[0, 128] = _bfrow([x0])[0]                     # k_0 = x0 e_0, k_1 = 0
        qkv[0, 256:] = _bfrow(np.ones(128))               # v_0 = 1, v_1 = 0
        out, lse = oracle.attn_fwd(qkv, 1, 1, 2)
        s0 = F(F(x0) * scale)
        p0 = oracle.prim("exp", np.array([s0], F))[0]
        l = F(p0 + F(1.0))
        il = F(F(1.0) / l)
        pt = bf(synth.to_bf16(np.array([p0], F)))[0]
        want = synth.to_bf16(np.array([F(pt * il)], F))[0]
        assert np.all(out[1] == want), x0
        assert lse[0, 0, 1] == F(F(0.0) + oracle.prim("log", np.array([l], F))[0])
        seen_unrounded += synth.to_bf16(np.array([F(p0 * il)], F))[0] != want
        seen_roundsum += synth.to_bf16(np.array([F(pt * F(F(1.0) / F(pt + F(1.0))))], F))[0] != want
    assert seen_unrounded >= 2 and seen_roundsum >= 1     # the cases do tell the readings apart


def test_attention_key_tile_is_128_and_earlier_tiles_are_rescaled():
    """Row 128 sees keys 0..128 with logits s_A0 > s_A1 at keys 0 and 1, a dominant logit 0 at key B, and logits so low
    everywhere else that their weights are exactly 0.  With B = 127 all three share the first tile:
    l = (exp(s_A0) + exp(s_A1)) + 1.  With B = 128 the first tile is normalised by its own maximum s_A0 and rescaled when
    the second tile arrives: l = (1 + exp(s_A1 - s_A0)) * exp(s_A0) + 1.  The two differ in the last bits, and a tile of
    64 or of 256 keys would put the boundary elsewhere.  exp and log are the oracle's own (pinned separately)."""
    scale = F(float.fromhex("0x1.6a09e6p-4"))
    ex = lambda x: oracle.prim("exp", np.array([x], F))[0]
    lg = lambda x: oracle.prim("log", np.array([x], F))[0]
    differ = 0
    for xa0, xa1 in ((-8.0, -16.0), (-16.0, -17.0), (-15.75, -16.5), (-15.5, -16.0), (-15.25, -20.0), (-1.0, -2.0)):
        sA0, sA1 = F(F(xa0) * scale), F(F(xa1) * scale)
        got = {}
        for Bk in (127, 128):
            S = 129
            qkv = _qkv_rows(S)
            qkv[128, 0] = _bfrow([1.0])[0]                            # q_128 = e_0
            qkv[:, 128] = _bfrow([-30000.0])[0]                       # every key far below ...
            qkv[0, 128] = _bfrow([xa0])[0]; qkv[1, 128] = _bfrow([xa1])[0]
            qkv[Bk, 128] = 0                                          # ... except A0, A1 and B
            out, lse = oracle.attn_fwd(qkv, 1, 1, S)
            got[Bk] = lse[0, 0, 128]
        same_tile = F(F(ex(sA0) + ex(sA1)) + F(1.0))
        two_tiles = F(F(F(F(1.0) + ex(F(sA1 - sA0))) * ex(F(sA0 - F(0.0)))) + F(1.0))
        assert got[127] == F(F(0.0) + lg(same_tile)), (xa0, xa1)
        assert got[128] == F(F(0.0) + lg(two_tiles)), (xa0, xa1)
        differ += same_tile != two_tiles
    assert differ >= 4


def test_attention_value_gradient_sums_queries_in_ascending_order():
    """Every row puts weight exactly 1 on key 0 (its logit is 0, every other logit is far below), so
    dV_0 = sum_i dO_i in binary32, queries ascending from +0.  Column 0 of dO is (2^24, 1, ..., 1, -2^24): ascending, the
    ones are lost and the total is 0; any other order keeps some of them.  Column 1 is (1, ..., 1, 2^24, -2^24): the 62
    ones are exact before the large terms arrive, total 62.  Column 2 is (2^24, -2^24, 1, ..., 1): total 62 as well."""
    S = 64
    qkv = _qkv_rows(S)
    qkv[:, 0] = _bfrow([1.0])[0]                                      # q_i = e_0
    qkv[1:, 128] = _bfrow([-30000.0])[0]                              # k_0 = 0, the others far below
    qkv[:, 256:] = synth.normal_bf16((S, 128), 1.0, seed=0, tid=68)
    out, lse = oracle.attn_fwd(qkv, 1, 1, S)
    assert np.all(lse == 0) and np.array_equal(out, np.tile(qkv[0, 256:], (S, 1)))
    dO = np.zeros((S, 128), F)
    dO[:, 0] = 1.0; dO[0, 0] = 2.0 ** 24; dO[S - 1, 0] = -2.0 ** 24
    dO[:, 1] = 1.0; dO[S - 2, 1] = 2.0 ** 24; dO[S - 1, 1] = -2.0 ** 24
    dO[:, 2] = 1.0; dO[0, 2] = 2.0 ** 24; dO[1, 2] = -2.0 ** 24
    d = oracle.attn_bwd(synth.to_bf16(dO), qkv, out, lse, 1, 1, S)
    dv0 = bf(d[0, 256:])
    assert dv0[0] == 0.0 and dv0[1] == 62.0 and dv0[2] == 62.0 and np.all(dv0[3:] == 0.0)
    assert np.all(bf(d[1:, 256:]) == 0.0)                             # no weight on the other keys


def test_attention_query_gradient_sums_keys_in_ascending_order():
    """q = 0 makes the weights of row 63 uniform, values alternating +1, -1 in one column make O = 0 exactly (so Delta = 0)
    and dP = +d, -d; dS_63,j is then +g, -g with ONE magnitude g.  Keys that carry the same alternating sign times
    (2^25, 1, ..., 1, -2^25) in column 3 give dQ_63,3 = g 2^25 + g + ... + g - g 2^25: in ascending (or descending) order
    every g is lost and the result is 0, in a tree the small terms meet first and survive.  Column 4 carries
    (1, ..., 1, 2^25, -2^25): ascending, the 62 small terms are summed exactly and then rounded against the large one;
    descending they would be added to an exact 0."""
    S = 64
    scale = F(float.fromhex("0x1.6a09e6p-4"))
    sign = np.where(np.arange(S) % 2 == 0, 1.0, -1.0).astype(F)
    t1 = np.ones(S, F); t1[0] = 2.0 ** 25; t1[-1] = -2.0 ** 25
    t2 = np.ones(S, F); t2[-2] = 2.0 ** 25; t2[-1] = -2.0 ** 25
    qkv = _qkv_rows(S)
    kk = np.zeros((S, 128), F); kk[:, 3] = sign * t1; kk[:, 4] = sign * t2
    vv = np.zeros((S, 128), F); vv[:, 7] = sign
    qkv[:, 128:256] = synth.to_bf16(kk)
    qkv[:, 256:] = synth.to_bf16(vv)
    out, lse = oracle.attn_fwd(qkv, 1, 1, S)
    assert np.all(bf(out)[S - 1] == 0.0)
    dO = np.zeros((S, 128), F); dO[S - 1, 7] = 1.0
    d = oracle.attn_bwd(synth.to_bf16(dO), qkv, out, lse, 1, 1, S)
    P = oracle.prim("exp", np.array([F(F(0.0) - lse[0, 0, S - 1])], F))[0]
    g = bf(synth.to_bf16(np.array([F(F(P * F(1.0)) * scale)], F)))[0]
    assert g > 0 and abs(g - 2.0 ** -3.5 / S) < 1e-4
    dq = bf(d[S - 1, :128])
    assert dq[3] == 0.0
    acc = F(0.0)
    for j in range(S):
        acc = F(acc + F(g * t2[j]))
    want = bf(synth.to_bf16(np.array([acc], F)))[0]
    assert dq[4] == want and want != bf(synth.to_bf16(np.array([F(62 * g)], F)))[0]    # 62 g is what a descending sum gives
    assert np.all(np.delete(dq, [3, 4]) == 0.0)


def test_attention_key_gradient_sums_queries_in_ascending_order():
    """Only keys 0 and 1 carry weight (logit 0; every other key far below), with values +1 and -1 in one column: every row
    i >= 1 has the same two weights, O = 0 exactly, Delta = 0 and dS_i0 = +g, ONE value for all rows.  The queries carry
    (2^25, 1, ..., 1, -2^25) in column 3 and (1, ..., 1, 2^25, -2^25) in column 4 (columns in which every key is 0, so the
    logits do not see them): dK_0 is 0 in column 3 for a sequential sum, and in column 4 the ascending value, which differs
    from the descending one (61 g) and from a tree's."""
    S = 64
    scale = F(float.fromhex("0x1.6a09e6p-4"))
    t1 = np.ones(S, F); t1[1] = 2.0 ** 25; t1[-1] = -2.0 ** 25; t1[0] = 0.0
    t2 = np.ones(S, F); t2[-2] = 2.0 ** 25; t2[-1] = -2.0 ** 25; t2[0] = 0.0
    qq = np.zeros((S, 128), F); qq[:, 0] = 1.0; qq[:, 3] = t1; qq[:, 4] = t2
    kk = np.zeros((S, 128), F); kk[2:, 0] = -30000.0
    vv = np.zeros((S, 128), F); vv[0, 7] = 1.0; vv[1, 7] = -1.0
    qkv = _qkv_rows(S)
    qkv[:, :128] = synth.to_bf16(qq); qkv[:, 128:256] = synth.to_bf16(kk); qkv[:, 256:] = synth.to_bf16(vv)
    out, lse = oracle.attn_fwd(qkv, 1, 1, S)
    assert np.all(bf(out)[1:] == 0.0) and np.all(lse[0, 0, 1:] == lse[0, 0, 1])
    dO = np.zeros((S, 128), F); dO[1:, 7] = 1.0
    d = oracle.attn_bwd(synth.to_bf16(dO), qkv, out, lse, 1, 1, S)
    P = oracle.prim("exp", np.array([F(F(0.0) - lse[0, 0, 1])], F))[0]
    g = bf(synth.to_bf16(np.array([F(F(P * F(1.0)) * scale)], F)))[0]
    assert abs(g - 2.0 ** -3.5 / 2) < 1e-3
    dk0 = bf(d[0, 128:256])
    assert dk0[3] == 0.0
    acc = F(0.0)
    for i in range(1, S):
        acc = F(acc + F(g * t2[i]))
    want = bf(synth.to_bf16(np.array([acc], F)))[0]
    assert dk0[4] == want and want != bf(synth.to_bf16(np.array([F(61 * g)], F)))[0]
    assert np.array_equal(bf(d[1, 128:256])[3:5], -dk0[3:5])                # key 1: the same sums with -g


def test_attention_backward_recomputes_the_weights_from_lse():
    """Two keys, dO_0 = 0, dO_1 = e_c: dV_0 = bf16(P_10) in column c, with P_10 = exp(s_0 - lse_1) recomputed from the
    stored logsumexp (not the forward's p / l) and rounded to bf16 once more by the output."""
    scale = F(float.fromhex("0x1.6a09e6p-4"))
    for x0 in (-2.0, -5.0, -9.0, 3.0):
        qkv = _qkv_rows(2)
        qkv[1, 0] = _bfrow([1.0])[0]
        qkv[0, 128] = _bfrow([x0])[0]
        qkv[:, 256:] = synth.normal_bf16((2, 128), 1.0, seed=0, tid=69)
        out, lse = oracle.attn_fwd(qkv, 1, 1, 2)
        dO = np.zeros((2, 128), F); dO[1, 5] = 1.0
        d = oracle.attn_bwd(synth.to_bf16(dO), qkv, out, lse, 1, 1, 2)
        s0 = F(F(x0) * scale)
        P10 = oracle.prim("exp", np.array([F(s0 - lse[0, 0, 1])], F))[0]
        assert d[0, 256 + 5] == synth.to_bf16(np.array([P10], F))[0], x0
        P11 = oracle.prim("exp", np.array([F(F(0.0) - lse[0, 0, 1])], F))[0]
        assert d[1, 256 + 5] == synth.to_bf16(np.array([P11], F))[0], x0


def test_attention_backward_against_float64():
    B, H, S = 2, 1, 160
    qkv = synth.normal_bf16((B * S, 3 * H * 128), 1.0, seed=0, tid=62)
    dout = synth.normal_bf16((B * S, H * 128), 0.1, seed=0, tid=63)
    out, lse = oracle.attn_fwd(qkv, B, H, S)
    dqkv = oracle.attn_bwd(dout, qkv, out, lse, B, H, S)
    q, k, v, p, o, _ = _attn_ref(qkv, B, H, S)
    do = bf(dout).astype(np.float64).reshape(B, S, H, 128).transpose(0, 2, 1, 3)
    dv = p.transpose(0, 1, 3, 2) @ do
    dp = do @ v.transpose(0, 1, 3, 2)
    ds = p * (dp - (do * o).sum(-1, keepdims=True)) / math.sqrt(128)
    dq = ds @ k; dk = ds.transpose(0, 1, 3, 2) @ q
    ref = np.stack([dq, dk, dv], 2).transpose(0, 3, 2, 1, 4).reshape(B * S, 3 * H * 128)
    got = bf(dqkv).astype(np.float64)
    for c in range(3):
        sl = slice(c * H * 128, (c + 1) * H * 128)
        assert rel_err(got[:, sl], ref[:, sl]) < 0.01
    # causal invariance of the backward: dq rows < 100 ignore later positions' inputs
    qkv2 = qkv.copy(); qkv2[B * S - 30:, :] = synth.normal_bf16((30, 3 * H * 128), 1.0, seed=2, tid=64)
    out2, lse2 = oracle.attn_fwd(qkv2, B, H, S)
    d2 = oracle.attn_bwd(dout, qkv2, out2, lse2, B, H, S)
    assert np.array_equal(d2[:S, :], dqkv[:S, :]) and np.array_equal(d2[S:S + 130 - 0, :H * 128], dqkv[S:S + 130, :H * 128])


def test_fixed_point_query_gradient_pins():
    """The 64-bit fixed-point accumulator of the query gradient (Sec. 3.2).  Hand values of the conversion; one block of
    keys: identical to the plain ordered sum wherever that sum is a multiple of 2^-48; several blocks: float64 reference,
    the other two gradients untouched, and the bf16 results at most one step away from the plain accumulator's."""
    two48 = 1 << 48
    assert oracle.fix48(1.0) == two48 and oracle.fix48(-0.75) == -3 * (1 << 46)
    assert oracle.fix48(2.0 ** -49) == 0 and oracle.fix48(3 * 2.0 ** -49) == 2      # ties go to the even integer
    assert oracle.fix48(-(2.0 ** -49)) == 0 and oracle.fix48(-3 * 2.0 ** -49) == -2
    assert oracle.fix48(5 * 2.0 ** -50) == 1 and oracle.fix48(7 * 2.0 ** -50) == 2   # 1.25 -> 1, 1.75 -> 2
    assert oracle.fix48(2.0 ** 15) == (1 << 63) - 1 and oracle.fix48(-(2.0 ** 15)) == -(1 << 63)   # saturation
    assert oracle.fix48(1e30) == (1 << 63) - 1 and oracle.fix48(-1e30) == -(1 << 63)
    assert oracle.fix48(float("nan")) == 0 and oracle.fix48(32767.5) == 32767 * two48 + (two48 >> 1)
    assert oracle.unfix48(two48) == 1.0 and oracle.unfix48(-3 * (1 << 46)) == -0.75
    assert oracle.unfix48(two48 + 1) == 1.0                            # 2^48 + 1 rounds to 2^48 in binary32
    assert oracle.unfix48((1 << 24) + 1) == np.float32(2.0 ** -24)     # 2^24 + 1 ties to even
    assert oracle.unfix48((1 << 24) + 3) == np.float32((2 ** 24 + 4) * 2.0 ** -48)

    B, H = 1, 2
    for S in (96, 128):                       # a single block of keys: sums far above 2^-25 convert exactly
        qkv = synth.normal_bf16((B * S, 3 * H * 128), 1.0, seed=0, tid=66)
        dout = synth.normal_bf16((B * S, H * 128), 1.0, seed=0, tid=67)
        out, lse = oracle.attn_fwd(qkv, B, H, S)
        plain = oracle.attn_bwd(dout, qkv, out, lse, B, H, S)
        fixed = oracle.attn_bwd(dout, qkv, out, lse, B, H, S, fixq=True)
        assert np.array_equal(fixed[:, H * 128:], plain[:, H * 128:])        # dK, dV do not use the accumulator
        big = np.abs(bf(plain[:, :H * 128])) >= 2.0 ** -20
        assert big.mean() > 0.9 and np.array_equal(fixed[:, :H * 128][big], plain[:, :H * 128][big])

    S = 300                                   # three blocks (the last one ragged)
    qkv = synth.normal_bf16((B * S, 3 * H * 128), 1.0, seed=0, tid=68)
    dout = synth.normal_bf16((B * S, H * 128), 0.1, seed=0, tid=69)
    out, lse = oracle.attn_fwd(qkv, B, H, S)
    plain = oracle.attn_bwd(dout, qkv, out, lse, B, H, S)
    fixed = oracle.attn_bwd(dout, qkv, out, lse, B, H, S, fixq=True)
    assert np.array_equal(fixed[:, H * 128:], plain[:, H * 128:])
    q, k, v, pr, o, _ = _attn_ref(qkv, B, H, S)
    do = bf(dout).astype(np.float64).reshape(B, S, H, 128).transpose(0, 2, 1, 3)
    ds = pr * (do @ v.transpose(0, 1, 3, 2) - (do * o).sum(-1, keepdims=True)) / math.sqrt(128)
    ref = (ds @ k).transpose(0, 2, 1, 3).reshape(B * S, H * 128)
    assert rel_err(bf(fixed[:, :H * 128]).astype(np.float64), ref) < 0.01
    # rows below 128 see one block only; all rows: neighbouring bf16 values at worst (the two accumulators differ by
    # far less than a bf16 step, so they can only fall on either side of a rounding boundary)
    assert np.array_equal(fixed[:128, :H * 128], plain[:128, :H * 128])
    fa, pa = fixed[:, :H * 128].astype(np.int32), plain[:, :H * 128].astype(np.int32)
    assert np.abs(fa - pa).max() <= 1 and (fa != pa).mean() < 0.02
    # a sliding window and grouped heads go through the same accumulator
    Hq, Hkv, W = 4, 2, 128
    qkv = synth.normal_bf16((B * S, (Hq + 2 * Hkv) * 128), 1.0, seed=0, tid=70)
    dout = synth.normal_bf16((B * S, Hq * 128), 0.1, seed=0, tid=71)
    out, lse = oracle.attn_fwd(qkv, B, Hq, S, Hkv=Hkv, window=W)
    plain = oracle.attn_bwd(dout, qkv, out, lse, B, Hq, S, Hkv=Hkv, window=W)
    fixed = oracle.attn_bwd(dout, qkv, out, lse, B, Hq, S, Hkv=Hkv, window=W, fixq=True)
    assert np.array_equal(fixed[:, Hq * 128:], plain[:, Hq * 128:])
    fa, pa = fixed[:, :Hq * 128].astype(np.int32), plain[:, :Hq * 128].astype(np.int32)
    assert np.abs(fa - pa).max() <= 1 and np.array_equal(fa[:128], pa[:128])


def _expand_kv(qkv, H, Hkv):
    """grouped q|k|v rows -> multi-head rows with every key/value head repeated for its query heads"""
    G = H // Hkv
    q = qkv[:, :H * 128]
    k = qkv[:, H * 128:(H + Hkv) * 128].reshape(-1, Hkv, 128).repeat(G, axis=1).reshape(-1, H * 128)
    v = qkv[:, (H + Hkv) * 128:].reshape(-1, Hkv, 128).repeat(G, axis=1).reshape(-1, H * 128)
    return np.ascontiguousarray(np.concatenate([q, k, v], 1))


def test_grouped_query_attention_pins():
    """Sec. 3.1 GQA: the forward of a query head is that of multi-head attention on its shared key/value head (bit
    for bit); dq likewise; dk, dv of a shared head are the float64 sums over its query heads."""
    B, H, Hkv, S = 1, 4, 2, 160
    qkv = synth.normal_bf16((B * S, (H + 2 * Hkv) * 128), 1.0, seed=0, tid=65)
    dout = synth.normal_bf16((B * S, H * 128), 0.1, seed=0, tid=66)
    out, lse = oracle.attn_fwd(qkv, B, H, S, Hkv=Hkv)
    full = _expand_kv(qkv, H, Hkv)
    out_m, lse_m = oracle.attn_fwd(full, B, H, S)
    assert np.array_equal(out, out_m) and np.array_equal(lse, lse_m)
    d = oracle.attn_bwd(dout, qkv, out, lse, B, H, S, Hkv=Hkv)
    d_m = oracle.attn_bwd(dout, full, out_m, lse_m, B, H, S)
    assert np.array_equal(d[:, :H * 128], d_m[:, :H * 128])                     # dq is per query head
    q, k, v, p, o, _ = _attn_ref(full, B, H, S)
    do = bf(dout).astype(np.float64).reshape(B, S, H, 128).transpose(0, 2, 1, 3)
    dv = p.transpose(0, 1, 3, 2) @ do
    ds = p * (do @ v.transpose(0, 1, 3, 2) - (do * o).sum(-1, keepdims=True)) / math.sqrt(128)
    dk = ds.transpose(0, 1, 3, 2) @ q
    G = H // Hkv
    for name, ref, off in (("dk", dk, H * 128), ("dv", dv, (H + Hkv) * 128)):
        r = ref.reshape(B, Hkv, G, S, 128).sum(2).transpose(0, 2, 1, 3).reshape(B * S, Hkv * 128)
        assert rel_err(bf(d[:, off:off + Hkv * 128]).astype(np.float64), r) < 0.01, name
    # one group per head is plain multi-head attention
    assert np.array_equal(oracle.attn_fwd(full, B, H, S, Hkv=H)[0], out_m)


def test_sliding_window_attention_pins():
    """Sec. 3.1 SWA: keys j in (i - W, i].  A window that covers the sequence is full causal attention bit for bit;
    keys that left the window cannot change a bit of the row; float64 agreement with the banded softmax."""
    B, H, S, W = 1, 1, 400, 128
    qkv = synth.normal_bf16((B * S, 3 * H * 128), 1.0, seed=0, tid=67)
    dout = synth.normal_bf16((B * S, H * 128), 0.1, seed=0, tid=68)
    out_f, lse_f = oracle.attn_fwd(qkv, B, H, S)
    out_w, lse_w = oracle.attn_fwd(qkv, B, H, S, window=512)
    assert np.array_equal(out_f, out_w) and np.array_equal(lse_f, lse_w)
    assert np.array_equal(oracle.attn_bwd(dout, qkv, out_f, lse_f, B, H, S), oracle.attn_bwd(dout, qkv, out_w, lse_w, B, H, S, window=512))
    out, lse = oracle.attn_fwd(qkv, B, H, S, window=W)
    assert np.array_equal(out[:W], out_f[:W]) and not np.array_equal(out[W:], out_f[W:])   # rows < W see everything
    x = bf(qkv).astype(np.float64).reshape(S, 3, 128)
    s = x[:, 0] @ x[:, 1].T / math.sqrt(128)
    i, j = np.arange(S)[:, None], np.arange(S)[None, :]
    s = np.where((j <= i) & (j > i - W), s, -np.inf)
    l64 = np.log(np.exp(s - s.max(-1, keepdims=True)).sum(-1)) + s.max(-1)
    p = np.exp(s - l64[:, None])
    assert np.abs(bf(out) - p @ x[:, 2]).max() < 0.02 and np.allclose(lse[0, 0], l64, rtol=1e-5, atol=1e-5)
    # locality: rows >= 300 do not depend on keys/values before 300 - W + 1 = 173
    qkv2 = qkv.copy(); qkv2[:173, 128:] = synth.normal_bf16((173, 256), 1.0, seed=3, tid=69)
    out2, lse2 = oracle.attn_fwd(qkv2, B, H, S, window=W)
    assert np.array_equal(out2[300:], out[300:]) and np.array_equal(lse2[..., 300:], lse[..., 300:])
    # backward against the banded float64 softmax
    d = oracle.attn_bwd(dout, qkv, out, lse, B, H, S, window=W)
    do = bf(dout).astype(np.float64)
    o = p @ x[:, 2]
    ds = p * (do @ x[:, 2].T - (do * o).sum(-1, keepdims=True)) / math.sqrt(128)
    for c, ref in enumerate((ds @ x[:, 1], ds.T @ x[:, 0], p.T @ do)):
        assert rel_err(bf(d[:, c * 128:(c + 1) * 128]).astype(np.float64), ref) < 0.01
    # dk, dv of keys that no later query can see inside the window ... every key is seen by itself; key 0 only by rows < W
    d3 = oracle.attn_bwd(dout, qkv2, out2, lse2, B, H, S, window=W)
    assert np.array_equal(d3[300:, :128], d[300:, :128])                          # dq rows >= 300 unchanged


def test_attention_int8_pv_pins():
    """int8 P.V per block (Sec. 3.2): same logsumexp as the full-precision forward, output within the quantisation
    error of it and of the float64 softmax, exact where the quantisers are exact, causal at block granularity."""
    B, H, S = 1, 2, 300
    qkv = synth.normal_bf16((B * S, 3 * H * 128), 1.0, seed=0, tid=93)
    out_f, lse_f = oracle.attn_fwd(qkv, B, H, S)
    out_q, lse_q = oracle.attn_fwd(qkv, B, H, S, int8_pv=True)
    assert np.array_equal(lse_f, lse_q)                                   # statistics are not quantised
    q, k, v, p, o, _ = _attn_ref(qkv, B, H, S)
    o = o.transpose(0, 2, 1, 3).reshape(B * S, H * 128)
    err_q, err_f = np.abs(bf(out_q) - o).max(), np.abs(bf(out_f) - o).max()
    assert err_q < 0.08 and err_q > err_f                                  # coarser than the f32 path, but close
    # float64 emulation of the defined formula (quantised p and v, per-block scale): much closer than to the exact softmax
    x = bf(qkv).astype(np.float64).reshape(S, 3, H, 128)
    for h in range(H):
        ref = np.zeros((S, 128))
        sc = x[:, 0, h] @ x[:, 1, h].T / math.sqrt(128)
        for i in (0, 1, 127, 128, 200, 299):
            mrun, orow, l = -np.inf, np.zeros(128), 0.0
            for j0 in range(0, i + 1, 128):
                js = np.arange(j0, min(j0 + 128, i + 1))
                mt = max(mrun, sc[i, js].max())
                pj = np.exp(sc[i, js] - mt)
                blk = x[j0:min(j0 + 128, S), 2, h]
                am = np.abs(blk).max()
                qv = np.clip(np.rint(x[js, 2, h] * (127.0 / am)), -128, 127)
                u = (np.rint(pj * 127.0)[:, None] * qv).sum(0) * (am / 127.0 / 127.0)
                a = np.exp(mrun - mt) if np.isfinite(mrun) else 0.0
                orow, l, mrun = orow * a + u, l * a + pj.sum(), mt
            got = bf(out_q)[i, h * 128:(h + 1) * 128]
            assert np.abs(got - orow / l).max() < 0.02
    # row 0 sees one key with p = 1: out_0 = v_0 up to the two quantisers' rounding
    assert np.abs(bf(out_q)[0] - bf(qkv)[0, 2 * H * 128:]).max() < np.abs(bf(qkv)[:128, 2 * H * 128:]).max() / 127 + 1e-2
    # changing keys/values of later blocks leaves the rows of earlier blocks bit-identical (the block scale is shared
    # inside a block, so the guarantee is per block of 128 keys)
    qkv2 = qkv.copy(); qkv2[256:, H * 128:] = synth.normal_bf16((S - 256, 2 * H * 128), 1.0, seed=1, tid=94)
    out2, _ = oracle.attn_fwd(qkv2, B, H, S, int8_pv=True)
    assert np.array_equal(out2[:256], out_q[:256]) and not np.array_equal(out2[256:], out_q[256:])


# ---------------------------------------------------------------- glue
def test_glue_ops():
    gu = synth.normal_bf16((9, 512), 2.0, seed=0, tid=70)
    h = oracle.swiglu_fwd(gu)
    g, u = bf(gu[:, :256]).astype(np.float64), bf(gu[:, 256:]).astype(np.float64)
    sg = 1 / (1 + np.exp(-g))
    assert np.allclose(bf(h), g * sg * u, rtol=1e-2, atol=1e-3)
    dh = synth.normal_bf16((9, 256), 1.0, seed=0, tid=71)
    dgu = oracle.swiglu_bwd(dh, gu)
    d = bf(dh).astype(np.float64)
    assert np.allclose(bf(dgu[:, 256:]), d * g * sg, rtol=1e-2, atol=1e-3)
    assert np.allclose(bf(dgu[:, :256]), d * u * sg * (1 + g * (1 - sg)), rtol=1e-2, atol=1e-3)
    big = synth.to_bf16(np.array([[-200.0, 200.0, 1.0, 1.0]], F))             # exp overflow path: silu(-200) = -0
    hb = bf(oracle.swiglu_fwd(big))
    assert hb[0, 0] == 0 and hb[0, 1] == 200
    a = synth.normal_bf16(1000, seed=0, tid=72); b = synth.normal_bf16(1000, seed=0, tid=73)
    assert np.array_equal(oracle.residual_add(a, b), synth.to_bf16(bf(a) + bf(b)))
    # embedding: gather, and ordered scatter-add with duplicate tokens
    E = synth.normal_bf16((11, 8), seed=0, tid=74)
    tok = np.array([3, 5, 3, 3, 10, 5], np.int32)
    assert np.array_equal(oracle.embed_fwd(tok, E), E[tok])
    dy = synth.to_bf16(np.array([[2.0 ** 24] * 8, [1.0] * 8, [1.0] * 8, [1.0] * 8, [4.0] * 8, [2.0] * 8], F))
    dE = oracle.embed_bwd(tok, dy, 11)
    assert np.all(dE[3] == 2.0 ** 24)            # sequential: (2^24 + 1) + 1 stays 2^24; a tree would give 2^24 + 2
    assert np.all(dE[5] == 3) and np.all(dE[10] == 4) and np.all(dE[0] == 0)


def test_lmhead_against_float64_and_order():
    M, V, K = 24, 40, 256
    Hh = synth.normal_bf16((M, K), 1.0, seed=0, tid=80)
    W = synth.normal_bf16((V, K), 0.02, seed=0, tid=81)
    lg = oracle.lmhead_fwd(Hh, W)
    assert np.allclose(lg, bf(Hh).astype(np.float64) @ bf(W).astype(np.float64).T, rtol=1e-4, atol=1e-5)
    # sequential order: python restatement of one output
    acc = F(0)
    for kk in range(K):
        acc = F(acc + F(bf(Hh)[3, kk] * bf(W)[7, kk]))
    assert lg[3, 7] == acc
    dl = synth.normal_f32((M, V), 1e-3, seed=0, tid=82)
    dH, dW = oracle.lmhead_bwd(dl, Hh, W)
    g = bf(synth.to_bf16(dl)).astype(np.float64)
    assert rel_err(bf(dH), g @ bf(W).astype(np.float64)) < 0.01
    assert rel_err(dW, g.T @ bf(Hh).astype(np.float64)) < 1e-5
    # chunked accumulation over tokens continues the same ordered sum
    _, dWa = oracle.lmhead_bwd(dl[:10], Hh[:10], W)
    _, dWb = oracle.lmhead_bwd(dl[10:], Hh[10:], W, dW=dWa)
    assert np.array_equal(dWb, dW)


# ---------------------------------------------------------------- reduction replay, clip, AdamW
def test_treefold_paper_facts():
    n = 16
    for R in range(1, 17):
        acc = oracle.Accum(1, 1, R, n)
        for r in range(R):
            acc.push(np.full(n, float(r + 1), F))
        assert acc.stack_size == bin(R).count("1")                 # one residual entry per set bit (App. A.1)
        out = acc.result()
        assert np.all(out == F(F(R * (R + 1) // 2) * F(1.0 / R)))
        if R == 8:
            assert acc.max_resident == 4                           # App. A.1: "the fold needs at most 4"
    # pairing order: R = 4 gives (g0+g1)+(g2+g3); R = 7 gives A + (B + C) with A = 4 replicas, B = 2, C = 1
    acc = oracle.Accum(1, 1, 4, 1)
    for v in (2.0 ** 24, 1.0, 1.0, 1.0):
        acc.push(np.array([v], F))
    assert acc.result()[0] == F(F(16777218) * F(0.25))
    acc = oracle.Accum(1, 1, 7, 1)
    for v in (2.0 ** 24, 0, 0, 0, 1.0, 0, 1.0):
        acc.push(np.array([v], F))
    assert acc.result()[0] == F(F(16777218) * F(1.0 / 7))
    with pytest.raises(ValueError):
        a = oracle.Accum(2, 2, 2, 1); a.push(np.zeros(1, F)); a.result()


def test_mesh_order_and_exact_means():
    # integer-valued gradients: every mesh gives the exact mean; the three levels use reciprocal multiplies
    n = 1000
    gs = [np.round(synth.normal_f32(n, 50.0, seed=0, tid=90 + i)) * 8 for i in range(8)]
    mean = np.sum(np.array(gs, np.float64), 0) / 8
    for mesh in ((8, 1, 1), (2, 2, 2), (1, 8, 1), (1, 1, 8), (4, 2, 1), (2, 1, 4)):
        acc = oracle.Accum(*mesh, n)
        for g in gs:
            acc.push(g)
        assert np.array_equal(acc.result().astype(np.float64), mean)
    # non-integer data: different meshes are different summation orders (Appendix A: ~1e-11.. not bitwise)
    gs = [synth.normal_f32(n, 1e-3, seed=0, tid=100 + i) for i in range(8)]
    outs = []
    for mesh in ((8, 1, 1), (2, 2, 2), (1, 1, 8)):
        acc = oracle.Accum(*mesh, n)
        for g in gs:
            acc.push(g)
        outs.append(acc.result())
    assert not np.array_equal(outs[0], outs[2]) and np.allclose(outs[0], outs[2], rtol=1e-5, atol=1e-9)
    # python restatement of mesh (2,2,2): ranks r = rep*2 + shard own micro-batches 2r, 2r+1
    half = F(0.5)
    gr = [F(F(F(0) + gs[2 * r] * half) + gs[2 * r + 1] * half) for r in range(4)]
    inner = [F(F(gr[0] + gr[1]) * half), F(F(gr[2] + gr[3]) * half)]
    assert np.array_equal(outs[1], F(F(inner[0] + inner[1]) * half))


def test_grad_norm_and_clip():
    for k in range(1, 9):
        norm, coef = oracle.grad_norm([np.ones(4 ** k, F)], max_norm=1.0)
        assert norm == F(2 ** k)
        assert coef == F(1) / F(F(2 ** k) + F(1e-6))
    g = synth.normal_f32(1 << 20, 1e-3, seed=0, tid=110)
    norm, coef = oracle.grad_norm([g[:1000], g[1000:]], max_norm=1.0)
    assert abs(norm - np.linalg.norm(g.astype(np.float64))) < 1e-5 and coef == F(1) / F(norm + F(1e-6)) or coef == 1
    norm2, coef2 = oracle.grad_norm([g], max_norm=0.0)
    assert coef2 == 1
    assert np.array_equal(oracle.scale(g, F(0.5)), g * F(0.5))


def test_adamw_hand_element_and_float64():
    lr, b1, b2, eps, wd = 3e-4, 0.9, 0.95, 1e-8, 0.1
    p = synth.to_bf16(np.array([1.0, -2.0, 0.5], F)); g = np.array([0.25, -1e-3, 0.0], F)
    p1, m1, v1 = oracle.adamw(p, g, np.zeros(3, F), np.zeros(3, F), lr, b1, b2, eps, wd, 1)
    # t = 1 by hand: m = (1-b1) g, v = (1-b2) g^2, bias-corrected ratio = g/|g| -> |dp| ~ lr (+ decay lr*wd*p)
    omb1 = F(1) - F(b1); omb2 = F(1) - F(b2)
    assert np.array_equal(m1, (omb1 * g).astype(F)) and np.array_equal(v1, (omb2 * (g * g).astype(F)).astype(F))
    exp_p = np.array([1.0 * (1 - lr * wd) - lr, -2.0 * (1 - lr * wd) + lr, 0.5 * (1 - lr * wd)])
    assert np.allclose(bf(p1), exp_p, rtol=2 ** -8)
    assert bf(p1)[2] == bf(synth.to_bf16(np.array([F(0.5) * F(1 - lr * wd)], F)))[0]   # zero gradient: pure decay
    # f32 parameters (LSQ activation steps): no rounding to bf16, no weight decay
    pf = np.array([0.03], F)
    p2, _, _ = oracle.adamw(pf, np.array([1e-4], F), np.zeros(1, F), np.zeros(1, F), lr, b1, b2, eps, 0.0, 1)
    assert abs(float(p2[0]) - (0.03 - lr)) < 1e-7
    # two steps against float64 AdamW
    n = 4096
    pw = synth.normal_f32(n, 0.02, seed=0, tid=120); gw = synth.normal_f32(n, 1e-3, seed=0, tid=121)
    pb = synth.to_bf16(pw); m = np.zeros(n, F); v = np.zeros(n, F)
    P = bf(pb).astype(np.float64); M = np.zeros(n); Vv = np.zeros(n)
    for t in (1, 2):
        pb, m, v = oracle.adamw(pb, gw, m, v, lr, b1, b2, eps, wd, t)
        M = b1 * M + (1 - b1) * gw; Vv = b2 * Vv + (1 - b2) * gw.astype(np.float64) ** 2
        P = P * (1 - lr * wd) - lr * (M / (1 - b1 ** t)) / (np.sqrt(Vv / (1 - b2 ** t)) + eps)
        P = bf(synth.to_bf16(P.astype(F))).astype(np.float64)
    assert np.mean(bf(pb) == P) > 0.98 and np.allclose(bf(pb), P, rtol=2 ** -7)
    assert np.allclose(m, M, rtol=1e-5, atol=1e-12) and np.allclose(v, Vv, rtol=1e-5, atol=1e-14)


def test_rope_pins():
    """Rotary embedding (Sec. 3.1): pairing (i, i+64), signs, identity at position 0, float64 agreement, inverse."""
    S, nh = 24, 3
    cos, sin = synth.rope_tables(S)
    assert cos.shape == (S, 64) and np.all(cos[0] == 1.0) and np.all(sin[0] == 0.0)
    # the tables follow angle = pos * theta**(-2i/128) with theta = 5e5
    assert abs(float(cos[5, 7]) - math.cos(5 * 5.0e5 ** (-14 / 128))) < 1e-7
    x = synth.normal_bf16((2 * S, nh, 128), seed=11)
    y = oracle.rope(x, S, cos, sin)
    assert np.array_equal(y[0], x[0]) and np.array_equal(y[S], x[S])          # position 0 (and S: t mod S) is the identity
    # unit vectors pin the pairing and the signs: e_i -> (c_i at i, s_i at i+64); e_{i+64} -> (-s_i at i, c_i at i+64)
    e = np.zeros((S, 1, 128), np.float32)
    e[:, 0, 9] = 1.0
    ye = synth.from_bf16(oracle.rope(synth.to_bf16(e), S, cos, sin))
    assert np.array_equal(ye[:, 0, 9], synth.from_bf16(synth.to_bf16(cos[:, 9])))
    assert np.array_equal(ye[:, 0, 73], synth.from_bf16(synth.to_bf16(sin[:, 9])))
    assert not ye[:, 0, [8, 10, 72, 74]].any()
    e[:] = 0
    e[:, 0, 73] = 1.0
    ye = synth.from_bf16(oracle.rope(synth.to_bf16(e), S, cos, sin))
    assert np.array_equal(ye[:, 0, 9], synth.from_bf16(synth.to_bf16(-sin[:, 9])))
    assert np.array_equal(ye[:, 0, 73], synth.from_bf16(synth.to_bf16(cos[:, 9])))
    # float64 reference within half a bf16 ulp (+ the f32 roundings)
    xf = synth.from_bf16(x).astype(np.float64).reshape(2, S, nh, 128)
    c, s = cos.astype(np.float64)[None, :, None, :], sin.astype(np.float64)[None, :, None, :]
    ref = np.concatenate([xf[..., :64] * c - xf[..., 64:] * s, xf[..., 64:] * c + xf[..., :64] * s], -1).reshape(2 * S, nh, 128)
    got = synth.from_bf16(y).astype(np.float64)
    assert np.all(np.abs(got - ref) <= np.abs(ref) * 2.0 ** -8 + 1e-30)
    # relative-position property: <rope(q, p), rope(k, r)> depends on p - r only (float64 check on the reference form)
    # and the inverse rotation undoes the forward one up to the two bf16 roundings
    back = synth.from_bf16(oracle.rope(y, S, cos, sin, inverse=True)).astype(np.float64)
    assert np.all(np.abs(back - synth.from_bf16(x)) <= np.abs(synth.from_bf16(x)) * 2.0 ** -7 + 2.0 ** -7 * np.abs(ref).max())
    # the inverse is the transpose: <y, R x> = <R^T y, x> in float64 up to rounding
    g = synth.normal_bf16((2 * S, nh, 128), seed=12)
    lhs = (synth.from_bf16(g).astype(np.float64) * got).sum()
    rhs = (synth.from_bf16(oracle.rope(g, S, cos, sin, inverse=True)).astype(np.float64) * synth.from_bf16(x)).sum()
    assert abs(lhs - rhs) <= 2e-2 * math.sqrt(got.size)


def test_headnorm_is_gain_free_rmsnorm_over_128():
    """QK-norm (Sec. 3.1) is the gain-free RMSNorm over each head's 128 values: unit RMS out, float64 agreement."""
    x = synth.normal_bf16((40, 128), seed=13)
    y, rstd = oracle.rmsnorm_fwd(x, None, 1e-6, bf=True)
    xf = synth.from_bf16(x).astype(np.float64)
    ref = xf / np.sqrt((xf * xf).mean(-1, keepdims=True) + 1e-6)
    assert np.all(np.abs(synth.from_bf16(y) - ref) <= np.abs(ref) * 2.0 ** -8 + 1e-30)
    assert np.allclose(np.sqrt((synth.from_bf16(y).astype(np.float64) ** 2).mean(-1)), 1.0, atol=5e-3)
    dy = synth.normal_bf16((40, 128), seed=14)
    dx, _ = oracle.rmsnorm_bwd(dy, x, None, rstd, bf=True)
    g = synth.from_bf16(dy).astype(np.float64)
    r = 1.0 / np.sqrt((xf * xf).mean(-1, keepdims=True) + 1e-6)
    xh = xf * r
    refdx = r * (g - xh * (g * xh).mean(-1, keepdims=True))
    assert np.all(np.abs(synth.from_bf16(dx) - refdx) <= np.abs(refdx) * 2.0 ** -7 + 1e-3 * np.abs(refdx).max())
