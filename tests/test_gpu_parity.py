"""GPU parity: every C-ABI entry point against the CPU oracle, bit for bit (0 ULP), on seeded inputs that
span several tiles and ragged tails."""
import ctypes

import numpy as np
import pytest

import oracle
import synth
from gpu_util import assert_same_bits, dev, empty, host, ws

pytestmark = pytest.mark.gpu
F = np.float32


@pytest.fixture(scope="module")
def det():
    import torch
    import paper_2609_17380_b200 as d
    d.load()
    assert torch.cuda.is_available()
    return d


def _sync():
    import torch
    torch.cuda.synchronize()


# ------------------------------------------------------------------ primitives
def test_primitives_bitwise(det):
    rng = np.random.default_rng(0)
    a = np.concatenate([synth.normal_f32(200000, 10.0, seed=1, tid=1), rng.uniform(-90, 90, 200000).astype(F),
                        np.array([0.0, -0.0, 1.0, -1.0, 2.0 ** -126, 2.0 ** -127, -2.0 ** -140, 2.0 ** -149, 88.7, 88.73, -87.3,
                                  -87.34, -100.0, 3.4e38, -np.inf, np.inf], F)])
    b = np.concatenate([synth.normal_f32(200000, 1e-20, seed=1, tid=2), rng.uniform(0.1, 4, 200000).astype(F),
                        np.array([1.0, 1.0, 2.0 ** -126, 0.5, 0.5, 2.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 10.0, 1.0, 1.0], F)])
    da, db, out = dev(a), dev(b), empty(a.shape, F)
    for name, op in oracle.OPS.items():
        x, y = a, b
        if name in ("sqrt", "log"):
            x = np.abs(a) + F(2.0 ** -100)
            x[~np.isfinite(x)] = 1.0
            da = dev(x)
        else:
            da = dev(a)
        det.det_test_prim(op, da, db, out)
        _sync()
        assert_same_bits(host(out), oracle.prim(name, x, y), "prim " + name)


def test_max_of_signed_zeros(det):
    a = np.array([0.0, -0.0, -0.0, 0.0], F)
    b = np.array([-0.0, 0.0, -0.0, 0.0], F)
    out = empty(a.shape, F)
    det.det_test_prim(oracle.OPS["max"], dev(a), dev(b), out)
    _sync()
    assert_same_bits(host(out), oracle.prim("max", a, b), "max of zeros")


def test_flush_boundary_probe(det):
    # products whose exact value lies just below 2^-126: rounding to the minimum normal must be kept on both sides
    fh = float.fromhex
    a = np.array([fh('0x1.fffffep-1'), fh('0x1.fffffcp-1'), fh('0x1.000002p+0'), fh('0x1.8p-1')], F)
    b = np.array([2.0 ** -126, 2.0 ** -126, fh('0x1.fffffep-1') * 2.0 ** -126, 2.0 ** -126], F)
    out = empty(a.shape, F)
    det.det_test_prim(oracle.OPS["mul"], dev(a), dev(b), out)
    _sync()
    assert_same_bits(host(out), oracle.prim("mul", a, b), "ftz boundary")
    # quotients: exact value (1 - 2^-24) * 2^-126 is a tie that IEEE would round up to the minimum normal
    a = np.array([fh('0x1.fffffep-1'), fh('0x1.fffffep-1'), 1.0, fh('0x1.fffffep-100'), 3.0], F)
    b = np.array([2.0 ** 126, 2.0 ** 125, 2.0 ** 126, 2.0 ** 27, fh('0x1.8p+127')], F)
    out = empty(a.shape, F)
    det.det_test_prim(oracle.OPS["div"], dev(a), dev(b), out)
    _sync()
    assert_same_bits(host(out), oracle.prim("div", a, b), "ftz boundary (div)")


def test_exp_all_bf16_arguments(det):
    h = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    x = oracle.bf2f(h)
    x = x[np.isfinite(x)]
    out = empty(x.shape, F)
    det.det_test_prim(oracle.OPS["exp"], dev(x), None, out)
    _sync()
    assert_same_bits(host(out), oracle.prim("exp", x), "exp")


def test_exp_for_softmax_arguments_has_the_bits_of_exp(det):
    """The softmax kernels evaluate the exponential of z - max <= 0 with the overflow range left out (test op 10): on
    every non-positive bf16 value, a dense grid over [-110, 0], every float near the flush threshold, near 0 and near
    the points where k changes, -inf and the negative subnormals it must give exactly the oracle's exp."""
    h = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    xb = oracle.bf2f(h)
    xb = xb[np.isfinite(xb) & (xb <= 0)]
    grid = np.linspace(-110.0, 0.0, 400001).astype(F)
    ends = []
    for c in (float.fromhex("-0x1.5d58a0p+6"), -0.0, -0.34657359, -1.0397208, -87.0, -1.0, -86.98):
        b = np.array([c], F).view(np.int32)[0]
        ends.append((np.arange(-40, 41, dtype=np.int64) + int(b)).astype(np.int32).view(F))
    x = np.concatenate([xb, grid] + ends + [np.array([-np.inf, -3.0e38, -1e-45, -1e-30, -0.0, 0.0], F)])
    x = x[~np.isnan(x)]
    x = x[x <= 0]
    out = empty(x.shape, F)
    det.det_test_prim(10, dev(x), None, out)
    _sync()
    assert_same_bits(host(out), oracle.prim("exp", x), "exp for arguments <= 0")


def test_exp_dense_grid_and_ends_of_the_range(det):
    """A dense f32 grid over [-100, 100], every float within a few ULP of the two thresholds of the definition (the
    largest argument with a finite result, the smallest with a non-zero one), of 0 and of the points where k changes,
    and the infinities: bit for bit (the device evaluates the sequence with selects instead of branches)."""
    grid = np.linspace(-100.0, 100.0, 400001).astype(F)
    ends = []
    for c in (float.fromhex("0x1.62e42ep+6"), float.fromhex("-0x1.5d58a0p+6"), 0.0, 0.34657359, -0.34657359, 88.0, -87.0, 1.0, -1.0):
        b = np.array([c], F).view(np.int32)[0]
        ends.append((np.arange(-40, 41, dtype=np.int64) + int(b)).astype(np.int32).view(F))
    x = np.concatenate([grid] + ends + [np.array([np.inf, -np.inf, 3.0e38, -3.0e38, 1e-45, -1e-45, 1e-30], F)])
    x = x[~np.isnan(x)]                       # the patterns just below +0 are NaNs; their payloads are not defined
    out = empty(x.shape, F)
    det.det_test_prim(oracle.OPS["exp"], dev(x), None, out)
    _sync()
    assert_same_bits(host(out), oracle.prim("exp", x), "exp")


def test_log_ends_of_the_domain_and_nan_logits(det):
    """det_log keeps a non-finite or non-positive argument visible; a NaN logit therefore gives a NaN loss, not a finite
    number that depends on the NaN's payload.  NaNs are compared as NaNs, everything else bit for bit."""
    import torch
    x = np.array([0.0, -0.0, 1e-40, np.inf, -1.0, -np.inf, np.nan, 1.0, 2.5, 50304.0], F)
    out = empty(x.shape, F)
    det.det_test_prim(oracle.OPS["log"], dev(x), None, out)
    _sync()
    got, want = host(out), oracle.prim("log", x)
    assert np.array_equal(np.isnan(got), np.isnan(want))
    assert np.array_equal(got[~np.isnan(got)].view(np.uint32), want[~np.isnan(want)].view(np.uint32))
    z = synth.normal_f32((6, 1000), 1.0, seed=31, tid=1)
    z[1, 10] = np.nan
    z[2, 20] = np.inf
    z[3, 30] = -np.inf
    z[4, :] = -np.inf
    tgt = np.array([5, 7, 9, 11, 13, 999], np.int32)
    lr, l2, lm, zm = empty((6,), F), empty((6,), F), empty((1,), F), empty((1,), F)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    det.det_xent_fwd(dev(z), dev(tgt), 6, 1000, 1e-4, lr, l2, lm, zm, ws(det.det_xent_ws_bytes(6, 1000)), status)
    _sync()
    olr, ol2, olm, ozm, _ = oracle.xent_fwd(z, tgt, 1e-4)
    for g, w, name in ((host(lr), olr, "loss_row"), (host(l2), ol2, "lse"), (host(lm), olm, "mean")):
        w = np.asarray(w, F).reshape(g.shape)
        assert np.array_equal(np.isnan(g), np.isnan(w)), name
        assert np.array_equal(g[~np.isnan(g)].view(np.uint32), w[~np.isnan(w)].view(np.uint32)), name
    assert np.isnan(host(lr)[1]) and np.isnan(host(lm)[0])


# ------------------------------------------------------------------ sums
@pytest.mark.parametrize("n", [0, 1, 2, 7, 255, 256, 257, 16383, 16384, 16385, 50304, 1000003, 16384 * 300 + 17])
def test_det_sum_lengths(det, n):
    x = synth.normal_f32(max(n, 1), 1.0, seed=2, tid=n % 97)[:n]
    dx = dev(x) if n else empty((4,), F)
    out = empty((1,), F)
    w = ws(det.det_sum_ws_bytes(n))
    for sq in (0, 1):
        det.det_sum(dx, n, sq, out, w)
        _sync()
        want = oracle.sumsq(x) if sq else oracle.det_sum(x)
        assert_same_bits(host(out), np.array([want], F), "det_sum n=%d sq=%d" % (n, sq))


def test_det_sum_order_pins_on_device(det):
    out = empty((1,), F)
    w = ws(256)
    for v, want in (([2.0 ** 24, 1, 1, 1], 16777218.0), ([2.0 ** 24, 0, 0, 0, 1, 0, 1], 16777218.0),
                    ([1, 2.0 ** 24, 0, 0, 0, 0, 1], 16777216.0)):
        x = np.array(v, F)
        det.det_sum(dev(np.concatenate([x, np.zeros(8, F)])), x.size, 0, out, w)
        _sync()
        assert host(out)[0] == F(want)
    x = np.full(5, -0.0, F)
    det.det_sum(dev(np.concatenate([x, np.zeros(3, F)])), 5, 0, out, w)
    _sync()
    assert host(out).view(np.uint32)[0] == 0x80000000


def test_grad_norm_and_scale(det):
    sizes = [4, 1000, 16384, 70001 * 4, 3 * 16384 + 12]
    gs = [synth.normal_f32(s, 1e-3, seed=3, tid=i) for i, s in enumerate(sizes)]
    dg = [dev(g) for g in gs]
    norm, coef = empty((1,), F), empty((1,), F)
    w = ws(det.det_grad_norm_ws_bytes(dg))
    for mx in (1.0, 1e-3, 0.0):
        det.det_grad_norm(dg, mx, norm, coef, w)
        _sync()
        on, oc = oracle.grad_norm(gs, mx)
        assert_same_bits(host(norm), np.array([on], F), "norm")
        assert_same_bits(host(coef), np.array([oc], F), "coef")
    det.det_grad_norm(dg, 1e-3, norm, coef, w)
    det.det_scale_inplace(dg[3], sizes[3], coef)
    _sync()
    assert_same_bits(host(dg[3]), oracle.scale(gs[3], oracle.grad_norm(gs, 1e-3)[1]), "scale")
    # all-ones of length 4^k has norm 2^k exactly
    ones = dev(np.ones(4 ** 9, F))
    det.det_grad_norm([ones], 1.0, norm, coef, ws(det.det_grad_norm_ws_bytes([ones])))
    _sync()
    assert host(norm)[0] == 512.0


# ------------------------------------------------------------------ RMSNorm
@pytest.mark.parametrize("bf,rows,D,gain", [(False, 300, 2048, True), (True, 300, 2048, True), (False, 33, 1000, False),
                                            (True, 17, 4096, True), (False, 9, 8, True), (True, 513, 256, False)])
def test_rmsnorm(det, bf, rows, D, gain):
    x = synth.normal_f32((rows, D), 1.0, seed=4, tid=1)
    g = (1 + synth.normal_f32(D, 0.02, seed=4, tid=2)) if gain else None
    dy = synth.normal_f32((rows, D), 1.0, seed=4, tid=3)
    if bf:
        x, dy = synth.to_bf16(x), synth.to_bf16(dy)
        g = synth.to_bf16(g) if gain else None
    dt = np.uint16 if bf else F
    y, rstd = empty((rows, D), dt), empty((rows,), F)
    dg_ = dev(g) if gain else None
    det.det_rmsnorm_fwd(int(bf), dev(x), dg_, rows, D, 1e-6, y, rstd)
    _sync()
    oy, orstd = oracle.rmsnorm_fwd(x, g, 1e-6, bf=bf)
    assert_same_bits(host(rstd), orstd, "rstd")
    assert_same_bits(host(y, dt), oy, "y")
    dx, dgam = empty((rows, D), dt), empty((D,), F)
    det.det_rmsnorm_bwd(int(bf), dev(dy), dev(x), dg_, rstd, rows, D, dx, dgam, ws(det.det_rmsnorm_bwd_ws_bytes(rows, D)))
    _sync()
    odx, odg = oracle.rmsnorm_bwd(dy, x, g, orstd, bf=bf)
    assert_same_bits(host(dx, dt), odx, "dx")
    assert_same_bits(host(dgam), odg, "dgamma")


# ------------------------------------------------------------------ per-head norm and rotary embedding
@pytest.mark.parametrize("T,nh,pad,S", [(300, 4, 0, 100), (129, 3, 256, 64), (7, 1, 8, 7)])
def test_headnorm_and_rope(det, T, nh, pad, S):
    """Rows of 128 inside wider token rows (stride = nh*128 + pad), against the oracle on the gathered rows."""
    ld = nh * 128 + pad
    buf = synth.normal_bf16((T, ld), seed=21)
    buf[::5, 3] = 0x0001                                        # a few subnormal and tiny inputs
    buf[1::7, 64] = synth.to_bf16(np.array([2.0 ** -70], F))[0]
    dyb = synth.normal_bf16((T, ld), seed=22)
    x = np.ascontiguousarray(buf[:, :nh * 128]).reshape(T * nh, 128)
    dy = np.ascontiguousarray(dyb[:, :nh * 128]).reshape(T * nh, 128)
    # forward norm into a second strided buffer
    ybuf, rstd = dev(np.zeros((T, ld), np.uint16)), empty((T * nh,), F)
    det.det_headnorm_fwd(dev(buf), ld, T, nh, 1e-6, ybuf, ld, rstd)
    _sync()
    oy, orstd = oracle.rmsnorm_fwd(x, None, 1e-6, bf=True)
    assert_same_bits(host(rstd), orstd, "headnorm rstd")
    gy = host(ybuf, np.uint16)
    assert_same_bits(gy[:, :nh * 128].reshape(T * nh, 128), oy, "headnorm y")
    assert not gy[:, nh * 128:].any()                           # nothing written outside the heads
    dxbuf = dev(np.zeros((T, ld), np.uint16))
    det.det_headnorm_bwd(dev(dyb), ld, dev(buf), ld, rstd, T, nh, dxbuf, ld)
    _sync()
    odx, _ = oracle.rmsnorm_bwd(dy, x, None, orstd, bf=True)
    assert_same_bits(host(dxbuf, np.uint16)[:, :nh * 128].reshape(T * nh, 128), odx, "headnorm dx")
    # rotary embedding, forward out of place and inverse in place
    cos, sin = synth.rope_tables(S)
    dc, ds = dev(cos), dev(sin)
    rbuf = dev(np.zeros((T, ld), np.uint16))
    det.det_rope(dev(buf), ld, T, nh, S, dc, ds, 0, rbuf, ld)
    _sync()
    orot = oracle.rope(x.reshape(T, nh, 128), S, cos, sin)
    assert_same_bits(host(rbuf, np.uint16)[:, :nh * 128].reshape(T, nh, 128), orot, "rope")
    det.det_rope(rbuf, ld, T, nh, S, dc, ds, 1, rbuf, ld)
    _sync()
    oinv = oracle.rope(orot, S, cos, sin, inverse=True)
    assert_same_bits(host(rbuf, np.uint16)[:, :nh * 128].reshape(T, nh, 128), oinv, "rope inverse in place")


# ------------------------------------------------------------------ cross-entropy
@pytest.mark.parametrize("rows,V,zw", [(24, 50304, 0.0), (8, 50304, 1e-4), (5, 1000, 0.0), (3, 4, 0.0), (2, 128256, 1e-4)])
def test_xent(det, rows, V, zw):
    z = synth.normal_f32((rows, V), 2.0, seed=5, tid=1)
    t = synth.randint(rows, V, seed=5, tid=2)
    dz = dev(z)
    dt_ = dev(t)
    loss_row, lse, lm, zm = empty((rows,), F), empty((rows,), F), empty((1,), F), empty((1,), F)
    import torch
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    det.det_xent_fwd(dz, dt_, rows, V, zw, loss_row, lse, lm, zm, ws(det.det_xent_ws_bytes(rows, V)), status)
    _sync()
    ol, olse, olm, ozm, bad = oracle.xent_fwd(z, t, zw)
    assert bad == 0 and int(status.item()) == 0
    assert_same_bits(host(lse), olse, "lse")
    assert_same_bits(host(loss_row), ol, "loss_row")
    assert_same_bits(host(lm), olm, "loss_mean")
    assert_same_bits(host(zm), ozm, "z_mean")
    det.det_xent_bwd(dz, dt_, lse, rows, V, zw, 1.0 / 64)
    _sync()
    assert_same_bits(host(dz), oracle.xent_bwd(z, t, olse, zw, 1.0 / 64), "dlogits")


def test_xent_backward_with_a_foreign_logsumexp(det):
    """det_xent_bwd takes lse as an input: with values below a row's own logsumexp some arguments z - lse are positive
    (up to the overflow of exp), and the kernel must leave its shortcut for non-positive arguments; with values far above,
    every probability underflows.  Both against the oracle, bit for bit, on a width with a ragged last block."""
    rows, V = 24, 6 * 2048 + 1024 + 36
    z = synth.normal_f32((rows, V), 2.0, seed=3, tid=70)
    t = synth.randint(rows, V, seed=3, tid=71)
    _, olse, _, _, _ = oracle.xent_fwd(z, t, 0.0)
    lse = olse.copy()
    lse[0::4] -= 3.0                       # some positive arguments
    lse[1::4] -= 95.0                      # arguments up to the edge of the overflow range
    lse[3::4] -= 110.0                     # exp overflows for the largest logits
    lse[2::4] += 100.0                     # every probability flushes to 0
    for zw in (0.0, 1e-4):
        dz = dev(z)
        det.det_xent_bwd(dz, dev(t), dev(lse), rows, V, zw, 0.5)
        _sync()
        got, want = host(dz), oracle.xent_bwd(z, t, lse, zw, 0.5)
        assert np.array_equal(np.isnan(got), np.isnan(want))
        fin = ~np.isnan(want)
        assert_same_bits(got[fin], want[fin], "dlogits with a foreign lse")
        assert np.all(want[2][np.arange(V) != t[2]] == 0) and not np.all(np.isfinite(want[3]))


def test_xent_closed_forms_and_bad_target(det):
    import torch
    V = 50304
    z = np.full((2, V), 3.25, F)
    t = np.array([7, V], np.int32)                 # second target is out of range
    loss_row, lse, lm, zm = empty((2,), F), empty((2,), F), empty((1,), F), empty((1,), F)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    det.det_xent_fwd(dev(z), dev(t), 2, V, 0.0, loss_row, lse, lm, zm, ws(det.det_xent_ws_bytes(2, V)), status)
    _sync()
    assert int(status.item()) & det.DEV_TARGET
    ol, olse, olm, _, bad = oracle.xent_fwd(z, t)
    assert bad == 1
    assert_same_bits(host(loss_row), ol, "loss")
    assert abs(float(host(loss_row)[0]) - np.log(V)) < 2e-6 and host(loss_row)[1] == 0


# ------------------------------------------------------------------ glue
def test_glue(det):
    rows, Fd = 37, 1024
    gu = synth.normal_bf16((rows, 2 * Fd), 2.0, seed=6, tid=1)
    gu[0, :4] = synth.to_bf16(np.array([-200.0, 200.0, 90.0, -90.0], F))
    dh = synth.normal_bf16((rows, Fd), 1.0, seed=6, tid=2)
    h = empty((rows, Fd), np.uint16)
    det.det_swiglu_fwd(dev(gu), rows, Fd, h)
    dgu = empty((rows, 2 * Fd), np.uint16)
    det.det_swiglu_bwd(dev(dh), dev(gu), rows, Fd, dgu)
    _sync()
    assert_same_bits(host(h, np.uint16), oracle.swiglu_fwd(gu), "swiglu")
    assert_same_bits(host(dgu, np.uint16), oracle.swiglu_bwd(dh, gu), "swiglu bwd")
    a = synth.normal_bf16(40000, 1.0, seed=6, tid=3)
    b = synth.normal_bf16(40000, 1.0, seed=6, tid=4)
    y = empty((40000,), np.uint16)
    det.det_residual_add(dev(a), dev(b), 40000, y)
    _sync()
    assert_same_bits(host(y, np.uint16), oracle.residual_add(a, b), "residual")


def test_producers_write_the_next_linears_int8_input(det):
    """The activation quantiser fused into RMSNorm, SwiGLU and the attention forward: the int8 copy equals the oracle's
    quantiser applied to the producer's bf16 output, the bf16 output itself is untouched, and the linear that takes the
    codes ready-made equals the oracle's linear forward.  Steps are chosen so that values saturate on both sides."""
    import torch
    rows, D = 264, 512
    x = synth.normal_bf16((rows, D), 3.0, seed=41, tid=1)
    g = synth.to_bf16(1 + synth.normal_f32(D, 0.02, seed=41, tid=2))
    s = np.array([0.021], F)
    y, rstd, qy = empty((rows, D), np.uint16), empty((rows,), F), empty((rows, D), np.int8)
    det.det_rmsnorm_fwd_q(dev(x), dev(g), rows, D, 1e-6, y, rstd, dev(s), qy)
    _sync()
    oy, orstd = oracle.rmsnorm_fwd(x, g, 1e-6, bf=True)
    assert_same_bits(host(y, np.uint16), oy, "rmsnorm y")
    assert_same_bits(host(rstd), orstd, "rstd")
    assert_same_bits(host(qy), oracle.lsq_quantize(oy, s, False), "rmsnorm int8 copy")
    assert (host(qy) == 127).any() and (host(qy) == -128).any()
    # SwiGLU
    Fd = 768
    gu = synth.normal_bf16((rows, 2 * Fd), 2.0, seed=41, tid=3)
    s2 = np.array([0.013], F)
    h, qh = empty((rows, Fd), np.uint16), empty((rows, Fd), np.int8)
    det.det_swiglu_fwd_q(dev(gu), rows, Fd, h, dev(s2), qh)
    _sync()
    oh = oracle.swiglu_fwd(gu)
    assert_same_bits(host(h, np.uint16), oh, "swiglu h")
    assert_same_bits(host(qh), oracle.lsq_quantize(oh, s2, False), "swiglu int8 copy")
    # attention (full causal and a sliding window), then the output projection on the ready-made codes
    B, H, S = 2, 2, 320
    HD = H * 128
    qkv = synth.normal_bf16((B * S, 3 * HD), 1.0, seed=41, tid=4)
    dq = dev(qkv)
    base = dq.data_ptr()
    s3 = np.array([0.004], F)
    for window in (0, 128):
        out, lse, qo = empty((B * S, HD), np.uint16), empty((B, H, S), F), empty((B * S, HD), np.int8)
        det.det_attn_fwd_q(base, base + 2 * HD, base + 4 * HD, 3 * HD, B, H, S, out, HD, lse, dev(s3), qo, window=window)
        _sync()
        oout, olse = oracle.attn_fwd(qkv, B, H, S, window=window)
        assert_same_bits(host(out, np.uint16), oout, "attention out")
        assert_same_bits(host(lse), olse, "lse")
        assert_same_bits(host(qo), oracle.lsq_quantize(oout, s3, False), "attention int8 copy")
    N = 384
    W = synth.normal_bf16((N, HD), 0.02, seed=41, tid=5)
    osw = oracle.lsq_weight_scale(W)
    qW = empty((N, HD), np.int8)
    det.det_lsq_quantize_weight(dev(W), dev(osw), N, HD, 128, qW, None, None, ws(256))
    Y = empty((B * S, N), np.uint16)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    det.det_linear_fwd_q(qo, qW, dev(s3), dev(osw), B * S, N, HD, Y, status)
    _sync()
    oY, _, _ = oracle.linear_fwd(oout, W, s3, osw)
    assert int(status.item()) == 0
    assert_same_bits(host(Y, np.uint16), oY, "linear on ready-made codes")


@pytest.mark.parametrize("M,V,K", [(128, 128, 128), (256, 384, 1024), (384, 256, 2048)])
def test_lmhead_forward_version_2(det, M, V, K):
    """The order-free contraction of arithmetic version 2 on the int8 tensor cores against its oracle, bit for bit: values
    over a wide range of exponents (so that slices are truncated), an all-zero row, subnormal inputs, a row with an
    infinity and one with a NaN."""
    import torch
    from oracle import v2
    rng = np.random.default_rng(M + V + K)
    Hh = synth.to_bf16((rng.standard_normal((M, K)) * np.exp2(rng.integers(-10, 4, (M, K)))).astype(F))
    W = synth.to_bf16((rng.standard_normal((V, K)) * 0.02 * np.exp2(rng.integers(-8, 3, (V, K)))).astype(F))
    Hh[3] = 0
    Hh[5, ::3] = 0x0001
    W[7, 11] = 0x7F80
    Hh[9, 0] = 0x7FC0
    lg = empty((M, V), F)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    det.det_lmhead_fwd_v2(dev(Hh), dev(W), M, V, K, lg, ws(det.det_lmhead_fwd_v2_ws_bytes(M, V, K)), status)
    _sync()
    assert int(status.item()) == 0
    got, want = host(lg), v2.lmhead_fwd(Hh, W)
    assert np.array_equal(np.isnan(got), np.isnan(want))
    assert np.isnan(want[9]).all() and np.isnan(want[:, 7]).all()
    ok = ~np.isnan(want)
    assert_same_bits(got[ok], want[ok], "version-2 logits")
    assert np.all(np.delete(got[3], 7).view(np.uint32) == 0)          # the all-zero row: +0 against every finite row of W


@pytest.mark.parametrize("M,V,K", [(128, 128, 128), (256, 384, 256), (384, 1152, 128)])
def test_lmhead_backward_version_2(det, M, V, K):
    """Both gradient contractions of arithmetic version 2 (column slicing with transposed output, f32 source rounded to
    bf16 first, bf16 and f32 results) against the oracle, bit for bit; gradients over a wide range of exponents, a
    subnormal one, an all-zero token, a non-finite one."""
    import torch
    from oracle import v2
    rng = np.random.default_rng(M + V + K + 1)
    Hh = synth.to_bf16((rng.standard_normal((M, K)) * np.exp2(rng.integers(-6, 4, (M, K)))).astype(F))
    W = synth.to_bf16((rng.standard_normal((V, K)) * 0.02 * np.exp2(rng.integers(-8, 3, (V, K)))).astype(F))
    dl = (rng.standard_normal((M, V)) * 1e-3 * np.exp2(rng.integers(-12, 2, (M, V)))).astype(F)
    dl[2] = 0
    dl[4, 5] = 1e-41
    dl[6, 9] = np.inf
    dH, dW = empty((M, K), np.uint16), empty((V, K), F)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    det.det_lmhead_bwd_v2(dev(dl), dev(Hh), dev(W), M, V, K, dH, dW, ws(det.det_lmhead_bwd_v2_ws_bytes(M, V, K)), status)
    _sync()
    assert int(status.item()) == 0
    wH, wW = v2.lmhead_bwd(dl, Hh, W)
    gH, gW = host(dH, np.uint16), host(dW)
    nanH, nanW = np.isnan(synth.from_bf16(wH)), np.isnan(wW)
    assert nanH[6].all() and nanW[9].all() and nanH.sum() == K and nanW.sum() == K
    assert np.array_equal(np.isnan(synth.from_bf16(gH)), nanH) and np.array_equal(np.isnan(gW), nanW)
    assert_same_bits(gH[~nanH], wH[~nanH], "version-2 dH")
    assert_same_bits(gW[~nanW], wW[~nanW], "version-2 dW")


@pytest.mark.parametrize("B,H,S", [(1, 1, 128), (1, 2, 384), (2, 3, 640), (1, 1, 2176)])   # 2176 > 2048: several leaves per warp
def test_attention_forward_version_2(det, B, H, S):
    """Causal attention in arithmetic version 2 (logits and P.V as order-free contractions on the int8 tensor cores, the
    softmax in binary32) against its oracle, bit for bit: output and logsumexp; operands over a range of exponents so that
    slices are truncated, a zero query row, a zero value column, subnormal inputs."""
    import torch
    from oracle import v2
    rng = np.random.default_rng(B * 1000 + H * 100 + S)
    x = rng.standard_normal((B * S, 3 * H * 128)) * np.exp2(rng.integers(-5, 2, (B * S, 3 * H * 128)))
    x[:, :H * 128] *= 1.5                                       # sharper softmax rows
    qkv = synth.to_bf16(x.astype(F))
    qkv[5, :128] = 0                                            # a zero query row: uniform weights
    qkv[:, 2 * H * 128 + 7] = 0                                 # a zero value column
    qkv[9, H * 128:H * 128 + 128:5] = 0x0001                    # subnormal keys (count as zero)
    ld = 3 * H * 128
    d_qkv = dev(qkv)
    flat = d_qkv.view(-1)
    out, lse = empty((B * S, H * 128), np.uint16), empty((B, H, S), F)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    det.det_attn_fwd_v2(flat, flat[H * 128:], flat[2 * H * 128:], ld, B, H, S, out, H * 128, lse,
                        ws(det.det_attn_fwd_v2_ws_bytes(B, H, S)), status)
    _sync()
    assert int(status.item()) == 0
    w_out, w_lse = v2.attn_fwd(qkv, B, H, S)
    assert_same_bits(host(lse), w_lse, "version-2 lse")
    assert_same_bits(host(out, np.uint16), w_out, "version-2 attention output")


def test_embedding(det):
    V, D, T = 1000, 512, 700
    E = synth.normal_bf16((V, D), 0.02, seed=7, tid=1)
    tok = synth.randint(T, 50, seed=7, tid=2)          # many duplicates
    tok[::7] = synth.randint((T + 6) // 7, V, seed=7, tid=3)
    y = empty((T, D), np.uint16)
    det.det_embed_fwd(dev(tok), T, dev(E), V, D, y)
    dy = synth.normal_bf16((T, D), 1.0, seed=7, tid=4)
    dE = empty((V, D), F)
    det.det_embed_bwd(dev(tok), T, dev(dy), V, D, dE)
    _sync()
    assert_same_bits(host(y, np.uint16), oracle.embed_fwd(tok, E), "embed")
    assert_same_bits(host(dE), oracle.embed_bwd(tok, dy, V), "embed bwd")


# ------------------------------------------------------------------ gradient accumulation, AdamW, hash
@pytest.mark.parametrize("mesh", [(8, 1, 1), (2, 2, 2), (1, 8, 1), (1, 1, 8), (1, 1, 7), (2, 1, 3), (1, 3, 2)])
def test_grad_accum(det, mesh):
    n = 40000
    accum, shard, rep = mesh
    total = accum * shard * rep
    gs = [synth.normal_f32(n, 1e-3, seed=8, tid=i) for i in range(total)]
    nb = det.det_grad_accum_nbufs(rep)
    bufs = empty((nb * n,), F)
    st = det.det_accum()
    det.det_grad_accum_init(st, accum, shard, rep, n, bufs)
    oa = oracle.Accum(accum, shard, rep, n)
    out = empty((n,), F)
    with pytest.raises(det.DetError):
        det.det_grad_accum_result(st, out)             # too few pushes
    for g in gs:
        det.det_grad_accum_push(st, dev(g))
        oa.push(g)
    det.det_grad_accum_result(st, out)
    _sync()
    assert_same_bits(host(out), oa.result(), "accum %s" % (mesh,))
    with pytest.raises(det.DetError):
        det.det_grad_accum_push(st, dev(gs[0]))        # too many pushes


@pytest.mark.parametrize("bf,n", [(True, 100003), (False, 96), (True, 4096)])
def test_adamw(det, bf, n):
    p = synth.normal_f32(n, 0.02, seed=9, tid=1)
    if bf:
        p = synth.to_bf16(p)
    m = np.zeros(n, F)
    v = np.zeros(n, F)
    dp, dm, dv = dev(p), dev(m), dev(v)
    for t in (1, 2, 3):
        g = synth.normal_f32(n, 1e-3, seed=9, tid=10 + t)
        wd = 0.1 if bf else 0.0
        desc = det.det_adamw_desc(3e-4, 0.9, 0.95, 1e-8, wd, t)
        det.det_adamw_step(desc, int(bf), dp, dev(g), dm, dv, n)
        _sync()
        p, m, v = oracle.adamw(p, g, m, v, 3e-4, 0.9, 0.95, 1e-8, wd, t)
        assert_same_bits(host(dp, p.dtype), p, "p t=%d" % t)
        assert_same_bits(host(dm), m, "m")
        assert_same_bits(host(dv), v, "v")


@pytest.mark.parametrize("n", [16, 4096, 4096 + 16, 3 * 65536 + 1000, 128 * 4096, 128 * 4096 + 16, 5000000,
                               128 * 128 * 4096 + 4096 + 48])
def test_tensor_hash(det, n):
    b = np.random.default_rng(n).integers(0, 256, n).astype(np.uint8)
    got = det.det_tensor_hash(dev(b), n, ws(det.det_tensor_hash_ws_bytes(n)))
    assert got == oracle.tensor_hash(b)


# ------------------------------------------------------------------ int8 GEMM and the LSQ linear layer
@pytest.mark.parametrize("I,J,K,one_cta", [(128, 128, 128, 0), (256, 512, 512, 0), (384, 256, 1024, 0), (128, 384, 2048, 0),
                                           (512, 768, 640, 0), (1024, 2048, 1152, 0), (256, 256, 128, 0), (256, 512, 512, 1),
                                           (1024, 2048, 1152, 1)])
def test_igemm_exact(det, I, J, K, one_cta):
    import torch
    rng = np.random.default_rng(I + J + K)
    A = rng.integers(-128, 128, (I, K)).astype(np.int8)
    B = rng.integers(-128, 128, (J, K)).astype(np.int8)
    Cd = empty((I, J), np.int32)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    det.det_test_igemm_tn(dev(A), dev(B), I, J, K, Cd, one_cta, status)   # one_cta: the one-CTA kernel where CTA pairs would apply
    _sync()
    assert int(status.item()) == 0
    want = A.astype(np.int32) @ B.astype(np.int32).T       # brute force, exact
    assert_same_bits(host(Cd), want, "igemm")


def _linear_case(M, N, K, seed):
    X = synth.normal_bf16((M, K), 1.0, seed=seed, tid=1)
    X.reshape(-1)[:7] = synth.to_bf16(np.array([40, -40, 30, -35, 50, 11.3, -11.3], F))
    W = synth.normal_bf16((N, K), 0.02, seed=seed, tid=2)
    dY = synth.normal_bf16((M, N), 0.01, seed=seed, tid=3)
    return X, W, dY


@pytest.mark.parametrize("M,N,K,per_tensor", [(256, 512, 512, False), (256, 512, 512, True), (384, 128, 1024, False),
                                              (128, 640, 256, False)])
def test_lsq_scales_quant_forward(det, M, N, K, per_tensor):
    import torch
    X, W, _ = _linear_case(M, N, K, 11)
    dX_, dW_ = dev(X), dev(W)
    s_w, s_x = empty((N,), F), empty((1,), F)
    det.det_lsq_weight_scale(dW_, N, K, int(per_tensor), s_w, ws(det.det_lsq_weight_scale_ws_bytes(N, K)))
    det.det_lsq_act_scale_init(dX_, M * K, s_x, ws(det.det_lsq_act_scale_init_ws_bytes(M * K)))
    _sync()
    osw = oracle.lsq_weight_scale(W, per_tensor)
    osx = oracle.lsq_act_scale_init(X)
    assert_same_bits(host(s_w), osw, "s_w")
    assert_same_bits(host(s_x), osx, "s_x")
    qW, qWt, s_u = empty((N, K), np.int8), empty((K, N), np.int8), empty((1,), F)
    det.det_lsq_quantize_weight(dW_, s_w, N, K, 128, qW, qWt, s_u, ws(det.det_lsq_quantize_weight_ws_bytes(N, K)))
    Y, qX = empty((M, N), np.uint16), empty((M, K), np.int8)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    det.det_linear_fwd(dX_, qW, s_x, s_w, M, N, K, Y, qX, status)
    _sync()
    assert int(status.item()) == 0
    oY, oqX, oqW = oracle.linear_fwd(X, W, osx, osw)
    assert_same_bits(host(qW), oqW, "qW")
    assert_same_bits(host(qX), oqX, "qX")
    assert_same_bits(host(Y, np.uint16), oY, "Y")


@pytest.mark.parametrize("M,N,K,hb", [(256, 512, 512, 128), (256, 512, 512, 0), (384, 128, 256, 128), (128, 256, 640, 128),
                                       (384, 512, 512, 128), (512, 256, 768, 128), (128, 384, 256, 128)])
def test_linear_backward(det, M, N, K, hb):
    """Shapes whose output dimensions are multiples of 256 run on CTA pairs, the others on the one-CTA kernel with 128- or
    256-wide tiles: (384, 512, 512) takes the one-CTA kernel with 256-wide tiles for the input gradient and CTA pairs for the
    weight gradient."""
    import torch
    X, W, dY = _linear_case(M, N, K, 12)
    osw = oracle.lsq_weight_scale(W)
    osx = oracle.lsq_act_scale_init(X)
    odX, odW, ods, dbg = oracle.linear_bwd(dY, X, W, osx, osw, hb=hb, debug=True)
    dX_, dW_, dY_ = dev(X), dev(W), dev(dY)
    s_w, s_x = dev(osw), dev(osx)
    qW, qWt, s_u = empty((N, K), np.int8), empty((K, N), np.int8), empty((1,), F)
    det.det_lsq_quantize_weight(dW_, s_w, N, K, hb, qW, qWt, s_u, ws(det.det_lsq_quantize_weight_ws_bytes(N, K)))
    Y, qX = empty((M, N), np.uint16), empty((M, K), np.int8)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    det.det_linear_fwd(dX_, qW, s_x, s_w, M, N, K, Y, qX, status)
    gX, gW, gs = empty((M, K), np.uint16), empty((N, K), F), empty((1,), F)
    w = ws(det.det_linear_bwd_ws_bytes(M, N, K))
    det.det_linear_bwd(dY_, dX_, qX, dW_, qWt, s_x, s_w, s_u, M, N, K, hb, gX, gW, gs, w, status)
    _sync()
    assert int(status.item()) == 0
    assert_same_bits(host(qWt), dbg["UqT"], "UqT")
    assert_same_bits(host(s_u), dbg["scales"][1:2], "s_u")
    assert_same_bits(host(gX, np.uint16), odX, "dX")
    assert_same_bits(host(gW), odW, "dW")
    assert_same_bits(host(gs), ods, "ds_x")


def test_linear_backward_per_tensor_weight_step(det):
    """The single-linear configuration (256 tokens, 512 -> 512) with ONE weight step for the whole tensor: the backward
    folds that step into dY and uses it in the weight mask exactly as it does a per-channel vector."""
    import torch
    M, N, K = 256, 512, 512
    X, W, dY = _linear_case(M, N, K, 0)
    osw = oracle.lsq_weight_scale(W, True)
    assert np.all(osw == osw[0])
    osx = oracle.lsq_act_scale_init(X)
    for hb in (128, 0):
        odX, odW, ods, dbg = oracle.linear_bwd(dY, X, W, osx, osw, hb=hb, debug=True)
        dX_, dW_, dY_ = dev(X), dev(W), dev(dY)
        s_w, s_x = empty((N,), F), dev(osx)
        det.det_lsq_weight_scale(dW_, N, K, 1, s_w, ws(det.det_lsq_weight_scale_ws_bytes(N, K)))
        qW, qWt, s_u = empty((N, K), np.int8), empty((K, N), np.int8), empty((1,), F)
        det.det_lsq_quantize_weight(dW_, s_w, N, K, hb, qW, qWt, s_u, ws(det.det_lsq_quantize_weight_ws_bytes(N, K)))
        Y, qX = empty((M, N), np.uint16), empty((M, K), np.int8)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        det.det_linear_fwd(dX_, qW, s_x, s_w, M, N, K, Y, qX, status)
        gX, gW, gs = empty((M, K), np.uint16), empty((N, K), F), empty((1,), F)
        det.det_linear_bwd(dY_, dX_, qX, dW_, qWt, s_x, s_w, s_u, M, N, K, hb, gX, gW, gs,
                           ws(det.det_linear_bwd_ws_bytes(M, N, K)), status)
        _sync()
        assert int(status.item()) == 0
        assert_same_bits(host(s_w), osw, "per-tensor s_w")
        oY, _, _ = oracle.linear_fwd(X, W, osx, osw)
        assert_same_bits(host(Y, np.uint16), oY, "Y")
        assert_same_bits(host(gX, np.uint16), odX, "dX hb=%d" % hb)
        assert_same_bits(host(gW), odW, "dW hb=%d" % hb)
        assert_same_bits(host(gs), ods, "ds_x hb=%d" % hb)


@pytest.mark.parametrize("case", ["zero_grad", "zero_weight", "zero_input", "heavy_tail", "saturated_input", "inf_grad",
                                  "nan_grad"])
def test_linear_backward_degenerate(det, case):
    """Degenerate operands of the LSQ linear: all-zero tensors (absmax 0 -> scale 0, codes 0), a gradient with a few
    huge entries (everything else quantises to 0 without the rotation's spreading), activations far outside the
    quantiser's range (straight-through mask zeroes their gradient)."""
    import torch
    M, N, K = 256, 256, 256
    X, W, dY = _linear_case(M, N, K, 13)
    if case == "zero_grad":
        dY[:] = 0
    if case == "zero_weight":
        W[:] = 0
    if case == "zero_input":
        X[:] = 0
    if case == "heavy_tail":
        dY[::37, ::41] = synth.to_bf16(np.array([3.0e4], F))[0]
    if case == "inf_grad":        # an infinite gradient: both absmax values are infinite, every code is 0 or the clamp of a NaN
        dY[5, 9] = 0x7F80
    if case == "nan_grad":        # a NaN does not enter the absmax; its 128-block rotates to NaNs, which quantise like the oracle's
        dY[100, 200] = 0x7FC0
    osw = oracle.lsq_weight_scale(W)
    osx = oracle.lsq_act_scale_init(X)
    if case == "saturated_input":
        X[::3, ::5] = synth.to_bf16(np.array([1.0e3], F))[0]      # far beyond 127 steps, after the step was fixed
    odX, odW, ods, dbg = oracle.linear_bwd(dY, X, W, osx, osw, hb=128, debug=True)
    dX_, dW_, dY_ = dev(X), dev(W), dev(dY)
    s_w, s_x = dev(osw), dev(osx)
    qW, qWt, s_u = empty((N, K), np.int8), empty((K, N), np.int8), empty((1,), F)
    det.det_lsq_quantize_weight(dW_, s_w, N, K, 128, qW, qWt, s_u, ws(det.det_lsq_quantize_weight_ws_bytes(N, K)))
    Y, qX = empty((M, N), np.uint16), empty((M, K), np.int8)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    det.det_linear_fwd(dX_, qW, s_x, s_w, M, N, K, Y, qX, status)
    oY, _, _ = oracle.linear_fwd(X, W, osx, osw)
    gX, gW, gs = empty((M, K), np.uint16), empty((N, K), F), empty((1,), F)
    det.det_linear_bwd(dY_, dX_, qX, dW_, qWt, s_x, s_w, s_u, M, N, K, 128, gX, gW, gs, ws(det.det_linear_bwd_ws_bytes(M, N, K)),
                       status)
    _sync()
    assert int(status.item()) == 0
    assert_same_bits(host(Y, np.uint16), oY, "Y")
    if case == "inf_grad":
        # infinite steps turn almost every gradient into a NaN; NaNs are compared as NaNs (their payload is not part of
        # the arithmetic's definition), everything else bit for bit
        for got, want, name in ((synth.from_bf16(host(gX, np.uint16)), synth.from_bf16(odX), "dX"), (host(gW), odW, "dW"),
                                (host(gs), ods, "ds_x")):
            gn, wn = np.isnan(got), np.isnan(want)
            assert np.array_equal(gn, wn), name + ": NaN positions differ"
            assert np.array_equal(got[~gn].view(np.uint32), want[~wn].view(np.uint32)), name
        assert np.isnan(odW).mean() > 0.9
        return
    assert_same_bits(host(gX, np.uint16), odX, "dX")
    assert_same_bits(host(gW), odW, "dW")
    assert_same_bits(host(gs), ods, "ds_x")
    if case == "zero_grad":
        assert not host(gX, np.uint16).any() and not host(gW).view(np.uint32).any()


# ------------------------------------------------------------------ LM head and attention (ordered FP32)
@pytest.mark.parametrize("M,V,K", [(128, 256, 256), (72, 1008, 64), (256, 50304 // 8, 128)])
def test_lmhead(det, M, V, K):
    Hh = synth.normal_bf16((M, K), 1.0, seed=13, tid=1)
    W = synth.normal_bf16((V, K), 0.02, seed=13, tid=2)
    lg = empty((M, V), F)
    det.det_lmhead_fwd(dev(Hh), dev(W), M, V, K, lg)
    _sync()
    assert_same_bits(host(lg), oracle.lmhead_fwd(Hh, W), "logits")
    dl = synth.normal_f32((M, V), 1e-3, seed=13, tid=3)
    dH, dW = empty((M, K), np.uint16), empty((V, K), F)
    h1 = M // 2 // 8 * 8
    det.det_lmhead_bwd(dev(dl[:h1]), dev(Hh[:h1]), dev(W), h1, V, K, dH[:h1], dW, 1)
    det.det_lmhead_bwd(dev(dl[h1:]), dev(Hh[h1:]), dev(W), M - h1, V, K, dH[h1:], dW, 0)
    _sync()
    oH, oW = oracle.lmhead_bwd(dl, Hh, W)
    assert_same_bits(host(dH, np.uint16), oH, "dH")
    assert_same_bits(host(dW), oW, "dW")


@pytest.mark.parametrize("B,H,S", [(1, 2, 64), (2, 2, 192), (1, 1, 320)])
def test_attention(det, B, H, S):
    HD = H * 128
    qkv = synth.normal_bf16((B * S, 3 * HD), 1.0, seed=14, tid=1)
    dout = synth.normal_bf16((B * S, HD), 0.1, seed=14, tid=2)
    dqkv_in = dev(qkv)
    base = dqkv_in.data_ptr()
    out, lse = empty((B * S, HD), np.uint16), empty((B, H, S), F)
    det.det_attn_fwd(base, base + 2 * HD, base + 4 * HD, 3 * HD, B, H, S, out, HD, lse)
    _sync()
    oout, olse = oracle.attn_fwd(qkv, B, H, S)
    assert_same_bits(host(lse), olse, "lse")
    assert_same_bits(host(out, np.uint16), oout, "out")
    dqkv = empty((B * S, 3 * HD), np.uint16)
    db = dqkv.data_ptr()
    det.det_attn_bwd(dev(dout), base, base + 2 * HD, base + 4 * HD, out, lse, 3 * HD, HD, B, H, S, db, db + 2 * HD,
                     db + 4 * HD, 3 * HD, ws(det.det_attn_bwd_ws_bytes(B, H, S)))
    _sync()
    want = oracle.attn_bwd(dout, qkv, oout, olse, B, H, S)
    got = host(dqkv, np.uint16)
    for name, c in (("dq", 0), ("dk", 1), ("dv", 2)):
        assert_same_bits(got[:, c * HD:(c + 1) * HD], want[:, c * HD:(c + 1) * HD], name)


@pytest.mark.parametrize("B,H,Hkv,S,W", [(1, 4, 2, 192, 0), (2, 4, 1, 128, 0), (1, 2, 2, 448, 128), (1, 1, 1, 640, 256),
                                         (1, 4, 2, 384, 128), (1, 2, 2, 256, 512)])
def test_attention_grouped_and_windowed(det, B, H, Hkv, S, W):
    """Grouped-query heads (Hkv < H) and sliding windows: forward and all three gradients bit for bit."""
    HD, KD = H * 128, Hkv * 128
    ld = HD + 2 * KD
    qkv = synth.normal_bf16((B * S, ld), 1.0, seed=15, tid=1)
    dout = synth.normal_bf16((B * S, HD), 0.1, seed=15, tid=2)
    dqkv_in = dev(qkv)
    base = dqkv_in.data_ptr()
    out, lse = empty((B * S, HD), np.uint16), empty((B, H, S), F)
    det.det_attn_fwd(base, base + 2 * HD, base + 2 * (HD + KD), ld, B, H, S, out, HD, lse, Hkv=Hkv, window=W)
    _sync()
    oout, olse = oracle.attn_fwd(qkv, B, H, S, Hkv=Hkv, window=W)
    assert_same_bits(host(lse), olse, "lse")
    assert_same_bits(host(out, np.uint16), oout, "out")
    dqkv = empty((B * S, ld), np.uint16)
    db = dqkv.data_ptr()
    det.det_attn_bwd(dev(dout), base, base + 2 * HD, base + 2 * (HD + KD), out, lse, ld, HD, B, H, S, db, db + 2 * HD,
                     db + 2 * (HD + KD), ld, ws(det.det_attn_bwd_ws_bytes(B, H, S, Hkv)), Hkv=Hkv, window=W)
    _sync()
    want = oracle.attn_bwd(dout, qkv, oout, olse, B, H, S, Hkv=Hkv, window=W)
    got = host(dqkv, np.uint16)
    for name, lo, hi in (("dq", 0, HD), ("dk", HD, HD + KD), ("dv", HD + KD, ld)):
        assert_same_bits(got[:, lo:hi], want[:, lo:hi], name)


@pytest.mark.parametrize("B,H,Hkv,S,W,scale", [(1, 2, 2, 64, 0, 0.1), (2, 2, 2, 192, 0, 0.1), (1, 4, 2, 448, 0, 1e-6),
                                               (1, 2, 1, 640, 256, 0.1), (1, 1, 1, 384, 128, 1e-9),
                                               (1, 1, 1, 320, 0, 3e4)])
def test_attention_backward_fixed_point_query_gradient(det, B, H, Hkv, S, W, scale):
    """dQ accumulated over the key blocks in 64-bit fixed point: all three gradients bit for bit, from gradients so small
    that most contributions round to a few units of 2^-48 up to ones that saturate the accumulator."""
    HD, KD = H * 128, Hkv * 128
    ld = HD + 2 * KD
    qkv = synth.normal_bf16((B * S, ld), 1.0, seed=16, tid=1)
    dout = synth.normal_bf16((B * S, HD), scale, seed=16, tid=2)
    dqkv_in = dev(qkv)
    base = dqkv_in.data_ptr()
    out, lse = empty((B * S, HD), np.uint16), empty((B, H, S), F)
    det.det_attn_fwd(base, base + 2 * HD, base + 2 * (HD + KD), ld, B, H, S, out, HD, lse, Hkv=Hkv, window=W)
    _sync()
    oout, olse = oracle.attn_fwd(qkv, B, H, S, Hkv=Hkv, window=W)
    dqkv = empty((B * S, ld), np.uint16)
    db = dqkv.data_ptr()
    w = ws(det.det_attn_bwd_fixq_ws_bytes(B, H, S, Hkv))
    w.fill_(255)                                       # stale scratch must not leak into the accumulators
    det.det_attn_bwd_fixq(dev(dout), base, base + 2 * HD, base + 2 * (HD + KD), out, lse, ld, HD, B, H, S, db, db + 2 * HD,
                          db + 2 * (HD + KD), ld, w, Hkv=Hkv, window=W)
    _sync()
    want = oracle.attn_bwd(dout, qkv, oout, olse, B, H, S, Hkv=Hkv, window=W, fixq=True)
    got = host(dqkv, np.uint16)
    for name, lo, hi in (("dq", 0, HD), ("dk", HD, HD + KD), ("dv", HD + KD, ld)):
        assert_same_bits(got[:, lo:hi], want[:, lo:hi], name)


@pytest.mark.parametrize("B,H,Hkv,S,W", [(1, 1, 1, 128, 0), (1, 2, 2, 320, 0), (2, 4, 2, 256, 0), (1, 2, 1, 512, 128)])
def test_attention_forward_int8_pv(det, B, H, Hkv, S, W):
    """P.V of every block on the int8 tensor cores: output and logsumexp bit for bit against the oracle's definition."""
    import torch
    HD, KD = H * 128, Hkv * 128
    ld = HD + 2 * KD
    qkv = synth.normal_bf16((B * S, ld), 1.0, seed=16, tid=1)
    qkv[5, HD + KD:] = 0                                         # a zero value row
    dq = dev(qkv)
    base = dq.data_ptr()
    out, lse = empty((B * S, HD), np.uint16), empty((B, H, S), F)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    det.det_attn_fwd_int8pv(base, base + 2 * HD, base + 2 * (HD + KD), ld, B, H, S, out, HD, lse, status, Hkv=Hkv, window=W)
    _sync()
    assert int(status.item()) == 0
    oout, olse = oracle.attn_fwd(qkv, B, H, S, Hkv=Hkv, window=W, int8_pv=True)
    assert_same_bits(host(lse), olse, "lse")
    assert_same_bits(host(out, np.uint16), oout, "out")


# ------------------------------------------------------------------ slabs whose products can underflow
def _sprinkle_tiny(a, seed, frac=0.002):
    """Overwrite a fraction of a bf16 tensor with magnitudes around 2^-64 .. 2^-62 (random signs)."""
    rng = np.random.default_rng(seed)
    flat = a.reshape(-1)
    idx = rng.choice(flat.size, max(4, int(flat.size * frac)), replace=False)
    vals = (2.0 ** rng.integers(-66, -61, idx.size)) * rng.choice([-1.0, 1.0, 1.5, -1.25], idx.size)
    flat[idx] = synth.to_bf16(vals.astype(F))
    return a


def test_lmhead_subnormal_products(det):
    # 1.5*2^-126 + 2^-127: the second product is subnormal, so multiply-flush-add keeps 1.5*2^-126 while a fused
    # multiply-add would give 2^-125; the kernel must notice the tiny factors and take the unfused sequence
    M, V, K = 128, 256, 64
    Hh = synth.normal_bf16((M, K), 1.0, seed=21, tid=1)
    W = synth.normal_bf16((V, K), 0.02, seed=21, tid=2)
    Hh[0] = 0
    W[0] = 0
    Hh[0, :2] = synth.to_bf16(np.array([2.0 ** -63, 2.0 ** -64], F))
    W[0, :2] = synth.to_bf16(np.array([1.5 * 2.0 ** -63, 2.0 ** -63], F))
    _sprinkle_tiny(Hh[1:], 1)
    _sprinkle_tiny(W[1:], 2)
    lg = empty((M, V), F)
    det.det_lmhead_fwd(dev(Hh), dev(W), M, V, K, lg)
    _sync()
    want = oracle.lmhead_fwd(Hh, W)
    assert want[0, 0] == F(1.5 * 2.0 ** -126)
    assert_same_bits(host(lg), want, "logits with subnormal products")
    dl = synth.normal_f32((M, V), 1e-3, seed=21, tid=3)
    dl.reshape(-1)[::97] = F(2.0 ** -65)
    dH, dW = empty((M, K), np.uint16), empty((V, K), F)
    det.det_lmhead_bwd(dev(dl), dev(Hh), dev(W), M, V, K, dH, dW, 1)
    _sync()
    oH, oW = oracle.lmhead_bwd(dl, Hh, W)
    assert_same_bits(host(dH, np.uint16), oH, "dH")
    assert_same_bits(host(dW), oW, "dW")


def test_attention_subnormal_products(det):
    B, H, S = 1, 2, 256
    HD = H * 128
    qkv = _sprinkle_tiny(synth.normal_bf16((B * S, 3 * HD), 1.0, seed=22, tid=1), 3, 0.01)
    qkv[5:9, :] = synth.to_bf16(np.full((4, 3 * HD), 2.0 ** -64, F))       # whole rows of tiny q, k, v
    dout = _sprinkle_tiny(synth.normal_bf16((B * S, HD), 0.1, seed=22, tid=2), 4, 0.01)
    dqkv_in = dev(qkv)
    base = dqkv_in.data_ptr()
    out, lse = empty((B * S, HD), np.uint16), empty((B, H, S), F)
    det.det_attn_fwd(base, base + 2 * HD, base + 4 * HD, 3 * HD, B, H, S, out, HD, lse)
    _sync()
    oout, olse = oracle.attn_fwd(qkv, B, H, S)
    assert_same_bits(host(lse), olse, "lse")
    assert_same_bits(host(out, np.uint16), oout, "out")
    dqkv = empty((B * S, 3 * HD), np.uint16)
    db = dqkv.data_ptr()
    det.det_attn_bwd(dev(dout), base, base + 2 * HD, base + 4 * HD, out, lse, 3 * HD, HD, B, H, S, db, db + 2 * HD,
                     db + 4 * HD, 3 * HD, ws(det.det_attn_bwd_ws_bytes(B, H, S)))
    _sync()
    assert_same_bits(host(dqkv, np.uint16), oracle.attn_bwd(dout, qkv, oout, olse, B, H, S), "dqkv")


def test_bounded_wait_times_out_and_context_survives(det):
    """A wait on a barrier that nothing completes gives up after its limit, reports DET_DEV_TIMEOUT through the status
    word and returns; the next launches run normally."""
    import torch
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    det.det_test_wait_timeout(status, 2000000)              # about a millisecond
    _sync()
    assert int(status.item()) == det.DET_DEV_TIMEOUT
    x = np.arange(1000, dtype=F)
    out = empty((1,), F)
    det.det_sum(dev(x), 1000, 0, out, ws(det.det_sum_ws_bytes(1000)))
    _sync()
    assert_same_bits(host(out), np.array([oracle.det_sum(x)], F), "sum after a timed-out wait")


def test_extreme_inputs(det):
    """Saturated softmax, zero rows and non-finite gradients: the degenerate corners of the floating-point ops."""
    import torch
    # attention with logits so large that most weights underflow to exactly 0 (flush-to-zero results of det_exp)
    B, H, S = 1, 1, 256
    HD = 128
    qkv = synth.normal_bf16((B * S, 3 * HD), 1.0, seed=17, tid=1)
    qkv[:, :HD] = synth.to_bf16(synth.from_bf16(qkv[:, :HD]) * F(40.0))          # logits of order +-400
    qkv[7, :HD] = 0                                                              # one all-zero query: uniform weights
    dout = synth.normal_bf16((B * S, HD), 0.1, seed=17, tid=2)
    dq = dev(qkv)
    base = dq.data_ptr()
    out, lse = empty((B * S, HD), np.uint16), empty((B, H, S), F)
    det.det_attn_fwd(base, base + 2 * HD, base + 4 * HD, 3 * HD, B, H, S, out, HD, lse)
    dqkv = empty((B * S, 3 * HD), np.uint16)
    db = dqkv.data_ptr()
    det.det_attn_bwd(dev(dout), base, base + 2 * HD, base + 4 * HD, out, lse, 3 * HD, HD, B, H, S, db, db + 2 * HD, db + 4 * HD,
                     3 * HD, ws(det.det_attn_bwd_ws_bytes(B, H, S)))
    _sync()
    oout, olse = oracle.attn_fwd(qkv, B, H, S)
    assert_same_bits(host(out, np.uint16), oout, "saturated attention out")
    assert_same_bits(host(lse), olse, "saturated attention lse")
    assert_same_bits(host(dqkv, np.uint16), oracle.attn_bwd(dout, qkv, oout, olse, B, H, S), "saturated attention grads")
    # RMSNorm of an all-zero row: rstd = 1/sqrt(eps), outputs 0
    x = synth.normal_f32((16, 256), 1.0, seed=18, tid=1)
    x[3] = 0
    y, rstd = empty((16, 256), F), empty((16,), F)
    det.det_rmsnorm_fwd(0, dev(x), None, 16, 256, 1e-6, y, rstd)
    _sync()
    oy, orstd = oracle.rmsnorm_fwd(x, None, 1e-6)
    assert_same_bits(host(y), oy, "rmsnorm zero row")
    assert_same_bits(host(rstd), orstd, "rstd zero row")
    assert not host(y)[3].any()
    # cross-entropy with a dominant logit and with huge negative logits
    z = synth.normal_f32((6, 1000), 1.0, seed=19, tid=1)
    z[0, 5] = 1.0e4
    z[1] = -3.0e4
    z[2, :] = 0.0
    tgt = np.array([5, 7, 9, 11, 13, 999], np.int32)
    loss_row, l2, lm, zm = empty((6,), F), empty((6,), F), empty((1,), F), empty((1,), F)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    det.det_xent_fwd(dev(z), dev(tgt), 6, 1000, 0.0, loss_row, l2, lm, zm, ws(det.det_xent_ws_bytes(6, 1000)), status)
    _sync()
    olr, ol2, olm, _, _ = oracle.xent_fwd(z, tgt, 0.0)
    assert_same_bits(host(loss_row), olr, "xent extreme rows")
    assert_same_bits(host(lm), olm, "xent mean")
    assert host(loss_row)[0] == 0.0                                             # dominant logit at the target
    # gradient norm: all zeros -> norm 0, coefficient 1; a NaN raises the non-finite flag
    g0 = dev(np.zeros(5000, F))
    norm, coef = empty((1,), F), empty((1,), F)
    det.det_grad_norm([g0], 1.0, norm, coef, ws(det.det_grad_norm_ws_bytes([g0])), status)
    _sync()
    on, oc = oracle.grad_norm([np.zeros(5000, F)], 1.0)
    assert_same_bits(host(norm), np.array([on], F), "zero norm")
    assert_same_bits(host(coef), np.array([oc], F), "zero-norm coefficient")
    bad = np.zeros(5000, F)
    bad[123] = np.nan
    status.zero_()
    det.det_grad_norm([dev(bad)], 1.0, norm, coef, ws(det.det_grad_norm_ws_bytes([g0])), status)
    _sync()
    assert int(status.item()) & det.DET_DEV_NONFINITE
