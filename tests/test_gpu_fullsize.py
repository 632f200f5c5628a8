"""Parity at the benchmark's full shapes (24-layer 1B block at 8192 tokens per micro-batch), in the launch configuration
the bench times: the GPU computes the whole operation, the oracle recomputes a sample of outputs that are independent of
the rest (rows, columns, heads), and those must agree bit for bit; whole-tensor quantities are checked through the
oracle's own reductions of the GPU's per-row results."""
import numpy as np
import pytest

import oracle
import synth
from gpu_util import assert_same_bits, dev, empty, host, ws

pytestmark = pytest.mark.gpu
F = np.float32
T, D, FF, V, H, S, B = 8192, 2048, 8192, 50304, 16, 2048, 4


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


def _bf16_normal(shape, std, seed):
    """Seeded N(0, std) as bf16 bit patterns (numpy generator: the counter-based one is too slow for 10^8 values)."""
    return synth.to_bf16((np.random.default_rng(seed).standard_normal(shape, dtype=np.float32) * F(std)))


# gate/up (CTA-pair tiles, short K) and down (long K) at the micro-batch's 8192 tokens, and both again at the 16384
# tokens of the 1B-shaped linear set
@pytest.mark.parametrize("T,N,K", [(8192, 2 * FF, D), (8192, D, FF), (16384, 2 * FF, D), (16384, D, FF)])
def test_linear_forward_full_shape_sampled(det, T, N, K):
    import torch
    X, W = _bf16_normal((T, K), 1.0, 1), _bf16_normal((N, K), 0.02, 2)
    dX_, dW_ = dev(X), dev(W)
    s_w, s_x = empty((N,), F), empty((1,), F)
    det.det_lsq_weight_scale(dW_, N, K, 0, s_w, ws(det.det_lsq_weight_scale_ws_bytes(N, K)))
    det.det_lsq_act_scale_init(dX_, T * K, s_x, ws(det.det_lsq_act_scale_init_ws_bytes(T * K)))
    qW, qWt, s_u = empty((N, K), np.int8), empty((K, N), np.int8), empty((1,), F)
    det.det_lsq_quantize_weight(dW_, s_w, N, K, 128, qW, qWt, s_u, ws(det.det_lsq_quantize_weight_ws_bytes(N, K)))
    Y, qX = empty((T, N), np.uint16), empty((T, K), np.int8)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    det.det_linear_fwd(dX_, qW, s_x, s_w, T, N, K, Y, qX, status)
    _sync()
    assert int(status.item()) == 0
    osx = oracle.lsq_act_scale_init(X)                              # whole-tensor reduction, cheap on the host
    assert_same_bits(host(s_x), osx, "s_x")
    rng = np.random.default_rng(3)
    rows = np.sort(rng.choice(T, 24, replace=False))
    rows[0], rows[-1] = 0, T - 1
    cols = np.sort(rng.choice(N, 96, replace=False))
    cols[0], cols[-1] = 0, N - 1
    osw = oracle.lsq_weight_scale(W[cols])                          # weight steps are per output channel
    assert_same_bits(host(s_w)[cols], osw, "s_w")
    oY, oqX, oqW = oracle.linear_fwd(X[rows], W[cols], osx, osw)
    assert_same_bits(host(qX)[rows], oqX, "qX rows")
    assert_same_bits(host(qW)[cols], oqW, "qW rows")
    assert_same_bits(host(Y, np.uint16)[np.ix_(rows, cols)], oY, "Y sample")


@pytest.mark.parametrize("T,N,K", [(8192, 2 * FF, D), (16384, 3 * D, D)])
def test_linear_backward_full_shape_sampled(det, T, N, K):
    """Gate/up projection backward at 8192 x 16384 x 2048 and the QKV projection backward at 16384 x 6144 x 2048 (the token
    count of the 1B-shaped linear set) with the Hadamard rotation: the operands' scales are maxima over whole tensors, so
    the oracle prepares them in full and evaluates the two contractions for sampled rows."""
    import torch
    X, W, dY = _bf16_normal((T, K), 1.0, 21), _bf16_normal((N, K), 0.02, 22), _bf16_normal((T, N), 0.01, 23)
    dX_, dW_, dY_ = dev(X), dev(W), dev(dY)
    s_w, s_x = empty((N,), F), empty((1,), F)
    det.det_lsq_weight_scale(dW_, N, K, 0, s_w, ws(det.det_lsq_weight_scale_ws_bytes(N, K)))
    det.det_lsq_act_scale_init(dX_, T * K, s_x, ws(det.det_lsq_act_scale_init_ws_bytes(T * K)))
    qW, qWt, s_u = empty((N, K), np.int8), empty((K, N), np.int8), empty((1,), F)
    det.det_lsq_quantize_weight(dW_, s_w, N, K, 128, qW, qWt, s_u, ws(det.det_lsq_quantize_weight_ws_bytes(N, K)))
    Y, qX = empty((T, N), np.uint16), empty((T, K), np.int8)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    det.det_linear_fwd(dX_, qW, s_x, s_w, T, N, K, Y, qX, status)
    gdX, gdW, gds = empty((T, K), np.uint16), empty((N, K), F), empty((1,), F)
    det.det_linear_bwd(dY_, dX_, qX, dW_, qWt, s_x, s_w, s_u, T, N, K, 128, gdX, gdW, gds,
                       ws(det.det_linear_bwd_ws_bytes(T, N, K)), status)
    _sync()
    assert int(status.item()) == 0
    rng = np.random.default_rng(24)
    rm = np.sort(rng.choice(T, 8, replace=False)).astype(np.int32)
    rm[0], rm[-1] = 0, T - 1
    rn = np.sort(rng.choice(N, 8, replace=False)).astype(np.int32)
    rn[0], rn[-1] = 0, N - 1
    odx, odw = oracle.linear_bwd_rows(dY, X, W, host(s_x), host(s_w), rm, rn)
    assert_same_bits(host(gdX, np.uint16)[rm], odx, "dX rows")
    assert_same_bits(gdW[rn.tolist()].cpu().numpy(), odw, "dW rows")


def test_lmhead_full_shape_sampled(det):
    Hh, W = _bf16_normal((T, D), 1.0, 4), _bf16_normal((V, D), 0.02, 5)
    logits = empty((T, V), F)
    det.det_lmhead_fwd(dev(Hh), dev(W), T, V, D, logits)
    _sync()
    rng = np.random.default_rng(6)
    rows = np.sort(rng.choice(T, 6, replace=False))
    rows[0], rows[-1] = 0, T - 1
    got = logits[rows.tolist()].cpu().numpy()
    assert_same_bits(got, oracle.lmhead_fwd(Hh[rows], W), "logit rows")
    # backward on a synthetic dlogits: dH rows need only their own dlogits row; dW rows need every token
    dl = (np.random.default_rng(7).standard_normal((T, V), dtype=np.float32) * F(1e-3))
    dH, dW = empty((T, D), np.uint16), empty((V, D), F)
    ddl = dev(dl)
    det.det_lmhead_bwd(ddl, dev(Hh), dev(W), T, V, D, dH, dW, 1)
    _sync()
    odH, _ = oracle.lmhead_bwd(dl[rows], Hh[rows], W)
    assert_same_bits(host(dH, np.uint16)[rows], odH, "dH rows")
    vs = np.sort(rng.choice(V, 12, replace=False))
    vs[0], vs[-1] = 0, V - 1
    _, odW = oracle.lmhead_bwd(np.ascontiguousarray(dl[:, vs]), Hh, W[vs])
    assert_same_bits(dW[vs.tolist()].cpu().numpy(), odW, "dW rows")


def test_lmhead_version_2_full_shape_sampled(det):
    """The order-free forward contraction (arithmetic version 2) at 8192 x 50304 x 2048: sampled rows against its oracle."""
    import torch
    from oracle import v2
    Hh, W = _bf16_normal((T, D), 1.0, 41), _bf16_normal((V, D), 0.02, 42)
    logits = empty((T, V), F)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    det.det_lmhead_fwd_v2(dev(Hh), dev(W), T, V, D, logits, ws(det.det_lmhead_fwd_v2_ws_bytes(T, V, D)), status)
    _sync()
    assert int(status.item()) == 0
    rows = np.sort(np.random.default_rng(43).choice(T, 6, replace=False))
    rows[0], rows[-1] = 0, T - 1
    assert_same_bits(logits[rows.tolist()].cpu().numpy(), v2.lmhead_fwd(Hh[rows], W), "version-2 logit rows")


def test_attention_full_shape_one_head(det):
    HD = H * 128
    qkv = _bf16_normal((B * S, 3 * HD), 1.0, 8)
    dout = _bf16_normal((B * S, HD), 0.1, 9)
    dq = dev(qkv)
    base = dq.data_ptr()
    out, lse = empty((B * S, HD), np.uint16), empty((B, H, S), F)
    det.det_attn_fwd(base, base + 2 * HD, base + 4 * HD, 3 * HD, B, H, S, out, HD, lse)
    dqkv = empty((B * S, 3 * HD), np.uint16)
    db = dqkv.data_ptr()
    det.det_attn_bwd(dev(dout), base, base + 2 * HD, base + 4 * HD, out, lse, 3 * HD, HD, B, H, S, db, db + 2 * HD,
                     db + 4 * HD, 3 * HD, ws(det.det_attn_bwd_ws_bytes(B, H, S)))
    _sync()
    gout, glse, gd = host(out, np.uint16), host(lse), host(dqkv, np.uint16)
    # every (batch, head) is independent of the others: two of them are replayed by the oracle as a batch of two
    # single-head problems
    picks = ((0, 0), (B - 1, H - 1))
    one = np.ascontiguousarray(np.concatenate(
        [np.concatenate([qkv[b * S:(b + 1) * S, c * HD + h * 128:c * HD + (h + 1) * 128] for c in range(3)], 1) for b, h in picks], 0))
    do1 = np.ascontiguousarray(np.concatenate([dout[b * S:(b + 1) * S, h * 128:(h + 1) * 128] for b, h in picks], 0))
    oo, ol = oracle.attn_fwd(one, 2, 1, S)
    od = oracle.attn_bwd(do1, one, oo, ol, 2, 1, S)
    for i, (b, h) in enumerate(picks):
        r, ro = slice(b * S, (b + 1) * S), slice(i * S, (i + 1) * S)
        assert_same_bits(gout[r, h * 128:(h + 1) * 128], oo[ro], "out head")
        assert_same_bits(glse[b, h], ol[i, 0], "lse head")
        for c, name in enumerate(("dq", "dk", "dv")):
            assert_same_bits(gd[r, c * HD + h * 128:c * HD + (h + 1) * 128], od[ro, c * 128:(c + 1) * 128], name)
    # the same backward with the query gradient accumulated over the 16 key blocks in 64-bit fixed point
    dqkv2 = empty((B * S, 3 * HD), np.uint16)
    db2 = dqkv2.data_ptr()
    det.det_attn_bwd_fixq(dev(dout), base, base + 2 * HD, base + 4 * HD, out, lse, 3 * HD, HD, B, H, S, db2, db2 + 2 * HD,
                          db2 + 4 * HD, 3 * HD, ws(det.det_attn_bwd_fixq_ws_bytes(B, H, S)))
    _sync()
    gd2 = host(dqkv2, np.uint16)
    assert_same_bits(gd2[:, HD:], gd[:, HD:], "dk, dv of the fixed-point variant")
    od2 = oracle.attn_bwd(do1, one, oo, ol, 2, 1, S, fixq=True)
    for i, (b, h) in enumerate(picks):
        r, ro = slice(b * S, (b + 1) * S), slice(i * S, (i + 1) * S)
        assert_same_bits(gd2[r, h * 128:(h + 1) * 128], od2[ro, :128], "dq fixed point")


def test_norm_and_loss_full_shape(det):
    import torch
    x, g = _bf16_normal((T, D), 1.0, 10), synth.to_bf16(1 + np.random.default_rng(11).standard_normal(D).astype(F) * F(0.02))
    y, rstd = empty((T, D), np.uint16), empty((T,), F)
    det.det_rmsnorm_fwd(1, dev(x), dev(g), T, D, 1e-6, y, rstd)
    _sync()
    oy, orstd = oracle.rmsnorm_fwd(x, g, 1e-6, bf=True)
    assert_same_bits(host(rstd), orstd, "rstd")
    assert_same_bits(host(y, np.uint16), oy, "y")
    dy = _bf16_normal((T, D), 1.0, 12)
    dx, dgam = empty((T, D), np.uint16), empty((D,), F)
    det.det_rmsnorm_bwd(1, dev(dy), dev(x), dev(g), rstd, T, D, dx, dgam, ws(det.det_rmsnorm_bwd_ws_bytes(T, D)))
    _sync()
    odx, odg = oracle.rmsnorm_bwd(dy, x, g, orstd, bf=True)
    assert_same_bits(host(dx, np.uint16), odx, "dx")
    assert_same_bits(host(dgam), odg, "dgamma (tree over 8192 rows)")
    # cross-entropy over [8192, 50304]: sampled rows bit for bit; the means through the oracle's tree over the GPU's rows
    z = np.random.default_rng(13).standard_normal((T, V), dtype=np.float32) * F(2.0)
    tgt = np.random.default_rng(14).integers(0, V, T).astype(np.int32)
    dz = dev(z)
    loss_row, lse, lm, zm = empty((T,), F), empty((T,), F), empty((1,), F), empty((1,), F)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    det.det_xent_fwd(dz, dev(tgt), T, V, 1e-4, loss_row, lse, lm, zm, ws(det.det_xent_ws_bytes(T, V)), status)
    _sync()
    rows = np.sort(np.random.default_rng(15).choice(T, 48, replace=False))
    rows[0], rows[-1] = 0, T - 1
    olr, olse, _, _, _ = oracle.xent_fwd(z[rows], tgt[rows], 1e-4)
    assert_same_bits(host(loss_row)[rows], olr, "loss rows")
    assert_same_bits(host(lse)[rows], olse, "lse rows")
    glr, glse = host(loss_row), host(lse)
    inv = np.array([1.0 / T], F)
    zmean = oracle.prim("mul", np.array([oracle.det_sum(oracle.prim("mul", glse, glse))], F), inv)
    assert_same_bits(host(zm), zmean, "z mean")
    ce = oracle.prim("mul", np.array([oracle.det_sum(glr)], F), inv)
    assert_same_bits(host(lm), oracle.prim("add", ce, oracle.prim("mul", np.array([1e-4], F), zmean)), "loss mean")
    det.det_xent_bwd(dz, dev(tgt), lse, T, V, 1e-4, 1.0 / T)
    _sync()
    odz = oracle.xent_bwd(z[rows], tgt[rows], glse[rows], 1e-4, F(1.0 / T))
    assert_same_bits(dz[rows.tolist()].cpu().numpy(), odz, "dlogits rows")


def test_grad_norm_1p2e9_elements(det):
    """Global gradient norm over 1.2e9 f32 ~ N(0, 1e-3) (the reductions configuration), split into three tensors of ragged
    lengths so that the per-tensor trees (four levels of 16384-element chunks for the largest) and the tree over the
    per-tensor sums both run: norm and clip coefficient bit for bit against the oracle's trees."""
    import torch
    n = 1_200_000_000
    g = np.random.default_rng(31).standard_normal(n, dtype=np.float32)
    g *= F(1e-3)
    cuts = [0, 700_000_000, 1_000_000_128, n]      # lengths 700000000, 300000128, 199999872; every start 16-byte aligned
    dg = dev(g)
    views = [dg[cuts[i]:cuts[i + 1]] for i in range(3)]
    norm, coef = empty((1,), F), empty((1,), F)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    det.det_grad_norm(views, 1.0, norm, coef, ws(det.det_grad_norm_ws_bytes(views)), status)
    _sync()
    onorm, ocoef = oracle.grad_norm([g[cuts[i]:cuts[i + 1]] for i in range(3)], 1.0)
    assert int(status.item()) == 0
    assert_same_bits(host(norm), np.array([onorm], F), "norm")
    assert_same_bits(host(coef), np.array([ocoef], F), "clip coefficient")
    assert abs(float(onorm) - 34.64) < 0.05                        # sqrt(1.2e9) * 1e-3
    # the whole vector as one tensor: one tree of five levels
    out = empty((1,), F)
    det.det_sum(dg, n, 1, out, ws(det.det_sum_ws_bytes(n)))
    _sync()
    assert_same_bits(host(out), np.array([oracle.sumsq(g)], F), "sum of squares, 1.2e9 elements")


def test_reduction_and_optimizer_at_scale(det):
    """Order-fixed reductions and the element-wise update on 2^27 + 1000 elements (ragged tail, many tree levels)."""
    import torch
    n = (1 << 27) + 1000
    g = np.random.default_rng(16).standard_normal(n, dtype=np.float32) * F(1e-3)
    dg = dev(g)
    out = empty((1,), F)
    det.det_sum(dg, n, 1, out, ws(det.det_sum_ws_bytes(n)))
    _sync()
    assert_same_bits(host(out), np.array([oracle.sumsq(g)], F), "sum of squares")
    # mesh (2,2,2): eight pushes of scaled copies, then the result
    bufs = torch.empty(det.det_grad_accum_nbufs(2) * n, dtype=torch.float32, device="cuda")
    st = det.det_accum()
    det.det_grad_accum_init(st, 2, 2, 2, n, bufs)
    acc = oracle.Accum(2, 2, 2, n)
    for m in range(8):
        gm = oracle.prim("mul", g, np.full(n, 1.0 + 0.125 * m, F))
        det.det_grad_accum_push(st, dev(gm))
        acc.push(gm)
    red = empty((n,), F)
    det.det_grad_accum_result(st, red)
    _sync()
    ored = acc.result()
    assert_same_bits(host(red), ored, "reduced gradient")
    p = _bf16_normal((n,), 0.02, 17)
    m0, v0 = np.zeros(n, F), np.zeros(n, F)
    dp, dm, dv = dev(p), dev(m0), dev(v0)
    desc = det.det_adamw_desc(3e-4, 0.9, 0.95, 1e-8, 0.1, 1)
    det.det_adamw_step(desc, det.DET_BF16, dp, red, dm, dv, n)
    _sync()
    op, om, ov = oracle.adamw(p, ored, m0, v0, 3e-4, 0.9, 0.95, 1e-8, 0.1, 1)
    assert_same_bits(host(dp, np.uint16), op, "parameters")
    assert_same_bits(host(dm), om, "m")
    assert_same_bits(host(dv), ov, "v")
    assert det.det_tensor_hash(dp, n * 2, ws(det.det_tensor_hash_ws_bytes(n * 2))) == oracle.tensor_hash(op)
