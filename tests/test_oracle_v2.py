"""Pins of the version-2 oracle (order-free, exactly defined LM-head contraction): hand-worked slices, a brute-force
restatement in exact rational arithmetic that starts from the VALUES (not the bit fields), the case in which nothing is
truncated and the result must be the correctly rounded exact dot product, order-freedom, an error bound against float64,
and the special rows."""
from fractions import Fraction

import numpy as np

import synth
from oracle import v2

F = np.float32


def _val(h):
    return float(synth.from_bf16(np.array([h], np.uint16))[0])


def _rn_f32(fr):
    """Exactly representable-in-double rational -> binary32, nearest even (one rounding), flushed below 2^-126."""
    d = float(fr)
    assert Fraction(d) == fr
    r = F(d)
    return F(np.copysign(0.0, r)) if abs(r) < 2.0 ** -126 else r


def _brute(a_bits, b_bits):
    """Version-2 contraction of two rows from their values: scale = 2^(floor(log2 max|x|) - 13), T = trunc(x / scale)."""
    def aligned(bits):
        vals = [Fraction(_val(h)) for h in bits]
        vals = [v if abs(v) >= Fraction(2) ** -126 else Fraction(0) for v in vals]      # flushed subnormals
        mx = max(abs(v) for v in vals)
        if mx == 0:
            return [0] * len(vals), Fraction(1)
        e = 0
        while Fraction(2) ** (e + 1) <= mx:
            e += 1
        while Fraction(2) ** e > mx:
            e -= 1
        scale = Fraction(2) ** (e - 13)
        T = [int(abs(v) / scale) * (1 if v >= 0 else -1) for v in vals]                  # truncation toward zero
        return T, scale
    Ta, sa = aligned(a_bits)
    Tb, sb = aligned(b_bits)
    return _rn_f32(sum(x * y for x, y in zip(Ta, Tb)) * sa * sb)


def test_slices_by_hand():
    x = synth.to_bf16(np.array([[1.0, 0.5, -3.0, 0.0, 3.0 * 2.0 ** -7, -2.0 ** -13, 2.0 ** -14]], F))
    hi, lo, E = v2.slice_rows(x)
    assert E[0] == 128                                   # 3.0 = 1.5 * 2^1
    T = hi.astype(np.int32) * 128 + lo.astype(np.int32)
    # units of 2^(128 - 140) = 2^-12: 1.0 -> 4096, 0.5 -> 2048, -3.0 -> -12288, 3 * 2^-7 -> 96, -2^-13 -> -0 (half a unit,
    # truncated), 2^-14 -> 0
    assert T[0].tolist() == [4096, 2048, -12288, 0, 96, 0, 0]
    assert hi[0].tolist() == [32, 16, -96, 0, 0, 0, 0] and lo[0].tolist() == [0, 0, 0, 0, 96, 0, 0]
    assert np.abs(hi.astype(np.int32)).max() <= 127 and np.abs(lo.astype(np.int32)).max() <= 127


def test_slices_reconstruct_the_truncated_values():
    x = synth.normal_bf16((5, 256), 1.0, seed=3, tid=1)
    x[1] = synth.to_bf16((synth.normal_f32(256, 1.0, seed=3, tid=2) * np.exp2(np.arange(256) % 20 - 10.0)).astype(F))   # wide range
    hi, lo, E = v2.slice_rows(x)
    T = hi.astype(np.int64) * 128 + lo.astype(np.int64)
    xv = synth.from_bf16(x).astype(np.float64)
    for r in range(5):
        unit = 2.0 ** (int(E[r]) - 140)
        want = np.trunc(xv[r] / unit)
        assert np.array_equal(T[r], want.astype(np.int64)), r
        assert np.max(np.abs(xv[r] - T[r] * unit)) < unit
        assert (hi[r].astype(np.int32) * lo[r].astype(np.int32) >= 0).all()      # both slices carry the sign


def test_brute_force_in_exact_rational_arithmetic():
    rng = np.random.default_rng(0)
    for trial in range(6):
        K = [1, 3, 8, 17, 32, 40][trial]
        a = synth.to_bf16((rng.standard_normal((3, K)) * np.exp2(rng.integers(-9, 9, (3, K)))).astype(F))
        b = synth.to_bf16((rng.standard_normal((4, K)) * np.exp2(rng.integers(-20, 3, (4, K)))).astype(F))
        got = v2.lmhead_fwd(a, b)
        for m in range(3):
            for n in range(4):
                want = _brute(a[m], b[n])
                assert got[m, n].view(np.uint32) == F(want).view(np.uint32), (trial, m, n, got[m, n], want)


def test_without_truncation_the_result_is_the_correctly_rounded_dot_product():
    """Rows whose values all lie within a factor 64 of the row's largest are kept exactly, so the contraction is the exact
    dot product of the bf16 values rounded once: a closed form that no ordered binary32 chain reaches in general."""
    rng = np.random.default_rng(1)
    K = 96
    a = synth.to_bf16((rng.uniform(1.0, 1.99, (4, K)) * np.exp2(rng.integers(-6, 1, (4, K))) * rng.choice([-1, 1], (4, K))).astype(F))
    b = synth.to_bf16((rng.uniform(1.0, 1.99, (5, K)) * np.exp2(rng.integers(-9, -3, (5, K))) * rng.choice([-1, 1], (5, K))).astype(F))
    a[:, 0] = synth.to_bf16(np.array([1.5], F))[0]          # pins the row exponents at the top of the range
    b[:, 0] = synth.to_bf16(np.array([2.0 ** -4 * 1.25], F))[0]
    got = v2.lmhead_fwd(a, b)
    av, bv = synth.from_bf16(a), synth.from_bf16(b)
    for m in range(4):
        for n in range(5):
            exact = sum(Fraction(float(x)) * Fraction(float(y)) for x, y in zip(av[m], bv[n]))
            assert got[m, n].view(np.uint32) == _rn_f32(exact).view(np.uint32), (m, n)


def test_order_free_and_close_to_float64():
    a = synth.normal_bf16((6, 512), 1.0, seed=5, tid=1)
    b = synth.normal_bf16((7, 512), 0.02, seed=5, tid=2)
    got = v2.lmhead_fwd(a, b)
    perm = np.random.default_rng(2).permutation(512)
    assert np.array_equal(v2.lmhead_fwd(a[:, perm], b[:, perm]).view(np.uint32), got.view(np.uint32))
    av, bv = synth.from_bf16(a).astype(np.float64), synth.from_bf16(b).astype(np.float64)
    ref = av @ bv.T
    _, _, Ea = v2.slice_rows(a)
    _, _, Eb = v2.slice_rows(b)
    ua, ub = np.exp2(Ea.astype(np.float64) - 140), np.exp2(Eb.astype(np.float64) - 140)
    # every operand is off by less than one unit of its row: |error| <= sum(|a| ub + |b| ua + ua ub) + half an ulp of the result
    bound = np.abs(av).sum(1)[:, None] * ub[None, :] + ua[:, None] * np.abs(bv).sum(1)[None, :] + 512 * ua[:, None] * ub[None, :]
    assert np.all(np.abs(got - ref) <= bound + np.abs(ref) * 2.0 ** -24)
    assert np.max(np.abs(got - ref)) < 2e-3 * np.max(np.abs(ref))      # and in practice far inside it


def test_special_rows():
    a = synth.normal_bf16((4, 64), 1.0, seed=6, tid=1)
    b = synth.normal_bf16((3, 64), 1.0, seed=6, tid=2)
    a[1] = 0
    a[2, 5] = 0x7F80                                   # +inf
    b[1, 9] = 0x7FC0                                   # NaN
    a[3, :] = 0x0001                                   # subnormal bf16 values count as zero
    got = v2.lmhead_fwd(a, b)
    assert got[1, 0].view(np.uint32) == 0 and got[3, 2].view(np.uint32) == 0        # +0
    assert np.isnan(got[2]).all() and np.isnan(got[:, 1]).all()
    assert np.isfinite(got[0, 0]) and np.isfinite(got[0, 2])
    _, _, E = v2.slice_rows(a)
    assert E[1] == 0 and E[3] == 0 and (E[2] >> 30) == 1


def test_backward_is_the_contraction_on_transposed_operands_and_close_to_float64():
    """dH and dW of version 2 against float64 (the bound of the forward applies), bf16 rounding of dlogits pinned against
    the shared input generator's converter, and shapes / dtypes."""
    rng = np.random.default_rng(7)
    M, V, K = 24, 40, 32
    Hh = synth.normal_bf16((M, K), 1.0, seed=8, tid=1)
    W = synth.normal_bf16((V, K), 0.02, seed=8, tid=2)
    dl = (rng.standard_normal((M, V)) * 1e-3).astype(F)
    dl[0, 0] = 1e-41                                       # a subnormal gradient is flushed before it is rounded
    assert np.array_equal(v2._f2bf(dl[1:]), synth.to_bf16(dl[1:])) and v2._f2bf(dl[:1])[0, 0] == 0
    dH, dW = v2.lmhead_bwd(dl, Hh, W)
    assert dH.shape == (M, K) and dH.dtype == np.uint16 and dW.shape == (V, K) and dW.dtype == F
    g = synth.from_bf16(v2._f2bf(dl)).astype(np.float64)
    rH = g @ synth.from_bf16(W).astype(np.float64)
    rW = g.T @ synth.from_bf16(Hh).astype(np.float64)
    assert np.max(np.abs(synth.from_bf16(dH) - rH)) <= np.max(np.abs(rH)) * 2.0 ** -8
    assert np.max(np.abs(dW - rW)) <= np.max(np.abs(rW)) * 1e-3
    # brute force of single elements in exact rational arithmetic from the values
    for (m, k) in ((0, 0), (5, 7), (23, 31)):
        want = _brute(v2._f2bf(dl)[m], np.ascontiguousarray(W[:, k]))
        assert synth.from_bf16(dH[m:m + 1, k:k + 1])[0, 0] == synth.from_bf16(synth.to_bf16(np.array([want], F)))[0]
    for (v, k) in ((0, 0), (11, 3), (39, 31)):
        want = _brute(np.ascontiguousarray(v2._f2bf(dl)[:, v]), np.ascontiguousarray(Hh[:, k]))
        assert dW[v, k].view(np.uint32) == F(want).view(np.uint32)


# ---------------------------------------------------------------- attention in version 2
def _qkv(S, H=1):
    return np.zeros((S, 3 * H * 128), np.uint16)


def test_attention_v2_uniform_weights_are_exact():
    """q = 0: every logit is 0, every weight exactly 1, l_i = i + 1 exactly, and u is the exact integer sum of small
    integer values (nothing is truncated: all within 2^-6 of the column's largest), so the output is
    bf16(fmul(sum_{j<=i} v_jc, fdiv(1, i + 1))) and lse_i = log(i + 1) by the oracle's own log."""
    import oracle
    S = 70
    rng = np.random.default_rng(3)
    qkv = _qkv(S)
    vals = rng.integers(-3, 4, (S, 128)).astype(F)
    vals[0] = 3.0                                            # every column's largest magnitude is 3: exponent 128
    qkv[:, 128:256] = synth.to_bf16(rng.standard_normal((S, 128)).astype(F))     # keys do not matter when q = 0
    qkv[:, 256:] = synth.to_bf16(vals)
    out, lse = v2.attn_fwd(qkv, 1, 1, S)
    csum = np.cumsum(vals.astype(np.int64), 0)
    for i in (0, 1, 2, 31, 63, 69):
        il = F(F(1.0) / F(i + 1))
        want = synth.to_bf16((csum[i].astype(F) * il).astype(F))
        assert np.array_equal(out[i], want), i
        assert lse[0, 0, i] == F(F(0.0) + oracle.prim("log", np.array([F(i + 1)], F))[0])


def test_attention_v2_logits_are_the_v2_contraction():
    """One query against itself and one earlier key (S = 2): lse_0 is the logit s_00 itself, and the pair of rows goes
    through the brute-force restatement of the contraction (exact rational arithmetic from the values)."""
    rng = np.random.default_rng(5)
    scale = F(float.fromhex("0x1.6a09e6p-4"))
    for t in range(4):
        qkv = _qkv(1)
        qkv[0, :128] = synth.to_bf16((rng.standard_normal(128) * np.exp2(rng.integers(-8, 3, 128))).astype(F))
        qkv[0, 128:256] = synth.to_bf16((rng.standard_normal(128) * np.exp2(rng.integers(-8, 3, 128))).astype(F))
        qkv[0, 256:] = synth.to_bf16(rng.standard_normal(128).astype(F))
        out, lse = v2.attn_fwd(qkv, 1, 1, 1)
        want = F(_brute(qkv[0, :128], qkv[0, 128:256]) * scale)
        assert lse[0, 0, 0] == want
        # a single key: weight 1, u = the value aligned to its own exponent (exact), l = 1
        assert np.array_equal(out[0], qkv[0, 256:])


def test_attention_v2_is_causal_and_close_to_float64():
    import math
    B, H, S = 1, 2, 200
    qkv = synth.normal_bf16((B * S, 3 * H * 128), 1.0, seed=0, tid=60)
    out, lse = v2.attn_fwd(qkv, B, H, S)
    x = synth.from_bf16(qkv).astype(np.float64).reshape(B, S, 3, H, 128)
    q, k, v = (x[:, :, i].transpose(0, 2, 1, 3) for i in range(3))
    s = q @ k.transpose(0, 1, 3, 2) / math.sqrt(128)
    s = np.where(np.tril(np.ones((S, S), bool)), s, -np.inf)
    l64 = np.log(np.exp(s - s.max(-1, keepdims=True)).sum(-1)) + s.max(-1)
    o64 = (np.exp(s - l64[..., None]) @ v).transpose(0, 2, 1, 3).reshape(B * S, H * 128)
    # truncation of the aligned values costs at most 2^-13 of the largest product per term; bf16 rounding of the weights and
    # of the output dominates
    assert np.abs(synth.from_bf16(out) - o64).max() < 0.02 and np.allclose(lse, l64, rtol=2e-4, atol=2e-4)
    # causality: later keys and values leave earlier rows bit-identical -- EXCEPT through the exponent of a value column,
    # which is taken over all keys of the sequence: keep the columns' largest magnitudes where they are
    qkv2 = qkv.copy()
    tail = synth.normal_bf16((S - 150, 2 * H * 128), 0.25, seed=1, tid=61)
    qkv2[150:, H * 128:] = tail
    e_before = ((qkv[:, 2 * H * 128:] >> 7) & 0xFF).max(0)
    e_after = ((qkv2[:, 2 * H * 128:] >> 7) & 0xFF).max(0)
    assert np.array_equal(e_before, e_after)                 # the recipe above keeps every column exponent
    out2, lse2 = v2.attn_fwd(qkv2, B, H, S)
    assert np.array_equal(out2[:150], out[:150]) and np.array_equal(lse2[:, :, :150], lse[:, :, :150])


def test_attention_v2_does_not_depend_on_the_order_of_the_head_dimensions():
    """The contraction over the 128 dimensions is order-free: permuting the dimensions of q and k together leaves every
    logit, hence lse and the output, bit-identical (version 1's ordered dot does not have this property)."""
    B, H, S = 1, 1, 96
    rng = np.random.default_rng(11)
    qkv = synth.to_bf16((rng.standard_normal((S, 384)) * np.exp2(rng.integers(-6, 3, (S, 384)))).astype(F))
    out, lse = v2.attn_fwd(qkv, B, H, S)
    perm = rng.permutation(128)
    qkv2 = qkv.copy()
    qkv2[:, :128] = qkv[:, :128][:, perm]
    qkv2[:, 128:256] = qkv[:, 128:256][:, perm]
    out2, lse2 = v2.attn_fwd(qkv2, B, H, S)
    assert np.array_equal(out, out2) and np.array_equal(lse, lse2)
