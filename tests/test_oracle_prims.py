"""Pins for the oracle's primitives: each is checked against something other than itself
(IEEE facts, closed forms, double-precision libm, hashlib, hand-worked values)."""
import hashlib
import math

import numpy as np

import oracle
import synth

F = np.float32


def ulp_diff(a, b):
    a = np.asarray(a, F).view(np.int32).astype(np.int64)
    b = np.asarray(b, F).view(np.int32).astype(np.int64)
    a = np.where(a < 0, -(a & 0x7FFFFFFF), a)
    b = np.where(b < 0, -(b & 0x7FFFFFFF), b)
    return np.abs(a - b)


def test_unfused_multiply_add():
    # Sec. 2.1: fused and unfused a*b+c differ by up to one ULP; the oracle must give the unfused value.
    rng = np.random.default_rng(1)
    a = (1 + rng.random(20000)).astype(F)
    b = (1 + rng.random(20000)).astype(F)
    prod = a.astype(np.float64) * b.astype(np.float64)       # exact: 48 significant bits
    fused = (prod + b.astype(np.float64)).astype(F)            # sum exact in double, one rounding
    unfused = (prod.astype(F).astype(np.float64) + b.astype(np.float64)).astype(F)  # two roundings
    differ = fused != unfused
    assert differ.sum() > 100 and ulp_diff(fused, unfused).max() == 1
    got = oracle.prim("mul_add", a, b)
    assert np.array_equal(got, unfused)


def test_flush_to_zero():
    tiny = F(2.0 ** -126)
    sub = F(2.0 ** -130)
    assert oracle.prim("add", [sub], [0])[0] == 0            # DAZ on input
    assert oracle.prim("mul", [tiny], [0.5])[0] == 0         # FTZ on result
    r = oracle.prim("mul", [-tiny], [0.5])
    assert r[0] == 0 and np.signbit(r[0])                    # sign-preserving zero
    assert oracle.prim("add", [tiny], [tiny])[0] == F(2.0 ** -125)
    assert oracle.prim("sub", [F(1.5) * tiny], [tiny])[0] == 0  # exact result 2^-127 is subnormal
    # tininess is judged on the exact value: (1 - 2^-24) * 2^-126 would round up to 2^-126 but is flushed
    almost_one = F(1 - 2.0 ** -24)
    assert oracle.prim("mul", [almost_one], [tiny])[0] == 0
    assert oracle.prim("div", [almost_one], [F(2.0 ** 126)])[0] == 0
    assert oracle.prim("mul", [F(1 + 2.0 ** -23)], [tiny])[0] == F((1 + 2.0 ** -23) * 2.0 ** -126)
    assert oracle.prim("max", [-0.0], [0.0]).view(np.uint32)[0] == 0
    assert oracle.prim("max", [0.0], [-0.0]).view(np.uint32)[0] == 0
    # a NaN operand of max is ignored, whichever side it is on (maxNum); only two NaNs give a NaN
    nan = F("nan")
    assert oracle.prim("max", [nan], [F(-3.0)])[0] == F(-3.0) and oracle.prim("max", [F(-3.0)], [nan])[0] == F(-3.0)
    assert np.isnan(oracle.prim("max", [nan], [nan])[0])


def test_bf16_roundtrip_and_ties():
    pats = np.arange(65536, dtype=np.uint32)
    exp = (pats >> 7) & 0xFF
    keep = (exp != 0xFF) & (exp != 0)           # finite, not subnormal
    h = pats[keep].astype(np.uint16)
    assert np.array_equal(oracle.f2bf(oracle.bf2f(h)), h)
    # ties to even: 0x3F808000 is half-way between 0x3F80 and 0x3F81 -> even (0x3F80)
    tie = np.array([0x3F808000, 0x3F818000, 0x3F808001, 0x3F807FFF], np.uint32).view(F)
    assert list(oracle.f2bf(tie)) == [0x3F80, 0x3F82, 0x3F81, 0x3F80]
    # agreement with an independent integer implementation on random data
    x = synth.normal_f32(100000, 3.0, seed=5)
    assert np.array_equal(oracle.f2bf(x), synth.to_bf16(x))


def test_det_sum_shape():
    assert oracle.det_sum(np.array([2 ** 24, 1, 1, 1], F)) == F(16777218)   # sequential gives 16777216
    assert oracle.det_sum(np.array([2 ** 24, 0, 0, 0, 1, 0, 1], F)) == F(16777218)  # A + (B + C)
    assert oracle.det_sum(np.array([1, 2 ** 24, 0, 0, 0, 0, 1], F)) == F(16777216)  # carry meets the block last
    z = oracle.det_sum(np.full(5, -0.0, F))
    assert z == 0 and np.signbit(z)                                          # carried, not padded with +0
    assert oracle.det_sum(np.zeros(0, F)) == 0
    x = np.arange(1, 5001, dtype=F)
    assert oracle.det_sum(x) == F(5000 * 5001 // 2)                          # integers below 2^24 are exact
    # pure-python restatement on a ragged length
    v = synth.normal_f32(1000, seed=3)
    cur = [F(t) for t in v]
    while len(cur) > 1:
        nxt = [F(cur[i] + cur[i + 1]) for i in range(0, len(cur) - 1, 2)]
        if len(cur) & 1:
            nxt.append(cur[-1])
        cur = nxt
    assert oracle.det_sum(v) == cur[0]


def test_det_sum_block_decomposition():
    # the tree over the whole vector equals the tree over trees of aligned power-of-two blocks
    v = synth.normal_f32(50304, 2.0, seed=9)
    leaves = [oracle.det_sum(v[i:i + 256]) for i in range(0, v.size, 256)]
    assert oracle.det_sum(np.array(leaves, F)) == oracle.det_sum(v)


def test_exp_pins():
    assert oracle.prim("exp", [0.0])[0] == 1.0
    assert oracle.prim("exp", [-np.inf, -200.0, -87.4])[0:3].tolist() == [0.0, 0.0, 0.0]
    assert np.isinf(oracle.prim("exp", [89.0])[0])
    x = np.linspace(-87.0, 88.0, 400001).astype(F)
    ref = np.exp(x.astype(np.float64))
    got = oracle.prim("exp", x)
    ok = ref > 2.0 ** -125
    assert ulp_diff(got[ok], ref[ok].astype(F)).max() <= 4
    # every bf16-representable argument in (-88, 0]: the softmax/attention use
    h = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    xb = oracle.bf2f(h)
    xb = xb[np.isfinite(xb) & (xb <= 0) & (xb > -87)]
    assert ulp_diff(oracle.prim("exp", xb), np.exp(xb.astype(np.float64)).astype(F)).max() <= 4


def test_log_pins():
    assert oracle.prim("log", [1.0]).view(np.uint32)[0] == 0           # +0 exactly
    got = oracle.prim("log", [50304.0])[0]
    assert ulp_diff(got, F(math.log(50304.0))) <= 2                     # 10.82583988
    x = np.concatenate([np.linspace(1.0, 4.0, 200001), np.logspace(0, 30, 100001)]).astype(F)
    assert ulp_diff(oracle.prim("log", x), np.log(x.astype(np.float64)).astype(F)).max() <= 4
    # the ends of the domain: a non-finite or non-positive argument stays visible (a NaN logit must not become a finite loss)
    edge = oracle.prim("log", np.array([0.0, -0.0, 1e-40, np.inf, -1.0, -np.inf, np.nan], F))
    assert edge[0] == -np.inf and edge[1] == -np.inf and edge[2] == -np.inf and edge[3] == np.inf   # 1e-40 is flushed to 0
    assert np.isnan(edge[4:]).all()


def test_reciprocal_multiply_vs_division():
    # Appendix A.3: x*(1/8) == x/8 bitwise; x*(1/6) differs from x/6 for some x (by at most one ULP)
    x = synth.normal_f32(100000, seed=11)
    assert np.array_equal(oracle.prim("mul", x, np.full_like(x, F(1 / 8))), oracle.prim("div", x, np.full_like(x, 8)))
    a = oracle.prim("mul", x, np.full_like(x, F(1.0 / 6.0)))
    b = oracle.prim("div", x, np.full_like(x, 6))
    d = ulp_diff(a, b)
    assert d.max() == 1 and (d > 0).any()


def test_sha256_and_tensor_hash():
    assert oracle.sha256(np.frombuffer(b"abc", np.uint8)) == \
        "ba7816bf8f01cfea414140de5dae2223b00361a396177a9cb410ff61f20015ad"      # FIPS 180-4 example
    assert oracle.sha256(np.zeros(0, np.uint8)) == hashlib.sha256(b"").hexdigest()
    msg = b"abcdbcdecdefdefgefghfghighijhijkijkljklmklmnlmnomnopnopq"
    assert oracle.sha256(np.frombuffer(msg, np.uint8)) == \
        "248d6a61d20638b8e5c026930c3e6039a33ce45964ff2167f6ecedd419db06c1"      # FIPS 180-4 example
    rng = np.random.default_rng(0)
    # 128 * 4096 bytes is the largest input with a single level, 128 * 128 * 4096 the largest with two
    for n in (0, 1, 55, 56, 63, 64, 65, 119, 120, 4095, 4096, 4097, 65537, 200001, 128 * 4096, 128 * 4096 + 1,
              3 * 128 * 4096 + 777, 128 * 128 * 4096 + 5000):
        b = rng.integers(0, 256, n).astype(np.uint8)
        assert oracle.sha256(b) == hashlib.sha256(b.tobytes()).hexdigest()
        d = b"".join(hashlib.sha256(b[i:i + 4096].tobytes()).digest() for i in range(0, n, 4096))
        while len(d) > 128 * 32:
            d = b"".join(hashlib.sha256(d[i:i + 4096]).digest() for i in range(0, len(d), 4096))
        root = hashlib.sha256(d + int(n).to_bytes(8, "little")).hexdigest()
        assert oracle.tensor_hash(b) == root


def test_philox_known_answers():
    kat = [((0, 0, 0, 0), (0, 0), "6627e8d5e169c58dbc57ac4c9b00dbd8"),
           ((0xFFFFFFFF,) * 4, (0xFFFFFFFF,) * 2, "408f276d41c83b0ea20bc7c66d5451fd"),
           ((0x243F6A88, 0x85A308D3, 0x13198A2E, 0x03707344), (0xA4093822, 0x299F31D0),
            "d16cfe0994fdcceb5001e42024126ea1")]
    for c, k, e in kat:
        r = synth.philox4x32_10(np.array([c], np.uint32), k)[0]
        assert "".join("%08x" % v for v in r) == e
    a = synth.normal_f32(10001, seed=1, tid=2)
    b = synth.normal_f32(20001, seed=1, tid=2)
    assert abs(a.mean()) < 0.05 and abs(a.std() - 1) < 0.05
    assert synth.normal_f32(7, seed=1, tid=2).shape == (7,) and b.size == 20001
