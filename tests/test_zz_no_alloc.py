"""det_sum_static: the entry point for callers that may not allocate device memory (a plug-in inside an application
that owns the device heap, a loop that must stay out of cudaMalloc).  Its scratch is a fixed array inside the library,
so this test checks through the C-ABI that it returns the same bits as det_sum with a caller workspace and as the
oracle's tree, on calls in a row (each call finds the previous call's leftovers in the shared array), at the ends of its
range (no element, one element, a length whose tree has three levels of chunk sums), and that oversize requests are
refused.  Collected last on purpose: a failure here cannot hide the result of any other test."""
import numpy as np
import pytest

import synth
from gpu_util import dev, empty, host, ws

pytestmark = pytest.mark.gpu
F = np.float32


def test_static_scratch_sum_matches_workspace_sum_twice():
    import torch
    import paper_2609_17380_b200 as det
    det.load()
    out_ref, out_new = empty((1,), F), empty((1,), F)
    # two calls in a row with different lengths, so the second one runs over what the first one left behind
    for n, seed in ((16384 * 37 + 1001, 1), (16384 * 5 + 3, 2), (300, 3)):
        x = dev(synth.normal_f32(n, 1.0, seed=seed, tid=42))
        for squares in (1, 0):
            det.det_sum(x, n, squares, out_ref, ws(det.det_sum_ws_bytes(n)))
            det.det_sum_static(x, n, squares, out_new)
            torch.cuda.synchronize()
            a, b = host(out_ref), host(out_new)
            assert a.view(np.uint32)[0] == b.view(np.uint32)[0], (n, squares, a, b)   # 0 ULP, as everywhere else
    # repeated call on the same input gives the same bits again
    det.det_sum_static(x, n, 0, out_new)
    torch.cuda.synchronize()
    assert host(out_new).view(np.uint32)[0] == host(out_ref).view(np.uint32)[0]


def test_static_scratch_sum_matches_oracle_at_the_ends_of_its_range():
    """n = 0 (+0 by definition), n = 1 (the element itself, flushed), and 16384^2 + 3 * 16384 + 5 elements: 16388 chunk sums,
    then 2, then 1, i.e. three levels, the deepest tree the fixed array is sized for short of its maximum length."""
    import torch
    import oracle
    import paper_2609_17380_b200 as det
    det.load()
    out_ref, out_new = empty((1,), F), empty((1,), F)
    big = 16384 * 16384 + 3 * 16384 + 5
    xs = np.random.default_rng(5).standard_normal(big, dtype=np.float32)
    xd = dev(xs)
    for n in (big, 1, 0, 257, big):          # the large case again after small ones: leftovers of every size in the array
        for squares in (0, 1):
            out_new.fill_(7.0)
            det.det_sum_static(xd, n, squares, out_new)
            det.det_sum(xd, n, squares, out_ref, ws(det.det_sum_ws_bytes(n)))
            torch.cuda.synchronize()
            want = oracle.sumsq(xs[:n]) if squares else oracle.det_sum(xs[:n])
            got = host(out_new).view(np.uint32)[0]
            assert got == np.array([want], F).view(np.uint32)[0], (n, squares, host(out_new), want)
            assert got == host(out_ref).view(np.uint32)[0], (n, squares)


def test_static_scratch_sum_rejects_oversize():
    import paper_2609_17380_b200 as det
    det.load()
    x = empty((16,), F)
    out = empty((1,), F)
    mx = det.det_sum_static_max_n()
    assert mx == 1 << 29
    with pytest.raises(det.DetError) as e:
        det.det_sum_static(x, mx + 1, 0, out)          # refused on the host before anything is launched
    assert e.value.code == -2
