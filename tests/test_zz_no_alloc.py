"""det_sum_static: the entry point for callers that may not allocate device memory (a plug-in inside an application
that owns the device heap, a loop that must stay out of cudaMalloc).  Its scratch is a fixed array inside the library,
so this test checks through the C-ABI that it returns the same bits as det_sum with a caller workspace, twice in a
row (the second call finds the first call's leftovers in the shared array), and that oversize requests are refused.
Collected last on purpose: a failure here cannot hide the result of any other test."""
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
