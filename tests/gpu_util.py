"""Helpers for the GPU parity tests: move seeded numpy inputs to the device and results back."""
import numpy as np
import torch


def dev(a):
    """numpy array -> contiguous CUDA tensor with the same bytes (uint16 bf16 bit patterns travel as int16)."""
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda()
    if a.dtype == np.uint32:
        return torch.from_numpy(a.view(np.int32)).cuda()
    return torch.from_numpy(a).cuda()


def host(t, dtype=None):
    a = t.detach().cpu().numpy()
    if dtype is not None:
        a = a.view(dtype)
    return a


def empty(shape, dtype):
    m = {np.float32: torch.float32, np.uint16: torch.int16, np.int8: torch.int8, np.int32: torch.int32,
         np.uint8: torch.uint8}
    return torch.empty(shape, dtype=m[dtype], device="cuda")


def ws(nbytes):
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device="cuda")


def same_bits(a, b):
    a = np.ascontiguousarray(a)
    b = np.ascontiguousarray(b)
    return a.shape == b.shape and a.dtype.itemsize == b.dtype.itemsize and np.array_equal(a.view(np.uint8), b.view(np.uint8))


def assert_same_bits(got, want, what=""):
    got = np.ascontiguousarray(got)
    want = np.ascontiguousarray(want)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    if not np.array_equal(got.view(np.uint8), want.view(np.uint8)):
        g = got.reshape(-1)
        w = want.reshape(-1)
        bad = np.nonzero(g.view(np.uint8).reshape(g.size, -1) != w.view(np.uint8).reshape(w.size, -1))[0]
        bad = np.unique(bad)
        i = int(bad[0])
        raise AssertionError("%s: %d of %d elements differ; first at %d: got %r want %r"
                             % (what, bad.size, g.size, i, g[i], w[i]))
