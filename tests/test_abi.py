"""The C-ABI library loads and exports every symbol that include/det.h and include/det_test.h declare (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = set()
    for h in ("det.h", "det_test.h"):
        src = open(os.path.join(ROOT, "include", h)).read()
        src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
        names |= set(re.findall(r"\b(det_[a-z0-9_]+)\s*\(", src))
    return sorted(names)


def test_header_symbols_are_exported():
    from paper_2609_17380_b200 import build
    so = build.build()
    lib = ctypes.CDLL(so)
    names = _declared()
    assert len(names) >= 35
    missing = [n for n in names if not hasattr(lib, n)]
    assert not missing, missing


def test_host_side_argument_checks():
    # error paths that return before any launch work without a GPU
    from paper_2609_17380_b200 import build
    lib = ctypes.CDLL(build.build())
    lib.det_sum_ws_bytes.restype = ctypes.c_size_t
    assert lib.det_sum_ws_bytes(ctypes.c_size_t(1200000000)) >= 4 * (1200000000 // 16384)
    assert lib.det_grad_accum_nbufs(8) == 5 and lib.det_grad_accum_nbufs(1) == 2 and lib.det_grad_accum_nbufs(7) == 4
    assert lib.det_grad_accum_nbufs(0) == -1
    assert lib.det_rmsnorm_fwd(0, None, None, 4, 8, ctypes.c_float(0), None, None, None) == -1      # DET_ERR_ARG
    buf = ctypes.create_string_buffer(4096)
    addr = ctypes.addressof(buf)
    a16 = ctypes.c_void_p((addr + 255) // 256 * 256)
    a1 = ctypes.c_void_p(a16.value + 4)
    assert lib.det_rmsnorm_fwd(0, a16, None, 4, 12, ctypes.c_float(0), a16, a16, None) == -2        # D % 8
    assert lib.det_rmsnorm_fwd(0, a1, None, 4, 8, ctypes.c_float(0), a16, a16, None) == -3          # alignment
    assert lib.det_linear_fwd(a16, a16, a16, a16, 100, 128, 128, a16, a16, None, None) == -2        # M % 128
    assert lib.det_linear_fwd(a16, a16, a16, a16, 128, 128, 1 << 17, a16, a16, None, None) == -5    # int32 range
    assert lib.det_attn_fwd(a16, a16, a16, 128, 1, 1, 1, 100, 0, a16, 128, a16, None) == -2         # S % 64
    assert lib.det_attn_fwd(a16, a16, a16, 512, 1, 4, 3, 128, 0, a16, 512, a16, None) == -2         # H % Hkv
    assert lib.det_attn_fwd(a16, a16, a16, 128, 1, 1, 1, 128, 100, a16, 128, a16, None) == -2       # window % 128
    assert lib.det_xent_fwd(a16, a16, 4, 8, ctypes.c_float(0), a16, a16, a16, a16, a16, ctypes.c_size_t(8), None, None) == -4
    # the attention forward of arithmetic version 2: shape limits, alignment, workspace size
    lib.det_attn_fwd_v2_ws_bytes.restype = ctypes.c_size_t
    need = lib.det_attn_fwd_v2_ws_bytes(1, 2, 256)
    assert need >= 2 * 256 * 256 * 6 and lib.det_attn_fwd_v2_ws_bytes(0, 2, 256) == 0
    big = ctypes.c_size_t(1 << 40)
    assert lib.det_attn_fwd_v2(a16, a16, a16, 768, 1, 2, 100, a16, 256, a16, a16, big, None, None) == -2      # S % 128
    assert lib.det_attn_fwd_v2(a16, a16, a16, 768, 1, 2, 16384, a16, 256, a16, a16, big, None, None) == -2    # S > 8192
    assert lib.det_attn_fwd_v2(a16, a16, a16, 128, 1, 2, 256, a16, 256, a16, a16, big, None, None) == -2      # ld < H * 128
    assert lib.det_attn_fwd_v2(a1, a16, a16, 768, 1, 2, 256, a16, 256, a16, a16, big, None, None) == -3       # alignment
    assert lib.det_attn_fwd_v2(a16, a16, a16, 768, 1, 2, 256, a16, 256, a16, a16, ctypes.c_size_t(need - 1), None, None) == -4
    assert lib.det_attn_fwd_v2(None, a16, a16, 768, 1, 2, 256, a16, 256, a16, a16, big, None, None) == -1     # null operand
