"""Per-kernel timing of libdet on one GPU: CUDA events around each C-ABI call, L2 flushed between iterations.

    python -m paper_2609_17380_b200.kbench [--case NAME ...] [--iters N] [--small] [--json]

Cases follow the benchmark configurations: the order-fixed reductions (RMSNorm 16384x2048 f32, cross-entropy
4096x50304, sum of squares over 1.2e9 f32), the 1B-shaped linear set at 8192 tokens per micro-batch, attention
(4 x 16 heads x 2048), the LM head, accumulation, AdamW and the hash.  `--small` shrinks every case to a few hundred
MB for profiler captures.  Rates are algorithmic bytes (or integer / floating-point operations) per second.
"""
import argparse
import json
import sys

import torch

import paper_2609_17380_b200 as det

F32, I16, I8, I32 = torch.float32, torch.int16, torch.int8, torch.int32
_flush = None


def flush_l2():
    global _flush
    if _flush is None:
        _flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    _flush.zero_()


def timeit(fn, iters, warm=2):
    for _ in range(warm):
        fn()
    ts = []
    for _ in range(iters):
        flush_l2()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1))
    ts.sort()
    return ts[len(ts) // 2]


def randn_bf16(n, std=1.0):
    return (torch.randn(n, device="cuda") * std).to(torch.bfloat16).view(I16)


def ws(nbytes):
    return torch.empty(int(nbytes) + 256, dtype=torch.uint8, device="cuda")


def case_sumsq(small):
    n = 100_000_000 if small else 1_200_000_000
    x = torch.randn(n, device="cuda") * 1e-3
    out = torch.empty(1, device="cuda")
    w = ws(det.det_sum_ws_bytes(n))
    return (lambda: det.det_sum(x, n, 1, out, w)), 4.0 * n, "B"


def case_grad_norm(small):
    """Global L2 norm and clip coefficient over one flat gradient of 1.2e9 f32 ~ N(0, 1e-3)."""
    n = 100_000_000 if small else 1_200_000_000
    x = torch.randn(n, device="cuda") * 1e-3
    norm, coef = torch.empty(1, device="cuda"), torch.empty(1, device="cuda")
    w = ws(det.det_grad_norm_ws_bytes([x]))
    return (lambda: det.det_grad_norm([x], 1.0, norm, coef, w)), 4.0 * n, "B"


def case_rmsnorm(small, bwd):
    rows, D = 16384, 2048
    x, dy = torch.randn(rows * D, device="cuda"), torch.randn(rows * D, device="cuda")
    g = 1 + 0.02 * torch.randn(D, device="cuda")
    y, rstd, dg = torch.empty_like(x), torch.empty(rows, device="cuda"), torch.empty(D, device="cuda")
    w = ws(det.det_rmsnorm_bwd_ws_bytes(rows, D))
    det.det_rmsnorm_fwd(det.DET_F32, x, g, rows, D, 1e-6, y, rstd)
    if bwd:
        return (lambda: det.det_rmsnorm_bwd(det.DET_F32, dy, x, g, rstd, rows, D, y, dg, w)), 12.0 * rows * D, "B"
    return (lambda: det.det_rmsnorm_fwd(det.DET_F32, x, g, rows, D, 1e-6, y, rstd)), 8.0 * rows * D, "B"


def case_xent(small, bwd):
    rows, V = (1024 if small else 4096), 50304
    z = torch.randn(rows * V, device="cuda") * 2
    t = torch.randint(0, V, (rows,), device="cuda", dtype=I32)
    lr, lse = torch.empty(rows, device="cuda"), torch.empty(rows, device="cuda")
    lm, zm = torch.empty(1, device="cuda"), torch.empty(1, device="cuda")
    w = ws(det.det_xent_ws_bytes(rows, V))
    det.det_xent_fwd(z, t, rows, V, 0.0, lr, lse, lm, zm, w)
    if bwd:
        z2 = z.clone()
        return (lambda: det.det_xent_bwd(z2, t, lse, rows, V, 0.0, 1.0 / rows)), 8.0 * rows * V, "B"
    return (lambda: det.det_xent_fwd(z, t, rows, V, 0.0, lr, lse, lm, zm, w)), 4.0 * rows * V, "B"


LINEAR_SHAPES = {"qkv": (6144, 2048), "o": (2048, 2048), "gu": (16384, 2048), "down": (2048, 8192)}


def _linear_setup(M, N, K):
    X, W, dY = randn_bf16(M * K), randn_bf16(N * K, 0.02), randn_bf16(M * N, 0.01)
    s_w, s_x, s_u = torch.empty(N, device="cuda"), torch.empty(1, device="cuda"), torch.empty(1, device="cuda")
    qW, qWt = torch.empty(N * K, dtype=I8, device="cuda"), torch.empty(N * K, dtype=I8, device="cuda")
    qX = torch.empty(M * K, dtype=I8, device="cuda")
    w = ws(max(det.det_linear_bwd_ws_bytes(M, N, K), det.det_lsq_act_scale_init_ws_bytes(M * K)))
    det.det_lsq_weight_scale(W, N, K, 0, s_w, w)
    det.det_lsq_act_scale_init(X, M * K, s_x, w)
    det.det_lsq_quantize_weight(W, s_w, N, K, 128, qW, qWt, s_u, w)
    Y = torch.empty(M * N, dtype=I16, device="cuda")
    status = torch.zeros(1, dtype=I32, device="cuda")
    det.det_linear_fwd(X, qW, s_x, s_w, M, N, K, Y, qX, status)
    return dict(X=X, W=W, dY=dY, s_w=s_w, s_x=s_x, s_u=s_u, qW=qW, qWt=qWt, qX=qX, Y=Y, w=w, status=status)


def case_igemm(small, which):
    M = 2048 if small else 8192
    N, K = LINEAR_SHAPES[which]
    A = torch.randint(-128, 128, (M * K,), dtype=I8, device="cuda")
    B = torch.randint(-128, 128, (N * K,), dtype=I8, device="cuda")
    C = torch.empty(M * N, dtype=I32, device="cuda")
    status = torch.zeros(1, dtype=I32, device="cuda")
    return (lambda: det.det_test_igemm_tn(A, B, M, N, K, C, 0, status)), 2.0 * M * N * K, "op"


def case_linear(small, which, bwd, M=None):
    M = M or (2048 if small else 8192)
    N, K = LINEAR_SHAPES[which]
    d = _linear_setup(M, N, K)
    if bwd:
        dX = torch.empty(M * K, dtype=I16, device="cuda")
        dW, ds = torch.empty(N * K, device="cuda"), torch.empty(1, device="cuda")
        return (lambda: det.det_linear_bwd(d["dY"], d["X"], d["qX"], d["W"], d["qWt"], d["s_x"], d["s_w"], d["s_u"], M, N, K,
                                           128, dX, dW, ds, d["w"], d["status"])), 4.0 * M * N * K, "op"
    return (lambda: det.det_linear_fwd(d["X"], d["qW"], d["s_x"], d["s_w"], M, N, K, d["Y"], d["qX"], d["status"])), \
        2.0 * M * N * K, "op"


def case_attn(small, bwd, int8pv=False, fixq=False):
    B, H, S = (1, 16, 2048) if small else (4, 16, 2048)
    HD = H * 128
    qkv = randn_bf16(B * S * 3 * HD)
    out, lse = torch.empty(B * S * HD, dtype=I16, device="cuda"), torch.empty(B * H * S, device="cuda")
    p = qkv.data_ptr()
    fwd = lambda: det.det_attn_fwd(p, p + 2 * HD, p + 4 * HD, 3 * HD, B, H, S, out, HD, lse)
    unit = B * H * (S * S // 2) * 128 * 2.0
    if int8pv:   # same nominal work as the full-precision forward (one of the two contractions runs on the tensor cores)
        st = torch.zeros(1, dtype=I32, device="cuda")
        return (lambda: det.det_attn_fwd_int8pv(p, p + 2 * HD, p + 4 * HD, 3 * HD, B, H, S, out, HD, lse, st)), 2 * unit, "flop"
    if not bwd:
        return fwd, 2 * unit, "flop"
    fwd()
    dout, dqkv = randn_bf16(B * S * HD, 0.1), torch.empty(B * S * 3 * HD, dtype=I16, device="cuda")
    w = ws(det.det_attn_bwd_fixq_ws_bytes(B, H, S) if fixq else det.det_attn_bwd_ws_bytes(B, H, S))
    dp = dqkv.data_ptr()
    bwd_fn = det.det_attn_bwd_fixq if fixq else det.det_attn_bwd
    return (lambda: bwd_fn(dout, p, p + 2 * HD, p + 4 * HD, out, lse, 3 * HD, HD, B, H, S, dp, dp + 2 * HD,
                           dp + 4 * HD, 3 * HD, w)), 5 * unit, "flop"


def case_attn_v2(small):
    """Attention forward in arithmetic version 2 (not the benchmark's arithmetic): same workload as attn_fwd."""
    B, H, S = (1 if small else 4), 16, 2048
    T, dm = B * S, H * 128
    qkv = randn_bf16(T * 3 * dm)
    q, k, v = qkv, qkv[dm:], qkv[2 * dm:]
    out, lse = torch.empty(T * dm, dtype=I16, device="cuda"), torch.empty(B * H * S, device="cuda")
    w = ws(det.det_attn_fwd_v2_ws_bytes(B, H, S))
    status = torch.zeros(1, dtype=I32, device="cuda")
    flops = 2 * 2.0 * B * H * (S * (S + 1) / 2) * 128
    return (lambda: det.det_attn_fwd_v2(q, k, v, 3 * dm, B, H, S, out, dm, lse, w, status)), flops, "flop"


def case_lmhead(small, bwd):
    M, V, K = (1024 if small else 8192), 50304, 2048
    Hh, W = randn_bf16(M * K), randn_bf16(V * K, 0.02)
    lg = torch.empty(M * V, device="cuda")
    if not bwd:
        return (lambda: det.det_lmhead_fwd(Hh, W, M, V, K, lg)), 2.0 * M * V * K, "flop"
    lg.normal_(0, 1e-3)
    dH, dW = torch.empty(M * K, dtype=I16, device="cuda"), torch.empty(V * K, device="cuda")
    return (lambda: det.det_lmhead_bwd(lg, Hh, W, M, V, K, dH, dW, 1)), 4.0 * M * V * K, "flop"


def case_lmhead_v2(small):
    """The order-free LM-head forward (arithmetic version 2) on the int8 tensor cores; same nominal work as lmhead_fwd."""
    M, V, K = (1024 if small else 8192), 50304, 2048
    Hh, W = randn_bf16(M * K), randn_bf16(V * K, 0.02)
    lg = torch.empty(M * V, device="cuda")
    w = ws(det.det_lmhead_fwd_v2_ws_bytes(M, V, K))
    st = torch.zeros(1, dtype=I32, device="cuda")
    return (lambda: det.det_lmhead_fwd_v2(Hh, W, M, V, K, lg, w, st)), 2.0 * M * V * K, "flop"


def case_lmhead_bwd_v2(small):
    """Both gradient contractions of the LM head in arithmetic version 2; same nominal work as lmhead_bwd."""
    M, V, K = (1024 if small else 8192), 50304, 2048
    Hh, W = randn_bf16(M * K), randn_bf16(V * K, 0.02)
    lg = torch.empty(M * V, device="cuda").normal_(0, 1e-3)
    dH, dW = torch.empty(M * K, dtype=I16, device="cuda"), torch.empty(V * K, device="cuda")
    w = ws(det.det_lmhead_bwd_v2_ws_bytes(M, V, K))
    st = torch.zeros(1, dtype=I32, device="cuda")
    return (lambda: det.det_lmhead_bwd_v2(lg, Hh, W, M, V, K, dH, dW, w, st)), 4.0 * M * V * K, "flop"


def case_accum(small):
    n = (1 << 26) if small else (1 << 28)
    g = torch.randn(n, device="cuda")
    bufs = torch.empty(det.det_grad_accum_nbufs(2) * n, device="cuda")

    def run():
        st = det.det_accum()
        det.det_grad_accum_init(st, 2, 2, 2, n, bufs)
        for _ in range(8):
            det.det_grad_accum_push(st, g)
    return run, 8 * 12.0 * n, "B"


def case_adamw(small):
    n = (1 << 26) if small else (1 << 28)
    p, g, m, v = randn_bf16(n, 0.02), torch.randn(n, device="cuda") * 1e-3, torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
    desc = det.det_adamw_desc(3e-4, 0.9, 0.95, 1e-8, 0.1, 1)
    return (lambda: det.det_adamw_step(desc, det.DET_BF16, p, g, m, v, n)), 24.0 * n, "B"


def case_hash(small):
    n = (1 << 28) if small else (1 << 30)
    b = torch.randint(0, 255, (n,), dtype=torch.uint8, device="cuda")
    w = ws(det.det_tensor_hash_ws_bytes(n))
    return (lambda: det.det_tensor_hash(b, n, w)), 1.0 * n, "B"


def build_cases():
    c = {"sumsq": case_sumsq, "grad_norm": case_grad_norm, "rmsnorm_fwd": lambda s: case_rmsnorm(s, False), "rmsnorm_bwd": lambda s: case_rmsnorm(s, True),
         "xent_fwd": lambda s: case_xent(s, False), "xent_bwd": lambda s: case_xent(s, True),
         "attn_fwd": lambda s: case_attn(s, False), "attn_bwd": lambda s: case_attn(s, True),
         "attn_fwd_int8pv": lambda s: case_attn(s, False, True), "attn_fwd_v2": case_attn_v2,
         "attn_bwd_fixq": lambda s: case_attn(s, True, False, True),
         "lmhead_fwd": lambda s: case_lmhead(s, False), "lmhead_fwd_v2": case_lmhead_v2, "lmhead_bwd_v2": case_lmhead_bwd_v2, "lmhead_bwd": lambda s: case_lmhead(s, True),
         "accum": case_accum, "adamw": case_adamw, "hash": case_hash}
    for k in LINEAR_SHAPES:
        c["igemm_" + k] = (lambda s, k=k: case_igemm(s, k))
        c["linear_fwd_" + k] = (lambda s, k=k: case_linear(s, k, False))
        c["linear_bwd_" + k] = (lambda s, k=k: case_linear(s, k, True))
        # the 1B-shaped linear set at 16384 tokens
        c["linear16k_fwd_" + k] = (lambda s, k=k: case_linear(s, k, False, M=16384))
        c["linear16k_bwd_" + k] = (lambda s, k=k: case_linear(s, k, True, M=16384))
    return c


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--case", nargs="*", default=None)
    ap.add_argument("--iters", type=int, default=5)
    ap.add_argument("--small", action="store_true")
    ap.add_argument("--no-flush", action="store_true")
    args = ap.parse_args()
    det.load()
    cases = build_cases()
    names = args.case or list(cases)
    res = {}
    for name in names:
        fn, work, unit = cases[name](args.small)
        torch.cuda.synchronize()
        ms = timeit(fn, args.iters, warm=1 if args.iters == 1 else 2)
        rate = work / (ms / 1e3)
        res[name] = {"ms": round(ms, 4), "rate": rate / 1e9 if unit == "B" else rate / 1e12,
                     "unit": "GB/s" if unit == "B" else ("TOP/s" if unit == "op" else "TFLOP/s")}
        print(json.dumps({name: res[name]}), flush=True)
        del fn
        torch.cuda.empty_cache()
    return res


if __name__ == "__main__":
    main()
