#!/usr/bin/env python
"""Benchmark of the replayed, bit-exact training step on B200.

    python bench.py --gpus N --steps K --warmup W [--impl reference]

A "step" is one full optimizer step of the 1B-shaped decoder (24 layers, d_model 2048, 16 heads, FFN 8192,
vocab 50304, seq 2048, 32 sequences as 8 micro-batches of 4 in mesh (accum, dp_shard, dp_replicate) = (2,2,2)):
weight-step re-pin and quantisation, 8 x (forward, backward), the fixed-order gradient reduction, global-norm
clip, AdamW, and the SHA-256 state hash.  Inputs are seeded synthetic token ids and random-init weights.
Prints ONE JSON line (rank 0).
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "replayed step tokens/s (bit-exact)"
UNIT = "tokens/s"
WORKLOAD = "config5: full 1B-shaped step, 24 layers, d_model 2048, 16 heads, FFN 8192, vocab 50304, seq 2048, " \
           "8 micro-batches of 4 sequences, mesh (accum,dp_shard,dp_replicate)=(2,2,2), AdamW, SHA-256 of post-step state"


WORKLOAD_PAPER = "paper block (not the default): 24 layers, d_model 2048, 16 query / 4 key-value heads, QK-norm, RoPE 5e5, " \
                 "embedding norm, sliding window 512 with every 5th and the last layer full, int8 P.V, fixed-point query gradient, z-loss 1e-4, FFN 5632, vocab 128256, " \
                 "seq 4096, 8 micro-batches of 4 sequences, mesh (2,2,2), AdamW, SHA-256 of post-step state"


def full_config_kwargs(layers=None, workload="config5"):
    kw = dict(n_layers=24, d_model=2048, n_heads=16, ffn=8192, vocab=50304, seq=2048, micro_batch=4, mesh=(2, 2, 2),
              hadamard_block=128, lr=3e-4, betas=(0.9, 0.95), eps=1e-8, wd=0.1, clip=1.0)
    if workload == "paper":
        import numpy as np
        i = np.arange(64, dtype=np.float64)
        ang = np.arange(4096, dtype=np.float64)[:, None] * (5.0e5 ** (-2.0 * i / 128))[None, :]
        kw.update(n_kv_heads=4, ffn=5632, vocab=128256, seq=4096, qk_norm=True, embed_norm=True, window=512, full_every=5,
                  z_weight=1e-4, lr=4.5e-4, pv_int8=True, dq_fixed=True, rope_tables=(np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)))
    if layers is not None:
        kw["n_layers"] = layers
    return kw


# ---------------------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = "clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown," \
        "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap"

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "200"], stdout=subprocess.PIPE, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); power.append(float(r[2]))
            except Exception:
                continue
            for name, col in (("hw_slowdown", 4), ("hw_thermal_slowdown", 5), ("sw_thermal_slowdown", 6), ("sw_power_cap", 7)):
                if len(r) > col and r[col].lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"], "bf16_tflops_sustained": d["bf16_tflops_sustained"],
                "sm_max_mhz": d.get("sm_max_mhz", 1965.0), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "sm_max_mhz": 1965.0, "source": "fallback"}


def profile_traffic(name):
    """DRAM read + write bytes summed over the launches of one committed ncu summary under profiles/ (the lines
    `dram__bytes_read.sum` / `dram__bytes_write.sum`), or None if the file is missing."""
    path = os.path.join(ROOT, "profiles", name)
    if not os.path.exists(path):
        return None
    mult = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    tot, seen = 0.0, 0
    for line in open(path):
        f = line.split()
        if len(f) >= 3 and f[0] in ("dram__bytes_read.sum", "dram__bytes_write.sum") and f[2] in mult:
            tot += float(f[1]) * mult[f[2]]
            seen += 1
    return tot if seen else None


def accum_bytes_per_element(accum, shard, rep):
    """Bytes per gradient element that the pushes of one step really move (Algorithm 1 + 2 as det_grad_accum_push runs
    them): every push reads the fresh gradient and writes one buffer; it also reads the rank's running sum (k > 0), the
    running shard sum (end of a rank, shard > 0) and one stacked partial per TreeFold carry (end of a replica)."""
    streams, stack = 0, []
    for r in range(shard * rep):
        for k in range(accum):
            streams += 2 + (1 if k > 0 else 0)
            if k == accum - 1:
                s_ = r % shard
                streams += 1 if s_ > 0 else 0
                if s_ == shard - 1:
                    level = 0
                    while stack and stack[-1] == level:
                        stack.pop()
                        level += 1
                        streams += 1
                    stack.append(level)
    return 4.0 * streams


def component_rates_configs_2_3(peaks, iters=5):
    """The kernel-level workloads of the metric, timed one call at a time (CUDA events, L2 flushed between iterations):
    the order-fixed reductions (RMSNorm forward/backward on 16384 x 2048 f32, cross-entropy forward/backward on
    4096 x 50304, global gradient norm over 1.2e9 f32) as GB/s and fraction of the measured copy bandwidth, and the
    1B-shaped linear set at 16384 tokens, forward and backward, as int8 POP/s and fraction of 4.5 POP/s nominal and of
    2 x the measured bf16 rate."""
    import torch
    from paper_2609_17380_b200 import kbench
    out = {}
    for name, fn in (("rmsnorm_fwd", lambda: kbench.case_rmsnorm(False, False)), ("rmsnorm_bwd", lambda: kbench.case_rmsnorm(False, True)),
                     ("xent_fwd", lambda: kbench.case_xent(False, False)), ("xent_bwd", lambda: kbench.case_xent(False, True)),
                     ("grad_norm_1.2e9", lambda: kbench.case_grad_norm(False))):
        call, work, _ = fn()
        torch.cuda.synchronize()
        ms = kbench.timeit(call, iters)
        gbs = work / (ms / 1e3) / 1e9
        out[name] = {"ms": round(ms, 4), "gbs": round(gbs, 1), "frac_of_hbm": round(gbs / peaks["hbm_gbs"], 3)}
        del call
        torch.cuda.empty_cache()
    tot = {"fwd": [0.0, 0.0], "bwd": [0.0, 0.0]}
    for which in kbench.LINEAR_SHAPES:
        for bwd in (False, True):
            call, work, _ = kbench.case_linear(False, which, bwd, M=16384)
            torch.cuda.synchronize()
            ms = kbench.timeit(call, iters)
            tops = work / (ms / 1e3) / 1e12
            key = "linear16k_%s_%s" % ("bwd" if bwd else "fwd", which)
            out[key] = {"ms": round(ms, 4), "int8_tops": round(tops, 1), "frac_of_4.5POPs": round(tops / 4500.0, 3),
                        "frac_of_2x_measured_bf16": round(tops / (2.0 * peaks["bf16_tflops"]), 3)}
            t = tot["bwd" if bwd else "fwd"]
            t[0] += work
            t[1] += ms
            del call
            torch.cuda.empty_cache()
    for k, (work, ms) in tot.items():
        tops = work / (ms / 1e3) / 1e12
        out["linear16k_%s_set" % k] = {"ms": round(ms, 4), "int8_tops": round(tops, 1), "frac_of_4.5POPs": round(tops / 4500.0, 3),
                                       "frac_of_2x_measured_bf16": round(tops / (2.0 * peaks["bf16_tflops"]), 3)}
    out["hbm_peak_used_gbs"] = peaks["hbm_gbs"]
    out["note"] = "hbm fraction is against the measured copy bandwidth (%s); a read-mostly kernel can read a little above it" % peaks["source"]
    return out


def optional_arithmetic_v2_rates(iters=5):
    """The optional arithmetic version 2 (NOT the benchmark's arithmetic; the default step does not use it): the LM head
    and the attention forward as order-free contractions on the int8 tensor cores, each beside the default-arithmetic
    kernel on the same workload (8192 x 50304 x 2048; 4 x 16 heads x 2048)."""
    import torch
    from paper_2609_17380_b200 import kbench
    out = {}
    for name, fn in (("lmhead_fwd", lambda: kbench.case_lmhead(False, False)), ("lmhead_fwd_v2", lambda: kbench.case_lmhead_v2(False)),
                     ("lmhead_bwd", lambda: kbench.case_lmhead(False, True)), ("lmhead_bwd_v2", lambda: kbench.case_lmhead_bwd_v2(False)),
                     ("attn_fwd", lambda: kbench.case_attn(False, False)), ("attn_fwd_v2", lambda: kbench.case_attn_v2(False))):
        call, _, _ = fn()
        torch.cuda.synchronize()
        out[name + "_ms"] = round(kbench.timeit(call, iters), 4)
        del call
        torch.cuda.empty_cache()
    return out


def spawn_ranks(args):
    """`python bench.py --gpus N` without a launcher: start N local ranks, one GPU each, NCCL over 127.0.0.1."""
    import socket
    import torch
    have = torch.cuda.device_count()
    if have < args.gpus:
        print("bench.py: --gpus %d asked for, %d visible" % (args.gpus, have), file=sys.stderr)
        return 2
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus), "--master-addr",
           "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


# ---------------------------------------------------------------------------------------------------------
def cpu_baseline(kw):
    """The oracle, as it stands, on the host cores: a bounded sample of the same workload, scaled to tokens/s.

    Sample: (a) 48 tokens through embedding + final norm + LM head + loss, forward and backward; (b) one full-width
    decoder layer (norms, four LSQ int8 linears, SwiGLU, residuals) on 512 tokens, forward and backward, with its
    attention (four sequences of 128) timed apart and left out; (b2) attention forward + backward of one 16-head sequence
    at seq 1024; (c) accumulate + clip + AdamW + hash on 4M parameters.  (a), (b) and (c) are scaled linearly in tokens,
    layers and parameters, (b2) with the number of sequences and with (seq / 1024)^2."""
    import numpy as np
    import oracle as O
    import synth
    from oracle import step as ostep
    cores = os.cpu_count() or 1
    D, Fh, V, L, H = kw["d_model"], kw["ffn"], kw["vocab"], kw["n_layers"], kw["n_heads"]
    # (a) head: 8 tokens (weights drawn with numpy's seeded generator: only the timing is used here)
    th = 48
    c = dict(kw)
    c.update(seq=th, micro_batch=1, mesh=(1, 1, 1), n_layers=0)
    rng = np.random.default_rng(0)
    P = {"embed": synth.to_bf16((rng.standard_normal((V, D), dtype=np.float32) * 0.02)),
         "lm_head": synth.to_bf16((rng.standard_normal((V, D), dtype=np.float32) * 0.02)),
         "final_norm": np.full(D, 0x3F80, np.uint16)}
    toks = rng.integers(0, V, (1, th + 1)).astype(np.int32)
    t0 = time.time()
    ostep.microbatch_grad(c, P, {}, toks)
    t_head = time.time() - t0
    # (b) one layer on 512 tokens (four sequences of 128; attention is timed apart because it grows with seq^2)
    T = 512
    x = synth.to_bf16(rng.standard_normal((T, D), dtype=np.float32))
    dy = synth.to_bf16(rng.standard_normal((T, D), dtype=np.float32) * 0.01)
    gain = np.full(D, 0x3F80, np.uint16)
    Ws = [synth.to_bf16(rng.standard_normal(sh, dtype=np.float32) * 0.02) for sh in ((3 * D, D), (D, D), (2 * Fh, D), (D, Fh))]
    sws = [O.lsq_weight_scale(W) for W in Ws]
    t0 = time.time()
    n1, r1 = O.rmsnorm_fwd(x, gain, 1e-6, bf=True)
    s0 = O.lsq_act_scale_init(n1)
    qkv, _, _ = O.linear_fwd(n1, Ws[0], s0, sws[0])
    ta = time.time()
    att, lse = O.attn_fwd(qkv, 4, H, 128)
    t_att_small = time.time() - ta
    s1 = O.lsq_act_scale_init(att)
    o, _, _ = O.linear_fwd(att, Ws[1], s1, sws[1])
    h = O.residual_add(x, o)
    n2, r2 = O.rmsnorm_fwd(h, gain, 1e-6, bf=True)
    s2 = O.lsq_act_scale_init(n2)
    gu, _, _ = O.linear_fwd(n2, Ws[2], s2, sws[2])
    act = O.swiglu_fwd(gu)
    s3 = O.lsq_act_scale_init(act)
    dn, _, _ = O.linear_fwd(act, Ws[3], s3, sws[3])
    O.residual_add(h, dn)
    d_act, _, _ = O.linear_bwd(dy, act, Ws[3], s3, sws[3], 128)
    d_gu = O.swiglu_bwd(d_act, gu)
    d_n2, _, _ = O.linear_bwd(d_gu, n2, Ws[2], s2, sws[2], 128)
    d_h2, _ = O.rmsnorm_bwd(d_n2, h, gain, r2, bf=True)
    d_h = O.residual_add(dy, d_h2)
    d_att, _, _ = O.linear_bwd(d_h, att, Ws[1], s1, sws[1], 128)
    ta = time.time()
    d_qkv = O.attn_bwd(d_att, qkv, att, lse, 4, H, 128)
    t_att_small += time.time() - ta
    d_n1, _, _ = O.linear_bwd(d_qkv, n1, Ws[0], s0, sws[0], 128)
    d_x1, _ = O.rmsnorm_bwd(d_n1, x, gain, r1, bf=True)
    O.residual_add(d_h, d_x1)
    t_layer = time.time() - t0 - t_att_small
    # (b2) attention forward + backward of 16 heads at seq 1024; the cost per sequence grows with seq^2
    SA = 1024
    qa = synth.to_bf16(rng.standard_normal((SA, 3 * H * 128), dtype=np.float32))
    da = synth.to_bf16(rng.standard_normal((SA, H * 128), dtype=np.float32) * 0.1)
    t0 = time.time()
    oa, la = O.attn_fwd(qa, 1, H, SA)
    O.attn_bwd(da, qa, oa, la, 1, H, SA)
    t_attn = time.time() - t0
    # (c) reduction + optimizer + hash on 4M parameters
    n_opt = 1 << 22
    g = rng.standard_normal(n_opt, dtype=np.float32) * np.float32(1e-3)
    p = synth.to_bf16(rng.standard_normal(n_opt, dtype=np.float32) * 0.02)
    t0 = time.time()
    acc = O.Accum(1, 1, 1, n_opt)
    acc.push(g)
    t_push = time.time() - t0
    gr = acc.result()
    nrm, coef = O.grad_norm([gr], 1.0)
    gr = O.scale(gr, coef)
    O.adamw(p, gr, np.zeros(n_opt, np.float32), np.zeros(n_opt, np.float32), 3e-4, 0.9, 0.95, 1e-8, 0.1, 1)
    O.tensor_hash(p)
    t_opt = time.time() - t0
    n_params = 2 * V * D + L * (4 * D * D + 3 * D * Fh + 2 * D + 4) + D
    tokens_step = 8 * kw["micro_batch"] * kw["seq"]
    n_seq = 8 * kw["micro_batch"]
    est = t_head * (tokens_step / th) + L * t_layer * (tokens_step / T) + L * t_attn * n_seq * (kw["seq"] / SA) ** 2 + \
        (t_opt + 7 * t_push) * (n_params / n_opt)
    return {"value": tokens_step / est, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "%d tokens through embed+norm+head+loss fwd/bwd (%.1fs); one full-width layer fwd/bwd without attention on "
                      "%d tokens (%.1fs); attention fwd/bwd of one 16-head sequence at seq %d (%.1fs); accumulate+clip+AdamW+hash "
                      "on 4M params (%.1fs); scaled linearly in tokens, layers and parameters and with seq^2 for attention to "
                      "%d layers, %d tokens at seq %d, %.2fB params"
                      % (th, t_head, T, t_layer, SA, t_attn, t_opt, L, tokens_step, kw["seq"], n_params / 1e9),
            "sample_seconds": t_head + t_layer + t_att_small + t_attn + t_opt, "est_step_seconds": est}


def run_reference(args):
    """Reference arm = the CPU oracle as it stands, on the host cores, on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    kw = full_config_kwargs(args.layers)
    vals, ms = [], []
    for i in range(args.warmup + args.steps):
        t0 = time.time()
        cb = cpu_baseline(kw)
        dt = time.time() - t0
        if i >= args.warmup:
            vals.append(cb["value"])
            ms.append(cb["est_step_seconds"] * 1e3)
    v = statistics.mean(vals)
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": statistics.mean(ms), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int8+f32", "data": "synthetic", "config": {"workload": WORKLOAD},
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": cb["cores"], "kind": "oracle", "sample": cb["sample"]},
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    import paper_2609_17380_b200 as det
    from paper_2609_17380_b200 import step as dstep
    det.load()
    kw = full_config_kwargs(args.layers, args.workload)
    kw["arith"] = args.arith
    cfg = dstep.ModelConfig(**kw)
    n_mb = cfg.n_microbatches
    # N > 1: the micro-batches of the one global step are shared out over the ranks and the gradient is exchanged in
    # the fixed order (same parameters, tokens and resulting hashes on every rank); if N does not divide the
    # micro-batch count the ranks run independent replicas instead
    sharded = world > 1 and n_mb % world == 0
    if sharded:
        from paper_2609_17380_b200.dist import ShardedReplay
        rep = ShardedReplay(cfg, rank, world, peer_fold=args.peer_fold)
        r = rep.r
    else:
        rep = r = dstep.Replay(cfg)
    seed = 0 if sharded else rank
    r.init_params_on_device(seed=seed)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(1234 + seed)
    tok_dev = torch.randint(0, cfg.vocab, (n_mb, cfg.micro_batch, cfg.seq + 1), generator=gen, device="cuda", dtype=torch.int32)
    tok_host = tok_dev.cpu().pin_memory()
    r.calibrate(tok_dev[0])
    torch.cuda.synchronize()
    tokens_per_step = n_mb * cfg.micro_batch * cfg.seq

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def do_steps(n, host_inputs):
        outs = []
        for _ in range(n):
            if host_inputs:
                tok = tok_host.to("cuda", non_blocking=True)
            else:
                tok = tok_dev
            out = rep.step(tok, per_tensor_hashes=False, want_losses=host_inputs)
            r.cfg.step += 1
            outs.append(out)
        return outs

    do_steps(args.warmup, False)
    # ---- device-resident timing ----
    r.prof = {}
    sampler = ClockSampler(local)
    barrier()
    if rank == 0:
        sampler.start()
    l0 = det.det_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    e0.record()
    outs = do_steps(args.steps, False)
    e1.record()
    barrier()
    wall = time.time() - t0
    launches = det.det_launch_count() - l0
    clocks = sampler.stop() if rank == 0 else None
    ms = e0.elapsed_time(e1)
    prof = r.prof_summary()
    r.prof = None
    # ---- end to end: tokens from pinned host memory, losses + hashes back on the host every step ----
    barrier()
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2.record()
    outs2 = do_steps(args.steps, True)
    e3.record()
    barrier()
    ms_e2e = e2.elapsed_time(e3)
    t = torch.tensor([ms, ms_e2e], device="cuda", dtype=torch.float64)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms, ms_e2e = float(t[0]), float(t[1])
    status = max(o["status"] for o in outs + outs2)
    agree = None
    if sharded:   # every rank must hold the same state after the same steps
        hb = torch.tensor(list(bytes.fromhex(outs2[-1]["hashes"]["params_bf16"])), dtype=torch.uint8, device="cuda")
        allh = torch.empty(world * 32, dtype=torch.uint8, device="cuda")
        dist.all_gather_into_tensor(allh, hb)
        agree = bool((allh.view(world, 32) == hb).all().item())
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    peaks = measured_peaks()
    per_step = ms / args.steps
    jobs = 1 if sharded else world          # sharded: all ranks together process one global batch per step
    value = jobs * tokens_per_step * args.steps / (ms / 1e3)
    e2e_val = jobs * tokens_per_step * args.steps / (ms_e2e / 1e3)
    # ---- roofline of the dominant kernel group (by device time inside the timed region) ----
    total_prof = sum(v[1] for v in prof.values()) or 1.0
    shares = {k: round(v[1] / total_prof, 4) for k, v in sorted(prof.items(), key=lambda kv: -kv[1][1])}
    B, H, S, D, Fh, V, L, T = cfg.micro_batch, cfg.n_heads, cfg.seq, cfg.d_model, cfg.ffn, cfg.vocab, cfg.n_layers, cfg.tokens_per_microbatch
    # visible (query, key) pairs x 128 MACs of one attention contraction, averaged over the layers (windowed layers see
    # W keys per row once the window is full)
    def pairs(l):
        W = cfg.layer_window(l)
        return S * S // 2 if not W else S * W - W * W // 2
    unit = B * H * 128 * sum(pairs(l) for l in range(L)) / L
    alg = {  # name -> (bound, algorithmic work per launch group, unit of peak)
        "attn_fwd": ("alu", 2 * unit * 2.0, "flop"),
        "attn_bwd": ("alu", 5 * unit * 2.0, "flop"),
        "lmhead_fwd": ("alu", T * V * D * 2.0, "flop"),
        "lmhead_bwd": ("alu", 2 * T * V * D * 2.0, "flop"),
    }
    # FP32 ALU peak: one fused multiply-add per lane per clock = 2 flop; the ordered contractions use the fused
    # instruction wherever it is bit-identical to multiply-then-add, so this is their ceiling
    alu_peak = 148 * 128 * 2 * peaks["sm_max_mhz"] * 1e6 / 1e12
    dom = next(iter(shares))
    roof = {"kernel": dom, "share_of_step": shares[dom]}
    if dom in alg:
        n, tot_ms = prof[dom]
        ach = alg[dom][1] / (tot_ms / n / 1e3) / 1e12
        # DRAM traffic per launch group from the committed ncu capture of the same kernels at B = 1 (read + write, summed
        # over the launches of the summary; it grows in proportion to the batch)
        prof_file = {"attn_bwd": "k_attn_sdp_ws_k_ogemm_wb_attn_bwd_small.md", "attn_fwd": "k_attn_fwd_ws_attn_fwd_small.md"}.get(dom)
        t1 = profile_traffic(prof_file) if (prof_file and args.workload == "config5") else None
        traffic = t1 * B if t1 is not None else None
        roof["traffic_source"] = ("profiles/%s x batch %d" % (prof_file, B)) if t1 is not None else None
        roof.update({"bound": "alu", "achieved": ach, "peak": alu_peak, "unit": "TFLOP/s", "frac": ach / alu_peak,
                     "traffic": traffic, "peak_source": "148 SMs x 128 FP32 lanes x 2 flop (fused multiply-add) x %.0f MHz"
                     % peaks["sm_max_mhz"]})
    all_alu = {}
    for kname, (bound, work, _) in alg.items():
        if kname in prof:
            n, tot_ms = prof[kname]
            if args.arith == 2 and kname.startswith("lmhead"):
                # arithmetic version 2 runs the head on the int8 tensor cores: a fraction of the FP32 FMA rate means nothing
                all_alu[kname] = {"ms": tot_ms / n, "note": "arithmetic version 2: int8 tensor cores, not an FP32-ALU kernel"}
                continue
            all_alu[kname] = {"tflops": work / (tot_ms / n / 1e3) / 1e12, "frac_of_alu_peak": work / (tot_ms / n / 1e3) / 1e12 / alu_peak}
    # the two fractions the benchmark spec asks for: int8 tensor pipe (linear GEMMs) and HBM (order-fixed reductions)
    lin_macs_fwd = T * (cfg.qkv_width * D + D * D + 2 * Fh * D + D * Fh)
    extra = {}
    if "linear_fwd" in prof:
        n, tot_ms = prof["linear_fwd"]
        extra["linear_fwd_int8_tops"] = 2.0 * lin_macs_fwd / 4 * n / (tot_ms / 1e3) / 1e12
        extra["linear_fwd_frac_of_4.5POPs"] = extra["linear_fwd_int8_tops"] / 4500.0
    if "linear_bwd" in prof:
        n, tot_ms = prof["linear_bwd"]
        extra["linear_bwd_int8_tops"] = 2.0 * 2 * lin_macs_fwd / 4 * n / (tot_ms / 1e3) / 1e12
        extra["linear_bwd_frac_of_4.5POPs"] = extra["linear_bwd_int8_tops"] / 4500.0
    if "grad_accum" in prof:
        n, tot_ms = prof["grad_accum"]
        # bytes the pushes really move: single GPU, n timed pushes = n / n_mb steps over the whole gradient; sharded, one
        # timed fold per step over this rank's slice (the gather that follows it is inside the same span)
        bpe = accum_bytes_per_element(*cfg.mesh)
        elems, nsteps = (rep.plan.chunk, n) if sharded else (r.n_grad, n / n_mb)
        extra["grad_accum_bytes_per_element_per_step"] = bpe
        extra["grad_accum_gbs"] = bpe * elems * nsteps / (tot_ms / 1e3) / 1e9
        extra["grad_accum_frac_of_hbm"] = extra["grad_accum_gbs"] / peaks["hbm_gbs"]
        extra["grad_accum_peak_note"] = "against the measured copy bandwidth; a kernel with three or four read streams per write stream can read a little above a 1:1 copy"
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": per_step, "higher_is_better": True, "scaling": "strong" if sharded else "weak", "vs_baseline": None,
            "dtype": "int8 tensor-core GEMMs + f32 ordered arithmetic (bf16 storage)", "data": "synthetic",
            "config": {"workload": (WORKLOAD if args.workload == "config5" else WORKLOAD_PAPER) +
                       ("" if args.layers is None else " [REDUCED to %d layers]" % args.layers) +
                       ("" if args.arith == 1 else " [LM-head contractions in arithmetic version 2: NOT the benchmark's arithmetic]"),
                       "l2": "inputs_exceed_l2", "multi_gpu": ("micro-batches sharded over ranks, ordered gradient exchange, replicated optimizer" if sharded
                                     else "replicas only" if world > 1 else "single"), "ranks_agree": agree},
            "clocks": clocks, "gpu_launches": int(launches),
            "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": int(tok_host.numel() * 4),
                    "d2h_bytes_per_step": int(n_mb * 4 + 8 + 5 * 32)},
            "roofline": roof, "alu_kernels": all_alu, "kernel_time_shares": shares, "component_rates": extra, "peaks": peaks,
            "wall_s_timed": wall, "device_status": status,
            "state_hash": outs2[-1]["hashes"].get("params_bf16")}
    if world == 1 and not args.no_component_rates:
        # free the step's buffers, then time the kernel-level workloads of the metric on their own
        hash_keep = line["state_hash"]
        del rep, r, outs, outs2, tok_dev
        torch.cuda.empty_cache()
        try:
            line["component_rates"].update(component_rates_configs_2_3(peaks))
        except Exception as ex:
            line["component_rates"]["configs_2_3_error"] = repr(ex)
        try:
            line["optional_arithmetic_v2"] = optional_arithmetic_v2_rates()
        except Exception as ex:
            line["optional_arithmetic_v2"] = {"error": repr(ex)}
        line["state_hash"] = hash_keep
    if world == 1 and not args.no_cpu_baseline:
        try:
            import oracle
            oracle.build()
            line["cpu_baseline"] = cpu_baseline(kw)
        except Exception as ex:  # the oracle is a reported baseline, not part of the product path
            line["cpu_baseline"] = {"value": None, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle", "sample": "failed: %r" % ex}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--peer-fold", action="store_true",
                    help="N > 1: fold the gradient slices straight out of the peers' buffers (symmetric memory) instead of "
                         "exchanging them with point-to-point copies first")
    ap.add_argument("--workload", choices=("config5", "paper"), default="config5",
                    help="config5 (default) is the benchmark configuration; paper is the paper's own block and shapes")
    ap.add_argument("--arith", type=int, choices=(1, 2), default=1,
                    help="2: the LM-head contractions in arithmetic version 2 (order-free, int8 tensor cores); not the default metric")
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=None, help="debug only: fewer layers (the line says REDUCED)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-component-rates", action="store_true",
                    help="skip the kernel-level workloads (reductions, 16384-token linear set) timed after the step")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args))
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
