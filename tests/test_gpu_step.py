"""Full replayed step on the GPU against the oracle's step: every post-step tensor hashes identically."""
import numpy as np
import pytest

import synth

pytestmark = pytest.mark.gpu


def _run(cfg_kwargs, seed=0):
    from oracle import step as ostep
    from paper_2609_17380_b200 import step as dstep
    cfg_kwargs = dict(cfg_kwargs)
    if cfg_kwargs.pop("rope", False):
        cfg_kwargs["rope_tables"] = synth.rope_tables(cfg_kwargs["seq"])
    cfg = dstep.ModelConfig(**cfg_kwargs)
    params = synth.model_params(cfg.as_dict(), seed=seed)
    tokens = synth.model_tokens(cfg.as_dict(), cfg.n_microbatches, seed=seed)
    got = dstep.run_step(cfg, params, tokens)
    want = ostep.run_step(cfg.as_dict(), params, tokens)
    return cfg, got, want


def _oracle_step(kw, seed):
    """The oracle's step for a configuration given as keyword arguments of ModelConfig (seeded inputs from synth)."""
    from oracle import step as ostep
    from paper_2609_17380_b200 import step as dstep
    cfg = dstep.ModelConfig(**kw).as_dict()
    n_mb = cfg["mesh"][0] * cfg["mesh"][1] * cfg["mesh"][2]
    return ostep.run_step(cfg, synth.model_params(cfg, seed=seed), synth.model_tokens(cfg, n_mb, seed=seed))


@pytest.mark.parametrize("kw", [
    dict(n_layers=2, d_model=256, n_heads=2, ffn=512, vocab=512, seq=128, micro_batch=1, mesh=(2, 2, 2)),
    dict(n_layers=1, d_model=256, n_heads=2, ffn=384, vocab=1024, seq=192, micro_batch=2, mesh=(1, 1, 3)),
    dict(n_layers=1, d_model=128, n_heads=1, ffn=256, vocab=256, seq=128, micro_batch=1, mesh=(1, 1, 1), hadamard_block=0,
         z_weight=1e-4),
    # the paper's block in miniature: grouped queries 4/1, QK-norm, RoPE, embedding norm, a sliding-window layer
    # followed by a full one, z-loss
    dict(n_layers=2, d_model=512, n_heads=4, n_kv_heads=1, ffn=384, vocab=512, seq=256, micro_batch=1, mesh=(1, 2, 1),
         qk_norm=True, rope=True, embed_norm=True, window=128, z_weight=1e-4),
    dict(n_layers=1, d_model=256, n_heads=2, n_kv_heads=2, ffn=256, vocab=256, seq=128, micro_batch=2, mesh=(1, 1, 1),
         qk_norm=True, rope=True),
    # forward P.V on the int8 tensor cores (the backward recomputes the weights in full precision)
    dict(n_layers=2, d_model=256, n_heads=2, n_kv_heads=1, ffn=256, vocab=256, seq=256, micro_batch=1, mesh=(2, 1, 1),
         pv_int8=True, window=128),
    # both integer devices of the attention: int8 P.V forward, query gradient in 64-bit fixed point backward
    dict(n_layers=2, d_model=256, n_heads=2, n_kv_heads=1, ffn=256, vocab=256, seq=384, micro_batch=1, mesh=(1, 2, 1),
         pv_int8=True, dq_fixed=True, qk_norm=True, rope=True),
])
def test_step_hashes_match_oracle(kw):
    cfg, got, want = _run(kw)
    assert got["status"] == 0
    assert got["losses"] == [np.float32(x) for x in want["losses"]]
    assert np.float32(got["grad_norm"]) == np.float32(want["grad_norm"])
    bad = [k for k, h in want["hashes"].items() if got["hashes"][k] != h]
    assert not bad, bad
    # the device state equals the oracle's post-step tensors element by element as well
    r = got["replay"]
    host = r.params_to_host()
    for name, arr in want["params"].items():
        assert np.array_equal(host[name].reshape(-1).view(np.uint8), np.ascontiguousarray(arr).reshape(-1).view(np.uint8)), name
    assert abs(got["loss"] - np.log(cfg.vocab)) < 0.5      # random init: loss ~ log V


def test_step_with_separate_quantiser_passes_gives_the_same_hashes():
    """The step driver lets the producers write the linears' int8 inputs; with that switched off every linear runs its own
    quantiser pass (the unfused definition): same hashes, and both equal the oracle's."""
    import torch
    from paper_2609_17380_b200 import step as dstep
    kw = dict(n_layers=2, d_model=256, n_heads=2, ffn=512, vocab=512, seq=128, micro_batch=1, mesh=(1, 2, 1))
    want = _oracle_step(kw, 11)
    cfg = dstep.ModelConfig(**kw)
    params = synth.model_params(cfg.as_dict(), seed=11)
    tok = torch.from_numpy(np.ascontiguousarray(synth.model_tokens(cfg.as_dict(), 2, seed=11), dtype=np.int32)).cuda()
    for fuse in (False, True):
        r = dstep.Replay(cfg)
        r.fuse_quant = fuse
        r.load_params(params)
        r.calibrate(tok[0])
        got = r.step(tok)
        assert got["status"] == 0
        assert not [k for k, h in want["hashes"].items() if got["hashes"][k] != h], fuse


def test_step_in_arithmetic_version_2_matches_its_oracle():
    """The step with the LM-head contractions in arithmetic version 2 (order-free, on the int8 tensor cores) against the
    oracle's step in the same version: every hash; and it is a different arithmetic from version 1 (the hashes differ)."""
    kw = dict(n_layers=1, d_model=256, n_heads=2, ffn=512, vocab=512, seq=128, micro_batch=2, mesh=(2, 1, 2))
    cfg, got, want = _run(dict(kw, arith=2), seed=12)
    assert got["status"] == 0
    assert got["losses"] == [np.float32(x) for x in want["losses"]]
    assert not [k for k, h in want["hashes"].items() if got["hashes"][k] != h]
    v1 = _oracle_step(kw, 12)
    assert v1["hashes"]["grad"] != want["hashes"]["grad"]
    assert abs(v1["loss"] - want["loss"]) < 1e-3


def test_full_width_step_matches_oracle():
    """One replayed step at the benchmark's full width (d_model 2048, 16 heads, FFN 8192, sequence 2048, micro-batch 4,
    Hadamard 128, CTA-pair GEMMs on every linear, the 268 MB attention workspace, the driver's shared scratch buffers at
    their real sizes), one layer and an 8192-entry vocabulary so that the oracle's step takes minutes, not hours.  The
    expected hashes are the oracle's: read from tests/golden/full_width_step.json (written by make_full_width_step.py,
    which imports only the oracle and the input generator) while the oracle's sources are the ones that file was made
    from, recomputed with the oracle otherwise."""
    import importlib.util
    import json
    import os
    from paper_2609_17380_b200 import step as dstep
    gdir = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
    spec = importlib.util.spec_from_file_location("make_full_width_step", os.path.join(gdir, "make_full_width_step.py"))
    mk = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mk)
    want = None
    if os.path.exists(mk.OUT):
        stored = json.load(open(mk.OUT))
        if stored.get("key") == mk.source_key():
            want = stored
    if want is None:
        want = mk.compute()
    cfg = dstep.ModelConfig(**mk.CASE)
    params = synth.model_params(cfg.as_dict(), seed=mk.SEED)
    tokens = synth.model_tokens(cfg.as_dict(), 1, seed=mk.SEED)
    got = dstep.run_step(cfg, params, tokens)
    assert got["status"] == 0
    assert [np.float32(x) for x in got["losses"]] == [np.float32(x) for x in want["losses"]]
    assert np.float32(got["grad_norm"]) == np.float32(want["grad_norm"])
    bad = [k for k, h in want["hashes"].items() if got["hashes"][k] != h]
    assert not bad, bad


@pytest.mark.parametrize("world", [1, 2, 4, 8])
def test_sharded_fold_on_device_matches_single_replay(world):
    """The multi-GPU step with its transport replaced by plain copies, all ranks played one after the other on one
    GPU: micro-batch gradients are cut into the ranks' slices, every slice is folded with the library's accumulator
    at its own offset and length, and the state after clip + AdamW hashes like the single-device replay."""
    import torch
    import paper_2609_17380_b200 as det
    from paper_2609_17380_b200 import step as dstep
    from paper_2609_17380_b200.dist import ShardPlan, fold_slices
    kw = dict(n_layers=1, d_model=256, n_heads=2, ffn=384, vocab=512, seq=128, micro_batch=1, mesh=(2, 2, 2))
    cfg = dstep.ModelConfig(**kw)
    params = synth.model_params(cfg.as_dict(), seed=3)
    tokens = synth.model_tokens(cfg.as_dict(), cfg.n_microbatches, seed=3)
    want = _oracle_step(kw, 3)                      # the expectation is the oracle's single-process step
    n = want["grad"].size
    plan = ShardPlan(cfg.n_microbatches, world, n)
    r = dstep.Replay(cfg, accum_len=plan.chunk, gout_len=plan.padded)
    r.load_params(params)
    tok = torch.from_numpy(np.ascontiguousarray(tokens, dtype=np.int32)).cuda()
    r.calibrate(tok[0])
    r.prepare_weights()
    recv = [torch.empty((plan.M, plan.chunk), dtype=torch.float32, device="cuda") for _ in range(world)]
    for rank in range(world):
        for m in plan.local_microbatches(rank):
            r.forward(tok[m])
            r.backward()
            for c in range(world):
                lo, hi = plan.bounds(c)
                recv[c][m, :hi - lo].copy_(r.gmb[lo:hi])
    for c in range(world):
        lo, hi = plan.bounds(c)
        if hi > lo:
            fold_slices(det, cfg.mesh, r.abufs, [recv[c][m, :hi - lo] for m in range(plan.M)],
                        r.gout_padded[c * plan.chunk:c * plan.chunk + hi - lo])
    r.optimizer()
    got = r.hashes()
    bad = [k for k, h in want["hashes"].items() if got[k] != h]
    assert not bad, bad


def test_sharded_replay_class_single_rank():
    """ShardedReplay with one rank takes no collective and must reproduce the plain replay."""
    import torch
    from paper_2609_17380_b200 import step as dstep
    from paper_2609_17380_b200.dist import ShardedReplay
    kw = dict(n_layers=1, d_model=256, n_heads=2, ffn=384, vocab=512, seq=128, micro_batch=1, mesh=(2, 1, 3))
    cfg = dstep.ModelConfig(**kw)
    params = synth.model_params(cfg.as_dict(), seed=5)
    tokens = synth.model_tokens(cfg.as_dict(), cfg.n_microbatches, seed=5)
    want = _oracle_step(kw, 5)
    rep = ShardedReplay(cfg, 0, 1)
    rep.r.load_params(params)
    tok = torch.from_numpy(np.ascontiguousarray(tokens, dtype=np.int32)).cuda()
    rep.calibrate(tok[0])
    got = rep.step(tok)
    assert got["status"] == 0 and got["losses"] == [np.float32(x) for x in want["losses"]]
    bad = [k for k, h in want["hashes"].items() if got["hashes"][k] != h]
    assert not bad, bad


def test_two_steps_and_replay_from_a_dump(tmp_path):
    """Two consecutive optimizer steps match the oracle's two steps; a replay that starts from the state dumped after
    the first step reproduces the second step's hashes."""
    import torch
    from oracle import step as ostep
    from paper_2609_17380_b200 import step as dstep
    kw = dict(n_layers=1, d_model=256, n_heads=2, ffn=256, vocab=512, seq=128, micro_batch=1, mesh=(2, 1, 2))
    cfg = dstep.ModelConfig(**kw)
    params = synth.model_params(cfg.as_dict(), seed=7)
    toks = [synth.model_tokens(cfg.as_dict(), cfg.n_microbatches, seed=70 + i) for i in range(2)]
    # oracle: step 1 (with calibration), then step 2 from its parameters and moments
    o1 = ostep.run_step(cfg.as_dict(), params, toks[0])
    c2 = dict(cfg.as_dict(), step=2)
    o2 = ostep.run_step(c2, o1["params"], toks[1], opt={"m": o1["m"], "v": o1["v"]}, calibrate=False)
    # device: two steps in one replay
    r = dstep.Replay(cfg)
    r.load_params(params)
    t0, t1 = (torch.from_numpy(np.ascontiguousarray(t, dtype=np.int32)).cuda() for t in toks)
    r.calibrate(t0[0])
    g1 = r.step(t0)
    dump = str(tmp_path / "after_step1.npz")
    r.cfg.step = 2
    r.save_state(dump)
    g2 = r.step(t1)
    assert not [k for k, h in o1["hashes"].items() if g1["hashes"][k] != h]
    assert not [k for k, h in o2["hashes"].items() if g2["hashes"][k] != h]
    # a fresh replay from the dump
    r2 = dstep.Replay(dstep.ModelConfig(**kw))
    r2.load_state(dump)
    assert r2.cfg.step == 2
    g2b = r2.step(t1)
    assert g2b["hashes"] == g2["hashes"] and g2b["losses"] == g2["losses"]


def _sharded_worker(rank, world, port, kw, outdir):
    """One rank of the sharded replay; both ranks share the one GPU (their kernels never wait on each other, only the
    host blocks in the process group), gloo carries the CUDA tensors."""
    import os
    import torch
    import torch.distributed as dist
    from paper_2609_17380_b200 import step as dstep
    from paper_2609_17380_b200.dist import ShardedReplay
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        torch.cuda.set_device(0)
        cfg = dstep.ModelConfig(**kw)
        params = synth.model_params(cfg.as_dict(), seed=9)
        tokens = synth.model_tokens(cfg.as_dict(), cfg.n_microbatches, seed=9)
        rep = ShardedReplay(cfg, rank, world)
        rep.r.load_params(params)
        tok = torch.from_numpy(np.ascontiguousarray(tokens, dtype=np.int32)).cuda()
        rep.calibrate(tok[0])
        out = rep.step(tok)
        with open(os.path.join(outdir, "rank%d.txt" % rank), "w") as f:
            f.write(repr((out["hashes"], out["losses"], out["status"])))
    finally:
        dist.destroy_process_group()


def test_sharded_replay_two_ranks_on_one_gpu(tmp_path):
    """The whole ShardedReplay step on two ranks (point-to-point slice exchange, fold, gather, replicated optimizer):
    both ranks end with the single-replay hashes."""
    import socket
    import torch.multiprocessing as mp
    from paper_2609_17380_b200 import step as dstep
    kw = dict(n_layers=1, d_model=256, n_heads=2, ffn=384, vocab=512, seq=128, micro_batch=1, mesh=(2, 2, 2))
    want = _oracle_step(kw, 9)
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    mp.spawn(_sharded_worker, args=(2, port, kw, str(tmp_path)), nprocs=2, join=True)
    for rank in range(2):
        hashes, losses, status = eval(open(tmp_path / ("rank%d.txt" % rank)).read())
        assert status == 0 and losses == [np.float32(x) for x in want["losses"]]
        assert not [k for k, h in want["hashes"].items() if hashes[k] != h], "rank %d" % rank


def _peer_worker_gpu(rank, world, port, outdir):
    """Symmetric-memory construction of the peer-fold reducer with a one-rank NCCL group: the stash is allocated and
    rendezvoused through torch's symmetric memory and the fold reads it through the raw addresses it reports."""
    import os
    import torch
    import torch.distributed as dist
    import paper_2609_17380_b200 as det
    from paper_2609_17380_b200.dist import ShardPlan, fold_slices, make_peer_reducer
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=torch.device("cuda", 0))
    try:
        mesh, n = (2, 2, 2), 100000
        plan = ShardPlan(8, 1, n)
        red = make_peer_reducer(plan, 0, "cuda")
        g = [torch.from_numpy(np.random.default_rng(50 + m).standard_normal(n).astype(np.float32)).cuda() for m in range(8)]
        for j in range(8):
            red.scatter(j, g[j])
        pool = torch.empty(det.det_grad_accum_nbufs(2) * plan.chunk, dtype=torch.float32, device="cuda")
        out = torch.zeros(plan.padded, dtype=torch.float32, device="cuda")
        got = red.fold_and_gather(lambda sl, o: fold_slices(det, mesh, pool, sl, o), out).cpu().numpy()
        import oracle                                   # the expectation is the oracle's accumulator (Algorithm 1 + 2)
        oa = oracle.Accum(2, 2, 2, n)
        for j in range(8):
            oa.push(g[j].cpu().numpy())
        same = np.array_equal(got[:n].view(np.uint32), oa.result().view(np.uint32))
        # the NCCL in-place all-gather of the slice exchange accepts a slice of its own output (one rank: a no-op copy)
        from paper_2609_17380_b200.dist import ShardedReducer
        sr = ShardedReducer(plan, 0, "cuda")
        before = out.clone()
        sr._gather(out, out[:plan.chunk])
        torch.cuda.synchronize()
        same = same and bool((out == before).all().item()) and not sr.host_stage
        with open(os.path.join(outdir, "ok.txt"), "w") as f:
            f.write("1" if same else "0")
    finally:
        dist.destroy_process_group()


def test_peer_fold_symmetric_memory_one_rank(tmp_path):
    import socket
    import torch.multiprocessing as mp
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    mp.spawn(_peer_worker_gpu, args=(1, port, str(tmp_path)), nprocs=1, join=True)
    assert open(tmp_path / "ok.txt").read() == "1"
