"""Oracle-side replay of one full training step (TEST INFRASTRUCTURE ONLY).

Plain numpy orchestration of the oracle's C functions in the order the paper states a step: forward,
gradient, reduction of the micro-batch gradients in the cluster's order (Algorithm 1 + 2), clip, AdamW,
hash.  Written independently of the CUDA-side driver; they share only the seeded inputs.
"""
import numpy as np

import oracle as O
from oracle import v2 as O2

LINEARS = ("w_qkv", "w_o", "w_gu", "w_down")


def _kv(cfg):
    return cfg.get("n_kv_heads") or cfg["n_heads"]


def _window(cfg, l):
    """Sliding-window layers (Sec. 3.1): every `full_every`-th layer and the last one attend to everything."""
    W = cfg.get("window", 0)
    if not W or l == cfg["n_layers"] - 1 or (l + 1) % cfg.get("full_every", 5) == 0:
        return 0
    return W


def _specs(cfg):
    D, Fh, V, L = cfg["d_model"], cfg["ffn"], cfg["vocab"], cfg["n_layers"]
    nq = D + 2 * 128 * _kv(cfg)
    s = [("embed", (V, D))]
    if cfg.get("embed_norm"):
        s += [("embed_norm", (D,))]
    for l in range(L):
        s += [("l%d.attn_norm" % l, (D,)), ("l%d.w_qkv" % l, (nq, D)), ("l%d.w_o" % l, (D, D)),
              ("l%d.ffn_norm" % l, (D,)), ("l%d.w_gu" % l, (2 * Fh, D)), ("l%d.w_down" % l, (D, Fh)),
              ("l%d.s_x" % l, (4,))]
    return s + [("final_norm", (D,)), ("lm_head", (V, D))]


def forward(cfg, P, sw, tok, calibrate=False):
    """Returns (saved activations, loss pieces).  With calibrate, every activation step is set from its input."""
    L, H, S, B = cfg["n_layers"], cfg["n_heads"], cfg["seq"], cfg["micro_batch"]
    Hkv, D = _kv(cfg), cfg["d_model"]
    inp = tok[:, :-1].reshape(-1)
    x = O.embed_fwd(inp, P["embed"])
    saved = {"inp": inp, "layers": []}
    if cfg.get("embed_norm"):
        saved["x_emb"] = x
        x, saved["rstd_emb"] = O.rmsnorm_fwd(x, P["embed_norm"], 1e-6, bf=True)
    rope = cfg.get("rope_tables")
    for l in range(L):
        sx = P["l%d.s_x" % l]
        a = {"x": x}
        a["n1"], a["rstd1"] = O.rmsnorm_fwd(x, P["l%d.attn_norm" % l], 1e-6, bf=True)
        if calibrate:
            sx[0] = O.lsq_act_scale_init(a["n1"])[0]
        a["qkv"], _, _ = O.linear_fwd(a["n1"], P["l%d.w_qkv" % l], sx[0:1], sw["l%d.w_qkv" % l])
        # the paper's block: gain-free RMS norm of every query and key head, then the rotary embedding
        qk = np.ascontiguousarray(a["qkv"][:, :D + 128 * Hkv]).reshape(-1, 128)
        if cfg.get("qk_norm"):
            a["qk_pre"] = qk
            qk, a["rstd_qk"] = O.rmsnorm_fwd(qk, None, 1e-6, bf=True)
        if rope is not None:
            qk = O.rope(qk.reshape(B * S, H + Hkv, 128), S, rope[0], rope[1]).reshape(-1, 128)
        a["qkr"] = np.ascontiguousarray(np.concatenate([qk.reshape(B * S, -1), a["qkv"][:, D + 128 * Hkv:]], 1))
        a["att"], a["lse"] = O.attn_fwd(a["qkr"], B, H, S, Hkv=Hkv, window=_window(cfg, l), int8_pv=bool(cfg.get("pv_int8")))
        if calibrate:
            sx[1] = O.lsq_act_scale_init(a["att"])[0]
        o, _, _ = O.linear_fwd(a["att"], P["l%d.w_o" % l], sx[1:2], sw["l%d.w_o" % l])
        a["h"] = O.residual_add(x, o)
        a["n2"], a["rstd2"] = O.rmsnorm_fwd(a["h"], P["l%d.ffn_norm" % l], 1e-6, bf=True)
        if calibrate:
            sx[2] = O.lsq_act_scale_init(a["n2"])[0]
        a["gu"], _, _ = O.linear_fwd(a["n2"], P["l%d.w_gu" % l], sx[2:3], sw["l%d.w_gu" % l])
        a["act"] = O.swiglu_fwd(a["gu"])
        if calibrate:
            sx[3] = O.lsq_act_scale_init(a["act"])[0]
        dn, _, _ = O.linear_fwd(a["act"], P["l%d.w_down" % l], sx[3:4], sw["l%d.w_down" % l])
        x = O.residual_add(a["h"], dn)
        saved["layers"].append(a)
    saved["xf"] = x
    saved["nf"], saved["rstdf"] = O.rmsnorm_fwd(x, P["final_norm"], 1e-6, bf=True)
    # arithmetic version 2 (cfg["arith"] == 2) replaces the LM-head contractions by the order-free ones of oracle/v2
    saved["logits"] = (O2 if cfg.get("arith", 1) == 2 else O).lmhead_fwd(saved["nf"], P["lm_head"])
    return saved


def microbatch_grad(cfg, P, sw, tok):
    """Forward + backward of one micro-batch; returns (flat f32 gradient in canonical order, mean loss)."""
    L, H, S, B = cfg["n_layers"], cfg["n_heads"], cfg["seq"], cfg["micro_batch"]
    hb = cfg.get("hadamard_block", 128)
    Hkv, D, rope = _kv(cfg), cfg["d_model"], cfg.get("rope_tables")
    sv = forward(cfg, P, sw, tok)
    labels = tok[:, 1:].reshape(-1).astype(np.int32)
    T = labels.size
    _, lse, loss_mean, _, _ = O.xent_fwd(sv["logits"], labels, cfg.get("z_weight", 0.0))
    dlog = O.xent_bwd(sv["logits"], labels, lse, cfg.get("z_weight", 0.0), np.float32(1.0 / T))
    G = {}
    d_nf, G["lm_head"] = (O2 if cfg.get("arith", 1) == 2 else O).lmhead_bwd(dlog, sv["nf"], P["lm_head"])
    dx, G["final_norm"] = O.rmsnorm_bwd(d_nf, sv["xf"], P["final_norm"], sv["rstdf"], bf=True)
    for l in reversed(range(L)):
        a = sv["layers"][l]
        sx = P["l%d.s_x" % l]
        ds = np.zeros(4, np.float32)
        d_act, G["l%d.w_down" % l], d3 = O.linear_bwd(dx, a["act"], P["l%d.w_down" % l], sx[3:4], sw["l%d.w_down" % l], hb)
        d_gu = O.swiglu_bwd(d_act, a["gu"])
        d_n2, G["l%d.w_gu" % l], d2 = O.linear_bwd(d_gu, a["n2"], P["l%d.w_gu" % l], sx[2:3], sw["l%d.w_gu" % l], hb)
        d_h2, G["l%d.ffn_norm" % l] = O.rmsnorm_bwd(d_n2, a["h"], P["l%d.ffn_norm" % l], a["rstd2"], bf=True)
        d_h = O.residual_add(dx, d_h2)
        d_att, G["l%d.w_o" % l], d1 = O.linear_bwd(d_h, a["att"], P["l%d.w_o" % l], sx[1:2], sw["l%d.w_o" % l], hb)
        d_qkv = O.attn_bwd(d_att, a["qkr"], a["att"], a["lse"], B, H, S, Hkv=Hkv, window=_window(cfg, l),
                           fixq=bool(cfg.get("dq_fixed")))
        dqk = np.ascontiguousarray(d_qkv[:, :D + 128 * Hkv]).reshape(-1, 128)
        if rope is not None:
            dqk = O.rope(dqk.reshape(B * S, H + Hkv, 128), S, rope[0], rope[1], inverse=True).reshape(-1, 128)
        if cfg.get("qk_norm"):
            dqk, _ = O.rmsnorm_bwd(dqk, a["qk_pre"], None, a["rstd_qk"], bf=True)
        d_qkv = np.ascontiguousarray(np.concatenate([dqk.reshape(B * S, -1), d_qkv[:, D + 128 * Hkv:]], 1))
        d_n1, G["l%d.w_qkv" % l], d0 = O.linear_bwd(d_qkv, a["n1"], P["l%d.w_qkv" % l], sx[0:1], sw["l%d.w_qkv" % l], hb)
        d_x1, G["l%d.attn_norm" % l] = O.rmsnorm_bwd(d_n1, a["x"], P["l%d.attn_norm" % l], a["rstd1"], bf=True)
        dx = O.residual_add(d_h, d_x1)
        ds[0], ds[1], ds[2], ds[3] = d0[0], d1[0], d2[0], d3[0]
        G["l%d.s_x" % l] = ds
    if cfg.get("embed_norm"):
        dx, G["embed_norm"] = O.rmsnorm_bwd(dx, sv["x_emb"], P["embed_norm"], sv["rstd_emb"], bf=True)
    G["embed"] = O.embed_bwd(sv["inp"], dx, cfg["vocab"])
    flat = np.concatenate([np.asarray(G[name], np.float32).reshape(-1) for name, _ in _specs(cfg)])
    return flat, float(loss_mean[0])


def run_step(cfg, params, tokens, opt=None, calibrate=True):
    """One optimizer step.  cfg: dict (n_layers, d_model, n_heads, ffn, vocab, seq, micro_batch, mesh=(accum,
    dp_shard, dp_replicate), optional hadamard_block, z_weight, lr, betas, eps, wd, clip, step; the paper's block:
    n_kv_heads, qk_norm, rope_tables=(cos, sin) f32 [seq, 64], embed_norm, window, full_every).
    params: dict name -> numpy (uint16 bf16 bits / float32 steps).  tokens: [n_mb, micro_batch, seq+1]."""
    P = {k: np.array(v, copy=True) for k, v in params.items()}
    specs = _specs(cfg)
    accum, shard, rep = cfg["mesh"]
    assert tokens.shape[0] == accum * shard * rep
    sw = {}
    for l in range(cfg["n_layers"]):
        for w in LINEARS:
            sw["l%d.%s" % (l, w)] = O.lsq_weight_scale(P["l%d.%s" % (l, w)])
    if calibrate:
        forward(cfg, P, sw, tokens[0], calibrate=True)
    n = sum(int(np.prod(s)) for _, s in specs)
    acc = O.Accum(accum, shard, rep, n)
    losses = []
    for mb in range(tokens.shape[0]):
        g, loss = microbatch_grad(cfg, P, sw, tokens[mb])
        acc.push(g)
        losses.append(loss)
    g = acc.result()
    offs = np.cumsum([0] + [int(np.prod(s)) for _, s in specs])
    views = [g[offs[i]:offs[i + 1]] for i in range(len(specs))]
    norm, coef = O.grad_norm(views, cfg.get("clip", 1.0))
    g = O.scale(g, coef)
    if opt is None:
        opt = {"m": np.zeros(n, np.float32), "v": np.zeros(n, np.float32)}
    m, v = opt["m"].copy(), opt["v"].copy()
    lr, (b1, b2), eps, wd, t = cfg.get("lr", 3e-4), cfg.get("betas", (0.9, 0.95)), cfg.get("eps", 1e-8), cfg.get("wd", 0.1), cfg.get("step", 1)
    hashes = {}
    for i, (name, shape) in enumerate(specs):
        sl = slice(offs[i], offs[i + 1])
        decay = wd if (name == "lm_head" or name.split(".")[-1] in LINEARS) else 0.0
        p, m[sl], v[sl] = O.adamw(P[name].reshape(-1), g[sl], m[sl], v[sl], lr, b1, b2, eps, decay, t)
        P[name] = p.reshape(shape)
        hashes[name] = O.tensor_hash(P[name])
    hashes["grad"] = O.tensor_hash(g)
    hashes["adam_m"] = O.tensor_hash(m)
    hashes["adam_v"] = O.tensor_hash(v)
    return {"params": P, "m": m, "v": v, "grad": g, "loss": float(np.mean(losses)), "losses": losses,
            "grad_norm": float(norm), "coef": float(coef), "hashes": hashes}
