"""Seeded synthetic inputs shared by the oracle-side and CUDA-side tests and by bench.py.

This module holds none of the method's arithmetic: it only draws numbers.  Values come from a
counter-based generator (Philox4x32-10: value = f(seed, tensor id, element index), independent of
how the work is split -- the property Sec. 2.1 "Random number generation" asks of every random
draw), turned into normals by Box-Muller in float64 and rounded to the requested storage type.

bf16 tensors are returned as numpy ``uint16`` bit patterns.
"""
import numpy as np

_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = 0x9E3779B9
_W1 = 0xBB67AE85
_MASK = np.uint64(0xFFFFFFFF)


def philox4x32_10(ctr, key):
    """ctr: uint32 array [..., 4]; key: (k0, k1).  Returns uint32 array [..., 4]."""
    c = [np.asarray(ctr[..., i], np.uint64) for i in range(4)]
    k0, k1 = int(key[0]) & 0xFFFFFFFF, int(key[1]) & 0xFFFFFFFF
    for _ in range(10):
        p0 = _M0 * c[0]
        p1 = _M1 * c[2]
        hi0, lo0 = p0 >> np.uint64(32), p0 & _MASK
        hi1, lo1 = p1 >> np.uint64(32), p1 & _MASK
        c = [hi1 ^ c[1] ^ np.uint64(k0), lo1, hi0 ^ c[3] ^ np.uint64(k1), lo0]
        k0 = (k0 + _W0) & 0xFFFFFFFF
        k1 = (k1 + _W1) & 0xFFFFFFFF
    return np.stack([x.astype(np.uint32) for x in c], axis=-1)


def _raw(n, seed, tid):
    """n uint32 draws for (seed, tensor id); element i comes from counter i // 4, lane i % 4."""
    nblk = (n + 3) // 4
    ctr = np.zeros((nblk, 4), np.uint32)
    idx = np.arange(nblk, dtype=np.uint64)
    ctr[:, 0] = (idx & _MASK).astype(np.uint32)
    ctr[:, 1] = (idx >> np.uint64(32)).astype(np.uint32)
    return philox4x32_10(ctr, (seed, tid)).reshape(-1)[:n]


def uniform01(n, seed, tid):
    """float64 in (0, 1)."""
    return (_raw(n, seed, tid).astype(np.float64) + 0.5) * (1.0 / 4294967296.0)


def normal_f32(shape, std=1.0, mean=0.0, seed=0, tid=0):
    n = int(np.prod(shape))
    h = (n + 1) // 2
    u = uniform01(2 * h, seed, tid)
    r = np.sqrt(-2.0 * np.log(u[:h]))
    z = np.concatenate([r * np.cos(2 * np.pi * u[h:]), r * np.sin(2 * np.pi * u[h:])])[:n]
    return (mean + std * z).astype(np.float32).reshape(shape)


def to_bf16(x):
    """float32 -> bf16 bit patterns (uint16), round-to-nearest-even; storage conversion of inputs only."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32).astype(np.uint64)
    u = u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))
    return (u >> np.uint64(16)).astype(np.uint16).reshape(np.shape(x))


def from_bf16(h):
    return (np.asarray(h, np.uint16).astype(np.uint32) << 16).view(np.float32)


def normal_bf16(shape, std=1.0, mean=0.0, seed=0, tid=0):
    return to_bf16(normal_f32(shape, std, mean, seed, tid))


def randint(shape, high, seed=0, tid=0):
    n = int(np.prod(shape))
    return (_raw(n, seed, tid).astype(np.uint64) % np.uint64(high)).astype(np.int32).reshape(shape)


# ---- model-shaped inputs --------------------------------------------------------------------------------
def model_param_specs(cfg):
    """Canonical parameter order: embedding; per layer attn-norm gain, W_qkv, W_o, ffn-norm gain, W_gate/up,
    W_down, the four activation steps; final-norm gain; LM head.  cfg: dict with n_layers, d_model, ffn, vocab and
    optionally n_kv_heads (grouped queries: W_qkv has (n_heads + 2 n_kv_heads) * 128 rows) and embed_norm (a gain
    after the embedding).  Returns a list of (name, shape, kind), kind in {"embed", "gain", "linear", "step", "head"}."""
    D, Fh, V, L = cfg["d_model"], cfg["ffn"], cfg["vocab"], cfg["n_layers"]
    nq = D + 2 * 128 * (cfg.get("n_kv_heads") or cfg["n_heads"]) if "n_heads" in cfg else 3 * D
    specs = [("embed", (V, D), "embed")]
    if cfg.get("embed_norm"):
        specs += [("embed_norm", (D,), "gain")]
    for l in range(L):
        specs += [("l%d.attn_norm" % l, (D,), "gain"), ("l%d.w_qkv" % l, (nq, D), "linear"),
                  ("l%d.w_o" % l, (D, D), "linear"), ("l%d.ffn_norm" % l, (D,), "gain"),
                  ("l%d.w_gu" % l, (2 * Fh, D), "linear"), ("l%d.w_down" % l, (D, Fh), "linear"),
                  ("l%d.s_x" % l, (4,), "step")]
    specs += [("final_norm", (D,), "gain"), ("lm_head", (V, D), "head")]
    return specs


def model_params(cfg, seed=0):
    """Random-init parameters: weights ~ N(0, 0.02) as bf16 bit patterns, gains = 1 (bf16), activation steps
    filled later by a calibration forward (zeros here, float32)."""
    out = {}
    for tid, (name, shape, kind) in enumerate(model_param_specs(cfg)):
        if kind == "gain":
            out[name] = np.full(shape, 0x3F80, np.uint16)
        elif kind == "step":
            out[name] = np.zeros(shape, np.float32)
        else:
            out[name] = normal_bf16(shape, 0.02, seed=seed, tid=1000 + tid)
    return out


def model_tokens(cfg, n_microbatches, seed=0):
    """Uniform random token ids, [n_microbatches, micro_batch, seq + 1] (inputs and shifted labels)."""
    return randint((n_microbatches, cfg["micro_batch"], cfg["seq"] + 1), cfg["vocab"], seed=seed, tid=777)


def rope_tables(S, base=5.0e5, dim=128):
    """cos/sin tables [S, dim/2] for rotary embeddings: angle = pos * base**(-2i/dim), evaluated in float64 and rounded
    to float32 once; the tables are inputs of the step (both implementations read the same arrays)."""
    i = np.arange(dim // 2, dtype=np.float64)
    inv = base ** (-2.0 * i / dim)
    ang = np.arange(S, dtype=np.float64)[:, None] * inv[None, :]
    return np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)
