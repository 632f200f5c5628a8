"""Replay of one full training step on one B200 through the C-ABI (Sec. 6, Algorithm 1: every virtual rank's
forward/backward in mesh order, gradients folded in the cluster's order, clip, AdamW, state hash).

This module only owns device memory (torch tensors) and the order of the calls; every arithmetic step runs
inside libdet.  It never imports the oracle.
"""
import math
from dataclasses import dataclass, field

import numpy as np
import torch

import paper_2609_17380_b200 as det

LINEARS = ("w_qkv", "w_o", "w_gu", "w_down")
I16, I8, F32, I32 = torch.int16, torch.int8, torch.float32, torch.int32


@dataclass
class ModelConfig:
    n_layers: int = 24
    d_model: int = 2048
    n_heads: int = 16
    ffn: int = 8192
    vocab: int = 50304
    seq: int = 2048
    micro_batch: int = 4
    mesh: tuple = (2, 2, 2)          # (accum, dp_shard, dp_replicate)
    hadamard_block: int = 128
    z_weight: float = 0.0
    lr: float = 3e-4
    betas: tuple = (0.9, 0.95)
    eps: float = 1e-8
    wd: float = 0.1
    clip: float = 1.0
    step: int = 1
    # the paper's block (Sec. 3.1); the defaults are the plain multi-head block of the benchmark configuration
    n_kv_heads: int = 0              # 0 = n_heads (multi-head); 4 with 16 query heads in the paper
    qk_norm: bool = False            # gain-free RMS norm of every query and key head before RoPE
    rope_tables: tuple = None        # (cos, sin) float32 numpy arrays [seq, 64], inputs of the step
    embed_norm: bool = False         # RMSNorm (with gain) on the embedding output
    window: int = 0                  # sliding-window width of the local layers (multiple of 128), 0 = all layers full
    full_every: int = 5              # every full_every-th layer and the last one attend to the whole prefix
    pv_int8: bool = False            # forward P.V of every block of 128 keys on the int8 tensor cores
    dq_fixed: bool = False           # query gradient accumulated over the key blocks in 64-bit fixed point
    arith: int = 1                   # 2: the LM-head contractions in arithmetic version 2 (order-free, int8 tensor cores)

    def as_dict(self):
        return dict(self.__dict__)

    @property
    def tokens_per_microbatch(self):
        return self.micro_batch * self.seq

    @property
    def n_microbatches(self):
        return self.mesh[0] * self.mesh[1] * self.mesh[2]

    @property
    def kv_heads(self):
        return self.n_kv_heads or self.n_heads

    @property
    def qkv_width(self):
        return (self.n_heads + 2 * self.kv_heads) * 128

    def layer_window(self, l):
        if not self.window or l == self.n_layers - 1 or (l + 1) % self.full_every == 0:
            return 0
        return self.window


def param_specs(cfg):
    D, Fh, V, L = cfg.d_model, cfg.ffn, cfg.vocab, cfg.n_layers
    s = [("embed", (V, D), "bf16")]
    if cfg.embed_norm:
        s += [("embed_norm", (D,), "bf16")]
    for l in range(L):
        s += [("l%d.attn_norm" % l, (D,), "bf16"), ("l%d.w_qkv" % l, (cfg.qkv_width, D), "bf16"), ("l%d.w_o" % l, (D, D), "bf16"),
              ("l%d.ffn_norm" % l, (D,), "bf16"), ("l%d.w_gu" % l, (2 * Fh, D), "bf16"), ("l%d.w_down" % l, (D, Fh), "bf16"),
              ("l%d.s_x" % l, (4,), "f32")]
    return s + [("final_norm", (D,), "bf16"), ("lm_head", (V, D), "bf16")]


def _numel(shape):
    n = 1
    for d in shape:
        n *= d
    return n


class Replay:
    """Device state of the replay: parameters, optimizer moments, gradient buffers, saved activations."""

    def __init__(self, cfg, device="cuda", accum_len=None, gout_len=None):
        """accum_len: elements per buffer of the accumulation pool (default: the whole gradient); gout_len: allocated
        length of the reduced-gradient buffer (default: the gradient length).  The sharded replay folds only a slice of
        the gradient on each GPU and gathers the slices into a padded buffer."""
        self.cfg = cfg
        self.dev = device
        self.specs = param_specs(cfg)
        D, Fh, V, L, T = cfg.d_model, cfg.ffn, cfg.vocab, cfg.n_layers, cfg.tokens_per_microbatch
        assert D == cfg.n_heads * 128, "head_dim is 128"
        self.goff, self.poff = {}, {}
        self.shape = dict((n, sh) for n, sh, _ in self.specs)
        g = p = 0
        for name, shape, kind in self.specs:
            self.goff[name] = g
            g += _numel(shape)
            if kind == "bf16":
                self.poff[name] = p
                p += _numel(shape)
        self.n_grad = g
        z = lambda n, dt: torch.zeros(n, dtype=dt, device=device)
        self.pbf = z(p, I16)                       # bf16 parameters (bit patterns), canonical order
        self.sx = z(L * 4, F32)                    # LSQ activation steps, [layer, (qkv, o, gu, down)]
        self.m, self.v = z(g, F32), z(g, F32)      # Adam moments, gradient layout
        self.gmb = z(g, F32)                       # gradient of the current micro-batch
        self.gout_padded = z(max(g, gout_len or 0), F32)
        self.gout = self.gout_padded[:g]           # reduced gradient
        self.nbufs = det.det_grad_accum_nbufs(cfg.mesh[2])
        self.abufs = z(self.nbufs * (accum_len or g), F32)
        self.lin = {}
        for l in range(L):
            for w, (N, K) in zip(LINEARS, ((cfg.qkv_width, D), (D, D), (2 * Fh, D), (D, Fh))):
                self.lin[(l, w)] = dict(N=N, K=K, s_w=z(N, F32), qW=z(N * K, I8), qWt=z(N * K, I8), s_u=z(1, F32))
        e = lambda n, dt: torch.empty(n, dtype=dt, device=device)
        QW, Hkv = cfg.qkv_width, cfg.kv_heads
        self.head_ops = cfg.qk_norm or cfg.rope_tables is not None
        if cfg.rope_tables is not None:
            self.rope_cos = torch.from_numpy(np.ascontiguousarray(cfg.rope_tables[0], dtype=np.float32)).to(device)
            self.rope_sin = torch.from_numpy(np.ascontiguousarray(cfg.rope_tables[1], dtype=np.float32)).to(device)
        self.act = [dict(x=e(T * D, I16), rstd1=e(T, F32), n1=e(T * D, I16), qx_qkv=e(T * D, I8), qkv=e(T * QW, I16),
                         qkr=e(T * QW if self.head_ops else 0, I16),
                         rstd_qk=e(T * (cfg.n_heads + Hkv) if cfg.qk_norm else 0, F32),
                         lse=e(T * cfg.n_heads, F32), att=e(T * D, I16), qx_o=e(T * D, I8), h=e(T * D, I16), rstd2=e(T, F32),
                         n2=e(T * D, I16), qx_gu=e(T * D, I8), gu=e(T * 2 * Fh, I16), a=e(T * Fh, I16),
                         qx_down=e(T * Fh, I8)) for _ in range(L)]
        self.xf, self.rstdf, self.nf = e(T * D, I16), e(T, F32), e(T * D, I16)
        self.x_emb, self.rstd_emb = (e(T * D, I16), e(T, F32)) if cfg.embed_norm else (None, None)
        self.logits = e(T * V, F32)
        self.loss_row, self.lse_x = e(T, F32), e(T, F32)
        self.loss_mean, self.z_mean = e(1, F32), e(1, F32)
        self.tmp = [e(T * max(QW, 2 * Fh), I16) for _ in range(3)]   # gradient scratch activations
        self.tok = e(T, I32)
        self.lab = e(T, I32)
        self.norm, self.coef = e(1, F32), e(1, F32)
        self.status = z(1, I32)
        self.roots = z(32 * 8, torch.uint8)        # hash roots of one step, read back with one copy
        B, H, S = cfg.micro_batch, cfg.n_heads, cfg.seq
        wsb = max(det.det_attn_bwd_fixq_ws_bytes(B, H, S, Hkv) if cfg.dq_fixed else det.det_attn_bwd_ws_bytes(B, H, S, Hkv),
                  det.det_xent_ws_bytes(T, V), det.det_rmsnorm_bwd_ws_bytes(T, D),
                  det.det_lsq_weight_scale_ws_bytes(2 * Fh, D), det.det_lsq_act_scale_init_ws_bytes(T * max(Fh, D)),
                  det.det_tensor_hash_ws_bytes(g * 4), det.det_sum_ws_bytes(g), 1 << 20,
                  (max(det.det_lmhead_fwd_v2_ws_bytes(T, V, D), det.det_lmhead_bwd_v2_ws_bytes(T, V, D)) if cfg.arith == 2 else 0),
                  *[det.det_linear_bwd_ws_bytes(T, N, K) for (N, K) in ((QW, D), (D, D), (2 * Fh, D), (D, Fh))])
        self.ws = e(wsb + 4096, torch.uint8)
        self.losses = []
        self.prof = None
        self.fuse_quant = True       # producers write the linears' int8 inputs (False: separate quantiser pass per linear)

    # ---- optional per-call-site device timing (CUDA events on the launching stream) --------------------
    class _Span:
        def __init__(self, owner, name):
            self.o, self.name = owner, name

        def __enter__(self):
            if self.o.prof is not None:
                self.e0 = torch.cuda.Event(enable_timing=True)
                self.e0.record()

        def __exit__(self, *a):
            if self.o.prof is not None:
                e1 = torch.cuda.Event(enable_timing=True)
                e1.record()
                self.o.prof.setdefault(self.name, []).append((self.e0, e1))

    def span(self, name):
        return Replay._Span(self, name)

    def prof_summary(self):
        """name -> (launch groups, total ms); call after a synchronize."""
        return {k: (len(v), sum(a.elapsed_time(b) for a, b in v)) for k, v in (self.prof or {}).items()}

    # ---- parameter access ------------------------------------------------------------------------------
    def p(self, name):
        shape = self.shape[name]
        if name.endswith("s_x"):
            l = int(name.split(".")[0][1:])
            return self.sx[4 * l:4 * l + 4]
        return self.pbf[self.poff[name]:self.poff[name] + _numel(shape)]

    def g(self, buf, name):
        shape = self.shape[name]
        return buf[self.goff[name]:self.goff[name] + _numel(shape)]

    def load_params(self, params):
        """params: dict name -> numpy (uint16 bf16 bits, float32 steps)."""
        for name, shape, kind in self.specs:
            a = np.ascontiguousarray(params[name]).reshape(-1)
            t = torch.from_numpy(a.view(np.int16) if kind == "bf16" else a)
            self.p(name).copy_(t.to(self.dev))

    def init_params_on_device(self, seed=0):
        """Seeded N(0, 0.02) weights drawn on the device (for shapes too large to draw on the host), gains = 1."""
        gen = torch.Generator(device=self.dev)
        gen.manual_seed(seed)
        for name, shape, kind in self.specs:
            if kind == "f32":
                continue
            dst = self.p(name)
            if name.endswith("norm"):
                dst.fill_(0x3F80)
            else:
                n = dst.numel()
                for o in range(0, n, 1 << 26):
                    c = min(1 << 26, n - o)
                    dst[o:o + c] = (torch.randn(c, generator=gen, device=self.dev) * 0.02).to(torch.bfloat16).view(I16)

    # ---- state dump: everything a later step depends on (Appendix B: replay from a saved state) ------------------
    def save_state(self, path):
        """Parameters (bf16 bits), activation steps, both Adam moments and the step counter, as one .npz file."""
        np.savez(path, pbf=self.pbf.cpu().numpy(), sx=self.sx.cpu().numpy(), m=self.m.cpu().numpy(), v=self.v.cpu().numpy(),
                 step=np.array([self.cfg.step], np.int64))

    def load_state(self, path):
        z = np.load(path)
        for name, dst in (("pbf", self.pbf), ("sx", self.sx), ("m", self.m), ("v", self.v)):
            a = z[name]
            if a.shape != tuple(dst.shape):
                raise ValueError("state file does not match this configuration: %s %s vs %s" % (name, a.shape, tuple(dst.shape)))
            dst.copy_(torch.from_numpy(a).to(self.dev))
        self.cfg.step = int(z["step"][0])

    def params_to_host(self):
        out = {}
        for name, shape, kind in self.specs:
            a = self.p(name).cpu().numpy()
            out[name] = (a.view(np.uint16) if kind == "bf16" else a).reshape(shape)
        return out

    # ---- step pieces --------------------------------------------------------------------------------------
    def prepare_weights(self):
        """Start of an optimizer step: re-pin every weight step from the current weights and quantise."""
        hb = self.cfg.hadamard_block
        for (l, w), d in self.lin.items():
            W = self.p("l%d.%s" % (l, w))
            det.det_lsq_weight_scale(W, d["N"], d["K"], 0, d["s_w"], self.ws)
            det.det_lsq_quantize_weight(W, d["s_w"], d["N"], d["K"], hb, d["qW"], d["qWt"], d["s_u"], self.ws)

    def _linear(self, l, w, idx, X, M, Y, qx, calibrate, prequantised=False):
        """prequantised: the kernel that produced X already wrote its int8 codes into qx."""
        d = self.lin[(l, w)]
        sx = self.sx[4 * l + idx:4 * l + idx + 1]
        if calibrate:
            det.det_lsq_act_scale_init(X, M * d["K"], sx, self.ws)
        with self.span("linear_fwd"):
            if prequantised:
                det.det_linear_fwd_q(qx, d["qW"], sx, d["s_w"], M, d["N"], d["K"], Y, self.status)
            else:
                det.det_linear_fwd(X, d["qW"], sx, d["s_w"], M, d["N"], d["K"], Y, qx, self.status)

    def forward(self, tokens_mb, calibrate=False):
        cfg = self.cfg
        D, Fh, V, L, T = cfg.d_model, cfg.ffn, cfg.vocab, cfg.n_layers, cfg.tokens_per_microbatch
        B, H, S = cfg.micro_batch, cfg.n_heads, cfg.seq
        self.tok.copy_(tokens_mb[:, :-1].reshape(-1))
        self.lab.copy_(tokens_mb[:, 1:].reshape(-1))
        x = self.tmp[0][:T * D]
        Hkv, QW = cfg.kv_heads, cfg.qkv_width
        if cfg.embed_norm:
            det.det_embed_fwd(self.tok, T, self.p("embed"), V, D, self.x_emb)
            det.det_rmsnorm_fwd(det.DET_BF16, self.x_emb, self.p("embed_norm"), T, D, 1e-6, x, self.rstd_emb)
        else:
            det.det_embed_fwd(self.tok, T, self.p("embed"), V, D, x)
        for l in range(L):
            a = self.act[l]
            a["x"].copy_(x)
            # outside the calibration pass every activation step is known before its activation is produced, so the
            # producers write the next linear's int8 input themselves (same bits as the separate quantiser pass)
            fuse = self.fuse_quant and not calibrate and D <= 2048
            sxl = self.sx[4 * l:4 * l + 4]
            if fuse:
                det.det_rmsnorm_fwd_q(a["x"], self.p("l%d.attn_norm" % l), T, D, 1e-6, a["n1"], a["rstd1"], sxl[0:1], a["qx_qkv"])
            else:
                det.det_rmsnorm_fwd(det.DET_BF16, a["x"], self.p("l%d.attn_norm" % l), T, D, 1e-6, a["n1"], a["rstd1"])
            self._linear(l, "w_qkv", 0, a["n1"], T, a["qkv"], a["qx_qkv"], calibrate, fuse)
            qp = vp = a["qkv"].data_ptr()
            if self.head_ops:
                # queries and keys (the first H + Hkv heads of every row) are normalised and rotated into qkr; the
                # values are read from qkv, which has the same row stride
                src = a["qkv"]
                if cfg.qk_norm:
                    det.det_headnorm_fwd(src, QW, T, H + Hkv, 1e-6, a["qkr"], QW, a["rstd_qk"])
                    src = a["qkr"]
                if cfg.rope_tables is not None:
                    det.det_rope(src, QW, T, H + Hkv, S, self.rope_cos, self.rope_sin, 0, a["qkr"], QW)
                qp = a["qkr"].data_ptr()
            with self.span("attn_fwd"):
                if cfg.pv_int8:
                    det.det_attn_fwd_int8pv(qp, qp + 2 * D, vp + 2 * (D + 128 * Hkv), QW, B, H, S, a["att"], D, a["lse"],
                                            self.status, Hkv=Hkv, window=cfg.layer_window(l))
                elif fuse:
                    det.det_attn_fwd_q(qp, qp + 2 * D, vp + 2 * (D + 128 * Hkv), QW, B, H, S, a["att"], D, a["lse"], sxl[1:2],
                                       a["qx_o"], Hkv=Hkv, window=cfg.layer_window(l))
                else:
                    det.det_attn_fwd(qp, qp + 2 * D, vp + 2 * (D + 128 * Hkv), QW, B, H, S, a["att"], D, a["lse"], Hkv=Hkv,
                                     window=cfg.layer_window(l))
            o = self.tmp[1][:T * D]
            self._linear(l, "w_o", 1, a["att"], T, o, a["qx_o"], calibrate, fuse and not cfg.pv_int8)
            det.det_residual_add(a["x"], o, T * D, a["h"])
            if fuse:
                det.det_rmsnorm_fwd_q(a["h"], self.p("l%d.ffn_norm" % l), T, D, 1e-6, a["n2"], a["rstd2"], sxl[2:3], a["qx_gu"])
            else:
                det.det_rmsnorm_fwd(det.DET_BF16, a["h"], self.p("l%d.ffn_norm" % l), T, D, 1e-6, a["n2"], a["rstd2"])
            self._linear(l, "w_gu", 2, a["n2"], T, a["gu"], a["qx_gu"], calibrate, fuse)
            if fuse:
                det.det_swiglu_fwd_q(a["gu"], T, Fh, a["a"], sxl[3:4], a["qx_down"])
            else:
                det.det_swiglu_fwd(a["gu"], T, Fh, a["a"])
            dn = self.tmp[1][:T * D]
            self._linear(l, "w_down", 3, a["a"], T, dn, a["qx_down"], calibrate, fuse)
            det.det_residual_add(a["h"], dn, T * D, x)
        self.xf.copy_(x)
        det.det_rmsnorm_fwd(det.DET_BF16, self.xf, self.p("final_norm"), T, D, 1e-6, self.nf, self.rstdf)
        with self.span("lmhead_fwd"):
            if cfg.arith == 2:
                det.det_lmhead_fwd_v2(self.nf, self.p("lm_head"), T, V, D, self.logits, self.ws, self.status)
            else:
                det.det_lmhead_fwd(self.nf, self.p("lm_head"), T, V, D, self.logits)
        with self.span("xent_fwd"):
            det.det_xent_fwd(self.logits, self.lab, T, V, cfg.z_weight, self.loss_row, self.lse_x, self.loss_mean,
                             self.z_mean, self.ws, self.status)

    def _linear_bwd(self, l, w, idx, dY, X, qx, M, dX):
        d = self.lin[(l, w)]
        name = "l%d.%s" % (l, w)
        sx = self.sx[4 * l + idx:4 * l + idx + 1]
        ds = self.g(self.gmb, "l%d.s_x" % l)[idx:idx + 1]
        with self.span("linear_bwd"):
            det.det_linear_bwd(dY, X, qx, self.p(name), d["qWt"], sx, d["s_w"], d["s_u"], M, d["N"], d["K"],
                               self.cfg.hadamard_block, dX, self.g(self.gmb, name), ds, self.ws, self.status)

    def backward(self):
        cfg = self.cfg
        D, Fh, V, L, T = cfg.d_model, cfg.ffn, cfg.vocab, cfg.n_layers, cfg.tokens_per_microbatch
        B, H, S = cfg.micro_batch, cfg.n_heads, cfg.seq
        with self.span("xent_bwd"):
            det.det_xent_bwd(self.logits, self.lab, self.lse_x, T, V, cfg.z_weight, 1.0 / T)
        t0, t1, t2 = self.tmp
        d_nf = t0[:T * D]
        with self.span("lmhead_bwd"):
            if cfg.arith == 2:
                det.det_lmhead_bwd_v2(self.logits, self.nf, self.p("lm_head"), T, V, D, d_nf, self.g(self.gmb, "lm_head"),
                                      self.ws, self.status)
            else:
                det.det_lmhead_bwd(self.logits, self.nf, self.p("lm_head"), T, V, D, d_nf, self.g(self.gmb, "lm_head"), 1)
        dx = t1[:T * D]
        det.det_rmsnorm_bwd(det.DET_BF16, d_nf, self.xf, self.p("final_norm"), self.rstdf, T, D, dx,
                            self.g(self.gmb, "final_norm"), self.ws)
        for l in reversed(range(L)):
            a = self.act[l]
            d_a = t0[:T * Fh]
            self._linear_bwd(l, "w_down", 3, dx, a["a"], a["qx_down"], T, d_a)
            d_gu = t2[:T * 2 * Fh]
            det.det_swiglu_bwd(d_a, a["gu"], T, Fh, d_gu)
            d_n2 = t0[:T * D]
            self._linear_bwd(l, "w_gu", 2, d_gu, a["n2"], a["qx_gu"], T, d_n2)
            d_h2 = t2[:T * D]
            det.det_rmsnorm_bwd(det.DET_BF16, d_n2, a["h"], self.p("l%d.ffn_norm" % l), a["rstd2"], T, D, d_h2,
                                self.g(self.gmb, "l%d.ffn_norm" % l), self.ws)
            d_h = t1[:T * D]
            det.det_residual_add(dx, d_h2, T * D, d_h)            # in place over dx
            d_att = t0[:T * D]
            self._linear_bwd(l, "w_o", 1, d_h, a["att"], a["qx_o"], T, d_att)
            Hkv, QW = cfg.kv_heads, cfg.qkv_width
            d_qkv = t2[:T * QW]
            vp, dp = a["qkv"].data_ptr(), d_qkv.data_ptr()
            qp = a["qkr"].data_ptr() if self.head_ops else vp
            with self.span("attn_bwd"):
                bwd = det.det_attn_bwd_fixq if cfg.dq_fixed else det.det_attn_bwd
                bwd(d_att, qp, qp + 2 * D, vp + 2 * (D + 128 * Hkv), a["att"], a["lse"], QW, D, B, H, S, dp,
                    dp + 2 * D, dp + 2 * (D + 128 * Hkv), QW, self.ws, Hkv=Hkv, window=cfg.layer_window(l))
            if cfg.rope_tables is not None:
                det.det_rope(d_qkv, QW, T, H + Hkv, S, self.rope_cos, self.rope_sin, 1, d_qkv, QW)
            if cfg.qk_norm:
                det.det_headnorm_bwd(d_qkv, QW, a["qkv"], QW, a["rstd_qk"], T, H + Hkv, d_qkv, QW)
            d_n1 = t0[:T * D]
            self._linear_bwd(l, "w_qkv", 0, d_qkv, a["n1"], a["qx_qkv"], T, d_n1)
            d_x1 = t2[:T * D]
            det.det_rmsnorm_bwd(det.DET_BF16, d_n1, a["x"], self.p("l%d.attn_norm" % l), a["rstd1"], T, D, d_x1,
                                self.g(self.gmb, "l%d.attn_norm" % l), self.ws)
            det.det_residual_add(d_h, d_x1, T * D, dx)            # dx aliases d_h: in place
        if cfg.embed_norm:
            d_emb = t0[:T * D]
            det.det_rmsnorm_bwd(det.DET_BF16, dx, self.x_emb, self.p("embed_norm"), self.rstd_emb, T, D, d_emb,
                                self.g(self.gmb, "embed_norm"), self.ws)
            dx = d_emb
        det.det_embed_bwd(self.tok, T, dx, V, D, self.g(self.gmb, "embed"))

    def optimizer(self):
        cfg = self.cfg
        views = [self.g(self.gout, name) for name, _, _ in self.specs]
        det.det_grad_norm(views, cfg.clip, self.norm, self.coef, self.ws, self.status)
        det.det_scale_inplace(self.gout, self.n_grad, self.coef)
        for name, shape, kind in self.specs:
            decay = cfg.wd if (name == "lm_head" or name.split(".")[-1] in LINEARS) else 0.0
            desc = det.det_adamw_desc(cfg.lr, cfg.betas[0], cfg.betas[1], cfg.eps, decay, cfg.step)
            det.det_adamw_step(desc, det.DET_BF16 if kind == "bf16" else det.DET_F32, self.p(name), self.g(self.gout, name),
                               self.g(self.m, name), self.g(self.v, name), _numel(shape))

    def hashes(self, per_tensor=True):
        """State hashes of the step (Appendix B).  Every hash is queued on the stream with its root finished on the
        device; the roots come back in ONE copy, so the whole set costs one synchronisation."""
        jobs = []
        if per_tensor:
            for name, shape, kind in self.specs:
                t = self.p(name)
                jobs.append((name, t, t.numel() * t.element_size()))
        else:
            jobs.append(("params_bf16", self.pbf, self.pbf.numel() * 2))
            jobs.append(("steps_f32", self.sx, self.sx.numel() * 4))
        jobs += [("grad", self.gout, self.n_grad * 4), ("adam_m", self.m, self.n_grad * 4), ("adam_v", self.v, self.n_grad * 4)]
        if self.roots.numel() < 32 * len(jobs):
            self.roots = torch.empty(32 * len(jobs), dtype=torch.uint8, device=self.dev)
        for i, (_, t, nbytes) in enumerate(jobs):
            det.det_tensor_hash_async(t, nbytes, self.roots[32 * i:32 * i + 32], self.ws)
        raw = self.roots[:32 * len(jobs)].cpu().numpy().tobytes()
        return {name: raw[32 * i:32 * i + 32].hex() for i, (name, _, _) in enumerate(jobs)}

    def calibrate(self, tokens_mb):
        """Untimed: set every activation step from the first micro-batch (LSQ initialisation rule)."""
        self.prepare_weights()
        self.forward(tokens_mb, calibrate=True)

    def step(self, tokens, per_tensor_hashes=True, want_losses=True):
        """tokens: device int32 [n_microbatches, micro_batch, seq+1] in mesh order.  One optimizer step."""
        cfg = self.cfg
        with self.span("prepare_weights"):
            self.prepare_weights()
        st = det.det_accum()
        det.det_grad_accum_init(st, cfg.mesh[0], cfg.mesh[1], cfg.mesh[2], self.n_grad, self.abufs)
        losses = torch.empty(tokens.shape[0], dtype=F32, device=self.dev)
        for mb in range(tokens.shape[0]):
            torch.cuda.nvtx.range_push("microbatch%d" % mb)      # lets a profiler select one micro-batch
            self.forward(tokens[mb])
            losses[mb:mb + 1].copy_(self.loss_mean)
            self.backward()
            with self.span("grad_accum"):
                det.det_grad_accum_push(st, self.gmb)
            torch.cuda.nvtx.range_pop()
        det.det_grad_accum_result(st, self.gout)
        with self.span("optimizer"):
            self.optimizer()
        with self.span("hash"):
            h = self.hashes(per_tensor_hashes)
        res = {"hashes": h, "status": int(self.status.item())}
        if want_losses:
            ls = losses.cpu().numpy()
            res.update(losses=[float(x) for x in ls], loss=float(np.mean(ls.astype(np.float64))),
                       grad_norm=float(self.norm.item()), coef=float(self.coef.item()))
        return res


def run_step(cfg, params, tokens, calibrate=True):
    """Convenience for tests: numpy params/tokens in, one replayed step, results and hashes out."""
    r = Replay(cfg)
    r.load_params(params)
    tok = torch.from_numpy(np.ascontiguousarray(tokens, dtype=np.int32)).cuda()
    if calibrate:
        r.calibrate(tok[0])
    out = r.step(tok)
    out["replay"] = r
    return out
