"""The replayed step sharded over several GPUs of one NVSwitch domain (Sec. 6: every virtual rank owns the
micro-batches m with m mod R = r; Appendix A: the gradient exchange is pure data movement followed by a sum in a
fixed order, so where a micro-batch was computed cannot change a bit of the result).

Units: the micro-batches of one optimizer step, in mesh order (replica-major, shard-minor, then the accumulation
index).  Rank q of W computes the contiguous block of M/W micro-batches starting at q*M/W.  The flat gradient is cut
into W slices; after each backward pass the slice c of the fresh micro-batch gradient travels to rank c (the
"all-to-all of shard chunks": movement only, no arithmetic), and when all M slices have arrived rank c folds them with
the same push sequence the single-device replay uses (Algorithm 1 inner sums, ascending shard sum, TreeFold across
replicas, reciprocal multiplies).  Every operation of that sequence is element-wise, so folding a slice gives
exactly the bits of the same elements of the single-device fold.  The reduced slices are then gathered on every rank,
and clip, AdamW and the state hash run replicated, which keeps the per-tensor reduction trees of the gradient norm
untouched.

The arithmetic is injected (`fold`), so the exchange and its ordering can be exercised with CPU tensors over the gloo
backend; on GPUs `ShardedReplay` plugs in the library's accumulator.  Only point-to-point send/recv and all_gather are
used, both available in NCCL and gloo.
"""
import torch
import torch.distributed as dist


class ShardPlan:
    """Who computes which micro-batch and who finishes which slice of the flat gradient."""

    def __init__(self, n_microbatches, world, n_grad, align=256):
        if world < 1 or n_microbatches % world:
            raise ValueError("the number of ranks (%d) must divide the micro-batches per step (%d)" % (world, n_microbatches))
        self.M, self.W, self.n = n_microbatches, world, n_grad
        self.per_rank = n_microbatches // world
        # equal slices, a multiple of `align` elements each so that every slice starts 16-byte aligned; the last one
        # is shorter and the gather buffer is padded to W * chunk
        per = (n_grad + world - 1) // world
        self.chunk = (per + align - 1) // align * align

    def owner(self, m):
        return m // self.per_rank

    def local_microbatches(self, rank):
        return range(rank * self.per_rank, (rank + 1) * self.per_rank)

    def bounds(self, c):
        lo = min(c * self.chunk, self.n)
        return lo, min(lo + self.chunk, self.n)

    @property
    def padded(self):
        return self.W * self.chunk


class ShardedReducer:
    """Movement and ordering of the gradient exchange.  `group` None = the default process group."""

    def __init__(self, plan, rank, device, group=None, dtype=torch.float32):
        self.plan, self.rank, self.group = plan, rank, group
        lo, hi = plan.bounds(rank)
        self.len = hi - lo
        # slice `rank` of every micro-batch gradient of the step, in mesh order
        # (rows are a whole chunk apart, so every row starts 16-byte aligned)
        self.recv = torch.empty((plan.M, plan.chunk), dtype=dtype, device=device)
        self.pending = []
        # a process group that cannot move device memory (gloo) gets the slices through host copies
        self.host_stage = torch.device(device).type == "cuda" and dist.is_initialized() and dist.get_backend(group) != "nccl"
        self.landing = []       # (host tensor, device destination) pairs of receives in flight

    def scatter(self, j, grad):
        """Send the slices of the j-th local micro-batch gradient (flat tensor of n elements) to their finishers and post
        the receives for the j-th micro-batch of every other rank.  Returns after posting; `wait` completes them.
        `grad` must stay untouched until then."""
        p = self.plan
        m = self.rank * p.per_rank + j
        lo, hi = p.bounds(self.rank)
        self.recv[m, :hi - lo].copy_(grad[lo:hi])
        ops = []
        for c in range(p.W):
            if c == self.rank:
                continue
            clo, chi = p.bounds(c)
            if chi > clo:
                src = grad[clo:chi].cpu() if self.host_stage else grad[clo:chi]
                ops.append(dist.P2POp(dist.isend, src, c, group=self.group))
            if hi > lo:
                dst = self.recv[c * p.per_rank + j, :hi - lo]
                if self.host_stage:
                    land = torch.empty(hi - lo, dtype=dst.dtype)
                    self.landing.append((land, dst))
                    dst = land
                ops.append(dist.P2POp(dist.irecv, dst, c, group=self.group))
        if ops:
            self.pending += dist.batch_isend_irecv(ops)

    def wait(self):
        for w in self.pending:
            w.wait()
        self.pending = []
        for land, dst in self.landing:
            dst.copy_(land)
        self.landing = []

    def _gather(self, out_padded, mine):
        p = self.plan
        if dist.get_backend(self.group) == "nccl":
            # in place: this rank's slice already sits at its position of the output
            dist.all_gather_into_tensor(out_padded, mine, group=self.group)
        elif out_padded.is_cuda:
            host = [torch.empty(p.chunk, dtype=mine.dtype) for _ in range(p.W)]
            dist.all_gather(host, mine.cpu(), group=self.group)
            for c in range(p.W):
                out_padded[c * p.chunk:(c + 1) * p.chunk].copy_(host[c])
        else:
            views = [out_padded[c * p.chunk:(c + 1) * p.chunk] for c in range(p.W)]
            dist.all_gather(views, mine.clone(), group=self.group)

    def fold_and_gather(self, fold, out_padded):
        """fold(list of M slice tensors in mesh order, out) writes the reduced slice (self.len elements) into out.  The
        reduced slices of all ranks are gathered into out_padded (W * chunk elements; element i of the gradient lands
        at index i)."""
        self.wait()
        p = self.plan
        mine = out_padded[self.rank * p.chunk:(self.rank + 1) * p.chunk]
        if self.len:
            fold([self.recv[m, :self.len] for m in range(p.M)], mine[:self.len])
        if self.len < p.chunk:
            mine[self.len:].zero_()
        if p.W > 1:
            self._gather(out_padded, mine)
        return out_padded[:p.n]


class PeerReducer:
    """The same exchange without staging copies: every rank keeps the gradients of its micro-batches in a buffer that its
    peers can address (symmetric memory over NVLink / NVSwitch), and the fold reads slice `rank` of every micro-batch
    straight out of the owners' buffers, so the accumulate kernel itself moves the data (plain peer loads, no multicast)
    and the arithmetic order is untouched.  Two barriers per step delimit the window in which peers read a buffer.

    `peer_view(owner, j, lo, hi)` returns what `fold` consumes for micro-batch j of rank `owner`, elements [lo, hi):
    a device address on GPUs, a tensor view in the CPU tests.  `barrier()` is a process-group barrier ordered with the
    device work of every rank."""

    def __init__(self, plan, rank, stash, peer_view, barrier, group=None):
        self.plan, self.rank, self.group = plan, rank, group
        self.stash_buf, self.peer_view, self.barrier = stash, peer_view, barrier
        lo, hi = plan.bounds(rank)
        self.len = hi - lo

    def wait(self):
        pass

    def scatter(self, j, grad):
        """Keep the j-th local micro-batch gradient where the peers can read it."""
        self.stash_buf[j].copy_(grad)

    def fold_and_gather(self, fold, out_padded):
        p = self.plan
        lo, hi = p.bounds(self.rank)
        self.barrier()                       # every rank's gradients are complete
        mine = out_padded[self.rank * p.chunk:(self.rank + 1) * p.chunk]
        if self.len:
            fold([self.peer_view(m // p.per_rank, m % p.per_rank, lo, hi) for m in range(p.M)], mine[:self.len])
        if self.len < p.chunk:
            mine[self.len:].zero_()
        self.barrier()                       # nobody reads a peer's buffer past this point
        if p.W > 1:
            if dist.get_backend(self.group) == "nccl":
                dist.all_gather_into_tensor(out_padded, mine, group=self.group)
            else:
                views = [out_padded[c * p.chunk:(c + 1) * p.chunk] for c in range(p.W)]
                dist.all_gather(views, mine.clone(), group=self.group)
        return out_padded[:p.n]


def make_peer_reducer(plan, rank, device, group=None):
    """GPU construction of a PeerReducer on torch's symmetric memory (one allocation of per_rank x n floats per rank)."""
    import torch.distributed._symmetric_memory as symm_mem
    n = plan.n
    flat = symm_mem.empty(plan.per_rank * n, dtype=torch.float32, device=device)
    hdl = symm_mem.rendezvous(flat, group if group is not None else dist.group.WORLD)
    ptrs = [int(x) for x in hdl.buffer_ptrs]
    stash = flat.view(plan.per_rank, n)

    def peer_view(owner, j, lo, hi):
        return ptrs[owner] + 4 * (j * n + lo)

    def barrier():
        # an NCCL collective on the compute stream: it starts on a rank only after that rank's earlier kernels, and
        # completes only when every rank has started it
        dist.barrier(group=group)

    red = PeerReducer(plan, rank, stash, peer_view, barrier, group)
    red._keepalive = (flat, hdl)
    return red


def fold_slices(det, mesh, pool, slices, out):
    """The single-device push sequence (Algorithm 1 + TreeFold) on one slice: `slices` are the M micro-batch slices in
    mesh order, `pool` the accumulation buffers (det_grad_accum_nbufs x len(out) floats), `out` the reduced slice."""
    st = det.det_accum()
    det.det_grad_accum_init(st, mesh[0], mesh[1], mesh[2], out.numel(), pool)
    for s in slices:
        det.det_grad_accum_push(st, s)
    det.det_grad_accum_result(st, out)


class ShardedReplay:
    """One optimizer step of the replay on W GPUs (one process per GPU, NCCL).  Wraps a `Replay` whose accumulation
    pool is sized for this rank's slice only; parameters, moments and the reduced gradient are replicated, so the
    state hashes of all ranks are equal to each other and to those of the single-device replay."""

    def __init__(self, cfg, rank, world, group=None, device="cuda", peer_fold=False):
        """peer_fold: fold straight out of the peers' gradient buffers (symmetric memory, plain peer loads inside the
        accumulate kernel) instead of exchanging slices with point-to-point copies first."""
        import paper_2609_17380_b200 as det
        from .step import Replay, param_specs, _numel
        n_grad = sum(_numel(sh) for _, sh, _ in param_specs(cfg))
        self.det = det
        self.plan = ShardPlan(cfg.n_microbatches, world, n_grad)
        self.rank, self.world, self.group = rank, world, group
        self.r = Replay(cfg, device, accum_len=self.plan.chunk, gout_len=self.plan.padded)
        self.peer_fold = bool(peer_fold) and world > 1
        if self.peer_fold:
            self.red = make_peer_reducer(self.plan, rank, device, group)
            self.stage = None
        else:
            self.red = ShardedReducer(self.plan, rank, device, group)
            # the fresh gradient is copied here so that the next backward pass can overwrite gmb while it travels
            self.stage = torch.empty(n_grad, dtype=torch.float32, device=device)

    def _fold(self, slices, out):
        fold_slices(self.det, self.r.cfg.mesh, self.r.abufs, slices, out)

    def calibrate(self, tokens_mb):
        self.r.calibrate(tokens_mb)

    def step(self, tokens, per_tensor_hashes=True, want_losses=True):
        """tokens: device int32 [n_microbatches, micro_batch, seq+1] in mesh order, the same on every rank."""
        r, p = self.r, self.plan
        with r.span("prepare_weights"):
            r.prepare_weights()
        losses = torch.zeros(p.M, dtype=torch.float32, device=r.dev)
        for j, m in enumerate(p.local_microbatches(self.rank)):
            r.forward(tokens[m])
            losses[m:m + 1].copy_(r.loss_mean)
            r.backward()
            with r.span("grad_exchange"):
                if self.peer_fold:
                    self.red.scatter(j, r.gmb)
                else:
                    self.red.wait()
                    self.stage.copy_(r.gmb)
                    self.red.scatter(j, self.stage)
        with r.span("grad_accum"):
            self.red.fold_and_gather(self._fold, r.gout_padded)
        with r.span("optimizer"):
            r.optimizer()
        with r.span("hash"):
            h = r.hashes(per_tensor_hashes)
        res = {"hashes": h, "status": int(r.status.item())}
        if want_losses:
            if self.world > 1:   # every entry is non-zero on exactly one rank
                if dist.get_backend(self.group) == "nccl":
                    dist.all_reduce(losses, group=self.group)
                else:
                    host = losses.cpu()
                    dist.all_reduce(host, group=self.group)
                    losses = host
            ls = losses.cpu().numpy()
            res.update(losses=[float(x) for x in ls], grad_norm=float(r.norm.item()), coef=float(r.coef.item()))
        return res
