"""Expert-parallel MoE layer forward (Sections 2.1, 3.1-3.3 of the paper) on top of the C-ABI entry points.

Rank c holds experts [c*L, (c+1)*L) and its own T_local tokens.  Per layer and rank: route the local tokens, all-gather
the top-k expert ids, build the dispatch schedule for the local experts (Algorithm 1 with R source ranks), run the
expert FFNs with the rows pulled from the source ranks' token buffers, wait for all ranks, and combine the k expert
rows of every local token from the serving ranks' output buffers in a fixed order.

Two drivers over the same library calls:
  * `forward_emulated`  -- every rank lives on ONE GPU in ONE process, phase by phase.  A local pointer is a valid peer
    pointer, so this exercises exactly the kernels and schedules of the multi-GPU path; it is what the GPU tests run.
  * `forward_distributed` -- one process per GPU under torch.distributed: buffers other ranks must read (x, y, pos) live
    in symmetric memory, the route all-gather and the barrier before the combine are torch.distributed collectives.
    It needs at least two GPUs connected by NVLink.
Argument marshalling and collective plumbing only; every step of the layer runs in the library's kernels.
"""
import torch

from . import mok


class RankState:
    """Buffers of one rank for fixed sizes: workspace, y / pos / y_shared, and (local) routing results."""

    def __init__(self, n_ranks, T_local, H, I, I_shared, E, k, device, alloc=None, mx=False):
        alloc = alloc or (lambda shape, dtype: torch.empty(shape, dtype=dtype, device=device))
        self.n_ranks, self.T_local, self.H, self.I, self.I_shared, self.E, self.k = n_ranks, T_local, H, I, I_shared, E, k
        n = (mok.mok_ep_mx_workspace_bytes if mx else mok.mok_ep_workspace_bytes)(n_ranks, T_local, H, I, I_shared, E, k)
        if n == 0:
            raise mok.MokError(mok.MOK_ERR_SHAPE)
        self.ws = torch.empty(n + 256, dtype=torch.uint8, device=device)
        self.route_ws = mok.alloc_workspace(T_local, H, max(I, 8), 0, E, k, device=device)
        self.y = alloc((mok.mok_ep_y_rows(n_ranks, T_local, E, k), H), torch.bfloat16)
        self.pos = alloc((n_ranks * T_local * k,), torch.int32)
        tpad = (T_local + 255) // 256 * 256
        self.y_shared = torch.empty((max(tpad, 256), H), dtype=torch.bfloat16, device=device) if I_shared else None
        # MXFP8 mode: this rank's quantised token rows and their scales, read by the peers' gather warps
        self.x_codes = alloc((T_local, H), torch.uint8) if mx else None
        self.x_scales = alloc((T_local, (H + 127) // 128 * 4), torch.uint8) if mx else None
        self.idx = self.w = None


def forward_emulated(xs, W_router, router_bias, W_gate_up, W_down, W_shared_gate_up, W_shared_down, k, config=None,
                     return_tables=False, mx=False):
    """All ranks on the current GPU.  xs: list of bf16 [T_local, H] (one per rank); W_gate_up [E, 2I, H] and
    W_down [E, H, I] hold ALL experts and are cut into per-rank shards here.  Returns the list of per-rank outputs
    (and, with return_tables, each rank's Algorithm 1 tables)."""
    R = len(xs)
    T_local, H = xs[0].shape
    E = W_router.shape[0]
    L = E // R
    I = W_gate_up.shape[1] // 2
    I_s = 0 if W_shared_gate_up is None else W_shared_gate_up.shape[0] // 2
    dev = xs[0].device
    st = [RankState(R, T_local, H, I, I_s, E, k, dev, mx=mx) for _ in range(R)]
    if mx:
        config = config or mok._config()
        config.precision = mok.MOK_PRECISION_MXFP8
    mxw = [None] * R
    for r in range(R):                                                  # 1. local routing (+ quantised rows for the peers)
        st[r].idx, st[r].w = mok.mok_route(xs[r], W_router, router_bias, k, st[r].route_ws)
        if mx:
            codes, scales = mok.mok_mx_quantize_rows(xs[r])
            st[r].x_codes.copy_(codes)
            st[r].x_scales.copy_(scales)
            mxw[r] = mok.MxWeights(W_gate_up[r * L:(r + 1) * L].contiguous(), W_down[r * L:(r + 1) * L].contiguous())
    idx_all = torch.stack([s.idx.reshape(-1) for s in st]).contiguous()  # 2. the all-gather of the routes
    x_ptrs = [x.data_ptr() for x in xs]
    xc_ptrs = [s.x_codes.data_ptr() for s in st] if mx else None
    xs_ptrs = [s.x_scales.data_ptr() for s in st] if mx else None
    tables = []
    for c in range(R):                                                  # 3. schedule + expert FFNs of rank c
        tables.append(mok.mok_ep_expert_ffn(c, x_ptrs, idx_all, W_gate_up[c * L:(c + 1) * L], W_down[c * L:(c + 1) * L],
                                            W_shared_gate_up, W_shared_down, E, k, st[c].y, st[c].pos, st[c].y_shared,
                                            st[c].ws, H, outputs=return_tables, config=config, mx_weights=mxw[c],
                                            x_codes_ptrs=xc_ptrs, x_scales_ptrs=xs_ptrs))
    # 4. the barrier: one stream, so every rank's y and pos are complete before the combines below start
    outs = []
    y_ptrs = [s.y.data_ptr() for s in st]
    pos_ptrs = [s.pos.data_ptr() for s in st]
    for r in range(R):                                                  # 5. owner-side combine
        out = torch.empty_like(xs[r])
        mok.mok_ep_combine(r, R, st[r].idx, st[r].w, y_ptrs, pos_ptrs, st[r].y_shared, E, out)
        outs.append(out)
    for s in st:
        status = mok.mok_read_status(s.ws)
        if status != 0:
            raise mok.MokError(status)
    return (outs, tables, idx_all) if return_tables else outs


def backward_emulated(xs, douts, idxs, ws_, W_gate_up, W_down, W_shared_gate_up, W_shared_down, config=None,
                      weight_grads=True):
    """The expert-parallel backward pass with all ranks on the current GPU, phase by phase (as forward_emulated).
    xs, douts: per-rank bf16 [T_local, H]; idxs, ws_: per-rank routing of the forward pass (int32 / fp32 [T_local, k]).
    Returns per rank {dx, dw, dW_gate_up (this rank's experts), dW_down, (dW_shared_gate_up, dW_shared_down: this rank's
    tokens' share of the shared expert's gradient)}."""
    R = len(xs)
    T_local, H = xs[0].shape
    k = idxs[0].shape[1]
    E = W_gate_up.shape[0]
    L = E // R
    I = W_gate_up.shape[1] // 2
    I_s = 0 if W_shared_gate_up is None else W_shared_gate_up.shape[0] // 2
    dev = xs[0].device
    idx_all = torch.stack([i.reshape(-1) for i in idxs]).contiguous()          # the "all-gather" of routes and weights
    w_all = torch.stack([w.reshape(-1) for w in ws_]).contiguous()
    rows = mok.mok_ep_y_rows(R, T_local, E, k)
    tpad = max((T_local + 255) // 256 * 256, 256)
    nbytes = mok.mok_ep_bwd_workspace_bytes(R, T_local, H, I, I_s, E, k)
    if nbytes == 0:
        raise mok.MokError(mok.MOK_ERR_SHAPE)
    st = []
    for r in range(R):
        st.append({"ws": torch.empty(nbytes + 256, dtype=torch.uint8, device=dev),
                   "dxg": torch.empty((rows, H), dtype=torch.bfloat16, device=dev),
                   "pos": torch.empty((R * T_local * k,), dtype=torch.int32, device=dev),
                   "dw_routes": torch.zeros((R * T_local * k,), dtype=torch.float32, device=dev),
                   "dx_shared": torch.empty((tpad, H), dtype=torch.bfloat16, device=dev) if I_s else None})
    x_ptrs = [int(x.data_ptr()) for x in xs]
    d_ptrs = [int(d.data_ptr()) for d in douts]
    out = []
    for r in range(R):                                                          # serving side, every rank
        g = mok.mok_ep_expert_bwd(r, x_ptrs, d_ptrs, idx_all, w_all, W_gate_up[r * L:(r + 1) * L].contiguous(),
                                  W_down[r * L:(r + 1) * L].contiguous(), W_shared_gate_up, W_shared_down, E, k, H,
                                  st[r]["dxg"], st[r]["pos"], st[r]["dw_routes"], st[r]["dx_shared"], st[r]["ws"],
                                  weight_grads=weight_grads, config=config)
        status = mok.mok_read_status(st[r]["ws"])
        if status != 0:
            raise mok.MokError(status)
        out.append(g)
    torch.cuda.synchronize()                                                    # the barrier over the ranks
    dxg_ptrs = [int(s_["dxg"].data_ptr()) for s_ in st]
    pos_ptrs = [int(s_["pos"].data_ptr()) for s_ in st]
    dw_ptrs = [int(s_["dw_routes"].data_ptr()) for s_ in st]
    for r in range(R):                                                          # owner side
        dx = torch.empty_like(xs[r])
        dw = torch.empty((T_local, k), dtype=torch.float32, device=dev)
        mok.mok_ep_bwd_combine(r, R, idxs[r], dxg_ptrs, pos_ptrs, dw_ptrs, st[r]["dx_shared"], E, dx, dw)
        out[r]["dx"], out[r]["dw"] = dx, dw
    torch.cuda.synchronize()
    return out


class DistributedLayer:
    """One process per rank under torch.distributed.  Buffers that peers read (x, y, pos) are allocated once and
    exchanged once; `forward` then makes no allocation a peer depends on.

    exchange = None: the buffers live in symmetric memory and the peers' addresses come from its rendezvous (one
    process per GPU, NCCL for the route all-gather and the barriers).
    exchange = callable(name, tensor) -> list of one tensor per rank (this rank's own included) that map the peers'
    buffers into this process, e.g. CUDA IPC handles passed through torch.multiprocessing queues.  The collectives
    then go through whatever backend the group has; with a CPU backend (gloo) the routes are staged through the host
    and every barrier synchronises the device first.  That form also runs with several processes on ONE GPU, since no
    kernel ever waits for another rank's kernel."""

    def __init__(self, T_local, H, I, I_shared, E, k, device, group=None, exchange=None, mx=False):
        import torch.distributed as dist
        self.dist = dist
        self.group = group or dist.group.WORLD
        self.R, self.rank = dist.get_world_size(self.group), dist.get_rank(self.group)
        self.E, self.k, self.H, self.mx = E, k, H, mx
        self.host_collectives = dist.get_backend(self.group) != "nccl"
        self._keep = []
        if exchange is None:
            import torch.distributed._symmetric_memory as symm

            def alloc(shape, dtype):
                return symm.empty(shape, dtype=dtype, device=device)

            def peers_of(name, t):
                h = symm.rendezvous(t, self.group)
                self._keep.append(h)
                return [int(p) for p in h.buffer_ptrs]
        else:
            def alloc(shape, dtype):
                return torch.empty(shape, dtype=dtype, device=device)

            def peers_of(name, t):
                peers = exchange(name, t)
                assert len(peers) == self.R
                self._keep.append(peers)                    # the mappings must outlive every kernel that reads them
                return [int(q.data_ptr()) for q in peers]
        self._alloc, self._peers_of, self.device = alloc, peers_of, device
        self.T_local, self.I, self.I_shared = T_local, I, I_shared
        self._bwd = None
        self.st = RankState(self.R, T_local, H, I, I_shared, E, k, device, alloc=alloc, mx=mx)
        self.x = alloc((T_local, H), torch.bfloat16)
        self.y_ptrs = peers_of("y", self.st.y)
        self.pos_ptrs = peers_of("pos", self.st.pos)
        self.x_ptrs = peers_of("x", self.x)
        self.xc_ptrs = peers_of("x_codes", self.st.x_codes) if mx else None
        self.xs_ptrs = peers_of("x_scales", self.st.x_scales) if mx else None
        self.idx_all = torch.empty((self.R, T_local * k), dtype=torch.int32, device=device)

    def _barrier(self):
        if self.host_collectives:
            torch.cuda.synchronize()
        self.dist.barrier(group=self.group)

    def _gather_routes(self, idx, dst=None):
        """All-gather of a per-route tensor (the top-k ids; in the backward pass also the router weights)."""
        dst = self.idx_all if dst is None else dst
        if not self.host_collectives:
            self.dist.all_gather_into_tensor(dst, idx.reshape(-1), group=self.group)
            return
        mine = idx.reshape(-1).cpu()                          # synchronises this rank's stream: its x is final too
        parts = [torch.empty_like(mine) for _ in range(self.R)]
        self.dist.all_gather(parts, mine, group=self.group)
        dst.copy_(torch.stack(parts))

    def forward(self, x_local, W_router, router_bias, W_gate_up_local, W_down_local, W_shared_gate_up, W_shared_down,
                out=None, config=None, mx_weights=None, timeline=None):
        """x_local: this rank's tokens, bf16 [T_local, H], on the device or in pinned host memory (it is copied into
        the peer-visible buffer either way).  mx_weights: this rank's experts pre-quantised (mok.MxWeights) when the
        layer was built with mx=True.  timeline: a list that receives (phase name, CUDA event recorded after it)."""
        st = self.st

        def mark(name):
            if timeline is not None:
                ev = torch.cuda.Event(enable_timing=True)
                ev.record()
                timeline.append((name, ev))

        mark("start")
        self._barrier()                         # peers have finished reading the previous layer's x / y / pos
        self.x.copy_(x_local, non_blocking=True)
        mark("stage_x")
        if self.mx:                             # this rank's token rows as the peers' gather warps will pull them
            codes, scales = mok.mok_mx_quantize_rows(self.x)
            st.x_codes.copy_(codes)
            st.x_scales.copy_(scales)
            config = config or mok._config()
            config.precision = mok.MOK_PRECISION_MXFP8
        st.idx, st.w = mok.mok_route(self.x, W_router, router_bias, self.k, st.route_ws)
        # the all-gather of the routes also orders every rank's x before any rank's pulls
        mark("route")
        self._gather_routes(st.idx)
        mark("gather_routes")
        mok.mok_ep_expert_ffn(self.rank, self.x_ptrs, self.idx_all, W_gate_up_local, W_down_local, W_shared_gate_up,
                              W_shared_down, self.E, self.k, st.y, st.pos, st.y_shared, st.ws, self.H, config=config,
                              mx_weights=mx_weights, x_codes_ptrs=self.xc_ptrs, x_scales_ptrs=self.xs_ptrs)
        mark("expert_ffn")
        self._barrier()                         # every rank's y and pos are complete
        mark("barrier")
        if out is None:
            out = torch.empty_like(self.x)
        mok.mok_ep_combine(self.rank, self.R, st.idx, st.w, self.y_ptrs, self.pos_ptrs, st.y_shared, self.E, out)
        mark("combine")
        return out

    def _init_backward(self):
        """Buffers of the backward pass, allocated and exchanged once (a collective: every rank calls it together)."""
        n = self.T_local * self.k
        nbytes = mok.mok_ep_bwd_workspace_bytes(self.R, self.T_local, self.H, self.I, self.I_shared, self.E, self.k)
        if nbytes == 0:
            raise mok.MokError(mok.MOK_ERR_SHAPE)
        b = {"ws": torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device),
             "dout": self._alloc((self.T_local, self.H), torch.bfloat16),
             "dxg": self._alloc(tuple(self.st.y.shape), torch.bfloat16),
             "dw_routes": self._alloc((self.R * n,), torch.float32),
             "w_all": torch.empty((self.R, n), dtype=torch.float32, device=self.device),
             "dx_shared": None if self.st.y_shared is None else torch.empty_like(self.st.y_shared)}
        b["dout_ptrs"] = self._peers_of("dout", b["dout"])
        b["dxg_ptrs"] = self._peers_of("dxg", b["dxg"])
        b["dw_ptrs"] = self._peers_of("dw_routes", b["dw_routes"])
        self._bwd = b

    def backward(self, dout_local, W_gate_up_local, W_down_local, W_shared_gate_up, W_shared_down, weight_grads=True,
                 config=None):
        """The backward pass of the last forward call (its tokens are still in the peer-visible buffer, its routing in
        this object).  dout_local: bf16 [T_local, H].  Returns {dx, dw, and with weight_grads the gradients of this
        rank's experts and its tokens' share of the shared expert's}."""
        if self.mx:
            raise mok.MokError(mok.MOK_ERR_UNSUPPORTED)
        if self._bwd is None:
            self._init_backward()
        st, b = self.st, self._bwd
        self._barrier()                         # peers have finished reading the previous call's buffers
        b["dout"].copy_(dout_local, non_blocking=True)
        # the all-gather of the router weights also orders every rank's dout before any rank's pulls
        self._gather_routes(st.w, b["w_all"])
        res = mok.mok_ep_expert_bwd(self.rank, self.x_ptrs, b["dout_ptrs"], self.idx_all, b["w_all"], W_gate_up_local,
                                    W_down_local, W_shared_gate_up, W_shared_down, self.E, self.k, self.H, b["dxg"], st.pos,
                                    b["dw_routes"], b["dx_shared"], b["ws"], weight_grads=weight_grads, config=config)
        self._barrier()                         # every rank's dxg, pos and dw_routes are complete
        res["dx"] = torch.empty((self.T_local, self.H), dtype=torch.bfloat16, device=self.device)
        res["dw"] = torch.empty((self.T_local, self.k), dtype=torch.float32, device=self.device)
        mok.mok_ep_bwd_combine(self.rank, self.R, st.idx, b["dxg_ptrs"], self.pos_ptrs, b["dw_ptrs"], b["dx_shared"],
                               self.E, res["dx"], res["dw"])
        return res

    def status(self):
        status = mok.mok_read_status(self.st.ws)
        if status == 0 and self._bwd is not None:
            status = mok.mok_read_status(self._bwd["ws"])
        return status


def forward_distributed(x_local, W_router, router_bias, W_gate_up_local, W_down_local, W_shared_gate_up, W_shared_down,
                        E, k, group=None, config=None):
    """One call of a DistributedLayer built for these sizes.  x_local bf16 [T_local, H]; W_gate_up_local [L, 2I, H] and
    W_down_local [L, H, I] are this rank's experts."""
    T_local, H = x_local.shape
    I = W_gate_up_local.shape[1] // 2
    I_s = 0 if W_shared_gate_up is None else W_shared_gate_up.shape[0] // 2
    layer = DistributedLayer(T_local, H, I, I_s, E, k, x_local.device, group)
    out = layer.forward(x_local, W_router, router_bias, W_gate_up_local, W_down_local, W_shared_gate_up, W_shared_down,
                        config=config)
    layer._barrier()                            # nobody frees y while a peer still reads it
    status = layer.status()
    if status != 0:
        raise mok.MokError(status)
    return out


def _ipc_rank(rank, world, queues, config_name, port, results, mx=False, tokens=0, config_kw=None):
    """One rank of the several-processes-on-one-GPU self-check: gloo collectives, peer buffers through CUDA IPC.
    tokens: total tokens over the ranks (0 = the workload's); config_kw: knobs of the expert-parallel calls."""
    import os
    import torch.distributed as dist
    from . import inputs
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = inputs.CONFIGS[config_name]
    if tokens:
        cfg = cfg.with_tokens(tokens)
    T_local, L = cfg.T // world, cfg.E // world
    conf = mok._config(**config_kw) if config_kw else None

    def exchange(name, t):
        # every rank puts its tensor on every other rank's queue (torch.multiprocessing ships a CUDA IPC handle) and
        # takes world - 1 tensors off its own; tags keep the three rounds apart
        for r in range(world):
            if r != rank:
                queues[r].put((name, rank, t))
        got = {rank: t}
        while len(got) < world:
            tag, src, peer = queues[rank].get()
            assert tag == name, (tag, name)
            got[src] = peer
        dist.barrier()
        return [got[r] for r in range(world)]

    d = inputs.make_inputs(cfg)
    g = {k: (None if d[k] is None else mok.to_device_bf16(d[k], dev)) for k in ("x", "W_gate_up", "W_down", "W_sgu", "W_sd")}
    W_r = torch.from_numpy(d["W_r"]).to(dev)
    bias = None if d["bias"] is None else torch.from_numpy(d["bias"]).to(dev)
    x_local = g["x"][rank * T_local:(rank + 1) * T_local].contiguous()
    layer = DistributedLayer(T_local, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k, dev, exchange=exchange, mx=mx)
    Wgu, Wd = g["W_gate_up"][rank * L:(rank + 1) * L].contiguous(), g["W_down"][rank * L:(rank + 1) * L].contiguous()
    mxw = mok.MxWeights(Wgu, Wd) if mx else None
    out = None
    for _ in range(2):                                         # twice: buffers are reused across layers
        out = layer.forward(x_local, W_r, bias, Wgu, Wd, g["W_sgu"], g["W_sd"], mx_weights=mxw, config=conf)
    layer._barrier()
    ws = mok.alloc_workspace(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k, device=dev, mx=mx)
    one = mok.mok_moe_forward_ex(g["x"], W_r, bias, g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], cfg.k, ws,
                                 config=mok._config(precision=int(mx)),
                                 mx_weights=mok.MxWeights(g["W_gate_up"], g["W_down"]) if mx else None)
    same = torch.equal(out.view(torch.int16), one[rank * T_local:(rank + 1) * T_local].view(torch.int16))
    if not mx:
        # the backward pass of that layer, twice on the same buffers: dx and dw against the one-rank backward pass
        gen = torch.Generator(device="cpu").manual_seed(7)
        dout = torch.randn((cfg.T, cfg.H), generator=gen).to(torch.bfloat16).to(dev)
        sl = slice(rank * T_local, (rank + 1) * T_local)
        for _ in range(2):
            res = layer.backward(dout[sl].contiguous(), Wgu, Wd, g["W_sgu"], g["W_sd"])
        layer._barrier()
        _, st1 = mok.mok_moe_forward_ex(g["x"], W_r, bias, g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], cfg.k, ws,
                                        stages=True)
        ref = mok.mok_moe_backward(g["x"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], st1["topk_idx"],
                                   st1["topk_w"], dout, weight_grads=False)
        same = same and torch.equal(res["dx"].view(torch.int16), ref["dx"][sl].view(torch.int16))
        same = same and torch.equal(res["dw"].view(torch.int32), ref["dw"][sl].view(torch.int32))
        same = same and bool(torch.isfinite(res["dW_gate_up"].float()).all())
    results.put((rank, bool(same) and layer.status() == 0))
    layer._barrier()                                           # peers may still read this rank's buffers until here
    dist.destroy_process_group()


def check_processes_on_one_gpu(world=2, config_name="tiny", port=29561, mx=False, tokens=0, config_kw=None):
    """Runs `world` ranks as separate processes on GPU 0 (each maps the others' x / y / pos through CUDA IPC) and
    returns True if every rank's output (and, in bf16 mode, its dx and dw of the backward pass) equals its slice of the
    one-rank layer's bit for bit."""
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    queues = [ctx.Queue() for _ in range(world)]
    results = ctx.Queue()
    procs = [ctx.Process(target=_ipc_rank, args=(r, world, queues, config_name, port, results, mx, tokens, config_kw))
             for r in range(world)]
    for p in procs:
        p.start()
    ok = []
    try:
        for _ in range(world):
            ok.append(results.get(timeout=240)[1])
    finally:
        for p in procs:
            p.join(timeout=60)
            if p.is_alive():
                p.kill()
    return len(ok) == world and all(ok) and all(p.exitcode == 0 for p in procs)


def main():
    """Self-check and timing of the distributed driver: `python -m paper_2609_36070_b200.ep [--config NAME]`, alone
    (a world of one rank) or under torch.distributed.run with one process per GPU.  Every rank builds the same seeded
    workload, keeps its slice of the tokens and its shard of the experts, runs the expert-parallel layer and compares
    its slice of the output bit for bit with the one-rank layer run on the whole batch on its own GPU.  Rank 0 prints
    one JSON line."""
    import argparse
    import json
    import os
    import torch.distributed as dist
    from . import inputs
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="tiny")
    ap.add_argument("--tokens", type=int, default=0, help="total tokens over all ranks (0 = the config's T)")
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    args = ap.parse_args()
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29541")
    os.environ.setdefault("TORCH_SYMM_MEM_DISABLE_MULTICAST", "1")   # plain peer pointers only
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    cfg = inputs.CONFIGS[args.config]
    if args.tokens:
        cfg = cfg.with_tokens(args.tokens)
    assert cfg.T % world == 0 and cfg.E % world == 0, "tokens and experts must divide over the ranks"
    T_local, L = cfg.T // world, cfg.E // world
    d = inputs.make_inputs(cfg)
    g = {k: (None if d[k] is None else mok.to_device_bf16(d[k], dev)) for k in ("x", "W_gate_up", "W_down", "W_sgu", "W_sd")}
    W_r = torch.from_numpy(d["W_r"]).to(dev)
    bias = None if d["bias"] is None else torch.from_numpy(d["bias"]).to(dev)
    x_local = g["x"][rank * T_local:(rank + 1) * T_local].contiguous()
    Wgu, Wd = g["W_gate_up"][rank * L:(rank + 1) * L].contiguous(), g["W_down"][rank * L:(rank + 1) * L].contiguous()
    layer = DistributedLayer(T_local, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k, dev)
    out = torch.empty_like(x_local)

    def step():
        layer.forward(x_local, W_r, bias, Wgu, Wd, g["W_sgu"], g["W_sd"], out=out)

    for _ in range(max(args.warmup, 1)):
        step()
    dist.barrier()
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    dist.barrier()
    torch.cuda.synchronize()
    ms = torch.tensor([ev0.elapsed_time(ev1) / max(args.steps, 1)], device=dev)
    dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    ws = mok.alloc_workspace(cfg.T, cfg.H, cfg.I, cfg.I_s, cfg.E, cfg.k, device=dev)
    one = mok.mok_moe_forward_ex(g["x"], W_r, bias, g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], cfg.k, ws)
    same = torch.equal(out.view(torch.int16), one[rank * T_local:(rank + 1) * T_local].view(torch.int16))
    # the backward pass of the same layer against the one-rank backward pass (dx, dw bit for bit)
    gen = torch.Generator(device="cpu").manual_seed(7)
    dout = torch.randn((cfg.T, cfg.H), generator=gen).to(torch.bfloat16).to(dev)
    sl = slice(rank * T_local, (rank + 1) * T_local)
    step()
    res = layer.backward(dout[sl].contiguous(), Wgu, Wd, g["W_sgu"], g["W_sd"], weight_grads=False)
    _, st1 = mok.mok_moe_forward_ex(g["x"], W_r, bias, g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], cfg.k, ws,
                                    stages=True)
    ref = mok.mok_moe_backward(g["x"], g["W_gate_up"], g["W_down"], g["W_sgu"], g["W_sd"], st1["topk_idx"], st1["topk_w"],
                               dout, weight_grads=False)
    same_bwd = (torch.equal(res["dx"].view(torch.int16), ref["dx"][sl].view(torch.int16)) and
                torch.equal(res["dw"].view(torch.int32), ref["dw"][sl].view(torch.int32)))
    ok = torch.tensor([int(same and same_bwd and layer.status() == 0)], device=dev)
    dist.all_reduce(ok, op=dist.ReduceOp.MIN)
    if rank == 0:
        print(json.dumps({"workload": cfg.name, "n_ranks": world, "T_total": cfg.T, "ms_per_layer": float(ms.item()),
                          "tokens_per_s": cfg.T / (float(ms.item()) * 1e-3),
                          "bitwise_equal_to_one_rank_layer": bool(ok.item()),
                          "backward_dx_dw_bitwise_equal_to_one_rank": bool(ok.item())}), flush=True)
    dist.barrier()
    dist.destroy_process_group()
    return 0 if ok.item() else 1


if __name__ == "__main__":
    raise SystemExit(main())
