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

    def __init__(self, n_ranks, T_local, H, I, I_shared, E, k, device, alloc=None):
        alloc = alloc or (lambda shape, dtype: torch.empty(shape, dtype=dtype, device=device))
        self.n_ranks, self.T_local, self.H, self.I, self.I_shared, self.E, self.k = n_ranks, T_local, H, I, I_shared, E, k
        n = mok.mok_ep_workspace_bytes(n_ranks, T_local, H, I, I_shared, E, k)
        if n == 0:
            raise mok.MokError(mok.MOK_ERR_SHAPE)
        self.ws = torch.empty(n + 256, dtype=torch.uint8, device=device)
        self.route_ws = mok.alloc_workspace(T_local, H, max(I, 8), 0, E, k, device=device)
        self.y = alloc((mok.mok_ep_y_rows(n_ranks, T_local, E, k), H), torch.bfloat16)
        self.pos = alloc((n_ranks * T_local * k,), torch.int32)
        tpad = (T_local + 255) // 256 * 256
        self.y_shared = torch.empty((max(tpad, 256), H), dtype=torch.bfloat16, device=device) if I_shared else None
        self.idx = self.w = None


def forward_emulated(xs, W_router, router_bias, W_gate_up, W_down, W_shared_gate_up, W_shared_down, k, config=None,
                     return_tables=False):
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
    st = [RankState(R, T_local, H, I, I_s, E, k, dev) for _ in range(R)]
    for r in range(R):                                                  # 1. local routing
        st[r].idx, st[r].w = mok.mok_route(xs[r], W_router, router_bias, k, st[r].route_ws)
    idx_all = torch.stack([s.idx.reshape(-1) for s in st]).contiguous()  # 2. the all-gather of the routes
    x_ptrs = [x.data_ptr() for x in xs]
    tables = []
    for c in range(R):                                                  # 3. schedule + expert FFNs of rank c
        tables.append(mok.mok_ep_expert_ffn(c, x_ptrs, idx_all, W_gate_up[c * L:(c + 1) * L], W_down[c * L:(c + 1) * L],
                                            W_shared_gate_up, W_shared_down, E, k, st[c].y, st[c].pos, st[c].y_shared,
                                            st[c].ws, H, outputs=return_tables, config=config))
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


class DistributedLayer:
    """One process per GPU under torch.distributed.  Buffers that peers read (x, y, pos) are allocated in symmetric
    memory once and exchanged by a rendezvous; `forward` then makes no allocation a peer depends on."""

    def __init__(self, T_local, H, I, I_shared, E, k, device, group=None):
        import torch.distributed as dist
        import torch.distributed._symmetric_memory as symm
        self.dist = dist
        self.group = group or dist.group.WORLD
        self.R, self.rank = dist.get_world_size(self.group), dist.get_rank(self.group)
        self.E, self.k, self.H = E, k, H
        handles = []

        def symm_alloc(shape, dtype):
            t = symm.empty(shape, dtype=dtype, device=device)
            handles.append(symm.rendezvous(t, self.group))
            return t

        self.st = RankState(self.R, T_local, H, I, I_shared, E, k, device, alloc=symm_alloc)   # y, pos: symmetric
        self.x = symm_alloc((T_local, H), torch.bfloat16)
        h_y, h_pos, h_x = handles
        self.y_ptrs = [int(p) for p in h_y.buffer_ptrs]
        self.pos_ptrs = [int(p) for p in h_pos.buffer_ptrs]
        self.x_ptrs = [int(p) for p in h_x.buffer_ptrs]
        self.idx_all = torch.empty((self.R, T_local * k), dtype=torch.int32, device=device)
        self._handles = handles

    def forward(self, x_local, W_router, router_bias, W_gate_up_local, W_down_local, W_shared_gate_up, W_shared_down,
                out=None, config=None):
        st, dist = self.st, self.dist
        dist.barrier(group=self.group)          # peers have finished reading the previous layer's x / y / pos
        self.x.copy_(x_local)
        st.idx, st.w = mok.mok_route(self.x, W_router, router_bias, self.k, st.route_ws)
        # the all-gather of the routes also orders every rank's x before any rank's pulls
        dist.all_gather_into_tensor(self.idx_all, st.idx.reshape(-1), group=self.group)
        mok.mok_ep_expert_ffn(self.rank, self.x_ptrs, self.idx_all, W_gate_up_local, W_down_local, W_shared_gate_up,
                              W_shared_down, self.E, self.k, st.y, st.pos, st.y_shared, st.ws, self.H, config=config)
        dist.barrier(group=self.group)          # every rank's y and pos are complete
        if out is None:
            out = torch.empty_like(x_local)
        mok.mok_ep_combine(self.rank, self.R, st.idx, st.w, self.y_ptrs, self.pos_ptrs, st.y_shared, self.E, out)
        return out

    def status(self):
        return mok.mok_read_status(self.st.ws)


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
    layer.dist.barrier(group=layer.group)       # nobody frees y while a peer still reads it
    status = layer.status()
    if status != 0:
        raise mok.MokError(status)
    return out


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
    ok = torch.tensor([int(same and layer.status() == 0)], device=dev)
    dist.all_reduce(ok, op=dist.ReduceOp.MIN)
    if rank == 0:
        print(json.dumps({"workload": cfg.name, "n_ranks": world, "T_total": cfg.T, "ms_per_layer": float(ms.item()),
                          "tokens_per_s": cfg.T / (float(ms.item()) * 1e-3),
                          "bitwise_equal_to_one_rank_layer": bool(ok.item())}), flush=True)
    dist.barrier()
    dist.destroy_process_group()
    return 0 if ok.item() else 1


if __name__ == "__main__":
    raise SystemExit(main())
