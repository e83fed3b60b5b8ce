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


def forward_distributed(x_local, W_router, router_bias, W_gate_up_local, W_down_local, W_shared_gate_up, W_shared_down,
                        E, k, group=None, config=None):
    """One process per GPU.  x_local bf16 [T_local, H]; W_gate_up_local [L, 2I, H] / W_down_local [L, H, I] are this
    rank's experts.  Buffers that peers read are allocated in symmetric memory and exchanged by a rendezvous; the
    function keeps them for the lifetime of the call only (a training loop would keep a RankState instead)."""
    import torch.distributed as dist
    import torch.distributed._symmetric_memory as symm
    group = group or dist.group.WORLD
    R, rank = dist.get_world_size(group), dist.get_rank(group)
    T_local, H = x_local.shape
    I = W_gate_up_local.shape[1] // 2
    I_s = 0 if W_shared_gate_up is None else W_shared_gate_up.shape[0] // 2
    dev = x_local.device
    handles = []

    def symm_alloc(shape, dtype):
        t = symm.empty(shape, dtype=dtype, device=dev)
        handles.append((t, symm.rendezvous(t, group)))
        return t

    st = RankState(R, T_local, H, I, I_s, E, k, dev, alloc=symm_alloc)      # y, pos: symmetric
    (_, h_y), (_, h_pos) = handles
    x_sym = symm_alloc(tuple(x_local.shape), torch.bfloat16)
    h_x = handles[-1][1]
    x_sym.copy_(x_local)
    st.idx, st.w = mok.mok_route(x_sym, W_router, router_bias, k, st.route_ws)
    idx_all = torch.empty((R, T_local * k), dtype=torch.int32, device=dev)
    dist.all_gather_into_tensor(idx_all, st.idx.reshape(-1), group=group)   # orders every rank's x before any pull
    mok.mok_ep_expert_ffn(rank, [int(p) for p in h_x.buffer_ptrs], idx_all, W_gate_up_local, W_down_local,
                          W_shared_gate_up, W_shared_down, E, k, st.y, st.pos, st.y_shared, st.ws, H, config=config)
    dist.barrier(group=group)                                               # all y / pos complete
    out = torch.empty_like(x_local)
    mok.mok_ep_combine(rank, R, st.idx, st.w, [int(p) for p in h_y.buffer_ptrs], [int(p) for p in h_pos.buffer_ptrs],
                       st.y_shared, E, out)
    dist.barrier(group=group)                                               # nobody frees y while a peer still reads
    status = mok.mok_read_status(st.ws)
    if status != 0:
        raise mok.MokError(status)
    return out
