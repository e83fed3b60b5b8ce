// Expert parallelism (Sections 2.1 and 3.1-3.3): Algorithm 1 for R source ranks on the device, the expert FFN whose
// gate/up GEMM pulls its rows from the source ranks' token buffers, and the owner-side deterministic combine.
//
// Algorithm 1 for rank c (L local experts, routes A[r, j] of every source rank r gathered beforehand):
//   M[r, l]  = number of routes of rank r to local expert l
//   S[l]     = exclusive prefix sum over l of sum_r M[r, l]
//   for a route (r, j) to local expert l with ordinal o (number of earlier routes of rank r to that expert):
//       p = sum_{r'} min(M[r', l], o) + |{ r' < r : M[r', l] > o }|,      Phi[S[l] + p] = (r, j)
// i.e. the rows of one expert cycle through the source ranks that still have routes, so consecutive pulls spread
// over the links.  Three kernels as for one rank (histograms per block, one scan block, scatter); blocks never
// straddle two source ranks, so the ordinal of a route is its block's exclusive prefix within the rank plus its
// stable position inside the block.  Integer arithmetic only: the result is unique and bit-reproducible.
#include "mok_internal.cuh"
#include "schedule_common.cuh"
#include <string.h>

namespace mok {

__global__ void __launch_bounds__(SCHED_THREADS)
ep_hist_kernel(const int32_t* __restrict__ a, int n, int bpr, int lo, int Lx, int32_t* __restrict__ blk_hist) {
    __shared__ int32_t hist[MAX_E];
    for (int e = threadIdx.x; e < Lx; e += SCHED_THREADS) hist[e] = 0;
    __syncthreads();
    const int r = blockIdx.x / bpr, cb = blockIdx.x - r * bpr;
    const size_t base = (size_t)r * n;
    for (int i = threadIdx.x; i < SCHED_CHUNK; i += SCHED_THREADS) {
        const int j = cb * SCHED_CHUNK + i;
        if (j < n) {
            const int l = a[base + j] - lo;
            if ((unsigned)l < (unsigned)Lx) atomicAdd(&hist[l], 1);   // integer atomics: order-independent result
        }
    }
    __syncthreads();
    for (int e = threadIdx.x; e < Lx; e += SCHED_THREADS) blk_hist[(size_t)blockIdx.x * Lx + e] = hist[e];
}

// One block of MAX_E threads.  Thread l walks the blocks of every source rank for local expert l: exclusive prefix
// within the rank (in place) and the rank's total M[r, l]; then the block scans over the experts.
__global__ void __launch_bounds__(MAX_E)
ep_scan_kernel(int32_t* __restrict__ blk_hist, int R, int bpr, int Lx, int max_mt, int tile_m,
               int32_t* __restrict__ M, int32_t* __restrict__ counts, int32_t* __restrict__ offsets,
               int32_t* __restrict__ pad_offsets, int32_t* __restrict__ mt_start, int32_t* __restrict__ tile_expert,
               int32_t* __restrict__ mt_start2, int32_t* __restrict__ tile_expert2, WsHeader* __restrict__ hdr,
               int32_t* __restrict__ M_out, int32_t* __restrict__ S_out) {
    __shared__ int32_t s_cnt[MAX_E], s_off[MAX_E + 1], s_mt[MAX_E + 1], s_pad[MAX_E + 1], s_mt2[MAX_E + 1];
    const int l = threadIdx.x;
    if (l < Lx) {
        int32_t total = 0;
        for (int r = 0; r < R; ++r) {
            int32_t run = 0;
            int32_t* col = blk_hist + (size_t)r * bpr * Lx + l;
            for (int b0 = 0; b0 < bpr; b0 += 8) {          // 8 independent loads in flight, then the serial prefix
                int32_t c[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) c[i] = (b0 + i < bpr) ? col[(size_t)(b0 + i) * Lx] : 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (b0 + i < bpr) col[(size_t)(b0 + i) * Lx] = run;
                    run += c[i];
                }
            }
            M[(size_t)r * Lx + l] = run;
            if (M_out) M_out[(size_t)r * Lx + l] = run;
            total += run;
        }
        s_cnt[l] = total;
    }
    __syncthreads();
    scan_tables(s_cnt, s_off, s_mt, s_pad, s_mt2, Lx, max_mt, tile_m, tile_m, counts, offsets, pad_offsets, mt_start,
                tile_expert, mt_start2, tile_expert2, hdr, nullptr, S_out);
}

__global__ void __launch_bounds__(SCHED_THREADS)
ep_scatter_kernel(const int32_t* __restrict__ a, int n, int bpr, int R, int lo, int Lx,
                  const int32_t* __restrict__ blk_base, const int32_t* __restrict__ M,
                  const int32_t* __restrict__ offsets, const int32_t* __restrict__ pad_offsets,
                  int32_t* __restrict__ phi_rank, int32_t* __restrict__ phi_index, int32_t* __restrict__ row_token,
                  int k, int tokens_per_rank, int32_t* __restrict__ pos_out,
                  int32_t* __restrict__ phi_rank_out, int32_t* __restrict__ phi_index_out) {
    extern __shared__ int32_t ssm[];                 // [SCHED_WARPS][Lx] running counters per warp
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int32_t* mine = ssm + warp * Lx;
    for (int e = threadIdx.x; e < SCHED_WARPS * Lx; e += SCHED_THREADS) ssm[e] = 0;
    __syncthreads();
    const int r = blockIdx.x / bpr, cb = blockIdx.x - r * bpr;
    const size_t base = (size_t)r * n;
    const int wbase = cb * SCHED_CHUNK + warp * ROUTES_PER_WARP;
    // pass 1: this warp's histogram over its contiguous routes
    for (int i = 0; i < ROUTES_PER_WARP; i += 32) {
        const int j = wbase + i + lane;
        bool valid = j < n;
        int l = valid ? a[base + j] - lo : -1 - lane;       // invalid lanes get unique keys
        if ((unsigned)l >= (unsigned)Lx) { valid = false; l = -1 - lane; }
        const unsigned peers = __match_any_sync(0xffffffffu, l);
        if (valid && lane == __ffs(peers) - 1) mine[l] += __popc(peers);
        __syncwarp();
    }
    __syncthreads();
    // warp-exclusive prefix over warps, plus the block's base within its source rank -> starting ordinal
    for (int e = threadIdx.x; e < Lx; e += SCHED_THREADS) {
        int32_t run = blk_base[(size_t)blockIdx.x * Lx + e];
        for (int wi = 0; wi < SCHED_WARPS; ++wi) {
            const int32_t c = ssm[wi * Lx + e];
            ssm[wi * Lx + e] = run;
            run += c;
        }
    }
    __syncthreads();
    // pass 2: ordinals in route order, then the position formula of Algorithm 1
    for (int i = 0; i < ROUTES_PER_WARP; i += 32) {
        const int j = wbase + i + lane;
        bool valid = j < n;
        int l = valid ? a[base + j] - lo : -1 - lane;
        if ((unsigned)l >= (unsigned)Lx) { valid = false; l = -1 - lane; }
        const unsigned peers = __match_any_sync(0xffffffffu, l);
        const int before = __popc(peers & ((1u << lane) - 1u));
        int32_t o = 0;
        if (valid) o = mine[l] + before;
        __syncwarp();
        if (valid && lane == __ffs(peers) - 1) mine[l] += __popc(peers);
        __syncwarp();
        if (valid) {
            int32_t p = 0;
            for (int rp = 0; rp < R; ++rp) {
                const int32_t m = __ldg(M + (size_t)rp * Lx + l);
                p += min(m, o) + ((rp < r && m > o) ? 1 : 0);
            }
            const int32_t row = offsets[l] + p;               // Phi[S_l + p] = (r, j)
            phi_rank[row] = r;
            phi_index[row] = j;
            if (phi_rank_out) phi_rank_out[row] = r;
            if (phi_index_out) phi_index_out[row] = j;
            const int32_t prow = pad_offsets[l] + p;          // row in the padded GEMM space = row of y
            row_token[prow] = r * tokens_per_rank + j / k;    // global token id: which rank to pull from, which row
            pos_out[base + j] = prow;
        }
    }
}

cudaError_t launch_ep_schedule(const int32_t* idx_all, int n_ranks, int rank, int routes_per_rank, int k,
                               int tokens_per_rank, int experts_local, int tile_m, const WsLayout& L, char* ws,
                               int32_t* pos_out, int32_t* M_out, int32_t* S_out, int32_t* phi_rank_out,
                               int32_t* phi_index_out, cudaStream_t s) {
    const int bpr = (routes_per_rank + SCHED_CHUNK - 1) / SCHED_CHUNK;
    int32_t* blk_hist = reinterpret_cast<int32_t*>(ws + L.blk_hist);
    int32_t* M = reinterpret_cast<int32_t*>(ws + L.w);       // the weights region is unused in this mode
    WsHeader* hdr = reinterpret_cast<WsHeader*>(ws + L.header);
    const int lo = rank * experts_local;
    ep_hist_kernel<<<n_ranks * bpr, SCHED_THREADS, 0, s>>>(idx_all, routes_per_rank, bpr, lo, experts_local, blk_hist);
    ep_scan_kernel<<<1, MAX_E, 0, s>>>(blk_hist, n_ranks, bpr, experts_local, L.max_mt, tile_m, M,
                                       reinterpret_cast<int32_t*>(ws + L.counts), reinterpret_cast<int32_t*>(ws + L.offsets),
                                       reinterpret_cast<int32_t*>(ws + L.pad_offsets),
                                       reinterpret_cast<int32_t*>(ws + L.mt_start), reinterpret_cast<int32_t*>(ws + L.tile_expert),
                                       reinterpret_cast<int32_t*>(ws + L.mt_start2), reinterpret_cast<int32_t*>(ws + L.tile_expert2),
                                       hdr, M_out, S_out);
    ep_scatter_kernel<<<n_ranks * bpr, SCHED_THREADS, sizeof(int32_t) * SCHED_WARPS * experts_local, s>>>(
        idx_all, routes_per_rank, bpr, n_ranks, lo, experts_local, blk_hist, M,
        reinterpret_cast<const int32_t*>(ws + L.offsets), reinterpret_cast<const int32_t*>(ws + L.pad_offsets),
        reinterpret_cast<int32_t*>(ws + L.inv), reinterpret_cast<int32_t*>(ws + L.perm),
        reinterpret_cast<int32_t*>(ws + L.row_token), k, tokens_per_rank, pos_out, phi_rank_out, phi_index_out);
    return cudaGetLastError();
}

// out[t,:] = ysh[t,:] + sum_{s=0}^{k-1} w[t,s] * y_{c(s)}[pos_{c(s)}[rank*n + t*k + s], :], c(s) = idx[t,s] / L:
// the owner pulls each of its k rows from the rank that served the route and reduces them in slot order in fp32.
struct EpCombineArgs {
    const __nv_bfloat16* y[MOK_MAX_RANKS];
    const int32_t* pos[MOK_MAX_RANKS];
    const __nv_bfloat16* ysh;
    const int32_t* idx;
    const float* w;
    __nv_bfloat16* out;
    int32_t T, H, k, Lx, route_base;
};

__global__ void __launch_bounds__(128)
ep_combine_kernel(const __grid_constant__ EpCombineArgs a) {
    __shared__ const __nv_bfloat16* s_row[MAX_K];
    __shared__ float s_w[MAX_K];
    const int t = blockIdx.x;
    if (threadIdx.x < a.k) {
        const size_t j = (size_t)t * a.k + threadIdx.x;
        const int c = a.idx[j] / a.Lx;
        const int32_t p = a.pos[c][(size_t)a.route_base + j];
        s_row[threadIdx.x] = a.y[c] + (size_t)p * a.H;
        s_w[threadIdx.x] = a.w ? a.w[j] : 1.f;          // w == NULL: plain sum (backward pass)
    }
    __syncthreads();
    const int chunks = a.H >> 3;
    for (int c = threadIdx.x; c < chunks; c += 128) {
        float acc[8];
        if (a.ysh) {
            const uint4 raw = *reinterpret_cast<const uint4*>(a.ysh + (size_t)t * a.H + c * 8);
            const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 f = __bfloat1622float2(p2[i]);
                acc[2 * i] = f.x;
                acc[2 * i + 1] = f.y;
            }
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] = 0.f;
        }
#pragma unroll 4
        for (int s = 0; s < a.k; ++s) {
            const uint4 raw = *reinterpret_cast<const uint4*>(s_row[s] + c * 8);
            const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
            const float ws = s_w[s];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 f = __bfloat1622float2(p2[i]);
                acc[2 * i] = fmaf(ws, f.x, acc[2 * i]);
                acc[2 * i + 1] = fmaf(ws, f.y, acc[2 * i + 1]);
            }
        }
        uint4 o;
        __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
        for (int i = 0; i < 4; ++i) o2[i] = __floats2bfloat162_rn(acc[2 * i], acc[2 * i + 1]);
        *reinterpret_cast<uint4*>(a.out + (size_t)t * a.H + c * 8) = o;
    }
}

// Workspace of one rank: the one-rank layout for n_ranks*T_local "tokens" and L experts without the router and
// gathered-copy regions, with room for the per-(rank, block) histograms and M.
bool ep_layout(int n_ranks, int T_local, int H, int I, int Is, int E, int k, WsLayout* L, bool mx) {
    if (n_ranks < 1 || n_ranks > MOK_MAX_RANKS || T_local < 0 || E < 1 || E % n_ranks) return false;
    if (H <= 0 || I <= 0 || Is < 0 || (H % 8) || (I % 8) || (Is % 8) || k < 1 || k > MAX_K || k > E || E > MAX_E) return false;
    const int Lx = E / n_ranks;
    const long long n = (long long)T_local * k, R = n * n_ranks;
    if (R >= (1ll << 31) / 256) return false;
    memset(L, 0, sizeof(*L));
    const long long nonempty_max = R < Lx ? R : Lx;
    long long Rpad = (R + nonempty_max * (2 * TILE_M - 1) + 2 * TILE_M - 1) / (2 * TILE_M) * (2 * TILE_M);
    if (Rpad < 2 * TILE_M) Rpad = 2 * TILE_M;
    L->R = (int32_t)R;
    L->Rpad = (int32_t)Rpad;
    L->max_mt = (int32_t)(Rpad / TILE_M);
    L->Tpad = (T_local + 2 * TILE_M - 1) / (2 * TILE_M) * (2 * TILE_M);
    if (L->Tpad < 2 * TILE_M) L->Tpad = 2 * TILE_M;
    const long long bpr = (n + SCHED_CHUNK - 1) / SCHED_CHUNK;
    L->n_blk = (int32_t)(bpr * n_ranks > 0 ? bpr * n_ranks : 1);
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    const size_t Rn = (size_t)(R > 0 ? R : 1);
    L->header = take(sizeof(WsHeader));
    L->w = take(sizeof(int32_t) * (size_t)n_ranks * Lx);          // M[r, l]
    L->counts = take(sizeof(int32_t) * Lx);
    L->offsets = take(sizeof(int32_t) * (Lx + 1));
    L->pad_offsets = take(sizeof(int32_t) * (Lx + 1));
    L->mt_start = take(sizeof(int32_t) * (Lx + 1));
    L->tile_expert = take(sizeof(int32_t) * (size_t)L->max_mt);
    L->mt_start2 = take(sizeof(int32_t) * (Lx + 1));
    L->tile_expert2 = take(sizeof(int32_t) * (size_t)L->max_mt);
    L->perm = take(sizeof(int32_t) * Rn);                          // Phi: source route index
    L->inv = take(sizeof(int32_t) * Rn);                           // Phi: source rank
    L->blk_hist = take(sizeof(int32_t) * (size_t)L->n_blk * Lx);
    L->row_token = take(sizeof(int32_t) * (size_t)Rpad);
    L->h = take(2 * (size_t)Rpad * I);
    L->hs = take(Is > 0 ? 2 * (size_t)L->Tpad * Is : 0);
    if (!mx) {   // one-launch expert FFN: its tile list and the two completion counters per 256-row tile
        const long long mt2 = Rpad / (2 * TILE_M), per = (I + 127) / 128 + (H + 255) / 256;
        const long long nt = mt2 * per;
        L->max_ftiles = nt < (1ll << 30) ? (int32_t)nt : 0;
        L->ftiles = take(sizeof(int4) * (size_t)L->max_ftiles);
        L->ready = take(4 * sizeof(int32_t) * (size_t)mt2);    // ready, consumed, staged, released
        L->xg = take(2 * (size_t)FFN_COMM_SLOTS * 2 * TILE_M * H);    // staging slots of the communication CTAs
    }
    {   // gang-start counters of the 256-row kernel: one per tile of the largest of the four GEMMs
        const long long mt2 = Rpad / (2 * TILE_M), mts = L->Tpad / (2 * TILE_M);
        const long long n_r = (I + 127) / 128 > (H + 255) / 256 ? (I + 127) / 128 : (H + 255) / 256;
        const long long n_s = (Is + 127) / 128 > (H + 255) / 256 ? (Is + 127) / 128 : (H + 255) / 256;
        long long tiles = mt2 * n_r > mts * n_s ? mt2 * n_r : mts * n_s;
        if (L->max_ftiles > tiles) tiles = L->max_ftiles;       // the one-launch FFN's list (static hand-out)
        L->gang_bytes = sizeof(int32_t) * (size_t)tiles;
        L->gang = take(L->gang_bytes);
    }
    if (mx) {
        if ((H % 32) || (I % 32)) return false;
        L->h8 = take((size_t)Rpad * I);
        L->sh = take((size_t)(Rpad / TILE_M) * ((I + 127) / 128) * 512);
    }
    L->total = off;
    return true;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace mok

using namespace mok;

extern "C" {

size_t mok_ep_workspace_bytes(int n_ranks, int T_local, int H, int I, int I_shared, int E, int k) {
    WsLayout L;
    return ep_layout(n_ranks, T_local, H, I, I_shared, E, k, &L) ? L.total : 0;
}

size_t mok_ep_mx_workspace_bytes(int n_ranks, int T_local, int H, int I, int I_shared, int E, int k) {
    WsLayout L;
    return ep_layout(n_ranks, T_local, H, I, I_shared, E, k, &L, true) ? L.total : 0;
}

long long mok_ep_y_rows(int n_ranks, int T_local, int E, int k) {
    WsLayout L;
    return ep_layout(n_ranks, T_local, 8, 8, 0, E, k, &L) ? (long long)L.Rpad : 0;
}

int mok_ep_expert_ffn(const mok_ep_args* a) {
    if (!a) return MOK_ERR_NULL;
    WsLayout L;
    if (a->config && (a->config->precision < 0 || a->config->precision > 1)) return MOK_ERR_SHAPE;
    const bool mx = a->config && a->config->precision == MOK_PRECISION_MXFP8;
    if (!ep_layout(a->n_ranks, a->T_local, a->H, a->I, a->I_shared, a->E, a->k, &L, mx)) return MOK_ERR_SHAPE;
    if (a->rank < 0 || a->rank >= a->n_ranks) return MOK_ERR_SHAPE;
    if ((a->I_shared > 0) != (a->W_shared_gate_up != nullptr) || (a->I_shared > 0) != (a->W_shared_down != nullptr))
        return MOK_ERR_SHAPE;
    if (a->config && (a->config->impl != MOK_IMPL_TCGEN05 || a->config->grid < 0 ||
                      (a->config->cta_group != 0 && a->config->cta_group != 1 && a->config->cta_group != 3) ||
                      a->config->comm_ctas < 0))
        return MOK_ERR_SHAPE;
    if (a->T_local == 0) return MOK_OK;
    if (!a->idx_all || !a->pos) return MOK_ERR_NULL;
    if (!a->schedule_only) {
        if (!a->y || (a->I_shared > 0 && !a->y_shared)) return MOK_ERR_NULL;
        if (mx) {
            if (!a->W_gate_up_codes || !a->W_gate_up_scales || !a->W_down_codes || !a->W_down_scales) return MOK_ERR_NULL;
            if (!aligned16(a->W_gate_up_codes) || !aligned16(a->W_gate_up_scales) || !aligned16(a->W_down_codes) ||
                !aligned16(a->W_down_scales))
                return MOK_ERR_ALIGN;
            if (a->I_shared > 0 && !a->x_peers[a->rank]) return MOK_ERR_NULL;
        } else if (!a->W_gate_up || !a->W_down) {
            return MOK_ERR_NULL;
        }
        for (int r = 0; r < a->n_ranks; ++r) {
            if (mx) {
                if (!a->x_codes_peers[r] || !a->x_scales_peers[r]) return MOK_ERR_NULL;
                if (!aligned16(a->x_codes_peers[r]) || (reinterpret_cast<uintptr_t>(a->x_scales_peers[r]) & 3u)) return MOK_ERR_ALIGN;
            } else {
                if (!a->x_peers[r]) return MOK_ERR_NULL;
                if (!aligned16(a->x_peers[r])) return MOK_ERR_ALIGN;
            }
        }
        if (!aligned16(a->W_gate_up) || !aligned16(a->W_down) || !aligned16(a->W_shared_gate_up) ||
            !aligned16(a->W_shared_down) || !aligned16(a->y) || !aligned16(a->y_shared))
            return MOK_ERR_ALIGN;
        if (a->y_rows < L.Rpad) return MOK_ERR_WORKSPACE;
    }
    if (!a->workspace || (reinterpret_cast<uintptr_t>(a->workspace) & 255u) || a->workspace_bytes < L.total)
        return MOK_ERR_WORKSPACE;

    cudaStream_t s = reinterpret_cast<cudaStream_t>(a->stream);
    char* ws = reinterpret_cast<char*>(a->workspace);
    WsHeader* hdr = reinterpret_cast<WsHeader*>(ws + L.header);
    cudaError_t e = cudaMemsetAsync(hdr, 0, sizeof(WsHeader), s);
    if (e != cudaSuccess) return cuda_fail(e);
    const int Lx = a->E / a->n_ranks, n = a->T_local * a->k;
    e = launch_ep_schedule(a->idx_all, a->n_ranks, a->rank, n, a->k, a->T_local, Lx, TILE_M, L, ws, a->pos, a->M, a->S,
                           a->phi_rank, a->phi_index, s);
    if (e != cudaSuccess) return cuda_fail(e);
    if (a->schedule_only) return MOK_OK;

    mok_config cfg;
    memset(&cfg, 0, sizeof(cfg));
    if (a->config) {
        cfg.grid = a->config->grid; cfg.cta_group = a->config->cta_group; cfg.gang_sync = a->config->gang_sync;
        cfg.fused_ffn = a->config->fused_ffn == 3 ? 2 : a->config->fused_ffn;     // (the combine is the owners' call here)
        cfg.fused_window = a->config->fused_window; cfg.tile_sched = a->config->tile_sched;
        cfg.comm_ctas = a->config->comm_ctas;
    }
    const __nv_bfloat16* x_own = reinterpret_cast<const __nv_bfloat16*>(a->x_peers[a->rank]);   // (may be NULL in MXFP8 mode without a shared expert)
    GemmArgs g;
    memset(&g, 0, sizeof(g));
    g.header = hdr;
    g.n_mtiles = &hdr->n_mtiles;
    g.tile_expert = reinterpret_cast<const int32_t*>(ws + L.tile_expert);
    g.mt_start = reinterpret_cast<const int32_t*>(ws + L.mt_start);
    g.max_mt = L.max_mt;
    g.tile_m = TILE_M;
    g.pad_offsets = reinterpret_cast<const int32_t*>(ws + L.pad_offsets);
    g.counts = reinterpret_cast<const int32_t*>(ws + L.counts);
    g.dbg_slot = -1;
    int rc;
    if (mx) {
        // routed experts on MXFP8 operands (Section 3.4): codes and scales of row (src_rank, token) are pulled from that
        // rank's quantised buffers; the gated activation is quantised in the gate/up epilogue
        e = cudaMemsetAsync(ws + L.sh, 127, (size_t)(L.Rpad / TILE_M) * ((a->I + 127) / 128) * 512, s);
        if (e != cudaSuccess) return cuda_fail(e);
        g.A = reinterpret_cast<const __nv_bfloat16*>(a->x_codes_peers[a->rank]);
        g.a_rows = a->T_local;
        g.row_token = reinterpret_cast<const int32_t*>(ws + L.row_token);
        g.peer_tokens = a->T_local;
        for (int r = 0; r < a->n_ranks; ++r) {
            g.peer_x[r] = reinterpret_cast<const __nv_bfloat16*>(a->x_codes_peers[r]);
            g.peer_sfa[r] = reinterpret_cast<const uint8_t*>(a->x_scales_peers[r]);
        }
        g.sfa = g.peer_sfa[a->rank];
        g.sfa_stride = (a->H + 127) / 128 * 4;
        g.B = reinterpret_cast<const __nv_bfloat16*>(a->W_gate_up_codes);
        g.sfb = reinterpret_cast<const uint8_t*>(a->W_gate_up_scales);
        g.C = ws + L.h8;
        g.sfc = reinterpret_cast<uint8_t*>(ws + L.sh);
        g.K = a->H; g.N = a->I; g.ldc = a->I; g.E = Lx; g.rows_pad = L.Rpad; g.dense_rows = 0;
        g.total_rows = n;
        e = launch_gemm_mx(g, EPI_SWIGLU, cfg.grid, s);
        if (e != cudaSuccess) return cuda_fail(e);
        g.row_token = nullptr;
        g.peer_tokens = 0;
        g.A = reinterpret_cast<const __nv_bfloat16*>(ws + L.h8);
        g.a_rows = L.Rpad;
        g.sfa = reinterpret_cast<const uint8_t*>(ws + L.sh);
        g.B = reinterpret_cast<const __nv_bfloat16*>(a->W_down_codes);
        g.sfb = reinterpret_cast<const uint8_t*>(a->W_down_scales);
        g.C = a->y;
        g.sfc = nullptr;
        g.K = a->I; g.N = a->H; g.ldc = a->H;
        e = launch_gemm_mx(g, EPI_BF16, cfg.grid, s);
        if (e != cudaSuccess) return cuda_fail(e);
        g.sfa = g.sfb = nullptr;
    } else {
        // routed experts of this rank: the gather warps pull row (src_rank, token) of the schedule from x_peers[src_rank]
        g.A = x_own;
        g.a_rows = a->T_local;
        g.row_token = reinterpret_cast<const int32_t*>(ws + L.row_token);
        g.peer_tokens = a->T_local;
        for (int r = 0; r < a->n_ranks; ++r) g.peer_x[r] = reinterpret_cast<const __nv_bfloat16*>(a->x_peers[r]);
        g.B = reinterpret_cast<const __nv_bfloat16*>(a->W_gate_up);
        g.C = ws + L.h;
        g.K = a->H; g.N = a->I; g.ldc = a->I; g.E = Lx; g.rows_pad = L.Rpad; g.dense_rows = 0;
        g.total_rows = n;   // expected share of this rank, for the kernel choice
        // the routed experts as ONE persistent launch where the one-rank layer would choose it (large expert matrices),
        // or on request: the same kernel, its gather warps pulling from the owners' buffers, its down tiles storing
        // into the peer-visible y
        bool fused_sync = false;
        const bool fused = fused_ffn_choice(&cfg, a->H, a->I, TILE_M, n, Lx, L.max_ftiles, &fused_sync);
        if (cfg.comm_ctas > 0 && !fused) return MOK_ERR_UNSUPPORTED;     // communication CTAs exist in that kernel only
        if (fused) {
            const bool dynamic = cfg.tile_sched == 1 || (cfg.tile_sched == 0 && !fused_sync);
            e = launch_fused_ffn(x_own, a->T_local, a->H, a->I, Lx, reinterpret_cast<const __nv_bfloat16*>(a->W_gate_up),
                                 reinterpret_cast<const __nv_bfloat16*>(a->W_down), L, ws, cfg.grid, cfg.fused_window, dynamic,
                                 fused_sync, false, 0, s, nullptr, 0, false, 0, a->x_peers, a->T_local, a->y, cfg.comm_ctas,
                                 cfg.comm_ctas > 0 ? ws + L.xg : nullptr);
            if (e != cudaSuccess) return cuda_fail(e);
        } else {
            if ((rc = run_gemm(g, true, &cfg, L, ws, s))) return rc;
            g.row_token = nullptr;
            g.peer_tokens = 0;
            g.a_rows = L.Rpad;
            g.A = reinterpret_cast<const __nv_bfloat16*>(ws + L.h);
            g.B = reinterpret_cast<const __nv_bfloat16*>(a->W_down);
            g.C = a->y;
            g.K = a->I; g.N = a->H; g.ldc = a->H;
            if ((rc = run_gemm(g, false, &cfg, L, ws, s))) return rc;
        }
        g.row_token = nullptr;
        g.peer_tokens = 0;
    }
    if (a->I_shared > 0) {   // shared expert on the rank's own tokens, natural order
        g.A = x_own;
        g.B = reinterpret_cast<const __nv_bfloat16*>(a->W_shared_gate_up);
        g.C = ws + L.hs;
        g.K = a->H; g.N = a->I_shared; g.ldc = a->I_shared; g.E = 1; g.rows_pad = L.Tpad; g.a_rows = a->T_local;
        g.dense_rows = a->T_local;
        if ((rc = run_gemm(g, true, &cfg, L, ws, s))) return rc;
        g.A = reinterpret_cast<const __nv_bfloat16*>(ws + L.hs);
        g.B = reinterpret_cast<const __nv_bfloat16*>(a->W_shared_down);
        g.C = a->y_shared;
        g.K = a->I_shared; g.N = a->H; g.ldc = a->H; g.a_rows = L.Tpad;
        if ((rc = run_gemm(g, false, &cfg, L, ws, s))) return rc;
    }
    return MOK_OK;
}

int mok_ep_combine(const mok_ep_combine_args* a) { return ep_combine_impl(a, false); }

}  // extern "C"

namespace mok {

int ep_combine_impl(const mok_ep_combine_args* a, bool unit_weights) {
    if (!a) return MOK_ERR_NULL;
    if (a->n_ranks < 1 || a->n_ranks > MOK_MAX_RANKS || a->rank < 0 || a->rank >= a->n_ranks || a->T_local < 0 ||
        a->H <= 0 || (a->H % 8) || a->E < 1 || a->E % a->n_ranks || a->k < 1 || a->k > MAX_K || a->k > a->E)
        return MOK_ERR_SHAPE;
    if (a->T_local == 0) return MOK_OK;
    if (!a->topk_idx || (!unit_weights && !a->topk_w) || !a->out) return MOK_ERR_NULL;
    if (!aligned16(a->out) || !aligned16(a->y_shared)) return MOK_ERR_ALIGN;
    EpCombineArgs c;
    memset(&c, 0, sizeof(c));
    for (int r = 0; r < a->n_ranks; ++r) {
        if (!a->y_peers[r] || !a->pos_peers[r]) return MOK_ERR_NULL;
        if (!aligned16(a->y_peers[r])) return MOK_ERR_ALIGN;
        c.y[r] = reinterpret_cast<const __nv_bfloat16*>(a->y_peers[r]);
        c.pos[r] = a->pos_peers[r];
    }
    c.ysh = reinterpret_cast<const __nv_bfloat16*>(a->y_shared);
    c.idx = a->topk_idx;
    c.w = unit_weights ? nullptr : a->topk_w;
    c.out = reinterpret_cast<__nv_bfloat16*>(a->out);
    c.T = a->T_local; c.H = a->H; c.k = a->k; c.Lx = a->E / a->n_ranks;
    c.route_base = a->rank * a->T_local * a->k;
    ep_combine_kernel<<<a->T_local, 128, 0, reinterpret_cast<cudaStream_t>(a->stream)>>>(c);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? MOK_OK : cuda_fail(e);
}

}  // namespace mok
