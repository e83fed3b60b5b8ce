// Dispatch schedule construction on the device: Algorithm 1 of the paper for one rank.
//
// With a single source rank Algorithm 1 reduces to a stable counting sort of the routes by expert:
// M_{0,l} = counts[l], S_l = exclusive prefix sum, the ordinal o of a route is the number of earlier routes
// to the same expert and its position is p = o, so Phi[S_l + o] = route.  Three kernels (one for small batches), no host readback
// (Section 3.3), integer arithmetic only, hence bit-reproducible:
//   1. sched_hist    per-block expert histograms of SCHED_CHUNK consecutive routes
//   2. sched_scan    one block: per-expert prefix over blocks, counts, offsets, and the internal tile tables
//                    (each expert's segment is padded to a multiple of pad_m rows -> pad_offsets; it is cut into
//                    tiles of tile_m rows -> mt_start, tile_expert.  pad_m = tile_m = 128 or 256 when tokens sit on the
//                    MMA's M side, pad_m = 16 and tile_m = 128 when they sit on its N side)
//   3. sched_scatter stable ranks inside each block (warp match + per-warp running counters) -> perm, inv, pos,
//                    row_token (padded row -> source token: the {src_index} column of the paper's schedule table)
// Exported offsets/perm are unpadded; the padding is internal to the GEMM row space.
#include "mok_internal.cuh"
#include "schedule_common.cuh"

namespace mok {

__global__ void __launch_bounds__(SCHED_THREADS)
sched_hist_kernel(const int32_t* __restrict__ a, int n, int E, int32_t* __restrict__ blk_hist) {
    __shared__ int32_t hist[MAX_E];
    pdl_enter();
    for (int e = threadIdx.x; e < E; e += SCHED_THREADS) hist[e] = 0;
    __syncthreads();
    int base = blockIdx.x * SCHED_CHUNK;
    for (int i = threadIdx.x; i < SCHED_CHUNK; i += SCHED_THREADS) {
        int j = base + i;
        if (j < n && (unsigned)a[j] < (unsigned)E) atomicAdd(&hist[a[j]], 1);   // integer atomics: order-independent result
    }
    __syncthreads();
    for (int e = threadIdx.x; e < E; e += SCHED_THREADS) blk_hist[(size_t)blockIdx.x * E + e] = hist[e];
}

// One block of MAX_E threads.  Thread e walks the blocks for expert e (exclusive prefix, in place), then the
// block scans over experts.
__global__ void __launch_bounds__(MAX_E)
sched_scan_kernel(int32_t* __restrict__ blk_hist, int n_blk, int E, int max_mt, int tile_m, int pad_m,
                  int32_t* __restrict__ counts, int32_t* __restrict__ offsets, int32_t* __restrict__ pad_offsets,
                  int32_t* __restrict__ mt_start, int32_t* __restrict__ tile_expert,
                  int32_t* __restrict__ mt_start2, int32_t* __restrict__ tile_expert2, WsHeader* __restrict__ hdr,
                  int32_t* __restrict__ counts_out, int32_t* __restrict__ offsets_out) {
    __shared__ int32_t s_cnt[MAX_E], s_off[MAX_E + 1], s_mt[MAX_E + 1], s_pad[MAX_E + 1], s_mt2[MAX_E + 1];
    pdl_enter();
    const int e = threadIdx.x;
    int32_t total = 0;
    if (e < E) {
        for (int b0 = 0; b0 < n_blk; b0 += 16) {         // 16 independent loads in flight, then the serial prefix
            int32_t c[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) c[i] = (b0 + i < n_blk) ? blk_hist[(size_t)(b0 + i) * E + e] : 0;
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                if (b0 + i < n_blk) blk_hist[(size_t)(b0 + i) * E + e] = total;
                total += c[i];
            }
        }
        s_cnt[e] = total;
    }
    __syncthreads();
    scan_tables(s_cnt, s_off, s_mt, s_pad, s_mt2, E, max_mt, tile_m, pad_m, counts, offsets, pad_offsets, mt_start,
                tile_expert, mt_start2, tile_expert2, hdr, counts_out, offsets_out);
}

__global__ void __launch_bounds__(SCHED_THREADS)
sched_scatter_kernel(const int32_t* __restrict__ a, int n, int E,
                     const int32_t* __restrict__ blk_base, const int32_t* __restrict__ offsets,
                     const int32_t* __restrict__ pad_offsets,
                     int32_t* __restrict__ perm, int32_t* __restrict__ inv, int32_t* __restrict__ pos,
                     int32_t* __restrict__ row_token, int k,
                     int32_t* __restrict__ perm_out, int32_t* __restrict__ inv_out, int32_t* __restrict__ row_route) {
    extern __shared__ int32_t ssm[];                 // [SCHED_WARPS][E] running counters per warp
    pdl_enter();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int32_t* mine = ssm + warp * E;
    for (int e = threadIdx.x; e < SCHED_WARPS * E; e += SCHED_THREADS) ssm[e] = 0;
    __syncthreads();
    const int wbase = blockIdx.x * SCHED_CHUNK + warp * ROUTES_PER_WARP;
    // pass 1: this warp's histogram over its contiguous routes
    for (int i = 0; i < ROUTES_PER_WARP; i += 32) {
        int j = wbase + i + lane;
        bool valid = j < n;
        int e = valid ? a[j] : -1 - lane;            // invalid lanes get unique keys
        if ((unsigned)e >= (unsigned)E) { valid = false; e = -1 - lane; }
        unsigned peers = __match_any_sync(0xffffffffu, e);
        if (valid && lane == __ffs(peers) - 1) mine[e] += __popc(peers);
        __syncwarp();
    }
    __syncthreads();
    // warp-exclusive prefix over warps, plus the block's base for each expert -> starting rank per (warp, expert)
    for (int e = threadIdx.x; e < E; e += SCHED_THREADS) {
        int32_t run = blk_base[(size_t)blockIdx.x * E + e];
        for (int wi = 0; wi < SCHED_WARPS; ++wi) {
            int32_t c = ssm[wi * E + e];
            ssm[wi * E + e] = run;
            run += c;
        }
    }
    __syncthreads();
    // pass 2: ranks in route order
    for (int i = 0; i < ROUTES_PER_WARP; i += 32) {
        int j = wbase + i + lane;
        bool valid = j < n;
        int e = valid ? a[j] : -1 - lane;
        if ((unsigned)e >= (unsigned)E) { valid = false; e = -1 - lane; }
        unsigned peers = __match_any_sync(0xffffffffu, e);
        int before = __popc(peers & ((1u << lane) - 1u));
        int32_t rank = 0;
        if (valid) rank = mine[e] + before;          // ordinal o of Algorithm 1
        __syncwarp();
        if (valid && lane == __ffs(peers) - 1) mine[e] += __popc(peers);
        __syncwarp();
        if (valid) {
            int32_t p = offsets[e] + rank;           // Phi[S_l + o] = route j
            perm[p] = j;
            inv[j] = p;
            const int32_t prow = pad_offsets[e] + rank;   // row in the padded GEMM space
            pos[j] = prow;
            row_token[prow] = j / k;                 // the schedule table's src_index column, as a token id
            if (row_route) row_route[prow] = j;      // ... and as the route itself (the backward pass needs the slot)
            if (perm_out) perm_out[p] = j;
            if (inv_out) inv_out[j] = p;
        }
    }
}

// The three kernels above as ONE block, for batches of at most SCHED_CHUNK routes (a few hundred tokens: the layer is
// then bound by launch latency, and two launches fewer are a tenth of it).  Same arithmetic: per-warp histograms of
// contiguous route ranges, a prefix over the warps, the block-wide scans of the tables, ranks in route order.
__global__ void __launch_bounds__(MAX_E)
sched_small_kernel(const int32_t* __restrict__ a, int n, int E, int max_mt, int tile_m, int pad_m,
                   int32_t* __restrict__ counts, int32_t* __restrict__ offsets, int32_t* __restrict__ pad_offsets,
                   int32_t* __restrict__ mt_start, int32_t* __restrict__ tile_expert,
                   int32_t* __restrict__ mt_start2, int32_t* __restrict__ tile_expert2, WsHeader* __restrict__ hdr,
                   int32_t* __restrict__ counts_out, int32_t* __restrict__ offsets_out,
                   int32_t* __restrict__ perm, int32_t* __restrict__ inv, int32_t* __restrict__ pos,
                   int32_t* __restrict__ row_token, int k,
                   int32_t* __restrict__ perm_out, int32_t* __restrict__ inv_out, int32_t* __restrict__ row_route) {
    extern __shared__ int32_t ssm[];                 // [SCHED_WARPS][E] running counters per warp
    __shared__ int32_t s_cnt[MAX_E], s_off[MAX_E + 1], s_mt[MAX_E + 1], s_pad[MAX_E + 1], s_mt2[MAX_E + 1];
    pdl_enter();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int32_t* mine = ssm + (warp < SCHED_WARPS ? warp : 0) * E;
    for (int e = threadIdx.x; e < SCHED_WARPS * E; e += blockDim.x) ssm[e] = 0;
    __syncthreads();
    const int wbase = warp * ROUTES_PER_WARP;
    if (warp < SCHED_WARPS) {
        for (int i = 0; i < ROUTES_PER_WARP; i += 32) {
            int j = wbase + i + lane;
            bool valid = j < n;
            int e = valid ? a[j] : -1 - lane;            // invalid lanes get unique keys
            if ((unsigned)e >= (unsigned)E) { valid = false; e = -1 - lane; }
            unsigned peers = __match_any_sync(0xffffffffu, e);
            if (valid && lane == __ffs(peers) - 1) mine[e] += __popc(peers);
            __syncwarp();
        }
    }
    __syncthreads();
    if ((int)threadIdx.x < E) {                          // exclusive prefix over the warps; the total is the expert's count
        const int e = threadIdx.x;
        int32_t run = 0;
        for (int wi = 0; wi < SCHED_WARPS; ++wi) {
            int32_t c = ssm[wi * E + e];
            ssm[wi * E + e] = run;
            run += c;
        }
        s_cnt[e] = run;
    }
    __syncthreads();
    scan_tables(s_cnt, s_off, s_mt, s_pad, s_mt2, E, max_mt, tile_m, pad_m, counts, offsets, pad_offsets, mt_start,
                tile_expert, mt_start2, tile_expert2, hdr, counts_out, offsets_out);
    __syncthreads();
    if (warp < SCHED_WARPS) {
        for (int i = 0; i < ROUTES_PER_WARP; i += 32) {
            int j = wbase + i + lane;
            bool valid = j < n;
            int e = valid ? a[j] : -1 - lane;
            if ((unsigned)e >= (unsigned)E) { valid = false; e = -1 - lane; }
            unsigned peers = __match_any_sync(0xffffffffu, e);
            int before = __popc(peers & ((1u << lane) - 1u));
            int32_t rank = 0;
            if (valid) rank = mine[e] + before;          // ordinal o of Algorithm 1
            __syncwarp();
            if (valid && lane == __ffs(peers) - 1) mine[e] += __popc(peers);
            __syncwarp();
            if (valid) {
                int32_t p = s_off[e] + rank;
                perm[p] = j;
                inv[j] = p;
                const int32_t prow = s_pad[e] + rank;
                pos[j] = prow;
                row_token[prow] = j / k;
                if (row_route) row_route[prow] = j;
                if (perm_out) perm_out[p] = j;
                if (inv_out) inv_out[j] = p;
            }
        }
    }
}

cudaError_t launch_schedule(const int32_t* idx, int T, int E, int k, int tile_m, int pad_m, const WsLayout& L, char* ws,
                            int32_t* counts_out, int32_t* offsets_out, int32_t* perm_out, int32_t* inv_out,
                            cudaStream_t s, int32_t* row_route) {
    const int n = T * k;
    int32_t* blk_hist = reinterpret_cast<int32_t*>(ws + L.blk_hist);
    int32_t* counts = reinterpret_cast<int32_t*>(ws + L.counts);
    int32_t* offsets = reinterpret_cast<int32_t*>(ws + L.offsets);
    int32_t* pad_offsets = reinterpret_cast<int32_t*>(ws + L.pad_offsets);
    int32_t* mt_start = reinterpret_cast<int32_t*>(ws + L.mt_start);
    int32_t* tile_expert = reinterpret_cast<int32_t*>(ws + L.tile_expert);
    WsHeader* hdr = reinterpret_cast<WsHeader*>(ws + L.header);
    if (n <= SCHED_CHUNK)
        return launch_pdl(sched_small_kernel, dim3(1), dim3(MAX_E), sizeof(int32_t) * SCHED_WARPS * E, s, idx, n, E, L.max_mt,
                          tile_m, pad_m, counts, offsets, pad_offsets, mt_start, tile_expert,
                          reinterpret_cast<int32_t*>(ws + L.mt_start2), reinterpret_cast<int32_t*>(ws + L.tile_expert2), hdr,
                          counts_out, offsets_out, reinterpret_cast<int32_t*>(ws + L.perm), reinterpret_cast<int32_t*>(ws + L.inv),
                          reinterpret_cast<int32_t*>(ws + L.pos), reinterpret_cast<int32_t*>(ws + L.row_token), k, perm_out,
                          inv_out, row_route);
    cudaError_t e = launch_pdl(sched_hist_kernel, dim3(L.n_blk), dim3(SCHED_THREADS), 0, s, idx, n, E, blk_hist);
    if (e != cudaSuccess) return e;
    e = launch_pdl(sched_scan_kernel, dim3(1), dim3(MAX_E), 0, s, blk_hist, L.n_blk, E, L.max_mt, tile_m, pad_m, counts, offsets,
                   pad_offsets, mt_start, tile_expert, reinterpret_cast<int32_t*>(ws + L.mt_start2),
                   reinterpret_cast<int32_t*>(ws + L.tile_expert2), hdr, counts_out, offsets_out);
    if (e != cudaSuccess) return e;
    return launch_pdl(sched_scatter_kernel, dim3(L.n_blk), dim3(SCHED_THREADS), sizeof(int32_t) * SCHED_WARPS * E, s,
                      idx, n, E, blk_hist, offsets, pad_offsets,
                      reinterpret_cast<int32_t*>(ws + L.perm), reinterpret_cast<int32_t*>(ws + L.inv),
                      reinterpret_cast<int32_t*>(ws + L.pos), reinterpret_cast<int32_t*>(ws + L.row_token), k, perm_out,
                      inv_out, row_route);
}

}  // namespace mok
