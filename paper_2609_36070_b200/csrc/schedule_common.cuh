// Pieces shared by the one-rank and the R-rank schedule kernels (Algorithm 1): block geometry and the step that
// turns per-expert row counts into offsets and the GEMMs' internal tile tables.
#pragma once
#include "mok_internal.cuh"

namespace mok {

constexpr int SCHED_THREADS = 256;
constexpr int SCHED_WARPS = SCHED_THREADS / 32;
constexpr int ROUTES_PER_WARP = SCHED_CHUNK / SCHED_WARPS;   // contiguous routes owned by one warp

// Called by every thread of a block of at least E threads (a multiple of 32, at most 1024) after s_cnt[0..E) is
// complete and the block has synchronised.  S_l (offsets) is the exclusive prefix sum of the counts (Algorithm 1);
// each expert's segment of the padded row space starts at a multiple of pad_m rows and is cut into tiles of tile_m
// and of 2*tile_m rows.  The four prefix sums are one block-wide scan (warp shuffles, then the warp totals).
__device__ __forceinline__ void scan_tables(const int32_t* s_cnt, int32_t* s_off, int32_t* s_mt, int32_t* s_pad,
                                            int32_t* s_mt2, int E, int max_mt, int tile_m, int pad_m,
                                            int32_t* __restrict__ counts, int32_t* __restrict__ offsets,
                                            int32_t* __restrict__ pad_offsets, int32_t* __restrict__ mt_start,
                                            int32_t* __restrict__ tile_expert, int32_t* __restrict__ mt_start2,
                                            int32_t* __restrict__ tile_expert2, WsHeader* __restrict__ hdr,
                                            int32_t* __restrict__ counts_out, int32_t* __restrict__ offsets_out) {
    __shared__ int32_t s_wtot[4][32];
    const int e = threadIdx.x, lane = e & 31, wid = e >> 5, n_warps = (blockDim.x + 31) >> 5;
    const int32_t c = (e < E) ? s_cnt[e] : 0;
    int32_t v[4] = {c, (c + tile_m - 1) / tile_m, (c + 2 * tile_m - 1) / (2 * tile_m), (c + pad_m - 1) / pad_m * pad_m};
    int32_t inc[4] = {v[0], v[1], v[2], v[3]};
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int32_t t = __shfl_up_sync(0xffffffffu, inc[q], off);
            if (lane >= off) inc[q] += t;
        }
    }
    if (lane == 31) {
#pragma unroll
        for (int q = 0; q < 4; ++q) s_wtot[q][wid] = inc[q];
    }
    __syncthreads();
    if (wid == 0) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int32_t mine = (lane < n_warps) ? s_wtot[q][lane] : 0;
            int32_t run = mine;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int32_t t = __shfl_up_sync(0xffffffffu, run, off);
                if (lane >= off) run += t;
            }
            s_wtot[q][lane] = run - mine;               // exclusive prefix of the warp totals
        }
    }
    __syncthreads();
    if (e < E) {
        const int32_t off = s_wtot[0][wid] + inc[0] - v[0], mt = s_wtot[1][wid] + inc[1] - v[1];
        const int32_t mt2 = s_wtot[2][wid] + inc[2] - v[2], pad = s_wtot[3][wid] + inc[3] - v[3];
        s_off[e] = off;
        s_mt[e] = mt;
        s_mt2[e] = mt2;
        s_pad[e] = pad;
        if (e == E - 1) {
            s_off[E] = off + v[0];
            s_mt[E] = mt + v[1];
            s_mt2[E] = mt2 + v[2];
            s_pad[E] = pad + v[3];
            hdr->n_mtiles = mt + v[1];
            hdr->n_mtiles2 = mt2 + v[2];
            if ((mt + v[1]) * (tile_m / TILE_M) > max_mt) hdr->status = MOK_ERR_SCHEDULE;
        }
    }
    __syncthreads();
    if (e < E) {
        counts[e] = s_cnt[e];
        offsets[e] = s_off[e];
        pad_offsets[e] = s_pad[e];
        mt_start[e] = s_mt[e];
        if (counts_out) counts_out[e] = s_cnt[e];
        if (offsets_out) offsets_out[e] = s_off[e];
        for (int q = s_mt[e]; q < s_mt[e + 1] && q < max_mt; ++q) tile_expert[q] = e;
        mt_start2[e] = s_mt2[e];
        for (int q = s_mt2[e]; q < s_mt2[e + 1] && q < max_mt; ++q) tile_expert2[q] = e;
    }
    if (e == 0) {
        offsets[E] = s_off[E];
        pad_offsets[E] = s_pad[E];
        mt_start[E] = s_mt[E];
        mt_start2[E] = s_mt2[E];
        if (offsets_out) offsets_out[E] = s_off[E];
    }
}

}  // namespace mok
