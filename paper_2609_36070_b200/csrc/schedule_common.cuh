// Pieces shared by the one-rank and the R-rank schedule kernels (Algorithm 1): block geometry and the step that
// turns per-expert row counts into offsets and the GEMMs' internal tile tables.
#pragma once
#include "mok_internal.cuh"

namespace mok {

constexpr int SCHED_THREADS = 256;
constexpr int SCHED_WARPS = SCHED_THREADS / 32;
constexpr int ROUTES_PER_WARP = SCHED_CHUNK / SCHED_WARPS;   // contiguous routes owned by one warp

// Called by every thread of a block of at least E threads after s_cnt[0..E) is complete and the block has
// synchronised.  S_l (offsets) is the exclusive prefix sum of the counts (Algorithm 1); each expert's segment of the
// padded row space starts at a multiple of pad_m rows and is cut into tiles of tile_m and of 2*tile_m rows.
__device__ __forceinline__ void scan_tables(const int32_t* s_cnt, int32_t* s_off, int32_t* s_mt, int32_t* s_pad,
                                            int32_t* s_mt2, int E, int max_mt, int tile_m, int pad_m,
                                            int32_t* __restrict__ counts, int32_t* __restrict__ offsets,
                                            int32_t* __restrict__ pad_offsets, int32_t* __restrict__ mt_start,
                                            int32_t* __restrict__ tile_expert, int32_t* __restrict__ mt_start2,
                                            int32_t* __restrict__ tile_expert2, WsHeader* __restrict__ hdr,
                                            int32_t* __restrict__ counts_out, int32_t* __restrict__ offsets_out) {
    const int e = threadIdx.x;
    if (e == 0) {   // E <= 512: a serial scan by one thread is a few hundred cycles
        int32_t off = 0, mt = 0, pad = 0, mt2 = 0;
        for (int i = 0; i < E; ++i) {
            s_off[i] = off;
            s_mt[i] = mt;
            s_mt2[i] = mt2;
            s_pad[i] = pad;
            off += s_cnt[i];
            mt += (s_cnt[i] + tile_m - 1) / tile_m;
            mt2 += (s_cnt[i] + 2 * tile_m - 1) / (2 * tile_m);
            pad += (s_cnt[i] + pad_m - 1) / pad_m * pad_m;
        }
        s_off[E] = off;
        s_mt[E] = mt;
        s_pad[E] = pad;
        s_mt2[E] = mt2;
        hdr->n_mtiles = mt;
        hdr->n_mtiles2 = mt2;
        if (mt * (tile_m / TILE_M) > max_mt) hdr->status = MOK_ERR_SCHEDULE;
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
