// Warp-level top-k selection and normalised router weights shared by the two router implementations
// (paper, Section 2.1: the router picks each token's k experts and gives each pick a weight).
#pragma once
#include <cuda_runtime.h>
#include <float.h>
#include <stdint.h>

namespace mok {

// Selection state of one warp working on one token: lane l remembers which of its experts (l, l+32, ...) are
// already taken, and lane s holds the logit and expert id of slot s.
struct TopkState {
    uint32_t taken;
    float v;
    int e;
};

// Fills slots [s_begin, s_end) with the next largest logits of lg[0..E), ordered by (logit desc, expert id asc).
__device__ __forceinline__ void warp_select(const float* __restrict__ lg, int E, int s_begin, int s_end, int lane,
                                            TopkState& st) {
    for (int s = s_begin; s < s_end; ++s) {
        float bv = -FLT_MAX;
        int be = 0x7fffffff;
        for (int j = 0, e = lane; e < E; ++j, e += 32) {
            if ((st.taken >> j) & 1u) continue;
            float v = lg[e];
            if (v > bv || be == 0x7fffffff) { bv = v; be = e; }   // ascending e + strict '>' keeps the lowest id on ties
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            float ov = __shfl_xor_sync(0xffffffffu, bv, off);
            int oe = __shfl_xor_sync(0xffffffffu, be, off);
            if (oe != 0x7fffffff && (be == 0x7fffffff || ov > bv || (ov == bv && oe < be))) { bv = ov; be = oe; }
        }
        if ((be & 31) == lane) st.taken |= 1u << (be >> 5);
        if (lane == s) { st.v = bv; st.e = be; }
    }
}

// w[s] = exp(l_s - l_0) / sum_s' exp(l_s' - l_0) over the k selected logits: the softmax over all E experts
// restricted to the selection and renormalised (the two are the same number).
__device__ __forceinline__ void warp_write_topk(const TopkState& st, int k, int lane,
                                                int32_t* __restrict__ idx_out, float* __restrict__ w_out) {
    float v0 = __shfl_sync(0xffffffffu, st.v, 0);
    float ex = (lane < k) ? expf(st.v - v0) : 0.f;
    float sum = ex;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
    if (lane < k) {
        idx_out[lane] = st.e;
        w_out[lane] = ex / sum;
    }
}

// One warp selects the top-k of `E` logits in shared memory and writes idx / w for one token.
__device__ __forceinline__ void warp_topk_softmax(const float* __restrict__ lg, int E, int k, int lane,
                                                  int32_t* __restrict__ idx_out, float* __restrict__ w_out) {
    TopkState st = {0u, 0.f, 0};
    warp_select(lg, E, 0, k, lane, st);
    warp_write_topk(st, k, lane, idx_out, w_out);
}

}  // namespace mok
