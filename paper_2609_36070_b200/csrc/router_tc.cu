// Router projection on the tensor cores without giving up fp32 router weights (paper, Section 2.1; Figure 1
// right: the GPU-side router projection and top-k that precede the expert kernels).
//
// A plain bf16 GEMM would round W_r to 8 mantissa bits and move logits by ~2e-3, which changes the top-k of tokens
// that are nowhere near a tie.  Instead every fp32 weight is split exactly into three bf16 terms,
//     W_r = hi + mid + lo,   hi = bf16(W_r), mid = bf16(W_r - hi), lo = bf16(W_r - hi - mid),
// x is bf16 already, so all products are exact in fp32 and the tensor cores only add rounding in the fp32
// accumulation.  Four kernels (up to 160 experts kernels 2 and 3 are one: router_fused.cu):
//   1. router_split_kernel  W_r [E,H] fp32 -> [ldl, H] bf16 rows: hi (0..E-1), mid (E..2E-1), lo (2E..3E-1), zero pad
//   2. the tcgen05 GEMM     x [T,H] . split^T -> partial logits fp32 [T, ldl]
//   3. router_topk_kernel   logit = (lo + mid) + hi + bias, warp-shuffle top-k and softmax weights; tokens with a
//                           pair of candidates closer than the accumulation error are put on a list
//   4. router_fixup_kernel  the listed tokens (about 1 % of them) are re-decided with exact FMAs.  A kernel of its own,
//                           because one such token costs a warp ~10 us of dependent L2 round trips: inside kernel 3
//                           that latency was the kernel's duration
#include "mok_internal.cuh"
#include "router_common.cuh"

namespace mok {

// rows of `out`: part * estride + e for part = hi, mid, lo (estride >= E); every other row is zero
__global__ void __launch_bounds__(256)
router_split_kernel(const float* __restrict__ Wr, int E, int estride, int H, int rows, __nv_bfloat16* __restrict__ out,
                    WsHeader* hdr) {
    if (hdr && blockIdx.x == 0 && threadIdx.x == 0) hdr->n_flag = 0;   // the near-tie list of this call starts empty
    const size_t n = (size_t)rows * H;
    for (size_t i = (size_t)blockIdx.x * 256 + threadIdx.x; i < n; i += (size_t)gridDim.x * 256) {
        const int row = (int)(i / H), h = (int)(i - (size_t)row * H);
        const int part = row / estride, e = row - part * estride;
        float v = 0.f;
        if (part < 3 && e < E) {
            const float wv = Wr[(size_t)e * H + h];
            const float hi = __bfloat162float(__float2bfloat16_rn(wv));
            const float r1 = wv - hi;                                   // exact
            const float mid = __bfloat162float(__float2bfloat16_rn(r1));
            const float r2 = r1 - mid;                                  // exact
            v = (part == 0) ? hi : (part == 1) ? mid : r2;
        }
        out[i] = __float2bfloat16_rn(v);
    }
}

// Exact (fp32 FMA) logits of one token against up to four experts at once, computed by a whole warp: lanes stride
// over h in 16-byte pieces of x (read once for the four experts), then a shuffle tree per expert.  Four independent
// weight streams keep enough loads in flight to hide the L2 latency.  Error ~1e-7 relative, far below the near-tie
// threshold.
__device__ __forceinline__ void warp_exact_logits4(const __nv_bfloat16* __restrict__ xrow, const float* __restrict__ Wr,
                                                   const int (&e)[4], int n, int H, int lane, float (&out)[4]) {
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    const float* wrow[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) wrow[c] = Wr + (size_t)e[c < n ? c : 0] * H;
#pragma unroll 4
    for (int h = lane * 8; h < H; h += 256) {
        const uint4 raw = *reinterpret_cast<const uint4*>(xrow + h);
        const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&raw);
        const float2 x0 = __bfloat1622float2(p[0]), x1 = __bfloat1622float2(p[1]);
        const float2 x2 = __bfloat1622float2(p[2]), x3 = __bfloat1622float2(p[3]);
        float4 w0[4], w1[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            w0[c] = *reinterpret_cast<const float4*>(wrow[c] + h);
            w1[c] = *reinterpret_cast<const float4*>(wrow[c] + h + 4);
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            float a = acc[c];
            a = fmaf(x0.x, w0[c].x, a); a = fmaf(x0.y, w0[c].y, a);
            a = fmaf(x1.x, w0[c].z, a); a = fmaf(x1.y, w0[c].w, a);
            a = fmaf(x2.x, w1[c].x, a); a = fmaf(x2.y, w1[c].y, a);
            a = fmaf(x3.x, w1[c].z, a); a = fmaf(x3.y, w1[c].w, a);
            acc[c] = a;
        }
    }
#pragma unroll
    for (int c = 0; c < 4; ++c) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], off);
        out[c] = acc[c];
    }
}

// Monotone map from float to unsigned: a > b  <=>  key(a) > key(b) (finite inputs).
__device__ __forceinline__ unsigned float_key(float v) {
    const unsigned u = __float_as_uint(v);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Selection with the logits in registers: lane l holds experts l, l+32, ... (VPL per lane).  One round = every lane's
// best remaining value, a hardware warp max of the keys (redux.sync), and a warp min of the expert ids that attain it
// (ties go to the lowest id): two reductions instead of a ten-shuffle tree.
template <int VPL>
__device__ __forceinline__ void reg_select(float (&v)[VPL], int lane, int s_begin, int s_end, float& slot_v, int& slot_e) {
    for (int s = s_begin; s < s_end; ++s) {
        float bv = v[0];
        int bj = 0;
#pragma unroll
        for (int j = 1; j < VPL; ++j)
            if (v[j] > bv) { bv = v[j]; bj = j; }             // strict '>' keeps the lowest id on ties inside a lane
        const unsigned key = float_key(bv);
        const unsigned kmax = __reduce_max_sync(0xffffffffu, key);
        const int e_mine = (key == kmax) ? lane + 32 * bj : 0x7fffffff;
        const int e_win = __reduce_min_sync(0xffffffffu, e_mine);
        if (e_mine == e_win) {
#pragma unroll
            for (int j = 0; j < VPL; ++j)
                if (j == bj) v[j] = -FLT_MAX;                    // taken
        }
        const float v_win = __shfl_sync(0xffffffffu, bv, e_win & 31);
        if (lane == s) { slot_v = v_win; slot_e = e_win; }
    }
}

// The tensor cores add the 16 products of one MMA step to the fp32 accumulator with truncation, so the logit
// of a long dot product carries a small bias that grows with H (measured on B200: up to 4.5e-5 at H = 7168,
// against an fp64 evaluation).  That is harmless for the weights but could reorder two logits that are closer than
// the error.  So: tokens whose top-(k+1) tensor-core logits contain an adjacent pair closer than
//     guard = H * 2^-26 * (1 + max|logit|)      (four times the modelled bound (H/16) * 2^-24 * |acc|)
// get the logits of their top-(k+4) candidates recomputed with plain fp32 FMAs and are selected again.
template <int VPL>
__device__ __forceinline__ void load_logits(const float* __restrict__ row, const float* __restrict__ bias, int E, int lane,
                                            float (&v)[VPL], bool summed = false) {
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
        const int e = lane + 32 * j;
        float val = -FLT_MAX;
        if (e < E) {
            if (summed) {
                val = row[e];                                  // written by the fused kernel, bias included
            } else {
                val = (row[2 * E + e] + row[E + e]) + row[e];  // smallest terms first
                if (bias) val += bias[e];
            }
        }
        v[j] = val;
    }
}

template <int VPL>
__global__ void __launch_bounds__(256)
router_topk_kernel(const float* __restrict__ part, const float* __restrict__ bias, int T, int H, int E, int k, int ldl,
                   int32_t* __restrict__ idx, float* __restrict__ w, WsHeader* hdr, int32_t* __restrict__ flagged) {
    pdl_enter();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_check = (k + 1 < E) ? k + 1 : E;        // slots compared pairwise
    const float guard_scale = (float)H * 1.4901161e-8f; // H * 2^-26
    for (int t = blockIdx.x * 8 + warp; t < T; t += gridDim.x * 8) {
        float v[VPL];
        load_logits<VPL>(part + (size_t)t * ldl, bias, E, lane, v);
        TopkState st = {0u, 0.f, 0};
        reg_select<VPL>(v, lane, 0, n_check, st.v, st.e);
        const float next_v = __shfl_down_sync(0xffffffffu, st.v, 1);
        float amax = (lane < n_check) ? fabsf(st.v) : 0.f;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, off));
        const bool close = (lane + 1 < n_check) && (st.v - next_v < guard_scale * (1.f + amax));
        if (__any_sync(0xffffffffu, close) && lane == 0) flagged[atomicAdd(&hdr->n_flag, 1)] = t;
        warp_write_topk(st, k, lane, idx + (size_t)t * k, w + (size_t)t * k);   // provisional for a listed token
    }
}

// One block per listed token: the logits of its top-(k+4) candidates are recomputed with plain fp32 FMAs, then the
// top-k is selected again from all E logits and overwrites the provisional result.  There are few such tokens, so the
// kernel's duration is the latency of one of them: warp 0 selects, all eight warps share the candidates' dot products
// (each lane keeps many independent loads in flight), warp 0 selects again.  The list's order (atomic appends) does
// not matter: every token is decided on its own.
template <int VPL>
__global__ void __launch_bounds__(256)
router_fixup_kernel(const float* __restrict__ part, const float* __restrict__ bias,
                    const __nv_bfloat16* __restrict__ x, const float* __restrict__ Wr, int H, int E, int k, int ldl,
                    bool summed, int32_t* __restrict__ idx, float* __restrict__ w, const WsHeader* hdr,
                    const int32_t* __restrict__ flagged) {
    __shared__ int s_e[32];
    __shared__ float s_ex[32];
    pdl_enter();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int n_cand = (k + 4 < E) ? k + 4 : E;               // candidates recomputed
    if (n_cand > 32) n_cand = 32;
    const int n_flag = hdr->n_flag;
    for (int i = blockIdx.x; i < n_flag; i += gridDim.x) {
        const int t = flagged[i];
        float orig[VPL], v[VPL];
        TopkState st = {0u, 0.f, 0};
        if (warp == 0) {
            load_logits<VPL>(part + (size_t)t * ldl, bias, E, lane, orig, summed);
#pragma unroll
            for (int j = 0; j < VPL; ++j) v[j] = orig[j];
            reg_select<VPL>(v, lane, 0, n_cand, st.v, st.e);
            if (lane < n_cand) s_e[lane] = st.e;
        }
        __syncthreads();
        {   // warp w recomputes candidates w, w + 8, w + 16, w + 24
            int e[4], n = 0;
            float ex[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int ci = warp + 8 * c;
                e[c] = s_e[ci < n_cand ? ci : 0];
                if (ci < n_cand) n = c + 1;
            }
            if (n > 0) {
                warp_exact_logits4(x + (size_t)t * H, Wr, e, n, H, lane, ex);
                if (lane == 0) {
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        if (c < n) s_ex[warp + 8 * c] = ex[c];
                }
            }
        }
        __syncthreads();
        if (warp == 0) {
            for (int c = 0; c < n_cand; ++c) {
                const int ec = s_e[c];
                if ((ec & 31) == lane) {
                    const float val = s_ex[c] + (bias ? bias[ec] : 0.f);
#pragma unroll
                    for (int j = 0; j < VPL; ++j)
                        if (j == (ec >> 5)) orig[j] = val;
                }
            }
#pragma unroll
            for (int j = 0; j < VPL; ++j) v[j] = orig[j];
            reg_select<VPL>(v, lane, 0, k, st.v, st.e);
            warp_write_topk(st, k, lane, idx + (size_t)t * k, w + (size_t)t * k);
        }
        __syncthreads();                                // s_e / s_ex are reused by the next token
    }
}

template <int VPL>
static cudaError_t launch_topk(const float* part, const float* bias, const __nv_bfloat16* x, const float* Wr, int T, int H,
                               int E, int k, int ldl, bool fused, int32_t* idx, float* w, WsHeader* hdr, int32_t* flagged,
                               cudaStream_t s) {
    if (!fused) {
        int tblocks = (T + 7) / 8;
        if (tblocks > 148 * 16) tblocks = 148 * 16;
        cudaError_t e = launch_pdl(router_topk_kernel<VPL>, dim3(tblocks), dim3(256), 0, s, part, bias, T, H, E, k, ldl, idx, w,
                                   hdr, flagged);
        if (e != cudaSuccess) return e;
    }
    // one block per listed token; 8 blocks fit on an SM at once, and blocks beyond the list's length leave at once
    return launch_pdl(router_fixup_kernel<VPL>, dim3(148 * 8), dim3(256), 0, s, part, bias, x, Wr, H, E, k, ldl, fused, idx, w,
                      (const WsHeader*)hdr, (const int32_t*)flagged);
}

cudaError_t launch_router_tc(const __nv_bfloat16* x, const float* Wr, const float* bias, int T, int H, int E, int k,
                             const WsLayout& L, char* ws, WsHeader* hdr, int grid, int tile_m, int variant, bool fused,
                             int32_t* idx, float* w, cudaStream_t s, const __nv_bfloat16* presplit, bool split_only) {
    fused = fused && router_fused_ok(E, k);
    const int ep = (E + 31) / 32 * 32;
    const int ldl = fused ? ep : (3 * E + 7) / 8 * 8;       // row stride of the logits buffer
    const int split_rows = fused ? 3 * ep : ldl;
    // W_r is a weight: its split can be made once (mok_router_prepare) and handed in, or is made here on every call
    const __nv_bfloat16* split = presplit && !split_only ? presplit : reinterpret_cast<const __nv_bfloat16*>(ws + L.wr_split);
    float* part = reinterpret_cast<float*>(ws + L.logits);
    // the near-tie list lives in the schedule's `perm` region (T*k entries), which is not written before the schedule runs
    int32_t* flagged = reinterpret_cast<int32_t*>(ws + L.perm);
    size_t n = (size_t)split_rows * H;
    int blocks = (int)((n + 255) / 256);
    if (blocks > 148 * 8) blocks = 148 * 8;
    cudaError_t e = cudaSuccess;
    if (split_only) {     // mok_router_prepare: `presplit` is the destination, no workspace is involved
        router_split_kernel<<<blocks, 256, 0, s>>>(Wr, E, fused ? ep : E, H, split_rows, const_cast<__nv_bfloat16*>(presplit), nullptr);
        return cudaGetLastError();
    }
    if (!presplit) {
        router_split_kernel<<<blocks, 256, 0, s>>>(Wr, E, fused ? ep : E, H, split_rows,
                                                   reinterpret_cast<__nv_bfloat16*>(ws + L.wr_split), hdr);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    if (fused) {
        e = launch_router_fused(x, split, bias, T, H, E, k, part, flagged, hdr, grid, idx, w, s);
    } else {
        GemmArgs g = {};
        g.A = x;
        g.B = split;
        g.C = part;
        g.K = H; g.N = ldl; g.E = 1; g.ldc = ldl;
        g.rows_pad = L.Tpad; g.a_rows = T; g.dense_rows = T;
        g.max_mt = L.Tpad / TILE_M;
        g.tile_m = tile_m;
        g.dbg_slot = -1;
        g.header = hdr;
        // Few tokens give few tiles (T = 64 with 256 experts: three tiles of 128 x 256, each streaming a third of the split
        // weights through one SM): up to 16 row tiles the 128-row kernel runs with N tiles of 32 to 128 columns instead.  An
        // output element is the same accumulation over K whatever the tile width, so the logits keep their bits.
        const int row_tiles = (T + TILE_M - 1) / TILE_M;
        if (variant != 2 && tile_m == TILE_M && row_tiles <= 16) {
            g.n_tile = row_tiles <= 4 ? 32 : row_tiles <= 8 ? 64 : 128;
            variant = 0;
        }
        e = variant == 2 ? launch_gemm_tn(g, EPI_F32, grid, s)
            : variant == 3 ? launch_gemm_m2(g, EPI_F32, grid, s) : launch_gemm_tc(g, EPI_F32, grid, s);
    }
    if (e != cudaSuccess) return e;
    const int vpl = (E + 31) / 32;
    if (vpl <= 1) return launch_topk<1>(part, bias, x, Wr, T, H, E, k, ldl, fused, idx, w, hdr, flagged, s);
    if (vpl <= 2) return launch_topk<2>(part, bias, x, Wr, T, H, E, k, ldl, fused, idx, w, hdr, flagged, s);
    if (vpl <= 4) return launch_topk<4>(part, bias, x, Wr, T, H, E, k, ldl, fused, idx, w, hdr, flagged, s);
    if (vpl <= 8) return launch_topk<8>(part, bias, x, Wr, T, H, E, k, ldl, fused, idx, w, hdr, flagged, s);
    return launch_topk<16>(part, bias, x, Wr, T, H, E, k, ldl, fused, idx, w, hdr, flagged, s);
}

}  // namespace mok
