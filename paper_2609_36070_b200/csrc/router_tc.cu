// Router projection on the tensor cores without giving up fp32 router weights (paper, Section 2.1; Figure 1
// right: the GPU-side router projection and top-k that precede the expert kernels).
//
// A plain bf16 GEMM would round W_r to 8 mantissa bits and move logits by ~2e-3, which changes the top-k of tokens
// that are nowhere near a tie.  Instead every fp32 weight is split exactly into three bf16 terms,
//     W_r = hi + mid + lo,   hi = bf16(W_r), mid = bf16(W_r - hi), lo = bf16(W_r - hi - mid),
// x is bf16 already, so all products are exact in fp32 and the tensor cores only add rounding in the fp32
// accumulation.  Three kernels:
//   1. router_split_kernel  W_r [E,H] fp32 -> [ldl, H] bf16 rows: hi (0..E-1), mid (E..2E-1), lo (2E..3E-1), zero pad
//   2. the tcgen05 GEMM     x [T,H] . split^T -> partial logits fp32 [T, ldl]
//   3. router_topk_kernel   logit = (lo + mid) + hi + bias, warp-shuffle top-k and softmax weights; tokens with a
//                           pair of candidates closer than the accumulation error are re-decided with exact FMAs
#include "mok_internal.cuh"
#include "router_common.cuh"

namespace mok {

__global__ void __launch_bounds__(256)
router_split_kernel(const float* __restrict__ Wr, int E, int H, int ldl, __nv_bfloat16* __restrict__ out) {
    const size_t n = (size_t)ldl * H;
    for (size_t i = (size_t)blockIdx.x * 256 + threadIdx.x; i < n; i += (size_t)gridDim.x * 256) {
        const int row = (int)(i / H), h = (int)(i - (size_t)row * H);
        float v = 0.f;
        if (row < 3 * E) {
            const int part = row / E, e = row - part * E;
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

// Exact (fp32 FMA) logit of one (token, expert) pair computed by a whole warp: lanes stride over h in 16-byte
// pieces, then a shuffle tree.  Error ~1e-7 relative, far below the near-tie threshold.
__device__ __forceinline__ float warp_exact_logit(const __nv_bfloat16* __restrict__ xrow, const float* __restrict__ wrow,
                                                  int H, int lane) {
    float acc = 0.f;
    for (int h = lane * 8; h < H; h += 256) {
        const uint4 raw = *reinterpret_cast<const uint4*>(xrow + h);
        const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&raw);
        const float4 w0 = *reinterpret_cast<const float4*>(wrow + h);
        const float4 w1 = *reinterpret_cast<const float4*>(wrow + h + 4);
        const float2 x0 = __bfloat1622float2(p[0]), x1 = __bfloat1622float2(p[1]);
        const float2 x2 = __bfloat1622float2(p[2]), x3 = __bfloat1622float2(p[3]);
        acc = fmaf(x0.x, w0.x, acc); acc = fmaf(x0.y, w0.y, acc);
        acc = fmaf(x1.x, w0.z, acc); acc = fmaf(x1.y, w0.w, acc);
        acc = fmaf(x2.x, w1.x, acc); acc = fmaf(x2.y, w1.y, acc);
        acc = fmaf(x3.x, w1.z, acc); acc = fmaf(x3.y, w1.w, acc);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    return acc;
}

// The tensor cores add the 16 products of one MMA step to the fp32 accumulator with truncation, so the logit
// of a long dot product carries a small bias that grows with H (measured on B200: up to 4.5e-5 at H = 7168,
// against an fp64 evaluation).  That is harmless for the weights but could reorder two logits that are closer than
// the error.  So: tokens whose top-(k+1) tensor-core logits contain an adjacent pair closer than
//     guard = H * 2^-26 * (1 + max|logit|)      (four times the modelled bound (H/16) * 2^-24 * |acc|)
// get the logits of their top-(k+4) candidates recomputed with plain fp32 FMAs and are selected again.
__global__ void __launch_bounds__(256)
router_topk_kernel(const float* __restrict__ part, const float* __restrict__ bias,
                   const __nv_bfloat16* __restrict__ x, const float* __restrict__ Wr,
                   int T, int H, int E, int k, int ldl, int32_t* __restrict__ idx, float* __restrict__ w) {
    extern __shared__ float tsm[];                      // [8][E]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float* lg = tsm + warp * E;
    const int n_check = (k + 1 < E) ? k + 1 : E;        // slots compared pairwise
    int n_cand = (k + 4 < E) ? k + 4 : E;               // candidates recomputed when a pair is too close
    if (n_cand > 32) n_cand = 32;
    const float guard_scale = (float)H * 1.4901161e-8f; // H * 2^-26
    for (int t = blockIdx.x * 8 + warp; t < T; t += gridDim.x * 8) {
        const float* row = part + (size_t)t * ldl;
        for (int e = lane; e < E; e += 32) {
            float v = (row[2 * E + e] + row[E + e]) + row[e];      // smallest terms first
            if (bias) v += bias[e];
            lg[e] = v;
        }
        __syncwarp();
        TopkState st = {0u, 0.f, 0};
        warp_select(lg, E, 0, n_check, lane, st);
        const float next_v = __shfl_down_sync(0xffffffffu, st.v, 1);
        float amax = (lane < n_check) ? fabsf(st.v) : 0.f;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, off));
        const bool close = (lane + 1 < n_check) && (st.v - next_v < guard_scale * (1.f + amax));
        if (__any_sync(0xffffffffu, close)) {
            warp_select(lg, E, n_check, n_cand, lane, st);
            for (int c = 0; c < n_cand; ++c) {
                const int e = __shfl_sync(0xffffffffu, st.e, c);
                float v = warp_exact_logit(x + (size_t)t * H, Wr + (size_t)e * H, H, lane);
                if (bias) v += bias[e];
                if (lane == 0) lg[e] = v;
            }
            __syncwarp();
            st.taken = 0u;
            warp_select(lg, E, 0, k, lane, st);
        }
        warp_write_topk(st, k, lane, idx + (size_t)t * k, w + (size_t)t * k);
        __syncwarp();
    }
}

cudaError_t launch_router_tc(const __nv_bfloat16* x, const float* Wr, const float* bias, int T, int H, int E, int k,
                             const WsLayout& L, char* ws, WsHeader* hdr, int grid, int tile_m, int32_t* idx, float* w,
                             cudaStream_t s) {
    const int ldl = (3 * E + 7) / 8 * 8;
    __nv_bfloat16* split = reinterpret_cast<__nv_bfloat16*>(ws + L.wr_split);
    float* part = reinterpret_cast<float*>(ws + L.logits);
    size_t n = (size_t)ldl * H;
    int blocks = (int)((n + 255) / 256);
    if (blocks > 148 * 8) blocks = 148 * 8;
    router_split_kernel<<<blocks, 256, 0, s>>>(Wr, E, H, ldl, split);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
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
    e = launch_gemm_tc(g, EPI_F32, grid, s);
    if (e != cudaSuccess) return e;
    int tblocks = (T + 7) / 8;
    if (tblocks > 148 * 16) tblocks = 148 * 16;
    router_topk_kernel<<<tblocks, 256, sizeof(float) * 8 * E, s>>>(part, bias, x, Wr, T, H, E, k, ldl, idx, w);
    return cudaGetLastError();
}

}  // namespace mok
