// Router projection, top-k selection and normalised weights (paper, Section 2.1; Figure 1 right: the
// GPU-side routing step that runs before the expert kernels).
//
//   logit[t,e] = sum_h x[t,h] * W_r[e,h] (+ bias[e])      fp32 accumulation, W_r kept in fp32
//   idx[t,0..k) = the k largest logits, ordered by (logit desc, expert id asc)
//   w[t,s]      = softmax over all E restricted to the selection and renormalised
//               = exp(l_s - l_0) / sum_s' exp(l_s' - l_0)   over the selected logits (same number)
//
// This file holds the fp32 FMA version: a 64-token x 64-expert shared-memory tiled product that leaves
// the block's logits in shared memory, followed by a warp-shuffle top-k (one warp per token).
#include "mok_internal.cuh"
#include "router_common.cuh"

namespace mok {

constexpr int RT_TOK = 64;   // tokens per block
constexpr int RT_EXP = 64;   // experts per pass
constexpr int RT_KC = 32;    // hidden-dimension chunk

__global__ void __launch_bounds__(256)
router_simt_kernel(const __nv_bfloat16* __restrict__ x, const float* __restrict__ Wr, const float* __restrict__ bias,
                   int T, int H, int E, int k, int32_t* __restrict__ idx, float* __restrict__ w) {
    extern __shared__ float rsm[];
    float* sx = rsm;                          // [RT_KC][RT_TOK]
    float* sw = sx + RT_KC * RT_TOK;          // [RT_KC][RT_EXP]
    float* slog = sw + RT_KC * RT_EXP;        // [RT_TOK][ldl]
    const int ldl = E + 1;
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int tok0 = blockIdx.x * RT_TOK;
    const int lrow = tid >> 2, lcol = (tid & 3) * 8;

    for (int e0 = 0; e0 < E; e0 += RT_EXP) {
        float acc[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
        for (int k0 = 0; k0 < H; k0 += RT_KC) {
            {   // x tile: 64 tokens x 32 hidden values, 8 bf16 (16 bytes) per thread
                float v[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) v[i] = 0.f;
                int t = tok0 + lrow;
                if (t < T && k0 + lcol < H) {
                    uint4 raw = *reinterpret_cast<const uint4*>(x + (size_t)t * H + k0 + lcol);
                    const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        float2 f = __bfloat1622float2(p[i]);
                        v[2 * i] = f.x;
                        v[2 * i + 1] = f.y;
                    }
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) sx[(lcol + i) * RT_TOK + lrow] = v[i];
            }
            {   // W_r tile: 64 experts x 32 hidden values, 8 floats per thread
                float v[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) v[i] = 0.f;
                int e = e0 + lrow;
                if (e < E && k0 + lcol < H) {
                    const float4* p = reinterpret_cast<const float4*>(Wr + (size_t)e * H + k0 + lcol);
                    float4 a = p[0], b = p[1];
                    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
                    v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) sw[(lcol + i) * RT_EXP + lrow] = v[i];
            }
            __syncthreads();
#pragma unroll
            for (int kk = 0; kk < RT_KC; ++kk) {
                float4 a = *reinterpret_cast<const float4*>(sx + kk * RT_TOK + ty * 4);
                float4 b = *reinterpret_cast<const float4*>(sw + kk * RT_EXP + tx * 4);
                const float av[4] = {a.x, a.y, a.z, a.w};
                const float bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
            }
            __syncthreads();
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                int e = e0 + tx * 4 + j;
                if (e < E) slog[(ty * 4 + i) * ldl + e] = acc[i][j] + (bias ? bias[e] : 0.f);
            }
    }
    __syncthreads();
    const int warp = tid >> 5, lane = tid & 31;
    for (int r = warp; r < RT_TOK; r += 8) {
        int t = tok0 + r;
        if (t < T) warp_topk_softmax(slog + r * ldl, E, k, lane, idx + (size_t)t * k, w + (size_t)t * k);
    }
}

cudaError_t launch_router_simt(const __nv_bfloat16* x, const float* Wr, const float* bias, int T, int H, int E, int k,
                               int32_t* idx, float* w, cudaStream_t s) {
    size_t smem = sizeof(float) * (RT_KC * RT_TOK + RT_KC * RT_EXP + (size_t)RT_TOK * (E + 1));
    cudaError_t err = cudaFuncSetAttribute(router_simt_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    router_simt_kernel<<<(T + RT_TOK - 1) / RT_TOK, 256, smem, s>>>(x, Wr, bias, T, H, E, k, idx, w);
    return cudaGetLastError();
}

}  // namespace mok
