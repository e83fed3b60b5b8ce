// Plain shared-memory FMA version of the grouped expert GEMMs (paper, Section 2.1: gate/up projection with
// gated activation, and down projection).  Slow by design: it is the on-device cross-check of the tcgen05
// kernel and shares only the argument block with it.
//   SWIGLU : C[r, c] = silu(A[r,:] . Bgate[e][c,:]) * (A[r,:] . Bup[e][c,:])      B = [E, 2N, K]
//   else   : C[r, c] = A[r,:] . B[e][c,:]                                         B = [E,  N, K]
// bf16 operands, fp32 accumulation in ascending k, bf16 result.
#include "mok_internal.cuh"

namespace mok {

template <bool SWIGLU>
__global__ void __launch_bounds__(256) gemm_simt_kernel(GemmArgs a) {
    __shared__ __align__(16) float As[16][64];
    __shared__ __align__(16) float Bg[16][64];
    __shared__ __align__(16) float Bu[SWIGLU ? 16 : 1][64];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int r0 = blockIdx.y * 64, c0 = blockIdx.x * 64;
    const int n_rows = (a.dense_rows > 0) ? (a.dense_rows + TILE_M - 1) / TILE_M * TILE_M : *a.n_mtiles * a.tile_m;
    if (r0 >= n_rows) return;
    const int e = (a.dense_rows > 0) ? 0 : a.tile_expert[r0 / a.tile_m];
    const size_t brow0 = (size_t)e * (SWIGLU ? 2 : 1) * a.N;
    const int lrow = tid >> 2, lk = (tid & 3) * 4;

    float accg[4][4], accu[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) { accg[i][j] = 0.f; accu[i][j] = 0.f; }

    for (int k0 = 0; k0 < a.K; k0 += 16) {
        const bool kok = (k0 + lk) < a.K;
        {
            float v[4] = {0.f, 0.f, 0.f, 0.f};
            if (kok && r0 + lrow < a.a_rows) {
                uint2 raw = *reinterpret_cast<const uint2*>(a.A + (size_t)(r0 + lrow) * a.K + k0 + lk);
                const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&raw);
                float2 f0 = __bfloat1622float2(p[0]), f1 = __bfloat1622float2(p[1]);
                v[0] = f0.x; v[1] = f0.y; v[2] = f1.x; v[3] = f1.y;
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) As[lk + i][lrow] = v[i];
        }
        {
            float v[4] = {0.f, 0.f, 0.f, 0.f}, u[4] = {0.f, 0.f, 0.f, 0.f};
            const int c = c0 + lrow;
            if (kok && c < a.N) {
                uint2 raw = *reinterpret_cast<const uint2*>(a.B + (brow0 + c) * a.K + k0 + lk);
                const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&raw);
                float2 f0 = __bfloat1622float2(p[0]), f1 = __bfloat1622float2(p[1]);
                v[0] = f0.x; v[1] = f0.y; v[2] = f1.x; v[3] = f1.y;
                if (SWIGLU) {
                    uint2 raw2 = *reinterpret_cast<const uint2*>(a.B + (brow0 + a.N + c) * a.K + k0 + lk);
                    const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&raw2);
                    float2 g0 = __bfloat1622float2(p2[0]), g1 = __bfloat1622float2(p2[1]);
                    u[0] = g0.x; u[1] = g0.y; u[2] = g1.x; u[3] = g1.y;
                }
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                Bg[lk + i][lrow] = v[i];
                if (SWIGLU) Bu[lk + i][lrow] = u[i];
            }
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
            float4 av4 = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
            float4 bg4 = *reinterpret_cast<const float4*>(&Bg[kk][tx * 4]);
            const float av[4] = {av4.x, av4.y, av4.z, av4.w};
            const float bg[4] = {bg4.x, bg4.y, bg4.z, bg4.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) accg[i][j] = fmaf(av[i], bg[j], accg[i][j]);
            if (SWIGLU) {
                float4 bu4 = *reinterpret_cast<const float4*>(&Bu[kk][tx * 4]);
                const float bu[4] = {bu4.x, bu4.y, bu4.z, bu4.w};
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) accu[i][j] = fmaf(av[i], bu[j], accu[i][j]);
            }
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = c0 + tx * 4 + j;
            if (c >= a.N) continue;
            float v = accg[i][j];
            if (SWIGLU) v = (v / (1.f + expf(-v))) * accu[i][j];
            reinterpret_cast<__nv_bfloat16*>(a.C)[(size_t)(r0 + ty * 4 + i) * a.ldc + c] = __float2bfloat16_rn(v);
        }
}

cudaError_t launch_gemm_simt(const GemmArgs& a, bool swiglu, cudaStream_t s) {
    const int mt = (a.dense_rows > 0) ? (a.dense_rows + TILE_M - 1) / TILE_M : a.max_mt;
    dim3 grid((a.N + 63) / 64, mt * 2);
    if (swiglu) gemm_simt_kernel<true><<<grid, 256, 0, s>>>(a);
    else gemm_simt_kernel<false><<<grid, 256, 0, s>>>(a);
    return cudaGetLastError();
}

}  // namespace mok
