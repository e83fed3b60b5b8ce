// Token gather ("pull dispatch") and deterministic weighted combine ("push combine" + router-weighted sum)
// for one GPU, where the paper's remote loads/stores (Section 3.1) become HBM row copies.
//
//   gather : Xg[p,:] = x[perm[...] / k, :] for every row p of the padded expert-sorted buffer (pad rows = 0)
//   combine: out[t,:] = ysh[t,:] + sum_{s=0}^{k-1} w[t,s] * y[pos[t*k+s], :]
//            fp32 FMA chain in slot order, one rounding to bf16, no atomics => bitwise reproducible
//            (Section 3.4 "Determinism": a temporary buffer reduced by another worker in a fixed order).
// Both are HBM-bound: 128-bit accesses, one warp (gather) or one block (combine) per row.
#include "mok_internal.cuh"

namespace mok {

__global__ void __launch_bounds__(256)
gather_kernel(const __nv_bfloat16* __restrict__ x, int H, int k, int tile_m,
              const WsHeader* __restrict__ hdr, const int32_t* __restrict__ tile_expert,
              const int32_t* __restrict__ pad_offsets, const int32_t* __restrict__ offsets,
              const int32_t* __restrict__ counts, const int32_t* __restrict__ perm,
              __nv_bfloat16* __restrict__ xg) {
    const int lane = threadIdx.x & 31;
    const int rows = hdr->n_mtiles * tile_m;
    const int chunks = H >> 3;
    for (int p = blockIdx.x * 8 + (threadIdx.x >> 5); p < rows; p += gridDim.x * 8) {
        const int e = tile_expert[p / tile_m];
        const int local = p - pad_offsets[e];
        uint4* dst = reinterpret_cast<uint4*>(xg + (size_t)p * H);
        if (local < counts[e]) {
            const int t = perm[offsets[e] + local] / k;
            const uint4* src = reinterpret_cast<const uint4*>(x + (size_t)t * H);
            for (int c = lane; c < chunks; c += 32) dst[c] = __ldg(src + c);
        } else {
            for (int c = lane; c < chunks; c += 32) dst[c] = make_uint4(0u, 0u, 0u, 0u);
        }
    }
}

__global__ void __launch_bounds__(128)
combine_kernel(const __nv_bfloat16* __restrict__ y, const __nv_bfloat16* __restrict__ ysh,
               const int32_t* __restrict__ pos, const float* __restrict__ w,
               int T, int H, int k, __nv_bfloat16* __restrict__ out) {
    __shared__ int32_t s_pos[MAX_K];
    __shared__ float s_w[MAX_K];
    pdl_enter();
    const int t = blockIdx.x;
    if (threadIdx.x < k) {
        s_pos[threadIdx.x] = pos[(size_t)t * k + threadIdx.x];
        s_w[threadIdx.x] = w ? w[(size_t)t * k + threadIdx.x] : 1.f;   // w == NULL: plain sum (backward pass)
    }
    __syncthreads();
    const int chunks = H >> 3;
    for (int c = threadIdx.x; c < chunks; c += 128) {
        float acc[8];
        if (ysh) {
            uint4 raw = *reinterpret_cast<const uint4*>(ysh + (size_t)t * H + c * 8);
            const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float2 f = __bfloat1622float2(p2[i]);
                acc[2 * i] = f.x;
                acc[2 * i + 1] = f.y;
            }
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] = 0.f;
        }
#pragma unroll 4
        for (int s = 0; s < k; ++s) {
            uint4 raw = *reinterpret_cast<const uint4*>(y + (size_t)s_pos[s] * H + c * 8);
            const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
            const float ws = s_w[s];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float2 f = __bfloat1622float2(p2[i]);
                acc[2 * i] = fmaf(ws, f.x, acc[2 * i]);
                acc[2 * i + 1] = fmaf(ws, f.y, acc[2 * i + 1]);
            }
        }
        uint4 o;
        __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
        for (int i = 0; i < 4; ++i) o2[i] = __floats2bfloat162_rn(acc[2 * i], acc[2 * i + 1]);
        *reinterpret_cast<uint4*>(out + (size_t)t * H + c * 8) = o;
    }
}

cudaError_t launch_gather(const __nv_bfloat16* x, int H, int k, int tile_m, const WsLayout& L, char* ws, cudaStream_t s,
                          __nv_bfloat16* dst) {
    int blocks = (L.Rpad + 7) / 8;
    if (blocks > 148 * 64) blocks = 148 * 64;
    gather_kernel<<<blocks, 256, 0, s>>>(x, H, k, tile_m, reinterpret_cast<const WsHeader*>(ws + L.header),
                                         reinterpret_cast<const int32_t*>(ws + L.tile_expert),
                                         reinterpret_cast<const int32_t*>(ws + L.pad_offsets),
                                         reinterpret_cast<const int32_t*>(ws + L.offsets),
                                         reinterpret_cast<const int32_t*>(ws + L.counts),
                                         reinterpret_cast<const int32_t*>(ws + L.perm),
                                         dst ? dst : reinterpret_cast<__nv_bfloat16*>(ws + L.xg));
    return cudaGetLastError();
}

cudaError_t launch_combine(const WsLayout& L, char* ws, int T, int H, int k, bool shared, __nv_bfloat16* out,
                           cudaStream_t s, bool unit_weights) {
    return launch_pdl(combine_kernel, dim3(T), dim3(128), 0, s, reinterpret_cast<const __nv_bfloat16*>(ws + L.y),
                      shared ? reinterpret_cast<const __nv_bfloat16*>(ws + L.ysh) : (const __nv_bfloat16*)nullptr,
                      reinterpret_cast<const int32_t*>(ws + L.pos),
                      unit_weights ? (const float*)nullptr : reinterpret_cast<const float*>(ws + L.w), T, H, k, out);
}

}  // namespace mok
