// MXFP8 quantisation (Section 3.4 "MXFP8 Support": weights are quantised ahead of time by a dedicated kernel,
// activations where they are produced).  Format of the microscaling paper the section cites: 32 consecutive
// elements along the contraction dimension share the scale X = 2^(floor(log2(amax)) - 8), stored as an E8M0 byte
// (exponent + 127); elements are v / X rounded to nearest-even on the FP8 E4M3 grid, magnitudes above 448 clamped.
//
// Inputs here are bf16, so amax, its exponent and v / X (a power-of-two scaling) are exact in fp32 and the codes
// are decided by one hardware conversion (cvt.rn.satfinite.e4m3x2.f32): the result is bit-reproducible.
//
// Scale layouts
//   row-major  : scales[row, kb], row stride padded to a multiple of 4 bytes (whole 128-element k-groups), pad = 127.
//                Used for the token rows, which the gate/up GEMM gathers one by one.
//   atoms      : the layout the block-scaled MMA consumes after a 32x128b.warpx4 shared -> tensor-memory copy: for
//                each (group, 128-row block, 128-element k-group) 512 bytes with the scale of (row r, block j of the
//                k-group) at (r % 32) * 16 + (r / 32) * 4 + j.  Rows / blocks outside the tensor hold 127 (= 1.0).
//                Used for the weights; a "group" is one [rows, K] matrix (an expert's gate, up or down projection).
#include "mok_internal.cuh"
#include <cuda_fp8.h>

namespace mok {

// E8M0 code of the block scale from the block's amax (fp32 bits): biased exponent - 8, clamped to [0, 254].
__device__ __forceinline__ int mx_scale_code(float amax) {
    const int field = (int)((__float_as_uint(amax) >> 23) & 0xFFu);
    int code = field - 8;
    code = code < 0 ? 0 : code;
    return code > 254 ? 254 : code;
}
// 2^(127 - code): the factor that maps values onto the E4M3 grid of a block with this scale code.
__device__ __forceinline__ float mx_inv_scale(int code) {
    const int e = 254 - code;                       // biased exponent of 2^(127 - code); 0 -> the subnormal 2^-127
    return e > 0 ? __uint_as_float((uint32_t)e << 23) : __uint_as_float(0x00400000u);
}

// One thread per 8 consecutive elements (16 bytes of bf16); the 4 threads of a 32-element block share the amax with
// two shuffles.  Each block of 256 threads walks whole rows (blockIdx.x, then grid stride), so no index is ever
// divided.  rows x K, K a multiple of 32.  Writes codes[rows, K] and the scales in the requested layout.
template <bool ATOMS>
__global__ void __launch_bounds__(256)
mx_quantize_kernel(const __nv_bfloat16* __restrict__ in, long long rows, int K, int rows_per_group,
                   uint8_t* __restrict__ codes, uint8_t* __restrict__ scales, int scale_stride) {
    const int chunks = K >> 3;                      // 8-element chunks per row (a multiple of 4)
    const int KG = (K + 127) / 128, NB = (rows_per_group + 127) / 128;
    const int rows_per_iter = ATOMS ? 1 : 4;        // token rows are short: four per block iteration
    for (long long row0 = (long long)blockIdx.x * rows_per_iter; row0 < rows; row0 += (long long)gridDim.x * rows_per_iter) {
        const int n_here = (int)min((long long)rows_per_iter, rows - row0);
        for (int i = threadIdx.x; i < ((n_here * chunks + 31) & ~31); i += 256) {
            const bool live = i < n_here * chunks;
            const int rsub = live ? i / chunks : 0;
            const long long row = row0 + rsub;
            const int c = live ? i - rsub * chunks : 0;
            uint4 raw = make_uint4(0u, 0u, 0u, 0u);
            if (live) raw = __ldg(reinterpret_cast<const uint4*>(in + row * K + c * 8));
            const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
            float v[8];
            float amax = 0.f;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float2 f = __bfloat1622float2(p2[q]);
                v[2 * q] = f.x;
                v[2 * q + 1] = f.y;
                amax = fmaxf(amax, fmaxf(fabsf(f.x), fabsf(f.y)));
            }
            amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
            amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
            if (!live) continue;
            const int code = mx_scale_code(amax);
            const float inv = mx_inv_scale(code);
            uint32_t out[2];
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2(v[4 * q] * inv, v[4 * q + 1] * inv), __NV_SATFINITE, __NV_E4M3);
                const uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2(v[4 * q + 2] * inv, v[4 * q + 3] * inv), __NV_SATFINITE, __NV_E4M3);
                out[q] = lo | (hi << 16);
            }
            *reinterpret_cast<uint2*>(codes + row * K + c * 8) = make_uint2(out[0], out[1]);
            if ((c & 3) == 0) {
                const int kb = c >> 2;              // 32-element block index along K
                if (ATOMS) {
                    const long long g = row / rows_per_group;
                    const int r = (int)(row - g * rows_per_group);
                    const size_t atom = ((size_t)(g * NB + (r >> 7)) * KG + (kb >> 2)) * 512;
                    scales[atom + (r & 31) * 16 + ((r & 127) >> 5) * 4 + (kb & 3)] = (uint8_t)code;
                } else {
                    scales[row * scale_stride + kb] = (uint8_t)code;
                }
            }
        }
    }
}

cudaError_t launch_mx_quantize_rows(const __nv_bfloat16* in, long long rows, int K, uint8_t* codes, uint8_t* scales,
                                    cudaStream_t s) {
    const int stride = (K + 127) / 128 * 4;
    cudaError_t e = cudaMemsetAsync(scales, 127, (size_t)rows * stride, s);
    if (e != cudaSuccess) return e;
    long long blocks = (rows + 3) / 4;
    if (blocks > 148 * 8) blocks = 148 * 8;
    if (blocks < 1) blocks = 1;
    mx_quantize_kernel<false><<<(int)blocks, 256, 0, s>>>(in, rows, K, 1, codes, scales, stride);
    return cudaGetLastError();
}

cudaError_t launch_mx_quantize_atoms(const __nv_bfloat16* in, int groups, int rows_per_group, int K, uint8_t* codes,
                                     uint8_t* scales, cudaStream_t s) {
    const size_t atoms = (size_t)groups * ((rows_per_group + 127) / 128) * ((K + 127) / 128);
    cudaError_t e = cudaMemsetAsync(scales, 127, atoms * 512, s);
    if (e != cudaSuccess) return e;
    const long long rows = (long long)groups * rows_per_group;
    long long blocks = rows;
    if (blocks > 148 * 16) blocks = 148 * 16;
    if (blocks < 1) blocks = 1;
    mx_quantize_kernel<true><<<(int)blocks, 256, 0, s>>>(in, rows, K, rows_per_group, codes, scales, 0);
    return cudaGetLastError();
}

}  // namespace mok
