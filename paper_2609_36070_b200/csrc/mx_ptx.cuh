// PTX wrappers and scale arithmetic shared by the MXFP8 GEMM kernels (Section 3.4 "MXFP8 Support").
#pragma once
#include "mok_internal.cuh"
#include "tc_ptx.cuh"
#include <cuda_fp8.h>

namespace mok {
namespace mx {

// Instruction descriptor of the block-scaled MMA: A and B E4M3 (format 0), both K-major, scales E8M0; m = rows of the
// MMA (128, or 256 for a CTA pair), n = its columns; the two scale ids (which byte of the 4-byte scale cell a K = 32
// step uses) are set per instruction.
__device__ __forceinline__ constexpr uint32_t make_idesc_mx(int m, int n, uint32_t sf_id) {
    return (sf_id << 4) | ((uint32_t)(n >> 3) << 17) | (1u << 23) | ((uint32_t)(m >> 4) << 24) | (sf_id << 29);
}
// Shared-memory descriptor of one scale atom for tcgen05.cp: 32 rows of 16 bytes, no swizzle, 8-row groups 128
// bytes apart.
__device__ __forceinline__ uint64_t make_sf_desc(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(128 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    return d;
}
// Scale atom shared memory -> 4 tensor-memory columns, replicated over the four lane quadrants.  For a CTA pair the
// one instruction makes each CTA copy from its own shared memory (same offset) into its own tensor memory.
template <int CTAS>
__device__ __forceinline__ void tc_cp_sf(uint32_t taddr, uint64_t sdesc) {
    if (CTAS == 1) asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
    else asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
template <int CTAS>
__device__ __forceinline__ void tc_mma_mx(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t sfa_tmem, uint32_t sfb_tmem, uint32_t accumulate) {
    if (CTAS == 1) {
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.b32 p, %6, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%4], [%5], p;\n\t}"
            ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(sfa_tmem), "r"(sfb_tmem), "r"(accumulate) : "memory");
    } else {
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.b32 p, %6, 0;\n\t"
            "tcgen05.mma.cta_group::2.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%4], [%5], p;\n\t}"
            ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(sfa_tmem), "r"(sfb_tmem), "r"(accumulate) : "memory");
    }
}
// Plain (untiled) bulk copy global -> shared, completing on an mbarrier; both addresses 16-byte aligned.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void cp_async_4(uint32_t dst, const void* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}

// E8M0 code of a block's scale from its amax, and the factor 2^(127 - code) that maps the block onto the E4M3 grid.
__device__ __forceinline__ int scale_code(float amax) {
    int code = (int)((__float_as_uint(amax) >> 23) & 0xFFu) - 8;
    code = code < 0 ? 0 : code;
    return code > 254 ? 254 : code;
}
__device__ __forceinline__ float inv_scale(int code) {
    const int e = 254 - code;
    return e > 0 ? __uint_as_float((uint32_t)e << 23) : __uint_as_float(0x00400000u);
}

}  // namespace mx
}  // namespace mok
