// Router projection, top-k and router weights in ONE tcgen05 kernel (paper, Section 2.1; Figure 1 right: the GPU-side
// router that precedes the expert kernels), for up to 160 experts.
//
// As in the three-kernel tensor-core router the fp32 router weights are split exactly into three bf16 terms
// (hi + mid + lo), so every product with the bf16 activations is exact in fp32.  Here the three partial logits of a
// 128-token tile stay in tensor memory (3 x EP fp32 columns, EP = E rounded up to 32, 3 EP <= 512) and the epilogue
// selects straight from there: thread = token row, logit = (lo + mid) + hi + bias in registers, k + 1 rounds of
// "largest remaining logit, lowest expert id on ties", softmax weights over the selection.  Nothing but idx and w goes
// back to HBM (the three-kernel path writes and re-reads 12 E bytes per token and takes one launch more).
// Tokens whose top-(k+1) logits contain a pair closer than the tensor cores' accumulation error are listed, with their
// logits, for the exact fix-up kernel, exactly as in the three-kernel path; the logits, the selection and the weights
// are bit-identical to that path's.
//
// Warp 0: TMA producer (128 x 64 tile of x, 3 EP x 64 tile of the split weights per stage), warp 1: MMA issuer (M = 128,
// N = 3 EP as one or two instructions), warps 2..5: epilogue.  One accumulator: while the epilogue selects, the next
// tile's MMAs already run (the accumulator is handed back as soon as it has been read into registers).
#include <float.h>
#include "mok_internal.cuh"
#include "tc_ptx.cuh"
#include "tensor_map.cuh"

namespace mok {
namespace rf {

using namespace tc;

constexpr int BM = 128, BK = 64, UMMA_K = 16;
constexpr int A_BYTES = BM * BK * 2;
constexpr int MAX_STAGES = 4;
constexpr int THREADS = 192;
constexpr int SMEM_CTRL = 1024;         // control block (256 bytes) + the router bias (up to 160 floats)
constexpr int SMEM_LIMIT = 232448;

struct Ctrl {
    uint64_t full[MAX_STAGES], empty[MAX_STAGES];
    uint64_t tfull, tempty;
    uint32_t tmem_base, abort;
};
static_assert(sizeof(Ctrl) <= 256, "control block too large");

struct Args {
    const float* bias;      // [E] or NULL
    int32_t* idx;           // [T, k]
    float* w;               // [T, k]
    float* rows;            // [T, EP]: logits of listed tokens (bias included)
    int32_t* flagged;       // near-tie list
    WsHeader* hdr;
    int32_t T, H, E, k, stages, n_tiles, k_blocks;
    uint32_t tmem_cols;
};

// 32 lanes x 16 consecutive fp32 columns
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}

// Monotone map from float to unsigned (a > b <=> key(a) > key(b), finite inputs) and its inverse.
__device__ __forceinline__ unsigned float_key(float v) {
    const unsigned u = __float_as_uint(v);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_float(unsigned key) {
    return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

__device__ __forceinline__ uint32_t idesc_n(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

template <int NJ>
__global__ void __launch_bounds__(THREADS, 1)
router_fused_kernel(const __grid_constant__ CUtensorMap tmapA, const __grid_constant__ CUtensorMap tmapB,
                    const __grid_constant__ Args a) {
    constexpr int EP = 32 * NJ;
    constexpr int B_BYTES = 3 * EP * BK * 2;
    constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    constexpr int N1 = (3 * EP > 256) ? 256 : 3 * EP, N2 = 3 * EP - N1;
    extern __shared__ uint8_t smem_raw[];
    pdl_enter();
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem + a.stages * STAGE_BYTES);
    float* s_bias = reinterpret_cast<float*>(smem + a.stages * STAGE_BYTES + 256);
    volatile uint32_t* abort_flag = &ctrl->abort;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int stages = a.stages;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(smem_u32(&ctrl->full[s]), 1);
            mbar_init(smem_u32(&ctrl->empty[s]), 1);
        }
        mbar_init(smem_u32(&ctrl->tfull), 1);
        mbar_init(smem_u32(&ctrl->tempty), 4);
        ctrl->abort = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (a.bias && threadIdx.x >= 64 && threadIdx.x - 64 < EP) s_bias[threadIdx.x - 64] = (threadIdx.x - 64 < a.E) ? a.bias[threadIdx.x - 64] : 0.f;
    if (EP > 128 && a.bias && threadIdx.x < EP - 128) s_bias[128 + threadIdx.x] = (128 + threadIdx.x < a.E) ? a.bias[128 + threadIdx.x] : 0.f;
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&ctrl->tmem_base)), "r"(a.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctrl->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < a.n_tiles && ok; tile += gridDim.x) {
                for (int kb = 0; kb < a.k_blocks; ++kb) {
                    ok = mbar_wait(smem_u32(&ctrl->empty[s]), ph ^ 1u, abort_flag, a.hdr, 21);
                    if (!ok) break;
                    const uint32_t full = smem_u32(&ctrl->full[s]);
                    const uint32_t sa = base + s * STAGE_BYTES, sb = sa + A_BYTES;
                    mbar_expect_tx(full, STAGE_BYTES);
                    tma_load_2d(sa, &tmapA, full, kb * BK, tile * BM);
#pragma unroll
                    for (int p = 0; p < 3; ++p) tma_load_2d(sb + p * (EP * BK * 2), &tmapB, full, kb * BK, p * EP);
                    if (++s == stages) { s = 0; ph ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0, aph = 0;
            const uint32_t id1 = idesc_n(N1), id2 = idesc_n(N2 > 0 ? N2 : 16);
            bool ok = true;
            for (int tile = blockIdx.x; tile < a.n_tiles && ok; tile += gridDim.x) {
                ok = mbar_wait(smem_u32(&ctrl->tempty), aph ^ 1u, abort_flag, a.hdr, 22);
                if (!ok) break;
                tc_fence_after();
                for (int kb = 0; kb < a.k_blocks; ++kb) {
                    ok = mbar_wait(smem_u32(&ctrl->full[s]), ph, abort_flag, a.hdr, 23);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t sa = base + s * STAGE_BYTES, sb = sa + A_BYTES;
                    const uint64_t ad = make_smem_desc(sa), b1 = make_smem_desc(sb), b2 = make_smem_desc(sb + N1 * BK * 2);
#pragma unroll
                    for (int j = 0; j < BK / UMMA_K; ++j) {
                        tc_mma<1>(tmem_base, ad + (uint64_t)(j * 2), b1 + (uint64_t)(j * 2), id1, (kb | j) ? 1u : 0u);
                        if (N2 > 0)
                            tc_mma<1>(tmem_base + N1, ad + (uint64_t)(j * 2), b2 + (uint64_t)(j * 2), id2, (kb | j) ? 1u : 0u);
                    }
                    tc_commit<1>(smem_u32(&ctrl->empty[s]));
                    if (++s == stages) { s = 0; ph ^= 1u; }
                }
                if (!ok) break;
                tc_commit<1>(smem_u32(&ctrl->tfull));
                aph ^= 1u;
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue: thread = token row
        const int quad = warp & 3;
        const int E = a.E, k = a.k;
        const int n_check = (k + 1 < E) ? k + 1 : E;
        const float guard_scale = (float)a.H * 1.4901161e-8f;   // H * 2^-26, as in the three-kernel path
        uint32_t aph = 0;
        for (int tile = blockIdx.x; tile < a.n_tiles; tile += gridDim.x) {
            bool ok = mbar_wait(smem_u32(&ctrl->tfull), aph, abort_flag, a.hdr, 24);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            aph ^= 1u;
            __syncwarp();                                 // lanes past the last token took a shorter way round
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16);
            unsigned key[EP];                               // monotone unsigned images of the logits
#pragma unroll
            for (int c = 0; c < EP; c += 16) {
                uint32_t hi[16], mid[16], lo[16];
                tc_ld16(taddr + 2 * EP + c, lo);
                tc_ld16(taddr + EP + c, mid);
                tc_ld16(taddr + c, hi);
                tc_wait_ld();
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int e = c + i;
                    float val = (__uint_as_float(lo[i]) + __uint_as_float(mid[i])) + __uint_as_float(hi[i]);   // smallest terms first
                    if (a.bias) val += s_bias[e];
                    key[e] = float_key((e < E) ? val : -FLT_MAX);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctrl->tempty));   // the next tile's MMAs may overwrite the accumulator

            const int t = tile * BM + quad * 32 + lane;
            if (t >= a.T) continue;
            // selection: n_check rounds over the row in registers.  Branch-free: every logit becomes a 64-bit key
            // (monotone image of the float, then EP - 1 - expert id, so that keys are unique and the lowest id wins a
            // tie); round s takes the largest key below the previous pick; four independent max chains per round.
            // (Compare-and-assign on (value, id) pairs compiles to divergent branches and ran 6 times slower.)
            unsigned long long prev = ~0ull;
            float sv[32];
            int se[32];
            for (int s = 0; s < n_check; ++s) {
                unsigned long long b[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
                for (int i = 0; i < EP; i += 4) {
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const unsigned long long kk = ((unsigned long long)key[i + c] << 32) | (unsigned)(EP - 1 - (i + c));
                        const unsigned long long cand = kk < prev ? kk : 0ull;
                        b[c] = cand > b[c] ? cand : b[c];
                    }
                }
                unsigned long long m = b[0] > b[1] ? b[0] : b[1];
                const unsigned long long m2 = b[2] > b[3] ? b[2] : b[3];
                m = m > m2 ? m : m2;
                prev = m;
                sv[s] = key_float((unsigned)(m >> 32));
                se[s] = EP - 1 - (int)(m & 0xffffffffu);
            }
            // near-tie check over the sorted top-(k+1)
            float amax = 0.f;
            for (int s = 0; s < n_check; ++s) amax = fmaxf(amax, fabsf(sv[s]));
            bool close = false;
            for (int s = 0; s + 1 < n_check; ++s) close = close || (sv[s] - sv[s + 1] < guard_scale * (1.f + amax));
            if (close) {
                float* row = a.rows + (size_t)t * EP;
#pragma unroll
                for (int i = 0; i < EP; ++i) row[i] = key_float(key[i]);
                a.flagged[atomicAdd(&a.hdr->n_flag, 1)] = t;
            }
            // weights: exp(l_s - l_0) / sum over the k selected, the sum taken as the warp-shuffle tree of the other
            // router kernels takes it (lanes >= k contribute 0), so that all paths give the same bits
            float ex[32];
            for (int s = 0; s < 32; ++s) ex[s] = (s < k) ? expf(sv[s] - sv[0]) : 0.f;
            float tr[16];
            for (int i = 0; i < 16; ++i) tr[i] = ex[i] + ex[i + 16];
            for (int i = 0; i < 8; ++i) tr[i] = tr[i] + tr[i + 8];
            for (int i = 0; i < 4; ++i) tr[i] = tr[i] + tr[i + 4];
            for (int i = 0; i < 2; ++i) tr[i] = tr[i] + tr[i + 2];
            const float sum = tr[0] + tr[1];
            int32_t* io = a.idx + (size_t)t * k;
            float* wo = a.w + (size_t)t * k;
            for (int s = 0; s < k; ++s) {
                io[s] = se[s];
                wo[s] = ex[s] / sum;
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    if (*abort_flag) {   // failure path only: give copies and MMAs already in flight time to land before leaving
        const unsigned long long t0 = globaltimer();
        while (globaltimer() - t0 < 200000ull) { }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(a.tmem_cols) : "memory");
    }
}

static bool make_map(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    return tmap::bf16_sw128(m, ptr, rows, cols, box_rows);
}

template <int NJ>
static cudaError_t launch_one(const CUtensorMap& mA, const CUtensorMap& mB, Args a, int grid, cudaStream_t s) {
    constexpr int EP = 32 * NJ;
    constexpr int STAGE_BYTES = A_BYTES + 3 * EP * BK * 2;
    int stages = (SMEM_LIMIT - 1024 - SMEM_CTRL) / STAGE_BYTES;
    if (stages > MAX_STAGES) stages = MAX_STAGES;
    if (stages < 2) return cudaErrorInvalidConfiguration;
    const int smem_bytes = stages * STAGE_BYTES + SMEM_CTRL + 1024;
    static PerDevice configured;      // per device: SM count once this instantiation has its shared-memory opt-in there
    int dev = 0, sms = 0;
    cudaError_t e = current_device(&dev);
    if (e != cudaSuccess) return e;
    e = configured.get(dev, &sms, [&](int d, int* n) {
        cudaError_t e2 = cudaFuncSetAttribute(router_fused_kernel<NJ>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
        return e2 != cudaSuccess ? e2 : device_sm_count(d, n);
    });
    if (e != cudaSuccess) return e;
    a.stages = stages;
    a.tmem_cols = 3 * EP <= 128 ? 128u : 3 * EP <= 256 ? 256u : 512u;
    int blocks = a.n_tiles < sms ? a.n_tiles : sms;
    if (grid > 0 && grid < blocks) blocks = grid;
    return launch_pdl(router_fused_kernel<NJ>, dim3(blocks), dim3(THREADS), (size_t)smem_bytes, s, mA, mB, a);
}

}  // namespace rf

bool router_fused_ok(int E, int k) { return E <= 160 && k <= 28; }

// split must hold 3 * EP rows of H bf16 (hi rows 0.., mid rows EP.., lo rows 2 EP.., EP = E rounded up to 32, pad rows
// zero); rows: [T, EP] floats; flagged: [T] ints.  The caller runs the split kernel before and the fix-up kernel after.
cudaError_t launch_router_fused(const __nv_bfloat16* x, const __nv_bfloat16* split, const float* bias, int T, int H, int E,
                                int k, float* rows, int32_t* flagged, WsHeader* hdr, int grid, int32_t* idx, float* w,
                                cudaStream_t s) {
    using namespace rf;
    const int nj = (E + 31) / 32, ep = 32 * nj;
    CUtensorMap mA, mB;
    if (!make_map(&mA, x, (uint64_t)T, (uint64_t)H, BM)) return cudaErrorInvalidValue;
    if (!make_map(&mB, split, (uint64_t)(3 * ep), (uint64_t)H, (uint32_t)ep)) return cudaErrorInvalidValue;
    Args a = {};
    a.bias = bias; a.idx = idx; a.w = w; a.rows = rows; a.flagged = flagged; a.hdr = hdr;
    a.T = T; a.H = H; a.E = E; a.k = k;
    a.n_tiles = (T + BM - 1) / BM;
    a.k_blocks = (H + BK - 1) / BK;
    switch (nj) {
        case 1: return launch_one<1>(mA, mB, a, grid, s);
        case 2: return launch_one<2>(mA, mB, a, grid, s);
        case 3: return launch_one<3>(mA, mB, a, grid, s);
        case 4: return launch_one<4>(mA, mB, a, grid, s);
        case 5: return launch_one<5>(mA, mB, a, grid, s);
    }
    return cudaErrorInvalidValue;
}

}  // namespace mok
