// Grouped expert GEMMs with the TOKENS on the N side of the MMA (paper, Section 2.1: the expert FFN; Section 3.2:
// tensor cores must stay saturated although per-expert batches are ragged).
//
// tcgen05.mma fixes M at 128 rows but lets N be any multiple of 16.  Experts own ragged numbers of rows, so this
// kernel puts the WEIGHT rows on the M side and the expert's tokens on the N side: C^T[feature, token] = W . X^T.  A
// tile is two 128-row weight sub-tiles (gate + up for SwiGLU, 256 consecutive output features otherwise) against up to
// 128 tokens; the last tile of an expert runs with N = its row count rounded up to 16, so padding costs at most 15
// rows per expert instead of 127, and its MMAs take proportionally less time.  Per k-block a CTA still moves 48 KB
// (2 x 16 KB of weights + 16 KB of tokens) for 2 x 128 x 128 x 64 MACs, the same ratio as a 128 x 256 tile.
//
//   warp 0      TMA producer : weight sub-tiles (and the token tile when it comes from a contiguous buffer)
//   warp 1      MMA issuer   : per K step two MMAs (M=128, N=rows) into two 128-column accumulators in TMEM
//   warps 2..5  epilogue     : thread = output feature, registers = tokens; (SwiGLU) -> bf16 -> transposed into a
//                              swizzled [token][feature] staging tile -> TMA stores of 16-row boxes
//   warps 6..9  gather       : GATHER only: token rows of x through the schedule's row -> token table (pull
//                              dispatch, Section 3.1) with 16-byte cp.async into the swizzled token stage
// Row space: expert e owns rows [pad_offsets[e], pad_offsets[e] + roundup16(counts[e])); token tile m of an expert
// starts at pad_offsets[e] + 128 m.  Tile order: expert, group of 16 token tiles, feature tile, token tile (fastest),
// so CTAs side by side share weight tiles in L2.  One tile = one fixed k order per output element, so results do
// not depend on the grid or on timing (Section 3.4 "Determinism").  All waits are bounded.
#include "mok_internal.cuh"
#include "tc_ptx.cuh"
#include "tensor_map.cuh"

namespace mok {
namespace tn {

using namespace tc;

constexpr int WM = 128;                        // weight rows per sub-tile (MMA M)
constexpr int NT = 128;                        // token rows per tile (MMA N; tail tiles use a multiple of 16)
constexpr int BK = 64, UMMA_K = 16, STAGES = 4;
constexpr int W_BYTES = WM * BK * 2;           // 16 KB
constexpr int X_BYTES = NT * BK * 2;           // 16 KB
constexpr int STAGE_BYTES = 2 * W_BYTES + X_BYTES;
constexpr int ACC_STAGES = 2, TMEM_COLS = 512, ACC_COLS = 256;   // two 128-column accumulators per stage
constexpr int THREADS = 192, GATHER_THREADS = 128;
constexpr int GROUP_TILES = 16;
constexpr int OUT_BYTES = NT * 128 * 2;        // staging: 128 tokens x 128 features bf16, as two [128 x 128 B] halves
constexpr int SMEM_CTRL = 256;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + OUT_BYTES + SMEM_CTRL + 1024;

struct Ctrl {
    uint64_t full[STAGES], empty[STAGES], tfull[ACC_STAGES], tempty[ACC_STAGES];
    uint32_t tmem_base, abort;
};
static_assert(sizeof(Ctrl) <= SMEM_CTRL, "control block too large");

struct Tile { int e, n, row0, rows, valid; };   // rows: multiple of 16 (MMA N); valid: real rows of this tile

__device__ __forceinline__ Tile decode_tile(const GemmArgs& a, int L, int n_nt, int n_mt_total) {
    Tile t;
    int mt0, m_cnt, pad0, cnt;
    if (a.dense_rows > 0) {
        t.e = 0; mt0 = 0; m_cnt = n_mt_total; pad0 = 0; cnt = a.dense_rows;
    } else {
        t.e = __ldg(a.tile_expert + L / n_nt);
        mt0 = __ldg(a.mt_start + t.e);
        m_cnt = __ldg(a.mt_start + t.e + 1) - mt0;
        pad0 = __ldg(a.pad_offsets + t.e);
        cnt = __ldg(a.counts + t.e);
    }
    const int r = L - n_nt * mt0;
    const int per_group = GROUP_TILES * n_nt;
    const int g = r / per_group;
    const int rem = r - g * per_group;
    const int in_group = min(GROUP_TILES, m_cnt - g * GROUP_TILES);
    t.n = rem / in_group;
    const int m = g * GROUP_TILES + (rem - t.n * in_group);
    t.row0 = pad0 + m * NT;
    t.valid = min(NT, cnt - m * NT);
    t.rows = (t.valid + 15) & ~15;
    return t;
}

__device__ __forceinline__ void st_shared_b16(uint32_t addr, uint16_t v) {
    asm volatile("st.shared.b16 [%0], %1;" ::"r"(addr), "h"(v) : "memory");
}
__device__ __forceinline__ void epi_bar() { asm volatile("bar.sync 1, 128;" ::: "memory"); }   // the 4 epilogue warps
__device__ __forceinline__ uint16_t bf16_bits(float v) {
    __nv_bfloat16 b = __float2bfloat16_rn(v);
    return *reinterpret_cast<uint16_t*>(&b);
}
// Byte offset of (token t, feature f) in the staging tile: two halves of 64 features, rows of 128 bytes, 16-byte chunks
// XOR-swizzled with the row index: the layout a 128-byte-swizzled TMA store of [16 rows x 64 columns] boxes expects.
__device__ __forceinline__ uint32_t out_offset(int t, int f) {
    return (uint32_t)((f >> 6) * (NT * 128) + t * 128 + ((((f & 63) >> 3) ^ (t & 7)) << 4) + ((f & 7) << 1));
}

template <int EPI, bool GATHER>
__global__ void __launch_bounds__(THREADS + (GATHER ? GATHER_THREADS : 0), 1)
gemm_tn_kernel(const __grid_constant__ CUtensorMap tmapW, const __grid_constant__ CUtensorMap tmapX,
               const __grid_constant__ CUtensorMap tmapC, const GemmArgs a, const int n_nt, const int k_blocks) {
    constexpr bool SWIGLU = (EPI == EPI_SWIGLU);
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem + STAGES * STAGE_BYTES + OUT_BYTES);
    volatile uint32_t* abort_flag = &ctrl->abort;
    const uint32_t out_base = base + STAGES * STAGE_BYTES;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    int n_mt_total = (a.dense_rows > 0) ? (a.dense_rows + NT - 1) / NT : *a.n_mtiles;
    if (n_mt_total > a.max_mt) n_mt_total = a.max_mt;
    const int total = n_mt_total * n_nt;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(smem_u32(&ctrl->full[s]), GATHER ? 1 + GATHER_THREADS : 1);
            mbar_init(smem_u32(&ctrl->empty[s]), 1);
        }
        for (int s = 0; s < ACC_STAGES; ++s) {
            mbar_init(smem_u32(&ctrl->tfull[s]), 1);
            mbar_init(smem_u32(&ctrl->tempty[s]), 4);
        }
        ctrl->abort = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&ctrl->tmem_base)), "r"((uint32_t)TMEM_COLS) : "memory");
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
            const int w_rows_per_expert = (SWIGLU ? 2 : 1) * a.N;
            for (int L = blockIdx.x; L < total; L += gridDim.x) {
                const Tile t = decode_tile(a, L, n_nt, n_mt_total);
                // weight sub-tiles: gate rows + the matching up rows for SwiGLU, 256 consecutive rows otherwise
                const int wrow0 = t.e * w_rows_per_expert + (SWIGLU ? t.n * WM : t.n * 2 * WM);
                const int wrow1 = SWIGLU ? wrow0 + a.N : wrow0 + WM;
                bool ok = true;
                for (int kb = 0; kb < k_blocks; ++kb) {
                    ok = mbar_wait(smem_u32(&ctrl->empty[s]), ph ^ 1u, abort_flag, a.header, 1);
                    if (!ok) break;
                    const uint32_t full = smem_u32(&ctrl->full[s]);
                    const uint32_t sw = base + s * STAGE_BYTES;
                    mbar_expect_tx(full, GATHER ? 2 * W_BYTES : STAGE_BYTES);
                    tma_load_2d(sw, &tmapW, full, kb * BK, wrow0);
                    tma_load_2d(sw + W_BYTES, &tmapW, full, kb * BK, wrow1);
                    if (!GATHER) tma_load_2d(sw + 2 * W_BYTES, &tmapX, full, kb * BK, t.row0);
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (!ok) break;
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            int s = 0, as = 0;
            uint32_t ph = 0, aph = 0;
            for (int L = blockIdx.x; L < total; L += gridDim.x) {
                const Tile t = decode_tile(a, L, n_nt, n_mt_total);
                // D fp32, A/B bf16, both K-major, M = 128, N = this tile's rows
                const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(t.rows >> 3) << 17) |
                                       ((uint32_t)(WM >> 4) << 24);
                bool ok = mbar_wait(smem_u32(&ctrl->tempty[as]), aph ^ 1u, abort_flag, a.header, 2);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d0 = tmem_base + (uint32_t)(as * ACC_COLS), d1 = d0 + NT;
                for (int kb = 0; kb < k_blocks; ++kb) {
                    ok = mbar_wait(smem_u32(&ctrl->full[s]), ph, abort_flag, a.header, 3);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t sw = base + s * STAGE_BYTES;
                    const uint64_t w0 = make_smem_desc(sw), w1 = make_smem_desc(sw + W_BYTES);
                    const uint64_t xd = make_smem_desc(sw + 2 * W_BYTES);
#pragma unroll
                    for (int j = 0; j < BK / UMMA_K; ++j) {
                        tc_mma<1>(d0, w0 + (uint64_t)(j * 2), xd + (uint64_t)(j * 2), idesc, (kb | j) ? 1u : 0u);
                        tc_mma<1>(d1, w1 + (uint64_t)(j * 2), xd + (uint64_t)(j * 2), idesc, (kb | j) ? 1u : 0u);
                    }
                    tc_commit<1>(smem_u32(&ctrl->empty[s]));
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (!ok) break;
                tc_commit<1>(smem_u32(&ctrl->tfull[as]));
                if (++as == ACC_STAGES) { as = 0; aph ^= 1u; }
            }
        }
        __syncwarp();
    } else if (GATHER && warp >= 6) {
        // ------------------------------------------------------------------ gather warps 6..9 (pull dispatch)
        // Warp gw owns token rows 32 gw .. 32 gw + 31 of the tile; lane = (sub-row 0..3, 16-byte chunk 0..7); pass i
        // covers rows 32 gw + 4 i + sub-row.  Chunk c of row r lands at r*128 + ((c ^ (r & 7)) * 16).  Rows between
        // `valid` and `rows` re-read the tile's first row (computed, never combined); rows >= `rows` are not read by
        // the MMA and are skipped.
        const int gw = warp - 6, sub = lane >> 3, chunk = lane & 7;
        int s = 0;
        uint32_t ph = 0;
        for (int L = blockIdx.x; L < total; L += gridDim.x) {
            const Tile t = decode_tile(a, L, n_nt, n_mt_total);
            const int tok0 = __ldg(a.row_token + t.row0);
            const __nv_bfloat16* src[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int r = gw * 32 + i * 4 + sub;
                const int tok = (r < t.valid) ? __ldg(a.row_token + t.row0 + r) : tok0;
                src[i] = a.A + (size_t)tok * a.K + chunk * 8;
            }
            bool ok = true;
            for (int kb = 0; kb < k_blocks; ++kb) {
                ok = mbar_wait(smem_u32(&ctrl->empty[s]), ph ^ 1u, abort_flag, a.header, 5);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const uint32_t sx = base + s * STAGE_BYTES + 2 * W_BYTES;
                const bool in_k = (kb * BK + chunk * 8) < a.K;            // K tail: zero-fill
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int r = gw * 32 + i * 4 + sub;
                    if (r < t.rows) {
                        const uint32_t dst = sx + r * 128 + ((chunk ^ (r & 7)) << 4);
                        cp_async_16(dst, in_k ? (const void*)(src[i] + kb * BK) : (const void*)a.A, in_k ? 16u : 0u);
                    }
                }
                cp_async_mbar_arrive(smem_u32(&ctrl->full[s]));
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
            if (!ok) break;
        }
        asm volatile("cp.async.wait_all;" ::: "memory");
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int quad = warp & 3;                            // TMEM lane quadrant = features 32 quad .. 32 quad + 31
        const int f = quad * 32 + lane;                       // this thread's feature inside a 128-row sub-tile
        const bool leader = (warp == 2 && lane == 0);         // issues the TMA stores
        int as = 0;
        uint32_t aph = 0;
        for (int L = blockIdx.x; L < total; L += gridDim.x) {
            const Tile t = decode_tile(a, L, n_nt, n_mt_total);
            bool ok = mbar_wait(smem_u32(&ctrl->tfull[as]), aph, abort_flag, a.header, 4);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(as * ACC_COLS);
            if (EPI == EPI_F32) {
                // logits[token][column]: for a fixed token the warp's 32 features are 32 consecutive floats
                float* cbase = reinterpret_cast<float*>(a.C) + (size_t)t.row0 * a.ldc;
#pragma unroll 1
                for (int sub_tile = 0; sub_tile < 2; ++sub_tile) {
                    const int col = t.n * 2 * WM + sub_tile * WM + f;
#pragma unroll 1
                    for (int c = 0; c < t.rows; c += 32) {
                        uint32_t r[32];
                        tc_ld32(taddr + sub_tile * NT + c, r);
                        tc_wait_ld();
                        if (col < a.N) {
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                if (c + i < t.rows) cbase[(size_t)(c + i) * a.ldc + col] = __uint_as_float(r[i]);
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctrl->tempty[as]));
            } else {
                constexpr int PASSES = SWIGLU ? 1 : 2;        // 128 output features per pass
#pragma unroll 1
                for (int pass = 0; pass < PASSES; ++pass) {
                    if (leader) tma_store_wait_read();        // the staging tile's previous stores have been read out
                    epi_bar();
#pragma unroll 1
                    for (int c = 0; c < t.rows; c += 32) {
                        uint32_t g[32];
                        if (SWIGLU) {
                            uint32_t u[32];
                            tc_ld32(taddr + c, g);
                            tc_ld32(taddr + NT + c, u);
                            tc_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) {
                                const float gv = __uint_as_float(g[i]);
                                const float hv = swiglu(gv, __uint_as_float(u[i]));
                                st_shared_b16(out_base + out_offset(c + i, f), bf16_bits(hv));
                            }
                        } else {
                            tc_ld32(taddr + pass * NT + c, g);
                            tc_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                st_shared_b16(out_base + out_offset(c + i, f), bf16_bits(__uint_as_float(g[i])));
                        }
                    }
                    if (pass == PASSES - 1) tc_fence_before();   // all TMEM reads of this tile are done
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    epi_bar();
                    if (pass == PASSES - 1 && lane == 0) mbar_arrive(smem_u32(&ctrl->tempty[as]));
                    if (leader) {
                        const int col0 = SWIGLU ? t.n * WM : t.n * 2 * WM + pass * WM;
#pragma unroll 1
                        for (int half = 0; half < 2; ++half) {
                            const int col = col0 + half * 64;
                            if (col >= a.N) break;
                            for (int r = 0; r < t.rows; r += 16)
                                tma_store_2d(&tmapC, out_base + half * (NT * 128) + r * 128, col, t.row0 + r);
                        }
                        tma_store_commit();
                    }
                }
            }
            if (++as == ACC_STAGES) { as = 0; aph ^= 1u; }
        }
        if (leader) tma_store_wait_all();
        __syncwarp();
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
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
    }
}

static bool make_map(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows, uint64_t stride) {
    return tmap::bf16_sw128(m, ptr, rows, cols, box_rows, stride);
}

template <int EPI, bool GATHER>
static cudaError_t launch_one(const CUtensorMap& mW, const CUtensorMap& mX, const CUtensorMap& mC, const GemmArgs& a,
                              int n_nt, int k_blocks, int grid, cudaStream_t s) {
    static PerDevice configured;      // per device: SM count once this instantiation has its shared-memory opt-in there
    int dev = 0, sm_count = 0;
    cudaError_t e = current_device(&dev);
    if (e != cudaSuccess) return e;
    e = configured.get(dev, &sm_count, [](int d, int* sms) {
        cudaError_t e2 = cudaFuncSetAttribute(gemm_tn_kernel<EPI, GATHER>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              SMEM_BYTES);
        return e2 != cudaSuccess ? e2 : device_sm_count(d, sms);
    });
    if (e != cudaSuccess) return e;
    if (grid <= 0 || grid > sm_count) grid = sm_count;
    gemm_tn_kernel<EPI, GATHER><<<grid, THREADS + (GATHER ? GATHER_THREADS : 0), SMEM_BYTES, s>>>(mW, mX, mC, a, n_nt,
                                                                                                 k_blocks);
    return cudaGetLastError();
}

}  // namespace tn

cudaError_t launch_gemm_tn(const GemmArgs& a, int epi, int grid, cudaStream_t s) {
    using namespace tn;
    const bool swiglu = (epi == EPI_SWIGLU), gather = (a.row_token != nullptr);
    CUtensorMap mW, mX, mC;
    const uint64_t w_rows = (uint64_t)a.E * (swiglu ? 2 : 1) * a.N;
    if (!make_map(&mW, a.B, w_rows, (uint64_t)a.K, WM, (uint64_t)a.K)) return cudaErrorInvalidValue;
    if (!make_map(&mX, a.A, (uint64_t)a.a_rows, (uint64_t)a.K, NT, (uint64_t)a.K)) return cudaErrorInvalidValue;
    if (epi == EPI_F32) mC = mW;      // the fp32 epilogue stores directly
    else if (!make_map(&mC, a.C, (uint64_t)a.rows_pad, (uint64_t)a.N, 16, (uint64_t)a.ldc)) return cudaErrorInvalidValue;
    const int n_nt = swiglu ? (a.N + WM - 1) / WM : (a.N + 2 * WM - 1) / (2 * WM);
    const int k_blocks = (a.K + BK - 1) / BK;
    if (epi == EPI_SWIGLU && gather) return launch_one<EPI_SWIGLU, true>(mW, mX, mC, a, n_nt, k_blocks, grid, s);
    if (epi == EPI_SWIGLU) return launch_one<EPI_SWIGLU, false>(mW, mX, mC, a, n_nt, k_blocks, grid, s);
    if (epi == EPI_BF16 && !gather) return launch_one<EPI_BF16, false>(mW, mX, mC, a, n_nt, k_blocks, grid, s);
    if (epi == EPI_F32 && !gather) return launch_one<EPI_F32, false>(mW, mX, mC, a, n_nt, k_blocks, grid, s);
    return cudaErrorInvalidValue;
}

}  // namespace mok
