// Grouped expert GEMMs on MXFP8 operands (Section 3.4 "MXFP8 Support"): E4M3 elements with one E8M0 scale per 32
// elements along K, multiplied by the block-scaled 5th-generation tensor-core instruction
// (tcgen05.mma.kind::mxf8f6f4.block_scale, M = 128, N = 256, K = 32, fp32 accumulators in TMEM).
//
// Same persistent, warp-specialised shape as the bf16 kernel with 128-row tiles:
//   warp 0       TMA producer : A tile [128 rows x 128 bytes] and B tile [256 x 128 bytes] (128-byte swizzle) plus
//                               their scale atoms (512 bytes per 128 rows and 128-element k-group) -> 4-stage ring
//   warp 1       MMA issuer   : per stage, copies the scale atoms from shared memory into tensor memory
//                               (tcgen05.cp 32x128b.warpx4: 4 columns per atom, replicated over the four lane
//                               quadrants), then issues four K = 32 MMAs that pick their scale byte by id 0..3
//   warps 2..9   epilogue     : two warps per TMEM lane quadrant, each draining half of the tile's columns
//   warps 10..13 gather       : GATHER only: pull dispatch of the quantised token rows (Section 3.1) with 16-byte
//                               cp.async, and of their scales (4 bytes per row and stage) into the atom layout
// CTAS = 2 (default): two CTAs of a cluster compute one 256 x 256 tile with cta_group::2 MMAs issued by the even CTA.
// Each CTA stages its own 128 rows of A, HALF of the weight tile, its rows' scale atom and both weight scale atoms
// (every CTA needs the scales of all 256 weight rows in its own tensor memory; one tcgen05.cp.cta_group::2 makes
// both CTAs copy from their own shared memory).  A k-stage then moves 33.5 KB instead of 49.5 KB from L2 into each
// SM for the same 512 tensor-pipe cycles: with one-byte operands the 128 x 256 tile of a single CTA asks for about
// twice the bytes per cycle that the L2 -> SM path delivers.  The odd CTA's TMA loads complete on the even CTA's
// mbarrier; its gathered rows are announced by its warp 1; commits are multicast to both CTAs.  No TMA multicast.
// Pair tiles are the 256-row tiles of the schedule's second tile table over the 128-row-padded row space: when an
// expert's last tile has at most 128 rows the odd CTA computes rows of the next segment and stores nothing.
// Tensor memory holds ONE 256-column accumulator (the scale atoms need columns too, so a second N = 256 accumulator
// does not fit into the 512 columns); the epilogue therefore hands the accumulator back as soon as its last
// tcgen05.ld has completed and does its arithmetic and stores afterwards.
//
//   EPI_SWIGLU : B tile = 128 gate rows + the matching 128 up rows; the epilogue computes h = silu(g) * u in fp32,
//                quantises it to MXFP8 along the output columns (the next GEMM's K) -- each thread holds the 32
//                consecutive columns of one block, so amax, scale and codes need no communication -- and writes the
//                codes to C [rows, N] and the scales straight into the atom layout the down GEMM loads ("fuses
//                activation quantization into ... the gated activation computation").
//   EPI_BF16   : C [rows, N] bf16 = A . B^T (the down projection; its output feeds the fp32 combine).
// K and N may be ragged: TMA zero-fills bytes past K and rows past the tensor, whose scales are 127 (= 1.0).
// All mbarrier waits are bounded; on a timeout the CTA records MOK_ERR_TIMEOUT and leaves cleanly.
#include "mok_internal.cuh"
#include "tc_ptx.cuh"
#include "tile_order.cuh"
#include "mx_ptx.cuh"
#include "tensor_map.cuh"

namespace mok {
namespace mx {

using namespace tc;

constexpr int BM = 128, BN = 256, BKB = 128;   // BM: rows per CTA; BKB: bytes = elements of K per stage (four K = 32 MMAs)
constexpr int A_BYTES = BM * BKB;              // 16 KB
constexpr int B_BYTES = BN * BKB;              // 32 KB (whole tile; a CTA of a pair stages half of it)
constexpr int RING_BYTES = 196608;             // 4 x 48 KB or 6 x 32 KB of swizzled operand tiles
constexpr int MAX_STAGES = 6;
constexpr int SF_BYTES = 1536;                 // per stage: the A rows' scale atom (512 bytes) + the B rows' two
constexpr int SF_REGION = RING_BYTES;
constexpr int SLAB_BYTES = 2048;               // per epilogue warp: 32 rows x 32 bf16 columns, for coalesced stores
constexpr int SLAB_REGION = SF_REGION + MAX_STAGES * SF_BYTES;
constexpr int TMEM_COLS = 512, SF_COL0 = BN, SF_COLS = 12;   // per stage: 4 columns for A's atom, 8 for B's two
constexpr int EPI_WARPS = 8;
constexpr int THREADS = 64 + 32 * EPI_WARPS;   // + 4 gather warps in the GATHER instantiation
constexpr int GATHER_THREADS = 128;
constexpr int SMEM_CTRL = 256;
constexpr int SMEM_BYTES = SLAB_REGION + EPI_WARPS * SLAB_BYTES + SMEM_CTRL + 1024;

struct Ctrl {
    uint64_t full[MAX_STAGES];     // this CTA's stage has landed (TMA bytes + gather arrivals)
    uint64_t pfull[MAX_STAGES];    // even CTA only: the odd CTA's gathered stage has landed
    uint64_t empty[MAX_STAGES];
    uint64_t tfull;
    uint64_t tempty;
    uint32_t tmem_base;
    uint32_t abort;
};
static_assert(sizeof(Ctrl) <= SMEM_CTRL, "control block too large");

// Source of a gathered token row (E4M3 codes) and of its scale bytes: this GPU's own buffers, or in expert-parallel
// mode (global token id = source_rank * peer_tokens + token) the owning rank's, read with plain peer loads.
__device__ __forceinline__ const uint8_t* mx_row(const GemmArgs& a, const uint8_t* xq, int tok) {
    if (a.peer_tokens > 0) {
        const int r = tok / a.peer_tokens;
        return reinterpret_cast<const uint8_t*>(a.peer_x[r]) + (size_t)(tok - r * a.peer_tokens) * a.K;
    }
    return xq + (size_t)tok * a.K;
}
__device__ __forceinline__ const uint8_t* mx_row_scales(const GemmArgs& a, int tok) {
    if (a.peer_tokens > 0) {
        const int r = tok / a.peer_tokens;
        return a.peer_sfa[r] + (size_t)(tok - r * a.peer_tokens) * a.sfa_stride;
    }
    return a.sfa + (size_t)tok * a.sfa_stride;
}

template <int EPI, bool GATHER, int CTAS>
__global__ void __launch_bounds__(THREADS + (GATHER ? GATHER_THREADS : 0), 1)
gemm_mx_kernel(const __grid_constant__ CUtensorMap tmapA, const __grid_constant__ CUtensorMap tmapB,
               const __grid_constant__ CUtensorMap tmapSFA, const __grid_constant__ CUtensorMap tmapSFB,
               const __grid_constant__ GemmArgs a, const int n_nt, const int k_blocks) {
    constexpr bool SWIGLU = (EPI == EPI_SWIGLU);
    constexpr int STAGES = (CTAS == 2) ? 6 : 4;
    constexpr int B_STAGE = B_BYTES / CTAS;
    constexpr int STAGE_BYTES = A_BYTES + B_STAGE;
    constexpr int TM = BM * CTAS;
    static_assert(STAGES * STAGE_BYTES == RING_BYTES, "ring size");
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem + SLAB_REGION + EPI_WARPS * SLAB_BYTES);
    volatile uint32_t* abort_flag = &ctrl->abort;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = (CTAS == 2) ? (int)cluster_ctarank() : 0;      // 0 = the CTA that issues the MMAs
    const int unit = blockIdx.x / CTAS, n_units = gridDim.x / CTAS;

    int n_mt_total = (a.dense_rows > 0) ? (a.dense_rows + TM - 1) / TM : *a.n_mtiles;
    if (n_mt_total > a.max_mt) n_mt_total = a.max_mt;
    const int total = n_mt_total * n_nt;
    const int KG = k_blocks;                                  // 128-element k-groups = scale atoms along K

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            // arrivals per phase: the producer's expect_tx (not in the odd CTA of a pair, whose TMA bytes complete on
            // the even CTA's barrier) + one per gather thread
            const int full_arrivals = ((CTAS == 2 && rank == 1) ? 0 : 1) + (GATHER ? GATHER_THREADS : 0);
            mbar_init(smem_u32(&ctrl->full[s]), full_arrivals > 0 ? full_arrivals : 1);
            mbar_init(smem_u32(&ctrl->pfull[s]), 1);
            mbar_init(smem_u32(&ctrl->empty[s]), 1);
        }
        mbar_init(smem_u32(&ctrl->tfull), 1);
        mbar_init(smem_u32(&ctrl->tempty), EPI_WARPS * CTAS);
        ctrl->abort = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        if (CTAS == 1) {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(&ctrl->tmem_base)), "r"((uint32_t)TMEM_COLS) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(&ctrl->tmem_base)), "r"((uint32_t)TMEM_COLS) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if (CTAS == 2) cluster_sync();          // the peer's barriers exist before anyone arrives on them remotely
    tc_fence_after();
    const uint32_t tmem_base = ctrl->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0 && !a.starve) {
            int s = 0;
            uint32_t ph = 0;
            const int b_rows_per_expert = (SWIGLU ? 2 : 1) * a.N;
            const int NB = (a.N + 127) / 128;                 // 128-row blocks of one weight matrix (scale atoms)
            for (int L = unit; L < total; L += n_units) {
                const Tile t = decode_tile(a, L, n_nt, n_mt_total, TM);
                const int brow0 = t.e * b_rows_per_expert + (SWIGLU ? t.n * (BN / 2) : t.n * BN);
                const int brow1 = SWIGLU ? brow0 + a.N : brow0 + BN / 2;
                // scale atoms of the two 128-row halves of the B tile, and of this CTA's 128 A rows
                int nb0, nb1;
                if (SWIGLU) { nb0 = (2 * t.e) * NB + t.n; nb1 = (2 * t.e + 1) * NB + t.n; }
                else { nb0 = t.e * NB + min(2 * t.n, NB - 1); nb1 = t.e * NB + min(2 * t.n + 1, NB - 1); }
                const int sfb0 = nb0 * KG, sfb1 = nb1 * KG;
                const int arow = t.row0 + rank * BM;
                const int sfa0 = (arow / BM) * KG;
                bool ok = true;
                for (int kb = 0; kb < k_blocks; ++kb) {
                    ok = mbar_wait(smem_u32(&ctrl->empty[s]), ph ^ 1u, abort_flag, a.header, 1);
                    if (!ok) break;
                    const uint32_t full = smem_u32(&ctrl->full[s]);
                    const uint32_t sa = base + s * STAGE_BYTES, sb = sa + A_BYTES;
                    const uint32_t sf = base + SF_REGION + s * SF_BYTES;
                    constexpr uint32_t per_cta = (uint32_t)(B_STAGE + 1024 + (GATHER ? 0 : A_BYTES + 512));
                    if (CTAS == 1) {
                        mbar_expect_tx(full, per_cta);
                        if (!GATHER) {
                            tma_load_2d(sa, &tmapA, full, kb * BKB, arow);
                            tma_load_2d(sf, &tmapSFA, full, 0, sfa0 + kb);
                        }
                        tma_load_2d(sb, &tmapB, full, kb * BKB, brow0);
                        tma_load_2d(sb + B_BYTES / 2, &tmapB, full, kb * BKB, brow1);
                        tma_load_2d(sf + 512, &tmapSFB, full, 0, sfb0 + kb);
                        tma_load_2d(sf + 1024, &tmapSFB, full, 0, sfb1 + kb);
                    } else if (rank == 0) {
                        // the even CTA's barrier collects the TMA bytes of both CTAs of the pair
                        mbar_expect_tx(full, 2 * per_cta);
                        if (!GATHER) {
                            tma_load_2d(sa, &tmapA, full, kb * BKB, arow);
                            tma_load_2d(sf, &tmapSFA, full, 0, sfa0 + kb);
                        }
                        tma_load_2d(sb, &tmapB, full, kb * BKB, brow0);
                        tma_load_2d(sf + 512, &tmapSFB, full, 0, sfb0 + kb);
                        tma_load_2d(sf + 1024, &tmapSFB, full, 0, sfb1 + kb);
                    } else {
                        if (!GATHER) {
                            tma_load_2d_peer(sa, &tmapA, full, kb * BKB, arow);
                            tma_load_2d_peer(sf, &tmapSFA, full, 0, sfa0 + kb);
                        }
                        tma_load_2d_peer(sb, &tmapB, full, kb * BKB, brow1);
                        tma_load_2d_peer(sf + 512, &tmapSFB, full, 0, sfb0 + kb);
                        tma_load_2d_peer(sf + 1024, &tmapSFB, full, 0, sfb1 + kb);
                    }
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (!ok) break;
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            // -------------------------------------------------------------- MMA issuer (even CTA of a pair)
            int s = 0;
            uint32_t ph = 0, aph = 0;
            const bool dbg = a.dbg_slot >= 0;
            long long d_full = 0, d_pfull = 0, d_tempty = 0, d_kb = 0;
            const long long d_t0 = dbg ? clock64() : 0;
            for (int L = unit; L < total; L += n_units) {
                long long w0 = dbg ? clock64() : 0;
                bool ok = mbar_wait(smem_u32(&ctrl->tempty), aph ^ 1u, abort_flag, a.header, 2);
                if (dbg) d_tempty += clock64() - w0;
                if (!ok) break;
                aph ^= 1u;
                tc_fence_after();
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (dbg) w0 = clock64();
                    ok = mbar_wait(smem_u32(&ctrl->full[s]), ph, abort_flag, a.header, 3);
                    if (dbg) { const long long w1 = clock64(); d_full += w1 - w0; w0 = w1; ++d_kb; }
                    if (ok && CTAS == 2 && GATHER) ok = mbar_wait(smem_u32(&ctrl->pfull[s]), ph, abort_flag, a.header, 6);
                    if (dbg) d_pfull += clock64() - w0;
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t sa = base + s * STAGE_BYTES, sb = sa + A_BYTES;
                    const uint32_t sf = base + SF_REGION + s * SF_BYTES;
                    const uint32_t sf_tmem = tmem_base + (uint32_t)(SF_COL0 + s * SF_COLS);
                    tc_cp_sf<CTAS>(sf_tmem, make_sf_desc(sf));
                    tc_cp_sf<CTAS>(sf_tmem + 4, make_sf_desc(sf + 512));
                    tc_cp_sf<CTAS>(sf_tmem + 8, make_sf_desc(sf + 1024));
                    const uint64_t adesc = make_smem_desc(sa), bdesc = make_smem_desc(sb);
#pragma unroll
                    for (int j = 0; j < 4; ++j)               // +32 bytes per K = 32 step inside the 128-byte swizzle row
                        tc_mma_mx<CTAS>(tmem_base, adesc + (uint64_t)(j * 2), bdesc + (uint64_t)(j * 2),
                                        make_idesc_mx(TM, BN, (uint32_t)j), sf_tmem, sf_tmem + 4, (kb | j) ? 1u : 0u);
                    tc_commit<CTAS>(smem_u32(&ctrl->empty[s]));
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (!ok) break;
                tc_commit<CTAS>(smem_u32(&ctrl->tfull));
            }
            if (dbg) {
                unsigned long long* d = a.header->dbg[a.dbg_slot];
                atomicAdd(d + DBG_MMA_WAIT_FULL, (unsigned long long)d_full);
                atomicAdd(d + DBG_MMA_WAIT_PFULL, (unsigned long long)d_pfull);
                atomicAdd(d + DBG_MMA_WAIT_TEMPTY, (unsigned long long)d_tempty);
                atomicAdd(d + DBG_MMA_TOTAL, (unsigned long long)(clock64() - d_t0));
                atomicAdd(d + DBG_KBLOCKS, (unsigned long long)d_kb);
            }
        } else if (lane == 0 && CTAS == 2 && GATHER) {
            // -------------------------------------------------------------- odd CTA: tell the even CTA that my stage landed
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int L = unit; L < total && ok; L += n_units) {
                for (int kb = 0; kb < k_blocks; ++kb) {
                    ok = mbar_wait(smem_u32(&ctrl->full[s]), ph, abort_flag, a.header, 7);
                    if (!ok) break;
                    mbar_arrive_remote(smem_u32(&ctrl->pfull[s]), 0);
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else if (GATHER && warp >= 2 + EPI_WARPS) {
        // ------------------------------------------------------------------ gather warps (pull dispatch)
        // Data: warp gw owns tile rows 32 gw .. 32 gw + 31 of this CTA's 128; lane = (sub-row 0..3, 16-byte chunk 0..7);
        // pass i covers rows 32 gw + 4 i + sub-row; chunk c of row r lands at r*128 + ((c ^ (r & 7)) * 16).  Scales:
        // thread q of the 128 copies the 4 scale bytes of row q for this k-group to (q % 32) * 16 + (q / 32) * 4 of the
        // atom.  Rows past the expert's segment re-read the tile's first row (computed, never stored or combined).
        const int gw = warp - (2 + EPI_WARPS), sub = lane >> 3, chunk = lane & 7;
        const int q = gw * 32 + lane;
        int s = 0;
        uint32_t ph = 0;
        const uint8_t* xq = reinterpret_cast<const uint8_t*>(a.A);
        for (int L = unit; L < total; L += n_units) {
            const Tile t = decode_tile(a, L, n_nt, n_mt_total, TM);
            const int valid = __ldg(a.counts + t.e) - t.m * TM - rank * BM;
            const int tok0 = __ldg(a.row_token + t.row0);
            const int* rows = a.row_token + t.row0 + rank * BM;
            const uint8_t* src[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int r = gw * 32 + i * 4 + sub;
                const int tok = (r < valid) ? __ldg(rows + r) : tok0;
                src[i] = mx_row(a, xq, tok) + chunk * 16;
            }
            const int tokq = (q < valid) ? __ldg(rows + q) : tok0;
            const uint8_t* sfsrc = mx_row_scales(a, tokq);
            const uint32_t sfdst = base + SF_REGION + (q & 31) * 16 + (q >> 5) * 4;
            bool ok = true;
            for (int kb = 0; kb < k_blocks; ++kb) {
                ok = mbar_wait(smem_u32(&ctrl->empty[s]), ph ^ 1u, abort_flag, a.header, 5);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const uint32_t sa = base + s * STAGE_BYTES;
                const bool in_k = (kb * BKB + chunk * 16) < a.K;          // K tail: zero-fill
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int r = gw * 32 + i * 4 + sub;
                    const uint32_t dst = sa + r * 128 + ((chunk ^ (r & 7)) << 4);
                    cp_async_16(dst, in_k ? (const void*)(src[i] + kb * BKB) : (const void*)xq, in_k ? 16u : 0u);
                }
                cp_async_4(sfdst + s * SF_BYTES, sfsrc + kb * 4);
                cp_async_mbar_arrive(smem_u32(&ctrl->full[s]));
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
            if (!ok) break;
        }
        asm volatile("cp.async.wait_all;" ::: "memory");
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..9)
        // Warp w drains TMEM lane quadrant w % 4 (32 of this CTA's 128 rows) and column half (w - 2) / 4 of the tile.
        const int quad = warp & 3, hh = (warp - 2) >> 2;
        uint32_t aph = 0;
        for (int L = unit; L < total; L += n_units) {
            const Tile t = decode_tile(a, L, n_nt, n_mt_total, TM);
            bool ok = mbar_wait(smem_u32(&ctrl->tfull), aph, abort_flag, a.header, 4);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            aph ^= 1u;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16);
            const int row0 = t.row0 + rank * BM;                       // first of this CTA's 128 rows
            const int row = row0 + quad * 32 + lane;
            // the odd CTA of a pair has nothing to store when the expert's remaining rows fit into the even CTA's half
            const bool store = (CTAS == 1) || rank == 0 ||
                               ((a.dense_rows > 0 ? a.dense_rows : __ldg(a.counts + t.e)) - t.m * TM > BM);
            if (SWIGLU) {
                // output columns [64 hh, 64 hh + 64) of the tile's 128: two 32-column MX blocks per thread.  Block 0 is
                // quantised while block 1's loads are in flight; the accumulator goes back to the MMA issuer as soon
                // as the last tcgen05.ld has completed.
                uint32_t o[2][8];
                int code[2];
#pragma unroll
                for (int b = 0; b < 2; ++b) {
                    uint32_t g[32], u[32];
                    tc_ld32(taddr + hh * 64 + b * 32, g);
                    tc_ld32(taddr + BN / 2 + hh * 64 + b * 32, u);
                    tc_wait_ld();
                    if (b == 1) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) {
                            if (rank == 0) mbar_arrive(smem_u32(&ctrl->tempty));
                            else mbar_arrive_remote(smem_u32(&ctrl->tempty), 0);
                        }
                    }
                    float amax = 0.f;
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const float hv = swiglu(__uint_as_float(g[i]), __uint_as_float(u[i]));
                        g[i] = __float_as_uint(hv);
                        amax = fmaxf(amax, fabsf(hv));
                    }
                    code[b] = scale_code(amax);
                    const float inv = inv_scale(code[b]);
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2(__uint_as_float(g[4 * i]) * inv, __uint_as_float(g[4 * i + 1]) * inv), __NV_SATFINITE, __NV_E4M3);
                        const uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2(__uint_as_float(g[4 * i + 2]) * inv, __uint_as_float(g[4 * i + 3]) * inv), __NV_SATFINITE, __NV_E4M3);
                        o[b][i] = lo | (hi << 16);
                    }
                }
                if (store) {
                    uint8_t* crow = reinterpret_cast<uint8_t*>(a.C) + (size_t)row * a.ldc;
                    uint8_t* atom = a.sfc + ((size_t)(row0 / BM) * ((a.N + 127) / 128) + t.n) * 512 + lane * 16 + quad * 4;
#pragma unroll
                    for (int b = 0; b < 2; ++b) {
                        const int col = t.n * (BN / 2) + hh * 64 + b * 32;
                        if (col >= a.N) continue;
                        *reinterpret_cast<uint4*>(crow + col) = make_uint4(o[b][0], o[b][1], o[b][2], o[b][3]);
                        *reinterpret_cast<uint4*>(crow + col + 16) = make_uint4(o[b][4], o[b][5], o[b][6], o[b][7]);
                        atom[hh * 2 + b] = (uint8_t)code[b];
                    }
                }
            } else {
                // output columns [128 hh, 128 hh + 128) of the tile's 256, as bf16
                uint32_t o[4][16];
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t r[32];
                    tc_ld32(taddr + hh * 128 + c * 32, r);
                    tc_wait_ld();
#pragma unroll
                    for (int i = 0; i < 16; ++i) o[c][i] = pack_bf16(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (rank == 0) mbar_arrive(smem_u32(&ctrl->tempty));
                    else mbar_arrive_remote(smem_u32(&ctrl->tempty), 0);
                }
                // Transpose through this warp's slab so that each store instruction writes whole 64-byte row segments
                // of 8 rows (full 32-byte sectors) instead of 16 bytes in each of 32 different rows.
                const uint32_t slab = base + SLAB_REGION + (warp - 2) * SLAB_BYTES;
                const int rr = lane >> 2, seg = lane & 3;            // read side: row within a group of 8, 16-byte segment
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const int col = t.n * BN + hh * 128 + c * 32;
                    __syncwarp();
#pragma unroll
                    for (int v = 0; v < 4; ++v)
                        st_shared_v4(slab + lane * 64 + ((v ^ ((lane >> 1) & 3)) << 4), o[c][4 * v], o[c][4 * v + 1], o[c][4 * v + 2], o[c][4 * v + 3]);
                    __syncwarp();
                    if (store && col + seg * 8 < a.N) {
#pragma unroll
                        for (int it = 0; it < 4; ++it) {
                            const int r = it * 8 + rr;
                            uint4 val;
                            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                                         : "=r"(val.x), "=r"(val.y), "=r"(val.z), "=r"(val.w)
                                         : "r"(slab + r * 64 + ((seg ^ ((r >> 1) & 3)) << 4)));
                            __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(a.C) + (size_t)(row0 + quad * 32 + r) * a.ldc + col + seg * 8;
                            *reinterpret_cast<uint4*>(dst) = val;
                        }
                    }
                }
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
    if (CTAS == 2) cluster_sync();          // neither CTA frees TMEM or exits while the other may still touch it
    if (warp == 1) {
        tc_fence_after();
        if (CTAS == 1)
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
    }
}

// 2D row-major byte tensor [rows, cols] -> tensor map with a [128 rows x 128 bytes] box and 128-byte swizzle.
static bool make_map(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t cols) {
    return tmap::encode_2d(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, ptr, rows, cols, cols, (uint32_t)BKB, 128, CU_TENSOR_MAP_SWIZZLE_128B);
}

// Scale atoms as a 2D tensor [atoms, 128 words]: one box = one 512-byte atom, no swizzle.
static bool make_sf_map(CUtensorMap* m, const void* ptr, uint64_t atoms) {
    return tmap::encode_2d(m, CU_TENSOR_MAP_DATA_TYPE_UINT32, ptr, atoms, 128, 512, 128, 1, CU_TENSOR_MAP_SWIZZLE_NONE);
}

}  // namespace mx

template <int EPI, bool GATHER, int CTAS>
static cudaError_t launch_one_mx(const CUtensorMap& mA, const CUtensorMap& mB, const CUtensorMap& mSFA,
                                 const CUtensorMap& mSFB, const GemmArgs& a, int n_nt, int k_blocks, int grid,
                                 cudaStream_t s) {
    using namespace mx;
    static PerDevice configured;      // per device: CTAs (or CTA pairs) of the persistent grid, once configured there
    int max_units = 0;
    const int threads = THREADS + (GATHER ? GATHER_THREADS : 0);
    auto kernel = gemm_mx_kernel<EPI, GATHER, CTAS>;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    cfg.blockDim = dim3(threads);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = s;
    cfg.numAttrs = 0;
    if (CTAS == 2) {
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
    }
    {
        int dev = 0;
        cudaError_t e = current_device(&dev);
        if (e != cudaSuccess) return e;
        e = configured.get(dev, &max_units, [&](int d, int* units) {
            cudaError_t e2 = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
            if (e2 != cudaSuccess) return e2;
            int sms = 0;
            if ((e2 = device_sm_count(d, &sms)) != cudaSuccess) return e2;
            if (CTAS == 2) {
                int clusters = 0;
                cfg.gridDim = dim3(sms / 2 * 2);
                e2 = cudaOccupancyMaxActiveClusters(&clusters, kernel, &cfg);
                if (e2 != cudaSuccess) return e2;
                if (clusters < 1) return cudaErrorInvalidConfiguration;
                *units = clusters < sms / 2 ? clusters : sms / 2;
            } else {
                *units = sms;
            }
            return cudaSuccess;
        });
        if (e != cudaSuccess) return e;
    }
    int units = (grid <= 0) ? max_units : (grid + CTAS - 1) / CTAS;
    if (units > max_units) units = max_units;
    cfg.gridDim = dim3(units * CTAS);
    return cudaLaunchKernelEx(&cfg, kernel, mA, mB, mSFA, mSFB, a, n_nt, k_blocks);
}

// a.A / a.B: E4M3 codes; a.K a multiple of 32 and, for EPI_SWIGLU, a.N a multiple of 32.  a.tile_m = 128: single
// CTAs on the 128-row tile table; 256: CTA pairs on the 256-row tile table (both over the 128-row-padded row space).
cudaError_t launch_gemm_mx(const GemmArgs& a, int epi, int grid, cudaStream_t s) {
    using namespace mx;
    const bool swiglu = (epi == EPI_SWIGLU), gather = (a.row_token != nullptr), pair = (a.tile_m == 2 * BM);
    if ((a.tile_m != BM && !pair) || (a.K % 32) || !a.sfa || !a.sfb || (swiglu && (!a.sfc || (a.N % 32))))
        return cudaErrorInvalidValue;
    CUtensorMap mA, mB, mSFA, mSFB;
    const uint64_t b_rows = (uint64_t)a.E * (swiglu ? 2 : 1) * a.N;
    const uint64_t KG = (uint64_t)(a.K + BKB - 1) / BKB;
    if (!make_map(&mA, a.A, (uint64_t)a.a_rows, (uint64_t)a.K)) return cudaErrorInvalidValue;
    if (!make_map(&mB, a.B, b_rows, (uint64_t)a.K)) return cudaErrorInvalidValue;
    if (!make_sf_map(&mSFB, a.sfb, (uint64_t)a.E * (swiglu ? 2 : 1) * ((a.N + 127) / 128) * KG)) return cudaErrorInvalidValue;
    if (gather) mSFA = mSFB;      // the gather warps fetch the rows' scales themselves
    else if (!make_sf_map(&mSFA, a.sfa, (uint64_t)(a.rows_pad / BM) * KG)) return cudaErrorInvalidValue;
    const int n_nt = swiglu ? (a.N + BN / 2 - 1) / (BN / 2) : (a.N + BN - 1) / BN;
    const int k_blocks = (int)KG;
    if (pair) {
        if (swiglu && gather) return launch_one_mx<EPI_SWIGLU, true, 2>(mA, mB, mSFA, mSFB, a, n_nt, k_blocks, grid, s);
        if (swiglu) return launch_one_mx<EPI_SWIGLU, false, 2>(mA, mB, mSFA, mSFB, a, n_nt, k_blocks, grid, s);
        if (epi == EPI_BF16 && !gather) return launch_one_mx<EPI_BF16, false, 2>(mA, mB, mSFA, mSFB, a, n_nt, k_blocks, grid, s);
    } else {
        if (swiglu && gather) return launch_one_mx<EPI_SWIGLU, true, 1>(mA, mB, mSFA, mSFB, a, n_nt, k_blocks, grid, s);
        if (swiglu) return launch_one_mx<EPI_SWIGLU, false, 1>(mA, mB, mSFA, mSFB, a, n_nt, k_blocks, grid, s);
        if (epi == EPI_BF16 && !gather) return launch_one_mx<EPI_BF16, false, 1>(mA, mB, mSFA, mSFB, a, n_nt, k_blocks, grid, s);
    }
    return cudaErrorInvalidValue;
}

}  // namespace mok
