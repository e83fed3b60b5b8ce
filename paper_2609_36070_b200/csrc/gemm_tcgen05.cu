// Grouped expert GEMMs on the 5th-generation tensor cores (paper, Section 2.1: f_i(x) = W_down(phi(W_gate x) .* W_up x);
// Section 3.2: expert FFNs run as persistent, fused kernels that keep the tensor cores fed by pipelining operands).
//
// Persistent kernel, one CTA per SM, warp-specialised:
//   warp 0      TMA producer : A tile [128 x 64] and B tile (bf16, 128-byte swizzle) -> shared-memory ring
//   warp 1      MMA issuer   : tcgen05.mma.kind::f16, N = 256, K = 16, fp32 accumulators in TMEM
//                              (2 accumulator stages x 256 columns = all 512 TMEM columns)
//   warps 2..5  epilogue     : tcgen05.ld -> registers -> (SwiGLU) -> bf16 -> swizzled smem slab -> TMA store
//   warps 6..9  gather       : only in the GATHER instantiation, see below
// CTAS = 1: every CTA computes 128 x 256 tiles on its own (cta_group::1, 4 stages of 48 KB).
// CTAS = 2: two CTAs of a cluster compute one 256 x 256 tile with cta_group::2 MMAs issued by the even CTA: each CTA
//           stages its own 128 rows of A and HALF of the B tile (128 of the 256 weight rows), so a k-block moves
//           32 KB instead of 48 KB from L2 into each SM and the ring holds 6 stages.  The odd CTA's TMA loads complete
//           on the even CTA's mbarrier (its gathered rows are announced by its warp 1); tcgen05.commit multicasts
//           "stage free" / "accumulator ready" to both CTAs; each CTA drains its own 128 accumulator rows.  No TMA multicast is used.
// Tiles are handed out statically (tile L -> CTA or pair L mod grid) in the order expert, M group, N tile, M tile, so
// that CTAs running side by side share the same weight tile through L2 while an expert's activations stay L2
// resident.  The tile tables come from the on-device schedule; nothing is read back.  Every output element is
// produced by exactly one tile with a fixed k order, so results do not depend on the grid size or on timing
// (Section 3.4 "Determinism").
//
//   EPI_SWIGLU : B = [E, 2N, K]; the 256-wide B tile is 128 gate rows followed by the matching 128 up rows and the
//                epilogue writes C[:, n*128 .. n*128+127] = silu(gate) * up (bf16).
//   EPI_BF16   : B = [E, N, K]; C[:, n*256 .. n*256+255] = A . B^T (bf16).
//   EPI_F32    : as EPI_BF16 with fp32 output (router logits).
//   GATHER     : the A rows of a tile are token rows of x picked through the row -> token table of the dispatch
//                schedule: the paper's pull dispatch (Section 3.1).  Four extra gather warps copy the rows with
//                16-byte cp.async straight into the swizzled A stage (8 lanes cover one 128-byte row segment, so a
//                warp instruction reads four whole segments), and the copies' completion arrives on the stage's
//                mbarrier; the expert-sorted copy of x never exists.  (TMA tile::gather4 computes the same thing
//                but measured 2x slower here: 32 instructions of 512 bytes per k-block outrun the TMA issue rate.)
// Tried and dropped: cp.async.bulk.prefetch.tensor of the weight boxes 8-12 k-blocks ahead (by every CTA, or only by
// the CTA holding a group's first M tile) made the operand waits longer, not shorter (+13 % kernel time).
// All mbarrier waits are bounded: on a timeout the CTA records MOK_ERR_TIMEOUT and leaves cleanly.
#include "mok_internal.cuh"
#include "tc_ptx.cuh"
#include "tensor_map.cuh"
#include "tile_order.cuh"

namespace mok {
namespace tc {

constexpr int BM = 128, BN = 256, BK = 64, UMMA_K = 16;
constexpr int A_BYTES = BM * BK * 2;           // 16 KB
constexpr int B_BYTES = BN * BK * 2;           // 32 KB (whole tile; a CTA of a pair stages half of it)
constexpr int MAX_STAGES = 6;
constexpr int ACC_STAGES = 2, TMEM_COLS = 512;
constexpr int THREADS = 192;                   // + 4 gather warps in the GATHER instantiation
constexpr int GATHER_THREADS = 128;
constexpr int SMEM_CTRL = 256;
constexpr int OUT_STAGE_BYTES = 4 * 8192;      // per epilogue warp: 32 rows x 128 bf16 columns, as two swizzled boxes
constexpr int RING_BYTES = 196608;             // 4 x 48 KB or 6 x 32 KB
constexpr int SMEM_BYTES = RING_BYTES + OUT_STAGE_BYTES + SMEM_CTRL + 1024;   // + slack for 1024-byte alignment

struct Ctrl {
    uint64_t full[MAX_STAGES];     // this CTA's stage has landed (TMA bytes + gather arrivals)
    uint64_t pfull[MAX_STAGES];    // even CTA only: the odd CTA's stage has landed
    uint64_t empty[MAX_STAGES];    // the MMAs reading the stage have retired
    uint64_t tfull[ACC_STAGES];    // accumulator stage complete
    uint64_t tempty[ACC_STAGES];   // accumulator stage drained by every epilogue warp (of both CTAs)
    uint32_t tmem_base;
    uint32_t abort;
};
static_assert(sizeof(Ctrl) <= SMEM_CTRL, "control block too large");

// Instruction descriptor: D fp32, A/B bf16, both K-major, dense, M = 128 x CTAS, N = 256.
template <int CTAS>
__device__ __forceinline__ constexpr uint32_t make_idesc() {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((BM * CTAS) >> 4) << 24);
}

template <int EPI, bool GATHER, int CTAS>
__global__ void __launch_bounds__(THREADS + (GATHER ? GATHER_THREADS : 0), 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmapA, const __grid_constant__ CUtensorMap tmapB,
               const __grid_constant__ CUtensorMap tmapC, const __grid_constant__ GemmArgs a, const int n_nt, const int k_blocks) {
    constexpr bool SWIGLU = (EPI == EPI_SWIGLU);
    constexpr int STAGES = (CTAS == 2) ? 6 : 4;
    constexpr int B_STAGE = B_BYTES / CTAS;                 // B bytes this CTA stages per k-block
    constexpr int STAGE_BYTES = A_BYTES + B_STAGE;
    constexpr int TM = BM * CTAS;                           // rows of one (pair) tile
    static_assert(STAGES * STAGE_BYTES == RING_BYTES, "ring size");
    extern __shared__ uint8_t smem_raw[];
    pdl_enter();
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem + RING_BYTES + OUT_STAGE_BYTES);
    volatile uint32_t* abort_flag = &ctrl->abort;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = (CTAS == 2) ? (int)cluster_ctarank() : 0;      // 0 = the CTA that issues the MMAs
    const int unit = blockIdx.x / CTAS, n_units = gridDim.x / CTAS;   // CTA (or pair) index in the static schedule
    const bool dbg = a.dbg_slot >= 0;

    int n_mt_total = (a.dense_rows > 0) ? (a.dense_rows + TM - 1) / TM : *a.n_mtiles;
    if (n_mt_total > a.max_mt) n_mt_total = a.max_mt;
    const int total = n_mt_total * n_nt;
    // columns of an N tile: 256, or fewer for the fp32 epilogue on single CTAs (GemmArgs::n_tile: more, narrower tiles
    // when a GEMM has too few tiles to fill the GPU; every output element is still one accumulation over K)
    const int n_width = (EPI == EPI_F32 && CTAS == 1 && a.n_tile > 0) ? a.n_tile : BN;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            // arrivals per phase: the producer's expect_tx (not in the odd CTA of a pair, whose TMA bytes complete on
            // the even CTA's barrier) + one per gather thread
            const int full_arrivals = ((CTAS == 2 && rank == 1) ? 0 : 1) + (GATHER ? GATHER_THREADS : 0);
            mbar_init(smem_u32(&ctrl->full[s]), full_arrivals > 0 ? full_arrivals : 1);   // (unused when it would be 0)
            mbar_init(smem_u32(&ctrl->pfull[s]), 1);
            mbar_init(smem_u32(&ctrl->empty[s]), 1);
        }
        for (int s = 0; s < ACC_STAGES; ++s) {
            mbar_init(smem_u32(&ctrl->tfull[s]), 1);
            mbar_init(smem_u32(&ctrl->tempty[s]), 4 * CTAS);       // one arrive per epilogue warp of each CTA
        }
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
            long long dbg_prod = 0;
            const int b_rows_per_expert = (SWIGLU ? 2 : 1) * a.N;
            for (int L = unit; L < total; L += n_units) {
                const Tile t = decode_tile(a, L, n_nt, n_mt_total, TM);
                // weight rows of this tile: [gate 128 | up 128] for SwiGLU, 256 consecutive rows otherwise; a CTA
                // of a pair stages only its half (rank 0: first 128 rows, rank 1: second 128 rows)
                const int brow0 = t.e * b_rows_per_expert + (SWIGLU ? t.n * (BN / 2) : t.n * n_width);
                const int brow1 = SWIGLU ? brow0 + a.N : brow0 + BN / 2;
                bool ok = true;
                for (int kb = 0; kb < k_blocks; ++kb) {
                    const long long w0 = dbg ? clock64() : 0;
                    ok = mbar_wait(smem_u32(&ctrl->empty[s]), ph ^ 1u, abort_flag, a.header, 1);
                    if (dbg) dbg_prod += clock64() - w0;
                    if (!ok) break;
                    const uint32_t full = smem_u32(&ctrl->full[s]);
                    const uint32_t sa = base + s * STAGE_BYTES, sb = sa + A_BYTES;
                    if (CTAS == 1 && n_width <= BN / 2) {
                        // narrow N tile (fp32 epilogue only): one box of n_width weight rows
                        mbar_expect_tx(full, (GATHER ? 0 : A_BYTES) + n_width * BK * 2);
                        if (!GATHER) tma_load_2d(sa, &tmapA, full, kb * BK, t.row0);
                        tma_load_2d(sb, &tmapB, full, kb * BK, brow0);
                    } else if (CTAS == 1) {
                        mbar_expect_tx(full, GATHER ? B_STAGE : STAGE_BYTES);
                        if (!GATHER) tma_load_2d(sa, &tmapA, full, kb * BK, t.row0);
                        tma_load_2d(sb, &tmapB, full, kb * BK, brow0);
                        tma_load_2d(sb + B_BYTES / 2, &tmapB, full, kb * BK, brow1);
                    } else if (rank == 0) {
                        // the even CTA's barrier collects the TMA bytes of both CTAs of the pair
                        mbar_expect_tx(full, 2 * (GATHER ? B_STAGE : STAGE_BYTES));
                        if (!GATHER) tma_load_2d(sa, &tmapA, full, kb * BK, t.row0);
                        tma_load_2d(sb, &tmapB, full, kb * BK, brow0);
                    } else {
                        if (!GATHER) tma_load_2d_peer(sa, &tmapA, full, kb * BK, t.row0 + BM);
                        tma_load_2d_peer(sb, &tmapB, full, kb * BK, brow1);
                    }
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (!ok) break;
            }
            if (dbg) atomicAdd(&a.header->dbg[a.dbg_slot][DBG_PROD_WAIT_EMPTY], (unsigned long long)dbg_prod);
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            // -------------------------------------------------------------- MMA issuer (even CTA of a pair)
            const uint32_t idesc = (make_idesc<CTAS>() & ~(0x3Fu << 17)) | ((uint32_t)(n_width >> 3) << 17);
            int s = 0, as = 0;
            uint32_t ph = 0, aph = 0;
            long long d_full = 0, d_pfull = 0, d_tempty = 0, d_kb = 0;
            const long long d_t0 = dbg ? clock64() : 0;
            const unsigned long long d_ns0 = dbg ? globaltimer() : 0ull;
            for (int L = unit; L < total; L += n_units) {
                long long w0 = dbg ? clock64() : 0;
                bool ok = mbar_wait(smem_u32(&ctrl->tempty[as]), aph ^ 1u, abort_flag, a.header, 2);
                if (dbg) d_tempty += clock64() - w0;
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(as * BN);
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (dbg) w0 = clock64();
                    ok = mbar_wait(smem_u32(&ctrl->full[s]), ph, abort_flag, a.header, 3);
                    if (dbg) { const long long w1 = clock64(); d_full += w1 - w0; w0 = w1; ++d_kb; }
                    if (ok && CTAS == 2 && GATHER) ok = mbar_wait(smem_u32(&ctrl->pfull[s]), ph, abort_flag, a.header, 6);
                    if (dbg) d_pfull += clock64() - w0;
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t sa = base + s * STAGE_BYTES, sb = sa + A_BYTES;
                    const uint64_t adesc = make_smem_desc(sa), bdesc = make_smem_desc(sb);
#pragma unroll
                    for (int j = 0; j < BK / UMMA_K; ++j)   // +32 bytes per K=16 step inside the 128-byte swizzle row
                        tc_mma<CTAS>(d_tmem, adesc + (uint64_t)(j * 2), bdesc + (uint64_t)(j * 2), idesc, (kb | j) ? 1u : 0u);
                    tc_commit<CTAS>(smem_u32(&ctrl->empty[s]));   // frees the smem stage (in both CTAs) when these MMAs retire
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (!ok) break;
                tc_commit<CTAS>(smem_u32(&ctrl->tfull[as]));      // accumulator complete (in both CTAs)
                if (++as == ACC_STAGES) { as = 0; aph ^= 1u; }
            }
            if (dbg) {
                unsigned long long* d = a.header->dbg[a.dbg_slot];
                atomicAdd(d + DBG_MMA_WAIT_FULL, (unsigned long long)d_full);
                atomicAdd(d + DBG_MMA_WAIT_PFULL, (unsigned long long)d_pfull);
                atomicAdd(d + DBG_MMA_WAIT_TEMPTY, (unsigned long long)d_tempty);
                const unsigned long long d_tot = (unsigned long long)(clock64() - d_t0);
                atomicAdd(d + DBG_MMA_TOTAL, d_tot);
                atomicMax(d + DBG_MMA_TOTAL_MAX, d_tot);
                atomicAdd(d + DBG_MMA_TOTAL_NS, globaltimer() - d_ns0);
                atomicAdd(d + DBG_KBLOCKS, (unsigned long long)d_kb);
                atomicAdd(d + DBG_CTAS, 1ull);
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
    } else if (GATHER && warp >= 6) {
        // ------------------------------------------------------------------ gather warps 6..9 (pull dispatch)
        // Warp gw owns tile rows 32 gw .. 32 gw + 31.  Lane = (sub-row 0..3, 16-byte chunk 0..7); pass i covers rows
        // 32 gw + 4 i + sub-row.  Chunk c of row r lands at r*128 + ((c ^ (r & 7)) * 16): the 128-byte swizzle the
        // UMMA descriptor expects.  Rows past the expert's segment re-read the tile's first row (never combined).
        const int gw = warp - 6, sub = lane >> 3, chunk = lane & 7;
        int s = 0;
        uint32_t ph = 0;
        for (int L = unit; L < total; L += n_units) {
            const Tile t = decode_tile(a, L, n_nt, n_mt_total, TM);
            const int valid = __ldg(a.counts + t.e) - t.m * TM - rank * BM;
            const int tok0 = __ldg(a.row_token + t.row0);
            const int* rows = a.row_token + t.row0 + rank * BM;
            const __nv_bfloat16* src[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int r = gw * 32 + i * 4 + sub;
                const int tok = (r < valid) ? __ldg(rows + r) : tok0;
                src[i] = gather_row(a, tok) + chunk * 8;
            }
            bool ok = true;
            for (int kb = 0; kb < k_blocks; ++kb) {
                ok = mbar_wait(smem_u32(&ctrl->empty[s]), ph ^ 1u, abort_flag, a.header, 5);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const uint32_t sa = base + s * STAGE_BYTES;
                const bool in_k = (kb * BK + chunk * 8) < a.K;            // K tail: zero-fill
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int r = gw * 32 + i * 4 + sub;
                    const uint32_t dst = sa + r * 128 + ((chunk ^ (r & 7)) << 4);
                    cp_async_16(dst, in_k ? (const void*)(src[i] + kb * BK) : (const void*)a.A, in_k ? 16u : 0u);
                }
                cp_async_mbar_arrive(smem_u32(&ctrl->full[s]));
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
            if (!ok) break;
        }
        asm volatile("cp.async.wait_all;" ::: "memory");
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        // TMEM -> registers -> (SwiGLU) -> bf16 -> this warp's swizzled staging slab -> TMA store.  Each warp owns
        // 32 accumulator rows and stages 128 output columns at a time as two [32 rows x 64 columns] boxes, so the
        // global writes are whole 128-byte lines and the warp only synchronises with itself.
        const int quad = warp & 3;                            // TMEM lane quadrant this warp may access
        const uint32_t slab = base + RING_BYTES + quad * 8192;
        int as = 0;
        uint32_t aph = 0;
        long long d_tfull = 0;
        const long long d_e0 = dbg ? clock64() : 0;
        for (int L = unit; L < total; L += n_units) {
            const Tile t = decode_tile(a, L, n_nt, n_mt_total, TM);
            const long long w0 = dbg ? clock64() : 0;
            bool ok = mbar_wait(smem_u32(&ctrl->tfull[as]), aph, abort_flag, a.header, 4);
            if (dbg) d_tfull += clock64() - w0;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(as * BN);
            const int row = t.row0 + rank * BM + quad * 32;
            if (EPI == EPI_F32) {
                float* frow = reinterpret_cast<float*>(a.C) + (size_t)(row + lane) * a.ldc;
                const int c0 = t.n * n_width;
#pragma unroll 1
                for (int c = 0; c < n_width; c += 32) {
                    uint32_t r[32];
                    tc_ld32(taddr + c, r);
                    tc_wait_ld();
#pragma unroll
                    for (int v = 0; v < 8; ++v) {
                        const int col = c0 + c + v * 4;
                        if (col < a.N)
                            *reinterpret_cast<uint4*>(frow + col) = make_uint4(r[4 * v], r[4 * v + 1], r[4 * v + 2], r[4 * v + 3]);
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (rank == 0) mbar_arrive(smem_u32(&ctrl->tempty[as]));
                    else mbar_arrive_remote(smem_u32(&ctrl->tempty[as]), 0);
                }
            } else {
                constexpr int HALVES = SWIGLU ? 1 : 2;        // 128 output columns per pass
                const int c0 = SWIGLU ? t.n * (BN / 2) : t.n * BN;
#pragma unroll 1
                for (int half = 0; half < HALVES; ++half) {
                    if (lane == 0) tma_store_wait_read();     // the slab's previous stores have been read out
                    __syncwarp();
#pragma unroll 1
                    for (int c = 0; c < 128; c += 32) {
                        uint32_t o[16];
                        if (SWIGLU) {
                            uint32_t g[32], u[32];
                            tc_ld32(taddr + c, g);
                            tc_ld32(taddr + BN / 2 + c, u);
                            tc_wait_ld();
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                float g0 = __uint_as_float(g[2 * i]), g1 = __uint_as_float(g[2 * i + 1]);
                                float h0 = swiglu(g0, __uint_as_float(u[2 * i]));
                                float h1 = swiglu(g1, __uint_as_float(u[2 * i + 1]));
                                o[i] = pack_bf16(h0, h1);
                            }
                        } else {
                            uint32_t r[32];
                            tc_ld32(taddr + half * 128 + c, r);
                            tc_wait_ld();
#pragma unroll
                            for (int i = 0; i < 16; ++i) o[i] = pack_bf16(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
                        }
                        // 32 columns = 4 chunks of 16 bytes in box (c / 64), chunk index ((c % 64) / 8 + v)
                        const uint32_t box = slab + (c >> 6) * 4096 + lane * 128;
#pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            const int cc = ((c & 63) >> 3) + v;
                            st_shared_v4(box + ((cc ^ (lane & 7)) << 4), o[4 * v], o[4 * v + 1], o[4 * v + 2], o[4 * v + 3]);
                        }
                    }
                    if (half == HALVES - 1) tc_fence_before();   // all TMEM reads of this tile are done
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) {
                        if (half == HALVES - 1) {             // hand the accumulator stage back to the MMA issuer
                            if (rank == 0) mbar_arrive(smem_u32(&ctrl->tempty[as]));
                            else mbar_arrive_remote(smem_u32(&ctrl->tempty[as]), 0);
                        }
                        const int col = c0 + half * 128;
                        if (col < a.N) tma_store_2d(&tmapC, slab, col, row);
                        if (col + 64 < a.N) tma_store_2d(&tmapC, slab + 4096, col + 64, row);
                        tma_store_commit();
                    }
                }
            }
            if (++as == ACC_STAGES) { as = 0; aph ^= 1u; }
        }
        if (lane == 0) tma_store_wait_all();
        __syncwarp();
        if (dbg && warp == 2 && lane == 0) {
            atomicAdd(&a.header->dbg[a.dbg_slot][DBG_EPI_WAIT_TFULL], (unsigned long long)d_tfull);
            atomicAdd(&a.header->dbg[a.dbg_slot][DBG_EPI_TOTAL], (unsigned long long)(clock64() - d_e0));
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

// 2D bf16 row-major tensor [rows, cols] -> tensor map with a [box_rows x 64] box and 128-byte swizzle.
static bool make_map(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows,
                     uint64_t row_stride_elems = 0) {
    return tmap::bf16_sw128(m, ptr, rows, cols, box_rows, row_stride_elems);
}

}  // namespace tc

// Grid of the persistent kernel: one CTA per SM, or as many CTA pairs as can be co-resident.
template <int EPI, bool GATHER, int CTAS>
static cudaError_t launch_one(const CUtensorMap& mA, const CUtensorMap& mB, const CUtensorMap& mC, const GemmArgs& a,
                              int n_nt, int k_blocks, int grid, cudaStream_t s) {
    using namespace tc;
    static PerDevice configured;      // per device: CTAs (or CTA pairs) of the persistent grid, once configured there
    int max_units = 0;
    const int threads = THREADS + (GATHER ? GATHER_THREADS : 0);
    auto kernel = gemm_tc_kernel<EPI, GATHER, CTAS>;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    cfg.blockDim = dim3(threads);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = s;
    cfg.numAttrs = 0;
    if (CTAS == 1 && g_pdl) {     // single CTAs: programmatically serialised with the kernel before (see pdl_enter)
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
    }
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
    return cudaLaunchKernelEx(&cfg, kernel, mA, mB, mC, a, n_nt, k_blocks);
}

cudaError_t launch_gemm_tc(const GemmArgs& a, int epi, int grid, cudaStream_t s) {
    using namespace tc;
    const bool swiglu = (epi == EPI_SWIGLU), gather = (a.row_token != nullptr), pair = (a.tile_m == 2 * BM);
    if (a.tile_m != BM && a.tile_m != 2 * BM) return cudaErrorInvalidValue;
    CUtensorMap mA, mB, mC;
    const uint64_t b_rows = (uint64_t)a.E * (swiglu ? 2 : 1) * a.N;
    if (!make_map(&mA, a.A, (uint64_t)a.a_rows, (uint64_t)a.K, BM)) return cudaErrorInvalidValue;
    int n_width = BN;
    if (a.n_tile > 0) {     // narrower N tiles: fp32 epilogue, single CTAs, 32 / 64 / 128 columns
        if (epi != EPI_F32 || pair || gather || (a.n_tile != 32 && a.n_tile != 64 && a.n_tile != 128)) return cudaErrorInvalidValue;
        n_width = a.n_tile;
    }
    if (!make_map(&mB, a.B, b_rows, (uint64_t)a.K, n_width < BN / 2 ? n_width : BN / 2)) return cudaErrorInvalidValue;
    if (epi == EPI_F32) mC = mB;      // the fp32 epilogue stores directly
    else if (!make_map(&mC, a.C, (uint64_t)a.rows_pad, (uint64_t)a.N, 32, (uint64_t)a.ldc)) return cudaErrorInvalidValue;
    const int n_nt = swiglu ? (a.N + BN / 2 - 1) / (BN / 2) : (a.N + n_width - 1) / n_width;
    const int k_blocks = (a.K + BK - 1) / BK;
    if (pair) {
        if (epi == EPI_SWIGLU && gather) return launch_one<EPI_SWIGLU, true, 2>(mA, mB, mC, a, n_nt, k_blocks, grid, s);
        if (epi == EPI_SWIGLU) return launch_one<EPI_SWIGLU, false, 2>(mA, mB, mC, a, n_nt, k_blocks, grid, s);
        if (epi == EPI_BF16 && !gather) return launch_one<EPI_BF16, false, 2>(mA, mB, mC, a, n_nt, k_blocks, grid, s);
        if (epi == EPI_F32 && !gather) return launch_one<EPI_F32, false, 2>(mA, mB, mC, a, n_nt, k_blocks, grid, s);
    } else {
        if (epi == EPI_SWIGLU && gather) return launch_one<EPI_SWIGLU, true, 1>(mA, mB, mC, a, n_nt, k_blocks, grid, s);
        if (epi == EPI_SWIGLU) return launch_one<EPI_SWIGLU, false, 1>(mA, mB, mC, a, n_nt, k_blocks, grid, s);
        if (epi == EPI_BF16 && !gather) return launch_one<EPI_BF16, false, 1>(mA, mB, mC, a, n_nt, k_blocks, grid, s);
        if (epi == EPI_BF16) return launch_one<EPI_BF16, true, 1>(mA, mB, mC, a, n_nt, k_blocks, grid, s);
        if (epi == EPI_F32 && !gather) return launch_one<EPI_F32, false, 1>(mA, mB, mC, a, n_nt, k_blocks, grid, s);
    }
    return cudaErrorInvalidValue;
}

}  // namespace mok
