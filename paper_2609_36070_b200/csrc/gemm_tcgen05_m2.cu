// Grouped expert GEMMs, 256-row tiles in ONE CTA (paper, Section 2.1: the expert FFN; Section 3 cost model: keep the
// tensor cores fed, T_comp, against the memory system, T_mem).
//
// The 128 x 256 kernel (gemm_tcgen05.cu) moves 48 KB per k-block and can hold four such stages; measured on B200 that
// is not enough bytes in flight to cover the ~1.4 us from TMA issue to landed data, and its MMA issuer waits for
// operands 20-30 % of the time.  Here a tile is TWO 128-row halves that share one 256-row weight tile: per k-block
// 16 + 16 KB of activations and 32 KB of weights feed twice the MMA work, so every stage in flight carries 1024
// tensor-pipe cycles instead of 512 (three 64 KB stages), and a third less data crosses L2 -> SM per FLOP.  This is
// what a CTA pair (cta_group::2) buys, without any cross-CTA signalling.  The price: both accumulators (2 x 256 TMEM
// columns) belong to one tile, so the epilogue of a tile does not overlap the next tile's MMAs; eight epilogue warps
// (four per accumulator) keep that bubble to the time it takes to read the accumulators out of TMEM.  The second half
// of a tile is skipped when the expert's remaining rows fit in the first, so expert segments are still padded to 128
// rows only.
//
//   warp 0        TMA producer : A halves (unless gathered) and the B tile -> 3-stage ring
//   warp 1        MMA issuer   : per k-block 4 MMAs into accumulator 0 and, for a two-half tile, 4 into accumulator 1
//   warps 2..5    epilogue of accumulator 0 (rows 0..127 of the tile);  warps 6..9: accumulator 1 (rows 128..255)
//   warps 10..13  gather (GATHER only): token rows of x through the schedule's row -> token table (pull dispatch,
//                 Section 3.1), 16-byte cp.async into the swizzled A halves
// Tile order, epilogue variants (EPI_SWIGLU / EPI_BF16 / EPI_F32), determinism and the bounded waits are those of
// gemm_tcgen05.cu.
#include "mok_internal.cuh"
#include "tc_ptx.cuh"
#include "tensor_map.cuh"

namespace mok {
namespace m2 {

using namespace tc;

constexpr int BM = 128, BN = 256, BK = 64, UMMA_K = 16, STAGES = 3;
constexpr int A_BYTES = BM * BK * 2;           // 16 KB per half
constexpr int B_BYTES = BN * BK * 2;           // 32 KB
constexpr int STAGE_BYTES = 2 * A_BYTES + B_BYTES;   // 64 KB
constexpr int TM = 2 * BM;                     // rows of a full tile
constexpr int TMEM_COLS = 512;
constexpr int EPI_WARPS = 8;
constexpr int THREADS = 64 + 32 * EPI_WARPS;   // producer + MMA + epilogue warps = 320
constexpr int GATHER_THREADS = 128;
constexpr int GROUP_TILES = 8;                 // 2048 rows per rasterisation group
constexpr int SLAB_BYTES = 4096;               // per epilogue warp: 32 rows x 64 bf16 columns (one swizzled box)
constexpr int SMEM_CTRL = 512;
constexpr int QSLOTS = 2;                      // tile ids the hardware scheduler hands out ahead (stolen mode)
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_WARPS * SLAB_BYTES + SMEM_CTRL + 1024;

struct Ctrl {
    uint64_t full[STAGES], empty[STAGES];
    uint64_t tfull[2], tempty[2];              // per accumulator
    uint32_t tmem_base, abort;
    // stolen mode (cluster launch control): the scheduler warp's queue of tile ids for the roles of this CTA
    alignas(16) uint8_t clc_response[16];
    uint64_t clc_done, q_full[QSLOTS], q_empty[QSLOTS];
    int32_t q_tile[QSLOTS];
};
static_assert(sizeof(Ctrl) <= SMEM_CTRL, "control block too large");

constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);

// valid: real rows of this tile (1..256); > 128 => both halves.  row0: first A row and first C row.  In the
// K-range mode (weight gradients, see GemmArgs::kgroup_rows) the A rows and the C rows differ and the contraction
// runs over kcol0 .. kcol0 + 64 kblocks of the operands' column space.
struct Tile { int e, n, row0, valid, crow0, kcol0, kblocks, gang_first, gang_size; };

template <bool KGROUP>
__device__ __forceinline__ Tile decode_tile(const GemmArgs& a, int L, int n_nt, int n_mt_total, int k_blocks) {
    Tile t;
    if (KGROUP) {
        // one output matrix [kgroup_rows, N] per expert; tiles in the order expert, N tile, M tile
        const int m_tiles = (a.kgroup_rows + TM - 1) / TM;
        const int per_e = m_tiles * n_nt;
        t.e = L / per_e;
        const int rem = L - t.e * per_e;
        t.n = rem / m_tiles;
        const int m = rem - t.n * m_tiles;
        t.row0 = m * TM;
        t.crow0 = t.e * a.kgroup_rows + m * TM;
        t.valid = min(TM, a.kgroup_rows - m * TM);
        t.gang_first = L;
        t.gang_size = 1;
        if (a.dense_rows > 0) {            // one group over all rows (shared expert)
            t.kcol0 = 0;
            t.kblocks = (a.dense_rows + 63) / 64;
        } else {                           // the expert's padded segment of the dispatch space
            t.kcol0 = __ldg(a.pad_offsets + t.e);
            t.kblocks = (__ldg(a.pad_offsets + t.e + 1) - t.kcol0) / 64;
        }
        return t;
    }
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
    t.gang_first = L - (rem - t.n * in_group);     // the in_group tiles [N tile][M tile 0 .. in_group) use one weight tile
    t.gang_size = in_group;
    t.row0 = pad0 + m * TM;
    t.crow0 = t.row0;
    t.valid = min(TM, cnt - m * TM);
    t.kcol0 = 0;
    t.kblocks = k_blocks;
    return t;
}

// Shared-memory matrix descriptor of an MN-major bf16 operand tile (the N index contiguous in global memory): groups of
// 64 N-elements x 64 K-rows, each a [K row][128 bytes] block with the 128-byte swizzle; consecutive N groups are
// `group_bytes` apart (leading byte offset), consecutive groups of 8 K-rows 1024 bytes (stride byte offset).
__device__ __forceinline__ uint64_t make_smem_desc_mn(uint32_t addr, uint32_t group_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(group_bytes >> 4) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// How a role walks over its tiles.  Static mode: tile L -> CTA L mod grid of a persistent grid.  Stolen mode (paper,
// Section 3.4 "Cluster Launch Control"): the grid has one CTA per tile; a CTA that runs computes its own tile and
// then cancels CTAs that have not started yet and computes theirs (clusterlaunchcontrol.try_cancel: hardware work
// stealing) -- CTAs come and go at tile granularity, so other work can get onto the SMs between them.  The scheduler
// warp steals; the other roles read the stolen ids from a two-entry queue in shared memory (bounded waits; an entry
// is released once every role has read it).  Ids at or past `total` (the grid is a host-side upper bound) are skipped.
template <bool CLC>
struct TileSeq {
    Ctrl* ctrl;
    volatile uint32_t* abort_flag;
    WsHeader* hdr;
    int total, slot;
    uint32_t ph;
    bool warp_role;       // all 32 lanes call next() together (epilogue, gather) / one lane calls it (producer, issuer)
    __device__ __forceinline__ TileSeq(Ctrl* c, volatile uint32_t* af, WsHeader* h, int tot, bool wr)
        : ctrl(c), abort_flag(af), hdr(h), total(tot), slot(0), ph(0), warp_role(wr) {}
    __device__ __forceinline__ int first() {
        if (!CLC) return blockIdx.x;
        return (int)blockIdx.x < total ? (int)blockIdx.x : next(0);
    }
    __device__ __forceinline__ int next(int L) {
        if (!CLC) return L + gridDim.x;
        bool ok = mbar_wait(smem_u32(&ctrl->q_full[slot]), ph, abort_flag, hdr, 30);
        if (warp_role) ok = __all_sync(0xffffffffu, ok);
        if (!ok) return total;
        const int t = *reinterpret_cast<volatile int32_t*>(&ctrl->q_tile[slot]);
        if (warp_role) __syncwarp();
        if (!warp_role || (threadIdx.x & 31) == 0) mbar_arrive(smem_u32(&ctrl->q_empty[slot]));
        if (++slot == QSLOTS) { slot = 0; ph ^= 1u; }
        return t < 0 ? total : t;
    }
};

// MODE 0: forward layout.  MODE 1 (KGROUP): the K-range mode (weight gradients).  MODE 2 (BMN): B is read MN-major,
// i.e. W[e] is [K, N] with N contiguous -- the weights as they sit in memory serve the transposed products of the
// backward pass (dL/dh = dy Wd, dXg = [dg|du] Wgu) without a transposed copy.  Compiled separately so that the
// forward kernels carry none of it.
template <int EPI, bool GATHER, int MODE, bool CLC>
__global__ void __launch_bounds__(THREADS + (GATHER ? GATHER_THREADS : 0) + (CLC ? 32 : 0), 1)
gemm_m2_kernel(const __grid_constant__ CUtensorMap tmapA, const __grid_constant__ CUtensorMap tmapB,
               const __grid_constant__ CUtensorMap tmapC, const __grid_constant__ CUtensorMap tmapB64,
               const __grid_constant__ GemmArgs a, const int n_nt, const int k_blocks) {
    constexpr bool SWIGLU = (EPI == EPI_SWIGLU);
    // MODE 3: the K-range mode with BOTH operands read MN-major: A = [rows of the dispatch space, M] and
    // B = [rows, N] as the backward pass produces them, no transposed copies
    constexpr bool KGROUP = (MODE == 1 || MODE == 3), BMN = (MODE == 2 || MODE == 3), AMN = (MODE == 3);
    pdl_enter();
    // SwiGLU tiles are [gate 128 | up 128] weight rows.  When the last N tile has at most 64 real columns (I mod 128 in
    // 1..64) it is loaded as [gate 64 | up 64] through a 64-row box and issued as an N = 128 MMA: half the tensor-pipe
    // time and half the weight bytes for the same outputs.
    const int last_cols = SWIGLU ? a.N - (n_nt - 1) * (BN / 2) : 0;
    const bool narrow_last = SWIGLU && MODE == 0 && last_cols <= BN / 4;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem + STAGES * STAGE_BYTES + EPI_WARPS * SLAB_BYTES);
    volatile uint32_t* abort_flag = &ctrl->abort;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    int n_mt_total = (a.dense_rows > 0) ? (a.dense_rows + TM - 1) / TM : *a.n_mtiles;
    if (n_mt_total > a.max_mt) n_mt_total = a.max_mt;
    const int total = KGROUP ? a.E * ((a.kgroup_rows + TM - 1) / TM) * n_nt : n_mt_total * n_nt;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(smem_u32(&ctrl->full[s]), GATHER ? 1 + GATHER_THREADS : 1);
            mbar_init(smem_u32(&ctrl->empty[s]), 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(smem_u32(&ctrl->tfull[s]), 1);
            mbar_init(smem_u32(&ctrl->tempty[s]), 4);           // one arrive per epilogue warp of that accumulator
        }
        if (CLC) {
            mbar_init(smem_u32(&ctrl->clc_done), 1);
            for (int q = 0; q < QSLOTS; ++q) {
                mbar_init(smem_u32(&ctrl->q_full[q]), 1);
                mbar_init(smem_u32(&ctrl->q_empty[q]), 2 + EPI_WARPS + (GATHER ? GATHER_THREADS / 32 : 0));   // every role
            }
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
        if (lane == 0 && !a.starve) {
            int s = 0;
            uint32_t ph = 0;
            const int b_rows_per_expert = (SWIGLU ? 2 : 1) * a.N;
            TileSeq<CLC> seq(ctrl, abort_flag, a.header, total, false);
            for (int L = seq.first(); L < total; L = seq.next(L)) {
                const Tile t = decode_tile<KGROUP>(a, L, n_nt, n_mt_total, k_blocks);
                const bool two = t.valid > BM;
                if (!KGROUP && !CLC && a.gang && t.gang_size > 1) {
                    // The row tiles of one expert that use the same weight tile sit at consecutive list positions, i.e.
                    // on neighbouring CTAs.  They only share that weight tile through L2 if they stream it at the same
                    // time; tiles of different length (an expert's last, half-empty row tile) pull the CTAs apart, each
                    // then fetches its own copy from DRAM, the extra traffic shortens the time a line stays in L2, and
                    // the grid never finds back (measured on the DeepSeek-like layer: 67 GB read per launch for 20 GB
                    // of operands).  So the producers of such a gang start the tile together: one arrival each on the
                    // gang's counter, then a bounded wait for the others.  No deadlock: a gang's members (consecutive
                    // list positions, at most GROUP_TILES of them) are on different CTAs because the grid is at
                    // least that large (the launcher checks), every CTA walks its tiles in list order, and the launch
                    // is cooperative (all CTAs resident) -- the first gang that is not yet complete only waits for
                    // CTAs that are busy with tiles of gangs before it.
                    int32_t* cnt = a.gang + t.gang_first;
                    asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(cnt) : "memory");
                    const unsigned long long t0 = globaltimer();
                    uint32_t spins = 0;
                    bool alive = true;
                    int seen;
                    for (;;) {
                        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(cnt) : "memory");
                        if (seen >= t.gang_size) break;
                        if ((++spins & 63u) == 0u) {
                            if (*abort_flag) { alive = false; break; }
                            const unsigned long long limit =
                                a.header->wait_limit_us ? 1000ull * a.header->wait_limit_us : WAIT_LIMIT_NS;
                            if (globaltimer() - t0 > limit) {
                                *abort_flag = 1u;
                                atomicCAS(&a.header->status, 0, (int)MOK_ERR_TIMEOUT);
                                a.header->where = 42;
                                alive = false;
                                break;
                            }
                        }
                    }
                    if (!alive) break;
                }
                // weight rows of this tile; in the K-range mode B is an activation matrix shared by all experts
                const int brow0 = KGROUP ? t.n * BN
                                                      : t.e * b_rows_per_expert + (SWIGLU ? t.n * (BN / 2) : t.n * BN);
                const int brow1 = SWIGLU ? brow0 + a.N : brow0 + BN / 2;
                bool ok = true;
                for (int kb = 0; kb < t.kblocks; ++kb) {
                    ok = mbar_wait(smem_u32(&ctrl->empty[s]), ph ^ 1u, abort_flag, a.header, 1);
                    if (!ok) break;
                    const uint32_t full = smem_u32(&ctrl->full[s]);
                    const uint32_t sa = base + s * STAGE_BYTES, sb = sa + 2 * A_BYTES;
                    // GATHER: the gather warps bring A (forward layout), or in MODE 3 the operand a.gather_mn names
                    const bool gA = GATHER && (!AMN || a.gather_mn == 1), gB = GATHER && AMN && a.gather_mn == 2;
                    const bool narrow = narrow_last && t.n == n_nt - 1;
                    mbar_expect_tx(full, (gB ? 0 : (narrow ? B_BYTES / 2 : B_BYTES)) + (gA ? 0 : (two ? 2 : 1) * A_BYTES));
                    if (AMN && !gA) {   // per half two boxes of 64 M-columns x 64 K-rows (K = rows of the dispatch space)
                        tma_load_2d(sa, &tmapA, full, t.row0, t.kcol0 + kb * BK);
                        tma_load_2d(sa + A_BYTES / 2, &tmapA, full, t.row0 + 64, t.kcol0 + kb * BK);
                        if (two) {
                            tma_load_2d(sa + A_BYTES, &tmapA, full, t.row0 + BM, t.kcol0 + kb * BK);
                            tma_load_2d(sa + A_BYTES + A_BYTES / 2, &tmapA, full, t.row0 + BM + 64, t.kcol0 + kb * BK);
                        }
                    } else if (!AMN && !GATHER) {
                        tma_load_2d(sa, &tmapA, full, t.kcol0 + kb * BK, t.row0);
                        if (two) tma_load_2d(sa + A_BYTES, &tmapA, full, t.kcol0 + kb * BK, t.row0 + BM);
                    }
                    if (gB) {
                    } else if (BMN) {   // four boxes of 64 N-columns x 64 K-rows: W[e] viewed as [E * K, N], or the shared B rows
                        const int krow = AMN ? t.kcol0 + kb * BK : t.e * a.K + kb * BK;
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            tma_load_2d(sb + q * (B_BYTES / 4), &tmapB, full, t.n * BN + q * 64, krow);
                    } else if (narrow) {
                        tma_load_2d(sb, &tmapB64, full, t.kcol0 + kb * BK, brow0);
                        tma_load_2d(sb + B_BYTES / 4, &tmapB64, full, t.kcol0 + kb * BK, brow1);
                    } else {
                        tma_load_2d(sb, &tmapB, full, t.kcol0 + kb * BK, brow0);
                        tma_load_2d(sb + B_BYTES / 2, &tmapB, full, t.kcol0 + kb * BK, brow1);
                    }
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (!ok) break;
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0, ap0 = 0, ap1 = 0;        // phases of tempty[0], tempty[1]: they advance per use
            const bool dbg = a.dbg_slot >= 0;
            long long d_full = 0, d_tempty = 0, d_kb = 0, d_rows = 0;
            const long long d_t0 = dbg ? clock64() : 0;
            const unsigned long long d_ns0 = dbg ? globaltimer() : 0ull;
            TileSeq<CLC> seq(ctrl, abort_flag, a.header, total, false);
            for (int L = seq.first(); L < total; L = seq.next(L)) {
                const Tile t = decode_tile<KGROUP>(a, L, n_nt, n_mt_total, k_blocks);
                if (KGROUP && t.kblocks == 0) continue;       // K-range mode: an expert without rows (output pre-zeroed)
                const bool two = t.valid > BM;
                // the last N tile of a plain output may be narrower than 256 columns: the MMA is told so (its duration is
                // proportional to N); the columns past it are never stored.  (A SwiGLU tile is [gate 128 | up 128].)
                constexpr uint32_t IDESC_K = IDESC | (BMN ? (1u << 16) : 0u) | (AMN ? (1u << 15) : 0u);
                uint32_t idesc = IDESC_K;
                if (!SWIGLU && a.N - t.n * BN < BN)
                    idesc = (IDESC_K & ~(0x3Fu << 17)) | ((uint32_t)(((a.N - t.n * BN + 15) & ~15) >> 3) << 17);
                if (narrow_last && t.n == n_nt - 1)
                    idesc = (IDESC_K & ~(0x3Fu << 17)) | ((uint32_t)((BN / 2) >> 3) << 17);
                long long w0 = dbg ? clock64() : 0;
                // Accumulator 0 is needed now, accumulator 1 only after the first k-block's MMAs into accumulator 0; and
                // accumulator 0 is published before the last k-block's MMAs into accumulator 1 are issued.  Each
                // accumulator's epilogue thus gets one k-block (512 tensor-pipe cycles) more to drain.
                bool ok = mbar_wait(smem_u32(&ctrl->tempty[0]), ap0 ^ 1u, abort_flag, a.header, 2);
                if (dbg) d_tempty += clock64() - w0;
                if (!ok) break;
                tc_fence_after();
                const uint32_t d0 = tmem_base, d1 = tmem_base + BN;
                for (int kb = 0; kb < t.kblocks; ++kb) {
                    if (dbg) w0 = clock64();
                    ok = mbar_wait(smem_u32(&ctrl->full[s]), ph, abort_flag, a.header, 3);
                    if (dbg) { d_full += clock64() - w0; d_kb += two ? 2 : 1; }
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t sa = base + s * STAGE_BYTES;
                    const uint64_t a0 = AMN ? make_smem_desc_mn(sa, A_BYTES / 2) : make_smem_desc(sa);
                    const uint64_t a1 = AMN ? make_smem_desc_mn(sa + A_BYTES, A_BYTES / 2) : make_smem_desc(sa + A_BYTES);
                    constexpr uint32_t ASTEP = AMN ? (2048 >> 4) : 2;
                    // K-major B: +32 bytes per K = 16 step inside the swizzled row; MN-major B: +2 groups of 8 K-rows
                    const uint64_t bd = BMN ? make_smem_desc_mn(sa + 2 * A_BYTES, B_BYTES / 4) : make_smem_desc(sa + 2 * A_BYTES);
                    constexpr uint32_t BSTEP = BMN ? (2048 >> 4) : 2;
#pragma unroll
                    for (int j = 0; j < BK / UMMA_K; ++j)
                        tc_mma<1>(d0, a0 + (uint64_t)(j * ASTEP), bd + (uint64_t)(j * BSTEP), idesc, (kb | j) ? 1u : 0u);
                    if (kb == t.kblocks - 1) { tc_commit<1>(smem_u32(&ctrl->tfull[0])); ap0 ^= 1u; }
                    if (two) {
                        if (kb == 0) {
                            if (dbg) w0 = clock64();
                            ok = mbar_wait(smem_u32(&ctrl->tempty[1]), ap1 ^ 1u, abort_flag, a.header, 8);
                            if (dbg) d_tempty += clock64() - w0;
                            if (!ok) break;
                            tc_fence_after();
                        }
#pragma unroll
                        for (int j = 0; j < BK / UMMA_K; ++j)
                            tc_mma<1>(d1, a1 + (uint64_t)(j * ASTEP), bd + (uint64_t)(j * BSTEP), idesc, (kb | j) ? 1u : 0u);
                    }
                    tc_commit<1>(smem_u32(&ctrl->empty[s]));
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (!ok) break;
                if (two) { tc_commit<1>(smem_u32(&ctrl->tfull[1])); ap1 ^= 1u; }
                if (dbg) d_rows += (long long)t.valid * t.kblocks;
            }
            if (dbg) {   // k_blocks counted in 128-row units so that the figures compare with the 128-row kernel
                unsigned long long* d = a.header->dbg[a.dbg_slot];
                atomicAdd(d + DBG_MMA_WAIT_FULL, (unsigned long long)d_full);
                atomicAdd(d + DBG_MMA_WAIT_TEMPTY, (unsigned long long)d_tempty);
                const unsigned long long d_tot = (unsigned long long)(clock64() - d_t0);
                atomicAdd(d + DBG_MMA_TOTAL, d_tot);
                atomicMax(d + DBG_MMA_TOTAL_MAX, d_tot);
                atomicAdd(d + DBG_MMA_TOTAL_NS, globaltimer() - d_ns0);
                atomicAdd(d + DBG_KBLOCKS, (unsigned long long)d_kb);
                atomicAdd(d + DBG_ROWS_KB, (unsigned long long)d_rows);
                atomicAdd(d + DBG_CTAS, 1ull);
            }
        }
        __syncwarp();
    } else if (CLC && warp == (THREADS + (GATHER ? GATHER_THREADS : 0)) / 32) {
        // ------------------------------------------------------------------ scheduler (stolen mode): steals tile ids
        if (lane == 0) {
            int slot = 0;
            uint32_t qph = 0, cph = 0;
            bool more = true;
            while (more) {
                int tile = -1;
                bool ok = true;
                while (ok) {
                    mbar_expect_tx(smem_u32(&ctrl->clc_done), 16);
                    asm volatile("clusterlaunchcontrol.try_cancel.async.shared::cta.mbarrier::complete_tx::bytes.b128 [%0], [%1];"
                                 ::"r"(smem_u32(ctrl->clc_response)), "r"(smem_u32(&ctrl->clc_done)) : "memory");
                    ok = mbar_wait(smem_u32(&ctrl->clc_done), cph, abort_flag, a.header, 31);
                    cph ^= 1u;
                    if (!ok) break;
                    uint32_t canceled = 0, bx = 0;
                    asm volatile("{\n\t.reg .b128 r;\n\t.reg .pred p;\n\t"
                                 "ld.shared.b128 r, [%2];\n\t"
                                 "clusterlaunchcontrol.query_cancel.is_canceled.pred.b128 p, r;\n\t"
                                 "selp.u32 %0, 1, 0, p;\n\t"
                                 "@p clusterlaunchcontrol.query_cancel.get_first_ctaid::x.b32.b128 %1, r;\n\t}"
                                 : "=r"(canceled), "=r"(bx) : "r"(smem_u32(ctrl->clc_response)) : "memory");
                    // refused: nothing is left to steal, or work of a higher stream priority is waiting for an SM -- then this
                    // CTA leaves and the tiles nobody stole start as CTAs of their own afterwards.  (No request may follow a
                    // refused one.)
                    if (!canceled) break;
                    if ((int)bx < total) { tile = (int)bx; break; }
                }
                if (!ok) break;
                if (!mbar_wait(smem_u32(&ctrl->q_empty[slot]), qph ^ 1u, abort_flag, a.header, 32)) break;
                *reinterpret_cast<volatile int32_t*>(&ctrl->q_tile[slot]) = tile;
                mbar_arrive(smem_u32(&ctrl->q_full[slot]));   // release semantics order the id before the arrive
                if (++slot == QSLOTS) { slot = 0; qph ^= 1u; }
                more = tile >= 0;
            }
        }
        __syncwarp();
    } else if (GATHER && warp >= 2 + EPI_WARPS && warp < 2 + EPI_WARPS + GATHER_THREADS / 32) {
        // ------------------------------------------------------------------ gather warps (pull dispatch)
        // Warp gw owns rows 32 gw .. 32 gw + 31 of each half; lane = (sub-row 0..3, 16-byte chunk 0..7); pass i of half
        // h covers row 128 h + 32 gw + 4 i + sub-row.  Chunk c of row r lands at r*128 + ((c ^ (r & 7)) * 16) inside
        // its half.  Rows past the expert's segment are written as zeros: their products are never combined, and zero
        // operands cost the tensor pipe far less power than live ones (the board runs at its power cap, so power
        // spent on padding is clock taken from the real rows).
        const int gw = warp - (2 + EPI_WARPS), sub = lane >> 3, chunk = lane & 7;
        int s = 0;
        uint32_t ph = 0;
        TileSeq<CLC> seq(ctrl, abort_flag, a.header, total, true);
        if (AMN) {
            // MODE 3 (weight gradients): the gathered operand is read MN-major, K = rows of the dispatch space.  One
            // k-block = 64 dispatch rows x 256 columns of x or dout, laid out as four 64-column groups of [K row][128
            // bytes] (chunk c of row kr at kr*128 + ((c ^ (kr & 7)) * 16) of its group), as the MMA descriptors expect.
            // Warp gw owns rows 16 gw .. 16 gw + 15; lane = (sub-row 0..3, 16-byte chunk 0..7), so eight lanes read 128
            // contiguous bytes of one row; a thread copies 4 rows x 4 column groups per k-block.  Rows past the expert's
            // count are written as zeros: they must not contribute to the sums over rows.  The row ids of the next two
            // k-blocks are loaded ahead.
            const bool gB = a.gather_mn == 2;
            const __nv_bfloat16* mat = gB ? a.B : a.A;
            const int ld = gB ? (a.ldb ? a.ldb : a.K) : (a.lda ? a.lda : a.K);
            const int col_lim = gB ? a.N : a.kgroup_rows;
            const uint32_t obase = gB ? 2u * A_BYTES : 0u;
            for (int L = seq.first(); L < total; L = seq.next(L)) {
                const Tile t = decode_tile<KGROUP>(a, L, n_nt, n_mt_total, k_blocks);
                if (t.kblocks == 0) continue;
                const bool second = gB || t.valid > BM;      // column groups 2, 3 are in use
                const int cnt = __ldg(a.counts + t.e);
                const int colbase = (gB ? t.n * BN : t.row0) + chunk * 8;
                const int32_t* rt = a.row_token + t.kcol0 + gw * 16 + sub;
                int tok_cur[4], tok_nxt[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int r = gw * 16 + q * 4 + sub;
                    tok_cur[q] = (r < cnt) ? __ldg(rt + q * 4) : -1;
                    tok_nxt[q] = (t.kblocks > 1 && 64 + r < cnt) ? __ldg(rt + 64 + q * 4) : -1;
                }
                bool ok = true;
                for (int kb = 0; kb < t.kblocks; ++kb) {
                    int tok_n2[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int r = (kb + 2) * 64 + gw * 16 + q * 4 + sub;
                        tok_n2[q] = (kb + 2 < t.kblocks && r < cnt) ? __ldg(rt + (kb + 2) * 64 + q * 4) : -1;
                    }
                    ok = mbar_wait(smem_u32(&ctrl->empty[s]), ph ^ 1u, abort_flag, a.header, 5);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    const uint32_t stage = base + s * STAGE_BYTES + obase;
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int kr = gw * 16 + q * 4 + sub;
                        // (expert-parallel mode: the row id names the owning rank, whose buffer holds the row)
                        const int tk = tok_cur[q] >= 0 ? tok_cur[q] : 0;
                        const int pr = a.peer_tokens > 0 ? tk / a.peer_tokens : 0;
                        const __nv_bfloat16* srow = (a.peer_tokens > 0 ? a.peer_x[pr] + (size_t)(tk - pr * a.peer_tokens) * ld
                                                                        : mat + (size_t)tk * ld) + colbase;
                        const uint32_t drow = stage + (uint32_t)kr * 128u + (uint32_t)((chunk ^ (kr & 7)) << 4);
#pragma unroll
                        for (int g4 = 0; g4 < 4; ++g4) {
                            if (g4 < 2 || second) {
                                const bool live = tok_cur[q] >= 0 && colbase + g4 * 64 < col_lim;
                                cp_async_16(drow + (uint32_t)g4 * 8192u, live ? (const void*)(srow + g4 * 64) : (const void*)a.A,
                                            live ? 16u : 0u);
                            }
                        }
                    }
                    cp_async_mbar_arrive(smem_u32(&ctrl->full[s]));
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
#pragma unroll
                    for (int q = 0; q < 4; ++q) { tok_cur[q] = tok_nxt[q]; tok_nxt[q] = tok_n2[q]; }
                }
                if (!ok) break;
            }
        } else
        for (int L = seq.first(); L < total; L = seq.next(L)) {
            const Tile t = decode_tile<KGROUP>(a, L, n_nt, n_mt_total, k_blocks);
            const bool two = t.valid > BM;
            const __nv_bfloat16* src[16];
            uint32_t live = 0u;                                           // bit i: row i of this thread is a real row
            int tok[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {   // sixteen independent loads (a pad row reads the tile's last real row id)
                const int r = (i >> 3) * BM + gw * 32 + (i & 7) * 4 + sub;
                tok[i] = __ldg(a.row_token + t.row0 + min(r, t.valid - 1));
            }
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int r = (i >> 3) * BM + gw * 32 + (i & 7) * 4 + sub;
                src[i] = gather_row(a, tok[i]) + chunk * 8;
                if (r < t.valid) live |= 1u << i;
            }
            bool ok = true;
            for (int kb = 0; kb < k_blocks; ++kb) {
                ok = mbar_wait(smem_u32(&ctrl->empty[s]), ph ^ 1u, abort_flag, a.header, 5);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const uint32_t sa = base + s * STAGE_BYTES;
                const bool in_k = (kb * BK + chunk * 8) < a.K;            // K tail: zero-fill
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    if (i < 8 || two) {
                        const int rr = gw * 32 + (i & 7) * 4 + sub;       // row inside the half
                        const uint32_t dst = sa + (i >> 3) * A_BYTES + rr * 128 + ((chunk ^ (rr & 7)) << 4);
                        const bool on = in_k && ((live >> i) & 1u);
                        cp_async_16(dst, on ? (const void*)(src[i] + kb * BK) : (const void*)a.A, on ? 16u : 0u);
                    }
                }
                cp_async_mbar_arrive(smem_u32(&ctrl->full[s]));
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
            if (!ok) break;
        }
        asm volatile("cp.async.wait_all;" ::: "memory");
    } else {
        // ------------------------------------------------------------------ epilogue: warps 2..5 -> accumulator 0,
        // warps 6..9 -> accumulator 1.  TMEM -> registers -> (SwiGLU) -> bf16 -> this warp's swizzled slab (32 rows x
        // 64 columns) -> TMA store; the accumulator is handed back right after its last TMEM read.
        const int acc = (warp - 2) >> 2;                      // which accumulator / half of the tile
        const int quad = warp & 3;                            // TMEM lane quadrant this warp may access
        const uint32_t slab = base + STAGES * STAGE_BYTES + (warp - 2) * SLAB_BYTES;
        uint32_t aph = 0;
        TileSeq<CLC> seq(ctrl, abort_flag, a.header, total, true);
        for (int L = seq.first(); L < total; L = seq.next(L)) {
            const Tile t = decode_tile<KGROUP>(a, L, n_nt, n_mt_total, k_blocks);
            if ((KGROUP && t.kblocks == 0) || (acc == 1 && t.valid <= BM)) continue;   // no rows to contract / no second half
            bool ok = mbar_wait(smem_u32(&ctrl->tfull[acc]), aph, abort_flag, a.header, 4);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            aph ^= 1u;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * BN);
            const int row = t.crow0 + acc * BM + quad * 32;
            // K-range mode: 32-row boxes past the expert's output matrix belong to the next expert
            const bool store_ok = !KGROUP || (row - t.e * a.kgroup_rows) < a.kgroup_rows;
            if (EPI == EPI_F32) {
                float* frow = reinterpret_cast<float*>(a.C) + (size_t)(row + lane) * a.ldc;
                const int c0 = t.n * BN;
#pragma unroll 1
                for (int c = 0; c < BN; c += 32) {
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
                if (lane == 0) mbar_arrive(smem_u32(&ctrl->tempty[acc]));
            } else if (EPI == EPI_BF16 && !GATHER) {
                // Plain bf16 output (this instantiation has registers to spare): the whole accumulator row is read and
                // packed first, the accumulator goes back to the MMA issuer, and only then do the four 64-column passes
                // through the slab start -- the hand-over no longer waits behind the first passes' stores.
                const int c0 = t.n * BN;
                uint32_t o[128];
#pragma unroll
                for (int c = 0; c < BN; c += 32) {
                    uint32_t r[32];
                    tc_ld32(taddr + c, r);
                    tc_wait_ld();
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        o[(c >> 1) + i] = pack_bf16(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctrl->tempty[acc]));
#pragma unroll
                for (int pass = 0; pass < 4; ++pass) {
                    if (lane == 0) tma_store_wait_read();     // the slab's previous store has been read out
                    __syncwarp();
                    const uint32_t line = slab + lane * 128;  // 64 columns = 8 chunks of 16 bytes
#pragma unroll
                    for (int v = 0; v < 8; ++v)
                        st_shared_v4(line + ((v ^ (lane & 7)) << 4), o[pass * 32 + 4 * v], o[pass * 32 + 4 * v + 1],
                                     o[pass * 32 + 4 * v + 2], o[pass * 32 + 4 * v + 3]);
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) {
                        const int col = c0 + pass * 64;
                        if (col < a.N && store_ok) tma_store_2d(&tmapC, slab, col, row);
                        tma_store_commit();
                    }
                }
            } else {
                // 64 output columns per pass.  The TMEM reads and the arithmetic of pass p+1 are done BEFORE waiting for
                // the slab that pass p is about to overwrite, so the accumulator goes back to the MMA issuer as soon as
                // its last column has been read, not after the stores.
                constexpr int PASSES = SWIGLU ? 2 : 4;
                const bool narrow = narrow_last && t.n == n_nt - 1;      // [gate 64 | up 64]: one pass, up at column 64
                const int passes = narrow ? 1 : PASSES;
                const uint32_t up_off = narrow ? BN / 4 : BN / 2;
                const int c0 = SWIGLU ? t.n * (BN / 2) : t.n * BN;
                uint32_t cur[32], nxt[32];                    // one pass = 64 columns = 32 packed bf16 pairs per row
                auto hand_back = [&]() {                       // the accumulator goes back to the MMA issuer
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&ctrl->tempty[acc]));
                };
                auto load_pass = [&](int pass, uint32_t (&o)[32]) {
#pragma unroll
                    for (int c = 0; c < 64; c += 32) {
                        if (SWIGLU) {
                            uint32_t g[32], u[32];
                            tc_ld32(taddr + pass * 64 + c, g);
                            tc_ld32(taddr + up_off + pass * 64 + c, u);
                            tc_wait_ld();
                            if (pass == passes - 1 && c == 32) hand_back();   // the tile's last TMEM read: arithmetic comes after
#pragma unroll
                            for (int i = 0; i < 16; ++i)
                                o[(c >> 1) + i] = pack_bf16(swiglu(__uint_as_float(g[2 * i]), __uint_as_float(u[2 * i])),
                                                            swiglu(__uint_as_float(g[2 * i + 1]), __uint_as_float(u[2 * i + 1])));
                        } else {
                            uint32_t r[32];
                            tc_ld32(taddr + pass * 64 + c, r);
                            tc_wait_ld();
                            if (pass == passes - 1 && c == 32) hand_back();
#pragma unroll
                            for (int i = 0; i < 16; ++i)
                                o[(c >> 1) + i] = pack_bf16(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
                        }
                    }
                };
                load_pass(0, nxt);
#pragma unroll
                for (int pass = 0; pass < PASSES; ++pass) {
                    if (pass >= passes) break;
#pragma unroll
                    for (int i = 0; i < 32; ++i) cur[i] = nxt[i];
                    if (pass + 1 < passes) {
                        load_pass(pass + 1, nxt);
                    }
                    if (lane == 0) tma_store_wait_read();     // the slab's previous store has been read out
                    __syncwarp();
                    const uint32_t line = slab + lane * 128;  // 64 columns = 8 chunks of 16 bytes
#pragma unroll
                    for (int v = 0; v < 8; ++v)
                        st_shared_v4(line + ((v ^ (lane & 7)) << 4), cur[4 * v], cur[4 * v + 1], cur[4 * v + 2], cur[4 * v + 3]);
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) {
                        const int col = c0 + pass * 64;
                        if (col < a.N && store_ok) tma_store_2d(&tmapC, slab, col, row);
                        tma_store_commit();
                    }
                }
            }
        }
        if (lane == 0) tma_store_wait_all();
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

template <int EPI, bool GATHER, int MODE = 0, bool CLC = false>
static cudaError_t launch_one(const CUtensorMap& mA, const CUtensorMap& mB, const CUtensorMap& mC, const CUtensorMap& mB64,
                              const GemmArgs& a, int n_nt, int k_blocks, int grid, cudaStream_t s) {
    static PerDevice configured;      // per device: SM count once this instantiation has its shared-memory opt-in there
    int dev = 0, sm_count = 0;
    cudaError_t e = current_device(&dev);
    if (e != cudaSuccess) return e;
    e = configured.get(dev, &sm_count, [](int d, int* sms) {
        cudaError_t e2 = cudaFuncSetAttribute(gemm_m2_kernel<EPI, GATHER, MODE, CLC>,
                                              cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        return e2 != cudaSuccess ? e2 : device_sm_count(d, sms);
    });
    if (e != cudaSuccess) return e;
    if (CLC) {
        // one CTA per tile: a host-side upper bound of the tile count (every expert with rows has at most one partial tile)
        const long long rows = a.total_rows > 0 ? a.total_rows : 0;
        const long long m_tiles = (rows + TM - 1) / TM + (rows < a.E ? rows : a.E);
        grid = (int)(m_tiles * n_nt);
        if (grid < 1) grid = 1;
    } else if (grid <= 0 || grid > sm_count) {
        grid = sm_count;
    }
    constexpr bool ROW_TILES = MODE == 0 || MODE == 2;     // tiles of expert rows against a weight tile (not K ranges)
    if (a.gang && !CLC && ROW_TILES && grid < GROUP_TILES) {
        // a gang's (up to GROUP_TILES) tiles must sit on different CTAs, or a CTA would wait for its own later tile
        GemmArgs b = a;
        b.gang = nullptr;
        gemm_m2_kernel<EPI, GATHER, MODE, CLC><<<grid, THREADS + (GATHER ? GATHER_THREADS : 0), SMEM_BYTES, s>>>(
            mA, mB, mC, mB64, b, n_nt, k_blocks);
        return cudaGetLastError();
    }
    if (a.gang && !CLC && ROW_TILES) {
        // gang starts wait for tiles of other CTAs: every CTA of the grid has to be resident (cooperative launch)
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeCooperative;
        attr[0].val.cooperative = 1;
        cfg.gridDim = dim3(grid);
        cfg.blockDim = dim3(THREADS + (GATHER ? GATHER_THREADS : 0));
        cfg.dynamicSmemBytes = SMEM_BYTES;
        cfg.stream = s;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        return cudaLaunchKernelEx(&cfg, gemm_m2_kernel<EPI, GATHER, MODE, CLC>, mA, mB, mC, mB64, a, n_nt, k_blocks);
    }
    if (CLC) {   // (tile stealing cancels CTAs that have not started: kept as a plain launch)
        gemm_m2_kernel<EPI, GATHER, MODE, CLC><<<grid, THREADS + (GATHER ? GATHER_THREADS : 0) + 32, SMEM_BYTES, s>>>(
            mA, mB, mC, mB64, a, n_nt, k_blocks);
        return cudaGetLastError();
    }
    return launch_pdl(gemm_m2_kernel<EPI, GATHER, MODE, CLC>, dim3(grid), dim3(THREADS + (GATHER ? GATHER_THREADS : 0)),
                      (size_t)SMEM_BYTES, s, mA, mB, mC, mB64, a, n_nt, k_blocks);
}

}  // namespace m2

cudaError_t launch_gemm_m2(const GemmArgs& a, int epi, int grid, cudaStream_t s) {
    using namespace m2;
    const bool swiglu = (epi == EPI_SWIGLU), gather = (a.row_token != nullptr);
    CUtensorMap mA, mB, mC;
    const uint64_t b_rows = (uint64_t)a.E * (swiglu ? 2 : 1) * a.N;
    if (a.kgroup_rows > 0 && (epi != EPI_BF16 || (gather && !a.b_mn) || (a.kgroup_rows % 32))) return cudaErrorInvalidValue;
    if (gather && a.kgroup_rows > 0 && (a.gather_mn < 1 || a.gather_mn > 2 || a.dense_rows > 0)) return cudaErrorInvalidValue;
    const uint64_t lda = a.lda ? (uint64_t)a.lda : (uint64_t)a.K, ldb = a.ldb ? (uint64_t)a.ldb : (uint64_t)a.K;
    if (a.kgroup_rows > 0 && a.b_mn) {
        // both operands as produced: A = [K rows, kgroup_rows columns], B = [K rows, N columns]; a.K = rows that exist
        // (a gathered operand is not read through its map: the map then only has to be a valid one over its a_rows rows)
        const uint64_t ra = (gather && a.gather_mn == 1) ? (uint64_t)a.a_rows : (uint64_t)a.K;
        const uint64_t rb = (gather && a.gather_mn == 2) ? (uint64_t)a.a_rows : (uint64_t)a.K;
        if (!make_map(&mA, a.A, ra, (uint64_t)a.kgroup_rows, 64, lda)) return cudaErrorInvalidValue;
        if (!make_map(&mB, a.B, rb, (uint64_t)a.N, 64, ldb)) return cudaErrorInvalidValue;
    } else if (!make_map(&mA, a.A, (uint64_t)a.a_rows, (uint64_t)a.K, BM, lda)) return cudaErrorInvalidValue;
    else if (a.b_mn) {   // W viewed as [E * K, N], N contiguous: boxes of 64 columns x 64 rows
        if (!make_map(&mB, a.B, (uint64_t)a.E * a.K, (uint64_t)a.N, 64, (uint64_t)a.N)) return cudaErrorInvalidValue;
    } else if (!make_map(&mB, a.B, a.kgroup_rows > 0 ? (uint64_t)a.N : b_rows, (uint64_t)a.K, BN / 2, ldb)) return cudaErrorInvalidValue;
    // the SwiGLU kernels' 64-row box over the same weights (narrow last N tile); a copy of mB where it is not used
    CUtensorMap mB64 = mB;
    if (swiglu && a.kgroup_rows == 0 && !a.b_mn && !make_map(&mB64, a.B, b_rows, (uint64_t)a.K, BN / 4, ldb)) return cudaErrorInvalidValue;
    if (epi == EPI_F32) mC = mB;      // the fp32 epilogue stores directly
    else if (!make_map(&mC, a.C, (uint64_t)a.rows_pad, (uint64_t)a.N, 32, (uint64_t)a.ldc)) return cudaErrorInvalidValue;
    const int n_nt = swiglu ? (a.N + BN / 2 - 1) / (BN / 2) : (a.N + BN - 1) / BN;
    const int k_blocks = (a.K + BK - 1) / BK;
    if (a.kgroup_rows > 0 && a.b_mn && gather) return launch_one<EPI_BF16, true, 3>(mA, mB, mC, mB64, a, n_nt, k_blocks, grid, s);
    if (a.kgroup_rows > 0 && a.b_mn) return launch_one<EPI_BF16, false, 3>(mA, mB, mC, mB64, a, n_nt, k_blocks, grid, s);
    if (a.kgroup_rows > 0) return launch_one<EPI_BF16, false, 1>(mA, mB, mC, mB64, a, n_nt, k_blocks, grid, s);
    if (a.b_mn) {
        if (epi != EPI_BF16) return cudaErrorInvalidValue;
        return gather ? launch_one<EPI_BF16, true, 2>(mA, mB, mC, mB64, a, n_nt, k_blocks, grid, s)
                      : launch_one<EPI_BF16, false, 2>(mA, mB, mC, mB64, a, n_nt, k_blocks, grid, s);
    }
    const bool stolen = a.tile_sched == 1 && a.dense_rows == 0;   // hardware tile stealing: routed forward GEMMs only
    if (stolen && epi == EPI_SWIGLU && gather) return launch_one<EPI_SWIGLU, true, 0, true>(mA, mB, mC, mB64, a, n_nt, k_blocks, grid, s);
    if (stolen && epi == EPI_BF16 && !gather) return launch_one<EPI_BF16, false, 0, true>(mA, mB, mC, mB64, a, n_nt, k_blocks, grid, s);
    if (epi == EPI_SWIGLU && gather) return launch_one<EPI_SWIGLU, true>(mA, mB, mC, mB64, a, n_nt, k_blocks, grid, s);
    if (epi == EPI_SWIGLU) return launch_one<EPI_SWIGLU, false>(mA, mB, mC, mB64, a, n_nt, k_blocks, grid, s);
    if (epi == EPI_BF16 && !gather) return launch_one<EPI_BF16, false>(mA, mB, mC, mB64, a, n_nt, k_blocks, grid, s);
    if (epi == EPI_BF16) return launch_one<EPI_BF16, true>(mA, mB, mC, mB64, a, n_nt, k_blocks, grid, s);
    if (epi == EPI_F32 && !gather) return launch_one<EPI_F32, false>(mA, mB, mC, mB64, a, n_nt, k_blocks, grid, s);
    return cudaErrorInvalidValue;
}

}  // namespace mok
