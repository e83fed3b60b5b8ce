// Routed expert FFN in ONE persistent launch: gate/up grouped GEMM + SwiGLU and the down grouped GEMM of the same rows
// (paper, Section 3.2 "Megakernel": the stages of an expert's FFN run depth-first inside one kernel and synchronise
// through GPU-local completion counters instead of kernel boundaries; Figure 1, left).
//
// The work is ONE list of 256-row tiles of two kinds:
//   G  gate/up tile: rows gathered from x through the schedule (pull dispatch, Section 3.1), weights [gate 128 | up 128]
//      by TMA, K = H; epilogue silu(g) * u -> h (bf16, TMA store), then the epilogue warps wait until their stores have
//      completed and add one arrival each to ready[M tile]
//   D  down tile: h rows and W_down by TMA, K = I; epilogue -> y (bf16, TMA store).  Its producer first waits until
//      ready[M tile] shows every gate/up tile of those rows (bounded wait; a time-out reports MOK_ERR_TIMEOUT).
//      One D entry of the list covers q = round(H / I) consecutive N tiles of its rows, so that an entry of either kind
//      keeps a CTA busy for about the same time.  That matters for DRAM traffic, not for balance: CTAs that work on
//      the same weight tile for different row tiles share it through L2 only while they stay in step, and they only
//      stay in step if the entries before them took equally long (measured with entries of unequal length: 43 % more
//      DRAM reads than the two-launch path, and a lower clock under the power cap)
// The list is built on the device by fused_tiles_kernel from the schedule's per-expert tables: M tiles are grouped
// (eight per group, one expert per group) and a group's tiles are laid out [N tile][M tile] so that CTAs working side
// by side share a weight tile in L2.  A group's D tiles are placed `window` M tiles behind its G tiles: with the
// persistent grid walking the list in order (tile L -> CTA L mod grid), the gate/up tiles a down tile depends on are
// then normally complete when its producer asks, and h is consumed while it is still in L2.
//
// No deadlock: every tile a D tile depends on has a smaller list index; a CTA works through its tiles in increasing
// order; the launch is cooperative, so all CTAs of the grid are resident.  Take the unfinished tile with the smallest
// index: everything it waits for is finished, so it makes progress.
//
// Two ways of handing out the list.  STATIC: tile L -> CTA L mod grid (cooperative launch: every CTA resident).  Gate/up
// and down tiles differ in length (K = H against K = I), so CTAs drift apart along the list and down tiles do wait.
// DYNAMIC: a scheduler warp per CTA draws the next list position from one global counter (a plain atomic add, a few
// tiles ahead of the CTA's other roles, which read the ids from a small queue in shared memory), so a CTA that got
// short tiles simply draws more of them and all CTAs stay within about one tile of each other.  The argument above
// holds unchanged: whoever drew a position runs, and everything it waits for was drawn earlier.
// (Tried and dropped: two draw counters with "the next down tile if its rows are complete, else a gate/up tile",
// claimed by compare-and-swap so that a claimed down tile never waits.  Correct, but a compare-and-swap chain hands
// out about one tile per L2 round trip for the whole GPU, an order of magnitude below the ~7 tiles per microsecond the
// grid consumes: the layer ran three times slower.)
//
// Determinism: every output element is still produced by exactly one tile with a fixed k order, so the bits equal
// those of the two separate launches whatever the interleaving (tested).
//
// Shared-memory ring, tensor-memory use and the epilogue arithmetic are those of gemm_tcgen05_m2.cu; during D tiles the
// gather warps skip ahead and the producer makes their arrivals on the ring's barriers.
//
// Optionally `h` is a RING of `ring` 256-row slots (Section 3.3: fixed-size buffers reused by the minibatches in flight):
// row tile mt lives in slot mt mod ring.  A gate/up tile of row tile mt >= ring may only store once every down entry of
// row tile mt - ring has loaded its rows: the MMA issuer adds one arrival to consumed[mt'] when all TMA loads of a down
// entry of mt' have landed, and the gate/up epilogue waits (bounded) for all entries' arrivals.  No deadlock: with
// ring >= window + 2 * GROUP_TILES (the launcher shortens the window to make it so) every down entry of row tile
// mt - ring sits at a smaller list position than every gate/up tile of row tile mt, so the argument above still holds.
// With the static window of two grids' worth of tiles the slots are rewritten while still in L2.
//
// Optionally some CTAs of the grid are COMMUNICATION CTAs (Section 3.4 "Computation-Communication SM Tuning"; Figure 1:
// dedicated SMs pull the tokens while the others compute).  They do no tiles: for row tile after row tile, in list
// order, they copy the tile's token rows (from x, or under expert parallelism from the owners' buffers) into one of
// COMM_SLOTS 256-row slots of a staging buffer and add an arrival to staged[mt]; the gate/up tiles of that row tile
// then take their A operand from the slot by TMA (the gather warps idle, as for down tiles) once staged[mt] is set, and
// the MMA issuer adds an arrival to released[mt] when a gate/up tile's loads have landed, which is what a communication
// CTA waits for (all n1 of them) before it reuses the slot for row tile mt + COMM_SLOTS.  So the latency of a pull --
// microseconds over NVLink -- is taken by CTAs that do nothing else, a whole row tile ahead of its use, instead of by
// gather warps that feed a three-stage ring.  No deadlock: communication CTAs walk the row tiles in increasing order,
// every gate/up tile of row tile mt - COMM_SLOTS has a smaller list position than any of row tile mt (COMM_SLOTS >=
// 2 * GROUP_TILES), the launch is cooperative; the unfinished item with the smallest position can always proceed.
//
// Optionally the COMBINE (Section 2.1: out[t] = shared[t] + sum_s w[t,s] * y[pos[t,s]]) runs in the same launch: a token's
// k rows lie anywhere in y, so it can only start when every down tile has been stored.  Every epilogue warp adds one
// arrival to a grid-wide counter once its last store has completed, waits (bounded) until all epilogue warps of the grid
// have arrived; then the epilogue and gather warps draw tokens from a global counter and combine them, one token per
// warp at a time, in the fixed slot order of the separate combine kernel (same bits).
#include "mok_internal.cuh"
#include "tc_ptx.cuh"
#include "tensor_map.cuh"
#include <string.h>

namespace mok {
namespace ff {

using namespace tc;

constexpr int BM = 128, BN = 256, BK = 64, UMMA_K = 16, STAGES = 3;
constexpr int A_BYTES = BM * BK * 2;
constexpr int B_BYTES = BN * BK * 2;
constexpr int STAGE_BYTES = 2 * A_BYTES + B_BYTES;
constexpr int TM = 2 * BM;
constexpr int TMEM_COLS = 512;
constexpr int EPI_WARPS = 8;
constexpr int GATHER_THREADS = 128;
constexpr int THREADS = 128 + 32 * EPI_WARPS + GATHER_THREADS;    // 512: four groups of four warps (see the kernel)
constexpr int GROUP_TILES = 8;
constexpr int SLAB_BYTES = 4096;
constexpr int SMEM_CTRL = 512;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_WARPS * SLAB_BYTES + SMEM_CTRL + 1024;
constexpr int QSLOTS = 4;                       // tile ids drawn ahead by the scheduler warp (dynamic mode)
constexpr int COMM_SLOTS = FFN_COMM_SLOTS;      // 256-row slots of the staging buffer of the communication CTAs
constexpr int COMM_ISSUERS = 4, COMM_BUFS = 3, COMM_PIECE = 16384;   // its copy pipelines: 4 threads x 3 buffers of 16 KB
static_assert(COMM_SLOTS >= 2 * GROUP_TILES, "a slot must not be reused inside the row group that still needs it");
constexpr int ROLE_READERS = 2 + EPI_WARPS + GATHER_THREADS / 32;      // one arrival per role warp and queue entry

struct Ctrl {
    uint64_t full[STAGES], empty[STAGES];
    uint64_t tfull[2], tempty[2];
    uint64_t q_full[QSLOTS], q_empty[QSLOTS];
    int32_t q_tile[QSLOTS];
    uint32_t tmem_base, abort;
    uint32_t combine_go;                 // in-launch combine: the grid has finished its tiles (written by the CTA's poller)
    uint64_t cbar[COMM_ISSUERS * COMM_BUFS];   // communication CTA: one barrier per staging buffer of its copy pipelines
};
static_assert(sizeof(Ctrl) <= SMEM_CTRL, "control block too large");

constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
__device__ __forceinline__ uint32_t idesc_n(int n) { return (IDESC & ~(0x3Fu << 17)) | ((uint32_t)(n >> 3) << 17); }

struct Tile { int row0, valid, kind, cnt, e, n, mt, gang_m, gang_size; };
// cnt: N tiles n .. n + cnt - 1 covered by this list entry; gang: the gang_size entries [L - gang_m, ...) use the same
// weight tiles (one per row tile of the group)
__device__ __forceinline__ Tile decode_tile(const int4 d) {
    Tile t;
    t.row0 = d.x;
    t.valid = d.y & 0x1FF;
    t.gang_m = (d.y >> 9) & 7;
    t.gang_size = ((d.y >> 12) & 7) + 1;
    t.kind = (d.y >> 16) & 1;
    t.cnt = (d.y >> 20) & 0xFF;
    t.e = d.z & 0xFFFF;
    t.n = (d.z >> 16) & 0xFFFF;
    t.mt = d.w;
    return t;
}

// The bounded mbarrier wait of tc_ptx.cuh, inlined: this kernel changes the register allocation of its warps
// (setmaxnreg), and a real function call from regions with different register counts does not compile.
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, WsHeader* hdr, int site) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = globaltimer();
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 127u) == 0u) {
            if (*abort_flag) return false;
            const unsigned long long limit = hdr->wait_limit_us ? 1000ull * hdr->wait_limit_us : WAIT_LIMIT_NS;
            if (globaltimer() - t0 > limit) {
                *abort_flag = 1u;
                atomicCAS(&hdr->status, 0, (int)MOK_ERR_TIMEOUT);
                hdr->where = site;
                return false;
            }
        }
    }
    return true;
}

// How a role walks over its tiles: static stride, or ids read from the scheduler warp's queue (bounded waits; an entry
// is released once every role has read it; a negative id ends the kernel).
template <bool DYN>
struct TileSeq {
    Ctrl* ctrl;
    volatile uint32_t* abort_flag;
    WsHeader* hdr;
    int total, slot, stride;
    uint32_t ph;
    bool warp_role;       // all 32 lanes call next() together / one lane calls it
    __device__ __forceinline__ TileSeq(Ctrl* c, volatile uint32_t* af, WsHeader* h, int tot, bool wr, int str)
        : ctrl(c), abort_flag(af), hdr(h), total(tot), slot(0), stride(str), ph(0), warp_role(wr) {}
    __device__ __forceinline__ int first() { return DYN ? next(0) : (int)blockIdx.x; }
    __device__ __forceinline__ int next(int L) {
        if (!DYN) return L + stride;             // (the compute CTAs of the grid: communication CTAs take no tiles)
        bool ok = wait_bar(smem_u32(&ctrl->q_full[slot]), ph, abort_flag, hdr, 30);
        if (warp_role) ok = __all_sync(0xffffffffu, ok);
        if (!ok) return total;
        const int t = *reinterpret_cast<volatile int32_t*>(&ctrl->q_tile[slot]);
        if (warp_role) __syncwarp();
        if (!warp_role || (threadIdx.x & 31) == 0) mbar_arrive(smem_u32(&ctrl->q_empty[slot]));
        if (++slot == QSLOTS) { slot = 0; ph ^= 1u; }
        return t < 0 ? total : t;
    }
};

// A role's walk over its tiles with the NEXT tile's descriptor already on its way: the 16-byte descriptor load of tile
// i + 1 is issued when the role starts tile i, so no role stalls on it at a tile boundary.
template <bool DYN>
struct TileWalk {
    TileSeq<DYN> seq;
    const int4* tiles;
    int total, L, Ln;
    int4 d, dn;
    __device__ __forceinline__ int4 fetch(int l) const { return l < total ? __ldg(tiles + l) : make_int4(0, 0, 0, 0); }
    __device__ __forceinline__ TileWalk(Ctrl* c, volatile uint32_t* af, WsHeader* h, const int4* tl, int tot, bool wr, int str)
        : seq(c, af, h, tot, wr, str), tiles(tl), total(tot) {
        L = seq.first();
        d = fetch(L);
        Ln = L < total ? seq.next(L) : total;
        dn = fetch(Ln);
    }
    __device__ __forceinline__ bool valid() const { return L < total; }
    __device__ __forceinline__ void advance() {
        L = Ln;
        d = dn;
        if (L < total) {
            Ln = seq.next(L);
            dn = fetch(Ln);
        }
    }
};

__device__ __forceinline__ int ld_acquire(const int32_t* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// ---------------------------------------------------------------------------------------------------------------
// Tile list.  One block of MAX_E threads per launch-grid slot; every block rebuilds the (tiny) per-expert group
// offsets in shared memory, then its warps take groups g = warp id, + number of warps, ...
//   ME(g) = M tiles up to and including group g;  MB(g) = ME(g - 1)
//   j(g)  = first group j >= g with ME(j) >= ME(g) + window (last group if none): D(g) follows G(j(g))
//   c(j)  = number of groups whose D tiles precede G(j) = #{g : ME(g) <= MB(j) - window}
//   pos_G(j) = n1 * MB(j) + n2 * MB(c(j));   pos_D(g) = n1 * ME(j(g)) + n2 * MB(g)
__global__ void __launch_bounds__(MAX_E)
fused_tiles_kernel(const int32_t* __restrict__ counts, const int32_t* __restrict__ pad_offsets,
                   const int32_t* __restrict__ mt_start2, int E, int n1, int n2_tiles, int q, int window, int max_tiles,
                   int4* __restrict__ tiles, int32_t* __restrict__ ready, int32_t* __restrict__ consumed,
                   int32_t* __restrict__ staged, int32_t* __restrict__ released, WsHeader* __restrict__ hdr) {
    __shared__ int32_t s_mt[MAX_E + 1], s_gofs[MAX_E + 1], s_wtot[32];
    pdl_enter();
    const int n2 = (n2_tiles + q - 1) / q;           // down entries per M tile: each covers up to q N tiles
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, n_warps = blockDim.x >> 5;
    int mc = 0;
    if (tid < E) {
        const int m0 = mt_start2[tid], m1 = mt_start2[tid + 1];
        s_mt[tid] = m0;
        if (tid == E - 1) s_mt[E] = m1;
        mc = m1 - m0;
    }
    const int ng = (mc + GROUP_TILES - 1) / GROUP_TILES;
    int inc = ng;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, inc, off);
        if (lane >= off) inc += t;
    }
    if (lane == 31) s_wtot[wid] = inc;
    __syncthreads();
    if (wid == 0) {
        const int mine = lane < n_warps ? s_wtot[lane] : 0;
        int run = mine;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, run, off);
            if (lane >= off) run += t;
        }
        s_wtot[lane] = run - mine;
    }
    __syncthreads();
    if (tid < E) {
        s_gofs[tid] = s_wtot[wid] + inc - ng;
        if (tid == E - 1) s_gofs[E] = s_wtot[wid] + inc;
    }
    __syncthreads();
    const int NG = s_gofs[E], NMT = s_mt[E];
    const long long total = (long long)NMT * (n1 + n2);
    if (blockIdx.x == 0 && tid == 0) {
        hdr->n_ftiles = total <= max_tiles ? (int32_t)total : 0;
        hdr->next_tile = 0;
        hdr->ffn_done = 0;
        hdr->combine_next = 0;
        if (total > max_tiles) atomicCAS(&hdr->status, 0, (int)MOK_ERR_SCHEDULE);
    }
    if (total > max_tiles) return;
    for (int i = blockIdx.x * blockDim.x + tid; i < NMT; i += gridDim.x * blockDim.x) {
        ready[i] = 0;
        consumed[i] = 0;
        staged[i] = 0;
        released[i] = 0;
    }

    // largest e in [0, E) with s_mt[e] <= v and a non-empty tail (the expert that holds M tile index v), for 0 <= v < NMT
    auto expert_of_tile = [&](int v) {
        int lo = 0, hi = E;                       // invariant: s_mt[lo] <= v < s_mt[hi]
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (s_mt[mid] <= v) lo = mid; else hi = mid;
        }
        return lo;
    };
    for (int g = blockIdx.x * n_warps + wid; g < NG; g += gridDim.x * n_warps) {
        // expert and position of group g: the last e with s_gofs[e] <= g (empty experts have no groups and are skipped
        // by taking the LAST such e)
        int lo = 0, hi = E;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (s_gofs[mid] <= g) lo = mid; else hi = mid;
        }
        const int e = lo, gi = g - s_gofs[e], m0 = gi * GROUP_TILES;
        const int mcnt = s_mt[e + 1] - s_mt[e];
        const int gm = min(GROUP_TILES, mcnt - m0);              // M tiles of this group
        const int MB = s_mt[e] + m0, ME = MB + gm;
        // j(g): the group in which the cumulative M-tile count first reaches ME + window
        int MEj;
        {
            const int target = ME + window;
            if (window == 0) {
                MEj = ME;
            } else if (target > NMT) {
                MEj = NMT;                                       // the last group
            } else {
                const int ej = expert_of_tile(target - 1);       // expert holding the target-th M tile
                const int within = target - s_mt[ej];            // 1 .. its M-tile count
                const int gj = (within + GROUP_TILES - 1) / GROUP_TILES;     // groups of ej needed to reach it
                MEj = s_mt[ej] + min(gj * GROUP_TILES, s_mt[ej + 1] - s_mt[ej]);
            }
        }
        // c(g): groups whose D tiles come before G(g): those ending at or before MB - window
        int MBc;                                                 // = MB(c(g)): M tiles of those groups
        {
            const int v = MB - window;
            if (v <= 0) {
                MBc = 0;
            } else if (window == 0) {
                MBc = MB;
            } else {
                const int ec = expert_of_tile(v - 1);            // expert holding the v-th M tile
                const int within = v - s_mt[ec];                 // M tiles of ec among the first v
                const int mce = s_mt[ec + 1] - s_mt[ec];
                // whole groups of ec inside the first v tiles (its last, partial group counts once all its tiles are in)
                MBc = s_mt[ec] + (within == mce ? mce : within / GROUP_TILES * GROUP_TILES);
            }
        }
        const long long posG = (long long)n1 * MB + (long long)n2 * MBc;
        const long long posD = (long long)n1 * MEj + (long long)n2 * MB;
        const int cnt = counts[e], pad0 = pad_offsets[e];
        for (int i = lane; i < (n1 + n2) * gm; i += 32) {
            const int kind = i >= n1 * gm;
            const int r = kind ? i - n1 * gm : i;
            const int nc = r / gm, m = m0 + (r - nc * gm);
            const int n = kind ? nc * q : nc;                       // first N tile of the entry
            const int span = kind ? min(q, n2_tiles - n) : 1;       // N tiles it covers
            int4 d;
            d.x = pad0 + m * TM;
            d.y = min(TM, cnt - m * TM) | ((m - m0) << 9) | ((gm - 1) << 12) | (kind << 16) | (span << 20);
            d.z = e | (n << 16);
            d.w = s_mt[e] + m;
            tiles[(kind ? posD : posG) + r] = d;
        }
    }
}

struct FusedArgs {
    const __nv_bfloat16* x;        // [T, H] token rows (gathered through row_token)
    // expert parallelism (Section 3.1, pull dispatch): with peer_tokens > 0 the ids in row_token are global,
    // id = source rank * peer_tokens + token, and the row is read from that rank's buffer with plain peer loads
    int32_t peer_tokens;
    const __nv_bfloat16* peer_x[MOK_MAX_RANKS];
    const int32_t* row_token;      // padded row -> token
    const int4* tiles;             // the tile list
    const int32_t* n_tiles;        // device: its length
    int32_t* next_tile;            // device: dynamic mode's draw counter (zeroed by the tile-list kernel)
    int32_t* gang;                 // static mode: per list position, arrivals of the entries that share weight tiles
                                   // (zeroed before the launch), or NULL: unsynchronised starts
    int32_t* ready;                // per 256-row M tile: epilogue-warp arrivals of its gate/up tiles
    int32_t* consumed;             // per 256-row M tile: down entries whose loads of h have landed (ring mode)
    // communication CTAs (comm_ctas > 0): the last comm_ctas CTAs of the grid stage the token rows of every row tile
    int32_t comm_ctas, n_compute;  // n_compute = gridDim.x - comm_ctas CTAs work on tiles
    __nv_bfloat16* xg;             // [COMM_SLOTS * 256, H] staging slots, row tile mt in slot mt % COMM_SLOTS
    int32_t* staged;               // per row tile: 1 once its rows are in the slot
    int32_t* released;             // per row tile: gate/up tiles whose loads from the slot have landed
    const int32_t* mt_start2;      // the schedule's 256-row tile tables (row tile -> expert, first row, valid rows)
    const int32_t* tile_expert2;
    const int32_t* counts;
    const int32_t* pad_offsets;
    const int32_t* n_mtiles2;
    int32_t max_mt2;
    int32_t ring;                  // > 0: h holds `ring` 256-row slots, row tile mt in slot mt % ring
    int32_t need_d;                // down entries per row tile
    int32_t max_tiles;
    int32_t H, I, E;
    int32_t n1, n2;                // N tiles of a gate/up row tile (ceil(I / 128)) and of a down row tile (ceil(H / 256))
    int32_t kb1, kb2;              // k-blocks of the two kinds
    int32_t dbg;                   // != 0: counters into header->dbg[1] (gate/up tiles) and [2] (down tiles)
    int32_t starve;                // test hooks: 1 = the producer issues nothing, 2 = nobody arrives on `consumed` / `ffn_done`
    WsHeader* header;
    // combine in the same launch (out != NULL)
    const __nv_bfloat16* y;        // [Rpad, H] rows of the down tiles
    const __nv_bfloat16* ysh;      // [T, H] shared expert's output, or NULL
    const int32_t* pos;            // [T * k] padded row of every route
    const float* w;                // [T * k] router weights
    __nv_bfloat16* out;            // [T, H], or NULL: no combine in this launch
    int32_t T, k;
};

// The combine of this launch, run warp by warp after a warp's last tile.  An epilogue warp first adds its arrival to the
// grid-wide counter (its stores have completed); every participating warp then waits (bounded) for all
// EPI_WARPS * gridDim.x arrivals and draws tokens from a global counter, one token per warp at a time: 16 bytes per
// lane and row, CH chunks of a row per pass with the k rows of every chunk loaded before the first multiply-add,
// accumulation in fp32 in slot order on top of the shared expert's row.
// (every epilogue and gather warp of the CTA calls this exactly once, whatever happened before: the two named barriers
//  below count all COMBINE_THREADS threads.  ONE thread per CTA polls the grid-wide counter: with every warp of the grid
//  polling, the polls swamp the L2 slice that also has to take the arrivals.)
constexpr int COMBINE_THREADS = 32 * EPI_WARPS + GATHER_THREADS;
template <int CH>
__device__ __forceinline__ void combine_tokens(const FusedArgs& a, Ctrl* ctrl, int lane, bool poller,
                                               volatile uint32_t* abort_flag, bool arrive) {
    int32_t* done = &a.header->ffn_done;
    const int need = EPI_WARPS * a.n_compute;
    if (lane == 0 && arrive && a.starve != 2 && !*abort_flag) {
        // (the warp's TMA stores have completed: make them visible to generic-proxy reads of other SMs, then arrive)
        asm volatile("fence.proxy.async;" ::: "memory");
        __threadfence();
        asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(done) : "memory");
    }
    asm volatile("bar.sync 1, %0;" ::"n"(COMBINE_THREADS) : "memory");      // this CTA's warps are through with their tiles
    if (poller && lane == 0) {
        uint32_t go = *abort_flag ? 0u : 1u;
        const unsigned long long t0 = globaltimer();
        uint32_t spins = 0;
        while (go && ld_acquire(done) < need) {
            __nanosleep(256);
            if ((++spins & 31u) == 0u) {
                if (*abort_flag) { go = 0u; break; }
                const unsigned long long limit = a.header->wait_limit_us ? 1000ull * a.header->wait_limit_us : WAIT_LIMIT_NS;
                if (globaltimer() - t0 > limit) {
                    *abort_flag = 1u;
                    atomicCAS(&a.header->status, 0, (int)MOK_ERR_TIMEOUT);
                    a.header->where = 44;
                    go = 0u;
                    break;
                }
            }
        }
        *reinterpret_cast<volatile uint32_t*>(&ctrl->combine_go) = go;
    }
    asm volatile("bar.sync 1, %0;" ::"n"(COMBINE_THREADS) : "memory");      // the poller's verdict is in shared memory
    if (!*reinterpret_cast<volatile uint32_t*>(&ctrl->combine_go)) return;
    const int chunks = a.H >> 3, k = a.k;
    for (;;) {
        int t = 0;
        if (lane == 0) t = atomicAdd(&a.header->combine_next, 1);
        t = __shfl_sync(0xffffffffu, t, 0);
        if (t >= a.T) break;
        int my_pos = 0;
        float my_w = 0.f;
        if (lane < k) {
            my_pos = __ldg(a.pos + (size_t)t * k + lane);
            my_w = __ldg(a.w + (size_t)t * k + lane);
        }
        // (the trip count is the same for every lane: the loop body exchanges values between lanes)
        for (int c0 = 0; c0 < chunks; c0 += 32 * CH) {
            float acc[CH][8];
#pragma unroll
            for (int u = 0; u < CH; ++u) {
                const int c = c0 + u * 32 + lane;
                if (a.ysh && c < chunks) {
                    const uint4 raw = __ldcg(reinterpret_cast<const uint4*>(a.ysh + (size_t)t * a.H) + c);
                    const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float2 f = __bfloat1622float2(p2[i]);
                        acc[u][2 * i] = f.x;
                        acc[u][2 * i + 1] = f.y;
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 8; ++i) acc[u][i] = 0.f;
                }
            }
            for (int s0 = 0; s0 < k; s0 += 8) {
                uint4 v[CH][8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int row = __shfl_sync(0xffffffffu, my_pos, (s0 + j) & 31);
#pragma unroll
                    for (int u = 0; u < CH; ++u) {
                        const int c = c0 + u * 32 + lane;
                        if (c < chunks && s0 + j < k) v[u][j] = __ldcg(reinterpret_cast<const uint4*>(a.y + (size_t)row * a.H) + c);
                    }
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float wv = __shfl_sync(0xffffffffu, my_w, (s0 + j) & 31);
#pragma unroll
                    for (int u = 0; u < CH; ++u) {
                        if (c0 + u * 32 + lane < chunks && s0 + j < k) {
                            const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&v[u][j]);
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const float2 f = __bfloat1622float2(p2[i]);
                                acc[u][2 * i] = fmaf(wv, f.x, acc[u][2 * i]);
                                acc[u][2 * i + 1] = fmaf(wv, f.y, acc[u][2 * i + 1]);
                            }
                        }
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < CH; ++u) {
                const int c = c0 + u * 32 + lane;
                uint4 o;
                __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
                for (int i = 0; i < 4; ++i) o2[i] = __floats2bfloat162_rn(acc[u][2 * i], acc[u][2 * i + 1]);
                if (c < chunks) *(reinterpret_cast<uint4*>(a.out + (size_t)t * a.H) + c) = o;
            }
        }
    }
}

// Registers are handed from the light roles to the epilogue (setmaxnreg, per group of four warps): the producer /
// issuer / scheduler group and the gather group give up most of theirs, and the two epilogue groups get enough to hold
// a whole 256-column accumulator row, so that an accumulator goes back to the MMA issuer right after its last TMEM read.
template <int N>
__device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N>
__device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
constexpr int REGS_CONTROL = 56, REGS_GATHER = 88, REGS_EPILOGUE = 184;      // (56 + 88 + 2 * 184) * 128 = 65536

//   warp 0 TMA producer | warp 1 MMA issuer (+ tensor-memory allocation) | warp 2 scheduler (dynamic mode) | warp 3 idle
//   warps 4..7  epilogue of accumulator 0 (rows 0..127 of a tile)     warps 8..11 epilogue of accumulator 1
//   warps 12..15 gather
template <bool DYN>
__global__ void __launch_bounds__(THREADS, 1)
fused_ffn_kernel(const __grid_constant__ CUtensorMap mapWgu, const __grid_constant__ CUtensorMap mapWgu64,
                 const __grid_constant__ CUtensorMap mapHst, const __grid_constant__ CUtensorMap mapHld,
                 const __grid_constant__ CUtensorMap mapWd, const __grid_constant__ CUtensorMap mapY,
                 const __grid_constant__ CUtensorMap mapXg, const __grid_constant__ FusedArgs a) {
    extern __shared__ uint8_t smem_raw[];
    pdl_enter();
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem + STAGES * STAGE_BYTES + EPI_WARPS * SLAB_BYTES);
    volatile uint32_t* abort_flag = &ctrl->abort;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    int total = *a.n_tiles;
    if (total > a.max_tiles) total = a.max_tiles;
    const int last_cols = a.I - (a.n1 - 1) * (BN / 2);
    const bool narrow_last = last_cols <= BN / 4;          // last gate/up N tile as [gate 64 | up 64], N = 128

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(smem_u32(&ctrl->full[s]), 1 + GATHER_THREADS);
            mbar_init(smem_u32(&ctrl->empty[s]), 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(smem_u32(&ctrl->tfull[s]), 1);
            mbar_init(smem_u32(&ctrl->tempty[s]), 4);
        }
        if (DYN) {
            for (int q = 0; q < QSLOTS; ++q) {
                mbar_init(smem_u32(&ctrl->q_full[q]), 1);
                mbar_init(smem_u32(&ctrl->q_empty[q]), ROLE_READERS);
            }
        }
        for (int q = 0; q < COMM_ISSUERS * COMM_BUFS; ++q) mbar_init(smem_u32(&ctrl->cbar[q]), 1);
        ctrl->abort = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    const bool is_comm = (int)blockIdx.x >= a.n_compute;
    if (warp == 1 && !is_comm) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&ctrl->tmem_base)), "r"((uint32_t)TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctrl->tmem_base;

    if (is_comm) {
        // ---------------------------------------------------------------------- communication CTA: stages token rows
        // Row tiles cr, cr + comm_ctas, ... in increasing order.  The copy goes through shared memory with bulk
        // asynchronous copies (global -> shared -> global), so that ~128 KB are in flight per SM whatever the latency of
        // the source: COMM_ISSUERS threads (lane 0 of warps 0..3) each run a pipeline over COMM_BUFS buffers of 16 KB and
        // take every fourth piece (a row, or 16 KB of a longer row).  Rows past the expert's count are written as zeros by
        // the other threads.
        const int cr = (int)blockIdx.x - a.n_compute;
        const int n_mt = min(*a.n_mtiles2, a.max_mt2);
        const int row_bytes = a.H * 2, ppr = (row_bytes + COMM_PIECE - 1) / COMM_PIECE;
        int32_t* s_tok = reinterpret_cast<int32_t*>(smem + STAGES * STAGE_BYTES);       // the tile's row -> token ids
        uint32_t cph[COMM_BUFS] = {0u, 0u, 0u};
        for (int mt = cr; mt < n_mt; mt += a.comm_ctas) {
            if (threadIdx.x == 0) {
                uint32_t go = 1u;
                if (mt >= COMM_SLOTS) {      // the slot's previous rows have been loaded by all their gate/up tiles
                    const int32_t* c = a.released + (mt - COMM_SLOTS);
                    const unsigned long long t0 = globaltimer();
                    uint32_t spins = 0;
                    while (ld_acquire(c) < a.n1) {
                        __nanosleep(256);
                        if ((++spins & 31u) == 0u) {
                            const unsigned long long limit =
                                a.header->wait_limit_us ? 1000ull * a.header->wait_limit_us : WAIT_LIMIT_NS;
                            if (a.header->status != 0 || globaltimer() - t0 > limit) {
                                atomicCAS(&a.header->status, 0, (int)MOK_ERR_TIMEOUT);
                                a.header->where = 46;
                                go = 0u;
                                break;
                            }
                        }
                    }
                }
                *reinterpret_cast<volatile uint32_t*>(&ctrl->combine_go) = go;
            }
            const int e = __ldg(a.tile_expert2 + mt);
            const int m = mt - __ldg(a.mt_start2 + e);
            const int row0 = __ldg(a.pad_offsets + e) + m * TM;
            const int valid = min(TM, __ldg(a.counts + e) - m * TM);
            const int rows = valid > BM ? TM : BM;                      // a tile with one half only loads one half
            if ((int)threadIdx.x < valid) s_tok[threadIdx.x] = __ldg(a.row_token + row0 + threadIdx.x);
            __syncthreads();
            if (!*reinterpret_cast<volatile uint32_t*>(&ctrl->combine_go)) break;
            __nv_bfloat16* dst0 = a.xg + (size_t)(mt % COMM_SLOTS) * TM * a.H;
            bool ok = true;
            if (warp < COMM_ISSUERS) {
                if (lane == 0) {
                    const int n_pieces = valid * ppr;
                    const uint32_t buf0 = base + (uint32_t)(warp * COMM_BUFS) * COMM_PIECE;
                    uint64_t* bars = ctrl->cbar + warp * COMM_BUFS;
                    auto piece = [&](int q, const char*& src, char*& dst, uint32_t& bytes) {
                        const int r = q / ppr, off = (q - r * ppr) * COMM_PIECE;
                        const int tok = s_tok[r];
                        const __nv_bfloat16* srow;
                        if (a.peer_tokens > 0) {
                            const int pr = tok / a.peer_tokens;
                            srow = a.peer_x[pr] + (size_t)(tok - pr * a.peer_tokens) * a.H;
                        } else {
                            srow = a.x + (size_t)tok * a.H;
                        }
                        src = reinterpret_cast<const char*>(srow) + off;
                        dst = reinterpret_cast<char*>(dst0 + (size_t)r * a.H) + off;
                        bytes = (uint32_t)min(COMM_PIECE, row_bytes - off);
                    };
                    auto load = [&](int q, int b) {
                        const char* src; char* dst; uint32_t bytes;
                        piece(q, src, dst, bytes);
                        const uint32_t bar = smem_u32(&bars[b]);
                        mbar_expect_tx(bar, bytes);
                        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                                     ::"r"(buf0 + (uint32_t)b * COMM_PIECE), "l"(src), "r"(bytes), "r"(bar) : "memory");
                    };
                    // this issuer's pieces: warp, warp + 4, ...; two loads ahead of the store
                    int q_load = warp, b_load = 0;
                    for (int pre = 0; pre < COMM_BUFS - 1 && q_load < n_pieces; ++pre) {
                        load(q_load, b_load);
                        q_load += COMM_ISSUERS;
                        b_load = (b_load + 1) % COMM_BUFS;
                    }
                    int b = 0;
                    for (int q = warp; q < n_pieces; q += COMM_ISSUERS) {
                        ok = wait_bar(smem_u32(&bars[b]), cph[b], abort_flag, a.header, 48);
                        if (!ok) break;
                        cph[b] ^= 1u;
                        const char* src; char* dst; uint32_t bytes;
                        piece(q, src, dst, bytes);
                        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                                     ::"l"(dst), "r"(buf0 + (uint32_t)b * COMM_PIECE), "r"(bytes) : "memory");
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                        // the buffer of the next load held the piece before this one: its store must have left shared memory
                        asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                        if (q_load < n_pieces) {
                            load(q_load, b_load);
                            q_load += COMM_ISSUERS;
                            b_load = (b_load + 1) % COMM_BUFS;
                        }
                        b = (b + 1) % COMM_BUFS;
                    }
                    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");      // every store of this issuer has completed
                    asm volatile("fence.proxy.async;" ::: "memory");
                    __threadfence();
                }
                ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
            } else {
                // padding rows of the tile, as zeros
                const int chunks = a.H >> 3;
                for (int r = valid + (warp - COMM_ISSUERS); r < rows; r += THREADS / 32 - COMM_ISSUERS) {
                    uint4* d = reinterpret_cast<uint4*>(dst0 + (size_t)r * a.H);
                    for (int c = lane; c < chunks; c += 32) d[c] = make_uint4(0u, 0u, 0u, 0u);
                }
                __threadfence();                 // visible at GPU scope before the arrival below
            }
            if (!__syncthreads_and((int)ok)) {
                // failure path only: give the copies already in flight into this CTA's shared memory time to land
                const unsigned long long t0 = globaltimer();
                while (globaltimer() - t0 < 200000ull) { }
                break;
            }
            if (threadIdx.x == 0) asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(a.staged + mt) : "memory");
        }
        if (warp < COMM_ISSUERS && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        return;                                  // (no tensor memory, no tiles: nothing to tear down)
    }

    if (warp < 4) {
        reg_dec<REGS_CONTROL>();
        if (warp == 0) {
            // -------------------------------------------------------------- TMA producer
            if (lane == 0 && a.starve != 1) {
                int s = 0;
                uint32_t ph = 0;
                long long d_ready = 0;
                int peek = 0;            // completion counter of the NEXT tile's rows, read during the current tile
                TileWalk<DYN> w(ctrl, abort_flag, a.header, a.tiles, total, false, a.n_compute);
                for (; w.valid(); w.advance()) {
                    const Tile t = decode_tile(w.d);
                    const bool two = t.valid > BM;
                    bool ok = true;
                    if (!DYN && a.gang && t.gang_size > 1) {
                        // entries that stream the same weight tiles start together (see gemm_tcgen05_m2.cu): with the
                        // static stride they sit on different CTAs (grid >= 8, checked by the launcher)
                        int32_t* cnt = a.gang + (w.L - t.gang_m);
                        asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(cnt) : "memory");
                        const unsigned long long t0 = globaltimer();
                        uint32_t spins = 0;
                        while (ld_acquire(cnt) < t.gang_size) {
                            if ((++spins & 63u) == 0u) {
                                if (*abort_flag) { ok = false; break; }
                                const unsigned long long limit =
                                    a.header->wait_limit_us ? 1000ull * a.header->wait_limit_us : WAIT_LIMIT_NS;
                                if (globaltimer() - t0 > limit) {
                                    *abort_flag = 1u;
                                    atomicCAS(&a.header->status, 0, (int)MOK_ERR_TIMEOUT);
                                    a.header->where = 43;
                                    ok = false;
                                    break;
                                }
                            }
                        }
                        if (!ok) break;
                    }
                    if (t.kind) {
                        // every gate/up tile of these rows has stored h: n1 tiles x 4 epilogue warps per 128-row half
                        const int need = a.n1 * (two ? 8 : 4);
                        const int32_t* flag = a.ready + t.mt;
                        if (peek < need && ld_acquire(flag) < need) {
                            const long long w0 = a.dbg ? clock64() : 0;
                            const unsigned long long t0 = globaltimer();
                            uint32_t spins = 0;
                            while (ld_acquire(flag) < need) {
                                __nanosleep(64);
                                if ((++spins & 63u) == 0u) {
                                    if (*abort_flag) { ok = false; break; }
                                    const unsigned long long limit =
                                        a.header->wait_limit_us ? 1000ull * a.header->wait_limit_us : WAIT_LIMIT_NS;
                                    if (globaltimer() - t0 > limit) {
                                        *abort_flag = 1u;
                                        atomicCAS(&a.header->status, 0, (int)MOK_ERR_TIMEOUT);
                                        a.header->where = 40;
                                        ok = false;
                                        break;
                                    }
                                }
                            }
                            if (a.dbg) d_ready += clock64() - w0;
                        }
                        if (!ok) break;
                        // the rows were written through the async proxy by other CTAs and are read through it below
                        asm volatile("fence.proxy.async;" ::: "memory");
                    }
                    const bool staged_a = !t.kind && a.comm_ctas > 0;     // the A rows come from the communication CTAs' slot
                    if (staged_a) {
                        const int32_t* flag = a.staged + t.mt;
                        if (ld_acquire(flag) < 1) {
                            const unsigned long long t0 = globaltimer();
                            uint32_t spins = 0;
                            while (ld_acquire(flag) < 1) {
                                __nanosleep(64);
                                if ((++spins & 63u) == 0u) {
                                    if (*abort_flag) { ok = false; break; }
                                    const unsigned long long limit =
                                        a.header->wait_limit_us ? 1000ull * a.header->wait_limit_us : WAIT_LIMIT_NS;
                                    if (globaltimer() - t0 > limit) {
                                        *abort_flag = 1u;
                                        atomicCAS(&a.header->status, 0, (int)MOK_ERR_TIMEOUT);
                                        a.header->where = 47;
                                        ok = false;
                                        break;
                                    }
                                }
                            }
                        }
                        if (!ok) break;
                        // the rows were written through the generic proxy by another CTA and are read through the async one
                        asm volatile("fence.proxy.async;" ::: "memory");
                    }
                    const int xrow = (t.mt % COMM_SLOTS) * TM;
                    const int kblocks = t.kind ? a.kb2 : a.kb1;
                    peek = 0;
                    for (int sub = 0; sub < t.cnt && ok; ++sub) {
                    const int n = t.n + sub;
                    const bool narrow = !t.kind && narrow_last && n == a.n1 - 1;
                    const int brow0 = t.kind ? t.e * a.H + n * BN : t.e * 2 * a.I + n * (BN / 2);
                    const int brow1 = t.kind ? brow0 + BN / 2 : brow0 + a.I;
                    for (int kb = 0; kb < kblocks; ++kb) {
                        if (sub == t.cnt - 1 && kb == (kblocks >> 1) && w.Ln < total) {   // the next entry's descriptor has arrived by now
                            const Tile tn = decode_tile(w.dn);
                            if (tn.kind) peek = ld_acquire(a.ready + tn.mt);
                        }
                        ok = wait_bar(smem_u32(&ctrl->empty[s]), ph ^ 1u, abort_flag, a.header, 1);
                        if (!ok) break;
                        const uint32_t full = smem_u32(&ctrl->full[s]);
                        const uint32_t sa = base + s * STAGE_BYTES, sb = sa + 2 * A_BYTES;
                        if (t.kind) {
                            // (the gather threads have nothing to bring: their arrivals on the stage are made here)
                            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(full), "r"((uint32_t)GATHER_THREADS) : "memory");
                            mbar_expect_tx(full, B_BYTES + (two ? 2 : 1) * A_BYTES);
                            const int hrow = a.ring ? (t.mt % a.ring) * TM : t.row0;
                            tma_load_2d(sa, &mapHld, full, kb * BK, hrow);
                            if (two) tma_load_2d(sa + A_BYTES, &mapHld, full, kb * BK, hrow + BM);
                            tma_load_2d(sb, &mapWd, full, kb * BK, brow0);
                            tma_load_2d(sb + B_BYTES / 2, &mapWd, full, kb * BK, brow1);
                        } else {
                            uint32_t a_bytes = 0;
                            if (staged_a) {     // (the gather threads have nothing to bring here either)
                                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(full), "r"((uint32_t)GATHER_THREADS) : "memory");
                                a_bytes = (two ? 2 : 1) * A_BYTES;
                            }
                            mbar_expect_tx(full, (narrow ? B_BYTES / 2 : B_BYTES) + a_bytes);
                            if (staged_a) {
                                tma_load_2d(sa, &mapXg, full, kb * BK, xrow);
                                if (two) tma_load_2d(sa + A_BYTES, &mapXg, full, kb * BK, xrow + BM);
                            }
                            if (narrow) {
                                tma_load_2d(sb, &mapWgu64, full, kb * BK, brow0);
                                tma_load_2d(sb + B_BYTES / 4, &mapWgu64, full, kb * BK, brow1);
                            } else {
                                tma_load_2d(sb, &mapWgu, full, kb * BK, brow0);
                                tma_load_2d(sb + B_BYTES / 2, &mapWgu, full, kb * BK, brow1);
                            }
                        }
                        if (++s == STAGES) { s = 0; ph ^= 1u; }
                    }
                    }
                    if (!ok) break;
                }
                if (a.dbg) atomicAdd(&a.header->dbg[2][DBG_PROD_WAIT_EMPTY], (unsigned long long)d_ready);
            }
        } else if (warp == 1) {
            // -------------------------------------------------------------- MMA issuer
            if (lane == 0) {
                int s = 0;
                uint32_t ph = 0, ap0 = 0, ap1 = 0;
                const bool dbg = a.dbg != 0;
                // debug counters: index 0 = gate/up tiles, 1 = down tiles
                long long d_full0 = 0, d_full1 = 0, d_te0 = 0, d_te1 = 0, d_kb0 = 0, d_kb1 = 0, d_rows0 = 0, d_rows1 = 0,
                          d_tot0 = 0, d_tot1 = 0;
                const unsigned long long d_ns0 = dbg ? globaltimer() : 0ull;
                const long long d_c0 = dbg ? clock64() : 0;
                TileWalk<DYN> w(ctrl, abort_flag, a.header, a.tiles, total, false, a.n_compute);
                for (; w.valid(); w.advance()) {
                    const Tile t = decode_tile(w.d);
                    const bool two = t.valid > BM;
                    const int kblocks = t.kind ? a.kb2 : a.kb1;
                    const long long tile0 = dbg ? clock64() : 0;
                    long long w0 = tile0, w_full = 0, w_te = 0;
                    bool ok = true;
                    for (int sub = 0; sub < t.cnt && ok; ++sub) {
                    const int n = t.n + sub;
                    uint32_t idesc = IDESC;
                    if (t.kind) {
                        if (a.H - n * BN < BN) idesc = idesc_n((a.H - n * BN + 15) & ~15);
                    } else if (narrow_last && n == a.n1 - 1) {
                        idesc = idesc_n(BN / 2);
                    }
                    if (dbg) w0 = clock64();
                    ok = wait_bar(smem_u32(&ctrl->tempty[0]), ap0 ^ 1u, abort_flag, a.header, 2);
                    if (dbg) w_te += clock64() - w0;
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t d0 = tmem_base, d1 = tmem_base + BN;
                    for (int kb = 0; kb < kblocks; ++kb) {
                        if (dbg) w0 = clock64();
                        ok = wait_bar(smem_u32(&ctrl->full[s]), ph, abort_flag, a.header, 3);
                        if (dbg) w_full += clock64() - w0;
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t sa = base + s * STAGE_BYTES;
                        const uint64_t a0 = make_smem_desc(sa), a1 = make_smem_desc(sa + A_BYTES);
                        const uint64_t bd = make_smem_desc(sa + 2 * A_BYTES);
#pragma unroll
                        for (int j = 0; j < BK / UMMA_K; ++j)
                            tc_mma<1>(d0, a0 + (uint64_t)(j * 2), bd + (uint64_t)(j * 2), idesc, (kb | j) ? 1u : 0u);
                        if (kb == kblocks - 1) { tc_commit<1>(smem_u32(&ctrl->tfull[0])); ap0 ^= 1u; }
                        if (two) {
                            if (kb == 0) {
                                if (dbg) w0 = clock64();
                                ok = wait_bar(smem_u32(&ctrl->tempty[1]), ap1 ^ 1u, abort_flag, a.header, 8);
                                if (dbg) w_te += clock64() - w0;
                                if (!ok) break;
                                tc_fence_after();
                            }
#pragma unroll
                            for (int j = 0; j < BK / UMMA_K; ++j)
                                tc_mma<1>(d1, a1 + (uint64_t)(j * 2), bd + (uint64_t)(j * 2), idesc, (kb | j) ? 1u : 0u);
                        }
                        tc_commit<1>(smem_u32(&ctrl->empty[s]));
                        if (++s == STAGES) { s = 0; ph ^= 1u; }
                    }
                    if (!ok) break;
                    if (two) { tc_commit<1>(smem_u32(&ctrl->tfull[1])); ap1 ^= 1u; }
                    }
                    if (!ok) break;
                    // ring mode: every load of h of this down entry has landed (its stages' full barriers were passed)
                    if (a.ring && t.kind && a.starve != 2)
                        asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(a.consumed + t.mt) : "memory");
                    // communication CTAs: every load of this gate/up tile from its staging slot has landed
                    if (a.comm_ctas > 0 && !t.kind && a.starve != 2)
                        asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(a.released + t.mt) : "memory");
                    if (dbg) {
                        const long long dt = clock64() - tile0, units = (long long)(two ? 2 : 1) * kblocks * t.cnt;
                        if (t.kind) { d_full1 += w_full; d_te1 += w_te; d_kb1 += units; d_rows1 += (long long)t.valid * kblocks * t.cnt; d_tot1 += dt; }
                        else        { d_full0 += w_full; d_te0 += w_te; d_kb0 += units; d_rows0 += (long long)t.valid * kblocks; d_tot0 += dt; }
                    }
                }
                if (dbg) {
                    const unsigned long long ns = globaltimer() - d_ns0, cyc = (unsigned long long)(clock64() - d_c0);
                    {   // slot 0: the whole kernel (imbalance of the tile hand-out, clock)
                        unsigned long long* d = a.header->dbg[0];
                        atomicAdd(d + DBG_MMA_TOTAL, cyc);
                        atomicMax(d + DBG_MMA_TOTAL_MAX, cyc);
                        atomicAdd(d + DBG_MMA_TOTAL_NS, ns);
                        atomicAdd(d + DBG_CTAS, 1ull);
                    }
                    const double both = (double)(d_tot0 + d_tot1);
                    for (int q = 0; q < 2; ++q) {
                        unsigned long long* d = a.header->dbg[1 + q];
                        const long long tot = q ? d_tot1 : d_tot0;
                        // the CTA's wall time is split between the two kinds in proportion to the cycles spent in their tiles
                        atomicAdd(d + DBG_MMA_WAIT_FULL, (unsigned long long)(q ? d_full1 : d_full0));
                        atomicAdd(d + DBG_MMA_WAIT_TEMPTY, (unsigned long long)(q ? d_te1 : d_te0));
                        atomicAdd(d + DBG_MMA_TOTAL, (unsigned long long)tot);
                        atomicMax(d + DBG_MMA_TOTAL_MAX, (unsigned long long)tot);
                        atomicAdd(d + DBG_MMA_TOTAL_NS, both > 0 ? (unsigned long long)((double)ns * (double)tot / both) : 0ull);
                        atomicAdd(d + DBG_KBLOCKS, (unsigned long long)(q ? d_kb1 : d_kb0));
                        atomicAdd(d + DBG_ROWS_KB, (unsigned long long)(q ? d_rows1 : d_rows0));
                        atomicAdd(d + DBG_CTAS, 1ull);
                    }
                }
            }
        } else if (DYN && warp == 2) {
            // -------------------------------------------------------------- scheduler (dynamic mode)
            if (lane == 0) {
                // draws list positions in order from one global counter, a few tiles ahead of the roles.  Whoever draws
                // a position runs, and everything a down tile waits for sits at smaller positions, which were drawn before.
                int slot = 0;
                uint32_t qph = 0;
                for (;;) {
                    const int L = atomicAdd(a.next_tile, 1);
                    if (!wait_bar(smem_u32(&ctrl->q_empty[slot]), qph ^ 1u, abort_flag, a.header, 32)) break;
                    *reinterpret_cast<volatile int32_t*>(&ctrl->q_tile[slot]) = L < total ? L : -1;
                    mbar_arrive(smem_u32(&ctrl->q_full[slot]));
                    if (++slot == QSLOTS) { slot = 0; qph ^= 1u; }
                    if (L >= total) break;
                }
            }
        }
        __syncwarp();
    } else if (warp >= 4 + EPI_WARPS) {
        // ------------------------------------------------------------------ gather warps (pull dispatch)
        reg_dec<REGS_GATHER>();
        const int gw = warp - (4 + EPI_WARPS), sub = lane >> 3, chunk = lane & 7;
        int s = 0;
        uint32_t ph = 0;
        TileWalk<DYN> w(ctrl, abort_flag, a.header, a.tiles, total, true, a.n_compute);
        for (; w.valid(); w.advance()) {
            const Tile t = decode_tile(w.d);
            bool ok = true;
            if (t.kind || a.comm_ctas > 0) {
                // down tile (or a gate/up tile whose rows the communication CTAs staged): both operands come by TMA and
                // the producer makes these threads' arrivals for them.  The warp
                // still follows the ring stage by stage (one polling lane): a parity wait is only meaningful while the
                // waiter is at most one phase ahead of the barrier, so it must not jump over the tile's stages.
                for (int kb = 0; kb < (t.kind ? a.kb2 : a.kb1) * t.cnt; ++kb) {
                    if (lane == 0) ok = wait_bar(smem_u32(&ctrl->empty[s]), ph ^ 1u, abort_flag, a.header, 5);
                    ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
                    if (!ok) break;
                    if (++s == STAGES) { s = 0; ph ^= 1u; }
                }
                if (!ok) break;
                continue;
            }
            const bool two = t.valid > BM;
            const __nv_bfloat16* src[16];
            uint32_t live = 0u;
            int tok[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {   // sixteen independent loads (a pad row reads the tile's last real row id)
                const int r = (i >> 3) * BM + gw * 32 + (i & 7) * 4 + sub;
                tok[i] = __ldg(a.row_token + t.row0 + min(r, t.valid - 1));
            }
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int r = (i >> 3) * BM + gw * 32 + (i & 7) * 4 + sub;
                if (a.peer_tokens > 0) {
                    const int pr = tok[i] / a.peer_tokens;
                    src[i] = a.peer_x[pr] + (size_t)(tok[i] - pr * a.peer_tokens) * a.H + chunk * 8;
                } else {
                    src[i] = a.x + (size_t)tok[i] * a.H + chunk * 8;
                }
                if (r < t.valid) live |= 1u << i;
            }
            for (int kb = 0; kb < a.kb1; ++kb) {
                ok = wait_bar(smem_u32(&ctrl->empty[s]), ph ^ 1u, abort_flag, a.header, 5);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const uint32_t sa = base + s * STAGE_BYTES;
                const bool in_k = (kb * BK + chunk * 8) < a.H;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    if (i < 8 || two) {
                        const int rr = gw * 32 + (i & 7) * 4 + sub;
                        const uint32_t dst = sa + (i >> 3) * A_BYTES + rr * 128 + ((chunk ^ (rr & 7)) << 4);
                        const bool on = in_k && ((live >> i) & 1u);    // pad rows and the K tail are written as zeros
                        cp_async_16(dst, on ? (const void*)(src[i] + kb * BK) : (const void*)a.x, on ? 16u : 0u);
                    }
                }
                cp_async_mbar_arrive(smem_u32(&ctrl->full[s]));
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
            if (!ok) break;
        }
        asm volatile("cp.async.wait_all;" ::: "memory");
        // (the gather warps help with the combine: more bytes in flight per SM)
        if (a.out != nullptr) combine_tokens<1>(a, ctrl, lane, false, abort_flag, false);
    } else {
        // ------------------------------------------------------------------ epilogue warps
        reg_inc<REGS_EPILOGUE>();
        const int acc = (warp - 4) >> 2;
        const int quad = warp & 3;                            // TMEM lane quadrant this warp may access
        const uint32_t slab = base + STAGES * STAGE_BYTES + (warp - 4) * SLAB_BYTES;
        uint32_t aph = 0;
        auto hand_back = [&]() {                               // the accumulator goes back to the MMA issuer
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctrl->tempty[acc]));
        };
        // one pass: 32 rows x 64 columns of packed bf16 through this warp's swizzled slab and out by TMA
        auto store_pass = [&](const uint32_t* v, const CUtensorMap* map, int col, int n_cols, int row) {
            if (lane == 0) tma_store_wait_read();             // the slab's previous store has been read out
            __syncwarp();
            const uint32_t line = slab + lane * 128;
#pragma unroll
            for (int q = 0; q < 8; ++q)
                st_shared_v4(line + ((q ^ (lane & 7)) << 4), v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
                if (col < n_cols) tma_store_2d(map, slab, col, row);
                tma_store_commit();
            }
        };
        TileWalk<DYN> w(ctrl, abort_flag, a.header, a.tiles, total, true, a.n_compute);
        for (; w.valid(); w.advance()) {
            const Tile t = decode_tile(w.d);
            if (acc == 1 && t.valid <= BM) continue;
            bool ok = true;
            for (int sub = 0; sub < t.cnt; ++sub) {
            const int n = t.n + sub;
            ok = wait_bar(smem_u32(&ctrl->tfull[acc]), aph, abort_flag, a.header, 4);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            aph ^= 1u;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * BN);
            const int row = t.row0 + acc * BM + quad * 32;
            if (t.kind) {
                // down tile: the whole 256-column accumulator row is read and packed first, the accumulator goes back to
                // the MMA issuer, and only then do the four 64-column passes through the slab start
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
                hand_back();
#pragma unroll
                for (int pass = 0; pass < 4; ++pass) store_pass(o + pass * 32, &mapY, n * BN + pass * 64, a.H, row);
            } else {
                // gate/up tile: silu(g) * u from columns c and c + 128 (c + 64 of a narrow last tile), 64 output columns
                // per pass; the next pass is read and computed before waiting for the slab of the current one
                int hrow = row;
                if (a.ring) {
                    hrow = (t.mt % a.ring) * TM + acc * BM + quad * 32;
                    if (t.mt >= a.ring) {
                        // the slot's previous rows (row tile mt - ring) must have been loaded by all their down entries
                        int free_ = 1;
                        if (lane == 0) {
                            const int32_t* c = a.consumed + (t.mt - a.ring);
                            if (ld_acquire(c) < a.need_d) {
                                const unsigned long long t0 = globaltimer();
                                uint32_t spins = 0;
                                while (ld_acquire(c) < a.need_d) {
                                    __nanosleep(64);
                                    if ((++spins & 63u) == 0u) {
                                        if (*abort_flag) { free_ = 0; break; }
                                        const unsigned long long limit =
                                            a.header->wait_limit_us ? 1000ull * a.header->wait_limit_us : WAIT_LIMIT_NS;
                                        if (globaltimer() - t0 > limit) {
                                            *abort_flag = 1u;
                                            atomicCAS(&a.header->status, 0, (int)MOK_ERR_TIMEOUT);
                                            a.header->where = 45;
                                            free_ = 0;
                                            break;
                                        }
                                    }
                                }
                            }
                            asm volatile("fence.proxy.async;" ::: "memory");
                        }
                        ok = __shfl_sync(0xffffffffu, free_, 0) != 0;
                        if (!ok) break;
                    }
                }
                const bool narrow = narrow_last && n == a.n1 - 1;
                const int passes = narrow ? 1 : 2;
                const uint32_t up_off = narrow ? BN / 4 : BN / 2;
                uint32_t cur[32], nxt[32];
                auto load_pass = [&](int pass, uint32_t (&o)[32]) {
#pragma unroll
                    for (int c = 0; c < 64; c += 32) {
                        uint32_t g[32], u[32];
                        tc_ld32(taddr + pass * 64 + c, g);
                        tc_ld32(taddr + up_off + pass * 64 + c, u);
                        tc_wait_ld();
                        if (pass == passes - 1 && c == 32) hand_back();   // the tile's last TMEM read: arithmetic comes after
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            o[(c >> 1) + i] = pack_bf16(swiglu(__uint_as_float(g[2 * i]), __uint_as_float(u[2 * i])),
                                                        swiglu(__uint_as_float(g[2 * i + 1]), __uint_as_float(u[2 * i + 1])));
                    }
                };
                load_pass(0, nxt);
#pragma unroll
                for (int pass = 0; pass < 2; ++pass) {
                    if (pass >= passes) break;
#pragma unroll
                    for (int i = 0; i < 32; ++i) cur[i] = nxt[i];
                    if (pass + 1 < passes) load_pass(pass + 1, nxt);
                    store_pass(cur, &mapHst, n * (BN / 2) + pass * 64, a.I, hrow);
                }
                if (lane == 0) {
                    // h of this warp's 32 rows is on its way: wait until the stores have completed (not only left shared
                    // memory), then publish one arrival for the M tile.  Release at GPU scope after a proxy fence: the
                    // down tiles read these rows through the async proxy from other SMs.
                    tma_store_wait_all();
                    asm volatile("fence.proxy.async;" ::: "memory");
                    __threadfence();
                    asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(a.ready + t.mt) : "memory");
                }
                __syncwarp();
            }
            }
            if (!ok) break;
        }
        if (lane == 0) tma_store_wait_all();
        __syncwarp();
        if (a.out != nullptr) combine_tokens<4>(a, ctrl, lane, warp == 4, abort_flag, true);
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

}  // namespace ff

template <bool DYN>
static cudaError_t launch_kernel(int grid, cudaStream_t s, const CUtensorMap& m0, const CUtensorMap& m1, const CUtensorMap& m2,
                                 const CUtensorMap& m3, const CUtensorMap& m4, const CUtensorMap& m5, const CUtensorMap& m6,
                                 const ff::FusedArgs& a) {
    using namespace ff;
    static PerDevice configured;
    int dev = 0, sm_count = 0;
    cudaError_t e = current_device(&dev);
    if (e != cudaSuccess) return e;
    e = configured.get(dev, &sm_count, [](int d, int* sms) {
        cudaError_t e2 = cudaFuncSetAttribute(fused_ffn_kernel<DYN>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        return e2 != cudaSuccess ? e2 : device_sm_count(d, sms);
    });
    if (e != cudaSuccess) return e;
    if (grid <= 0 || grid > sm_count) grid = sm_count;
    // Dynamic draw: a position is only drawn by a CTA that runs: an ordinary (programmatically serialised) launch --
    // unless tiles wait for communication CTAs, which then have to be resident like everybody else.
    if (DYN && a.comm_ctas == 0)
        return launch_pdl(fused_ffn_kernel<DYN>, dim3(grid), dim3(THREADS), (size_t)SMEM_BYTES, s, m0, m1, m2, m3, m4, m5, m6, a);
    // static list: tiles wait for tiles of other CTAs, so every CTA of the grid must be resident (cooperative launch).
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, fused_ffn_kernel<DYN>, m0, m1, m2, m3, m4, m5, m6, a);
}

// Host side.  `window_tiles`: distance (in list positions) between a group's gate/up tiles and its down tiles; 0 = the
// default (eight grids' worth of tiles with the dynamic draw, two with the static stride: measured best), -1 = none
// (a group's down tiles directly behind its gate/up tiles).
cudaError_t launch_fused_ffn(const __nv_bfloat16* x, int T, int H, int I, int E, const __nv_bfloat16* Wgu,
                             const __nv_bfloat16* Wd, const WsLayout& L, char* ws, int grid, int window_tiles, bool dynamic,
                             bool gang_sync, bool dbg, int starve, cudaStream_t s, __nv_bfloat16* combine_out, int k,
                             bool shared, int h_ring_tiles, const void* const* peer_x, int peer_tokens, void* y_out,
                             int comm_ctas, void* xg) {
    using namespace ff;
    int dev = 0, sm_count = 0;
    cudaError_t e = current_device(&dev);
    if (e != cudaSuccess) return e;
    if ((e = device_sm_count(dev, &sm_count)) != cudaSuccess) return e;
    if (grid <= 0 || grid > sm_count) grid = sm_count;
    // communication CTAs come out of the grid; at least one CTA computes
    if (comm_ctas < 0 || (comm_ctas > 0 && !xg)) return cudaErrorInvalidValue;
    if (comm_ctas >= grid) comm_ctas = grid - 1;
    const int total_grid = grid;
    grid -= comm_ctas;                                  // from here on: the CTAs that work on tiles
    WsHeader* hdr = reinterpret_cast<WsHeader*>(ws + L.header);
    const int n1 = (I + BN / 2 - 1) / (BN / 2), n2 = (H + BN - 1) / BN;
    // N tiles per down entry: as many as make its k-blocks about those of a gate/up entry (K = H against K = I)
    int q = ((H + BK - 1) / BK + (I + BK - 1) / BK / 2) / ((I + BK - 1) / BK);
    if (q < 1) q = 1;
    if (q > n2) q = n2;
    if (window_tiles == 0) window_tiles = dynamic ? 8 * grid : 2 * grid;
    int window = window_tiles < 0 ? 0 : (window_tiles + n1 - 1) / n1;      // in M tiles
    // ring of h: only as many slots as there are row tiles are ever used; the window must leave 2 * GROUP_TILES slots
    const int max_mt2 = L.max_mt / 2;
    const int ring = h_ring_tiles > 0 && h_ring_tiles < max_mt2 ? h_ring_tiles : 0;
    if (ring > 0 && ring < H_RING_MIN_TILES) return cudaErrorInvalidValue;
    if (ring > 0 && window > ring - 2 * GROUP_TILES) window = ring - 2 * GROUP_TILES;
    int4* tiles = reinterpret_cast<int4*>(ws + L.ftiles);
    int32_t* ready = reinterpret_cast<int32_t*>(ws + L.ready);
    // enough blocks for one warp per group of a large batch; every block rebuilds the per-expert offsets itself
    int tblocks = (int)((L.max_mt / 2 / GROUP_TILES + E) / (MAX_E / 32)) + 1;
    if (tblocks > sm_count) tblocks = sm_count;
    e = launch_pdl(fused_tiles_kernel, dim3(tblocks), dim3(MAX_E), 0, s, reinterpret_cast<const int32_t*>(ws + L.counts),
                   reinterpret_cast<const int32_t*>(ws + L.pad_offsets), reinterpret_cast<const int32_t*>(ws + L.mt_start2), E,
                   n1, n2, q, window, L.max_ftiles, tiles, ready, ready + max_mt2, ready + 2 * max_mt2, ready + 3 * max_mt2, hdr);
    if (e != cudaSuccess) return e;

    CUtensorMap mWgu, mWgu64, mHst, mHld, mWd, mY, mXg;
    void* h = ws + L.h;
    void* y = y_out ? y_out : ws + L.y;
    if (!tmap::bf16_sw128(&mWgu, Wgu, (uint64_t)E * 2 * I, (uint64_t)H, BN / 2) ||
        !tmap::bf16_sw128(&mWgu64, Wgu, (uint64_t)E * 2 * I, (uint64_t)H, BN / 4) ||
        !tmap::bf16_sw128(&mHst, h, (uint64_t)(ring ? ring * TM : L.Rpad), (uint64_t)I, 32) ||
        !tmap::bf16_sw128(&mHld, h, (uint64_t)(ring ? ring * TM : L.Rpad), (uint64_t)I, BM) ||
        !tmap::bf16_sw128(&mWd, Wd, (uint64_t)E * H, (uint64_t)I, BN / 2) ||
        !tmap::bf16_sw128(&mY, y, (uint64_t)L.Rpad, (uint64_t)H, 32))
        return cudaErrorInvalidValue;
    mXg = mHld;      // (unused without communication CTAs)
    if (comm_ctas > 0 && !tmap::bf16_sw128(&mXg, xg, (uint64_t)COMM_SLOTS * TM, (uint64_t)H, BM)) return cudaErrorInvalidValue;
    FusedArgs a;
    memset(&a, 0, sizeof(a));
    a.x = x;
    a.peer_tokens = peer_x ? peer_tokens : 0;
    for (int r = 0; peer_x && r < MOK_MAX_RANKS; ++r) a.peer_x[r] = reinterpret_cast<const __nv_bfloat16*>(peer_x[r]);
    a.row_token = reinterpret_cast<const int32_t*>(ws + L.row_token);
    a.tiles = tiles;
    a.n_tiles = &hdr->n_ftiles;
    a.next_tile = &hdr->next_tile;
    a.gang = nullptr;
    if (!dynamic && gang_sync && grid >= GROUP_TILES && L.gang_bytes >= sizeof(int32_t) * (size_t)L.max_ftiles) {
        e = cudaMemsetAsync(ws + L.gang, 0, sizeof(int32_t) * (size_t)L.max_ftiles, s);
        if (e != cudaSuccess) return e;
        a.gang = reinterpret_cast<int32_t*>(ws + L.gang);
    }
    a.ready = ready;
    a.consumed = ready + max_mt2;
    a.staged = ready + 2 * max_mt2;
    a.released = ready + 3 * max_mt2;
    a.comm_ctas = comm_ctas;
    a.n_compute = grid;
    a.xg = reinterpret_cast<__nv_bfloat16*>(xg);
    a.mt_start2 = reinterpret_cast<const int32_t*>(ws + L.mt_start2);
    a.tile_expert2 = reinterpret_cast<const int32_t*>(ws + L.tile_expert2);
    a.counts = reinterpret_cast<const int32_t*>(ws + L.counts);
    a.pad_offsets = reinterpret_cast<const int32_t*>(ws + L.pad_offsets);
    a.n_mtiles2 = &hdr->n_mtiles2;
    a.max_mt2 = max_mt2;
    a.ring = ring;
    a.need_d = (n2 + q - 1) / q;
    a.max_tiles = L.max_ftiles;
    a.H = H; a.I = I; a.E = E;
    a.n1 = n1; a.n2 = n2;
    a.kb1 = (H + BK - 1) / BK;
    a.kb2 = (I + BK - 1) / BK;
    a.dbg = dbg ? 1 : 0;
    a.starve = starve;
    a.header = hdr;
    a.y = reinterpret_cast<const __nv_bfloat16*>(y);
    a.ysh = shared ? reinterpret_cast<const __nv_bfloat16*>(ws + L.ysh) : nullptr;
    a.pos = reinterpret_cast<const int32_t*>(ws + L.pos);
    a.w = reinterpret_cast<const float*>(ws + L.w);
    a.out = combine_out;
    a.T = T;
    a.k = k;

    return dynamic ? launch_kernel<true>(total_grid, s, mWgu, mWgu64, mHst, mHld, mWd, mY, mXg, a)
                   : launch_kernel<false>(total_grid, s, mWgu, mWgu64, mHst, mHld, mWd, mY, mXg, a);
}

}  // namespace mok
