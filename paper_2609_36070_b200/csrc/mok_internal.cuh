// Internal declarations shared by the translation units of libmok (not part of the public ABI).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda.h>
#include <stdint.h>
#include <stddef.h>
#include <atomic>
#include "mok.h"

namespace mok {

constexpr int TILE_M = 128;          // rows of one CTA's GEMM tile; expert segments are padded internally to tile_m =
                                     // 128 (single CTAs) or 256 (CTA pairs) rows
constexpr int SCHED_CHUNK = 2048;    // routes handled by one block of the schedule kernels
constexpr int MAX_E = 512;
constexpr int MAX_K = 32;

// Device-side control block at the start of the workspace.
struct WsHeader {
    int32_t status;        // 0 or a negative mok_status written by a kernel
    int32_t n_mtiles;      // number of tile_m-row tiles of the padded dispatch buffer (written by the schedule)
    int32_t n_mtiles2;     // number of 2*tile_m-row tiles of the same buffer (second tile table)
    int32_t where;         // diagnostic: which wait gave up (site number inside the kernel)
    uint32_t wait_limit_us; // 0 = default (2 s): bound of every mbarrier wait, in microseconds
    int32_t n_flag;        // tensor-core router: tokens on the near-tie list of the current call
    int32_t n_ftiles;      // length of the fused expert-FFN kernel's tile list (gate/up tiles + down tiles)
    int32_t next_tile;     // its dynamic hand-out: the next list position to draw
    int32_t ffn_done;      // that kernel's epilogue warps whose last store has completed (gate of its in-launch combine)
    int32_t combine_next;  // its in-launch combine: the next token to draw
    int32_t pad[54];
    // optional counters of the tcgen05 GEMMs (config.debug): [slot][counter]; SM cycles summed over CTAs unless stated
    unsigned long long dbg[4][MOK_DEBUG_COUNTERS];
};
enum { DBG_MMA_WAIT_FULL = 0, DBG_MMA_WAIT_PFULL, DBG_MMA_WAIT_TEMPTY, DBG_MMA_TOTAL, DBG_KBLOCKS,
       DBG_PROD_WAIT_EMPTY, DBG_EPI_WAIT_TFULL, DBG_EPI_TOTAL,
       DBG_MMA_TOTAL_MAX,     // the busiest CTA's MMA-issuer time (cycles, maximum over CTAs)
       DBG_MMA_TOTAL_NS,      // MMA-issuer time in nanoseconds of the global timer, summed over CTAs (cycles / ns = SM clock)
       DBG_ROWS_KB,           // valid (non-padding) rows x k-blocks issued (256-row kernel only)
       DBG_CTAS };            // CTAs that reported

// Byte offsets of every workspace region, computed on the host from the sizes alone (no readback).
struct WsLayout {
    size_t header, idx, w, counts, offsets, pad_offsets, mt_start, tile_expert, perm, inv, pos, blk_hist;
    size_t mt_start2, tile_expert2;   // the same segments cut into tiles of 2*tile_m rows
    size_t row_token;     // int32 [Rpad]: source token of every row of the padded dispatch space (pad rows undefined)
    size_t wr_split;      // bf16 [ldl, H]: W_r split into hi/mid/lo parts for the tensor-core router
    size_t logits;        // fp32 [Tpad, ldl] partial logits of the tensor-core router (ldl = 3E rounded up to 8, or
                          // 3 * (E rounded up to 32) if larger: the one-kernel router pads each part to 32 rows)
    size_t xg, h, y, hs, ysh;
    size_t x8, sx, h8, sh;   // MXFP8 mode: quantised token rows + row-major scales, quantised gated activation + scale atoms
    size_t ftiles, ready;    // fused expert-FFN kernel: tile list (int4 per tile) and per-M-tile completion counters
                             // (two int32 per 256-row tile: gate/up arrivals, then down-tile arrivals at + max_mt / 2)
    int32_t h_ring;          // > 0: `h` holds only this many 256-row tiles (a ring), and there is no `xg` region
    size_t gang;             // 256-row kernel: gang-start counters, one int32 per list position of the largest GEMM
    size_t gang_bytes;
    int32_t max_ftiles;
    size_t total;
    int32_t R;            // T*k
    int32_t Rpad;         // upper bound on padded rows for either tile_m (multiple of 256)
    int32_t max_mt;       // Rpad / 128
    int32_t Tpad;         // T rounded up to 256
    int32_t n_blk;        // schedule blocks
};

bool ws_layout(int T, int H, int I, int Is, int E, int k, WsLayout* L, bool mx = false, int h_ring_tiles = 0);

// Arguments of the grouped GEMM (both implementations).  Rows live in a padded space: expert e owns rows
// [128*mt_start[e], 128*mt_start[e+1]); tile q belongs to expert tile_expert[q].  In dense mode (shared
// expert) there is one expert and ceil(dense_rows/128) tiles.
struct GemmArgs {
    const __nv_bfloat16* A;      // [a_rows, K]; with row_token set, A = x [T, K] and rows are gathered through it
    const __nv_bfloat16* B;      // SWIGLU: [E, 2*N, K] (gate rows then up rows); else [E, N, K]
    void* C;                     // [rows_pad, ldc] bf16 (fp32 for the router logits)
    int32_t K, N, E;
    int32_t ldc;                 // elements between consecutive rows of C
    const int32_t* row_token;    // device [rows_pad] or NULL: padded row -> token (gather fused into the A loads)
    const int32_t* counts;       // device [E]
    const int32_t* pad_offsets;  // device [E+1]: first row of each expert in the padded row space
    int32_t rows_pad;            // allocated rows of C (multiple of 128)
    int32_t a_rows;              // allocated rows of A (reads beyond it are treated as zero)
    int32_t dense_rows;          // > 0: dense mode with this many valid rows
    int32_t total_rows;          // routed mode: T*k (host-side hint for choosing the kernel; not read on the device)
    const int32_t* n_mtiles;     // device (routed mode)
    const int32_t* tile_expert;  // device [max_mt]
    const int32_t* mt_start;     // device [E+1]
    int32_t max_mt;
    int32_t tile_m;              // rows of one tile of the padded row space: 128, or 256 for CTA pairs
    int32_t dbg_slot;            // >= 0: accumulate wait-time counters into header->dbg[dbg_slot]
    int32_t starve;              // test hook: the TMA producer issues nothing, so the kernel's waits run out
    int32_t n_tile;              // 128-row kernel, fp32 epilogue: columns per N tile (32 / 64 / 128; 0 = 256)
    int32_t tile_sched;          // 256-row kernel, routed forward GEMMs: 1 = tiles handed out by cluster launch control
    int32_t* gang;               // 256-row kernel, forward layout: per list position, arrivals of the row tiles that share
                                 // one weight tile (zeroed before the launch), or NULL: no synchronised tile starts
    // K-range mode of the 256-row kernel (weight gradients): C holds E matrices [kgroup_rows, N]; A is ONE matrix
    // [kgroup_rows, K extent] and B ONE matrix [N, K extent] whose columns are the rows of the dispatch space; expert e
    // contracts over its padded segment [pad_offsets[e], pad_offsets[e+1]) (dense_rows > 0: one group over columns
    // 0 .. dense_rows).  lda / ldb: elements between consecutive rows of A / B (0 = K).
    int32_t kgroup_rows;
    int32_t lda, ldb;
    int32_t b_mn;                // 256-row kernel: B is W[e] = [K, N] with N contiguous (read MN-major), EPI_BF16 only
    int32_t gather_mn;           // K-range mode with both operands MN-major and row_token set: 1 = A, 2 = B is x or dout in
                                 // TOKEN order ([a_rows tokens, columns]) and its rows are pulled through row_token by the
                                 // gather warps (rows past an expert's count read as zero)
    WsHeader* header;
    // Expert-parallel pull dispatch (Section 3.1): with peer_tokens > 0 the ids in row_token are global,
    // id = source_rank * peer_tokens + token, and row `id` is read from peer_x[source_rank] (this GPU's own tokens
    // or a peer's, mapped into this process) with plain 16-byte asynchronous copies -- never a multicast load.
    int32_t peer_tokens;
    const __nv_bfloat16* peer_x[MOK_MAX_RANKS];
    // MXFP8 mode (Section 3.4): A and B hold E4M3 codes (one byte per element) and these are the E8M0 block scales.
    const uint8_t* sfa;          // GATHER: row-major [tokens, sfa_stride] of x; else 512-byte atoms [rows_pad/128][KG]
    const uint8_t* sfb;          // 512-byte atoms [E (x2 for gate, up)][ceil(N/128)][KG] of the weights
    uint8_t* sfc;                // SWIGLU epilogue: scale atoms of the quantised gated activation [rows_pad/128][ceil(N/128)]
    int32_t sfa_stride;          // bytes between the scale rows of consecutive tokens (GATHER)
    const uint8_t* peer_sfa[MOK_MAX_RANKS];   // expert-parallel MXFP8: every rank's row-major token scales (with peer_x
                                              // holding every rank's E4M3 token rows)
};

// Source row of the fused gather: row `tok` of A, or of the owning rank's token buffer in expert-parallel mode.
__device__ __forceinline__ const __nv_bfloat16* gather_row(const GemmArgs& a, int tok) {
    if (a.peer_tokens > 0) {
        const int r = tok / a.peer_tokens;
        return a.peer_x[r] + (size_t)(tok - r * a.peer_tokens) * a.K;
    }
    return a.A + (size_t)tok * a.K;
}

// kernels' host launchers (each returns a cudaError_t from the launch)
cudaError_t launch_router_simt(const __nv_bfloat16* x, const float* Wr, const float* bias, int T, int H, int E, int k,
                               int32_t* idx, float* w, cudaStream_t s);
cudaError_t launch_schedule(const int32_t* idx, int T, int E, int k, int tile_m, int pad_m, const WsLayout& L, char* ws,
                            int32_t* counts_out, int32_t* offsets_out, int32_t* perm_out, int32_t* inv_out,
                            cudaStream_t s, int32_t* row_route = nullptr);
cudaError_t launch_gather(const __nv_bfloat16* x, int H, int k, int tile_m, const WsLayout& L, char* ws, cudaStream_t s,
                          __nv_bfloat16* dst = nullptr);   // dst = NULL: the workspace's own expert-sorted buffer
cudaError_t launch_combine(const WsLayout& L, char* ws, int T, int H, int k, bool shared, __nv_bfloat16* out,
                           cudaStream_t s, bool unit_weights = false);
cudaError_t launch_ep_schedule(const int32_t* idx_all, int n_ranks, int rank, int routes_per_rank, int k, int tokens_per_rank,
                               int experts_local, int tile_m, const WsLayout& L, char* ws, int32_t* pos_out, int32_t* M_out,
                               int32_t* S_out, int32_t* phi_rank_out, int32_t* phi_index_out, cudaStream_t s);
// the expert-parallel owner-side combine; unit_weights: plain sum of the k rows (backward pass)
int ep_combine_impl(const mok_ep_combine_args* a, bool unit_weights);
// workspace layout of one expert-parallel rank (ep.cu)
bool ep_layout(int n_ranks, int T_local, int H, int I, int Is, int E, int k, WsLayout* L, bool mx = false);
int run_gemm(GemmArgs g, bool swiglu, const mok_config* cfg, const WsLayout& L, char* ws, cudaStream_t s);
int gang_prepare(GemmArgs& g, bool swiglu, const mok_config* cfg, const WsLayout& L, char* ws, cudaStream_t s);
int tile_rows(const mok_config* cfg, int I);
bool fused_gather(const mok_config* cfg, int I);
int cuda_fail(cudaError_t e);
cudaError_t launch_gemm_simt(const GemmArgs& a, bool swiglu, cudaStream_t s);
enum { EPI_BF16 = 0, EPI_SWIGLU = 1, EPI_F32 = 2 };
cudaError_t launch_gemm_tc(const GemmArgs& a, int epi, int grid, cudaStream_t s);
cudaError_t launch_gemm_tn(const GemmArgs& a, int epi, int grid, cudaStream_t s);   // tokens on the MMA's N side
cudaError_t launch_gemm_m2(const GemmArgs& a, int epi, int grid, cudaStream_t s);   // 256-row tiles, two accumulators
cudaError_t launch_gemm_mx(const GemmArgs& a, int epi, int grid, cudaStream_t s);   // MXFP8 operands, block-scaled MMA
// routed gate/up + SwiGLU + down in one persistent launch (tile list + kernel); needs the schedule's 256-row tile table
cudaError_t launch_fused_ffn(const __nv_bfloat16* x, int T, int H, int I, int E, const __nv_bfloat16* Wgu,
                             const __nv_bfloat16* Wd, const WsLayout& L, char* ws, int grid, int window_tiles, bool dynamic,
                             bool gang_sync, bool dbg, int starve, cudaStream_t s, __nv_bfloat16* combine_out = nullptr,
                             int k = 0, bool shared = false,    // combine_out != NULL: the combine runs in the same launch
                             int h_ring_tiles = 0,              // > 0: h is a ring of that many 256-row tiles
                             const void* const* peer_x = nullptr, int peer_tokens = 0,   // expert parallelism: every rank's token rows
                             void* y_out = nullptr,             // where the down tiles go (NULL: the workspace's y)
                             int comm_ctas = 0, void* xg = nullptr);   // communication CTAs and their staging slots
constexpr int FFN_COMM_SLOTS = 24;       // 256-row slots of that staging buffer ([FFN_COMM_SLOTS * 256, H] bf16)
// whether the routed expert FFN runs as the one launch for these sizes and knobs; *sync: with synchronised tile starts
bool fused_ffn_choice(const mok_config* cfg, int H, int I, int tile_m, long long rows, int experts, int max_ftiles, bool* sync);
constexpr int H_RING_MIN_TILES = 24;     // smallest ring of the gated activation (see gemm_fused.cu)
cudaError_t launch_mx_quantize_rows(const __nv_bfloat16* in, long long rows, int K, uint8_t* codes, uint8_t* scales,
                                    cudaStream_t s);
cudaError_t launch_mx_quantize_atoms(const __nv_bfloat16* in, int groups, int rows_per_group, int K, uint8_t* codes,
                                     uint8_t* scales, cudaStream_t s);
cudaError_t launch_router_tc(const __nv_bfloat16* x, const float* Wr, const float* bias, int T, int H, int E, int k,
                             const WsLayout& L, char* ws, WsHeader* hdr, int grid, int tile_m, int variant, bool fused,
                             int32_t* idx, float* w, cudaStream_t s, const __nv_bfloat16* presplit = nullptr,
                             bool split_only = false);
bool router_fused_ok(int E, int k);     // the one-kernel projection + top-k serves this shape
cudaError_t launch_router_fused(const __nv_bfloat16* x, const __nv_bfloat16* split, const float* bias, int T, int H, int E,
                                int k, float* rows, int32_t* flagged, WsHeader* hdr, int grid, int32_t* idx, float* w,
                                cudaStream_t s);

inline __host__ __device__ size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Programmatic dependent launch: the kernels of one forward call are launched with the "programmatic stream
// serialization" attribute, so that a kernel's CTAs are scheduled (launch latency, parameter fetch) while its
// predecessor in the stream is still running.  Device side, first thing in every such kernel: let the successor be
// scheduled in turn, then wait until every predecessor grid has completed and its memory is visible.  Without the
// attribute both instructions do nothing.
__device__ __forceinline__ void pdl_enter() {
#if defined(__CUDA_ARCH__)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
#endif
}
extern thread_local bool g_pdl;       // set per forward call from config.serial_launches
template <class... P, class... A>
inline cudaError_t launch_pdl(void (*kernel)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, A&&... args) {
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = g_pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<P>(args)...);
}

// Launch state that belongs to ONE device.  cudaFuncSetAttribute (the opt-in to more than 48 KB of dynamic shared
// memory) applies to the device that is current when it is called, and the SM count is a property of that device, so
// a launcher that remembers "configured" per process would launch unconfigured kernels on a second GPU of the same
// process.  Each launcher keeps one PerDevice per kernel instantiation: value(dev) is 0 until `configure` has
// succeeded on that device and then holds what it returned (the SM count, or the number of co-resident CTA pairs).
// Concurrent first calls may both configure (the calls are idempotent) and store the same value.
constexpr int MAX_DEVICES = 64;
struct PerDevice {
    std::atomic<int> v[MAX_DEVICES];
    // configure(dev, &value) -> cudaError_t; value must come back > 0
    template <class F>
    cudaError_t get(int dev, int* out, F configure) {
        if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
        int cur = v[dev].load(std::memory_order_acquire);
        if (cur == 0) {
            cudaError_t e = configure(dev, &cur);
            if (e != cudaSuccess) return e;
            if (cur <= 0) return cudaErrorInvalidConfiguration;
            v[dev].store(cur, std::memory_order_release);
        }
        *out = cur;
        return cudaSuccess;
    }
};
inline cudaError_t current_device(int* dev) { return cudaGetDevice(dev); }
inline cudaError_t device_sm_count(int dev, int* sms) {
    return cudaDeviceGetAttribute(sms, cudaDevAttrMultiProcessorCount, dev);
}

}  // namespace mok
