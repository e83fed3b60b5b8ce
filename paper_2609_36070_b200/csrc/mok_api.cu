// Host side of libmok: argument validation, workspace layout and the launch sequence of the MoE layer forward
// (paper, Figure 1: router projection + top-k, dispatch scheduling, then dispatch / expert FFNs / combine).
// Nothing here synchronises with the device or reads counts back (Section 3.3), except mok_read_status and
// mok_moe_forward_host, which say so.
#include "mok_internal.cuh"
#include <string.h>

namespace mok {

static thread_local int g_last_cuda_error = 0;
thread_local bool g_pdl = true;
constexpr int M2_MIN_K = 512;    // shortest K for which the 256-row-tile kernel is chosen by default

int cuda_fail(cudaError_t e) {
    g_last_cuda_error = (int)e;
    return MOK_ERR_CUDA;
}

// Event sets of the per-stage profiler (mok_profile_begin / mok_profile_end).
struct Profiler {
    cudaEvent_t* ev = nullptr;      // [max_calls][MOK_STAGE_COUNT + 1]: event 0 opens the call, event st + 1 closes stage st
    uint8_t* pred = nullptr;        // [max_calls][MOK_STAGE_COUNT]: the event recorded just before stage st's closing event
                                    // (stages do not always run in the order of their numbers)
    int max_calls = 0, n_calls = 0;
};
static Profiler g_prof;

struct ProfileMarks {
    cudaEvent_t* ev = nullptr;
    uint8_t* pred = nullptr;
    int last = 0;
    cudaStream_t s = nullptr;
    void open() { if (ev) cudaEventRecord(ev[0], s); }
    void close(int stage) {
        if (!ev) return;
        cudaEventRecord(ev[stage + 1], s);
        pred[stage] = (uint8_t)last;
        last = stage + 1;
    }
};

static ProfileMarks profile_slot(const mok_config* cfg, cudaStream_t s) {
    ProfileMarks m;
    if (!cfg || !cfg->profile || !g_prof.ev || g_prof.n_calls >= g_prof.max_calls) return m;
    const int c = g_prof.n_calls++;
    m.ev = g_prof.ev + (size_t)c * (MOK_STAGE_COUNT + 1);
    m.pred = g_prof.pred + (size_t)c * MOK_STAGE_COUNT;
    m.s = s;
    return m;
}

static bool sizes_ok(int T, int H, int I, int Is, int E, int k) {
    if (T < 0 || H <= 0 || I <= 0 || Is < 0 || E <= 0 || k < 1) return false;
    if (k > E || k > MAX_K || E > MAX_E) return false;
    if ((H % 8) || (I % 8) || (Is % 8)) return false;
    if ((long long)T * k >= (1ll << 31) / 256) return false;
    return true;
}

bool ws_layout(int T, int H, int I, int Is, int E, int k, WsLayout* L, bool mx, int h_ring_tiles) {
    if (!sizes_ok(T, H, I, Is, E, k)) return false;
    if (mx && ((H % 32) || (I % 32))) return false;
    if (h_ring_tiles < 0 || (h_ring_tiles > 0 && (h_ring_tiles < H_RING_MIN_TILES || mx))) return false;
    memset(L, 0, sizeof(*L));
    L->h_ring = h_ring_tiles;
    const long long R = (long long)T * k;
    const long long nonempty_max = R < E ? R : E;
    long long Rpad = (R + nonempty_max * (2 * TILE_M - 1) + 2 * TILE_M - 1) / (2 * TILE_M) * (2 * TILE_M);
    if (Rpad < 2 * TILE_M) Rpad = 2 * TILE_M;
    L->R = (int32_t)R;
    L->Rpad = (int32_t)Rpad;
    L->max_mt = (int32_t)(Rpad / TILE_M);
    L->Tpad = (T + 2 * TILE_M - 1) / (2 * TILE_M) * (2 * TILE_M);
    if (L->Tpad < 2 * TILE_M) L->Tpad = 2 * TILE_M;
    L->n_blk = (int32_t)((R + SCHED_CHUNK - 1) / SCHED_CHUNK);
    if (L->n_blk < 1) L->n_blk = 1;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    L->header = take(sizeof(WsHeader));
    L->idx = take(sizeof(int32_t) * (size_t)(R > 0 ? R : 1));
    L->w = take(sizeof(float) * (size_t)(R > 0 ? R : 1));
    L->counts = take(sizeof(int32_t) * E);
    L->offsets = take(sizeof(int32_t) * (E + 1));
    L->pad_offsets = take(sizeof(int32_t) * (E + 1));
    L->mt_start = take(sizeof(int32_t) * (E + 1));
    L->tile_expert = take(sizeof(int32_t) * (size_t)L->max_mt);
    L->mt_start2 = take(sizeof(int32_t) * (E + 1));
    L->tile_expert2 = take(sizeof(int32_t) * (size_t)L->max_mt);
    L->perm = take(sizeof(int32_t) * (size_t)(R > 0 ? R : 1));
    L->inv = take(sizeof(int32_t) * (size_t)(R > 0 ? R : 1));
    L->pos = take(sizeof(int32_t) * (size_t)(R > 0 ? R : 1));
    L->blk_hist = take(sizeof(int32_t) * (size_t)L->n_blk * E);
    L->row_token = take(sizeof(int32_t) * (size_t)Rpad);
    size_t ldl = (size_t)(3 * E + 7) / 8 * 8;
    if (ldl < 3 * (size_t)((E + 31) / 32 * 32)) ldl = 3 * (size_t)((E + 31) / 32 * 32);
    L->wr_split = take(2 * ldl * H);
    L->logits = take(sizeof(float) * (size_t)L->Tpad * ldl);
    // (a ring of the gated activation belongs to the one-launch expert FFN, which gathers its rows itself: no copy of x)
    L->xg = take(h_ring_tiles > 0 ? 0 : 2 * (size_t)Rpad * H);
    const long long h_rows = h_ring_tiles > 0 && (long long)h_ring_tiles * 2 * TILE_M < Rpad ? (long long)h_ring_tiles * 2 * TILE_M : Rpad;
    L->h = take(2 * (size_t)h_rows * I);
    L->y = take(2 * (size_t)Rpad * H);
    {   // fused expert-FFN kernel: every 256-row tile times (gate/up N tiles + down N tiles), one counter per row tile
        const long long mt2 = Rpad / (2 * TILE_M), per = (I + 127) / 128 + (H + 255) / 256;
        const long long nt = mt2 * per;
        L->max_ftiles = nt < (1ll << 30) ? (int32_t)nt : 0;
        L->ftiles = take(sizeof(int4) * (size_t)L->max_ftiles);
        L->ready = take(4 * sizeof(int32_t) * (size_t)mt2);    // ready, consumed, staged, released
    }
    {   // gang-start counters of the 256-row kernel: one per tile of the largest of the four GEMMs
        const long long mt2 = Rpad / (2 * TILE_M), mts = L->Tpad / (2 * TILE_M);
        long long n_r = (I + 127) / 128 > (H + 255) / 256 ? (I + 127) / 128 : (H + 255) / 256;
        long long n_s = (Is + 127) / 128 > (H + 255) / 256 ? (Is + 127) / 128 : (H + 255) / 256;
        long long tiles = mt2 * n_r > mts * n_s ? mt2 * n_r : mts * n_s;
        if (L->max_ftiles > tiles) tiles = L->max_ftiles;       // the one-launch FFN's list (static hand-out)
        L->gang_bytes = sizeof(int32_t) * (size_t)tiles;
        L->gang = take(L->gang_bytes);
    }
    L->hs = take(Is > 0 ? 2 * (size_t)L->Tpad * Is : 0);
    L->ysh = take(Is > 0 ? 2 * (size_t)L->Tpad * H : 0);
    if (mx) {
        L->x8 = take((size_t)(T > 0 ? T : 1) * H);
        L->sx = take((size_t)(T > 0 ? T : 1) * ((H + 127) / 128 * 4));
        L->h8 = take((size_t)Rpad * I);
        L->sh = take((size_t)(Rpad / TILE_M) * ((I + 127) / 128) * 512);
    }
    L->total = off;
    return true;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static bool use_mx(const mok_config* cfg) { return cfg && cfg->precision == MOK_PRECISION_MXFP8; }
// MXFP8 GEMMs on CTA pairs (each CTA stages half of the weight tile): cta_group = 2 asks for them, 1 for single CTAs.
static bool mx_pairs(const mok_config* cfg) { return cfg && cfg->cta_group == 2; }

static int validate(const mok_args* a, WsLayout* L, size_t extra_ws) {
    if (!a) return MOK_ERR_NULL;
    if (a->config && (a->config->precision < 0 || a->config->precision > 1)) return MOK_ERR_SHAPE;
    if (a->config && (a->config->tile_sched < 0 || a->config->tile_sched > 2)) return MOK_ERR_SHAPE;
    const bool mx = use_mx(a->config);
    if (mx && a->config->impl != MOK_IMPL_TCGEN05) return MOK_ERR_SHAPE;
    const int ring = a->config ? a->config->h_ring_tiles : 0;
    if (ring < 0 || (ring > 0 && ring < H_RING_MIN_TILES)) return MOK_ERR_SHAPE;
    if (ring > 0 && mx) return MOK_ERR_UNSUPPORTED;
    if (!ws_layout(a->T, a->H, a->I, a->I_shared, a->E, a->k, L, mx, ring)) return MOK_ERR_SHAPE;
    if ((a->I_shared > 0) != (a->W_shared_gate_up != nullptr) || (a->I_shared > 0) != (a->W_shared_down != nullptr))
        return MOK_ERR_SHAPE;
    if (a->T == 0) return MOK_OK;
    if (!a->W_router) return MOK_ERR_NULL;
    if (mx) {
        if (!a->W_gate_up_codes || !a->W_gate_up_scales || !a->W_down_codes || !a->W_down_scales) return MOK_ERR_NULL;
        if (!aligned16(a->W_gate_up_codes) || !aligned16(a->W_gate_up_scales) || !aligned16(a->W_down_codes) ||
            !aligned16(a->W_down_scales))
            return MOK_ERR_ALIGN;
    } else if (!a->W_gate_up || !a->W_down) {
        return MOK_ERR_NULL;
    }
    if (!aligned16(a->W_router_split)) return MOK_ERR_ALIGN;
    if (!aligned16(a->W_router) || !aligned16(a->W_gate_up) || !aligned16(a->W_down) ||
        !aligned16(a->W_shared_gate_up) || !aligned16(a->W_shared_down))
        return MOK_ERR_ALIGN;
    if (!a->workspace || (reinterpret_cast<uintptr_t>(a->workspace) & 255u) || a->workspace_bytes < L->total + extra_ws)
        return MOK_ERR_WORKSPACE;
    if (a->config && (a->config->impl < 0 || a->config->impl > 2 || a->config->grid < 0 ||
                      a->config->router_impl < 0 || a->config->router_impl > 2 ||
                      a->config->gather_mode < 0 || a->config->gather_mode > 2 ||
                      a->config->cta_group < 0 || a->config->cta_group > 3 ||
                      a->config->host_chunks < 0 || a->config->host_chunks > MOK_MAX_HOST_CHUNKS ||
                      a->config->fused_ffn < 0 || a->config->fused_ffn > 3 || a->config->fused_window < -1 ||
                      a->config->gang_sync < 0 || a->config->gang_sync > 2 || a->config->serial_launches < 0 ||
                      a->config->serial_launches > 1 || a->config->h_ring_tiles < 0 || a->config->shared_overlap < 0 ||
                      a->config->shared_overlap > 2 || a->config->comm_ctas < 0))
        return MOK_ERR_SHAPE;
    return MOK_OK;
}

static bool use_simt(const mok_config* cfg) { return cfg && cfg->impl == MOK_IMPL_SIMT; }
static bool use_tn(const mok_config* cfg) { return cfg && cfg->impl == MOK_IMPL_TCGEN05_TN; }
static bool use_simt_router(const mok_config* cfg, int k) {
    if (k > 28) return true;   // the tensor-core router keeps k + 4 candidates in one warp's 32 lanes
    return cfg && (cfg->router_impl == 1 || (cfg->router_impl == 0 && cfg->impl == MOK_IMPL_SIMT));
}

// Projection + top-k in one kernel (router_fused.cu) whenever the shape allows it; router_impl = 2 keeps the
// three-kernel tensor-core path (split, GEMM, top-k), which also serves more than 160 experts.
static bool use_fused_router(const mok_config* cfg, int E, int k) {
    if (use_simt_router(cfg, k) || (cfg && cfg->router_impl == 2)) return false;
    return router_fused_ok(E, k);
}

// Whether the routed gate/up GEMM gathers its rows itself.  The fused path re-gathers the rows once per N tile
// through the load/store units; the separate kernel writes the expert-sorted copy once and the GEMM then uses
// plain TMA tile loads.  Measured on B200: fused wins at 6, 16 and 23 N tiles (ceil(I / 128)), loses at 112.
bool fused_gather(const mok_config* cfg, int I) {
    if (use_simt(cfg)) return false;
    if (use_tn(cfg)) return true;
    if (cfg && cfg->gather_mode == 1) return true;
    if (cfg && cfg->gather_mode == 2) return false;
    return (I + 127) / 128 <= 32;
}

// Rows of one tile of the padded row space: 256 when the GEMMs run on CTA pairs (cta_group::2), else 128.
// Measured on B200: pairs are 5-19 % faster per k-block than single 128-row tiles for GEMMs whose A operand comes
// through TMA, but slower for the fused-gather GEMM (its odd CTA has to announce its gathered rows in software) and
// they double the padding of every expert segment.  The 256-row tiles of ONE CTA (use_m2) get the same saving without
// either drawback, so pairs are only used on request (cta_group = 2).
int tile_rows(const mok_config* cfg, int I) {
    if (use_simt(cfg) || use_tn(cfg)) return TILE_M;
    if (cfg && cfg->cta_group == 2) return 2 * TILE_M;
    if (cfg && cfg->cta_group == 1) return TILE_M;
    (void)I;
    return TILE_M;   // default: 128-row padding; the 256-row-tile kernel works on it through the second tile table
}

// 256-row tiles with two accumulators in one CTA (gemm_tcgen05_m2.cu): used on the 128-padded row space through the
// second tile table.  cta_group = 3 forces it; by default it serves GEMMs whose K is long enough to amortise the
// accumulator hand-over between tiles.
static bool use_m2(const mok_config* cfg, int K, int tile_m, long long rows, int experts) {
    if (use_simt(cfg) || use_tn(cfg) || tile_m != TILE_M) return false;
    if (cfg && cfg->cta_group == 3) return true;
    if (cfg && cfg->cta_group != 0) return false;
    // With few rows per expert nearly every tile has one half only and the layer is bound by streaming the weights
    // once: there the 128-row kernel, whose four stages are all weight and activation bytes, is the faster one
    // (measured on the DeepSeek-like shape: 3.39 vs 3.62 ms at 2 rows per expert, 5.58 vs 5.31 ms at 128).
    return K >= M2_MIN_K && rows >= 96ll * experts;
}

// Whether synchronised tile starts (gemm_tcgen05_m2.cu, "gang") pay for a grouped GEMM whose experts own weight matrices
// of `w_bytes` bytes and `rows` rows in total: an expert's matrix is large against L2 (>= 12 MB: a few experts' tiles in
// flight fill it, so a tile only survives in L2 while its users run in step) and an expert has fewer than eight full
// row tiles (the half-empty last tile is what pulls CTAs apart).  Measured on B200, layer time with / without:
// DeepSeek-like -13 %, GPT-OSS-like -4 %; Qwen3-like (6 MB per expert) +2 %, Mixtral-like (eight equal row tiles per
// expert) +1.5 %.
static bool gang_pays(long long w_bytes, long long rows, int experts) {
    return w_bytes >= (12ll << 20) && rows < 8ll * 256 * experts;
}

// Routed gate/up + SwiGLU + down as ONE persistent launch (gemm_fused.cu).  Chosen by default for large expert
// matrices (both GEMMs' weights of an expert >= 12 MB, fewer than eight row tiles per expert: there it equals or beats
// the two launches: DeepSeek-like -1.6 %, GPT-OSS-like -4 to -13 %, variants alternating in one process); elsewhere the
// two launches are 1-2 % faster from a rested board and stay the default.
// fused_ffn = 1 / 2 force the two launches / the one launch; 3 = the one launch with the combine at its end.
static bool large_experts(int H, int I, long long rows, int experts) {
    return gang_pays(4ll * I * H, rows, experts) && gang_pays(2ll * H * I, rows, experts);
}
// ... with synchronised tile starts on the static stride where an expert has three or more row tiles on average (the
// DeepSeek-like layer: 23.7 against 29-31 ms with the dynamic draw), with the dynamic draw and no gangs below that (the
// GPT-OSS-like layer, two row tiles per expert and K = 2880: 3.20-3.24 against 3.41-3.48 ms under the power cap).
static bool fused_gang(const mok_config* cfg, int H, int I, long long rows, int experts) {
    const int mode = cfg ? cfg->gang_sync : 0;
    if (mode == 1) return false;
    if (mode == 2) return true;
    return large_experts(H, I, rows, experts) && rows >= 768ll * experts;
}
static bool use_fused_ffn(const mok_config* cfg, int H, int I, int tile_m, long long rows, int experts, int max_ftiles) {
    if (use_simt(cfg) || use_tn(cfg) || use_mx(cfg) || tile_m != TILE_M || max_ftiles <= 0) return false;
    if (cfg && (cfg->fused_ffn == 1 || cfg->cta_group == 1 || cfg->cta_group == 2)) return false;
    if (!fused_gather(cfg, I)) return false;
    if (cfg && (cfg->fused_ffn >= 2 || cfg->h_ring_tiles > 0 || cfg->comm_ctas > 0)) return true;
    if (cfg && cfg->tile_sched == 1) return false;          // (tile stealing belongs to the two-launch path)
    // (at least two row tiles per expert on average: with single tiles there is nothing to start together, and the
    //  weight-streaming regime of small batches is served better by the two launches: 4.64 vs 4.80 ms at 128 rows)
    return use_m2(cfg, H, tile_m, rows, experts) && use_m2(cfg, I, tile_m, rows, experts) &&
           rows >= 512ll * experts && large_experts(H, I, rows, experts) && !(cfg && cfg->gang_sync == 1);
}

// Synchronised starts of the row tiles that share a weight tile (see gemm_tcgen05_m2.cu) for one launch of the 256-row
// kernel: where they pay (or are forced), the gang counters are cleared and handed to the kernel.  Not with stolen
// tiles, not for the K-range products of the backward pass, and off with gang_sync = 1.
int gang_prepare(GemmArgs& g, bool swiglu, const mok_config* cfg, const WsLayout& L, char* ws, cudaStream_t s) {
    const long long w_bytes = 2ll * (swiglu ? 2 : 1) * g.N * g.K;
    const long long rows_all = g.dense_rows > 0 ? g.dense_rows : g.total_rows;
    const bool pays = gang_pays(w_bytes, rows_all, g.dense_rows > 0 ? 1 : g.E);
    const int mode = cfg ? cfg->gang_sync : 0;
    g.gang = nullptr;
    if (L.gang_bytes > 0 && g.kgroup_rows == 0 && g.tile_sched != 1 && (mode == 2 || (mode == 0 && pays))) {
        const long long rows = g.dense_rows > 0 ? g.dense_rows : g.rows_pad;
        const long long n_nt = swiglu ? (g.N + 127) / 128 : (g.N + 255) / 256;
        const size_t bytes = sizeof(int32_t) * (size_t)((rows + 255) / 256 * n_nt);
        if (bytes <= L.gang_bytes) {        // (a GEMM with more tiles than the region was sized for runs without)
            cudaError_t eg = cudaMemsetAsync(ws + L.gang, 0, bytes, s);
            if (eg != cudaSuccess) return cuda_fail(eg);
            g.gang = reinterpret_cast<int32_t*>(ws + L.gang);
        }
    }
    return MOK_OK;
}

bool fused_ffn_choice(const mok_config* cfg, int H, int I, int tile_m, long long rows, int experts, int max_ftiles, bool* sync) {
    if (sync) *sync = fused_gang(cfg, H, I, rows, experts);
    return use_fused_ffn(cfg, H, I, tile_m, rows, experts, max_ftiles);
}

int run_gemm(GemmArgs g, bool swiglu, const mok_config* cfg, const WsLayout& L, char* ws, cudaStream_t s) {
    const int epi = swiglu ? EPI_SWIGLU : EPI_BF16, grid = cfg ? cfg->grid : 0;
    if (use_m2(cfg, g.K, g.tile_m, g.dense_rows > 0 ? g.dense_rows : g.total_rows, g.dense_rows > 0 ? 1 : g.E)) {
        WsHeader* hdr = reinterpret_cast<WsHeader*>(ws + L.header);
        const int rcg = gang_prepare(g, swiglu, cfg, L, ws, s);
        if (rcg) return rcg;
        g.n_mtiles = &hdr->n_mtiles2;
        g.mt_start = reinterpret_cast<const int32_t*>(ws + L.mt_start2);
        g.tile_expert = reinterpret_cast<const int32_t*>(ws + L.tile_expert2);
        cudaError_t e2 = launch_gemm_m2(g, epi, grid, s);
        return e2 == cudaSuccess ? MOK_OK : cuda_fail(e2);
    }
    cudaError_t e = use_simt(cfg) ? launch_gemm_simt(g, swiglu, s)
                    : use_tn(cfg) ? launch_gemm_tn(g, epi, grid, s) : launch_gemm_tc(g, epi, grid, s);
    return e == cudaSuccess ? MOK_OK : cuda_fail(e);
}

static int route_stage(const mok_args* a, const WsLayout& L, char* ws, const __nv_bfloat16* x, cudaStream_t s) {
    int32_t* idx = reinterpret_cast<int32_t*>(ws + L.idx);
    float* w = reinterpret_cast<float*>(ws + L.w);
    cudaError_t e;
    if (use_simt_router(a->config, a->k))
        e = launch_router_simt(x, a->W_router, a->router_bias, a->T, a->H, a->E, a->k, idx, w, s);
    else
        e = launch_router_tc(x, a->W_router, a->router_bias, a->T, a->H, a->E, a->k, L, ws,
                             reinterpret_cast<WsHeader*>(ws + L.header), a->config ? a->config->grid : 0,
                             tile_rows(a->config, a->I > 0 ? a->I : 8),
                             use_tn(a->config) ? 2 : use_m2(a->config, a->H, tile_rows(a->config, a->I > 0 ? a->I : 8), a->T, 1) ? 3 : 0,
                             use_fused_router(a->config, a->E, a->k), idx, w, s,
                             reinterpret_cast<const __nv_bfloat16*>(a->W_router_split));
    if (e != cudaSuccess) return cuda_fail(e);
    if (a->topk_idx) {
        e = cudaMemcpyAsync(a->topk_idx, idx, sizeof(int32_t) * (size_t)L.R, cudaMemcpyDeviceToDevice, s);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    if (a->topk_w) {
        e = cudaMemcpyAsync(a->topk_w, w, sizeof(float) * (size_t)L.R, cudaMemcpyDeviceToDevice, s);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    return MOK_OK;
}

// A second, library-owned stream per device for the shared expert (see forward_device): forked from and joined to the
// caller's stream with two events, so the caller sees one stream's worth of ordering (and a stream capture of the call
// captures both).
struct SidePipe {
    cudaStream_t stream = nullptr;
    cudaEvent_t fork = nullptr, join = nullptr;
    bool ready = false;
};
static SidePipe g_side[64];
static int side_pipe(SidePipe** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= 64) return MOK_ERR_UNSUPPORTED;
    SidePipe& p = g_side[dev];
    if (!p.ready) {
        if ((e = cudaStreamCreateWithFlags(&p.stream, cudaStreamNonBlocking)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaEventCreateWithFlags(&p.fork, cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaEventCreateWithFlags(&p.join, cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e);
        p.ready = true;
    }
    *out = &p;
    return MOK_OK;
}
constexpr int SIDE_CTAS = 16;           // persistent CTAs of the shared expert's GEMMs while they run beside the routed ones

// Shared expert beside the routed experts (Section 3.4 "Shared Expert": it does not depend on the dispatch, so it can
// fill time the routed path leaves idle).  On one GPU that pays for SMALL layers only, whose kernels are a few tiles
// each and bound by launch and pipeline-fill latency: there the shared expert's two GEMMs run while router, schedule
// and routed GEMMs go through their own latencies (tiny workload: 47 against 60 us per layer).  It does not pay where
// the routed GEMMs stream expert weights from DRAM (few rows per expert, large experts): a CTA pulls about 40 GB/s, so
// that phase needs every SM to reach the DRAM bandwidth, and each SM given to the shared expert is lost to it
// (DeepSeek-like layer at 64 / 4096 tokens: 3.59 against 3.40 ms, 6.6 against 4.9 ms).  Nor with many rows per expert,
// where both are bound by the tensor cores or the power cap and a split of the SMs conserves the work.
static bool shared_beside_routed(const mok_config* cfg, int H, int I, int I_shared, long long rows, int experts) {
    if (I_shared <= 0) return false;
    const int mode = cfg ? cfg->shared_overlap : 0;
    if (mode == 1) return false;
    if (cfg && (cfg->debug == MOK_DEBUG_STARVE || cfg->debug == MOK_DEBUG_NO_ARRIVALS || cfg->fused_ffn == 3)) return false;
    if (mode == 2) return true;
    return rows <= 160ll * experts && 6ll * experts * H * I <= (64ll << 20);
}

// The shared expert's two GEMMs (every token in natural order, no gather) on stream ss with the knobs cs.
static int shared_expert_gemms(const mok_args* a, const WsLayout& L, char* ws, WsHeader* hdr, const __nv_bfloat16* x,
                               int tile_m, bool dbg, const mok_config* cs, cudaStream_t ss, ProfileMarks* marks) {
    if (a->I_shared <= 0) {
        if (marks) { marks->close(MOK_STAGE_SHARED_GEMM1); marks->close(MOK_STAGE_SHARED_GEMM2); }
        return MOK_OK;
    }
    GemmArgs gs;
    memset(&gs, 0, sizeof(gs));
    gs.header = hdr;
    gs.n_mtiles = &hdr->n_mtiles;          // (dense mode derives its tiles from dense_rows: the schedule's tables are not read)
    gs.tile_expert = reinterpret_cast<const int32_t*>(ws + L.tile_expert);
    gs.mt_start = reinterpret_cast<const int32_t*>(ws + L.mt_start);
    gs.max_mt = L.max_mt;
    gs.tile_m = tile_m;
    gs.pad_offsets = reinterpret_cast<const int32_t*>(ws + L.pad_offsets);
    gs.counts = reinterpret_cast<const int32_t*>(ws + L.counts);
    gs.dbg_slot = dbg ? 3 : -1;
    gs.A = x;
    gs.B = reinterpret_cast<const __nv_bfloat16*>(a->W_shared_gate_up);
    gs.C = ws + L.hs;
    gs.K = a->H; gs.N = a->I_shared; gs.ldc = a->I_shared; gs.E = 1; gs.rows_pad = L.Tpad; gs.a_rows = a->T;
    gs.dense_rows = a->T;
    int rc = run_gemm(gs, true, cs, L, ws, ss);
    if (rc) return rc;
    if (marks) marks->close(MOK_STAGE_SHARED_GEMM1);
    gs.A = reinterpret_cast<const __nv_bfloat16*>(ws + L.hs);
    gs.B = reinterpret_cast<const __nv_bfloat16*>(a->W_shared_down);
    gs.C = ws + L.ysh;
    gs.K = a->I_shared; gs.N = a->H; gs.ldc = a->H; gs.a_rows = L.Tpad;
    if ((rc = run_gemm(gs, false, cs, L, ws, ss))) return rc;
    if (marks) marks->close(MOK_STAGE_SHARED_GEMM2);
    return MOK_OK;
}

// The whole layer on device pointers.  x / out may differ from a->x / a->out (host-buffer variant).
static int forward_device(const mok_args* a, const WsLayout& L, const __nv_bfloat16* x, __nv_bfloat16* out,
                          bool reset_header = true) {
    cudaStream_t s = reinterpret_cast<cudaStream_t>(a->stream);
    char* ws = reinterpret_cast<char*>(a->workspace);
    WsHeader* hdr = reinterpret_cast<WsHeader*>(ws + L.header);
    // (later macrobatches of one call keep the header: its status word is sticky, the tile counts are rewritten anyway)
    cudaError_t e = reset_header ? cudaMemsetAsync(hdr, 0, sizeof(WsHeader), s)
                                 : cudaMemsetAsync(&hdr->n_flag, 0, sizeof(hdr->n_flag), s);
    if (e != cudaSuccess) return cuda_fail(e);
    // a private copy of the knobs: the grid of the routed kernels shrinks while the shared expert runs beside them
    mok_config cfg_main;
    if (a->config) cfg_main = *a->config; else memset(&cfg_main, 0, sizeof(cfg_main));
    mok_args a_main = *a;
    a_main.config = &cfg_main;
    a = &a_main;
    g_pdl = !cfg_main.serial_launches;
    ProfileMarks marks = profile_slot(a->config, s);
#define MOK_MARK(i) marks.close((i) - 1)
    marks.open();
    int rc = MOK_OK;
    const int tile_m = use_mx(a->config) ? TILE_M : tile_rows(a->config, a->I);
    SidePipe* side = nullptr;
    mok_config cfg_side = cfg_main;
    if (shared_beside_routed(&cfg_main, a->H, a->I, a->I_shared, L.R, a->E)) {
        int dev = 0, sms = 0;
        if ((e = current_device(&dev)) != cudaSuccess || (e = device_sm_count(dev, &sms)) != cudaSuccess) return cuda_fail(e);
        if (sms >= 4 * SIDE_CTAS) {
            if ((rc = side_pipe(&side))) return rc;
            cfg_side.grid = cfg_main.grid > 0 && cfg_main.grid < SIDE_CTAS ? cfg_main.grid : SIDE_CTAS;
            cfg_side.gang_sync = 1;                                 // (the gang counters belong to the routed kernels)
            // The persistent kernels of the caller's stream leave the side kernels their SMs: every GEMM CTA takes a
            // whole SM, and with programmatic launches the routed GEMM's CTAs become resident (and wait) while router
            // and schedule still run -- a full grid of them would keep the side kernels off the GPU until it is done.
            if (cfg_main.grid == 0) cfg_main.grid = sms - SIDE_CTAS;
            if ((e = cudaEventRecord(side->fork, s)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaStreamWaitEvent(side->stream, side->fork, 0)) != cudaSuccess) return cuda_fail(e);
            // its two GEMMs need x and the weights only: enqueued first, so that they are on the GPU first
            if ((rc = shared_expert_gemms(a, L, ws, hdr, x, tile_m, cfg_main.debug == 1, &cfg_side, side->stream, nullptr)))
                return rc;
            if ((e = cudaEventRecord(side->join, side->stream)) != cudaSuccess) return cuda_fail(e);
        }
    }
    rc = route_stage(a, L, ws, x, s);
    if (rc) return rc;
    MOK_MARK(MOK_STAGE_ROUTER + 1);
    const int pad_m = use_tn(a->config) ? 16 : tile_m;   // tokens on the MMA's N side need 16-row granularity only
    e = launch_schedule(reinterpret_cast<const int32_t*>(ws + L.idx), a->T, a->E, a->k, tile_m, pad_m, L, ws,
                        a->counts, a->offsets, a->perm, a->inv_perm, s);
    if (e != cudaSuccess) return cuda_fail(e);
    MOK_MARK(MOK_STAGE_SCHEDULE + 1);
    const bool mx = use_mx(a->config);
    const bool simt = !mx && !fused_gather(a->config, a->I);
    if (L.h_ring > 0 && (simt || mx)) return MOK_ERR_UNSUPPORTED;   // (that layout has no room for a copy of x)
    if (simt) {   // materialise the expert-sorted copy of x
        e = launch_gather(x, a->H, a->k, tile_m, L, ws, s);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    if (mx) {     // quantise the token rows once; the gate/up GEMM pulls codes and scales of the rows it needs
        e = launch_mx_quantize_rows(x, a->T, a->H, reinterpret_cast<uint8_t*>(ws + L.x8),
                                    reinterpret_cast<uint8_t*>(ws + L.sx), s);
        if (e != cudaSuccess) return cuda_fail(e);
        // scale atoms of the gated activation: blocks past I keep 127 (= 1.0)
        e = cudaMemsetAsync(ws + L.sh, 127, (size_t)(L.Rpad / TILE_M) * ((a->I + 127) / 128) * 512, s);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    MOK_MARK(MOK_STAGE_GATHER + 1);

    GemmArgs g;
    memset(&g, 0, sizeof(g));
    g.header = hdr;
    g.n_mtiles = &hdr->n_mtiles;
    g.tile_expert = reinterpret_cast<const int32_t*>(ws + L.tile_expert);
    g.mt_start = reinterpret_cast<const int32_t*>(ws + L.mt_start);
    g.max_mt = L.max_mt;
    g.tile_m = tile_m;
    g.pad_offsets = reinterpret_cast<const int32_t*>(ws + L.pad_offsets);
    g.counts = reinterpret_cast<const int32_t*>(ws + L.counts);
    const bool dbg = a->config && a->config->debug == 1;
    g.dbg_slot = dbg ? 1 : -1;
    if (a->config && (a->config->debug == MOK_DEBUG_STARVE || a->config->debug == MOK_DEBUG_NO_ARRIVALS)) {
        // test hooks (see mok.h): the gate/up GEMM's producer stays silent, or the one-launch kernel's completion
        // counters get no arrivals; every wait gives up after 2 ms
        const uint32_t limit_us = 2000;
        e = cudaMemcpyAsync(&hdr->wait_limit_us, &limit_us, sizeof(limit_us), cudaMemcpyHostToDevice, s);
        if (e != cudaSuccess) return cuda_fail(e);
        g.starve = a->config->debug == MOK_DEBUG_STARVE ? 1 : 2;
    }
    bool combine_in_launch = false;
    if (mx) {
        // routed experts on MXFP8 operands (Section 3.4): h = Q(silu(Q(x) Wg_q^T) * (Q(x) Wu_q^T));  y = h Wd_q^T
        const int grid = a->config->grid;
        if (mx_pairs(a->config)) {   // CTA pairs on the 256-row tile table (over the same 128-row-padded row space)
            g.tile_m = 2 * TILE_M;
            g.n_mtiles = &hdr->n_mtiles2;
            g.mt_start = reinterpret_cast<const int32_t*>(ws + L.mt_start2);
            g.tile_expert = reinterpret_cast<const int32_t*>(ws + L.tile_expert2);
        }
        g.A = reinterpret_cast<const __nv_bfloat16*>(ws + L.x8);
        g.a_rows = a->T;
        g.row_token = reinterpret_cast<const int32_t*>(ws + L.row_token);
        g.sfa = reinterpret_cast<const uint8_t*>(ws + L.sx);
        g.sfa_stride = (a->H + 127) / 128 * 4;
        g.B = reinterpret_cast<const __nv_bfloat16*>(a->W_gate_up_codes);
        g.sfb = reinterpret_cast<const uint8_t*>(a->W_gate_up_scales);
        g.C = ws + L.h8;
        g.sfc = reinterpret_cast<uint8_t*>(ws + L.sh);
        g.K = a->H; g.N = a->I; g.ldc = a->I; g.E = a->E; g.rows_pad = L.Rpad; g.dense_rows = 0;
        g.total_rows = L.R;
        e = launch_gemm_mx(g, EPI_SWIGLU, grid, s);
        if (e != cudaSuccess) return cuda_fail(e);
        MOK_MARK(MOK_STAGE_GEMM1 + 1);
        g.row_token = nullptr;
        g.starve = 0;
        g.dbg_slot = dbg ? 2 : -1;
        g.A = reinterpret_cast<const __nv_bfloat16*>(ws + L.h8);
        g.a_rows = L.Rpad;
        g.sfa = reinterpret_cast<const uint8_t*>(ws + L.sh);
        g.B = reinterpret_cast<const __nv_bfloat16*>(a->W_down_codes);
        g.sfb = reinterpret_cast<const uint8_t*>(a->W_down_scales);
        g.C = ws + L.y;
        g.sfc = nullptr;
        g.K = a->I; g.N = a->H; g.ldc = a->H;
        e = launch_gemm_mx(g, EPI_BF16, grid, s);
        if (e != cudaSuccess) return cuda_fail(e);
        g.sfa = g.sfb = nullptr;
        g.tile_m = tile_m;
        g.n_mtiles = &hdr->n_mtiles;
        g.mt_start = reinterpret_cast<const int32_t*>(ws + L.mt_start);
        g.tile_expert = reinterpret_cast<const int32_t*>(ws + L.tile_expert);
    } else {
        // routed experts: h = silu(Xg Wg^T) * (Xg Wu^T);  y = h Wd^T
        if (simt) {
            g.A = reinterpret_cast<const __nv_bfloat16*>(ws + L.xg);
            g.a_rows = L.Rpad;
        } else {
            g.A = x;
            g.a_rows = a->T;
            g.row_token = reinterpret_cast<const int32_t*>(ws + L.row_token);
            g.counts = reinterpret_cast<const int32_t*>(ws + L.counts);
        }
        g.B = reinterpret_cast<const __nv_bfloat16*>(a->W_gate_up);
        g.C = ws + L.h;
        g.K = a->H; g.N = a->I; g.ldc = a->I; g.E = a->E; g.rows_pad = L.Rpad; g.dense_rows = 0;
        g.total_rows = L.R;
        g.tile_sched = a->config ? a->config->tile_sched : 0;
        const bool fused = !simt && use_fused_ffn(a->config, a->H, a->I, tile_m, L.R, a->E, L.max_ftiles);
        if (L.h_ring > 0 && !fused) return MOK_ERR_UNSUPPORTED;     // the ring exists in the one-launch kernel only
        if (!fused && g.starve == 2) g.starve = 0;                  // (that hook only exists in the one-launch kernel)
        combine_in_launch = fused && a->config && a->config->fused_ffn == 3;
        // (the shared expert's output is an input of that launch: it then runs first)
        if (combine_in_launch && (rc = shared_expert_gemms(a, L, ws, hdr, x, tile_m, dbg, a->config, s, &marks))) return rc;
        // its hand-out: synchronised starts need the static stride (a CTA that draws ahead could hold two tiles of a gang)
        const bool fused_sync = fused_gang(a->config, a->H, a->I, L.R, a->E);
        const int sched = a->config ? a->config->tile_sched : 0;
        // (with a ring of h the window is short; the static stride keeps a row group's tiles closest together: measured
        //  1.29 against 1.56 ms on the Qwen3-like layer with 72 slots)
        const bool fused_dynamic = sched == 1 || (sched == 0 && !fused_sync && L.h_ring == 0);
        // communication CTAs exist in the one-launch kernel; their staging slots take the place of the gathered copy of x
        const int comm_ctas = a->config ? a->config->comm_ctas : 0;
        if (comm_ctas > 0 && (!fused || L.h_ring > 0 || (long long)L.Rpad < (long long)FFN_COMM_SLOTS * 2 * TILE_M))
            return MOK_ERR_UNSUPPORTED;
        if (fused) {
            e = launch_fused_ffn(x, a->T, a->H, a->I, a->E, reinterpret_cast<const __nv_bfloat16*>(a->W_gate_up),
                                 reinterpret_cast<const __nv_bfloat16*>(a->W_down), L, ws, a->config ? a->config->grid : 0,
                                 a->config ? a->config->fused_window : 0, fused_dynamic, fused_sync, dbg, g.starve, s,
                                 combine_in_launch ? out : nullptr, a->k, a->I_shared > 0, L.h_ring, nullptr, 0, nullptr,
                                 comm_ctas, comm_ctas > 0 ? ws + L.xg : nullptr);
            if (e != cudaSuccess) return cuda_fail(e);
        } else if ((rc = run_gemm(g, true, a->config, L, ws, s))) return rc;
        g.row_token = nullptr;
        g.starve = 0;
        g.a_rows = L.Rpad;
        g.dbg_slot = dbg ? 2 : -1;
        MOK_MARK(MOK_STAGE_GEMM1 + 1);
        g.A = reinterpret_cast<const __nv_bfloat16*>(ws + L.h);
        g.B = reinterpret_cast<const __nv_bfloat16*>(a->W_down);
        g.C = ws + L.y;
        g.K = a->I; g.N = a->H; g.ldc = a->H;
        if (!fused && (rc = run_gemm(g, false, a->config, L, ws, s))) return rc;
        g.tile_sched = 0;
    }
    MOK_MARK(MOK_STAGE_GEMM2 + 1);
    if (!combine_in_launch) {
        if (side) {
            MOK_MARK(MOK_STAGE_SHARED_GEMM1 + 1);
            MOK_MARK(MOK_STAGE_SHARED_GEMM2 + 1);
            if ((e = cudaStreamWaitEvent(s, side->join, 0)) != cudaSuccess) return cuda_fail(e);
        } else if ((rc = shared_expert_gemms(a, L, ws, hdr, x, tile_m, dbg, a->config, s, &marks))) return rc;
        e = launch_combine(L, ws, a->T, a->H, a->k, a->I_shared > 0, out, s);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    MOK_MARK(MOK_STAGE_COMBINE + 1);
#undef MOK_MARK
    return MOK_OK;
}

// Library-owned workspace of mok_moe_forward, one per device, grown on demand.
struct OwnedWs { void* ptr; size_t bytes; };
static OwnedWs g_owned[64];

}  // namespace mok

using namespace mok;

extern "C" {

size_t mok_mx_workspace_bytes(int T, int H, int I, int I_shared, int E, int k) {
    WsLayout L;
    return ws_layout(T, H, I, I_shared, E, k, &L, true) ? L.total : 0;
}

size_t mok_mx_scale_bytes(int groups, int rows, int K) {
    if (groups < 1 || rows < 1 || K < 32 || (K % 32)) return 0;
    return (size_t)groups * ((rows + 127) / 128) * ((K + 127) / 128) * 512;
}

int mok_mx_quantize_weights(const void* W, int groups, int rows, int K, void* codes, void* scales, void* stream) {
    if (!W || !codes || !scales) return MOK_ERR_NULL;
    if (mok_mx_scale_bytes(groups, rows, K) == 0) return MOK_ERR_SHAPE;
    if (!aligned16(W) || !aligned16(codes) || !aligned16(scales)) return MOK_ERR_ALIGN;
    cudaError_t e = launch_mx_quantize_atoms(reinterpret_cast<const __nv_bfloat16*>(W), groups, rows, K,
                                             reinterpret_cast<uint8_t*>(codes), reinterpret_cast<uint8_t*>(scales),
                                             reinterpret_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? MOK_OK : cuda_fail(e);
}

int mok_mx_quantize_rows(const void* x, int rows, int K, void* codes, void* scales, void* stream) {
    if (!x || !codes || !scales) return MOK_ERR_NULL;
    if (rows < 0 || K < 32 || (K % 32)) return MOK_ERR_SHAPE;
    if (rows == 0) return MOK_OK;
    if (!aligned16(x) || !aligned16(codes) || !aligned16(scales)) return MOK_ERR_ALIGN;
    cudaError_t e = launch_mx_quantize_rows(reinterpret_cast<const __nv_bfloat16*>(x), rows, K,
                                            reinterpret_cast<uint8_t*>(codes), reinterpret_cast<uint8_t*>(scales),
                                            reinterpret_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? MOK_OK : cuda_fail(e);
}

size_t mok_workspace_bytes(int T, int H, int I, int I_shared, int E, int k) {
    WsLayout L;
    return ws_layout(T, H, I, I_shared, E, k, &L) ? L.total : 0;
}

size_t mok_workspace_bytes_ring(int T, int H, int I, int I_shared, int E, int k, int h_ring_tiles) {
    WsLayout L;
    if (h_ring_tiles < H_RING_MIN_TILES) return 0;
    return ws_layout(T, H, I, I_shared, E, k, &L, false, h_ring_tiles) ? L.total : 0;
}

size_t mok_router_prepared_bytes(int E, int H) {
    if (E <= 0 || E > MAX_E || H <= 0 || (H % 8)) return 0;
    return align_up(2 * (size_t)3 * ((E + 31) / 32 * 32) * H, 256);      // either layout fits: 3 * E rows rounded up
}

int mok_router_prepare(const float* W_router, int E, int H, int k, const mok_config* config, void* out, size_t out_bytes,
                       void* stream) {
    if (!W_router || !out) return MOK_ERR_NULL;
    const size_t need = mok_router_prepared_bytes(E, H);
    if (need == 0 || k < 1 || k > E || k > MAX_K) return MOK_ERR_SHAPE;
    if (use_simt_router(config, k)) return MOK_ERR_UNSUPPORTED;        // the fp32-FMA router reads W_router itself
    if (!aligned16(W_router) || !aligned16(out)) return MOK_ERR_ALIGN;
    if (out_bytes < need) return MOK_ERR_WORKSPACE;
    WsLayout L;
    memset(&L, 0, sizeof(L));
    cudaError_t e = launch_router_tc(nullptr, W_router, nullptr, 0, H, E, k, L, nullptr, nullptr, 0, TILE_M, 0,
                                     use_fused_router(config, E, k), nullptr, nullptr,
                                     reinterpret_cast<cudaStream_t>(stream), reinterpret_cast<const __nv_bfloat16*>(out), true);
    return e == cudaSuccess ? MOK_OK : cuda_fail(e);
}

int mok_moe_forward_ex(const mok_args* a) {
    WsLayout L;
    if (!a) return MOK_ERR_NULL;
    const int mb = a->config ? a->config->macrobatch_tokens : 0;
    if (mb < 0) return MOK_ERR_SHAPE;
    if (mb > 0 && a->T > mb) {
        // Fixed-size macrobatches (Section 3.3): the tokens pass through a workspace sized for `mb` tokens, one macrobatch
        // after the other on the same stream.  A token's output depends only on its own row of x, so the bits equal
        // those of the single pass.  The schedule tables describe one macrobatch each, so only the per-token stage
        // outputs can be returned.
        if (a->counts || a->offsets || a->perm || a->inv_perm) return MOK_ERR_UNSUPPORTED;
        mok_args ac = *a;
        ac.T = mb;
        int rc = validate(&ac, &L, 0);
        if (rc) return rc;
        if (!a->x || !a->out) return MOK_ERR_NULL;
        if (!aligned16(a->x) || !aligned16(a->out)) return MOK_ERR_ALIGN;
        const __nv_bfloat16* x = reinterpret_cast<const __nv_bfloat16*>(a->x);
        __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(a->out);
        for (int t0 = 0; t0 < a->T; t0 += mb) {
            ac.T = a->T - t0 < mb ? a->T - t0 : mb;
            if (!ws_layout(ac.T, a->H, a->I, a->I_shared, a->E, a->k, &L, use_mx(a->config), a->config->h_ring_tiles))
                return MOK_ERR_SHAPE;
            ac.topk_idx = a->topk_idx ? a->topk_idx + (size_t)t0 * a->k : nullptr;
            ac.topk_w = a->topk_w ? a->topk_w + (size_t)t0 * a->k : nullptr;
            rc = forward_device(&ac, L, x + (size_t)t0 * a->H, out + (size_t)t0 * a->H, t0 == 0);
            if (rc) return rc;
        }
        return MOK_OK;
    }
    int rc = validate(a, &L, 0);
    if (rc || a->T == 0) return rc;
    if (!a->x || !a->out) return MOK_ERR_NULL;
    if (!aligned16(a->x) || !aligned16(a->out)) return MOK_ERR_ALIGN;
    return forward_device(a, L, reinterpret_cast<const __nv_bfloat16*>(a->x), reinterpret_cast<__nv_bfloat16*>(a->out));
}

// Copy streams and events of mok_moe_forward_host, created once per device.
struct HostPipe {
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t start = nullptr, out_done = nullptr, in_done[MOK_MAX_HOST_CHUNKS] = {}, fwd_done[MOK_MAX_HOST_CHUNKS] = {};
    // asynchronous submissions: two staging slots used in turn; slot_free[i] fires when slot i's result has left the device
    cudaEvent_t a_in[2] = {}, a_fwd[2] = {}, slot_free[2] = {};
    bool slot_used[2] = {false, false};
    unsigned long long n_async = 0;
    unsigned long long n_since_wait = 0;     // submissions since the last mok_host_wait
    bool ready = false;
};
static HostPipe g_pipe[64];

static int host_pipe(HostPipe** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= 64) return MOK_ERR_UNSUPPORTED;
    HostPipe& p = g_pipe[dev];
    if (!p.ready) {
        if ((e = cudaStreamCreateWithFlags(&p.s_in, cudaStreamNonBlocking)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaStreamCreateWithFlags(&p.s_out, cudaStreamNonBlocking)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaEventCreateWithFlags(&p.out_done, cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e);
        for (int c = 0; c < MOK_MAX_HOST_CHUNKS; ++c) {
            if ((e = cudaEventCreateWithFlags(&p.in_done[c], cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaEventCreateWithFlags(&p.fwd_done[c], cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e);
        }
        for (int c = 0; c < 2; ++c) {
            if ((e = cudaEventCreateWithFlags(&p.a_in[c], cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaEventCreateWithFlags(&p.a_fwd[c], cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaEventCreateWithFlags(&p.slot_free[c], cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e);
        }
        p.ready = true;
    }
    *out = &p;
    return MOK_OK;
}

// Every token's output depends only on its own row of x, so the batch can be cut into token chunks: the upload of
// chunk c+1 and the download of chunk c-1 run on two copy streams while chunk c computes.  The bits of the result
// do not depend on the number of chunks.
int mok_moe_forward_host(const mok_args* a, const void* x_host, void* out_host) {
    WsLayout L;
    if (!a) return MOK_ERR_NULL;
    const size_t act = 2 * (size_t)(a->T > 0 ? a->T : 0) * (size_t)(a->H > 0 ? a->H : 0);
    const size_t act_al = align_up(act, 256);
    int rc = validate(a, &L, 2 * act_al);
    if (rc || a->T == 0) return rc;
    if (!x_host || !out_host) return MOK_ERR_NULL;
    int chunks = a->config ? a->config->host_chunks : 0;
    if (chunks < 0 || chunks > MOK_MAX_HOST_CHUNKS) return MOK_ERR_SHAPE;
    const bool stages = a->topk_idx || a->topk_w || a->counts || a->offsets || a->perm || a->inv_perm;
    if (chunks == 0) chunks = a->T >= 8192 ? 4 : (a->T >= 2048 ? 2 : 1);
    if (stages) chunks = 1;                    // stage outputs describe one schedule over the whole batch
    // Chunk boundaries: with three or more chunks the first and the last get half the weight of the inner ones, so
    // that the upload nobody can hide (first chunk) and the download nobody can hide (last chunk) are short.
    int bound[MOK_MAX_HOST_CHUNKS + 1];
    {
        const int units = (chunks >= 3) ? 2 * chunks - 2 : chunks;
        int acc_units = 0, n = 0;
        bound[0] = 0;
        for (int c = 0; c < chunks; ++c) {
            acc_units += (chunks >= 3 && c > 0 && c < chunks - 1) ? 2 : 1;
            int end = (int)(((long long)a->T * acc_units / units + 2 * TILE_M - 1) / (2 * TILE_M) * (2 * TILE_M));
            if (end > a->T || c == chunks - 1) end = a->T;
            if (end > bound[n]) bound[++n] = end;
        }
        chunks = n;
    }
    HostPipe* p = nullptr;
    if ((rc = host_pipe(&p))) return rc;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(a->stream);
    char* ws = reinterpret_cast<char*>(a->workspace);
    __nv_bfloat16* xd = reinterpret_cast<__nv_bfloat16*>(ws + L.total);
    __nv_bfloat16* od = reinterpret_cast<__nv_bfloat16*>(ws + L.total + act_al);
    const char* xh = reinterpret_cast<const char*>(x_host);
    char* oh = reinterpret_cast<char*>(out_host);
    cudaError_t e;
    // the copy streams start after whatever already sits in the caller's stream (it may still use the staging area)
    if ((e = cudaEventRecord(p->start, s)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaStreamWaitEvent(p->s_in, p->start, 0)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaStreamWaitEvent(p->s_out, p->start, 0)) != cudaSuccess) return cuda_fail(e);
    for (int c = 0; c < chunks; ++c) {
        const int t0 = bound[c], tc = bound[c + 1] - bound[c];
        const size_t off = 2 * (size_t)t0 * a->H, bytes = 2 * (size_t)tc * a->H;
        if ((e = cudaMemcpyAsync(reinterpret_cast<char*>(xd) + off, xh + off, bytes, cudaMemcpyHostToDevice, p->s_in)) != cudaSuccess)
            return cuda_fail(e);
        if ((e = cudaEventRecord(p->in_done[c], p->s_in)) != cudaSuccess) return cuda_fail(e);
    }
    for (int c = 0; c < chunks; ++c) {
        const int t0 = bound[c], tc = bound[c + 1] - bound[c];
        const size_t off = 2 * (size_t)t0 * a->H, bytes = 2 * (size_t)tc * a->H;
        mok_args ac = *a;
        ac.T = tc;
        WsLayout Lc;
        if (!ws_layout(tc, a->H, a->I, a->I_shared, a->E, a->k, &Lc, use_mx(a->config), a->config ? a->config->h_ring_tiles : 0))
            return MOK_ERR_SHAPE;
        if ((e = cudaStreamWaitEvent(s, p->in_done[c], 0)) != cudaSuccess) return cuda_fail(e);
        // only the first chunk clears the header: a device-side failure of any chunk stays in the status word
        rc = forward_device(&ac, Lc, xd + (size_t)t0 * a->H, od + (size_t)t0 * a->H, c == 0);
        if (rc) return rc;
        if ((e = cudaEventRecord(p->fwd_done[c], s)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaStreamWaitEvent(p->s_out, p->fwd_done[c], 0)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaMemcpyAsync(oh + off, reinterpret_cast<char*>(od) + off, bytes, cudaMemcpyDeviceToHost, p->s_out)) != cudaSuccess)
            return cuda_fail(e);
    }
    if ((e = cudaEventRecord(p->out_done, p->s_out)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaStreamWaitEvent(s, p->out_done, 0)) != cudaSuccess) return cuda_fail(e);
    e = cudaStreamSynchronize(s);
    return e == cudaSuccess ? MOK_OK : cuda_fail(e);
}

// Submission without waiting: upload on the input copy stream, layer on the caller's stream, download on the output copy
// stream, chained by events; two staging slots at the end of the workspace alternate, so the upload of submission
// i+1 and the download of submission i-1 overlap the layer of submission i.  Nothing here blocks the host.
int mok_moe_forward_host_async(const mok_args* a, const void* x_host, void* out_host) {
    WsLayout L;
    if (!a) return MOK_ERR_NULL;
    const size_t act = 2 * (size_t)(a->T > 0 ? a->T : 0) * (size_t)(a->H > 0 ? a->H : 0);
    const size_t act_al = align_up(act, 256);
    int rc = validate(a, &L, 4 * act_al);
    if (rc || a->T == 0) return rc;
    if (!x_host || !out_host) return MOK_ERR_NULL;
    if (a->topk_idx || a->topk_w || a->counts || a->offsets || a->perm || a->inv_perm) return MOK_ERR_UNSUPPORTED;
    HostPipe* p = nullptr;
    if ((rc = host_pipe(&p))) return rc;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(a->stream);
    char* ws = reinterpret_cast<char*>(a->workspace);
    const int slot = (int)(p->n_async & 1ull);
    __nv_bfloat16* xd = reinterpret_cast<__nv_bfloat16*>(ws + L.total + (size_t)slot * 2 * act_al);
    __nv_bfloat16* od = reinterpret_cast<__nv_bfloat16*>(ws + L.total + (size_t)slot * 2 * act_al + act_al);
    cudaError_t e;
    // the slot's x copy is free once the layer that read it has run; its out copy once that result has been downloaded.
    // Three stages of about equal length (upload, layer, download) thus stay busy with two slots.
    if (p->slot_used[slot] && (e = cudaStreamWaitEvent(p->s_in, p->a_fwd[slot], 0)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaMemcpyAsync(xd, x_host, act, cudaMemcpyHostToDevice, p->s_in)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaEventRecord(p->a_in[slot], p->s_in)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaStreamWaitEvent(s, p->a_in[slot], 0)) != cudaSuccess) return cuda_fail(e);
    if (p->slot_used[slot] && (e = cudaStreamWaitEvent(s, p->slot_free[slot], 0)) != cudaSuccess) return cuda_fail(e);
    // The status word is shared by every submission on this workspace: only the first submission after a
    // mok_host_wait clears it, so a device-side failure of ANY submission is still there when the caller reads it.
    if ((rc = forward_device(a, L, xd, od, p->n_since_wait == 0))) return rc;
    ++p->n_since_wait;
    if ((e = cudaEventRecord(p->a_fwd[slot], s)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaStreamWaitEvent(p->s_out, p->a_fwd[slot], 0)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaMemcpyAsync(out_host, od, act, cudaMemcpyDeviceToHost, p->s_out)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaEventRecord(p->slot_free[slot], p->s_out)) != cudaSuccess) return cuda_fail(e);
    p->slot_used[slot] = true;
    ++p->n_async;
    return MOK_OK;
}

int mok_host_wait(void) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= 64) return MOK_ERR_UNSUPPORTED;
    HostPipe& p = g_pipe[dev];
    if (!p.ready) return MOK_OK;
    // every download is ordered after its layer and its upload, and the output stream runs in order
    e = cudaStreamSynchronize(p.s_out);
    p.n_since_wait = 0;
    return e == cudaSuccess ? MOK_OK : cuda_fail(e);
}

int mok_moe_forward(const void* x, const float* W_router, const void* W_gate_up, const void* W_down,
                    const void* W_shared_gate_up, const void* W_shared_down,
                    int T, int H, int I, int I_shared, int E, int k, void* out, void* stream) {
    WsLayout L;
    if (!ws_layout(T, H, I, I_shared, E, k, &L)) return MOK_ERR_SHAPE;
    if (T == 0) return MOK_OK;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= 64) return MOK_ERR_UNSUPPORTED;
    OwnedWs& o = g_owned[dev];
    if (o.bytes < L.total) {
        if (o.ptr) {
            e = cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(stream));
            if (e != cudaSuccess) return cuda_fail(e);
            cudaFree(o.ptr);
            o.ptr = nullptr;
            o.bytes = 0;
        }
        e = cudaMalloc(&o.ptr, L.total);
        if (e != cudaSuccess) { o.ptr = nullptr; return cuda_fail(e); }
        o.bytes = L.total;
    }
    mok_args a;
    memset(&a, 0, sizeof(a));
    a.x = x; a.W_router = W_router; a.W_gate_up = W_gate_up; a.W_down = W_down;
    a.W_shared_gate_up = W_shared_gate_up; a.W_shared_down = W_shared_down;
    a.T = T; a.H = H; a.I = I; a.I_shared = I_shared; a.E = E; a.k = k;
    a.out = out; a.workspace = o.ptr; a.workspace_bytes = o.bytes; a.stream = stream;
    return mok_moe_forward_ex(&a);
}

int mok_route(const void* x, const float* W_router, const float* router_bias, int T, int H, int E, int k,
              int32_t* topk_idx, float* topk_w, void* workspace, size_t workspace_bytes,
              const mok_config* config, void* stream) {
    WsLayout L;
    if (!ws_layout(T, H, 8, 0, E, k, &L)) return MOK_ERR_SHAPE;
    if (T == 0) return MOK_OK;
    if (!x || !W_router || !topk_idx || !topk_w) return MOK_ERR_NULL;
    if (!aligned16(x) || !aligned16(W_router)) return MOK_ERR_ALIGN;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < L.total) return MOK_ERR_WORKSPACE;
    mok_args a;
    memset(&a, 0, sizeof(a));
    a.W_router = W_router; a.router_bias = router_bias; a.T = T; a.H = H; a.E = E; a.k = k;
    a.topk_idx = topk_idx; a.topk_w = topk_w; a.config = config;
    return route_stage(&a, L, reinterpret_cast<char*>(workspace), reinterpret_cast<const __nv_bfloat16*>(x),
                       reinterpret_cast<cudaStream_t>(stream));
}

int mok_schedule(const int32_t* topk_idx, int T, int E, int k, int32_t* counts, int32_t* offsets, int32_t* perm,
                 int32_t* inv_perm, void* workspace, size_t workspace_bytes, void* stream) {
    WsLayout L;
    if (!ws_layout(T, 8, 8, 0, E, k, &L)) return MOK_ERR_SHAPE;
    if (T == 0) return MOK_OK;
    if (!topk_idx) return MOK_ERR_NULL;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < L.total) return MOK_ERR_WORKSPACE;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    char* ws = reinterpret_cast<char*>(workspace);
    cudaError_t e = cudaMemsetAsync(ws + L.header, 0, sizeof(WsHeader), s);
    if (e != cudaSuccess) return cuda_fail(e);
    e = launch_schedule(topk_idx, T, E, k, TILE_M, TILE_M, L, ws, counts, offsets, perm, inv_perm, s);
    return e == cudaSuccess ? MOK_OK : cuda_fail(e);
}

int mok_read_status(const void* workspace, void* stream) {
    if (!workspace) return MOK_ERR_NULL;
    cudaError_t e = cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e);
    WsHeader h;
    e = cudaMemcpy(&h, workspace, sizeof(h), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e);
    return h.status;
}

int mok_debug_counters(const void* workspace, void* stream, unsigned long long* out) {
    if (!workspace || !out) return MOK_ERR_NULL;
    cudaError_t e = cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e);
    WsHeader h;
    e = cudaMemcpy(&h, workspace, sizeof(h), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e);
    memcpy(out, h.dbg, sizeof(h.dbg));
    return MOK_OK;
}

int mok_launch_count(int T, int H, int I, int I_shared, int E, int k, const mok_config* config) {
    WsLayout L;
    if (!ws_layout(T, H, I, I_shared, E, k, &L) || T == 0) return 0;
    // router (1 fp32-FMA kernel, or split + GEMM + top-k + near-tie fix-up), 3 schedule kernels (1 up to 2048 routes), (gather on the SIMT path),
    // 2 routed GEMMs, (2 shared GEMMs), combine
    // (MXFP8 mode: the token-row quantiser instead of the gather kernel; its two memsets are not counted)
    const int pre = use_mx(config) ? 1 : (fused_gather(config, I) ? 0 : 1);
    // (with mok_args.W_router_split the router's split kernel is not launched: one launch less than counted here;
    //  with config.fused_ffn = 2 the two routed GEMMs are the tile-list kernel + ONE persistent kernel: the same count)
    //  with config.fused_ffn = 3 that kernel also does the combine: one launch less)
    const int tile_m = use_mx(config) ? TILE_M : tile_rows(config, I);
    const int combine = config && config->fused_ffn == 3 && use_fused_ffn(config, H, I, tile_m, L.R, E, L.max_ftiles) ? 0 : 1;
    const int sched = (long long)T * k <= SCHED_CHUNK ? 1 : 3;       // small batches: the schedule is one block
    return (use_simt_router(config, k) ? 1 : use_fused_router(config, E, k) ? 3 : 4) + sched + pre + 2 + (I_shared > 0 ? 2 : 0) + combine;
}

int mok_profile_begin(int max_calls) {
    if (max_calls <= 0) return MOK_ERR_SHAPE;
    if (g_prof.ev) return MOK_ERR_SHAPE;            // a session is already open
    const size_t n = (size_t)max_calls * (MOK_STAGE_COUNT + 1);
    g_prof.ev = new cudaEvent_t[n];
    for (size_t i = 0; i < n; ++i) {
        cudaError_t e = cudaEventCreate(&g_prof.ev[i]);
        if (e != cudaSuccess) {
            for (size_t j = 0; j < i; ++j) cudaEventDestroy(g_prof.ev[j]);
            delete[] g_prof.ev;
            g_prof.ev = nullptr;
            return cuda_fail(e);
        }
    }
    g_prof.pred = new uint8_t[(size_t)max_calls * MOK_STAGE_COUNT];
    for (size_t i = 0; i < (size_t)max_calls * MOK_STAGE_COUNT; ++i) g_prof.pred[i] = (uint8_t)(i % MOK_STAGE_COUNT);
    g_prof.max_calls = max_calls;
    g_prof.n_calls = 0;
    return MOK_OK;
}

int mok_profile_end(float* ms, int max_calls_out, int* n_calls) {
    if (!g_prof.ev) return MOK_ERR_SHAPE;
    int rc = MOK_OK;
    const int n = g_prof.n_calls < max_calls_out ? g_prof.n_calls : max_calls_out;
    if (g_prof.n_calls > 0) {
        cudaError_t e = cudaEventSynchronize(g_prof.ev[(size_t)(g_prof.n_calls - 1) * (MOK_STAGE_COUNT + 1) + MOK_STAGE_COUNT]);
        if (e != cudaSuccess) rc = cuda_fail(e);
    }
    for (int c = 0; c < n && rc == MOK_OK && ms; ++c) {
        cudaEvent_t* ev = g_prof.ev + (size_t)c * (MOK_STAGE_COUNT + 1);
        for (int st = 0; st < MOK_STAGE_COUNT; ++st) {
            float t = 0.f;
            cudaError_t e = cudaEventElapsedTime(&t, ev[g_prof.pred[(size_t)c * MOK_STAGE_COUNT + st]], ev[st + 1]);
            if (e != cudaSuccess) { rc = cuda_fail(e); break; }
            ms[(size_t)c * MOK_STAGE_COUNT + st] = t;
        }
    }
    if (n_calls) *n_calls = n;
    const size_t total = (size_t)g_prof.max_calls * (MOK_STAGE_COUNT + 1);
    for (size_t i = 0; i < total; ++i) cudaEventDestroy(g_prof.ev[i]);
    delete[] g_prof.ev;
    delete[] g_prof.pred;
    g_prof = Profiler();
    return rc;
}

int mok_last_cuda_error(void) { return g_last_cuda_error; }

int mok_selftest_per_device(void) {
    // walks the per-device launch-state cache with a stand-in for the configuration step; no CUDA call is made
    static PerDevice cache;
    int calls = 0, fail_next = 0, out = 0;
    auto configure = [&](int dev, int* value) {
        ++calls;
        if (fail_next) { fail_next = 0; return cudaErrorInvalidValue; }
        *value = 100 + dev;
        return cudaSuccess;
    };
    for (int d = 0; d < MAX_DEVICES; ++d) cache.v[d].store(0);
    if (cache.get(3, &out, configure) != cudaSuccess || out != 103 || calls != 1) return 1;
    if (cache.get(3, &out, configure) != cudaSuccess || out != 103 || calls != 1) return 2;   // cached
    if (cache.get(5, &out, configure) != cudaSuccess || out != 105 || calls != 2) return 3;   // a second device configures again
    if (cache.get(3, &out, configure) != cudaSuccess || out != 103 || calls != 2) return 4;
    fail_next = 1;                                                                           // a failure is not remembered
    if (cache.get(7, &out, configure) != cudaErrorInvalidValue || calls != 3) return 5;
    if (cache.get(7, &out, configure) != cudaSuccess || out != 107 || calls != 4) return 6;
    if (cache.get(-1, &out, configure) != cudaErrorInvalidDevice || cache.get(MAX_DEVICES, &out, configure) != cudaErrorInvalidDevice)
        return 7;
    if (calls != 4) return 8;
    return MOK_OK;
}

const char* mok_status_string(int status) {
    switch (status) {
        case MOK_OK: return "ok";
        case MOK_ERR_NULL: return "a required pointer is NULL";
        case MOK_ERR_SHAPE: return "unsupported or inconsistent sizes";
        case MOK_ERR_ALIGN: return "a tensor pointer is not 16-byte aligned";
        case MOK_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case MOK_ERR_CUDA: return "a CUDA call failed";
        case MOK_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out";
        case MOK_ERR_SCHEDULE: return "the dispatch schedule failed its consistency check";
        case MOK_ERR_UNSUPPORTED: return "unsupported device";
        default: return "unknown status";
    }
}

int mok_version(void) { return 100; }

}  // extern "C"
