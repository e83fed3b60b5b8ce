// Backward pass of the MoE layer (paper, Section 3.4: the router-weight gradient fused into the backward chain, activations recomputed instead of stored;
// Section 4.1: backward = dgrad + wgrad, twice the forward FLOPs).  The paper prints no formulas; this is the chain
// rule of the Section 2.1 definition, arranged so that every contraction runs on the forward pass's grouped tcgen05
// GEMM kernels:
//
//   saved from the forward pass: only the routing (top-k ids and weights).  Everything else is recomputed from x
//   (Section 3.4): the dispatch schedule from the ids, the pre-activations gu = [g | u] = Xg Wgu^T.
//
//   activation gradients (dgrad)
//     dhu  = gather(dout) Wd            grouped GEMM, rows pulled from dout through the schedule (K = H, N = I)
//     per row p (route j = (t, s), weight w):                                       [swiglu_bwd_kernel]
//         h = silu(g) u,   dw[t,s] = <dhu, h>   (the router-weight gradient, fused: y is never rebuilt)
//         dh = w dhu,  dg = dh u sig (1 + g (1 - sig)),  du = dh silu(g),  hw = w h
//     dXg  = [dg | du] Wgu              grouped GEMM (K = 2I, N = H)
//     dx[t] = dx_shared[t] + sum_s dXg[pos[t,s]]      the forward combine kernel with unit weights (fixed order)
//   weight gradients (wgrad), per expert e over its rows (a contraction over the ROW index):
//     dWd_e  = gather(dout)_e^T hw_e    [H, I]        dWgu_e = [dg | du]_e^T Xg_e    [2I, H]
//   Both operands of these products are activations whose contraction index is the row, so they are transposed once
//   ([rows, C] -> [C, rows], pad rows zero) and fed to the same kernel in its "K range per expert" mode.
//   The shared expert is the same computation on every token with w = 1 and no dw.
//   The weights enter dgrad transposed (Wd^T, Wgu^T as K-contiguous operands): they are transposed into the workspace
//   at the start of every call (they change between training steps).
// Intermediates (gu, dhu, dg|du, hw, dXg) are bf16 like the forward pass's h and y; accumulation is fp32 in TMEM;
// dw is accumulated in fp32.  Deterministic: fixed tile order, fixed k order, fixed combine order, no float atomics.
#include "mok_internal.cuh"
#include <string.h>

namespace mok {

// [B, R, C] -> [B, C, R] for bf16 (C a multiple of 8), 128 x 128 tiles through shared memory with 16-byte global
// accesses on both sides: a block reads 128 row segments of 256 bytes and writes 128 column segments of 256 bytes.
// With `route_of_row` the source rows are gathered on the fly: row p of the (padded) dispatch space is token
// route_of_row[p] / k of `in` when p is a real row of its expert, and zero when it is padding -- the gather and the
// transpose of the weight-gradient operands in one pass.  Rows >= R of the last tile are not written (out_ld >= R).
constexpr int TT = 128;                                       // transpose tile: 128 x 128 elements
__global__ void __launch_bounds__(256)
transpose_kernel(const __nv_bfloat16* __restrict__ in, __nv_bfloat16* __restrict__ out, int R, int C, long long in_batch,
                 long long out_batch, int out_ld, const int32_t* __restrict__ route_of_row, int k,
                 const int32_t* __restrict__ tile_expert, const int32_t* __restrict__ pad_offsets,
                 const int32_t* __restrict__ counts, const WsHeader* __restrict__ hdr) {
    // 32-bit words, row r at word r * PW + (r >> 3): the skew of one word per 8 rows keeps the column reads of the
    // write phase (rows 8 apart across the lanes) on different banks
    extern __shared__ __align__(16) uint32_t tile[];
    constexpr int PW = TT / 2 + 4;
    const __nv_bfloat16* src = in + (size_t)blockIdx.z * in_batch;
    __nv_bfloat16* dst = out + (size_t)blockIdx.z * out_batch;
    const int r0 = blockIdx.y * TT, c0 = blockIdx.x * TT;
    const int rows_live = route_of_row ? hdr->n_mtiles * TILE_M : R;   // gather mode: rows beyond the schedule are zero
    uint4 v[8];
#pragma unroll
    for (int pass = 0; pass < 8; ++pass) {                     // 8 independent 16-byte loads per thread in flight
        const int r = (threadIdx.x >> 4) + pass * 16, ch = threadIdx.x & 15;
        v[pass] = make_uint4(0u, 0u, 0u, 0u);
        const int p = r0 + r;
        if (p < R && c0 + ch * 8 < C) {
            long long srow = p;
            if (route_of_row) {
                srow = -1;
                if (p < rows_live) {
                    const int e = tile_expert[p / TILE_M];
                    if (p - pad_offsets[e] < counts[e]) srow = route_of_row[p] / k;
                }
            }
            if (srow >= 0) v[pass] = __ldg(reinterpret_cast<const uint4*>(src + (size_t)srow * C + c0 + ch * 8));
        }
    }
#pragma unroll
    for (int pass = 0; pass < 8; ++pass) {
        const int r = (threadIdx.x >> 4) + pass * 16, ch = threadIdx.x & 15;
        uint32_t* row = tile + r * PW + (r >> 3) + ch * 4;
        row[0] = v[pass].x; row[1] = v[pass].y; row[2] = v[pass].z; row[3] = v[pass].w;
    }
    __syncthreads();
#pragma unroll
    for (int pass = 0; pass < 8; ++pass) {
        const int c = (threadIdx.x >> 4) + pass * 16, rc = threadIdx.x & 15;
        if (c0 + c >= C || r0 + rc * 8 >= R) continue;
        uint32_t wv[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int r = rc * 8 + j;
            wv[j] = tile[r * PW + (r >> 3) + (c >> 1)];
        }
        const uint32_t sel = (c & 1) ? 0x7632u : 0x5410u;          // high or low halves of two words
        uint4 o;
        o.x = __byte_perm(wv[0], wv[1], sel); o.y = __byte_perm(wv[2], wv[3], sel);
        o.z = __byte_perm(wv[4], wv[5], sel); o.w = __byte_perm(wv[6], wv[7], sel);
        *reinterpret_cast<uint4*>(dst + (size_t)(c0 + c) * out_ld + r0 + rc * 8) = o;
    }
}

// R must be a multiple of 8 wherever the output rows are written 16 bytes at a time: here R is Rpad, Tpad-padded T (the
// tail chunk past R is written with the zeros read for p >= R; out_ld covers it) or a weight dimension (multiple of 32).
static cudaError_t launch_transpose(const __nv_bfloat16* in, __nv_bfloat16* out, int batch, int R, int C, int out_ld,
                                    cudaStream_t s, const int32_t* route_of_row = nullptr, int k = 1,
                                    const int32_t* tile_expert = nullptr, const int32_t* pad_offsets = nullptr,
                                    const int32_t* counts = nullptr, const WsHeader* hdr = nullptr) {
    if (batch <= 0 || R <= 0 || C <= 0) return cudaSuccess;
    static PerDevice configured;      // per device: 1 once the kernel has its shared-memory opt-in there
    constexpr int smem = (TT * (TT / 2 + 4) + TT / 8) * 4;
    int dev = 0, done = 0;
    cudaError_t e = current_device(&dev);
    if (e != cudaSuccess) return e;
    e = configured.get(dev, &done, [&](int, int* flag) {
        *flag = 1;
        return cudaFuncSetAttribute(transpose_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    });
    if (e != cudaSuccess) return e;
    dim3 grid((C + TT - 1) / TT, (R + TT - 1) / TT, batch);
    transpose_kernel<<<grid, 256, smem, s>>>(in, out, R, C, (long long)R * C, (long long)C * out_ld, out_ld, route_of_row, k,
                                          tile_expert, pad_offsets, counts, hdr);
    return cudaGetLastError();
}

// SwiGLU backward, one warp per row of the (padded) dispatch space, or per token for the shared expert.
//   gu [rows, 2I] = [g | u] (bf16), dhu [rows, I] = dL/dh before the router weight (bf16)
//   -> dgu [rows, 2I] = [dg | du], hw [rows, I] = w h, dw[route] = <dhu, h>.
// Routed mode: row p belongs to expert tile_expert[p / 128]; rows past the expert's count are padding and get zeros
// (the weight-gradient products run over whole padded segments).  Dense mode (row_route == NULL): w = 1, no dw.
__global__ void __launch_bounds__(256)
swiglu_bwd_kernel(const __nv_bfloat16* __restrict__ gu, const __nv_bfloat16* __restrict__ dhu, int I, int rows_dense,
                  const WsHeader* __restrict__ hdr, const int32_t* __restrict__ tile_expert,
                  const int32_t* __restrict__ pad_offsets, const int32_t* __restrict__ counts,
                  const int32_t* __restrict__ row_route, const float* __restrict__ w,
                  __nv_bfloat16* __restrict__ dgu, __nv_bfloat16* __restrict__ hw, float* __restrict__ dw) {
    const int lane = threadIdx.x & 31;
    const int rows = row_route ? hdr->n_mtiles * TILE_M : rows_dense;
    const int chunks = I >> 3;
    for (int p = blockIdx.x * 8 + (threadIdx.x >> 5); p < rows; p += gridDim.x * 8) {
        float wt = 1.f;
        int route = -1;
        bool valid = true;
        if (row_route) {
            const int e = tile_expert[p / TILE_M];
            valid = (p - pad_offsets[e]) < counts[e];
            if (valid) { route = row_route[p]; wt = w[route]; }
        }
        const uint4* g4 = reinterpret_cast<const uint4*>(gu + (size_t)p * 2 * I);
        const uint4* u4 = reinterpret_cast<const uint4*>(gu + (size_t)p * 2 * I + I);
        const uint4* d4 = reinterpret_cast<const uint4*>(dhu + (size_t)p * I);
        uint4* dg4 = reinterpret_cast<uint4*>(dgu + (size_t)p * 2 * I);
        uint4* du4 = reinterpret_cast<uint4*>(dgu + (size_t)p * 2 * I + I);
        uint4* hw4 = reinterpret_cast<uint4*>(hw + (size_t)p * I);
        float dot = 0.f;
        for (int c = lane; c < chunks; c += 32) {
            uint4 og = make_uint4(0u, 0u, 0u, 0u), ou = og, oh = og;
            if (valid) {
                const uint4 rg = g4[c], ru = u4[c], rd = d4[c];
                const __nv_bfloat162* pg = reinterpret_cast<const __nv_bfloat162*>(&rg);
                const __nv_bfloat162* pu = reinterpret_cast<const __nv_bfloat162*>(&ru);
                const __nv_bfloat162* pd = reinterpret_cast<const __nv_bfloat162*>(&rd);
                __nv_bfloat162* qg = reinterpret_cast<__nv_bfloat162*>(&og);
                __nv_bfloat162* qu = reinterpret_cast<__nv_bfloat162*>(&ou);
                __nv_bfloat162* qh = reinterpret_cast<__nv_bfloat162*>(&oh);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float2 g = __bfloat1622float2(pg[q]), u = __bfloat1622float2(pu[q]), d = __bfloat1622float2(pd[q]);
                    float r0[3], r1[3];
                    {
                        const float sig = 1.f / (1.f + __expf(-g.x)), a = g.x * sig, h = a * u.x, dh = wt * d.x;
                        dot = fmaf(d.x, h, dot);
                        r0[0] = dh * u.x * sig * (1.f + g.x * (1.f - sig)); r0[1] = dh * a; r0[2] = wt * h;
                    }
                    {
                        const float sig = 1.f / (1.f + __expf(-g.y)), a = g.y * sig, h = a * u.y, dh = wt * d.y;
                        dot = fmaf(d.y, h, dot);
                        r1[0] = dh * u.y * sig * (1.f + g.y * (1.f - sig)); r1[1] = dh * a; r1[2] = wt * h;
                    }
                    qg[q] = __floats2bfloat162_rn(r0[0], r1[0]);
                    qu[q] = __floats2bfloat162_rn(r0[1], r1[1]);
                    qh[q] = __floats2bfloat162_rn(r0[2], r1[2]);
                }
            }
            dg4[c] = og;
            du4[c] = ou;
            hw4[c] = oh;
        }
        if (dw && row_route) {
            // fixed-order reduction over the warp (every lane takes part; `valid` is the same for the whole warp)
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
            if (lane == 0 && valid) dw[route] = dot;
        }
    }
}

// Workspace of the backward pass: the forward layout (schedule tables; its h / y / hs / ysh regions hold hw, dXg, the
// shared expert's h and dx) followed by the regions only the backward pass needs.
struct BwdLayout {
    WsLayout F;
    size_t row_route, gu, dhu, dgu, WdT, WguT, WsdT, WsguT, gus, dhus, dgus;
    size_t doutT, hwT, dguT, xgT;      // transposed activations of the weight-gradient products
    size_t total;
};

static bool bwd_layout(int T, int H, int I, int Is, int E, int k, BwdLayout* B) {
    if ((H % 32) || (I % 32) || (Is % 32)) return false;
    if (!ws_layout(T, H, I, Is, E, k, &B->F)) return false;
    const WsLayout& F = B->F;
    size_t off = F.total;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    const size_t Rp = (size_t)F.Rpad, Tp = (size_t)F.Tpad;
    B->row_route = take(sizeof(int32_t) * Rp);
    B->gu = take(2 * Rp * 2 * I);
    B->dhu = take(2 * Rp * I);
    B->dgu = take(2 * Rp * 2 * I);
    B->WdT = take(2 * (size_t)E * I * H);
    B->WguT = take(2 * (size_t)E * H * 2 * I);
    B->WsdT = take(2 * (size_t)Is * H);
    B->WsguT = take(2 * (size_t)H * 2 * Is);
    B->gus = take(2 * Tp * 2 * Is);
    B->dhus = take(2 * Tp * Is);
    B->dgus = take(2 * Tp * 2 * Is);
    const size_t Rm = Rp > Tp ? Rp : Tp;
    B->doutT = take(2 * (size_t)H * Rm);
    B->hwT = take(2 * (size_t)(I > Is ? I : Is) * Rm);
    B->dguT = take(2 * (size_t)2 * (I > Is ? I : Is) * Rm);
    B->xgT = take(2 * (size_t)H * Rm);
    B->total = off;
    return true;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// What the expert-parallel backward adds to the one-rank chain (see backward_chain).
struct EpBwd {
    int n_ranks, T_local;
    long long routes_expected;                         // expected share of this rank, for the kernel choice
    const __nv_bfloat16* x_peers[MOK_MAX_RANKS];
    const __nv_bfloat16* dout_peers[MOK_MAX_RANKS];
    const float* w_all;                                // [n_ranks * T_local * k] router weights of every rank's routes
    float* dw_routes;                                  // [n_ranks * T_local * k] dL/dw of the routes served here
    __nv_bfloat16* dxg;                                // [rows, H] dL/d(gathered x) of the rows served here
    __nv_bfloat16* dx_shared;                          // [Tpad, H] shared expert's dx of this rank's tokens
};
int backward_chain(const mok_bwd_args* a, const BwdLayout& B, const WsLayout& L, const EpBwd* ep);

}  // namespace mok

using namespace mok;

extern "C" {

size_t mok_bwd_workspace_bytes(int T, int H, int I, int I_shared, int E, int k) {
    BwdLayout B;
    return bwd_layout(T, H, I, I_shared, E, k, &B) ? B.total : 0;
}

int mok_moe_backward(const mok_bwd_args* a) {
    if (!a) return MOK_ERR_NULL;
    BwdLayout B;
    if (!bwd_layout(a->T, a->H, a->I, a->I_shared, a->E, a->k, &B)) return MOK_ERR_SHAPE;
    if ((a->I_shared > 0) != (a->W_shared_gate_up != nullptr) || (a->I_shared > 0) != (a->W_shared_down != nullptr))
        return MOK_ERR_SHAPE;
    if (a->T == 0) return MOK_OK;
    if (!a->x || !a->W_gate_up || !a->W_down || !a->topk_idx || !a->topk_w || !a->dout || !a->dx) return MOK_ERR_NULL;
    if (!aligned16(a->x) || !aligned16(a->W_gate_up) || !aligned16(a->W_down) || !aligned16(a->W_shared_gate_up) ||
        !aligned16(a->W_shared_down) || !aligned16(a->dout) || !aligned16(a->dx) || !aligned16(a->dW_gate_up) ||
        !aligned16(a->dW_down) || !aligned16(a->dW_shared_gate_up) || !aligned16(a->dW_shared_down))
        return MOK_ERR_ALIGN;
    if (!a->workspace || (reinterpret_cast<uintptr_t>(a->workspace) & 255u) || a->workspace_bytes < B.total)
        return MOK_ERR_WORKSPACE;
    if (a->config && (a->config->impl != MOK_IMPL_TCGEN05 || a->config->grid < 0 || a->config->precision != MOK_PRECISION_BF16 ||
                      a->config->gather_mode < 0 || a->config->gather_mode > 2 ||
                      (a->config->cta_group != 0 && a->config->cta_group != 1 && a->config->cta_group != 3)))
        return MOK_ERR_SHAPE;
    const bool want_w = a->dW_gate_up || a->dW_down || a->dW_shared_gate_up || a->dW_shared_down;
    if (want_w && (!a->dW_gate_up || !a->dW_down || (a->I_shared > 0 && (!a->dW_shared_gate_up || !a->dW_shared_down))))
        return MOK_ERR_NULL;
    return backward_chain(a, B, B.F, nullptr);
}

}  // extern "C"

namespace mok {

// The chain of the backward pass on one rank's dispatch space.  a: the one-rank arguments (T = tokens of the shared
// expert and of dx, E = experts of the schedule tables, x / dout = this rank's token rows).  ep == NULL: one rank -- the
// schedule is rebuilt from a->topk_idx and the chain ends with the combine into a->dx.  ep != NULL: expert parallelism --
// the caller has built the schedule for the local experts (row_token holds global token ids, row_route global route
// ids), rows are pulled from the owners' buffers, and the chain leaves dL/d(gathered x) and the shared expert's dx in
// the caller's buffers for the owners' combine.
int backward_chain(const mok_bwd_args* a, const BwdLayout& B, const WsLayout& L, const EpBwd* ep) {
    const int T = a->T, H = a->H, I = a->I, Is = a->I_shared, E = a->E, k = a->k;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(a->stream);
    char* ws = reinterpret_cast<char*>(a->workspace);
    WsHeader* hdr = reinterpret_cast<WsHeader*>(ws + L.header);
    const __nv_bfloat16* x = reinterpret_cast<const __nv_bfloat16*>(a->x);
    const __nv_bfloat16* dout = reinterpret_cast<const __nv_bfloat16*>(a->dout);
    auto bf = [&](size_t off) { return reinterpret_cast<__nv_bfloat16*>(ws + off); };
    const bool want_w = a->dW_gate_up || a->dW_down || a->dW_shared_gate_up || a->dW_shared_down;
    mok_config cfg;
    memset(&cfg, 0, sizeof(cfg));
    if (a->config) { cfg.grid = a->config->grid; cfg.cta_group = a->config->cta_group; cfg.gang_sync = a->config->gang_sync; }
    cudaError_t e = cudaSuccess;
    if (!ep) {
        e = cudaMemsetAsync(hdr, 0, sizeof(WsHeader), s);
        if (e != cudaSuccess) return cuda_fail(e);
        // the dispatch schedule again, from the saved routing (no host readback)
        e = launch_schedule(a->topk_idx, T, E, k, TILE_M, TILE_M, L, ws, nullptr, nullptr, nullptr, nullptr, s,
                            reinterpret_cast<int32_t*>(ws + B.row_route));
        if (e != cudaSuccess) return cuda_fail(e);
    }
    const float* w_routes = ep ? ep->w_all : a->topk_w;
    float* dw_routes = ep ? ep->dw_routes : a->dw;
    __nv_bfloat16* dxg = ep ? ep->dxg : bf(L.y);
    __nv_bfloat16* dx_shared = ep ? ep->dx_shared : bf(L.ysh);
    // rows pulled from the owners' buffers (expert parallelism): which buffers a gathering GEMM reads
    auto pull_from = [&](GemmArgs& q, const __nv_bfloat16* const* peers) {
        q.peer_tokens = 0;
        if (!ep) return;
        q.peer_tokens = ep->T_local;
        for (int r = 0; r < ep->n_ranks; ++r) q.peer_x[r] = peers[r];
    };
    // The transposed products of dgrad read the weights MN-major, as they sit in memory (W[e] = [K, N], N contiguous).
    // config.gather_mode = 2 selects the older path instead: K-contiguous transposed copies made at every call.
    const bool wT = !ep && a->config && a->config->gather_mode == 2;
    if (wT) {
        if ((e = launch_transpose(reinterpret_cast<const __nv_bfloat16*>(a->W_down), bf(B.WdT), E, H, I, H, s)) != cudaSuccess) return cuda_fail(e);
        if ((e = launch_transpose(reinterpret_cast<const __nv_bfloat16*>(a->W_gate_up), bf(B.WguT), E, 2 * I, H, 2 * I, s)) != cudaSuccess) return cuda_fail(e);
    }
    auto dgrad_gemm = [&](GemmArgs& q, const void* W, size_t WT_off) -> int {
        if (wT) { q.B = bf(WT_off); q.b_mn = 0; return run_gemm(q, false, &cfg, L, ws, s); }
        q.B = reinterpret_cast<const __nv_bfloat16*>(W); q.b_mn = 1;
        WsHeader* h2 = hdr;
        q.n_mtiles = q.dense_rows > 0 ? q.n_mtiles : &h2->n_mtiles2;        // the 256-row kernel's tile table
        const int32_t* mt = q.mt_start; const int32_t* te = q.tile_expert;
        if (q.dense_rows == 0) {
            q.mt_start = reinterpret_cast<const int32_t*>(ws + L.mt_start2);
            q.tile_expert = reinterpret_cast<const int32_t*>(ws + L.tile_expert2);
        }
        // (the row tiles of an expert share a tile of W here as in the forward products: synchronised starts where they pay)
        const int rcg = gang_prepare(q, false, &cfg, L, ws, s);
        if (rcg) return rcg;
        cudaError_t ee = launch_gemm_m2(q, EPI_BF16, cfg.grid, s);
        q.n_mtiles = &h2->n_mtiles; q.mt_start = mt; q.tile_expert = te; q.b_mn = 0; q.gang = nullptr;
        return ee == cudaSuccess ? MOK_OK : cuda_fail(ee);
    };

    GemmArgs g;
    memset(&g, 0, sizeof(g));
    g.header = hdr;
    g.n_mtiles = &hdr->n_mtiles;
    g.tile_expert = reinterpret_cast<const int32_t*>(ws + L.tile_expert);
    g.mt_start = reinterpret_cast<const int32_t*>(ws + L.mt_start);
    g.max_mt = L.max_mt;
    g.tile_m = TILE_M;
    g.pad_offsets = reinterpret_cast<const int32_t*>(ws + L.pad_offsets);
    g.counts = reinterpret_cast<const int32_t*>(ws + L.counts);
    g.dbg_slot = -1;
    g.E = E; g.rows_pad = L.Rpad; g.dense_rows = 0; g.total_rows = ep ? ep->routes_expected : L.R;
    int rc;
    // Four products need the rows of x or dout in dispatch order.  Up to I = 2048 each of them pulls the rows through the
    // schedule's row_token table inside the GEMM, as the forward pass does (K-major for the recomputation and the dgrad
    // product, MN-major for the weight gradients): no expert-sorted copies (bench workload 3.47 vs 3.73 ms).  A GEMM
    // re-gathers its rows once per tile along the other output dimension (2I/256 or I/256 times), so for wide experts
    // the copies are made once instead (I = 14336: 13.3 vs 13.9 ms, I = 2880: 10.9 vs 11.2 ms), padding rows zero.
    const int32_t* row_token = reinterpret_cast<const int32_t*>(ws + L.row_token);
    const bool pull = !wT && (I <= 2048 || ep);       // (expert parallelism always pulls: there is no local copy to make)
    __nv_bfloat16* XG = bf(L.xg);
    __nv_bfloat16* DG = bf(B.doutT);
    if (!wT && !pull) {
        if ((e = launch_gather(x, H, k, TILE_M, L, ws, s, XG)) != cudaSuccess) return cuda_fail(e);
        if ((e = launch_gather(dout, H, k, TILE_M, L, ws, s, DG)) != cudaSuccess) return cuda_fail(e);
    }
    // gu = Xg Wgu^T  (activation recomputation)
    if (wT || pull) { g.A = x; g.a_rows = T; g.row_token = row_token; if (ep) pull_from(g, ep->x_peers); }
    else { g.A = XG; g.a_rows = L.Rpad; g.row_token = nullptr; }
    g.B = reinterpret_cast<const __nv_bfloat16*>(a->W_gate_up);
    g.C = ws + B.gu; g.K = H; g.N = 2 * I; g.ldc = 2 * I;
    if ((rc = run_gemm(g, false, &cfg, L, ws, s))) return rc;
    // dhu = gather(dout) Wd
    g.A = (wT || pull) ? dout : DG; g.C = ws + B.dhu; g.K = H; g.N = I; g.ldc = I;
    if (ep) pull_from(g, ep->dout_peers);
    if ((rc = dgrad_gemm(g, a->W_down, B.WdT))) return rc;
    g.peer_tokens = 0;
    // SwiGLU backward + router-weight gradient
    {
        int blocks = (L.Rpad + 7) / 8;
        if (blocks > 148 * 16) blocks = 148 * 16;
        swiglu_bwd_kernel<<<blocks, 256, 0, s>>>(bf(B.gu), bf(B.dhu), I, 0, hdr, g.tile_expert, g.pad_offsets, g.counts,
                                                 reinterpret_cast<const int32_t*>(ws + B.row_route), w_routes, bf(B.dgu),
                                                 bf(L.h), dw_routes);
        if ((e = cudaGetLastError()) != cudaSuccess) return cuda_fail(e);
    }
    // dXg = [dg | du] Wgu
    g.row_token = nullptr;
    g.A = bf(B.dgu); g.a_rows = L.Rpad; g.C = dxg; g.K = 2 * I; g.N = H; g.ldc = H;
    if ((rc = dgrad_gemm(g, a->W_gate_up, B.WguT))) return rc;
    if (Is > 0) {   // shared expert: the same chain on every token, w = 1
        if (wT) {
            if ((e = launch_transpose(reinterpret_cast<const __nv_bfloat16*>(a->W_shared_down), bf(B.WsdT), 1, H, Is, H, s)) != cudaSuccess) return cuda_fail(e);
            if ((e = launch_transpose(reinterpret_cast<const __nv_bfloat16*>(a->W_shared_gate_up), bf(B.WsguT), 1, 2 * Is, H, 2 * Is, s)) != cudaSuccess) return cuda_fail(e);
        }
        g.E = 1; g.rows_pad = L.Tpad; g.dense_rows = T; g.a_rows = T;
        g.A = x; g.B = reinterpret_cast<const __nv_bfloat16*>(a->W_shared_gate_up); g.C = ws + B.gus; g.K = H; g.N = 2 * Is; g.ldc = 2 * Is;
        if ((rc = run_gemm(g, false, &cfg, L, ws, s))) return rc;
        g.A = dout; g.C = ws + B.dhus; g.K = H; g.N = Is; g.ldc = Is;
        if ((rc = dgrad_gemm(g, a->W_shared_down, B.WsdT))) return rc;
        int blocks = (T + 7) / 8;
        if (blocks > 148 * 16) blocks = 148 * 16;
        swiglu_bwd_kernel<<<blocks, 256, 0, s>>>(bf(B.gus), bf(B.dhus), Is, T, hdr, nullptr, nullptr, nullptr, nullptr,
                                                 nullptr, bf(B.dgus), bf(L.hs), nullptr);
        if ((e = cudaGetLastError()) != cudaSuccess) return cuda_fail(e);
        g.A = bf(B.dgus); g.a_rows = L.Tpad; g.C = dx_shared; g.K = 2 * Is; g.N = H; g.ldc = H;
        if ((rc = dgrad_gemm(g, a->W_shared_gate_up, B.WsguT))) return rc;
    }
    if (!ep) {
        // dx[t] = dx_shared[t] + sum_s dXg[pos[t,s]]: the forward combine with unit weights, same fixed order
        e = launch_combine(L, ws, T, H, k, Is > 0, reinterpret_cast<__nv_bfloat16*>(a->dx), s, /*unit_weights=*/true);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    if (!want_w) return MOK_OK;

    // ------------------------------------------------------------------ weight gradients
    // Experts without rows keep the zeros written here; every other output element is written by exactly one tile.
    if ((e = cudaMemsetAsync(a->dW_down, 0, 2 * (size_t)E * H * I, s)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaMemsetAsync(a->dW_gate_up, 0, 2 * (size_t)E * 2 * I * H, s)) != cudaSuccess) return cuda_fail(e);
    GemmArgs q;
    memset(&q, 0, sizeof(q));
    q.header = hdr;
    q.n_mtiles = &hdr->n_mtiles;
    q.tile_expert = g.tile_expert; q.mt_start = g.mt_start; q.max_mt = L.max_mt; q.tile_m = TILE_M;
    q.pad_offsets = g.pad_offsets; q.counts = g.counts;
    q.dbg_slot = -1;
    const int Rp = L.Rpad, Tp = L.Tpad;
    if (!wT) {
        // Both operands of a weight-gradient product are read MN-major, exactly as the chain above left them:
        // A = [rows, M] and B = [rows, N] with the row index as K; the operand that is a gathered x or dout is pulled
        // through row_token by the kernel's gather warps (rows past an expert's count read as zero).
        q.b_mn = 1; q.E = E; q.dense_rows = 0; q.K = Rp;
        if (pull) { q.row_token = row_token; q.a_rows = T; }   // dout / x stay in token order: their rows are pulled by the GEMM
        q.kgroup_rows = H; q.A = pull ? dout : DG; q.lda = H; q.gather_mn = pull ? 1 : 0; q.B = bf(L.h); q.N = I; q.ldb = I;
        q.C = a->dW_down; q.rows_pad = E * H; q.ldc = I;
        if (ep) pull_from(q, ep->dout_peers);
        if ((e = launch_gemm_m2(q, EPI_BF16, cfg.grid, s)) != cudaSuccess) return cuda_fail(e);
        q.kgroup_rows = 2 * I; q.A = bf(B.dgu); q.lda = 2 * I; q.B = pull ? x : XG; q.N = H; q.ldb = H; q.gather_mn = pull ? 2 : 0;
        q.C = a->dW_gate_up; q.rows_pad = E * 2 * I; q.ldc = H;
        if (ep) pull_from(q, ep->x_peers);
        if ((e = launch_gemm_m2(q, EPI_BF16, cfg.grid, s)) != cudaSuccess) return cuda_fail(e);
        q.row_token = nullptr; q.gather_mn = 0; q.peer_tokens = 0;
        if (Is > 0) {   // shared expert: one K range over the T tokens (rows past T are zero-filled by the tensor maps)
            q.E = 1; q.dense_rows = T; q.K = T;
            q.kgroup_rows = H; q.A = dout; q.lda = H; q.B = bf(L.hs); q.N = Is; q.ldb = Is;
            q.C = a->dW_shared_down; q.rows_pad = H; q.ldc = Is;
            if ((e = launch_gemm_m2(q, EPI_BF16, cfg.grid, s)) != cudaSuccess) return cuda_fail(e);
            q.kgroup_rows = 2 * Is; q.A = bf(B.dgus); q.lda = 2 * Is; q.B = x; q.N = H; q.ldb = H;
            q.C = a->dW_shared_gate_up; q.rows_pad = 2 * Is; q.ldc = H;
            if ((e = launch_gemm_m2(q, EPI_BF16, cfg.grid, s)) != cudaSuccess) return cuda_fail(e);
        }
        return MOK_OK;
    }
    // dWd_e = gather(dout)_e^T (w h)_e: both operands transposed so that the row index is the contiguous (K) one
    const int32_t* rr = reinterpret_cast<const int32_t*>(ws + B.row_route);
    if ((e = launch_transpose(dout, bf(B.doutT), 1, Rp, H, Rp, s, rr, k, g.tile_expert, g.pad_offsets, g.counts, hdr)) != cudaSuccess)
        return cuda_fail(e);
    if ((e = launch_transpose(bf(L.h), bf(B.hwT), 1, Rp, I, Rp, s)) != cudaSuccess) return cuda_fail(e);
    q.E = E; q.kgroup_rows = H; q.A = bf(B.doutT); q.a_rows = H; q.K = Rp; q.lda = Rp;
    q.B = bf(B.hwT); q.N = I; q.ldb = Rp; q.C = a->dW_down; q.rows_pad = E * H; q.ldc = I; q.dense_rows = 0;
    if ((e = launch_gemm_m2(q, EPI_BF16, cfg.grid, s)) != cudaSuccess) return cuda_fail(e);
    // dWgu_e = [dg | du]_e^T Xg_e
    if ((e = launch_transpose(x, bf(B.xgT), 1, Rp, H, Rp, s, rr, k, g.tile_expert, g.pad_offsets, g.counts, hdr)) != cudaSuccess)
        return cuda_fail(e);
    if ((e = launch_transpose(bf(B.dgu), bf(B.dguT), 1, Rp, 2 * I, Rp, s)) != cudaSuccess) return cuda_fail(e);
    q.kgroup_rows = 2 * I; q.A = bf(B.dguT); q.a_rows = 2 * I; q.B = bf(B.xgT); q.N = H; q.C = a->dW_gate_up;
    q.rows_pad = E * 2 * I; q.ldc = H;
    if ((e = launch_gemm_m2(q, EPI_BF16, cfg.grid, s)) != cudaSuccess) return cuda_fail(e);
    if (Is > 0) {   // shared expert: one group over all T tokens (K tail past T is zero-filled by the tensor map)
        if ((e = launch_transpose(dout, bf(B.doutT), 1, T, H, Tp, s)) != cudaSuccess) return cuda_fail(e);
        if ((e = launch_transpose(bf(L.hs), bf(B.hwT), 1, T, Is, Tp, s)) != cudaSuccess) return cuda_fail(e);
        q.E = 1; q.dense_rows = T; q.K = T; q.lda = Tp; q.ldb = Tp;
        q.kgroup_rows = H; q.A = bf(B.doutT); q.a_rows = H; q.B = bf(B.hwT); q.N = Is; q.C = a->dW_shared_down;
        q.rows_pad = H; q.ldc = Is;
        if ((e = launch_gemm_m2(q, EPI_BF16, cfg.grid, s)) != cudaSuccess) return cuda_fail(e);
        if ((e = launch_transpose(x, bf(B.xgT), 1, T, H, Tp, s)) != cudaSuccess) return cuda_fail(e);
        if ((e = launch_transpose(bf(B.dgus), bf(B.dguT), 1, T, 2 * Is, Tp, s)) != cudaSuccess) return cuda_fail(e);
        q.kgroup_rows = 2 * Is; q.A = bf(B.dguT); q.a_rows = 2 * Is; q.B = bf(B.xgT); q.N = H; q.C = a->dW_shared_gate_up;
        q.rows_pad = 2 * Is; q.ldc = H;
        if ((e = launch_gemm_m2(q, EPI_BF16, cfg.grid, s)) != cudaSuccess) return cuda_fail(e);
    }
    return MOK_OK;
}

}  // namespace mok

namespace mok {

// padded row -> global route id (source rank * routes per rank + route) from the schedule's `pos` table
__global__ void __launch_bounds__(256)
ep_row_route_kernel(const int32_t* __restrict__ idx_all, const int32_t* __restrict__ pos, int total_routes, int lo, int Lx,
                    int32_t* __restrict__ row_route) {
    for (int g = blockIdx.x * 256 + threadIdx.x; g < total_routes; g += gridDim.x * 256) {
        const int e = idx_all[g];
        if (e >= lo && e < lo + Lx) row_route[pos[g]] = g;
    }
}

// dw[t, s] of this rank's routes, from the rank that served each route
struct EpDwArgs {
    const float* dw[MOK_MAX_RANKS];
    const int32_t* idx;
    float* out;
    int32_t n, Lx, route_base;
};
__global__ void __launch_bounds__(256)
ep_dw_kernel(const __grid_constant__ EpDwArgs a) {
    for (int j = blockIdx.x * 256 + threadIdx.x; j < a.n; j += gridDim.x * 256)
        a.out[j] = a.dw[a.idx[j] / a.Lx][(size_t)a.route_base + j];
}

static bool ep_bwd_layout(int n_ranks, int T_local, int H, int I, int Is, int E, int k, BwdLayout* B) {
    if ((H % 32) || (I % 32) || (Is % 32)) return false;
    if (!ep_layout(n_ranks, T_local, H, I, Is, E, k, &B->F)) return false;
    const WsLayout& F = B->F;
    size_t off = F.total;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    const size_t Rp = (size_t)F.Rpad, Tp = (size_t)F.Tpad;
    B->row_route = take(sizeof(int32_t) * Rp);
    B->gu = take(2 * Rp * 2 * I);
    B->dhu = take(2 * Rp * I);
    B->dgu = take(2 * Rp * 2 * I);
    B->gus = take(2 * Tp * 2 * Is);
    B->dhus = take(2 * Tp * Is);
    B->dgus = take(2 * Tp * 2 * Is);
    B->WdT = B->WguT = B->WsdT = B->WsguT = B->doutT = B->hwT = B->dguT = B->xgT = 0;    // (paths the pull mode never takes)
    B->total = off;
    return true;
}

}  // namespace mok

extern "C" {

size_t mok_ep_bwd_workspace_bytes(int n_ranks, int T_local, int H, int I, int I_shared, int E, int k) {
    BwdLayout B;
    return ep_bwd_layout(n_ranks, T_local, H, I, I_shared, E, k, &B) ? B.total : 0;
}

int mok_ep_expert_bwd(const mok_ep_bwd_args* a) {
    if (!a) return MOK_ERR_NULL;
    BwdLayout B;
    if (a->n_ranks < 1 || a->n_ranks > MOK_MAX_RANKS || a->rank < 0 || a->rank >= a->n_ranks) return MOK_ERR_SHAPE;
    if (!ep_bwd_layout(a->n_ranks, a->T_local, a->H, a->I, a->I_shared, a->E, a->k, &B)) return MOK_ERR_SHAPE;
    if ((a->I_shared > 0) != (a->W_shared_gate_up != nullptr) || (a->I_shared > 0) != (a->W_shared_down != nullptr))
        return MOK_ERR_SHAPE;
    if (a->config && (a->config->impl != MOK_IMPL_TCGEN05 || a->config->grid < 0 || a->config->precision != MOK_PRECISION_BF16 ||
                      (a->config->cta_group != 0 && a->config->cta_group != 1 && a->config->cta_group != 3)))
        return MOK_ERR_SHAPE;
    if (a->T_local == 0) return MOK_OK;
    if (!a->idx_all || !a->w_all || !a->W_gate_up || !a->W_down || !a->dxg || !a->pos || !a->dw_routes) return MOK_ERR_NULL;
    if (a->I_shared > 0 && !a->dx_shared) return MOK_ERR_NULL;
    for (int r = 0; r < a->n_ranks; ++r) {
        if (!a->x_peers[r] || !a->dout_peers[r]) return MOK_ERR_NULL;
        if (!aligned16(a->x_peers[r]) || !aligned16(a->dout_peers[r])) return MOK_ERR_ALIGN;
    }
    if (!aligned16(a->W_gate_up) || !aligned16(a->W_down) || !aligned16(a->W_shared_gate_up) || !aligned16(a->W_shared_down) ||
        !aligned16(a->dxg) || !aligned16(a->dx_shared) || !aligned16(a->dW_gate_up) || !aligned16(a->dW_down) ||
        !aligned16(a->dW_shared_gate_up) || !aligned16(a->dW_shared_down))
        return MOK_ERR_ALIGN;
    const bool want_w = a->dW_gate_up || a->dW_down || a->dW_shared_gate_up || a->dW_shared_down;
    if (want_w && (!a->dW_gate_up || !a->dW_down || (a->I_shared > 0 && (!a->dW_shared_gate_up || !a->dW_shared_down))))
        return MOK_ERR_NULL;
    const WsLayout& L = B.F;
    if (a->dxg_rows < L.Rpad) return MOK_ERR_WORKSPACE;
    if (!a->workspace || (reinterpret_cast<uintptr_t>(a->workspace) & 255u) || a->workspace_bytes < B.total)
        return MOK_ERR_WORKSPACE;

    cudaStream_t s = reinterpret_cast<cudaStream_t>(a->stream);
    char* ws = reinterpret_cast<char*>(a->workspace);
    WsHeader* hdr = reinterpret_cast<WsHeader*>(ws + L.header);
    cudaError_t e = cudaMemsetAsync(hdr, 0, sizeof(WsHeader), s);
    if (e != cudaSuccess) return cuda_fail(e);
    const int Lx = a->E / a->n_ranks, n = a->T_local * a->k;
    // Algorithm 1 for this rank's experts, as in the forward pass (same tables, same positions)
    e = launch_ep_schedule(a->idx_all, a->n_ranks, a->rank, n, a->k, a->T_local, Lx, TILE_M, L, ws, a->pos, nullptr, nullptr,
                           nullptr, nullptr, s);
    if (e != cudaSuccess) return cuda_fail(e);
    {
        const int total = a->n_ranks * n;
        int blocks = (total + 255) / 256;
        if (blocks > 148 * 8) blocks = 148 * 8;
        ep_row_route_kernel<<<blocks, 256, 0, s>>>(a->idx_all, a->pos, total, a->rank * Lx, Lx,
                                                   reinterpret_cast<int32_t*>(ws + B.row_route));
        if ((e = cudaGetLastError()) != cudaSuccess) return cuda_fail(e);
    }
    EpBwd ep;
    memset(&ep, 0, sizeof(ep));
    ep.n_ranks = a->n_ranks;
    ep.T_local = a->T_local;
    ep.routes_expected = n;
    for (int r = 0; r < a->n_ranks; ++r) {
        ep.x_peers[r] = reinterpret_cast<const __nv_bfloat16*>(a->x_peers[r]);
        ep.dout_peers[r] = reinterpret_cast<const __nv_bfloat16*>(a->dout_peers[r]);
    }
    ep.w_all = a->w_all;
    ep.dw_routes = a->dw_routes;
    ep.dxg = reinterpret_cast<__nv_bfloat16*>(a->dxg);
    ep.dx_shared = reinterpret_cast<__nv_bfloat16*>(a->dx_shared);
    mok_bwd_args b;
    memset(&b, 0, sizeof(b));
    b.x = a->x_peers[a->rank];
    b.dout = a->dout_peers[a->rank];
    b.W_gate_up = a->W_gate_up; b.W_down = a->W_down;
    b.W_shared_gate_up = a->W_shared_gate_up; b.W_shared_down = a->W_shared_down;
    b.T = a->T_local; b.H = a->H; b.I = a->I; b.I_shared = a->I_shared; b.E = Lx; b.k = a->k;
    b.dW_gate_up = a->dW_gate_up; b.dW_down = a->dW_down;
    b.dW_shared_gate_up = a->dW_shared_gate_up; b.dW_shared_down = a->dW_shared_down;
    b.workspace = a->workspace; b.workspace_bytes = a->workspace_bytes;
    b.config = a->config;
    b.stream = a->stream;
    return backward_chain(&b, B, L, &ep);
}

int mok_ep_bwd_combine(const mok_ep_bwd_combine_args* a) {
    if (!a) return MOK_ERR_NULL;
    if (a->n_ranks < 1 || a->n_ranks > MOK_MAX_RANKS || a->rank < 0 || a->rank >= a->n_ranks || a->T_local < 0 ||
        a->H <= 0 || (a->H % 8) || a->E < 1 || a->E % a->n_ranks || a->k < 1 || a->k > MAX_K || a->k > a->E)
        return MOK_ERR_SHAPE;
    if (a->T_local == 0) return MOK_OK;
    if (!a->topk_idx || !a->dx) return MOK_ERR_NULL;
    // dx: the forward's owner-side combine with unit weights over the serving ranks' dL/d(gathered x) rows
    mok_ep_combine_args c;
    memset(&c, 0, sizeof(c));
    c.rank = a->rank; c.n_ranks = a->n_ranks; c.T_local = a->T_local; c.H = a->H; c.E = a->E; c.k = a->k;
    c.topk_idx = a->topk_idx;
    c.topk_w = nullptr;                       // unit weights
    for (int r = 0; r < a->n_ranks; ++r) { c.y_peers[r] = a->dxg_peers[r]; c.pos_peers[r] = a->pos_peers[r]; }
    c.y_shared = a->dx_shared;
    c.out = a->dx;
    c.stream = a->stream;
    int rc = ep_combine_impl(&c, true);
    if (rc) return rc;
    if (a->dw) {
        EpDwArgs d;
        memset(&d, 0, sizeof(d));
        for (int r = 0; r < a->n_ranks; ++r) {
            if (!a->dw_peers[r]) return MOK_ERR_NULL;
            d.dw[r] = a->dw_peers[r];
        }
        d.idx = a->topk_idx;
        d.out = a->dw;
        d.n = a->T_local * a->k;
        d.Lx = a->E / a->n_ranks;
        d.route_base = a->rank * d.n;
        int blocks = (d.n + 255) / 256;
        if (blocks > 148 * 8) blocks = 148 * 8;
        ep_dw_kernel<<<blocks, 256, 0, reinterpret_cast<cudaStream_t>(a->stream)>>>(d);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return cuda_fail(e);
    }
    return MOK_OK;
}

}  // extern "C"
