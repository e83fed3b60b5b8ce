// Router projection on the tensor cores without giving up fp32 router weights (paper, Section 2.1; Figure 1
// right: the GPU-side router projection and top-k that precede the expert kernels).
//
// A plain bf16 GEMM would round W_r to 8 mantissa bits and move logits by ~2e-3, which changes the top-k of tokens
// that are nowhere near a tie.  Instead every fp32 weight is split exactly into three bf16 terms,
//     W_r = hi + mid + lo,   hi = bf16(W_r), mid = bf16(W_r - hi), lo = bf16(W_r - hi - mid),
// x is bf16 already, so all products are exact in fp32 and the tensor cores only add rounding in the fp32
// accumulation.  Three kernels:
//   1. router_split_kernel  W_r [E,H] fp32 -> [ldl, H] bf16 rows: hi (0..E-1), mid (E..2E-1), lo (2E..3E-1), zero pad
//   2. the tcgen05 GEMM     x [T,H] . split^T -> partial logits fp32 [T, ldl]
//   3. router_topk_kernel   logit = (lo + mid) + hi + bias, warp-shuffle top-k and softmax weights; tokens with a
//                           pair of candidates closer than the accumulation error are re-decided with exact FMAs
#include "mok_internal.cuh"
#include "router_common.cuh"

namespace mok {

__global__ void __launch_bounds__(256)
router_split_kernel(const float* __restrict__ Wr, int E, int H, int ldl, __nv_bfloat16* __restrict__ out) {
    const size_t n = (size_t)ldl * H;
    for (size_t i = (size_t)blockIdx.x * 256 + threadIdx.x; i < n; i += (size_t)gridDim.x * 256) {
        const int row = (int)(i / H), h = (int)(i - (size_t)row * H);
        float v = 0.f;
        if (row < 3 * E) {
            const int part = row / E, e = row - part * E;
            const float wv = Wr[(size_t)e * H + h];
            const float hi = __bfloat162float(__float2bfloat16_rn(wv));
            const float r1 = wv - hi;                                   // exact
            const float mid = __bfloat162float(__float2bfloat16_rn(r1));
            const float r2 = r1 - mid;                                  // exact
            v = (part == 0) ? hi : (part == 1) ? mid : r2;
        }
        out[i] = __float2bfloat16_rn(v);
    }
}

// Exact (fp32 FMA) logits of one token against up to four experts at once, computed by a whole warp: lanes stride
// over h in 16-byte pieces of x (read once for the four experts), then a shuffle tree per expert.  Four independent
// weight streams keep enough loads in flight to hide the L2 latency.  Error ~1e-7 relative, far below the near-tie
// threshold.
__device__ __forceinline__ void warp_exact_logits4(const __nv_bfloat16* __restrict__ xrow, const float* __restrict__ Wr,
                                                   const int (&e)[4], int n, int H, int lane, float (&out)[4]) {
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    const float* wrow[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) wrow[c] = Wr + (size_t)e[c < n ? c : 0] * H;
    for (int h = lane * 8; h < H; h += 256) {
        const uint4 raw = *reinterpret_cast<const uint4*>(xrow + h);
        const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&raw);
        const float2 x0 = __bfloat1622float2(p[0]), x1 = __bfloat1622float2(p[1]);
        const float2 x2 = __bfloat1622float2(p[2]), x3 = __bfloat1622float2(p[3]);
        float4 w0[4], w1[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            w0[c] = *reinterpret_cast<const float4*>(wrow[c] + h);
            w1[c] = *reinterpret_cast<const float4*>(wrow[c] + h + 4);
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            float a = acc[c];
            a = fmaf(x0.x, w0[c].x, a); a = fmaf(x0.y, w0[c].y, a);
            a = fmaf(x1.x, w0[c].z, a); a = fmaf(x1.y, w0[c].w, a);
            a = fmaf(x2.x, w1[c].x, a); a = fmaf(x2.y, w1[c].y, a);
            a = fmaf(x3.x, w1[c].z, a); a = fmaf(x3.y, w1[c].w, a);
            acc[c] = a;
        }
    }
#pragma unroll
    for (int c = 0; c < 4; ++c) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], off);
        out[c] = acc[c];
    }
}

// Monotone map from float to unsigned: a > b  <=>  key(a) > key(b) (finite inputs).
__device__ __forceinline__ unsigned float_key(float v) {
    const unsigned u = __float_as_uint(v);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Selection with the logits in registers: lane l holds experts l, l+32, ... (VPL per lane).  One round = every lane's
// best remaining value, a hardware warp max of the keys (redux.sync), and a warp min of the expert ids that attain it
// (ties go to the lowest id): two reductions instead of a ten-shuffle tree.
template <int VPL>
__device__ __forceinline__ void reg_select(float (&v)[VPL], int lane, int s_begin, int s_end, float& slot_v, int& slot_e) {
    for (int s = s_begin; s < s_end; ++s) {
        float bv = v[0];
        int bj = 0;
#pragma unroll
        for (int j = 1; j < VPL; ++j)
            if (v[j] > bv) { bv = v[j]; bj = j; }             // strict '>' keeps the lowest id on ties inside a lane
        const unsigned key = float_key(bv);
        const unsigned kmax = __reduce_max_sync(0xffffffffu, key);
        const int e_mine = (key == kmax) ? lane + 32 * bj : 0x7fffffff;
        const int e_win = __reduce_min_sync(0xffffffffu, e_mine);
        if (e_mine == e_win) {
#pragma unroll
            for (int j = 0; j < VPL; ++j)
                if (j == bj) v[j] = -FLT_MAX;                    // taken
        }
        const float v_win = __shfl_sync(0xffffffffu, bv, e_win & 31);
        if (lane == s) { slot_v = v_win; slot_e = e_win; }
    }
}

// The tensor cores add the 16 products of one MMA step to the fp32 accumulator with truncation, so the logit
// of a long dot product carries a small bias that grows with H (measured on B200: up to 4.5e-5 at H = 7168,
// against an fp64 evaluation).  That is harmless for the weights but could reorder two logits that are closer than
// the error.  So: tokens whose top-(k+1) tensor-core logits contain an adjacent pair closer than
//     guard = H * 2^-26 * (1 + max|logit|)      (four times the modelled bound (H/16) * 2^-24 * |acc|)
// get the logits of their top-(k+4) candidates recomputed with plain fp32 FMAs and are selected again.
template <int VPL>
__global__ void __launch_bounds__(256)
router_topk_kernel(const float* __restrict__ part, const float* __restrict__ bias,
                   const __nv_bfloat16* __restrict__ x, const float* __restrict__ Wr,
                   int T, int H, int E, int k, int ldl, int32_t* __restrict__ idx, float* __restrict__ w) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_check = (k + 1 < E) ? k + 1 : E;        // slots compared pairwise
    int n_cand = (k + 4 < E) ? k + 4 : E;               // candidates recomputed when a pair is too close
    if (n_cand > 32) n_cand = 32;
    const float guard_scale = (float)H * 1.4901161e-8f; // H * 2^-26
    for (int t = blockIdx.x * 8 + warp; t < T; t += gridDim.x * 8) {
        const float* row = part + (size_t)t * ldl;
        float orig[VPL], v[VPL];
#pragma unroll
        for (int j = 0; j < VPL; ++j) {
            const int e = lane + 32 * j;
            float val = -FLT_MAX;
            if (e < E) {
                val = (row[2 * E + e] + row[E + e]) + row[e];      // smallest terms first
                if (bias) val += bias[e];
            }
            orig[j] = val;
            v[j] = val;
        }
        TopkState st = {0u, 0.f, 0};
        reg_select<VPL>(v, lane, 0, n_check, st.v, st.e);
        const float next_v = __shfl_down_sync(0xffffffffu, st.v, 1);
        float amax = (lane < n_check) ? fabsf(st.v) : 0.f;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, off));
        const bool close = (lane + 1 < n_check) && (st.v - next_v < guard_scale * (1.f + amax));
        if (__any_sync(0xffffffffu, close)) {
            reg_select<VPL>(v, lane, n_check, n_cand, st.v, st.e);
            for (int c0 = 0; c0 < n_cand; c0 += 4) {
                int e[4];
                float ex[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) e[c] = __shfl_sync(0xffffffffu, st.e, (c0 + c < n_cand) ? c0 + c : c0);
                const int n = (n_cand - c0 < 4) ? n_cand - c0 : 4;
                warp_exact_logits4(x + (size_t)t * H, Wr, e, n, H, lane, ex);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    if (c < n && (e[c] & 31) == lane) {
                        const float val = ex[c] + (bias ? bias[e[c]] : 0.f);
#pragma unroll
                        for (int j = 0; j < VPL; ++j)
                            if (j == (e[c] >> 5)) orig[j] = val;
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < VPL; ++j) v[j] = orig[j];
            reg_select<VPL>(v, lane, 0, k, st.v, st.e);
        }
        warp_write_topk(st, k, lane, idx + (size_t)t * k, w + (size_t)t * k);
    }
}

cudaError_t launch_router_tc(const __nv_bfloat16* x, const float* Wr, const float* bias, int T, int H, int E, int k,
                             const WsLayout& L, char* ws, WsHeader* hdr, int grid, int tile_m, int variant, int32_t* idx,
                             float* w, cudaStream_t s) {
    const int ldl = (3 * E + 7) / 8 * 8;
    __nv_bfloat16* split = reinterpret_cast<__nv_bfloat16*>(ws + L.wr_split);
    float* part = reinterpret_cast<float*>(ws + L.logits);
    size_t n = (size_t)ldl * H;
    int blocks = (int)((n + 255) / 256);
    if (blocks > 148 * 8) blocks = 148 * 8;
    router_split_kernel<<<blocks, 256, 0, s>>>(Wr, E, H, ldl, split);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    GemmArgs g = {};
    g.A = x;
    g.B = split;
    g.C = part;
    g.K = H; g.N = ldl; g.E = 1; g.ldc = ldl;
    g.rows_pad = L.Tpad; g.a_rows = T; g.dense_rows = T;
    g.max_mt = L.Tpad / TILE_M;
    g.tile_m = tile_m;
    g.dbg_slot = -1;
    g.header = hdr;
    e = variant == 2 ? launch_gemm_tn(g, EPI_F32, grid, s)
        : variant == 3 ? launch_gemm_m2(g, EPI_F32, grid, s) : launch_gemm_tc(g, EPI_F32, grid, s);
    if (e != cudaSuccess) return e;
    int tblocks = (T + 7) / 8;
    if (tblocks > 148 * 16) tblocks = 148 * 16;
    const int vpl = (E + 31) / 32;
    if (vpl <= 1) router_topk_kernel<1><<<tblocks, 256, 0, s>>>(part, bias, x, Wr, T, H, E, k, ldl, idx, w);
    else if (vpl <= 2) router_topk_kernel<2><<<tblocks, 256, 0, s>>>(part, bias, x, Wr, T, H, E, k, ldl, idx, w);
    else if (vpl <= 4) router_topk_kernel<4><<<tblocks, 256, 0, s>>>(part, bias, x, Wr, T, H, E, k, ldl, idx, w);
    else if (vpl <= 8) router_topk_kernel<8><<<tblocks, 256, 0, s>>>(part, bias, x, Wr, T, H, E, k, ldl, idx, w);
    else router_topk_kernel<16><<<tblocks, 256, 0, s>>>(part, bias, x, Wr, T, H, E, k, ldl, idx, w);
    return cudaGetLastError();
}

}  // namespace mok
