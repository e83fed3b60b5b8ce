/*
 * mok.h -- C ABI of libmok: the fused Mixture-of-Experts layer forward pass on one B200 (sm_100a).
 *
 * The layer (paper, Section 2.1):
 *     MoE(x, s) = f_shared(x) + sum_{i in top-k} s_i / (sum_j s_j) * f_i(x),
 *     f_i(x)    = W_down_i ( silu(W_gate_i x) .* (W_up_i x) ).
 * One call runs, on the device and without any host synchronisation or count readback (Section 3.3):
 *   router projection and top-k with normalised weights (Section 2.1; Figure 1, right),
 *   dispatch schedule construction (Algorithm 1 with one rank: counts, offsets, stable permutation),
 *   the token gather in expert order ("pull dispatch", Section 3.1),
 *   the routed and shared SwiGLU expert FFNs as grouped bf16 GEMMs (Section 2.1),
 *   and the deterministic weighted combine back to token order ("push combine" + router-weighted sum,
 *   Sections 3.1 and 3.4 "Determinism").
 *
 * General rules for every entry point
 *   - Pointers are DEVICE pointers unless the argument is documented as HOST.  The caller owns every
 *     buffer; the library borrows it for the duration of the enqueued work and never frees it.
 *   - bf16 tensors are row-major with the last index contiguous; they must be 16-byte aligned and
 *     H, I, I_shared must be multiples of 8 (16-byte rows).
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = default stream).  Calls return
 *     as soon as the work is enqueued, unless stated otherwise.
 *   - Return value: MOK_OK (0) or a negative mok_status.  Nothing throws or exits.  Argument errors are
 *     detected before anything is launched.
 *   - Inputs must be finite; behaviour on NaN/Inf is unspecified.
 *   - Limits: 1 <= k <= 32, k <= E <= 512, T*k < 2^31 / 256.
 */
#ifndef MOK_H_
#define MOK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum mok_status {
    MOK_OK = 0,
    MOK_ERR_NULL = -1,       /* a required pointer is NULL */
    MOK_ERR_SHAPE = -2,      /* unsupported or inconsistent sizes */
    MOK_ERR_ALIGN = -3,      /* a tensor pointer is not 16-byte aligned */
    MOK_ERR_WORKSPACE = -4,  /* workspace missing, misaligned or too small */
    MOK_ERR_CUDA = -5,       /* a CUDA runtime/driver call failed; see mok_last_cuda_error() */
    MOK_ERR_TIMEOUT = -6,    /* device side: a bounded wait inside a kernel ran out (reported by mok_read_status) */
    MOK_ERR_SCHEDULE = -7,   /* device side: the schedule failed its consistency check */
    MOK_ERR_UNSUPPORTED = -8 /* the device is not an sm_100 part */
} mok_status;

/* Which grouped-GEMM kernel runs the expert FFNs. */
enum {
    MOK_IMPL_TCGEN05 = 0, /* warp-specialised persistent kernel: TMA -> smem ring -> tcgen05.mma -> TMEM (default) */
    MOK_IMPL_SIMT = 1,    /* plain shared-memory FMA kernel; slow; the on-device cross-check of the above */
    MOK_IMPL_TCGEN05_TN = 2 /* tcgen05 kernel with the tokens on the MMA's N side (expert padding 16 rows, not 128) */
};

#define MOK_MAX_HOST_CHUNKS 8
#define MOK_DEBUG_STARVE 2

/* Optional tuning / debugging knobs.  Zero-initialise for defaults. */
typedef struct mok_config {
    int32_t impl;         /* MOK_IMPL_* */
    int32_t grid;         /* persistent grid size override for the tcgen05 kernels (0 = number of SMs).  The
                             output bits do not depend on it (Section 3.4 "Determinism"). */
    int32_t router_impl;  /* 0 = default, 1 = fp32 FMA router, 2 = split-bf16 tensor-core router */
    int32_t profile;      /* != 0: record CUDA events around every stage of this call (see mok_profile_begin) */
    int32_t gather_mode;  /* token gather of the routed gate/up GEMM: 0 = choose by shape, 1 = fused into the GEMM's
                             operand loads (no expert-sorted copy of x), 2 = separate gather kernel + TMA loads */
    int32_t cta_group;    /* tcgen05 GEMMs: 0 = choose by shape, 1 = one CTA per 128-row tile, 2 = CTA pairs sharing a
                             256-row tile (cta_group::2; halves the weight traffic into each SM), 3 = one CTA per
                             256-row tile with two accumulators (same traffic saving, no cross-CTA signalling) */
    int32_t debug;        /* 1: the tcgen05 GEMMs accumulate wait-time counters (see mok_debug_counters).
                             MOK_DEBUG_STARVE: test hook for the bounded waits -- the gate/up GEMM's TMA producer
                             issues nothing and every wait gives up after 2 ms, so the call must end with
                             mok_read_status() == MOK_ERR_TIMEOUT and a usable context (output undefined) */
    int32_t host_chunks;  /* mok_moe_forward_host: token chunks whose copies overlap compute (0 = choose by T,
                             at most MOK_MAX_HOST_CHUNKS) */
} mok_config;

/*
 * Arguments of mok_moe_forward_ex.  Zero-initialise, then fill.  Shapes follow the paper's notation:
 * T tokens, H hidden size (D in the paper), I expert intermediate size, E routed experts, k routes/token.
 */
typedef struct mok_args {
    /* inputs */
    const void*  x;                 /* bf16 [T, H] */
    const float* W_router;          /* fp32 [E, H] */
    const float* router_bias;       /* fp32 [E] or NULL: logit[t,e] += bias[e] (enters selection and weights) */
    const void*  W_gate_up;         /* bf16 [E, 2I, H]: rows 0..I-1 = W_gate, rows I..2I-1 = W_up */
    const void*  W_down;            /* bf16 [E, H, I] */
    const void*  W_shared_gate_up;  /* bf16 [2*I_shared, H] or NULL */
    const void*  W_shared_down;     /* bf16 [H, I_shared]   or NULL */
    int32_t T, H, I, I_shared, E, k;
    /* output */
    void* out;                      /* bf16 [T, H] */
    /* scratch, caller-owned: >= mok_workspace_bytes(...) bytes, 256-byte aligned.  Its contents are
       undefined between calls; calls that share a workspace must not overlap on the device. */
    void*  workspace;
    size_t workspace_bytes;
    /* optional stage outputs (NULL = not wanted); written by the same enqueued work */
    int32_t* topk_idx;   /* [T, k]  selected experts, descending logit, ties to the lowest id */
    float*   topk_w;     /* [T, k]  normalised router weights (sum to 1 per token) */
    int32_t* counts;     /* [E]     routes per expert */
    int32_t* offsets;    /* [E+1]   exclusive prefix sum of counts (unpadded) */
    int32_t* perm;       /* [T*k]   route id (t*k+s) at dispatch-buffer position p: Algorithm 1's table for one rank */
    int32_t* inv_perm;   /* [T*k]   inverse of perm */
    const mok_config* config;       /* NULL = defaults */
    void* stream;
} mok_args;

/*
 * The MoE layer forward (Section 2.1 equation; Figure 1).  out[t,:] = f_shared(x[t]) + sum_s w[t,s] f_{idx[t,s]}(x[t]).
 * Scores are softmax over all E router logits, the k largest are selected (ties to the lowest expert id) and
 * renormalised.  I_shared == 0 <=> both shared pointers NULL.  T == 0 returns MOK_OK without launching.
 * Uses a library-owned per-device workspace that grows on demand with cudaMalloc (so the first call for a
 * new size is not capturable and not thread-safe); use mok_moe_forward_ex to supply your own.
 */
int mok_moe_forward(const void* x, const float* W_router,
                    const void* W_gate_up, const void* W_down,
                    const void* W_shared_gate_up, const void* W_shared_down,
                    int T, int H, int I, int I_shared, int E, int k,
                    void* out, void* stream);

/* Bytes of scratch mok_moe_forward_ex needs for these sizes (0 if the sizes are invalid). */
size_t mok_workspace_bytes(int T, int H, int I, int I_shared, int E, int k);

/* Same layer with a router bias, caller-owned workspace, stage outputs and knobs (see mok_args). */
int mok_moe_forward_ex(const mok_args* args);

/*
 * Same layer with the activations in HOST memory: x_host (bf16 [T,H]) is copied to the device, the layer
 * runs, and out_host (bf16 [T,H]) is copied back; the call returns after the result has arrived (it
 * synchronises `stream`).  Pinned host buffers make the copies asynchronous DMA.  Because each token's output
 * depends only on its own row of x, the batch is cut into token chunks (config.host_chunks) and the upload of the
 * next chunk and the download of the previous one run on two library-owned copy streams while a chunk computes;
 * the result bits do not depend on the number of chunks.  Stage outputs force a single chunk.  The first call on a
 * device creates the copy streams and events.  Weights, bias and
 * workspace stay DEVICE pointers as in mok_args; args->x and args->out are ignored.  The workspace must
 * have mok_workspace_bytes(...) + 2 * T*H*2 bytes (the staging copies of x and out live at its end).
 */
int mok_moe_forward_host(const mok_args* args, const void* x_host, void* out_host);

/*
 * Stage entry points (used by tests and profiling; each is the corresponding step of mok_moe_forward_ex).
 *   mok_route    : router projection + top-k + weights (Section 2.1)          -> topk_idx [T,k], topk_w [T,k]
 *   mok_schedule : Algorithm 1 for one rank from topk_idx [T*k]               -> counts, offsets, perm, inv_perm
 * `workspace` as for mok_moe_forward_ex (same size query).
 */
int mok_route(const void* x, const float* W_router, const float* router_bias, int T, int H, int E, int k,
              int32_t* topk_idx, float* topk_w, void* workspace, size_t workspace_bytes,
              const mok_config* config, void* stream);
int mok_schedule(const int32_t* topk_idx, int T, int E, int k,
                 int32_t* counts, int32_t* offsets, int32_t* perm, int32_t* inv_perm,
                 void* workspace, size_t workspace_bytes, void* stream);

/*
 * mok_schedule without a workspace and without any allocation.  The paper has no counterpart of this entry point;
 * it exists for callers that cannot allocate device memory where they need a schedule: serving loops that must not
 * take cudaMalloc's device-wide synchronisation, processes whose framework already owns all of HBM, plug-ins that
 * are handed only input and output buffers.  Inputs and outputs are as for mok_schedule (device pointers; any of the
 * four outputs may be NULL).  The scratch lives in a fixed 1.5 MiB array inside the library image: one copy per GPU
 * that loads the library, held until the process exits.
 *   - Limit: T*k <= MOK_NOALLOC_MAX_ROUTES (and E <= 512); larger sizes return MOK_ERR_SHAPE and launch nothing.
 *   - The first call on each device looks up the array's device address (a host-side set-up step); make that first
 *     call outside of any stream capture.  No call allocates or frees memory.
 *   - All calls on a device share the array and it keeps the previous call's contents (the words that must start at
 *     zero are cleared by every call): calls that overlap on the device race, so serialise them on one stream.
 */
#define MOK_NOALLOC_MAX_ROUTES 32768
int mok_schedule_noalloc(const int32_t* topk_idx, int T, int E, int k,
                         int32_t* counts, int32_t* offsets, int32_t* perm, int32_t* inv_perm, void* stream);

/*
 * Reads the device-side status word of a workspace after synchronising `stream` -- the only call besides
 * mok_moe_forward_host that blocks the host.  Returns MOK_OK, MOK_ERR_TIMEOUT or MOK_ERR_SCHEDULE
 * (or MOK_ERR_CUDA if the stream itself is in error).
 */
int mok_read_status(const void* workspace, void* stream);

/*
 * Per-stage device timing with CUDA events recorded on the call's stream (measurement aid; the paper reports
 * CUDA-side latencies, Section 4.1).  mok_profile_begin reserves event sets for up to max_calls forward calls;
 * every later forward call whose config has profile != 0 fills the next set without synchronising.
 * mok_profile_end synchronises on the last recorded event, writes ms[call][stage] (row-major,
 * MOK_STAGE_COUNT floats per call) for the calls recorded (at most max_calls_out rows), stores their number in
 * *n_calls and releases the events.  Not thread-safe.
 */
enum {
    MOK_STAGE_ROUTER = 0, MOK_STAGE_SCHEDULE, MOK_STAGE_GATHER, MOK_STAGE_GEMM1, MOK_STAGE_GEMM2,
    MOK_STAGE_SHARED_GEMM1, MOK_STAGE_SHARED_GEMM2, MOK_STAGE_COMBINE, MOK_STAGE_COUNT
};
int mok_profile_begin(int max_calls);
int mok_profile_end(float* ms, int max_calls_out, int* n_calls);

/*
 * Wait-time counters of the tcgen05 GEMM kernels of the last forward call that ran with config.debug != 0
 * (measurement aid; Section 3 cost model: T_sync).  Synchronises `stream`, then writes 4 x 8 values: slot 1 = routed
 * gate/up GEMM, 2 = routed down GEMM, 3 = shared GEMMs; per slot, SM cycles summed over CTAs: MMA issuer waiting for
 * operands, for the peer CTA's operands, for a free accumulator; MMA issuer total; k-blocks issued; TMA producer
 * waiting for a free stage; epilogue waiting for an accumulator; epilogue total.
 */
int mok_debug_counters(const void* workspace, void* stream, unsigned long long* out);

/* Number of kernels one mok_moe_forward_ex call enqueues for these arguments (the memset of the workspace header
   is not counted); 0 on bad sizes. */
int mok_launch_count(int T, int H, int I, int I_shared, int E, int k, const mok_config* config);

int mok_last_cuda_error(void);          /* cudaError_t of the most recent failed CUDA call on this thread */
const char* mok_status_string(int status);
int mok_version(void);                  /* major*10000 + minor*100 + patch */

#ifdef __cplusplus
}
#endif
#endif /* MOK_H_ */
