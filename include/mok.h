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

enum { MOK_PRECISION_BF16 = 0, MOK_PRECISION_MXFP8 = 1 };

#define MOK_MAX_HOST_CHUNKS 8
#define MOK_DEBUG_STARVE 2
#define MOK_DEBUG_NO_ARRIVALS 3

/* Optional tuning / debugging knobs.  Zero-initialise for defaults. */
typedef struct mok_config {
    int32_t impl;         /* MOK_IMPL_* */
    int32_t grid;         /* persistent grid size override for the tcgen05 kernels (0 = number of SMs).  The
                             output bits do not depend on it (Section 3.4 "Determinism"). */
    int32_t router_impl;  /* 0 = default (split-bf16 tensor-core router; projection and top-k in one kernel for up to
                             160 experts), 1 = fp32 FMA router, 2 = split-bf16 tensor-core router as three kernels
                             (split, GEMM, top-k); 0 and 2 give the same bits */
    int32_t profile;      /* != 0: record CUDA events around every stage of this call (see mok_profile_begin) */
    int32_t gather_mode;  /* token gather of the routed gate/up GEMM: 0 = choose by shape, 1 = fused into the GEMM's
                             operand loads (no expert-sorted copy of x), 2 = separate gather kernel + TMA loads */
    int32_t cta_group;    /* tcgen05 GEMMs: 0 = choose by shape, 1 = one CTA per 128-row tile, 2 = CTA pairs sharing a
                             256-row tile (cta_group::2; halves the weight traffic into each SM), 3 = one CTA per
                             256-row tile with two accumulators (same traffic saving, no cross-CTA signalling) */
    int32_t debug;        /* 1: the tcgen05 GEMMs accumulate wait-time counters (see mok_debug_counters).
                             MOK_DEBUG_STARVE: test hook for the bounded waits -- the gate/up GEMM's TMA producer
                             issues nothing and every wait gives up after 2 ms, so the call must end with
                             mok_read_status() == MOK_ERR_TIMEOUT and a usable context (output undefined).
                             MOK_DEBUG_NO_ARRIVALS: the same for the completion counters of the one-launch expert FFN
                             that gate a ring slot's reuse (h_ring_tiles) and the in-launch combine (fused_ffn = 3):
                             nobody arrives on them, so those waits run out */
    int32_t host_chunks;  /* mok_moe_forward_host: token chunks whose copies overlap compute (0 = choose by T,
                             at most MOK_MAX_HOST_CHUNKS) */
    int32_t precision;    /* MOK_PRECISION_BF16 (0, default) or MOK_PRECISION_MXFP8: routed experts on MXFP8 operands
                             (Section 3.4 "MXFP8 Support"); needs the pre-quantised weights in mok_args and a workspace
                             of mok_mx_workspace_bytes(...) */
    int32_t tile_sched;   /* routed expert GEMMs of the forward pass (256-row-tile kernel): 0 = persistent grid, tile L on
                             CTA L mod grid; 1 = one CTA per tile, running CTAs steal the tiles of CTAs that have not
                             started through cluster launch control (Section 3.4 "Cluster Launch Control": hardware
                             work stealing).  The hardware refuses the request while work of a higher stream priority
                             waits for an SM; the CTA then leaves and the tiles nobody stole start as CTAs of their own
                             afterwards, so such work gets onto the SMs at the next tile boundary instead of at the end
                             of the kernel.  Same bits either way.  With the one-launch expert FFN (fused_ffn): 1 = dynamic
                             draw of list positions, 2 = static stride. */
    int32_t macrobatch_tokens; /* mok_moe_forward_ex: > 0 and < T: the tokens pass through the workspace in macrobatches of
                             this many tokens, one after the other (Section 3.3: a fixed-size buffer through which the
                             tokens cycle, instead of buffers sized for the whole batch).  The workspace then only needs
                             mok_workspace_bytes(macrobatch_tokens, ...); every macrobatch streams the expert weights
                             again.  Same bits as the single pass; counts / offsets / perm / inv_perm (tables of ONE
                             schedule) cannot be returned: MOK_ERR_UNSUPPORTED. */
    int32_t fused_ffn;    /* routed experts, bf16: 1 = gate/up GEMM and down GEMM as two launches, 0 = choose (the one launch
                             for large expert matrices -- an expert's weights of either GEMM at least 12 MB, two to
                             eight row tiles per expert; else the two launches),
                             2 = ONE persistent launch over a list of gate/up tiles and down tiles; a down tile runs
                             once a per-row-tile completion counter, advanced by the gate/up epilogues, shows that its
                             rows of the gated activation exist (Section 3.2: megakernel, GPU-local synchronisation
                             instead of kernel boundaries).  3 = as 2, and the combine runs at the end of the same launch:
                             the shared expert is then computed first, every epilogue warp reports its last store on a
                             grid-wide counter, waits (bounded) for all of them and combines its share of the tokens in
                             the slot order of the separate combine kernel.  Same bits in every mode. */
    int32_t fused_window; /* fused_ffn: list positions between a row group's gate/up tiles and its down tiles (0 = a
                             default of two to eight grids' worth of tiles; -1 = none: directly behind them, which makes
                             every down tile wait -- a test setting).  The list is walked with stride grid and
                             synchronised tile starts where experts have three or more row tiles on average, else
                             handed out dynamically (each CTA draws the next position from a global counter);
                             tile_sched = 1 / 2 force the draw / the stride. */
    int32_t gang_sync;    /* 256-row-tile GEMM kernel: the row tiles of an expert that use the same weight tile start that
                             tile together (a counter per such gang, bounded wait, cooperative launch), so that the weight
                             tile is read from DRAM once and shared through L2 instead of once per row tile.
                             0 = where it pays (large expert matrices, fewer than eight row tiles per expert), 1 = never,
                             2 = always (grids of fewer than eight CTAs excepted).  Same bits. */
    int32_t serial_launches; /* 0 = the kernels of a forward call are launched with programmatic stream serialization (a
                             kernel's CTAs are scheduled while its predecessor still runs; every kernel waits for its
                             predecessors' completion before it touches their data), 1 = plain launches.  Same bits. */
    int32_t h_ring_tiles; /* 0 = the gated activation h has a row for every padded route.  > 0: h is a RING of that many
                             256-row slots (at least MOK_H_RING_MIN_TILES) that the row tiles in flight reuse (Section 3.3:
                             fixed-size buffers; Section 3.2: the intermediate is consumed depth-first and stays in the
                             caches).  Only the one-launch expert FFN can do that (it is then used whatever fused_ffn says;
                             MOK_ERR_UNSUPPORTED where it cannot run: MXFP8, impl != 0, cta_group 1 / 2, a separate gather
                             kernel): a gate/up tile stores into its slot once every down tile of the slot's previous
                             rows has loaded them (completion counters, bounded waits); the distance between a row
                             group's gate/up and down tiles is cut to the ring size minus 16 tiles.  The workspace is
                             then the smaller one of mok_workspace_bytes_ring (no h rows beyond the ring, no gathered
                             copy of x).  Same bits. */
    int32_t shared_overlap; /* shared expert: 2 = its two GEMMs run on a library-owned second stream on 16 SMs beside the
                             router, the schedule and the routed experts (forked from and joined to `stream` by events,
                             before the combine; the routed kernels then take the other SMs); 1 = in line, after the
                             routed experts; 0 = beside them for small layers only (at most 160 routed rows per expert
                             and 64 MB of expert weights), whose kernels are bound by launch and fill latency rather
                             than by DRAM or the tensor cores (Section 3.4 "Shared Expert").  Same bits.  The second
                             stream and its two events exist once per device: host threads that call the library
                             concurrently on one device must set 1. */
    int32_t comm_ctas;    /* one-launch expert FFN (used whatever fused_ffn says; MOK_ERR_UNSUPPORTED where it cannot run, or
                             with h_ring_tiles): that many CTAs of the grid are COMMUNICATION CTAs (Section 3.4
                             "Computation-Communication SM Tuning"): they do no tiles but copy the token rows of one row
                             tile after the other -- from x, under expert parallelism from the owners' buffers -- into
                             a ring of 24 staging slots, from which the gate/up tiles then load their A operand by
                             TMA; completion counters (bounded waits) order staging, use and reuse of a slot.  The
                             latency of a pull is then taken by CTAs that do nothing else, a row tile ahead of its
                             use, instead of by the gather warps of the computing CTAs.  0 = none: the gather warps
                             pull.  Same bits. */
} mok_config;
#define MOK_H_RING_MIN_TILES 24

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
    /* MXFP8 mode only (config->precision == MOK_PRECISION_MXFP8): the routed weights pre-quantised by
       mok_mx_quantize_weights; the bf16 W_gate_up / W_down are then not read and may be NULL */
    const void* W_gate_up_codes;    /* E4M3 [E, 2I, H] */
    const void* W_gate_up_scales;   /* E8M0 scale atoms of the 2E matrices [I, H] */
    const void* W_down_codes;       /* E4M3 [E, H, I] */
    const void* W_down_scales;      /* E8M0 scale atoms of the E matrices [H, I] */
    /* optional: W_router split ahead of time by mok_router_prepare (same E, H, k and config.router_impl as this call);
       NULL = the split is redone inside every call.  W_router is still needed (near-ties are re-decided in fp32). */
    const void* W_router_split;
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
/* The same for calls with config.h_ring_tiles = h_ring_tiles > 0 (Section 3.3: buffers of fixed size): the gated
 * activation takes min(h_ring_tiles * 256, padded routes) rows and the gathered copy of x does not exist.  0 if the sizes
 * are invalid or h_ring_tiles < MOK_H_RING_MIN_TILES.  A workspace of mok_workspace_bytes is always large enough too. */
size_t mok_workspace_bytes_ring(int T, int H, int I, int I_shared, int E, int k, int h_ring_tiles);

/* Same layer with a router bias, caller-owned workspace, stage outputs and knobs (see mok_args). */
int mok_moe_forward_ex(const mok_args* args);

/*
 * Router weights prepared once (Section 2.1 router projection; Figure 1, right: the routing step precedes the expert
 * kernels on every call, but W_router is a weight).  The tensor-core router multiplies x by an exact three-way bf16
 * split of the fp32 W_router (hi + mid + lo); mok_router_prepare writes that split for the given E, H, k and
 * config->router_impl into `out` (device, 16-byte aligned, at least mok_router_prepared_bytes(E, H) bytes; the
 * caller owns it), and mok_args.W_router_split hands it to later forward calls, which then skip their own split
 * kernel.  Same result bits either way.  MOK_ERR_UNSUPPORTED when the configuration routes with the fp32-FMA kernel
 * (config->router_impl = 1, config->impl = MOK_IMPL_SIMT with router_impl = 0, or k > 28), which has no split.
 */
size_t mok_router_prepared_bytes(int E, int H);
int mok_router_prepare(const float* W_router, int E, int H, int k, const mok_config* config, void* out, size_t out_bytes,
                       void* stream);

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
 * The host-buffer call without the wait at its end, for a stream of batches (this entry point and the wait below are
 * this library's own; the paper measures device-side latency only, Section 4.1).  It enqueues: upload of x_host on the
 * library's input copy stream, the layer on args->stream, download into out_host on the library's output copy stream,
 * chained by events, and returns at once.  Two staging slots at the end of the workspace are used in turn, so
 * consecutive submissions overlap: while batch i computes, batch i+1 uploads and batch i-1 downloads (PCIe is full
 * duplex).  A slot's copy of x is reused once the layer that read it has run, its copy of out once that result has left
 * the device (event waits on the device, not on the host).  The result bits equal those of mok_moe_forward_ex.
 *   - x_host must stay unchanged, and out_host must not be read, until mok_host_wait() has returned; use a
 *     different out_host for submissions that are in flight together.  Pinned buffers are needed for the overlap.
 *   - The workspace must have mok_workspace_bytes(...) + 4 * T*H*2 bytes (each slot: x and out, 256-byte aligned)
 *     and must serve these submissions only while any is in flight; all submissions in flight use the same T and H.
 *   - Stage outputs are not supported here (MOK_ERR_UNSUPPORTED); the other errors are those of mok_moe_forward_ex,
 *     reported before anything is enqueued.  Device-side failures show in mok_read_status after the wait: the status
 *     word is cleared by the first submission after a mok_host_wait only, so it covers every submission since then.
 * mok_host_wait blocks until every submission made so far on the current device has delivered its result.
 */
int mok_moe_forward_host_async(const mok_args* args, const void* x_host, void* out_host);
int mok_host_wait(void);

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
 * Expert parallelism over n_ranks GPUs of one NVLink domain (Sections 2.1 and 3.1-3.3; Algorithm 1 with R source
 * ranks).  Rank c holds the L = E / n_ranks experts [cL, (c+1)L) and T_local tokens.  One layer is, on every rank:
 *   1. mok_route on the rank's own tokens                                  -> topk_idx, topk_w      (local)
 *   2. an all-gather of topk_idx over the ranks (the caller's collective; Section 3.1: every rank learns all routes)
 *   3. mok_ep_expert_ffn: Algorithm 1 for this rank from the gathered routes (M, S, Phi; no host readback), then
 *      the routed gate/up GEMM whose gather warps PULL each scheduled row straight from its source rank's token
 *      buffer x_peers[src_rank] into shared memory ("pull dispatch": plain 16-byte asynchronous copies over NVLink,
 *      never a multicast load), SwiGLU, and the down GEMM, which leaves this rank's expert outputs in y in schedule
 *      order; pos tells every token owner where its routes' rows sit in this rank's y
 *   4. a barrier over the ranks (the caller's; every rank's y and pos must be complete before any rank combines)
 *   5. mok_ep_combine: each token owner reads its k rows from the serving ranks' y buffers and reduces them, with the
 *      shared expert's output, in slot order in fp32 -- fixed order, no atomics, bitwise reproducible (Section 3.4).
 *      The paper has the expert's rank push rows into a buffer of the owner, which the owner then reduces; here the
 *      owner pulls the same rows, so each row still crosses NVLink once and the only cross-rank signal is step 4.
 * x_peers / y_peers / pos_peers hold device pointers valid in the calling process: the rank's own buffers and the
 * peers' buffers mapped into it (symmetric memory or IPC handles; the caller's plumbing).  On one GPU the same entry
 * points serve any number of emulated ranks, since a local pointer is a valid peer pointer.
 * Limits: n_ranks <= MOK_MAX_RANKS, E a multiple of n_ranks, and the sizes of mok_moe_forward_ex with
 * T = n_ranks * T_local.  The dispatch buffers are sized for the worst case (every route of every rank served by this
 * rank): mok_ep_y_rows rows.
 */
#define MOK_MAX_RANKS 16
typedef struct mok_ep_args {
    int32_t rank, n_ranks;
    int32_t T_local, H, I, I_shared, E, k;
    const void* x_peers[MOK_MAX_RANKS];  /* bf16 [T_local, H] of every rank; x_peers[rank] is this rank's own */
    const int32_t* idx_all;              /* int32 [n_ranks, T_local*k]: gathered top-k expert ids, rank-major */
    const void* W_gate_up;               /* bf16 [L, 2I, H]: this rank's experts */
    const void* W_down;                  /* bf16 [L, H, I] */
    const void* W_shared_gate_up;        /* bf16 [2*I_shared, H] or NULL: shared expert, run on the rank's own tokens */
    const void* W_shared_down;           /* bf16 [H, I_shared] or NULL */
    void* y;                             /* out: bf16 [y_rows, H] expert outputs in schedule order (peers read it) */
    int64_t y_rows;                      /* rows allocated for y: at least mok_ep_y_rows(...) */
    int32_t* pos;                        /* out: int32 [n_ranks*T_local*k]: row of y of every route this rank serves;
                                            entries of routes served elsewhere are left untouched (peers read it) */
    void* y_shared;                      /* out: bf16 [T_local rounded up to a multiple of 256, H]: the shared expert's
                                            output for the rank's own tokens; required when I_shared > 0 */
    void* workspace;                     /* mok_ep_workspace_bytes(...) bytes, 256-byte aligned */
    size_t workspace_bytes;
    /* optional outputs of Algorithm 1 (any may be NULL) */
    int32_t* M;                          /* int32 [n_ranks, L]: routes from source rank r to local expert l */
    int32_t* S;                          /* int32 [L+1]: exclusive prefix sums of the per-expert totals */
    int32_t* phi_rank;                   /* int32 [n_ranks*T_local*k]: source rank of schedule row p < S[L] */
    int32_t* phi_index;                  /* int32 [n_ranks*T_local*k]: source route index (token*k + slot) of row p */
    int32_t schedule_only;               /* non-zero: stop after Algorithm 1 (y untouched; pos and the outputs written) */
    const mok_config* config;            /* grid, cta_group 0/1/3, precision; impl must be MOK_IMPL_TCGEN05 */
    void* stream;
    /* MXFP8 mode only (config->precision == MOK_PRECISION_MXFP8, Section 3.4; workspace of
       mok_ep_mx_workspace_bytes): every rank quantises its own token rows with mok_mx_quantize_rows into buffers the
       peers can read, and this rank's routed weights come pre-quantised; x_peers is then only used for the shared
       expert (x_peers[rank]) and W_gate_up / W_down may be NULL */
    const void* x_codes_peers[MOK_MAX_RANKS];   /* E4M3 [T_local, H] of every rank */
    const void* x_scales_peers[MOK_MAX_RANKS];  /* E8M0 [T_local, 4 * ceil(H / 128)] of every rank */
    const void* W_gate_up_codes;         /* E4M3 [L, 2I, H] */
    const void* W_gate_up_scales;        /* scale atoms of the 2L matrices [I, H] (mok_mx_quantize_weights) */
    const void* W_down_codes;            /* E4M3 [L, H, I] */
    const void* W_down_scales;           /* scale atoms of the L matrices [H, I] */
} mok_ep_args;

typedef struct mok_ep_combine_args {
    int32_t rank, n_ranks;
    int32_t T_local, H, E, k;
    const int32_t* topk_idx;             /* int32 [T_local, k]: this rank's routes */
    const float* topk_w;                 /* fp32 [T_local, k] */
    const void* y_peers[MOK_MAX_RANKS];  /* every rank's y */
    const int32_t* pos_peers[MOK_MAX_RANKS]; /* every rank's pos */
    const void* y_shared;                /* this rank's y_shared from mok_ep_expert_ffn, or NULL: no shared term */
    void* out;                           /* bf16 [T_local, H] */
    void* stream;
} mok_ep_combine_args;

size_t mok_ep_workspace_bytes(int n_ranks, int T_local, int H, int I, int I_shared, int E, int k);
size_t mok_ep_mx_workspace_bytes(int n_ranks, int T_local, int H, int I, int I_shared, int E, int k);
long long mok_ep_y_rows(int n_ranks, int T_local, int E, int k);
int mok_ep_expert_ffn(const mok_ep_args* args);
int mok_ep_combine(const mok_ep_combine_args* args);

/*
 * MXFP8 mode of the routed experts (Section 3.4 "MXFP8 Support"; the shared expert, the router and the combine stay
 * as in bf16 mode).  Format: the microscaling format the section cites -- along the contraction dimension every 32
 * consecutive elements share the scale 2^(floor(log2(amax)) - 8), stored as one E8M0 byte (exponent + 127), and hold
 * v / scale rounded to nearest-even on the FP8 E4M3 grid, magnitudes above 448 clamped; an all-zero block has scale
 * byte 0.  H and I must be multiples of 32.
 *   mok_mx_quantize_weights : the weight pre-quantisation kernel.  W is bf16 [groups, rows, K] (W_gate_up: groups = 2E
 *       matrices of [I, H], i.e. each expert's gate then up projection; W_down: groups = E matrices of [H, I]);
 *       codes receives groups*rows*K bytes in the same order; scales receives mok_mx_scale_bytes(groups, rows, K)
 *       bytes in the layout the block-scaled tensor-core instruction loads: for each (group, 128-row block,
 *       128-element k-group) 512 bytes with the scale of row r, 32-element block j of the k-group at
 *       (r % 32) * 16 + ((r % 128) / 32) * 4 + j; entries outside the tensor hold 127 (= 1.0).
 *   mok_mx_quantize_rows    : the activation quantiser as a stage entry point (tests): x bf16 [rows, K] -> codes
 *       [rows, K] and row-major scales [rows, 4 * ceil(K / 128)] (entries past K / 32 hold 127).
 *   The forward pass in this mode quantises the token rows once (a pre-pass instead of re-quantising every row k
 *   times inside the dispatch), the gate/up GEMM pulls codes and scales of its rows, its epilogue quantises the gated
 *   activation as it is produced, and the down GEMM writes bf16 for the fp32 combine.
 */
size_t mok_mx_scale_bytes(int groups, int rows, int K);
int mok_mx_quantize_weights(const void* W, int groups, int rows, int K, void* codes, void* scales, void* stream);
int mok_mx_quantize_rows(const void* x, int rows, int K, void* codes, void* scales, void* stream);
size_t mok_mx_workspace_bytes(int T, int H, int I, int I_shared, int E, int k);

/*
 * Backward pass of the layer (Section 3.4: the router-weight gradient is computed inside the backward chain and the
 * activations are recomputed rather than stored; Section 4.1: dgrad + wgrad).  The paper prints no formulas: this is the chain rule of the Section 2.1 definition.
 * Inputs: the forward pass's inputs, its routing (topk_idx, topk_w as returned by mok_moe_forward_ex -- the only
 * thing that has to be kept from the forward pass; every activation is recomputed) and dout = dL/dout.
 * Outputs: dx = dL/dx through the experts (bf16 [T, H]; the router's own path from x to the logits is not part of
 * the layer's backward), dw = dL/dtopk_w (fp32 [T, k], the router-weight gradient, or NULL), and the weight
 * gradients in bf16 with the shapes of the weights (all four NULL = activation gradients only; otherwise all that
 * belong to present experts must be given).  bf16 mode only; H, I and I_shared must be multiples of 32.
 * Deterministic like the forward pass: no float atomics, fixed reduction orders.
 */
typedef struct mok_bwd_args {
    const void* x;                  /* bf16 [T, H] */
    const void* W_gate_up;          /* bf16 [E, 2I, H] */
    const void* W_down;             /* bf16 [E, H, I] */
    const void* W_shared_gate_up;   /* bf16 [2*I_shared, H] or NULL */
    const void* W_shared_down;      /* bf16 [H, I_shared]   or NULL */
    int32_t T, H, I, I_shared, E, k;
    const int32_t* topk_idx;        /* int32 [T, k] from the forward pass */
    const float* topk_w;            /* fp32 [T, k]  from the forward pass */
    const void* dout;               /* bf16 [T, H] */
    void* dx;                       /* out: bf16 [T, H] */
    float* dw;                      /* out: fp32 [T, k] or NULL */
    void* dW_gate_up;               /* out: bf16 [E, 2I, H] or NULL */
    void* dW_down;                  /* out: bf16 [E, H, I] or NULL */
    void* dW_shared_gate_up;        /* out: bf16 [2*I_shared, H] or NULL */
    void* dW_shared_down;           /* out: bf16 [H, I_shared] or NULL */
    void* workspace;                /* mok_bwd_workspace_bytes(...) bytes, 256-byte aligned */
    size_t workspace_bytes;
    const mok_config* config;       /* grid, cta_group 0/1/3 */
    void* stream;
} mok_bwd_args;
size_t mok_bwd_workspace_bytes(int T, int H, int I, int I_shared, int E, int k);
int mok_moe_backward(const mok_bwd_args* args);

/*
 * Backward pass under expert parallelism (Section 3.1: the backward pass moves the same rows the other way -- the rank
 * that serves a route pulls the row of dL/dout from the token's owner, the owner pulls dL/d(gathered x) from the
 * serving rank; Section 3.4: router-weight gradient inside the chain, activations recomputed).  Two calls per rank,
 * mirroring mok_ep_expert_ffn / mok_ep_combine, with a barrier over the ranks between them:
 *   mok_ep_expert_bwd : Algorithm 1 for this rank's experts from the all-gathered routes (the forward pass's tables and
 *       positions), then the one-rank chain on the rows served here -- x and dout rows pulled from the owners' buffers
 *       inside the GEMMs -- which leaves dL/d(gathered x) in dxg, dL/dw of the served routes in dw_routes (indexed by
 *       source rank * T_local * k + route; other entries untouched), the shared expert's dx of this rank's own tokens
 *       in dx_shared, and the weight gradients of the local experts (all four NULL: activation gradients only).
 *   mok_ep_bwd_combine : the owner sums the k rows of dxg it pulls from the serving ranks (through their pos tables)
 *       on top of dx_shared, in slot order in fp32, and fetches its routes' dw.
 * dx and dw equal the one-rank backward pass on the concatenated batch bit for bit; the weight gradients sum an
 * expert's rows in Algorithm 1's order, so they agree with it up to fp32 summation order.  bf16 mode only; H, I and
 * I_shared multiples of 32.  The paper prints no formulas for the backward pass: this is the chain rule of Section 2.1.
 */
typedef struct mok_ep_bwd_args {
    int32_t rank, n_ranks;
    int32_t T_local, H, I, I_shared, E, k;
    const void* x_peers[MOK_MAX_RANKS];      /* every rank's token rows, bf16 [T_local, H] (device addresses) */
    const void* dout_peers[MOK_MAX_RANKS];   /* every rank's dL/dout, bf16 [T_local, H] */
    const int32_t* idx_all;                  /* int32 [n_ranks, T_local * k]: all-gathered routes */
    const float* w_all;                      /* fp32 [n_ranks, T_local * k]: all-gathered router weights */
    const void* W_gate_up;                   /* bf16 [E / n_ranks, 2I, H]: this rank's experts */
    const void* W_down;                      /* bf16 [E / n_ranks, H, I] */
    const void* W_shared_gate_up;            /* bf16 [2 * I_shared, H] or NULL */
    const void* W_shared_down;               /* bf16 [H, I_shared] or NULL */
    void* dxg;                               /* out, read by the peers: bf16 [dxg_rows, H], dxg_rows >= mok_ep_y_rows(...) */
    long long dxg_rows;
    int32_t* pos;                            /* out, read by the peers: int32 [n_ranks * T_local * k] */
    float* dw_routes;                        /* out, read by the peers: fp32 [n_ranks * T_local * k] */
    void* dx_shared;                         /* out: bf16 [T_local rounded up to 256, H], or NULL without a shared expert */
    void* dW_gate_up;                        /* out: bf16 [E / n_ranks, 2I, H] or NULL */
    void* dW_down;                           /* out: bf16 [E / n_ranks, H, I] or NULL */
    void* dW_shared_gate_up;                 /* out: bf16 [2 * I_shared, H] or NULL (this rank's tokens' share) */
    void* dW_shared_down;                    /* out: bf16 [H, I_shared] or NULL */
    void* workspace;                         /* mok_ep_bwd_workspace_bytes(...) bytes, 256-byte aligned */
    size_t workspace_bytes;
    const mok_config* config;                /* grid, cta_group 0/1/3, gang_sync */
    void* stream;
} mok_ep_bwd_args;

typedef struct mok_ep_bwd_combine_args {
    int32_t rank, n_ranks;
    int32_t T_local, H, E, k;
    const int32_t* topk_idx;                 /* int32 [T_local, k]: this rank's routes */
    const void* dxg_peers[MOK_MAX_RANKS];    /* every rank's dxg */
    const int32_t* pos_peers[MOK_MAX_RANKS]; /* every rank's pos */
    const float* dw_peers[MOK_MAX_RANKS];    /* every rank's dw_routes (needed when dw != NULL) */
    const void* dx_shared;                   /* this rank's dx_shared, or NULL */
    void* dx;                                /* out: bf16 [T_local, H] */
    float* dw;                               /* out: fp32 [T_local, k], or NULL */
    void* stream;
} mok_ep_bwd_combine_args;

size_t mok_ep_bwd_workspace_bytes(int n_ranks, int T_local, int H, int I, int I_shared, int E, int k);
int mok_ep_expert_bwd(const mok_ep_bwd_args* args);
int mok_ep_bwd_combine(const mok_ep_bwd_combine_args* args);

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
 * Counters of the tcgen05 GEMM kernels of the last forward call that ran with config.debug != 0 (measurement aid;
 * Section 3 cost model: T_comp against T_sync).  Synchronises `stream`, then writes 4 x MOK_DEBUG_COUNTERS values:
 * slot 1 = routed gate/up GEMM, 2 = routed down GEMM, 3 = shared GEMMs (with config.fused_ffn the routed GEMMs are one
 * launch: slots 1 and 2 hold its gate/up tiles and its down tiles, [5] of slot 2 the time its producers waited for
 * gate/up tiles to complete, and slot 0 the whole kernel: [3], [8], [9], [11]).  Per slot, SM cycles summed over CTAs:
 * [0] MMA issuer waiting for operands, [1] for the peer CTA's operands, [2] for a free accumulator; [3] MMA issuer
 * total; [4] k-blocks issued (in 128-row units); [5] TMA producer waiting for a free stage; [6] epilogue waiting for an
 * accumulator; [7] epilogue total; then [8] the busiest CTA's MMA-issuer total (cycles, maximum over CTAs: [8] against
 * [3] / [11] is the load imbalance of the tile -> CTA rule); [9] MMA issuer total in nanoseconds of the global timer
 * ([3] / [9] = the SM clock the kernel really ran at, in GHz); [10] valid rows x k-blocks issued (256-row kernel
 * only, else 0: 128 x [4] minus this is the MMA work spent on padding rows); [11] CTAs that reported.
 */
#define MOK_DEBUG_COUNTERS 12
int mok_debug_counters(const void* workspace, void* stream, unsigned long long* out);

/* Number of kernels one mok_moe_forward_ex call enqueues for these arguments (the memset of the workspace header
   is not counted); 0 on bad sizes. */
int mok_launch_count(int T, int H, int I, int I_shared, int E, int k, const mok_config* config);

/* Host-only self-test of the per-device launch-state cache (the shared-memory opt-in of every kernel and the SM
   count are remembered per device, not per process, so that one process can drive several GPUs).  Makes no CUDA
   call; returns MOK_OK or the number of the failed check. */
int mok_selftest_per_device(void);

int mok_last_cuda_error(void);          /* cudaError_t of the most recent failed CUDA call on this thread */
const char* mok_status_string(int status);
int mok_version(void);                  /* major*10000 + minor*100 + patch */

#ifdef __cplusplus
}
#endif
#endif /* MOK_H_ */
