/*
 * mok_ref.c -- CPU oracle for the MoE layer forward pass.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 evaluation of what the layer computes, written from the paper's
 * definition.  Nothing on the product path may call it: only the test suite, the smoke check
 * and the benchmark's cpu-baseline leg load this library.  It shares no code, header, table or
 * helper with the CUDA path.
 *
 * Conventions
 *   - bf16 tensors arrive as uint16_t bit patterns and are widened exactly to double.
 *   - x[T,H] row-major; W_r[E,H] fp32; bias[E] fp32 or NULL;
 *     W_gate_up[E,2I,H] (rows 0..I-1 = W_gate, rows I..2I-1 = W_up); W_down[E,H,I];
 *     shared expert: W_sgu[2*I_s,H], W_sd[H,I_s] (NULL / I_s = 0 when absent).
 *   - routes are flattened token-major: route j = t*k + s.
 *
 * What follows which passage of the paper
 *   mok_ref_logits / mok_ref_topk / mok_ref_weights : Section 2.1 (the router projects every token
 *       onto the experts, keeps its k best and weights each of them) and the normalised weights
 *       s_i / sum_j s_j of the MoE equation in Section 2.1.  Score = softmax over all E logits
 *       (the benchmark configuration's reading); ties go to the lowest expert id.
 *   mok_ref_schedule : the dispatch schedule of one rank as Section 3.1 restates Algorithm 1: the
 *       routes in ascending order of (expert, route id).
 *   mok_ref_alg1     : the pull schedule of one destination rank for R source ranks, from the same
 *       restatement: the routes in ascending order of (local expert, ordinal, source rank).  The
 *       printed algorithm's closed-form row position is NOT used here; the pins evaluate it instead.
 *   mok_ref_ffn_tokens / mok_ref_forward : the MoE equation and the expert FFN
 *       f_i(x) = W_down (phi(W_gate x) .* W_up x) of Section 2.1, phi = SiLU.
 *
 * Parity pins live in tests/test_oracle_*.py (golden example, closed forms, brute force,
 * library special cases).  No function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static inline double bf16_to_f64(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* round-to-nearest-even of a double to the bf16 grid, returned as double (diagnostic "mimic" mode) */
static double round_bf16(double v) {
    float f = (float)v; /* double -> float RNE; bf16 grid is far coarser, double rounding is negligible here */
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7F800000u) == 0x7F800000u) return (double)f;
    u = (u + 0x7FFFu + ((u >> 16) & 1u)) & 0xFFFF0000u;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int mok_ref_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Section 2.1, router projection: logit[t,e] = sum_h x[t,h] * W_r[e,h] (+ bias[e]), h ascending. */
int mok_ref_logits(const uint16_t* x, const float* W_r, const float* bias,
                   int T, int H, int E, double* logits) {
    if (!x || !W_r || !logits || T < 0 || H <= 0 || E <= 0) return -1;
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {
        for (int e = 0; e < E; ++e) {
            double acc = 0.0;
            for (int h = 0; h < H; ++h)
                acc += bf16_to_f64(x[(size_t)t * H + h]) * (double)W_r[(size_t)e * H + h];
            if (bias) acc += (double)bias[e];
            logits[(size_t)t * E + e] = acc;
        }
    }
    return 0;
}

/*
 * Section 2.1, top-k selection.  Experts of a token are ordered by (logit descending, expert id
 * ascending); idx[t,0..k-1] are the first k of that order.  gap[t] is the distance between the
 * k-th and the (k+1)-th logit of that order (+inf when k == E): a token with a small gap is a
 * near-tie whose selection legitimately depends on rounding.
 */
int mok_ref_topk(const double* logits, int T, int E, int k, int32_t* idx, double* gap) {
    if (!logits || !idx || k < 1 || k > E) return -1;
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {
        const double* l = logits + (size_t)t * E;
        char* taken = (char*)calloc((size_t)E, 1);
        for (int s = 0; s <= k; ++s) {
            int best = -1;
            for (int e = 0; e < E; ++e) { /* ascending id + strict '>' => lowest id wins ties */
                if (taken[e]) continue;
                if (best < 0 || l[e] > l[best]) best = e;
            }
            if (s < k) {
                idx[(size_t)t * k + s] = best;
                taken[best] = 1;
            } else if (gap) {
                gap[t] = (best < 0) ? INFINITY : l[idx[(size_t)t * k + k - 1]] - l[best];
            }
        }
        free(taken);
    }
    return 0;
}

/*
 * Section 2.1, normalised router weights: s = softmax over ALL E logits; the weight of a selected
 * expert is s_i / sum_{j in selected} s_j.  `idx` may be any selection (the oracle's own, or the
 * device's for tokens whose near-tie was resolved the other way).
 */
int mok_ref_weights(const double* logits, const int32_t* idx, int T, int E, int k, double* w) {
    if (!logits || !idx || !w) return -1;
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {
        const double* l = logits + (size_t)t * E;
        double mx = l[0];
        for (int e = 1; e < E; ++e) if (l[e] > mx) mx = l[e];
        double den = 0.0;
        for (int e = 0; e < E; ++e) den += exp(l[e] - mx);
        double sel = 0.0;
        for (int s = 0; s < k; ++s) sel += exp(l[idx[(size_t)t * k + s]] - mx) / den;
        for (int s = 0; s < k; ++s)
            w[(size_t)t * k + s] = (exp(l[idx[(size_t)t * k + s]] - mx) / den) / sel;
    }
    return 0;
}

/*
 * Algorithm 1 with one rank, in the form of its restatement (Section 3.1): routes sorted by
 * (expert ascending, route id ascending).  counts[e] = number of routes to e; offsets = exclusive
 * prefix sum (offsets[E] = n); perm[p] = route at buffer position p; inv[perm[p]] = p.
 */
int mok_ref_schedule(const int32_t* a, int n, int E,
                     int32_t* counts, int32_t* offsets, int32_t* perm, int32_t* inv) {
    if (!a || !counts || !offsets || !perm || !inv || n < 0 || E <= 0) return -1;
    for (int e = 0; e < E; ++e) counts[e] = 0;
    for (int j = 0; j < n; ++j) {
        if (a[j] < 0 || a[j] >= E) return -2;
        counts[a[j]]++;
    }
    offsets[0] = 0;
    for (int e = 0; e < E; ++e) offsets[e + 1] = offsets[e] + counts[e];
    int p = 0;
    for (int e = 0; e < E; ++e)
        for (int j = 0; j < n; ++j)
            if (a[j] == e) { perm[p] = j; inv[j] = p; ++p; }
    return 0;
}

/*
 * The pull schedule of one destination rank for R source ranks (Section 3.1), from its defining order rather
 * than from the position arithmetic of the printed algorithm: rank c owns global experts cL .. cL+L-1, and the
 * rows it receives are the routes (r, j) with A[r,j] in that range, laid out in ascending order of the key
 *     ( local expert l,  ordinal o of the route among rank r's routes to that expert,  source rank r ).
 * Sorting by l gives each expert one contiguous run; inside a run, ordinal-major order takes one route from every
 * rank that still has one before taking anybody's next, i.e. consecutive rows cycle over the source ranks.
 * S[l] = first row of expert l (S[L] = rows received); phi_rank / phi_idx give the source of every row and must
 * hold at least S[L] entries (R*NK always suffices).  A[r*NK + j] in [0, R*L).
 */
typedef struct { int32_t l, o, r, j; } pull_key;

static int pull_key_cmp(const void* pa, const void* pb) {
    const pull_key* a = (const pull_key*)pa;
    const pull_key* b = (const pull_key*)pb;
    if (a->l != b->l) return a->l < b->l ? -1 : 1;
    if (a->o != b->o) return a->o < b->o ? -1 : 1;
    if (a->r != b->r) return a->r < b->r ? -1 : 1;
    return 0;                       /* (l, o, r) identifies a route: never reached for two different routes */
}

int mok_ref_alg1(const int32_t* A, int R, int NK, int L, int c,
                 int32_t* S, int32_t* phi_rank, int32_t* phi_idx) {
    if (!A || !S || !phi_rank || !phi_idx || R <= 0 || NK < 0 || L <= 0 || c < 0 || c >= R) return -1;
    pull_key* keys = (pull_key*)malloc(sizeof(pull_key) * ((size_t)R * NK + 1));
    int32_t* seen = (int32_t*)malloc(sizeof(int32_t) * (size_t)L);
    if (!keys || !seen) { free(keys); free(seen); return -3; }
    size_t n = 0;
    for (int l = 0; l <= L; ++l) S[l] = 0;
    for (int r = 0; r < R; ++r) {
        for (int l = 0; l < L; ++l) seen[l] = 0;          /* routes of rank r to local expert l met so far */
        for (int j = 0; j < NK; ++j) {
            int g = A[(size_t)r * NK + j];
            if (g < 0 || g >= R * L) { free(keys); free(seen); return -2; }
            if (g / L != c) continue;
            pull_key q = { g - c * L, seen[g - c * L]++, r, j };
            keys[n++] = q;
            S[q.l + 1]++;                                   /* rows of expert l, turned into prefix sums below */
        }
    }
    for (int l = 0; l < L; ++l) S[l + 1] += S[l];
    qsort(keys, n, sizeof(pull_key), pull_key_cmp);
    for (size_t p = 0; p < n; ++p) { phi_rank[p] = keys[p].r; phi_idx[p] = keys[p].j; }
    free(keys);
    free(seen);
    return 0;
}

/* f(v) = W_d ( silu(W_g v) .* (W_u v) ) accumulated as out[0..H) += scale * f(v);  silu(z) = z / (1 + exp(-z)) */
static void ffn_accumulate(const double* v, const uint16_t* Wgu, const uint16_t* Wd,
                           int H, int I, double scale, int mimic, double* hbuf, double* out) {
    for (int i = 0; i < I; ++i) {
        const uint16_t* wg = Wgu + (size_t)i * H;
        const uint16_t* wu = Wgu + (size_t)(I + i) * H;
        double g = 0.0, u = 0.0;
        for (int h = 0; h < H; ++h) {
            g += bf16_to_f64(wg[h]) * v[h];
            u += bf16_to_f64(wu[h]) * v[h];
        }
        double a = (g / (1.0 + exp(-g))) * u;
        hbuf[i] = mimic ? round_bf16(a) : a;
    }
    for (int h = 0; h < H; ++h) {
        const uint16_t* wd = Wd + (size_t)h * I;
        double y = 0.0;
        for (int i = 0; i < I; ++i) y += bf16_to_f64(wd[i]) * hbuf[i];
        if (mimic) y = round_bf16(y);
        out[h] += scale * y;
    }
}

/*
 * MoE(x, s) = f_shared(x) + sum_{i in selected} w_i f_i(x), evaluated from the definition for the
 * n_tok tokens listed in `tokens` (token ids into x / idx / w).  out[n_tok, H] in fp64.
 * It never looks at the dispatch schedule.  mimic_bf16 != 0 rounds the gated activation and each
 * expert output to bf16 the way a bf16 pipeline would (a diagnostic, not the reference).
 */
int mok_ref_ffn_tokens(const uint16_t* x, const uint16_t* W_gate_up, const uint16_t* W_down,
                       const uint16_t* W_sgu, const uint16_t* W_sd,
                       int H, int I, int I_s, int E, int k,
                       const int32_t* idx, const double* w,
                       const int32_t* tokens, int n_tok, int mimic_bf16, double* out) {
    if (!x || !out || !tokens || H <= 0 || n_tok < 0) return -1;
    if (k > 0 && (!W_gate_up || !W_down || !idx || !w || I <= 0)) return -1;
    if ((I_s > 0) != (W_sgu != NULL) || (I_s > 0) != (W_sd != NULL)) return -1;
    int Imax = I > I_s ? I : I_s;
    int bad = 0;
#pragma omp parallel
    {
        double* v = (double*)malloc(sizeof(double) * (size_t)H);
        double* hbuf = (double*)malloc(sizeof(double) * (size_t)(Imax > 0 ? Imax : 1));
#pragma omp for schedule(dynamic, 1)
        for (int n = 0; n < n_tok; ++n) {
            int t = tokens[n];
            double* o = out + (size_t)n * H;
            for (int h = 0; h < H; ++h) { v[h] = bf16_to_f64(x[(size_t)t * H + h]); o[h] = 0.0; }
            if (I_s > 0) ffn_accumulate(v, W_sgu, W_sd, H, I_s, 1.0, mimic_bf16, hbuf, o);
            for (int s = 0; s < k; ++s) {
                int e = idx[(size_t)t * k + s];
                if (e < 0 || e >= E) { bad = 1; continue; }
                ffn_accumulate(v, W_gate_up + (size_t)e * 2 * I * H, W_down + (size_t)e * H * I,
                               H, I, w[(size_t)t * k + s], mimic_bf16, hbuf, o);
            }
        }
        free(v);
        free(hbuf);
    }
    return bad ? -2 : 0;
}

/* Whole layer: route every token, then evaluate every token.  Optional outputs may be NULL. */
int mok_ref_forward(const uint16_t* x, const float* W_r, const float* bias,
                    const uint16_t* W_gate_up, const uint16_t* W_down,
                    const uint16_t* W_sgu, const uint16_t* W_sd,
                    int T, int H, int I, int I_s, int E, int k,
                    double* out, int32_t* idx_out, double* w_out) {
    if (T == 0) return 0;
    double* logits = (double*)malloc(sizeof(double) * (size_t)T * E);
    int32_t* idx = (int32_t*)malloc(sizeof(int32_t) * (size_t)T * k);
    double* w = (double*)malloc(sizeof(double) * (size_t)T * k);
    int32_t* tokens = (int32_t*)malloc(sizeof(int32_t) * (size_t)T);
    int rc = -3;
    if (logits && idx && w && tokens) {
        rc = mok_ref_logits(x, W_r, bias, T, H, E, logits);
        if (!rc) rc = mok_ref_topk(logits, T, E, k, idx, NULL);
        if (!rc) rc = mok_ref_weights(logits, idx, T, E, k, w);
        for (int t = 0; t < T; ++t) tokens[t] = t;
        if (!rc) rc = mok_ref_ffn_tokens(x, W_gate_up, W_down, W_sgu, W_sd, H, I, I_s, E, k,
                                         idx, w, tokens, T, 0, out);
        if (!rc && idx_out) memcpy(idx_out, idx, sizeof(int32_t) * (size_t)T * k);
        if (!rc && w_out) memcpy(w_out, w, sizeof(double) * (size_t)T * k);
    }
    free(logits); free(idx); free(w); free(tokens);
    return rc;
}
