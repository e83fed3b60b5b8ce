/*
 * mok_ref_bwd.c -- CPU oracle for the backward pass of the MoE layer.  TEST INFRASTRUCTURE ONLY
 * (same rules as mok_ref.c: nothing on the product path may call it; no code shared with the CUDA path).
 *
 * What follows which passage of the paper
 *   Section 2.1 defines the layer, out[t] = f_shared(x[t]) + sum_s w[t,s] f_{idx[t,s]}(x[t]) with
 *   f(v) = W_down (silu(W_gate v) .* (W_up v)); Section 3.4 ("Fused router weight gradient", "activation
 *   recomputation") and Section 4.1 (backward = dgrad + wgrad, twice the forward FLOPs) name what the backward
 *   pass produces.  The paper prints no formulas for it: this file is the derivative of the definition, written
 *   out by the chain rule in fp64.  The router weights w[t,s] are treated as inputs: their gradient dw is an
 *   output ("router weight gradient"), the router's own backward is outside the layer.
 *
 *   Given dout[t,:] = dL/dout[t,:], for every route (t, s) with expert e and weight w:
 *       g = Wg_e x,  u = Wu_e x,  sig = 1/(1+exp(-g)),  a = g sig (= silu),  h = a .* u,  y = Wd_e h
 *       dw[t,s]  = <dout[t], y>
 *       dy       = w dout[t]
 *       dh       = Wd_e^T dy
 *       dg       = dh .* u .* sig .* (1 + g .* (1 - sig)),     du = dh .* a
 *       dx[t]   += Wg_e^T dg + Wu_e^T du
 *       dWd_e   += dy h^T,   dWg_e += dg x^T,   dWu_e += du x^T
 *   and the same for the shared expert with w = 1 (no dw).
 * Pins: tests/test_oracle_bwd_pins.py (central finite differences of an independent fp64 forward, special cases).
 * No function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_f64(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* One expert applied to one token: accumulates dx (if non-NULL) and the weight gradients (if non-NULL); returns
 * <dout, y> through *dot.  scratch: 5*I + H doubles. */
static void expert_backward(const double* v, const uint16_t* Wgu, const uint16_t* Wd, int H, int I,
                            double w, const double* dout, double* dx, double* dWgu, double* dWd, double* dot,
                            double* scratch) {
    double* g = scratch;
    double* u = g + I;
    double* h = u + I;
    double* dg = h + I;
    double* du = dg + I;
    for (int i = 0; i < I; ++i) {
        double gg = 0.0, uu = 0.0;
        for (int c = 0; c < H; ++c) {
            gg += bf16_f64(Wgu[(size_t)i * H + c]) * v[c];
            uu += bf16_f64(Wgu[(size_t)(I + i) * H + c]) * v[c];
        }
        g[i] = gg; u[i] = uu;
        h[i] = gg / (1.0 + exp(-gg)) * uu;
    }
    double d = 0.0;
    for (int c = 0; c < H; ++c) {
        double y = 0.0;
        for (int i = 0; i < I; ++i) y += bf16_f64(Wd[(size_t)c * I + i]) * h[i];
        d += dout[c] * y;
    }
    if (dot) *dot = d;
    for (int i = 0; i < I; ++i) {
        double dh = 0.0;
        for (int c = 0; c < H; ++c) dh += bf16_f64(Wd[(size_t)c * I + i]) * (w * dout[c]);
        const double sig = 1.0 / (1.0 + exp(-g[i]));
        dg[i] = dh * u[i] * sig * (1.0 + g[i] * (1.0 - sig));
        du[i] = dh * (g[i] * sig);
    }
    if (dx)
        for (int c = 0; c < H; ++c) {
            double acc = 0.0;
            for (int i = 0; i < I; ++i)
                acc += bf16_f64(Wgu[(size_t)i * H + c]) * dg[i] + bf16_f64(Wgu[(size_t)(I + i) * H + c]) * du[i];
            dx[c] += acc;
        }
    if (dWd)
        for (int c = 0; c < H; ++c)
            for (int i = 0; i < I; ++i) dWd[(size_t)c * I + i] += (w * dout[c]) * h[i];
    if (dWgu)
        for (int i = 0; i < I; ++i)
            for (int c = 0; c < H; ++c) {
                dWgu[(size_t)i * H + c] += dg[i] * v[c];
                dWgu[(size_t)(I + i) * H + c] += du[i] * v[c];
            }
}

/*
 * Backward of the whole layer for all T tokens.  dout[T,H] fp64.  Outputs (any may be NULL): dx[T,H], dw[T,k],
 * dWgu[E,2I,H], dWd[E,H,I], dWsgu[2Is,H], dWsd[H,Is]; weight gradients are overwritten (not accumulated into).
 */
int mok_ref_backward(const uint16_t* x, const uint16_t* W_gate_up, const uint16_t* W_down,
                     const uint16_t* W_sgu, const uint16_t* W_sd,
                     int T, int H, int I, int I_s, int E, int k, const int32_t* idx, const double* w,
                     const double* dout, double* dx, double* dw, double* dWgu, double* dWd, double* dWsgu,
                     double* dWsd) {
    if (!x || !dout || T < 0 || H <= 0 || I <= 0 || E <= 0 || k < 1 || !W_gate_up || !W_down || !idx || !w) return -1;
    if ((I_s > 0) != (W_sgu != NULL) || (I_s > 0) != (W_sd != NULL)) return -1;
    const int Imax = I > I_s ? I : I_s;
    if (dx) memset(dx, 0, sizeof(double) * (size_t)T * H);
    /* token side: dx and dw, parallel over tokens */
#pragma omp parallel
    {
        double* v = (double*)malloc(sizeof(double) * (size_t)H);
        double* scratch = (double*)malloc(sizeof(double) * (size_t)(5 * Imax + H));
#pragma omp for schedule(dynamic, 1)
        for (int t = 0; t < T; ++t) {
            for (int c = 0; c < H; ++c) v[c] = bf16_f64(x[(size_t)t * H + c]);
            const double* dr = dout + (size_t)t * H;
            if (I_s > 0 && dx) expert_backward(v, W_sgu, W_sd, H, I_s, 1.0, dr, dx + (size_t)t * H, NULL, NULL, NULL, scratch);
            for (int s = 0; s < k; ++s) {
                const int e = idx[(size_t)t * k + s];
                double d = 0.0;
                expert_backward(v, W_gate_up + (size_t)e * 2 * I * H, W_down + (size_t)e * H * I, H, I,
                                w[(size_t)t * k + s], dr, dx ? dx + (size_t)t * H : NULL, NULL, NULL, &d, scratch);
                if (dw) dw[(size_t)t * k + s] = d;
            }
        }
        free(v); free(scratch);
    }
    /* weight side: parallel over experts, every expert scans the routes that selected it, in token order */
    if (dWgu || dWd) {
        if (dWgu) memset(dWgu, 0, sizeof(double) * (size_t)E * 2 * I * H);
        if (dWd) memset(dWd, 0, sizeof(double) * (size_t)E * H * I);
#pragma omp parallel
        {
            double* v = (double*)malloc(sizeof(double) * (size_t)H);
            double* scratch = (double*)malloc(sizeof(double) * (size_t)(5 * Imax + H));
#pragma omp for schedule(dynamic, 1)
            for (int e = 0; e < E; ++e)
                for (int t = 0; t < T; ++t)
                    for (int s = 0; s < k; ++s) {
                        if (idx[(size_t)t * k + s] != e) continue;
                        for (int c = 0; c < H; ++c) v[c] = bf16_f64(x[(size_t)t * H + c]);
                        expert_backward(v, W_gate_up + (size_t)e * 2 * I * H, W_down + (size_t)e * H * I, H, I,
                                        w[(size_t)t * k + s], dout + (size_t)t * H, NULL,
                                        dWgu ? dWgu + (size_t)e * 2 * I * H : NULL, dWd ? dWd + (size_t)e * H * I : NULL,
                                        NULL, scratch);
                    }
            free(v); free(scratch);
        }
    }
    if (I_s > 0 && (dWsgu || dWsd)) {
        if (dWsgu) memset(dWsgu, 0, sizeof(double) * (size_t)2 * I_s * H);
        if (dWsd) memset(dWsd, 0, sizeof(double) * (size_t)H * I_s);
        double* v = (double*)malloc(sizeof(double) * (size_t)H);
        double* scratch = (double*)malloc(sizeof(double) * (size_t)(5 * Imax + H));
        for (int t = 0; t < T; ++t) {
            for (int c = 0; c < H; ++c) v[c] = bf16_f64(x[(size_t)t * H + c]);
            expert_backward(v, W_sgu, W_sd, H, I_s, 1.0, dout + (size_t)t * H, NULL, dWsgu, dWsd, NULL, scratch);
        }
        free(v); free(scratch);
    }
    return 0;
}

/*
 * Token side of the backward pass for a list of tokens only (full-size checks): dx[n_tok, H] and dw[n_tok, k] of the
 * listed tokens, from the same chain rule.  idx, w and dout are indexed by token id.
 */
int mok_ref_backward_tokens(const uint16_t* x, const uint16_t* W_gate_up, const uint16_t* W_down,
                            const uint16_t* W_sgu, const uint16_t* W_sd,
                            int H, int I, int I_s, int E, int k, const int32_t* idx, const double* w,
                            const double* dout, const int32_t* tokens, int n_tok, double* dx, double* dw) {
    if (!x || !dout || !tokens || !dx || n_tok < 0 || H <= 0 || I <= 0 || E <= 0 || k < 1 || !W_gate_up || !W_down || !idx || !w)
        return -1;
    if ((I_s > 0) != (W_sgu != NULL) || (I_s > 0) != (W_sd != NULL)) return -1;
    const int Imax = I > I_s ? I : I_s;
    memset(dx, 0, sizeof(double) * (size_t)n_tok * H);
    int bad = 0;
#pragma omp parallel
    {
        double* v = (double*)malloc(sizeof(double) * (size_t)H);
        double* scratch = (double*)malloc(sizeof(double) * (size_t)(5 * Imax + H));
#pragma omp for schedule(dynamic, 1)
        for (int n = 0; n < n_tok; ++n) {
            const int t = tokens[n];
            for (int c = 0; c < H; ++c) v[c] = bf16_f64(x[(size_t)t * H + c]);
            const double* dr = dout + (size_t)t * H;
            if (I_s > 0) expert_backward(v, W_sgu, W_sd, H, I_s, 1.0, dr, dx + (size_t)n * H, NULL, NULL, NULL, scratch);
            for (int s = 0; s < k; ++s) {
                const int e = idx[(size_t)t * k + s];
                if (e < 0 || e >= E) { bad = 1; continue; }
                double d = 0.0;
                expert_backward(v, W_gate_up + (size_t)e * 2 * I * H, W_down + (size_t)e * H * I, H, I,
                                w[(size_t)t * k + s], dr, dx + (size_t)n * H, NULL, NULL, &d, scratch);
                if (dw) dw[(size_t)n * k + s] = d;
            }
        }
        free(v); free(scratch);
    }
    return bad ? -2 : 0;
}
