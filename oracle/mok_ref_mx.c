/*
 * mok_ref_mx.c -- CPU oracle for the MXFP8 mode of the routed experts.  TEST INFRASTRUCTURE ONLY
 * (same rules as mok_ref.c: nothing on the product path may call it; no code shared with the CUDA path).
 *
 * What follows which passage of the paper
 *   Section 3.4 "MXFP8 Support": routed experts run on MXFP8 operands, the shared expert stays in
 *   bf16; weights are quantised ahead of time; activations are quantised where they are produced
 *   (the dispatched token rows, and the gated activation between the two GEMMs).
 *   The format is the one of the microscaling paper the section cites: blocks of 32 consecutive
 *   elements along the contraction dimension share one power-of-two scale X = 2^(floor(log2(amax)) - 8)
 *   stored as an 8-bit exponent (E8M0, code = exponent + 127), and every element is v / X rounded to
 *   nearest-even on the FP8 E4M3 grid with magnitudes above the largest normal (448) clamped to it.
 *   A block of zeros gets the smallest scale (code 0).
 *
 * Everything is evaluated in fp64: a quantised operand is the exact real number code * X, products and
 * sums are fp64, the gated activation is quantised from its fp64 value.
 * Pins: tests/test_oracle_mx_pins.py.  No function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_bits_to_f64(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* E4M3 ("fn" variant: no infinities, 0x7F/0xFF are NaN, largest finite 448): sign, 4 exponent bits (bias 7),
 * 3 mantissa bits; exponent field 0 = subnormals m/8 * 2^-6. */
double mok_ref_e4m3_decode(uint8_t c) {
    int s = c >> 7, e = (c >> 3) & 15, m = c & 7;
    double v;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) v = ldexp((double)m / 8.0, -6);
    else v = ldexp(1.0 + (double)m / 8.0, e - 7);
    return s ? -v : v;
}

/* Nearest E4M3 value, ties to the even code, magnitudes beyond 448 clamped to 448.  v must be finite. */
uint8_t mok_ref_e4m3_encode(double v) {
    uint8_t sign = (v < 0.0 || (v == 0.0 && signbit(v))) ? 0x80 : 0x00;
    double a = fabs(v);
    if (a >= 448.0) return sign | 0x7E;                 /* 448 = 1.75 * 2^8: exponent field 15, mantissa 6 */
    /* the grid spacing around a: 2^-9 below 2^-6 (subnormals), else 2^(floor(log2 a) - 3) */
    int ex;
    (void)frexp(a, &ex);                                /* a = f * 2^ex, f in [0.5, 1)  ->  floor(log2 a) = ex - 1 */
    int e = (a == 0.0) ? -6 : ex - 1;
    if (e < -6) e = -6;
    double step = ldexp(1.0, e - 3);
    double q = a / step;                                /* exact: a power-of-two scaling */
    double r = nearbyint(q);                            /* default rounding mode: to nearest, ties to even */
    /* r counts steps from zero: r in [0, 8] in the subnormal range, [8, 16] in a normal binade */
    int steps = (int)r;
    int field, mant;
    if (e == -6 && steps < 8) { field = 0; mant = steps; }
    else {
        if (steps == 16) { steps = 8; e += 1; }         /* rounded up into the next binade */
        field = e + 7;
        mant = steps - 8;
    }
    if (field > 15 || (field == 15 && mant > 6)) return sign | 0x7E;
    return sign | (uint8_t)(field << 3) | (uint8_t)mant;
}

/* Shared scale of one block: E8M0 code of 2^(floor(log2(amax)) - 8), clamped to the representable exponents. */
uint8_t mok_ref_mx_scale_code(const double* v, int n) {
    double amax = 0.0;
    for (int i = 0; i < n; ++i) { double a = fabs(v[i]); if (a > amax) amax = a; }
    if (amax == 0.0) return 0;
    int ex;
    (void)frexp(amax, &ex);
    int code = (ex - 1) - 8 + 127;
    if (code < 0) code = 0;
    if (code > 254) code = 254;
    return (uint8_t)code;
}

/* Quantise rows of `cols` fp64 values (cols a multiple of 32): codes[rows, cols], scales[rows, cols/32]. */
int mok_ref_mx_quantize(const double* v, long long rows, int cols, uint8_t* codes, uint8_t* scales) {
    if (!v || !codes || !scales || rows < 0 || cols <= 0 || cols % 32) return -1;
    const int nb = cols / 32;
#pragma omp parallel for schedule(static)
    for (long long r = 0; r < rows; ++r)
        for (int b = 0; b < nb; ++b) {
            const double* blk = v + (size_t)r * cols + (size_t)b * 32;
            uint8_t sc = mok_ref_mx_scale_code(blk, 32);
            scales[(size_t)r * nb + b] = sc;
            double X = ldexp(1.0, (int)sc - 127);
            for (int i = 0; i < 32; ++i) codes[(size_t)r * cols + (size_t)b * 32 + i] = mok_ref_e4m3_encode(blk[i] / X);
        }
    return 0;
}

/* The real numbers a quantised tensor stands for: out = decode(code) * 2^(scale - 127). */
int mok_ref_mx_dequantize(const uint8_t* codes, const uint8_t* scales, long long rows, int cols, double* out) {
    if (!codes || !scales || !out || rows < 0 || cols <= 0 || cols % 32) return -1;
    const int nb = cols / 32;
#pragma omp parallel for schedule(static)
    for (long long r = 0; r < rows; ++r)
        for (int c = 0; c < cols; ++c)
            out[(size_t)r * cols + c] = mok_ref_e4m3_decode(codes[(size_t)r * cols + c]) *
                                        ldexp(1.0, (int)scales[(size_t)r * nb + c / 32] - 127);
    return 0;
}

/* bf16 bit patterns -> quantise -> the fp32 number each element stands for (exact: 4 significant bits times a
 * power of two).  Used to pre-quantise weights once. */
int mok_ref_mx_roundtrip_bf16(const uint16_t* in, long long rows, int cols, float* out) {
    if (!in || !out || rows < 0 || cols <= 0 || cols % 32) return -1;
    const int nb = cols / 32;
#pragma omp parallel for schedule(static)
    for (long long r = 0; r < rows; ++r) {
        double blk[32];
        for (int b = 0; b < nb; ++b) {
            for (int i = 0; i < 32; ++i) blk[i] = bf16_bits_to_f64(in[(size_t)r * cols + (size_t)b * 32 + i]);
            double X = ldexp(1.0, (int)mok_ref_mx_scale_code(blk, 32) - 127);
            for (int i = 0; i < 32; ++i)
                out[(size_t)r * cols + (size_t)b * 32 + i] = (float)(mok_ref_e4m3_decode(mok_ref_e4m3_encode(blk[i] / X)) * X);
        }
    }
    return 0;
}

static void quantize_in_place(double* v, int n) {      /* n a multiple of 32 */
    for (int b = 0; b < n; b += 32) {
        double X = ldexp(1.0, (int)mok_ref_mx_scale_code(v + b, 32) - 127);
        for (int i = 0; i < 32; ++i) v[b + i] = mok_ref_e4m3_decode(mok_ref_e4m3_encode(v[b + i] / X)) * X;
    }
}

/* routed expert in MXFP8: vq = Q(x row) along H; g = Wg_q vq, u = Wu_q vq; h = Q(silu(g) * u) along I; y = Wd_q h */
static void ffn_mx_accumulate(const double* vq, const float* Wgu_q, const float* Wd_q, int H, int I, double scale,
                              double* hbuf, double* out) {
    for (int i = 0; i < I; ++i) {
        const float* wg = Wgu_q + (size_t)i * H;
        const float* wu = Wgu_q + (size_t)(I + i) * H;
        double g = 0.0, u = 0.0;
        for (int h = 0; h < H; ++h) { g += (double)wg[h] * vq[h]; u += (double)wu[h] * vq[h]; }
        hbuf[i] = (g / (1.0 + exp(-g))) * u;
    }
    quantize_in_place(hbuf, I);
    for (int h = 0; h < H; ++h) {
        const float* wd = Wd_q + (size_t)h * I;
        double y = 0.0;
        for (int i = 0; i < I; ++i) y += (double)wd[i] * hbuf[i];
        out[h] += scale * y;
    }
}

static void ffn_bf16_accumulate(const double* v, const uint16_t* Wgu, const uint16_t* Wd, int H, int I, double* hbuf,
                                double* out) {
    for (int i = 0; i < I; ++i) {
        double g = 0.0, u = 0.0;
        for (int h = 0; h < H; ++h) {
            g += bf16_bits_to_f64(Wgu[(size_t)i * H + h]) * v[h];
            u += bf16_bits_to_f64(Wgu[(size_t)(I + i) * H + h]) * v[h];
        }
        hbuf[i] = (g / (1.0 + exp(-g))) * u;
    }
    for (int h = 0; h < H; ++h) {
        double y = 0.0;
        for (int i = 0; i < I; ++i) y += bf16_bits_to_f64(Wd[(size_t)h * I + i]) * hbuf[i];
        out[h] += y;
    }
}

/*
 * The MoE equation of Section 2.1 with the routed experts in MXFP8 (Section 3.4) and the shared expert in bf16,
 * per token from the definition, for the listed tokens.  Wgu_q [E,2I,H] and Wd_q [E,H,I] are the pre-quantised
 * routed weights as the numbers they stand for (mok_ref_mx_roundtrip_bf16 along their last index).
 * H and I must be multiples of 32.
 */
int mok_ref_ffn_tokens_mx(const uint16_t* x, const float* Wgu_q, const float* Wd_q,
                          const uint16_t* W_sgu, const uint16_t* W_sd,
                          int H, int I, int I_s, int E, int k, const int32_t* idx, const double* w,
                          const int32_t* tokens, int n_tok, double* out) {
    if (!x || !out || !tokens || !Wgu_q || !Wd_q || !idx || !w || H <= 0 || I <= 0 || n_tok < 0) return -1;
    if (H % 32 || I % 32) return -1;
    if ((I_s > 0) != (W_sgu != NULL) || (I_s > 0) != (W_sd != NULL)) return -1;
    int Imax = I > I_s ? I : I_s;
    int bad = 0;
#pragma omp parallel
    {
        double* v = (double*)malloc(sizeof(double) * (size_t)H);
        double* vq = (double*)malloc(sizeof(double) * (size_t)H);
        double* hbuf = (double*)malloc(sizeof(double) * (size_t)Imax);
#pragma omp for schedule(dynamic, 1)
        for (int n = 0; n < n_tok; ++n) {
            int t = tokens[n];
            double* o = out + (size_t)n * H;
            for (int h = 0; h < H; ++h) { v[h] = bf16_bits_to_f64(x[(size_t)t * H + h]); vq[h] = v[h]; o[h] = 0.0; }
            quantize_in_place(vq, H);
            if (I_s > 0) ffn_bf16_accumulate(v, W_sgu, W_sd, H, I_s, hbuf, o);
            for (int s = 0; s < k; ++s) {
                int e = idx[(size_t)t * k + s];
                if (e < 0 || e >= E) { bad = 1; continue; }
                ffn_mx_accumulate(vq, Wgu_q + (size_t)e * 2 * I * H, Wd_q + (size_t)e * H * I, H, I,
                                  w[(size_t)t * k + s], hbuf, o);
            }
        }
        free(v); free(vq); free(hbuf);
    }
    return bad ? -2 : 0;
}
