/*
 * CPU oracle for the DynaMo quantized-MoE hot path.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, float64 restatement of what the path computes, written from the
 * paper's description of the method (expert-level uniform mixed-precision
 * quantization, Section IV-A; channel cache and channel-level switching,
 * Sections IV-B and V-A; packed low-bit weights dequantized and multiplied,
 * Section V-B; Top-K expert selection, Section II-A).  It shares no code with
 * the CUDA library and is never called by it.  Only the tests, the smoke check
 * and the benchmark's CPU-baseline leg may load this file.
 *
 * No blocking, fusion or reordering beyond what each definition states: every
 * function below is the definition written out as loops.  Floating point is
 * IEEE double; build with -ffp-contract=off so that no multiply-add is fused.
 *
 * Parity pins (see tests): fp16 conversion against a library conversion over
 * all half-ulp midpoints; quantizer against brute-force nearest-level search,
 * the lossless construction and the error bound; pack/unpack round trip;
 * routing against a stable sort; permutation against Python's sorted();
 * the FFN against a dense float64 matmul of the dequantized weights, and the
 * all-channels-switched identity.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ---- number formats --------------------------------------------------------------- */

/* bf16 bit pattern -> double (exact). */
double orc_bf16_to_f64(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* fp16 bit pattern -> double (exact; subnormals, infinities and NaN handled). */
double orc_f16_to_f64(uint16_t h) {
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1f;
    int frac = h & 0x3ff;
    double v;
    if (e == 0) v = ldexp((double)frac, -24);
    else if (e == 31) v = frac ? NAN : INFINITY;
    else v = ldexp((double)(frac | 0x400), e - 25);
    return sign ? -v : v;
}

/* double -> fp16 bit pattern in ONE rounding: round-to-nearest, ties to even,
 * subnormals kept, overflow to infinity. */
uint16_t orc_f64_to_f16(double x) {
    uint16_t sign = signbit(x) ? 0x8000 : 0;
    if (isnan(x)) return (uint16_t)(sign | 0x7e00);
    double a = fabs(x);
    if (isinf(a)) return (uint16_t)(sign | 0x7c00);
    if (a == 0.0) return sign;
    int ex;
    (void)frexp(a, &ex); /* a = f * 2^ex, f in [0.5, 1) -> a in [2^(ex-1), 2^ex) */
    int e = ex - 1;      /* unbiased exponent of a */
    if (e < -14) e = -14; /* subnormal range: fixed quantum 2^-24 */
    /* quantum of the target format at this exponent: 2^(e-10) */
    double scaled = ldexp(a, 10 - e); /* exact: power-of-two scaling */
    double r = nearbyint(scaled);     /* default rounding mode: nearest, ties to even */
    /* r in [0, 2048]; mantissa overflow moves to the next exponent */
    if (r >= 2048.0) { r = 1024.0; e += 1; }
    if (e > 15) return (uint16_t)(sign | 0x7c00);
    uint32_t ri = (uint32_t)r;
    if (ri < 1024) { /* subnormal (e == -14 here) or zero */
        return (uint16_t)(sign | ri);
    }
    return (uint16_t)(sign | ((uint32_t)(e + 15) << 10) | (ri - 1024));
}

/* ---- C1: group-wise asymmetric uniform quantizer (Section IV-A, "uniform quantization") ---
 * W is [N, K] row-major bf16 bit patterns; groups are G consecutive k of one row.
 * Per group: lo/hi = min/max; scale s = fp16((hi - lo) / L), L = 2^bits - 1 (s := 1 if it
 * rounds to 0); zero m = fp16(lo); code q = clamp(rint((w - m) / s), 0, L) with true
 * division and ties-to-even.  q is [N, K] uint8, s and m are [N, K/G] fp16 bit patterns. */
void orc_quantize(const uint16_t* w, int64_t N, int64_t K, int G, int bits,
                  uint8_t* q, uint16_t* s_out, uint16_t* m_out) {
    const double L = (double)((1 << bits) - 1);
    const int64_t ng = K / G;
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        for (int64_t g = 0; g < ng; ++g) {
            const uint16_t* wp = w + n * K + g * G;
            double lo = orc_bf16_to_f64(wp[0]), hi = lo;
            for (int i = 1; i < G; ++i) {
                double v = orc_bf16_to_f64(wp[i]);
                if (v < lo) lo = v;
                if (v > hi) hi = v;
            }
            uint16_t sb = orc_f64_to_f16((hi - lo) / L);
            if (orc_f16_to_f64(sb) == 0.0) sb = 0x3c00; /* 1.0 */
            uint16_t mb = orc_f64_to_f16(lo);
            const double s = orc_f16_to_f64(sb), m = orc_f16_to_f64(mb);
            s_out[n * ng + g] = sb;
            m_out[n * ng + g] = mb;
            for (int i = 0; i < G; ++i) {
                double v = orc_bf16_to_f64(wp[i]);
                double t = nearbyint((v - m) / s);
                if (t < 0.0) t = 0.0;
                if (t > L) t = L;
                q[n * K + g * G + i] = (uint8_t)t;
            }
        }
    }
}

/* Dequantized value of one element: s*q + m in double (exact). */
static inline double deq(const uint8_t* q, const uint16_t* s, const uint16_t* m,
                         int64_t n, int64_t k, int64_t K, int G) {
    const int64_t ng = K / G;
    return orc_f16_to_f64(s[n * ng + k / G]) * (double)q[n * K + k] + orc_f16_to_f64(m[n * ng + k / G]);
}

void orc_dequantize(const uint8_t* q, const uint16_t* s, const uint16_t* m,
                    int64_t N, int64_t K, int G, double* out) {
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n)
        for (int64_t k = 0; k < K; ++k) out[n * K + k] = deq(q, s, m, n, k, K, G);
}

/* ---- C2: canonical bit packing (Section V-B, "pack multiple low-precision data into an INT32") --
 * Code k of a row occupies bits [bits*k, bits*k + bits) of the row's little-endian bit stream,
 * stored in uint32 words; a row takes ceil(K*bits/32) words. */
int64_t orc_packed_words(int64_t K, int bits) { return (K * bits + 31) / 32; }

void orc_pack_rows(const uint8_t* q, int64_t N, int64_t K, int bits, uint32_t* out) {
    const int64_t nw = orc_packed_words(K, bits);
    memset(out, 0, (size_t)(N * nw) * sizeof(uint32_t));
    for (int64_t n = 0; n < N; ++n)
        for (int64_t k = 0; k < K; ++k)
            for (int b = 0; b < bits; ++b) {
                int64_t pos = k * bits + b;
                if ((q[n * K + k] >> b) & 1) out[n * nw + pos / 32] |= (uint32_t)1 << (pos % 32);
            }
}

void orc_unpack_rows(const uint32_t* in, int64_t N, int64_t K, int bits, uint8_t* q) {
    const int64_t nw = orc_packed_words(K, bits);
    for (int64_t n = 0; n < N; ++n)
        for (int64_t k = 0; k < K; ++k) {
            unsigned v = 0;
            for (int b = 0; b < bits; ++b) {
                int64_t pos = k * bits + b;
                v |= ((in[n * nw + pos / 32] >> (pos % 32)) & 1u) << b;
            }
            q[n * K + k] = (uint8_t)v;
        }
}

/* ---- router scores (Section II-A: the gating network scores every expert for a token) -------
 * scores[t][e] = sum_c x[t][c] * w_r[e][c] + bias[e]; x and w_r are bf16 bit patterns, every product and
 * the sum in double (a product of two bf16 values is exact in double; the sum of d of them rounds at 2^-53). */
void orc_router_scores(const uint16_t* x, const uint16_t* w_r, const float* bias, int64_t T, int64_t d, int E,
                       double* scores) {
    for (int64_t t = 0; t < T; ++t)
        for (int e = 0; e < E; ++e) {
            double acc = 0.0;
            for (int64_t c = 0; c < d; ++c) acc += orc_bf16_to_f64(x[t * d + c]) * orc_bf16_to_f64(w_r[(int64_t)e * d + c]);
            scores[t * E + e] = acc + (bias ? (double)bias[e] : 0.0);
        }
}

/* ---- C3: Top-K routing (Section II-A: a fixed number of experts per token) ------------
 * idx[t, :] = the k experts with the largest logits, descending, ties -> lower index.
 * p = softmax(logits[t, :]) in double over all E; w = p[idx] (divided by their sum if renorm). */
void orc_route(const float* logits, int64_t T, int E, int k, int renorm, int32_t* idx, double* w) {
    for (int64_t t = 0; t < T; ++t) {
        const float* l = logits + t * E;
        double mx = (double)l[0];
        for (int e = 1; e < E; ++e) if ((double)l[e] > mx) mx = (double)l[e];
        double den = 0.0;
        for (int e = 0; e < E; ++e) den += exp((double)l[e] - mx);
        for (int j = 0; j < k; ++j) {
            int best = -1;
            for (int e = 0; e < E; ++e) {
                int taken = 0;
                for (int i = 0; i < j; ++i) if (idx[t * k + i] == e) taken = 1;
                if (taken) continue;
                if (best < 0 || l[e] > l[best]) best = e; /* strict >: ties keep the lower index */
            }
            idx[t * k + j] = best;
            w[t * k + j] = exp((double)l[best] - mx) / den;
        }
        if (renorm) {
            double sum = 0.0;
            for (int j = 0; j < k; ++j) sum += w[t * k + j];
            for (int j = 0; j < k; ++j) w[t * k + j] /= sum;
        }
    }
}

/* ---- C4: permutation (Section II-A: one token is dispatched to several experts) -----------
 * offsets = exclusive scan of the per-expert pair counts; sorted row r in expert e's segment
 * lists that expert's (token, slot) pairs in ascending token; perm[r] = t*k + j. */
void orc_permute(const int32_t* idx, int64_t T, int k, int E, int32_t* offsets, int32_t* perm) {
    for (int e = 0; e <= E; ++e) offsets[e] = 0;
    for (int64_t i = 0; i < T * k; ++i) offsets[idx[i] + 1] += 1;
    for (int e = 0; e < E; ++e) offsets[e + 1] += offsets[e];
    int32_t* cur = (int32_t*)malloc(sizeof(int32_t) * (size_t)(E > 0 ? E : 1));
    for (int e = 0; e < E; ++e) cur[e] = offsets[e];
    for (int64_t t = 0; t < T; ++t)
        for (int j = 0; j < k; ++j) {
            int e = idx[t * k + j];
            perm[cur[e]++] = (int32_t)(t * k + j);
        }
    free(cur);
}

/* ---- C5 + C6: one expert's SwiGLU FFN over effective weights ------------------------------
 * Effective weight (Sections IV-B, V-A: significant channels are served from the channel cache
 * at the higher precision, the rest at the expert's base precision):
 *   W_eff[n, c] = s8[n, c/G]*q8[n, c] + m8[n, c/G]   if mask != NULL and mask[c]   (gate, up: c an input channel
 *                                                       in [0, d); down: mask_d over its input channels [0, f))
 *               = sb[n, c/G]*qb[n, c] + mb[n, c/G]   otherwise.
 * FFN:  g = W_gate,eff x,  u = W_up,eff x,  h = g / (1 + exp(-g)) * u,  y = W_down h,
 * all in double with no intermediate rounding.  x rows are bf16 bit patterns [T, d];
 * rows[i] selects the token of output row i; out is [n_rows, d] double. */
void orc_expert_ffn(const uint16_t* x, const int32_t* rows, int64_t n_rows, int64_t d, int64_t f, int G,
                    const uint8_t* qg, const uint16_t* sg, const uint16_t* mg,
                    const uint8_t* qu, const uint16_t* su, const uint16_t* mu,
                    const uint8_t* qd, const uint16_t* sd, const uint16_t* md,
                    const uint8_t* q8g, const uint16_t* s8g, const uint16_t* m8g,
                    const uint8_t* q8u, const uint16_t* s8u, const uint16_t* m8u,
                    const uint8_t* mask,
                    const uint8_t* q8d, const uint16_t* s8d, const uint16_t* m8d, const uint8_t* mask_d,
                    double* out) {
    double* h = (double*)malloc(sizeof(double) * (size_t)(n_rows * f > 0 ? n_rows * f : 1));
    double* xd = (double*)malloc(sizeof(double) * (size_t)(n_rows * d > 0 ? n_rows * d : 1));
    for (int64_t i = 0; i < n_rows; ++i)
        for (int64_t c = 0; c < d; ++c) xd[i * d + c] = orc_bf16_to_f64(x[(int64_t)rows[i] * d + c]);
#pragma omp parallel
    {
        double* wg = (double*)malloc(sizeof(double) * (size_t)d);
        double* wu = (double*)malloc(sizeof(double) * (size_t)d);
#pragma omp for schedule(static)
        for (int64_t n = 0; n < f; ++n) {
            for (int64_t c = 0; c < d; ++c) {
                if (mask && mask[c]) {
                    wg[c] = deq(q8g, s8g, m8g, n, c, d, G);
                    wu[c] = deq(q8u, s8u, m8u, n, c, d, G);
                } else {
                    wg[c] = deq(qg, sg, mg, n, c, d, G);
                    wu[c] = deq(qu, su, mu, n, c, d, G);
                }
            }
            for (int64_t i = 0; i < n_rows; ++i) {
                double g = 0.0, u = 0.0;
                const double* xr = xd + i * d;
                for (int64_t c = 0; c < d; ++c) { g += wg[c] * xr[c]; u += wu[c] * xr[c]; }
                h[i * f + n] = g / (1.0 + exp(-g)) * u;
            }
        }
        free(wg);
        free(wu);
        double* wd = (double*)malloc(sizeof(double) * (size_t)f);
#pragma omp for schedule(static)
        for (int64_t n = 0; n < d; ++n) {
            for (int64_t c = 0; c < f; ++c)
                wd[c] = (mask_d && mask_d[c]) ? deq(q8d, s8d, m8d, n, c, f, G) : deq(qd, sd, md, n, c, f, G);
            for (int64_t i = 0; i < n_rows; ++i) {
                double y = 0.0;
                const double* hr = h + i * f;
                for (int64_t c = 0; c < f; ++c) y += wd[c] * hr[c];
                out[i * d + n] = y;
            }
        }
        free(wd);
    }
    free(h);
    free(xd);
}

/* Number of OpenMP threads the FFN loops will use (reported beside timings). */
#ifdef _OPENMP
#include <omp.h>
int orc_threads(void) { return omp_get_max_threads(); }
void orc_set_threads(int n) { omp_set_num_threads(n); }
#else
int orc_threads(void) { return 1; }
void orc_set_threads(int n) { (void)n; }
#endif
