/*
 * CPU oracle for the block-scaled FP8 quantized forward (QaRL, Sec. 2.2 and Sec. 3.1).
 *
 * THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, obviously-correct restatement of what
 * the quantized forward computes, written from the paper's formulas and the e4m3 format
 * definition.  It shares no code with the CUDA path and must never be called from it; only
 * the tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * Parity status: every function below is pinned by tests that do not call this file's own
 * formulas (library casts, closed forms, brute force, exact-arithmetic special cases) except
 * one: the ORDER in which block partial sums are promoted and in which the top-k
 * contributions are added (oracle_linear_q's kb-ascending chain, oracle_combine's
 * ascending-expert chain) is "parity unpinned" by the paper -- App. C only requires that
 * some fixed order be used.  The order chosen here is stated beside each function.
 * Likewise "parity unpinned" by the paper, each stated beside its function: the group size of
 * the two 4-bit weight formats (128 along K), and the router's top-k softmax rule (the paper
 * names a router but gives no formula); what follows from those choices is pinned as above.
 *
 * Build: gcc -O2 -fopenmp -ffp-contract=off -fno-fast-math -shared -fPIC (see oracle/build.py).
 * OpenMP is used over independent rows / experts only, never inside a reduction whose
 * order is specified.
 *
 * Notation follows the paper: s = max|W| / alpha, W_q = [W / s]_FP8, W^ = s * W_q,
 * Y ~= (s_x s_w) (X_q W_q), alpha = 448 for e4m3 (Sec. 2.2, "Floating-point quantization").
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define QBLOCK 128            /* block edge: 128x128 weight blocks, 1x128 activation groups */
#define E4M3_ALPHA 448.0f     /* Sec. 2.2: alpha = 448 for e4m3 => the no-infinity variant  */
#define AMAX_FLOOR 0x1p-40f   /* reading for an all-zero block (paper is silent)            */

/* ---------------------------------------------------------------------------------------
 * bf16 helpers.  bf16 is the upper half of an IEEE fp32.
 * ------------------------------------------------------------------------------------- */
static inline float bf16_to_f32(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* fp32 -> bf16, round to nearest, ties to even. */
uint16_t oracle_bf16_rne(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u); /* NaN */
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

float oracle_bf16_to_f32(uint16_t b) { return bf16_to_f32(b); }

/* ---------------------------------------------------------------------------------------
 * e4m3 ("fn": no infinities, max finite 448 -- fixed by alpha = 448 in Sec. 2.2).
 * code = s eeee mmm.  e = 0: (-1)^s * m * 2^-9.  1 <= e <= 15: (-1)^s * (1 + m/8) * 2^(e-7).
 * 0x7F and 0xFF are NaN.
 * ------------------------------------------------------------------------------------- */
double oracle_e4m3_decode(uint8_t c) {
    int s = c >> 7, e = (c >> 3) & 15, m = c & 7;
    if (e == 15 && m == 7) return NAN;
    double v = (e == 0) ? ldexp((double)m, -9) : ldexp(1.0 + m / 8.0, e - 7);
    return s ? -v : v;
}

/* The code's value as an integer count of 2^-9 (exact; |.| <= 448 * 512 = 229376). */
static inline int32_t e4m3_units(uint8_t c) {
    int s = c >> 7, e = (c >> 3) & 15, m = c & 7;
    int32_t v = (e == 0) ? m : ((8 + m) << (e - 1));
    return s ? -v : v;
}

/* fp32 -> e4m3: round to nearest on the e4m3 grid, ties to the even mantissa code,
 * magnitudes above 448 saturate to +-448, the sign is kept (also for zero / underflow).
 * The paper only writes [.]_FPk ("casting"); rounding and overflow mode are this reading. */
uint8_t oracle_e4m3_encode(float f) {
    if (isnan(f)) return 0x7f;
    uint8_t sign = signbit(f) ? 0x80 : 0x00;
    double a = fabs((double)f);
    if (a > 448.0) return sign | 0x7e;
    if (a < 0x1p-6) {
        /* subnormal grid, spacing 2^-9; q = 8 lands on the smallest normal (code 0x08) */
        int q = (int)nearbyint(ldexp(a, 9));
        return sign | (uint8_t)q;
    }
    int ex;
    (void)frexp(a, &ex);          /* a = f * 2^ex, f in [0.5, 1) => floor(log2 a) = ex - 1 */
    int e_unb = ex - 1;
    int q = (int)nearbyint(ldexp(a, 3 - e_unb));   /* in [8, 16] */
    if (q == 16) { q = 8; e_unb += 1; }
    return sign | (uint8_t)(((e_unb + 7) << 3) | (q - 8));
}

/* Array forms of the two casts (for exhaustive tests). */
void oracle_e4m3_encode_array(const float *v, int64_t n, uint8_t *out) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) out[i] = oracle_e4m3_encode(v[i]);
}

void oracle_bf16_rne_array(const float *v, int64_t n, uint16_t *out) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) out[i] = oracle_bf16_rne(v[i]);
}

/* ---------------------------------------------------------------------------------------
 * Scale and code of one block (Sec. 2.2): s = max|W| / 448, W_q = [W / s]_FP8.
 * Readings where the paper is silent or ambiguous:
 *   - an all-zero block uses amax_c = max(amax, 2^-40);
 *   - W / s is evaluated as W * inv with inv = fl(448 / amax_c), one fp32 multiply per
 *     element; the stored scale is still s = fl(amax_c / 448).
 * ------------------------------------------------------------------------------------- */
static inline float block_scale(float amax, float *inv) {
    float amax_c = amax > AMAX_FLOOR ? amax : AMAX_FLOOR;
    *inv = E4M3_ALPHA / amax_c;
    return amax_c / E4M3_ALPHA;
}

/* W bf16 [E, N, K] -> codes u8 [E, N, K], scales f32 [E, N/128, K/128]; 128x128 blocks. */
int oracle_quantize_weight(const uint16_t *w, int64_t E, int64_t N, int64_t K,
                           uint8_t *codes, float *scales) {
    if (N % QBLOCK || K % QBLOCK) return -2;
    int64_t nb = N / QBLOCK, kb = K / QBLOCK;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t e = 0; e < E; ++e)
        for (int64_t bn = 0; bn < nb; ++bn)
            for (int64_t bk = 0; bk < kb; ++bk) {
                const uint16_t *base = w + (e * N + bn * QBLOCK) * K + bk * QBLOCK;
                float amax = 0.0f;
                for (int r = 0; r < QBLOCK; ++r)
                    for (int c = 0; c < QBLOCK; ++c) {
                        float a = fabsf(bf16_to_f32(base[(int64_t)r * K + c]));
                        if (a > amax) amax = a;
                    }
                float inv;
                float s = block_scale(amax, &inv);
                scales[(e * nb + bn) * kb + bk] = s;
                uint8_t *cb = codes + (e * N + bn * QBLOCK) * K + bk * QBLOCK;
                for (int r = 0; r < QBLOCK; ++r)
                    for (int c = 0; c < QBLOCK; ++c) {
                        float v = bf16_to_f32(base[(int64_t)r * K + c]) * inv;
                        cb[(int64_t)r * K + c] = oracle_e4m3_encode(v);
                    }
            }
    return 0;
}

/* X bf16 [M, K] (row stride ldx elements) -> codes u8 [M, K], scales f32 [M, K/128];
 * 1x128 groups along K. */
int oracle_quantize_act(const uint16_t *x, int64_t M, int64_t K, int64_t ldx,
                        uint8_t *codes, float *scales) {
    if (K % QBLOCK) return -2;
    int64_t kb = K / QBLOCK;
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t g = 0; g < kb; ++g) {
            const uint16_t *base = x + m * ldx + g * QBLOCK;
            float amax = 0.0f;
            for (int c = 0; c < QBLOCK; ++c) {
                float a = fabsf(bf16_to_f32(base[c]));
                if (a > amax) amax = a;
            }
            float inv;
            float s = block_scale(amax, &inv);
            scales[m * kb + g] = s;
            for (int c = 0; c < QBLOCK; ++c)
                codes[m * K + g * QBLOCK + c] = oracle_e4m3_encode(bf16_to_f32(base[c]) * inv);
        }
    return 0;
}

/* ---------------------------------------------------------------------------------------
 * Block-scaled linear (Eq. "Y ~= (s_x s_w)(X_q W_q)" of Sec. 2.2, applied per 128-wide
 * K-block, accumulating in higher precision = fp32):
 *   y[m,n] = sum_kb  fl(s_x[m,kb] * s_w[n/128,kb]) * p[m,n,kb],
 *   p = the EXACT dot product of the 128 code values of the block, rounded once to fp32.
 * Order (parity unpinned by the paper, App. C only asks for a fixed one): acc starts at
 * 0.0f and takes acc = fmaf(sc, p, acc) for kb = 0, 1, 2, ... ascending.
 * The block sum is exact: each code is an integer multiple of 2^-9, so products are
 * integers in units of 2^-18 and 128 of them stay below 2^43.
 *
 * w_row_block_of(n): scale row for weight row n is n / 128.
 * Outputs: y32 (fp32, may be NULL) and y16 (bf16 bits, may be NULL), both [M, N].
 * ------------------------------------------------------------------------------------- */
static void linear_rows(const uint8_t *xc, const float *xs, int64_t M, int64_t K,
                        const uint8_t *wc, const float *ws, int64_t N,
                        float *y32, uint16_t *y16, int64_t ldy) {
    int64_t kb = K / QBLOCK;
    /* decode the weight codes once: int32 units of 2^-9 */
    int32_t *wi = (int32_t *)malloc((size_t)N * K * sizeof(int32_t));
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < N * K; ++i) wi[i] = e4m3_units(wc[i]);
    int32_t *xi = (int32_t *)malloc((size_t)(M > 0 ? M : 1) * K * sizeof(int32_t));
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < M * K; ++i) xi[i] = e4m3_units(xc[i]);
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            float acc = 0.0f;
            const int32_t *xr = xi + m * K;
            const int32_t *wr = wi + n * K;
            for (int64_t b = 0; b < kb; ++b) {
                int64_t isum = 0;
                for (int c = 0; c < QBLOCK; ++c)
                    isum += (int64_t)xr[b * QBLOCK + c] * (int64_t)wr[b * QBLOCK + c];
                float p = (float)ldexp((double)isum, -18);   /* exact, then one rounding */
                float sc = xs[m * kb + b] * ws[(n / QBLOCK) * kb + b];
                acc = fmaf(sc, p, acc);
            }
            if (y32) y32[m * ldy + n] = acc;
            if (y16) y16[m * ldy + n] = oracle_bf16_rne(acc);
        }
    free(xi);
    free(wi);
}

int oracle_linear_q(const uint8_t *xc, const float *xs, int64_t M, int64_t K,
                    const uint8_t *wc, const float *ws, int64_t N,
                    float *y32, uint16_t *y16) {
    if (N % QBLOCK || K % QBLOCK) return -2;
    linear_rows(xc, xs, M, K, wc, ws, N, y32, y16, N);
    return 0;
}

/* y = blockscaled(quantize_act(x), W): the dense projection as one call. */
int oracle_linear(const uint16_t *x, int64_t M, int64_t K,
                  const uint8_t *wc, const float *ws, int64_t N,
                  float *y32, uint16_t *y16) {
    if (N % QBLOCK || K % QBLOCK) return -2;
    uint8_t *xc = (uint8_t *)malloc((size_t)(M > 0 ? M : 1) * K);
    float *xs = (float *)malloc((size_t)(M > 0 ? M : 1) * (K / QBLOCK) * sizeof(float));
    oracle_quantize_act(x, M, K, K, xc, xs);
    linear_rows(xc, xs, M, K, wc, ws, N, y32, y16, N);
    free(xc);
    free(xs);
    return 0;
}

/* ---------------------------------------------------------------------------------------
 * Expert permutation (the grouping step of the routed MoE; not in the paper's text, fixed
 * by the problem statement): flat pair id p = t*k + j; pairs stably sorted by expert id
 * (ties by ascending p).  offsets[e] = first sorted position of expert e, offsets[E] = P.
 * Returns -8 for an id outside [0, E) or the same expert twice in one token.
 * ------------------------------------------------------------------------------------- */
int oracle_permute(const int32_t *ids, int64_t M, int64_t k, int64_t E,
                   int32_t *offsets, int32_t *sorted_pair, int32_t *pos_of_pair) {
    int64_t P = M * k;
    for (int64_t t = 0; t < M; ++t)
        for (int64_t j = 0; j < k; ++j) {
            int32_t e = ids[t * k + j];
            if (e < 0 || e >= E) return -8;
            for (int64_t j2 = 0; j2 < j; ++j2)
                if (ids[t * k + j2] == e) return -8;
        }
    int64_t *count = (int64_t *)calloc((size_t)E + 1, sizeof(int64_t));
    for (int64_t p = 0; p < P; ++p) count[ids[p]]++;
    int64_t run = 0;
    for (int64_t e = 0; e < E; ++e) {
        offsets[e] = (int32_t)run;
        run += count[e];
    }
    offsets[E] = (int32_t)run;
    int64_t *cursor = (int64_t *)malloc((size_t)E * sizeof(int64_t));
    for (int64_t e = 0; e < E; ++e) cursor[e] = offsets[e];
    for (int64_t p = 0; p < P; ++p) {     /* ascending p => stable */
        int64_t pos = cursor[ids[p]]++;
        if (sorted_pair) sorted_pair[pos] = (int32_t)p;
        if (pos_of_pair) pos_of_pair[p] = (int32_t)pos;
    }
    free(count);
    free(cursor);
    return 0;
}

/* ---------------------------------------------------------------------------------------
 * SwiGLU on bf16 operands: h = bf16( silu(g) * u ), silu(g) = g / (1 + exp(-g)), evaluated
 * in double and rounded once to fp32, then to bf16.  g and u are the bf16-rounded gate / up
 * projections (every tensor crossing an op boundary is bf16 -- a reading; the paper does
 * not discuss the activation).  gate_up is [P, 2I] with gate in columns 0..I-1.
 * ------------------------------------------------------------------------------------- */
void oracle_swiglu(const uint16_t *gate_up, int64_t P, int64_t I, uint16_t *h) {
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < P; ++p)
        for (int64_t i = 0; i < I; ++i) {
            double g = (double)bf16_to_f32(gate_up[p * 2 * I + i]);
            double u = (double)bf16_to_f32(gate_up[p * 2 * I + I + i]);
            double v = g / (1.0 + exp(-g)) * u;
            h[p * I + i] = oracle_bf16_rne((float)v);
        }
}


/* ---------------------------------------------------------------------------------------
 * Backward of SwiGLU on the bf16 gate / up saved by the forward: with s = 1 / (1 + exp(-g)),
 *   dG = dH * u * s * (1 + g (1 - s)),   dU = dH * g * s,
 * evaluated in double, rounded once to fp32 and then to bf16.  dgu is [P, 2I], gate part first.
 * ------------------------------------------------------------------------------------- */
void oracle_swiglu_bwd(const uint16_t *gate_up, const uint16_t *dh, int64_t P, int64_t I, uint16_t *dgu) {
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < P; ++p)
        for (int64_t i = 0; i < I; ++i) {
            double g = (double)bf16_to_f32(gate_up[p * 2 * I + i]);
            double u = (double)bf16_to_f32(gate_up[p * 2 * I + I + i]);
            double d = (double)bf16_to_f32(dh[p * I + i]);
            double s = 1.0 / (1.0 + exp(-g));
            dgu[p * 2 * I + i] = oracle_bf16_rne((float)(d * u * s * (1.0 + g * (1.0 - s))));
            dgu[p * 2 * I + I + i] = oracle_bf16_rne((float)(d * g * s));
        }
}

/* ---------------------------------------------------------------------------------------
 * Top-k weighted combine.  For token t the k contributions are visited in ASCENDING EXPERT
 * ID (a canonical order that does not depend on the caller's slot order; parity unpinned
 * by the paper):  c_j = bf16( fl(w[t,j] * y32_j) );  sum = 0.0f; sum += float(c_j);
 * out = bf16(sum).   y32 is [P, H] indexed by flat pair id p = t*k + j.
 * ------------------------------------------------------------------------------------- */
void oracle_combine(const float *y32, const int32_t *ids, const float *wts,
                    int64_t M, int64_t k, int64_t H, uint16_t *out) {
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < M; ++t) {
        int64_t order[64];
        for (int64_t j = 0; j < k; ++j) order[j] = j;
        for (int64_t a = 1; a < k; ++a) {            /* insertion sort by expert id */
            int64_t v = order[a], b = a;
            while (b > 0 && ids[t * k + order[b - 1]] > ids[t * k + v]) {
                order[b] = order[b - 1];
                --b;
            }
            order[b] = v;
        }
        for (int64_t c = 0; c < H; ++c) {
            float sum = 0.0f;
            for (int64_t a = 0; a < k; ++a) {
                int64_t j = order[a];
                float cj = bf16_to_f32(oracle_bf16_rne(wts[t * k + j] * y32[(t * k + j) * H + c]));
                sum = sum + cj;
            }
            out[t * H + c] = oracle_bf16_rne(sum);
        }
    }
}

/* ---------------------------------------------------------------------------------------
 * One routed MoE FFN layer on quantized weights, per pair p = (t, j) with expert e:
 *   x_q          = quantize_act(x[t])                         (1x128 groups along H)
 *   gate_up[p]   = bf16( blockscaled(x_q, W13_e) )            [2I]
 *   h[p]         = swiglu(gate_up[p])                         [I], bf16
 *   h_q          = quantize_act(h[p])                         (1x128 groups along I)
 *   y32[p]       = blockscaled(h_q, W2_e)                     [H], fp32
 *   out[t]       = combine over the token's k pairs
 * w13 codes [E, 2I, H] (rows 0..I-1 gate, I..2I-1 up; scale blocks over the concatenated
 * [2I, H] matrix), w2 codes [E, H, I].
 * Optional dumps (NULL to skip), all indexed by flat pair id p = t*k + j:
 *   d_gate_up bf16 [P, 2I], d_h bf16 [P, I], d_hc u8 [P, I], d_hs f32 [P, I/128],
 *   d_y32 f32 [P, H].
 * ------------------------------------------------------------------------------------- */
int oracle_moe(const uint16_t *x, const int32_t *ids, const float *wts,
               int64_t M, int64_t H, int64_t I, int64_t E, int64_t k,
               const uint8_t *w13c, const float *w13s, const uint8_t *w2c, const float *w2s,
               uint16_t *out, uint16_t *d_gate_up, uint16_t *d_h, uint8_t *d_hc, float *d_hs,
               float *d_y32) {
    if (H % QBLOCK || I % QBLOCK || k > 64) return -2;
    int64_t P = M * k;
    int32_t *offsets = (int32_t *)malloc(((size_t)E + 1) * sizeof(int32_t));
    int32_t *sorted = (int32_t *)malloc((size_t)(P > 0 ? P : 1) * sizeof(int32_t));
    int rc = oracle_permute(ids, M, k, E, offsets, sorted, NULL);
    if (rc) { free(offsets); free(sorted); return rc; }

    int64_t hb = H / QBLOCK, ib = I / QBLOCK;
    size_t Pn = (size_t)(P > 0 ? P : 1), Mn = (size_t)(M > 0 ? M : 1);
    uint8_t *xc = (uint8_t *)malloc(Mn * H);
    float *xs = (float *)malloc(Mn * hb * sizeof(float));
    oracle_quantize_act(x, M, H, H, xc, xs);

    uint16_t *gate_up = d_gate_up ? d_gate_up : (uint16_t *)malloc(Pn * 2 * I * sizeof(uint16_t));
    uint16_t *h = d_h ? d_h : (uint16_t *)malloc(Pn * I * sizeof(uint16_t));
    uint8_t *hc = d_hc ? d_hc : (uint8_t *)malloc(Pn * I);
    float *hs = d_hs ? d_hs : (float *)malloc(Pn * ib * sizeof(float));
    float *y32 = d_y32 ? d_y32 : (float *)malloc(Pn * H * sizeof(float));

    /* gate_up, one expert group at a time (rows gathered into a contiguous scratch) */
    for (int64_t e = 0; e < E; ++e) {
        int64_t g0 = offsets[e], g1 = offsets[e + 1], G = g1 - g0;
        if (G == 0) continue;
        uint8_t *gc = (uint8_t *)malloc((size_t)G * H);
        float *gs = (float *)malloc((size_t)G * hb * sizeof(float));
        uint16_t *gy = (uint16_t *)malloc((size_t)G * 2 * I * sizeof(uint16_t));
        for (int64_t r = 0; r < G; ++r) {
            int64_t t = sorted[g0 + r] / k;
            memcpy(gc + r * H, xc + t * H, (size_t)H);
            memcpy(gs + r * hb, xs + t * hb, (size_t)hb * sizeof(float));
        }
        linear_rows(gc, gs, G, H, w13c + e * 2 * I * H, w13s + e * (2 * I / QBLOCK) * hb,
                    2 * I, NULL, gy, 2 * I);
        for (int64_t r = 0; r < G; ++r)
            memcpy(gate_up + (int64_t)sorted[g0 + r] * 2 * I, gy + r * 2 * I,
                   (size_t)2 * I * sizeof(uint16_t));
        free(gc); free(gs); free(gy);
    }
    oracle_swiglu(gate_up, P, I, h);
    oracle_quantize_act(h, P, I, I, hc, hs);
    for (int64_t e = 0; e < E; ++e) {
        int64_t g0 = offsets[e], g1 = offsets[e + 1], G = g1 - g0;
        if (G == 0) continue;
        uint8_t *gc = (uint8_t *)malloc((size_t)G * I);
        float *gs = (float *)malloc((size_t)G * ib * sizeof(float));
        float *gy = (float *)malloc((size_t)G * H * sizeof(float));
        for (int64_t r = 0; r < G; ++r) {
            int64_t p = sorted[g0 + r];
            memcpy(gc + r * I, hc + p * I, (size_t)I);
            memcpy(gs + r * ib, hs + p * ib, (size_t)ib * sizeof(float));
        }
        linear_rows(gc, gs, G, I, w2c + e * H * I, w2s + e * hb * ib, H, gy, NULL, H);
        for (int64_t r = 0; r < G; ++r)
            memcpy(y32 + (int64_t)sorted[g0 + r] * H, gy + r * H, (size_t)H * sizeof(float));
        free(gc); free(gs); free(gy);
    }
    oracle_combine(y32, ids, wts, M, k, H, out);

    if (!d_gate_up) free(gate_up);
    if (!d_h) free(h);
    if (!d_hc) free(hc);
    if (!d_hs) free(hs);
    if (!d_y32) free(y32);
    free(xc); free(xs); free(offsets); free(sorted);
    return 0;
}

/* =======================================================================================
 * W4A16: 4-bit integer weight-only quantization (Sec. 2.2, "Integer quantization"), the format
 * the paper's headline results use (Sec. 3.1 item 1: W4A16 for larger MoE models).
 *   Quant:   W_q = clamp( round(W / s) + z, q_min, q_max ),   Dequant:  W^ = s (W_q - z)
 * Readings where the paper is silent: unsigned 4-bit codes (q_min = 0, q_max = 15); one
 * (s, z) per group of 128 consecutive K elements of one weight row (the group size is not in the
 * paper: "parity unpinned" on this point, for this format and the FP4 one below); asymmetric min/max
 * calibration with zero kept representable: lo = min(0, min W), hi = max(0, max W),
 * s = bf16( fl(max(hi - lo, 2^-40) / 15) ) -- the group scale is kept in the model's 16-bit type,
 * as W4A16 checkpoints store it, and is returned here as the fp32 of that bf16 value --
 * z = clamp(rint(-lo / s), 0, 15); round() is round to nearest, ties to even; W / s and -lo / s
 * are IEEE fp32 divisions by that stored s.  The GEMM consumes the dequantized weight rounded
 * to bf16, w^ = bf16( s * (W_q - z) ): s has 8 significant bits and |W_q - z| <= 15, so the
 * product is exact before its one rounding.  Activations stay bf16 ("A16"), accumulation is
 * higher precision (fp32).
 * Packed layout: byte j of a row holds code 2j in its low nibble and code 2j+1 in its high nibble.
 * ===================================================================================== */
int oracle_quantize_weight_w4(const uint16_t *w, int64_t E, int64_t N, int64_t K,
                              uint8_t *packed, float *scales, uint8_t *zeros) {
    if (K % QBLOCK) return -2;
    int64_t kb = K / QBLOCK;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < E * N; ++r)
        for (int64_t g = 0; g < kb; ++g) {
            const uint16_t *base = w + r * K + g * QBLOCK;
            float lo = 0.0f, hi = 0.0f;
            for (int c = 0; c < QBLOCK; ++c) {
                float v = bf16_to_f32(base[c]);
                if (v < lo) lo = v;
                if (v > hi) hi = v;
            }
            float range = hi - lo;
            if (range < AMAX_FLOOR) range = AMAX_FLOOR;
            float s = bf16_to_f32(oracle_bf16_rne(range / 15.0f));
            float zf = nearbyintf(-lo / s);
            if (zf < 0.0f) zf = 0.0f;
            if (zf > 15.0f) zf = 15.0f;
            scales[r * kb + g] = s;
            zeros[r * kb + g] = (uint8_t)zf;
            for (int c = 0; c < QBLOCK; c += 2) {
                int q[2];
                for (int t = 0; t < 2; ++t) {
                    float v = nearbyintf(bf16_to_f32(base[c + t]) / s) + zf;
                    if (v < 0.0f) v = 0.0f;
                    if (v > 15.0f) v = 15.0f;
                    q[t] = (int)v;
                }
                packed[r * (K / 2) + (g * QBLOCK + c) / 2] = (uint8_t)(q[0] | (q[1] << 4));
            }
        }
    return 0;
}

/* w^ bf16 bits [rows, K] from packed codes, scales and zeros (rows = E*N). */
void oracle_dequant_w4(const uint8_t *packed, const float *scales, const uint8_t *zeros,
                       int64_t rows, int64_t K, uint16_t *w_hat) {
    int64_t kb = K / QBLOCK;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t k = 0; k < K; ++k) {
            uint8_t b = packed[r * (K / 2) + k / 2];
            int q = (k & 1) ? (b >> 4) : (b & 15);
            float s = scales[r * kb + k / QBLOCK];
            int z = zeros[r * kb + k / QBLOCK];
            w_hat[r * K + k] = oracle_bf16_rne(s * (float)(q - z));
        }
}

/* =======================================================================================
 * FP4 (e2m1) weight-only quantization (Sec. 2.2, "Floating-point quantization"):
 *   s = max|W| / alpha,   W_q = [W / s]_FP4,   W^ = s * W_q,   alpha = 6 (largest finite e2m1 value).
 * An e2m1 code has a sign bit (bit 3), two exponent bits (bits 2..1, bias 1) and one mantissa
 * bit (bit 0); exponent field 0 is subnormal.  The eight magnitudes are 0, 0.5, 1, 1.5, 2, 3, 4, 6;
 * there is no infinity and no NaN.
 * Readings where the paper is silent (the same ones as for the integer format, so that the two
 * 4-bit formats share storage and GEMM): one s per group of 128 consecutive K elements of one
 * weight row; s = bf16( fl(max(amax, 2^-40) / 6) ), returned as the fp32 of that bf16 value;
 * W / s is an IEEE fp32 division by the stored s; [.]_FP4 rounds to the nearest representable
 * value, ties to the even code, and saturates at +-6; zero keeps the sign of W (code 8 for -0
 * and for negative values that round to zero: it decodes to -0 = 0).  The GEMM consumes
 * w^ = bf16(s * value): the value has two significant bits and s eight, so the product is exact
 * before its one rounding.
 * Packed layout as for the integer format: byte j of a row holds code 2j in its low nibble.
 * ===================================================================================== */
static const float E2M1_MAGNITUDES[8] = {0.0f, 0.5f, 1.0f, 1.5f, 2.0f, 3.0f, 4.0f, 6.0f};

double oracle_e2m1_decode(uint8_t code) {
    int ee = (code >> 1) & 3, m = code & 1;
    double mag = ee ? ldexp(1.0 + 0.5 * m, ee - 1) : 0.5 * m;
    return (code & 8) ? -mag : mag;
}

/* Round a finite fp32 to e2m1: nearest magnitude, ties to the even code, saturating. */
uint8_t oracle_e2m1_encode(float f) {
    uint8_t sign = signbit(f) ? 8 : 0;
    double a = fabs((double)f);
    int best = 7;                                   /* everything at or above 6 saturates */
    for (int c = 0; c < 7; ++c) {
        double lo = E2M1_MAGNITUDES[c], hi = E2M1_MAGNITUDES[c + 1];
        if (a > hi) continue;
        double dl = a - lo, dh = hi - a;            /* a in [lo, hi]: both exact in double */
        if (dl < dh) best = c;
        else if (dl > dh) best = c + 1;
        else best = (c & 1) ? c + 1 : c;            /* tie: the code with mantissa bit 0 */
        break;
    }
    return (uint8_t)(sign | best);
}

int oracle_quantize_weight_fp4(const uint16_t *w, int64_t E, int64_t N, int64_t K,
                               uint8_t *packed, float *scales) {
    if (K % QBLOCK) return -2;
    int64_t kb = K / QBLOCK;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < E * N; ++r)
        for (int64_t g = 0; g < kb; ++g) {
            const uint16_t *base = w + r * K + g * QBLOCK;
            float amax = 0.0f;
            for (int c = 0; c < QBLOCK; ++c) {
                float v = fabsf(bf16_to_f32(base[c]));
                if (v > amax) amax = v;
            }
            if (amax < AMAX_FLOOR) amax = AMAX_FLOOR;
            float s = bf16_to_f32(oracle_bf16_rne(amax / 6.0f));
            scales[r * kb + g] = s;
            for (int c = 0; c < QBLOCK; c += 2) {
                uint8_t q0 = oracle_e2m1_encode(bf16_to_f32(base[c]) / s);
                uint8_t q1 = oracle_e2m1_encode(bf16_to_f32(base[c + 1]) / s);
                packed[r * (K / 2) + (g * QBLOCK + c) / 2] = (uint8_t)(q0 | (q1 << 4));
            }
        }
    return 0;
}

/* w^ bf16 bits [rows, K] from packed e2m1 codes and group scales (rows = E*N). */
void oracle_dequant_fp4(const uint8_t *packed, const float *scales, int64_t rows, int64_t K,
                        uint16_t *w_hat) {
    int64_t kb = K / QBLOCK;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t k = 0; k < K; ++k) {
            uint8_t b = packed[r * (K / 2) + k / 2];
            uint8_t q = (k & 1) ? (b >> 4) : (b & 15);
            float s = scales[r * kb + k / QBLOCK];
            w_hat[r * K + k] = oracle_bf16_rne(s * (float)oracle_e2m1_decode(q));
        }
}

/* y[m,n] = sum_k x[m,k] * w^[n,k]: bf16 operands, products and sum exact in double (each
 * product has <= 16 significant bits), rounded once to fp32, then to bf16.  The paper asks
 * only for "higher precision" accumulation; the GPU's tensor-core order is compared with this
 * ideal within the stated tolerance. */
void oracle_linear_bf16(const uint16_t *x, int64_t M, int64_t K, const uint16_t *w_hat, int64_t N,
                        float *y32, uint16_t *y16) {
    float *wf = (float *)malloc((size_t)N * K * sizeof(float));
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < N * K; ++i) wf[i] = bf16_to_f32(w_hat[i]);
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int64_t k = 0; k < K; ++k)
                acc += (double)bf16_to_f32(x[m * K + k]) * (double)wf[n * K + k];
            float a = (float)acc;
            if (y32) y32[m * N + n] = a;
            if (y16) y16[m * N + n] = oracle_bf16_rne(a);
        }
    free(wf);
}

/* One routed MoE FFN layer with W4A16 weights: activations stay bf16 between the GEMMs.
 *   gate_up[p] = bf16( x[t] . W13^_e ),  h[p] = swiglu(gate_up[p]),  y32[p] = h[p] . W2^_e (fp32),
 *   out[t] = combine (same rule as the FP8 layer).  w13_hat [E, 2I, H], w2_hat [E, H, I] bf16. */
int oracle_moe_w4a16(const uint16_t *x, const int32_t *ids, const float *wts,
                     int64_t M, int64_t H, int64_t I, int64_t E, int64_t k,
                     const uint16_t *w13_hat, const uint16_t *w2_hat, uint16_t *out,
                     uint16_t *d_gate_up, uint16_t *d_h, float *d_y32) {
    if (k > 64) return -2;
    int64_t P = M * k;
    for (int64_t p = 0; p < P; ++p)
        if (ids[p] < 0 || ids[p] >= E) return -8;
    size_t Pn = (size_t)(P > 0 ? P : 1);
    uint16_t *gate_up = d_gate_up ? d_gate_up : (uint16_t *)malloc(Pn * 2 * I * sizeof(uint16_t));
    uint16_t *h = d_h ? d_h : (uint16_t *)malloc(Pn * I * sizeof(uint16_t));
    float *y32 = d_y32 ? d_y32 : (float *)malloc(Pn * H * sizeof(float));
    for (int64_t p = 0; p < P; ++p) {
        int64_t t = p / k, e = ids[p];
        oracle_linear_bf16(x + t * H, 1, H, w13_hat + e * 2 * I * H, 2 * I, NULL, gate_up + p * 2 * I);
    }
    oracle_swiglu(gate_up, P, I, h);
    for (int64_t p = 0; p < P; ++p) {
        int64_t e = ids[p];
        oracle_linear_bf16(h + p * I, 1, I, w2_hat + e * H * I, H, y32 + p * H, NULL);
    }
    oracle_combine(y32, ids, wts, M, k, H, out);
    if (!d_gate_up) free(gate_up);
    if (!d_h) free(h);
    if (!d_y32) free(y32);
    return 0;
}


/* =======================================================================================
 * Training-side backward of a quantized linear layer (Sec. 3.1 item 2: the forward runs in low
 * bit, the backward in full precision; gradients pass the quantizer by the straight-through
 * estimator and are applied to the bf16 master weights).  Reading: with y = x . W^T computed on
 * Quant(W), the backward treats Quant as the identity and uses the bf16 masters themselves:
 *   dX[m,k] = sum_n dY[m,n] W[n,k]      dW[n,k] = sum_m dY[m,n] X[m,k]
 * bf16 operands; every product and the whole sum exact in double, rounded once to fp32
 * (dX additionally to bf16, dW stays fp32 as the gradient a master-weight optimizer consumes).
 * ===================================================================================== */
void oracle_linear_bwd(const uint16_t *dy, const uint16_t *x, const uint16_t *w,
                       int64_t M, int64_t N, int64_t K, float *dx32, uint16_t *dx16, float *dw32) {
    float *dyf = (float *)malloc((size_t)(M > 0 ? M : 1) * N * sizeof(float));
    for (int64_t i = 0; i < M * N; ++i) dyf[i] = bf16_to_f32(dy[i]);
    if (dx32 || dx16) {
#pragma omp parallel for schedule(static)
        for (int64_t m = 0; m < M; ++m)
            for (int64_t k = 0; k < K; ++k) {
                double acc = 0.0;
                for (int64_t n = 0; n < N; ++n)
                    acc += (double)dyf[m * N + n] * (double)bf16_to_f32(w[n * K + k]);
                float a = (float)acc;
                if (dx32) dx32[m * K + k] = a;
                if (dx16) dx16[m * K + k] = oracle_bf16_rne(a);
            }
    }
    if (dw32) {
#pragma omp parallel for schedule(static)
        for (int64_t n = 0; n < N; ++n)
            for (int64_t k = 0; k < K; ++k) {
                double acc = 0.0;
                for (int64_t m = 0; m < M; ++m)
                    acc += (double)dyf[m * N + n] * (double)bf16_to_f32(x[m * K + k]);
                dw32[n * K + k] = (float)acc;
            }
    }
    free(dyf);
}


/* =======================================================================================
 * TBPO: the sequence-level surrogate of Sec. 3.2 ("Trust Band Policy Optimization"; ratio and
 * weight as written out in the appendix "Detail of TBPO").  For a response o of L tokens:
 *   a = (1/L) sum_t (log pi_current-learner - log pi_old-learner)(o_t),  r = exp(a)   (r_seq-prox)
 *   b = (1/L) sum_t (log pi_old-learner - log pi_old-sampler)(o_t),      w = exp(b)   (w_seq-mismatch)
 *   w~ = two-sided cap of w with c > 1 (Eq. "tis");  r~ = clip(r, 0, 1 + eps_h) if A >= 0,
 *   clip(r, 1 - delta_l, 1 + delta_h) if A < 0 (Eq. "clip");  J = w~ r~ A.
 * Readings: the cap is printed as clip(w, [-log c, log c]): taken in the log domain, i.e.
 * w~ = exp(clip(b, -log c, log c)) in [1/c, c].  The batch objective is the mean of J over the B
 * responses (the expectation over sampled responses), loss = -mean J.  A clipped r~ is a constant:
 * the response then sends no gradient (the paper's "mask out the entire response"); bounds are
 * inclusive (lo <= r <= hi passes the gradient).  w~ carries no gradient (neither old policy depends
 * on theta).  Gradient of the loss with respect to every token log-prob of the current learner in
 * response i:  -(1/B) w~ A r / L  if r is inside its band, else 0.  An empty response (L = 0)
 * contributes J = 0 and still counts in B.  All arithmetic in double on fp32 inputs; the token
 * differences are formed in double, summed in token order.
 * flags: bit 0 = r outside its band (no gradient), bit 1 = w capped, bit 2 = empty response.
 * ===================================================================================== */
void oracle_tbpo(const float *lp_cur, const float *lp_old_learner, const float *lp_old_sampler,
                 const int64_t *offsets, const float *adv, int64_t B,
                 double eps_h, double delta_l, double delta_h, double cap,
                 double *r_seq, double *w_seq, double *j_seq, int32_t *flags, float *grad, double *loss) {
    double total = 0.0;
    double logc = log(cap);
    for (int64_t i = 0; i < B; ++i) {
        int64_t t0 = offsets[i], t1 = offsets[i + 1], L = t1 - t0;
        if (L <= 0) {
            r_seq[i] = 1.0; w_seq[i] = 1.0; j_seq[i] = 0.0; flags[i] = 4;
            continue;
        }
        double sa = 0.0, sb = 0.0;
        for (int64_t t = t0; t < t1; ++t) {
            sa += (double)lp_cur[t] - (double)lp_old_learner[t];
            sb += (double)lp_old_learner[t] - (double)lp_old_sampler[t];
        }
        double a = sa / (double)L, b = sb / (double)L;
        double r = exp(a), w = exp(b);
        int f = 0;
        double bc = b;
        if (bc > logc) { bc = logc; f |= 2; }
        if (bc < -logc) { bc = -logc; f |= 2; }
        double wt = exp(bc);
        double A = (double)adv[i];
        double lo = A >= 0.0 ? 0.0 : 1.0 - delta_l;
        double hi = A >= 0.0 ? 1.0 + eps_h : 1.0 + delta_h;
        double rt = r;
        if (rt < lo) { rt = lo; f |= 1; }
        if (rt > hi) { rt = hi; f |= 1; }
        double J = wt * rt * A;
        r_seq[i] = r; w_seq[i] = w; j_seq[i] = J; flags[i] = f;
        total += J;
        if (grad) {
            float g = (f & 1) ? 0.0f : (float)(-(wt * A * r) / ((double)L * (double)B));
            for (int64_t t = t0; t < t1; ++t) grad[t] = g;
        }
    }
    *loss = B > 0 ? -total / (double)B : 0.0;
}


/* =======================================================================================
 * Router of the MoE block ("router shift", Sec. 4.2: the routing decision is part of the forward
 * the sampler and the learner must agree on).  The paper gives no formula; reading (the common
 * top-k softmax router of the Qwen3-MoE family the paper trains): logits = x . W_r^T on bf16
 * operands (exact sum, rounded once to fp32); the k largest logits of a token, ties to the lower
 * expert id, in descending order; weights = softmax over the k selected fp32 logits (exp of
 * logit - max in double, normalised, rounded to fp32).  The router stays in bf16: it is not
 * quantized.  The rule itself is "parity unpinned" (nothing in the paper fixes it); the tests pin what
 * the rule implies (sorted selection, ties, weights summing to one, the softmax closed form).
 * ===================================================================================== */
void oracle_router_topk(const float *logits, int64_t M, int64_t E, int64_t k, int32_t *ids, float *wts) {
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        const float *l = logits + m * E;
        char *taken = (char *)calloc((size_t)E, 1);
        double mx = 0.0, den = 0.0;
        for (int64_t j = 0; j < k; ++j) {
            int64_t best = -1;
            for (int64_t e = 0; e < E; ++e)
                if (!taken[e] && (best < 0 || l[e] > l[best])) best = e;   /* strict >: ties keep the lower id */
            taken[best] = 1;
            ids[m * k + j] = (int32_t)best;
            if (j == 0) mx = (double)l[best];
        }
        for (int64_t j = 0; j < k; ++j) den += exp((double)l[ids[m * k + j]] - mx);
        for (int64_t j = 0; j < k; ++j) wts[m * k + j] = (float)(exp((double)l[ids[m * k + j]] - mx) / den);
        free(taken);
    }
}

/* Number of OpenMP threads the oracle will use (reported beside its timing). */
#ifdef _OPENMP
#include <omp.h>
int oracle_num_threads(void) { return omp_get_max_threads(); }
#else
int oracle_num_threads(void) { return 1; }
#endif
