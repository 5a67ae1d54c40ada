/*
 * CPU oracle for the HyQuant prefill path.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 restatement of what the paper defines:
 *   - vertical-line token identification          (Algorithm 1)
 *   - per-tile symmetric quantization             (Algorithm 2, Stage 2)
 *   - hybrid-precision causal attention           (Eq. 6-7; Algorithm 2, Stage 3)
 * It shares no code with the CUDA library and is only ever called by the test
 * suite, the smoke check and the CPU-baseline leg of the benchmark.
 *
 * Every function below is pinned by CPU tests against something other than
 * itself (library routines, brute force, closed forms); nothing here is
 * "parity unpinned".
 *
 * Conventions: tensors are contiguous row-major, Q [B,Hq,L,D], K/V [B,Hkv,L,D];
 * bf16 values arrive as their 16-bit patterns; kv(h) = h / (Hq/Hkv).
 * Build: gcc -O2 -fopenmp -ffp-contract=off (no -ffast-math).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { FMT_INT8 = 0, FMT_FP8_E4M3 = 1, FMT_INT4 = 2 };

static inline float bf16_to_f32(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* ------------------------------------------------------------------------- */
/* FP8 e4m3 ("fn": no infinities, max finite 448), written from the format's  */
/* definition: 1 sign, 4 exponent (bias 7), 3 mantissa bits, subnormals with  */
/* step 2^-9.                                                                 */
/* ------------------------------------------------------------------------- */

/* value of an e4m3 byte (NaN patterns never produced by the encoder) */
static double e4m3_value(uint8_t c) {
    int sign = c >> 7, e = (c >> 3) & 0xF, m = c & 7;
    double v = (e == 0) ? ldexp((double)m, -9) : ldexp(1.0 + m / 8.0, e - 7);
    return sign ? -v : v;
}

/* round-to-nearest-even onto the e4m3 grid, saturating at +-448, sign kept */
static uint8_t e4m3_encode_rne_sat(float y) {
    uint8_t sign = signbit(y) ? 0x80 : 0;
    double a = fabs((double)y);
    if (!(a < 448.0)) return sign | 0x7E;                   /* saturate (0x7E = 448) */
    if (a == 0.0) return sign;
    int ex;
    frexp(a, &ex);                                          /* a = f * 2^ex, f in [0.5,1) */
    int e = ex - 1;                                         /* a in [2^e, 2^(e+1)) */
    if (e < -6) e = -6;                                     /* subnormal range shares the 2^-9 step */
    double step = ldexp(1.0, e - 3);
    double n = nearbyint(a / step);                         /* default mode: ties to even; a/step exact */
    double r = n * step;
    if (r > 448.0) r = 448.0;
    /* re-derive fields from the rounded value */
    if (r < ldexp(1.0, -6)) return sign | (uint8_t)(r / ldexp(1.0, -9));
    frexp(r, &ex);
    e = ex - 1;
    int m = (int)((r / ldexp(1.0, e) - 1.0) * 8.0);
    return sign | (uint8_t)(((e + 7) << 3) | m);
}

/* ------------------------------------------------------------------------- */
/* Algorithm 2, Stage 2: per-tile quantization.                               */
/* One tile = block_tokens consecutive tokens x all D channels of one head,   */
/* cut by original position (ragged last tile allowed).                       */
/*   scale = absmax / c,  code = round(x * (c / absmax))                      */
/* c = 127 (INT8), 448 (FP8 e4m3), 7 (INT4).  fp32 arithmetic, one rounding   */
/* per operation, round-half-to-even.  A tile with absmax < 2^-100 gets scale */
/* 0 and all-zero codes.  INT4: two's-complement nibbles, even channel low.   */
/* ------------------------------------------------------------------------- */
int oracle_quantize(const uint16_t* x, int B, int H, int L, int D, int block_tokens,
                    int fmt, uint8_t* codes, float* scales) {
    if (fmt != FMT_INT8 && fmt != FMT_FP8_E4M3 && fmt != FMT_INT4) return 1;
    if (fmt == FMT_INT4 && (D & 1)) return 1;
    const float c = (fmt == FMT_INT8) ? 127.0f : (fmt == FMT_FP8_E4M3) ? 448.0f : 7.0f;
    const int nb = (L + block_tokens - 1) / block_tokens;
    const long row_bytes = (fmt == FMT_INT4) ? D / 2 : D;
#pragma omp parallel for collapse(2) schedule(static)
    for (long bh = 0; bh < (long)B * H; ++bh) {
        for (int n = 0; n < nb; ++n) {
            const int t0 = n * block_tokens;
            const int t1 = (t0 + block_tokens < L) ? t0 + block_tokens : L;
            const uint16_t* xb = x + (bh * L + t0) * (long)D;
            float amax = 0.0f;
            for (long e = 0; e < (long)(t1 - t0) * D; ++e) {
                float a = fabsf(bf16_to_f32(xb[e]));
                if (a > amax) amax = a;
            }
            const int dead = !(amax >= 0x1p-100f);
            volatile float scale_v = dead ? 0.0f : amax / c;   /* volatile: one fp32 rounding each */
            volatile float inv_v = dead ? 0.0f : c / amax;
            const float inv = inv_v;
            scales[bh * nb + n] = scale_v;
            for (int t = t0; t < t1; ++t) {
                const uint16_t* xr = x + (bh * L + t) * (long)D;
                uint8_t* cr = codes + (bh * L + t) * row_bytes;
                if (fmt == FMT_INT4) memset(cr, 0, (size_t)row_bytes);
                for (int d = 0; d < D; ++d) {
                    volatile float y_v = bf16_to_f32(xr[d]) * inv;
                    const float y = y_v;
                    if (fmt == FMT_FP8_E4M3) {
                        cr[d] = dead ? 0 : e4m3_encode_rne_sat(y);
                    } else {
                        int q = dead ? 0 : (int)nearbyintf(y);
                        if (q > (int)c) q = (int)c;
                        if (q < -(int)c) q = -(int)c;
                        if (fmt == FMT_INT8) cr[d] = (uint8_t)(int8_t)q;
                        else cr[d >> 1] |= (uint8_t)((q & 0xF) << ((d & 1) * 4));
                    }
                }
            }
        }
    }
    return 0;
}

/* dequantized value of channel d of a code row: code * scale, exact in fp64 */
static inline double dequant(const uint8_t* row, int d, int fmt, double scale) {
    if (fmt == FMT_INT8) return (double)(int8_t)row[d] * scale;
    if (fmt == FMT_FP8_E4M3) return e4m3_value(row[d]) * scale;
    int nib = (row[d >> 1] >> ((d & 1) * 4)) & 0xF;
    if (nib >= 8) nib -= 16;
    return (double)nib * scale;
}

/* ------------------------------------------------------------------------- */
/* Algorithm 1: vertical token identification.                                */
/*   P = max(0, Lk - W); empty result when P = 0 (or k = 0)                   */
/*   t = n_tail, or min(W, Lq) when n_tail = 0                                */
/*   qbar = mean of the last t query rows (fp64 sum in row order, one divide) */
/*   S[p] = qbar . K[kv(h), p, :]  for p in [0, P)   (fp64 fma chain over d)  */
/*   keep the k largest; equal scores: the lower position wins; the set is    */
/*   written in ascending position order.                                     */
/* ------------------------------------------------------------------------- */
typedef struct { double s; int p; } scored_t;

static int cmp_scored(const void* a, const void* b) {
    const scored_t* x = (const scored_t*)a;
    const scored_t* y = (const scored_t*)b;
    if (x->s > y->s) return -1;
    if (x->s < y->s) return 1;
    return (x->p > y->p) - (x->p < y->p);
}
static int cmp_int(const void* a, const void* b) {
    int x = *(const int*)a, y = *(const int*)b;
    return (x > y) - (x < y);
}

int oracle_select(const uint16_t* q, const uint16_t* k_, int B, int Hq, int Hkv, int Lq, int Lk,
                  int D, int W, int n_tail, int k, int32_t* idx_out, double* scores_out) {
    if (Hkv <= 0 || Hq % Hkv) return 1;
    const int g = Hq / Hkv;
    const int P = (Lk - W > 0) ? Lk - W : 0;
    if (P == 0 || k == 0) return 0;
    if (k > P || k < 0) return 1;
    const int t = n_tail ? n_tail : (W < Lq ? W : Lq);
    if (t <= 0 || t > Lq) return 1;
    int err = 0;
#pragma omp parallel for schedule(dynamic)
    for (int bh = 0; bh < B * Hq; ++bh) {
        const int b = bh / Hq, h = bh % Hq, kvh = h / g;
        double* qbar = (double*)malloc(sizeof(double) * D);
        scored_t* sc = (scored_t*)malloc(sizeof(scored_t) * P);
        if (!qbar || !sc) { err = 2; free(qbar); free(sc); continue; }
        for (int d = 0; d < D; ++d) {
            double sum = 0.0;
            for (int i = Lq - t; i < Lq; ++i)
                sum += (double)bf16_to_f32(q[(((long)b * Hq + h) * Lq + i) * D + d]);
            qbar[d] = sum / (double)t;
        }
        for (int p = 0; p < P; ++p) {
            const uint16_t* kr = k_ + (((long)b * Hkv + kvh) * Lk + p) * D;
            double s = 0.0;
            for (int d = 0; d < D; ++d) s = fma(qbar[d], (double)bf16_to_f32(kr[d]), s);
            sc[p].s = s;
            sc[p].p = p;
            if (scores_out) scores_out[(long)bh * P + p] = s;
        }
        qsort(sc, P, sizeof(scored_t), cmp_scored);
        int32_t* out = idx_out + (long)bh * k;
        for (int c = 0; c < k; ++c) out[c] = sc[c].p;
        qsort(out, k, sizeof(int32_t), cmp_int);
        free(qbar);
        free(sc);
    }
    return err;
}

/* ------------------------------------------------------------------------- */
/* Eq. 4-5: vertical-line score as accumulated column mass.                    */
/*   a_{t,j} = softmax over the keys j <= pos(t) of alpha * <q_t, k_j>         */
/*   S(p)    = sum over the query set T of a_{t,p},   p in the prefix [0, P)    */
/*   I       = TopK(S, k), ties towards the lower position, ascending          */
/* T is the last n_queries query rows (0: min(W, Lq), Algorithm 1's tail); the   */
/* query block is end-aligned with the keys: row i sits at position            */
/* Lk - Lq + i.  n_queries <= W, so every prefix key is visible to every t.    */
/*                                                                             */
/* This function is the library's REPRODUCIBILITY CONTRACT, not the definition: */
/* the definition is oracle_select_mass_plain below (two-pass softmax, libm exp, */
/* sequential sums), to which this one is pinned at 1e-12 of the largest score.  */
/* So that the GPU can return the same set bit for bit, the arithmetic is fixed  */
/* operation by operation (all fp64, round to nearest):                          */
/*   s       = (fma chain over channels 0..D-1 from 0) * alpha                 */
/*   exp     = exp_det below (range reduction by ln2 in two parts, degree-13   */
/*             Taylor polynomial by Horner fma, exact scaling by 2^n)          */
/*   row sum = per chunk of 64 consecutive keys (aligned at multiples of 64):  */
/*             m_c = max, z_c = balanced pairwise tree over exp(s - m_c) with  */
/*             masked keys contributing 0; then m = max_c m_c and              */
/*             Z = sum_c z_c * exp(m_c - m), added in ascending chunk order    */
/*   S(p)    = sum over t ascending of exp(s - m_t) / Z_t                      */
/* ------------------------------------------------------------------------- */
static double exp_det(double x) {
    if (!(x >= -690.0)) return 0.0;                 /* also -inf; the caller never passes x > 0 by much */
    const double n = rint(x * 1.4426950408889634);
    double r = fma(n, -6.93147180369123816490e-01, x);
    r = fma(n, -1.90821492927058770002e-10, r);
    double p = 1.0 / 6227020800.0;                  /* 1/13! */
    p = fma(p, r, 1.0 / 479001600.0);
    p = fma(p, r, 1.0 / 39916800.0);
    p = fma(p, r, 1.0 / 3628800.0);
    p = fma(p, r, 1.0 / 362880.0);
    p = fma(p, r, 1.0 / 40320.0);
    p = fma(p, r, 1.0 / 5040.0);
    p = fma(p, r, 1.0 / 720.0);
    p = fma(p, r, 1.0 / 120.0);
    p = fma(p, r, 1.0 / 24.0);
    p = fma(p, r, 1.0 / 6.0);
    p = fma(p, r, 0.5);
    p = fma(p, r, 1.0);
    p = fma(p, r, 1.0);
    union { uint64_t u; double d; } two_n;
    two_n.u = (uint64_t)((int64_t)n + 1023) << 52;  /* n >= -996: a normal number */
    return p * two_n.d;
}

void oracle_exp_det(const double* x, long n, double* out) {
    for (long i = 0; i < n; ++i) out[i] = exp_det(x[i]);
}

static double tree_sum64(double* e) {               /* balanced pairwise tree: (0,1),(2,3).. then pairs of pairs */
    for (int step = 1; step < 64; step <<= 1)
        for (int i = 0; i < 64; i += 2 * step) e[i] = e[i] + e[i + step];
    return e[0];
}

int oracle_select_mass(const uint16_t* q, const uint16_t* k_, int B, int Hq, int Hkv, int Lq, int Lk, int D, int W,
                       int n_queries, int k, double alpha, int32_t* idx_out, double* scores_out) {
    if (Hkv <= 0 || Hq % Hkv) return 1;
    const int g = Hq / Hkv;
    const int P = (Lk - W > 0) ? Lk - W : 0;
    if (P == 0 || k == 0) return 0;
    if (k > P || k < 0 || Lq > Lk) return 1;
    const int nT = n_queries ? n_queries : (W < Lq ? W : Lq);
    if (nT <= 0 || nT > Lq || nT > W) return 1;
    const int n_chunks = (Lk + 63) / 64;
    int err = 0;
#pragma omp parallel for schedule(dynamic)
    for (int bh = 0; bh < B * Hq; ++bh) {
        const int b = bh / Hq, h = bh % Hq, kvh = h / g;
        const uint16_t* kh = k_ + ((long)b * Hkv + kvh) * Lk * D;
        double* S = (double*)calloc((size_t)P, sizeof(double));
        double* srow = (double*)malloc(sizeof(double) * (size_t)Lk);
        double* mc = (double*)malloc(sizeof(double) * (size_t)n_chunks);
        double* zc = (double*)malloc(sizeof(double) * (size_t)n_chunks);
        scored_t* sc = (scored_t*)malloc(sizeof(scored_t) * (size_t)P);
        if (!S || !srow || !mc || !zc || !sc) { err = 2; free(S); free(srow); free(mc); free(zc); free(sc); continue; }
        for (int i = Lq - nT; i < Lq; ++i) {        /* t ascending */
            const int pos = Lk - Lq + i;
            const uint16_t* qr = q + (((long)b * Hq + h) * Lq + i) * D;
            for (int j = 0; j <= pos; ++j) {
                double acc = 0.0;
                for (int d = 0; d < D; ++d)
                    acc = fma((double)bf16_to_f32(qr[d]), (double)bf16_to_f32(kh[(long)j * D + d]), acc);
                srow[j] = acc * alpha;
            }
            const int nc = pos / 64 + 1;
            double m = -INFINITY;
            for (int c = 0; c < nc; ++c) {
                double e[64], cm = -INFINITY;
                for (int u = 0; u < 64; ++u) {
                    const int j = 64 * c + u;
                    if (j <= pos && srow[j] > cm) cm = srow[j];
                }
                for (int u = 0; u < 64; ++u) {
                    const int j = 64 * c + u;
                    e[u] = j <= pos ? exp_det(srow[j] - cm) : 0.0;
                }
                mc[c] = cm;
                zc[c] = tree_sum64(e);
                if (cm > m) m = cm;
            }
            double Z = 0.0;
            for (int c = 0; c < nc; ++c) Z = Z + zc[c] * exp_det(mc[c] - m);
            for (int p = 0; p < P; ++p) S[p] = S[p] + exp_det(srow[p] - m) / Z;
        }
        for (int p = 0; p < P; ++p) {
            sc[p].s = S[p];
            sc[p].p = p;
            if (scores_out) scores_out[(long)bh * P + p] = S[p];
        }
        qsort(sc, P, sizeof(scored_t), cmp_scored);
        int32_t* out = idx_out + (long)bh * k;
        for (int c = 0; c < k; ++c) out[c] = sc[c].p;
        qsort(out, k, sizeof(int32_t), cmp_int);
        free(S); free(srow); free(mc); free(zc); free(sc);
    }
    return err;
}

/* ------------------------------------------------------------------------- */
/* Eq. 4-5 by the plain definition (the reference for oracle_select_mass and    */
/* for the validity of any selected set): per tail query t a two-pass fp64     */
/* softmax over the keys j <= pos(t) - libm exp, running maximum and running   */
/* sum in ascending key order - and S(p) = sum of a_{t,p} over t in ascending  */
/* query order.  Top-k by (score descending, position ascending), emitted      */
/* ascending.  No blocking, no polynomial, no reordering.                      */
/* ------------------------------------------------------------------------- */
int oracle_select_mass_plain(const uint16_t* q, const uint16_t* k_, int B, int Hq, int Hkv, int Lq, int Lk, int D, int W,
                             int n_queries, int k, double alpha, int32_t* idx_out, double* scores_out) {
    if (Hkv <= 0 || Hq % Hkv) return 1;
    const int g = Hq / Hkv;
    const int P = (Lk - W > 0) ? Lk - W : 0;
    if (P == 0 || k == 0) return 0;
    if (k > P || k < 0 || Lq > Lk) return 1;
    const int nT = n_queries ? n_queries : (W < Lq ? W : Lq);
    if (nT <= 0 || nT > Lq || nT > W) return 1;
    int err = 0;
#pragma omp parallel for schedule(dynamic)
    for (int bh = 0; bh < B * Hq; ++bh) {
        const int b = bh / Hq, h = bh % Hq, kvh = h / g;
        const uint16_t* kh = k_ + ((long)b * Hkv + kvh) * Lk * D;
        double* S = (double*)calloc((size_t)P, sizeof(double));
        double* srow = (double*)malloc(sizeof(double) * (size_t)Lk);
        scored_t* sc = (scored_t*)malloc(sizeof(scored_t) * (size_t)P);
        if (!S || !srow || !sc) { err = 2; free(S); free(srow); free(sc); continue; }
        for (int i = Lq - nT; i < Lq; ++i) {
            const int pos = Lk - Lq + i;
            const uint16_t* qr = q + (((long)b * Hq + h) * Lq + i) * D;
            double m = -INFINITY;
            for (int j = 0; j <= pos; ++j) {
                double acc = 0.0;
                for (int d = 0; d < D; ++d) acc += (double)bf16_to_f32(qr[d]) * (double)bf16_to_f32(kh[(long)j * D + d]);
                srow[j] = alpha * acc;
                if (srow[j] > m) m = srow[j];
            }
            double Z = 0.0;
            for (int j = 0; j <= pos; ++j) Z += exp(srow[j] - m);
            for (int p = 0; p < P; ++p) S[p] += exp(srow[p] - m) / Z;
        }
        for (int p = 0; p < P; ++p) {
            sc[p].s = S[p];
            sc[p].p = p;
            if (scores_out) scores_out[(long)bh * P + p] = S[p];
        }
        qsort(sc, P, sizeof(scored_t), cmp_scored);
        int32_t* out = idx_out + (long)bh * k;
        for (int c = 0; c < k; ++c) out[c] = sc[c].p;
        qsort(out, k, sizeof(int32_t), cmp_int);
        free(S); free(srow); free(sc);
    }
    return err;
}

/* ------------------------------------------------------------------------- */
/* Eq. 6-7: hybrid-precision causal attention, by its definition.             */
/* For query row i of head h and every key j <= i:                            */
/*   the pair is full precision (FP) when j is a vertical-line key of (b,h)   */
/*   or lies in the sliding window (i - j < W); otherwise it is low-bit.      */
/*   s_ij = alpha * <q_i, k_j>   with the bf16 originals for FP pairs and     */
/*                               the dequantized codes for low-bit pairs      */
/*   O_i  = sum_j softmax_j(s_i.) * v_j   with v_j = V (FP) or V^ (low-bit)   */
/* One softmax over the whole row (two passes, fp64).                         */
/* rows[] selects the query rows to compute (same rows for every head);       */
/* out is [B,Hq,n_rows,D] fp64, lse (optional) is [B,Hq,n_rows].              */
/* fp_pairs (optional) returns the number of FP pairs met.                    */
/* ------------------------------------------------------------------------- */
/* L: number of keys (L_K).  Lq: number of query rows (the query block of Algorithm 2), end-aligned with
   the keys: query row i sits at position L - Lq + i.  Lq = L is the whole prefill.  q, q_codes and q_scales
   hold Lq rows (quantization blocks counted from the first row of the block).
   fixed_window: 0 = per-row sliding window (key j is a window key of the row at position i iff i - j < W);
   1 = Algorithm 2's K_Win taken literally: the last W keys, [L - W, L), for every row of the block. */
typedef struct {
    int B, Hq, Hkv, L, Lq, fixed_window, D, W, k, block_tokens;
    int q_fmt, k_fmt, v_fmt;
    double alpha;
    const uint16_t *q, *k_, *v;
    const uint8_t *q_codes, *k_codes, *v_codes;
    const float *q_scales, *k_scales, *v_scales;
    const int32_t* vl_idx;
} attn_in_t;

static long code_row_bytes(int fmt, int D) { return fmt == FMT_INT4 ? D / 2 : D; }

static void mark_vl(const attn_in_t* a, int b, int h, uint8_t* is_vl) {
    memset(is_vl, 0, (size_t)a->L);
    for (int c = 0; c < a->k; ++c) {
        int j = a->vl_idx[((long)b * a->Hq + h) * a->k + c];
        if (j >= 0 && j < a->L) is_vl[j] = 1;
    }
}

/* x^ = code * scale for one head, materialised as [L,D] fp64 (exact products) */
static double* dequant_head(const uint8_t* codes, const float* scales, int fmt, int L, int D, int bt) {
    double* xh = (double*)malloc(sizeof(double) * (size_t)L * D);
    if (!xh) return NULL;
    for (int t = 0; t < L; ++t)
        for (int d = 0; d < D; ++d)
            xh[(long)t * D + d] = dequant(codes + (long)t * code_row_bytes(fmt, D), d, fmt, (double)scales[t / bt]);
    return xh;
}

/* the bf16 originals of one head widened to [L,D] fp64 (exact) */
static double* widen_head(const uint16_t* x, int L, int D) {
    double* xd = (double*)malloc(sizeof(double) * (size_t)L * D);
    if (!xd) return NULL;
    for (long e = 0; e < (long)L * D; ++e) xd[e] = (double)bf16_to_f32(x[e]);
    return xd;
}

typedef struct { double *qf, *qh, *kf, *kh, *vf, *vh; } head_views_t;

static int load_head(const attn_in_t* a, int b, int h, head_views_t* hv) {
    const int g = a->Hq / a->Hkv, kvh = h / g, L = a->L, Lq = a->Lq, D = a->D, bt = a->block_tokens;
    const int nb = (L + bt - 1) / bt, nbq = (Lq + bt - 1) / bt;
    const long qo = ((long)b * a->Hq + h), ko = ((long)b * a->Hkv + kvh);
    hv->qf = widen_head(a->q + qo * Lq * D, Lq, D);
    hv->kf = widen_head(a->k_ + ko * L * D, L, D);
    hv->vf = widen_head(a->v + ko * L * D, L, D);
    hv->qh = dequant_head(a->q_codes + qo * Lq * code_row_bytes(a->q_fmt, D), a->q_scales + qo * nbq, a->q_fmt, Lq, D, bt);
    hv->kh = dequant_head(a->k_codes + ko * L * code_row_bytes(a->k_fmt, D), a->k_scales + ko * nb, a->k_fmt, L, D, bt);
    hv->vh = dequant_head(a->v_codes + ko * L * code_row_bytes(a->v_fmt, D), a->v_scales + ko * nb, a->v_fmt, L, D, bt);
    return (hv->qf && hv->kf && hv->vf && hv->qh && hv->kh && hv->vh) ? 0 : 2;
}
static void free_head(head_views_t* hv) {
    free(hv->qf); free(hv->qh); free(hv->kf); free(hv->kh); free(hv->vf); free(hv->vh);
}

/* is key j a window key of the query row at position i? */
static int in_window(const attn_in_t* a, int i, int j) {
    return a->fixed_window ? (j >= a->L - a->W) : (i - j < a->W);
}

/* alpha * <q_i, k_j> in the pair's class */
static double pair_score(const attn_in_t* a, const head_views_t* hv, int i, int j, int fp) {
    const int D = a->D;
    const double* qr = (fp ? hv->qf : hv->qh) + (long)i * D;
    const double* kr = (fp ? hv->kf : hv->kh) + (long)j * D;
    double s = 0.0;
    for (int d = 0; d < D; ++d) s += qr[d] * kr[d];
    return a->alpha * s;
}

int oracle_attention_rows(const attn_in_t* a, const int32_t* rows, int n_rows, double* out,
                          double* lse, long long* fp_pairs) {
    if (a->Hkv <= 0 || a->Hq % a->Hkv || a->Lq <= 0 || a->Lq > a->L) return 1;
    const int D = a->D, L = a->L, off = a->L - a->Lq;   /* query row r sits at position off + r */
    long long fp_total = 0;
    int err = 0;
    for (int bh = 0; bh < a->B * a->Hq && !err; ++bh) {
        const int b = bh / a->Hq, h = bh % a->Hq;
        uint8_t* is_vl = (uint8_t*)malloc((size_t)L);
        head_views_t hv;
        if (!is_vl || load_head(a, b, h, &hv)) return 2;
        mark_vl(a, b, h, is_vl);
#pragma omp parallel for schedule(dynamic) reduction(+ : fp_total)
        for (int r = 0; r < n_rows; ++r) {
            const int qi = rows[r], i = qi + off;      /* row of the query block, its position among the keys */
            double* o = out + ((long)bh * n_rows + r) * D;
            if (qi < 0 || qi >= a->Lq) { err = 1; continue; }
            double* s = (double*)malloc(sizeof(double) * (i + 1));
            uint8_t* fp = (uint8_t*)malloc((size_t)(i + 1));
            if (!s || !fp) { err = 2; free(s); free(fp); continue; }
            double m = -INFINITY;
            for (int j = 0; j <= i; ++j) {
                fp[j] = (uint8_t)(is_vl[j] || in_window(a, i, j));
                fp_total += fp[j];
                s[j] = pair_score(a, &hv, qi, j, fp[j]);
                if (s[j] > m) m = s[j];
            }
            double denom = 0.0;
            for (int j = 0; j <= i; ++j) { s[j] = exp(s[j] - m); denom += s[j]; }
            for (int d = 0; d < D; ++d) o[d] = 0.0;
            for (int j = 0; j <= i; ++j) {
                const double* vr = (fp[j] ? hv.vf : hv.vh) + (long)j * D;
                for (int d = 0; d < D; ++d) o[d] += s[j] * vr[d];
            }
            for (int d = 0; d < D; ++d) o[d] /= denom;
            if (lse) lse[(long)bh * n_rows + r] = m + log(denom);
            free(s);
            free(fp);
        }
        free(is_vl);
        free_head(&hv);
    }
    if (fp_pairs) *fp_pairs = fp_total;
    return err;
}

/* ------------------------------------------------------------------------- */
/* Algorithm 2, Stage 3, taken literally: three segments scanned in tiles of  */
/* tile_n keys with the running (m, l, acc) update                            */
/*   m' = max(m, rowmax);  l' = l e^{m-m'} + sum e^{s-m'};                     */
/*   acc' = acc e^{m-m'} + sum e^{s-m'} v                                     */
/* Segment A: low-bit keys; Segment B: vertical-line keys outside the window; */
/* Segment C: window keys.  Must agree with oracle_attention_rows up to       */
/* rounding order.                                                            */
/* ------------------------------------------------------------------------- */
static void flash_os(const double* s, const double* const* vals, int n, int D, double* m, double* l,
                     double* acc) {
    if (n == 0) return;
    double mx = *m;
    for (int c = 0; c < n; ++c) if (s[c] > mx) mx = s[c];
    const double corr = (*m == -INFINITY) ? 0.0 : exp(*m - mx);
    *l *= corr;
    for (int d = 0; d < D; ++d) acc[d] *= corr;
    for (int c = 0; c < n; ++c) {
        const double p = exp(s[c] - mx);
        *l += p;
        for (int d = 0; d < D; ++d) acc[d] += p * vals[c][d];
    }
    *m = mx;
}

int oracle_attention_segmented_rows(const attn_in_t* a, const int32_t* rows, int n_rows, int tile_n,
                                    double* out) {
    if (a->Hkv <= 0 || a->Hq % a->Hkv || tile_n <= 0 || a->Lq <= 0 || a->Lq > a->L) return 1;
    const int D = a->D, L = a->L, off = a->L - a->Lq;
    for (int bh = 0; bh < a->B * a->Hq; ++bh) {
        const int b = bh / a->Hq, h = bh % a->Hq;
        uint8_t* is_vl = (uint8_t*)malloc((size_t)L);
        head_views_t hv;
        if (!is_vl || load_head(a, b, h, &hv)) return 2;
        mark_vl(a, b, h, is_vl);
#pragma omp parallel for schedule(dynamic)
        for (int r = 0; r < n_rows; ++r) {
            const int qi = rows[r], i = qi + off;
            double* o = out + ((long)bh * n_rows + r) * D;
            double m = -INFINITY, l = 0.0;
            double* acc = (double*)calloc((size_t)D, sizeof(double));
            double* s = (double*)malloc(sizeof(double) * tile_n);
            const double** vals = (const double**)malloc(sizeof(double*) * (size_t)tile_n);
            int* members = (int*)malloc(sizeof(int) * (i + 1));
            for (int seg = 0; seg < 3; ++seg) {
                int n_mem = 0;                      /* keys of this segment, in position order */
                for (int j = 0; j <= i; ++j) {
                    const int cls = in_window(a, i, j) ? 2 : (is_vl[j] ? 1 : 0);
                    if (cls == seg) members[n_mem++] = j;
                }
                for (int t0 = 0; t0 < n_mem; t0 += tile_n) {
                    const int n = (n_mem - t0 < tile_n) ? n_mem - t0 : tile_n;
                    for (int c = 0; c < n; ++c) {
                        const int j = members[t0 + c];
                        s[c] = pair_score(a, &hv, qi, j, seg != 0);
                        vals[c] = ((seg != 0) ? hv.vf : hv.vh) + (long)j * D;
                    }
                    flash_os(s, vals, n, D, &m, &l, acc);
                }
            }
            for (int d = 0; d < D; ++d) o[d] = acc[d] / l;
            free(acc); free(s); free(vals); free(members);
        }
        free(is_vl);
        free_head(&hv);
    }
    return 0;
}

/* element-wise access to the e4m3 encoder / decoder (pinned by the tests against a library cast) */
void oracle_e4m3_encode(const float* y, long n, uint8_t* out) {
    for (long e = 0; e < n; ++e) out[e] = e4m3_encode_rne_sat(y[e]);
}
void oracle_e4m3_decode(const uint8_t* c, long n, double* out) {
    for (long e = 0; e < n; ++e) out[e] = e4m3_value(c[e]);
}

int oracle_num_threads(void) {
    int n = 1;
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    n = omp_get_max_threads();
#endif
    return n;
}
