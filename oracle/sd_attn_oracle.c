/*
 * sd_attn_oracle.c -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, obviously-correct CPU statement of scaled-dot-product attention,
 *
 *     Attention(Q, K, V) = softmax(Q K^T * s) V            (paper Eq. 3, s = 1/sqrt(d))
 *
 * with the softmax written exactly as the paper splits it (Eq. 4): a row maximum
 * L_i = max_j a_ij, a shifted exponential sum S_i = sum_j exp(a_ij - L_i), and the
 * element-wise normalisation p_ij = exp(a_ij - L_i) / S_i.  FlashAttention (Sec. 3.2.2)
 * and the partially fused softmax (Sec. 3.2.1) are exact reformulations of this result,
 * so the definition itself is the oracle for every GPU kernel of the library.
 *
 * Everything is IEEE double: inputs (binary16 or binary32) are widened exactly, every
 * product of two binary16 values is exact in double, sums run in index order, exp() is
 * libm's.  No blocking, no fusion, no reordering.  The only parallelism is OpenMP over
 * independent query rows, which cannot change any result bit.
 *
 * Only tests, the smoke check and the benchmark's cpu_baseline leg may call this file.
 * It shares no code with the CUDA path (own binary16 decoder, no CUDA headers).
 *
 * Parity pins: every exported function is pinned by CPU tests against closed forms,
 * brute force in another formulation, invariants of the definition and scipy's softmax.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_ERR_ARG 1
#define ORACLE_ERR_NOMEM 2

#define ORACLE_F16 0
#define ORACLE_F32 1

/* IEEE 754 binary16 -> double, exact (sign, 5-bit exponent, 10-bit fraction). */
static double half_bits_to_double(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int expo = (h >> 10) & 0x1f;
    int frac = h & 0x3ff;
    double mag;
    if (expo == 0) {
        mag = ldexp((double)frac, -24);               /* zero and subnormals: frac * 2^-24 */
    } else if (expo == 31) {
        mag = frac ? NAN : INFINITY;
    } else {
        mag = ldexp((double)(frac | 0x400), expo - 25); /* (1024+frac) * 2^(expo-15-10) */
    }
    return sign ? -mag : mag;
}

static double load_elem(const void *base, int64_t idx, int dtype)
{
    if (dtype == ORACLE_F16)
        return half_bits_to_double(((const uint16_t *)base)[idx]);
    return (double)((const float *)base)[idx];
}

int sd_attn_oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void sd_attn_oracle_set_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* exact widening of a binary16 array, exported so tests can pin the decoder itself */
void sd_attn_oracle_half_to_double(const uint16_t *src, double *dst, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) dst[i] = half_bits_to_double(src[i]);
}

/*
 * One query row of Eq. 3 / Eq. 4.  qrow: d doubles.  kd, vd: Nk x d doubles.
 * a, e: scratch of Nk doubles.  Writes o[d]; returns L and S through pointers.
 * If p_out is non-NULL it receives the Nk normalised weights p_ij.
 */
static void attention_row(const double *qrow, const double *kd, const double *vd,
                          int Nk, int d, double s, double *a, double *e,
                          double *o, double *L_out, double *S_out, double *p_out)
{
    /* scores: a_j = s * sum_k q_k k_jk   (Eq. 3, the matrix A of Sec. 3.2.1) */
    for (int j = 0; j < Nk; ++j) {
        double dot = 0.0;
        for (int c = 0; c < d; ++c) dot += qrow[c] * kd[(int64_t)j * d + c];
        a[j] = s * dot;
    }
    /* reductions (Eq. 4): L = max_j a_j ; S = sum_j exp(a_j - L) */
    double L = a[0];
    for (int j = 1; j < Nk; ++j) if (a[j] > L) L = a[j];
    double S = 0.0;
    for (int j = 0; j < Nk; ++j) { e[j] = exp(a[j] - L); S += e[j]; }
    /* element-wise normalisation and the product with V (Eq. 3) */
    for (int c = 0; c < d; ++c) {
        double acc = 0.0;
        for (int j = 0; j < Nk; ++j) acc += e[j] * vd[(int64_t)j * d + c];
        o[c] = acc / S;
    }
    if (p_out) for (int j = 0; j < Nk; ++j) p_out[j] = e[j] / S;
    *L_out = L;
    *S_out = S;
}

/*
 * q: [B][H][Nq][d], k, v: [B][H][Nk][d], dense, d innermost, dtype ORACLE_F16 / ORACLE_F32.
 * rows == NULL : every row; out is [B][H][Nq][d] doubles, L and S (optional) are [B][H][Nq].
 * rows != NULL : n_rows flattened row ids r = (b*H + h)*Nq + i; out is [n_rows][d],
 *                L and S are [n_rows].  Row ids must be grouped by (b,h) only for speed,
 *                never for correctness.
 * probs (optional, may be NULL): receives p_ij, [rows or all rows][Nk].
 */
int sd_attn_oracle_forward(const void *q, const void *k, const void *v,
                           double *out, double *L, double *S, double *probs,
                           int B, int H, int Nq, int Nk, int d, float scale, int dtype,
                           const int64_t *rows, int64_t n_rows)
{
    if (!q || !k || !v || !out) return ORACLE_ERR_ARG;
    if (B <= 0 || H <= 0 || Nq < 0 || Nk <= 0 || d <= 0) return ORACLE_ERR_ARG;
    if (dtype != ORACLE_F16 && dtype != ORACLE_F32) return ORACLE_ERR_ARG;
    const int64_t BH = (int64_t)B * H;
    const int64_t total_rows = rows ? n_rows : BH * Nq;
    if (total_rows == 0) return ORACLE_OK;
    if (rows)
        for (int64_t r = 0; r < n_rows; ++r)
            if (rows[r] < 0 || rows[r] >= BH * Nq) return ORACLE_ERR_ARG;
    const double s = (double)scale; /* the caller's binary32 scale, widened exactly */

    /* widen K and V once: exact, and it keeps the row loop readable */
    const int64_t kv_elems = BH * Nk * d;
    double *kd = (double *)malloc(sizeof(double) * (size_t)kv_elems);
    double *vd = (double *)malloc(sizeof(double) * (size_t)kv_elems);
    if (!kd || !vd) { free(kd); free(vd); return ORACLE_ERR_NOMEM; }
    for (int64_t t = 0; t < kv_elems; ++t) {
        kd[t] = load_elem(k, t, dtype);
        vd[t] = load_elem(v, t, dtype);
    }

    int failed = 0;
#pragma omp parallel
    {
        double *a = (double *)malloc(sizeof(double) * (size_t)Nk);
        double *e = (double *)malloc(sizeof(double) * (size_t)Nk);
        double *qrow = (double *)malloc(sizeof(double) * (size_t)d);
        if (!a || !e || !qrow) {
#pragma omp atomic write
            failed = 1;
        } else {
#pragma omp for schedule(dynamic, 16)
            for (int64_t t = 0; t < total_rows; ++t) {
                const int64_t r = rows ? rows[t] : t;
                const int64_t bh = r / Nq;
                for (int c = 0; c < d; ++c) qrow[c] = load_elem(q, r * d + c, dtype);
                double Lr, Sr;
                attention_row(qrow, kd + bh * Nk * d, vd + bh * Nk * d, Nk, d, s, a, e,
                              out + t * d, &Lr, &Sr, probs ? probs + t * Nk : NULL);
                if (L) L[t] = Lr;
                if (S) S[t] = Sr;
            }
        }
        free(a); free(e); free(qrow);
    }
    free(kd); free(vd);
    return failed ? ORACLE_ERR_NOMEM : ORACLE_OK;
}
