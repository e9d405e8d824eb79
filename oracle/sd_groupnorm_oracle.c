/*
 * CPU oracle for the fused group normalisation -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * Sec. 3.1 of the paper runs "reshape, mean, variance, normalize" of group normalisation as one kernel without
 * intermediate tensors.  Per sample n and group g (the C channels are divided into G groups of C/G consecutive
 * channels), over the (C/G) * HW values of the group:
 *
 *     mu = mean(x),   sigma^2 = mean((x - mu)^2),   xhat = (x - mu) / sigma                          (Eq. 1)
 *     y[n][c][p] = xhat * gamma[c] + beta[c]
 *
 * Readings: Eq. 1 shows neither the epsilon nor the per-channel affine of the operation the paper cites for it; both
 * are part of that operation as the UNet uses it, so sigma = sqrt(sigma^2 + eps) with eps an argument (the variance is
 * the biased one), and gamma / beta are optional arguments (NULL: 1 and 0).  Layout: x and y are [N][C][HW], HW
 * innermost (the model's NCHW), so a group is one contiguous run of (C/G) * HW values.
 *
 * Evaluated in IEEE double from the stored fp16 (or fp32) values, two passes over the group (mean first, then the
 * centred squares).  Plain loops, one OpenMP "parallel for" over (n, g).  Shares no code with the CUDA library.
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>

static double half_to_double(uint16_t h)
{
    const int sign = h >> 15, e = (h >> 10) & 31, m = h & 1023;
    double v;
    if (e == 0) v = ldexp((double)m, -24);
    else if (e == 31) v = m ? NAN : INFINITY;
    else v = ldexp((double)(m + 1024), e - 25);
    return sign ? -v : v;
}

static double elem(const void *base, int64_t i, int dtype)
{
    if (dtype == 0) return half_to_double(((const uint16_t *)base)[i]);
    return (double)((const float *)base)[i];
}

/* x: [N][C][HW]; gamma, beta: [C] in the same dtype, or NULL; y: [N][C][HW] doubles; mean, rstd: [N][G] doubles or NULL.
 * dtype 0 = fp16 bits, 1 = fp32.  Returns 0, or 1 on bad arguments (C not divisible by G included). */
int sd_groupnorm_oracle_forward(const void *x, const void *gamma, const void *beta, double *y, double *mean, double *rstd,
                                int64_t N, int64_t C, int64_t HW, int64_t G, double eps, int dtype)
{
    if (!x || !y || N < 0 || C <= 0 || HW <= 0 || G <= 0 || C % G || (dtype != 0 && dtype != 1)) return 1;
    const int64_t cpg = C / G, n_group = cpg * HW;
#pragma omp parallel for schedule(static)
    for (int64_t ng = 0; ng < N * G; ++ng) {
        const int64_t n = ng / G, g = ng % G;
        const int64_t base = (n * C + g * cpg) * HW;
        double sum = 0.0;
        for (int64_t i = 0; i < n_group; ++i) sum += elem(x, base + i, dtype);
        const double mu = sum / (double)n_group;
        double sq = 0.0;
        for (int64_t i = 0; i < n_group; ++i) {
            const double dlt = elem(x, base + i, dtype) - mu;
            sq += dlt * dlt;
        }
        const double r = 1.0 / sqrt(sq / (double)n_group + eps);
        if (mean) mean[ng] = mu;
        if (rstd) rstd[ng] = r;
        for (int64_t c = 0; c < cpg; ++c) {
            const double ga = gamma ? elem(gamma, g * cpg + c, dtype) : 1.0;
            const double be = beta ? elem(beta, g * cpg + c, dtype) : 0.0;
            for (int64_t p = 0; p < HW; ++p) {
                const int64_t i = base + c * HW + p;
                y[i] = (elem(x, i, dtype) - mu) * r * ga + be;
            }
        }
    }
    return 0;
}
