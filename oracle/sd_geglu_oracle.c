/*
 * CPU oracle for the fused GEGLU step -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * The feed-forward blocks of the UNet's transformer layers project to 2C channels, split the result in two halves,
 * apply GELU to one half and multiply it into the other; the paper (Sec. 3.1, Eq. 2) runs the error-function
 * arithmetic together with "its accompanied split and multiplication ops" as one kernel.  What that computes, per row
 * r and channel c < C of an input x of shape [R][2C]:
 *
 *     out[r][c] = x[r][c] * GELU(x[r][C + c]),      GELU(g) = g/2 * (1 + erf(g / sqrt 2))            (Eq. 2)
 *
 * Reading: the paper does not say which half is gated; the Stable Diffusion feed-forward block it accelerates applies
 * GELU to the SECOND half, which is what is taken here.
 *
 * Evaluated in IEEE double from the stored fp16 (or fp32) values.  1 + erf(z) is written as erfc(-z): the two are the
 * same function, and libm's erfc keeps its relative accuracy where erf is within an ulp of -1.
 * Plain loops, one OpenMP "parallel for" over rows (rows are independent).  Shares no code with the CUDA library.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

static double half_to_double(uint16_t h)
{
    const int sign = h >> 15, e = (h >> 10) & 31, m = h & 1023;
    double v;
    if (e == 0) v = ldexp((double)m, -24);                       /* zero and subnormals */
    else if (e == 31) v = m ? NAN : INFINITY;
    else v = ldexp((double)(m + 1024), e - 25);
    return sign ? -v : v;
}

static double elem(const void *base, int64_t i, int dtype)
{
    if (dtype == 0) return half_to_double(((const uint16_t *)base)[i]);
    return (double)((const float *)base)[i];
}

/* GELU of Eq. 2 in double. */
double sd_geglu_oracle_gelu(double g)
{
    return 0.5 * g * erfc(-g / sqrt(2.0));
}

/* x: [rows][2C] (dtype 0 = fp16 bits, 1 = fp32), out: [rows][C] doubles.  Returns 0, or 1 on bad arguments. */
int sd_geglu_oracle_forward(const void *x, double *out, int64_t rows, int64_t C, int dtype)
{
    if (!x || !out || rows < 0 || C <= 0 || (dtype != 0 && dtype != 1)) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < C; ++c) {
            const double a = elem(x, r * 2 * C + c, dtype);
            const double g = elem(x, r * 2 * C + C + c, dtype);
            out[r * C + c] = a * sd_geglu_oracle_gelu(g);
        }
    return 0;
}
