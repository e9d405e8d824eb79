/*
 * CPU oracle for the 3x3 convolution that the Winograd step computes -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * Sec. 3.3 of the paper replaces the UNet's 3x3 convolutions by Winograd convolution with a 4x4 output tile.  In
 * exact arithmetic Winograd's algorithm gives the result of the convolution itself, so the oracle is that
 * definition written out (stride 1, zero padding 1, as every 3x3 convolution of the model):
 *
 *     y[n][i][j][k] = bias[k] + sum_{r=0..2} sum_{s=0..2} sum_{c} x[n][i + r - 1][j + s - 1][c] * w[k][r][s][c]
 *
 * with x taken as zero outside the image.  This is the cross-correlation every deep-learning framework calls a
 * convolution (the filter is not flipped).  Layout: x [N][H][W][C] and y [N][H][W][K] channels-last, w [K][3][3][C].
 *
 * Evaluated in IEEE double from the stored fp16 (or fp32) values, in the order of the formula.  Plain loops, one
 * OpenMP "parallel for" over output pixels.  Shares no code with the CUDA library.
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

/* x: [N][H][W][C]; w: [K][3][3][C]; bias: [K] or NULL, all in `dtype` (0 = fp16 bits, 1 = fp32); y: [N][H][W][K]
 * doubles.  Returns 0, or 1 on bad arguments. */
int sd_conv3x3_oracle_forward(const void *x, const void *w, const void *bias, double *y, int64_t N, int64_t H,
                              int64_t W, int64_t C, int64_t K, int dtype)
{
    if (!x || !w || !y || N < 0 || H <= 0 || W <= 0 || C <= 0 || K <= 0 || (dtype != 0 && dtype != 1)) return 1;
    const int64_t pixels = N * H * W;
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < pixels; ++p) {
        const int64_t n = p / (H * W), i = (p / W) % H, j = p % W;
        for (int64_t k = 0; k < K; ++k) {
            double acc = bias ? elem(bias, k, dtype) : 0.0;
            for (int r = 0; r < 3; ++r) {
                const int64_t ii = i + r - 1;
                if (ii < 0 || ii >= H) continue;
                for (int s = 0; s < 3; ++s) {
                    const int64_t jj = j + s - 1;
                    if (jj < 0 || jj >= W) continue;
                    const int64_t xo = ((n * H + ii) * W + jj) * C, wo = ((k * 3 + r) * 3 + s) * C;
                    for (int64_t c = 0; c < C; ++c) acc += elem(x, xo + c, dtype) * elem(w, wo + c, dtype);
                }
            }
            y[p * K + k] = acc;
        }
    }
    return 0;
}
