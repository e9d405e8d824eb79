/*
 * sd_winograd.h -- C ABI of the Winograd 3x3 convolution (Sec. 3.3 of the paper: the UNet's 3x3 convolutions as
 * matrix multiplications in a transformed domain, with the 4x4 output tile that Table 2 selects).
 *
 *     y[n][i][j][k] = bias[k] + sum_{r,s in 0..2} sum_c x[n][i + r - 1][j + s - 1][c] * w[k][r][s][c]
 *
 * stride 1, zero padding 1, the filter not flipped.  Tensors are DEVICE memory, channels-last, IEEE binary16:
 * x [N][H][W][C], w [K][3][3][C], bias [K] (or NULL), y [N][H][W][K]; C and K multiples of 8; every pointer
 * 16-byte aligned.  Arithmetic: transforms in binary32, the transformed filter U and the transformed input V
 * rounded once to binary16, products accumulated in binary32 on the tensor cores, output rounded once to binary16.
 * Winograd's algorithm is exact in exact arithmetic; in this arithmetic its result differs from the directly
 * evaluated convolution by the roundings of U and V amplified by the output transform (about 3e-3 of the output's
 * r.m.s. in relative L2 for the UNet's layer sizes), which is the numerical error the paper names.
 *
 * The filter is transformed once per layer (sd_winograd_transform_filter: 36 K C values from 9 K C, the "Weight x4"
 * of Table 2); a forward call transforms the input into caller-lent scratch (the "Tensor x2.25" of Table 2, plus
 * the binary32 products), runs 36 matrix multiplications and transforms back.  The entry points are stateless:
 * they act on the current device, allocate nothing, enqueue their kernels on `stream` and do not synchronise.
 * Status codes are those of sd_attn.h (sd_attn_status_string names them).
 */
#ifndef SD_WINOGRAD_H
#define SD_WINOGRAD_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Number of binary16 values of the transformed filter U for K output and C input channels: 36 * K * C. */
size_t sd_winograd_filter_elems(int K, int C);

/*
 * U = 128 * G w G^T for every (k, c): w [K][3][3][C] -> U [36][K][C], both binary16 on the device.  (The factor
 * 128 keeps small weights out of binary16's subnormals; the forward call removes it.  |w| must stay below 512.)
 * Errors: INVALID_VALUE (null pointer, K or C <= 0), UNSUPPORTED (K or C not a multiple of 8), ALIGNMENT, ARCH, CUDA.
 */
int sd_winograd_transform_filter(const void *w, void *U, int K, int C, void *stream);

/* Bytes of device scratch a forward call of this shape needs (256-byte aligned): V, binary16 [36][T][C], then the
 * products M, binary32 [36][T][K], with T = N * ceil(H/4) * ceil(W/4) tiles.  0 for a bad shape. */
size_t sd_winograd_workspace_bytes(int N, int H, int W, int C, int K);

/*
 * y = conv3x3(x, w) + bias through the transformed domain.  U is what sd_winograd_transform_filter wrote for w.
 * `workspace` is caller-owned device scratch of at least sd_winograd_workspace_bytes(...) bytes, 256-byte aligned;
 * its contents after the call are unspecified.  N == 0 is an OK no-op.
 * Errors: INVALID_VALUE (null pointer, non-positive size), UNSUPPORTED (C or K not a multiple of 8, more than
 * 2^31 - 1 tiles or elements of a scratch plane), ALIGNMENT, WORKSPACE (scratch null, misaligned or too small),
 * ARCH, CUDA.  A bounded wait inside the kernel that expires sets a status block the next call of
 * sd_winograd_query_status reports.
 */
int sd_winograd_conv3x3_forward(const void *x, const void *U, const void *bias, void *y, void *workspace,
                                size_t workspace_bytes, int N, int H, int W, int C, int K, void *stream);

/* Synchronise `stream` and report (and clear) whether a kernel of this file's calls gave up on a wait on the current
 * device: SD_ATTN_OK or SD_ATTN_ERR_DEVICE_TIMEOUT; detail (may be NULL) receives four ints: flag, site, index, block. */
int sd_winograd_query_status(void *stream, int *detail);

#ifdef __cplusplus
}
#endif
#endif
