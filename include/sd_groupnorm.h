/*
 * sd_groupnorm.h -- C ABI of the fused group normalisation of the B200 (sm_100a) library.
 *
 * Group normalisation sits in front of every convolution block and every transformer block of the Stable Diffusion
 * 1.4 UNet.  Sec. 3.1 of the paper runs its "reshape, mean, variance, normalize" as ONE kernel without intermediate
 * tensors; so does this entry point.  Per sample n and group g (G groups of C/G consecutive channels), over the
 * (C/G) * HW values of the group:
 *
 *     mu = mean(x),  sigma^2 = mean((x - mu)^2),  y[n][c][p] = (x[n][c][p] - mu) / sqrt(sigma^2 + eps) * gamma[c] + beta[c]
 *
 * (Eq. 1 of the paper; the epsilon and the per-channel affine are those of the operation it cites.)  Status codes are
 * those of sd_attn.h.
 */
#ifndef SD_GROUPNORM_H_
#define SD_GROUPNORM_H_

#include "sd_attn.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 *   x, y        DEVICE pointers, caller-owned: dense [N][C][HW], HW innermost (NCHW), 16-byte aligned; y may be x
 *               (in place) but must not overlap it otherwise
 *   gamma, beta DEVICE pointers to [C] values of the same dtype, or NULL (1 and 0)
 *   N, C, HW, G sizes: samples, channels, values per channel, groups; C must be a multiple of G; N == 0 is an OK no-op
 *   eps         added to the (biased) variance under the root; finite and >= 0
 *   dtype       SD_ATTN_F16 (binary16 storage, binary32 statistics and arithmetic) or SD_ATTN_F32
 *   stream      cudaStream_t passed as void* (NULL = the legacy default stream)
 * Asynchronous and stream-ordered: enqueues one kernel (one thread block per (sample, group)), does not synchronise,
 * allocate or read back; no handle.  The FIRST call in a process raises the kernel's shared-memory limit (a host-side
 * attribute call); make it outside any stream capture.  A non-OK return means nothing was enqueued.
 * Errors: INVALID_VALUE (null x or y, a size <= 0, C % G != 0, eps negative or not finite, more than 2^31 - 1 groups),
 * UNSUPPORTED (dtype), ALIGNMENT, ARCH (device not compute capability 10.x), CUDA.
 */
int sd_groupnorm_forward(const void *x, const void *gamma, const void *beta, void *y, int N, int C, long long HW, int G,
                         float eps, int dtype, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* SD_GROUPNORM_H_ */
