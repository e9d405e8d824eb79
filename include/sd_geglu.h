/*
 * sd_geglu.h -- C ABI of the fused GEGLU step of the B200 (sm_100a) library.
 *
 * The feed-forward block of every transformer layer of the Stable Diffusion 1.4 UNet projects to 2C channels,
 * splits the result into two halves, applies GELU to one and multiplies it into the other.  Sec. 3.1 of the paper
 * runs the error-function arithmetic of Eq. 2 together with the split and the multiplication as ONE kernel, with no
 * intermediate tensor; so does this entry point:
 *
 *     out[r][c] = x[r][c] * GELU(x[r][C + c]),     GELU(g) = g/2 * (1 + erf(g / sqrt 2))       (Eq. 2)
 *
 * for r in [0, rows), c in [0, C).  (The paper does not say which half is gated; the second is, as in the model it
 * accelerates.)  Status codes are those of sd_attn.h.
 */
#ifndef SD_GEGLU_H_
#define SD_GEGLU_H_

#include "sd_attn.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 *   x      DEVICE pointer, caller-owned: dense [rows][2 C], the 2 C channels of a row contiguous, 16-byte aligned
 *   out    DEVICE pointer, caller-owned: dense [rows][C], 16-byte aligned; must not overlap x
 *   rows   number of rows (tokens); 0 is an OK no-op
 *   C      channels of ONE half (the input has 2 C per row); any positive value, fastest when a multiple of 8
 *   dtype  SD_ATTN_F16 (binary16 in and out, binary32 arithmetic) or SD_ATTN_F32
 *   stream cudaStream_t passed as void* (NULL = the legacy default stream)
 * Asynchronous and stream-ordered: enqueues one kernel, does not synchronise, allocate or read back; needs no handle
 * (the operation has no state).  Validation happens before the launch: a non-OK return means nothing was enqueued.
 * Errors: INVALID_VALUE (null pointer, rows < 0, C <= 0, more than 2^31 - 1 sixteen-byte pieces per tensor... see
 * the limit below), UNSUPPORTED (dtype), ALIGNMENT, ARCH (the current device is not compute capability 10.x), CUDA.
 * Limit: rows * C < 2^40 elements.
 */
int sd_geglu_forward(const void *x, void *out, long long rows, int C, int dtype, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* SD_GEGLU_H_ */
