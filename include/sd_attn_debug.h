/*
 * sd_attn_debug.h -- bring-up hooks of the attention library.  Not part of the stable ABI.
 */
#ifndef SD_ATTN_DEBUG_H_
#define SD_ATTN_DEBUG_H_

#include "sd_attn.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Ask later CROSS-mode forwards of this handle to also store the raw tensor-core scores
 * q.k (before scaling; the matrix A of Sec. 3.2.1 divided by the scale) into `device_buffer`, a
 * caller-owned DEVICE array of binary32 laid out [B*H][ceil(Nq/128)][128][Nk rounded up to 16].
 * NULL switches the dump off (the default).  Returns an sd_attn_status.
 */
int sd_attn_debug_dump_cross_scores(sd_attn_handle *h, float *device_buffer);

#ifdef __cplusplus
}
#endif
#endif /* SD_ATTN_DEBUG_H_ */
