/*
 * sd_attn.h -- C ABI of the B200 (sm_100a) attention library.
 *
 * One operation:  out = softmax(Q K^T * scale) V  per (batch, head)      (paper Eq. 3),
 * the scaled-dot-product attention inside every transformer block of the Stable Diffusion
 * 1.4 UNet: self-attention (Nk == Nq = 4096/1024/256/64 latent tokens, head dim 40/80/160)
 * and cross-attention against Nk = 77 text tokens.  Sec. 3.2 of the paper describes two ways
 * to evaluate it -- a partially fused softmax over a materialised score matrix (Sec. 3.2.1,
 * Eq. 4) and FlashAttention (Sec. 3.2.2); both are exact, so every mode below returns the
 * same result up to rounding.
 *
 * Conventions that hold for every entry point
 *   - Pointers named q, k, v, out, workspace are DEVICE pointers owned by the caller; the
 *     library never allocates, frees or keeps them.  `stream` is a cudaStream_t passed as
 *     void* (NULL = the legacy default stream).  Handles are HOST objects; the status block a
 *     handle owns is DEVICE memory, read back only by sd_attn_query_status.
 *   - Layout: q and out are dense [B][H][Nq][d], k and v dense [B][H][Nk][d], d innermost,
 *     no strides -- or, after sd_attn_set_layout(SD_ATTN_LAYOUT_BNHD), dense [B][Nq][H][d] and
 *     [B][Nk][H][d]; `d` is the true head dim (padding to tensor-core widths is internal).
 *     `out` must not overlap any input.
 *   - Every function returns an sd_attn_status.  No function throws, aborts or exits.
 *     sd_attn_forward and sd_attn_forward_twopass_static validate before any launch: an argument
 *     error from them means nothing was enqueued (ERR_CUDA can come from a launch itself, in
 *     TWOPASS mode from the second of its two).  sd_attn_forward_batch and sd_attn_forward_host
 *     enqueue piece by piece: when they return an error, earlier problems or slices may already
 *     be enqueued, and the library's own streams have been joined back into `stream` in every case.
 *   - A handle belongs to the device that was current at sd_attn_create; every call that takes a
 *     handle returns INVALID_VALUE when another device is current.
 *   - sd_attn_forward is asynchronous and stream-ordered: it does not synchronise, allocate
 *     or read back.  One handle serves one host thread and one stream at a time (its status
 *     block and the streams of the host and batch entry points are per handle).
 */
#ifndef SD_ATTN_H_
#define SD_ATTN_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sd_attn_handle sd_attn_handle; /* opaque; created and destroyed by the library */

typedef enum {
    SD_ATTN_OK = 0,
    SD_ATTN_ERR_INVALID_VALUE = 1,  /* null pointer, non-positive size, non-finite scale, bad mode */
    SD_ATTN_ERR_UNSUPPORTED = 2,    /* dtype/d/Nk outside what the requested mode implements   */
    SD_ATTN_ERR_ALIGNMENT = 3,      /* a tensor pointer is not 16-byte aligned                  */
    SD_ATTN_ERR_WORKSPACE = 4,      /* two-pass mode without enough caller-provided scratch     */
    SD_ATTN_ERR_ARCH = 5,           /* the current device is not compute capability 10.x        */
    SD_ATTN_ERR_CUDA = 6,           /* a CUDA runtime/driver call failed                        */
    SD_ATTN_ERR_DEVICE_TIMEOUT = 7  /* a bounded wait inside a kernel expired (see query_status) */
} sd_attn_status;

typedef enum {
    SD_ATTN_F16 = 0, /* IEEE binary16 q/k/v/out, binary32 accumulation            */
    SD_ATTN_F32 = 1, /* binary32 throughout (plain FMA arithmetic, no TF32)        */
    SD_ATTN_BF16 = 2 /* bfloat16 q/k/v/out, binary32 accumulation; the softmax weights enter the second product
                        rounded to bfloat16 (8 significant bits), so results are about 8x coarser than F16's.
                        Implemented by FUSED, CROSS and SIMT; TWOPASS mode answers UNSUPPORTED.              */
} sd_attn_dtype;

typedef enum {
    SD_ATTN_MODE_AUTO = 0,    /* F16: CROSS when Nk fits one key tile, else FUSED.  F32: SIMT */
    SD_ATTN_MODE_FUSED = 1,   /* single-pass online softmax (FlashAttention, Sec. 3.2.2)      */
    SD_ATTN_MODE_CROSS = 2,   /* all keys in one shared-memory tile, plain softmax            */
    SD_ATTN_MODE_TWOPASS = 3, /* partially fused softmax of Sec. 3.2.1: scores and [L,S] in HBM */
    SD_ATTN_MODE_SIMT = 4     /* CUDA-core kernel, F16 or F32 storage, fp32 arithmetic        */
} sd_attn_mode;

typedef enum {
    SD_ATTN_LAYOUT_BHND = 0, /* head-major: q, out [B][H][Nq][d]; k, v [B][H][Nk][d] (the default)              */
    SD_ATTN_LAYOUT_BNHD = 1  /* token-major: q, out [B][Nq][H][d]; k, v [B][Nk][H][d] -- what a projection to
                                H*d channels leaves, so the head split before and the head merge after the
                                attention (Sec. 3.2) are views, not copies                                      */
} sd_attn_layout;

/* Largest Nk the CROSS mode accepts (one key tile). */
#define SD_ATTN_CROSS_MAX_NK 128
/* Largest head dim any mode accepts; F16 tensor-core modes need d to be a multiple of 8. */
#define SD_ATTN_MAX_D 160

/*
 * Choices a caller (or a test) can make when a handle is created.  All zero = the defaults; every non-default
 * choice selects a slower variant that exists for comparison and testing, with the same results within the
 * tolerance.  Nothing in the library's kernel selection depends on the process environment.
 */
typedef struct {
    size_t struct_size;    /* sizeof(sd_attn_options): lets the struct grow without breaking callers       */
    int no_pdl;            /* 1: launch every kernel the ordinary way.  By default the tensor-core kernels are
                              launched with programmatic stream serialization: a kernel may run its set-up
                              while the previous kernel of the stream finishes, and waits for that kernel to
                              complete before it reads or writes global memory, so stream order is kept      */
    int fused_tiles;       /* 1..4: fixed number of query tiles per CTA of the FUSED kernel (0: by problem size) */
    int fused_split;       /* FUSED with one query tile per CTA: 2 or 4 warpgroups share its key tiles, 1 none
                              (0: by head dim)                                                                */
    int fused_shares;      /* 1: FUSED deals the (group of query tiles, key tile) steps of a problem out in equal
                              shares to one CTA per SM, so that no SM idles in a last, partly filled wave; a group
                              whose key range is cut between CTAs is finished through scratch the handle then owns
                              (136 MB), by whichever piece arrives last, in a fixed order (the bits repeat).
                              Measured slower than whole groups on every shape tried (4096 tokens: 97 against 86
                              microseconds): off by default, kept as the tested basis of that scheme              */
    int cross_one_tile;    /* 1: CROSS runs one tile per CTA also for 65..80 keys                             */
    int host_one_slice;    /* 1: sd_attn_forward_host uses one slice, copies and kernel all on the caller's stream */
    int batch_serial;      /* 1: sd_attn_forward_batch runs its problems one after another on the caller's stream */
} sd_attn_options;

/*
 * Create a handle on the CURRENT CUDA device.  Checks the architecture (ERR_ARCH unless compute capability
 * 10.x), resolves the driver's tensor-map encoder, raises the kernels' dynamic shared-memory limits, allocates
 * the handle's device memory -- one 64-byte status block (and the scratch of `fused_shares`, if asked for) -- and
 * creates the two copy streams and ten events sd_attn_forward_host uses, and the three streams and four events of
 * sd_attn_forward_batch.  No stream work.  *out receives the handle (NULL on failure).
 * sd_attn_create(out) is sd_attn_create_ex(NULL, out): the defaults.  `options` may be NULL; it is read during
 * the call only.  Errors: INVALID_VALUE (null `out`, an option out of range, struct_size not that of a known
 * version), ARCH, CUDA.
 */
int sd_attn_create(sd_attn_handle **out);
int sd_attn_create_ex(const sd_attn_options *options, sd_attn_handle **out);

/*
 * out = softmax(q k^T * scale) v, Eq. 3, for every (b, h); see the conventions above.
 *   B, H, Nq, Nk, d : sizes; all > 0 except Nq == 0, which is an OK no-op.  Nk == 0 is
 *                     INVALID_VALUE (a softmax over no keys is undefined).
 *   scale           : the multiplier applied to q.k (1/sqrt(d) in the paper); any finite
 *                     value, used as given.
 *   dtype           : sd_attn_dtype of all four tensors.
 * Errors: INVALID_VALUE, UNSUPPORTED (d > SD_ATTN_MAX_D; F16 tensor-core modes with d % 8 != 0;
 * CROSS with Nk > SD_ATTN_CROSS_MAX_NK; F32 in a tensor-core mode), ALIGNMENT, WORKSPACE
 * (TWOPASS only), CUDA.
 */
int sd_attn_forward(sd_attn_handle *h, const void *q, const void *k, const void *v, void *out,
                    int B, int H, int Nq, int Nk, int d, float scale, int dtype, void *stream);

/* One problem of a batch: the arguments of sd_attn_forward. */
typedef struct {
    const void *q, *k, *v; /* device pointers, 16-byte aligned, in the handle's layout */
    void *out;
    int B, H, Nq, Nk, d;
    float scale;
} sd_attn_problem;

/*
 * `count` INDEPENDENT problems of Eq. 3 -- e.g. the attention calls of several UNet blocks evaluated side by side,
 * or of several requests -- as one piece of stream-ordered work on `stream`: no problem's output may be another's
 * input or output.  Problems of the same shape (B, H, Nq, Nk, d) that the same kernel serves become ONE launch of
 * that kernel over all of them (up to eight per launch for FUSED, five for the 77-key CROSS kernel; the 32 calls
 * of a UNet step are eight launches); the launches of different shapes are spread over `stream` and three streams
 * of the handle, forked from `stream` and joined back by events -- the launch with the most work first, on a stream
 * of the device's highest priority, so that the small shapes run in the SMs that its last wave leaves idle,
 * whatever the order of the problems in the list.  Capturable into a CUDA graph through `stream`.  All problems share `dtype`, the handle's mode and
 * layout; every problem is validated as by sd_attn_forward BEFORE anything is enqueued, and the first error is
 * returned with nothing enqueued (an error of a launch itself, ERR_CUDA, can leave earlier launches enqueued; the
 * streams are joined in every case).  Results are bitwise those of the same problems run one by one.
 * In TWOPASS mode (one workspace), in SIMT mode and with `batch_serial` set at creation the problems run one
 * after another on `stream`.  `problems` is a HOST array, read during the call only.
 * Errors: INVALID_VALUE (null handle, negative count, null array), then as sd_attn_forward.
 */
int sd_attn_forward_batch(sd_attn_handle *h, const sd_attn_problem *problems, int count, int dtype,
                          void *stream);

/*
 * The same operation (Eq. 3) for callers whose tensors live in HOST memory: q, k, v, out are HOST
 * pointers (pinned memory makes the copies asynchronous; pageable memory works but serialises).
 * `staging` is caller-owned DEVICE scratch of at least sd_attn_host_staging_bytes(...) bytes,
 * 256-byte aligned.  The work is the host-to-device copies of q, k and v, sd_attn_forward on the
 * staged tensors and the device-to-host copy of the result.  K and V are copied whole; Q and the result
 * are cut along the (batch, head) range into up to four slices (independent problems) whose copies run on
 * two streams owned by the handle, so that the copies of one slice overlap the kernel of another; the
 * slices are forked from `stream` and joined back into it by events, so for the caller the call is one
 * piece of stream-ordered work on `stream`.  (One slice, everything on `stream`, in TWOPASS mode or when a head of q or k is not a
 * multiple of 16 bytes.)  Does not synchronise: `out` is valid once the stream has drained.  Errors
 * as sd_attn_forward, plus WORKSPACE if `staging` is NULL, misaligned or too small.
 */
int sd_attn_forward_host(sd_attn_handle *h, const void *q, const void *k, const void *v, void *out,
                         void *staging, size_t staging_bytes, int B, int H, int Nq, int Nk, int d,
                         float scale, int dtype, void *stream);

/* Device scratch sd_attn_forward_host needs: q, k, v and out, each rounded up to 256 bytes. */
size_t sd_attn_host_staging_bytes(int B, int H, int Nq, int Nk, int d, int dtype);

/* Destroy a handle and its status block.  NULL is an OK no-op. */
int sd_attn_destroy(sd_attn_handle *h);

/* Choose the kernel family for later forwards (default AUTO). */
int sd_attn_set_mode(sd_attn_handle *h, int mode);

/*
 * Choose where the heads of q, k, v and out lie for later forwards (sd_attn_layout; default BHND).  All four
 * tensors of a call share the layout; each is dense in it.  BNHD is implemented by FUSED, CROSS and SIMT modes
 * (every dtype); TWOPASS mode answers UNSUPPORTED for it.  sd_attn_forward_host takes either layout (BNHD in
 * one slice).
 * Errors: INVALID_VALUE (null handle, unknown layout).
 */
int sd_attn_set_layout(sd_attn_handle *h, int layout);

/*
 * Scratch the TWOPASS mode needs for a call of this shape: the score matrix
 * A = q k^T * scale as binary32 [B][H][Nq][Nk] (Sec. 3.2.1) followed by the row statistics
 * [L, S] of Eq. 4 as binary32 [B][H][Nq][2].  Zero for every other mode.
 */
size_t sd_attn_workspace_bytes(int mode, int B, int H, int Nq, int Nk, int d, int dtype);

/* Lend caller-owned device scratch (256-byte aligned) to the handle; (NULL, 0) withdraws it. */
int sd_attn_set_workspace(sd_attn_handle *h, void *workspace, size_t bytes);

/*
 * After a TWOPASS forward: device pointers into the workspace of that call's score matrix and
 * [L,S] tensor (valid until the workspace is reused).  Either output pointer may be NULL.
 */
int sd_attn_twopass_buffers(sd_attn_handle *h, const float **scores, const float **row_stats);

/*
 * Synchronise `stream`, then read and clear the device status block.  Returns OK,
 * ERR_DEVICE_TIMEOUT (a kernel gave up a bounded wait and returned early: the outputs of the
 * calls since the last query are not valid) or ERR_CUDA.  If `detail` is non-NULL it receives
 * four host ints: {code, block index, wait site, tile index} of the first failure.  After a
 * time-out the handle's scratch counters are cleared as well, so the handle stays usable.
 */
int sd_attn_query_status(sd_attn_handle *h, void *stream, int *detail);

/*
 * Self-test of the failure path behind SD_ATTN_ERR_DEVICE_TIMEOUT (Eq. 3 has no part in it): enqueues on `stream`
 * a one-block kernel that takes the steps a tensor-core kernel of this library takes when a bounded wait runs
 * out -- with the same primitives, but a budget of a few thousand polls (under a millisecond): a thread waits on
 * a barrier nothing ever arrives on, gives up, raises the block's abort flag and records {1, block 0, site 99,
 * tile 7} in the handle's status block; a second waiter leaves on seeing the flag; the block releases its tensor
 * memory and returns normally.  Nothing traps, faults or waits without a limit.  The next sd_attn_query_status
 * returns ERR_DEVICE_TIMEOUT with that detail and clears it; the handle and the context stay usable.
 * Errors: INVALID_VALUE (null handle, wrong device), CUDA.
 */
int sd_attn_selftest_wait_timeout(sd_attn_handle *h, void *stream);

/*
 * Instruction-rate probes behind the joint roofline of the FUSED kernel (Eq. 3 costs one exponential and a few
 * multiply-adds per score element next to its 4 d tensor-core FLOPs; which unit bounds a head dim depends on their
 * rates).  Runs, twice, one block of 512 threads per SM that repeats `iters` (1 .. 2^20) trips of independent
 * chains of ONE operation on registers -- op 0: ex2.approx.ftz.f32; 1: fma.rn.f32; 2: fma.rn.f32x2 (two results per
 * instruction); 3: the kernels' exp2 / row-sum / binary16-pack sweep over 32 scores, every exponential on the
 * special-function unit; 4: the same with the share of them the d <= 48 kernel sends to the FMA pipe -- then
 * synchronises `stream` and returns, from the second run, the results per clock per SM (mean over the SMs) and the
 * SM clock in MHz that was in effect (clock64 against globaltimer).  At iters = 4096 a run takes 0.07 ms (op 1, 2) to
 * 2.2 ms (op 3); allocates nothing.  Errors: INVALID_VALUE, ARCH, CUDA.
 */
int sd_attn_ubench(int op, int iters, void *stream, double *results_per_clk_per_sm, double *sm_mhz);

/* Which kernel family the last successful forward used (an sd_attn_mode, never AUTO). */
int sd_attn_last_mode(const sd_attn_handle *h);

/* How many kernels of this library the handle has launched since it was created. */
long long sd_attn_launch_count(const sd_attn_handle *h);

/*
 * The two-pass evaluation for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this entry point exists for deployment, not for the method.)
 *
 * Who needs it: code that runs where cudaMalloc is unavailable or forbidden -- inside a host framework
 * that owns the whole device heap, in a process whose device memory was carved up at start-up, or on a
 * path where an allocation's implicit device-wide synchronisation is unacceptable.  Such callers can
 * neither create a handle (sd_attn_create allocates) nor lend a workspace.  Here the scratch of the
 * two-pass path (the binary32 score matrix and the [L, S] row statistics of Eq. 4) is a fixed array of
 * SD_ATTN_STATIC_MAX_SCRATCH bytes built into the library image; every GPU that loads the library holds
 * that array until the process exits, used or not.
 *
 * Arguments, layout and result are those of sd_attn_forward in TWOPASS mode with dtype SD_ATTN_F16 (q, k,
 * v, out are caller-owned DEVICE pointers; no handle).  The call allocates nothing: no cudaMalloc, no
 * cudaFree, no allocating library routine.
 *   - A call whose scratch need, sd_attn_workspace_bytes(SD_ATTN_MODE_TWOPASS, ...), exceeds
 *     SD_ATTN_STATIC_MAX_SCRATCH returns SD_ATTN_ERR_WORKSPACE and enqueues nothing (with SD_ATTN_LOG set
 *     the two sizes are printed).  F32 data or d % 8 != 0 is SD_ATTN_ERR_UNSUPPORTED.
 *   - The FIRST call on each device looks up the device address of the built-in array (with that device
 *     current) and raises the kernels' shared-memory limits; make that first call outside any stream
 *     capture.  Later calls only enqueue work on `stream`.
 *   - All calls on a device share the one array, which keeps whatever the previous call left in it; every
 *     call overwrites what it reads, so calls that follow one another on a stream are independent.  Calls
 *     that OVERLAP on the GPU (different streams, or different host threads without ordering) race on the
 *     array and produce garbage: serialise them.
 *   - A bounded wait that expires inside a kernel is recorded in a status word beside the array (zero from the
 *     first call's set-up on; written only by a kernel that gives up; read and cleared by
 *     sd_attn_static_query_status: there is no handle to query).
 *   - The array's device address is looked up once per device and kept for the life of the process: after a
 *     cudaDeviceReset of that device the kept address is stale and this entry point must not be used again in
 *     the process (the library cannot see the reset).
 */
#define SD_ATTN_STATIC_MAX_SCRATCH ((size_t)34 * 1024 * 1024)
int sd_attn_forward_twopass_static(const void *q, const void *k, const void *v, void *out, int B, int H,
                                   int Nq, int Nk, int d, float scale, int dtype, void *stream);

/*
 * The status word of sd_attn_forward_twopass_static on the current device (the paper has no counterpart
 * either): synchronises `stream`, reads and clears the word.  OK, ERR_DEVICE_TIMEOUT (a kernel of a static
 * call since the last query gave up a bounded wait: that call's output is not valid) or ERR_CUDA; `detail`
 * as for sd_attn_query_status.  Allocates nothing (a stream synchronisation and one small copy to the host).
 */
int sd_attn_static_query_status(void *stream, int *detail);

/* Static, NUL-terminated description of a status code. */
const char *sd_attn_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* SD_ATTN_H_ */
