// Host side of the C ABI declared in include/sd_attn.h: handle management, argument validation,
// kernel selection, TMA tensor-map construction and launches.  No entry point here synchronises
// (except query_status, whose job it is), allocates in forward, or touches caller tensors on the host.
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
#include <mutex>

#include "../../include/sd_attn.h"
#include "../../include/sd_geglu.h"
#include "../../include/sd_groupnorm.h"
#include "../../include/sd_winograd.h"
#include "cross_kernel.cuh"
#include "cross2_kernel.cuh"
#include "geglu_kernel.cuh"
#include "groupnorm_kernel.cuh"
#include "winograd_kernel.cuh"
#include "fused4s_kernel.cuh"
#include "selftest_kernel.cuh"
#include "simt_kernel.cuh"
#include "twopass_kernel.cuh"
#include "ubench_kernel.cuh"

using namespace sd_attn;

typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// A tensor map depends only on (base address, shape, tile rows): encoding costs a few microseconds on
// the host, so the handle remembers the most recent ones.  Entries own nothing and are never dereferenced
// on the host; a stale entry is harmless because the key includes everything the encoding reads.
struct TmapCacheEntry {
    const void* base;
    int BH, N, d, box_rows;
    int heads;   // heads per batch entry of a token-major tensor, 0 for a head-major one
    int bf16;    // bfloat16 elements (binary16 otherwise)
    CUtensorMap map;
};
constexpr int TMAP_CACHE_ENTRIES = 128;

#ifndef SD_ATTN_BATCH_LANES
#define SD_ATTN_BATCH_LANES 3
#endif
constexpr int BATCH_LANES = SD_ATTN_BATCH_LANES;   // sd_attn_forward_batch spreads independent problems over the caller's stream and these

constexpr int HOST_SLICES = 4;   // sd_attn_forward_host cuts the (batch, head) range into at most this many slices

// Scratch of the FUSED kernel's shares mode (see fused4s_kernel.cuh): pieces and their arrival counters.
constexpr size_t PART_BYTES = (size_t)136 << 20;   // five 4096-token d = 40 problems in one launch need 128 MB
constexpr int PART_COUNTERS = 1 << 16;             // (problem, unit, tile) counters of one launch

struct sd_attn_handle {
    TmapCacheEntry tmap_cache[TMAP_CACHE_ENTRIES];
    int tmap_cache_next;
    int device;
    int mode;
    int layout;
    int last_mode;
    sd_attn_options opt;
    cudaStream_t batch_lane[BATCH_LANES];   // sd_attn_forward_batch: lanes beside the caller's stream
    cudaEvent_t ev_batch_fork, ev_batch_join[BATCH_LANES];
    int batch_lanes_ok;
    long long launches;
    int* dev_status;          // DEV_STATUS_INTS ints on the device
    float* part;              // PART_BYTES of pieces (FUSED, shares mode)
    int* part_count;          // PART_COUNTERS arrival counters, zero between launches
    void* workspace;          // caller-owned
    size_t workspace_bytes;
    const float* tp_scores;   // where the last TWOPASS call put A and [L,S]
    const float* tp_stats;
    encode_tiled_fn encode_tiled;
    cudaError_t last_cuda_error;
    int sm_count;
    int fused4s_ok;           // the register hand-over inside these kernels fits their launch allocation
    int cross2_four_ok;
    // sd_attn_forward_host: copies of one slice of heads overlap the kernel of another (see there)
    cudaStream_t copy_in, copy_out;
    cudaEvent_t ev_fork, ev_join, ev_in[HOST_SLICES], ev_done[HOST_SLICES];
    int host_overlap;         // the streams and events above exist
};

static const float LOG2E = 1.4426950408889634f;

extern "C" const char* sd_attn_status_string(int status) {
    switch (status) {
        case SD_ATTN_OK: return "ok";
        case SD_ATTN_ERR_INVALID_VALUE: return "invalid value";
        case SD_ATTN_ERR_UNSUPPORTED: return "unsupported dtype, head dim or size for the requested mode";
        case SD_ATTN_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
        case SD_ATTN_ERR_WORKSPACE: return "two-pass workspace missing or too small";
        case SD_ATTN_ERR_ARCH: return "device is not compute capability 10.x (sm_100)";
        case SD_ATTN_ERR_CUDA: return "a CUDA call failed";
        case SD_ATTN_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel expired";
        default: return "unknown status";
    }
}

static int cuda_fail(sd_attn_handle* h, cudaError_t e) {
    if (h) h->last_cuda_error = e;
    if (getenv("SD_ATTN_LOG")) fprintf(stderr, "[sd_attn] CUDA error: %s\n", cudaGetErrorString(e));
    return SD_ATTN_ERR_CUDA;
}

// Launch with the programmatic-stream-serialization attribute: the kernel may begin its set-up while the previous
// kernel of the stream is still running and waits for it (griddepcontrol.wait) before it touches global memory.
// Only the kernels that contain that wait are launched this way.
template <typename... KArgs, typename... Args>
static cudaError_t launch_overlapped_if(bool overlap, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                        cudaStream_t stream, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
template <typename... KArgs, typename... Args>
static cudaError_t launch_overlapped(const sd_attn_handle* h, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                     cudaStream_t stream, Args&&... args) {
    return launch_overlapped_if(!h->opt.no_pdl, kernel, grid, block, smem, stream, static_cast<Args&&>(args)...);
}

template <typename K>
static cudaError_t raise_smem_limit(K kernel, size_t bytes) {
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

// Two copy streams and the events that tie them to the caller's stream in sd_attn_forward_host.
static cudaError_t create_host_overlap(sd_attn_handle* h) {
    cudaError_t e = cudaStreamCreateWithFlags(&h->copy_in, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&h->copy_out, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming);
    for (int c = 0; c < HOST_SLICES && e == cudaSuccess; ++c) {
        e = cudaEventCreateWithFlags(&h->ev_in[c], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_done[c], cudaEventDisableTiming);
    }
    h->host_overlap = e == cudaSuccess && !h->opt.host_one_slice;
    // the lanes of sd_attn_forward_batch
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_batch_fork, cudaEventDisableTiming);
    // The first lane has the device's highest priority: it takes the launch with the most work of a batch, whose
    // CTAs then win every SM that frees up, and the small launches run in what its last, partly filled wave leaves
    // idle instead of pushing its waves back (measured on the 32 calls of a UNet step: see sd_attn_forward_batch).
    int prio_least = 0, prio_greatest = 0;
    if (e == cudaSuccess) e = cudaDeviceGetStreamPriorityRange(&prio_least, &prio_greatest);
    for (int l = 0; l < BATCH_LANES && e == cudaSuccess; ++l) {
        e = cudaStreamCreateWithPriority(&h->batch_lane[l], cudaStreamNonBlocking, l == 0 ? prio_greatest : prio_least);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_batch_join[l], cudaEventDisableTiming);
    }
    h->batch_lanes_ok = e == cudaSuccess && !h->opt.batch_serial;
    return e;
}

static void destroy_host_overlap(sd_attn_handle* h) {   // the handle was calloc'ed: what was never created is null
    for (int c = 0; c < HOST_SLICES; ++c) {
        if (h->ev_in[c]) cudaEventDestroy(h->ev_in[c]);
        if (h->ev_done[c]) cudaEventDestroy(h->ev_done[c]);
    }
    if (h->ev_fork) cudaEventDestroy(h->ev_fork);
    if (h->ev_join) cudaEventDestroy(h->ev_join);
    if (h->copy_in) cudaStreamDestroy(h->copy_in);
    if (h->copy_out) cudaStreamDestroy(h->copy_out);
    h->host_overlap = 0;
    for (int l = 0; l < BATCH_LANES; ++l) {
        if (h->ev_batch_join[l]) cudaEventDestroy(h->ev_batch_join[l]);
        if (h->batch_lane[l]) cudaStreamDestroy(h->batch_lane[l]);
    }
    if (h->ev_batch_fork) cudaEventDestroy(h->ev_batch_fork);
    h->batch_lanes_ok = 0;
}

// The kernels AUTO selects exist for binary16 and for bfloat16 tensors (BF); each needs its shared-memory limit raised.
template <bool BF>
static cudaError_t raise_layout_kernels() {
    cudaError_t e = raise_smem_limit(cross_attention_kernel<BF>, cross_smem_bytes(3, 128));
    if (e == cudaSuccess) e = raise_smem_limit(cross2_attention_kernel<2, BF, 1>, X2_SMEM_BUDGET + 1024);
    if (e == cudaSuccess) e = raise_smem_limit(cross2_attention_kernel<3, BF, 1>, X2_SMEM_BUDGET + 1024);
    if (e == cudaSuccess) e = raise_smem_limit(cross2_attention_kernel<4, BF, 1>, X2_SMEM_BUDGET + 1024);
    if (e == cudaSuccess) e = raise_smem_limit(cross2_attention_kernel<2, BF, X2_GROUP_MAX>, X2_SMEM_BUDGET + 1024);
    if (e == cudaSuccess) e = raise_smem_limit(cross2_attention_kernel<3, BF, X2_GROUP_MAX>, X2_SMEM_BUDGET + 1024);
    if (e == cudaSuccess) e = raise_smem_limit(cross2_attention_kernel<4, BF, X2_GROUP_MAX>, X2_SMEM_BUDGET + 1024);
    if (e == cudaSuccess) e = raise_smem_limit(fused4s_attention_kernel<F4S_POLY_PER8, 1, 1, BF>, F4S_SMEM_BUDGET + 1024);
    if (e == cudaSuccess) e = raise_smem_limit(fused4s_attention_kernel<0, 1, 1, BF>, F4S_SMEM_BUDGET + 1024);
    if (e == cudaSuccess) e = raise_smem_limit(fused4s_attention_kernel<0, 2, 1, BF>, F4S_SMEM_BUDGET + 1024);
    if (e == cudaSuccess) e = raise_smem_limit(fused4s_attention_kernel<0, 3, 1, BF>, F4S_SMEM_BUDGET + 1024);
    if (e == cudaSuccess) e = raise_smem_limit(fused4s_attention_kernel<F4S_POLY_PER8, 1, 4, BF>, F4S_SMEM_BUDGET + 1024);
    if (e == cudaSuccess) e = raise_smem_limit(fused4s_attention_kernel<F4S_POLY_PER8, 1, 2, BF>, F4S_SMEM_BUDGET + 1024);
    if (e == cudaSuccess) e = raise_smem_limit(fused4s_attention_kernel<F4S_POLY_PER8, 2, 2, BF>, F4S_SMEM_BUDGET + 1024);
    if (e == cudaSuccess) e = raise_smem_limit(fused4s_attention_kernel<F4S_POLY_PER8, 3, 2, BF>, F4S_SMEM_BUDGET + 1024);
    return e;
}

// Register budgets of the warp-specialised kernels (setmaxnreg pools must fit the launch allocation).
template <bool BF>
static cudaError_t check_register_pools(sd_attn_handle* h) {
    cudaFuncAttributes fa;
    cudaError_t e = cudaSuccess;
    const void* f4s[8] = {(const void*)fused4s_attention_kernel<F4S_POLY_PER8, 1, 1, BF>, (const void*)fused4s_attention_kernel<0, 1, 1, BF>,
                          (const void*)fused4s_attention_kernel<0, 2, 1, BF>, (const void*)fused4s_attention_kernel<0, 3, 1, BF>,
                          (const void*)fused4s_attention_kernel<F4S_POLY_PER8, 1, 4, BF>, (const void*)fused4s_attention_kernel<F4S_POLY_PER8, 1, 2, BF>,
                          (const void*)fused4s_attention_kernel<F4S_POLY_PER8, 2, 2, BF>,
                          (const void*)fused4s_attention_kernel<F4S_POLY_PER8, 3, 2, BF>};
    for (int i = 0; i < 8 && e == cudaSuccess; ++i) {
        e = cudaFuncGetAttributes(&fa, f4s[i]);
        if (e == cudaSuccess && F4_THREADS * fa.numRegs < 512 * F4S_SOFTMAX_REGS + 256 * F4S_CONTROL_REGS) h->fused4s_ok = 0;
    }
    if (e == cudaSuccess) e = cudaFuncGetAttributes(&fa, cross2_attention_kernel<4, BF, 1>);
    if (e == cudaSuccess && cross2_threads(4) * fa.numRegs < 512 * X2_SOFTMAX_REGS + 128 * X2_EPILOGUE_REGS + 128 * X2_CONTROL_REGS)
        h->cross2_four_ok = 0;
    if (e == cudaSuccess) e = cudaFuncGetAttributes(&fa, cross2_attention_kernel<4, BF, X2_GROUP_MAX>);
    if (e == cudaSuccess && cross2_threads(4) * fa.numRegs < 512 * X2_SOFTMAX_REGS + 128 * X2_EPILOGUE_REGS + 128 * X2_CONTROL_REGS)
        h->cross2_four_ok = 0;
    return e;
}

extern "C" int sd_attn_create_ex(const sd_attn_options* options, sd_attn_handle** out) {
    if (!out) return SD_ATTN_ERR_INVALID_VALUE;
    *out = nullptr;
    sd_attn_options opt;
    memset(&opt, 0, sizeof(opt));
    if (options) {
        if (options->struct_size != sizeof(sd_attn_options)) return SD_ATTN_ERR_INVALID_VALUE;
        opt = *options;
        const int flags[] = {opt.no_pdl, opt.cross_one_tile, opt.host_one_slice, opt.batch_serial};
        for (int f : flags)
            if (f != 0 && f != 1) return SD_ATTN_ERR_INVALID_VALUE;
        if (opt.fused_tiles < 0 || opt.fused_tiles > F4_TILES) return SD_ATTN_ERR_INVALID_VALUE;
        if (opt.fused_shares < 0 || opt.fused_shares > 1) return SD_ATTN_ERR_INVALID_VALUE;
        if (opt.fused_split != 0 && opt.fused_split != 1 && opt.fused_split != 2 && opt.fused_split != 4)
            return SD_ATTN_ERR_INVALID_VALUE;
    }
    opt.struct_size = sizeof(sd_attn_options);
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(nullptr, e);
    int major = 0, sms = 0;
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return cuda_fail(nullptr, e);
    if (major != 10) return SD_ATTN_ERR_ARCH;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);

    sd_attn_handle* h = (sd_attn_handle*)calloc(1, sizeof(sd_attn_handle));
    if (!h) return SD_ATTN_ERR_INVALID_VALUE;
    h->device = dev;
    h->mode = SD_ATTN_MODE_AUTO;
    h->last_mode = SD_ATTN_MODE_AUTO;
    h->sm_count = sms;
    h->opt = opt;

    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) {
        free(h);
        return cuda_fail(nullptr, e != cudaSuccess ? e : cudaErrorUnknown);
    }
    h->encode_tiled = (encode_tiled_fn)fn;

    // dynamic shared memory ceilings of every kernel, once
    e = raise_layout_kernels<false>();
    if (e == cudaSuccess) e = raise_layout_kernels<true>();
    if (e == cudaSuccess) e = raise_smem_limit(twopass_scores_kernel, twopass_scores_smem_bytes(3));
    if (e == cudaSuccess) e = raise_smem_limit(twopass_pv_kernel, twopass_pv_smem_bytes(3));
    if (e == cudaSuccess) e = raise_smem_limit(simt_attention_kernel<float, 5>, simt_smem_bytes(160));
    if (e == cudaSuccess) e = raise_smem_limit(simt_attention_kernel<__half, 5>, simt_smem_bytes(160));
    if (e == cudaSuccess) e = raise_smem_limit(simt_attention_kernel<float, 4>, simt_smem_bytes(128));
    if (e == cudaSuccess) e = raise_smem_limit(simt_attention_kernel<__half, 4>, simt_smem_bytes(128));
    if (e == cudaSuccess) e = raise_smem_limit(simt_attention_kernel<__nv_bfloat16, 5>, simt_smem_bytes(160));
    if (e == cudaSuccess) e = raise_smem_limit(simt_attention_kernel<__nv_bfloat16, 4>, simt_smem_bytes(128));
    // setmaxnreg budgets (see the kernels): a kernel whose increases its decreases do not cover is never launched
    if (e == cudaSuccess) {
        h->fused4s_ok = 1;
        h->cross2_four_ok = 1;
        e = check_register_pools<false>(h);
        if (e == cudaSuccess) e = check_register_pools<true>(h);
    }
    if (e == cudaSuccess) e = cudaMalloc((void**)&h->dev_status, sizeof(int) * DEV_STATUS_INTS);
    if (e == cudaSuccess) e = cudaMemset(h->dev_status, 0, sizeof(int) * DEV_STATUS_INTS);
    if (e == cudaSuccess && opt.fused_shares == 1) {   // (the scratch of the shares mode, only where it is asked for)
        e = cudaMalloc((void**)&h->part, PART_BYTES);
        if (e == cudaSuccess) e = cudaMalloc((void**)&h->part_count, sizeof(int) * PART_COUNTERS);
        if (e == cudaSuccess) e = cudaMemset(h->part_count, 0, sizeof(int) * PART_COUNTERS);
    }
    if (e == cudaSuccess) e = create_host_overlap(h);
    if (e != cudaSuccess) {
        destroy_host_overlap(h);
        if (h->dev_status) cudaFree(h->dev_status);
        if (h->part) cudaFree(h->part);
        if (h->part_count) cudaFree(h->part_count);
        free(h);
        return cuda_fail(nullptr, e);
    }
    *out = h;
    return SD_ATTN_OK;
}

extern "C" int sd_attn_create(sd_attn_handle** out) { return sd_attn_create_ex(nullptr, out); }

// A handle's kernels, status block and scratch belong to the device it was created on.
static bool on_handle_device(const sd_attn_handle* h) {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == h->device;
}

extern "C" int sd_attn_destroy(sd_attn_handle* h) {
    if (!h) return SD_ATTN_OK;
    cudaError_t e = cudaSuccess;
    destroy_host_overlap(h);
    if (h->dev_status) e = cudaFree(h->dev_status);
    if (h->part) cudaFree(h->part);
    if (h->part_count) cudaFree(h->part_count);
    free(h);
    return e == cudaSuccess ? SD_ATTN_OK : SD_ATTN_ERR_CUDA;
}

extern "C" int sd_attn_set_mode(sd_attn_handle* h, int mode) {
    if (!h || mode < SD_ATTN_MODE_AUTO || mode > SD_ATTN_MODE_SIMT) return SD_ATTN_ERR_INVALID_VALUE;
    h->mode = mode;
    return SD_ATTN_OK;
}

extern "C" int sd_attn_set_layout(sd_attn_handle* h, int layout) {
    if (!h || (layout != SD_ATTN_LAYOUT_BHND && layout != SD_ATTN_LAYOUT_BNHD)) return SD_ATTN_ERR_INVALID_VALUE;
    h->layout = layout;
    return SD_ATTN_OK;
}

extern "C" size_t sd_attn_workspace_bytes(int mode, int B, int H, int Nq, int Nk, int d, int dtype) {
    (void)d;
    (void)dtype;
    if (mode != SD_ATTN_MODE_TWOPASS || B <= 0 || H <= 0 || Nq <= 0 || Nk <= 0) return 0;
    const size_t rows = (size_t)B * H * Nq;
    const size_t scores = (rows * (size_t)Nk * sizeof(float) + 255) & ~(size_t)255;
    return scores + rows * 2 * sizeof(float);
}

extern "C" int sd_attn_set_workspace(sd_attn_handle* h, void* workspace, size_t bytes) {
    if (!h) return SD_ATTN_ERR_INVALID_VALUE;
    if ((workspace == nullptr) != (bytes == 0)) return SD_ATTN_ERR_INVALID_VALUE;
    if (((uintptr_t)workspace & 255u) != 0) return SD_ATTN_ERR_ALIGNMENT;
    h->workspace = workspace;
    h->workspace_bytes = bytes;
    return SD_ATTN_OK;
}

extern "C" int sd_attn_twopass_buffers(sd_attn_handle* h, const float** scores, const float** row_stats) {
    if (!h || !h->tp_scores) return SD_ATTN_ERR_INVALID_VALUE;
    if (scores) *scores = h->tp_scores;
    if (row_stats) *row_stats = h->tp_stats;
    return SD_ATTN_OK;
}

extern "C" int sd_attn_selftest_wait_timeout(sd_attn_handle* h, void* stream) {
    if (!h || !on_handle_device(h)) return SD_ATTN_ERR_INVALID_VALUE;
    selftest_wait_timeout_kernel<<<1, 128, 0, (cudaStream_t)stream>>>(h->dev_status, nullptr);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(h, e);
    h->launches += 1;
    return SD_ATTN_OK;
}

extern "C" int sd_attn_last_mode(const sd_attn_handle* h) { return h ? h->last_mode : SD_ATTN_MODE_AUTO; }
extern "C" long long sd_attn_launch_count(const sd_attn_handle* h) { return h ? h->launches : 0; }

extern "C" int sd_attn_query_status(sd_attn_handle* h, void* stream, int* detail) {
    if (!h || !on_handle_device(h)) return SD_ATTN_ERR_INVALID_VALUE;
    int host[DEV_STATUS_INTS];
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e = cudaStreamSynchronize(s);
    if (e == cudaSuccess) e = cudaMemcpy(host, h->dev_status, sizeof(host), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(h, e);
    if (detail) memcpy(detail, host, 4 * sizeof(int));
    if (host[0] != 0) {
        e = cudaMemset(h->dev_status, 0, sizeof(host));
        // a kernel that gave up may have left arrival counters of the shares mode behind
        if (e == cudaSuccess && h->part_count) e = cudaMemset(h->part_count, 0, sizeof(int) * PART_COUNTERS);
        if (e != cudaSuccess) return cuda_fail(h, e);
        return SD_ATTN_ERR_DEVICE_TIMEOUT;
    }
    return SD_ATTN_OK;
}

// The heads of a call's tensors: `heads` per batch entry when the tensors are token-major, 0 when head-major.
static HeadLayout head_layout(int heads, int BH, int N, int d) {
    HeadLayout l;
    if (heads > 0) {
        l.heads = heads; l.ld = heads * d; l.head_stride = d; l.batch_stride = (long long)N * heads * d;
    } else {
        l.heads = BH; l.ld = d; l.head_stride = (long long)N * d; l.batch_stride = (long long)BH * N * d;
    }
    return l;
}

static CUresult encode_tmap(encode_tiled_fn enc, CUtensorMap* map, const void* base, int heads, int BH, int N, int d,
                            int box_rows, int bf16 = 0) {
    const HeadLayout l = head_layout(heads, BH, N, d);
    cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)N, (cuuint64_t)l.heads, (cuuint64_t)(BH / l.heads)};
    cuuint64_t strides[3] = {(cuuint64_t)l.ld * 2, (cuuint64_t)l.head_stride * 2, (cuuint64_t)l.batch_stride * 2};
    cuuint32_t box[4] = {(cuuint32_t)CHUNK_COLS, (cuuint32_t)box_rows, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    return enc(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4,
               const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

// The same tensor as unswizzled tiles of exactly d columns by 128 rows: a tile lands in (or leaves) shared memory as
// dense rows of 2d bytes.  For the 77-key kernel's raw Q ring and output staging when a head's rows are not one
// contiguous run of memory (token-major tensors).
static CUresult encode_row_tmap(encode_tiled_fn enc, CUtensorMap* map, const void* base, int heads, int BH, int N, int d,
                                int bf16) {
    const HeadLayout l = head_layout(heads, BH, N, d);
    cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)N, (cuuint64_t)l.heads, (cuuint64_t)(BH / l.heads)};
    cuuint64_t strides[3] = {(cuuint64_t)l.ld * 2, (cuuint64_t)l.head_stride * 2, (cuuint64_t)l.batch_stride * 2};
    cuuint32_t box[4] = {(cuuint32_t)d, (cuuint32_t)TILE_M, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    return enc(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4,
               const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

// An fp16 tensor of BH heads of N rows of d values seen by the TMA as (x = d, y = N, z = head, w = batch): tiles are
// 64 columns wide (one 128-byte swizzled row) by `box_rows` rows.  Columns >= d and rows >= N read as zero.
static int make_tmap(sd_attn_handle* h, CUtensorMap* map, const void* base, int BH, int N, int d, int box_rows,
                     int heads = 0, int bf16 = 0) {
    for (int i = 0; i < TMAP_CACHE_ENTRIES; ++i) {
        const TmapCacheEntry& e = h->tmap_cache[i];
        if (e.base == base && e.BH == BH && e.N == N && e.d == d && e.box_rows == box_rows && e.heads == heads && e.bf16 == bf16) {
            *map = e.map;
            return SD_ATTN_OK;
        }
    }
    CUresult r = encode_tmap(h->encode_tiled, map, base, heads, BH, N, d, box_rows, bf16);
    if (r != CUDA_SUCCESS) {
        if (getenv("SD_ATTN_LOG")) fprintf(stderr, "[sd_attn] cuTensorMapEncodeTiled failed: %d\n", (int)r);
        h->last_cuda_error = cudaErrorInvalidValue;
        return SD_ATTN_ERR_CUDA;
    }
    TmapCacheEntry& slot = h->tmap_cache[h->tmap_cache_next];
    h->tmap_cache_next = (h->tmap_cache_next + 1) % TMAP_CACHE_ENTRIES;
    slot.base = base; slot.BH = BH; slot.N = N; slot.d = d; slot.box_rows = box_rows; slot.heads = heads; slot.bf16 = bf16;
    slot.map = *map;
    return SD_ATTN_OK;
}

static int next_pow2_cols(int cols) {
    int p = 32;
    while (p < cols) p <<= 1;
    return p;
}

struct Problem {
    const void *q, *k, *v;
    void* out;
    int BH, Nq, Nk, d;
    float scale;
    cudaStream_t stream;
    int heads;   // token-major tensors: heads per batch entry; head-major: 0
    int bf16;    // bfloat16 tensors (binary16 otherwise); tensor-core kernels only
};

template <typename T>
static int launch_simt(sd_attn_handle* h, const Problem& p) {
    dim3 grid((p.Nq + SIMT_BLOCK_ROWS - 1) / SIMT_BLOCK_ROWS, p.BH), block(SIMT_WARPS * 32);
    const size_t smem = simt_smem_bytes(p.d);
    const T *q = (const T*)p.q, *k = (const T*)p.k, *v = (const T*)p.v;
    T* o = (T*)p.out;
    const HeadLayout lq = head_layout(p.heads, p.BH, p.Nq, p.d), lk = head_layout(p.heads, p.BH, p.Nk, p.d);
    switch ((p.d + 31) / 32) {
        case 1: simt_attention_kernel<T, 1><<<grid, block, smem, p.stream>>>(q, k, v, o, p.Nq, p.Nk, p.d, p.scale, lq, lk); break;
        case 2: simt_attention_kernel<T, 2><<<grid, block, smem, p.stream>>>(q, k, v, o, p.Nq, p.Nk, p.d, p.scale, lq, lk); break;
        case 3: simt_attention_kernel<T, 3><<<grid, block, smem, p.stream>>>(q, k, v, o, p.Nq, p.Nk, p.d, p.scale, lq, lk); break;
        case 4: simt_attention_kernel<T, 4><<<grid, block, smem, p.stream>>>(q, k, v, o, p.Nq, p.Nk, p.d, p.scale, lq, lk); break;
        default: simt_attention_kernel<T, 5><<<grid, block, smem, p.stream>>>(q, k, v, o, p.Nq, p.Nk, p.d, p.scale, lq, lk); break;
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(h, e);
    h->launches += 1;
    return SD_ATTN_OK;
}

// 65..80 keys (the 77 text tokens): one persistent CTA per SM walks a range of (head, tile) items of `n` problems of
// ONE shape (BH, Nq, Nk, d, layout, dtype alike) -- one launch.
template <int NP>
static int launch_cross2_np(sd_attn_handle* h, const Problem* ps, int n) {
    const Problem& p = ps[0];
    Cross2ArgsT<NP> a;
    a.n_prob = n; a.BH = p.BH;
    a.lay = head_layout(p.heads, p.BH, p.Nq, p.d);
    a.Nq = p.Nq; a.Nk = p.Nk; a.d = p.d;
    a.dpad = (p.d + 15) / 16 * 16;
    a.nch = (p.d + CHUNK_COLS - 1) / CHUNK_COLS;
    a.stages = cross2_stages(a.nch);
    a.tiles_per_bh = (p.Nq + TILE_M - 1) / TILE_M;
    a.n_items = n * p.BH * a.tiles_per_bh;
    a.status = h->dev_status;
    int groups = cross2_groups(p.d);
    if (groups >= 4 && !h->cross2_four_ok) groups = 3;
    // The four-group variant moves whole Q and output tiles: as single contiguous runs when the tensors are
    // head-major, as unswizzled tiles of d columns (two more tensor maps) when they are token-major.
    a.strided_rows = (groups >= 4 && p.heads > 0) ? 1 : 0;
    for (int i = 0; i < n; ++i) {
        const Problem& pi = ps[i];
        Cross2Problem& cp = a.prob[i];
        int rc = make_tmap(h, &cp.tq, pi.q, pi.BH, pi.Nq, pi.d, TILE_M, pi.heads, pi.bf16);
        if (rc == SD_ATTN_OK) rc = make_tmap(h, &cp.tk, pi.k, pi.BH, pi.Nk, pi.d, X2_KN, pi.heads, pi.bf16);
        if (rc == SD_ATTN_OK) rc = make_tmap(h, &cp.tv, pi.v, pi.BH, pi.Nk, pi.d, X2_KN, pi.heads, pi.bf16);
        if (rc != SD_ATTN_OK) return rc;
        cp.tq_rows = cp.tq;
        cp.tout_rows = cp.tq;
        if (a.strided_rows) {
            if (encode_row_tmap(h->encode_tiled, &cp.tq_rows, pi.q, pi.heads, pi.BH, pi.Nq, pi.d, pi.bf16) != CUDA_SUCCESS ||
                encode_row_tmap(h->encode_tiled, &cp.tout_rows, pi.out, pi.heads, pi.BH, pi.Nq, pi.d, pi.bf16) != CUDA_SUCCESS) {
                h->last_cuda_error = cudaErrorInvalidValue;
                return SD_ATTN_ERR_CUDA;
            }
        }
        cp.q = (const __half*)pi.q;
        cp.out = (__half*)pi.out;
        cp.scale_log2e = fabsf(pi.scale) * LOG2E;
        cp.negate = pi.scale < 0.f;
    }
    const int grid = a.n_items < h->sm_count ? a.n_items : h->sm_count;
    size_t smem = cross2_smem_bytes(a.nch);
    if (groups >= 4) {   // d <= 48: Q tiles arrive as raw bulk copies and are rewritten in shared memory
        a.stages = cross2_dense_stages(p.d);
        smem = cross2_dense_smem_bytes(p.d);
    }
    const dim3 g(grid);
    if (p.bf16) {
        if (groups >= 4) launch_overlapped(h, cross2_attention_kernel<4, true, NP>, g, dim3(cross2_threads(4)), smem, p.stream, a);
        else if (groups == 3) launch_overlapped(h, cross2_attention_kernel<3, true, NP>, g, dim3(cross2_threads(3)), smem, p.stream, a);
        else launch_overlapped(h, cross2_attention_kernel<2, true, NP>, g, dim3(cross2_threads(2)), smem, p.stream, a);
    } else {
        if (groups >= 4) launch_overlapped(h, cross2_attention_kernel<4, false, NP>, g, dim3(cross2_threads(4)), smem, p.stream, a);
        else if (groups == 3) launch_overlapped(h, cross2_attention_kernel<3, false, NP>, g, dim3(cross2_threads(3)), smem, p.stream, a);
        else launch_overlapped(h, cross2_attention_kernel<2, false, NP>, g, dim3(cross2_threads(2)), smem, p.stream, a);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(h, e);
    h->launches += 1;
    return SD_ATTN_OK;
}

static int launch_cross2_group(sd_attn_handle* h, const Problem* ps, int n) {
    if (n < 1 || n > X2_GROUP_MAX) return SD_ATTN_ERR_INVALID_VALUE;
    return n == 1 ? launch_cross2_np<1>(h, ps, 1) : launch_cross2_np<X2_GROUP_MAX>(h, ps, n);
}

static int launch_cross2(sd_attn_handle* h, const Problem& p) { return launch_cross2_group(h, &p, 1); }

static int launch_cross(sd_attn_handle* h, const Problem& p) {
    if (cross2_supports(p.Nk, p.d) && !h->opt.cross_one_tile) return launch_cross2(h, p);
    CrossArgs a;
    a.out = (__half*)p.out;
    a.lay = head_layout(p.heads, p.BH, p.Nq, p.d);
    a.Nq = p.Nq; a.Nk = p.Nk; a.d = p.d;
    a.kn = (p.Nk + 15) / 16 * 16;
    a.dpad = (p.d + 15) / 16 * 16;
    a.nch = (p.d + CHUNK_COLS - 1) / CHUNK_COLS;
    a.tmem_cols = next_pow2_cols(a.kn + a.dpad);
    a.scale_log2e = fabsf(p.scale) * LOG2E;
    a.negate = p.scale < 0.f;
    a.status = h->dev_status;
    CUtensorMap tq, tk, tv;
    int rc = make_tmap(h, &tq, p.q, p.BH, p.Nq, p.d, TILE_M, p.heads, p.bf16);
    if (rc == SD_ATTN_OK) rc = make_tmap(h, &tk, p.k, p.BH, p.Nk, p.d, a.kn, p.heads, p.bf16);
    if (rc == SD_ATTN_OK) rc = make_tmap(h, &tv, p.v, p.BH, p.Nk, p.d, a.kn, p.heads, p.bf16);
    if (rc != SD_ATTN_OK) return rc;
    dim3 grid((p.Nq + TILE_M - 1) / TILE_M, p.BH), block(CROSS_THREADS);
    if (p.bf16)
        launch_overlapped(h, cross_attention_kernel<true>, grid, block, cross_smem_bytes(a.nch, a.kn), p.stream, tq, tk, tv, a);
    else
        launch_overlapped(h, cross_attention_kernel<false>, grid, block, cross_smem_bytes(a.nch, a.kn), p.stream, tq, tk, tv, a);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(h, e);
    h->launches += 1;
    return SD_ATTN_OK;
}

template <bool BF>
static void dispatch_fused4s(sd_attn_handle* h, int split, const Fused4Args& a, dim3 grid, dim3 block, size_t smem,
                             cudaStream_t stream) {
    if (split == 4 && a.nch == 1)
        launch_overlapped(h, fused4s_attention_kernel<F4S_POLY_PER8, 1, 4, BF>, grid, block, smem, stream, a);
    else if (split == 2 && a.nch == 1)
        launch_overlapped(h, fused4s_attention_kernel<F4S_POLY_PER8, 1, 2, BF>, grid, block, smem, stream, a);
    else if (split == 2 && a.nch == 2)
        launch_overlapped(h, fused4s_attention_kernel<F4S_POLY_PER8, 2, 2, BF>, grid, block, smem, stream, a);
    else if (split == 2 && a.nch == 3)
        launch_overlapped(h, fused4s_attention_kernel<F4S_POLY_PER8, 3, 2, BF>, grid, block, smem, stream, a);
    // the polynomial share of the exponentials only pays where four tiles saturate the special function unit
    else if (a.dpad <= 48)
        launch_overlapped(h, fused4s_attention_kernel<F4S_POLY_PER8, 1, 1, BF>, grid, block, smem, stream, a);
    else if (a.nch == 1)
        launch_overlapped(h, fused4s_attention_kernel<0, 1, 1, BF>, grid, block, smem, stream, a);
    else if (a.nch == 2)
        launch_overlapped(h, fused4s_attention_kernel<0, 2, 1, BF>, grid, block, smem, stream, a);
    else
        launch_overlapped(h, fused4s_attention_kernel<0, 3, 1, BF>, grid, block, smem, stream, a);
}

// How the FUSED kernel lays a problem out: query tiles per unit, whole units or shares.  A function of the problem's
// shape alone, so that a problem gets the same arithmetic whatever else shares its launch.
struct FusedPlan {
    int tiles_per_cta, units_per_head, n_units, n_kv;
    int shares;       // every CTA takes a share of every problem's (unit, key tile) steps; 0: one CTA per unit
    int slot_floats;  // shares: floats of one piece slot
    int grid;         // shares: CTAs (one per SM, but never more than a problem has steps: no CTA without a step)
    int max_group;    // problems of this shape one launch can take (shares: the scratch bounds it)
};

static FusedPlan plan_fused(const sd_attn_handle* h, const Problem& p) {
    const int dpad = (p.d + 15) / 16 * 16, nch = (p.d + CHUNK_COLS - 1) / CHUNK_COLS;
    const int q_tile_bytes = nch * TILE_M * CHUNK_ROW_BYTES, stage_bytes = 2 * nch * F4_BN * CHUNK_ROW_BYTES;
    // Tiles per unit: the fewest key-tile steps per CTA times the cost of one step of a CTA with that many tiles
    // (clocks, measured at d = 40: four tiles share the exponential unit, one tile alone is bound by its hand-off
    // chain), among the counts tensor memory and shared memory (at least two K/V stages) have room for.  Dealing a
    // problem's steps out in shares (only on request: sd_attn_options::fused_shares) costs, measured on the 4096-token
    // call, about five steps' time at every change of segment (the last tiles' epilogue, the barriers, the refill of
    // the pipeline) and about seven for a piece's trip through the scratch and the combination at the end.
    static const int step_cost[F4_TILES + 1] = {0, 1000, 1400, 1900, 2400};
    const int tiles_per_head = (p.Nq + TILE_M - 1) / TILE_M;
    int max_tiles = f4s_max_tiles(dpad);
    // (at least three K/V stages: the issuer of the rotation's last tile asks for key tile j + 2 before it multiplies
    // key tile j, which a ring of two could never deliver)
    while (max_tiles > 1 && F4S_SMEM_BUDGET - max_tiles * q_tile_bytes < 3 * stage_bytes) --max_tiles;
    FusedPlan best = {};
    double best_cost = -1.0;
    const int n_kv = (p.Nk + F4_BN - 1) / F4_BN;
    for (int tpc = 1; tpc <= max_tiles; ++tpc) {
        if (h->opt.fused_tiles > 0 && h->opt.fused_tiles <= max_tiles && tpc != h->opt.fused_tiles) continue;
        FusedPlan f = {};
        f.tiles_per_cta = tpc;
        f.units_per_head = (tiles_per_head + tpc - 1) / tpc;
        f.n_units = f.units_per_head * p.BH;
        f.n_kv = n_kv;
        f.slot_floats = tpc * (dpad + 2) * TILE_M;   // per tile: dpad columns of O, anchor, row sum; 128 rows each
        const double whole_steps = (double)((f.n_units + h->sm_count - 1) / h->sm_count) * n_kv;
        double steps = whole_steps;
        f.max_group = F4_GROUP_MAX;
        // shares: the handle has the scratch, two slots per CTA fit it, one counter per (unit, tile); W below 2^31
        const size_t slots_bytes = (size_t)2 * h->sm_count * f.slot_floats * sizeof(float);
        const bool can_share = tpc >= 2 && h->part && h->opt.fused_shares == 1 && slots_bytes <= PART_BYTES &&
                               (long)f.n_units * F4_TILES <= PART_COUNTERS && f.n_units >= 2 &&
                               (long long)f.n_units * n_kv < (1ll << 30);
        if (can_share) {
            const long W = (long)f.n_units * n_kv;
            f.grid = W < h->sm_count ? (int)W : h->sm_count;
            const double share = (double)W / f.grid;                          // steps of the problem per CTA
            const double segments = share / n_kv + 1.0;                       // about: a cut begins a new one
            steps = share + 5.0 * (segments - 1.0) + 7.0;
            f.shares = 1;
            const long by_slots = (long)(PART_BYTES / slots_bytes), by_counters = PART_COUNTERS / ((long)f.n_units * F4_TILES);
            const long cap = by_slots < by_counters ? by_slots : by_counters;
            if (cap < f.max_group) f.max_group = (int)cap;
        }
        const double cost = steps * step_cost[tpc];
        if (best_cost < 0 || cost < best_cost) {
            best_cost = cost;
            best = f;
        }
    }
    return best;
}

// The single-pass kernel for `n` problems of ONE shape (BH, Nq, Nk, d, layout, dtype alike): one launch.
static int launch_fused_group(sd_attn_handle* h, const Problem* ps, int n) {
    if (!h->fused4s_ok) return SD_ATTN_ERR_UNSUPPORTED;
    const Problem& p = ps[0];
    const FusedPlan plan = plan_fused(h, p);
    if (n < 1 || n > plan.max_group) return SD_ATTN_ERR_INVALID_VALUE;
    Fused4Args a;
    a.lay = head_layout(p.heads, p.BH, p.Nq, p.d);
    a.n_prob = n; a.BH = p.BH;
    a.Nq = p.Nq; a.Nk = p.Nk; a.d = p.d;
    a.dpad = (p.d + 15) / 16 * 16;
    a.nch = (p.d + CHUNK_COLS - 1) / CHUNK_COLS;
    a.tiles_per_cta = plan.tiles_per_cta;
    a.units_per_head = plan.units_per_head;
    a.n_units = plan.n_units;
    a.n_kv = plan.n_kv;
    a.shares = plan.shares;
    a.status = h->dev_status;
    a.part = h->part;
    a.part_count = h->part_count;
    a.part_slot_floats = plan.slot_floats;
    const int q_tile_bytes = a.nch * TILE_M * CHUNK_ROW_BYTES, stage_bytes = 2 * a.nch * F4_BN * CHUNK_ROW_BYTES;
    // one chunk per row: the kernel lays out four tile slots and eight stages whatever tiles_per_cta is (192 KB)
    const int tile_slots = a.nch == 1 ? F4_TILES : a.tiles_per_cta;
    a.stages = (F4S_SMEM_BUDGET - tile_slots * q_tile_bytes) / stage_bytes;
    if (a.stages > F4_STAGES) a.stages = F4_STAGES;
    if (a.stages < 3) return SD_ATTN_ERR_UNSUPPORTED;   // (cannot happen for d <= SD_ATTN_MAX_D: one 160-wide tile leaves three)
    const size_t smem = (size_t)tile_slots * q_tile_bytes + (size_t)a.stages * stage_bytes + 1024;
    for (int i = 0; i < n; ++i) {
        const Problem& pi = ps[i];
        Fused4Problem& fp = a.prob[i];
        int rc = make_tmap(h, &fp.tq, pi.q, pi.BH, pi.Nq, pi.d, TILE_M, pi.heads, pi.bf16);
        if (rc == SD_ATTN_OK) rc = make_tmap(h, &fp.tk, pi.k, pi.BH, pi.Nk, pi.d, F4_BN, pi.heads, pi.bf16);
        if (rc == SD_ATTN_OK) rc = make_tmap(h, &fp.tv, pi.v, pi.BH, pi.Nk, pi.d, F4_BN, pi.heads, pi.bf16);
        if (rc != SD_ATTN_OK) return rc;
        fp.out = (__half*)pi.out;
        fp.scale_log2e = fabsf(pi.scale) * LOG2E;
        fp.negate = pi.scale < 0.f;
    }
    dim3 grid(plan.shares ? plan.grid : plan.n_units * n), block(F4_THREADS);
    // One tile per unit: its key tiles are dealt out among 4 or 2 warpgroups (parts), each with an accumulator of its
    // own in tensor memory next to the score buffers, whose number is a multiple of the parts (a buffer then always
    // meets the same part) and smaller than the K/V ring (a buffer ahead is a key tile ahead).
    int split = 1;
    a.split_buffers = 2;
    if (a.tiles_per_cta == 1 && h->opt.fused_split != 1) {
        split = 4 * F4_BN + 4 * a.dpad <= 512 ? 4 : 2;
        if (h->opt.fused_split == 2) split = 2;
        a.split_buffers = (4 * F4_BN + split * a.dpad <= 512 && a.stages >= 5) ? 4 : 2;
        if (a.split_buffers < split || 2 * F4_BN + 2 * a.dpad > 512) split = 1;   // (no room: d > 192)
    }
    if (p.bf16)
        dispatch_fused4s<true>(h, split, a, grid, block, smem, p.stream);
    else
        dispatch_fused4s<false>(h, split, a, grid, block, smem, p.stream);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(h, e);
    h->launches += 1;
    return SD_ATTN_OK;
}

static int launch_fused(sd_attn_handle* h, const Problem& p) { return launch_fused_group(h, &p, 1); }

static int launch_twopass(sd_attn_handle* h, const Problem& p) {
    // (the comparator is head-major binary16 only and needs its workspace: validate_problem has checked both)
    const size_t rows = (size_t)p.BH * p.Nq;
    float* scores = (float*)h->workspace;
    float* stats = (float*)((char*)h->workspace + ((rows * (size_t)p.Nk * sizeof(float) + 255) & ~(size_t)255));
    TwoPassArgs a;
    twopass_fill_args(&a, scores, stats, (__half*)p.out, p.Nq, p.Nk, p.d, p.scale, h->dev_status);
    CUtensorMap tq, tk, tv;
    int rc = make_tmap(h, &tq, p.q, p.BH, p.Nq, p.d, TILE_M);
    if (rc == SD_ATTN_OK) rc = make_tmap(h, &tk, p.k, p.BH, p.Nk, p.d, TWOPASS_BN);
    if (rc == SD_ATTN_OK) rc = make_tmap(h, &tv, p.v, p.BH, p.Nk, p.d, TWOPASS_BN);
    if (rc != SD_ATTN_OK) return rc;
    dim3 grid((p.Nq + TILE_M - 1) / TILE_M, p.BH);
    // pass 1 (Sec. 3.2.1): A = q k^T * scale to HBM, per-block partial (max, sum), final [L, S]
    twopass_scores_kernel<<<grid, TWOPASS_THREADS, twopass_scores_smem_bytes(a.nch), p.stream>>>(tq, tk, a);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(h, e);
    // pass 2: exp(a - L) / S applied while A is loaded as the left operand of the product with V
    twopass_pv_kernel<<<grid, TWOPASS_THREADS, twopass_pv_smem_bytes(a.nch), p.stream>>>(tv, a);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(h, e);
    h->launches += 2;
    h->tp_scores = scores;
    h->tp_stats = stats;
    return SD_ATTN_OK;
}

// Argument checks of one problem, before anything is enqueued; *mode_out receives the kernel family that serves it.
// Returns OK with *mode_out = -1 for an empty problem (Nq == 0).
static int validate_problem(const sd_attn_handle* h, const void* q, const void* k, const void* v, const void* out, int B,
                            int H, int Nq, int Nk, int d, float scale, int dtype, int* mode_out) {
    *mode_out = -1;
    if (B <= 0 || H <= 0 || Nq < 0 || Nk <= 0 || d <= 0) return SD_ATTN_ERR_INVALID_VALUE;
    if (!isfinite(scale)) return SD_ATTN_ERR_INVALID_VALUE;
    if (dtype != SD_ATTN_F16 && dtype != SD_ATTN_F32 && dtype != SD_ATTN_BF16) return SD_ATTN_ERR_UNSUPPORTED;
    if (d > SD_ATTN_MAX_D) return SD_ATTN_ERR_UNSUPPORTED;
    if ((long long)B * H > 65535) return SD_ATTN_ERR_UNSUPPORTED;
    if (Nq == 0) return SD_ATTN_OK;
    if (!q || !k || !v || !out) return SD_ATTN_ERR_INVALID_VALUE;
    if ((((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out) & 15u) != 0) return SD_ATTN_ERR_ALIGNMENT;
    int mode = h->mode;
    const bool tensor_ok = (dtype == SD_ATTN_F16 || dtype == SD_ATTN_BF16) && (d % 8 == 0);
    if (mode == SD_ATTN_MODE_AUTO) {
        if (!tensor_ok) mode = SD_ATTN_MODE_SIMT;
        else mode = (Nk <= SD_ATTN_CROSS_MAX_NK) ? SD_ATTN_MODE_CROSS : SD_ATTN_MODE_FUSED;
    }
    if (mode != SD_ATTN_MODE_SIMT && !tensor_ok) return SD_ATTN_ERR_UNSUPPORTED;
    if (mode == SD_ATTN_MODE_CROSS && Nk > SD_ATTN_CROSS_MAX_NK) return SD_ATTN_ERR_UNSUPPORTED;
    if (mode == SD_ATTN_MODE_TWOPASS) {
        if (h->layout == SD_ATTN_LAYOUT_BNHD || dtype == SD_ATTN_BF16) return SD_ATTN_ERR_UNSUPPORTED;
        const size_t need = sd_attn_workspace_bytes(SD_ATTN_MODE_TWOPASS, B, H, Nq, Nk, d, dtype);
        if (!h->workspace || h->workspace_bytes < need) return SD_ATTN_ERR_WORKSPACE;
    }
    *mode_out = mode;
    return SD_ATTN_OK;
}

static Problem make_problem(const sd_attn_handle* h, const void* q, const void* k, const void* v, void* out, int B, int H,
                            int Nq, int Nk, int d, float scale, int dtype, cudaStream_t stream) {
    Problem p = {q, k, v, out, B * H, Nq, Nk, d, scale, stream, h->layout == SD_ATTN_LAYOUT_BNHD ? H : 0,
                 dtype == SD_ATTN_BF16 ? 1 : 0};
    return p;
}

static int launch_one(sd_attn_handle* h, const Problem& p, int mode, int dtype) {
    switch (mode) {
        case SD_ATTN_MODE_SIMT:
            return dtype == SD_ATTN_F16    ? launch_simt<__half>(h, p)
                   : dtype == SD_ATTN_BF16 ? launch_simt<__nv_bfloat16>(h, p)
                                           : launch_simt<float>(h, p);
        case SD_ATTN_MODE_CROSS: return launch_cross(h, p);
        case SD_ATTN_MODE_FUSED: return launch_fused(h, p);
        case SD_ATTN_MODE_TWOPASS: return launch_twopass(h, p);
        default: return SD_ATTN_ERR_INVALID_VALUE;
    }
}

extern "C" int sd_attn_forward(sd_attn_handle* h, const void* q, const void* k, const void* v, void* out, int B, int H,
                               int Nq, int Nk, int d, float scale, int dtype, void* stream) {
    if (!h) return SD_ATTN_ERR_INVALID_VALUE;
    int mode;
    int rc = validate_problem(h, q, k, v, out, B, H, Nq, Nk, d, scale, dtype, &mode);
    if (rc != SD_ATTN_OK || mode < 0) return rc;
    if (!on_handle_device(h)) return SD_ATTN_ERR_INVALID_VALUE;
    const Problem p = make_problem(h, q, k, v, out, B, H, Nq, Nk, d, scale, dtype, (cudaStream_t)stream);
    rc = launch_one(h, p, mode, dtype);
    if (rc == SD_ATTN_OK) h->last_mode = mode;
    if (rc == SD_ATTN_OK && getenv("SD_ATTN_LOG"))
        fprintf(stderr, "[sd_attn] forward BH=%d Nq=%d Nk=%d d=%d dtype=%d -> mode %d\n", B * H, Nq, Nk, d, dtype, mode);
    return rc;
}

// A rough cost of one launch in microseconds, only to balance the lanes of a batch: a floor for the fixed part of
// a launch, tensor time at the rate the single-pass kernel reaches, memory time at the rate the cross kernel reaches.
static double group_cost_us(const Problem& p, int n, int dtype) {
    const double bh = (double)p.BH * n, es = dtype == SD_ATTN_F32 ? 4.0 : 2.0;
    const double flops = 4.0 * bh * p.Nq * (double)p.Nk * p.d;
    const double bytes = es * bh * p.d * (2.0 * p.Nq + 2.0 * p.Nk);
    const double t = flops / 450e6, m = bytes / 2.5e6;
    const double c = t > m ? t : m;
    return c > 8.0 ? c : 8.0;
}

constexpr int BATCH_MAX_GROUP = F4_GROUP_MAX > X2_GROUP_MAX ? F4_GROUP_MAX : X2_GROUP_MAX;

extern "C" int sd_attn_forward_batch(sd_attn_handle* h, const sd_attn_problem* problems, int count, int dtype,
                                     void* stream) {
    if (!h || count < 0 || (count > 0 && !problems)) return SD_ATTN_ERR_INVALID_VALUE;
    if (count == 0) return SD_ATTN_OK;
    cudaStream_t s = (cudaStream_t)stream;
    // every problem is checked before anything is enqueued
    int* modes = (int*)malloc(sizeof(int) * (size_t)count * 2);
    if (!modes) return SD_ATTN_ERR_INVALID_VALUE;
    int* taken = modes + count;
    for (int i = 0; i < count; ++i) {
        const sd_attn_problem& p = problems[i];
        const int rc = validate_problem(h, p.q, p.k, p.v, p.out, p.B, p.H, p.Nq, p.Nk, p.d, p.scale, dtype, &modes[i]);
        if (rc != SD_ATTN_OK) {
            free(modes);
            return rc;
        }
        taken[i] = modes[i] < 0;   // an empty problem: nothing to launch
    }
    if (!on_handle_device(h)) {
        free(modes);
        return SD_ATTN_ERR_INVALID_VALUE;
    }
    // TWOPASS lends ONE workspace to every call and the CUDA-core kernel gains nothing from company: one after another
    bool serial = !h->batch_lanes_ok || count == 1;
    for (int i = 0; i < count; ++i)
        if (modes[i] == SD_ATTN_MODE_TWOPASS || modes[i] == SD_ATTN_MODE_SIMT) serial = true;
    int rc = SD_ATTN_OK;
    if (serial) {
        for (int i = 0; i < count && rc == SD_ATTN_OK; ++i) {
            if (taken[i]) continue;
            const sd_attn_problem& p = problems[i];
            rc = launch_one(h, make_problem(h, p.q, p.k, p.v, p.out, p.B, p.H, p.Nq, p.Nk, p.d, p.scale, dtype, s), modes[i], dtype);
            if (rc == SD_ATTN_OK) h->last_mode = modes[i];
        }
        free(modes);
        return rc;
    }
    // Fork the lanes from the caller's stream; problems of one shape and kernel become one launch; every launch goes
    // to the lane with the least work so far (FUSED launches that deal their steps out in shares use the handle's
    // one scratch and therefore all stay on the caller's stream); join the lanes back: for the caller one piece of
    // stream-ordered work, capturable in a graph.
    cudaError_t e = cudaEventRecord(h->ev_batch_fork, s);
    for (int l = 0; l < BATCH_LANES && e == cudaSuccess; ++l) e = cudaStreamWaitEvent(h->batch_lane[l], h->ev_batch_fork, 0);
    if (e != cudaSuccess) {
        free(modes);
        return cuda_fail(h, e);
    }
    // pass 1: the groups (members of group g: member[first[g]] .. member[first[g + 1] - 1]) and the one with the most work
    int* member = (int*)malloc(sizeof(int) * ((size_t)count * 2 + 1));
    if (!member) {
        free(modes);
        return SD_ATTN_ERR_INVALID_VALUE;   // (nothing was enqueued but the fork, which the join below would need: give up early)
    }
    int* first = member + count;
    int n_groups = 0, n_members = 0, biggest = -1;
    double biggest_cost = 0.0;
    for (int i = 0; i < count; ++i) {
        if (taken[i]) continue;
        const sd_attn_problem& p0 = problems[i];
        const bool x2 = modes[i] == SD_ATTN_MODE_CROSS && cross2_supports(p0.Nk, p0.d) && !h->opt.cross_one_tile;
        int cap = x2 ? X2_GROUP_MAX : 1;
        if (modes[i] == SD_ATTN_MODE_FUSED)
            cap = plan_fused(h, make_problem(h, p0.q, p0.k, p0.v, p0.out, p0.B, p0.H, p0.Nq, p0.Nk, p0.d, p0.scale, dtype, s)).max_group;
        first[n_groups] = n_members;
        int n = 0;
        for (int j = i; j < count && n < cap; ++j) {
            const sd_attn_problem& p = problems[j];
            if (taken[j] || modes[j] != modes[i] || p.B != p0.B || p.H != p0.H || p.Nq != p0.Nq || p.Nk != p0.Nk || p.d != p0.d)
                continue;
            member[n_members++] = j;
            taken[j] = 1;
            ++n;
        }
        const double cost = group_cost_us(make_problem(h, p0.q, p0.k, p0.v, p0.out, p0.B, p0.H, p0.Nq, p0.Nk, p0.d, p0.scale, dtype, s), n, dtype);
        if (cost > biggest_cost) {
            biggest_cost = cost;
            biggest = n_groups;
        }
        ++n_groups;
    }
    first[n_groups] = n_members;
    // pass 2: the biggest group first, on the high-priority lane (unless it deals key ranges out: those launches share
    // the handle's one scratch and stay on the caller's stream); every other launch to the lane with the least work so
    // far among the caller's stream and the other lanes
    double load[BATCH_LANES + 1] = {0};
    for (int k = 0; k < n_groups && rc == SD_ATTN_OK; ++k) {
        const int g = k == 0 ? biggest : (k <= biggest ? k - 1 : k);
        const int i = member[first[g]], n = first[g + 1] - first[g];
        const sd_attn_problem& p0 = problems[i];
        const bool x2 = modes[i] == SD_ATTN_MODE_CROSS && cross2_supports(p0.Nk, p0.d) && !h->opt.cross_one_tile;
        Problem group[BATCH_MAX_GROUP];
        for (int m = 0; m < n; ++m) {
            const sd_attn_problem& p = problems[member[first[g] + m]];
            group[m] = make_problem(h, p.q, p.k, p.v, p.out, p.B, p.H, p.Nq, p.Nk, p.d, p.scale, dtype, s);
        }
        const bool shares = modes[i] == SD_ATTN_MODE_FUSED && plan_fused(h, group[0]).shares;
        int lane = 0;   // 0: the caller's stream; l >= 1: batch_lane[l - 1]
        if (!shares) {
            if (k == 0 && n_groups > 1) lane = 1;
            else
                for (int l = 2; l <= BATCH_LANES; ++l)
                    if (load[l] < load[lane]) lane = l;
        }
        load[lane] += group_cost_us(group[0], n, dtype);
        cudaStream_t target = lane == 0 ? s : h->batch_lane[lane - 1];
        for (int m = 0; m < n; ++m) group[m].stream = target;
        if (modes[i] == SD_ATTN_MODE_FUSED) rc = launch_fused_group(h, group, n);
        else if (x2) rc = launch_cross2_group(h, group, n);
        else rc = launch_one(h, group[0], modes[i], dtype);
        if (rc == SD_ATTN_OK) h->last_mode = modes[i];
    }
    free(member);
    free(modes);
    // join in every case: the caller's stream must not run ahead of work that was enqueued
    for (int l = 0; l < BATCH_LANES; ++l) {
        cudaError_t ej = cudaEventRecord(h->ev_batch_join[l], h->batch_lane[l]);
        if (ej == cudaSuccess) ej = cudaStreamWaitEvent(s, h->ev_batch_join[l], 0);
        if (ej != cudaSuccess && e == cudaSuccess) e = ej;
    }
    if (rc != SD_ATTN_OK) return rc;
    return e == cudaSuccess ? SD_ATTN_OK : cuda_fail(h, e);
}

static size_t round256(size_t x) { return (x + 255) & ~(size_t)255; }

extern "C" size_t sd_attn_host_staging_bytes(int B, int H, int Nq, int Nk, int d, int dtype) {
    if (B <= 0 || H <= 0 || Nq < 0 || Nk <= 0 || d <= 0) return 0;
    const size_t es = dtype == SD_ATTN_F32 ? 4 : 2;
    const size_t qb = round256((size_t)B * H * Nq * d * es), kb = round256((size_t)B * H * Nk * d * es);
    return 2 * qb + 2 * kb;
}

extern "C" int sd_attn_forward_host(sd_attn_handle* h, const void* q, const void* k, const void* v, void* out,
                                    void* staging, size_t staging_bytes, int B, int H, int Nq, int Nk, int d,
                                    float scale, int dtype, void* stream) {
    if (!h) return SD_ATTN_ERR_INVALID_VALUE;
    if (B <= 0 || H <= 0 || Nq < 0 || Nk <= 0 || d <= 0) return SD_ATTN_ERR_INVALID_VALUE;
    if (dtype != SD_ATTN_F16 && dtype != SD_ATTN_F32 && dtype != SD_ATTN_BF16) return SD_ATTN_ERR_UNSUPPORTED;
    if (Nq == 0) return SD_ATTN_OK;
    if (!q || !k || !v || !out) return SD_ATTN_ERR_INVALID_VALUE;
    if (!on_handle_device(h)) return SD_ATTN_ERR_INVALID_VALUE;
    const size_t need = sd_attn_host_staging_bytes(B, H, Nq, Nk, d, dtype);
    if (!staging || staging_bytes < need || ((uintptr_t)staging & 255u)) return SD_ATTN_ERR_WORKSPACE;
    const size_t es = dtype == SD_ATTN_F32 ? 4 : 2;
    const size_t q_bytes = (size_t)B * H * Nq * d * es, k_bytes = (size_t)B * H * Nk * d * es;
    char* dq = (char*)staging;
    char* dk = dq + round256(q_bytes);
    char* dv = dk + round256(k_bytes);
    char* dout = dv + round256(k_bytes);
    cudaStream_t s = (cudaStream_t)stream;
    // Slices of the (batch, head) range are independent problems.  With more than one, the copies run on two streams
    // of the handle -- host to device of slice c + 1 and device to host of slice c - 1 while the kernel of slice c
    // runs on the caller's stream -- forked from and joined back into the caller's stream by events, so that for the
    // caller the call is still one piece of stream-ordered work.  (Not in TWOPASS mode: its workspace and the
    // pointers sd_attn_twopass_buffers returns describe one whole call.)
    const int BH = B * H;
    const size_t q_head = (size_t)Nq * d * es, k_head = (size_t)Nk * d * es;
    const bool sliceable = h->host_overlap && h->mode != SD_ATTN_MODE_TWOPASS && h->layout == SD_ATTN_LAYOUT_BHND &&
                           q_head % 16 == 0 && k_head % 16 == 0;   // every slice starts 16-byte aligned
    const int slices = sliceable ? (BH < HOST_SLICES ? BH : HOST_SLICES) : 1;
    if (slices > 1) {
        cudaError_t e = cudaEventRecord(h->ev_fork, s);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(h->copy_in, h->ev_fork, 0);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(h->copy_out, h->ev_fork, 0);
        if (e != cudaSuccess) return cuda_fail(h, e);
        int rc = SD_ATTN_OK;
        // Every copy costs the copy engine about 8 us on top of its bytes (measured: twelve copies of 1.3 MB run at
        // 40 GB/s, one of 15.7 MB at 54), so K and V go over whole, one copy each, and only Q and the output are cut.
        e = cudaMemcpyAsync(dk, k, k_bytes, cudaMemcpyHostToDevice, h->copy_in);
        if (e == cudaSuccess) e = cudaMemcpyAsync(dv, v, k_bytes, cudaMemcpyHostToDevice, h->copy_in);
        for (int c = 0; c < slices && e == cudaSuccess && rc == SD_ATTN_OK; ++c) {
            const int h0 = (int)((long long)BH * c / slices), h1 = (int)((long long)BH * (c + 1) / slices);
            const size_t qo = q_head * h0, ko = k_head * h0, qn = q_head * (h1 - h0);
            e = cudaMemcpyAsync(dq + qo, (const char*)q + qo, qn, cudaMemcpyHostToDevice, h->copy_in);
            if (e == cudaSuccess) e = cudaEventRecord(h->ev_in[c], h->copy_in);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(s, h->ev_in[c], 0);
            if (e != cudaSuccess) break;
            rc = sd_attn_forward(h, dq + qo, dk + ko, dv + ko, dout + qo, 1, h1 - h0, Nq, Nk, d, scale, dtype, stream);
            if (rc != SD_ATTN_OK) break;
            e = cudaEventRecord(h->ev_done[c], s);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(h->copy_out, h->ev_done[c], 0);
            if (e == cudaSuccess) e = cudaMemcpyAsync((char*)out + qo, dout + qo, qn, cudaMemcpyDeviceToHost, h->copy_out);
        }
        // join in every case: the caller's stream must not run ahead of copies that were enqueued
        cudaError_t ej = cudaEventRecord(h->ev_join, h->copy_out);
        if (ej == cudaSuccess) ej = cudaStreamWaitEvent(s, h->ev_join, 0);
        if (ej == cudaSuccess) ej = cudaEventRecord(h->ev_join, h->copy_in);
        if (ej == cudaSuccess) ej = cudaStreamWaitEvent(s, h->ev_join, 0);
        if (rc != SD_ATTN_OK) return rc;
        if (e != cudaSuccess || ej != cudaSuccess) return cuda_fail(h, e != cudaSuccess ? e : ej);
        return SD_ATTN_OK;
    }
    cudaError_t e = cudaMemcpyAsync(dq, q, q_bytes, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(dk, k, k_bytes, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(dv, v, k_bytes, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return cuda_fail(h, e);
    const int rc = sd_attn_forward(h, dq, dk, dv, dout, B, H, Nq, Nk, d, scale, dtype, stream);
    if (rc != SD_ATTN_OK) return rc;
    e = cudaMemcpyAsync(out, dout, q_bytes, cudaMemcpyDeviceToHost, s);
    return e == cudaSuccess ? SD_ATTN_OK : cuda_fail(h, e);
}

// ------------------------------------------------------------------------------------------------
// Two-pass attention for callers that cannot allocate device memory.
//
// Some hosts of this library run where cudaMalloc is off limits: inside a framework that owns the whole
// device heap and forbids side allocations, in a process whose memory was carved up front, or on a
// latency path where an allocation (an implicit device synchronisation) is not acceptable.  Such a
// caller cannot create a handle either (sd_attn_create allocates the status block), nor lend a
// workspace it does not have.  For them the scratch of the two-pass path -- the score matrix A and
// the [L, S] row statistics -- lives in a fixed array inside the library image.
//
// The array is part of every GPU's copy of the module from the moment the library is loaded until the
// process exits, whether or not this entry point is ever called; hence the modest size.
constexpr size_t SD_ATTN_STATIC_SCRATCH_BYTES = SD_ATTN_STATIC_MAX_SCRATCH;
static __device__ __align__(256) unsigned char g_static_scratch[SD_ATTN_STATIC_SCRATCH_BYTES];
static __device__ __align__(256) int g_static_status[DEV_STATUS_INTS];

// In host code the names above are only host-side handles of the device symbols, not device addresses:
// the real addresses are looked up once per device (with that device current) and kept here.
constexpr int STATIC_MAX_DEVICES = 64;
struct StaticDeviceState {
    int ready;
    unsigned char* scratch;
    int* status;
    encode_tiled_fn encode_tiled;
};
static StaticDeviceState g_static_state[STATIC_MAX_DEVICES];
static std::mutex g_static_mutex;   // two host threads may make their first call on a device together

static int static_setup(int dev, StaticDeviceState** out) {
    if (dev < 0 || dev >= STATIC_MAX_DEVICES) return SD_ATTN_ERR_UNSUPPORTED;
    StaticDeviceState* st = &g_static_state[dev];
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!st->ready) {
        int major = 0;
        cudaError_t e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (e != cudaSuccess) return cuda_fail(nullptr, e);
        if (major != 10) return SD_ATTN_ERR_ARCH;
        void* scratch = nullptr;
        void* status = nullptr;
        e = cudaGetSymbolAddress(&scratch, g_static_scratch);
        if (e == cudaSuccess) e = cudaGetSymbolAddress(&status, g_static_status);
        if (e != cudaSuccess || !scratch || !status) return cuda_fail(nullptr, e != cudaSuccess ? e : cudaErrorUnknown);
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn)
            return cuda_fail(nullptr, e != cudaSuccess ? e : cudaErrorUnknown);
        e = raise_smem_limit(twopass_scores_kernel, twopass_scores_smem_bytes(3));
        if (e == cudaSuccess) e = raise_smem_limit(twopass_pv_kernel, twopass_pv_smem_bytes(3));
        // the status word must start at zero (a kernel only ever writes it when a wait expires)
        if (e == cudaSuccess) e = cudaMemset(status, 0, sizeof(int) * DEV_STATUS_INTS);
        if (e != cudaSuccess) return cuda_fail(nullptr, e);
        st->scratch = (unsigned char*)scratch;
        st->status = (int*)status;
        st->encode_tiled = (encode_tiled_fn)fn;
        st->ready = 1;
    }
    *out = st;
    return SD_ATTN_OK;
}

static int static_tmap(encode_tiled_fn enc, CUtensorMap* map, const void* base, int BH, int N, int d, int box_rows) {
    return encode_tmap(enc, map, base, 0, BH, N, d, box_rows) == CUDA_SUCCESS ? SD_ATTN_OK : SD_ATTN_ERR_CUDA;
}

extern "C" int sd_attn_forward_twopass_static(const void* q, const void* k, const void* v, void* out, int B, int H,
                                              int Nq, int Nk, int d, float scale, int dtype, void* stream) {
    if (B <= 0 || H <= 0 || Nq < 0 || Nk <= 0 || d <= 0) return SD_ATTN_ERR_INVALID_VALUE;
    if (!isfinite(scale)) return SD_ATTN_ERR_INVALID_VALUE;
    if (dtype != SD_ATTN_F16 || d > SD_ATTN_MAX_D || d % 8 != 0) return SD_ATTN_ERR_UNSUPPORTED;
    if ((long long)B * H > 65535) return SD_ATTN_ERR_UNSUPPORTED;
    if (Nq == 0) return SD_ATTN_OK;
    if (!q || !k || !v || !out) return SD_ATTN_ERR_INVALID_VALUE;
    if ((((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out) & 15u) != 0) return SD_ATTN_ERR_ALIGNMENT;
    const size_t need = sd_attn_workspace_bytes(SD_ATTN_MODE_TWOPASS, B, H, Nq, Nk, d, dtype);
    if (need > SD_ATTN_STATIC_SCRATCH_BYTES) {
        if (getenv("SD_ATTN_LOG"))
            fprintf(stderr, "[sd_attn] static two-pass scratch: call needs %zu bytes, the built-in array holds %zu\n", need,
                    (size_t)SD_ATTN_STATIC_SCRATCH_BYTES);
        return SD_ATTN_ERR_WORKSPACE;
    }
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(nullptr, e);
    StaticDeviceState* st = nullptr;
    int rc = static_setup(dev, &st);
    if (rc != SD_ATTN_OK) return rc;

    const int BH = B * H;
    const size_t rows = (size_t)BH * Nq;
    float* scores = (float*)st->scratch;
    float* stats = (float*)(st->scratch + ((rows * (size_t)Nk * sizeof(float) + 255) & ~(size_t)255));
    cudaStream_t s = (cudaStream_t)stream;
    TwoPassArgs a;
    twopass_fill_args(&a, scores, stats, (__half*)out, Nq, Nk, d, scale, st->status);
    CUtensorMap tq, tk, tv;
    rc = static_tmap(st->encode_tiled, &tq, q, BH, Nq, d, TILE_M);
    if (rc == SD_ATTN_OK) rc = static_tmap(st->encode_tiled, &tk, k, BH, Nk, d, TWOPASS_BN);
    if (rc == SD_ATTN_OK) rc = static_tmap(st->encode_tiled, &tv, v, BH, Nk, d, TWOPASS_BN);
    if (rc != SD_ATTN_OK) return rc;
    dim3 grid((Nq + TILE_M - 1) / TILE_M, BH);
    twopass_scores_kernel<<<grid, TWOPASS_THREADS, twopass_scores_smem_bytes(a.nch), s>>>(tq, tk, a);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(nullptr, e);
    twopass_pv_kernel<<<grid, TWOPASS_THREADS, twopass_pv_smem_bytes(a.nch), s>>>(tv, a);
    e = cudaGetLastError();
    return e == cudaSuccess ? SD_ATTN_OK : cuda_fail(nullptr, e);
}

extern "C" int sd_attn_static_query_status(void* stream, int* detail) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(nullptr, e);
    StaticDeviceState* st = nullptr;
    const int rc = static_setup(dev, &st);
    if (rc != SD_ATTN_OK) return rc;
    int host[DEV_STATUS_INTS];
    e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaMemcpy(host, st->status, sizeof(host), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(nullptr, e);
    if (detail) memcpy(detail, host, 4 * sizeof(int));
    if (host[0] != 0) {
        e = cudaMemset(st->status, 0, sizeof(host));
        if (e != cudaSuccess) return cuda_fail(nullptr, e);
        return SD_ATTN_ERR_DEVICE_TIMEOUT;
    }
    return SD_ATTN_OK;
}

// ------------------------------------------------------------------------------------------------
// Fused GEGLU (Sec. 3.1, Eq. 2): stateless, one kernel.
extern "C" int sd_geglu_forward(const void* x, void* out, long long rows, int C, int dtype, void* stream) {
    if (rows < 0 || C <= 0) return SD_ATTN_ERR_INVALID_VALUE;
    if (dtype != SD_ATTN_F16 && dtype != SD_ATTN_F32) return SD_ATTN_ERR_UNSUPPORTED;
    if (rows == 0) return SD_ATTN_OK;
    if (!x || !out) return SD_ATTN_ERR_INVALID_VALUE;
    if (rows > (1ll << 40) / C) return SD_ATTN_ERR_INVALID_VALUE;
    if (((uintptr_t)x & 15u) || ((uintptr_t)out & 15u)) return SD_ATTN_ERR_ALIGNMENT;
    int dev = 0, major = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return cuda_fail(nullptr, e);
    if (major != 10) return SD_ATTN_ERR_ARCH;
    cudaStream_t s = (cudaStream_t)stream;
    const long long elems = rows * C;
    const int vec = dtype == SD_ATTN_F16 ? 8 : 4;
    // a small multiple of the SM count walks the tensor with a stride; fewer blocks for a small tensor
    auto blocks_for = [&](long long work_items) {
        long long b = (work_items + GEGLU_THREADS - 1) / GEGLU_THREADS;
        const long long cap = (long long)sms * GEGLU_BLOCKS_PER_SM;
        return (unsigned)(b < cap ? b : cap);
    };
    if (C % vec == 0) {
        const long long pieces = elems / vec;
        const unsigned blocks = blocks_for((pieces + GEGLU_UNROLL - 1) / GEGLU_UNROLL);
        if (dtype == SD_ATTN_F16)
            geglu_vector_kernel<__half, 8><<<blocks, GEGLU_THREADS, 0, s>>>((const __half*)x, (__half*)out, pieces, C / 8);
        else
            geglu_vector_kernel<float, 4><<<blocks, GEGLU_THREADS, 0, s>>>((const float*)x, (float*)out, pieces, C / 4);
    } else {
        const unsigned blocks = blocks_for(elems);
        if (dtype == SD_ATTN_F16)
            geglu_scalar_kernel<__half><<<blocks, GEGLU_THREADS, 0, s>>>((const __half*)x, (__half*)out, elems, C);
        else
            geglu_scalar_kernel<float><<<blocks, GEGLU_THREADS, 0, s>>>((const float*)x, (float*)out, elems, C);
    }
    e = cudaGetLastError();
    return e == cudaSuccess ? SD_ATTN_OK : cuda_fail(nullptr, e);
}

// ------------------------------------------------------------------------------------------------
// Fused group normalisation (Sec. 3.1, Eq. 1): stateless, one kernel, one thread block per (sample, group).
static std::mutex g_gn_mutex;
static int g_gn_limits_raised[STATIC_MAX_DEVICES];

extern "C" int sd_groupnorm_forward(const void* x, const void* gamma, const void* beta, void* y, int N, int C,
                                    long long HW, int G, float eps, int dtype, void* stream) {
    if (N < 0 || C <= 0 || HW <= 0 || G <= 0 || C % G != 0) return SD_ATTN_ERR_INVALID_VALUE;
    if (!(eps >= 0.f) || !isfinite(eps)) return SD_ATTN_ERR_INVALID_VALUE;
    if (dtype != SD_ATTN_F16 && dtype != SD_ATTN_F32) return SD_ATTN_ERR_UNSUPPORTED;
    if (N == 0) return SD_ATTN_OK;
    if (!x || !y) return SD_ATTN_ERR_INVALID_VALUE;
    if ((long long)N * G > 2147483647ll) return SD_ATTN_ERR_INVALID_VALUE;
    const size_t es = dtype == SD_ATTN_F16 ? 2 : 4;
    if (((uintptr_t)x & 15u) || ((uintptr_t)y & 15u) || ((uintptr_t)gamma & (es - 1)) || ((uintptr_t)beta & (es - 1)))
        return SD_ATTN_ERR_ALIGNMENT;
    int dev = 0, major = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return cuda_fail(nullptr, e);
    if (major != 10) return SD_ATTN_ERR_ARCH;
    if (dev < 0 || dev >= STATIC_MAX_DEVICES) return SD_ATTN_ERR_UNSUPPORTED;
    {
        std::lock_guard<std::mutex> lock(g_gn_mutex);
        if (!g_gn_limits_raised[dev]) {
            e = raise_smem_limit(groupnorm_staged_kernel<__half, 8>, GN_MAX_STAGED_BYTES);
            if (e == cudaSuccess) e = raise_smem_limit(groupnorm_staged_kernel<float, 4>, GN_MAX_STAGED_BYTES);
            if (e != cudaSuccess) return cuda_fail(nullptr, e);
            g_gn_limits_raised[dev] = 1;
        }
    }
    GroupNormArgs a;
    a.x = x; a.gamma = gamma; a.beta = beta; a.y = y;
    a.C = C; a.G = G; a.HW = HW; a.eps = eps;
    cudaStream_t s = (cudaStream_t)stream;
    const long long group_elems = (long long)(C / G) * HW;
    const long long group_bytes = group_elems * (long long)es;
    const int vec = (int)(16 / es);
    const unsigned blocks = (unsigned)((long long)N * G);
    // staged: the group fits shared memory and neither a channel nor the group ends inside a 16-byte piece
    const bool staged = group_bytes <= GN_MAX_STAGED_BYTES && HW % vec == 0;
    if (staged && dtype == SD_ATTN_F16) {
        groupnorm_staged_kernel<__half, 8><<<blocks, GN_THREADS, (size_t)group_bytes, s>>>(a);
    } else if (staged) {
        groupnorm_staged_kernel<float, 4><<<blocks, GN_THREADS, (size_t)group_bytes, s>>>(a);
    } else if (dtype == SD_ATTN_F16)
        groupnorm_streaming_kernel<__half><<<blocks, GN_THREADS, 0, s>>>(a);
    else
        groupnorm_streaming_kernel<float><<<blocks, GN_THREADS, 0, s>>>(a);
    e = cudaGetLastError();
    return e == cudaSuccess ? SD_ATTN_OK : cuda_fail(nullptr, e);
}

// ------------------------------------------------------------------------------------------------
// Winograd F(4x4, 3x3) convolution (Sec. 3.3): stateless; filter transform once, then input transform, 36 GEMMs on
// the tensor cores and output transform per call.
static __device__ __align__(256) int g_winograd_status[DEV_STATUS_INTS];
static std::mutex g_wg_mutex;
struct WinogradDeviceState {
    int ready;
    int* status;
    encode_tiled_fn encode_tiled;
};
static WinogradDeviceState g_wg_state[STATIC_MAX_DEVICES];

static int winograd_setup(WinogradDeviceState** out) {
    int dev = 0, major = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return cuda_fail(nullptr, e);
    if (major != 10) return SD_ATTN_ERR_ARCH;
    if (dev < 0 || dev >= STATIC_MAX_DEVICES) return SD_ATTN_ERR_UNSUPPORTED;
    WinogradDeviceState* st = &g_wg_state[dev];
    std::lock_guard<std::mutex> lock(g_wg_mutex);
    if (!st->ready) {
        void* status = nullptr;
        e = cudaGetSymbolAddress(&status, g_winograd_status);
        if (e != cudaSuccess || !status) return cuda_fail(nullptr, e != cudaSuccess ? e : cudaErrorUnknown);
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn)
            return cuda_fail(nullptr, e != cudaSuccess ? e : cudaErrorUnknown);
        e = raise_smem_limit(winograd_gemm_kernel, winograd_gemm_smem_bytes(WG_MAX_N_CHUNK, WG_MAX_STAGES));
        if (e == cudaSuccess) e = cudaMemset(status, 0, sizeof(int) * DEV_STATUS_INTS);
        if (e != cudaSuccess) return cuda_fail(nullptr, e);
        st->status = (int*)status;
        st->encode_tiled = (encode_tiled_fn)fn;
        st->ready = 1;
    }
    *out = st;
    return SD_ATTN_OK;
}

extern "C" size_t sd_winograd_filter_elems(int K, int C) {
    return (K > 0 && C > 0) ? (size_t)WG_XI * (size_t)K * (size_t)C : 0;
}

static long long winograd_tiles(int N, int H, int W) {
    return (long long)N * ((H + WG_TILE - 1) / WG_TILE) * ((W + WG_TILE - 1) / WG_TILE);
}

extern "C" size_t sd_winograd_workspace_bytes(int N, int H, int W, int C, int K) {
    if (N <= 0 || H <= 0 || W <= 0 || C <= 0 || K <= 0) return 0;
    const size_t T = (size_t)winograd_tiles(N, H, W);
    return round256((size_t)WG_XI * T * C * sizeof(__half)) + round256((size_t)WG_XI * T * K * sizeof(float));
}

extern "C" int sd_winograd_transform_filter(const void* w, void* U, int K, int C, void* stream) {
    if (!w || !U || K <= 0 || C <= 0) return SD_ATTN_ERR_INVALID_VALUE;
    if (K % 8 != 0 || C % 8 != 0) return SD_ATTN_ERR_UNSUPPORTED;
    if (((uintptr_t)w & 15u) || ((uintptr_t)U & 15u)) return SD_ATTN_ERR_ALIGNMENT;
    WinogradDeviceState* st = nullptr;
    const int rc = winograd_setup(&st);
    if (rc != SD_ATTN_OK) return rc;
    const long long n = (long long)K * C;
    winograd_filter_kernel<<<(unsigned)((n + 255) / 256), 256, 0, (cudaStream_t)stream>>>((const __half*)w, (__half*)U, K, C);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? SD_ATTN_OK : cuda_fail(nullptr, e);
}

// A [36][rows][C] fp16 scratch plane seen by the TMA as (x = C, y = rows, z = 36): tiles of 64 columns by box_rows.
static CUresult winograd_tmap(encode_tiled_fn enc, CUtensorMap* map, const void* base, long long rows, int C, int box_rows) {
    cuuint64_t dims[3] = {(cuuint64_t)C, (cuuint64_t)rows, (cuuint64_t)WG_XI};
    cuuint64_t strides[2] = {(cuuint64_t)C * 2, (cuuint64_t)rows * C * 2};
    cuuint32_t box[3] = {(cuuint32_t)CHUNK_COLS, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

extern "C" int sd_winograd_conv3x3_forward(const void* x, const void* U, const void* bias, void* y, void* workspace,
                                           size_t workspace_bytes, int N, int H, int W, int C, int K, void* stream) {
    if (N < 0 || H <= 0 || W <= 0 || C <= 0 || K <= 0) return SD_ATTN_ERR_INVALID_VALUE;
    if (C % 8 != 0 || K % 8 != 0) return SD_ATTN_ERR_UNSUPPORTED;
    if (N == 0) return SD_ATTN_OK;
    if (!x || !U || !y) return SD_ATTN_ERR_INVALID_VALUE;
    if (((uintptr_t)x & 15u) || ((uintptr_t)U & 15u) || ((uintptr_t)y & 15u) || ((uintptr_t)bias & 3u))
        return SD_ATTN_ERR_ALIGNMENT;
    const long long T = winograd_tiles(N, H, W);
    // (tile indices are ints; the transform grids are T * C / 256 and T * K / 256 blocks)
    if (T > 2147483647ll || T * (C > K ? C : K) / 256 > 2147483647ll) return SD_ATTN_ERR_UNSUPPORTED;
    const size_t need = sd_winograd_workspace_bytes(N, H, W, C, K);
    if (!workspace || workspace_bytes < need || ((uintptr_t)workspace & 255u)) return SD_ATTN_ERR_WORKSPACE;
    WinogradDeviceState* st = nullptr;
    int rc = winograd_setup(&st);
    if (rc != SD_ATTN_OK) return rc;

    WinogradArgs a;
    a.N = N; a.H = H; a.W = W; a.C = C; a.K = K;
    a.tiles_y = (H + WG_TILE - 1) / WG_TILE;
    a.tiles_x = (W + WG_TILE - 1) / WG_TILE;
    a.T = (int)T;
    const int chunks = (K + WG_MAX_N_CHUNK - 1) / WG_MAX_N_CHUNK;
    a.n_chunk = ((K + chunks - 1) / chunks + 15) / 16 * 16;
    a.tmem_cols = next_pow2_cols(a.n_chunk);
    // two CTAs per SM (shared memory and the 512 columns of tensor memory allow it): one's epilogue under the other's loads
    a.stages = 3;
    a.status = st->status;
    __half* V = (__half*)workspace;
    float* M = (float*)((char*)workspace + round256((size_t)WG_XI * T * C * sizeof(__half)));
    CUtensorMap tv, tu;
    if (winograd_tmap(st->encode_tiled, &tv, V, T, C, TILE_M) != CUDA_SUCCESS ||
        winograd_tmap(st->encode_tiled, &tu, U, K, C, a.n_chunk) != CUDA_SUCCESS)
        return SD_ATTN_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    const long long in_threads = T * (C / 4), out_threads = T * (K / 2);
    // Each of the three kernels lets the next one of the stream start its set-up early and waits for its
    // predecessor to complete before it touches global memory.
    const bool overlap = true;
    cudaError_t e = launch_overlapped_if(overlap, winograd_input_kernel, dim3((unsigned)((in_threads + 127) / 128)), dim3(128), 0, s,
                                         (const __half*)x, V, a);
    if (e != cudaSuccess) return cuda_fail(nullptr, e);
    dim3 grid((unsigned)((T + TILE_M - 1) / TILE_M), (unsigned)chunks, WG_XI);
    e = launch_overlapped_if(overlap, winograd_gemm_kernel, grid, dim3(WG_THREADS), winograd_gemm_smem_bytes(a.n_chunk, a.stages), s,
                             tv, tu, M, a);
    if (e != cudaSuccess) return cuda_fail(nullptr, e);
    e = launch_overlapped_if(overlap, winograd_output_kernel, dim3((unsigned)((out_threads + 127) / 128)), dim3(128), 0, s,
                             (const float*)M, (const __half*)bias, (__half*)y, a);
    return e == cudaSuccess ? SD_ATTN_OK : cuda_fail(nullptr, e);
}

extern "C" int sd_winograd_query_status(void* stream, int* detail) {
    WinogradDeviceState* st = nullptr;
    const int rc = winograd_setup(&st);
    if (rc != SD_ATTN_OK) return rc;
    int host[DEV_STATUS_INTS];
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaMemcpy(host, st->status, sizeof(host), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(nullptr, e);
    if (detail) memcpy(detail, host, 4 * sizeof(int));
    if (host[0] != 0) {
        e = cudaMemset(st->status, 0, sizeof(host));
        if (e != cudaSuccess) return cuda_fail(nullptr, e);
        return SD_ATTN_ERR_DEVICE_TIMEOUT;
    }
    return SD_ATTN_OK;
}


// ------------------------------------------------------------------------------------------------
// Instruction-rate probes for the joint roofline (see ubench_kernel.cuh): stateless, allocate nothing.
constexpr int UBENCH_MAX_BLOCKS = 1024;
static __device__ __align__(256) long long g_ubench_out[2 * UBENCH_MAX_BLOCKS];
static __device__ float g_ubench_sink[4];

extern "C" int sd_attn_ubench(int op, int iters, void* stream, double* results_per_clk_per_sm, double* sm_mhz) {
    if (op < 0 || op >= UBENCH_OPS || iters <= 0 || iters > (1 << 20) || !results_per_clk_per_sm || !sm_mhz)
        return SD_ATTN_ERR_INVALID_VALUE;
    int dev = 0, major = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return cuda_fail(nullptr, e);
    if (major != 10) return SD_ATTN_ERR_ARCH;
    if (sms > UBENCH_MAX_BLOCKS) sms = UBENCH_MAX_BLOCKS;
    long long* out = nullptr;
    float* sink = nullptr;
    e = cudaGetSymbolAddress((void**)&out, g_ubench_out);
    if (e == cudaSuccess) e = cudaGetSymbolAddress((void**)&sink, g_ubench_sink);
    if (e != cudaSuccess) return cuda_fail(nullptr, e);
    cudaStream_t s = (cudaStream_t)stream;
    for (int rep = 0; rep < 2; ++rep) {   // the second run is the measurement (the first warms the clocks and the code)
        switch (op) {
            case UBENCH_EX2: ubench_kernel<UBENCH_EX2><<<sms, UBENCH_THREADS, 0, s>>>(iters, 0.5f, out, sink); break;
            case UBENCH_FMA: ubench_kernel<UBENCH_FMA><<<sms, UBENCH_THREADS, 0, s>>>(iters, 0.5f, out, sink); break;
            case UBENCH_FMA_X2: ubench_kernel<UBENCH_FMA_X2><<<sms, UBENCH_THREADS, 0, s>>>(iters, 0.5f, out, sink); break;
            case UBENCH_SWEEP: ubench_kernel<UBENCH_SWEEP><<<sms, UBENCH_THREADS, 0, s>>>(iters, 0.5f, out, sink); break;
            default: ubench_kernel<UBENCH_SWEEP_POLY><<<sms, UBENCH_THREADS, 0, s>>>(iters, 0.5f, out, sink); break;
        }
    }
    e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    static long long host[2 * UBENCH_MAX_BLOCKS];
    if (e == cudaSuccess) e = cudaMemcpy(host, out, sizeof(long long) * 2 * sms, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(nullptr, e);
    double clk = 0, ns = 0;
    for (int b = 0; b < sms; ++b) { clk += (double)host[2 * b]; ns += (double)host[2 * b + 1]; }
    clk /= sms; ns /= sms;
    *results_per_clk_per_sm = (double)UBENCH_THREADS * iters * ubench_results_per_trip(op) / clk;
    *sm_mhz = clk / ns * 1e3;
    return SD_ATTN_OK;
}
