// Thin inline-PTX layer for the sm_100a tensor-core kernels: mbarriers with BOUNDED waits,
// TMA tile loads, tensor-memory (TMEM) management, tcgen05 MMA issue and TMEM <-> register moves,
// plus the shared-memory matrix descriptor and instruction descriptor encoders.
//
// Every wait in this file gives up after a fixed number of polls and reports through a status
// block instead of spinning for ever; callers then drain and return normally.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace sd_attn {

// ------------------------------------------------------------------ device status block
// int[0] code (0 = fine), int[1] block index, int[2] wait site, int[3] tile index.
constexpr int DEV_STATUS_INTS = 16;
constexpr int DEV_ERR_TIMEOUT = 1;

// Poll budget of one wait.  Each failed poll past the first few sleeps ~100 ns, so the budget
// is a few hundred milliseconds: far above any legitimate wait of these microsecond kernels.
constexpr uint32_t WAIT_POLL_LIMIT = 1u << 21;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void report_timeout(int* status, int site, int tile) {
    if (atomicCAS(status, 0, DEV_ERR_TIMEOUT) == 0) {
        status[1] = static_cast<int>(blockIdx.x + gridDim.x * blockIdx.y);
        status[2] = site;
        status[3] = tile;
        __threadfence();
    }
}

// True in exactly one (converged) lane of the warp.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(pred));
    return pred != 0;
}

// Re-balance the register file between warpgroups (all four warps of a warpgroup must execute it).
template <int REGS>
__device__ __forceinline__ void setmaxnreg_inc() {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS));
}
template <int REGS>
__device__ __forceinline__ void setmaxnreg_dec() {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS));
}

// ------------------------------------------------------------------ mbarrier
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t arrivals) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(arrivals) : "memory");
}
// Retire a barrier that has no operation pending, so that its memory may be initialised again.
__device__ __forceinline__ void mbar_inval(uint32_t bar) {
    asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
// Make freshly initialised barriers visible to the async proxy (TMA, tcgen05.commit).
__device__ __forceinline__ void mbar_init_fence() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    return done != 0;
}
// Non-blocking test of a phase (try_wait may suspend the thread for a while when the phase is pending).
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    return done != 0;
}
// Bounded wait.  `abort_flag` is a shared-memory int that any role sets when it gives up; every
// waiter polls it so that one expired wait releases the whole block.  Returns false on abort.
// LIMIT is the poll budget (the kernels use the default; the library's self-test of this path a small one).
template <uint32_t LIMIT = WAIT_POLL_LIMIT>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          int* status, int site, int tile) {
    // try_wait itself suspends the thread for a hardware-chosen slice, so the first polls add no
    // sleep: a sleeping poller would see a completed phase up to a sleep period late, and that
    // delay sits on the MMA-issue round trip of the fused kernels.
    for (uint32_t i = 0; i < LIMIT; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 63) == 63) {
            if (*abort_flag) return false;
            if (i > (1u << 14)) __nanosleep(256);
        }
    }
    *abort_flag = 1;
    report_timeout(status, site, tile);
    return false;
}

// The same for a waiter that is far ahead of what it waits for (a producer with a deep ring): it sleeps between polls
// from the first failed one on, so that its polling does not take issue slots from the warps that share its
// scheduler.  The poll budget is the same number of polls, so the bound in time is longer.
__device__ __forceinline__ bool mbar_wait_lazy(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                               int* status, int site, int tile) {
    for (uint32_t i = 0; i < WAIT_POLL_LIMIT; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        __nanosleep(400);
        if ((i & 15) == 15 && *abort_flag) return false;
    }
    *abort_flag = 1;
    report_timeout(status, site, tile);
    return false;
}

// The same for a wait on the hand-over path of the fused kernels: the first polls are plain tests (no suspension by
// the hardware, so a completed phase is seen at once), then the bounded wait above takes over.
template <uint32_t SPIN = 4096>
__device__ __forceinline__ bool mbar_wait_eager(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                                int* status, int site, int tile) {
    for (uint32_t i = 0; i < SPIN; ++i)
        if (mbar_test(bar, parity)) return true;
    return mbar_wait(bar, parity, abort_flag, status, site, tile);
}

// After a block gave up: give copies that may still be in flight a bounded chance to land before
// shared memory is released.  Ignores the abort flag, reports nothing.
__device__ __forceinline__ void mbar_drain(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < (1u << 14); ++i) {
        if (mbar_try_wait(bar, parity)) return;
        __nanosleep(64);
    }
}

// 16-byte shared-memory accesses by 32-bit shared address
__device__ __forceinline__ uint4 ld_shared_v4(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint4 v) {
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// ------------------------------------------------------------------ programmatic dependent launch
// A kernel launched with the programmatic-stream-serialization attribute may start while the kernel before it
// in the stream is still running.  pdl_launch_dependents() lets the NEXT kernel start that early (it takes effect
// once every CTA of this grid has called it or exited); pdl_wait() blocks until the PREVIOUS grid has completed
// and its memory is visible.  Both are no-ops for a kernel launched the ordinary way.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ------------------------------------------------------------------ TMA (bulk tensor copies)
__device__ __forceinline__ void tma_prefetch_desc(const void* tmap) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(tmap)) : "memory");
}
// 3-D tile load global -> shared, completion counted in bytes on `bar`.  Coordinates are
// (x = innermost element, y = row, z = batch*head); x must make x*elem_size a multiple of 16.
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const void* tmap, uint32_t bar, int x, int y,
                                            int z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(tmap)), "r"(bar), "r"(x), "r"(y), "r"(z)
        : "memory");
}
// Where the heads of a tensor lie.  A (batch, head) index bh splits into batch = bh / heads and head = bh % heads;
// row r of that head starts batch * batch_stride + head * head_stride + r * ld elements into the tensor.
// Head-major [B][H][N][d] is {heads = B*H, ld = d, head_stride = N*d} (the batch index is always 0); token-major
// [B][N][H][d] -- the layout a projection to H*d channels leaves, so that the head split and merge around the
// attention cost no copy -- is {heads = H, ld = H*d, head_stride = d, batch_stride = N*H*d}.
struct HeadLayout {
    int heads;
    int ld;
    long long head_stride;
    long long batch_stride;
};
template <typename T>
__device__ __forceinline__ T* head_row(T* base, const HeadLayout& lay, int bh, int row) {
    const int batch = bh / lay.heads, head = bh - batch * lay.heads;
    return base + batch * lay.batch_stride + head * lay.head_stride + (long long)row * lay.ld;
}
// 4-D tile load global -> shared: (x = innermost element, y = row, z = head, w = batch); x as for the 3-D load.
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const void* tmap, uint32_t bar, int x, int y, int z,
                                            int w) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5, %6}], [%2];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(tmap)), "r"(bar), "r"(x), "r"(y), "r"(z), "r"(w)
        : "memory");
}
// Untiled bulk copy global -> shared, completion counted in bytes on `bar`.  Both addresses 16-byte aligned, the
// size a multiple of 16 bytes.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar)
                 : "memory");
}
// Untiled bulk copy shared -> global in the executing thread's bulk group (addresses 16-byte aligned, size a multiple
// of 16 bytes); bulk_commit closes the group, bulk_wait_read<N> waits until all but the last N groups have READ their
// shared-memory source (it may then be overwritten), bulk_wait_all until every group has completed.
__device__ __forceinline__ void bulk_store(void* dst, uint32_t src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(reinterpret_cast<uint64_t>(dst)),
                 "r"(src), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// Barrier among `threads` threads of the CTA (a multiple of 32) on hardware barrier `id` (1..15; 0 is __syncthreads).
__device__ __forceinline__ void named_barrier(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
// The same with an AND reduction of a predicate: every participant receives the conjunction.
__device__ __forceinline__ bool named_barrier_and(int id, int threads, bool pred) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %3, 0;\n\t"
        "bar.red.and.pred p, %1, %2, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "r"(id), "r"(threads), "r"((uint32_t)pred)
        : "memory");
    return r != 0;
}
// 3-D tile store shared -> global (rows/columns outside the tensor are clipped by the hardware).
__device__ __forceinline__ void tma_store_3d(const void* tmap, uint32_t src, int x, int y, int z) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(
                     reinterpret_cast<uint64_t>(tmap)),
                 "r"(src), "r"(x), "r"(y), "r"(z)
                 : "memory");
}
// 4-D tile store shared -> global, coordinates as for the 4-D load.
__device__ __forceinline__ void tma_store_4d(const void* tmap, uint32_t src, int x, int y, int z, int w) {
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];" ::"l"(
                     reinterpret_cast<uint64_t>(tmap)),
                 "r"(src), "r"(x), "r"(y), "r"(z), "r"(w)
                 : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Wait until the committed stores have finished READING shared memory (it may then be reused).
__device__ __forceinline__ void tma_store_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// Generic-proxy writes to shared memory -> visible to the async proxy (TMA store, tcgen05.mma).
__device__ __forceinline__ void fence_proxy_async_smem() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// ------------------------------------------------------------------ tensor memory
// TMEM address: bits 31..16 lane, bits 15..0 column (32-bit cells).  One warp allocates.
__device__ __forceinline__ void tmem_alloc(uint32_t smem_result, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_result),
                 "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after_sync() {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Arrive on `bar` once every tcgen05 operation this thread issued so far has completed.
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
                 : "memory");
}

// D[tmem] (+)= A[smem] * B[smem]; fp16 inputs, fp32 accumulate.  One thread issues.
__device__ __forceinline__ void mma_f16_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                           bool accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate ? 1u : 0u)
        : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]: A is a 128 x 16 fp16 slab held as 8 packed 32-bit columns.
__device__ __forceinline__ void mma_f16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                           bool accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
        "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate ? 1u : 0u)
        : "memory");
}

// 32 lanes x 32-bit, 16 consecutive columns: thread t of the warp receives lane (base lane + t).
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&r)[8]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"r"(taddr),
                 "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}

// 32 consecutive columns at once (pointer to 32 registers of a fully unrolled array).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, "
        "%23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, "
        "%24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
        "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
        "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}

// ------------------------------------------------------------------ descriptors
// Shared-memory matrix descriptor, 128-byte swizzle.  A tile is stored as rows of 128 bytes
// (64 fp16); eight rows form one 1024-byte swizzle atom, and the tile base is 1024-byte aligned.
//   bits  0..13 start address >> 4        bits 16..29 leading-dimension byte offset >> 4
//   bits 32..45 stride-dimension byte offset >> 4      bits 46..47 descriptor version (1)
//   bits 61..63 swizzle mode (2 = 128 B)
// K-major operand (rows = M or N index, the 128 bytes run along the contraction):
//   stride offset = distance between 8-row groups (1024), leading offset unused (1).
// MN-major operand (rows = contraction index, the 128 bytes run along N):
//   stride offset = distance between 8-row groups (1024), leading offset = distance between
//   successive 64-element column chunks of the tile.
__host__ __device__ constexpr uint64_t smem_desc_sw128(uint32_t byte_addr, uint32_t lbo_bytes,
                                                       uint32_t sbo_bytes) {
    return (uint64_t)((byte_addr & 0x3FFFFu) >> 4) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | (2ull << 61);
}

// Instruction descriptor for kind::f16 with fp16 (or bf16) A/B and fp32 D.
//   bits 4..5 D format (1 = f32)   bits 7..9 A format (0 = f16, 1 = bf16)   bits 10..12 B format (likewise)
//   bit 13 negate A   bit 14 negate B   bit 15 A is MN-major   bit 16 B is MN-major
//   bits 17..22 N >> 3   bits 24..28 M >> 4
__host__ __device__ constexpr uint32_t idesc_f16(int m, int n, bool a_mn_major, bool b_mn_major,
                                                 bool negate_a, bool bf16 = false) {
    return (1u << 4) | (bf16 ? ((1u << 7) | (1u << 10)) : 0u) | (negate_a ? (1u << 13) : 0u) | (a_mn_major ? (1u << 15) : 0u) |
           (b_mn_major ? (1u << 16) : 0u) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// ------------------------------------------------------------------ small math helpers
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// 2^x on the FMA pipe, for x <= ~100: the special-function unit retires only 16 exponentials per
// clock per SM, so a share of them is computed here instead.  x = n + f with n = floor(x) taken from
// the low mantissa bits of (x + 1.5*2^23) rounded down, 2^f by a degree-3 polynomial fitted to
// [0, 1) (max relative error 7.5e-5, below the fp16 rounding of the weights), and n added into
// the exponent field.  Inputs are clamped to [-127, 127] (the exponent field would wrap outside).
__device__ __forceinline__ float ex2_poly(float x) {
    x = fminf(fmaxf(x, -127.f), 127.f);
    const float t = __fadd_rd(x, 12582912.f);
    const float f = x - (t - 12582912.f);
    float p = fmaf(f, 0.07802452f, 0.22606716f);
    p = fmaf(p, f, 0.69583356f);
    p = fmaf(p, f, 0.9999252f);
    return __int_as_float(__float_as_int(p) + (__float_as_int(t) << 23));
}
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
    __half2 h = __floats2half2_rn(lo, hi);  // .x (low 16 bits) = lo
    return *reinterpret_cast<uint32_t*>(&h);
}
// Two values rounded to the storage type of the call -- binary16, or bfloat16 when BF -- low 16 bits = lo.
template <bool BF>
__device__ __forceinline__ uint32_t pack_16x2(float lo, float hi) {
    if (BF) {
        uint32_t r;
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
        return r;
    }
    return pack_half2(lo, hi);
}

}  // namespace sd_attn
