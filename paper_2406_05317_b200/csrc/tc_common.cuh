// Thin inline-PTX wrappers for the sm_100a features the tensor-core kernels use:
// mbarrier, bulk async copies (TMA engine), cp.async, tcgen05 (TMEM alloc, MMA, ld, commit).
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

namespace lococo {
namespace tc {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ----------------------------------------------------------------- mbarrier
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
// Must precede a second mbarrier.init on the same shared-memory word (a CTA that runs several work items).
__device__ __forceinline__ void mbar_inval(uint32_t bar) {
    asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bounded wait: gives up after `limit` polls, records the failure in *status (global)
// and in *failed (shared, makes later waits give up quickly), and returns false.
// The caller carries on, so the kernel always terminates and frees its TMEM.
constexpr uint32_t kWaitLimit = 1u << 22;
static __device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, int* status, volatile int* failed, int code,
                                                    uint32_t max_polls = kWaitLimit) {
    const uint32_t limit = *failed ? 64u : max_polls;
    for (uint32_t i = 0; i < limit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
    }
    *failed = 1;
    atomicCAS(status, 0, code);
    return false;
}
// The first poll is inlined and touches nothing else: the thread that issues MMAs runs a
// dependent instruction chain, so every extra instruction on this path delays the tensor pipe.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int* status, volatile int* failed, int code) {
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, status, failed, code);
}

__device__ __forceinline__ void fence_barrier_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
// Makes generic-proxy writes to shared memory visible to the async proxy (TMA, tcgen05.mma).
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// ----------------------------------------------------------------- copies
// Linear bulk copy global -> shared through the TMA engine; both addresses 16-byte aligned,
// bytes a multiple of 16; completion is signalled on the mbarrier as transaction bytes.
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
// Tiled copy global -> shared through the tensor copy engine, rank 4, one box of the tensor map at
// coordinates (x, y, z, w); x times the element size must be a multiple of 16 bytes. Elements outside
// the tensor arrive as zeros. Completion is signalled on the mbarrier as transaction bytes.
__device__ __forceinline__ void tma_load_4d(uint32_t dst_smem, const void* tensor_map, int x, int y, int z, int w, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];" ::"r"(dst_smem),
        "l"(tensor_map), "r"(x), "r"(y), "r"(z), "r"(w), "r"(bar)
        : "memory");
}
// Tiled copy shared -> global through the tensor copy engine, rank 4, one box of the tensor map at coordinates
// (x, y, z, w), all of them inside the tensor and x times the element size a multiple of 16 bytes. The copy belongs to
// the thread's current bulk group; the shared-memory source must stay untouched until the group's reads are done.
__device__ __forceinline__ void tma_store_4d(const void* tensor_map, uint32_t src_smem, int x, int y, int z, int w) {
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5}], [%1];" ::"l"(tensor_map),
                 "r"(src_smem), "r"(x), "r"(y), "r"(z), "r"(w)
                 : "memory");
}
// Closes the thread's bulk group and waits until its copies have read their shared-memory sources.
__device__ __forceinline__ void bulk_stores_read() {
    asm volatile("cp.async.bulk.commit_group;\n\tcp.async.bulk.wait_group.read 0;" ::: "memory");
}
// Makes a tensor map that was written to global memory before this kernel started (by a copy on the
// same stream) the one the copy engine uses, whatever an earlier kernel read from that address.
__device__ __forceinline__ void tensormap_acquire(const void* tensor_map) {
    asm volatile("fence.proxy.tensormap::generic.acquire.gpu [%0], 128;" ::"l"(tensor_map) : "memory");
}
// 16-byte cp.async; src_bytes = 0 writes zeros. The .ca form goes through L1, which merges the
// sixteen 16-byte pieces of a 256-byte row into full lines: measured 64-74 GB/s per SM for the
// tile-staging pattern here, against 24 GB/s for .cg (each piece its own L2 request).
__device__ __forceinline__ void cp_async16(uint32_t dst_smem, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;" ::"r"(dst_smem), "l"(src), "r"(src_bytes) : "memory");
}
// The .cg form bypasses L1: for data that another SM may have rewritten during this kernel.
__device__ __forceinline__ void cp_async16_cg(uint32_t dst_smem, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst_smem), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}

// ----------------------------------------------------------------- TMEM
// Whole warp. ncols: power of two >= 32. The base address is written to *dst_smem.
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// ----------------------------------------------------------------- descriptors
// Shared-memory matrix descriptor, no swizzle ("interleaved" canonical layout): the
// operand is stored as 8x(16-byte) core matrices, 128 contiguous bytes each.
//   K-major  : lbo = byte stride between the two 8-element K halves of one MMA,
//              sbo = byte stride between 8-row groups along M/N.
//   MN-major : sbo = byte stride between 8-element groups along M/N,
//              lbo = byte stride between 8-row groups along K.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)((lbo >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;  // descriptor version of sm_100
    return d;                // base offset 0, layout type 0 (no swizzle)
}
// Shared-memory matrix descriptor for the 128-byte swizzle (the layout the tensor copy engine writes
// for a box whose inner extent is 128 bytes): rows of 128 bytes, the 16-byte chunk index XORed with
// (row mod 8); tiles start on 1024-byte boundaries.
//   K-major  : a row holds 64 consecutive K elements; sbo = byte stride between 8-row groups (1024
//              when rows are dense), lbo is not used (one 16-byte unit); the k-th MMA of a row
//              (16 elements) starts 32*k bytes into the tile.
//   MN-major : a row holds 64 consecutive M/N elements of one K index; lbo = byte stride between
//              64-element blocks along M/N, sbo = byte stride between 8-row groups along K.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)((lbo >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;  // descriptor version of sm_100
    d |= (uint64_t)2 << 61;  // layout type: 128-byte swizzle
    return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N multiple of 16.
__device__ __forceinline__ uint32_t instr_desc_bf16(int n, bool a_mn_major, bool b_mn_major) {
    uint32_t d = 0;
    d |= 1u << 4;   // D format fp32
    d |= 1u << 7;   // A format bf16
    d |= 1u << 10;  // B format bf16
    d |= (a_mn_major ? 1u : 0u) << 15;
    d |= (b_mn_major ? 1u : 0u) << 16;
    d |= (uint32_t)(n >> 3) << 17;
    d |= (uint32_t)(128 >> 4) << 24;
    return d;
}
// D[tmem] (+)= A[smem] * B[smem]; one thread issues.
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Eight MMAs of one K loop (128 elements in steps of 16) from ONE instruction block: descriptors advance by fixed steps,
// the first MMA overwrites the accumulator when `acc_first` is 0. Keeps the issuing thread's instruction count per MMA
// below the MMA's own duration at small N.
__device__ __forceinline__ void umma_ss_k8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t astep, uint32_t bstep,
                                           uint32_t idesc, uint32_t acc_first) {
    asm volatile(
        "{\n\t.reg .pred p0, p1;\n\t.reg .b64 a, b, sa, sb;\n\t"
        "setp.ne.b32 p0, %6, 0;\n\tsetp.eq.b32 p1, 0, 0;\n\t"
        "cvt.u64.u32 sa, %4;\n\tcvt.u64.u32 sb, %5;\n\t"
        "mov.b64 a, %1;\n\tmov.b64 b, %2;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, p0;\n\t"
        "add.u64 a, a, sa;\n\tadd.u64 b, b, sb;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, p1;\n\t"
        "add.u64 a, a, sa;\n\tadd.u64 b, b, sb;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, p1;\n\t"
        "add.u64 a, a, sa;\n\tadd.u64 b, b, sb;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, p1;\n\t"
        "add.u64 a, a, sa;\n\tadd.u64 b, b, sb;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, p1;\n\t"
        "add.u64 a, a, sa;\n\tadd.u64 b, b, sb;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, p1;\n\t"
        "add.u64 a, a, sa;\n\tadd.u64 b, b, sb;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, p1;\n\t"
        "add.u64 a, a, sa;\n\tadd.u64 b, b, sb;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, p1;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(astep), "r"(bstep), "r"(acc_first)
        : "memory");
}

// The same for a K loop of four steps (64 elements).
__device__ __forceinline__ void umma_ss_k4(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t astep, uint32_t bstep,
                                           uint32_t idesc, uint32_t acc_first) {
    asm volatile(
        "{\n\t.reg .pred p0, p1;\n\t.reg .b64 a, b, sa, sb;\n\t"
        "setp.ne.b32 p0, %6, 0;\n\tsetp.eq.b32 p1, 0, 0;\n\t"
        "cvt.u64.u32 sa, %4;\n\tcvt.u64.u32 sb, %5;\n\t"
        "mov.b64 a, %1;\n\tmov.b64 b, %2;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, p0;\n\t"
        "add.u64 a, a, sa;\n\tadd.u64 b, b, sb;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, p1;\n\t"
        "add.u64 a, a, sa;\n\tadd.u64 b, b, sb;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, p1;\n\t"
        "add.u64 a, a, sa;\n\tadd.u64 b, b, sb;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, p1;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(astep), "r"(bstep), "r"(acc_first)
        : "memory");
}
// The mbarrier receives one arrival when all MMAs issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 32 lanes x 32 columns of fp32: thread l of the warp gets lane (base lane + l), columns c..c+31.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}
// The reverse: thread l writes lane (base lane + l), columns c..c+31.
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
        "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]),
        "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]), "r"(v[18]),
        "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]),
        "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

}  // namespace tc
}  // namespace lococo
