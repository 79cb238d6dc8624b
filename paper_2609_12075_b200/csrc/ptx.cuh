// Thin wrappers over the sm_100a PTX used by the tensor-core kernels: mbarriers with bounded
// waits, TMA tile loads, tcgen05 (TMEM allocation, MMA issue, commit, loads) and programmatic
// dependent launch.  Every wait is bounded: on expiry the caller records ADIT_E_TIMEOUT and unwinds.
#pragma once
#include <cuda.h>
#include <stdint.h>

namespace adit {
namespace ptx {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint64_t globaltimer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// ---- mbarrier ---------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Non-blocking test (try_wait may suspend the thread for a while when the phase is not complete).
__device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
#ifndef ADIT_WAIT_TRIES
#define ADIT_WAIT_TRIES 1
#endif
// Bounded wait: gives up after `limit_ns` (checked every 1024 polls) and returns false.  The clock read after
// the first failed test doubles as a short back-off (it takes a few hundred nanoseconds), which measurably
// helps the warps that share a scheduler with the waiting one.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, uint64_t limit_ns = 2000000000ull) {
#pragma unroll 1
  for (int i = 0; i < ADIT_WAIT_TRIES; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = globaltimer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 1024; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (globaltimer_ns() - t0 > limit_ns) return false;
  }
}

// ---- TMA --------------------------------------------------------------------------------------
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* m) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(m) : "memory");
}
// Tensor maps that a kernel wrote to global memory: the writer releases, the thread that is going to use the map
// for a copy acquires (the copy engine reads maps through a cache of its own).
__device__ __forceinline__ void tensormap_release() { asm volatile("fence.proxy.tensormap::generic.release.gpu;" ::: "memory"); }
__device__ __forceinline__ void tensormap_acquire(const CUtensorMap* m) {
  asm volatile("fence.proxy.tensormap::generic.acquire.gpu [%0], 128;" ::"l"(m) : "memory");
}
// 2-D tiled load global -> shared, completion counted in bytes on `bar`.  x = innermost (element)
// coordinate, which must be a multiple of 16 bytes worth of elements; y = row.
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          smem_u32(smem_dst)),
      "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(void* smem_dst, const CUtensorMap* map, int x, int y, int z, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(
          smem_u32(smem_dst)),
      "l"(map), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void tma_load_2d_hint(void* smem_dst, const CUtensorMap* map, int x, int y, uint64_t* bar,
                                                 uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, "
      "%3}], [%4], %5;" ::"r"(smem_u32(smem_dst)),
      "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}

// ---- tcgen05 / tensor memory ------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_result, uint32_t ncols) {  // whole warp
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)),
               "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {  // whole warp
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {  // whole warp
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem desc] * B[smem desc]^T, bf16/f16 inputs, one thread issues.
__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                         uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The same with the A operand in tensor memory: lane = row, each 32-bit column holds two consecutive k elements
// (bf16, the lower k in the low half); a product of 16 k elements reads 8 columns starting at a_tmem.
__device__ __forceinline__ void umma_f16_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The mbarrier receives one arrival once all tcgen05 operations issued so far by this thread are done.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
// 32 lanes x 32 consecutive fp32 columns: thread i of the warp gets lane (base lane + i).
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
// Store 32 lanes x 32 consecutive fp32 columns from registers (thread i writes lane base + i).
__device__ __forceinline__ void tmem_st_32x32(uint32_t taddr, const float* v) {
  const uint32_t* r = reinterpret_cast<const uint32_t*>(v);
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
      "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
      "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
// Store 32 lanes x 16 consecutive 32-bit columns from registers.
__device__ __forceinline__ void tmem_st_32x16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major bf16 tile whose rows are 128 bytes (64 elements)
// stored with the 128-byte swizzle TMA produces: 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);  // start address
  d |= (uint64_t)1 << 16;                       // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;             // stride byte offset: 8 rows x 128 B
  d |= (uint64_t)1 << 46;                       // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                       // 128-byte swizzle
  return d;
}
// Descriptor of an MN-major bf16 operand (the N index is contiguous in memory), 128-byte swizzle: the tile is
// a row of boxes, each 64 N-elements (128 bytes) wide and as many K rows as the k-block has; `box_bytes` is the
// distance between boxes, 8-row K groups are 1024 bytes apart.  (Checked against a plain product on B200.)
__device__ __forceinline__ uint64_t smem_desc_mn_sw128(uint32_t smem_addr, uint32_t box_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);
  d |= (uint64_t)((box_bytes >> 4) & 0x3FFF) << 16;  // leading byte offset: next box along N
  d |= (uint64_t)(1024 >> 4) << 32;                  // stride byte offset: next 8 rows along K
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M x N tile.
__device__ __forceinline__ uint32_t idesc_bf16_f32(int m, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// ---- one k-block (64 deep = four products of 16) issued as a single instruction sequence ------------------------
// The issuing thread has nothing to hide its own instruction latencies behind, and a product should leave it every
// 60-130 cycles: descriptors are therefore kept as 32-bit halves (only the low half, which holds the address, changes
// from product to product: + 2 per 32 bytes along k) and the four products of a k-block are one asm block.
// `lo` halves: see smem_desc_lo; `hi`: smem_desc_hi_sw128 (the same for every K-major 128-byte-swizzled operand).
__device__ __forceinline__ uint32_t smem_desc_lo(uint32_t smem_addr) { return ((smem_addr & 0x3FFFF) >> 4) | (1u << 16); }
__device__ __forceinline__ uint32_t smem_desc_hi_sw128() { return (uint32_t)(1024 >> 4) | (1u << 14) | (2u << 29); }
#define ADIT_UMMA_KBLOCK(NAME, GROUP)                                                                              \
  __device__ __forceinline__ void NAME(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc, \
                                       uint32_t acc_first) {                                                       \
    asm volatile(                                                                                                  \
        "{\n\t.reg .pred p, q;\n\t.reg .b64 a, b;\n\t.reg .b32 al, bl;\n\t"                                        \
        "setp.ne.b32 p, %5, 0;\n\t"                                                                                \
        "setp.eq.b32 q, 0, 0;\n\t"                                                                                 \
        "mov.b64 a, {%1, %3};\n\tmov.b64 b, {%2, %3};\n\t"                                                         \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%0], a, b, %4, p;\n\t"                                        \
        "add.u32 al, %1, 2;\n\tadd.u32 bl, %2, 2;\n\tmov.b64 a, {al, %3};\n\tmov.b64 b, {bl, %3};\n\t"             \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%0], a, b, %4, q;\n\t"                                        \
        "add.u32 al, %1, 4;\n\tadd.u32 bl, %2, 4;\n\tmov.b64 a, {al, %3};\n\tmov.b64 b, {bl, %3};\n\t"             \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%0], a, b, %4, q;\n\t"                                        \
        "add.u32 al, %1, 6;\n\tadd.u32 bl, %2, 6;\n\tmov.b64 a, {al, %3};\n\tmov.b64 b, {bl, %3};\n\t"             \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%0], a, b, %4, q;\n\t}" ::"r"(d_tmem),                        \
        "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(acc_first)                                                  \
        : "memory");                                                                                               \
  }
ADIT_UMMA_KBLOCK(umma_kblock_f16, "1")
ADIT_UMMA_KBLOCK(umma_kblock_f16_pair, "2")
#undef ADIT_UMMA_KBLOCK
// The same for a gate/up pair: two accumulators (d_tmem, d_tmem2), two weight operands, one token operand.
#define ADIT_UMMA_KBLOCK2(NAME, GROUP)                                                                             \
  __device__ __forceinline__ void NAME(uint32_t d_tmem, uint32_t d_tmem2, uint32_t a_lo, uint32_t a2_lo,           \
                                       uint32_t b_lo, uint32_t hi, uint32_t idesc, uint32_t acc_first) {           \
    asm volatile(                                                                                                  \
        "{\n\t.reg .pred p, q;\n\t.reg .b64 a, a2, b;\n\t.reg .b32 al, a2l, bl;\n\t"                               \
        "setp.ne.b32 p, %7, 0;\n\t"                                                                                \
        "setp.eq.b32 q, 0, 0;\n\t"                                                                                 \
        "mov.b64 a, {%2, %5};\n\tmov.b64 a2, {%3, %5};\n\tmov.b64 b, {%4, %5};\n\t"                                \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%0], a, b, %6, p;\n\t"                                        \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%1], a2, b, %6, p;\n\t"                                       \
        "add.u32 al, %2, 2;\n\tadd.u32 a2l, %3, 2;\n\tadd.u32 bl, %4, 2;\n\t"                                      \
        "mov.b64 a, {al, %5};\n\tmov.b64 a2, {a2l, %5};\n\tmov.b64 b, {bl, %5};\n\t"                               \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%0], a, b, %6, q;\n\t"                                        \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%1], a2, b, %6, q;\n\t"                                       \
        "add.u32 al, %2, 4;\n\tadd.u32 a2l, %3, 4;\n\tadd.u32 bl, %4, 4;\n\t"                                      \
        "mov.b64 a, {al, %5};\n\tmov.b64 a2, {a2l, %5};\n\tmov.b64 b, {bl, %5};\n\t"                               \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%0], a, b, %6, q;\n\t"                                        \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%1], a2, b, %6, q;\n\t"                                       \
        "add.u32 al, %2, 6;\n\tadd.u32 a2l, %3, 6;\n\tadd.u32 bl, %4, 6;\n\t"                                      \
        "mov.b64 a, {al, %5};\n\tmov.b64 a2, {a2l, %5};\n\tmov.b64 b, {bl, %5};\n\t"                               \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%0], a, b, %6, q;\n\t"                                        \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%1], a2, b, %6, q;\n\t}" ::"r"(d_tmem),                       \
        "r"(d_tmem2), "r"(a_lo), "r"(a2_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(acc_first)                        \
        : "memory");                                                                                               \
  }
ADIT_UMMA_KBLOCK2(umma_kblock2_f16, "1")
ADIT_UMMA_KBLOCK2(umma_kblock2_f16_pair, "2")
#undef ADIT_UMMA_KBLOCK2

// A whole step of the issuing thread's k loop as one instruction sequence: test the NEXT stage's "filled" barrier
// (result wanted one step later), issue this k-block's four products (eight for a gate/up pair), commit them to this
// stage's "free" barrier, and only then read the test's result - so that the barrier test's latency is hidden behind
// the products' issue instead of stalling the (in-order) thread.  Returns whether the next stage is already filled.
// The two-SM form commits to the same barrier offset in both blocks of the pair (two commits: the issuing block's own
// barrier and, through its cluster address, the partner's - rank 1 of the two-block cluster).  Barriers are given as 32-bit
// shared-memory addresses (smem_u32), which the caller keeps in registers: every instruction of this thread counts.
#define ADIT_COMMIT_1 "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%7];\n\t"
#define ADIT_COMMIT_2 "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%7];\n\tmapa.shared::cluster.u32 pa, %7, 1;\n\ttcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [pa];\n\t"
#define ADIT_UMMA_STEP(NAME, GROUP, COMMIT)                                                                          \
  __device__ __forceinline__ bool NAME(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc,   \
                                       uint32_t acc_first, uint32_t free_bar, uint32_t next_full, uint32_t parity) { \
    uint32_t ready;                                                                                                  \
    asm volatile(                                                                                                    \
        "{\n\t.reg .pred p, q, r;\n\t.reg .b64 a, b;\n\t.reg .b32 al, bl;\n\t.reg .b32 pa;\n\t"     \
        "mbarrier.test_wait.parity.shared::cta.b64 r, [%8], %9;\n\t"                                                 \
        "setp.ne.b32 p, %6, 0;\n\t"                                                                                  \
        "setp.eq.b32 q, 0, 0;\n\t"                                                                                   \
        "mov.b64 a, {%2, %4};\n\tmov.b64 b, {%3, %4};\n\t"                                                           \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%1], a, b, %5, p;\n\t"                                          \
        "add.u32 al, %2, 2;\n\tadd.u32 bl, %3, 2;\n\tmov.b64 a, {al, %4};\n\tmov.b64 b, {bl, %4};\n\t"               \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%1], a, b, %5, q;\n\t"                                          \
        "add.u32 al, %2, 4;\n\tadd.u32 bl, %3, 4;\n\tmov.b64 a, {al, %4};\n\tmov.b64 b, {bl, %4};\n\t"               \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%1], a, b, %5, q;\n\t"                                          \
        "add.u32 al, %2, 6;\n\tadd.u32 bl, %3, 6;\n\tmov.b64 a, {al, %4};\n\tmov.b64 b, {bl, %4};\n\t"               \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%1], a, b, %5, q;\n\t" COMMIT                                   \
        "selp.u32 %0, 1, 0, r;\n\t}"                                                                                 \
        : "=r"(ready)                                                                                                \
        : "r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(acc_first), "r"(free_bar),                     \
          "r"(next_full), "r"(parity)                                                                      \
        : "memory");                                                                                                 \
    return ready != 0;                                                                                               \
  }
ADIT_UMMA_STEP(umma_step_f16, "1", ADIT_COMMIT_1)
ADIT_UMMA_STEP(umma_step_f16_pair, "2", ADIT_COMMIT_2)
#undef ADIT_UMMA_STEP
#undef ADIT_COMMIT_1
#undef ADIT_COMMIT_2
#define ADIT_COMMIT_1 "tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%9];\n\t"
#define ADIT_COMMIT_2 "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%9];\n\tmapa.shared::cluster.u32 pa, %9, 1;\n\ttcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [pa];\n\t"
#define ADIT_UMMA_STEP2(NAME, GROUP, COMMIT)                                                                         \
  __device__ __forceinline__ bool NAME(uint32_t d_tmem, uint32_t d_tmem2, uint32_t a_lo, uint32_t a2_lo, uint32_t b_lo, \
                                       uint32_t hi, uint32_t idesc, uint32_t acc_first, uint32_t free_bar,           \
                                       uint32_t next_full, uint32_t parity) {                                       \
    uint32_t ready;                                                                                                  \
    asm volatile(                                                                                                    \
        "{\n\t.reg .pred p, q, r;\n\t.reg .b64 a, a2, b;\n\t.reg .b32 al, a2l, bl;\n\t.reg .b32 pa;\n\t" \
        "mbarrier.test_wait.parity.shared::cta.b64 r, [%10], %11;\n\t"                                               \
        "setp.ne.b32 p, %8, 0;\n\t"                                                                                  \
        "setp.eq.b32 q, 0, 0;\n\t"                                                                                   \
        "mov.b64 a, {%3, %6};\n\tmov.b64 a2, {%4, %6};\n\tmov.b64 b, {%5, %6};\n\t"                                  \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%1], a, b, %7, p;\n\t"                                          \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%2], a2, b, %7, p;\n\t"                                         \
        "add.u32 al, %3, 2;\n\tadd.u32 a2l, %4, 2;\n\tadd.u32 bl, %5, 2;\n\t"                                        \
        "mov.b64 a, {al, %6};\n\tmov.b64 a2, {a2l, %6};\n\tmov.b64 b, {bl, %6};\n\t"                                 \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%1], a, b, %7, q;\n\t"                                          \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%2], a2, b, %7, q;\n\t"                                         \
        "add.u32 al, %3, 4;\n\tadd.u32 a2l, %4, 4;\n\tadd.u32 bl, %5, 4;\n\t"                                        \
        "mov.b64 a, {al, %6};\n\tmov.b64 a2, {a2l, %6};\n\tmov.b64 b, {bl, %6};\n\t"                                 \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%1], a, b, %7, q;\n\t"                                          \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%2], a2, b, %7, q;\n\t"                                         \
        "add.u32 al, %3, 6;\n\tadd.u32 a2l, %4, 6;\n\tadd.u32 bl, %5, 6;\n\t"                                        \
        "mov.b64 a, {al, %6};\n\tmov.b64 a2, {a2l, %6};\n\tmov.b64 b, {bl, %6};\n\t"                                 \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%1], a, b, %7, q;\n\t"                                          \
        "tcgen05.mma.cta_group::" GROUP ".kind::f16 [%2], a2, b, %7, q;\n\t" COMMIT                                  \
        "selp.u32 %0, 1, 0, r;\n\t}"                                                                                 \
        : "=r"(ready)                                                                                                \
        : "r"(d_tmem), "r"(d_tmem2), "r"(a_lo), "r"(a2_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(acc_first),          \
          "r"(free_bar), "r"(next_full), "r"(parity)                                             \
        : "memory");                                                                                                 \
    return ready != 0;                                                                                               \
  }
ADIT_UMMA_STEP2(umma_step2_f16, "1", ADIT_COMMIT_1)
ADIT_UMMA_STEP2(umma_step2_f16_pair, "2", ADIT_COMMIT_2)
#undef ADIT_UMMA_STEP2
#undef ADIT_COMMIT_1
#undef ADIT_COMMIT_2

__device__ __forceinline__ bool mbar_test_wait_addr(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait for a thread that must react at once (the product issuer): non-blocking tests in a tight loop for
// about ten microseconds before the clocked, slower loop of mbar_wait takes over.
__device__ __forceinline__ bool mbar_wait_hot(uint64_t* bar, uint32_t parity) {
#pragma unroll 1
  for (int i = 0; i < 2048; ++i)
    if (mbar_test_wait(bar, parity)) return true;
  return mbar_wait(bar, parity);
}
// hot_polls: non-blocking tests before the clocked loop (0 = go to the clock at once: its read takes a few hundred
// nanoseconds, which is a welcome back-off where the data is known to be far away)
__device__ __noinline__ bool mbar_wait_hot_addr(uint32_t bar, uint32_t parity, int hot_polls = 2048) {  // (the slow path: kept out of line)
#pragma unroll 1
  for (int i = 0; i < hot_polls; ++i)
    if (mbar_test_wait_addr(bar, parity)) return true;
  const uint64_t t0 = globaltimer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 1024; ++i)
      if (mbar_test_wait_addr(bar, parity)) return true;
    if (globaltimer_ns() - t0 > 2000000000ull) return false;
  }
}

// ---- the two-SM forms (cta_group::2): a pair of blocks of one cluster (ranks 2i, 2i + 1) works on one product ------
// Every tcgen05 instruction of a kernel names the same cta_group, so a kernel uses either these or the forms above.
// Allocation and release are executed by one warp of each block of the pair; both get the same column range.
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* smem_result, uint32_t ncols) {  // whole warp
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)),
               "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {  // whole warp
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {  // whole warp
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// D (+)= A * B^T over the pair: M = 256 (each block holds 128 rows of A in its shared memory and the matching 128
// lanes of D in its tensor memory), N columns of which each block's shared memory holds one half of B (the even
// block the first half).  Issued by one thread of the even block; the descriptors are offsets into either block's
// shared memory, so both blocks lay their operands out alike.
__device__ __forceinline__ void umma_f16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                              uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ uint32_t mapa_shared(uint32_t local, int rank);
// One arrival on the mbarrier at this shared-memory offset in the blocks of `cta_mask` (bit 0: the issuing, even block;
// bit 1: its partner, rank 1 of the two-block cluster) once all tcgen05 operations issued so far by this thread are
// done: one commit per block, the partner's through its cluster address.
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar, uint16_t cta_mask) {
  const uint32_t local = smem_u32(bar);
  if (cta_mask & 1)
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(local) : "memory");
  if (cta_mask & 2)
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(mapa_shared(local, 1)) : "memory");
}
// 2-D tiled load into this block's shared memory whose completion is counted on an mbarrier that may live in the
// other block of the pair (`bar_cluster` is a shared::cluster address, see mapa_shared).
__device__ __forceinline__ void tma_load_2d_pair(void* smem_dst, const CUtensorMap* map, int x, int y, uint32_t bar_cluster) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          smem_u32(smem_dst)),
      "l"(map), "r"(x), "r"(y), "r"(bar_cluster)
      : "memory");
}

// One step of a copy-issuing thread as a single instruction sequence: test the NEXT stage's "free" barrier (result
// wanted one step later), announce `expect_bytes` on `expect_bar` (skipped when 0), issue the 2-D tiled load, and only
// then read the test's result - the test's latency would otherwise stall the in-order thread at every stage.
// `bar_cluster` is the shared::cluster address of the barrier that counts the copy's bytes (it may live in the other
// block of a pair: the cta_group::2 form).  Returns whether the next stage is already free.
__device__ __forceinline__ bool tma_load_2d_pair_step(void* smem_dst, const CUtensorMap* map, int x, int y, uint32_t bar_cluster,
                                                      uint64_t* expect_bar, uint32_t expect_bytes, uint64_t* next_free,
                                                      uint32_t parity) {
  uint32_t ready;
  asm volatile(
      "{\n\t.reg .pred r, e;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 r, [%8], %9;\n\t"
      "setp.ne.b32 e, %7, 0;\n\t"
      "@e mbarrier.arrive.expect_tx.shared::cta.b64 _, [%6], %7;\n\t"
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%1], [%2, {%3, %4}], [%5];\n\t"
      "selp.u32 %0, 1, 0, r;\n\t}"
      : "=r"(ready)
      : "r"(smem_u32(smem_dst)), "l"(map), "r"(x), "r"(y), "r"(bar_cluster), "r"(smem_u32(expect_bar)), "r"(expect_bytes),
        "r"(smem_u32(next_free)), "r"(parity)
      : "memory");
  return ready != 0;
}

// ---- thread-block clusters and distributed shared memory --------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_arrive_release() { asm volatile("barrier.cluster.arrive.release;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait_acquire() { asm volatile("barrier.cluster.wait.acquire;" ::: "memory"); }
// Address of this block's shared-memory location `local` in the block of rank `rank` of the cluster.
__device__ __forceinline__ uint32_t mapa_shared(uint32_t local, int rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
  return r;
}
// Bulk copy from this block's shared memory into a peer block's shared memory; completion is counted
// in bytes on an mbarrier that lives in the destination block.  Addresses: dst and bar are
// shared::cluster addresses (mapa), src is a shared::cta address; 16-byte aligned, size % 16 == 0.
__device__ __forceinline__ void bulk_copy_to_peer(uint32_t dst_cluster, uint32_t src_cta, uint32_t bytes,
                                                  uint32_t bar_cluster) {
  asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   dst_cluster),
               "r"(src_cta), "r"(bytes), "r"(bar_cluster)
               : "memory");
}
// Bulk store shared -> global (contiguous, 16-byte aligned, size % 16 == 0), tracked by the thread's bulk group.
__device__ __forceinline__ void bulk_store(void* gdst, uint32_t src_cta, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(src_cta), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Wait until the bulk stores of this thread have finished READING shared memory (it may then be reused).
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ float ld_shared_cluster_f32(uint32_t addr) {
  float v;
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ void st_shared_cluster_f32(uint32_t addr, float v) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}

// ---- cross-block signalling inside one kernel ---------------------------------------------------
__device__ __forceinline__ uint32_t ld_acquire_gpu(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_release_gpu_add(uint32_t* p, uint32_t v) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void fence_acq_rel_gpu() { asm volatile("fence.acq_rel.gpu;" ::: "memory"); }
// Orders generic-proxy accesses (of any state space) with later asynchronous-proxy accesses (TMA) of this thread.
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

// mbarrier test with acquire semantics at cluster scope: the data that peers of the cluster pushed into this
// block's shared memory (st.async, counted in bytes on the barrier) is visible once the phase has completed.
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_test_wait_cluster(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// One arrival (release, cluster scope) on an mbarrier of a peer block; `bar_cluster` is a shared::cluster address.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t bar_cluster) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster) : "memory");
}
// The same as a pure signal (no data is published with it): relaxed, so that it does not wait for this thread's
// earlier global stores the way a release would.
__device__ __forceinline__ void mbar_arrive_remote_relaxed(uint32_t bar_cluster) {
  asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster) : "memory");
}
__device__ __forceinline__ uint32_t ld_relaxed_gpu(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
// Asynchronous 16-byte store into a peer block's shared memory; the destination block's mbarrier counts the bytes.
__device__ __forceinline__ void st_async_v4(uint32_t dst_cluster, uint32_t a, uint32_t b, uint32_t c, uint32_t d,
                                            uint32_t bar_cluster) {
  asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];" ::"r"(
                   dst_cluster),
               "r"(a), "r"(b), "r"(c), "r"(d), "r"(bar_cluster)
               : "memory");
}
__device__ __forceinline__ void st_async_v2(uint32_t dst_cluster, uint32_t a, uint32_t b, uint32_t bar_cluster) {
  asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.v2.b32 [%0], {%1, %2}, [%3];" ::"r"(dst_cluster),
               "r"(a), "r"(b), "r"(bar_cluster)
               : "memory");
}

// ---- programmatic dependent launch ------------------------------------------------------------
__device__ __forceinline__ void pdl_wait_prior_grids() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
}

}  // namespace ptx
}  // namespace adit
