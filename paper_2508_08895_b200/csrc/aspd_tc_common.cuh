// PTX wrappers shared by the tensor-core attention kernels: mbarriers with bounded waits, bulk
// copies, tcgen05 MMA / commit / TMEM load and store, shared-memory and instruction descriptors.
#pragma once

#include "aspd_internal.cuh"

namespace aspd {
namespace {

constexpr long long kWaitCycles = 3000000000LL; // ~1.5 s at 1.9 GHz

// ------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// The same question without any waiting (try_wait may suspend the thread for a while before it answers).
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: false means "give up" (time limit hit here or in another role).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          long long limit = kWaitCycles) {
  if (mbar_try(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    if (mbar_try(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > limit) { *abort_flag = 1; return false; }
  }
}
__device__ __forceinline__ void bulk_copy(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
// The same two, executed by a whole warp with warp-uniform operands; lane 0 alone issues.  With
// uniform control flow around them the descriptors stay in the uniform datapath.
__device__ __forceinline__ void tc_commit_lane0(uint32_t bar) {
  asm volatile(
      "{\n\t.reg .pred e;\n\t.reg .u32 l;\n\t"
      "mov.u32 l, %%laneid;\n\t"
      "setp.eq.u32 e, l, 0;\n\t"
      "@e tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_lane0(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p, e;\n\t.reg .u32 l;\n\t"
      "mov.u32 l, %%laneid;\n\t"
      "setp.eq.u32 e, l, 0;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
// A operand in tensor memory (M = 128: lane = row, 16-bit elements packed two to a column).
__device__ __forceinline__ void tc_mma_ts_lane0(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p, e;\n\t.reg .u32 l;\n\t"
      "mov.u32 l, %%laneid;\n\t"
      "setp.eq.u32 e, l, 0;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
// Whole operations in one statement each, so that the issuing warp spends a handful of instructions
// per MMA (it shares its scheduler with softmax warps; descriptor arithmetic per MMA made an
// operation of 8 take ~600 cycles to issue).  A descriptor's low bits are the address / 16, so the
// k-steps are additions to the first descriptor.
//
// Eight k-steps of a 128 x N x 128 product with both operands in shared memory (K-major, 128-byte
// swizzle): k-step ks reads A at +32 (ks % 4) bytes in half ks / 4 (a_half bytes apart), B likewise
// with halves b_half bytes apart.  Lane 0 issues; the first k-step overwrites the accumulator.
template <uint32_t A_HALF, uint32_t B_HALF>
__device__ __forceinline__ void tc_mma_ss_k128_lane0(uint32_t d_tmem, uint64_t a0, uint64_t b0, uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred e, z, o;\n\t.reg .u32 l;\n\t.reg .b64 a, b;\n\t"
      "mov.u32 l, %%laneid;\n\t"
      "setp.eq.u32 e, l, 0;\n\t"
      "setp.ne.b32 z, 0, 0;\n\t"
      "setp.eq.b32 o, 0, 0;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, z;\n\t"
      "add.s64 a, %1, 2;\n\tadd.s64 b, %2, 2;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, o;\n\t"
      "add.s64 a, %1, 4;\n\tadd.s64 b, %2, 4;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, o;\n\t"
      "add.s64 a, %1, 6;\n\tadd.s64 b, %2, 6;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, o;\n\t"
      "add.s64 a, %1, %4;\n\tadd.s64 b, %2, %5;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, o;\n\t"
      "add.s64 a, %1, %4 + 2;\n\tadd.s64 b, %2, %5 + 2;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, o;\n\t"
      "add.s64 a, %1, %4 + 4;\n\tadd.s64 b, %2, %5 + 4;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, o;\n\t"
      "add.s64 a, %1, %4 + 6;\n\tadd.s64 b, %2, %5 + 6;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, o;\n\t}"
      ::"r"(d_tmem), "l"(a0), "l"(b0), "r"(idesc), "n"(A_HALF / 16), "n"(B_HALF / 16) : "memory");
}
// Up to four k-steps of 16 keys of O += P . V: P (bf16) in tensor memory, 8 columns per k-step; V
// pages of 4096 bytes in shared memory.  `first_acc` = 0 overwrites the accumulator at the first k-step.
__device__ __forceinline__ void tc_mma_ts_pv_lane0(uint32_t d_tmem, uint32_t p_tmem, uint64_t v0, uint32_t idesc, uint32_t first_acc, int n) {
  asm volatile(
      "{\n\t.reg .pred e, f, o, q;\n\t.reg .u32 l;\n\t.reg .b32 t;\n\t.reg .b64 b;\n\t"
      "mov.u32 l, %%laneid;\n\t"
      "setp.eq.u32 e, l, 0;\n\t"
      "setp.ne.b32 f, %4, 0;\n\t"
      "setp.eq.b32 o, 0, 0;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, f;\n\t"
      "setp.gt.and.s32 q, %5, 1, e;\n\t"
      "add.u32 t, %1, 8;\n\tadd.s64 b, %2, 256;\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], [t], b, %3, o;\n\t"
      "setp.gt.and.s32 q, %5, 2, e;\n\t"
      "add.u32 t, %1, 16;\n\tadd.s64 b, %2, 512;\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], [t], b, %3, o;\n\t"
      "setp.gt.and.s32 q, %5, 3, e;\n\t"
      "add.u32 t, %1, 24;\n\tadd.s64 b, %2, 768;\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], [t], b, %3, o;\n\t}"
      ::"r"(d_tmem), "r"(p_tmem), "l"(v0), "r"(idesc), "r"(first_acc), "r"(n) : "memory");
}
// Up to eight k-steps of 16 keys of O += P . V with both operands in shared memory: P K-major in two
// spans of 64 keys (A_HALF bytes apart), V pages of 4096 bytes.  `first_acc` = 0 overwrites the
// accumulator at the first k-step; k-steps at and beyond n are skipped.
template <uint32_t A_HALF>
__device__ __forceinline__ void tc_mma_ss_pv_lane0(uint32_t d_tmem, uint64_t p0, uint64_t v0, uint32_t idesc, uint32_t first_acc, int n) {
  asm volatile(
      "{\n\t.reg .pred e, f, o, q;\n\t.reg .u32 l;\n\t.reg .b64 a, b;\n\t"
      "mov.u32 l, %%laneid;\n\t"
      "setp.eq.u32 e, l, 0;\n\t"
      "setp.ne.b32 f, %4, 0;\n\t"
      "setp.eq.b32 o, 0, 0;\n\t"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, f;\n\t"
      "setp.gt.and.s32 q, %5, 1, e;\n\t"
      "add.s64 a, %1, 2;\n\tadd.s64 b, %2, 256;\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, o;\n\t"
      "setp.gt.and.s32 q, %5, 2, e;\n\t"
      "add.s64 a, %1, 4;\n\tadd.s64 b, %2, 512;\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, o;\n\t"
      "setp.gt.and.s32 q, %5, 3, e;\n\t"
      "add.s64 a, %1, 6;\n\tadd.s64 b, %2, 768;\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, o;\n\t"
      "setp.gt.and.s32 q, %5, 4, e;\n\t"
      "add.s64 a, %1, %6;\n\tadd.s64 b, %2, 1024;\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, o;\n\t"
      "setp.gt.and.s32 q, %5, 5, e;\n\t"
      "add.s64 a, %1, %6 + 2;\n\tadd.s64 b, %2, 1280;\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, o;\n\t"
      "setp.gt.and.s32 q, %5, 6, e;\n\t"
      "add.s64 a, %1, %6 + 4;\n\tadd.s64 b, %2, 1536;\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, o;\n\t"
      "setp.gt.and.s32 q, %5, 7, e;\n\t"
      "add.s64 a, %1, %6 + 6;\n\tadd.s64 b, %2, 1792;\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], a, b, %3, o;\n\t}"
      ::"r"(d_tmem), "l"(p0), "l"(v0), "r"(idesc), "r"(first_acc), "r"(n), "n"(A_HALF / 16) : "memory");
}
__device__ __forceinline__ void named_sync(int id, int n) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n) : "memory"); }
// Barrier among n threads that also ORs a predicate, so that all of them take the same exit.
__device__ __forceinline__ bool named_sync_or(int id, int n, bool pred) {
  uint32_t out;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 q, %3, 0;\n\t"
      "bar.red.or.pred p, %1, %2, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(out) : "r"(id), "r"(n), "r"((uint32_t)pred) : "memory");
  return out != 0;
}

#define ASPD_R32(v, o) "=f"(v[o + 0]), "=f"(v[o + 1]), "=f"(v[o + 2]), "=f"(v[o + 3]), "=f"(v[o + 4]), "=f"(v[o + 5]),  \
    "=f"(v[o + 6]), "=f"(v[o + 7]), "=f"(v[o + 8]), "=f"(v[o + 9]), "=f"(v[o + 10]), "=f"(v[o + 11]), "=f"(v[o + 12]),    \
    "=f"(v[o + 13]), "=f"(v[o + 14]), "=f"(v[o + 15]), "=f"(v[o + 16]), "=f"(v[o + 17]), "=f"(v[o + 18]),                 \
    "=f"(v[o + 19]), "=f"(v[o + 20]), "=f"(v[o + 21]), "=f"(v[o + 22]), "=f"(v[o + 23]), "=f"(v[o + 24]),                 \
    "=f"(v[o + 25]), "=f"(v[o + 26]), "=f"(v[o + 27]), "=f"(v[o + 28]), "=f"(v[o + 29]), "=f"(v[o + 30]), "=f"(v[o + 31])
#define ASPD_W32(v, o) "f"(v[o + 0]), "f"(v[o + 1]), "f"(v[o + 2]), "f"(v[o + 3]), "f"(v[o + 4]), "f"(v[o + 5]),        \
    "f"(v[o + 6]), "f"(v[o + 7]), "f"(v[o + 8]), "f"(v[o + 9]), "f"(v[o + 10]), "f"(v[o + 11]), "f"(v[o + 12]),           \
    "f"(v[o + 13]), "f"(v[o + 14]), "f"(v[o + 15]), "f"(v[o + 16]), "f"(v[o + 17]), "f"(v[o + 18]), "f"(v[o + 19]),       \
    "f"(v[o + 20]), "f"(v[o + 21]), "f"(v[o + 22]), "f"(v[o + 23]), "f"(v[o + 24]), "f"(v[o + 25]), "f"(v[o + 26]),       \
    "f"(v[o + 27]), "f"(v[o + 28]), "f"(v[o + 29]), "f"(v[o + 30]), "f"(v[o + 31])

// 32 consecutive fp32 columns of this thread's TMEM lane -> v[o .. o+31]
#define ASPD_TMEM_LD32(taddr, v, o)                                                                               \
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, "  \
               "%13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, " \
               "[%32];" : ASPD_R32(v, o) : "r"(taddr) : "memory")
#define ASPD_TMEM_ST32(taddr, v, o)                                                                               \
  asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, " \
               "%12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, "   \
               "%31};" ::ASPD_W32(v, o), "r"(taddr) : "memory")
#define ASPD_U32(v, o) "r"(v[o + 0]), "r"(v[o + 1]), "r"(v[o + 2]), "r"(v[o + 3]), "r"(v[o + 4]), "r"(v[o + 5]), "r"(v[o + 6]),   \
    "r"(v[o + 7]), "r"(v[o + 8]), "r"(v[o + 9]), "r"(v[o + 10]), "r"(v[o + 11]), "r"(v[o + 12]), "r"(v[o + 13]), "r"(v[o + 14]),  \
    "r"(v[o + 15]), "r"(v[o + 16]), "r"(v[o + 17]), "r"(v[o + 18]), "r"(v[o + 19]), "r"(v[o + 20]), "r"(v[o + 21]),              \
    "r"(v[o + 22]), "r"(v[o + 23]), "r"(v[o + 24]), "r"(v[o + 25]), "r"(v[o + 26]), "r"(v[o + 27]), "r"(v[o + 28]),              \
    "r"(v[o + 29]), "r"(v[o + 30]), "r"(v[o + 31])
// 32 uint32 of this thread -> 32 consecutive columns of its TMEM lane
#define ASPD_TMEM_ST32U(taddr, v, o)                                                                              \
  asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, " \
               "%12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, "   \
               "%31};" ::ASPD_U32(v, o), "r"(taddr) : "memory")
#define ASPD_TMEM_LD16(taddr, v, o)                                                                               \
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, "  \
               "%13, %14, %15}, [%16];"                                                                          \
               : "=f"(v[o + 0]), "=f"(v[o + 1]), "=f"(v[o + 2]), "=f"(v[o + 3]), "=f"(v[o + 4]), "=f"(v[o + 5]),  \
                 "=f"(v[o + 6]), "=f"(v[o + 7]), "=f"(v[o + 8]), "=f"(v[o + 9]), "=f"(v[o + 10]), "=f"(v[o + 11]), \
                 "=f"(v[o + 12]), "=f"(v[o + 13]), "=f"(v[o + 14]), "=f"(v[o + 15])                               \
               : "r"(taddr) : "memory")
// 16 lanes x 256 bits per block, N blocks along the columns: thread t of the warp gets, per block of 8
// columns, columns 2 (t % 4), + 1 of lane t / 4 (registers 4 n, 4 n + 1) and of lane t / 4 + 8 (4 n + 2,
// 4 n + 3): the accumulator of an M = 64 MMA keeps 16 rows in lanes 0..15 of each 32-lane quadrant.
#define ASPD_TMEM_LD16x256_X4(taddr, v)                                                                             \
  asm volatile("tcgen05.ld.sync.aligned.16x256b.x4.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, "    \
               "%13, %14, %15}, [%16];"                                                                            \
               : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7]),    \
                 "=f"(v[8]), "=f"(v[9]), "=f"(v[10]), "=f"(v[11]), "=f"(v[12]), "=f"(v[13]), "=f"(v[14]), "=f"(v[15]) \
               : "r"(taddr) : "memory")
#define ASPD_TMEM_LD16x256_X8(taddr, v)                                                                             \
  asm volatile("tcgen05.ld.sync.aligned.16x256b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, "    \
               "%13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, "   \
               "[%32];" : ASPD_R32(v, 0) : "r"(taddr) : "memory")
#define ASPD_TMEM_ST16x256_X4(taddr, v)                                                                             \
  asm volatile("tcgen05.st.sync.aligned.16x256b.x4.b32 [%16], {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, "  \
               "%12, %13, %14, %15};"                                                                              \
               ::"f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]), "f"(v[8]), \
                 "f"(v[9]), "f"(v[10]), "f"(v[11]), "f"(v[12]), "f"(v[13]), "f"(v[14]), "f"(v[15]), "r"(taddr) : "memory")
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle, descriptor version 1.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128 (or 64), A K-major.
__device__ __forceinline__ uint32_t instr_desc(uint32_t n, uint32_t b_mn_major, uint32_t m = 128u) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major << 16) | ((n >> 3) << 17) | ((m >> 4) << 24);
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// 2^x for two values on the FMA and integer pipes instead of the special-function unit (which takes
// a warp's instruction only every 8 cycles): x = n + f with n the nearest integer (the magic-number
// addition leaves n in the low bits), 2^f by a cubic (largest relative error 8e-5 on [-1/2, 1/2],
// a twenty-fifth of what rounding the result to bf16 costs), n added to the exponent bits.  The
// argument is clamped to the exponent range, so that a huge value still ends far above 2^40 and a
// tiny one near 2^-126.
__device__ __forceinline__ float2 ex2_fma2(float2 x) {
  x.x = fminf(fmaxf(x.x, -126.f), 127.f);
  x.y = fminf(fmaxf(x.y, -126.f), 127.f);
  const float2 magic = make_float2(12582912.f, 12582912.f);
  const float2 t = __fadd2_rn(x, magic);
  const float2 n = __fadd2_rn(t, make_float2(-12582912.f, -12582912.f));
  const float2 f = __ffma2_rn(n, make_float2(-1.f, -1.f), x);
  float2 p = __ffma2_rn(f, make_float2(0.05519810691f, 0.05519810691f), make_float2(0.24267712235f, 0.24267712235f));
  p = __ffma2_rn(p, f, make_float2(0.69326180220f, 0.69326180220f));
  p = __ffma2_rn(p, f, make_float2(0.99992275238f, 0.99992275238f));
  return make_float2(__int_as_float(__float_as_int(p.x) + (__float_as_int(t.x) << 23)),
                     __int_as_float(__float_as_int(p.y) + (__float_as_int(t.y) << 23)));
}
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}

}  // namespace
}  // namespace aspd
