// Blackwell (sm_100a) building blocks in inline PTX: mbarriers with bounded waits, TMA tensor
// loads, TMEM allocation, tcgen05.mma with shared-memory descriptors, tcgen05.ld.
//
// Every wait in here has an iteration limit.  A wait that runs out sets the CTA's abort flag;
// all roles poll that flag, leave their loops, and the kernel reports TWKV_ERR_TIMEOUT through
// the cache's status word instead of hanging the GPU.
#pragma once
#include <cuda.h>
#include "twkv_dev.h"

namespace twkv {
namespace tc {

// try_wait attempts of a bounded wait.  An attempt on a barrier that does not complete suspends the thread for about
// 4 microseconds (measured: 16384 attempts take 66 ms), so a wait gives up after about one second; the longest
// legitimate wait in any kernel of the library is a few milliseconds.
constexpr uint32_t SPIN_LIMIT = 1u << 18;

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_init_fence() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
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
// Bounded wait.  Returns false if the wait ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait_limited(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t limit) {
  for (uint32_t i = 0; i < limit; ++i) {
    if (mbar_try(bar, parity)) return true;
    if ((i & 63u) == 63u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  return mbar_wait_limited(bar, parity, abort_flag, SPIN_LIMIT);
}

// The same wait for a role that runs on one thread and must spend few instructions: one attempt inline, the bounded
// loop out of line.
static __device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  return mbar_wait(bar, parity, abort_flag);
}
__device__ __forceinline__ bool mbar_wait_thin(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, abort_flag);
}

// Used only after a give-up: lets copies already in flight land before the CTA exits.
__device__ __forceinline__ void mbar_wait_drain(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < (1u << 16); ++i)
    if (mbar_try(bar, parity)) return;
}

// 2-D tiled TMA load (no multicast): box lands in shared memory, completion counted on `bar`.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// TMEM allocation: one full warp, power-of-two column count >= 32; base address lands in shared memory.
__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t base, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(base), "r"(cols) : "memory");
}
__device__ __forceinline__ void fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major operand tile stored as rows of 128 bytes with the
// 128-byte swizzle (what a TMA box of 64 16-bit elements x R rows with SWIZZLE_128B writes):
// 8-row groups are 1024 bytes apart.  The tile base must be 1024-byte aligned; advancing along K
// by 16 elements adds 32 bytes to the start address.
__device__ __forceinline__ uint64_t kmajor_sw128_desc(uint32_t addr) {
  return (uint64_t)((addr >> 4) & 0x3fffu) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor, kind::f16: fp32 accumulate, A and B both `fmt` (0 = f16, 1 = bf16), both K-major.
__host__ __device__ constexpr uint32_t idesc_f16(int fmt, int M, int N) {
  return (1u << 4) | ((uint32_t)fmt << 7) | ((uint32_t)fmt << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// D[tmem] (+)= A[smem] * B[smem]^T, issued by one thread.
__device__ __forceinline__ void mma_f16_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// Descriptor halves: the low word carries the start address (>> 4) and the leading byte offset, the high word the
// stride (1024 bytes between 8-row groups), the version and the swizzle mode; K steps of 16 elements and whole
// panels only move the low word, so a single thread can step descriptors with 32-bit adds.
__device__ __forceinline__ uint32_t kmajor_sw128_desc_lo(uint32_t addr) { return ((addr >> 4) & 0x3fffu) | (1u << 16); }
constexpr uint32_t KMAJOR_SW128_DESC_HI = 64u | (1u << 14) | (2u << 29);
// Four MMAs over one 64-wide K panel (K steps of 16): D (+)= A[panel] * B[panel]^T, accumulate = 0 overwrites D first.
// CG = 2: the CTA-pair form (M = 256 over the pair, each CTA supplies its own A rows and half of B's rows).
#define TWKV_SS_PANEL_ASM(CGS)                                                                                          \
  asm volatile(                                                                                                         \
      "{\n\t.reg .pred p0, p1;\n\t.reg .b64 da, db;\n\t.reg .b32 al, bl;\n\t"                                          \
      "setp.ne.b32 p0, %4, 0;\n\t"                                                                                      \
      "setp.eq.b32 p1, %4, %4;\n\t"                                                                                     \
      "mov.b64 da, {%1, %5};\n\tmov.b64 db, {%2, %5};\n\t"                                                             \
      "tcgen05.mma.cta_group::" CGS ".kind::f16 [%0], da, db, %3, p0;\n\t"                                              \
      "add.u32 al, %1, 2;\n\tadd.u32 bl, %2, 2;\n\tmov.b64 da, {al, %5};\n\tmov.b64 db, {bl, %5};\n\t"                \
      "tcgen05.mma.cta_group::" CGS ".kind::f16 [%0], da, db, %3, p1;\n\t"                                              \
      "add.u32 al, %1, 4;\n\tadd.u32 bl, %2, 4;\n\tmov.b64 da, {al, %5};\n\tmov.b64 db, {bl, %5};\n\t"                \
      "tcgen05.mma.cta_group::" CGS ".kind::f16 [%0], da, db, %3, p1;\n\t"                                              \
      "add.u32 al, %1, 6;\n\tadd.u32 bl, %2, 6;\n\tmov.b64 da, {al, %5};\n\tmov.b64 db, {bl, %5};\n\t"                \
      "tcgen05.mma.cta_group::" CGS ".kind::f16 [%0], da, db, %3, p1;\n\t}"                                             \
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(KMAJOR_SW128_DESC_HI) : "memory")
template <int CG>
__device__ __forceinline__ void mma_f16_ss_panel_cg(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc, uint32_t accumulate) {
  if constexpr (CG == 2) TWKV_SS_PANEL_ASM("2"); else TWKV_SS_PANEL_ASM("1");
}
#define TWKV_TS_K128_ASM(CGS)                                                                                           \
  asm volatile(                                                                                                         \
      "{\n\t.reg .pred p0, p1;\n\t.reg .b64 db;\n\t.reg .b32 bl, b2, ta;\n\t"                                          \
      "setp.ne.b32 p0, %4, 0;\n\t"                                                                                      \
      "setp.eq.b32 p1, %4, %4;\n\t"                                                                                     \
      "add.u32 b2, %2, %6;\n\t"                                                                                         \
      "mov.b64 db, {%2, %5};\n\t"                                                                                       \
      "tcgen05.mma.cta_group::" CGS ".kind::f16 [%0], [%1], db, %3, p0;\n\t"                                            \
      "add.u32 ta, %1, 8;\n\tadd.u32 bl, %2, 2;\n\tmov.b64 db, {bl, %5};\n\t"                                          \
      "tcgen05.mma.cta_group::" CGS ".kind::f16 [%0], [ta], db, %3, p1;\n\t"                                            \
      "add.u32 ta, %1, 16;\n\tadd.u32 bl, %2, 4;\n\tmov.b64 db, {bl, %5};\n\t"                                         \
      "tcgen05.mma.cta_group::" CGS ".kind::f16 [%0], [ta], db, %3, p1;\n\t"                                            \
      "add.u32 ta, %1, 24;\n\tadd.u32 bl, %2, 6;\n\tmov.b64 db, {bl, %5};\n\t"                                         \
      "tcgen05.mma.cta_group::" CGS ".kind::f16 [%0], [ta], db, %3, p1;\n\t"                                            \
      "add.u32 ta, %1, 32;\n\tmov.b64 db, {b2, %5};\n\t"                                                               \
      "tcgen05.mma.cta_group::" CGS ".kind::f16 [%0], [ta], db, %3, p1;\n\t"                                            \
      "add.u32 ta, %1, 40;\n\tadd.u32 bl, b2, 2;\n\tmov.b64 db, {bl, %5};\n\t"                                         \
      "tcgen05.mma.cta_group::" CGS ".kind::f16 [%0], [ta], db, %3, p1;\n\t"                                            \
      "add.u32 ta, %1, 48;\n\tadd.u32 bl, b2, 4;\n\tmov.b64 db, {bl, %5};\n\t"                                         \
      "tcgen05.mma.cta_group::" CGS ".kind::f16 [%0], [ta], db, %3, p1;\n\t"                                            \
      "add.u32 ta, %1, 56;\n\tadd.u32 bl, b2, 6;\n\tmov.b64 db, {bl, %5};\n\t"                                         \
      "tcgen05.mma.cta_group::" CGS ".kind::f16 [%0], [ta], db, %3, p1;\n\t}"                                           \
      ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(KMAJOR_SW128_DESC_HI), "r"(panel_step) : "memory")
// Eight MMAs over K = 128 with A in tensor memory (8 columns per K step) and B as two 64-wide K panels
// `panel_step` (in 16-byte units) apart.
template <int CG>
__device__ __forceinline__ void mma_f16_ts_k128_cg(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t panel_step, uint32_t idesc,
                                                   uint32_t accumulate) {
  if constexpr (CG == 2) TWKV_TS_K128_ASM("2"); else TWKV_TS_K128_ASM("1");
}
__device__ __forceinline__ void mma_f16_ss_panel(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p0, p1;\n\t.reg .b64 da, db;\n\t.reg .b32 al, bl;\n\t"
      "setp.ne.b32 p0, %4, 0;\n\t"
      "setp.eq.b32 p1, %4, %4;\n\t"
      "mov.b64 da, {%1, %5};\n\tmov.b64 db, {%2, %5};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p0;\n\t"
      "add.u32 al, %1, 2;\n\tadd.u32 bl, %2, 2;\n\tmov.b64 da, {al, %5};\n\tmov.b64 db, {bl, %5};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p1;\n\t"
      "add.u32 al, %1, 4;\n\tadd.u32 bl, %2, 4;\n\tmov.b64 da, {al, %5};\n\tmov.b64 db, {bl, %5};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p1;\n\t"
      "add.u32 al, %1, 6;\n\tadd.u32 bl, %2, 6;\n\tmov.b64 da, {al, %5};\n\tmov.b64 db, {bl, %5};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p1;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(KMAJOR_SW128_DESC_HI) : "memory");
}
// Eight MMAs over K = 128 with A in tensor memory (8 columns per K step) and B as two 64-wide K panels
// `panel_step` (in 16-byte units) apart.
__device__ __forceinline__ void mma_f16_ts_k128(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t panel_step, uint32_t idesc,
                                                uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p0, p1;\n\t.reg .b64 db;\n\t.reg .b32 bl, b2, ta;\n\t"
      "setp.ne.b32 p0, %4, 0;\n\t"
      "setp.eq.b32 p1, %4, %4;\n\t"
      "add.u32 b2, %2, %6;\n\t"
      "mov.b64 db, {%2, %5};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %3, p0;\n\t"
      "add.u32 ta, %1, 8;\n\tadd.u32 bl, %2, 2;\n\tmov.b64 db, {bl, %5};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [ta], db, %3, p1;\n\t"
      "add.u32 ta, %1, 16;\n\tadd.u32 bl, %2, 4;\n\tmov.b64 db, {bl, %5};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [ta], db, %3, p1;\n\t"
      "add.u32 ta, %1, 24;\n\tadd.u32 bl, %2, 6;\n\tmov.b64 db, {bl, %5};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [ta], db, %3, p1;\n\t"
      "add.u32 ta, %1, 32;\n\tmov.b64 db, {b2, %5};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [ta], db, %3, p1;\n\t"
      "add.u32 ta, %1, 40;\n\tadd.u32 bl, b2, 2;\n\tmov.b64 db, {bl, %5};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [ta], db, %3, p1;\n\t"
      "add.u32 ta, %1, 48;\n\tadd.u32 bl, b2, 4;\n\tmov.b64 db, {bl, %5};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [ta], db, %3, p1;\n\t"
      "add.u32 ta, %1, 56;\n\tadd.u32 bl, b2, 6;\n\tmov.b64 db, {bl, %5};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [ta], db, %3, p1;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(KMAJOR_SW128_DESC_HI), "r"(panel_step) : "memory");
}
// Arrive on `bar` once every tcgen05 operation issued so far by this thread has completed.
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// tcgen05.ld / tcgen05.st, shape 32x32b: thread i of the warp owns TMEM lane (lane base + i) and
// moves N consecutive 32-bit columns starting at the address's column.  A warp may only touch
// the lane quarter 32 * (warp index % 4).
__device__ __forceinline__ void tmem_ld1(uint32_t taddr, uint32_t* r) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];"
               : "=r"(r[0]) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld2(uint32_t taddr, uint32_t* r) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x2.b32 {%0, %1}, [%2];"
               : "=r"(r[0]), "=r"(r[1]) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld4(uint32_t taddr, uint32_t* r) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t* r) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t* r) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               :: "r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]) : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
               :: "r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) { tmem_ld32(taddr, reinterpret_cast<uint32_t*>(v)); }
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// D[tmem] (+)= A[tmem] * B[smem]^T: A is read from tensor memory (lane = row, two 16-bit K
// elements per 32-bit column, the lower K index in the lower half).
__device__ __forceinline__ void mma_f16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// Makes generic-proxy writes to shared memory visible to the async proxy (TMA, tcgen05.mma operand reads).
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// Two floats -> packed f16x2 (lo in bits 0..15), round to nearest, saturating to the finite range.
__device__ __forceinline__ uint32_t pack_f16x2_sat(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}

__device__ __forceinline__ void named_bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
}

// ---- CTA pairs (cta_group::2): two CTAs of a cluster on neighbouring SMs share one MMA ----
__device__ __forceinline__ uint32_t cluster_cta_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of the same shared-memory object in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t cluster_map(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}
// TMA load whose completion is counted on a barrier that may live in the partner CTA (no multicast).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster_addr, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar_cluster_addr), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t slot_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t base, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(base), "r"(cols) : "memory");
}
__device__ __forceinline__ void mma_f16_ss_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// arrives, once the pair's MMAs issued so far have retired, on one barrier (of the issuing CTA)
__device__ __forceinline__ void mma_commit_pair(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// arrives, once the pair's MMAs issued so far have retired, on the barrier at this offset in both CTAs
__device__ __forceinline__ void mma_commit_pair_both(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((unsigned short)3) : "memory");
}

// ---- the main loop shared by the dense kernels whose operands stream through a ring (gate logits, projection) ----
// A ring stage holds one K = 64 panel of the row operand (`x_bytes` at offset 0: 128 rows of this CTA) and one of the
// column operand (at `b_off`: N rows, or this CTA's half of them in a pair).  An accumulator is KP stages; accumulators
// alternate between two 256-column TMEM buffers.  CG = 2: the CTA-pair form (both CTAs produce, the even CTA issues;
// `full` and `acc_empty` live in the even CTA, `empty` and `acc_full` are signalled in both by a multicast commit).
//
// Producer: one elected thread issues every copy in ring order.  coord(a, map_x, map_w, m0, n0) names the tensor maps
// and the first rows of accumulator a's operands.
template <int CG, class Coord>
__device__ __forceinline__ void ring_gemm_produce(uint32_t n_acc, int KP, uint32_t stages, uint32_t sA, uint32_t stage_bytes, uint32_t b_off,
                                                  uint32_t tx_bytes, uint32_t full, uint32_t empty, uint32_t crank,
                                                  volatile int* abort_flag, Coord coord) {
  uint32_t st = 0, ph = 0;
  for (uint32_t a = 0; a < n_acc; ++a) {
    const CUtensorMap *map_x, *map_w;
    int m0, n0;
    coord(a, map_x, map_w, m0, n0);
    for (int p = 0; p < KP; ++p) {
      if (!mbar_wait_thin(empty + 8 * st, ph ^ 1u, abort_flag)) return;
      if constexpr (CG == 2) {
        const uint32_t full_even = cluster_map(full + 8 * st, 0);              // the even CTA's barrier of this stage
        if (crank == 0) mbar_expect_tx(full + 8 * st, tx_bytes);                // both CTAs' two copies
        tma_load_2d_pair(sA + st * stage_bytes, map_x, full_even, p * TWKV_PANEL_ELEMS, m0);
        tma_load_2d_pair(sA + st * stage_bytes + b_off, map_w, full_even, p * TWKV_PANEL_ELEMS, n0);
      } else {
        mbar_expect_tx(full + 8 * st, tx_bytes);
        tma_load_2d(sA + st * stage_bytes, map_x, full + 8 * st, p * TWKV_PANEL_ELEMS, m0);
        tma_load_2d(sA + st * stage_bytes + b_off, map_w, full + 8 * st, p * TWKV_PANEL_ELEMS, n0);
      }
      if (++st == stages) { st = 0; ph ^= 1u; }
    }
  }
}
// Issuer: one elected thread (of the even CTA in a pair); four MMAs per stage, the stage handed back when they retire.
template <int CG>
__device__ __forceinline__ void ring_gemm_issue(uint32_t n_acc, int KP, uint32_t stages, uint32_t sA, uint32_t stage_bytes, uint32_t b_off,
                                                uint32_t idesc, uint32_t tmem_base, uint32_t full, uint32_t empty, uint32_t acc_full,
                                                uint32_t acc_empty, volatile int* abort_flag) {
  const uint64_t adesc0 = kmajor_sw128_desc(sA), bdesc0 = kmajor_sw128_desc(sA + b_off);
  uint32_t st = 0, ph = 0;
  for (uint32_t ac = 0; ac < n_acc; ++ac) {
    const uint32_t buf = ac & 1u;
    if (!mbar_wait(acc_empty + 8 * buf, ((ac >> 1) & 1u) ^ 1u, abort_flag)) return;
    fence_after_sync();
    const uint32_t dcol = tmem_base + buf * 256;
    for (int p = 0; p < KP; ++p) {
      if (!mbar_wait(full + 8 * st, ph, abort_flag)) return;
      fence_after_sync();
      const uint64_t adesc = adesc0 + (uint64_t)(st * (stage_bytes >> 4));
      const uint64_t bdesc = bdesc0 + (uint64_t)(st * (stage_bytes >> 4));
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
        if constexpr (CG == 2) mma_f16_ss_pair(dcol, adesc + 2 * ks, bdesc + 2 * ks, idesc, (p > 0 || ks > 0) ? 1u : 0u);
        else mma_f16_ss(dcol, adesc + 2 * ks, bdesc + 2 * ks, idesc, (p > 0 || ks > 0) ? 1u : 0u);
      }
      if constexpr (CG == 2) mma_commit_pair_both(empty + 8 * st); else mma_commit(empty + 8 * st);
      if (++st == stages) { st = 0; ph ^= 1u; }
    }
    if constexpr (CG == 2) mma_commit_pair_both(acc_full + 8 * buf); else mma_commit(acc_full + 8 * buf);
  }
}

}  // namespace tc

// Tensor maps the decode path needs: the block pool as rows of 64 elements, and the layer's transposed U_K^-1.
// `scores`: the score scratch for the V pass's TMA copies, or null when the head count does not allow them.
struct TcMaps { CUtensorMap blocks, uinvT_k; const CUtensorMap* scores; };
// Tensor maps of the fused gate kernel: the call's K and V states, and the layer's transposed gate weights.
// `raw`: the same four operands as plain pointers (states row-major, weights transposed), for the rows the kernel
// decides again in fp32.
// fix_list / fix_counters: rows handed to the fix-up kernel (two int4 per row) and {entries, finished CTAs}.
struct GateRaw { const unsigned short *xk, *xv, *wkT, *wvT; int4* fix_list; int* fix_counters; };
struct GateMaps { CUtensorMap xk, xv, wk, wv; GateRaw raw; };
// Tensor maps of the projection kernel: the call's raw states, the transposed bases, and the outputs.
struct ProjectMaps { CUtensorMap xk, xv, uk, uv, ok, ov; };

// Host side: 2-D tensor map over a row-major 16-bit matrix [rows][cols], box [box_rows][64], 128-byte swizzle.
bool make_tmap_2d(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint64_t row_stride_bytes, uint32_t box_rows);

}  // namespace twkv
