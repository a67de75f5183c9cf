// Inline-PTX wrappers for the Blackwell (sm_100a) features the tensor-core kernels
// use: mbarriers with bounded waits, TMA tiled loads/stores (no multicast), TMEM
// allocation, tcgen05.mma with shared-memory descriptors, tcgen05.ld.
//
// Every wait in this file gives up after a clock budget and reports failure to the
// caller, which records an error code and unwinds (frees TMEM, returns) instead of
// spinning forever.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace la {
namespace ptx {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---- mbarrier ------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
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

// ---- proxy / tcgen05 fences -------------------------------------------------------------------
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after_sync() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}

// 2^x on the special-function unit (relative error 2^-22, denormal results flush to zero).
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ---- TMA (tiled, this CTA only; never multicast) ------------------------------------------------
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* m) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(m)) : "memory");
}
__device__ __forceinline__ void tma_load_3d(void* smem_dst, const CUtensorMap* m, uint64_t* bar, int c0,
                                            int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(c0), "r"(c1),
      "r"(c2)
      : "memory");
}
// The same for 4-D maps {feature, token, head, batch}.
__device__ __forceinline__ void tma_load_4d(void* smem_dst, const CUtensorMap* m, uint64_t* bar, int c0, int c1, int c2,
                                            int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2),
      "r"(c3)
      : "memory");
}
__device__ __forceinline__ void tma_prefetch_4d(const CUtensorMap* m, int c0, int c1, int c2, int c3) {
  asm volatile("cp.async.bulk.prefetch.tensor.4d.L2.global.tile [%0, {%1, %2, %3, %4}];" ::"l"(
                   reinterpret_cast<uint64_t>(m)),
               "r"(c0), "r"(c1), "r"(c2), "r"(c3)
               : "memory");
}
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* m, const void* smem_src, int c0, int c1, int c2, int c3) {
  asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];" ::"l"(
                   reinterpret_cast<uint64_t>(m)),
               "r"(smem_u32(smem_src)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
               : "memory");
}
// Brings a box into L2 only (no shared-memory destination, no barrier).
__device__ __forceinline__ void tma_prefetch_3d(const CUtensorMap* m, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(reinterpret_cast<uint64_t>(m)),
               "r"(c0), "r"(c1), "r"(c2)
               : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* m, const void* smem_src, int c0, int c1,
                                             int c2) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(
                   reinterpret_cast<uint64_t>(m)),
               "r"(smem_u32(smem_src)), "r"(c0), "r"(c1), "r"(c2)
               : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Waits until the smem sources of all committed bulk stores have been read.
__device__ __forceinline__ void tma_store_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// 32-byte store to global memory (one whole sector; address 32-byte aligned).
__device__ __forceinline__ void st_global_v8(void* gptr, const uint32_t* w) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(gptr), "r"(w[0]), "r"(w[1]), "r"(w[2]),
               "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
               : "memory");
}

// ---- TMEM ----------------------------------------------------------------------------------------
// One full warp allocates `ncols` (power of two >= 32) columns; the base address lands in *slot.
__device__ __forceinline__ void tmem_alloc(uint32_t* slot_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot_smem)),
               "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// ---- UMMA descriptors ------------------------------------------------------------------------------
// Shared-memory matrix descriptor, 128-byte swizzle, bf16.  Addresses/offsets in bytes.
//   K-major operand  (rows x K, K contiguous, 64 elements = one 128-byte row per panel):
//       sbo = distance between 8-row groups (1024 for a dense panel); lbo unused.
//   MN-major operand (K x MN, MN contiguous): lbo = distance between 64-element MN chunks,
//       sbo = distance between 8-row K groups (1024 for a dense panel).
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);        // bits [0,14)
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;   // bits [16,30)
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;   // bits [32,46)
  d |= (uint64_t)1 << 46;                              // descriptor version (sm_100)
  d |= (uint64_t)2 << 61;                              // layout type: 128-byte swizzle
  return d;
}
// The same descriptor as two 32-bit halves.  Only the low half depends on the address, and a
// byte offset `off` (multiple of 16) inside one buffer moves it by off >> 4 (shared-memory
// addresses stay below 2^18, so the 14-bit field cannot carry).
__device__ __forceinline__ uint32_t umma_desc_lo(uint32_t smem_addr, uint32_t lbo_bytes) {
  return ((smem_addr & 0x3FFFFu) >> 4) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
}
constexpr uint32_t UMMA_DESC_HI_SBO1024 = (1024u >> 4) | (1u << 14) | (2u << 29);  // sbo = 1024, version, 128-byte swizzle

// Instruction descriptor for kind::f16 with bf16 A/B and fp32 accumulation.
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int M, int N, bool a_mn_major, bool b_mn_major) {
  return (1u << 4)                       // D format: f32
         | (1u << 7)                     // A format: bf16
         | (1u << 10)                    // B format: bf16
         | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16) |
         ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// D[tmem] (+)= A[smem] * B[smem]; issued by one thread.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives on the mbarrier once all tcgen05.mma issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}

// ---- TMEM loads: 32 lanes x 32-bit, N consecutive columns per thread ------------------------------
__device__ __forceinline__ void tmem_ld_x16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---- TMEM stores: 32 lanes x 32-bit, 8 consecutive columns per thread ---------------------------
__device__ __forceinline__ void tmem_st_x8(uint32_t taddr, const uint32_t (&r)[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"r"(taddr),
               "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// D[tmem] (+)= A[tmem] * B[smem].  A is M x 16 bf16 for one instruction: row m in lane m, the 16
// elements packed two per 32-bit column (element 2c in the low half of column c) over 8 columns.
__device__ __forceinline__ void umma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// ---- warp-convergent issue -------------------------------------------------------------------------
// Used by the state-only kernel: the MMA-issuing warp runs its whole loop with all 32 lanes converged and
// only predicates the tcgen05 instructions themselves on one elected lane.  Measured on B200 in a
// micro-benchmark: issued from inside a divergent `if (lane == 0)` region, an MMA costs the issuing warp
// enough instruction slots that FMA-bound warps on the same scheduler stretch it from 48 to 122 clocks
// per instruction; issued convergently it stays at the tensor pipe's own 46 clocks.
__device__ __forceinline__ uint32_t elect_one() {
  uint32_t el;
  asm volatile("{\n\t.reg .pred q;\n\telect.sync _|q, 0xffffffff;\n\tselp.u32 %0, 1, 0, q;\n\t}" : "=r"(el));
  return el;
}
// D[tmem] (+)= A[smem] * B[smem] with descriptors as (low half, common high half); takes effect only
// in lanes with go != 0.
__device__ __forceinline__ void umma_bf16_lh(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi,
                                             uint32_t idesc, uint32_t accumulate, uint32_t go) {
  asm volatile(
      "{\n\t.reg .pred p, g;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 g, %6, 0;\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 da, {%1, %3};\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "@g tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}" ::"r"(d_tmem),
      "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate), "r"(go)
      : "memory");
}
// The same with the A operand read from tensor memory.
__device__ __forceinline__ void umma_bf16_ts_lh(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t desc_hi,
                                                uint32_t idesc, uint32_t accumulate, uint32_t go) {
  asm volatile(
      "{\n\t.reg .pred p, g;\n\t.reg .b64 db;\n\t"
      "setp.ne.b32 g, %6, 0;\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "@g tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate), "r"(go)
      : "memory");
}
// A whole K loop in one instruction sequence: NK tensor-core instructions D[tmem] (+)= A_k * B_k, k = 0..NK-1,
// all predicated on `go`, the first one accumulating only if `acc0`.  Operand k is operand 0 moved by a
// compile-time step: for shared-memory operands the low descriptor half advances by step(k) (16-byte units),
// AK / BK select the step pattern (true: K-major tile of two 64-element panels 16 KB apart, 32 bytes per K step
// inside a panel; false: MN-major tile, 2 KB per K step); for a tensor-memory A operand the column advances by
// 16 per K step.  One predicate set-up for the group instead of one per instruction keeps the issuing warp's
// instruction count per MMA at three.
template <bool K_MAJOR>
__host__ __device__ constexpr uint32_t umma_kstep(int k) {
  return K_MAJOR ? (uint32_t)((k >> 2) * 1024 + (k & 3) * 2) : (uint32_t)(k * 128);
}
#define LA_UMMA_SS_STEP(AI, BI)                                  \
  "add.u32 al, %1, " #AI ";\n\tmov.b64 da, {al, %3};\n\t"        \
  "add.u32 bl, %2, " #BI ";\n\tmov.b64 db, {bl, %3};\n\t"        \
  "@g tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, t;\n\t"
template <int NK, bool AK, bool BK>
__device__ __forceinline__ void umma_group_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi,
                                              uint32_t idesc, uint32_t acc0, uint32_t go) {
  static_assert(NK == 4 || NK == 8, "K steps per group");
  if (NK == 8) {
    asm volatile(
        "{\n\t.reg .pred p, g, t;\n\t.reg .b64 da, db;\n\t.reg .b32 al, bl;\n\t"
        "setp.ne.b32 g, %6, 0;\n\tsetp.ne.b32 p, %5, 0;\n\tsetp.eq.b32 t, 0, 0;\n\t"
        "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
        "@g tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t"
        LA_UMMA_SS_STEP(%7, %14) LA_UMMA_SS_STEP(%8, %15) LA_UMMA_SS_STEP(%9, %16) LA_UMMA_SS_STEP(%10, %17)
        LA_UMMA_SS_STEP(%11, %18) LA_UMMA_SS_STEP(%12, %19) LA_UMMA_SS_STEP(%13, %20)
        "}" ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(acc0), "r"(go),
        "n"(umma_kstep<AK>(1)), "n"(umma_kstep<AK>(2)), "n"(umma_kstep<AK>(3)), "n"(umma_kstep<AK>(4)),
        "n"(umma_kstep<AK>(5)), "n"(umma_kstep<AK>(6)), "n"(umma_kstep<AK>(7)),
        "n"(umma_kstep<BK>(1)), "n"(umma_kstep<BK>(2)), "n"(umma_kstep<BK>(3)), "n"(umma_kstep<BK>(4)),
        "n"(umma_kstep<BK>(5)), "n"(umma_kstep<BK>(6)), "n"(umma_kstep<BK>(7))
        : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p, g, t;\n\t.reg .b64 da, db;\n\t.reg .b32 al, bl;\n\t"
        "setp.ne.b32 g, %6, 0;\n\tsetp.ne.b32 p, %5, 0;\n\tsetp.eq.b32 t, 0, 0;\n\t"
        "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
        "@g tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t"
        LA_UMMA_SS_STEP(%7, %10) LA_UMMA_SS_STEP(%8, %11) LA_UMMA_SS_STEP(%9, %12)
        "}" ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(acc0), "r"(go),
        "n"(umma_kstep<AK>(1)), "n"(umma_kstep<AK>(2)), "n"(umma_kstep<AK>(3)),
        "n"(umma_kstep<BK>(1)), "n"(umma_kstep<BK>(2)), "n"(umma_kstep<BK>(3))
        : "memory");
  }
}
#undef LA_UMMA_SS_STEP
// Eight K steps with A in tensor memory (16 columns per step) and an MN-major B tile in shared memory.
#define LA_UMMA_TS_STEP(AI, BI)                                  \
  "add.u32 at, %1, " #AI ";\n\t"                                 \
  "add.u32 bl, %2, " #BI ";\n\tmov.b64 db, {bl, %3};\n\t"        \
  "@g tcgen05.mma.cta_group::1.kind::f16 [%0], [at], db, %4, t;\n\t"
__device__ __forceinline__ void umma_group_ts8(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t desc_hi,
                                               uint32_t idesc, uint32_t acc0, uint32_t go) {
  asm volatile(
      "{\n\t.reg .pred p, g, t;\n\t.reg .b64 db;\n\t.reg .b32 at, bl;\n\t"
      "setp.ne.b32 g, %6, 0;\n\tsetp.ne.b32 p, %5, 0;\n\tsetp.eq.b32 t, 0, 0;\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "@g tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t"
      LA_UMMA_TS_STEP(16, 128) LA_UMMA_TS_STEP(32, 256) LA_UMMA_TS_STEP(48, 384) LA_UMMA_TS_STEP(64, 512)
      LA_UMMA_TS_STEP(80, 640) LA_UMMA_TS_STEP(96, 768) LA_UMMA_TS_STEP(112, 896)
      "}" ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(acc0), "r"(go)
      : "memory");
}
#undef LA_UMMA_TS_STEP
__device__ __forceinline__ void umma_commit_if(uint64_t* bar, uint32_t go) {
  asm volatile(
      "{\n\t.reg .pred g;\n\tsetp.ne.b32 g, %1, 0;\n\t"
      "@g tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}" ::"r"(smem_u32(bar)),
      "r"(go)
      : "memory");
}

}  // namespace ptx
}  // namespace la
