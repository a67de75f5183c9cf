// Tensor-core kernels of the generic decayed linear-attention operator for
// bf16 inputs with Da = Ec = 128 (block formulas: la_common.cuh).
//
// One thread block walks the 128-token blocks of one (batch*head, segment,
// half of the value columns).  Per block it issues, on the 5th-generation
// tensor cores (tcgen05.mma, fp32 accumulators in tensor memory):
//   M1  S        = a b^T                          128x128, K = 128
//   M2  O_inter  = a Z_hi (+ a Z_lo)              128x64,  K = 128   (state of the previous block)
//   M3  dZ       = b^T fc_hi (+ b^T fc_lo)        128x64,  K = 128   (fc = diag(f_state) c)
//   M4  O_intra  = P_hi c (+ P_lo c)              128x64,  K = 128   (P = S (.) D)
// and combines out = O_intra + diag(f_out) O_inter, Z <- Gamma Z + dZ on the CUDA
// cores.  Operands that are formed on chip from fp32 values (P, fc, Z) are carried
// as two bf16 terms hi + lo = x (to 2^-17), so that the only rounding left is the
// fp32 accumulation the method prescribes; each split can be turned off.
//
// Warp roles (192 threads): warp 0 issues TMA loads, warp 1 owns tensor memory and
// issues every MMA from one lane, warps 2-5 (one per 32-lane quarter of tensor
// memory) turn accumulators into the next operands and into the output tile.  All
// hand-offs are mbarriers; every wait is bounded and an expired wait makes the
// whole block unwind (flag set, copies drained, tensor memory freed).
//
// Shared-memory operand layouts are the canonical 128-byte-swizzled ones: K-major
// tiles as two [128 rows][64 elements] panels (what a TMA box of 64x128 with
// CU_TENSOR_MAP_SWIZZLE_128B writes), MN-major tiles as [K rows][64 elements].
// The value-like tile c and the state operand are MN-major B operands, b is used
// K-major in M1 and MN-major (as b^T) in M3 from the same bytes.
#include <cuda.h>

#include <mutex>

#include "la_common.cuh"
#include "sm100_ptx.cuh"

namespace la {

__device__ unsigned int g_tc_status = 0;  // first non-zero failure code of any block (0 = none)

namespace {
using namespace ptx;

constexpr int TC_THREADS = 192;
constexpr int TMEM_COLS = 512;
constexpr uint32_t COL_S = 0, COL_OI = 128, COL_OE = 192, COL_DZ = 256;
constexpr long long WAIT_BUDGET = 2000000000LL;  // clocks (~1 s)

enum Bar {
  FULL_AB = 0, FULL_C, AB_FREE, C_FREE, S_READY, FC_READY, P_READY, DZ_READY, O_READY, Z_READY, O_FREE,
  STAGE_READY, STAGE_FREE, DRAIN, NUM_BARS
};

struct alignas(1024) TcSmem {
  __nv_bfloat16 a[2][128 * 64];
  __nv_bfloat16 b[2][128 * 64];
  __nv_bfloat16 c[128 * 64];
  __nv_bfloat16 p_hi[2][128 * 64];  // also the output staging tile
  __nv_bfloat16 p_lo[2][128 * 64];
  __nv_bfloat16 fc_hi[128 * 64];
  __nv_bfloat16 fc_lo[128 * 64];
  __nv_bfloat16 z_hi[128 * 64];
  __nv_bfloat16 z_lo[128 * 64];
  float dtab[128];
  uint64_t bars[NUM_BARS];
  uint32_t tmem_slot;
  int abort;
};

struct TcArgs {
  const float* entry;
  float* local_out;
  float* final_out;
  int BH, H, N, seg_len, nseg;
  int precision;
};

__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  unsigned spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 31u) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > WAIT_BUDGET) return false;
    }
  }
  return true;
}

// Used only while unwinding after a failure: waits (bounded) for work this thread started.
__device__ __forceinline__ void drain_wait(uint64_t* bar, uint32_t parity) {
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity) && clock64() - t0 < WAIT_BUDGET) {
  }
}

__device__ __forceinline__ void split2(float x0, float x1, uint32_t& hi, uint32_t& lo) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
  const float2 hf = __bfloat1622float2(h);
  const __nv_bfloat162 l = __floats2bfloat162_rn(x0 - hf.x, x1 - hf.y);
  hi = *reinterpret_cast<const uint32_t*>(&h);
  lo = *reinterpret_cast<const uint32_t*>(&l);
}

// Writes 8 consecutive fp32 values of row `row` (elements col8*8 .. col8*8+7 of a 64-element
// swizzled row) as bf16 hi (and lo) 16-byte chunks.
__device__ __forceinline__ void store_split8(__nv_bfloat16* hi_tile, __nv_bfloat16* lo_tile, int row, int col8,
                                             const float (&x)[8], bool want_lo) {
  uint4 h, l;
  split2(x[0], x[1], h.x, l.x);
  split2(x[2], x[3], h.y, l.y);
  split2(x[4], x[5], h.z, l.z);
  split2(x[6], x[7], h.w, l.w);
  const int off = row * 64 + ((col8 ^ (row & 7)) << 3);
  *reinterpret_cast<uint4*>(hi_tile + off) = h;
  if (want_lo) *reinterpret_cast<uint4*>(lo_tile + off) = l;
}

#define TC_WAIT(barid, par, code)                                        \
  do {                                                                   \
    if (!wait_or_abort(&sm.bars[barid], (par), &sm.abort)) {             \
      if (!sm.abort) atomicCAS(&g_tc_status, 0u, (unsigned)(code));      \
      sm.abort = 1;                                                      \
      goto teardown;                                                     \
    }                                                                    \
  } while (0)

template <bool REV, bool STATE_ONLY, typename TOut>
__global__ void __launch_bounds__(TC_THREADS, 1)
tc_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
          const __grid_constant__ CUtensorMap tm_c, const __grid_constant__ CUtensorMap tm_out,
          const TcArgs args, const DecayTable tab) {
  extern __shared__ unsigned char smem_raw[];
  TcSmem& sm = *reinterpret_cast<TcSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int ehalf = blockIdx.x & 1;
  const int segid = blockIdx.x >> 1;
  const int bh = segid / args.nseg, seg = segid % args.nseg;
  const int seg_t0 = seg * args.seg_len;
  const int seg_t1 = min(args.N, seg_t0 + args.seg_len);
  const int nblk = (seg_t1 - seg_t0 + 127) >> 7;
  const float s2 = (float)tab.s2[bh % args.H];
  const bool split_p = (args.precision & 1) != 0;
  const bool split_z = (args.precision & 2) != 0;
  const bool split_c = (args.precision & 4) != 0;

  if (tid == 0) {
    mbar_init(&sm.bars[FULL_AB], 1);
    mbar_init(&sm.bars[FULL_C], 1);
    mbar_init(&sm.bars[AB_FREE], 1);
    mbar_init(&sm.bars[C_FREE], 1);
    mbar_init(&sm.bars[S_READY], 1);
    mbar_init(&sm.bars[FC_READY], 128);
    mbar_init(&sm.bars[P_READY], 128);
    mbar_init(&sm.bars[DZ_READY], 1);
    mbar_init(&sm.bars[O_READY], 1);
    mbar_init(&sm.bars[Z_READY], 128);
    mbar_init(&sm.bars[O_FREE], 128);
    mbar_init(&sm.bars[STAGE_READY], 128);
    mbar_init(&sm.bars[STAGE_FREE], 1);
    mbar_init(&sm.bars[DRAIN], 1);
    sm.abort = 0;
    fence_mbar_init();
    tma_prefetch_desc(&tm_a);
    tma_prefetch_desc(&tm_b);
    tma_prefetch_desc(&tm_c);
    tma_prefetch_desc(&tm_out);
  }
  if (warp == 1) {
    tmem_alloc(&sm.tmem_slot, TMEM_COLS);
    tmem_relinquish();
  }
  if (tid >= 64) sm.dtab[tid - 64] = exp2f(-s2 * (float)(tid - 64));
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = sm.tmem_slot;
  bool issued_mma = false;
  int ab_armed = 0, c_armed = 0;  // producer: block iterations whose a/b and c loads were issued

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      for (int it = 0; it < nblk; ++it) {
        const int blk = REV ? (nblk - 1 - it) : it;
        const int t0 = seg_t0 + blk * 128;
        if (it > 0) TC_WAIT(AB_FREE, (it - 1) & 1, 1);
        if (!STATE_ONLY) {
          mbar_arrive_expect_tx(&sm.bars[FULL_AB], 65536);
          tma_load_3d(&sm.a[0][0], &tm_a, &sm.bars[FULL_AB], 0, t0, bh);
          tma_load_3d(&sm.a[1][0], &tm_a, &sm.bars[FULL_AB], 64, t0, bh);
        } else {
          mbar_arrive_expect_tx(&sm.bars[FULL_AB], 32768);
        }
        tma_load_3d(&sm.b[0][0], &tm_b, &sm.bars[FULL_AB], 0, t0, bh);
        tma_load_3d(&sm.b[1][0], &tm_b, &sm.bars[FULL_AB], 64, t0, bh);
        ab_armed = it + 1;
        if (it > 0) TC_WAIT(C_FREE, (it - 1) & 1, 2);
        mbar_arrive_expect_tx(&sm.bars[FULL_C], 16384);
        tma_load_3d(&sm.c[0], &tm_c, &sm.bars[FULL_C], ehalf * 64, t0, bh);
        c_armed = it + 1;
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0) {
      const uint32_t a0 = smem_u32(&sm.a[0][0]), b0 = smem_u32(&sm.b[0][0]), c0 = smem_u32(&sm.c[0]);
      const uint32_t ph0 = smem_u32(&sm.p_hi[0][0]), pl0 = smem_u32(&sm.p_lo[0][0]);
      const uint32_t fh0 = smem_u32(&sm.fc_hi[0]), fl0 = smem_u32(&sm.fc_lo[0]);
      const uint32_t zh0 = smem_u32(&sm.z_hi[0]), zl0 = smem_u32(&sm.z_lo[0]);
      constexpr uint32_t ID_S = umma_idesc_bf16(128, 128, false, false);  // a (K-major) x b (K-major)
      constexpr uint32_t ID_KN = umma_idesc_bf16(128, 64, false, true);   // K-major A x MN-major B
      constexpr uint32_t ID_MN = umma_idesc_bf16(128, 64, true, true);    // MN-major A (b^T) x MN-major B
      for (int it = 0; it < nblk; ++it) {
        const uint32_t par = it & 1;
        TC_WAIT(FULL_AB, par, 3);
        tc_fence_after_sync();
        if (!STATE_ONLY) {
          // M1: S = a b^T
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const uint32_t ko = (k >> 2) * 16384 + (k & 3) * 32;
            umma_bf16(tmem + COL_S, umma_desc_sw128(a0 + ko, 16, 1024), umma_desc_sw128(b0 + ko, 16, 1024), ID_S,
                      k > 0);
          }
          issued_mma = true;
          umma_commit(&sm.bars[S_READY]);
          // M2: O_inter = a Z   (state operand of the previous block / the entry state)
          TC_WAIT(Z_READY, par, 4);
          if (it > 0) TC_WAIT(O_FREE, (it - 1) & 1, 5);
          tc_fence_after_sync();
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const uint32_t ko = (k >> 2) * 16384 + (k & 3) * 32;
            umma_bf16(tmem + COL_OE, umma_desc_sw128(a0 + ko, 16, 1024),
                      umma_desc_sw128(zh0 + k * 2048, 16384, 1024), ID_KN, k > 0);
          }
          if (split_z) {
#pragma unroll
            for (int k = 0; k < 8; ++k) {
              const uint32_t ko = (k >> 2) * 16384 + (k & 3) * 32;
              umma_bf16(tmem + COL_OE, umma_desc_sw128(a0 + ko, 16, 1024),
                        umma_desc_sw128(zl0 + k * 2048, 16384, 1024), ID_KN, 1);
            }
          }
        }
        // M3: dZ = b^T fc
        TC_WAIT(FC_READY, par, 6);
        tc_fence_after_sync();
#pragma unroll
        for (int k = 0; k < 8; ++k)
          umma_bf16(tmem + COL_DZ, umma_desc_sw128(b0 + k * 2048, 16384, 1024),
                    umma_desc_sw128(fh0 + k * 2048, 16384, 1024), ID_MN, STATE_ONLY ? (it > 0 || k > 0) : (k > 0));
        if (split_c) {
#pragma unroll
          for (int k = 0; k < 8; ++k)
            umma_bf16(tmem + COL_DZ, umma_desc_sw128(b0 + k * 2048, 16384, 1024),
                      umma_desc_sw128(fl0 + k * 2048, 16384, 1024), ID_MN, 1);
        }
        issued_mma = true;
        umma_commit(&sm.bars[DZ_READY]);
        umma_commit(&sm.bars[AB_FREE]);
        if (STATE_ONLY) {
          umma_commit(&sm.bars[C_FREE]);
          continue;
        }
        // M4: O_intra = P c
        TC_WAIT(P_READY, par, 7);
        TC_WAIT(FULL_C, par, 8);
        tc_fence_after_sync();
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const uint32_t ko = (k >> 2) * 16384 + (k & 3) * 32;
          umma_bf16(tmem + COL_OI, umma_desc_sw128(ph0 + ko, 16, 1024), umma_desc_sw128(c0 + k * 2048, 16384, 1024),
                    ID_KN, k > 0);
        }
        if (split_p) {
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const uint32_t ko = (k >> 2) * 16384 + (k & 3) * 32;
            umma_bf16(tmem + COL_OI, umma_desc_sw128(pl0 + ko, 16, 1024),
                      umma_desc_sw128(c0 + k * 2048, 16384, 1024), ID_KN, 1);
          }
        }
        umma_commit(&sm.bars[O_READY]);
        umma_commit(&sm.bars[C_FREE]);
      }
    }
  } else {
    // ------------------------------ transform / epilogue warps ------------------------------
    const int q = warp & 3;          // quarter of tensor memory this warp may read
    const int r = q * 32 + lane;     // row owned by this thread: token i / token j / state row k
    const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
    float zreg[64];
    if (!STATE_ONLY) {
      if (args.entry) {
        const float4* src = reinterpret_cast<const float4*>(
            args.entry + ((size_t)bh * args.nseg + seg) * (128 * 128) + (size_t)r * 128 + ehalf * 64);
#pragma unroll
        for (int x = 0; x < 16; ++x) {
          const float4 v = __ldg(src + x);
          zreg[4 * x] = v.x; zreg[4 * x + 1] = v.y; zreg[4 * x + 2] = v.z; zreg[4 * x + 3] = v.w;
        }
      } else {
#pragma unroll
        for (int x = 0; x < 64; ++x) zreg[x] = 0.f;
      }
#pragma unroll
      for (int c8 = 0; c8 < 8; ++c8) {
        float x8[8];
#pragma unroll
        for (int x = 0; x < 8; ++x) x8[x] = zreg[c8 * 8 + x];
        store_split8(sm.z_hi, sm.z_lo, r, c8, x8, split_z);
      }
      fence_proxy_async_smem();
      mbar_arrive(&sm.bars[Z_READY]);
    }

    for (int it = 0; it < nblk; ++it) {
      const uint32_t par = it & 1;
      const int blk = REV ? (nblk - 1 - it) : it;
      const int t0 = seg_t0 + blk * 128;
      const int Cr = min(128, seg_t1 - t0);

      // ---- X1: fc = diag(f_state) c, as hi/lo bf16 ----
      TC_WAIT(FULL_C, par, 9);
      if (STATE_ONLY && it > 0) TC_WAIT(DZ_READY, (it - 1) & 1, 10);  // previous M3 has read fc
      {
        float f = 0.f;
        if (r < Cr) {
          if (STATE_ONLY) f = REV ? exp2f(-s2 * (float)(t0 + r - seg_t0 + 1)) : exp2f(-s2 * (float)(seg_t1 - 1 - t0 - r));
          else f = REV ? exp2f(-s2 * (float)(r + 1)) : exp2f(-s2 * (float)(Cr - 1 - r));
        }
#pragma unroll
        for (int c8 = 0; c8 < 8; ++c8) {
          const int off = r * 64 + ((c8 ^ (r & 7)) << 3);
          const uint4 raw = *reinterpret_cast<const uint4*>(&sm.c[off]);
          const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
          float x8[8];
#pragma unroll
          for (int x = 0; x < 4; ++x) {
            const float2 v = __bfloat1622float2(h2[x]);
            x8[2 * x] = v.x * f;
            x8[2 * x + 1] = v.y * f;
          }
          store_split8(sm.fc_hi, sm.fc_lo, r, c8, x8, split_c);
        }
        fence_proxy_async_smem();
        mbar_arrive(&sm.bars[FC_READY]);
      }
      if (STATE_ONLY) continue;

      // ---- X2: P = S (.) D as hi/lo bf16 (row i = r) ----
      TC_WAIT(S_READY, par, 11);
      if (it > 0) TC_WAIT(STAGE_FREE, (it - 1) & 1, 12);  // staging tile aliases p_hi
      tc_fence_after_sync();
#pragma unroll 1
      for (int cc = 0; cc < 4; ++cc) {
        const bool all_masked = REV ? (cc < q) : (cc > q);  // whole 32x32 sub-tile is outside the causal band
        uint32_t sreg[32];
        if (!all_masked) {
          tmem_ld_x32(lane_addr + COL_S + cc * 32, sreg);
          tmem_ld_wait();
        }
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          float x8[8];
#pragma unroll
          for (int x = 0; x < 8; ++x) {
            const int j = cc * 32 + g * 8 + x;
            const int n = REV ? (j - r) : (r - j);
            float p = 0.f;
            if (!all_masked && n >= 0) p = __uint_as_float(sreg[g * 8 + x]) * sm.dtab[n];
            x8[x] = p;
          }
          store_split8(&sm.p_hi[cc >> 1][0], &sm.p_lo[cc >> 1][0], r, (cc & 1) * 4 + g, x8, split_p);
        }
      }
      tc_fence_before_sync();
      fence_proxy_async_smem();
      mbar_arrive(&sm.bars[P_READY]);

      // ---- X3: Z <- Gamma Z + dZ (row k = r), new state operand ----
      TC_WAIT(DZ_READY, par, 13);
      tc_fence_after_sync();
      {
        const float gamma = exp2f(-s2 * (float)Cr);
#pragma unroll
        for (int hcol = 0; hcol < 2; ++hcol) {
          uint32_t dz[32];
          tmem_ld_x32(lane_addr + COL_DZ + hcol * 32, dz);
          tmem_ld_wait();
#pragma unroll
          for (int x = 0; x < 32; ++x) zreg[hcol * 32 + x] = fmaf(gamma, zreg[hcol * 32 + x], __uint_as_float(dz[x]));
        }
        if (it + 1 < nblk) {
#pragma unroll
          for (int c8 = 0; c8 < 8; ++c8) {
            float x8[8];
#pragma unroll
            for (int x = 0; x < 8; ++x) x8[x] = zreg[c8 * 8 + x];
            store_split8(sm.z_hi, sm.z_lo, r, c8, x8, split_z);
          }
        }
        tc_fence_before_sync();
        fence_proxy_async_smem();
        mbar_arrive(&sm.bars[Z_READY]);
      }

      // ---- X4: out = O_intra + diag(f_out) O_inter (row i = r) ----
      TC_WAIT(O_READY, par, 14);
      tc_fence_after_sync();
      {
        float f = 0.f;
        if (r < Cr) f = REV ? exp2f(-s2 * (float)(Cr - 1 - r)) : exp2f(-s2 * (float)(r + 1));
        unsigned char* stage = reinterpret_cast<unsigned char*>(&sm.p_hi[0][0]);
#pragma unroll
        for (int hcol = 0; hcol < 2; ++hcol) {
          uint32_t oi[32], oe[32];
          tmem_ld_x32(lane_addr + COL_OI + hcol * 32, oi);
          tmem_ld_x32(lane_addr + COL_OE + hcol * 32, oe);
          tmem_ld_wait();
          if (hcol == 1) {
            tc_fence_before_sync();
            mbar_arrive(&sm.bars[O_FREE]);  // both accumulators are in registers now
          }
          if (sizeof(TOut) == 4) {
            // fp32 staging: panel hcol = [128 rows][32 floats], 16-byte chunks swizzled by row
#pragma unroll
            for (int c4 = 0; c4 < 8; ++c4) {
              float4 v;
              v.x = fmaf(f, __uint_as_float(oe[4 * c4 + 0]), __uint_as_float(oi[4 * c4 + 0]));
              v.y = fmaf(f, __uint_as_float(oe[4 * c4 + 1]), __uint_as_float(oi[4 * c4 + 1]));
              v.z = fmaf(f, __uint_as_float(oe[4 * c4 + 2]), __uint_as_float(oi[4 * c4 + 2]));
              v.w = fmaf(f, __uint_as_float(oe[4 * c4 + 3]), __uint_as_float(oi[4 * c4 + 3]));
              *reinterpret_cast<float4*>(stage + hcol * 16384 + r * 128 + ((c4 ^ (r & 7)) << 4)) = v;
            }
          } else {
            // bf16 staging: one panel [128 rows][64 bf16]
#pragma unroll
            for (int c8 = 0; c8 < 4; ++c8) {
              uint4 v;
              uint32_t* vw = reinterpret_cast<uint32_t*>(&v);
#pragma unroll
              for (int x = 0; x < 4; ++x) {
                const float y0 = fmaf(f, __uint_as_float(oe[8 * c8 + 2 * x]), __uint_as_float(oi[8 * c8 + 2 * x]));
                const float y1 = fmaf(f, __uint_as_float(oe[8 * c8 + 2 * x + 1]), __uint_as_float(oi[8 * c8 + 2 * x + 1]));
                const __nv_bfloat162 h = __floats2bfloat162_rn(y0, y1);
                vw[x] = *reinterpret_cast<const uint32_t*>(&h);
              }
              const int chunk = hcol * 4 + c8;
              *reinterpret_cast<uint4*>(stage + r * 128 + ((chunk ^ (r & 7)) << 4)) = v;
            }
          }
        }
        fence_proxy_async_smem();
        mbar_arrive(&sm.bars[STAGE_READY]);
        if (tid == 64) {
          TC_WAIT(STAGE_READY, par, 15);
          if (sizeof(TOut) == 4) {
            tma_store_3d(&tm_out, stage, ehalf * 64, t0, bh);
            tma_store_3d(&tm_out, stage + 16384, ehalf * 64 + 32, t0, bh);
          } else {
            tma_store_3d(&tm_out, stage, ehalf * 64, t0, bh);
          }
          tma_store_commit();
          tma_store_wait_read();
          mbar_arrive(&sm.bars[STAGE_FREE]);
        }
      }
    }

    if (STATE_ONLY) {
      // segment-local state = accumulated dZ
      TC_WAIT(DZ_READY, (nblk - 1) & 1, 16);
      tc_fence_after_sync();
      float* dst = args.local_out + ((size_t)bh * args.nseg + seg) * (128 * 128) + (size_t)r * 128 + ehalf * 64;
#pragma unroll
      for (int hcol = 0; hcol < 2; ++hcol) {
        uint32_t dz[32];
        tmem_ld_x32(lane_addr + COL_DZ + hcol * 32, dz);
        tmem_ld_wait();
#pragma unroll
        for (int x = 0; x < 8; ++x)
          *reinterpret_cast<float4*>(dst + hcol * 32 + 4 * x) =
              make_float4(__uint_as_float(dz[4 * x]), __uint_as_float(dz[4 * x + 1]), __uint_as_float(dz[4 * x + 2]),
                          __uint_as_float(dz[4 * x + 3]));
      }
      tc_fence_before_sync();
    } else {
      const bool last_processed = REV ? (seg == 0) : (seg == args.nseg - 1);
      if (args.final_out && last_processed) {
        float* dst = args.final_out + (size_t)bh * (128 * 128) + (size_t)r * 128 + ehalf * 64;
#pragma unroll
        for (int x = 0; x < 16; ++x)
          *reinterpret_cast<float4*>(dst + 4 * x) = make_float4(zreg[4 * x], zreg[4 * x + 1], zreg[4 * x + 2], zreg[4 * x + 3]);
      }
      if (tid == 64) tma_store_wait_all();
    }
  }

teardown:
  // After an expired wait: drain what this thread started so nothing is in flight when the
  // block exits (loads into shared memory, tensor-core work on tensor memory, bulk stores).
  if (sm.abort) {
    if (warp == 0 && lane == 0) {
      if (ab_armed > 0) drain_wait(&sm.bars[FULL_AB], (ab_armed - 1) & 1);
      if (c_armed > 0) drain_wait(&sm.bars[FULL_C], (c_armed - 1) & 1);
    }
    if (warp == 1 && lane == 0 && issued_mma) {
      umma_commit(&sm.bars[DRAIN]);
      drain_wait(&sm.bars[DRAIN], 0);
    }
    if (tid == 64) tma_store_wait_all();
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, TMEM_COLS);
}

// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess) return nullptr;
    if (q != cudaDriverEntryPointSuccess) return nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// Tensor map over a [BH, N, 128] tensor (feature dimension innermost) with a box of
// box_inner x 128 rows x 1, 128-byte swizzle; out-of-range rows read as zero / are not written.
bool make_map(CUtensorMap* m, const void* ptr, bool is_f32, int N, int BH, int box_inner) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return false;
  const cuuint64_t esz = is_f32 ? 4 : 2;
  cuuint64_t dims[3] = {128, (cuuint64_t)N, (cuuint64_t)BH};
  cuuint64_t strides[2] = {128 * esz, (cuuint64_t)N * 128 * esz};
  cuuint32_t box[3] = {(cuuint32_t)box_inner, 128, 1};
  cuuint32_t es[3] = {1, 1, 1};
  return enc(m, is_f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3,
             const_cast<void*>(ptr), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <bool REV, bool STATE_ONLY, typename TOut>
cudaError_t launch_t(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc, const CUtensorMap& mo,
                     const TcArgs& ta, const DecayTable& tab, cudaStream_t stream) {
  const size_t smem = sizeof(TcSmem) + 1024;
  auto kern = tc_kernel<REV, STATE_ONLY, TOut>;
  cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (err != cudaSuccess) return err;
  KernelTimer timer(STATE_ONLY ? K_PREPASS : K_WALK, stream);
  kern<<<(unsigned)(ta.BH * ta.nseg * 2), TC_THREADS, smem, stream>>>(ma, mb, mc, mo, ta, tab);
  count_launch();
  return cudaGetLastError();
}

}  // namespace

bool tc_supported() { return encode_fn() != nullptr; }

cudaError_t launch_tc_walk(const OpArgs& args, const DecayTable& tab, int out_dt, int precision,
                           cudaStream_t stream) {
  CUtensorMap ma, mb, mc, mo;
  const bool f32 = (out_dt == DT_F32);
  if (!make_map(&ma, args.a, false, args.N, args.BH, 64) || !make_map(&mb, args.b, false, args.N, args.BH, 64) ||
      !make_map(&mc, args.c, false, args.N, args.BH, 64) ||
      !make_map(&mo, args.out, f32, args.N, args.BH, f32 ? 32 : 64))
    return cudaErrorInvalidValue;
  TcArgs ta{args.entry, nullptr, args.final_out, args.BH, args.H, args.N, args.seg_len, args.nseg, precision};
  if (args.reverse)
    return f32 ? launch_t<true, false, float>(ma, mb, mc, mo, ta, tab, stream)
               : launch_t<true, false, __nv_bfloat16>(ma, mb, mc, mo, ta, tab, stream);
  return f32 ? launch_t<false, false, float>(ma, mb, mc, mo, ta, tab, stream)
             : launch_t<false, false, __nv_bfloat16>(ma, mb, mc, mo, ta, tab, stream);
}

cudaError_t launch_tc_prepass(const OpArgs& args, const DecayTable& tab, int precision, cudaStream_t stream) {
  CUtensorMap mb, mc;
  if (!make_map(&mb, args.b, false, args.N, args.BH, 64) || !make_map(&mc, args.c, false, args.N, args.BH, 64))
    return cudaErrorInvalidValue;
  TcArgs ta{nullptr, args.local_out, nullptr, args.BH, args.H, args.N, args.seg_len, args.nseg, precision};
  // the a / out maps are unused by the state-only kernel; pass valid descriptors anyway
  return args.reverse ? launch_t<true, true, float>(mb, mb, mc, mc, ta, tab, stream)
                      : launch_t<false, true, float>(mb, mb, mc, mc, ta, tab, stream);
}

unsigned int tc_read_status(bool clear) {
  unsigned int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_tc_status, sizeof(v)) != cudaSuccess) return 0xFFFFFFFFu;
  if (clear && v != 0) {
    const unsigned int zero = 0;
    cudaMemcpyToSymbol(g_tc_status, &zero, sizeof(zero));
  }
  return v;
}

}  // namespace la
