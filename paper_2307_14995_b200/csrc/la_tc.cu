// Tensor-core kernels of the generic decayed linear-attention operator for
// bf16 inputs with Da = Ec = D, D = 128 or 64 (block formulas: la_common.cuh).  Two kernels share this file's
// launchers: the half-width kernel below (every D = 64 launch, the state-only pre-pass at both head sizes, and the
// D = 128 walk when an output is aligned to 16 but not 32 bytes) and the full-width walk of la_tc_full.cuh
// (D = 128: one thread block per (batch*head, segment) with all four 128x128 accumulators in tensor memory),
// which launch_walk_d prefers.  The text below describes the half-width kernel at D = 128; the differences at
// D = 64 are described at the kernel's template parameter.
//
// One thread block walks the 128-token blocks of one (batch*head, segment,
// half of the value columns).  Per block it issues, on the 5th-generation
// tensor cores (tcgen05.mma, fp32 accumulators in tensor memory):
//   M1  S        = a b^T                          128x128, K = 128
//   M2  O_inter  = a Z_hi (+ a Z_lo)              128x64,  K = 128   (state of the previous block)
//   M3  dZ       = b^T fc_hi (+ b^T fc_lo)        128x64,  K = 128   (fc = diag(f_state) c; the state-only
//                                                                      pre-pass uses one N = 128 product)
//   M4  O_intra  = P_hi c (+ P_lo c)              128x64,  K = 128   (P = S (.) D, read from tensor memory)
// and combines out = O_intra + diag(f_out) O_inter, Z <- Gamma Z + dZ on the CUDA
// cores.  Operands that are formed on chip from fp32 values (P, fc, Z) are carried
// as two bf16 terms hi + lo = x (to 2^-17), so that the only rounding left is the
// fp32 accumulation the method prescribes; each split can be turned off.
//
// Tensor memory (512 columns) is full: 2 x 128 (S/P, double-buffered) + 64 (O_intra) +
// 2 x 64 (O_inter, double-buffered so that M2 of the next block need not wait until the
// output group has read this block's accumulators) + 64 (dZ).  (Measured on B200: one
// tcgen05.mma of M = 128, K = 16 occupies the tensor pipe for about 64 clocks whether N is
// 64 or 128, so the N = 64 products run at half the pipe's rate; wider tiles do not fit.)
//
// Warp roles (24 warps; every group has whole multiples of four warps because a warp
// can only touch the 32-lane quarter of tensor memory given by its index mod 4):
//   warp 0       TMA producer: a, b, c tiles into a 2-stage shared-memory ring
//   warp 1       owns tensor memory and issues every MMA: the whole warp stays converged through the waits and
//                one elected lane issues each group of eight K-steps (a lone lane looping over the products
//                was measurably slower: its barrier polls and descriptor arithmetic did not overlap)
//   warps 4-11   "P" group (two warps per quarter, two 32-column chunks each): S (fp32) ->
//                masked, decayed P as packed bf16 hi/lo, written back over S in tensor
//                memory, where M4 reads it as its A operand
//   warps 12-19  "Z" group (two warps per quarter, 32 state columns each): owns the fp32 state
//                in registers (Z <- Gamma Z + dZ), rewrites the bf16 state operand, and forms
//                fc = diag(f_state) c of the next block
//   warps 20-23  "O" group: out = O_intra + diag(f_out) O_inter; 128 bytes of every output row are
//                staged in the dead c tile and leave through bulk tensor stores
// In the state-only pre-pass warps 4-19 all form fc, and the MMA warp issues converged.
// All hand-offs are mbarriers; every wait is bounded and an expired wait makes the whole
// block unwind (flag set, copies drained, tensor memory freed).  Barrier operations on the MMA
// warp are kept few, since each costs it a few hundred clocks (measured): per block it
// waits for Z_READY (state operand and fc, both written by the Z group), FULL_B of the next block
// (a and b tiles travel together), P_READY (P written AND the previous block's accumulators read
// by the output group: 8 + 4 arrivals) and FULL_C, and commits to DZ_READY, A_FREE (which the
// producer and the Z group both wait for), S_READY and O_READY.
//
// The only chain that is sequential across blocks is dZ -> Z -> O_inter; S, P and fc of
// block n+1 do not depend on block n.  The MMA warp therefore issues, per block n:
// M3(n), M2(n), M1(n+1), M4(n): the state chain first (it never waits for a load), then the
// next score tile so that the P group always has work, then the product that needs P.
//
// Shared-memory operand layouts are the canonical 128-byte-swizzled ones: K-major
// tiles as two [128 rows][64 elements] panels (what a TMA box of 64x128 with
// CU_TENSOR_MAP_SWIZZLE_128B writes), MN-major tiles as [K rows][64 elements].
// The value-like tile c and the state operand are MN-major B operands, b is used
// K-major in M1 and MN-major (as b^T) in M3 from the same bytes.
#include <cuda.h>

#include "la_common.cuh"
#include "sm100_ptx.cuh"

namespace la {

__device__ unsigned int g_tc_status = 0;       // first non-zero failure code of any block (0 = none)
__device__ unsigned int g_tc_status_read = 0;  // where status_exchange_kernel leaves the value it took

namespace {
using namespace ptx;

constexpr int TC_THREADS = 768;
constexpr int TMEM_COLS = 512;
// tensor-memory columns: two S/P buffers, O_intra, two O_inter buffers, dZ
constexpr uint32_t COL_S0 = 0, COL_S1 = 128, COL_OI = 256, COL_OE0 = 320, COL_OE1 = 384, COL_DZ = 448;
constexpr long long WAIT_BUDGET = 2000000000LL;  // clocks (~1 s)

enum Bar {
  FULL_B0 = 0, FULL_B1, FULL_B2, FULL_C0, FULL_C1, FULL_C2,   // TMA -> consumers (FULL_B: b, and a in the walk kernel)
  A_FREE0, A_FREE1, B_FREE0, B_FREE1, B_FREE2, C_FREE0, C_FREE1, C_FREE2,  // consumers -> TMA (third stage: state-only kernel)
  S_READY0, S_READY1, P_READY0, P_READY1,
  FC_READY0, FC_READY1, FC_FREE0, FC_FREE1,                   // (second buffer: state-only kernel)
  DZ_READY, Z_READY, O_READY, OG_SYNC, DRAIN,
  NUM_BARS
};

struct Stage {
  __nv_bfloat16 a[2][128 * 64];  // query-like tile (two K panels)
  __nv_bfloat16 b[2][128 * 64];  // key-like tile
  __nv_bfloat16 c[128 * 64];     // this block's 64 value columns; afterwards the output scratch
};

struct alignas(1024) TcSmem {
  Stage st[2];
  __nv_bfloat16 fc_hi[128 * 64];  // fc_hi and fc_lo are adjacent: one MN-major B operand with N = 128
  __nv_bfloat16 fc_lo[128 * 64];
  __nv_bfloat16 z_hi[128 * 64];   // state operand; in the state-only kernel: second fc buffer
  __nv_bfloat16 z_lo[128 * 64];
  uint64_t bars[NUM_BARS];
  uint32_t tmem_slot;
  int abort;
};

// One launch carries one job, or two jobs that walk the same tokens in the same direction (the dV and dK walks of
// the backward pass: they read the same four tensors, so the second read of each tile is an L2 hit).
struct TcJob {
  const void* c;  // value-like tensor, also read row-wise straight from global memory by the Z group
  void* out;
  const float* entry;
  float* final_out;
  // gate epilogue of the forward walk (full-width kernel only): y = SRMSNorm(out) (.) u
  const void* u;
  void* y;
  float* rstd;
};

struct TcMaps {
  CUtensorMap a, b, c, out;
};

struct TcArgs {
  TcJob job[2];
  float* local_out;
  const int* seq_start;  // packed batch (see OpArgs): DEVICE arrays, or NULL
  const int* seq_len;
  const int* seq_order;
  int njobs;
  int BH, H, N, seg_len, nseg;
  int precision;
  long long sT, sH, sB;  // element offset of token t of (b,h): b*sB + h*sH + t*sT (rows of D contiguous features)
};

__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                              long long budget = WAIT_BUDGET) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  // each try blocks in hardware for the default time limit (it returns early when the phase completes);
  // measured: giving a suspend-time hint of 1, 20 or 200 us instead makes the walk kernel 4 % slower
  while (!mbar_try_wait(bar, parity)) {
    if (*abort_flag) return false;
    if (clock64() - t0 > budget) return false;
  }
  return true;
}

// Used only while unwinding after a failure: waits (bounded) for work this thread started.
__device__ __forceinline__ void drain_wait(uint64_t* bar, uint32_t parity) {
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity) && clock64() - t0 < WAIT_BUDGET) {
  }
}

// x[0..15] -> packed bf16 pairs hi[0..7] and lo[0..7] with hi + lo = x to 2^-17.  Written as
// separate passes so that the 8 conversion chains are independent in program order.
__device__ __forceinline__ void split16(const float (&x)[16], uint32_t (&hi)[8], uint32_t (&lo)[8]) {
  __nv_bfloat162 h[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) h[i] = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);
  float r[16];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float2 hf = __bfloat1622float2(h[i]);
    r[2 * i] = x[2 * i] - hf.x;
    r[2 * i + 1] = x[2 * i + 1] - hf.y;
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const __nv_bfloat162 l = __floats2bfloat162_rn(r[2 * i], r[2 * i + 1]);
    hi[i] = *reinterpret_cast<const uint32_t*>(&h[i]);
    lo[i] = *reinterpret_cast<const uint32_t*>(&l);
  }
}

// Eight-element variant (fewer live registers; used where a thread also carries state rows).
__device__ __forceinline__ void split8(const float (&x)[8], uint4& hi, uint4& lo) {
  __nv_bfloat162 h[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);
  float r[8];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 hf = __bfloat1622float2(h[i]);
    r[2 * i] = x[2 * i] - hf.x;
    r[2 * i + 1] = x[2 * i + 1] - hf.y;
  }
  uint32_t hw[4], lw[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const __nv_bfloat162 l = __floats2bfloat162_rn(r[2 * i], r[2 * i + 1]);
    hw[i] = *reinterpret_cast<const uint32_t*>(&h[i]);
    lw[i] = *reinterpret_cast<const uint32_t*>(&l);
  }
  hi = make_uint4(hw[0], hw[1], hw[2], hw[3]);
  lo = make_uint4(lw[0], lw[1], lw[2], lw[3]);
}

#define TC_WAIT(barid, par, code)                                        \
  do {                                                                   \
    if (!wait_or_abort(&sm.bars[barid], (par), &sm.abort)) {             \
      if (!sm.abort) atomicCAS(&g_tc_status, 0u, (unsigned)(code));      \
      sm.abort = 1;                                                      \
      goto teardown;                                                     \
    }                                                                    \
  } while (0)

// The same for a whole warp waiting together: the outcome is made warp-uniform so that the
// warp-level synchronisation of the elected arrivals below can never be entered by a part of a warp.
#define TC_WAIT_WARP(barid, par, code)                                                    \
  do {                                                                                    \
    const bool ok_ = wait_or_abort(&sm.bars[barid], (par), &sm.abort);                    \
    if (!__all_sync(0xffffffffu, ok_)) {                                                  \
      if (!ok_ && !sm.abort) atomicCAS(&g_tc_status, 0u, (unsigned)(code));               \
      sm.abort = 1;                                                                       \
      goto teardown;                                                                      \
    }                                                                                     \
  } while (0)

// One arrival per warp: every lane has fenced its own writes, the warp synchronises, lane 0
// arrives.  (A barrier that 256 threads arrive on costs 256 serialised shared-memory atomics per
// phase; at six such barriers per block that was a third of the kernel's shared-memory traffic.)
#define WARP_ARRIVE(barid)                               \
  do {                                                   \
    __syncwarp();                                        \
    if (lane == 0) mbar_arrive(&sm.bars[barid]);         \
  } while (0)

template <bool REV, bool STATE_ONLY, typename TOut, int D, int NJOBS>
__global__ void __launch_bounds__(TC_THREADS, 1)
tc_kernel(const __grid_constant__ TcMaps maps0, const __grid_constant__ TcMaps maps1, const TcArgs args,
          const DecayTable tab) {
  extern __shared__ unsigned char smem_raw[];
  // 1024-byte alignment by pointer arithmetic on the shared array itself, so that the compiler keeps
  // the shared address space (ld.shared / st.shared rather than generic accesses)
  TcSmem& sm = *reinterpret_cast<TcSmem*>(smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u));

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // D = 128: two thread blocks per (head, segment), one per half of the value columns.  D = 64: one
  // thread block; the feature halves 64..127 of the a and b tiles do not exist (the K steps over them are
  // skipped, and the second b panel, which M3 reads as rows 64..127 of b^T, is zeroed once below), so rows
  // 64..127 of the state stay zero and are neither loaded nor stored.
  static_assert(D == 64 || D == 128, "feature dimension");
  constexpr int KD = D / 16;  // K steps over the feature dimension
  // With two jobs the thread blocks of one (head, segment) -- both jobs, both value halves -- have adjacent
  // indices, so they run at the same time and share their tiles through L2.
  const int jobid = (NJOBS == 2) ? (int)(blockIdx.x & 1) : 0;
  const unsigned bidx = (NJOBS == 2) ? (blockIdx.x >> 1) : blockIdx.x;
  TcJob job = args.job[0];
  if (NJOBS == 2 && jobid) job = args.job[1];
  const CUtensorMap* const tm_a = (NJOBS == 2 && jobid) ? &maps1.a : &maps0.a;
  const CUtensorMap* const tm_b = (NJOBS == 2 && jobid) ? &maps1.b : &maps0.b;
  const CUtensorMap* const tm_c = (NJOBS == 2 && jobid) ? &maps1.c : &maps0.c;
  const CUtensorMap* const tm_out = (NJOBS == 2 && jobid) ? &maps1.out : &maps0.out;
  const int ehalf = (D == 128) ? (int)(bidx & 1) : 0;
  const int segid = (D == 128) ? (int)(bidx >> 1) : (int)bidx;
  const int seg = segid % args.nseg;
  int bh = segid / args.nseg;
  if (args.seq_order) bh = args.seq_order[bh / args.H] * args.H + bh % args.H;  // packed batch: longest sequences first
  const int hh_ = bh % args.H;  // head coordinate of the 4-D tensor maps
  // Packed batch (state-only kernel; the walk of a packed batch is the full-width kernel's): entry bh / H is a
  // sequence of its own length starting at token tok0 of one [tokens, H, D] tensor, the maps' batch coordinate is 0.
  const int n_tok = args.seq_len ? args.seq_len[bh / args.H] : args.N;
  const int tok0 = args.seq_start ? args.seq_start[bh / args.H] : 0;
  const int bb_ = args.seq_start ? 0 : bh / args.H;
  if (seg * args.seg_len >= n_tok) return;  // the grid covers the longest sequence; nothing has been set up yet
  const size_t head_off = (size_t)bb_ * args.sB + (size_t)hh_ * args.sH + (size_t)tok0 * args.sT;
  const int seg_t0 = seg * args.seg_len;
  const int seg_t1 = min(n_tok, seg_t0 + args.seg_len);
  const float s2 = (float)tab.s2[bh % args.H];
  int nblk = (seg_t1 - seg_t0 + 127) >> 7;
  int it0 = 0;  // forward pre-pass: index of the first block that is walked
  if (STATE_ONLY && s2 > 0.f) {
    // The pre-pass weighs every token by its decay to the edge the state leaves the segment through.  Once
    // s2 * distance exceeds 150 that weight is exactly zero in fp32 (exp2f underflows past the smallest
    // subnormal), so whole blocks far from the edge add exactly nothing and are not loaded at all: the blocks
    // kept are those whose nearest token is within 160 / s2 + 128 tokens of the edge (the margin makes the
    // skipped weights zero whatever the rounding of this bound).  Results are those of walking every block.
    const float reach = 160.f / s2;  // tokens
    int keep;
    if (REV) {
      keep = (int)fminf(ceilf((reach - 1.f) * (1.f / 128.f)) + 2.f, (float)nblk);
    } else {
      const float x = ((float)(seg_t1 - seg_t0) - reach) * (1.f / 128.f);  // blocks before the reach
      const int skip = max(0, min(nblk - 1, (int)floorf(x - 1.f)));
      keep = nblk - skip;
      it0 = skip;
    }
    keep = max(1, min(keep, nblk));
    nblk = keep;  // the reverse pre-pass walks blocks nblk-1 .. 0, the forward one it0 .. it0+nblk-1
  }
  const bool split_p = (args.precision & 1) != 0;
  const bool split_z = (args.precision & 2) != 0;
  // lambda == 1: the decayed rows equal the bf16 inputs, their lo term is identically zero
  const bool split_c = (args.precision & 4) != 0 && s2 != 0.f;

  if (tid == 0) {
    for (int i = 0; i < NUM_BARS; ++i) {
      uint32_t count = 1;
      // barriers that a compute group arrives on: one arrival per warp
      if (i == P_READY0 || i == P_READY1 || i == FC_READY0 || i == FC_READY1 || i == Z_READY)
        count = (STATE_ONLY && (i == FC_READY0 || i == FC_READY1)) ? 16 : 8;
      // P_READY of a block completes when the P group has written P AND the output group has read the
      // previous block's accumulators (both are what M4 waits for): 8 + 4 warps
      if (i == P_READY0 || i == P_READY1) count = 12;
      if (i == OG_SYNC) count = 4;
      // the c tile is released by the warps that read it (state-only) / by the thread that stores from it (walk)
      if (i == C_FREE0 || i == C_FREE1 || i == C_FREE2) count = STATE_ONLY ? 16 : 1;
      mbar_init(&sm.bars[i], count);
    }
    sm.abort = 0;
    fence_mbar_init();
    tma_prefetch_desc(tm_a);
    tma_prefetch_desc(tm_b);
    tma_prefetch_desc(tm_c);
    if (!STATE_ONLY) tma_prefetch_desc(tm_out);
  }
  if (warp == 1) {
    tmem_alloc(&sm.tmem_slot, TMEM_COLS);
    tmem_relinquish();
  }
  if (D == 64) {
    for (int i = tid; i < 2 * 1024; i += TC_THREADS)
      reinterpret_cast<uint4*>(&sm.st[i >> 10].b[1][0])[i & 1023] = make_uint4(0u, 0u, 0u, 0u);
    if (STATE_ONLY)  // the third load stage keeps its b tile where the walk kernel has stage 0's a tile
      for (int i = tid; i < 1024; i += TC_THREADS)
        reinterpret_cast<uint4*>(&sm.st[0].a[1][0])[i] = make_uint4(0u, 0u, 0u, 0u);
    fence_proxy_async_smem();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = sm.tmem_slot;
  bool issued_mma = false;
  uint32_t mma_elected = 0;  // set in the lane of warp 1 that issues the tensor-core instructions
  int armed_b[3] = {0, 0, 0}, armed_c[3] = {0, 0, 0};  // producer: uses armed per stage
  // State-only kernel: three load stages (the a tiles, which it never loads, hold the third stage's b and c), so
  // that a thread block running alone at the end of the launch has 144 KB in flight instead of 96 KB: its time per
  // block is the latency of HBM divided by the stages in flight.  The fc buffers stay two deep (it & 1).
  constexpr int NLS = STATE_ONLY ? 3 : 2;
  auto b_tile = [&](int ls) { return ls == 0 ? &sm.st[0].b[0][0] : (ls == 1 ? &sm.st[1].b[0][0] : &sm.st[0].a[0][0]); };
  auto c_tile = [&](int ls) { return ls == 0 ? &sm.st[0].c[0] : (ls == 1 ? &sm.st[1].c[0] : &sm.st[1].a[0][0]); };

  if (warp == 0) {
    // ------------------------------------ TMA producer ------------------------------------
    if (lane == 0) {
      for (int it = 0; it < nblk; ++it) {
        const int s = STATE_ONLY ? it % NLS : (it & 1);
        const int use = STATE_ONLY ? it / NLS : (it >> 1);  // how often this stage has been used before
        const uint32_t prev = (use - 1) & 1;                // parity of this stage's previous use
        const int blk = REV ? (nblk - 1 - it) : (it + it0);
        const int t0 = tok0 + seg_t0 + blk * 128;  // token coordinate of the maps
        // State-only kernel: the tiles a few blocks ahead are pulled into L2 now, so that the loads proper are
        // L2 hits (measured: 0.276 -> 0.245 ms per launch; the same in the walk kernel made it slower).
        if (STATE_ONLY && it + NLS < nblk) {
          const int tp = tok0 + seg_t0 + (REV ? (nblk - 1 - NLS - it) : (it + NLS + it0)) * 128;
          tma_prefetch_4d(tm_b, 0, tp, hh_, bb_);
          if (D == 128) tma_prefetch_4d(tm_b, 64, tp, hh_, bb_);
          tma_prefetch_4d(tm_c, ehalf * 64, tp, hh_, bb_);
        }
        if (STATE_ONLY) {
          if (it >= NLS) TC_WAIT(B_FREE0 + s, prev, 1);
          mbar_arrive_expect_tx(&sm.bars[FULL_B0 + s], D * 256);
          tma_load_4d(b_tile(s), tm_b, &sm.bars[FULL_B0 + s], 0, t0, hh_, bb_);
          if (D == 128) tma_load_4d(b_tile(s) + 128 * 64, tm_b, &sm.bars[FULL_B0 + s], 64, t0, hh_, bb_);
        } else {
          Stage& stg = sm.st[s];
          // walk kernel: the a and b tiles of a stage travel together (one barrier for both, FULL_B); A_FREE
          // is committed after M2, the last product of the block that reads either of them
          if (it >= 2) TC_WAIT(A_FREE0 + s, prev, 3);
          mbar_arrive_expect_tx(&sm.bars[FULL_B0 + s], D * 512);
          tma_load_4d(&stg.b[0][0], tm_b, &sm.bars[FULL_B0 + s], 0, t0, hh_, bb_);
          if (D == 128) tma_load_4d(&stg.b[1][0], tm_b, &sm.bars[FULL_B0 + s], 64, t0, hh_, bb_);
          tma_load_4d(&stg.a[0][0], tm_a, &sm.bars[FULL_B0 + s], 0, t0, hh_, bb_);
          if (D == 128) tma_load_4d(&stg.a[1][0], tm_a, &sm.bars[FULL_B0 + s], 64, t0, hh_, bb_);
        }
        armed_b[s] = use + 1;
        if (it >= NLS) TC_WAIT(C_FREE0 + s, prev, 2);
        mbar_arrive_expect_tx(&sm.bars[FULL_C0 + s], 16384);
        tma_load_4d(c_tile(s), tm_c, &sm.bars[FULL_C0 + s], ehalf * 64, t0, hh_, bb_);
        armed_c[s] = use + 1;
      }
    }
  } else if (warp == 1 && STATE_ONLY) {
    // ------------------------------------ MMA issuer, state-only kernel ------------------------------------
    // All 32 lanes run this loop converged (waits included); the tensor-core instructions and their commits
    // take effect in the one elected lane only.  Issued this way the instructions cost the warp few issue
    // slots (measured: 0.242 -> 0.229 ms per launch against the single-lane form the walk kernel uses,
    // which did not gain from it).
    {
      constexpr uint32_t ID_MN64 = umma_idesc_bf16(128, 64, true, true);   // b^T (MN-major A) x MN-major B
      constexpr uint32_t ID_MN128 = umma_idesc_bf16(128, 128, true, true); // same with [fc_hi | fc_lo], N = 128
      constexpr uint32_t HI = UMMA_DESC_HI_SBO1024;
      const uint32_t go = elect_one();
      mma_elected = go;
      // low descriptor halves (MN-major: 64-element chunks 16 KB apart); K step k adds k * 2 KB >> 4
      const uint32_t bm0 = umma_desc_lo(smem_u32(b_tile(0)), 16384), bm1 = umma_desc_lo(smem_u32(b_tile(1)), 16384);
      const uint32_t bm2 = umma_desc_lo(smem_u32(b_tile(2)), 16384);
      const uint32_t fh_lo = umma_desc_lo(smem_u32(&sm.fc_hi[0]), 16384), zh_lo = umma_desc_lo(smem_u32(&sm.z_hi[0]), 16384);
      for (int it = 0; it < nblk; ++it) {
        const int ls = it % NLS;   // load stage of the b tile
        const int s = it & 1;      // fc buffer
        const uint32_t par2 = (it >> 1) & 1;
        const uint32_t bm = ls == 0 ? bm0 : (ls == 1 ? bm1 : bm2);
        const uint32_t fbuf_lo = s ? zh_lo : fh_lo;  // fc buffer of this iteration (hi then lo, 16 KB apart)
        TC_WAIT_WARP(FULL_B0 + ls, (it / NLS) & 1, 4);
        TC_WAIT_WARP(FC_READY0 + s, par2, 5);
        tc_fence_after_sync();
        // tensor memory is otherwise unused here, so hi and lo share one N = 128 instruction
        // ([fc_hi | fc_lo]) into columns 0..127; the halves are summed at the end
#pragma unroll
        for (int k = 0; k < 8; ++k)
          umma_bf16_lh(tmem + COL_S0, bm + k * 128, fbuf_lo + k * 128, HI, split_c ? ID_MN128 : ID_MN64,
                       (it > 0 || k > 0), go);
        issued_mma = true;
        umma_commit_if(&sm.bars[B_FREE0 + ls], go);
        umma_commit_if(&sm.bars[FC_FREE0 + s], go);
      }
      umma_commit_if(&sm.bars[DZ_READY], go);
    }
  } else if (warp == 1) {
    // ------------------------------------ MMA issuer, walk kernel ------------------------------------
    // All 32 lanes run this loop converged (waits included); the tensor-core instructions and their commits take
    // effect in one elected lane only, a whole K loop per instruction sequence (measured: 4 % faster than issuing
    // from inside an `if (lane == 0)` region).
    {
      constexpr uint32_t ID_S = umma_idesc_bf16(128, 128, false, false);
      constexpr uint32_t ID_KN = umma_idesc_bf16(128, 64, false, true);
      constexpr uint32_t ID_MN64 = umma_idesc_bf16(128, 64, true, true);
      constexpr uint32_t HI = UMMA_DESC_HI_SBO1024;
      const uint32_t go = elect_one();
      mma_elected = go;
      // low descriptor halves.  K-major tiles (a, b in M1; a in M2): K step k adds (k >> 2) * 16 KB + (k & 3) * 32 B;
      // MN-major tiles (b^T in M3, fc, the state operand, c): K step k adds k * 2 KB.
      const uint32_t ak0 = umma_desc_lo(smem_u32(&sm.st[0].a[0][0]), 16), ak1 = umma_desc_lo(smem_u32(&sm.st[1].a[0][0]), 16);
      const uint32_t bk0 = umma_desc_lo(smem_u32(&sm.st[0].b[0][0]), 16), bk1 = umma_desc_lo(smem_u32(&sm.st[1].b[0][0]), 16);
      const uint32_t bm0 = umma_desc_lo(smem_u32(&sm.st[0].b[0][0]), 16384), bm1 = umma_desc_lo(smem_u32(&sm.st[1].b[0][0]), 16384);
      const uint32_t cm0 = umma_desc_lo(smem_u32(&sm.st[0].c[0]), 16384), cm1 = umma_desc_lo(smem_u32(&sm.st[1].c[0]), 16384);
      const uint32_t fh = umma_desc_lo(smem_u32(&sm.fc_hi[0]), 16384), fl = umma_desc_lo(smem_u32(&sm.fc_lo[0]), 16384);
      const uint32_t zh = umma_desc_lo(smem_u32(&sm.z_hi[0]), 16384), zl = umma_desc_lo(smem_u32(&sm.z_lo[0]), 16384);
      TC_WAIT_WARP(FULL_B0, 0, 7);
      tc_fence_after_sync();
      umma_group_ss<KD, true, true>(tmem + COL_S0, ak0, bk0, HI, ID_S, 0, go);
      issued_mma = true;
      umma_commit_if(&sm.bars[S_READY0], go);
      for (int it = 0; it < nblk; ++it) {
        const int s = it & 1;
        const uint32_t par1 = it & 1, par2 = (it >> 1) & 1;
        const uint32_t col_p = s ? COL_S1 : COL_S0;
        const uint32_t aks = s ? ak1 : ak0, bms = s ? bm1 : bm0, cms = s ? cm1 : cm0;
        const uint32_t akn = s ? ak0 : ak1, bkn = s ? bk0 : bk1;  // the other stage (next block)
        TC_WAIT_WARP(Z_READY, par1, 12);
        tc_fence_after_sync();
        umma_group_ss<8, false, false>(tmem + COL_DZ, bms, fh, HI, ID_MN64, 0, go);
        if (split_c) umma_group_ss<8, false, false>(tmem + COL_DZ, bms, fl, HI, ID_MN64, 1, go);
        umma_commit_if(&sm.bars[DZ_READY], go);
        const uint32_t col_oe = (it & 1) ? COL_OE1 : COL_OE0;
        umma_group_ss<KD, true, false>(tmem + col_oe, aks, zh, HI, ID_KN, 0, go);
        if (split_z) umma_group_ss<KD, true, false>(tmem + col_oe, aks, zl, HI, ID_KN, 1, go);
        umma_commit_if(&sm.bars[A_FREE0 + s], go);
        if (it + 1 < nblk) {
          const int s1 = s ^ 1;
          TC_WAIT_WARP(FULL_B0 + s1, ((it + 1) >> 1) & 1, 11);
          tc_fence_after_sync();
          umma_group_ss<KD, true, true>(tmem + (s1 ? COL_S1 : COL_S0), akn, bkn, HI, ID_S, 0, go);
          umma_commit_if(&sm.bars[S_READY0 + s1], go);
        }
        TC_WAIT_WARP(P_READY0 + s, par2, 14);
        TC_WAIT_WARP(FULL_C0 + s, par2, 15);
        tc_fence_after_sync();
        umma_group_ts8(tmem + COL_OI, tmem + col_p, cms, HI, ID_KN, 0, go);
        if (split_p) umma_group_ts8(tmem + COL_OI, tmem + col_p + 8, cms, HI, ID_KN, 1, go);
        umma_commit_if(&sm.bars[O_READY], go);
      }
    }
  } else if (STATE_ONLY && warp >= 4 && warp < 20) {
    // ------------------------------------ state-only kernel: fc producers ------------------------------------
    // Sixteen warps (the walk kernel's P and Z groups) form fc = diag(f_state) c: row r = 32 (w % 4) + lane,
    // sixteen of the 64 value columns each (two 16-byte chunks), hi and lo written to the buffer of stage s.
    const int w16 = warp - 4, q = w16 & 3, cq = w16 >> 2;
    const int r = q * 32 + lane;
    for (int it = 0; it < nblk; ++it) {
      const int s = it & 1;
      const int blk = REV ? (nblk - 1 - it) : (it + it0);
      const int t0 = seg_t0 + blk * 128;
      // decay from token t0 + r to the edge of the segment that the state leaves through
      float f = 0.f;
      if (r < min(128, seg_t1 - t0))
        f = REV ? exp2f(-s2 * (float)(t0 + r - seg_t0 + 1)) : exp2f(-s2 * (float)(seg_t1 - 1 - t0 - r));
      const int ls = it % NLS;  // load stage of the c tile
      TC_WAIT_WARP(FULL_C0 + ls, (it / NLS) & 1, 18);
      if (it >= 2) TC_WAIT_WARP(FC_FREE0 + s, ((it >> 1) - 1) & 1, 19);  // the MMA two blocks back has read this buffer
      const __nv_bfloat16* ctile = c_tile(ls);
      __nv_bfloat16* hi_tile = s ? sm.z_hi : sm.fc_hi;
      __nv_bfloat16* lo_tile = s ? sm.z_lo : sm.fc_lo;
#pragma unroll
      for (int x2 = 0; x2 < 2; ++x2) {
        const int off = r * 64 + (((2 * cq + x2) ^ (r & 7)) << 3);
        const uint4 raw = *reinterpret_cast<const uint4*>(ctile + off);
        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
        float x8[8];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          const float2 v = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[x]));
          x8[2 * x] = v.x * f;
          x8[2 * x + 1] = v.y * f;
        }
        uint4 h, l;
        split8(x8, h, l);
        *reinterpret_cast<uint4*>(hi_tile + off) = h;
        if (split_c) *reinterpret_cast<uint4*>(lo_tile + off) = l;
      }
      fence_proxy_async_smem();
      WARP_ARRIVE(FC_READY0 + s);
      if (lane == 0) mbar_arrive(&sm.bars[C_FREE0 + ls]);
    }
    if (warp >= 12) {
      // segment-local state = accumulated dZ (hi-part + lo-part); this warp's 32 state columns of row r
      const int zh = (warp - 12) >> 2;
      const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
      TC_WAIT_WARP(DZ_READY, 0, 20);
      tc_fence_after_sync();
      float* dst = args.local_out + ((size_t)bh * args.nseg + seg) * (D * D) + (size_t)r * D + ehalf * 64 + zh * 32;
#pragma unroll
      for (int pc = 0; pc < 2; ++pc) {
        if (r >= D) break;  // D = 64: state rows 64..127 do not exist (warp-uniform: r = 32 q + lane)
        uint32_t dh[16], dl[16];
        tmem_ld_x16(lane_addr + COL_S0 + zh * 32 + pc * 16, dh);
        if (split_c) tmem_ld_x16(lane_addr + COL_S0 + 64 + zh * 32 + pc * 16, dl);
        tmem_ld_wait();
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          float4 v;
          v.x = __uint_as_float(dh[4 * x]) + (split_c ? __uint_as_float(dl[4 * x]) : 0.f);
          v.y = __uint_as_float(dh[4 * x + 1]) + (split_c ? __uint_as_float(dl[4 * x + 1]) : 0.f);
          v.z = __uint_as_float(dh[4 * x + 2]) + (split_c ? __uint_as_float(dl[4 * x + 2]) : 0.f);
          v.w = __uint_as_float(dh[4 * x + 3]) + (split_c ? __uint_as_float(dl[4 * x + 3]) : 0.f);
          *reinterpret_cast<float4*>(dst + pc * 16 + 4 * x) = v;
        }
      }
      tc_fence_before_sync();
    }
  } else if (warp >= 4 && warp < 12) {
    // ------------------------------------ P group ------------------------------------
    if (!STATE_ONLY) {
      const int q = warp & 3;
      const int half = (warp - 4) >> 2;  // which two of the four 32-column chunks this warp converts
      const int r = q * 32 + lane;       // score row i
      const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
      for (int it = 0; it < nblk; ++it) {
        const int s = it & 1;
        const uint32_t colS = lane_addr + (s ? COL_S1 : COL_S0);
        TC_WAIT_WARP(S_READY0 + s, (it >> 1) & 1, 17);
        tc_fence_after_sync();
#pragma unroll 1
        for (int ci = 0; ci < 2; ++ci) {
          const int cc = half * 2 + ci;
          const bool all_masked = REV ? (cc < q) : (cc > q);  // 32x32 sub-tile outside the causal band
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {  // 16 columns per pass
            uint32_t h8[8], l8[8];
            if (all_masked) {
#pragma unroll
              for (int x = 0; x < 8; ++x) h8[x] = l8[x] = 0u;
            } else {
              uint32_t sreg[16];
              tmem_ld_x16(colS + cc * 32 + hh * 16, sreg);
              float d[16];
              // lambda^n on the special-function unit (idle otherwise); n < 0 is masked out below
              const float n0 = (float)(REV ? (cc * 32 + hh * 16 - r) : (r - cc * 32 - hh * 16));
#pragma unroll
              for (int x = 0; x < 16; ++x) d[x] = ex2_approx(-s2 * (REV ? n0 + (float)x : n0 - (float)x));
              tmem_ld_wait();
#pragma unroll
              for (int x = 0; x < 16; ++x) {
                const int j = cc * 32 + hh * 16 + x;
                const int n = REV ? (j - r) : (r - j);
                // a select, not a multiply by zero: masked-out tokens can never leak
                d[x] = (n >= 0) ? __uint_as_float(sreg[x]) * d[x] : 0.f;
              }
              split16(d, h8, l8);
            }
            // in place: the 16 fp32 columns just read become 8 columns of hi pairs + 8 of lo pairs
            tmem_st_x8(colS + cc * 32 + hh * 16, h8);
            if (split_p) tmem_st_x8(colS + cc * 32 + hh * 16 + 8, l8);
          }
        }
        tmem_st_wait();
        tc_fence_before_sync();
        WARP_ARRIVE(P_READY0 + s);
      }
    }
  } else if (warp >= 12 && warp < 20) {
    // ------------------------------------ Z group (walk kernel) ------------------------------------
    const int q = warp & 3;
    const int zh = (warp - 12) >> 2;  // which 32 of the 64 state / value columns this warp owns
    const int r = q * 32 + lane;      // token row j of c / state row k of Z
    const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);

    // fc = diag(f_state) c is formed 16 bytes (8 columns) at a time: piece i of this thread is chunk (zt & 7) of
    // token row 32 i + (zt >> 3), so a warp reads whole 128-byte lines of c per load instruction (four rows of this
    // block's 64 value columns) and writes whole rows of the operand tile; row-per-thread loads would touch 32
    // lines per instruction, and the load/store unit's time per line is what every group's shared-memory traffic
    // then waits behind (measured on the full-width kernel: 7 % of a step).
    const int zt = (warp - 12) * 32 + lane;  // 0 .. 255
    const int frow = zt >> 3, fch = zt & 7;
    // decay factor of token row `row` of block iteration `it` in the state update
    auto state_factor = [&](int it, int row) -> float {
      const int blk = REV ? (nblk - 1 - it) : it;
      const int t0 = seg_t0 + blk * 128;
      const int Cr = min(128, seg_t1 - t0);
      if (row >= Cr) return 0.f;
      return REV ? exp2f(-s2 * (float)(row + 1)) : exp2f(-s2 * (float)(Cr - 1 - row));
    };
    auto make_fc = [&](const uint4 (&raw)[4], int it, __nv_bfloat16* hi_tile, __nv_bfloat16* lo_tile) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int row = 32 * i + frow;
        const float f = state_factor(it, row);
        const uint32_t w[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
        float x8[8];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          const float2 v = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[x]));
          x8[2 * x] = v.x * f;
          x8[2 * x + 1] = v.y * f;
        }
        uint4 h, l;
        split8(x8, h, l);
        const int off = row * 64 + ((fch ^ (row & 7)) << 3);
        *reinterpret_cast<uint4*>(hi_tile + off) = h;
        if (split_c) *reinterpret_cast<uint4*>(lo_tile + off) = l;
      }
      fence_proxy_async_smem();
    };
    // this thread's four pieces of c straight from global memory (keeps the shared c tile off the state chain, so
    // that tile only has to arrive in time for M4); rows beyond N read as zero
    auto c_from_global = [&](int it, uint4 (&raw)[4]) {
      const int blk = REV ? (nblk - 1 - it) : it;
      const int t0 = seg_t0 + blk * 128;
      const __nv_bfloat16* src = static_cast<const __nv_bfloat16*>(job.c) + head_off + (size_t)(t0 + frow) * args.sT +
                                 ehalf * 64 + fch * 8;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (t0 + 32 * i + frow < args.N) raw[i] = __ldg(reinterpret_cast<const uint4*>(src + (size_t)(32 * i) * args.sT));
        else raw[i] = make_uint4(0u, 0u, 0u, 0u);
      }
    };

    {
      float zreg[32];
      if (job.entry && r < D) {
        const float4* src = reinterpret_cast<const float4*>(
            job.entry + ((size_t)bh * args.nseg + seg) * (D * D) + (size_t)r * D + ehalf * 64 + zh * 32);
#pragma unroll
        for (int x = 0; x < 8; ++x) {
          const float4 v = __ldg(src + x);
          zreg[4 * x] = v.x; zreg[4 * x + 1] = v.y; zreg[4 * x + 2] = v.z; zreg[4 * x + 3] = v.w;
        }
      } else {
#pragma unroll
        for (int x = 0; x < 32; ++x) zreg[x] = 0.f;
      }
      // bf16 hi/lo operand of the current state rows (this warp's 32 columns)
      auto write_state_operand = [&]() {
#pragma unroll
        for (int x4 = 0; x4 < 4; ++x4) {
          float x8[8];
#pragma unroll
          for (int x = 0; x < 8; ++x) x8[x] = zreg[x4 * 8 + x];
          uint4 h, l;
          split8(x8, h, l);
          const int off = r * 64 + (((4 * zh + x4) ^ (r & 7)) << 3);
          *reinterpret_cast<uint4*>(sm.z_hi + off) = h;
          if (split_z) *reinterpret_cast<uint4*>(sm.z_lo + off) = l;
        }
        fence_proxy_async_smem();
      };
      uint4 cnext[4];  // row slice of the next block's c, fetched one block ahead
      c_from_global(0, cnext);
      make_fc(cnext, 0, sm.fc_hi, sm.fc_lo);
      if (nblk > 1) c_from_global(1, cnext);
      write_state_operand();
      WARP_ARRIVE(Z_READY);

      for (int it = 0; it < nblk; ++it) {
        const int blk = REV ? (nblk - 1 - it) : it;
        const int Cr = min(128, seg_t1 - (seg_t0 + blk * 128));
        // ---- Z <- Gamma Z + dZ ----
        TC_WAIT_WARP(DZ_READY, it & 1, 22);
        tc_fence_after_sync();
        {
          const float gamma = exp2f(-s2 * (float)Cr);
#pragma unroll
          for (int pc = 0; pc < 2; ++pc) {
            uint32_t dh[16];
            tmem_ld_x16(lane_addr + COL_DZ + zh * 32 + pc * 16, dh);
            tmem_ld_wait();
#pragma unroll
            for (int x = 0; x < 16; ++x) zreg[pc * 16 + x] = fmaf(gamma, zreg[pc * 16 + x], __uint_as_float(dh[x]));
          }
          tc_fence_before_sync();  // ordered before the Z_READY arrival below, which is what M3 of the next block waits for
        }
        if (it + 1 < nblk) {
          // DZ_READY also says M3 of this block is done, so the fc buffer may be rewritten
          make_fc(cnext, it + 1, sm.fc_hi, sm.fc_lo);
          if (it + 2 < nblk) c_from_global(it + 2, cnext);
          // A_FREE of this block's stage: M2 of this block is done, so it has read the old state operand
          TC_WAIT_WARP(A_FREE0 + (it & 1), (it >> 1) & 1, 23);
          write_state_operand();
          WARP_ARRIVE(Z_READY);
        }
      }
      const bool last_processed = REV ? (seg == 0) : (seg == args.nseg - 1);
      if (job.final_out && last_processed && r < D) {
        float* dst = job.final_out + (size_t)bh * (D * D) + (size_t)r * D + ehalf * 64 + zh * 32;
#pragma unroll
        for (int x = 0; x < 8; ++x)
          *reinterpret_cast<float4*>(dst + 4 * x) = make_float4(zreg[4 * x], zreg[4 * x + 1], zreg[4 * x + 2], zreg[4 * x + 3]);
      }
    }
  } else if (warp >= 20) {
    // ------------------------------------ O group ------------------------------------
    if (!STATE_ONLY) {
      const int q = warp & 3;
      const int r = q * 32 + lane;  // output row i
      const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
      uint32_t og_uses = 0;  // phases of the group's own barrier used so far
      if (lane == 0) mbar_arrive(&sm.bars[P_READY0]);  // block 0 has no earlier accumulators to wait for
      for (int it = 0; it < nblk; ++it) {
        const int s = it & 1;
        const int blk = REV ? (nblk - 1 - it) : it;
        const int t0 = seg_t0 + blk * 128;
        const int Cr = min(128, seg_t1 - t0);
        float f = 0.f;
        if (r < Cr) f = REV ? exp2f(-s2 * (float)(Cr - 1 - r)) : exp2f(-s2 * (float)(r + 1));
        // staging tile for the bulk stores: the c tile of this block, dead once M4 is done
        unsigned char* stg = reinterpret_cast<unsigned char*>(&sm.st[s].c[0]);
        // O_READY: every MMA up to M4 of this block is done
        TC_WAIT_WARP(O_READY, it & 1, 25);
        tc_fence_after_sync();
        constexpr int PASSES = (sizeof(TOut) == 4) ? 2 : 1;  // 128 bytes of each output row per pass
        constexpr int PIECES = (sizeof(TOut) == 4) ? 2 : 4;  // 16-column accumulator pieces per pass
#pragma unroll
        for (int pass = 0; pass < PASSES; ++pass) {
          uint32_t w[32];  // this thread's 128 bytes of the pass
#pragma unroll
          for (int pc = 0; pc < PIECES; ++pc) {
            const int col = (pass * PIECES + pc) * 16;
            uint32_t oi[16], oe[16];
            tmem_ld_x16(lane_addr + COL_OI + col, oi);
            tmem_ld_x16(lane_addr + ((it & 1) ? COL_OE1 : COL_OE0) + col, oe);
            tmem_ld_wait();
            if (pass == PASSES - 1 && pc == PIECES - 1) {
              tc_fence_before_sync();
              // both accumulators are in registers now: M4 of the next block may overwrite O_intra
              if (it + 1 < nblk) WARP_ARRIVE(P_READY0 + (s ^ 1));
            }
            if (sizeof(TOut) == 4) {
#pragma unroll
              for (int x = 0; x < 16; ++x)
                w[pc * 16 + x] = __float_as_uint(fmaf(f, __uint_as_float(oe[x]), __uint_as_float(oi[x])));
            } else {
#pragma unroll
              for (int x = 0; x < 8; ++x) {
                const __nv_bfloat162 h = __floats2bfloat162_rn(
                    fmaf(f, __uint_as_float(oe[2 * x]), __uint_as_float(oi[2 * x])),
                    fmaf(f, __uint_as_float(oe[2 * x + 1]), __uint_as_float(oi[2 * x + 1])));
                w[pc * 8 + x] = *reinterpret_cast<const uint32_t*>(&h);
              }
            }
          }
          if (pass > 0) {
            // the staging tile still feeds the previous pass's store until its source has been read
            if (warp == 20 && lane == 0) tma_store_wait_read();
            WARP_ARRIVE(OG_SYNC);
            TC_WAIT_WARP(OG_SYNC, og_uses & 1, 27);
            ++og_uses;
          }
          // row r of the [128 rows][128 bytes] staging tile, 16-byte chunks swizzled as the store expects
#pragma unroll
          for (int c = 0; c < 8; ++c)
            *reinterpret_cast<uint4*>(stg + r * 128 + ((c ^ (r & 7)) << 4)) =
                make_uint4(w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
          fence_proxy_async_smem();
          WARP_ARRIVE(OG_SYNC);
          TC_WAIT_WARP(OG_SYNC, og_uses & 1, 28);
          ++og_uses;
          if (warp == 20 && lane == 0) {
            // rows beyond N are clipped by the tensor map (a ragged block is always the last of the sequence)
            tma_store_4d(tm_out, stg, ehalf * 64 + pass * (int)(128 / sizeof(TOut)), t0, hh_, bb_);
            tma_store_commit();
          }
        }
        if (warp == 20 && lane == 0) {
          tma_store_wait_read();
          mbar_arrive(&sm.bars[C_FREE0 + s]);  // the c tile of this stage may be reloaded
        }
      }
    }
  }

teardown:
  // the storing thread's bulk stores must have read their shared-memory source before the block exits
  if (!STATE_ONLY && warp == 20 && lane == 0) tma_store_wait_all();
  // After an expired wait: drain what this thread started so nothing is in flight when the
  // block exits (loads into shared memory, tensor-core work on tensor memory).
  if (sm.abort) {
    if (warp == 0 && lane == 0) {
      for (int s = 0; s < 3; ++s) {
        if (armed_b[s] > 0) drain_wait(&sm.bars[FULL_B0 + s], (armed_b[s] - 1) & 1);
        if (armed_c[s] > 0) drain_wait(&sm.bars[FULL_C0 + s], (armed_c[s] - 1) & 1);
      }
    }
    if (warp == 1 && mma_elected && issued_mma) {
      umma_commit(&sm.bars[DRAIN]);
      drain_wait(&sm.bars[DRAIN], 0);
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, TMEM_COLS);
}

// Self-test of the failure path: one warp waits, with the kernels' own bounded wait, on a barrier that
// nothing ever arrives on; when the budget runs out it records code 99 like a real block would and returns.
__global__ void bounded_wait_selftest_kernel(long long budget) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    fence_mbar_init();
  }
  __syncthreads();
  if (!wait_or_abort(&bar, 0, &abort_flag, budget)) {
    if (threadIdx.x == 0) atomicCAS(&g_tc_status, 0u, 99u);
  }
}

#include "la_tc_full.cuh"

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

// Tensor map over a token tensor seen as {feature D, token N, head H, batch B} with element strides {1, sT, sH, sB}
// (D = 64 or 128, bf16 or fp32), a box of 128 bytes x 128 tokens x 1 x 1 and 128-byte swizzle; tokens beyond N read
// as zero and are not written.
bool make_map(CUtensorMap* m, const void* ptr, const OpArgs& a, int D, bool f32 = false) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return false;
  const cuuint64_t esz = f32 ? 4 : 2;
  // packed batch: one [total_tokens, H, D] tensor, batch extent 1
  const int B = a.seq_start ? 1 : a.BH / a.H;
  const int tokens = a.seq_start ? a.total_tokens : a.N;
  cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)tokens, (cuuint64_t)a.H, (cuuint64_t)B};
  cuuint64_t strides[3] = {(cuuint64_t)a.sT * esz, (cuuint64_t)a.sH * esz, (cuuint64_t)a.sB * esz};
  cuuint32_t box[4] = {(cuuint32_t)(128 / esz), 128, 1, 1};
  cuuint32_t es[4] = {1, 1, 1, 1};
  return enc(m, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr),
             dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
             CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <bool REV, bool STATE_ONLY, typename TOut, int D, int NJOBS>
cudaError_t launch_t(const TcMaps& m0, const TcMaps& m1, const TcArgs& ta, const DecayTable& tab, cudaStream_t stream) {
  const size_t smem = sizeof(TcSmem) + 1024;
  auto kern = tc_kernel<REV, STATE_ONLY, TOut, D, NJOBS>;
  cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (err != cudaSuccess) return err;
  KernelTimer timer(STATE_ONLY ? K_PREPASS : (NJOBS == 2 ? K_WALK_PAIR : K_WALK), stream);
  kern<<<(unsigned)(ta.BH * ta.nseg * (D == 128 ? 2 : 1) * NJOBS), TC_THREADS, smem, stream>>>(m0, m1, ta, tab);
  count_launch();
  return cudaGetLastError();
}

bool make_maps(TcMaps* m, const OpArgs& args, int D, bool f32) {
  return make_map(&m->a, args.a, args, D) && make_map(&m->b, args.b, args, D) && make_map(&m->c, args.c, args, D) &&
         make_map(&m->out, args.out ? args.out : args.y, args, D, f32);  // (gated walk without `out`: y)
}

// One walk (second == nullptr) or two walks of the same direction over the same tokens in one launch.
template <int D>
cudaError_t launch_walk_d(const OpArgs& args, const OpArgs* second, const DecayTable& tab, int out_dt, int precision,
                          cudaStream_t stream) {
  TcMaps m0, m1;
  const bool f32 = (out_dt == DT_F32);
  if (!make_maps(&m0, args, D, f32)) return cudaErrorInvalidValue;
  if (second) {
    if (!make_maps(&m1, *second, D, f32)) return cudaErrorInvalidValue;
  } else {
    m1 = m0;
  }
  TcArgs ta{};
  ta.job[0] = TcJob{args.c, args.out, args.entry, args.final_out, args.u, args.y, args.rstd};
  ta.job[1] = second ? TcJob{second->c, second->out, second->entry, second->final_out, nullptr, nullptr, nullptr} : ta.job[0];
  ta.local_out = nullptr;
  ta.njobs = second ? 2 : 1;
  ta.BH = args.BH; ta.H = args.H; ta.N = args.N; ta.seg_len = args.seg_len; ta.nseg = args.nseg;
  ta.precision = precision;
  ta.sT = args.sT; ta.sH = args.sH; ta.sB = args.sB;
  ta.seq_start = args.seq_start;
  ta.seq_len = args.seq_len;
  ta.seq_order = args.seq_order;
  if (args.seq_start && !tc_walk_is_full(D, args.out, second ? second->out : nullptr))
    return cudaErrorInvalidValue;  // only the full-width kernel walks packed batches (the caller checks first)
  if (args.u) {
    // forward walk with the gate epilogue: only the full-width kernel has it (the caller asks tc_can_fuse_gate first)
    if (D != 128 || second || args.reverse || !tc_can_fuse_gate(args, D)) return cudaErrorInvalidValue;
    return f32 ? launch_full_t<false, float, 1, true>(m0, m1, ta, tab, stream)
               : launch_full_t<false, __nv_bfloat16, 1, true>(m0, m1, ta, tab, stream);
  }
  if (D == 128 && !(reinterpret_cast<uintptr_t>(args.out) & 31u) &&
      !(second && (reinterpret_cast<uintptr_t>(second->out) & 31u))) {
    // full-width kernel: one thread block per (head, segment).  Its 32-byte output stores need that alignment;
    // an output that is only 16-byte aligned (the contract's minimum) takes the half-width kernels below.
    if (second) {
      if (!args.reverse) return cudaErrorInvalidValue;
      return f32 ? launch_full_t<true, float, 2, false>(m0, m1, ta, tab, stream)
                 : launch_full_t<true, __nv_bfloat16, 2, false>(m0, m1, ta, tab, stream);
    }
    if (args.reverse)
      return f32 ? launch_full_t<true, float, 1, false>(m0, m1, ta, tab, stream)
                 : launch_full_t<true, __nv_bfloat16, 1, false>(m0, m1, ta, tab, stream);
    return f32 ? launch_full_t<false, float, 1, false>(m0, m1, ta, tab, stream)
               : launch_full_t<false, __nv_bfloat16, 1, false>(m0, m1, ta, tab, stream);
  }
  if (second) {  // only the reverse direction is ever paired
    if (!args.reverse) return cudaErrorInvalidValue;
    return f32 ? launch_t<true, false, float, D, 2>(m0, m1, ta, tab, stream)
               : launch_t<true, false, __nv_bfloat16, D, 2>(m0, m1, ta, tab, stream);
  }
  if (args.reverse)
    return f32 ? launch_t<true, false, float, D, 1>(m0, m1, ta, tab, stream)
               : launch_t<true, false, __nv_bfloat16, D, 1>(m0, m1, ta, tab, stream);
  return f32 ? launch_t<false, false, float, D, 1>(m0, m1, ta, tab, stream)
             : launch_t<false, false, __nv_bfloat16, D, 1>(m0, m1, ta, tab, stream);
}

template <int D>
cudaError_t launch_prepass_d(const OpArgs& args, const DecayTable& tab, int precision, cudaStream_t stream) {
  TcMaps m;
  // the a and out maps are unused by the state-only kernel; valid descriptors are passed anyway
  if (!make_map(&m.b, args.b, args, D) || !make_map(&m.c, args.c, args, D))
    return cudaErrorInvalidValue;
  m.a = m.b;
  m.out = m.c;
  TcArgs ta{};
  ta.job[0] = TcJob{args.c, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
  ta.job[1] = ta.job[0];
  ta.local_out = args.local_out;
  ta.njobs = 1;
  ta.BH = args.BH; ta.H = args.H; ta.N = args.N; ta.seg_len = args.seg_len; ta.nseg = args.nseg;
  ta.precision = precision;
  ta.sT = args.sT; ta.sH = args.sH; ta.sB = args.sB;
  ta.seq_start = args.seq_start;
  ta.seq_len = args.seq_len;
  ta.seq_order = args.seq_order;
  return args.reverse ? launch_t<true, true, float, D, 1>(m, m, ta, tab, stream)
                      : launch_t<false, true, float, D, 1>(m, m, ta, tab, stream);
}

}  // namespace

bool tc_supported() { return encode_fn() != nullptr; }

cudaError_t launch_tc_walk(const OpArgs& args, const DecayTable& tab, int D, int out_dt, int precision,
                           cudaStream_t stream) {
  return D == 128 ? launch_walk_d<128>(args, nullptr, tab, out_dt, precision, stream)
                  : launch_walk_d<64>(args, nullptr, tab, out_dt, precision, stream);
}

bool tc_full_width() { return true; }

bool tc_walk_is_full(int D, const void* out0, const void* out1) {
  return D == 128 && !((reinterpret_cast<uintptr_t>(out0) | reinterpret_cast<uintptr_t>(out1)) & 31u);
}

bool tc_can_fuse_gate(const OpArgs& args, int D) {
  if (D != 128 || !args.u || !args.y) return false;
  if (reinterpret_cast<uintptr_t>(args.y) & 31u) return false;
  if (args.out && (reinterpret_cast<uintptr_t>(args.out) & 31u)) return false;
  return true;
}

cudaError_t launch_tc_walk_pair(const OpArgs& first, const OpArgs& second, const DecayTable& tab, int D, int out_dt,
                                int precision, cudaStream_t stream) {
  if (first.reverse != second.reverse || first.N != second.N || first.BH != second.BH || first.nseg != second.nseg ||
      first.seg_len != second.seg_len)
    return cudaErrorInvalidValue;
  return D == 128 ? launch_walk_d<128>(first, &second, tab, out_dt, precision, stream)
                  : launch_walk_d<64>(first, &second, tab, out_dt, precision, stream);
}

cudaError_t launch_tc_prepass(const OpArgs& args, const DecayTable& tab, int D, int precision, cudaStream_t stream) {
  return D == 128 ? launch_prepass_d<128>(args, tab, precision, stream) : launch_prepass_d<64>(args, tab, precision, stream);
}

cudaError_t launch_bounded_wait_selftest(long long budget_clocks, cudaStream_t stream) {
  bounded_wait_selftest_kernel<<<1, 32, 0, stream>>>(budget_clocks);
  count_launch();
  return cudaGetLastError();
}

// Reads the failure flag and clears it in one atomic exchange on the device, so that a code recorded between
// a separate read and a separate clear cannot be lost.
__global__ void status_exchange_kernel(bool clear) {
  g_tc_status_read = clear ? atomicExch(&g_tc_status, 0u) : atomicAdd(&g_tc_status, 0u);
}

unsigned int tc_read_status(bool clear) {
  unsigned int v = 0;
  status_exchange_kernel<<<1, 1, 0, cudaStreamPerThread>>>(clear);
  if (cudaGetLastError() != cudaSuccess) return 0xFFFFFFFFu;
  if (cudaStreamSynchronize(cudaStreamPerThread) != cudaSuccess) return 0xFFFFFFFFu;
  if (cudaMemcpyFromSymbol(&v, g_tc_status_read, sizeof(v)) != cudaSuccess) return 0xFFFFFFFFu;
  return v;
}

}  // namespace la
