// Full-width block walk for D = 128 (included by la_tc.cu, inside its anonymous namespace, after the helpers).
//
// One thread block walks the 128-token blocks of one (batch*head, segment) and produces all 128 value columns,
// so every tensor-core product is 128 x 128 (N = 128) and the score tile S and its conversion to P are computed
// once per block instead of once per value half:
//   M1  S        = a b^T                              K = 128     8 instructions
//   M3  dZ       = b^T fc_hi (+ b^T fc_lo)            K = 128     8 (+ 8)
//   M2  O_inter  = a Z_hi (+ a Z_lo)                  K = 128     8 (+ 8)
//   M4  O_intra  = P_hi c (+ P_lo c)                  K = 128     8 (+ 8), P read from tensor memory
// Per 128 tokens that is 56 instructions of N = 128 where two half-width thread blocks issue 112 (96 of them
// N = 64, which fetch as many operand bytes from shared memory per instruction for half the work), and half the
// CUDA-core work on scores.  The price is space: the four 128 x 128 accumulators fill tensor memory
// (S/P, O_intra, O_inter, dZ: 4 x 128 columns) and the operands fill shared memory (a, b, c, fc hi/lo, state
// hi/lo: 7 x 32 KB), so nothing is double-buffered.  What makes that affordable is the order of the products:
//   per block n:  M3(n)  M2(n)  M4(n)  M1(n+1)
// - b(n) is free after M3(n) and a(n) after M2(n); each is reloaded at once, while the later products of the
//   block run, and both are needed again by M1(n+1);
// - c(n) is free after M4(n) and c(n+1) is needed a whole block later;
// - S/P is rewritten by M1(n+1) right after M4(n) has read P(n); the P group converts S(n+1) while M3(n+1) and
//   M2(n+1) keep the tensor pipe busy;
// - dZ(n), O_inter(n), O_intra(n) are each read by their group at least one product group before they are
//   overwritten.
// Output rows leave as 32-byte stores straight from registers (there is no shared memory left to stage them),
// after a four-lane transpose that makes every store instruction write whole 128-byte lines.
//
// Warp roles (32 warps): 0 TMA producer, 1 MMA issuer (all lanes converged, instructions on one elected lane),
// 4-7 P group, 8-11 and 28-31 O group (two warps per 32 rows, half of the columns each), 12-27 Z group (state rows
// in registers, 32 columns per warp).  Registers are re-divided between the roles with setmaxnreg after start-up.
// (Measured on B200 at the 7B-like shape: pulling the tiles into L2 two blocks ahead with TMA prefetches made the
// kernel 1 % slower, so there is none.)

constexpr int F_THREADS = 1024;
constexpr uint32_t FCOL_S = 0, FCOL_OI = 128, FCOL_OE = 256, FCOL_DZ = 384;

enum FBar {
  F_FULL_AB = 0,            // TMA -> MMA: b (requested when M3 of the previous block is done) and a (when M2 is)
  F_AB_FREE,                // M2 done: a and the state operand may be overwritten
  F_S_READY,
  F_M4_OK,                  // P written by the P group (8 arrivals) and c landed (the producer's arrival and bytes)
  F_DZ_READY, F_Z_READY,
  F_O_READY,                // M4 done: accumulators complete, c may be overwritten
  F_O_FREE,                 // the output group has read both accumulators
  F_DRAIN,
  F_NUM_BARS
};

struct alignas(1024) FSmem {
  __nv_bfloat16 a[2][128 * 64];      // query-like tile, K-major, two K panels
  __nv_bfloat16 b[2][128 * 64];      // key-like tile (K-major in M1, read as b^T MN-major in M3)
  __nv_bfloat16 c[2][128 * 64];      // value-like tile, MN-major B operand: two 64-column chunks
  __nv_bfloat16 fc_hi[2][128 * 64];  // decayed value rows, hi and lo terms
  __nv_bfloat16 fc_lo[2][128 * 64];
  __nv_bfloat16 z_hi[2][128 * 64];   // state operand, hi and lo terms
  __nv_bfloat16 z_lo[2][128 * 64];
  uint64_t bars[F_NUM_BARS];
  uint32_t tmem_slot;
  int abort;
};

// Clears, in the P tile a warp has just written to tensor memory (its 32 rows, 128 columns as 8 passes of 16:
// words 0..7 of a pass hold the hi terms of column pairs (2x, 2x + 1), words 8..15 the lo terms), the columns from
// `first` on.  Called once per thread block at most, by the whole warp; kept out of line so that the P group's
// loop is compiled exactly as it is without it (a bound inside the loop cost the dense walk 1.5 %, this block
// inlined behind it 0.4 %).
__device__ __noinline__ void clear_keys_past_end(uint32_t colS, int first) {
  tmem_st_wait();
  for (int pass = first >> 4; pass < 8; ++pass) {
    uint32_t w16[16];
    tmem_ld_x16(colS + pass * 16, w16);
    tmem_ld_wait();
    uint32_t h8[8], l8[8];
#pragma unroll
    for (int x = 0; x < 8; ++x) {
      const int j = pass * 16 + 2 * x;
      const uint32_t keep = (j < first ? 0x0000ffffu : 0u) | (j + 1 < first ? 0xffff0000u : 0u);
      h8[x] = w16[x] & keep;
      l8[x] = w16[8 + x] & keep;
    }
    tmem_st_x8(colS + pass * 16, h8);
    tmem_st_x8(colS + pass * 16 + 8, l8);
  }
}

template <int N>
__device__ __forceinline__ void reg_dec() {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N>
__device__ __forceinline__ void reg_inc() {
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}

// NJOBS = 2: two walks of the same direction over the same tokens in one launch (the dV and dK walks of the backward
// pass, which between them read Q, K, V and dO); the thread blocks of the two jobs alternate, so that the two
// readers of a tile run side by side and the tile comes from HBM once.
// GATED (forward, single job): the epilogue y = SRMSNorm(out) (.) u of Eq. 3 with Eq. 8 is applied to the rows
// before they leave (job.u, job.y; job.out and job.rstd optional).
template <bool REV, typename TOut, int NJOBS, bool GATED>
__global__ void __launch_bounds__(F_THREADS, 1)
tc_walk_full_kernel(const __grid_constant__ TcMaps maps0, const __grid_constant__ TcMaps maps1, const TcArgs args,
                    const DecayTable tab) {
  extern __shared__ unsigned char smem_raw[];
  FSmem& sm = *reinterpret_cast<FSmem*>(smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u));

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int jobid = (NJOBS == 2) ? (int)(blockIdx.x & 1) : 0;
  const int bidx = (NJOBS == 2) ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  TcJob job = args.job[0];
  if (NJOBS == 2 && jobid) job = args.job[1];
  const TcMaps& maps = (NJOBS == 2 && jobid) ? maps1 : maps0;
  const int seg = bidx % args.nseg;
  int bh = bidx / args.nseg;
  // packed batch: thread blocks take the sequences longest first, so that a long one is not what the launch ends on
  if (args.seq_order) bh = args.seq_order[bh / args.H] * args.H + bh % args.H;
  const int hh_ = bh % args.H;  // head coordinate of the 4-D tensor maps
  // Packed batch: "batch" entry bh / H is a sequence of its own length inside one [tokens, H, D] tensor; tok0 is its
  // first token, and the maps' batch coordinate is 0.  Dense batch: tok0 = 0, every entry has N tokens.
  const int n_tok = args.seq_len ? args.seq_len[bh / args.H] : args.N;
  const int tok0 = args.seq_start ? args.seq_start[bh / args.H] : 0;
  const int bb_ = args.seq_start ? 0 : bh / args.H;
  const int nseg_own = (n_tok + args.seg_len - 1) / args.seg_len;
  if (seg >= nseg_own) return;  // the grid covers the longest sequence; nothing has been set up yet
  const size_t head_off = (size_t)bb_ * args.sB + (size_t)hh_ * args.sH + (size_t)tok0 * args.sT;
  const int seg_t0 = seg * args.seg_len;
  const int seg_t1 = min(n_tok, seg_t0 + args.seg_len);
  const int nblk = (seg_t1 - seg_t0 + 127) >> 7;
  const float s2 = (float)tab.s2[bh % args.H];
  const bool split_p = (args.precision & 1) != 0;
  const bool split_z = (args.precision & 2) != 0;
  const bool split_c = (args.precision & 4) != 0 && s2 != 0.f;  // lambda == 1: the lo term is identically zero

  if (tid == 0) {
    for (int i = 0; i < F_NUM_BARS; ++i) {
      uint32_t count = 1;
      if (i == F_M4_OK) count = 5;     // one arrival per warp of the P group + the producer's for c
      if (i == F_FULL_AB) count = 2;   // the producer arrives once for b and once for a
      if (i == F_Z_READY) count = 16;
      if (i == F_O_FREE) count = 8;
      mbar_init(&sm.bars[i], count);
    }
    sm.abort = 0;
    fence_mbar_init();
    tma_prefetch_desc(&maps.a);
    tma_prefetch_desc(&maps.b);
    tma_prefetch_desc(&maps.c);
  }
  if (warp == 1) {
    tmem_alloc(&sm.tmem_slot, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = sm.tmem_slot;
  bool issued_mma = false;
  uint32_t mma_elected = 0;
  int armed_ab = 0, armed_c = 0;  // producer: loads armed so far

  if (warp < 4) {
    reg_dec<32>();
    if (warp == 0) {
      // ------------------------------------ TMA producer ------------------------------------
      if (lane == 0) {
        for (int it = 0; it < nblk; ++it) {
          const int t0 = tok0 + seg_t0 + (REV ? (nblk - 1 - it) : it) * 128;  // token coordinate of the maps
          // b is free once M3 of the previous block has read it (DZ_READY), a once M2 has (AB_FREE): each is
          // reloaded as soon as it falls free; both count towards the one barrier M1 of this block waits for
          if (it >= 1) TC_WAIT(F_DZ_READY, (it - 1) & 1, 3);
          mbar_arrive_expect_tx(&sm.bars[F_FULL_AB], 32768);
          tma_load_4d(&sm.b[0][0], &maps.b, &sm.bars[F_FULL_AB], 0, t0, hh_, bb_);
          tma_load_4d(&sm.b[1][0], &maps.b, &sm.bars[F_FULL_AB], 64, t0, hh_, bb_);
          if (it >= 1) TC_WAIT(F_AB_FREE, (it - 1) & 1, 5);
          mbar_arrive_expect_tx(&sm.bars[F_FULL_AB], 32768);
          tma_load_4d(&sm.a[0][0], &maps.a, &sm.bars[F_FULL_AB], 0, t0, hh_, bb_);
          tma_load_4d(&sm.a[1][0], &maps.a, &sm.bars[F_FULL_AB], 64, t0, hh_, bb_);
          armed_ab = it + 1;
          if (it >= 1) TC_WAIT(F_O_READY, (it - 1) & 1, 2);
          mbar_arrive_expect_tx(&sm.bars[F_M4_OK], 32768);
          tma_load_4d(&sm.c[0][0], &maps.c, &sm.bars[F_M4_OK], 0, t0, hh_, bb_);
          tma_load_4d(&sm.c[1][0], &maps.c, &sm.bars[F_M4_OK], 64, t0, hh_, bb_);
          armed_c = it + 1;
        }
      }
    } else if (warp == 1) {
      // ------------------------------------ MMA issuer ------------------------------------
      constexpr uint32_t ID_S = umma_idesc_bf16(128, 128, false, false);   // a (K-major) x b (K-major)
      constexpr uint32_t ID_KN = umma_idesc_bf16(128, 128, false, true);   // K-major or tensor-memory A x MN-major B
      constexpr uint32_t ID_MN = umma_idesc_bf16(128, 128, true, true);    // b^T (MN-major A) x MN-major B
      constexpr uint32_t HI = UMMA_DESC_HI_SBO1024;
      const uint32_t go = elect_one();
      mma_elected = go;
      const uint32_t ak = umma_desc_lo(smem_u32(&sm.a[0][0]), 16), bk = umma_desc_lo(smem_u32(&sm.b[0][0]), 16);
      const uint32_t bm = umma_desc_lo(smem_u32(&sm.b[0][0]), 16384), cm = umma_desc_lo(smem_u32(&sm.c[0][0]), 16384);
      const uint32_t fh = umma_desc_lo(smem_u32(&sm.fc_hi[0][0]), 16384), fl = umma_desc_lo(smem_u32(&sm.fc_lo[0][0]), 16384);
      const uint32_t zh = umma_desc_lo(smem_u32(&sm.z_hi[0][0]), 16384), zl = umma_desc_lo(smem_u32(&sm.z_lo[0][0]), 16384);
      TC_WAIT_WARP(F_FULL_AB, 0, 7);
      tc_fence_after_sync();
      umma_group_ss<8, true, true>(tmem + FCOL_S, ak, bk, HI, ID_S, 0, go);
      issued_mma = true;
      umma_commit_if(&sm.bars[F_S_READY], go);
      for (int it = 0; it < nblk; ++it) {
        const uint32_t par = it & 1;
        // M3: dZ = b^T fc   (the state operand and fc of this block are in place; dZ of the previous block has been read)
        TC_WAIT_WARP(F_Z_READY, par, 12);
        tc_fence_after_sync();
        umma_group_ss<8, false, false>(tmem + FCOL_DZ, bm, fh, HI, ID_MN, 0, go);
        if (split_c) umma_group_ss<8, false, false>(tmem + FCOL_DZ, bm, fl, HI, ID_MN, 1, go);
        umma_commit_if(&sm.bars[F_DZ_READY], go);
        // M2: O_inter = a Z   (the output group has read the accumulators of the previous block)
        if (it > 0) {
          TC_WAIT_WARP(F_O_FREE, (it - 1) & 1, 13);
          tc_fence_after_sync();
        }
        umma_group_ss<8, true, false>(tmem + FCOL_OE, ak, zh, HI, ID_KN, 0, go);
        if (split_z) umma_group_ss<8, true, false>(tmem + FCOL_OE, ak, zl, HI, ID_KN, 1, go);
        umma_commit_if(&sm.bars[F_AB_FREE], go);
        // M4: O_intra = P c
        TC_WAIT_WARP(F_M4_OK, par, 14);  // P is written and c has landed
        tc_fence_after_sync();
        umma_group_ts8(tmem + FCOL_OI, tmem + FCOL_S, cm, HI, ID_KN, 0, go);
        if (split_p) umma_group_ts8(tmem + FCOL_OI, tmem + FCOL_S + 8, cm, HI, ID_KN, 1, go);
        umma_commit_if(&sm.bars[F_O_READY], go);
        // M1 of the next block, over the P just consumed (the tensor pipe runs the products in issue order)
        if (it + 1 < nblk) {
          TC_WAIT_WARP(F_FULL_AB, (it + 1) & 1, 11);
          tc_fence_after_sync();
          umma_group_ss<8, true, true>(tmem + FCOL_S, ak, bk, HI, ID_S, 0, go);
          umma_commit_if(&sm.bars[F_S_READY], go);
        }
      }
    }
  } else if (warp < 8) {
    // ------------------------------------ P group ------------------------------------
    const int q = warp & 3;
    const int r = q * 32 + lane;       // score row
    const uint32_t colS = tmem + ((uint32_t)(q * 32) << 16) + FCOL_S;
    for (int it = 0; it < nblk; ++it) {
      TC_WAIT_WARP(F_S_READY, it & 1, 17);
      tc_fence_after_sync();
#pragma unroll 1
      for (int cc = 0; cc < 4; ++cc) {  // the four 32-column chunks of this warp's 32 rows
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
            // lambda^n on the special-function unit; n < 0 is masked out below
            const float n0 = (float)(REV ? (cc * 32 + hh * 16 - r) : (r - cc * 32 - hh * 16));
#pragma unroll
            for (int x = 0; x < 16; ++x) d[x] = ex2_approx(-s2 * (REV ? n0 + (float)x : n0 - (float)x));
            tmem_ld_wait();
            if (REV ? (cc > q) : (cc < q)) {
              // 32x32 sub-tile wholly inside the causal band: nothing to mask
#pragma unroll
              for (int x = 0; x < 16; ++x) d[x] = __uint_as_float(sreg[x]) * d[x];
            } else {
#pragma unroll
              for (int x = 0; x < 16; ++x) {
                const int j = cc * 32 + hh * 16 + x;
                const int n = REV ? (j - r) : (r - j);
                // a select, not a multiply by zero: masked-out tokens can never leak
                d[x] = (n >= 0) ? __uint_as_float(sreg[x]) * d[x] : 0.f;
              }
            }
            split16(d, h8, l8);
          }
          // in place: the 16 fp32 columns just read become 8 columns of hi pairs + 8 of lo pairs
          tmem_st_x8(colS + cc * 32 + hh * 16, h8);
          if (split_p) tmem_st_x8(colS + cc * 32 + hh * 16 + 8, l8);
        }
      }
      // Reverse walk of a packed batch, the block that holds the sequence's last tokens: the keys past the end lie
      // inside the band, and there they are the next sequence's tokens, not the zero fill a dense batch has.
      if (REV && it == 0 && args.seq_start && seg_t1 - (seg_t0 + (nblk - 1) * 128) < 128)
        clear_keys_past_end(colS, seg_t1 - (seg_t0 + (nblk - 1) * 128));
      tmem_st_wait();
      tc_fence_before_sync();
      WARP_ARRIVE(F_M4_OK);
    }
  } else if (warp >= 12 && warp < 28) {
    // ------------------------------------ Z group ------------------------------------
    reg_inc<72>();
    const int q = warp & 3;
    const int cg = (warp - 12) >> 2;  // which 32 of the 128 state / value columns this warp owns
    const int r = q * 32 + lane;      // token row j of c / state row k of Z
    const uint32_t colDZ = tmem + ((uint32_t)(q * 32) << 16) + FCOL_DZ + cg * 32;
    // this thread's four 16-byte chunks in a swizzled MN-major operand tile (two 64-column chunks of 16 KB)
    const int off_base = (cg >> 1) * (128 * 64) + r * 64;
    const int chunk0 = 4 * (cg & 1);

    // fc = diag(f_state) c is formed 16 bytes (8 columns) at a time: piece i of this thread is chunk (zt & 15) of
    // token row 32 i + (zt >> 4), so a warp reads two whole rows of c (512 contiguous bytes) per load instruction
    // and writes whole 128-byte rows of the operand tile -- row-per-thread loads would touch 32 lines each.
    const int zt = (warp - 12) * 32 + lane;  // 0 .. 511
    const int frow = zt >> 4, fch = zt & 15;
    // decay factor of token row `row` of block iteration `it` in the state update
    auto state_factor = [&](int it, int row) -> float {
      const int t0 = seg_t0 + (REV ? (nblk - 1 - it) : it) * 128;
      const int Cr = min(128, seg_t1 - t0);
      if (row >= Cr) return 0.f;
      return REV ? ex2_approx(-s2 * (float)(row + 1)) : ex2_approx(-s2 * (float)(Cr - 1 - row));
    };
    auto make_fc = [&](const uint4 (&raw)[4], int it) {
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
        // MN-major operand tile: two 64-column chunks of 16 KB, rows of 128 bytes, 16-byte units swizzled by row
        const int off = (fch >> 3) * (128 * 64) + row * 64 + (((fch & 7) ^ (row & 7)) << 3);
        *reinterpret_cast<uint4*>(&sm.fc_hi[0][0] + off) = h;
        if (split_c) *reinterpret_cast<uint4*>(&sm.fc_lo[0][0] + off) = l;
      }
      fence_proxy_async_smem();
    };
    // this thread's four pieces of c straight from global memory; rows beyond N read as zero
    auto c_from_global = [&](int it, uint4 (&raw)[4]) {
      const int t0 = seg_t0 + (REV ? (nblk - 1 - it) : it) * 128;
      const __nv_bfloat16* src = static_cast<const __nv_bfloat16*>(job.c) + head_off + (size_t)(t0 + frow) * args.sT + fch * 8;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (t0 + 32 * i + frow < n_tok) raw[i] = __ldg(reinterpret_cast<const uint4*>(src + (size_t)(32 * i) * args.sT));
        else raw[i] = make_uint4(0u, 0u, 0u, 0u);
      }
    };
    {
      float zreg[32];
      if (job.entry) {
        const float4* src = reinterpret_cast<const float4*>(job.entry + ((size_t)bh * args.nseg + seg) * (128 * 128) +
                                                            (size_t)r * 128 + cg * 32);
#pragma unroll
        for (int x = 0; x < 8; ++x) {
          const float4 v = __ldg(src + x);
          zreg[4 * x] = v.x; zreg[4 * x + 1] = v.y; zreg[4 * x + 2] = v.z; zreg[4 * x + 3] = v.w;
        }
      } else {
#pragma unroll
        for (int x = 0; x < 32; ++x) zreg[x] = 0.f;
      }
      auto write_state_operand = [&]() {
#pragma unroll
        for (int x4 = 0; x4 < 4; ++x4) {
          float x8[8];
#pragma unroll
          for (int x = 0; x < 8; ++x) x8[x] = zreg[x4 * 8 + x];
          uint4 h, l;
          split8(x8, h, l);
          const int off = off_base + (((chunk0 + x4) ^ (r & 7)) << 3);
          *reinterpret_cast<uint4*>(&sm.z_hi[0][0] + off) = h;
          if (split_z) *reinterpret_cast<uint4*>(&sm.z_lo[0][0] + off) = l;
        }
        fence_proxy_async_smem();
      };
      uint4 cnext[4];  // row slice of the next block's c, fetched one block ahead
      c_from_global(0, cnext);
      make_fc(cnext, 0);
      if (nblk > 1) c_from_global(1, cnext);
      write_state_operand();
      WARP_ARRIVE(F_Z_READY);

      for (int it = 0; it < nblk; ++it) {
        const int Cr = min(128, seg_t1 - (seg_t0 + (REV ? (nblk - 1 - it) : it) * 128));
        // ---- Z <- Gamma Z + dZ ----
        TC_WAIT_WARP(F_DZ_READY, it & 1, 22);
        tc_fence_after_sync();
        {
          const float gamma = ex2_approx(-s2 * (float)Cr);
#pragma unroll
          for (int pc = 0; pc < 2; ++pc) {
            uint32_t dh[16];
            tmem_ld_x16(colDZ + pc * 16, dh);
            tmem_ld_wait();
#pragma unroll
            for (int x = 0; x < 16; ++x) zreg[pc * 16 + x] = fmaf(gamma, zreg[pc * 16 + x], __uint_as_float(dh[x]));
          }
          tc_fence_before_sync();  // ordered before the Z_READY arrival below, which M3 of the next block waits for
        }
        if (it + 1 < nblk) {
          // DZ_READY also says M3 of this block is done, so the fc buffer may be rewritten
          make_fc(cnext, it + 1);
          if (it + 2 < nblk) c_from_global(it + 2, cnext);
          // M2 of this block is done: it has read the old state operand
          TC_WAIT_WARP(F_AB_FREE, it & 1, 23);
          write_state_operand();
          WARP_ARRIVE(F_Z_READY);
        }
      }
      const bool last_processed = REV ? (seg == 0) : (seg == nseg_own - 1);
      if (job.final_out && last_processed) {
        float* dst = job.final_out + (size_t)bh * (128 * 128) + (size_t)r * 128 + cg * 32;
#pragma unroll
        for (int x = 0; x < 8; ++x)
          *reinterpret_cast<float4*>(dst + 4 * x) = make_float4(zreg[4 * x], zreg[4 * x + 1], zreg[4 * x + 2], zreg[4 * x + 3]);
      }
    }
  } else {
    // ------------------------------------ O group ------------------------------------
    // out = O_intra + diag(f_out) O_inter, stored straight from registers (there is no shared memory left to stage
    // the rows for a bulk store).  A thread holds one row, so a plain store instruction would touch 32 different
    // lines, and the load/store unit's time per line is what the other groups' shared-memory traffic then waits
    // behind (measured: 2048 line accesses per block cost 2500 clocks of a 9100-clock block, 512 cost 700).  So each
    // 128-byte piece of four rows is first transposed among four lanes with two exchanges by shuffles: afterwards lane
    // g of a quad holds the g-th 32 bytes of its quad's four rows, and one store instruction writes whole 128-byte
    // lines (8 rows per instruction instead of 32 quarter-lines).
    const int q = warp & 3;
    const int r = q * 32 + lane;  // output row
    const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
    const bool b0 = (lane & 1) != 0, b1 = (lane & 2) != 0;
    const int g = lane & 3;
    // columns per 128-byte piece: 32 fp32 or 64 bf16; with the gate the rows stay fp32 until they are stored
    constexpr bool F32ROWS = GATED || sizeof(TOut) == 4;
    constexpr int COLS = F32ROWS ? 32 : 64;
    constexpr int NPIECE = 128 / COLS;             // 4 or 2
    const int ohalf = (warp >= 28) ? 1 : 0;        // warps 8..11 take the first half of the pieces, 28..31 the second
    for (int it = 0; it < nblk; ++it) {
      const int t0 = seg_t0 + (REV ? (nblk - 1 - it) : it) * 128;
      const int Cr = min(128, seg_t1 - t0);
      float f = 0.f;
      if (r < Cr) f = REV ? ex2_approx(-s2 * (float)(Cr - 1 - r)) : ex2_approx(-s2 * (float)(r + 1));
      // element offset of the first row of this thread's quad; the other rows are sT elements apart
      const size_t quad_row0 = head_off + (size_t)(t0 + (r & ~3)) * args.sT;
      unsigned char* const quad_base = static_cast<unsigned char*>(job.out) + quad_row0 * sizeof(TOut) + g * 32;
      // O_READY: every product up to M4 of this block is done
      TC_WAIT_WARP(F_O_READY, it & 1, 25);
      tc_fence_after_sync();
      float srow[4] = {0.f, 0.f, 0.f, 0.f};  // gate: sqrt(128) / ||row|| of the rows of lanes ^ 0..3
      if (GATED) {
        // first pass over the whole row (both halves of the columns: each warp of a pair does this for itself, which
        // costs tensor-memory reads but no exchange between warps): sum of squares of out = O_intra + f O_inter
        float ss = 0.f;
#pragma unroll
        for (int sub = 0; sub < 8; ++sub) {
          uint32_t oi[16], oe[16];
          tmem_ld_x16(lane_addr + FCOL_OI + sub * 16, oi);
          tmem_ld_x16(lane_addr + FCOL_OE + sub * 16, oe);
          tmem_ld_wait();
#pragma unroll
          for (int x = 0; x < 16; ++x) {
            const float v = fmaf(f, __uint_as_float(oe[x]), __uint_as_float(oi[x]));
            ss = fmaf(v, v, ss);
          }
        }
        const float s = ss > 0.f ? rsqrtf(ss * (1.f / 128.f)) : 0.f;
        // rstd has the layout of the token tensors without the feature dimension
        if (job.rstd && ohalf == 0 && r < Cr) job.rstd[(head_off + (size_t)(t0 + r) * args.sT) >> 7] = s;
#pragma unroll
        for (int k = 0; k < 4; ++k) srow[k] = __shfl_xor_sync(0xffffffffu, s, k);
      }
#pragma unroll
      for (int pcl = 0; pcl < NPIECE / 2; ++pcl) {
        const int pc = ohalf * (NPIECE / 2) + pcl;
        uint32_t w[32];  // this thread's 128 bytes of the piece: four 32-byte chunks
#pragma unroll
        for (int sub = 0; sub < COLS / 16; ++sub) {
          const int col = pc * COLS + sub * 16;
          uint32_t oi[16], oe[16];
          tmem_ld_x16(lane_addr + FCOL_OI + col, oi);
          tmem_ld_x16(lane_addr + FCOL_OE + col, oe);
          tmem_ld_wait();
          if (pcl == NPIECE / 2 - 1 && sub == COLS / 16 - 1) {
            tc_fence_before_sync();
            WARP_ARRIVE(F_O_FREE);  // both accumulators are in registers: M2 and M4 of the next block may overwrite them
          }
          if (F32ROWS) {
#pragma unroll
            for (int x = 0; x < 16; ++x)
              w[sub * 16 + x] = __float_as_uint(fmaf(f, __uint_as_float(oe[x]), __uint_as_float(oi[x])));
          } else {
#pragma unroll
            for (int x = 0; x < 8; ++x) {
              const __nv_bfloat162 h = __floats2bfloat162_rn(fmaf(f, __uint_as_float(oe[2 * x]), __uint_as_float(oi[2 * x])),
                                                             fmaf(f, __uint_as_float(oe[2 * x + 1]), __uint_as_float(oi[2 * x + 1])));
              w[sub * 8 + x] = *reinterpret_cast<const uint32_t*>(&h);
            }
          }
        }
        // first exchange, partner lane ^ 1: the even lane keeps chunks 0 and 2 and sends 1 and 3, the odd lane the other way
        // round; afterwards chunk slots hold (own row, chunk b0), (partner row, chunk b0), (own, 2 + b0), (partner, 2 + b0)
#pragma unroll
        for (int x = 0; x < 8; ++x) {
          const uint32_t k0 = b0 ? w[8 + x] : w[x], s0 = b0 ? w[x] : w[8 + x];
          const uint32_t k2 = b0 ? w[24 + x] : w[16 + x], s2x = b0 ? w[16 + x] : w[24 + x];
          w[x] = k0;
          w[8 + x] = __shfl_xor_sync(0xffffffffu, s0, 1);
          w[16 + x] = k2;
          w[24 + x] = __shfl_xor_sync(0xffffffffu, s2x, 1);
        }
        // second exchange, partner lane ^ 2: lanes 0, 1 of the quad keep the chunk-b0 pair and send the chunk-(2 + b0) pair,
        // lanes 2, 3 the other way round; afterwards slot k holds chunk g of the row of lane ^ k
#pragma unroll
        for (int x = 0; x < 8; ++x) {
          const uint32_t k0 = b1 ? w[16 + x] : w[x], s0 = b1 ? w[x] : w[16 + x];
          const uint32_t k1 = b1 ? w[24 + x] : w[8 + x], s1 = b1 ? w[8 + x] : w[24 + x];
          w[x] = k0;
          w[8 + x] = k1;
          w[16 + x] = __shfl_xor_sync(0xffffffffu, s0, 2);
          w[24 + x] = __shfl_xor_sync(0xffffffffu, s1, 2);
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int row_in_quad = g ^ k;  // slot k holds the row of lane ^ k
          if ((r & ~3) + row_in_quad >= Cr) continue;
          if (!GATED) {
            st_global_v8(quad_base + (size_t)row_in_quad * args.sT * sizeof(TOut) + pc * 128, &w[8 * k]);
          } else {
            // slot k: columns pc * 32 + 8 g .. + 8 of that row, still fp32
            const size_t elem = quad_row0 + (size_t)row_in_quad * args.sT + pc * 32 + g * 8;
            const uint4 uraw = __ldg(reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(job.u) + elem));
            const uint32_t uw[4] = {uraw.x, uraw.y, uraw.z, uraw.w};
            uint32_t yv[8];
#pragma unroll
            for (int x = 0; x < 4; ++x) {
              const float2 ug = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&uw[x]));
              yv[2 * x] = __float_as_uint(__uint_as_float(w[8 * k + 2 * x]) * srow[k] * ug.x);
              yv[2 * x + 1] = __float_as_uint(__uint_as_float(w[8 * k + 2 * x + 1]) * srow[k] * ug.y);
            }
            if (sizeof(TOut) == 4) {
              st_global_v8(static_cast<float*>(job.y) + elem, yv);
              if (job.out) st_global_v8(static_cast<float*>(job.out) + elem, &w[8 * k]);
            } else {
              uint4 yp, op;
              uint32_t* ypw = reinterpret_cast<uint32_t*>(&yp);
              uint32_t* opw = reinterpret_cast<uint32_t*>(&op);
#pragma unroll
              for (int x = 0; x < 4; ++x) {
                const __nv_bfloat162 a = __floats2bfloat162_rn(__uint_as_float(yv[2 * x]), __uint_as_float(yv[2 * x + 1]));
                const __nv_bfloat162 b = __floats2bfloat162_rn(__uint_as_float(w[8 * k + 2 * x]), __uint_as_float(w[8 * k + 2 * x + 1]));
                ypw[x] = *reinterpret_cast<const uint32_t*>(&a);
                opw[x] = *reinterpret_cast<const uint32_t*>(&b);
              }
              *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(job.y) + elem) = yp;
              if (job.out) *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(job.out) + elem) = op;
            }
          }
        }
      }
    }
  }

teardown:
  // After an expired wait: drain what this thread started so nothing is in flight when the block exits.
  if (sm.abort) {
    if (warp == 0 && lane == 0) {
      // (a block that gave up between the two halves of an a/b load, or before the P group's arrivals, leaves these
      // phases incomplete; the drain wait is bounded like every other)
      if (armed_ab > 0) drain_wait(&sm.bars[F_FULL_AB], (armed_ab - 1) & 1);
      if (armed_c > 0) drain_wait(&sm.bars[F_M4_OK], (armed_c - 1) & 1);
    }
    if (warp == 1 && mma_elected && issued_mma) {
      umma_commit(&sm.bars[F_DRAIN]);
      drain_wait(&sm.bars[F_DRAIN], 0);
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, TMEM_COLS);
}

template <bool REV, typename TOut, int NJOBS, bool GATED>
cudaError_t launch_full_t(const TcMaps& m0, const TcMaps& m1, const TcArgs& ta, const DecayTable& tab, cudaStream_t stream) {
  const size_t smem = sizeof(FSmem) + 1024;
  auto kern = tc_walk_full_kernel<REV, TOut, NJOBS, GATED>;
  cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (err != cudaSuccess) return err;
  KernelTimer timer(NJOBS == 2 ? K_WALK_PAIR : K_WALK, stream);
  kern<<<(unsigned)(ta.BH * ta.nseg * NJOBS), F_THREADS, smem, stream>>>(m0, m1, ta, tab);
  count_launch();
  return cudaGetLastError();
}
