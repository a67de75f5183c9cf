// fp32 CUDA-core kernels of the generic decayed linear-attention operator
// (see la_common.cuh for the block formulas).  They serve the fp32 workload,
// head dimension 64, and are the full-precision second opinion for the
// tensor-core kernels.  All arithmetic is fp32 FMA with fp32 accumulation;
// bf16 inputs are widened exactly on load.
//
// Block size C = 32 tokens, 256 threads per thread block, one thread block per
// (batch*head, segment).  Shared memory holds the a/b/c tiles (a and b also
// transposed so that every inner loop reads consecutive addresses), the masked
// score tile and the Da x Ec state.
#include "la_common.cuh"

namespace la {

namespace {

constexpr int C = 32;
constexpr int THREADS = 256;
constexpr int AP = C + 4;  // padded row length of the transposed tiles

template <int DA, int EC>
struct Smem {
  float aT[DA][AP];  // aT[k][i] = a[i][k]
  float bT[DA][AP];
  float b[C][DA];
  float c[C][EC];
  float pT[C][AP];  // pT[j][i] = masked score of (row i, column j)
  float Z[DA][EC];
  float dtab[C];     // lambda^n, n = 0..C-1
  float f_out[C];
  float f_state[C];
  float gamma;
};

template <typename TIn, int W>
__device__ __forceinline__ void load_tile_natural(float (*dst)[W], const TIn* src, long long row_stride, int rows_valid) {
  // dst[i][k] = src[i*row_stride + k] for i < rows_valid, else 0
  for (int idx = threadIdx.x; idx < C * W; idx += THREADS) {
    const int i = idx / W, k = idx % W;
    dst[i][k] = (i < rows_valid) ? to_f32<TIn>(src[(size_t)i * row_stride + k]) : 0.f;
  }
}

template <typename TIn, int W>
__device__ __forceinline__ void load_tile_transposed(float (*dstT)[AP], const TIn* src, long long row_stride,
                                                     int rows_valid) {
  for (int idx = threadIdx.x; idx < C * W; idx += THREADS) {
    const int i = idx / W, k = idx % W;
    dstT[k][i] = (i < rows_valid) ? to_f32<TIn>(src[(size_t)i * row_stride + k]) : 0.f;
  }
}

template <typename TIn, typename TOut, int DA, int EC, bool REV>
__global__ void __launch_bounds__(THREADS, 1)
simt_walk_kernel(const OpArgs args, const DecayTable tab) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  Smem<DA, EC>& sm = *reinterpret_cast<Smem<DA, EC>*>(smem_raw);

  const int tid = threadIdx.x;
  const int bh = blockIdx.x / args.nseg;
  const int seg = blockIdx.x % args.nseg;
  const double s2 = tab.s2[bh % args.H];
  const int seg_t0 = seg * args.seg_len;
  const int seg_t1 = min(args.N, seg_t0 + args.seg_len);
  const int nblk = (seg_t1 - seg_t0 + C - 1) / C;

  const size_t head_off = (size_t)(bh / args.H) * args.sB + (size_t)(bh % args.H) * args.sH;
  const long long sT = args.sT;  // elements between consecutive tokens
  const TIn* a = static_cast<const TIn*>(args.a) + head_off;
  const TIn* b = static_cast<const TIn*>(args.b) + head_off;
  const TIn* c = static_cast<const TIn*>(args.c) + head_off;
  TOut* out = static_cast<TOut*>(args.out) + head_off;

  // state entering this segment
  {
    const float* zin = args.entry ? args.entry + ((size_t)bh * args.nseg + seg) * DA * EC : nullptr;
    float* zf = &sm.Z[0][0];
    for (int idx = tid; idx < DA * EC; idx += THREADS) zf[idx] = zin ? zin[idx] : 0.f;
  }
  if (tid < C) sm.dtab[tid] = decay_pow_d(s2, (double)tid);

  for (int ib = 0; ib < nblk; ++ib) {
    const int blk = REV ? (nblk - 1 - ib) : ib;
    const int t0 = seg_t0 + blk * C;
    const int Cr = min(C, seg_t1 - t0);

    if (tid < C) {
      const int i = tid;
      if (!REV) {
        sm.f_out[i] = decay_pow_d(s2, (double)(i + 1));
        sm.f_state[i] = (i < Cr) ? decay_pow_d(s2, (double)(Cr - 1 - i)) : 0.f;
      } else {
        sm.f_out[i] = (i < Cr) ? decay_pow_d(s2, (double)(Cr - 1 - i)) : 0.f;
        sm.f_state[i] = decay_pow_d(s2, (double)(i + 1));
      }
      if (i == 0) sm.gamma = decay_pow_d(s2, (double)Cr);
    }
    load_tile_transposed<TIn, DA>(sm.aT, a + (size_t)t0 * sT, sT, Cr);
    load_tile_transposed<TIn, DA>(sm.bT, b + (size_t)t0 * sT, sT, Cr);
    load_tile_natural<TIn, DA>(sm.b, b + (size_t)t0 * sT, sT, Cr);
    load_tile_natural<TIn, EC>(sm.c, c + (size_t)t0 * sT, sT, Cr);
    __syncthreads();

    // (1) masked scores: pT[j][i] = (a_i . b_j) * D_ij
    {
      const int ty = tid / 16, tx = tid % 16;
      float acc[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
#pragma unroll 8
      for (int k = 0; k < DA; ++k) {
        const float a0 = sm.aT[k][2 * ty], a1 = sm.aT[k][2 * ty + 1];
        const float b0 = sm.bT[k][2 * tx], b1 = sm.bT[k][2 * tx + 1];
        acc[0][0] = fmaf(a0, b0, acc[0][0]);
        acc[0][1] = fmaf(a0, b1, acc[0][1]);
        acc[1][0] = fmaf(a1, b0, acc[1][0]);
        acc[1][1] = fmaf(a1, b1, acc[1][1]);
      }
#pragma unroll
      for (int r = 0; r < 2; ++r)
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {
          const int i = 2 * ty + r, j = 2 * tx + cc;
          const int n = REV ? (j - i) : (i - j);
          // a select, not a multiply by zero: masked-out tokens can never leak
          sm.pT[j][i] = (n >= 0) ? acc[r][cc] * sm.dtab[n] : 0.f;
        }
    }
    __syncthreads();

    // (2)+(3) out = P c + diag(f_out) a Z
    {
      constexpr int EM = EC / 32;
      const int ty = tid / 32, tx = tid % 32;
      const int i0 = 4 * ty;
      float intra[4][EM], inter[4][EM];
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int m = 0; m < EM; ++m) intra[r][m] = inter[r][m] = 0.f;
#pragma unroll 4
      for (int j = 0; j < C; ++j) {
        float p[4], cv[EM];
#pragma unroll
        for (int r = 0; r < 4; ++r) p[r] = sm.pT[j][i0 + r];
#pragma unroll
        for (int m = 0; m < EM; ++m) cv[m] = sm.c[j][tx + 32 * m];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
          for (int m = 0; m < EM; ++m) intra[r][m] = fmaf(p[r], cv[m], intra[r][m]);
      }
#pragma unroll 4
      for (int k = 0; k < DA; ++k) {
        float av[4], zv[EM];
#pragma unroll
        for (int r = 0; r < 4; ++r) av[r] = sm.aT[k][i0 + r];
#pragma unroll
        for (int m = 0; m < EM; ++m) zv[m] = sm.Z[k][tx + 32 * m];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
          for (int m = 0; m < EM; ++m) inter[r][m] = fmaf(av[r], zv[m], inter[r][m]);
      }
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int i = i0 + r;
        if (i < Cr) {
          const float f = sm.f_out[i];
#pragma unroll
          for (int m = 0; m < EM; ++m)
            out[(size_t)(t0 + i) * sT + tx + 32 * m] = from_f32<TOut>(fmaf(f, inter[r][m], intra[r][m]));
        }
      }
    }
    __syncthreads();

    // (4) Z <- Gamma Z + b^T diag(f_state) c
    {
      constexpr int RK = DA / 16, RE = EC / 16;
      const int ty = tid / 16, tx = tid % 16;
      float acc[RK][RE];
#pragma unroll
      for (int r = 0; r < RK; ++r)
#pragma unroll
        for (int m = 0; m < RE; ++m) acc[r][m] = 0.f;
#pragma unroll 2
      for (int j = 0; j < C; ++j) {
        float bv[RK], cv[RE];
        const float f = sm.f_state[j];
#pragma unroll
        for (int r = 0; r < RK; ++r) bv[r] = sm.b[j][ty + 16 * r];
#pragma unroll
        for (int m = 0; m < RE; ++m) cv[m] = f * sm.c[j][tx + 16 * m];
#pragma unroll
        for (int r = 0; r < RK; ++r)
#pragma unroll
          for (int m = 0; m < RE; ++m) acc[r][m] = fmaf(bv[r], cv[m], acc[r][m]);
      }
      const float g = sm.gamma;
#pragma unroll
      for (int r = 0; r < RK; ++r)
#pragma unroll
        for (int m = 0; m < RE; ++m) {
          float& z = sm.Z[ty + 16 * r][tx + 16 * m];
          z = fmaf(g, z, acc[r][m]);
        }
    }
    __syncthreads();
  }

  const bool last_processed = REV ? (seg == 0) : (seg == args.nseg - 1);
  if (args.final_out && last_processed) {
    float* dst = args.final_out + (size_t)bh * DA * EC;
    const float* zf = &sm.Z[0][0];
    for (int idx = tid; idx < DA * EC; idx += THREADS) dst[idx] = zf[idx];
  }
}

// Segment-local state: sum over the segment's tokens of decay-to-segment-edge * b_t c_t^T.
//   forward: edge = last token of the segment, factor lambda^(t1-1-t)
//   reverse: edge = first token, in the gauge the reverse walk carries: lambda^(t-t0+1)
template <typename TIn, int DA, int EC>
struct PreSmem {
  float b[C][DA];
  float c[C][EC];
  float f_state[C];
};

template <typename TIn, int DA, int EC, bool REV>
__global__ void __launch_bounds__(THREADS, 2)
simt_prepass_kernel(const OpArgs args, const DecayTable tab) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  PreSmem<TIn, DA, EC>& sm = *reinterpret_cast<PreSmem<TIn, DA, EC>*>(smem_raw);
  const int tid = threadIdx.x;
  const int bh = blockIdx.x / args.nseg;
  const int seg = blockIdx.x % args.nseg;
  const double s2 = tab.s2[bh % args.H];
  const int seg_t0 = seg * args.seg_len;
  const int seg_t1 = min(args.N, seg_t0 + args.seg_len);
  const int nblk = (seg_t1 - seg_t0 + C - 1) / C;
  const size_t head_off = (size_t)(bh / args.H) * args.sB + (size_t)(bh % args.H) * args.sH;
  const long long sT = args.sT;
  const TIn* b = static_cast<const TIn*>(args.b) + head_off;
  const TIn* c = static_cast<const TIn*>(args.c) + head_off;

  constexpr int RK = DA / 16, RE = EC / 16;
  const int ty = tid / 16, tx = tid % 16;
  float acc[RK][RE];
#pragma unroll
  for (int r = 0; r < RK; ++r)
#pragma unroll
    for (int m = 0; m < RE; ++m) acc[r][m] = 0.f;

  for (int blk = 0; blk < nblk; ++blk) {
    const int t0 = seg_t0 + blk * C;
    const int Cr = min(C, seg_t1 - t0);
    if (tid < C) {
      const int t = t0 + tid;
      float f = 0.f;
      if (tid < Cr) f = REV ? decay_pow_d(s2, (double)(t - seg_t0 + 1)) : decay_pow_d(s2, (double)(seg_t1 - 1 - t));
      sm.f_state[tid] = f;
    }
    load_tile_natural<TIn, DA>(sm.b, b + (size_t)t0 * sT, sT, Cr);
    load_tile_natural<TIn, EC>(sm.c, c + (size_t)t0 * sT, sT, Cr);
    __syncthreads();
#pragma unroll 2
    for (int j = 0; j < C; ++j) {
      float bv[RK], cv[RE];
      const float f = sm.f_state[j];
#pragma unroll
      for (int r = 0; r < RK; ++r) bv[r] = sm.b[j][ty + 16 * r];
#pragma unroll
      for (int m = 0; m < RE; ++m) cv[m] = f * sm.c[j][tx + 16 * m];
#pragma unroll
      for (int r = 0; r < RK; ++r)
#pragma unroll
        for (int m = 0; m < RE; ++m) acc[r][m] = fmaf(bv[r], cv[m], acc[r][m]);
    }
    __syncthreads();
  }
  float* dst = args.local_out + ((size_t)bh * args.nseg + seg) * DA * EC;
#pragma unroll
  for (int r = 0; r < RK; ++r)
#pragma unroll
    for (int m = 0; m < RE; ++m) dst[(size_t)(ty + 16 * r) * EC + tx + 16 * m] = acc[r][m];
}

// Turns segment-local states into the state entering each segment, in place:
//   forward: x_0 = Z_in, x_{p+1} = lambda^(L_p) x_p + local_p
//   reverse: x_{last} = Z_in, x_{p-1} = lambda^(L_p) x_p + local_p
// One thread block per 32x32 tile of one (batch*head) state; each thread carries four elements
// across the short sequential walk over segments.  The optional transposed copy goes through a
// shared-memory tile so that both copies are written with coalesced stores.
constexpr int SCAN_MAX_SEG = 1024;
__global__ void __launch_bounds__(256) scan_kernel(const ScanArgs args, const DecayTable tab) {
  __shared__ float gamma[SCAN_MAX_SEG];
  __shared__ float tile[32][33];
  const int Da = args.Da, Ec = args.Ec, DE = Da * Ec;
  const int bh = blockIdx.x;
  const int tiles_y = Ec / 32;
  const int x0 = (blockIdx.y / tiles_y) * 32, y0 = (blockIdx.y % tiles_y) * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;  // 32 x 8
  const double s2 = tab.s2[bh % args.H];
  // this (batch, head)'s own length and segment count (a packed batch has sequences of different lengths)
  const int n_tok = args.seq_len ? args.seq_len[bh / args.H] : args.N;
  const int nseg = (n_tok + args.seg_len - 1) / args.seg_len;
  for (int p = threadIdx.x; p < nseg; p += 256) {
    const int L = min(n_tok, (p + 1) * args.seg_len) - p * args.seg_len;
    gamma[p] = decay_pow_d(s2, (double)L);
  }
  float z[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int x = x0 + ty + 8 * k, y = y0 + tx;
    z[k] = 0.f;
    if (args.z_in) z[k] = args.z_in[(size_t)bh * DE + (args.z_in_transposed ? (y * Da + x) : (x * Ec + y))];
  }
  __syncthreads();
  // the local state of a segment is fetched one step ahead of its use: the chain over segments is
  // sequential, and this keeps one global-memory round trip out of every step
  auto seg_of = [&](int ip) { return args.reverse ? (nseg - 1 - ip) : ip; };
  float loc[4];
#pragma unroll
  for (int k = 0; k < 4; ++k)
    loc[k] = (nseg > 1) ? args.buf[((size_t)bh * args.nseg + seg_of(0)) * DE + (size_t)(x0 + ty + 8 * k) * Ec + y0 + tx] : 0.f;
  for (int ip = 0; ip < nseg; ++ip) {
    const int p = seg_of(ip);
    const size_t off = ((size_t)bh * args.nseg + p) * DE;
    const bool more = (ip + 1 < nseg);
    float nxt[4] = {0.f, 0.f, 0.f, 0.f};
    if (ip + 2 < nseg) {
      const size_t offn = ((size_t)bh * args.nseg + seg_of(ip + 1)) * DE;
#pragma unroll
      for (int k = 0; k < 4; ++k) nxt[k] = args.buf[offn + (size_t)(x0 + ty + 8 * k) * Ec + y0 + tx];
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) args.buf[off + (size_t)(x0 + ty + 8 * k) * Ec + y0 + tx] = z[k];
    if (args.buf_t) {
#pragma unroll
      for (int k = 0; k < 4; ++k) tile[ty + 8 * k][tx] = z[k];
      __syncthreads();
#pragma unroll
      for (int k = 0; k < 4; ++k)
        args.buf_t[off + (size_t)(y0 + ty + 8 * k) * Da + x0 + tx] = tile[tx][ty + 8 * k];
      __syncthreads();
    }
    if (more) {
      const float g = gamma[p];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        z[k] = fmaf(g, z[k], loc[k]);
        loc[k] = nxt[k];
      }
    }
  }
}

template <typename TIn, typename TOut, int DA, int EC>
cudaError_t launch_walk_t(const OpArgs& args, const DecayTable& tab, cudaStream_t stream) {
  const size_t smem = sizeof(Smem<DA, EC>);
  const dim3 grid((unsigned)(args.BH * args.nseg)), block(THREADS);
  cudaError_t err;
  KernelTimer timer(K_WALK, stream);
  if (args.reverse) {
    auto kern = simt_walk_kernel<TIn, TOut, DA, EC, true>;
    err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    kern<<<grid, block, smem, stream>>>(args, tab);
  } else {
    auto kern = simt_walk_kernel<TIn, TOut, DA, EC, false>;
    err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    kern<<<grid, block, smem, stream>>>(args, tab);
  }
  count_launch();
  return cudaGetLastError();
}

template <typename TIn, int DA, int EC>
cudaError_t launch_prepass_t(const OpArgs& args, const DecayTable& tab, cudaStream_t stream) {
  const size_t smem = sizeof(PreSmem<TIn, DA, EC>);
  const dim3 grid((unsigned)(args.BH * args.nseg)), block(THREADS);
  cudaError_t err;
  KernelTimer timer(K_PREPASS, stream);
  if (args.reverse) {
    auto kern = simt_prepass_kernel<TIn, DA, EC, true>;
    err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    kern<<<grid, block, smem, stream>>>(args, tab);
  } else {
    auto kern = simt_prepass_kernel<TIn, DA, EC, false>;
    err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    kern<<<grid, block, smem, stream>>>(args, tab);
  }
  count_launch();
  return cudaGetLastError();
}

template <int DA, int EC>
cudaError_t launch_walk_dims(const OpArgs& args, const DecayTable& tab, int in_dt, int out_dt,
                             cudaStream_t stream) {
  if (in_dt == DT_F32 && out_dt == DT_F32) return launch_walk_t<float, float, DA, EC>(args, tab, stream);
  if (in_dt == DT_BF16 && out_dt == DT_F32)
    return launch_walk_t<__nv_bfloat16, float, DA, EC>(args, tab, stream);
  if (in_dt == DT_BF16 && out_dt == DT_BF16)
    return launch_walk_t<__nv_bfloat16, __nv_bfloat16, DA, EC>(args, tab, stream);
  return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t launch_simt_walk(const OpArgs& args, const DecayTable& tab, int Da, int Ec, int in_dt,
                             int out_dt, cudaStream_t stream) {
  if (Da == 64 && Ec == 64) return launch_walk_dims<64, 64>(args, tab, in_dt, out_dt, stream);
  if (Da == 128 && Ec == 128) return launch_walk_dims<128, 128>(args, tab, in_dt, out_dt, stream);
  return cudaErrorInvalidValue;
}

cudaError_t launch_simt_prepass(const OpArgs& args, const DecayTable& tab, int Da, int Ec, int in_dt,
                                cudaStream_t stream) {
  if (Da == 64 && Ec == 64) {
    return in_dt == DT_F32 ? launch_prepass_t<float, 64, 64>(args, tab, stream)
                           : launch_prepass_t<__nv_bfloat16, 64, 64>(args, tab, stream);
  }
  if (Da == 128 && Ec == 128) {
    return in_dt == DT_F32 ? launch_prepass_t<float, 128, 128>(args, tab, stream)
                           : launch_prepass_t<__nv_bfloat16, 128, 128>(args, tab, stream);
  }
  return cudaErrorInvalidValue;
}

// dst[m] = src[m]^T for `count` row-major Da x Ec matrices (32x32 tiles through shared memory).
__global__ void __launch_bounds__(256) transpose_states_kernel(const float* __restrict__ src, float* __restrict__ dst,
                                                               int Da, int Ec) {
  __shared__ float tile[32][33];
  const size_t m = blockIdx.x;
  const int tiles_y = Ec / 32;
  const int x0 = (blockIdx.y / tiles_y) * 32, y0 = (blockIdx.y % tiles_y) * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const float* s = src + m * Da * Ec;
  float* d = dst + m * Da * Ec;
#pragma unroll
  for (int k = 0; k < 4; ++k) tile[ty + 8 * k][tx] = s[(size_t)(x0 + ty + 8 * k) * Ec + y0 + tx];
  __syncthreads();
#pragma unroll
  for (int k = 0; k < 4; ++k) d[(size_t)(y0 + ty + 8 * k) * Da + x0 + tx] = tile[tx][ty + 8 * k];
}

cudaError_t launch_transpose_states(const float* src, float* dst, long count, int Da, int Ec, cudaStream_t stream) {
  if ((Da % 32) != 0 || (Ec % 32) != 0 || count < 1 || count > 2147483647L) return cudaErrorInvalidValue;
  const dim3 grid((unsigned)count, (unsigned)((Da / 32) * (Ec / 32)));
  KernelTimer timer(K_SCAN, stream);
  transpose_states_kernel<<<grid, 256, 0, stream>>>(src, dst, Da, Ec);
  count_launch();
  return cudaGetLastError();
}

// One thread per four consecutive state elements; the pieces are few (ranks of a sequence-parallel group, or the
// segments of one chunk), so the sequential chain is short and every access is a coalesced 16-byte one.
__global__ void __launch_bounds__(256) chain_kernel(const ChainArgs args, const DecayTable tab) {
  const long per_head = args.DE / 4;
  const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (long)args.BH * per_head) return;
  const int bh = (int)(i / per_head);
  const size_t e0 = (size_t)(i % per_head) * 4;
  const double s2 = tab.s2[bh % args.H];
  float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
  if (args.z_in) z = *reinterpret_cast<const float4*>(args.z_in + (size_t)bh * args.DE + e0);
  int j = args.first;
  for (int n = 0; n < args.count; ++n, j += args.step) {
    const long long t0 = (long long)j * args.piece_len;
    const long long t1 = (t0 + args.piece_len < args.N) ? t0 + args.piece_len : args.N;
    const float g = decay_pow_d(s2, (double)(t1 - t0));
    const float4 x = *reinterpret_cast<const float4*>(args.src + (size_t)j * args.stride_j + (size_t)bh * args.stride_bh + e0);
    z.x = fmaf(g, z.x, x.x);
    z.y = fmaf(g, z.y, x.y);
    z.z = fmaf(g, z.z, x.z);
    z.w = fmaf(g, z.w, x.w);
  }
  *reinterpret_cast<float4*>(args.out + (size_t)bh * args.DE + e0) = z;
}

cudaError_t launch_chain(const ChainArgs& args, const DecayTable& tab, cudaStream_t stream) {
  if (args.DE % 4 != 0 || args.BH < 1 || args.count < 0 || args.piece_len < 1) return cudaErrorInvalidValue;
  const long threads = (long)args.BH * (args.DE / 4);
  KernelTimer timer(K_SCAN, stream);
  chain_kernel<<<(unsigned)((threads + 255) / 256), 256, 0, stream>>>(args, tab);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_scan(const ScanArgs& args, const DecayTable& tab, cudaStream_t stream) {
  if (args.nseg > SCAN_MAX_SEG || (args.Da % 32) != 0 || (args.Ec % 32) != 0) return cudaErrorInvalidValue;
  const dim3 grid((unsigned)args.BH, (unsigned)((args.Da / 32) * (args.Ec / 32)));
  KernelTimer timer(K_SCAN, stream);
  scan_kernel<<<grid, 256, 0, stream>>>(args, tab);
  count_launch();
  return cudaGetLastError();
}

}  // namespace la
