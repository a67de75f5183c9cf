// Recurrent decode (iterations of Algorithm 2) for all (batch, head) pairs:
//   kv <- lambda kv + k v^T,   o <- kv^T q,   kv fp32 [BH, d, e] updated in place,
// for T >= 1 consecutive tokens per launch (q, k [BH, T, d], v, o [BH, T, e]): the state is read once, kept in
// registers over the T tokens and written once, so a few tokens decoded together (speculative or chunked
// decoding) cost one pass over the state instead of T.
//
// The step moves 2*d*e*4 bytes of state per (b,h) against 5*d*e flops, so it is
// bound by HBM bandwidth and runs on the plain fp32 ALUs.  One thread block owns
// one (b,h) state: every thread keeps a fixed group of four value columns and
// strides over the key rows, so a warp touches whole 512-byte rows with 16-byte
// accesses, all row loads are issued before the first use, and the column sums
// for o are reduced inside the block (no atomics, bitwise reproducible).
#include "la_common.cuh"

namespace la {
namespace {

constexpr int THREADS = 256;

template <typename TIn, typename TOut, int D, int E>
__global__ void __launch_bounds__(THREADS)
decode_kernel(const TIn* __restrict__ q, const TIn* __restrict__ k, const TIn* __restrict__ v,
              float* __restrict__ kv, TOut* __restrict__ o, int H, int T, long long sT, long long sH, long long sB,
              const DecayTable tab) {
  constexpr int LPR = E / 4;              // lanes per state row (float4 each)
  constexpr int RPP = THREADS / LPR;      // rows per pass
  constexpr int PASSES = D / RPP;
  static_assert(D % RPP == 0 && THREADS % LPR == 0, "shape");

  __shared__ float sq[D];
  __shared__ float sk[D];
  __shared__ float4 red[RPP][LPR];

  const int bh = blockIdx.x;
  const int tid = threadIdx.x;
  const float lam = (float)exp2(-tab.s2[bh % H]);
  const int col4 = tid % LPR;
  const int row0 = tid / LPR;

  float4* state = reinterpret_cast<float4*>(kv + (size_t)bh * D * E);
  const size_t head_off = (size_t)(bh / H) * sB + (size_t)(bh % H) * sH;  // token t of this (b,h): + t * sT

  // issue every state load first: PASSES independent 16-byte loads per thread
  float4 s[PASSES];
#pragma unroll
  for (int p = 0; p < PASSES; ++p) s[p] = __ldcs(&state[(size_t)(row0 + p * RPP) * LPR + col4]);

  for (int t = 0; t < T; ++t) {
    if (tid < D) {
      sq[tid] = to_f32<TIn>(q[head_off + (size_t)t * sT + tid]);
      sk[tid] = to_f32<TIn>(k[head_off + (size_t)t * sT + tid]);
    }
    float4 vv;
    {
      const TIn* vp = v + head_off + (size_t)t * sT + 4 * col4;
      vv = make_float4(to_f32<TIn>(vp[0]), to_f32<TIn>(vp[1]), to_f32<TIn>(vp[2]), to_f32<TIn>(vp[3]));
    }
    __syncthreads();

    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int p = 0; p < PASSES; ++p) {
      const int i = row0 + p * RPP;
      const float ki = sk[i], qi = sq[i];
      float4 x = s[p];
      x.x = fmaf(lam, x.x, ki * vv.x);
      x.y = fmaf(lam, x.y, ki * vv.y);
      x.z = fmaf(lam, x.z, ki * vv.z);
      x.w = fmaf(lam, x.w, ki * vv.w);
      s[p] = x;
      if (t == T - 1) __stcs(&state[(size_t)i * LPR + col4], x);  // the state leaves once, after the last token
      acc.x = fmaf(x.x, qi, acc.x);
      acc.y = fmaf(x.y, qi, acc.y);
      acc.z = fmaf(x.z, qi, acc.z);
      acc.w = fmaf(x.w, qi, acc.w);
    }
    red[row0][col4] = acc;
    __syncthreads();
    if (tid < LPR) {
      float4 sum = red[0][tid];
#pragma unroll
      for (int r = 1; r < RPP; ++r) {
        const float4 u = red[r][tid];
        sum.x += u.x; sum.y += u.y; sum.z += u.z; sum.w += u.w;
      }
      TOut* op = o + head_off + (size_t)t * sT + 4 * tid;
      op[0] = from_f32<TOut>(sum.x);
      op[1] = from_f32<TOut>(sum.y);
      op[2] = from_f32<TOut>(sum.z);
      op[3] = from_f32<TOut>(sum.w);
    }
    // (the next token's q, k are written to sq, sk only after every thread has passed the barrier above; red is
    // rewritten only after the next barrier)
  }
}

template <typename TIn, typename TOut, int D, int E>
cudaError_t launch_t(const void* q, const void* k, const void* v, float* kv, void* o, int BH, int H, int T,
                     long long sT, long long sH, long long sB, const DecayTable& tab, cudaStream_t stream) {
  KernelTimer timer(K_DECODE, stream);
  decode_kernel<TIn, TOut, D, E><<<BH, THREADS, 0, stream>>>(
      static_cast<const TIn*>(q), static_cast<const TIn*>(k), static_cast<const TIn*>(v), kv,
      static_cast<TOut*>(o), H, T, sT, sH, sB, tab);
  count_launch();
  return cudaGetLastError();
}

template <int D, int E>
cudaError_t launch_dims(const void* q, const void* k, const void* v, float* kv, void* o, int BH, int H, int T,
                        int in_dt, int out_dt, long long sT, long long sH, long long sB, const DecayTable& tab,
                        cudaStream_t stream) {
  if (in_dt == DT_F32 && out_dt == DT_F32)
    return launch_t<float, float, D, E>(q, k, v, kv, o, BH, H, T, sT, sH, sB, tab, stream);
  if (in_dt == DT_BF16 && out_dt == DT_F32)
    return launch_t<__nv_bfloat16, float, D, E>(q, k, v, kv, o, BH, H, T, sT, sH, sB, tab, stream);
  if (in_dt == DT_BF16 && out_dt == DT_BF16)
    return launch_t<__nv_bfloat16, __nv_bfloat16, D, E>(q, k, v, kv, o, BH, H, T, sT, sH, sB, tab, stream);
  return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t launch_decode(const void* q, const void* k, const void* v, float* kv, void* o, int BH,
                          int H, int T, int d, int e, int in_dt, int out_dt, long long sT, long long sH, long long sB,
                          const DecayTable& tab, cudaStream_t stream) {
  if (T < 1) return cudaErrorInvalidValue;
  if (d == 64 && e == 64) return launch_dims<64, 64>(q, k, v, kv, o, BH, H, T, in_dt, out_dt, sT, sH, sB, tab, stream);
  if (d == 128 && e == 128)
    return launch_dims<128, 128>(q, k, v, kv, o, BH, H, T, in_dt, out_dt, sT, sH, sB, tab, stream);
  return cudaErrorInvalidValue;
}

}  // namespace la
