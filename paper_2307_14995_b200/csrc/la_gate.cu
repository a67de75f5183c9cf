// SimpleRMSNorm followed by the gate (Eq. 3 "Gated Linear Attention" with Eq. 8 "SimpleRMSNorm") as stand-alone
// row kernels:   y = o / (||o||_2 / sqrt(e)) (.) u   per row of e values, and the gradients of <y, dy>
//   du = dy (.) n,   do = s (g - n (n . g) / e)   with  n = o s,  s = sqrt(e) / ||o||_2,  g = dy (.) u.
// A row with ||o||_2 = 0 gives y = 0 and zero gradients (Eq. 8 has no epsilon).
//
// The forward kernel is the fallback of la_fwd_gated where the epilogue is not fused into the walk kernel
// (d = 64, the fp32 path, outputs aligned to 16 bytes only); the backward kernel is la_gate_bwd.  Both are
// bound by HBM: e / 4 lanes share a row, each lane moves 4 consecutive elements with one vector access per
// tensor, and the row sums are reduced with shuffles.
#include "la_common.cuh"

namespace la {
namespace {

// sum over the e / 4 lanes that share a row (a power of two <= 32)
__device__ __forceinline__ float row_sum(float x, int lanes) {
  for (int o = lanes >> 1; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

// TO: dtype of o and y (the library's out_dtype), TU: dtype of u (in_dtype).  o and y may be the same buffer.
template <typename TO, typename TU>
__global__ void __launch_bounds__(256) norm_gate_fwd_kernel(const TO* o, const TU* __restrict__ u, TO* y,
                                                            float* __restrict__ rstd, long rows, int e) {
  const int lanes = e >> 2;  // lanes per row: 16 or 32
  const long gthread = (long)blockIdx.x * blockDim.x + threadIdx.x;
  const long nthreads = (long)gridDim.x * blockDim.x;
  const long total = rows * lanes;
  const long padded = (total + 31) / 32 * 32;  // whole warps stay together in the shuffles
  for (long i = gthread; i < padded; i += nthreads) {
    const bool valid = i < total;
    const long row = valid ? i / lanes : 0;
    const int c0 = valid ? (int)(i % lanes) * 4 : 0;
    float x[4] = {0.f, 0.f, 0.f, 0.f}, g[4] = {0.f, 0.f, 0.f, 0.f};
    if (valid) {
      Vec4<TO>::load(o + row * e + c0, x);
      Vec4<TU>::load(u + row * e + c0, g);
    }
    const float ss = row_sum(x[0] * x[0] + x[1] * x[1] + x[2] * x[2] + x[3] * x[3], lanes);
    const float s = ss > 0.f ? rsqrtf(ss / (float)e) : 0.f;
    if (rstd && valid && c0 == 0) rstd[row] = s;
#pragma unroll
    for (int k = 0; k < 4; ++k) x[k] = x[k] * s * g[k];
    if (valid) Vec4<TO>::store(y + row * e + c0, x);
  }
}

// o in TO (out_dtype); u, dy and d_o in TU (in_dtype: d_o feeds la_bwd); d_u in TO.
template <typename TO, typename TU>
__global__ void __launch_bounds__(256) norm_gate_bwd_kernel(const TO* __restrict__ o, const TU* __restrict__ u,
                                                            const TU* __restrict__ dy, TU* __restrict__ d_o,
                                                            TO* __restrict__ d_u, long rows, int e) {
  const int lanes = e >> 2;
  const long gthread = (long)blockIdx.x * blockDim.x + threadIdx.x;
  const long nthreads = (long)gridDim.x * blockDim.x;
  const long total = rows * lanes;
  const long padded = (total + 31) / 32 * 32;
  const float inv_e = 1.f / (float)e;
  for (long i = gthread; i < padded; i += nthreads) {
    const bool valid = i < total;
    const long row = valid ? i / lanes : 0;
    const int c0 = valid ? (int)(i % lanes) * 4 : 0;
    float x[4] = {0.f, 0.f, 0.f, 0.f}, uu[4] = {0.f, 0.f, 0.f, 0.f}, gy[4] = {0.f, 0.f, 0.f, 0.f};
    if (valid) {
      Vec4<TO>::load(o + row * e + c0, x);
      Vec4<TU>::load(u + row * e + c0, uu);
      Vec4<TU>::load(dy + row * e + c0, gy);
    }
    const float ss = row_sum(x[0] * x[0] + x[1] * x[1] + x[2] * x[2] + x[3] * x[3], lanes);
    const float s = ss > 0.f ? rsqrtf(ss * inv_e) : 0.f;
    float n[4], g[4], part = 0.f;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      n[k] = x[k] * s;
      g[k] = gy[k] * uu[k];
      part = fmaf(n[k], g[k], part);
    }
    const float ng = row_sum(part, lanes) * inv_e;
    float dox[4], dux[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      dux[k] = gy[k] * n[k];
      dox[k] = s * (g[k] - n[k] * ng);
    }
    if (valid) {
      Vec4<TU>::store(d_o + row * e + c0, dox);
      Vec4<TO>::store(d_u + row * e + c0, dux);
    }
  }
}

unsigned grid_for(long rows, int e) {
  const long total = rows * (e / 4);
  long blocks = (total + 255) / 256;
  const long cap = 148L * 16;  // a few waves of a grid-stride loop
  return (unsigned)(blocks < cap ? blocks : cap);
}

}  // namespace

cudaError_t launch_norm_gate_fwd(const void* o, const void* u, void* y, float* rstd, long rows, int e, int in_dt,
                                 int out_dt, cudaStream_t stream) {
  if ((e != 64 && e != 128) || rows < 1) return cudaErrorInvalidValue;
  KernelTimer timer(K_GATE, stream);
  const unsigned grid = grid_for(rows, e);
  if (out_dt == DT_F32 && in_dt == DT_F32)
    norm_gate_fwd_kernel<float, float><<<grid, 256, 0, stream>>>((const float*)o, (const float*)u, (float*)y, rstd, rows, e);
  else if (out_dt == DT_F32)
    norm_gate_fwd_kernel<float, __nv_bfloat16><<<grid, 256, 0, stream>>>((const float*)o, (const __nv_bfloat16*)u, (float*)y,
                                                                        rstd, rows, e);
  else if (in_dt == DT_BF16)
    norm_gate_fwd_kernel<__nv_bfloat16, __nv_bfloat16><<<grid, 256, 0, stream>>>(
        (const __nv_bfloat16*)o, (const __nv_bfloat16*)u, (__nv_bfloat16*)y, rstd, rows, e);
  else
    return cudaErrorInvalidValue;
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_norm_gate_bwd(const void* o, const void* u, const void* dy, void* d_o, void* d_u, long rows, int e,
                                 int in_dt, int out_dt, cudaStream_t stream) {
  if ((e != 64 && e != 128) || rows < 1) return cudaErrorInvalidValue;
  KernelTimer timer(K_GATE, stream);
  const unsigned grid = grid_for(rows, e);
  if (out_dt == DT_F32 && in_dt == DT_F32)
    norm_gate_bwd_kernel<float, float><<<grid, 256, 0, stream>>>((const float*)o, (const float*)u, (const float*)dy,
                                                                 (float*)d_o, (float*)d_u, rows, e);
  else if (out_dt == DT_F32)
    norm_gate_bwd_kernel<float, __nv_bfloat16><<<grid, 256, 0, stream>>>(
        (const float*)o, (const __nv_bfloat16*)u, (const __nv_bfloat16*)dy, (__nv_bfloat16*)d_o, (float*)d_u, rows, e);
  else if (in_dt == DT_BF16)
    norm_gate_bwd_kernel<__nv_bfloat16, __nv_bfloat16><<<grid, 256, 0, stream>>>(
        (const __nv_bfloat16*)o, (const __nv_bfloat16*)u, (const __nv_bfloat16*)dy, (__nv_bfloat16*)d_o,
        (__nv_bfloat16*)d_u, rows, e);
  else
    return cudaErrorInvalidValue;
  count_launch();
  return cudaGetLastError();
}

}  // namespace la
