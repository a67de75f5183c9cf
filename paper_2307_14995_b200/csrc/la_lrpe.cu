// LRPE-d (Eq. 1): the decayed score times a learnable rotation of the relative position,
//   a_ts = lambda^(t-s) sum_i q_t[i] k_s[i] cos(theta[h][i] (t - s)),   s <= t   (real part of the printed form).
// The rotation splits into one factor per position, cos(a - b) = cos a cos b + sin a sin b, so with the features
//   x_c[t] = x[t] cos(theta t),  x_s[t] = x[t] sin(theta t)       (t the absolute position)
// the score is q_c.k_c + q_s.k_s and the output is the sum of two runs of the decayed operator,
//   O = op(Q_c, K_c, V) + op(Q_s, K_s, V),
// each with its own d x e state (the state of the doubled feature dimension 2d, stored as [2,B,H,d,e]).
// This file holds the element-wise kernels around those two runs -- the feature map, the sum of the two
// results, the chain rule back through the feature map including the gradient of the angles -- and the
// entry points that sequence them with la_fwd / la_bwd on the caller's stream.
//
// Angles: theta t is formed in double and reduced to [-pi, pi] before the fp32 sincos, so positions far into a
// long context lose nothing to the size of the product.  The gradient of theta is a position-weighted sum,
//   dtheta_i = sum_t t (q_c gs - q_s gc)_i + the same for k,     gc, gs = gradients of the two feature halves,
// whose two parts cancel down to the relative-position result; per-tile partial sums are written out and
// added in a fixed order (double) by a second kernel, so the result is reproducible bit for bit.
#include <cstdint>
#include <initializer_list>

#include "../../include/la.h"
#include "la_common.cuh"

namespace la {
namespace {

constexpr int TILE_TOKENS = 256;  // tokens of one (b,h) per block in the gradient kernel

__device__ __forceinline__ void rotation(float theta, long long pos, float* c, float* s) {
  double a = (double)theta * (double)pos;
  a -= 6.283185307179586476925 * rint(a * 0.159154943091895335769);
  sincosf((float)a, s, c);
}

struct Geometry {   // where token t of (b,h) lives: element offset b*sB + h*sH + t*sT (+ feature)
  long long sT, sH, sB;
  int B, H, N, d;
};

// x -> x cos(theta t), x sin(theta t), same layout as x.  d/4 lanes share a token (four features each) and walk a
// run of RUN consecutive tokens of one (b,h): the first angle of the run is exact (double product, reduced), the
// following ones come from rotating (cos, sin) by the feature's own step angle, four multiply-adds instead of a
// sincos per element; over RUN = 16 steps the recurrence drifts by a few 1e-7, far below the bf16 features' 2^-9.
constexpr int RUN = 16;

template <typename T>
__global__ void __launch_bounds__(256) lrpe_feature_kernel(const T* __restrict__ x, const float* __restrict__ theta,
                                                           T* __restrict__ xc, T* __restrict__ xs, Geometry g,
                                                           long long pos0) {
  const int lanes = g.d >> 2;
  const int groups = 256 / lanes;
  const int lane = threadIdx.x % lanes, grp = threadIdx.x / lanes;
  const int c0 = lane * 4;
  const int runs_per_head = (g.N + RUN - 1) / RUN;
  const long total = (long)g.B * g.H * runs_per_head;
  for (long run = (long)blockIdx.x * groups + grp; run < total; run += (long)gridDim.x * groups) {
    const int t_first = (int)(run % runs_per_head) * RUN;
    const long bh = run / runs_per_head;
    const int h = (int)(bh % g.H), b = (int)(bh / g.H);
    const float4 th = *reinterpret_cast<const float4*>(theta + (size_t)h * g.d + c0);
    const float tv[4] = {th.x, th.y, th.z, th.w};
    float c[4], s[4], cs[4], ss[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      rotation(tv[k], pos0 + t_first, &c[k], &s[k]);
      rotation(tv[k], 1, &cs[k], &ss[k]);
    }
    const size_t base = (size_t)b * g.sB + (size_t)h * g.sH + c0;
    const int t_end = min(g.N, t_first + RUN);
    for (int t = t_first; t < t_end; ++t) {
      const size_t off = base + (size_t)t * g.sT;
      float v[4], oc[4], os[4];
      Vec4<T>::load(x + off, v);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        oc[k] = v[k] * c[k];
        os[k] = v[k] * s[k];
        const float cn = fmaf(c[k], cs[k], -s[k] * ss[k]);
        s[k] = fmaf(s[k], cs[k], c[k] * ss[k]);
        c[k] = cn;
      }
      Vec4<T>::store(xc + off, oc);
      Vec4<T>::store(xs + off, os);
    }
  }
}

// dst = a + b (fp32 operands; dst may be a itself), four elements per thread.
template <typename TOut>
__global__ void __launch_bounds__(256) lrpe_sum_kernel(const float* a, const float* __restrict__ b, TOut* dst, long n4) {
  const long nthreads = (long)gridDim.x * blockDim.x;
  for (long i = (long)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += nthreads) {
    float x[4], y[4];
    Vec4<float>::load(a + 4 * i, x);
    Vec4<float>::load(b + 4 * i, y);
#pragma unroll
    for (int k = 0; k < 4; ++k) x[k] += y[k];
    Vec4<TOut>::store(dst + 4 * i, x);
  }
}

// Chain rule through the feature map for one of q, k:
//   dx = gc cos + gs sin,     part[(bh, tile), i] = sum over the tile's tokens of t (x cos gs - x sin gc)_i.
// Block = one tile of TILE_TOKENS tokens of one (b,h); d/4 lanes per token, 256/(d/4) tokens per pass.
template <typename TIn, typename TOut>
__global__ void __launch_bounds__(256) lrpe_grad_kernel(const TIn* __restrict__ x, const float* __restrict__ gc,
                                                        const float* __restrict__ gs, const float* __restrict__ theta,
                                                        TOut* __restrict__ dx, float* __restrict__ part, Geometry g,
                                                        long long pos0, int ntiles) {
  __shared__ float red[2048];  // [tokens per pass][d]: 8 x 128 or 16 x 64
  const int lanes = g.d >> 2;
  const int rows_per_pass = 256 / lanes;  // 8 (d = 128) or 16 (d = 64)
  const int lane = threadIdx.x % lanes, row0 = threadIdx.x / lanes;
  const int tile = blockIdx.x % ntiles, bh = blockIdx.x / ntiles;
  const int h = bh % g.H, b = bh / g.H;
  const int c0 = lane * 4;
  const size_t head_off = (size_t)b * g.sB + (size_t)h * g.sH + c0;
  const float4 th = *reinterpret_cast<const float4*>(theta + (size_t)h * g.d + c0);
  const float tv[4] = {th.x, th.y, th.z, th.w};
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  // each group of d/4 lanes walks its own run of consecutive tokens, rotating (cos, sin) from an exact start
  const int run = TILE_TOKENS / rows_per_pass;  // 32 (d = 128) or 16 (d = 64)
  const int t_first = tile * TILE_TOKENS + row0 * run;
  const int t_end = min(g.N, t_first + run);
  float c[4], s[4], cs[4], ss[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    rotation(tv[k], pos0 + t_first, &c[k], &s[k]);
    rotation(tv[k], 1, &cs[k], &ss[k]);
  }
  for (int t = t_first; t < t_end; ++t) {
    const size_t off = head_off + (size_t)t * g.sT;
    float v[4], a[4], bb[4], o[4];
    Vec4<TIn>::load(x + off, v);
    Vec4<float>::load(gc + off, a);
    Vec4<float>::load(gs + off, bb);
    const float pos = (float)(pos0 + t);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      o[k] = fmaf(a[k], c[k], bb[k] * s[k]);
      acc[k] = fmaf(pos, v[k] * (c[k] * bb[k] - s[k] * a[k]), acc[k]);
      const float cn = fmaf(c[k], cs[k], -s[k] * ss[k]);
      s[k] = fmaf(s[k], cs[k], c[k] * ss[k]);
      c[k] = cn;
    }
    Vec4<TOut>::store(dx + off, o);
  }
  // fixed-order sum over the token rows of the block
#pragma unroll
  for (int k = 0; k < 4; ++k) red[row0 * g.d + c0 + k] = acc[k];
  __syncthreads();
  if (threadIdx.x < g.d) {
    float s = 0.f;
    for (int r = 0; r < rows_per_pass; ++r) s += red[r * g.d + threadIdx.x];
    part[((size_t)bh * ntiles + tile) * g.d + threadIdx.x] = s;
  }
}

// dtheta[h][i] = sum over the batch and the tiles of the two partial arrays, in double, in an order that depends on
// the shape only (32 slices per feature: slice l adds the partials l, l + 32, ...; the slices are then added in
// order through shared memory), so the result is reproducible bit for bit.  Eight consecutive features per block.
__global__ void __launch_bounds__(256) lrpe_theta_reduce_kernel(const float* __restrict__ part_q,
                                                                const float* __restrict__ part_k,
                                                                float* __restrict__ dtheta, int B, int H, int ntiles, int d) {
  const int slice = threadIdx.x >> 3, fi = threadIdx.x & 7;
  const int idx = blockIdx.x * 8 + fi;  // feature index in [0, H*d)
  __shared__ double red[32][8];
  double s = 0.0;
  if (idx < H * d) {
    const int h = idx / d, i = idx % d;
    const int n = B * ntiles;
    for (int j = slice; j < n; j += 32) {
      const int b = j / ntiles, tl = j % ntiles;
      const size_t at = ((size_t)(b * H + h) * ntiles + tl) * d + i;
      s += (double)part_q[at] + (double)part_k[at];
    }
  }
  red[slice][fi] = s;
  __syncthreads();
  if (slice == 0 && idx < H * d) {
    double t = 0.0;
    for (int j = 0; j < 32; ++j) t += red[j][fi];
    dtheta[idx] = (float)t;
  }
}

unsigned grid_for(long threads_needed) {
  long blocks = (threads_needed + 255) / 256;
  const long cap = 148L * 16;
  return (unsigned)(blocks < 1 ? 1 : (blocks < cap ? blocks : cap));
}

Geometry geometry(const la_shape* s) {
  Geometry g;
  g.B = s->B; g.H = s->H; g.N = s->N; g.d = s->d;
  if (s->layout == LA_LAYOUT_BNHD) {
    g.sT = (long long)s->H * s->d; g.sH = s->d; g.sB = (long long)s->N * s->H * s->d;
  } else {
    g.sT = s->d; g.sH = (long long)s->N * s->d; g.sB = (long long)s->H * s->N * s->d;
  }
  return g;
}

cudaError_t run_features(const la_shape* s, const void* x, const float* theta, void* xc, void* xs, long long pos0,
                         cudaStream_t st) {
  KernelTimer timer(K_LRPE, st);
  const Geometry g = geometry(s);
  const unsigned grid = grid_for((long)s->B * s->H * ((s->N + RUN - 1) / RUN) * (s->d / 4));
  if (s->in_dtype == LA_BF16)
    lrpe_feature_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)x, theta, (__nv_bfloat16*)xc,
                                                            (__nv_bfloat16*)xs, g, pos0);
  else
    lrpe_feature_kernel<float><<<grid, 256, 0, st>>>((const float*)x, theta, (float*)xc, (float*)xs, g, pos0);
  count_launch();
  return cudaGetLastError();
}

cudaError_t run_sum(const la_shape* s, const float* a, const float* b, void* dst, cudaStream_t st) {
  KernelTimer timer(K_LRPE, st);
  const long n4 = (long)s->B * s->H * s->N * s->e / 4;
  const unsigned grid = grid_for(n4);
  if (s->out_dtype == LA_BF16)
    lrpe_sum_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(a, b, (__nv_bfloat16*)dst, n4);
  else
    lrpe_sum_kernel<float><<<grid, 256, 0, st>>>(a, b, (float*)dst, n4);
  count_launch();
  return cudaGetLastError();
}

cudaError_t run_grad(const la_shape* s, const void* x, const float* gc, const float* gs, const float* theta, void* dx,
                     float* part, long long pos0, int ntiles, cudaStream_t st) {
  KernelTimer timer(K_LRPE, st);
  const Geometry g = geometry(s);
  const unsigned grid = (unsigned)((long)s->B * s->H * ntiles);
  const bool ib = s->in_dtype == LA_BF16, ob = s->out_dtype == LA_BF16;
  if (ib && ob)
    lrpe_grad_kernel<__nv_bfloat16, __nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)x, gc, gs, theta,
                                                                        (__nv_bfloat16*)dx, part, g, pos0, ntiles);
  else if (ib)
    lrpe_grad_kernel<__nv_bfloat16, float><<<grid, 256, 0, st>>>((const __nv_bfloat16*)x, gc, gs, theta, (float*)dx,
                                                                part, g, pos0, ntiles);
  else if (!ob)
    lrpe_grad_kernel<float, float><<<grid, 256, 0, st>>>((const float*)x, gc, gs, theta, (float*)dx, part, g, pos0,
                                                        ntiles);
  else
    return cudaErrorInvalidValue;
  count_launch();
  return cudaGetLastError();
}

size_t up256(size_t x) { return (x + 255) / 256 * 256; }

// What la_fwd / la_bwd would reject, checked before the feature kernels are launched.
bool plain_args_ok(const la_shape* s, const float* lambda_host, std::initializer_list<const void*> ptrs) {
  if (!lambda_host) return false;
  for (int h = 0; h < s->H; ++h)
    if (!(lambda_host[h] > 0.f && lambda_host[h] <= 1.f)) return false;
  for (const void* p : ptrs)
    if (reinterpret_cast<uintptr_t>(p) & 15u) return false;
  return true;
}

// Workspace layout shared by the size query and the two entry points.
struct Carve {
  size_t feat;       // bytes of one feature tensor (in_dtype)
  size_t f32;        // bytes of one fp32 temporary of the tensors' size
  size_t part;       // bytes of one partial-sum array for dtheta
  size_t op;         // workspace of the inner la_fwd / la_bwd
  int ntiles;
  int n_f32;         // fp32 temporaries
  size_t total;
};

bool carve(int op, const la_shape* s, Carve* c) {
  la_shape inner = *s;
  inner.out_dtype = LA_F32;
  const size_t op_ws = la_workspace_bytes(op, &inner);
  if (op_ws == (size_t)-1 || s->d != s->e) return false;
  const size_t elems = (size_t)s->B * s->H * s->N * s->d;
  c->feat = up256(elems * (s->in_dtype == LA_BF16 ? 2 : 4));
  c->f32 = up256(elems * 4);
  c->ntiles = (s->N + TILE_TOKENS - 1) / TILE_TOKENS;
  c->part = up256((size_t)s->B * s->H * c->ntiles * s->d * 4);
  c->op = up256(op_ws);
  const bool out32 = s->out_dtype == LA_F32;
  if (op == LA_OP_FWD) {
    c->n_f32 = out32 ? 1 : 2;                    // the second run's result (and the first's when o is bf16)
    c->total = 4 * c->feat + c->n_f32 * c->f32 + c->op;
  } else {
    c->n_f32 = 4 + (out32 ? 1 : 2);              // gradients of the four feature tensors, dv of the runs
    c->total = 4 * c->feat + c->n_f32 * c->f32 + 2 * c->part + c->op;
  }
  return true;
}

}  // namespace
}  // namespace la

using namespace la;

extern "C" {

size_t la_lrpe_workspace_bytes(int op, const la_shape* shape) {
  Carve c;
  if (!shape || (op != LA_OP_FWD && op != LA_OP_BWD) || !carve(op, shape, &c)) return (size_t)-1;
  return c.total;
}

la_status la_lrpe_fwd(const la_shape* shape, const void* q, const void* k, const void* v, const float* theta,
                      const float* lambda_host, long long pos0, void* o, const float* kv_in, float* kv_out,
                      void* workspace, size_t workspace_bytes, void* stream) {
  Carve c;
  if (!shape || !carve(LA_OP_FWD, shape, &c)) return shape ? LA_ERR_UNSUPPORTED : LA_ERR_INVALID_ARG;
  if (!q || !k || !v || !theta || !o || pos0 < 0) return LA_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(theta) & 15u) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return LA_ERR_INVALID_ARG;
  if (!workspace || workspace_bytes < c.total) return LA_ERR_WORKSPACE;
  if (!plain_args_ok(shape, lambda_host, {q, k, v, o, kv_in, kv_out})) return LA_ERR_INVALID_ARG;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  char* w = static_cast<char*>(workspace);
  void* qc = w; void* qs = w + c.feat; void* kc = w + 2 * c.feat; void* ks = w + 3 * c.feat;
  float* tmp = reinterpret_cast<float*>(w + 4 * c.feat);
  void* op_ws = w + 4 * c.feat + c.n_f32 * c.f32;
  const bool out32 = shape->out_dtype == LA_F32;
  la_shape inner = *shape;
  inner.out_dtype = LA_F32;
  const size_t state = (size_t)shape->B * shape->H * shape->d * shape->e;

  if (run_features(shape, q, theta, qc, qs, pos0, cs) != cudaSuccess) return LA_ERR_CUDA;
  if (run_features(shape, k, theta, kc, ks, pos0, cs) != cudaSuccess) return LA_ERR_CUDA;
  float* first = out32 ? static_cast<float*>(o) : tmp + c.f32 / 4;
  la_status st = la_fwd(&inner, qc, kc, v, lambda_host, first, kv_in, kv_out, op_ws, c.op, stream);
  if (st != LA_OK) return st;
  st = la_fwd(&inner, qs, ks, v, lambda_host, tmp, kv_in ? kv_in + state : nullptr, kv_out ? kv_out + state : nullptr,
              op_ws, c.op, stream);
  if (st != LA_OK) return st;
  if (run_sum(shape, first, tmp, o, cs) != cudaSuccess) return LA_ERR_CUDA;
  return LA_OK;
}

la_status la_lrpe_bwd(const la_shape* shape, const void* q, const void* k, const void* v, const void* d_o,
                      const float* theta, const float* lambda_host, long long pos0, void* dq, void* dk, void* dv,
                      float* d_theta, const float* kv_in, const float* grad_kv_out, float* grad_kv_in, void* workspace,
                      size_t workspace_bytes, void* stream) {
  Carve c;
  if (!shape || !carve(LA_OP_BWD, shape, &c)) return shape ? LA_ERR_UNSUPPORTED : LA_ERR_INVALID_ARG;
  if (!q || !k || !v || !d_o || !theta || !dq || !dk || !dv || !d_theta || pos0 < 0) return LA_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(theta) & 15u) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return LA_ERR_INVALID_ARG;
  if (!workspace || workspace_bytes < c.total) return LA_ERR_WORKSPACE;
  if (!plain_args_ok(shape, lambda_host, {q, k, v, d_o, dq, dk, dv, d_theta, kv_in, grad_kv_out, grad_kv_in}))
    return LA_ERR_INVALID_ARG;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  char* w = static_cast<char*>(workspace);
  void* qc = w; void* qs = w + c.feat; void* kc = w + 2 * c.feat; void* ks = w + 3 * c.feat;
  w += 4 * c.feat;
  float* g_qc = reinterpret_cast<float*>(w);
  float* g_kc = reinterpret_cast<float*>(w + c.f32);
  float* g_qs = reinterpret_cast<float*>(w + 2 * c.f32);
  float* g_ks = reinterpret_cast<float*>(w + 3 * c.f32);
  float* dv_s = reinterpret_cast<float*>(w + 4 * c.f32);
  const bool out32 = shape->out_dtype == LA_F32;
  float* dv_c = out32 ? static_cast<float*>(dv) : reinterpret_cast<float*>(w + 5 * c.f32);
  w += c.n_f32 * c.f32;
  float* part_q = reinterpret_cast<float*>(w);
  float* part_k = reinterpret_cast<float*>(w + c.part);
  void* op_ws = w + 2 * c.part;
  la_shape inner = *shape;
  inner.out_dtype = LA_F32;
  const size_t state = (size_t)shape->B * shape->H * shape->d * shape->e;

  if (run_features(shape, q, theta, qc, qs, pos0, cs) != cudaSuccess) return LA_ERR_CUDA;
  if (run_features(shape, k, theta, kc, ks, pos0, cs) != cudaSuccess) return LA_ERR_CUDA;
  la_status st = la_bwd(&inner, qc, kc, v, d_o, lambda_host, g_qc, g_kc, dv_c, kv_in, grad_kv_out, grad_kv_in, op_ws,
                        c.op, stream);
  if (st != LA_OK) return st;
  st = la_bwd(&inner, qs, ks, v, d_o, lambda_host, g_qs, g_ks, dv_s, kv_in ? kv_in + state : nullptr,
              grad_kv_out ? grad_kv_out + state : nullptr, grad_kv_in ? grad_kv_in + state : nullptr, op_ws, c.op,
              stream);
  if (st != LA_OK) return st;
  if (run_sum(shape, dv_c, dv_s, dv, cs) != cudaSuccess) return LA_ERR_CUDA;
  if (run_grad(shape, q, g_qc, g_qs, theta, dq, part_q, pos0, c.ntiles, cs) != cudaSuccess) return LA_ERR_CUDA;
  if (run_grad(shape, k, g_kc, g_ks, theta, dk, part_k, pos0, c.ntiles, cs) != cudaSuccess) return LA_ERR_CUDA;
  {
    KernelTimer timer(K_LRPE, cs);
    const int n = shape->H * shape->d;
    lrpe_theta_reduce_kernel<<<(n + 7) / 8, 256, 0, cs>>>(part_q, part_k, d_theta, shape->B, shape->H, c.ntiles, shape->d);
    count_launch();
    if (cudaGetLastError() != cudaSuccess) return LA_ERR_CUDA;
  }
  return LA_OK;
}

}  // extern "C"
