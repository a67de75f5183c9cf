// C-ABI entry points (declared in include/la.h): argument validation, the
// segment plan, workspace carving and the launch sequences.  Nothing here
// computes attention; every step of the path runs in the kernels.
#include <algorithm>
#include <atomic>
#include <mutex>
#include <vector>
#include <cmath>
#include <cstdint>
#include <cstdlib>

#include "../../include/la.h"
#include "la_common.cuh"

namespace la {

static std::atomic<unsigned long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

// ---- optional benchmark profiling ----------------------------------------------------------
struct ProfRecord { int kind; cudaEvent_t start, stop; };
static std::mutex g_prof_mu;
static std::atomic<bool> g_prof_on{false};
static std::vector<ProfRecord> g_prof;

KernelTimer::KernelTimer(int kind, cudaStream_t stream)
    : kind_(kind), stream_(stream), start_(nullptr), active_(false) {
  if (!g_prof_on.load(std::memory_order_relaxed)) return;
  if (cudaEventCreate(&start_) != cudaSuccess) return;
  cudaEventRecord(start_, stream_);
  active_ = true;
}
KernelTimer::~KernelTimer() {
  if (!active_) return;
  cudaEvent_t stop;
  if (cudaEventCreate(&stop) != cudaSuccess) { cudaEventDestroy(start_); return; }
  cudaEventRecord(stop, stream_);
  std::lock_guard<std::mutex> lock(g_prof_mu);
  g_prof.push_back({kind_, start_, stop});
}

namespace {

// A packed batch: sequences of different lengths one after the other in [total_tokens, H, D] tensors (DEVICE arrays
// of first tokens and lengths, one entry per sequence); the shape that goes with it has B = sequences, N = longest.
struct Packed {
  const int* start;
  const int* len;
  const int* order;  // sequence indices, longest first
  int total_tokens;
};

struct Plan {
  int BH, seg_len, nseg;
  bool tensor;      // tensor-core kernels
  int precision;    // LA_SPLIT_* bits (tensor path)
  Packed pk;        // start == NULL: dense batch
};

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

la_status check_shape(const la_shape* s, bool need_n) {
  if (!s) return LA_ERR_INVALID_ARG;
  if (s->B < 1 || s->H < 1 || s->d < 1 || s->e < 1) return LA_ERR_INVALID_ARG;
  if (need_n && s->N < 1) return LA_ERR_INVALID_ARG;
  if (s->in_dtype != LA_BF16 && s->in_dtype != LA_F32) return LA_ERR_INVALID_ARG;
  if (s->out_dtype != LA_BF16 && s->out_dtype != LA_F32) return LA_ERR_INVALID_ARG;
  if (s->seg_len < 0 || (s->seg_len % 128) != 0) return LA_ERR_INVALID_ARG;
  if (s->path < LA_PATH_AUTO || s->path > LA_PATH_TENSOR) return LA_ERR_INVALID_ARG;
  if (s->precision != LA_PRECISION_DEFAULT && (s->precision < 0 || s->precision > 7))
    return LA_ERR_INVALID_ARG;
  if (s->layout != LA_LAYOUT_BHND && s->layout != LA_LAYOUT_BNHD) return LA_ERR_INVALID_ARG;
  if (s->H > LA_MAX_H) return LA_ERR_UNSUPPORTED;
  if (!(s->d == s->e && (s->d == 64 || s->d == 128))) return LA_ERR_UNSUPPORTED;
  if (s->in_dtype == LA_F32 && s->out_dtype != LA_F32) return LA_ERR_UNSUPPORTED;
  // element counts must fit the 32-bit coordinates the kernels and tensor maps use
  const double tokens = (double)s->B * s->H * (need_n ? s->N : 1);
  if (tokens * s->d >= 2147483648.0 * 64.0 || (double)s->B * s->H >= 2147483648.0 ||
      (need_n && (double)s->N >= 1073741824.0))
    return LA_ERR_UNSUPPORTED;
  return LA_OK;
}

bool tensor_path_available(const la_shape* s) {
  return tc_supported() && s->in_dtype == LA_BF16 && s->d == s->e && (s->d == 128 || s->d == 64);
}

la_status make_plan(const la_shape* s, Plan* p) {
  p->pk = Packed{nullptr, nullptr, nullptr, 0};
  p->BH = s->B * s->H;
  if (s->path == LA_PATH_TENSOR && !tensor_path_available(s)) return LA_ERR_UNSUPPORTED;
  p->tensor = (s->path == LA_PATH_TENSOR) || (s->path == LA_PATH_AUTO && tensor_path_available(s));
  p->precision = (s->precision == LA_PRECISION_DEFAULT)
                     ? (LA_SPLIT_SCORES | LA_SPLIT_STATE | LA_SPLIT_DECAYED)
                     : s->precision;
  long seg_len = s->seg_len;
  if (seg_len == 0) {
    // One thread block per (batch*head, segment[, value-column half]) and one block per SM at a
    // time: pick the segment count that minimises (waves over the 148 SMs) x (blocks walked per
    // segment + pipeline fill), with segments no shorter than 1024 tokens so that the
    // per-segment state traffic stays small.  Depends on the shape only.
    // at d = 128 the half-width tensor kernels also split the value columns over two thread blocks
    const long slices = (p->tensor && s->d == 128 && !tc_full_width()) ? 2 : 1;
    const long sms = 148, fill = 2;
    long most = s->N / 1024;
    if (most < 1) most = 1;
    if (most > 1024) most = 1024;
    long best_n = 1, best_cost = -1;
    for (long n = 1; n <= most; ++n) {
      const long len = ((s->N + n - 1) / n + 127) / 128 * 128;
      const long nseg = (s->N + len - 1) / len;
      const long waves = (p->BH * slices * nseg + sms - 1) / sms;
      const long cost = waves * (len / 128 + fill);
      if (best_cost < 0 || cost < best_cost) {
        best_cost = cost;
        best_n = n;
      }
    }
    seg_len = ((s->N + best_n - 1) / best_n + 127) / 128 * 128;
  }
  p->seg_len = (int)seg_len;
  p->nseg = (int)((s->N + seg_len - 1) / seg_len);
  if (p->nseg > 1024) return LA_ERR_UNSUPPORTED;  // the state scan keeps one decay factor per segment on chip
  return LA_OK;
}

size_t state_set_bytes(const la_shape* s, const Plan& p) {
  return (size_t)p.BH * p.nseg * s->d * s->e * sizeof(float);
}

la_status make_table(const la_shape* s, const float* lambda_host, DecayTable* tab) {
  if (!lambda_host) return LA_ERR_INVALID_ARG;
  for (int h = 0; h < s->H; ++h) {
    const float lam = lambda_host[h];
    if (!(std::isfinite(lam) && lam > 0.f && lam <= 1.f)) return LA_ERR_INVALID_ARG;
    const double s2 = -std::log2((double)lam);
    tab->s2[h] = (s2 > 0.0) ? s2 : 0.0;  // lambda == 1 gives exactly 0 (never -0)
  }
  for (int h = s->H; h < LA_MAX_H; ++h) tab->s2[h] = 0.0;
  return LA_OK;
}

la_status check_device() {
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return LA_ERR_CUDA;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
    return LA_ERR_CUDA;
  return major == 10 ? LA_OK : LA_ERR_ARCH;
}

#define LA_TRY_CUDA(expr)                       \
  do {                                          \
    if ((expr) != cudaSuccess) return LA_ERR_CUDA; \
  } while (0)

// One generic-operator call: optional pre-pass + scan (when the sequence is cut
// into segments or the incoming state needs transposing), then the walk.
struct OpCall {
  const void *a, *b, *c;
  void* out;
  int reverse;
  const float* z_in;     // user state entering the sequence (kernel orientation unless transposed)
  bool z_in_transposed;
  float* final_out;      // state leaving the sequence, kernel orientation, or NULL
  float* buf;            // [BH,nseg,D*E] scratch for entry states (may be NULL if not needed)
};

// Element strides of the token tensors for the shape's layout (d == e in every supported shape).
void set_strides(const la_shape* s, int tokens, OpArgs* a) {
  const long long D = s->d;
  if (s->layout == LA_LAYOUT_BNHD) {
    a->sT = (long long)s->H * D;
    a->sH = D;
    a->sB = (long long)tokens * s->H * D;
  } else {
    a->sT = D;
    a->sH = (long long)tokens * D;
    a->sB = (long long)s->H * tokens * D;
  }
}

cudaError_t run_prepass(const la_shape* s, const Plan& p, const DecayTable& tab, const void* b,
                        const void* c, int reverse, float* local_out, cudaStream_t st) {
  OpArgs args{};
  args.b = b;
  args.c = c;
  args.local_out = local_out;
  args.BH = p.BH;
  args.H = s->H;
  args.N = s->N;
  args.seg_len = p.seg_len;
  args.nseg = p.nseg;
  args.reverse = reverse;
  args.seq_start = p.pk.start;
  args.seq_len = p.pk.len;
  args.seq_order = p.pk.order;
  args.total_tokens = p.pk.total_tokens;
  set_strides(s, p.pk.start ? p.pk.total_tokens : s->N, &args);
  if (p.tensor) return launch_tc_prepass(args, tab, s->d, p.precision, st);
  return launch_simt_prepass(args, tab, s->d, s->e, (int)s->in_dtype, st);
}

cudaError_t run_scan(const la_shape* s, const Plan& p, const DecayTable& tab, float* buf, float* buf_t,
                     const float* z_in, bool z_in_transposed, int reverse, cudaStream_t st) {
  ScanArgs sa{};
  sa.buf = buf;
  sa.buf_t = buf_t;
  sa.z_in = z_in;
  sa.z_in_transposed = z_in_transposed ? 1 : 0;
  sa.BH = p.BH;
  sa.H = s->H;
  sa.N = s->N;
  sa.seg_len = p.seg_len;
  sa.nseg = p.nseg;
  sa.seq_len = p.pk.len;
  sa.Da = s->d;  // d == e in every supported shape, so both orientations are square
  sa.Ec = s->e;
  sa.reverse = reverse;
  return launch_scan(sa, tab, st);
}

OpArgs walk_args(const la_shape* s, const Plan& p, const void* a, const void* b, const void* c, void* out,
                 const float* entry, float* final_out, int reverse) {
  OpArgs args{};
  args.a = a;
  args.b = b;
  args.c = c;
  args.out = out;
  args.entry = entry;
  args.final_out = final_out;
  args.BH = p.BH;
  args.H = s->H;
  args.N = s->N;
  args.seg_len = p.seg_len;
  args.nseg = p.nseg;
  args.reverse = reverse;
  args.seq_start = p.pk.start;
  args.seq_len = p.pk.len;
  args.seq_order = p.pk.order;
  args.total_tokens = p.pk.total_tokens;
  set_strides(s, p.pk.start ? p.pk.total_tokens : s->N, &args);
  return args;
}

cudaError_t run_walk(const la_shape* s, const Plan& p, const DecayTable& tab, const void* a,
                     const void* b, const void* c, void* out, const float* entry, float* final_out,
                     int reverse, cudaStream_t st) {
  const OpArgs args = walk_args(s, p, a, b, c, out, entry, final_out, reverse);
  if (p.tensor) return launch_tc_walk(args, tab, s->d, (int)s->out_dtype, p.precision, st);
  return launch_simt_walk(args, tab, s->d, s->e, (int)s->in_dtype, (int)s->out_dtype, st);
}

la_status fwd_impl(const la_shape* shape, const void* q, const void* k, const void* v, const void* u,
                   const float* lambda_host, void* y, void* o, float* rstd, const float* kv_in, float* kv_out,
                   void* workspace, size_t workspace_bytes, void* stream, const Packed* pk = nullptr);
la_status bwd_impl(const la_shape* shape, const void* q, const void* k, const void* v, const void* d_o,
                   const float* lambda_host, void* dq, void* dk, void* dv, const float* kv_in,
                   const float* grad_kv_out, float* grad_kv_in, const void* fwd_workspace, void* workspace,
                   size_t workspace_bytes, void* stream, const Packed* pk);
la_status decode_impl(const la_shape* shape, int T, const void* q, const void* k, const void* v,
                      const float* lambda_host, float* kv, void* o, void* stream);

}  // namespace
}  // namespace la

using namespace la;

extern "C" {

size_t la_workspace_bytes(int op, const la_shape* shape) {
  if (op != LA_OP_FWD && op != LA_OP_BWD && op != LA_OP_DECODE) return (size_t)-1;
  if (check_shape(shape, op != LA_OP_DECODE) != LA_OK) return (size_t)-1;
  if (op == LA_OP_DECODE) return 0;
  Plan p;
  if (make_plan(shape, &p) != LA_OK) return (size_t)-1;
  const size_t one = state_set_bytes(shape, p);
  if (op == LA_OP_FWD) return p.nseg > 1 ? 2 * one : 0;  // the states entering each segment, and their transposes
  return 3 * one;
}

int la_segment_length(const la_shape* shape) {
  if (check_shape(shape, true) != LA_OK) return 0;
  Plan p;
  if (make_plan(shape, &p) != LA_OK) return 0;
  return p.seg_len;
}

la_status la_fwd(const la_shape* shape, const void* q, const void* k, const void* v,
                 const float* lambda_host, void* o, const float* kv_in, float* kv_out,
                 void* workspace, size_t workspace_bytes, void* stream) {
  return fwd_impl(shape, q, k, v, nullptr, lambda_host, nullptr, o, nullptr, kv_in, kv_out, workspace, workspace_bytes,
                  stream);
}

la_status la_fwd_gated(const la_shape* shape, const void* q, const void* k, const void* v, const void* u,
                       const float* lambda_host, void* y, void* o, float* rstd, const float* kv_in, float* kv_out,
                       void* workspace, size_t workspace_bytes, void* stream) {
  if (!u || !y) return LA_ERR_INVALID_ARG;
  return fwd_impl(shape, q, k, v, u, lambda_host, y, o, rstd, kv_in, kv_out, workspace, workspace_bytes, stream);
}

la_status la_gate_fwd(const la_shape* shape, const void* o, const void* u, void* y, float* rstd, void* stream) {
  la_status st = check_shape(shape, true);
  if (st != LA_OK) return st;
  if (!o || !u || !y) return LA_ERR_INVALID_ARG;
  if (!aligned16(o) || !aligned16(u) || !aligned16(y) || !aligned16(rstd)) return LA_ERR_INVALID_ARG;
  if ((st = check_device()) != LA_OK) return st;
  LA_TRY_CUDA(launch_norm_gate_fwd(o, u, y, rstd, (long)shape->B * shape->H * shape->N, shape->e, (int)shape->in_dtype,
                                   (int)shape->out_dtype, static_cast<cudaStream_t>(stream)));
  return LA_OK;
}

la_status la_gate_bwd(const la_shape* shape, const void* o, const void* u, const void* d_y, void* d_o, void* d_u,
                      void* stream) {
  la_status st = check_shape(shape, true);
  if (st != LA_OK) return st;
  if (!o || !u || !d_y || !d_o || !d_u) return LA_ERR_INVALID_ARG;
  if (!aligned16(o) || !aligned16(u) || !aligned16(d_y) || !aligned16(d_o) || !aligned16(d_u)) return LA_ERR_INVALID_ARG;
  if ((st = check_device()) != LA_OK) return st;
  LA_TRY_CUDA(launch_norm_gate_bwd(o, u, d_y, d_o, d_u, (long)shape->B * shape->H * shape->N, shape->e,
                                   (int)shape->in_dtype, (int)shape->out_dtype, static_cast<cudaStream_t>(stream)));
  return LA_OK;
}

}  // extern "C"

namespace la {
namespace {
// la_fwd and la_fwd_gated: u == NULL is the plain forward pass (o required); with u the rows leave as
// y = SRMSNorm(o) (.) u, fused into the walk where the kernel can, else by a row kernel behind it.
la_status fwd_impl(const la_shape* shape, const void* q, const void* k, const void* v, const void* u,
                   const float* lambda_host, void* y, void* o, float* rstd, const float* kv_in, float* kv_out,
                   void* workspace, size_t workspace_bytes, void* stream, const Packed* pk) {
  la_status st = check_shape(shape, true);
  if (st != LA_OK) return st;
  if (!q || !k || !v || (!u && !o)) return LA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(kv_in) ||
      !aligned16(kv_out) || !aligned16(u) || !aligned16(y) || !aligned16(rstd))
    return LA_ERR_INVALID_ARG;
  DecayTable tab;
  if ((st = make_table(shape, lambda_host, &tab)) != LA_OK) return st;
  Plan p;
  if ((st = make_plan(shape, &p)) != LA_OK) return st;
  if (pk) p.pk = *pk;
  const size_t one = state_set_bytes(shape, p);
  const size_t need = p.nseg > 1 ? 2 * one : 0;
  if (need > 0 && (!workspace || workspace_bytes < need)) return LA_ERR_WORKSPACE;
  if (need > 0 && (reinterpret_cast<uintptr_t>(workspace) & 255u)) return LA_ERR_INVALID_ARG;
  if ((st = check_device()) != LA_OK) return st;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);

  const float* entry = kv_in;  // single segment: the caller's state is the entry state
  if (p.nseg > 1) {
    float* buf = static_cast<float*>(workspace);
    LA_TRY_CUDA(run_prepass(shape, p, tab, k, v, 0, buf, cs));
    // the transposed copy (second set) is what the dQ walk of la_bwd_reuse starts from
    LA_TRY_CUDA(run_scan(shape, p, tab, buf, buf + one / sizeof(float), kv_in, false, 0, cs));
    entry = buf;
  }
  if (!u) {
    LA_TRY_CUDA(run_walk(shape, p, tab, q, k, v, o, entry, kv_out, 0, cs));
    return LA_OK;
  }
  OpArgs wa = walk_args(shape, p, q, k, v, o, entry, kv_out, 0);
  wa.u = u;
  wa.y = y;
  wa.rstd = rstd;
  if (p.tensor && tc_can_fuse_gate(wa, shape->d)) {
    LA_TRY_CUDA(launch_tc_walk(wa, tab, shape->d, (int)shape->out_dtype, p.precision, cs));
    return LA_OK;
  }
  // not fused: the attention output goes to o (or, if it is not wanted, to y itself) and a row kernel turns it into y
  void* att = o ? o : y;
  LA_TRY_CUDA(run_walk(shape, p, tab, q, k, v, att, entry, kv_out, 0, cs));
  LA_TRY_CUDA(launch_norm_gate_fwd(att, u, y, rstd, (long)p.BH * shape->N, shape->e, (int)shape->in_dtype,
                                   (int)shape->out_dtype, cs));
  return LA_OK;
}
}  // namespace
}  // namespace la

extern "C" {

la_status la_bwd(const la_shape* shape, const void* q, const void* k, const void* v,
                 const void* d_o, const float* lambda_host, void* dq, void* dk, void* dv,
                 const float* kv_in, const float* grad_kv_out, float* grad_kv_in,
                 void* workspace, size_t workspace_bytes, void* stream) {
  return la_bwd_reuse(shape, q, k, v, d_o, lambda_host, dq, dk, dv, kv_in, grad_kv_out, grad_kv_in, nullptr,
                      workspace, workspace_bytes, stream);
}

la_status la_bwd_reuse(const la_shape* shape, const void* q, const void* k, const void* v,
                       const void* d_o, const float* lambda_host, void* dq, void* dk, void* dv,
                       const float* kv_in, const float* grad_kv_out, float* grad_kv_in,
                       const void* fwd_workspace, void* workspace, size_t workspace_bytes, void* stream) {
  return bwd_impl(shape, q, k, v, d_o, lambda_host, dq, dk, dv, kv_in, grad_kv_out, grad_kv_in, fwd_workspace,
                  workspace, workspace_bytes, stream, nullptr);
}

}  // extern "C"

namespace la {
namespace {
la_status bwd_impl(const la_shape* shape, const void* q, const void* k, const void* v, const void* d_o,
                   const float* lambda_host, void* dq, void* dk, void* dv, const float* kv_in,
                   const float* grad_kv_out, float* grad_kv_in, const void* fwd_workspace, void* workspace,
                   size_t workspace_bytes, void* stream, const Packed* pk) {
  la_status st = check_shape(shape, true);
  if (st != LA_OK) return st;
  if (!q || !k || !v || !d_o || !dq || !dk || !dv) return LA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(d_o) || !aligned16(dq) ||
      !aligned16(dk) || !aligned16(dv) || !aligned16(kv_in) || !aligned16(grad_kv_out) ||
      !aligned16(grad_kv_in) || !aligned16(fwd_workspace))
    return LA_ERR_INVALID_ARG;
  DecayTable tab;
  if ((st = make_table(shape, lambda_host, &tab)) != LA_OK) return st;
  Plan p;
  if ((st = make_plan(shape, &p)) != LA_OK) return st;
  if (pk) p.pk = *pk;
  const size_t one = state_set_bytes(shape, p);
  if (!workspace || workspace_bytes < 3 * one) return LA_ERR_WORKSPACE;
  if (fwd_workspace == workspace) return LA_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return LA_ERR_INVALID_ARG;
  if ((st = check_device()) != LA_OK) return st;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);

  float* buf_kvt = static_cast<float*>(workspace);                 // KV^T entering each segment
  float* buf_e = buf_kvt + one / sizeof(float);                    // dKV entering each segment (from the right)
  float* buf_et = buf_e + one / sizeof(float);                     // its transpose
  const bool multi = p.nseg > 1;

  // dQ = fwd(a = dO, b = V, c = K); its state is KV^T, so the caller's kv_in enters transposed.
  const float* entry_q = nullptr;
  if (multi && fwd_workspace) {
    // la_fwd left KV entering each segment (kv_in included) and its transpose in its workspace: no pre-pass, no scan
    entry_q = static_cast<const float*>(fwd_workspace) + one / sizeof(float);
  } else if (multi || kv_in) {
    if (multi) LA_TRY_CUDA(run_prepass(shape, p, tab, v, k, 0, buf_kvt, cs));
    LA_TRY_CUDA(run_scan(shape, p, tab, buf_kvt, nullptr, kv_in, true, 0, cs));
    entry_q = buf_kvt;
  }
  LA_TRY_CUDA(run_walk(shape, p, tab, d_o, v, k, dq, entry_q, nullptr, 0, cs));

  // dV = rev(a = K, b = Q, c = dO) carries dKV; dK = rev(a = V, b = dO, c = Q) carries dKV^T.
  const float* entry_v = nullptr;
  const float* entry_k = nullptr;
  if (multi) LA_TRY_CUDA(run_prepass(shape, p, tab, q, d_o, 1, buf_e, cs));
  if (multi || grad_kv_out) {
    LA_TRY_CUDA(run_scan(shape, p, tab, buf_e, buf_et, grad_kv_out, false, 1, cs));
    entry_v = buf_e;
    entry_k = buf_et;
  }
  if (p.tensor) {
    // both reverse walks in one launch: together they read Q, K, V and dO, and the thread blocks of the two are
    // interleaved so that each of those tiles comes from HBM once (Algorithm 4 accumulates dK_j and dV_j in the
    // same outer iteration for the same reason)
    const OpArgs walk_v = walk_args(shape, p, k, q, d_o, dv, entry_v, grad_kv_in, 1);
    const OpArgs walk_k = walk_args(shape, p, v, d_o, q, dk, entry_k, nullptr, 1);
    LA_TRY_CUDA(launch_tc_walk_pair(walk_v, walk_k, tab, shape->d, (int)shape->out_dtype, p.precision, cs));
  } else {
    LA_TRY_CUDA(run_walk(shape, p, tab, k, q, d_o, dv, entry_v, grad_kv_in, 1, cs));
    LA_TRY_CUDA(run_walk(shape, p, tab, v, d_o, q, dk, entry_k, nullptr, 1, cs));
  }
  return LA_OK;
}
}  // namespace
}  // namespace la

extern "C" {

la_status la_decode_step(const la_shape* shape, const void* q, const void* k, const void* v,
                         const float* lambda_host, float* kv, void* o, void* stream) {
  return decode_impl(shape, 1, q, k, v, lambda_host, kv, o, stream);
}

la_status la_decode_steps(const la_shape* shape, const void* q, const void* k, const void* v,
                          const float* lambda_host, float* kv, void* o, void* stream) {
  if (!shape || shape->N < 1) return LA_ERR_INVALID_ARG;
  return decode_impl(shape, shape->N, q, k, v, lambda_host, kv, o, stream);
}

}  // extern "C"

namespace la {
namespace {
la_status decode_impl(const la_shape* shape, int T, const void* q, const void* k, const void* v,
                      const float* lambda_host, float* kv, void* o, void* stream) {
  la_status st = check_shape(shape, false);
  if (st != LA_OK) return st;
  if (!q || !k || !v || !kv || !o) return LA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(kv) || !aligned16(o))
    return LA_ERR_INVALID_ARG;
  DecayTable tab;
  if ((st = make_table(shape, lambda_host, &tab)) != LA_OK) return st;
  if ((st = check_device()) != LA_OK) return st;
  OpArgs strides{};
  set_strides(shape, T, &strides);
  LA_TRY_CUDA(launch_decode(q, k, v, kv, o, shape->B * shape->H, shape->H, T, shape->d, shape->e,
                            (int)shape->in_dtype, (int)shape->out_dtype, strides.sT, strides.sH, strides.sB, tab,
                            static_cast<cudaStream_t>(stream)));
  return LA_OK;
}
}  // namespace
}  // namespace la

extern "C" {

static size_t round256(size_t n) { return (n + 255) / 256 * 256; }

size_t la_host_arena_bytes(const la_shape* shape) {
  const size_t wf = la_workspace_bytes(LA_OP_FWD, shape);
  const size_t wb = la_workspace_bytes(LA_OP_BWD, shape);
  if (wf == (size_t)-1 || wb == (size_t)-1) return (size_t)-1;
  const size_t tokens = (size_t)shape->B * shape->H * shape->N;
  const size_t in_sz = shape->in_dtype == LA_BF16 ? 2 : 4;
  const size_t out_sz = shape->out_dtype == LA_BF16 ? 2 : 4;
  size_t total = 0;
  total += 2 * round256(tokens * shape->d * in_sz) + 2 * round256(tokens * shape->e * in_sz);
  total += 2 * round256(tokens * shape->d * out_sz) + 2 * round256(tokens * shape->e * out_sz);
  total += round256(wf) + round256(wb);
  return total;
}

// Side streams and events of the host-buffer entry point: created once per device, on first use
// (streams and events are not device memory; nothing here allocates any).
namespace {
constexpr int kHostLanes = 3;
struct HostPipe {
  bool ready = false;
  cudaStream_t lane[kHostLanes];
  cudaEvent_t done[kHostLanes];
  cudaEvent_t start;
};
std::mutex g_pipe_mu;
std::mutex g_pipe_enqueue_mu;  // one host thread at a time records and waits on the shared events
HostPipe g_pipe[64];

HostPipe* host_pipe() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(g_pipe_mu);
  HostPipe& hp = g_pipe[dev];
  if (!hp.ready) {
    for (int i = 0; i < kHostLanes; ++i) {
      if (cudaStreamCreateWithFlags(&hp.lane[i], cudaStreamNonBlocking) != cudaSuccess) return nullptr;
      if (cudaEventCreateWithFlags(&hp.done[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
    }
    if (cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    hp.ready = true;
  }
  return &hp;
}
}  // namespace

la_status la_fwd_bwd_host(const la_shape* shape, const void* q_host, const void* k_host,
                          const void* v_host, const void* d_o_host, const float* lambda_host,
                          void* o_host, void* dq_host, void* dk_host, void* dv_host,
                          void* device_arena, size_t arena_bytes, void* stream) {
  const size_t need = la_host_arena_bytes(shape);
  if (need == (size_t)-1) return check_shape(shape, true) != LA_OK ? check_shape(shape, true) : LA_ERR_UNSUPPORTED;
  if (shape->layout != LA_LAYOUT_BHND) return LA_ERR_UNSUPPORTED;  // the head groups must be contiguous slices
  if (!q_host || !k_host || !v_host || !d_o_host || !o_host || !dq_host || !dk_host || !dv_host)
    return LA_ERR_INVALID_ARG;
  if (!device_arena || arena_bytes < need) return LA_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(device_arena) & 255u) return LA_ERR_INVALID_ARG;
  const size_t tokens = (size_t)shape->B * shape->H * shape->N;
  const size_t in_sz = shape->in_dtype == LA_BF16 ? 2 : 4;
  const size_t out_sz = shape->out_dtype == LA_BF16 ? 2 : 4;
  const size_t bq = tokens * shape->d * in_sz, bv = tokens * shape->e * in_sz;
  const size_t bdq = tokens * shape->d * out_sz, bdv = tokens * shape->e * out_sz;
  char* p = static_cast<char*>(device_arena);
  auto take = [&p](size_t n) { char* r = p; p += round256(n); return r; };
  char *dq_in = take(bq), *dk_in = take(bq), *dv_in = take(bv), *ddo_in = take(bv);
  char *d_o = take(bdv), *d_dq = take(bdq), *d_dk = take(bdq), *d_dv = take(bdv);
  char* ws = p;
  const size_t ws_bytes = arena_bytes - (size_t)(ws - static_cast<char*>(device_arena));
  cudaStream_t cs = static_cast<cudaStream_t>(stream);

  // Heads are independent, so the work is cut into groups of heads that run as
  // copy-in -> forward -> backward -> copy-out chains on three side streams: while one group
  // computes, the next one's inputs arrive and the previous one's results leave, and the two copy
  // directions share the link in full duplex.  Every group keeps the segment length of the whole
  // shape, so its workspace is its heads' share of the whole workspace; the three streams use
  // three disjoint thirds of it.
  la_shape sub = *shape;
  sub.B = 1;
  sub.seg_len = la_segment_length(shape);
  int group = shape->H / 8;
  if (group < 1) group = 1;
  size_t slot = 0;
  HostPipe* hp = nullptr;
  if (shape->H >= 3 * group) {
    sub.H = group;
    const size_t wf_g = la_workspace_bytes(LA_OP_FWD, &sub), wb_g = la_workspace_bytes(LA_OP_BWD, &sub);
    if (wf_g != (size_t)-1 && wb_g != (size_t)-1) {
      slot = round256(wf_g) + round256(wb_g);
      if (slot * kHostLanes <= ws_bytes) hp = host_pipe();
    }
  }
  if (!hp) {
    // small shapes: one chain on the caller's stream
    LA_TRY_CUDA(cudaMemcpyAsync(dq_in, q_host, bq, cudaMemcpyHostToDevice, cs));
    LA_TRY_CUDA(cudaMemcpyAsync(dk_in, k_host, bq, cudaMemcpyHostToDevice, cs));
    LA_TRY_CUDA(cudaMemcpyAsync(dv_in, v_host, bv, cudaMemcpyHostToDevice, cs));
    LA_TRY_CUDA(cudaMemcpyAsync(ddo_in, d_o_host, bv, cudaMemcpyHostToDevice, cs));
    la_status st = la_fwd(shape, dq_in, dk_in, dv_in, lambda_host, d_o, nullptr, nullptr, ws, ws_bytes, stream);
    if (st != LA_OK) return st;
    // the forward workspace (first state set) feeds the backward pass, which uses the space behind it
    const size_t wf = round256(la_workspace_bytes(LA_OP_FWD, shape));
    st = la_bwd_reuse(shape, dq_in, dk_in, dv_in, ddo_in, lambda_host, d_dq, d_dk, d_dv, nullptr, nullptr, nullptr,
                      wf > 0 ? ws : nullptr, ws + wf, ws_bytes - wf, stream);
    if (st != LA_OK) return st;
    LA_TRY_CUDA(cudaMemcpyAsync(o_host, d_o, bdv, cudaMemcpyDeviceToHost, cs));
    LA_TRY_CUDA(cudaMemcpyAsync(dq_host, d_dq, bdq, cudaMemcpyDeviceToHost, cs));
    LA_TRY_CUDA(cudaMemcpyAsync(dk_host, d_dk, bdq, cudaMemcpyDeviceToHost, cs));
    LA_TRY_CUDA(cudaMemcpyAsync(dv_host, d_dv, bdv, cudaMemcpyDeviceToHost, cs));
    return LA_OK;
  }

  // the side streams start after everything already queued on the caller's stream ...
  std::lock_guard<std::mutex> enqueue_lock(g_pipe_enqueue_mu);
  LA_TRY_CUDA(cudaEventRecord(hp->start, cs));
  for (int i = 0; i < kHostLanes; ++i) LA_TRY_CUDA(cudaStreamWaitEvent(hp->lane[i], hp->start, 0));
  int g = 0;
  for (int b = 0; b < shape->B; ++b) {
    for (int h0 = 0; h0 < shape->H; h0 += group, ++g) {
      const int hc = shape->H - h0 < group ? shape->H - h0 : group;
      sub.H = hc;
      cudaStream_t ls = hp->lane[g % kHostLanes];
      char* wsg = ws + (size_t)(g % kHostLanes) * slot;
      const size_t head = (size_t)b * shape->H + h0;  // first (b,h) slice of the group
      const size_t oq = head * shape->N * shape->d * in_sz, ov = head * shape->N * shape->e * in_sz;
      const size_t odq = head * shape->N * shape->d * out_sz, odv = head * shape->N * shape->e * out_sz;
      const size_t nq = (size_t)hc * shape->N * shape->d * in_sz, nv = (size_t)hc * shape->N * shape->e * in_sz;
      const size_t ndq = (size_t)hc * shape->N * shape->d * out_sz, ndv = (size_t)hc * shape->N * shape->e * out_sz;
      LA_TRY_CUDA(cudaMemcpyAsync(dq_in + oq, static_cast<const char*>(q_host) + oq, nq, cudaMemcpyHostToDevice, ls));
      LA_TRY_CUDA(cudaMemcpyAsync(dk_in + oq, static_cast<const char*>(k_host) + oq, nq, cudaMemcpyHostToDevice, ls));
      LA_TRY_CUDA(cudaMemcpyAsync(dv_in + ov, static_cast<const char*>(v_host) + ov, nv, cudaMemcpyHostToDevice, ls));
      LA_TRY_CUDA(cudaMemcpyAsync(ddo_in + ov, static_cast<const char*>(d_o_host) + ov, nv, cudaMemcpyHostToDevice, ls));
      const size_t wf = round256(la_workspace_bytes(LA_OP_FWD, &sub));
      la_status st = la_fwd(&sub, dq_in + oq, dk_in + oq, dv_in + ov, lambda_host + h0, d_o + odv, nullptr, nullptr,
                            wsg, slot, ls);
      if (st != LA_OK) return st;
      st = la_bwd_reuse(&sub, dq_in + oq, dk_in + oq, dv_in + ov, ddo_in + ov, lambda_host + h0, d_dq + odq, d_dk + odq,
                        d_dv + odv, nullptr, nullptr, nullptr, wf > 0 ? wsg : nullptr, wsg + wf, slot - wf, ls);
      if (st != LA_OK) return st;
      LA_TRY_CUDA(cudaMemcpyAsync(static_cast<char*>(o_host) + odv, d_o + odv, ndv, cudaMemcpyDeviceToHost, ls));
      LA_TRY_CUDA(cudaMemcpyAsync(static_cast<char*>(dq_host) + odq, d_dq + odq, ndq, cudaMemcpyDeviceToHost, ls));
      LA_TRY_CUDA(cudaMemcpyAsync(static_cast<char*>(dk_host) + odq, d_dk + odq, ndq, cudaMemcpyDeviceToHost, ls));
      LA_TRY_CUDA(cudaMemcpyAsync(static_cast<char*>(dv_host) + odv, d_dv + odv, ndv, cudaMemcpyDeviceToHost, ls));
    }
  }
  // ... and the caller's stream continues after all of them
  for (int i = 0; i < kHostLanes; ++i) {
    LA_TRY_CUDA(cudaEventRecord(hp->done[i], hp->lane[i]));
    LA_TRY_CUDA(cudaStreamWaitEvent(cs, hp->done[i], 0));
  }
  return LA_OK;
}

// ---- one sequence cut into chunks (sequence parallelism): the state is all that crosses a cut ---------------------
size_t la_chunk_state_workspace_bytes(const la_shape* shape) {
  if (check_shape(shape, true) != LA_OK) return (size_t)-1;
  Plan p;
  if (make_plan(shape, &p) != LA_OK) return (size_t)-1;
  return state_set_bytes(shape, p);
}

la_status la_chunk_state(const la_shape* shape, int reverse, const void* b, const void* c, const float* lambda_host,
                         float* state_out, void* workspace, size_t workspace_bytes, void* stream) {
  la_status st = check_shape(shape, true);
  if (st != LA_OK) return st;
  if (!b || !c || !state_out || (reverse != 0 && reverse != 1)) return LA_ERR_INVALID_ARG;
  if (!aligned16(b) || !aligned16(c) || !aligned16(state_out)) return LA_ERR_INVALID_ARG;
  DecayTable tab;
  if ((st = make_table(shape, lambda_host, &tab)) != LA_OK) return st;
  Plan p;
  if ((st = make_plan(shape, &p)) != LA_OK) return st;
  const size_t need = state_set_bytes(shape, p);
  if (!workspace || workspace_bytes < need) return LA_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return LA_ERR_INVALID_ARG;
  if ((st = check_device()) != LA_OK) return st;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  float* buf = static_cast<float*>(workspace);
  LA_TRY_CUDA(run_prepass(shape, p, tab, b, c, reverse, buf, cs));
  ChainArgs ca{};
  ca.src = buf;
  ca.DE = shape->d * shape->e;
  ca.stride_j = ca.DE;
  ca.stride_bh = (long long)p.nseg * ca.DE;
  ca.z_in = nullptr;
  ca.out = state_out;
  ca.BH = p.BH;
  ca.H = shape->H;
  ca.first = reverse ? p.nseg - 1 : 0;
  ca.count = p.nseg;
  ca.step = reverse ? -1 : 1;
  ca.N = shape->N;
  ca.piece_len = p.seg_len;
  LA_TRY_CUDA(launch_chain(ca, tab, cs));
  return LA_OK;
}

la_status la_chain_states(const la_shape* shape, long long total_tokens, long long chunk_tokens, int reverse,
                          const float* states, int num_chunks, int chunk, const float* boundary,
                          const float* lambda_host, float* state_out, void* stream) {
  la_status st = check_shape(shape, false);
  if (st != LA_OK) return st;
  if (!states || !state_out || (reverse != 0 && reverse != 1)) return LA_ERR_INVALID_ARG;
  if (!aligned16(states) || !aligned16(state_out) || !aligned16(boundary)) return LA_ERR_INVALID_ARG;
  if (num_chunks < 1 || chunk_tokens < 1 || total_tokens < 1) return LA_ERR_INVALID_ARG;
  if ((total_tokens + chunk_tokens - 1) / chunk_tokens != num_chunks) return LA_ERR_INVALID_ARG;
  // forward: the state entering chunk `chunk` (0 .. num_chunks; num_chunks = after the last chunk);
  // reverse: the state gradient entering chunk `chunk` from the right (-1 .. num_chunks - 1; -1 = before the first)
  if (reverse ? (chunk < -1 || chunk > num_chunks - 1) : (chunk < 0 || chunk > num_chunks)) return LA_ERR_INVALID_ARG;
  DecayTable tab;
  if ((st = make_table(shape, lambda_host, &tab)) != LA_OK) return st;
  if ((st = check_device()) != LA_OK) return st;
  ChainArgs ca{};
  ca.src = states;
  ca.DE = shape->d * shape->e;
  ca.BH = shape->B * shape->H;
  ca.stride_j = (long long)ca.BH * ca.DE;
  ca.stride_bh = ca.DE;
  ca.z_in = boundary;
  ca.out = state_out;
  ca.H = shape->H;
  ca.first = reverse ? num_chunks - 1 : 0;
  ca.count = reverse ? num_chunks - 1 - chunk : chunk;
  ca.step = reverse ? -1 : 1;
  ca.N = total_tokens;
  ca.piece_len = chunk_tokens;
  LA_TRY_CUDA(launch_chain(ca, tab, static_cast<cudaStream_t>(stream)));
  return LA_OK;
}

// ---- packed batches of sequences of different lengths -------------------------------------------------------
namespace {
// Checks the packed description and returns, through `sub`, the shape of one sequence (N filled in per sequence).
la_status varlen_check(const la_shape* shape, const int* cu, int S, la_shape* sub) {
  la_status st = check_shape(shape, true);
  if (st != LA_OK) return st;
  if (!cu || S < 1) return LA_ERR_INVALID_ARG;
  if (shape->B != 1 || shape->layout != LA_LAYOUT_BNHD) return LA_ERR_UNSUPPORTED;
  if (cu[0] != 0 || cu[S] != shape->N) return LA_ERR_INVALID_ARG;
  for (int i = 0; i < S; ++i)
    if (cu[i + 1] <= cu[i]) return LA_ERR_INVALID_ARG;  // empty sequences are not allowed
  *sub = *shape;
  return LA_OK;
}
size_t esize(int dt) { return dt == LA_BF16 ? 2 : 4; }

// The single-launch form: every sequence is a "batch" entry of its own length inside the packed tensors, and the
// full-width tensor-core walk (with the state-only pre-pass and the scan where the longest sequence is cut into
// segments) runs over all of them at once.  It exists for bf16 inputs at d = e = 128 with outputs aligned to 32
// bytes; everything else runs one call per sequence.  `sp` is the shape that goes with it: B = sequences, N = longest.
bool packed_shape(const la_shape* shape, const int* cu, int S, la_shape* sp) {
  if (S < 2 || shape->d != 128 || shape->in_dtype != LA_BF16 || shape->path == LA_PATH_SIMT || !tc_supported())
    return false;
  int longest = 0;
  for (int i = 0; i < S; ++i) longest = std::max(longest, cu[i + 1] - cu[i]);
  *sp = *shape;
  sp->B = S;
  sp->N = longest;
  return check_shape(sp, true) == LA_OK;
}
size_t packed_table_bytes(int S) { return ((size_t)3 * S * sizeof(int) + 255) / 256 * 256; }

// Copies first tokens and lengths to the head of the workspace (stream-ordered) and describes them.
la_status packed_upload(const int* cu, int S, int total, void* workspace, cudaStream_t cs, Packed* pk) {
  std::vector<int> host(3 * (size_t)S);
  for (int i = 0; i < S; ++i) {
    host[i] = cu[i];
    host[S + i] = cu[i + 1] - cu[i];
    host[2 * S + i] = i;
  }
  // longest first (ties in the caller's order): the thread blocks of a launch are handed out in index order
  std::stable_sort(host.begin() + 2 * S, host.end(), [&](int a, int b) { return host[S + a] > host[S + b]; });
  // pageable source: the runtime has taken its copy of the table by the time the call returns
  if (cudaMemcpyAsync(workspace, host.data(), host.size() * sizeof(int), cudaMemcpyHostToDevice, cs) != cudaSuccess)
    return LA_ERR_CUDA;
  pk->start = static_cast<const int*>(workspace);
  pk->len = pk->start + S;
  pk->order = pk->start + 2 * S;
  pk->total_tokens = total;
  return LA_OK;
}
}  // namespace

size_t la_varlen_workspace_bytes(int op, const la_shape* shape, const int* cu_seqlens_host, int num_seqs) {
  la_shape sub;
  if (op != LA_OP_FWD && op != LA_OP_BWD) return (size_t)-1;
  if (varlen_check(shape, cu_seqlens_host, num_seqs, &sub) != LA_OK) return (size_t)-1;
  size_t most = 0;
  for (int i = 0; i < num_seqs; ++i) {
    sub.N = cu_seqlens_host[i + 1] - cu_seqlens_host[i];
    const size_t w = la_workspace_bytes(op, &sub);
    if (w == (size_t)-1) return (size_t)-1;
    if (w > most) most = w;
  }
  la_shape sp;
  if (packed_shape(shape, cu_seqlens_host, num_seqs, &sp)) {  // the single-launch form: its table and its state sets
    const size_t w = la_workspace_bytes(op, &sp);
    if (w != (size_t)-1 && packed_table_bytes(num_seqs) + w > most) most = packed_table_bytes(num_seqs) + w;
  }
  return most;
}

la_status la_fwd_varlen(const la_shape* shape, const void* q, const void* k, const void* v, const float* lambda_host,
                        void* o, const int* cu_seqlens_host, int num_seqs, const float* kv_in, float* kv_out,
                        void* workspace, size_t workspace_bytes, void* stream) {
  la_shape sub;
  la_status st = varlen_check(shape, cu_seqlens_host, num_seqs, &sub);
  if (st != LA_OK) return st;
  if (!q || !k || !v || !o) return LA_ERR_INVALID_ARG;
  la_shape sp;
  if (packed_shape(shape, cu_seqlens_host, num_seqs, &sp) && tc_walk_is_full(shape->d, o, nullptr)) {
    const size_t tb = packed_table_bytes(num_seqs);
    if (!workspace || workspace_bytes < tb || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return LA_ERR_WORKSPACE;
    if ((st = check_device()) != LA_OK) return st;
    Packed pk;
    if ((st = packed_upload(cu_seqlens_host, num_seqs, shape->N, workspace, static_cast<cudaStream_t>(stream), &pk)) != LA_OK)
      return st;
    return fwd_impl(&sp, q, k, v, nullptr, lambda_host, nullptr, o, nullptr, kv_in, kv_out,
                    static_cast<char*>(workspace) + tb, workspace_bytes - tb, stream, &pk);
  }
  const size_t row_in = (size_t)shape->H * shape->d * esize(shape->in_dtype);
  const size_t row_out = (size_t)shape->H * shape->e * esize(shape->out_dtype);
  const size_t state = (size_t)shape->H * shape->d * shape->e;
  for (int i = 0; i < num_seqs; ++i) {
    const size_t t0 = (size_t)cu_seqlens_host[i];
    sub.N = cu_seqlens_host[i + 1] - cu_seqlens_host[i];
    st = la_fwd(&sub, static_cast<const char*>(q) + t0 * row_in, static_cast<const char*>(k) + t0 * row_in,
                static_cast<const char*>(v) + t0 * row_in, lambda_host, static_cast<char*>(o) + t0 * row_out,
                kv_in ? kv_in + i * state : nullptr, kv_out ? kv_out + i * state : nullptr, workspace, workspace_bytes,
                stream);
    if (st != LA_OK) return st;
  }
  return LA_OK;
}

la_status la_bwd_varlen(const la_shape* shape, const void* q, const void* k, const void* v, const void* d_o,
                        const float* lambda_host, void* dq, void* dk, void* dv, const int* cu_seqlens_host, int num_seqs,
                        const float* kv_in, const float* grad_kv_out, float* grad_kv_in, void* workspace,
                        size_t workspace_bytes, void* stream) {
  la_shape sub;
  la_status st = varlen_check(shape, cu_seqlens_host, num_seqs, &sub);
  if (st != LA_OK) return st;
  if (!q || !k || !v || !d_o || !dq || !dk || !dv) return LA_ERR_INVALID_ARG;
  la_shape sp;
  if (packed_shape(shape, cu_seqlens_host, num_seqs, &sp) && tc_walk_is_full(shape->d, dq, dk) &&
      tc_walk_is_full(shape->d, dv, nullptr)) {
    const size_t tb = packed_table_bytes(num_seqs);
    if (!workspace || workspace_bytes < tb || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return LA_ERR_WORKSPACE;
    if ((st = check_device()) != LA_OK) return st;
    Packed pk;
    if ((st = packed_upload(cu_seqlens_host, num_seqs, shape->N, workspace, static_cast<cudaStream_t>(stream), &pk)) != LA_OK)
      return st;
    return bwd_impl(&sp, q, k, v, d_o, lambda_host, dq, dk, dv, kv_in, grad_kv_out, grad_kv_in, nullptr,
                    static_cast<char*>(workspace) + tb, workspace_bytes - tb, stream, &pk);
  }
  const size_t row_in = (size_t)shape->H * shape->d * esize(shape->in_dtype);
  const size_t row_out = (size_t)shape->H * shape->e * esize(shape->out_dtype);
  const size_t state = (size_t)shape->H * shape->d * shape->e;
  for (int i = 0; i < num_seqs; ++i) {
    const size_t t0 = (size_t)cu_seqlens_host[i];
    sub.N = cu_seqlens_host[i + 1] - cu_seqlens_host[i];
    st = la_bwd(&sub, static_cast<const char*>(q) + t0 * row_in, static_cast<const char*>(k) + t0 * row_in,
                static_cast<const char*>(v) + t0 * row_in, static_cast<const char*>(d_o) + t0 * row_in, lambda_host,
                static_cast<char*>(dq) + t0 * row_out, static_cast<char*>(dk) + t0 * row_out,
                static_cast<char*>(dv) + t0 * row_out, kv_in ? kv_in + i * state : nullptr,
                grad_kv_out ? grad_kv_out + i * state : nullptr, grad_kv_in ? grad_kv_in + i * state : nullptr, workspace,
                workspace_bytes, stream);
    if (st != LA_OK) return st;
  }
  return LA_OK;
}

la_status la_selftest_bounded_wait(unsigned long long budget_clocks, void* stream) {
  if (budget_clocks == 0 || budget_clocks > 2000000000ull) return LA_ERR_INVALID_ARG;
  const la_status dev = check_device();
  if (dev != LA_OK) return dev;
  if (launch_bounded_wait_selftest((long long)budget_clocks, static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return LA_ERR_CUDA;
  return LA_OK;
}

la_status la_device_status(unsigned int* code) {
  if (cudaDeviceSynchronize() != cudaSuccess) return LA_ERR_CUDA;
  const unsigned int v = tc_read_status(true);
  if (code) *code = v;
  if (v == 0xFFFFFFFFu) return LA_ERR_CUDA;
  return v == 0 ? LA_OK : LA_ERR_DEVICE_TIMEOUT;
}

const char* la_status_string(la_status s) {
  switch (s) {
    case LA_OK: return "ok";
    case LA_ERR_INVALID_ARG: return "invalid argument";
    case LA_ERR_UNSUPPORTED: return "unsupported shape or dtype";
    case LA_ERR_WORKSPACE: return "workspace missing or too small";
    case LA_ERR_CUDA: return "CUDA call or launch failed";
    case LA_ERR_ARCH: return "device is not sm_100";
    case LA_ERR_DEVICE_TIMEOUT: return "bounded device-side wait expired";
    case LA_ERR_SCRATCH_LIMIT: return "shape needs more scratch than the built-in static buffer holds";
  }
  return "unknown status";
}

int la_version(void) { return 100; }

void la_profile_enable(int on) { g_prof_on.store(on != 0, std::memory_order_relaxed); }

la_status la_profile_collect(double* ms, unsigned long long* launches) {
  if (!ms || !launches) return LA_ERR_INVALID_ARG;
  for (int i = 0; i < LA_NUM_KERNEL_KINDS; ++i) { ms[i] = 0.0; launches[i] = 0; }
  std::lock_guard<std::mutex> lock(g_prof_mu);
  la_status st = LA_OK;
  for (const ProfRecord& r : g_prof) {
    float t = 0.f;
    if (cudaEventSynchronize(r.stop) != cudaSuccess ||
        cudaEventElapsedTime(&t, r.start, r.stop) != cudaSuccess)
      st = LA_ERR_CUDA;
    if (r.kind >= 0 && r.kind < LA_NUM_KERNEL_KINDS) { ms[r.kind] += t; launches[r.kind] += 1; }
    cudaEventDestroy(r.start);
    cudaEventDestroy(r.stop);
  }
  g_prof.clear();
  return st;
}

unsigned long long la_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
