// Shared declarations of the CUDA side: kernel parameter blocks and the launch
// helpers that the C-ABI entry points in la_api.cu call.
//
// One generic operator covers forward and all three gradients.  With a
// "query-like" a [N,Da], a "key-like" b [N,Da] and a "value-like" c [N,Ec]:
//
//   forward direction   out_t = sum_{s<=t} lambda^(t-s) (a_t.b_s) c_s + lambda^(t+1)   Z_in^T a_t
//   reverse direction   out_t = sum_{s>=t} lambda^(s-t) (a_t.b_s) c_s + lambda^(N-1-t) Z_in^T a_t
//
// where Z is the Da x Ec running state sum_s decay * b_s c_s^T.  Then
//   O  = fwd(a=Q,  b=K,  c=V)        state = KV          (Algorithm 2 / Algorithm 3)
//   dQ = fwd(a=dO, b=V,  c=K)        state = KV^T        (Algorithm 4, dQ line)
//   dK = rev(a=V,  b=dO, c=Q)        state = (dKV)^T     (Algorithm 4, dK line)
//   dV = rev(a=K,  b=Q,  c=dO)       state = dKV         (Algorithm 4, dV line)
// The sequence is processed in blocks of C tokens (block-local index i, j):
//   out_blk = ((a b^T) (.) D) c + diag(f_out) a Z,      Z <- Gamma Z + b^T diag(f_state) c
// with every decay factor a non-negative power of lambda:
//   forward: D_ij = lambda^(i-j) [i>=j], f_out_i = lambda^(i+1),    f_state_j = lambda^(Cr-1-j)
//   reverse: D_ij = lambda^(j-i) [j>=i], f_out_i = lambda^(Cr-1-i), f_state_j = lambda^(j+1)
//   Gamma = lambda^Cr, Cr = number of real tokens in the block (a ragged last block
//   uses its own Cr so that no state is decayed through padding).
// Factors are evaluated as exp2(-s2 * n) with s2 = -log2(lambda) >= 0, never as a
// ratio of powers, so nothing can overflow and underflow only flushes to the
// correct limit 0 (this is what the prescaled form of Algorithm 1 cannot offer).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#define LA_MAX_H 256

namespace la {

struct DecayTable {
  double s2[LA_MAX_H];  // -log2(lambda_h) >= 0, computed in double on the host
};

// Arguments of one generic-operator launch (either the walking kernel or the
// state-only pre-pass).
struct OpArgs {
  const void* a;      // [BH, N, Da]  (unused by the pre-pass)
  const void* b;      // [BH, N, Da]
  const void* c;      // [BH, N, Ec]
  void* out;          // [BH, N, Ec]  (unused by the pre-pass)
  const float* entry; // [BH, nseg, Da*Ec] state entering each segment, or NULL = zeros
  float* local_out;   // pre-pass: [BH, nseg, Da*Ec] segment-local states
  float* final_out;   // [BH, Da*Ec] state leaving the last-processed segment, or NULL
  int BH, H, N;
  int seg_len, nseg;  // seg_len is a multiple of 128
  int reverse;        // 0 forward, 1 reverse
  // Where token t of (batch b, head h) sits in a, b, c, out, u, y: element offset b*sB + h*sH + t*sT of a row of
  // Da / Ec contiguous features.  [B,H,N,D]: sT = D, sH = N*D, sB = H*N*D; [B,N,H,D]: sT = H*D, sH = D, sB = N*H*D
  // (D = Da = Ec in every supported shape).
  long long sT, sH, sB;
  // Optional epilogue of the forward walk (Eq. 3 with Eq. 8): y = SRMSNorm(out) (.) u per row.  With u set, y is
  // written, `out` becomes optional (NULL = the attention output itself is not wanted) and rstd [BH, N] optional.
  const void* u;      // [BH, N, Ec] gate, input dtype
  void* y;            // [BH, N, Ec] output dtype
  float* rstd;        // [BH, N] sqrt(Ec) / ||out row||_2, or NULL
  // Packed batch of sequences of different lengths (tensor-core kernels at Da = Ec = 128 only; NULL elsewhere):
  // the token tensors are [total_tokens, H, D] with the sequences one after the other, "batch" entry b is
  // sequence b with seq_len[b] tokens starting at token seq_start[b] (DEVICE arrays of BH / H ints), N is the
  // longest length (it fixes the segment grid; thread blocks of segments a sequence does not have return at once)
  // and sB is unused.  Rows past a sequence's end belong to its neighbour, not to a zero-filled margin, so every
  // bound below is the sequence's own length.
  const int* seq_start;
  const int* seq_len;
  const int* seq_order;  // the order in which thread blocks take the sequences (longest first), or NULL
  int total_tokens;
};

struct ScanArgs {
  float* buf;          // [BH, nseg, Da*Ec]: in = segment-local states, out = entry states
  float* buf_t;        // optional transposed copy of the entry states [BH, nseg, Ec*Da]
  const float* z_in;   // [BH, Da*Ec] (or [BH, Ec*Da] if z_in_transposed), or NULL = zeros
  int z_in_transposed;
  int BH, H, N, seg_len, nseg, Da, Ec, reverse;
  const int* seq_len;  // packed batch: DEVICE array of BH / H lengths (N is then the longest), or NULL
};

// Chain of piece-local states into the state at one boundary (a cut of the sequence):
//   forward (first <= last):  z = z_in;  for j = first .. last:      z = lambda^(L_j) z + src_j
//   reverse (first >  last):  z = z_in;  for j = first down to last: z = lambda^(L_j) z + src_j
// with L_j = tokens of piece j = min(N, (j+1) piece_len) - j piece_len.  count == 0 copies z_in (or zeros).
struct ChainArgs {
  const float* src;         // element i of piece j of (b,h): src[j * stride_j + bh * stride_bh + i]
  long long stride_j, stride_bh;
  const float* z_in;        // [BH, DE] or NULL = zeros
  float* out;               // [BH, DE]
  int BH, H, DE;
  int first, count, step;   // pieces first, first + step, ... (count of them), step = +1 or -1
  long long N, piece_len;
};

// dtype tags as in la.h
enum { DT_BF16 = 0, DT_F32 = 1 };

// Each returns cudaGetLastError() of its launch.
cudaError_t launch_simt_walk(const OpArgs& args, const DecayTable& tab, int Da, int Ec, int in_dt,
                             int out_dt, cudaStream_t stream);
cudaError_t launch_simt_prepass(const OpArgs& args, const DecayTable& tab, int Da, int Ec, int in_dt,
                                cudaStream_t stream);
cudaError_t launch_scan(const ScanArgs& args, const DecayTable& tab, cudaStream_t stream);
cudaError_t launch_chain(const ChainArgs& args, const DecayTable& tab, cudaStream_t stream);
// dst[m] = transpose(src[m]) for `count` row-major Da x Ec fp32 matrices.
cudaError_t launch_transpose_states(const float* src, float* dst, long count, int Da, int Ec, cudaStream_t stream);
// T >= 1 consecutive tokens per (batch, head); token t of (b,h) is the row at element offset b*sB + h*sH + t*sT.
cudaError_t launch_decode(const void* q, const void* k, const void* v, float* kv, void* o, int BH,
                          int H, int T, int d, int e, int in_dt, int out_dt, long long sT, long long sH, long long sB,
                          const DecayTable& tab, cudaStream_t stream);

// SimpleRMSNorm followed by the gate as stand-alone row kernels (la_gate.cu): y = SRMSNorm(o) (.) u (o and y may be
// the same buffer), and the gradients of <y, dy> with respect to o (written in the input dtype) and u.
cudaError_t launch_norm_gate_fwd(const void* o, const void* u, void* y, float* rstd, long rows, int e, int in_dt,
                                 int out_dt, cudaStream_t stream);
cudaError_t launch_norm_gate_bwd(const void* o, const void* u, const void* dy, void* d_o, void* d_u, long rows, int e,
                                 int in_dt, int out_dt, cudaStream_t stream);

// Tensor-core (tcgen05) kernels: bf16 inputs, Da = Ec = D with D = 64 or 128.
bool tc_supported();
cudaError_t launch_tc_walk(const OpArgs& args, const DecayTable& tab, int D, int out_dt, int precision,
                           cudaStream_t stream);
// Whether launch_tc_walk can fuse the epilogue described by args.u / args.y into the walk (d = 128, y and out
// aligned to 32 bytes); otherwise the caller runs the walk and then launch_norm_gate_fwd.
// True when launch_tc_walk / launch_tc_walk_pair take the full-width kernel for these outputs (D = 128, aligned to 32 bytes).
bool tc_walk_is_full(int D, const void* out0, const void* out1);
bool tc_can_fuse_gate(const OpArgs& args, int D);
// Two walks of the same direction over the same tokens (same N, BH, segments) in one launch; the thread blocks of
// the two are interleaved so that tiles both read come from HBM once.
// Whether the d = 128 walk normally runs as one full-width thread block per (head, segment) rather than two
// half-width ones (the segment plan counts thread blocks accordingly).
bool tc_full_width();
cudaError_t launch_tc_walk_pair(const OpArgs& first, const OpArgs& second, const DecayTable& tab, int D, int out_dt,
                                int precision, cudaStream_t stream);
cudaError_t launch_tc_prepass(const OpArgs& args, const DecayTable& tab, int D, int precision,
                              cudaStream_t stream);

// One warp runs the kernels' bounded wait on a barrier nothing arrives on (budget in SM clocks).
cudaError_t launch_bounded_wait_selftest(long long budget_clocks, cudaStream_t stream);

// Failure code recorded by a tensor-core block whose bounded wait expired (0 = none);
// copies it from the device (blocking) and optionally clears it.
unsigned int tc_read_status(bool clear);

void count_launch(int n = 1);

// Brackets one kernel launch with CUDA events when benchmark profiling is enabled
// (la_profile_enable); otherwise does nothing.  kind is one of LA_KERNEL_*.
struct KernelTimer {
  KernelTimer(int kind, cudaStream_t stream);
  ~KernelTimer();
  int kind_;
  cudaStream_t stream_;
  cudaEvent_t start_;
  bool active_;
};
enum { K_PREPASS = 0, K_SCAN = 1, K_WALK = 2, K_DECODE = 3, K_WALK_PAIR = 4, K_GATE = 5, K_LRPE = 6, K_NUM = 7 };

// ---- small device helpers --------------------------------------------------
__device__ __forceinline__ float decay_pow(float s2, float n) {
  // lambda^n for n >= 0; s2 == 0 (lambda == 1) gives exactly 1.
  return exp2f(-s2 * n);
}
__device__ __forceinline__ float decay_pow_d(double s2, double n) {
  // Same in double, rounded once; used where a handful of factors per block are tabulated.
  return (float)exp2(-s2 * n);
}

// four consecutive elements as one vector access, widened to fp32
template <typename T> struct Vec4;
template <> struct Vec4<float> {
  static __device__ __forceinline__ void load(const float* p, float (&x)[4]) {
    const float4 v = *reinterpret_cast<const float4*>(p);
    x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
  }
  static __device__ __forceinline__ void store(float* p, const float (&x)[4]) {
    *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
  }
};
template <> struct Vec4<__nv_bfloat16> {
  static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&x)[4]) {
    const uint2 v = *reinterpret_cast<const uint2*>(p);
    const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v.x));
    const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v.y));
    x[0] = a.x; x[1] = a.y; x[2] = b.x; x[3] = b.y;
  }
  static __device__ __forceinline__ void store(__nv_bfloat16* p, const float (&x)[4]) {
    const __nv_bfloat162 a = __floats2bfloat162_rn(x[0], x[1]), b = __floats2bfloat162_rn(x[2], x[3]);
    uint2 v;
    v.x = *reinterpret_cast<const uint32_t*>(&a);
    v.y = *reinterpret_cast<const uint32_t*>(&b);
    *reinterpret_cast<uint2*>(p) = v;
  }
};

template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) {
  return __bfloat162float(x);
}
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) {
  return __float2bfloat16_rn(x);
}

}  // namespace la
