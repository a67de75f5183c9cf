/*
 * la.h -- C ABI of the B200 (sm_100a) library for causal linear attention with
 * per-head exponential decay.
 *
 * What is computed (per batch b and head h, independently):
 *
 *   forward   o_t = sum_{s<=t} lambda_h^(t-s) (q_t . k_s) v_s
 *             i.e. O = (Q K^T (.) M) V with M_ts = lambda^(t-s) for t >= s, else 0
 *             (Section 3.2.1 "Lightning Attention", Algorithm 3), which equals the
 *             recurrence kv_t = lambda kv_{t-1} + k_t v_t^T, o_t = kv_t^T q_t
 *             (Algorithm 2 "Robust Inference"; equivalence: Appendix C).
 *             No softmax and no 1/sqrt(d) scaling (Section 3.1.4).
 *   backward  dQ = dA K, dK = dA^T Q, dV = A^T dO with A = (Q K^T) (.) M and
 *             dA = (dO V^T) (.) M (Algorithm 4), for the loss <O, dO>.
 *   decode    one iteration of Algorithm 2 on a state kept by the caller.
 *
 * Conventions that hold for every entry point
 *   - Tensors are dense row-major with the feature dimension fastest:
 *     q,k,dq,dk [B,H,N,d]; v,o,dO,dv [B,H,N,e] (or [B,N,H,.] with la_shape.layout =
 *     LA_LAYOUT_BNHD); states [B,H,d,e] fp32 with kv[b,h,i,j] = sum_s lambda^(t-s) k_s[i] v_s[j].
 *   - Every tensor pointer is DEVICE memory, 16-byte aligned, owned by the caller.
 *     The library allocates no device memory, never frees and never synchronises
 *     the stream (la_device_status and la_profile_collect are the two calls that
 *     wait, and say so).  Inputs are not modified; outputs are fully overwritten;
 *     inputs and outputs must not alias (except the state of la_decode_step, which
 *     is updated in place).
 *   - State the library keeps between calls (everything else is per call): (1) one
 *     failure flag per device, shared by all streams and callers, written by a
 *     tensor-core block whose bounded wait expired and read by la_device_status;
 *     (2) per device, the three side streams and events of la_fwd_bwd_host,
 *     created on its first use; (3) the per-kernel timing records and the launch
 *     counter of the benchmark helpers (process-wide, off by default);
 *     (4) the fixed scratch array of la_fwd_noalloc, shared by all its callers on
 *     a device.  la_fwd, la_bwd, la_bwd_reuse and la_decode_step touch none of
 *     these except that their kernels may set (1), so concurrent calls from
 *     several host threads on different streams are safe.
 *   - `lambda_host` is HOST memory: H floats, each finite and in (0, 1].  It is
 *     read during the call (validated, converted to -log2(lambda) in double) and
 *     passed to the kernels by value; it need not outlive the call.
 *   - All work is enqueued on `stream`; the call returns without waiting.
 *   - Errors are reported by return code only.  Argument errors are found
 *     before anything is launched.  There is no CPU fallback: on a device that
 *     is not sm_100 the calls return LA_ERR_ARCH.
 *   - Supported in this version: d == e in {64, 128}; H <= 256;
 *     in_dtype BF16 with out_dtype F32 or BF16, or in = out = F32.
 *     Accumulation and states are always fp32.
 */
#ifndef LA_B200_H
#define LA_B200_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  LA_OK = 0,
  LA_ERR_INVALID_ARG = 1, /* null/misaligned pointer, bad size, lambda outside (0,1] */
  LA_ERR_UNSUPPORTED = 2, /* shape or dtype combination not built */
  LA_ERR_WORKSPACE = 3,   /* workspace missing or smaller than la_workspace_bytes() */
  LA_ERR_CUDA = 4,        /* a CUDA runtime/driver call or a launch failed */
  LA_ERR_ARCH = 5,        /* current device is not sm_100 */
  LA_ERR_DEVICE_TIMEOUT = 6, /* a bounded device-side wait expired (see la_device_status) */
  LA_ERR_SCRATCH_LIMIT = 7   /* la_fwd_noalloc: the shape needs more scratch than the built-in buffer holds */
} la_status;

typedef enum { LA_BF16 = 0, LA_F32 = 1 } la_dtype;

/* Which kernels run.  AUTO picks the tensor-core kernels where they exist
 * (bf16 inputs, d = e = 128 or d = e = 64) and the fp32 CUDA-core kernels otherwise
 * (fp32 inputs).  TENSOR fails with LA_ERR_UNSUPPORTED where they do not exist. */
typedef enum { LA_PATH_AUTO = 0, LA_PATH_SIMT = 1, LA_PATH_TENSOR = 2 } la_path;

/* la_shape.precision, tensor-core path only: bf16 operands formed on chip from fp32
 * values are carried as two bf16 terms (hi + lo).  Default: both bits set. */
#define LA_SPLIT_SCORES 1 /* the masked score tile (Q K^T) (.) D                      */
#define LA_SPLIT_STATE 2  /* the running state used as a matrix operand              */
#define LA_SPLIT_DECAYED 4 /* the decay-scaled value rows entering the state update  */
#define LA_PRECISION_DEFAULT (-1)

/* Layout of the token tensors (q, k, v, dO, o, dq, dk, dv, u, y): feature dimension always fastest.
 * LA_LAYOUT_BHND: [B,H,N,d] as in the operation's definition.  LA_LAYOUT_BNHD: [B,N,H,d], the layout a fused
 * Q/K/V/U projection of the token mixer leaves its output in (Eq. 3: the heads of one token are adjacent); rstd
 * follows as [B,N,H].  States are [B,H,d,e] in both.  la_fwd_bwd_host takes LA_LAYOUT_BHND only. */
typedef enum { LA_LAYOUT_BHND = 0, LA_LAYOUT_BNHD = 1 } la_layout;

typedef struct {
  int B, H, N, d, e;  /* N >= 1 (ignored by la_decode_step) */
  la_dtype in_dtype;  /* q, k, v, dO */
  la_dtype out_dtype; /* o, dq, dk, dv */
  int seg_len;        /* 0 = library chooses.  Otherwise the sequence is cut into
                         segments of this many tokens (a positive multiple of 128)
                         that run as independent thread blocks joined by a state scan. */
  int path;           /* la_path */
  int precision;      /* LA_PRECISION_DEFAULT or an OR of LA_SPLIT_* */
  int layout;         /* la_layout */
} la_shape;

#define LA_OP_FWD 0
#define LA_OP_BWD 1
#define LA_OP_DECODE 2

/* Bytes of device scratch the given op needs for this shape (0 is possible).
 * Returns (size_t)-1 if the shape is invalid or unsupported.  Linear in
 * B*H*d*e*ceil(N/seg_len); never grows with N^2: sets of [B,H,nseg,d,e] fp32 states,
 * two for the forward pass (0 with a single segment), three for the backward pass. */
size_t la_workspace_bytes(int op, const la_shape* shape);

/* The segment length the library will use for this shape (after applying
 * shape->seg_len), or 0 if the shape is invalid. */
int la_segment_length(const la_shape* shape);

/*
 * Forward pass (Section 3.2.1; Algorithm 3 defines the result, Algorithm 2 the
 * state).  o [B,H,N,e] <- (Q K^T (.) M) V, optionally continuing from a state:
 *   kv_in   [B,H,d,e] fp32 state before token 0, or NULL for zeros;
 *   kv_out  [B,H,d,e] fp32 state after the last token (no extra decay), or NULL.
 * With kv_in the result is o_t = kv_t^T q_t where kv_{-1} = kv_in.
 * workspace: device scratch of at least la_workspace_bytes(LA_OP_FWD, shape)
 * bytes, 256-byte aligned; may be NULL when that size is 0.  Calls that share a
 * workspace must be stream-ordered.  Afterwards the workspace holds the state
 * entering each segment and its transpose; la_bwd_reuse can take it to skip recomputing those.
 */
la_status la_fwd(const la_shape* shape, const void* q, const void* k, const void* v,
                 const float* lambda_host, void* o, const float* kv_in, float* kv_out,
                 void* workspace, size_t workspace_bytes, void* stream /* cudaStream_t */);

/*
 * Forward pass with the rest of the token mixer's output stage fused in (Eq. 3 "Gated Linear Attention" with
 * Eq. 8 "SimpleRMSNorm"): per batch, head and token, with o the e attention outputs of la_fwd,
 *   y = o / (||o||_2 / sqrt(e)) (.) u
 * (each head's e values are normalised on their own, as in the model-parallel form of Eq. 3; Eq. 8 has no
 * epsilon: a row with ||o||_2 = 0 gives y = 0).
 *   u     [B,H,N,e] gate, in_dtype;
 *   y     [B,H,N,e] out_dtype;
 *   o     [B,H,N,e] out_dtype, the attention output itself, or NULL if it is not wanted (inference); the
 *         backward of this stage (la_gate_bwd) needs it;
 *   rstd  [B,H,N] fp32, sqrt(e) / ||o||_2 per row, or NULL.
 * Everything else as for la_fwd.  At d = e = 128 on the tensor-core path, with y (and o) aligned to 32 bytes, the
 * epilogue runs inside the walk kernel and o is never written unless asked for; otherwise the attention output is
 * written (to o, or to y if o is NULL) and a row kernel turns it into y.
 */
la_status la_fwd_gated(const la_shape* shape, const void* q, const void* k, const void* v, const void* u,
                       const float* lambda_host, void* y, void* o, float* rstd, const float* kv_in, float* kv_out,
                       void* workspace, size_t workspace_bytes, void* stream);

/*
 * The same output stage on its own (Eq. 3 with Eq. 8), for an attention output that already sits in memory:
 *   y = o / (||o||_2 / sqrt(e)) (.) u;  o, y [B,H,N,e] out_dtype (they may be the same buffer), u in_dtype,
 *   rstd [B,H,N] fp32 or NULL.  One bandwidth-bound row kernel; this is what la_fwd_gated runs behind the walk
 *   where it cannot fuse.  shape->d is ignored.
 */
la_status la_gate_fwd(const la_shape* shape, const void* o, const void* u, void* y, float* rstd, void* stream);

/*
 * Backward of that output stage (the chain rule through Eq. 3 / Eq. 8): from d_y = dL/dy
 *   d_u = d_y (.) n,      d_o = s (g - n (n . g) / e),      n = o s,  s = sqrt(e) / ||o||_2,  g = d_y (.) u.
 *   o [B,H,N,e] out_dtype (as written by la_fwd_gated); u, d_y [B,H,N,e] in_dtype;
 *   d_o [B,H,N,e] in_dtype (it is what la_bwd takes as d_o); d_u [B,H,N,e] out_dtype.
 * One bandwidth-bound row kernel; needs no workspace.  shape->d is ignored.
 */
la_status la_gate_bwd(const la_shape* shape, const void* o, const void* u, const void* d_y, void* d_o, void* d_u,
                      void* stream);

/*
 * Backward pass (Algorithm 4 defines the result): gradients of
 * L = <O, dO> + <kv_out, grad_kv_out> with respect to q, k, v (and kv_in).
 *   d_o          [B,H,N,e] in in_dtype;
 *   dq, dk       [B,H,N,d], dv [B,H,N,e] in out_dtype;
 *   kv_in        the state given to la_fwd, or NULL;
 *   grad_kv_out  IN, [B,H,d,e] fp32, dL/d(kv_out), or NULL for zeros;
 *   grad_kv_in   OUT, [B,H,d,e] fp32, dL/d(kv_in), or NULL if not wanted.
 * lambda has no gradient (it is not learnable, Section 3.1.1).
 * workspace as for la_fwd with LA_OP_BWD.
 */
la_status la_bwd(const la_shape* shape, const void* q, const void* k, const void* v,
                 const void* d_o, const float* lambda_host, void* dq, void* dk, void* dv,
                 const float* kv_in, const float* grad_kv_out, float* grad_kv_in,
                 void* workspace, size_t workspace_bytes, void* stream);

/*
 * la_bwd that reuses the forward pass's segment states.  fwd_workspace is the workspace
 * a preceding la_fwd used for the SAME shape (incl. seg_len/path), inputs, lambda and
 * kv_in, untouched since; the dQ part of Algorithm 4 then starts from those states
 * instead of re-reading K and V in a pre-pass.  NULL, or a shape with a single segment,
 * makes it identical to la_bwd.  fwd_workspace must not overlap `workspace`.
 */
la_status la_bwd_reuse(const la_shape* shape, const void* q, const void* k, const void* v,
                       const void* d_o, const float* lambda_host, void* dq, void* dk, void* dv,
                       const float* kv_in, const float* grad_kv_out, float* grad_kv_in,
                       const void* fwd_workspace, void* workspace, size_t workspace_bytes, void* stream);

/*
 * One recurrent decode step (one iteration of Algorithm 2) for every (b,h):
 *   kv <- lambda_h kv + k v^T   (kv [B,H,d,e] fp32, updated IN PLACE)
 *   o  <- kv^T q                (o [B,H,e] in out_dtype)
 * q,k [B,H,d], v [B,H,e] in in_dtype.  shape->N is ignored.  Needs no workspace.
 * Holds no host state between calls, so a loop of steps may be stream-captured.
 */
la_status la_decode_step(const la_shape* shape, const void* q, const void* k, const void* v,
                         const float* lambda_host, float* kv, void* o, void* stream);

/*
 * LRPE-d (Eq. 1): decay times a learnable rotation of the relative position,
 *   a_ts = lambda^(t-s) sum_i q_t[i] k_s[i] cos(theta[h][i] (t-s)),  s <= t;   o_t = sum_{s<=t} a_ts v_s
 * (the real part of the printed complex form; one angle per head and feature).  The rotation splits into the
 * position features [x cos(theta t), x sin(theta t)], i.e. a doubled feature dimension 2d, and the result is the
 * sum of two runs of the decayed operator on the two halves, which is how these calls compute it.
 *   theta        DEVICE, [H,d] fp32, 16-byte aligned;       d_theta  OUT, DEVICE, [H,d] fp32 (overwritten);
 *   pos0         absolute position of the first token (>= 0; chunks of one sequence pass their offset);
 *   kv_in, kv_out, grad_kv_out, grad_kv_in   [2,B,H,d,e] fp32 (cos half, then sin half) or NULL;
 *   other arguments as in la_fwd / la_bwd; requires d == e.
 * Workspace: la_lrpe_workspace_bytes(op, shape), 256-byte aligned: the four feature tensors, fp32 temporaries of
 * the tensors' size (1-2 forward, 5-6 backward) and the inner calls' own workspace.
 * d_theta is a position-weighted sum whose q and k parts cancel down to the relative-position result; with
 * bf16 features its error grows with the absolute positions (see the tests for the bound that is checked).
 */
size_t la_lrpe_workspace_bytes(int op, const la_shape* shape);
la_status la_lrpe_fwd(const la_shape* shape, const void* q, const void* k, const void* v, const float* theta,
                      const float* lambda_host, long long pos0, void* o, const float* kv_in, float* kv_out,
                      void* workspace, size_t workspace_bytes, void* stream);
la_status la_lrpe_bwd(const la_shape* shape, const void* q, const void* k, const void* v, const void* d_o,
                      const float* theta, const float* lambda_host, long long pos0, void* dq, void* dk, void* dv,
                      float* d_theta, const float* kv_in, const float* grad_kv_out, float* grad_kv_in, void* workspace,
                      size_t workspace_bytes, void* stream);

/*
 * One sequence cut into consecutive chunks of chunk_tokens tokens (the last may be shorter), e.g. one chunk per GPU
 * of a sequence-parallel group.  Only Algorithm 2's d x e state crosses a cut, so the exchange between the chunks'
 * owners is one gather of [B,H,d,e] fp32 states per direction:
 *
 *   la_chunk_state   the chunk's own contribution, from its tokens alone:
 *                      reverse = 0:  b = k, c = v:    state_out = sum_s lambda^(n-1-s) k_s v_s^T
 *                                    (what la_fwd would return as kv_out from a zero kv_in);
 *                      reverse = 1:  b = q, c = d_o:  state_out = sum_t lambda^(t+1) q_t do_t^T
 *                                    (what la_bwd would return as grad_kv_in for a zero grad_kv_out).
 *                    shape describes the chunk (N = its tokens).  workspace: la_chunk_state_workspace_bytes(shape),
 *                    256-byte aligned.
 *   la_chain_states  the state at a cut from the gathered contributions `states` [num_chunks,B,H,d,e]:
 *                      reverse = 0:  state_out = the state entering chunk `chunk` (kv_in of its la_fwd / la_bwd),
 *                                    z = boundary; for j = 0 .. chunk-1: z = lambda^(n_j) z + states[j];
 *                                    chunk = num_chunks gives the kv_out of the whole sequence;
 *                      reverse = 1:  state_out = grad_kv_out of chunk `chunk`'s la_bwd,
 *                                    z = boundary; for j = num_chunks-1 down to chunk+1: z = lambda^(n_j) z + states[j];
 *                                    chunk = -1 gives the grad_kv_in of the whole sequence.
 *                    boundary: the whole sequence's kv_in (reverse = 0) or grad_kv_out (reverse = 1), or NULL.
 *                    shape gives B, H, d, e (N is ignored); total_tokens and chunk_tokens give every n_j.
 * The results of la_fwd / la_bwd on the chunks with these states are those of the whole sequence on one device.
 */
size_t la_chunk_state_workspace_bytes(const la_shape* shape);
la_status la_chunk_state(const la_shape* shape, int reverse, const void* b, const void* c, const float* lambda_host,
                         float* state_out, void* workspace, size_t workspace_bytes, void* stream);
la_status la_chain_states(const la_shape* shape, long long total_tokens, long long chunk_tokens, int reverse,
                          const float* states, int num_chunks, int chunk, const float* boundary,
                          const float* lambda_host, float* state_out, void* stream);

/*
 * Packed batches of sequences of different lengths (the serving-side form of Algorithm 2: every sequence has its
 * own state).  The token tensors are [T, H, d] with the num_seqs sequences one after the other: shape->B = 1,
 * shape->N = T, shape->layout = LA_LAYOUT_BNHD; cu_seqlens_host (HOST memory, num_seqs + 1 ints, cu[0] = 0,
 * cu[num_seqs] = T, strictly increasing) gives the first token of each sequence.  Sequence i runs
 * from the state kv_in[i] (or zero) and leaves kv_out[i]; kv_in, kv_out, grad_kv_out, grad_kv_in are
 * [num_seqs, H, d, e] fp32 or NULL.  Results are those of la_fwd / la_bwd on each sequence alone.
 * bf16 inputs at d = e = 128 with outputs aligned to 32 bytes (and more than one sequence) run as ONE set of
 * launches over all sequences: every (sequence, head[, segment]) is a thread block of the tensor-core kernels, which
 * take each sequence's first token and length from a small table the call copies to the head of the workspace
 * (a host-to-device copy on `stream` from pageable memory: such a call cannot be captured into a graph).  Other
 * shapes enqueue one la_fwd / la_bwd per sequence on `stream`.  la_varlen_workspace_bytes covers both.
 */
size_t la_varlen_workspace_bytes(int op, const la_shape* shape, const int* cu_seqlens_host, int num_seqs);
la_status la_fwd_varlen(const la_shape* shape, const void* q, const void* k, const void* v, const float* lambda_host,
                        void* o, const int* cu_seqlens_host, int num_seqs, const float* kv_in, float* kv_out,
                        void* workspace, size_t workspace_bytes, void* stream);
la_status la_bwd_varlen(const la_shape* shape, const void* q, const void* k, const void* v, const void* d_o,
                        const float* lambda_host, void* dq, void* dk, void* dv, const int* cu_seqlens_host, int num_seqs,
                        const float* kv_in, const float* grad_kv_out, float* grad_kv_in, void* workspace,
                        size_t workspace_bytes, void* stream);

/*
 * Several recurrent decode steps in one call (Algorithm 2 iterated over shape->N >= 1 consecutive tokens): for
 * t = 0 .. N-1 in order,  kv <- lambda_h kv + k_t v_t^T,  o_t <- kv^T q_t.
 *   q, k [B,H,N,d], v [B,H,N,e] in in_dtype; o [B,H,N,e] in out_dtype; kv [B,H,d,e] fp32, updated IN PLACE once.
 * The state is read once, kept on chip over the N tokens and written once, so a handful of tokens decoded together
 * (speculative decoding, a short chunk of a prompt) costs one pass over the state instead of N.  The tokens are
 * processed one after the other; for long chunks la_fwd with kv_in / kv_out is the faster route.  Same result
 * as N calls of la_decode_step, bit for bit.  Needs no workspace, keeps no host state.
 */
la_status la_decode_steps(const la_shape* shape, const void* q, const void* k, const void* v,
                          const float* lambda_host, float* kv, void* o, void* stream);

/*
 * Forward pass without caller-provided scratch (the paper has no counterpart; this is a
 * deployment convenience).  Same result as la_fwd, but the per-segment state scratch comes
 * from a fixed LA_NOALLOC_SCRATCH_BYTES array that is part of the library's device image,
 * for callers that cannot allocate device memory when they call: a server that gave all
 * device memory to its own pool at start-up, a latency-critical loop that must avoid the
 * device-wide synchronisation of an allocation, or a plug-in that is handed only tensor
 * pointers and a stream.  Inputs and outputs are still the caller's.
 *   - Every GPU that loads the library holds the 32 MiB array until the process exits.
 *     With lazy module loading (the CUDA default) the array may only be materialised
 *     when its address is first asked for, that is, inside the first call on a device:
 *     make that warm-up call before the caller's own pool takes the rest of the
 *     device memory, or it can fail with LA_ERR_CUDA for lack of room.
 *   - Shapes with la_workspace_bytes(LA_OP_FWD, shape) > LA_NOALLOC_SCRATCH_BYTES are
 *     rejected with LA_ERR_SCRATCH_LIMIT before anything is launched.
 *   - The first call on each device looks up the array's device address (once, with that
 *     device current); make that first call before any stream capture begins.
 *   - All calls on a device share the array: calls that can overlap on the GPU (different
 *     streams) race on it; calls ordered on one stream are safe.  The array keeps the last
 *     call's contents, which needs no clearing: the forward pass writes every scratch
 *     element before reading it.
 * The call itself performs no cudaMalloc / cudaFree and uses no allocating library routine.
 */
#define LA_NOALLOC_SCRATCH_BYTES (32u << 20)
la_status la_fwd_noalloc(const la_shape* shape, const void* q, const void* k, const void* v,
                         const float* lambda_host, void* o, const float* kv_in, float* kv_out,
                         void* stream);

/*
 * Forward + backward with HOST tensors (end-to-end convenience; the paper has no
 * counterpart).  q,k,v,d_o and o,dq,dk,dv are host pointers with the layouts and
 * dtypes of la_fwd / la_bwd (pinned memory makes the copies asynchronous).  The
 * call enqueues the four host-to-device copies, la_fwd, la_bwd (zero initial
 * state, no state gradients) and the four device-to-host copies.  Heads are
 * independent, so for H >= 3 the work is cut into groups of heads that run as
 * copy-in -> forward -> backward -> copy-out chains on three side streams owned
 * by the library (created on first use, one set per device): copies of one
 * group overlap the kernels and the opposite-direction copies of its
 * neighbours.  The side streams start after all work queued on `stream` before
 * the call, and `stream` continues only after they have finished, so to the
 * caller the call behaves as if everything had been enqueued on `stream`.
 * Calls from several host threads are enqueued one at a time and share the side
 * streams, so they run one after the other on the device.  device_arena is caller-owned device scratch of at least
 * la_host_arena_bytes(shape) bytes, 256-byte aligned; it holds the device copies
 * of all eight tensors and the workspace.  Host outputs are valid once `stream`
 * has been synchronised by the caller.
 */
size_t la_host_arena_bytes(const la_shape* shape);
la_status la_fwd_bwd_host(const la_shape* shape, const void* q_host, const void* k_host,
                          const void* v_host, const void* d_o_host, const float* lambda_host,
                          void* o_host, void* dq_host, void* dk_host, void* dv_host,
                          void* device_arena, size_t arena_bytes, void* stream);

/*
 * Device-side failure flag (no counterpart in the paper).  The tensor-core kernels
 * never spin without limit: a thread block whose wait on a copy or on the tensor
 * cores expires records a code, drains what it started and returns, leaving its
 * part of the output unwritten; la_fwd / la_bwd have returned LA_OK long before,
 * so a caller that wants to know asks here.  The flag is one word per DEVICE, not
 * per stream or per call: it keeps the first code any block recorded since it was
 * last cleared, whoever launched that block.  This call waits until the whole
 * device is idle (cudaDeviceSynchronize), takes the flag and clears it in one
 * atomic exchange on the device, stores the raw code in *code if code is not
 * NULL, and returns LA_OK if no block failed, else LA_ERR_DEVICE_TIMEOUT.  With
 * several callers on one device, whoever calls first sees (and clears) the code.
 */
la_status la_device_status(unsigned int* code);

/*
 * Self-test of that failure path (no counterpart in the paper): launches one warp
 * that waits, with the kernels' own bounded wait, on a barrier nothing ever arrives
 * on.  After budget_clocks SM clocks (1 .. 2e9; 2e6 is about a millisecond) the
 * wait gives up, records code 99 and the kernel returns normally; the next
 * la_device_status() reports LA_ERR_DEVICE_TIMEOUT with that code and the context
 * stays usable.  Nothing faults, traps or spins without limit.
 */
la_status la_selftest_bounded_wait(unsigned long long budget_clocks, void* stream);

/* Human-readable name of a status code (static string). */
const char* la_status_string(la_status s);

/* Library version: major*10000 + minor*100 + patch. */
int la_version(void);

/* Number of kernels this library has launched in the calling process since load
 * (monotonic counter, relaxed atomics; for benchmarks that report launch counts). */
unsigned long long la_launch_count(void);

/*
 * Optional per-kernel timing for benchmarks (no counterpart in the paper).
 * While enabled, every kernel the library launches is bracketed by a pair of
 * CUDA events recorded on the caller's stream.  la_profile_collect waits for
 * those events, adds the elapsed milliseconds and launch counts per kernel kind
 * into ms[LA_NUM_KERNEL_KINDS] / launches[LA_NUM_KERNEL_KINDS] (both are
 * overwritten), releases the events and returns LA_OK.  The records are
 * process-wide state; profiling is off by default, guarded by a mutex, and must
 * not be enabled while a stream is being captured.  It adds event records between
 * the launches, so a loop timed as a whole should run with it off.
 */
#define LA_KERNEL_PREPASS 0 /* segment-local states            */
#define LA_KERNEL_SCAN 1    /* state scan across segments      */
#define LA_KERNEL_WALK 2    /* block walk producing o/dq/dk/dv */
#define LA_KERNEL_DECODE 3  /* recurrent decode step           */
#define LA_KERNEL_WALK_PAIR 4 /* the dV and dK walks of the backward pass in one launch */
#define LA_KERNEL_GATE 5      /* stand-alone SRMSNorm-and-gate kernels (la_fwd_gated fallback, la_gate_bwd) */
#define LA_KERNEL_LRPE 6      /* element-wise kernels of la_lrpe_fwd / la_lrpe_bwd */
#define LA_NUM_KERNEL_KINDS 7
void la_profile_enable(int on);
la_status la_profile_collect(double* ms, unsigned long long* launches);

#ifdef __cplusplus
}
#endif
#endif /* LA_B200_H */
