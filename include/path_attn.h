/*
 * path_attn.h -- C ABI of the PaTH attention library for NVIDIA B200 (sm_100a).
 *
 * PaTH attention (paper Sec. 2.1-2.2) is causal softmax attention whose logit
 * between query i and key j <= i is
 *
 *     s_ij = scale * k_j^T ( H_{j+1} H_{j+2} ... H_i ) q_i + sum_{t=j+1..i} log f_t ,
 *     H_t  = I - beta_t w_t w_t^T ,
 *
 * where the log f_t term (PaTH-FoX, paper Sec. 2.2 "Extension") is optional.
 * The library computes it blockwise (paper Sec. 3.1-3.3): a per-chunk compact
 * (UT transform) representation of the Householder products, boundary-adjusted
 * queries and keys, chunk products, and a FlashAttention-style sweep with an
 * online softmax.
 *
 * Conventions shared by every entry point
 *   - All data pointers are DEVICE pointers owned by the caller, 16-byte
 *     aligned, contiguous row-major.  q, k, v, w, o, d_o, dq, dk, dv, dw are
 *     [B, H, L, d] in the I/O dtype `dt`; beta, log_f, lse, dbeta, dlog_f are
 *     [B, H, L] float32.  d is 64 or 128; L >= 1 is arbitrary.
 *   - Inputs are read-only.  Outputs are fully overwritten.  Nothing is
 *     allocated: scratch memory is the caller's `workspace` of at least
 *     path_attn_workspace_bytes(...) bytes (256-byte aligned), which a call may
 *     overwrite entirely.  Two calls may run concurrently only with distinct
 *     workspaces.
 *   - Calls are asynchronous on `cuda_stream` (a cudaStream_t passed as void*;
 *     NULL is the default stream) and never synchronise it.
 *   - Return value: PATH_OK or a negative path_status_t.  Argument errors are
 *     detected on the host before anything is launched.  There is no CPU
 *     fallback: an unsupported argument is an error.
 *   - w and beta are used as given (no normalisation, no clipping).  `scale`
 *     multiplies the bilinear term only; the gate is added after scaling.
 *   - Device-side waits are bounded.  If one runs out, the kernel records it in
 *     a status word at the start of the workspace and returns; read it with
 *     path_attn_device_status after synchronising the stream.
 */
#ifndef PATH_ATTN_H_
#define PATH_ATTN_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

/* I/O dtype of q, k, v, w, o and their gradients.
 * PATH_BF16: bf16 tensor-core products with float32 accumulation (the training path, forward and backward).
 * PATH_FP32: forward only; the definition of Sec. 2.2 evaluated in float32 on the CUDA cores (one warp per query
 * position carrying u <- H_j u over the keys), O(L^2 d) work: an accuracy path for float32 tensors, not a fast one.
 * path_attn_bwd and for_backward = 1 do not accept it. */
typedef enum { PATH_BF16 = 0, PATH_FP32 = 1 } path_dtype_t;

typedef enum {
    PATH_OK = 0,
    PATH_ERR_NULL = -1,      /* a required pointer is NULL, or dlog_f / log_f given without the other */
    PATH_ERR_SHAPE = -2,     /* d not in {64,128}, or B, H, L < 1, or sizes overflow */
    PATH_ERR_DTYPE = -3,     /* unknown dtype, or dtype not supported by this entry point */
    PATH_ERR_ALIGN = -4,     /* a pointer is not 16-byte aligned (workspace: 256-byte) */
    PATH_ERR_WORKSPACE = -5, /* workspace_bytes too small */
    PATH_ERR_ARCH = -6,      /* current device is not compute capability 10.x */
    PATH_ERR_LAUNCH = -7,    /* a CUDA runtime / driver call failed (see path_attn_last_cuda_error) */
    PATH_ERR_TIMEOUT = -8,   /* reported by path_attn_device_status: a bounded device wait ran out */
    PATH_ERR_STATIC_LIMIT = -9, /* path_attn_fwd_static: the problem needs more scratch than the built-in buffer holds */
    PATH_ERR_STATE = -10     /* reported by path_attn_device_status after path_attn_bwd_reuse: the workspace does not
                                hold the forward state of this problem; the gradients of that call are invalid */
} path_status_t;

/* Bytes of scratch memory path_attn_fwd (for_backward = 0) or path_attn_bwd
 * (for_backward = 1) needs for this problem.  Returns 0 for invalid arguments
 * (PATH_FP32 with for_backward = 1 is one). */
size_t path_attn_workspace_bytes(int B, int H, int L, int d, path_dtype_t dt, int has_gate,
                                 int for_backward);

/*
 * Forward (paper Sec. 3.3): o_i = sum_{j<=i} softmax_j(s_ij) v_j and
 * lse_i = log sum_{j<=i} exp(s_ij) (natural log, scale and gate included).
 *   q,k,v,w : [B,H,L,d] in dt          beta  : [B,H,L] float32
 *   log_f   : [B,H,L] float32 per-step log f_t, or NULL for plain PaTH
 *   o       : [B,H,L,d] in dt (out)    lse   : [B,H,L] float32 (out)
 * Bitwise reproducible from run to run.
 */
int path_attn_fwd(const void* q, const void* k, const void* v, const void* w, const float* beta,
                  const float* log_f, void* o, float* lse, int B, int H, int L, int d, float scale,
                  path_dtype_t dt, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Backward of the same function (the paper gives no backward; this is the chain
 * rule through the Sec. 3.1-3.3 formulation): given d_o it returns the gradients
 * of sum(o * d_o).
 *   o, lse  : the forward's outputs for the same inputs
 *   d_o     : [B,H,L,d] in dt
 *   dq,dk,dv,dw : [B,H,L,d] in dt (out)   dbeta : [B,H,L] float32 (out)
 *   dlog_f  : [B,H,L] float32 (out); must be NULL exactly when log_f is NULL
 * dt must be PATH_BF16.  Bitwise reproducible from run to run, like the forward
 * (nothing on this path is accumulated atomically).
 *
 * path_attn_bwd always recomputes the chunk preparation (Sec. 3.1 / 3.3
 * quantities) from q, k, w, beta, log_f: it depends on nothing a previous call
 * left in the workspace.
 *
 * path_attn_bwd_reuse (same arguments) is the explicit request to skip that
 * recomputation.  Contract: the last call on `workspace` was path_attn_fwd for
 * this very problem (same pointers q, k, v, w, beta, log_f, same shape and,
 * when log_f is given, the same scale), the workspace was at least
 * path_attn_workspace_bytes(..., for_backward = 1) bytes in that call too, and
 * since then neither the workspace nor the contents of q, k, w, beta, log_f
 * have been written to.  A forward that runs on a backward-sized workspace ends
 * by writing a record of its problem into the workspace; path_attn_bwd_reuse
 * compares that record on the device before anything reads the state, and a
 * mismatch (another problem, a forward-sized forward, a call in between) is
 * reported by path_attn_device_status as PATH_ERR_STATE, in which case the
 * outputs of the call are invalid.  The record cannot see a caller that
 * rewrites an input buffer in place: that is the caller's side of the contract.
 * Holding the state costs the whole backward-sized workspace from forward to
 * backward; recomputing costs the preparation stages once more.
 */
int path_attn_bwd(const void* q, const void* k, const void* v, const void* w, const float* beta,
                  const float* log_f, const void* o, const float* lse, const void* d_o, void* dq,
                  void* dk, void* dv, void* dw, float* dbeta, float* dlog_f, int B, int H, int L,
                  int d, float scale, path_dtype_t dt, void* workspace, size_t workspace_bytes,
                  void* cuda_stream);
int path_attn_bwd_reuse(const void* q, const void* k, const void* v, const void* w, const float* beta,
                        const float* log_f, const void* o, const float* lse, const void* d_o, void* dq,
                        void* dk, void* dv, void* dw, float* dbeta, float* dlog_f, int B, int H, int L,
                        int d, float scale, path_dtype_t dt, void* workspace, size_t workspace_bytes,
                        void* cuda_stream);

/*
 * Forward pass for callers that cannot allocate device memory (the paper has no
 * counterpart; this is a packaging variant of path_attn_fwd).
 *
 * Some hosts of this library may not call cudaMalloc at the point where they
 * need attention: code running while a stream is being captured into a CUDA
 * graph, plug-ins inside a serving runtime that has already handed every free
 * byte of the device to its own pool, and latency-critical loops in which the
 * implicit device synchronisation of cudaMalloc / cudaFree is not acceptable.
 * For them the scratch memory is not a caller workspace but a fixed buffer of
 * PATH_ATTN_STATIC_SCRATCH_BYTES that is part of the library image itself: every
 * GPU on which the library is loaded holds that buffer until the process exits.
 *
 * Arguments are those of path_attn_fwd without the workspace.  The call computes
 * exactly what path_attn_fwd computes and allocates nothing: no cudaMalloc, no
 * cudaFree, no allocating library routine.  A problem whose
 * path_attn_workspace_bytes(..., for_backward = 0) exceeds
 * PATH_ATTN_STATIC_SCRATCH_BYTES is rejected with PATH_ERR_STATIC_LIMIT before
 * anything is launched (roughly: B*H*L up to a few thousand tokens at d = 128).
 *
 * The first call on each device looks up the buffer's device address (once per
 * device, with that device current) and may trigger the driver's one-time module
 * loading; make that first call outside of any stream capture.
 * All calls on one device share the one buffer, and it keeps whatever the
 * previous call left in it: the call clears the status word it needs at zero and
 * overwrites every other region before reading it, so back-to-back calls on one
 * stream are safe, but two calls that overlap on the GPU (different streams, or
 * different host threads) race on the buffer and must be serialised by the caller.
 * Stage timing (path_attn_profile_enable) is ignored by this entry point.
 * If scratch_out is not NULL it receives the buffer's device address, which may
 * be passed to path_attn_device_status as the `workspace` of this call.
 */
#define PATH_ATTN_STATIC_SCRATCH_BYTES (16u << 20)
int path_attn_fwd_static(const void* q, const void* k, const void* v, const void* w, const float* beta,
                         const float* log_f, void* o, float* lse, int B, int H, int L, int d, float scale,
                         path_dtype_t dt, void* cuda_stream, void** scratch_out);

/*
 * Inference with a key cache (paper Sec. 3.4).  For every past position j the cache holds the key as the transitions
 * after it have left it, kc_j = H_{t-1} ... H_{j+1} k_j, so that a new query needs plain dot products:
 *   kc : [B,H,cap,d] float32 (float32 because every decoding step rewrites the whole cache in place)
 *   vc : [B,H,cap,d] bf16 values as given          gc : [B,H,cap] float32 gate prefix sums (PaTH-FoX), or NULL
 * cap >= 1 is the capacity in tokens; dt must be PATH_BF16 (dtype of the per-token inputs and of o).
 *
 * path_attn_prefill_cache fills positions 0..L-1 from a whole prompt: kc[.,.,j,:] = H_{L-1} ... H_{j+1} k_j, vc <- v
 * and, when log_f and gc are given (both or neither), gc <- inclusive prefix sums of log_f.  Needs
 * path_attn_workspace_bytes(B, H, L, d, PATH_BF16, has_gate, 0) bytes of workspace, which it overwrites.
 *
 * path_attn_decode_step processes the token at position t = number of cached tokens (0 <= t < cap):
 *   kc_j <- kc_j - beta_t w_t (w_t . kc_j) for j < t;  kc_t <- k_t, vc_t <- v_t, gc_t <- gc_{t-1} + log_f_t;
 *   o_t = sum_{j<=t} softmax_j(scale * q_t . kc_j + gc_t - gc_j) vc_j,   lse_t = log of the softmax's normaliser.
 * q_t, k_t, v_t, w_t, o_t : [B,H,d] bf16;  beta_t, log_f_t, lse_t : [B,H] float32 (log_f_t NULL iff gc NULL).
 * One pass over the cache (memory-bound).  Needs path_attn_decode_workspace_bytes(B, H, cap, d) bytes.
 * Same conventions as the entry points above: device pointers, asynchronous on cuda_stream, no allocation.
 */
int path_attn_prefill_cache(const void* k, const void* v, const void* w, const float* beta, const float* log_f,
                            float* kc, void* vc, float* gc, int B, int H, int L, int d, int cap, path_dtype_t dt,
                            void* workspace, size_t workspace_bytes, void* cuda_stream);
size_t path_attn_decode_workspace_bytes(int B, int H, int cap, int d);
int path_attn_decode_step(const void* q_t, const void* k_t, const void* v_t, const void* w_t, const float* beta_t,
                          const float* log_f_t, float* kc, void* vc, float* gc, int t, int cap, void* o_t,
                          float* lse_t, int B, int H, int d, float scale, path_dtype_t dt, void* workspace,
                          size_t workspace_bytes, void* cuda_stream);

/*
 * Context-parallel PaTH (paper Sec. 3.5, "Compatibility with context-parallelism"): the sequence is cut into
 * contiguous segments, one per device; every device first handles its own segment, then the (transformed keys, values,
 * segment product) of each EARLIER segment pass by, nearest first, and are attended by the resident queries.  These calls
 * are the per-device arithmetic of that scheme; they run on one GPU and know nothing about how a message travels
 * (paper_2505_16381_b200/ring.py holds a ring schedule over torch.distributed send / recv, which copies every incoming
 * message into this GPU's own memory before a kernel reads it).
 *
 *   path_attn_cp_prepare   this device's segment q, k, v, w [B,H,L,d] bf16, beta, log_f (or NULL) [B,H,L] float32
 *        -> `state`   (path_attn_cp_state_bytes): the queries pulled back to the segment's start, x_i = (H_s ... H_i q_i)
 *                     with s the segment's first position, as bf16 tiles; their gate terms; and the running result
 *                     (float32 O, normalised, with its LSE) initialised with the segment's own causal attention;
 *        -> `message` (path_attn_cp_message_bytes): the keys advanced to the segment's end, H_e ... H_{j+1} k_j with e
 *                     the segment's last position (Sec. 3.4's key transform), the values, the product of the segment's
 *                     transitions P = H_s ... H_e as a bf16 hi + lo pair, and the gate sums from each key to the
 *                     segment's end.  One contiguous buffer: what travels along the ring.
 *   path_attn_cp_step      `state` (Lq positions) meets the `message` of an earlier segment (Lk positions): plain
 *        softmax attention of x against the transformed keys (no mask: every key is earlier), merged into the
 *        running (O, LSE); then the queries move on past that segment, x <- x P  (the paper's in-place query update),
 *        and their gate terms grow by the segment's total.  Messages must arrive nearest segment first.
 *   path_attn_cp_finish    o [B,H,L,d] bf16 and lse [B,H,L] float32 from the state.
 * After prepare, step for every earlier segment and finish, (o, lse) equal path_attn_fwd's rows for this segment on
 * the whole sequence, up to rounding (x is re-rounded to bf16 once per step; the running result is float32).
 * Forward only.  state, message and workspace are device buffers, 256-byte aligned, caller-owned;
 * path_attn_cp_workspace_bytes(B, H, L, d, has_gate) covers prepare and step for a state of L positions.  Segments
 * may differ in length.  dt must be PATH_BF16.  Same conventions as above (asynchronous, no allocation, error codes;
 * the status word is at the start of `workspace`).
 */
size_t path_attn_cp_state_bytes(int B, int H, int L, int d);
size_t path_attn_cp_message_bytes(int B, int H, int L, int d);
size_t path_attn_cp_workspace_bytes(int B, int H, int L, int d, int has_gate);
int path_attn_cp_prepare(const void* q, const void* k, const void* v, const void* w, const float* beta,
                         const float* log_f, void* state, void* message, int B, int H, int L, int d, float scale,
                         path_dtype_t dt, void* workspace, size_t workspace_bytes, void* cuda_stream);
int path_attn_cp_step(void* state, const void* message, int B, int H, int Lq, int Lk, int d, float scale,
                      void* workspace, size_t workspace_bytes, void* cuda_stream);
int path_attn_cp_finish(const void* state, void* o, float* lse, int B, int H, int L, int d, void* cuda_stream);

/*
 * Layer front-end: how a PaTH layer obtains the operator's w, beta and log_f (paper Sec. 2.2, footnote to the
 * definition of H_t; gate of Sec. 2.4).  The low-rank layer giving z is path_attn_lowrank_fwd / _bwd below; the two
 * logits u^T x + b are one matrix-vector product per head and stay with the caller; these two calls are the rest:
 *   y_t[c]  = conv_w[c][0] z_{t-2}[c] + conv_w[c][1] z_{t-1}[c] + conv_w[c][2] z_t[c]   (causal, depthwise, z = 0 before t = 0)
 *   w_t     = y_t / sqrt(sum over the head's d channels of y_t^2 + eps)               (per head)
 *   beta_t  = 2 sigmoid(beta_logit_t),      log_f_t = log sigmoid(gate_logit_t)
 * Layouts: z, dz : [B,L,H*d] bf16 (head h owns channels h*d .. h*d+d-1);  conv_w, dconv_w : [H*d,3] float32;
 *   beta_logit, gate_logit and their gradients : [B,L,H] float32;  w, dw : [B,H,L,d] bf16;
 *   beta, log_f, dbeta, dlog_f : [B,H,L] float32  (the operator's layouts: the calls also do the change of layout).
 * gate_logit, log_f, dlog_f, dgate_logit are all NULL for plain PaTH and all given for PaTH-FoX.  eps >= 0.
 * path_attn_frontend_bwd returns the gradients of sum(w*dw) + sum(beta*dbeta) + sum(log_f*dlog_f); dconv_w is
 * summed with float32 atomics (reproducible to rounding, not bitwise).  Float32 arithmetic, one pass over the
 * tensors (memory-bound), no workspace.  Same conventions as above: device pointers, outputs fully overwritten,
 * asynchronous on cuda_stream, argument errors detected on the host.
 */
/*
 * The low-rank linear layer in front of them (paper Sec. 2.2, same footnote: "a low-rank linear layer followed by a
 * short convolution and L2 normalisation"), forward and backward, as tcgen05 products inside this library:
 *     t = x W1^T  [M, r],    z = t W2^T  [M, C]              x : [M, D] bf16 (M = B*L rows of the layer's input)
 *     dt = dz W2,  dW2 = dz^T t,  dx = dt W1,  dW1 = dt^T x    W1 : [r, D], W2 : [C, r] bf16 (nn.Linear layouts), C = H*d
 * t, z, dx are bf16 (t is the forward's by-product the backward takes back); dW1 [r, D] and dW2 [C, r] are float32,
 * fully overwritten, summed over the M rows with float32 atomics (reproducible to rounding).  D and C multiples of 64,
 * r = 64 or 128.  z is what path_attn_frontend_fwd takes (viewed as [B, L, H*d]) and dz what path_attn_frontend_bwd
 * returns.  workspace: path_attn_lowrank_workspace_bytes(M, D, r, C) bytes, 256-byte aligned (status word + dt).
 * Same conventions as above: device pointers, asynchronous on cuda_stream, no allocation, error codes.
 */
size_t path_attn_lowrank_workspace_bytes(long long M, int D, int r, int C);
int path_attn_lowrank_fwd(const void* x, const void* w1, const void* w2, void* t, void* z, long long M, int D, int r, int C,
                          void* workspace, size_t workspace_bytes, void* cuda_stream);
int path_attn_lowrank_bwd(const void* x, const void* w1, const void* w2, const void* t, const void* dz, void* dx,
                          float* dw1, float* dw2, long long M, int D, int r, int C, void* workspace, size_t workspace_bytes,
                          void* cuda_stream);

int path_attn_frontend_fwd(const void* z, const float* conv_w, const float* beta_logit, const float* gate_logit,
                           void* w, float* beta, float* log_f, int B, int H, int L, int d, float eps,
                           void* cuda_stream);
int path_attn_frontend_bwd(const void* z, const float* conv_w, const float* beta_logit, const float* gate_logit,
                           const void* dw, const float* dbeta, const float* dlog_f, void* dz, float* dconv_w,
                           float* dbeta_logit, float* dgate_logit, int B, int H, int L, int d, float eps,
                           void* cuda_stream);

/*
 * Block skipping in gated problems (the paper notes, Sec. 2.4, that PaTH-FoX stays compatible with FoX's pruning of
 * negligible blocks).  When log_f is given, path_attn_fwd leaves out every (query chunk, key chunk) pair of 128 x 128
 * positions whose logits are all provably more than 30 nats below the largest logit of their rows (the bound uses
 * |k| |q|, the norm bounds of the H_t in between and the accumulated gate; exp(-30) is far below bf16 resolution), and
 * with it every farther key chunk of that query chunk.  Results are unchanged within the stated tolerances; plain PaTH
 * (log_f == NULL) never skips.  This call reports, for the last gated path_attn_fwd on `workspace` (until another call
 * uses the workspace), how many chunk pairs were computed and how many a full causal sweep has.  Synchronises
 * `cuda_stream`.
 */
int path_attn_skipped_chunk_pairs(const void* workspace, void* cuda_stream, unsigned long long* kept,
                                  unsigned long long* all);

/* Reads the device status word the last call on this workspace left behind.
 * Synchronises `cuda_stream`.  Returns PATH_OK, PATH_ERR_TIMEOUT (a bounded
 * wait ran out), PATH_ERR_STATE (path_attn_bwd_reuse found no matching forward
 * state), or PATH_ERR_LAUNCH if the copy itself failed.  If `detail` is not
 * NULL it receives the raw status word (0 = clean; otherwise a code naming the
 * wait: 0x1xx forward sweep, 0x2xx dK/dV sweep, 0x3xx dQ sweep, 0x401 chunk
 * preparation, 0x501 chunk chain rule, 0x601 level kernels, 0x701 state
 * mismatch, 0x7f1 the self-test below). */
int path_attn_device_status(const void* workspace, void* cuda_stream, unsigned int* detail);

/*
 * Self-test of the bounded-wait machinery (no counterpart in the paper).  Every
 * device-side wait of the library (on an mbarrier fed by TMA or by tcgen05
 * commits) gives up after a time limit, raises its CTA's abort flag, lets the
 * kernel wind down and leaves a code in the status word.  This call runs that
 * very wait routine on a barrier nothing ever arrives on, with a limit of
 * `limit_us` microseconds (1 .. 100000) instead of the library's ~1 s, so that
 * the path from an expired wait to PATH_ERR_TIMEOUT can be exercised without a
 * fault or a hang: afterwards path_attn_device_status(workspace, ...) returns
 * PATH_ERR_TIMEOUT with detail 0x7f1.  Only the first 256 bytes of `workspace`
 * (256-byte aligned) are written.  Asynchronous on cuda_stream.
 */
int path_attn_selftest_timeout(void* workspace, unsigned int limit_us, void* cuda_stream);

/* Static description of a status code. */
const char* path_attn_strerror(int status);

/*
 * Optional stage timing for benchmarks (no counterpart in the paper).  After
 * path_attn_profile_enable(1), every fwd / bwd call of the calling thread records
 * CUDA events on its stream around its stages: "chunk_prep" (UT transform and
 * boundary-adjusted tiles, Sec. 3.1/3.3, one kernel), "levels_fwd" (run products
 * and versions, several launches), "fa_fwd" (the fused sweep, one kernel); and
 * for bwd "bwd_chunk_prep" and "bwd_levels_fwd" (the same preparation,
 * recomputed), "rowstats", "fa_bwd_dkv", "fa_bwd_dq", "bwd_chunk_chain" (one
 * kernel each), "bwd_levels" (several launches) and "bwd_gate".  path_attn_profile_read waits for those events and writes the
 * milliseconds per stage of the most recent fwd and the most recent bwd call
 * into ms[0..n) (-1 for a stage that did not run); it returns the number of entries written or a
 * negative status.  The events are created on first use and live until the
 * thread exits; nothing else is allocated.
 */
int path_attn_profile_enable(int on);
int path_attn_profile_read(float* ms, int n);
const char* path_attn_profile_stage_name(int i);

/* cudaError_t (as int) of the CUDA call behind the calling thread's most recent PATH_ERR_LAUNCH. */
int path_attn_last_cuda_error(void);

/* Number of kernel launches the calling thread's most recent fwd / bwd call issued. */
int path_attn_last_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* PATH_ATTN_H_ */
