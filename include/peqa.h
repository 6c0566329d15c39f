/*
 * peqa.h -- C ABI of the B200 (sm_100a) PEQA quantized-linear library.
 *
 * PEQA (arXiv 2305.14152) freezes a b-bit integer matrix Q and a zero-point z
 * and trains only the quantization scale s; the effective weight of a linear
 * layer is W_hat = s * (Q - z) (Eq. 2, Sec. 3.2).  This library is the layer's
 * hot path: quantize once (Eq. 1), forward, backward (dX and the scale
 * gradient dS, without ever materialising dW), small-batch decode, and AdamW
 * on the scales.
 *
 * Conventions for every entry point
 *   - All tensor pointers are DEVICE pointers owned by the caller, dense and
 *     row-major, 16-byte aligned, unless an argument says "host".  The library
 *     allocates no device memory.
 *   - N = out_features (rows of W, the paper's n), K = in_features (columns,
 *     the paper's m), T = tokens.  group_size g: 0 or K means one (s, z) per
 *     output row ("per-channel", Sec. 3.2); otherwise g is a multiple of 32
 *     that divides K and (s, z) are shared by runs of g input columns within
 *     a row (Sec. 4.2, "Group-wise Quantization").  G = K / g.
 *   - bits b is 3 or 4.
 *   - Packed layout of Q: each row is a little-endian bit string in which
 *     column j occupies bits [b*j, b*j+b), stored as uint32 words; a row has
 *     K*b/32 words (8 codes per word for b=4, 32 codes per 3 words for b=3).
 *   - Activations and their gradients are bf16; scales and dS are fp32;
 *     zero-points are uint8 integers in [0, 2^b-1].
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *     Calls validate their arguments on the host, enqueue work and return
 *     without synchronising (peqa_train_step_host and peqa_check_status
 *     synchronise, as documented).
 *   - Return value: PEQA_OK or a negative peqa_status code.  Nothing is
 *     enqueued when an argument check fails.
 *   - Kernels that wait on hardware barriers give every wait a bound; a wait
 *     that runs out records PEQA_ERR_DEVICE_TIMEOUT in a device status word
 *     that peqa_check_status() reads back.  Outputs are undefined after it.
 */
#ifndef PEQA_H_
#define PEQA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  PEQA_OK = 0,
  PEQA_ERR_NULL = -1,           /* a required pointer is NULL */
  PEQA_ERR_BAD_BITS = -2,       /* bits not in {3, 4} */
  PEQA_ERR_BAD_SHAPE = -3,      /* non-positive size, K % 32, bad group size, unsupported tile constraint */
  PEQA_ERR_ALIGNMENT = -4,      /* a pointer is not aligned as required */
  PEQA_ERR_WORKSPACE = -5,      /* workspace missing or smaller than peqa_workspace_bytes() */
  PEQA_ERR_ARCH = -6,           /* current device is not compute capability 10.x */
  PEQA_ERR_CUDA = -7,           /* a CUDA runtime/driver call failed; see peqa_last_cuda_error() */
  PEQA_ERR_DEVICE_TIMEOUT = -8, /* a bounded device-side wait expired */
  PEQA_ERR_TOO_LARGE = -9       /* size exceeds a documented fixed capacity */
} peqa_status;

/* Frozen part (Q, z) and trainable scale s of one PEQA linear layer. */
typedef struct {
  int32_t bits;            /* 3 or 4 */
  int32_t out_features;    /* N */
  int32_t in_features;     /* K, multiple of 32 */
  int32_t group_size;      /* 0 or K: per-channel; else multiple of 32 dividing K */
  const uint32_t* qweight; /* [N, K*bits/32] packed codes */
  const uint8_t* zeros;    /* [N, G] */
  const float* scales;     /* [N, G] */
} peqa_qweight_t;

typedef enum {
  PEQA_OP_FWD = 0,
  PEQA_OP_BWD = 1,
  PEQA_OP_DECODE = 2,
  PEQA_OP_BWD_DS_FROM_Y = 3,
  PEQA_OP_BWD_DSDZ = 4
} peqa_op;

/* Library version, major*10000 + minor*100 + patch. */
int peqa_version(void);

/* cudaError_t of the most recent failing CUDA call made by this library on
 * the calling thread (0 if none). */
int peqa_last_cuda_error(void);

/*
 * Asymmetric round-to-nearest quantization, Eq. 1 (Sec. 3.2), per (row, group):
 *   mn, mx = min/max of the group;  s = (mx - mn) / (2^b - 1)  (s = 1 if mx == mn)
 *   z = clamp(rint(-mn / s), 0, 2^b - 1);   Q = clamp(rint(W / s) + z, 0, 2^b - 1)
 * evaluated in IEEE binary32, round-half-to-even, true division, no FMA.
 *   W        in   fp32 [N, K]
 *   qweight  out  uint32 [N, K*bits/32]  packed Q
 *   zeros    out  uint8 [N, G]
 *   scales   out  fp32 [N, G]
 * W must be finite.  K % 32 == 0 and K <= 65536 (else PEQA_ERR_TOO_LARGE).
 */
int peqa_quantize_rtn(const float* W, int N, int K, int bits, int group_size,
                      uint32_t* qweight, uint8_t* zeros, float* scales, void* stream);

/*
 * Quantization with a searched clipping range.  Sec. 3.2 says s0 and z0 "are
 * initialized to minimize" the Frobenius error of Eq. 1 without giving a
 * procedure; this entry point reads it as a search over shrunken ranges.  Per
 * (row, group), candidate k = 0 .. n_candidates-1 scales the group's extremes by
 * p_k = 1 - k/64 and applies Eq. 1 in binary32 exactly as peqa_quantize_rtn does
 * (lo = p*mn, hi = p*mx, s = (hi-lo)/(2^b-1), z = clamp(rint(-lo/s)),
 * q = clamp(rint(w/s) + z)); its error is sum_j (w_j - s*(q_j - z))^2 with binary32
 * terms summed in binary64 in column order.  The first candidate with the smallest
 * error wins, so the result is never worse than peqa_quantize_rtn (candidate 0).
 *   W in fp32 [N, K];  qweight, zeros, scales out as in peqa_quantize_rtn;
 *   chosen  out  uint8 [N, G], the winning k (may be NULL).
 * 1 <= n_candidates <= 64.  An initialisation step (about n_candidates times the
 * work of peqa_quantize_rtn), not part of the training or serving loop.
 */
int peqa_quantize_search(const float* W, int N, int K, int bits, int group_size, int n_candidates,
                         uint32_t* qweight, uint8_t* zeros, float* scales, uint8_t* chosen,
                         void* stream);

/* Pack one code per byte (values in [0, 2^bits-1], upper bits ignored) into the
 * packed layout above, and the inverse.  codes is uint8 [N, K]; K % 32 == 0.
 * (The paper only states that the weights are a b-bit integer matrix, Sec. 3.3.) */
int peqa_pack(const uint8_t* codes, int N, int K, int bits, uint32_t* qweight, void* stream);
int peqa_unpack(const uint32_t* qweight, int N, int K, int bits, uint8_t* codes, void* stream);

/* Bytes of caller-provided scratch the given operation (peqa_op) needs for T
 * tokens (0 if none).  The workspace must be 256-byte aligned.  Its contents
 * are overwritten by each call; calls that may overlap need distinct workspaces. */
size_t peqa_workspace_bytes(int op, int T, const peqa_qweight_t* w);

/*
 * Forward of the PEQA layer, Y = X * W_hat^T with W_hat = s*(Q - z) (Eq. 2):
 *   Y[t,i] = sum_j X[t,j] * s[i,g(j)] * (Q[i,j] - z[i,g(j)])
 *   X  in   bf16 [T, K]
 *   Y  out  bf16 [T, N]  (fp32 accumulation, rounded to nearest even)
 * Requires K % 64 == 0, N % 8 == 0, T >= 1.  workspace may be NULL.
 */
int peqa_qlinear_fwd(const peqa_qweight_t* w, const void* X_bf16, int T, void* Y_bf16,
                     void* workspace, size_t workspace_bytes, void* stream);

/*
 * Backward of the PEQA layer (chain rule on Eq. 2; Q and z are frozen, s is
 * the only trainable tensor, Sec. 3.2):
 *   dX[t,j]  = sum_i dY[t,i] * s[i,g(j)] * (Q[i,j] - z[i,g(j)])
 *   dS[i,gi] = sum_{j in group gi} (Q[i,j] - z[i,gi]) * sum_t dY[t,i] * X[t,j]
 *   X   in   bf16 [T, K]  (only needed for dS)      dY  in  bf16 [T, N]
 *   dX  out  bf16 [T, K]      (may be NULL: skipped)
 *   dS  out  fp32 [N, G]      (may be NULL: skipped) OVERWRITTEN, not accumulated
 * dW = dY^T X exists only tile by tile in tensor memory and registers.
 * Requires K % 64 == 0, N % 8 == 0, T >= 1.  Needs a workspace of
 * peqa_workspace_bytes(PEQA_OP_BWD, T, w) bytes when that is non-zero.
 */
int peqa_qlinear_bwd(const peqa_qweight_t* w, const void* X_bf16, const void* dY_bf16, int T,
                     void* dX_bf16, float* dS, void* workspace, size_t workspace_bytes,
                     void* stream);

/*
 * Scale gradient followed at once by the AdamW step on the scales (chain rule
 * on Eq. 2, then App. A's optimizer): what peqa_qlinear_bwd (dS only) and
 * peqa_scale_adamw would do in two launches, done where each dS value becomes
 * final, so the scales, m and v are touched once and no second kernel runs.
 * Results are bit-identical to the two calls.
 *   X  in  bf16 [T, K]   dY  in  bf16 [T, N]   dS  out  fp32 [N, G]  OVERWRITTEN
 *   m, v  in/out  fp32 [N, G];  w->scales is updated in place (it must be writable)
 * Same shape rules and workspace as peqa_qlinear_bwd; step >= 1.
 */
int peqa_qlinear_bwd_ds_adamw(const peqa_qweight_t* w, const void* X_bf16, const void* dY_bf16,
                              int T, float* dS, float* m, float* v, float lr, float beta1,
                              float beta2, float eps, float weight_decay, int64_t step,
                              void* workspace, size_t workspace_bytes, void* stream);

/*
 * One training step of several PEQA linears in one call: for each linear, in the
 * order given, the forward of Eq. 2, then dX and dS by the chain rule on it and,
 * when apply_adamw is non-zero, App. A's AdamW step on its scales where dS becomes
 * final (the calls peqa_qlinear_fwd, peqa_qlinear_bwd (dX only) and
 * peqa_qlinear_bwd_ds_adamw would make, enqueued back to back with every
 * argument of every linear checked before the first launch).  A transformer
 * layer's quantized projections -- q, k, v, o, gate, up, down -- are such a list.
 * Each linear has its own activations X [T, K_i], upstream gradient dY [T, N_i]
 * and outputs Y [T, N_i], dX [T, K_i], dS [N_i, G_i] (overwritten); composing the
 * layer (attention, residuals, summing the dX of projections that share an
 * input) stays with the caller.  With apply_adamw == 0 the scales are left as
 * they are and m, v may be NULL: a data-parallel caller sums dS over its ranks
 * first and then calls peqa_scale_adamw.
 *   workspace: peqa_workspace_bytes(PEQA_OP_BWD, T, &w) bytes per linear, 256-byte
 *   aligned (may be NULL when that is 0); the linears may share one workspace,
 *   since their kernels run in stream order.
 * 1 <= n_linears <= PEQA_LAYER_MAX_LINEARS.  Shape rules and return codes as for
 * the single calls; nothing is enqueued when a check fails.
 */
#define PEQA_LAYER_MAX_LINEARS 16
typedef struct {
  peqa_qweight_t w;       /* w.scales must be writable when apply_adamw != 0 */
  const void* X_bf16;     /* [T, K] */
  const void* dY_bf16;    /* [T, N] */
  void* Y_bf16;           /* [T, N] out */
  void* dX_bf16;          /* [T, K] out */
  float* dS;              /* [N, G] out */
  float* m;               /* [N, G] in/out, AdamW first moment */
  float* v;               /* [N, G] in/out, AdamW second moment */
  void* workspace;
  size_t workspace_bytes;
} peqa_layer_linear_t;
int peqa_layer_train_step(const peqa_layer_linear_t* linears, int n_linears, int T, int apply_adamw,
                          float lr, float beta1, float beta2, float eps, float weight_decay,
                          int64_t step, void* stream);

/*
 * Scale gradient and zero-point gradient together (App. K trains z as well as
 * s).  By the chain rule on Eq. 2, with dW = dY^T X never leaving the chip,
 *   dS[i,gi] = sum_{j in group gi} (Q[i,j] - z[i,gi]) * dW[i,j]     (as peqa_qlinear_bwd)
 *   dZ[i,gi] = -s[i,gi] * sum_{j in group gi} dW[i,j]
 * Both come from the same dW tiles in one pass.  z itself stays the stored
 * integer: the gradient is what an optimizer of a real-valued copy would use.
 *   X  in  bf16 [T, K]   dY  in  bf16 [T, N]   dS, dZ  out  fp32 [N, G]  OVERWRITTEN
 * Requires K % 64 == 0, N % 8 == 0, T >= 1 and a workspace of
 * peqa_workspace_bytes(PEQA_OP_BWD_DSDZ, T, w) bytes when that is non-zero.
 */
int peqa_qlinear_bwd_dsdz(const peqa_qweight_t* w, const void* X_bf16, const void* dY_bf16, int T,
                          float* dS, float* dZ, void* workspace, size_t workspace_bytes,
                          void* stream);

/*
 * The layer with a real-valued zero-point.  App. K also trains the zero-points
 * ("zero-points only", "both zero-points and quantization scales"); z then leaves
 * the integer grid, and Eq. 2's weight is W_hat[i,j] = s[i,g] * (Q[i,j] - z[i,g])
 * with z a binary32 tensor zeros_f [N, G] that replaces w->zeros (which may be
 * NULL here).  Forward and dX fold s*(Q - z) into the bf16 operand, for every
 * group size, as (Q - zi)*s - (z - zi)*s with zi = clamp(rint(z), 0, 2^b-1), one
 * fused multiply-add on exact integers.  The gradients follow from the chain rule
 * on Eq. 2:
 *   dS[i,g] = sum_{j in g} (Q[i,j] - z[i,g]) * dW[i,j]
 *   dZ[i,g] = -s[i,g] * sum_{j in g} dW[i,j],          dW = dY^T X (never stored)
 * peqa_qlinear_bwd_zf: dX may be NULL (skipped); dS and dZ are both given or both
 * NULL; they need X and a workspace of peqa_workspace_bytes(PEQA_OP_BWD_DSDZ, T, w)
 * bytes when that is non-zero.  Shape rules as peqa_qlinear_fwd / _bwd.
 * One training step of a mode of App. K is then: peqa_qlinear_fwd_zf,
 * peqa_qlinear_bwd_zf, and peqa_scale_adamw on s and/or peqa_zero_adamw on z
 * (the same AdamW step, App. A, applied to the zero-points with dZ).
 */
int peqa_qlinear_fwd_zf(const peqa_qweight_t* w, const float* zeros_f, const void* X_bf16, int T,
                        void* Y_bf16, void* stream);
int peqa_qlinear_bwd_zf(const peqa_qweight_t* w, const float* zeros_f, const void* X_bf16,
                        const void* dY_bf16, int T, void* dX_bf16, float* dS, float* dZ,
                        void* workspace, size_t workspace_bytes, void* stream);
int peqa_zero_adamw(float* zeros_f, const float* dZ, float* m, float* v, int64_t numel, float lr,
                    float beta1, float beta2, float eps, float weight_decay, int64_t step,
                    void* stream);

/*
 * Scale gradient of a per-channel layer (group_size 0 or K, the paper's main
 * setting, Sec. 3.2) from the output the forward pass stored.  Eq. 2 with one
 * scale per channel reads Y[t,i] = s[i] * sum_j X[t,j] (Q[i,j] - z[i]), so
 *   dS[i] = ( sum_t dY[t,i] * Y[t,i] ) / s[i]
 * and the third contraction of the backward pass is not needed: the call reads
 * dY and Y once (4*T*N bytes).  Y must be the bf16 tensor peqa_qlinear_fwd wrote
 * for the same X and the same scales; its bf16 rounding carries into dS (about
 * 1e-3 relative).  A channel whose scale is 0 gets inf or NaN.
 *   dY, Y  in   bf16 [T, N]        dS  out  fp32 [N]  OVERWRITTEN
 * Requires one scale per channel (else PEQA_ERR_BAD_SHAPE), N % 8 == 0 and a
 * workspace of peqa_workspace_bytes(PEQA_OP_BWD_DS_FROM_Y, T, w) bytes.
 */
int peqa_qlinear_bwd_ds_from_y(const peqa_qweight_t* w, const void* dY_bf16, const void* Y_bf16,
                               int T, float* dS, void* workspace, size_t workspace_bytes,
                               void* stream);

/*
 * Small-batch forward for token generation (the memory-bound matrix-vector
 * regime of Sec. 3.1 / 3.3): same definition as peqa_qlinear_fwd with
 * T = M in [1, 16], implemented as a streaming fused dequant GEMV / skinny GEMM.
 * Requires K % 128 == 0 and N % 8 == 0.
 */
int peqa_qlinear_decode(const peqa_qweight_t* w, const void* X_bf16, int M, void* Y_bf16,
                        void* workspace, size_t workspace_bytes, void* stream);

/*
 * Small-batch forward for several tasks at once (Sec. 3.3: one frozen Q and z
 * serve every task, only the scales are task-specific, so a server switches
 * tasks by switching s).  Token m is multiplied by the scales of its own task:
 *   Y[m,i] = S[task_ids[m]][i] * sum_j X[m,j] * (Q[i,j] - z[i])
 *   scale_table  in  fp32 [n_tasks, N]   (w->scales is not read)
 *   task_ids     in  int32 [M], device memory; values are clamped to [0, n_tasks-1]
 *   X  in  bf16 [M, K]     Y  out  bf16 [M, N]     1 <= M <= 16
 * One scale per channel only (group_size 0 or K), K % 128 == 0, N % 8 == 0, and
 * M*K small enough for the streaming kernel (M*K <= 32768); otherwise
 * PEQA_ERR_BAD_SHAPE.
 */
int peqa_qlinear_decode_multitask(const peqa_qweight_t* w, const float* scale_table, int n_tasks,
                                  const int32_t* task_ids, const void* X_bf16, int M,
                                  void* Y_bf16, void* stream);

/*
 * One AdamW step on the scales, in place (App. A names AdamW; decoupled weight
 * decay, bias-corrected moments, step counted from 1):
 *   s <- s*(1 - lr*wd);  m <- b1*m + (1-b1)*dS;  v <- b2*v + (1-b2)*dS^2
 *   s <- s - lr * (m/(1-b1^step)) / (sqrt(v/(1-b2^step)) + eps)
 * scales, dS, m, v are fp32 [numel].
 */
int peqa_scale_adamw(float* scales, const float* dS, float* m, float* v, int64_t numel,
                     float lr, float beta1, float beta2, float eps, float weight_decay,
                     int64_t step, void* stream);

/*
 * One training step of a PEQA layer with HOST activations (composition of
 * Eq. 2's forward/backward with App. A's optimizer): copies h_X [T,K] and
 * h_dY [T,N] (host bf16, pinned or pageable) into the caller's device staging
 * buffers d_X, d_dY, runs forward, backward and AdamW on the stream, and
 * copies Y [T,N], dX [T,K] (host bf16) and dS [N,G] (host fp32) back.  Every
 * d_* pointer is device memory of the size of its host counterpart; d_m, d_v
 * are the optimizer state [N,G].  w->scales is updated in place (it must be
 * writable).  Synchronises the stream before returning.  The tokens travel in
 * chunks over two auxiliary streams of the library, so that the copies in, the
 * kernels and the copies out overlap (pinned host buffers are needed for that);
 * those streams (2) and events (35) are created on the first call on a device
 * and kept until the process ends, so make that first call outside any stream
 * capture.  They are shared by all calls on the device: concurrent calls from
 * several host threads are serialised by the library.  Every argument is checked
 * before anything is enqueued; if a CUDA call fails later, the streams are
 * drained before the error is returned.  h_* and d_* buffers must not be
 * touched by other work until the call returns.
 */
int peqa_train_step_host(const peqa_qweight_t* w, int T,
                         const void* h_X_bf16, const void* h_dY_bf16,
                         void* h_Y_bf16, void* h_dX_bf16, float* h_dS,
                         void* d_X, void* d_dY, void* d_Y, void* d_dX, float* d_dS,
                         float* d_m, float* d_v,
                         float lr, float beta1, float beta2, float eps, float weight_decay,
                         int64_t step, void* workspace, size_t workspace_bytes, void* stream);

/*
 * The same host-buffer step for several linears in one call (a layer's
 * projections, as for peqa_layer_train_step): for each linear, in the order
 * given, what peqa_train_step_host does, with the copies of the next linear
 * already on their way while the kernels of the current one run, and the copies
 * out of a linear overlapping the kernels of the next.  For that every linear
 * brings device staging buffers of its own: d_X, d_dY, d_Y, d_dX of different
 * linears must not overlap (PEQA_ERR_BAD_SHAPE otherwise); the workspace may be
 * shared.  The AdamW step (App. A) is applied to each linear's scales with the
 * same hyper-parameters and step.  Every argument of every linear is checked
 * before anything is enqueued; the stream is synchronised before returning; the
 * library's streams and events are those of peqa_train_step_host.
 */
typedef struct {
  peqa_qweight_t w;       /* w.scales is updated in place */
  const void* h_X;        /* host bf16 [T, K] in */
  const void* h_dY;       /* host bf16 [T, N] in */
  void* h_Y;              /* host bf16 [T, N] out */
  void* h_dX;             /* host bf16 [T, K] out */
  float* h_dS;            /* host fp32 [N, G] out */
  void* d_X;              /* device staging, sizes of the host counterparts */
  void* d_dY;
  void* d_Y;
  void* d_dX;
  float* d_dS;
  float* d_m;             /* device fp32 [N, G] in/out, AdamW moments */
  float* d_v;
  void* workspace;        /* peqa_workspace_bytes(PEQA_OP_BWD, T, &w) bytes, may be shared */
  size_t workspace_bytes;
} peqa_layer_host_linear_t;
int peqa_layer_train_step_host(const peqa_layer_host_linear_t* linears, int n_linears, int T,
                               float lr, float beta1, float beta2, float eps, float weight_decay,
                               int64_t step, void* stream);

/*
 * Scale gradient dS alone, for callers that cannot allocate device memory and
 * therefore cannot hand peqa_qlinear_bwd a workspace: code that runs where
 * cudaMalloc is off limits, or that is given nothing but its input and output
 * buffers.  (The paper has no counterpart to this call; it is the dS half of
 * peqa_qlinear_bwd with the scratch moved inside the library.)
 *   X in bf16 [T, K];  dY in bf16 [T, N];  dS out fp32 [N, G], overwritten.
 * The partial sums go to a fixed 8 MiB array that is part of the library's
 * device image (each GPU that loads the library holds it until the process
 * ends); peqa_bwd_ds_static_capacity_bytes() returns that size.  A layer
 * whose peqa_workspace_bytes(PEQA_OP_BWD, T, w) exceeds it is refused with
 * PEQA_ERR_TOO_LARGE and nothing is enqueued.  The first call on each device
 * looks the array's device address up (with that device current) and caches
 * it; that lookup and the first launch make the driver load the module that
 * carries the array, so make that first call outside any stream capture.
 * After it, a call allocates nothing of any kind.  All calls on a device share the one
 * array: it keeps whatever the previous call left, every value that is read
 * is rewritten first, and two calls whose kernels may overlap on the GPU
 * (different streams) race on it -- serialise them.  Same shape rules and
 * return codes as peqa_qlinear_bwd.
 */
int peqa_qlinear_bwd_ds_static(const peqa_qweight_t* w, const void* X_bf16, const void* dY_bf16,
                               int T, float* dS, void* stream);
size_t peqa_bwd_ds_static_capacity_bytes(void);

/*
 * Decode from a prepared copy of the frozen weights.  Q never changes after
 * quantization and is shared by every task (Sec. 3.3), so a server may keep it
 * in the order the small-batch kernel streams best.  The canonical packed
 * layout above stays the interchange format; the prepared buffer holds exactly
 * the same codes, rearranged (zero codes fill columns K .. 512*T - 1 and the row
 * group that completes an odd count of row groups):
 *   rg = row / 8, r = row % 8, step t = column / 512, T = ceil(K / 512), C = bits;
 *   block (rg, t) is C*512 bytes at byte offset (((rg/2)*T + t)*2 + rg%2)*C*512
 *   and consists of C chunks of 32 lanes of 16 bytes, chunk-major: word wo of
 *   chunk c of lane l is the lane's word wi = 4*c + wo;
 *   lane l = 4*r + c4 holds, of row 8*rg + r, columns 8*c4 .. 8*c4 + 7 of each of
 *   the step's sixteen 32-column runs; its 4*C words are four strings of C words
 *   (string s = words s*C .. s*C + C - 1 = runs 4s .. 4s + 3 of the step);
 *   a string is a little-endian bit string of 32 code positions (position p =
 *   bits [bits*p, bits*p + bits)); the code of string column
 *   cs = 8*(run % 4) + column % 8 is stored at position lo(cs/2) when cs is even
 *   and hi(cs/2) when cs is odd, where for bits = 4: lo(k) = 8*(k/4) + k%4,
 *   hi(k) = lo(k) + 4, and for bits = 3:
 *   lo = {1,0,3,2,4,9,12,11,15,14,18,21,24,23,26,25},
 *   hi = {5,6,7,8,10,13,16,17,19,20,22,27,28,29,30,31}.
 * peqa_decode_unprepare(peqa_decode_prepare(Q)) == Q bit for bit.
 * Requires K % 128 == 0 and N % 8 == 0; the prepared buffer has
 * peqa_decode_prepared_bytes(w) = 2*ceil(N/16) * T * bits * 512 bytes (N*K*bits/8
 * when K % 512 == 0 and N % 16 == 0; 0 for an unsupported shape) and must be
 * 16-byte aligned.  Only
 * bits, out_features, in_features and group_size of *w are read by
 * prepared_bytes and unprepare; prepare also reads w->qweight.
 */
size_t peqa_decode_prepared_bytes(const peqa_qweight_t* w);
int peqa_decode_prepare(const peqa_qweight_t* w, uint32_t* prepared, void* stream);
int peqa_decode_unprepare(const peqa_qweight_t* w, const uint32_t* prepared, uint32_t* qweight_out,
                          void* stream);

/*
 * Small-batch forward (Sec. 3.1 / 3.3) reading the prepared weights:
 *   Y[m,i] = sum_g s_m[i,g] * sum_{j in g} X[m,j] * (Q[i,j] - z[i,g]),   1 <= M <= 16
 * for one scale per channel (group_size 0 or K), groups of 64, 128 or 256
 * columns, and groups that are multiples of 512 columns (Sec. 4.2; other group
 * sizes: PEQA_ERR_BAD_SHAPE, use peqa_qlinear_decode).  s_m = w->scales, or,
 * when task_ids is not NULL, entry clamp(task_ids[m], 0, n_tasks-1) of
 * scale_table (fp32 [n_tasks, N, G]): token m is served with the scales of its
 * own task (Sec. 3.3).  w->qweight is not read.
 *   X  in  bf16 [M, K]    Y  out  bf16 [M, N]    task_ids  in  int32 [M] (device)
 * No workspace.  More than eight tokens are served by two launches of at most
 * eight tokens each.  The kernel is launched so that it may begin while earlier work
 * on `stream` is still draining: it starts to read `prepared` before that work
 * is known to be complete (X, the zero-points and the scales are read and Y is
 * written only after it has completed).  `prepared` must therefore be final when
 * the call is made -- synchronise once after peqa_decode_prepare.
 */
int peqa_qlinear_decode_prepared(const peqa_qweight_t* w, const uint32_t* prepared,
                                 const void* X_bf16, int M, void* Y_bf16,
                                 const float* scale_table, int n_tasks, const int32_t* task_ids,
                                 void* stream);

/*
 * Measurement aid (the paper has no counterpart): reads `bytes` bytes (a
 * multiple of 16, 16-byte aligned) with one CTA per SM, each CTA a contiguous
 * range, and does nothing else.  Its duration is the ceiling for any kernel that
 * must stream that many bytes from HBM under the same launch conditions; the
 * benchmark reports decode times next to it (Sec. 3.1: small-batch generation is
 * bound by the weight read).  sink: device scratch of at least 4 bytes per SM.
 */
int peqa_probe_read(const void* src, size_t bytes, uint32_t* sink, size_t sink_bytes, void* stream);

/*
 * Synchronises `stream`, then reads and clears the status word of that stream.
 * Returns PEQA_OK, PEQA_ERR_DEVICE_TIMEOUT (a bounded wait of a kernel launched on
 * `stream` expired since the last check; its outputs are undefined) or
 * PEQA_ERR_CUDA.  Status words live in the library's device image, one per stream
 * (the first 31 streams seen on a device get a word of their own, any further
 * streams share one); entry points without a workspace argument have nowhere
 * else to report to.  The table is initialised by the first call of any entry
 * point on a device with a blocking copy: make that call outside stream capture.
 */
int peqa_check_status(void* stream);

/*
 * Self-test of the bounded waits (the paper has no counterpart).  Sets, for
 * kernels launched afterwards on the current device, the bound of a single
 * device-side wait to wait_limit_us microseconds (0 restores the default of two
 * seconds) and, when starve_forward is non-zero, makes peqa_qlinear_fwd's
 * CTA-pair kernel announce one byte more than its copies deliver, so that its
 * first stage never fills: the kernel must then leave through its time-out path,
 * free its tensor memory and report PEQA_ERR_DEVICE_TIMEOUT through
 * peqa_check_status, leaving the context usable.  Synchronises the device and
 * clears all status words.  For tests only; never leave it set.
 */
int peqa_selftest_configure(int wait_limit_us, int starve_forward);

#ifdef __cplusplus
}
#endif
#endif /* PEQA_H_ */
