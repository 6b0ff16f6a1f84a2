/*
 * qalora.h -- C ABI of the QA-LoRA linear layer for NVIDIA B200 (sm_100a).
 *
 * The layer (arXiv 2309.14717, "QA-LoRA"): a weight matrix W [D_in x D_out]
 * quantized group-wise with min-max quantization (Eq. 1 applied per group of
 * `group_size` consecutive input channels and per output column, Section 3.3),
 * plus a low-rank adapter that sees the input summed over each group
 * (Algorithm 1; Appendix B Eq. 3 and Eq. 4):
 *
 *     y = x * W~  +  s * (pool(x) * A) * B
 *     W~[k, n]   = alpha[k / g, n] * c[k, n] + beta[k / g, n]
 *     pool(x)[m, q] = sum of x[m, k] over the g channels k of group q
 *
 * Notation used below: K = d_in, N = d_out, g = group_size, G = K / g (the
 * paper's symbol L is this NUMBER of groups), r = rank (the paper's D_int),
 * b = bits, s = scale, M = number of token rows.
 *
 * Conventions that hold for every entry point
 *   - Every data pointer is DEVICE memory owned by the caller unless the
 *     comment says "host".  The library allocates no device memory.
 *   - All matrices are dense row-major.  x, y, dy, dx, A, B are bfloat16
 *     (passed as void*); alpha/beta (qparams), dA, dB and W are float32.
 *   - Pointers must be 16-byte aligned.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL
 *     is the legacy default stream); calls do not synchronize the host.
 *   - Outputs are overwritten, never accumulated into.
 *   - Return value: QALORA_OK or a negative qalora_status.  Nothing is
 *     launched when an argument is rejected.  No call traps or aborts.
 *
 * Packed code layout (version QALORA_LAYOUT_VERSION; the paper only says the
 * codes are stored as b-bit integers, Section 3.1 -- the arrangement is this
 * library's own).  A pack unit is 32 consecutive input channels (k-block
 * kb = k / 32) of one output column n; j = k % 32.  `codes` is a little-endian
 * uint32 array [K/32][N][words]:
 *   b = 4: 4 words; position j lives in word j/8,  e = j%8,  at bit 16*(e&1) + 4*(e>>1)
 *   b = 2: 2 words; position j lives in word j/16, e = j%16, at bit 16*(e&1) + 2*(e>>1)
 *   b = 3: 3 words; words 0..1 hold (c & 3) in the b = 2 arrangement, word 2
 *          holds (c >> 2) of position j at bit 16*(j&1) + (j>>1)
 * `qparams` is float32 [G][N][2] = {alpha, beta} per (group, column).
 */
#ifndef QALORA_H_
#define QALORA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define QALORA_LAYOUT_VERSION 1

/* Most token rows a call takes (2^22): beyond it QALORA_ERR_INVALID_ARG. */
#define QALORA_MAX_ROWS 4194304

typedef enum qalora_status {
  QALORA_OK = 0,
  QALORA_ERR_INVALID_ARG = -1,      /* a size or enum outside its domain        */
  QALORA_ERR_NULL_POINTER = -2,     /* a required pointer is NULL               */
  QALORA_ERR_UNSUPPORTED_SHAPE = -3,/* see qalora_desc                          */
  QALORA_ERR_MISALIGNED = -4,       /* a pointer is not 16-byte aligned         */
  QALORA_ERR_WORKSPACE_TOO_SMALL = -5,
  QALORA_ERR_CUDA = -6,             /* a CUDA call or launch failed             */
  QALORA_ERR_STATIC_SCRATCH_EXCEEDED = -7 /* qalora_forward_static: the call needs more
                                       than QALORA_STATIC_SCRATCH_BYTES of scratch */
} qalora_status;

/* Shape and hyper-parameters of one layer.  Supported: d_in a multiple of
 * group_size; group_size a multiple of 32; d_out a multiple of 8; bits in
 * {2, 3, 4}; 0 <= rank <= 256 and a multiple of 8.  rank == 0 is the plain
 * (merged, deployed) quantized layer: A and B are then ignored and may be NULL. */
typedef struct qalora_desc {
  int32_t d_in;        /* K */
  int32_t d_out;       /* N */
  int32_t group_size;  /* g */
  int32_t bits;        /* b */
  int32_t rank;        /* r */
  float   scale;       /* s */
} qalora_desc;

/* QALORA_OP_TRAIN: one workspace shared by qalora_forward_train and qalora_backward_train. */
typedef enum qalora_op { QALORA_OP_FORWARD = 0, QALORA_OP_BACKWARD = 1, QALORA_OP_TRAIN = 2 } qalora_op;

/* Library version * 100 + QALORA_LAYOUT_VERSION. */
int qalora_version(void);

/* Static, NUL-terminated description of a status code (host memory, never freed). */
const char* qalora_status_string(int status);

/* Sizes in bytes of the packed `codes` array and of `qparams` for a layer.
 * Both outputs are host pointers. */
int qalora_packed_bytes(const qalora_desc* desc, size_t* code_bytes, size_t* qparam_bytes);

/* Bytes of scratch `workspace` that qalora_forward / qalora_backward need for
 * `m` token rows (host pointer out; may be 0).  The workspace holds the pooled
 * input, the rank-r intermediates and split-K partial sums; its content is
 * undefined on entry.  On exit its first int32 is a device status word: 0, or
 * 1 when a bounded wait inside a tensor-core kernel expired (the outputs of
 * that call are then invalid; nothing hangs or traps).  The size is for exactly
 * `m` rows and does not grow monotonically with m: a smaller batch may take a
 * kernel that cuts its reduction into more parts and keeps larger partial sums,
 * so a workspace that serves several batch sizes takes the largest of their sizes. */
int qalora_workspace_bytes(const qalora_desc* desc, int64_t m, int op, size_t* bytes);

/* Group-wise min-max quantization, Eq. 1 per (group, column) (Section 3.3):
 *   lo, hi = min, max of W[q*g .. (q+1)*g - 1, n];  beta = lo;
 *   alpha = (hi - lo) / (2^b - 1), or 1 when hi == lo;
 *   c = clamp(round_half_even((W - beta) / alpha), 0, 2^b - 1)
 * evaluated in IEEE float32, one correctly rounded operation at a time.
 *   W        in : float32 [K][N]
 *   codes    out: packed codes, qalora_packed_bytes() bytes
 *   qparams  out: float32 [G][N][2]
 *   dev_status out, optional: one int32 in device memory; bit 0 is OR-ed in
 *            when a non-finite weight is met (the codes of that group are then
 *            unspecified).  The caller zeroes it.  May be NULL. */
int qalora_quantize(const qalora_desc* desc, const float* W, void* codes, float* qparams,
                    int32_t* dev_status, void* cuda_stream);

/* Forward pass, Algorithm 1 / Appendix B Eq. 4:
 *   y = x * W~ + s * (pool(x) * A) * B.
 *   x bf16 [m][K];  A bf16 [G][r];  B bf16 [r][N];  y out bf16 [m][N].
 * Products are bf16 x bf16 accumulated in float32.  Any m with 0 <= m <= QALORA_MAX_ROWS
 * is accepted by every call that takes a row count, more is QALORA_ERR_INVALID_ARG
 * (element and byte offsets are 64-bit: tensors of more than 2^31 elements are fine, a
 * test runs 200 000 rows of an 11008-wide layer; tile counts are 32-bit); the
 * kernel is chosen from m (a bandwidth-bound path for a few rows, a
 * tensor-core path otherwise).  The few-token kernel of a layer without adapter may
 * start while the kernel before it in the stream is still running (programmatic dependent
 * launch): it then reads only codes and qparams early and waits for that kernel's
 * completion before it reads x or writes y.  Codes and qparams must therefore not be
 * outputs of a kernel that itself lets its successors start early; no kernel of this
 * library that writes them (quantize, merge, the format conversions) does. */
int qalora_forward(const qalora_desc* desc, int64_t m, const void* x, const void* codes,
                   const float* qparams, const void* A, const void* B, void* y,
                   void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The forward pass of SEVERAL layers in one call, for serving a merged model a few tokens at
 * a time (Section 3.2 states efficient deployment as the method's second goal; Section 4.2:
 * the merged model stays quantized and is therefore faster at inference).  The layers are
 * independent: each has its own input x, e.g. the q, k and v projections or the gate and up
 * projections of a transformer block (which read the same x), or any layers whose inputs are
 * ready.  Layer l computes what qalora_forward computes,
 *     y_l = x_l * W~_l  (+ s_l * (pool(x_l) * A_l) * B_l  when its rank is not 0),
 * on the same number m of token rows.  When every layer is a plain quantized layer (rank 0),
 * m <= 16, there are at most 8 layers, all with the same bit width, all with group size 32 or
 * all with group size 64/128, and every shape has d_out and d_in multiples of 128, the whole
 * group runs as ONE kernel launch (launch, cluster set-up and first-byte latency are paid once,
 * and the layers' blocks fill the GPU together); otherwise the layers run one after the other
 * exactly as qalora_forward would run them.  Results do not depend on which way was taken
 * beyond the summation order of the reduction slices.
 *   layers   : HOST array of n descriptors with DEVICE pointers (A, B ignored when rank == 0)
 *   workspace: DEVICE scratch of qalora_forward_group_workspace_bytes() bytes; its first int32
 *              is the status word described at qalora_workspace_bytes, for the whole group
 * Errors are those of qalora_forward; every layer is checked before anything is launched. */
typedef struct qalora_group_layer {
  qalora_desc desc;
  const void* x;          /* bf16 [m][d_in]  */
  const void* codes;
  const float* qparams;
  const void* A;          /* bf16 [G][r], or NULL when rank == 0 */
  const void* B;          /* bf16 [r][d_out], or NULL when rank == 0 */
  void* y;                /* bf16 [m][d_out], out */
} qalora_group_layer;
int qalora_forward_group_workspace_bytes(const qalora_group_layer* layers, int n, int64_t m, size_t* bytes);
int qalora_forward_group(const qalora_group_layer* layers, int n, int64_t m,
                         void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Backward pass with the base weights frozen (Section 3.1: only A and B are
 * adjusted).  With l the loss and dy = dl/dy:
 *   dT = s * dy * B^T;   dx = dy * W~^T + repeat_g(dT * A^T);
 *   dA = pool(x)^T * dT; dB = s * (pool(x) * A)^T * dy.
 *   x bf16 [m][K]; dy bf16 [m][N];
 *   dx out bf16 [m][K]; dA out float32 [G][r]; dB out float32 [r][N].
 * rank must be > 0.  dx, dA or dB may be NULL to skip that output.
 * With more than 16 rows the dB product runs beside dT and dA on a stream of the library's
 * own (made on first use by the calling host thread, one per device, never destroyed), forked
 * from `cuda_stream` and joined to it by events inside the call: to the caller the call is
 * ordered in `cuda_stream` like any other, also inside a stream capture. */
int qalora_backward(const qalora_desc* desc, int64_t m, const void* x, const void* dy,
                    const void* codes, const float* qparams, const void* A, const void* B,
                    void* dx, float* dA, float* dB,
                    void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The same two passes for a fine-tuning step, sharing one workspace of
 * qalora_workspace_bytes(desc, m, QALORA_OP_TRAIN) bytes (Algorithm 1's forward and its
 * gradients; Section 3.1).  The pooled input pool(x) and T = s * pool(x) * A are needed by
 * both passes: qalora_forward_train computes them once and leaves them in the workspace,
 * qalora_backward_train takes them from there instead of streaming x a second time.  The
 * caller must pass the SAME workspace, desc, m, x and A to both and must not write to the
 * workspace in between.  Results are identical to qalora_forward / qalora_backward.  The
 * status word is cleared by qalora_forward_train only, so that after the pair it tells
 * whether either pass gave up a wait.  rank must be > 0. */
int qalora_forward_train(const qalora_desc* desc, int64_t m, const void* x, const void* codes,
                         const float* qparams, const void* A, const void* B, void* y,
                         void* workspace, size_t workspace_bytes, void* cuda_stream);
int qalora_backward_train(const qalora_desc* desc, int64_t m, const void* x, const void* dy,
                          const void* codes, const float* qparams, const void* A, const void* B,
                          void* dx, float* dA, float* dB,
                          void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Merge for deployment (Algorithm 1, merge_with_quantization; Appendix B
 * Eq. 7): folds s*A*B into the zero factors, after which the plain quantized
 * layer (rank 0) reproduces the adapted one.  For the additive zero of Eq. 1:
 *   beta'[q, n] = beta[q, n] + s * sum_i A[q, i] * B[i, n]   (alpha unchanged)
 * which is the paper's zero-point update z' = z - s*A*B/alpha under
 * z = -beta/alpha.  qparams_out may alias qparams_in. */
int qalora_merge(const qalora_desc* desc, const float* qparams_in, const void* A, const void* B,
                 float* qparams_out, void* cuda_stream);

/* One fine-tuning step of the layer driven from HOST buffers: copies x and dy to
 * the device, runs qalora_forward and qalora_backward (Algorithm 1 and its
 * gradients, as above), and copies y, dx, dA and dB back.  The call returns
 * without synchronizing; everything it enqueues starts after the work already on
 * `cuda_stream`, and `cuda_stream` ends after the last copy, so the host outputs
 * are valid once that stream has been synchronized.  Batches of 2048 rows and
 * more are cut into up to 8 row chunks (multiples of 256 rows, at least 1024):
 * the copies run on two streams of the library's own (made on first use, one
 * pair per device), so that a chunk's inputs arrive while the previous chunk
 * computes and the one before that returns.  Rows are independent in y and dx:
 * the full chunks' rows are the same bits as from one qalora_forward /
 * qalora_backward over all rows; a shorter last chunk may take another kernel
 * (another summation order: its rows agree to within one bf16 step).  dA and dB
 * are then the sums of the chunks' results in chunk order (a different, fixed,
 * summation order).
 * Calls from several host threads are serialized by the library.
 *   x_host, dy_host   in : HOST memory (pinned for asynchronous copies), bf16 [m][K], [m][N]
 *   codes, qparams, A, B : DEVICE memory, as for qalora_forward
 *   y_host, dx_host   out: HOST bf16 [m][N], [m][K];  dA_host, dB_host out: HOST float32
 *   staging              : DEVICE scratch of qalora_step_host_bytes() bytes (device copies
 *                          of the inputs and outputs plus the workspaces); its first
 *                          int32 is the status word described at qalora_workspace_bytes
 * rank must be > 0. */
int qalora_step_host_bytes(const qalora_desc* desc, int64_t m, size_t* bytes);
int qalora_step_host(const qalora_desc* desc, int64_t m, const void* x_host, const void* dy_host,
                     const void* codes, const float* qparams, const void* A, const void* B,
                     void* y_host, void* dx_host, float* dA_host, float* dB_host,
                     void* staging, size_t staging_bytes, void* cuda_stream);

/* Dequantizes the whole weight matrix, W~[k][n] = alpha[k/g][n] * c[k][n] + beta[k/g][n]
 * (Eq. 1), e.g. to export a merged layer or to feed a 16-bit baseline.
 *   codes, qparams in : DEVICE, as written by qalora_quantize / qalora_merge
 *   W              out: DEVICE [d_in][d_out] row-major, float32 (out_bf16 == 0) or bf16
 *                       (out_bf16 != 0; the float32 value rounded to nearest even)
 * Pointers 16-byte aligned.  One launch on `cuda_stream`, no synchronization. */
int qalora_dequantize(const qalora_desc* desc, const void* codes, const float* qparams, void* W,
                      int out_bf16, void* cuda_stream);

/* The zero-point form of Algorithm 1 (pre_quantization / merge_with_quantization):
 * W~ = alpha * (c - z), against Eq. 1's W~ = alpha * c + beta; the two describe the same
 * weights when beta = -alpha * z.  qalora_qparams_from_zero_point imports scales and zero
 * points (integer ones of an asymmetric integer quantizer, stored as float32, or the real
 * ones Algorithm 1's merge leaves) into the library's qparams; qalora_qparams_to_zero_point
 * exports them, z = -beta / alpha (alpha is never 0 in qparams written by this library).
 *   alpha, zero : DEVICE float32 [G][d_out];  qparams : DEVICE float32 [G][d_out][2]
 * Pointers 16-byte aligned.  One launch each on `cuda_stream`, no synchronization. */
int qalora_qparams_from_zero_point(const qalora_desc* desc, const float* alpha, const float* zero,
                                   float* qparams, void* cuda_stream);
int qalora_qparams_to_zero_point(const qalora_desc* desc, const float* qparams, float* alpha,
                                 float* zero, void* cuda_stream);

/* Adapter update of one fine-tuning step (Section 4.1, training details: AdamW with a
 * maximum gradient norm of 0.3 and a constant learning rate; only A and B are trained,
 * Section 3.3).  All trained values of the step lie in ONE flat array of n float32
 * (the caller lays the layers' A and B out in it, e.g. as the all-reduce bucket of a
 * data-parallel step), so the gradient norm is the joint norm over all of them:
 *     norm = ||grad||_2,  coef = max_grad_norm > 0 ? min(1, max_grad_norm / (norm + 1e-6)) : 1
 *     g = coef * grad;  param *= 1 - lr * weight_decay
 *     m = beta1 * m + (1 - beta1) * g;  v = beta2 * v + (1 - beta2) * g * g
 *     param -= lr * (m / (1 - beta1^step)) / (sqrt(v / (1 - beta2^step)) + eps)
 *     param_bf16 = bf16(param)           (round to nearest even; what qalora_forward reads)
 * The paper does not state beta1, beta2, eps or weight_decay; they are the caller's.
 *   hyper        in : HOST struct; step counts from 1
 *   grad         in : DEVICE float32 [n]
 *   param, exp_avg, exp_avg_sq  in/out: DEVICE float32 [n] (master copy and both moments)
 *   param_bf16   out: DEVICE bf16 [n]
 *   norm_out     out: DEVICE float32 [2] = {norm, coef}, or NULL
 *   workspace       : DEVICE scratch of qalora_adamw_workspace_bytes() bytes, caller-owned
 * All device pointers 16-byte aligned.  Two launches on `cuda_stream`, no synchronization,
 * no allocation; results are reproducible bit for bit for a given n and device.
 * Errors: QALORA_ERR_NULL_POINTER, QALORA_ERR_MISALIGNED, QALORA_ERR_INVALID_ARG (n < 0,
 * step < 1, a beta outside [0, 1), lr, eps or weight_decay negative or not finite),
 * QALORA_ERR_WORKSPACE_TOO_SMALL, QALORA_ERR_CUDA. */
typedef struct qalora_adamw_hyper {
  float lr, beta1, beta2, eps, weight_decay, max_grad_norm;
  int64_t step;
} qalora_adamw_hyper;
int qalora_adamw_workspace_bytes(size_t* bytes);
int qalora_adamw_step(const qalora_adamw_hyper* hyper, int64_t n, const float* grad, float* param,
                      float* exp_avg, float* exp_avg_sq, void* param_bf16, float* norm_out,
                      void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Forward pass for callers that cannot allocate device memory (the paper has no
 * counterpart; this is a convenience of the library).  Some hosts of this code
 * may not call cudaMalloc at all: a plugin running inside an engine that owns
 * the whole device heap, code on a real-time or already-capturing path where an
 * allocation would stall or is forbidden, or a process started with its memory
 * budget fully handed out.  qalora_forward asks such a caller for a workspace it
 * has no way to provide.  This variant computes exactly what qalora_forward
 * computes (same arguments, same kernels, same results) but takes its scratch
 * from a fixed array of QALORA_STATIC_SCRATCH_BYTES that is part of the
 * library's device image.  It calls no cudaMalloc/cudaFree and no allocating
 * routine.
 *   - Limit: qalora_workspace_bytes(desc, m, QALORA_OP_FORWARD) must not exceed
 *     QALORA_STATIC_SCRATCH_BYTES.  That is about m * rank * 6 bytes + 1 KiB where the
 *     few-token kernel runs (m <= 16; m <= 32 on layers whose grid fills the GPU evenly)
 *     and for m > 512, e.g. 2048 tokens at rank 64.  For 17 <= m <= 512 on the tensor-core
 *     path the forward pass also keeps float32 partial results of its reduction, several
 *     times m * d_out * 4 bytes, which is beyond 1 MiB on LLaMA-sized layers (d_out = 4096:
 *     m = 64 needs 4 MiB).  Larger requests return QALORA_ERR_STATIC_SCRATCH_EXCEEDED;
 *     a call that is rejected, for this or any reason qalora_forward would reject it for,
 *     launches nothing and does not touch the CUDA runtime.
 *   - Cost: every GPU on which the library's device code is loaded holds the
 *     array until the process exits, whether or not this function is used.
 *   - The first call on each device looks up the array's device address (with
 *     that device current).  Make that first call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps the previous
 *     call's contents; the function clears the part that must start at zero.
 *     Two calls whose GPU work overlaps (different streams, or different
 *     threads without ordering) race on it: serialize them. */
#define QALORA_STATIC_SCRATCH_BYTES (1 << 20)
int qalora_forward_static(const qalora_desc* desc, int64_t m, const void* x, const void* codes,
                          const float* qparams, const void* A, const void* B, void* y,
                          void* cuda_stream);

/* ---- Instrumentation (no counterpart in the paper) ------------------------ */

/* Number of CUDA kernels this library has launched in this process so far
 * (all threads; monotonically increasing). */
uint64_t qalora_kernel_launches(void);

/* Arms a one-shot probe on the calling thread: the next main contraction kernel
 * (the x * W~ product of qalora_forward or the dy * W~^T product of
 * qalora_backward) launched from this thread records `start_event` just before
 * and `stop_event` just after that one launch, on the launch stream.  Both are
 * cudaEvent_t handles created with timing enabled, passed as void*; NULL
 * disarms.  Host pointers are not retained after the launch. */
int qalora_profile_next_main_kernel(void* start_event, void* stop_event);

/* Name of the main contraction kernel chosen by the most recent qalora_forward
 * or qalora_backward call on this thread ("" before any call).  Static host
 * string. */
const char* qalora_main_kernel_name(void);

/* Bounds-check build.  The same sources compiled with -DQALORA_DEBUG (libqalora_debug.so)
 * test every index, offset, tensor-memory column and copy coordinate a kernel computes
 * against its limit before the access, skip an access that would fall outside, and put a
 * 256-byte guard behind every region of a workspace (qalora_workspace_bytes and the other
 * size queries grow accordingly), written before a pass and verified after it.  Nothing
 * faults: failures are recorded.  qalora_debug_checks() returns 1 in that build and 0 in the
 * ordinary one.  qalora_debug_report() waits for the current device's work, copies the
 * record to `words8` (HOST array of 8 int32) and clears it:
 *   [0] flags: 2 = an index check failed, 4 = a guard word was overwritten;
 *   [1] first failed check, source file ordinal * 100000 + line;  [2], [3] its index (low,
 *   high word);  [4], [5] its limit;  [6] failed checks in all;  [7] first overwritten guard,
 *   region ordinal * 65536 + word + 1.
 * In the ordinary build it writes zeros.  Both are host functions; the report is the one
 * call of this library that synchronizes the device, and the bounds-check build the one
 * that allocates device memory (the 32-byte record, once per device). */
int qalora_debug_checks(void);
int qalora_debug_report(int32_t* words8);

#ifdef __cplusplus
}
#endif
#endif /* QALORA_H_ */
