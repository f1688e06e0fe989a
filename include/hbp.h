/* hbp.h - C ABI of the Highway-backpropagation hot path (arXiv 2501.17086) on one GPU.
 *
 * Model (Section 3, Eq. 1-2): a stack of L residual steps
 *     x_{l+1} = a_l (.) x_l + f_l(x_l),      l = 0..L-1,
 * where f_l is the expensive block (Jacobian J, only ever multiplied by a
 * vector) and diag(a_l) is the cheap residual Jacobian K.  The loss is a sum of
 * per-state losses (Section 3); delta_l = dLoss_l/dx_l is an INPUT of the
 * backward calls, so any loss can be used.
 *
 * Highway-BP (Theorem 2, Section 4.3): g^0 = CumSumProd(delta, K) (Eq. 10); each
 * iteration computes u_l = J_l^T g_{l+1} for every l from the previous iterate
 * (Eq. 8) and then g_l = delta_l + a_l (.) g_{l+1} + u_l for l = L-1..0 (Eq. 9
 * and 11 folded into one recurrence, which is the same thing by linearity).
 * After k iterations g_l is the sum of all gradient paths through at most k
 * blocks; it is the exact gradient for l >= L-k, and everywhere once k >= L.
 * Parameter gradients use the final estimate (last sentence of Section 4.2).
 *
 * Shifted split (Appendix C.3, Eq. 17): with cfg.gamma > 0 (plain residual connections only, cfg.gate ==
 * HBP_GATE_ONE) a layer x + Block(x) is split as r(x, z) = (1 - gamma) x + z around g(x) = Block(x) + gamma x: the
 * forward pass and exact backpropagation are unchanged, while every Highway-BP iteration uses K = (1 - gamma) I and
 * adds gamma g_{l+1} (from the previous iterate) to each block VJP.  gamma = 1 is the fixed-point iteration of
 * Section 5.2.1.
 *
 * Conventions
 *  - Every pointer named below is a DEVICE pointer unless it says "host".
 *    All device buffers are allocated and owned by the caller and are only
 *    borrowed until the enqueued work has finished.  The library allocates no
 *    device memory and frees none.
 *  - All tensors are row-major with the channel dimension contiguous:
 *    states [L+1][N][d], weights [layer][out][in].  Element type is
 *    cfg.dtype (float or bf16); parameter gradients are always float.
 *  - Device pointers must be 16-byte aligned and d, hidden, in_dim must be
 *    multiples of 8 (bf16) or 4 (float): all access is 128-bit.
 *  - Calls enqueue work on `cuda_stream` (a cudaStream_t, may be NULL for the
 *    default stream) and return without synchronising, except
 *    hbp_sync_status.  They are not thread-safe per context.
 *  - Errors are returned as status codes.  Nothing aborts, throws or traps.
 */
#ifndef HBP_H_
#define HBP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct hbp_ctx hbp_ctx; /* opaque, host memory, made by hbp_create */

typedef enum {
  HBP_OK = 0,
  HBP_ERR_INVALID_ARG = 1, /* NULL where a pointer is required, k < 0, ...          */
  HBP_ERR_SHAPE = 2,       /* a size is <= 0 or violates the alignment rule        */
  HBP_ERR_DTYPE = 3,
  HBP_ERR_STATE = 4,       /* backward / exact before any forward                  */
  HBP_ERR_WORKSPACE = 5,   /* workspace too small or misaligned                    */
  HBP_ERR_UNSUPPORTED = 6,
  HBP_ERR_CUDA = 7,        /* a CUDA runtime call or launch failed                 */
  HBP_ERR_TIMEOUT = 8      /* a bounded device-side wait expired (status word)     */
} hbp_status;

/* Block kinds f_l (Table 1; Section 5.1.1 for the Transformer split; Section 5.2 for the RNN).
 *  MLP               f(x) = W2 gelu(W1 x)                     (exact erf GELU, no biases)
 *  PRELN_MLP         f(x) = W2 gelu(W1 LN(x))                 (LN without affine, biased variance)
 *  RNN_TANH          f_t(h) = tanh(W h + U x_t), weights shared over t; L is the sequence length
 *  PRELN_TRANSFORMER L decoder blocks = 2L residual steps: causal softmax MHA(LN(x)) Wo, then PRELN_MLP
 *  GRU               Table 1, row "GRU": h' = z (.) h + (1 - z) (.) n with r = sigmoid(U_r x_t + W_r h),
 *                    z = sigmoid(U_z x_t + W_z h), n = tanh(U_n x_t + r (.) W_n h), no biases, weights shared over
 *                    t.  The residual gate is the update gate z_t itself, K = diag(z_t): it depends on the state,
 *                    is produced by hbp_forward and kept in the workspace; cfg.gate must be HBP_GATE_ONE (there is
 *                    no further constant gate) and cfg.gamma 0.
 *  LSTM              Table 1, row "LSTM": the state is [c, h] (d = 2 * hidden wide); [i, f, g, o] = [sigmoid, sigmoid,
 *                    tanh, sigmoid](U x_t + W h), c' = f (.) c + i (.) g, h' = o (.) tanh(c'), no biases.  The residual
 *                    gate is [f_t, 0] (only the cell state has a linear path), produced by hbp_forward like the GRU's;
 *                    cfg.gate must be HBP_GATE_ONE, cfg.gamma 0, cfg.hidden = d / 2 = the number of units.
 *  RELU_MLP          Table 1, row "ResNet": x' = ReLU(x + W2 gelu(W1 x)).  The residual gate is the ReLU's 0/1 mask
 *                    [x + Block(x) > 0], produced by hbp_forward and kept in the workspace; the block Jacobian is
 *                    the mask times the MLP's.  cfg.gate must be HBP_GATE_ONE, cfg.gamma 0, cfg.dtype HBP_F32 (a mask
 *                    decided in bf16 arithmetic flips on elements near zero; HBP_ERR_UNSUPPORTED).
 *  POSTLN_MLP        Table 1, row "Transformer (Post-LN)" and Appendix C.3 with alpha = 1, beta = 0:
 *                    x' = LN(x + W2 gelu(W1 x)) = a(x) (.) x + b(x) with the row-wise gate a = 1 / sigma(x + Block(x)),
 *                    produced by hbp_forward; the block Jacobian is the rest of the layer's.  cfg.gate must be
 *                    HBP_GATE_ONE.  cfg.gamma > 0 uses the shifted split of Appendix C.3, K = (1 - gamma) diag(a)
 *                    (without a shift the truncated sums diverge on the directions LayerNorm removes). */
typedef enum {
  HBP_BLOCK_MLP = 0, HBP_BLOCK_PRELN_MLP = 1, HBP_BLOCK_RNN_TANH = 2, HBP_BLOCK_PRELN_TRANSFORMER = 3, HBP_BLOCK_GRU = 4,
  HBP_BLOCK_LSTM = 5, HBP_BLOCK_RELU_MLP = 6, HBP_BLOCK_POSTLN_MLP = 7
} hbp_block;
typedef enum { HBP_F32 = 0, HBP_BF16 = 1 } hbp_dtype;
/* Residual gate a_l, the diagonal of K (Eq. 2): all ones, one vector a[d] for every step, or a[steps][d]. */
typedef enum { HBP_GATE_ONE = 0, HBP_GATE_CHANNEL_SHARED = 1, HBP_GATE_CHANNEL_PER_STEP = 2 } hbp_gate;
/* Where the loss acts (Section 3): on the last state only (delta is [N][d]) or on every state
 * (delta is [steps+1][N][d]; delta[0] belongs to x_0 and is usually zero). */
typedef enum { HBP_LOSS_FINAL = 0, HBP_LOSS_EVERY_STEP = 1 } hbp_loss;

typedef struct {
  int32_t block;    /* hbp_block */
  int32_t dtype;    /* hbp_dtype */
  int32_t gate;     /* hbp_gate  */
  int32_t loss;     /* hbp_loss  */
  int32_t L;        /* residual steps (MLP kinds), time steps (RNN), decoder blocks (Transformer) */
  int32_t d;        /* state width */
  int32_t hidden;   /* MLP hidden width (MLP kinds, Transformer); LSTM: units */
  int32_t in_dim;   /* RNN / GRU / LSTM input width */
  int32_t n_heads;  /* Transformer: n_heads * head_dim == d */
  int32_t head_dim;
  int32_t seq;      /* Transformer: tokens == batch * seq */
  int32_t batch;    /* Transformer: sequences; RNN / GRU: rows (== tokens) */
  int64_t tokens;   /* N: rows of one state */
  float ln_eps;
  float gamma;      /* shift of the residual split, 0 <= gamma <= 1 (Appendix C.3, Eq. 17); 0 = the plain split */
} hbp_config;

/* Borrowed parameter pointers; those the block kind does not use are ignored.
 *  MLP kinds:    W1 [L][hidden][d], W2 [L][d][hidden]
 *  RNN:          W [d][d], U [d][in_dim]
 *  GRU:          W [3d][d], U [3d][in_dim]: the rows of the r, z and n parts stacked in that order
 *  LSTM:         W [4u][u], U [4u][in_dim], u = hidden: the rows of the i, f, g and o parts stacked in that order
 *  Transformer:  Wq, Wk, Wv, Wo [L][d][d], W1 [L][hidden][d], W2 [L][d][hidden]
 *  gate:         a [d] or [steps][d] when cfg.gate != HBP_GATE_ONE (steps = 2L for the Transformer) */
typedef struct {
  const void *W1, *W2;
  const void *W, *U;
  const void *Wq, *Wk, *Wv, *Wo;
  const void *a;
} hbp_params;

/* Caller-owned float outputs with the shapes of the parameters; OVERWRITTEN, not accumulated.
 * da has the shape of the gate and may be NULL to skip it. */
typedef struct {
  float *dW1, *dW2;
  float *dW, *dU;
  float *dWq, *dWk, *dWv, *dWo;
  float *da;
} hbp_grads;

/* Bytes of caller-provided device workspace a context for `cfg` needs (activation caches of the
 * last forward, per-iteration scratch, a status word).  HBP_ERR_SHAPE / _DTYPE / _UNSUPPORTED on a
 * bad config. */
hbp_status hbp_workspace_bytes(const hbp_config* cfg, size_t* bytes);

/* Makes a context over `workspace` (device, 256-byte aligned, >= hbp_workspace_bytes).  The
 * workspace is borrowed until hbp_destroy.  *out is host memory owned by the library. */
hbp_status hbp_create(const hbp_config* cfg, void* workspace, size_t workspace_bytes, hbp_ctx** out);

/* Section 3, h_i = f_i(h_{i-1}): runs the steps from x0 [N][d] and stores every state in
 * x_all [steps+1][N][d] (x_all[0] = x0) plus, in the workspace, what the block VJPs need.
 * `inputs` is the recurrent kinds' x [L][batch][in_dim] (NULL otherwise). */
hbp_status hbp_forward(hbp_ctx* ctx, const hbp_params* params, const void* x0, const void* inputs,
                       void* x_all, void* cuda_stream);

/* Theorem 2 / Eq. 8-11: k Highway-BP iterations from the caches of the last hbp_forward.
 * delta: see hbp_loss.  g_all [steps+1][N][d] receives g^k (g_all[steps] = delta_L always).
 * grads == NULL skips the parameter-gradient pass; otherwise it is computed from g^k (Section 4.2).
 * k >= steps returns the exact gradient (the loop stops there).  x_all and inputs must be the
 * buffers the last hbp_forward used. */
hbp_status hbp_backward(hbp_ctx* ctx, const hbp_params* params, int32_t k, const void* delta,
                        const void* x_all, const void* inputs, void* g_all, const hbp_grads* grads,
                        void* cuda_stream);

/* Section 2.2: sequential exact backpropagation, l = L-1..0, through the same block kernels. */
hbp_status hbp_exact(hbp_ctx* ctx, const hbp_params* params, const void* delta, const void* x_all,
                     const void* inputs, void* g_all, const hbp_grads* grads, void* cuda_stream);

/* The pieces of hbp_backward on their own, for callers that run the iterations themselves - in particular for
 * splitting the stack over several GPUs by layers (Section 6's layer-parallel setting: every GPU holds a contiguous
 * range of layers as its own context and the scan's carry crosses GPUs between the calls).
 *  hbp_iterate      one iteration in place (Eq. 8, then Eq. 9 and 11): u_l = J_l^T g_all[l+1] for every step from the
 *                   iterate as given (g_all[steps] included: the owner of the following layers supplies it), then
 *                   g_all[steps] = delta_L and g_all[l] = delta_l + a_l (.) g_all[l+1] + u_l.  g^0 followed by k calls
 *                   with the loss gradient as delta is hbp_backward(k).  A GPU that does not hold the last layer passes
 *                   zeros as delta: its scan then starts from a zero carry.
 *  hbp_add_carry    g_all[l] += carry [N][d] for l = 0..steps: applies the true carry to a scan that was started from
 *                   zero.  Only for gates that are all one (then every state depends on the carry with coefficient one);
 *                   HBP_ERR_UNSUPPORTED otherwise.
 *  hbp_param_grads  Section 4.2: the parameter gradients from the estimate in g_all. */
hbp_status hbp_iterate(hbp_ctx* ctx, const hbp_params* params, const void* delta, const void* x_all, const void* inputs,
                       void* g_all, void* cuda_stream);
hbp_status hbp_add_carry(hbp_ctx* ctx, const void* carry, void* g_all, void* cuda_stream);
hbp_status hbp_param_grads(hbp_ctx* ctx, const hbp_params* params, const void* x_all, const void* inputs,
                           const void* g_all, const hbp_grads* grads, void* cuda_stream);

/* Eq. 9 / Eq. 12 on its own: g[L] = delta_L and g[l] = delta_l + a_l (.) g[l+1] + u[l] for l = L-1..0,
 * i.e. the reverse CumSumProd with diagonal K.  u [L][rows][d] (NULL = zeros), delta as in hbp_loss
 * (`loss`), a as in hbp_gate (`gate`), g [L+1][rows][d].  `scratch` is device memory of at least
 * hbp_cumsumprod_scratch_bytes(...) bytes (may be NULL when that is 0).
 * hbp_cumsumprod_status is the same call with a device status word: `status` (device, one int, 4-byte aligned) is
 * where a kernel of the scan records HBP_ERR_TIMEOUT if one of its bounded waits gives up; the caller zeroes it
 * beforehand and reads it once the stream has finished.  hbp_cumsumprod (and hbp_cumsumprod_static) have no such
 * word: there a wait that gives up still ends the kernel, but goes unreported and leaves g partly unwritten. */
hbp_status hbp_cumsumprod_scratch_bytes(int32_t dtype, int32_t L, int64_t rows, int32_t d, size_t* bytes);
hbp_status hbp_cumsumprod(int32_t dtype, int32_t gate, int32_t loss, int32_t L, int64_t rows, int32_t d,
                          const void* u, const void* delta, const void* a, void* g,
                          void* scratch, size_t scratch_bytes, void* cuda_stream);
hbp_status hbp_cumsumprod_status(int32_t dtype, int32_t gate, int32_t loss, int32_t L, int64_t rows, int32_t d,
                                 const void* u, const void* delta, const void* a, void* g,
                                 void* scratch, size_t scratch_bytes, int32_t* status, void* cuda_stream);

/* The same scan for callers that cannot allocate device memory.  (The paper has no counterpart: this is a
 * packaging variant of hbp_cumsumprod, not a step of the method.)  Some hosts hand all device memory to
 * their own pool at start-up, or forbid cudaMalloc/cudaFree once they are running (latency-critical loops,
 * sandboxed plug-ins); they have no way to provide the scratch that the time-chunked scan needs.  Here the
 * scratch is a fixed array inside the library's device image of hbp_cumsumprod_static_max_bytes() bytes
 * (32 MiB), held by every GPU that loads the library until the process exits.  The call allocates nothing and
 * frees nothing.  Problems whose hbp_cumsumprod_scratch_bytes(...) exceeds the fixed size are refused with
 * HBP_ERR_WORKSPACE.  The first call on each device looks the array's device address up (a one-time set-up
 * with that device current): make that first call before starting any stream capture.  All calls share the
 * one array per device, so two calls whose kernels may overlap on the GPU (different streams) race on it;
 * serialise them.  Contents left by an earlier call are harmless: the scan writes every partial result
 * before reading it. */
size_t hbp_cumsumprod_static_max_bytes(void);
hbp_status hbp_cumsumprod_static(int32_t dtype, int32_t gate, int32_t loss, int32_t L, int64_t rows, int32_t d,
                                 const void* u, const void* delta, const void* a, void* g, void* cuda_stream);

/* Agreement of two gradient estimates, the quantities behind Figure 5 (cosine similarity of the k-iteration estimate
 * with the true gradient; norm of an iteration's step relative to the total): a and b hold `segments` consecutive
 * blocks of `elems` elements of `dtype` (states g_l, or float parameter gradients); out [segments][4] doubles (device)
 * receives <a,b>, |a|^2, |b|^2, |a-b|^2 per segment, summed in double in a fixed order.  scratch: device memory of
 * hbp_compare_scratch_bytes(segments) bytes, 8-byte aligned.  cos = out[0] / sqrt(out[1] out[2]); relative step =
 * sqrt(out[3] / out[2]). */
size_t hbp_compare_scratch_bytes(int32_t segments);
hbp_status hbp_compare(int32_t dtype, int32_t segments, int64_t elems, const void* a, const void* b, double* out,
                       void* scratch, size_t scratch_bytes, void* cuda_stream);

/* Copies the context's device status word to the host after synchronising the stream: HBP_OK, or the
 * error a kernel recorded (HBP_ERR_TIMEOUT when a bounded wait gave up).  An error is reported once: the word is
 * cleared after a non-zero read, and the context stays usable (a kernel whose wait gave up has released its
 * tensor memory and ended normally; its outputs are incomplete).  The only synchronising call. */
hbp_status hbp_sync_status(hbp_ctx* ctx, void* cuda_stream);

/* Diagnostic, not part of the method: exercises the failure path of the tensor-core kernels' bounded waits.
 * Enqueues one tile of the GEMM kernel whose copy role expects bytes that it never requests, with every wait limited
 * to limit_ns (1 us .. 1 s) instead of the usual 4 s: the wait runs out, the kernel records HBP_ERR_TIMEOUT in the
 * context's status word, all of its roles leave, the tensor memory is freed and the kernel ends.  The next
 * hbp_sync_status returns HBP_ERR_TIMEOUT.  scratch: device memory, 256-byte aligned, >= 128 KiB (contents
 * irrelevant, may be overwritten).  Nothing waits without a limit at any point. */
hbp_status hbp_selftest_wait_timeout(hbp_ctx* ctx, void* scratch, size_t scratch_bytes, uint64_t limit_ns,
                                     void* cuda_stream);

/* Device time per phase of the path, for the backward / exact calls made while profiling is on.  CUDA
 * events are recorded on the call's stream around each phase: the reverse scans (Eq. 9-11), the block VJPs
 * (Eq. 8), the parameter-gradient pass (Section 4.2) and everything else.  hbp_profile_enable(ctx, 1)
 * clears the totals; hbp_profile_read waits for the recorded events, adds them up into ms[HBP_PHASE_COUNT]
 * and launches[HBP_PHASE_COUNT] (either may be NULL) and clears the record. */
typedef enum { HBP_PHASE_SCAN = 0, HBP_PHASE_VJP = 1, HBP_PHASE_WGRAD = 2, HBP_PHASE_OTHER = 3, HBP_PHASE_COUNT = 4 } hbp_phase;
hbp_status hbp_profile_enable(hbp_ctx* ctx, int32_t on);
hbp_status hbp_profile_read(hbp_ctx* ctx, float* ms, int64_t* launches);

/* Number of kernels this context has launched since creation (host counter). */
int64_t hbp_launch_count(const hbp_ctx* ctx);

/* Kernel-selection modes of a context, fixed when it was created from the environment of that moment:
 * bit 0 = HBP_FORCE_SIMT=1 (every contraction on the CUDA-core kernels, a cross-check of the tensor-core ones),
 * bit 1 = the tensor-core GEMM pairs CTAs (tcgen05 cta_group::2, 256 x 256 tiles): the default; HBP_GEMM_PAIR=0
 * keeps single CTAs (128 x 256 tiles),
 * bit 2 = on the float tanh RNN the reverse scan between two all-step VJPs (Eq. 9 followed by Eq. 8) also writes
 * the next VJP's left operand g_{t+1} * tanh'(z_t), split for the tensor cores, instead of the intermediate
 * iterate: the default; HBP_SCAN_OPERAND=0 keeps the separate pass (same bits in every result, a cross-check).
 * The modes belong to the context: contexts created
 * under other settings, before or after, keep their own.  One-time kernel set-up is likewise remembered per
 * device, so one process may hold contexts on several GPUs (each used with its device current). */
int32_t hbp_context_modes(const hbp_ctx* ctx);

const char* hbp_status_string(hbp_status s);
void hbp_destroy(hbp_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* HBP_H_ */
