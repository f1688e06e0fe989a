// Internal declarations shared by the CUDA translation units of libhbp.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "hbp.h"

namespace hbp {

typedef __nv_bfloat16 bf16;

// ---------------------------------------------------------------- GEMM description
// D(m, n) = sum_k A(m, k) * B(n, k) per batch entry, fp32 accumulation, followed by an epilogue.
// A(m, k) lives at A + batch*a_sb + m*a_sm + k*a_sk (element strides), B(n, k) likewise.
enum Epilogue {
  EPI_STORE = 0,     // D = acc
  EPI_GELU_FWD = 1,  // D = gelu(acc), D2 = gelu'(acc): the two activation caches of the MLP block
  EPI_RESID = 2,     // v = gate[n] * r + acc with r = R ? R[m,n] : E[m,n];  R = v (if R);  D = v
  EPI_MUL = 3,       // D = acc * E[m,n]   (dZ = dA * gelu'(Z) with the cached derivative)
  EPI_AFFINE = 4,    // D = (E ? E[m,n] : 0) + gate[n] * E2[m,n] + acc
  EPI_STORE_LN = 6,  // D = acc, plus per-row partial sums (sum acc, sum acc * E[m,n]) per 64 columns -> stats
  EPI_ADD = 7,       // D = acc + E[m,n]   (u_t + delta_t: the scan then reads one tensor less)
  EPI_RNN_FWD = 5,   // c = tanh(acc + E[m,n]);  D2 = 1 - c^2;  D = gate[n] * E2[m,n] + c
};

struct GemmArgs {
  int M = 0, N = 0, K = 0, batch = 1;
  int in_dtype = HBP_F32;  // element type of A, A2, B, D2, E, E2, gate and of D unless d_f32
  const void* A = nullptr;
  int64_t a_sm = 0, a_sk = 0, a_sb = 0;
  const void* A2 = nullptr;  // if set, the A operand is the elementwise product A * A2, A2 indexed like A
  const void* B = nullptr;
  int64_t b_sn = 0, b_sk = 0, b_sb = 0;
  int epi = EPI_STORE;
  void* D = nullptr;
  int64_t ldd = 0, d_sb = 0;
  bool d_f32 = false;  // D is float regardless of in_dtype
  void* D2 = nullptr;
  int64_t ldd2 = 0, d2_sb = 0;
  const void* E = nullptr;
  int64_t lde = 0, e_sb = 0;
  const void* E2 = nullptr;
  int64_t lde2 = 0, e2_sb = 0;
  const void* gate = nullptr;  // [N] per batch entry (stride gate_sb), nullptr = ones
  int64_t gate_sb = 0;
  float* R = nullptr;  // fp32 master copy of the residual stream [M][N], leading dim N
  bool relu = false;   // EPI_RESID on the CUDA-core kernel only: v = max(v, 0) and D2[m,n] = (v > 0) as 0/1 (the mask that gates this step)
  float2* stats = nullptr;  // EPI_STORE_LN: [batch][M][stats_slots] partial sums; batch stride stats_sb (in float2)
  int64_t stats_sb = 0;
  // float operands for the tensor cores: each of A (after the A2 product) and B split into a tf32-exact
  // high part and a tf32-rounded remainder, written with the contraction index contiguous (their own
  // strides below).  The tensor-core kernel forms A_hi B_lo + A_lo B_hi + A_hi B_hi (three tf32 products,
  // fp32 accumulation, the small terms first).
  const float *A_hi = nullptr, *A_lo = nullptr, *B_hi = nullptr, *B_lo = nullptr;
  int64_t hl_a_sm = 0, hl_a_sk = 0, hl_b_sn = 0, hl_b_sk = 0;
  int splitk = 1;      // > 1: partial sums to `partial` [splitk][batch][M][N], reduced in fixed order
  float* partial = nullptr;
  // self-test of the tensor-core kernel's bounded waits (hbp_selftest_wait_timeout): a wait limit other than the
  // default, and a producer that arms its first pipeline stage without issuing the copies
  uint64_t wait_limit_ns = 0;
  int test_stall = 0;
  bool dry_run = false;  // gemm_tc only: answer whether it would take this product, launch nothing
};

// Per-device memo for one-time set-up that CUDA keeps per device (kernel attributes, device properties): a
// process may drive several GPUs, each from its own context, so nothing of that kind is cached process-wide.
constexpr int kMaxDevices = 64;
inline int current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
  return dev;
}
template <typename T>
struct PerDevice {
  T v[kMaxDevices] = {};
  T& here() { return v[current_device()]; }
};

// Counts launches and remembers the first CUDA error; carries the kernel-selection modes of the context it runs for.
struct Launcher {
  cudaStream_t stream = nullptr;
  int64_t* launches = nullptr;
  cudaError_t err = cudaSuccess;
  bool force_simt = false;  // keep every GEMM and attention product on the CUDA-core kernels (cross-checks)
  bool gemm_pair = true;    // tensor-core GEMM pairs CTAs (cta_group::2, 256 x 256 tiles) where there are two row blocks
  void count(int n = 1) {
    if (launches) *launches += n;
  }
  void check() {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess && err == cudaSuccess) err = e;
  }
};

// CUDA-core GEMM for any strides and both dtypes (gemm_simt.cu).
void gemm_simt(Launcher& lc, const GemmArgs& g);
// tcgen05 / TMEM / TMA GEMM for bf16 operands; returns false if the problem does not meet its
// alignment rules, in which case nothing was launched (gemm_tc.cu).
bool gemm_tc(Launcher& lc, const GemmArgs& g, int* status_word);
// Picks gemm_tc when it applies, else gemm_simt (EPI_STORE_LN then degrades to EPI_STORE); returns
// whether the tensor-core kernel ran.
bool gemm(Launcher& lc, const GemmArgs& g, int* status_word);
// Number of 64-column slots of partial sums the tensor-core kernel writes per row for N columns.
int gemm_tc_stats_slots(int N);

// ---------------------------------------------------------------- scans and elementwise (scan.cu)
// Internal gate kind beside the public hbp_gate values: a[L][rows][d], one gate per element and step (the
// state-dependent gate of a GRU, produced by its forward pass).
constexpr int kGateElement = 3;
// ... and a[L][rows] in float, one gate per row and step (ScanArgs::row_gate; post-LN layers: 1 / sigma of the row)
constexpr int kGateRow = 4;
struct ScanArgs {
  int dtype = HBP_F32;
  int L = 0;               // number of steps in the buffers
  int l_lo = 0, l_hi = 0;  // processes l = l_hi-1 .. l_lo, carry-in read from g[l_hi]
  int64_t rows = 0;
  int d = 0;
  const void* u = nullptr;      // [L][rows][d] or nullptr (zeros)
  // Shifted split: g_l = delta_l + keep * a_l * g_{l+1} + u_l + gamma * (g_{l+1} of the previous iterate, read from
  // the g buffer before it is overwritten).  keep = 1 - gamma during Highway-BP, 1 otherwise.
  float keep = 1.0f, gamma = 0.0f;
  bool u_has_delta = false;     // u[l] already contains delta_l for l < L (added by the producing GEMM)
  const void* delta = nullptr;  // per hbp_loss
  int loss = HBP_LOSS_FINAL;
  const float* row_gate = nullptr;  // kGateRow only
  const void* u2 = nullptr;         // optional second additive tensor [L][rows][d] (serial depth scan only)
  const void* a = nullptr;  // gate
  int gate = HBP_GATE_ONE;  // an hbp_gate value, or kGateElement
  void* g = nullptr;  // [L+1][rows][d]
  // LayerNorm-backward finish: u is dY; the kernel forms rstd * (dy - mean(dy) - xhat * mean(dy*xhat)).
  // xhat [L][rows][d] in dtype, rstd [L][rows] float.
  const void* xhat = nullptr;
  const float* rstd = nullptr;
  // If set, [L][rows] of {rstd, mean(dy), mean(dy*xhat), 0} prepared by ln_stats_finish: the kernel then
  // needs no reduction of its own and streams like the plain scan.
  const float4* lnstat = nullptr;
  void* scratch = nullptr;  // time-chunked variant only
  size_t scratch_bytes = 0;
  int* status = nullptr;  // device status word for bounded waits (may be null)
  // Optional by-product for the float tanh RNN, written only by the TMA-ring kernel (which then sets *op_done):
  // the next all-step VJP's left operand g_{l+1} * coef_l, already split for the 3 x tf32 product, into rows
  // l = l_lo-1 .. l_hi-1 (l >= 0) of op_hi / op_lo ([L][rows][d] float, like op_coef).  With op_skip_g the kernel
  // leaves g alone (an intermediate iterate nobody reads).
  const float* op_coef = nullptr;
  float* op_hi = nullptr;
  float* op_lo = nullptr;
  bool op_skip_g = false;
  bool* op_done = nullptr;
};
size_t scan_scratch_bytes(int dtype, int L, int64_t rows, int d);
void scan_reverse(Launcher& lc, const ScanArgs& s);
// TMA-ring scan, serial in time, for few channels (scan_ring.cu); false if the problem does not qualify
// (nothing launched then).
bool scan_ring(Launcher& lc, const ScanArgs& s);
// lnstat[l][row] = {rstd, sum_slots s1 / d, sum_slots s2 / d, 0} from the GEMM's partial sums.
void ln_stats_finish(Launcher& lc, const float2* stats, int slots, const float* rstd, float4* lnstat, int64_t count,
                     int d);
void copy_state(Launcher& lc, int dtype, void* dst, const void* src, int64_t elems);
// dst[i] = a[i] * b[i] (dtype), elems a multiple of the 16-byte vector
void mul_elementwise(Launcher& lc, int dtype, void* dst, const void* a, const void* b, int64_t elems);
// states[s][e] += carry[e] for s in [0, count)
void add_to_states(Launcher& lc, int dtype, void* states, const void* carry, int count, int64_t elems);
// LayerNorm forward of one state: x (float master or dtype) -> xhat (dtype), rstd (float).
// (master, if given, receives the normalised values in float as well)
void layernorm_fwd(Launcher& lc, int dtype, const void* x, bool x_is_f32, void* xhat, float* rstd, int64_t rows,
                   int d, float eps, float* master = nullptr);
// t = rstd (g - mean g - xo mean(g xo)) and c = t - rstd g per row (post-LN layers; xo = the layer's output state)
void postln_prepass(Launcher& lc, int dtype, const void* g, const void* xo, const float* rstd, void* t_out, void* c_out,
                    int64_t rows, int d);
void convert_to_f32(Launcher& lc, int dtype, const void* src, float* dst, int64_t elems);
// da[c] = sum over rows of g[r][c] * x[r][c] (deterministic two-stage reduction; partial holds blocks*d floats).
void gate_grad(Launcher& lc, int dtype, const void* g, const void* x, int64_t rows_total, int d, float* da,
               float* partial, int blocks);
void reduce_splitk(Launcher& lc, const float* partial, float* out, int splits, int64_t elems);
// hi = tf32-exact part of v, lo = tf32 rounding of (v - hi), with v = a[i] * (b ? b[i] : 1).
void split_tf32(Launcher& lc, const float* a, const float* b, float* hi, float* lo, int64_t elems);
// The same for a [rows][cols] matrix, written transposed: hiT, loT are [cols][rows].
// (ld = elements between rows of a and b; 0 = cols)
void split_tf32_transposed(Launcher& lc, const float* a, const float* b, float* hiT, float* loT, int64_t rows, int cols,
                           int64_t ld = 0);

// ---------------------------------------------------------------- RNN forward step (rnn.cu)
// z = W h + U x_t in double from the double master state h_in; writes h_out (double), the cached
// derivative 1 - tanh(z)^2 and the next stored state (both in dtype).
void rnn_forward_step(Launcher& lc, int dtype, const void* W, const void* U, const void* x_t, const void* gate,
                      const double* h_in, double* h_out, void* deriv, void* state_out, int B, int d, int in_dim);
// g_t = delta_t + a * g_{t+1} + (g_{t+1} * deriv_t) W in double from the double master g_in.
void rnn_backward_step(Launcher& lc, int dtype, const void* W, const void* deriv, const void* delta, const void* gate,
                       const double* g_in, double* g_out, void* g_store, int B, int d);
void convert_to_f64(Launcher& lc, int dtype, const void* src, double* dst, int64_t elems);
// The same recurrences as ONE launch over all T steps (rnn_persistent.cu): clusters of 16 CTAs own 4 batch rows
// each, the recurrent matrix stays in registers, the state moves between the CTAs through distributed shared
// memory.  status: device status word for the kernel's bounded waits.  P is scratch of rnn_persistent_proj_bytes(...) bytes for U x_t of every step in double (0 = the width is
// not one this form takes).  Both return false when nothing was done for the recurrence (unsupported width, or
// clusters of 16 cannot be scheduled on this device): the caller then runs the per-step kernels.
size_t rnn_persistent_proj_bytes(int T, int64_t B, int d);
bool rnn_forward_persistent(Launcher& lc, int dtype, const void* W, const void* U, const void* X, const void* gate,
                            const void* x0, double* P, void* x_all, void* deriv, int T, int B, int d, int in_dim, int* status);
bool rnn_backward_persistent(Launcher& lc, int dtype, const void* W, const void* gate, const void* deriv,
                             const void* delta, void* g_all, int T, int B, int d, int* status);

// ---------------------------------------------------------------- diagnostics (diag.cu)
// out[seg][4] = {<a,b>, |a|^2, |b|^2, |a-b|^2} over `elems` elements per segment; scratch holds
// compare_scratch_bytes(segments) bytes.
size_t compare_scratch_bytes(int segments);
void compare_segments(Launcher& lc, int dtype, const void* a, const void* b, int segments, int64_t elems, double* out,
                      double* scratch);

// ---------------------------------------------------------------- GRU (gru.cu)
// One forward step in double from the double master state; writes the new master, the stored state, the
// gate z [B][d] and the VJP coefficients c4 [B][4d] = [c_r | c_z | c_nr | c_n].
void gru_forward_step(Launcher& lc, int dtype, const void* W, const void* U, const void* x_t, const double* h_in,
                      double* h_out, void* zc, void* c4, void* state_out, int B, int d, int in_dim);
// g_t = delta_t + z_t * g_{t+1} + (g_{t+1} * [c_r | c_z | c_nr]) W in double from the double master g_in.
void gru_backward_step(Launcher& lc, int dtype, const void* W, const void* zc, const void* c4, const void* delta,
                       const double* g_in, double* g_out, void* g_store, int B, int d);
// a4[row][q*d + c] = g[row][c] * c4[row][q*d + c], in dtype.
void gru_operand(Launcher& lc, int dtype, const void* g, const void* c4, void* a4, int64_t rows, int d);
// tf32 high/low split of g * c4: columns [0, 3d) as [rows][3d], or all of it transposed as [4d][rows].
void gru_split(Launcher& lc, const float* g, const float* c4, float* hi, float* lo, int64_t rows, int d);
void gru_split_transposed(Launcher& lc, const float* g, const float* c4, float* hiT, float* loT, int64_t rows, int d);

// ---------------------------------------------------------------- LSTM (lstm.cu); u units, state [c | h] 2u wide
// One forward step in double from the double master state; writes the new master, the stored state, the scan's
// gate fg [B][2u] = [f | 0] and the VJP coefficients c5 [B][5u] = [c_i | c_f | c_g | c_o | c_h].
void lstm_forward_step(Launcher& lc, int dtype, const void* W, const void* U, const void* x_t, const double* s_in,
                       double* s_out, void* fg, void* c5, void* state_out, int B, int u, int in_dim);
// exact backpropagation through one step in double from the double master g_in
void lstm_backward_step(Launcher& lc, int dtype, const void* W, const void* fg, const void* c5, const void* delta,
                        const double* g_in, double* g_out, void* g_store, int B, int u);
// a4 [rows][4u] = [t c_i | t c_f | t c_g | g_h c_o], t = g_c + g_h c_h, from g [rows][2u]; if uo is given also the
// cell-state half of the block VJP, uo[row][0..u) = f g_h c_h (+ delta), rows of uo 2u wide
void lstm_operand(Launcher& lc, int dtype, const void* g, const void* c5, const void* fg, const void* delta, void* a4,
                  void* uo, int64_t rows, int u);
// the same operand as tf32 high/low parts: [rows][4u] (with the optional uo), or transposed [4u][rows]
void lstm_split(Launcher& lc, const float* g, const float* c5, const float* fg, const float* delta, float* hi, float* lo,
                float* uo, int64_t rows, int u);
void lstm_split_transposed(Launcher& lc, const float* g, const float* c5, float* hiT, float* loT, int64_t rows, int u);

// ---------------------------------------------------------------- attention (attention.cu)
struct AttnArgs {
  int dtype = HBP_BF16;
  int batch = 0, seq = 0, heads = 0, head_dim = 0;
  // q, k, v are column blocks of one [tokens][3d] buffer (ld = 3d); o, d_o are [tokens][d].
  const void* qkv = nullptr;
  void* o = nullptr;
  float* lse = nullptr;  // [batch][heads][seq]
  const void* d_o = nullptr;
  void* d_qkv = nullptr;        // [tokens][3d]
  float* delta_rows = nullptr;  // scratch [batch][heads][seq]: rowsum(dO * O)
  // If set (head dimension 64 only): rowsum(dO * O) already sits in the .y of d_stats[token][d_slots + head],
  // written by the epilogue of the GEMM that produced dO; the row-dot pass is then skipped.
  const float2* d_stats = nullptr;
  int d_slots = 0;
  int* status = nullptr;        // device status word for the bounded waits of the tensor-core kernels
};
void attention_fwd(Launcher& lc, const AttnArgs& a);
void attention_bwd(Launcher& lc, const AttnArgs& a);
// Tensor-core dQ/dK/dV (attention_tc.cu); false if the problem does not qualify (nothing launched).
bool attention_bwd_tc(Launcher& lc, const AttnArgs& a, int* status_word);
// Tensor-core forward (attention_tc.cu), same conditions.
bool attention_fwd_tc(Launcher& lc, const AttnArgs& a, int* status_word);

// ---------------------------------------------------------------- device math
__device__ __forceinline__ float gelu_f(float z) { return 0.5f * z * (1.0f + erff(z * 0.70710678118654752440f)); }
__device__ __forceinline__ float gelu_prime_f(float z) {
  return 0.5f * (1.0f + erff(z * 0.70710678118654752440f)) + z * expf(-0.5f * z * z) * 0.39894228040143267794f;
}
// v rounded to tf32 precision (13 low mantissa bits cleared, round to nearest even)
__device__ __forceinline__ float round_tf32(float v) {
  uint32_t u = __float_as_uint(v);
  u += 0x00000fffu + ((u >> 13) & 1u);
  return __uint_as_float(u & 0xffffe000u);
}
__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(bf16 v) { return __bfloat162float(v); }
template <typename T>
__device__ __forceinline__ T from_f(float v);
template <>
__device__ __forceinline__ float from_f<float>(float v) {
  return v;
}
template <>
__device__ __forceinline__ bf16 from_f<bf16>(float v) {
  return __float2bfloat16_rn(v);
}

}  // namespace hbp
