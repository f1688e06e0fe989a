// One forward step of the gated tanh RNN (Section 5.2: the cell at time t is layer f_t):
//     z = W h_t + U x_t,  c = tanh(z),  h_{t+1} = a * h_t + c,  and the cached derivative 1 - c^2.
// The recurrence is carried in double precision (a master copy of h beside the stored states) so
// that thousands of dependent steps do not accumulate float rounding; the stored state and the cached
// derivative are the roundings of the double values.  4096 such steps are latency-bound by design:
// this is the sequential part that the time-parallel backward removes.
#include "hbp_internal.h"

namespace hbp {

namespace {

constexpr int kTile = 32;

template <typename T>
__global__ void __launch_bounds__(256) rnn_step_kernel(const T* __restrict__ W, const T* __restrict__ U,
                                                       const T* __restrict__ x_t, const T* __restrict__ gate,
                                                       const double* __restrict__ h_in, double* __restrict__ h_out,
                                                       T* __restrict__ deriv, T* __restrict__ state_out, int B, int d,
                                                       int in_dim) {
  __shared__ double Hs[kTile][kTile + 1];
  __shared__ float Ws[kTile][kTile + 1];
  const int tx = threadIdx.x % kTile, ty = threadIdx.x / kTile;  // ty in 0..7
  const int n0 = blockIdx.x * kTile, m0 = blockIdx.y * kTile;
  double acc[4] = {0.0, 0.0, 0.0, 0.0};
  const int ktotal = d + in_dim;
  for (int k0 = 0; k0 < ktotal; k0 += kTile) {
    // rows of the chunk come from h (k < d) or from x_t (k >= d); d and in_dim are multiples of 4,
    // chunks may straddle the boundary, so the source is picked per element
    for (int i = ty; i < kTile; i += 8) {
      const int k = k0 + tx;
      const int m = m0 + i, n = n0 + i;
      double hv = 0.0;
      float wv = 0.0f;
      if (k < ktotal) {
        if (m < B) hv = k < d ? h_in[(int64_t)m * d + k] : (double)to_f(x_t[(int64_t)m * in_dim + (k - d)]);
        if (n < d) wv = k < d ? to_f(W[(int64_t)n * d + k]) : to_f(U[(int64_t)n * in_dim + (k - d)]);
      }
      Hs[i][tx] = hv;
      Ws[i][tx] = wv;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kTile; ++kk) {
      const double w = (double)Ws[tx][kk];
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[j] = fma(Hs[ty + 8 * j][kk], w, acc[j]);
    }
    __syncthreads();
  }
  const int n = n0 + tx;
  if (n >= d) return;
  const double a = gate ? (double)to_f(gate[n]) : 1.0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int m = m0 + ty + 8 * j;
    if (m >= B) continue;
    const double z = acc[j];
    const double e = exp(-2.0 * fabs(z));
    const double c = copysign((1.0 - e) / (1.0 + e), z);
    const double s = 4.0 * e / ((1.0 + e) * (1.0 + e));  // 1 - tanh(z)^2 without cancellation
    const double hn = a * h_in[(int64_t)m * d + n] + c;
    h_out[(int64_t)m * d + n] = hn;
    deriv[(int64_t)m * d + n] = from_f<T>((float)s);
    state_out[(int64_t)m * d + n] = from_f<T>((float)hn);
  }
}

// One step of exact backpropagation through time, carried in double like the forward recurrence:
//     g_t = delta_t + a * g_{t+1} + (g_{t+1} * tanh'(z_t)) W
// from the double master copy of g_{t+1}; writes the new master and its rounding g[t].
template <typename T>
__global__ void __launch_bounds__(256) rnn_bwd_step_kernel(const T* __restrict__ W, const T* __restrict__ deriv,
                                                           const T* __restrict__ delta, const T* __restrict__ gate,
                                                           const double* __restrict__ g_in, double* __restrict__ g_out,
                                                           T* __restrict__ g_store, int B, int d) {
  __shared__ double Hs[kTile][kTile + 1];
  __shared__ float Ws[kTile][kTile + 1];
  const int tx = threadIdx.x % kTile, ty = threadIdx.x / kTile;
  const int n0 = blockIdx.x * kTile, m0 = blockIdx.y * kTile;
  double acc[4] = {0.0, 0.0, 0.0, 0.0};
  for (int k0 = 0; k0 < d; k0 += kTile) {
    for (int i = ty; i < kTile; i += 8) {
      const int m = m0 + i, k = k0 + tx;
      Hs[i][tx] = (m < B && k < d) ? g_in[(int64_t)m * d + k] * (double)to_f(deriv[(int64_t)m * d + k]) : 0.0;
      const int kk = k0 + i, n = n0 + tx;  // W[k][n]: contiguous in n
      Ws[tx][i] = (kk < d && n < d) ? to_f(W[(int64_t)kk * d + n]) : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kTile; ++kk) {
      const double w = (double)Ws[tx][kk];
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[j] = fma(Hs[ty + 8 * j][kk], w, acc[j]);
    }
    __syncthreads();
  }
  const int n = n0 + tx;
  if (n >= d) return;
  const double a = gate ? (double)to_f(gate[n]) : 1.0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int m = m0 + ty + 8 * j;
    if (m >= B) continue;
    const int64_t idx = (int64_t)m * d + n;
    const double v = (delta ? (double)to_f(delta[idx]) : 0.0) + a * g_in[idx] + acc[j];
    g_out[idx] = v;
    g_store[idx] = from_f<T>((float)v);
  }
}

// ---- the same two steps with all operands of a block staged in shared memory at once ------------------------
// The tiled kernels above wait for global memory once per 32 of K (24 times per step on d = 512, in = 256) and
// use d / 32 blocks.  Here a block owns 16 rows x 8 columns of the step's output, issues every load it needs in
// one go (the state rows in double, its 8 weight rows converted to double once), and two threads per output
// split the contraction; one exposed memory latency per step instead of 24, and d / 8 x B / 16 blocks.
constexpr int kSRows = 16, kSCols = 8;

__device__ __forceinline__ double dot_halves(const double* __restrict__ a, const double* __restrict__ w, int n, int half) {
  double acc0 = 0.0, acc1 = 0.0, acc2 = 0.0, acc3 = 0.0;
  int k = half;
  for (; k + 6 < n; k += 8) {
    acc0 = fma(a[k], w[k], acc0);
    acc1 = fma(a[k + 2], w[k + 2], acc1);
    acc2 = fma(a[k + 4], w[k + 4], acc2);
    acc3 = fma(a[k + 6], w[k + 6], acc3);
  }
  for (; k < n; k += 2) acc0 = fma(a[k], w[k], acc0);
  return (acc0 + acc1) + (acc2 + acc3);
}

__device__ __forceinline__ double as_double(double v) { return v; }
__device__ __forceinline__ double as_double(float v) { return (double)v; }
__device__ __forceinline__ double as_double(bf16 v) { return (double)to_f(v); }

// dst[r * lda + col0 + c] = src[(r0 + r) * ld + c] as double for r < R, c < ncols (zero where r0 + r >= rmax).  A thread
// walks columns and issues the loads of all R rows of a column before the first store: the block has its whole tile in
// flight at once, and no index needs a division.
template <int R, typename S>
__device__ __forceinline__ void stage_tile(double* __restrict__ dst, int lda, int col0, const S* __restrict__ src, int64_t ld,
                                           int r0, int rmax, int ncols) {
  for (int c = threadIdx.x; c < ncols; c += blockDim.x) {
    double v[R];
#pragma unroll
    for (int r = 0; r < R; ++r) v[r] = r0 + r < rmax ? as_double(src[(int64_t)(r0 + r) * ld + c]) : 0.0;
#pragma unroll
    for (int r = 0; r < R; ++r) dst[r * lda + col0 + c] = v[r];
  }
}

template <typename T>
__global__ void __launch_bounds__(256) rnn_step_staged_kernel(const T* __restrict__ W, const T* __restrict__ U,
                                                              const T* __restrict__ x_t, const T* __restrict__ gate,
                                                              const double* __restrict__ h_in, double* __restrict__ h_out,
                                                              T* __restrict__ deriv, T* __restrict__ state_out, int B,
                                                              int d, int in_dim) {
  extern __shared__ double sm[];
  const int ktot = d + in_dim, lda = ktot + 2;  // padded rows: the 8 weight rows of a warp fall on distinct banks
  double* As = sm;                     // [kSRows][lda]: h | x_t
  double* Ws = sm + kSRows * lda;      // [kSCols][lda]: W row | U row
  const int n0 = blockIdx.x * kSCols, m0 = blockIdx.y * kSRows;
  stage_tile<kSRows, double>(As, lda, 0, h_in, d, m0, B, d);
  stage_tile<kSRows, T>(As, lda, d, x_t, in_dim, m0, B, in_dim);
  stage_tile<kSCols, T>(Ws, lda, 0, W, d, n0, d, d);
  stage_tile<kSCols, T>(Ws, lda, d, U, in_dim, n0, d, in_dim);
  __syncthreads();
  const int o = threadIdx.x >> 1, half = threadIdx.x & 1, m = o / kSCols, c = o % kSCols;
  double z = dot_halves(As + m * lda, Ws + c * lda, ktot, half);
  z += __shfl_xor_sync(0xffffffffu, z, 1);
  const int gm = m0 + m, n = n0 + c;
  if (half != 0 || gm >= B || n >= d) return;
  const double a = gate ? (double)to_f(gate[n]) : 1.0;
  const double e = exp(-2.0 * fabs(z));
  const double cth = copysign((1.0 - e) / (1.0 + e), z);
  const double sl = 4.0 * e / ((1.0 + e) * (1.0 + e));  // 1 - tanh(z)^2 without cancellation
  const double hn = a * As[m * lda + n] + cth;
  const int64_t idx = (int64_t)gm * d + n;
  h_out[idx] = hn;
  deriv[idx] = from_f<T>((float)sl);
  state_out[idx] = from_f<T>((float)hn);
}

template <typename T>
__global__ void __launch_bounds__(256) rnn_bwd_step_staged_kernel(const T* __restrict__ W, const T* __restrict__ deriv,
                                                                  const T* __restrict__ delta, const T* __restrict__ gate,
                                                                  const double* __restrict__ g_in, double* __restrict__ g_out,
                                                                  T* __restrict__ g_store, int B, int d) {
  extern __shared__ double sm[];
  const int lda = d + 2;
  double* As = sm;                   // [kSRows][lda]: g_{t+1} * tanh'(z_t)
  double* Ws = sm + kSRows * lda;    // [kSCols][lda]: columns n0.. of W, one per row here
  const int n0 = blockIdx.x * kSCols, m0 = blockIdx.y * kSRows;
  for (int k = threadIdx.x; k < d; k += blockDim.x) {  // all rows of a column in flight before the first store
    double gv[kSRows];
    float dv[kSRows];
#pragma unroll
    for (int m = 0; m < kSRows; ++m) {
      const bool okm = m0 + m < B;
      gv[m] = okm ? g_in[(int64_t)(m0 + m) * d + k] : 0.0;
      dv[m] = okm ? to_f(deriv[(int64_t)(m0 + m) * d + k]) : 0.0f;
    }
#pragma unroll
    for (int m = 0; m < kSRows; ++m) As[m * lda + k] = gv[m] * (double)dv[m];
  }
#pragma unroll 8
  for (int idx = threadIdx.x; idx < kSCols * d; idx += blockDim.x) {
    const int k = idx / kSCols, c = idx - k * kSCols, n = n0 + c;  // 8 neighbouring columns of row k: one 32-byte read
    Ws[c * lda + k] = n < d ? (double)to_f(W[(int64_t)k * d + n]) : 0.0;
  }
  __syncthreads();
  const int o = threadIdx.x >> 1, half = threadIdx.x & 1, m = o / kSCols, c = o % kSCols;
  double acc = dot_halves(As + m * lda, Ws + c * lda, d, half);
  acc += __shfl_xor_sync(0xffffffffu, acc, 1);
  const int gm = m0 + m, n = n0 + c;
  if (half != 0 || gm >= B || n >= d) return;
  const double a = gate ? (double)to_f(gate[n]) : 1.0;
  const int64_t idx = (int64_t)gm * d + n;
  const double v = (delta ? (double)to_f(delta[idx]) : 0.0) + a * g_in[idx] + acc;
  g_out[idx] = v;
  g_store[idx] = from_f<T>((float)v);
}

constexpr size_t kStagedSmemLimit = 200 * 1024;
inline size_t staged_bytes(int k_a, int k_w) { return ((size_t)kSRows * (k_a + 2) + (size_t)kSCols * (k_w + 2)) * sizeof(double); }
template <typename K>
bool allow_smem(K kernel, size_t bytes, size_t* configured) {
  if (bytes <= *configured) return true;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  *configured = bytes;
  return true;
}

template <typename T>
__global__ void to_f64_kernel(const T* __restrict__ src, double* __restrict__ dst, int64_t n) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = (double)to_f(src[i]);
}

}  // namespace

void rnn_forward_step(Launcher& lc, int dtype, const void* W, const void* U, const void* x_t, const void* gate,
                      const double* h_in, double* h_out, void* deriv, void* state_out, int B, int d, int in_dim) {
  const size_t staged = staged_bytes(d + in_dim, d + in_dim);
  if (staged <= kStagedSmemLimit) {
    static PerDevice<size_t> cfg_f_on, cfg_b_on;  // per-device kernel attributes
    size_t &cfg_f = cfg_f_on.here(), &cfg_b = cfg_b_on.here();
    dim3 sgrid((d + kSCols - 1) / kSCols, (B + kSRows - 1) / kSRows);
    if (dtype == HBP_F32 && allow_smem(rnn_step_staged_kernel<float>, staged, &cfg_f)) {
      rnn_step_staged_kernel<float><<<sgrid, 256, staged, lc.stream>>>((const float*)W, (const float*)U, (const float*)x_t,
                                                                       (const float*)gate, h_in, h_out, (float*)deriv,
                                                                       (float*)state_out, B, d, in_dim);
      lc.count();
      lc.check();
      return;
    }
    if (dtype == HBP_BF16 && allow_smem(rnn_step_staged_kernel<bf16>, staged, &cfg_b)) {
      rnn_step_staged_kernel<bf16><<<sgrid, 256, staged, lc.stream>>>((const bf16*)W, (const bf16*)U, (const bf16*)x_t,
                                                                      (const bf16*)gate, h_in, h_out, (bf16*)deriv,
                                                                      (bf16*)state_out, B, d, in_dim);
      lc.count();
      lc.check();
      return;
    }
  }
  dim3 grid((d + kTile - 1) / kTile, (B + kTile - 1) / kTile);
  if (dtype == HBP_F32)
    rnn_step_kernel<float><<<grid, 256, 0, lc.stream>>>((const float*)W, (const float*)U, (const float*)x_t,
                                                        (const float*)gate, h_in, h_out, (float*)deriv,
                                                        (float*)state_out, B, d, in_dim);
  else
    rnn_step_kernel<bf16><<<grid, 256, 0, lc.stream>>>((const bf16*)W, (const bf16*)U, (const bf16*)x_t,
                                                       (const bf16*)gate, h_in, h_out, (bf16*)deriv, (bf16*)state_out,
                                                       B, d, in_dim);
  lc.count();
  lc.check();
}

void rnn_backward_step(Launcher& lc, int dtype, const void* W, const void* deriv, const void* delta, const void* gate,
                       const double* g_in, double* g_out, void* g_store, int B, int d) {
  const size_t staged = staged_bytes(d, d);
  if (staged <= kStagedSmemLimit) {
    static PerDevice<size_t> cfg_f_on, cfg_b_on;  // per-device kernel attributes
    size_t &cfg_f = cfg_f_on.here(), &cfg_b = cfg_b_on.here();
    dim3 sgrid((d + kSCols - 1) / kSCols, (B + kSRows - 1) / kSRows);
    if (dtype == HBP_F32 && allow_smem(rnn_bwd_step_staged_kernel<float>, staged, &cfg_f)) {
      rnn_bwd_step_staged_kernel<float><<<sgrid, 256, staged, lc.stream>>>((const float*)W, (const float*)deriv,
                                                                           (const float*)delta, (const float*)gate, g_in,
                                                                           g_out, (float*)g_store, B, d);
      lc.count();
      lc.check();
      return;
    }
    if (dtype == HBP_BF16 && allow_smem(rnn_bwd_step_staged_kernel<bf16>, staged, &cfg_b)) {
      rnn_bwd_step_staged_kernel<bf16><<<sgrid, 256, staged, lc.stream>>>((const bf16*)W, (const bf16*)deriv,
                                                                          (const bf16*)delta, (const bf16*)gate, g_in,
                                                                          g_out, (bf16*)g_store, B, d);
      lc.count();
      lc.check();
      return;
    }
  }
  dim3 grid((d + kTile - 1) / kTile, (B + kTile - 1) / kTile);
  if (dtype == HBP_F32)
    rnn_bwd_step_kernel<float><<<grid, 256, 0, lc.stream>>>((const float*)W, (const float*)deriv, (const float*)delta,
                                                            (const float*)gate, g_in, g_out, (float*)g_store, B, d);
  else
    rnn_bwd_step_kernel<bf16><<<grid, 256, 0, lc.stream>>>((const bf16*)W, (const bf16*)deriv, (const bf16*)delta,
                                                           (const bf16*)gate, g_in, g_out, (bf16*)g_store, B, d);
  lc.count();
  lc.check();
}

void convert_to_f64(Launcher& lc, int dtype, const void* src, double* dst, int64_t elems) {
  const unsigned grid = (unsigned)((elems + 255) / 256);
  if (dtype == HBP_F32) to_f64_kernel<float><<<grid, 256, 0, lc.stream>>>((const float*)src, dst, elems);
  else to_f64_kernel<bf16><<<grid, 256, 0, lc.stream>>>((const bf16*)src, dst, elems);
  lc.count();
  lc.check();
}

}  // namespace hbp
