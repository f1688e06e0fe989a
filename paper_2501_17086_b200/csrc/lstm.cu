// LSTM cell as a residual step on the state x = [c, h] (Table 1, row "LSTM"), u units, state width 2u:
//     [i, f, g, o] = [sigmoid, sigmoid, tanh, sigmoid](U x_t + W h),   c' = f * c + i * g,   h' = o * tanh(c').
// K = diag([f, 0]) is the cheap Jacobian (only the cell state has a linear path).  With the upstream gradient
// [g_c, g_h], t = g_c + g_h * c_h is what reaches c' (c_h = o (1 - tanh(c')^2)), and the block VJP is
//     u_c = f * g_h * c_h,     u_h = [t c_i | t c_f | t c_g | g_h c_o] W
// with the per-element coefficients c_i = g i (1 - i), c_f = c f (1 - f), c_g = i (1 - g^2), c_o = tanh(c') o (1 - o),
// computed once, in double, by the forward step and stored as C5 = [c_i | c_f | c_g | c_o | c_h] per row.  The
// parameter gradients contract the same four-block operand with h and with x_t.  As for the other recurrent cells,
// the recurrence itself and exact backpropagation through time are carried in double beside the stored values.
#include "cluster_split.cuh"

namespace hbp {

namespace {

constexpr int kTile = 32;

// acc[q][j] += sum_k src[m_j][k] * Wm[q * u + n][k] over k in [k_lo, k_hi) (k_lo a multiple of the tile); src rows are
// src_ld apart
template <typename T, bool kSrcDouble>
__device__ __forceinline__ void lstm_accumulate(const void* __restrict__ src, int64_t src_ld, const T* __restrict__ Wm,
                                                int kdim, int B, int u, int m0, int n0, double (*Hs)[kTile + 1],
                                                float (*Ws)[kTile][kTile + 1], double (*acc)[4], int k_lo, int k_hi) {
  if (k_lo >= k_hi) return;
  const int tx = threadIdx.x % kTile, ty = threadIdx.x / kTile;
  // The next tile's global loads are issued into registers before the current tile is multiplied, so the loop
  // waits for memory once, not once per tile.
  double hreg[4];
  float wreg[4][4];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int i = ty + 8 * j;
      const int k = k0 + tx, m = m0 + i, n = n0 + i;
      double hv = 0.0;
      if (k < kdim && m < B)
        hv = kSrcDouble ? ((const double*)src)[(int64_t)m * src_ld + k] : (double)to_f(((const T*)src)[(int64_t)m * src_ld + k]);
      hreg[j] = hv;
#pragma unroll
      for (int q = 0; q < 4; ++q) wreg[q][j] = (k < kdim && n < u) ? to_f(Wm[((int64_t)q * u + n) * kdim + k]) : 0.0f;
    }
  };
  fetch(k_lo);
  for (int k0 = k_lo; k0 < k_hi; k0 += kTile) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int i = ty + 8 * j;
      Hs[i][tx] = hreg[j];
#pragma unroll
      for (int q = 0; q < 4; ++q) Ws[q][i][tx] = wreg[q][j];
    }
    __syncthreads();
    if (k0 + kTile < k_hi) fetch(k0 + kTile);
#pragma unroll 8
    for (int kk = 0; kk < kTile; ++kk) {
      double w[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) w[q] = (double)Ws[q][tx][kk];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const double hv = Hs[ty + 8 * j][kk];
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[q][j] = fma(hv, w[q], acc[q][j]);
      }
    }
    __syncthreads();
  }
}

__device__ __forceinline__ double sigmoid_d(double v) { return 1.0 / (1.0 + exp(-v)); }
// tanh(v) and 1 - tanh(v)^2 = 4e / (1 + e)^2 with e = exp(-2|v|): no cancellation near saturation
__device__ __forceinline__ void tanh_and_slope(double v, double& t, double& s) {
  const double e = exp(-2.0 * fabs(v));
  t = copysign((1.0 - e) / (1.0 + e), v);
  s = 4.0 * e / ((1.0 + e) * (1.0 + e));
}

template <typename T, bool kCluster>
__global__ void __launch_bounds__(256) lstm_step_kernel(const T* __restrict__ W, const T* __restrict__ U,
                                                        const T* __restrict__ x_t, const double* __restrict__ s_in,
                                                        double* __restrict__ s_out, T* __restrict__ fg,
                                                        T* __restrict__ c5, T* __restrict__ state_out, int B, int u,
                                                        int in_dim) {
  __shared__ double Hs[kTile][kTile + 1];
  __shared__ float Ws[4][kTile][kTile + 1];
  extern __shared__ double red[];  // partial sums of the cluster's other ranks (see cluster_splitk_reduce)
  const int tx = threadIdx.x % kTile, ty = threadIdx.x / kTile;
  const int n0 = blockIdx.x * kTile, m0 = blockIdx.y * kTile;
  double flat[16];  // [gate][row]
#pragma unroll
  for (int i = 0; i < 16; ++i) flat[i] = 0.0;
  double (*acc)[4] = reinterpret_cast<double (*)[4]>(flat);
  // the CTAs of a cluster share the k-tiles of both products out and add their partial sums
  // (a kernel that reads the cluster registers is launched as a cluster even alone, which costs microseconds per launch:
  // the form without a split does not touch them)
  const int ks = kCluster ? (int)tc::cluster_nctarank() : 1, rank = kCluster ? (int)tc::cluster_ctarank() : 0;
  // the previous cell state of this thread's outputs, fetched before the products so that the epilogue does not wait
  double cprev[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int m = m0 + ty + 8 * j, n = n0 + tx;
    cprev[j] = (m < B && n < u) ? s_in[(int64_t)m * 2 * u + n] : 0.0;
  }
  const int nt_h = (u + kTile - 1) / kTile, nt_x = (in_dim + kTile - 1) / kTile;
  lstm_accumulate<T, true>(s_in + u, 2 * u, W, u, B, u, m0, n0, Hs, Ws, acc, (nt_h * rank / ks) * kTile,
                           min(u, (nt_h * (rank + 1) / ks) * kTile));   // W h: h is the second half of the state
  lstm_accumulate<T, false>(x_t, in_dim, U, in_dim, B, u, m0, n0, Hs, Ws, acc, (nt_x * rank / ks) * kTile,
                            min(in_dim, (nt_x * (rank + 1) / ks) * kTile));  // + U x_t
  if (kCluster && !tc::cluster_splitk_reduce(flat, red)) return;
  const int n = n0 + tx;
  if (n >= u) return;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int m = m0 + ty + 8 * j;
    if (m >= B) continue;
    const double i = sigmoid_d(acc[0][j]), i1 = sigmoid_d(-acc[0][j]);
    const double f = sigmoid_d(acc[1][j]), f1 = sigmoid_d(-acc[1][j]);
    const double o = sigmoid_d(acc[3][j]), o1 = sigmoid_d(-acc[3][j]);
    double g, dg, tc, dtc;
    tanh_and_slope(acc[2][j], g, dg);
    const double c = cprev[j];
    const double cn = f * c + i * g;
    tanh_and_slope(cn, tc, dtc);
    const double hn = o * tc;
    const int64_t so = (int64_t)m * 2 * u + n;
    s_out[so] = cn;
    s_out[so + u] = hn;
    state_out[so] = from_f<T>((float)cn);
    state_out[so + u] = from_f<T>((float)hn);
    fg[so] = from_f<T>((float)f);
    fg[so + u] = from_f<T>(0.0f);
    T* k = c5 + (int64_t)m * 5 * u + n;
    k[0] = from_f<T>((float)(g * i * i1));
    k[u] = from_f<T>((float)(c * f * f1));
    k[2 * u] = from_f<T>((float)(i * dg));
    k[3 * u] = from_f<T>((float)(tc * o * o1));
    k[4 * u] = from_f<T>((float)(o * dtc));
  }
}

__device__ __forceinline__ double as_d(double v) { return v; }
__device__ __forceinline__ double as_d(float v) { return (double)v; }

// element (row, column k of the [4u] operand) from the upstream gradient [g_c | g_h] and the coefficients
// (C = the type to compute in: double for exact backpropagation, float for GEMM operands)
template <typename C, typename T, typename G>
__device__ __forceinline__ C operand_value(const G* __restrict__ g_row, const T* __restrict__ c5_row, int u, int k) {
  const int q = k / u, n = k - q * u;
  const C gh = (C)as_d(g_row[u + n]);
  if (q == 3) return gh * (C)to_f(c5_row[3 * u + n]);
  const C t = (C)as_d(g_row[n]) + gh * (C)to_f(c5_row[4 * u + n]);
  return t * (C)to_f(c5_row[q * u + n]);
}

// the four operand values of (row, unit n) at once
template <typename T>
__device__ __forceinline__ void operand_quad(const T* __restrict__ g_row, const T* __restrict__ c5_row, int u, int n, float* v) {
  const float gh = to_f(g_row[u + n]);
  const float t = to_f(g_row[n]) + gh * to_f(c5_row[4 * u + n]);
  v[0] = t * to_f(c5_row[n]);
  v[1] = t * to_f(c5_row[u + n]);
  v[2] = t * to_f(c5_row[2 * u + n]);
  v[3] = gh * to_f(c5_row[3 * u + n]);
}

// Exact backpropagation through one step in double: g_t = delta_t + [f * g_c, 0] + [u_c, u_h].
template <typename T, bool kCluster>
__global__ void __launch_bounds__(256) lstm_bwd_step_kernel(const T* __restrict__ W, const T* __restrict__ fg,
                                                            const T* __restrict__ c5, const T* __restrict__ delta,
                                                            const double* __restrict__ g_in, double* __restrict__ g_out,
                                                            T* __restrict__ g_store, int B, int u) {
  __shared__ double Hs[kTile][kTile + 1];
  __shared__ float Ws[kTile][kTile + 1];
  __shared__ double red[(tc::kMaxClusterSplit - 1) * 4 * 256];
  const int tx = threadIdx.x % kTile, ty = threadIdx.x / kTile;
  const int n0 = blockIdx.x * kTile, m0 = blockIdx.y * kTile;
  double acc[4] = {0.0, 0.0, 0.0, 0.0};
  // the CTAs of a cluster share the k-tiles out (one step has too few output tiles to fill the GPU) and add their
  // partial sums at the end
  const int ntiles = (4 * u + kTile - 1) / kTile;
  // (a kernel that reads the cluster registers is launched as a cluster even alone, which costs microseconds per launch:
  // the form without a split does not touch them)
  const int ks = kCluster ? (int)tc::cluster_nctarank() : 1, rank = kCluster ? (int)tc::cluster_ctarank() : 0;
  const int k_lo = (ntiles * rank / ks) * kTile, k_hi = min(4 * u, (ntiles * (rank + 1) / ks) * kTile);
  // the next tile's operands are fetched into registers before the current tile is multiplied
  double hreg[4];
  float wreg[4];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int i = ty + 8 * j;
      const int m = m0 + i, k = k0 + tx;
      hreg[j] = (m < B && k < 4 * u) ? operand_value<double, T, double>(g_in + (int64_t)m * 2 * u, c5 + (int64_t)m * 5 * u, u, k) : 0.0;
      const int kk = k0 + i, n = n0 + tx;  // W[k][n]: contiguous in n
      wreg[j] = (kk < 4 * u && n < u) ? to_f(W[(int64_t)kk * u + n]) : 0.0f;
    }
  };
  if (k_lo < k_hi) fetch(k_lo);
  for (int k0 = k_lo; k0 < k_hi; k0 += kTile) {  // u is a multiple of 4, not of the tile: blocks may straddle gates
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      Hs[ty + 8 * j][tx] = hreg[j];
      Ws[tx][ty + 8 * j] = wreg[j];
    }
    __syncthreads();
    if (k0 + kTile < k_hi) fetch(k0 + kTile);
#pragma unroll
    for (int kk = 0; kk < kTile; ++kk) {
      const double w = (double)Ws[tx][kk];
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[j] = fma(Hs[ty + 8 * j][kk], w, acc[j]);
    }
    __syncthreads();
  }
  if (kCluster && !tc::cluster_splitk_reduce(acc, red)) return;
  const int n = n0 + tx;
  if (n >= u) return;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int m = m0 + ty + 8 * j;
    if (m >= B) continue;
    const int64_t so = (int64_t)m * 2 * u + n;
    const double f = (double)to_f(fg[so]), ch = (double)to_f(c5[(int64_t)m * 5 * u + 4 * u + n]);
    const double gc = g_in[so], gh = g_in[so + u];
    const double vc = (delta ? (double)to_f(delta[so]) : 0.0) + f * (gc + gh * ch);
    const double vh = (delta ? (double)to_f(delta[so + u]) : 0.0) + acc[j];
    g_out[so] = vc;
    g_out[so + u] = vh;
    g_store[so] = from_f<T>((float)vc);
    g_store[so + u] = from_f<T>((float)vh);
  }
}

// The cell-state half of the block VJP (+ delta when given): uo[row][n] = f g_h c_h, n < u.  uo rows are 2u wide.
template <typename T>
__device__ __forceinline__ void write_uc(const T* g_row, const T* c5_row, const T* fg_row, const T* delta_row, T* uo_row,
                                         int u, int n) {
  float v = to_f(fg_row[n]) * to_f(g_row[u + n]) * to_f(c5_row[4 * u + n]);
  if (delta_row) v += to_f(delta_row[n]);
  uo_row[n] = from_f<T>(v);
}

// a4[row][k] = operand (in dtype) for the GEMMs that do not take the tf32 splits; optionally the u_c half.
// One block row per row of the operand, one thread per unit (its four columns are u apart).
template <typename T>
__global__ void __launch_bounds__(256) lstm_operand_kernel(const T* __restrict__ g, const T* __restrict__ c5,
                                                           const T* __restrict__ fg, const T* __restrict__ delta,
                                                           T* __restrict__ a4, T* __restrict__ uo, int u) {
  const int64_t row = blockIdx.x;
  const int n = blockIdx.y * blockDim.x + threadIdx.x;
  if (n >= u) return;
  const T* g_row = g + row * 2 * u;
  float v[4];
  operand_quad<T>(g_row, c5 + row * 5 * u, u, n, v);
#pragma unroll
  for (int q = 0; q < 4; ++q) a4[row * 4 * u + q * u + n] = from_f<T>(v[q]);
  if (uo) write_uc<T>(g_row, c5 + row * 5 * u, fg + row * 2 * u, delta ? delta + row * 2 * u : nullptr, uo + row * 2 * u, u, n);
}

// tf32 split of the operand as [rows][4u]; optionally the u_c half (float data)
__global__ void __launch_bounds__(256) lstm_split_kernel(const float* __restrict__ g, const float* __restrict__ c5,
                                                         const float* __restrict__ fg, const float* __restrict__ delta,
                                                         float* __restrict__ hi, float* __restrict__ lo,
                                                         float* __restrict__ uo, int u) {
  const int64_t row = blockIdx.x;
  const int n = blockIdx.y * blockDim.x + threadIdx.x;
  if (n >= u) return;
  const float* g_row = g + row * 2 * u;
  float v[4];
  operand_quad<float>(g_row, c5 + row * 5 * u, u, n, v);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const float h = round_tf32(v[q]);
    hi[row * 4 * u + q * u + n] = h;
    lo[row * 4 * u + q * u + n] = round_tf32(v[q] - h);
  }
  if (uo) write_uc<float>(g_row, c5 + row * 5 * u, fg + row * 2 * u, delta ? delta + row * 2 * u : nullptr, uo + row * 2 * u, u, n);
}

// the same operand written transposed, [4u][rows] (the weight-gradient GEMMs contract over rows)
__global__ void __launch_bounds__(256) lstm_split_transposed_kernel(const float* __restrict__ g, const float* __restrict__ c5,
                                                                    float* __restrict__ hiT, float* __restrict__ loT,
                                                                    int64_t rows, int u) {
  __shared__ float th[32][33], tl[32][33];
  const int64_t r0 = (int64_t)blockIdx.x * 32;
  const int c0 = blockIdx.y * 32;
  const int tx = threadIdx.x % 32, ty = threadIdx.x / 32;
  for (int i = ty; i < 32; i += 8) {
    const int64_t r = r0 + i;
    const int c = c0 + tx;
    float v = 0.0f;
    if (r < rows && c < 4 * u) v = operand_value<float, float, float>(g + r * 2 * u, c5 + r * 5 * u, u, c);
    const float h = round_tf32(v);
    th[i][tx] = h;
    tl[i][tx] = round_tf32(v - h);
  }
  __syncthreads();
  for (int i = ty; i < 32; i += 8) {
    const int c = c0 + i;
    const int64_t r = r0 + tx;
    if (c < 4 * u && r < rows) {
      hiT[(int64_t)c * rows + r] = th[tx][i];
      loT[(int64_t)c * rows + r] = tl[tx][i];
    }
  }
}

}  // namespace

void lstm_forward_step(Launcher& lc, int dtype, const void* W, const void* U, const void* x_t, const double* s_in,
                       double* s_out, void* fg, void* c5, void* state_out, int B, int u, int in_dim) {
  dim3 grid((u + kTile - 1) / kTile, (B + kTile - 1) / kTile);
  // at most two ways: a rank hands 16 partial sums per thread over, 32 KB of the leader's shared memory per peer
  const int ks = tc::cluster_split_for((int)(grid.x * grid.y), (int)grid.x, tc::sm_count(), 2, 4);
  const size_t smem = (size_t)(ks - 1) * 16 * 256 * sizeof(double);
  static PerDevice<bool> attr_done;  // per-device kernel attribute
  if (ks > 1 && !attr_done.here()) {
    cudaFuncSetAttribute(lstm_step_kernel<float, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 16 * 256 * (int)sizeof(double));
    cudaFuncSetAttribute(lstm_step_kernel<bf16, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 16 * 256 * (int)sizeof(double));
    attr_done.here() = true;
  }
  bool launched = false;
  if (ks > 1) {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr;
    tc::cluster_launch_config(cfg, attr, grid, ks, smem, lc.stream);
    cudaError_t e;
    if (dtype == HBP_F32) e = cudaLaunchKernelEx(&cfg, lstm_step_kernel<float, true>, (const float*)W, (const float*)U, (const float*)x_t, s_in, s_out,
                           (float*)fg, (float*)c5, (float*)state_out, B, u, in_dim);
    else e = cudaLaunchKernelEx(&cfg, lstm_step_kernel<bf16, true>, (const bf16*)W, (const bf16*)U, (const bf16*)x_t, s_in, s_out,
                           (bf16*)fg, (bf16*)c5, (bf16*)state_out, B, u, in_dim);
    launched = e == cudaSuccess;
    if (!launched) cudaGetLastError();  // clusters of this size cannot be placed here: run unsplit
  }
  if (!launched) {  // no cluster: the plain launch path is the cheaper one, and these launches are latency-bound
    if (dtype == HBP_F32) lstm_step_kernel<float, false><<<grid, 256, 0, lc.stream>>>((const float*)W, (const float*)U, (const float*)x_t, s_in, s_out,
                           (float*)fg, (float*)c5, (float*)state_out, B, u, in_dim);
    else lstm_step_kernel<bf16, false><<<grid, 256, 0, lc.stream>>>((const bf16*)W, (const bf16*)U, (const bf16*)x_t, s_in, s_out,
                           (bf16*)fg, (bf16*)c5, (bf16*)state_out, B, u, in_dim);
  }
  lc.count();
  lc.check();
}

void lstm_backward_step(Launcher& lc, int dtype, const void* W, const void* fg, const void* c5, const void* delta,
                        const double* g_in, double* g_out, void* g_store, int B, int u) {
  dim3 grid((u + kTile - 1) / kTile, (B + kTile - 1) / kTile);
  const int ks = tc::cluster_split_for((int)(grid.x * grid.y), (4 * u + kTile - 1) / kTile, tc::sm_count());
  bool launched = false;
  if (ks > 1) {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr;
    tc::cluster_launch_config(cfg, attr, grid, ks, 0, lc.stream);
    cudaError_t e;
    if (dtype == HBP_F32) e = cudaLaunchKernelEx(&cfg, lstm_bwd_step_kernel<float, true>, (const float*)W, (const float*)fg, (const float*)c5,
                           (const float*)delta, g_in, g_out, (float*)g_store, B, u);
    else e = cudaLaunchKernelEx(&cfg, lstm_bwd_step_kernel<bf16, true>, (const bf16*)W, (const bf16*)fg, (const bf16*)c5,
                           (const bf16*)delta, g_in, g_out, (bf16*)g_store, B, u);
    launched = e == cudaSuccess;
    if (!launched) cudaGetLastError();  // clusters of this size cannot be placed here: run unsplit
  }
  if (!launched) {  // no cluster: the plain launch path is the cheaper one, and these launches are latency-bound
    if (dtype == HBP_F32) lstm_bwd_step_kernel<float, false><<<grid, 256, 0, lc.stream>>>((const float*)W, (const float*)fg, (const float*)c5,
                           (const float*)delta, g_in, g_out, (float*)g_store, B, u);
    else lstm_bwd_step_kernel<bf16, false><<<grid, 256, 0, lc.stream>>>((const bf16*)W, (const bf16*)fg, (const bf16*)c5,
                           (const bf16*)delta, g_in, g_out, (bf16*)g_store, B, u);
  }
  lc.count();
  lc.check();
}

void lstm_operand(Launcher& lc, int dtype, const void* g, const void* c5, const void* fg, const void* delta, void* a4,
                  void* uo, int64_t rows, int u) {
  dim3 grid((unsigned)rows, (unsigned)((u + 255) / 256));
  if (dtype == HBP_F32)
    lstm_operand_kernel<float><<<grid, 256, 0, lc.stream>>>((const float*)g, (const float*)c5, (const float*)fg,
                                                            (const float*)delta, (float*)a4, (float*)uo, u);
  else
    lstm_operand_kernel<bf16><<<grid, 256, 0, lc.stream>>>((const bf16*)g, (const bf16*)c5, (const bf16*)fg,
                                                           (const bf16*)delta, (bf16*)a4, (bf16*)uo, u);
  lc.count();
  lc.check();
}

void lstm_split(Launcher& lc, const float* g, const float* c5, const float* fg, const float* delta, float* hi, float* lo,
                float* uo, int64_t rows, int u) {
  dim3 grid((unsigned)rows, (unsigned)((u + 255) / 256));
  lstm_split_kernel<<<grid, 256, 0, lc.stream>>>(g, c5, fg, delta, hi, lo, uo, u);
  lc.count();
  lc.check();
}

void lstm_split_transposed(Launcher& lc, const float* g, const float* c5, float* hiT, float* loT, int64_t rows, int u) {
  dim3 grid((unsigned)((rows + 31) / 32), (unsigned)((4 * u + 31) / 32));
  lstm_split_transposed_kernel<<<grid, 256, 0, lc.stream>>>(g, c5, hiT, loT, rows, u);
  lc.count();
  lc.check();
}

}  // namespace hbp
