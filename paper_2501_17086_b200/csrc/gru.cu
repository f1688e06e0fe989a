// GRU cell as a residual step with a state-dependent gate (Table 1, row "GRU"):
//     r = sigmoid(U_r x_t + W_r h),  z = sigmoid(U_z x_t + W_z h),  n = tanh(U_n x_t + r * (W_n h)),
//     h' = z * h + (1 - z) * n,
// so K = diag(z) is the cheap Jacobian and J^T g = (g * [c_r | c_z | c_nr]) W is the block VJP, with the
// per-element coefficients
//     c_n  = (1 - z)(1 - n^2)        (dLoss/d(pre-activation of n) per unit of g)
//     c_z  = (h - n) z (1 - z)
//     c_r  = c_n * (W_n h) * r (1 - r)
//     c_nr = c_n * r
// which the forward step computes once, in double, from the pre-activations (no cancellation near saturated
// gates) and stores as C4 = [c_r | c_z | c_nr | c_n] per row.  The input-weight gradient uses
// [c_r | c_z | c_n] instead of the first three.  Like the tanh RNN, the recurrence itself and exact
// backpropagation through time are carried in double beside the stored values.
#include "cluster_split.cuh"

namespace hbp {

namespace {

constexpr int kTile = 32;

// acc[gate][j] += sum_k src[m_j][k] * Wm[gate * d + n][k] over k in [k_lo, k_hi) (k_lo a multiple of the tile)
template <typename T, bool kSrcDouble>
__device__ __forceinline__ void gru_accumulate(const void* __restrict__ src, const T* __restrict__ Wm, int kdim, int B,
                                               int d, int m0, int n0, double (*Hs)[kTile + 1],
                                               float (*Ws)[kTile][kTile + 1], double (*acc)[4], int k_lo, int k_hi) {
  if (k_lo >= k_hi) return;
  const int tx = threadIdx.x % kTile, ty = threadIdx.x / kTile;
  // The next tile's global loads are issued into registers before the current tile is multiplied, so the loop
  // waits for memory once, not once per tile.
  double hreg[4];
  float wreg[3][4];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int i = ty + 8 * j;
      const int k = k0 + tx, m = m0 + i, n = n0 + i;
      double hv = 0.0;
      if (k < kdim && m < B)
        hv = kSrcDouble ? ((const double*)src)[(int64_t)m * kdim + k] : (double)to_f(((const T*)src)[(int64_t)m * kdim + k]);
      hreg[j] = hv;
#pragma unroll
      for (int q = 0; q < 3; ++q) wreg[q][j] = (k < kdim && n < d) ? to_f(Wm[((int64_t)q * d + n) * kdim + k]) : 0.0f;
    }
  };
  fetch(k_lo);
  for (int k0 = k_lo; k0 < k_hi; k0 += kTile) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int i = ty + 8 * j;
      Hs[i][tx] = hreg[j];
#pragma unroll
      for (int q = 0; q < 3; ++q) Ws[q][i][tx] = wreg[q][j];
    }
    __syncthreads();
    if (k0 + kTile < k_hi) fetch(k0 + kTile);
#pragma unroll 8
    for (int kk = 0; kk < kTile; ++kk) {
      double w[3];
#pragma unroll
      for (int q = 0; q < 3; ++q) w[q] = (double)Ws[q][tx][kk];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const double hv = Hs[ty + 8 * j][kk];
#pragma unroll
        for (int q = 0; q < 3; ++q) acc[q][j] = fma(hv, w[q], acc[q][j]);
      }
    }
    __syncthreads();
  }
}

__device__ __forceinline__ double sigmoid_d(double v) { return 1.0 / (1.0 + exp(-v)); }

template <typename T, bool kCluster>
__global__ void __launch_bounds__(256) gru_step_kernel(const T* __restrict__ W, const T* __restrict__ U,
                                                       const T* __restrict__ x_t, const double* __restrict__ h_in,
                                                       double* __restrict__ h_out, T* __restrict__ zc,
                                                       T* __restrict__ c4, T* __restrict__ state_out, int B, int d,
                                                       int in_dim) {
  __shared__ double Hs[kTile][kTile + 1];
  __shared__ float Ws[3][kTile][kTile + 1];
  extern __shared__ double red[];  // partial sums of the cluster's other ranks (see cluster_splitk_reduce)
  const int tx = threadIdx.x % kTile, ty = threadIdx.x / kTile;
  const int n0 = blockIdx.x * kTile, m0 = blockIdx.y * kTile;
  double acc[24];  // [rec | pre][gate][row]
#pragma unroll
  for (int i = 0; i < 24; ++i) acc[i] = 0.0;
  double (*rec)[4] = reinterpret_cast<double (*)[4]>(acc);
  double (*pre)[4] = reinterpret_cast<double (*)[4]>(acc + 12);
  // the previous state of this thread's outputs, fetched before the products so that the epilogue does not wait for it
  double hprev[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int m = m0 + ty + 8 * j, n = n0 + tx;
    hprev[j] = (m < B && n < d) ? h_in[(int64_t)m * d + n] : 0.0;
  }
  // the CTAs of a cluster share the k-tiles of both products out and add their partial sums
  // (a kernel that reads the cluster registers is launched as a cluster even alone, which costs microseconds per launch:
  // the form without a split does not touch them)
  const int ks = kCluster ? (int)tc::cluster_nctarank() : 1, rank = kCluster ? (int)tc::cluster_ctarank() : 0;
  const int nt_h = (d + kTile - 1) / kTile, nt_x = (in_dim + kTile - 1) / kTile;
  gru_accumulate<T, true>(h_in, W, d, B, d, m0, n0, Hs, Ws, rec, (nt_h * rank / ks) * kTile,
                          min(d, (nt_h * (rank + 1) / ks) * kTile));
  gru_accumulate<T, false>(x_t, U, in_dim, B, d, m0, n0, Hs, Ws, pre, (nt_x * rank / ks) * kTile,
                           min(in_dim, (nt_x * (rank + 1) / ks) * kTile));
  if (kCluster && !tc::cluster_splitk_reduce(acc, red)) return;
  const int n = n0 + tx;
  if (n >= d) return;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int m = m0 + ty + 8 * j;
    if (m >= B) continue;
    const int64_t idx = (int64_t)m * d + n;
    const double ar = pre[0][j] + rec[0][j], az = pre[1][j] + rec[1][j];
    const double r = sigmoid_d(ar), r1 = sigmoid_d(-ar);  // r and 1 - r
    const double z = sigmoid_d(az), z1 = sigmoid_d(-az);
    const double an = pre[2][j] + r * rec[2][j];
    const double e = exp(-2.0 * fabs(an));
    const double nn = copysign((1.0 - e) / (1.0 + e), an);
    const double dn = 4.0 * e / ((1.0 + e) * (1.0 + e));  // 1 - tanh(an)^2
    const double h = hprev[j];
    const double hn = z * h + z1 * nn;
    const double cn = z1 * dn;
    h_out[idx] = hn;
    state_out[idx] = from_f<T>((float)hn);
    zc[idx] = from_f<T>((float)z);
    T* c = c4 + (int64_t)m * 4 * d + n;
    c[0] = from_f<T>((float)(cn * rec[2][j] * r * r1));
    c[d] = from_f<T>((float)((h - nn) * z * z1));
    c[2 * d] = from_f<T>((float)(cn * r));
    c[3 * d] = from_f<T>((float)cn);
  }
}

// Exact backpropagation through one GRU step in double:
//     g_t = delta_t + z_t * g_{t+1} + (g_{t+1} * [c_r | c_z | c_nr]) W.
template <typename T, bool kCluster>
__global__ void __launch_bounds__(256) gru_bwd_step_kernel(const T* __restrict__ W, const T* __restrict__ zc,
                                                           const T* __restrict__ c4, const T* __restrict__ delta,
                                                           const double* __restrict__ g_in, double* __restrict__ g_out,
                                                           T* __restrict__ g_store, int B, int d) {
  __shared__ double Hs[kTile][kTile + 1];
  __shared__ float Ws[kTile][kTile + 1];
  __shared__ double red[(tc::kMaxClusterSplit - 1) * 4 * 256];
  const int tx = threadIdx.x % kTile, ty = threadIdx.x / kTile;
  const int n0 = blockIdx.x * kTile, m0 = blockIdx.y * kTile;
  double acc[4] = {0.0, 0.0, 0.0, 0.0};
  // the next tile's operands are fetched into registers before the current tile is multiplied; tiles are numbered
  // through the three gate blocks.  The CTAs of a cluster share the tiles out (one step has too few output tiles to
  // fill the GPU) and add their partial sums at the end.
  const int tiles_per_gate = (d + kTile - 1) / kTile, ntiles = 3 * tiles_per_gate;
  // (a kernel that reads the cluster registers is launched as a cluster even alone, which costs microseconds per launch:
  // the form without a split does not touch them)
  const int ks = kCluster ? (int)tc::cluster_nctarank() : 1, rank = kCluster ? (int)tc::cluster_ctarank() : 0;
  const int t_lo = ntiles * rank / ks, t_hi = ntiles * (rank + 1) / ks;
  double hreg[4];
  float wreg[4];
  auto fetch = [&](int t) {
    const int q = t / tiles_per_gate, k0 = (t - q * tiles_per_gate) * kTile;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int i = ty + 8 * j;
      const int m = m0 + i, k = k0 + tx;
      hreg[j] = (m < B && k < d) ? g_in[(int64_t)m * d + k] * (double)to_f(c4[(int64_t)m * 4 * d + (int64_t)q * d + k]) : 0.0;
      const int kk = k0 + i, n = n0 + tx;  // W[q*d + k][n]: contiguous in n
      wreg[j] = (kk < d && n < d) ? to_f(W[((int64_t)q * d + kk) * d + n]) : 0.0f;
    }
  };
  if (t_lo < t_hi) fetch(t_lo);
  {
    for (int t = t_lo; t < t_hi; ++t) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        Hs[ty + 8 * j][tx] = hreg[j];
        Ws[tx][ty + 8 * j] = wreg[j];
      }
      __syncthreads();
      if (t + 1 < t_hi) fetch(t + 1);
#pragma unroll
      for (int kk = 0; kk < kTile; ++kk) {
        const double w = (double)Ws[tx][kk];
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[j] = fma(Hs[ty + 8 * j][kk], w, acc[j]);
      }
      __syncthreads();
    }
  }
  if (kCluster && !tc::cluster_splitk_reduce(acc, red)) return;
  const int n = n0 + tx;
  if (n >= d) return;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int m = m0 + ty + 8 * j;
    if (m >= B) continue;
    const int64_t idx = (int64_t)m * d + n;
    const double v = (delta ? (double)to_f(delta[idx]) : 0.0) + (double)to_f(zc[idx]) * g_in[idx] + acc[j];
    g_out[idx] = v;
    g_store[idx] = from_f<T>((float)v);
  }
}

// a4[row][q*d + c] = g[row][c] * c4[row][q*d + c] for q = 0..3 (the operand of the CUDA-core GEMMs).
template <typename T>
__global__ void gru_operand_kernel(const T* __restrict__ g, const T* __restrict__ c4, T* __restrict__ a4, int64_t rows,
                                   int d) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= rows * 4 * d) return;
  const int64_t row = i / (4 * d);
  const int c = (int)(i % d);
  a4[i] = from_f<T>(to_f(g[row * d + c]) * to_f(c4[i]));
}

// tf32 split of g * [c_r | c_z | c_nr] as [rows][3d] (the VJP's A operand, contraction index contiguous)
__global__ void gru_split_kernel(const float* __restrict__ g, const float* __restrict__ c4, float4* __restrict__ hi,
                                 float4* __restrict__ lo, int64_t rows, int d) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;  // one float4 of the [rows][3d] output
  const int vrow = 3 * d / 4;
  if (i >= rows * vrow) return;
  const int64_t row = i / vrow;
  const int col = (int)(i % vrow) * 4;  // column in [0, 3d); never straddles a block since d % 4 == 0
  const float4 gv = *reinterpret_cast<const float4*>(g + row * d + col % d);
  const float4 cv = *reinterpret_cast<const float4*>(c4 + row * 4 * d + col);
  const float v[4] = {gv.x * cv.x, gv.y * cv.y, gv.z * cv.z, gv.w * cv.w};
  float h[4], l[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    h[k] = round_tf32(v[k]);
    l[k] = round_tf32(v[k] - h[k]);
  }
  hi[i] = make_float4(h[0], h[1], h[2], h[3]);
  lo[i] = make_float4(l[0], l[1], l[2], l[3]);
}

// tf32 split of g * C4 written transposed, [4d][rows] (the weight-gradient GEMMs contract over rows)
__global__ void __launch_bounds__(256) gru_split_transposed_kernel(const float* __restrict__ g,
                                                                   const float* __restrict__ c4, float* __restrict__ hiT,
                                                                   float* __restrict__ loT, int64_t rows, int d) {
  __shared__ float th[32][33], tl[32][33];
  const int64_t r0 = (int64_t)blockIdx.x * 32;
  const int c0 = blockIdx.y * 32;  // column of C4 in [0, 4d)
  const int tx = threadIdx.x % 32, ty = threadIdx.x / 32;
  for (int i = ty; i < 32; i += 8) {
    const int64_t r = r0 + i;
    const int c = c0 + tx;
    float v = 0.0f;
    if (r < rows && c < 4 * d) v = g[r * d + c % d] * c4[r * 4 * d + c];
    const float h = round_tf32(v);
    th[i][tx] = h;
    tl[i][tx] = round_tf32(v - h);
  }
  __syncthreads();
  for (int i = ty; i < 32; i += 8) {
    const int c = c0 + i;
    const int64_t r = r0 + tx;
    if (c < 4 * d && r < rows) {
      hiT[(int64_t)c * rows + r] = th[tx][i];
      loT[(int64_t)c * rows + r] = tl[tx][i];
    }
  }
}

}  // namespace

void gru_forward_step(Launcher& lc, int dtype, const void* W, const void* U, const void* x_t, const double* h_in,
                      double* h_out, void* zc, void* c4, void* state_out, int B, int d, int in_dim) {
  dim3 grid((d + kTile - 1) / kTile, (B + kTile - 1) / kTile);
  // at most two ways: a rank hands 24 partial sums per thread over, 48 KB of the leader's shared memory per peer
  const int ks = tc::cluster_split_for((int)(grid.x * grid.y), (int)grid.x, tc::sm_count(), 2, 4);
  const size_t smem = (size_t)(ks - 1) * 24 * 256 * sizeof(double);
  static PerDevice<bool> attr_done;  // per-device kernel attribute
  if (ks > 1 && !attr_done.here()) {
    cudaFuncSetAttribute(gru_step_kernel<float, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 24 * 256 * (int)sizeof(double));
    cudaFuncSetAttribute(gru_step_kernel<bf16, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 24 * 256 * (int)sizeof(double));
    attr_done.here() = true;
  }
  bool launched = false;
  if (ks > 1) {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr;
    tc::cluster_launch_config(cfg, attr, grid, ks, smem, lc.stream);
    cudaError_t e;
    if (dtype == HBP_F32) e = cudaLaunchKernelEx(&cfg, gru_step_kernel<float, true>, (const float*)W, (const float*)U, (const float*)x_t, h_in, h_out,
                           (float*)zc, (float*)c4, (float*)state_out, B, d, in_dim);
    else e = cudaLaunchKernelEx(&cfg, gru_step_kernel<bf16, true>, (const bf16*)W, (const bf16*)U, (const bf16*)x_t, h_in, h_out,
                           (bf16*)zc, (bf16*)c4, (bf16*)state_out, B, d, in_dim);
    launched = e == cudaSuccess;
    if (!launched) cudaGetLastError();  // clusters of this size cannot be placed here: run unsplit
  }
  if (!launched) {  // no cluster: the plain launch path is the cheaper one, and these launches are latency-bound
    if (dtype == HBP_F32) gru_step_kernel<float, false><<<grid, 256, 0, lc.stream>>>((const float*)W, (const float*)U, (const float*)x_t, h_in, h_out,
                           (float*)zc, (float*)c4, (float*)state_out, B, d, in_dim);
    else gru_step_kernel<bf16, false><<<grid, 256, 0, lc.stream>>>((const bf16*)W, (const bf16*)U, (const bf16*)x_t, h_in, h_out,
                           (bf16*)zc, (bf16*)c4, (bf16*)state_out, B, d, in_dim);
  }
  lc.count();
  lc.check();
}

void gru_backward_step(Launcher& lc, int dtype, const void* W, const void* zc, const void* c4, const void* delta,
                       const double* g_in, double* g_out, void* g_store, int B, int d) {
  dim3 grid((d + kTile - 1) / kTile, (B + kTile - 1) / kTile);
  const int ks = tc::cluster_split_for((int)(grid.x * grid.y), 3 * (int)grid.x, tc::sm_count());
  bool launched = false;
  if (ks > 1) {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr;
    tc::cluster_launch_config(cfg, attr, grid, ks, 0, lc.stream);
    cudaError_t e;
    if (dtype == HBP_F32) e = cudaLaunchKernelEx(&cfg, gru_bwd_step_kernel<float, true>, (const float*)W, (const float*)zc, (const float*)c4,
                           (const float*)delta, g_in, g_out, (float*)g_store, B, d);
    else e = cudaLaunchKernelEx(&cfg, gru_bwd_step_kernel<bf16, true>, (const bf16*)W, (const bf16*)zc, (const bf16*)c4,
                           (const bf16*)delta, g_in, g_out, (bf16*)g_store, B, d);
    launched = e == cudaSuccess;
    if (!launched) cudaGetLastError();  // clusters of this size cannot be placed here: run unsplit
  }
  if (!launched) {  // no cluster: the plain launch path is the cheaper one, and these launches are latency-bound
    if (dtype == HBP_F32) gru_bwd_step_kernel<float, false><<<grid, 256, 0, lc.stream>>>((const float*)W, (const float*)zc, (const float*)c4,
                           (const float*)delta, g_in, g_out, (float*)g_store, B, d);
    else gru_bwd_step_kernel<bf16, false><<<grid, 256, 0, lc.stream>>>((const bf16*)W, (const bf16*)zc, (const bf16*)c4,
                           (const bf16*)delta, g_in, g_out, (bf16*)g_store, B, d);
  }
  lc.count();
  lc.check();
}

void gru_operand(Launcher& lc, int dtype, const void* g, const void* c4, void* a4, int64_t rows, int d) {
  const int64_t n = rows * 4 * d;
  const unsigned grid = (unsigned)((n + 255) / 256);
  if (dtype == HBP_F32) gru_operand_kernel<float><<<grid, 256, 0, lc.stream>>>((const float*)g, (const float*)c4, (float*)a4, rows, d);
  else gru_operand_kernel<bf16><<<grid, 256, 0, lc.stream>>>((const bf16*)g, (const bf16*)c4, (bf16*)a4, rows, d);
  lc.count();
  lc.check();
}

void gru_split(Launcher& lc, const float* g, const float* c4, float* hi, float* lo, int64_t rows, int d) {
  const int64_t nvec = rows * (3 * d / 4);
  gru_split_kernel<<<(unsigned)((nvec + 255) / 256), 256, 0, lc.stream>>>(g, c4, (float4*)hi, (float4*)lo, rows, d);
  lc.count();
  lc.check();
}

void gru_split_transposed(Launcher& lc, const float* g, const float* c4, float* hiT, float* loT, int64_t rows, int d) {
  dim3 grid((unsigned)((rows + 31) / 32), (unsigned)((4 * d + 31) / 32));
  gru_split_transposed_kernel<<<grid, 256, 0, lc.stream>>>(g, c4, hiT, loT, rows, d);
  lc.count();
  lc.check();
}

}  // namespace hbp
