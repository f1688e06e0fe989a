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

template <typename T>
__global__ void to_f64_kernel(const T* __restrict__ src, double* __restrict__ dst, int64_t n) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = (double)to_f(src[i]);
}

}  // namespace

void rnn_forward_step(Launcher& lc, int dtype, const void* W, const void* U, const void* x_t, const void* gate,
                      const double* h_in, double* h_out, void* deriv, void* state_out, int B, int d, int in_dim) {
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
