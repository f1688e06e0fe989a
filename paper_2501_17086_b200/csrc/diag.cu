// Agreement between two gradient estimates (the quantities of the paper's Figure 5: cosine similarity between the
// Highway-BP estimate and the true gradient, and the norm of one iteration's step relative to the total): per
// segment the four sums <a,b>, |a|^2, |b|^2, |a-b|^2 in double, by a two-stage reduction in a fixed order
// (deterministic).  HBM-bound: each input is read once.
#include "hbp_internal.h"

namespace hbp {

namespace {

constexpr int kSlices = 64;  // blocks per segment

template <typename T>
__global__ void __launch_bounds__(256) compare_partial_kernel(const T* __restrict__ a, const T* __restrict__ b,
                                                              int64_t elems, double* __restrict__ partial) {
  __shared__ double red[8][4];
  const int seg = blockIdx.y, slice = blockIdx.x;
  const T* pa = a + (int64_t)seg * elems;
  const T* pb = b + (int64_t)seg * elems;
  const int64_t per = (elems + kSlices - 1) / kSlices;
  const int64_t lo = (int64_t)slice * per, hi = min(elems, lo + per);
  double s[4] = {0.0, 0.0, 0.0, 0.0};
  for (int64_t i = lo + threadIdx.x; i < hi; i += blockDim.x) {
    const float x = to_f(pa[i]), y = to_f(pb[i]), d = x - y;
    s[0] += (double)x * y;
    s[1] += (double)x * x;
    s[2] += (double)y * y;
    s[3] += (double)d * d;
  }
#pragma unroll
  for (int k = 0; k < 4; ++k)
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s[k] += __shfl_xor_sync(0xffffffffu, s[k], o);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0)
    for (int k = 0; k < 4; ++k) red[warp][k] = s[k];
  __syncthreads();
  if (threadIdx.x < 4) {
    double t = 0.0;
    for (int w = 0; w < 8; ++w) t += red[w][threadIdx.x];
    partial[((int64_t)seg * kSlices + slice) * 4 + threadIdx.x] = t;
  }
}

__global__ void compare_final_kernel(const double* __restrict__ partial, double* __restrict__ out, int segments) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= segments * 4) return;
  const int seg = i / 4, k = i % 4;
  double t = 0.0;
  for (int s = 0; s < kSlices; ++s) t += partial[((int64_t)seg * kSlices + s) * 4 + k];
  out[i] = t;
}

}  // namespace

size_t compare_scratch_bytes(int segments) { return (size_t)segments * kSlices * 4 * sizeof(double); }

void compare_segments(Launcher& lc, int dtype, const void* a, const void* b, int segments, int64_t elems, double* out,
                      double* scratch) {
  dim3 grid(kSlices, segments);
  if (dtype == HBP_F32) compare_partial_kernel<float><<<grid, 256, 0, lc.stream>>>((const float*)a, (const float*)b, elems, scratch);
  else compare_partial_kernel<bf16><<<grid, 256, 0, lc.stream>>>((const bf16*)a, (const bf16*)b, elems, scratch);
  compare_final_kernel<<<(segments * 4 + 127) / 128, 128, 0, lc.stream>>>(scratch, out, segments);
  lc.count(2);
  lc.check();
}

}  // namespace hbp
