// Reverse diagonal scan over depth or time (Eq. 9 / Eq. 12 with diagonal K) and the row-wise
// elementwise kernels around it.  All access is 128-bit and coalesced along the channel axis; the
// running value is kept in float and rounded only when stored.
#include "hbp_internal.h"

namespace hbp {

namespace {

template <typename T>
struct Vec;  // 16-byte vector of T
template <>
struct Vec<float> {
  static constexpr int N = 4;
  float4 raw;
  __device__ __forceinline__ void get(float* f) const { f[0] = raw.x; f[1] = raw.y; f[2] = raw.z; f[3] = raw.w; }
  __device__ __forceinline__ void set(const float* f) { raw = make_float4(f[0], f[1], f[2], f[3]); }
};
template <>
struct Vec<bf16> {
  static constexpr int N = 8;
  uint4 raw;
  __device__ __forceinline__ void get(float* f) const {
    const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float2 t = __bfloat1622float2(p[i]);
      f[2 * i] = t.x;
      f[2 * i + 1] = t.y;
    }
  }
  __device__ __forceinline__ void set(const float* f) {
    __nv_bfloat162* p = reinterpret_cast<__nv_bfloat162*>(&raw);
#pragma unroll
    for (int i = 0; i < 4; ++i) p[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
  }
};

template <typename T>
__device__ __forceinline__ Vec<T> ldv(const T* p) {
  Vec<T> v;
  v.raw = *reinterpret_cast<const decltype(v.raw)*>(p);
  return v;
}
template <typename T>
__device__ __forceinline__ Vec<T> ldv_stream(const T* p) {  // read-once data: evict first
  Vec<T> v;
  v.raw = __ldcs(reinterpret_cast<const decltype(v.raw)*>(p));
  return v;
}
template <typename T>
__device__ __forceinline__ void stv(T* p, const Vec<T>& v) {
  *reinterpret_cast<decltype(v.raw)*>(p) = v.raw;
}

// delta pointer for state l (nullptr = zero)
template <typename T>
__device__ __forceinline__ const T* delta_at(const ScanArgs& s, int l, int64_t state_elems) {
  if (!s.delta) return nullptr;
  if (s.loss == HBP_LOSS_EVERY_STEP) return (const T*)s.delta + (int64_t)l * state_elems;
  return (l == s.L) ? (const T*)s.delta : nullptr;
}
template <typename T>
__device__ __forceinline__ const T* gate_at(const ScanArgs& s, int l) {
  if (s.gate == HBP_GATE_ONE || !s.a) return nullptr;
  return (const T*)s.a + (s.gate == HBP_GATE_CHANNEL_PER_STEP ? (int64_t)l * s.d : 0);
}

// One step of the recurrence for a 16-byte channel group: val = a * carry + u + delta.
template <typename T>
__device__ __forceinline__ void scan_step(const ScanArgs& s, int l, int64_t state_elems, int64_t off, int ch,
                                          const float* carry, float* val) {
  constexpr int V = Vec<T>::N;
  const T* gp = gate_at<T>(s, l);
  if (gp) {
    float a[V];
    ldv<T>(gp + ch).get(a);
#pragma unroll
    for (int i = 0; i < V; ++i) val[i] = a[i] * carry[i];
  } else {
#pragma unroll
    for (int i = 0; i < V; ++i) val[i] = carry[i];
  }
  if (s.u) {
    float u[V];
    ldv_stream<T>((const T*)s.u + (int64_t)l * state_elems + off).get(u);
#pragma unroll
    for (int i = 0; i < V; ++i) val[i] += u[i];
  }
  const T* dp = delta_at<T>(s, l, state_elems);
  if (dp) {
    float dl[V];
    ldv_stream<T>(dp + off).get(dl);
#pragma unroll
    for (int i = 0; i < V; ++i) val[i] += dl[i];
  }
}

// ---- depth scan, no LayerNorm: one thread per 16-byte channel group, serial over l -----------------
template <typename T>
__global__ void __launch_bounds__(256) scan_depth_kernel(const ScanArgs s) {
  constexpr int V = Vec<T>::N;
  const int64_t state_elems = s.rows * s.d;
  const int64_t nvec = state_elems / V;
  const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (v >= nvec) return;
  const int64_t off = v * V;
  const int ch = (int)(off % s.d);
  T* g = (T*)s.g;
  float carry[V];
  ldv<T>(g + (int64_t)s.l_hi * state_elems + off).get(carry);
  for (int l = s.l_hi - 1; l >= s.l_lo; --l) {
    float val[V];
    scan_step<T>(s, l, state_elems, off, ch, carry, val);
    Vec<T> out;
    out.set(val);
    stv<T>(g + (int64_t)l * state_elems + off, out);
#pragma unroll
    for (int i = 0; i < V; ++i) carry[i] = val[i];
  }
}

// ---- depth scan with the LayerNorm-backward finish: one block per row ------------------------------
// u holds dY = dL/d(LN(x)); the step's VJP is rstd * (dy - mean(dy) - xhat * mean(dy * xhat)).
template <typename T>
__global__ void __launch_bounds__(1024) scan_depth_ln_kernel(const ScanArgs s) {
  constexpr int V = Vec<T>::N;
  __shared__ float red[2][32][2];
  const int64_t row = blockIdx.x;
  const int tpr = s.d / V;
  const bool active = (int)threadIdx.x < tpr;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
  const int64_t state_elems = s.rows * s.d;
  const int64_t off = row * s.d + (int64_t)threadIdx.x * V;
  T* g = (T*)s.g;
  float carry[V], dy[V], xh[V];
#pragma unroll
  for (int i = 0; i < V; ++i) carry[i] = dy[i] = xh[i] = 0.0f;
  if (active) {
    ldv<T>(g + (int64_t)s.l_hi * state_elems + off).get(carry);
    ldv_stream<T>((const T*)s.u + (int64_t)(s.l_hi - 1) * state_elems + off).get(dy);
    ldv_stream<T>((const T*)s.xhat + (int64_t)(s.l_hi - 1) * state_elems + off).get(xh);
  }
  const float inv_d = 1.0f / (float)s.d;
  for (int l = s.l_hi - 1; l >= s.l_lo; --l) {
    float s1 = 0.0f, s2 = 0.0f;
#pragma unroll
    for (int i = 0; i < V; ++i) {
      s1 += dy[i];
      s2 = fmaf(dy[i], xh[i], s2);
    }
    // fetch the next step's operands before waiting on the reduction
    float ndy[V], nxh[V];
#pragma unroll
    for (int i = 0; i < V; ++i) ndy[i] = nxh[i] = 0.0f;
    if (active && l > s.l_lo) {
      ldv_stream<T>((const T*)s.u + (int64_t)(l - 1) * state_elems + off).get(ndy);
      ldv_stream<T>((const T*)s.xhat + (int64_t)(l - 1) * state_elems + off).get(nxh);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      s1 += __shfl_xor_sync(0xffffffffu, s1, o);
      s2 += __shfl_xor_sync(0xffffffffu, s2, o);
    }
    const int buf = l & 1;  // two buffers: one barrier per step is enough
    if (lane == 0) {
      red[buf][warp][0] = s1;
      red[buf][warp][1] = s2;
    }
    __syncthreads();
    float t1 = 0.0f, t2 = 0.0f;
    for (int w = 0; w < nwarps; ++w) {
      t1 += red[buf][w][0];
      t2 += red[buf][w][1];
    }
    const float m1 = t1 * inv_d, m2 = t2 * inv_d;
    const float r = s.rstd[(int64_t)l * s.rows + row];
    if (active) {
      float val[V];
      const T* gp = gate_at<T>(s, l);
      if (gp) {
        float a[V];
        ldv<T>(gp + threadIdx.x * V).get(a);
#pragma unroll
        for (int i = 0; i < V; ++i) val[i] = a[i] * carry[i];
      } else {
#pragma unroll
        for (int i = 0; i < V; ++i) val[i] = carry[i];
      }
#pragma unroll
      for (int i = 0; i < V; ++i) val[i] += r * (dy[i] - m1 - xh[i] * m2);
      const T* dp = delta_at<T>(s, l, state_elems);
      if (dp) {
        float dl[V];
        ldv_stream<T>(dp + off).get(dl);
#pragma unroll
        for (int i = 0; i < V; ++i) val[i] += dl[i];
      }
      Vec<T> out;
      out.set(val);
      stv<T>(g + (int64_t)l * state_elems + off, out);
#pragma unroll
      for (int i = 0; i < V; ++i) carry[i] = val[i];
    }
#pragma unroll
    for (int i = 0; i < V; ++i) {
      dy[i] = ndy[i];
      xh[i] = nxh[i];
    }
  }
}
