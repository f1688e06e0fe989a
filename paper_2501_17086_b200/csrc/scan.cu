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
  template <typename F>
  __device__ __forceinline__ void get(F* f) const { f[0] = raw.x; f[1] = raw.y; f[2] = raw.z; f[3] = raw.w; }
  template <typename F>
  __device__ __forceinline__ void set(const F* f) { raw = make_float4((float)f[0], (float)f[1], (float)f[2], (float)f[3]); }
};
template <>
struct Vec<bf16> {
  static constexpr int N = 8;
  uint4 raw;
  template <typename F>
  __device__ __forceinline__ void get(F* f) const {
    const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float2 t = __bfloat1622float2(p[i]);
      f[2 * i] = t.x;
      f[2 * i + 1] = t.y;
    }
  }
  template <typename F>
  __device__ __forceinline__ void set(const F* f) {
    __nv_bfloat162* p = reinterpret_cast<__nv_bfloat162*>(&raw);
#pragma unroll
    for (int i = 0; i < 4; ++i) p[i] = __floats2bfloat162_rn((float)f[2 * i], (float)f[2 * i + 1]);
  }
};

// The running value of the recurrence: double for float data (thousands of steps must stay within 1e-5 of
// an exact evaluation), float for bf16 data.
template <typename T>
struct Acc {
  typedef float type;
};
template <>
struct Acc<float> {
  typedef double type;
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
  if (s.loss == HBP_LOSS_EVERY_STEP) return (s.u_has_delta && l < s.L) ? nullptr : (const T*)s.delta + (int64_t)l * state_elems;
  return (l == s.L) ? (const T*)s.delta : nullptr;
}
// gate vector of step l for the 16-byte group at element `off` of the state, channel `ch` (nullptr = ones)
template <typename T>
__device__ __forceinline__ const T* gate_at(const ScanArgs& s, int l, int64_t state_elems, int64_t off, int ch) {
  if (s.gate == HBP_GATE_ONE || s.gate == kGateRow || !s.a) return nullptr;
  if (s.gate == kGateElement) return (const T*)s.a + (int64_t)l * state_elems + off;
  return (const T*)s.a + (s.gate == HBP_GATE_CHANNEL_PER_STEP ? (int64_t)l * s.d : 0) + ch;
}

// One step of the recurrence for a 16-byte channel group: val = a * carry + u + delta.
template <typename T>
__device__ __forceinline__ void scan_step(const ScanArgs& s, int l, int64_t state_elems, int64_t off, int ch,
                                          const typename Acc<T>::type* carry, typename Acc<T>::type* val,
                                          int64_t row = 0) {
  constexpr int V = Vec<T>::N;
  const T* gp = gate_at<T>(s, l, state_elems, off, ch);
  if (s.gate == kGateRow) {  // one gate value per row and step (a float table [L][rows])
    const float a = s.keep * __ldg(s.row_gate + (int64_t)l * s.rows + row);
#pragma unroll
    for (int i = 0; i < V; ++i) val[i] = a * carry[i];
  } else if (gp) {
    float a[V];
    ldv<T>(gp).get(a);
#pragma unroll
    for (int i = 0; i < V; ++i) val[i] = a[i] * carry[i];
  } else {
#pragma unroll
    for (int i = 0; i < V; ++i) val[i] = s.keep * carry[i];
  }
  if (s.u2) {
    float w[V];
    ldv_stream<T>((const T*)s.u2 + (int64_t)l * state_elems + off).get(w);
#pragma unroll
    for (int i = 0; i < V; ++i) val[i] += w[i];
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
// kShift: the shifted split (gamma > 0), which also reads the previous iterate; compiled apart so that the plain
// scan carries no registers for it
template <typename T, bool kShift>
__global__ void __launch_bounds__(256) scan_depth_kernel(const ScanArgs s) {
  constexpr int V = Vec<T>::N;
  const int64_t state_elems = s.rows * s.d;
  const int64_t nvec = state_elems / V;
  const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (v >= nvec) return;
  const int64_t off = v * V;
  const int64_t row = off / s.d;  // once per thread: the per-row gate of post-LN layers is looked up by it
  const int ch = (int)(off - row * s.d);
  T* g = (T*)s.g;
  typedef typename Acc<T>::type A;
  A carry[V];
  ldv<T>(g + (int64_t)s.l_hi * state_elems + off).get(carry);
  float old_next[kShift ? V : 1];  // shifted split: g_{l+1} of the previous iterate
  if (kShift) {
#pragma unroll
    for (int i = 0; i < V; ++i) old_next[i] = (float)carry[i];
  }
#pragma unroll 4
  for (int l = s.l_hi - 1; l >= s.l_lo; --l) {  // unrolled: the loads of four steps in flight per thread
    A val[V];
    scan_step<T>(s, l, state_elems, off, ch, carry, val, row);
    if (kShift) {
      // the shifted part of the split acts on the previous iterate: gamma * a * g_{l+1} (a = 1 unless the gate is per row)
      const float ga = s.gate == kGateRow ? s.gamma * __ldg(s.row_gate + (int64_t)l * s.rows + row) : s.gamma;
#pragma unroll
      for (int i = 0; i < V; ++i) val[i] += ga * old_next[i];
      ldv<T>(g + (int64_t)l * state_elems + off).get(old_next);  // before it is overwritten below
    }
    Vec<T> out;
    out.set(val);
    stv<T>(g + (int64_t)l * state_elems + off, out);
#pragma unroll
    for (int i = 0; i < V; ++i) carry[i] = val[i];
  }
}

// ---- depth scan with the LayerNorm-backward finish from prepared row statistics ---------------------
// Same streaming form as above: lnstat[l][row] = {rstd, mean(dy), mean(dy * xhat)} comes from the GEMM that
// produced dy, so no reduction is needed here.  u holds dy, the VJP is rstd * (dy - m1 - xhat * m2).
template <typename T, bool kShift>
__global__ void __launch_bounds__(256) scan_depth_lnstat_kernel(const ScanArgs s) {
  constexpr int V = Vec<T>::N;
  const int64_t state_elems = s.rows * s.d;
  const int64_t nvec = state_elems / V;
  const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (v >= nvec) return;
  const int64_t off = v * V;
  const int64_t row = off / s.d;
  const int ch = (int)(off - row * s.d);
  T* g = (T*)s.g;
  float carry[V], old_next[kShift ? V : 1];
  ldv<T>(g + (int64_t)s.l_hi * state_elems + off).get(carry);
  if (kShift) {
#pragma unroll
    for (int i = 0; i < V; ++i) old_next[i] = carry[i];
  }
  // the loads of a step do not depend on the running value: unrolled, those of four steps are in flight per thread
#pragma unroll 4
  for (int l = s.l_hi - 1; l >= s.l_lo; --l) {
    float dy[V], xh[V], val[V];
    ldv_stream<T>((const T*)s.u + (int64_t)l * state_elems + off).get(dy);
    ldv_stream<T>((const T*)s.xhat + (int64_t)l * state_elems + off).get(xh);
    const float4 st = __ldg(s.lnstat + (int64_t)l * s.rows + row);
    const T* gp = gate_at<T>(s, l, state_elems, off, ch);
    if (gp) {
      float a[V];
      ldv<T>(gp).get(a);
#pragma unroll
      for (int i = 0; i < V; ++i) val[i] = a[i] * carry[i];
    } else {
#pragma unroll
      for (int i = 0; i < V; ++i) val[i] = s.keep * carry[i];
    }
#pragma unroll
    for (int i = 0; i < V; ++i) val[i] += st.x * (dy[i] - st.y - xh[i] * st.z);
    if (kShift) {
#pragma unroll
      for (int i = 0; i < V; ++i) val[i] += s.gamma * old_next[i];
      ldv<T>(g + (int64_t)l * state_elems + off).get(old_next);
    }
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
}

__global__ void ln_stats_finish_kernel(const float2* __restrict__ stats, int slots, const float* __restrict__ rstd,
                                       float4* __restrict__ lnstat, int64_t count, float inv_d) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= count) return;
  float s1 = 0.0f, s2 = 0.0f;
  for (int k = 0; k < slots; ++k) {  // fixed order: deterministic
    const float2 t = stats[i * slots + k];
    s1 += t.x;
    s2 += t.y;
  }
  lnstat[i] = make_float4(rstd[i], s1 * inv_d, s2 * inv_d, 0.0f);
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
  float carry[V], dy[V], xh[V], old_next[V];
#pragma unroll
  for (int i = 0; i < V; ++i) carry[i] = dy[i] = xh[i] = old_next[i] = 0.0f;
  if (active) {
    ldv<T>(g + (int64_t)s.l_hi * state_elems + off).get(carry);
    ldv<T>(g + (int64_t)s.l_hi * state_elems + off).get(old_next);
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
      const T* gp = gate_at<T>(s, l, state_elems, off, (int)threadIdx.x * V);
      if (gp) {
        float a[V];
        ldv<T>(gp).get(a);
#pragma unroll
        for (int i = 0; i < V; ++i) val[i] = a[i] * carry[i];
      } else {
#pragma unroll
        for (int i = 0; i < V; ++i) val[i] = s.keep * carry[i];
      }
#pragma unroll
      for (int i = 0; i < V; ++i) val[i] += r * (dy[i] - m1 - xh[i] * m2);
      if (s.gamma != 0.0f) {
#pragma unroll
        for (int i = 0; i < V; ++i) val[i] += s.gamma * old_next[i];
        ldv<T>(g + (int64_t)l * state_elems + off).get(old_next);
      }
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

// ---- time-chunked scan for long L and few channels (three phases) ----------------------------------
// Phase 1: per (chunk, channel group) local scan with zero carry-in -> S (value at the chunk's first
// step) and P (product of the gates over the chunk).  Phase 2: per channel, serial over the chunks:
// carry-in of chunk c = G_{c+1}, G_c = S_c + P_c * G_{c+1}.  Phase 3: local scan again with the
// carry-in, writing g.  Scratch: S (then the carry-ins) [nchunks][rows*d] and P likewise, in the
// accumulator type (double for float data).
constexpr int kChunk = 32;

template <typename T, bool kApply>
__global__ void __launch_bounds__(128) scan_chunk_kernel(const ScanArgs s, typename Acc<T>::type* __restrict__ S,
                                                         typename Acc<T>::type* __restrict__ P) {
  typedef typename Acc<T>::type A;
  constexpr int V = Vec<T>::N;
  const int64_t state_elems = s.rows * s.d;
  const int64_t nvec = state_elems / V;
  const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (v >= nvec) return;
  const int c = blockIdx.y;
  const int lo = s.l_lo + c * kChunk, hi = min(s.l_hi, lo + kChunk);
  const int64_t off = v * V;
  const int ch = (int)(off % s.d);
  T* g = (T*)s.g;
  A carry[V], prod[V];
#pragma unroll
  for (int i = 0; i < V; ++i) {
    carry[i] = kApply ? S[(int64_t)c * state_elems + off + i] : (A)0;
    prod[i] = (A)1;
  }
  for (int l = hi - 1; l >= lo; --l) {
    A val[V];
    scan_step<T>(s, l, state_elems, off, ch, carry, val);
    if (kApply) {
      Vec<T> out;
      out.set(val);
      stv<T>(g + (int64_t)l * state_elems + off, out);
    } else {
      const T* gp = gate_at<T>(s, l, state_elems, off, ch);
      if (gp) {
        float a[V];
        ldv<T>(gp).get(a);
#pragma unroll
        for (int i = 0; i < V; ++i) prod[i] *= a[i];
      }
    }
#pragma unroll
    for (int i = 0; i < V; ++i) carry[i] = val[i];
  }
  if (!kApply) {
#pragma unroll
    for (int i = 0; i < V; ++i) {
      S[(int64_t)c * state_elems + off + i] = carry[i];
      P[(int64_t)c * state_elems + off + i] = prod[i];
    }
  }
}

template <typename T>
__global__ void __launch_bounds__(128) scan_carry_kernel(const ScanArgs s, typename Acc<T>::type* __restrict__ S,
                                                         const typename Acc<T>::type* __restrict__ P, int nchunks) {
  typedef typename Acc<T>::type A;
  const int64_t state_elems = s.rows * s.d;
  const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= state_elems) return;
  A G = (A)to_f(((const T*)s.g)[(int64_t)s.l_hi * state_elems + e]);
  for (int c = nchunks - 1; c >= 0; --c) {
    const A sc = S[(int64_t)c * state_elems + e], pc = P[(int64_t)c * state_elems + e];
    S[(int64_t)c * state_elems + e] = G;  // carry-in of chunk c
    G = sc + pc * G;
  }
}

// ---- row-wise helpers ----------------------------------------------------------------------------
template <typename T>
__global__ void copy_kernel(T* __restrict__ dst, const T* __restrict__ src, int64_t nvec) {
  int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (v < nvec) stv<T>(dst + v * Vec<T>::N, ldv<T>(src + v * Vec<T>::N));
}

template <typename T>
__global__ void mul_kernel(T* __restrict__ dst, const T* __restrict__ a, const T* __restrict__ b, int64_t nvec) {
  constexpr int V = Vec<T>::N;
  const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (v >= nvec) return;
  float x[V], y[V];
  ldv_stream<T>(a + v * V).get(x);
  ldv_stream<T>(b + v * V).get(y);
#pragma unroll
  for (int i = 0; i < V; ++i) x[i] *= y[i];
  Vec<T> out;
  out.set(x);
  stv<T>(dst + v * V, out);
}

// states[s] += carry for every state s (the carry of a scan whose gates are all one, applied after the fact)
template <typename T>
__global__ void add_to_states_kernel(T* __restrict__ states, const T* __restrict__ carry, int64_t elems) {
  constexpr int V = Vec<T>::N;
  const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (v * V >= elems) return;
  T* p = states + (int64_t)blockIdx.y * elems + v * V;
  float a[V], c[V];
  ldv<T>(p).get(a);
  ldv<T>(carry + v * V).get(c);
#pragma unroll
  for (int i = 0; i < V; ++i) a[i] += c[i];
  Vec<T> out;
  out.set(a);
  stv<T>(p, out);
}

template <typename T>
__global__ void to_f32_kernel(const T* __restrict__ src, float* __restrict__ dst, int64_t n) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = to_f(src[i]);
}

// xhat = (x - mean) * rstd over the last axis, biased variance; one block per row, two passes in registers.
template <typename T, typename X>
__global__ void __launch_bounds__(1024) layernorm_fwd_kernel(const X* __restrict__ x, T* __restrict__ xhat,
                                                             float* __restrict__ rstd, int d, float eps,
                                                             float* __restrict__ master) {
  constexpr int V = Vec<T>::N;
  __shared__ float red[2][32];
  const int64_t row = blockIdx.x;
  const bool active = (int)threadIdx.x * V < d;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
  float val[V];
#pragma unroll
  for (int i = 0; i < V; ++i) val[i] = active ? to_f(x[row * d + threadIdx.x * V + i]) : 0.0f;
  float s1 = 0.0f;
#pragma unroll
  for (int i = 0; i < V; ++i) s1 += val[i];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s1 += __shfl_xor_sync(0xffffffffu, s1, o);
  if (lane == 0) red[0][warp] = s1;
  __syncthreads();
  float t = 0.0f;
  for (int w = 0; w < nwarps; ++w) t += red[0][w];
  const float mu = t / (float)d;
  float s2 = 0.0f;
#pragma unroll
  for (int i = 0; i < V; ++i) {
    const float c = active ? val[i] - mu : 0.0f;
    s2 = fmaf(c, c, s2);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s2 += __shfl_xor_sync(0xffffffffu, s2, o);
  if (lane == 0) red[1][warp] = s2;
  __syncthreads();
  t = 0.0f;
  for (int w = 0; w < nwarps; ++w) t += red[1][w];
  const float r = rsqrtf(t / (float)d + eps);
  if (threadIdx.x == 0) rstd[row] = r;
  if (active) {
    float o[V];
#pragma unroll
    for (int i = 0; i < V; ++i) o[i] = (val[i] - mu) * r;
    Vec<T> out;
    out.set(o);
    stv<T>(xhat + row * d + threadIdx.x * V, out);
    if (master) {  // the float copy of the residual stream continues from the normalised values (post-LN layers)
#pragma unroll
      for (int i = 0; i < V; ++i) master[row * d + threadIdx.x * V + i] = o[i];
    }
  }
}

// Post-LN layers: per row, t = LayerNorm-backward of g through the layer's own output xo (the normalised state):
// t = rstd (g - mean g - xo mean(g xo)), and c = t - rstd g, the part of the layer's VJP that is not the block's.
template <typename T>
__global__ void __launch_bounds__(1024) postln_prepass_kernel(const T* __restrict__ g, const T* __restrict__ xo,
                                                              const float* __restrict__ rstd, T* __restrict__ t_out,
                                                              T* __restrict__ c_out, int d) {
  constexpr int V = Vec<T>::N;
  __shared__ float red[2][32];
  const int64_t row = blockIdx.x;
  const bool active = (int)threadIdx.x * V < d;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
  const int64_t off = row * d + (int64_t)threadIdx.x * V;
  float gv[V], xv[V];
#pragma unroll
  for (int i = 0; i < V; ++i) gv[i] = xv[i] = 0.0f;
  if (active) {
    ldv<T>(g + off).get(gv);
    ldv<T>(xo + off).get(xv);
  }
  float s1 = 0.0f, s2 = 0.0f;
#pragma unroll
  for (int i = 0; i < V; ++i) {
    s1 += gv[i];
    s2 = fmaf(gv[i], xv[i], s2);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    s1 += __shfl_xor_sync(0xffffffffu, s1, o);
    s2 += __shfl_xor_sync(0xffffffffu, s2, o);
  }
  if (lane == 0) {
    red[0][warp] = s1;
    red[1][warp] = s2;
  }
  __syncthreads();
  float t1 = 0.0f, t2 = 0.0f;
  for (int w = 0; w < nwarps; ++w) {
    t1 += red[0][w];
    t2 += red[1][w];
  }
  if (!active) return;
  const float m1 = t1 / (float)d, m2 = t2 / (float)d, r = rstd[row];
  float tv[V], cv[V];
#pragma unroll
  for (int i = 0; i < V; ++i) {
    cv[i] = r * (-m1 - xv[i] * m2);
    tv[i] = fmaf(r, gv[i], cv[i]);
  }
  Vec<T> a, b;
  a.set(tv);
  b.set(cv);
  stv<T>(t_out + off, a);
  stv<T>(c_out + off, b);
}

// partial[b][c] = sum over the block's rows of g[r][c] * x[r][c]
template <typename T>
__global__ void __launch_bounds__(256) gate_grad_kernel(const T* __restrict__ g, const T* __restrict__ x,
                                                        int64_t rows, int d, float* __restrict__ partial) {
  const int64_t per = (rows + gridDim.x - 1) / gridDim.x;
  const int64_t r0 = (int64_t)blockIdx.x * per, r1 = min(rows, r0 + per);
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    // four running sums over interleaved rows: eight loads in flight per thread instead of two, fixed order
    float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    int64_t r = r0;
    for (; r + 4 <= r1; r += 4) {
      float gv[4], xv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        gv[i] = to_f(g[(r + i) * d + c]);
        xv[i] = to_f(x[(r + i) * d + c]);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[i] = fmaf(gv[i], xv[i], acc[i]);
    }
    for (; r < r1; ++r) acc[0] = fmaf(to_f(g[r * d + c]), to_f(x[r * d + c]), acc[0]);
    partial[(int64_t)blockIdx.x * d + c] = (acc[0] + acc[1]) + (acc[2] + acc[3]);
  }
}

// v = a * b (b optional); hi = v rounded to tf32 precision, lo = the same rounding of v - hi.  hi + lo carries
// 21+ bits of v, and both are exact tf32 operands.
__global__ void split_tf32_kernel(const float4* __restrict__ a, const float4* __restrict__ b, float4* __restrict__ hi,
                                  float4* __restrict__ lo, int64_t nvec) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= nvec) return;
  float4 v = a[i];
  if (b) {
    const float4 w = b[i];
    v.x *= w.x; v.y *= w.y; v.z *= w.z; v.w *= w.w;
  }
  float4 h, l;
  h.x = round_tf32(v.x); h.y = round_tf32(v.y); h.z = round_tf32(v.z); h.w = round_tf32(v.w);
  l.x = round_tf32(v.x - h.x); l.y = round_tf32(v.y - h.y); l.z = round_tf32(v.z - h.z); l.w = round_tf32(v.w - h.w);
  hi[i] = h;
  lo[i] = l;
}
__global__ void __launch_bounds__(256) split_tf32_transposed_kernel(const float* __restrict__ a, const float* __restrict__ b,
                                                                    float* __restrict__ hiT, float* __restrict__ loT,
                                                                    int64_t rows, int cols, int64_t ld) {
  __shared__ float th[32][33], tl[32][33];
  const int64_t r0 = (int64_t)blockIdx.x * 32;
  const int c0 = blockIdx.y * 32;
  const int tx = threadIdx.x % 32, ty = threadIdx.x / 32;  // ty in 0..7
  for (int i = ty; i < 32; i += 8) {
    const int64_t r = r0 + i;
    const int c = c0 + tx;
    float v = 0.0f;
    if (r < rows && c < cols) {
      v = a[r * ld + c];
      if (b) v *= b[r * ld + c];
    }
    const float h = round_tf32(v);
    th[i][tx] = h;
    tl[i][tx] = round_tf32(v - h);
  }
  __syncthreads();
  for (int i = ty; i < 32; i += 8) {
    const int c = c0 + i;
    const int64_t r = r0 + tx;
    if (c < cols && r < rows) {
      hiT[(int64_t)c * rows + r] = th[tx][i];
      loT[(int64_t)c * rows + r] = tl[tx][i];
    }
  }
}

inline int row_block_threads(int d, int V) {
  int t = (d / V + 31) / 32 * 32;
  return t < 32 ? 32 : t;
}

}  // namespace

size_t scan_scratch_bytes(int dtype, int L, int64_t rows, int d) {
  const int V = dtype == HBP_F32 ? 4 : 8;
  const int64_t nvec = rows * d / V;
  if (nvec >= 148 * 512 || L < 4 * kChunk) return 0;  // enough channels (or too short) for the serial form
  const int nchunks = (L + kChunk - 1) / kChunk;
  return (size_t)2 * nchunks * rows * d * (dtype == HBP_F32 ? sizeof(double) : sizeof(float));
}

void scan_reverse(Launcher& lc, const ScanArgs& s) {
  if (s.l_hi <= s.l_lo || s.rows <= 0) return;
  const int V = s.dtype == HBP_F32 ? 4 : 8;
  const int64_t nvec = s.rows * s.d / V;
  if (s.xhat && s.lnstat) {
    const unsigned grid = (unsigned)((nvec + 255) / 256);
    const bool shift = s.gamma != 0.0f;
    if (s.dtype == HBP_F32) {
      if (shift) scan_depth_lnstat_kernel<float, true><<<grid, 256, 0, lc.stream>>>(s);
      else scan_depth_lnstat_kernel<float, false><<<grid, 256, 0, lc.stream>>>(s);
    } else {
      if (shift) scan_depth_lnstat_kernel<bf16, true><<<grid, 256, 0, lc.stream>>>(s);
      else scan_depth_lnstat_kernel<bf16, false><<<grid, 256, 0, lc.stream>>>(s);
    }
    lc.count();
    lc.check();
    return;
  }
  if (s.xhat) {
    const int threads = row_block_threads(s.d, V);
    if (s.dtype == HBP_F32) scan_depth_ln_kernel<float><<<(unsigned)s.rows, threads, 0, lc.stream>>>(s);
    else scan_depth_ln_kernel<bf16><<<(unsigned)s.rows, threads, 0, lc.stream>>>(s);
    lc.count();
    lc.check();
    return;
  }
  const int steps = s.l_hi - s.l_lo;
  const size_t need = scan_scratch_bytes(s.dtype, steps, s.rows, s.d);
  // few channels, many steps: one serial pass in time behind a ring of TMA loads reads and writes every byte
  // once; the three-phase form below remains for what that kernel does not take (a gate table per step)
  const bool depth_only = s.u2 || s.gate == kGateRow;  // forms only the serial depth scan takes
  if (need > 0 && !depth_only && scan_ring(lc, s)) return;
  if (need > 0 && !depth_only && s.scratch && s.scratch_bytes >= need && s.keep == 1.0f && s.gamma == 0.0f) {
    const int nchunks = (steps + kChunk - 1) / kChunk;
    dim3 grid((unsigned)((nvec + 127) / 128), nchunks);
    const unsigned cgrid = (unsigned)((s.rows * s.d + 127) / 128);
    if (s.dtype == HBP_F32) {
      double* S = (double*)s.scratch;
      double* P = S + (int64_t)nchunks * s.rows * s.d;
      scan_chunk_kernel<float, false><<<grid, 128, 0, lc.stream>>>(s, S, P);
      scan_carry_kernel<float><<<cgrid, 128, 0, lc.stream>>>(s, S, P, nchunks);
      scan_chunk_kernel<float, true><<<grid, 128, 0, lc.stream>>>(s, S, P);
    } else {
      float* S = (float*)s.scratch;
      float* P = S + (int64_t)nchunks * s.rows * s.d;
      scan_chunk_kernel<bf16, false><<<grid, 128, 0, lc.stream>>>(s, S, P);
      scan_carry_kernel<bf16><<<cgrid, 128, 0, lc.stream>>>(s, S, P, nchunks);
      scan_chunk_kernel<bf16, true><<<grid, 128, 0, lc.stream>>>(s, S, P);
    }
    lc.count(3);
    lc.check();
    return;
  }
  const unsigned grid = (unsigned)((nvec + 255) / 256);
  const bool shift = s.gamma != 0.0f;
  if (s.dtype == HBP_F32) {
    if (shift) scan_depth_kernel<float, true><<<grid, 256, 0, lc.stream>>>(s);
    else scan_depth_kernel<float, false><<<grid, 256, 0, lc.stream>>>(s);
  } else {
    if (shift) scan_depth_kernel<bf16, true><<<grid, 256, 0, lc.stream>>>(s);
    else scan_depth_kernel<bf16, false><<<grid, 256, 0, lc.stream>>>(s);
  }
  lc.count();
  lc.check();
}

void ln_stats_finish(Launcher& lc, const float2* stats, int slots, const float* rstd, float4* lnstat, int64_t count,
                     int d) {
  ln_stats_finish_kernel<<<(unsigned)((count + 255) / 256), 256, 0, lc.stream>>>(stats, slots, rstd, lnstat, count,
                                                                                1.0f / (float)d);
  lc.count();
  lc.check();
}

void copy_state(Launcher& lc, int dtype, void* dst, const void* src, int64_t elems) {
  if (dtype == HBP_F32)
    copy_kernel<float><<<(unsigned)((elems / 4 + 255) / 256), 256, 0, lc.stream>>>((float*)dst, (const float*)src, elems / 4);
  else
    copy_kernel<bf16><<<(unsigned)((elems / 8 + 255) / 256), 256, 0, lc.stream>>>((bf16*)dst, (const bf16*)src, elems / 8);
  lc.count();
  lc.check();
}

void postln_prepass(Launcher& lc, int dtype, const void* g, const void* xo, const float* rstd, void* t_out, void* c_out,
                    int64_t rows, int d) {
  const int V = dtype == HBP_F32 ? 4 : 8;
  const int threads = row_block_threads(d, V);
  if (dtype == HBP_F32)
    postln_prepass_kernel<float><<<(unsigned)rows, threads, 0, lc.stream>>>((const float*)g, (const float*)xo, rstd,
                                                                           (float*)t_out, (float*)c_out, d);
  else
    postln_prepass_kernel<bf16><<<(unsigned)rows, threads, 0, lc.stream>>>((const bf16*)g, (const bf16*)xo, rstd,
                                                                          (bf16*)t_out, (bf16*)c_out, d);
  lc.count();
  lc.check();
}

void mul_elementwise(Launcher& lc, int dtype, void* dst, const void* a, const void* b, int64_t elems) {
  const int V = dtype == HBP_F32 ? 4 : 8;
  const unsigned grid = (unsigned)((elems / V + 255) / 256);
  if (dtype == HBP_F32) mul_kernel<float><<<grid, 256, 0, lc.stream>>>((float*)dst, (const float*)a, (const float*)b, elems / V);
  else mul_kernel<bf16><<<grid, 256, 0, lc.stream>>>((bf16*)dst, (const bf16*)a, (const bf16*)b, elems / V);
  lc.count();
  lc.check();
}

void add_to_states(Launcher& lc, int dtype, void* states, const void* carry, int count, int64_t elems) {
  const int V = dtype == HBP_F32 ? 4 : 8;
  dim3 grid((unsigned)((elems / V + 255) / 256), (unsigned)count);
  if (dtype == HBP_F32) add_to_states_kernel<float><<<grid, 256, 0, lc.stream>>>((float*)states, (const float*)carry, elems);
  else add_to_states_kernel<bf16><<<grid, 256, 0, lc.stream>>>((bf16*)states, (const bf16*)carry, elems);
  lc.count();
  lc.check();
}

void convert_to_f32(Launcher& lc, int dtype, const void* src, float* dst, int64_t elems) {
  const unsigned grid = (unsigned)((elems + 255) / 256);
  if (dtype == HBP_F32) to_f32_kernel<float><<<grid, 256, 0, lc.stream>>>((const float*)src, dst, elems);
  else to_f32_kernel<bf16><<<grid, 256, 0, lc.stream>>>((const bf16*)src, dst, elems);
  lc.count();
  lc.check();
}

void layernorm_fwd(Launcher& lc, int dtype, const void* x, bool x_is_f32, void* xhat, float* rstd, int64_t rows,
                   int d, float eps, float* master) {
  const int V = dtype == HBP_F32 ? 4 : 8;
  const int threads = row_block_threads(d, V);
  if (dtype == HBP_F32)
    layernorm_fwd_kernel<float, float><<<(unsigned)rows, threads, 0, lc.stream>>>((const float*)x, (float*)xhat, rstd, d, eps, master);
  else if (x_is_f32)
    layernorm_fwd_kernel<bf16, float><<<(unsigned)rows, threads, 0, lc.stream>>>((const float*)x, (bf16*)xhat, rstd, d, eps, master);
  else
    layernorm_fwd_kernel<bf16, bf16><<<(unsigned)rows, threads, 0, lc.stream>>>((const bf16*)x, (bf16*)xhat, rstd, d, eps, master);
  lc.count();
  lc.check();
}

void split_tf32(Launcher& lc, const float* a, const float* b, float* hi, float* lo, int64_t elems) {
  const int64_t nvec = elems / 4;
  split_tf32_kernel<<<(unsigned)((nvec + 255) / 256), 256, 0, lc.stream>>>((const float4*)a, (const float4*)b, (float4*)hi,
                                                                          (float4*)lo, nvec);
  lc.count();
  lc.check();
}

void split_tf32_transposed(Launcher& lc, const float* a, const float* b, float* hiT, float* loT, int64_t rows, int cols,
                           int64_t ld) {
  dim3 grid((unsigned)((rows + 31) / 32), (unsigned)((cols + 31) / 32));
  split_tf32_transposed_kernel<<<grid, 256, 0, lc.stream>>>(a, b, hiT, loT, rows, cols, ld > 0 ? ld : cols);
  lc.count();
  lc.check();
}

void gate_grad(Launcher& lc, int dtype, const void* g, const void* x, int64_t rows_total, int d, float* da,
               float* partial, int blocks) {
  if (dtype == HBP_F32)
    gate_grad_kernel<float><<<blocks, 256, 0, lc.stream>>>((const float*)g, (const float*)x, rows_total, d, partial);
  else
    gate_grad_kernel<bf16><<<blocks, 256, 0, lc.stream>>>((const bf16*)g, (const bf16*)x, rows_total, d, partial);
  lc.count();
  lc.check();
  reduce_splitk(lc, partial, da, blocks, d);
}

}  // namespace hbp
