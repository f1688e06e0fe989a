// Causal softmax attention, forward and flash-style backward (scores recomputed from Q, K and the
// stored log-sum-exp; the S x S matrix is never written).  CUDA-core version: every row is owned by
// four threads that split the head dimension; tiles of the opposite side are staged in shared memory.
//   forward:  P = softmax(Q K^T / sqrt(dh) + causal mask),  O = P V,  lse_i = log sum_j exp(s_ij)
//   backward: D_i = sum(dO_i * O_i);  dV = P^T dO;  dP = dO V^T;  dS = P * (dP - D);
//             dQ = dS K / sqrt(dh);  dK = dS^T Q / sqrt(dh)
#include "hbp_internal.h"

namespace hbp {

namespace {

constexpr int kRows = 32;     // rows (queries or keys) per block
constexpr int kThreads = 128; // 4 threads per row

// expf for float data (1e-5 accuracy target), the fast intrinsic for bf16 data
template <typename T>
__device__ __forceinline__ float exp_t(float x) {
  if constexpr (sizeof(T) == 4) return expf(x);
  else return __expf(x);
}

__device__ __forceinline__ float quad_sum(float v) {
  v += __shfl_xor_sync(0xffffffffu, v, 1);
  v += __shfl_xor_sync(0xffffffffu, v, 2);
  return v;
}

template <typename T, int DH>
__device__ __forceinline__ void load_tile(float (*dst)[DH + 4], const T* base, int64_t ld, int row0, int nrows_valid) {
  // dst[r][c] = base[(row0 + r) * ld + c] for r < kRows, zero beyond nrows_valid
  for (int idx = threadIdx.x; idx < kRows * DH; idx += kThreads) {
    int r = idx / DH, c = idx % DH;
    dst[r][c] = (r < nrows_valid) ? to_f(base[(int64_t)(row0 + r) * ld + c]) : 0.0f;
  }
}

template <typename T, int DH>
__global__ void __launch_bounds__(kThreads) attn_fwd_kernel(const AttnArgs a) {
  constexpr int DP = DH / 4;
  __shared__ float Ks[kRows][DH + 4];
  __shared__ float Vs[kRows][DH + 4];
  const int S = a.seq, d = a.heads * DH, ld = 3 * d;
  const int qt = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int r = threadIdx.x / 4, part = threadIdx.x % 4;
  const int qi = qt * kRows + r;
  const bool valid = qi < S;
  const T* base = (const T*)a.qkv + (int64_t)b * S * ld + h * DH;
  const float scale = rsqrtf((float)DH);
  float q[DP], o[DP];
#pragma unroll
  for (int i = 0; i < DP; ++i) {
    q[i] = valid ? to_f(base[(int64_t)qi * ld + part * DP + i]) * scale : 0.0f;
    o[i] = 0.0f;
  }
  float mrun = -INFINITY, lrun = 0.0f;
  const int last_key = min(S, (qt + 1) * kRows);  // causal: keys < this
  for (int k0 = 0; k0 < last_key; k0 += kRows) {
    const int nvalid = min(kRows, S - k0);
    __syncthreads();
    load_tile<T, DH>(Ks, base + d, ld, k0, nvalid);
    load_tile<T, DH>(Vs, base + 2 * d, ld, k0, nvalid);
    __syncthreads();
    float sc[kRows];
    float tmax = -INFINITY;
#pragma unroll
    for (int j = 0; j < kRows; ++j) {
      float p = 0.0f;
#pragma unroll
      for (int i = 0; i < DP; ++i) p = fmaf(q[i], Ks[j][part * DP + i], p);
      p = quad_sum(p);
      const bool ok = (k0 + j <= qi) && (j < nvalid);
      sc[j] = ok ? p : -INFINITY;
      tmax = fmaxf(tmax, sc[j]);
    }
    const float mnew = fmaxf(mrun, tmax);
    if (mnew == -INFINITY) continue;  // (only rows past the end) nothing visible yet
    const float corr = exp_t<T>(mrun - mnew);
    lrun *= corr;
#pragma unroll
    for (int i = 0; i < DP; ++i) o[i] *= corr;
#pragma unroll
    for (int j = 0; j < kRows; ++j) {
      const float p = exp_t<T>(sc[j] - mnew);
      lrun += p;
#pragma unroll
      for (int i = 0; i < DP; ++i) o[i] = fmaf(p, Vs[j][part * DP + i], o[i]);
    }
    mrun = mnew;
  }
  if (valid) {
    const float inv = 1.0f / lrun;
    T* op = (T*)a.o + ((int64_t)b * S + qi) * d + h * DH + part * DP;
#pragma unroll
    for (int i = 0; i < DP; ++i) op[i] = from_f<T>(o[i] * inv);
    if (part == 0) a.lse[((int64_t)b * a.heads + h) * S + qi] = mrun + logf(lrun);
  }
}

// D_i = sum_c dO[i][c] * O[i][c] per (batch, head, query)
template <typename T, int DH>
__global__ void __launch_bounds__(kThreads) attn_rowdot_kernel(const AttnArgs a) {
  constexpr int DP = DH / 4;
  const int S = a.seq, d = a.heads * DH;
  const int qi = blockIdx.x * kRows + threadIdx.x / 4, part = threadIdx.x % 4;
  const int h = blockIdx.y, b = blockIdx.z;
  float acc = 0.0f;
  if (qi < S) {
    const int64_t off = ((int64_t)b * S + qi) * d + h * DH + part * DP;
#pragma unroll
    for (int i = 0; i < DP; ++i) acc = fmaf(to_f(((const T*)a.d_o)[off + i]), to_f(((const T*)a.o)[off + i]), acc);
  }
  acc = quad_sum(acc);
  if (qi < S && part == 0) a.delta_rows[((int64_t)b * a.heads + h) * S + qi] = acc;
}

// dQ: one query row per thread quad, loop over visible key tiles.
template <typename T, int DH>
__global__ void __launch_bounds__(kThreads) attn_bwd_dq_kernel(const AttnArgs a) {
  constexpr int DP = DH / 4;
  __shared__ float Ks[kRows][DH + 4];
  __shared__ float Vs[kRows][DH + 4];
  const int S = a.seq, d = a.heads * DH, ld = 3 * d;
  const int qt = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int r = threadIdx.x / 4, part = threadIdx.x % 4;
  const int qi = qt * kRows + r;
  const bool valid = qi < S;
  const T* base = (const T*)a.qkv + (int64_t)b * S * ld + h * DH;
  const float scale = rsqrtf((float)DH);
  float q[DP], dO[DP], dq[DP];
  const int64_t orow = ((int64_t)b * S + qi) * d + h * DH + part * DP;
#pragma unroll
  for (int i = 0; i < DP; ++i) {
    q[i] = valid ? to_f(base[(int64_t)qi * ld + part * DP + i]) * scale : 0.0f;
    dO[i] = valid ? to_f(((const T*)a.d_o)[orow + i]) : 0.0f;
    dq[i] = 0.0f;
  }
  const int64_t stat = ((int64_t)b * a.heads + h) * S + qi;
  const float lse = valid ? a.lse[stat] : 0.0f, Di = valid ? a.delta_rows[stat] : 0.0f;
  const int last_key = min(S, (qt + 1) * kRows);
  for (int k0 = 0; k0 < last_key; k0 += kRows) {
    const int nvalid = min(kRows, S - k0);
    __syncthreads();
    load_tile<T, DH>(Ks, base + d, ld, k0, nvalid);
    load_tile<T, DH>(Vs, base + 2 * d, ld, k0, nvalid);
    __syncthreads();
#pragma unroll 4
    for (int j = 0; j < kRows; ++j) {
      float s = 0.0f, dp = 0.0f;
#pragma unroll
      for (int i = 0; i < DP; ++i) {
        s = fmaf(q[i], Ks[j][part * DP + i], s);
        dp = fmaf(dO[i], Vs[j][part * DP + i], dp);
      }
      s = quad_sum(s);
      dp = quad_sum(dp);
      const bool ok = valid && (k0 + j <= qi) && (j < nvalid);
      const float p = ok ? exp_t<T>(s - lse) : 0.0f;
      const float ds = p * (dp - Di);
#pragma unroll
      for (int i = 0; i < DP; ++i) dq[i] = fmaf(ds, Ks[j][part * DP + i], dq[i]);
    }
  }
  if (valid) {
    T* out = (T*)a.d_qkv + ((int64_t)b * S + qi) * ld + h * DH + part * DP;
#pragma unroll
    for (int i = 0; i < DP; ++i) out[i] = from_f<T>(dq[i] * scale);
  }
}

// dK, dV: one key row per thread quad, loop over the query tiles that can see it.
template <typename T, int DH>
__global__ void __launch_bounds__(kThreads) attn_bwd_dkv_kernel(const AttnArgs a) {
  constexpr int DP = DH / 4;
  __shared__ float Qs[kRows][DH + 4];
  __shared__ float Os[kRows][DH + 4];  // dO tile
  __shared__ float lse_s[kRows], D_s[kRows];
  const int S = a.seq, d = a.heads * DH, ld = 3 * d;
  const int kt = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int r = threadIdx.x / 4, part = threadIdx.x % 4;
  const int kj = kt * kRows + r;
  const bool valid = kj < S;
  const T* base = (const T*)a.qkv + (int64_t)b * S * ld + h * DH;
  const T* dObase = (const T*)a.d_o + (int64_t)b * S * d + h * DH;
  const float scale = rsqrtf((float)DH);
  float kk[DP], vv[DP], dk[DP], dv[DP];
#pragma unroll
  for (int i = 0; i < DP; ++i) {
    kk[i] = valid ? to_f(base[(int64_t)kj * ld + d + part * DP + i]) * scale : 0.0f;
    vv[i] = valid ? to_f(base[(int64_t)kj * ld + 2 * d + part * DP + i]) : 0.0f;
    dk[i] = dv[i] = 0.0f;
  }
  for (int q0 = kt * kRows; q0 < S; q0 += kRows) {
    const int nvalid = min(kRows, S - q0);
    __syncthreads();
    load_tile<T, DH>(Qs, base, ld, q0, nvalid);
    load_tile<T, DH>(Os, dObase, d, q0, nvalid);
    if (threadIdx.x < kRows) {
      const bool ok = threadIdx.x < nvalid;
      const int64_t stat = ((int64_t)b * a.heads + h) * S + q0 + threadIdx.x;
      lse_s[threadIdx.x] = ok ? a.lse[stat] : 0.0f;
      D_s[threadIdx.x] = ok ? a.delta_rows[stat] : 0.0f;
    }
    __syncthreads();
#pragma unroll 4
    for (int i2 = 0; i2 < kRows; ++i2) {
      float s = 0.0f, dp = 0.0f;
#pragma unroll
      for (int i = 0; i < DP; ++i) {
        s = fmaf(kk[i], Qs[i2][part * DP + i], s);
        dp = fmaf(vv[i], Os[i2][part * DP + i], dp);
      }
      s = quad_sum(s);
      dp = quad_sum(dp);
      const bool ok = valid && (q0 + i2 >= kj) && (i2 < nvalid);
      const float p = ok ? exp_t<T>(s - lse_s[i2]) : 0.0f;
      const float ds = p * (dp - D_s[i2]);
#pragma unroll
      for (int i = 0; i < DP; ++i) {
        dv[i] = fmaf(p, Os[i2][part * DP + i], dv[i]);
        dk[i] = fmaf(ds, Qs[i2][part * DP + i], dk[i]);
      }
    }
  }
  if (valid) {
    T* out = (T*)a.d_qkv + ((int64_t)b * S + kj) * ld + h * DH + part * DP;
#pragma unroll
    for (int i = 0; i < DP; ++i) {
      out[d + i] = from_f<T>(dk[i] * scale);
      out[2 * d + i] = from_f<T>(dv[i]);
    }
  }
}

template <typename T, int DH>
void launch_fwd(Launcher& lc, const AttnArgs& a) {
  dim3 grid((a.seq + kRows - 1) / kRows, a.heads, a.batch);
  attn_fwd_kernel<T, DH><<<grid, kThreads, 0, lc.stream>>>(a);
  lc.count();
  lc.check();
}
template <typename T, int DH>
void launch_bwd(Launcher& lc, const AttnArgs& a) {
  dim3 grid((a.seq + kRows - 1) / kRows, a.heads, a.batch);
  if (a.d_stats && !lc.force_simt && attention_bwd_tc(lc, a, a.status)) return;  // row dots came with dO
  attn_rowdot_kernel<T, DH><<<grid, kThreads, 0, lc.stream>>>(a);
  lc.count();
  lc.check();
  AttnArgs plain = a;
  plain.d_stats = nullptr;
  if (!lc.force_simt && attention_bwd_tc(lc, plain, a.status)) return;  // bf16, head dimension 64: tensor cores
  attn_bwd_dq_kernel<T, DH><<<grid, kThreads, 0, lc.stream>>>(a);
  attn_bwd_dkv_kernel<T, DH><<<grid, kThreads, 0, lc.stream>>>(a);
  lc.count(2);
  lc.check();
}

}  // namespace

#define HBP_ATTN_DISPATCH(fn)                                                      \
  if (a.dtype == HBP_F32) {                                                        \
    if (a.head_dim == 32) fn<float, 32>(lc, a);                                    \
    else if (a.head_dim == 64) fn<float, 64>(lc, a);                               \
    else fn<float, 128>(lc, a);                                                    \
  } else {                                                                         \
    if (a.head_dim == 32) fn<bf16, 32>(lc, a);                                     \
    else if (a.head_dim == 64) fn<bf16, 64>(lc, a);                                \
    else fn<bf16, 128>(lc, a);                                                     \
  }

void attention_fwd(Launcher& lc, const AttnArgs& a) {
  if (!lc.force_simt && attention_fwd_tc(lc, a, a.status)) return;  // bf16, head dimension 64: tensor cores
  HBP_ATTN_DISPATCH(launch_fwd)
}
void attention_bwd(Launcher& lc, const AttnArgs& a) { HBP_ATTN_DISPATCH(launch_bwd) }

}  // namespace hbp
