// CUDA-core (FFMA) GEMM with arbitrary operand strides, fp32 accumulation and fused epilogues.
// Serves the float configurations (where 1e-5 accuracy rules out reduced-precision tensor-core
// inputs) and every bf16 problem whose shape the tcgen05 kernel does not take.
#include "hbp_internal.h"

namespace hbp {

namespace {

template <typename T>
__device__ __forceinline__ float load_a(const T* A, const T* A2, int64_t off) {
  float v = to_f(A[off]);
  if (A2) v *= to_f(A2[off]);
  return v;
}

template <typename T>
__device__ __forceinline__ void epilogue_store(const GemmArgs& g, int b, int m, int n, float acc) {
  const int64_t dn = (int64_t)m * g.ldd + n;
  switch (g.epi) {
    case EPI_STORE_LN:
    case EPI_STORE: {
      if (g.d_f32) ((float*)g.D)[b * g.d_sb + dn] = acc;
      else ((T*)g.D)[b * g.d_sb + dn] = from_f<T>(acc);
    } break;
    case EPI_GELU_FWD: {
      ((T*)g.D)[b * g.d_sb + dn] = from_f<T>(gelu_f(acc));
      ((T*)g.D2)[b * g.d2_sb + (int64_t)m * g.ldd2 + n] = from_f<T>(gelu_prime_f(acc));
    } break;
    case EPI_RESID: {
      float gate = g.gate ? to_f(((const T*)g.gate)[b * g.gate_sb + n]) : 1.0f;
      float r = g.R ? g.R[(int64_t)m * g.N + n] : to_f(((const T*)g.E)[b * g.e_sb + (int64_t)m * g.lde + n]);
      float v = gate * r + acc;
      if (g.relu) {
        ((T*)g.D2)[b * g.d2_sb + (int64_t)m * g.ldd2 + n] = from_f<T>(v > 0.0f ? 1.0f : 0.0f);
        v = fmaxf(v, 0.0f);
      }
      if (g.R) g.R[(int64_t)m * g.N + n] = v;
      ((T*)g.D)[b * g.d_sb + dn] = from_f<T>(v);
    } break;
    case EPI_ADD: {
      float e = to_f(((const T*)g.E)[b * g.e_sb + (int64_t)m * g.lde + n]);
      if (g.d_f32) ((float*)g.D)[b * g.d_sb + dn] = acc + e;
      else ((T*)g.D)[b * g.d_sb + dn] = from_f<T>(acc + e);
    } break;
    case EPI_MUL: {
      float e = to_f(((const T*)g.E)[b * g.e_sb + (int64_t)m * g.lde + n]);
      ((T*)g.D)[b * g.d_sb + dn] = from_f<T>(acc * e);
    } break;
    case EPI_AFFINE: {
      float gate = g.gate ? to_f(((const T*)g.gate)[b * g.gate_sb + n]) : 1.0f;
      float e = g.E ? to_f(((const T*)g.E)[b * g.e_sb + (int64_t)m * g.lde + n]) : 0.0f;
      float e2 = to_f(((const T*)g.E2)[b * g.e2_sb + (int64_t)m * g.lde2 + n]);
      ((T*)g.D)[b * g.d_sb + dn] = from_f<T>(e + gate * e2 + acc);
    } break;
    case EPI_RNN_FWD: {
      float gate = g.gate ? to_f(((const T*)g.gate)[b * g.gate_sb + n]) : 1.0f;
      float z = acc + to_f(((const T*)g.E)[b * g.e_sb + (int64_t)m * g.lde + n]);
      // tanh and its derivative 1 - tanh^2 = 4e / (1 + e)^2 with e = exp(-2|z|): no cancellation near |c| = 1
      float e = expf(-2.0f * fabsf(z));
      float c = copysignf((1.0f - e) / (1.0f + e), z);
      float h = to_f(((const T*)g.E2)[b * g.e2_sb + (int64_t)m * g.lde2 + n]);
      ((T*)g.D2)[b * g.d2_sb + (int64_t)m * g.ldd2 + n] = from_f<T>(4.0f * e / ((1.0f + e) * (1.0f + e)));
      ((T*)g.D)[b * g.d_sb + dn] = from_f<T>(gate * h + c);
    } break;
  }
}

// 256 threads, BM x BN output tile, BK = 16, (BM/16) x (BN/16) register micro-tile.
template <typename T, int BM, int BN>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const GemmArgs g) {
  constexpr int BK = 16, TM = BM / 16, TN = BN / 16;
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];
  const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
  const int b = blockIdx.z / g.splitk, split = blockIdx.z % g.splitk;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  const T* A = (const T*)g.A + (int64_t)b * g.a_sb;
  const T* A2 = g.A2 ? (const T*)g.A2 + (int64_t)b * g.a_sb : nullptr;
  const T* B = (const T*)g.B + (int64_t)b * g.b_sb;
  // K range of this split (multiples of BK except the last)
  const int ktiles = (g.K + BK - 1) / BK;
  const int per = (ktiles + g.splitk - 1) / g.splitk;
  const int kbeg = split * per * BK;
  const int kend = min(g.K, (split + 1) * per * BK);

  float acc[TM][TN];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc[i][j] = 0.0f;

  const bool a_kmajor = (g.a_sk == 1), b_kmajor = (g.b_sk == 1);
  for (int k0 = kbeg; k0 < kend; k0 += BK) {
#pragma unroll
    for (int i = 0; i < (BM * BK) / 256; ++i) {
      int idx = tid + i * 256;
      int kk = a_kmajor ? idx % BK : idx / BM;
      int mm = a_kmajor ? idx / BK : idx % BM;
      int m = m0 + mm, k = k0 + kk;
      float v = 0.0f;
      if (m < g.M && k < kend) v = load_a<T>(A, A2, (int64_t)m * g.a_sm + (int64_t)k * g.a_sk);
      As[kk][mm] = v;
    }
#pragma unroll
    for (int i = 0; i < (BN * BK) / 256; ++i) {
      int idx = tid + i * 256;
      int kk = b_kmajor ? idx % BK : idx / BN;
      int nn = b_kmajor ? idx / BK : idx % BN;
      int n = n0 + nn, k = k0 + kk;
      float v = 0.0f;
      if (n < g.N && k < kend) v = to_f(B[(int64_t)n * g.b_sn + (int64_t)k * g.b_sk]);
      Bs[kk][nn] = v;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[TM], bb[TN];
#pragma unroll
      for (int i = 0; i < TM; ++i) a[i] = As[kk][ty + 16 * i];
#pragma unroll
      for (int j = 0; j < TN; ++j) bb[j] = Bs[kk][tx + 16 * j];
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], bb[j], acc[i][j]);
    }
    __syncthreads();
  }

#pragma unroll
  for (int i = 0; i < TM; ++i) {
    int m = m0 + ty + 16 * i;
    if (m >= g.M) continue;
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      int n = n0 + tx + 16 * j;
      if (n >= g.N) continue;
      if (g.splitk > 1) {
        g.partial[(((int64_t)split * g.batch + b) * g.M + m) * g.N + n] = acc[i][j];
      } else {
        epilogue_store<T>(g, b, m, n, acc[i][j]);
      }
    }
  }
}

__global__ void reduce_splitk_kernel(const float* __restrict__ partial, float* __restrict__ out, int splits,
                                     int64_t elems) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= elems) return;
  double s = 0.0;
  for (int k = 0; k < splits; ++k) s += (double)partial[(int64_t)k * elems + i];  // fixed order: deterministic
  out[i] = (float)s;
}

template <typename T>
void launch_simt(Launcher& lc, const GemmArgs& g) {
  const int64_t ctas128 = (int64_t)((g.M + 127) / 128) * ((g.N + 127) / 128) * g.batch * g.splitk;
  if (ctas128 >= 148 && g.M >= 128 && g.N >= 128) {
    dim3 grid((g.N + 127) / 128, (g.M + 127) / 128, g.batch * g.splitk);
    gemm_simt_kernel<T, 128, 128><<<grid, 256, 0, lc.stream>>>(g);
  } else if (g.M > 32) {
    dim3 grid((g.N + 63) / 64, (g.M + 63) / 64, g.batch * g.splitk);
    gemm_simt_kernel<T, 64, 64><<<grid, 256, 0, lc.stream>>>(g);
  } else {
    dim3 grid((g.N + 31) / 32, (g.M + 31) / 32, g.batch * g.splitk);
    gemm_simt_kernel<T, 32, 32><<<grid, 256, 0, lc.stream>>>(g);
  }
  lc.count();
  lc.check();
}

}  // namespace

void reduce_splitk(Launcher& lc, const float* partial, float* out, int splits, int64_t elems) {
  reduce_splitk_kernel<<<(unsigned)((elems + 255) / 256), 256, 0, lc.stream>>>(partial, out, splits, elems);
  lc.count();
  lc.check();
}

void gemm_simt(Launcher& lc, const GemmArgs& g) {
  if (g.M <= 0 || g.N <= 0 || g.batch <= 0) return;
  if (g.in_dtype == HBP_F32) launch_simt<float>(lc, g);
  else launch_simt<bf16>(lc, g);
  // split-K supports a plain contiguous float store only
  if (g.splitk > 1) reduce_splitk(lc, g.partial, (float*)g.D, g.splitk, (int64_t)g.batch * g.M * g.N);
}

}  // namespace hbp
