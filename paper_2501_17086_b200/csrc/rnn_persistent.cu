// The sequential recurrences of the gated tanh RNN (Section 5.2) as ONE launch over all T steps instead of T launches:
//     forward     h_{t+1} = a * h_t + tanh(W h_t + U x_t)                      (plus the cache 1 - tanh^2)
//     exact BPTT  g_t     = delta_t + a * g_{t+1} + (g_{t+1} * tanh'(z_t)) W   (Section 2.2)
// Batch rows are independent, so a thread-block cluster that owns whole rows never waits on any other cluster.
// A cluster of 16 CTAs owns 4 batch rows; CTA c owns d / 16 output channels and keeps its slice of the recurrent
// matrix in REGISTERS for the whole sequence (d / 16 doubles per thread: the matrix is float, held as double so that
// the inner loop is pure FP64 FMA).  Per step a CTA multiplies its slice with the 4 rows' current vector (shared
// memory, broadcast reads), the 16 partial sums per output are added in a fixed tree, and the new value is sent to
// the shared memory of all 16 CTAs with asynchronous distributed-shared-memory stores that count bytes on the
// receiver's mbarrier: the arrival of the data is the signal, there is no separate barrier round trip per step
// (a hardware cluster barrier per step cost about 1900 cycles of a 5000-cycle step when measured).
//
// Waits are bounded (about 2 s); a wait that gives up records HBP_ERR_TIMEOUT in the status word, the whole CTA
// leaves the step loop together, and every CTA still meets its peers at the final hardware cluster barrier, so no
// CTA ends while a peer may still write into its shared memory.
//
// The recurrence is carried in double like the per-step kernels of rnn.cu (a float carry drifts from the fp64
// reference over thousands of steps).  The input projection U x_t of all steps has no dependence on h and is
// formed beforehand by one FP64 GEMM (proj_f64_kernel).
#include "hbp_internal.h"

namespace hbp {

namespace {

constexpr int kCS = 16;  // CTAs per cluster
constexpr int kR = 4;    // batch rows per cluster
constexpr int kKP = 16;  // parts the contraction index is split into (threads per output)
constexpr uint64_t kWaitLimitNs = 2000000000ull;

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t cta_rank_in_cluster() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_index() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t peer_addr(uint32_t local, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
  return r;
}
// 8 bytes into a peer's shared memory; the peer's mbarrier `bar` (same CTA as `addr`) counts them on arrival
__device__ __forceinline__ void send_peer(uint32_t addr, double v, uint32_t bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b64 [%0], %1, [%2];" ::"r"(addr),
               "l"(__double_as_longlong(v)), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void cluster_barrier() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint64_t now_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ bool bar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// false once the time limit has passed (or a thread of this CTA has already given up)
__device__ __forceinline__ bool bar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  uint64_t t0 = 0;
  for (uint32_t spin = 0;; ++spin) {
    if (bar_try(bar, parity)) return true;
    if ((spin & 255u) == 255u) {
      if (*abort_flag) return false;
      const uint64_t now = now_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        return false;
      }
    }
  }
}

struct PersistArgs {
  const void* W;       // [d][d]
  const void* gate;    // [d] or null (ones)
  const double* P;     // forward: U x_t for every step, [T][B][d] in double
  const void* x0;      // forward: h_0 [B][d]
  void* states;        // forward: x_all [T+1][B][d];  backward: g [T+1][B][d] (g[T] already holds delta_T)
  void* deriv;         // [T][B][d]: written by the forward, read by the backward
  const void* delta;   // backward: [T+1][B][d] (per-step loss) or null
  int* status;         // device status word (may be null)
  int T, B, d;
};

// NW = d / kKP elements of the contraction per thread; block = (d / kCS) x kKP threads
template <typename T, int NW, bool BWD>
__global__ void __launch_bounds__(NW * kKP / kCS * kKP, 1) rnn_persistent_kernel(const PersistArgs p) {
  constexpr int D = NW * kKP, DC = D / kCS, NT = DC * kKP;
  extern __shared__ __align__(16) unsigned char persist_smem[];
  // the vector the matrix multiplies, double-buffered over steps; the partial sums; bytes received into vbuf[b]
  double (*vbuf)[kR][D] = reinterpret_cast<double (*)[kR][D]>(persist_smem);
  double (*partial)[kR][DC] = reinterpret_cast<double (*)[kR][DC]>(persist_smem + 2 * kR * D * sizeof(double));
  uint64_t* bars = reinterpret_cast<uint64_t*>(persist_smem + (2 * kR * D + kKP * kR * DC) * sizeof(double));
  volatile int& abort_flag = *reinterpret_cast<volatile int*>(bars + 2);
  const int tid = threadIdx.x, c = tid % DC, kp = tid / DC;
  const uint32_t rank = cta_rank_in_cluster();
  const int row0 = (int)cluster_index() * kR, col = (int)rank * DC + c;
  const T* W = (const T*)p.W;
  const T* deriv = (const T*)p.deriv;
  T* states = (T*)p.states;
  const int64_t state = (int64_t)p.B * D;
  constexpr uint32_t kBufBytes = kR * D * sizeof(double);

  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr(&bars[0])));
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr(&bars[1])));
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // this thread's slice of the matrix, kept for the whole sequence.  forward: row `col` of W (z = W h);
  // backward: column `col` of W (u = v W)
  double w[NW];
#pragma unroll
  for (int j = 0; j < NW; ++j) {
    const int k = kp * NW + j;
    w[j] = (double)to_f(BWD ? W[(int64_t)k * D + col] : W[(int64_t)col * D + k]);
  }
  // the first vector, every CTA its own copy: h_0, or v_{T-1} = g_T * tanh'(z_{T-1})
  for (int i = tid; i < kR * D; i += NT) {
    const int r = i / D, k = i - r * D, row = row0 + r;
    double v = 0.0;
    if (row < p.B) {
      if (BWD) v = (double)to_f(states[(int64_t)p.T * state + (int64_t)row * D + k]) *
                   (double)to_f(deriv[(int64_t)(p.T - 1) * state + (int64_t)row * D + k]);
      else v = (double)to_f(((const T*)p.x0)[(int64_t)row * D + k]);
    }
    vbuf[0][r][k] = v;
  }
  // finisher threads own one output (row fr, channel col) and keep its running value in a register
  const bool finisher = tid < kR * DC;
  const int fr = finisher ? tid / DC : 0;
  const int frow = row0 + fr;
  const bool live = finisher && frow < p.B;
  const int64_t fidx = (int64_t)frow * D + col;
  const double a = (live && p.gate) ? (double)to_f(((const T*)p.gate)[col]) : 1.0;
  double own = 0.0;  // h_t or g_{t+1} of this output
  if (live) own = BWD ? (double)to_f(states[(int64_t)p.T * state + fidx]) : (double)to_f(((const T*)p.x0)[fidx]);
  uint32_t peers[kCS], peer_bar[kCS];  // buffer 0 / barrier 0 of every CTA of the cluster
  {
    const uint32_t local = smem_addr(&vbuf[0][fr][col]), lbar = smem_addr(&bars[0]);
#pragma unroll
    for (int q = 0; q < kCS; ++q) {
      peers[q] = peer_addr(local, (uint32_t)q);
      peer_bar[q] = peer_addr(lbar, (uint32_t)q);
    }
  }
  cluster_barrier();  // every CTA of the cluster has started: its barriers exist and its first vector is in place

  bool ok = true;
  for (int s = 0; s < p.T; ++s) {
    const int t = BWD ? p.T - 1 - s : s;
    const int cur = s & 1, nxt = cur ^ 1;
    // this step's outputs of all 16 CTAs will land in vbuf[nxt]: expect their bytes (bytes that arrive before this
    // line only make the count negative for a moment)
    if (tid == 0 && s + 1 < p.T)
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(&bars[nxt])), "r"(kBufBytes) : "memory");
    // operands of the finishing step, requested before the products so that their latency is hidden
    double add = 0.0, scale = 0.0;
    if (live) {
      if (BWD) {
        if (p.delta) add = (double)to_f(((const T*)p.delta)[(int64_t)t * state + fidx]);
        if (t > 0) scale = (double)to_f(deriv[(int64_t)(t - 1) * state + fidx]);
      } else {
        add = p.P[(int64_t)t * state + fidx];
      }
    }
    double acc[kR];
#pragma unroll
    for (int r = 0; r < kR; ++r) acc[r] = 0.0;
    const double* vb = &vbuf[cur][0][kp * NW];
#pragma unroll
    for (int j = 0; j < NW; j += 2) {
#pragma unroll
      for (int r = 0; r < kR; ++r) {
        const double2 v = *reinterpret_cast<const double2*>(vb + r * D + j);
        acc[r] = fma(w[j], v.x, acc[r]);
        acc[r] = fma(w[j + 1], v.y, acc[r]);
      }
    }
#pragma unroll
    for (int r = 0; r < kR; ++r) partial[kp][r][c] = acc[r];
    __syncthreads();
    if (finisher) {
      double q[kKP];
#pragma unroll
      for (int i = 0; i < kKP; ++i) q[i] = partial[i][fr][c];
#pragma unroll
      for (int w2 = 1; w2 < kKP; w2 *= 2)  // fixed tree: ((q0 + q1) + (q2 + q3)) + ...
#pragma unroll
        for (int i = 0; i < kKP; i += 2 * w2) q[i] += q[i + w2];
      double z = q[0], out, push;
      if (BWD) {
        out = add + a * own + z;        // g_t
        push = out * scale;             // v_{t-1} = g_t * tanh'(z_{t-1})
        if (live) states[(int64_t)t * state + fidx] = from_f<T>((float)out);
      } else {
        z += add;
        const double e = exp(-2.0 * fabs(z));
        const double rcp = 1.0 / (1.0 + e);
        const double th = copysign((1.0 - e) * rcp, z);
        const double sl = 4.0 * e * rcp * rcp;  // 1 - tanh(z)^2 without cancellation
        out = a * own + th;             // h_{t+1}
        push = out;
        if (live) {
          states[(int64_t)(t + 1) * state + fidx] = from_f<T>((float)out);
          ((T*)p.deriv)[(int64_t)t * state + fidx] = from_f<T>((float)sl);
        }
      }
      own = out;
      if (!live) push = 0.0;
      if (s + 1 < p.T) {  // nobody reads what the last step would send
        const uint32_t off = (uint32_t)nxt * kBufBytes, boff = (uint32_t)nxt * 8u;
#pragma unroll
        for (int i = 0; i < kCS; ++i) send_peer(peers[i] + off, push, peer_bar[i] + boff);
      }
    }
    if (s + 1 < p.T) {
      // the next step reads vbuf[nxt]: wait until all of it has arrived.  This is use number s / 2 of that barrier.
      const bool got = bar_wait(smem_addr(&bars[nxt]), (uint32_t)((s >> 1) & 1), (volatile int*)(bars + 2));
      if (__syncthreads_or(!got)) {  // the whole CTA leaves together
        ok = false;
        break;
      }
    }
  }
  if (!ok) {
    if (tid == 0 && p.status) atomicExch(p.status, (int)HBP_ERR_TIMEOUT);
    // give stores that peers may still have in flight towards this CTA time to land before anybody leaves
    const uint64_t t0 = now_ns();
    while (now_ns() - t0 < 2000000ull) {
    }
  }
  cluster_barrier();  // no CTA ends while a peer may still address its shared memory
}

// P[m][n] = sum_k X[m][k] U[n][k] in double (operands of type T), M = T * B rows, N = d, K = in_dim.
// 64 x 64 tiles, 16 of K per stage, 4 x 4 outputs per thread.
template <typename T>
__global__ void __launch_bounds__(256) proj_f64_kernel(const T* __restrict__ X, const T* __restrict__ U,
                                                       double* __restrict__ P, int64_t M, int N, int K) {
  __shared__ __align__(16) double Xs[16][64 + 2];
  __shared__ __align__(16) double Us[16][64 + 2];
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  const int64_t m0 = (int64_t)blockIdx.y * 64;
  const int n0 = blockIdx.x * 64;
  double acc[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += 16) {
    for (int i = threadIdx.x; i < 64 * 16; i += 256) {
      const int r = i / 16, kk = i % 16, k = k0 + kk;
      Xs[kk][r] = (m0 + r < M && k < K) ? (double)to_f(X[(m0 + r) * K + k]) : 0.0;
      Us[kk][r] = (n0 + r < N && k < K) ? (double)to_f(U[(int64_t)(n0 + r) * K + k]) : 0.0;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      double xa[4], ub[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) xa[i] = Xs[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) ub[j] = Us[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fma(xa[i], ub[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t m = m0 + ty * 4 + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n < N) P[m * N + n] = acc[i][j];
    }
  }
}

template <typename T, int NW, bool BWD>
bool launch_persistent(Launcher& lc, const PersistArgs& a) {
  static PerDevice<int> state;  // 0 = not set up yet, 1 = usable on this device, -1 = clusters of 16 not schedulable here
  int& st = state.here();
  auto kernel = rnn_persistent_kernel<T, NW, BWD>;
  constexpr int NT = NW * kKP / kCS * kKP, D = NW * kKP;
  constexpr size_t kSmem = (2 * kR * D + kKP * kR * (D / kCS)) * sizeof(double) + 32;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(((a.B + kR - 1) / kR) * kCS));
  cfg.blockDim = dim3(NT);
  cfg.dynamicSmemBytes = kSmem;
  cfg.stream = lc.stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = kCS;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (st == 0) {
    st = -1;
    int clusters = 0;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem) == cudaSuccess &&
        cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess &&
        cudaOccupancyMaxActiveClusters(&clusters, kernel, &cfg) == cudaSuccess && clusters >= 1)
      st = 1;
    cudaGetLastError();
  }
  if (st != 1) return false;
  cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, a);
  if (e != cudaSuccess && lc.err == cudaSuccess) lc.err = e;
  lc.count();
  lc.check();
  return true;
}

template <typename T, bool BWD>
bool dispatch_persistent(Launcher& lc, const PersistArgs& a) {
  switch (a.d) {
    case 128: return launch_persistent<T, 128 / kKP, BWD>(lc, a);
    case 256: return launch_persistent<T, 256 / kKP, BWD>(lc, a);
    case 512: return launch_persistent<T, 512 / kKP, BWD>(lc, a);
    default: return false;  // other widths stay on the per-step kernels
  }
}

}  // namespace

size_t rnn_persistent_proj_bytes(int T, int64_t B, int d) {
  if (d != 128 && d != 256 && d != 512) return 0;
  return (size_t)T * (size_t)B * (size_t)d * sizeof(double);
}

bool rnn_forward_persistent(Launcher& lc, int dtype, const void* W, const void* U, const void* X, const void* gate,
                            const void* x0, double* P, void* x_all, void* deriv, int T, int B, int d, int in_dim, int* status) {
  if (!P || T <= 0 || B <= 0 || (d != 128 && d != 256 && d != 512)) return false;
  PersistArgs a = {};
  a.W = W; a.gate = gate; a.P = P; a.x0 = x0; a.states = x_all; a.deriv = deriv; a.delta = nullptr; a.status = status;
  a.T = T; a.B = B; a.d = d;
  const int64_t M = (int64_t)T * B;
  dim3 grid((unsigned)((d + 63) / 64), (unsigned)((M + 63) / 64));
  // (where clusters of 16 cannot be scheduled the dispatch returns false after the projection has been enqueued:
  // harmless, the caller then runs the per-step kernels)
  if (dtype == HBP_F32) {
    proj_f64_kernel<float><<<grid, 256, 0, lc.stream>>>((const float*)X, (const float*)U, P, M, d, in_dim);
    lc.count();
    lc.check();
    return dispatch_persistent<float, false>(lc, a);
  }
  proj_f64_kernel<bf16><<<grid, 256, 0, lc.stream>>>((const bf16*)X, (const bf16*)U, P, M, d, in_dim);
  lc.count();
  lc.check();
  return dispatch_persistent<bf16, false>(lc, a);
}

bool rnn_backward_persistent(Launcher& lc, int dtype, const void* W, const void* gate, const void* deriv, const void* delta,
                             void* g_all, int T, int B, int d, int* status) {
  if (T <= 0 || B <= 0 || (d != 128 && d != 256 && d != 512)) return false;
  PersistArgs a = {};
  a.W = W; a.gate = gate; a.P = nullptr; a.x0 = nullptr; a.states = g_all; a.deriv = const_cast<void*>(deriv); a.delta = delta; a.status = status;
  a.T = T; a.B = B; a.d = d;
  if (dtype == HBP_F32) return dispatch_persistent<float, true>(lc, a);
  return dispatch_persistent<bf16, true>(lc, a);
}

}  // namespace hbp
