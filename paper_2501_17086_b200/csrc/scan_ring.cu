// Reverse scan over time for problems with few channels (Eq. 9 / Eq. 12 with diagonal K; the recurrent
// workloads: hundreds to thousands of steps, 10^4..10^5 channels).  There are too few independent recurrences
// to hide memory latency with threads, so each block hides it with a deep ring of TMA loads instead: a block
// owns 512 bytes of channels (128 floats / 256 bf16) and walks all steps serially, one 32-bit word of channels
// per lane; a producer warp keeps the ring of {8..64 steps x 512 bytes} boxes full per input stream (u, a
// separately given delta, an element-wise gate), and four consumer warps - one per scheduler, so that the
// float <-> double conversions of the running value spread over all four conversion pipes - apply
// g = a * g + u step by step and store g.  Every input byte is read once and every output byte written once,
// with no scratch, no hand-over between blocks and nothing to wait for but this block's own loads.
#include <type_traits>

#include "tc_common.cuh"

namespace hbp {

namespace {

using namespace tc;

constexpr int kMaxRows = 64;                    // steps per ring stage (one TMA box per stream): 8, 16, 32 or 64
constexpr int kSubRows = 8;                     // steps a consumer takes from shared memory at a time
constexpr int kRowBytes = 512;                  // channel bytes per block
constexpr int kRingBudget = 192 * 1024;         // shared memory an SM gives to rings, split among its blocks
constexpr int kMaxStages = 24;
constexpr int kConsumerWarps = 4;

template <typename T>
struct RingAcc {
  typedef float type;
};
template <>
struct RingAcc<float> {
  typedef double type;  // thousands of dependent steps at 1e-5: the running value is carried in double
};

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
               "l"(tm), "r"(bar), "r"(c0), "r"(c1)
               : "memory");
}

template <typename T>
__device__ __forceinline__ void unpack_word(uint32_t w, float* f);
template <>
__device__ __forceinline__ void unpack_word<float>(uint32_t w, float* f) {
  f[0] = __uint_as_float(w);
}
template <>
__device__ __forceinline__ void unpack_word<bf16>(uint32_t w, float* f) {
  f[0] = __uint_as_float(w << 16);
  f[1] = __uint_as_float(w & 0xffff0000u);
}

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* tm, uint32_t src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(tm), "r"(src), "r"(c0), "r"(c1)
               : "memory");
}

struct RingMaps {
  CUtensorMap m0, m1, mg, mc;  // loads: the additive streams, the element gate, the operand's coefficients
  CUtensorMap og, oh, ol;      // stores: g, and the two terms of the operand
};

// NS additive streams (0..2: u and/or a per-step delta), kElemGate: a gate value per element and step.
// m0, m1: maps of the additive streams, mg: map of the gate; all [steps][rows * d] with boxes of
// {512 bytes, rows_ps}.  Row y of every map is step y.
//
// Results leave the way the inputs came: a consumer puts g_l where it took u_l (or the gate, when there is no
// additive stream) from the ring, and when a stage is done the block's one control lane sends it to global memory as
// one TMA box, waits until the box has been read, and refills the slot with loads.  The serial chain (one warp per
// scheduler, thousands of dependent steps) so never issues a global store.  Only a stage that reaches below the
// first step (or, for the operand, below row 0) is stored by the threads themselves: a TMA store may not start at
// a negative coordinate, and rows outside [l_lo, l_hi) are not this call's to write.
//
// kOp (float only): a further stream mc, the coefficients of the next all-step VJP, read one step lower than the
// others (step l takes row l - 1), so that the kernel can write row l - 1 of that product's left operand
// g_l * coef_{l-1}, split into its two tf32 terms: the operand never makes a round trip through g.  Four further
// warps - again one per scheduler - turn a stage the consumers have finished into operand rows, in place over g_l
// and the coefficients; g itself is then stored only on request (by the consumers' own stores).
template <typename T, int NS, bool kElemGate, bool kOp>
__global__ void __launch_bounds__((kConsumerWarps * (kOp ? 2 : 1) + 1) * 32) scan_ring_kernel(const ScanArgs s,
                                                                                            const __grid_constant__ RingMaps m,
                                                                                            int nstages, int rows_ps) {
  typedef typename RingAcc<T>::type A;
  constexpr int EPT = 4 / (int)sizeof(T);  // channels per lane: one 32-bit word
  static_assert(!kOp || EPT == 1, "the operand by-product is a float path");
  constexpr int STREAMS = NS + (kElemGate ? 1 : 0) + (kOp ? 1 : 0);
  constexpr int OP_STREAM = STREAMS - 1;
  const int kRows = rows_ps;                       // steps per ring stage
  const int kStageBytes = rows_ps * kRowBytes;  // per stream
  extern __shared__ __align__(128) unsigned char ring_raw[];
  unsigned char* ring = reinterpret_cast<unsigned char*>(((uintptr_t)ring_raw + 127) & ~(uintptr_t)127);
  uint64_t* bars = reinterpret_cast<uint64_t*>(ring + (size_t)nstages * STREAMS * kStageBytes);
  constexpr int kBarsPerStage = 2 + (kOp ? kConsumerWarps : 0);
  int* abort_flag = reinterpret_cast<int*>(bars + kBarsPerStage * nstages);
  int* local_status = abort_flag + 1;
  auto full_bar = [&](int i) { return smem_u32(bars + i); };            // the loads of stage i have landed
  auto done_bar = [&](int i) { return smem_u32(bars + nstages + i); };  // the results of stage i are in place
  // kOp: consumer warp w has left its g values in stage i
  auto chain_bar = [&](int i, int w) { return smem_u32(bars + 2 * nstages + i * kConsumerWarps + w); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t state = s.rows * s.d;
  const int x0 = (int)((int64_t)blockIdx.x * (kRowBytes / (int)sizeof(T)));
  const int nsteps = s.l_hi - s.l_lo;
  const int niter = (nsteps + kRows - 1) / kRows;
  int* status = s.status ? s.status : local_status;
  const bool store_g = !(kOp && s.op_skip_g);
  // the lowest first step of a stage that still goes out as a box (see above)
  const int l_box = kOp ? (s.l_lo > 1 ? s.l_lo : 1) : s.l_lo;

  if (threadIdx.x == 0) {
    for (int i = 0; i < nstages; ++i) {
      mbar_init(full_bar(i), 1);
      mbar_init(done_bar(i), kConsumerWarps);
      if (kOp)
        for (int w = 0; w < kConsumerWarps; ++w) mbar_init(chain_bar(i, w), 1);
    }
    *abort_flag = 0;
    *local_status = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  __syncthreads();

  if (warp == kConsumerWarps) {
    // ---- control: one lane keeps the ring full and sends finished stages out ---------------------------------
    if (lane == 0) {
      auto load_stage = [&](int k) {
        const int slot = k % nstages;
        mbar_expect_tx(full_bar(slot), STREAMS * kStageBytes);
        const int y = s.l_hi - (k + 1) * kRows;  // may start below step 0 in the last stage: zero fill
        const uint32_t dst = smem_u32(ring + (size_t)slot * STREAMS * kStageBytes);
        if (NS >= 1) tma_load_2d(dst, &m.m0, full_bar(slot), x0, y);
        if (NS >= 2) tma_load_2d(dst + kStageBytes, &m.m1, full_bar(slot), x0, y);
        if (kElemGate) tma_load_2d(dst + NS * kStageBytes, &m.mg, full_bar(slot), x0, y);
        if (kOp) tma_load_2d(dst + OP_STREAM * kStageBytes, &m.mc, full_bar(slot), x0, y - 1);  // rows below 0: zero fill
      };
      int issued = 0, taken = 0;
      for (; issued < niter && issued < nstages; ++issued) load_stage(issued);
      for (int k = 0; k < niter; ++k) {
        const int slot = k % nstages;
        if (!mbar_wait(done_bar(slot), (uint32_t)((k / nstages) & 1), abort_flag, status)) break;
        taken = k + 1;
        const int l_base = s.l_hi - (k + 1) * kRows;
        if (l_base >= l_box) {
          const uint32_t src = smem_u32(ring + (size_t)slot * STREAMS * kStageBytes);
          if (kOp) {
            tma_store_2d(&m.oh, src, x0, l_base - 1);
            tma_store_2d(&m.ol, src + OP_STREAM * kStageBytes, x0, l_base - 1);
          } else {
            tma_store_2d(&m.og, src, x0, l_base);
          }
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          tma_store_wait_read();  // the slot may be overwritten once the box has been read out of it
        }
        if (issued < niter) load_stage(issued++);
      }
      // nothing of this block may still be in flight when it ends: loads that no one took (only after an abort) ...
      for (int k = taken; k < issued; ++k) {
        const uint64_t t0 = global_ns();
        while (!mbar_try_wait(full_bar(k % nstages), (uint32_t)((k / nstages) & 1)))
          if (global_ns() - t0 > WAIT_LIMIT_NS) {  // a copy that never landed: say so, then leave
            atomicExch(status, (int)HBP_ERR_TIMEOUT);
            break;
          }
      }
      tma_store_wait_all();  // ... and the boxes on their way out
    }
    return;
  }

  if (kOp && warp > kConsumerWarps) {
    // ---- operand warps: warp w takes the words of consumer warp w; row l - 1 of the operand is g_l * coef_{l-1} ----
    const int cw = warp - kConsumerWarps - 1;
    const int word = cw * 32 + lane;
    const int64_t e0 = (int64_t)x0 + word;
    const bool live = e0 < state;
    auto split = [](float gl, float coef, float& h, float& l) {
      const float v = gl * coef;
      h = round_tf32(v);
      l = round_tf32(v - h);
    };
    if (live && s.l_hi >= 1) {  // the top row comes from the carry-in
      float h, l;
      split(((const float*)s.g)[(int64_t)s.l_hi * state + e0], s.op_coef[(int64_t)(s.l_hi - 1) * state + e0], h, l);
      s.op_hi[(int64_t)(s.l_hi - 1) * state + e0] = h;
      s.op_lo[(int64_t)(s.l_hi - 1) * state + e0] = l;
    }
    for (int k = 0; k < niter; ++k) {
      const int slot = k % nstages;
      if (!mbar_wait(chain_bar(slot, cw), (uint32_t)((k / nstages) & 1), abort_flag, status)) break;
      unsigned char* stg = ring + (size_t)slot * STREAMS * kStageBytes + word * 4;
      const int l_base = s.l_hi - (k + 1) * kRows;
      const bool box = l_base >= l_box;  // else: this stage reaches below the first row, its rows go out one by one
#pragma unroll 1
      for (int sb = kRows / kSubRows - 1; sb >= 0; --sb) {
        unsigned char* sub = stg + sb * kSubRows * kRowBytes;
        float hh[kSubRows], ll[kSubRows];
#pragma unroll
        for (int r = 0; r < kSubRows; ++r)
          split(*reinterpret_cast<const float*>(sub + r * kRowBytes),
                *reinterpret_cast<const float*>(sub + OP_STREAM * kStageBytes + r * kRowBytes), hh[r], ll[r]);
        if (box) {
#pragma unroll
          for (int r = 0; r < kSubRows; ++r) {
            *reinterpret_cast<float*>(sub + r * kRowBytes) = hh[r];
            *reinterpret_cast<float*>(sub + OP_STREAM * kStageBytes + r * kRowBytes) = ll[r];
          }
        } else {
#pragma unroll
          for (int r = kSubRows - 1; r >= 0; --r) {
            const int l = l_base + sb * kSubRows + r;
            if (live && l >= l_box) {
              s.op_hi[(int64_t)(l - 1) * state + e0] = hh[r];
              s.op_lo[(int64_t)(l - 1) * state + e0] = ll[r];
            }
          }
        }
      }
      fence_async_smem();  // the box is read by the async proxy
      __syncwarp();
      if (lane == 0) mbar_arrive(done_bar(slot));
    }
    return;
  }

  // ---- consumers: warp w owns 32-bit words [32 w, 32 (w + 1)) of the block's 512-byte row ---------------
  const int word = warp * 32 + lane;
  const int64_t e0 = (int64_t)x0 + (int64_t)word * EPT;
  const bool live = e0 < state;
  T* g = (T*)s.g;
  A carry[EPT];
  float a0[EPT];
#pragma unroll
  for (int e = 0; e < EPT; ++e) {
    carry[e] = live ? (A)to_f(g[(int64_t)s.l_hi * state + e0 + e]) : (A)0;
    a0[e] = 1.0f;
  }
  if (!kElemGate && live && s.a && s.gate == HBP_GATE_CHANNEL_SHARED) {
#pragma unroll
    for (int e = 0; e < EPT; ++e) a0[e] = to_f(((const T*)s.a)[(e0 + e) % s.d]);
  }
  T* gp = g + (int64_t)(s.l_hi - 1) * state + e0;  // where the next step's value goes
  // kSub rows of one stage, later steps first.  direct = the threads store g themselves (a stage that reaches below
  // the first step, where they also stop there; or g wanted beside the operand)
  auto sub_block = [&](unsigned char* stg, int l_top, auto direct_t, auto check_t) {
    constexpr bool kDirect = decltype(direct_t)::value, kCheck = decltype(check_t)::value;
    float uu[kSubRows][EPT], aa[kSubRows][EPT];
#pragma unroll
    for (int r = 0; r < kSubRows; ++r) {
#pragma unroll
      for (int e = 0; e < EPT; ++e) {
        uu[r][e] = 0.0f;
        aa[r][e] = a0[e];
      }
      if (NS >= 1) unpack_word<T>(*reinterpret_cast<const uint32_t*>(stg + r * kRowBytes), uu[r]);
      if (NS >= 2) {
        float t[EPT];
        unpack_word<T>(*reinterpret_cast<const uint32_t*>(stg + kStageBytes + r * kRowBytes), t);
#pragma unroll
        for (int e = 0; e < EPT; ++e) uu[r][e] += t[e];
      }
      if (kElemGate) unpack_word<T>(*reinterpret_cast<const uint32_t*>(stg + NS * kStageBytes + r * kRowBytes), aa[r]);
    }
#pragma unroll
    for (int r = kSubRows - 1; r >= 0; --r) {
      if (kCheck && l_top - (kSubRows - 1 - r) < s.l_lo) break;
#pragma unroll
      for (int e = 0; e < EPT; ++e) carry[e] = (A)aa[r][e] * carry[e] + (A)uu[r][e];
      uint32_t out;  // g_l as it is stored: one float, or two bf16
      if (EPT == 1) {
        out = __float_as_uint((float)carry[0]);
      } else {
        const __nv_bfloat162 b2 = __floats2bfloat162_rn((float)carry[0], (float)carry[EPT - 1]);
        out = *reinterpret_cast<const uint32_t*>(&b2);
      }
      if (kDirect && live) *reinterpret_cast<uint32_t*>(gp) = out;
      gp -= state;
      // left in the first stream's place: for the box that goes out, or for the operand warps
      if (!kDirect || kOp) *reinterpret_cast<uint32_t*>(stg + r * kRowBytes) = out;
    }
  };
  for (int k = 0; k < niter; ++k) {
    const int slot = k % nstages;
    if (!mbar_wait(full_bar(slot), (uint32_t)((k / nstages) & 1), abort_flag, status)) break;
    unsigned char* stg = ring + (size_t)slot * STREAMS * kStageBytes + word * 4;
    const int l_base = s.l_hi - (k + 1) * kRows;
    if (l_base < s.l_lo) {
#pragma unroll 1
      for (int sb = kRows / kSubRows - 1; sb >= 0; --sb) {
        if (store_g) sub_block(stg + sb * kSubRows * kRowBytes, l_base + sb * kSubRows + kSubRows - 1, std::true_type(), std::true_type());
        else sub_block(stg + sb * kSubRows * kRowBytes, l_base + sb * kSubRows + kSubRows - 1, std::false_type(), std::true_type());
      }
    } else if (kOp ? store_g : l_base < l_box) {
#pragma unroll 1
      for (int sb = kRows / kSubRows - 1; sb >= 0; --sb)
        sub_block(stg + sb * kSubRows * kRowBytes, l_base + sb * kSubRows + kSubRows - 1, std::true_type(), std::false_type());
    } else {
#pragma unroll 1
      for (int sb = kRows / kSubRows - 1; sb >= 0; --sb)
        sub_block(stg + sb * kSubRows * kRowBytes, l_base + sb * kSubRows + kSubRows - 1, std::false_type(), std::false_type());
    }
    if (!kOp) fence_async_smem();  // the box is read by the async proxy
    __syncwarp();
    if (lane == 0) mbar_arrive(kOp ? chain_bar(slot, warp) : done_bar(slot));
  }
}

bool make_map2(CUtensorMap* tm, const void* base, bool f32, int64_t steps, int64_t state, int rows_ps) {
  EncodeTiledFn fn = encode_fn();
  if (!fn || ((uintptr_t)base & 15u)) return false;
  const cuuint64_t es = f32 ? 4 : 2;
  if ((state * es) % 16) return false;
  cuuint64_t dims[2] = {(cuuint64_t)state, (cuuint64_t)steps};
  cuuint64_t strides[1] = {(cuuint64_t)state * es};
  cuuint32_t box[2] = {(cuuint32_t)(kRowBytes / es), (cuuint32_t)rows_ps}, estr[2] = {1, 1};
  return fn(tm, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims,
            strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <typename T, int NS, bool kElemGate, bool kOp>
void launch_ring(Launcher& lc, const ScanArgs& s, const RingMaps& m, unsigned grid, int nstages, int rows_ps, size_t smem) {
  static PerDevice<size_t> configured_on;  // per-device kernel attribute
  size_t& configured = configured_on.here();
  if (smem > configured) {
    cudaFuncSetAttribute(scan_ring_kernel<T, NS, kElemGate, kOp>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    configured = smem;
  }
  scan_ring_kernel<T, NS, kElemGate, kOp>
      <<<grid, (kConsumerWarps * (kOp ? 2 : 1) + 1) * 32, smem, lc.stream>>>(s, m, nstages, rows_ps);
  lc.count();
  lc.check();
}

template <typename T>
void dispatch_ring(Launcher& lc, const ScanArgs& s, int ns, bool eg, bool op, const RingMaps& m, unsigned grid, int nstages,
                   int rows_ps, size_t smem) {
  if constexpr (std::is_same<T, float>::value) {
    if (op) {  // never together with an element gate (see scan_ring)
      if (ns == 1) launch_ring<T, 1, false, true>(lc, s, m, grid, nstages, rows_ps, smem);
      else launch_ring<T, 2, false, true>(lc, s, m, grid, nstages, rows_ps, smem);
      return;
    }
  }
  if (eg) {
    if (ns == 0) launch_ring<T, 0, true, false>(lc, s, m, grid, nstages, rows_ps, smem);
    else if (ns == 1) launch_ring<T, 1, true, false>(lc, s, m, grid, nstages, rows_ps, smem);
    else launch_ring<T, 2, true, false>(lc, s, m, grid, nstages, rows_ps, smem);
  } else {
    if (ns == 1) launch_ring<T, 1, false, false>(lc, s, m, grid, nstages, rows_ps, smem);
    else launch_ring<T, 2, false, false>(lc, s, m, grid, nstages, rows_ps, smem);
  }
}

}  // namespace

bool scan_ring(Launcher& lc, const ScanArgs& s) {
  if (s.xhat || s.keep != 1.0f || s.gamma != 0.0f) return false;
  if (s.gate == HBP_GATE_CHANNEL_PER_STEP && s.a) return false;  // a small [steps][d] table: not a stream of this shape
  const bool f32 = s.dtype == HBP_F32;
  const int64_t state = s.rows * s.d;
  const int nsteps = s.l_hi - s.l_lo;
  if (nsteps < 4 * kSubRows || state <= 0 || state > 0x7fffffff) return false;
  const int row_elems = kRowBytes / (f32 ? 4 : 2);
  const unsigned grid = (unsigned)((state + row_elems - 1) / row_elems);
  // the additive streams: u, and delta when it is given per step and not already inside u
  const void* streams[2] = {nullptr, nullptr};
  int64_t stream_rows[2] = {0, 0};
  int ns = 0;
  if (s.u) {
    streams[ns] = s.u;
    stream_rows[ns++] = s.L;
  }
  if (s.delta && s.loss == HBP_LOSS_EVERY_STEP && !(s.u && s.u_has_delta)) {
    streams[ns] = s.delta;
    stream_rows[ns++] = (int64_t)s.L + 1;
  }
  const bool eg = s.a && s.gate == kGateElement;
  if (ns == 0 && !eg) return false;  // nothing to stream: a pure broadcast
  // the operand by-product: float, a constant gate, and at least one additive stream to ride along with
  const bool op = f32 && !eg && ns >= 1 && s.op_coef && s.op_hi && s.op_lo;
  const int nstreams = ns + (eg ? 1 : 0) + (op ? 1 : 0);
  const int sms = sm_count();
  int per_sm = (int)((grid + sms - 1) / sms);
  if (per_sm > 4) per_sm = 4;
  // the longest stage (fewest producer round trips) that still leaves a ring of at least four stages
  const int budget = kRingBudget / per_sm / nstreams;
  int rows_ps = kMaxRows;
  while (rows_ps > kSubRows && (budget / (rows_ps * kRowBytes) < 4 || nsteps < 2 * rows_ps)) rows_ps /= 2;
  int nstages = budget / (rows_ps * kRowBytes);
  const int niter = (nsteps + rows_ps - 1) / rows_ps;
  if (nstages > niter) nstages = niter;
  if (nstages > kMaxStages) nstages = kMaxStages;
  if (nstages < 2) return false;
  RingMaps m;
  if (ns >= 1 && !make_map2(&m.m0, streams[0], f32, stream_rows[0], state, rows_ps)) return false;
  if (ns >= 2 && !make_map2(&m.m1, streams[1], f32, stream_rows[1], state, rows_ps)) return false;
  if (eg && !make_map2(&m.mg, s.a, f32, s.L, state, rows_ps)) return false;
  if (op && !make_map2(&m.mc, s.op_coef, true, s.L, state, rows_ps)) return false;
  if (ns == 0) m.m0 = m.mg;  // unused maps still have to be valid objects
  if (ns < 2) m.m1 = m.m0;
  if (!eg) m.mg = m.m0;
  if (!op) m.mc = m.m0;
  // the ways out: g [L + 1 rows], and the operand's two terms [L rows]
  if (!make_map2(&m.og, s.g, f32, (int64_t)s.L + 1, state, rows_ps)) return false;
  if (op && (!make_map2(&m.oh, s.op_hi, true, s.L, state, rows_ps) || !make_map2(&m.ol, s.op_lo, true, s.L, state, rows_ps)))
    return false;
  if (!op) m.oh = m.ol = m.og;
  const size_t smem = (size_t)nstages * nstreams * rows_ps * kRowBytes + (size_t)nstages * (op ? 16 + 8 * kConsumerWarps : 16) + 16 + 128;
  if (f32) dispatch_ring<float>(lc, s, ns, eg, op, m, grid, nstages, rows_ps, smem);
  else dispatch_ring<bf16>(lc, s, ns, eg, false, m, grid, nstages, rows_ps, smem);
  if (op && s.op_done) *s.op_done = true;
  return true;
}

}  // namespace hbp
