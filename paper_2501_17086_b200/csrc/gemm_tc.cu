// bf16 GEMM on the 5th-generation tensor cores: tcgen05.mma with the accumulator in tensor memory,
// operands staged in shared memory by TMA (128-byte swizzle), fused epilogues read back with tcgen05.ld.
//
//   D(m, n) = sum_k A(m, k) B(n, k), fp32 accumulate, batched (one launch covers all layers of a group).
//
// Persistent kernel, one CTA per SM, 320 threads:
//   warp 0      TMA producer (one lane): fills a 4-stage ring of {A 128x64, B 256x64} bf16 tiles
//   warp 1      MMA issuer (one lane): 4 x tcgen05.mma 128x256x16 per stage; owns the TMEM allocation
//   warps 2..9  epilogue: two warps per 32-lane TMEM quarter, 128 accumulator columns each; each warp
//               stages 32-row chunks through a private 4 KB swizzled buffer, so every global access of
//               the epilogue is a TMA tile copy (the cached gelu' in, the result out)
// The 512 TMEM columns hold two 128x256 fp32 accumulators, so the epilogue of tile i overlaps the main
// loop of tile i+1.  Either operand may be K-major (contraction index contiguous in memory) or MN-major
// (row/column index contiguous); both are supported natively through the matrix descriptors, so neither
// weights nor activations are ever transposed in memory.
//
// Every wait on an mbarrier is bounded: after ~4 s it raises a shared abort flag, records
// HBP_ERR_TIMEOUT in the status word, and all roles drain and leave through the common exit that
// frees the tensor memory.
#include "tc_common.cuh"

namespace hbp {

using namespace tc;

namespace {

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int A_BYTES = BM * BK * 2;
// Single CTA: a 128 x 256 tile, stages of {A 128 x 64, B 256 x 64} (B 64 or 128 rows for a product at most that wide).
// CTA pair (two CTAs of a cluster on one 256 x 256 tile, tcgen05 cta_group::2): each CTA stages its own 128 rows of A
// and its own 128 of the 256 columns of B, so a stage is 32 KB instead of 48 KB for the same flops per SM, and six
// stages fit.
template <bool kPair>
struct Mode {
  static constexpr int kBRows = kPair ? 128 : 256;
  static constexpr int kTileM = kPair ? 256 : 128;
};
constexpr int PAIR_STAGES = 6, PAIR_STAGE_BYTES = A_BYTES + 128 * BK * 2;
constexpr int RING_BYTES = 4 * (A_BYTES + 256 * BK * 2);  // = 6 stages of the pair mode
constexpr int EPI_WARPS = 8, THREADS = 64 + 32 * EPI_WARPS;
constexpr uint32_t TMEM_COLS = 512;
constexpr int EPI_BUF_BYTES = 4096;  // 32 rows x 128 bytes per epilogue warp
constexpr int SMEM_BYTES = RING_BYTES + EPI_WARPS * EPI_BUF_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;

struct TcParams {
  int M, N, K, batch;
  int m_tiles, n_tiles, num_tiles, k_blocks;
  int a_mn, b_mn;  // 1: the operand is MN-major
  int tf32;        // operands are float, multiplied as tf32 (else bf16)
  int n_mma;       // columns one MMA covers: 256, or 64 / 128 for a narrow single-CTA product (N <= 128), whose B tiles,
                   // instructions and epilogue then leave the padding columns out
  int segs;        // K segments, each with its own pair of operand maps (3 for the split-float product)
  int splits, kb_per_split;  // split-K: tile z index = split * batch + b; each split covers kb_per_split k-blocks
  int epi, d_f32;
  void* D; int64_t ldd, d_sb;
  void* D2; int64_t ldd2, d2_sb;
  const void* E; int64_t lde, e_sb;
  const void* gate; int64_t gate_sb;
  float* R;
  float2* stats; int64_t stats_sb;
  int* status;
  uint64_t wait_limit_ns;  // limit of every barrier wait
  int stall;               // self-test of the bounded waits only: the producer arms its first stage and copies nothing
};

// ------------------------------------------------------------------------------------------- epilogue math
// Phi(z) and the normal density for bf16 outputs: erf by Abramowitz & Stegun 7.1.26 (|error| < 1.5e-7),
// sharing exp(-z^2/2) between erf and the density; the tail is formed without cancellation.
__device__ __forceinline__ void normal_cdf_pdf(float z, float& cdf, float& pdf) {
  const float ax = fabsf(z) * 0.70710678118654752440f;
  float t;  // 1 / (1 + p |z| / sqrt 2) by the hardware reciprocal (relative error 2^-23: far below the formula's own)
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t) : "f"(fmaf(0.3275911f, ax, 1.0f)));
  const float e = __expf(-0.5f * z * z);
  float poly = fmaf(t, 1.061405429f, -1.453152027f);
  poly = fmaf(t, poly, 1.421413741f);
  poly = fmaf(t, poly, -0.284496736f);
  poly = fmaf(t, poly, 0.254829592f);
  const float half_tail = 0.5f * poly * t * e;  // 0.5 * erfc(|z| / sqrt 2)
  cdf = z < 0.0f ? half_tail : 1.0f - half_tail;
  pdf = e * 0.39894228040143267794f;
}

// Residual update of the forward pass, written straight from registers (not on the hot path):
// one thread owns `row` and the 32 accumulator columns starting at col0.
__device__ __forceinline__ void residual_chunk(const TcParams& p, int b, int row, int col0, float* v) {
  if (row >= p.M) return;
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    const int col = col0 + 8 * g;
    if (col >= p.N) break;  // N is a multiple of 8: groups are all-in or all-out
    float* a = v + 8 * g;
    float gt[8], r[8];
    if (p.gate) {
      unpack8(*reinterpret_cast<const uint4*>((const bf16*)p.gate + (int64_t)b * p.gate_sb + col), gt);
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) gt[i] = 1.0f;
    }
    if (p.R) {
      float4* rp = reinterpret_cast<float4*>(p.R + (int64_t)row * p.N + col);
      const float4 r0 = rp[0], r1 = rp[1];
      r[0] = r0.x; r[1] = r0.y; r[2] = r0.z; r[3] = r0.w;
      r[4] = r1.x; r[5] = r1.y; r[6] = r1.z; r[7] = r1.w;
#pragma unroll
      for (int i = 0; i < 8; ++i) a[i] = fmaf(gt[i], r[i], a[i]);
      rp[0] = make_float4(a[0], a[1], a[2], a[3]);
      rp[1] = make_float4(a[4], a[5], a[6], a[7]);
    } else {
      unpack8(*reinterpret_cast<const uint4*>((const bf16*)p.E + (int64_t)b * p.e_sb + (int64_t)row * p.lde + col), r);
#pragma unroll
      for (int i = 0; i < 8; ++i) a[i] = fmaf(gt[i], r[i], a[i]);
    }
    *reinterpret_cast<uint4*>((bf16*)p.D + (int64_t)b * p.d_sb + (int64_t)row * p.ldd + col) = pack8(a);
  }
}

// ------------------------------------------------------------------------------------------- kernel
template <bool kPair, bool kTf32>
__global__ void __launch_bounds__(THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmA1, const __grid_constant__ CUtensorMap tmB1,
               const __grid_constant__ CUtensorMap tmA2, const __grid_constant__ CUtensorMap tmB2,
               const __grid_constant__ CUtensorMap tmD, const __grid_constant__ CUtensorMap tmD2,
               const __grid_constant__ CUtensorMap tmE, const TcParams p) {
  // single CTAs size their stages by the B tile they load (a narrow product: 64 or 128 rows instead of 256), so the
  // same 192 KB ring is 4, 6 or 8 stages deep: the bytes in flight, not the stage count, hide the load latency
  constexpr int MAX_STAGES = 8;
  const int STAGE_BYTES = kPair ? PAIR_STAGE_BYTES : A_BYTES + p.n_mma * 128;
  const int STAGES = kPair ? PAIR_STAGES : RING_BYTES / STAGE_BYTES;
  constexpr int B_ROWS = Mode<kPair>::kBRows, TILE_M = Mode<kPair>::kTileM;
  // pair mode: rank of this CTA in its pair; the even CTA (leader) owns the pipeline's full barriers and
  // issues the MMAs, its peer's tile loads signal the leader's barriers
  const uint32_t rank = kPair ? cluster_ctarank() : 0u;
  const bool leader = rank == 0;
  const int first_tile = kPair ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int tile_step = kPair ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  extern __shared__ uint8_t smem_raw[];
  // the swizzled tiles need 1024-byte alignment
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* aligned = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t epi_base = base + RING_BYTES;  // EPI_WARPS x 4 KB, each 1024-byte aligned
  uint64_t* bars = reinterpret_cast<uint64_t*>(aligned + RING_BYTES + EPI_WARPS * EPI_BUF_BYTES);
  // with S = MAX_STAGES: bars[0..S) full, [S..2S) empty, [2S..2S+2) accumulator full, [2S+2..2S+4) accumulator empty,
  // [2S+4] drain, [2S+5 .. 2S+5+EPI_WARPS) one per epilogue warp for its staged operand loads
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (MAX_STAGES + s); };
  auto accf_bar = [&](int a) { return bar0 + 8u * (2 * MAX_STAGES + a); };
  auto acce_bar = [&](int a) { return bar0 + 8u * (2 * MAX_STAGES + 2 + a); };
  const uint32_t drain_bar = bar0 + 8u * (2 * MAX_STAGES + 4);
  auto epi_bar = [&](int w) { return bar0 + 8u * (2 * MAX_STAGES + 5 + w); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * MAX_STAGES + 5 + EPI_WARPS);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(accf_bar(a), 1);
      mbar_init(acce_bar(a), kPair ? 2 * EPI_WARPS : EPI_WARPS);  // pair: both CTAs' epilogue warps arrive at the leader
    }
    mbar_init(drain_bar, 1);
    for (int w = 0; w < EPI_WARPS; ++w) mbar_init(epi_bar(w), 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    if (kPair) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                   "r"(TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                   "r"(TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if (kPair) cluster_sync();  // the peer's barriers and tensor memory exist before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int tiles_per_batch = p.m_tiles * p.n_tiles;
  // per element size: elements per 128-byte row (= K elements per stage), bytes of one MN-major block
  const int row_elems = kTf32 ? 32 : 64;
  const uint32_t mn_block = kTf32 ? 4096u : 8192u;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      uint32_t issued_mask = 0, issued_parity = 0;
      bool ok = true;
      for (int tile = first_tile; tile < p.num_tiles && ok; tile += tile_step) {
        const int zc = tile / tiles_per_batch, r = tile % tiles_per_batch;
        const int b = zc % p.batch, split = zc / p.batch;
        // n fastest: a wave shares few A row-panels.  This CTA's rows of A and (pair) its half of B's columns
        const int m0 = (r / p.n_tiles) * TILE_M + (int)rank * BM, n0 = (r % p.n_tiles) * BN + (int)rank * (BN - B_ROWS);
        const int kb_lo = split * p.kb_per_split, kb_hi = min(p.k_blocks, kb_lo + p.kb_per_split);
        for (int seg = 0; seg < p.segs && ok; ++seg) {
          const CUtensorMap* mA = seg == 0 ? &tmA : (seg == 1 ? &tmA1 : &tmA2);
          const CUtensorMap* mB = seg == 0 ? &tmB : (seg == 1 ? &tmB1 : &tmB2);
          for (int kb = kb_lo; kb < kb_hi; ++kb) {
            if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status, p.wait_limit_ns)) { ok = false; break; }
            const uint32_t sA = base + stage * STAGE_BYTES, sB = sA + A_BYTES;
            // pair: all four tile loads of a stage (two per CTA) complete on the leader's barrier
            const uint32_t fb = kPair ? map_to_cta(full_bar(stage), 0) : full_bar(stage);
            if (leader) mbar_expect_tx(full_bar(stage), kPair ? 2 * STAGE_BYTES : A_BYTES + p.n_mma * 128);
            issued_mask |= 1u << stage;
            issued_parity = (issued_parity & ~(1u << stage)) | (phase << stage);
            if (p.stall) { ok = false; break; }  // self-test: bytes are expected that nobody sends
            const int k0 = kb * row_elems;
            auto load = [&](uint32_t dst, const CUtensorMap* tm, int c0, int c1) {
              if (kPair) tma_load_3d_pair(dst, tm, fb, c0, c1, b);
              else tma_load_3d(dst, tm, fb, c0, c1, b);
            };
            if (p.a_mn) {
              for (int i = 0; i < BM / row_elems; ++i) load(sA + i * mn_block, mA, m0 + row_elems * i, k0);
            } else {
              load(sA, mA, k0, m0);
            }
            if (p.b_mn) {
              for (int i = 0; i < (kPair ? B_ROWS : p.n_mma) / row_elems; ++i) load(sB + i * mn_block, mB, n0 + row_elems * i, k0);
            } else {
              load(sB, mB, k0, n0);
            }
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
          }
        }
      }
      if (!ok && leader) {
        // leave no copy of ours in flight: wait (bounded) for every stage armed last
        for (int s = 0; s < STAGES; ++s)
          if (issued_mask & (1u << s)) {
            uint64_t t0 = global_ns();
            const uint64_t lim = p.wait_limit_ns < 100000000ull ? p.wait_limit_ns : 100000000ull;
            while (!mbar_try_wait(full_bar(s), (issued_parity >> s) & 1u) && global_ns() - t0 < lim) {
            }
          }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    // The whole warp runs this loop converged (waits, tests and address arithmetic in every lane, which lets the
    // compiler keep them on the uniform datapath); only the tcgen05 instructions are predicated on one elected lane.
    if (leader) {
      uint32_t elected;
      asm volatile("{\n\t.reg .pred q;\n\telect.sync _|q, 0xffffffff;\n\tselp.u32 %0, 1, 0, q;\n\t}" : "=r"(elected));
      const bool issuer = elected != 0;
      const uint32_t fmt = kTf32 ? 2u : 1u;  // operand format: tf32 or bf16
      const uint32_t idesc = (1u << 4) /*fp32 accumulate*/ | (fmt << 7) | (fmt << 10) | ((uint32_t)p.a_mn << 15) |
                             ((uint32_t)p.b_mn << 16) | ((uint32_t)((kPair ? BN : p.n_mma) >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24);
      // one instruction consumes 32 bytes of K: 32 bytes along a K-major row, or 16 rows of an MN-major bf16 block.
      // Descriptors differ between stages and k-steps only in their start address (bits 0..13, in 16-byte units):
      // they are formed once and advanced by adding to the low word.
      const uint32_t a_step16 = (p.a_mn ? 2048u : 32u) >> 4, b_step16 = (p.b_mn ? 2048u : 32u) >> 4;
      const uint64_t adesc0 = make_desc(base, p.a_mn ? mn_block : 16u, 1024u);
      const uint64_t bdesc0 = make_desc(base + A_BYTES, p.b_mn ? mn_block : 16u, 1024u);
      const uint32_t kStage16 = (uint32_t)STAGE_BYTES >> 4;
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      // The tensor core idles whenever this thread takes longer between two MMAs than one MMA runs, so nothing that
      // has to wait for an answer sits between them: the barrier of the NEXT stage (and of the next tile's
      // accumulator) is only tested, without blocking, before the current stage's MMAs go out, and the answer is
      // looked at afterwards; the blocking wait is the fallback when that test said "not yet".
      bool stage_ready = false, acc_ready = false;
      for (int tile = first_tile; tile < p.num_tiles && ok; tile += tile_step) {
        if (!acc_ready && !mbar_wait(acce_bar(acc), acc_phase ^ 1u, abort_flag, p.status, p.wait_limit_ns)) { ok = false; break; }
        acc_ready = false;
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)acc * BN;
        const int split = (tile / tiles_per_batch) / p.batch;
        const int kb_lo = split * p.kb_per_split, kb_hi = min(p.k_blocks, kb_lo + p.kb_per_split);
        uint32_t accum = 0;
        const int n_it = (kb_hi - kb_lo) * p.segs;
        for (int it = 0; it < n_it; ++it) {
          if (!stage_ready && !mbar_wait(full_bar(stage), phase, abort_flag, p.status, p.wait_limit_ns)) { ok = false; break; }
          const int next_stage = stage + 1 == STAGES ? 0 : stage + 1;
          const uint32_t next_phase = next_stage == 0 ? phase ^ 1u : phase;
          const bool peek = mbar_test_wait(full_bar(next_stage), next_phase);
          bool peek_acc = false;
          if (it == n_it - 1) peek_acc = mbar_test_wait(acce_bar(acc ^ 1), (acc == 1 ? acc_phase ^ 1u : acc_phase) ^ 1u);
          const uint64_t ad = adesc0 + (uint64_t)((uint32_t)stage * kStage16), bd = bdesc0 + (uint64_t)((uint32_t)stage * kStage16);
          if (issuer) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const uint64_t adk = ad + (uint64_t)(k * a_step16), bdk = bd + (uint64_t)(k * b_step16);
              const uint32_t acc_k = k == 0 ? accum : 1u;
              if (kPair) {
                if (kTf32) tc_mma_tf32_pair(tmem_d, adk, bdk, idesc, acc_k);
                else tc_mma_pair(tmem_d, adk, bdk, idesc, acc_k);
              } else {
                if (kTf32) tc_mma_tf32(tmem_d, adk, bdk, idesc, acc_k);
                else tc_mma(tmem_d, adk, bdk, idesc, acc_k);
              }
            }
            // frees the stage (in both CTAs of a pair) once these MMAs have read it
            if (kPair) tc_commit_pair(empty_bar(stage));
            else tc_commit(empty_bar(stage));
          }
          accum = 1;
          stage_ready = peek;
          if (it == n_it - 1) acc_ready = peek_acc;
          stage = next_stage;
          phase = next_phase;
        }
        if (!ok) break;
        if (issuer) {
          if (kPair) tc_commit_pair(accf_bar(acc));  // accumulator complete (each CTA holds its 128 rows of it)
          else tc_commit(accf_bar(acc));
        }
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
      if (!ok) {  // let issued MMAs finish before the tensor memory is freed
        if (issuer) {
          if (kPair) tc_commit_pair(drain_bar);
          else tc_commit(drain_bar);
        }
        uint64_t t0 = global_ns();
        while (!mbar_try_wait(drain_bar, 0) && global_ns() - t0 < 100000000ull) {
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int quarter = warp & 3, half = (warp - 2) >> 2, ew = warp - 2;
    const uint32_t buf = epi_base + ew * EPI_BUF_BYTES;
    const uint32_t ebar = epi_bar(ew);
    uint32_t e_phase = 0;
    bool e_pending = false;  // lane 0: a staged operand load is in flight
    int acc = 0;
    uint32_t acc_phase = 0;
    const bool staged = p.epi != EPI_RESID;
    const bool has_e = p.epi == EPI_MUL || p.epi == EPI_STORE_LN || p.epi == EPI_ADD;
    const int cw = p.d_f32 ? 32 : 64;      // accumulator columns per staged chunk (128 bytes of output per row)
    // columns of this warp's half that the MMAs write: a narrow product leaves the rest of the tile out
    const int my_cols = min(128, max(0, (kPair ? BN : p.n_mma) - half * 128));
    const int nchunks = (my_cols + cw - 1) / cw;
    const uint32_t acce_target[2] = {kPair ? map_to_cta(acce_bar(0), 0) : acce_bar(0),
                                     kPair ? map_to_cta(acce_bar(1), 0) : acce_bar(1)};
    auto release_acc = [&](int a) {
      if (kPair) mbar_arrive_cluster(acce_target[a]);
      else mbar_arrive(acce_bar(a));
    };
    for (int tile = first_tile; tile < p.num_tiles; tile += tile_step) {
      // b indexes the outputs: with split-K it is split * batch + batch entry (partial sums [split][batch][M][N])
      const int b = tile / tiles_per_batch, r = tile % tiles_per_batch;
      const int m0 = (r / p.n_tiles) * TILE_M + (int)rank * BM, n0 = (r % p.n_tiles) * BN;  // this CTA's 128 rows
      const int row0 = m0 + quarter * 32, colw = n0 + half * 128;
      if (has_e && lane == 0 && nchunks > 0) {  // the buffer is free here: fetch the first chunk of E while the MMAs still run
        mbar_expect_tx(ebar, EPI_BUF_BYTES);
        tma_load_3d(buf, &tmE, ebar, colw, row0, b);
        e_pending = true;
      }
      if (!mbar_wait(accf_bar(acc), acc_phase, abort_flag, p.status, p.wait_limit_ns)) break;
      tc_fence_after();
      const uint32_t tsrc = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN + half * 128);
      if (nchunks == 0) {  // nothing of a narrow product in this half: only hand the accumulator back
        tc_fence_before();
        __syncwarp();
        if (lane == 0) release_acc(acc);
      } else if (!staged) {
#pragma unroll 1
        for (int c = 0; c < (my_cols + 31) / 32; ++c) {
          float v[32];
          tc_ld32(tsrc + c * 32, v);
          residual_chunk(p, b, row0 + lane, colw + c * 32, v);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) release_acc(acc);
      } else {
        bool ok = true;
        float s1 = 0.0f, s2 = 0.0f;  // EPI_STORE_LN: row sums of acc and acc * E over the current 64 columns
#pragma unroll 1
        for (int c = 0; c < nchunks; ++c) {
          float v[64];
          tc_ld32(tsrc + c * cw, v);
          if (!p.d_f32) tc_ld32(tsrc + c * cw + 32, v + 32);
          if (c == nchunks - 1) {  // last read of this accumulator: hand it back to the MMA warp
            tc_fence_before();
            __syncwarp();
            if (lane == 0) release_acc(acc);
          }
          const int col = colw + c * cw;
          if (has_e) {
            if (!mbar_wait(ebar, e_phase, abort_flag, p.status, p.wait_limit_ns)) { ok = false; break; }
            e_phase ^= 1u;
            e_pending = false;
            if (p.epi == EPI_ADD) {  // float tile: 32 columns
#pragma unroll
              for (int u = 0; u < 8; ++u) {
                const uint4 raw = ld_shared16(swz(buf, lane, u));
                v[4 * u] += __uint_as_float(raw.x);
                v[4 * u + 1] += __uint_as_float(raw.y);
                v[4 * u + 2] += __uint_as_float(raw.z);
                v[4 * u + 3] += __uint_as_float(raw.w);
              }
            } else
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              float e[8];
              unpack8(ld_shared16(swz(buf, lane, u)), e);
              if (p.epi == EPI_MUL) {
#pragma unroll
                for (int i = 0; i < 8; ++i) v[8 * u + i] *= e[i];
              } else {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                  s1 += v[8 * u + i];
                  s2 = fmaf(v[8 * u + i], e[i], s2);
                }
              }
            }
          }
          if (p.epi == EPI_STORE_LN) {  // one slot of row sums per 64 columns
            if (row0 + lane < p.M)
              p.stats[(int64_t)b * p.stats_sb + (int64_t)(row0 + lane) * (4 * p.n_tiles) + 4 * (n0 / BN) + 2 * half + c] =
                  make_float2(s1, s2);
            s1 = s2 = 0.0f;
          }
          if (p.d_f32) {
#pragma unroll
            for (int u = 0; u < 8; ++u)
              st_shared16(swz(buf, lane, u), make_uint4(__float_as_uint(v[4 * u]), __float_as_uint(v[4 * u + 1]),
                                                        __float_as_uint(v[4 * u + 2]), __float_as_uint(v[4 * u + 3])));
          } else if (p.epi == EPI_GELU_FWD) {
            float dv[64];
#pragma unroll
            for (int i = 0; i < 64; ++i) {
              float cdf, pdf;
              normal_cdf_pdf(v[i], cdf, pdf);
              dv[i] = fmaf(v[i], pdf, cdf);
              v[i] *= cdf;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) st_shared16(swz(buf, lane, u), pack8(dv + 8 * u));
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
              tma_store_3d(&tmD2, buf, col, row0, b);
              tma_store_wait_read();
            }
            __syncwarp();
#pragma unroll
            for (int u = 0; u < 8; ++u) st_shared16(swz(buf, lane, u), pack8(v + 8 * u));
          } else {
#pragma unroll
            for (int u = 0; u < 8; ++u) st_shared16(swz(buf, lane, u), pack8(v + 8 * u));
          }
          fence_async_smem();
          __syncwarp();
          if (lane == 0) {
            tma_store_3d(&tmD, buf, col, row0, b);
            tma_store_wait_read();  // the buffer may be overwritten once the copy has read it
            if (has_e && c + 1 < nchunks) {
              mbar_expect_tx(ebar, EPI_BUF_BYTES);
              tma_load_3d(buf, &tmE, ebar, col + cw, row0, b);
              e_pending = true;
            }
          }
          __syncwarp();
        }
        if (!ok) break;
      }
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    if (lane == 0) {
      tma_store_wait_all();
      if (e_pending) {  // only after an abort: do not leave with a copy into our buffer in flight
        uint64_t t0 = global_ns();
        while (!mbar_try_wait(ebar, e_phase) && global_ns() - t0 < 100000000ull) {
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (kPair) cluster_sync();  // neither CTA leaves (or frees) while its peer may still read its tiles or signal its barriers
  if (warp == 1) {
    tc_fence_after();
    if (kPair) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// ------------------------------------------------------------------------------------------- host
// Tensor map of one operand: element (mn, k, b) at base + b*sb + mn*s_mn + k*s_k (element strides).
bool make_map(CUtensorMap* tm, const void* base, int extent_mn, int K, int batch, int64_t s_mn, int64_t s_k,
              int64_t s_b, bool mn_major, int box_mn, bool f32) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3], strides[2];
  cuuint32_t box[3], estr[3] = {1, 1, 1};
  const int64_t row_stride = mn_major ? s_k : s_mn;
  dims[0] = mn_major ? (cuuint64_t)extent_mn : (cuuint64_t)K;
  dims[1] = mn_major ? (cuuint64_t)K : (cuuint64_t)extent_mn;
  dims[2] = (cuuint64_t)batch;
  const cuuint64_t es = f32 ? 4 : 2;
  const cuuint32_t row_elems = f32 ? 32 : 64;  // 128 bytes
  strides[0] = (cuuint64_t)row_stride * es;
  strides[1] = batch > 1 ? (cuuint64_t)s_b * es : (cuuint64_t)row_stride * es * dims[1];
  box[0] = row_elems;
  box[1] = mn_major ? row_elems : (cuuint32_t)box_mn;
  box[2] = 1;
  return fn(tm, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor map of an epilogue operand [batch][M][N] (leading dimension ld, batch stride sb, in elements):
// boxes of 32 rows x 128 bytes, the chunk one epilogue warp stages.
bool make_map_epi(CUtensorMap* tm, const void* base, bool f32, int M, int N, int batch, int64_t ld, int64_t sb) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t es = f32 ? 4 : 2;
  cuuint64_t dims[3] = {(cuuint64_t)N, (cuuint64_t)M, (cuuint64_t)batch};
  cuuint64_t strides[2] = {(cuuint64_t)ld * es, batch > 1 ? (cuuint64_t)sb * es : (cuuint64_t)ld * es * (cuuint64_t)M};
  cuuint32_t box[3] = {f32 ? 32u : 64u, 32u, 1u}, estr[3] = {1, 1, 1};
  return fn(tm, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims,
            strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

// An operand qualifies if one of its two strides is 1 and the others keep every row 16-byte aligned.
bool operand_ok(const void* base, int64_t s_mn, int64_t s_k, int64_t s_b, int batch, bool* mn_major, int vec) {
  if (!aligned16(base)) return false;
  if (batch > 1 && (s_b % vec != 0 || s_b <= 0)) return false;
  if (s_k == 1 && s_mn % vec == 0 && s_mn > 0) { *mn_major = false; return true; }
  if (s_mn == 1 && s_k % vec == 0 && s_k > 0) { *mn_major = true; return true; }
  return false;
}

}  // namespace

namespace tc {
EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)ptr;
  }
  return fn;
}

int sm_count() {
  static PerDevice<int> count;
  int& n = count.here();
  if (n == 0) {
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, current_device());
    if (n <= 0) n = 1;
  }
  return n;
}

}  // namespace tc

int gemm_tc_stats_slots(int N) { return 4 * ((N + BN - 1) / BN); }

bool gemm_tc(Launcher& lc, const GemmArgs& g, int* status_word) {
  if (!status_word) return false;
  const bool f32 = g.in_dtype == HBP_F32;
  if (f32 && (!g.A_hi || !g.A_lo || !g.B_hi || !g.B_lo)) return false;  // float needs the split operands
  if (!f32 && g.A2) return false;
  if (g.M <= 0 || g.N <= 0 || g.K <= 0 || g.batch <= 0) return false;
  const int vec = f32 ? 4 : 8;  // elements per 16 bytes
  if (g.N % vec || g.K % vec) return false;
  if (g.epi != EPI_STORE && g.epi != EPI_GELU_FWD && g.epi != EPI_MUL && g.epi != EPI_RESID && g.epi != EPI_STORE_LN &&
      g.epi != EPI_ADD)
    return false;
  if (g.epi == EPI_ADD && (!g.E || !(g.d_f32 || g.in_dtype == HBP_F32) || g.splitk > 1)) return false;  // float outputs only
  if (g.epi == EPI_STORE_LN && (!g.stats || !g.E)) return false;
  const bool out_f32 = g.d_f32 || f32;
  if (out_f32 && g.epi != EPI_STORE && g.epi != EPI_ADD) return false;
  if (g.splitk > 1 && (g.epi != EPI_STORE || !out_f32 || !g.partial || g.ldd != g.N || (g.batch > 1 && g.d_sb != (int64_t)g.M * g.N)))
    return false;
  const void* A0 = f32 ? (const void*)g.A_hi : g.A;
  const void* B0 = f32 ? (const void*)g.B_hi : g.B;
  // strides of the operands the kernel reads (the split float copies have their own layout)
  const int64_t a_sm = f32 && g.hl_a_sm ? g.hl_a_sm : g.a_sm, a_sk = f32 && g.hl_a_sk ? g.hl_a_sk : g.a_sk;
  const int64_t b_sn = f32 && g.hl_b_sn ? g.hl_b_sn : g.b_sn, b_sk = f32 && g.hl_b_sk ? g.hl_b_sk : g.b_sk;
  bool a_mn = false, b_mn = false;
  if (!operand_ok(A0, a_sm, a_sk, g.a_sb, g.batch, &a_mn, vec)) return false;
  if (!operand_ok(B0, b_sn, b_sk, g.b_sb, g.batch, &b_mn, vec)) return false;
  if (f32 && (!aligned16(g.A_lo) || !aligned16(g.B_lo))) return false;
  // 32-bit MN-major operands need a shared-memory layout of their own that this kernel does not build:
  // float operands must be K-major (the callers write the split copies that way)
  if (f32 && (a_mn || b_mn || g.batch != 1)) return false;
  if (a_mn && g.M % vec) return false;
  // epilogue operands: 16-byte vectors
  const int dv = out_f32 ? 4 : 8;
  if (!aligned16(g.D) || g.ldd % dv || g.d_sb % dv) return false;
  if (g.D2 && (!aligned16(g.D2) || g.ldd2 % 8 || g.d2_sb % 8)) return false;
  if (g.E && (!aligned16(g.E) || g.lde % (g.epi == EPI_ADD ? 4 : 8) || g.e_sb % (g.epi == EPI_ADD ? 4 : 8))) return false;
  if (g.gate && (!aligned16(g.gate) || g.gate_sb % 8)) return false;
  if (g.R && (!aligned16(g.R) || g.N % 4)) return false;
  if (g.epi == EPI_GELU_FWD && !g.D2) return false;
  if (g.epi == EPI_MUL && !g.E) return false;
  if (g.epi == EPI_RESID && !g.R && !g.E) return false;

  // CTA pairs wherever there are at least two 128-row blocks (unless the context asks for single CTAs): a stage is
  // 32 KB instead of 48 KB for the same flops per SM, so the ring is six stages deep and draws a third less from L2
  const int sms = sm_count();
  // A product at most 128 columns wide runs on single CTAs with MMAs of 64 or 128 columns, so that most of the tile is
  // not padding (64-wide recurrent states).  The LayerNorm row sums keep the full tile: their slots are per 64 columns.
  const bool narrow = g.N <= 128 && g.epi != EPI_STORE_LN;
  const bool pair = lc.gemm_pair && sms >= 2 && g.M > BM && !narrow;
  const int n_mma = !narrow ? BN : (g.N <= 64 ? 64 : 128);
  const int b_rows = pair ? Mode<true>::kBRows : n_mma;
  CUtensorMap tmA, tmB;
  if (!make_map(&tmA, A0, g.M, g.K, g.batch, a_sm, a_sk, g.a_sb, a_mn, BM, f32)) return false;
  if (!make_map(&tmB, B0, g.N, g.K, g.batch, b_sn, b_sk, g.b_sb, b_mn, b_rows, f32)) return false;
  // float: segments A_hi B_lo, A_lo B_hi, A_hi B_hi - the small terms first, so that only the last segment adds
  // to an accumulator of full magnitude (the tensor core's fp32 accumulation does not round to nearest)
  CUtensorMap tmA1 = tmA, tmB1 = tmB, tmA2 = tmA, tmB2 = tmB;
  if (f32) {
    CUtensorMap a_lo, b_lo;
    if (!make_map(&b_lo, g.B_lo, g.N, g.K, g.batch, b_sn, b_sk, g.b_sb, b_mn, b_rows, true)) return false;
    if (!make_map(&a_lo, g.A_lo, g.M, g.K, g.batch, a_sm, a_sk, g.a_sb, a_mn, BM, true)) return false;
    tmA2 = tmA; tmB2 = tmB;      // segment 2: hi x hi
    tmA1 = a_lo; tmB1 = tmB;     // segment 1: lo x hi
    tmB = b_lo;                  // segment 0: hi x lo (tmA stays A_hi)
  }
  const int row_elems = f32 ? 32 : 64;
  const int k_blocks = (g.K + row_elems - 1) / row_elems;
  int splits = g.splitk > 1 ? g.splitk : 1;
  if (splits > k_blocks) splits = k_blocks;
  const int kb_per_split = (k_blocks + splits - 1) / splits;
  splits = (k_blocks + kb_per_split - 1) / kb_per_split;  // no empty split
  // epilogue operands that are staged through shared memory (everything but the forward residual update)
  CUtensorMap tmD = tmA, tmD2 = tmA, tmE = tmA;  // placeholders when unused
  if (g.epi != EPI_RESID) {
    if (g.batch > 1 && g.d_sb <= 0) return false;
    if (splits > 1) {
      if (!make_map_epi(&tmD, g.partial, true, g.M, g.N, g.batch * splits, g.N, (int64_t)g.M * g.N)) return false;
    } else if (!make_map_epi(&tmD, g.D, out_f32, g.M, g.N, g.batch, g.ldd, g.d_sb)) return false;
    if (g.epi == EPI_GELU_FWD && !make_map_epi(&tmD2, g.D2, false, g.M, g.N, g.batch, g.ldd2, g.d2_sb)) return false;
    if ((g.epi == EPI_MUL || g.epi == EPI_STORE_LN) && !make_map_epi(&tmE, g.E, false, g.M, g.N, g.batch, g.lde, g.e_sb))
      return false;
    if (g.epi == EPI_ADD && !make_map_epi(&tmE, g.E, true, g.M, g.N, g.batch, g.lde, g.e_sb)) return false;
  }

  if (g.dry_run) return true;
  static PerDevice<bool> attr_done;  // the shared-memory opt-in is a per-device attribute of the kernel
  bool& attr_set = attr_done.here();
  if (!attr_set) {
    if (cudaFuncSetAttribute(gemm_tc_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess ||
        cudaFuncSetAttribute(gemm_tc_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess ||
        cudaFuncSetAttribute(gemm_tc_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess ||
        cudaFuncSetAttribute(gemm_tc_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess) {
      cudaGetLastError();
      return false;
    }
    attr_set = true;
  }
  TcParams p;
  p.M = g.M; p.N = g.N; p.K = g.K; p.batch = g.batch;
  p.m_tiles = pair ? (g.M + 255) / 256 : (g.M + BM - 1) / BM;
  p.n_tiles = (g.N + BN - 1) / BN;
  p.num_tiles = p.m_tiles * p.n_tiles * g.batch * splits;
  p.k_blocks = k_blocks;
  p.a_mn = a_mn; p.b_mn = b_mn;
  p.tf32 = f32; p.segs = f32 ? 3 : 1;
  p.n_mma = n_mma;
  p.splits = splits; p.kb_per_split = kb_per_split;
  p.epi = g.epi; p.d_f32 = out_f32;
  p.D = g.D; p.ldd = g.ldd; p.d_sb = g.d_sb;
  p.D2 = g.D2; p.ldd2 = g.ldd2; p.d2_sb = g.d2_sb;
  p.E = g.E; p.lde = g.lde; p.e_sb = g.e_sb;
  p.gate = g.gate; p.gate_sb = g.gate_sb;
  p.R = g.R;
  p.stats = g.stats; p.stats_sb = g.stats_sb;
  p.status = status_word;
  p.wait_limit_ns = g.wait_limit_ns ? g.wait_limit_ns : WAIT_LIMIT_NS;
  p.stall = g.test_stall;
  if (pair) {
    const int pairs = p.num_tiles < sms / 2 ? p.num_tiles : sms / 2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * pairs);
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = lc.stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = f32 ? cudaLaunchKernelEx(&cfg, gemm_tc_kernel<true, true>, tmA, tmB, tmA1, tmB1, tmA2, tmB2, tmD, tmD2, tmE, p)
                        : cudaLaunchKernelEx(&cfg, gemm_tc_kernel<true, false>, tmA, tmB, tmA1, tmB1, tmA2, tmB2, tmD, tmD2, tmE, p);
    if (e != cudaSuccess && lc.err == cudaSuccess) lc.err = e;
  } else {
    const int grid = p.num_tiles < sms ? p.num_tiles : sms;
    if (f32) gemm_tc_kernel<false, true><<<grid, THREADS, SMEM_BYTES, lc.stream>>>(tmA, tmB, tmA1, tmB1, tmA2, tmB2, tmD, tmD2, tmE, p);
    else gemm_tc_kernel<false, false><<<grid, THREADS, SMEM_BYTES, lc.stream>>>(tmA, tmB, tmA1, tmB1, tmA2, tmB2, tmD, tmD2, tmE, p);
  }
  lc.count();
  lc.check();
  if (splits > 1) reduce_splitk(lc, g.partial, (float*)g.D, splits, (int64_t)g.batch * g.M * g.N);
  return true;
}

}  // namespace hbp
