// Flash-style causal attention backward on the tensor cores (bf16, head dimension 64).
//
// The S x S score matrix is never stored: each CTA recomputes the blocks it needs from Q, K and the
// forward's log-sum-exp.  Two kernels, so that every output is owned by exactly one CTA (no atomics, runs
// are bitwise reproducible):
//   attn_dkv_kernel  one CTA per 128 keys; loops over blocks of 64 queries that can see them:
//                       S^T = K Q^T, dP^T = V dO^T            (tcgen05.mma 128x64x16, accumulators in TMEM)
//                       P^T = exp(S^T/sqrt(dh) - lse), dS^T = P^T * (dP^T - D)   (8 warps, one key row per lane, 32 query columns per thread)
//                       dV += P^T dO,  dK += dS^T Q           (P^T, dS^T go back through shared memory as bf16)
//   attn_dq_kernel   one CTA per 128 queries; loops over blocks of 64 keys up to the diagonal:
//                       S = Q K^T, dP = dO V^T, dS = P * (dP - D),  dQ += dS K
// with D_i = sum(dO_i * O_i).  All tiles are moved by TMA (128-byte swizzle); the same shared-memory tile
// serves as a K-major operand (contraction over the head dimension) and as an MN-major operand (contraction
// over its rows).  Each CTA uses at most 256 TMEM columns and ~100 KB of shared memory, so two CTAs share an
// SM and the softmax of one overlaps the MMAs of the other.  All mbarrier waits are bounded.
#include "tc_common.cuh"

namespace hbp {

using namespace tc;

namespace {

constexpr int DH = 64;
constexpr int BIG = 128, SMALL = 64;
constexpr int BIG_BYTES = BIG * DH * 2, SMALL_BYTES = SMALL * DH * 2, PS_BYTES = BIG * SMALL * 2;
constexpr int THREADS = 320;  // warp 0 TMA, warp 1 MMA, warps 2..9 softmax / epilogue (two warps per TMEM lane quarter)
constexpr int SOFTMAX_WARPS = 8;
constexpr uint32_t TMEM_COLS = 256;
constexpr float LOG2E = 1.4426950408889634f;

struct AttnTcParams {
  int S, H, B;
  const float* lse;   // [B][H][S]
  const float* drow;  // rowsum(dO * O) of (batch b, head h, query q) at drow[b * d_sb + h * d_sh + q * d_sq]
  int64_t d_sb, d_sh, d_sq;
  float scale;
  int* status;
};

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// A global load that stays where it is written: left to the compiler, a load whose value is first used one loop
// iteration later is moved down to that use, and its latency is then waited for instead of hidden.
__device__ __forceinline__ float ld_pinned(const float* ptr) {
  float v;
  asm volatile("ld.global.nc.f32 %0, [%1];" : "=f"(v) : "l"(ptr));
  return v;
}
__device__ __forceinline__ void named_barrier_softmax() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = 64, A K-major, B K-major or MN-major
constexpr uint32_t make_idesc(int b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn << 16) | ((uint32_t)(SMALL >> 3) << 17) |
         ((uint32_t)(BIG >> 4) << 24);
}
constexpr uint32_t IDESC_KK = make_idesc(0), IDESC_KMN = make_idesc(1);

// One lane of a converged warp.  The MMA warps below stay converged through their whole loop - every lane runs the
// waits and the address arithmetic, which the compiler can then keep on the uniform datapath - and only the
// tcgen05 instructions themselves are predicated on the elected lane.  Issued from inside an `if (lane == 0)`
// region instead, with descriptors formed per instruction, one MMA cost the issuing thread about 120 cycles,
// four times what a 128 x 64 x 16 MMA takes to run; converged and with descriptors formed once, about 50.
__device__ __forceinline__ bool elect_one() {
  uint32_t is_leader;
  asm volatile("{\n\t.reg .pred q;\n\telect.sync _|q, 0xffffffff;\n\tselp.u32 %0, 1, 0, q;\n\t}" : "=r"(is_leader));
  return is_leader != 0;
}
// descriptor `d` moved by `bytes` within shared memory (the start address sits in the low bits, in 16-byte units)
__device__ __forceinline__ uint64_t desc_add(uint64_t d, uint32_t bytes) { return d + (uint64_t)(bytes >> 4); }

// Barrier slots (8 bytes each):
// 0 big tiles loaded, 1-2 full[2], 3-4 empty[2], 5 scores ready, 6 probabilities ready, 7 all MMAs done,
// 8 scores copied out of tensor memory (the next block's score MMAs may overwrite them), 9 / 10 full / empty of the
// dQ kernel's third buffer.
__device__ __forceinline__ uint32_t bar_at(uint32_t bars, int i) { return bars + 8u * i; }

template <bool kDKV>
__global__ void __launch_bounds__(THREADS, 2)
attn_bwd_tc_kernel(const __grid_constant__ CUtensorMap tmBig0, const __grid_constant__ CUtensorMap tmBig1,
                   const __grid_constant__ CUtensorMap tmSmall0, const __grid_constant__ CUtensorMap tmSmall1,
                   const __grid_constant__ CUtensorMap tmOut0, const __grid_constant__ CUtensorMap tmOut1,
                   const AttnTcParams p) {
  // kDKV: big tiles = K, V (rows = keys), small tiles = Q, dO (rows = queries), outputs dK (Out0), dV (Out1).
  // else: big tiles = Q, dO (rows = queries), small tiles = K, V (rows = keys), output dQ (Out0).
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* aligned = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sBig0 = base, sBig1 = base + BIG_BYTES;
  const uint32_t sSmall = base + 2 * BIG_BYTES;            // [buf][2 tiles]
  const uint32_t sP = sSmall + 4 * SMALL_BYTES;            // P^T (dkv only)
  const uint32_t sDS = sP + PS_BYTES;                      // dS^T / dS
  constexpr int VEC_OFF = 2 * BIG_BYTES + 4 * SMALL_BYTES + 2 * PS_BYTES;
  uint64_t* bar_mem = reinterpret_cast<uint64_t*>(aligned + VEC_OFF + 1024);
  const uint32_t bars = smem_u32(bar_mem);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_mem + 12);
  // The dQ kernel does not stage P, so the place of P^T holds a third buffer of small tiles: its K / V tiles come a
  // block earlier, which is what its MMA warp was waiting for.  Slots of the buffers' barriers: full 1, 2, 9; empty 3, 4, 10.
  constexpr int NBUF = kDKV ? 2 : 3;
  auto full_bar = [&](int buf) { return bar_at(bars, buf < 2 ? 1 + buf : 9); };
  auto empty_bar = [&](int buf) { return bar_at(bars, buf < 2 ? 3 + buf : 10); };
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int blk = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int big0 = blk * BIG;  // first key (dkv) or first query (dq) of this CTA
  // inner blocks: dkv: queries from big0 on; dq: keys up to the last query of the block
  const int n_small = (p.S + SMALL - 1) / SMALL;
  const int it_beg = kDKV ? (big0 / SMALL) : 0;
  const int it_end = kDKV ? n_small : min(n_small, (min(p.S, big0 + BIG) + SMALL - 1) / SMALL);
  const int n_it = it_end - it_beg;

  if (threadIdx.x == 0) {
    mbar_init(bar_at(bars, 0), 1);
    mbar_init(bar_at(bars, 1), 1);
    mbar_init(bar_at(bars, 2), 1);
    mbar_init(bar_at(bars, 3), 1);
    mbar_init(bar_at(bars, 4), 1);
    mbar_init(bar_at(bars, 5), 1);
    mbar_init(bar_at(bars, 6), SOFTMAX_WARPS);
    mbar_init(bar_at(bars, 7), 1);
    mbar_init(bar_at(bars, 8), SOFTMAX_WARPS);
    mbar_init(bar_at(bars, 9), 1);
    mbar_init(bar_at(bars, 10), 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // TMEM columns: scores [0,64), dP [64,128), accumulator 0 [128,192), accumulator 1 [192,256)
  const uint32_t tS = tmem, tDP = tmem + 64, tAcc0 = tmem + 128, tAcc1 = tmem + 192;

  if (warp == 0) {
    if (lane == 0) {
      mbar_expect_tx(bar_at(bars, 0), 2 * BIG_BYTES);
      tma_load_4d(sBig0, &tmBig0, bar_at(bars, 0), 0, big0, h, b);
      tma_load_4d(sBig1, &tmBig1, bar_at(bars, 0), 0, big0, h, b);
      bool ok = true;
      int last_buf_parity[3] = {-1, -1, -1};
      for (int it = 0; it < n_it && ok; ++it) {
        const int buf = it % NBUF;
        const uint32_t ph = (uint32_t)(it / NBUF) & 1u;
        if (!mbar_wait(empty_bar(buf), ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
        const int r0 = (it_beg + it) * SMALL;
        mbar_expect_tx(full_bar(buf), 2 * SMALL_BYTES);
        last_buf_parity[buf] = (int)ph;
        tma_load_4d(sSmall + (2 * buf) * SMALL_BYTES, &tmSmall0, full_bar(buf), 0, r0, h, b);
        tma_load_4d(sSmall + (2 * buf + 1) * SMALL_BYTES, &tmSmall1, full_bar(buf), 0, r0, h, b);
      }
      if (!ok) {  // leave no copy of ours in flight
        for (int buf = 0; buf < NBUF; ++buf)
          if (last_buf_parity[buf] >= 0) {
            const uint64_t t0 = global_ns();
            while (!mbar_try_wait(full_bar(buf), (uint32_t)last_buf_parity[buf]) &&
                   global_ns() - t0 < 100000000ull) {
            }
          }
        const uint64_t t0 = global_ns();
        while (!mbar_try_wait(bar_at(bars, 0), 0) && global_ns() - t0 < 100000000ull) {
        }
      }
    }
  } else if (warp == 1) {
    // Software pipeline: the score MMAs of block it+1 are issued as soon as the softmax warps have copied the
    // scores of block it out of tensor memory, so they run under the exp / pack work of block it; the
    // accumulating MMAs of block it follow once its probabilities are in shared memory.
    const bool leader = elect_one();
    // descriptors of every tile, formed once (buffer 1 of the small tiles lies 2 * SMALL_BYTES after buffer 0)
    const uint64_t dBig0 = make_desc(sBig0, 16, 1024), dBig1 = make_desc(sBig1, 16, 1024);
    const uint64_t dS0kk = make_desc(sSmall, 16, 1024), dS1kk = make_desc(sSmall + SMALL_BYTES, 16, 1024);
    const uint64_t dS0mn = make_desc(sSmall, 8192, 1024), dS1mn = make_desc(sSmall + SMALL_BYTES, 8192, 1024);
    const uint64_t dPt = make_desc(sP, 16, 1024), dDSt = make_desc(sDS, 16, 1024);
    auto issue_scores = [&](int it) {
      const uint32_t boff = (uint32_t)(it % NBUF) * (2 * SMALL_BYTES);
      if (leader) {
        // scores and dP: contraction over the head dimension, both operands K-major
#pragma unroll
        for (int k = 0; k < DH / 16; ++k) tc_mma(tS, desc_add(dBig0, 32 * k), desc_add(dS0kk, boff + 32 * k), IDESC_KK, k != 0);
#pragma unroll
        for (int k = 0; k < DH / 16; ++k) tc_mma(tDP, desc_add(dBig1, 32 * k), desc_add(dS1kk, boff + 32 * k), IDESC_KK, k != 0);
        tc_commit(bar_at(bars, 5));
      }
    };
    bool ok = mbar_wait(bar_at(bars, 0), 0, abort_flag, p.status);
    ok = ok && mbar_wait(full_bar(0), 0, abort_flag, p.status);
    tc_fence_after();
    if (ok) issue_scores(0);
    for (int it = 0; it < n_it && ok; ++it) {
      const int buf = it % NBUF;
      const uint32_t itp = (uint32_t)it & 1u;
      if (it + 1 < n_it) {
        const int nb = (it + 1) % NBUF;
        if (!mbar_wait(full_bar(nb), (uint32_t)((it + 1) / NBUF) & 1u, abort_flag, p.status)) { ok = false; break; }
        if (!mbar_wait(bar_at(bars, 8), itp, abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        issue_scores(it + 1);
      }
      if (!mbar_wait(bar_at(bars, 6), itp, abort_flag, p.status)) { ok = false; break; }
      tc_fence_after();
      // accumulate: contraction over the 64 rows of the small tiles, which are MN-major B operands here
      const uint32_t acc_on = it != 0 ? 1u : 0u;
      const uint32_t boff = (uint32_t)buf * (2 * SMALL_BYTES);
      if (leader) {
        if (kDKV) {
#pragma unroll
          for (int k = 0; k < SMALL / 16; ++k)  // dV += P^T dO
            tc_mma(tAcc1, desc_add(dPt, 32 * k), desc_add(dS1mn, boff + 2048 * k), IDESC_KMN, acc_on | (k != 0));
        }
#pragma unroll
        for (int k = 0; k < SMALL / 16; ++k)  // dK += dS^T Q   /   dQ += dS K
          tc_mma(tAcc0, desc_add(dDSt, 32 * k), desc_add(dS0mn, boff + 2048 * k), IDESC_KMN, acc_on | (k != 0));
        tc_commit(empty_bar(buf));
      }
    }
    if (leader) tc_commit(bar_at(bars, 7));
    if (!ok) {
      const uint64_t t0 = global_ns();
      while (!mbar_try_wait(bar_at(bars, 7), 0) && global_ns() - t0 < 100000000ull) {
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax and epilogue (128 threads)
    const int t = threadIdx.x - 64;             // 0..255
    const int ch = (warp - 2) >> 2;             // which 32 of the block's 64 columns this warp handles
    const int quarter = warp & 3;               // TMEM lane quarter this warp may read
    const int row = quarter * 32 + lane;        // row of the big tile (key for dkv, query for dq)
    const int grow = big0 + row;                // its index in the sequence
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const float scale2 = p.scale * LOG2E;
    const int64_t stat_base = ((int64_t)b * p.H + h) * p.S;
    float my_lse = 0.0f, my_d = 0.0f;
    if (!kDKV) {  // one query per lane: its statistics are scalars
      my_lse = grow < p.S ? p.lse[stat_base + grow] * LOG2E : INFINITY;
      my_d = grow < p.S ? p.drow[(int64_t)b * p.d_sb + (int64_t)h * p.d_sh + (int64_t)grow * p.d_sq] : 0.0f;
    }
    bool ok = true;  // false after a wait gave up: keep pace with the named barriers, do no more work
    // dkv: thread t < 64 fetches the log-sum-exp of query t of a block, thread 64 + t its D
    // dkv: the statistics belong to the block's queries (columns).  Lane c of a warp fetches those of column
    // ch * 32 + c one block ahead (raw values: nothing waits for the loads) and the lanes exchange them by shuffle in
    // the element loop: no staging through shared memory, no barrier among the softmax warps per block.
    auto load_lse = [&](int it) -> float {
      const int q = (it_beg + it) * SMALL + ch * 32 + lane;
      return q < p.S ? ld_pinned(p.lse + stat_base + q) : INFINITY;
    };
    auto load_dd = [&](int it) -> float {
      const int q = (it_beg + it) * SMALL + ch * 32 + lane;
      return q < p.S ? ld_pinned(p.drow + (int64_t)b * p.d_sb + (int64_t)h * p.d_sh + (int64_t)q * p.d_sq) : 0.0f;
    };
    float lse_next = (kDKV && n_it > 0) ? load_lse(0) : 0.0f, dd_next = (kDKV && n_it > 0) ? load_dd(0) : 0.0f;
    for (int it = 0; it < n_it; ++it) {
      const int c0 = (it_beg + it) * SMALL;  // first query (dkv) / key (dq) of the small block
      float col_lse = 0.0f, col_dd = 0.0f;  // dkv: this lane's column statistics of the current block
      if (kDKV) {
        col_lse = lse_next * LOG2E;
        col_dd = dd_next;
        if (it + 1 < n_it) {
          lse_next = load_lse(it + 1);
          dd_next = load_dd(it + 1);
        }
      }
      if (!ok) continue;
      if (!mbar_wait(bar_at(bars, 5), (uint32_t)it & 1u, abort_flag, p.status)) { ok = false; continue; }
      tc_fence_after();
      // copy this warp's 32 score columns out of tensor memory and release it for the next block's score MMAs
      float sc[32], dp[32];
      tc_ld32_async(tS + lane_addr + ch * 32, sc);
      tc_ld32_async(tDP + lane_addr + ch * 32, dp);
      tc_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_at(bars, 8));
      // only blocks that touch the diagonal (or the end of the sequence) need the per-element mask
      const bool full = kDKV ? (c0 >= big0 + BIG - 1 && big0 + BIG <= p.S) : (c0 + SMALL - 1 <= big0 && c0 + SMALL <= p.S);
      if (full) {
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          const float lse2 = kDKV ? __shfl_sync(0xffffffffu, col_lse, c) : my_lse;
          const float dd = kDKV ? __shfl_sync(0xffffffffu, col_dd, c) : my_d;
          const float pr = fast_exp2(fmaf(sc[c], scale2, -lse2));
          sc[c] = pr;
          dp[c] = pr * (dp[c] - dd);
        }
      } else {
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          const int col = c0 + ch * 32 + c;
          const float lse2 = kDKV ? __shfl_sync(0xffffffffu, col_lse, c) : my_lse;
          const float dd = kDKV ? __shfl_sync(0xffffffffu, col_dd, c) : my_d;
          // dkv: row = key, column = query; dq: row = query, column = key
          const bool vis = kDKV ? ((col >= grow) && (grow < p.S)) : ((col <= grow) && (col < p.S));
          const float pr = vis ? fast_exp2(fmaf(sc[c], scale2, -lse2)) : 0.0f;
          sc[c] = pr;
          dp[c] = pr * (dp[c] - dd);
        }
      }
      // the accumulating MMAs of the previous block read the probability tiles: wait until they are done
      if (it > 0 && !mbar_wait(empty_bar((it - 1) % NBUF), (uint32_t)((it - 1) / NBUF) & 1u, abort_flag, p.status)) {
        ok = false;
        continue;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (kDKV) st_shared16(swz(sP, row, ch * 4 + u), pack8(sc + 8 * u));
        st_shared16(swz(sDS, row, ch * 4 + u), pack8(dp + 8 * u));
      }
      fence_async_smem();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_at(bars, 6));
    }
    // ---- epilogue: accumulators -> bf16 -> shared -> TMA store
    ok = ok && mbar_wait(bar_at(bars, 7), 0, abort_flag, p.status);
    if (ok) {
      tc_fence_after();
#pragma unroll 1
      for (int o = 0; o < (kDKV ? 2 : 1); ++o) {
        const uint32_t dst = o == 0 ? sDS : sP;          // staging: the probability tiles are free now
        const float mul = o == 0 ? p.scale : 1.0f;       // dK and dQ carry the 1/sqrt(dh) factor, dV does not
        float v[32];
        tc_ld32((o == 0 ? tAcc0 : tAcc1) + lane_addr + ch * 32, v);
#pragma unroll
        for (int c = 0; c < 32; ++c) v[c] *= mul;
#pragma unroll
        for (int u = 0; u < 4; ++u) st_shared16(swz(dst, row, ch * 4 + u), pack8(v + 8 * u));
      }
      fence_async_smem();
    }
    named_barrier_softmax();
    if (t == 0 && ok) {
      tma_store_4d(&tmOut0, sDS, 0, big0, h, b);
      if (kDKV) tma_store_4d(&tmOut1, sP, 0, big0, h, b);
      tma_store_wait_all();
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
  }
}

// ------------------------------------------------------------------------------------------- forward
// Causal attention forward, one CTA per 128 queries (bf16, head dimension 64), in two sweeps over the key blocks
// so that the output accumulator in tensor memory never has to be rescaled:
//   sweep 1:  S = Q K^T per 64-key block; every softmax thread keeps the running maximum and sum of exponentials of
//             its row over its 32 columns; the two halves of a row are merged into the row's log-sum-exp;
//   sweep 2:  S again, P = exp(S/sqrt(dh) - lse) (already normalised), O += P V.
// Same roles, barriers and pipelining as the backward kernels: the score MMAs of the next block run under the
// exponentials of the current one.  Barrier slots: 1-2 full[2], 3-4 empty[2], 5 scores ready, 6 probabilities
// ready, 7 all MMAs done, 8 scores copied out, 0 the Q tile.
constexpr uint32_t FWD_TMEM_COLS = 128;  // scores [0,64), output accumulator [64,128)
constexpr int FWD_SMEM_BYTES = BIG_BYTES + 4 * SMALL_BYTES + PS_BYTES + 2048 /*row statistics*/ + 256 /*barriers*/ + 1024;

__global__ void __launch_bounds__(THREADS, 3)
attn_fwd_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                   const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO, float* lse_out,
                   const AttnTcParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* aligned = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sQ = base;
  const uint32_t sSmall = base + BIG_BYTES;       // [buf][K tile, V tile]
  const uint32_t sP = sSmall + 4 * SMALL_BYTES;   // P as bf16, later the output staging
  constexpr int VEC_OFF = BIG_BYTES + 4 * SMALL_BYTES + PS_BYTES;
  float* vec = reinterpret_cast<float*>(aligned + VEC_OFF);  // [2 halves][128 rows] of {max, sum}
  uint64_t* bar_mem = reinterpret_cast<uint64_t*>(aligned + VEC_OFF + 2048);
  const uint32_t bars = smem_u32(bar_mem);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar_mem + 10);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int blk = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int q0 = blk * BIG;
  const int n_kb = min((p.S + SMALL - 1) / SMALL, (min(p.S, q0 + BIG) + SMALL - 1) / SMALL);  // key blocks up to the diagonal
  const int n_it = 2 * n_kb;  // sweep 1 then sweep 2

  if (threadIdx.x == 0) {
    for (int i = 0; i < 9; ++i) mbar_init(bar_at(bars, i), (i == 6 || i == 8) ? SOFTMAX_WARPS : 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(FWD_TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tS = tmem, tO = tmem + 64;

  if (warp == 0) {
    if (lane == 0) {
      mbar_expect_tx(bar_at(bars, 0), BIG_BYTES);
      tma_load_4d(sQ, &tmQ, bar_at(bars, 0), 0, q0, h, b);
      bool ok = true;
      int last_buf_parity[2] = {-1, -1};
      for (int it = 0; it < n_it && ok; ++it) {
        const int buf = it & 1;
        const uint32_t ph = (uint32_t)(it >> 1) & 1u;
        if (!mbar_wait(bar_at(bars, 3 + buf), ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
        const bool second = it >= n_kb;
        const int r0 = (second ? it - n_kb : it) * SMALL;
        mbar_expect_tx(bar_at(bars, 1 + buf), second ? 2 * SMALL_BYTES : SMALL_BYTES);
        last_buf_parity[buf] = (int)ph;
        tma_load_4d(sSmall + (2 * buf) * SMALL_BYTES, &tmK, bar_at(bars, 1 + buf), 0, r0, h, b);
        if (second) tma_load_4d(sSmall + (2 * buf + 1) * SMALL_BYTES, &tmV, bar_at(bars, 1 + buf), 0, r0, h, b);
      }
      if (!ok) {  // leave no copy of ours in flight
        for (int buf = 0; buf < 2; ++buf)
          if (last_buf_parity[buf] >= 0) {
            const uint64_t t0 = global_ns();
            while (!mbar_try_wait(bar_at(bars, 1 + buf), (uint32_t)last_buf_parity[buf]) &&
                   global_ns() - t0 < 100000000ull) {
            }
          }
        const uint64_t t0 = global_ns();
        while (!mbar_try_wait(bar_at(bars, 0), 0) && global_ns() - t0 < 100000000ull) {
        }
      }
    }
  } else if (warp == 1) {
    // converged warp, one elected lane issues (see elect_one); descriptors formed once
    const bool leader = elect_one();
    const uint64_t dQt = make_desc(sQ, 16, 1024), dKkk = make_desc(sSmall, 16, 1024);
    const uint64_t dVmn = make_desc(sSmall + SMALL_BYTES, 8192, 1024), dPt = make_desc(sP, 16, 1024);
    auto issue_scores = [&](int it) {
      const uint32_t boff = (uint32_t)(it & 1) * (2 * SMALL_BYTES);
      if (leader) {
#pragma unroll
        for (int k = 0; k < DH / 16; ++k) tc_mma(tS, desc_add(dQt, 32 * k), desc_add(dKkk, boff + 32 * k), IDESC_KK, k != 0);
        tc_commit(bar_at(bars, 5));
        if (it < n_kb) tc_commit(bar_at(bars, 3 + (it & 1)));  // sweep 1: the K tile is free once the scores are formed
      }
    };
    bool ok = mbar_wait(bar_at(bars, 0), 0, abort_flag, p.status);
    ok = ok && mbar_wait(bar_at(bars, 1), 0, abort_flag, p.status);
    tc_fence_after();
    if (ok) issue_scores(0);
    for (int it = 0; it < n_it && ok; ++it) {
      const int buf = it & 1;
      if (it + 1 < n_it) {
        const int nb = (it + 1) & 1;
        if (!mbar_wait(bar_at(bars, 1 + nb), (uint32_t)((it + 1) >> 1) & 1u, abort_flag, p.status)) { ok = false; break; }
        if (!mbar_wait(bar_at(bars, 8), (uint32_t)it & 1u, abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        issue_scores(it + 1);
      }
      if (it < n_kb) continue;
      const int j = it - n_kb;
      if (!mbar_wait(bar_at(bars, 6), (uint32_t)j & 1u, abort_flag, p.status)) { ok = false; break; }
      tc_fence_after();
      const uint32_t boff = (uint32_t)buf * (2 * SMALL_BYTES);
      if (leader) {
#pragma unroll
        for (int k = 0; k < SMALL / 16; ++k)  // O += P V: contraction over the 64 keys, V is an MN-major operand
          tc_mma(tO, desc_add(dPt, 32 * k), desc_add(dVmn, boff + 2048 * k), IDESC_KMN, (j != 0 ? 1u : 0u) | (k != 0));
        tc_commit(bar_at(bars, 3 + buf));
      }
    }
    if (leader) tc_commit(bar_at(bars, 7));
    if (!ok) {
      const uint64_t t0 = global_ns();
      while (!mbar_try_wait(bar_at(bars, 7), 0) && global_ns() - t0 < 100000000ull) {
      }
    }
  } else {
    const int ch = (warp - 2) >> 2;        // which 32 of the block's 64 key columns this warp handles
    const int quarter = warp & 3;          // TMEM lane quarter this warp may read
    const int row = quarter * 32 + lane;   // query row of the tile
    const int grow = q0 + row;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const float scale2 = p.scale * LOG2E;
    float m_run = -INFINITY, l_run = 0.0f, lse2 = 0.0f;
    bool ok = true;  // false after a wait gave up: keep pace with the named barriers, do no more work
    for (int it = 0; it < n_it; ++it) {
      const bool second = it >= n_kb;
      const int j = second ? it - n_kb : it;
      const int c0 = j * SMALL;
      if (it == n_kb) {  // between the sweeps: merge the two halves of every row into its log-sum-exp
        vec[ch * 256 + row] = m_run;
        vec[ch * 256 + 128 + row] = l_run;
        named_barrier_softmax();
        const float m0 = vec[row], l0 = vec[128 + row], m1 = vec[256 + row], l1 = vec[256 + 128 + row];
        const float mm = fmaxf(m0, m1);  // finite: key 0 is visible to every query
        const float ll = l0 * fast_exp2(m0 - mm) + l1 * fast_exp2(m1 - mm);
        lse2 = mm + __log2f(ll);
        if (ch == 0 && grow < p.S && ok) lse_out[((int64_t)b * p.H + h) * p.S + grow] = lse2 * (1.0f / LOG2E);
      }
      if (!ok) continue;
      if (!mbar_wait(bar_at(bars, 5), (uint32_t)it & 1u, abort_flag, p.status)) { ok = false; continue; }
      tc_fence_after();
      float sc[32];
      tc_ld32(tS + lane_addr + ch * 32, sc);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_at(bars, 8));
      const bool full = (c0 + SMALL - 1 <= q0) && (c0 + SMALL <= p.S);  // no element of the block is masked
      if (!second) {
        float bm = -INFINITY;
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          const int col = c0 + ch * 32 + c;
          const bool vis = full || ((col <= grow) && (col < p.S));
          sc[c] = vis ? sc[c] * scale2 : -INFINITY;
          bm = fmaxf(bm, sc[c]);
        }
        if (bm > -INFINITY) {
          const float mn = fmaxf(m_run, bm);
          float sum = 0.0f;
#pragma unroll
          for (int c = 0; c < 32; ++c) sum += fast_exp2(sc[c] - mn);
          l_run = l_run * fast_exp2(m_run - mn) + sum;
          m_run = mn;
        }
      } else {
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          const int col = c0 + ch * 32 + c;
          const bool vis = full || ((col <= grow) && (col < p.S));
          sc[c] = vis ? fast_exp2(fmaf(sc[c], scale2, -lse2)) : 0.0f;
        }
        // the accumulating MMAs of the previous block read the probability tile: wait until they are done
        if (j > 0 && !mbar_wait(bar_at(bars, 3 + ((it - 1) & 1)), (uint32_t)((it - 1) >> 1) & 1u, abort_flag, p.status)) {
          ok = false;
          continue;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) st_shared16(swz(sP, row, ch * 4 + u), pack8(sc + 8 * u));
        fence_async_smem();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_at(bars, 6));
      }
    }
    // ---- epilogue: O -> bf16 -> shared -> TMA store
    ok = ok && mbar_wait(bar_at(bars, 7), 0, abort_flag, p.status);
    if (ok) {
      tc_fence_after();
      float v[32];
      tc_ld32(tO + lane_addr + ch * 32, v);
#pragma unroll
      for (int u = 0; u < 4; ++u) st_shared16(swz(sP, row, ch * 4 + u), pack8(v + 8 * u));
      fence_async_smem();
    }
    named_barrier_softmax();
    if (threadIdx.x == 64 && ok) {
      tma_store_4d(&tmO, sP, 0, q0, h, b);
      tma_store_wait_all();
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(FWD_TMEM_COLS) : "memory");
  }
}

constexpr int SMEM_BYTES = 2 * BIG_BYTES + 4 * SMALL_BYTES + 2 * PS_BYTES + 1024 /*vectors*/ + 256 /*barriers*/ + 1024;

// 4-D map {dh, sequence, head, batch} of one [tokens][ld] tensor's column block starting at `base`.
bool make_map4(CUtensorMap* tm, const void* base, int S, int H, int B, int64_t ld, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[4] = {(cuuint64_t)DH, (cuuint64_t)S, (cuuint64_t)H, (cuuint64_t)B};
  cuuint64_t strides[3] = {(cuuint64_t)ld * 2, (cuuint64_t)DH * 2, (cuuint64_t)S * (cuuint64_t)ld * 2};
  cuuint32_t box[4] = {(cuuint32_t)DH, (cuuint32_t)box_rows, 1, 1}, estr[4] = {1, 1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// Runs dQ, dK, dV of attention_bwd on the tensor cores; delta_rows must already hold rowsum(dO * O).
// Returns false (nothing launched) when the problem does not fit this kernel.
bool attention_bwd_tc(Launcher& lc, const AttnArgs& a, int* status_word) {
  if (a.dtype != HBP_BF16 || a.head_dim != DH || !status_word) return false;
  const int d = a.heads * DH;
  const int64_t ld3 = 3 * (int64_t)d;
  if (((uintptr_t)a.qkv | (uintptr_t)a.d_o | (uintptr_t)a.d_qkv) & 15u) return false;
  if (d % 8) return false;
  const bf16* qkv = (const bf16*)a.qkv;
  bf16* dqkv = (bf16*)a.d_qkv;
  CUtensorMap qB, qS, kB, kS, vB, vS, oB, oS, dq, dk, dv;
  bool ok = make_map4(&qB, qkv, a.seq, a.heads, a.batch, ld3, BIG) && make_map4(&qS, qkv, a.seq, a.heads, a.batch, ld3, SMALL) &&
            make_map4(&kB, qkv + d, a.seq, a.heads, a.batch, ld3, BIG) && make_map4(&kS, qkv + d, a.seq, a.heads, a.batch, ld3, SMALL) &&
            make_map4(&vB, qkv + 2 * d, a.seq, a.heads, a.batch, ld3, BIG) && make_map4(&vS, qkv + 2 * d, a.seq, a.heads, a.batch, ld3, SMALL) &&
            make_map4(&oB, a.d_o, a.seq, a.heads, a.batch, d, BIG) && make_map4(&oS, a.d_o, a.seq, a.heads, a.batch, d, SMALL) &&
            make_map4(&dq, dqkv, a.seq, a.heads, a.batch, ld3, BIG) && make_map4(&dk, dqkv + d, a.seq, a.heads, a.batch, ld3, BIG) &&
            make_map4(&dv, dqkv + 2 * d, a.seq, a.heads, a.batch, ld3, BIG);
  if (!ok) return false;
  static PerDevice<bool> attr_done;  // per-device kernel attribute
  bool& attr_set = attr_done.here();
  if (!attr_set) {
    if (cudaFuncSetAttribute(attn_bwd_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess ||
        cudaFuncSetAttribute(attn_bwd_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess) {
      cudaGetLastError();
      return false;
    }
    attr_set = true;
  }
  AttnTcParams p;
  p.S = a.seq; p.H = a.heads; p.B = a.batch;
  p.lse = a.lse;
  if (a.d_stats) {  // float2 {sum dO, sum dO * O} per token and 64-column slot: the .y of slot `head`
    p.drow = reinterpret_cast<const float*>(a.d_stats) + 1;
    p.d_sb = (int64_t)a.seq * a.d_slots * 2; p.d_sh = 2; p.d_sq = (int64_t)a.d_slots * 2;
  } else {
    p.drow = a.delta_rows;
    p.d_sb = (int64_t)a.heads * a.seq; p.d_sh = a.seq; p.d_sq = 1;
  }
  p.scale = 1.0f / sqrtf((float)DH);
  p.status = status_word;
  dim3 grid((a.seq + BIG - 1) / BIG, a.heads, a.batch);
  // dK, dV: big tiles K, V; small tiles Q, dO
  attn_bwd_tc_kernel<true><<<grid, THREADS, SMEM_BYTES, lc.stream>>>(kB, vB, qS, oS, dk, dv, p);
  // dQ: big tiles Q, dO; small tiles K, V
  attn_bwd_tc_kernel<false><<<grid, THREADS, SMEM_BYTES, lc.stream>>>(qB, oB, kS, vS, dq, dq, p);
  lc.count(2);
  lc.check();
  return true;
}

// Causal attention forward (O and the log-sum-exp) on the tensor cores; false (nothing launched) when the problem
// does not fit this kernel.
bool attention_fwd_tc(Launcher& lc, const AttnArgs& a, int* status_word) {
  if (a.dtype != HBP_BF16 || a.head_dim != DH || !status_word) return false;
  const int d = a.heads * DH;
  const int64_t ld3 = 3 * (int64_t)d;
  if (((uintptr_t)a.qkv | (uintptr_t)a.o) & 15u) return false;
  if (d % 8) return false;
  const bf16* qkv = (const bf16*)a.qkv;
  CUtensorMap q, k, v, o;
  if (!(make_map4(&q, qkv, a.seq, a.heads, a.batch, ld3, BIG) && make_map4(&k, qkv + d, a.seq, a.heads, a.batch, ld3, SMALL) &&
        make_map4(&v, qkv + 2 * d, a.seq, a.heads, a.batch, ld3, SMALL) && make_map4(&o, a.o, a.seq, a.heads, a.batch, d, BIG)))
    return false;
  static PerDevice<bool> attr_done;  // per-device kernel attribute
  bool& attr_set = attr_done.here();
  if (!attr_set) {
    if (cudaFuncSetAttribute(attn_fwd_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, FWD_SMEM_BYTES) != cudaSuccess) {
      cudaGetLastError();
      return false;
    }
    attr_set = true;
  }
  AttnTcParams p;
  p.S = a.seq; p.H = a.heads; p.B = a.batch;
  p.lse = nullptr; p.drow = nullptr; p.d_sb = p.d_sh = p.d_sq = 0;
  p.scale = 1.0f / sqrtf((float)DH);
  p.status = status_word;
  dim3 grid((a.seq + BIG - 1) / BIG, a.heads, a.batch);
  attn_fwd_tc_kernel<<<grid, THREADS, FWD_SMEM_BYTES, lc.stream>>>(q, k, v, o, a.lse, p);
  lc.count();
  lc.check();
  return true;
}

}  // namespace hbp
