// A contraction that has too few output tiles to fill the GPU, split over the CTAs of a thread-block cluster: device
// side hand-over of the partial sums through distributed shared memory, host side choice of the split and the launch
// configuration.  Used by the per-step recurrent kernels (one launch per time step, B * d / 1024 tiles).
#pragma once
#include "tc_common.cuh"

namespace hbp {
namespace tc {

__device__ __forceinline__ uint32_t cluster_nctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
  return r;
}
// A contraction split over the CTAs of a cluster (cluster dims (1, 1, ks), ks <= kMaxClusterSplit, 256 threads per
// CTA): every rank but 0 hands its NACC partial sums per thread to rank 0 through distributed shared memory, one
// hardware cluster barrier orders the hand-over, and rank 0 adds them in rank order (the same bits every run).  `red`
// is the same shared array [ks - 1][NACC][256] (static or dynamic, same offset) in every CTA.  Returns true in the CTA that now
// holds the totals.  Every thread of every CTA of the cluster must call it.
constexpr int kMaxClusterSplit = 4;
template <int NACC>
__device__ __forceinline__ bool cluster_splitk_reduce(double (&acc)[NACC], double* red) {
  const uint32_t ks = cluster_nctarank();
  if (ks == 1) return true;
  const uint32_t rank = cluster_ctarank();
  if (rank != 0) {
#pragma unroll
    for (int j = 0; j < NACC; ++j) {
      const uint32_t remote = map_to_cta(smem_u32(red + ((rank - 1) * NACC + j) * 256 + threadIdx.x), 0);
      asm volatile("st.shared::cluster.f64 [%0], %1;" ::"r"(remote), "d"(acc[j]) : "memory");
    }
  }
  cluster_sync();
  if (rank != 0) return false;
  for (uint32_t r = 1; r < ks; ++r)
#pragma unroll
    for (int j = 0; j < NACC; ++j) acc[j] += red[((r - 1) * NACC + j) * 256 + threadIdx.x];
  return true;
}
// Launch configuration for such a kernel: how many ways to split (1, 2 or 4) so that about two CTAs per SM run, given
// the CTAs there are without a split and the k-tiles there are to share out (at least min_tiles per rank: the
// hand-over costs a cluster barrier and, for many accumulators, tens of KB through distributed shared memory).
inline int cluster_split_for(int base_ctas, int k_tiles, int sms, int max_split = kMaxClusterSplit, int min_tiles = 1) {
  int ks = 1;
  while (ks < max_split && base_ctas * ks * 2 <= 2 * sms && ks * 2 * min_tiles <= k_tiles) ks *= 2;
  return ks;
}
// Fills a launch configuration for 256-thread CTAs in clusters of (1, 1, ks); attr must outlive the launch call.
inline void cluster_launch_config(cudaLaunchConfig_t& cfg, cudaLaunchAttribute& attr, dim3 grid, int ks, size_t smem,
                                  cudaStream_t stream) {
  grid.z = (unsigned)ks;
  cfg = cudaLaunchConfig_t{};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(256);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = 1;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = (unsigned)ks;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
}

}  // namespace tc
}  // namespace hbp
