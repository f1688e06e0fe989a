// hbp_cumsumprod_static: the reverse scan for callers that cannot allocate device memory.
//
// The time-chunked form of the scan needs scratch (per-chunk partial results).  hbp_cumsumprod takes
// that scratch from the caller; this variant keeps it in a fixed array that is part of the library's
// device image, so the call needs no allocation by anybody.  The array is file-scope device memory:
// every GPU on which the library is loaded holds kStaticScratchBytes from load until the process ends.
#include "hbp_internal.h"

namespace {

constexpr size_t kStaticScratchBytes = (size_t)32 << 20;  // 32 MiB

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// The array's name is only a host-side handle; the device address is looked up once per device
// (with that device current) and remembered.
void* g_scratch_addr[hbp::kMaxDevices] = {};

hbp_status static_scratch(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= hbp::kMaxDevices) return HBP_ERR_CUDA;
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
      cudaGetLastError();
      return HBP_ERR_CUDA;
    }
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return HBP_OK;
}

}  // namespace

extern "C" {

size_t hbp_cumsumprod_static_max_bytes(void) { return kStaticScratchBytes; }

hbp_status hbp_cumsumprod_static(int32_t dtype, int32_t gate, int32_t loss, int32_t L, int64_t rows, int32_t d,
                                 const void* u, const void* delta, const void* a, void* g, void* cuda_stream) {
  size_t need = 0;
  hbp_status st = hbp_cumsumprod_scratch_bytes(dtype, L, rows, d, &need);
  if (st != HBP_OK) return st;
  if (need > kStaticScratchBytes) return HBP_ERR_WORKSPACE;  // problem too large for the built-in scratch
  void* scratch = nullptr;
  st = static_scratch(&scratch);
  if (st != HBP_OK) return st;
  // Same kernels as hbp_cumsumprod.  Nothing in the scratch has to start at zero: the first phase writes
  // every partial result before the later phases read it, so what the previous call left behind is harmless.
  return hbp_cumsumprod(dtype, gate, loss, L, rows, d, u, delta, a, g, need ? scratch : nullptr, need, cuda_stream);
}

}  // extern "C"
