// prac_weight_grad_static: the weight-gradient entry point for callers that cannot hand the
// library a workspace.  The scratch that prac_weight_grad takes from its `ws` argument (the
// bf16 M' matrix between the two stages and the fp32 split-K partial tiles) lives here in a
// fixed-size array in device global memory that is part of the loaded library image.
#include <cuda_runtime.h>

#include <mutex>

#include "internal.h"

namespace {

constexpr size_t kStaticScratchBytes = 32u << 20;  // 32 MiB on every device that loads the library

// Host code sees only a stand-in for this symbol; its device address is looked up once per
// device with cudaGetSymbolAddress and that pointer is what the kernels receive.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void* g_scratch_ptr[kMaxDevices] = {};

int scratch_of_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PRAC_ECUDA;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (g_scratch_ptr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return PRAC_ECUDA;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return PRAC_OK;
}

}  // namespace

extern "C" {

size_t prac_static_scratch_bytes(void) { return kStaticScratchBytes; }

int prac_weight_grad_static(const prac_basis* basis, const void* dY, int64_t lddy, int64_t d_out,
                            const void* Z, int64_t ldz, int64_t N, double c_override, void* dW,
                            int64_t lddw, int32_t dw_dtype, int32_t accumulate, void* stream) {
  if (!basis) return PRAC_EINVAL;
  void* scratch = nullptr;
  const int st = scratch_of_current_device(&scratch);
  if (st != PRAC_OK) return st;
  // prac_weight_grad checks the size before launching anything: a problem whose scratch need
  // exceeds the array comes back as PRAC_EWORKSPACE.
  return prac_weight_grad(basis, dY, lddy, d_out, Z, ldz, N, c_override, dW, lddw, dw_dtype, accumulate,
                          scratch, kStaticScratchBytes, stream);
}

}  // extern "C"
