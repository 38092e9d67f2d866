// Device status word: a kernel whose bounded wait (mbarrier, flag) runs out records a code here and
// leaves through its normal exit path instead of spinning forever; the host reads it after a sync.
#include <stdlib.h>
#include "kernels.h"

namespace mk {

__device__ unsigned int g_mk_status = 0;

int current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return -1; }
  return dev >= 0 && dev < kMaxDevices ? dev : -1;
}

// Every device that loads the library has its own copy of g_mk_status at its own address.
static std::atomic<unsigned int*> g_status_addr[kMaxDevices];

unsigned int* kernel_status_ptr() {
  const int dev = current_device();
  if (dev < 0) return nullptr;
  unsigned int* p = g_status_addr[dev].load(std::memory_order_acquire);
  if (!p) {
    void* a = nullptr;
    if (cudaGetSymbolAddress(&a, g_mk_status) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    p = (unsigned int*)a;
    g_status_addr[dev].store(p, std::memory_order_release);   // a racing thread stores the same address
  }
  return p;
}

bool pdl_enabled(unsigned family) {
  static const unsigned mask = [] {
    const char* v = getenv("MK_NO_PDL");
    if (v && v[0] && v[0] != '0') return 0u;
    const char* m = getenv("MK_PDL_MASK");
    // Default: the kernels that fill an SM by themselves (shared memory) and the GroupNorm pass that follows the
    // convolution.  The row and elementwise kernels are small enough to become resident BESIDE a running GEMM; as
    // dependents they did (blocked in their wait) and slowed it by 3 % (measured), so they keep plain stream order.
    return m && m[0] ? (unsigned)strtoul(m, nullptr, 0) : (unsigned)(PDL_GEMM | PDL_ATTENTION | PDL_CONV | PDL_GROUPNORM);
  }();
  return (mask & family) != 0;
}

cudaError_t kernel_status_fetch_and_clear(unsigned int* out) {
  unsigned int* p = kernel_status_ptr();
  if (!p) return cudaErrorInvalidSymbol;
  cudaError_t e = cudaMemcpy(out, p, sizeof(unsigned int), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return e;
  if (*out) e = cudaMemset(p, 0, sizeof(unsigned int));
  return e;
}

}  // namespace mk
