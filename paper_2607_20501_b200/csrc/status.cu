// Device status word: a kernel whose bounded wait (mbarrier, flag) runs out records a code here and
// leaves through its normal exit path instead of spinning forever; the host reads it after a sync.
#include "kernels.h"

namespace mk {

__device__ unsigned int g_mk_status = 0;

unsigned int* kernel_status_ptr() {
  static unsigned int* p = nullptr;
  if (!p) {
    void* a = nullptr;
    if (cudaGetSymbolAddress(&a, g_mk_status) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    p = (unsigned int*)a;
  }
  return p;
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
