// Allocation-free GroupNorm entry point.
//
// Some callers cannot hand the library a workspace because they cannot allocate device memory at
// the point where they call it: code running inside a framework's memory-planned region, a plugin
// whose host gives it only its input and output buffers, a real-time loop where cudaMalloc's
// implicit synchronisation is not acceptable.  For them the two-pass GroupNorm keeps its partial
// sums in a fixed array that is part of the library image instead of in caller-provided workspace.
// The price: the array's 1 MiB is resident on every GPU that loads the library until the process
// exits, it bounds the problem size, and all calls share it.
#include "../../include/mk.h"
#include "kernels.h"

namespace mk {
namespace {

constexpr size_t kStaticScratchBytes = 1u << 20;  // 1 MiB
static __device__ __align__(256) unsigned char g_groupnorm_scratch[kStaticScratchBytes];

struct PerDevice {
  std::atomic<float*> scratch{nullptr};  // device address of g_groupnorm_scratch on that device
  std::atomic<int> sm_count{0};
};
PerDevice g_dev[kMaxDevices];

// In host code the array's name is only a handle for the runtime, not an address a kernel can use:
// the device address has to be asked for, once per device, with that device current.  Two host
// threads that make a device's first call together both ask and both store the same two values;
// the address is published last, so whoever sees it also sees the SM count.
mk_status setup_current_device(int* dev_out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return MK_ERR_NO_DEVICE; }
  if (dev < 0 || dev >= kMaxDevices) return MK_ERR_INVALID_ARG;
  if (!g_dev[dev].scratch.load(std::memory_order_acquire)) {
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_groupnorm_scratch);
    if (e != cudaSuccess || !p) { cudaGetLastError(); return MK_ERR_CUDA; }
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess || sms < 1) { cudaGetLastError(); return MK_ERR_CUDA; }
    g_dev[dev].sm_count.store(sms, std::memory_order_relaxed);
    g_dev[dev].scratch.store(static_cast<float*>(p), std::memory_order_release);
  }
  *dev_out = dev;
  return MK_OK;
}

}  // namespace
}  // namespace mk

extern "C" MK_API mk_status mk_groupnorm_nhwc_noalloc(int32_t dtype, const void* dev_x, void* dev_y, const void* dev_gamma,
                                                       const void* dev_beta, int64_t n, int64_t h, int64_t w, int64_t c,
                                                       int32_t groups, double eps, void* cuda_stream) {
  using namespace mk;
  if (dtype != MK_F32 && dtype != MK_BF16) return MK_ERR_INVALID_ARG;
  if (!dev_x || !dev_y || ((uintptr_t)dev_x & 15) || ((uintptr_t)dev_y & 15)) return MK_ERR_INVALID_ARG;
  if (((uintptr_t)dev_gamma & 15) || ((uintptr_t)dev_beta & 15)) return MK_ERR_INVALID_ARG;
  if (!(eps >= 0.0)) return MK_ERR_INVALID_ARG;
  if (n < 1 || h < 1 || w < 1 || c < 1 || groups < 1 || c % groups) return MK_ERR_SHAPE_MISMATCH;
  // Sizes the kernels cannot index are refused before anything is multiplied: an image count beyond the
  // grid's second dimension, and extents whose products would leave 64 bits or the kernels' 32-bit channel index.
  constexpr int64_t kMaxImages = 65535, kMaxExtent = int64_t(1) << 31;
  if (n > kMaxImages || h >= kMaxExtent || w >= kMaxExtent || c >= kMaxExtent || h * w >= kMaxExtent) return MK_ERR_SHAPE_MISMATCH;
  int dev = -1;
  mk_status st = setup_current_device(&dev);
  if (st != MK_OK) return st;
  const int sms = g_dev[dev].sm_count.load(std::memory_order_relaxed);
  const int64_t hw = h * w;
  // n <= 65535, chunks <= 64, groups < 2^31: the product below stays far inside 64 bits
  if (groupnorm_scratch_bytes(n, hw, c, groups, sms) > kStaticScratchBytes) return MK_ERR_WORKSPACE_TOO_SMALL;
  const int chunks = groupnorm_chunks(n, hw, sms);
  float* scratch = g_dev[dev].scratch.load(std::memory_order_acquire);
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const int d = dtype == MK_F32 ? DT_F32 : DT_BF16;
  EpiProgram none;  // no elementwise ops ahead of the norm
  // The statistics pass overwrites every partial-sum slot the second pass reads, so nothing in the
  // shared array has to start at zero and the previous call's contents are harmless.
  cudaError_t e = launch_groupnorm_stats(d, dev_x, n, hw, c, groups, none, scratch, chunks, s);
  if (e == cudaSuccess)
    e = launch_groupnorm_apply(d, dev_x, dev_y, n, hw, c, groups, dev_gamma, dev_beta, (float)eps, none, scratch, chunks, s);
  if (e != cudaSuccess) { cudaGetLastError(); return MK_ERR_CUDA; }
  return MK_OK;
}
