// Host-callable launchers of the sm_100a kernels.  One function = one kernel launch on the
// given stream; none of them allocates, synchronises or copies.  Pointers are device pointers.
#pragma once

#include <cuda_runtime.h>
#include <atomic>
#include <stddef.h>
#include <stdint.h>

namespace mk {

// dtype codes mirror mk_dtype
constexpr int DT_F32 = 0;
constexpr int DT_BF16 = 1;

// ---- elementwise program: the tail a producing kernel applies before its store -----------------
// (paper, decomposition rules: GEMM + elementwise, elementwise chains, bias after matmul and the
// residual add are fused into one subkernel)
enum EpiKind : int32_t {
  EPI_BIAS = 1,      // v += bias[col]            ptr = bias vector
  EPI_RELU = 2,
  EPI_GELU_TANH = 3,
  EPI_SILU = 4,
  EPI_SCALE = 5,     // v *= a
  EPI_CLAMP = 6,     // v = min(max(v, a), b)
  EPI_RESIDUAL = 7,  // v += res[row * ld + col]  ptr = residual tensor, ld = output width
  EPI_GELU_ERF = 8   // 0.5 v (1 + erf(v / sqrt 2))
};
constexpr int EPI_MAX = 8;
struct EpiOp {
  int32_t kind;
  float a, b;
  int32_t ptr_dtype;  // element type behind ptr (a residual may be fp32 in a bf16 module)
  const void* ptr;
};
struct EpiProgram {
  int32_t n = 0;
  int32_t dtype = DT_BF16;  // the module's storage type (bias vectors, default for everything)
  EpiOp op[EPI_MAX];
};

// ---- per-device host state ---------------------------------------------------------------------------------
// One process may hold contexts on several GPUs, and may use them from several host threads: everything the
// launchers cache (the device address of a __device__ symbol, a kernel's opt-in to more than 48 KB of dynamic
// shared memory) is a property of ONE device and is therefore kept per device ordinal, in atomics.
constexpr int kMaxDevices = 64;
int current_device();   // ordinal of the calling thread's current device; -1 on error or beyond kMaxDevices

// Largest dynamic shared-memory size the kernels of one launcher have opted into, per device.
struct SmemOptIn {
  std::atomic<size_t> have[kMaxDevices] = {};
  // Raise cudaFuncAttributeMaxDynamicSharedMemorySize of every kernel in `fn` to `need` bytes on the current
  // device unless that device has been given at least as much before.  Two threads that race here set the
  // same attribute twice, which is harmless.
  template <typename... Fn>
  cudaError_t ensure(size_t need, Fn... fn) {
    const int dev = current_device();
    if (dev < 0) return cudaErrorInvalidDevice;
    if (need <= have[dev].load(std::memory_order_acquire)) return cudaSuccess;
    cudaError_t r = cudaSuccess;
    ((r = (r == cudaSuccess ? cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)need) : r)), ...);
    if (r == cudaSuccess) have[dev].store(need, std::memory_order_release);
    return r;
  }
};

// Blocks of one kernel that can be resident on the current device at once (SM count x blocks per SM at the kernel's
// register and shared-memory footprint), asked once per device: the grid size of a persistent launch.
struct ResidentBlocks {
  std::atomic<int> n[kMaxDevices] = {};
  cudaError_t last_error = cudaSuccess;   // why get() returned 0
  template <typename K>
  int get(K kernel, int block_threads, size_t dyn_smem = 0) {
    const int dev = current_device();
    if (dev < 0) return 0;
    int v = n[dev].load(std::memory_order_acquire);
    if (v > 0) return v;
    int per_sm = 0, sms = 0;
    const cudaError_t e1 = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, block_threads, dyn_smem);
    const cudaError_t e2 = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e1 != cudaSuccess || e2 != cudaSuccess || per_sm < 1 || sms < 1) {
      last_error = e1 != cudaSuccess ? e1 : e2 != cudaSuccess ? e2 : cudaErrorInvalidConfiguration;
      cudaGetLastError();
      return 0;
    }
    v = per_sm * sms;
    n[dev].store(v, std::memory_order_release);
    return v;
  }
};

// ---- device status word (bounded-wait expiry codes) --------------------------------------------------
unsigned int* kernel_status_ptr();   // address on the current device, nullptr without one
cudaError_t kernel_status_fetch_and_clear(unsigned int* out);   // of the current device

// Self-test of the bounded-wait exit (selftest.cu): one CTA waits, through the kernels' own wait routine, on a
// barrier nobody arrives at; out6 = six int64 in device memory (see the kernel).
cudaError_t launch_bounded_wait_selftest(long long limit_cycles, long long* out6, cudaStream_t s);

// ---- programmatic dependent launch ----------------------------------------------------------------------
// A kernel launched through LaunchCfg may be scheduled while the kernel before it on the stream is still
// draining: its CTAs become resident as the predecessor's CTAs retire, run their set-up, and block in
// pdl_wait() (device_common.cuh) until the predecessor has completed and its writes are visible.  Only
// kernels that execute pdl_wait() before their first read of global data may be launched this way.
// MK_NO_PDL=1 in the environment turns the attribute off (plain stream order); MK_PDL_MASK=<bits> sets which
// kernel families (PDL_* below) are launched as dependents (default: GEMM, attention, convolution, GroupNorm pass).
enum PdlFamily : unsigned { PDL_GEMM = 1, PDL_ATTENTION = 2, PDL_CONV = 4, PDL_ROWOP = 8, PDL_ELTWISE = 16, PDL_GROUPNORM = 32 };
bool pdl_enabled(unsigned family);
struct LaunchCfg {
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr[2];
  LaunchCfg(unsigned family, dim3 grid, dim3 block, size_t smem, cudaStream_t s, int cluster = 1) {
    cfg = cudaLaunchConfig_t{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    int n = 0;
    if (cluster > 1) {
      attr[n].id = cudaLaunchAttributeClusterDimension;
      attr[n].val.clusterDim.x = (unsigned)cluster;
      attr[n].val.clusterDim.y = 1;
      attr[n].val.clusterDim.z = 1;
      ++n;
    }
    if (pdl_enabled(family)) {
      attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[n].val.programmaticStreamSerializationAllowed = 1;
      ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = (unsigned)n;
  }
};

// ---- HBM-bound kernels ------------------------------------------------------------------------------
// y[rows, cols] = program(x).  swiglu: x is [rows, 2*cols] = [gate | up] and the program runs on
// silu(gate) * up.  x has the module dtype; y has out_dtype (fp32 for an fp32 residual stream).
cudaError_t launch_eltwise(int dtype, int out_dtype, const void* x, void* y, int64_t rows, int64_t cols, bool swiglu,
                           const EpiProgram& p, int sm_count, cudaStream_t s);

enum RowMode : int32_t { ROW_LAYERNORM = 0, ROW_RMSNORM = 1, ROW_SOFTMAX = 2 };
// Row-wise reduction over the last dimension of program(x)[rows, n]; gamma/beta may be null.
// x has in_dtype (fp32 when it is an fp32 residual stream), y / gamma / beta have dtype.
cudaError_t launch_rowop(int dtype, int in_dtype, int mode, const void* x, void* y, int64_t rows, int64_t n,
                         const void* gamma, const void* beta, float eps, const EpiProgram& pre,
                         cudaStream_t s);

// GroupNorm over NHWC [nb, hw, c]: stats writes per-(image, chunk, group) partial sums into
// scratch, apply reduces them and normalises.  scratch must hold groupnorm_scratch_bytes().
int groupnorm_chunks(int64_t nb, int64_t hw, int sm_count);
// One launch, one pass over HBM: a thread-block cluster holds an image in its shared memory (groupnorm_cluster.cu).
// supported: the image fits a cluster of at most eight CTAs, 16-byte-aligned tensors, vectorisable channel count.
bool groupnorm_cluster_supported(int dtype, const void* x, const void* y, int64_t nb, int64_t hw, int64_t c, int groups, int sm_count);
cudaError_t launch_groupnorm_cluster(int dtype, const void* x, void* y, int64_t nb, int64_t hw, int64_t c, int groups, const void* gamma,
                                     const void* beta, float eps, const EpiProgram& pre, int sm_count, cudaStream_t s);
size_t groupnorm_scratch_bytes(int64_t nb, int64_t hw, int64_t c, int groups, int sm_count);
cudaError_t launch_groupnorm_stats(int dtype, const void* x, int64_t nb, int64_t hw, int64_t c,
                                   int groups, const EpiProgram& pre, float* scratch, int chunks,
                                   cudaStream_t s);
cudaError_t launch_groupnorm_apply(int dtype, const void* x, void* y, int64_t nb, int64_t hw,
                                   int64_t c, int groups, const void* gamma, const void* beta,
                                   float eps, const EpiProgram& pre, const float* scratch, int chunks,
                                   cudaStream_t s);
// Normalisation alone, from partial sums float [nb][stat_slots][groups][2] written by the producer of x
// (the convolution's epilogue).  Needs c to be a multiple of the 16-byte vector and at most 2048.
bool groupnorm_apply_partials_supported(int dtype, int64_t c, int groups);
cudaError_t launch_groupnorm_apply_partials(int dtype, const void* x, void* y, int64_t nb, int64_t hw, int64_t c, int groups,
                                            const void* gamma, const void* beta, float eps, const float* stats, int stat_slots,
                                            int sm_count, cudaStream_t s);

// Pooling over NHWC [nb, h, w, c], square window k, stride, no padding: mode 0 mean, 1 maximum, 2 p-norm.
enum PoolMode : int32_t { POOL_AVG = 0, POOL_MAX = 1, POOL_LP = 2 };
cudaError_t launch_pool_nhwc(int dtype, int mode, const void* x, void* y, int64_t nb, int64_t h, int64_t w, int64_t c, int k,
                             int stride, float p, int sm_count, cudaStream_t s);

// ---- plain-ALU (SIMT) kernels: any shape, fp32 or bf16, fp32 accumulation -------------------------
// Y[M, N] = program(A[M, K] @ W); W is [K, N] row-major, or [N, K] when w_transposed.
// swiglu: W has 2N logical columns [gate | up] and Y = program(silu(A Wg) * (A Wu)).
cudaError_t launch_gemm_simt(int dtype, int out_dtype, const void* a, const void* w, bool w_transposed, void* y,
                             int64_t m, int64_t n, int64_t k, bool swiglu, const EpiProgram& p,
                             cudaStream_t s);
// Block-scaled fp8 GEMM on the plain ALUs (any m, n; k a multiple of 128): xq [m, k] e4m3, sx [m, k / 128], wq [k, n] or
// [n, k] when w_transposed, sw [ceil(n / 128), k / 128]; y = program(...) in `dtype` (bf16).
cudaError_t launch_gemm_fp8_simt(const void* xq, const float* sx, const void* wq, bool w_transposed, const float* sw, void* y, int64_t m,
                                 int64_t n, int64_t k, const EpiProgram& p, cudaStream_t s);
// Small-shape fused chain: one CTA owns whole rows, so the row norm follows the GEMM in-kernel.
// Y = rownorm(program(A @ W)); n <= 1024.
cudaError_t launch_linear_rownorm_simt(int dtype, const void* a, const void* w, bool w_transposed,
                                       void* y, int64_t m, int64_t n, int64_t k, const EpiProgram& p,
                                       int mode, const void* gamma, const void* beta, float eps,
                                       cudaStream_t s);
cudaError_t launch_conv3x3_simt(int dtype, const void* x, const void* w, void* y, int64_t nb, int64_t h,
                                int64_t wd, int64_t c, int64_t co, const EpiProgram& p, cudaStream_t s);

// Strided view of Q, K, V: element (b, h, s, d) sits at base + b*sb + h*sh + s*ss + d (elements).
struct AttnView {
  const void* q;
  const void* k;
  const void* v;
  int64_t sb, sh, ss;
  int64_t B, H, S, D;
  bool causal;   // mask keys after the query (diagonal kept); false: every key is visible
};
// O is the dense [B*S, H*D] matrix.
cudaError_t launch_attention_simt(int dtype, const AttnView& a, void* o, cudaStream_t s);

}  // namespace mk
