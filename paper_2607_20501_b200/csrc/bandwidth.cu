// HBM-bound subkernels: elementwise chains, row reductions (LayerNorm / RMSNorm / softmax) and
// NHWC GroupNorm.  All global traffic is 128-bit wide on the vector paths; statistics are fp32;
// rows stay in registers between the reduction and the normalising pass, so each element is read
// once and written once.
#include <stdlib.h>
#include "device_common.cuh"

namespace mk {

static inline int ceil_div_i64(int64_t a, int64_t b) { return (int)((a + b - 1) / b); }

// =====================================================================================================
// elementwise chain
// =====================================================================================================
// Thread (cx, ry) of a block owns one 16-byte column vector and walks down the rows, four rows in
// flight at a time: no per-element index arithmetic (a 64-bit division per vector made the first
// version of this kernel ALU-bound), the bias slice of a thread never changes, and every access of a
// warp is a contiguous run of a row.  tx = threads along a row (power of two <= 256).
template <typename T, typename TO, bool SWIGLU>
__global__ void __launch_bounds__(256) eltwise_vec_kernel(const T* __restrict__ x, TO* __restrict__ y, int64_t rows,
                                                          int64_t cols, int tx, const __grid_constant__ EpiProgram p) {
  constexpr int VE = Elem<T>::VEC;
  constexpr int UNROLL = 4;
  pdl_launch_dependents();
  pdl_wait();
  const int vpr = (int)(cols / VE);
  const int cx = threadIdx.x & (tx - 1), ry = threadIdx.x / tx, rpb = 256 / tx;
  const int vc = blockIdx.x * tx + cx;
  if (vc >= vpr) return;
  const int64_t col = (int64_t)vc * VE;
  const int64_t in_ld = SWIGLU ? 2 * cols : cols;
  const int64_t rstride = (int64_t)gridDim.y * rpb;
  for (int64_t r0 = (int64_t)blockIdx.y * rpb + ry; r0 < rows; r0 += rstride * UNROLL) {
    float v[UNROLL][VE];
    float u[UNROLL][VE];
#pragma unroll
    for (int q = 0; q < UNROLL; ++q) {
      const int64_t r = r0 + q * rstride;
      if (r < rows) {
        ld_vec(x + r * in_ld + col, v[q]);
        if (SWIGLU) ld_vec(x + r * in_ld + cols + col, u[q]);
      }
    }
#pragma unroll
    for (int q = 0; q < UNROLL; ++q) {
      const int64_t r = r0 + q * rstride;
      if (r < rows) {
        if (SWIGLU) {
#pragma unroll
          for (int e = 0; e < VE; ++e) v[q][e] = silu_f(v[q][e]) * u[q][e];
        }
        epi_apply_vec<T, VE>(p, v[q], r, col, cols);
        st_vec_as<TO, VE>(y + r * cols + col, v[q]);
      }
    }
  }
}

template <typename T, typename TO, bool SWIGLU>
__global__ void __launch_bounds__(256) eltwise_scalar_kernel(const T* __restrict__ x, TO* __restrict__ y, int64_t rows,
                                                             int64_t cols, const __grid_constant__ EpiProgram p) {
  const int64_t total = rows * cols;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  const int64_t in_ld = SWIGLU ? 2 * cols : cols;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
    const int64_t r = i / cols, c = i - r * cols;
    float v = Elem<T>::ld(x + r * in_ld + c);
    if (SWIGLU) v = silu_f(v) * Elem<T>::ld(x + r * in_ld + cols + c);
    Elem<TO>::st(y + i, epi_apply(p, v, r, c, cols));
  }
}

template <typename T, typename TO>
static cudaError_t eltwise_dispatch(const void* x, void* y, int64_t rows, int64_t cols, bool swiglu, const EpiProgram& p,
                                    int sm_count, cudaStream_t s) {
  constexpr int VE = Elem<T>::VEC;
  const T* xp = (const T*)x;
  TO* yp = (TO*)y;
  if (rows * cols == 0) return cudaSuccess;
  if (cols % VE == 0 && cols / VE <= INT32_MAX / 2) {
    const int vpr = (int)(cols / VE);
    int tx = 1;
    while (tx < vpr && tx < 256) tx *= 2;
    const int rpb = 256 / tx;
    const int gx = (vpr + tx - 1) / tx;
    // enough row blocks to fill the machine 8 CTAs deep, each thread taking >= 4 rows when there are that many
    int64_t gy = (rows + (int64_t)rpb * 4 - 1) / ((int64_t)rpb * 4);
    const int64_t cap = ((int64_t)sm_count * 8 + gx - 1) / gx;
    if (gy > cap) gy = cap;
    if (gy < 1) gy = 1;
    if (gy > 65535) gy = 65535;
    dim3 grid((unsigned)gx, (unsigned)gy);
    LaunchCfg lc(PDL_ELTWISE, grid, dim3(256), 0, s);
    if (swiglu) return cudaLaunchKernelEx(&lc.cfg, eltwise_vec_kernel<T, TO, true>, xp, yp, rows, cols, tx, p);
    return cudaLaunchKernelEx(&lc.cfg, eltwise_vec_kernel<T, TO, false>, xp, yp, rows, cols, tx, p);
  } else {
    int grid = ceil_div_i64(rows * cols, 256);
    grid = grid > sm_count * 8 ? sm_count * 8 : grid;
    if (swiglu) eltwise_scalar_kernel<T, TO, true><<<grid, 256, 0, s>>>(xp, yp, rows, cols, p);
    else eltwise_scalar_kernel<T, TO, false><<<grid, 256, 0, s>>>(xp, yp, rows, cols, p);
  }
  return cudaGetLastError();
}

cudaError_t launch_eltwise(int dtype, int out_dtype, const void* x, void* y, int64_t rows, int64_t cols, bool swiglu,
                           const EpiProgram& p, int sm_count, cudaStream_t s) {
  if (dtype == DT_F32) return out_dtype == DT_F32 ? eltwise_dispatch<float, float>(x, y, rows, cols, swiglu, p, sm_count, s) : cudaErrorInvalidValue;
  return out_dtype == DT_F32 ? eltwise_dispatch<__nv_bfloat16, float>(x, y, rows, cols, swiglu, p, sm_count, s)
                             : eltwise_dispatch<__nv_bfloat16, __nv_bfloat16>(x, y, rows, cols, swiglu, p, sm_count, s);
}

// =====================================================================================================
// row reductions: one warp per row at a time, the row lives in registers; warps walk the rows with a
// grid-wide stride so a launch is a few resident waves, not one block per handful of rows
// =====================================================================================================
template <typename TI, typename T, int VPL, int MODE>
__global__ void __launch_bounds__(256) rowop_warp_kernel(const TI* __restrict__ x, T* __restrict__ y, int64_t rows, int n,
                                                         const T* __restrict__ gamma, const T* __restrict__ beta, float eps,
                                                         const __grid_constant__ EpiProgram pre) {
  constexpr int VE = Elem<T>::VEC;
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int nvec = n / VE;
  const int64_t wstride = (int64_t)gridDim.x * (blockDim.x >> 5);
  const int64_t row_first = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  // the NEXT row is kept in flight while the current one is reduced, unless that would double an already
  // large register footprint (fp32 input next to bf16 output: 32 raw bytes per 8 elements; measured with the
  // prefetch: one block per SM instead of two and 24.5 us instead of 19.1 for 8192 rows of 2048)
  constexpr bool PREFETCH = sizeof(TI) == sizeof(T);
  RawVec<TI, VE> raw[VPL];
  if (PREFETCH && row_first < rows) {
#pragma unroll
    for (int i = 0; i < VPL; ++i)
      if (lane + 32 * i < nvec) raw[i].load(x + row_first * n + (lane + 32 * i) * VE);
  }
  for (int64_t row = row_first; row < rows; row += wstride) {
  float v[VPL][VE];
#pragma unroll
  for (int i = 0; i < VPL; ++i) {
    const int vi = lane + 32 * i;
    if (vi < nvec) {
      if (!PREFETCH) raw[i].load(x + row * n + vi * VE);
      raw[i].unpack(v[i]);
      epi_apply_vec<T, VE>(pre, v[i], row, (int64_t)vi * VE, n);
    } else {
#pragma unroll
      for (int e = 0; e < VE; ++e) v[i][e] = (MODE == ROW_SOFTMAX) ? -INFINITY : 0.0f;
    }
  }
  if (PREFETCH && row + wstride < rows) {
#pragma unroll
    for (int i = 0; i < VPL; ++i)
      if (lane + 32 * i < nvec) raw[i].load(x + (row + wstride) * n + (lane + 32 * i) * VE);
  }
  const float inv_n = 1.0f / (float)n;
  float mean = 0.0f, mul = 1.0f;
  if (MODE == ROW_LAYERNORM) {
    float s = 0.0f;
#pragma unroll
    for (int i = 0; i < VPL; ++i)
#pragma unroll
      for (int e = 0; e < VE; ++e) s += v[i][e];
    mean = warp_sum(s) * inv_n;
    float q = 0.0f;
#pragma unroll
    for (int i = 0; i < VPL; ++i)
      if (lane + 32 * i < nvec) {
#pragma unroll
        for (int e = 0; e < VE; ++e) { const float d = v[i][e] - mean; q += d * d; }
      }
    mul = rsqrtf(warp_sum(q) * inv_n + eps);
  } else if (MODE == ROW_RMSNORM) {
    float q = 0.0f;
#pragma unroll
    for (int i = 0; i < VPL; ++i)
#pragma unroll
      for (int e = 0; e < VE; ++e) q += v[i][e] * v[i][e];
    mul = rsqrtf(warp_sum(q) * inv_n + eps);
  } else {
    float mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < VPL; ++i)
#pragma unroll
      for (int e = 0; e < VE; ++e) mx = fmaxf(mx, v[i][e]);
    mx = warp_max(mx);
    float s = 0.0f;
#pragma unroll
    for (int i = 0; i < VPL; ++i)
#pragma unroll
      for (int e = 0; e < VE; ++e) { v[i][e] = __expf(v[i][e] - mx); s += v[i][e]; }
    mul = 1.0f / warp_sum(s);
  }
  T* yr = y + row * n;
#pragma unroll
  for (int i = 0; i < VPL; ++i) {
    const int vi = lane + 32 * i;
    if (vi < nvec) {
      float o[VE];
#pragma unroll
      for (int e = 0; e < VE; ++e) o[e] = MODE == ROW_LAYERNORM ? (v[i][e] - mean) * mul : v[i][e] * mul;
      if (MODE != ROW_SOFTMAX) {
        if (gamma) {
          float g[VE];
          ld_vec(gamma + vi * VE, g);
#pragma unroll
          for (int e = 0; e < VE; ++e) o[e] *= g[e];
        }
        if (MODE == ROW_LAYERNORM && beta) {
          float b[VE];
          ld_vec(beta + vi * VE, b);
#pragma unroll
          for (int e = 0; e < VE; ++e) o[e] += b[e];
        }
      }
      st_vec(yr + vi * VE, o);
    }
  }
  }  // row loop
}

// Fallback for rows that do not fit the register path or are not a multiple of the vector width:
// one CTA per row, three passes over the row (it stays in L1/L2 between them).
template <int MODE>
__device__ __forceinline__ float block_reduce(float v, float* sh) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
  v = (MODE == 1) ? warp_max(v) : warp_sum(v);
  __syncthreads();
  if (lane == 0) sh[w] = v;
  __syncthreads();
  float r = (MODE == 1) ? -INFINITY : 0.0f;
  for (int i = 0; i < nw; ++i) r = (MODE == 1) ? fmaxf(r, sh[i]) : r + sh[i];
  return r;
}

template <typename TI, typename T, int MODE>
__global__ void __launch_bounds__(256) rowop_block_kernel(const TI* __restrict__ x, T* __restrict__ y, int64_t rows, int64_t n,
                                                          const T* __restrict__ gamma, const T* __restrict__ beta, float eps,
                                                          const __grid_constant__ EpiProgram pre) {
  __shared__ float sh[32];
  const int64_t row = blockIdx.x;
  const TI* xr = x + row * n;
  T* yr = y + row * n;
  const float inv_n = 1.0f / (float)n;
  float mean = 0.0f, mul = 1.0f, mx = 0.0f;
  if (MODE == ROW_LAYERNORM) {
    float s = 0.0f;
    for (int64_t c = threadIdx.x; c < n; c += blockDim.x) s += epi_apply(pre, Elem<TI>::ld(xr + c), row, c, n);
    mean = block_reduce<0>(s, sh) * inv_n;
    float q = 0.0f;
    for (int64_t c = threadIdx.x; c < n; c += blockDim.x) { const float d = epi_apply(pre, Elem<TI>::ld(xr + c), row, c, n) - mean; q += d * d; }
    mul = rsqrtf(block_reduce<0>(q, sh) * inv_n + eps);
  } else if (MODE == ROW_RMSNORM) {
    float q = 0.0f;
    for (int64_t c = threadIdx.x; c < n; c += blockDim.x) { const float d = epi_apply(pre, Elem<TI>::ld(xr + c), row, c, n); q += d * d; }
    mul = rsqrtf(block_reduce<0>(q, sh) * inv_n + eps);
  } else {
    float m = -INFINITY;
    for (int64_t c = threadIdx.x; c < n; c += blockDim.x) m = fmaxf(m, epi_apply(pre, Elem<TI>::ld(xr + c), row, c, n));
    mx = block_reduce<1>(m, sh);
    float s = 0.0f;
    for (int64_t c = threadIdx.x; c < n; c += blockDim.x) s += __expf(epi_apply(pre, Elem<TI>::ld(xr + c), row, c, n) - mx);
    mul = 1.0f / block_reduce<0>(s, sh);
  }
  for (int64_t c = threadIdx.x; c < n; c += blockDim.x) {
    const float v = epi_apply(pre, Elem<TI>::ld(xr + c), row, c, n);
    float o;
    if (MODE == ROW_SOFTMAX) {
      o = __expf(v - mx) * mul;
    } else {
      o = (v - mean) * mul;
      if (gamma) o *= Elem<T>::ld(gamma + c);
      if (MODE == ROW_LAYERNORM && beta) o += Elem<T>::ld(beta + c);
    }
    Elem<T>::st(yr + c, o);
  }
}

template <typename TI, typename T, int MODE>
static cudaError_t rowop_mode(const TI* x, T* y, int64_t rows, int64_t n, const T* g, const T* b, float eps,
                              const EpiProgram& pre, cudaStream_t s) {
  constexpr int VE = Elem<T>::VEC;
  if (rows == 0) return cudaSuccess;
  const int64_t nvec = n / VE;
  if (n % VE == 0 && nvec <= 32 * 16) {
    const int ni = (int)n;
    // Grid: every warp should walk about three rows (the next one in flight while the current one is reduced), and
    // beyond one resident wave the hardware's block scheduler is the load balancer: up to three waves of blocks
    // when there are rows enough, exactly one resident wave when there are not (a grid of rows / 8 blocks, most of
    // which start only when an earlier one has retired, gives a warp one row and the prefetch nothing to do).
    // Measured at 2048-element rows: 8192 rows 18.4 -> 16.4 us with one wave; 32768 rows 47 us with three, 50 with one.
    auto go = [&](auto kernel, ResidentBlocks& rb) -> cudaError_t {
      const int resident = rb.get(kernel, 256);
      if (resident <= 0) return rb.last_error != cudaSuccess ? rb.last_error : cudaErrorInvalidDevice;
      const int64_t want = ceil_div_i64(rows, 24);
      int64_t grid = 2 * want <= 3 * (int64_t)resident ? resident : (want < 3 * (int64_t)resident ? want : 3 * (int64_t)resident);
      if (sizeof(TI) != sizeof(T)) grid = 148 * 8;   // no prefetch (fp32 in, bf16 out): a row per warp, the block scheduler does the rest
      if (grid > ceil_div_i64(rows, 8)) grid = ceil_div_i64(rows, 8);
      LaunchCfg lc(PDL_ROWOP, dim3((unsigned)grid), dim3(256), 0, s);
      return cudaLaunchKernelEx(&lc.cfg, kernel, x, y, rows, ni, g, b, eps, pre);
    };
    static ResidentBlocks rb1, rb2, rb4, rb8, rb16;   // per instantiation (this function is one) and kernel
    if (nvec <= 32) return go(rowop_warp_kernel<TI, T, 1, MODE>, rb1);
    if (nvec <= 64) return go(rowop_warp_kernel<TI, T, 2, MODE>, rb2);
    if (nvec <= 128) return go(rowop_warp_kernel<TI, T, 4, MODE>, rb4);
    if (nvec <= 256) return go(rowop_warp_kernel<TI, T, 8, MODE>, rb8);
    return go(rowop_warp_kernel<TI, T, 16, MODE>, rb16);
  } else {
    rowop_block_kernel<TI, T, MODE><<<(unsigned)rows, 256, 0, s>>>(x, y, rows, n, g, b, eps, pre);
  }
  return cudaGetLastError();
}

template <typename TI, typename T>
static cudaError_t rowop_dispatch(int mode, const void* x, void* y, int64_t rows, int64_t n, const void* g, const void* b,
                                  float eps, const EpiProgram& pre, cudaStream_t s) {
  const TI* xp = (const TI*)x; T* yp = (T*)y; const T* gp = (const T*)g; const T* bp = (const T*)b;
  switch (mode) {
    case ROW_LAYERNORM: return rowop_mode<TI, T, ROW_LAYERNORM>(xp, yp, rows, n, gp, bp, eps, pre, s);
    case ROW_RMSNORM: return rowop_mode<TI, T, ROW_RMSNORM>(xp, yp, rows, n, gp, bp, eps, pre, s);
    default: return rowop_mode<TI, T, ROW_SOFTMAX>(xp, yp, rows, n, gp, bp, eps, pre, s);
  }
}

cudaError_t launch_rowop(int dtype, int in_dtype, int mode, const void* x, void* y, int64_t rows, int64_t n, const void* gamma,
                         const void* beta, float eps, const EpiProgram& pre, cudaStream_t s) {
  if (dtype == DT_F32) return in_dtype == DT_F32 ? rowop_dispatch<float, float>(mode, x, y, rows, n, gamma, beta, eps, pre, s) : cudaErrorInvalidValue;
  return in_dtype == DT_F32 ? rowop_dispatch<float, __nv_bfloat16>(mode, x, y, rows, n, gamma, beta, eps, pre, s)
                            : rowop_dispatch<__nv_bfloat16, __nv_bfloat16>(mode, x, y, rows, n, gamma, beta, eps, pre, s);
}

// =====================================================================================================
// Pooling NHWC (mean / maximum / p-norm of k x k windows, no padding).  HBM-bound: every input element is read
// once when stride >= k.  One thread per 128-bit channel vector of an output pixel; consecutive threads walk the
// channels, so a warp reads contiguous runs of every window pixel; fp32 accumulation.
// =====================================================================================================
template <typename T, int MODE>
__global__ void __launch_bounds__(256, 4) pool_nhwc_kernel(const T* __restrict__ x, T* __restrict__ y, int64_t nb, int h, int w, int c, int oh,
                                                        int ow, int k, int stride, float p, float inv_p) {
  // A block = 32 consecutive output vectors (lane) x R window-row slots (warp): warp r takes window rows r, r + R, ...,
  // so a 7 x 7 window is 7 loads per thread instead of 49 in a row, and the grid has R times as many threads.
  constexpr int VE = Elem<T>::VEC;
  __shared__ float part[8][32][VE + 1];
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31, r = threadIdx.x >> 5, R = blockDim.x >> 5;
  const int cv = c / VE;
  const int64_t total = nb * oh * ow * cv;
  for (int64_t i0 = (int64_t)blockIdx.x * 32; i0 < total; i0 += (int64_t)gridDim.x * 32) {
    const int64_t i = i0 + lane;
    float acc[VE];
#pragma unroll
    for (int e = 0; e < VE; ++e) acc[e] = MODE == POOL_MAX ? -INFINITY : 0.0f;
    if (i < total) {
      const int vc = (int)(i % cv);
      int64_t q = i / cv;
      const int ox = (int)(q % ow);
      q /= ow;
      const int oy = (int)(q % oh);
      const int64_t n = q / oh;
      const T* base = x + ((n * h + (int64_t)oy * stride) * w + (int64_t)ox * stride) * c + vc * VE;
      for (int a = r; a < k; a += R) {
        // a window row in pieces of up to eight pixels: all of a piece's loads are issued before any is used
        for (int b0 = 0; b0 < k; b0 += 8) {
          RawVec<T, VE> raw[8];
#pragma unroll
          for (int u = 0; u < 8; ++u)
            if (b0 + u < k) raw[u].load(base + ((int64_t)a * w + b0 + u) * c);
#pragma unroll
          for (int u = 0; u < 8; ++u)
            if (b0 + u < k) {
              float v[VE];
              raw[u].unpack(v);
#pragma unroll
              for (int e = 0; e < VE; ++e) {
                if (MODE == POOL_AVG) acc[e] += v[e];
                else if (MODE == POOL_MAX) acc[e] = fmaxf(acc[e], v[e]);
                else acc[e] += p == 2.0f ? v[e] * v[e] : __powf(fabsf(v[e]), p);
              }
            }
        }
      }
    }
    if (R > 1) {
#pragma unroll
      for (int e = 0; e < VE; ++e) part[r][lane][e] = acc[e];
      __syncthreads();
      if (r == 0) {
        for (int rr = 1; rr < R; ++rr)
#pragma unroll
          for (int e = 0; e < VE; ++e) acc[e] = MODE == POOL_MAX ? fmaxf(acc[e], part[rr][lane][e]) : acc[e] + part[rr][lane][e];
      }
    }
    if (r == 0 && i < total) {
      const float inv_n = 1.0f / (float)(k * k);
#pragma unroll
      for (int e = 0; e < VE; ++e) {
        if (MODE == POOL_AVG) acc[e] *= inv_n;
        else if (MODE == POOL_LP) acc[e] = p == 2.0f ? sqrtf(acc[e]) : __powf(acc[e], inv_p);
      }
      st_vec(y + i * VE, acc);
    }
    if (R > 1) __syncthreads();
  }
}
// any channel count: one thread per output element
template <typename T, int MODE>
__global__ void __launch_bounds__(256) pool_nhwc_scalar_kernel(const T* __restrict__ x, T* __restrict__ y, int64_t nb, int h, int w, int c,
                                                               int oh, int ow, int k, int stride, float p, float inv_p) {
  const int64_t total = nb * oh * ow * c;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int ch = (int)(i % c);
    int64_t r = i / c;
    const int ox = (int)(r % ow);
    r /= ow;
    const int oy = (int)(r % oh);
    const int64_t n = r / oh;
    float acc = MODE == POOL_MAX ? -INFINITY : 0.0f;
    const T* base = x + ((n * h + (int64_t)oy * stride) * w + (int64_t)ox * stride) * c + ch;
    for (int a = 0; a < k; ++a)
      for (int b = 0; b < k; ++b) {
        const float v = Elem<T>::ld(base + ((int64_t)a * w + b) * c);
        if (MODE == POOL_AVG) acc += v;
        else if (MODE == POOL_MAX) acc = fmaxf(acc, v);
        else acc += p == 2.0f ? v * v : powf(fabsf(v), p);
      }
    if (MODE == POOL_AVG) acc *= 1.0f / (float)(k * k);
    else if (MODE == POOL_LP) acc = p == 2.0f ? sqrtf(acc) : powf(acc, inv_p);
    Elem<T>::st(y + i, acc);
  }
}

template <typename T, int MODE>
static cudaError_t pool_launch(const void* x, void* y, int64_t nb, int64_t h, int64_t w, int64_t c, int k, int stride, float p, int sm_count,
                               cudaStream_t s) {
  const int oh = (int)((h - k) / stride + 1), ow = (int)((w - k) / stride + 1);
  const bool vec = c % Elem<T>::VEC == 0;
  const int64_t total = nb * oh * ow * (vec ? c / Elem<T>::VEC : c);
  if (total == 0) return cudaSuccess;
  int64_t grid = (total + 255) / 256;
  if (grid > (int64_t)sm_count * 16) grid = (int64_t)sm_count * 16;
  if (vec) {
    const int R = k < 8 ? k : 8;
    grid = (total + 31) / 32;
    if (grid > (int64_t)sm_count * 32) grid = (int64_t)sm_count * 32;
    LaunchCfg lc(PDL_ELTWISE, dim3((unsigned)grid), dim3(32 * R), 0, s);   // plain order by default: as a dependent it measured 2 % slower
    return cudaLaunchKernelEx(&lc.cfg, pool_nhwc_kernel<T, MODE>, (const T*)x, (T*)y, nb, (int)h, (int)w, (int)c, oh, ow, k, stride, p, 1.0f / p);
  }
  pool_nhwc_scalar_kernel<T, MODE><<<(unsigned)grid, 256, 0, s>>>((const T*)x, (T*)y, nb, (int)h, (int)w, (int)c, oh, ow, k, stride, p, 1.0f / p);
  return cudaGetLastError();
}
template <typename T>
static cudaError_t pool_mode(int mode, const void* x, void* y, int64_t nb, int64_t h, int64_t w, int64_t c, int k, int stride, float p,
                             int sm_count, cudaStream_t s) {
  if (mode == POOL_AVG) return pool_launch<T, POOL_AVG>(x, y, nb, h, w, c, k, stride, p, sm_count, s);
  if (mode == POOL_MAX) return pool_launch<T, POOL_MAX>(x, y, nb, h, w, c, k, stride, p, sm_count, s);
  return pool_launch<T, POOL_LP>(x, y, nb, h, w, c, k, stride, p, sm_count, s);
}
cudaError_t launch_pool_nhwc(int dtype, int mode, const void* x, void* y, int64_t nb, int64_t h, int64_t w, int64_t c, int k, int stride,
                             float p, int sm_count, cudaStream_t s) {
  if (k < 1 || stride < 1 || k > h || k > w || mode < 0 || mode > 2) return cudaErrorInvalidValue;
  if (h > INT32_MAX || w > INT32_MAX || c > INT32_MAX) return cudaErrorInvalidValue;
  return dtype == DT_F32 ? pool_mode<float>(mode, x, y, nb, h, w, c, k, stride, p, sm_count, s)
                         : pool_mode<__nv_bfloat16>(mode, x, y, nb, h, w, c, k, stride, p, sm_count, s);
}

// =====================================================================================================
// GroupNorm NHWC: the statistics of one (image, group) span the whole image, a global
// synchronisation, so it takes two launches: partial sums per (image, pixel chunk, group), then a
// pass that reduces the partials (a few dozen values) and normalises.
// scratch layout: float [nb][chunks][groups][2] = (sum, sum of squares)
// =====================================================================================================
constexpr int GN_THREADS = 256;
constexpr int GN_MAX_C = 2048;
#ifndef MK_GN_RESIDENT
#define MK_GN_RESIDENT 2
#endif
constexpr int GN_RESIDENT = MK_GN_RESIDENT;    // CTAs per SM the two-pass kernels are compiled for
#ifndef MK_GN_UN
#define MK_GN_UN 4
#endif
constexpr int GN_UN = MK_GN_UN;                // independent 16-byte loads per thread and batch (8 and 16 measured slower)

int groupnorm_chunks(int64_t nb, int64_t hw, int sm_count) {
  // as many CTAs as are resident at once (GN_RESIDENT per SM: both kernels are built for it), never one more: a
  // CTA walks its pixels in a few dependent batches, so a second, nearly empty wave would double the kernel's time;
  // at least 32 pixels each
  int64_t want = (GN_RESIDENT * (int64_t)sm_count) / nb;
  int64_t maxc = hw / 32 > 0 ? hw / 32 : 1;
  int64_t c = want < 1 ? 1 : want;
  if (c > maxc) c = maxc;
  if (c > 64) c = 64;
  return (int)c;
}
size_t groupnorm_scratch_bytes(int64_t nb, int64_t hw, int64_t, int groups, int sm_count) {
  return (size_t)nb * groupnorm_chunks(nb, hw, sm_count) * groups * 2 * sizeof(float);
}


template <typename T>
__host__ __device__ inline bool gn_fast_ok(int64_t c) {
  const int64_t vpp = c / Elem<T>::VEC;
  return c % Elem<T>::VEC == 0 && vpp >= 1 && vpp <= GN_THREADS && (GN_THREADS % vpp) == 0 && c <= GN_MAX_C;
}

// The statistics are sums of differences from a pivot, not of the values themselves: with E[x^2] - mean^2 taken about
// zero, a group whose mean is fifty standard deviations from zero loses the variance to cancellation in fp32.  The
// pivot of (image, group) is the group's own first element (first pixel, first channel, after the elementwise
// prefix): a sample of the data, so (mean - pivot)^2 is of the order of the variance.  Both passes read it from the
// same address; the partial sums keep their layout.
template <typename T>
__device__ __forceinline__ float gn_pivot(const T* __restrict__ x, int64_t img, int64_t hw, int64_t c, int64_t g, int64_t cg, const EpiProgram& pre) {
  const int64_t r = img * hw, ch = g * cg;
  return epi_apply(pre, Elem<T>::ld(x + r * c + ch), r, ch, c);
}

// A thread's walk over its 16-byte vectors (one per pixel row of the thread grid): batches of UN independent loads,
// the next batch asked for before the current one is used, pointers advanced by a fixed stride, no per-load
// bounds test.  f(raw, i) receives the i-th vector of the walk.  These kernels are issue-bound before they are
// bandwidth-bound (a profile of the first form showed 94 warp instructions per vector, a third of all issue slots
// taken, 1.7 TB/s), so the loop carries nothing but the loads and the arithmetic.
template <int UN, typename F>
__device__ __forceinline__ void walk16(const uint4* __restrict__ ptr, size_t step, int n, F f) {
  int i = 0;
  uint4 cur[UN];
  if (n >= UN) {
#pragma unroll
    for (int u = 0; u < UN; ++u) cur[u] = ptr[u * step];
  }
  for (; i + UN <= n; i += UN) {
    uint4 nxt[UN];
    const bool more = i + 2 * UN <= n;
    if (more) {
#pragma unroll
      for (int u = 0; u < UN; ++u) nxt[u] = ptr[(UN + u) * step];
    }
    ptr += UN * step;
#pragma unroll
    for (int u = 0; u < UN; ++u) f(cur[u], i + u);
    if (more) {
#pragma unroll
      for (int u = 0; u < UN; ++u) cur[u] = nxt[u];
    }
  }
  for (; i < n; ++i) {
    const uint4 t = *ptr;
    ptr += step;
    f(t, i);
  }
}
template <typename T> __device__ __forceinline__ void unpack16(const uint4& r, float (&v)[Elem<T>::VEC]) {
  if constexpr (sizeof(T) == 4) {
    v[0] = __uint_as_float(r.x); v[1] = __uint_as_float(r.y); v[2] = __uint_as_float(r.z); v[3] = __uint_as_float(r.w);
  } else {
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) { v[2 * k] = __uint_as_float(w[k] << 16); v[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u); }
  }
}
template <typename T> __device__ __forceinline__ uint4 pack16(const float (&v)[Elem<T>::VEC]) {
  if constexpr (sizeof(T) == 4) {
    return make_uint4(__float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]), __float_as_uint(v[3]));
  } else {
    return make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]), pack_bf16x2(v[6], v[7]));
  }
}

template <typename T>
__global__ void __launch_bounds__(GN_THREADS, GN_RESIDENT) groupnorm_stats_kernel(const T* __restrict__ x, int64_t hw, int c, int groups,
                                                                     const __grid_constant__ EpiProgram pre,
                                                                     float* __restrict__ scratch) {
  constexpr int VE = Elem<T>::VEC;
  __shared__ float sh_s[GN_THREADS * VE];
  __shared__ float sh_q[GN_THREADS * VE];
  const int chunks = gridDim.x, chunk = blockIdx.x;
  const int64_t img = blockIdx.y;
  const int vpp = c / VE;
  const int vcol = threadIdx.x % vpp, prow = threadIdx.x / vpp, pstride = GN_THREADS / vpp;
  const int64_t p0 = hw * chunk / chunks, p1 = hw * (chunk + 1) / chunks;
  float s[VE], q[VE], piv[VE];
  const int cg_ = c / groups;
#pragma unroll
  for (int e = 0; e < VE; ++e) { s[e] = 0.0f; q[e] = 0.0f; piv[e] = gn_pivot(x, img, hw, c, (vcol * VE + e) / cg_, cg_, pre); }
  {
    const int64_t first = p0 + prow;
    const int n_my = first < p1 ? (int)((p1 - first + pstride - 1) / pstride) : 0;
    const uint4* ptr = reinterpret_cast<const uint4*>(x + (img * hw + first) * c + vcol * VE);
    const size_t step = (size_t)pstride * c / VE;             // 16-byte vectors between two pixels of this thread
    if (pre.n == 0) {
      walk16<GN_UN>(ptr, step, n_my, [&](const uint4& raw, int) {
        float v[VE];
        unpack16<T>(raw, v);
#pragma unroll
        for (int e = 0; e < VE; ++e) { const float d = v[e] - piv[e]; s[e] += d; q[e] = fmaf(d, d, q[e]); }
      });
    } else {
      walk16<GN_UN>(ptr, step, n_my, [&](const uint4& raw, int i) {
        float v[VE];
        unpack16<T>(raw, v);
        epi_apply_vec<T, VE>(pre, v, img * hw + first + (int64_t)i * pstride, (int64_t)vcol * VE, c);
#pragma unroll
        for (int e = 0; e < VE; ++e) { const float d = v[e] - piv[e]; s[e] += d; q[e] = fmaf(d, d, q[e]); }
      });
    }
  }
#pragma unroll
  for (int e = 0; e < VE; ++e) {
    sh_s[prow * c + vcol * VE + e] = s[e];
    sh_q[prow * c + vcol * VE + e] = q[e];
  }
  __syncthreads();
  const int cg = c / groups;
  for (int g = threadIdx.x; g < groups; g += GN_THREADS) {
    float ts = 0.0f, tq = 0.0f;
    for (int ch = g * cg; ch < (g + 1) * cg; ++ch)
      for (int r = 0; r < pstride; ++r) { ts += sh_s[r * c + ch]; tq += sh_q[r * c + ch]; }
    float* o = scratch + ((img * chunks + chunk) * groups + g) * 2;
    o[0] = ts;
    o[1] = tq;
  }
}

// Column sums of float [stat_slots][ncol] (ncol = 2 * groups <= 2 * GN_MAX_C partial sums per slot) into sh_stat[ncol],
// by the whole CTA; the caller synchronises before reading sh_stat.
__device__ __forceinline__ void gn_reduce_slots(const float* __restrict__ st, int stat_slots, int ncol, float* sh_stat, float (*sh_part)[2 * 64]) {
  // Reduction of the partials: 2 * groups columns, the slots of a column split over as many threads as
  // the CTA can spare, sixteen independent loads in flight per thread.
  int parts = GN_THREADS / ncol;
  if (parts < 1) parts = 1;
  if (parts > 8) parts = 8;
  const bool small = ncol <= 128 && parts > 1;
  const int quads = ncol / 4;                         // 16-byte pieces per slot
  if (ncol % 4 == 0 && quads <= 16 && GN_THREADS / quads <= 16 && stat_slots <= 8 * (GN_THREADS / quads)) {
    // a slot is a few hundred contiguous bytes: 16-byte loads, every thread's (at most eight) in flight at once,
    // so the whole reduction costs one round trip to L2 instead of two or more
    const int lanes = GN_THREADS / quads;             // slots read side by side
    const int qd = threadIdx.x % quads, sl = threadIdx.x / quads;
    float4 t[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int k = sl + u * lanes;
      t[u] = (sl < lanes && k < stat_slots) ? *reinterpret_cast<const float4*>(st + (int64_t)k * ncol + qd * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    float4 a = t[0];
#pragma unroll
    for (int u = 1; u < 8; ++u) { a.x += t[u].x; a.y += t[u].y; a.z += t[u].z; a.w += t[u].w; }
    float* pp = &sh_part[0][0];                        // [lanes <= 16][ncol <= 64] floats: 8 x 128 are enough
    if (sl < lanes) *reinterpret_cast<float4*>(pp + sl * ncol + qd * 4) = a;
    __syncthreads();
    if ((int)threadIdx.x < ncol) {
      float acc = 0.0f;
      for (int p = 0; p < lanes; ++p) acc += pp[p * ncol + threadIdx.x];
      sh_stat[threadIdx.x] = acc;
    }
  } else if (small) {
    const int col = threadIdx.x % ncol, part = threadIdx.x / ncol;
    if (part < parts) {
      float acc = 0.0f;
      for (int k0 = part; k0 < stat_slots; k0 += 16 * parts) {
        float t[16];
#pragma unroll
        for (int u = 0; u < 16; ++u) {
          const int k = k0 + u * parts;
          t[u] = k < stat_slots ? st[(int64_t)k * ncol + col] : 0.0f;
        }
#pragma unroll
        for (int u = 0; u < 16; ++u) acc += t[u];
      }
      sh_part[part][col] = acc;
    }
    __syncthreads();
    if ((int)threadIdx.x < ncol) {
      float acc = 0.0f;
      for (int p = 0; p < parts; ++p) acc += sh_part[p][threadIdx.x];
      sh_stat[threadIdx.x] = acc;
    }
  } else {
    for (int idx = threadIdx.x; idx < ncol; idx += GN_THREADS) {
      float acc = 0.0f;
      for (int k0 = 0; k0 < stat_slots; k0 += 16) {
        float t[16];
#pragma unroll
        for (int u = 0; u < 16; ++u) t[u] = k0 + u < stat_slots ? st[(int64_t)(k0 + u) * ncol + idx] : 0.0f;
#pragma unroll
        for (int u = 0; u < 16; ++u) acc += t[u];
      }
      sh_stat[idx] = acc;
    }
  }
}

template <typename T>
__global__ void __launch_bounds__(GN_THREADS, GN_RESIDENT) groupnorm_apply_kernel(const T* __restrict__ x, T* __restrict__ y, int64_t hw,
                                                                     int c, int groups, const T* __restrict__ gamma,
                                                                     const T* __restrict__ beta, float eps,
                                                                     const __grid_constant__ EpiProgram pre,
                                                                     const float* __restrict__ scratch) {
  constexpr int VE = Elem<T>::VEC;
  __shared__ float sh_scale[GN_MAX_C];
  __shared__ float sh_shift[GN_MAX_C];
  __shared__ float sh_stat[2 * GN_MAX_C];
  __shared__ float sh_part[8][2 * 64];
  const int chunks = gridDim.x, chunk = blockIdx.x;
  const int64_t img = blockIdx.y;
  const int cg = c / groups;
  const int vpp = c / VE;
  const int vcol = threadIdx.x % vpp, prow = threadIdx.x / vpp, pstride = GN_THREADS / vpp;
  const int64_t p0 = hw * chunk / chunks, p1 = hw * (chunk + 1) / chunks;
  const T* xin = x + (img * hw) * c + vcol * VE;
  T* yout = y + (img * hw) * c + vcol * VE;
  gn_reduce_slots(scratch + img * chunks * groups * 2, chunks, 2 * groups, sh_stat, sh_part);
  __syncthreads();
  const float inv_cnt = 1.0f / ((float)hw * (float)cg);
  for (int ch = threadIdx.x; ch < c; ch += GN_THREADS) {
    const int g = ch / cg;
    const float md = sh_stat[2 * g] * inv_cnt;                       // mean - pivot
    const float mean = gn_pivot(x, img, hw, c, g, cg, pre) + md;
    const float var = fmaxf(sh_stat[2 * g + 1] * inv_cnt - md * md, 0.0f);
    const float rstd = rsqrtf(var + eps);
    const float ga = gamma ? Elem<T>::ld(gamma + ch) : 1.0f;
    const float be = beta ? Elem<T>::ld(beta + ch) : 0.0f;
    sh_scale[ch] = rstd * ga;
    sh_shift[ch] = be - mean * rstd * ga;
  }
  __syncthreads();
  float sc[VE], sf[VE];
#pragma unroll
  for (int e = 0; e < VE; ++e) { sc[e] = sh_scale[vcol * VE + e]; sf[e] = sh_shift[vcol * VE + e]; }
  const int64_t first = p0 + prow;
  const int n_my = first < p1 ? (int)((p1 - first + pstride - 1) / pstride) : 0;
  const size_t step = (size_t)pstride * c / VE;
  const uint4* ptr = reinterpret_cast<const uint4*>(xin + first * c);
  uint4* out = reinterpret_cast<uint4*>(yout + first * c);
  if (pre.n == 0) {
    walk16<GN_UN>(ptr, step, n_my, [&](const uint4& raw, int i) {
      float v[VE];
      unpack16<T>(raw, v);
#pragma unroll
      for (int e = 0; e < VE; ++e) v[e] = fmaf(v[e], sc[e], sf[e]);
      out[(size_t)i * step] = pack16<T>(v);
    });
  } else {
    walk16<GN_UN>(ptr, step, n_my, [&](const uint4& raw, int i) {
      float v[VE];
      unpack16<T>(raw, v);
      epi_apply_vec<T, VE>(pre, v, img * hw + first + (int64_t)i * pstride, (int64_t)vcol * VE, c);
#pragma unroll
      for (int e = 0; e < VE; ++e) v[e] = fmaf(v[e], sc[e], sf[e]);
      out[(size_t)i * step] = pack16<T>(v);
    });
  }
}

// Any channel count: scalar accesses, shared-memory atomics for the group sums.
template <typename T>
__global__ void __launch_bounds__(GN_THREADS) groupnorm_stats_generic(const T* __restrict__ x, int64_t hw, int64_t c, int groups,
                                                                      const __grid_constant__ EpiProgram pre,
                                                                      float* __restrict__ scratch) {
  const int chunks = gridDim.x, chunk = blockIdx.x;
  const int64_t img = blockIdx.y;
  const int64_t cg = c / groups;
  const int64_t p0 = hw * chunk / chunks, p1 = hw * (chunk + 1) / chunks;
  float* out = scratch + (img * chunks + chunk) * groups * 2;
  for (int g = 0; g < groups; ++g) {  // one group at a time keeps shared memory constant-size
    __shared__ float sh[32];
    float s = 0.0f, q = 0.0f;
    const int64_t cnt = (p1 - p0) * cg;
    const float piv = gn_pivot(x, img, hw, c, g, cg, pre);
    for (int64_t i = threadIdx.x; i < cnt; i += GN_THREADS) {
      const int64_t pix = p0 + i / cg, ch = g * cg + i % cg;
      const int64_t r = img * hw + pix;
      const float d = epi_apply(pre, Elem<T>::ld(x + r * c + ch), r, ch, c) - piv;
      s += d;
      q = fmaf(d, d, q);
    }
    s = block_reduce<0>(s, sh);
    q = block_reduce<0>(q, sh);
    if (threadIdx.x == 0) { out[g * 2] = s; out[g * 2 + 1] = q; }
  }
}

template <typename T>
__global__ void __launch_bounds__(GN_THREADS) groupnorm_apply_generic(const T* __restrict__ x, T* __restrict__ y, int64_t hw,
                                                                      int64_t c, int groups, const T* __restrict__ gamma,
                                                                      const T* __restrict__ beta, float eps,
                                                                      const __grid_constant__ EpiProgram pre,
                                                                      const float* __restrict__ scratch) {
  const int chunks = gridDim.x, chunk = blockIdx.x;
  const int64_t img = blockIdx.y;
  const int64_t cg = c / groups;
  const float inv_cnt = 1.0f / ((float)hw * (float)cg);
  const int64_t p0 = hw * chunk / chunks, p1 = hw * (chunk + 1) / chunks;
  for (int64_t i = threadIdx.x; i < (p1 - p0) * c; i += GN_THREADS) {
    const int64_t pix = p0 + i / c, ch = i % c;
    const int g = (int)(ch / cg);
    float ts = 0.0f, tq = 0.0f;
    for (int k = 0; k < chunks; ++k) {
      const float* o = scratch + ((img * chunks + k) * groups + g) * 2;
      ts += o[0];
      tq += o[1];
    }
    const float md = ts * inv_cnt;                                   // mean - pivot
    const float mean = gn_pivot(x, img, hw, c, g, cg, pre) + md;
    const float rstd = rsqrtf(fmaxf(tq * inv_cnt - md * md, 0.0f) + eps);
    const int64_t r = img * hw + pix;
    float v = (epi_apply(pre, Elem<T>::ld(x + r * c + ch), r, ch, c) - mean) * rstd;
    if (gamma) v *= Elem<T>::ld(gamma + ch);
    if (beta) v += Elem<T>::ld(beta + ch);
    Elem<T>::st(y + r * c + ch, v);
  }
}

// Normalisation from partial sums that another kernel (the convolution's epilogue) has left behind:
// float [nb][stat_slots][groups][2].  One CTA = one pixel chunk of one image.  The first batch of
// activation loads is issued BEFORE the statistics are reduced (they do not depend on them), and the
// main loop keeps a batch of 16-byte loads in flight while it normalises and stores the previous one.
template <typename T>
__global__ void __launch_bounds__(GN_THREADS, 3) groupnorm_apply_partials_kernel(const T* __restrict__ x, T* __restrict__ y, int64_t hw, int c,
                                                                              int groups, const T* __restrict__ gamma,
                                                                              const T* __restrict__ beta, float eps,
                                                                              const float* __restrict__ stats, int stat_slots) {
  constexpr int VE = Elem<T>::VEC;
  constexpr int UN = 4;
  __shared__ float sh_scale[GN_MAX_C];
  __shared__ float sh_shift[GN_MAX_C];
  __shared__ float sh_stat[2 * GN_MAX_C];
  __shared__ float sh_part[8][2 * 64];
  const int chunks = gridDim.x, chunk = blockIdx.x;
  const int64_t img = blockIdx.y;
  const int cg = c / groups;
  const int vpp = c / VE;
  const int vcol = threadIdx.x % vpp, prow = threadIdx.x / vpp, pstride = GN_THREADS / vpp;
  const int64_t p0 = hw * chunk / chunks, p1 = hw * (chunk + 1) / chunks;
  const T* xin = x + (img * hw) * c + vcol * VE;
  T* yout = y + (img * hw) * c + vcol * VE;
  pdl_launch_dependents();
  pdl_wait();   // x and the partial sums come from the kernel before this one
  RawVec<T, VE> cur[UN];
  int64_t pix = p0 + prow;
#pragma unroll
  for (int u = 0; u < UN; ++u)
    if (pix + (int64_t)u * pstride < p1) cur[u].load(xin + (pix + (int64_t)u * pstride) * c);

  gn_reduce_slots(stats + img * stat_slots * groups * 2, stat_slots, 2 * groups, sh_stat, sh_part);
  __syncthreads();
  const float inv_cnt = 1.0f / ((float)hw * (float)cg);
  for (int ch = threadIdx.x; ch < c; ch += GN_THREADS) {
    const int g = ch / cg;
    const float mean = sh_stat[2 * g] * inv_cnt;
    const float var = fmaxf(sh_stat[2 * g + 1] * inv_cnt - mean * mean, 0.0f);
    const float rstd = rsqrtf(var + eps);
    const float ga = gamma ? Elem<T>::ld(gamma + ch) : 1.0f;
    const float be = beta ? Elem<T>::ld(beta + ch) : 0.0f;
    sh_scale[ch] = rstd * ga;
    sh_shift[ch] = be - mean * rstd * ga;
  }
  __syncthreads();
  float sc[VE], sf[VE];
#pragma unroll
  for (int e = 0; e < VE; ++e) { sc[e] = sh_scale[vcol * VE + e]; sf[e] = sh_shift[vcol * VE + e]; }
  for (; pix < p1; pix += (int64_t)UN * pstride) {
    RawVec<T, VE> nxt[UN];
    const int64_t npix = pix + (int64_t)UN * pstride;
#pragma unroll
    for (int u = 0; u < UN; ++u)
      if (npix + (int64_t)u * pstride < p1) nxt[u].load(xin + (npix + (int64_t)u * pstride) * c);
#pragma unroll
    for (int u = 0; u < UN; ++u) {
      const int64_t pp = pix + (int64_t)u * pstride;
      if (pp < p1) {
        float v[VE];
        cur[u].unpack(v);
#pragma unroll
        for (int e = 0; e < VE; ++e) v[e] = fmaf(v[e], sc[e], sf[e]);
        st_vec(yout + pp * c, v);
      }
    }
#pragma unroll
    for (int u = 0; u < UN; ++u) cur[u] = nxt[u];
  }
}

bool groupnorm_apply_partials_supported(int dtype, int64_t c, int groups) {
  if (groups < 1 || c % groups) return false;
  return dtype == DT_F32 ? gn_fast_ok<float>(c) : gn_fast_ok<__nv_bfloat16>(c);
}
cudaError_t launch_groupnorm_apply_partials(int dtype, const void* x, void* y, int64_t nb, int64_t hw, int64_t c, int groups,
                                            const void* gamma, const void* beta, float eps, const float* stats, int stat_slots,
                                            int sm_count, cudaStream_t s) {
  if (nb == 0) return cudaSuccess;
  if (!groupnorm_apply_partials_supported(dtype, c, groups)) return cudaErrorInvalidValue;
  // exactly one wave: as many pixel chunks per image as the resident CTAs of the whole GPU allow
  int occ = 0;
  cudaError_t oe = dtype == DT_F32
                       ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, groupnorm_apply_partials_kernel<float>, GN_THREADS, 0)
                       : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, groupnorm_apply_partials_kernel<__nv_bfloat16>, GN_THREADS, 0);
  if (oe != cudaSuccess) return oe;
  if (occ < 1) occ = 1;
  int64_t chunks = ((int64_t)occ * sm_count) / nb;
  const int64_t maxc = hw / 64 > 0 ? hw / 64 : 1;
  if (chunks > maxc) chunks = maxc;
  if (chunks < 1) chunks = 1;
  dim3 grid((unsigned)chunks, (unsigned)nb);
  LaunchCfg lc(PDL_GROUPNORM, grid, dim3(GN_THREADS), 0, s);
  if (dtype == DT_F32)
    return cudaLaunchKernelEx(&lc.cfg, groupnorm_apply_partials_kernel<float>, (const float*)x, (float*)y, hw, (int)c, groups, (const float*)gamma,
                              (const float*)beta, eps, stats, stat_slots);
  return cudaLaunchKernelEx(&lc.cfg, groupnorm_apply_partials_kernel<__nv_bfloat16>, (const __nv_bfloat16*)x, (__nv_bfloat16*)y, hw, (int)c, groups,
                            (const __nv_bfloat16*)gamma, (const __nv_bfloat16*)beta, eps, stats, stat_slots);
}

template <typename T>
static cudaError_t gn_stats(const void* x, int64_t nb, int64_t hw, int64_t c, int groups, const EpiProgram& pre, float* scratch,
                            int chunks, cudaStream_t s) {
  if (nb == 0) return cudaSuccess;
  dim3 grid(chunks, (unsigned)nb);
  if (gn_fast_ok<T>(c)) groupnorm_stats_kernel<T><<<grid, GN_THREADS, 0, s>>>((const T*)x, hw, (int)c, groups, pre, scratch);
  else groupnorm_stats_generic<T><<<grid, GN_THREADS, 0, s>>>((const T*)x, hw, c, groups, pre, scratch);
  return cudaGetLastError();
}
template <typename T>
static cudaError_t gn_apply(const void* x, void* y, int64_t nb, int64_t hw, int64_t c, int groups, const void* g, const void* b,
                            float eps, const EpiProgram& pre, const float* scratch, int chunks, cudaStream_t s) {
  if (nb == 0) return cudaSuccess;
  dim3 grid(chunks, (unsigned)nb);
  if (gn_fast_ok<T>(c))
    groupnorm_apply_kernel<T><<<grid, GN_THREADS, 0, s>>>((const T*)x, (T*)y, hw, (int)c, groups, (const T*)g, (const T*)b, eps, pre, scratch);
  else
    groupnorm_apply_generic<T><<<grid, GN_THREADS, 0, s>>>((const T*)x, (T*)y, hw, c, groups, (const T*)g, (const T*)b, eps, pre, scratch);
  return cudaGetLastError();
}

cudaError_t launch_groupnorm_stats(int dtype, const void* x, int64_t nb, int64_t hw, int64_t c, int groups, const EpiProgram& pre,
                                   float* scratch, int chunks, cudaStream_t s) {
  return dtype == DT_F32 ? gn_stats<float>(x, nb, hw, c, groups, pre, scratch, chunks, s)
                         : gn_stats<__nv_bfloat16>(x, nb, hw, c, groups, pre, scratch, chunks, s);
}
cudaError_t launch_groupnorm_apply(int dtype, const void* x, void* y, int64_t nb, int64_t hw, int64_t c, int groups,
                                   const void* gamma, const void* beta, float eps, const EpiProgram& pre, const float* scratch,
                                   int chunks, cudaStream_t s) {
  return dtype == DT_F32 ? gn_apply<float>(x, y, nb, hw, c, groups, gamma, beta, eps, pre, scratch, chunks, s)
                         : gn_apply<__nv_bfloat16>(x, y, nb, hw, c, groups, gamma, beta, eps, pre, scratch, chunks, s);
}

}  // namespace mk
