// Plain-ALU subkernels: any shape, fp32 or bf16 storage, fp32 FMA accumulation (no TF32: the fp32
// tolerance rtol 1e-4 / atol 1e-5 rules it out, as the paper's own fp32 setting does).  They are the
// always-legal implementations the composer falls back to for shapes the tensor-core kernels do
// not take, the alternatives a submodule can be swapped to, and — for the small fp32 chain — the
// fused single-launch kernel in which one CTA owns whole rows so the row norm needs no second pass
// over memory.
#include "device_common.cuh"
#include "tc_common.cuh"

namespace mk {

// =====================================================================================================
// tiled GEMM, 64x64 tile, 16x16 threads, 4x4 micro-tile
// =====================================================================================================
template <typename T, typename TO, bool SWIGLU>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const T* __restrict__ a, const T* __restrict__ w, bool wt,
                                                        TO* __restrict__ y, int64_t M, int64_t N, int64_t K,
                                                        const __grid_constant__ EpiProgram p) {
  constexpr int BM = 64, BN = 64, BK = 16;
  __shared__ float As[BK][BM + 1];
  __shared__ float Ws[SWIGLU ? 2 : 1][BK][BN + 1];
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  const int64_t m0 = (int64_t)blockIdx.y * BM, n0 = (int64_t)blockIdx.x * BN;
  const int64_t ldw = SWIGLU ? 2 * N : N;  // logical columns of W
  float acc[4][4] = {};
  float acc2[SWIGLU ? 4 : 1][4] = {};
  for (int64_t k0 = 0; k0 < K; k0 += BK) {
    for (int i = threadIdx.x; i < BM * BK; i += 256) {
      const int mm = i / BK, kk = i % BK;
      const int64_t gm = m0 + mm, gk = k0 + kk;
      As[kk][mm] = (gm < M && gk < K) ? Elem<T>::ld(a + gm * K + gk) : 0.0f;
    }
    for (int i = threadIdx.x; i < BN * BK; i += 256) {
      int nn, kk;
      if (wt) { nn = i / BK; kk = i % BK; } else { kk = i / BN; nn = i % BN; }
      const int64_t gn = n0 + nn, gk = k0 + kk;
      const bool ok = gn < N && gk < K;
      Ws[0][kk][nn] = ok ? Elem<T>::ld(wt ? w + gn * K + gk : w + gk * ldw + gn) : 0.0f;
      if (SWIGLU) Ws[1][kk][nn] = ok ? Elem<T>::ld(wt ? w + (N + gn) * K + gk : w + gk * ldw + N + gn) : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float av[4], bv[4], cv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) av[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        bv[j] = Ws[0][kk][tx * 4 + j];
        if (SWIGLU) cv[j] = Ws[1][kk][tx * 4 + j];
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
          if (SWIGLU) acc2[i][j] = fmaf(av[i], cv[j], acc2[i][j]);
        }
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int64_t gm = m0 + ty * 4 + i, gn = n0 + tx * 4 + j;
      if (gm < M && gn < N) {
        float v = acc[i][j];
        if (SWIGLU) v = silu_f(v) * acc2[i][j];
        Elem<TO>::st(y + gm * N + gn, epi_apply(p, v, gm, gn, N));
      }
    }
}

template <typename T, typename TO>
static cudaError_t gemm_simt_dispatch(const void* a, const void* w, bool wt, void* y, int64_t m, int64_t n, int64_t k, bool swiglu,
                                      const EpiProgram& p, cudaStream_t s) {
  if (m == 0 || n == 0) return cudaSuccess;
  dim3 grid((unsigned)((n + 63) / 64), (unsigned)((m + 63) / 64));
  if (swiglu) gemm_simt_kernel<T, TO, true><<<grid, 256, 0, s>>>((const T*)a, (const T*)w, wt, (TO*)y, m, n, k, p);
  else gemm_simt_kernel<T, TO, false><<<grid, 256, 0, s>>>((const T*)a, (const T*)w, wt, (TO*)y, m, n, k, p);
  return cudaGetLastError();
}

// =====================================================================================================
// The same fused chain on a thread-block cluster, for the small problems whose whole time is latency (N <= 256):
// a cluster of eight CTAs owns eight rows, each CTA a slice of the columns, so a CTA loads an eighth of W
// instead of all of it; the row statistics meet through distributed shared memory (every CTA writes its
// partial sums into all eight CTAs' slots, one cluster barrier per statistic).  Two-pass LayerNorm
// (mean, then centred squares), as in the single-CTA form.
// =====================================================================================================
constexpr int LC_CL = 8;         // CTAs per cluster
constexpr int LC_RB = 8;         // rows per cluster
constexpr int LC_THREADS = 256;
constexpr int LC_MAXNC = 32;     // columns per CTA: N <= LC_CL * LC_MAXNC

__device__ __forceinline__ void st_cluster_f32(uint32_t cluster_addr, float v) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(cluster_addr), "f"(v) : "memory");
}

template <typename T>
__global__ void __launch_bounds__(LC_THREADS) linear_rownorm_cluster_kernel(const T* __restrict__ a, const T* __restrict__ w, bool wt,
                                                                            T* __restrict__ y, int M, int N, int K, int NC,
                                                                            const __grid_constant__ EpiProgram p, int mode,
                                                                            const T* __restrict__ gamma, const T* __restrict__ beta,
                                                                            float eps) {
  extern __shared__ float smem[];
  const int KP = K + 1;                                    // odd pitch: threads of different columns hit different banks
  float* xs = smem;                                        // [LC_RB][K]
  float* ws = xs + LC_RB * K;                              // [NC][KP]: this CTA's columns of W, K contiguous
  float* part = ws + NC * KP;                              // [KS][LC_RB * NC]
  __shared__ float val[LC_RB][LC_MAXNC];                   // this CTA's outputs after the elementwise tail
  __shared__ float slot[2][LC_CL][LC_RB];                  // row partial sums of every CTA of the cluster (two statistics)
  __shared__ float stat[2][LC_RB];
  pdl_launch_dependents();
  // A CTA may write into a peer's shared memory only once that peer is running: every CTA announces itself
  // here and waits for the others just before its first remote store, so the rendezvous costs nothing.
  tc::cluster_arrive();
  pdl_wait();
  const uint32_t rank = tc::cluster_ctarank();
  const int m0 = (int)(blockIdx.x / LC_CL) * LC_RB, c0 = (int)rank * NC;
  const int nc = min(NC, N - c0) > 0 ? min(NC, N - c0) : 0;   // columns of this CTA that exist
  // Everything that is read late - the norm's scale and shift, a bias vector inside the elementwise tail - is asked
  // for now: a dependent global load at the end of this kernel would be a tenth of its whole duration.
  float ga = 1.0f, be = 0.0f;
  {
    const int rj = threadIdx.x, j = rj % NC;
    if (rj < LC_RB * NC && j < nc) {
      if (gamma) ga = Elem<T>::ld(gamma + c0 + j);
      if (mode == ROW_LAYERNORM && beta) be = Elem<T>::ld(beta + c0 + j);
      for (int i = 0; i < p.n; ++i)
        if (p.op[i].kind == EPI_BIAS && p.op[i].ptr)
          asm volatile("prefetch.global.L1 [%0];" ::"l"(reinterpret_cast<const char*>(p.op[i].ptr) + (size_t)(c0 + j) * sizeof(T)));
    }
  }
  constexpr int VE = Elem<T>::VEC;
  if (K % VE == 0) {
    // 16-byte loads, all of a thread's in flight together: the whole kernel is a few round trips to L2 long
    const int kv = K / VE;
    for (int i = threadIdx.x; i < LC_RB * kv; i += LC_THREADS) {
      const int r = i / kv, k = (i - r * kv) * VE;
      float v[VE];
      if (m0 + r < M) {
        ld_vec(a + (int64_t)(m0 + r) * K + k, v);
      } else {
#pragma unroll
        for (int e = 0; e < VE; ++e) v[e] = 0.0f;
      }
#pragma unroll
      for (int e = 0; e < VE; ++e) xs[r * K + k + e] = v[e];
    }
  } else {
    for (int i = threadIdx.x; i < LC_RB * K; i += LC_THREADS) {
      const int r = i / K, k = i - r * K;
      xs[i] = (m0 + r < M) ? Elem<T>::ld(a + (int64_t)(m0 + r) * K + k) : 0.0f;
    }
  }
  if (wt && K % VE == 0) {
    const int kv = K / VE;
    for (int i = threadIdx.x; i < nc * kv; i += LC_THREADS) {
      const int j = i / kv, k = (i - j * kv) * VE;
      float v[VE];
      ld_vec(w + (int64_t)(c0 + j) * K + k, v);
#pragma unroll
      for (int e = 0; e < VE; ++e) ws[j * KP + k + e] = v[e];
    }
  } else if (wt) {
    for (int i = threadIdx.x; i < nc * K; i += LC_THREADS) {
      const int j = i / K, k = i - j * K;                   // consecutive threads walk K: contiguous in memory
      ws[j * KP + k] = Elem<T>::ld(w + (int64_t)(c0 + j) * K + k);
    }
  } else {
    for (int i = threadIdx.x; i < nc * K; i += LC_THREADS) {
      const int k = i / nc, j = i - k * nc;                 // consecutive threads walk the columns: contiguous in memory
      ws[j * KP + k] = Elem<T>::ld(w + (int64_t)k * N + c0 + j);
    }
  }
  __syncthreads();
  // outputs r * NC + j; the threads beyond them split K
  const int outs = LC_RB * NC;
  const int KS = LC_THREADS / outs > 0 ? LC_THREADS / outs : 1;
  for (int o = threadIdx.x; o < outs * KS; o += LC_THREADS) {
    const int ks = o / outs, rj = o - ks * outs, r = rj / NC, j = rj - r * NC;
    const int kper = (K + KS - 1) / KS, kb = ks * kper, ke = min(K, kb + kper);
    float acc = 0.0f;
    if (j < nc) {
      const float* xr = xs + r * K;
      const float* wr = ws + j * KP;
#pragma unroll 8
      for (int k = kb; k < ke; ++k) acc = fmaf(xr[k], wr[k], acc);
    }
    part[ks * outs + rj] = acc;
  }
  __syncthreads();
  for (int rj = threadIdx.x; rj < outs; rj += LC_THREADS) {
    const int r = rj / NC, j = rj - r * NC;
    float v = 0.0f;
    for (int q = 0; q < KS; ++q) v += part[q * outs + rj];       // fixed order
    val[r][j] = j < nc ? epi_apply(p, v, m0 + r, c0 + j, N) : 0.0f;
  }
  __syncthreads();
  tc::cluster_wait();   // all eight CTAs of the cluster are resident from here on
  const float inv_n = 1.0f / (float)N;
  // statistic 0: the row sums (LayerNorm) -> mean
  if (mode == ROW_LAYERNORM) {
    if (threadIdx.x < LC_RB) {
      float sm = 0.0f;
      for (int j = 0; j < nc; ++j) sm += val[threadIdx.x][j];
      const uint32_t local = tc::smem_u32(&slot[0][rank][threadIdx.x]);
      for (uint32_t c = 0; c < LC_CL; ++c) st_cluster_f32(tc::map_to_cta(local, c), sm);
    }
    tc::cluster_sync();
    if (threadIdx.x < LC_RB) {
      float sm = 0.0f;
      for (int c = 0; c < LC_CL; ++c) sm += slot[0][c][threadIdx.x];   // the same order in every CTA
      stat[0][threadIdx.x] = sm * inv_n;
    }
  } else if (threadIdx.x < LC_RB) {
    stat[0][threadIdx.x] = 0.0f;
  }
  __syncthreads();
  // statistic 1: centred squares -> 1 / sqrt(var + eps)  (RMSNorm: squares about zero)
  if (threadIdx.x < LC_RB) {
    const float mean = stat[0][threadIdx.x];
    float q = 0.0f;
    for (int j = 0; j < nc; ++j) { const float d = val[threadIdx.x][j] - mean; q += d * d; }
    const uint32_t local = tc::smem_u32(&slot[1][rank][threadIdx.x]);
    for (uint32_t c = 0; c < LC_CL; ++c) st_cluster_f32(tc::map_to_cta(local, c), q);
  }
  tc::cluster_sync();
  if (threadIdx.x < LC_RB) {
    float q = 0.0f;
    for (int c = 0; c < LC_CL; ++c) q += slot[1][c][threadIdx.x];
    stat[1][threadIdx.x] = rsqrtf(q * inv_n + eps);
  }
  __syncthreads();
  for (int rj = threadIdx.x; rj < outs; rj += LC_THREADS) {
    const int r = rj / NC, j = rj - r * NC;
    if (j < nc && m0 + r < M) {
      const int c = c0 + j;
      const float o = (val[r][j] - stat[0][r]) * stat[1][r] * ga + be;
      Elem<T>::st(y + (int64_t)(m0 + r) * N + c, o);
    }
  }
  // nobody writes into a peer's shared memory after the second cluster barrier: a CTA may retire here
}

template <typename T>
static cudaError_t linear_rownorm_cluster_launch(const void* a, const void* w, bool wt, void* y, int64_t m, int64_t n, int64_t k,
                                                 const EpiProgram& p, int mode, const void* g, const void* b, float eps, cudaStream_t s) {
  int NC = (int)((n + LC_CL - 1) / LC_CL);
  // a power of two keeps LC_RB * NC a divisor of the CTA size, so the idle threads split K evenly
  int pw = 1;
  while (pw < NC) pw *= 2;
  NC = pw;
  const int outs = LC_RB * NC, KS = LC_THREADS / outs > 0 ? LC_THREADS / outs : 1;
  const size_t smem = sizeof(float) * ((size_t)LC_RB * k + (size_t)NC * (k + 1) + (size_t)KS * outs);
  static SmemOptIn opt_in;   // one per instantiation (T)
  if (smem > 48 * 1024) {
    cudaError_t e = opt_in.ensure(smem, linear_rownorm_cluster_kernel<T>);
    if (e != cudaSuccess) return e;
  }
  const unsigned grid = (unsigned)((m + LC_RB - 1) / LC_RB) * LC_CL;
  LaunchCfg lc(PDL_ELTWISE, dim3(grid), dim3(LC_THREADS), smem, s, LC_CL);
  return cudaLaunchKernelEx(&lc.cfg, linear_rownorm_cluster_kernel<T>, (const T*)a, (const T*)w, wt, (T*)y, (int)m, (int)n, (int)k, NC, p, mode,
                            (const T*)g, (const T*)b, eps);
}
// what the cluster form takes: a row norm with two statistics at most, few columns, operands that fit
static bool linear_rownorm_cluster_ok(int64_t m, int64_t n, int64_t k, int mode) {
  if (mode != ROW_LAYERNORM && mode != ROW_RMSNORM) return false;
  if (n > LC_CL * LC_MAXNC || n < LC_CL || k > 2048 || m > (1 << 20)) return false;
  return sizeof(float) * ((size_t)(LC_RB + LC_MAXNC) * (k + 1) + LC_THREADS) <= 160 * 1024;
}

template <typename T>
static cudaError_t linear_rownorm_dispatch(const void* a, const void* w, bool wt, void* y, int64_t m, int64_t n, int64_t k,
                                           const EpiProgram& p, int mode, const void* g, const void* b, float eps,
                                           cudaStream_t s);

cudaError_t launch_gemm_simt(int dtype, int out_dtype, const void* a, const void* w, bool w_transposed, void* y, int64_t m, int64_t n,
                             int64_t k, bool swiglu, const EpiProgram& p, cudaStream_t s) {
  // A problem too small to fill the machine with 64 x 64 tiles runs faster row by row with K split inside
  // the CTA (the small-shape kernel below without its norm).
  if (!swiglu && dtype == out_dtype && m * n <= 64 * 1024 && n <= 1024 && k <= 8192) {
    cudaError_t e = dtype == DT_F32 ? linear_rownorm_dispatch<float>(a, w, w_transposed, y, m, n, k, p, -1, nullptr, nullptr, 0.0f, s)
                                    : linear_rownorm_dispatch<__nv_bfloat16>(a, w, w_transposed, y, m, n, k, p, -1, nullptr, nullptr, 0.0f, s);
    if (e != cudaErrorInvalidValue) return e;
  }
  if (dtype == DT_F32) return out_dtype == DT_F32 ? gemm_simt_dispatch<float, float>(a, w, w_transposed, y, m, n, k, swiglu, p, s) : cudaErrorInvalidValue;
  return out_dtype == DT_F32 ? gemm_simt_dispatch<__nv_bfloat16, float>(a, w, w_transposed, y, m, n, k, swiglu, p, s)
                             : gemm_simt_dispatch<__nv_bfloat16, __nv_bfloat16>(a, w, w_transposed, y, m, n, k, swiglu, p, s);
}

// =====================================================================================================
// small-shape fused chain: linear -> elementwise tail -> row norm, one launch
// CTA = LR_ROWS rows x all N columns; K is split over LR_THREADS / NT thread groups whose partial
// sums meet in shared memory; then one warp per row normalises.
// =====================================================================================================
constexpr int LR_ROWS = 2;
constexpr int LR_THREADS = 512;
constexpr int LR_MAXC = 4;  // columns per thread: N <= NT * LR_MAXC

template <typename T>
__global__ void __launch_bounds__(LR_THREADS) linear_rownorm_kernel(const T* __restrict__ a, const T* __restrict__ w, bool wt,
                                                                    T* __restrict__ y, int M, int N, int K, int NT,
                                                                    const __grid_constant__ EpiProgram p, int mode,
                                                                    const T* __restrict__ gamma, const T* __restrict__ beta,
                                                                    float eps) {
  extern __shared__ float smem[];
  float* xs = smem;                         // [LR_ROWS][K]
  float* part = smem + LR_ROWS * K;         // [KS][LR_ROWS][N]
  const int KS = LR_THREADS / NT;
  const int ct = threadIdx.x % NT, ks = threadIdx.x / NT;
  const int m0 = blockIdx.x * LR_ROWS;
  for (int i = threadIdx.x; i < LR_ROWS * K; i += LR_THREADS) {
    const int r = i / K, k = i - r * K;
    xs[i] = (m0 + r < M) ? Elem<T>::ld(a + (int64_t)(m0 + r) * K + k) : 0.0f;
  }
  __syncthreads();
  const int kper = (K + KS - 1) / KS;
  const int kb = ks * kper, ke = min(K, kb + kper);
  float acc[LR_ROWS][LR_MAXC] = {};
  constexpr int VE = Elem<T>::VEC;
  const bool vec_k = wt && K % VE == 0 && kper % VE == 0;
  if (ks < KS && vec_k) {
    // W stored [N, K]: a column's K-slice is contiguous, so every thread streams 16-byte vectors of its own
    // columns (a scalar load here would fetch a whole sector per lane for one element)
#pragma unroll 4
    for (int k = kb; k < ke; k += VE) {
      float wv[LR_MAXC][VE];
#pragma unroll
      for (int j = 0; j < LR_MAXC; ++j) {
        const int c = ct + j * NT;
        if (c < N) {
          ld_vec(w + (int64_t)c * K + k, wv[j]);
        } else {
#pragma unroll
          for (int e = 0; e < VE; ++e) wv[j][e] = 0.0f;
        }
      }
#pragma unroll
      for (int r = 0; r < LR_ROWS; ++r)
#pragma unroll
        for (int e = 0; e < VE; ++e) {
          const float xv = xs[r * K + k + e];
#pragma unroll
          for (int j = 0; j < LR_MAXC; ++j) acc[r][j] = fmaf(xv, wv[j][e], acc[r][j]);
        }
    }
  } else if (ks < KS) {
#pragma unroll 8
    for (int k = kb; k < ke; ++k) {
      float wv[LR_MAXC];
#pragma unroll
      for (int j = 0; j < LR_MAXC; ++j) {
        const int c = ct + j * NT;
        wv[j] = (c < N) ? Elem<T>::ld(wt ? w + (int64_t)c * K + k : w + (int64_t)k * N + c) : 0.0f;
      }
#pragma unroll
      for (int r = 0; r < LR_ROWS; ++r)
#pragma unroll
        for (int j = 0; j < LR_MAXC; ++j) acc[r][j] = fmaf(xs[r * K + k], wv[j], acc[r][j]);
    }
#pragma unroll
    for (int r = 0; r < LR_ROWS; ++r)
#pragma unroll
      for (int j = 0; j < LR_MAXC; ++j) {
        const int c = ct + j * NT;
        if (c < N) part[(ks * LR_ROWS + r) * N + c] = acc[r][j];
      }
  }
  if (ks < KS && vec_k) {
#pragma unroll
    for (int r = 0; r < LR_ROWS; ++r)
#pragma unroll
      for (int j = 0; j < LR_MAXC; ++j) {
        const int c = ct + j * NT;
        if (c < N) part[(ks * LR_ROWS + r) * N + c] = acc[r][j];
      }
  }
  __syncthreads();
  // sum the K-slices in a fixed order, apply the elementwise tail; result overwrites slice 0
  for (int i = threadIdx.x; i < LR_ROWS * N; i += LR_THREADS) {
    const int r = i / N, c = i - r * N;
    float v = 0.0f;
    for (int q = 0; q < KS; ++q) v += part[(q * LR_ROWS + r) * N + c];
    part[r * N + c] = epi_apply(p, v, m0 + r, c, N);
  }
  __syncthreads();
  if (mode < 0) {
    // no row norm: the fused linear + elementwise tail of a small problem
    for (int i = threadIdx.x; i < LR_ROWS * N; i += LR_THREADS) {
      const int r = i / N, c = i - r * N;
      if (m0 + r < M) Elem<T>::st(y + (int64_t)(m0 + r) * N + c, part[r * N + c]);
    }
    return;
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (warp < LR_ROWS && m0 + warp < M) {
    const float* row = part + warp * N;
    const float inv_n = 1.0f / (float)N;
    float mean = 0.0f;
    if (mode == ROW_LAYERNORM) {
      float s = 0.0f;
      for (int c = lane; c < N; c += 32) s += row[c];
      mean = warp_sum(s) * inv_n;
    }
    float q = 0.0f;
    for (int c = lane; c < N; c += 32) { const float d = row[c] - mean; q += d * d; }
    const float rstd = rsqrtf(warp_sum(q) * inv_n + eps);
    T* yr = y + (int64_t)(m0 + warp) * N;
    for (int c = lane; c < N; c += 32) {
      float o = (row[c] - mean) * rstd;
      if (gamma) o *= Elem<T>::ld(gamma + c);
      if (mode == ROW_LAYERNORM && beta) o += Elem<T>::ld(beta + c);
      Elem<T>::st(yr + c, o);
    }
  }
}

template <typename T>
static cudaError_t linear_rownorm_dispatch(const void* a, const void* w, bool wt, void* y, int64_t m, int64_t n, int64_t k,
                                           const EpiProgram& p, int mode, const void* g, const void* b, float eps,
                                           cudaStream_t s) {
  if (m == 0) return cudaSuccess;
  if (linear_rownorm_cluster_ok(m, n, k, mode)) return linear_rownorm_cluster_launch<T>(a, w, wt, y, m, n, k, p, mode, g, b, eps, s);
  // fewest column threads that cover N with LR_MAXC columns each: the rest of the CTA splits K, which
  // shortens every thread's chain of loads
  int NT = 32;
  while ((int64_t)NT * LR_MAXC < n && NT < 256) NT *= 2;
  if ((int64_t)NT * LR_MAXC < n) return cudaErrorInvalidValue;
  const int KS = LR_THREADS / NT;
  const size_t smem = sizeof(float) * ((size_t)LR_ROWS * k + (size_t)KS * LR_ROWS * n);
  if (smem > 200 * 1024) return cudaErrorInvalidValue;
  static SmemOptIn opt_in;   // one per instantiation (T)
  {
    cudaError_t e = opt_in.ensure(200 * 1024, linear_rownorm_kernel<T>);
    if (e != cudaSuccess) return e;
  }
  const int grid = (int)((m + LR_ROWS - 1) / LR_ROWS);
  linear_rownorm_kernel<T><<<grid, LR_THREADS, smem, s>>>((const T*)a, (const T*)w, wt, (T*)y, (int)m, (int)n, (int)k, NT, p, mode,
                                                          (const T*)g, (const T*)b, eps);
  return cudaGetLastError();
}

cudaError_t launch_linear_rownorm_simt(int dtype, const void* a, const void* w, bool w_transposed, void* y, int64_t m, int64_t n,
                                       int64_t k, const EpiProgram& p, int mode, const void* gamma, const void* beta, float eps,
                                       cudaStream_t s) {
  return dtype == DT_F32 ? linear_rownorm_dispatch<float>(a, w, w_transposed, y, m, n, k, p, mode, gamma, beta, eps, s)
                         : linear_rownorm_dispatch<__nv_bfloat16>(a, w, w_transposed, y, m, n, k, p, mode, gamma, beta, eps, s);
}

// =====================================================================================================
// direct 3x3 convolution, NHWC, one thread per output element
// =====================================================================================================
template <typename T>
__global__ void __launch_bounds__(256) conv3x3_simt_kernel(const T* __restrict__ x, const T* __restrict__ w, T* __restrict__ y,
                                                           int64_t nb, int h, int wd, int c, int co,
                                                           const __grid_constant__ EpiProgram p) {
  const int64_t total = nb * h * wd * co;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int o = (int)(i % co);
    const int64_t pix = i / co;
    const int px = (int)(pix % wd);
    const int py = (int)((pix / wd) % h);
    const int64_t n = pix / ((int64_t)wd * h);
    float acc = 0.0f;
    for (int a = 0; a < 3; ++a) {
      const int iy = py + a - 1;
      if (iy < 0 || iy >= h) continue;
      for (int b = 0; b < 3; ++b) {
        const int ix = px + b - 1;
        if (ix < 0 || ix >= wd) continue;
        const T* xp = x + ((n * h + iy) * wd + ix) * c;
        const T* wp = w + ((int64_t)(o * 3 + a) * 3 + b) * c;
        for (int ch = 0; ch < c; ++ch) acc = fmaf(Elem<T>::ld(xp + ch), Elem<T>::ld(wp + ch), acc);
      }
    }
    Elem<T>::st(y + i, epi_apply(p, acc, pix, o, co));
  }
}

cudaError_t launch_conv3x3_simt(int dtype, const void* x, const void* w, void* y, int64_t nb, int64_t h, int64_t wd, int64_t c,
                                int64_t co, const EpiProgram& p, cudaStream_t s) {
  const int64_t total = nb * h * wd * co;
  if (total == 0) return cudaSuccess;
  int64_t g = (total + 255) / 256;
  if (g > 148 * 64) g = 148 * 64;
  if (dtype == DT_F32)
    conv3x3_simt_kernel<float><<<(unsigned)g, 256, 0, s>>>((const float*)x, (const float*)w, (float*)y, nb, (int)h, (int)wd, (int)c, (int)co, p);
  else
    conv3x3_simt_kernel<__nv_bfloat16><<<(unsigned)g, 256, 0, s>>>((const __nv_bfloat16*)x, (const __nv_bfloat16*)w, (__nv_bfloat16*)y, nb,
                                                                   (int)h, (int)wd, (int)c, (int)co, p);
  return cudaGetLastError();
}

// =====================================================================================================
// causal attention, one warp per (batch, head, query); online softmax over the keys j <= i
// =====================================================================================================
template <typename T>
__global__ void __launch_bounds__(128) attention_simt_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                                                             T* __restrict__ o, int64_t sb, int64_t sh, int64_t ss, int64_t B, int H,
                                                             int S, int D, int causal) {
  constexpr int MAXE = 8;  // D <= 256
  const int lane = threadIdx.x & 31;
  const int64_t wid = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (wid >= B * H * S) return;
  const int i = (int)(wid % S);
  const int h = (int)((wid / S) % H);
  const int64_t b = wid / ((int64_t)S * H);
  const int64_t base = b * sb + h * sh;
  float qv[MAXE], acc[MAXE];
#pragma unroll
  for (int e = 0; e < MAXE; ++e) {
    const int d = lane + 32 * e;
    qv[e] = d < D ? Elem<T>::ld(q + base + i * ss + d) : 0.0f;
    acc[e] = 0.0f;
  }
  const float scale = rsqrtf((float)D);
  float m = -INFINITY, l = 0.0f;
  const int last = causal ? i : S - 1;
  for (int j = 0; j <= last; ++j) {
    float dot = 0.0f;
#pragma unroll
    for (int e = 0; e < MAXE; ++e) {
      const int d = lane + 32 * e;
      if (d < D) dot = fmaf(qv[e], Elem<T>::ld(k + base + j * ss + d), dot);
    }
    const float sc = warp_sum(dot) * scale;
    const float mn = fmaxf(m, sc);
    const float alpha = expf(m - mn), pj = expf(sc - mn);
    l = l * alpha + pj;
#pragma unroll
    for (int e = 0; e < MAXE; ++e) {
      const int d = lane + 32 * e;
      if (d < D) acc[e] = acc[e] * alpha + pj * Elem<T>::ld(v + base + j * ss + d);
    }
    m = mn;
  }
  const float inv = 1.0f / l;
  T* orow = o + ((b * S + i) * H + h) * D;
#pragma unroll
  for (int e = 0; e < MAXE; ++e) {
    const int d = lane + 32 * e;
    if (d < D) Elem<T>::st(orow + d, acc[e] * inv);
  }
}

cudaError_t launch_attention_simt(int dtype, const AttnView& a, void* o, cudaStream_t s) {
  const int64_t warps = a.B * a.H * a.S;
  if (warps == 0) return cudaSuccess;
  const unsigned grid = (unsigned)((warps + 3) / 4);
  if (dtype == DT_F32)
    attention_simt_kernel<float><<<grid, 128, 0, s>>>((const float*)a.q, (const float*)a.k, (const float*)a.v, (float*)o, a.sb, a.sh, a.ss, a.B,
                                                      (int)a.H, (int)a.S, (int)a.D, a.causal ? 1 : 0);
  else
    attention_simt_kernel<__nv_bfloat16><<<grid, 128, 0, s>>>((const __nv_bfloat16*)a.q, (const __nv_bfloat16*)a.k, (const __nv_bfloat16*)a.v,
                                                              (__nv_bfloat16*)o, a.sb, a.sh, a.ss, a.B, (int)a.H, (int)a.S, (int)a.D,
                                                              a.causal ? 1 : 0);
  return cudaGetLastError();
}

}  // namespace mk
