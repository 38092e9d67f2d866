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
// (mean, M2) of its slice of each row into all eight CTAs' slots, one cluster barrier).  The merged variance is what
// the single-CTA form's two passes give.
// =====================================================================================================
constexpr int LC_CL = 8;         // CTAs per cluster
constexpr int LC_RB = 8;         // rows per cluster
#ifndef MK_LC_THREADS
#define MK_LC_THREADS 512
#endif
constexpr int LC_THREADS = MK_LC_THREADS;   // the threads beyond the CTA's outputs split K: more of them, shorter dot products
constexpr int LC_MAXNC = 32;     // columns per CTA: N <= LC_CL * LC_MAXNC

__device__ __forceinline__ void st_cluster_f32(uint32_t cluster_addr, float v) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(cluster_addr), "f"(v) : "memory");
}

// The end of both cluster forms: thread (r, j) holds output v of row m0 + r, column c0 + j (has: that output exists;
// in_outs: the thread is one of the CTA's LC_RB * NC output threads).  Called by every thread of the CTA.
template <typename T>
__device__ __forceinline__ void lc_norm_tail(float v, bool has, bool in_outs, int r, int j, int nc, int NC, int N, int M, int m0, int c0,
                                             uint32_t rank, int mode, float eps, float ga, float be, float (&slot)[2][LC_CL][LC_RB],
                                             T* __restrict__ y) {
  if (mode != ROW_LAYERNORM && mode != ROW_RMSNORM) {   // the chain without its norm (a tiny GEMM + elementwise tail)
    if (has && m0 + r < M) Elem<T>::st(y + (int64_t)(m0 + r) * N + c0 + j, v);
    return;
  }
  // One exchange for both statistics.  LayerNorm: every CTA sends, per row, the mean of its columns and their squared
  // deviations from that mean; the receiver merges the eight (count, mean, M2) triples, M2 = sum of M2_c + n_c *
  // (mean_c - mean)^2, which is what a second pass about the global mean would have summed, so no second round is
  // needed.  RMSNorm: the squares about zero.  A row's NC values sit in NC adjacent lanes (NC is a power of two <= 32).
  if (__any_sync(0xffffffffu, in_outs)) {
    float mc = 0.0f, q;
    if (mode == ROW_LAYERNORM) {
      float sm = v;
      for (int o = NC >> 1; o; o >>= 1) sm += __shfl_xor_sync(0xffffffffu, sm, o);
      mc = nc > 0 ? sm / (float)nc : 0.0f;
      const float d = has ? v - mc : 0.0f;
      q = d * d;
    } else {
      q = v * v;
    }
    for (int o = NC >> 1; o; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
    if (in_outs) {
      const uint32_t l0 = tc::smem_u32(&slot[0][rank][r]), l1 = tc::smem_u32(&slot[1][rank][r]);
      for (uint32_t c = (uint32_t)j; c < LC_CL; c += (uint32_t)NC) {   // the row's lanes share the eight destinations
        st_cluster_f32(tc::map_to_cta(l0, c), mc);
        st_cluster_f32(tc::map_to_cta(l1, c), q);
      }
    }
  }
  tc::cluster_sync();
  if (has && m0 + r < M) {
    float mean = 0.0f, m2 = 0.0f;
    const float inv_n = 1.0f / (float)N;
    if (mode == ROW_LAYERNORM) {
      for (int c = 0; c < LC_CL; ++c) mean += (float)max(0, min(NC, N - c * NC)) * slot[0][c][r];   // the same order everywhere
      mean *= inv_n;
      for (int c = 0; c < LC_CL; ++c) {
        const float d = slot[0][c][r] - mean;
        m2 += slot[1][c][r] + (float)max(0, min(NC, N - c * NC)) * d * d;
      }
    } else {
      for (int c = 0; c < LC_CL; ++c) m2 += slot[1][c][r];
    }
    const float o = (v - mean) * rsqrtf(m2 * inv_n + eps) * ga + be;
    Elem<T>::st(y + (int64_t)(m0 + r) * N + c0 + j, o);
  }
}

template <typename T>
__global__ void __launch_bounds__(LC_THREADS) linear_rownorm_cluster_kernel(const T* __restrict__ a, const T* __restrict__ w, bool wt,
                                                                            T* __restrict__ y, int M, int N, int K, int NC,
                                                                            const __grid_constant__ EpiProgram p, int mode,
                                                                            const T* __restrict__ gamma, const T* __restrict__ beta,
                                                                            float eps) {
  extern __shared__ float smem[];
  // row pitches of K + 4 floats: rows stay 16-byte aligned for the vector reads of the dot products, and the rows (of X)
  // or columns (of W) that a quarter warp reads together start four banks apart
  const int KP = K + 4;
  const int XP = K + 4;
  float* xs = smem;                                        // [LC_RB][XP]
  float* ws = xs + LC_RB * XP;                             // [NC][KP]: this CTA's columns of W, K contiguous
  float* part = ws + NC * KP;                              // [KS][LC_RB * NC]
  __shared__ float slot[2][LC_CL][LC_RB];                  // every CTA's (mean, M2) of its slice of each row
#ifdef MK_TRACE_C1
  long long tr_[8]; tr_[0] = clock64();
#define C1T(i) tr_[i] = clock64()
#else
#define C1T(i) do {} while (0)
#endif
  pdl_launch_dependents();
  // A CTA may write into a peer's shared memory only once that peer is running: every CTA announces itself
  // here and waits for the others just before its first remote store, so the rendezvous costs nothing.
  tc::cluster_arrive_relaxed();
  pdl_wait();
  const uint32_t rank = tc::cluster_ctarank();
  const int m0 = (int)(blockIdx.x / LC_CL) * LC_RB, c0 = (int)rank * NC;
  const int nc = min(NC, N - c0) > 0 ? min(NC, N - c0) : 0;   // columns of this CTA that exist
  // Everything that is read late - the norm's scale and shift, the first bias vector of the elementwise tail - is
  // asked for now: a dependent global load at the end of this kernel would be a tenth of its whole duration.
  float ga = 1.0f, be = 0.0f, bias_v = 0.0f;
  int bias_i = -1;
  {
    const int rj = threadIdx.x, j = rj % NC;
    if (rj < LC_RB * NC && j < nc) {
      if (gamma) ga = Elem<T>::ld(gamma + c0 + j);
      if (mode == ROW_LAYERNORM && beta) be = Elem<T>::ld(beta + c0 + j);
      for (int i = 0; i < p.n && bias_i < 0; ++i)
        if (p.op[i].kind == EPI_BIAS && p.op[i].ptr) bias_i = i;
      if (bias_i >= 0) bias_v = epi_ptr_ld(p.op[bias_i].ptr, p.dtype, c0 + j);
    }
  }
  constexpr int VE = Elem<T>::VEC;
  // how W is read: 1 = 16-byte vectors along K (stored [N, K]), 2 = 16-byte vectors along N (stored [K, N]), 0 = scalars
  const int wmode = wt ? (K % VE == 0 ? 1 : 0) : ((N % VE == 0 && NC % VE == 0 && nc % VE == 0) ? 2 : 0);
  if (K % VE == 0 && wmode != 0) {
    // 16-byte loads; a thread's load of X and its load of W are in flight together: the whole kernel is a few round
    // trips to L2 long
    const int kv = K / VE, nx = LC_RB * kv, nv = nc / VE;
    const int nw = wmode == 1 ? nc * kv : K * nv;
    for (int base = 0; base < max(nx, nw); base += LC_THREADS) {
      const int i = base + threadIdx.x;
      const bool hx = i < nx, hw = i < nw;
      float vx[VE], vw[VE];
      int r = 0, kx = 0, jw = 0, kw = 0;
      if (hx) {
        r = i / kv; kx = (i - r * kv) * VE;
        if (m0 + r < M) {
          ld_vec(a + (int64_t)(m0 + r) * K + kx, vx);
        } else {
#pragma unroll
          for (int e = 0; e < VE; ++e) vx[e] = 0.0f;
        }
      }
      if (hw) {
        if (wmode == 1) { jw = i / kv; kw = (i - jw * kv) * VE; ld_vec(w + (int64_t)(c0 + jw) * K + kw, vw); }
        else { kw = i / nv; jw = (i - kw * nv) * VE; ld_vec(w + (int64_t)kw * N + c0 + jw, vw); }
      }
      if (hx) {
#pragma unroll
        for (int e = 0; e < VE; ++e) xs[r * XP + kx + e] = vx[e];
      }
      if (hw) {
#pragma unroll
        for (int e = 0; e < VE; ++e) {
          if (wmode == 1) ws[jw * KP + kw + e] = vw[e];
          else ws[(jw + e) * KP + kw] = vw[e];
        }
      }
    }
  } else {
    for (int i = threadIdx.x; i < LC_RB * K; i += LC_THREADS) {
      const int r = i / K, k = i - r * K;
      xs[r * XP + k] = (m0 + r < M) ? Elem<T>::ld(a + (int64_t)(m0 + r) * K + k) : 0.0f;
    }
    if (wt) {
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
  }
  __syncthreads();
  C1T(1);
  // outputs r * NC + j; the threads beyond them split K
  const int outs = LC_RB * NC;
  const int KS = LC_THREADS / outs > 0 ? LC_THREADS / outs : 1;
  for (int o = threadIdx.x; o < outs * KS; o += LC_THREADS) {
    const int ks = o / outs, rj = o - ks * outs, r = rj / NC, j = rj - r * NC;
    const int kper = (K + KS - 1) / KS, kb = ks * kper, ke = min(K, kb + kper);
    float acc = 0.0f, acc1 = 0.0f;   // two chains: a dependent FMA every four cycles is half of what the loop can issue
    if (j < nc) {
      const float* xr = xs + r * XP;
      const float* wr = ws + j * KP;
      if (((kb | ke | K) & 3) == 0) {   // K itself too: the row pitches are K + 4
        // 16-byte reads: the dot products are bound by shared-memory wavefronts, and a vector read of X (two distinct
        // rows per warp) costs one wavefront for four k where scalar reads cost four
        for (int k = kb; k < ke; k += 4) {
          const float4 xv = *reinterpret_cast<const float4*>(xr + k), wv = *reinterpret_cast<const float4*>(wr + k);
          acc = fmaf(xv.x, wv.x, acc);
          acc1 = fmaf(xv.y, wv.y, acc1);
          acc = fmaf(xv.z, wv.z, acc);
          acc1 = fmaf(xv.w, wv.w, acc1);
        }
      } else {
        int k = kb;
#pragma unroll 4
        for (; k + 1 < ke; k += 2) {
          acc = fmaf(xr[k], wr[k], acc);
          acc1 = fmaf(xr[k + 1], wr[k + 1], acc1);
        }
        if (k < ke) acc = fmaf(xr[k], wr[k], acc);
      }
    }
    part[ks * outs + rj] = acc + acc1;
  }
  __syncthreads();
  C1T(2);
  // from here on a thread owns one output (outs <= LC_THREADS): row r, column j of this CTA's slice, kept in a register
  const int rj = threadIdx.x, r = rj / NC, j = rj - r * NC;
  const bool has = rj < outs && j < nc;
  float v = 0.0f;
  if (has) {
    for (int q = 0; q < KS; ++q) v += part[q * outs + rj];       // fixed order
    v = epi_apply_pre(p, v, m0 + r, c0 + j, N, bias_i, bias_v);
  }
  C1T(3);
  tc::cluster_wait();   // all eight CTAs of the cluster are resident from here on
  C1T(4);
  lc_norm_tail<T>(v, has, rj < outs, r, j, nc, NC, N, M, m0, c0, rank, mode, eps, ga, be, slot, y);
#ifdef MK_TRACE_C1
  C1T(7);
  if (blockIdx.x == 0 && threadIdx.x == 0) printf("c1 loads %lld fma %lld tail %lld wait %lld stats %lld sync %lld out %lld\n", tr_[1]-tr_[0], tr_[2]-tr_[1], tr_[3]-tr_[2], tr_[4]-tr_[3], tr_[5]-tr_[4], tr_[6]-tr_[5], tr_[7]-tr_[6]);
#endif
  // nobody writes into a peer's shared memory after the cluster barrier: a CTA may retire here
}

// The register form of the same kernel, for the shapes where it applies (K <= LC_KPER * LC_THREADS / NC, K a multiple of
// LC_KPER): nothing is staged in shared memory.  A thread owns one column and LC_KPER consecutive k: it loads its
// LC_KPER weights and the eight rows' LC_KPER activations straight into registers (all loads in flight at once; the
// lanes that share a k slice read the same addresses of X, which the load unit serves as one request), multiplies, and
// leaves eight partial sums in shared memory; an output thread adds its column's slices.  The staged form is bound by
// shared-memory wavefronts in its dot products (two reads per FMA, the read of X a broadcast); this one has none.
constexpr int LC_KPER = 8;

template <typename T>
__global__ void __launch_bounds__(LC_THREADS) linear_rownorm_cluster_reg_kernel(const T* __restrict__ a, const T* __restrict__ w, bool wt,
                                                                                T* __restrict__ y, int M, int N, int K, int NC,
                                                                                const __grid_constant__ EpiProgram p, int mode,
                                                                                const T* __restrict__ gamma, const T* __restrict__ beta,
                                                                                float eps) {
  __shared__ float part[LC_THREADS * LC_RB];               // [k slice][LC_RB][NC]
  __shared__ float slot[2][LC_CL][LC_RB];                  // every CTA's (mean, M2) of its slice of each row
  pdl_launch_dependents();
  tc::cluster_arrive_relaxed();                                    // see the staged form: met again just before the remote stores
  pdl_wait();
  const uint32_t rank = tc::cluster_ctarank();
  const int m0 = (int)(blockIdx.x / LC_CL) * LC_RB, c0 = (int)rank * NC;
  const int nc = min(NC, N - c0) > 0 ? min(NC, N - c0) : 0;
  const int outs = LC_RB * NC;
  const int j = threadIdx.x % NC, sl = threadIdx.x / NC, kb = sl * LC_KPER;
  float ga = 1.0f, be = 0.0f, bias_v = 0.0f;
  int bias_i = -1;
  if (threadIdx.x < outs && j < nc) {
    if (gamma) ga = Elem<T>::ld(gamma + c0 + j);
    if (mode == ROW_LAYERNORM && beta) be = Elem<T>::ld(beta + c0 + j);
    for (int i = 0; i < p.n && bias_i < 0; ++i)
      if (p.op[i].kind == EPI_BIAS && p.op[i].ptr) bias_i = i;
    if (bias_i >= 0) bias_v = epi_ptr_ld(p.op[bias_i].ptr, p.dtype, c0 + j);
  }
  constexpr int VE = Elem<T>::VEC;
  static_assert(LC_KPER % VE == 0, "a thread's k slice is whole 16-byte vectors");
  float acc[LC_RB];
#pragma unroll
  for (int r = 0; r < LC_RB; ++r) acc[r] = 0.0f;
  if (kb < K && j < nc) {
    float wv[LC_KPER], xr[LC_RB][LC_KPER];
    if (wt) {
#pragma unroll
      for (int e0 = 0; e0 < LC_KPER; e0 += VE) {
        float t[VE];
        ld_vec(w + (int64_t)(c0 + j) * K + kb + e0, t);
#pragma unroll
        for (int e = 0; e < VE; ++e) wv[e0 + e] = t[e];
      }
    } else {
#pragma unroll
      for (int e = 0; e < LC_KPER; ++e) wv[e] = Elem<T>::ld(w + (int64_t)(kb + e) * N + c0 + j);
    }
#pragma unroll
    for (int r = 0; r < LC_RB; ++r) {
#pragma unroll
      for (int e0 = 0; e0 < LC_KPER; e0 += VE) {
        float t[VE];
        if (m0 + r < M) {
          ld_vec(a + (int64_t)(m0 + r) * K + kb + e0, t);
        } else {
#pragma unroll
          for (int e = 0; e < VE; ++e) t[e] = 0.0f;
        }
#pragma unroll
        for (int e = 0; e < VE; ++e) xr[r][e0 + e] = t[e];
      }
    }
#pragma unroll
    for (int e = 0; e < LC_KPER; ++e) {
#pragma unroll
      for (int r = 0; r < LC_RB; ++r) acc[r] = fmaf(xr[r][e], wv[e], acc[r]);
    }
  }
#pragma unroll
  for (int r = 0; r < LC_RB; ++r) part[(sl * LC_RB + r) * NC + j] = acc[r];
  __syncthreads();
  const int rj = threadIdx.x, r = rj / NC;
  const bool has = rj < outs && j < nc;
  float v = 0.0f;
  if (has) {
    const int ns = K / LC_KPER;
    for (int q = 0; q < ns; ++q) v += part[(q * LC_RB + r) * NC + j];   // fixed order
    v = epi_apply_pre(p, v, m0 + r, c0 + j, N, bias_i, bias_v);
  }
  tc::cluster_wait();   // all eight CTAs of the cluster are resident from here on
  lc_norm_tail<T>(v, has, rj < outs, r, j, nc, NC, N, M, m0, c0, rank, mode, eps, ga, be, slot, y);
}

template <typename T>
static cudaError_t linear_rownorm_cluster_launch(const void* a, const void* w, bool wt, void* y, int64_t m, int64_t n, int64_t k,
                                                 const EpiProgram& p, int mode, const void* g, const void* b, float eps, cudaStream_t s) {
  int NC = (int)((n + LC_CL - 1) / LC_CL);
  // a power of two keeps LC_RB * NC a divisor of the CTA size, so the idle threads split K evenly
  int pw = 1;
  while (pw < NC) pw *= 2;
  NC = pw;
  const unsigned grid = (unsigned)((m + LC_RB - 1) / LC_RB) * LC_CL;
  if (k % LC_KPER == 0 && k <= (int64_t)LC_KPER * (LC_THREADS / NC) && (!wt || k % Elem<T>::VEC == 0)) {
    LaunchCfg lc(PDL_ELTWISE, dim3(grid), dim3(LC_THREADS), 0, s, LC_CL);
    return cudaLaunchKernelEx(&lc.cfg, linear_rownorm_cluster_reg_kernel<T>, (const T*)a, (const T*)w, wt, (T*)y, (int)m, (int)n, (int)k, NC, p,
                              mode, (const T*)g, (const T*)b, eps);
  }
  const int outs = LC_RB * NC, KS = LC_THREADS / outs > 0 ? LC_THREADS / outs : 1;
  const size_t smem = sizeof(float) * ((size_t)LC_RB * (k + 4) + (size_t)NC * (k + 4) + (size_t)KS * outs);
  static SmemOptIn opt_in;   // one per instantiation (T)
  if (smem > 48 * 1024) {
    cudaError_t e = opt_in.ensure(smem, linear_rownorm_cluster_kernel<T>);
    if (e != cudaSuccess) return e;
  }
  LaunchCfg lc(PDL_ELTWISE, dim3(grid), dim3(LC_THREADS), smem, s, LC_CL);
  return cudaLaunchKernelEx(&lc.cfg, linear_rownorm_cluster_kernel<T>, (const T*)a, (const T*)w, wt, (T*)y, (int)m, (int)n, (int)k, NC, p, mode,
                            (const T*)g, (const T*)b, eps);
}
// what the cluster form takes: a row norm with two statistics at most, few columns, operands that fit
static bool linear_rownorm_cluster_ok(int64_t m, int64_t n, int64_t k, int mode) {
  if (mode != ROW_LAYERNORM && mode != ROW_RMSNORM && mode != -1) return false;   // -1: no norm, the column split alone
  if (n > LC_CL * LC_MAXNC || n < LC_CL || k > 2048 || m > (1 << 20)) return false;
  return sizeof(float) * ((size_t)(LC_RB + LC_MAXNC) * (k + 4) + LC_THREADS) <= 160 * 1024;
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
