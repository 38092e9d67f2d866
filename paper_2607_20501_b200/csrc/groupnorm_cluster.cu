// GroupNorm over an NHWC tensor with the image resident in the shared memory of a thread-block cluster.
//
// The statistics of one (image, group) span the whole image, which is why the plain form takes two launches
// and reads the tensor twice.  Here the 2, 4 or 8 CTAs of a cluster hold one image between them (a CTA owns a
// contiguous run of pixels, up to ~200 KB): every CTA brings its pixels in with a handful of asynchronous bulk
// copies (global -> shared, one mbarrier per piece, so the whole share is in flight from the first
// instruction), sums each piece as it lands, exchanges one (mean, M2) pair per group with its peers through
// distributed shared memory (st.shared::cluster into every peer's slot, one cluster barrier), merges them in
// rank order with Chan's formula, and normalises its pixels out of shared memory straight into global memory.
// HBM sees the tensor once in each direction; nothing else is read but gamma and beta.
//
// Statistics: sums of differences from a pivot (the CTA's own first pixel, the group's first channel, after the
// elementwise prefix), so a group whose mean is many standard deviations from zero keeps its variance in fp32;
// the partial results leave the CTA as (mean, sum of squared deviations from it), which merge without
// cancellation.  The merge visits the ranks in the same order in every CTA: the result is the same in all of
// them and from launch to launch.
//
// Waits: the only spin is on the load barriers, bounded (status word, abort flag) like every other wait of the
// library; a CTA whose wait ran out skips its arithmetic but still takes part in every cluster barrier, so its
// peers are never left waiting for it.
#include <cstdio>
#include "device_common.cuh"
#include "tc_common.cuh"
#include "kernels.h"

namespace mk {
namespace {

#ifndef MK_GC_THREADS
#define MK_GC_THREADS 256
#endif
constexpr int GC_THREADS = MK_GC_THREADS;   // measured: 512 threads 18.4 us, 256 threads 17.9 us on 32 x 56 x 56 x 128
constexpr int GC_MAX_C = 512;            // one thread per (statistic, channel) column in the reduction
constexpr int GC_PIECES = 8;            // bulk copies per CTA
constexpr int GC_MAX_CL = 8;            // CTAs per cluster (the portable maximum)
constexpr size_t GC_SMEM_MAX = 227 * 1024;

struct GcLayout {
  size_t data, red, slot, mr, piv, table, bars, total;   // byte offsets of the regions, and the total
};
// data: this CTA's pixels; red: partial sums [2][gc_red_rows][c]; slot: float2 [cluster][groups];
// mr: float2 [groups] = (mean, 1 / std); piv: float [groups]; table: float [2][c] = scale, shift;
// bars: GC_PIECES mbarriers + flag
// rows of the reduction buffer: the lanes of a warp that hold the same channels (pixel rows of the thread grid inside
// one warp) are summed by shuffles first, so a warp leaves one row when a pixel takes at most a warp's width
__host__ __device__ inline int gc_red_rows(int c, int ve) {
  const int vpp = c / ve;
  return vpp <= 32 ? GC_THREADS / 32 : GC_THREADS / vpp;
}
__host__ __device__ inline GcLayout gc_layout(int64_t pix_max, int c, int groups, int esz, int ve, int cl) {
  GcLayout l;
  l.data = 0;
  size_t o = ((size_t)pix_max * c * esz + 127) & ~(size_t)127;
  l.red = o; o += (size_t)2 * gc_red_rows(c, ve) * c * 4;
  l.slot = o; o += (size_t)cl * groups * 8;
  l.mr = o; o += (size_t)groups * 8;
  l.piv = o; o += (size_t)groups * 4;
  l.table = o; o += (size_t)2 * c * 4;
  o = (o + 15) & ~(size_t)15;
  l.bars = o; o += GC_PIECES * 8 + 16;
  l.total = o + 128;   // slack for aligning the dynamic region's base
  return l;
}

__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(tc::smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(tc::smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void st_cluster_f32x2_(uint32_t cluster_addr, float a, float b) {
  asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(cluster_addr), "f"(a), "f"(b) : "memory");
}

#ifdef MK_TRACE_GC
__device__ __forceinline__ unsigned long long gc_gtime() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
#define GCT(i) do { if (threadIdx.x == 0 && blockIdx.x == 0 && blockIdx.y == 0) gct[i] = gc_gtime(); } while (0)
#else
#define GCT(i) do {} while (0)
#endif

template <typename T>
__global__ void __launch_bounds__(GC_THREADS, 1)
groupnorm_cluster_kernel(const T* __restrict__ x, T* __restrict__ y, int64_t hw, int c, int groups, const T* __restrict__ gamma,
                         const T* __restrict__ beta, float eps, const __grid_constant__ EpiProgram pre, unsigned int* status) {
  constexpr int VE = Elem<T>::VEC;
#ifdef MK_TRACE_GC
  unsigned long long gct[32] = {};
#endif
  GCT(0);
  extern __shared__ uint8_t gc_smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(gc_smem_raw) + 127) & ~(uintptr_t)127);
  const int cl = (int)gridDim.x;                       // the cluster spans the grid's x dimension
  const uint32_t rank = tc::cluster_ctarank();
  const int64_t img = blockIdx.y;
  const int64_t pix_max = (hw + cl - 1) / cl;
  const GcLayout L = gc_layout(pix_max, c, groups, (int)sizeof(T), VE, cl);
  T* data = reinterpret_cast<T*>(base + L.data);
  float* red_s = reinterpret_cast<float*>(base + L.red);
  const int red_rows = gc_red_rows(c, VE);
  float* red_q = red_s + red_rows * c;
  float2* slot = reinterpret_cast<float2*>(base + L.slot);
  float2* mr = reinterpret_cast<float2*>(base + L.mr);
  float* pivg = reinterpret_cast<float*>(base + L.piv);
  float* scale = reinterpret_cast<float*>(base + L.table);
  float* shift = scale + c;
  uint64_t* bars = reinterpret_cast<uint64_t*>(base + L.bars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + GC_PIECES);

  const int64_t p0 = hw * (int64_t)rank / cl, p1 = hw * ((int64_t)rank + 1) / cl;
  const int npix = (int)(p1 - p0);
  const int cg = c / groups;
  const int vpp = c / VE;
  const int vcol = threadIdx.x % vpp, prow = threadIdx.x / vpp, pstride = GC_THREADS / vpp;
  auto piece_lo = [&](int k) { return (int)((int64_t)npix * k / GC_PIECES); };

  if (threadIdx.x == 0) {
    for (int k = 0; k < GC_PIECES; ++k) tc::mbar_init(&bars[k], 1);
    *abort_flag = 0;
    tc::fence_barrier_init();
  }
  __syncthreads();
  tc::cluster_arrive_relaxed();        // "this CTA runs": waited for before the first store into a peer's shared memory
  pdl_launch_dependents();
  pdl_wait();                  // x may come from the kernel before this one
  const T* xin = x + (img * hw + p0) * c;
  T* yout = y + (img * hw + p0) * c;
  // gamma and beta of this thread's table entries, asked for now: they are not needed before the statistics are
  float ga_pf[(GC_MAX_C + GC_THREADS - 1) / GC_THREADS], be_pf[(GC_MAX_C + GC_THREADS - 1) / GC_THREADS];
#pragma unroll
  for (int i = 0; i < (GC_MAX_C + GC_THREADS - 1) / GC_THREADS; ++i) {
    const int ch = threadIdx.x + i * GC_THREADS;
    ga_pf[i] = (gamma && ch < c) ? Elem<T>::ld(gamma + ch) : 1.0f;
    be_pf[i] = (beta && ch < c) ? Elem<T>::ld(beta + ch) : 0.0f;
  }
  GCT(1);
  // The whole share is asked for at once: GC_PIECES bulk copies, a barrier each, so the sums below start on the
  // first piece while the rest is in flight.  (Measured against it: the last three pieces fetched by the threads'
  // own 16-byte loads at the same time, eight in flight each, 22.9 us against 18.8 us.)
  if (threadIdx.x == 0) {
    for (int k = 0; k < GC_PIECES; ++k) {
      const int a = piece_lo(k), b = piece_lo(k + 1);
      if (b > a) {
        const uint32_t bytes = (uint32_t)(b - a) * (uint32_t)c * (uint32_t)sizeof(T);
        tc::mbar_expect_tx(&bars[k], bytes);
        bulk_g2s(data + (int64_t)a * c, xin + (int64_t)a * c, bytes, &bars[k]);
      }
    }
  }

  // ---------------------------------------------------------------- sums about the pivot, piece by piece
  float s[VE], q[VE], piv[VE];
#pragma unroll
  for (int e = 0; e < VE; ++e) { s[e] = 0.0f; q[e] = 0.0f; piv[e] = 0.0f; }
  bool ok = true;
  for (int k = 0; k < GC_PIECES && ok; ++k) {
    const int a = piece_lo(k), b = piece_lo(k + 1);
    if (b <= a) continue;               // uniform over the CTA
    // the same answer in every thread: what follows has CTA-wide barriers in it
    ok = __syncthreads_and(tc::mbar_wait(&bars[k], 0, abort_flag, status, tc::WAIT_SMEM_FULL) ? 1 : 0) != 0;
    if (!ok) break;
    GCT(2 + k);
    if (a == 0) {
      // the pivots: the CTA's first pixel, the first channel of each group, after the elementwise prefix; taken
      // before the prefix is written back over the pixels
      for (int g = threadIdx.x; g < groups; g += GC_THREADS) pivg[g] = epi_apply(pre, Elem<T>::ld(data + g * cg), img * hw + p0, g * cg, c);
      __syncthreads();
#pragma unroll
      for (int e = 0; e < VE; ++e) piv[e] = pivg[(vcol * VE + e) / cg];
    }
    for (int pix = a + prow; pix < b; pix += pstride) {
      float v[VE];
      T* src = data + (int64_t)pix * c + vcol * VE;
      ld_vec(src, v);
      if (pre.n > 0) {
        epi_apply_vec<T, VE>(pre, v, img * hw + p0 + pix, (int64_t)vcol * VE, c);
        st_vec(src, v);                 // the normalisation pass reads what the prefix left (rounded to T, as it would be in memory)
        ld_vec(src, v);
      }
#pragma unroll
      for (int e = 0; e < VE; ++e) { const float d = v[e] - piv[e]; s[e] += d; q[e] = fmaf(d, d, q[e]); }
    }
  }
  // Per-channel totals through the reduction buffer: column j < c is the sum of channel j over the thread grid's
  // pixel rows, column c + j that of its squares.  They land in the table region, free until the statistics are known.
  if (vpp < 32) {
    // 32 / vpp pixel rows of the thread grid sit in one warp (vpp divides 32: it divides the block size, a power of two)
    for (int off = vpp; off < 32; off <<= 1) {
#pragma unroll
      for (int e = 0; e < VE; ++e) {
        s[e] += __shfl_xor_sync(0xffffffffu, s[e], off);
        q[e] += __shfl_xor_sync(0xffffffffu, q[e], off);
      }
    }
  }
  {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int rrow = vpp <= 32 ? warp : prow;
    if (vpp > 32 || lane < vpp) {
#pragma unroll
      for (int e = 0; e < VE; ++e) {
        red_s[rrow * c + vcol * VE + e] = s[e];
        red_q[rrow * c + vcol * VE + e] = q[e];
      }
    }
  }
  __syncthreads();
  for (int col = threadIdx.x; col < 2 * c; col += GC_THREADS) {
    const float* src = col < c ? red_s + col : red_q + (col - c);
    float acc = 0.0f;
    for (int row = 0; row < red_rows; ++row) acc += src[row * c];
    scale[col] = acc;             // scale[0, c): sums; shift[0, c) = scale[c, 2c): sums of squares
  }
  __syncthreads();
  GCT(10);
  ok = *abort_flag == 0;
  tc::cluster_wait();          // every CTA of the cluster is running: its shared memory may be written
  if (ok) {
    for (int g = threadIdx.x; g < groups; g += GC_THREADS) {
      float ts = 0.0f, tq = 0.0f;
      for (int ch = g * cg; ch < (g + 1) * cg; ++ch) { ts += scale[ch]; tq += shift[ch]; }
      const float n_r = (float)npix * (float)cg;
      const float pv = pivg[g];
      const float md = npix > 0 ? ts / n_r : 0.0f;
      const float mean_r = pv + md;
      const float m2_r = fmaxf(tq - ts * md, 0.0f);
      const uint32_t local = tc::smem_u32(&slot[rank * groups + g]);
      for (int peer = 0; peer < cl; ++peer) st_cluster_f32x2_(tc::map_to_cta(local, (uint32_t)peer), mean_r, m2_r);
    }
  }
  GCT(11);
  tc::cluster_sync();          // the peers' partial results are in this CTA's slots
  GCT(12);
  if (ok) {
    for (int g = threadIdx.x; g < groups; g += GC_THREADS) {
      // Chan's pairwise update, ranks in order
      float n = 0.0f, mean = 0.0f, m2 = 0.0f;
      for (int r = 0; r < cl; ++r) {
        const float n_r = (float)(hw * ((int64_t)r + 1) / cl - hw * (int64_t)r / cl) * (float)cg;
        if (n_r <= 0.0f) continue;
        const float2 pr = slot[r * groups + g];
        const float nn = n + n_r, delta = pr.x - mean;
        mean += delta * (n_r / nn);
        m2 += pr.y + delta * delta * (n * n_r / nn);
        n = nn;
      }
      mr[g] = make_float2(mean, rsqrtf(m2 / n + eps));
    }
  }
  __syncthreads();
  if (ok) {
#pragma unroll
    for (int i = 0; i < (GC_MAX_C + GC_THREADS - 1) / GC_THREADS; ++i) {
      const int ch = threadIdx.x + i * GC_THREADS;
      if (ch < c) {
        const float2 st = mr[ch / cg];
        scale[ch] = st.y * ga_pf[i];
        shift[ch] = be_pf[i] - st.x * st.y * ga_pf[i];
      }
    }
  }
  __syncthreads();

  // ---------------------------------------------------------------- normalise out of shared memory, store
  // Four pixels per thread and step, 16-byte stores straight to global memory.  (Measured against it: normalising in
  // place and sending each piece out with a bulk copy shared -> global, 19.4 us against 18.8 us.)
  if (ok) {
    float sc[VE], sf[VE];
#pragma unroll
    for (int e = 0; e < VE; ++e) { sc[e] = scale[vcol * VE + e]; sf[e] = shift[vcol * VE + e]; }
    for (int pix = prow; pix < npix; pix += 4 * pstride) {
      uint4 raw[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (pix + u * pstride < npix) raw[u] = *reinterpret_cast<const uint4*>(data + (int64_t)(pix + u * pstride) * c + vcol * VE);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (pix + u * pstride < npix) {
          float v[VE];
          RawVec<T, VE> rv;
          rv.r[0] = raw[u];
          rv.unpack(v);
#pragma unroll
          for (int e = 0; e < VE; ++e) v[e] = fmaf(v[e], sc[e], sf[e]);
          st_vec(yout + (int64_t)(pix + u * pstride) * c + vcol * VE, v);
        }
      }
    }
  }
#ifdef MK_TRACE_GC
  GCT(21);
  if (threadIdx.x == 0 && blockIdx.x == 0 && blockIdx.y == 0) {
    printf("gc:");
    for (int i = 1; i < 24; ++i) printf(" [%d]%llu", i, gct[i] - gct[0]);
    printf("\n");
  }
#endif
  if (!ok) {
    // give a copy in that may still be in flight time to land before the CTA retires
    const long long t0 = clock64();
    while (clock64() - t0 < 4000000LL) {}
  }
  __syncthreads();
}

template <typename T> bool gc_shape_ok(int64_t c) {
  constexpr int VE = Elem<T>::VEC;
  const int64_t vpp = c / VE;
  return c % VE == 0 && vpp >= 1 && vpp <= GC_THREADS && GC_THREADS % vpp == 0 && c <= GC_MAX_C;
}

// the cluster size for this shape: the image must fit; among those that do, the largest that still leaves every
// cluster resident at once (one CTA per SM), else the smallest
int gc_cluster_size(int dtype, int64_t nb, int64_t hw, int64_t c, int groups, int sm_count) {
  const int esz = dtype == DT_F32 ? 4 : 2, ve = dtype == DT_F32 ? 4 : 8;
  int smallest = 0, best = 0;
  for (int cl = 1; cl <= GC_MAX_CL; cl *= 2) {
    if (hw < cl) break;
    const GcLayout l = gc_layout((hw + cl - 1) / cl, (int)c, groups, esz, ve, cl);
    if (l.total > GC_SMEM_MAX) continue;
    if (!smallest) smallest = cl;
    if (nb * cl <= (int64_t)sm_count * 9 / 10) best = cl;   // clusters of 4 / 8 do not pack every SM: leave a margin
  }
  return best ? best : smallest;
}

}  // namespace

bool groupnorm_cluster_supported(int dtype, const void* x, const void* y, int64_t nb, int64_t hw, int64_t c, int groups, int sm_count) {
  if (nb < 1 || nb > 65535 || hw < 1 || groups < 1 || c % groups || c > 4096) return false;
  if (((uintptr_t)x & 15) != 0 || ((uintptr_t)y & 15) != 0) return false;
  if (!(dtype == DT_F32 ? gc_shape_ok<float>(c) : gc_shape_ok<__nv_bfloat16>(c))) return false;
  return gc_cluster_size(dtype, nb, hw, c, groups, sm_count) > 0;
}

template <typename T>
static cudaError_t gc_launch(const void* x, void* y, int64_t nb, int64_t hw, int64_t c, int groups, const void* gamma, const void* beta,
                             float eps, const EpiProgram& pre, int cl, cudaStream_t s) {
  static SmemOptIn opt_in;
  const GcLayout l = gc_layout((hw + cl - 1) / cl, (int)c, groups, (int)sizeof(T), Elem<T>::VEC, cl);
  cudaError_t e = opt_in.ensure(GC_SMEM_MAX, groupnorm_cluster_kernel<T>);
  if (e != cudaSuccess) return e;
  LaunchCfg lc(PDL_GROUPNORM, dim3((unsigned)cl, (unsigned)nb), dim3(GC_THREADS), l.total, s, cl);
  return cudaLaunchKernelEx(&lc.cfg, groupnorm_cluster_kernel<T>, (const T*)x, (T*)y, hw, (int)c, groups, (const T*)gamma, (const T*)beta, eps,
                            pre, kernel_status_ptr());
}

cudaError_t launch_groupnorm_cluster(int dtype, const void* x, void* y, int64_t nb, int64_t hw, int64_t c, int groups, const void* gamma,
                                     const void* beta, float eps, const EpiProgram& pre, int sm_count, cudaStream_t s) {
  if (!groupnorm_cluster_supported(dtype, x, y, nb, hw, c, groups, sm_count)) return cudaErrorInvalidValue;
  const int cl = gc_cluster_size(dtype, nb, hw, c, groups, sm_count);
  return dtype == DT_F32 ? gc_launch<float>(x, y, nb, hw, c, groups, gamma, beta, eps, pre, cl, s)
                         : gc_launch<__nv_bfloat16>(x, y, nb, hw, c, groups, gamma, beta, eps, pre, cl, s);
}

}  // namespace mk
