// K1, two-SM form: bf16 GEMM with fused elementwise tail, one 256x256 output tile per CTA PAIR.
//
//   D[M, N] = tail(A[M, K] @ W[K, N])        A row-major (K-major), W stored [N, K] (K-major)
//
// A cluster of two CTAs (two SMs) shares one tcgen05.mma.cta_group::2 of shape 256x256x16: each CTA
// stages its own 128 rows of A and its own 128 of the 256 W rows, so every byte of W is fetched and
// held once per pair and each SM reads half as much B from shared memory per MMA as the one-SM form
// does.  No TMA multicast is used: each CTA issues plain tile loads for its own halves, and both
// CTAs' loads complete on the leader CTA's "full" barrier.
//
// Per CTA, 6 warps:
//   warp 0        TMA producer: A tile 128x64 + W tile 128x64 per stage (32 KB), 128-byte swizzle,
//                 6-stage ring; waits on its own "empty" barrier, which the leader's
//                 tcgen05.commit signals in both CTAs
//   warp 1        allocates TMEM (512 columns, both CTAs); in the leader CTA one lane issues the MMAs,
//                 commits the stage back to both producers and, after the last K block, publishes the
//                 accumulator to both epilogues
//   warps 2..5    epilogue of this CTA's 128 rows: tcgen05.ld, elementwise program, bf16 stores; the
//                 accumulator is double-buffered so it overlaps the next tile's MMAs; when done each
//                 warp arrives on the leader's "tmem empty" barrier
// SwiGLU mode: the leader's W half holds 128 gate rows, the peer's the matching 128 up rows.
// Every mbarrier wait is bounded (tc_common.cuh); both CTAs leave through a cluster barrier.
#include "device_common.cuh"
#include "tc_common.cuh"
#include "tc_epilogue.cuh"
#include "tc_plans.h"

namespace mk {

namespace {

constexpr int BM = 128;        // rows per CTA (256 per pair)
constexpr int BN = 256;        // accumulator columns
constexpr int BK = 64, UMMA_K = 16;
constexpr int STAGES = 6;
constexpr int A_BYTES = BM * BK * 2, B_BYTES = (BN / 2) * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int THREADS = 192;
constexpr int GROUP_M = 8;     // in 256-row tiles
constexpr size_t SMEM_BYTES = (size_t)STAGES * STAGE_BYTES + 1024 + 256;

struct Shared {
  uint64_t full[STAGES];
  uint64_t empty[STAGES];
  uint64_t tfull[2];
  uint64_t tempty[2];
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// tile load into this CTA's shared memory, completion bytes go to the barrier at cluster address `bar`
__device__ __forceinline__ void tma_load_2d_pair(void* dst, const CUtensorMap* m, uint32_t bar_cluster_addr, int32_t x, int32_t y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(
          tc::smem_u32(dst)),
      "l"(reinterpret_cast<uint64_t>(m)), "r"(bar_cluster_addr), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void umma_ss_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// one arrival on the barrier at this offset in BOTH CTAs once all MMAs issued so far have finished
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(tc::smem_u32(bar)),
               "h"((uint16_t)3)
               : "memory");
}

__device__ __forceinline__ void tile_coords(int t, int num_m, int num_n, int& mi, int& ni) {
  const int per_group = GROUP_M * num_n;
  const int g = t / per_group;
  const int first_m = g * GROUP_M;
  const int gsz = min(num_m - first_m, GROUP_M);
  const int r = t - g * per_group;
  mi = first_m + r % gsz;
  ni = r / gsz;
}

template <bool SWIGLU>
__global__ void __launch_bounds__(THREADS, 1)
gemm_tc2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, __nv_bfloat16* __restrict__ out, int M,
                int N, int K, int up_row_offset, const __grid_constant__ EpiProgram epi, unsigned int* status) {
  constexpr int OUT_N = SWIGLU ? BN / 2 : BN;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  Shared* sh = reinterpret_cast<Shared*>(tiles + (size_t)STAGES * STAGE_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const int cluster_id = blockIdx.x >> 1, num_clusters = gridDim.x >> 1;
  const int num_m = (M + 2 * BM - 1) / (2 * BM), num_n = (N + OUT_N - 1) / OUT_N;
  const int total_tiles = num_m * num_n;
  const int num_kb = (K + BK - 1) / BK;
  volatile int* abort_flag = &sh->abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&sh->full[s], 1); tc::mbar_init(&sh->empty[s], 1); }
    for (int b = 0; b < 2; ++b) { tc::mbar_init(&sh->tfull[b], 1); tc::mbar_init(&sh->tempty[b], 8); }
    sh->abort_flag = 0;
    tc::fence_barrier_init();
    tc::tma_prefetch_desc(&tmA);
    tc::tma_prefetch_desc(&tmB);
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc::smem_u32(&sh->tmem_base)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc::tc_fence_before();
  __syncthreads();
  cluster_sync();  // both CTAs' barriers are initialised before anything remote touches them
  tc::tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (both CTAs)
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int t = cluster_id; t < total_tiles && ok; t += num_clusters) {
      int mi, ni;
      tile_coords(t, num_m, num_n, mi, ni);
      const int m0 = (mi * 2 + (int)rank) * BM;
      const int n0 = ni * OUT_N;
      const int b_row = SWIGLU ? (leader ? n0 : up_row_offset + n0) : n0 + (int)rank * (BN / 2);
      for (int kb = 0; kb < num_kb && ok; ++kb) {
        if (lane == 0) {
          ok = tc::mbar_wait(&sh->empty[stage], phase ^ 1, abort_flag, status, tc::WAIT_SMEM_EMPTY);
          if (ok) {
            uint8_t* a_dst = tiles + (size_t)stage * STAGE_BYTES;
            const uint32_t full_leader = map_to_cta(tc::smem_u32(&sh->full[stage]), 0);
            if (leader) tc::mbar_expect_tx(&sh->full[stage], 2 * STAGE_BYTES);
            tma_load_2d_pair(a_dst, &tmA, full_leader, kb * BK, m0);
            tma_load_2d_pair(a_dst + A_BYTES, &tmB, full_leader, kb * BK, b_row);
          }
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (++stage == STAGES) { stage = 0; phase ^= 1; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader CTA only)
    if (leader) {
      constexpr uint32_t idesc = tc::idesc_bf16_f32(2 * BM, BN, 0, 0);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int it = 0;
      for (int t = cluster_id; t < total_tiles && ok; t += num_clusters, ++it) {
        const int acc = it & 1;
        const uint32_t acc_phase = (it >> 1) & 1;
        const uint32_t d_tmem = tmem_base + acc * BN;
        if (lane == 0) {
          ok = tc::mbar_wait(&sh->tempty[acc], acc_phase ^ 1, abort_flag, status, tc::WAIT_TMEM_EMPTY);
          tc::tc_fence_after();
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        for (int kb = 0; kb < num_kb && ok; ++kb) {
          if (lane == 0) {
            ok = tc::mbar_wait(&sh->full[stage], phase, abort_flag, status, tc::WAIT_SMEM_FULL);
            if (ok) {
              tc::tc_fence_after();
              const uint32_t a_addr = tc::smem_u32(tiles + (size_t)stage * STAGE_BYTES);
              const uint64_t adesc = tc::smem_desc_sw128(a_addr, 16, 1024);
              const uint64_t bdesc = tc::smem_desc_sw128(a_addr + A_BYTES, 16, 1024);
#pragma unroll
              for (int k = 0; k < BK / UMMA_K; ++k)
                umma_ss_pair(d_tmem, adesc + (uint64_t)(k * UMMA_K * 2 / 16), bdesc + (uint64_t)(k * UMMA_K * 2 / 16), idesc,
                             (kb > 0 || k > 0) ? 1u : 0u);
              umma_commit_pair(&sh->empty[stage]);
              if (kb == num_kb - 1) umma_commit_pair(&sh->tfull[acc]);
            }
          }
          ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (both CTAs, own 128 rows)
    const int q = warp & 3;
    bool ok = true;
    int it = 0;
    for (int t = cluster_id; t < total_tiles && ok; t += num_clusters, ++it) {
      int mi, ni;
      tile_coords(t, num_m, num_n, mi, ni);
      const int acc = it & 1;
      const uint32_t acc_phase = (it >> 1) & 1;
      ok = tc::mbar_wait(&sh->tfull[acc], acc_phase, abort_flag, status, tc::WAIT_TMEM_FULL);
      ok = __all_sync(0xffffffffu, ok ? 1 : 0) != 0;
      if (!ok) break;
      tc::tc_fence_after();
      const int64_t row = (int64_t)(mi * 2 + (int)rank) * BM + q * 32 + lane;
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN;
#pragma unroll 1
      for (int c = 0; c < OUT_N / 32; ++c) {
        uint32_t r[32];
        float v[32];
        tc::tmem_ld32(t_row + c * 32, r);
        tc::tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
        if (SWIGLU) {
          tc::tmem_ld32(t_row + BN / 2 + c * 32, r);
          tc::tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = silu_fast(v[j]) * __uint_as_float(r[j]);
        }
        epi_store32(epi, v, out, row, (int64_t)ni * OUT_N + c * 32, M, N);
      }
      tc::tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_cta(tc::smem_u32(&sh->tempty[acc]), 0));
    }
  }

  if (*abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 4000000LL) {}
  }
  tc::tc_fence_before();
  __syncthreads();
  cluster_sync();  // the peer's shared memory and barriers stay alive until both CTAs are done
  if (warp == 1) {
    tc::tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

}  // namespace

cudaError_t gemm_tc2_plan(GemmTcPlan* p, const void* a, const void* w_nk, void* y, int64_t m, int64_t n, int64_t k, bool swiglu,
                          const EpiProgram& epi, int sm_count) {
  if (k % 8 || n % 8 || m < 1 || n < 1 || k < 1) return cudaErrorInvalidValue;
  if (m > INT32_MAX || n > INT32_MAX || k > INT32_MAX) return cudaErrorInvalidValue;
  const int64_t w_rows = swiglu ? 2 * n : n;
  cudaError_t e = encode_tmap_2d_bf16(&p->tm_a, a, (uint64_t)m, (uint64_t)k, (uint64_t)k, BM, BK);
  if (e != cudaSuccess) return e;
  e = encode_tmap_2d_bf16(&p->tm_b, w_nk, (uint64_t)w_rows, (uint64_t)k, (uint64_t)k, BN / 2, BK);
  if (e != cudaSuccess) return e;
  p->out = y;
  p->m = (int)m; p->n = (int)n; p->k = (int)k;
  p->swiglu = swiglu;
  p->epi = epi;
  const int out_n = swiglu ? BN / 2 : BN;
  const int64_t tiles = ((m + 2 * BM - 1) / (2 * BM)) * ((n + out_n - 1) / out_n);
  const int64_t clusters = tiles < sm_count / 2 ? tiles : sm_count / 2;
  p->grid = (int)(2 * clusters);
  return cudaSuccess;
}

cudaError_t launch_gemm_tc2(const GemmTcPlan& p, cudaStream_t s) {
  static bool attr_done = false;
  if (!attr_done) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tc2_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tc2_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attr_done = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)p.grid);
  cfg.blockDim = dim3(THREADS);
  cfg.dynamicSmemBytes = SMEM_BYTES;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  unsigned int* status = kernel_status_ptr();
  __nv_bfloat16* out = (__nv_bfloat16*)p.out;
  if (p.swiglu) return cudaLaunchKernelEx(&cfg, gemm_tc2_kernel<true>, p.tm_a, p.tm_b, out, p.m, p.n, p.k, p.n, p.epi, status);
  return cudaLaunchKernelEx(&cfg, gemm_tc2_kernel<false>, p.tm_a, p.tm_b, out, p.m, p.n, p.k, 0, p.epi, status);
}

}  // namespace mk
