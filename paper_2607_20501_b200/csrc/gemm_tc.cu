// K1: bf16 GEMM with fused elementwise tail on the 5th-generation tensor cores.
//
//   D[M, N] = tail(A[M, K] @ W[K, N])        A row-major (K-major), W stored [N, K] (K-major)
//
// One persistent CTA per SM, 6 warps:
//   warp 0        TMA producer: A tile 128x64 and W tile 256x64 per stage, 128-byte swizzle,
//                 4-stage mbarrier ring (192 KB of shared memory)
//   warp 1        allocates TMEM (512 columns = two 128x256 fp32 accumulators) and issues
//                 tcgen05.mma 128x256x16, four per stage; tcgen05.commit frees the stage and,
//                 after the last K block, publishes the accumulator
//   warps 2..5    epilogue: tcgen05.ld 32 lanes x 32 columns, the elementwise program in fp32
//                 registers, bf16 pack, 16-byte global stores; runs on accumulator t while the
//                 tensor cores fill accumulator t+1
// SwiGLU mode: the 256 accumulator columns are 128 gate columns and the matching 128 up columns
// (two TMA boxes of W), and the tile's output is silu(gate) * up, 128 columns wide.
//
// Every mbarrier wait is bounded; see tc_common.cuh.
#include "device_common.cuh"
#include "tc_common.cuh"
#include "tc_plans.h"
#include "tc_epilogue.cuh"

namespace mk {

namespace {

constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4, UMMA_K = 16;
constexpr int A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int GEMM_THREADS = 192;
constexpr int GROUP_M = 16;
constexpr size_t GEMM_SMEM = (size_t)STAGES * STAGE_BYTES + 1024 /*alignment*/ + 256 /*barriers*/;

struct Shared {
  uint64_t full[STAGES];
  uint64_t empty[STAGES];
  uint64_t tfull[2];
  uint64_t tempty[2];
  uint32_t tmem_base;
  int abort_flag;
};

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
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, __nv_bfloat16* __restrict__ out, int M,
               int N, int K, int up_row_offset, const __grid_constant__ EpiProgram epi, unsigned int* status) {
  constexpr int OUT_N = SWIGLU ? BN / 2 : BN;  // output columns per tile
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  Shared* sh = reinterpret_cast<Shared*>(tiles + (size_t)STAGES * STAGE_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_m = (M + BM - 1) / BM, num_n = (N + OUT_N - 1) / OUT_N;
  const int total_tiles = num_m * num_n;
  const int num_kb = (K + BK - 1) / BK;
  volatile int* abort_flag = &sh->abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&sh->full[s], 1); tc::mbar_init(&sh->empty[s], 1); }
    for (int b = 0; b < 2; ++b) { tc::mbar_init(&sh->tfull[b], 1); tc::mbar_init(&sh->tempty[b], 4); }
    sh->abort_flag = 0;
    tc::fence_barrier_init();
    tc::tma_prefetch_desc(&tmA);
    tc::tma_prefetch_desc(&tmB);
  }
  if (warp == 1) {
    tc::tmem_alloc(&sh->tmem_base, 512);
    tc::tmem_relinquish();
  }
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
      int mi, ni;
      tile_coords(t, num_m, num_n, mi, ni);
      for (int kb = 0; kb < num_kb && ok; ++kb) {
        if (lane == 0) {
          ok = tc::mbar_wait(&sh->empty[stage], phase ^ 1, abort_flag, status, tc::WAIT_SMEM_EMPTY);
          if (ok) {
            uint8_t* a_dst = tiles + (size_t)stage * STAGE_BYTES;
            uint8_t* b_dst = a_dst + A_BYTES;
            tc::mbar_expect_tx(&sh->full[stage], STAGE_BYTES);
            tc::tma_load_2d(a_dst, &tmA, &sh->full[stage], kb * BK, mi * BM);
            const int n0 = ni * OUT_N;
            tc::tma_load_2d(b_dst, &tmB, &sh->full[stage], kb * BK, n0);
            tc::tma_load_2d(b_dst + B_BYTES / 2, &tmB, &sh->full[stage], kb * BK, SWIGLU ? up_row_offset + n0 : n0 + BN / 2);
          }
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (++stage == STAGES) { stage = 0; phase ^= 1; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    constexpr uint32_t idesc = tc::idesc_bf16_f32(BM, BN, 0, 0);
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    int it = 0;
    for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++it) {
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
              tc::umma_ss(d_tmem, adesc + (uint64_t)(k * UMMA_K * 2 / 16), bdesc + (uint64_t)(k * UMMA_K * 2 / 16), idesc,
                          (kb > 0 || k > 0) ? 1u : 0u);
            tc::umma_commit(&sh->empty[stage]);
            if (kb == num_kb - 1) tc::umma_commit(&sh->tfull[acc]);
          }
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (++stage == STAGES) { stage = 0; phase ^= 1; }
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue
    const int q = warp & 3;  // TMEM lane quarter this warp may read
    bool ok = true;
    int it = 0;
    for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++it) {
      int mi, ni;
      tile_coords(t, num_m, num_n, mi, ni);
      const int acc = it & 1;
      const uint32_t acc_phase = (it >> 1) & 1;
      ok = tc::mbar_wait(&sh->tfull[acc], acc_phase, abort_flag, status, tc::WAIT_TMEM_FULL);
      ok = __all_sync(0xffffffffu, ok ? 1 : 0) != 0;
      if (!ok) break;
      tc::tc_fence_after();
      const int64_t row = (int64_t)mi * BM + q * 32 + lane;
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN;
      __nv_bfloat16* orow = out + row * N;
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
        const int64_t col0 = (int64_t)ni * OUT_N + c * 32;
        if (row < M && col0 < N) {
          if (col0 + 32 <= N) {
            epi32(epi, v, row, col0, N);
#pragma unroll
            for (int j = 0; j < 32; j += 8) {
              uint4 pk;
              pk.x = pack_bf16x2(v[j], v[j + 1]);
              pk.y = pack_bf16x2(v[j + 2], v[j + 3]);
              pk.z = pack_bf16x2(v[j + 4], v[j + 5]);
              pk.w = pack_bf16x2(v[j + 6], v[j + 7]);
              *reinterpret_cast<uint4*>(orow + col0 + j) = pk;
            }
          } else {
            for (int j = 0; j < 32 && col0 + j < N; ++j) orow[col0 + j] = __float2bfloat16_rn(epi_apply(epi, v[j], row, col0 + j, N));
          }
        }
      }
      tc::tc_fence_before();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&sh->tempty[acc]);
    }
  }

  // common exit: on an aborted run give copies in flight time to land before the CTA retires
  if (*abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 4000000LL) {}
  }
  tc::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc::tc_fence_after();
    tc::tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace

cudaError_t gemm_tc_plan(GemmTcPlan* p, const void* a, const void* w_nk, void* y, int64_t m, int64_t n, int64_t k, bool swiglu,
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
  const int64_t tiles = ((m + BM - 1) / BM) * ((n + out_n - 1) / out_n);
  p->grid = (int)(tiles < sm_count ? tiles : sm_count);
  return cudaSuccess;
}

cudaError_t launch_gemm_tc(const GemmTcPlan& p, cudaStream_t s) {
  static bool attr_done = false;
  if (!attr_done) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GEMM_SMEM);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gemm_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GEMM_SMEM);
    if (e != cudaSuccess) return e;
    attr_done = true;
  }
  unsigned int* status = kernel_status_ptr();
  if (p.swiglu)
    gemm_tc_kernel<true><<<p.grid, GEMM_THREADS, GEMM_SMEM, s>>>(p.tm_a, p.tm_b, (__nv_bfloat16*)p.out, p.m, p.n, p.k, p.n, p.epi, status);
  else
    gemm_tc_kernel<false><<<p.grid, GEMM_THREADS, GEMM_SMEM, s>>>(p.tm_a, p.tm_b, (__nv_bfloat16*)p.out, p.m, p.n, p.k, 0, p.epi, status);
  return cudaGetLastError();
}

}  // namespace mk
