// LINEAR_FP8: block-scaled fp8 (e4m3) GEMM on tcgen05, the contraction of the paper's FP8 MoE inference task
// (appendix "LLM Inference Kernel Results").
//
//   y[m, n] = tail( sum_kb sx[m, kb] * sw[n / 128, kb] * sum_{k in block kb} xq[m, k] * wq[k, n] )      blocks of 128 along K
//
// The scale changes from one K block to the next, so it cannot be applied after the sum: the tensor core
// accumulates ONE K block (four kind::f8f6f4 MMAs of K = 32, fp32 in tensor memory), and the epilogue warps
// drain that partial tile, multiply it by the block's two scales and add it into fp32 accumulators in registers
// while the tensor core works on the next block in another tensor-memory buffer (four buffers of 128 columns).
// Two-SM form: a CTA pair computes a 256 x 128 tile with tcgen05.mma.cta_group::2; each CTA stages its own 128
// rows of xq and 64 of the tile's 128 weight rows per 128-byte-swizzled stage (TMA, no multicast).  One tile
// column is exactly one 128-wide weight scale block.  The activation scales of the CTA's rows for every K block
// are copied to shared memory a tile ahead (cp.async), so the drain never waits for global memory.
// A plain-ALU kernel serves the shapes this one declines and is the second implementation Swap can bind.
// Measured (4096 x 7168 x 4096): 186 us, 1.29 PFLOP/s; with two commits per K block (one more for the operand
// stage) 200 us, and then the tensor pipe was busy 27 % of the time and L2 at a quarter of its throughput: the
// kernel is bound by the hand-shake per K block (barrier waits and a commit per four MMAs on the issuing thread,
// a tensor-memory round trip and a barrier arrival per drain), not by the drain's own work (sixteen epilogue
// warps with a 32 x 32 chunk each: 218 us) and not by operand traffic.
#include <stdlib.h>

#include "device_common.cuh"
#include "tc_common.cuh"
#include "tc_epilogue.cuh"
#include "tc_plans.h"

namespace mk {
namespace {

constexpr int BM = 128, BN = 128, BK = 128, UMMA_K = 32;
constexpr int EPI_WARPS = 8;
constexpr int THREADS = 64 + 32 * EPI_WARPS;
constexpr int STAGES = 5;
constexpr int A_BYTES = BM * BK, B_BYTES = (BN / 2) * BK, STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int ACC_BUFS = 4;                 // tensor-memory buffers of BN columns
constexpr int KB_MAX = 64;                  // K <= 8192
constexpr int SCALE_BYTES = 2 * (KB_MAX * BM + KB_MAX) * 4;   // two buffers of sx[kb][row] and sw[kb]

struct SharedF8 {
  uint64_t full[STAGES];
  uint64_t empty[STAGES];
  uint64_t tfull[ACC_BUFS];
  uint64_t tempty[ACC_BUFS];
  uint32_t tmem_base;
  int abort_flag;
  EpiProgram epi;
};
constexpr size_t SMEM_F8 = (size_t)STAGES * STAGE_BYTES + EPI_WARPS * EPI_WARP_BYTES + SCALE_BYTES + 1024 + 512;
static_assert(sizeof(SharedF8) <= 512, "barrier block");
static_assert(SMEM_F8 <= 227 * 1024, "shared memory of one SM");

__device__ __forceinline__ void cp_async4(uint32_t smem_dst, const void* gsrc) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_dst), "l"(gsrc) : "memory");
}

__global__ void __launch_bounds__(THREADS, 1)
gemm_fp8_tc2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmOut,
                    void* __restrict__ out, const float* __restrict__ sx, const float* __restrict__ sw, int M, int N, int K,
                    const __grid_constant__ EpiProgram epi_param, unsigned int* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* staging = tiles + (size_t)STAGES * STAGE_BYTES;
  float* scales = reinterpret_cast<float*>(staging + EPI_WARPS * EPI_WARP_BYTES);      // [2][KB_MAX * BM + KB_MAX]
  SharedF8* sh = reinterpret_cast<SharedF8*>(reinterpret_cast<uint8_t*>(scales) + SCALE_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = tc::cluster_ctarank();
  const bool leader = rank == 0;
  const int unit_id = blockIdx.x >> 1, num_units = gridDim.x >> 1;
  const int num_m = (M + 2 * BM - 1) / (2 * BM), num_n = (N + BN - 1) / BN;
  const int total_tiles = num_m * num_n;
  const int num_kb = K / BK;
  volatile int* abort_flag = &sh->abort_flag;
  // tiles walked column by column inside groups of 16 tile rows (their xq rows and the weight slabs stay in L2)
  auto tile_coords = [&](int t, int& mi, int& ni) {
    constexpr int G = 16;
    const int per_group = G * num_n, g = t / per_group, first_m = g * G, gsz = min(num_m - first_m, G), r = t - g * per_group;
    mi = first_m + r % gsz;
    ni = r / gsz;
  };

  epi_copy_to_smem(&sh->epi, epi_param, threadIdx.x, THREADS);
  const EpiProgram& epi = sh->epi;
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&sh->full[s], 1); tc::mbar_init(&sh->empty[s], 1); }
    for (int b = 0; b < ACC_BUFS; ++b) { tc::mbar_init(&sh->tfull[b], 1); tc::mbar_init(&sh->tempty[b], EPI_WARPS * 2); }
    sh->abort_flag = 0;
    tc::fence_barrier_init();
    tc::tma_prefetch_desc(&tmA);
    tc::tma_prefetch_desc(&tmB);
    tc::tma_prefetch_desc(&tmOut);
  }
  if (warp == 1) tc::tmem_alloc_pair(&sh->tmem_base, 512);
  tc::tc_fence_before();
  __syncthreads();
  tc::cluster_sync();
  tc::tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;
  pdl_launch_dependents();
  pdl_wait();

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      const uint32_t full_base = tc::smem_u32(&sh->full[0]);
      for (int t = unit_id; t < total_tiles && ok; t += num_units) {
        int mi, ni;
        tile_coords(t, mi, ni);
        const int m0 = (mi * 2 + (int)rank) * BM, n0 = ni * BN;
        for (int kb = 0; kb < num_kb; ++kb) {
          ok = tc::mbar_wait(&sh->empty[stage], phase ^ 1, abort_flag, status, tc::WAIT_SMEM_EMPTY);
          if (!ok) break;
          uint8_t* a_dst = tiles + (size_t)stage * STAGE_BYTES;
          const uint32_t full_leader = tc::map_to_cta(full_base + (uint32_t)stage * 8u, 0);
          tc::tma_load_2d_pair(a_dst, &tmA, full_leader, kb * BK, m0);
          if (leader) tc::mbar_expect_tx(&sh->full[stage], 2 * STAGE_BYTES);
          tc::tma_load_2d_pair(a_dst + A_BYTES, &tmB, full_leader, kb * BK, n0 + (int)rank * (BN / 2));
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer: one tensor-memory buffer per K block
    if (leader && lane == 0) {
      constexpr uint32_t idesc = tc::idesc_e4m3_f32(2 * BM, BN);
      const uint32_t a_lo0 = tc::desc_lo_sw128(tc::smem_u32(tiles));
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      uint32_t cnt = 0;   // K blocks issued so far: buffer = cnt % ACC_BUFS, the buffer's use count = cnt / ACC_BUFS
      for (int t = unit_id; t < total_tiles && ok; t += num_units) {
        for (int kb = 0; kb < num_kb; ++kb, ++cnt) {
          const uint32_t b = cnt % ACC_BUFS;
          ok = tc::mbar_wait(&sh->tempty[b], ((cnt / ACC_BUFS) & 1) ^ 1, abort_flag, status, tc::WAIT_TMEM_EMPTY);
          if (!ok) break;
          ok = tc::mbar_wait(&sh->full[stage], phase, abort_flag, status, tc::WAIT_SMEM_FULL);
          if (!ok) break;
          tc::tc_fence_after();
          const uint32_t d_tmem = tmem_base + b * BN;
          const uint32_t a_lo = a_lo0 + (uint32_t)stage * (STAGE_BYTES >> 4);
          const uint32_t b_lo = a_lo + (A_BYTES >> 4);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) tc::umma_fp8_pair_lohi(d_tmem, a_lo + 2 * k, b_lo + 2 * k, idesc, k > 0 ? 1u : 0u);
          // ONE commit per K block: its completion says both "the buffer is full" and "the stage has been read";
          // the stage is handed back to the producer by an epilogue warp that has seen it (a commit costs the
          // issuing thread about as long as two of the four MMAs it follows)
          tc::umma_commit_pair(&sh->tfull[b]);
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ epilogue: drain, scale, accumulate; then tail and store
    const int q = warp & 3;                 // tensor-memory lane quarter: tile rows [32 q, 32 q + 32)
    const int half = (warp - 2) >> 2;       // columns [64 half, 64 half + 64) of the tile
    const int et = (int)threadIdx.x - 64;   // 0 .. 255
    EpiWarp ew;
    ew.init(staging + (warp - 2) * EPI_WARP_BYTES, epi, lane, false);
    bool ok = true;
    uint32_t cnt = 0;
    int it = 0;
    const int scale_floats = KB_MAX * BM + KB_MAX;
    // scales of tile t into buffer `buf`: sx[kb][row] for this CTA's 128 rows (thread et: row et % 128, every
    // second K block) and sw[kb] of the tile's weight block column
    auto fetch_scales = [&](int t, int buf) {
      if (t < total_tiles) {
        int mi, ni;
        tile_coords(t, mi, ni);
        float* dst = scales + buf * scale_floats;
        const int row = et & (BM - 1);
        const int64_t grow = (int64_t)(mi * 2 + (int)rank) * BM + row;
        if (grow < M)
          for (int kb = et >> 7; kb < num_kb; kb += 2) cp_async4(tc::smem_u32(dst + kb * BM + row), sx + grow * num_kb + kb);
        if (et < num_kb) cp_async4(tc::smem_u32(dst + KB_MAX * BM + et), sw + (int64_t)ni * num_kb + et);
      }
      tc::cp_async_commit();
    };
    const uint32_t tempty_leader = tc::map_to_cta(tc::smem_u32(&sh->tempty[0]), 0);
    fetch_scales(unit_id, 0);
    for (int t = unit_id; t < total_tiles && ok; t += num_units, ++it) {
      int mi, ni;
      tile_coords(t, mi, ni);
      const int buf = it & 1;
      // this tile's scales have landed (every epilogue thread's copies), the next tile's are requested
      tc::cp_async_wait<0>();
      asm volatile("bar.sync 1, %0;" ::"n"(32 * EPI_WARPS) : "memory");
      fetch_scales(t + num_units, buf ^ 1);
      const float* sxs = scales + buf * scale_floats + q * 32 + lane;     // + kb * BM
      const float* sws = scales + buf * scale_floats + KB_MAX * BM;
      float acc[2][32];
#pragma unroll
      for (int c = 0; c < 2; ++c)
#pragma unroll
        for (int j = 0; j < 32; ++j) acc[c][j] = 0.0f;
      for (int kb = 0; kb < num_kb; ++kb, ++cnt) {
        const uint32_t b = cnt % ACC_BUFS;
        const float f = sxs[kb * BM] * sws[kb];
        ok = tc::mbar_wait_spin(&sh->tfull[b], (cnt / ACC_BUFS) & 1, abort_flag, status, tc::WAIT_TMEM_FULL);
        ok = __all_sync(0xffffffffu, ok ? 1 : 0) != 0;
        if (!ok) break;
        tc::tc_fence_after();
        // the MMAs of this K block are complete, so its operand stage has been read: this CTA's producer may refill it
        if (warp == 2 && lane == 0) tc::mbar_arrive(&sh->empty[cnt % STAGES]);
        const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + b * BN + half * 64;
        {
          // both chunks in flight at once: a tensor-memory load takes several hundred cycles beside running MMAs
          uint32_t r0[32], r1[32];
          tc::tmem_ld32(t_row, r0);
          tc::tmem_ld32(t_row + 32, r1);
          tc::tmem_ld_wait();
          // the buffer is free as soon as its values are in registers
          tc::tc_fence_before();
          __syncwarp();
          // (a relaxed arrival: nothing written to memory has to be published, see tc_common.cuh; with the release form
          // at cluster scope this kernel took 381 us instead of 200 on the 4096 x 7168 x 4096 problem)
          if (lane == 0) tc::mbar_arrive_cluster_relaxed(tempty_leader + b * 8u);
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            acc[0][j] = fmaf(__uint_as_float(r0[j]), f, acc[0][j]);
            acc[1][j] = fmaf(__uint_as_float(r1[j]), f, acc[1][j]);
          }
        }
      }
      if (!ok) break;
      // tail program, bf16, store
      const int64_t row0 = (int64_t)(mi * 2 + (int)rank) * BM + q * 32;
      auto rowmap = [&](int rr) -> int64_t { const int64_t g = row0 + rr; return g < M ? g : -1; };
      const int64_t col_base = (int64_t)ni * BN;
      uint4 res_regs[8];
      ew.load_bias(epi, col_base, BN, N);
      ew.prefetch_res(epi, rowmap, col_base + half * 64, N, res_regs);
      ew.chunk_out(epi, acc[0], rowmap, out, col_base + half * 64, half * 64, (int64_t)N, res_regs, col_base + half * 64 + 32, &tmOut, row0);
      ew.chunk_out(epi, acc[1], rowmap, out, col_base + half * 64 + 32, half * 64 + 32, (int64_t)N, res_regs, -1, &tmOut, row0);
    }
    tc::cp_async_wait<0>();
    if (lane == 0) tc::tma_store_wait_all();
  }

  if (*abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 4000000LL) {}
  }
  tc::tc_fence_before();
  __syncthreads();
  tc::cluster_sync();
  if (warp == 1) {
    tc::tc_fence_after();
    tc::tmem_dealloc_pair(tmem_base, 512);
  }
}

// ---- plain-ALU form: one thread per output element, the definition written out ---------------------------------
__device__ __forceinline__ float e4m3_to_float(uint8_t b) {
  const uint32_t sign = (uint32_t)(b & 0x80) << 24, e = (b >> 3) & 0xF, mt = b & 7;
  float v;
  if (e == 0) v = (float)mt * 0.001953125f;                         // subnormal: mt * 2^-9
  else if (e == 15 && mt == 7) v = __int_as_float(0x7fc00000);      // the one NaN pattern per sign
  else v = __uint_as_float(((e + 120u) << 23) | (mt << 20));        // (1 + mt / 8) * 2^(e - 7)
  return __uint_as_float(__float_as_uint(v) | sign);
}

__global__ void __launch_bounds__(256) gemm_fp8_simt_kernel(const uint8_t* __restrict__ xq, const float* __restrict__ sx,
                                                            const uint8_t* __restrict__ wq, int w_transposed, const float* __restrict__ sw,
                                                            __nv_bfloat16* __restrict__ y, int M, int N, int K,
                                                            const __grid_constant__ EpiProgram p) {
  const int n = blockIdx.x * 32 + (threadIdx.x & 31);
  const int m = blockIdx.y * 8 + (threadIdx.x >> 5);
  if (m >= M || n >= N) return;
  const int num_kb = K / 128;
  float acc = 0.0f;
  for (int kb = 0; kb < num_kb; ++kb) {
    float part = 0.0f;
    for (int k = kb * 128; k < kb * 128 + 128; ++k) {
      const uint8_t wb = w_transposed ? wq[(int64_t)n * K + k] : wq[(int64_t)k * N + n];
      part = fmaf(e4m3_to_float(xq[(int64_t)m * K + k]), e4m3_to_float(wb), part);
    }
    acc = fmaf(part, sx[(int64_t)m * num_kb + kb] * sw[(int64_t)(n / 128) * num_kb + kb], acc);
  }
  y[(int64_t)m * N + n] = __float2bfloat16_rn(epi_apply(p, acc, m, n, N));
}

}  // namespace

bool gemm_fp8_tc2_supported(int64_t m, int64_t n, int64_t k) {
  return m >= 1 && m <= INT32_MAX && n >= 8 && n <= INT32_MAX && n % 8 == 0 && k >= 128 && k % 128 == 0 && k / 128 <= KB_MAX;
}

cudaError_t gemm_fp8_tc2_plan(GemmFp8Plan* p, const void* xq, const float* sx, const void* wq_nk, const float* sw, void* y, int64_t m,
                              int64_t n, int64_t k, const EpiProgram& epi, int sm_count) {
  if (!gemm_fp8_tc2_supported(m, n, k) || !sx || !sw) return cudaErrorInvalidValue;
  cudaError_t e = encode_tmap_2d_u8(&p->tm_a, xq, (uint64_t)m, (uint64_t)k, (uint64_t)k, BM);
  if (e != cudaSuccess) return e;
  e = encode_tmap_2d_u8(&p->tm_b, wq_nk, (uint64_t)n, (uint64_t)k, (uint64_t)k, BN / 2);
  if (e != cudaSuccess) return e;
  e = encode_tmap_2d_bf16_store(&p->tm_out, y, (uint64_t)m, (uint64_t)n, (uint64_t)n);
  if (e != cudaSuccess) return e;
  p->sx = sx; p->sw = sw; p->out = y;
  p->m = (int)m; p->n = (int)n; p->k = (int)k;
  p->epi = epi;
  const int64_t tiles = ((m + 2 * BM - 1) / (2 * BM)) * ((n + BN - 1) / BN);
  const int64_t units = tiles < sm_count / 2 ? tiles : sm_count / 2;
  p->grid = (int)(2 * units);
  return cudaSuccess;
}

cudaError_t launch_gemm_fp8_tc2(const GemmFp8Plan& p, cudaStream_t s) {
  static SmemOptIn opt_in;
  cudaError_t e = opt_in.ensure(SMEM_F8, gemm_fp8_tc2_kernel);
  if (e != cudaSuccess) return e;
  LaunchCfg lc(PDL_GEMM, dim3((unsigned)p.grid), dim3(THREADS), SMEM_F8, s, 2);
  return cudaLaunchKernelEx(&lc.cfg, gemm_fp8_tc2_kernel, p.tm_a, p.tm_b, p.tm_out, p.out, p.sx, p.sw, p.m, p.n, p.k, p.epi, kernel_status_ptr());
}

cudaError_t launch_gemm_fp8_simt(const void* xq, const float* sx, const void* wq, bool w_transposed, const float* sw, void* y, int64_t m,
                                 int64_t n, int64_t k, const EpiProgram& p, cudaStream_t s) {
  if (m < 1 || n < 1 || k < 128 || k % 128 || m > INT32_MAX || n > INT32_MAX || k > INT32_MAX) return cudaErrorInvalidValue;
  dim3 grid((unsigned)((n + 31) / 32), (unsigned)((m + 7) / 8));
  if (grid.y > 65535) return cudaErrorInvalidValue;
  gemm_fp8_simt_kernel<<<grid, 256, 0, s>>>((const uint8_t*)xq, sx, (const uint8_t*)wq, w_transposed ? 1 : 0, sw, (__nv_bfloat16*)y, (int)m, (int)n,
                                            (int)k, p);
  return cudaGetLastError();
}

}  // namespace mk
