// GEMM + elementwise tail + LayerNorm / RMSNorm over the whole output row in ONE tensor-core kernel that
// writes the normalised row once: the paper's projection + residual + norm fusion (its listings fuse the
// output projection, the residual add and the LayerNorm into one subkernel) at tensor-core shape.
//
// A thread-block cluster of P CTA pairs (2P CTAs, P in {1, 2, 4}) owns a block of 256 rows; pair p computes the
// 256 x 256 tiles of its columns with tcgen05.mma.cta_group::2 exactly as the plain two-SM GEMM does (TMA ring,
// accumulators in TMEM), one tile per row block (N <= 256 P, accumulators double-buffered so that the epilogue of
// one row block overlaps the MMAs of the next) or two (N <= 512 P, all of TMEM taken by one row block).
// The rows stay in TMEM until their statistics are known:
//   pass 1   an epilogue warp reads its accumulator chunks, applies the elementwise tail (bias, residual, ...),
//            writes the result back to TMEM - and to global memory too when the value before the norm is needed
//            later (a residual stream) - and sums it;
//   pass 2   (LayerNorm) squares about the warp's own mean, again out of TMEM;
//   exchange every warp leaves (mean, M2) or the sum of squares of its 32 rows in the shared memory of the P CTAs
//            that hold the other columns of those rows (st.shared::cluster), fences, and arrives on their barrier;
//   pass 3   after the barrier each lane combines the 2P partials of its own row (Chan's formula: no
//            cancellation between a large mean and a small variance), normalises straight out of TMEM and the
//            block leaves by a bulk tensor store.
// Nothing un-normalised is written and read back: against GEMM + row kernel this saves one write and one read of
// the activation and a launch.  No TMA multicast: every CTA loads its own operands.
#include <stdlib.h>

#include "device_common.cuh"
#include "tc_common.cuh"
#include "tc_epilogue.cuh"
#include "tc_plans.h"

namespace mk {
namespace {

constexpr int BM = 128, BN = 256, BK = 64, UMMA_K = 16;
constexpr int EPI_WARPS = 8;
constexpr int THREADS = 64 + 32 * EPI_WARPS;
constexpr int STAGES = 5;
constexpr int A_BYTES = BM * BK * 2, B_BYTES = (BN / 2) * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int MAX_PAIRS = 4, MAX_NT = 2;
constexpr int COLVEC_BYTES = 2 * MAX_NT * BN * 4;                  // gamma and beta of this pair's columns, fp32
constexpr int PART_BYTES = 2 * MAX_PAIRS * 2 * BM * 8;             // [buffer][source pair][column half][row] float2

struct SharedCl {
  uint64_t full[STAGES];
  uint64_t empty[STAGES];
  uint64_t tfull[2];
  uint64_t tempty[2];
  uint64_t stat_bar[2];
  uint32_t tmem_base;
  int abort_flag;
  EpiProgram epi;
};
constexpr size_t SMEM_CL = (size_t)STAGES * STAGE_BYTES + EPI_WARPS * EPI_WARP_BYTES + COLVEC_BYTES + PART_BYTES + 1024 + 512;
static_assert(sizeof(SharedCl) <= 512, "barrier block");
static_assert(SMEM_CL <= 227 * 1024, "shared memory of one SM");

// valid columns among the chunks half, half + 2, ... of the NT tiles of pair `pi`
__device__ __forceinline__ int warp_cols(int pi, int half, int NT, int N) {
  int n = 0;
  for (int j = 0; j < NT; ++j)
    for (int c = half; c < BN / 32; c += 2) {
      const int c0 = (pi * NT + j) * BN + c * 32;
      n += min(max(N - c0, 0), 32);
    }
  return n;
}

__global__ void __launch_bounds__(THREADS, 1)
gemm_rownorm_cl_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmOut,
                       __nv_bfloat16* __restrict__ out, void* __restrict__ mid_out, int mid_f32, int M, int N, int K, int P, int NT,
                       const __grid_constant__ EpiProgram epi_param, const __nv_bfloat16* __restrict__ gamma,
                       const __nv_bfloat16* __restrict__ beta, float eps, int mode, unsigned int* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* staging = tiles + (size_t)STAGES * STAGE_BYTES;
  float* gvec = reinterpret_cast<float*>(staging + EPI_WARPS * EPI_WARP_BYTES);   // [NT * 256]
  float* bvec = gvec + MAX_NT * BN;
  float2* part = reinterpret_cast<float2*>(reinterpret_cast<uint8_t*>(gvec) + COLVEC_BYTES);
  SharedCl* sh = reinterpret_cast<SharedCl*>(reinterpret_cast<uint8_t*>(part) + PART_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t crank = tc::cluster_ctarank();
  const uint32_t r = crank & 1u, leader_rank = crank & ~1u;
  const int pi = (int)(crank >> 1);
  const bool leader = r == 0;
  const int csize = 2 * P;
  const int cluster_id = blockIdx.x / csize, num_clusters = gridDim.x / csize;
  const int num_rb = (M + 2 * BM - 1) / (2 * BM);
  const int num_kb = (K + BK - 1) / BK;
  volatile int* abort_flag = &sh->abort_flag;

  epi_copy_to_smem(&sh->epi, epi_param, threadIdx.x, THREADS);
  const EpiProgram& epi = sh->epi;
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&sh->full[s], 1); tc::mbar_init(&sh->empty[s], 1); }
    for (int b = 0; b < 2; ++b) {
      tc::mbar_init(&sh->tfull[b], 1);
      tc::mbar_init(&sh->tempty[b], EPI_WARPS * 2);
      tc::mbar_init(&sh->stat_bar[b], EPI_WARPS * P);     // every epilogue warp of the P CTAs that share these rows
    }
    sh->abort_flag = 0;
    tc::fence_barrier_init();
    tc::tma_prefetch_desc(&tmA);
    tc::tma_prefetch_desc(&tmB);
    tc::tma_prefetch_desc(&tmOut);
  }
  if (warp == 1) tc::tmem_alloc_pair(&sh->tmem_base, 512);
  // the norm's scale and shift for this pair's columns (parameters: they are not the preceding kernel's output)
  for (int i = threadIdx.x; i < NT * BN; i += THREADS) {
    const int col = pi * NT * BN + i;
    gvec[i] = (gamma && col < N) ? __bfloat162float(gamma[col]) : 1.0f;
    bvec[i] = (beta && mode == ROW_LAYERNORM && col < N) ? __bfloat162float(beta[col]) : 0.0f;
  }
  tc::tc_fence_before();
  __syncthreads();
  tc::cluster_sync();   // every CTA's barriers exist before anything remote touches them
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
      for (int rb = cluster_id; rb < num_rb && ok; rb += num_clusters) {
        const int m0 = (rb * 2 + (int)r) * BM;
        for (int j = 0; j < NT && ok; ++j) {
          const int n0 = (pi * NT + j) * BN;
          for (int kb = 0; kb < num_kb; ++kb) {
            ok = tc::mbar_wait(&sh->empty[stage], phase ^ 1, abort_flag, status, tc::WAIT_SMEM_EMPTY);
            if (!ok) break;
            uint8_t* a_dst = tiles + (size_t)stage * STAGE_BYTES;
            uint8_t* b_dst = a_dst + A_BYTES;
            const uint32_t full_leader = tc::map_to_cta(full_base + (uint32_t)stage * 8u, leader_rank);
            tc::tma_load_2d_pair(a_dst, &tmA, full_leader, kb * BK, m0);
            if (leader) tc::mbar_expect_tx(&sh->full[stage], 2 * STAGE_BYTES);
            tc::tma_load_2d_pair(b_dst, &tmB, full_leader, kb * BK, n0 + (int)r * (BN / 2));
            if (++stage == STAGES) { stage = 0; phase ^= 1; }
          }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (one lane of each pair's leader)
    if (leader && lane == 0) {
      constexpr uint32_t idesc = tc::idesc_bf16_f32(2 * BM, BN, 0, 0);
      const uint32_t a_lo0 = tc::desc_lo_sw128(tc::smem_u32(tiles));
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int use = 0;     // accumulator uses so far: slot = use & 1, the slot's use count = use >> 1
      for (int rb = cluster_id; rb < num_rb && ok; rb += num_clusters) {
        for (int j = 0; j < NT && ok; ++j, ++use) {
          const int slot = use & 1;
          const uint32_t d_tmem = tmem_base + slot * BN;
          ok = tc::mbar_wait(&sh->tempty[slot], ((use >> 1) & 1) ^ 1, abort_flag, status, tc::WAIT_TMEM_EMPTY);
          if (!ok) break;
          tc::tc_fence_after();
          uint32_t accumulate = 0;
          for (int kb = 0; kb < num_kb; ++kb) {
            ok = tc::mbar_wait(&sh->full[stage], phase, abort_flag, status, tc::WAIT_SMEM_FULL);
            if (!ok) break;
            tc::tc_fence_after();
            const uint32_t a_lo = a_lo0 + (uint32_t)stage * (STAGE_BYTES >> 4);
            const uint32_t b_lo = a_lo + (A_BYTES >> 4);
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k) {
              tc::umma_ss_pair_lohi(d_tmem, a_lo + 2 * k, b_lo + 2 * k, idesc, accumulate);
              accumulate = 1;
            }
            tc::umma_commit_pair_at(&sh->empty[stage], leader_rank);
            if (++stage == STAGES) { stage = 0; phase ^= 1; }
          }
          if (!ok) break;
          tc::umma_commit_pair_at(&sh->tfull[slot], leader_rank);
        }
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ epilogue: this CTA's 128 rows of the block
    const int q = warp & 3;
    const int half = (warp - 2) >> 2;
    constexpr int CHUNKS = BN / 32;
    EpiWarp ew;
    ew.init(staging + (warp - 2) * EPI_WARP_BYTES, epi, lane, mid_f32 != 0);
    ew.store = mid_out != nullptr;
    bool ok = true;
    int use = 0, it = 0;
    const float inv_n = 1.0f / (float)N;
    const int n_w = warp_cols(pi, half, NT, N);
    const float inv_nw = n_w > 0 ? 1.0f / (float)n_w : 0.0f;
    const uint32_t part_local = tc::smem_u32(part);
    const uint32_t stat_local = tc::smem_u32(&sh->stat_bar[0]);
    for (int rb = cluster_id; rb < num_rb && ok; rb += num_clusters, ++it) {
      const int64_t row0 = (int64_t)(rb * 2 + (int)r) * BM + q * 32;
      auto rowmap = [&](int rr) -> int64_t { const int64_t g = row0 + rr; return g < M ? g : -1; };
      const int use0 = use;
      // the last bulk store of the row block before has finished reading the staging buffer, which pass 1 reuses
      if (lane == 0) tc::tma_store_wait_read();
      __syncwarp();
      float s1 = 0.0f, s2 = 0.0f;   // this lane's row over the warp's columns: sum, then sum of squares (about the warp's mean for LayerNorm)
      // ---- pass 1: tail, write-back, sums
      for (int j = 0; j < NT && ok; ++j, ++use) {
        const int slot = use & 1;
        const int64_t col_base = (int64_t)(pi * NT + j) * BN;
        uint4 res_regs[8];
        ew.load_bias(epi, col_base, BN, N);
        ew.prefetch_res(epi, rowmap, col_base + half * 32, N, res_regs);
        ok = tc::mbar_wait(&sh->tfull[slot], (use >> 1) & 1, abort_flag, status, tc::WAIT_TMEM_FULL);
        ok = __all_sync(0xffffffffu, ok ? 1 : 0) != 0;
        if (!ok) break;
        tc::tc_fence_after();
        const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + slot * BN;
#pragma unroll 1
        for (int c = half; c < CHUNKS; c += 2) {
          const int64_t c0 = col_base + c * 32;
          if (c0 >= N) break;            // warp-uniform; nothing of this tile is left
          uint32_t rg[32];
          float v[32];
          tc::tmem_ld32(t_row + c * 32, rg);
          tc::tmem_ld_wait();
#pragma unroll
          for (int k = 0; k < 32; ++k) v[k] = __uint_as_float(rg[k]);
          ew.chunk_out(epi, v, rowmap, mid_out, c0, c * 32, (int64_t)N, res_regs, c + 2 < CHUNKS ? col_base + (c + 2) * 32 : -1);
#pragma unroll
          for (int k = 0; k < 32; ++k) {
            if (c0 + k >= N) v[k] = 0.0f;
            rg[k] = __float_as_uint(v[k]);
          }
          tc::tmem_st32(t_row + c * 32, rg);
          if (mode == ROW_LAYERNORM) {
#pragma unroll
            for (int k = 0; k < 32; ++k) s1 += v[k];
          } else {
#pragma unroll
            for (int k = 0; k < 32; ++k) s2 = fmaf(v[k], v[k], s2);
          }
        }
        tc::tmem_st_wait();
      }
      if (!ok) break;
      // ---- pass 2 (LayerNorm): squares about this warp's own mean
      float mean_w = 0.0f;
      if (mode == ROW_LAYERNORM) {
        mean_w = s1 * inv_nw;
        for (int j = 0; j < NT; ++j) {
          const int slot = (use0 + j) & 1;
          const int64_t col_base = (int64_t)(pi * NT + j) * BN;
          const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + slot * BN;
#pragma unroll 1
          for (int c = half; c < CHUNKS; c += 2) {
            const int64_t c0 = col_base + c * 32;
            if (c0 >= N) break;
            uint32_t rg[32];
            tc::tmem_ld32(t_row + c * 32, rg);
            tc::tmem_ld_wait();
#pragma unroll
            for (int k = 0; k < 32; ++k) {
              const float d = __uint_as_float(rg[k]) - mean_w;
              if (c0 + k < N) s2 = fmaf(d, d, s2);
            }
          }
        }
      }
      // ---- exchange: this warp's partial for its 32 rows goes to the P CTAs that hold the rest of those rows
      {
        const int buf = it & 1;
        const uint32_t slot_off = (uint32_t)((((buf * MAX_PAIRS + pi) * 2 + half) * BM + q * 32 + lane) * 8);
        for (int pj = 0; pj < P; ++pj)
          tc::st_cluster_f32x2(tc::map_to_cta(part_local + slot_off, (uint32_t)(2 * pj) + r), mean_w, s2);
        tc::fence_acq_rel_cluster();
        __syncwarp();
        if (lane == 0)
          for (int pj = 0; pj < P; ++pj) tc::mbar_arrive_cluster(tc::map_to_cta(stat_local + (uint32_t)buf * 8u, (uint32_t)(2 * pj) + r));
        ok = tc::mbar_wait_cluster(&sh->stat_bar[buf], (it >> 1) & 1, abort_flag, status, tc::WAIT_ROW_STATS);
        ok = __all_sync(0xffffffffu, ok ? 1 : 0) != 0;
        if (!ok) break;
      }
      // ---- combine the 2P partials of this lane's row
      float mean = 0.0f, rstd;
      {
        const int buf = it & 1;
        const float2* pp = part + (size_t)buf * MAX_PAIRS * 2 * BM + q * 32 + lane;
        if (mode == ROW_LAYERNORM) {
          float sm = 0.0f;
          for (int pj = 0; pj < P; ++pj)
            for (int h = 0; h < 2; ++h) sm += (float)warp_cols(pj, h, NT, N) * pp[(pj * 2 + h) * BM].x;
          mean = sm * inv_n;
          float m2 = 0.0f;
          for (int pj = 0; pj < P; ++pj)
            for (int h = 0; h < 2; ++h) {
              const float2 t = pp[(pj * 2 + h) * BM];
              const float d = t.x - mean;
              m2 += t.y + (float)warp_cols(pj, h, NT, N) * d * d;
            }
          rstd = rsqrtf(m2 * inv_n + eps);
        } else {
          float sq = 0.0f;
          for (int pj = 0; pj < P; ++pj)
            for (int h = 0; h < 2; ++h) sq += pp[(pj * 2 + h) * BM].y;
          rstd = rsqrtf(sq * inv_n + eps);
        }
      }
      // ---- pass 3: normalise out of TMEM, store, hand the accumulator back
      const float nm = -mean * rstd;
      for (int j = 0; j < NT; ++j) {
        const int slot = (use0 + j) & 1;
        const int64_t col_base = (int64_t)(pi * NT + j) * BN;
        const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + slot * BN;
        const int64_t my_row = rowmap(lane);
#pragma unroll 1
        for (int c = half; c < CHUNKS; c += 2) {
          const int64_t c0 = col_base + c * 32;
          if (c0 >= N) break;
          uint32_t rg[32];
          tc::tmem_ld32(t_row + c * 32, rg);
          tc::tmem_ld_wait();
          const float* gv = gvec + j * BN + c * 32;
          const float* bv = bvec + j * BN + c * 32;
          float y[32];
#pragma unroll
          for (int k = 0; k < 32; ++k) {
            const float g = gv[k];
            y[k] = fmaf(fmaf(__uint_as_float(rg[k]), rstd, nm), g, bv[k]);
          }
          if (c0 + 32 <= N) {
            if (lane == 0) tc::tma_store_wait_read();     // the previous block has left the staging buffer
            __syncwarp();
            uint4 mine[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              mine[k].x = pack_bf16x2(y[8 * k + 0], y[8 * k + 1]);
              mine[k].y = pack_bf16x2(y[8 * k + 2], y[8 * k + 3]);
              mine[k].z = pack_bf16x2(y[8 * k + 4], y[8 * k + 5]);
              mine[k].w = pack_bf16x2(y[8 * k + 6], y[8 * k + 7]);
            }
            ew.own_row_to_global_bulk(mine, &tmOut, (int32_t)c0, (int32_t)row0);
          } else if (my_row >= 0) {
#pragma unroll
            for (int k = 0; k < 32; ++k)
              if (c0 + k < N) out[my_row * N + c0 + k] = __float2bfloat16_rn(y[k]);
          }
        }
        tc::tc_fence_before();
        __syncwarp();
        if (lane == 0) tc::mbar_arrive_cluster(tc::map_to_cta(tc::smem_u32(&sh->tempty[slot]), leader_rank));
      }
    }
    if (lane == 0) tc::tma_store_wait_all();
  }

  // common exit: on an aborted run give copies in flight time to land before the CTA retires
  if (*abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 4000000LL) {}
  }
  tc::tc_fence_before();
  __syncthreads();
  tc::cluster_sync();   // peers' shared memory and barriers stay alive until every CTA of the cluster is done
  if (warp == 1) {
    tc::tc_fence_after();
    tc::tmem_dealloc_pair(tmem_base, 512);
  }
}

}  // namespace

bool gemm_rownorm_cl_supported(int64_t m, int64_t n, int64_t k) {
  return m > 128 && m <= INT32_MAX && k >= 8 && k <= INT32_MAX && k % 8 == 0 && n % 8 == 0 && n >= 8 && n <= (int64_t)MAX_PAIRS * MAX_NT * BN;
}

cudaError_t gemm_rownorm_cl_plan(GemmRowNormClPlan* p, const void* a, const void* w_nk, void* y, void* mid_out, bool mid_f32, int64_t m,
                                 int64_t n, int64_t k, const EpiProgram& epi, int mode, const void* gamma, const void* beta, float eps,
                                 int sm_count) {
  if (!gemm_rownorm_cl_supported(m, n, k) || (mode != ROW_LAYERNORM && mode != ROW_RMSNORM)) return cudaErrorInvalidValue;
  cudaError_t e = encode_tmap_2d_bf16(&p->tm_a, a, (uint64_t)m, (uint64_t)k, (uint64_t)k, BM, BK);
  if (e != cudaSuccess) return e;
  e = encode_tmap_2d_bf16(&p->tm_b, w_nk, (uint64_t)n, (uint64_t)k, (uint64_t)k, BN / 2, BK);
  if (e != cudaSuccess) return e;
  e = encode_tmap_2d_bf16_store(&p->tm_out, y, (uint64_t)m, (uint64_t)n, (uint64_t)n);
  if (e != cudaSuccess) return e;
  // fewest pairs (a power of two) whose one or two tiles each cover the row; one tile per pair while that fits a cluster of eight
  const int tiles_n = (int)((n + BN - 1) / BN);
  int P = 1;
  while (P < MAX_PAIRS && P < tiles_n) P *= 2;
  const int NT = (tiles_n + P - 1) / P;
  if (NT > MAX_NT) return cudaErrorInvalidValue;
  p->pairs = P;
  p->nt = NT;
  p->out = y; p->mid_out = mid_out; p->mid_f32 = mid_f32;
  p->m = (int)m; p->n = (int)n; p->k = (int)k;
  p->epi = epi; p->gamma = gamma; p->beta = beta; p->eps = eps; p->mode = mode;
  const int64_t row_blocks = (m + 2 * BM - 1) / (2 * BM);
  int64_t clusters = sm_count / (2 * P);
  const char* ov = getenv("MK_ROWNORM_CLUSTERS");
  if (ov && ov[0]) clusters = atoi(ov);
  if (clusters > row_blocks) clusters = row_blocks;
  if (clusters < 1) clusters = 1;
  p->grid = (int)(clusters * 2 * P);
  return cudaSuccess;
}

cudaError_t launch_gemm_rownorm_cl(const GemmRowNormClPlan& p, cudaStream_t s) {
  static SmemOptIn opt_in;
  cudaError_t e = opt_in.ensure(SMEM_CL, gemm_rownorm_cl_kernel);
  if (e != cudaSuccess) return e;
  LaunchCfg lc(PDL_GEMM, dim3((unsigned)p.grid), dim3(THREADS), SMEM_CL, s, 2 * p.pairs);
  return cudaLaunchKernelEx(&lc.cfg, gemm_rownorm_cl_kernel, p.tm_a, p.tm_b, p.tm_out, (__nv_bfloat16*)p.out, p.mid_out, p.mid_f32 ? 1 : 0, p.m, p.n,
                            p.k, p.pairs, p.nt, p.epi, (const __nv_bfloat16*)p.gamma, (const __nv_bfloat16*)p.beta, p.eps, p.mode,
                            kernel_status_ptr());
}

}  // namespace mk
