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
//            later (a residual stream) - and accumulates, per row, the sum and the sum of squares of the
//            differences from a pivot (the row's first value in this warp's columns: sums about a value of
//            the row itself lose nothing to cancellation when the mean is far from zero);
//   exchange every lane sends (mean, M2) of its row over the warp's columns - for RMSNorm the sum of squares - to
//            the P CTAs that hold the other columns of that row, as asynchronous stores into their shared memory
//            that complete a transaction on their barrier (data and signal travel together);
//   pass 2   after the barrier each lane combines the 2P partials of its own row (Chan's formula), normalises
//            straight out of TMEM and the block leaves by a bulk tensor store.
// A bf16 residual is copied into shared memory (cp.async, all of the tile's chunks for this warp) while the MMAs of
// the row block run, so pass 1 never waits for global memory.
// Nothing un-normalised is written and read back: against GEMM + row kernel this saves one write and one read of
// the activation and a launch.  No TMA multicast: every CTA loads its own operands.
#include <stdlib.h>
#include <cstdio>

#include "device_common.cuh"
#include "tc_common.cuh"
#include "tc_epilogue.cuh"
#include "tc_plans.h"

namespace mk {
namespace {

constexpr int BM = 128, BN = 256, BK = 64, UMMA_K = 16;
constexpr int EPI_WARPS = 8;
constexpr int THREADS = 64 + 32 * EPI_WARPS;
constexpr int STAGES = 4;
constexpr int A_BYTES = BM * BK * 2, B_BYTES = (BN / 2) * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int MAX_PAIRS = 4, MAX_NT = 2;
constexpr int COLVEC_BYTES = 2 * MAX_NT * BN * 4;                  // gamma and beta of this pair's columns, fp32
constexpr int PART_BYTES = 2 * MAX_PAIRS * 2 * BM * 8;             // [buffer][source pair][column half][row] float2
constexpr int RES_SLOT_BYTES = 32 * 64;                           // one 32-row x 32-column bf16 residual chunk
constexpr int RES_EXTRA_SLOTS = 3;                                // per epilogue warp, beside its staging buffer
constexpr int RES_BYTES = EPI_WARPS * RES_EXTRA_SLOTS * RES_SLOT_BYTES;
static_assert(RES_SLOT_BYTES <= EPI_WARP_STAGE, "the staging buffer serves as the first residual slot");

struct SharedCl {
  uint64_t full[STAGES];
  uint64_t empty[STAGES];
  uint64_t tfull[2];
  uint64_t tempty[2];
  uint64_t stat_bar[2];
  uint32_t tmem_base;
  int abort_flag;
  float ncols[MAX_PAIRS * 2];   // valid columns of every (pair, column half) warp: the weights of the partial means
  EpiProgram epi;
};
constexpr size_t SMEM_CL = (size_t)STAGES * STAGE_BYTES + EPI_WARPS * EPI_WARP_BYTES + COLVEC_BYTES + PART_BYTES + RES_BYTES + 1024 + 512;
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
  uint8_t* res_slots = reinterpret_cast<uint8_t*>(part) + PART_BYTES;
  SharedCl* sh = reinterpret_cast<SharedCl*>(res_slots + RES_BYTES);
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
      tc::mbar_init(&sh->stat_bar[b], 1);     // one local arrival that announces the bytes the P CTAs sharing these rows will send
    }
    for (int i = 0; i < MAX_PAIRS * 2; ++i) sh->ncols[i] = (float)warp_cols(i >> 1, i & 1, NT, N);
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
    const float n_w = sh->ncols[pi * 2 + half];
    const float inv_nw = n_w > 0.0f ? 1.0f / n_w : 0.0f;
    const uint32_t part_local = tc::smem_u32(part);
    const uint32_t stat_local = tc::smem_u32(&sh->stat_bar[0]);
    // A bf16 residual, when nothing else needs the staging buffer during pass 1 (no second output), is staged in
    // shared memory: this warp's four chunks of a tile land in four slots (the staging buffer and three more) while
    // the tile's MMAs run.  Slot layout as the bulk store's: a lane reads its own 64-byte row without conflicts.
    const bool res_ring = ew.res_idx >= 0 && !ew.res_f32 && mid_out == nullptr && NT == 1;
    uint8_t* my_slots = res_slots + (warp - 2) * RES_EXTRA_SLOTS * RES_SLOT_BYTES;
    auto slot_ptr = [&](int i) -> uint8_t* { return i == 0 ? ew.stage : my_slots + (i - 1) * RES_SLOT_BYTES; };
    auto ring_fill = [&](int64_t r0, int64_t col_base) {
      const uint8_t* res = reinterpret_cast<const uint8_t*>(epi.op[ew.res_idx].ptr);
      const int sub_row = lane >> 2, seg = lane & 3;
      int i = 0;
      for (int c = half; c < CHUNKS; c += 2, ++i) {
        const int64_t c0 = col_base + c * 32;
        if (c0 + 32 > N) break;
        const uint32_t dst0 = tc::smem_u32(slot_ptr(i));
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int rr = sub_row + 8 * k;
          if (r0 + rr < M) tc::cp_async16(dst0 + rr * 64 + ((seg ^ ((rr >> 1) & 3)) * 16), res + ((r0 + rr) * (int64_t)N + c0) * 2 + seg * 16);
        }
      }
      tc::cp_async_commit();
    };
    for (int rb = cluster_id; rb < num_rb && ok; rb += num_clusters, ++it) {
      const int64_t row0 = (int64_t)(rb * 2 + (int)r) * BM + q * 32;
      auto rowmap = [&](int rr) -> int64_t { const int64_t g = row0 + rr; return g < M ? g : -1; };
      const int use0 = use;
      const int buf = it & 1;
#ifdef MK_TRACE_RN
      long long tr[8];
      tr[0] = clock64();
#endif
      // the last bulk store of the row block before has finished reading the staging buffer, which pass 1 reuses
      if (lane == 0) tc::tma_store_wait_read();
      __syncwarp();
      // announce what this row block's partials will bring to this CTA's barrier (one thread per CTA)
      if (warp == 2 && lane == 0) tc::mbar_expect_tx(&sh->stat_bar[buf], (uint32_t)(P * EPI_WARPS * 32 * 8));
      if (res_ring) ring_fill(row0, (int64_t)pi * BN);
      // this lane's row over the warp's columns: for LayerNorm sums of (x - pivot) and (x - pivot)^2, for RMSNorm the sum of squares
      float s1 = 0.0f, s2 = 0.0f, pivot = 0.0f;
      bool have_pivot = false;
      // ---- pass 1: tail, write-back, sums
      for (int j = 0; j < NT && ok; ++j, ++use) {
        const int slot = use & 1;
        const int64_t col_base = (int64_t)(pi * NT + j) * BN;
        uint4 res_regs[8];
        ew.load_bias(epi, col_base, BN, N);
        if (!res_ring) ew.prefetch_res(epi, rowmap, col_base + half * 32, N, res_regs);
        ok = tc::mbar_wait(&sh->tfull[slot], (use >> 1) & 1, abort_flag, status, tc::WAIT_TMEM_FULL);
        ok = __all_sync(0xffffffffu, ok ? 1 : 0) != 0;
        if (!ok) break;
        tc::tc_fence_after();
#ifdef MK_TRACE_RN
        if (j == 0) tr[1] = clock64();
#endif
        if (res_ring) {
          tc::cp_async_wait<0>();
          __syncwarp();
        }
        const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + slot * BN;
        int ci = 0;
#pragma unroll 1
        for (int c = half; c < CHUNKS; c += 2, ++ci) {
          const int64_t c0 = col_base + c * 32;
          if (c0 >= N) break;            // warp-uniform; nothing of this tile is left
          uint32_t rg[32];
          float v[32];
          tc::tmem_ld32(t_row + c * 32, rg);
          tc::tmem_ld_wait();
#pragma unroll
          for (int k = 0; k < 32; ++k) v[k] = __uint_as_float(rg[k]);
          if (res_ring) {
            const uint8_t* src = slot_ptr(ci) + lane * 64;
            const int f = (lane >> 1) & 3;
            auto get = [&](uint4 (&ra)[4], uint4 (&)[4]) -> int {
#pragma unroll
              for (int k = 0; k < 4; ++k) ra[k] = *reinterpret_cast<const uint4*>(src + ((k ^ f) * 16));
              return 1;
            };
            auto skip = [&]() {};
            ew.chunk_out_from(epi, v, rowmap, mid_out, c0, c * 32, (int64_t)N, get, skip);
          } else {
            ew.chunk_out(epi, v, rowmap, mid_out, c0, c * 32, (int64_t)N, res_regs, c + 2 < CHUNKS ? col_base + (c + 2) * 32 : -1);
          }
          if (!have_pivot) { pivot = v[0]; have_pivot = true; }
#pragma unroll
          for (int k = 0; k < 32; ++k) {
            if (c0 + k >= N) v[k] = 0.0f;
            rg[k] = __float_as_uint(v[k]);
          }
          tc::tmem_st32(t_row + c * 32, rg);
          if (mode == ROW_LAYERNORM) {
#pragma unroll
            for (int k = 0; k < 32; ++k) {
              const float d = v[k] - pivot;
              if (c0 + k < N) { s1 += d; s2 = fmaf(d, d, s2); }
            }
          } else {
#pragma unroll
            for (int k = 0; k < 32; ++k) s2 = fmaf(v[k], v[k], s2);
          }
        }
        tc::tmem_st_wait();
      }
      if (!ok) break;
#ifdef MK_TRACE_RN
      tr[2] = clock64();
      tr[3] = tr[2];
#endif
      // ---- exchange: this lane's partial goes to the P CTAs that hold the rest of its row
      {
        float mean_w = 0.0f, m2_w = s2;
        if (mode == ROW_LAYERNORM) {
          mean_w = pivot + s1 * inv_nw;
          m2_w = fmaxf(s2 - s1 * s1 * inv_nw, 0.0f);
        }
        const uint32_t slot_off = (uint32_t)((((buf * MAX_PAIRS + pi) * 2 + half) * BM + q * 32 + lane) * 8);
        for (int pj = 0; pj < P; ++pj) {
          const uint32_t dst_rank = (uint32_t)(2 * pj) + r;
          tc::st_async_f32x2(tc::map_to_cta(part_local + slot_off, dst_rank), mean_w, m2_w, tc::map_to_cta(stat_local + (uint32_t)buf * 8u, dst_rank));
        }
        ok = tc::mbar_wait(&sh->stat_bar[buf], (it >> 1) & 1, abort_flag, status, tc::WAIT_ROW_STATS);
        ok = __all_sync(0xffffffffu, ok ? 1 : 0) != 0;
        if (!ok) break;
      }
#ifdef MK_TRACE_RN
      tr[4] = clock64();
#endif
      // ---- combine the 2P partials of this lane's row
      float mean = 0.0f, rstd;
      {
        const float2* pp = part + (size_t)buf * MAX_PAIRS * 2 * BM + q * 32 + lane;
        if (mode == ROW_LAYERNORM) {
          float sm = 0.0f;
          for (int i = 0; i < 2 * P; ++i) sm += sh->ncols[i] * pp[i * BM].x;
          mean = sm * inv_n;
          float m2 = 0.0f;
          for (int i = 0; i < 2 * P; ++i) {
            const float2 t = pp[i * BM];
            const float d = t.x - mean;
            m2 += t.y + sh->ncols[i] * d * d;
          }
          rstd = rsqrtf(m2 * inv_n + eps);
        } else {
          float sq = 0.0f;
          for (int i = 0; i < 2 * P; ++i) sq += pp[i * BM].y;
          rstd = rsqrtf(sq * inv_n + eps);
        }
      }
#ifdef MK_TRACE_RN
      tr[5] = clock64();
#endif
      // ---- pass 2: normalise out of TMEM, store, hand the accumulator back
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
        // (a relaxed arrival: the warp's reads of tensor memory are over, nothing has to be published)
        if (lane == 0) tc::mbar_arrive_cluster_relaxed(tc::map_to_cta(tc::smem_u32(&sh->tempty[slot]), leader_rank));
      }
#ifdef MK_TRACE_RN
      tr[6] = clock64();
      if (blockIdx.x == 0 && lane == 0 && (warp == 2 || warp == 9))
        printf("rn w%d it%d: wait_full %lld p1 %lld p2 %lld exch %lld comb %lld p3 %lld total %lld\n", warp, it, tr[1] - tr[0], tr[2] - tr[1],
               tr[3] - tr[2], tr[4] - tr[3], tr[5] - tr[4], tr[6] - tr[5], tr[6] - tr[0]);
#endif
    }
    if (res_ring) tc::cp_async_wait<0>();
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
  // A cluster lives inside one GPC, so fewer clusters of eight fit the machine than SMs / 8 (16 on a B200 whose
  // GPCs have 18 or 20 SMs): a cluster beyond that number would only start when another has finished and
  // double the kernel's time.  Ask the runtime how many can be resident at once.
  int64_t clusters = sm_count / (2 * P);
  {
    static SmemOptIn opt_in;
    cudaError_t e2 = opt_in.ensure(SMEM_CL, gemm_rownorm_cl_kernel);
    if (e2 != cudaSuccess) return e2;
    LaunchCfg lc(0, dim3((unsigned)(clusters * 2 * P)), dim3(THREADS), SMEM_CL, nullptr, 2 * P);
    int active = 0;
    if (cudaOccupancyMaxActiveClusters(&active, gemm_rownorm_cl_kernel, &lc.cfg) == cudaSuccess && active > 0) {
      if (active < clusters) clusters = active;
    } else {
      cudaGetLastError();
    }
  }
  const char* ov = getenv("MK_ROWNORM_CLUSTERS");
  if (ov && ov[0]) clusters = atoi(ov);
  if (clusters > row_blocks) clusters = row_blocks;
  if (clusters < 1) clusters = 1;
  if (getenv("MK_DEBUG_PLAN")) fprintf(stderr, "gemm_rownorm_cl plan: m %d n %d k %d pairs %d nt %d clusters %d\n", (int)m, (int)n, (int)k, P, NT, (int)clusters);
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
