// K1: bf16 GEMM with fused elementwise tail on the 5th-generation tensor cores.
//
//   D[M, N] = tail(A[M, K] @ W[K, N])        A row-major (K-major), W stored [N, K] (K-major)
//
// Two forms of one kernel:
//   CTAS = 2  a cluster of two CTAs (two SMs) shares one tcgen05.mma.cta_group::2 of shape 256x256x16.
//             Each CTA stages its own 128 rows of A and its own 128 of the tile's 256 W rows (32 KB per
//             stage, 6 stages), so each W byte crosses L2 -> SM once per pair.  No TMA multicast: each
//             CTA issues plain tile loads for its halves and both CTAs' loads complete on the leader's
//             "full" barrier; the leader's tcgen05.commit (multicast of a barrier arrival, not of data)
//             frees the stage in both CTAs and publishes the accumulator to both epilogues.
//   CTAS = 1  one CTA per 128x256 tile (48 KB per stage, 4 stages), for M <= 128.
//
// Per CTA, 10 warps:
//   warp 0        TMA producer (one lane): 128-byte-swizzled tiles into an mbarrier ring
//   warp 1        TMEM allocation (512 columns = two 128x256 fp32 accumulators); one lane of the leader
//                 CTA issues the MMAs.  The issue loop is kept to a few instructions per MMA: a single
//                 thread issuing dependent instructions can starve the tensor pipe (a 256x256x16 MMA
//                 lasts 128 cycles)
//   warps 2..9    epilogue of this CTA's 128 rows (two warps per TMEM lane quarter, alternating 32-column
//                 chunks): tcgen05.ld, elementwise program in fp32, bf16 pack, shared-memory transpose,
//                 coalesced stores; overlaps the next tile's MMAs through the second accumulator
// SwiGLU mode: accumulator columns [0,128) are gate columns and [128,256) the matching up columns
// (two TMA boxes of W; in the pair form the leader holds gate rows, the peer up rows); the tile's
// output is silu(gate) * up, 128 columns wide.
// Ragged M / N / K: TMA zero-fills out-of-range rows and K columns; stores are guarded.
// Every mbarrier wait is bounded (tc_common.cuh); a CTA pair leaves through a cluster barrier.
#include "device_common.cuh"
#include <stdlib.h>
#include "tc_common.cuh"
#include "tc_epilogue.cuh"
#include "tc_plans.h"

namespace mk {

namespace {

constexpr int BM = 128;   // rows per CTA
constexpr int BN = 256;   // accumulator columns
constexpr int BK = 64, UMMA_K = 16;
constexpr int EPI_WARPS = 8;
constexpr int THREADS = 64 + 32 * EPI_WARPS;
constexpr int GROUP_M_MAX = 16;  // most tile rows walked together for L2 reuse (the plan picks fewer for a long K)

template <int CTAS> struct Cfg {
  static constexpr int STAGES = CTAS == 2 ? 6 : 4;
  static constexpr int A_BYTES = BM * BK * 2;
  static constexpr int B_BYTES = (BN / CTAS) * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr size_t SMEM = (size_t)STAGES * STAGE_BYTES + EPI_WARPS * EPI_WARP_BYTES + 1024 /*alignment*/ + 512 /*barriers, program*/;
};

template <int STAGES> struct Shared {
  uint64_t full[STAGES];
  uint64_t empty[STAGES];
  uint64_t tfull[2];
  uint64_t tempty[2];
  uint32_t tmem_base;
  int abort_flag;
  EpiProgram epi;   // the kernel parameter, copied once (see epi_copy_to_smem)
  // fused row norm: first row of the 32-row block each epilogue warp completed with its last tile (-1: none),
  // double-buffered by tile parity
  long long fix_row0[2][EPI_WARPS];
  uint64_t fix_bar;   // the epilogue warps meet here once per tile (bounded wait, like every other)
};

__device__ __forceinline__ void tile_coords(int t, int num_m, int num_n, int group_m, int& mi, int& ni) {
  const int per_group = group_m * num_n;
  const int g = t / per_group;
  const int first_m = g * group_m;
  const int gsz = min(num_m - first_m, group_m);
  const int r = t - g * per_group;
  mi = first_m + r % gsz;
  ni = r / gsz;
}

// Normalise rows [row0 + first, row0 + first + count) of the bf16 matrix out[M, N] in place, from the partial
// sums every epilogue warp left behind.  One warp: lane l < count sums the partials of row l, then the whole
// warp streams each row with all of a row's loads in flight at once (16 bytes per lane, read through L2:
// other SMs wrote these bytes; a load-compute-store loop would pay one L2 round trip per 512 bytes).
__device__ __forceinline__ void rownorm_fixup(const RowNormArgs& na, __nv_bfloat16* out, int64_t row0, int first, int count, int M, int N,
                                              int slots, int lane) {
  const int64_t my = row0 + first + lane;
  float sm = 0.0f, sq = 0.0f;
  if (lane < count && my < M) {
    const float2* p = reinterpret_cast<const float2*>(na.partials) + my * slots;
    for (int k = 0; k < slots; ++k) {
      const float2 v = __ldcg(p + k);
      sm += v.x;
      sq += v.y;
    }
  }
  const float inv_n = 1.0f / (float)N;
  const float mean = na.mode == ROW_LAYERNORM ? sm * inv_n : 0.0f;
  const float rstd = rsqrtf(fmaxf(sq * inv_n - mean * mean, 0.0f) + na.eps);
  const __nv_bfloat16* gamma = reinterpret_cast<const __nv_bfloat16*>(na.gamma);
  const __nv_bfloat16* beta = na.mode == ROW_LAYERNORM ? reinterpret_cast<const __nv_bfloat16*>(na.beta) : nullptr;
#pragma unroll 1
  for (int r = 0; r < count; ++r) {
    const int64_t gr = row0 + first + r;
    if (gr >= M) break;
    const float mr = __shfl_sync(0xffffffffu, mean, r), rs = __shfl_sync(0xffffffffu, rstd, r);
    __nv_bfloat16* rowp = out + gr * N;
#pragma unroll 1
    for (int base = 0; base < N; base += 8 * 256) {
      uint4 raw[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int c0 = base + u * 256 + lane * 8;
        if (c0 < N) raw[u] = __ldcg(reinterpret_cast<const uint4*>(rowp + c0));
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int c0 = base + u * 256 + lane * 8;
        if (c0 >= N) continue;
        const uint32_t w[4] = {raw[u].x, raw[u].y, raw[u].z, raw[u].w};
        float x[8], g[8], b[8];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          x[2 * k] = __uint_as_float(w[k] << 16);
          x[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
        }
        if (gamma) ld_vec(gamma + c0, g);
        if (beta) ld_vec(beta + c0, b);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          float y = (x[k] - mr) * rs;
          if (gamma) y *= g[k];
          if (beta) y += b[k];
          x[k] = y;
        }
        st_vec(rowp + c0, x);
      }
    }
  }
}

// RING (two-SM form): one pipeline stage less, and its shared memory holds, per epilogue warp, two 32-row x 64-byte
// slots into which a bf16 residual is copied asynchronously two chunks ahead of its use (RES_RING_BYTES in all).
constexpr int RES_SLOT_BYTES = 32 * 64;
constexpr int RES_RING_BYTES = EPI_WARPS * 2 * RES_SLOT_BYTES;
static_assert(RES_RING_BYTES <= Cfg<2>::STAGE_BYTES, "the residual ring takes the place of one pipeline stage");

template <int CTAS, bool SWIGLU, bool NORM = false, bool RING = false, bool PRE = false>
__global__ void __launch_bounds__(THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmBh,
               const __grid_constant__ CUtensorMap tmOut, int bulk_store, void* __restrict__ out, int out_f32, int M, int N, int K, int up_row_offset, int tail_first, int group_m,
               const __grid_constant__ EpiProgram epi_param, const __grid_constant__ RowNormArgs na, unsigned int* status,
               const __grid_constant__ CUtensorMap tmAux, const __grid_constant__ PreNormArgs pn) {
  using C = Cfg<CTAS>;
  static_assert(!RING || (CTAS == 2 && !SWIGLU && !NORM), "the residual ring exists in the plain two-SM form only");
  static_assert(!PRE || (CTAS == 2 && !NORM && !RING), "the folded pre-norm exists in the plain two-SM form only");
  constexpr int STAGES = C::STAGES - (RING ? 1 : 0);
  constexpr int OUT_N = SWIGLU ? BN / 2 : BN;  // output columns per tile
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* res_ring = tiles + (size_t)STAGES * C::STAGE_BYTES;       // RING only: the space of the stage given up
  uint8_t* staging = tiles + (size_t)C::STAGES * C::STAGE_BYTES;
  Shared<C::STAGES>* sh = reinterpret_cast<Shared<C::STAGES>*>(staging + EPI_WARPS * EPI_WARP_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = CTAS == 2 ? tc::cluster_ctarank() : 0;
  const bool leader = rank == 0;
  const int unit_id = blockIdx.x / CTAS, num_units = gridDim.x / CTAS;   // a unit = a CTA or a CTA pair
  const int num_m = (M + CTAS * BM - 1) / (CTAS * BM), num_n = (N + OUT_N - 1) / OUT_N;
  const int total_tiles = num_m * num_n;
  // Work units: tiles [0, tail_first) whole; each tile from tail_first on as two units of half the columns
  // (256 x 128, N = 128 MMAs), so that a last wave that would leave more than half of the machine idle is
  // spread over twice as many CTA pairs.  tail_first = total_tiles: no split.
  const int total_units = tail_first + 2 * (total_tiles - tail_first);
  auto decode = [&](int u, int& tile, int& nhalf) {
    if (u < tail_first) { tile = u; nhalf = -1; }
    else { tile = tail_first + ((u - tail_first) >> 1); nhalf = (u - tail_first) & 1; }
  };
  const int num_kb = (K + BK - 1) / BK;
  volatile int* abort_flag = &sh->abort_flag;
  MK_TR_DECL
  MK_TR_INIT;

  static_assert(sizeof(Shared<C::STAGES>) <= 512, "barrier block");
  epi_copy_to_smem(&sh->epi, epi_param, threadIdx.x, THREADS);
  const EpiProgram& epi = sh->epi;
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&sh->full[s], 1); tc::mbar_init(&sh->empty[s], 1); }
    for (int b = 0; b < 2; ++b) { tc::mbar_init(&sh->tfull[b], 1); tc::mbar_init(&sh->tempty[b], EPI_WARPS * CTAS); }
    tc::mbar_init(&sh->fix_bar, EPI_WARPS);
    sh->abort_flag = 0;
    tc::fence_barrier_init();
    tc::tma_prefetch_desc(&tmA);
    tc::tma_prefetch_desc(&tmB);
  }
  if (warp == 1) {
    if (CTAS == 2) tc::tmem_alloc_pair(&sh->tmem_base, 512);
    else { tc::tmem_alloc(&sh->tmem_base, 512); tc::tmem_relinquish(); }
  }
  tc::tc_fence_before();
  __syncthreads();
  if (CTAS == 2) tc::cluster_sync();  // both CTAs' barriers exist before anything remote touches them
  tc::tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;
  // set-up done: the next kernel may be scheduled as this grid drains; nothing of the previous kernel's
  // output (A, a residual) is read before it has completed
  pdl_launch_dependents();
  pdl_wait();

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int u = unit_id; u < total_units && ok; u += num_units) {
        int t, nhalf;
        decode(u, t, nhalf);
        int mi, ni;
        tile_coords(t, num_m, num_n, group_m, mi, ni);
        const int m0 = (mi * CTAS + (int)rank) * BM;
        const int n0 = ni * OUT_N;
#ifdef MK_TRACE
        unsigned long long esum = 0;
#endif
        for (int kb = 0; kb < num_kb; ++kb) {
#ifdef MK_TRACE
          const unsigned long long w0_ = tc::gtime();
#endif
          ok = tc::mbar_wait(&sh->empty[stage], phase ^ 1, abort_flag, status, tc::WAIT_SMEM_EMPTY);
#ifdef MK_TRACE
          esum += tc::gtime() - w0_;
          if (kb == num_kb - 1 && blockIdx.x == 0) mk_tr[70 + (u - unit_id) / num_units] = mk_tr[0] + esum;
#endif
          if (!ok) break;
          uint8_t* a_dst = tiles + (size_t)stage * C::STAGE_BYTES;
          uint8_t* b_dst = a_dst + C::A_BYTES;
          if (CTAS == 2) {
            const uint32_t full_leader = tc::map_to_cta(tc::smem_u32(&sh->full[stage]), 0);
            tc::tma_load_2d_pair(a_dst, &tmA, full_leader, kb * BK, m0);
            if (nhalf < 0) {
              if (leader) tc::mbar_expect_tx(&sh->full[stage], 2 * C::STAGE_BYTES);
              const int b_row = SWIGLU ? (leader ? n0 : up_row_offset + n0) : n0 + (int)rank * (BN / 2);
              tc::tma_load_2d_pair(b_dst, &tmB, full_leader, kb * BK, b_row);
            } else {
              // half the columns: 64 W rows per CTA
              if (leader) tc::mbar_expect_tx(&sh->full[stage], 2 * (C::A_BYTES + C::B_BYTES / 2));
              tc::tma_load_2d_pair(b_dst, &tmBh, full_leader, kb * BK, n0 + nhalf * (BN / 2) + (int)rank * (BN / 4));
            }
          } else {
            tc::mbar_expect_tx(&sh->full[stage], C::STAGE_BYTES);
            tc::tma_load_2d(a_dst, &tmA, &sh->full[stage], kb * BK, m0);
            tc::tma_load_2d(b_dst, &tmB, &sh->full[stage], kb * BK, n0);
            tc::tma_load_2d(b_dst + C::B_BYTES / 2, &tmB, &sh->full[stage], kb * BK, SWIGLU ? up_row_offset + n0 : n0 + BN / 2);
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (one lane of the leader)
    if (leader && lane == 0) {
      constexpr uint32_t idesc_full = tc::idesc_bf16_f32(CTAS * BM, BN, 0, 0);
      constexpr uint32_t idesc_half = tc::idesc_bf16_f32(CTAS * BM, BN / 2, 0, 0);
      const uint32_t a_lo0 = tc::desc_lo_sw128(tc::smem_u32(tiles));
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int it = 0;
      for (int u = unit_id; u < total_units && ok; u += num_units, ++it) {
        const uint32_t idesc = u < tail_first ? idesc_full : idesc_half;
        const int acc = it & 1;
        const uint32_t d_tmem = tmem_base + acc * BN;
        ok = tc::mbar_wait(&sh->tempty[acc], ((it >> 1) & 1) ^ 1, abort_flag, status, tc::WAIT_TMEM_EMPTY);
        if (!ok) break;
        tc::tc_fence_after();
        MK_TR(1 + it * 8);                       // MMA: accumulator free, tile starts
        uint32_t accumulate = 0;
#ifdef MK_TRACE
        unsigned long long wsum = 0;
#endif
        for (int kb = 0; kb < num_kb; ++kb) {
#ifdef MK_TRACE
          const unsigned long long w0_ = tc::gtime();
#endif
          ok = tc::mbar_wait(&sh->full[stage], phase, abort_flag, status, tc::WAIT_SMEM_FULL);
#ifdef MK_TRACE
          wsum += tc::gtime() - w0_;
          if (kb == num_kb - 1 && blockIdx.x == 0) mk_tr[60 + it] = mk_tr[0] + wsum;
#endif
          if (!ok) break;
          tc::tc_fence_after();
          const uint32_t a_lo = a_lo0 + (uint32_t)stage * (C::STAGE_BYTES >> 4);
          const uint32_t b_lo = a_lo + (C::A_BYTES >> 4);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            if (CTAS == 2) tc::umma_ss_pair_lohi(d_tmem, a_lo + 2 * k, b_lo + 2 * k, idesc, accumulate);
            else tc::umma_ss_lohi(d_tmem, a_lo + 2 * k, b_lo + 2 * k, idesc, accumulate);
            accumulate = 1;
          }
          if (CTAS == 2) tc::umma_commit_pair(&sh->empty[stage]);
          else tc::umma_commit(&sh->empty[stage]);
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        MK_TR(2 + it * 8);                       // MMA: last MMA of the tile issued
        if (CTAS == 2) tc::umma_commit_pair(&sh->tfull[acc]);
        else tc::umma_commit(&sh->tfull[acc]);
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ epilogue: this CTA's 128 rows
    // eight warps: warp w reads TMEM lane quarter w % 4 (the hardware's rule) and takes every other
    // 32-column chunk, so each scheduler has two epilogue warps to interleave
    const int q = warp & 3;
    const int half = (warp - 2) >> 2;
    constexpr int CHUNKS = OUT_N / 32;
    EpiWarp ew;
    ew.init(staging + (warp - 2) * EPI_WARP_BYTES, epi, lane, out_f32 != 0);
    bool ok = true;
    int it = 0;
    // RING: the warp's chunks form one sequence across its tiles (unit u, chunk c = half, half + 2, ...).  A cursor
    // runs two chunks ahead of the one being stored; every chunk, once its residual has been read out of its slot,
    // starts the copy of the chunk at the cursor into that slot (16 bytes per lane and row, swizzled like the store
    // staging so that the lane's read of its own 64-byte row is free of bank conflicts), one commit group per chunk.
    uint8_t* my_ring = res_ring + (warp - 2) * 2 * RES_SLOT_BYTES;
    int pf_u = unit_id, pf_c = half, res_slot = 0;
    // what the cursor's tile fixes, recomputed when the cursor moves to another tile and not once per chunk: its first
    // row of this warp, its first column, its number of chunks, and this lane's first source address
    int64_t pf_r0 = 0, pf_cb = 0;
    int pf_chunks = 0;
    const uint8_t* pf_src = nullptr;
    auto ring_tile = [&]() {
      if (pf_u >= total_units) return;
      int t, nhalf;
      decode(pf_u, t, nhalf);
      int mi, ni;
      tile_coords(t, num_m, num_n, group_m, mi, ni);
      pf_r0 = (int64_t)(mi * CTAS + (int)rank) * BM + q * 32;
      pf_cb = (int64_t)ni * OUT_N + (nhalf > 0 ? BN / 2 : 0);
      pf_chunks = nhalf < 0 ? CHUNKS : CHUNKS / 2;
      pf_src = reinterpret_cast<const uint8_t*>(epi.op[ew.res_idx].ptr) + ((pf_r0 + (lane >> 2)) * (int64_t)N + pf_cb) * 2 + (lane & 3) * 16;
    };
    auto ring_issue = [&](int slot) {
      if (pf_u < total_units) {
        if (pf_cb + pf_c * 32 + 32 <= N) {
          const int sub_row = lane >> 2, seg = lane & 3;
          const uint32_t dst0 = tc::smem_u32(my_ring + slot * RES_SLOT_BYTES);
          const uint8_t* src = pf_src + pf_c * 64;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int r = sub_row + 8 * i;
            if (pf_r0 + r < M) tc::cp_async16(dst0 + r * 64 + ((seg ^ ((r >> 1) & 3)) * 16), src + (int64_t)(8 * i) * N * 2);
          }
        }
        pf_c += 2;
        if (pf_c >= pf_chunks) { pf_u += num_units; pf_c = half; ring_tile(); }
      }
      tc::cp_async_commit();
    };
    auto ring_get = [&](uint4 (&ra)[4], uint4 (&)[4]) -> int {
      tc::cp_async_wait<1>();      // this chunk's group (the older of the two in flight) has landed
      __syncwarp();                // ... for every lane
      const uint8_t* src = my_ring + res_slot * RES_SLOT_BYTES + lane * 64;
      const int f = (lane >> 1) & 3;
#pragma unroll
      for (int i = 0; i < 4; ++i) ra[i] = *reinterpret_cast<const uint4*>(src + ((i ^ f) * 16));
      __syncwarp();                // every lane has read its row: the slot may be refilled
      ring_issue(res_slot);
      res_slot ^= 1;
      return 1;
    };
    auto ring_skip = [&]() {
      tc::cp_async_wait<1>();
      __syncwarp();
      ring_issue(res_slot);
      res_slot ^= 1;
    };
    if (RING) {
      ring_tile();
      ring_issue(0);
      ring_issue(1);
    }
    for (int u = unit_id; u < total_units && ok; u += num_units, ++it) {
      int t, nhalf;
      decode(u, t, nhalf);
      int mi, ni;
      tile_coords(t, num_m, num_n, group_m, mi, ni);
      const int acc = it & 1;
      const int64_t row0 = (int64_t)(mi * CTAS + (int)rank) * BM + q * 32;
      auto rowmap = [&](int r) -> int64_t { const int64_t g = row0 + r; return g < M ? g : -1; };
      const int64_t col_base = (int64_t)ni * OUT_N + (nhalf > 0 ? BN / 2 : 0);
      // chunks of this unit; without the ring (whose cursor counts every chunk of every tile) only those that begin inside N
      const int chunks_unit = nhalf < 0 ? CHUNKS : CHUNKS / 2;
      const int chunks_here = RING ? chunks_unit : (int)min((int64_t)chunks_unit, (N - col_base + 31) / 32);
      uint4 res_regs[8];
      ew.load_bias(epi, col_base, nhalf < 0 ? OUT_N : OUT_N / 2, N);
      if (!RING) ew.prefetch_res(epi, rowmap, col_base + half * 32, N, res_regs);
      float pre_rstd = 1.0f;
      if (PRE && pn.part_in) {
        // this lane's row: the partial sums of squares its producer left, read while the accumulator is still filling
        const int64_t my = row0 + lane;
        float sq = 0.0f;
        if (my < M) {
          const float* pp = pn.part_in + my * pn.slots_in;
          if ((pn.slots_in & 3) == 0) {
            for (int k = 0; k < pn.slots_in; k += 4) {
              const float4 t4 = *reinterpret_cast<const float4*>(pp + k);
              sq += (t4.x + t4.y) + (t4.z + t4.w);
            }
          } else {
            for (int k = 0; k < pn.slots_in; ++k) sq += pp[k];
          }
        }
        pre_rstd = rsqrtf(sq * pn.inv_n_in + pn.eps_in);
      }
      if (threadIdx.x == 64) MK_TR(7 + it * 8);  // epilogue: bias in shared memory, about to wait for the accumulator
      ok = tc::mbar_wait(&sh->tfull[acc], (it >> 1) & 1, abort_flag, status, tc::WAIT_TMEM_FULL);
      ok = __all_sync(0xffffffffu, ok ? 1 : 0) != 0;
      if (!ok) break;
      if (threadIdx.x == 64) MK_TR(3 + it * 8);  // epilogue: accumulator ready
      tc::tc_fence_after();
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + acc * BN;
      float rsum = 0.0f, rsq = 0.0f;   // NORM: this lane's row, over the columns this warp stores (PRE producer: rsq alone)
#pragma unroll 1
      for (int c = half; c < chunks_here; c += 2) {
        uint32_t r[32];
        float v[32];
        float gl = 1.0f;               // PRE producer: gamma of column c0 + lane, asked for before the accumulator is read
        if (PRE && pn.part_out) {
          const int64_t gc = col_base + c * 32 + lane;
          if (pn.gamma && gc < N) gl = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(pn.gamma)[gc]);
          // the previous chunk's bulk store of xg has finished reading the staging buffer
          if (lane == 0) tc::tma_store_wait_read();
          __syncwarp();
        }
#ifdef MK_TRACE
        ew.tr = (threadIdx.x == 64 && it == 2 && c == half + 2 && blockIdx.x == 0) ? &mk_tr[50] : nullptr;
        if (ew.tr) ew.tr[-1] = (unsigned long long)clock64();
#endif
        tc::tmem_ld32(t_row + c * 32, r);
        tc::tmem_ld_wait();
#ifdef MK_TRACE
        if (ew.tr) ew.tr[0] = (unsigned long long)clock64();
#endif
        if (threadIdx.x == 64 && c == half + 2) MK_TR(5 + it * 8);  // epilogue: second chunk in registers
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
        if (PRE && pn.part_in) {
          // consumer of a folded RMSNorm: the row's 1 / rms multiplies the accumulator before anything else
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] *= pre_rstd;
        }
        if (SWIGLU) {
          tc::tmem_ld32(t_row + BN / 2 + c * 32, r);
          tc::tmem_ld_wait();
          if (PRE && pn.part_in) {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = silu_fast(v[j]) * (__uint_as_float(r[j]) * pre_rstd);
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = silu_fast(v[j]) * __uint_as_float(r[j]);
          }
        }
        if (RING)
          ew.chunk_out_from(epi, v, rowmap, out, col_base + c * 32, c * 32, (int64_t)N, ring_get, ring_skip, bulk_store ? &tmOut : nullptr, row0);
        else
          ew.chunk_out(epi, v, rowmap, out, col_base + c * 32, c * 32, (int64_t)N, res_regs, c + 2 < chunks_here ? col_base + (c + 2) * 32 : -1,
                       (!NORM && bulk_store) ? &tmOut : nullptr, row0);
        if (threadIdx.x == 64 && c == half + 2) MK_TR(6 + it * 8);  // epilogue: second chunk handed to the store
        if (NORM) {
          // v now holds the values after the elementwise tail (what was just stored, before its bf16 rounding)
          const int64_t c0 = col_base + c * 32;
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (c0 + j < N) { rsum += v[j]; rsq = fmaf(v[j], v[j], rsq); }
        }
        if (PRE && pn.part_out) {
          // producer of a folded RMSNorm: v is the norm's input (after this GEMM's tail).  Its squares go to the row's
          // partial sum, and xg = bf16(v * gamma) leaves beside the main output, as a bulk tensor store.
          const int64_t c0 = col_base + c * 32;
          if (c0 < N) {
            const int64_t my_row = rowmap(lane);
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              if (c0 + j < N) rsq = fmaf(v[j], v[j], rsq);
              v[j] *= __shfl_sync(0xffffffffu, gl, j);
            }
            if (c0 + 32 <= N) {
              uint4 mine[4];
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                mine[k].x = pack_bf16x2(v[8 * k + 0], v[8 * k + 1]);
                mine[k].y = pack_bf16x2(v[8 * k + 2], v[8 * k + 3]);
                mine[k].z = pack_bf16x2(v[8 * k + 4], v[8 * k + 5]);
                mine[k].w = pack_bf16x2(v[8 * k + 6], v[8 * k + 7]);
              }
              // a bf16 main output has just left through the same staging buffer
              if (lane == 0) tc::tma_store_wait_read();
              __syncwarp();
              ew.own_row_to_global_bulk(mine, &tmAux, (int32_t)c0, (int32_t)row0);
            } else if (my_row >= 0) {
              __nv_bfloat16* xg = reinterpret_cast<__nv_bfloat16*>(pn.xg);
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (c0 + j < N) xg[my_row * N + c0 + j] = __float2bfloat16_rn(v[j]);
            }
          }
        }
      }
      if (PRE && pn.part_out) {
        const int64_t my = row0 + lane;
        if (my < M) pn.part_out[my * (2 * num_n) + ni * 2 + half] = rsq;
      }
      tc::tc_fence_before();
      __syncwarp();
      if (threadIdx.x == 64) MK_TR(4 + it * 8);  // epilogue: tile stored
      if (lane == 0) {
        // a relaxed arrival: what must be over are this warp's reads of tensor memory (tcgen05.wait::ld and the fence
        // above), nothing written to memory has to be published; the release form at cluster scope held each warp
        // for some two thousand cycles per tile
        if (CTAS == 2) tc::mbar_arrive_cluster_relaxed(tc::map_to_cta(tc::smem_u32(&sh->tempty[acc]), 0));
        else tc::mbar_arrive(&sh->tempty[acc]);
      }
      if (threadIdx.x == 64 && it) MK_TR(it * 8);  // epilogue: accumulator handed back
      if (NORM) {
        // partial sums of this warp's share of the rows, then count this warp in; the warp that completes the
        // block of 32 rows (2 * column tiles arrivals: both column halves of every tile) normalises it
        const int slots = 2 * num_n;
        const int64_t my = row0 + lane;
        if (my < M) reinterpret_cast<float2*>(na.partials)[my * slots + ni * 2 + half] = make_float2(rsum, rsq);
        __threadfence();
        __syncwarp();
        int old = 0;
        if (lane == 0) old = atomicAdd(na.counters + ((mi * CTAS + (int)rank) * 4 + q), 1);
        old = __shfl_sync(0xffffffffu, old, 0);
        // A completed block is normalised by all eight epilogue warps of this CTA together (four rows each): one
        // warp alone would spend tens of microseconds on it.  Every warp posts what it completed, the warps
        // meet, and each takes its rows of every posted block.
        const int ew_id = warp - 2;
        if (lane == 0) sh->fix_row0[it & 1][ew_id] = old == slots - 1 ? (long long)row0 : -1LL;
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(&sh->fix_bar);
        ok = tc::mbar_wait(&sh->fix_bar, it & 1, abort_flag, status, tc::WAIT_TMEM_FULL);
        ok = __all_sync(0xffffffffu, ok ? 1 : 0) != 0;
        if (!ok) break;
#pragma unroll 1
        for (int w_ = 0; w_ < EPI_WARPS; ++w_) {
          const long long fr = sh->fix_row0[it & 1][w_];
          if (fr < 0) continue;
          __threadfence();
          rownorm_fixup(na, reinterpret_cast<__nv_bfloat16*>(out), fr, ew_id * (32 / EPI_WARPS), 32 / EPI_WARPS, M, N, slots, lane);
        }
      }
    }
    if (RING) tc::cp_async_wait<0>();           // no copy into shared memory is in flight when the CTA retires
    if (lane == 0) tc::tma_store_wait_all();   // bulk stores of this warp are complete before the CTA retires
  }

  MK_TR_PRINT("gemm");

  // common exit: on an aborted run give copies in flight time to land before the CTA retires
  if (*abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < 4000000LL) {}
  }
  tc::tc_fence_before();
  __syncthreads();
  if (CTAS == 2) tc::cluster_sync();  // the peer's shared memory and barriers stay alive until both are done
  if (warp == 1) {
    tc::tc_fence_after();
    if (CTAS == 2) tc::tmem_dealloc_pair(tmem_base, 512);
    else tc::tmem_dealloc(tmem_base, 512);
  }
}

template <int CTAS>
cudaError_t plan_impl(GemmTcPlan* p, const void* a, const void* w_nk, void* y, bool out_f32, int64_t m, int64_t n, int64_t k, bool swiglu,
                      const EpiProgram& epi, int sm_count) {
  if (k % 8 || n % 8 || m < 1 || n < 1 || k < 1) return cudaErrorInvalidValue;
  if (m > INT32_MAX || n > INT32_MAX || k > INT32_MAX) return cudaErrorInvalidValue;
  const int64_t w_rows = swiglu ? 2 * n : n;
  cudaError_t e = encode_tmap_2d_bf16(&p->tm_a, a, (uint64_t)m, (uint64_t)k, (uint64_t)k, BM, BK);
  if (e != cudaSuccess) return e;
  e = encode_tmap_2d_bf16(&p->tm_b, w_nk, (uint64_t)w_rows, (uint64_t)k, (uint64_t)k, BN / 2, BK);
  if (e != cudaSuccess) return e;
  e = encode_tmap_2d_bf16(&p->tm_b_half, w_nk, (uint64_t)w_rows, (uint64_t)k, (uint64_t)k, BN / 4, BK);
  if (e != cudaSuccess) return e;
  p->out = y;
  p->out_f32 = out_f32;
  p->use_tm_out = false;
  e = out_f32 ? encode_tmap_2d_f32_store(&p->tm_out, y, (uint64_t)m, (uint64_t)n, (uint64_t)n)
              : encode_tmap_2d_bf16_store(&p->tm_out, y, (uint64_t)m, (uint64_t)n, (uint64_t)n);
  if (e != cudaSuccess) return e;
  p->use_tm_out = true;   // bf16 and fp32 outputs both leave by bulk tensor stores (fp32: 71 -> 68 us on 8192 x 2048 x 2048)
  p->m = (int)m; p->n = (int)n; p->k = (int)k;
  p->swiglu = swiglu;
  p->epi = epi;
  p->tm_aux = p->tm_a;   // never read unless a folded pre-norm replaces it
  p->pre = PreNormArgs{};
  p->use_pre = false;
  const int out_n = swiglu ? BN / 2 : BN;
  const int64_t tiles = ((m + CTAS * BM - 1) / (CTAS * BM)) * ((n + out_n - 1) / out_n);
  const int64_t units = tiles < sm_count / CTAS ? tiles : sm_count / CTAS;
  p->grid = (int)(CTAS * units);
  // a last wave that fills at most half of the CTA pairs is run as half-width units (two-SM form only)
  // a bf16 residual of the plain two-SM form travels through the shared-memory ring
  p->res_ring = false;
  if (CTAS == 2 && !swiglu) {
    int idx = -1, cnt = 0;
    for (int i = 0; i < epi.n; ++i)
      if (epi.op[i].kind == EPI_RESIDUAL) { idx = i; ++cnt; }
    p->res_ring = cnt == 1 && epi.op[idx].ptr_dtype == DT_BF16;
  }
  // When the whole of W fits in L2 beside the A rows in flight (up to 48 MB), walking one tile row at a time is
  // fastest: its column tiles run on neighbouring pairs at the same moment and share each A row while it passes
  // (measured over groups of 1, 2, 4, 8, 16: 8192 x 2048 x 8192 185.7 ... 193.1 us, 8192 x 6144 x 2048 131.8 ... 133.7 us,
  // 32768 x 2048 x 2048 177.3 ... 179.0 us; with 67 MB of W, 8192 x 16384 x 2048, the order turns round: 382.8 ... 352.4 us).
  // Tile rows walked together: their A rows (group_m x CTAS x 128 rows of K) plus the W slabs in flight should stay
  // in L2 for the walk across the columns.  With K = 8192 sixteen tile rows are 67 MB of A and the DRAM traffic
  // doubles (measured: 541 MB for 302 MB algorithmic); the budget below keeps a group's A rows under ~36 MB.
  {
    int g = GROUP_M_MAX;
    const char* ov = getenv("MK_GEMM_GROUP_M");
    if (ov && ov[0]) g = atoi(ov);
    else if ((int64_t)(swiglu ? 2 : 1) * n * k * 2 <= (int64_t)48 << 20) g = 1;   // W stays in L2 whatever the walk: see below
    else while (g > 2 && (int64_t)g * CTAS * BM * k * 2 > (int64_t)36 << 20) g /= 2;
    p->group_m = g < 1 ? 1 : g;
  }
  const int64_t tail = tiles % units;
  p->tail_first = (int)tiles;
  if (CTAS == 2 && !swiglu && tiles > units && tail > 0 && 2 * tail <= units) p->tail_first = (int)(tiles - tail);
  return cudaSuccess;
}

template <int CTAS>
cudaError_t launch_impl(const GemmTcPlan& p, cudaStream_t s) {
  static SmemOptIn opt_in;
  cudaError_t e0 = opt_in.ensure(Cfg<CTAS>::SMEM, gemm_tc_kernel<CTAS, false>, gemm_tc_kernel<CTAS, true>, gemm_tc_kernel<CTAS, false, false, CTAS == 2>);
  if (e0 != cudaSuccess) return e0;
  LaunchCfg lc(PDL_GEMM, dim3((unsigned)p.grid), dim3(THREADS), Cfg<CTAS>::SMEM, s, CTAS == 2 ? 2 : 0);
  cudaLaunchConfig_t& cfg = lc.cfg;
  unsigned int* status = kernel_status_ptr();
  const int out_f32 = p.out_f32 ? 1 : 0;
  if constexpr (CTAS == 2) {
    if (p.use_pre) {
      static SmemOptIn opt_in_pre;
      cudaError_t e1 = opt_in_pre.ensure(Cfg<2>::SMEM, gemm_tc_kernel<2, false, false, false, true>, gemm_tc_kernel<2, true, false, false, true>);
      if (e1 != cudaSuccess) return e1;
      if (p.swiglu)
        return cudaLaunchKernelEx(&cfg, gemm_tc_kernel<2, true, false, false, true>, p.tm_a, p.tm_b, p.tm_b_half, p.tm_out, p.use_tm_out ? 1 : 0, p.out, out_f32, p.m, p.n,
                                  p.k, p.n, p.tail_first, p.group_m, p.epi, p.norm, status, p.tm_aux, p.pre);
      return cudaLaunchKernelEx(&cfg, gemm_tc_kernel<2, false, false, false, true>, p.tm_a, p.tm_b, p.tm_b_half, p.tm_out, p.use_tm_out ? 1 : 0, p.out, out_f32, p.m,
                                p.n, p.k, 0, p.tail_first, p.group_m, p.epi, p.norm, status, p.tm_aux, p.pre);
    }
  }
  if (p.swiglu)
    return cudaLaunchKernelEx(&cfg, gemm_tc_kernel<CTAS, true>, p.tm_a, p.tm_b, p.tm_b_half, p.tm_out, p.use_tm_out ? 1 : 0, p.out, out_f32, p.m, p.n, p.k, p.n, p.tail_first, p.group_m, p.epi,
                              p.norm, status, p.tm_aux, p.pre);
  if (CTAS == 2 && p.res_ring)
    return cudaLaunchKernelEx(&cfg, gemm_tc_kernel<2, false, false, true>, p.tm_a, p.tm_b, p.tm_b_half, p.tm_out, p.use_tm_out ? 1 : 0, p.out, out_f32, p.m, p.n, p.k, 0,
                              p.tail_first, p.group_m, p.epi, p.norm, status, p.tm_aux, p.pre);
  return cudaLaunchKernelEx(&cfg, gemm_tc_kernel<CTAS, false>, p.tm_a, p.tm_b, p.tm_b_half, p.tm_out, p.use_tm_out ? 1 : 0, p.out, out_f32, p.m, p.n, p.k, 0, p.tail_first, p.group_m, p.epi,
                            p.norm, status, p.tm_aux, p.pre);
}

cudaError_t launch_norm_impl(const GemmTcPlan& p, cudaStream_t s) {
  static SmemOptIn opt_in;
  cudaError_t e0 = opt_in.ensure(Cfg<2>::SMEM, gemm_tc_kernel<2, false, true>);
  if (e0 != cudaSuccess) return e0;
  const int64_t row_blocks = ((p.m + 2 * BM - 1) / (2 * BM)) * 2 * 4;
  cudaError_t e = cudaMemsetAsync(p.norm.counters, 0, (size_t)row_blocks * sizeof(int), s);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)p.grid);
  cfg.blockDim = dim3(THREADS);
  cfg.dynamicSmemBytes = Cfg<2>::SMEM;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, gemm_tc_kernel<2, false, true>, p.tm_a, p.tm_b, p.tm_b_half, p.tm_out, 0, p.out, 0, p.m, p.n, p.k, 0, p.tail_first, p.group_m, p.epi, p.norm,
                            kernel_status_ptr(), p.tm_aux, p.pre);
}

}  // namespace

size_t gemm_rownorm_tc2_scratch(int64_t m, int64_t n) {
  const int64_t num_n = (n + BN - 1) / BN, num_m = (m + 2 * BM - 1) / (2 * BM);
  const size_t partials = (size_t)m * (size_t)(2 * num_n) * sizeof(float2);
  return (partials + 255) / 256 * 256 + (size_t)num_m * 2 * 4 * sizeof(int);
}
cudaError_t gemm_rownorm_tc2_plan(GemmTcPlan* p, const void* a, const void* w_nk, void* y, int64_t m, int64_t n, int64_t k,
                                  const EpiProgram& epi, int mode, const void* gamma, const void* beta, float eps, void* scratch,
                                  int sm_count) {
  cudaError_t e = plan_impl<2>(p, a, w_nk, y, false, m, n, k, false, epi, sm_count);
  if (e != cudaSuccess) return e;
  p->tail_first = (int)(((m + 2 * BM - 1) / (2 * BM)) * ((n + BN - 1) / BN));   // whole tiles only: the arrival count assumes it
  const int64_t num_n = (n + BN - 1) / BN;
  const size_t partials = (size_t)m * (size_t)(2 * num_n) * sizeof(float2);
  p->norm.partials = reinterpret_cast<float*>(scratch);
  p->norm.counters = reinterpret_cast<int*>(reinterpret_cast<char*>(scratch) + (partials + 255) / 256 * 256);
  p->norm.gamma = gamma;
  p->norm.beta = beta;
  p->norm.eps = eps;
  p->norm.mode = mode;
  return cudaSuccess;
}
cudaError_t launch_gemm_rownorm_tc2(const GemmTcPlan& p, cudaStream_t s) { return launch_norm_impl(p, s); }

size_t gemm_prenorm_scratch(int64_t m, int64_t n1) {
  const int64_t num_n = (n1 + BN - 1) / BN;
  const size_t xg = ((size_t)m * (size_t)n1 * 2 + 255) / 256 * 256;
  return xg + (size_t)m * (size_t)(2 * num_n) * sizeof(float);
}
cudaError_t gemm_prenorm_pair_plan(GemmTcPlan* p1, GemmTcPlan* p2, const void* a, const void* w1_nk, void* y1, bool y1_f32, int64_t m, int64_t n1,
                                   int64_t k1, const EpiProgram& epi1, const void* gamma, float eps, const void* w2_nk, void* y2, int64_t n2,
                                   bool swiglu2, const EpiProgram& epi2, void* scratch, int sm_count) {
  if (!scratch || ((uintptr_t)scratch & 255)) return cudaErrorInvalidValue;
  cudaError_t e = plan_impl<2>(p1, a, w1_nk, y1, y1_f32, m, n1, k1, false, epi1, sm_count);
  if (e != cudaSuccess) return e;
  const int64_t num_n1 = (n1 + BN - 1) / BN;
  void* xg = scratch;
  float* part = reinterpret_cast<float*>(reinterpret_cast<char*>(scratch) + ((size_t)m * (size_t)n1 * 2 + 255) / 256 * 256);
  e = encode_tmap_2d_bf16_store(&p1->tm_aux, xg, (uint64_t)m, (uint64_t)n1, (uint64_t)n1);
  if (e != cudaSuccess) return e;
  p1->tail_first = (int)(((m + 2 * BM - 1) / (2 * BM)) * num_n1);   // whole tiles only: one partial-sum slot per (tile column, epilogue half)
  p1->res_ring = false;
  p1->use_pre = true;
  p1->pre.part_out = part;
  p1->pre.xg = xg;
  p1->pre.gamma = gamma;
  e = plan_impl<2>(p2, xg, w2_nk, y2, false, m, n2, n1, swiglu2, epi2, sm_count);
  if (e != cudaSuccess) return e;
  p2->tail_first = (int)(((m + 2 * BM - 1) / (2 * BM)) * ((n2 + (swiglu2 ? BN / 2 : BN) - 1) / (swiglu2 ? BN / 2 : BN)));
  p2->res_ring = false;
  p2->use_pre = true;
  p2->pre.part_in = part;
  p2->pre.slots_in = (int)(2 * num_n1);
  p2->pre.inv_n_in = 1.0f / (float)n1;
  p2->pre.eps_in = eps;
  return cudaSuccess;
}

cudaError_t gemm_tc_plan(GemmTcPlan* p, const void* a, const void* w_nk, void* y, bool out_f32, int64_t m, int64_t n, int64_t k, bool swiglu,
                         const EpiProgram& epi, int sm_count) {
  return plan_impl<1>(p, a, w_nk, y, out_f32, m, n, k, swiglu, epi, sm_count);
}
cudaError_t launch_gemm_tc(const GemmTcPlan& p, cudaStream_t s) { return launch_impl<1>(p, s); }
cudaError_t gemm_tc2_plan(GemmTcPlan* p, const void* a, const void* w_nk, void* y, bool out_f32, int64_t m, int64_t n, int64_t k, bool swiglu,
                          const EpiProgram& epi, int sm_count) {
  return plan_impl<2>(p, a, w_nk, y, out_f32, m, n, k, swiglu, epi, sm_count);
}
cudaError_t launch_gemm_tc2(const GemmTcPlan& p, cudaStream_t s) { return launch_impl<2>(p, s); }

}  // namespace mk
