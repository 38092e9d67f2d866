// K2: 3x3 convolution (stride 1, zero pad 1, NHWC, bf16) as an implicit GEMM on tcgen05, with the
// elementwise tail fused into the store.
//
//   Y[n,h,w,co] = tail( sum_{kh,kw,ci} Xpad[n, h+kh-1, w+kw-1, ci] * W[co,kh,kw,ci] )
//
// GEMM view: M = output pixels, N = C_out, K = 9 * C_in, K index = (kh*3 + kw) * C_in + ci, which is
// the weight tensor's own memory order.  Design, per CTA PAIR (cluster of 2, cta_group::2):
//
//  * Weights stay in shared memory for the whole kernel: each CTA holds its half of the C_out rows
//    for all of K ((C_out/2) * 9*C_in * 2 bytes, 144 KB for 128->128 channels), loaded once.
//  * The input is staged once per tile, not once per tap: a CTA's tile is 2 output rows, and ONE TMA
//    box {64 channels, 64 pixels, 4 rows} starting at (w = -1, h = h0 - 1) brings the 4 input rows
//    with their halo (out-of-range coordinates are zero-filled: that is the padding) into a patch of
//    256 rows x 128 bytes, pixel pitch 64.  Output pixel (hl, w) is tile row r = hl*64 + w, and the
//    A operand of tap (kh, kw) is the patch seen from row kh*64 + kw on: 128 consecutive rows.  A tap
//    is therefore just another shared-memory descriptor with a shifted start address (the 128-byte
//    swizzle follows absolute shared-memory address bits, so a row-shifted view stays consistent),
//    and the 9 taps x 4 MMAs of a channel block re-read the same 32 KB.
//    The last two rows of each 64, and rows with w >= W, are junk and never stored (56 of 64 useful at W = 56).  An
//    image row wider than 62 pixels is covered by several tiles of 62 pixels each (the box starts at w = 62 s - 1).
//  * L2 -> SM traffic per tile and CTA is the patch alone; the kernel is bound by the tensor pipe.
//
// Warp roles as in the GEMM: warp 0 TMA producer, warp 1 TMEM allocation + (leader) MMA issue with a
// fully unrolled tap loop (a 256x128x16 MMA lasts 64 cycles, so the issuing thread may spend only a
// handful of instructions per MMA), warps 2..9 epilogue (two per TMEM lane quarter) with a double-buffered
// accumulator, coalesced stores and, on request, the GroupNorm partial sums of the stored values.  No TMA multicast.  Bounded waits.
#include "device_common.cuh"
#include "tc_common.cuh"
#include "tc_epilogue.cuh"
#include "tc_plans.h"

namespace mk {

namespace {

constexpr int PITCH = 64;                 // pixel pitch of the patch
constexpr int SEG = PITCH - 2;            // output pixels of one image row a tile covers; wider rows take several tiles
constexpr int TILE_ROWS = 2;              // output rows per CTA
constexpr int PATCH_ROWS = TILE_ROWS + 2; // input rows per CTA incl. halo
constexpr int PATCH_BYTES = PATCH_ROWS * PITCH * 128;  // one 64-channel block: 32 KB
constexpr int A_STAGES = 2;
constexpr int EPI_WARPS = 8;              // two per TMEM lane quarter, each taking half of the channel chunks
constexpr int THREADS = 64 + 32 * EPI_WARPS;
constexpr int STG_BYTES = 32 * 64;        // transpose buffer per epilogue warp: 32 rows x 64 bytes, XOR-swizzled
constexpr int BIAS_BYTES = 512;           // one copy of the bias (C_out <= 256 bf16) per CTA

// The timeline of -DMK_TRACE builds lives in global memory here: this kernel leaves no shared memory for it.
#ifdef MK_TRACE
__device__ unsigned long long conv_tr[96];
__device__ long long conv_clk0;
#define CTR_INIT do { if (blockIdx.x == 0 && threadIdx.x == 0) { for (int i_ = 0; i_ < 96; ++i_) conv_tr[i_] = 0; conv_tr[0] = tc::gtime(); conv_clk0 = clock64(); } } while (0)
#define CTR(slot) do { if (blockIdx.x == 0 && (slot) < 96) conv_tr[slot] = tc::gtime(); } while (0)
#define CTR_PRINT do { __threadfence(); __syncthreads(); if (blockIdx.x == 0 && threadIdx.x == 0) { printf("conv end=%llu cycles=%lld :", tc::gtime() - conv_tr[0], clock64() - conv_clk0); \
    for (int i_ = 1; i_ < 96; ++i_) if (conv_tr[i_]) printf(" [%d]%llu", i_, conv_tr[i_] - conv_tr[0]); printf("\n"); } } while (0)
#else
#define CTR_INIT do {} while (0)
#define CTR(slot) do {} while (0)
#define CTR_PRINT do {} while (0)
#endif

struct Shared {
  uint64_t a_full[A_STAGES];
  uint64_t a_empty[A_STAGES];
  uint64_t b_full[2];      // weights of channel block 0 / 1 (the MMAs start when the first has landed)
  uint64_t tfull[4];
  uint64_t tempty[4];
  uint32_t tmem_base;
  int abort_flag;
  EpiProgram epi;   // the kernel parameter, copied once (see epi_copy_to_smem)
};

// Sum over the warp's 32 rows of N per-lane values, N a power of two: each step halves the number of
// values a lane carries (it keeps one half and receives the partner's other half), so N values cost N
// shuffles instead of 5 N.  On return lane L holds, in a[0], the total of value L >> (5 - log2 N)
// (every lane of that group of lanes holds the same total).
template <int N>
__device__ __forceinline__ void fold_rows(float* a, int lane, int m) {
  if constexpr (N > 1) {
    const bool up = (lane & m) != 0;
#pragma unroll
    for (int i = 0; i < N / 2; ++i) {
      const float send = up ? a[i] : a[i + N / 2];
      const float keep = up ? a[i + N / 2] : a[i];
      a[i] = keep + __shfl_xor_sync(0xffffffffu, send, m);
    }
    fold_rows<N / 2>(a, lane, m >> 1);
  } else {
    for (; m >= 1; m >>= 1) a[0] += __shfl_xor_sync(0xffffffffu, a[0], m);
  }
}
// GroupNorm partial sums of one 32-channel chunk over the warp's 32 pixels: groups of CPG adjacent
// channels; dst = float[32 / CPG][2] = (sum, sum of squares) per group.  Rows that are not stored count 0.
template <int CPG>
__device__ __forceinline__ void chunk_stats(const float (&v)[32], bool valid, int lane, float* __restrict__ dst) {
  constexpr int GPC = 32 / CPG, NV = 2 * GPC;
  float a[NV];
#pragma unroll
  for (int g = 0; g < GPC; ++g) {
    float sm = 0.0f, sq = 0.0f;
#pragma unroll
    for (int e = 0; e < CPG; ++e) {
      const float x = valid ? v[g * CPG + e] : 0.0f;
      sm += x;
      sq = fmaf(x, x, sq);
    }
    a[2 * g] = sm;
    a[2 * g + 1] = sq;
  }
  fold_rows<NV>(a, lane, 16);
  constexpr int LOG = NV == 32 ? 5 : NV == 16 ? 4 : NV == 8 ? 3 : NV == 4 ? 2 : 1;
  if ((lane & ((1 << (5 - LOG)) - 1)) == 0) dst[lane >> (5 - LOG)] = a[0];
}

// Four MMAs of one tap (K = 64 channels in steps of 16): the two descriptors advance by 32 bytes (2 in
// the address field) per step, done on the low words inside the block, so the issuing thread spends three
// instructions per 64-cycle MMA.  acc0 = 0 makes the first MMA overwrite the accumulator.
__device__ __forceinline__ void umma_ss_pair_x4(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc0) {
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t.reg .b32 alo, ahi, blo, bhi;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "setp.eq.b32 q, %3, %3;\n\t"
      "mov.b64 {alo, ahi}, %1;\n\t"
      "mov.b64 {blo, bhi}, %2;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t"
      "add.u32 alo, alo, 2;\n\tadd.u32 blo, blo, 2;\n\tmov.b64 da, {alo, ahi};\n\tmov.b64 db, {blo, bhi};\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, q;\n\t"
      "add.u32 alo, alo, 2;\n\tadd.u32 blo, blo, 2;\n\tmov.b64 da, {alo, ahi};\n\tmov.b64 db, {blo, bhi};\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, q;\n\t"
      "add.u32 alo, alo, 2;\n\tadd.u32 blo, blo, 2;\n\tmov.b64 da, {alo, ahi};\n\tmov.b64 db, {blo, bhi};\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, q;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc0)
      : "memory");
}


// CB = C_in / 64 channel blocks; WIDE: image rows of more than SEG pixels (several tiles per row)
template <int CB, bool WIDE>
__global__ void __launch_bounds__(THREADS, 1)
conv3x3_tc2_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmY,
                   const __grid_constant__ CUtensorMap tmY30,
                   int NB, int H, int W, int C_OUT, const __grid_constant__ EpiProgram epi_param, float* __restrict__ stats, int cpg,
                   unsigned int* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int b_rows = C_OUT / 2;                       // weight rows held by this CTA
  const int b_block_bytes = b_rows * 128;             // one 64-wide K block of them
  const int b_bytes = 9 * CB * b_block_bytes;
  uint8_t* a_tiles = base;                            // A_STAGES patches (+ 1 KB the last tap's junk rows may touch)
  uint8_t* b_tiles = base + A_STAGES * PATCH_BYTES + 1024;
  uint8_t* staging = b_tiles + b_bytes;
  Shared* sh = reinterpret_cast<Shared*>(staging + EPI_WARPS * STG_BYTES + BIAS_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = tc::cluster_ctarank();
  const bool leader = rank == 0;
  const int cluster_id = blockIdx.x >> 1, num_clusters = gridDim.x >> 1;
  const int quads = (H + 2 * TILE_ROWS - 1) / (2 * TILE_ROWS);   // row groups (four output rows per CTA pair) per image
  const int nseg = WIDE ? (W + SEG - 1) / SEG : 1;               // SEG-pixel segments per image row
  const int total_tiles = NB * quads * nseg;                     // tile t = ((n * quads + hq) * nseg + sg)
  volatile int* abort_flag = &sh->abort_flag;
  CTR_INIT;
  static_assert(sizeof(Shared) <= 512, "barrier block");
  epi_copy_to_smem(&sh->epi, epi_param, threadIdx.x, THREADS);
  const EpiProgram& epi = sh->epi;

  if (threadIdx.x == 0) {
    for (int s = 0; s < A_STAGES; ++s) { tc::mbar_init(&sh->a_full[s], 1); tc::mbar_init(&sh->a_empty[s], 1); }
    tc::mbar_init(&sh->b_full[0], 1);
    tc::mbar_init(&sh->b_full[1], 1);
    for (int b = 0; b < 4; ++b) { tc::mbar_init(&sh->tfull[b], 1); tc::mbar_init(&sh->tempty[b], 2 * EPI_WARPS); }
    sh->abort_flag = 0;
    tc::fence_barrier_init();
    tc::tma_prefetch_desc(&tmX);
    tc::tma_prefetch_desc(&tmW);
    tc::tma_prefetch_desc(&tmY);
    if (nseg > 1) tc::tma_prefetch_desc(&tmY30);
  }
  if (warp == 1) tc::tmem_alloc_pair(&sh->tmem_base, 512);
  tc::tc_fence_before();
  __syncthreads();
  tc::cluster_sync();
  tc::tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;
  // Accumulators: the 512 TMEM columns as four buffers of 128 when C_out <= 128, else two of 256.  With four, the
  // MMAs of tile i + 2 never wait for the epilogue of tile i (the barrier's round trip through both CTAs' sixteen
  // epilogue warps was 0.2 us per tile with two).
  const int nacc = C_OUT <= 128 ? 4 : 2, acc_shift = C_OUT <= 128 ? 2 : 1;
  const uint32_t acc_cols = 512u / (uint32_t)nacc;
  // Weights: this CTA's C_out half, every K block, once; channel block by channel block, in the order the MMAs
  // consume them (K block index = tap * CB + cb).  They are parameters, not the output of the kernel before this
  // one on the stream, so their load is issued BEFORE the wait for that kernel: as a programmatic dependent this
  // CTA is resident while its predecessor drains, and the 2 x 144 KB land meanwhile (measured: C3 41.0 -> 40.2 us).
  // Measured and not kept: a barrier per kernel row instead of per channel block, so that the first MMAs could
  // start on a third of the weights (the waits between MMA groups cost more than the earlier start: +0.9 us), and
  // the last wave's four tiles run as eight units of half the output channels (+0.3 us: the slowest of eight
  // pairs ends later than the slowest of four, and a 256 x 64 MMA reads as many patch bytes as a 256 x 128 one).
  if (warp == 0 && lane == 0) {
    for (int cb = 0; cb < CB; ++cb) {
      const uint32_t bfull_leader = tc::map_to_cta(tc::smem_u32(&sh->b_full[cb]), 0);
      if (leader) tc::mbar_expect_tx(&sh->b_full[cb], 2u * 9u * (uint32_t)b_block_bytes);
      for (int tap = 0; tap < 9; ++tap) {
        const int kb = tap * CB + cb;
        tc::tma_load_2d_pair(b_tiles + (size_t)kb * b_block_bytes, &tmW, bfull_leader, kb * 64, (int)rank * b_rows);
      }
    }
  }
  pdl_launch_dependents();
  pdl_wait();   // X may come from the kernel before this one

  if (warp == 0) {
    // ------------------------------------------------------------ producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int t = cluster_id; t < total_tiles && ok; t += num_clusters) {
        const int sg = nseg == 1 ? 0 : t % nseg, nq = nseg == 1 ? t : t / nseg;
        const int n = nq / quads, hq = nq - n * quads;
        const int h0 = hq * 2 * TILE_ROWS + (int)rank * TILE_ROWS;   // first output row of this CTA
        // No L2 prefetch of the next tile's patches: with one issued here, a whole tile early, the step measured
        // 39.9 us against 39.4 us without (32 x 56 x 56 x 128, inputs rotated through more than L2).
        for (int cb = 0; cb < CB; ++cb) {
          ok = tc::mbar_wait(&sh->a_empty[stage], phase ^ 1, abort_flag, status, tc::WAIT_SMEM_EMPTY);
          if (!ok) break;
          const uint32_t full_leader = tc::map_to_cta(tc::smem_u32(&sh->a_full[stage]), 0);
          if (leader) tc::mbar_expect_tx(&sh->a_full[stage], 2 * PATCH_BYTES);
          tc::tma_load_4d_pair(a_tiles + (size_t)stage * PATCH_BYTES, &tmX, full_leader, cb * 64, sg * SEG - 1, h0 - 1, n);
          if (++stage == A_STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (one lane of the leader)
    if (leader && lane == 0) {
      const uint32_t idesc = tc::idesc_bf16_f32(256, C_OUT, 0, 0);
      const uint32_t patch_lo0 = tc::desc_lo_sw128(tc::smem_u32(a_tiles));
      const uint32_t b_lo0 = tc::desc_lo_sw128(tc::smem_u32(b_tiles));
      const uint32_t b_step = (uint32_t)b_block_bytes >> 4;
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int it = 0;
      for (int t = cluster_id; t < total_tiles && ok; t += num_clusters, ++it) {
        const int acc = it & (nacc - 1);
        const uint32_t d_tmem = tmem_base + acc * acc_cols;
        ok = tc::mbar_wait(&sh->tempty[acc], ((it >> acc_shift) & 1) ^ 1, abort_flag, status, tc::WAIT_TMEM_EMPTY);
        if (!ok) break;
        tc::tc_fence_after();
        if (it > 0) CTR(it * 8);               // MMA: accumulator free
        uint32_t accumulate = 0;
#pragma unroll
        for (int cb = 0; cb < CB; ++cb) {
          if (it == 0) {
            ok = tc::mbar_wait(&sh->b_full[cb], 0, abort_flag, status, tc::WAIT_SMEM_FULL);
            if (!ok) break;
          }
          ok = tc::mbar_wait(&sh->a_full[stage], phase, abort_flag, status, tc::WAIT_SMEM_FULL);
          if (!ok) break;
          tc::tc_fence_after();
          CTR(1 + it * 8 + cb);                // MMA: patch cb landed
          const uint64_t patch_desc = ((uint64_t)tc::kDescHiSw128 << 32) | (patch_lo0 + (uint32_t)stage * (PATCH_BYTES >> 4));
          uint64_t b_desc = ((uint64_t)tc::kDescHiSw128 << 32) | (b_lo0 + (uint32_t)cb * b_step);
          // fully unrolled on purpose: as a compact loop (nine iterations, the offsets advanced at run time) the
          // kernel is 3 us slower, the extra instructions between two MMAs being time the tensor pipe waits
#pragma unroll
          for (int tap = 0; tap < 9; ++tap) {
            const int kh = tap / 3, kw = tap % 3;                                   // compile-time after unrolling
            umma_ss_pair_x4(d_tmem, patch_desc + (uint64_t)(((kh * PITCH + kw) * 128) >> 4), b_desc, idesc, accumulate);
            accumulate = 1;
            b_desc += (uint64_t)((uint32_t)CB * b_step);
          }
          CTR(6 + it * 8 + cb);                  // MMA: channel block issued
          tc::umma_commit_pair(&sh->a_empty[stage]);
          if (++stage == A_STAGES) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        CTR(3 + it * 8);                       // MMA: tile issued
        tc::umma_commit_pair(&sh->tfull[acc]);
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ epilogue: 128 tile rows = 2 output rows x 64 pitch
    // Warps w and w + 4 share TMEM lane quarter q (tile rows [32q, 32q + 32)) and split its channel chunks.
    const int ew = warp - 2, q = warp & 3, half = ew >> 2;
    uint8_t* stg = staging + ew * STG_BYTES;
    uint8_t* bias_sh = staging + EPI_WARPS * STG_BYTES;
    const int bias_idx = epi_single_index(epi, EPI_BIAS);
    if (bias_idx >= 0) {
      // the bias slice is the same for every tile: one copy per CTA, once
      for (int i = (int)threadIdx.x - 64; i < C_OUT / 8; i += 32 * EPI_WARPS)
        reinterpret_cast<uint4*>(bias_sh)[i] = reinterpret_cast<const uint4*>(epi.op[bias_idx].ptr)[i];
    }
    asm volatile("bar.sync 1, %0;" ::"n"(32 * EPI_WARPS) : "memory");
    const int chunks = C_OUT / 32, c_mid = (chunks + 1) / 2;
    const int c_lo = half ? c_mid : 0, c_hi = half ? chunks : c_mid;
    const int groups = stats ? C_OUT / cpg : 0;
    const int stat_slots = quads * nseg * 2 * 4;   // partial sums per image: one per (pair-tile, CTA, lane quarter)
    const uint4 no_res[4] = {};
    bool ok = true;
    int it = 0;
    for (int t = cluster_id; t < total_tiles && ok; t += num_clusters, ++it) {
      const int sg = nseg == 1 ? 0 : t % nseg, nq = nseg == 1 ? t : t / nseg;
      const int n = nq / quads, hq = nq - n * quads;
      const int acc = it & (nacc - 1);
      // warp q covers tile rows [32q, 32q + 32): output row hl = q / 2, pixels w0 .. w0 + 31 of the image row, of
      // which those inside the segment (the first SEG of the tile row's 64) and inside the image are real
      const int hl = q >> 1, w0 = sg * SEG + (q & 1) * 32;
      const int w_end = (sg + 1) * SEG < W ? (sg + 1) * SEG : W;
      const int h = hq * 2 * TILE_ROWS + (int)rank * TILE_ROWS + hl;
      const int64_t pix0 = ((int64_t)n * H + h) * W;
      const bool row_ok = h < H;
      auto rowmap = [&](int r) -> int64_t { return (row_ok && w0 + r < w_end) ? pix0 + w0 + r : -1; };
      const int64_t my_row = rowmap(lane);
      ok = tc::mbar_wait(&sh->tfull[acc], (it >> acc_shift) & 1, abort_flag, status, tc::WAIT_TMEM_FULL);
      ok = __all_sync(0xffffffffu, ok ? 1 : 0) != 0;
      if (!ok) break;
      if (threadIdx.x == 64) CTR(4 + it * 8);  // epilogue: accumulator ready
      tc::tc_fence_after();
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + acc * acc_cols;
      float* stat_dst = stats ? stats + (((int64_t)n * stat_slots + ((hq * nseg + sg) * 2 + (int)rank) * 4 + q) * groups) * 2 : nullptr;
#pragma unroll 1
      for (int c = c_lo; c < c_hi; ++c) {
        uint32_t rr[32];
        float v[32];
        tc::tmem_ld32(t_row + c * 32, rr);
        tc::tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(rr[j]);
        if (my_row >= 0) epi32(epi, v, my_row, (int64_t)c * 32, (int64_t)C_OUT, bias_idx >= 0 ? bias_sh + c * 64 : nullptr, 0, no_res, no_res);
        if (stats) {
          float* d = stat_dst + (c * 32 / cpg) * 2;
          switch (cpg) {
            case 2: chunk_stats<2>(v, my_row >= 0, lane, d); break;
            case 4: chunk_stats<4>(v, my_row >= 0, lane, d); break;
            case 8: chunk_stats<8>(v, my_row >= 0, lane, d); break;
            case 16: chunk_stats<16>(v, my_row >= 0, lane, d); break;
            default: chunk_stats<32>(v, my_row >= 0, lane, d); break;
          }
        }
        uint4 mine[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          mine[k].x = pack_bf16x2(v[8 * k + 0], v[8 * k + 1]);
          mine[k].y = pack_bf16x2(v[8 * k + 2], v[8 * k + 3]);
          mine[k].z = pack_bf16x2(v[8 * k + 4], v[8 * k + 5]);
          mine[k].w = pack_bf16x2(v[8 * k + 6], v[8 * k + 7]);
        }
        // the lane's own 64 bytes into the staging buffer (64-byte swizzle), then one bulk tensor store of the
        // 32 pixels x 32 channels; pixels past the end of the image row are clipped by the copy engine
        if (lane == 0) tc::tma_store_wait_read();   // the previous chunk's store has finished reading the buffer
        __syncwarp();
        {
          const int f = (lane >> 1) & 3;
#pragma unroll
          for (int sgm = 0; sgm < 4; ++sgm) *reinterpret_cast<uint4*>(stg + lane * 64 + ((sgm ^ f) * 16)) = mine[sgm];
        }
        tc::fence_proxy_async();
        __syncwarp();
        // the second half of a tile row holds 30 pixels of the segment: where the image row goes on behind it, its box
        // is 30 pixels long, so that the two junk rows are not written over the next segment's first pixels
        if (lane == 0 && row_ok && w0 < W) {
          tc::tma_store_4d((nseg > 1 && (q & 1)) ? &tmY30 : &tmY, stg, c * 32, w0, h, n);
          tc::tma_store_commit();
        }
      }
      tc::tc_fence_before();
      __syncwarp();
      if (threadIdx.x == 64) CTR(5 + it * 8);  // epilogue: tile stored
      // (a relaxed arrival: the warp's reads of tensor memory are over, nothing has to be published)
      if (lane == 0) tc::mbar_arrive_cluster_relaxed(tc::map_to_cta(tc::smem_u32(&sh->tempty[acc]), 0));
    }
  }

  if (warp >= 2 && lane == 0) tc::tma_store_wait_all();   // this warp's bulk stores are complete before the CTA retires
  CTR_PRINT;
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

size_t conv_smem_bytes(int c_in, int c_out) {
  return (size_t)A_STAGES * PATCH_BYTES + 1024 + (size_t)(c_out / 2) * 9 * c_in * 2 + EPI_WARPS * STG_BYTES + BIAS_BYTES + 1024 + 512;
}

}  // namespace

int conv3x3_tc2_stat_slots(int64_t h, int64_t w) {
  return (int)(((h + 2 * TILE_ROWS - 1) / (2 * TILE_ROWS)) * ((w + SEG - 1) / SEG)) * 2 * 4;
}

bool conv3x3_tc2_supported(int64_t nb, int64_t h, int64_t w, int64_t c_in, int64_t c_out) {
  if (nb < 1 || h < 1 || w < 1) return false;
  if (nb * ((h + 2 * TILE_ROWS - 1) / (2 * TILE_ROWS)) * ((w + SEG - 1) / SEG) > INT32_MAX) return false;
  if (c_in != 64 && c_in != 128) return false;
  if (c_out < 32 || c_out > 256 || c_out % 32) return false;
  return conv_smem_bytes((int)c_in, (int)c_out) <= 227 * 1024;
}

cudaError_t conv3x3_tc2_plan(ConvTcPlan* p, const void* x, const void* w, void* y, int64_t nb, int64_t h, int64_t wd, int64_t c_in,
                             int64_t c_out, const EpiProgram& epi, int sm_count) {
  if (!conv3x3_tc2_supported(nb, h, wd, c_in, c_out)) return cudaErrorInvalidValue;
  {
    const uint64_t dims[4] = {(uint64_t)c_in, (uint64_t)wd, (uint64_t)h, (uint64_t)nb};
    const uint64_t strides[3] = {(uint64_t)c_in * 2, (uint64_t)wd * c_in * 2, (uint64_t)h * wd * c_in * 2};
    const uint32_t box[4] = {64, PITCH, PATCH_ROWS, 1};
    cudaError_t e = encode_tmap_bf16(&p->tm_x, x, 4, dims, strides, box, true);
    if (e != cudaSuccess) return e;
  }
  cudaError_t e = encode_tmap_2d_bf16(&p->tm_w, w, (uint64_t)c_out, (uint64_t)(9 * c_in), (uint64_t)(9 * c_in), (uint32_t)(c_out / 2), 64);
  if (e != cudaSuccess) return e;
  e = encode_tmap_nhwc_bf16_store(&p->tm_y, y, (uint64_t)nb, (uint64_t)h, (uint64_t)wd, (uint64_t)c_out, 32);
  if (e != cudaSuccess) return e;
  e = encode_tmap_nhwc_bf16_store(&p->tm_y30, y, (uint64_t)nb, (uint64_t)h, (uint64_t)wd, (uint64_t)c_out, 30);
  if (e != cudaSuccess) return e;
  p->y = y;
  p->stats = nullptr;
  p->cpg = 0;
  p->nb = (int)nb; p->h = (int)h; p->w = (int)wd; p->c_in = (int)c_in; p->c_out = (int)c_out;
  p->epi = epi;
  const int64_t tiles = nb * ((h + 2 * TILE_ROWS - 1) / (2 * TILE_ROWS)) * ((wd + SEG - 1) / SEG);
  const int64_t clusters = tiles < sm_count / 2 ? tiles : sm_count / 2;
  p->grid = (int)(2 * clusters);
  p->smem = conv_smem_bytes((int)c_in, (int)c_out);
  return cudaSuccess;
}

cudaError_t launch_conv3x3_tc2(const ConvTcPlan& p, cudaStream_t s) {
  static SmemOptIn opt_in;
  {
    cudaError_t e = opt_in.ensure(p.smem, conv3x3_tc2_kernel<1, false>, conv3x3_tc2_kernel<2, false>, conv3x3_tc2_kernel<1, true>,
                                  conv3x3_tc2_kernel<2, true>);
    if (e != cudaSuccess) return e;
  }
  LaunchCfg lc(PDL_CONV, dim3((unsigned)p.grid), dim3(THREADS), p.smem, s, 2);
  cudaLaunchConfig_t& cfg = lc.cfg;
  unsigned int* status = kernel_status_ptr();
  const bool wide = p.w > SEG;
#define MK_CONV_LAUNCH(CB_, WIDE_)                                                                                                          \
  return cudaLaunchKernelEx(&cfg, conv3x3_tc2_kernel<CB_, WIDE_>, p.tm_x, p.tm_w, p.tm_y, p.tm_y30, p.nb, p.h, p.w, p.c_out, p.epi, p.stats, \
                            p.cpg, status)
  if (p.c_in == 64) {
    if (wide) MK_CONV_LAUNCH(1, true);
    MK_CONV_LAUNCH(1, false);
  }
  if (wide) MK_CONV_LAUNCH(2, true);
  MK_CONV_LAUNCH(2, false);
#undef MK_CONV_LAUNCH
}

}  // namespace mk
