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
//    Rows with w >= W are junk and never stored (W <= 62; 56 of 64 useful at W = 56).
//  * L2 -> SM traffic per tile and CTA is the patch alone; the kernel is bound by the tensor pipe.
//
// Warp roles as in the GEMM: warp 0 TMA producer, warp 1 TMEM allocation + (leader) MMA issue with a
// fully unrolled tap loop (a 256x128x16 MMA lasts 64 cycles, so the issuing thread may spend only a
// handful of instructions per MMA), warps 2..5 epilogue with a double-buffered accumulator and
// coalesced stores.  No TMA multicast.  Bounded waits.
#include "device_common.cuh"
#include "tc_common.cuh"
#include "tc_epilogue.cuh"
#include "tc_plans.h"

namespace mk {

namespace {

constexpr int PITCH = 64;                 // pixel pitch of the patch (>= W + 2)
constexpr int TILE_ROWS = 2;              // output rows per CTA
constexpr int PATCH_ROWS = TILE_ROWS + 2; // input rows per CTA incl. halo
constexpr int PATCH_BYTES = PATCH_ROWS * PITCH * 128;  // one 64-channel block: 32 KB
constexpr int A_STAGES = 2;
constexpr int THREADS = 192;

struct Shared {
  uint64_t a_full[A_STAGES];
  uint64_t a_empty[A_STAGES];
  uint64_t b_full;
  uint64_t tfull[2];
  uint64_t tempty[2];
  uint32_t tmem_base;
  int abort_flag;
};

// CB = C_in / 64 channel blocks
template <int CB>
__global__ void __launch_bounds__(THREADS, 1)
conv3x3_tc2_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW, __nv_bfloat16* __restrict__ y,
                   int NB, int H, int W, int C_OUT, const __grid_constant__ EpiProgram epi, unsigned int* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int b_rows = C_OUT / 2;                       // weight rows held by this CTA
  const int b_block_bytes = b_rows * 128;             // one 64-wide K block of them
  const int b_bytes = 9 * CB * b_block_bytes;
  uint8_t* a_tiles = base;                            // A_STAGES patches (+ 1 KB the last tap's junk rows may touch)
  uint8_t* b_tiles = base + A_STAGES * PATCH_BYTES + 1024;
  uint8_t* staging = b_tiles + b_bytes;
  Shared* sh = reinterpret_cast<Shared*>(staging + 4 * EPI_WARP_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = tc::cluster_ctarank();
  const bool leader = rank == 0;
  const int cluster_id = blockIdx.x >> 1, num_clusters = gridDim.x >> 1;
  const int quads = (H + 2 * TILE_ROWS - 1) / (2 * TILE_ROWS);   // pair-tiles per image
  const int total_tiles = NB * quads;
  volatile int* abort_flag = &sh->abort_flag;
  MK_TR_DECL
  MK_TR_INIT;

  if (threadIdx.x == 0) {
    for (int s = 0; s < A_STAGES; ++s) { tc::mbar_init(&sh->a_full[s], 1); tc::mbar_init(&sh->a_empty[s], 1); }
    tc::mbar_init(&sh->b_full, 1);
    for (int b = 0; b < 2; ++b) { tc::mbar_init(&sh->tfull[b], 1); tc::mbar_init(&sh->tempty[b], 8); }
    sh->abort_flag = 0;
    tc::fence_barrier_init();
    tc::tma_prefetch_desc(&tmX);
    tc::tma_prefetch_desc(&tmW);
  }
  if (warp == 1) tc::tmem_alloc_pair(&sh->tmem_base, 512);
  tc::tc_fence_before();
  __syncthreads();
  tc::cluster_sync();
  tc::tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------ producer
    if (lane == 0) {
      // weights: this CTA's C_out half, every K block, once
      const uint32_t bfull_leader = tc::map_to_cta(tc::smem_u32(&sh->b_full), 0);
      if (leader) tc::mbar_expect_tx(&sh->b_full, 2u * (uint32_t)b_bytes);
      for (int kb = 0; kb < 9 * CB; ++kb)
        tc::tma_load_2d_pair(b_tiles + (size_t)kb * b_block_bytes, &tmW, bfull_leader, kb * 64, (int)rank * b_rows);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int t = cluster_id; t < total_tiles && ok; t += num_clusters) {
        const int n = t / quads, hq = t - n * quads;
        const int h0 = hq * 2 * TILE_ROWS + (int)rank * TILE_ROWS;   // first output row of this CTA
        for (int cb = 0; cb < CB; ++cb) {
          ok = tc::mbar_wait(&sh->a_empty[stage], phase ^ 1, abort_flag, status, tc::WAIT_SMEM_EMPTY);
          if (!ok) break;
          const uint32_t full_leader = tc::map_to_cta(tc::smem_u32(&sh->a_full[stage]), 0);
          if (leader) tc::mbar_expect_tx(&sh->a_full[stage], 2 * PATCH_BYTES);
          tc::tma_load_4d_pair(a_tiles + (size_t)stage * PATCH_BYTES, &tmX, full_leader, cb * 64, -1, h0 - 1, n);
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
      bool ok = tc::mbar_wait(&sh->b_full, 0, abort_flag, status, tc::WAIT_SMEM_FULL);
      MK_TR(90);                                 // weights resident
      int it = 0;
      for (int t = cluster_id; t < total_tiles && ok; t += num_clusters, ++it) {
        const int acc = it & 1;
        const uint32_t d_tmem = tmem_base + acc * 256;
        ok = tc::mbar_wait(&sh->tempty[acc], ((it >> 1) & 1) ^ 1, abort_flag, status, tc::WAIT_TMEM_EMPTY);
        if (!ok) break;
        tc::tc_fence_after();
        uint32_t accumulate = 0;
#pragma unroll
        for (int cb = 0; cb < CB; ++cb) {
          ok = tc::mbar_wait(&sh->a_full[stage], phase, abort_flag, status, tc::WAIT_SMEM_FULL);
          if (!ok) break;
          tc::tc_fence_after();
          MK_TR(1 + it * 8 + cb);                // MMA: patch cb landed
          const uint32_t patch_lo = patch_lo0 + (uint32_t)stage * (PATCH_BYTES >> 4);
          uint32_t b_lo = b_lo0 + (uint32_t)cb * b_step;
#pragma unroll
          for (int tap = 0; tap < 9; ++tap) {
            const int kh = tap / 3, kw = tap % 3;                                   // compile-time after unrolling
            const uint32_t a_lo = patch_lo + (uint32_t)(((kh * PITCH + kw) * 128) >> 4);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              tc::umma_ss_pair_lohi(d_tmem, a_lo + 2 * k, b_lo + 2 * k, idesc, accumulate);
              accumulate = 1;
            }
            b_lo += (uint32_t)CB * b_step;
          }
          tc::umma_commit_pair(&sh->a_empty[stage]);
          if (++stage == A_STAGES) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        MK_TR(3 + it * 8);                       // MMA: tile issued
        tc::umma_commit_pair(&sh->tfull[acc]);
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ epilogue: 128 tile rows = 2 output rows x 64 pitch
    const int q = warp & 3;
    EpiWarp ew;
    ew.init(staging + q * EPI_WARP_BYTES, epi, lane, false);
    ew.load_bias(epi, 0, C_OUT, C_OUT);          // the bias slice is the same for every tile: once
    const int chunks = C_OUT / 32;
    bool ok = true;
    int it = 0;
    for (int t = cluster_id; t < total_tiles && ok; t += num_clusters, ++it) {
      const int n = t / quads, hq = t - n * quads;
      const int acc = it & 1;
      // warp q covers tile rows [32q, 32q + 32): output row hl = q / 2, pixels w0 .. w0 + 31
      const int hl = q >> 1, w0 = (q & 1) * 32;
      const int h = hq * 2 * TILE_ROWS + (int)rank * TILE_ROWS + hl;
      const int64_t pix0 = ((int64_t)n * H + h) * W;
      const bool row_ok = h < H;
      auto rowmap = [&](int r) -> int64_t { return (row_ok && w0 + r < W) ? pix0 + w0 + r : -1; };
      uint4 res_regs[8];
      ew.prefetch_res(epi, rowmap, 0, C_OUT, res_regs);
      ok = tc::mbar_wait(&sh->tfull[acc], (it >> 1) & 1, abort_flag, status, tc::WAIT_TMEM_FULL);
      ok = __all_sync(0xffffffffu, ok ? 1 : 0) != 0;
      if (!ok) break;
      if (threadIdx.x == 64) MK_TR(4 + it * 8);  // epilogue: accumulator ready
      tc::tc_fence_after();
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + acc * 256;
#pragma unroll 1
      for (int c = 0; c < chunks; ++c) {
        uint32_t rr[32];
        float v[32];
        tc::tmem_ld32(t_row + c * 32, rr);
        tc::tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(rr[j]);
        ew.chunk_out(epi, v, rowmap, y, (int64_t)c * 32, c * 32, (int64_t)C_OUT, res_regs, c + 1 < chunks ? (int64_t)(c + 1) * 32 : -1);
      }
      tc::tc_fence_before();
      __syncwarp();
      if (threadIdx.x == 64) MK_TR(5 + it * 8);  // epilogue: tile stored
      if (lane == 0) tc::mbar_arrive_cluster(tc::map_to_cta(tc::smem_u32(&sh->tempty[acc]), 0));
    }
  }

  MK_TR_PRINT("conv");
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
  return (size_t)A_STAGES * PATCH_BYTES + 1024 + (size_t)(c_out / 2) * 9 * c_in * 2 + 4 * EPI_WARP_BYTES + 1024 + 256;
}

}  // namespace

bool conv3x3_tc2_supported(int64_t nb, int64_t h, int64_t w, int64_t c_in, int64_t c_out) {
  if (nb < 1 || h < 1 || w < 1 || w > PITCH - 2) return false;
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
  p->y = y;
  p->nb = (int)nb; p->h = (int)h; p->w = (int)wd; p->c_in = (int)c_in; p->c_out = (int)c_out;
  p->epi = epi;
  const int64_t tiles = nb * ((h + 2 * TILE_ROWS - 1) / (2 * TILE_ROWS));
  const int64_t clusters = tiles < sm_count / 2 ? tiles : sm_count / 2;
  p->grid = (int)(2 * clusters);
  p->smem = conv_smem_bytes((int)c_in, (int)c_out);
  return cudaSuccess;
}

cudaError_t launch_conv3x3_tc2(const ConvTcPlan& p, cudaStream_t s) {
  static size_t attr_bytes = 0;   // largest dynamic shared-memory size opted into so far
  if (p.smem > attr_bytes) {
    cudaError_t e = cudaFuncSetAttribute(conv3x3_tc2_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(conv3x3_tc2_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem);
    if (e != cudaSuccess) return e;
    attr_bytes = p.smem;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)p.grid);
  cfg.blockDim = dim3(THREADS);
  cfg.dynamicSmemBytes = p.smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  unsigned int* status = kernel_status_ptr();
  __nv_bfloat16* y = (__nv_bfloat16*)p.y;
  if (p.c_in == 64) return cudaLaunchKernelEx(&cfg, conv3x3_tc2_kernel<1>, p.tm_x, p.tm_w, y, p.nb, p.h, p.w, p.c_out, p.epi, status);
  return cudaLaunchKernelEx(&cfg, conv3x3_tc2_kernel<2>, p.tm_x, p.tm_w, y, p.nb, p.h, p.w, p.c_out, p.epi, status);
}

}  // namespace mk
