// K7: fused causal attention on tcgen05 / TMEM, head_dim 128, bf16 in, fp32 softmax and accumulation.
//
//   O = softmax(mask_{j<=i}(Q K^T / sqrt(D))) V        online softmax, the S x S matrix never leaves the SM
//
// One CTA = one (batch, head, 128-query tile); it walks the key tiles 0..diagonal (128 keys each).
//   warp 0      TMA: Q once; K and V tiles through separate 2-stage rings (128-byte swizzle)
//   warp 1      TMEM allocation; one lane issues   S_j = Q K_j^T   (SS form, 128x128x16 x 8)
//                                           and   O_j = P_j V_j   (TS form: P is read from TMEM,
//                                                                   V from shared memory, MN-major)
//   warps 2..9  two threads per query row, each owning half of the row's columns: two passes over S_j in TMEM (row max; then
//               p = exp2(s * scale*log2e - m), row sum), P_j written back into TMEM as packed bf16
//               OVER the columns of S_j that are already consumed; then O_{j-1} is read from TMEM and
//               folded into a register accumulator  o = o * alpha + O_{j-1}  (alpha = exp2(m_old - m_new)).
//               Keeping the running O in registers means no rescale round trip through TMEM.
// TMEM (512 columns): S/P double buffer (2 x 128) + O_j double buffer (2 x 128), so S_{j+1} is being
// computed while the softmax of tile j runs, and P_j V_j runs while the softmax of tile j+1 runs.
// The diagonal tile is masked (key > query -> -inf, diagonal kept); tiles left of it need no mask;
// tiles right of it are never visited.  CTAs are ordered head by head (L2 reuse of K/V), heavy query
// tiles first within a head.
// Output rows go through the shared-memory transpose of the common epilogue (coalesced stores) to the
// [B*S, H*D] matrix.  Every mbarrier wait is bounded.
#include "device_common.cuh"
#include "tc_common.cuh"
#include "tc_epilogue.cuh"
#include "tc_plans.h"

namespace mk {

namespace {

constexpr int BQ = 128, BKV = 128;
constexpr int SUB_BYTES = 128 * 64 * 2;    // a 128 x 64 sub-tile (one 128-byte swizzle row per query / key): 16 KB
// a Q / K / V tile: 128 rows x head_dim = one sub-tile (head_dim 64) or two (head_dim 128)
constexpr int tile_bytes(int hd) { return 128 * hd * 2; }
constexpr int KV_STAGES = 2;
constexpr int SOFTMAX_WARPS = 8;
constexpr int THREADS = 64 + 32 * SOFTMAX_WARPS;
constexpr size_t attn_smem(int hd) { return (size_t)tile_bytes(hd) * (1 + 2 * KV_STAGES) + SOFTMAX_WARPS * EPI_WARP_BYTES + 1024 + 256 + 2048; }

struct Shared {
  uint64_t q_full;
  uint64_t k_full[KV_STAGES], k_empty[KV_STAGES];
  uint64_t v_full[KV_STAGES], v_empty[KV_STAGES];
  uint64_t s_full[2], p_ready[2], o_full[2], o_free[2];
  uint32_t tmem_base;
  int abort_flag;
  float xch[2][128][2];   // row maximum / row sum exchange between the two threads of a row
};

// D[tmem] (+)= A[tmem] * B[smem], descriptor given as low word + constant high word
__device__ __forceinline__ void umma_ts_lohi(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]),
      "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}

// HD: head dimension, 64 or 128.  causal != 0: query i sees keys 0..i; else every key (the last key tile may be
// ragged: keys past S are hidden the way the diagonal hides them, with one limit for every row).
template <int HD>
__global__ void __launch_bounds__(THREADS, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                    __nv_bfloat16* __restrict__ out, int B, int H, int S, int causal, float scale_log2, unsigned int* status) {
  static_assert(HD == 64 || HD == 128, "head dimension");
  constexpr int TILE_BYTES = tile_bytes(HD);
  constexpr int OC = HD / 64;                    // 32-column chunks of O per softmax thread (it owns HD / 2 columns)
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* q_tile = base;
  uint8_t* k_tiles = base + TILE_BYTES;
  uint8_t* v_tiles = k_tiles + KV_STAGES * TILE_BYTES;
  uint8_t* staging = v_tiles + KV_STAGES * TILE_BYTES;
  Shared* sh = reinterpret_cast<Shared*>(staging + SOFTMAX_WARPS * EPI_WARP_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_q = (S + BQ - 1) / BQ;
  // consecutive CTAs = the query tiles of ONE (batch, head), heaviest first: the CTAs resident at any
  // time then share a handful of K/V tensors, which stay in L2, instead of each streaming its own
  // head's K/V from HBM
  const int bh = blockIdx.x / num_q;
  const int qt = num_q - 1 - blockIdx.x % num_q;
  const int b = bh / H, h = bh - b * H;
  const int T = causal ? qt + 1 : num_q;              // key tiles 0 .. diagonal, or all of them
  volatile int* abort_flag = &sh->abort_flag;
  MK_TR_DECL
  MK_TR_INIT;

  if (threadIdx.x == 0) {
    tc::mbar_init(&sh->q_full, 1);
    for (int s = 0; s < KV_STAGES; ++s) {
      tc::mbar_init(&sh->k_full[s], 1); tc::mbar_init(&sh->k_empty[s], 1);
      tc::mbar_init(&sh->v_full[s], 1); tc::mbar_init(&sh->v_empty[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      tc::mbar_init(&sh->s_full[i], 1); tc::mbar_init(&sh->p_ready[i], 32 * SOFTMAX_WARPS);
      tc::mbar_init(&sh->o_full[i], 1); tc::mbar_init(&sh->o_free[i], 32 * SOFTMAX_WARPS);
    }
    sh->abort_flag = 0;
    tc::fence_barrier_init();
    tc::tma_prefetch_desc(&tmQ);
    tc::tma_prefetch_desc(&tmK);
    tc::tma_prefetch_desc(&tmV);
  }
  if (warp == 1) { tc::tmem_alloc(&sh->tmem_base, 512); tc::tmem_relinquish(); }
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;
  const uint32_t tmem_s = tmem_base;            // S/P buffers: columns [0,128) and [128,256)
  const uint32_t tmem_o = tmem_base + 256;      // O_j buffers: columns [256,384) and [384,512)

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tc::mbar_expect_tx(&sh->q_full, TILE_BYTES);
      tc::tma_load_4d(q_tile, &tmQ, &sh->q_full, 0, qt * BQ, h, b);
      if (HD == 128) tc::tma_load_4d(q_tile + SUB_BYTES, &tmQ, &sh->q_full, 64, qt * BQ, h, b);
      bool ok = true;
      auto load_k = [&](int j) {
        const int st = j % KV_STAGES;
        ok = tc::mbar_wait(&sh->k_empty[st], ((j / KV_STAGES) & 1) ^ 1, abort_flag, status, tc::WAIT_SMEM_EMPTY);
        if (!ok) return;
        uint8_t* kd = k_tiles + (size_t)st * TILE_BYTES;
        tc::mbar_expect_tx(&sh->k_full[st], TILE_BYTES);
        tc::tma_load_4d(kd, &tmK, &sh->k_full[st], 0, j * BKV, h, b);
        if (HD == 128) tc::tma_load_4d(kd + SUB_BYTES, &tmK, &sh->k_full[st], 64, j * BKV, h, b);
      };
      auto load_v = [&](int j) {
        const int st = j % KV_STAGES;
        ok = tc::mbar_wait(&sh->v_empty[st], ((j / KV_STAGES) & 1) ^ 1, abort_flag, status, tc::WAIT_SMEM_EMPTY);
        if (!ok) return;
        uint8_t* vd = v_tiles + (size_t)st * TILE_BYTES;
        tc::mbar_expect_tx(&sh->v_full[st], TILE_BYTES);
        tc::tma_load_4d(vd, &tmV, &sh->v_full[st], 0, j * BKV, h, b);
        if (HD == 128) tc::tma_load_4d(vd + SUB_BYTES, &tmV, &sh->v_full[st], 64, j * BKV, h, b);
      };
      // Loads are issued in the order their ring slots come free, which is the order the MMAs retire:
      // QK(0) QK(1) PV(0) QK(2) PV(1) QK(3) ...  (a K load queued behind a V slot that frees later would
      // stall the next Q K^T)
      load_k(0);
      if (ok && T > 1) load_k(1);
      for (int j = 0; j < T && ok; ++j) {
        load_v(j);
        if (ok && j + 2 < T) load_k(j + 2);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_qk = tc::idesc_bf16_f32(BQ, BKV, 0, 0);   // A, B K-major
      constexpr uint32_t idesc_pv = tc::idesc_bf16_f32(BQ, HD, 0, 1);    // B (= V) MN-major
      // V, MN-major with 128-byte swizzle: 64 head-dim elements are contiguous (one 128-byte row per
      // key), 8-key groups are 1024 B apart (SBO), the second 64 head-dim elements sit SUB_BYTES on (LBO)
      constexpr uint32_t v_hi = ((1024u >> 4) & 0x3FFF) | (1u << 14) | (2u << 29);
      const uint32_t q_lo = tc::desc_lo_sw128(tc::smem_u32(q_tile));
      const uint32_t k_lo0 = tc::desc_lo_sw128(tc::smem_u32(k_tiles));
      const uint32_t v_lo0 = ((tc::smem_u32(v_tiles) & 0x3FFFF) >> 4) | ((uint32_t)(SUB_BYTES >> 4) << 16);
      bool ok = tc::mbar_wait(&sh->q_full, 0, abort_flag, status, tc::WAIT_SMEM_FULL);
      auto issue_qk = [&](int j) {
        const int st = j % KV_STAGES;
        ok = tc::mbar_wait(&sh->k_full[st], (j / KV_STAGES) & 1, abort_flag, status, tc::WAIT_SMEM_FULL);
        if (!ok) return;
        tc::tc_fence_after();
        const uint32_t k_lo = k_lo0 + (uint32_t)st * (TILE_BYTES >> 4);
        const uint32_t d = tmem_s + (j & 1) * 128;
#pragma unroll
        for (int k = 0; k < HD / 16; ++k) {
          const uint32_t off = (uint32_t)((k >> 2) * (SUB_BYTES >> 4) + (k & 3) * 2);
          tc::umma_ss_lohi(d, q_lo + off, k_lo + off, idesc_qk, k > 0 ? 1u : 0u);
        }
        tc::umma_commit(&sh->k_empty[st]);
        tc::umma_commit(&sh->s_full[j & 1]);
      };
      if (ok) issue_qk(0);
      for (int j = 0; j < T && ok; ++j) {
        if (j + 1 < T) issue_qk(j + 1);
        if (!ok) break;
        const int st = j % KV_STAGES, buf = j & 1;
        const uint32_t use = (j >> 1) & 1;
        if (j < 11) MK_TR(6 + j * 8);                        // QK(j+1) issued, now waiting for P_j
        ok = tc::mbar_wait(&sh->p_ready[buf], use, abort_flag, status, tc::WAIT_ATTN);
        if (j < 11) MK_TR(7 + j * 8);                        // P_j seen
        if (ok) ok = tc::mbar_wait(&sh->v_full[st], (j / KV_STAGES) & 1, abort_flag, status, tc::WAIT_SMEM_FULL);
        if (j < 10) MK_TR(8 + j * 8);                        // V_j seen
        if (ok) ok = tc::mbar_wait(&sh->o_free[buf], use ^ 1, abort_flag, status, tc::WAIT_TMEM_EMPTY);
        if (!ok) break;
        tc::tc_fence_after();
        const uint32_t v_lo = v_lo0 + (uint32_t)st * (TILE_BYTES >> 4);
        // P_j: packed bf16, 16 keys = 8 columns; keys 0..63 sit in columns [0,32) of the S/P buffer, keys
        // 64..127 in columns [64,96) (each softmax thread overwrites only S columns it has consumed itself)
        const uint32_t p_tmem = tmem_s + buf * 128;
        const uint32_t d = tmem_o + buf * 128;
#pragma unroll
        for (int k = 0; k < BKV / 16; ++k)
          umma_ts_lohi(d, p_tmem + (k < 4 ? k * 8 : 64 + (k - 4) * 8), v_lo + (uint32_t)(k * ((16 * 128) >> 4)), v_hi, idesc_pv, k > 0 ? 1u : 0u);
        tc::umma_commit(&sh->v_empty[st]);
        tc::umma_commit(&sh->o_full[buf]);
        if (j < 11) MK_TR(5 + j * 8);                        // P_j V_j issued
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ softmax + O accumulation
    // Eight warps: warps w and w + 4 share TMEM lane quarter w % 4, i.e. the same 32 query rows; each
    // thread owns one row and one half of its columns (64 keys of S_j, HD / 2 head-dim columns of O).  The
    // two threads of a row meet once per tile to agree on the row maximum (shared memory + a 64-thread
    // named barrier) and once at the end to add their row sums.
    const int q = warp & 3, hf = (warp - 2) >> 2;
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    const int row_in_tile = q * 32 + lane;
    float o[HD / 2];
#pragma unroll
    for (int i = 0; i < HD / 2; ++i) o[i] = 0.0f;
    float m = -INFINITY, l = 0.0f, alpha_prev = 0.0f;
    bool ok = true;
    for (int j = 0; j < T; ++j) {
      const int buf = j & 1;
      const uint32_t use = (j >> 1) & 1;
      ok = tc::mbar_wait(&sh->s_full[buf], use, abort_flag, status, tc::WAIT_TMEM_FULL);
      ok = __all_sync(0xffffffffu, ok ? 1 : 0) != 0;
      if (!ok) break;
      if (threadIdx.x == 64 && j < 11) MK_TR(1 + j * 8);   // S_j ready
      tc::tc_fence_after();
      const uint32_t s_addr = tmem_s + buf * 128 + lane_off + hf * 64;
      // the tile with hidden keys: the diagonal one (limit = the row's own index), or an unmasked head's ragged last
      // tile (limit = the last real key, the same for every row)
      const bool diag = j == T - 1 && (causal || (S & (BKV - 1)) != 0);
      const int lim = causal ? row_in_tile : S - 1 - j * BKV;
      const int col_base = hf * 64;                          // key index (inside the tile) of this thread's first column
      // pass 1: maximum of the raw scores (four independent chains), then into log2 units
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t r[32];
        tc::tmem_ld32(s_addr + c * 32, r);
        tc::tmem_ld_wait();
        if (!diag) {
#pragma unroll
          for (int i = 0; i < 32; ++i) mx4[i & 3] = fmaxf(mx4[i & 3], __uint_as_float(r[i]));
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (col_base + c * 32 + i <= lim) mx4[i & 3] = fmaxf(mx4[i & 3], __uint_as_float(r[i]));
        }
      }
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * scale_log2;
      sh->xch[j & 1][row_in_tile][hf] = mx;
      asm volatile("bar.sync %0, %1;" ::"r"(1 + q), "r"(64) : "memory");
      const float mx_other = sh->xch[j & 1][row_in_tile][hf ^ 1];
      if (threadIdx.x == 64 && j < 11) MK_TR(2 + j * 8);   // pass 1 done
      const float m_new = fmaxf(m, fmaxf(mx, mx_other));
      const float alpha = tc::ex2_fast(m - m_new);           // 0 on the first tile (m = -inf)
      const float neg_m = -m_new;
      // pass 2: probabilities, row sum, P -> TMEM as packed bf16 over S columns this thread has consumed
      float sum4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t r[32];
        uint32_t pk[16];
        tc::tmem_ld32(s_addr + c * 32, r);
        tc::tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          float p0 = tc::ex2_fast(fmaf(__uint_as_float(r[i]), scale_log2, neg_m));
          float p1 = tc::ex2_fast(fmaf(__uint_as_float(r[i + 1]), scale_log2, neg_m));
          if (diag) {
            if (col_base + c * 32 + i > lim) p0 = 0.0f;
            if (col_base + c * 32 + i + 1 > lim) p1 = 0.0f;
          }
          sum4[(i >> 1) & 3] += p0 + p1;
          pk[i >> 1] = pack_bf16x2(p0, p1);
        }
        tmem_st16(s_addr + c * 16, pk);
      }
      tc::tmem_st_wait();
      l = l * alpha + ((sum4[0] + sum4[1]) + (sum4[2] + sum4[3]));
      m = m_new;
      tc::tc_fence_before();
      tc::mbar_arrive(&sh->p_ready[buf]);
      if (threadIdx.x == 64 && j < 11) MK_TR(3 + j * 8);   // P_j written
      // fold the previous tile's P V into the register accumulator
      if (j >= 1) {
        const int pb = (j - 1) & 1;
        ok = tc::mbar_wait(&sh->o_full[pb], ((j - 1) >> 1) & 1, abort_flag, status, tc::WAIT_TMEM_FULL);
        ok = __all_sync(0xffffffffu, ok ? 1 : 0) != 0;
        if (!ok) break;
        tc::tc_fence_after();
        const uint32_t o_addr = tmem_o + pb * 128 + lane_off + hf * (HD / 2);
#pragma unroll
        for (int c = 0; c < OC; ++c) {
          uint32_t r[32];
          tc::tmem_ld32(o_addr + c * 32, r);
          tc::tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) o[c * 32 + i] = fmaf(o[c * 32 + i], alpha_prev, __uint_as_float(r[i]));
        }
        tc::tc_fence_before();
        tc::mbar_arrive(&sh->o_free[pb]);
        if (threadIdx.x == 64 && j < 11) MK_TR(4 + j * 8);   // O_{j-1} folded in
      }
      alpha_prev = alpha;
    }
    if (ok) {
      const int pb = (T - 1) & 1;
      ok = tc::mbar_wait(&sh->o_full[pb], ((T - 1) >> 1) & 1, abort_flag, status, tc::WAIT_TMEM_FULL);
      ok = __all_sync(0xffffffffu, ok ? 1 : 0) != 0;
    }
    if (ok) {
      tc::tc_fence_after();
      // the row sum is the sum of the two halves' sums (both are in units of the same final maximum)
      sh->xch[T & 1][row_in_tile][hf] = l;
      asm volatile("bar.sync %0, %1;" ::"r"(1 + q), "r"(64) : "memory");
      const float inv_l = 1.0f / (l + sh->xch[T & 1][row_in_tile][hf ^ 1]);
      const uint32_t o_addr = tmem_o + ((T - 1) & 1) * 128 + lane_off + hf * (HD / 2);
#pragma unroll
      for (int c = 0; c < OC; ++c) {
        uint32_t r[32];
        tc::tmem_ld32(o_addr + c * 32, r);
        tc::tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) o[c * 32 + i] = fmaf(o[c * 32 + i], alpha_prev, __uint_as_float(r[i])) * inv_l;
      }
      // store: rows (b*S + query), this thread's HD / 2 of the columns h*D .. h*D + HD - 1 of the [B*S, H*D] matrix
      EpiProgram none;
      none.n = 0;
      EpiWarp ew;
      ew.init(staging + (warp - 2) * EPI_WARP_BYTES, none, lane, false);
      const int64_t row0 = (int64_t)b * S + (int64_t)qt * BQ + q * 32;
      const int64_t row_end = (int64_t)b * S + S;
      auto rowmap = [&](int r) -> int64_t { const int64_t g = row0 + r; return g < row_end ? g : -1; };
      uint4 none_regs[8];
      const int64_t n_cols = (int64_t)H * HD;
#pragma unroll
      for (int c = 0; c < OC; ++c) {
        float v[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = o[c * 32 + i];
        ew.chunk_out(none, v, rowmap, out, (int64_t)h * HD + hf * (HD / 2) + c * 32, 0, n_cols, none_regs, -1);
      }
    }
  }

  MK_TR_PRINT("attn");
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

bool attention_tc_supported(const AttnView& a) {
  if ((a.D != 64 && a.D != 128) || a.B < 1 || a.H < 1 || a.S < 1) return false;
  if ((a.ss * 2) % 16 || (a.sh * 2) % 16 || (a.sb * 2) % 16) return false;
  if (a.B * a.H * ((a.S + BQ - 1) / BQ) > INT32_MAX) return false;
  return true;
}

cudaError_t attention_tc_plan(AttnTcPlan* p, const AttnView& a, void* o) {
  if (!attention_tc_supported(a)) return cudaErrorInvalidValue;
  const uint64_t dims[4] = {(uint64_t)a.D, (uint64_t)a.S, (uint64_t)a.H, (uint64_t)a.B};
  const uint64_t strides[3] = {(uint64_t)a.ss * 2, (uint64_t)a.sh * 2, (uint64_t)a.sb * 2};
  const uint32_t box[4] = {64, 128, 1, 1};
  cudaError_t e = encode_tmap_bf16(&p->tm_q, a.q, 4, dims, strides, box, true);
  if (e == cudaSuccess) e = encode_tmap_bf16(&p->tm_k, a.k, 4, dims, strides, box, true);
  if (e == cudaSuccess) e = encode_tmap_bf16(&p->tm_v, a.v, 4, dims, strides, box, true);
  if (e != cudaSuccess) return e;
  p->out = o;
  p->B = (int)a.B; p->H = (int)a.H; p->S = (int)a.S; p->D = (int)a.D;
  p->causal = a.causal;
  p->scale_log2 = (float)(1.4426950408889634 / sqrt((double)a.D));
  p->grid = (int)(a.B * a.H * ((a.S + BQ - 1) / BQ));
  return cudaSuccess;
}

cudaError_t launch_attention_tc(const AttnTcPlan& p, cudaStream_t s) {
  static SmemOptIn opt_in;
  {
    cudaError_t e = opt_in.ensure(attn_smem(128), attention_tc_kernel<64>, attention_tc_kernel<128>);
    if (e != cudaSuccess) return e;
  }
  if (p.D == 64)
    attention_tc_kernel<64><<<p.grid, THREADS, attn_smem(64), s>>>(p.tm_q, p.tm_k, p.tm_v, (__nv_bfloat16*)p.out, p.B, p.H, p.S, p.causal ? 1 : 0,
                                                                  p.scale_log2, kernel_status_ptr());
  else
    attention_tc_kernel<128><<<p.grid, THREADS, attn_smem(128), s>>>(p.tm_q, p.tm_k, p.tm_v, (__nv_bfloat16*)p.out, p.B, p.H, p.S,
                                                                    p.causal ? 1 : 0, p.scale_log2, kernel_status_ptr());
  return cudaGetLastError();
}

}  // namespace mk
