// K7, two-query-tile form: fused attention (causal, or unmasked with a run-time flag) on tcgen05 / TMEM, head_dim 128, bf16 in, fp32 softmax
// and accumulation.
//
//   O = softmax(mask_{j<=i}(Q K^T / sqrt(D))) V        online softmax, the S x S matrix never leaves the SM
//
// Persistent CTAs.  A work item is (batch, head, 256 consecutive queries) = two 128-query tiles ("streams"
// 0 and 1) that share every K/V tile they both need; items are handed out as complementary pairs (the
// heaviest query block of a head with its lightest), so every CTA gets the same number of key tiles.
//
//   warps 0-3    softmax of stream 0: one thread per query row.  S_j (128 fp32 columns of TMEM) -> registers,
//                p = exp2(s * scale*log2e - m), row sum, P_j back into TMEM as packed bf16 over the columns
//                of S_j.  The reference m is raised (and the running O and l rescaled) only on an item's first
//                and diagonal tiles or when a row sum would leave a safe range: see role_softmax.
//   warps 4-7    the same for stream 1.
//   warps 8-11   output: at the end of an item they read O from TMEM, divide by the row sum and store it.
//   warp 12      TMA: Q tiles per item, K and V tiles through two-stage rings (128-byte swizzle).
//   warp 13      TMEM allocation; one lane issues every MMA, the two streams interleaved:
//                   S_t = Q_t K_j^T (SS form, 128x128x16 x 8),   O_t (+)= P_t V_j (TS form: P from TMEM,
//                   V from shared memory, MN-major).  While one stream's softmax runs, the tensor pipe
//                   works for the other.
// TMEM (512 columns): S/P of stream 0 and 1 (2 x 128), O of stream 0 and 1 (2 x 128); O accumulates in TMEM.
// Causal: the diagonal tile is masked (key > query -> -inf, diagonal kept); tiles right of it are never visited.
// Unmasked: every stream visits every key tile; only the keys past S in a ragged last tile are hidden.
// Every mbarrier wait is bounded.
#include "device_common.cuh"
#include "tc_common.cuh"
#include "tc_epilogue.cuh"
#include "tc_plans.h"

namespace mk {

namespace {

constexpr int BQ = 128, BKV = 128, HD = 128;
constexpr int TILE_BYTES = 128 * HD * 2;   // 32 KB: two 128 x 64 sub-tiles of 16 KB
constexpr int SUB_BYTES = TILE_BYTES / 2;
constexpr int KV_STAGES = 2;
constexpr int THREADS = 512;

#ifdef MK_TRACE
__shared__ unsigned long long mk_tr[96];
#endif
#define TR2(cond, slot) do { if (cond) MK_TR(slot); } while (0)
#define TRM(jj, k) TR2(gbase == 0 && (jj) >= 2 && (jj) < 7, 1 + ((jj) - 2) * 16 + (k))

struct Shared {
  uint64_t q_full[2], q_free[2];
  uint64_t k_full[KV_STAGES], k_empty[KV_STAGES];
  uint64_t v_full[KV_STAGES], v_empty[KV_STAGES];
  uint64_t s_lo_full[2], s_hi_full[2], b_free[2], p_ready[2], o_final[2], l_ready[2], o_free[2];
  uint32_t tmem_base;
  int abort_flag;
  float l[2][128];
};
constexpr size_t ATTN2_SMEM = (size_t)TILE_BYTES * (2 + 2 * KV_STAGES) + 4 * EPI_WARP_BYTES + 1024 + ((sizeof(Shared) + 255) / 256) * 256;

// One work item: two query tiles of one (batch, head).  n0, n1 = number of key tiles stream 0, 1 visits
// (0: the stream has no queries in this item), nk = key tiles loaded for the item.
struct Item {
  int b, h, q0;
  int n0, n1;
  int nk;
};

// Every role walks the same list: super-items blockIdx.x, + gridDim.x, ...; super-item s of a head is the
// query block P-1-s followed by block s.
struct ItemIter {
  int sidx, half, n_super, SP, P, num_q, H;
  bool causal;
  __device__ __forceinline__ void init(int S, int B, int H_, bool causal_) {
    causal = causal_;
    num_q = (S + BQ - 1) / BQ;
    P = (num_q + 1) / 2;
    SP = (P + 1) / 2;
    H = H_;
    n_super = B * H * SP;
    sidx = blockIdx.x;
    half = 0;
  }
  __device__ __forceinline__ bool next(Item& it) {
    while (sidx < n_super) {
      const int bh = sidx / SP, s = sidx - bh * SP;
      const int hi = P - 1 - s;
      int p;
      if (half == 0) {
        p = hi;
        half = 1;
      } else {
        half = 0;
        sidx += gridDim.x;
        if (s == hi) continue;
        p = s;
      }
      it.b = bh / H;
      it.h = bh - it.b * H;
      it.q0 = p * 2 * BQ;
      // causal: the query tile at index i sees key tiles 0..i; unmasked: every stream sees all of them
      it.n0 = causal ? 2 * p + 1 : num_q;
      it.n1 = (2 * p + 1 < num_q) ? (causal ? 2 * p + 2 : num_q) : 0;
      it.nk = it.n1 ? it.n1 : it.n0;
      return true;
    }
    return false;
  }
};

struct Ctx {
  Shared* sh;
  volatile int* abort_flag;
  unsigned int* status;
  __device__ __forceinline__ bool wait(uint64_t* bar, uint32_t parity, unsigned code) const {
    return tc::mbar_wait(bar, parity, abort_flag, status, code);
  }
  // the same for a whole warp (its next instruction is warp-collective)
  __device__ __forceinline__ bool wait_warp(uint64_t* bar, uint32_t parity, unsigned code) const {
    const bool ok = tc::mbar_wait(bar, parity, abort_flag, status, code);
    return __all_sync(0xffffffffu, ok ? 1 : 0) != 0;
  }
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
// Eight MMAs (one 128-wide K or key tile).  The descriptors are formed inside the block from two base words and
// compile-time offsets (two adds and two moves per MMA, which run while the MMA before executes): the issuing
// thread keeps four words in registers across its waits instead of thirty-two.
// a_lo / b_lo: low descriptor words (address >> 4 | ...) of the first K slice; slice k sits OFF(k) further, where
// OFF(k) = (k / 4) * (SUB_BYTES >> 4) + (k % 4) * 2 (two 64-element sub-tiles of four 16-element slices each).
#define MK_SS_STEP(OFF, PRED)                                   \
  "add.u32 la, %2, " #OFF ";\n\tadd.u32 lb, %3, " #OFF ";\n\t" \
  "mov.b64 da, {la, %4};\n\tmov.b64 db, {lb, %4};\n\t"         \
  "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %1, " #PRED ";\n\t"
__device__ __forceinline__ void umma_ss_x8(uint32_t d, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc) {
  static_assert((SUB_BYTES >> 4) == 1024, "offsets below");
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t.reg .b32 la, lb;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p, %1, %1;\n\t"
      "setp.eq.b32 q, %1, %1;\n\t"
      MK_SS_STEP(0, p) MK_SS_STEP(2, q) MK_SS_STEP(4, q) MK_SS_STEP(6, q)
      MK_SS_STEP(1024, q) MK_SS_STEP(1026, q) MK_SS_STEP(1028, q) MK_SS_STEP(1030, q)
      "}" ::"r"(d), "r"(idesc), "r"(a_lo), "r"(b_lo), "r"(desc_hi)
      : "memory");
}
#undef MK_SS_STEP
// D (+)= A[tmem] B[smem]; the first MMA accumulates only if acc0 != 0.  A: 8 TMEM columns per 16-key slice;
// B (= V, MN-major): 16 keys = 16 rows of 128 bytes = 128 descriptor units per slice.
#define MK_TS_STEP(K, PRED)                                             \
  "add.u32 ta, %3, " #K "*8;\n\tadd.u32 lb, %4, " #K "*128;\n\t"       \
  "mov.b64 db, {lb, %5};\n\t"                                          \
  "tcgen05.mma.cta_group::1.kind::f16 [%0], [ta], db, %1, " #PRED ";\n\t"
__device__ __forceinline__ void umma_ts_x8(uint32_t d, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc, uint32_t acc0) {
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t.reg .b32 ta, lb;\n\t.reg .b64 db;\n\t"
      "setp.ne.b32 p, %2, 0;\n\t"
      "setp.eq.b32 q, %1, %1;\n\t"
      MK_TS_STEP(0, p) MK_TS_STEP(1, q) MK_TS_STEP(2, q) MK_TS_STEP(3, q)
      MK_TS_STEP(4, q) MK_TS_STEP(5, q) MK_TS_STEP(6, q) MK_TS_STEP(7, q)
      "}" ::"r"(d), "r"(idesc), "r"(acc0), "r"(a_tmem), "r"(b_lo), "r"(b_hi)
      : "memory");
}
#undef MK_TS_STEP
// keep a value computed before a wait in a register across it
__device__ __forceinline__ void pin(uint32_t& x) { asm volatile("" : "+r"(x)); }
__device__ __forceinline__ void pin(uint64_t& x) { asm volatile("" : "+l"(x)); }

__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]),
      "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}

// ------------------------------------------------------------------------------------------ TMA producer
// Order per item: Q0, K0, Q1, V0, K1, V1, ... : the order in which the slots come free (the MMAs retire
// as QK(j) of both streams, PV(j) of both, QK(j+1) ...), so no load queues behind a slot that frees later.
__device__ __forceinline__ void role_loader(const Ctx& cx, const CUtensorMap* tmQ, const CUtensorMap* tmK, const CUtensorMap* tmV,
                                            uint8_t* q_tiles, uint8_t* k_tiles, uint8_t* v_tiles, int B, int H, int S, bool causal) {
  Shared* sh = cx.sh;
  ItemIter iter;
  iter.init(S, B, H, causal);
  Item it;
  uint32_t n_items[2] = {0, 0};
  uint32_t g = 0;   // key tiles loaded so far by this CTA (ring position)
  while (iter.next(it)) {
    auto load_q = [&](int t) -> bool {
      if (!cx.wait(&sh->q_free[t], (n_items[t] & 1) ^ 1, tc::WAIT_SMEM_EMPTY)) return false;
      ++n_items[t];
      uint8_t* qd = q_tiles + (size_t)t * TILE_BYTES;
      tc::mbar_expect_tx(&sh->q_full[t], TILE_BYTES);
      tc::tma_load_4d(qd, tmQ, &sh->q_full[t], 0, it.q0 + t * BQ, it.h, it.b);
      tc::tma_load_4d(qd + SUB_BYTES, tmQ, &sh->q_full[t], 64, it.q0 + t * BQ, it.h, it.b);
      return true;
    };
    auto load_kv = [&](int j, bool is_v) -> bool {
      const uint32_t gg = g + (uint32_t)j;
      const int st = gg % KV_STAGES;
      uint64_t* empty = is_v ? &sh->v_empty[st] : &sh->k_empty[st];
      uint64_t* full = is_v ? &sh->v_full[st] : &sh->k_full[st];
      if (!cx.wait(empty, ((gg / KV_STAGES) & 1) ^ 1, tc::WAIT_SMEM_EMPTY)) return false;
      uint8_t* dst = (is_v ? v_tiles : k_tiles) + (size_t)st * TILE_BYTES;
      const CUtensorMap* tm = is_v ? tmV : tmK;
      tc::mbar_expect_tx(full, TILE_BYTES);
      tc::tma_load_4d(dst, tm, full, 0, j * BKV, it.h, it.b);
      tc::tma_load_4d(dst + SUB_BYTES, tm, full, 64, j * BKV, it.h, it.b);
      return true;
    };
    if (!load_q(0)) return;
    if (!load_kv(0, false)) return;
    if (it.n1 && !load_q(1)) return;
    if (!load_kv(0, true)) return;
    for (int j = 1; j < it.nk; ++j) {
      if (!load_kv(j, false)) return;
      if (!load_kv(j, true)) return;
    }
    g += (uint32_t)it.nk;
  }
}

// ------------------------------------------------------------------------------------------ MMA issuer
// One issuing thread per stream (warps 13 and 14).  Stream t's order is S_t(0), [O_t(0), S_t(1)], [O_t(1), S_t(2)], ...
// straight across items: P_t aliases S_t, so QK_t(j+1) has to follow PV_t(j) anyway, and PV_t(j) waits
// for the stream's softmax; the pair in brackets is issued as one run of sixteen MMAs, so the path from
// "P is ready" to "the next S is ready" holds no waits, descriptor arithmetic or bookkeeping.  During the
// wait for P the other thread keeps the tensor pipe busy.  Two threads
// because the pipe accepts an MMA only about when it can start it: the issuing thread is blocked for
// the whole run of its eight MMAs, and its waits, commits and bookkeeping (about as long again) would
// otherwise leave the pipe idle.  The streams synchronise only through the K/V ring: a slot is
// released by two commit arrivals, one per stream (both from the same thread for a tile only it reads).
// The stream index is a run-time value on purpose: one copy of the code for both warps.
__device__ __forceinline__ void role_mma(const Ctx& cx, uint32_t tmem_base, int t, uint8_t* q_tiles, uint8_t* k_tiles, uint8_t* v_tiles, int B,
                                         int H, int S, bool causal) {
  Shared* sh = cx.sh;
  constexpr uint32_t idesc_qk64 = tc::idesc_bf16_f32(BQ, 64, 0, 0);  // A, B K-major, half a key tile
  constexpr uint32_t idesc_pv = tc::idesc_bf16_f32(BQ, HD, 0, 1);    // B (= V) MN-major
  // V, MN-major with 128-byte swizzle: 64 head-dim elements are contiguous (one 128-byte row per key),
  // 8-key groups are 1024 B apart (SBO), the second 64 head-dim elements sit SUB_BYTES on (LBO)
  constexpr uint32_t v_hi = ((1024u >> 4) & 0x3FFF) | (1u << 14) | (2u << 29);
  const uint32_t q_lo0 = tc::desc_lo_sw128(tc::smem_u32(q_tiles));
  const uint32_t k_lo0 = tc::desc_lo_sw128(tc::smem_u32(k_tiles));
  const uint32_t v_lo0 = ((tc::smem_u32(v_tiles) & 0x3FFFF) >> 4) | ((uint32_t)(SUB_BYTES >> 4) << 16);
  uint32_t par_qfull = 0;     // parity of the next q_full[t] phase to wait for
  uint32_t par_ofree = 1;     // parity to wait for on o_free[t] (starts "already free")
  uint32_t par_pv = 0;
  const uint32_t q_lo = q_lo0 + (uint32_t)t * (TILE_BYTES >> 4);
  const uint32_t s_tmem = tmem_base + (uint32_t)t * 128;          // S, and P over it (packed bf16: 16 keys = 8 columns)
  const uint32_t o_tmem = tmem_base + 256 + (uint32_t)t * 128;

  // one key tile of this stream: j-th of nt in an item whose tiles start at ring position g
  struct Pos {
    int n0, n1, nt, j;
    uint32_t g;
    bool valid;
  };
  ItemIter iter;
  iter.init(S, B, H, causal);
  uint32_t g_next = 0;
  auto next_item = [&](Pos& p) {
    Item it;
    p.valid = false;
    while (iter.next(it)) {
      const int nt = t ? it.n1 : it.n0;
      const uint32_t g = g_next;
      g_next += (uint32_t)it.nk;
      if (nt > 0) {
        p.n0 = it.n0; p.n1 = it.n1; p.nt = nt; p.j = 0; p.g = g; p.valid = true;
        return;
      }
    }
  };
  // One step: O_t (+)= P_t V for tile a (if do_pv) and S_t = Q_t K^T for the following tile b (if do_qk), S in two
  // halves of 64 keys:
  //   S_lo(b) (keys 0..63)   -> columns [64, 128) of the stream's S region ("region B"), as soon as the
  //                             softmax has read S_lo(a) out of it: while softmax(a) is still busy with its second half;
  //   P V(a), then S_hi(b)   -> columns [0, 64) ("region A", which also holds P(a)), once P(a) is there.
  // So when softmax(a) ends, half of the next S is already waiting for it, and the other half arrives while it
  // works on the first: the chain softmax -> P V -> Q K^T -> softmax no longer has the MMAs in it.
  // Operands are precomputed before the waits.  The two issuing threads do not take turns: a lock around each
  // run of MMAs (tried) makes the short early Q K^T wait for the other stream's whole run.
  bool first_qk = true;
  uint32_t par_bfree = 0;
  auto issue = [&](const Pos& a, bool do_pv, const Pos& b, bool do_qk) -> bool {
    const uint32_t ga = a.g + (uint32_t)a.j, gb = b.g + (uint32_t)b.j;
    const int sta = ga % KV_STAGES, stb = gb % KV_STAGES;
    bool lo_done = false, hi_done = false;
    uint32_t v_lo = v_lo0 + (uint32_t)sta * (TILE_BYTES >> 4);
    uint32_t k_lo = k_lo0 + (uint32_t)stb * (TILE_BYTES >> 4);
    pin(v_lo);
    pin(k_lo);
    auto issue_lo = [&]() {
      umma_ss_x8(s_tmem + 64, q_lo, k_lo, tc::kDescHiSw128, idesc_qk64);
      tc::umma_commit(&sh->s_lo_full[t]);
    };
    auto issue_hi = [&]() {
      umma_ss_x8(s_tmem, q_lo, k_lo + (uint32_t)((64 * 128) >> 4), tc::kDescHiSw128, idesc_qk64);   // key rows 64..127 of the K tile
      tc::umma_commit(&sh->s_hi_full[t]);
    };
    if (do_qk) {
      if (!first_qk) {
        // region B has been read (the softmax signals it half-way through tile a)
        if (!cx.wait(&sh->b_free[t], par_bfree, tc::WAIT_TMEM_EMPTY)) return false;
        par_bfree ^= 1u;
      }
      first_qk = false;
      // Early only if Q and K are already there: waiting for them here, before this tile's P V is issued, could
      // wait for a load that is queued behind a slot this very P V releases.
      bool ready = true;
      if (do_pv) {
        ready = (b.j != 0 || tc::mbar_test_wait(&sh->q_full[t], par_qfull)) && tc::mbar_test_wait(&sh->k_full[stb], (gb / KV_STAGES) & 1);
      } else {
        if (b.j == 0 && !cx.wait(&sh->q_full[t], par_qfull, tc::WAIT_SMEM_FULL)) return false;
        if (!cx.wait(&sh->k_full[stb], (gb / KV_STAGES) & 1, tc::WAIT_SMEM_FULL)) return false;
      }
      if (ready) {
        tc::tc_fence_after();
        issue_lo();
        if (!do_pv) { issue_hi(); hi_done = true; }
        lo_done = true;
      }
    }
    if (do_pv) {
      if (a.j == 0) {
        // the previous item's O of this stream has been read out
        if (!cx.wait(&sh->o_free[t], par_ofree, tc::WAIT_TMEM_EMPTY)) return false;
        par_ofree ^= 1u;
      }
      if (!cx.wait(&sh->v_full[sta], (ga / KV_STAGES) & 1, tc::WAIT_SMEM_FULL)) return false;
      if (!tc::mbar_wait_spin(&sh->p_ready[t], par_pv, cx.abort_flag, cx.status, tc::WAIT_ATTN)) return false;
      par_pv ^= 1u;
      TR2(a.g == 0 && a.j < 11, (t ? 8 : 4) + a.j * 8);
      tc::tc_fence_after();
      umma_ts_x8(o_tmem, s_tmem, v_lo, v_hi, idesc_pv, a.j > 0 ? 1u : 0u);
      if (do_qk && lo_done) { issue_hi(); hi_done = true; }
      // a K/V slot is released by two arrivals: one per stream, or both from the only stream that reads it
      if (a.j == a.nt - 1) tc::umma_commit(&sh->o_final[t]);
      tc::umma_commit(&sh->v_empty[sta]);
      if (!(a.j < a.n0 && a.j < a.n1)) tc::umma_commit(&sh->v_empty[sta]);
    }
    if (do_qk) {
      if (!hi_done) {
        if (b.j == 0 && !cx.wait(&sh->q_full[t], par_qfull, tc::WAIT_SMEM_FULL)) return false;
        if (!cx.wait(&sh->k_full[stb], (gb / KV_STAGES) & 1, tc::WAIT_SMEM_FULL)) return false;
        tc::tc_fence_after();
        if (!lo_done) issue_lo();
        issue_hi();
      }
      if (b.j == 0) par_qfull ^= 1u;
      tc::umma_commit(&sh->k_empty[stb]);
      if (!(b.j < b.n0 && b.j < b.n1)) tc::umma_commit(&sh->k_empty[stb]);
      if (b.j == b.nt - 1) tc::umma_commit(&sh->q_free[t]);
    }
    return true;
  };

  Pos a, b;
  next_item(a);
  if (!a.valid) return;
  if (!issue(a, false, a, true)) return;
  while (true) {
    b = a;
    if (b.j + 1 < b.nt) ++b.j;
    else next_item(b);
    if (!issue(a, true, b, b.valid)) return;
    if (!b.valid) break;
    a = b;
  }
}

// Two fp32 multiply-adds / adds in one instruction (sm_100 packed fp32): the softmax's issue slots are as
// scarce as its special-function slots.
__device__ __forceinline__ void fma2(float& d0, float& d1, float a0, float a1, float b, float c) {
  asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\t"
      "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %4};\n\tmov.b64 rc, {%5, %5};\n\t"
      "fma.rn.f32x2 rd, ra, rb, rc;\n\t"
      "mov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d0), "=f"(d1)
      : "f"(a0), "f"(a1), "f"(b), "f"(c));
}
__device__ __forceinline__ void add2(float& s0, float& s1, float a0, float a1) {
  asm("{\n\t.reg .b64 ra, rs;\n\t"
      "mov.b64 ra, {%2, %3};\n\tmov.b64 rs, {%0, %1};\n\t"
      "add.rn.f32x2 rs, rs, ra;\n\t"
      "mov.b64 {%0, %1}, rs;\n\t}"
      : "+f"(s0), "+f"(s1)
      : "f"(a0), "f"(a1));
}

// ------------------------------------------------------------------------------------------ softmax
// One thread per query row of stream T.  m is the reference maximum in log2 units (scores times
// scale * log2 e): p = exp2(s * scale*log2e - m).  Any m gives the same O / l as long as nothing
// overflows, so m is NOT kept equal to the running row maximum; it is raised (and the running O in TMEM,
// l, and whatever of this tile's P is already computed, rescaled by exp2(m_old - m_new)) only
// when a half-row sum leaves the safe range (above 2^60; or, on an item's very first half, where m is a
// mere guess of 0, underflowed) - then from that half's own maximum.  The common tile is therefore one pass
// over S with no maximum at all.  On the diagonal tile (an item's last) a warp masks the one 32-key chunk
// that holds its own diagonal by writing -inf over the hidden scores in TMEM, and skips the chunks right of it.
// S arrives in two halves: keys 0..63 in columns [64, 128) of the stream's S region (B), keys 64..127 in
// columns [0, 64) (A).  As soon as the first half has been turned into probabilities (kept in registers),
// region B is handed back (b_free) and the tensor pipe computes the next tile's first half into it while this
// thread works on the second half.  P (packed bf16, 64 columns) goes over region A at the end.
// O may be touched only after S_hi of the same tile is visible: Q K^T_hi(j) is issued after P V(j-1), the
// pipe runs in order, and the next P V is not issued before this thread's p_ready arrival.
__device__ __forceinline__ void role_softmax(const Ctx& cx, uint32_t tmem_base, int T, int warp, int lane, int B, int H, int S,
                                             bool causal, float scale_log2) {
  Shared* sh = cx.sh;
  const int q = warp & 3;
  const int row = q * 32 + lane;
  const uint32_t lane_off = (uint32_t)(q * 32) << 16;
  const uint32_t s_addr = tmem_base + (uint32_t)T * 128 + lane_off;     // region A; region B = s_addr + 64
  const uint32_t o_addr = tmem_base + 256 + (uint32_t)T * 128 + lane_off;
  ItemIter iter;
  iter.init(S, B, H, causal);
  Item it;
  uint32_t n_tiles = 0, n_items = 0;
  while (iter.next(it)) {
    const int nt = T ? it.n1 : it.n0;
    if (nt == 0) continue;
    // m = 0 is the first guess of an item (scores of the usual size then need no maximum at all); `fresh`
    // says that nothing of this item has been accumulated yet, so m may still be set freely
    float m = 0.0f, l = 0.0f;
    bool fresh = true;
#pragma unroll 1
    for (int j = 0; j < nt; ++j) {
      const uint32_t par = n_tiles & 1;
      ++n_tiles;
      auto wait_half = [&](uint64_t* bar) -> bool {
        const bool ok = tc::mbar_wait_spin(bar, par, cx.abort_flag, cx.status, tc::WAIT_TMEM_FULL);
        const bool all = __all_sync(0xffffffffu, ok ? 1 : 0) != 0;
        if (all) tc::tc_fence_after();
        return all;
      };
      // m := max(m, mx); the running O (not on an item's first tile) and l follow
      auto raise = [&](float mx) -> float {
        if (fresh) {
          m = mx;                          // nothing to rescale yet
          return 1.0f;
        }
        float alpha = 1.0f;
        if (mx > m) {
          alpha = tc::ex2_fast(m - mx);
          m = mx;
        }
        if (j > 0 && __any_sync(0xffffffffu, alpha != 1.0f)) {
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            tc::tmem_ld32(o_addr + c * 32, r);
            tc::tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
            tc::tmem_st32(o_addr + c * 32, r);
          }
          tc::tmem_st_wait();
        }
        l *= alpha;
        return alpha;
      };
      // maximum (log2 units) of 64 scores starting at TMEM address `base`
      auto half_max = [&](uint32_t base, int nchunks) -> float {
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll 1
        for (int c = 0; c < nchunks; ++c) {
          uint32_t r[32];
          tc::tmem_ld32(base + c * 32, r);
          tc::tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) mx4[i & 3] = fmaxf(mx4[i & 3], __uint_as_float(r[i]));
        }
        return fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * scale_log2;
      };

      // Chunks of 32 keys this warp's rows can see at all: every one off the diagonal; on the diagonal tile
      // (the item's last) chunk q holds the warp's own diagonal (key i of it is visible to lane >= i) and the
      // chunks right of it are skipped outright.
      // Without the causal mask only a ragged last key tile has anything hidden: keys from `rem` on, the same
      // for every row.  All of these conditions are the same for the whole warp.
      const int rem = S - (nt - 1) * BKV;                       // keys of the item's last tile that exist
      const bool diag = j == nt - 1 && (causal || rem < BKV);
      const int vis = !diag ? 4 : causal ? q + 1 : (rem + 31) >> 5;
      if (diag) {
        if (!wait_half(&sh->s_lo_full[T])) return;
        if (!wait_half(&sh->s_hi_full[T])) return;
        // -inf over the hidden scores of the one partly visible chunk, in place, so that the main pass needs no
        // mask code: chunk mc, elements above `lim`
        const int mc = causal ? q : ((rem & 31) ? rem >> 5 : -1);
        const int lim = causal ? lane : (rem & 31) - 1;
        if (mc >= 0) {
          const uint32_t addr = s_addr + (mc < 2 ? 64 + mc * 32 : (mc - 2) * 32);
          uint32_t r[32];
          tc::tmem_ld32(addr, r);
          tc::tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (i > lim) r[i] = 0xff800000u;
          tc::tmem_st32(addr, r);
          tc::tmem_st_wait();
        }
      }

      uint32_t pk[64];
      float sum_lo = 0.0f, sum_hi = 0.0f;
      // ---- first half: keys 0..63 from region B
      if (!wait_half(&sh->s_lo_full[T])) return;
      TR2(T == 0 && threadIdx.x == 0 && n_items == 0 && j < 11, 1 + j * 8);
      TR2(T == 1 && threadIdx.x == 128 && n_items == 0 && j < 11, 5 + j * 8);
#pragma unroll 1
      for (int attempt = 0; attempt < 2; ++attempt) {
        const float neg_m = -m;
        float sum4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          if (c >= vis) {
#pragma unroll
            for (int i = 0; i < 16; ++i) pk[c * 16 + i] = 0u;
            continue;
          }
          uint32_t r[32];
          tc::tmem_ld32(s_addr + 64 + c * 32, r);
          tc::tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            float x0, x1;
            fma2(x0, x1, __uint_as_float(r[i]), __uint_as_float(r[i + 1]), scale_log2, neg_m);
            const float p0 = tc::ex2_fast(x0), p1 = tc::ex2_fast(x1);
            add2(sum4[(i >> 1) & 1 ? 2 : 0], sum4[(i >> 1) & 1 ? 3 : 1], p0, p1);
            pk[c * 16 + (i >> 1)] = pack_bf16x2(p0, p1);
          }
        }
        sum_lo = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
        // safe range: below 2^60 (also false for inf / NaN) and, while m is still the first guess, not underflowed
        const bool bad = !(sum_lo < 1.152921504606847e18f) || (fresh && !(sum_lo > 8.673617379884035e-19f));
        if (attempt == 1 || !__any_sync(0xffffffffu, bad)) break;
        // out of range: raise m to this half's maximum (O is safe to touch once S_hi is visible), then once more
        if (!wait_half(&sh->s_hi_full[T])) return;
        raise(half_max(s_addr + 64, vis < 2 ? vis : 2));
      }
      fresh = false;
      tc::tc_fence_before();
      tc::mbar_arrive(&sh->b_free[T]);
      TR2(T == 0 && threadIdx.x == 0 && n_items == 0 && j < 11, 2 + j * 8);
      // ---- second half: keys 64..127 from region A
      if (!wait_half(&sh->s_hi_full[T])) return;
      TR2(T == 0 && threadIdx.x == 0 && n_items == 0 && j < 11, 6 + j * 8);
#pragma unroll 1
      for (int attempt = 0; attempt < 2; ++attempt) {
        const float neg_m = -m;
        float sum4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          if (2 + c >= vis) {
#pragma unroll
            for (int i = 0; i < 16; ++i) pk[32 + c * 16 + i] = 0u;
            continue;
          }
          uint32_t r[32];
          tc::tmem_ld32(s_addr + c * 32, r);
          tc::tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            float x0, x1;
            fma2(x0, x1, __uint_as_float(r[i]), __uint_as_float(r[i + 1]), scale_log2, neg_m);
            const float p0 = tc::ex2_fast(x0), p1 = tc::ex2_fast(x1);
            add2(sum4[(i >> 1) & 1 ? 2 : 0], sum4[(i >> 1) & 1 ? 3 : 1], p0, p1);
            pk[32 + c * 16 + (i >> 1)] = pack_bf16x2(p0, p1);
          }
        }
        sum_hi = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
        if (attempt == 1 || !__any_sync(0xffffffffu, !(sum_hi < 1.152921504606847e18f))) break;
        // out of range: raise m to this half's maximum; the first half's probabilities and sum follow
        const float alpha = raise(half_max(s_addr, vis - 2 > 0 ? vis - 2 : 0));
        sum_lo *= alpha;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const float a0 = __uint_as_float(pk[i] << 16) * alpha, a1 = __uint_as_float(pk[i] & 0xffff0000u) * alpha;
          pk[i] = pack_bf16x2(a0, a1);
        }
      }
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t part[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) part[i] = pk[c * 16 + i];
        tmem_st16(s_addr + c * 16, part);
      }
      l += sum_lo + sum_hi;
      tc::tmem_st_wait();
      tc::tc_fence_before();
      tc::mbar_arrive(&sh->p_ready[T]);
      TR2(T == 0 && threadIdx.x == 0 && n_items == 0 && j < 11, 3 + j * 8);
      TR2(T == 1 && threadIdx.x == 128 && n_items == 0 && j < 11, 7 + j * 8);
    }
    // the previous item's row sums have been read (a stream whose items are one tile long can otherwise
    // finish two items before the output warps have finished one)
    if (!cx.wait_warp(&sh->o_free[T], (n_items & 1) ^ 1, tc::WAIT_TMEM_EMPTY)) return;
    ++n_items;
    sh->l[T][row] = l;
    tc::mbar_arrive(&sh->l_ready[T]);
  }
}

// ------------------------------------------------------------------------------------------ output
// At the end of an item: O / l, to bf16, through the shared-memory transpose to the [B*S, H*D] matrix.
__device__ __forceinline__ void role_output(const Ctx& cx, uint32_t tmem_base, uint8_t* staging, int warp, int lane,
                                            __nv_bfloat16* __restrict__ out, int B, int H, int S, bool causal) {
  Shared* sh = cx.sh;
  const int q = warp & 3;
  const int row = q * 32 + lane;
  const uint32_t lane_off = (uint32_t)(q * 32) << 16;
  EpiProgram none;
  none.n = 0;
  EpiWarp ew;
  ew.init(staging + q * EPI_WARP_BYTES, none, lane, false);
  ItemIter iter;
  iter.init(S, B, H, causal);
  Item it;
  uint32_t par_item = 0;   // bit t: parity of stream t's next phase
  const int64_t row_bytes = (int64_t)H * HD * 2;
  while (iter.next(it)) {
#pragma unroll 1
    for (int t = 0; t < 2; ++t) {
      if ((t ? it.n1 : it.n0) == 0) continue;
      if (!cx.wait_warp(&sh->l_ready[t], (par_item >> t) & 1, tc::WAIT_ATTN)) return;
      if (!cx.wait_warp(&sh->o_final[t], (par_item >> t) & 1, tc::WAIT_TMEM_FULL)) return;
      par_item ^= 1u << t;
      tc::tc_fence_after();
      const float inv_l = 1.0f / sh->l[t][row];
      const uint32_t o_addr = tmem_base + 256 + (uint32_t)t * 128 + lane_off;
      const int q_row0 = it.q0 + t * BQ + q * 32;                       // query index of this warp's first row
      const int64_t g_row0 = (int64_t)it.b * S + q_row0;
      auto rowmap = [&](int r) -> int64_t { return q_row0 + r < S ? g_row0 + r : -1; };
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        uint32_t r[32];
        tc::tmem_ld32(o_addr + c * 32, r);
        tc::tmem_ld_wait();
        if (c == 3) {
          // O has left TMEM: the next item's first P V of this stream may overwrite it
          tc::tc_fence_before();
          tc::mbar_arrive(&sh->o_free[t]);
        }
        uint4 mine[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          mine[k].x = pack_bf16x2(__uint_as_float(r[8 * k + 0]) * inv_l, __uint_as_float(r[8 * k + 1]) * inv_l);
          mine[k].y = pack_bf16x2(__uint_as_float(r[8 * k + 2]) * inv_l, __uint_as_float(r[8 * k + 3]) * inv_l);
          mine[k].z = pack_bf16x2(__uint_as_float(r[8 * k + 4]) * inv_l, __uint_as_float(r[8 * k + 5]) * inv_l);
          mine[k].w = pack_bf16x2(__uint_as_float(r[8 * k + 6]) * inv_l, __uint_as_float(r[8 * k + 7]) * inv_l);
        }
        ew.own_row_to_global(mine, rowmap, reinterpret_cast<uint8_t*>(out), row_bytes, ((int64_t)it.h * HD + c * 32) * 2);
      }
    }
  }
}

__global__ void __launch_bounds__(THREADS, 1)
attention_tc2_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                     __nv_bfloat16* __restrict__ out, int B, int H, int S, int causal_i, float scale_log2, unsigned int* status) {
  const bool causal = causal_i != 0;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* q_tiles = base;
  uint8_t* k_tiles = q_tiles + 2 * TILE_BYTES;
  uint8_t* v_tiles = k_tiles + KV_STAGES * TILE_BYTES;
  uint8_t* staging = v_tiles + KV_STAGES * TILE_BYTES;
  Shared* sh = reinterpret_cast<Shared*>(staging + 4 * EPI_WARP_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  MK_TR_INIT;

  if (threadIdx.x == 0) {
    for (int t = 0; t < 2; ++t) {
      tc::mbar_init(&sh->q_full[t], 1); tc::mbar_init(&sh->q_free[t], 1);
      tc::mbar_init(&sh->s_lo_full[t], 1); tc::mbar_init(&sh->s_hi_full[t], 1); tc::mbar_init(&sh->b_free[t], 128);
      tc::mbar_init(&sh->p_ready[t], 128);
      tc::mbar_init(&sh->o_final[t], 1); tc::mbar_init(&sh->l_ready[t], 128); tc::mbar_init(&sh->o_free[t], 128);
    }
    for (int s = 0; s < KV_STAGES; ++s) {
      tc::mbar_init(&sh->k_full[s], 1); tc::mbar_init(&sh->k_empty[s], 2);
      tc::mbar_init(&sh->v_full[s], 1); tc::mbar_init(&sh->v_empty[s], 2);
    }
    sh->abort_flag = 0;
    tc::fence_barrier_init();
    tc::tma_prefetch_desc(&tmQ);
    tc::tma_prefetch_desc(&tmK);
    tc::tma_prefetch_desc(&tmV);
  }
  if (warp == 13) { tc::tmem_alloc(&sh->tmem_base, 512); tc::tmem_relinquish(); }
  tc::tc_fence_before();
  __syncthreads();
  tc::tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;
  Ctx cx{sh, &sh->abort_flag, status};
  pdl_launch_dependents();
  pdl_wait();   // Q, K, V may come from the kernel before this one

  if (warp < 8) {
    role_softmax(cx, tmem_base, warp >> 2, warp, lane, B, H, S, causal, scale_log2);
  } else if (warp < 12) {
    role_output(cx, tmem_base, staging, warp, lane, out, B, H, S, causal);
  } else {
    if (warp == 12 && lane == 0) role_loader(cx, &tmQ, &tmK, &tmV, q_tiles, k_tiles, v_tiles, B, H, S, causal);
    if ((warp == 13 || warp == 14) && lane == 0) role_mma(cx, tmem_base, warp - 13, q_tiles, k_tiles, v_tiles, B, H, S, causal);
    __syncwarp();
  }

  MK_TR_PRINT("attn2");
  if (sh->abort_flag) {
    // give copies in flight time to land before shared memory and TMEM are handed back
    const long long t0 = clock64();
    while (clock64() - t0 < 4000000LL) {}
  }
  tc::tc_fence_before();
  __syncthreads();
  if (warp == 13) {
    tc::tc_fence_after();
    tc::tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace

bool attention_tc2_supported(const AttnView& a) {
  if (a.D != HD || a.B < 1 || a.H < 1 || a.S < 1) return false;
  if ((a.ss * 2) % 16 || (a.sh * 2) % 16 || (a.sb * 2) % 16) return false;
  if (a.B * a.H * ((a.S + BQ - 1) / BQ) > INT32_MAX / 4) return false;
  return true;
}

cudaError_t attention_tc2_plan(AttnTcPlan* p, const AttnView& a, void* o, int sm_count) {
  if (!attention_tc2_supported(a)) return cudaErrorInvalidValue;
  const uint64_t dims[4] = {(uint64_t)a.D, (uint64_t)a.S, (uint64_t)a.H, (uint64_t)a.B};
  const uint64_t strides[3] = {(uint64_t)a.ss * 2, (uint64_t)a.sh * 2, (uint64_t)a.sb * 2};
  const uint32_t box[4] = {64, 128, 1, 1};
  cudaError_t e = encode_tmap_bf16(&p->tm_q, a.q, 4, dims, strides, box, true);
  if (e == cudaSuccess) e = encode_tmap_bf16(&p->tm_k, a.k, 4, dims, strides, box, true);
  if (e == cudaSuccess) e = encode_tmap_bf16(&p->tm_v, a.v, 4, dims, strides, box, true);
  if (e != cudaSuccess) return e;
  p->out = o;
  p->B = (int)a.B; p->H = (int)a.H; p->S = (int)a.S;
  p->causal = a.causal;
  p->scale_log2 = (float)(1.4426950408889634 / sqrt((double)a.D));
  const int64_t num_q = (a.S + BQ - 1) / BQ, pairs = (num_q + 1) / 2, n_super = a.B * a.H * ((pairs + 1) / 2);
  p->grid = (int)(n_super < sm_count ? n_super : sm_count);
  return cudaSuccess;
}

cudaError_t launch_attention_tc2(const AttnTcPlan& p, cudaStream_t s) {
  static SmemOptIn opt_in;
  {
    cudaError_t e = opt_in.ensure(ATTN2_SMEM, attention_tc2_kernel);
    if (e != cudaSuccess) return e;
  }
  LaunchCfg lc(PDL_ATTENTION, dim3((unsigned)p.grid), dim3(THREADS), ATTN2_SMEM, s);
  return cudaLaunchKernelEx(&lc.cfg, attention_tc2_kernel, p.tm_q, p.tm_k, p.tm_v, (__nv_bfloat16*)p.out, p.B, p.H, p.S, p.causal ? 1 : 0, p.scale_log2,
                            kernel_status_ptr());
}

}  // namespace mk
