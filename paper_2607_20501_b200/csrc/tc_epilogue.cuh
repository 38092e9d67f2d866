// Epilogue shared by the tensor-core kernels.
//
// An epilogue warp owns 32 accumulator rows (one per lane, straight from tcgen05.ld) and walks its
// share of the tile 32 columns at a time.  Three things keep it off the critical path:
//   * no dependent global load inside a chunk: the tile's bias slice is copied to shared memory when
//     the warp starts the tile (before it waits for the accumulator), and a residual chunk is
//     fetched into registers one chunk ahead (a global load under TMA traffic costs ~1 us of
//     latency, and with one or two warps per scheduler nothing else would hide it);
//   * coalesced global access: a lane's own bytes sit a whole output row from its neighbour's, so
//     stores (and residual loads) go through a shared-memory transpose, one 32-row x 64-byte slab at
//     a time, and each instruction moves 8 rows x 64 contiguous bytes instead of 32 half-filled
//     sectors;
//   * hardware-approximate tanh / exp2 (relative error ~2^-11, below bf16's half-ulp of 2^-9).
// The residual operand and the output may each be bf16 or fp32 (an fp32 residual stream next to
// bf16 activations): an fp32 chunk is two slabs.
// Everything indexes the accumulator array with compile-time constants: one run-time index would
// move the whole array, for its whole lifetime, from registers to local memory.
#pragma once

#include "device_common.cuh"
#include "tc_common.cuh"

namespace mk {

constexpr int EPI_ROW_PITCH = 80;                   // bytes per staged row: 64 + 16 of padding (bank-conflict free)
constexpr int EPI_WARP_STAGE = 32 * EPI_ROW_PITCH;  // transpose buffer per epilogue warp
constexpr int EPI_WARP_BIAS = 512;                  // up to 256 bf16 bias values per warp
constexpr int EPI_WARP_BYTES = EPI_WARP_STAGE + EPI_WARP_BIAS;

__device__ __forceinline__ float gelu_fast(float x) {
  const float u = 0.7978845608028654f * (x + 0.044715f * x * x * x);
  return 0.5f * x * (1.0f + tc::tanh_fast(u));
}
__device__ __forceinline__ float silu_fast(float x) { return __fdividef(x, 1.0f + tc::ex2_fast(-1.4426950408889634f * x)); }

// Elementwise program on 32 consecutive columns of one row.  bias32: the 64 bytes of bias for these
// columns in shared memory (null: read them from global memory).  res_mode 1: the row's 32 residual
// values as bf16 in ra; 2: as fp32 in ra (columns 0..15) and rb (16..31); 0: a residual op reads
// global memory.
__device__ __forceinline__ void epi32(const EpiProgram& p, float (&v)[32], int64_t row, int64_t col0, int64_t ld, const uint8_t* bias32,
                                      int res_mode, const uint4 (&ra)[4], const uint4 (&rb)[4]) {
#pragma unroll 1
  for (int i = 0; i < p.n; ++i) {
    const EpiOp& o = p.op[i];
    switch (o.kind) {
      case EPI_BIAS: {
        const __nv_bfloat16* b = bias32 ? reinterpret_cast<const __nv_bfloat16*>(bias32) : reinterpret_cast<const __nv_bfloat16*>(o.ptr) + col0;
#pragma unroll
        for (int j = 0; j < 32; j += 8) {
          float t[8];
          ld_vec(b + j, t);
#pragma unroll
          for (int q = 0; q < 8; ++q) v[j + q] += t[q];
        }
        break;
      }
      case EPI_RESIDUAL: {
        if (res_mode == 1) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const uint32_t w[4] = {ra[i].x, ra[i].y, ra[i].z, ra[i].w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              v[8 * i + 2 * k] += __uint_as_float(w[k] << 16);
              v[8 * i + 2 * k + 1] += __uint_as_float(w[k] & 0xffff0000u);
            }
          }
        } else if (res_mode == 2) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            v[4 * i] += __uint_as_float(ra[i].x); v[4 * i + 1] += __uint_as_float(ra[i].y);
            v[4 * i + 2] += __uint_as_float(ra[i].z); v[4 * i + 3] += __uint_as_float(ra[i].w);
            v[16 + 4 * i] += __uint_as_float(rb[i].x); v[16 + 4 * i + 1] += __uint_as_float(rb[i].y);
            v[16 + 4 * i + 2] += __uint_as_float(rb[i].z); v[16 + 4 * i + 3] += __uint_as_float(rb[i].w);
          }
        } else if (o.ptr_dtype == DT_F32) {
          const float* r = reinterpret_cast<const float*>(o.ptr) + row * ld + col0;
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            float t[4];
            ld_vec(r + j, t);
#pragma unroll
            for (int q = 0; q < 4; ++q) v[j + q] += t[q];
          }
        } else {
          const __nv_bfloat16* r = reinterpret_cast<const __nv_bfloat16*>(o.ptr) + row * ld + col0;
#pragma unroll
          for (int j = 0; j < 32; j += 8) {
            float t[8];
            ld_vec(r + j, t);
#pragma unroll
            for (int q = 0; q < 8; ++q) v[j + q] += t[q];
          }
        }
        break;
      }
      case EPI_RELU:
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = fmaxf(v[j], 0.0f);
        break;
      case EPI_GELU_TANH:
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = gelu_fast(v[j]);
        break;
      case EPI_GELU_ERF:
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = gelu_erf_f(v[j]);   // fully unrolled like the rest: a run-time index would put v in local memory
        break;
      case EPI_SILU:
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = silu_fast(v[j]);
        break;
      case EPI_SCALE:
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] *= o.a;
        break;
      case EPI_CLAMP:
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = fminf(fmaxf(v[j], o.a), o.b);
        break;
      default: break;
    }
  }
}

// The elementwise program arrives as a kernel parameter and is interpreted per 32-column chunk through a
// reference.  The tensor-core kernels copy it to shared memory once, before their first __syncthreads, so
// the interpreter's run-time-indexed reads are shared-memory broadcasts whatever the compiler makes of a
// reference to the parameter space.  (Measured: no change in kernel time; kept for the predictable latency.)
__device__ __forceinline__ void epi_copy_to_smem(EpiProgram* dst, const EpiProgram& src, int tid, int nthreads) {
  constexpr int WORDS = (int)(sizeof(EpiProgram) / 4);
  static_assert(sizeof(EpiProgram) % 4 == 0, "EpiProgram is copied word by word");
  const uint32_t* s = reinterpret_cast<const uint32_t*>(&src);
  uint32_t* d = reinterpret_cast<uint32_t*>(dst);
  for (int i = tid; i < WORDS; i += nthreads) d[i] = s[i];
}

// index of the op of kind `kind` if the program has exactly one, else -1 (then that kind is read
// straight from global memory inside epi32)
__device__ __forceinline__ int epi_single_index(const EpiProgram& p, int kind) {
  int idx = -1, cnt = 0;
  for (int i = 0; i < p.n; ++i)
    if (p.op[i].kind == kind) { idx = i; ++cnt; }
  return cnt == 1 ? idx : -1;
}

struct EpiWarp {
  uint8_t* stage;  // EPI_WARP_STAGE bytes, this warp's transpose buffer
  uint8_t* bias;   // EPI_WARP_BIAS bytes, this warp's copy of the tile's bias slice
  int bias_idx, res_idx;
  bool res_f32, out_f32;
  bool store = true;   // false: chunk_out applies the program to v and stores nothing (the caller goes on with v)
  int lane;
#ifdef MK_TRACE
  unsigned long long* tr = nullptr;   // trace builds: where the chunk being timed leaves its clock readings (null: not timed)
#define MK_TRC(k) do { if (tr) tr[k] = (unsigned long long)clock64(); } while (0)
#else
#define MK_TRC(k) do {} while (0)
#endif
  __device__ __forceinline__ void init(uint8_t* warp_smem, const EpiProgram& p, int lane_, bool out_f32_) {
    stage = warp_smem;
    bias = warp_smem + EPI_WARP_STAGE;
    bias_idx = epi_single_index(p, EPI_BIAS);
    res_idx = epi_single_index(p, EPI_RESIDUAL);
    res_f32 = res_idx >= 0 && p.op[res_idx].ptr_dtype == DT_F32;
    out_f32 = out_f32_;
    lane = lane_;
  }
  // Copy bias[col_base, col_base + width) (width <= 256) into shared memory; call before waiting for
  // the accumulator.  Segments past n_cols are skipped (their columns are never stored).
  __device__ __forceinline__ void load_bias(const EpiProgram& p, int64_t col_base, int width, int64_t n_cols) {
    if (bias_idx < 0) return;
    __syncwarp();
    const int64_t c = col_base + lane * 8;
    if (lane * 8 < width && c + 8 <= n_cols)
      *reinterpret_cast<uint4*>(bias + lane * 16) = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p.op[bias_idx].ptr) + c);
    __syncwarp();
  }
  // Fetch the residual chunk [32 rows x 32 columns at col0] into registers, coalesced (8 rows x 64 B
  // per instruction; an fp32 chunk is two 64-byte slabs per row).  A chunk that is ragged in N is left
  // to the element-wise path.
  template <typename RowMap>
  __device__ __forceinline__ void prefetch_res(const EpiProgram& p, RowMap rowmap, int64_t col0, int64_t n_cols, uint4 (&regs)[8]) {
    if (res_idx < 0 || col0 + 32 > n_cols) return;
    const uint8_t* res = reinterpret_cast<const uint8_t*>(p.op[res_idx].ptr);
    const int sub_row = lane >> 2, seg = lane & 3;
    const int esz = res_f32 ? 4 : 2;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int64_t gr = rowmap(sub_row + 8 * i);
      const uint8_t* src = res + (gr * n_cols + col0) * esz + seg * 16;
      regs[i] = gr >= 0 ? *reinterpret_cast<const uint4*>(src) : make_uint4(0, 0, 0, 0);
      if (res_f32) regs[4 + i] = gr >= 0 ? *reinterpret_cast<const uint4*>(src + 64) : make_uint4(0, 0, 0, 0);
    }
  }
  // registers (transposed role) -> staging -> this lane's own 64 bytes.  No barrier after the own-row
  // reads: whatever follows either touches only the lane's own row or starts with its own barrier.
  __device__ __forceinline__ void slab_to_own_row(const uint4& r0, const uint4& r1, const uint4& r2, const uint4& r3, uint4 (&mine)[4],
                                                  bool sync_first) {
    const int sub_row = lane >> 2, seg = lane & 3;
    if (sync_first) __syncwarp();
    *reinterpret_cast<uint4*>(stage + (sub_row + 0) * EPI_ROW_PITCH + seg * 16) = r0;
    *reinterpret_cast<uint4*>(stage + (sub_row + 8) * EPI_ROW_PITCH + seg * 16) = r1;
    *reinterpret_cast<uint4*>(stage + (sub_row + 16) * EPI_ROW_PITCH + seg * 16) = r2;
    *reinterpret_cast<uint4*>(stage + (sub_row + 24) * EPI_ROW_PITCH + seg * 16) = r3;
    __syncwarp();
#pragma unroll
    for (int i = 0; i < 4; ++i) mine[i] = *reinterpret_cast<const uint4*>(stage + lane * EPI_ROW_PITCH + i * 16);
  }
  // this lane's own 64 bytes -> staging -> coalesced global store at byte offset `byte_off` of each row
  template <typename RowMap>
  __device__ __forceinline__ void own_row_to_global(const uint4 (&mine)[4], RowMap rowmap, uint8_t* out, int64_t row_bytes, int64_t byte_off) {
    const int sub_row = lane >> 2, seg = lane & 3;
#pragma unroll
    for (int i = 0; i < 4; ++i) *reinterpret_cast<uint4*>(stage + lane * EPI_ROW_PITCH + i * 16) = mine[i];
    __syncwarp();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int r = sub_row + 8 * i;
      const int64_t gr = rowmap(r);
      if (gr >= 0) *reinterpret_cast<uint4*>(out + gr * row_bytes + byte_off + seg * 16) = *reinterpret_cast<const uint4*>(stage + r * EPI_ROW_PITCH + seg * 16);
    }
    __syncwarp();
  }
  // this lane's own 64 bytes -> staging (64-byte rows, the bulk store's 64-byte swizzle) -> one asynchronous
  // bulk tensor store of the 32 x 64-byte block at column x (elements), row y; lane 0 issues and tracks it.
  // Rows and columns beyond the tensor are clipped by the copy engine.
  __device__ __forceinline__ void own_row_to_global_bulk(const uint4 (&mine)[4], const CUtensorMap* tm, int32_t x, int32_t y) {
    const int f = (lane >> 1) & 3;
#pragma unroll
    for (int i = 0; i < 4; ++i) *reinterpret_cast<uint4*>(stage + lane * 64 + ((i ^ f) * 16)) = mine[i];
    MK_TRC(4);
    tc::fence_proxy_async();
    __syncwarp();
    MK_TRC(5);
    if (lane == 0) {
      tc::tma_store_2d(tm, stage, x, y);
      tc::tma_store_commit();
    }
    MK_TRC(6);
  }
  // One chunk: program, pack, transposed coalesced store.
  //   v            the lane's fp32 values for columns [col0, col0 + 32) of its row
  //   bias_off     offset (elements) of col0 inside the bias slice loaded by load_bias
  //   rowmap(r)    global row of warp-local row r in [0, 32), or -1 if that row is not stored
  //   res_regs     this chunk's residual (from prefetch_res); on return the next chunk's, if next_col0 >= 0
  //   tm_store     if not null (a map of the output in its own type, rows of the warp consecutive from global row y0):
  //                the block leaves by bulk tensor stores (one for bf16, two for fp32) instead of 16-byte stores
  template <typename RowMap>
  __device__ __forceinline__ void chunk_out(const EpiProgram& epi, float (&v)[32], RowMap rowmap, void* __restrict__ out_v, int64_t col0,
                                            int bias_off, int64_t n_cols, uint4 (&res_regs)[8], int64_t next_col0,
                                            const CUtensorMap* tm_store = nullptr, int64_t y0 = 0) {
    if (col0 >= n_cols) return;  // warp-uniform
    // the residual through registers: this chunk's values were fetched one chunk ago, the next chunk's are fetched now
    auto get = [&](uint4 (&ra)[4], uint4 (&rb)[4]) -> int {
      if (res_idx < 0) return 0;
      slab_to_own_row(res_regs[0], res_regs[1], res_regs[2], res_regs[3], ra, false);
      if (res_f32) slab_to_own_row(res_regs[4], res_regs[5], res_regs[6], res_regs[7], rb, true);
      if (next_col0 >= 0) prefetch_res(epi, rowmap, next_col0, n_cols, res_regs);
      return res_f32 ? 2 : 1;
    };
    auto skip = [&]() {
      if (res_idx >= 0 && next_col0 >= 0) prefetch_res(epi, rowmap, next_col0, n_cols, res_regs);
    };
    chunk_out_from(epi, v, rowmap, out_v, col0, bias_off, n_cols, get, skip, tm_store, y0);
  }
  // The same with the residual supplied by the caller:
  //   get(ra, rb)  called once for a chunk that is stored whole: fills the lane's own 32 residual values (bf16 in ra:
  //                returns 1; fp32 in ra, rb: returns 2; no residual operand prepared: returns 0) and may start the
  //                fetch of a later chunk
  //   skip()       called instead for a chunk that is ragged in N (its residual is read element by element)
  template <typename RowMap, typename Get, typename Skip>
  __device__ __forceinline__ void chunk_out_from(const EpiProgram& epi, float (&v)[32], RowMap rowmap, void* __restrict__ out_v, int64_t col0,
                                                 int bias_off, int64_t n_cols, Get get, Skip skip, const CUtensorMap* tm_store = nullptr,
                                                 int64_t y0 = 0) {
    if (col0 >= n_cols) {  // warp-uniform
      skip();
      return;
    }
    if (tm_store) {
      // the previous chunk's bulk store has finished reading the staging buffer (the residual slabs go through it too)
      if (lane == 0) tc::tma_store_wait_read();
      __syncwarp();
    }
    MK_TRC(1);
    const int64_t my_row = rowmap(lane);
    uint8_t* out = reinterpret_cast<uint8_t*>(out_v);
    if (col0 + 32 <= n_cols) {
      uint4 ra[4], rb[4];
      const int res_mode = get(ra, rb);
      MK_TRC(2);
      if (my_row >= 0) epi32(epi, v, my_row, col0, n_cols, bias_idx >= 0 ? bias + bias_off * 2 : nullptr, res_mode, ra, rb);
      MK_TRC(3);
      uint4 mine[4];
      if (!store) {
        // program only
      } else if (!out_f32) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          mine[j].x = pack_bf16x2(v[8 * j + 0], v[8 * j + 1]);
          mine[j].y = pack_bf16x2(v[8 * j + 2], v[8 * j + 3]);
          mine[j].z = pack_bf16x2(v[8 * j + 4], v[8 * j + 5]);
          mine[j].w = pack_bf16x2(v[8 * j + 6], v[8 * j + 7]);
        }
        if (tm_store) own_row_to_global_bulk(mine, tm_store, (int32_t)col0, (int32_t)y0);
        else own_row_to_global(mine, rowmap, out, n_cols * 2, col0 * 2);
      } else {
        // an fp32 chunk is two 64-byte slabs per row
#pragma unroll
        for (int j = 0; j < 4; ++j)
          mine[j] = make_uint4(__float_as_uint(v[4 * j]), __float_as_uint(v[4 * j + 1]), __float_as_uint(v[4 * j + 2]), __float_as_uint(v[4 * j + 3]));
        if (tm_store) own_row_to_global_bulk(mine, tm_store, (int32_t)col0, (int32_t)y0);
        else own_row_to_global(mine, rowmap, out, n_cols * 4, col0 * 4);
#pragma unroll
        for (int j = 0; j < 4; ++j)
          mine[j] = make_uint4(__float_as_uint(v[16 + 4 * j]), __float_as_uint(v[16 + 4 * j + 1]), __float_as_uint(v[16 + 4 * j + 2]),
                               __float_as_uint(v[16 + 4 * j + 3]));
        if (tm_store) {
          if (lane == 0) tc::tma_store_wait_read();   // the first slab has left the staging buffer
          __syncwarp();
          own_row_to_global_bulk(mine, tm_store, (int32_t)col0 + 16, (int32_t)y0);
        } else {
          own_row_to_global(mine, rowmap, out, n_cols * 4, col0 * 4 + 64);
        }
      }
    } else {
      // ragged last chunk of the row: element by element, operands from global memory
      if (my_row >= 0) {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (col0 + j < n_cols) {
            const float r = epi_apply(epi, v[j], my_row, col0 + j, n_cols);
            v[j] = r;   // callers that go on with the chunk (row statistics) see the values after the tail
            if (!store) continue;
            if (out_f32) reinterpret_cast<float*>(out)[my_row * n_cols + col0 + j] = r;
            else reinterpret_cast<__nv_bfloat16*>(out)[my_row * n_cols + col0 + j] = __float2bfloat16_rn(r);
          }
      }
      skip();
    }
  }
};

}  // namespace mk
