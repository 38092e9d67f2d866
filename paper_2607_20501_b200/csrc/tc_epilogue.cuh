// Epilogue shared by the tensor-core kernels.
//
// An epilogue warp owns 32 accumulator rows (one per lane, straight from tcgen05.ld) and walks its
// share of the tile 32 columns at a time.  Three things keep it off the critical path:
//   * no dependent global load inside a chunk: the tile's bias slice is copied to shared memory when
//     the warp starts the tile (before it waits for the accumulator), and a residual chunk is
//     fetched into registers one chunk ahead (a global load under TMA traffic costs ~1 us of
//     latency, and with one warp per scheduler nothing else would hide it);
//   * coalesced global access: a lane's own 64 bytes sit 2*N bytes from its neighbour's, so stores
//     (and residual loads) go through a shared-memory transpose and each instruction moves
//     8 rows x 64 contiguous bytes instead of 32 half-filled sectors;
//   * hardware-approximate tanh / exp2 (the output is bf16, whose half-ulp of 2^-9 dwarfs their 2^-11
//     relative error).
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

// Elementwise program on 32 consecutive columns of one row.  bias32 / res_row: the 64 bytes of bias /
// residual for these columns in shared memory (null: read them from global memory).
__device__ __forceinline__ void epi32(const EpiProgram& p, float (&v)[32], int64_t row, int64_t col0, int64_t ld, const uint8_t* bias32,
                                      const uint8_t* res_row) {
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
        const __nv_bfloat16* r = res_row ? reinterpret_cast<const __nv_bfloat16*>(res_row)
                                         : reinterpret_cast<const __nv_bfloat16*>(o.ptr) + row * ld + col0;
#pragma unroll
        for (int j = 0; j < 32; j += 8) {
          float t[8];
          ld_vec(r + j, t);
#pragma unroll
          for (int q = 0; q < 8; ++q) v[j + q] += t[q];
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
  int lane;
  __device__ __forceinline__ void init(uint8_t* warp_smem, const EpiProgram& p, int lane_) {
    stage = warp_smem;
    bias = warp_smem + EPI_WARP_STAGE;
    bias_idx = epi_single_index(p, EPI_BIAS);
    res_idx = epi_single_index(p, EPI_RESIDUAL);
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
  // per instruction).  A chunk that is ragged in N is left to the element-wise path.
  template <typename RowMap>
  __device__ __forceinline__ void prefetch_res(const EpiProgram& p, RowMap rowmap, int64_t col0, int64_t n_cols, uint4 (&regs)[4]) {
    if (res_idx < 0 || col0 + 32 > n_cols) return;
    const __nv_bfloat16* res = reinterpret_cast<const __nv_bfloat16*>(p.op[res_idx].ptr);
    const int sub_row = lane >> 2, seg = lane & 3;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int64_t gr = rowmap(sub_row + 8 * i);
      regs[i] = gr >= 0 ? *reinterpret_cast<const uint4*>(res + gr * n_cols + col0 + seg * 8) : make_uint4(0, 0, 0, 0);
    }
  }
  // One chunk: program, bf16 pack, transposed coalesced store.
  //   v            the lane's fp32 values for columns [col0, col0 + 32) of its row
  //   bias_off     offset of col0 inside the bias slice loaded by load_bias
  //   rowmap(r)    global row of warp-local row r in [0, 32), or -1 if that row is not stored
  //   res_regs     this chunk's residual (from prefetch_res); on return the next chunk's, if next_col0 >= 0
  template <typename RowMap>
  __device__ __forceinline__ void chunk_out(const EpiProgram& epi, float (&v)[32], RowMap rowmap, __nv_bfloat16* __restrict__ out,
                                            int64_t col0, int bias_off, int64_t n_cols, uint4 (&res_regs)[4], int64_t next_col0) {
    if (col0 >= n_cols) return;  // warp-uniform
    const int64_t my_row = rowmap(lane);
    const int sub_row = lane >> 2, seg = lane & 3;  // transposed role: 8 rows x 4 segments of 16 B per pass
    if (col0 + 32 <= n_cols) {
      const uint8_t* res_row = nullptr;
      if (res_idx >= 0) {
#pragma unroll
        for (int i = 0; i < 4; ++i) *reinterpret_cast<uint4*>(stage + (sub_row + 8 * i) * EPI_ROW_PITCH + seg * 16) = res_regs[i];
        __syncwarp();
        res_row = stage + lane * EPI_ROW_PITCH;  // only this lane reads, then overwrites, its own row
        if (next_col0 >= 0) prefetch_res(epi, rowmap, next_col0, n_cols, res_regs);
      }
      if (my_row >= 0) epi32(epi, v, my_row, col0, n_cols, bias_idx >= 0 ? bias + bias_off * 2 : nullptr, res_row);
      uint4* dst = reinterpret_cast<uint4*>(stage + lane * EPI_ROW_PITCH);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        uint4 pk;
        pk.x = pack_bf16x2(v[8 * j + 0], v[8 * j + 1]);
        pk.y = pack_bf16x2(v[8 * j + 2], v[8 * j + 3]);
        pk.z = pack_bf16x2(v[8 * j + 4], v[8 * j + 5]);
        pk.w = pack_bf16x2(v[8 * j + 6], v[8 * j + 7]);
        dst[j] = pk;
      }
      __syncwarp();
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int r = sub_row + 8 * i;
        const int64_t gr = rowmap(r);
        if (gr >= 0)
          *reinterpret_cast<uint4*>(out + gr * n_cols + col0 + seg * 8) = *reinterpret_cast<const uint4*>(stage + r * EPI_ROW_PITCH + seg * 16);
      }
      __syncwarp();
    } else {
      // ragged last chunk of the row: element by element, operands from global memory
      // (fully unrolled with a predicate: a run-time index into v[] would push the whole array, for its
      // whole lifetime, out of registers into local memory)
      if (my_row >= 0) {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (col0 + j < n_cols) out[my_row * n_cols + col0 + j] = __float2bfloat16_rn(epi_apply(epi, v[j], my_row, col0 + j, n_cols));
      }
      if (res_idx >= 0 && next_col0 >= 0) prefetch_res(epi, rowmap, next_col0, n_cols, res_regs);
    }
  }
};

}  // namespace mk
