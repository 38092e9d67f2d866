// Epilogue shared by the tensor-core kernels: the elementwise program on 32 consecutive fp32
// accumulator columns of one row, with hardware-approximate tanh / exp2 (the output is bf16, whose
// half-ulp of 2^-9 dwarfs their 2^-11 relative error), and the bf16 row store.
#pragma once

#include "device_common.cuh"
#include "tc_common.cuh"

namespace mk {

__device__ __forceinline__ float gelu_fast(float x) {
  const float u = 0.7978845608028654f * (x + 0.044715f * x * x * x);
  return 0.5f * x * (1.0f + tc::tanh_fast(u));
}
__device__ __forceinline__ float silu_fast(float x) { return __fdividef(x, 1.0f + tc::ex2_fast(-1.4426950408889634f * x)); }

// elementwise program on 32 consecutive columns of one row, fast transcendental forms (bf16 output)
__device__ __forceinline__ void epi32(const EpiProgram& p, float (&v)[32], int64_t row, int64_t col0, int64_t ld) {
  for (int i = 0; i < p.n; ++i) {
    const EpiOp& o = p.op[i];
    switch (o.kind) {
      case EPI_BIAS: {
        const __nv_bfloat16* b = reinterpret_cast<const __nv_bfloat16*>(o.ptr) + col0;
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
        const __nv_bfloat16* r = reinterpret_cast<const __nv_bfloat16*>(o.ptr) + row * ld + col0;
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

// fp32 accumulator chunk -> program -> bf16 -> global, for columns [col0, col0 + 32) of `row`
__device__ __forceinline__ void epi_store32(const EpiProgram& epi, float (&v)[32], __nv_bfloat16* __restrict__ out, int64_t row,
                                            int64_t col0, int64_t M, int64_t N) {
  if (row >= M || col0 >= N) return;
  __nv_bfloat16* orow = out + row * N;
  if (col0 + 32 <= N) {
    epi32(epi, v, row, col0, N);
#pragma unroll
    for (int j = 0; j < 32; j += 8) {
      uint4 pk;
      pk.x = pack_bf16x2(v[j], v[j + 1]);
      pk.y = pack_bf16x2(v[j + 2], v[j + 3]);
      pk.z = pack_bf16x2(v[j + 4], v[j + 5]);
      pk.w = pack_bf16x2(v[j + 6], v[j + 7]);
      *reinterpret_cast<uint4*>(orow + col0 + j) = pk;
    }
  } else {
    for (int j = 0; j < 32 && col0 + j < N; ++j) orow[col0 + j] = __float2bfloat16_rn(epi_apply(epi, v[j], row, col0 + j, N));
  }
}

}  // namespace mk
