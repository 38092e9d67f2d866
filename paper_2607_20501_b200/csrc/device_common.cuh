// Device helpers shared by the kernels: storage conversion, 128-bit access, warp reductions and the
// elementwise-program interpreter.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kernels.h"

namespace mk {

// Programmatic dependent launch, device side.  pdl_launch_dependents(): the next kernel on the stream (if it was
// launched as a dependent) may start being scheduled once every CTA of this grid has said so or retired.
// pdl_wait(): block until every kernel this grid depends on has completed and its writes are visible; a no-op
// for a grid launched in plain stream order.  Nothing produced by an earlier kernel may be read before it.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename T> struct Elem;
template <> struct Elem<float> {
  static constexpr int VEC = 4;  // elements per 128-bit access
  __device__ __forceinline__ static float ld(const float* p) { return *p; }
  __device__ __forceinline__ static void st(float* p, float v) { *p = v; }
};
template <> struct Elem<__nv_bfloat16> {
  static constexpr int VEC = 8;
  __device__ __forceinline__ static float ld(const __nv_bfloat16* p) { return __bfloat162float(*p); }
  __device__ __forceinline__ static void st(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
};

// 128-bit load of VEC consecutive elements into fp32 registers (pointer 16-byte aligned)
__device__ __forceinline__ void ld_vec(const float* p, float (&v)[4]) {
  const float4 t = *reinterpret_cast<const float4*>(p);
  v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}
__device__ __forceinline__ void ld_vec(const __nv_bfloat16* p, float (&v)[8]) {
  const uint4 t = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}
// raw 128-bit load now, conversion later (software pipelining: the next row's loads are in flight
// while the current row is reduced)
__device__ __forceinline__ uint4 ld_raw(const void* p) { return *reinterpret_cast<const uint4*>(p); }
__device__ __forceinline__ void unpack_raw(const uint4& t, float (&v)[4]) {
  v[0] = __uint_as_float(t.x); v[1] = __uint_as_float(t.y); v[2] = __uint_as_float(t.z); v[3] = __uint_as_float(t.w);
}
__device__ __forceinline__ void unpack_raw(const uint4& t, float (&v)[8]) {
  const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}
__device__ __forceinline__ void st_vec(float* p, const float (&v)[4]) {
  *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
}
__device__ __forceinline__ void st_vec(__nv_bfloat16* p, const float (&v)[8]) {
  uint4 t;
  t.x = pack_bf16x2(v[0], v[1]);
  t.y = pack_bf16x2(v[2], v[3]);
  t.z = pack_bf16x2(v[4], v[5]);
  t.w = pack_bf16x2(v[6], v[7]);
  *reinterpret_cast<uint4*>(p) = t;
}

// NV fp32 registers -> NV consecutive elements of type TO (16-byte aligned destination)
template <typename TO, int NV>
__device__ __forceinline__ void st_vec_as(TO* p, const float (&v)[NV]) {
  if constexpr (sizeof(TO) == 4) {
#pragma unroll
    for (int j = 0; j < NV; j += 4) *reinterpret_cast<float4*>(reinterpret_cast<float*>(p) + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
  } else {
#pragma unroll
    for (int j = 0; j < NV; j += 8) {
      uint4 t;
      t.x = pack_bf16x2(v[j], v[j + 1]);
      t.y = pack_bf16x2(v[j + 2], v[j + 3]);
      t.z = pack_bf16x2(v[j + 4], v[j + 5]);
      t.w = pack_bf16x2(v[j + 6], v[j + 7]);
      *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p) + j) = t;
    }
  }
}
// NV consecutive elements of type TI, raw (16-byte pieces), and their later conversion to fp32
template <typename TI, int NV> struct RawVec {
  static constexpr int N16 = NV * (int)sizeof(TI) / 16;
  uint4 r[N16];
  __device__ __forceinline__ void load(const TI* p) {
#pragma unroll
    for (int i = 0; i < N16; ++i) r[i] = *reinterpret_cast<const uint4*>(reinterpret_cast<const uint8_t*>(p) + 16 * i);
  }
  __device__ __forceinline__ void unpack(float (&v)[NV]) const {
    if constexpr (sizeof(TI) == 4) {
#pragma unroll
      for (int i = 0; i < N16; ++i) {
        v[4 * i] = __uint_as_float(r[i].x); v[4 * i + 1] = __uint_as_float(r[i].y);
        v[4 * i + 2] = __uint_as_float(r[i].z); v[4 * i + 3] = __uint_as_float(r[i].w);
      }
    } else {
#pragma unroll
      for (int i = 0; i < N16; ++i) {
        const uint32_t w[4] = {r[i].x, r[i].y, r[i].z, r[i].w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          v[8 * i + 2 * k] = __uint_as_float(w[k] << 16);
          v[8 * i + 2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
        }
      }
    }
  }
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

__device__ __forceinline__ float gelu_tanh_f(float x) {
  const float u = 0.7978845608028654f * (x + 0.044715f * x * x * x);
  return 0.5f * x * (1.0f + tanhf(u));
}
__device__ __forceinline__ float gelu_erf_f(float x) { return 0.5f * x * (1.0f + erff(x * 0.7071067811865476f)); }
__device__ __forceinline__ float silu_f(float x) { return x / (1.0f + __expf(-x)); }
// hardware tanh (relative error ~2^-11): only where the result is stored as bf16 (half-ulp 2^-9)
__device__ __forceinline__ float gelu_tanh_bf16_f(float x) {
  const float u = 0.7978845608028654f * (x + 0.044715f * x * x * x);
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(u));
  return 0.5f * x * (1.0f + t);
}

__device__ __forceinline__ float epi_ptr_ld(const void* p, int dtype, int64_t i) {
  return dtype == DT_F32 ? reinterpret_cast<const float*>(p)[i]
                         : __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[i]);
}

// Run the program on one value sitting at (row, col) of a [*, ld] output.
__device__ __forceinline__ float epi_apply(const EpiProgram& p, float v, int64_t row, int64_t col, int64_t ld) {
  for (int i = 0; i < p.n; ++i) {
    const EpiOp& o = p.op[i];
    switch (o.kind) {
      case EPI_BIAS: v += epi_ptr_ld(o.ptr, p.dtype, col); break;
      case EPI_RELU: v = fmaxf(v, 0.0f); break;
      case EPI_GELU_TANH: v = gelu_tanh_f(v); break;
      case EPI_GELU_ERF: v = gelu_erf_f(v); break;
      case EPI_SILU: v = silu_f(v); break;
      case EPI_SCALE: v *= o.a; break;
      case EPI_CLAMP: v = fminf(fmaxf(v, o.a), o.b); break;
      case EPI_RESIDUAL: v += epi_ptr_ld(o.ptr, o.ptr_dtype, row * ld + col); break;
      default: break;
    }
  }
  return v;
}

// The same with the value of one bias op (index pre_idx, -1: none) already in a register: kernels whose whole time is
// latency ask for it in their first instructions instead of at the end.
__device__ __forceinline__ float epi_apply_pre(const EpiProgram& p, float v, int64_t row, int64_t col, int64_t ld, int pre_idx, float pre_val) {
  for (int i = 0; i < p.n; ++i) {
    const EpiOp& o = p.op[i];
    switch (o.kind) {
      case EPI_BIAS: v += i == pre_idx ? pre_val : epi_ptr_ld(o.ptr, p.dtype, col); break;
      case EPI_RELU: v = fmaxf(v, 0.0f); break;
      case EPI_GELU_TANH: v = gelu_tanh_f(v); break;
      case EPI_GELU_ERF: v = gelu_erf_f(v); break;
      case EPI_SILU: v = silu_f(v); break;
      case EPI_SCALE: v *= o.a; break;
      case EPI_CLAMP: v = fminf(fmaxf(v, o.a), o.b); break;
      case EPI_RESIDUAL: v += epi_ptr_ld(o.ptr, o.ptr_dtype, row * ld + col); break;
      default: break;
    }
  }
  return v;
}

// Run the program on NV consecutive columns of one row; col0 is a multiple of NV and the program's
// pointers are 16-byte aligned, so bias and residual are fetched with 128-bit loads.
template <typename T, int NV>
__device__ __forceinline__ void epi_apply_vec(const EpiProgram& p, float (&v)[NV], int64_t row, int64_t col0, int64_t ld) {
  static_assert(NV % Elem<T>::VEC == 0, "vector width");
  constexpr int VE = Elem<T>::VEC;
  for (int i = 0; i < p.n; ++i) {
    const EpiOp& o = p.op[i];
    switch (o.kind) {
      case EPI_BIAS: {
        const T* b = reinterpret_cast<const T*>(o.ptr) + col0;
#pragma unroll
        for (int j = 0; j < NV; j += VE) {
          float t[VE];
          ld_vec(b + j, t);
#pragma unroll
          for (int q = 0; q < VE; ++q) v[j + q] += t[q];
        }
        break;
      }
      case EPI_RESIDUAL: {
        if (o.ptr_dtype == DT_F32) {   // an fp32 residual stream next to bf16 activations
          const float* r = reinterpret_cast<const float*>(o.ptr) + row * ld + col0;
#pragma unroll
          for (int j = 0; j < NV; j += 4) {
            float t[4];
            ld_vec(r + j, t);
#pragma unroll
            for (int q = 0; q < 4; ++q) v[j + q] += t[q];
          }
        } else {
          const T* r = reinterpret_cast<const T*>(o.ptr) + row * ld + col0;
#pragma unroll
          for (int j = 0; j < NV; j += VE) {
            float t[VE];
            ld_vec(r + j, t);
#pragma unroll
            for (int q = 0; q < VE; ++q) v[j + q] += t[q];
          }
        }
        break;
      }
      case EPI_RELU:
#pragma unroll
        for (int j = 0; j < NV; ++j) v[j] = fmaxf(v[j], 0.0f);
        break;
      case EPI_GELU_TANH:
#pragma unroll
        for (int j = 0; j < NV; ++j) v[j] = sizeof(T) == 2 ? gelu_tanh_bf16_f(v[j]) : gelu_tanh_f(v[j]);
        break;
      case EPI_GELU_ERF:
#pragma unroll
        for (int j = 0; j < NV; ++j) v[j] = gelu_erf_f(v[j]);
        break;
      case EPI_SILU:
#pragma unroll
        for (int j = 0; j < NV; ++j) v[j] = silu_f(v[j]);
        break;
      case EPI_SCALE:
#pragma unroll
        for (int j = 0; j < NV; ++j) v[j] *= o.a;
        break;
      case EPI_CLAMP:
#pragma unroll
        for (int j = 0; j < NV; ++j) v[j] = fminf(fmaxf(v[j], o.a), o.b);
        break;
      default: break;
    }
  }
}

}  // namespace mk
