// Launch plans of the tensor-core kernels: TMA descriptors are encoded once when a submodule is
// planned and reused by every forward, so a launch does no host-side encoding.
#pragma once

#include <cuda.h>

#include "kernels.h"

namespace mk {

struct GemmTcPlan {
  CUtensorMap tm_a, tm_b;
  void* out = nullptr;
  int m = 0, n = 0, k = 0;  // n = output columns
  bool swiglu = false;
  int grid = 0;
  EpiProgram epi;
};
// A [m, k] row-major; W stored [n, k] row-major ([2n, k] = [gate ; up] rows with swiglu); bf16.
// Needs k % 8 == 0 and n % 8 == 0 (16-byte rows for TMA and for the vector stores).
cudaError_t gemm_tc_plan(GemmTcPlan* p, const void* a, const void* w_nk, void* y, int64_t m, int64_t n, int64_t k, bool swiglu,
                         const EpiProgram& epi, int sm_count);
cudaError_t launch_gemm_tc(const GemmTcPlan& p, cudaStream_t s);

}  // namespace mk

namespace mk {
// Two-SM form (CTA pairs, tcgen05 cta_group::2, 256x256 tiles); same contract as gemm_tc_plan.
cudaError_t gemm_tc2_plan(GemmTcPlan* p, const void* a, const void* w_nk, void* y, int64_t m, int64_t n, int64_t k, bool swiglu,
                          const EpiProgram& epi, int sm_count);
cudaError_t launch_gemm_tc2(const GemmTcPlan& p, cudaStream_t s);
}  // namespace mk
