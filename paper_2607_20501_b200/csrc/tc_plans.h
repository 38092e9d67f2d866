// Launch plans of the tensor-core kernels: TMA descriptors are encoded once when a submodule is
// planned and reused by every forward, so a launch does no host-side encoding.
#pragma once

#include <cuda.h>

#include "kernels.h"

namespace mk {

// Row norm fused behind the GEMM's tail (LayerNorm or RMSNorm over the whole output row, which spans
// several tiles): every epilogue warp leaves per-row partial sums of what it stores and counts itself
// in; the warp that completes a block of 32 rows normalises those rows in place.
struct RowNormArgs {
  float* partials = nullptr;   // [m][2 * column tiles][2] = (sum, sum of squares) per row and epilogue-warp slot
  int* counters = nullptr;     // [row blocks of 32]; zeroed before every launch
  const void* gamma = nullptr; // bf16 [n] or null
  const void* beta = nullptr;  // bf16 [n] or null (LayerNorm only)
  float eps = 0.f;
  int mode = 0;                // RowMode
};

// RMSNorm folded across two GEMMs (the norm's reduction blocks fusion into ONE kernel, but not its arithmetic:
// rstd is a scalar per row, so (rstd x * gamma) W = rstd ((x * gamma) W)).  The GEMM that PRODUCES the norm's input
// also writes xg = bf16(x * gamma) and, per row and epilogue-warp slot, the sum of x^2 over the columns that warp
// stored; the GEMM that CONSUMES the norm's output takes xg as its A operand and multiplies every accumulator row
// by rstd = 1 / sqrt(sum of the row's partials / n + eps) before its own tail.  No pass over the activation is left.
struct PreNormArgs {
  // producer side (null: none)
  float* part_out = nullptr;      // [m][2 * column tiles] sums of squares
  void* xg = nullptr;             // bf16 [m, n]
  const void* gamma = nullptr;    // bf16 [n] or null
  // consumer side (null: none)
  const float* part_in = nullptr; // [m][slots_in]
  int slots_in = 0;
  float inv_n_in = 0.f;           // 1 / (row length of the normalised tensor)
  float eps_in = 0.f;
};

struct GemmTcPlan {
  CUtensorMap tm_a, tm_b;
  CUtensorMap tm_aux;       // producer of a folded pre-norm: store map of xg (never read otherwise)
  PreNormArgs pre;
  bool use_pre = false;
  RowNormArgs norm;         // used by the fused GEMM + row norm form only
  CUtensorMap tm_b_half;    // W with a box of half as many rows, for the half-width units of the last wave
  CUtensorMap tm_out;       // the output in its own type (bf16 or fp32), for the epilogue's bulk stores (use_tm_out)
  bool use_tm_out = false;
  bool res_ring = false;    // a bf16 residual is staged through shared memory two chunks ahead (one pipeline stage less)
  int tail_first = 0;       // tiles from this index on run as two half-width units (= tile count: none)
  int group_m = 16;         // tile rows walked together, column by column, so that their A rows and the W slabs stay in L2
  void* out = nullptr;
  bool out_f32 = false;     // output stored as fp32 (an fp32 residual stream), else bf16
  int m = 0, n = 0, k = 0;  // n = output columns
  bool swiglu = false;
  int grid = 0;
  EpiProgram epi;
};
// A [m, k] row-major; W stored [n, k] row-major ([2n, k] = [gate ; up] rows with swiglu); bf16.
// Needs k % 8 == 0 and n % 8 == 0 (16-byte rows for TMA and for the vector stores).
cudaError_t gemm_tc_plan(GemmTcPlan* p, const void* a, const void* w_nk, void* y, bool out_f32, int64_t m, int64_t n, int64_t k, bool swiglu,
                         const EpiProgram& epi, int sm_count);
cudaError_t launch_gemm_tc(const GemmTcPlan& p, cudaStream_t s);

}  // namespace mk

namespace mk {
// Two-SM form (CTA pairs, tcgen05 cta_group::2, 256x256 tiles); same contract as gemm_tc_plan.
cudaError_t gemm_tc2_plan(GemmTcPlan* p, const void* a, const void* w_nk, void* y, bool out_f32, int64_t m, int64_t n, int64_t k, bool swiglu,
                          const EpiProgram& epi, int sm_count);
cudaError_t launch_gemm_tc2(const GemmTcPlan& p, cudaStream_t s);
// The pair of GEMMs around a folded RMSNorm (see PreNormArgs).  Scratch: gemm_prenorm_scratch(m, n1) bytes =
// xg [m, n1] bf16 followed by the partial sums.  First plan: y1 = tail1(A W1) (bf16 or fp32), n1 columns; second:
// y2 = tail2(swiglu?(rmsnorm(y1; gamma, eps) W2)).
size_t gemm_prenorm_scratch(int64_t m, int64_t n1);
cudaError_t gemm_prenorm_pair_plan(GemmTcPlan* p1, GemmTcPlan* p2, const void* a, const void* w1_nk, void* y1, bool y1_f32, int64_t m, int64_t n1,
                                   int64_t k1, const EpiProgram& epi1, const void* gamma, float eps, const void* w2_nk, void* y2, int64_t n2,
                                   bool swiglu2, const EpiProgram& epi2, void* scratch, int sm_count);
// Fused GEMM + tail + row norm (bf16 out).  Scratch: gemm_rownorm_tc2_scratch(m, n) bytes, laid out by the plan.
size_t gemm_rownorm_tc2_scratch(int64_t m, int64_t n);
cudaError_t gemm_rownorm_tc2_plan(GemmTcPlan* p, const void* a, const void* w_nk, void* y, int64_t m, int64_t n, int64_t k,
                                  const EpiProgram& epi, int mode, const void* gamma, const void* beta, float eps, void* scratch,
                                  int sm_count);
cudaError_t launch_gemm_rownorm_tc2(const GemmTcPlan& p, cudaStream_t s);

// GEMM + tail + row norm with the rows held in tensor memory until their statistics are known (a cluster of CTA
// pairs covers whole rows and exchanges partial sums through distributed shared memory): y = norm(tail(A W)),
// bf16; mid_out (optional, bf16 or fp32) also receives tail(A W), the value before the norm.
struct GemmRowNormClPlan {
  CUtensorMap tm_a, tm_b, tm_out;
  void* out = nullptr;
  void* mid_out = nullptr;
  bool mid_f32 = false;
  int m = 0, n = 0, k = 0;
  int pairs = 1, nt = 1;     // CTA pairs per cluster; 256-column tiles per pair and row block
  int grid = 0;
  EpiProgram epi;
  const void* gamma = nullptr;
  const void* beta = nullptr;
  float eps = 0.f;
  int mode = 0;
};
// m > 128, k % 8 == 0, n % 8 == 0, n <= 2048
bool gemm_rownorm_cl_supported(int64_t m, int64_t n, int64_t k);
cudaError_t gemm_rownorm_cl_plan(GemmRowNormClPlan* p, const void* a, const void* w_nk, void* y, void* mid_out, bool mid_f32, int64_t m,
                                 int64_t n, int64_t k, const EpiProgram& epi, int mode, const void* gamma, const void* beta, float eps,
                                 int sm_count);
cudaError_t launch_gemm_rownorm_cl(const GemmRowNormClPlan& p, cudaStream_t s);
}  // namespace mk

namespace mk {
// Block-scaled fp8 GEMM (LINEAR_FP8): y = tail( sum_kb sx[m, kb] * sw[n / 128, kb] * (xq[m, kb-th block] . wq[kb-th block, n]) ), bf16 out.
struct GemmFp8Plan {
  CUtensorMap tm_a, tm_b, tm_out;
  const float* sx = nullptr;   // [m, k / 128]
  const float* sw = nullptr;   // [ceil(n / 128), k / 128]
  void* out = nullptr;
  int m = 0, n = 0, k = 0;
  int grid = 0;
  EpiProgram epi;
};
// xq [m, k] and wq stored [n, k], both e4m3 bytes; k % 128 == 0, k <= 8192, n % 8 == 0
bool gemm_fp8_tc2_supported(int64_t m, int64_t n, int64_t k);
cudaError_t gemm_fp8_tc2_plan(GemmFp8Plan* p, const void* xq, const float* sx, const void* wq_nk, const float* sw, void* y, int64_t m,
                              int64_t n, int64_t k, const EpiProgram& epi, int sm_count);
cudaError_t launch_gemm_fp8_tc2(const GemmFp8Plan& p, cudaStream_t s);
}  // namespace mk

namespace mk {
struct ConvTcPlan {
  CUtensorMap tm_x, tm_w;
  CUtensorMap tm_y, tm_y30; // the output, for the epilogue's bulk stores: boxes of 32 and of 30 pixels
  void* y = nullptr;
  // optional GroupNorm partial sums of the stored output: float [nb][conv3x3_tc2_stat_slots(h, w)][c_out / cpg][2]
  // = (sum, sum of squares) per group of cpg adjacent channels (cpg in {2, 4, 8, 16, 32}); null: none
  float* stats = nullptr;
  int cpg = 0;
  int nb = 0, h = 0, w = 0, c_in = 0, c_out = 0;
  int grid = 0;
  size_t smem = 0;
  EpiProgram epi;
};
// NHWC bf16 3x3 conv (stride 1, pad 1) + elementwise tail; weights [C_out, 3, 3, C_in].
// Supported: C_in in {64, 128}, C_out multiple of 32 up to 256, any H and W, and half the weights
// plus two input patches must fit one SM's shared memory.
bool conv3x3_tc2_supported(int64_t nb, int64_t h, int64_t w, int64_t c_in, int64_t c_out);
int conv3x3_tc2_stat_slots(int64_t h, int64_t w);
cudaError_t conv3x3_tc2_plan(ConvTcPlan* p, const void* x, const void* w, void* y, int64_t nb, int64_t h, int64_t wd, int64_t c_in,
                             int64_t c_out, const EpiProgram& epi, int sm_count);
cudaError_t launch_conv3x3_tc2(const ConvTcPlan& p, cudaStream_t s);
}  // namespace mk

namespace mk {
struct AttnTcPlan {
  CUtensorMap tm_q, tm_k, tm_v;
  void* out = nullptr;
  int B = 0, H = 0, S = 0, D = 128;
  bool causal = true;
  float scale_log2 = 0.f;
  int grid = 0;
};
// Attention (causal or unmasked), bf16, head_dim 64 or 128, any strided [B, H, S, D] view whose strides are
// multiples of 16 bytes; output the dense [B*S, H*D] matrix.  One 128-query tile per CTA.
bool attention_tc_supported(const AttnView& a);
cudaError_t attention_tc_plan(AttnTcPlan* p, const AttnView& a, void* o);
cudaError_t launch_attention_tc(const AttnTcPlan& p, cudaStream_t s);
// Two-query-tile persistent form (256 queries per work item, O accumulated in TMEM); same contract, and also
// the unmasked operator (AttnView::causal false).
bool attention_tc2_supported(const AttnView& a);
cudaError_t attention_tc2_plan(AttnTcPlan* p, const AttnView& a, void* o, int sm_count);
cudaError_t launch_attention_tc2(const AttnTcPlan& p, cudaStream_t s);
}  // namespace mk
