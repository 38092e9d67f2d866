// Implementation registry: each entry is a kernel family with the legality predicate that says
// which operator ranges it can run as ONE fused piece, following the paper's fusion rules
// (appendix "Prompts", decomposition: GEMM + elementwise tail, elementwise chains, bias after
// matmul and residual add fuse; a reduction that needs the whole row / group before its result is
// used blocks fusion unless one CTA owns the whole row).
//
// Order = the composer's preference among implementations that accept the same range.
#include <stdio.h>
#include <stdlib.h>
#include <memory>

#include "mk_internal.h"
#include "tc_plans.h"

namespace mk {
namespace {

int dt(const Module& m) { return m.dtype == MK_F32 ? DT_F32 : DT_BF16; }
int dt_of(const mk_tensor_spec& s) { return s.dtype == MK_F32 ? DT_F32 : DT_BF16; }
// the piece's first input / its output stored in the module's dtype (not an fp32 residual stream)
bool in_is_module_dtype(const Module& m, int lo) { return m.vspec(m.ops[lo].in_id[0]).dtype == m.dtype; }
bool out_is_module_dtype(const Module& m, int hi) { return m.vspec(m.ops[hi - 1].out_id).dtype == m.dtype; }

// ops lo+1.. read their predecessor as first input; nothing but the last value leaves the piece;
// residual operands come from outside the piece.
bool is_chain(const Module& m, int lo, int hi) {
  if (hi <= lo) return false;
  for (int j = lo + 1; j < hi; ++j)
    if (m.ops[j].in_id[0] != m.ops[j - 1].out_id) return false;
  for (int j = lo; j < hi - 1; ++j)
    if (m.escapes(j, lo, hi)) return false;
  for (int j = lo; j < hi; ++j)
    if (m.ops[j].d.kind == MK_OP_RESIDUAL_ADD) {
      const int prod = m.values[m.ops[j].in_id[1]].producer;
      if (prod >= lo && prod < hi) return false;
    }
  return true;
}
bool all_eltwise(const Module& m, int a, int b) {
  if (b - a > EPI_MAX) return false;
  for (int j = a; j < b; ++j)
    if (!is_eltwise(m.ops[j].d.kind)) return false;
  return true;
}
size_t no_scratch(const Module&, int, int) { return 0; }

int64_t last_dim(const mk_tensor_spec& s) { return s.shape[s.rank - 1]; }
int64_t rows_of(const mk_tensor_spec& s) { return numel(s) / last_dim(s); }

// ------------------------------------------------------------------ eltwise chain
bool eltwise_match(const Module& m, int lo, int hi) {
  if (!is_chain(m, lo, hi) || !in_is_module_dtype(m, lo)) return false;
  const bool sw = m.ops[lo].d.kind == MK_OP_SWIGLU;
  return all_eltwise(m, lo + (sw ? 1 : 0), hi);
}
mk_status eltwise_emit(const Module& m, int lo, int hi, const Resolved& r, std::vector<Launch>& out, std::string& err) {
  const bool sw = m.ops[lo].d.kind == MK_OP_SWIGLU;
  EpiProgram p;
  mk_status st = build_epi(m, lo + (sw ? 1 : 0), hi, r, p, err);
  if (st != MK_OK) return st;
  const void* x = r.value_ptr[m.ops[lo].in_id[0]];
  void* y = r.value_ptr[m.ops[hi - 1].out_id];
  const mk_tensor_spec& ys = m.vspec(m.ops[hi - 1].out_id);
  const int64_t rows = rows_of(ys), cols = last_dim(ys);
  const int d = dt(m), od = dt_of(ys), sms = m.ctx->sm_count;
  out.push_back([=](cudaStream_t s) { return launch_eltwise(d, od, x, y, rows, cols, sw, p, sms, s); });
  return MK_OK;
}

// ------------------------------------------------------------------ pooling
bool is_pool(int32_t k) { return k == MK_OP_AVGPOOL2D || k == MK_OP_MAXPOOL2D || k == MK_OP_LPPOOL2D; }
bool pool_match(const Module& m, int lo, int hi) { return hi - lo == 1 && is_pool(m.ops[lo].d.kind) && in_is_module_dtype(m, lo); }
mk_status pool_emit(const Module& m, int lo, int, const Resolved& r, std::vector<Launch>& out, std::string&) {
  const Op& op = m.ops[lo];
  const mk_tensor_spec& xs = m.vspec(op.in_id[0]);
  const void* x = r.value_ptr[op.in_id[0]];
  void* y = r.value_ptr[op.out_id];
  const int d = dt(m), sms = m.ctx->sm_count;
  const int mode = op.d.kind == MK_OP_AVGPOOL2D ? POOL_AVG : op.d.kind == MK_OP_MAXPOOL2D ? POOL_MAX : POOL_LP;
  const int64_t nb = xs.shape[0], h = xs.shape[1], w = xs.shape[2], c = xs.shape[3];
  const int k = (int)op.d.i[0], st = (int)op.d.i[1];
  const float p = (float)op.d.f[0];
  out.push_back([=](cudaStream_t s) { return launch_pool_nhwc(d, mode, x, y, nb, h, w, c, k, st, p, sms, s); });
  return MK_OK;
}

// ------------------------------------------------------------------ row reductions
bool is_rowop(int32_t k) { return k == MK_OP_LAYERNORM || k == MK_OP_RMSNORM || k == MK_OP_SOFTMAX; }
int row_mode(int32_t k) { return k == MK_OP_LAYERNORM ? ROW_LAYERNORM : k == MK_OP_RMSNORM ? ROW_RMSNORM : ROW_SOFTMAX; }

bool rowop_match(const Module& m, int lo, int hi) {
  if (!is_chain(m, lo, hi) || !is_rowop(m.ops[hi - 1].d.kind) || !all_eltwise(m, lo, hi - 1)) return false;
  // an fp32 residual-stream input is taken by the norm itself, not through an elementwise prefix
  return in_is_module_dtype(m, lo) || hi - lo == 1;
}
mk_status rowop_emit(const Module& m, int lo, int hi, const Resolved& r, std::vector<Launch>& out, std::string& err) {
  EpiProgram p;
  mk_status st = build_epi(m, lo, hi - 1, r, p, err);
  if (st != MK_OK) return st;
  const Op& op = m.ops[hi - 1];
  const void* x = r.value_ptr[m.ops[lo].in_id[0]];
  void* y = r.value_ptr[op.out_id];
  const mk_tensor_spec& ys = m.vspec(op.out_id);
  const int64_t rows = rows_of(ys), n = last_dim(ys);
  const void* g = op.param[0].set ? op.param[0].ptr : nullptr;
  const void* b = op.param[1].set ? op.param[1].ptr : nullptr;
  const float eps = (float)op.d.f[0];
  const int mode = row_mode(op.d.kind), d = dt(m), id = dt_of(m.vspec(m.ops[lo].in_id[0]));
  out.push_back([=](cudaStream_t s) { return launch_rowop(d, id, mode, x, y, rows, n, g, b, eps, p, s); });
  return MK_OK;
}

// ------------------------------------------------------------------ GroupNorm (two launches + scratch)
bool groupnorm_match(const Module& m, int lo, int hi) {
  return is_chain(m, lo, hi) && m.ops[hi - 1].d.kind == MK_OP_GROUPNORM && all_eltwise(m, lo, hi - 1) && in_is_module_dtype(m, lo);
}
size_t groupnorm_scratch(const Module& m, int, int hi) {
  const mk_tensor_spec& s = m.vspec(m.ops[hi - 1].out_id);
  return groupnorm_scratch_bytes(s.shape[0], s.shape[1] * s.shape[2], s.shape[3], m.ops[hi - 1].d.i[0], m.ctx->sm_count);
}
mk_status groupnorm_emit(const Module& m, int lo, int hi, const Resolved& r, std::vector<Launch>& out, std::string& err) {
  EpiProgram p;
  mk_status st = build_epi(m, lo, hi - 1, r, p, err);
  if (st != MK_OK) return st;
  const Op& op = m.ops[hi - 1];
  const void* x = r.value_ptr[m.ops[lo].in_id[0]];
  void* y = r.value_ptr[op.out_id];
  const mk_tensor_spec& s = m.vspec(op.out_id);
  const int64_t nb = s.shape[0], hw = s.shape[1] * s.shape[2], c = s.shape[3];
  const int groups = op.d.i[0];
  const void* g = op.param[0].set ? op.param[0].ptr : nullptr;
  const void* b = op.param[1].set ? op.param[1].ptr : nullptr;
  const float eps = (float)op.d.f[0];
  const int d = dt(m);
  const int sms = m.ctx->sm_count;
  if (getenv("MK_DEBUG_PLAN"))
    fprintf(stderr, "groupnorm_nhwc: nb %lld hw %lld c %lld groups %d -> %s\n", (long long)nb, (long long)hw, (long long)c, groups,
            groupnorm_cluster_supported(d, x, y, nb, hw, c, groups, sms) ? "cluster form" : "two passes");
  if (!getenv("MK_GN_TWO_PASS") && groupnorm_cluster_supported(d, x, y, nb, hw, c, groups, sms)) {
    // the image fits a cluster's shared memory: one launch, the tensor read once
    out.push_back([=](cudaStream_t st_) { return launch_groupnorm_cluster(d, x, y, nb, hw, c, groups, g, b, eps, p, sms, st_); });
    return MK_OK;
  }
  const int chunks = groupnorm_chunks(nb, hw, m.ctx->sm_count);
  float* scratch = (float*)r.scratch;
  out.push_back([=](cudaStream_t st_) { return launch_groupnorm_stats(d, x, nb, hw, c, groups, p, scratch, chunks, st_); });
  out.push_back([=](cudaStream_t st_) { return launch_groupnorm_apply(d, x, y, nb, hw, c, groups, g, b, eps, p, scratch, chunks, st_); });
  return MK_OK;
}

// ------------------------------------------------------------------ GEMM family
// LINEAR [SWIGLU] [elementwise]*
bool gemm_shape(const Module& m, int lo, int hi, bool* swiglu, int* tail_lo) {
  if (!is_chain(m, lo, hi) || m.ops[lo].d.kind != MK_OP_LINEAR || !in_is_module_dtype(m, lo)) return false;
  int t = lo + 1;
  *swiglu = t < hi && m.ops[t].d.kind == MK_OP_SWIGLU;
  if (*swiglu) ++t;
  *tail_lo = t;
  return all_eltwise(m, t, hi);
}
bool gemm_simt_match(const Module& m, int lo, int hi) {
  bool sw; int t;
  return gemm_shape(m, lo, hi, &sw, &t);
}
mk_status gemm_simt_emit(const Module& m, int lo, int hi, const Resolved& r, std::vector<Launch>& out, std::string& err) {
  bool sw; int t;
  gemm_shape(m, lo, hi, &sw, &t);
  EpiProgram p;
  mk_status st = build_epi(m, t, hi, r, p, err);
  if (st != MK_OK) return st;
  const Op& op = m.ops[lo];
  const void* a = r.value_ptr[op.in_id[0]];
  const void* w = op.param[0].ptr;
  void* y = r.value_ptr[m.ops[hi - 1].out_id];
  const mk_tensor_spec& xs = m.vspec(op.in_id[0]);
  const int64_t M = rows_of(xs), K = last_dim(xs), N = last_dim(m.vspec(m.ops[hi - 1].out_id));
  const bool wt = op.d.i[1] == MK_LAYOUT_TRANSPOSED;
  const int d = dt(m), od = dt_of(m.vspec(m.ops[hi - 1].out_id));
  out.push_back([=](cudaStream_t s) { return launch_gemm_simt(d, od, a, w, wt, y, M, N, K, sw, p, s); });
  return MK_OK;
}

// tcgen05 GEMM: bf16, W stored [N, K], 16-byte rows
bool gemm_tc_match(const Module& m, int lo, int hi) {
  bool sw; int t;
  if (!gemm_shape(m, lo, hi, &sw, &t)) return false;
  if (m.dtype != MK_BF16) return false;
  const Op& op = m.ops[lo];
  if (op.d.i[1] != MK_LAYOUT_TRANSPOSED) return false;
  const int64_t K = last_dim(m.vspec(op.in_id[0]));
  const int64_t N = last_dim(m.vspec(m.ops[hi - 1].out_id));
  return K % 8 == 0 && N % 8 == 0;
}
mk_status gemm_tc_emit_impl(const Module& m, int lo, int hi, const Resolved& r, std::vector<Launch>& out, std::string& err, bool pair) {
  bool sw; int t;
  gemm_shape(m, lo, hi, &sw, &t);
  EpiProgram p;
  mk_status st = build_epi(m, t, hi, r, p, err);
  if (st != MK_OK) return st;
  const Op& op = m.ops[lo];
  const mk_tensor_spec& xs = m.vspec(op.in_id[0]);
  const int64_t M = rows_of(xs), K = last_dim(xs), N = last_dim(m.vspec(m.ops[hi - 1].out_id));
  auto plan = std::make_shared<GemmTcPlan>();
  const void* a = r.value_ptr[op.in_id[0]];
  void* y = r.value_ptr[m.ops[hi - 1].out_id];
  const bool of32 = m.vspec(m.ops[hi - 1].out_id).dtype == MK_F32;
  cudaError_t e = pair ? gemm_tc2_plan(plan.get(), a, op.param[0].ptr, y, of32, M, N, K, sw, p, m.ctx->sm_count)
                       : gemm_tc_plan(plan.get(), a, op.param[0].ptr, y, of32, M, N, K, sw, p, m.ctx->sm_count);
  if (e != cudaSuccess) { err = std::string("gemm_tc plan: ") + cudaGetErrorString(e); return MK_ERR_CUDA; }
  if (pair) out.push_back([plan](cudaStream_t s) { return launch_gemm_tc2(*plan, s); });
  else out.push_back([plan](cudaStream_t s) { return launch_gemm_tc(*plan, s); });
  return MK_OK;
}
mk_status gemm_tc_emit(const Module& m, int lo, int hi, const Resolved& r, std::vector<Launch>& out, std::string& err) {
  return gemm_tc_emit_impl(m, lo, hi, r, out, err, false);
}
// two-SM form: worth it once a tile pair has more than one CTA's worth of rows
bool gemm_tc2_match(const Module& m, int lo, int hi) {
  return gemm_tc_match(m, lo, hi) && rows_of(m.vspec(m.ops[lo].in_id[0])) > 128;
}
mk_status gemm_tc2_emit(const Module& m, int lo, int hi, const Resolved& r, std::vector<Launch>& out, std::string& err) {
  return gemm_tc_emit_impl(m, lo, hi, r, out, err, true);
}

// LINEAR_FP8 [elementwise]*: block-scaled fp8 contraction (the paper's FP8 MoE inference task), bf16 out
bool gemm_fp8_shape(const Module& m, int lo, int hi) {
  return is_chain(m, lo, hi) && m.ops[lo].d.kind == MK_OP_LINEAR_FP8 && all_eltwise(m, lo + 1, hi) && out_is_module_dtype(m, hi) && m.dtype == MK_BF16;
}
bool gemm_fp8_simt_match(const Module& m, int lo, int hi) { return gemm_fp8_shape(m, lo, hi); }
bool gemm_fp8_tc2_match(const Module& m, int lo, int hi) {
  if (!gemm_fp8_shape(m, lo, hi) || m.ops[lo].d.i[1] != MK_LAYOUT_TRANSPOSED) return false;
  const mk_tensor_spec& xs = m.vspec(m.ops[lo].in_id[0]);
  return gemm_fp8_tc2_supported(rows_of(xs), m.ops[lo].d.i[0], last_dim(xs));
}
mk_status gemm_fp8_emit_impl(const Module& m, int lo, int hi, const Resolved& r, std::vector<Launch>& out, std::string& err, bool tc) {
  EpiProgram p;
  mk_status st = build_epi(m, lo + 1, hi, r, p, err);
  if (st != MK_OK) return st;
  const Op& op = m.ops[lo];
  const mk_tensor_spec& xs = m.vspec(op.in_id[0]);
  const int64_t M = rows_of(xs), K = last_dim(xs), N = op.d.i[0];
  const void* xq = r.value_ptr[op.in_id[0]];
  const float* sx = (const float*)r.value_ptr[op.in_id[1]];
  const void* wq = op.param[0].ptr;
  const float* sw = (const float*)op.param[1].ptr;
  void* y = r.value_ptr[m.ops[hi - 1].out_id];
  if (tc) {
    auto plan = std::make_shared<GemmFp8Plan>();
    cudaError_t e = gemm_fp8_tc2_plan(plan.get(), xq, sx, wq, sw, y, M, N, K, p, m.ctx->sm_count);
    if (e != cudaSuccess) { err = std::string("gemm_fp8_tc2 plan: ") + cudaGetErrorString(e); return MK_ERR_CUDA; }
    out.push_back([plan](cudaStream_t s) { return launch_gemm_fp8_tc2(*plan, s); });
  } else {
    const bool wt = op.d.i[1] == MK_LAYOUT_TRANSPOSED;
    out.push_back([=](cudaStream_t s) { return launch_gemm_fp8_simt(xq, sx, wq, wt, sw, y, M, N, K, p, s); });
  }
  return MK_OK;
}
mk_status gemm_fp8_tc2_emit(const Module& m, int lo, int hi, const Resolved& r, std::vector<Launch>& out, std::string& err) {
  return gemm_fp8_emit_impl(m, lo, hi, r, out, err, true);
}
mk_status gemm_fp8_simt_emit(const Module& m, int lo, int hi, const Resolved& r, std::vector<Launch>& out, std::string& err) {
  return gemm_fp8_emit_impl(m, lo, hi, r, out, err, false);
}

// LINEAR [elementwise]* (LAYERNORM | RMSNORM) on the tensor cores: the norm's statistics come out of the GEMM's
// epilogue and the warp that completes a block of rows normalises it in place - the paper's projection +
// residual + norm fusion at tensor-core shape, without a pass of its own over the activation.
bool gemm_rownorm_tc2_match(const Module& m, int lo, int hi) {
  if (hi - lo < 2 || !is_chain(m, lo, hi)) return false;
  const int32_t k = m.ops[hi - 1].d.kind;
  if (k != MK_OP_LAYERNORM && k != MK_OP_RMSNORM) return false;
  if (!gemm_tc2_match(m, lo, hi - 1)) return false;
  bool sw; int t;
  if (!gemm_shape(m, lo, hi - 1, &sw, &t) || sw) return false;
  // the value handed to the norm and the norm's result are both bf16 (the row is normalised in place)
  if (m.vspec(m.ops[hi - 2].out_id).dtype != MK_BF16 || m.vspec(m.ops[hi - 1].out_id).dtype != MK_BF16) return false;
  const int64_t N = last_dim(m.vspec(m.ops[hi - 1].out_id));
  return N <= 16384;
}
size_t gemm_rownorm_tc2_scratch_fn(const Module& m, int lo, int hi) {
  const mk_tensor_spec& xs = m.vspec(m.ops[lo].in_id[0]);
  return gemm_rownorm_tc2_scratch(rows_of(xs), last_dim(m.vspec(m.ops[hi - 1].out_id)));
}
mk_status gemm_rownorm_tc2_emit(const Module& m, int lo, int hi, const Resolved& r, std::vector<Launch>& out, std::string& err) {
  bool sw; int t;
  gemm_shape(m, lo, hi - 1, &sw, &t);
  EpiProgram p;
  mk_status st = build_epi(m, t, hi - 1, r, p, err);
  if (st != MK_OK) return st;
  const Op& op = m.ops[lo];
  const Op& nop = m.ops[hi - 1];
  const mk_tensor_spec& xs = m.vspec(op.in_id[0]);
  const int64_t M = rows_of(xs), K = last_dim(xs), N = last_dim(m.vspec(nop.out_id));
  const void* g = nop.param[0].set ? nop.param[0].ptr : nullptr;
  const void* b = nop.param[1].set ? nop.param[1].ptr : nullptr;
  auto plan = std::make_shared<GemmTcPlan>();
  cudaError_t e = gemm_rownorm_tc2_plan(plan.get(), r.value_ptr[op.in_id[0]], op.param[0].ptr, r.value_ptr[nop.out_id], M, N, K, p,
                                        row_mode(nop.d.kind), g, b, (float)nop.d.f[0], r.scratch, m.ctx->sm_count);
  if (e != cudaSuccess) { err = std::string("gemm_rownorm_tc2 plan: ") + cudaGetErrorString(e); return MK_ERR_CUDA; }
  out.push_back([plan](cudaStream_t s) { return launch_gemm_rownorm_tc2(*plan, s); });
  return MK_OK;
}

// The same operator range with the rows kept in tensor memory until their statistics are known (a cluster of CTA
// pairs covers whole rows): one store of the normalised row, nothing read back.  The value handed to the norm may
// itself be needed later (a residual stream): it is then written as well, from the same pass.
bool chain_with_open_prenorm(const Module& m, int lo, int hi) {
  if (hi - lo < 2) return false;
  for (int j = lo + 1; j < hi; ++j)
    if (m.ops[j].in_id[0] != m.ops[j - 1].out_id) return false;
  for (int j = lo; j < hi - 2; ++j)
    if (m.escapes(j, lo, hi)) return false;
  for (int j = lo; j < hi; ++j)
    if (m.ops[j].d.kind == MK_OP_RESIDUAL_ADD) {
      const int prod = m.values[m.ops[j].in_id[1]].producer;
      if (prod >= lo && prod < hi) return false;
    }
  return true;
}
bool gemm_rownorm_cl_match(const Module& m, int lo, int hi) {
  if (!chain_with_open_prenorm(m, lo, hi)) return false;
  const int32_t k = m.ops[hi - 1].d.kind;
  if (k != MK_OP_LAYERNORM && k != MK_OP_RMSNORM) return false;
  const Op& op = m.ops[lo];
  if (op.d.kind != MK_OP_LINEAR || !in_is_module_dtype(m, lo) || m.dtype != MK_BF16) return false;
  if (op.d.i[1] != MK_LAYOUT_TRANSPOSED || !all_eltwise(m, lo + 1, hi - 1)) return false;
  if (m.vspec(m.ops[hi - 1].out_id).dtype != MK_BF16) return false;
  const mk_tensor_spec& xs = m.vspec(op.in_id[0]);
  return gemm_rownorm_cl_supported(rows_of(xs), last_dim(m.vspec(m.ops[hi - 1].out_id)), last_dim(xs));
}
mk_status gemm_rownorm_cl_emit(const Module& m, int lo, int hi, const Resolved& r, std::vector<Launch>& out, std::string& err) {
  EpiProgram p;
  mk_status st = build_epi(m, lo + 1, hi - 1, r, p, err);
  if (st != MK_OK) return st;
  const Op& op = m.ops[lo];
  const Op& nop = m.ops[hi - 1];
  const mk_tensor_spec& xs = m.vspec(op.in_id[0]);
  const int64_t M = rows_of(xs), K = last_dim(xs), N = last_dim(m.vspec(nop.out_id));
  const void* g = nop.param[0].set ? nop.param[0].ptr : nullptr;
  const void* b = nop.param[1].set ? nop.param[1].ptr : nullptr;
  const int pre = m.ops[hi - 2].out_id;
  void* mid = m.escapes(hi - 2, lo, hi) ? r.value_ptr[pre] : nullptr;
  const bool mid_f32 = m.vspec(pre).dtype == MK_F32;
  auto plan = std::make_shared<GemmRowNormClPlan>();
  cudaError_t e = gemm_rownorm_cl_plan(plan.get(), r.value_ptr[op.in_id[0]], op.param[0].ptr, r.value_ptr[nop.out_id], mid, mid_f32, M, N, K, p,
                                       row_mode(nop.d.kind), g, b, (float)nop.d.f[0], m.ctx->sm_count);
  if (e != cudaSuccess) { err = std::string("gemm_rownorm_cl plan: ") + cudaGetErrorString(e); return MK_ERR_CUDA; }
  out.push_back([plan](cudaStream_t s) { return launch_gemm_rownorm_cl(*plan, s); });
  return MK_OK;
}

// LINEAR [elementwise]* RMSNORM LINEAR [SWIGLU] [elementwise]* as TWO tensor-core GEMMs and no pass over the
// activation in between: the paper's fusion across a norm boundary in the form that survives a reduction over the
// whole row.  The norm's scale 1 / rms is one scalar per row, so it commutes with the second contraction: the first
// GEMM's epilogue also leaves xg = bf16(x * gamma) and per-row partial sums of x^2, the second takes xg as its A
// operand and multiplies its accumulator rows by 1 / rms before its own tail.  The value handed to the norm must be
// needed later anyway (a residual stream): it is the first GEMM's ordinary output.
bool gemm_prenorm_find(const Module& m, int lo, int hi, int* norm_at, bool* swiglu2, int* tail2_lo) {
  if (hi - lo < 3 || m.dtype != MK_BF16) return false;
  int r = -1;
  for (int j = lo + 1; j < hi; ++j)
    if (m.ops[j].d.kind == MK_OP_RMSNORM) { r = j; break; }
  if (r < 0 || r + 1 >= hi) return false;
  // structure: a chain; only the norm's input may leave the piece early, and it must; the norm's output feeds the second GEMM alone
  for (int j = lo + 1; j < hi; ++j)
    if (m.ops[j].in_id[0] != m.ops[j - 1].out_id) return false;
  for (int j = lo; j < hi - 1; ++j)
    if (m.escapes(j, lo, hi) != (j == r - 1)) return false;
  for (int j = lo; j < hi; ++j)
    if (m.ops[j].d.kind == MK_OP_RESIDUAL_ADD) {
      const int prod = m.values[m.ops[j].in_id[1]].producer;
      if (prod >= lo && prod < hi) return false;
    }
  const Op& l1 = m.ops[lo];
  const Op& l2 = m.ops[r + 1];
  if (l1.d.kind != MK_OP_LINEAR || l2.d.kind != MK_OP_LINEAR || !in_is_module_dtype(m, lo)) return false;
  if (l1.d.i[1] != MK_LAYOUT_TRANSPOSED || l2.d.i[1] != MK_LAYOUT_TRANSPOSED) return false;
  if (!all_eltwise(m, lo + 1, r)) return false;
  int t = r + 2;
  *swiglu2 = t < hi && m.ops[t].d.kind == MK_OP_SWIGLU;
  if (*swiglu2) ++t;
  if (!all_eltwise(m, t, hi) || !out_is_module_dtype(m, hi)) return false;
  const mk_tensor_spec& xs = m.vspec(l1.in_id[0]);
  const int64_t M = rows_of(xs), K1 = last_dim(xs), N1 = l1.d.i[0], N2 = last_dim(m.vspec(m.ops[hi - 1].out_id));
  if (M <= 128 || K1 % 8 || N1 % 8 || N2 % 8) return false;
  *norm_at = r;
  *tail2_lo = t;
  return true;
}
bool gemm_prenorm_match(const Module& m, int lo, int hi) {
  int r, t; bool sw;
  return gemm_prenorm_find(m, lo, hi, &r, &sw, &t);
}
size_t gemm_prenorm_scratch_fn(const Module& m, int lo, int) {
  return gemm_prenorm_scratch(rows_of(m.vspec(m.ops[lo].in_id[0])), m.ops[lo].d.i[0]);
}
mk_status gemm_prenorm_emit(const Module& m, int lo, int hi, const Resolved& r, std::vector<Launch>& out, std::string& err) {
  int nr, t2; bool sw2;
  gemm_prenorm_find(m, lo, hi, &nr, &sw2, &t2);
  EpiProgram p1, p2;
  mk_status st = build_epi(m, lo + 1, nr, r, p1, err);
  if (st == MK_OK) st = build_epi(m, t2, hi, r, p2, err);
  if (st != MK_OK) return st;
  const Op& l1 = m.ops[lo];
  const Op& nop = m.ops[nr];
  const Op& l2 = m.ops[nr + 1];
  const mk_tensor_spec& xs = m.vspec(l1.in_id[0]);
  const int64_t M = rows_of(xs), K1 = last_dim(xs), N1 = l1.d.i[0], N2 = last_dim(m.vspec(m.ops[hi - 1].out_id));
  const int pre = m.ops[nr - 1].out_id;
  auto plan1 = std::make_shared<GemmTcPlan>();
  auto plan2 = std::make_shared<GemmTcPlan>();
  cudaError_t e = gemm_prenorm_pair_plan(plan1.get(), plan2.get(), r.value_ptr[l1.in_id[0]], l1.param[0].ptr, r.value_ptr[pre], m.vspec(pre).dtype == MK_F32,
                                         M, N1, K1, p1, nop.param[0].set ? nop.param[0].ptr : nullptr, (float)nop.d.f[0], l2.param[0].ptr,
                                         r.value_ptr[m.ops[hi - 1].out_id], N2, sw2, p2, r.scratch, m.ctx->sm_count);
  if (e != cudaSuccess) { err = std::string("gemm_prenorm_gemm_tc2 plan: ") + cudaGetErrorString(e); return MK_ERR_CUDA; }
  out.push_back([plan1](cudaStream_t s) { return launch_gemm_tc2(*plan1, s); });
  out.push_back([plan2](cudaStream_t s) { return launch_gemm_tc2(*plan2, s); });
  return MK_OK;
}

// LINEAR [elementwise]* (LAYERNORM | RMSNORM), fp32, one CTA owns whole rows
bool linear_rownorm_match(const Module& m, int lo, int hi) {
  if (hi - lo < 2 || !is_chain(m, lo, hi) || m.ops[lo].d.kind != MK_OP_LINEAR) return false;
  const int32_t k = m.ops[hi - 1].d.kind;
  if (k != MK_OP_LAYERNORM && k != MK_OP_RMSNORM) return false;
  if (!all_eltwise(m, lo + 1, hi - 1)) return false;
  if (m.dtype != MK_F32) return false;
  return m.ops[lo].d.i[0] <= 1024;
}
mk_status linear_rownorm_emit(const Module& m, int lo, int hi, const Resolved& r, std::vector<Launch>& out, std::string& err) {
  EpiProgram p;
  mk_status st = build_epi(m, lo + 1, hi - 1, r, p, err);
  if (st != MK_OK) return st;
  const Op& op = m.ops[lo];
  const Op& nop = m.ops[hi - 1];
  const void* a = r.value_ptr[op.in_id[0]];
  const void* w = op.param[0].ptr;
  void* y = r.value_ptr[nop.out_id];
  const mk_tensor_spec& xs = m.vspec(op.in_id[0]);
  const int64_t M = rows_of(xs), K = last_dim(xs), N = op.d.i[0];
  const bool wt = op.d.i[1] == MK_LAYOUT_TRANSPOSED;
  const void* g = nop.param[0].set ? nop.param[0].ptr : nullptr;
  const void* b = nop.param[1].set ? nop.param[1].ptr : nullptr;
  const float eps = (float)nop.d.f[0];
  const int mode = row_mode(nop.d.kind), d = dt(m);
  out.push_back([=](cudaStream_t s) { return launch_linear_rownorm_simt(d, a, w, wt, y, M, N, K, p, mode, g, b, eps, s); });
  return MK_OK;
}

// ------------------------------------------------------------------ convolution
bool conv_simt_match(const Module& m, int lo, int hi) {
  return is_chain(m, lo, hi) && m.ops[lo].d.kind == MK_OP_CONV2D_3X3 && all_eltwise(m, lo + 1, hi) && out_is_module_dtype(m, hi);
}
mk_status conv_simt_emit(const Module& m, int lo, int hi, const Resolved& r, std::vector<Launch>& out, std::string& err) {
  EpiProgram p;
  mk_status st = build_epi(m, lo + 1, hi, r, p, err);
  if (st != MK_OK) return st;
  const Op& op = m.ops[lo];
  const void* x = r.value_ptr[op.in_id[0]];
  const void* w = op.param[0].ptr;
  void* y = r.value_ptr[m.ops[hi - 1].out_id];
  const mk_tensor_spec& xs = m.vspec(op.in_id[0]);
  const int64_t nb = xs.shape[0], h = xs.shape[1], wd = xs.shape[2], c = xs.shape[3], co = op.d.i[0];
  const int d = dt(m);
  out.push_back([=](cudaStream_t s) { return launch_conv3x3_simt(d, x, w, y, nb, h, wd, c, co, p, s); });
  return MK_OK;
}

// tcgen05 implicit GEMM, weights resident in shared memory
bool conv_tc2_match(const Module& m, int lo, int hi) {
  if (!conv_simt_match(m, lo, hi) || m.dtype != MK_BF16) return false;
  const mk_tensor_spec& xs = m.vspec(m.ops[lo].in_id[0]);
  return conv3x3_tc2_supported(xs.shape[0], xs.shape[1], xs.shape[2], xs.shape[3], m.ops[lo].d.i[0]);
}
mk_status conv_tc2_emit(const Module& m, int lo, int hi, const Resolved& r, std::vector<Launch>& out, std::string& err) {
  EpiProgram p;
  mk_status st = build_epi(m, lo + 1, hi, r, p, err);
  if (st != MK_OK) return st;
  const Op& op = m.ops[lo];
  const mk_tensor_spec& xs = m.vspec(op.in_id[0]);
  auto plan = std::make_shared<ConvTcPlan>();
  cudaError_t e = conv3x3_tc2_plan(plan.get(), r.value_ptr[op.in_id[0]], op.param[0].ptr, r.value_ptr[m.ops[hi - 1].out_id], xs.shape[0],
                                   xs.shape[1], xs.shape[2], xs.shape[3], op.d.i[0], p, m.ctx->sm_count);
  if (e != cudaSuccess) { err = std::string("conv3x3_tc2 plan: ") + cudaGetErrorString(e); return MK_ERR_CUDA; }
  out.push_back([plan](cudaStream_t s) { return launch_conv3x3_tc2(*plan, s); });
  return MK_OK;
}

// CONV2D_3x3 [elementwise]* GROUPNORM: the convolution's epilogue leaves the GroupNorm partial sums of
// what it stores, so the statistics pass over the activation disappears; the activation itself sits in
// scratch between the two launches (the normalisation needs the whole image's statistics first).
size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
bool conv_gn_tc2_match(const Module& m, int lo, int hi) {
  if (hi - lo < 2 || m.ops[hi - 1].d.kind != MK_OP_GROUPNORM || !is_chain(m, lo, hi)) return false;
  if (!conv_tc2_match(m, lo, hi - 1)) return false;
  const mk_tensor_spec& s = m.vspec(m.ops[hi - 1].out_id);
  const int64_t c = s.shape[3];
  const int groups = m.ops[hi - 1].d.i[0];
  if (groups < 1 || c % groups) return false;
  const int64_t cpg = c / groups;
  if (cpg != 2 && cpg != 4 && cpg != 8 && cpg != 16 && cpg != 32) return false;
  return groupnorm_apply_partials_supported(dt(m), c, groups);
}
size_t conv_gn_tc2_scratch(const Module& m, int, int hi) {
  const mk_tensor_spec& s = m.vspec(m.ops[hi - 1].out_id);
  const size_t act = (size_t)s.shape[0] * s.shape[1] * s.shape[2] * s.shape[3] * 2;
  const size_t st = (size_t)s.shape[0] * conv3x3_tc2_stat_slots(s.shape[1], s.shape[2]) * m.ops[hi - 1].d.i[0] * 2 * sizeof(float);
  return align_up(act, 1024) + st;
}
mk_status conv_gn_tc2_emit(const Module& m, int lo, int hi, const Resolved& r, std::vector<Launch>& out, std::string& err) {
  EpiProgram p;
  mk_status st = build_epi(m, lo + 1, hi - 1, r, p, err);
  if (st != MK_OK) return st;
  const Op& op = m.ops[lo];
  const Op& gn = m.ops[hi - 1];
  const mk_tensor_spec& xs = m.vspec(op.in_id[0]);
  const mk_tensor_spec& ys = m.vspec(gn.out_id);
  const int64_t nb = ys.shape[0], hw = ys.shape[1] * ys.shape[2], c = ys.shape[3];
  const int groups = gn.d.i[0];
  char* act = (char*)r.scratch;
  float* stats = (float*)(act + align_up((size_t)nb * hw * c * 2, 1024));
  const int slots = conv3x3_tc2_stat_slots(ys.shape[1], ys.shape[2]);
  auto plan = std::make_shared<ConvTcPlan>();
  cudaError_t e = conv3x3_tc2_plan(plan.get(), r.value_ptr[op.in_id[0]], op.param[0].ptr, act, xs.shape[0], xs.shape[1], xs.shape[2],
                                   xs.shape[3], op.d.i[0], p, m.ctx->sm_count);
  if (e != cudaSuccess) { err = std::string("conv3x3_tc2 plan: ") + cudaGetErrorString(e); return MK_ERR_CUDA; }
  plan->stats = stats;
  plan->cpg = (int)(c / groups);
  out.push_back([plan](cudaStream_t s) { return launch_conv3x3_tc2(*plan, s); });
  void* y = r.value_ptr[gn.out_id];
  const void* g = gn.param[0].set ? gn.param[0].ptr : nullptr;
  const void* b = gn.param[1].set ? gn.param[1].ptr : nullptr;
  const float eps = (float)gn.d.f[0];
  const int d = dt(m), sms = m.ctx->sm_count;
  out.push_back([=](cudaStream_t s_) { return launch_groupnorm_apply_partials(d, act, y, nb, hw, c, groups, g, b, eps, stats, slots, sms, s_); });
  return MK_OK;
}

// ------------------------------------------------------------------ attention
AttnView attn_view(const Module& m, const Op& op, const Resolved& r) {
  AttnView a{};
  a.causal = op.d.kind == MK_OP_ATTENTION_CAUSAL;
  const int64_t H = op.d.i[0], D = op.d.i[1];
  const size_t es = dtype_size(m.dtype);
  if (op.d.i[2] == 0) {
    const mk_tensor_spec& q = m.vspec(op.in_id[0]);
    a.q = r.value_ptr[op.in_id[0]];
    a.k = r.value_ptr[op.in_id[1]];
    a.v = r.value_ptr[op.in_id[2]];
    a.B = q.shape[0]; a.H = H; a.S = q.shape[2]; a.D = D;
    a.sb = H * a.S * D; a.sh = a.S * D; a.ss = D;
  } else {
    const char* base = (const char*)r.value_ptr[op.in_id[0]];
    const int64_t E = H * D;
    a.q = base;
    a.k = base + E * es;
    a.v = base + 2 * E * es;
    a.B = op.d.i[2]; a.H = H; a.S = op.d.i[3]; a.D = D;
    a.sb = a.S * 3 * E; a.sh = D; a.ss = 3 * E;
  }
  return a;
}
bool is_attention(int32_t k) { return k == MK_OP_ATTENTION_CAUSAL || k == MK_OP_ATTENTION; }
bool attn_tc_match(const Module& m, int lo, int hi) {
  if (hi - lo != 1 || !is_attention(m.ops[lo].d.kind) || m.dtype != MK_BF16) return false;
  Resolved none;
  none.value_ptr.assign(m.values.size(), nullptr);
  return attention_tc_supported(attn_view(m, m.ops[lo], none));
}
mk_status attn_tc_emit(const Module& m, int lo, int, const Resolved& r, std::vector<Launch>& out, std::string& err) {
  const Op& op = m.ops[lo];
  auto plan = std::make_shared<AttnTcPlan>();
  cudaError_t e = attention_tc_plan(plan.get(), attn_view(m, op, r), r.value_ptr[op.out_id]);
  if (e != cudaSuccess) { err = std::string("attention_tc plan: ") + cudaGetErrorString(e); return MK_ERR_CUDA; }
  out.push_back([plan](cudaStream_t s) { return launch_attention_tc(*plan, s); });
  return MK_OK;
}
bool attn_tc2_match(const Module& m, int lo, int hi) {
  if (hi - lo != 1 || !is_attention(m.ops[lo].d.kind) || m.dtype != MK_BF16) return false;
  Resolved none;
  none.value_ptr.assign(m.values.size(), nullptr);
  return attention_tc2_supported(attn_view(m, m.ops[lo], none));
}
mk_status attn_tc2_emit(const Module& m, int lo, int, const Resolved& r, std::vector<Launch>& out, std::string& err) {
  const Op& op = m.ops[lo];
  auto plan = std::make_shared<AttnTcPlan>();
  cudaError_t e = attention_tc2_plan(plan.get(), attn_view(m, op, r), r.value_ptr[op.out_id], m.ctx->sm_count);
  if (e != cudaSuccess) { err = std::string("attention_tc2 plan: ") + cudaGetErrorString(e); return MK_ERR_CUDA; }
  out.push_back([plan](cudaStream_t s) { return launch_attention_tc2(*plan, s); });
  return MK_OK;
}
bool attn_simt_match(const Module& m, int lo, int hi) {
  return hi - lo == 1 && (m.ops[lo].d.kind == MK_OP_ATTENTION_CAUSAL || m.ops[lo].d.kind == MK_OP_ATTENTION) && m.ops[lo].d.i[1] <= 256;
}
mk_status attn_simt_emit(const Module& m, int lo, int, const Resolved& r, std::vector<Launch>& out, std::string&) {
  const Op& op = m.ops[lo];
  const AttnView a = attn_view(m, op, r);
  void* o = r.value_ptr[op.out_id];
  const int d = dt(m);
  out.push_back([=](cudaStream_t s) { return launch_attention_simt(d, a, o, s); });
  return MK_OK;
}

}  // namespace

const std::vector<Impl>& registry() {
  static const std::vector<Impl> reg = {
      {"linear_rownorm_simt", linear_rownorm_match, no_scratch, linear_rownorm_emit},
      {"gemm_prenorm_gemm_tc2", gemm_prenorm_match, gemm_prenorm_scratch_fn, gemm_prenorm_emit, false},
      {"gemm_rownorm_cl", gemm_rownorm_cl_match, no_scratch, gemm_rownorm_cl_emit, false},
      {"gemm_rownorm_tc2", gemm_rownorm_tc2_match, gemm_rownorm_tc2_scratch_fn, gemm_rownorm_tc2_emit, false},
      {"gemm_tc2", gemm_tc2_match, no_scratch, gemm_tc2_emit},
      {"gemm_tc", gemm_tc_match, no_scratch, gemm_tc_emit},
      {"gemm_simt", gemm_simt_match, no_scratch, gemm_simt_emit},
      {"gemm_fp8_tc2", gemm_fp8_tc2_match, no_scratch, gemm_fp8_tc2_emit},
      {"gemm_fp8_simt", gemm_fp8_simt_match, no_scratch, gemm_fp8_simt_emit},
      {"conv3x3_gn_tc2", conv_gn_tc2_match, conv_gn_tc2_scratch, conv_gn_tc2_emit},
      {"conv3x3_tc2", conv_tc2_match, no_scratch, conv_tc2_emit},
      {"conv3x3_simt", conv_simt_match, no_scratch, conv_simt_emit},
      {"attention_tc2", attn_tc2_match, no_scratch, attn_tc2_emit},
      {"attention_tc", attn_tc_match, no_scratch, attn_tc_emit},
      {"attention_simt", attn_simt_match, no_scratch, attn_simt_emit},
      {"rowop", rowop_match, no_scratch, rowop_emit},
      {"groupnorm_nhwc", groupnorm_match, groupnorm_scratch, groupnorm_emit},
      {"eltwise", eltwise_match, no_scratch, eltwise_emit},
      {"pool_nhwc", pool_match, no_scratch, pool_emit},
  };
  return reg;
}

}  // namespace mk
