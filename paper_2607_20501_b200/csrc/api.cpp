// extern "C" surface declared in include/mk.h: argument checking and transactional edits around
// the composer.  No math here.
#include <cstring>
#include <new>

#include "mk_internal.h"

using namespace mk;

struct mk_ctx : Ctx {};
struct mk_module : Module {};

namespace {

mk_status fail(const Ctx* c, mk_status st, const std::string& msg) {
  if (c) c->err = msg;
  return st;
}

mk_status bind_all_default(Module& m, const std::vector<int>& cuts, std::vector<Binding>& out, std::string& err) {
  out.clear();
  const int n = (int)cuts.size();
  for (int s = 0; s < n; ++s) {
    const int lo = cuts[s], hi = s + 1 < n ? cuts[s + 1] : (int)m.ops.size();
    Binding b;
    mk_status st = default_binding(m, lo, hi, b, err);
    if (st != MK_OK) {
      err = "submodule " + std::to_string(s) + ": " + err;
      return st;
    }
    out.push_back(std::move(b));
  }
  return MK_OK;
}

void invalidate(Module& m) {
  m.layout_valid = false;
  m.plan_valid = false;
}

}  // namespace

extern "C" {

const char* mk_status_str(mk_status s) {
  switch (s) {
    case MK_OK: return "MK_OK";
    case MK_ERR_INVALID_ARG: return "MK_ERR_INVALID_ARG";
    case MK_ERR_SHAPE_MISMATCH: return "MK_ERR_SHAPE_MISMATCH";
    case MK_ERR_NO_IMPL: return "MK_ERR_NO_IMPL";
    case MK_ERR_CONTRACT_VIOLATION: return "MK_ERR_CONTRACT_VIOLATION";
    case MK_ERR_WORKSPACE_TOO_SMALL: return "MK_ERR_WORKSPACE_TOO_SMALL";
    case MK_ERR_UNSUPPORTED_ARCH: return "MK_ERR_UNSUPPORTED_ARCH";
    case MK_ERR_CUDA: return "MK_ERR_CUDA";
    case MK_ERR_DEVICE_TIMEOUT: return "MK_ERR_DEVICE_TIMEOUT";
    case MK_ERR_NO_DEVICE: return "MK_ERR_NO_DEVICE";
    case MK_ERR_PARAM_MISSING: return "MK_ERR_PARAM_MISSING";
    default: return "MK_ERR_UNKNOWN";
  }
}

mk_status mk_ctx_create(int32_t device, mk_ctx** out) {
  if (!out || device < -1) return MK_ERR_INVALID_ARG;
  mk_ctx* c = new (std::nothrow) mk_ctx();
  if (!c) return MK_ERR_INVALID_ARG;
  c->device = device;
  if (device >= 0) {
    int n = 0;
    if (cudaGetDeviceCount(&n) != cudaSuccess || device >= n) {
      cudaGetLastError();
      delete c;
      return MK_ERR_NO_DEVICE;
    }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { delete c; return MK_ERR_CUDA; }
    if (prop.major != 10) { delete c; return MK_ERR_UNSUPPORTED_ARCH; }
    c->sm_count = prop.multiProcessorCount;
    if (cudaSetDevice(device) != cudaSuccess) { delete c; return MK_ERR_CUDA; }
  } else {
    c->sm_count = 148;  // planning only
  }
  *out = c;
  return MK_OK;
}

void mk_ctx_destroy(mk_ctx* ctx) { delete ctx; }

const char* mk_last_error(const mk_ctx* ctx) { return ctx ? ctx->err.c_str() : ""; }

mk_status mk_ctx_check(mk_ctx* ctx) {
  if (!ctx) return MK_ERR_INVALID_ARG;
  if (ctx->device < 0) return MK_ERR_NO_DEVICE;
  if (current_device() != ctx->device)
    return fail(ctx, MK_ERR_INVALID_ARG, "the context's device must be the calling thread's current CUDA device");
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return fail(ctx, MK_ERR_CUDA, cudaGetErrorString(e));
  unsigned int flag = 0;
  e = kernel_status_fetch_and_clear(&flag);
  if (e != cudaSuccess) return fail(ctx, MK_ERR_CUDA, cudaGetErrorString(e));
  if (flag) return fail(ctx, MK_ERR_DEVICE_TIMEOUT, "a bounded wait inside a kernel expired (code " + std::to_string(flag) + ")");
  return MK_OK;
}

mk_status mk_selftest_bounded_wait(mk_ctx* ctx, int64_t limit_cycles, int64_t* dev_out6, void* cuda_stream) {
  if (!ctx || !dev_out6 || ((uintptr_t)dev_out6 & 7)) return MK_ERR_INVALID_ARG;
  if (ctx->device < 0) return MK_ERR_NO_DEVICE;
  // a limit a test can afford: between a microsecond and a tenth of a second of SM cycles
  if (limit_cycles < 1000 || limit_cycles > 200000000) return fail(ctx, MK_ERR_INVALID_ARG, "limit_cycles must lie in [1e3, 2e8]");
  if (current_device() != ctx->device)
    return fail(ctx, MK_ERR_INVALID_ARG, "the context's device must be the calling thread's current CUDA device");
  cudaError_t e = launch_bounded_wait_selftest((long long)limit_cycles, (long long*)dev_out6, (cudaStream_t)cuda_stream);
  if (e != cudaSuccess) return fail(ctx, MK_ERR_CUDA, cudaGetErrorString(e));
  return MK_OK;
}

mk_status mk_module_create(mk_ctx* ctx, const mk_op_desc* ops, int32_t n_ops, const mk_tensor_spec* inputs,
                           int32_t n_inputs, mk_module** out) {
  if (!ctx || !out) return MK_ERR_INVALID_ARG;
  if (!ops || n_ops < 1 || !inputs || n_inputs < 1) return fail(ctx, MK_ERR_INVALID_ARG, "ops and inputs must be non-empty");
  mk_module* m = new (std::nothrow) mk_module();
  if (!m) return MK_ERR_INVALID_ARG;
  m->ctx = ctx;
  m->n_inputs = n_inputs;
  m->values.resize((size_t)n_inputs + n_ops);
  for (int k = 0; k < n_inputs; ++k) m->values[k].spec = inputs[k];
  m->ops.resize(n_ops);
  for (int j = 0; j < n_ops; ++j) m->ops[j].d = ops[j];
  std::string err;
  mk_status st = infer_shapes(*m, err);
  if (st == MK_OK) {
    std::vector<int> cuts(n_ops);
    for (int j = 0; j < n_ops; ++j) cuts[j] = j;
    std::vector<Binding> b;
    st = bind_all_default(*m, cuts, b, err);
    if (st == MK_OK) { m->cuts = cuts; m->bind = std::move(b); }
  }
  if (st != MK_OK) { delete m; return fail(ctx, st, err); }
  *out = m;
  return MK_OK;
}

void mk_module_destroy(mk_module* m) { delete m; }

mk_status mk_module_n_ops(const mk_module* m, int32_t* n) {
  if (!m || !n) return MK_ERR_INVALID_ARG;
  *n = (int32_t)m->ops.size();
  return MK_OK;
}

mk_status mk_module_value_spec(const mk_module* m, int32_t value_id, mk_tensor_spec* out) {
  if (!m || !out) return MK_ERR_INVALID_ARG;
  if (value_id < 0 || value_id >= (int)m->values.size()) return fail(m->ctx, MK_ERR_INVALID_ARG, "value id out of range");
  *out = m->values[value_id].spec;
  return MK_OK;
}

mk_status mk_module_set_decomposition(mk_module* m, const int32_t* first, int32_t n_sub) {
  if (!m || !first) return MK_ERR_INVALID_ARG;
  const int n_ops = (int)m->ops.size();
  if (n_sub < 1 || n_sub > n_ops || first[0] != 0)
    return fail(m->ctx, MK_ERR_CONTRACT_VIOLATION, "a decomposition starts at operator 0 and has 1..n_ops submodules");
  for (int s = 1; s < n_sub; ++s)
    if (first[s] <= first[s - 1] || first[s] >= n_ops)
      return fail(m->ctx, MK_ERR_CONTRACT_VIOLATION, "submodules must be contiguous, non-empty and cover every operator exactly once");
  std::vector<int> cuts(first, first + n_sub);
  std::vector<Binding> b;
  std::string err;
  mk_status st = bind_all_default(*m, cuts, b, err);
  if (st != MK_OK) return fail(m->ctx, st, err);
  // keep explicit bindings of submodules whose operator range did not change
  for (int s = 0; s < n_sub; ++s) {
    const int lo = cuts[s], hi = s + 1 < n_sub ? cuts[s + 1] : n_ops;
    for (int t = 0; t < m->n_sub(); ++t)
      if (m->sub_lo(t) == lo && m->sub_hi(t) == hi && m->bind[t].explicit_bind) b[s] = m->bind[t];
  }
  m->cuts = std::move(cuts);
  m->bind = std::move(b);
  invalidate(*m);
  return MK_OK;
}

mk_status mk_module_n_sub(const mk_module* m, int32_t* n) {
  if (!m || !n) return MK_ERR_INVALID_ARG;
  *n = m->n_sub();
  return MK_OK;
}

mk_status mk_module_get_decomposition(const mk_module* m, int32_t* first, int32_t* n_sub) {
  if (!m || !first || !n_sub) return MK_ERR_INVALID_ARG;
  if (*n_sub < m->n_sub()) return fail(m->ctx, MK_ERR_INVALID_ARG, "array too small");
  for (int s = 0; s < m->n_sub(); ++s) first[s] = m->cuts[s];
  *n_sub = m->n_sub();
  return MK_OK;
}

mk_status mk_module_split(mk_module* m, int32_t sub, int32_t at_op) {
  if (!m) return MK_ERR_INVALID_ARG;
  if (sub < 0 || sub >= m->n_sub()) return fail(m->ctx, MK_ERR_INVALID_ARG, "submodule index out of range");
  if (at_op <= m->sub_lo(sub) || at_op >= m->sub_hi(sub))
    return fail(m->ctx, MK_ERR_CONTRACT_VIOLATION, "split point must lie strictly inside the submodule: both halves non-empty");
  std::vector<int32_t> cuts(m->cuts.begin(), m->cuts.end());
  cuts.insert(cuts.begin() + sub + 1, at_op);
  return mk_module_set_decomposition(m, cuts.data(), (int32_t)cuts.size());
}

mk_status mk_module_fuse(mk_module* m, int32_t first_sub, int32_t count) {
  if (!m) return MK_ERR_INVALID_ARG;
  if (first_sub < 0 || count < 2 || first_sub + count > m->n_sub())
    return fail(m->ctx, MK_ERR_INVALID_ARG, "fuse needs count >= 2 adjacent submodules inside the decomposition");
  std::vector<int32_t> cuts(m->cuts.begin(), m->cuts.end());
  cuts.erase(cuts.begin() + first_sub + 1, cuts.begin() + first_sub + count);
  return mk_module_set_decomposition(m, cuts.data(), (int32_t)cuts.size());
}

mk_status mk_module_total_fuse(mk_module* m) {
  if (!m) return MK_ERR_INVALID_ARG;
  const int32_t zero = 0;
  return mk_module_set_decomposition(m, &zero, 1);
}

mk_status mk_module_get_contract(const mk_module* m, int32_t sub, int32_t* in_ids, mk_tensor_spec* in_specs, int32_t* n_in,
                                 int32_t* out_ids, mk_tensor_spec* out_specs, int32_t* n_out) {
  if (!m || !n_in || !n_out) return MK_ERR_INVALID_ARG;
  if (sub < 0 || sub >= m->n_sub()) return fail(m->ctx, MK_ERR_INVALID_ARG, "submodule index out of range");
  std::vector<int> ins, outs;
  contract_of(*m, m->sub_lo(sub), m->sub_hi(sub), ins, outs);
  if (((in_ids || in_specs) && *n_in < (int)ins.size()) || ((out_ids || out_specs) && *n_out < (int)outs.size()))
    return fail(m->ctx, MK_ERR_INVALID_ARG, "contract arrays too small");
  for (size_t i = 0; i < ins.size(); ++i) {
    if (in_ids) in_ids[i] = ins[i];
    if (in_specs) in_specs[i] = m->values[ins[i]].spec;
  }
  for (size_t i = 0; i < outs.size(); ++i) {
    if (out_ids) out_ids[i] = outs[i];
    if (out_specs) out_specs[i] = m->values[outs[i]].spec;
  }
  *n_in = (int32_t)ins.size();
  *n_out = (int32_t)outs.size();
  return MK_OK;
}

mk_status mk_impl_count(const mk_module* m, int32_t sub, int32_t* n) {
  if (!m || !n) return MK_ERR_INVALID_ARG;
  if (sub < 0 || sub >= m->n_sub()) return fail(m->ctx, MK_ERR_INVALID_ARG, "submodule index out of range");
  int c = 0;
  for (const Impl& im : registry())
    if (im.match(*m, m->sub_lo(sub), m->sub_hi(sub))) ++c;
  *n = c;
  return MK_OK;
}

mk_status mk_impl_name(const mk_module* m, int32_t sub, int32_t i, const char** name) {
  if (!m || !name) return MK_ERR_INVALID_ARG;
  if (sub < 0 || sub >= m->n_sub()) return fail(m->ctx, MK_ERR_INVALID_ARG, "submodule index out of range");
  int c = 0;
  for (const Impl& im : registry())
    if (im.match(*m, m->sub_lo(sub), m->sub_hi(sub))) {
      if (c == i) { *name = im.name; return MK_OK; }
      ++c;
    }
  return fail(m->ctx, MK_ERR_INVALID_ARG, "implementation index out of range");
}

mk_status mk_module_bind(mk_module* m, int32_t sub, const char* impl_name) {
  if (!m) return MK_ERR_INVALID_ARG;
  if (sub < 0 || sub >= m->n_sub()) return fail(m->ctx, MK_ERR_INVALID_ARG, "submodule index out of range");
  Binding b;
  std::string err;
  mk_status st = impl_name ? explicit_binding(*m, m->sub_lo(sub), m->sub_hi(sub), impl_name, b, err)
                           : default_binding(*m, m->sub_lo(sub), m->sub_hi(sub), b, err);
  if (st != MK_OK) return fail(m->ctx, st, err);
  m->bind[sub] = std::move(b);
  invalidate(*m);
  return MK_OK;
}

mk_status mk_module_bound_impl(const mk_module* m, int32_t sub, const char** name) {
  if (!m || !name) return MK_ERR_INVALID_ARG;
  if (sub < 0 || sub >= m->n_sub()) return fail(m->ctx, MK_ERR_INVALID_ARG, "submodule index out of range");
  *name = m->bind[sub].name.c_str();
  return MK_OK;
}

mk_status mk_module_set_param(mk_module* m, int32_t op, int32_t slot, const void* dev_ptr, const mk_tensor_spec* spec) {
  if (!m || !spec) return MK_ERR_INVALID_ARG;
  if (op < 0 || op >= (int)m->ops.size() || slot < 0 || slot > 1) return fail(m->ctx, MK_ERR_INVALID_ARG, "operator or slot out of range");
  if (!dev_ptr || ((uintptr_t)dev_ptr & 15)) return fail(m->ctx, MK_ERR_INVALID_ARG, "parameter pointer must be non-null and 16-byte aligned");
  Op& o = m->ops[op];
  const mk_tensor_spec& x = m->values[o.in_id[0]].spec;
  const int64_t last = x.shape[x.rank - 1];
  mk_tensor_spec want{};
  want.dtype = m->dtype;   // parameters always have the module's storage type
  bool ok = false;
  switch (o.d.kind) {
    case MK_OP_LINEAR:
      if (slot == 0) { want.rank = 2; want.shape[0] = last; want.shape[1] = o.d.i[0]; want.layout = o.d.i[1]; ok = true; }
      break;
    case MK_OP_LINEAR_FP8:
      if (slot == 0) { want.dtype = MK_FP8_E4M3; want.rank = 2; want.shape[0] = last; want.shape[1] = o.d.i[0]; want.layout = o.d.i[1]; ok = true; }
      else { want.dtype = MK_F32; want.rank = 2; want.shape[0] = (o.d.i[0] + 127) / 128; want.shape[1] = last / 128; ok = true; }
      break;
    case MK_OP_CONV2D_3X3:
      if (slot == 0) { want.rank = 4; want.shape[0] = o.d.i[0]; want.shape[1] = 3; want.shape[2] = 3; want.shape[3] = last; ok = true; }
      break;
    case MK_OP_BIAS_ADD:
    case MK_OP_RMSNORM:
      if (slot == 0) { want.rank = 1; want.shape[0] = last; ok = true; }
      break;
    case MK_OP_LAYERNORM:
    case MK_OP_GROUPNORM:
      want.rank = 1; want.shape[0] = last; ok = true;
      break;
    default:
      break;
  }
  if (!ok) return fail(m->ctx, MK_ERR_INVALID_ARG, "this operator has no such parameter slot");
  if (!same_spec(want, *spec)) return fail(m->ctx, MK_ERR_SHAPE_MISMATCH, "parameter spec does not match what the operator expects");
  o.param[slot].ptr = dev_ptr;
  o.param[slot].spec = *spec;
  o.param[slot].set = true;
  m->plan_valid = false;
  return MK_OK;
}

mk_status mk_module_keep_intermediates(mk_module* m, int32_t keep) {
  if (!m) return MK_ERR_INVALID_ARG;
  m->keep_intermediates = keep != 0;
  invalidate(*m);
  return MK_OK;
}

mk_status mk_module_workspace_size(mk_module* m, size_t* bytes) {
  if (!m || !bytes) return MK_ERR_INVALID_ARG;
  if (!m->layout_valid) {
    std::string err;
    mk_status st = plan_layout(*m, err);
    if (st != MK_OK) return fail(m->ctx, st, err);
  }
  *bytes = m->workspace_bytes;
  return MK_OK;
}

static mk_status ensure_plan(mk_module* m, const void* const* in_ptrs, void* const* out_ptrs, void* ws, size_t ws_bytes) {
  if (!m || !in_ptrs || !out_ptrs) return MK_ERR_INVALID_ARG;
  if (m->ctx->device < 0) return fail(m->ctx, MK_ERR_NO_DEVICE, "host-only planning context cannot launch");
  // Launches go to the calling thread's current device; the module's buffers, descriptors and status word
  // belong to its context's device.  A process may hold contexts on several GPUs, so the two must agree.
  if (current_device() != m->ctx->device)
    return fail(m->ctx, MK_ERR_INVALID_ARG, "the context's device (" + std::to_string(m->ctx->device) +
                                               ") must be the calling thread's current CUDA device");
  std::string err;
  mk_status st = build_plan(*m, in_ptrs, out_ptrs, ws, ws_bytes, err);
  if (st != MK_OK) return fail(m->ctx, st, err);
  return MK_OK;
}

mk_status mk_module_launch_count(mk_module* m, int32_t* n) {
  if (!m || !n) return MK_ERR_INVALID_ARG;
  if (!m->plan_valid) return fail(m->ctx, MK_ERR_INVALID_ARG, "no launch plan yet: run a forward first");
  *n = (int32_t)m->launches.size();
  return MK_OK;
}

mk_status mk_module_forward(mk_module* m, const void* const* in_ptrs, void* const* out_ptrs, void* workspace,
                            size_t workspace_bytes, void* cuda_stream) {
  mk_status st = ensure_plan(m, in_ptrs, out_ptrs, workspace, workspace_bytes);
  if (st != MK_OK) return st;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  for (size_t q = 0; q < m->launches.size(); ++q) {
    cudaError_t e = m->launches[q](s);
    if (e != cudaSuccess) {
      const int sub = q < m->launch_sub.size() ? m->launch_sub[q] : -1;
      return fail(m->ctx, MK_ERR_CUDA, "launch " + std::to_string(q) + " (submodule " + std::to_string(sub) + ", " +
                                           (sub >= 0 && sub < (int)m->bind.size() ? m->bind[sub].name : std::string("?")) + "): " + cudaGetErrorString(e));
    }
  }
  return MK_OK;
}

mk_status mk_module_forward_sub(mk_module* m, const void* const* in_ptrs, void* const* out_ptrs, void* workspace,
                                size_t workspace_bytes, void* cuda_stream, int32_t first_sub, int32_t count) {
  mk_status st = ensure_plan(m, in_ptrs, out_ptrs, workspace, workspace_bytes);
  if (st != MK_OK) return st;
  if (first_sub < 0 || count < 1 || first_sub + count > m->n_sub()) return fail(m->ctx, MK_ERR_INVALID_ARG, "submodule range outside the decomposition");
  cudaStream_t s = (cudaStream_t)cuda_stream;
  for (size_t q = 0; q < m->launches.size(); ++q) {
    const int sub = m->launch_sub[q];
    if (sub < first_sub || sub >= first_sub + count) continue;
    cudaError_t e = m->launches[q](s);
    if (e != cudaSuccess)
      return fail(m->ctx, MK_ERR_CUDA, "launch " + std::to_string(q) + " (submodule " + std::to_string(sub) + ", " + m->bind[sub].name + "): " + cudaGetErrorString(e));
  }
  return MK_OK;
}

mk_status mk_module_profile(mk_module* m, const void* const* in_ptrs, void* const* out_ptrs, void* workspace,
                            size_t workspace_bytes, void* cuda_stream, int32_t iters, float* ms_per_sub) {
  if (!ms_per_sub || iters < 1) return MK_ERR_INVALID_ARG;
  mk_status st = ensure_plan(m, in_ptrs, out_ptrs, workspace, workspace_bytes);
  if (st != MK_OK) return st;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const int ns = m->n_sub();
  std::vector<cudaEvent_t> ev(ns + 1);
  for (auto& e : ev)
    if (cudaEventCreate(&e) != cudaSuccess) return fail(m->ctx, MK_ERR_CUDA, "cudaEventCreate failed");
  std::vector<double> acc(ns, 0.0);
  mk_status ret = MK_OK;
  for (int it = 0; it < iters && ret == MK_OK; ++it) {
    cudaEventRecord(ev[0], s);
    size_t q = 0;
    for (int sub = 0; sub < ns; ++sub) {
      while (q < m->launches.size() && m->launch_sub[q] == sub) {
        cudaError_t e = m->launches[q](s);
        if (e != cudaSuccess) { ret = fail(m->ctx, MK_ERR_CUDA, cudaGetErrorString(e)); break; }
        ++q;
      }
      cudaEventRecord(ev[sub + 1], s);
    }
    cudaError_t e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) { ret = fail(m->ctx, MK_ERR_CUDA, cudaGetErrorString(e)); break; }
    for (int sub = 0; sub < ns; ++sub) {
      float ms = 0.f;
      cudaEventElapsedTime(&ms, ev[sub], ev[sub + 1]);
      acc[sub] += ms;
    }
  }
  for (auto& e : ev) cudaEventDestroy(e);
  if (ret == MK_OK)
    for (int sub = 0; sub < ns; ++sub) ms_per_sub[sub] = (float)(acc[sub] / iters);
  return ret;
}

mk_status mk_module_swap(mk_module* m, const void* const* in_ptrs, void* const* out_ptrs, void* workspace, size_t workspace_bytes,
                         void* cuda_stream, int32_t iters, double tau, int32_t* n_swapped, float* ms_before_after) {
  if (!m || iters < 1 || !(tau > 0.0) || tau > 1.0) return MK_ERR_INVALID_ARG;
  if (n_swapped) *n_swapped = 0;
  const int ns = m->n_sub();
  std::vector<float> base(ns, 0.f), ms(ns, 0.f);
  mk_status st = mk_module_profile(m, in_ptrs, out_ptrs, workspace, workspace_bytes, cuda_stream, iters, base.data());
  if (st != MK_OK) return st;
  if (ms_before_after)
    for (int s_ = 0; s_ < ns; ++s_) ms_before_after[2 * s_] = ms_before_after[2 * s_ + 1] = base[s_];
  if (ns < 2) return MK_OK;
  int swapped = 0;
  for (int sub = 0; sub < ns; ++sub) {
    const Binding original = m->bind[sub];
    std::string best_name = original.name;
    float best_ms = base[sub];
    std::vector<const char*> cands;
    for (const Impl& im : registry())
      if (im.match(*m, m->sub_lo(sub), m->sub_hi(sub)) && original.name != im.name) cands.push_back(im.name);
    for (const char* cand : cands) {
      if (mk_module_bind(m, sub, cand) != MK_OK) continue;
      size_t need = 0;
      if (mk_module_workspace_size(m, &need) != MK_OK || need > workspace_bytes) continue;
      // one run first: it builds the plan and shows whether the alternative is in the race at all
      if (mk_module_profile(m, in_ptrs, out_ptrs, workspace, workspace_bytes, cuda_stream, 1, ms.data()) != MK_OK) continue;
      if (ms[sub] > 4.0f * best_ms) continue;
      if (mk_module_profile(m, in_ptrs, out_ptrs, workspace, workspace_bytes, cuda_stream, iters, ms.data()) != MK_OK) continue;
      if (ms[sub] < best_ms) { best_ms = ms[sub]; best_name = cand; }
    }
    // the bound one keeps its place unless it reaches less than tau of the fastest one's speed
    if (best_name != original.name && (double)best_ms < tau * (double)base[sub]) {
      st = mk_module_bind(m, sub, best_name.c_str());
      if (st != MK_OK) { m->bind[sub] = original; invalidate(*m); return st; }
      ++swapped;
      if (ms_before_after) ms_before_after[2 * sub + 1] = best_ms;
    } else {
      m->bind[sub] = original;
      invalidate(*m);
    }
  }
  if (n_swapped) *n_swapped = swapped;
  // leave a valid result of the final composition in the caller's output
  size_t need = 0;
  st = mk_module_workspace_size(m, &need);
  if (st != MK_OK) return st;
  return mk_module_profile(m, in_ptrs, out_ptrs, workspace, workspace_bytes, cuda_stream, 1, ms.data());
}

mk_status mk_module_intermediate(const mk_module* m, int32_t value_id, const void** dev_ptr, mk_tensor_spec* spec) {
  if (!m || !dev_ptr) return MK_ERR_INVALID_ARG;
  if (value_id < 0 || value_id >= (int)m->values.size()) return fail(m->ctx, MK_ERR_INVALID_ARG, "value id out of range");
  if (!m->plan_valid || !m->keep_intermediates)
    return fail(m->ctx, MK_ERR_INVALID_ARG, "needs keep_intermediates and a completed forward");
  void* p = m->last_value_ptr[value_id];
  if (!p) return fail(m->ctx, MK_ERR_INVALID_ARG, "value is internal to a fused subkernel: it never reaches memory");
  *dev_ptr = p;
  if (spec) *spec = m->values[value_id].spec;
  return MK_OK;
}

}  // extern "C"
