// Composer host logic: shape inference over the operator sequence, contracts of a contiguous
// decomposition, implementation choice (widest legal fused piece first), workspace layout and
// the launch plan.  Paper: Methodology (codebase = subkernels + a top-level module that only
// chains them; Split / Fuse / TotalFuse edits) and the decomposition rules of its appendix
// "Prompts" (what fuses, what blocks fusion).
#include <algorithm>
#include <cstring>

#include "mk_internal.h"

namespace mk {

int64_t numel(const mk_tensor_spec& s) {
  int64_t n = 1;
  for (int i = 0; i < s.rank; ++i) n *= s.shape[i];
  return n;
}
size_t dtype_size(int32_t dtype) { return dtype == MK_F32 ? 4 : dtype == MK_FP8_E4M3 ? 1 : 2; }
size_t spec_bytes(const mk_tensor_spec& s) { return (size_t)numel(s) * dtype_size(s.dtype); }
bool same_spec(const mk_tensor_spec& a, const mk_tensor_spec& b) {
  if (a.dtype != b.dtype || a.rank != b.rank || a.layout != b.layout) return false;
  for (int i = 0; i < a.rank; ++i)
    if (a.shape[i] != b.shape[i]) return false;
  return true;
}
static bool same_shape(const mk_tensor_spec& a, const mk_tensor_spec& b) {
  if (a.rank != b.rank || a.layout != b.layout) return false;
  for (int i = 0; i < a.rank; ++i)
    if (a.shape[i] != b.shape[i]) return false;
  return true;
}
bool is_eltwise(int32_t kind) {
  switch (kind) {
    case MK_OP_BIAS_ADD:
    case MK_OP_RELU:
    case MK_OP_GELU_TANH:
    case MK_OP_GELU_ERF:
    case MK_OP_SILU:
    case MK_OP_SCALE:
    case MK_OP_CLAMP:
    case MK_OP_RESIDUAL_ADD:
      return true;
    default:
      return false;
  }
}

static mk_tensor_spec make_spec(int32_t dtype, std::initializer_list<int64_t> shape) {
  mk_tensor_spec s{};
  s.dtype = dtype;
  s.rank = (int32_t)shape.size();
  int i = 0;
  for (int64_t v : shape) s.shape[i++] = v;
  s.layout = MK_LAYOUT_ROW_MAJOR;
  return s;
}

static int n_inputs_of(const mk_op_desc& d) {
  if (d.kind == MK_OP_RESIDUAL_ADD || d.kind == MK_OP_LINEAR_FP8) return 2;
  if (d.kind == MK_OP_ATTENTION_CAUSAL || d.kind == MK_OP_ATTENTION) return d.i[2] == 0 ? 3 : 1;
  return 1;
}

mk_status infer_shapes(Module& m, std::string& err) {
  const int n_in = m.n_inputs;
  if (n_in < 1) { err = "a module needs at least one input"; return MK_ERR_INVALID_ARG; }
  // the activations' storage type: that of the inputs; a module with an fp8 input is a bf16 module whose other
  // inputs may be fp32 (block scales) or bf16
  bool has_fp8 = false;
  for (int k = 0; k < n_in; ++k) has_fp8 = has_fp8 || m.values[k].spec.dtype == MK_FP8_E4M3;
  m.dtype = has_fp8 ? MK_BF16 : m.values[0].spec.dtype;
  const int32_t dtype = m.dtype;
  for (int k = 0; k < n_in; ++k) {
    const mk_tensor_spec& s = m.values[k].spec;
    if (s.dtype != MK_F32 && s.dtype != MK_BF16 && s.dtype != MK_FP8_E4M3) { err = "input dtype must be MK_F32, MK_BF16 or MK_FP8_E4M3"; return MK_ERR_INVALID_ARG; }
    if (s.dtype != dtype && !has_fp8) { err = "all module inputs must share one dtype"; return MK_ERR_INVALID_ARG; }
    if (s.rank < 1 || s.rank > MK_MAX_RANK) { err = "input rank out of range"; return MK_ERR_INVALID_ARG; }
    if (s.layout != MK_LAYOUT_ROW_MAJOR) { err = "module inputs must be row-major"; return MK_ERR_INVALID_ARG; }
    for (int i = 0; i < s.rank; ++i)
      if (s.shape[i] < 1) { err = "input dimensions must be positive"; return MK_ERR_INVALID_ARG; }
  }
  for (int j = 0; j < (int)m.ops.size(); ++j) {
    Op& op = m.ops[j];
    const mk_op_desc& d = op.d;
    const std::string at = "op " + std::to_string(j) + ": ";
    op.n_in = n_inputs_of(d);
    op.out_id = n_in + j;
    for (int k = 0; k < 3; ++k) {
      int id = d.in[k];
      if (k >= op.n_in) { op.in_id[k] = MK_NONE; continue; }
      if (id == MK_PREV) id = (j == 0) ? 0 : n_in + j - 1;
      if (id < 0 || id >= op.out_id) { err = at + "reads a value that is not defined before it"; return MK_ERR_INVALID_ARG; }
      op.in_id[k] = id;
    }
    const mk_tensor_spec x = m.values[op.in_id[0]].spec;
    const int64_t last = x.shape[x.rank - 1];
    mk_tensor_spec y = x;
    y.dtype = dtype;
    // an fp32 value inside a bf16 module (an fp32 residual stream) may only feed a residual add or a row norm
    const bool takes_f32 = d.kind == MK_OP_RESIDUAL_ADD || d.kind == MK_OP_RMSNORM || d.kind == MK_OP_LAYERNORM;
    for (int k = 0; k < op.n_in && d.kind != MK_OP_LINEAR_FP8; ++k) {
      const int32_t vd = m.values[op.in_id[k]].spec.dtype;
      if (vd == MK_FP8_E4M3) { err = at + "an fp8 value may only feed LINEAR_FP8"; return MK_ERR_SHAPE_MISMATCH; }
      if (vd != dtype && !takes_f32) { err = at + "this operator does not take an fp32 residual-stream value"; return MK_ERR_SHAPE_MISMATCH; }
    }
    switch (d.kind) {
      case MK_OP_LINEAR_FP8: {
        const mk_tensor_spec& sx = m.values[op.in_id[1]].spec;
        if (x.rank != 2 || x.dtype != MK_FP8_E4M3) { err = at + "LINEAR_FP8 takes a rank-2 MK_FP8_E4M3 input"; return MK_ERR_SHAPE_MISMATCH; }
        if (x.shape[1] % 128) { err = at + "LINEAR_FP8 needs K to be a multiple of the 128-element scale block"; return MK_ERR_SHAPE_MISMATCH; }
        if (sx.rank != 2 || sx.dtype != MK_F32 || sx.shape[0] != x.shape[0] || sx.shape[1] != x.shape[1] / 128) { err = at + "LINEAR_FP8 scales must be MK_F32 [M, K / 128]"; return MK_ERR_SHAPE_MISMATCH; }
        if (d.i[0] < 1) { err = at + "LINEAR_FP8 needs i[0] = N >= 1"; return MK_ERR_INVALID_ARG; }
        if (d.i[1] != MK_LAYOUT_ROW_MAJOR && d.i[1] != MK_LAYOUT_TRANSPOSED) { err = at + "LINEAR_FP8 i[1] must be an mk_layout"; return MK_ERR_INVALID_ARG; }
        y = make_spec(dtype, {x.shape[0], d.i[0]});
        break;
      }
      case MK_OP_LINEAR: {
        // any rank >= 2: the contraction runs over the last dimension, the leading ones are rows (on an NHWC tensor
        // this is the 1 x 1 convolution)
        if (x.rank < 2) { err = at + "LINEAR takes an input of rank 2 or more"; return MK_ERR_SHAPE_MISMATCH; }
        if (d.i[0] < 1) { err = at + "LINEAR needs i[0] = N >= 1"; return MK_ERR_INVALID_ARG; }
        if (d.i[1] != MK_LAYOUT_ROW_MAJOR && d.i[1] != MK_LAYOUT_TRANSPOSED) { err = at + "LINEAR i[1] must be an mk_layout"; return MK_ERR_INVALID_ARG; }
        y = x;
        y.dtype = dtype;
        y.shape[x.rank - 1] = d.i[0];
        break;
      }
      case MK_OP_CONV2D_3X3: {
        if (x.rank != 4) { err = at + "CONV2D_3X3 takes an NHWC rank-4 input"; return MK_ERR_SHAPE_MISMATCH; }
        if (d.i[0] < 1) { err = at + "CONV2D_3X3 needs i[0] = C_out >= 1"; return MK_ERR_INVALID_ARG; }
        y = make_spec(dtype, {x.shape[0], x.shape[1], x.shape[2], d.i[0]});
        break;
      }
      case MK_OP_BIAS_ADD:
      case MK_OP_RELU:
      case MK_OP_GELU_TANH:
      case MK_OP_GELU_ERF:
      case MK_OP_SILU:
      case MK_OP_SCALE:
        break;
      case MK_OP_CLAMP:
        if (!(d.f[0] <= d.f[1])) { err = at + "CLAMP needs f[0] <= f[1]"; return MK_ERR_INVALID_ARG; }
        break;
      case MK_OP_RESIDUAL_ADD:
        if (!same_shape(x, m.values[op.in_id[1]].spec)) { err = at + "RESIDUAL_ADD operands differ in shape"; return MK_ERR_SHAPE_MISMATCH; }
        if (d.i[0] != 0 && d.i[0] != 1) { err = at + "RESIDUAL_ADD i[0] must be 0 (module dtype) or 1 (fp32 store)"; return MK_ERR_INVALID_ARG; }
        if (d.i[0] == 1) y.dtype = MK_F32;
        break;
      case MK_OP_SWIGLU:
        if (last % 2) { err = at + "SWIGLU needs an even last dimension"; return MK_ERR_SHAPE_MISMATCH; }
        y.shape[y.rank - 1] = last / 2;
        break;
      case MK_OP_LAYERNORM:
      case MK_OP_RMSNORM:
        if (!(d.f[0] >= 0.0)) { err = at + "eps must be >= 0"; return MK_ERR_INVALID_ARG; }
        break;
      case MK_OP_SOFTMAX:
        break;
      case MK_OP_GROUPNORM:
        if (x.rank != 4) { err = at + "GROUPNORM takes an NHWC rank-4 input"; return MK_ERR_SHAPE_MISMATCH; }
        if (d.i[0] < 1 || last % d.i[0]) { err = at + "GROUPNORM: channels must be divisible by groups"; return MK_ERR_SHAPE_MISMATCH; }
        if (!(d.f[0] >= 0.0)) { err = at + "eps must be >= 0"; return MK_ERR_INVALID_ARG; }
        break;
      case MK_OP_AVGPOOL2D:
      case MK_OP_MAXPOOL2D:
      case MK_OP_LPPOOL2D: {
        const int64_t k = d.i[0], st = d.i[1];
        if (x.rank != 4) { err = at + "pooling takes an NHWC rank-4 input"; return MK_ERR_SHAPE_MISMATCH; }
        if (k < 1 || st < 1) { err = at + "pooling needs i[0] = window >= 1 and i[1] = stride >= 1"; return MK_ERR_INVALID_ARG; }
        if (k > x.shape[1] || k > x.shape[2]) { err = at + "pooling window larger than the image"; return MK_ERR_SHAPE_MISMATCH; }
        if (d.kind == MK_OP_LPPOOL2D && !(d.f[0] >= 1.0)) { err = at + "LPPOOL2D needs f[0] = p >= 1"; return MK_ERR_INVALID_ARG; }
        y = make_spec(dtype, {x.shape[0], (x.shape[1] - k) / st + 1, (x.shape[2] - k) / st + 1, x.shape[3]});
        break;
      }
      case MK_OP_ATTENTION_CAUSAL:
      case MK_OP_ATTENTION: {
        const int64_t H = d.i[0], D = d.i[1];
        if (H < 1 || D < 1) { err = at + "attention needs i[0] = heads, i[1] = head_dim"; return MK_ERR_INVALID_ARG; }
        if (d.i[2] == 0) {
          if (x.rank != 4 || x.shape[1] != H || x.shape[3] != D) { err = at + "q must be [B, H, S, D]"; return MK_ERR_SHAPE_MISMATCH; }
          if (!same_spec(x, m.values[op.in_id[1]].spec) || !same_spec(x, m.values[op.in_id[2]].spec)) { err = at + "q, k, v differ in shape"; return MK_ERR_SHAPE_MISMATCH; }
          y = make_spec(dtype, {x.shape[0] * x.shape[2], H * D});
        } else {
          const int64_t B = d.i[2], S = d.i[3];
          if (B < 1 || S < 1) { err = at + "packed attention needs i[2] = B, i[3] = S"; return MK_ERR_INVALID_ARG; }
          if (x.rank != 2 || x.shape[0] != B * S || x.shape[1] != 3 * H * D) { err = at + "packed qkv must be [B*S, 3*H*D]"; return MK_ERR_SHAPE_MISMATCH; }
          y = make_spec(dtype, {B * S, H * D});
        }
        break;
      }
      default:
        err = at + "unknown operator kind";
        return MK_ERR_INVALID_ARG;
    }
    m.values[op.out_id].spec = y;
    m.values[op.out_id].producer = j;
  }
  // Every operator's result must be read by a later operator, except the last one's, which is the module's output:
  // a value nobody reads would get no buffer, and the kernel that produces it nowhere to write.
  std::vector<char> used(m.values.size(), 0);
  for (const Op& op : m.ops)
    for (int k = 0; k < op.n_in; ++k) used[op.in_id[k]] = 1;
  for (int j = 0; j + 1 < (int)m.ops.size(); ++j)
    if (!used[m.ops[j].out_id]) { err = "op " + std::to_string(j) + ": its result is never read and is not the module's output"; return MK_ERR_INVALID_ARG; }
  return MK_OK;
}

bool Module::escapes(int i, int lo, int hi) const {
  if (i == (int)ops.size() - 1) return true;
  const int v = n_inputs + i;
  for (int j = 0; j < (int)ops.size(); ++j) {
    if (j >= lo && j < hi) continue;
    for (int k = 0; k < ops[j].n_in; ++k)
      if (ops[j].in_id[k] == v) return true;
  }
  return false;
}

void contract_of(const Module& m, int lo, int hi, std::vector<int>& in_ids, std::vector<int>& out_ids) {
  in_ids.clear();
  out_ids.clear();
  for (int j = lo; j < hi; ++j) {
    for (int k = 0; k < m.ops[j].n_in; ++k) {
      const int id = m.ops[j].in_id[k];
      const int prod = m.values[id].producer;
      if (prod >= lo && prod < hi) continue;
      if (std::find(in_ids.begin(), in_ids.end(), id) == in_ids.end()) in_ids.push_back(id);
    }
  }
  for (int j = lo; j < hi; ++j)
    if (m.escapes(j, lo, hi)) out_ids.push_back(m.ops[j].out_id);
}

static std::string kind_name(int32_t k) {
  static const char* names[] = {"?", "LINEAR", "CONV2D_3X3", "BIAS_ADD", "RELU", "GELU_TANH", "SILU", "SCALE", "CLAMP",
                                "RESIDUAL_ADD", "SWIGLU", "LAYERNORM", "RMSNORM", "GROUPNORM", "SOFTMAX", "ATTENTION_CAUSAL", "ATTENTION",
                                "AVGPOOL2D", "MAXPOOL2D", "LPPOOL2D", "LINEAR_FP8", "GELU_ERF"};
  return (k >= 1 && k <= 21) ? names[k] : "?";
}

mk_status default_binding(const Module& m, int lo, int hi, Binding& out, std::string& err) {
  out.pieces.clear();
  out.name.clear();
  out.explicit_bind = false;
  int p = lo;
  while (p < hi) {
    const Impl* best = nullptr;
    int best_end = p;
    for (int end = hi; end > p && !best; --end) {
      for (const Impl& im : registry()) {
        if (im.default_pick && im.match(m, p, end)) { best = &im; best_end = end; break; }
      }
    }
    if (!best) {
      err = "no implementation accepts operator " + std::to_string(p) + " (" + kind_name(m.ops[p].d.kind) + ")";
      return MK_ERR_NO_IMPL;
    }
    Piece pc;
    pc.lo = p; pc.hi = best_end; pc.impl = best;
    out.pieces.push_back(pc);
    if (!out.name.empty()) out.name += "+";
    out.name += best->name;
    p = best_end;
  }
  return MK_OK;
}

mk_status explicit_binding(const Module& m, int lo, int hi, const char* name, Binding& out, std::string& err) {
  for (const Impl& im : registry()) {
    if (std::strcmp(im.name, name) != 0) continue;
    if (!im.match(m, lo, hi)) {
      err = std::string("implementation '") + name + "' does not accept this submodule";
      return MK_ERR_NO_IMPL;
    }
    out.pieces.clear();
    Piece pc;
    pc.lo = lo; pc.hi = hi; pc.impl = &im;
    out.pieces.push_back(pc);
    out.name = name;
    out.explicit_bind = true;
    return MK_OK;
  }
  err = std::string("no implementation is named '") + name + "'";
  return MK_ERR_NO_IMPL;
}

// ---- workspace layout ---------------------------------------------------------------------------
namespace {
constexpr size_t kAlign = 1024;
size_t round_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

struct Block { size_t off, size; int last_use; };

size_t place(std::vector<Block>& live, size_t size, int last_use) {
  size = round_up(std::max<size_t>(size, 1));
  std::sort(live.begin(), live.end(), [](const Block& a, const Block& b) { return a.off < b.off; });
  size_t cur = 0;
  for (const Block& b : live) {
    if (b.off >= cur + size) break;
    cur = std::max(cur, b.off + b.size);
  }
  live.push_back({cur, size, last_use});
  return cur;
}
}  // namespace

mk_status plan_layout(Module& m, std::string& err) {
  (void)err;
  const int n_val = (int)m.values.size();
  m.value_off.assign(n_val, -1);
  m.piece_scratch_off.clear();
  std::vector<const Piece*> pieces;
  for (const Binding& b : m.bind)
    for (const Piece& pc : b.pieces) pieces.push_back(&pc);
  const int np = (int)pieces.size();
  const int final_id = m.ops.back().out_id;
  // last piece reading each value
  std::vector<int> last_use(n_val, -1);
  for (int p = 0; p < np; ++p)
    for (int j = pieces[p]->lo; j < pieces[p]->hi; ++j)
      for (int k = 0; k < m.ops[j].n_in; ++k) last_use[m.ops[j].in_id[k]] = std::max(last_use[m.ops[j].in_id[k]], p);
  std::vector<Block> live;
  size_t top = 0;
  for (int p = 0; p < np; ++p) {
    if (!m.keep_intermediates)
      live.erase(std::remove_if(live.begin(), live.end(), [&](const Block& b) { return b.last_use < p; }), live.end());
    std::vector<int> in_ids, out_ids;
    contract_of(m, pieces[p]->lo, pieces[p]->hi, in_ids, out_ids);
    for (int id : out_ids) {
      if (id == final_id) continue;
      const size_t off = place(live, spec_bytes(m.values[id].spec), m.keep_intermediates ? np : last_use[id]);
      m.value_off[id] = (int64_t)off;
      top = std::max(top, off + round_up(spec_bytes(m.values[id].spec)));
    }
    const size_t sc = pieces[p]->impl->scratch(m, pieces[p]->lo, pieces[p]->hi);
    if (sc) {
      const size_t off = place(live, sc, p);
      m.piece_scratch_off.push_back(off);
      top = std::max(top, off + round_up(sc));
    } else {
      m.piece_scratch_off.push_back(0);
    }
  }
  m.workspace_bytes = top;
  m.layout_valid = true;
  m.plan_valid = false;
  return MK_OK;
}

mk_status build_plan(Module& m, const void* const* in_ptrs, void* const* out_ptrs, void* ws, size_t ws_bytes,
                     std::string& err) {
  if (!m.layout_valid) {
    mk_status st = plan_layout(m, err);
    if (st != MK_OK) return st;
  }
  if (ws_bytes < m.workspace_bytes || (m.workspace_bytes && !ws)) {
    err = "workspace too small: need " + std::to_string(m.workspace_bytes) + " bytes";
    return MK_ERR_WORKSPACE_TOO_SMALL;
  }
  if (((uintptr_t)ws & 255) != 0) { err = "workspace must be 256-byte aligned"; return MK_ERR_INVALID_ARG; }
  bool same = m.plan_valid && m.plan_out == out_ptrs[0] && m.plan_ws == ws && (int)m.plan_in.size() == m.n_inputs;
  for (int k = 0; same && k < m.n_inputs; ++k) same = m.plan_in[k] == in_ptrs[k];
  if (same) return MK_OK;

  for (int j = 0; j < (int)m.ops.size(); ++j) {
    const Op& op = m.ops[j];
    const bool need0 = op.d.kind == MK_OP_LINEAR || op.d.kind == MK_OP_CONV2D_3X3 || op.d.kind == MK_OP_BIAS_ADD || op.d.kind == MK_OP_LINEAR_FP8;
    if (need0 && !op.param[0].set) {
      err = "op " + std::to_string(j) + ": parameter 0 has not been set";
      return MK_ERR_PARAM_MISSING;
    }
    if (op.d.kind == MK_OP_LINEAR_FP8 && !op.param[1].set) {
      err = "op " + std::to_string(j) + ": parameter 1 (the weight scales) has not been set";
      return MK_ERR_PARAM_MISSING;
    }
  }
  Resolved r;
  r.value_ptr.assign(m.values.size(), nullptr);
  for (int k = 0; k < m.n_inputs; ++k) {
    if (!in_ptrs[k] || ((uintptr_t)in_ptrs[k] & 15)) { err = "input pointers must be non-null and 16-byte aligned"; return MK_ERR_INVALID_ARG; }
    r.value_ptr[k] = const_cast<void*>(in_ptrs[k]);
  }
  if (!out_ptrs[0] || ((uintptr_t)out_ptrs[0] & 15)) { err = "output pointer must be non-null and 16-byte aligned"; return MK_ERR_INVALID_ARG; }
  r.value_ptr[m.ops.back().out_id] = out_ptrs[0];
  for (size_t id = 0; id < m.values.size(); ++id)
    if (m.value_off[id] >= 0) r.value_ptr[id] = (char*)ws + m.value_off[id];

  m.launches.clear();
  m.launch_sub.clear();
  int p = 0;
  for (int s = 0; s < m.n_sub(); ++s) {
    for (const Piece& pc : m.bind[s].pieces) {
      r.scratch_bytes = pc.impl->scratch(m, pc.lo, pc.hi);
      r.scratch = r.scratch_bytes ? (char*)ws + m.piece_scratch_off[p] : nullptr;
      const size_t before = m.launches.size();
      mk_status st = pc.impl->emit(m, pc.lo, pc.hi, r, m.launches, err);
      if (st != MK_OK) { m.launches.clear(); m.launch_sub.clear(); m.plan_valid = false; return st; }
      for (size_t q = before; q < m.launches.size(); ++q) m.launch_sub.push_back(s);
      ++p;
    }
  }
  m.plan_in.assign(in_ptrs, in_ptrs + m.n_inputs);
  m.plan_out = out_ptrs[0];
  m.plan_ws = ws;
  m.last_value_ptr = r.value_ptr;
  m.plan_valid = true;
  return MK_OK;
}

mk_status build_epi(const Module& m, int lo, int hi, const Resolved& r, EpiProgram& p, std::string& err) {
  p.n = 0;
  p.dtype = m.dtype == MK_F32 ? DT_F32 : DT_BF16;
  for (int j = lo; j < hi; ++j) {
    const Op& op = m.ops[j];
    if (p.n >= EPI_MAX) { err = "elementwise tail longer than the kernel's program"; return MK_ERR_NO_IMPL; }
    EpiOp e{};
    switch (op.d.kind) {
      case MK_OP_BIAS_ADD:
        if (!op.param[0].set) { err = "op " + std::to_string(j) + ": bias has not been set"; return MK_ERR_PARAM_MISSING; }
        e.kind = EPI_BIAS; e.ptr = op.param[0].ptr; e.ptr_dtype = p.dtype; break;
      case MK_OP_RELU: e.kind = EPI_RELU; break;
      case MK_OP_GELU_TANH: e.kind = EPI_GELU_TANH; break;
      case MK_OP_GELU_ERF: e.kind = EPI_GELU_ERF; break;
      case MK_OP_SILU: e.kind = EPI_SILU; break;
      case MK_OP_SCALE: e.kind = EPI_SCALE; e.a = (float)op.d.f[0]; break;
      case MK_OP_CLAMP: e.kind = EPI_CLAMP; e.a = (float)op.d.f[0]; e.b = (float)op.d.f[1]; break;
      case MK_OP_RESIDUAL_ADD:
        e.kind = EPI_RESIDUAL; e.ptr = r.value_ptr[op.in_id[1]];
        e.ptr_dtype = m.values[op.in_id[1]].spec.dtype == MK_F32 ? DT_F32 : DT_BF16;
        if (!e.ptr) { err = "residual operand is not materialised"; return MK_ERR_CONTRACT_VIOLATION; }
        break;
      default:
        err = "operator is not elementwise";
        return MK_ERR_INVALID_ARG;
    }
    p.op[p.n++] = e;
  }
  return MK_OK;
}

}  // namespace mk
