// Internal structures of the composer: module description, decomposition, implementation
// registry and launch plan.  Host code; the kernels see only kernels.h.
#pragma once

#include <cuda_runtime.h>

#include <functional>
#include <string>
#include <vector>

#include "../../include/mk.h"
#include "kernels.h"

namespace mk {

struct Param {
  const void* ptr = nullptr;
  mk_tensor_spec spec{};
  bool set = false;
};

struct Op {
  mk_op_desc d{};
  int n_in = 0;
  int in_id[3] = {MK_NONE, MK_NONE, MK_NONE};  // resolved value ids
  int out_id = -1;
  Param param[2];
};

struct Value {
  mk_tensor_spec spec{};
  int producer = -1;  // op index, -1 for module inputs
};

int64_t numel(const mk_tensor_spec& s);
size_t dtype_size(int32_t dtype);
size_t spec_bytes(const mk_tensor_spec& s);
bool same_spec(const mk_tensor_spec& a, const mk_tensor_spec& b);
bool is_eltwise(int32_t kind);  // pure elementwise kinds an epilogue program can hold

struct Module;

// Where every value lives for one forward call.
struct Resolved {
  std::vector<void*> value_ptr;  // per value id (nullptr: internal to a fused kernel)
  char* scratch = nullptr;       // scratch range of the piece being emitted
  size_t scratch_bytes = 0;
};

using Launch = std::function<cudaError_t(cudaStream_t)>;

// One registered implementation: a kernel family with a legality predicate.
struct Impl {
  const char* name;
  // Does this implementation accept operators [lo, hi) of m as one fused piece?
  bool (*match)(const Module& m, int lo, int hi);
  // Scratch bytes (global memory beyond inputs/outputs) the piece needs.
  size_t (*scratch)(const Module& m, int lo, int hi);
  // Append the piece's kernel launches.
  mk_status (*emit)(const Module& m, int lo, int hi, const Resolved& r, std::vector<Launch>& out,
                    std::string& err);
  // false: legal and bindable by name (and a candidate for Swap, which decides by measured time), but the
  // composer's default cover does not pick it - for variants that are not (yet) faster than what they replace
  bool default_pick = true;
};
const std::vector<Impl>& registry();

struct Piece {
  int lo = 0, hi = 0;
  const Impl* impl = nullptr;
};

struct Binding {
  std::vector<Piece> pieces;  // one for a single implementation, several for a chain
  std::string name;
  bool explicit_bind = false;
};

struct Ctx {
  int device = -1;
  int sm_count = 0;
  mutable std::string err;
  unsigned int* dev_status = nullptr;  // unused unless a kernel reports a bounded-wait expiry
};

struct Module {
  Ctx* ctx = nullptr;
  int n_inputs = 0;
  int32_t dtype = MK_BF16;       // storage type of the activations (MK_F32 or MK_BF16), set by infer_shapes
  std::vector<Op> ops;
  std::vector<Value> values;
  std::vector<int> cuts;         // first op of each submodule
  std::vector<Binding> bind;     // one per submodule
  bool keep_intermediates = false;

  // ---- plan (rebuilt when the decomposition, bindings, params or pointers change)
  bool layout_valid = false;
  std::vector<int64_t> value_off;  // workspace offset per value, -1 if not in the workspace
  std::vector<size_t> piece_scratch_off;
  size_t workspace_bytes = 0;
  bool plan_valid = false;
  std::vector<const void*> plan_in;
  void* plan_out = nullptr;
  void* plan_ws = nullptr;
  std::vector<Launch> launches;
  std::vector<int> launch_sub;   // submodule of each launch
  std::vector<void*> last_value_ptr;

  int n_sub() const { return (int)cuts.size(); }
  int sub_lo(int s) const { return cuts[s]; }
  int sub_hi(int s) const { return s + 1 < (int)cuts.size() ? cuts[s + 1] : (int)ops.size(); }
  const mk_tensor_spec& vspec(int id) const { return values[id].spec; }
  // Is the value produced by op `i` read by any op outside [lo, hi), or the module output?
  bool escapes(int i, int lo, int hi) const;
};

// composer.cpp
mk_status infer_shapes(Module& m, std::string& err);
mk_status default_binding(const Module& m, int lo, int hi, Binding& out, std::string& err);
mk_status explicit_binding(const Module& m, int lo, int hi, const char* name, Binding& out,
                           std::string& err);
void contract_of(const Module& m, int lo, int hi, std::vector<int>& in_ids, std::vector<int>& out_ids);
mk_status plan_layout(Module& m, std::string& err);
mk_status build_plan(Module& m, const void* const* in_ptrs, void* const* out_ptrs, void* ws,
                     size_t ws_bytes, std::string& err);

// Builds the elementwise program for ops [lo, hi) (all must satisfy is_eltwise); pointers come
// from the parameters (bias) and the resolved values (residual).
mk_status build_epi(const Module& m, int lo, int hi, const Resolved& r, EpiProgram& p,
                    std::string& err);

}  // namespace mk
