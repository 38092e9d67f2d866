/*
 * mk.h — C ABI of the composed-subkernel library (sm_100a).
 *
 * The library executes a PyTorch-style module as a programmatic composition of
 * subkernels.  The calls follow the paper's statement of the problem
 * (Methodology; Algorithms 1 and 2):
 *
 *   1. describe the module as an operator sequence            mk_module_create
 *   2. register / edit its decomposition into submodules,     mk_module_set_decomposition,
 *      each with a fixed input/output contract                mk_module_split / _fuse / _total_fuse,
 *                                                             mk_module_get_contract
 *   3. bind one subkernel implementation per submodule,       mk_impl_count / mk_impl_name,
 *      and swap it without touching the neighbours            mk_module_bind
 *   4. run the composed forward                               mk_module_set_param,
 *                                                             mk_module_workspace_size,
 *                                                             mk_module_forward
 *   5. observe: per-subkernel time, boundary tensors;         mk_module_profile,
 *      swap what is slower than an alternative                mk_module_intermediate,
 *                                                             mk_module_swap
 *
 * Conventions
 *   - Every pointer named dev_* / in_ptrs[i] / out_ptrs[i] / workspace is a DEVICE pointer
 *     owned by the caller; the library borrows it and never allocates, frees or copies
 *     device memory.  All other pointers are HOST pointers.
 *   - A module's activations have ONE storage type, MK_F32 or MK_BF16: that of its inputs.  A module that has
 *     an MK_FP8_E4M3 input is a bf16 module; beside its fp8 inputs it may have MK_F32 inputs (the block scales)
 *     and MK_BF16 ones.  fp8 and scale tensors may only feed LINEAR_FP8.
 *   - Tensors are dense, row-major, innermost dimension last.  Device pointers must be
 *     16-byte aligned.
 *   - Every function returns an mk_status (0 = MK_OK, negative = error) and never throws or
 *     aborts.  A failed edit or bind leaves the module exactly as it was (the paper's
 *     Split/Fuse agents return the previous decomposition on failure).
 *   - mk_module_forward is asynchronous on the given stream: no host synchronisation, no
 *     allocation and no host<->device copy.
 *   - There is no CPU fallback.  A submodule with no matching implementation yields
 *     MK_ERR_NO_IMPL; a device that is not sm_100 yields MK_ERR_UNSUPPORTED_ARCH.
 *   - One thread uses a module at a time.  Different modules, and contexts on different
 *     devices, may be used from different threads at once: what the library caches per device
 *     (kernel attributes, the address of its status word) is kept per device, in atomics.
 *   - A context belongs to one CUDA device.  A process may hold contexts on several devices;
 *     every call that launches or synchronises (mk_module_forward / _profile / _swap,
 *     mk_ctx_check) requires the context's device to be the calling thread's current device and
 *     returns MK_ERR_INVALID_ARG otherwise.
 *   - Parameters (weights, biases, norm scales) must not be written on the stream while a
 *     forward that reads them is in flight, and not between two forwards that are meant to
 *     overlap: kernels launched as programmatic dependents may read parameters before the
 *     preceding kernel on the stream has completed.
 */
#ifndef MK_H_
#define MK_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define MK_API __attribute__((visibility("default")))
#else
#define MK_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t mk_status;
enum {
  MK_OK = 0,
  MK_ERR_INVALID_ARG = -1,
  MK_ERR_SHAPE_MISMATCH = -2,
  MK_ERR_NO_IMPL = -3,
  MK_ERR_CONTRACT_VIOLATION = -4,
  MK_ERR_WORKSPACE_TOO_SMALL = -5,
  MK_ERR_UNSUPPORTED_ARCH = -6,
  MK_ERR_CUDA = -7,
  MK_ERR_DEVICE_TIMEOUT = -8,
  MK_ERR_NO_DEVICE = -9,
  MK_ERR_PARAM_MISSING = -10
};

/* MK_FP8_E4M3: 8-bit float, 4 exponent bits (bias 7), 3 mantissa bits, no infinities, 0x7f / 0xff are NaN, largest
 * finite value 448 (the "fn" variant).  Only LINEAR_FP8 reads it. */
typedef enum { MK_F32 = 0, MK_BF16 = 1, MK_FP8_E4M3 = 2 } mk_dtype;

/* Physical layout of a rank-2 tensor.  MK_LAYOUT_TRANSPOSED stores the logical [R, C] matrix
 * as its transpose, i.e. a dense row-major [C, R] array (a linear weight kept [out, in]). */
typedef enum { MK_LAYOUT_ROW_MAJOR = 0, MK_LAYOUT_TRANSPOSED = 1 } mk_layout;

#define MK_MAX_RANK 4
typedef struct mk_tensor_spec {
  int32_t dtype;               /* mk_dtype */
  int32_t rank;                /* 1..MK_MAX_RANK */
  int64_t shape[MK_MAX_RANK];  /* logical shape */
  int32_t layout;              /* mk_layout (rank 2 only; 0 otherwise) */
  int32_t reserved;
} mk_tensor_spec;

/* Operator kinds.  "x" is the operator's first input.
 *   LINEAR          y[..., N] = x[..., K] @ W[K,N]      param 0 = W (logical [K,N]); i[0] = N,
 *                   (rank >= 2; the leading dimensions   i[1] = mk_layout of W's storage
 *                   are rows: on NHWC a 1 x 1 convolution)
 *   CONV2D_3X3      NHWC cross-correlation, stride 1, zero pad 1; param 0 = W [C_out,3,3,C_in];
 *                                                       i[0] = C_out
 *   BIAS_ADD        y = x + b[last dim]                 param 0 = b
 *   RELU, GELU_TANH, GELU_ERF, SILU                     elementwise (GELU_ERF: 0.5 x (1 + erf(x / sqrt 2)), the exact form)
 *   SCALE           y = f[0] * x
 *   CLAMP           y = min(max(x, f[0]), f[1])
 *   RESIDUAL_ADD    y = x + in[1]                       (same shape).  i[0] = 1: the sum is stored as fp32
 *                                                       whatever the module dtype (an fp32 residual
 *                                                       stream); such a value may only feed another
 *                                                       RESIDUAL_ADD (either operand), LAYERNORM or RMSNORM
 *   SWIGLU          x[..., 2F] = [gate | up]; y[..., F] = silu(gate) * up
 *   LAYERNORM       rows over the last dim, biased variance, f[0] = eps inside the root;
 *                                                       param 0 = gamma, param 1 = beta (either may be absent)
 *   RMSNORM         y = x / sqrt(mean(x^2) + f[0]) * gamma;  param 0 = gamma (may be absent)
 *   GROUPNORM       NHWC, i[0] = groups of adjacent channels, f[0] = eps; params as LAYERNORM
 *   SOFTMAX         safe softmax over the last dim
 *   ATTENTION_CAUSAL  softmax(mask_{j<=i}(Q K^T / sqrt(D))) V, diagonal kept.
 *                   i[0] = heads H, i[1] = head_dim D.
 *                   i[2] = 0: three inputs q, k, v, each [B, H, S, D];
 *                   i[2] = B > 0: one input, packed [B*S, 3*H*D] with columns [Q | K | V],
 *                                 each head-major, and i[3] = S.
 *                   Output is the logical [B*S, H*D] matrix (head-major columns).
 *   ATTENTION       the same without the mask: softmax(Q K^T / sqrt(D)) V over every key (the encoder
 *                   attention of the paper's transformer-block example); attributes and layouts as above.
 *   AVGPOOL2D, MAXPOOL2D, LPPOOL2D   NHWC, square window i[0] = k, stride i[1], no padding, output
 *                   [N, (H - k) / stride + 1, (W - k) / stride + 1, C] (whole windows only).  Mean, maximum, and
 *                   the p-norm (sum |x|^p)^(1/p) with p = f[0] >= 1 of each window: the pooling subkernel of the
 *                   paper's MobileNetV1 example and the two variants of its transfer study.
 *   LINEAR_FP8      block-scaled fp8 GEMM, the contraction of the paper's FP8 MoE inference task:
 *                   y[M,N] = sum over K blocks kb of sx[m,kb] * sw[n/128,kb] * sum_{k in block kb} xq[m,k] * wq[k,n]
 *                   with blocks of 128 along K (activations: one scale per row and block; weights: one per
 *                   128 x 128 block).  in[0] = xq [M,K] MK_FP8_E4M3, in[1] = sx [M, K/128] MK_F32;
 *                   param 0 = wq (logical [K,N], MK_FP8_E4M3; i[1] = mk_layout of its storage),
 *                   param 1 = sw [ceil(N/128), K/128] MK_F32; i[0] = N; K must be a multiple of 128.
 *                   The result has the module's activation type (bf16 in a module that has fp8 inputs); the
 *                   products are accumulated in fp32 and every block's partial sum is scaled in fp32.
 * Definitions: the paper's subkernel listings (linear with W stored [K, N]; LayerNorm; online-
 * softmax attention) and its correctness appendix (safe softmax, tril(diagonal=0) mask, fp32
 * accumulation); RMSNorm, GroupNorm, SwiGLU, tanh-GELU and the 3x3 convolution follow the
 * workload list.
 */
typedef enum {
  MK_OP_LINEAR = 1,
  MK_OP_CONV2D_3X3 = 2,
  MK_OP_BIAS_ADD = 3,
  MK_OP_RELU = 4,
  MK_OP_GELU_TANH = 5,
  MK_OP_SILU = 6,
  MK_OP_SCALE = 7,
  MK_OP_CLAMP = 8,
  MK_OP_RESIDUAL_ADD = 9,
  MK_OP_SWIGLU = 10,
  MK_OP_LAYERNORM = 11,
  MK_OP_RMSNORM = 12,
  MK_OP_GROUPNORM = 13,
  MK_OP_SOFTMAX = 14,
  MK_OP_ATTENTION_CAUSAL = 15,
  MK_OP_ATTENTION = 16,
  MK_OP_AVGPOOL2D = 17,
  MK_OP_MAXPOOL2D = 18,
  MK_OP_LPPOOL2D = 19,
  MK_OP_LINEAR_FP8 = 20,
  MK_OP_GELU_ERF = 21
} mk_op_kind;

/* Value numbering: module input k has id k; operator j produces id n_inputs + j.
 * MK_PREV names the previous operator's output (module input 0 for operator 0).
 * The last operator's output is the module's output. */
#define MK_PREV (-1)
#define MK_NONE (-2)

typedef struct mk_op_desc {
  int32_t kind;   /* mk_op_kind */
  int32_t in[3];  /* value ids read; unused entries MK_NONE */
  double f[2];    /* scalar attributes, see the table above */
  int32_t i[4];   /* integer attributes, see the table above */
} mk_op_desc;

typedef struct mk_ctx mk_ctx;
typedef struct mk_module mk_module;

/* ---- context ------------------------------------------------------------------------------
 * (Methodology: the codebase is a set of subkernels K plus one top-level module S; a context is
 * where the library keeps what belongs to neither: the device and the last error.)
 * device >= 0: binds the context to that CUDA device (must be compute capability 10.x, else
 * MK_ERR_UNSUPPORTED_ARCH; MK_ERR_NO_DEVICE if there is none) and makes it the calling thread's
 * current device.  device = -1: a host-only planning context — describing, decomposing, binding
 * and contract queries work, launching returns MK_ERR_NO_DEVICE.  *out is written only on success. */
MK_API mk_status mk_ctx_create(int32_t device, mk_ctx** out);
MK_API void mk_ctx_destroy(mk_ctx* ctx);
MK_API const char* mk_status_str(mk_status s);
/* Text of the last error raised through this context ("" if none).  Valid until the next call. */
MK_API const char* mk_last_error(const mk_ctx* ctx);
/* Synchronises the context's device and reports a bounded-wait expiry inside a kernel
 * (MK_ERR_DEVICE_TIMEOUT) or a CUDA error (MK_ERR_CUDA).  Clears the timeout flag.  (Experiments,
 * "Setup": an evaluation that does not finish within its time limit counts as failed; here a
 * kernel that cannot make progress gives up by itself and says so.) */
MK_API mk_status mk_ctx_check(mk_ctx* ctx);

/* Self-test of the exit every bounded wait takes when it runs out (the one path a correct run never
 * executes).  Launches one small CTA that waits, through the same routine the tensor-core kernels
 * use, on a barrier nobody arrives at, gives up after `limit_cycles` SM cycles (1e3 .. 2e8; about
 * a millisecond at 2e6), records its code in the device status word and returns normally; the next
 * mk_ctx_check then reports MK_ERR_DEVICE_TIMEOUT once and clears the flag.  No copies, no tensor
 * memory, nothing left behind: the device stays usable.  dev_out6: six int64 in device memory
 * (8-byte aligned): [0] / [1] what the wait returned in the thread that gave up and in a second
 * thread released by the abort flag (0 = gave up), [2] / [3] the cycles they spent, [4] / [5] the
 * same for a wait started after the expiry (it must return at once).  Asynchronous on the stream.
 * (Experiments, "Setup": evaluations run under a time limit; a kernel that stalls must end as a
 * reported failure, not as a hung device.) */
MK_API mk_status mk_selftest_bounded_wait(mk_ctx* ctx, int64_t limit_cycles, int64_t* dev_out6,
                                          void* cuda_stream);

/* ---- 1. describe a module as an operator sequence -------------------------------------------
 * (Methodology, LLMDecompose: the input is a PyTorch module; the top-level module delegates all
 * mathematical computation to the submodules.  Here the module is its operator sequence.)
 * ops[n_ops] and inputs[n_inputs] are copied.  Shapes of all values are inferred here;
 * an inconsistent sequence gives MK_ERR_SHAPE_MISMATCH / MK_ERR_INVALID_ARG.  The initial
 * decomposition is one submodule per operator, each bound to the composer's default choice. */
MK_API mk_status mk_module_create(mk_ctx* ctx, const mk_op_desc* ops, int32_t n_ops,
                           const mk_tensor_spec* inputs, int32_t n_inputs, mk_module** out);
MK_API void mk_module_destroy(mk_module* m);
MK_API mk_status mk_module_n_ops(const mk_module* m, int32_t* n);
/* Spec of value `value_id` (inputs first, then one per operator). */
MK_API mk_status mk_module_value_spec(const mk_module* m, int32_t value_id, mk_tensor_spec* out);

/* ---- 2. the decomposition: a partition of [0, n_ops) into contiguous submodules -----------
 * (Methodology, LLMDecompose and its programmatic checks: the subproblems must fully and
 * exclusively cover what the top-level module needs.)
 * first_op_of_sub[n_sub] must start at 0 and increase strictly; every operator then lies in
 * exactly one submodule ("fully and exclusively cover").  Every new submodule is bound to
 * the composer's default choice; MK_ERR_NO_IMPL if some submodule cannot be implemented. */
MK_API mk_status mk_module_set_decomposition(mk_module* m, const int32_t* first_op_of_sub, int32_t n_sub);
MK_API mk_status mk_module_n_sub(const mk_module* m, int32_t* n);
/* Writes n_sub entries into first_op_of_sub (capacity checked against *n_sub on entry). */
MK_API mk_status mk_module_get_decomposition(const mk_module* m, int32_t* first_op_of_sub, int32_t* n_sub);
/* Split submodule `sub` into exactly two at operator `at_op` (first_op < at_op <= last op).
 * (Methodology, LLMSplit: a subproblem is split into exactly 2; Algorithm 2 applies it to failing
 * subkernels.  On failure the previous decomposition is kept.) */
MK_API mk_status mk_module_split(mk_module* m, int32_t sub, int32_t at_op);
/* Fuse `count` >= 2 adjacent submodules starting at `first_sub` into one.
 * (Methodology, LLMFuse: any number of subproblems are fused into a larger one; Algorithm 2's
 * fusion branch.  On failure the previous decomposition is kept.) */
MK_API mk_status mk_module_fuse(mk_module* m, int32_t first_sub, int32_t count);
/* Collapse to the monolithic problem: one submodule holding every operator.
 * (Algorithm 2, TotalFuse: taken when the local and the global correctness checks disagree.) */
MK_API mk_status mk_module_total_fuse(mk_module* m);
/* The submodule's I/O contract: value ids and specs it reads from outside and those it
 * produces for later submodules or as the module output.  (Appendix "Prompts", subproblem
 * decomposition: every subproblem states its input and output tensors with shapes and dtypes and
 * its verification criteria; LLMDecompose's forward-shape-coverage check.)  On entry *n_in / *n_out hold the
 * capacities of the arrays (ids and specs may each be NULL); on return the counts. */
MK_API mk_status mk_module_get_contract(const mk_module* m, int32_t sub, int32_t* in_ids,
                                 mk_tensor_spec* in_specs, int32_t* n_in, int32_t* out_ids,
                                 mk_tensor_spec* out_specs, int32_t* n_out);

/* ---- 3. implementations: list, bind, swap ----------------------------------------------------
 * (Introduction and Methodology: each subkernel solves one explicitly defined subproblem and can
 * be replaced by an alternative implementation without touching the rest; the composer's fusion
 * rules are those of the appendix "Prompts": GEMM + elementwise tail, elementwise chains, bias
 * after matmul and the residual add fuse, a reduction over a whole row or group blocks fusion.)
 * mk_impl_count/_name enumerate the registered single-kernel-family implementations whose
 * legality predicate accepts submodule `sub` as a whole.  mk_module_bind(sub, name) binds one
 * of them (MK_ERR_NO_IMPL if it does not accept the submodule; the old binding stays).
 * name = NULL asks the composer: it takes the widest legal fused implementation, and if no
 * single one covers the submodule it covers it with a chain of them (longest match first),
 * keeping the chain's intermediates in the workspace.  mk_module_bound_impl returns the bound
 * name (a chain reads "a+b+c"); the string lives until the next edit or bind. */
MK_API mk_status mk_impl_count(const mk_module* m, int32_t sub, int32_t* n);
MK_API mk_status mk_impl_name(const mk_module* m, int32_t sub, int32_t i, const char** name);
MK_API mk_status mk_module_bind(mk_module* m, int32_t sub, const char* impl_name);
MK_API mk_status mk_module_bound_impl(const mk_module* m, int32_t sub, const char** name);

/* ---- 4. parameters, workspace, run --------------------------------------------------------------
 * (Appendix "Example Solution", top-level module: it owns the parameters, hands each subkernel
 * its tensors and chains the calls; appendix "Prompts", memory and dataflow: intermediates are
 * materialised in global memory only at subproblem boundaries.)
 * set_param: operator `op`, slot as listed per kind; dev_ptr is borrowed and must stay valid;
 * spec must equal what the operator expects (MK_ERR_SHAPE_MISMATCH otherwise). */
MK_API mk_status mk_module_set_param(mk_module* m, int32_t op, int32_t slot, const void* dev_ptr,
                              const mk_tensor_spec* spec);
/* keep != 0: every submodule-boundary tensor keeps its own workspace range so that
 * mk_module_intermediate can read it after a forward; keep = 0 (default) lets boundary
 * tensors whose lifetimes do not overlap share memory. */
MK_API mk_status mk_module_keep_intermediates(mk_module* m, int32_t keep);
/* Bytes of workspace the current decomposition and bindings need (boundary tensors plus
 * kernel scratch). */
MK_API mk_status mk_module_workspace_size(mk_module* m, size_t* bytes);
/* Kernel launches one forward issues under the current decomposition and bindings. */
MK_API mk_status mk_module_launch_count(mk_module* m, int32_t* n);
/* Composed forward (Algorithm 1, Evaluate: the end-to-end kernel is the top-level module running
 * its subkernels in order).  in_ptrs[n_inputs], out_ptrs[1]: device tensors matching the specs.
 * workspace: device memory of at least workspace_size bytes, 256-byte aligned, may be NULL
 * when the size is 0.  cuda_stream: a cudaStream_t (NULL = the default stream).
 * Errors: MK_ERR_PARAM_MISSING, MK_ERR_WORKSPACE_TOO_SMALL, MK_ERR_NO_DEVICE, MK_ERR_CUDA,
 * MK_ERR_INVALID_ARG (the context's device is not the current device). */
MK_API mk_status mk_module_forward(mk_module* m, const void* const* in_ptrs, void* const* out_ptrs,
                            void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The same for submodules [first_sub, first_sub + count) alone: their launches of the cached plan, nothing else.
 * What they read from earlier submodules must already be in the workspace (run a whole forward first, with
 * mk_module_keep_intermediates on so that no later submodule has reused those ranges).  This is how one subkernel
 * is evaluated or timed in isolation on the inputs the composition gives it (Methodology, LLMEvolveKernel: every
 * subkernel is verified and profiled on its own subproblem; Algorithm 2: local checks beside the global one).
 * Errors: as mk_module_forward; MK_ERR_INVALID_ARG for a range outside the decomposition. */
MK_API mk_status mk_module_forward_sub(mk_module* m, const void* const* in_ptrs, void* const* out_ptrs,
                                void* workspace, size_t workspace_bytes, void* cuda_stream,
                                int32_t first_sub, int32_t count);

/* ---- 5. observability ---------------------------------------------------------------------------
 * profile: runs `iters` forwards with a CUDA event pair around every submodule, synchronises,
 * and writes the mean milliseconds per submodule into ms_per_sub[n_sub].  (Methodology,
 * AllocateLLMBudget: the budget follows each subkernel's runtime observed during the last
 * end-to-end evaluation; Swap reads the same per-subkernel figure.) */
MK_API mk_status mk_module_profile(mk_module* m, const void* const* in_ptrs, void* const* out_ptrs,
                            void* workspace, size_t workspace_bytes, void* cuda_stream,
                            int32_t iters, float* ms_per_sub);
/* Swap (paper, Algorithm 1's Swap step and the "MKEvolve (Swap)" variant: a subkernel that is slower
 * than an available alternative by more than a threshold is replaced, the rest of the composition is
 * left alone).  For every submodule in turn: time every registered implementation that accepts the whole
 * submodule (mk_module_profile's event pairs, on the caller's buffers: the tensors are overwritten
 * with valid results of whichever binding ran last) and, if the bound one runs at less than `tau`
 * (paper: 0.9; 0 < tau <= 1) of the fastest one's speed, rebind the submodule to the fastest; otherwise
 * the original binding - a composer-chosen chain included - is restored.  Modules with fewer than two
 * submodules are left alone, as in the paper.  An alternative that needs more workspace than
 * workspace_bytes, or whose first run takes more than four times the best time so far, is skipped.
 * n_swapped (optional): number of submodules rebound.  ms_before_after (optional): float
 * [n_sub][2], each submodule's time with its old and with its final binding.  Synchronises the stream.
 * Errors: as mk_module_profile; the bindings are valid (old or new) on every return. */
MK_API mk_status mk_module_swap(mk_module* m, const void* const* in_ptrs, void* const* out_ptrs, void* workspace,
                         size_t workspace_bytes, void* cuda_stream, int32_t iters, double tau,
                         int32_t* n_swapped, float* ms_before_after);
/* Device pointer and spec of the tensor produced by value `value_id` at a submodule boundary
 * during the last forward (requires keep_intermediates; MK_ERR_INVALID_ARG if the value is
 * internal to a submodule or no forward has run).  (Algorithm 2: local correctness checks, one
 * per subkernel, beside the global one; appendix on correctness checking: every intermediate
 * tensor is compared with its own calibrated tolerance.) */
MK_API mk_status mk_module_intermediate(const mk_module* m, int32_t value_id, const void** dev_ptr,
                                 mk_tensor_spec* spec);

/* ---- allocation-free GroupNorm ----------------------------------------------------------------
 * (The paper has no counterpart: this entry point exists for callers, not for the method.)
 * NHWC GroupNorm, the same two kernels the composed path launches, for callers that cannot
 * allocate device memory where they call the library and so cannot provide a workspace: code
 * inside a memory-planned region of a framework, a plugin that is handed only its input and
 * output buffers, a latency-critical loop that must not hit cudaMalloc's implicit
 * synchronisation.  The partial sums live in a 1 MiB array inside the library image, resident
 * on every GPU that loads the library until the process exits.
 *   dev_x, dev_y       [n, h, w, c] tensors of `dtype` (mk_dtype), 16-byte aligned, caller-owned
 *   dev_gamma/dev_beta [c] or NULL
 *   groups             must divide c; eps >= 0, inside the square root
 *   n <= 65535 images; h * w < 2^31 pixels per image
 * The call allocates nothing, is asynchronous on `cuda_stream` and does not synchronise.
 * The first call on each device looks up the array's device address (a host-side query, made
 * with that device current): make that first call before starting any stream capture.
 * All calls share the one array and it keeps the last call's contents; the kernels overwrite
 * every slot they later read, so nothing needs clearing, but two calls whose kernels overlap on
 * the GPU (different streams, no dependency) race on it — order them.  Host threads may call
 * concurrently as far as the host side goes (the per-device set-up is kept in atomics); the
 * shared array still requires their kernels to be ordered on the GPU.
 * Errors: MK_ERR_WORKSPACE_TOO_SMALL if n * chunks * groups * 8 bytes exceeds 1 MiB (chunks <= 64
 * pixel chunks per image; e.g. n = 32, groups = 32 needs 80 KiB), MK_ERR_SHAPE_MISMATCH (a
 * size outside the limits above, groups not dividing c), MK_ERR_INVALID_ARG (a NULL or unaligned
 * tensor pointer, an unknown dtype, eps < 0 or NaN), MK_ERR_NO_DEVICE, MK_ERR_CUDA. */
MK_API mk_status mk_groupnorm_nhwc_noalloc(int32_t dtype, const void* dev_x, void* dev_y,
                                           const void* dev_gamma, const void* dev_beta, int64_t n,
                                           int64_t h, int64_t w, int64_t c, int32_t groups,
                                           double eps, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* MK_H_ */
