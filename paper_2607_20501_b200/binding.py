"""ctypes binding of libmk.so: the same names as include/mk.h, argument marshalling only.

Every step of the composed forward runs in the library's CUDA kernels.  There is no
Python or CPU fallback: if the shared library is missing, importing this module
raises.  PyTorch appears only as the owner of device memory and streams.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmk.so")
if not os.path.exists(LIB_PATH):
    raise RuntimeError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2607_20501_b200.build` "
        "(there is no fallback path)")
lib = C.CDLL(LIB_PATH)

# ---- constants (mirror include/mk.h) --------------------------------------------------------------
MK_OK = 0
STATUS = {
    0: "MK_OK", -1: "MK_ERR_INVALID_ARG", -2: "MK_ERR_SHAPE_MISMATCH", -3: "MK_ERR_NO_IMPL",
    -4: "MK_ERR_CONTRACT_VIOLATION", -5: "MK_ERR_WORKSPACE_TOO_SMALL", -6: "MK_ERR_UNSUPPORTED_ARCH",
    -7: "MK_ERR_CUDA", -8: "MK_ERR_DEVICE_TIMEOUT", -9: "MK_ERR_NO_DEVICE", -10: "MK_ERR_PARAM_MISSING",
}
for _code, _name in STATUS.items():
    globals()[_name] = _code
MK_F32, MK_BF16, MK_FP8_E4M3 = 0, 1, 2
MK_LAYOUT_ROW_MAJOR, MK_LAYOUT_TRANSPOSED = 0, 1
MK_MAX_RANK = 4
MK_PREV, MK_NONE = -1, -2
OP = {
    "linear": 1, "conv2d_3x3": 2, "bias_add": 3, "relu": 4, "gelu_tanh": 5, "gelu_erf": 21, "silu": 6, "scale": 7,
    "clamp": 8, "residual_add": 9, "swiglu": 10, "layernorm": 11, "rmsnorm": 12, "groupnorm": 13,
    "softmax": 14, "attention_causal": 15, "attention": 16, "avgpool": 17, "maxpool": 18, "lppool": 19,
    "linear_fp8": 20,
}
DTYPE = {"f32": MK_F32, "bf16": MK_BF16, "fp8": MK_FP8_E4M3}


class mk_tensor_spec(C.Structure):
    _fields_ = [("dtype", C.c_int32), ("rank", C.c_int32), ("shape", C.c_int64 * MK_MAX_RANK),
                ("layout", C.c_int32), ("reserved", C.c_int32)]


class mk_op_desc(C.Structure):
    _fields_ = [("kind", C.c_int32), ("in_", C.c_int32 * 3), ("f", C.c_double * 2), ("i", C.c_int32 * 4)]


_P = C.c_void_p
_PP = C.POINTER(C.c_void_p)
_I32P = C.POINTER(C.c_int32)
_SPECP = C.POINTER(mk_tensor_spec)


def _sig(name, res, *args):
    fn = getattr(lib, name)
    fn.restype = res
    fn.argtypes = list(args)
    globals()[name] = fn
    return fn


_sig("mk_ctx_create", C.c_int32, C.c_int32, _PP)
_sig("mk_ctx_destroy", None, _P)
_sig("mk_status_str", C.c_char_p, C.c_int32)
_sig("mk_last_error", C.c_char_p, _P)
_sig("mk_ctx_check", C.c_int32, _P)
_sig("mk_selftest_bounded_wait", C.c_int32, _P, C.c_int64, _P, _P)
_sig("mk_module_create", C.c_int32, _P, C.POINTER(mk_op_desc), C.c_int32, _SPECP, C.c_int32, _PP)
_sig("mk_module_destroy", None, _P)
_sig("mk_module_n_ops", C.c_int32, _P, _I32P)
_sig("mk_module_value_spec", C.c_int32, _P, C.c_int32, _SPECP)
_sig("mk_module_set_decomposition", C.c_int32, _P, _I32P, C.c_int32)
_sig("mk_module_n_sub", C.c_int32, _P, _I32P)
_sig("mk_module_get_decomposition", C.c_int32, _P, _I32P, _I32P)
_sig("mk_module_split", C.c_int32, _P, C.c_int32, C.c_int32)
_sig("mk_module_fuse", C.c_int32, _P, C.c_int32, C.c_int32)
_sig("mk_module_total_fuse", C.c_int32, _P)
_sig("mk_module_get_contract", C.c_int32, _P, C.c_int32, _I32P, _SPECP, _I32P, _I32P, _SPECP, _I32P)
_sig("mk_impl_count", C.c_int32, _P, C.c_int32, _I32P)
_sig("mk_impl_name", C.c_int32, _P, C.c_int32, C.c_int32, C.POINTER(C.c_char_p))
_sig("mk_module_bind", C.c_int32, _P, C.c_int32, C.c_char_p)
_sig("mk_module_bound_impl", C.c_int32, _P, C.c_int32, C.POINTER(C.c_char_p))
_sig("mk_module_set_param", C.c_int32, _P, C.c_int32, C.c_int32, _P, _SPECP)
_sig("mk_module_keep_intermediates", C.c_int32, _P, C.c_int32)
_sig("mk_module_workspace_size", C.c_int32, _P, C.POINTER(C.c_size_t))
_sig("mk_module_launch_count", C.c_int32, _P, _I32P)
_sig("mk_module_forward", C.c_int32, _P, _PP, _PP, _P, C.c_size_t, _P)
_sig("mk_module_forward_sub", C.c_int32, _P, _PP, _PP, _P, C.c_size_t, _P, C.c_int32, C.c_int32)
_sig("mk_module_profile", C.c_int32, _P, _PP, _PP, _P, C.c_size_t, _P, C.c_int32, C.POINTER(C.c_float))
_sig("mk_module_swap", C.c_int32, _P, _PP, _PP, _P, C.c_size_t, _P, C.c_int32, C.c_double, C.POINTER(C.c_int32), C.POINTER(C.c_float))
_sig("mk_module_intermediate", C.c_int32, _P, C.c_int32, _PP, _SPECP)
_sig("mk_groupnorm_nhwc_noalloc", C.c_int32, C.c_int32, _P, _P, _P, _P, C.c_int64, C.c_int64, C.c_int64,
     C.c_int64, C.c_int32, C.c_double, _P)

EXPORTS = [n for n in dir() if n.startswith("mk_") and callable(globals()[n]) and n not in
           ("mk_tensor_spec", "mk_op_desc")]


class MkError(RuntimeError):
    def __init__(self, status, text=""):
        self.status = status
        super().__init__(f"{STATUS.get(status, status)}: {text}")


def make_spec(dtype, shape, layout=MK_LAYOUT_ROW_MAJOR) -> mk_tensor_spec:
    s = mk_tensor_spec()
    s.dtype = DTYPE[dtype] if isinstance(dtype, str) else int(dtype)
    s.rank = len(shape)
    for i, v in enumerate(shape):
        s.shape[i] = int(v)
    s.layout = layout
    return s


def spec_tuple(s: mk_tensor_spec):
    return (s.dtype, tuple(s.shape[i] for i in range(s.rank)), s.layout)


class Context:
    """mk_ctx owner.  device=-1 gives the host-only planning context."""

    def __init__(self, device=0):
        h = C.c_void_p()
        st = mk_ctx_create(device, C.byref(h))
        if st != MK_OK:
            raise MkError(st, "mk_ctx_create")
        self.h = h
        self.device = device

    def last_error(self):
        return mk_last_error(self.h).decode()

    def check(self):
        st = mk_ctx_check(self.h)
        if st != MK_OK:
            raise MkError(st, self.last_error())

    def __del__(self):
        try:
            if getattr(self, "h", None):
                mk_ctx_destroy(self.h)
                self.h = None
        except Exception:       # interpreter shutdown: the module globals may already be gone
            pass


def _ptr(t):
    """Device (or host) address of a torch tensor / raw int."""
    return int(t) if isinstance(t, int) else int(t.data_ptr())


class Module:
    """mk_module owner built from a declarative operator list.

    ops: list of dicts {"kind", "out", "in": [names], "params": {...}, "attrs": {...}};
    inputs: ordered dict name -> (dtype, shape).  Names are resolved to value ids here;
    weight_layout picks how LINEAR weights are stored (MK_LAYOUT_*).
    """

    PARAM_SLOTS = {"linear": ("w",), "linear_fp8": ("w", "sw"), "conv2d_3x3": ("w",), "bias_add": ("b",), "rmsnorm": ("gamma",),
                   "layernorm": ("gamma", "beta"), "groupnorm": ("gamma", "beta")}

    def __init__(self, ctx: Context, ops, inputs, weight_layout=MK_LAYOUT_TRANSPOSED):
        self.ctx = ctx
        self.ops = ops
        self.input_names = list(inputs)
        self.weight_layout = weight_layout
        ids = {n: k for k, n in enumerate(self.input_names)}
        n_in = len(ids)
        descs = (mk_op_desc * len(ops))()
        shapes = {n: tuple(inputs[n][1]) for n in inputs}
        for j, op in enumerate(ops):
            d = descs[j]
            d.kind = OP[op["kind"]]
            for k in range(3):
                d.in_[k] = ids[op["in"][k]] if k < len(op["in"]) else MK_NONE
            a = op.get("attrs", {})
            kind = op["kind"]
            if kind == "scale":
                d.f[0] = a["s"]
            elif kind == "clamp":
                d.f[0], d.f[1] = a["lo"], a["hi"]
            elif kind in ("layernorm", "rmsnorm"):
                d.f[0] = a["eps"]
            elif kind == "groupnorm":
                d.f[0] = a["eps"]
                d.i[0] = a["groups"]
            elif kind == "residual_add":
                d.i[0] = 1 if a.get("store") == "f32" else 0
            elif kind in ("linear", "linear_fp8"):
                d.i[0] = int(a["n"])
                d.i[1] = weight_layout
            elif kind == "conv2d_3x3":
                d.i[0] = int(a["c_out"])
            elif kind in ("avgpool", "maxpool", "lppool"):
                d.i[0], d.i[1] = int(a["k"]), int(a["stride"])
                if kind == "lppool":
                    d.f[0] = float(a["p"])
            elif kind in ("attention_causal", "attention"):
                d.i[0], d.i[1] = a["heads"], a["head_dim"]
                if a["layout"] == "packed_qkv":
                    d.i[2], d.i[3] = a["batch"], a["seq"]
            ids[op["out"]] = n_in + j
        self.value_id = ids
        specs = (mk_tensor_spec * n_in)()
        for k, n in enumerate(self.input_names):
            specs[k] = make_spec(inputs[n][0], inputs[n][1])
        h = C.c_void_p()
        st = mk_module_create(ctx.h, descs, len(ops), specs, n_in, C.byref(h))
        if st != MK_OK:
            raise MkError(st, ctx.last_error())
        self.h = h
        self._keep = []          # tensors whose pointers the library borrows
        self._ws = None

    # -- helpers -------------------------------------------------------------------------------------
    def _ck(self, st):
        if st != MK_OK:
            raise MkError(st, self.ctx.last_error())

    def __del__(self):
        try:
            if getattr(self, "h", None):
                mk_module_destroy(self.h)
                self.h = None
        except Exception:       # interpreter shutdown: the module globals may already be gone
            pass

    # -- description ---------------------------------------------------------------------------------
    def n_ops(self):
        n = C.c_int32()
        self._ck(mk_module_n_ops(self.h, C.byref(n)))
        return n.value

    def value_spec(self, value):
        vid = self.value_id[value] if isinstance(value, str) else value
        s = mk_tensor_spec()
        self._ck(mk_module_value_spec(self.h, vid, C.byref(s)))
        return spec_tuple(s)

    # -- decomposition -------------------------------------------------------------------------------
    def set_decomposition(self, cuts):
        arr = (C.c_int32 * len(cuts))(*cuts)
        self._ck(mk_module_set_decomposition(self.h, arr, len(cuts)))

    def n_sub(self):
        n = C.c_int32()
        self._ck(mk_module_n_sub(self.h, C.byref(n)))
        return n.value

    def decomposition(self):
        n = C.c_int32(self.n_ops())
        arr = (C.c_int32 * n.value)()
        self._ck(mk_module_get_decomposition(self.h, arr, C.byref(n)))
        return list(arr[: n.value])

    def split(self, sub, at_op):
        self._ck(mk_module_split(self.h, sub, at_op))

    def fuse(self, first_sub, count):
        self._ck(mk_module_fuse(self.h, first_sub, count))

    def total_fuse(self):
        self._ck(mk_module_total_fuse(self.h))

    def contract(self, sub):
        cap = 64
        n_in, n_out = C.c_int32(cap), C.c_int32(cap)
        in_ids, out_ids = (C.c_int32 * cap)(), (C.c_int32 * cap)()
        in_specs, out_specs = (mk_tensor_spec * cap)(), (mk_tensor_spec * cap)()
        self._ck(mk_module_get_contract(self.h, sub, in_ids, in_specs, C.byref(n_in), out_ids, out_specs,
                                        C.byref(n_out)))
        return ([(in_ids[i], spec_tuple(in_specs[i])) for i in range(n_in.value)],
                [(out_ids[i], spec_tuple(out_specs[i])) for i in range(n_out.value)])

    # -- implementations -----------------------------------------------------------------------------
    def impls(self, sub):
        n = C.c_int32()
        self._ck(mk_impl_count(self.h, sub, C.byref(n)))
        out = []
        for i in range(n.value):
            s = C.c_char_p()
            self._ck(mk_impl_name(self.h, sub, i, C.byref(s)))
            out.append(s.value.decode())
        return out

    def bind(self, sub, name=None):
        self._ck(mk_module_bind(self.h, sub, name.encode() if name is not None else None))

    def bound_impl(self, sub):
        s = C.c_char_p()
        self._ck(mk_module_bound_impl(self.h, sub, C.byref(s)))
        return s.value.decode()

    # -- parameters, run -----------------------------------------------------------------------------
    def set_param(self, op_index, slot, tensor, dtype, shape, layout=MK_LAYOUT_ROW_MAJOR):
        spec = make_spec(dtype, shape, layout)
        self._ck(mk_module_set_param(self.h, op_index, slot, _ptr(tensor), C.byref(spec)))
        self._keep.append(tensor)

    def set_params(self, device_params, dtype, param_dtypes=None):
        """device_params: name -> (tensor on the device, logical shape).  LINEAR weights must
        already be stored in this module's weight_layout.  param_dtypes: name -> storage type of the
        parameters that do not have the module's (fp8 weights and their fp32 block scales)."""
        for j, op in enumerate(self.ops):
            for slot, key in enumerate(self.PARAM_SLOTS.get(op["kind"], ())):
                name = op["params"].get(key)
                if name is None:
                    continue
                t, shape = device_params[name]
                layout = self.weight_layout if (op["kind"] in ("linear", "linear_fp8") and slot == 0) else MK_LAYOUT_ROW_MAJOR
                self.set_param(j, slot, t, (param_dtypes or {}).get(name, dtype), shape, layout)

    def keep_intermediates(self, keep=True):
        self._ck(mk_module_keep_intermediates(self.h, 1 if keep else 0))

    def workspace_size(self):
        n = C.c_size_t()
        self._ck(mk_module_workspace_size(self.h, C.byref(n)))
        return n.value

    def launch_count(self):
        n = C.c_int32()
        self._ck(mk_module_launch_count(self.h, C.byref(n)))
        return n.value

    def _marshal(self, inputs, output):
        ins = (C.c_void_p * len(inputs))(*[_ptr(t) for t in inputs])
        outs = (C.c_void_p * 1)(_ptr(output))
        return ins, outs

    def forward(self, inputs, output, workspace=None, workspace_bytes=0, stream=0):
        ins, outs = self._marshal(inputs, output)
        ws = _ptr(workspace) if workspace is not None else None
        self._ck(mk_module_forward(self.h, ins, outs, ws, workspace_bytes, stream))

    def forward_sub(self, inputs, output, first_sub, count=1, workspace=None, workspace_bytes=0, stream=0):
        ins, outs = self._marshal(inputs, output)
        ws = _ptr(workspace) if workspace is not None else None
        self._ck(mk_module_forward_sub(self.h, ins, outs, ws, workspace_bytes, stream, first_sub, count))

    def profile(self, inputs, output, workspace=None, workspace_bytes=0, stream=0, iters=10):
        ins, outs = self._marshal(inputs, output)
        ws = _ptr(workspace) if workspace is not None else None
        ms = (C.c_float * self.n_sub())()
        self._ck(mk_module_profile(self.h, ins, outs, ws, workspace_bytes, stream, iters, ms))
        return list(ms)

    def swap(self, inputs, output, workspace=None, workspace_bytes=0, stream=0, iters=5, tau=0.9):
        """Rebind every submodule that runs at less than `tau` of its fastest alternative's speed.
        Returns (number rebound, [(ms before, ms after)] per submodule)."""
        ins, outs = self._marshal(inputs, output)
        ws = _ptr(workspace) if workspace is not None else None
        n = C.c_int32(0)
        ms = (C.c_float * (2 * self.n_sub()))()
        self._ck(mk_module_swap(self.h, ins, outs, ws, workspace_bytes, stream, iters, tau, C.byref(n), ms))
        return n.value, [(ms[2 * i], ms[2 * i + 1]) for i in range(self.n_sub())]

    def intermediate(self, value):
        vid = self.value_id[value] if isinstance(value, str) else value
        p = C.c_void_p()
        s = mk_tensor_spec()
        self._ck(mk_module_intermediate(self.h, vid, C.byref(p), C.byref(s)))
        return p.value, spec_tuple(s)
