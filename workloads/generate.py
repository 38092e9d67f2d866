"""Counter-based seeded tensors for the workloads C1..C5.

Every tensor is drawn from its own Philox stream keyed by (seed, tensor id),
so changing one tensor's shape never changes another tensor's values.  Values
are rounded once to their storage type (fp32, or bf16 with round-to-nearest-
even); `Tensor.store` holds exactly the bytes a device buffer receives and
`Tensor.f64()` widens those same bytes, without further rounding, for the CPU
oracle.

Distribution notation follows the workload list: "N(0, 1/fan_in)" gives the
variance, "N(0, 0.02)" / "N(1, 0.02)" give the standard deviation (the usual
GPT-style init), U(a, b) is uniform on the open interval.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


# --------------------------------------------------------------------------
# storage formats
# --------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round-to-nearest-even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounding = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + rounding) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


# fp8 e4m3 ("fn" variant: bias 7, no infinities, 0x7f / 0xff NaN, largest finite 448, subnormals of 2^-9)
def _e4m3_table() -> np.ndarray:
    t = np.empty(256, np.float64)
    for b in range(256):
        e, m = (b >> 3) & 0xF, b & 7
        if e == 15 and m == 7:
            v = np.nan
        elif e == 0:
            v = m * 2.0 ** -9
        else:
            v = (1.0 + m / 8.0) * 2.0 ** (e - 7)
        t[b] = -v if b & 0x80 else v
    return t


E4M3_VALUES = _e4m3_table()
E4M3_MAX = 448.0


def f32_to_e4m3_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> e4m3 codes (uint8), round-to-nearest-even, magnitudes beyond 448 saturate to 448."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    sign = (np.signbit(x)).astype(np.uint8) << 7
    a = np.minimum(np.abs(x).astype(np.float64), E4M3_MAX)
    f, ex = np.frexp(a)                      # a = f * 2^ex, f in [0.5, 1)
    e = ex - 1                               # a = (2 f) * 2^e, 2 f in [1, 2)
    normal = a >= 2.0 ** -6
    mant = np.rint((2.0 * f - 1.0) * 8.0)    # ties to even
    carry = mant == 8
    e = np.where(carry, e + 1, e)
    mant = np.where(carry, 0, mant)
    nb = ((e + 7).astype(np.int64) << 3) | mant.astype(np.int64)
    sb = np.rint(a * 2.0 ** 9).astype(np.int64)   # subnormals: multiples of 2^-9; 8 is the smallest normal's code
    bits = np.where(normal, nb, sb)
    bits = np.minimum(bits, 0x7E)
    return (bits.astype(np.uint8) | sign).astype(np.uint8)


def e4m3_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return E4M3_VALUES[b]


@dataclass
class Tensor:
    """One named tensor in its storage format.

    dtype "f32": `store` is float32.  dtype "bf16": `store` is uint16 holding
    bf16 bit patterns.  dtype "fp8": `store` is uint8 holding e4m3 codes.
    Shapes are logical, row-major, innermost last.
    """

    name: str
    dtype: str
    store: np.ndarray

    @property
    def shape(self):
        return tuple(self.store.shape)

    def f64(self) -> np.ndarray:
        if self.dtype == "bf16":
            return bf16_bits_to_f64(self.store)
        if self.dtype == "fp8":
            return e4m3_bits_to_f64(self.store)
        return self.store.astype(np.float64)

    def nbytes(self) -> int:
        return int(self.store.nbytes)


def make(name: str, dtype: str, values_f32: np.ndarray) -> Tensor:
    """Round fp32 values to the storage type and wrap them."""
    v = np.ascontiguousarray(values_f32, dtype=np.float32)
    if dtype == "bf16":
        return Tensor(name, "bf16", f32_to_bf16_bits(v))
    if dtype == "f32":
        return Tensor(name, "f32", v)
    if dtype == "fp8":
        return Tensor(name, "fp8", f32_to_e4m3_bits(v))
    raise ValueError(f"unknown dtype {dtype!r}")


def quantize_blocks(name: str, values_f32: np.ndarray, block_rows: int, block_cols: int):
    """Synthesis of a block-scaled fp8 tensor from fp32 values: one fp32 scale per block_rows x block_cols block,
    scale = amax / 448, codes = e4m3(value / scale).  Returns (codes Tensor [R, C], scales Tensor
    [ceil(R / block_rows), ceil(C / block_cols)]).  This only MAKES inputs; what a consumer computes from
    codes and scales is defined where it is computed."""
    v = np.ascontiguousarray(values_f32, dtype=np.float32)
    R, Cc = v.shape
    nr, nc = -(-R // block_rows), -(-Cc // block_cols)
    pad = np.zeros((nr * block_rows, nc * block_cols), np.float32)
    pad[:R, :Cc] = v
    blk = pad.reshape(nr, block_rows, nc, block_cols)
    amax = np.abs(blk).max(axis=(1, 3))
    scale = (np.maximum(amax, np.float32(1e-10)) / np.float32(E4M3_MAX)).astype(np.float32)
    q = (blk / scale[:, None, :, None]).astype(np.float32).reshape(nr * block_rows, nc * block_cols)[:R, :Cc]
    return Tensor(name, "fp8", f32_to_e4m3_bits(q)), Tensor(name + "_scale", "f32", scale)


# --------------------------------------------------------------------------
# draws
# --------------------------------------------------------------------------
def _rng(seed: int, tensor_id: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed), int(tensor_id)]))


def _normal(seed, tid, shape, mean=0.0, std=1.0) -> np.ndarray:
    x = _rng(seed, tid).standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    if mean != 0.0:
        x += np.float32(mean)
    return x


def _uniform(seed, tid, shape, lo, hi) -> np.ndarray:
    u = _rng(seed, tid).random(size=shape, dtype=np.float32)  # [0, 1)
    # open interval: move exact 0 draws half a step inside
    u = np.where(u == 0.0, np.float32(2.0 ** -25), u)
    return (np.float32(lo) + (np.float32(hi) - np.float32(lo)) * u).astype(np.float32)


def int_valued(seed: int, tid: int, shape, lo: int, hi: int, dtype: str, name="t") -> Tensor:
    """Integers in [lo, hi]: exact in bf16, fp32 and fp64 alike, so a
    contraction over them has one exact answer in every precision."""
    v = _rng(seed, tid).integers(lo, hi + 1, size=shape).astype(np.float32)
    return make(name, dtype, v)


@dataclass
class Workload:
    """Inputs and parameters of one composed module, plus its op sequence.

    `ops` is declarative: each entry names an operator kind, the values it
    reads, the parameters it uses and its scalar attributes.  `partitions`
    maps a decomposition name to the list of first-op indices of its
    submodules.
    """

    name: str
    dtype: str
    inputs: dict = field(default_factory=dict)
    params: dict = field(default_factory=dict)
    ops: list = field(default_factory=list)
    partitions: dict = field(default_factory=dict)
    flops: float = 0.0
    min_bytes: float = 0.0


def _op(kind, out, ins, params=None, **attrs):
    return {"kind": kind, "out": out, "in": list(ins), "params": dict(params or {}), "attrs": attrs}


# --------------------------------------------------------------------------
# C1: fp32 linear -> +bias -> ReLU -> row LayerNorm
# --------------------------------------------------------------------------
def c1(seed=0, M=64, K=256, N=128, dtype="f32") -> Workload:
    w = Workload("c1", dtype)
    w.inputs["x"] = make("x", dtype, _normal(seed, 0, (M, K)))
    w.params["W"] = make("W", dtype, _normal(seed, 1, (K, N), std=(1.0 / K) ** 0.5))
    w.params["b"] = make("b", dtype, _uniform(seed, 2, (N,), -0.1, 0.1))
    w.params["gamma"] = make("gamma", dtype, np.ones((N,), np.float32))
    w.params["beta"] = make("beta", dtype, np.zeros((N,), np.float32))
    w.ops = [
        _op("linear", "y0", ["x"], {"w": "W"}, n=N),
        _op("bias_add", "y1", ["y0"], {"b": "b"}),
        _op("relu", "y2", ["y1"]),
        _op("layernorm", "y3", ["y2"], {"gamma": "gamma", "beta": "beta"}, eps=1e-5),
    ]
    w.partitions = {"fused": [0], "split": [0, 2, 3], "per_op": [0, 1, 2, 3]}
    w.flops = 2.0 * M * K * N
    esz = 4 if dtype == "f32" else 2
    w.min_bytes = esz * (M * K + K * N + N + M * N)
    return w


# --------------------------------------------------------------------------
# C2: bf16 GEMM -> +bias -> GELU(tanh) -> x0.5 -> clamp[-1, 1]
# --------------------------------------------------------------------------
def c2(seed=0, M=4096, K=4096, N=4096, dtype="bf16") -> Workload:
    w = Workload("c2", dtype)
    w.inputs["x"] = make("x", dtype, _normal(seed, 0, (M, K)))
    w.params["W"] = make("W", dtype, _normal(seed, 1, (K, N), std=(1.0 / K) ** 0.5))
    w.params["bias"] = make("bias", dtype, _normal(seed, 2, (N,), std=0.02))
    w.ops = [
        _op("linear", "y0", ["x"], {"w": "W"}, n=N),
        _op("bias_add", "y1", ["y0"], {"b": "bias"}),
        _op("gelu_tanh", "y2", ["y1"]),
        _op("scale", "y3", ["y2"], s=0.5),
        _op("clamp", "y4", ["y3"], lo=-1.0, hi=1.0),
    ]
    w.partitions = {"fused": [0], "split": [0, 2, 3, 4]}
    w.flops = 2.0 * M * K * N
    esz = 4 if dtype == "f32" else 2
    w.min_bytes = esz * (M * K + K * N + N + M * N)
    return w


# --------------------------------------------------------------------------
# C3: bf16 NHWC conv3x3 -> +bias -> ReLU -> GroupNorm
# --------------------------------------------------------------------------
def c3(seed=0, NB=32, H=56, W=56, C=128, CO=128, G=32, dtype="bf16") -> Workload:
    w = Workload("c3", dtype)
    w.inputs["x"] = make("x", dtype, _normal(seed, 0, (NB, H, W, C)))
    # logical weight layout [C_out, kh, kw, C_in]
    w.params["Wc"] = make("Wc", dtype, _normal(seed, 1, (CO, 3, 3, C), std=(1.0 / (9 * C)) ** 0.5))
    w.params["bias"] = make("bias", dtype, _normal(seed, 2, (CO,), std=0.02))
    w.params["gamma"] = make("gamma", dtype, _normal(seed, 3, (CO,), mean=1.0, std=0.02))
    w.params["beta"] = make("beta", dtype, _normal(seed, 4, (CO,), std=0.02))
    w.ops = [
        _op("conv2d_3x3", "y0", ["x"], {"w": "Wc"}, c_out=CO),
        _op("bias_add", "y1", ["y0"], {"b": "bias"}),
        _op("relu", "y2", ["y1"]),
        _op("groupnorm", "y3", ["y2"], {"gamma": "gamma", "beta": "beta"}, groups=G, eps=1e-5),
    ]
    w.partitions = {"fused": [0], "split2": [0, 3], "split3": [0, 2, 3]}
    w.flops = 2.0 * NB * H * W * CO * 9 * C
    w.min_bytes = 2 * (NB * H * W * C + CO * 9 * C + 3 * CO + NB * H * W * CO)
    return w


# --------------------------------------------------------------------------
# C4: bf16 causal attention -> out-proj + residual -> RMSNorm
# --------------------------------------------------------------------------
def c4(seed=0, B=16, H=16, S=2048, D=128, dtype="bf16") -> Workload:
    w = Workload("c4", dtype)
    E = H * D
    w.inputs["q"] = make("q", dtype, _normal(seed, 0, (B, H, S, D)))
    w.inputs["k"] = make("k", dtype, _normal(seed, 1, (B, H, S, D)))
    w.inputs["v"] = make("v", dtype, _normal(seed, 2, (B, H, S, D)))
    w.inputs["r"] = make("r", dtype, _normal(seed, 3, (B * S, E)))
    w.params["Wo"] = make("Wo", dtype, _normal(seed, 4, (E, E), std=0.02))
    w.params["gamma"] = make("gamma", dtype, np.ones((E,), np.float32))
    w.ops = [
        # attention output is logically [B*S, H*D], head-major columns
        _op("attention_causal", "a", ["q", "k", "v"], layout="bhsd", heads=H, head_dim=D),
        _op("linear", "p", ["a"], {"w": "Wo"}, n=E),
        _op("residual_add", "h", ["p", "r"]),
        _op("rmsnorm", "y", ["h"], {"gamma": "gamma"}, eps=1e-6),
    ]
    w.partitions = {"split3": [0, 1, 3], "per_op": [0, 1, 2, 3], "fused": [0]}
    w.flops = 4.0 * B * H * D * (S * (S + 1) / 2) + 2.0 * B * S * E * E
    w.min_bytes = 2 * (3 * B * H * S * D + B * S * E + E * E + E + B * S * E)
    return w


# --------------------------------------------------------------------------
# C5: bf16 4-layer pre-norm decoder (RMSNorm, causal MHA, SwiGLU FFN)
# --------------------------------------------------------------------------
def c5(seed=0, B=8, S=1024, E=2048, H=16, F=8192, L=4, dtype="bf16", stream="f32") -> Workload:
    """`stream`: storage type of the residual stream (the running sum x).  fp32 by default: with a
    bf16 stream the four layers' rounding errors, amplified layer over layer, put a few hundred of
    the 16.8 M outputs outside rtol/atol 2e-2 even for exact kernels; every other activation and all
    weights are `dtype`."""
    w = Workload("c5", dtype)
    D = E // H
    w.inputs["x"] = make("x", dtype, _normal(seed, 0, (B * S, E)))
    w.params["ones"] = make("ones", dtype, np.ones((E,), np.float32))
    cur = "x"
    tid = 1
    layer_starts = []
    for l in range(L):
        layer_starts.append(len(w.ops))
        # W_qkv columns are [Q | K | V], each head-major; W_gu columns are [gate | up]
        w.params[f"Wqkv{l}"] = make(f"Wqkv{l}", dtype, _normal(seed, tid + 0, (E, 3 * E), std=0.02))
        w.params[f"Wo{l}"] = make(f"Wo{l}", dtype, _normal(seed, tid + 1, (E, E), std=0.02))
        w.params[f"Wgu{l}"] = make(f"Wgu{l}", dtype, _normal(seed, tid + 2, (E, 2 * F), std=0.02))
        w.params[f"Wd{l}"] = make(f"Wd{l}", dtype, _normal(seed, tid + 3, (F, E), std=0.02))
        tid += 4
        w.ops += [
            _op("rmsnorm", f"n1_{l}", [cur], {"gamma": "ones"}, eps=1e-6),
            _op("linear", f"qkv_{l}", [f"n1_{l}"], {"w": f"Wqkv{l}"}, n=3 * E),
            _op("attention_causal", f"att_{l}", [f"qkv_{l}"], layout="packed_qkv", heads=H,
                head_dim=D, batch=B, seq=S),
            _op("linear", f"o_{l}", [f"att_{l}"], {"w": f"Wo{l}"}, n=E),
            _op("residual_add", f"x1_{l}", [f"o_{l}", cur], store=stream),
            _op("rmsnorm", f"n2_{l}", [f"x1_{l}"], {"gamma": "ones"}, eps=1e-6),
            _op("linear", f"gu_{l}", [f"n2_{l}"], {"w": f"Wgu{l}"}, n=2 * F),
            _op("swiglu", f"hid_{l}", [f"gu_{l}"]),
            _op("linear", f"d_{l}", [f"hid_{l}"], {"w": f"Wd{l}"}, n=E),
            _op("residual_add", f"x2_{l}", [f"d_{l}", f"x1_{l}"], store=stream),
        ]
        cur = f"x2_{l}"
    w.ops.append(_op("rmsnorm", "y", [cur], {"gamma": "ones"}, eps=1e-6))
    n_ops = len(w.ops)
    # default decomposition: GEMMs carry their elementwise tails, norms and attention stand alone
    fused_cuts = []
    for s in layer_starts:
        fused_cuts += [s + 0, s + 1, s + 2, s + 3, s + 5, s + 6, s + 8]
    fused_cuts.append(n_ops - 1)
    w.partitions = {"fused_tails": fused_cuts, "per_op": list(range(n_ops)), "fused": [0]}
    T = B * S
    per_layer = (2.0 * T * E * 3 * E + 4.0 * B * H * D * (S * (S + 1) / 2) + 2.0 * T * E * E
                 + 2.0 * T * E * 2 * F + 2.0 * T * F * E)
    w.flops = L * per_layer
    w.min_bytes = 2 * (2 * T * E + L * (3 * E * E + E * E + 3 * E * F))
    return w


# --------------------------------------------------------------------------
# C6: bf16 post-norm encoder layers (unmasked MHA with biases, LayerNorm, ReLU FFN): the shape of
# the transformer block in the paper's ConvolutionalVisionTransformer example, at a head_dim the
# tensor-core attention kernel takes
# --------------------------------------------------------------------------
def c6(seed=0, B=16, S=512, E=1024, H=8, F=4096, L=2, dtype="bf16") -> Workload:
    w = Workload("c6", dtype)
    D = E // H
    w.inputs["x"] = make("x", dtype, _normal(seed, 0, (B * S, E)))
    cur = "x"
    tid = 1
    layer_starts = []
    for l in range(L):
        layer_starts.append(len(w.ops))
        shapes = {"Wqkv": (E, 3 * E), "Wo": (E, E), "W1": (E, F), "W2": (F, E)}
        for i, (nm, shp) in enumerate(shapes.items()):
            w.params[f"{nm}{l}"] = make(f"{nm}{l}", dtype, _normal(seed, tid + i, shp, std=0.02))
            w.params[f"b{nm[1:]}{l}"] = make(f"b{nm[1:]}{l}", dtype, _normal(seed, tid + 4 + i, (shp[1],), std=0.02))
        for i, nm in enumerate(("g1", "g2")):
            w.params[f"{nm}_{l}"] = make(f"{nm}_{l}", dtype, 1.0 + _normal(seed, tid + 8 + i, (E,), std=0.02))
            w.params[f"{nm}b_{l}"] = make(f"{nm}b_{l}", dtype, _normal(seed, tid + 10 + i, (E,), std=0.02))
        tid += 12
        w.ops += [
            _op("linear", f"qkv0_{l}", [cur], {"w": f"Wqkv{l}"}, n=3 * E),
            _op("bias_add", f"qkv_{l}", [f"qkv0_{l}"], {"b": f"bqkv{l}"}),
            _op("attention", f"att_{l}", [f"qkv_{l}"], layout="packed_qkv", heads=H, head_dim=D, batch=B, seq=S),
            _op("linear", f"o0_{l}", [f"att_{l}"], {"w": f"Wo{l}"}, n=E),
            _op("bias_add", f"o1_{l}", [f"o0_{l}"], {"b": f"bo{l}"}),
            _op("residual_add", f"r1_{l}", [f"o1_{l}", cur]),
            _op("layernorm", f"x1_{l}", [f"r1_{l}"], {"gamma": f"g1_{l}", "beta": f"g1b_{l}"}, eps=1e-5),
            _op("linear", f"h0_{l}", [f"x1_{l}"], {"w": f"W1{l}"}, n=F),
            _op("bias_add", f"h1_{l}", [f"h0_{l}"], {"b": f"b1{l}"}),
            _op("relu", f"h_{l}", [f"h1_{l}"]),
            _op("linear", f"d0_{l}", [f"h_{l}"], {"w": f"W2{l}"}, n=E),
            _op("bias_add", f"d1_{l}", [f"d0_{l}"], {"b": f"b2{l}"}),
            _op("residual_add", f"r2_{l}", [f"d1_{l}", f"x1_{l}"]),
            _op("layernorm", f"x2_{l}", [f"r2_{l}"], {"gamma": f"g2_{l}", "beta": f"g2b_{l}"}, eps=1e-5),
        ]
        cur = f"x2_{l}"
    n_ops = len(w.ops)
    # default decomposition: GEMMs carry bias, activation and residual; attention and the norms stand alone
    fused_cuts = []
    for s in layer_starts:
        fused_cuts += [s + 0, s + 2, s + 3, s + 6, s + 7, s + 10, s + 13]
    w.partitions = {"fused_tails": fused_cuts, "per_op": list(range(n_ops)), "fused": [0]}
    T = B * S
    per_layer = 2.0 * T * E * 3 * E + 4.0 * B * H * D * S * S + 2.0 * T * E * E + 4.0 * T * E * F
    w.flops = L * per_layer
    w.min_bytes = 2 * (2 * T * E + L * (4 * E * E + 2 * E * F))
    return w


# --------------------------------------------------------------------------
# C7: bf16 conv3x3 -> +bias -> ReLU -> pooling (mean / maximum / p-norm): the convolution stage and the
# swappable pooling subkernel of the paper's MobileNetV1 transfer study, at C3's convolution shape
# --------------------------------------------------------------------------
def c7(seed=0, NB=32, H=56, W=56, C=128, CO=128, pool="avg", k=7, stride=7, p=2.0, dtype="bf16") -> Workload:
    w = Workload("c7", dtype)
    w.inputs["x"] = make("x", dtype, _normal(seed, 0, (NB, H, W, C)))
    w.params["Wc"] = make("Wc", dtype, _normal(seed, 1, (CO, 3, 3, C), std=(1.0 / (9 * C)) ** 0.5))
    w.params["bias"] = make("bias", dtype, _normal(seed, 2, (CO,), std=0.02))
    attrs = {"k": k, "stride": stride}
    if pool == "lp":
        attrs["p"] = p
    w.ops = [
        _op("conv2d_3x3", "y0", ["x"], {"w": "Wc"}, c_out=CO),
        _op("bias_add", "y1", ["y0"], {"b": "bias"}),
        _op("relu", "y2", ["y1"]),
        _op(pool + "pool", "y3", ["y2"], **attrs),
    ]
    w.partitions = {"fused": [0], "split2": [0, 3], "per_op": [0, 1, 2, 3]}
    oh, ow = (H - k) // stride + 1, (W - k) // stride + 1
    w.flops = 2.0 * NB * H * W * CO * 9 * C
    w.min_bytes = 2 * (NB * H * W * C + CO * 9 * C + CO + NB * oh * ow * CO)
    return w


# --------------------------------------------------------------------------
# C8: block-scaled fp8 GEMM, the contraction of the paper's FP8 MoE inference task: activations quantised per
# token and 128-channel block, weights per 128 x 128 block, fp32 scales, bf16 result (the expert projection
# shape hidden 7168 -> 4096 by default)
# --------------------------------------------------------------------------
def c8(seed=0, M=4096, K=7168, N=4096, bias=False) -> Workload:
    w = Workload("c8", "bf16")
    xq, sx = quantize_blocks("xq", _normal(seed, 0, (M, K)), 1, 128)
    wq, sw = quantize_blocks("Wq", _normal(seed, 1, (K, N), std=(1.0 / K) ** 0.5), 128, 128)
    w.inputs["xq"], w.inputs["sx"] = xq, Tensor("sx", "f32", sx.store)
    w.params["Wq"], w.params["sw"] = wq, Tensor("sw", "f32", np.ascontiguousarray(sw.store.T))   # [N / 128, K / 128]
    w.ops = [_op("linear_fp8", "y0", ["xq", "sx"], {"w": "Wq", "sw": "sw"}, n=N)]
    if bias:
        w.params["bias"] = make("bias", "bf16", _normal(seed, 2, (N,), std=0.02))
        w.ops += [_op("bias_add", "y1", ["y0"], {"b": "bias"}), _op("silu", "y2", ["y1"])]
    w.partitions = {"fused": [0], "per_op": list(range(len(w.ops)))}
    w.flops = 2.0 * M * K * N
    w.min_bytes = M * K + K * N + 4 * (sx.store.size + sw.store.size) + 2 * M * N
    return w


# --------------------------------------------------------------------------
# C9: a residual bottleneck block on an NHWC feature map: 1 x 1 convolution (C -> CM) + bias + ReLU, 3 x 3
# convolution (CM -> CM) + bias + ReLU, 1 x 1 convolution (CM -> C) + bias + skip connection + ReLU.  A 1 x 1
# convolution is a LINEAR over the channel dimension, so the whole block is three tensor-core launches.
# --------------------------------------------------------------------------
def c9(seed=0, NB=32, H=56, W=56, C=256, CM=64, dtype="bf16") -> Workload:
    w = Workload("c9", dtype)
    w.inputs["x"] = make("x", dtype, _normal(seed, 0, (NB, H, W, C)))
    w.params["W1"] = make("W1", dtype, _normal(seed, 1, (C, CM), std=(1.0 / C) ** 0.5))
    w.params["b1"] = make("b1", dtype, _normal(seed, 2, (CM,), std=0.02))
    w.params["Wc"] = make("Wc", dtype, _normal(seed, 3, (CM, 3, 3, CM), std=(2.0 / (9 * CM)) ** 0.5))
    w.params["b2"] = make("b2", dtype, _normal(seed, 4, (CM,), std=0.02))
    w.params["W3"] = make("W3", dtype, _normal(seed, 5, (CM, C), std=(2.0 / CM) ** 0.5))
    w.params["b3"] = make("b3", dtype, _normal(seed, 6, (C,), std=0.02))
    w.ops = [
        _op("linear", "a0", ["x"], {"w": "W1"}, n=CM),
        _op("bias_add", "a1", ["a0"], {"b": "b1"}),
        _op("relu", "a2", ["a1"]),
        _op("conv2d_3x3", "c0", ["a2"], {"w": "Wc"}, c_out=CM),
        _op("bias_add", "c1", ["c0"], {"b": "b2"}),
        _op("relu", "c2", ["c1"]),
        _op("linear", "d0", ["c2"], {"w": "W3"}, n=C),
        _op("bias_add", "d1", ["d0"], {"b": "b3"}),
        _op("residual_add", "d2", ["d1", "x"]),
        _op("relu", "y", ["d2"]),
    ]
    w.partitions = {"fused": [0], "split3": [0, 3, 6], "per_op": list(range(10))}
    w.flops = 2.0 * NB * H * W * (C * CM + 9 * CM * CM + CM * C)
    w.min_bytes = 2 * (2 * NB * H * W * C + 2 * C * CM + 9 * CM * CM + 2 * CM + C)
    return w


WORKLOADS = {"c1": c1, "c2": c2, "c3": c3, "c4": c4, "c5": c5, "c6": c6, "c7": c7, "c8": c8, "c9": c9}
