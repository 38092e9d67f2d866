"""fp64 CPU oracle: one plain function per operator.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package may import this
module; only the tests, the smoke check and the benchmark's CPU-baseline leg
do.  It shares no code with the CUDA path.

Every function is the operator's definition written out in numpy float64, with
no blocking, fusion or reordering.  numpy's matmul serves as the contraction
step.  Inputs are float64 arrays that already hold the storage-rounded values;
no intermediate is rounded.

Sources for the definitions: the paper's subkernel listings in its appendix
"Example Solution for ConvolutionalVisionTransformer" (linear as x @ W with W
stored [K, N], LayerNorm with biased variance and eps inside the square root,
attention as scale -> mask -> softmax over keys -> weighted sum), its appendix
"Modular Kernel Generation Enables Better Correctness Checking" (safe softmax,
causal mask keeps the diagonal, fp32-or-wider accumulation, the exact GELU
versus its sigmoid approximation), and the workload list for the operators the
paper only names (RMSNorm, GroupNorm, SwiGLU, tanh-form GELU, 3x3 convolution).

Pins: every function here is checked in tests/test_oracle_*.py against brute
force on tiny shapes, closed forms, invariants and library special cases; no
function is "parity unpinned".
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


def _f64(x):
    a = np.asarray(x)
    if a.dtype != F64:
        raise TypeError("oracle operators take float64 arrays")
    return a


# ---------------------------------------------------------------- contraction
def linear(x, w):
    """Y[m, n] = sum_k X[m, k] * W[k, n]; W is the logical [K, N] matrix
    (paper: linear subkernel, weight pre-transposed to [K, N])."""
    x, w = _f64(x), _f64(w)
    if x.shape[-1] != w.shape[0]:
        raise ValueError("linear: inner dimensions differ")
    return x @ w


def linear_fp8_block(xq, sx, wq, sw, block=128):
    """Block-scaled fp8 contraction (the paper's FP8 MoE inference task; blocks as in that task: activations one
    scale per row and 128-wide K block, weights one per 128 x 128 block):
        Y[m, n] = sum_kb sx[m, kb] * sw[n // 128, kb] * sum_{k in block kb} xq[m, k] * wq[k, n]
    xq [M, K] and wq [K, N] hold the decoded fp8 values (exact in fp64), sx [M, K/128], sw [ceil(N/128), K/128].
    Written as the definition: dequantise, then the plain contraction."""
    xq, sx, wq, sw = _f64(xq), _f64(sx), _f64(wq), _f64(sw)
    M, K = xq.shape
    N = wq.shape[1]
    assert K % block == 0 and sx.shape == (M, K // block) and sw.shape == (-(-N // block), K // block)
    x = xq * np.repeat(sx, block, axis=1)
    wscale = np.repeat(np.repeat(sw.T, block, axis=0), block, axis=1)[:K, :N]      # [K, N]
    return x @ (wq * wscale)


def conv2d_3x3_nhwc(x, w):
    """Y[n,h,w,co] = sum_{kh,kw,ci} Xpad[n, h+kh-1, w+kw-1, ci] * W[co,kh,kw,ci]

    Cross-correlation (no kernel flip), stride 1, zero padding 1, NHWC
    activations, weights [C_out, 3, 3, C_in]."""
    x, w = _f64(x), _f64(w)
    nb, h, wd, c = x.shape
    co, kh, kw, ci = w.shape
    if (kh, kw) != (3, 3) or ci != c:
        raise ValueError("conv2d_3x3_nhwc: bad weight shape")
    xp = np.zeros((nb, h + 2, wd + 2, c), F64)
    xp[:, 1:h + 1, 1:wd + 1, :] = x
    y = np.zeros((nb, h, wd, co), F64)
    for a in range(3):
        for b in range(3):
            y += xp[:, a:a + h, b:b + wd, :] @ w[:, a, b, :].T
    return y


# ---------------------------------------------------------------- elementwise
def bias_add(x, b):
    """y[..., n] = x[..., n] + b[n] (bias after matmul)."""
    x, b = _f64(x), _f64(b)
    if b.shape != (x.shape[-1],):
        raise ValueError("bias_add: bias must match the last dimension")
    return x + b


def relu(x):
    return np.maximum(_f64(x), 0.0)


GELU_C0 = 0.7978845608028654  # sqrt(2 / pi)
GELU_C1 = 0.044715


def gelu_tanh(x):
    """0.5 * x * (1 + tanh(sqrt(2/pi) * (x + 0.044715 x^3)))."""
    x = _f64(x)
    return 0.5 * x * (1.0 + np.tanh(GELU_C0 * (x + GELU_C1 * x * x * x)))


def gelu_erf(x):
    """0.5 * x * (1 + erf(x / sqrt 2)): the exact GELU the tanh form approximates (paper, appendix on numerical
    precision: erf is the exact form)."""
    import math
    x = _f64(x)
    return 0.5 * x * (1.0 + np.vectorize(math.erf, otypes=[np.float64])(x / math.sqrt(2.0)))


def silu(x):
    """x / (1 + exp(-x))."""
    x = _f64(x)
    return x / (1.0 + np.exp(-x))


def scale(x, s):
    return _f64(x) * F64(s)


def clamp(x, lo, hi):
    return np.minimum(np.maximum(_f64(x), F64(lo)), F64(hi))


def residual_add(x, r):
    x, r = _f64(x), _f64(r)
    if x.shape != r.shape:
        raise ValueError("residual_add: shapes differ")
    return x + r


def swiglu(gu):
    """Input [..., 2F] holds [gate | up]; y = silu(gate) * up, shape [..., F]."""
    gu = _f64(gu)
    f2 = gu.shape[-1]
    if f2 % 2:
        raise ValueError("swiglu: last dimension must be even")
    f = f2 // 2
    return silu(gu[..., :f]) * gu[..., f:]


# ---------------------------------------------------------------- reductions
def layernorm(x, gamma, beta, eps):
    """Row-wise: mu = mean(x); var = mean((x-mu)^2) (biased, two-pass);
    y = (x-mu) / sqrt(var + eps) * gamma + beta."""
    x = _f64(x)
    mu = x.mean(axis=-1, keepdims=True)
    d = x - mu
    var = (d * d).mean(axis=-1, keepdims=True)
    y = d / np.sqrt(var + F64(eps))
    if gamma is not None:
        y = y * _f64(gamma)
    if beta is not None:
        y = y + _f64(beta)
    return y


def rmsnorm(x, gamma, eps):
    """Row-wise: y = x / sqrt(mean(x^2) + eps) * gamma."""
    x = _f64(x)
    ms = (x * x).mean(axis=-1, keepdims=True)
    y = x / np.sqrt(ms + F64(eps))
    if gamma is not None:
        y = y * _f64(gamma)
    return y


def softmax(x):
    """Row-wise safe softmax over the last dimension."""
    x = _f64(x)
    m = x.max(axis=-1, keepdims=True)
    e = np.exp(x - m)
    return e / e.sum(axis=-1, keepdims=True)


def groupnorm_nhwc(x, gamma, beta, groups, eps):
    """x [N, H, W, C]; group g = channels [g*C/G, (g+1)*C/G); per (n, g) the
    mean and the biased variance run over H*W*C/G elements;
    y = (x-mu)/sqrt(var+eps) * gamma_c + beta_c."""
    x = _f64(x)
    nb, h, w, c = x.shape
    if c % groups:
        raise ValueError("groupnorm: C must be divisible by groups")
    cg = c // groups
    xg = x.reshape(nb, h * w, groups, cg)
    mu = xg.mean(axis=(1, 3), keepdims=True)
    d = xg - mu
    var = (d * d).mean(axis=(1, 3), keepdims=True)
    y = (d / np.sqrt(var + F64(eps))).reshape(nb, h, w, c)
    if gamma is not None:
        y = y * _f64(gamma)
    if beta is not None:
        y = y + _f64(beta)
    return y


# ---------------------------------------------------------------- pooling (NHWC, square window, no padding)
def _windows(x, k, stride):
    """x [N, H, W, C] -> [N, OH, OW, k*k, C]: every window written out, OH = (H - k)//stride + 1."""
    x = _f64(x)
    n, h, w, c = x.shape
    if k < 1 or stride < 1 or k > h or k > w:
        raise ValueError("pooling: bad window")
    oh, ow = (h - k) // stride + 1, (w - k) // stride + 1
    out = np.empty((n, oh, ow, k * k, c), F64)
    for i in range(oh):
        for j in range(ow):
            out[:, i, j] = x[:, i * stride:i * stride + k, j * stride:j * stride + k, :].reshape(n, k * k, c)
    return out


def avgpool_nhwc(x, k, stride):
    """Mean over each k x k window (the pooling of the paper's MobileNetV1 example)."""
    return _windows(x, k, stride).mean(axis=3)


def maxpool_nhwc(x, k, stride):
    """Maximum over each window (first variant of the paper's transfer study)."""
    return _windows(x, k, stride).max(axis=3)


def lppool_nhwc(x, k, stride, p):
    """p-norm of each window, (sum |x|^p)^(1/p) (second variant of the transfer study)."""
    if not p >= 1.0:
        raise ValueError("lppool: p must be >= 1")
    return (np.abs(_windows(x, k, stride)) ** F64(p)).sum(axis=3) ** (1.0 / F64(p))


# ---------------------------------------------------------------- attention
def attention_causal_bhsd(q, k, v):
    """q, k, v [B, H, S, D].  S_ij = (q_i . k_j)/sqrt(D) for j <= i, masked
    out otherwise (diagonal kept); P = softmax over keys; O = P V.
    Returns the logical [B*S, H*D] matrix, head-major columns."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    b, h, s, d = q.shape
    out = np.empty((b, s, h, d), F64)
    keep = np.tril(np.ones((s, s), dtype=bool))  # j <= i
    for bi in range(b):
        for hi in range(h):
            sc = (q[bi, hi] @ k[bi, hi].T) / np.sqrt(F64(d))
            sc = np.where(keep, sc, -np.inf)
            out[bi, :, hi, :] = softmax(sc) @ v[bi, hi]
    return out.reshape(b * s, h * d)


def attention_causal_packed(qkv, batch, seq, heads, head_dim):
    """qkv [B*S, 3*H*D] with columns [Q | K | V], each head-major.
    Same computation as attention_causal_bhsd; returns [B*S, H*D]."""
    qkv = _f64(qkv)
    e = heads * head_dim
    if qkv.shape != (batch * seq, 3 * e):
        raise ValueError("attention_causal_packed: bad shape")
    t = qkv.reshape(batch, seq, 3, heads, head_dim)
    q = np.ascontiguousarray(t[:, :, 0].transpose(0, 2, 1, 3))
    k = np.ascontiguousarray(t[:, :, 1].transpose(0, 2, 1, 3))
    v = np.ascontiguousarray(t[:, :, 2].transpose(0, 2, 1, 3))
    return attention_causal_bhsd(q, k, v)


def attention_bhsd(q, k, v):
    """Unmasked (encoder) attention: q, k, v [B, H, S, D]; S_ij = (q_i . k_j)/sqrt(D) for every
    pair; P = softmax over keys; O = P V.  This is the paper's transformer-block attention
    (its ConvolutionalVisionTransformer example): scale, softmax over all keys, weighted sum.
    Returns the logical [B*S, H*D] matrix, head-major columns."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    b, h, s, d = q.shape
    out = np.empty((b, s, h, d), F64)
    for bi in range(b):
        for hi in range(h):
            sc = (q[bi, hi] @ k[bi, hi].T) / np.sqrt(F64(d))
            out[bi, :, hi, :] = softmax(sc) @ v[bi, hi]
    return out.reshape(b * s, h * d)


def attention_packed(qkv, batch, seq, heads, head_dim):
    """qkv [B*S, 3*H*D] with columns [Q | K | V], each head-major.
    Same computation as attention_bhsd; returns [B*S, H*D]."""
    qkv = _f64(qkv)
    e = heads * head_dim
    if qkv.shape != (batch * seq, 3 * e):
        raise ValueError("attention_packed: bad shape")
    t = qkv.reshape(batch, seq, 3, heads, head_dim)
    q = np.ascontiguousarray(t[:, :, 0].transpose(0, 2, 1, 3))
    k = np.ascontiguousarray(t[:, :, 1].transpose(0, 2, 1, 3))
    v = np.ascontiguousarray(t[:, :, 2].transpose(0, 2, 1, 3))
    return attention_bhsd(q, k, v)
