"""CPU oracle for the Hadamard-quantized layer forward -- TEST INFRASTRUCTURE, not product code.

``hq_oracle.c`` holds the arithmetic (plain loops, fp64 / int64); this module only compiles
it with gcc, marshals numpy arrays into it, and chains its steps in the order the paper
gives them (Eq. 10 transform -> Eq. 3 quantize -> Eq. 12 / Eq. 14 integer product -> rescale).
Nothing here imports or calls the CUDA library, and the CUDA library never calls this.
Only the tests, the smoke check and the benchmark's CPU-baseline legs may import it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_DIR, "hq_oracle.c")
_LIB = os.path.join(_DIR, "libhq_oracle.so")
_lock = threading.Lock()
_lib = None

i64 = C.c_longlong


def build(force: bool = False) -> str:
    """Compile hq_oracle.c into libhq_oracle.so next to it (gcc -O2 -fopenmp)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    with _lock:
        if _lib is None:
            L = C.CDLL(build())
            p = C.c_void_p
            L.hqo_hadamard_raw.argtypes = [C.c_int, p]
            L.hqo_transform.argtypes = [p, i64, i64, C.c_int, p]
            L.hqo_quantize.argtypes = [p, i64, i64, C.c_int, C.c_int, C.c_float, p, p, p]
            L.hqo_pack_nibbles.argtypes = [p, i64, p]
            L.hqo_unpack_nibbles.argtypes = [p, i64, p]
            L.hqo_weight_quantize.argtypes = [p, i64, i64, C.c_int, p, p]
            L.hqo_weight_fold.argtypes = [p, i64, i64, i64, C.c_int, p]
            L.hqo_weight_double.argtypes = [p, i64, i64, i64, C.c_int, C.c_int, p, p]
            L.hqo_limb_split.argtypes = [p, i64, p, p]
            L.hqo_gemm_int.argtypes = [p, p, i64, i64, i64, p]
            L.hqo_gemm_int.restype = i64
            L.hqo_conv2d_int.argtypes = [p, p, i64, i64, i64, i64, i64, C.c_int, C.c_int, C.c_int, C.c_int, p]
            L.hqo_conv2d_int.restype = i64
            L.hqo_dequant.argtypes = [p, i64, i64, p, C.c_int, p, p, C.c_double, p]
            L.hqo_conv2d_dequant_perpixel.argtypes = [p, p, p, i64, i64, i64, i64, i64, C.c_int, C.c_int,
                                                      C.c_int, C.c_int, p, p, C.c_double, p]
            L.hqo_groupnorm_silu.argtypes = [p, i64, i64, i64, i64, C.c_int, p, p, C.c_double, p]
            L.hqo_layernorm_affine.argtypes = [p, i64, i64, p, p, i64, C.c_double, p]
            L.hqo_transform_width.argtypes = [p, i64, i64, i64, i64, C.c_int, p]
            L.hqo_codes_inverse_width.argtypes = [p, i64, i64, i64, i64, C.c_int, p]
            L.hqo_conv2d_int_z.argtypes = [p, p, i64, i64, i64, i64, i64, C.c_int, C.c_int, C.c_int, C.c_int, p]
            L.hqo_conv2d_int_z.restype = i64
            L.hqo_groupnorm.argtypes = [p, i64, i64, i64, i64, C.c_int, p, p, C.c_double, C.c_int, p]
            L.hqo_attention.argtypes = [p, i64, i64, i64, C.c_int, p]
            L.hqo_upsample_nearest2x.argtypes = [p, i64, i64, i64, i64, p]
            L.hqo_timestep_embedding.argtypes = [p, i64, i64, C.c_double, p]
            L.hqo_conv2d_float.argtypes = [p, p, p, i64, i64, i64, i64, i64, C.c_int, C.c_int, C.c_int, C.c_int, p]
            _lib = L
    return _lib


def num_threads() -> int:
    """Threads the OpenMP loops use (OMP_NUM_THREADS or the core count)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env and env.isdigit() and int(env) > 0:
        return int(env)
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dt):
    return np.ascontiguousarray(a, dtype=dt)


def _chk(rc, what):
    if rc != 0:
        raise ValueError(f"oracle {what} failed with code {rc}")


def qmax(bits: int) -> int:
    return (1 << (bits - 1)) - 1


def qmin(bits: int) -> int:
    return -(1 << (bits - 1))


# ----------------------------------------------------------------------------- steps

def hadamard_raw(n: int) -> np.ndarray:
    """H_raw (n x n, entries +-1) by the Sylvester recurrence -- Eq. 5 without the 1/sqrt(2), Eq. 7."""
    H = np.empty((n, n), np.int8)
    _chk(lib().hqo_hadamard_raw(n, _ptr(H)), "hadamard_raw")
    return H


def transform(x, had_block: int) -> np.ndarray:
    """u = x * BlockDiag(H_k) with the orthonormal H_k, along the last axis -- Eq. 10, Eq. 7."""
    x = _c(x, np.float64)
    cols = x.shape[-1]
    u = np.empty_like(x)
    _chk(lib().hqo_transform(_ptr(x), x.size // cols, cols, had_block, _ptr(u)), "transform")
    return u


def quantize(u, bits: int, static_scale: float | None = None, want_v: bool = False):
    """Eq. 3 along the last axis.  Returns (codes int8, scales fp32 [rows] or [1][, v = u/S before rounding])."""
    u = _c(u, np.float64)
    cols = u.shape[-1]
    rows = u.size // cols
    q = np.empty(u.shape, np.int8)
    mode = 0 if static_scale is None else 1
    scales = np.empty((rows if mode == 0 else 1,), np.float32)
    v = np.empty(u.shape, np.float64) if want_v else None
    _chk(lib().hqo_quantize(_ptr(u), rows, cols, bits, mode, float(static_scale or 0.0), _ptr(q), _ptr(scales),
                            _ptr(v)), "quantize")
    return (q, scales, v) if want_v else (q, scales)


def pack_nibbles(q) -> np.ndarray:
    q = _c(q, np.int8)
    out = np.empty(q.shape[:-1] + (q.shape[-1] // 2,), np.uint8)
    _chk(lib().hqo_pack_nibbles(_ptr(q), q.size, _ptr(out)), "pack_nibbles")
    return out


def unpack_nibbles(b) -> np.ndarray:
    b = _c(b, np.uint8)
    q = np.empty(b.shape[:-1] + (b.shape[-1] * 2,), np.int8)
    _chk(lib().hqo_unpack_nibbles(_ptr(b), q.size, _ptr(q)), "unpack_nibbles")
    return q


def weight_quantize(w, w_bits: int):
    """w [N][...]: per-output-channel Eq. 3.  Returns (W_int int32 same shape, S_w fp32 [N])."""
    w = _c(w, np.float64)
    N = w.shape[0]
    w_int = np.empty(w.shape, np.int32)
    s_w = np.empty((N,), np.float32)
    _chk(lib().hqo_weight_quantize(_ptr(w), N, w.size // N, w_bits, _ptr(w_int), _ptr(s_w)), "weight_quantize")
    return w_int, s_w


def weight_fold(w_int, had_block: int) -> np.ndarray:
    """B = H_raw * W_int over the input-channel (last) axis -- the inner product of Eq. 12 / Eq. 14."""
    w_int = _c(w_int, np.int32)
    N, Cc = w_int.shape[0], w_int.shape[-1]
    B = np.empty_like(w_int)
    _chk(lib().hqo_weight_fold(_ptr(w_int), N, w_int.size // (N * Cc), Cc, had_block, _ptr(B)), "weight_fold")
    return B


def weight_double(w, w_bits: int, had_block: int):
    """Double-Hadamard weights Q(H^T W).  Returns (B int32, S_w fp32 [N])."""
    w = _c(w, np.float64)
    N, Cc = w.shape[0], w.shape[-1]
    B = np.empty(w.shape, np.int32)
    s_w = np.empty((N,), np.float32)
    _chk(lib().hqo_weight_double(_ptr(w), N, w.size // (N * Cc), Cc, w_bits, had_block, _ptr(B), _ptr(s_w)),
         "weight_double")
    return B, s_w


def limb_split(B):
    B = _c(B, np.int32)
    hi = np.empty(B.shape, np.int8)
    lo = np.empty(B.shape, np.int8)
    _chk(lib().hqo_limb_split(_ptr(B), B.size, _ptr(hi), _ptr(lo)), "limb_split")
    return hi, lo


def gemm_int(q, B) -> np.ndarray:
    """acc[m][o] = sum_k q[m][k] * B[o][k], int64 -- the integer product of Eq. 12."""
    q = _c(q, np.int8)
    B = _c(B, np.int32)
    M, K = q.shape
    N = B.shape[0]
    assert B.shape[1] == K
    acc = np.empty((M, N), np.int64)
    bad = lib().hqo_gemm_int(_ptr(q), _ptr(B), M, N, K, _ptr(acc))
    if bad:
        raise OverflowError(f"{bad} accumulators exceed int32")
    return acc


def conv2d_int(q, B, stride: int, pad: int) -> np.ndarray:
    """Direct integer convolution, q NHWC int8, B [Cout][R][S][C] int32 -> int64 NHWC -- Eq. 14."""
    q = _c(q, np.int8)
    B = _c(B, np.int32)
    Nb, H, W, Cc = q.shape
    Cout, R, S, _ = B.shape
    Ho, Wo = (H + 2 * pad - R) // stride + 1, (W + 2 * pad - S) // stride + 1
    acc = np.empty((Nb, Ho, Wo, Cout), np.int64)
    bad = lib().hqo_conv2d_int(_ptr(q), _ptr(B), Nb, H, W, Cc, Cout, R, S, stride, pad, _ptr(acc))
    if bad:
        raise OverflowError(f"{bad} accumulators exceed int32")
    return acc


def dequant(acc, s_a, s_w, bias, alpha: float) -> np.ndarray:
    """y = alpha * S_a[m] * S_w[o] * acc + bias[o] in fp64 (S_a of size 1 is a scalar)."""
    acc = _c(acc, np.int64)
    N = acc.shape[-1]
    M = acc.size // N
    s_a = _c(s_a, np.float32).reshape(-1)
    s_w = _c(s_w, np.float32)
    b = None if bias is None else _c(bias, np.float32)
    y = np.empty(acc.shape, np.float64)
    scalar = 1 if s_a.size == 1 else 0
    assert scalar or s_a.size == M
    _chk(lib().hqo_dequant(_ptr(acc), M, N, _ptr(s_a), scalar, _ptr(s_w), _ptr(b), float(alpha), _ptr(y)), "dequant")
    return y


def conv2d_dequant_perpixel(q, s_a, B, stride: int, pad: int, s_w, bias, alpha: float) -> np.ndarray:
    """Convolution with one activation scale per input pixel (rescale per tap)."""
    q = _c(q, np.int8)
    B = _c(B, np.int32)
    Nb, H, W, Cc = q.shape
    Cout, R, S, _ = B.shape
    s_a = _c(s_a, np.float32).reshape(-1)
    assert s_a.size == Nb * H * W
    s_w = _c(s_w, np.float32)
    b = None if bias is None else _c(bias, np.float32)
    Ho, Wo = (H + 2 * pad - R) // stride + 1, (W + 2 * pad - S) // stride + 1
    y = np.empty((Nb, Ho, Wo, Cout), np.float64)
    _chk(lib().hqo_conv2d_dequant_perpixel(_ptr(q), _ptr(s_a), _ptr(B), Nb, H, W, Cc, Cout, R, S, stride, pad,
                                           _ptr(s_w), _ptr(b), float(alpha), _ptr(y)), "conv2d_dequant_perpixel")
    return y


def groupnorm_silu(x, groups: int, gamma, beta, eps: float = 1e-6) -> np.ndarray:
    """GroupNorm over `groups` groups of consecutive channels of an NHWC tensor, affine, then SiLU (fp64)."""
    x = _c(x, np.float64)
    Nb, H, W, Cc = x.shape
    gamma, beta = _c(gamma, np.float64), _c(beta, np.float64)
    out = np.empty_like(x)
    _chk(lib().hqo_groupnorm_silu(_ptr(x), Nb, H, W, Cc, groups, _ptr(gamma), _ptr(beta), float(eps), _ptr(out)),
         "groupnorm_silu")
    return out


def layernorm_affine(x, weight=None, bias=None, rows_per_group: int = 0, eps: float = 1e-6) -> np.ndarray:
    """LayerNorm over the last axis of x [rows, cols] (biased variance), then y * weight[g] + bias[g] with
    g = row // rows_per_group (one vector pair for all rows when rows_per_group <= 0); fp64."""
    x = _c(x, np.float64)
    rows, cols = x.shape
    w = None if weight is None else _c(np.asarray(weight, np.float64).reshape(-1, cols), np.float64)
    b = None if bias is None else _c(np.asarray(bias, np.float64).reshape(-1, cols), np.float64)
    groups = (rows + rows_per_group - 1) // rows_per_group if rows_per_group > 0 else 1
    for v in (w, b):
        if v is not None and v.shape[0] != groups:
            raise ValueError("one affine vector per group of rows is needed")
    out = np.empty_like(x)
    _chk(lib().hqo_layernorm_affine(_ptr(x), rows, cols, _ptr(w) if w is not None else None,
                                    _ptr(b) if b is not None else None, int(rows_per_group), float(eps), _ptr(out)),
         "layernorm_affine")
    return out


def groupnorm(x, groups: int, gamma, beta, eps: float = 1e-5, act: str = "none") -> np.ndarray:
    """GroupNorm of an NHWC tensor with the activation selectable ("none" or "silu"); fp64."""
    x = _c(x, np.float64)
    Nb, H, W, Cc = x.shape
    gamma, beta = _c(gamma, np.float64), _c(beta, np.float64)
    out = np.empty_like(x)
    _chk(lib().hqo_groupnorm(_ptr(x), Nb, H, W, Cc, groups, _ptr(gamma), _ptr(beta), float(eps),
                             {"none": 0, "silu": 1}[act], _ptr(out)), "groupnorm")
    return out


def silu(x) -> np.ndarray:
    """x * sigmoid(x), fp64."""
    x = np.asarray(x, np.float64)
    return x / (1.0 + np.exp(-x))


def round_bf16(x) -> np.ndarray:
    """The value a bf16 store keeps: fp64 -> fp32 -> the nearest number with 8 significant bits (ties to even), back
    as fp64.  Used where a tensor is defined to be held in bf16 between two layers."""
    f = np.ascontiguousarray(np.asarray(x, np.float64).astype(np.float32))
    u = f.view(np.uint32).astype(np.uint64)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16) << 16
    out = r.astype(np.uint32).view(np.float32).astype(np.float64)
    return np.where(np.isfinite(f), out, f.astype(np.float64))


def attention(qkv, heads: int) -> np.ndarray:
    """Self-attention core on qkv [Nb, L, 3C] (query | key | value column thirds, heads contiguous inside each):
    softmax(q k^T / sqrt(dh)) v per sample and head -> [Nb, L, C]; fp64."""
    qkv = _c(qkv, np.float64)
    Nb, L, C3 = qkv.shape
    Cc = C3 // 3
    assert 3 * Cc == C3
    out = np.empty((Nb, L, Cc), np.float64)
    _chk(lib().hqo_attention(_ptr(qkv), Nb, L, Cc, heads, _ptr(out)), "attention")
    return out


def upsample_nearest2x(x) -> np.ndarray:
    x = _c(x, np.float64)
    Nb, H, W, Cc = x.shape
    out = np.empty((Nb, 2 * H, 2 * W, Cc), np.float64)
    _chk(lib().hqo_upsample_nearest2x(_ptr(x), Nb, H, W, Cc, _ptr(out)), "upsample_nearest2x")
    return out


def timestep_embedding(t, dim: int, max_period: float = 10000.0) -> np.ndarray:
    """[cos(t f_i) | sin(t f_i)], f_i = max_period^(-i / (dim/2)); t [Nb] -> [Nb, dim]; fp64."""
    t = _c(t, np.float64).reshape(-1)
    out = np.empty((t.size, dim), np.float64)
    _chk(lib().hqo_timestep_embedding(_ptr(t), t.size, dim, float(max_period), _ptr(out)), "timestep_embedding")
    return out


def conv2d_float(x, w, bias, stride: int, pad: int) -> np.ndarray:
    """Floating-point convolution, x NHWC, w [Cout][R][S][C], zero padding; fp64."""
    x, w = _c(x, np.float64), _c(w, np.float64)
    Nb, H, W, Cc = x.shape
    Cout, R, S, _ = w.shape
    b = None if bias is None else _c(bias, np.float64)
    Ho, Wo = (H + 2 * pad - R) // stride + 1, (W + 2 * pad - S) // stride + 1
    out = np.empty((Nb, Ho, Wo, Cout), np.float64)
    _chk(lib().hqo_conv2d_float(_ptr(x), _ptr(w), _ptr(b), Nb, H, W, Cc, Cout, R, S, stride, pad, _ptr(out)),
         "conv2d_float")
    return out


def transform_width(x, had_block: int) -> np.ndarray:
    """u = X~ * BlockDiag(H_k) along the WIDTH axis of an NHWC tensor (orthonormal H_k) -- the product before Eq. 13."""
    x = _c(x, np.float64)
    Nb, H, W, Cc = x.shape
    u = np.empty_like(x)
    _chk(lib().hqo_transform_width(_ptr(x), Nb, H, W, Cc, had_block, _ptr(u)), "transform_width")
    return u


def codes_inverse_width(q, had_block: int) -> np.ndarray:
    """z = q * H_raw along the width axis (exact int32) -- the factor "(X H_c)_int * H_c" of Eq. 14 without 2^(-k/2)."""
    q = _c(q, np.int8)
    Nb, H, W, Cc = q.shape
    z = np.empty(q.shape, np.int32)
    _chk(lib().hqo_codes_inverse_width(_ptr(q), Nb, H, W, Cc, had_block, _ptr(z)), "codes_inverse_width")
    return z


def conv2d_int_z(z, B, stride: int, pad: int) -> np.ndarray:
    """Direct integer convolution of int32 NHWC activations with B [Cout][R][S][C] -> int64 NHWC (Eq. 14)."""
    z = _c(z, np.int32)
    B = _c(B, np.int32)
    Nb, H, W, Cc = z.shape
    Cout, R, S, _ = B.shape
    Ho, Wo = (H + 2 * pad - R) // stride + 1, (W + 2 * pad - S) // stride + 1
    acc = np.empty((Nb, Ho, Wo, Cout), np.int64)
    bad = lib().hqo_conv2d_int_z(_ptr(z), _ptr(B), Nb, H, W, Cc, Cout, R, S, stride, pad, _ptr(acc))
    if bad:
        raise OverflowError(f"{bad} accumulators exceed int32")
    return acc


# ----------------------------------------------------------------------------- chained layers

def alpha_for(weight_mode: str, had_block: int) -> float:
    """Folded weights carry H_raw, not the orthonormal H, so the second 2^(-k/2) of Eq. 12 sits in alpha."""
    if weight_mode == "folded" and had_block > 1:
        return float(2.0 ** (-0.5 * np.log2(had_block)))
    return 1.0


def prepare_weights(w, w_bits: int, had_block: int, weight_mode: str):
    """Offline weight side.  weight_mode: 'plain' B = Q(W); 'folded' B = H_raw*Q(W) (Eq. 12); 'double' B = Q(H^T W)."""
    if weight_mode == "plain":
        B, s_w = weight_quantize(w, w_bits)
    elif weight_mode == "folded":
        w_int, s_w = weight_quantize(w, w_bits)
        B = weight_fold(w_int, had_block)
    elif weight_mode == "double":
        B, s_w = weight_double(w, w_bits, had_block)
    else:
        raise ValueError(weight_mode)
    return B, s_w


def qlinear(x, w, bias, *, a_bits: int, w_bits: int, had_block: int, weight_mode: str = "folded",
            static_scale: float | None = None) -> dict:
    """Quantized linear layer, Eq. 12: x [M][K], w [N][K].  Returns every intermediate."""
    u = transform(x, had_block)
    q, s_a, v = quantize(u, a_bits, static_scale, want_v=True)
    B, s_w = prepare_weights(w, w_bits, had_block, weight_mode)
    acc = gemm_int(q, B.reshape(B.shape[0], -1))
    alpha = alpha_for(weight_mode, had_block)
    y = dequant(acc, s_a, s_w, bias, alpha)
    return dict(u=u, q=q, s_a=s_a, v=v, B=B, s_w=s_w, acc=acc, alpha=alpha, y=y)


def qconv(x, w, bias, *, a_bits: int, w_bits: int, had_block: int, stride: int, pad: int,
          weight_mode: str = "folded", static_scale: float | None = None) -> dict:
    """Quantized convolution, Eq. 14 with the transform over input channels: x NHWC, w [Cout][R][S][C]."""
    u = transform(x, had_block)
    q, s_a, v = quantize(u, a_bits, static_scale, want_v=True)
    B, s_w = prepare_weights(w, w_bits, had_block, weight_mode)
    alpha = alpha_for(weight_mode, had_block)
    acc = conv2d_int(q, B, stride, pad)
    if static_scale is None:
        y = conv2d_dequant_perpixel(q, s_a, B, stride, pad, s_w, bias, alpha)
    else:
        y = dequant(acc, s_a, s_w, bias, alpha)
    return dict(u=u, q=q, s_a=s_a, v=v, B=B, s_w=s_w, acc=acc, alpha=alpha, y=y)


def qconv_width(x, w, bias, *, a_bits: int, w_bits: int, had_block_w: int, stride: int, pad: int,
                static_scale: float) -> dict:
    """Quantized convolution exactly as Eq. 13-14 state it: the transform runs along the WIDTH axis, the weights are
    quantized untransformed, and the integer core is Conv((X~ H_c)_int * H_c, W_int) with one activation scale:
    y = 2^(-k/2) * S * S_w[o] * Conv(q * H_raw, W_int) + bias.   x NHWC, w [Cout][R][S][C]."""
    u = transform_width(x, had_block_w)
    q, s_a, v = quantize(u, a_bits, static_scale, want_v=True)      # elementwise with a static scale
    z = codes_inverse_width(q, had_block_w)
    w_int, s_w = weight_quantize(w, w_bits)
    acc = conv2d_int_z(z, w_int, stride, pad)
    alpha = float(2.0 ** (-0.5 * np.log2(had_block_w))) if had_block_w > 1 else 1.0
    y = dequant(acc, s_a, s_w, bias, alpha)
    return dict(u=u, q=q, s_a=s_a, v=v, z=z, B=w_int, s_w=s_w, acc=acc, alpha=alpha, y=y)
