"""ctypes binding of the C-ABI library ``libhq.so`` (declared in ``include/hq.h``).

Argument marshalling only: every function here forwards to the entry point of the same name.
Device buffers are torch CUDA tensors (torch is used for memory and streams, nothing else);
their ``data_ptr()`` is what crosses the boundary.  Importing this module loads the CUDA
library and raises if it has not been built -- there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_DIR, "libhq.so")

HQ_OK = 0
HQ_F32, HQ_BF16 = 0, 1
HQ_CODES_NIBBLE, HQ_CODES_INT8 = 0, 1
HQ_SCALE_PER_ROW, HQ_SCALE_STATIC = 0, 1
HQ_W_PLAIN, HQ_W_FOLDED, HQ_W_DOUBLE, HQ_W_PLAIN_A2 = 0, 1, 2, 3
WEIGHT_MODES = {"plain": HQ_W_PLAIN, "folded": HQ_W_FOLDED, "double": HQ_W_DOUBLE, "plain_a2": HQ_W_PLAIN_A2}

EXPORTS = ["hq_version", "hq_status_string", "hq_check_status", "hq_hadamard_quant", "hq_weight_blob_bytes",
           "hq_weight_prepare", "hq_qgemm", "hq_qconv2d", "hq_workspace_size", "hq_qlinear", "hq_qconv",
           "hq_alpha_for", "hq_mma_i8_probe", "hq_qlinear_noalloc", "hq_hadamard_quant_width", "hq_qconv_width", "hq_gn_silu_quant",
           "hq_ln_quant", "hq_ln_qlinear", "hq_gn_silu_qconv", "hq_gn_qlinear", "hq_silu", "hq_add", "hq_add_rows_bcast",
           "hq_class_embed_add", "hq_timestep_embedding", "hq_upsample_nearest2x", "hq_concat_channels", "hq_groupnorm_act",
           "hq_conv2d_direct", "hq_attention", "hq_hadamard_quant_width2", "hq_qlinear_fused", "hq_set_pair_gemm", "hq_mma_i8_probe_pair",
           "hq_hadamard_quant_cat", "hq_gn_silu_quant_cat", "hq_gn_silu_qconv_cat", "hq_qconv_cat"]
HQ_NOALLOC_SCRATCH_BYTES = 8 * 1024 * 1024


class HqError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {status_string(status)} (hq_status {status})")


class WeightDesc(C.Structure):
    _fields_ = [("N", C.c_int64), ("C", C.c_int64), ("RS", C.c_int32), ("w_bits", C.c_int32),
                ("had_block", C.c_int32), ("mode", C.c_int32), ("limbs", C.c_int32), ("container", C.c_int32),
                ("C_pad", C.c_int64), ("N_pad", C.c_int64), ("bytes", C.c_int64), ("max_abs_b", C.c_int32),
                ("reserved", C.c_int32)]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2512_05746_b200.build` "
                          "(there is no CPU fallback for the CUDA path)")
    L = C.CDLL(LIB_PATH)
    p, i64, i32 = C.c_void_p, C.c_int64, C.c_int
    L.hq_version.restype = C.c_int
    L.hq_status_string.restype = C.c_char_p
    L.hq_status_string.argtypes = [C.c_int]
    L.hq_check_status.argtypes = [p]
    L.hq_hadamard_quant.argtypes = [p, i32, i64, i64, i64, i32, i32, i32, p, p, i32, i64, p, p]
    L.hq_weight_blob_bytes.restype = i64
    L.hq_weight_blob_bytes.argtypes = [i64, C.c_int32, i64, C.c_int32, C.c_int32, i32]
    L.hq_weight_prepare.argtypes = [p, i64, C.c_int32, i64, C.c_int32, C.c_int32, i32, i32, p, i64, p,
                                    C.POINTER(WeightDesc)]
    L.hq_qgemm.argtypes = [p, i32, i32, i64, i64, i64, C.POINTER(WeightDesc), p, p, i32, p, p, C.c_float, p, p, i32,
                           i64, p, p]
    L.hq_qconv2d.argtypes = [p, i32, i32, i64, i64, i64, i64, C.POINTER(WeightDesc), p, i32, i32, i32, i32, p, i32,
                             p, p, C.c_float, p, p, i32, p, p]
    L.hq_workspace_size.argtypes = [i64, i64, i32, C.POINTER(C.c_size_t)]
    L.hq_qlinear.argtypes = [p, i32, i64, i64, i64, C.POINTER(WeightDesc), p, p, p, i32, i32, p, p, i32, i64, p,
                             C.c_size_t, p, p]
    L.hq_qconv.argtypes = [p, i32, i64, i64, i64, i64, C.POINTER(WeightDesc), p, i32, i32, i32, i32, p, p, i32, i32,
                           p, p, i32, p, C.c_size_t, p, p]
    L.hq_qlinear_noalloc.argtypes = [p, i32, i64, i64, i64, C.POINTER(WeightDesc), p, p, p, i32, i32, p, p, i32, i64,
                                     p, p]
    L.hq_hadamard_quant_width.argtypes = [p, i32, i64, i64, i64, i64, i32, i32, p, p, p, p]
    L.hq_mma_i8_probe_pair.argtypes = [i32, i32, p, p]
    L.hq_mma_i8_probe_pair.restype = C.c_int
    L.hq_set_pair_gemm.argtypes = [i32]
    L.hq_set_pair_gemm.restype = C.c_int
    L.hq_qlinear_fused.argtypes = [p, i32, i64, i64, i64, C.POINTER(WeightDesc), p, p, p, i32, i32, p, p, i64, p, p]
    L.hq_qlinear_fused.restype = C.c_int
    L.hq_hadamard_quant_width2.argtypes = [p, i32, i64, i64, i64, i64, i32, i32, p, p, p, p]
    L.hq_hadamard_quant_width2.restype = C.c_int
    L.hq_qconv_width.argtypes = [p, i32, i64, i64, i64, i64, C.POINTER(WeightDesc), p, i32, i32, i32, i32, p, p, i32, i32,
                                 p, p, i32, p, C.c_size_t, p, p]
    L.hq_gn_silu_quant.argtypes = [p, i32, i64, i64, i64, i64, i32, p, p, p, C.c_float, i32, i32, i32, p, p, i32, i64, p, p,
                                   C.c_size_t, p]
    L.hq_ln_quant.argtypes = [p, i32, i64, i64, i64, p, p, i64, C.c_float, i32, i32, i32, p, p, i32, i64, p, p]
    L.hq_ln_qlinear.argtypes = [p, i32, i64, i64, i64, p, p, i64, C.c_float, C.POINTER(WeightDesc), p, p, p, i32, p, i32, i64,
                                p, C.c_size_t, p, p]
    L.hq_gn_silu_qconv.argtypes = [p, i32, i64, i64, i64, i64, i32, p, p, p, C.c_float, C.POINTER(WeightDesc), p, i32, i32, i32,
                                   i32, p, p, i32, i32, p, p, i32, p, C.c_size_t, p, C.c_size_t, p, p]
    L.hq_gn_qlinear.argtypes = [p, i32, i64, i64, i64, i32, p, p, C.c_float, i32, C.POINTER(WeightDesc), p, p, p, i32, p, i32,
                                i64, p, C.c_size_t, p, C.c_size_t, p, p]
    L.hq_silu.argtypes = [p, i64, p, p]
    L.hq_add.argtypes = [p, p, i64, p, p]
    L.hq_add_rows_bcast.argtypes = [p, p, i64, i64, i64, p]
    L.hq_class_embed_add.argtypes = [p, p, p, i64, i64, i64, p]
    L.hq_timestep_embedding.argtypes = [p, i64, i64, C.c_float, p, p]
    L.hq_upsample_nearest2x.argtypes = [p, i64, i64, i64, i64, p, p]
    L.hq_concat_channels.argtypes = [p, i64, p, i64, i64, p, p]
    L.hq_groupnorm_act.argtypes = [p, i64, i64, i64, i64, i32, p, p, C.c_float, i32, p, p, C.c_size_t, p]
    L.hq_conv2d_direct.argtypes = [p, i32, p, p, i64, i64, i64, i64, i64, i32, i32, i32, p, i32, p]
    L.hq_attention.argtypes = [p, i64, i64, i64, i32, p, p, p]
    L.hq_alpha_for.restype = C.c_float
    L.hq_hadamard_quant_cat.argtypes = [p, i64, p, i64, i64, i32, i64, i64, i32, i32, i32, p, p, i32, i64, p, p]
    L.hq_gn_silu_quant_cat.argtypes = [p, p, i64, i32, i64, i64, i64, i64, i32, p, p, p, C.c_float, i32, i32, i32, p, p, i32,
                                       i64, p, p, C.c_size_t, p]
    L.hq_gn_silu_qconv_cat.argtypes = [p, p, i64, i32, i64, i64, i64, i64, i32, p, p, p, C.c_float, C.POINTER(WeightDesc), p,
                                       i32, i32, i32, i32, p, p, i32, i32, p, p, i32, p, C.c_size_t, p, C.c_size_t, p, p]
    L.hq_qconv_cat.argtypes = [p, p, i64, i32, i64, i64, i64, i64, C.POINTER(WeightDesc), p, i32, i32, i32, i32, p, p, i32,
                               i32, p, p, i32, p, C.c_size_t, p, p]
    L.hq_alpha_for.argtypes = [C.POINTER(WeightDesc)]
    L.hq_mma_i8_probe.argtypes = [i32, i32, p, p]
    for name in ("hq_check_status", "hq_hadamard_quant", "hq_weight_prepare", "hq_qgemm", "hq_qconv2d",
                 "hq_workspace_size", "hq_qlinear", "hq_qconv", "hq_mma_i8_probe", "hq_qlinear_noalloc",
                 "hq_hadamard_quant_width", "hq_qconv_width", "hq_gn_silu_quant", "hq_ln_quant", "hq_ln_qlinear", "hq_gn_silu_qconv",
                 "hq_gn_qlinear", "hq_silu", "hq_add", "hq_add_rows_bcast", "hq_class_embed_add", "hq_timestep_embedding",
                 "hq_upsample_nearest2x", "hq_concat_channels", "hq_groupnorm_act", "hq_conv2d_direct", "hq_attention",
                 "hq_hadamard_quant_cat", "hq_gn_silu_quant_cat", "hq_gn_silu_qconv_cat", "hq_qconv_cat"):
        getattr(L, name).restype = C.c_int
    return L


lib = _load()


def status_string(status: int) -> str:
    return lib.hq_status_string(int(status)).decode()


def _check(status: int, what: str):
    if status != HQ_OK:
        raise HqError(status, what)


def _dptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _dtype_code(t):
    import torch
    if t.dtype == torch.float32:
        return HQ_F32
    if t.dtype == torch.bfloat16:
        return HQ_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def hq_version() -> int:
    return lib.hq_version()


def hq_check_status(dev_status) -> None:
    """dev_status: a torch int32 tensor of one element (device); raises HqError on a recorded timeout."""
    host = np.array([int(dev_status.cpu()[0])], dtype=np.int32)
    _check(lib.hq_check_status(host.ctypes.data_as(C.c_void_p)), "hq_check_status")


def hq_hadamard_quant(x, had_block: int, bits: int, codes, container: int, scales=None, static_scale=None,
                      stream=None, x2=None) -> None:
    """x [rows, cols] (fp32/bf16, last dim contiguous) -> codes (uint8 [rows, pitch]) and scales (fp32).  With x2
    [rows, cols2] the input is the column concatenation [x | x2], read in place."""
    rows, cols = x.shape
    mode = HQ_SCALE_PER_ROW if static_scale is None else HQ_SCALE_STATIC
    if x2 is not None:
        _check(lib.hq_hadamard_quant_cat(_dptr(x), x.stride(0), _dptr(x2), x2.stride(0), cols, _dtype_code(x), rows,
                                         cols + x2.shape[1], had_block, bits, mode, _dptr(static_scale), _dptr(codes),
                                         container, codes.stride(0), _dptr(scales), _stream(stream)), "hq_hadamard_quant_cat")
        return
    _check(lib.hq_hadamard_quant(_dptr(x), _dtype_code(x), rows, cols, x.stride(0), had_block, bits, mode,
                                 _dptr(static_scale), _dptr(codes), container, codes.stride(0), _dptr(scales),
                                 _stream(stream)), "hq_hadamard_quant")


class PreparedWeight:
    """Result of hq_weight_prepare: host blob + scales + descriptor, and (after .to_device()) device copies."""

    def __init__(self, desc: WeightDesc, blob: np.ndarray, s_w: np.ndarray):
        self.desc, self.blob, self.s_w = desc, blob, s_w
        self.blob_dev = None
        self.s_w_dev = None

    def to_device(self, device="cuda"):
        import torch
        self.blob_dev = torch.from_numpy(self.blob).to(device)
        self.s_w_dev = torch.from_numpy(self.s_w).to(device)
        return self

    @property
    def alpha(self) -> float:
        return float(lib.hq_alpha_for(C.byref(self.desc)))


def hq_weight_blob_bytes(N: int, RS: int, Cin: int, w_bits: int, had_block: int, mode: int) -> int:
    return int(lib.hq_weight_blob_bytes(N, RS, Cin, w_bits, had_block, mode))


def hq_weight_prepare(w: np.ndarray, w_bits: int, had_block: int, mode: int, container: int) -> PreparedWeight:
    """w: host fp32 [N, C] or [N, R, S, C]."""
    w = np.ascontiguousarray(w, dtype=np.float32)
    N, Cin = w.shape[0], w.shape[-1]
    RS = w.size // (N * Cin)
    nbytes = hq_weight_blob_bytes(N, RS, Cin, w_bits, had_block, mode)
    blob = np.zeros((max(nbytes, 1),), np.int8)
    s_w = np.zeros((N,), np.float32)
    desc = WeightDesc()
    _check(lib.hq_weight_prepare(w.ctypes.data_as(C.c_void_p), N, RS, Cin, w_bits, had_block, mode, container,
                                 blob.ctypes.data_as(C.c_void_p), nbytes, s_w.ctypes.data_as(C.c_void_p),
                                 C.byref(desc)), "hq_weight_prepare")
    return PreparedWeight(desc, blob, s_w)


def hq_qgemm(a_codes, container: int, a_bits: int, K: int, pw: PreparedWeight, scale_a=None, bias=None,
             alpha: float = 1.0, acc_out=None, y=None, dev_status=None, stream=None) -> None:
    M = a_codes.shape[0]
    scalar = 1 if (scale_a is not None and scale_a.numel() == 1) else 0
    ydt = _dtype_code(y) if y is not None else HQ_BF16
    ldy = y.stride(0) if y is not None else 0
    _check(lib.hq_qgemm(_dptr(a_codes), container, a_bits, M, K, a_codes.stride(0), C.byref(pw.desc),
                        _dptr(pw.blob_dev), _dptr(scale_a), scalar, _dptr(pw.s_w_dev), _dptr(bias), alpha,
                        _dptr(acc_out), _dptr(y), ydt, ldy, _dptr(dev_status), _stream(stream)), "hq_qgemm")


def hq_qconv2d(a_codes, container: int, a_bits: int, Nb: int, H: int, W: int, Cin: int, pw: PreparedWeight, R: int,
               S: int, stride: int, pad: int, scale_a=None, bias=None, alpha: float = 1.0, acc_out=None, y=None,
               dev_status=None, stream=None) -> None:
    scalar = 1 if (scale_a is None or scale_a.numel() == 1) else 0
    ydt = _dtype_code(y) if y is not None else HQ_BF16
    _check(lib.hq_qconv2d(_dptr(a_codes), container, a_bits, Nb, H, W, Cin, C.byref(pw.desc), _dptr(pw.blob_dev), R,
                          S, stride, pad, _dptr(scale_a), scalar, _dptr(pw.s_w_dev), _dptr(bias), alpha,
                          _dptr(acc_out), _dptr(y), ydt, _dptr(dev_status), _stream(stream)), "hq_qconv2d")


def hq_workspace_size(rows: int, cols: int, container: int) -> int:
    out = C.c_size_t(0)
    _check(lib.hq_workspace_size(rows, cols, container, C.byref(out)), "hq_workspace_size")
    return int(out.value)


def hq_qlinear(x, pw: PreparedWeight, bias, a_bits: int, y, workspace, static_scale=None, dev_status=None,
               stream=None) -> None:
    M, K = x.shape
    mode = HQ_SCALE_PER_ROW if static_scale is None else HQ_SCALE_STATIC
    _check(lib.hq_qlinear(_dptr(x), _dtype_code(x), M, K, x.stride(0), C.byref(pw.desc), _dptr(pw.blob_dev),
                          _dptr(pw.s_w_dev), _dptr(bias), a_bits, mode, _dptr(static_scale), _dptr(y), _dtype_code(y),
                          y.stride(0), _dptr(workspace), workspace.numel() * workspace.element_size(),
                          _dptr(dev_status), _stream(stream)), "hq_qlinear")


def hq_qlinear_noalloc(x, pw: PreparedWeight, bias, a_bits: int, y, static_scale=None, dev_status=None,
                       stream=None) -> None:
    """hq_qlinear without a workspace: the intermediate codes and scales use the library's built-in 8 MiB device
    array, for callers that have no way to allocate one.  Raises HqError(9) when the layer does not fit."""
    M, K = x.shape
    mode = HQ_SCALE_PER_ROW if static_scale is None else HQ_SCALE_STATIC
    _check(lib.hq_qlinear_noalloc(_dptr(x), _dtype_code(x), M, K, x.stride(0), C.byref(pw.desc), _dptr(pw.blob_dev),
                                  _dptr(pw.s_w_dev), _dptr(bias), a_bits, mode, _dptr(static_scale), _dptr(y),
                                  _dtype_code(y), y.stride(0), _dptr(dev_status), _stream(stream)),
           "hq_qlinear_noalloc")


def hq_qconv(x, pw: PreparedWeight, R: int, S: int, stride: int, pad: int, bias, a_bits: int, y, workspace,
             static_scale=None, dev_status=None, stream=None, x2=None) -> None:
    """The fused convolution layer on x NHWC, or (x2 given) on the channel concatenation [x | x2] read in place."""
    Nb, H, W, Cin = x.shape
    mode = HQ_SCALE_PER_ROW if static_scale is None else HQ_SCALE_STATIC
    if x2 is not None:
        _check(lib.hq_qconv_cat(_dptr(x), _dptr(x2), Cin, _dtype_code(x), Nb, H, W, Cin + x2.shape[3], C.byref(pw.desc),
                                _dptr(pw.blob_dev), R, S, stride, pad, _dptr(pw.s_w_dev), _dptr(bias), a_bits, mode,
                                _dptr(static_scale), _dptr(y), _dtype_code(y), _dptr(workspace),
                                workspace.numel() * workspace.element_size(), _dptr(dev_status), _stream(stream)),
               "hq_qconv_cat")
        return
    _check(lib.hq_qconv(_dptr(x), _dtype_code(x), Nb, H, W, Cin, C.byref(pw.desc), _dptr(pw.blob_dev), R, S, stride,
                        pad, _dptr(pw.s_w_dev), _dptr(bias), a_bits, mode, _dptr(static_scale), _dptr(y),
                        _dtype_code(y), _dptr(workspace), workspace.numel() * workspace.element_size(),
                        _dptr(dev_status), _stream(stream)), "hq_qconv")


def hq_gn_silu_quant(x, groups: int, gamma, beta, eps: float, had_block: int, bits: int, codes, container: int,
                     scratch, scales=None, static_scale=None, stream=None, pre_bias=None, x2=None) -> None:
    """GroupNorm(groups) + SiLU of x NHWC (of x + pre_bias[n, c] when a bf16 [Nb, C] addend is given; of the channel
    concatenation [x | x2] when x2 is given), then transform over channels + quantization into codes [Nb*H*W, pitch]."""
    Nb, H, W, Cin = x.shape
    mode = HQ_SCALE_PER_ROW if static_scale is None else HQ_SCALE_STATIC
    if x2 is not None:
        _check(lib.hq_gn_silu_quant_cat(_dptr(x), _dptr(x2), Cin, _dtype_code(x), Nb, H, W, Cin + x2.shape[3], groups,
                                        _dptr(gamma), _dptr(beta), _dptr(pre_bias), eps, had_block, bits, mode,
                                        _dptr(static_scale), _dptr(codes), container, codes.stride(0), _dptr(scales),
                                        _dptr(scratch), scratch.numel() * scratch.element_size(), _stream(stream)),
               "hq_gn_silu_quant_cat")
        return
    _check(lib.hq_gn_silu_quant(_dptr(x), _dtype_code(x), Nb, H, W, Cin, groups, _dptr(gamma), _dptr(beta), _dptr(pre_bias), eps, had_block,
                                bits, mode, _dptr(static_scale), _dptr(codes), container, codes.stride(0), _dptr(scales),
                                _dptr(scratch), scratch.numel() * scratch.element_size(), _stream(stream)),
           "hq_gn_silu_quant")


def hq_gn_silu_qconv(x, groups: int, gamma, beta, eps: float, pw: PreparedWeight, R: int, S: int, stride: int, pad: int,
                     bias, a_bits: int, y, workspace, scratch, static_scale=None, dev_status=None, stream=None,
                     pre_bias=None, x2=None) -> None:
    """The fused convolution layer with GroupNorm + SiLU in front (x NHWC; pre_bias: bf16 [Nb, C] added to x before the
    normalisation, or None; x2: the input is the channel concatenation [x | x2], read in place)."""
    Nb, H, W, Cin = x.shape
    mode = HQ_SCALE_PER_ROW if static_scale is None else HQ_SCALE_STATIC
    if x2 is not None:
        _check(lib.hq_gn_silu_qconv_cat(_dptr(x), _dptr(x2), Cin, _dtype_code(x), Nb, H, W, Cin + x2.shape[3], groups,
                                        _dptr(gamma), _dptr(beta), _dptr(pre_bias), eps, C.byref(pw.desc), _dptr(pw.blob_dev),
                                        R, S, stride, pad, _dptr(pw.s_w_dev), _dptr(bias), a_bits, mode, _dptr(static_scale),
                                        _dptr(y), _dtype_code(y), _dptr(workspace),
                                        workspace.numel() * workspace.element_size(), _dptr(scratch),
                                        scratch.numel() * scratch.element_size(), _dptr(dev_status), _stream(stream)),
               "hq_gn_silu_qconv_cat")
        return
    _check(lib.hq_gn_silu_qconv(_dptr(x), _dtype_code(x), Nb, H, W, Cin, groups, _dptr(gamma), _dptr(beta), _dptr(pre_bias), eps,
                                C.byref(pw.desc), _dptr(pw.blob_dev), R, S, stride, pad, _dptr(pw.s_w_dev), _dptr(bias),
                                a_bits, mode, _dptr(static_scale), _dptr(y), _dtype_code(y), _dptr(workspace),
                                workspace.numel() * workspace.element_size(), _dptr(scratch),
                                scratch.numel() * scratch.element_size(), _dptr(dev_status), _stream(stream)),
           "hq_gn_silu_qconv")


def hq_ln_quant(x, weight, bias, rows_per_group: int, eps: float, had_block: int, bits: int, codes, container: int,
                scales=None, static_scale=None, stream=None) -> None:
    """LayerNorm over each row of x [rows, cols] with the affine vectors weight/bias [groups, cols] (or None) of the row's
    group, then transform + quantization into codes [rows, pitch]."""
    rows, cols = x.shape
    mode = HQ_SCALE_PER_ROW if static_scale is None else HQ_SCALE_STATIC
    _check(lib.hq_ln_quant(_dptr(x), _dtype_code(x), rows, cols, x.stride(0), _dptr(weight), _dptr(bias), rows_per_group,
                           eps, had_block, bits, mode, _dptr(static_scale), _dptr(codes), container, codes.stride(0),
                           _dptr(scales), _stream(stream)), "hq_ln_quant")


def hq_ln_qlinear(x, ln_weight, ln_bias, rows_per_group: int, eps: float, pw: PreparedWeight, bias, a_bits: int, y,
                  workspace, dev_status=None, stream=None) -> None:
    """The fused linear layer with LayerNorm + per-sample affine in front (per-row activation scales)."""
    M, K = x.shape
    _check(lib.hq_ln_qlinear(_dptr(x), _dtype_code(x), M, K, x.stride(0), _dptr(ln_weight), _dptr(ln_bias), rows_per_group,
                             eps, C.byref(pw.desc), _dptr(pw.blob_dev), _dptr(pw.s_w_dev), _dptr(bias), a_bits, _dptr(y),
                             _dtype_code(y), y.stride(0), _dptr(workspace), workspace.numel() * workspace.element_size(),
                             _dptr(dev_status), _stream(stream)), "hq_ln_qlinear")


def hq_hadamard_quant_width(x, had_block_w: int, bits: int, static_scale, z, scale_out=None, stream=None) -> None:
    """x NHWC (fp32/bf16, dense) -> z int8 NHWC = clamp(rint(x H_c / S)) * H_raw along the width axis (Eq. 13-14)."""
    Nb, H, W, Cin = x.shape
    _check(lib.hq_hadamard_quant_width(_dptr(x), _dtype_code(x), Nb, H, W, Cin, had_block_w, bits, _dptr(static_scale),
                                       _dptr(z), _dptr(scale_out), _stream(stream)), "hq_hadamard_quant_width")


def hq_hadamard_quant_width2(x, had_block_w: int, bits: int, static_scale, z_limbs, scale_out=None, stream=None) -> None:
    """As hq_hadamard_quant_width for blocks of up to 64 positions: z_limbs int8 NHWC [Nb, H, W, 2C] = [hi | lo]."""
    Nb, H, W, Cin = x.shape
    _check(lib.hq_hadamard_quant_width2(_dptr(x), _dtype_code(x), Nb, H, W, Cin, had_block_w, bits, _dptr(static_scale),
                                        _dptr(z_limbs), _dptr(scale_out), _stream(stream)), "hq_hadamard_quant_width2")


def hq_qconv_width(x, pw: PreparedWeight, R: int, S: int, stride: int, pad: int, bias, a_bits: int, had_block_w: int,
                   static_scale, y, workspace, dev_status=None, stream=None) -> None:
    """The convolution layer with the width-axis transform (Eq. 13-14); pw: PLAIN weights for the INT8 container."""
    Nb, H, W, Cin = x.shape
    _check(lib.hq_qconv_width(_dptr(x), _dtype_code(x), Nb, H, W, Cin, C.byref(pw.desc), _dptr(pw.blob_dev), R, S, stride,
                              pad, _dptr(pw.s_w_dev), _dptr(bias), a_bits, had_block_w, _dptr(static_scale), _dptr(y),
                              _dtype_code(y), _dptr(workspace), workspace.numel() * workspace.element_size(),
                              _dptr(dev_status), _stream(stream)), "hq_qconv_width")


def hq_mma_i8_probe(ctas: int, iters: int, dev_status=None, stream=None) -> None:
    _check(lib.hq_mma_i8_probe(ctas, iters, _dptr(dev_status), _stream(stream)), "hq_mma_i8_probe")


def hq_gn_qlinear(x, Nb: int, groups: int, gamma, beta, eps: float, silu: bool, pw: PreparedWeight, bias, a_bits: int, y,
                  workspace, scratch, dev_status=None, stream=None) -> None:
    """The fused linear layer on the pixels of x [Nb * rows_per_sample, C] with GroupNorm (+ SiLU) in front."""
    M, Cin = x.shape
    _check(lib.hq_gn_qlinear(_dptr(x), _dtype_code(x), Nb, M // Nb, Cin, groups, _dptr(gamma), _dptr(beta), eps, int(silu),
                             C.byref(pw.desc), _dptr(pw.blob_dev), _dptr(pw.s_w_dev), _dptr(bias), a_bits, _dptr(y),
                             _dtype_code(y), y.stride(0), _dptr(workspace), workspace.numel() * workspace.element_size(),
                             _dptr(scratch), scratch.numel() * scratch.element_size(), _dptr(dev_status), _stream(stream)),
           "hq_gn_qlinear")


def hq_silu(x, out, stream=None) -> None:
    _check(lib.hq_silu(_dptr(x), x.numel(), _dptr(out), _stream(stream)), "hq_silu")


def hq_add(a, b, out, stream=None) -> None:
    _check(lib.hq_add(_dptr(a), _dptr(b), a.numel(), _dptr(out), _stream(stream)), "hq_add")


def hq_add_rows_bcast(h, e, stream=None) -> None:
    """h [Nb, ..., C] += e [Nb, C] in place."""
    Nb, Cc = e.shape
    _check(lib.hq_add_rows_bcast(_dptr(h), _dptr(e), Nb, h.numel() // (Nb * Cc), Cc, _stream(stream)), "hq_add_rows_bcast")


def hq_class_embed_add(emb, table, labels, stream=None) -> None:
    Nb, dim = emb.shape
    _check(lib.hq_class_embed_add(_dptr(emb), _dptr(table), _dptr(labels), Nb, dim, table.shape[0], _stream(stream)),
           "hq_class_embed_add")


def hq_timestep_embedding(t, out, max_period: float = 10000.0, stream=None) -> None:
    Nb, dim = out.shape
    _check(lib.hq_timestep_embedding(_dptr(t), Nb, dim, max_period, _dptr(out), _stream(stream)), "hq_timestep_embedding")


def hq_upsample_nearest2x(x, out, stream=None) -> None:
    Nb, H, W, Cc = x.shape
    _check(lib.hq_upsample_nearest2x(_dptr(x), Nb, H, W, Cc, _dptr(out), _stream(stream)), "hq_upsample_nearest2x")


def hq_concat_channels(a, b, out, stream=None) -> None:
    Ca, Cb = a.shape[-1], b.shape[-1]
    _check(lib.hq_concat_channels(_dptr(a), Ca, _dptr(b), Cb, a.numel() // Ca, _dptr(out), _stream(stream)),
           "hq_concat_channels")


def hq_groupnorm_act(x, groups: int, gamma, beta, eps: float, silu: bool, out, scratch, stream=None) -> None:
    Nb, H, W, Cc = x.shape
    _check(lib.hq_groupnorm_act(_dptr(x), Nb, H, W, Cc, groups, _dptr(gamma), _dptr(beta), eps, int(silu), _dptr(out),
                                _dptr(scratch), scratch.numel() * scratch.element_size(), _stream(stream)), "hq_groupnorm_act")


def hq_conv2d_direct(x, w, bias, R: int, stride: int, pad: int, y, stream=None) -> None:
    """Floating-point convolution: x NHWC, w device fp32 [Cout, R, R, C], y NHWC."""
    Nb, H, W, Cc = x.shape
    _check(lib.hq_conv2d_direct(_dptr(x), _dtype_code(x), _dptr(w), _dptr(bias), Nb, H, W, Cc, w.shape[0], R, stride, pad,
                                _dptr(y), _dtype_code(y), _stream(stream)), "hq_conv2d_direct")


def hq_attention(qkv, Nb: int, heads: int, out, dev_status=None, stream=None) -> None:
    """qkv [Nb * L, 3C] -> out [Nb * L, C]."""
    M, C3 = qkv.shape
    _check(lib.hq_attention(_dptr(qkv), Nb, M // Nb, C3 // 3, heads, _dptr(out), _dptr(dev_status), _stream(stream)),
           "hq_attention")


def hq_qlinear_fused(x, pw: PreparedWeight, bias, a_bits: int, y, static_scale=None, dev_status=None, stream=None) -> None:
    """The fused linear layer as one kernel (transform and quantization inside the product kernel; no workspace)."""
    M, K = x.shape
    mode = HQ_SCALE_PER_ROW if static_scale is None else HQ_SCALE_STATIC
    _check(lib.hq_qlinear_fused(_dptr(x), _dtype_code(x), M, K, x.stride(0), C.byref(pw.desc), _dptr(pw.blob_dev),
                                _dptr(pw.s_w_dev), _dptr(bias), a_bits, mode, _dptr(static_scale), _dptr(y), y.stride(0),
                                _dptr(dev_status), _stream(stream)), "hq_qlinear_fused")


def hq_set_pair_gemm(mode: int) -> int:
    """Where products run on pairs of SMs (cta_group::2): 0 nowhere, 1 (or True) wherever covered, 2 (the default) where
    it measured faster (streamed weights, convolutions); returns the previous mode."""
    return int(lib.hq_set_pair_gemm(int(mode)))


def hq_mma_i8_probe_pair(pairs: int, iters: int, dev_status=None, stream=None) -> None:
    _check(lib.hq_mma_i8_probe_pair(pairs, iters, _dptr(dev_status), _stream(stream)), "hq_mma_i8_probe_pair")
