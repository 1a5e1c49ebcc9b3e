"""GPU parity of the fused layer calls (hq_qlinear, hq_qconv): transform -> quantize -> integer product -> rescale.

Two checks per case.  (1) The codes and scales the call left in its workspace follow the code acceptance rule
against the oracle's.  (2) The output equals the oracle's rescale of the oracle's integer product of THOSE codes
(the device's own), within the float tolerance -- so a code that legitimately differs at a rounding tie does not
blur the output check.  For the small configurations the end-to-end distance to the all-oracle layer is bounded too.
"""
import numpy as np
import pytest

from paper_2512_05746_b200 import inputs
from hq_testutil import (SCALE_RTOL, Y_BF16_RTOL, check_codes, rel_err, unpack_nibbles_np, weight_integers,
                         workspace_views)

pytestmark = pytest.mark.gpu


def rms_rel(y, y_ref):
    """||y - y_ref|| / ||y_ref||: the end-to-end distance to the all-oracle layer.  A code that differs at a rounding
    tie moves a few outputs by one weight step, which the element-wise maximum would blow up; the norm does not."""
    return float(np.sqrt(np.mean((y.astype(np.float64) - y_ref) ** 2)) / np.sqrt(np.mean(y_ref ** 2)))


@pytest.fixture(scope="module")
def env():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2512_05746_b200 import binding as hq
    return torch, hq


def _codes_from_ws(hq, ws, rows, cols, container):
    codes, scales = workspace_views(ws, rows, cols, container)
    c = codes.cpu().numpy()
    q = unpack_nibbles_np(c[:, : cols // 2]) if container == hq.HQ_CODES_NIBBLE else c[:, :cols].view(np.int8)
    return q, scales.cpu().numpy()


def run_linear(torch, hq, oracle, x, w, b, a_bits, had_block, mode, container, rows_checked=None):
    M, K = x.shape
    N = w.shape[0]
    pw = hq.hq_weight_prepare(w, 4, had_block, hq.WEIGHT_MODES[mode], container).to_device()
    y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros((hq.hq_workspace_size(M, K, container),), dtype=torch.uint8, device="cuda")
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    hq.hq_qlinear(torch.from_numpy(x).cuda(), pw, None if b is None else torch.from_numpy(b).cuda(), a_bits, y, ws,
                  dev_status=status)
    torch.cuda.synchronize()
    hq.hq_check_status(status)
    q_gpu, s_gpu = _codes_from_ws(hq, ws, M, K, container)
    idx = np.arange(M) if rows_checked is None else rows_checked
    ref = oracle.qlinear(x[idx], w, b, a_bits=a_bits, w_bits=4, had_block=had_block, weight_mode=mode)
    assert np.allclose(s_gpu[idx], ref["s_a"], rtol=SCALE_RTOL, atol=0)
    check_codes(q_gpu[idx], ref["q"], ref["v"], "fused linear")
    B = weight_integers(oracle, pw, w, 4, had_block, mode)
    y_own = oracle.dequant(oracle.gemm_int(q_gpu[idx], B), s_gpu[idx], pw.s_w, b, pw.alpha)
    y_gpu = y.float().cpu().numpy()[idx]
    assert rel_err(y_gpu, y_own) <= Y_BF16_RTOL
    return y_gpu, ref["y"]


@pytest.mark.parametrize("mode,container,a_bits", [("folded", 0, 4), ("folded", 1, 4), ("plain", 0, 3), ("double", 1, 4)])
def test_qlinear_small_configuration(env, oracle, mode, container, a_bits):
    """X [256,256] with 4 outlier channels, W [256,256], Hadamard block 256, per-token INT4 / INT3, bf16 output."""
    torch, hq = env
    cfg = inputs.config_linear_small(0)
    y_gpu, y_ref = run_linear(torch, hq, oracle, cfg["x"], cfg["w"], None, a_bits, 256, mode, container)
    if mode != "plain":        # without the weight-side transform the layer is not meant to reproduce X W
        assert rms_rel(y_gpu, y_ref) <= Y_BF16_RTOL


@pytest.mark.parametrize("which", ["qkv", "ff2"])
def test_qlinear_full_size_sampled_rows(env, oracle, which):
    """A transformer-block linear at the benchmark's size (32768 tokens), checked on sampled rows."""
    torch, hq = env
    cfg = inputs.config_transformer_linear(which)
    rows = np.sort(np.random.default_rng(1).choice(cfg["M"], size=64, replace=False))
    rows[0], rows[-1] = 0, cfg["M"] - 1
    run_linear(torch, hq, oracle, cfg["x"], cfg["w"], cfg["bias"], 4, cfg["had_block"], "folded", 0, rows_checked=rows)


@pytest.mark.parametrize("K,N", [(1152, 3456), (4608, 1152)])
def test_qlinear_block_diagonal_128(env, oracle, K, N):
    """Linears of a width-1152 transformer: 9 (or 36) Hadamard blocks of 128 channels per token, ragged row count."""
    torch, hq = env
    M = 700
    x = inputs.activations((M, K), dist="student_t3", outlier_count=max(1, K // 200), outlier_scale=30.0, seed=K)
    w = inputs.weights((N, K), seed=N)
    b = inputs.bias(N, seed=3)
    rows = np.sort(np.random.default_rng(2).choice(M, size=96, replace=False))
    run_linear(torch, hq, oracle, x, w, b, 4, 128, "folded", 0, rows_checked=rows)


@pytest.mark.parametrize("a_bits,static", [(4, False), (3, False), (4, True)])
def test_qconv_small_configuration(env, oracle, a_bits, static):
    """NHWC [8,32,32,256] x [256,3,3,256], stride 1, pad 1, Hadamard over the input channels, per-pixel INT4 / INT3
    (each tap rescaled by the scale of the pixel it read) or one static scale; bf16 output."""
    torch, hq = env
    cfg = inputs.config_conv_small(0)
    x, w, b = cfg["x"], cfg["w"], cfg["bias"]
    Nb, H, W, C = x.shape
    Cout = w.shape[0]
    pw = hq.hq_weight_prepare(w, 4, 256, hq.HQ_W_FOLDED, hq.HQ_CODES_NIBBLE).to_device()
    y = torch.zeros((Nb, H, W, Cout), dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros((hq.hq_workspace_size(Nb * H * W, C, hq.HQ_CODES_NIBBLE),), dtype=torch.uint8, device="cuda")
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    s0 = 0.8 if static else None
    ss = torch.tensor([s0], dtype=torch.float32, device="cuda") if static else None
    hq.hq_qconv(torch.from_numpy(x).cuda(), pw, 3, 3, 1, 1, torch.from_numpy(b).cuda(), a_bits, y, ws, static_scale=ss,
                dev_status=status)
    torch.cuda.synchronize()
    hq.hq_check_status(status)
    ref = oracle.qconv(x, w, b, a_bits=a_bits, w_bits=4, had_block=256, stride=1, pad=1, weight_mode="folded",
                       static_scale=s0)
    q_gpu, s_gpu = _codes_from_ws(hq, ws, Nb * H * W, C, hq.HQ_CODES_NIBBLE)
    v = ref["v"].reshape(-1, C)
    if static:
        v = np.clip(v, oracle.qmin(a_bits) - 0.25, oracle.qmax(a_bits) + 0.25)
        assert s_gpu[0] == np.float32(s0)
    else:
        assert np.allclose(s_gpu, ref["s_a"], rtol=SCALE_RTOL, atol=0)
    check_codes(q_gpu, ref["q"].reshape(-1, C), v, "fused conv")
    B = weight_integers(oracle, pw, w, 4, 256, "folded").reshape(Cout, 3, 3, C)
    qg = q_gpu.reshape(Nb, H, W, C)
    if static:
        y_own = oracle.dequant(oracle.conv2d_int(qg, B, 1, 1), np.array([s0], np.float32), pw.s_w, b, pw.alpha)
    else:
        y_own = oracle.conv2d_dequant_perpixel(qg, s_gpu, B, 1, 1, pw.s_w, b, pw.alpha)
    assert rel_err(y.float().cpu().numpy(), y_own) <= Y_BF16_RTOL
    assert rms_rel(y.float().cpu().numpy(), ref["y"]) <= Y_BF16_RTOL


@pytest.mark.parametrize("M,K,N,n,rpg,container", [(512, 1152, 384, 128, 256, 1), (320, 512, 200, 512, 32, 0)])
def test_ln_qlinear_layer(env, oracle, M, K, N, n, rpg, container):
    """LayerNorm + per-sample affine -> transform -> quantize -> integer product -> rescale in one call: the output
    equals the oracle's rescale of the integer product of the codes and scales the call left in its workspace, and the
    whole layer follows the oracle chain (normalise, quantize, multiply) to the layers' end-to-end bound."""
    torch, hq = env
    rng = np.random.default_rng(M + K)
    x = inputs.activations((M, K), outlier_count=max(1, K // 100), outlier_scale=8.0, seed=K) + np.float32(0.3)
    groups = (M + rpg - 1) // rpg
    lw = (1.0 + 0.2 * rng.standard_normal((groups, K))).astype(np.float32)
    lb = (0.3 * rng.standard_normal((groups, K))).astype(np.float32)
    w, b = inputs.weights((N, K), seed=N), inputs.bias(N, seed=N)
    pw = hq.hq_weight_prepare(w, 4, n, hq.HQ_W_FOLDED, container).to_device()
    y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros((hq.hq_workspace_size(M, K, container),), dtype=torch.uint8, device="cuda")
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    hq.hq_ln_qlinear(torch.from_numpy(x).cuda(), torch.from_numpy(lw).cuda(), torch.from_numpy(lb).cuda(), rpg, 1e-6, pw,
                     torch.from_numpy(b).cuda(), 4, y, ws, dev_status=status)
    torch.cuda.synchronize()
    hq.hq_check_status(status)
    q_gpu, s_gpu = _codes_from_ws(hq, ws, M, K, container)
    B = weight_integers(oracle, pw, w, 4, n, "folded")
    y_own = oracle.dequant(oracle.gemm_int(q_gpu, B), s_gpu, pw.s_w, b, pw.alpha)
    y_gpu = y.float().cpu().numpy()
    assert rel_err(y_gpu, y_own) <= Y_BF16_RTOL
    xn = oracle.layernorm_affine(x, lw, lb, rows_per_group=rpg, eps=1e-6)
    ref = oracle.qlinear(xn.astype(np.float32), w, b, a_bits=4, w_bits=4, had_block=n, weight_mode="folded")
    assert rms_rel(y_gpu, ref["y"]) <= 1e-2


@pytest.mark.parametrize("container,static", [(1, True), (0, False)])
def test_gn_silu_qconv_layer(env, oracle, container, static):
    """GroupNorm(32) + SiLU -> transform -> quantize -> integer 3x3 convolution -> rescale in one call, with one static
    scale or per-pixel scales: the output equals the oracle's rescale of the integer convolution of the codes and scales
    the call left in its workspace, and the whole layer follows the oracle chain to the layers' end-to-end bound."""
    torch, hq = env
    rng = np.random.default_rng(7)
    Nb, H, W, C, Cout, G = 2, 16, 16, 256, 128, 32
    x = inputs.activations((Nb, H, W, C), outlier_count=3, outlier_scale=8.0, seed=11) + np.float32(0.5)
    gamma = (1.0 + 0.2 * rng.standard_normal(C)).astype(np.float32)
    beta = (0.1 * rng.standard_normal(C)).astype(np.float32)
    w, b = inputs.weights((Cout, 3, 3, C), seed=5), inputs.bias(Cout, seed=5)
    pw = hq.hq_weight_prepare(w, 4, 256, hq.HQ_W_FOLDED, container).to_device()
    y = torch.zeros((Nb, H, W, Cout), dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros((hq.hq_workspace_size(Nb * H * W, C, container),), dtype=torch.uint8, device="cuda")
    scratch = torch.zeros((Nb * G * 24,), dtype=torch.uint8, device="cuda")
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    xn = oracle.groupnorm_silu(x, G, gamma, beta, 1e-5).astype(np.float32)
    s0 = float(np.float32(np.abs(oracle.transform(xn.reshape(-1, C), 256)).max() / 7.0)) if static else None
    ss = torch.tensor([s0], dtype=torch.float32, device="cuda") if static else None
    hq.hq_gn_silu_qconv(torch.from_numpy(x).cuda(), G, torch.from_numpy(gamma).cuda(), torch.from_numpy(beta).cuda(), 1e-5, pw,
                        3, 3, 1, 1, torch.from_numpy(b).cuda(), 4, y, ws, scratch, static_scale=ss, dev_status=status)
    torch.cuda.synchronize()
    hq.hq_check_status(status)
    q_gpu, s_gpu = _codes_from_ws(hq, ws, Nb * H * W, C, container)
    B = weight_integers(oracle, pw, w, 4, 256, "folded").reshape(Cout, 3, 3, C)
    qg = q_gpu.reshape(Nb, H, W, C)
    if static:
        y_own = oracle.dequant(oracle.conv2d_int(qg, B, 1, 1), np.array([s0], np.float32), pw.s_w, b, pw.alpha)
    else:
        y_own = oracle.conv2d_dequant_perpixel(qg, s_gpu, B, 1, 1, pw.s_w, b, pw.alpha)
    y_gpu = y.float().cpu().numpy()
    assert rel_err(y_gpu, y_own) <= Y_BF16_RTOL
    ref = oracle.qconv(xn, w, b, a_bits=4, w_bits=4, had_block=256, stride=1, pad=1, weight_mode="folded", static_scale=s0)
    assert rms_rel(y_gpu, ref["y"]) <= 1e-2


def test_qconv_benchmark_configuration_sampled_images(env, oracle):
    """The 3x3 convolution as the benchmark step runs it: batch 32 (32768 pixels), one code per byte, one static
    activation scale calibrated as the largest per-pixel scale, bf16 output.  Three sampled images (a convolution
    with zero padding never looks across images) go through the whole oracle layer."""
    torch, hq = env
    cfg = inputs.config_conv_small(0, batch=32)
    x, w, b = cfg["x"], cfg["w"], cfg["bias"]
    Nb, H, W, C = x.shape
    Cout = w.shape[0]
    cont = hq.HQ_CODES_INT8
    pw = hq.hq_weight_prepare(w, 4, 256, hq.HQ_W_FOLDED, cont).to_device()
    xd = torch.from_numpy(x).cuda()
    codes = torch.empty((Nb * H * W, C), dtype=torch.uint8, device="cuda")
    sc = torch.empty((Nb * H * W,), dtype=torch.float32, device="cuda")
    hq.hq_hadamard_quant(xd.view(-1, C), 256, 4, codes, cont, scales=sc)
    static = sc.max().reshape(1).contiguous()
    s0 = float(static.cpu()[0])
    y = torch.zeros((Nb, H, W, Cout), dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros((hq.hq_workspace_size(Nb * H * W, C, cont),), dtype=torch.uint8, device="cuda")
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    hq.hq_qconv(xd, pw, 3, 3, 1, 1, torch.from_numpy(b).cuda(), 4, y, ws, static_scale=static, dev_status=status)
    torch.cuda.synchronize()
    hq.hq_check_status(status)
    q_all, s_gpu = _codes_from_ws(hq, ws, Nb * H * W, C, cont)
    assert s_gpu[0] == np.float32(s0)
    q_all = q_all.reshape(Nb, H, W, C)
    imgs = [0, 13, Nb - 1]
    ref = oracle.qconv(x[imgs], w, b, a_bits=4, w_bits=4, had_block=256, stride=1, pad=1, weight_mode="folded",
                       static_scale=s0)
    # the calibrated scale equals the largest per-pixel scale of the oracle's dynamic quantizer on the whole tensor
    s_dyn = oracle.quantize(oracle.transform(x.reshape(-1, C), 256), 4)[1]
    assert np.isclose(s0, s_dyn.max(), rtol=SCALE_RTOL, atol=0)
    check_codes(q_all[imgs].reshape(-1, C), ref["q"].reshape(-1, C), ref["v"].reshape(-1, C), "bench conv, static scale")
    B = weight_integers(oracle, pw, w, 4, 256, "folded").reshape(Cout, 3, 3, C)
    y_own = oracle.dequant(oracle.conv2d_int(q_all[imgs], B, 1, 1), np.array([s0], np.float32), pw.s_w, b, pw.alpha)
    y_gpu = y.float().cpu().numpy()[imgs]
    assert rel_err(y_gpu, y_own) <= Y_BF16_RTOL
    assert rms_rel(y_gpu, ref["y"]) <= Y_BF16_RTOL


@pytest.mark.parametrize("M,K,N,n", [(1000, 512, 384, 512), (300, 1024, 200, 256)])
def test_qlinear_w8a8(env, oracle, M, K, N, n):
    """The fused layer at W8A8: 8-bit codes in the one-byte container, 8-bit Double-Hadamard weights Q(H^T W)
    (one limb), online transform in front."""
    torch, hq = env
    x = inputs.activations((M, K), outlier_count=max(1, K // 100), outlier_scale=20.0, seed=M + K)
    w, b = inputs.weights((N, K), seed=N), inputs.bias(N, seed=N)
    cont = hq.HQ_CODES_INT8
    pw = hq.hq_weight_prepare(w, 8, n, hq.HQ_W_DOUBLE, cont).to_device()
    y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros((hq.hq_workspace_size(M, K, cont),), dtype=torch.uint8, device="cuda")
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    hq.hq_qlinear(torch.from_numpy(x).cuda(), pw, torch.from_numpy(b).cuda(), 8, y, ws, dev_status=status)
    torch.cuda.synchronize()
    hq.hq_check_status(status)
    q_gpu, s_gpu = _codes_from_ws(hq, ws, M, K, cont)
    ref = oracle.qlinear(x, w, b, a_bits=8, w_bits=8, had_block=n, weight_mode="double")
    assert np.allclose(s_gpu, ref["s_a"], rtol=SCALE_RTOL, atol=0)
    check_codes(q_gpu, ref["q"], ref["v"], "fused linear W8A8")
    B = weight_integers(oracle, pw, w, 8, n, "double")
    y_own = oracle.dequant(oracle.gemm_int(q_gpu, B), s_gpu, pw.s_w, b, pw.alpha)
    y_gpu = y.float().cpu().numpy()
    assert rel_err(y_gpu, y_own) <= Y_BF16_RTOL
    # with 8 bits on both sides the Double-Hadamard layer is close to the float product
    xw = x.astype(np.float64) @ w.astype(np.float64).T + b
    assert rms_rel(y_gpu, xw) <= 2e-2


FUSED_CASES = [
    # M, K, N, had_block, mode, a_bits, dtype, static
    (256, 256, 256, 256, "folded", 4, "f32", False),      # the small linear configuration
    (1000, 512, 384, 512, "folded", 4, "f32", False),     # ragged rows, three column tiles
    (777, 512, 200, 256, "folded", 4, "bf16", False),     # two Hadamard blocks per row, ragged columns
    (300, 128, 72, 128, "plain", 3, "f32", False),        # one K block, one weight limb
    (2500, 256, 520, 64, "double", 4, "bf16", False),     # four blocks per row; several row tiles per CTA range
    (640, 512, 256, 32, "folded", 4, "f32", True),        # static scale, 16 blocks per row (one lane each)
    (40000, 512, 640, 512, "folded", 4, "f32", False),    # more tiles than CTAs: ranges that start inside a row tile
]


@pytest.mark.parametrize("M,K,N,n,mode,a_bits,dt,static", FUSED_CASES)
def test_qlinear_fused_single_kernel(env, oracle, M, K, N, n, mode, a_bits, dt, static):
    """The one-kernel fused layer: its output against the oracle's rescale of the integer product of the ORACLE's codes
    (the codes never leave the chip), allowing for the few codes on rounding ties; and bit-for-bit against the two-kernel
    hq_qlinear, which runs the same arithmetic."""
    torch, hq = env
    x = inputs.activations((M, K), dist="student_t3", outlier_count=max(1, K // 100), outlier_scale=30.0, seed=M + K)
    w, b = inputs.weights((N, K), seed=N), inputs.bias(N, seed=N)
    xt = torch.from_numpy(x).cuda()
    if dt == "bf16":
        xt = xt.to(torch.bfloat16)
        x = xt.float().cpu().numpy()
    cont = hq.HQ_CODES_INT8
    pw = hq.hq_weight_prepare(w, 4, n, hq.WEIGHT_MODES[mode], cont).to_device()
    bd = torch.from_numpy(b).cuda()
    s0 = None
    ss = None
    if static:
        s0 = float(np.float32(np.abs(oracle.transform(x, n)).max() / oracle.qmax(a_bits) / 3.0))
        ss = torch.tensor([s0], dtype=torch.float32, device="cuda")
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    y = torch.full((M, N), 9.0, dtype=torch.bfloat16, device="cuda")
    hq.hq_qlinear_fused(xt, pw, bd, a_bits, y, static_scale=ss, dev_status=status)
    y2 = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros((hq.hq_workspace_size(M, K, cont),), dtype=torch.uint8, device="cuda")
    hq.hq_qlinear(xt, pw, bd, a_bits, y2, ws, static_scale=ss, dev_status=status)
    torch.cuda.synchronize()
    hq.hq_check_status(status)
    assert torch.equal(y, y2), "one-kernel and two-kernel layers differ"
    idx = np.arange(M) if M <= 3000 else np.sort(np.random.default_rng(5).choice(M, size=192, replace=False))
    ref = oracle.qlinear(x[idx], w, b, a_bits=a_bits, w_bits=4, had_block=n, weight_mode=mode, static_scale=s0)
    q_gpu, s_gpu = _codes_from_ws(hq, ws, M, K, cont)            # the two-kernel path's codes: the same arithmetic
    v = ref["v"] if not static else np.clip(ref["v"], oracle.qmin(a_bits) - 0.25, oracle.qmax(a_bits) + 0.25)
    check_codes(q_gpu[idx], ref["q"], v, "fused one-kernel linear")
    B = weight_integers(oracle, pw, w, 4, n, mode)
    sa = s_gpu[idx] if not static else np.array([s0], np.float32)
    y_own = oracle.dequant(oracle.gemm_int(q_gpu[idx], B), sa, pw.s_w, b, pw.alpha)
    assert rel_err(y.float().cpu().numpy()[idx], y_own) <= Y_BF16_RTOL


def test_qlinear_fused_refuses_other_shapes(env):
    torch, hq = env
    x = torch.zeros((64, 1024), device="cuda")
    pw = hq.hq_weight_prepare(inputs.weights((128, 1024), seed=0), 4, 1024, hq.HQ_W_FOLDED, hq.HQ_CODES_INT8).to_device()
    with pytest.raises(hq.HqError) as e:
        hq.hq_qlinear_fused(x, pw, None, 4, torch.zeros((64, 128), dtype=torch.bfloat16, device="cuda"))
    assert e.value.status == 3
