"""GPU parity: integer GEMM / convolution with the rescale epilogue (hq_qgemm, hq_qconv2d) against the CPU oracle.
Integer accumulators must be bit-exact; float outputs within the stated tolerances."""
import numpy as np
import pytest

from paper_2512_05746_b200 import inputs
import hq_testutil as hqt
from hq_testutil import Y_BF16_RTOL, Y_F32_RTOL, pack_nibbles_np, rel_err, weight_integers

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2512_05746_b200 import binding as hq
    return torch, hq


def to_container(torch, hq, q_np, container):
    """int8 codes [..., K] -> device uint8 tensor in the requested container (rows densely packed)."""
    if container == hq.HQ_CODES_NIBBLE:
        b = pack_nibbles_np(q_np)
    else:
        b = q_np.view(np.uint8)
    return torch.from_numpy(np.ascontiguousarray(b)).cuda()


def gemm_case(torch, hq, oracle, M, K, N, a_bits, w_bits, had_block, mode, container, seed=0, with_bias=True):
    q = inputs.codes((M, K), a_bits, seed=seed)
    w = inputs.weights((N, K), seed=seed)
    pw = hq.hq_weight_prepare(w, w_bits, had_block, hq.WEIGHT_MODES[mode], container).to_device()
    B_ref = weight_integers(oracle, pw, w, w_bits, had_block, mode)
    s_a = inputs.positive_scales(M, seed=seed)
    b = inputs.bias(N, seed=seed) if with_bias else None
    a_dev = to_container(torch, hq, q, container)
    acc = torch.full((M, N), 12345, dtype=torch.int32, device="cuda")
    y16 = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    y32 = torch.zeros((M, N), dtype=torch.float32, device="cuda")
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    sa_dev = torch.from_numpy(s_a).cuda()
    b_dev = None if b is None else torch.from_numpy(b).cuda()
    hq.hq_qgemm(a_dev, container, a_bits, K, pw, scale_a=sa_dev, bias=b_dev, alpha=pw.alpha, acc_out=acc, y=y16,
                dev_status=status)
    hq.hq_qgemm(a_dev, container, a_bits, K, pw, scale_a=sa_dev, bias=b_dev, alpha=pw.alpha, y=y32, dev_status=status)
    # bf16 output alone: the launch configuration the layers and the benchmark use (bulk-store epilogue)
    y16_only = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    hq.hq_qgemm(a_dev, container, a_bits, K, pw, scale_a=sa_dev, bias=b_dev, alpha=pw.alpha, y=y16_only, dev_status=status)
    torch.cuda.synchronize()
    hq.hq_check_status(status)
    acc_ref = oracle.gemm_int(q, B_ref)
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), acc_ref), "int32 accumulators differ"
    y_ref = oracle.dequant(acc_ref, s_a, pw.s_w, b, pw.alpha)
    assert rel_err(y32.cpu().numpy(), y_ref) <= Y_F32_RTOL
    assert rel_err(y16.float().cpu().numpy(), y_ref) <= Y_BF16_RTOL
    assert rel_err(y16_only.float().cpu().numpy(), y_ref) <= Y_BF16_RTOL
    return pw


GEMM_CASES = [
    # M, K, N, a_bits, w_bits, had_block, mode, container
    (256, 256, 256, 4, 4, 256, "plain", 1),
    (256, 256, 256, 4, 4, 256, "folded", 1),
    (256, 256, 256, 4, 4, 256, "folded", 0),
    (256, 256, 256, 4, 4, 256, "plain", 0),
    (1000, 512, 384, 4, 4, 512, "folded", 1),     # ragged M, N = 1.5 tiles
    (1000, 512, 384, 3, 4, 512, "plain", 0),
    (130, 2048, 512, 4, 4, 2048, "folded", 0),
    (513, 768, 200, 4, 4, 256, "plain", 1),       # N not a multiple of 8, K = 6 blocks
    (300, 320, 72, 8, 8, 64, "plain", 1),         # W8A8, K tail (320 = 2.5 blocks)
    (97, 1024, 640, 4, 4, 16, "folded", 0),       # folded weights that still fit one limb
    (4096, 1024, 1280, 4, 4, 1024, "folded", 0),  # several tiles per CTA
    (64, 4096, 256, 4, 4, 4096, "folded", 1),
    (1, 256, 256, 4, 4, 256, "double", 0),
    # one code per byte with short reductions / one resident limb: the fragment-layout epilogue and its second issuer
    (1000, 256, 200, 4, 4, 256, "folded", 1),     # two limbs, K = 2 blocks, ragged M, N = 1.56 tiles
    (777, 512, 328, 4, 4, 512, "plain", 1),       # one limb, resident weights, several weight tiles per CTA range
    (130, 128, 72, 4, 4, 128, "folded", 1),       # K = 1 block
    (40000, 256, 384, 4, 4, 256, "double", 1),    # many tiles per CTA, weight tile changes inside a CTA's range
    (5000, 1152, 136, 4, 4, 128, "plain", 1),     # one limb with streamed weights (row-per-lane epilogue)
]


@pytest.mark.parametrize("M,K,N,a_bits,w_bits,had_block,mode,container", GEMM_CASES)
def test_qgemm_matches_oracle(env, oracle, M, K, N, a_bits, w_bits, had_block, mode, container):
    torch, hq = env
    gemm_case(torch, hq, oracle, M, K, N, a_bits, w_bits, had_block, mode, container, seed=M + K + N)


@pytest.mark.parametrize("seed", range(24))
def test_qgemm_random_shapes(env, oracle, seed):
    """Seeded random draws over reduction length, Hadamard block, ragged M / N, weight mode and container: every launch
    form of gemm_case (accumulators + bf16, fp32, bf16 alone) against the oracle."""
    torch, hq = env
    rng = np.random.default_rng(1000 + seed)
    K = int(rng.choice([128, 256, 384, 512, 640, 1024, 1152]))
    hb = int(rng.choice([h for h in (32, 128, 256, 512) if K % h == 0]))
    N = int(rng.choice([8, 72, 128, 136, 200, 256, 384, 520]))
    M = int(rng.choice([1, 127, 128, 129, 1000, 2500]))
    mode = ["folded", "plain", "double"][int(rng.integers(3))]
    container = int(rng.integers(2))
    gemm_case(torch, hq, oracle, M, K, N, 4, 4, hb, mode, container, seed=seed, with_bias=bool(rng.integers(2)))


def test_qgemm_extreme_magnitudes(env, oracle):
    """Largest accumulators the path can produce: (a) folded weights with a constant channel (B = -8*n at one index,
    so the high limb is at its extreme) against sign-matched extreme codes; (b) W8A8 with every product at 127*128."""
    torch, hq = env
    M, K, N = 128, 2048, 128
    w = inputs.weights((N, K), seed=3)
    w[0, :] = -1.0                                                  # W_int = -7 everywhere -> B[0][0] = -7*1024
    for container in (0, 1):
        pw = hq.hq_weight_prepare(w, 4, 1024, hq.HQ_W_FOLDED, container).to_device()
        B = weight_integers(oracle, pw, w, 4, 1024, "folded")
        assert np.abs(B).max() >= 7 * 1024
        q = np.where(B[1] > 0, -8, 7).astype(np.int8)[None, :].repeat(M, axis=0)    # |acc| of channel 1 = sum |q||B|
        q[1::2] = -8
        acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
        hq.hq_qgemm(to_container(torch, hq, q, container), container, 4, K, pw, acc_out=acc)
        torch.cuda.synchronize()
        ref = oracle.gemm_int(q, B)
        assert np.abs(ref).max() > 2 ** 19
        assert np.array_equal(acc.cpu().numpy().astype(np.int64), ref)
    K8 = 8192
    w8 = -np.ones((N, K8), np.float32)
    pw = hq.hq_weight_prepare(w8, 8, 1, hq.HQ_W_PLAIN, hq.HQ_CODES_INT8).to_device()
    q8 = np.full((M, K8), -128, np.int8)
    acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    hq.hq_qgemm(to_container(torch, hq, q8, 1), 1, 8, K8, pw, acc_out=acc)
    torch.cuda.synchronize()
    assert int(acc.min()) == int(acc.max()) == 127 * 128 * K8


def test_qgemm_scalar_scale_and_determinism(env, oracle):
    torch, hq = env
    M, K, N = 700, 512, 512
    q = inputs.codes((M, K), 4, seed=5)
    w = inputs.weights((N, K), seed=5)
    pw = hq.hq_weight_prepare(w, 4, 512, hq.HQ_W_FOLDED, hq.HQ_CODES_NIBBLE).to_device()
    a = to_container(torch, hq, q, hq.HQ_CODES_NIBBLE)
    s = torch.tensor([0.037], device="cuda")
    outs = []
    for _ in range(3):
        y = torch.zeros((M, N), dtype=torch.float32, device="cuda")
        hq.hq_qgemm(a, hq.HQ_CODES_NIBBLE, 4, K, pw, scale_a=s, alpha=pw.alpha, y=y)
        outs.append(y.cpu().numpy())
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], outs[2])
    y_ref = oracle.dequant(oracle.gemm_int(q, weight_integers(oracle, pw, w, 4, 512, "folded")), np.array([0.037], np.float32), pw.s_w,
                           None, pw.alpha)
    assert rel_err(outs[0], y_ref) <= Y_F32_RTOL


CONV_CASES = [
    # Nb, H, W, C, Cout, R, pad, a_bits, mode, container
    (8, 32, 32, 256, 256, 3, 1, 4, "folded", 0),     # the small conv configuration
    (8, 32, 32, 256, 256, 3, 1, 3, "folded", 1),
    (2, 16, 16, 128, 384, 3, 1, 4, "plain", 1),
    (3, 8, 8, 256, 128, 3, 1, 4, "folded", 0),       # tiles span two images
    (2, 64, 64, 128, 128, 3, 1, 4, "plain", 0),      # two output rows per tile
    (1, 20, 12, 128, 64, 3, 1, 4, "plain", 1),       # width that does not divide 128
    (2, 16, 16, 256, 256, 1, 0, 4, "folded", 0),     # 1x1
    (1, 10, 10, 160, 96, 3, 0, 4, "plain", 1),       # no padding, channel tail (160 = 1.25 blocks)
    (4, 16, 16, 256, 320, 1, 0, 4, "folded", 1),     # 1x1, K = 2 blocks: fragment-layout epilogue on a convolution
    (5, 8, 8, 384, 200, 1, 0, 4, "plain", 1),        # 1x1, one limb, tiles span two images, last tile partly empty
]


@pytest.mark.parametrize("Nb,H,W,C,Cout,R,pad,a_bits,mode,container", CONV_CASES)
def test_qconv2d_matches_oracle(env, oracle, Nb, H, W, C, Cout, R, pad, a_bits, mode, container):
    torch, hq = env
    hb = 128 if C % 128 == 0 else 32
    q = inputs.codes((Nb, H, W, C), a_bits, seed=H + W + C)
    w = inputs.weights((Cout, R, R, C), seed=C + Cout)
    pw = hq.hq_weight_prepare(w, 4, hb, hq.WEIGHT_MODES[mode], container).to_device()
    B_ref = weight_integers(oracle, pw, w, 4, hb, mode).reshape(Cout, R, R, C)
    b = inputs.bias(Cout, seed=1)
    Ho, Wo = H + 2 * pad - R + 1, W + 2 * pad - R + 1
    acc = torch.full((Nb, Ho, Wo, Cout), 777, dtype=torch.int32, device="cuda")
    y = torch.zeros((Nb, Ho, Wo, Cout), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    s_a = torch.tensor([0.05], device="cuda")
    hq.hq_qconv2d(to_container(torch, hq, q, container), container, a_bits, Nb, H, W, C, pw, R, R, 1, pad, scale_a=s_a,
                  bias=torch.from_numpy(b).cuda(), alpha=pw.alpha, acc_out=acc, y=y, dev_status=status)
    torch.cuda.synchronize()
    hq.hq_check_status(status)
    acc_ref = oracle.conv2d_int(q, B_ref, 1, pad)
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), acc_ref)
    y_ref = oracle.dequant(acc_ref, np.array([0.05], np.float32), pw.s_w, b, pw.alpha)
    assert rel_err(y.float().cpu().numpy(), y_ref) <= Y_BF16_RTOL
    # bf16 output alone: the launch configuration the layers and the benchmark use
    y2 = torch.zeros((Nb, Ho, Wo, Cout), dtype=torch.bfloat16, device="cuda")
    hq.hq_qconv2d(to_container(torch, hq, q, container), container, a_bits, Nb, H, W, C, pw, R, R, 1, pad, scale_a=s_a,
                  bias=torch.from_numpy(b).cuda(), alpha=pw.alpha, y=y2, dev_status=status)
    torch.cuda.synchronize()
    hq.hq_check_status(status)
    assert rel_err(y2.float().cpu().numpy(), y_ref) <= Y_BF16_RTOL


STRIDE2_CASES = [
    # Nb, H, W, C, Cout, R, pad, mode, container
    (2, 32, 32, 256, 256, 3, 1, "folded", 0),        # the down-sampling convolution of a UNet level
    (3, 16, 16, 128, 192, 3, 1, "plain", 1),
    (1, 17, 13, 128, 64, 3, 1, "plain", 0),          # odd sizes: the last window hangs over the padding
    (2, 16, 16, 256, 128, 1, 0, "folded", 1),        # 1x1 stride 2 (a strided skip projection)
]


@pytest.mark.parametrize("Nb,H,W,C,Cout,R,pad,mode,container", STRIDE2_CASES)
def test_qconv2d_stride2_matches_oracle(env, oracle, Nb, H, W, C, Cout, R, pad, mode, container):
    torch, hq = env
    q = inputs.codes((Nb, H, W, C), 4, seed=H + C)
    w = inputs.weights((Cout, R, R, C), seed=Cout)
    pw = hq.hq_weight_prepare(w, 4, 128, hq.WEIGHT_MODES[mode], container).to_device()
    B_ref = weight_integers(oracle, pw, w, 4, 128, mode).reshape(Cout, R, R, C)
    Ho, Wo = (H + 2 * pad - R) // 2 + 1, (W + 2 * pad - R) // 2 + 1
    acc = torch.full((Nb, Ho, Wo, Cout), 777, dtype=torch.int32, device="cuda")
    y = torch.zeros((Nb, Ho, Wo, Cout), dtype=torch.float32, device="cuda")
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    s_a = torch.tensor([0.03], device="cuda")
    hq.hq_qconv2d(to_container(torch, hq, q, container), container, 4, Nb, H, W, C, pw, R, R, 2, pad, scale_a=s_a,
                  alpha=pw.alpha, acc_out=acc, y=y, dev_status=status)
    torch.cuda.synchronize()
    hq.hq_check_status(status)
    acc_ref = oracle.conv2d_int(q, B_ref, 2, pad)
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), acc_ref)
    y_ref = oracle.dequant(acc_ref, np.array([0.03], np.float32), pw.s_w, None, pw.alpha)
    assert rel_err(y.cpu().numpy(), y_ref) <= Y_F32_RTOL


PERPIXEL_CASES = [
    # Nb, H, W, C, Cout, stride, a_bits, mode, container, out dtype
    (8, 32, 32, 256, 256, 1, 4, "folded", 0, "bf16"),    # the small conv configuration with its per-pixel scales
    (8, 32, 32, 256, 256, 1, 3, "folded", 0, "bf16"),    # W4A3
    (2, 16, 16, 128, 200, 1, 4, "folded", 1, "f32"),     # ragged Cout
    (2, 16, 16, 128, 320, 1, 4, "plain", 1, "f32"),      # one weight limb: two column passes
    (1, 20, 12, 128, 64, 1, 4, "plain", 0, "bf16"),      # ragged tiles
    (2, 32, 32, 128, 128, 2, 4, "folded", 0, "f32"),     # stride 2
]


@pytest.mark.parametrize("Nb,H,W,C,Cout,stride,a_bits,mode,container,odt", PERPIXEL_CASES)
def test_qconv2d_per_pixel_scales(env, oracle, Nb, H, W, C, Cout, stride, a_bits, mode, container, odt):
    """One activation scale per input pixel under a 3x3 window: every tap is rescaled by the scale of the pixel it
    read.  The integer sums over the whole window are requested in the same call and must still be bit-exact."""
    torch, hq = env
    q = inputs.codes((Nb, H, W, C), a_bits, seed=H + W + C + a_bits)
    w = inputs.weights((Cout, 3, 3, C), seed=Cout)
    pw = hq.hq_weight_prepare(w, 4, 128, hq.WEIGHT_MODES[mode], container).to_device()
    B_ref = weight_integers(oracle, pw, w, 4, 128, mode).reshape(Cout, 3, 3, C)
    b = inputs.bias(Cout, seed=3)
    s_a = inputs.positive_scales(Nb * H * W, seed=7)
    Ho, Wo = (H + 2 - 3) // stride + 1, (W + 2 - 3) // stride + 1
    acc = torch.full((Nb, Ho, Wo, Cout), 777, dtype=torch.int32, device="cuda")
    y = torch.zeros((Nb, Ho, Wo, Cout), dtype=torch.bfloat16 if odt == "bf16" else torch.float32, device="cuda")
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    hq.hq_qconv2d(to_container(torch, hq, q, container), container, a_bits, Nb, H, W, C, pw, 3, 3, stride, 1,
                  scale_a=torch.from_numpy(s_a).cuda(), bias=torch.from_numpy(b).cuda(), alpha=pw.alpha, acc_out=acc,
                  y=y, dev_status=status)
    torch.cuda.synchronize()
    hq.hq_check_status(status)
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), oracle.conv2d_int(q, B_ref, stride, 1))
    y_ref = oracle.conv2d_dequant_perpixel(q, s_a, B_ref, stride, 1, pw.s_w, b, pw.alpha)
    assert rel_err(y.float().cpu().numpy(), y_ref) <= (Y_BF16_RTOL if odt == "bf16" else Y_F32_RTOL)


def test_int8_tensor_pipe_probe_runs(env):
    torch, hq = env
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    hq.hq_mma_i8_probe(4, 64, dev_status=status)
    torch.cuda.synchronize()
    hq.hq_check_status(status)


def test_qgemm_sweep_corner_sampled(env, oracle):
    """The largest point of the shape sweep, 65536 x 4096 x 4096 with the folded two-limb weights of a 4096-point
    block: int32 accumulators of sampled rows and output channels (first and last of each axis included) against the
    oracle's integer product.  The codes are drawn on the device (seeded); the sampled rows are copied back."""
    torch, hq = env
    M, K, N = 65536, 4096, 4096
    gen = torch.Generator(device="cuda")
    gen.manual_seed(7)
    a = torch.randint(-8, 8, (M, K), generator=gen, device="cuda", dtype=torch.int8)
    w = inputs.weights((N, K), seed=4096)
    pw = hq.hq_weight_prepare(w, 4, K, hq.HQ_W_FOLDED, hq.HQ_CODES_INT8).to_device()
    assert pw.desc.limbs == 2
    acc = torch.empty((M, N), dtype=torch.int32, device="cuda")
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    hq.hq_qgemm(a.view(torch.uint8), hq.HQ_CODES_INT8, 4, K, pw, acc_out=acc, dev_status=status)
    torch.cuda.synchronize()
    hq.hq_check_status(status)
    rng = np.random.default_rng(3)
    rows = np.sort(np.concatenate(([0, 127, 128, M - 1], rng.choice(M, size=60, replace=False))))
    cols = np.sort(np.concatenate(([0, 127, 128, N - 1], rng.choice(N, size=60, replace=False))))
    w_int, _ = oracle.weight_quantize(w[cols], 4)
    B = oracle.weight_fold(w_int, K)                                  # exact integers, only the sampled channels
    assert np.array_equal(B, hqt.decode_blob(pw).reshape(N, K)[cols])
    ridx = torch.from_numpy(rows).cuda()
    q = a[ridx].cpu().numpy()
    ref = oracle.gemm_int(q, B)
    got = acc[ridx][:, torch.from_numpy(cols).cuda()].cpu().numpy().astype(np.int64)
    assert np.array_equal(got, ref)


PAIR_CASES = [
    # M, K, N, had_block, mode
    (512, 256, 256, 256, "folded"),
    (1000, 512, 384, 512, "folded"),      # ragged rows (3.9 pair tiles), three column tiles
    (777, 512, 328, 512, "plain"),        # one weight limb, ragged columns
    (300, 128, 72, 128, "folded"),        # one K block
    (40000, 256, 384, 256, "double"),     # more pair tiles than clusters; the weight tile changes inside a pair's range
    (40000, 512, 384, 512, "folded"),     # the same with four K blocks and two limbs: what the default dispatch sends to pairs
    (256, 384, 136, 128, "folded"),       # three K blocks
    # reductions beyond the resident weight tile: weights streamed through the pair's ring
    (1000, 1024, 384, 1024, "folded"),    # eight K blocks, ragged rows, three column tiles
    (4096, 2048, 512, 2048, "folded"),    # the shape of the step's FF2 at an eighth of its rows
    (777, 640, 328, 128, "plain"),        # five K blocks, one weight limb, ragged columns
    (38000, 768, 256, 256, "folded"),     # more pair tiles than clusters: tiles c, c + G, ... per pair
    (300, 1152, 72, 128, "double"),       # nine K blocks
]


@pytest.mark.parametrize("M,K,N,n,mode", PAIR_CASES)
def test_qgemm_on_sm_pairs_matches_oracle(env, oracle, M, K, N, n, mode):
    """The product on pairs of SMs (tcgen05.mma.cta_group::2, each CTA of a cluster holding half of the weight tile):
    bf16 output against the oracle's rescale of the oracle's integer product, and bit for bit against the one-CTA
    kernel."""
    torch, hq = env
    q = inputs.codes((M, K), 4, seed=M + N)
    w = inputs.weights((N, K), seed=N)
    pw = hq.hq_weight_prepare(w, 4, n, hq.WEIGHT_MODES[mode], hq.HQ_CODES_INT8).to_device()
    B = weight_integers(oracle, pw, w, 4, n, mode)
    s_a = inputs.positive_scales(M, seed=M)
    b = inputs.bias(N, seed=N)
    a_dev = to_container(torch, hq, q, hq.HQ_CODES_INT8)
    sa_dev, b_dev = torch.from_numpy(s_a).cuda(), torch.from_numpy(b).cuda()
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    y_one = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    y_pair = torch.full((M, N), 3.0, dtype=torch.bfloat16, device="cuda")
    before = hq.hq_set_pair_gemm(0)
    try:
        hq.hq_qgemm(a_dev, 1, 4, K, pw, scale_a=sa_dev, bias=b_dev, alpha=pw.alpha, y=y_one, dev_status=status)
        hq.hq_set_pair_gemm(1)
        hq.hq_qgemm(a_dev, 1, 4, K, pw, scale_a=sa_dev, bias=b_dev, alpha=pw.alpha, y=y_pair, dev_status=status)
        hq.hq_set_pair_gemm(2)                 # the default: whichever kernel the library picks for this shape
        y_def = torch.full((M, N), 5.0, dtype=torch.bfloat16, device="cuda")
        hq.hq_qgemm(a_dev, 1, 4, K, pw, scale_a=sa_dev, bias=b_dev, alpha=pw.alpha, y=y_def, dev_status=status)
        torch.cuda.synchronize()
    finally:
        hq.hq_set_pair_gemm(before)
    hq.hq_check_status(status)
    y_ref = oracle.dequant(oracle.gemm_int(q, B), s_a, pw.s_w, b, pw.alpha)
    assert rel_err(y_pair.float().cpu().numpy(), y_ref) <= Y_BF16_RTOL
    assert torch.equal(y_pair, y_one)
    assert torch.equal(y_def, y_one)


def test_paired_tensor_pipe_probe_runs(env):
    torch, hq = env
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    hq.hq_mma_i8_probe_pair(2, 64, dev_status=status)
    torch.cuda.synchronize()
    hq.hq_check_status(status)


PAIR_CONV_CASES = [
    # Nb, H, W, C, Cout, R, stride, pad, mode
    (8, 32, 32, 256, 256, 3, 1, 1, "folded"),      # the small conv configuration: 64 tiles of 128 pixels, two column tiles
    (3, 8, 8, 256, 128, 3, 1, 1, "folded"),        # tiles span two images; an odd number of tiles (the peer's last tile is empty)
    (2, 64, 64, 128, 128, 3, 1, 1, "plain"),       # two output rows per tile, one weight limb
    (2, 32, 32, 256, 256, 3, 2, 1, "folded"),      # the down-sampling convolution of a UNet level
    (4, 16, 16, 768, 320, 1, 1, 0, "folded"),      # 1x1 skip convolution with six K blocks, ragged columns
    (5, 16, 16, 384, 256, 3, 1, 1, "double"),      # 27 K blocks, five images of two tiles each
]


@pytest.mark.parametrize("Nb,H,W,C,Cout,R,stride,pad,mode", PAIR_CONV_CASES)
def test_qconv2d_on_sm_pairs_matches_oracle(env, oracle, Nb, H, W, C, Cout, R, stride, pad, mode):
    """The implicit-GEMM convolution on pairs of SMs (weights streamed, each CTA half of every weight K block): bf16 output
    against the oracle's rescale of the oracle's integer convolution, and bit for bit against the one-CTA kernel."""
    torch, hq = env
    hb = 128
    q = inputs.codes((Nb, H, W, C), 4, seed=H + C + Cout)
    w = inputs.weights((Cout, R, R, C), seed=C + Cout)
    pw = hq.hq_weight_prepare(w, 4, hb, hq.WEIGHT_MODES[mode], hq.HQ_CODES_INT8).to_device()
    B_ref = weight_integers(oracle, pw, w, 4, hb, mode).reshape(Cout, R, R, C)
    b = inputs.bias(Cout, seed=2)
    Ho, Wo = (H + 2 * pad - R) // stride + 1, (W + 2 * pad - R) // stride + 1
    a_dev = to_container(torch, hq, q, hq.HQ_CODES_INT8)
    # one static scale; the 1x1 convolution takes one scale per pixel instead (the skip projections of the UNet)
    sa_np = inputs.positive_scales(Nb * H * W, seed=H) if R == 1 else np.array([0.05], np.float32)
    s_a = torch.from_numpy(sa_np).cuda()
    b_dev = torch.from_numpy(b).cuda()
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    y_one = torch.zeros((Nb, Ho, Wo, Cout), dtype=torch.bfloat16, device="cuda")
    y_pair = torch.full((Nb, Ho, Wo, Cout), 3.0, dtype=torch.bfloat16, device="cuda")
    before = hq.hq_set_pair_gemm(0)
    try:
        hq.hq_qconv2d(a_dev, hq.HQ_CODES_INT8, 4, Nb, H, W, C, pw, R, R, stride, pad, scale_a=s_a, bias=b_dev, alpha=pw.alpha,
                      y=y_one, dev_status=status)
        hq.hq_set_pair_gemm(1)
        hq.hq_qconv2d(a_dev, hq.HQ_CODES_INT8, 4, Nb, H, W, C, pw, R, R, stride, pad, scale_a=s_a, bias=b_dev, alpha=pw.alpha,
                      y=y_pair, dev_status=status)
        torch.cuda.synchronize()
    finally:
        hq.hq_set_pair_gemm(before)
    hq.hq_check_status(status)
    acc_ref = oracle.conv2d_int(q, B_ref, stride, pad)
    y_ref = oracle.dequant(acc_ref.reshape(-1, Cout), sa_np, pw.s_w, b, pw.alpha).reshape(acc_ref.shape)
    assert rel_err(y_pair.float().cpu().numpy(), y_ref) <= Y_BF16_RTOL
    assert torch.equal(y_pair, y_one)
