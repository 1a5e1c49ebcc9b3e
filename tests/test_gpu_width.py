"""GPU parity of the convolution with the width-axis transform (Eq. 13-14 as the paper states them) against the
CPU oracle: the int8 activations z = clamp(rint(x H_c / S)) * H_raw, then the whole layer."""
import numpy as np
import pytest

from paper_2512_05746_b200 import inputs
from hq_testutil import CODE_MISMATCH_FRAC, CODE_TIE_REL, PARITY_STATS, Y_BF16_RTOL, Y_F32_RTOL, decode_blob, rel_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2512_05746_b200 import binding as hq
    return torch, hq


def codes_from_z(z, n, closed_H):
    """z = q * H_raw  =>  q = z * H_raw / n (exact): recovers the device's codes from its int8 activations."""
    Nb, H, W, C = z.shape
    zz = np.einsum("nhbic,ij->nhbjc", z.astype(np.int64).reshape(Nb, H, W // n, n, C), closed_H).reshape(z.shape)
    assert np.all(zz % n == 0)
    return (zz // n).astype(np.int64)


def closed_form_H(n):
    i = np.arange(n)
    pc = np.vectorize(lambda v: bin(v).count("1"))(i[:, None] & i[None, :])
    return (1 - 2 * (pc & 1)).astype(np.int64)


CASES = [
    # Nb, H, W, C, had_block_w, bits, dtype
    (2, 8, 32, 64, 16, 4, "f32"),
    (3, 5, 48, 32, 16, 4, "f32"),       # three blocks along w
    (2, 6, 32, 128, 32, 3, "f32"),      # 32-point blocks are allowed at 3 bits
    (1, 7, 8, 20, 8, 4, "bf16"),        # C not a multiple of 16, bf16 input
    (2, 4, 16, 64, 4, 8, "f32"),        # 8-bit codes: only 1-point ... 1*128: block must be 1
    (2, 4, 16, 64, 1, 8, "f32"),
]


@pytest.mark.parametrize("Nb,H,W,C,n,bits,dt", CASES)
def test_width_quant_matches_oracle(env, oracle, Nb, H, W, C, n, bits, dt):
    torch, hq = env
    x = inputs.activations((Nb, H, W, C), outlier_count=max(1, C // 50), outlier_scale=20.0, seed=W + C + n)
    xt = torch.from_numpy(x).cuda()
    if dt == "bf16":
        xt = xt.to(torch.bfloat16)
        x = xt.float().cpu().numpy()
    u = oracle.transform_width(x, n)
    S = float(np.float32(np.abs(u).max() / oracle.qmax(bits) / 2.5))          # clamps the largest values
    z = torch.full((Nb, H, W, C), 77, dtype=torch.int8, device="cuda")
    so = torch.zeros((1,), dtype=torch.float32, device="cuda")
    ss = torch.tensor([S], dtype=torch.float32, device="cuda")
    if n * 2 ** (bits - 1) > 128:
        with pytest.raises(hq.HqError) as e:
            hq.hq_hadamard_quant_width(xt, n, bits, ss, z, so)
        assert e.value.status == 6
        return
    hq.hq_hadamard_quant_width(xt, n, bits, ss, z, so)
    torch.cuda.synchronize()
    q_ref, _, v = oracle.quantize(u, bits, static_scale=S, want_v=True)
    z_gpu = z.cpu().numpy()
    q_gpu = codes_from_z(z_gpu, n, closed_form_H(n)) if n > 1 else z_gpu.astype(np.int64)
    bad = q_gpu != q_ref
    # Only rounding ties may differ, by one.  One static scale serves the whole tensor and the largest values are
    # clamped, so the full scale the fp32 error of a pre-rounding value is proportional to is the UNCLAMPED maximum
    # of |v| (2.5 x qmax here), not the clamp range.
    full = max(float(np.abs(v).max()), 1.0)
    dist = np.abs(v - (np.floor(v) + 0.5))
    PARITY_STATS.append(dict(what=f"width-axis {Nb}x{H}x{W}x{C} n={n} b={bits} {dt}", codes=int(q_ref.size),
                             mismatch_frac=float(bad.mean()), max_tie_rel=float((dist[bad] / full).max()) if bad.any() else 0.0))
    if bad.any():
        assert np.abs(q_gpu - q_ref)[bad].max() == 1 and bad.mean() <= CODE_MISMATCH_FRAC
        assert np.all(dist[bad] <= CODE_TIE_REL * full)
    assert np.array_equal(z_gpu.astype(np.int64), oracle.codes_inverse_width(q_gpu.astype(np.int8), n).astype(np.int64))
    assert q_gpu.min() == oracle.qmin(bits) and q_gpu.max() == oracle.qmax(bits)
    assert np.isclose(float(so.cpu()[0]), np.float32(S) * 2.0 ** (-0.5 * np.log2(n)), rtol=1e-6)


@pytest.mark.parametrize("Nb,H,W,C,Cout,R,stride,n,bits,odt", [
    (8, 32, 32, 256, 256, 3, 1, 16, 4, "bf16"),      # the small conv configuration, transform along the width
    (2, 16, 16, 128, 200, 3, 1, 16, 4, "f32"),
    (2, 32, 32, 64, 64, 3, 2, 16, 3, "f32"),         # stride 2, W4A3
    (2, 16, 16, 128, 128, 1, 1, 8, 4, "bf16"),       # 1x1
])
def test_qconv_width_layer_matches_oracle(env, oracle, Nb, H, W, C, Cout, R, stride, n, bits, odt):
    torch, hq = env
    x = inputs.activations((Nb, H, W, C), outlier_count=max(1, C // 100), outlier_scale=20.0, seed=H + C)
    w = inputs.weights((Cout, R, R, C), seed=Cout + R)
    b = inputs.bias(Cout, seed=2)
    pad = R // 2
    S = float(np.float32(np.abs(oracle.transform_width(x, n)).max() / oracle.qmax(bits) / 2.0))
    pw = hq.hq_weight_prepare(w, 4, 1, hq.HQ_W_PLAIN, hq.HQ_CODES_INT8).to_device()
    Ho, Wo = (H + 2 * pad - R) // stride + 1, (W + 2 * pad - R) // stride + 1
    y = torch.zeros((Nb, Ho, Wo, Cout), dtype=torch.bfloat16 if odt == "bf16" else torch.float32, device="cuda")
    ws = torch.zeros((hq.hq_workspace_size(Nb * H * W, C, hq.HQ_CODES_INT8),), dtype=torch.uint8, device="cuda")
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    hq.hq_qconv_width(torch.from_numpy(x).cuda(), pw, R, R, stride, pad, torch.from_numpy(b).cuda(), bits, n,
                      torch.tensor([S], dtype=torch.float32, device="cuda"), y, ws, dev_status=status)
    torch.cuda.synchronize()
    hq.hq_check_status(status)
    ref = oracle.qconv_width(x, w, b, a_bits=bits, w_bits=4, had_block_w=n, stride=stride, pad=pad, static_scale=S)
    # the device's own integer activations (they may differ from the oracle's at rounding ties) -> oracle conv + rescale
    z_gpu = ws[: Nb * H * W * C].view(torch.int8).cpu().numpy().reshape(Nb, H, W, C)
    assert (z_gpu.astype(np.int64) != ref["z"]).mean() <= 16 * CODE_MISMATCH_FRAC
    B = ref["B"]
    assert np.array_equal(decode_blob(pw).reshape(Cout, R, R, C), B) and np.array_equal(pw.s_w, ref["s_w"])
    y_own = oracle.dequant(oracle.conv2d_int_z(z_gpu.astype(np.int32), B, stride, pad), ref["s_a"], pw.s_w, b, ref["alpha"])
    assert rel_err(y.float().cpu().numpy(), y_own) <= (Y_BF16_RTOL if odt == "bf16" else Y_F32_RTOL)
    rms = np.sqrt(np.mean((y.float().cpu().numpy() - ref["y"]) ** 2)) / np.sqrt(np.mean(ref["y"] ** 2))
    assert rms <= Y_BF16_RTOL


WIDE_CASES = [
    # Nb, H, W, C, had_block_w, bits, dtype
    (2, 6, 32, 64, 32, 4, "f32"),       # the full width of a 32-wide map as one block
    (1, 5, 64, 32, 64, 4, "bf16"),      # ... of a 64-wide map
    (2, 3, 64, 16, 32, 4, "f32"),       # two 32-blocks
    (2, 4, 64, 8, 64, 3, "f32"),
]


@pytest.mark.parametrize("Nb,H,W,C,n,bits,dt", WIDE_CASES)
def test_width_quant_two_limbs_matches_oracle(env, oracle, Nb, H, W, C, n, bits, dt):
    """Blocks of 32 and 64 positions: z = q * H_raw leaves as two int8 limbs per channel, [hi | lo] per pixel."""
    torch, hq = env
    x = inputs.activations((Nb, H, W, C), outlier_count=max(1, C // 50), outlier_scale=20.0, seed=W + C + n)
    x[:, :, ::n, 1] = 1000.0         # a spike at the head of every block of channel 1: flat after the transform, so that
    xt = torch.from_numpy(x).cuda()  # all n codes sit at qmax and z = q * H_raw reaches n * qmax, beyond a signed byte
    if dt == "bf16":
        xt = xt.to(torch.bfloat16)
        x = xt.float().cpu().numpy()
    u = oracle.transform_width(x, n)
    S = float(np.float32(np.abs(u).max() / oracle.qmax(bits) / 2.5))
    zl = torch.full((Nb, H, W, 2 * C), 77, dtype=torch.int8, device="cuda")
    so = torch.zeros((1,), dtype=torch.float32, device="cuda")
    hq.hq_hadamard_quant_width2(xt, n, bits, torch.tensor([S], dtype=torch.float32, device="cuda"), zl, so)
    torch.cuda.synchronize()
    zz = zl.cpu().numpy().astype(np.int64)
    hi, lo = zz[..., :C], zz[..., C:]
    assert lo.min() >= -128 and lo.max() <= 127
    z_gpu = 256 * hi + lo
    q_ref, _, v = oracle.quantize(u, bits, static_scale=S, want_v=True)
    q_gpu = codes_from_z(z_gpu, n, closed_form_H(n))
    bad = q_gpu != q_ref
    full = max(float(np.abs(v).max()), 1.0)
    dist = np.abs(v - (np.floor(v) + 0.5))
    PARITY_STATS.append(dict(what=f"width-axis two limbs {Nb}x{H}x{W}x{C} n={n} b={bits} {dt}", codes=int(q_ref.size),
                             mismatch_frac=float(bad.mean()), max_tie_rel=float((dist[bad] / full).max()) if bad.any() else 0.0))
    if bad.any():
        assert np.abs(q_gpu - q_ref)[bad].max() == 1 and bad.mean() <= CODE_MISMATCH_FRAC
        assert np.all(dist[bad] <= CODE_TIE_REL * full)
    assert np.array_equal(z_gpu, oracle.codes_inverse_width(q_gpu.astype(np.int8), n).astype(np.int64))
    assert np.abs(z_gpu).max() > 127                           # the case needs the second limb
    assert np.isclose(float(so.cpu()[0]), np.float32(S) * 2.0 ** (-0.5 * np.log2(n)), rtol=1e-6)


@pytest.mark.parametrize("Nb,H,W,C,Cout,R,stride,n,odt", [
    (2, 32, 32, 128, 128, 3, 1, 32, "bf16"),     # the full-width transform of Eq. 13 on a 32-wide map
    (1, 16, 64, 64, 200, 3, 1, 64, "f32"),       # ... on a 64-wide map, ragged Cout
    (2, 32, 32, 64, 64, 3, 2, 32, "f32"),        # stride 2
])
def test_qconv_width_two_limbs_layer_matches_oracle(env, oracle, Nb, H, W, C, Cout, R, stride, n, odt):
    torch, hq = env
    x = inputs.activations((Nb, H, W, C), outlier_count=max(1, C // 100), outlier_scale=20.0, seed=H + C)
    w = inputs.weights((Cout, R, R, C), seed=Cout + R)
    b = inputs.bias(Cout, seed=2)
    pad = R // 2
    S = float(np.float32(np.abs(oracle.transform_width(x, n)).max() / 7 / 2.0))
    pw = hq.hq_weight_prepare(w, 4, 1, hq.HQ_W_PLAIN_A2, hq.HQ_CODES_INT8).to_device()
    assert pw.desc.C == 2 * C and pw.desc.limbs == 2
    Ho, Wo = (H + 2 * pad - R) // stride + 1, (W + 2 * pad - R) // stride + 1
    y = torch.zeros((Nb, Ho, Wo, Cout), dtype=torch.bfloat16 if odt == "bf16" else torch.float32, device="cuda")
    ws = torch.zeros((hq.hq_workspace_size(Nb * H * W, 2 * C, hq.HQ_CODES_INT8),), dtype=torch.uint8, device="cuda")
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    hq.hq_qconv_width(torch.from_numpy(x).cuda(), pw, R, R, stride, pad, torch.from_numpy(b).cuda(), 4, n,
                      torch.tensor([S], dtype=torch.float32, device="cuda"), y, ws, dev_status=status)
    torch.cuda.synchronize()
    hq.hq_check_status(status)
    ref = oracle.qconv_width(x, w, b, a_bits=4, w_bits=4, had_block_w=n, stride=stride, pad=pad, static_scale=S)
    zz = ws[: Nb * H * W * 2 * C].view(torch.int8).cpu().numpy().reshape(Nb, H, W, 2 * C).astype(np.int64)
    z_gpu = 256 * zz[..., :C] + zz[..., C:]
    assert (z_gpu != ref["z"]).mean() <= n * CODE_MISMATCH_FRAC          # one code touches the n positions of its block
    assert np.array_equal(pw.s_w, ref["s_w"])
    y_own = oracle.dequant(oracle.conv2d_int_z(z_gpu.astype(np.int32), ref["B"], stride, pad), ref["s_a"], pw.s_w, b, ref["alpha"])
    assert rel_err(y.float().cpu().numpy(), y_own) <= (Y_BF16_RTOL if odt == "bf16" else Y_F32_RTOL)
    rms = np.sqrt(np.mean((y.float().cpu().numpy() - ref["y"]) ** 2)) / np.sqrt(np.mean(ref["y"] ** 2))
    assert rms <= Y_BF16_RTOL
