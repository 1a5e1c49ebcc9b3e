"""GPU parity of GroupNorm + SiLU fused in front of the transform + quantization (hq_gn_silu_quant) against the CPU
oracle.  The prologue runs in fp32 with the hardware's approximate exponential and reciprocal; the transform that follows sums
a whole block of such values, over which their independent errors average out, so the codes are held to the same rule
as the plain kernel's (one step of difference only within 1e-6 of the row's full scale from a rounding boundary, for at
most 1e-4 of the codes) and the scales to the same 1e-6.  Measured on these cases: no differing code in 1.0 M codes
(GroupNorm) and 2.9e-6 of the codes at a tie distance of 1.5e-8 (LayerNorm); scales within 2.4e-7."""
import numpy as np
import pytest

from paper_2512_05746_b200 import inputs
from hq_testutil import CODE_MISMATCH_FRAC, CODE_TIE_REL, PARITY_STATS, check_codes, unpack_nibbles_np

pytestmark = pytest.mark.gpu

GN_TIE_REL = CODE_TIE_REL
GN_MISMATCH_FRAC = CODE_MISMATCH_FRAC
GN_SCALE_RTOL = 1e-6


@pytest.fixture(scope="module")
def env():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2512_05746_b200 import binding as hq
    return torch, hq


@pytest.mark.parametrize("Nb,H,W,C,G,n,bits,dt,static", [
    (2, 16, 16, 256, 32, 256, 4, "f32", False),
    (2, 16, 16, 256, 32, 256, 4, "bf16", False),
    (3, 8, 8, 512, 32, 256, 4, "bf16", False),      # two Hadamard blocks per pixel
    (2, 8, 8, 768, 32, 256, 3, "f32", False),       # 24 channels per group, three blocks
    (2, 16, 16, 128, 32, 128, 4, "f32", True),      # static scale, 4 channels per group
    (1, 32, 32, 512, 32, 512, 4, "f32", False),
])
def test_gn_silu_quant_matches_oracle(env, oracle, Nb, H, W, C, G, n, bits, dt, static):
    torch, hq = env
    rng = np.random.default_rng(C + H)
    x = inputs.activations((Nb, H, W, C), outlier_count=max(1, C // 100), outlier_scale=8.0, seed=C + G) + np.float32(0.7)
    gamma = (1.0 + 0.2 * rng.standard_normal(C)).astype(np.float32)
    beta = (0.1 * rng.standard_normal(C)).astype(np.float32)
    xt = torch.from_numpy(x).cuda()
    if dt == "bf16":
        xt = xt.to(torch.bfloat16)
        x = xt.float().cpu().numpy()
    eps = 1e-6
    rows = Nb * H * W
    codes = torch.full((rows, C // 2), 0x5A, dtype=torch.uint8, device="cuda")
    scales = torch.full((rows,), -1.0, dtype=torch.float32, device="cuda")
    scratch = torch.empty((Nb * G * 24,), dtype=torch.uint8, device="cuda")
    y_ref = oracle.groupnorm_silu(x, G, gamma, beta, eps)
    u = oracle.transform(y_ref.reshape(rows, C), n)
    s0 = float(np.float32(np.abs(u).max() / oracle.qmax(bits) / 2.0)) if static else None
    ss = torch.tensor([s0], dtype=torch.float32, device="cuda") if static else None
    hq.hq_gn_silu_quant(xt, G, torch.from_numpy(gamma).cuda(), torch.from_numpy(beta).cuda(), eps, n, bits, codes,
                        hq.HQ_CODES_NIBBLE, scratch, scales=scales, static_scale=ss)
    torch.cuda.synchronize()
    q = unpack_nibbles_np(codes.cpu().numpy())
    q_ref, s_ref, v = oracle.quantize(u, bits, static_scale=s0, want_v=True)
    if static:
        assert float(scales.cpu()[0]) == np.float32(s0)
        v = np.clip(v, oracle.qmin(bits) - 0.25, oracle.qmax(bits) + 0.25)
    else:
        dev = float(np.abs(scales.cpu().numpy() / s_ref - 1.0).max())
        PARITY_STATS.append(dict(what=f"groupnorm prologue scales {Nb}x{H}x{W}x{C} {dt}", max_scale_rel=dev))
        assert dev <= GN_SCALE_RTOL
    check_codes(q, q_ref, v, f"groupnorm prologue {Nb}x{H}x{W}x{C} {dt}", tie_rel=GN_TIE_REL, mismatch_frac=GN_MISMATCH_FRAC)
    # the dequantized values are the normalised, activated, transformed input within half a step (Eq. 3)
    s_gpu = scales.cpu().numpy()[:, None] if not static else np.float32(s0)
    inside = np.abs(v) < oracle.qmax(bits)
    assert np.all(np.abs(u - s_gpu * q)[inside] <= 0.5 * np.max(s_gpu) * (1 + 1e-3) + 1e-6)


@pytest.mark.parametrize("Nb,H,W,C,G,n,dt", [(3, 8, 8, 256, 32, 256, "bf16"), (2, 8, 8, 128, 32, 128, "f32"),
                                             (5, 4, 8, 512, 32, 256, "bf16")])
def test_gn_silu_quant_with_a_per_sample_addend(env, oracle, Nb, H, W, C, G, n, dt):
    """pre_bias[n, c] (the projected step embedding of a residual block) is added in front of the normalisation without
    the sum being stored: codes and scales against the oracle applied to x + pre_bias."""
    torch, hq = env
    x = inputs.activations((Nb, H, W, C), outlier_count=2, outlier_scale=8.0, seed=C + Nb) + np.float32(0.3)
    e = (1.5 * inputs.activations((Nb, C), seed=Nb)).astype(np.float32)
    rng = np.random.default_rng(C)
    gamma = (1.0 + 0.2 * rng.standard_normal(C)).astype(np.float32)
    beta = (0.1 * rng.standard_normal(C)).astype(np.float32)
    xt = torch.from_numpy(x).cuda()
    if dt == "bf16":
        xt = xt.to(torch.bfloat16)
        x = xt.float().cpu().numpy()
    et = torch.from_numpy(e).cuda().to(torch.bfloat16)
    e = et.float().cpu().numpy()
    rows = Nb * H * W
    codes = torch.zeros((rows, C // 2), dtype=torch.uint8, device="cuda")
    scales = torch.zeros((rows,), dtype=torch.float32, device="cuda")
    scratch = torch.empty((Nb * G * 24,), dtype=torch.uint8, device="cuda")
    hq.hq_gn_silu_quant(xt, G, torch.from_numpy(gamma).cuda(), torch.from_numpy(beta).cuda(), 1e-5, n, 4, codes,
                        hq.HQ_CODES_NIBBLE, scratch, scales=scales, pre_bias=et)
    torch.cuda.synchronize()
    xe = x.astype(np.float64) + e.astype(np.float64)[:, None, None, :]
    u = oracle.transform(oracle.groupnorm_silu(xe, G, gamma, beta, 1e-5).reshape(rows, C), n)
    q_ref, s_ref, v = oracle.quantize(u, 4, want_v=True)
    assert float(np.abs(scales.cpu().numpy() / s_ref - 1.0).max()) <= GN_SCALE_RTOL
    check_codes(unpack_nibbles_np(codes.cpu().numpy()), q_ref, v, f"groupnorm prologue with addend {Nb}x{H}x{W}x{C} {dt}",
                tie_rel=GN_TIE_REL, mismatch_frac=GN_MISMATCH_FRAC)
    # and the addend matters: without it the codes are others
    hq.hq_gn_silu_quant(xt, G, torch.from_numpy(gamma).cuda(), torch.from_numpy(beta).cuda(), 1e-5, n, 4, codes,
                        hq.HQ_CODES_NIBBLE, scratch, scales=scales)
    torch.cuda.synchronize()
    assert (unpack_nibbles_np(codes.cpu().numpy()) != q_ref).mean() > 0.2


@pytest.mark.parametrize("Nb,H,W,c1,c2,G,n,pre", [(3, 8, 8, 256, 512, 32, 256, False), (2, 8, 8, 128, 128, 32, 128, True),
                                                  (5, 4, 8, 512, 256, 32, 256, True)])
def test_gn_silu_quant_of_a_concatenation_read_in_place(env, oracle, Nb, H, W, c1, c2, G, n, pre):
    """GroupNorm + SiLU + transform + quantize of [x | x2] without the concatenation being written: the groups' statistics
    run over both tensors (a group may lie in either), codes and scales as the oracle's on the concatenated tensor and
    bit-identical to the call on the written-out concatenation."""
    torch, hq = env
    C = c1 + c2
    a = inputs.activations((Nb, H, W, c1), outlier_count=2, outlier_scale=8.0, seed=c1) + np.float32(0.3)
    b = inputs.activations((Nb, H, W, c2), outlier_count=1, outlier_scale=4.0, seed=c2 + 3) * np.float32(2.0) - np.float32(0.5)
    ta, tb = torch.from_numpy(a).cuda().to(torch.bfloat16), torch.from_numpy(b).cuda().to(torch.bfloat16)
    cat = torch.cat([ta, tb], dim=3).contiguous()
    x = cat.float().cpu().numpy().astype(np.float64)
    rng = np.random.default_rng(C)
    gamma = (1.0 + 0.2 * rng.standard_normal(C)).astype(np.float32)
    beta = (0.1 * rng.standard_normal(C)).astype(np.float32)
    et = torch.from_numpy(inputs.activations((Nb, C), seed=9)).cuda().to(torch.bfloat16) if pre else None
    if pre:
        x = x + et.float().cpu().numpy().astype(np.float64)[:, None, None, :]
    rows = Nb * H * W
    out = []
    for two in (True, False):
        codes = torch.zeros((rows, C // 2), dtype=torch.uint8, device="cuda")
        scales = torch.zeros((rows,), dtype=torch.float32, device="cuda")
        scratch = torch.empty((Nb * G * 24,), dtype=torch.uint8, device="cuda")
        hq.hq_gn_silu_quant(ta if two else cat, G, torch.from_numpy(gamma).cuda(), torch.from_numpy(beta).cuda(), 1e-5, n, 4,
                            codes, hq.HQ_CODES_NIBBLE, scratch, scales=scales, pre_bias=et, x2=tb if two else None)
        torch.cuda.synchronize()
        out.append((codes.cpu().numpy(), scales.cpu().numpy()))
    assert np.array_equal(out[0][0], out[1][0]) and np.array_equal(out[0][1], out[1][1])
    u = oracle.transform(oracle.groupnorm_silu(x, G, gamma, beta, 1e-5).reshape(rows, C), n)
    q_ref, s_ref, v = oracle.quantize(u, 4, want_v=True)
    assert float(np.abs(out[0][1] / s_ref - 1.0).max()) <= GN_SCALE_RTOL
    check_codes(unpack_nibbles_np(out[0][0]), q_ref, v, f"groupnorm prologue on a concatenation {Nb}x{H}x{W}x({c1}+{c2})",
                tie_rel=GN_TIE_REL, mismatch_frac=GN_MISMATCH_FRAC)


def test_gn_silu_quant_on_an_input_aligned_to_8_bytes_only(env, oracle):
    """A bf16 tensor that starts 8 bytes into an allocation: the statistics pass then reads four channels per load."""
    torch, hq = env
    Nb, H, W, C, G, n = 2, 8, 8, 128, 32, 128
    x = inputs.activations((Nb, H, W, C), outlier_count=1, outlier_scale=8.0, seed=3) + np.float32(0.5)
    rng = np.random.default_rng(5)
    gamma = (1.0 + 0.2 * rng.standard_normal(C)).astype(np.float32)
    beta = (0.1 * rng.standard_normal(C)).astype(np.float32)
    store = torch.zeros((x.size + 4,), dtype=torch.bfloat16, device="cuda")
    xt = store[4:].view(Nb, H, W, C)
    xt.copy_(torch.from_numpy(x).cuda().to(torch.bfloat16))
    assert xt.data_ptr() % 16 == 8
    x = xt.float().cpu().numpy()
    rows = Nb * H * W
    codes = torch.zeros((rows, C // 2), dtype=torch.uint8, device="cuda")
    scales = torch.zeros((rows,), dtype=torch.float32, device="cuda")
    scratch = torch.empty((Nb * G * 24,), dtype=torch.uint8, device="cuda")
    hq.hq_gn_silu_quant(xt, G, torch.from_numpy(gamma).cuda(), torch.from_numpy(beta).cuda(), 1e-6, n, 4, codes,
                        hq.HQ_CODES_NIBBLE, scratch, scales=scales)
    torch.cuda.synchronize()
    u = oracle.transform(oracle.groupnorm_silu(x, G, gamma, beta, 1e-6).reshape(rows, C), n)
    q_ref, s_ref, v = oracle.quantize(u, 4, want_v=True)
    assert float(np.abs(scales.cpu().numpy() / s_ref - 1.0).max()) <= GN_SCALE_RTOL
    check_codes(unpack_nibbles_np(codes.cpu().numpy()), q_ref, v, "groupnorm prologue, 8-byte aligned input",
                tie_rel=GN_TIE_REL, mismatch_frac=GN_MISMATCH_FRAC)


LN_TIE_REL = CODE_TIE_REL
LN_MISMATCH_FRAC = CODE_MISMATCH_FRAC
LN_SCALE_RTOL = 1e-6


@pytest.mark.parametrize("rows,cols,n,rpg,bits,dt,cont,static,affine", [
    (512, 1152, 128, 256, 4, "bf16", 1, False, True),    # the diffusion-transformer width: nine 128-blocks, two samples
    (300, 1152, 128, 0, 4, "f32", 0, False, True),       # ragged row count, one affine pair for all rows
    (256, 512, 512, 32, 3, "f32", 1, False, True),       # one block per row, eight samples
    (192, 4608, 128, 64, 4, "bf16", 1, False, True),     # the MLP's hidden width (36 blocks)
    (128, 256, 256, 0, 4, "f32", 0, True, False),        # static scale, no affine
    (96, 2048, 2048, 32, 4, "f32", 1, False, True),      # 64 values per thread
])
def test_ln_quant_matches_oracle(env, oracle, rows, cols, n, rpg, bits, dt, cont, static, affine):
    torch, hq = env
    rng = np.random.default_rng(rows + cols)
    x = inputs.activations((rows, cols), outlier_count=max(1, cols // 100), outlier_scale=8.0, seed=cols + n) * np.float32(1.7) \
        + np.float32(0.4)
    groups = (rows + rpg - 1) // rpg if rpg > 0 else 1
    w = (1.0 + 0.3 * rng.standard_normal((groups, cols))).astype(np.float32) if affine else None
    b = (0.5 * rng.standard_normal((groups, cols))).astype(np.float32) if affine else None
    xt = torch.from_numpy(x).cuda()
    if dt == "bf16":
        xt = xt.to(torch.bfloat16)
        x = xt.float().cpu().numpy()
    eps = 1e-6
    pitch = cols // 2 if cont == 0 else cols
    codes = torch.full((rows, pitch), 0x5A, dtype=torch.uint8, device="cuda")
    scales = torch.full((rows,), -1.0, dtype=torch.float32, device="cuda")
    y_ref = oracle.layernorm_affine(x, w, b, rows_per_group=rpg, eps=eps)
    u = oracle.transform(y_ref, n)
    s0 = float(np.float32(np.abs(u).max() / oracle.qmax(bits) / 2.0)) if static else None
    ss = torch.tensor([s0], dtype=torch.float32, device="cuda") if static else None
    hq.hq_ln_quant(xt, None if w is None else torch.from_numpy(w).cuda(), None if b is None else torch.from_numpy(b).cuda(),
                   rpg, eps, n, bits, codes, cont, scales=scales, static_scale=ss)
    torch.cuda.synchronize()
    q = unpack_nibbles_np(codes.cpu().numpy()) if cont == 0 else codes.cpu().numpy().view(np.int8)
    q_ref, s_ref, v = oracle.quantize(u, bits, static_scale=s0, want_v=True)
    if static:
        assert float(scales.cpu()[0]) == np.float32(s0)
        v = np.clip(v, oracle.qmin(bits) - 0.25, oracle.qmax(bits) + 0.25)
    else:
        dev = float(np.abs(scales.cpu().numpy() / s_ref - 1.0).max())
        PARITY_STATS.append(dict(what=f"layernorm prologue scales {rows}x{cols} {dt}", max_scale_rel=dev))
        assert dev <= LN_SCALE_RTOL
    check_codes(q, q_ref, v, f"layernorm prologue {rows}x{cols} {dt}", tie_rel=LN_TIE_REL, mismatch_frac=LN_MISMATCH_FRAC)
    s_gpu = scales.cpu().numpy()[:, None] if not static else np.float32(s0)
    inside = np.abs(v) < oracle.qmax(bits)
    assert np.all(np.abs(u - s_gpu * q)[inside] <= 0.5 * np.max(s_gpu) * (1 + 1e-3) + 1e-6)


def test_ln_quant_refuses_what_it_cannot_do(env):
    torch, hq = env
    x = torch.zeros((64, 1152), device="cuda")
    codes = torch.zeros((64, 1152), dtype=torch.uint8, device="cuda")
    sc = torch.zeros((64,), device="cuda")
    with pytest.raises(hq.HqError):                       # groups of 10 rows cannot be split over whole CTAs
        hq.hq_ln_quant(x, None, None, 10, 1e-6, 128, 4, codes, 1, scales=sc)
    with pytest.raises(hq.HqError):                       # a block size the fast kernel does not take
        hq.hq_ln_quant(x, None, None, 0, 1e-6, 16, 4, codes, 1, scales=sc)
