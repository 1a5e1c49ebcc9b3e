"""GPU parity of the unquantized operations between the quantized layers (SiLU, additions, embeddings, up-sampling,
concatenation, GroupNorm, float convolution, attention core) against the CPU oracle.  Inputs are rounded to bf16 first,
so both sides see the same values; outputs are bf16 (or fp32 where stated)."""
import numpy as np
import pytest

from paper_2512_05746_b200 import inputs
from hq_testutil import PARITY_STATS, Y_BF16_RTOL, Y_F32_RTOL, attention_bound, rel_err

pytestmark = pytest.mark.gpu

BF16_HALF_ULP = 2.0 ** -8        # largest relative rounding error of one bf16 store (8 significant bits)


@pytest.fixture(scope="module")
def env():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2512_05746_b200 import binding as hq
    return torch, hq


def bf16(torch, a):
    """numpy fp32 -> (device bf16 tensor, the same values as numpy fp64)."""
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda().to(torch.bfloat16)
    return t, t.float().cpu().numpy().astype(np.float64)


def close_bf16(got, want, extra=0.0):
    """Element-wise: one bf16 rounding of the exact result (plus `extra` relative slack for fp32 arithmetic)."""
    got = got.astype(np.float64)
    return np.all(np.abs(got - want) <= (BF16_HALF_ULP + extra) * np.abs(want) + 1e-30)


def test_silu_add_bcast(env, oracle):
    torch, hq = env
    x, xr = bf16(torch, inputs.activations((64, 1024), seed=1) * 3.0)
    out = torch.empty_like(x)
    hq.hq_silu(x, out)
    assert close_bf16(out.float().cpu().numpy(), oracle.silu(xr), extra=2e-6)
    b, br = bf16(torch, inputs.activations((64, 1024), seed=2))
    hq.hq_add(x, b, out)
    assert close_bf16(out.float().cpu().numpy(), xr + br)
    h, hr = bf16(torch, inputs.activations((3, 5, 7, 64), seed=3))
    e, er = bf16(torch, inputs.activations((3, 64), seed=4))
    hq.hq_add_rows_bcast(h, e)
    assert close_bf16(h.float().cpu().numpy(), hr + er[:, None, None, :])


def test_step_and_class_embedding(env, oracle):
    torch, hq = env
    t = np.array([0.0, 1.0, 37.0, 999.0], np.float32)
    out = torch.empty((4, 256), dtype=torch.bfloat16, device="cuda")
    hq.hq_timestep_embedding(torch.from_numpy(t).cuda(), out)
    want = oracle.timestep_embedding(t.astype(np.float64), 256)
    # fp32 sine / cosine of arguments up to 999: absolute error about 1e-4 of the unit amplitude, then one bf16 rounding
    assert np.abs(out.float().cpu().numpy() - want).max() <= 2.0 ** -8 + 2e-4
    emb, er = bf16(torch, inputs.activations((4, 256), seed=5))
    table, tr = bf16(torch, inputs.activations((10, 256), seed=6))
    labels = np.array([3, 0, 9, 3], np.int32)
    hq.hq_class_embed_add(emb, table, torch.from_numpy(labels).cuda())
    assert close_bf16(emb.float().cpu().numpy(), er + tr[labels])


def test_upsample_and_concat(env, oracle):
    torch, hq = env
    x, xr = bf16(torch, inputs.activations((2, 5, 3, 24), seed=7))
    up = torch.zeros((2, 10, 6, 24), dtype=torch.bfloat16, device="cuda")
    hq.hq_upsample_nearest2x(x, up)
    assert np.array_equal(up.float().cpu().numpy(), oracle.upsample_nearest2x(xr))
    b, br = bf16(torch, inputs.activations((2, 5, 3, 40), seed=8))
    cat = torch.zeros((2, 5, 3, 64), dtype=torch.bfloat16, device="cuda")
    hq.hq_concat_channels(x, b, cat)
    assert np.array_equal(cat.float().cpu().numpy(), np.concatenate([xr, br], axis=-1))


@pytest.mark.parametrize("silu", [False, True])
@pytest.mark.parametrize("Nb,H,W,C,G", [
    (2, 8, 8, 128, 32),         # four channels per group: the two channel quads of a 16-byte piece lie in different groups
    (3, 4, 4, 384, 32),         # twelve channels per group, 48 pieces per pixel (not a divisor of the CTA size)
    (1, 16, 16, 64, 8),
    (70, 3, 7, 64, 8),          # 21 pixels per sample: a CTA's share of the pixels crosses several sample boundaries
    (2, 40, 40, 256, 32),       # 1600 pixels per sample: shares end inside a sample, rounds of loads with a ragged tail
])
def test_groupnorm_act(env, oracle, silu, Nb, H, W, C, G):
    torch, hq = env
    x, xr = bf16(torch, inputs.activations((Nb, H, W, C), outlier_count=2, outlier_scale=8.0, seed=C) + np.float32(0.4))
    rng = np.random.default_rng(C)
    gamma = (1.0 + 0.2 * rng.standard_normal(C)).astype(np.float32)
    beta = (0.1 * rng.standard_normal(C)).astype(np.float32)
    out = torch.empty_like(x)
    scratch = torch.empty((Nb * G * 24,), dtype=torch.uint8, device="cuda")
    hq.hq_groupnorm_act(x, G, torch.from_numpy(gamma).cuda(), torch.from_numpy(beta).cuda(), 1e-5, silu, out, scratch)
    want = oracle.groupnorm(xr, G, gamma, beta, 1e-5, "silu" if silu else "none")
    assert rel_err(out.float().cpu().numpy(), want) <= Y_BF16_RTOL


@pytest.mark.parametrize("Nb,H,W,C,Cout,xdt", [(2, 16, 16, 3, 128, "bf16"), (1, 9, 7, 4, 64, "f32"), (2, 8, 8, 3, 256, "bf16")])
def test_first_convolution(env, oracle, Nb, H, W, C, Cout, xdt):
    torch, hq = env
    x32 = inputs.activations((Nb, H, W, C), seed=H)
    if xdt == "bf16":
        x, xr = bf16(torch, x32)
    else:
        x, xr = torch.from_numpy(x32).cuda(), x32.astype(np.float64)
    w, b = inputs.weights((Cout, 3, 3, C), std=0.2, seed=Cout), inputs.bias(Cout, seed=1)
    y = torch.zeros((Nb, H, W, Cout), dtype=torch.bfloat16, device="cuda")
    hq.hq_conv2d_direct(x, torch.from_numpy(w).cuda(), torch.from_numpy(b).cuda(), 3, 1, 1, y)
    want = oracle.conv2d_float(xr, w, b, 1, 1)
    assert rel_err(y.float().cpu().numpy(), want) <= Y_BF16_RTOL


@pytest.mark.parametrize("Nb,H,W,C,Cout", [(2, 16, 16, 128, 3), (1, 9, 7, 264, 3), (2, 8, 8, 256, 4)])
def test_last_convolution(env, oracle, Nb, H, W, C, Cout):
    torch, hq = env
    x, xr = bf16(torch, inputs.activations((Nb, H, W, C), seed=C))
    w, b = inputs.weights((Cout, 3, 3, C), std=0.05, seed=Cout), inputs.bias(Cout, seed=2)
    y = torch.zeros((Nb, H, W, Cout), dtype=torch.float32, device="cuda")
    hq.hq_conv2d_direct(x, torch.from_numpy(w).cuda(), torch.from_numpy(b).cuda(), 3, 1, 1, y)
    want = oracle.conv2d_float(xr, w, b, 1, 1)
    assert rel_err(y.cpu().numpy(), want) <= Y_F32_RTOL
    with pytest.raises(hq.HqError):                       # a shape neither kernel covers
        hq.hq_conv2d_direct(x, torch.zeros((64, 3, 3, C), device="cuda"), None, 3, 1, 1,
                            torch.zeros((Nb, H, W, 64), dtype=torch.float32, device="cuda"))


ATTN_CASES = [
    # Nb, L, C, heads
    (2, 64, 256, 8),        # dh 32, one partly filled key block
    (2, 256, 384, 8),       # dh 48, two key blocks
    (1, 1024, 512, 8),      # dh 64, eight key blocks: the 32x32 level
    (2, 256, 768, 8),       # dh 96: the 16x16 level
    (3, 64, 1024, 8),       # dh 128: the 8x8 level
    (1, 200, 128, 2),       # ragged: 200 = 128 + 72 queries and keys
    (1, 16, 64, 2),         # a 4x4 map
    (3, 200, 128, 2),       # dh 64, ragged, several samples: the last key block of a sample reaches into the next one's rows
    (2, 72, 256, 2),        # dh 128, ragged, two samples
]


@pytest.mark.parametrize("Nb,L,C,heads", ATTN_CASES)
def test_attention_matches_oracle(env, oracle, Nb, L, C, heads):
    torch, hq = env
    scale = 2.0 if L >= 256 else 1.0                      # sharper softmax on the long sequences: the maximum moves
    qkv, qr = bf16(torch, inputs.activations((Nb * L, 3 * C), seed=L + C) * np.float32(scale))
    out = torch.full((Nb * L, C), 7.0, dtype=torch.bfloat16, device="cuda")
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    hq.hq_attention(qkv, Nb, heads, out, dev_status=status)
    torch.cuda.synchronize()
    hq.hq_check_status(status)
    want = oracle.attention(qr.reshape(Nb, L, 3 * C), heads).reshape(Nb * L, C)
    err = np.abs(out.float().cpu().numpy().astype(np.float64) - want)
    bound = attention_bound(oracle, qr, Nb, L, C, heads, want)
    PARITY_STATS.append(dict(what=f"attention {Nb}x{L}x{C} heads {heads}", max_err_over_bound=float((err / bound).max()),
                             rms_rel=float(np.sqrt((err ** 2).mean() / (want ** 2).mean()))))
    assert np.all(err <= bound), f"largest error / bound = {(err / bound).max():.3f}"
    assert np.sqrt((err ** 2).mean() / (want ** 2).mean()) <= Y_BF16_RTOL


@pytest.mark.parametrize("C,heads", [(128, 2), (256, 2), (96, 2)])
def test_attention_follows_a_late_maximum(env, oracle, C, heads):
    """Scores that grow by far more than the kernel's lazy-rescale threshold from one key block to the next: the keys of
    each block of 64 are scaled up block by block, so the running maximum of every row has to move (and the output
    accumulator has to be rescaled) at every block."""
    torch, hq = env
    Nb, L = 2, 320
    x = inputs.activations((Nb * L, 3 * C), seed=77).reshape(Nb, L, 3 * C).copy()
    x[:, :, :C] = np.abs(x[:, :, :C])                    # q, k >= 0: every score of a later block is larger
    x[:, :, C:2 * C] = np.abs(x[:, :, C:2 * C]) * (1.0 + 1.5 * (np.arange(L) // 64))[None, :, None]
    qkv, qr = bf16(torch, x.reshape(Nb * L, 3 * C).astype(np.float32))
    out = torch.empty((Nb * L, C), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    hq.hq_attention(qkv, Nb, heads, out, dev_status=status)
    torch.cuda.synchronize()
    hq.hq_check_status(status)
    want = oracle.attention(qr.reshape(Nb, L, 3 * C), heads).reshape(Nb * L, C)
    err = np.abs(out.float().cpu().numpy().astype(np.float64) - want)
    assert np.all(err <= attention_bound(oracle, qr, Nb, L, C, heads, want))


def test_attention_refuses_unsupported_head_width(env):
    torch, hq = env
    qkv = torch.zeros((64, 3 * 80), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(hq.HqError):
        hq.hq_attention(qkv, 1, 2, torch.zeros((64, 80), dtype=torch.bfloat16, device="cuda"))     # dh = 40
