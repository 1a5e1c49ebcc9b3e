"""Pins of the oracle's network glue (attention core, GroupNorm, up-sampling, step embedding, float convolution) against
torch's CPU routines in fp64 and closed forms.  No GPU, no CUDA library.  Each test names the mistake it would catch."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F


def rnd(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


@pytest.mark.parametrize("Nb,L,C,heads", [(2, 16, 32, 4), (1, 64, 48, 2), (3, 7, 8, 8)])
def test_attention_equals_torch_sdpa(oracle, Nb, L, C, heads):
    """torch's scaled_dot_product_attention works on [N, heads, L, dh] tensors: a wrong head split, a missing
    1/sqrt(dh), a softmax over the wrong axis or q and k swapped all fail here."""
    qkv = rnd((Nb, L, 3 * C), L + C)
    dh = C // heads
    t = torch.from_numpy(qkv)
    q, k, v = (t[:, :, i * C:(i + 1) * C].reshape(Nb, L, heads, dh).permute(0, 2, 1, 3) for i in range(3))
    want = F.scaled_dot_product_attention(q, k, v).permute(0, 2, 1, 3).reshape(Nb, L, C).numpy()
    got = oracle.attention(qkv, heads)
    assert np.allclose(got, want, rtol=1e-12, atol=1e-13)


def test_attention_closed_forms(oracle):
    Nb, L, C, heads = 1, 5, 4, 2
    qkv = rnd((Nb, L, 3 * C), 1)
    # zero queries: uniform weights -> the mean of the values
    z = qkv.copy()
    z[:, :, :C] = 0.0
    assert np.allclose(oracle.attention(z, heads)[0], np.broadcast_to(z[0, :, 2 * C:].mean(axis=0), (L, C)), atol=1e-14)
    # one key that dominates every query: the output is that key's value vector
    d = qkv.copy()
    d[:, :, :C] = 1.0
    d[:, :, C:2 * C] = 0.0
    d[0, 3, C:2 * C] = 1000.0
    assert np.allclose(oracle.attention(d, heads)[0], np.broadcast_to(d[0, 3, 2 * C:], (L, C)), atol=1e-12)
    # heads do not mix: changing head 1's inputs leaves head 0's output alone
    e = qkv.copy()
    e[:, :, [2, 3, C + 2, C + 3, 2 * C + 2, 2 * C + 3]] += 1.0
    assert np.array_equal(oracle.attention(e, heads)[..., :2], oracle.attention(qkv, heads)[..., :2])
    # rows of the softmax sum to one: constant values come back
    c = qkv.copy()
    c[:, :, 2 * C:] = 2.5
    assert np.allclose(oracle.attention(c, heads), 2.5, atol=1e-14)
    with pytest.raises(ValueError):
        oracle.attention(qkv, 3)


@pytest.mark.parametrize("act", ["none", "silu"])
@pytest.mark.parametrize("Nb,H,W,C,G", [(2, 4, 4, 32, 8), (1, 3, 5, 24, 4)])
def test_groupnorm_equals_torch(oracle, act, Nb, H, W, C, G):
    x = rnd((Nb, H, W, C), C) * 2.0 + 0.3
    gamma, beta = 1.0 + 0.2 * rnd((C,), 1), 0.1 * rnd((C,), 2)
    t = torch.from_numpy(x).permute(0, 3, 1, 2)
    want = F.group_norm(t, G, torch.from_numpy(gamma), torch.from_numpy(beta), eps=1e-5)
    if act == "silu":
        want = F.silu(want)
    got = oracle.groupnorm(x, G, gamma, beta, 1e-5, act)
    assert np.allclose(got, want.permute(0, 2, 3, 1).numpy(), rtol=1e-12, atol=1e-12)
    if act == "silu":      # the older entry point is the same function
        assert np.array_equal(got, oracle.groupnorm_silu(x, G, gamma, beta, 1e-5))


def test_silu_values(oracle):
    assert oracle.silu(0.0) == 0.0
    assert np.isclose(oracle.silu(1.0), 1.0 / (1.0 + np.exp(-1.0)), rtol=1e-15)
    assert np.allclose(oracle.silu(np.array([-30.0, 30.0])), [-30.0 * np.exp(-30.0), 30.0], rtol=1e-12)
    x = rnd((50,), 0)
    assert np.allclose(oracle.silu(x), F.silu(torch.from_numpy(x)).numpy(), rtol=1e-14)


def test_upsample_equals_torch_and_replicates(oracle):
    x = rnd((2, 3, 5, 4), 0)
    want = F.interpolate(torch.from_numpy(x).permute(0, 3, 1, 2), scale_factor=2, mode="nearest").permute(0, 2, 3, 1).numpy()
    got = oracle.upsample_nearest2x(x)
    assert got.shape == (2, 6, 10, 4) and np.array_equal(got, want)
    assert np.array_equal(got[:, 0::2, 1::2], x) and np.array_equal(got[:, 1::2, 0::2], x)


def test_timestep_embedding_closed_forms(oracle):
    e = oracle.timestep_embedding([0.0, 1.0, 250.0], 8, 10000.0)
    assert np.array_equal(e[0], [1, 1, 1, 1, 0, 0, 0, 0])                       # cos 0 | sin 0
    f = 10000.0 ** (-np.arange(4) / 4.0)                                        # 1, 0.1, 0.01, 0.001
    assert np.allclose(f, [1.0, 0.1, 0.01, 0.001])
    assert np.allclose(e[1], np.concatenate([np.cos(f), np.sin(f)]), rtol=1e-14)
    assert np.allclose(e[2], np.concatenate([np.cos(250.0 * f), np.sin(250.0 * f)]), rtol=1e-12, atol=1e-14)
    assert np.allclose(e[:, :4] ** 2 + e[:, 4:] ** 2, 1.0, atol=1e-14)          # a swapped half would still pass this,
    assert e[1, 4] == np.sin(1.0)                                               # ... this one pins the order
    with pytest.raises(ValueError):
        oracle.timestep_embedding([1.0], 7)


@pytest.mark.parametrize("R,stride,pad,C,Cout", [(3, 1, 1, 3, 8), (3, 1, 1, 16, 3), (1, 1, 0, 5, 4), (3, 2, 1, 4, 6)])
def test_conv2d_float_equals_torch(oracle, R, stride, pad, C, Cout):
    x, w, b = rnd((2, 6, 7, C), C), rnd((Cout, R, R, C), Cout), rnd((Cout,), 3)
    want = F.conv2d(torch.from_numpy(x).permute(0, 3, 1, 2), torch.from_numpy(w).permute(0, 3, 1, 2), torch.from_numpy(b),
                    stride=stride, padding=pad).permute(0, 2, 3, 1).numpy()
    assert np.allclose(oracle.conv2d_float(x, w, b, stride, pad), want, rtol=1e-12, atol=1e-12)
    # and it is the integer convolution when the operands are integers (the pinned direct loops of Eq. 14)
    xi = np.random.default_rng(1).integers(-8, 8, size=(1, 5, 5, C)).astype(np.int8)
    wi = np.random.default_rng(2).integers(-8, 8, size=(Cout, R, R, C)).astype(np.int32)
    assert np.array_equal(oracle.conv2d_float(xi, wi, None, stride, pad), oracle.conv2d_int(xi, wi, stride, pad))


def test_round_bf16_equals_torch_conversion(oracle):
    """Ties go to even, the sign is kept, values already representable come back unchanged."""
    x = np.concatenate([rnd((4000,), 5) * 10.0 ** rnd((4000,), 6), [0.0, -0.0, 1.0, 1.00390625, 1.01171875, -3.0e38, 1e-40]])
    want = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).float().numpy().astype(np.float64)
    got = oracle.round_bf16(x)
    assert np.array_equal(got, want)
    assert oracle.round_bf16(1.00390625) == 1.0 and oracle.round_bf16(1.01171875) == 1.015625      # ties: to even
    assert np.array_equal(oracle.round_bf16(got), got)
