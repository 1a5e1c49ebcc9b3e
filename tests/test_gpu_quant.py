"""GPU parity: fused Hadamard transform + quantization (hq_hadamard_quant) against the CPU oracle."""
import numpy as np
import pytest

from paper_2512_05746_b200 import inputs
from hq_testutil import SCALE_RTOL, check_codes, unpack_nibbles_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2512_05746_b200 import binding as hq
    return torch, hq


def run_quant(torch, hq, x_np, had_block, bits, container, static_scale=None, dtype=None, ldx=None):
    rows, cols = x_np.shape
    dev = "cuda"
    if ldx is None:
        x = torch.from_numpy(x_np).to(dev)
    else:
        buf = torch.zeros((rows, ldx), dtype=torch.float32, device=dev)
        buf[:, :cols] = torch.from_numpy(x_np).to(dev)
        x = buf[:, :cols]
    if dtype is not None:
        x = x.to(dtype)
    pitch = ((cols // 2 if container == hq.HQ_CODES_NIBBLE else cols) + 15) // 16 * 16
    codes = torch.full((max(rows, 1), pitch), 0x5A, dtype=torch.uint8, device=dev)[:rows]
    if static_scale is None:
        scales = torch.full((max(rows, 1),), -1.0, dtype=torch.float32, device=dev)
        ss = None
    else:
        scales = torch.full((1,), -1.0, dtype=torch.float32, device=dev)
        ss = torch.tensor([static_scale], dtype=torch.float32, device=dev)
    hq.hq_hadamard_quant(x, had_block, bits, codes, container, scales=scales, static_scale=ss)
    torch.cuda.synchronize()
    c = codes.cpu().numpy()
    if container == hq.HQ_CODES_NIBBLE:
        q = unpack_nibbles_np(c[:, : cols // 2])
    else:
        q = c[:, :cols].view(np.int8)
    return q, scales.cpu().numpy(), (x.float().cpu().numpy() if dtype is not None else x_np)


CASES = [
    # rows, cols, had_block, bits, container(0 nibble / 1 int8)
    (256, 256, 256, 4, 0),
    (1000, 768, 256, 4, 0),      # m = 3, ragged row count
    (333, 1280, 256, 3, 0),      # m = 5, INT3
    (77, 1792, 256, 8, 1),       # m = 7, INT8 container
    (300, 512, 512, 4, 0),
    (300, 1024, 1024, 3, 1),
    (300, 2048, 2048, 4, 0),
    (150, 4096, 4096, 4, 0),
    (64, 8192, 4096, 4, 1),      # two 4096-blocks per row
    (50, 2048, 1024, 8, 1),
    (200, 384, 128, 4, 0),       # generic path
    (200, 64, 16, 4, 0),
    (100, 24, 1, 4, 0),          # identity bypass
    (100, 96, 32, 3, 1),
    (5, 256, 256, 4, 0),
    (300, 1152, 128, 4, 0),      # 9 blocks of 128 (a transformer of width 1152): 36 threads per row
    (100, 4608, 128, 4, 1),      # 36 blocks of 128
    (130, 1152, 64, 3, 0),
    (257, 640, 32, 4, 0),        # one thread per block
    (64, 3200, 128, 4, 0),       # 100 threads per row: too wide for whole-warp CTAs, generic kernel
]


@pytest.mark.parametrize("rows,cols,had_block,bits,container", CASES)
def test_quant_matches_oracle(env, oracle, rows, cols, had_block, bits, container):
    torch, hq = env
    x = inputs.activations((rows, cols), outlier_count=max(1, cols // 100), outlier_scale=20.0, seed=rows + cols)
    x[rows // 2] = 0.0                                             # an all-zero row
    q, s, _ = run_quant(torch, hq, x, had_block, bits, container)
    u = oracle.transform(x, had_block)
    q_ref, s_ref, v = oracle.quantize(u, bits, want_v=True)
    assert s[rows // 2] == 1.0 and np.all(q[rows // 2] == 0)
    assert np.allclose(s, s_ref, rtol=SCALE_RTOL, atol=0)
    check_codes(q, q_ref, v, f"{rows}x{cols} n={had_block} b={bits}")


@pytest.mark.parametrize("dist", ["student_t3"])
@pytest.mark.parametrize("cols,had_block", [(512, 512), (2048, 2048)])
def test_quant_heavy_tail_inputs(env, oracle, dist, cols, had_block):
    torch, hq = env
    x = inputs.activations((512, cols), dist=dist, outlier_count=max(1, round(0.005 * cols)), outlier_scale=30.0, seed=3)
    for bits in (4, 3):
        q, s, _ = run_quant(torch, hq, x, had_block, bits, hq.HQ_CODES_NIBBLE)
        q_ref, s_ref, v = oracle.quantize(oracle.transform(x, had_block), bits, want_v=True)
        assert np.allclose(s, s_ref, rtol=SCALE_RTOL)
        check_codes(q, q_ref, v, f"t3 {cols} b={bits}")


def test_quant_worked_vectors_on_gpu(env):
    """Eq. 15 / Eq. 16 directly on the device: c*e_i -> +-qmax with the sign pattern of H_raw row i; c*1 -> qmax*e_1."""
    torch, hq = env
    n, c = 256, 3.0
    x = np.zeros((4, n), np.float32)
    x[0, 0] = c
    x[1, 5] = c
    x[2, :] = c
    x[3, n - 1] = -c
    q, s, _ = run_quant(torch, hq, x, n, 4, hq.HQ_CODES_NIBBLE)
    j = np.arange(n)
    sign = lambda i: 1 - 2 * (np.array([bin(int(v)).count("1") for v in (i & j)]) & 1)
    assert np.all(q[0] == 7)
    assert np.array_equal(q[1], 7 * sign(5))
    assert q[2, 0] == 7 and np.all(q[2, 1:] == 0)
    assert np.array_equal(q[3], -7 * sign(n - 1))
    assert np.allclose(s[[0, 1, 3]], c / 16 / 7, rtol=1e-6) and np.isclose(s[2], c * 16 / 7, rtol=1e-6)


@pytest.mark.parametrize("cols,had_block,bits,container", [(256, 256, 4, 0), (1024, 1024, 3, 0), (96, 32, 8, 1)])
def test_quant_static_scale_clamps(env, oracle, cols, had_block, bits, container):
    torch, hq = env
    x = inputs.activations((130, cols), outlier_count=2, outlier_scale=20.0, seed=11)
    u = oracle.transform(x, had_block)
    s0 = float(np.float32(np.abs(u).max() / oracle.qmax(bits) / 3.0))      # forces saturation of the largest values
    q, s, _ = run_quant(torch, hq, x, had_block, bits, container, static_scale=s0)
    q_ref, s_ref, v = oracle.quantize(u, bits, static_scale=s0, want_v=True)
    assert s[0] == np.float32(s0)
    assert q.min() == oracle.qmin(bits) and q.max() == oracle.qmax(bits)
    # saturated values are far from any boundary that matters; clip v so the tie rule looks at the clamp range only
    check_codes(q, q_ref, np.clip(v, oracle.qmin(bits) - 0.25, oracle.qmax(bits) + 0.25), "static")


def test_quant_bf16_input_and_row_pitch(env, oracle):
    torch, hq = env
    x = inputs.activations((200, 512), outlier_count=3, outlier_scale=20.0, seed=5)
    q, s, xb = run_quant(torch, hq, x, 256, 4, hq.HQ_CODES_NIBBLE, dtype=torch.bfloat16)
    q_ref, s_ref, v = oracle.quantize(oracle.transform(xb, 256), 4, want_v=True)
    assert np.allclose(s, s_ref, rtol=SCALE_RTOL)
    check_codes(q, q_ref, v, "bf16")
    q, s, _ = run_quant(torch, hq, x, 512, 4, hq.HQ_CODES_INT8, ldx=640)
    q_ref, s_ref, v = oracle.quantize(oracle.transform(x, 512), 4, want_v=True)
    assert np.allclose(s, s_ref, rtol=SCALE_RTOL)
    check_codes(q, q_ref, v, "pitch")


def test_quant_zero_rows_and_guard_bytes(env):
    torch, hq = env
    x = torch.zeros((0, 256), dtype=torch.float32, device="cuda")
    codes = torch.zeros((1, 128), dtype=torch.uint8, device="cuda")[:0]
    scales = torch.zeros((1,), dtype=torch.float32, device="cuda")
    hq.hq_hadamard_quant(x, 256, 4, codes, hq.HQ_CODES_NIBBLE, scales=scales)
    # rows beyond `rows` and bytes beyond the row must stay untouched
    xx = torch.randn((37, 256), device="cuda")
    buf = torch.full((64, 160), 0x5A, dtype=torch.uint8, device="cuda")
    sc = torch.full((64,), -1.0, device="cuda")
    hq.hq_hadamard_quant(xx, 256, 4, buf[:37], hq.HQ_CODES_NIBBLE, scales=sc[:37])
    torch.cuda.synchronize()
    assert bool((buf[37:] == 0x5A).all()) and bool((buf[:37, 128:] == 0x5A).all()) and bool((sc[37:] == -1).all())


def test_quant_full_size_sampled_rows(env, oracle):
    """The benchmark's largest transformer shape (32768 x 2048, block 2048): sampled rows against the oracle."""
    torch, hq = env
    cfg = inputs.config_transformer_linear("ff2")
    x = cfg["x"]
    rows, cols = x.shape
    q, s, _ = run_quant(torch, hq, x, cfg["had_block"], 4, hq.HQ_CODES_NIBBLE)
    idx = np.random.default_rng(0).choice(rows, size=96, replace=False)
    idx[:3] = [0, rows - 1, rows // 2]
    q_ref, s_ref, v = oracle.quantize(oracle.transform(x[idx], cfg["had_block"]), 4, want_v=True)
    assert np.allclose(s[idx], s_ref, rtol=SCALE_RTOL)
    check_codes(q[idx], q_ref, v, "ff2 sampled")
    # properties that hold for every row: codes in range, each row reaches +-qmax
    assert q.min() >= -7 and q.max() <= 7
    assert np.all(np.abs(q).max(axis=1) == 7)


@pytest.mark.parametrize("rows,c1,c2,had_block,dt,static", [
    (300, 256, 512, 256, "bf16", False),        # [h | skip] of the up-sampling path: the blocks of a row come from two tensors
    (130, 128, 128, 128, "f32", True),
    (64, 1024, 768, 256, "bf16", False),
])
def test_quant_of_a_concatenation_read_in_place(env, oracle, rows, c1, c2, had_block, dt, static):
    """hq_hadamard_quant with a second source: codes and scales are those of the oracle on the concatenated matrix, and
    bit-identical to the call on the written-out concatenation."""
    torch, hq = env
    a = inputs.activations((rows, c1), outlier_count=2, outlier_scale=10.0, seed=c1)
    b = inputs.activations((rows, c2), outlier_count=1, outlier_scale=5.0, seed=c2 + 1) * np.float32(0.5)
    ta, tb = torch.from_numpy(a).cuda(), torch.from_numpy(b).cuda()
    if dt == "bf16":
        ta, tb = ta.to(torch.bfloat16), tb.to(torch.bfloat16)
    cat = torch.cat([ta, tb], dim=1).contiguous()
    x = cat.float().cpu().numpy()
    cols = c1 + c2
    ss = torch.tensor([0.37], dtype=torch.float32, device="cuda") if static else None
    out = []
    for two in (True, False):
        codes = torch.full((rows, cols // 2), 0x5A, dtype=torch.uint8, device="cuda")
        scales = torch.full((rows,), -1.0, dtype=torch.float32, device="cuda")
        if two:
            hq.hq_hadamard_quant(ta, had_block, 4, codes, hq.HQ_CODES_NIBBLE, scales=scales, static_scale=ss, x2=tb)
        else:
            hq.hq_hadamard_quant(cat, had_block, 4, codes, hq.HQ_CODES_NIBBLE, scales=scales, static_scale=ss)
        torch.cuda.synchronize()
        out.append((codes.cpu().numpy(), scales.cpu().numpy()))
    assert np.array_equal(out[0][0], out[1][0]) and np.array_equal(out[0][1], out[1][1])
    u = oracle.transform(x, had_block)
    q_ref, s_ref, v = oracle.quantize(u, 4, static_scale=0.37 if static else None, want_v=True)
    if static:
        v = np.clip(v, oracle.qmin(4) - 0.25, oracle.qmax(4) + 0.25)
    else:
        assert np.allclose(out[0][1], s_ref, rtol=SCALE_RTOL, atol=0)
    check_codes(unpack_nibbles_np(out[0][0]), q_ref, v, f"concatenated input {rows}x({c1}+{c2}) {dt}")


def test_quant_of_a_concatenation_refuses_a_block_across_the_seam(env):
    torch, hq = env
    ta = torch.zeros((32, 128), dtype=torch.bfloat16, device="cuda")
    tb = torch.zeros((32, 384), dtype=torch.bfloat16, device="cuda")
    codes = torch.zeros((32, 256), dtype=torch.uint8, device="cuda")
    scales = torch.zeros((32,), dtype=torch.float32, device="cuda")
    with pytest.raises(hq.HqError):
        hq.hq_hadamard_quant(ta, 256, 4, codes, hq.HQ_CODES_NIBBLE, scales=scales, x2=tb)     # 128 is not a multiple of 256
