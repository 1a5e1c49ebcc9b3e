"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU, no CUDA library).

Each test states which plausible mistake it would catch.
"""
import itertools
import os

import numpy as np
import pytest

from paper_2512_05746_b200 import inputs

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _lines(name):
    with open(os.path.join(GOLD, name)) as f:
        return [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]


def closed_form_H(n):
    """Entry (i,j) of the Sylvester matrix is (-1)^popcount(i & j)."""
    i = np.arange(n)
    pc = np.vectorize(lambda v: bin(v).count("1"))(i[:, None] & i[None, :])
    return (1 - 2 * (pc & 1)).astype(np.int64)


def butterfly_fwht(v):
    """Textbook in-place radix-2 fast Walsh-Hadamard transform (natural/Sylvester order), unnormalised."""
    v = np.array(v, dtype=np.int64).copy()
    n, h = v.size, 1
    while h < n:
        for s in range(0, n, 2 * h):
            for j in range(s, s + h):
                a, b = v[j], v[j + h]
                v[j], v[j + h] = a + b, a - b
        h *= 2
    return v


# ------------------------------------------------------------------ Hadamard matrix (Eq. 5-7)

def test_hadamard_golden_small(oracle):
    rows = [[int(t) for t in ln.split()] for ln in _lines("hadamard_small.txt")]
    H1, H2 = np.array(rows[:2]), np.array(rows[2:6])
    assert np.array_equal(oracle.hadamard_raw(2), H1)
    assert np.array_equal(oracle.hadamard_raw(4), H2)
    assert np.array_equal(oracle.hadamard_raw(1), [[1]])


@pytest.mark.parametrize("n", [1, 2, 8, 64, 256, 1024])
def test_hadamard_orthogonal_symmetric_closed_form(oracle, n):
    H = oracle.hadamard_raw(n).astype(np.int64)
    assert set(np.unique(H)) <= {-1, 1}
    assert np.array_equal(H @ H.T, n * np.eye(n, dtype=np.int64))      # Eq. 6 times n (wrong sign block fails)
    assert np.array_equal(H, H.T)                                       # Eq. 6, symmetry
    assert np.array_equal(H, closed_form_H(n))                          # swapped blocks in the recurrence fail
    assert (H[0] == 1).all() and (H[:, 0] == 1).all()


def test_hadamard_rejects_non_power_of_two(oracle):
    with pytest.raises(ValueError):
        oracle.hadamard_raw(12)


# ------------------------------------------------------------------ transform (Eq. 10, 15, 16)

def test_transform_worked_vectors_golden(oracle):
    for ln in _lines("worked_vectors.txt"):
        k, xin, want = [p.strip() for p in ln.split("|")]
        x = np.array([float(t) for t in xin.split()])
        w = np.array([float(t) for t in want.split()])
        assert x.size == 2 ** int(k)
        got = oracle.transform(x[None, :], x.size)[0]
        assert np.allclose(got, w, rtol=0, atol=1e-15)


@pytest.mark.parametrize("k", [4, 8, 9, 11])
def test_transform_basis_vectors(oracle, k):
    n = 2 ** k
    c = 3.25
    Hc = closed_form_H(n)
    for i in (0, 1, n // 2 + 3, n - 1):
        e = np.zeros((1, n)); e[0, i] = c
        u = oracle.transform(e, n)[0]
        assert np.allclose(np.abs(u), c * 2.0 ** (-k / 2), rtol=1e-15)       # Eq. 15: flat magnitude
        assert np.array_equal(np.sign(u), Hc[i])                              # sign pattern = row i of H_raw
    u = oracle.transform(np.full((1, n), c), n)[0]                            # Eq. 16
    assert np.isclose(u[0], c * 2.0 ** (k / 2), rtol=1e-15) and np.all(u[1:] == 0)


@pytest.mark.parametrize("n", [2, 4, 16, 64])
def test_transform_equals_butterfly_on_integers(oracle, n):
    rng = np.random.default_rng(n)
    x = rng.integers(-50, 50, size=(5, n))
    u = oracle.transform(x.astype(np.float64), n) * np.sqrt(n)               # back to H_raw
    for r in range(x.shape[0]):
        assert np.array_equal(np.rint(u[r]).astype(np.int64), butterfly_fwht(x[r]))
        assert np.allclose(u[r], np.rint(u[r]), atol=1e-9)


@pytest.mark.parametrize("n,m", [(16, 1), (64, 3), (256, 5), (512, 2)])
def test_transform_involution_parseval_blockdiag(oracle, n, m):
    rng = np.random.default_rng(7)
    x = rng.standard_normal((6, n * m))
    u = oracle.transform(x, n)
    assert np.allclose(oracle.transform(u, n), x, atol=1e-12)                 # H^2 = I (after Eq. 10)
    assert np.allclose(np.linalg.norm(u, axis=1), np.linalg.norm(x, axis=1), rtol=1e-13)
    for b in range(m):                                                        # blocks are independent
        ub = oracle.transform(x[:, b * n:(b + 1) * n], n)
        assert np.array_equal(ub, u[:, b * n:(b + 1) * n])
    # a block transform is NOT the full-width transform (would catch ignoring had_block)
    if m > 1 and (n * m) & (n * m - 1) == 0:
        assert not np.allclose(oracle.transform(x, n * m), u)


def test_transform_identity_bypass_and_errors(oracle):
    x = np.random.default_rng(0).standard_normal((3, 24))
    assert np.array_equal(oracle.transform(x, 1), x)
    assert np.array_equal(oracle.transform(x, 0), x)
    with pytest.raises(ValueError):
        oracle.transform(x, 16)        # 24 is not a multiple of 16
    with pytest.raises(ValueError):
        oracle.transform(x, 12)        # not a power of two


# ------------------------------------------------------------------ quantizer (Eq. 3)

def test_quantizer_golden_cases(oracle):
    for ln in _lines("quantizer_cases.txt"):
        bits, scale, xin, want = [p.strip() for p in ln.split("|")]
        x = np.array([[float(t) for t in xin.split()]])
        q, s = oracle.quantize(x, int(bits), static_scale=float(scale))
        assert s.shape == (1,) and s[0] == np.float32(scale)
        assert q[0].tolist() == [int(t) for t in want.split()], ln


@pytest.mark.parametrize("bits", [3, 4, 8])
def test_quantizer_dynamic_error_bound(oracle, bits):
    rng = np.random.default_rng(bits)
    u = rng.standard_normal((64, 96)) * rng.uniform(0.1, 30, size=(64, 1))
    q, s, v = oracle.quantize(u, bits, want_v=True)
    qm = oracle.qmax(bits)
    s64 = s.astype(np.float64)[:, None]
    assert np.all(np.abs(u - s64 * q) <= s64 / 2 * (1 + 1e-6))               # nothing clamps in dynamic mode
    assert q.max() <= qm and q.min() >= -qm                                   # qmin unreachable dynamically
    am = np.abs(u).argmax(axis=1)
    assert np.all(np.abs(q[np.arange(64), am]) == qm)                         # absmax element -> +-qmax
    assert np.allclose(s64[:, 0], np.abs(u).max(axis=1) / qm, rtol=1e-7)      # scale = absmax / qmax
    assert np.allclose(v, u / s64)


def test_quantizer_static_clamps_and_zero_row(oracle):
    u = np.array([[0.0, 0.0, 0.0, 0.0], [10.0, -10.0, 0.3, -0.3]])
    q, s = oracle.quantize(u, 4)
    assert s[0] == 1.0 and np.all(q[0] == 0)
    q, s = oracle.quantize(u, 4, static_scale=0.5)
    assert q[1].tolist() == [7, -8, 1, -1]                                    # 0.6 -> 1; clamp to [-8, 7]
    inside = np.abs(u / 0.5) <= 7
    assert np.all(np.abs(u - 0.5 * q)[inside] <= 0.25 + 1e-12)


def test_pack_unpack_nibbles(oracle):
    allv = np.arange(-8, 8, dtype=np.int8)
    pairs = np.array(list(itertools.product(allv, allv)), dtype=np.int8).reshape(-1)
    packed = oracle.pack_nibbles(pairs)
    assert np.array_equal(oracle.unpack_nibbles(packed), pairs)
    assert oracle.pack_nibbles(np.array([1, -1], np.int8)).tolist() == [0xF1]   # element 0 in the low nibble
    assert oracle.pack_nibbles(np.array([-8, 7], np.int8)).tolist() == [0x78]
    assert oracle.unpack_nibbles(np.array([0x8F], np.uint8)).tolist() == [-1, -8]


def test_limb_split(oracle):
    B = np.arange(-32768 - 128, 127 * 256 + 127 + 1, dtype=np.int32)     # the whole representable range
    hi, lo = oracle.limb_split(B)
    assert np.array_equal(256 * hi.astype(np.int64) + lo, B)
    assert lo.min() == -128 and lo.max() == 127
    assert oracle.limb_split(np.array([127, 128, -128, -129], np.int32))[0].tolist() == [0, 1, 0, -1]
    with pytest.raises(ValueError):
        oracle.limb_split(np.array([32640], np.int32))      # hi would be 128


# ------------------------------------------------------------------ weights (Eq. 3, Eq. 12)

def test_weight_quantize_per_channel(oracle):
    w = inputs.weights((8, 3, 3, 16), seed=3)
    w[2] = 0
    w_int, s_w = oracle.weight_quantize(w, 4)
    assert s_w[2] == 1.0 and np.all(w_int[2] == 0)
    flat = w.reshape(8, -1).astype(np.float64)
    for o in (0, 1, 3, 7):
        assert np.isclose(s_w[o], np.abs(flat[o]).max() / 7, rtol=1e-7)
        assert np.abs(w_int[o]).max() == 7
        assert np.all(np.abs(flat[o] - np.float64(s_w[o]) * w_int[o].reshape(-1)) <= s_w[o] / 2 * (1 + 1e-6))


@pytest.mark.parametrize("n,C", [(4, 4), (16, 48), (64, 64)])
def test_weight_fold_is_H_times_W_and_associative(oracle, n, C):
    rng = np.random.default_rng(n)
    w_int = rng.integers(-8, 8, size=(5, 2, C)).astype(np.int32)
    B = oracle.weight_fold(w_int, n)
    H = closed_form_H(n)
    for b in range(C // n):
        blk = slice(b * n, (b + 1) * n)
        assert np.array_equal(B[..., blk], np.einsum("ij,otj->oti", H, w_int[..., blk].astype(np.int64)))
    # Eq. 12: ((XH)_int * H_raw) * W_int == (XH)_int * (H_raw * W_int)
    q = inputs.codes((7, C), 4, seed=n)
    Hbd = np.kron(np.eye(C // n, dtype=np.int64), H)
    left = (q.astype(np.int64) @ Hbd) @ w_int[:, 0, :].astype(np.int64).T
    right = oracle.gemm_int(q, B[:, 0, :])
    assert np.array_equal(left, right)
    assert np.array_equal(oracle.weight_fold(w_int, 1), w_int)


def test_weight_double_close_to_HtW(oracle):
    w = inputs.weights((6, 1, 64), seed=5).astype(np.float64)
    B, s_w = oracle.weight_double(w, 8, 64)
    Hn = closed_form_H(64) / 8.0
    target = np.einsum("jc,otj->otc", Hn, w)       # (H^T W)[c, o]
    assert np.all(np.abs(target - s_w[:, None, None].astype(np.float64) * B) <= s_w[:, None, None] / 2 * (1 + 1e-6))


# ------------------------------------------------------------------ integer GEMM / conv (Eq. 12, 14)

def test_gemm_int_bruteforce_and_permutation(oracle):
    q = inputs.codes((5, 12), 4, seed=1)
    B = np.random.default_rng(2).integers(-2000, 2000, size=(4, 12)).astype(np.int32)
    acc = oracle.gemm_int(q, B)
    for m in range(5):
        for o in range(4):
            assert acc[m, o] == sum(int(q[m, k]) * int(B[o, k]) for k in range(12))
    perm = np.random.default_rng(3).permutation(12)
    assert np.array_equal(oracle.gemm_int(q[:, perm], B[:, perm]), acc)
    # not symmetric in its operands' roles: a transposed B must differ
    q2 = inputs.codes((4, 4), 4, seed=9)
    B2 = np.arange(16, dtype=np.int32).reshape(4, 4)
    assert np.array_equal(oracle.gemm_int(q2, B2), q2.astype(np.int64) @ B2.T.astype(np.int64))
    assert not np.array_equal(oracle.gemm_int(q2, B2), q2.astype(np.int64) @ B2.astype(np.int64))


def test_gemm_int_overflow_detected(oracle):
    q = np.full((1, 4096), -8, np.int8)
    B = np.full((1, 4096), -70000, np.int32)
    with pytest.raises(OverflowError):
        oracle.gemm_int(q, B)


def _im2col(q, R, S, stride, pad):
    Nb, H, W, C = q.shape
    Ho, Wo = (H + 2 * pad - R) // stride + 1, (W + 2 * pad - S) // stride + 1
    qp = np.zeros((Nb, H + 2 * pad, W + 2 * pad, C), q.dtype)
    qp[:, pad:pad + H, pad:pad + W] = q
    cols = np.empty((Nb, Ho, Wo, R, S, C), q.dtype)
    for r in range(R):
        for s in range(S):
            cols[:, :, :, r, s] = qp[:, r:r + stride * Ho:stride, s:s + stride * Wo:stride]
    return cols.reshape(Nb * Ho * Wo, R * S * C), (Nb, Ho, Wo)


@pytest.mark.parametrize("R,stride,pad,H,W", [(3, 1, 1, 6, 5), (3, 2, 1, 8, 6), (1, 1, 0, 4, 4), (3, 1, 0, 5, 5),
                                              (3, 2, 1, 7, 5)])
def test_conv_equals_im2col_gemm(oracle, R, stride, pad, H, W):
    C, Cout = 8, 6
    q = inputs.codes((2, H, W, C), 4, seed=H * W)
    B = np.random.default_rng(4).integers(-100, 100, size=(Cout, R, R, C)).astype(np.int32)
    acc = oracle.conv2d_int(q, B, stride, pad)
    cols, oshape = _im2col(q, R, R, stride, pad)
    ref = oracle.gemm_int(cols, B.reshape(Cout, -1)).reshape(*oshape, Cout)
    assert np.array_equal(acc, ref)
    if stride == 2:
        full = oracle.conv2d_int(q, B, 1, pad)
        assert np.array_equal(acc, full[:, ::2, ::2][:, :acc.shape[1], :acc.shape[2]])


def test_conv_bruteforce_tiny_and_1x1_is_linear(oracle):
    q = inputs.codes((1, 3, 3, 2), 4, seed=11)
    B = np.random.default_rng(5).integers(-9, 9, size=(2, 3, 3, 2)).astype(np.int32)
    acc = oracle.conv2d_int(q, B, 1, 1)
    for ho in range(3):
        for wo in range(3):
            for co in range(2):
                t = 0
                for r in range(3):
                    for s in range(3):
                        hi, wi = ho + r - 1, wo + s - 1
                        if 0 <= hi < 3 and 0 <= wi < 3:
                            t += sum(int(q[0, hi, wi, c]) * int(B[co, r, s, c]) for c in range(2))
                assert acc[0, ho, wo, co] == t
    q1 = inputs.codes((2, 4, 4, 8), 4, seed=12)
    B1 = np.random.default_rng(6).integers(-9, 9, size=(5, 1, 1, 8)).astype(np.int32)
    assert np.array_equal(oracle.conv2d_int(q1, B1, 1, 0).reshape(-1, 5), oracle.gemm_int(q1.reshape(-1, 8), B1.reshape(5, 8)))


# ------------------------------------------------------------------ rescale

def test_dequant_hand_values(oracle):
    acc = np.array([[10, -4], [3, 0]], np.int64)
    y = oracle.dequant(acc, np.array([0.5, 2.0], np.float32), np.array([0.25, 1.0], np.float32),
                       np.array([1.0, -1.0], np.float32), 0.5)
    assert np.array_equal(y, [[0.5 * 0.5 * 0.25 * 10 + 1, 0.5 * 0.5 * 1.0 * -4 - 1], [0.5 * 2 * 0.25 * 3 + 1, -1.0]])
    y = oracle.dequant(acc, np.array([2.0], np.float32), np.array([1.0, 1.0], np.float32), None, 1.0)
    assert np.array_equal(y, 2.0 * acc)


def test_perpixel_conv_dequant(oracle):
    q = inputs.codes((2, 5, 4, 8), 4, seed=21)
    B = np.random.default_rng(8).integers(-60, 60, size=(3, 3, 3, 8)).astype(np.int32)
    s_w = inputs.positive_scales(3, seed=1)
    b = inputs.bias(3, seed=1)
    # equal scales factor out of the sum over taps
    s_a = np.full(2 * 5 * 4, 0.125, np.float32)
    y = oracle.conv2d_dequant_perpixel(q, s_a, B, 1, 1, s_w, b, 0.5)
    ref = oracle.dequant(oracle.conv2d_int(q, B, 1, 1), np.array([0.125], np.float32), s_w, b, 0.5)
    assert np.allclose(y, ref, rtol=1e-13, atol=1e-13)
    # distinct scales: scaling the codes of one pixel by 2 (exactly) equals doubling that pixel's scale
    s_a = inputs.positive_scales(2 * 5 * 4, seed=2)
    qs = np.clip(q, -3, 3).astype(np.int8)                      # leave room to double one pixel
    y1 = oracle.conv2d_dequant_perpixel(qs, s_a, B, 1, 1, s_w, None, 1.0)
    q2, s2 = qs.copy(), s_a.copy()
    q2[1, 2, 3] *= 2
    s2[(1 * 5 + 2) * 4 + 3] /= 2
    y2 = oracle.conv2d_dequant_perpixel(q2, s2, B, 1, 1, s_w, None, 1.0)
    assert np.allclose(y1, y2, rtol=1e-12, atol=1e-12)
    # brute force: it equals the fp64 convolution of the dequantized activations with the integer weights
    xhat = qs.astype(np.float64) * s_a.astype(np.float64).reshape(2, 5, 4, 1)
    cols, oshape = _im2col(xhat, 3, 3, 1, 1)
    ref = (cols @ B.reshape(3, -1).T.astype(np.float64)).reshape(*oshape, 3) * s_w.astype(np.float64)
    assert np.allclose(y1, ref, rtol=1e-12, atol=1e-12)


# ------------------------------------------------------------------ whole layer (Eq. 11-12)

@pytest.mark.parametrize("n,m", [(16, 1), (64, 2), (256, 1)])
def test_folded_layer_recovers_X_times_What_without_rounding(oracle, n, m):
    """If XH/S is already integral nothing is lost by Eq. 3, and Eq. 12 must give X * (S_w W_int) exactly.
    Fails if H is applied once instead of twice, if 2^(-k/2) is dropped or doubled, or if the fold uses the
    wrong operand order."""
    K, N, M = n * m, 10, 9
    rng = np.random.default_rng(n + m)
    q0 = rng.integers(-7, 8, size=(M, K)).astype(np.int8)
    q0[:, 0] = 7                                                   # absmax -> scale = s exactly
    s = (2.0 ** rng.integers(-4, 3, size=(M, 1))).astype(np.float64)
    Hn = np.kron(np.eye(m), closed_form_H(n)) / np.sqrt(n)
    X = (s * q0) @ Hn                                              # inverse transform of the codes (Eq. 11)
    w = inputs.weights((N, K), seed=n)
    out = oracle.qlinear(X, w, None, a_bits=4, w_bits=4, had_block=n, weight_mode="folded")
    assert np.array_equal(out["q"], q0)
    assert np.allclose(out["s_a"], s[:, 0], rtol=1e-6)
    W_hat = out["s_w"].astype(np.float64)[:, None] * oracle.weight_quantize(w, 4)[0]
    assert np.allclose(out["y"], X @ W_hat.T, rtol=1e-6, atol=1e-9)
    # the plain (unfolded) product with the same codes is a different number: the two readings are distinguishable
    plain = oracle.qlinear(X, w, None, a_bits=4, w_bits=4, had_block=n, weight_mode="plain")
    assert not np.allclose(plain["y"], X @ W_hat.T, rtol=1e-2, atol=1e-6)


def test_double_hadamard_layer_approximates_XW(oracle):
    cfg = inputs.config_linear_small(0)
    x, w = cfg["x"][:64].astype(np.float64), cfg["w"]
    ref = x @ w.astype(np.float64).T
    out = oracle.qlinear(x, w, None, a_bits=8, w_bits=8, had_block=256, weight_mode="double")
    err = np.linalg.norm(out["y"] - ref) / np.linalg.norm(ref)
    assert err < 0.03


def test_transform_lowers_layer_error_on_outlier_inputs(oracle):
    """Direction only: with a few dominant channels, quantizing XH loses less than quantizing X."""
    cfg = inputs.config_linear_small(0)
    x, w = cfg["x"][:128].astype(np.float64), cfg["w"]
    W_hat = oracle.weight_quantize(w, 4)
    ref = x @ (W_hat[1].astype(np.float64)[:, None] * W_hat[0]).T
    with_h = oracle.qlinear(x, w, None, a_bits=4, w_bits=4, had_block=256, weight_mode="folded")["y"]
    without = oracle.qlinear(x, w, None, a_bits=4, w_bits=4, had_block=1, weight_mode="folded")["y"]
    e_h = np.linalg.norm(with_h - ref) / np.linalg.norm(ref)
    e_0 = np.linalg.norm(without - ref) / np.linalg.norm(ref)
    assert e_h < e_0
    # crest factor per token drops
    u = oracle.transform(x, 256)
    crest = lambda a: (np.abs(a).max(axis=1) / np.sqrt((a ** 2).mean(axis=1))).mean()
    assert crest(u) < crest(x)


def test_qconv_layer_consistency(oracle):
    """1x1 conv with per-pixel scales is the linear layer on flattened pixels; static-scale 3x3 conv has one drain."""
    x = inputs.activations((1, 4, 4, 32), outlier_count=1, outlier_scale=20.0, seed=4)
    w1 = inputs.weights((8, 1, 1, 32), seed=4)
    b = inputs.bias(8, seed=4)
    c = oracle.qconv(x, w1, b, a_bits=4, w_bits=4, had_block=32, stride=1, pad=0)
    l = oracle.qlinear(x.reshape(16, 32), w1.reshape(8, 32), b, a_bits=4, w_bits=4, had_block=32)
    assert np.allclose(c["y"].reshape(16, 8), l["y"], rtol=1e-13, atol=1e-13)
    w3 = inputs.weights((8, 3, 3, 32), seed=5)
    cs = oracle.qconv(x, w3, b, a_bits=3, w_bits=4, had_block=32, stride=1, pad=1, static_scale=0.4)
    assert cs["q"].min() >= -4 and cs["q"].max() <= 3
    ref = oracle.dequant(cs["acc"], np.array([0.4], np.float32), cs["s_w"], b, cs["alpha"])
    assert np.array_equal(cs["y"], ref)


# ------------------------------------------------------------------ width-axis convolution (Eq. 13-14 as stated)

@pytest.mark.parametrize("W,n", [(8, 8), (16, 4), (32, 16), (12, 4)])
def test_width_transform_is_the_row_transform_on_the_moved_axis(oracle, W, n):
    """Transforming along w of NHWC must equal the (already pinned) last-axis transform of the tensor with w moved
    last -- the reshape to (B*Cin*h) x w of the paper.  A wrong stride or a transposed H fails here."""
    x = inputs.activations((2, 3, W, 5), outlier_count=1, outlier_scale=20.0, seed=W + n).astype(np.float64)
    got = oracle.transform_width(x, n)
    want = np.moveaxis(oracle.transform(np.moveaxis(x, 2, 3), n), 3, 2)
    assert np.allclose(got, want, rtol=0, atol=1e-12)
    assert np.allclose(oracle.transform_width(got, n), x, rtol=0, atol=1e-12)      # H_c H_c = I
    with pytest.raises(ValueError):
        oracle.transform_width(x, 2 * W)                                            # block does not divide w


@pytest.mark.parametrize("W,n", [(8, 8), (16, 4), (32, 16)])
def test_codes_inverse_width_closed_form_and_involution(oracle, W, n):
    q = inputs.codes((2, 3, W, 4), 4, seed=W)
    z = oracle.codes_inverse_width(q, n)
    Hc = closed_form_H(n)
    want = np.einsum("nhbic,ij->nhbjc", q.astype(np.int64).reshape(2, 3, W // n, n, 4), Hc).reshape(2, 3, W, 4)
    assert np.array_equal(z, want)
    assert np.abs(z).max() <= n * 8
    # H_raw H_raw = n I: applying the integer factor twice returns n times the codes
    zz = np.einsum("nhbic,ij->nhbjc", z.astype(np.int64).reshape(2, 3, W // n, n, 4), Hc).reshape(2, 3, W, 4)
    assert np.array_equal(zz, n * q.astype(np.int64))


def test_conv2d_int_z_equals_conv2d_int_on_small_values(oracle):
    q = inputs.codes((2, 6, 5, 8), 4, seed=1)
    B = inputs.codes((4, 3, 3, 8), 4, seed=2).astype(np.int32)
    for stride, pad in ((1, 1), (2, 1), (1, 0)):
        assert np.array_equal(oracle.conv2d_int_z(q.astype(np.int32), B, stride, pad), oracle.conv2d_int(q, B, stride, pad))


def test_width_conv_layer_is_conv_of_dequantized_activations(oracle):
    """Eq. 13 then Eq. 14: the layer output equals an ordinary float convolution of x_hat = S (XH)_int H_c with
    W_hat = S_w W_int (im2col in numpy), and x_hat is within S/2 * sqrt(n) ... of x where nothing clamps."""
    x = inputs.activations((2, 6, 16, 8), outlier_count=1, outlier_scale=10.0, seed=3).astype(np.float64)
    w = inputs.weights((5, 3, 3, 8), seed=4)
    b = inputs.bias(5, seed=5)
    n, S = 8, 0.9
    out = oracle.qconv_width(x, w, b, a_bits=4, w_bits=4, had_block_w=n, stride=1, pad=1, static_scale=S)
    x_hat = np.float32(S) * oracle.transform_width(out["q"].astype(np.float64), n)      # S * q * H_c (orthonormal)
    assert np.allclose(x_hat, np.float64(np.float32(S)) * 2.0 ** (-0.5 * np.log2(n)) * out["z"], rtol=0, atol=1e-12)
    w_hat = out["s_w"].astype(np.float64)[:, None, None, None] * out["B"]
    xp = np.pad(x_hat, ((0, 0), (1, 1), (1, 1), (0, 0)))
    y = np.zeros((2, 6, 16, 5))
    for r in range(3):
        for s in range(3):
            y += np.einsum("nhwc,oc->nhwo", xp[:, r:r + 6, s:s + 16, :], w_hat[:, r, s, :])
    assert np.allclose(out["y"], y + b, rtol=1e-12, atol=1e-12)
    # inside the clamp range the transformed values are within S/2 of their codes (Eq. 3), hence by Parseval the
    # recovered activations are within S/2 * sqrt(n) of the originals per block
    inside = np.abs(out["v"]) <= 7
    assert np.all(np.abs(out["u"] - np.float32(S) * out["q"])[inside] <= 0.5 * np.float32(S) + 1e-12)


def test_width_conv_recovers_plain_conv_when_quantization_is_fine(oracle):
    """With 8-bit codes and a scale that nothing clamps at, the layer approaches Conv(x, W_hat): the error shrinks
    with the scale (direction check of H_c H_c^T = I in Eq. 14)."""
    x = inputs.activations((1, 5, 8, 4), seed=6).astype(np.float64)
    w = inputs.weights((3, 3, 3, 4), seed=7)
    errs = []
    for S in (0.2, 0.05):
        out = oracle.qconv_width(x, w, None, a_bits=8, w_bits=8, had_block_w=8, stride=1, pad=1, static_scale=S)
        w_hat = out["s_w"].astype(np.float64)[:, None, None, None] * out["B"]
        xp = np.pad(x, ((0, 0), (1, 1), (1, 1), (0, 0)))
        y = np.zeros((1, 5, 8, 3))
        for r in range(3):
            for s in range(3):
                y += np.einsum("nhwc,oc->nhwo", xp[:, r:r + 5, s:s + 8, :], w_hat[:, r, s, :])
        errs.append(np.abs(out["y"] - y).max())
    assert errs[1] < errs[0] and errs[1] < 0.02


# ------------------------------------------------------------------ GroupNorm + SiLU prologue

def test_groupnorm_silu_against_library_routine(oracle):
    """The written-out definition against torch's group_norm + silu on the CPU in fp64 (a library routine), plus two
    closed forms: a constant input gives silu(beta); with gamma = 1, beta = 0 each group of the normalised tensor has
    mean 0 and variance 1 / (1 + eps / var)."""
    import torch
    rng = np.random.default_rng(0)
    x = rng.standard_normal((3, 5, 4, 24)) * 3.0 + 1.5
    gamma, beta = rng.standard_normal(24), rng.standard_normal(24)
    got = oracle.groupnorm_silu(x, 6, gamma, beta, eps=1e-5)
    xt = torch.from_numpy(x).permute(0, 3, 1, 2)                                  # NCHW for the library
    want = torch.nn.functional.silu(torch.nn.functional.group_norm(xt, 6, torch.from_numpy(gamma), torch.from_numpy(beta), 1e-5))
    assert np.allclose(got, want.permute(0, 2, 3, 1).numpy(), rtol=1e-12, atol=1e-12)
    const = oracle.groupnorm_silu(np.full((1, 2, 2, 8), 7.0), 2, gamma[:8], beta[:8], eps=1e-6)
    assert np.allclose(const, beta[:8] / (1 + np.exp(-beta[:8])), atol=1e-9)
    with pytest.raises(ValueError):
        oracle.groupnorm_silu(x, 5, gamma, beta)                                   # 24 channels do not split into 5 groups


# ------------------------------------------------------------------ LayerNorm + per-sample affine prologue

def test_layernorm_affine_against_library_routine(oracle):
    """The written-out definition against torch's layer_norm on the CPU in fp64 (a library routine) followed by the
    modulation y * (1 + scale) + shift of a diffusion-transformer block, plus closed forms: without an affine every row
    has mean 0 and variance 1 / (1 + eps / var); a constant row gives the bias; a per-row shift and a positive per-row
    scale of x leave the result unchanged (up to the eps term)."""
    import torch
    rng = np.random.default_rng(1)
    rows, cols, rpg = 12, 40, 4
    x = rng.standard_normal((rows, cols)) * 2.5 + 0.7
    scale, shift = rng.standard_normal((3, cols)) * 0.3, rng.standard_normal((3, cols))
    got = oracle.layernorm_affine(x, 1.0 + scale, shift, rows_per_group=rpg, eps=1e-6)
    ln = torch.nn.functional.layer_norm(torch.from_numpy(x), (cols,), None, None, 1e-6).numpy()
    want = ln * (1.0 + np.repeat(scale, rpg, axis=0)) + np.repeat(shift, rpg, axis=0)
    assert np.allclose(got, want, rtol=1e-12, atol=1e-12)
    plain = oracle.layernorm_affine(x, eps=1e-6)
    assert np.allclose(plain.mean(axis=1), 0.0, atol=1e-12)
    assert np.allclose(plain.var(axis=1), 1.0 / (1.0 + 1e-6 / x.var(axis=1)), rtol=1e-12)
    const = oracle.layernorm_affine(np.full((2, cols), 3.0), np.ones((1, cols)), shift[:1], eps=1e-6)
    assert np.allclose(const, np.repeat(shift[:1], 2, axis=0), atol=1e-12)
    moved = oracle.layernorm_affine(x * 3.0 + rng.standard_normal((rows, 1)), 1.0 + scale, shift, rows_per_group=rpg, eps=1e-12)
    assert np.allclose(moved, oracle.layernorm_affine(x, 1.0 + scale, shift, rows_per_group=rpg, eps=1e-12), atol=1e-9)
    with pytest.raises(ValueError):
        oracle.layernorm_affine(x, scale[:2], shift, rows_per_group=rpg)          # 12 rows in groups of 4 need 3 vectors


# ------------------------------------------------------------------ Single vs Double Hadamard on the weight side

def test_double_hadamard_raises_error_of_low_outlier_weights_and_lowers_it_for_outlier_weights(oracle):
    """Direction of the "Single Hadamard Transformation" paragraph and of Table 6 on synthetic weights: transforming
    weights that have few outliers (bounded, or a flat component: Eq. 16) adds outliers and raises their 4-bit
    quantization error, and with it the layer error of the Double scheme; weights that do have outlier input channels
    gain from the transform; iid Gaussian weights are indifferent.  A transform applied along the wrong weight axis,
    or a Double scheme that reuses the scales of W, changes these directions."""
    from oracle import weight_error_study as st
    rows = {r["family"]: r for r in st.study(w_bits=4, a_bits=4, had_block=256)}
    g, u, o, x = rows["gaussian"], rows["uniform"], rows["offset"], rows["outlier-in"]
    assert 0.9 < g["werr_double"] / g["werr_single"] < 1.1
    assert abs(g["layer_double"] - g["layer_single"]) < 0.05 * g["layer_single"]
    for r in (u, o):
        assert r["werr_double"] > 2.0 * r["werr_single"]
        assert r["layer_double"] > 1.2 * r["layer_single"]
        assert r["after"]["kurtosis"] > r["before"]["kurtosis"]
        assert r["after"]["max_over_sigma"] > 1.5 * r["before"]["max_over_sigma"]
    assert u["before"]["beyond_3sigma"] == 0.0 and u["after"]["beyond_3sigma"] > 1e-3
    assert x["werr_double"] < 0.2 * x["werr_single"]
    assert x["layer_double"] < 0.5 * x["layer_single"]
    # Eq. 16 on the weight side: the flat component c * 1 of a channel lands in one coefficient, c * 2^(k/2)
    w = st.make_weights("offset")
    hw = oracle.transform(w.astype(np.float64), 256)
    assert np.allclose(hw[:, 0], 16.0 * w.astype(np.float64).mean(axis=1), rtol=1e-12, atol=1e-12)
