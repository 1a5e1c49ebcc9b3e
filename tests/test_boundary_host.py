"""CPU-only checks of the C-ABI library: it loads, exports what include/hq.h declares, validates arguments
before touching the GPU, and its offline weight preparation agrees with the oracle."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2512_05746_b200 import inputs
from hq_testutil import decode_blob

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def hq():
    from paper_2512_05746_b200 import build
    build.build()
    from paper_2512_05746_b200 import binding
    return binding


def test_library_exports_every_declared_symbol(hq):
    text = open(os.path.join(ROOT, "include", "hq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(hq_[a-z0-9_]+)\s*\(", text))
    assert declared, "no declarations found"
    assert declared == set(hq.EXPORTS)
    for name in declared:
        assert hasattr(hq.lib, name), name
    assert hq.hq_version() >= 100
    assert hq.status_string(0) == "ok" and "overflow" in hq.status_string(6)


def test_check_status_decodes_timeout_word(hq):
    ok = np.zeros(1, np.int32)
    bad = np.array([0x300], np.int32)
    assert hq.lib.hq_check_status(ok.ctypes.data_as(C.c_void_p)) == 0
    assert hq.lib.hq_check_status(bad.ctypes.data_as(C.c_void_p)) == 8
    assert hq.lib.hq_check_status(None) == 1


def test_argument_validation_without_gpu(hq):
    L = hq.lib
    fake = C.c_void_p(0x1000)
    # NULL pointers
    assert L.hq_hadamard_quant(None, 0, 4, 256, 256, 256, 4, 0, None, fake, 0, 128, fake, None) == 1
    # cols not a multiple of the block / block not a power of two
    assert L.hq_hadamard_quant(fake, 0, 4, 384, 384, 256, 4, 0, None, fake, 0, 192, fake, None) == 2
    assert L.hq_hadamard_quant(fake, 0, 4, 384, 384, 96, 4, 0, None, fake, 0, 192, fake, None) == 2
    # bits outside {3,4,8}; 8-bit codes in a nibble container
    assert L.hq_hadamard_quant(fake, 0, 4, 256, 256, 256, 5, 0, None, fake, 0, 128, fake, None) == 1
    assert L.hq_hadamard_quant(fake, 0, 4, 256, 256, 256, 8, 0, None, fake, 0, 128, fake, None) == 2
    # static mode without a scale
    assert L.hq_hadamard_quant(fake, 0, 4, 256, 256, 256, 4, 1, None, fake, 0, 128, fake, None) == 1
    # zero rows is a no-op
    assert L.hq_hadamard_quant(fake, 0, 0, 256, 256, 256, 4, 0, None, fake, 0, 128, fake, None) == 0
    out = C.c_size_t(0)
    assert L.hq_workspace_size(128, 256, 0, C.byref(out)) == 0 and out.value >= 128 * 128 + 128 * 4
    assert L.hq_workspace_size(128, 256, 1, C.byref(out)) == 0 and out.value >= 128 * 256 + 128 * 4
    assert L.hq_workspace_size(128, 0, 0, C.byref(out)) == 2


def test_gemm_validation_without_gpu(hq):
    w = inputs.weights((256, 256), seed=0)
    pw = hq.hq_weight_prepare(w, 4, 256, hq.HQ_W_FOLDED, hq.HQ_CODES_INT8)
    L = hq.lib
    fake = C.c_void_p(0x1000)
    d = C.byref(pw.desc)
    # container mismatch with the blob
    assert L.hq_qgemm(fake, 0, 4, 128, 256, 128, d, fake, fake, 0, fake, None, 1.0, fake, None, 1, 256, None, None) == 2
    # K mismatch
    assert L.hq_qgemm(fake, 1, 4, 128, 512, 512, d, fake, fake, 0, fake, None, 1.0, fake, None, 1, 256, None, None) == 2
    # neither output requested
    assert L.hq_qgemm(fake, 1, 4, 128, 256, 256, d, fake, fake, 0, fake, None, 1.0, None, None, 1, 256, None, None) == 1
    # 8-bit activations against 2-limb folded weights whose integers are large: K * 128 * max|B| >= 2^31
    w8 = np.ones((128, 4096), np.float32)
    pw8 = hq.hq_weight_prepare(w8, 8, 256, hq.HQ_W_FOLDED, hq.HQ_CODES_INT8)
    assert L.hq_qgemm(fake, 1, 8, 128, 4096, 4096, C.byref(pw8.desc), fake, fake, 0, fake, None, 1.0, fake, None, 1,
                      128, None, None) == 6
    # conv: unsupported filter size
    wc = inputs.weights((128, 3, 3, 128), seed=2)
    pwc = hq.hq_weight_prepare(wc, 4, 128, hq.HQ_W_PLAIN, hq.HQ_CODES_INT8)
    assert L.hq_qconv2d(fake, 1, 4, 1, 8, 8, 128, C.byref(pwc.desc), fake, 5, 5, 1, 1, fake, 1, fake, None, 1.0, fake,
                        None, 1, None, None) == 3


@pytest.mark.parametrize("mode", ["plain", "folded"])
@pytest.mark.parametrize("container", [0, 1])
@pytest.mark.parametrize("shape,had_block,w_bits", [((40, 256), 256, 4), ((130, 3, 3, 128), 128, 4),
                                                     ((16, 64), 16, 4), ((300, 768), 256, 4), ((8, 512), 512, 8),
                                                     ((5, 1, 1, 24), 8, 4)])
def test_weight_prepare_matches_oracle(hq, oracle, mode, container, shape, had_block, w_bits):
    w = inputs.weights(shape, seed=len(shape) + had_block)
    pw = hq.hq_weight_prepare(w, w_bits, had_block, hq.WEIGHT_MODES[mode], container)
    B_ref, s_ref = oracle.prepare_weights(w.reshape(shape[0], -1, shape[-1]), w_bits, had_block, mode)
    assert np.array_equal(pw.s_w, s_ref)
    assert np.array_equal(decode_blob(pw), B_ref)
    d = pw.desc
    assert d.bytes == hq.hq_weight_blob_bytes(shape[0], d.RS, shape[-1], w_bits, had_block, hq.WEIGHT_MODES[mode])
    assert d.max_abs_b == np.abs(B_ref).max()
    expect_limbs = 2 if (mode == "folded" and had_block * 2 ** (w_bits - 1) > 128) else 1
    assert d.limbs == expect_limbs
    a = 2.0 ** (-0.5 * np.log2(had_block)) if mode == "folded" else 1.0
    assert np.isclose(pw.alpha, a, rtol=1e-7)


def test_weight_prepare_double_close_to_oracle(hq, oracle):
    w = inputs.weights((64, 512), seed=9)
    pw = hq.hq_weight_prepare(w, 4, 512, hq.HQ_W_DOUBLE, hq.HQ_CODES_INT8)
    B_ref, s_ref = oracle.prepare_weights(w.reshape(64, 1, 512), 4, 512, "double")
    assert np.allclose(pw.s_w, s_ref, rtol=1e-6)
    diff = decode_blob(pw) != B_ref          # butterfly vs dense summation order: only exact ties may differ
    assert diff.mean() <= 1e-4
    assert pw.desc.limbs == 1 and pw.alpha == 1.0


def test_weight_prepare_errors(hq):
    w = inputs.weights((8, 48), seed=0)
    with pytest.raises(hq.HqError) as e:
        hq.hq_weight_prepare(w, 4, 32, hq.HQ_W_FOLDED, hq.HQ_CODES_INT8)    # 48 % 32 != 0
    assert e.value.status == 2
    with pytest.raises(hq.HqError) as e:
        hq.hq_weight_prepare(w, 5, 16, hq.HQ_W_PLAIN, hq.HQ_CODES_INT8)
    assert e.value.status == 1


def test_unet_layer_list_matches_the_workload_description():
    """Base 256, multipliers (1,2,3,4), 2 residual blocks per level, attention at 32/16/8, batch 64 on a 64x64 latent:
    121 quantized layers of 47 distinct shapes, 16.0 TOP per forward counted with one weight limb."""
    from paper_2512_05746_b200 import unet
    layers = unet.quantized_layers()
    assert len(layers) == 121 and len(unet.distinct_shapes(layers)) == 47
    assert abs(2 * sum(L["macs"] for L in layers) / 1e12 - 16.04) < 0.01
    for L in layers:
        cin = L["C"] if L["kind"] == "conv" else L["K"]
        assert cin % L["had_block"] == 0 and L["had_block"] == 256
    assert sum(1 for L in layers if L["kind"] == "conv" and L["stride"] == 2) == 3
    assert sum(1 for L in layers if L["kind"] == "conv" and L["R"] == 1) == 15
    assert max(L["C"] for L in layers if L["kind"] == "conv") == 2048       # skip concatenation at the deepest level


def test_dit_layer_list():
    """Width 1152 = 9 x 128, depth 28, MLP ratio 4, batch 32 x 256 tokens: 28 x 5 + 3 quantized linears."""
    from paper_2512_05746_b200 import dit
    layers = dit.quantized_layers()
    assert len(layers) == 28 * 5 + 3
    assert all(L["K"] % L["had_block"] == 0 and L["had_block"] == 128 for L in layers)
    big = [L for L in layers if L["M"] == 32 * 256]
    assert len(big) == 28 * 4 and {(L["K"], L["N"]) for L in big} == {(1152, 3456), (1152, 1152), (1152, 4608), (4608, 1152)}
