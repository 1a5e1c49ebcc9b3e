"""GPU check of hq_qlinear_noalloc, the fused linear layer for callers that cannot allocate device memory.

Some users of the library have no allocator to call when a layer runs: their memory was handed out at start-up,
or the host application they live in keeps the allocator to itself.  For them the library carries its own fixed
8 MiB device array for the codes and scales that sit between the two kernels of a layer.  This file checks, through
the C ABI, that the entry point gives what hq_qlinear gives with a caller-supplied workspace -- on two calls in a
row with different shapes, because every call reuses the same array and finds the previous call's bytes in it --
and that a layer too large for the array is refused before anything is launched.

The file name sorts last on purpose: a run that stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest

from paper_2512_05746_b200 import inputs
from hq_testutil import Y_BF16_RTOL, Y_F32_RTOL, rel_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2512_05746_b200 import binding as hq
    return torch, hq


def _both_ways(torch, hq, M, K, N, had_block, container, ydtype, seed, static=None):
    x = torch.from_numpy(inputs.activations((M, K), outlier_count=3, outlier_scale=20.0, seed=seed)).cuda()
    pw = hq.hq_weight_prepare(inputs.weights((N, K), seed=seed), 4, had_block, hq.HQ_W_FOLDED, container).to_device()
    b = torch.from_numpy(inputs.bias(N, seed=seed)).cuda()
    ss = None if static is None else torch.tensor([static], dtype=torch.float32, device="cuda")
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    ws = torch.empty((hq.hq_workspace_size(M, K, container),), dtype=torch.uint8, device="cuda")
    y_ref = torch.zeros((M, N), dtype=ydtype, device="cuda")
    hq.hq_qlinear(x, pw, b, 4, y_ref, ws, static_scale=ss, dev_status=status)
    y = torch.zeros((M, N), dtype=ydtype, device="cuda")
    hq.hq_qlinear_noalloc(x, pw, b, 4, y, static_scale=ss, dev_status=status)
    torch.cuda.synchronize()
    hq.hq_check_status(status)
    # the two entry points run the same kernels on the same inputs: beyond the tolerances below, the outputs must
    # be the same bits (left-over bytes of an earlier call that leaked into this one would show here first)
    assert torch.equal(y, y_ref), "hq_qlinear_noalloc and hq_qlinear differ"
    return y.float().cpu().numpy(), y_ref.float().cpu().numpy().astype(np.float64)


def test_noalloc_matches_workspace_version_twice_in_a_row(env):
    torch, hq = env
    # first call: large enough to fill most of the array (4096 x 2048 nibble codes = 4 MiB)
    y, y_ref = _both_ways(torch, hq, 4096, 2048, 384, 2048, hq.HQ_CODES_NIBBLE, torch.bfloat16, seed=1)
    assert rel_err(y, y_ref) <= Y_BF16_RTOL
    # second call straight after it: other shape, other container, ragged rows, static scale; the array still
    # holds the first call's codes
    y, y_ref = _both_ways(torch, hq, 1000, 512, 200, 512, hq.HQ_CODES_INT8, torch.float32, seed=2, static=0.4)
    assert rel_err(y, y_ref) <= Y_F32_RTOL
    # and the first shape again, so stale bytes of a smaller call sit under a larger one
    y, y_ref = _both_ways(torch, hq, 4096, 2048, 384, 2048, hq.HQ_CODES_NIBBLE, torch.bfloat16, seed=3)
    assert rel_err(y, y_ref) <= Y_BF16_RTOL


def test_noalloc_layer_that_fills_the_array_to_its_last_bytes(env):
    """8160 rows of 1024 one-byte codes plus their 8160 scales need 8388480 of the 8388608 bytes: the scales sit at the
    very end of the array, and one more row would not fit."""
    torch, hq = env
    M, K, N = 8160, 1024, 136
    assert hq.HQ_NOALLOC_SCRATCH_BYTES - 128 == hq.hq_workspace_size(M, K, hq.HQ_CODES_INT8)
    assert hq.hq_workspace_size(M + 1, K, hq.HQ_CODES_INT8) > hq.HQ_NOALLOC_SCRATCH_BYTES
    y, y_ref = _both_ways(torch, hq, M, K, N, 1024, hq.HQ_CODES_INT8, torch.bfloat16, seed=4)
    assert rel_err(y, y_ref) <= Y_BF16_RTOL


def test_noalloc_call_takes_no_device_memory(env):
    """What the entry point is for: once the library is loaded and the first call on the device has been made, a
    call leaves the amount of free device memory where it was."""
    torch, hq = env
    M, K, N = 2048, 512, 256
    x = torch.from_numpy(inputs.activations((M, K), outlier_count=2, outlier_scale=20.0, seed=5)).cuda()
    pw = hq.hq_weight_prepare(inputs.weights((N, K), seed=5), 4, 512, hq.HQ_W_FOLDED, hq.HQ_CODES_INT8).to_device()
    y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    hq.hq_qlinear_noalloc(x, pw, None, 4, y)                    # first call on the device: resolves the array's address
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        hq.hq_qlinear_noalloc(x, pw, None, 4, y)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after >= free_before, f"free device memory fell by {free_before - free_after} bytes"


def test_noalloc_refuses_layers_beyond_its_array(env):
    torch, hq = env
    M, K, N = 8192, 2048, 128                                   # 8192 * (1024 + 4) bytes > 8 MiB
    assert hq.hq_workspace_size(M, K, hq.HQ_CODES_NIBBLE) > hq.HQ_NOALLOC_SCRATCH_BYTES
    x = torch.zeros((M, K), dtype=torch.float32, device="cuda")
    pw = hq.hq_weight_prepare(inputs.weights((N, K), seed=0), 4, 2048, hq.HQ_W_FOLDED, hq.HQ_CODES_NIBBLE).to_device()
    y = torch.full((M, N), 3.0, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(hq.HqError) as e:
        hq.hq_qlinear_noalloc(x, pw, None, 4, y)
    assert e.value.status == 9 and "scratch" in str(e.value)
    torch.cuda.synchronize()
    assert bool((y == 3.0).all())                               # nothing was launched
