"""Multi-process (gloo, CPU) checks of the row-sharded layout used for more than one GPU: shards partition the
rows, a sharded layer equals the unsharded one row for row (so the data path needs no collective), and the timing
reduction returns the slowest rank's value on every rank."""
import os
import socket
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_shards_partition_rows():
    from paper_2512_05746_b200.sharding import shard_images, shard_rows
    for rows in (0, 1, 7, 32768, 100003):
        for world in (1, 2, 3, 8):
            spans = [shard_rows(rows, r, world) for r in range(world)]
            assert spans[0][0] == 0 and sum(c for _, c in spans) == rows
            for (a, ca), (b, _) in zip(spans, spans[1:]):
                assert a + ca == b
            assert max(c for _, c in spans) - min(c for _, c in spans) <= 1
    assert shard_images(64, 1, 2) == (32, 32)
    with pytest.raises(ValueError):
        shard_rows(10, 2, 2)


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import oracle
    from paper_2512_05746_b200 import inputs
    from paper_2512_05746_b200.sharding import max_over_ranks, shard_images, shard_rows
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # linear layer: this rank's rows only
        M, K, N = 301, 64, 40
        x = inputs.activations((M, K), outlier_count=2, outlier_scale=20.0, seed=5)
        w = inputs.weights((N, K), seed=5)
        first, count = shard_rows(M, rank, world)
        y_lin = oracle.qlinear(x[first:first + count], w, None, a_bits=4, w_bits=4, had_block=64)["y"]
        # convolution: this rank's images only (per-pixel scales)
        xc = inputs.activations((5, 6, 6, 32), outlier_count=1, outlier_scale=20.0, seed=6)
        wc = inputs.weights((16, 3, 3, 32), seed=6)
        f_img, n_img = shard_images(5, rank, world)
        y_conv = oracle.qconv(xc[f_img:f_img + n_img], wc, None, a_bits=4, w_bits=4, had_block=32, stride=1, pad=1)["y"]
        slowest = max_over_ranks(10.0 + rank)
        np.savez(out, first=first, count=count, y_lin=y_lin, f_img=f_img, n_img=n_img, y_conv=y_conv, slowest=slowest)
    finally:
        dist.destroy_process_group()


def test_sharded_layer_equals_unsharded_world2(tmp_path, oracle):
    import torch.multiprocessing as mp
    from paper_2512_05746_b200 import inputs
    world = 2
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    outs = [str(tmp_path / f"rank{r}.npz") for r in range(world)]
    procs = [ctx.Process(target=_worker, args=(r, world, port, outs[r])) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    parts = [np.load(o) for o in outs]
    x = inputs.activations((301, 64), outlier_count=2, outlier_scale=20.0, seed=5)
    w = inputs.weights((40, 64), seed=5)
    whole = oracle.qlinear(x, w, None, a_bits=4, w_bits=4, had_block=64)["y"]
    assert np.array_equal(np.concatenate([p["y_lin"] for p in parts]), whole)
    xc = inputs.activations((5, 6, 6, 32), outlier_count=1, outlier_scale=20.0, seed=6)
    wc = inputs.weights((16, 3, 3, 32), seed=6)
    whole_c = oracle.qconv(xc, wc, None, a_bits=4, w_bits=4, had_block=32, stride=1, pad=1)["y"]
    assert np.array_equal(np.concatenate([p["y_conv"] for p in parts]), whole_c)
    assert all(float(p["slowest"]) == 11.0 for p in parts)
