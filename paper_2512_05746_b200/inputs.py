"""Seeded synthetic inputs for the quantized-layer forward.

Only random draws and reshapes live here: no transform, no quantizer, no GEMM.
Every generator is a pure function of its arguments (counter-based Philox stream
keyed by ``seed`` and a per-tensor ``stream`` id), so the CUDA path and the CPU
checker are always handed byte-identical host arrays.

The shapes and value distributions follow the workloads this repository is
measured on: Gaussian or heavy-tailed (Student-t) activations in which a small
fraction of channels is scaled up to act as outlier channels, and small
zero-mean Gaussian weights.
"""
from __future__ import annotations

import numpy as np


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[np.uint64(seed), np.uint64(stream)]))


def outlier_channels(channels: int, count: int, seed: int, stream: int = 1000) -> np.ndarray:
    """``count`` distinct channel indices, sorted."""
    count = int(min(max(count, 0), channels))
    return np.sort(_rng(seed, stream).choice(channels, size=count, replace=False))


def activations(shape, *, dist: str = "normal", outlier_count: int = 0, outlier_scale: float = 1.0,
                seed: int = 0, stream: int = 0, dtype=np.float32) -> np.ndarray:
    """Activation tensor whose last axis is the channel axis.

    dist: "normal" -> N(0,1); "student_t3" -> Student-t with 3 degrees of freedom.
    ``outlier_count`` channels (chosen by the same seed) are multiplied by ``outlier_scale``.
    """
    rng = _rng(seed, stream)
    if dist == "normal":
        x = rng.standard_normal(size=shape, dtype=np.float32)
    elif dist == "student_t3":
        x = rng.standard_t(3.0, size=shape).astype(np.float32)
    else:
        raise ValueError(f"unknown dist {dist!r}")
    if outlier_count > 0:
        ch = outlier_channels(shape[-1], outlier_count, seed, stream + 1000)
        x[..., ch] *= np.float32(outlier_scale)
    return np.ascontiguousarray(x.astype(dtype, copy=False))


def weights(shape, *, std: float = 0.02, seed: int = 0, stream: int = 1) -> np.ndarray:
    """Weight tensor ~ N(0, std^2), fp32, C-contiguous, in whatever shape is asked for."""
    w = _rng(seed, stream).standard_normal(size=shape, dtype=np.float32) * np.float32(std)
    return np.ascontiguousarray(w)


def bias(n: int, *, std: float = 0.01, seed: int = 0, stream: int = 2) -> np.ndarray:
    return np.ascontiguousarray(_rng(seed, stream).standard_normal(size=(n,), dtype=np.float32) * np.float32(std))


def codes(shape, bits: int, *, seed: int = 0, stream: int = 3) -> np.ndarray:
    """Uniform random signed integers in the full ``bits``-bit two's-complement range, as int8."""
    lo, hi = -(1 << (bits - 1)), (1 << (bits - 1)) - 1
    return _rng(seed, stream).integers(lo, hi + 1, size=shape, dtype=np.int8)


def positive_scales(n: int, *, lo: float = 0.01, hi: float = 0.2, seed: int = 0, stream: int = 4) -> np.ndarray:
    return _rng(seed, stream).uniform(lo, hi, size=(n,)).astype(np.float32)


# ---------------------------------------------------------------------------------------------
# Named workloads.  Each returns a dict of plain numpy arrays and python scalars.
# ---------------------------------------------------------------------------------------------

def config_linear_small(seed: int = 0) -> dict:
    """Single quantized linear: X [256,256] ~N(0,1) with 4 channels x20; W [N=256][K=256] ~N(0,0.02)."""
    M = K = N = 256
    return dict(name="linear_small", M=M, K=K, N=N, had_block=256, a_bits=4, w_bits=4,
                x=activations((M, K), outlier_count=4, outlier_scale=20.0, seed=seed, stream=10),
                w=weights((N, K), seed=seed, stream=11), bias=None)


def config_conv_small(seed: int = 0, batch: int = 8) -> dict:
    """Single quantized 3x3 conv: X NHWC [8,32,32,256] ~N(0,1), 1% channels x20; W [256,3,3,256]."""
    Nb, H, W, C, Cout = batch, 32, 32, 256, 256
    return dict(name="conv_small", Nb=Nb, H=H, W=W, C=C, Cout=Cout, R=3, S=3, stride=1, pad=1, had_block=256,
                w_bits=4,
                x=activations((Nb, H, W, C), outlier_count=max(1, round(0.01 * C)), outlier_scale=20.0,
                              seed=seed, stream=20),
                w=weights((Cout, 3, 3, C), seed=seed, stream=21), bias=bias(Cout, seed=seed, stream=22))


TRANSFORMER_LINEARS = (
    # name, K, N, had_block
    ("qkv", 512, 1536, 512),
    ("out_proj", 512, 512, 512),
    ("ff1", 512, 2048, 512),
    ("ff2", 2048, 512, 2048),
)


def config_transformer_linear(which: str, M: int = 32768, seed: int = 0) -> dict:
    """One of the transformer-block linears of a latent UNet at 32x32 latent, batch 32 (M = 32768 tokens)."""
    for i, (name, K, N, hb) in enumerate(TRANSFORMER_LINEARS):
        if name == which:
            return dict(name=name, M=M, K=K, N=N, had_block=hb, w_bits=4,
                        x=activations((M, K), dist="student_t3", outlier_count=max(1, round(0.005 * K)),
                                      outlier_scale=30.0, seed=seed, stream=30 + 4 * i),
                        w=weights((N, K), seed=seed, stream=31 + 4 * i),
                        bias=bias(N, seed=seed, stream=32 + 4 * i))
    raise KeyError(which)


def config_sweep_point(M: int, K: int, N: int, seed: int = 0) -> dict:
    """One point of the shape sweep: X ~N(0,1) with 1% channels x20, Hadamard block = K."""
    return dict(name=f"sweep_{M}x{K}x{N}", M=M, K=K, N=N, had_block=K, w_bits=4,
                x=activations((M, K), outlier_count=max(1, round(0.01 * K)), outlier_scale=20.0,
                              seed=seed, stream=50),
                w=weights((N, K), seed=seed, stream=51), bias=bias(N, seed=seed, stream=52))


# ---------------------------------------------------------------------------------------------
# A latent-diffusion UNet: configuration and seeded random parameters (names and shapes only).
# ---------------------------------------------------------------------------------------------

def unet_config(batch: int = 64, latent: int = 64, in_ch: int = 3, base: int = 256, mults=(1, 2, 3, 4),
                res_blocks: int = 2, attn_resolutions=(32, 16, 8), heads: int = 8, groups: int = 32,
                classes: int = 1000, had_block: int = 256) -> dict:
    """The noise-prediction network the workload names: residual blocks of GroupNorm + SiLU + 3x3 convolution, a step
    + class embedding fed into every residual block, self-attention at the listed resolutions, stride-2 convolutions
    down, nearest up-sampling + convolution up, skip connections by channel concatenation."""
    return dict(batch=batch, latent=latent, in_ch=in_ch, base=base, mults=tuple(mults), res_blocks=res_blocks,
                attn_resolutions=tuple(attn_resolutions), heads=heads, groups=groups, classes=classes, had_block=had_block)


def unet_params(cfg: dict, seed: int = 0) -> dict:
    """name -> fp32 array for every parameter of the network, drawn from the seeded stream in a fixed order.
    Convolution weights are [Cout, R, R, Cin], linear weights [N, K], both ~N(0, 1/fan_in) so that activations keep
    their scale through the network; biases ~N(0, 0.01); norm gains 1 + 0.1 N(0,1), offsets 0.1 N(0,1); the class
    table ~N(0, 0.3)."""
    P = {}
    counter = [0]

    def draw(shape, std):
        counter[0] += 1
        return np.ascontiguousarray(_rng(seed, 2000 + counter[0]).standard_normal(size=shape, dtype=np.float32) * np.float32(std))

    def conv(name, cin, cout, R):
        P[name + ".w"] = draw((cout, R, R, cin), 1.0 / np.sqrt(R * R * cin))
        P[name + ".b"] = draw((cout,), 0.01)

    def linear(name, K, N):
        P[name + ".w"] = draw((N, K), 1.0 / np.sqrt(K))
        P[name + ".b"] = draw((N,), 0.01)

    def norm(name, ch):
        P[name + ".gamma"] = np.ascontiguousarray(1.0 + draw((ch,), 0.1), dtype=np.float32)
        P[name + ".beta"] = draw((ch,), 0.1)

    def resblock(name, cin, cout):
        norm(name + ".norm1", cin)
        conv(name + ".conv1", cin, cout, 3)
        linear(name + ".emb", temb, cout)
        norm(name + ".norm2", cout)
        conv(name + ".conv2", cout, cout, 3)
        if cin != cout:
            conv(name + ".skip", cin, cout, 1)

    def attention(name, ch):
        norm(name + ".norm", ch)
        linear(name + ".qkv", ch, 3 * ch)
        linear(name + ".proj", ch, ch)

    base, mults, nres = cfg["base"], cfg["mults"], cfg["res_blocks"]
    temb = 4 * base
    linear("time_embed.0", base, temb)
    linear("time_embed.2", temb, temb)
    P["label_emb"] = draw((cfg["classes"], temb), 0.3)
    conv("in_conv", cfg["in_ch"], base, 3)
    ch, res = base, cfg["latent"]
    skips = [ch]
    for lvl, m in enumerate(mults):
        for b in range(nres):
            resblock(f"down{lvl}.res{b}", ch, m * base)
            ch = m * base
            if res in cfg["attn_resolutions"]:
                attention(f"down{lvl}.attn{b}", ch)
            skips.append(ch)
        if lvl + 1 < len(mults):
            conv(f"down{lvl}.downsample", ch, ch, 3)
            res //= 2
            skips.append(ch)
    resblock("mid.res0", ch, ch)
    attention("mid.attn", ch)
    resblock("mid.res1", ch, ch)
    for lvl in reversed(range(len(mults))):
        m = mults[lvl]
        for b in range(nres + 1):
            resblock(f"up{lvl}.res{b}", ch + skips.pop(), m * base)
            ch = m * base
            if res in cfg["attn_resolutions"]:
                attention(f"up{lvl}.attn{b}", ch)
        if lvl > 0:
            res *= 2
            conv(f"up{lvl}.upsample", ch, ch, 3)
    norm("out_norm", ch)
    conv("out_conv", ch, cfg["in_ch"], 3)
    return P


def unet_inputs(cfg: dict, seed: int = 0) -> dict:
    """Latent x NHWC ~N(0,1), denoising steps t in [0, 1000), class labels."""
    r = _rng(seed, 1999)
    Nb, S = cfg["batch"], cfg["latent"]
    return dict(x=np.ascontiguousarray(r.standard_normal(size=(Nb, S, S, cfg["in_ch"]), dtype=np.float32)),
                t=r.integers(0, 1000, size=(Nb,)).astype(np.float32),
                y=r.integers(0, cfg["classes"], size=(Nb,)).astype(np.int32))
