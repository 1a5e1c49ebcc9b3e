"""One denoising step of the latent-diffusion UNet on the oracle's operations -- TEST INFRASTRUCTURE.

The method is applied to every linear and convolution of the noise-prediction network except its first and last
convolution (overview figure of the framework; Experiments).  This module chains the oracle's steps in the network's
order, in fp64 between layers: quantized layers through `oracle.qconv` / `oracle.qlinear` (Eq. 12 / Eq. 14 with the
folded weights), everything else through the oracle's plain definitions (GroupNorm, SiLU, attention core, up-sampling,
embeddings, float convolution).  It walks the network on its own (it shares no code with the CUDA-side runner); the two
only agree on the parameter names of `inputs.unet_params`.

3x3 convolutions use one static activation scale each, given by name in `static` (the learned per-layer scale of the
method; a parameter here); 1x1 convolutions and linears use one dynamic scale per row.

`store` is applied to every tensor that the network keeps between two operations (identity by default).  A network
whose layers are defined with bf16 outputs passes `oracle.round_bf16`: the quantizer of Eq. 3 is discontinuous, so a
storage rounding of 2^-9 in front of it moves a few per cent of the 4-bit codes by a whole step, and a forward that
keeps fp64 between layers is a different function from one that keeps bf16, not a more exact version of it.
"""
from __future__ import annotations

import numpy as np

import oracle

EPS = 1e-5


def forward(cfg: dict, P: dict, x, t, y, static: dict, a_bits: int = 4, w_bits: int = 4, trace: dict | None = None,
            store=None):
    """x NHWC [Nb, S, S, in_ch], t [Nb], y [Nb] -> eps [Nb, S, S, in_ch] (fp64).  trace: receives every block output."""
    st = store if store is not None else (lambda v: v)
    G, heads, hb = cfg["groups"], cfg["heads"], cfg["had_block"]
    base, mults, nres = cfg["base"], cfg["mults"], cfg["res_blocks"]

    def keep(name, v):
        if trace is not None:
            trace[name] = v
        return v

    def had_for(K):
        return hb if K % hb == 0 else 1

    def conv3(name, h, norm=None, stride=1):
        if norm:
            h = oracle.groupnorm(h, G, P[norm + ".gamma"], P[norm + ".beta"], EPS, "silu")
        return st(oracle.qconv(h, P[name + ".w"], P[name + ".b"], a_bits=a_bits, w_bits=w_bits, had_block=had_for(h.shape[-1]),
                               stride=stride, pad=1, weight_mode="folded", static_scale=float(static[name]))["y"])

    def conv1(name, h):
        return st(oracle.qconv(h, P[name + ".w"], P[name + ".b"], a_bits=a_bits, w_bits=w_bits, had_block=had_for(h.shape[-1]),
                               stride=1, pad=0, weight_mode="folded")["y"])

    def linear(name, h2d):
        return st(oracle.qlinear(h2d, P[name + ".w"], P[name + ".b"], a_bits=a_bits, w_bits=w_bits,
                                 had_block=had_for(h2d.shape[-1]), weight_mode="folded")["y"])

    def resblock(name, h, semb):
        cin, cout = h.shape[-1], P[name + ".conv1.w"].shape[0]
        a = conv3(name + ".conv1", h, norm=name + ".norm1")
        a = a + linear(name + ".emb", semb)[:, None, None, :]     # feeds the normalisation directly: not a kept tensor
        a = conv3(name + ".conv2", a, norm=name + ".norm2")
        skip = h if cin == cout else conv1(name + ".skip", h)
        return keep(name, st(skip + a))

    def attention(name, h):
        Nb, H, W, ch = h.shape
        hn = oracle.groupnorm(h, G, P[name + ".norm.gamma"], P[name + ".norm.beta"], EPS, "none")
        qkv = linear(name + ".qkv", hn.reshape(Nb * H * W, ch))
        a = st(oracle.attention(qkv.reshape(Nb, H * W, 3 * ch), heads).reshape(Nb * H * W, ch))
        return keep(name, st(h + linear(name + ".proj", a).reshape(h.shape)))

    x = np.asarray(x, np.float64)
    temb = st(oracle.timestep_embedding(np.asarray(t, np.float64), base))
    e = linear("time_embed.0", temb)
    e = linear("time_embed.2", st(oracle.silu(e)))
    e = st(e + np.asarray(P["label_emb"], np.float64)[np.asarray(y, np.int64)])
    semb = st(oracle.silu(e))

    h = keep("in_conv", st(oracle.conv2d_float(x, P["in_conv.w"], P["in_conv.b"], 1, 1)))
    res = cfg["latent"]
    skips = [h]
    for lvl in range(len(mults)):
        for b in range(nres):
            h = resblock(f"down{lvl}.res{b}", h, semb)
            if res in cfg["attn_resolutions"]:
                h = attention(f"down{lvl}.attn{b}", h)
            skips.append(h)
        if lvl + 1 < len(mults):
            h = keep(f"down{lvl}.downsample", conv3(f"down{lvl}.downsample", h, stride=2))
            res //= 2
            skips.append(h)
    h = resblock("mid.res0", h, semb)
    h = attention("mid.attn", h)
    h = resblock("mid.res1", h, semb)
    for lvl in reversed(range(len(mults))):
        for b in range(nres + 1):
            h = resblock(f"up{lvl}.res{b}", np.concatenate([h, skips.pop()], axis=-1), semb)
            if res in cfg["attn_resolutions"]:
                h = attention(f"up{lvl}.attn{b}", h)
        if lvl > 0:
            res *= 2
            h = keep(f"up{lvl}.upsample", conv3(f"up{lvl}.upsample", oracle.upsample_nearest2x(h)))
    h = st(oracle.groupnorm(h, G, P["out_norm.gamma"], P["out_norm.beta"], EPS, "silu"))
    return oracle.conv2d_float(h, P["out_conv.w"], P["out_conv.b"], 1, 1)
