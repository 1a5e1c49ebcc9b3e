"""Layer list of the quantized convolutions and linears of a latent-diffusion UNet (shapes only, no arithmetic).

The noise-prediction network the method is applied to is a UNet over a latent image; every convolution except the
first and the last, and every linear layer, runs as the Hadamard-quantized layer.  This module walks the usual
encoder / middle / decoder structure and emits one record per quantized layer, so that the benchmark can run them
with synthetic activations and random weights:

  level l of the encoder: `res_blocks` residual blocks (3x3 conv, time-embedding linear, 3x3 conv, 1x1 skip conv when
  the channel count changes), each followed by a self-attention block (QKV linear, output projection) at the
  resolutions listed in `attn_resolutions`; a stride-2 3x3 convolution goes down to the next level;
  middle: residual block, attention, residual block;
  decoder: `res_blocks + 1` residual blocks per level, fed with the concatenation of the running tensor and the
  matching encoder output, attention as in the encoder, and a 3x3 convolution after each nearest-neighbour upsampling;
  the time embedding itself is a two-layer MLP.

Normalisation, activation functions, the attention product, up/down-sampling and the first / last convolution are
not quantized layers and are not listed.
"""
from __future__ import annotations


def quantized_layers(batch: int = 64, latent: int = 64, base: int = 256, mults=(1, 2, 3, 4), res_blocks: int = 2,
                     attn_resolutions=(32, 16, 8), had_block: int = 256) -> list[dict]:
    """One dict per quantized layer, in execution order.

    kind 'conv': Nb, H, W (INPUT size), C, Cout, R (1 or 3), stride, pad;  kind 'linear': M, K, N.
    Every record also carries `had_block`, `macs` (multiply-accumulates) and a `name`."""
    layers: list[dict] = []
    temb = 4 * base

    def conv(name, res, cin, cout, R=3, stride=1):
        ho = res // stride
        layers.append(dict(kind="conv", name=name, Nb=batch, H=res, W=res, C=cin, Cout=cout, R=R, stride=stride,
                           pad=R // 2, had_block=had_block, macs=batch * ho * ho * cout * R * R * cin))

    def linear(name, M, K, N):
        layers.append(dict(kind="linear", name=name, M=M, K=K, N=N, had_block=min(had_block, K),
                           macs=M * N * K))

    def resblock(name, res, cin, cout):
        conv(f"{name}.conv1", res, cin, cout)
        linear(f"{name}.emb", batch, temb, cout)
        conv(f"{name}.conv2", res, cout, cout)
        if cin != cout:
            conv(f"{name}.skip", res, cin, cout, R=1)

    def attention(name, res, ch):
        linear(f"{name}.qkv", batch * res * res, ch, 3 * ch)
        linear(f"{name}.proj", batch * res * res, ch, ch)

    linear("time_embed.0", batch, base, temb)
    linear("time_embed.2", batch, temb, temb)

    ch, res = base, latent
    skips = [ch]                                   # output of the (unquantized) first convolution
    for lvl, m in enumerate(mults):
        for b in range(res_blocks):
            resblock(f"down{lvl}.res{b}", res, ch, m * base)
            ch = m * base
            if res in attn_resolutions:
                attention(f"down{lvl}.attn{b}", res, ch)
            skips.append(ch)
        if lvl + 1 < len(mults):
            conv(f"down{lvl}.downsample", res, ch, ch, R=3, stride=2)
            res //= 2
            skips.append(ch)
    resblock("mid.res0", res, ch, ch)
    attention("mid.attn", res, ch)
    resblock("mid.res1", res, ch, ch)
    for lvl in reversed(range(len(mults))):
        m = mults[lvl]
        for b in range(res_blocks + 1):
            resblock(f"up{lvl}.res{b}", res, ch + skips.pop(), m * base)
            ch = m * base
            if res in attn_resolutions:
                attention(f"up{lvl}.attn{b}", res, ch)
        if lvl > 0:
            res *= 2
            conv(f"up{lvl}.upsample", res, ch, ch)
    return layers


def distinct_shapes(layers: list[dict]) -> list[tuple]:
    """The set of distinct layer shapes, as sortable tuples."""
    out = set()
    for L in layers:
        if L["kind"] == "conv":
            out.add(("conv", L["Nb"], L["H"], L["C"], L["Cout"], L["R"], L["stride"]))
        else:
            out.add(("linear", L["M"], L["K"], L["N"]))
    return sorted(out)
