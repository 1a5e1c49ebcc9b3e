"""A latent-diffusion UNet on the Hadamard-quantized layers: the layer list (shapes only) and the forward pass.

`quantized_layers` lists the quantized convolutions and linears of the network, for workloads that run them on their
own.  `UNet` runs one denoising step of the whole network: every call below is an entry point of the C library (the
quantized layers with their fused normalisation prologues, and the unquantized operations between them); this module
only decides the order of the calls and owns the buffers.

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


class UNet:
    """One denoising step eps = net(x, t, y) of the network `inputs.unet_config` describes.

    Every convolution except the first and the last, and every linear, is a Hadamard-quantized layer (W4, `a_bits`
    activations, folded weights).  3x3 convolutions take one static activation scale each (the per-layer learned scale
    of the method; here calibrated once by `calibrate`), 1x1 convolutions and linears one dynamic scale per row.
    GroupNorm + SiLU in front of a residual block's convolutions and GroupNorm in front of an attention block's QKV
    projection are fused into the quantized layer's transform kernel.  Activations are bf16 NHWC.

    `build(Nb)` allocates every buffer and records the sequence of library calls; `run` replays it.  Calls are tagged
    "q" (a quantized layer, including its fused normalisation) or "g" (everything else), so that the two parts can be
    timed separately on the buffers of a complete forward."""

    EPS = 1e-5

    def __init__(self, cfg: dict, params: dict, hq, device, container: int | None = None, a_bits: int = 4):
        import torch
        self.torch, self.hq, self.cfg, self.dev, self.a_bits = torch, hq, cfg, device, a_bits
        self.cont = hq.HQ_CODES_INT8 if container is None else container
        self.had = cfg["had_block"]
        self.pw, self.f32, self.bf = {}, {}, {}
        for name, arr in params.items():
            stem, leaf = name.rsplit(".", 1) if "." in name else (name, "")
            if name == "label_emb":
                self.bf[name] = torch.from_numpy(arr).to(device).to(torch.bfloat16)
            elif leaf == "w" and stem not in ("in_conv", "out_conv"):
                K = arr.shape[-1]
                hb = self.had if K % self.had == 0 else 1
                self.pw[stem] = hq.hq_weight_prepare(arr, 4, hb, hq.HQ_W_FOLDED, self.cont).to_device(device)
            else:
                self.f32[name] = torch.from_numpy(arr).to(device)
        self.static = {}            # name of a 3x3 convolution -> device tensor [1]
        self.status = torch.zeros((1,), dtype=torch.int32, device=device)
        self.tape = []
        self.calibrating = False
        self.recording = None

    # ------------------------------------------------------------------ recording helpers
    def _emit(self, tag, name, fn, rec=None):
        """Adds one library call to the tape.  rec: () -> dict of tensors to keep when a recording is requested."""
        def call():
            fn()
            if self.recording is not None and rec is not None:
                self.torch.cuda.synchronize()
                self.recording.append(dict(name=name, **{k: (v.clone() if hasattr(v, "clone") else v) for k, v in rec().items()}))
        self.tape.append((tag, name, call))

    def _new(self, shape, dtype=None):
        return self.torch.empty(shape, dtype=dtype or self.torch.bfloat16, device=self.dev)

    def _need_ws(self, rows, cols):
        self._ws_need = max(self._ws_need, self.hq.hq_workspace_size(rows, cols, self.cont))

    def _ws_views(self, rows, cols):
        row_bytes = cols // 2 if self.cont == self.hq.HQ_CODES_NIBBLE else cols
        pitch = (row_bytes + 15) // 16 * 16
        off = (rows * pitch + 255) // 256 * 256
        return self.ws[: rows * pitch].view(rows, pitch), self.ws[off: off + rows * 4].view(self.torch.float32)

    # ------------------------------------------------------------------ layers
    def _conv3(self, name, x, norm=None, stride=1, pre_bias=None, x2=None):
        """x2: the layer's input is the channel concatenation [x | x2], which is read in place and never written."""
        hq, t = self.hq, self.torch
        Nb, H, W, Cin = x.shape
        Cin += x2.shape[3] if x2 is not None else 0
        pw = self.pw[name]
        self._need_ws(Nb * H * W, Cin)
        y = self._new((Nb, H // stride, W // stride, pw.desc.N))
        bias = self.f32[name + ".b"]
        ss = self.static.setdefault(name, t.ones((1,), dtype=t.float32, device=self.dev))
        g = (self.f32[norm + ".gamma"], self.f32[norm + ".beta"]) if norm else None
        G = self.cfg["groups"]

        def calibrate():
            if not self.calibrating:
                return
            codes, sc = self._ws_views(Nb * H * W, Cin)
            if g:
                hq.hq_gn_silu_quant(x, G, g[0], g[1], self.EPS, pw.desc.had_block, self.a_bits, codes, self.cont, self.scratch,
                                    scales=sc, pre_bias=pre_bias, x2=x2)
            else:
                hq.hq_hadamard_quant(x.view(-1, x.shape[3]), pw.desc.had_block, self.a_bits, codes, self.cont, scales=sc,
                                     x2=None if x2 is None else x2.view(-1, x2.shape[3]))
            ss.copy_(sc.max().reshape(1))

        def run():
            calibrate()
            if g:
                hq.hq_gn_silu_qconv(x, G, g[0], g[1], self.EPS, pw, 3, 3, stride, 1, bias, self.a_bits, y, self.ws, self.scratch,
                                    static_scale=ss, dev_status=self.status, pre_bias=pre_bias, x2=x2)
            else:
                hq.hq_qconv(x, pw, 3, 3, stride, 1, bias, self.a_bits, y, self.ws, static_scale=ss, dev_status=self.status,
                            x2=x2)

        self._emit("q", name, run, lambda: dict(op="conv3", x=x, x2=x2, y=y, norm=norm, stride=stride, static=ss, pre_bias=pre_bias,
                                                codes=self._ws_views(Nb * H * W, Cin)[0]))
        return y

    def _conv1(self, name, x, x2=None):
        hq = self.hq
        Nb, H, W, Cin = x.shape
        Cin += x2.shape[3] if x2 is not None else 0
        pw = self.pw[name]
        self._need_ws(Nb * H * W, Cin)
        y = self._new((Nb, H, W, pw.desc.N))
        bias = self.f32[name + ".b"]
        self._emit("q", name, lambda: hq.hq_qconv(x, pw, 1, 1, 1, 0, bias, self.a_bits, y, self.ws, dev_status=self.status,
                                                      x2=x2),
                   lambda: dict(op="conv1", x=x, x2=x2, y=y, codes=self._ws_views(Nb * H * W, Cin)[0],
                                scales=self._ws_views(Nb * H * W, Cin)[1]))
        return y

    def _linear(self, name, x, norm=None, Nb=None):
        hq = self.hq
        M, K = x.shape
        pw = self.pw[name]
        self._need_ws(M, K)
        y = self._new((M, pw.desc.N))
        bias = self.f32[name + ".b"]
        if norm:
            gm, bt = self.f32[norm + ".gamma"], self.f32[norm + ".beta"]
            fn = lambda: hq.hq_gn_qlinear(x, Nb, self.cfg["groups"], gm, bt, self.EPS, False, pw, bias, self.a_bits, y, self.ws,
                                          self.scratch, dev_status=self.status)
        else:
            fn = lambda: hq.hq_qlinear(x, pw, bias, self.a_bits, y, self.ws, dev_status=self.status)
        self._emit("q", name, fn, lambda: dict(op="linear", x=x, y=y, norm=norm, Nb=Nb, codes=self._ws_views(M, K)[0],
                                               scales=self._ws_views(M, K)[1]))
        return y

    def _glue(self, name, op, fn, **tensors):
        self._emit("g", name, fn, lambda: dict(op=op, **tensors))

    def _resblock(self, name, x, semb, x2=None):
        """x2: the block's input is the channel concatenation [x | x2] (a skip connection joining the up-sampling path);
        its two consumers, the first convolution and the 1x1 skip convolution, read the two tensors in place."""
        hq = self.hq
        cin, cout = x.shape[-1] + (x2.shape[-1] if x2 is not None else 0), self.pw[name + ".conv1"].desc.N
        h = self._conv3(name + ".conv1", x, norm=name + ".norm1", x2=x2)
        e = self._linear(name + ".emb", semb)
        # h + e is never stored: the second convolution's normalisation takes the embedding as a per-sample addend
        h2 = self._conv3(name + ".conv2", h, norm=name + ".norm2", pre_bias=e)
        assert x2 is None or cin != cout       # a concatenated input always changes the channel count here
        xs = x if cin == cout else self._conv1(name + ".skip", x, x2=x2)
        out = self._new(h2.shape)
        self._glue(name + ".residual", "add", lambda: hq.hq_add(xs, h2, out), a=xs, b=h2, out=out)
        return out

    def _attention(self, name, x):
        hq = self.hq
        Nb, H, W, ch = x.shape
        x2 = x.view(Nb * H * W, ch)
        qkv = self._linear(name + ".qkv", x2, norm=name + ".norm", Nb=Nb)
        a = self._new((Nb * H * W, ch))
        heads = self.cfg["heads"]
        self.attn_flops += 4.0 * Nb * float(H * W) ** 2 * ch
        self._glue(name + ".core", "attention", lambda: hq.hq_attention(qkv, Nb, heads, a, dev_status=self.status),
                   qkv=qkv, out=a, Nb=Nb, heads=heads)
        pr = self._linear(name + ".proj", a)
        out = self._new(x.shape)
        self._glue(name + ".residual", "add", lambda: hq.hq_add(x2, pr, out), a=x2, b=pr, out=out)
        return out

    # ------------------------------------------------------------------ the network
    def build(self, Nb: int):
        """Allocates the buffers of a forward at batch Nb and records its sequence of library calls."""
        t, hq, cfg = self.torch, self.hq, self.cfg
        S, base, mults, nres = cfg["latent"], cfg["base"], cfg["mults"], cfg["res_blocks"]
        temb = 4 * base
        self.tape = []
        self.Nb = Nb
        self.attn_flops = 0.0          # 4 L^2 C per sample and attention block (QK^T and PV)
        self._ws_need = 256
        self.scratch = t.empty((Nb * cfg["groups"] * 24,), dtype=t.uint8, device=self.dev)
        self.x_in = t.empty((Nb, S, S, cfg["in_ch"]), dtype=t.bfloat16, device=self.dev)
        self.t_in = t.empty((Nb,), dtype=t.float32, device=self.dev)
        self.y_in = t.empty((Nb,), dtype=t.int32, device=self.dev)

        te = self._new((Nb, base))
        self._glue("time_embed.sin", "timestep_embedding", lambda: hq.hq_timestep_embedding(self.t_in, te), t=self.t_in, out=te)
        e1 = self._linear("time_embed.0", te)
        e1s = self._new(e1.shape)
        self._glue("time_embed.act", "silu", lambda: hq.hq_silu(e1, e1s), x=e1, out=e1s)
        emb = self._linear("time_embed.2", e1s)
        table = self.bf["label_emb"]
        self._glue("label_emb.add", "class_embed_add", lambda: hq.hq_class_embed_add(emb, table, self.y_in),
                   labels=self.y_in, out=emb)
        semb = self._new(emb.shape)
        self._glue("emb.act", "silu", lambda: hq.hq_silu(emb, semb), x=emb, out=semb)

        h = self._new((Nb, S, S, base))
        w_in, b_in = self.f32["in_conv.w"], self.f32["in_conv.b"]
        self._glue("in_conv", "conv_float", (lambda o=h: hq.hq_conv2d_direct(self.x_in, w_in, b_in, 3, 1, 1, o)), x=self.x_in,
                   out=h)
        ch, res = base, S
        skips = [h]
        for lvl, m in enumerate(mults):
            for b in range(nres):
                h = self._resblock(f"down{lvl}.res{b}", h, semb)
                if res in cfg["attn_resolutions"]:
                    h = self._attention(f"down{lvl}.attn{b}", h)
                skips.append(h)
            if lvl + 1 < len(mults):
                h = self._conv3(f"down{lvl}.downsample", h, stride=2)
                res //= 2
                skips.append(h)
        h = self._resblock("mid.res0", h, semb)
        h = self._attention("mid.attn", h)
        h = self._resblock("mid.res1", h, semb)
        for lvl in reversed(range(len(mults))):
            for b in range(nres + 1):
                sk = skips.pop()
                h = self._resblock(f"up{lvl}.res{b}", h, semb, x2=sk)         # [h | skip], never written out
                if res in cfg["attn_resolutions"]:
                    h = self._attention(f"up{lvl}.attn{b}", h)
            if lvl > 0:
                up = self._new((Nb, 2 * res, 2 * res, h.shape[3]))
                self._glue(f"up{lvl}.upsample.nearest", "upsample", (lambda a=h, o=up: hq.hq_upsample_nearest2x(a, o)), x=h, out=up)
                res *= 2
                h = self._conv3(f"up{lvl}.upsample", up)
        hn = self._new(h.shape)
        gm, bt = self.f32["out_norm.gamma"], self.f32["out_norm.beta"]
        self._glue("out_norm", "groupnorm_silu", (lambda a=h: hq.hq_groupnorm_act(a, cfg["groups"], gm, bt, self.EPS, True, hn,
                                                                                   self.scratch)), x=h, out=hn)
        self.eps_out = t.empty((Nb, S, S, cfg["in_ch"]), dtype=t.float32, device=self.dev)
        w_o, b_o = self.f32["out_conv.w"], self.f32["out_conv.b"]
        self._glue("out_conv", "conv_float", lambda: hq.hq_conv2d_direct(hn, w_o, b_o, 3, 1, 1, self.eps_out), x=hn,
                   out=self.eps_out)
        # one workspace for the codes and scales of whichever quantized layer is running (sized for the largest)
        self.ws = t.empty((self._ws_need,), dtype=t.uint8, device=self.dev)
        return self

    def set_inputs(self, x, t, y):
        """x NHWC (any float dtype), t [Nb] denoising steps, y [Nb] class labels (device or host tensors)."""
        self.x_in.copy_(x)
        self.t_in.copy_(t)
        self.y_in.copy_(y)

    def run(self, tags=("q", "g")):
        for tag, _, call in self.tape:
            if tag in tags:
                call()

    def calibrate(self, x, t, y):
        """One forward in which every 3x3 convolution first measures its input: its static activation scale becomes the
        largest per-pixel scale of that input."""
        self.set_inputs(x, t, y)
        self.calibrating = True
        try:
            self.run()
        finally:
            self.calibrating = False
        self.torch.cuda.synchronize()
        self.hq.hq_check_status(self.status)

    def forward(self, x, t, y, record=None):
        """eps [Nb, S, S, in_ch] fp32.  record: a list that receives, per library call, its name and copies of the tensors
        it read and wrote (for layer-by-layer checks)."""
        self.set_inputs(x, t, y)
        self.recording = record
        try:
            self.run()
        finally:
            self.recording = None
        return self.eps_out
