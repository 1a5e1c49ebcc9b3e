#!/usr/bin/env python
"""Benchmark of the Hadamard-quantized layer forward on B200.

One step = one pass of the whole hot path over one batch of synthetic activations shaped like the
transformer block and ResBlock convolution of a latent UNet at 32x32 latent, batch 32 (M = 32768 tokens /
pixels per layer):
    4 fused quantized linears  (QKV 512->1536, out-proj 512->512, FF1 512->2048, FF2 2048->512; Hadamard block = K)
  + 1 fused quantized 3x3 conv (NHWC [32,32,32,256] x [256,3,3,256], stride 1, pad 1; Hadamard over Cin = 256)
each as  online Hadamard transform -> INT4 quantize -> int8 tensor-core product with the folded (2-limb) weights of
the Single-Hadamard scheme -> rescale + bias -> bf16.  W4A4.

Prints ONE JSON line (see the keys below).  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2512_05746_b200 import inputs  # noqa: E402

METRIC = "int8 tensor TOPS (2*M*N*K*limbs) of the fused Hadamard-quant W4A4 linear+conv step"
UNIT = "TOPS"
M_TOKENS = 32768
CONV = dict(Nb=32, H=32, W=32, C=256, Cout=256, R=3, S=3, stride=1, pad=1, had_block=256)
WORKLOAD = ("configs[2] transformer-block linears (M=32768; QKV, out-proj, FF1, FF2) + configs[1] 3x3 conv at "
            "batch 32 (M=32768, K=2304, N=256); W4A4, folded 2-limb weights, bf16 out")
A_BITS, W_BITS = 4, 4
CLOCK_WINDOW_S = 0.7       # how long the load is kept running for the clock samples after the timed region
# Container of the 4-bit activation codes between the two kernels of a layer: 0 = HQ_CODES_NIBBLE (two per byte,
# unpacked inside the GEMM kernel), 1 = HQ_CODES_INT8 (one per byte); set by --codes.
CODES = [1]


def code_pitch(cols):
    """Bytes per row of `cols` codes in the selected container."""
    return cols // 2 if CODES[0] == 0 else cols


def codes_name():
    return "nibble" if CODES[0] == 0 else "int8"


def ws_views(torch, ws, rows, cols):
    """Codes [rows, pitch] and scales [rows] inside the workspace of a fused layer call (the documented layout)."""
    pitch = (code_pitch(cols) + 15) // 16 * 16
    off = (rows * pitch + 255) // 256 * 256
    return ws[: rows * pitch].view(rows, pitch), ws[off: off + rows * 4].view(torch.float32)
# dram__bytes_read.sum + dram__bytes_write.sum per launch at the full size of the default step, from the one-pass ncu
# capture of this command (a summary is kept under profiles/; taken with these kernel versions: set an entry to
# None when its kernel changes).  Outputs partly stay in L2 past the end of a launch, so these are below the
# algorithmic bytes.
NCU_DRAM_CODES = 1      # container the counters below were taken with (1 = one code per byte)
NCU_DRAM_BYTES = {"gemm": {"qkv": 66.2e6, "ff1": 100.7e6, "ff2": 73.4e6, "conv3x3": 9.6e6, "out_proj": 17.5e6},
                  "quant": {"qkv": 67.3e6, "out_proj": 67.2e6, "ff1": 68.7e6, "ff2": 278.2e6, "conv3x3": 33.6e6}}


def layer_list():
    layers = []
    for name, K, N, hb in inputs.TRANSFORMER_LINEARS:
        layers.append(dict(kind="linear", name=name, M=M_TOKENS, K=K, N=N, had_block=hb))
    c = CONV
    c["Nb"] = max(1, M_TOKENS // (c["H"] * c["W"]))
    layers.append(dict(kind="conv", name="conv3x3", M=c["Nb"] * c["H"] * c["W"], K=c["R"] * c["S"] * c["C"],
                       N=c["Cout"], had_block=c["had_block"]))
    return layers


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_burst=float(p["bf16_tflops"]),
                    bf16_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.gpu), "-lms", "100"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for ln in self.proc.stdout:
            self.lines.append(ln.strip())

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1])); mx.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no samples"])
        return dict(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))


# ------------------------------------------------------------------------------------------------ CUDA arm

def build_layers(torch, hq, device, seed):
    """Synthetic inputs and offline-prepared weights for every layer of the step, resident on `device`."""
    layers = layer_list()
    for i, L in enumerate(layers):
        if L["kind"] == "linear":
            cfg = inputs.config_transformer_linear(L["name"], M=L["M"], seed=seed)
            x_host, w, b = cfg["x"], cfg["w"], cfg["bias"]
        else:
            c = CONV
            cfg = inputs.config_conv_small(seed=seed, batch=c["Nb"])
            x_host, w, b = cfg["x"], cfg["w"], cfg["bias"]
        pw = hq.hq_weight_prepare(w, W_BITS, L["had_block"], hq.HQ_W_FOLDED, CODES[0]).to_device(device)
        L["pw"] = pw
        L["limbs"] = pw.desc.limbs
        L["x_host"] = torch.from_numpy(x_host).pin_memory()
        L["x"] = L["x_host"].to(device, non_blocking=True)
        L["bias"] = torch.from_numpy(b).to(device)
        rows, cols = (L["M"], L["K"]) if L["kind"] == "linear" else (L["M"], CONV["C"])
        L["rows"], L["cols"] = rows, cols
        ws_bytes = hq.hq_workspace_size(rows, cols, CODES[0])
        L["ws"] = torch.empty((ws_bytes,), dtype=torch.uint8, device=device)
        oshape = (L["M"], L["N"]) if L["kind"] == "linear" else (CONV["Nb"], CONV["H"], CONV["W"], CONV["Cout"])
        L["y"] = torch.empty(oshape, dtype=torch.bfloat16, device=device)
        L["y_host"] = torch.empty(oshape, dtype=torch.bfloat16).pin_memory()
        L["ops"] = 2.0 * L["M"] * L["N"] * L["K"] * L["limbs"]
        L["ops_1limb"] = 2.0 * L["M"] * L["N"] * L["K"]
        # algorithmic HBM bytes of the two kernels (fp32 in, codes out + scales; codes + weights in, bf16 out)
        cb = float(code_pitch(2)) / 2.0                                      # bytes per code
        L["quant_bytes"] = rows * cols * 4.0 + rows * cols * cb + rows * 4.0
        L["gemm_bytes"] = (L["M"] * L["K"] * cb if L["kind"] == "linear" else rows * cols * cb) + \
            L["N"] * L["K"] * L["limbs"] + L["M"] * L["N"] * 2.0 + 4.0 * L["M"] + 8.0 * L["N"]
        L["static_scale"] = None
    torch.cuda.synchronize()
    # The conv uses one static activation scale (the paper's learned per-tensor scale): calibrate it once with the
    # library's own dynamic pass: S = max over pixels of the per-pixel scale.
    for L in layers:
        if L["kind"] == "conv":
            x2d = L["x"].view(L["rows"], L["cols"])
            pitch = code_pitch(L["cols"])
            codes = torch.empty((L["rows"], pitch), dtype=torch.uint8, device=device)
            scales = torch.empty((L["rows"],), dtype=torch.float32, device=device)
            hq.hq_hadamard_quant(x2d, L["had_block"], A_BITS, codes, CODES[0], scales=scales)
            L["static_scale"] = scales.max().reshape(1).contiguous()
    torch.cuda.synchronize()
    return layers


def run_step(hq, layers, status, stream=None):
    for L in layers:
        if L["kind"] == "linear":
            hq.hq_qlinear(L["x"], L["pw"], L["bias"], A_BITS, L["y"], L["ws"], dev_status=status, stream=stream)
        else:
            c = CONV
            hq.hq_qconv(L["x"], L["pw"], c["R"], c["S"], c["stride"], c["pad"], L["bias"], A_BITS, L["y"], L["ws"],
                        static_scale=L["static_scale"], dev_status=status, stream=stream)


def run_step_split(torch, hq, layers, status, evs):
    """Same kernels as run_step, launched through the unfused entry points with an event between them."""
    stream = torch.cuda.current_stream()
    for L in layers:
        rows, cols = L["rows"], L["cols"]
        pitch = code_pitch(cols)
        codes = L["ws"][: rows * pitch].view(rows, pitch)
        off = (rows * pitch + 255) // 256 * 256
        scales = L["ws"][off: off + rows * 4].view(torch.float32)
        x2d = L["x"].view(rows, cols)
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        e0.record(stream)
        if L["kind"] == "linear":
            hq.hq_hadamard_quant(x2d, L["had_block"], A_BITS, codes, CODES[0], scales=scales)
            e1.record(stream)
            hq.hq_qgemm(codes, CODES[0], A_BITS, L["K"], L["pw"], scale_a=scales, bias=L["bias"],
                        alpha=L["pw"].alpha, y=L["y"], dev_status=status)
        else:
            c = CONV
            hq.hq_hadamard_quant(x2d, L["had_block"], A_BITS, codes, CODES[0], scales=scales[:1],
                                 static_scale=L["static_scale"])
            e1.record(stream)
            hq.hq_qconv2d(codes, CODES[0], A_BITS, c["Nb"], c["H"], c["W"], c["C"], L["pw"], c["R"], c["S"],
                          c["stride"], c["pad"], scale_a=L["static_scale"], bias=L["bias"], alpha=L["pw"].alpha,
                          y=L["y"], dev_status=status)
        e2.record(stream)
        evs.append((L, e0, e1, e2))


def oracle_sample_step(orc, sample_rows, seed):
    """One bounded sample of the step on the CPU oracle; returns (ops done, seconds)."""
    ops, t0 = 0.0, time.perf_counter()
    for name, K, N, hb in inputs.TRANSFORMER_LINEARS:
        cfg = inputs.config_transformer_linear(name, M=sample_rows, seed=seed)
        out = orc.qlinear(cfg["x"], cfg["w"], cfg["bias"], a_bits=A_BITS, w_bits=W_BITS, had_block=hb,
                          weight_mode="folded")
        ops += 2.0 * sample_rows * N * K * 2
        del out
    c = CONV
    cfg = inputs.config_conv_small(seed=seed, batch=max(1, sample_rows // (c["H"] * c["W"])))
    nb = cfg["x"].shape[0]
    orc.qconv(cfg["x"], cfg["w"], cfg["bias"], a_bits=A_BITS, w_bits=W_BITS, had_block=c["had_block"], stride=1, pad=1,
              weight_mode="folded", static_scale=0.5)
    ops += 2.0 * nb * c["H"] * c["W"] * c["Cout"] * c["R"] * c["S"] * c["C"] * 2
    return ops, time.perf_counter() - t0


def cpu_baseline(sample_rows=8192, seed=0):
    import oracle as orc
    orc.lib()
    ops, sec = oracle_sample_step(orc, sample_rows, seed)
    return dict(value=ops / sec / 1e12, unit=UNIT, cores=orc.num_threads(), kind="oracle",
                sample=f"{sample_rows} of {M_TOKENS} rows of each linear and {max(1, sample_rows // 1024)} of 32 images "
                       f"of the conv, whole oracle layer (dense Hadamard, quantize, weight prep, triple-loop product, "
                       f"rescale); {sec:.1f} s")


def main_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle as orc
    orc.lib()
    sample_rows = 2048
    for _ in range(min(args.warmup, 1)):
        oracle_sample_step(orc, 64, 0)
    tot_ops, tot_sec = 0.0, 0.0
    for _ in range(args.steps):
        ops, sec = oracle_sample_step(orc, sample_rows, 0)
        tot_ops += ops
        tot_sec += sec
    value = tot_ops / tot_sec / 1e12
    line = dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=tot_sec / args.steps * 1e3, higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="int64", data="synthetic",
                config=dict(workload=WORKLOAD, sample=f"{sample_rows} rows per layer per step"),
                cpu_baseline=dict(value=value, unit=UNIT, cores=orc.num_threads(), kind="oracle",
                                  sample=f"{sample_rows} rows per layer per step"),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))


def main_layer_list(args, which):
    """All quantized layers of a network-shaped workload, one after the other on one stream, bf16 activations,
    W4A4 with folded two-limb weights.  3x3 convolutions use one static activation scale, 1x1 convolutions and linears
    per-row scales.  The bf16 glue between the layers is not part of this path.
    unet: 121 layers of the UNet-shaped workload (batch 64, 64x64 latent); dit: 143 linears of a width-1152,
    depth-28 diffusion transformer (batch 32, 256 tokens)."""
    import torch
    from paper_2512_05746_b200 import binding as hq
    from paper_2512_05746_b200 import dit, unet
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    if which == "unet":
        layers = unet.quantized_layers()
        label = "the 121 quantized layers of the UNet-shaped workload (batch 64, 64x64 latent)"
        wl = "configs[3] quantized layers only: 121 layers, 47 distinct shapes"
    else:
        layers = dit.quantized_layers()
        label = "the 143 quantized linears of the DiT-XL/2-shaped workload (batch 32, 256 tokens, width 1152 = 9 x 128)"
        wl = "DiT-XL/2-shaped quantized linears: 28 blocks x (adaLN, QKV, proj, FC1, FC2) + embedding MLP"
    gen = torch.Generator(device=dev)
    gen.manual_seed(0)
    cache = {}

    def key(L):
        return ("conv", L["Nb"], L["H"], L["C"], L["Cout"], L["R"], L["stride"]) if L["kind"] == "conv" else \
               ("linear", L["M"], L["K"], L["N"])

    status = torch.zeros((1,), dtype=torch.int32, device=dev)
    for L in layers:
        k = key(L)
        if k in cache:
            L["res"] = cache[k]
            continue
        if L["kind"] == "conv":
            rows, cin, cout = L["Nb"] * L["H"] * L["W"], L["C"], L["Cout"]
            wshape = (cout, L["R"], L["R"], cin)
            ho = L["H"] // L["stride"]
            oshape = (L["Nb"], ho, ho, cout)
        else:
            rows, cin, cout = L["M"], L["K"], L["N"]
            wshape = (cout, cin)
            oshape = (rows, cout)
        x = torch.randn((rows, cin), generator=gen, device=dev, dtype=torch.float32)
        nout = max(1, round(0.01 * cin))
        x[:, torch.randperm(cin, generator=gen, device=dev)[:nout]] *= 20.0          # outlier channels
        x = x.to(torch.bfloat16)
        pw = hq.hq_weight_prepare(inputs.weights(wshape, seed=len(cache)), W_BITS, L["had_block"], hq.HQ_W_FOLDED,
                                  CODES[0]).to_device(dev)
        res = dict(x=x.view((L["Nb"], L["H"], L["W"], cin)) if L["kind"] == "conv" else x, pw=pw,
                   bias=torch.from_numpy(inputs.bias(cout, seed=len(cache))).to(dev),
                   y=torch.empty(oshape, dtype=torch.bfloat16, device=dev),
                   ws=torch.empty((hq.hq_workspace_size(rows, cin, CODES[0]),), dtype=torch.uint8, device=dev),
                   static=None)
        if L["kind"] == "conv" and L["R"] == 3:           # calibrate the static scale with one dynamic pass
            codes = torch.empty((rows, code_pitch(cin)), dtype=torch.uint8, device=dev)
            sc = torch.empty((rows,), dtype=torch.float32, device=dev)
            hq.hq_hadamard_quant(x, L["had_block"], A_BITS, codes, CODES[0], scales=sc)
            res["static"] = sc.max().reshape(1).contiguous()
            del codes, sc
        cache[k] = res
        L["res"] = res
    torch.cuda.synchronize()

    def forward():
        for L in layers:
            r = L["res"]
            if L["kind"] == "conv":
                hq.hq_qconv(r["x"], r["pw"], L["R"], L["R"], L["stride"], L["pad"], r["bias"], A_BITS, r["y"], r["ws"],
                            static_scale=r["static"], dev_status=status)
            else:
                hq.hq_qlinear(r["x"], r["pw"], r["bias"], A_BITS, r["y"], r["ws"], dev_status=status)

    steps, warmup = max(1, min(args.steps, 10)), max(3, min(args.warmup, 5))
    for _ in range(warmup):
        forward()
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        forward()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    t_stop = time.time() + CLOCK_WINDOW_S      # nvidia-smi samples every 100 ms: keep the same load running for them
    while time.time() < t_stop:
        forward()
        torch.cuda.synchronize()
    clocks = sampler.stop()
    clocks["window"] = f"timed region + {CLOCK_WINDOW_S} s of the same forwards, untimed"
    hq.hq_check_status(status)
    # one more pass with an event after every layer: time and TOPS per distinct shape
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(len(layers) + 1)]
    evs[0].record()
    for i, L in enumerate(layers):
        r = L["res"]
        if L["kind"] == "conv":
            hq.hq_qconv(r["x"], r["pw"], L["R"], L["R"], L["stride"], L["pad"], r["bias"], A_BITS, r["y"], r["ws"],
                        static_scale=r["static"], dev_status=status)
        else:
            hq.hq_qlinear(r["x"], r["pw"], r["bias"], A_BITS, r["y"], r["ws"], dev_status=status)
        evs[i + 1].record()
    torch.cuda.synchronize()
    per_shape = {}
    for i, L in enumerate(layers):
        d = per_shape.setdefault(str(key(L)), dict(count=0, ms=0.0, macs=L["macs"], limbs=L["res"]["pw"].desc.limbs))
        d["count"] += 1
        d["ms"] += evs[i].elapsed_time(evs[i + 1])
    for d in per_shape.values():
        d["ms_each"] = d["ms"] / d["count"]
        d["tops"] = 2.0 * d["macs"] * d["limbs"] / (d["ms_each"] * 1e-3) / 1e12
    # The UNet's residual-block convolutions take SiLU(GroupNorm32(h)) as input: the same forward with that prologue
    # fused into the transform kernel of those layers (statistics pass + normalise-on-load), reported beside the main figure.
    gn_extra = None
    if which == "unet":
        gn_layers = [L for L in layers if L["kind"] == "conv" and L["R"] == 3 and L["stride"] == 1 and
                     (".conv1" in L["name"] or ".conv2" in L["name"])]
        for L in gn_layers:
            r = L["res"]
            if "gn" in r:
                continue
            cin, rows = L["C"], L["Nb"] * L["H"] * L["W"]
            g = dict(gamma=torch.ones((cin,), device=dev), beta=torch.zeros((cin,), device=dev),
                     scratch=torch.empty((L["Nb"] * 32 * 24,), dtype=torch.uint8, device=dev))
            codes, sc = ws_views(torch, r["ws"], rows, cin)
            hq.hq_gn_silu_quant(r["x"], 32, g["gamma"], g["beta"], 1e-5, L["had_block"], A_BITS, codes, CODES[0], g["scratch"],
                                scales=sc)
            g["static"] = sc.max().reshape(1).contiguous()          # one static scale, calibrated on the normalised input
            r["gn"] = g
        torch.cuda.synchronize()
        gn_names = {L["name"] for L in gn_layers}

        def forward_gn():
            for L in layers:
                r = L["res"]
                if L["name"] in gn_names:
                    g = r["gn"]
                    hq.hq_gn_silu_qconv(r["x"], 32, g["gamma"], g["beta"], 1e-5, r["pw"], L["R"], L["R"], L["stride"], L["pad"],
                                        r["bias"], A_BITS, r["y"], r["ws"], g["scratch"], static_scale=g["static"],
                                        dev_status=status)
                elif L["kind"] == "conv":
                    hq.hq_qconv(r["x"], r["pw"], L["R"], L["R"], L["stride"], L["pad"], r["bias"], A_BITS, r["y"], r["ws"],
                                static_scale=r["static"], dev_status=status)
                else:
                    hq.hq_qlinear(r["x"], r["pw"], r["bias"], A_BITS, r["y"], r["ws"], dev_status=status)

        for _ in range(3):
            forward_gn()
        torch.cuda.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for _ in range(steps):
            forward_gn()
        g1.record()
        torch.cuda.synchronize()
        hq.hq_check_status(status)
        gn_extra = dict(ms_per_step=g0.elapsed_time(g1) / steps, layers_with_prologue=len(gn_layers),
                        note="GroupNorm(32) + SiLU fused in front of the residual-block 3x3 convolutions "
                             "(hq_gn_silu_qconv)")
    # The transformer's QKV and FC1 linears take modulate(LayerNorm(x), shift, scale) as input: the same forward with that
    # prologue fused into the transform kernel of those layers (row statistics from the registers that hold the row).
    ln_extra = None
    if which == "dit":
        ln_names = {L["name"] for L in layers if L["name"].endswith(".qkv") or L["name"].endswith(".fc1")}
        tokens = 256
        for L in layers:
            r = L["res"]
            if L["name"] in ln_names and "ln" not in r:
                groups = L["M"] // tokens
                r["ln"] = dict(w=1.0 + 0.1 * torch.randn((groups, L["K"]), generator=gen, device=dev),
                               b=0.1 * torch.randn((groups, L["K"]), generator=gen, device=dev))

        def forward_ln():
            for L in layers:
                r = L["res"]
                if L["name"] in ln_names:
                    hq.hq_ln_qlinear(r["x"], r["ln"]["w"], r["ln"]["b"], tokens, 1e-6, r["pw"], r["bias"], A_BITS, r["y"], r["ws"],
                                     dev_status=status)
                else:
                    hq.hq_qlinear(r["x"], r["pw"], r["bias"], A_BITS, r["y"], r["ws"], dev_status=status)

        for _ in range(3):
            forward_ln()
        torch.cuda.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for _ in range(steps):
            forward_ln()
        g1.record()
        torch.cuda.synchronize()
        hq.hq_check_status(status)
        # the prologue alone against the plain transform on the block input (8192 x 1152 bf16)
        Lq = next(L for L in layers if L["name"].endswith(".qkv"))
        rq = Lq["res"]
        cq, sq = ws_views(torch, rq["ws"], Lq["M"], Lq["K"])

        def t_of(fn):
            for _ in range(5):
                fn()
            torch.cuda.synchronize()
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record()
            for _ in range(20):
                fn()
            a1.record()
            torch.cuda.synchronize()
            return a0.elapsed_time(a1) / 20

        ln_us = 1e3 * t_of(lambda: hq.hq_ln_quant(rq["x"], rq["ln"]["w"], rq["ln"]["b"], tokens, 1e-6, Lq["had_block"], A_BITS,
                                                  cq, CODES[0], scales=sq))
        pl_us = 1e3 * t_of(lambda: hq.hq_hadamard_quant(rq["x"], Lq["had_block"], A_BITS, cq, CODES[0], scales=sq))
        ln_extra = dict(ms_per_step=g0.elapsed_time(g1) / steps, layers_with_prologue=len(ln_names),
                        ln_quant_us=ln_us, plain_quant_us=pl_us,
                        note="LayerNorm + per-sample modulation fused in front of the QKV and FC1 linears (hq_ln_qlinear)")
    macs = sum(L["macs"] for L in layers)
    ops_limbs = sum(2.0 * L["macs"] * L["res"]["pw"].desc.limbs for L in layers)
    print(json.dumps(dict(metric="forwards/s of " + label,
                          value=1e3 / ms, unit="forwards/s", n_gpus=1, steps=steps, warmup=warmup, ms_per_step=ms,
                          higher_is_better=True, scaling="weak", vs_baseline=None, dtype="int8", data="synthetic",
                          config=dict(workload=wl + f", bf16 in/out, W4A{A_BITS} folded two-limb weights, " + codes_name() + " codes",
                                      layers=len(layers),
                                      layers_per_s=len(layers) * 1e3 / ms, tops_limbs=ops_limbs / ms / 1e9,
                                      tops_1limb_equiv=2.0 * macs / ms / 1e9,
                                      l2="activations of the large layers exceed L2"),
                          clocks=clocks, gpu_launches=2 * len(layers) * steps, per_shape=per_shape,
                          with_groupnorm_prologue=gn_extra, with_layernorm_prologue=ln_extra)))


def main_sweep(args):
    """Shape sweep of transform+quantize followed by the integer GEMM: M x K x N grid, Hadamard block = K, for
    W4A4 with the folded two-limb weights, W4A4 with plain one-limb weights (codes in the container --codes selects) and
    W8A8 (plain weights).  W4A3 runs the same kernels as W4A4 (only the quantizer range differs).  One JSON
    line with one record per point: int TOPS of the GEMM, GB/s of the quantize stage, and the roofline fraction of
    the GEMM (slower of tensor peak and algorithmic bytes over the measured copy bandwidth)."""
    import torch
    from paper_2512_05746_b200 import binding as hq
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    pk = peaks()
    int8_peak = 2.0 * pk["bf16_sustained"]
    Ms, Ks, Ns = (4096, 16384, 65536), (256, 512, 1024, 2048, 4096), (512, 1280, 4096)
    if args.rows != M_TOKENS:
        Ms = (int(args.rows),)
    variants = (("W4A4 folded", 4, 4, hq.HQ_W_FOLDED, CODES[0]),
                ("W4A4 plain", 4, 4, hq.HQ_W_PLAIN, CODES[0]),
                ("W8A8 plain", 8, 8, hq.HQ_W_PLAIN, hq.HQ_CODES_INT8))
    status = torch.zeros((1,), dtype=torch.int32, device=dev)
    gen = torch.Generator(device=dev)
    gen.manual_seed(0)
    reps = max(3, min(args.steps, 50))
    points = []

    def timed(fn):
        for _ in range(10):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    for K in Ks:
        for N in Ns:
            w = inputs.weights((N, K), seed=K + N)
            pws = {v[0]: hq.hq_weight_prepare(w, v[2], K, v[3], v[4]).to_device(dev) for v in variants}
            b = torch.from_numpy(inputs.bias(N, seed=N)).to(dev)
            for M in Ms:
                x = torch.randn((M, K), generator=gen, device=dev, dtype=torch.float32)
                x[:, torch.randperm(K, generator=gen, device=dev)[: max(1, round(0.01 * K))]] *= 20.0
                y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
                for name, a_bits, w_bits, mode, cont in variants:
                    pw = pws[name]
                    pitch = K // 2 if cont == hq.HQ_CODES_NIBBLE else K
                    codes = torch.empty((M, pitch), dtype=torch.uint8, device=dev)
                    sc = torch.empty((M,), dtype=torch.float32, device=dev)
                    q_ms = timed(lambda: hq.hq_hadamard_quant(x, K, a_bits, codes, cont, scales=sc))
                    g_ms = timed(lambda: hq.hq_qgemm(codes, cont, a_bits, K, pw, scale_a=sc, bias=b, alpha=pw.alpha, y=y,
                                                     dev_status=status))
                    limbs = pw.desc.limbs
                    ops = 2.0 * M * N * K * limbs
                    gbytes = M * pitch + N * K * limbs + M * N * 2.0 + 4.0 * M + 8.0 * N
                    t_tensor, t_hbm = ops / (int8_peak * 1e12), gbytes / (pk["hbm_gbs"] * 1e9)
                    qbytes = M * K * 4.0 + M * pitch + 4.0 * M
                    points.append(dict(M=M, K=K, N=N, variant=name, limbs=limbs, quant_us=q_ms * 1e3, gemm_us=g_ms * 1e3,
                                       gemm_tops=ops / g_ms / 1e9, quant_gbs=qbytes / q_ms / 1e6,
                                       bound="tensor" if t_tensor >= t_hbm else "hbm",
                                       roofline_frac=max(t_tensor, t_hbm) / (g_ms * 1e-3),
                                       quant_frac=qbytes / q_ms / 1e6 / pk["hbm_gbs"]))
                del x, y
    hq.hq_check_status(status)
    best = max(points, key=lambda d: d["gemm_tops"])
    print(json.dumps(dict(metric="shape sweep: int TOPS of the GEMM and GB/s of transform+quantize per point", value=best["gemm_tops"],
                          unit="TOPS (best point)", n_gpus=1, steps=reps, warmup=10, higher_is_better=True, dtype="int8",
                          data="synthetic", vs_baseline=None,
                          config=dict(workload="configs[4] shape sweep, " + codes_name() + " codes for W4A4", int8_peak_tops=int8_peak, hbm_gbs=pk["hbm_gbs"],
                                      peak_source=pk["source"]), points=points)))


def main_gn(args):
    """GroupNorm(32) + SiLU + transform + quantize on one NHWC bf16 tensor (64 x 64 x 64 x 256, the input of a UNet
    residual-block convolution), beside the plain transform + quantize of the same tensor."""
    import torch
    from paper_2512_05746_b200 import binding as hq
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    Nb, H, W, Cc = 64, 64, 64, 256
    gen = torch.Generator(device=dev)
    gen.manual_seed(0)
    x = (torch.randn((Nb, H, W, Cc), generator=gen, device=dev) * 1.5 + 0.3).to(torch.bfloat16)
    gamma = torch.rand((Cc,), generator=gen, device=dev) + 0.5
    beta = torch.randn((Cc,), generator=gen, device=dev) * 0.1
    rows = Nb * H * W
    codes = torch.empty((rows, code_pitch(Cc)), dtype=torch.uint8, device=dev)
    sc = torch.empty((rows,), dtype=torch.float32, device=dev)
    scratch = torch.empty((Nb * 32 * 24,), dtype=torch.uint8, device=dev)
    steps, warmup = max(1, min(args.steps, 20)), max(3, min(args.warmup, 5))

    def timed(fn):
        for _ in range(warmup):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps

    gn_ms = timed(lambda: hq.hq_gn_silu_quant(x, 32, gamma, beta, 1e-5, 256, A_BITS, codes, CODES[0], scratch, scales=sc))
    plain_ms = timed(lambda: hq.hq_hadamard_quant(x.view(rows, Cc), 256, A_BITS, codes, CODES[0], scales=sc))
    cb = code_pitch(2) / 2.0
    gbytes = x.numel() * (2 * 2.0 + cb) + rows * 4.0                     # x read twice, codes and scales written
    pk = peaks()
    print(json.dumps(dict(metric="GB/s of GroupNorm+SiLU+transform+quantize (x read twice + codes written)",
                          value=gbytes / gn_ms / 1e6, unit="GB/s", n_gpus=1, steps=steps, warmup=warmup, ms_per_step=gn_ms,
                          higher_is_better=True, dtype="f32", data="synthetic", vs_baseline=None,
                          config=dict(workload=f"GroupNorm(32)+SiLU prologue on {Nb}x{H}x{W}x{Cc} bf16, {codes_name()} codes"),
                          plain_transform_quantize_ms=plain_ms, frac_of_copy_bandwidth=gbytes / gn_ms / 1e6 / pk["hbm_gbs"],
                          gpu_launches=3 * steps)))


def main():
    global M_TOKENS, WORKLOAD, A_BITS, METRIC
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workload", default="step", choices=["step", "unet", "dit", "sweep", "gn"],
                    help="step: the benchmark step (default); unet / dit: the quantized layers of the UNet- / DiT-shaped workload; "
                         "sweep: the M x K x N shape sweep; gn: the GroupNorm+SiLU prologue on one tensor")
    ap.add_argument("--a-bits", type=int, default=4, choices=[3, 4],
                    help="activation bits of the step / unet / dit workloads (INT3 codes travel in the same containers)")
    ap.add_argument("--codes", default="int8", choices=["nibble", "int8"],
                    help="container of the 4-bit activation codes between the transform and the GEMM kernel: one per "
                         "byte (default, the faster one) or two per byte (half the workspace)")
    ap.add_argument("--rows", type=int, default=M_TOKENS,
                    help="rows per layer (default: the full 32768; smaller values are for profiler captures only)")
    args = ap.parse_args()
    CODES[0] = 0 if args.codes == "nibble" else 1
    WORKLOAD = WORKLOAD + f", {args.codes} codes"
    if args.a_bits != 4:
        A_BITS = int(args.a_bits)
        WORKLOAD = WORKLOAD.replace("W4A4", f"W4A{A_BITS}")
        METRIC = METRIC.replace("W4A4", f"W4A{A_BITS}")
    if args.rows != M_TOKENS:
        M_TOKENS = int(args.rows)
        WORKLOAD = f"REDUCED to {M_TOKENS} rows per layer (profiling case, not a benchmark number): " + WORKLOAD
    if args.impl == "reference":
        return main_reference(args)
    if args.workload in ("unet", "dit"):
        return main_layer_list(args, args.workload)
    if args.workload == "sweep":
        return main_sweep(args)
    if args.workload == "gn":
        return main_gn(args)

    import torch
    import torch.distributed as dist
    from paper_2512_05746_b200 import binding as hq

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (the CUDA path has no CPU fallback)")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

    warmup = max(args.warmup, 3)
    layers = build_layers(torch, hq, device, seed=rank)
    status = torch.zeros((1,), dtype=torch.int32, device=device)
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident throughput ---------------------------------------------------------------
    for _ in range(warmup):
        run_step(hq, layers, status)
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for _ in range(args.steps):
        run_step(hq, layers, status)
    e1.record(stream)
    barrier()
    ms = e0.elapsed_time(e1)
    # The timed region lasts a few milliseconds and nvidia-smi samples every 100 ms: keep the identical load running
    # (untimed) for a moment longer so that the samples are taken under it.
    t_stop = time.time() + CLOCK_WINDOW_S
    while time.time() < t_stop:
        for _ in range(20):
            run_step(hq, layers, status)
        torch.cuda.synchronize()
    clocks = sampler.stop()
    clocks["window"] = f"timed region + {CLOCK_WINDOW_S} s of the same steps, untimed"
    hq.hq_check_status(status)

    # ---- per-kernel attribution (same kernels, events between the two launches of each layer) -----------
    evs = []
    for _ in range(args.steps):
        run_step_split(torch, hq, layers, status, evs)
    torch.cuda.synchronize()
    per = {}
    for L, a, b, c in evs:
        d = per.setdefault(L["name"], dict(quant_ms=0.0, gemm_ms=0.0, n=0, L=L))
        d["quant_ms"] += a.elapsed_time(b)
        d["gemm_ms"] += b.elapsed_time(c)
        d["n"] += 1

    # ---- the same convolution with the width-axis transform (the paper's literal form; one weight limb) ----------
    width = None
    if rank == 0:
        Lc = [L for L in layers if L["kind"] == "conv"][0]
        c = CONV
        pw_w = hq.hq_weight_prepare(inputs.config_conv_small(seed=rank, batch=1)["w"], W_BITS, 1, hq.HQ_W_PLAIN,
                                    hq.HQ_CODES_INT8).to_device(device)
        ws_w = torch.empty((hq.hq_workspace_size(Lc["rows"], Lc["cols"], hq.HQ_CODES_INT8),), dtype=torch.uint8, device=device)
        zbuf = torch.empty((Lc["rows"], Lc["cols"]), dtype=torch.int8, device=device)

        def width_layer():
            hq.hq_qconv_width(Lc["x"], pw_w, c["R"], c["S"], c["stride"], c["pad"], Lc["bias"], A_BITS, 16,
                              Lc["static_scale"], Lc["y"], ws_w, dev_status=status)

        def width_quant():
            hq.hq_hadamard_quant_width(Lc["x"], 16, A_BITS, Lc["static_scale"], zbuf.view(Lc["x"].shape))

        res = []
        for fn in (width_layer, width_quant):
            for _ in range(3):
                fn()
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            g0.record(stream)
            for _ in range(args.steps):
                fn()
            g1.record(stream)
            torch.cuda.synchronize()
            res.append(g0.elapsed_time(g1) / args.steps)
        width = dict(layer_ms=res[0], quant_ms=res[1], tops_1limb=Lc["ops_1limb"] / (res[0] * 1e-3) / 1e12,
                     quant_gbs=Lc["rows"] * Lc["cols"] * 5.0 / (res[1] * 1e-3) / 1e9,
                     note="3x3 conv of the step with the transform along the width axis (16-point blocks), "
                          "untransformed one-limb weights, int8 activations")

    # ---- end to end: pinned host input -> device -> fused call -> host output -----------------------
    e2e_steps = max(2, min(args.steps, 5))
    h2d = sum(L["x_host"].numel() * L["x_host"].element_size() for L in layers)
    d2h = sum(L["y_host"].numel() * L["y_host"].element_size() for L in layers)

    # Three streams: inputs go up on one, the layer calls run on the main one as each input lands, results come down
    # on the third as each layer finishes; the timed region is bracketed on the main stream, which waits for the last
    # download of a step before the next step's uploads may overwrite anything.
    up, down = torch.cuda.Stream(device=device), torch.cuda.Stream(device=device)

    def e2e_step():
        ev_start = torch.cuda.Event()
        ev_start.record(stream)
        up.wait_event(ev_start)
        landed, done = [], []
        with torch.cuda.stream(up):
            for L in layers:
                L["x"].copy_(L["x_host"], non_blocking=True)
                e = torch.cuda.Event()
                e.record(up)
                landed.append(e)
        for L, e in zip(layers, landed):
            stream.wait_event(e)
            if L["kind"] == "linear":
                hq.hq_qlinear(L["x"], L["pw"], L["bias"], A_BITS, L["y"], L["ws"], dev_status=status, stream=stream)
            else:
                c = CONV
                hq.hq_qconv(L["x"], L["pw"], c["R"], c["S"], c["stride"], c["pad"], L["bias"], A_BITS, L["y"], L["ws"],
                            static_scale=L["static_scale"], dev_status=status, stream=stream)
            e2 = torch.cuda.Event()
            e2.record(stream)
            done.append(e2)
        with torch.cuda.stream(down):
            for L, e2 in zip(layers, done):
                down.wait_event(e2)
                L["y_host"].copy_(L["y"], non_blocking=True)
            ev_end = torch.cuda.Event()
            ev_end.record(down)
        stream.wait_event(ev_end)

    e2e_step()
    barrier()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    f1.record(stream)
    barrier()
    e2e_ms = f0.elapsed_time(f1)

    from paper_2512_05746_b200.sharding import max_over_ranks
    ms, e2e_ms = max_over_ranks(ms, device), max_over_ranks(e2e_ms, device)

    ops_step = sum(L["ops"] for L in layers)
    ops_step_1 = sum(L["ops_1limb"] for L in layers)
    value = ops_step * args.steps * world / (ms * 1e-3) / 1e12
    e2e_value = ops_step * e2e_steps * world / (e2e_ms * 1e-3) / 1e12

    if rank == 0:
        pk = peaks()
        int8_peak = 2.0 * pk["bf16_sustained"]          # int8 : bf16 nominal dense ratio is 2 (4.5 : 2.25 PFLOP/s)
        dom = max(per.values(), key=lambda d: d["gemm_ms"])      # dominant kernel: the longest GEMM launch
        L = dom["L"]
        gemm_ms = dom["gemm_ms"] / dom["n"]
        ach = L["ops"] / (gemm_ms * 1e-3) / 1e12
        roofline = dict(bound="tensor", kernel=f"qgemm_kernel<{codes_name()}> ({L['name']}: M={L['M']} K={L['K']} N={L['N']} "
                                                f"limbs={L['limbs']})",
                        achieved=ach, peak=int8_peak, unit="TOPS", frac=ach / int8_peak,
                        traffic=NCU_DRAM_BYTES["gemm"].get(L["name"]) if (M_TOKENS == 32768 and CODES[0] == NCU_DRAM_CODES) else None,
                        algorithmic_bytes=L["gemm_bytes"],
                        peak_source=f"2 x bf16 sustained ({pk['source']})", launch_ms=gemm_ms)
        qd = max(per.values(), key=lambda d: d["quant_ms"])
        q_ms = qd["quant_ms"] / qd["n"]
        q_gbs = qd["L"]["quant_bytes"] / (q_ms * 1e-3) / 1e9
        roofline_quant = dict(bound="hbm", kernel=f"fwht_quant_fast ({qd['L']['name']}: {qd['L']['rows']}x{qd['L']['cols']})",
                              achieved=q_gbs, peak=pk["hbm_gbs"], unit="GB/s", frac=q_gbs / pk["hbm_gbs"],
                              traffic=NCU_DRAM_BYTES["quant"].get(qd["L"]["name"]) if (M_TOKENS == 32768 and CODES[0] == NCU_DRAM_CODES) else None,
                              algorithmic_bytes=qd["L"]["quant_bytes"],
                              peak_source=f"copy bandwidth ({pk['source']})", launch_ms=q_ms)
        per_layer = {k: dict(quant_ms=d["quant_ms"] / d["n"], gemm_ms=d["gemm_ms"] / d["n"],
                             gemm_tops=d["L"]["ops"] / (d["gemm_ms"] / d["n"] * 1e-3) / 1e12,
                             quant_gbs=d["L"]["quant_bytes"] / (d["quant_ms"] / d["n"] * 1e-3) / 1e9)
                     for k, d in per.items()}
        line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=warmup,
                    ms_per_step=ms / args.steps, higher_is_better=True, scaling="weak", vs_baseline=None,
                    dtype="int8", data="synthetic",
                    config=dict(workload=WORKLOAD, l2="inputs larger than L2 (0.5 GB read per step)",
                                tops_1limb_equiv=ops_step_1 * args.steps * world / (ms * 1e-3) / 1e12,
                                layers_per_s=len(layers) * args.steps * world / (ms * 1e-3)),
                    clocks=clocks, gpu_launches=2 * len(layers) * args.steps,
                    e2e=dict(value=e2e_value, unit=UNIT, h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h,
                             steps=e2e_steps, ms_per_step=e2e_ms / e2e_steps),
                    roofline=roofline, roofline_fwht_quant=roofline_quant, per_layer=per_layer,
                    width_axis_conv=width)
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline()
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
