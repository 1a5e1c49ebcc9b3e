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

METRIC = "int TOPS (2*M*N*K, the W4A4 layers' own work) of the fused Hadamard-quant linear+conv step"
UNIT = "TOPS"
PASSES_PER_STEP = 100      # one step = this many passes over the batch, so that 20 steps last about 0.6 s on the device
M_TOKENS = 32768
CONV = dict(Nb=32, H=32, W=32, C=256, Cout=256, R=3, S=3, stride=1, pad=1, had_block=256)
WORKLOAD = ("configs[2] transformer-block linears (M=32768; QKV, out-proj, FF1, FF2) + configs[1] 3x3 conv at "
            "batch 32 (M=32768, K=2304, N=256); W4A4, folded 2-limb weights, bf16 out")
A_BITS, W_BITS = 4, 4
# Container of the 4-bit activation codes between the two kernels of a layer: 0 = HQ_CODES_NIBBLE (two per byte,
# unpacked inside the GEMM kernel), 1 = HQ_CODES_INT8 (one per byte); set by --codes.
CODES = [1]


def code_pitch(cols):
    """Bytes per row of `cols` codes in the selected container."""
    return cols // 2 if CODES[0] == 0 else cols


def codes_name():
    return "nibble" if CODES[0] == 0 else "int8"


def gemm_kernel_name(L):
    """The kernel the library's default dispatch takes for a layer of the step (see hq_set_pair_gemm in include/hq.h)."""
    if codes_name() != "int8":
        return "qgemm_kernel<nibble>"
    if L["kind"] == "conv" or L["K"] > 512:
        return "qgemm_pair_stream_kernel (pairs of SMs, streamed weights)"
    if L["K"] == 512 and L.get("limbs", 2) == 2:
        return "qgemm_pair_kernel (pairs of SMs, resident weights, two K blocks per ring stage)"
    return "qgemm_kernel<int8>"


def ws_views(torch, ws, rows, cols):
    """Codes [rows, pitch] and scales [rows] inside the workspace of a fused layer call (the documented layout)."""
    pitch = (code_pitch(cols) + 15) // 16 * 16
    off = (rows * pitch + 255) // 256 * 256
    return ws[: rows * pitch].view(rows, pitch), ws[off: off + rows * 4].view(torch.float32)


STEP_KERNEL_SOURCES = ("hq_common.cuh", "hq_fwht.cuh", "hq_quant.cu", "hq_gemm_kernel.cuh", "hq_gemm.cu", "hq_gemm_pair.cu", "hq_api.cu",
                       "hq_gemm_inst_i8_gemm.cu", "hq_gemm_inst_i8_conv.cu", "hq_gemm_inst_nibble_gemm.cu",
                       "hq_gemm_inst_nibble_conv.cu")


def csrc_digest():
    """SHA-256 over the sources of the kernels the default step launches (transform + quantize, integer GEMM / conv and
    their launchers): identifies the kernels a profile was taken with."""
    import hashlib
    h = hashlib.sha256()
    for name in STEP_KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2512_05746_b200", "csrc", name), "rb") as fh:
            h.update(name.encode() + b"\0" + fh.read())
    return h.hexdigest()[:16]


def measured_traffic():
    """dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu capture recorded in
    profiles/dram_traffic.json, or {} when the kernels have changed since it was taken (the record carries the digest of
    the sources it was captured with), or when it was taken with another container or row count."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(path):
        return {}
    with open(path) as f:
        rec = json.load(f)
    if rec.get("csrc_digest") != csrc_digest() or rec.get("rows") != M_TOKENS or rec.get("codes") != codes_name():
        return {}
    return rec


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

def build_layers(torch, hq, device, seed, cont=None, share=None, weight_mode=None):
    """Synthetic inputs and offline-prepared weights for every layer of the step, resident on `device`.
    cont: container of the codes (default: the one --codes selected); share: layers built earlier whose inputs, biases
    and outputs are reused (only weights and workspaces are made anew); weight_mode: default FOLDED."""
    cont = CODES[0] if cont is None else cont
    mode = hq.HQ_W_FOLDED if weight_mode is None else weight_mode
    cb = 0.5 if cont == 0 else 1.0                                           # bytes per code
    layers = layer_list()
    for i, L in enumerate(layers):
        if L["kind"] == "linear":
            cfg = inputs.config_transformer_linear(L["name"], M=64 if share else L["M"], seed=seed)
        else:
            cfg = inputs.config_conv_small(seed=seed, batch=1 if share else CONV["Nb"])
        w, b = cfg["w"], cfg["bias"]
        pw = hq.hq_weight_prepare(w, W_BITS, L["had_block"], mode, cont).to_device(device)
        L["pw"] = pw
        L["limbs"] = pw.desc.limbs
        rows, cols = (L["M"], L["K"]) if L["kind"] == "linear" else (L["M"], CONV["C"])
        L["rows"], L["cols"] = rows, cols
        oshape = (L["M"], L["N"]) if L["kind"] == "linear" else (CONV["Nb"], CONV["H"], CONV["W"], CONV["Cout"])
        if share:
            for key in ("x_host", "x", "bias", "y", "y_host", "static_scale"):
                L[key] = share[i][key]
        else:
            L["x_host"] = torch.from_numpy(cfg["x"]).pin_memory()
            L["x"] = L["x_host"].to(device, non_blocking=True)
            L["bias"] = torch.from_numpy(b).to(device)
            L["y"] = torch.empty(oshape, dtype=torch.bfloat16, device=device)
            L["y_host"] = torch.empty(oshape, dtype=torch.bfloat16).pin_memory()
            L["static_scale"] = None
        L["cont"] = cont
        L["ws"] = torch.empty((hq.hq_workspace_size(rows, cols, cont),), dtype=torch.uint8, device=device)
        L["ops"] = 2.0 * L["M"] * L["N"] * L["K"] * L["limbs"]
        L["ops_1limb"] = 2.0 * L["M"] * L["N"] * L["K"]
        # algorithmic HBM bytes of the two kernels (fp32 in, codes out + scales; codes + weights in, bf16 out)
        L["quant_bytes"] = rows * cols * 4.0 + rows * cols * cb + rows * 4.0
        L["gemm_bytes"] = rows * cols * cb + L["N"] * L["K"] * L["limbs"] + L["M"] * L["N"] * 2.0 + 4.0 * L["M"] + 8.0 * L["N"]
    torch.cuda.synchronize()
    # The conv uses one static activation scale (the paper's learned per-tensor scale): calibrate it once with the
    # library's own dynamic pass: S = max over pixels of the per-pixel scale.
    for L in layers:
        if L["kind"] == "conv" and L["static_scale"] is None:
            x2d = L["x"].view(L["rows"], L["cols"])
            pitch = L["cols"] // 2 if cont == 0 else L["cols"]
            codes = torch.empty((L["rows"], pitch), dtype=torch.uint8, device=device)
            scales = torch.empty((L["rows"],), dtype=torch.float32, device=device)
            hq.hq_hadamard_quant(x2d, L["had_block"], A_BITS, codes, cont, scales=scales)
            L["static_scale"] = scales.max().reshape(1).contiguous()
    torch.cuda.synchronize()
    return layers


def run_step(hq, layers, status, stream=None, a_bits=None, per_pixel_conv=False):
    """One pass: every layer of the step through its fused entry point."""
    a_bits = A_BITS if a_bits is None else a_bits
    for L in layers:
        if L["kind"] == "linear":
            hq.hq_qlinear(L["x"], L["pw"], L["bias"], a_bits, L["y"], L["ws"], dev_status=status, stream=stream)
        else:
            c = CONV
            hq.hq_qconv(L["x"], L["pw"], c["R"], c["S"], c["stride"], c["pad"], L["bias"], a_bits, L["y"], L["ws"],
                        static_scale=None if per_pixel_conv else L["static_scale"], dev_status=status, stream=stream)


def split_views(torch, L):
    rows, cols = L["rows"], L["cols"]
    pitch = cols // 2 if L["cont"] == 0 else cols
    codes = L["ws"][: rows * pitch].view(rows, pitch)
    off = (rows * pitch + 255) // 256 * 256
    return codes, L["ws"][off: off + rows * 4].view(torch.float32)


def run_step_split(torch, hq, layers, status, evs, gemm_only=False):
    """Same kernels as run_step, launched through the unfused entry points with an event between them."""
    stream = torch.cuda.current_stream()
    for L in layers:
        rows, cols, cont = L["rows"], L["cols"], L["cont"]
        codes, scales = split_views(torch, L)
        x2d = L["x"].view(rows, cols)
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        e0.record(stream)
        if L["kind"] == "linear":
            if not gemm_only:
                hq.hq_hadamard_quant(x2d, L["had_block"], A_BITS, codes, cont, scales=scales)
            e1.record(stream)
            hq.hq_qgemm(codes, cont, A_BITS, L["K"], L["pw"], scale_a=scales, bias=L["bias"],
                        alpha=L["pw"].alpha, y=L["y"], dev_status=status)
        else:
            c = CONV
            if not gemm_only:
                hq.hq_hadamard_quant(x2d, L["had_block"], A_BITS, codes, cont, scales=scales[:1],
                                     static_scale=L["static_scale"])
            e1.record(stream)
            hq.hq_qconv2d(codes, cont, A_BITS, c["Nb"], c["H"], c["W"], c["C"], L["pw"], c["R"], c["S"],
                          c["stride"], c["pad"], scale_a=L["static_scale"], bias=L["bias"], alpha=L["pw"].alpha,
                          y=L["y"], dev_status=status)
        e2.record(stream)
        evs.append((L, e0, e1, e2))


def measure_variants(torch, hq, device, layers, status, stream, rank):
    """The measurements that sit beside the headline in the same JSON line: the step with two codes per byte (the packed
    layout, unpacked inside the GEMM kernel), with INT3 activations, the 3x3 convolution with per-pixel scales (accumulator
    drained per filter tap), every GEMM with one-limb weights (what the fold of Eq. 12 costs), and the convolution in the
    paper's width-axis form."""
    out = {}
    reps = 200

    def per_pass(fn):
        for _ in range(10):
            fn()
        return timed_region(torch, fn, reps, stream) / reps

    ops1 = sum(L["ops_1limb"] for L in layers)
    # --- the other container
    other = 0 if layers[0]["cont"] == 1 else 1
    alt = build_layers(torch, hq, device, seed=rank, cont=other, share=layers)
    ms_alt = per_pass(lambda: run_step(hq, alt, status))
    evs = []
    for _ in range(30):
        run_step_split(torch, hq, alt, status, evs)
    torch.cuda.synchronize()
    per = {}
    for L, a, b, c in evs:
        d = per.setdefault(L["name"], dict(q=[], g=[], L=L))
        d["q"].append(a.elapsed_time(b))
        d["g"].append(b.elapsed_time(c))
    out["nibble_container" if other == 0 else "int8_container"] = dict(
        ms_per_pass=ms_alt, tops=ops1 / (ms_alt * 1e-3) / 1e12,
        per_layer={k: dict(quant_ms=float(np.median(d["q"])), gemm_ms=float(np.median(d["g"])),
                           quant_gbs=d["L"]["quant_bytes"] / (float(np.median(d["q"])) * 1e-3) / 1e9,
                           gemm_tops=d["L"]["ops_1limb"] / (float(np.median(d["g"])) * 1e-3) / 1e12) for k, d in per.items()},
        note="quantize bytes counted on this container's layout (4.5 B per element for two codes per byte)")
    del alt
    # --- INT3 activations (same kernels and containers; the quantizer range differs)
    ms_a3 = per_pass(lambda: run_step(hq, layers, status, a_bits=3))
    out["w4a3"] = dict(ms_per_pass=ms_a3, tops=ops1 / (ms_a3 * 1e-3) / 1e12)
    # --- the 3x3 convolution with one scale per pixel: per-tap drain of the accumulator
    Lc = [L for L in layers if L["kind"] == "conv"][0]
    c = CONV

    def conv_pp():
        hq.hq_qconv(Lc["x"], Lc["pw"], c["R"], c["S"], c["stride"], c["pad"], Lc["bias"], A_BITS, Lc["y"], Lc["ws"],
                    dev_status=status, stream=stream)

    def conv_static():
        hq.hq_qconv(Lc["x"], Lc["pw"], c["R"], c["S"], c["stride"], c["pad"], Lc["bias"], A_BITS, Lc["y"], Lc["ws"],
                    static_scale=Lc["static_scale"], dev_status=status, stream=stream)

    ms_pp, ms_st = per_pass(conv_pp), per_pass(conv_static)
    out["conv3x3_per_pixel_scales"] = dict(layer_ms=ms_pp, tops=Lc["ops_1limb"] / (ms_pp * 1e-3) / 1e12,
                                           static_scale_layer_ms=ms_st,
                                           note="3x3 conv of the step, batch 32, per-pixel INT4 scales: each tap rescaled by "
                                                "the scale of the pixel it read")
    # --- one-limb weights: the same GEMMs with PLAIN weights (codes already in the workspaces)
    plain = build_layers(torch, hq, device, seed=rank, cont=layers[0]["cont"], share=layers, weight_mode=hq.HQ_W_PLAIN)
    for Lp, L0 in zip(plain, layers):
        Lp["ws"] = L0["ws"]
    evs = []
    for _ in range(40):
        run_step_split(torch, hq, plain, status, evs, gemm_only=True)
    torch.cuda.synchronize()
    g = {}
    for L, a, b, c2 in evs[len(plain) * 10:]:
        g.setdefault(L["name"], []).append(b.elapsed_time(c2))
    out["one_limb_gemm_ms"] = {k: float(np.median(v)) for k, v in g.items()}
    del plain
    # --- the short-reduction products on pairs of SMs (tcgen05.mma.cta_group::2), GEMM only, codes already in the workspaces
    if layers[0]["cont"] == 1:
        def gemm_only_ms(sub):
            evs2 = []
            for _ in range(40):
                run_step_split(torch, hq, sub, status, evs2, gemm_only=True)
            torch.cuda.synchronize()
            acc = {}
            for L, a, b, c2 in evs2[len(sub) * 10:]:
                acc.setdefault(L["name"], []).append(b.elapsed_time(c2))
            return {k: float(np.median(v)) for k, v in acc.items()}
        lin = [L for L in layers if L["kind"] == "linear" and L["K"] <= 512]
        before = hq.hq_set_pair_gemm(0)
        try:
            one_cta = gemm_only_ms(lin)
            hq.hq_set_pair_gemm(1)
            paired = gemm_only_ms(lin)
        finally:
            hq.hq_set_pair_gemm(before)
        sms = torch.cuda.get_device_properties(device).multi_processor_count
        pr_ms = per_pass(lambda: hq.hq_mma_i8_probe_pair(sms // 2, 20000, dev_status=status, stream=stream))
        out["gemm_on_sm_pairs"] = dict(per_layer={k: dict(one_cta_ms=one_cta[k], pair_ms=paired[k]) for k in one_cta},
                                       paired_mma_probe_tops=(sms // 2) * 20000 * 2.0 * 256 * 256 * 32 / (pr_ms * 1e-3) / 1e12,
                                       note="hq_set_pair_gemm(1): 2-CTA clusters, each CTA half of the weight tile; GEMM launches only")
    # --- transform + quantization fused into the product kernel's operand tile (one kernel, no codes in memory)
    if layers[0]["cont"] == 1:
        fused = {}
        for L in layers:
            if L["kind"] != "linear" or L["K"] not in (128, 256, 512):
                continue
            one = per_pass(lambda: hq.hq_qlinear_fused(L["x"], L["pw"], L["bias"], A_BITS, L["y"], dev_status=status, stream=stream))
            two = per_pass(lambda: hq.hq_qlinear(L["x"], L["pw"], L["bias"], A_BITS, L["y"], L["ws"], dev_status=status, stream=stream))
            fused[L["name"]] = dict(one_kernel_ms=one, two_kernels_ms=two)
        out["fused_operand_load"] = dict(per_layer=fused,
                                         note="hq_qlinear_fused (activation tile stationary, transform by the epilogue warps) "
                                              "against hq_qlinear (two kernels, dependent launch), whole layer")
    # --- the same convolution with the width-axis transform (the paper's literal form; one weight limb)
    pw_w = hq.hq_weight_prepare(inputs.config_conv_small(seed=rank, batch=1)["w"], W_BITS, 1, hq.HQ_W_PLAIN,
                                hq.HQ_CODES_INT8).to_device(device)
    ws_w = torch.empty((hq.hq_workspace_size(Lc["rows"], Lc["cols"], hq.HQ_CODES_INT8),), dtype=torch.uint8, device=device)
    zbuf = torch.empty((Lc["rows"], Lc["cols"]), dtype=torch.int8, device=device)

    def width_layer():
        hq.hq_qconv_width(Lc["x"], pw_w, c["R"], c["S"], c["stride"], c["pad"], Lc["bias"], A_BITS, 16,
                          Lc["static_scale"], Lc["y"], ws_w, dev_status=status)

    def width_quant():
        hq.hq_hadamard_quant_width(Lc["x"], 16, A_BITS, Lc["static_scale"], zbuf.view(Lc["x"].shape))

    wl, wq = per_pass(width_layer), per_pass(width_quant)
    out["width_axis_conv"] = dict(layer_ms=wl, quant_ms=wq, tops=Lc["ops_1limb"] / (wl * 1e-3) / 1e12,
                                  quant_gbs=Lc["rows"] * Lc["cols"] * 5.0 / (wq * 1e-3) / 1e9,
                                  note="3x3 conv of the step with the transform along the width axis (16-point blocks), "
                                       "untransformed one-limb weights, int8 activations")
    hq.hq_check_status(status)
    return out


def oracle_sample_step(orc, sample_rows, seed):
    """One bounded sample of the step on the CPU oracle; returns (ops done, seconds)."""
    ops, t0 = 0.0, time.perf_counter()
    for name, K, N, hb in inputs.TRANSFORMER_LINEARS:
        cfg = inputs.config_transformer_linear(name, M=sample_rows, seed=seed)
        out = orc.qlinear(cfg["x"], cfg["w"], cfg["bias"], a_bits=A_BITS, w_bits=W_BITS, had_block=hb,
                          weight_mode="folded")
        ops += 2.0 * sample_rows * N * K
        del out
    c = CONV
    cfg = inputs.config_conv_small(seed=seed, batch=max(1, sample_rows // (c["H"] * c["W"])))
    nb = cfg["x"].shape[0]
    orc.qconv(cfg["x"], cfg["w"], cfg["bias"], a_bits=A_BITS, w_bits=W_BITS, had_block=c["had_block"], stride=1, pad=1,
              weight_mode="folded", static_scale=0.5)
    ops += 2.0 * nb * c["H"] * c["W"] * c["Cout"] * c["R"] * c["S"] * c["C"]
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
    """The quantized linears of the DiT-shaped workload, one after the other on one stream, bf16 activations, W4A4 with
    folded two-limb weights, per-row scales: 143 linears of a width-1152, depth-28 diffusion transformer (batch 32,
    256 tokens).  The attention core and the other glue between them are not part of this workload."""
    import torch
    from paper_2512_05746_b200 import binding as hq
    from paper_2512_05746_b200 import dit
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
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

    warmup = max(3, min(args.warmup, 5))
    for _ in range(warmup):
        forward()
    t_one = timed_region(torch, forward, 2, torch.cuda.current_stream()) / 2
    steps = max(args.steps, int(600.0 / max(t_one, 1e-3)) + 1)       # at least 0.6 s of forwards in the timed region
    sampler = ClockSampler(0)
    sampler.start()
    ms = timed_region(torch, forward, steps, torch.cuda.current_stream()) / steps
    clocks = sampler.stop()
    clocks["window"] = "the timed region"
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
                          with_layernorm_prologue=ln_extra)))


def main_unet(args):
    """One denoising step of the UNet-shaped network (batch 64, 64x64x3 latent, base 256, multipliers (1,2,3,4), two
    residual blocks per level, 8-head self-attention at 32/16/8, step + class embedding): every convolution but the first
    and last and every linear is a Hadamard-quantized W4A4 layer (3x3 convolutions with a calibrated static scale and
    GroupNorm + SiLU fused into their transform kernel), data flows from layer to layer, and the bf16 operations between
    them (attention core, additions, concatenation, up-sampling, embeddings, first / last convolution) run in the
    library's own kernels.  Reports the full forward, and the quantized layers and the glue timed on their own over the
    buffers of a complete forward."""
    import torch
    from paper_2512_05746_b200 import binding as hq
    from paper_2512_05746_b200.unet import UNet, quantized_layers
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    if args.pair_gemm:
        hq.hq_set_pair_gemm(1)
    batch = 64 if args.rows == 32768 else max(1, int(args.rows))          # --rows N: a reduced batch for profiler captures
    cfg = inputs.unet_config(batch=batch)
    t_setup = time.time()
    P = inputs.unet_params(cfg, seed=0)
    I = inputs.unet_inputs(cfg, seed=0)
    net = UNet(cfg, P, hq, dev, container=CODES[0], a_bits=A_BITS).build(batch)
    del P
    x, t, y = torch.from_numpy(I["x"]), torch.from_numpy(I["t"]), torch.from_numpy(I["y"])
    net.calibrate(x, t, y)
    t_setup = time.time() - t_setup
    stream = torch.cuda.current_stream()
    for _ in range(max(3, min(args.warmup, 5))):
        net.run()
    if args.profile_forward:
        torch.cuda.synchronize()
        torch.cuda.profiler.start()
        net.run()
        torch.cuda.synchronize()
        torch.cuda.profiler.stop()
        hq.hq_check_status(net.status)
        print(json.dumps(dict(workload="unet", batch=batch, profiled_forwards=1, library_calls=len(net.tape))))
        return
    t_one = timed_region(torch, net.run, 2, stream) / 2
    steps = max(args.steps, int(600.0 / max(t_one, 1e-3)) + 1)          # at least 0.6 s in the timed region
    sampler = ClockSampler(0)
    sampler.start()
    ms_full = timed_region(torch, net.run, steps, stream) / steps
    clocks = sampler.stop()
    clocks["window"] = "the timed region (full forwards)"
    reps = max(5, steps // 3)
    ms_q = timed_region(torch, lambda: net.run(tags=("q",)), reps, stream) / reps
    ms_g = timed_region(torch, lambda: net.run(tags=("g",)), reps, stream) / reps
    hq.hq_check_status(net.status)
    # one forward with an event after every call: time per kind of operation
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(len(net.tape) + 1)]
    evs[0].record(stream)
    for i, (_, _, call) in enumerate(net.tape):
        call()
        evs[i + 1].record(stream)
    torch.cuda.synchronize()
    by_kind = {}
    for i, (tag, name, _) in enumerate(net.tape):
        if tag == "q":
            kind = "quantized " + ("conv3x3" if (".conv" in name or "sample" in name) else "conv1x1" if name.endswith(".skip") else "linear")
        else:
            kind = ("attention core" if name.endswith(".core") else "residual / embedding add" if ("residual" in name or "emb_add" in name)
                    else "concat" if name.endswith(".concat") else "upsample" if name.endswith(".nearest")
                    else "first / last conv" if name in ("in_conv", "out_conv") else "final groupnorm" if name == "out_norm"
                    else "embedding path")
        d = by_kind.setdefault(kind, dict(calls=0, ms=0.0))
        d["calls"] += 1
        d["ms"] += evs[i].elapsed_time(evs[i + 1])
    layers = quantized_layers(batch=batch)
    macs = sum(L["macs"] for L in layers)
    nq = sum(1 for tag, _, _ in net.tape if tag == "q")
    attn_flops = net.attn_flops
    print(json.dumps(dict(metric="UNet forwards/s: one denoising step of the UNet-shaped network, batch 64 per forward",
                          value=1e3 / ms_full, unit="forwards/s", n_gpus=1, steps=steps, warmup=max(3, min(args.warmup, 5)),
                          ms_per_step=ms_full, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="int8",
                          data="synthetic",
                          config=dict(workload=f"configs[3] UNet forward: batch {batch}, 64x64x3 latent, base 256, mult (1,2,3,4), attention at "
                                               f"32/16/8 with 8 heads, 1000 classes; W4A{A_BITS}, folded weights, {codes_name()} codes, bf16 activations",
                                      quantized_layers=nq, library_calls=len(net.tape), samples_per_s=batch * 1e3 / ms_full,
                                      l2="activations of the large layers exceed L2", setup_s=t_setup),
                          full_forward_ms=ms_full, quantized_only_ms=ms_q, glue_ms=ms_g,
                          quantized_tops=2.0 * macs / (ms_q * 1e-3) / 1e12,
                          attention_tflops=attn_flops / (by_kind.get("attention core", dict(ms=1e30))["ms"] * 1e-3) / 1e12,
                          by_kind={k: dict(calls=v["calls"], ms=round(v["ms"], 4)) for k, v in sorted(by_kind.items())},
                          clocks=clocks, gpu_launches=len(net.tape) * steps)))


def main_sweep(args):
    """Shape sweep of transform+quantize followed by the integer GEMM: M x K x N grid, Hadamard block = K, for
    W4A4 with the folded two-limb weights, W4A4 with plain one-limb weights (codes in the container --codes selects) and
    W8A8 (plain weights).  W4A3 runs the same kernels as W4A4 (only the quantizer range differs).  Small shapes rotate
    through enough copies of their buffers that every launch's inputs and outputs come from and go to DRAM, not L2.
    One JSON line with one record per point: int TOPS of the GEMM (2*M*N*K), GB/s of the quantize stage, and the
    roofline fraction of the GEMM (slower of the tensor ceiling for its limb count and algorithmic bytes over the
    measured copy bandwidth)."""
    import torch
    from paper_2512_05746_b200 import binding as hq
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    pk = peaks()
    status = torch.zeros((1,), dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    probe = probe_int8_pipe(torch, hq, 0, status, stream, seconds=0.4)
    int8_peak = probe["tops"]                      # at the probe's own (power-capped) clock
    Ms, Ks, Ns = (4096, 16384, 65536), (256, 512, 1024, 2048, 4096), (512, 1280, 4096)
    if args.rows != M_TOKENS:
        Ms = (int(args.rows),)
    variants = (("W4A4 folded", 4, 4, hq.HQ_W_FOLDED, CODES[0]),
                ("W4A4 plain", 4, 4, hq.HQ_W_PLAIN, CODES[0]),
                ("W8A8 plain", 8, 8, hq.HQ_W_PLAIN, hq.HQ_CODES_INT8))
    gen = torch.Generator(device=dev)
    gen.manual_seed(0)
    reps = max(3, min(args.steps, 50))
    ROTATE_BYTES = 192e6                           # more than the 126 MB L2
    points = []

    def timed(fns):
        n = len(fns)
        for i in range(10):
            fns[i % n]()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(reps):
            fns[i % n]()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    for K in Ks:
        for N in Ns:
            w = inputs.weights((N, K), seed=K + N)
            pws = {v[0]: hq.hq_weight_prepare(w, v[2], K, v[3], v[4]).to_device(dev) for v in variants}
            b = torch.from_numpy(inputs.bias(N, seed=N)).to(dev)
            for M in Ms:
                set_bytes = M * K * 5.0 + M * N * 2.0
                nrot = int(min(16, max(1, -(-ROTATE_BYTES // set_bytes))))
                xs = []
                for _ in range(nrot):
                    x = torch.randn((M, K), generator=gen, device=dev, dtype=torch.float32)
                    x[:, torch.randperm(K, generator=gen, device=dev)[: max(1, round(0.01 * K))]] *= 20.0
                    xs.append(x)
                ys = [torch.empty((M, N), dtype=torch.bfloat16, device=dev) for _ in range(nrot)]
                for name, a_bits, w_bits, mode, cont in variants:
                    pw = pws[name]
                    pitch = K // 2 if cont == hq.HQ_CODES_NIBBLE else K
                    cds = [torch.empty((M, pitch), dtype=torch.uint8, device=dev) for _ in range(nrot)]
                    scs = [torch.empty((M,), dtype=torch.float32, device=dev) for _ in range(nrot)]
                    q_ms = timed([(lambda i=i: hq.hq_hadamard_quant(xs[i], K, a_bits, cds[i], cont, scales=scs[i]))
                                  for i in range(nrot)])
                    g_ms = timed([(lambda i=i: hq.hq_qgemm(cds[i], cont, a_bits, K, pw, scale_a=scs[i], bias=b, alpha=pw.alpha,
                                                           y=ys[i], dev_status=status)) for i in range(nrot)])
                    limbs = pw.desc.limbs
                    ops = 2.0 * M * N * K
                    gbytes = M * pitch + N * K * limbs + M * N * 2.0 + 4.0 * M + 8.0 * N
                    t_tensor, t_hbm = ops * limbs / (int8_peak * 1e12), gbytes / (pk["hbm_gbs"] * 1e9)
                    qbytes = M * K * 4.0 + M * pitch + 4.0 * M
                    points.append(dict(M=M, K=K, N=N, variant=name, limbs=limbs, rotated_sets=nrot, quant_us=q_ms * 1e3,
                                       gemm_us=g_ms * 1e3, gemm_tops=ops / g_ms / 1e9, gemm_tops_limbs=ops * limbs / g_ms / 1e9,
                                       quant_gbs=qbytes / q_ms / 1e6,
                                       bound="tensor" if t_tensor >= t_hbm else "hbm",
                                       roofline_frac=max(t_tensor, t_hbm) / (g_ms * 1e-3),
                                       quant_frac=qbytes / q_ms / 1e6 / pk["hbm_gbs"]))
                    del cds, scs
                del xs, ys
    hq.hq_check_status(status)
    best = max(points, key=lambda d: d["gemm_tops_limbs"])
    print(json.dumps(dict(metric="shape sweep: int TOPS of the GEMM and GB/s of transform+quantize per point", value=best["gemm_tops_limbs"],
                          unit="TOPS issued (best point)", n_gpus=1, steps=reps, warmup=10, higher_is_better=True, dtype="int8",
                          data="synthetic", vs_baseline=None,
                          config=dict(workload="configs[4] shape sweep, " + codes_name() + " codes for W4A4",
                                      int8_peak_tops=int8_peak, int8_peak_source="kind::i8 issue-rate probe of this run",
                                      probe_sm_mhz=probe["sm_mhz"], hbm_gbs=pk["hbm_gbs"], peak_source=pk["source"],
                                      l2=f"buffers of a point rotate through at least {ROTATE_BYTES / 1e6:.0f} MB"),
                          points=points)))


def main_attn(args):
    """The self-attention core of the UNet's 32x32 level (1024 tokens, 8 heads of 64) on its own: TFLOP/s of hq_attention.
    --rows sets the batch (default 64; smaller for profiler captures)."""
    import torch
    from paper_2512_05746_b200 import binding as hq
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    Nb = 64 if args.rows == 32768 else max(1, int(args.rows))
    L, Cc, heads = 1024, 512, 8
    gen = torch.Generator(device=dev)
    gen.manual_seed(0)
    status = torch.zeros((1,), dtype=torch.int32, device=dev)
    sets = [(torch.randn((Nb * L, 3 * Cc), generator=gen, device=dev).to(torch.bfloat16),
             torch.empty((Nb * L, Cc), dtype=torch.bfloat16, device=dev)) for _ in range(2)]
    i = [0]

    def call():
        i[0] ^= 1
        hq.hq_attention(sets[i[0]][0], Nb, heads, sets[i[0]][1], dev_status=status)

    steps, warmup = max(1, min(args.steps, 50)), max(3, min(args.warmup, 5))
    for _ in range(warmup):
        call()
    ms = timed_region(torch, call, steps, torch.cuda.current_stream()) / steps
    hq.hq_check_status(status)
    flops = 4.0 * Nb * L * L * Cc
    print(json.dumps(dict(metric="TFLOP/s of the self-attention core (bf16 tensor cores, 4 L^2 C per sample)",
                          value=flops / (ms * 1e-3) / 1e12, unit="TFLOP/s", n_gpus=1, steps=steps, warmup=warmup, ms_per_step=ms,
                          higher_is_better=True, dtype="bf16", data="synthetic", vs_baseline=None,
                          config=dict(workload=f"attention core: batch {Nb}, 1024 tokens, 8 heads x 64"), gpu_launches=steps)))


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
                          gpu_launches=2 * steps)))


def launch_command(n_gpus, argv, port=None):
    """The command that starts one rank per GPU for `bench.py --gpus N` when it was not started by a launcher."""
    import socket
    if port is None:
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={int(n_gpus)}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def timed_region(torch, fn, reps, stream):
    """Device time (ms) of `reps` calls of fn, events on `stream`, synchronised on both sides."""
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(reps):
        fn()
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1)


def probe_int8_pipe(torch, hq, local, status, stream, seconds=0.5):
    """Issue-rate ceiling of the int8 tensor pipe for the kernel's MMA shape (128x256x32 from shared memory, no global
    traffic), measured in this process: back-to-back probe launches for about `seconds`, with the SM clock sampled
    meanwhile.  Returns TOPS and the clock they were reached at."""
    sms = torch.cuda.get_device_properties(local).multi_processor_count
    iters = 20000
    for _ in range(3):
        hq.hq_mma_i8_probe(sms, iters, dev_status=status, stream=stream)
    ms1 = timed_region(torch, lambda: hq.hq_mma_i8_probe(sms, iters, dev_status=status, stream=stream), 3, stream) / 3
    reps = max(3, int(seconds * 1e3 / max(ms1, 1e-3)))
    sampler = ClockSampler(local)
    sampler.start()
    ms = timed_region(torch, lambda: hq.hq_mma_i8_probe(sms, iters, dev_status=status, stream=stream), reps, stream)
    clk = sampler.stop()
    ops = float(reps) * sms * iters * 2.0 * 128 * 256 * 32
    return dict(tops=ops / (ms * 1e-3) / 1e12, sm_mhz=clk.get("sm_mhz"), reasons=clk.get("reasons"), ctas=sms,
                seconds=ms * 1e-3)


def main():
    global M_TOKENS, WORKLOAD, A_BITS, METRIC
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the variant measurements (nibble container, INT3, per-pixel conv, one-limb weights, probe)")
    ap.add_argument("--passes-per-step", type=int, default=PASSES_PER_STEP,
                    help="passes over the batch that make up one step (profiler captures use 1)")
    ap.add_argument("--workload", default="step", choices=["step", "unet", "dit", "sweep", "gn", "attn"],
                    help="step: the benchmark step (default); unet: one denoising step of the UNet-shaped network; dit: the "
                         "quantized linears of the DiT-shaped workload; sweep: the M x K x N shape sweep; gn: the "
                         "GroupNorm+SiLU prologue on one tensor")
    ap.add_argument("--a-bits", type=int, default=4, choices=[3, 4],
                    help="activation bits of the step / unet / dit workloads (INT3 codes travel in the same containers)")
    ap.add_argument("--codes", default="int8", choices=["nibble", "int8"],
                    help="container of the 4-bit activation codes between the transform and the GEMM kernel: one per "
                         "byte (default, the faster one) or two per byte (half the workspace)")
    ap.add_argument("--rows", type=int, default=M_TOKENS,
                    help="rows per layer (default: the full 32768; smaller values are for profiler captures only)")
    ap.add_argument("--pair-gemm", action="store_true",
                    help="run every covered product on pairs of SMs (hq_set_pair_gemm(1)); the default mode 2 takes pairs where they "
                         "measured faster")
    ap.add_argument("--print-csrc-digest", action="store_true", help="print the digest profiles/dram_traffic.json records")
    ap.add_argument("--profile-forward", action="store_true",
                    help="--workload unet: run one forward between cudaProfilerStart / Stop and exit (for a profiler's "
                         "launch list with --profile-from-start off)")
    args = ap.parse_args()
    if args.print_csrc_digest:
        print(csrc_digest())
        return
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
    # `--gpus N` started by hand: start one rank per GPU (a launcher that already did sets WORLD_SIZE)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.workload == "step":
        import torch
        have = torch.cuda.device_count()
        if have < args.gpus:
            raise SystemExit(f"bench.py --gpus {args.gpus}: only {have} CUDA device(s) visible")
        env = dict(os.environ)
        env.setdefault("NCCL_DEBUG", "INFO")
        raise SystemExit(subprocess.call(launch_command(args.gpus, sys.argv[1:]), env=env))
    if args.workload == "unet":
        return main_unet(args)
    if args.workload == "dit":
        return main_layer_list(args, "dit")
    if args.workload == "sweep":
        return main_sweep(args)
    if args.workload == "gn":
        return main_gn(args)
    if args.workload == "attn":
        return main_attn(args)

    import torch
    import torch.distributed as dist
    from paper_2512_05746_b200 import binding as hq

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (the CUDA path has no CPU fallback)")
    if world != args.gpus:
        raise SystemExit(f"bench.py --gpus {args.gpus} was started with WORLD_SIZE={world}")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
        world = dist.get_world_size()

    warmup = max(args.warmup, 3)
    R = max(1, args.passes_per_step)
    if args.pair_gemm:
        hq.hq_set_pair_gemm(1)
        WORKLOAD = WORKLOAD + ", every covered product on SM pairs"
    layers = build_layers(torch, hq, device, seed=rank)
    status = torch.zeros((1,), dtype=torch.int32, device=device)
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def one_step():
        for _ in range(R):
            run_step(hq, layers, status)

    # ---- device-resident throughput: K steps of R passes each, clocks sampled over the timed region --------------
    for _ in range(warmup):
        one_step()
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for _ in range(args.steps):
        one_step()
    e1.record(stream)
    barrier()
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop()
    clocks["window"] = "the timed region"
    hq.hq_check_status(status)

    # ---- per-kernel attribution (same kernels, events between the two launches of each layer) -----------
    attr_reps = max(20, min(200, args.steps * R // 10))
    for _ in range(10):
        run_step(hq, layers, status)
    evs = []
    for _ in range(attr_reps):
        run_step_split(torch, hq, layers, status, evs)
    torch.cuda.synchronize()
    per = {}
    for L, a, b, c in evs:
        d = per.setdefault(L["name"], dict(quant=[], gemm=[], L=L))
        d["quant"].append(a.elapsed_time(b))
        d["gemm"].append(b.elapsed_time(c))
    for d in per.values():
        d["quant_ms"], d["gemm_ms"] = float(np.median(d["quant"])), float(np.median(d["gemm"]))
        d["quant_best"], d["gemm_best"] = float(np.min(d["quant"])), float(np.min(d["gemm"]))

    extras = {}
    probe = None
    width = None
    if rank == 0 and not args.no_extras:
        probe = probe_int8_pipe(torch, hq, local, status, stream)
        extras = measure_variants(torch, hq, device, layers, status, stream, rank)
        width = extras.pop("width_axis_conv", None)

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

    passes = args.steps * R
    ops_pass_limbs = sum(L["ops"] for L in layers)
    ops_pass = sum(L["ops_1limb"] for L in layers)
    value = ops_pass * passes * world / (ms * 1e-3) / 1e12
    e2e_value = ops_pass * e2e_steps * world / (e2e_ms * 1e-3) / 1e12

    if rank == 0:
        pk = peaks()
        traffic = measured_traffic()
        f_step = clocks.get("sm_mhz")
        # int8 tensor ceiling: the issue-rate probe measured in this run, scaled from the clock it ran at to the clock of
        # the timed region (both power-capped); cross-checks: 2 x the measured bf16 figures (nominal dense ratio 4.5 : 2.25)
        # and the nominal 4.5 POPS
        if probe is not None and probe.get("sm_mhz") and f_step:
            int8_peak = probe["tops"] * f_step / probe["sm_mhz"]
            peak_source = (f"kind::i8 issue-rate probe of this run ({probe['tops']:.0f} TOPS at {probe['sm_mhz']:.0f} MHz) "
                           f"scaled to the timed region's {f_step:.0f} MHz")
        elif probe is not None:
            int8_peak, peak_source = probe["tops"], "kind::i8 issue-rate probe of this run (no clock samples)"
        else:
            int8_peak, peak_source = 2.0 * pk["bf16_sustained"], f"2 x bf16 sustained ({pk['source']}); probe skipped"
        dom = max(per.values(), key=lambda d: d["gemm_ms"])      # dominant kernel: the longest GEMM launch
        L = dom["L"]
        gemm_ms = dom["gemm_ms"]
        ach = L["ops"] / (gemm_ms * 1e-3) / 1e12
        roofline = dict(bound="tensor", kernel=f"{gemm_kernel_name(L)} ({L['name']}: M={L['M']} K={L['K']} N={L['N']} "
                                                f"limbs={L['limbs']})",
                        achieved=ach, peak=int8_peak, unit="TOPS", frac=ach / int8_peak,
                        achieved_counts="2*M*N*K*limbs (the tensor work issued; the layer's own 2*M*N*K is achieved/limbs)",
                        traffic=(traffic.get("gemm") or {}).get(L["name"]),
                        algorithmic_bytes=L["gemm_bytes"], peak_source=peak_source,
                        peak_probe_tops=None if probe is None else probe["tops"],
                        peak_probe_mhz=None if probe is None else probe["sm_mhz"],
                        frac_vs_2x_bf16_sustained=ach / (2.0 * pk["bf16_sustained"]),
                        frac_vs_2x_bf16_burst=ach / (2.0 * pk["bf16_burst"]),
                        frac_vs_nominal_4500=ach / 4500.0,
                        launch_ms=gemm_ms, launch_ms_best=dom["gemm_best"])
        qd = max(per.values(), key=lambda d: d["quant_ms"])
        q_ms = qd["quant_ms"]
        q_gbs = qd["L"]["quant_bytes"] / (q_ms * 1e-3) / 1e9
        roofline_quant = dict(bound="hbm", kernel=f"fwht_quant_fast ({qd['L']['name']}: {qd['L']['rows']}x{qd['L']['cols']})",
                              achieved=q_gbs, peak=pk["hbm_gbs"], unit="GB/s", frac=q_gbs / pk["hbm_gbs"],
                              frac_vs_nominal_8000=q_gbs / 8000.0,
                              traffic=(traffic.get("quant") or {}).get(qd["L"]["name"]),
                              algorithmic_bytes=qd["L"]["quant_bytes"],
                              peak_source=f"copy bandwidth ({pk['source']})", launch_ms=q_ms, launch_ms_best=qd["quant_best"])
        per_layer = {}
        for k, d in per.items():
            Lk = d["L"]
            t_tensor = Lk["ops"] / (int8_peak * 1e12)
            t_hbm = Lk["gemm_bytes"] / (pk["hbm_gbs"] * 1e9)
            per_layer[k] = dict(quant_ms=d["quant_ms"], gemm_ms=d["gemm_ms"], limbs=Lk["limbs"],
                                gemm_tops_limbs=Lk["ops"] / (d["gemm_ms"] * 1e-3) / 1e12,
                                gemm_tops=Lk["ops_1limb"] / (d["gemm_ms"] * 1e-3) / 1e12,
                                quant_gbs=Lk["quant_bytes"] / (d["quant_ms"] * 1e-3) / 1e9,
                                quant_frac=Lk["quant_bytes"] / (d["quant_ms"] * 1e-3) / 1e9 / pk["hbm_gbs"],
                                gemm_bound="tensor" if t_tensor >= t_hbm else "hbm",
                                gemm_roofline_frac=max(t_tensor, t_hbm) / (d["gemm_ms"] * 1e-3))
            if k in (extras.get("one_limb_gemm_ms") or {}):
                per_layer[k]["gemm_ms_one_limb_weights"] = extras["one_limb_gemm_ms"][k]
        extras.pop("one_limb_gemm_ms", None)
        ms_step = ms / args.steps
        line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=warmup,
                    ms_per_step=ms_step, higher_is_better=True, scaling="weak", vs_baseline=None,
                    dtype="int8", data="synthetic",
                    config=dict(workload=WORKLOAD, passes_per_step=R, ms_per_pass=ms_step / R,
                                l2="inputs larger than L2 (0.5 GB read per pass)",
                                tensor_tops_limbs=ops_pass_limbs * passes * world / (ms * 1e-3) / 1e12,
                                layers_per_s=len(layers) * passes * world / (ms * 1e-3),
                                ms_per_pass_x_sm_mhz=None if not f_step else ms_step / R * f_step,
                                timed_region_s=ms * 1e-3),
                    clocks=clocks, gpu_launches=2 * len(layers) * passes,
                    e2e=dict(value=e2e_value, unit=UNIT, h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h,
                             steps=e2e_steps, ms_per_step=e2e_ms / e2e_steps,
                             note="one pass per end-to-end step: every pass uploads its inputs and downloads its outputs"),
                    roofline=roofline, roofline_fwht_quant=roofline_quant, per_layer=per_layer,
                    variants=extras, width_axis_conv=width)
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline()
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
