"""Weight-side error of the Single and the Double Hadamard scheme on synthetic weights -- TEST INFRASTRUCTURE.

The "Single Hadamard Transformation" paragraph argues that quantizing H^T W instead of W adds outliers when W has
few of them (a flat vector becomes a spike, Eq. 16), and Table 6 compares the two schemes.  The trained weights are
not available, so this script measures the direction of that claim on four synthetic weight families with the CPU
oracle only (nothing here touches the CUDA library):

  gaussian   iid N(0, 0.02)                         -- invariant in distribution under an orthonormal transform
  uniform    iid U(-0.035, 0.035)                   -- bounded, kurtosis 1.8: "low-outlier"
  offset     N(0, 0.02) + one mean per out-channel  -- the flat component of Eq. 16 (c * 1 -> c * 2^(k/2) e_1)
  outlier-in N(0, 0.02), 3 input channels x 20      -- weights that DO have outliers along the transformed axis

For every family: statistics of W and of H^T W along the input-channel axis (max|.|/sigma, kurtosis, share beyond
3 sigma: the three quantities of the paper's weight-outlier figure), the relative 4-bit quantization error of Q(W)
and of Q(H^T W) (measured in the same space: H is orthonormal), and the relative error of the W4A4 layer output
against the float product X W on outlier activations for the Single (folded) and the Double scheme, which share the
activation codes and differ in the weights only.

Run `python -m oracle.weight_error_study` to print the table that the design notes quote.
"""
from __future__ import annotations

import numpy as np

import oracle
from paper_2512_05746_b200 import inputs

FAMILIES = ("gaussian", "uniform", "offset", "outlier-in")


def make_weights(family: str, N: int = 256, K: int = 256, seed: int = 0) -> np.ndarray:
    """fp32 [N][K] (output channel, input channel)."""
    rng = np.random.default_rng(1000 + seed)
    if family == "gaussian":
        w = rng.normal(0.0, 0.02, size=(N, K))
    elif family == "uniform":
        w = rng.uniform(-0.035, 0.035, size=(N, K))
    elif family == "offset":
        w = rng.normal(0.0, 0.02, size=(N, K)) + rng.normal(0.0, 0.01, size=(N, 1))
    elif family == "outlier-in":
        w = rng.normal(0.0, 0.02, size=(N, K))
        w[:, rng.choice(K, size=3, replace=False)] *= 20.0
    else:
        raise ValueError(family)
    return w.astype(np.float32)


def axis_stats(a: np.ndarray) -> dict:
    """Mean over output channels of max|a|/sigma, kurtosis and the share of entries beyond 3 sigma (per channel)."""
    a = a.astype(np.float64)
    mu = a.mean(axis=1, keepdims=True)
    sd = a.std(axis=1, keepdims=True)
    z = (a - mu) / sd
    return dict(max_over_sigma=float((np.abs(a).max(axis=1) / sd[:, 0]).mean()),
                kurtosis=float((z ** 4).mean(axis=1).mean()),
                beyond_3sigma=float((np.abs(z) > 3.0).mean()))


def weight_errors(w: np.ndarray, w_bits: int, had_block: int) -> dict:
    """Relative squared error of Q(W) against W and of Q(H^T W) against H^T W, summed over the matrix."""
    w64 = w.astype(np.float64)
    w_int, s_w = oracle.weight_quantize(w, w_bits)
    e_single = float(((w64 - s_w.astype(np.float64)[:, None] * w_int) ** 2).sum() / (w64 ** 2).sum())
    hw = oracle.transform(w64, had_block)                    # rows are output channels: this is (H^T W)^T
    B, s_d = oracle.weight_double(w, w_bits, had_block)
    e_double = float(((hw - s_d.astype(np.float64)[:, None] * B) ** 2).sum() / (hw ** 2).sum())
    return dict(single=e_single, double=e_double, hw=hw)


def layer_errors(w: np.ndarray, a_bits: int, w_bits: int, had_block: int, rows: int = 128) -> dict:
    """Relative error of the quantized layer against the float product on outlier activations (config-1 inputs)."""
    x = inputs.config_linear_small(0)["x"][:rows].astype(np.float64)
    ref = x @ w.astype(np.float64).T
    out = {}
    for mode in ("folded", "double"):
        y = oracle.qlinear(x, w, None, a_bits=a_bits, w_bits=w_bits, had_block=had_block, weight_mode=mode)["y"]
        out[mode] = float(np.linalg.norm(y - ref) / np.linalg.norm(ref))
    return out


def study(w_bits: int = 4, a_bits: int = 4, had_block: int = 256) -> list[dict]:
    rows = []
    for fam in FAMILIES:
        w = make_weights(fam)
        we = weight_errors(w, w_bits, had_block)
        le = layer_errors(w, a_bits, w_bits, had_block)
        rows.append(dict(family=fam, before=axis_stats(w), after=axis_stats(we["hw"]), werr_single=we["single"],
                         werr_double=we["double"], layer_single=le["folded"], layer_double=le["double"]))
    return rows


def markdown(rows: list[dict]) -> str:
    out = ["| weights | max/sigma W -> H^T W | kurtosis | beyond 3 sigma | rel. err Q(W) | rel. err Q(H^T W) | ratio | "
           "layer err Single | layer err Double |", "|---|---|---|---|---|---|---|---|---|"]
    for r in rows:
        b, a = r["before"], r["after"]
        out.append(f"| {r['family']} | {b['max_over_sigma']:.2f} -> {a['max_over_sigma']:.2f} | "
                   f"{b['kurtosis']:.2f} -> {a['kurtosis']:.2f} | {100 * b['beyond_3sigma']:.2f} % -> "
                   f"{100 * a['beyond_3sigma']:.2f} % | {r['werr_single']:.4f} | {r['werr_double']:.4f} | "
                   f"{r['werr_double'] / r['werr_single']:.2f} | {r['layer_single']:.4f} | {r['layer_double']:.4f} |")
    return "\n".join(out)


if __name__ == "__main__":
    print(markdown(study()))
