"""Helpers shared by the GPU parity tests: acceptance rules written out once."""
import numpy as np

# Codes must equal the oracle's, except where the oracle's pre-rounding value v = u/S lies within
# CODE_TIE_REL * (full scale of the row) of a rounding boundary (a half-integer); there +-1 is allowed,
# for at most CODE_MISMATCH_FRAC of all codes.  The full scale of a row is max|v| (= qmax in dynamic mode),
# which is what the fp32 rounding error of the transform is proportional to.
CODE_TIE_REL = 1e-6
CODE_MISMATCH_FRAC = 1e-4
SCALE_RTOL = 1e-6
Y_BF16_RTOL = 1e-2      # final bf16 outputs: max relative error
Y_F32_RTOL = 1e-4       # fp32 epilogue path


def unpack_nibbles_np(b: np.ndarray) -> np.ndarray:
    """uint8 [..., n/2] -> int8 [..., n]; element 2j in the low nibble (test-side reimplementation)."""
    lo = (b & 0xF).astype(np.int16)
    hi = (b >> 4).astype(np.int16)
    lo = np.where(lo >= 8, lo - 16, lo)
    hi = np.where(hi >= 8, hi - 16, hi)
    out = np.empty(b.shape[:-1] + (b.shape[-1] * 2,), np.int8)
    out[..., 0::2] = lo
    out[..., 1::2] = hi
    return out


def pack_nibbles_np(q: np.ndarray) -> np.ndarray:
    u = q.astype(np.uint8) & 0xF
    return (u[..., 0::2] | (u[..., 1::2] << 4)).astype(np.uint8)


def check_codes(q_gpu: np.ndarray, q_ref: np.ndarray, v_ref: np.ndarray, what: str = ""):
    """Apply the code acceptance rule; returns the mismatch fraction."""
    assert q_gpu.shape == q_ref.shape, (q_gpu.shape, q_ref.shape)
    bad = q_gpu != q_ref
    nbad = int(bad.sum())
    if nbad == 0:
        return 0.0
    frac = nbad / q_ref.size
    d = np.abs(q_gpu.astype(np.int32) - q_ref.astype(np.int32))[bad]
    assert d.max() == 1, f"{what}: code differs by {d.max()}"
    full = np.maximum(np.abs(v_ref).reshape(-1, v_ref.shape[-1]).max(axis=1), 1.0)
    full = np.broadcast_to(full.reshape(v_ref.shape[:-1] + (1,)), v_ref.shape)
    dist = np.abs(v_ref - (np.floor(v_ref) + 0.5))[bad]
    lim = CODE_TIE_REL * full[bad]
    assert np.all(dist <= lim), f"{what}: mismatch {dist.max():.3e} away from a boundary (limit {lim.max():.3e})"
    assert frac <= CODE_MISMATCH_FRAC, f"{what}: {frac:.2e} of codes differ"
    return frac


def rel_err(y: np.ndarray, y_ref: np.ndarray) -> float:
    """max |y - y_ref| / max(|y_ref|, 2^-6 * rms(y_ref))."""
    y = y.astype(np.float64)
    rms = float(np.sqrt(np.mean(y_ref ** 2))) if y_ref.size else 0.0
    den = np.maximum(np.abs(y_ref), 2.0 ** -6 * rms + 1e-300)
    return float((np.abs(y - y_ref) / den).max()) if y.size else 0.0
