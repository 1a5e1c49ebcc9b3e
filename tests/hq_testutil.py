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


# (test name, mismatch fraction, largest distance of a mismatching code from a rounding boundary relative to the row's full
# scale) of every code comparison of the session; written to the file named by $HQ_PARITY_STATS when the session ends.
PARITY_STATS = []


def check_codes(q_gpu: np.ndarray, q_ref: np.ndarray, v_ref: np.ndarray, what: str = "", tie_rel: float = CODE_TIE_REL,
                mismatch_frac: float = CODE_MISMATCH_FRAC):
    """Apply the code acceptance rule; returns the mismatch fraction."""
    assert q_gpu.shape == q_ref.shape, (q_gpu.shape, q_ref.shape)
    bad = q_gpu != q_ref
    nbad = int(bad.sum())
    if nbad == 0:
        PARITY_STATS.append(dict(what=what, codes=int(q_ref.size), mismatch_frac=0.0, max_tie_rel=0.0))
        return 0.0
    frac = nbad / q_ref.size
    d = np.abs(q_gpu.astype(np.int32) - q_ref.astype(np.int32))[bad]
    full = np.maximum(np.abs(v_ref).reshape(-1, v_ref.shape[-1]).max(axis=1), 1.0)
    full = np.broadcast_to(full.reshape(v_ref.shape[:-1] + (1,)), v_ref.shape)
    dist = np.abs(v_ref - (np.floor(v_ref) + 0.5))[bad]
    PARITY_STATS.append(dict(what=what, codes=int(q_ref.size), mismatch_frac=frac,
                             max_tie_rel=float((dist / full[bad]).max()), max_code_diff=int(d.max())))
    assert d.max() == 1, f"{what}: code differs by {d.max()}"
    lim = tie_rel * full[bad]
    assert np.all(dist <= lim), f"{what}: mismatch {dist.max():.3e} away from a boundary (limit {lim.max():.3e})"
    assert frac <= mismatch_frac, f"{what}: {frac:.2e} of codes differ"
    return frac


def rel_err(y: np.ndarray, y_ref: np.ndarray) -> float:
    """max |y - y_ref| / max(|y_ref|, 2^-6 * rms(y_ref))."""
    y = y.astype(np.float64)
    rms = float(np.sqrt(np.mean(y_ref ** 2))) if y_ref.size else 0.0
    den = np.maximum(np.abs(y_ref), 2.0 ** -6 * rms + 1e-300)
    return float((np.abs(y - y_ref) / den).max()) if y.size else 0.0


def workspace_views(workspace, rows: int, cols: int, container: int):
    """The codes [rows, pitch] (uint8) and scales [rows] (fp32) a fused layer call left in its workspace: the layout
    hq_workspace_size documents (codes at offset 0 with a 16-byte row pitch, scales at the next multiple of 256)."""
    import torch
    row_bytes = cols // 2 if container == 0 else cols
    pitch = (row_bytes + 15) // 16 * 16
    off = (rows * pitch + 255) // 256 * 256
    codes = workspace[: rows * pitch].view(rows, pitch)
    scales = workspace[off: off + rows * 4].view(torch.float32)
    return codes, scales


def decode_blob(pw) -> np.ndarray:
    """Test-side inverse of the prepared-weight blob layout: the weight integers B as int32 [N, RS, C] (byte shuffling
    and 256*hi + lo only).  The host tests compare it with the oracle's weight integers."""
    d = pw.desc
    Kp = d.RS * d.C_pad
    rows = pw.blob[: d.N_pad * d.limbs * Kp].reshape(-1, Kp).astype(np.int32)
    o = np.arange(d.N)
    if d.limbs == 1:
        full = rows[o]
    else:
        hi = rows[(o // 128) * 256 + (o % 128)]
        lo = rows[(o // 128) * 256 + 128 + (o % 128)]
        full = 256 * hi + lo
    full = full.reshape(d.N, d.RS, d.C_pad)[:, :, : d.C]
    if d.container == 0:                       # nibble container: channels of every 8 stored as 0,2,4,6,1,3,5,7
        c = np.arange(d.C)
        r = c & 7
        slot = np.where(r & 1, 4 + (r >> 1), r >> 1)
        full = full[:, :, (c & ~7) + slot]
    return np.ascontiguousarray(full)


def weight_integers(oracle, pw, w, w_bits: int, had_block: int, mode: str) -> np.ndarray:
    """The weight integers B [N, RS*C] a GPU product is checked against.  PLAIN and FOLDED: the oracle's own integers
    (exact arithmetic), which the prepared blob must reproduce.  DOUBLE: Q(H^T W) rounds floating-point values, and
    the library's butterfly sums differ from the oracle's dense sums in the last bit, so exact ties may round the
    other way: there the blob's integers are taken, after checking that they differ from the oracle's by at most one
    in at most 1e-4 of the entries."""
    B_blob = decode_blob(pw).reshape(pw.desc.N, -1)
    B_orc = oracle.prepare_weights(w, w_bits, had_block, mode)[0].reshape(pw.desc.N, -1)
    if mode != "double":
        assert np.array_equal(B_blob, B_orc), "prepared weight integers differ from the oracle's"
        return B_orc
    diff = B_blob != B_orc
    assert diff.mean() <= 1e-4 and (not diff.any() or np.abs(B_blob - B_orc)[diff].max() == 1)
    return B_blob


def attention_bound(oracle, qr, Nb, L, C, heads, want):
    """Element-wise error bound of the attention core from its arithmetic.  A bf16 rounding moves a value by at most
    2^-8 of itself (8 significant bits).  The softmax weights p_j are rounded to bf16 before they multiply the values,
    so an output sum_j p_j v_j / sum_j p_j may move by up to 2^-8 * sum_j p_j |v_j| through the numerator and by 2^-8 of
    itself through the denominator; the result is rounded to bf16 once more (2^-8 of itself); the fp32 accumulation
    and the approximate exp2 are far below that.  sum_j p_j |v_j| is the oracle's own attention applied to |v|."""
    qa = qr.reshape(Nb, L, 3 * C).copy()
    qa[:, :, 2 * C:] = np.abs(qa[:, :, 2 * C:])
    A = oracle.attention(qa, heads).reshape(Nb * L, C)
    return 2.0 ** -8 * A + 2.0 ** -7 * np.abs(want) + 1e-6 * A
