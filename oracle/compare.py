"""Comparison metrics between a candidate implementation and the oracle (test infrastructure).

Nothing here knows about CUDA: candidates arrive as NumPy arrays.
"""
import numpy as np


def _signed_index(codes, mag_bits):
    codes = np.asarray(codes).astype(np.int64)
    mag = codes & ((1 << mag_bits) - 1)
    sign = (codes >> mag_bits) & 1
    return np.where(sign == 1, -mag, mag)        # +0 and -0 coincide


def code_mismatch(cand, ref, mag_bits=7):
    """(fraction of elements whose code differs, largest distance in code steps).

    mag_bits = 7 for E4M3 bytes, 3 for E2M1 nibbles.  Sign-magnitude codes are ordered
    like the values they encode, so a rounding tie shows up as a distance of one step.
    """
    a, b = _signed_index(cand, mag_bits), _signed_index(ref, mag_bits)
    diff = np.abs(a - b)
    return float(np.mean(diff != 0)), int(diff.max(initial=0))


def assert_codes_close(cand, ref, mag_bits=7, max_frac=1e-3, what="codes"):
    """Identical except for at most 0.1% of elements, and those one code step apart."""
    frac, dist = code_mismatch(cand, ref, mag_bits)
    assert dist <= 1, f"{what}: a code differs by {dist} steps"
    assert frac <= max_frac, f"{what}: {frac:.2e} of the codes differ (limit {max_frac:.0e})"
    return frac


def output_metrics(cand, ref, v_absmax):
    """max |delta| / max|V|, cosine similarity, PSNR (peak = max |ref|) of an output block."""
    c = np.asarray(cand, dtype=np.float64)
    r = np.asarray(ref, dtype=np.float64)
    err = np.abs(c - r)
    cos = float((c * r).sum() / (np.linalg.norm(c) * np.linalg.norm(r) + 1e-300))
    mse = float((err ** 2).mean())
    peak = float(np.abs(r).max())
    psnr = float("inf") if mse == 0 else 10.0 * np.log10(peak * peak / mse)
    return {"max_err_over_vmax": float(err.max() / v_absmax), "cos": cos, "psnr_db": psnr,
            "frac_over_tol": float(np.mean(err > 2e-2 * v_absmax))}


def unpack_nibbles(packed):
    """uint8 [.., n/2] -> uint8 [.., n] with the even index in the low nibble."""
    p = np.asarray(packed, dtype=np.uint8)
    out = np.empty(p.shape[:-1] + (p.shape[-1] * 2,), dtype=np.uint8)
    out[..., 0::2] = p & 0xF
    out[..., 1::2] = p >> 4
    return out


def pack_nibbles(codes):
    c = np.asarray(codes, dtype=np.uint8)
    return (c[..., 0::2] | (c[..., 1::2] << 4)).astype(np.uint8)
