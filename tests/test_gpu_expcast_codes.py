"""The ExpCast-FP8 code (Eq. 7) as the attention kernels' softmax stage forms it, taken out of the
kernel through the library's test hook and compared byte for byte.

Two references.  (1) The oracle's Eq. 7 (oracle/codecs.py): z = s * cs and u = z - m are rounded
to fp32 one after the other there, while the kernel folds both into one fused multiply-add, so a
code may differ by one step where 8 u + 120 + beta lies within an fp32 rounding of a half: at most
one step, and only where the exact value is a tie to within 1e-4.  (2) The kernel's own arithmetic written out exactly (rational
numbers, one rounding to fp32 where the kernel has one): every byte must agree, whatever route the
kernel takes to the integer (here: a product that is subnormal and a saturating pack)."""
from fractions import Fraction

import numpy as np
import pytest
import torch

import paper_2609_15810_b200 as vc
from oracle import codecs as OC

pytestmark = pytest.mark.gpu


def _scores(n, cs, m, seed):
    """fp32 scores at or below m / cs: dense near the top, a long tail, and the special values."""
    rng = np.random.default_rng(seed)
    top = np.float32(m) / np.float32(cs)
    drop = np.concatenate([rng.exponential(3.0, n // 2), rng.uniform(0.0, 24.0, n - n // 2)])   # binades below the maximum
    s = (top - np.float32(1.0) / np.float32(cs) * drop.astype(np.float32)).astype(np.float32)
    s = np.round(s * 4.0) / 4.0                         # sums of products of codes: a coarse grid, many ties
    s = np.minimum(s.astype(np.float32), np.nextafter(top, np.float32(-np.inf)))
    s[0] = np.nextafter(top, np.float32(-np.inf))       # the row maximum itself
    s[1] = -np.inf                                      # a masked (padded) key
    s[2] = np.float32(-1.0e30)
    s[3] = np.minimum(np.float32(0.0), s[0])            # (no score exceeds the running maximum)
    return s.astype(np.float32)


def _kernel_arithmetic_exact(s, cs, m, beta):
    """t = fl32(s * fa + fb) with fa = cs / 16, fb = fl32(fl32(120 + beta - fl32(8 m)) / 128); code =
    nearest-even integer of 128 t, 0 below zero.  Exact rational arithmetic, fp32 roundings where the
    kernel rounds."""
    f32 = np.float32
    fa = f32(cs) * f32(0.0625)
    fb = f32(f32(f32(120.0) + f32(beta)) - f32(8.0) * f32(m)) * f32(0.0078125)
    out = np.zeros(s.shape, np.uint8)
    for i, x in enumerate(s):
        if not np.isfinite(x):
            continue                                    # -inf: code 0
        exact = Fraction(float(x)) * Fraction(float(fa)) + Fraction(float(fb))
        # one rounding to fp32, to nearest, ties to the even mantissa (float() rounds to double first,
        # so the neighbours of that guess are compared with the exact sum)
        t0 = f32(float(exact))
        cands = {float(t0), float(np.nextafter(t0, f32(-np.inf))), float(np.nextafter(t0, f32(np.inf)))}
        t = f32(min(cands, key=lambda c: (abs(Fraction(c) - exact), int(f32(c).view(np.uint32)) & 1)))
        if t <= 0:
            continue
        c128 = Fraction(float(t)) * 128
        fl = c128.numerator // c128.denominator
        rem = c128 - fl
        code = fl + (1 if (rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1)) else 0)
        out[i] = min(code, 255)
    return out


@pytest.mark.parametrize("cs,m,beta", [(3.1e-5, 17.3, 0.0), (0.37, -4.21875, 0.0), (1.0 / 128.0, 2.0, -0.5), (7.7e-4, 0.0, 0.0)])
def test_expcast_codes_against_eq7_and_against_the_kernels_own_arithmetic(cs, m, beta):
    n = 1 << 16
    s = _scores(n, cs, m, seed=int(abs(m) * 1000) + 7)
    got = vc.vc_test_expcast_codes(torch.from_numpy(s).cuda(), cs, m, beta).cpu().numpy()
    b = beta if beta != 0.0 else OC.EXPCAST_BETA
    # (1) the oracle's Eq. 7, two fp32 roundings before the fused multiply-add of the code
    z = (s * np.float32(cs)).astype(np.float32)
    u = (z - np.float32(m)).astype(np.float32)
    u = np.where(np.isfinite(u), u, np.float32(-1.0e30)).astype(np.float32)
    want = OC.expcast_code(u, beta=b)
    diff = np.abs(got.astype(np.int32) - want.astype(np.int32))
    assert diff.max() <= 1, (diff.max(), s[diff.argmax()])
    # a differing byte is a tie broken by the order of the fp32 roundings: the exact value of
    # 8 (s cs - m) + 120 + beta lies within 1e-4 of a half there
    bad = np.nonzero(diff)[0]
    c = 8.0 * (s[bad].astype(np.float64) * float(np.float32(cs)) - float(np.float32(m))) + 120.0 + float(np.float32(b))
    assert np.all(np.abs(c - np.floor(c) - 0.5) < 1e-4), c[:8]
    assert bad.size <= n // 100
    assert got[0] == 120 and got[1] == 0 and got[2] == 0          # the maximum, a masked key, a huge negative score
    # (2) the kernel's arithmetic, exactly: on a sample (rational arithmetic is slow) that holds every mismatch of (1)
    idx = np.unique(np.concatenate([np.arange(0, n, 37), np.nonzero(diff)[0], np.arange(16)]))
    exact = _kernel_arithmetic_exact(s[idx], cs, m, b)
    assert np.array_equal(got[idx], exact), np.nonzero(got[idx] != exact)[0][:8]


def test_expcast_codes_hook_rejects_bad_arguments():
    s = torch.zeros(8, dtype=torch.float32, device="cuda")
    with pytest.raises(vc.VcError):
        vc.vc_test_expcast_codes(s[:6], 1.0, 0.0)                  # not a multiple of 4
    with pytest.raises(vc.VcError):
        vc.vc_test_expcast_codes(s, 0.0, 0.0)                      # the factor must be positive
    assert vc.vc_test_expcast_codes(s[:0], 1.0, 0.0).numel() == 0
