"""Pins for the oracle's number formats and the ExpCast-FP8 map (CPU only).

Each check ties the oracle to something other than itself: the format definition
evaluated by hand, an independent library cast (torch), or a value the paper prints
(tests/golden/*.txt).
"""
import os

import numpy as np
import torch

from oracle import codecs as C

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden_constants():
    out = {}
    with open(os.path.join(GOLDEN, "expcast_constants.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                name, value, tol = line.split()
                out[name] = (float(value), float(tol))
    return out


# ----------------------------------------------------------------------------- E4M3
def test_e4m3_decode_by_hand():
    # 2^(e-7)(1+m/8), Sec. 3.3; subnormals (m/8) 2^-6
    assert C.e4m3_decode(0x38) == 1.0            # e=7, m=0
    assert C.e4m3_decode(0x7E) == 448.0          # e=15, m=6
    assert C.e4m3_decode(0x78) == 256.0          # code 120
    assert C.e4m3_decode(107) == 88.0            # 8*13+3 -> 2^6 * 1.375
    assert C.e4m3_decode(0x01) == 2.0 ** -9
    assert C.e4m3_decode(0x07) == 7 * 2.0 ** -9
    assert C.e4m3_decode(0x08) == 2.0 ** -6
    assert C.e4m3_decode(0xB8) == -1.0
    assert np.isnan(C.e4m3_decode(0x7F)) and np.isnan(C.e4m3_decode(0xFF))


def test_e4m3_exhaustive_roundtrip():
    codes = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=np.uint8)
    vals = C.e4m3_decode(codes)
    assert np.array_equal(C.e4m3_encode(vals), codes)
    # decoded values are strictly increasing in the magnitude code
    pos = C.e4m3_decode(np.arange(0, 127, dtype=np.uint8))
    assert np.all(np.diff(pos) > 0)


def test_e4m3_ties_to_even_and_saturation():
    pos = C.e4m3_decode(np.arange(0, 127, dtype=np.uint8))
    mid = 0.5 * (pos[:-1] + pos[1:])                 # exact midpoints
    enc = C.e4m3_encode(mid).astype(int)
    lo = np.arange(0, 126)
    expect = np.where(lo % 2 == 0, lo, lo + 1)       # the neighbour with the even code
    assert np.array_equal(enc, expect)
    # just off the midpoint goes to the nearer neighbour
    assert np.array_equal(C.e4m3_encode(np.nextafter(mid, np.inf)).astype(int), lo + 1)
    assert np.array_equal(C.e4m3_encode(np.nextafter(mid, -np.inf)).astype(int), lo)
    assert C.e4m3_encode(np.array([449.0, 464.0, 1e9]))[-3:].tolist() == [0x7E] * 3
    assert C.e4m3_encode(np.array([-1e9]))[0] == 0xFE


def test_e4m3_encode_matches_library_cast():
    rng = np.random.default_rng(7)
    x = np.concatenate([rng.standard_normal(200000) * 30.0,
                        rng.standard_normal(50000) * 0.01,
                        rng.uniform(-448, 448, 50000)]).astype(np.float32)
    x = x[np.abs(x) <= 448.0]
    lib = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    mine = C.e4m3_encode(x)
    # the library has one zero code per sign as well; compare decoded magnitudes and signs
    assert np.array_equal(C.e4m3_decode(mine), C.e4m3_decode(lib))


# ----------------------------------------------------------------------------- E2M1
def test_e2m1_values_and_rounding():
    assert C.e2m1_decode(np.arange(8)).tolist() == [0, 0.5, 1, 1.5, 2, 3, 4, 6]
    assert C.e2m1_decode(np.arange(8, 16)).tolist() == [-0.0, -0.5, -1, -1.5, -2, -3, -4, -6]
    codes = np.arange(16, dtype=np.uint8)
    assert np.array_equal(C.e2m1_encode(C.e2m1_decode(codes)), codes)
    # ties go to the even code: by hand from the value list
    ties = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0])
    assert C.e2m1_decode(C.e2m1_encode(ties)).tolist() == [0.0, 1.0, 1.0, 2.0, 2.0, 4.0, 4.0]
    near = np.array([0.2501, 0.7499, 2.51, 4.99, 5.01, 7.0, 100.0, -9.0])
    assert C.e2m1_decode(C.e2m1_encode(near)).tolist() == [0.5, 0.5, 3.0, 4.0, 6.0, 6.0, 6.0, -6.0]


def test_nvfp4_group_quantizer_brute_force():
    """Against a brute-force nearest-value search over the 16 x 8 grid of one group."""
    rng = np.random.default_rng(3)
    x = (rng.standard_normal((64, 32)) * rng.uniform(0.01, 20, (64, 1))).astype(np.float32)
    codes, micro, deq = C.nvfp4_quantize_groups(x)
    grid = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6])
    for r in range(x.shape[0]):
        for g in range(2):
            seg = x[r, 16 * g:16 * g + 16].astype(np.float64)
            s = C.e4m3_decode(micro[r, g])
            # microscale = E4M3 value nearest to amax / 6
            allv = C.e4m3_decode(np.arange(0, 127, dtype=np.uint8))
            target = np.float32(np.abs(seg).max()) * np.float32(1.0 / 6.0)
            assert abs(s - target) == np.min(np.abs(allv - target))
            y = seg / s
            best = np.abs(np.abs(y)[:, None] - grid[None, :]).min(axis=1)
            got = np.abs(np.abs(deq[r, 16 * g:16 * g + 16]) / s - np.abs(y))
            # nearest grid point up to the fp32 rounding of the reciprocal multiply
            assert np.all(got <= best + 1e-5)
    z, mz, dz = C.nvfp4_quantize_groups(np.zeros((1, 16), np.float32))
    assert not z.any() and not mz.any() and not dz.any()


def test_mxfp4_group_quantizer_brute_force():
    """E2M1 under a power-of-two factor per 32: the factor is the smallest power of two that
    leaves the group maximum inside the E2M1 range (checked by exhaustive search over the
    exponent), elements are the nearest grid values, and a power-of-two input is reproduced."""
    rng = np.random.default_rng(5)
    x = (rng.standard_normal((48, 64)) * rng.uniform(1e-3, 50, (48, 1))).astype(np.float32)
    x[0, :32] = 0.0
    x[1, :32] = 4.0 * np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6] * 4, np.float32) * rng.choice([-1.0, 1.0], 32)   # grid values x 2^2
    x[2, :32] = np.float32(6.0000005) * 4                                         # just above: next power
    codes, sc, deq = C.mxfp4_quantize_groups(x)
    grid = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6])
    for r in range(x.shape[0]):
        for g in range(2):
            seg = x[r, 32 * g:32 * g + 32].astype(np.float64)
            amax = np.abs(seg).max()
            if amax == 0:
                assert sc[r, g] == 0 and not codes[r, 32 * g:32 * g + 32].any()
                continue
            e = int(sc[r, g]) - 127
            es = [k for k in range(-40, 40) if amax <= 6.0 * 2.0 ** k]
            assert e == min(es)                                   # no clipping, and no smaller factor does that
            y = np.abs(seg) / 2.0 ** e
            best = np.abs(y[:, None] - grid[None, :]).min(axis=1)
            got = np.abs(np.abs(deq[r, 32 * g:32 * g + 32]) / 2.0 ** e - y)
            assert np.array_equal(got, best)                      # exact scaling: the nearest value, no slack
    assert np.array_equal(deq[1, :32], x[1, :32].astype(np.float64))
    assert sc[2, 0] == 127 + 3 and C.ue8m0_decode(sc[2, 0]) == 8.0


# ----------------------------------------------------------------------------- bf16
def test_bf16_round_matches_library_cast():
    rng = np.random.default_rng(11)
    x = (rng.standard_normal(300000) * np.exp(rng.uniform(-20, 20, 300000))).astype(np.float32)
    ties = (np.arange(1, 4001, dtype=np.uint32) << np.uint32(16) | np.uint32(0x8000)).view(np.float32) * 1e3
    x = np.concatenate([x, ties.astype(np.float32)])
    lib = torch.from_numpy(x).to(torch.bfloat16).float().numpy()
    assert np.array_equal(C.bf16_round(x), lib)
    assert np.array_equal(C.bf16_bits(lib), torch.from_numpy(lib).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))


# ----------------------------------------------------------------------------- ExpCast-FP8
def test_expcast_worked_example_from_the_paper():
    with open(os.path.join(GOLDEN, "expcast_worked_example.txt")) as f:
        row = [l for l in f if not l.startswith("#") and l.strip()][0].split()
    u, affine, byte, e, m, decoded, p_exact, decoded_cast = map(float, row)
    assert abs((8 * (u + 8) + 56 + C.EXPCAST_BETA) - affine) < 1e-9
    code = int(C.expcast_code(np.float32(u)))
    assert code == int(byte) == 8 * int(e) + int(m)
    assert C.e4m3_decode(code) == decoded
    assert abs(2.0 ** (u + 8) - p_exact) < 0.05
    assert C.e4m3_decode(C.exp_then_cast_code(np.float32(u))) == decoded_cast


def test_expcast_printed_constants():
    g = _golden_constants()
    # one doubling of the probability, dense grid (every unit interval of u looks the same)
    u = (-3.0 + (np.arange(2_000_000) + 0.5) / 2_000_000).astype(np.float64)
    direct = C.expcast_code(u.astype(np.float32)).astype(int)
    cast = C.exp_then_cast_code(u.astype(np.float32)).astype(int)
    share = np.mean(direct == cast)
    assert abs(share - g["same_byte_share"][0]) <= g["same_byte_share"][1]
    assert np.abs(direct - cast).max() == g["max_code_gap"][0]
    exact = np.exp2(u + 8.0)
    rel = np.abs(C.e4m3_decode(direct) / exact - 1.0).max()
    assert abs(rel - g["max_rel_error"][0]) <= g["max_rel_error"][1]
    ratio = C.e4m3_decode(direct) / exact
    assert abs(ratio.min() - g["ratio_lo"][0]) <= g["ratio_lo"][1]
    assert abs(ratio.max() - g["ratio_hi"][0]) <= g["ratio_hi"][1]
    a, b = g["ratio_lo"][0], g["ratio_hi"][0]
    tv = (np.sqrt(b) - np.sqrt(a)) / (np.sqrt(b) + np.sqrt(a))
    assert tv < g["tv_bound"][0] and abs(tv - g["tv_bound"][0]) <= g["tv_bound"][1]
    # Mitchell's straight-line error scaled to E4M3 codes and its minimax centering
    f = np.linspace(0, 1, 1_000_001)
    e = 8.0 * (f - (np.exp2(f) - 1.0))
    assert e.min() >= 0 and abs(e.max() - g["mitchell_range_hi"][0]) <= g["mitchell_range_hi"][1]
    assert abs(-e.max() / 2 - g["minimax_shift"][0]) <= g["minimax_shift"][1]
    assert C.EXPCAST_BETA == g["beta"][0]
    # the row maximum (u = 0) lands at 256 and nothing exceeds it
    assert int(C.expcast_code(np.float32(0.0))) == g["top_code"][0]
    assert C.e4m3_decode(int(g["top_code"][0])) == 256.0
    assert direct.max() <= 120
    # underflow maps to zero, codes never leave [0, 120]
    assert int(C.expcast_code(np.float32(-40.0))) == 0
    assert int(C.expcast_code(np.float32(-14.97))) == 0 and int(C.expcast_code(np.float32(-14.8))) == 1


def test_expcast_row_total_variation_bound():
    """Prop. 3.1: TV(p, p_hat) < 0.0364 on rows in the normal range, + tau with a tail."""
    rng = np.random.default_rng(5)
    worst = 0.0
    for trial in range(300):
        n = int(rng.integers(2, 400))
        u = -rng.uniform(0, 14, n) * rng.uniform(0.05, 1.0)
        u[rng.integers(n)] = 0.0                       # the row maximum
        u = u.astype(np.float32)
        w = np.exp2(u.astype(np.float64))
        p = w / w.sum()
        wh = C.e4m3_decode(C.expcast_code(u))
        ph = wh / wh.sum()
        tv = 0.5 * np.abs(p - ph).sum()
        worst = max(worst, tv)
        assert tv < 0.0364
    assert worst > 0.003                               # the bound is not vacuous on these rows
    for trial in range(100):                           # rows with an underflow tail
        n = int(rng.integers(8, 400))
        u = -rng.uniform(0, 30, n)
        u[0] = 0.0
        u = u.astype(np.float32)
        w = np.exp2(u.astype(np.float64)); p = w / w.sum()
        wh = C.e4m3_decode(C.expcast_code(u)); ph = wh / wh.sum()
        tail = u < -14
        tau = max(p[tail].sum(), ph[tail].sum())
        assert 0.5 * np.abs(p - ph).sum() < 0.0364 + tau
