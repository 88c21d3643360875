"""Pins for the oracle's block quantizers (CPU only): the 8-bit Q/K quantizer, NVFP4 groups
under an outer scale, the NVFP4 probability format and the quantized branches of the V pass.

Every check recomputes the result element by element with plain Python loops and a
brute-force nearest-value search over the decoded code table (the tables themselves are
pinned exhaustively in test_oracle_codecs.py), on inputs with planted maxima, exact rounding
ties, zero groups and a ragged last block, so that a wrong axis, a wrong top value, a per-row
instead of a per-block scale or a dropped scale fails.
"""
import numpy as np
import pytest

from oracle import attention as A
from oracle import codecs as C
from oracle import prep as P

F = np.float32

# decoded magnitudes of the two small formats, straight from the format definitions
E4M3_MAG = [float(C.e4m3_decode(c)) for c in range(127)]          # codes 0 .. 126 (127 is NaN)
E2M1_MAG = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]


def nearest_code(y, table):
    """Code of the table magnitude nearest to |y|, ties to the even code, saturating; the sign
    bit sits above the magnitude bits.  Brute force: every code is tried."""
    a = abs(float(y))
    best, best_d = 0, None
    for c, v in enumerate(table):
        d = abs(a - v)
        if best_d is None or d < best_d or (d == best_d and c % 2 == 0 and best % 2 == 1):
            best, best_d = c, d
    sign_bit = 128 if len(table) > 8 else 8
    return best | (sign_bit if np.signbit(F(y)) else 0)


def test_nearest_code_agrees_with_the_library_cast():
    """The brute-force search itself, against torch's independent E4M3 cast."""
    import torch
    rng = np.random.default_rng(0)
    y = np.concatenate([rng.uniform(-448, 448, 300), rng.standard_normal(300) * 0.02, [0.0, 448.0, 20.0, 22.0]]).astype(F)
    lib = torch.from_numpy(y).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    mine = np.array([nearest_code(v, E4M3_MAG) for v in y], dtype=np.uint8)
    assert np.array_equal(C.e4m3_decode(mine), C.e4m3_decode(lib))


# ----------------------------------------------------------------------------- 8-bit Q/K
def test_e4m3_block_quantizer_follows_its_definition():
    """Per block of 128 ROWS (not per row, not per tensor): s = amax / 448, code = E4M3 of
    x * (448 / amax) with both operations single fp32 operations, ties to even."""
    rng = np.random.default_rng(11)
    x = rng.normal(size=(256, 16)).astype(F)
    x[3, 5] = 7.0                                  # amax of block 0: its code must be 448 = 0x7E
    x[3, 6] = F(7.0 * 21.0 / 448.0)                # 21 = midpoint of 20 and 22 (step 2 in [16, 32))
    x[200, 2] = -5.5                               # amax of block 1, negative
    x[130] *= F(0.01)                              # a small row: a per-row scale would blow it up
    codes, scale, deq = P.quantize_e4m3_blocks(x)
    assert codes.dtype == np.uint8 and scale.shape == (2,)
    assert codes[3, 5] == 0x7E and codes[200, 2] == 0xFE
    for blk in range(2):
        rows = slice(128 * blk, 128 * (blk + 1))
        amax = F(np.abs(x[rows]).max())
        assert scale[blk] == F(amax / F(448.0))
        inv = F(F(448.0) / amax)
        for r in range(128 * blk, 128 * (blk + 1)):
            for c in range(16):
                y = F(x[r, c] * inv)
                want = nearest_code(y, E4M3_MAG)
                got = int(codes[r, c])
                assert (got & 0x7F) == (want & 0x7F), (r, c, float(y))
                assert (got & 0x7F) == 0 or got == want            # sign of a nonzero code
    y_tie = float(F(x[3, 6] * F(F(448.0) / F(7.0))))
    assert y_tie == 21.0 and (codes[3, 6] & 0x7F) == nearest_code(20.0, E4M3_MAG)   # tie -> the even code (20)
    # the small row keeps small codes: the scale is the block's, not the row's
    assert np.abs(C.e4m3_decode(codes[130])).max() < 0.05 * 448
    # dequantized values: code times the block scale, within half a step of the input
    assert np.array_equal(deq, C.e4m3_decode(codes) * np.repeat(scale.astype(np.float64), 128)[:, None])
    assert np.abs(deq - x).max() <= 0.5 * (32.0 / 448.0) * 7.0 + 1e-6              # widest step is 32 below 448
    z, s0, _ = P.quantize_e4m3_blocks(np.zeros((128, 8), dtype=F))
    assert s0[0] == 1.0 and not z.any()


# ----------------------------------------------------------------------------- NVFP4 groups
def _nvfp4_group_by_hand(g16, outer):
    """One group of 16 fp32 values -> (codes, micro code, decoded values without the outer scale)."""
    inv6 = F(F(1.0) / F(F(6.0) * outer))
    amax = F(max(abs(float(v)) for v in g16))
    sb = nearest_code(F(amax * inv6), E4M3_MAG) & 0x7F
    sdec = F(E4M3_MAG[sb])
    if sdec == 0:
        return [0] * 16, sb, [0.0] * 16
    rcp = F(F(1.0) / F(outer * sdec))
    codes = [nearest_code(F(v * rcp), E2M1_MAG) for v in g16]
    dec = [(-1.0 if c & 8 else 1.0) * E2M1_MAG[c & 7] * float(sdec) for c in codes]
    return codes, sb, dec


@pytest.mark.parametrize("outer", [1.0, 0.37, 5.25e-3])
def test_nvfp4_groups_with_outer_scale(outer):
    """E2M1 elements under an unsigned E4M3 microscale per 16 elements of the LAST axis, the
    whole under one outer scale g (the per-head scale of the 4-bit Q and K)."""
    outer = F(outer)
    rng = np.random.default_rng(5)
    x = (rng.standard_normal((6, 48)) * 20.0 * float(outer)).astype(F)
    x[0, :16] = 0.0                                     # a zero group: microscale 0, codes 0
    x[1, 16:32] *= F(1e-4)                              # a tiny group: its own microscale
    x[2, 3] = F(6.0 * 448.0) * outer                    # the head maximum: microscale 448, element 6
    x[3, 40] = -x[2, 3]
    codes, micro, deq = C.nvfp4_quantize_groups(x, outer_scale=outer)
    assert codes.shape == x.shape and micro.shape == (6, 3) and codes.max() <= 15
    assert micro[0, 0] == 0 and not codes[0, :16].any()
    assert micro[2, 0] == 0x7E and codes[2, 3] == 7 and codes[3, 40] == 15
    for r in range(6):
        for g in range(3):
            want_c, want_sb, want_dec = _nvfp4_group_by_hand(x[r, 16 * g:16 * g + 16], outer)
            assert micro[r, g] == want_sb, (r, g)
            got = codes[r, 16 * g:16 * g + 16].tolist()
            assert [c & 7 for c in got] == [c & 7 for c in want_c], (r, g)
            assert all((a & 7) == 0 or a == b for a, b in zip(got, want_c))
            assert np.allclose(deq[r, 16 * g:16 * g + 16], want_dec, rtol=0, atol=0)
    # decoded x outer reproduces the input within half an element step of its group (widest E2M1
    # gap is 2); a group whose maximum / 6 rounds to microscale 0 (below 2^-10) is dropped whole
    step = np.repeat(C.e4m3_decode(micro), 16, axis=1) * float(outer)
    assert np.all(np.abs(deq * float(outer) - x) <= np.maximum(step, 6.0 * 2.0 ** -10 * float(outer)) * (1 + 1e-6))


# ----------------------------------------------------------------------------- NVFP4 probabilities
def test_nvfp4_probability_format_by_brute_force():
    """P = 2^u * (6 * 448) quantized in groups of 16 KEYS of a row: the row maximum (u = 0)
    becomes element 6 under microscale 448, i.e. exactly 2688."""
    rng = np.random.default_rng(9)
    u = -np.abs(rng.standard_normal((4, 64)) * 3.0).astype(F)
    u[0, 17] = 0.0                                       # the running maximum of row 0
    u[1, :16] = -200.0                                   # a group that underflows completely
    u[2, 5] = 0.0
    p_hat = np.asarray(A.probability_codes(u, A.P_NVFP4, C.EXPCAST_BETA), dtype=np.float64)
    assert p_hat.shape == u.shape
    assert p_hat[0, 17] == 6.0 * 448.0 and p_hat[2, 5] == 2688.0
    assert not p_hat[1, :16].any()
    for r in range(4):
        p = [F(np.exp2(np.float64(v)) * A.NVFP4_P_SCALE) for v in u[r]]
        for g in range(4):
            _, _, want = _nvfp4_group_by_hand(p[16 * g:16 * g + 16], F(1.0))
            assert p_hat[r, 16 * g:16 * g + 16].tolist() == want, (r, g)
    # the groups follow the keys of a row, not the rows of a key: scaling one ROW's scores
    # changes only that row
    u2 = u.copy()
    u2[3] -= 4.0
    q2 = np.asarray(A.probability_codes(u2, A.P_NVFP4, C.EXPCAST_BETA))
    assert np.array_equal(q2[:3], p_hat[:3]) and not np.array_equal(q2[3], p_hat[3])


# ----------------------------------------------------------------------------- V pass, quantized
def _v_case(N=300, d=16, seed=21):
    rng = np.random.default_rng(seed)
    nb = (N + 127) // 128
    v = rng.standard_normal((N, d)) + 2.0 * np.repeat(rng.standard_normal((nb, d)), 128, 0)[:N]
    v[:, 3] *= 40.0                                      # one channel far larger than the others
    v[:, 7] = 1.25                                       # a constant channel: zero residual
    v = C.bf16_round(v.astype(F))
    perm = rng.permutation(N)
    cfg = lambda bits, **kw: P.PrepConfig(N=N, d=d, grid=(3, 10, 10), bits=bits, **kw)
    return v, perm, cfg


def _v_residual_by_hand(v, perm, N, d, mean_as_stored=False):
    n_pad = 128 * ((N + 127) // 128)
    x = [[0.0] * d for _ in range(n_pad)]
    for t in range(N):
        x[t] = [float(a) for a in v[perm[t]]]
    mu, r = [], [[F(0.0)] * d for _ in range(n_pad)]
    for j in range(n_pad // 128):
        n = min(128, N - 128 * j)
        m = [F(sum(x[128 * j + i][c] for i in range(n)) / n) for c in range(d)]   # Eq. 4, valid rows only
        if mean_as_stored:        # 4 bits: the bf16 mean that Eq. 6 adds back is the one subtracted
            m = [F(a) for a in C.bf16_round(np.array(m, dtype=F))]
        mu.append(m)
        for i in range(n):
            for c in range(d):
                r[128 * j + i][c] = F(x[128 * j + i][c] - float(m[c]))
    return mu, r, n_pad


def test_prep_v_8bit_by_loops():
    """8 bits: one scale per CHANNEL over all tokens of the residual, codes E4M3 of
    r * (448 / amax_c), block means stored divided by the scale and rounded to bf16 (App. B)."""
    N, d = 300, 16
    v, perm, cfg = _v_case(N, d)
    out = P.prep_v(v, perm, cfg(8))
    mu, r, n_pad = _v_residual_by_hand(v, perm, N, d)
    assert out["v_codes"].shape == (n_pad, d) and out["v_scale"].shape == (d,) and out["v_means"].shape == (3, d)
    for c in range(d):
        amax = F(max(abs(float(r[t][c])) for t in range(n_pad)))
        if amax == 0:                                   # the constant channel
            assert out["v_scale"][c] == 1.0 and not out["v_codes"][:, c].any()
            for j in range(3):
                assert out["v_means"][j, c] == C.bf16_round(np.array([mu[j][c]], dtype=F))[0]
            continue
        assert out["v_scale"][c] == F(amax / F(448.0))
        inv = F(F(448.0) / amax)
        for t in range(n_pad):
            want = nearest_code(F(r[t][c] * inv), E4M3_MAG)
            got = int(out["v_codes"][t, c])
            assert (got & 0x7F) == (want & 0x7F) and ((got & 0x7F) == 0 or got == want), (t, c)
        for j in range(3):
            assert out["v_means"][j, c] == C.bf16_round(np.array([F(mu[j][c] * inv)], dtype=F))[0]
    assert (out["v_codes"][:, 3] & 0x7F).max() == 0x7E and (out["v_codes"][:, 0] & 0x7F).max() == 0x7E   # every channel reaches its own top
    assert not out["v_codes"][N:].any()                 # padding rows: zero residual code
    # decoded residual times the scale, plus the restored mean, reproduces the gathered V
    rec = C.e4m3_decode(out["v_codes"][:N]) * out["v_scale"].astype(np.float64) + \
        np.repeat(out["v_means"].astype(np.float64) * out["v_scale"].astype(np.float64), 128, 0)[:N]
    err = np.abs(rec - v[perm].astype(np.float64))
    live = [c for c in range(d) if c != 7]              # half the widest code step (32) plus the bf16 mean
    bound = out["v_scale"].astype(np.float64) * 16.0 + np.abs(np.repeat(np.array(mu, dtype=np.float64), 128, 0)[:N]) * 2.0 ** -8
    assert np.all(err[:, live] <= bound[:, live] + 1e-6)


@pytest.mark.parametrize("fmt", ["nvfp4", "mxfp4"])
def test_prep_v_4bit_by_loops(fmt):
    """4 bits: groups of 16 (NVFP4) or 32 (power-of-two factors) consecutive PERMUTED TOKENS of
    one channel, no tensor-level scale, block means stored unscaled in bf16 (App. B)."""
    N, d = 300, 16
    v, perm, cfg = _v_case(N, d)
    out = P.prep_v(v, perm, cfg(4, v_format=fmt))
    mu, r, n_pad = _v_residual_by_hand(v, perm, N, d, mean_as_stored=True)
    G = 16 if fmt == "nvfp4" else 32
    assert out["v_codes"].shape == (n_pad, d) and out["v_micro"].shape == (n_pad // G, d)
    assert np.all(out["v_scale"] == 1.0)
    for j in range(3):
        assert np.array_equal(out["v_means"][j], np.array(mu[j], dtype=F))
    # Eq. 6 at 4 bits: residual plus STORED mean is the gathered value again, exactly
    assert np.array_equal((out["v_pre"][:N].astype(np.float64) + np.repeat(out["v_means"].astype(np.float64), 128, 0)[:N]).astype(F),
                          v[perm])
    for c in range(d):
        for g in range(n_pad // G):
            col = [r[G * g + i][c] for i in range(G)]
            if fmt == "nvfp4":
                want_c, want_sb, want_dec = _nvfp4_group_by_hand(col, F(1.0))
            else:
                amax = max(abs(float(a)) for a in col)
                if amax == 0:
                    want_c, want_sb, want_dec = [0] * G, 0, [0.0] * G
                else:
                    e = -200
                    while 6.0 * 2.0 ** e < amax:         # smallest power of two that avoids clipping
                        e += 1
                    want_sb = e + 127
                    want_c = [nearest_code(F(float(a) / 2.0 ** e), E2M1_MAG) for a in col]
                    want_dec = [(-1.0 if k & 8 else 1.0) * E2M1_MAG[k & 7] * 2.0 ** e for k in want_c]
            assert out["v_micro"][g, c] == want_sb, (g, c)
            got = out["v_codes"][G * g:G * g + G, c].tolist()
            assert [a & 7 for a in got] == [a & 7 for a in want_c], (g, c)
            assert all((a & 7) == 0 or a == b for a, b in zip(got, want_c))
            assert out["v_deq"][G * g:G * g + G, c].tolist() == want_dec
    assert not out["v_codes"][:, 7].any() and not out["v_codes"][N:].any()
