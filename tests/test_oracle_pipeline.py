"""Pins for the oracle's preprocessing chain and attention recurrence (CPU only).

Identities the paper states (Hadamard orthogonality, softmax invariance to the K mean,
permutation invariance Eq. 3, energy identity Eq. 5, exact mean restoration Eq. 6) and
brute-force attention on tiny inputs with quantization switched off.
"""
import numpy as np
import pytest
import torch

import vc_inputs
import vc_kmeans_harness
from oracle import attention as A
from oracle import codecs as C
from oracle import prep as P


def _tiny(N=320, d=64, grid=(5, 8, 8), seed=0, k_off=3.0, v_shift=1.0):
    rng = np.random.default_rng(seed)
    bf = lambda x: C.bf16_round(x.astype(np.float32))
    q = bf(rng.standard_normal((N, d)))
    k = bf(rng.standard_normal((N, d)) + k_off * rng.standard_normal((1, d)))
    nb = (N + 127) // 128
    v = bf(rng.standard_normal((N, d)) + v_shift * np.repeat(rng.standard_normal((nb, d)), 128, 0)[:N])
    return q, k, v


def _brute_force(q, k, v, scale):
    """Attention with explicit Python loops (tiny inputs only)."""
    N, d = q.shape
    out = np.zeros((N, v.shape[1]))
    for i in range(N):
        s = np.array([sum(float(q[i, c]) * float(k[j, c]) for c in range(d)) for j in range(k.shape[0])]) * scale
        w = np.exp(s - s.max())
        w /= w.sum()
        out[i] = w @ v.astype(np.float64)
    return out


# ----------------------------------------------------------------------------- building blocks
@pytest.mark.parametrize("d", [64, 128])
def test_hadamard_is_orthogonal_and_preserves_scores(d):
    H = P.hadamard_matrix(d)
    assert np.array_equal(H @ H.T, d * np.eye(d, dtype=np.int64))
    assert np.array_equal(H, H.T) and set(np.unique(H)) == {-1, 1}
    assert np.all(H[0] == 1) and H[1, :4].tolist() == [1, -1, 1, -1]      # natural (Sylvester) order
    rng = np.random.default_rng(1)
    q, k = rng.standard_normal((9, d)), rng.standard_normal((11, d))
    Hn = H / np.sqrt(d)
    assert np.abs((q @ Hn) @ (k @ Hn).T - q @ k.T).max() < 1e-12
    x32 = rng.standard_normal((5, d)).astype(np.float32)
    assert np.abs(P.hadamard_apply(x32) - x32.astype(np.float64) @ Hn).max() < 1e-6


def test_rope_relative_position_and_identity():
    cfg = P.PrepConfig(N=4 * 6 * 8, d=64, grid=(4, 6, 8))
    cos, sin = P.rope_tables(cfg)
    assert np.all(cos[0] == 1.0) and np.all(sin[0] == 0.0)          # position 0: identity
    rng = np.random.default_rng(2)
    qv, kv = rng.standard_normal(64), rng.standard_normal(64)
    q = np.tile(qv, (cfg.N, 1)).astype(np.float32)
    k = np.tile(kv, (cfg.N, 1)).astype(np.float32)
    qr, kr = P.rope_apply(q, cos, sin).astype(np.float64), P.rope_apply(k, cos, sin).astype(np.float64)
    s = qr @ kr.T
    T, Hg, Wg = cfg.grid
    idx = lambda t, y, x: (t * Hg + y) * Wg + x
    # the score depends only on the per-axis offset between the two tokens
    ref = s[idx(2, 3, 5), idx(1, 1, 2)]
    for (t, y, x) in [(1, 2, 3), (3, 4, 7), (2, 5, 4)]:
        assert abs(s[idx(t, y, x), idx(t - 1, y - 2, x - 3)] - ref) < 2e-4
    assert abs(s[idx(2, 3, 5), idx(1, 1, 3)] - ref) > 1e-3            # a different offset differs
    # a rotation preserves the norm of every pair
    assert np.allclose((qr ** 2).reshape(cfg.N, 32, 2).sum(-1), (q.astype(np.float64) ** 2).reshape(cfg.N, 32, 2).sum(-1), atol=1e-5)
    # the three axes own disjoint channel ranges: moving along x leaves the t and y pairs alone
    dt, dy, dx = cfg.rope_dims
    assert np.allclose(qr[idx(1, 2, 0), :dt + dy], qr[idx(1, 2, 7), :dt + dy])
    assert not np.allclose(qr[idx(1, 2, 0), dt + dy:], qr[idx(1, 2, 7), dt + dy:])
    # first pair of the t axis has frequency 1: angle = t
    assert abs(cos[idx(3, 0, 0), 0] - np.cos(3.0)) < 1e-7 and abs(sin[idx(3, 0, 0), 0] - np.sin(3.0)) < 1e-7
    assert abs(cos[idx(0, 0, 5), (dt + dy) // 2 + 1] - np.cos(5.0 * 10000.0 ** (-2.0 / dx))) < 1e-7


def test_k_mean_subtraction_leaves_softmax_unchanged():
    q, k, v = _tiny()
    kbar = k.astype(np.float64).mean(axis=0)
    o = A.exact_attention(q, k, v)
    o2 = A.exact_attention(q, k.astype(np.float64) - kbar, v)
    assert np.abs(o - o2).max() < 1e-12


def test_permutation_invariance_eq3():
    q, k, v = _tiny()
    perm = np.random.default_rng(3).permutation(q.shape[0])
    assert np.abs(A.exact_attention(q, k[perm], v[perm]) - A.exact_attention(q, k, v)).max() < 1e-12


def test_exact_attention_is_brute_force():
    q, k, v = _tiny(N=40, d=8, grid=(2, 4, 5))
    assert np.abs(A.exact_attention(q, k, v) - _brute_force(q, k, v, 1 / np.sqrt(8))).max() < 1e-12


def test_block_demeaning_energy_identity_eq5():
    q, k, v = _tiny(N=300, d=64, grid=(3, 10, 10))
    cfg = P.PrepConfig(N=300, d=64, grid=(3, 10, 10), bits=0)
    perm = np.random.default_rng(4).permutation(300)
    out = P.prep_v(v, perm, cfg)
    mu, r = out["v_means"], out["v_deq"]
    vp = v[perm].astype(np.float64)
    for j in range(cfg.n_blocks):
        blk = vp[128 * j:128 * (j + 1)]
        n = blk.shape[0]
        assert np.abs(mu[j] - blk.mean(axis=0)).max() < 1e-12            # Eq. 4, partial block / n valid
        rj = r[128 * j:128 * j + n]
        assert np.abs(rj + mu[j] - blk).max() < 1e-12
        assert abs((rj ** 2).sum() - ((blk ** 2).sum() - n * (mu[j] ** 2).sum())) < 1e-8
        c = np.random.default_rng(j).standard_normal(64)
        lhs = ((blk - c) ** 2).sum()
        assert abs(lhs - ((rj ** 2).sum() + n * ((c - mu[j]) ** 2).sum())) < 1e-8
    assert not r[300:].any()                                              # padding rows: zero residual


# ----------------------------------------------------------------------------- recurrence
@pytest.mark.parametrize("tile", [128, 64])
def test_recurrence_exact_equals_brute_force_with_mean_restoration(tile):
    """Quantization off: Eq. 1 + Eq. 6 reproduce attention exactly (1e-10), ragged tail
    included, for any tile size."""
    N, d = 200, 16
    q, k, v = _tiny(N=N, d=d, grid=(2, 10, 10))
    cfg = P.PrepConfig(N=N, d=d, grid=(2, 10, 10), bits=0)
    perm = np.random.default_rng(6).permutation(N)
    vv = P.prep_v(v, perm, cfg)
    kp = P.pad_rows(k[perm].astype(np.float64), cfg.n_pad)
    qp = P.pad_rows(q.astype(np.float64), cfg.n_pad)
    scale = A.LOG2E / np.sqrt(d)
    if tile == 128:
        means = vv["v_means"]
        vdeq = vv["v_deq"]
    else:   # tile size must not change the unquantized result: hand it per-64 means
        vpad = P.pad_rows(v[perm].astype(np.float64), cfg.n_pad)
        means = np.zeros((cfg.n_pad // 128, d))
        vdeq = vpad
    o = A.recurrence(qp, kp, vdeq, means, N, scale, A.P_EXACT, exact=True, tile=tile)
    ref = _brute_force(q, k, v, 1 / np.sqrt(d))
    assert np.abs(o - ref).max() < 1e-10
    # rows subset
    rows = np.array([0, 5, 127, 128, 199])
    o2 = A.recurrence(qp, kp, vdeq, means, N, scale, A.P_EXACT, exact=True, rows=rows, tile=tile)
    assert np.abs(o2 - ref[rows]).max() < 1e-10


def test_mean_restoration_with_quantized_p_is_exact():
    """With l and r summing the decoded codes, P_hat (R + 1 mu^T) = P_hat V' holds for the
    quantized probabilities too (Eq. 6): V-Smooth on/off agree when R is left unquantized."""
    N, d = 384, 32
    q, k, v = _tiny(N=N, d=d, grid=(6, 8, 8))
    cfg = P.PrepConfig(N=N, d=d, grid=(6, 8, 8), bits=0)
    perm = np.arange(N)
    on = P.prep_v(v, perm, cfg)
    scale = np.float32(A.LOG2E / np.sqrt(d))
    qd, kd = q.astype(np.float64), k.astype(np.float64)
    o_on = A.recurrence(qd, kd, on["v_deq"], on["v_means"], N, scale, A.P_EXPCAST, exact=True)
    o_off = A.recurrence(qd, kd, v.astype(np.float64), np.zeros_like(on["v_means"]), N, scale, A.P_EXPCAST, exact=True)
    assert np.abs(o_on - o_off).max() < 1e-10
    # and the ExpCast row obeys the output bound of Prop. 3.1 with its tail
    ref = A.exact_attention(q, k, v)
    diam = np.sqrt(((v[:, None, :].astype(np.float64) - v[None, :, :]) ** 2).sum(-1)).max()
    assert np.linalg.norm(o_off - ref, axis=1).max() <= (0.0364 + 0.01) * diam


def test_size_of_the_8bit_mean_rounding_offset():
    """At 8 bits the block mean is stored as bf16(mu / s_V) and restored as s_V times that (App. B),
    so what Eq. 6 adds back differs from what Eq. 4 subtracted by at most one bf16 rounding of the
    mean: |s_V bf16(mu / s_V) - mu| <= 2^-8 |mu| (half an ulp of an 8-bit significand, plus the
    fp32 roundings).  Because the probabilities of a row sum to one, that offset reaches the output
    unchanged: with every other quantizer switched off, the output with stored means differs from
    the output with exact means by no more than the largest offset."""
    N, d = 384, 32
    q, k, v = _tiny(N=N, d=d, grid=(6, 8, 8), seed=4, v_shift=3.0)
    cfg8 = P.PrepConfig(N=N, d=d, grid=(6, 8, 8), bits=8)
    b8 = P.prep_v(v, np.arange(N), cfg8)
    mu = b8["v_mu"].astype(np.float64)
    restored = b8["v_means"].astype(np.float64) * b8["v_scale"].astype(np.float64)[None, :]
    off = np.abs(restored - mu)
    assert np.all(off <= 2.0 ** -8 * np.abs(mu) * (1 + 1e-3) + 1e-12) and off.max() > 0
    exact = P.prep_v(v, np.arange(N), P.PrepConfig(N=N, d=d, grid=(6, 8, 8), bits=0))
    scale = np.float32(A.LOG2E / np.sqrt(d))
    qd, kd = q.astype(np.float64), k.astype(np.float64)
    o_exact = A.recurrence(qd, kd, exact["v_deq"], exact["v_means"], N, scale, A.P_EXPCAST, exact=True)
    o_stored = A.recurrence(qd, kd, exact["v_deq"], restored, N, scale, A.P_EXPCAST, exact=True)
    assert np.abs(o_stored - o_exact).max() <= off.max() * (1 + 1e-9)
    assert np.abs(o_stored - o_exact).max() > 0.1 * off.max()          # and it is that offset, not something smaller


def test_running_max_and_alpha_follow_eq1():
    """Trace the recurrence on one row by hand."""
    N, d = 256, 16
    q, k, v = _tiny(N=N, d=d, grid=(4, 8, 8), seed=9)
    tr = []
    A.recurrence(q, k, v, np.zeros((2, d)), N, np.float32(0.3), A.P_EXPCAST, rows=np.array([7]), trace=tr)
    z = (q[7].astype(np.float64) @ k.astype(np.float64).T).astype(np.float32) * np.float32(0.3)
    m0, m1 = z[:128].max(), max(z[:128].max(), z[128:].max())
    assert tr[0]["m"][0] == m0 and tr[1]["m"][0] == m1
    assert tr[0]["alpha"][0] == 0.0 and abs(tr[1]["alpha"][0] - 2.0 ** (float(m0) - float(m1))) < 1e-7
    assert tr[0]["p_hat"][0].max() == 256.0                           # the tile maximum sits at code 120
    assert np.array_equal(tr[1]["p_hat"][0], C.e4m3_decode(C.expcast_code(z[128:] - m1)))
    assert tr[1]["r"][0] == tr[1]["p_hat"][0].sum()


# ----------------------------------------------------------------------------- whole pipeline
@pytest.mark.parametrize("perm_kind", ["identity", "random"])
def test_pipeline_without_quantization_matches_exact(perm_kind):
    """RoPE, K smoothing, permutation, Hadamard, block demeaning and restoration leave the
    output unchanged (up to the fp32 rounding between stages)."""
    w = vc_inputs.Workload("t", 1, 1, 300, 64, (3, 10, 10), (8,), 5, "gauss")
    q, k, v = [t[0, 0].float().numpy() for t in vc_inputs.make_qkv(w)]
    cfg = P.PrepConfig(N=300, d=64, grid=w.grid, bits=0)
    perm = None if perm_kind == "identity" else np.random.default_rng(8).permutation(300)
    b = P.prep_head(q, k, v, perm, cfg)
    o = A.recurrence(b["q_deq"], b["k_deq"], b["v_deq"], b["v_means"], 300,
                     A.LOG2E / np.sqrt(64), A.P_EXACT, exact=True)
    ref = A.reference_head(q, k, v, cfg)
    assert np.abs(o - ref).max() < 2e-4


@pytest.mark.parametrize("bits,cos_min,tol", [(8, 0.9995, 2e-2), (4, 0.995, 8e-2)])
def test_quantized_pipeline_tracks_exact_attention(bits, cos_min, tol):
    w = vc_inputs.WORKLOADS["c1"]
    q, k, v = [t[0, 0].float().numpy() for t in vc_inputs.make_qkv(w, heads=[0])]
    cfg = P.PrepConfig(N=w.N, d=w.d, grid=w.grid, bits=bits)
    rows = np.arange(0, w.N, 7)
    ref = A.reference_head(q, k, v, cfg, rows=rows)
    b = P.prep_head(q, k, v, None, cfg)
    o = A.emulate_head(b, cfg, rows=rows).astype(np.float64)
    cos = (o * ref).sum() / np.linalg.norm(o) / np.linalg.norm(ref)
    assert cos > cos_min
    assert np.abs(o - ref).max() < tol * np.abs(v).max()


def test_hybrid_4bit_arrangement_tracks_exact_attention():
    """ExpCast-FP8 P over 4-bit Q, K and values under power-of-two factors per 32 tokens: the
    value codes decode to the residual within half a grid step of their group, and the output
    is closer to exact attention than with the NVFP4 probability."""
    w = vc_inputs.WORKLOADS["c1"]
    q, k, v = [t[0, 0].float().numpy() for t in vc_inputs.make_qkv(w, heads=[0])]
    rows = np.arange(0, w.N, 7)
    cfg = P.PrepConfig(N=w.N, d=w.d, grid=w.grid, bits=4, v_format="mxfp4")
    b = P.prep_head(q, k, v, None, cfg)
    assert b["v_micro"].shape == (cfg.n_pad // 32, w.d)
    step = np.repeat(np.exp2(b["v_micro"].astype(np.float64) - 127.0), 32, axis=0)   # factor per element
    assert np.all(np.abs(b["v_deq"] - b["v_pre"]) <= step + 1e-12)                    # widest E2M1 gap is 2: half of it
    ref = A.reference_head(q, k, v, cfg, rows=rows)
    o = A.emulate_head(b, cfg, rows=rows, p_format=A.P_EXPCAST).astype(np.float64)
    cos = (o * ref).sum() / np.linalg.norm(o) / np.linalg.norm(ref)
    assert cos > 0.995 and np.abs(o - ref).max() < 8e-2 * np.abs(v).max()
    b4 = P.prep_head(q, k, v, None, P.PrepConfig(N=w.N, d=w.d, grid=w.grid, bits=4))
    o4 = A.emulate_head(b4, cfg, rows=rows).astype(np.float64)
    assert np.sqrt(((o - ref) ** 2).mean()) < 1.05 * np.sqrt(((o4 - ref) ** 2).mean())


def test_smoothing_helps_on_data_it_is_meant_for():
    """K smoothing on K with channel offsets, V smoothing on V with block shifts: each must
    lower the error against exact attention (the directions the paper claims)."""
    w = vc_inputs.WORKLOADS["c1"]
    q, k, v = [t[0, 0].float().numpy() for t in vc_inputs.make_qkv(w, heads=[1])]
    rows = np.arange(0, w.N, 5)
    err = {}
    for name, kw in {"both": {}, "no_k": {"k_smooth": False}, "no_v": {"v_smooth": False}}.items():
        cfg = P.PrepConfig(N=w.N, d=w.d, grid=w.grid, bits=8, **kw)
        ref = A.reference_head(q, k, v, cfg, rows=rows)
        o = A.emulate_head(P.prep_head(q, k, v, None, cfg), cfg, rows=rows, p_format=A.P_EXP_E4M3)
        err[name] = np.sqrt(((o - ref) ** 2).mean())
    assert err["both"] < err["no_k"] and err["both"] < err["no_v"]


def test_error_decomposition_eq2():
    """O - O_q = (P - P_q) V + P_q (V - V_q) with P_q the normalized decoded codes."""
    N, d = 256, 32
    q, k, v = _tiny(N=N, d=d, grid=(4, 8, 8), seed=12)
    cfg = P.PrepConfig(N=N, d=d, grid=(4, 8, 8), bits=8, rope=False, hadamard=False, k_smooth=False, v_smooth=False)
    b = P.prep_head(q, k, v, None, cfg)
    tr = []
    o_q = A.emulate_head(b, cfg, rows=np.arange(N), p_format=A.P_EXP_E4M3, trace=tr).astype(np.float64)
    # rebuild P_q from the trace (rescale each tile's codes to the final maximum)
    m_fin = tr[-1]["m"].astype(np.float64)
    cols = [t["p_hat"] * np.exp2(t["m"].astype(np.float64) - m_fin)[:, None] for t in tr]
    pq = np.concatenate(cols, axis=1)
    pq /= pq.sum(axis=1, keepdims=True)
    vq = b["v_deq"][:N] * b["v_scale"].astype(np.float64)[None, :]
    s = q.astype(np.float64) @ k.astype(np.float64).T / np.sqrt(d)
    p = np.exp(s - s.max(1, keepdims=True)); p /= p.sum(1, keepdims=True)
    vv = v.astype(np.float64)
    lhs = p @ vv - pq @ vq
    rhs = (p - pq) @ vv + pq @ (vv - vq)
    assert np.abs(lhs - rhs).max() < 1e-12
    assert np.abs(pq @ vq - o_q).max() < 0.02 * np.abs(vv).max()      # o_q is that product, bf16-rounded


def test_inputs_are_reproducible_and_shaped():
    w = vc_inputs.WORKLOADS["c1"]
    a = vc_inputs.make_qkv(w)
    b = vc_inputs.make_qkv(w, heads=[1])
    assert a[0].shape == (1, 2, 1024, 128) and a[0].dtype == torch.bfloat16
    assert torch.equal(a[1][:, 1], b[1][:, 0])
    k = a[1][0, 0].float()
    assert k.mean(0).std() > 1.5                                          # channel offsets ~ N(0, 9)
    p = vc_inputs.random_perm(1, 2, 1024, 3)
    assert sorted(p[0, 1].tolist()) == list(range(1024))
    pk, _ = vc_kmeans_harness.kmeans_perm(a[2][0, 0], k=8)
    assert sorted(pk.tolist()) == list(range(1024))


def test_int8_qk_codes_follow_their_definition():
    """INT8 Q/K quantizer (Fig. 3): symmetric per-128-row scale amax/127, round to nearest even,
    checked element by element with Python's own round() on a block with exact ties."""
    from oracle import prep as OP
    rng = np.random.default_rng(3)
    x = rng.normal(size=(256, 16)).astype(np.float32)
    x[0, 0] = 4.0                                  # amax of block 0 -> code 127
    x[0, 1] = np.float32(4.0 * 2.5 / 127.0)        # lands (nearly) on a tie
    codes, scale, deq = OP.quantize_int8_blocks(x)
    assert codes.dtype == np.int8 and codes.min() >= -127 and codes.max() == 127
    for blk in range(2):
        amax = float(np.abs(x[128 * blk:128 * (blk + 1)]).max())
        assert scale[blk] == np.float32(amax) / np.float32(127.0)
        inv = np.float32(127.0) / np.float32(amax)
        for r in range(128 * blk, 128 * blk + 128, 17):
            for c in range(16):
                y = float(np.float32(x[r, c] * inv))
                assert codes[r, c] == max(-127, min(127, round(y)))      # Python rounds ties to even
    assert np.abs(deq - x).max() <= 0.5 * float(scale.max()) * (1 + 1e-6)
    z = np.zeros((128, 8), dtype=np.float32)
    c0, s0, _ = OP.quantize_int8_blocks(z)
    assert s0[0] == 1.0 and not c0.any()
