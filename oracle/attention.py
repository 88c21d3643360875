"""Exact attention and the emulated low-bit recurrence -- oracle side (test infrastructure).

* ``exact_attention``   O = softmax(Q K^T / sqrt(d)) V in fp64 (Sec. 3.1 "Online softmax",
                        first sentence), the textbook definition written out.
* ``recurrence``        the tiled online-softmax update of Eq. 1 with the V-Smooth mean
                        restoration of Eq. 6 and the probability formats of Sec. 3.3 /
                        App. A, tile by tile over 128 permuted keys, in the paper's order:
                        row maximum, alpha, probability code, numerator, normalizer.

Readings fixed by this build: the normalizer l and the per-tile row sum r_ij are sums of
the *decoded* probability codes (the same numbers that multiply the residual), so that
softmax-weights-sum-to-one holds exactly for the quantized row and P (V - mu) + mu = P V;
codes are taken relative to the running maximum after the current tile (no lazy
rescaling: with the row maximum at code 120 there is less than one binade of headroom);
ExpCast codes 1..7 decode as E4M3 subnormals, as the tensor core reads those bytes.
"""
import numpy as np

from . import codecs as C
from .prep import BLOCK

P_EXACT = "exact"            # quantization off (pins only)
P_EXPCAST = "expcast_e4m3"   # Eq. 7
P_EXP_E4M3 = "exp_e4m3"      # exponentiate, then cast (Fig. 4a upper box)
P_NVFP4 = "nvfp4"            # App. A "Scope of ExpCast-FP8": E2M1 under a per-16 E4M3 microscale

LOG2E = 1.4426950408889634
NVFP4_P_SCALE = 6.0 * C.E4M3_MAX   # the row maximum maps to 6 * 448 so the top microscale is 448


def exact_attention(q, k, v, scale=None, rows=None):
    """fp64 attention for one head.  q,k,v: [N, d] (already rotated if RoPE applies)."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    if rows is not None:
        q = q[rows]
    if scale is None:
        scale = 1.0 / np.sqrt(q.shape[1])
    s = (q @ k.T) * scale
    s = s - s.max(axis=1, keepdims=True)
    p = np.exp(s)
    p = p / p.sum(axis=1, keepdims=True)
    return p @ v


def probability_codes(u, p_format, beta):
    """One tile of log2-domain scores u = z - m' (<= 0) -> decoded probabilities p_hat."""
    if p_format == P_EXPCAST:
        return C.e4m3_decode(C.expcast_code(u, beta))
    if p_format == P_EXP_E4M3:
        return C.e4m3_decode(C.exp_then_cast_code(u))
    if p_format == P_NVFP4:
        p = (np.exp2(u.astype(np.float64)) * NVFP4_P_SCALE).astype(np.float32)
        _, _, deq = C.nvfp4_quantize_groups(p)       # groups of 16 keys along the row
        return deq
    if p_format == P_EXACT:
        return np.exp2(np.asarray(u, dtype=np.float64))
    raise ValueError(p_format)


def recurrence(q_deq, k_deq, v_deq, v_means, n_valid, score_scale, p_format,
               beta=C.EXPCAST_BETA, rows=None, exact=False, tile=BLOCK, trace=None):
    """Eq. 1 + Eq. 6 for one head.

    q_deq   [n_pad, d]  decoded Q operand WITHOUT its per-block scale (code units)
    k_deq   [n_pad, d]  decoded permuted K operand, code units
    v_deq   [n_pad, d]  decoded residual R_q, code units (x s_V happens in the epilogue)
    v_means [n_blocks, d] block means in the same units as v_deq (0 if V-Smooth is off)
    n_valid             number of real keys; keys >= n_valid are padding and are excluded
    score_scale         callable (q_block, k_block) -> fp32 factor turning the code-unit
                        dot product into the log2-domain score z (folds s_Q s_K / sqrt(d)
                        and log2 e), or a scalar
    rows                query rows to evaluate (default: all n_valid)
    exact               all arithmetic in fp64, nothing rounded (pins)
    Returns A / l as fp64 [len(rows), d] (no epilogue scale, no bf16 rounding).
    """
    wt = np.float64 if exact else np.float32
    n_pad, d = k_deq.shape
    assert n_pad % tile == 0
    rows = np.arange(n_valid) if rows is None else np.asarray(rows)
    Q = np.asarray(q_deq, dtype=np.float64)[rows]
    qblk = rows // BLOCK
    R = len(rows)
    m = np.full(R, -np.inf, dtype=wt)
    l = np.zeros(R, dtype=wt)
    A = np.zeros((R, d), dtype=wt)
    for j in range(n_pad // tile):
        ks = slice(j * tile, (j + 1) * tile)
        nv = min(tile, n_valid - j * tile)
        if nv <= 0:
            break
        s_acc = (Q @ np.asarray(k_deq[ks], dtype=np.float64).T).astype(wt)
        if callable(score_scale):
            c = np.array([score_scale(b, (j * tile) // BLOCK) for b in qblk], dtype=wt)
        else:
            c = np.full(R, score_scale, dtype=wt)
        z = (s_acc * c[:, None]).astype(wt)                       # log2-domain scores
        z_valid = z[:, :nv]
        m_new = np.maximum(m, z_valid.max(axis=1)).astype(wt)     # m' = max(m, rowmax S_ij)
        alpha = np.exp2(m.astype(np.float64) - m_new.astype(np.float64)).astype(wt)
        u = (z - m_new[:, None]).astype(wt)
        p_hat = np.array(probability_codes(u, p_format, beta), dtype=np.float64)
        p_hat[:, nv:] = 0.0                                       # padded keys carry code 0
        r = p_hat.sum(axis=1)                                     # r_ij = P~_ij 1  (Eq. 6)
        mu = np.asarray(v_means[(j * tile) // BLOCK], dtype=np.float64)
        upd = (alpha.astype(np.float64)[:, None] * A.astype(np.float64)
               + p_hat @ np.asarray(v_deq[ks], dtype=np.float64)
               + r[:, None] * mu[None, :])
        A = upd.astype(wt)                                        # A <- a A + P R + r mu^T
        l = (alpha.astype(np.float64) * l.astype(np.float64) + r).astype(wt)
        m = m_new
        if trace is not None:
            trace.append({"j": j, "m": m.copy(), "alpha": alpha.copy(), "r": r.copy(),
                          "p_hat": p_hat.copy(), "u": u.copy()})
    return A.astype(np.float64) / l.astype(np.float64)[:, None]


def emulate_head(bundle, cfg, p_format=None, softmax_scale=None, beta=C.EXPCAST_BETA,
                 rows=None, trace=None):
    """O1 for one head from the oracle's prep bundle: the recurrence plus the epilogue.

    8-bit:  z = S_acc * (s_Q[i-block] * s_K[j]) * (scale * log2 e);  O = bf16(s_V * A / l)
    4-bit:  z = S_acc * (g_Q * g_K) * (scale * log2 e) with the microscales inside the
            decoded operands;  O = bf16(A / l)  (means added unscaled, App. B)
    """
    d = cfg.d
    if softmax_scale is None:
        softmax_scale = 1.0 / np.sqrt(d)
    sl = np.float32(softmax_scale * LOG2E)
    if cfg.bits == 8:
        p_format = p_format or P_EXPCAST
        sq, sk = bundle["q_scale"], bundle["k_scale"]
        scale_fn = lambda bq, bk: np.float32(np.float32(sq[bq] * sk[bk]) * sl)
        if cfg.qk_format == "int8":
            q_deq, k_deq = bundle["q_codes"].astype(np.float64), bundle["k_codes"].astype(np.float64)
        else:
            q_deq, k_deq = C.e4m3_decode(bundle["q_codes"]), C.e4m3_decode(bundle["k_codes"])
    elif cfg.bits == 4:
        p_format = p_format or P_NVFP4
        scale_fn = float(np.float32(np.float32(bundle["q_g"] * bundle["k_g"]) * sl))
        q_deq = bundle["q_deq"] / float(bundle["q_g"])
        k_deq = bundle["k_deq"] / float(bundle["k_g"])
    else:
        raise ValueError("emulate_head needs a quantized bundle; use recurrence(exact=True)")
    a_over_l = recurrence(q_deq, k_deq, bundle["v_deq"], bundle["v_means"], cfg.N, scale_fn,
                          p_format, beta=beta, rows=rows, trace=trace)
    o = (a_over_l.astype(np.float32) * bundle["v_scale"].astype(np.float32)[None, :]).astype(np.float32)
    return C.bf16_round(o)


def reference_scores(q, k, cfg, row, softmax_scale=None):
    """Exact fp64 scores (natural-log domain) of one query row of the rotated Q against all rotated
    keys: what the softmax of Sec. 3.1 sees (a diagnostic: effective keys 1 / sum p^2 of a row)."""
    from .prep import rope_tables
    q = np.asarray(q, dtype=np.float64)[row:row + 1]
    k = np.asarray(k, dtype=np.float64)
    if cfg.rope:
        cos, sin = rope_tables(cfg)
        def rot(x, c, s):
            out = np.empty_like(x)
            out[:, 0::2] = x[:, 0::2] * c - x[:, 1::2] * s
            out[:, 1::2] = x[:, 0::2] * s + x[:, 1::2] * c
            return out
        q, k = rot(q, cos[row:row + 1], sin[row:row + 1]), rot(k, cos, sin)
    scale = 1.0 / np.sqrt(q.shape[1]) if softmax_scale is None else softmax_scale
    return (q @ k.T)[0] * scale


def reference_head(q, k, v, cfg, rows=None, softmax_scale=None):
    """O0: exact fp64 attention of the rotated Q, K (no permutation, smoothing or
    Hadamard: each of them leaves the exact output unchanged)."""
    from .prep import rope_tables, rope_apply
    q = np.asarray(q, dtype=np.float32)
    k = np.asarray(k, dtype=np.float32)
    if cfg.rope:
        cos, sin = rope_tables(cfg)
        # rotate in fp64 without the fp32 rounding of the pipeline
        def rot(x):
            x = x.astype(np.float64)
            out = np.empty_like(x)
            out[:, 0::2] = x[:, 0::2] * cos - x[:, 1::2] * sin
            out[:, 1::2] = x[:, 0::2] * sin + x[:, 1::2] * cos
            return out
        q, k = rot(q), rot(k)
    return exact_attention(q, k, v, scale=softmax_scale, rows=rows)
