"""Synthetic analogues of the paper's value-side analysis -- CPU, TEST INFRASTRUCTURE.

The paper measures these quantities on tensors captured from video models; here the same
definitions are evaluated on whatever value tensor is handed in (the harness passes
synthetic ones), so only the SHAPE of the findings can be compared, never the numbers.

* value_rmse            Table "token order" (Sec. 3.2): relative squared error of the value
                        operand after block demeaning (Eq. 4) and per-channel E4M3
                        quantization, for a given token order, with or without a Hadamard
                        rotation of the value channels
* energy_share_removed  the share of a block's energy its mean removes (Eq. 5), block average
* error_decomposition   Eq. 2:  O - O_q = (P - P_q) V + P_q (V - V_q)
* token orders          sequence, static cube (a fixed 4 x 2 x 16 spatiotemporal brick per
                        128-token block), k-means (oracle.grouping)

All arithmetic in fp64; the quantizer is the one of oracle.prep / oracle.codecs.
"""
import numpy as np

from . import codecs as C
from . import grouping as G
from .prep import BLOCK, hadamard_apply


def sequence_order(n):
    return np.arange(n, dtype=np.int64)


def static_cube_order(grid, cube=(4, 2, 16)):
    """Tokens of a (T, H, W) grid regrouped into bricks of cube[0] x cube[1] x cube[2] tokens
    (128 with the default), bricks in raster order, tokens inside a brick in raster order.
    Ragged edges simply give smaller bricks; the order is a permutation either way."""
    T, H, W = grid
    t, y, x = np.meshgrid(np.arange(T), np.arange(H), np.arange(W), indexing="ij")
    key = np.stack([t // cube[0], y // cube[1], x // cube[2], t, y, x], axis=-1).reshape(-1, 6)
    return np.lexsort(key.T[::-1]).astype(np.int64)


def kmeans_order(v, k=64, iters=4):
    labels, _, _, _ = G.kmeans(np.asarray(v, dtype=np.float64), k, iters)
    return G.stable_argsort(labels)


def _blocks(x):
    n, d = x.shape
    n_pad = BLOCK * ((n + BLOCK - 1) // BLOCK)
    xp = np.zeros((n_pad, d), dtype=np.float64)
    xp[:n] = x
    valid = (np.arange(n_pad) < n).reshape(-1, BLOCK)
    return xp.reshape(-1, BLOCK, d), valid


def energy_share_removed(v, order):
    """Mean over blocks of B ||mu_j||^2 / ||V'_j||_F^2 (Eq. 5), valid rows only."""
    xb, valid = _blocks(np.asarray(v, dtype=np.float64)[order])
    shares = []
    for blk, ok in zip(xb, valid):
        rows = blk[ok]
        mu = rows.mean(axis=0)
        total = float((rows * rows).sum())
        if total > 0:
            shares.append(rows.shape[0] * float(mu @ mu) / total)
    return float(np.mean(shares))


def value_rmse(v, order, demean=True, hadamard=False):
    """|| V' - V'_q ||_F^2 / || V' ||_F^2 of the value operand under `order`: block means
    removed (Eq. 4), residual quantized to E4M3 with one scale per channel, means kept in
    bf16 (App. B), everything put back together.  `hadamard` rotates the value channels first
    and back afterwards (the alternative the paper's table prices)."""
    x = np.asarray(v, dtype=np.float64)[order]
    if hadamard:
        x = hadamard_apply(x.astype(np.float32)).astype(np.float64)
    xb, valid = _blocks(x)
    mu = np.zeros((xb.shape[0], x.shape[1]))
    if demean:
        for j, (blk, ok) in enumerate(zip(xb, valid)):
            mu[j] = blk[ok].mean(axis=0)
    res = (xb - mu[:, None, :]) * valid[:, :, None]
    amax = np.abs(res).max(axis=(0, 1))
    scale = np.where(amax > 0, amax / C.E4M3_MAX, 1.0)
    codes = C.e4m3_encode((res / scale).astype(np.float32))
    mu_q = C.bf16_round((mu / scale).astype(np.float32)).astype(np.float64) * scale
    rec = (C.e4m3_decode(codes) * scale + mu_q[:, None, :]) * valid[:, :, None]
    err = float(((rec - xb * valid[:, :, None]) ** 2).sum())
    return err / float((x * x).sum())


def error_decomposition(p, p_q, v, v_q):
    """Eq. 2.  Returns (O - O_q, (P - P_q) V, P_q (V - V_q)); the first equals the sum of the
    other two identically."""
    p, p_q, v, v_q = (np.asarray(a, dtype=np.float64) for a in (p, p_q, v, v_q))
    return p @ v - p_q @ v_q, (p - p_q) @ v, p_q @ (v - v_q)


def report(v, grid, k=64, iters=4):
    """The analogue of the paper's token-order table for one value tensor [N, d]."""
    n = v.shape[0]
    orders = {"sequence": sequence_order(n), "static cube 4x2x16": static_cube_order(grid),
              "k-means": kmeans_order(v, k, iters)}
    rows = [("sequence", value_rmse(v, orders["sequence"]), energy_share_removed(v, orders["sequence"])),
            ("Hadamard on V", value_rmse(v, orders["sequence"], hadamard=True), energy_share_removed(v, orders["sequence"]))]
    for name in ("static cube 4x2x16", "k-means"):
        rows.append((name, value_rmse(v, orders[name]), energy_share_removed(v, orders[name])))
    return rows
