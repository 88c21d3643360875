"""The preprocessing chain of VC-Attention -- oracle side (test infrastructure only).

Per (batch, head), following Sec. 3.4 "Fused preprocessing" and App. B "Fused
Preprocessing, Operand by Operand":

  Q : RoPE -> Hadamard rotation -> quantize
  K : RoPE -> channel mean over all tokens -> gather by pi -> subtract mean ->
      Hadamard rotation -> pad -> quantize
  V : gather by pi -> pad -> per-128-token block mean (Eq. 4) -> residual -> quantize,
      block means written next to the residual codes (divided by the per-channel value
      scale at 8 bits, unscaled at 4 bits)

Rule for precision: a stage is evaluated in fp64 from fp32 inputs and its output is
rounded once to fp32; the operations that decide an integer code (the multiplication by
the reciprocal scale and the rounding to the code grid) are single IEEE fp32 operations,
spelled out below, so that an fp32 implementation can take the same decision.

Readings fixed by this build where the paper is silent (listed in the design document):
RoPE is a 3-axis (t, y, x) rotary embedding on interleaved channel pairs; Q/K 8-bit
scales are one per 128-row block; the 8-bit V scale is one per channel over all tokens;
NVFP4 groups run along the contraction axis (channels for Q/K, tokens for V); the NVFP4
outer scale of Q/K is one fp32 per (batch, head), V has none.
"""
from dataclasses import dataclass, field
import numpy as np

from . import codecs as C

BLOCK = 128   # B_v of Eq. 4, and the row block of the Q/K scales


@dataclass
class PrepConfig:
    N: int
    d: int
    grid: tuple                      # (T, Hg, Wg), T*Hg*Wg == N, row-major t, y, x
    bits: int = 8                    # 8 or 4; 0 = no quantization (pins only)
    rope: bool = True
    hadamard: bool = True
    k_smooth: bool = True
    v_smooth: bool = True
    rope_dims: tuple = None          # channels per axis, sum == d
    rope_theta: float = 10000.0
    qk_format: str = "e4m3"          # 8-bit Q/K codes: "e4m3", or "int8" (the INT8 Q K^T of Fig. 3)
    v_format: str = "nvfp4"          # 4-bit V codes: "nvfp4" (E4M3 factor per 16 tokens), or "mxfp4"
                                     # (power-of-two factor per 32 tokens: the hybrid arrangement,
                                     # ExpCast-FP8 P times 4-bit values)

    def __post_init__(self):
        if self.rope_dims is None:
            self.rope_dims = default_rope_dims(self.d)
        assert sum(self.rope_dims) == self.d and all(x % 2 == 0 for x in self.rope_dims)
        assert self.grid[0] * self.grid[1] * self.grid[2] == self.N

    @property
    def n_pad(self):
        return BLOCK * ((self.N + BLOCK - 1) // BLOCK)

    @property
    def n_blocks(self):
        return self.n_pad // BLOCK


def default_rope_dims(d):
    """Channel split over (t, y, x) used by the harness: d - 4*(d//6), 2*(d//6), 2*(d//6)."""
    s = 2 * (d // 6)
    return (d - 2 * s, s, s)


# ----------------------------------------------------------------------------- RoPE
def rope_tables(cfg):
    """cos/sin [N, d/2] in fp32 (computed in fp64, rounded once).

    Pair p rotates channels (2p, 2p+1).  The first d_t/2 pairs follow the t coordinate,
    the next d_y/2 the y coordinate, the rest x; pair i of an axis with d_a channels has
    frequency theta^(-2i/d_a).  Token n sits at (n // (Hg*Wg), (n // Wg) % Hg, n % Wg).
    """
    T, Hg, Wg = cfg.grid
    n = np.arange(cfg.N, dtype=np.int64)
    pos = (n // (Hg * Wg), (n // Wg) % Hg, n % Wg)
    cols = []
    for axis, d_a in enumerate(cfg.rope_dims):
        i = np.arange(d_a // 2, dtype=np.float64)
        freq = np.power(float(cfg.rope_theta), -2.0 * i / d_a)
        cols.append(pos[axis][:, None].astype(np.float64) * freq[None, :])
    phi = np.concatenate(cols, axis=1)
    return np.cos(phi).astype(np.float32), np.sin(phi).astype(np.float32)


def rope_apply(x, cos, sin):
    """(x0, x1) -> (x0 c - x1 s, x0 s + x1 c) on interleaved pairs; fp64 inside, fp32 out."""
    x = np.asarray(x, dtype=np.float64)
    x0, x1 = x[:, 0::2], x[:, 1::2]
    c, s = cos.astype(np.float64), sin.astype(np.float64)
    out = np.empty_like(x)
    out[:, 0::2] = x0 * c - x1 * s
    out[:, 1::2] = x0 * s + x1 * c
    return out.astype(np.float32)


# ----------------------------------------------------------------------------- Hadamard
def hadamard_matrix(d):
    """Sylvester construction, natural order: H_1 = [1], H_2n = [[H, H], [H, -H]]."""
    H = np.array([[1]], dtype=np.int64)
    while H.shape[0] < d:
        H = np.block([[H, H], [H, -H]])
    assert H.shape[0] == d, "head dimension must be a power of two"
    return H


def hadamard_apply(x):
    """X H_d / sqrt(d); fp64 inside, fp32 out."""
    d = x.shape[-1]
    H = hadamard_matrix(d).astype(np.float64)
    return ((np.asarray(x, dtype=np.float64) @ H) / np.sqrt(float(d))).astype(np.float32)


# ----------------------------------------------------------------------------- helpers
def pad_rows(x, n_pad):
    out = np.zeros((n_pad,) + x.shape[1:], dtype=x.dtype)
    out[: x.shape[0]] = x
    return out


def quantize_e4m3_blocks(x):
    """Per block of 128 rows: s = amax/448 (1 if amax = 0); code = E4M3(x * (448/amax)).

    x: [n_pad, d] fp32.  Returns (codes u8, scales fp32 [n_blocks], dequantized fp64).
    """
    n_pad, d = x.shape
    xb = x.reshape(n_pad // BLOCK, BLOCK * d)
    amax = np.max(np.abs(xb), axis=1).astype(np.float32)
    f448 = np.float32(C.E4M3_MAX)
    with np.errstate(divide="ignore", invalid="ignore"):
        scale = np.where(amax > 0, (amax / f448).astype(np.float32), np.float32(1.0))
        inv = np.where(amax > 0, (f448 / amax).astype(np.float32), np.float32(0.0))
    y = (xb * inv[:, None]).astype(np.float32)
    codes = C.e4m3_encode(y).reshape(n_pad, d)
    deq = C.e4m3_decode(codes) * np.repeat(scale.astype(np.float64), BLOCK)[:, None]
    return codes, scale.astype(np.float32), deq


def quantize_int8_blocks(x):
    """INT8 Q/K codes (Fig. 3: INT8 Q K^T, FP8 softmax output, FP8 P V).  The paper gives no
    scale convention; taken here: symmetric, per block of 128 rows s = amax/127 (1 if amax = 0),
    code = round-to-nearest-even(x * (127/amax)) clamped to [-127, 127].

    x: [n_pad, d] fp32.  Returns (codes int8, scales fp32 [n_blocks], dequantized fp64).
    """
    n_pad, d = x.shape
    xb = x.reshape(n_pad // BLOCK, BLOCK * d)
    amax = np.max(np.abs(xb), axis=1).astype(np.float32)
    f127 = np.float32(127.0)
    with np.errstate(divide="ignore", invalid="ignore"):
        scale = np.where(amax > 0, (amax / f127).astype(np.float32), np.float32(1.0))
        inv = np.where(amax > 0, (f127 / amax).astype(np.float32), np.float32(0.0))
    y = (xb * inv[:, None]).astype(np.float32)
    codes = np.clip(np.rint(y.astype(np.float64)), -127, 127).astype(np.int8).reshape(n_pad, d)   # rint: ties to even
    deq = codes.astype(np.float64) * np.repeat(scale.astype(np.float64), BLOCK)[:, None]
    return codes, scale.astype(np.float32), deq


# ----------------------------------------------------------------------------- operands
def prep_q(q, cfg, cos=None, sin=None):
    """Q: RoPE, Hadamard, pad, quantize (App. B).  q: [N, d] fp32 holding bf16 values."""
    x = np.asarray(q, dtype=np.float32)
    if cfg.rope:
        x = rope_apply(x, cos, sin)
    if cfg.hadamard:
        x = hadamard_apply(x)
    x = pad_rows(x, cfg.n_pad)
    return _quantize_qk(x, cfg, "q")


def prep_k(k, perm, cfg, cos=None, sin=None):
    """K: RoPE at the original positions, channel mean over all tokens, gather by pi,
    mean subtraction, Hadamard, pad, quantize (App. B).  The mean is taken after RoPE:
    only a token-independent vector shifts every score of a row by the same constant."""
    x = np.asarray(k, dtype=np.float32)
    if cfg.rope:
        x = rope_apply(x, cos, sin)
    if cfg.k_smooth:
        k_mean = (x.astype(np.float64).sum(axis=0) / cfg.N).astype(np.float32)
    else:
        k_mean = np.zeros(cfg.d, dtype=np.float32)
    x = x[perm]                                                   # K' = K[pi]  (Eq. 3)
    x = (x.astype(np.float64) - k_mean.astype(np.float64)).astype(np.float32)
    if cfg.hadamard:
        x = hadamard_apply(x)
    x = pad_rows(x, cfg.n_pad)
    out = _quantize_qk(x, cfg, "k")
    out["k_mean"] = k_mean
    return out


def _quantize_qk(x, cfg, name):
    out = {name + "_pre": x}                   # the high-precision operand, for diagnostics
    if cfg.bits == 8:
        codes, scale, deq = quantize_int8_blocks(x) if cfg.qk_format == "int8" else quantize_e4m3_blocks(x)
        out.update({name + "_codes": codes, name + "_scale": scale, name + "_deq": deq})
    elif cfg.bits == 4:
        amax = np.float32(np.max(np.abs(x)))
        g = (amax / np.float32(6.0 * C.E4M3_MAX)).astype(np.float32) if amax > 0 else np.float32(1.0)
        codes, micro, deq = C.nvfp4_quantize_groups(x, outer_scale=g)
        out.update({name + "_codes": codes, name + "_micro": micro, name + "_g": np.float32(g),
                    name + "_deq": deq * float(g)})
    else:                                       # quantization off
        out.update({name + "_deq": x.astype(np.float64)})
    return out


def prep_v(v, perm, cfg):
    """V: gather by pi, pad, block means, residual, quantize, scaled means (Eq. 4, App. B).

    A partial last block divides by its number of valid rows and its padding rows have a
    zero residual.
    """
    x = np.asarray(v, dtype=np.float32)[perm]                     # V' = V[pi]  (Eq. 3)
    x = pad_rows(x, cfg.n_pad)
    nb, d = cfg.n_blocks, cfg.d
    valid = (np.arange(cfg.n_pad) < cfg.N)
    n_valid = valid.reshape(nb, BLOCK).sum(axis=1)
    if cfg.v_smooth:
        mu = (x.astype(np.float64).reshape(nb, BLOCK, d).sum(axis=1)
              / n_valid[:, None]).astype(np.float32)              # mu_j  (Eq. 4)
    else:
        mu = np.zeros((nb, d), dtype=np.float32)
    # Eq. 6 restores exactly what Eq. 4 subtracted only if the two means are the same number.  At 4
    # bits the mean is stored as bf16 and added back unscaled (App. B), so the mean that is
    # subtracted is that bf16 value.  (At 8 bits the stored mean is bf16(mu / s_V), restored as
    # s_V times that: it differs from mu by at most 2^-9 |mu|, a constant offset per block that the
    # probabilities, which sum to one, pass straight to the output; pinned in the tests.)
    mu_sub = C.bf16_round(mu) if cfg.bits == 4 else mu
    r = (x.astype(np.float64) - np.repeat(mu_sub.astype(np.float64), BLOCK, axis=0)).astype(np.float32)
    r = np.where(valid[:, None], r, np.float32(0.0))              # R_j  (Eq. 4)
    out = {"v_pre": r, "v_mu": mu}
    if cfg.bits == 8:
        amax = np.max(np.abs(r), axis=0).astype(np.float32)       # per channel, all tokens
        f448 = np.float32(C.E4M3_MAX)
        with np.errstate(divide="ignore", invalid="ignore"):
            scale = np.where(amax > 0, (amax / f448).astype(np.float32), np.float32(1.0))
            inv = np.where(amax > 0, (f448 / amax).astype(np.float32), np.float32(0.0))
        codes = C.e4m3_encode((r * inv[None, :]).astype(np.float32))
        means = C.bf16_round((mu * inv[None, :]).astype(np.float32))   # stored / s_V  (App. B)
        means = np.where(amax[None, :] > 0, means, C.bf16_round(mu))
        out.update({"v_codes": codes, "v_scale": scale, "v_means": means,
                    "v_deq": C.e4m3_decode(codes)})                # in code units; x s_V in the epilogue
    elif cfg.bits == 4:
        # groups of 16 consecutive permuted tokens per channel: quantize the transpose
        # (nvfp4), or of 32 under a power-of-two factor (mxfp4)
        quant = C.mxfp4_quantize_groups if cfg.v_format == "mxfp4" else C.nvfp4_quantize_groups
        codes_t, micro_t, deq_t = quant(np.ascontiguousarray(r.T))
        out.update({"v_codes": np.ascontiguousarray(codes_t.T),    # [n_pad, d]
                    "v_micro": np.ascontiguousarray(micro_t.T),    # [n_pad/16, d] (mxfp4: [n_pad/32, d])
                    "v_means": C.bf16_round(mu),                   # unscaled  (App. B)
                    "v_scale": np.ones(d, dtype=np.float32),
                    "v_deq": np.ascontiguousarray(deq_t.T)})
    else:
        out.update({"v_means": mu.astype(np.float64), "v_scale": np.ones(d), "v_deq": r.astype(np.float64)})
        if cfg.v_smooth:                          # exact arithmetic for the pins
            mu64 = x.astype(np.float64).reshape(nb, BLOCK, d).sum(axis=1) / n_valid[:, None]
            r64 = np.where(valid[:, None], x.astype(np.float64) - np.repeat(mu64, BLOCK, axis=0), 0.0)
            out.update({"v_means": mu64, "v_deq": r64})
    return out


def prep_head(q, k, v, perm, cfg):
    """The whole chain for one (batch, head).  perm=None means the identity."""
    if perm is None:
        perm = np.arange(cfg.N)
    perm = np.asarray(perm, dtype=np.int64)
    assert np.array_equal(np.sort(perm), np.arange(cfg.N)), "perm must be a permutation"
    cos = sin = None
    if cfg.rope:
        cos, sin = rope_tables(cfg)
    out = {}
    out.update(prep_q(q, cfg, cos, sin))
    out.update(prep_k(k, perm, cfg, cos, sin))
    out.update(prep_v(v, perm, cfg))
    return out
