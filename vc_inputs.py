"""Seeded synthetic inputs shaped like the paper's video-DiT workloads.

This module serves both the CPU oracle and the CUDA path and holds none of the method's
arithmetic: it only draws Q, K, V (bf16) and uniformly random token permutations.  The paper measures on
tensors captured from Wan2.2 / HunyuanVideo runs; those are not available, so the
generator stands in for them with the structure the paper describes: Q/K outliers live in
a few channels shared by all tokens, V outliers sit in tokens and move with the block,
and tokens are spatiotemporally smooth (Sec. 3.1 "The value quantization bottleneck").

Every (tensor, batch, head, call) has its own generator seed, so any single head can be
regenerated on its own.  CPU and CUDA generators give different streams for the same
seed; a comparison must hand the *same buffers* to both sides.
"""
from dataclasses import dataclass
import math
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    N: int
    d: int
    grid: tuple            # (T, Hg, Wg), row-major t, y, x
    bits: tuple            # bit widths the config asks for
    seed: int
    kind: str              # "gauss" | "field"
    outliers: bool = False

    @property
    def flops(self):
        return 4.0 * self.B * self.H * float(self.N) ** 2 * self.d


WORKLOADS = {
    # tiny correctness case: the oracle finishes in seconds
    "c1": Workload("c1", 1, 2, 1024, 128, (4, 16, 16), (8,), 1001, "gauss"),
    # Wan-1.3B-shaped
    "c2": Workload("c2", 1, 12, 32760, 128, (21, 30, 52), (8,), 1002, "field"),
    # Wan-14B-shaped: the headline configuration
    "c3": Workload("c3", 1, 40, 32760, 128, (21, 30, 52), (8, 4), 1003, "field"),
    # HunyuanVideo-shaped long sequence with outlier channels
    "c4": Workload("c4", 1, 24, 118800, 128, (33, 45, 80), (4,), 1004, "field", True),
}
# mixed sweep for the roofline plot
for _d in (64, 128):
    for _n, _g in ((4096, (4, 32, 32)), (16384, (16, 32, 32)), (65536, (16, 64, 64))):
        WORKLOADS[f"c5_d{_d}_n{_n}"] = Workload(f"c5_d{_d}_n{_n}", 2, 16, _n, _d, _g, (8, 4), 1005, "field")


def _gen(device, *key):
    g = torch.Generator(device=device)
    s = 0x9E3779B97F4A7C15
    for k in key:
        s = (s * 6364136223846793005 + int(k) + 1442695040888963407) & ((1 << 63) - 1)
    g.manual_seed(s)
    return g


def _field(w, gen, device):
    """Sum of 8 random sinusoids over (t, y, x) per channel, unit variance: [N, d] fp32."""
    T, Hg, Wg = w.grid
    n = torch.arange(w.N, device=device)
    pos = torch.stack([(n // (Hg * Wg)).float() / T,
                       ((n // Wg) % Hg).float() / Hg,
                       (n % Wg).float() / Wg], dim=1)                        # [N, 3]
    f = torch.rand(w.d, 8, 3, generator=gen, device=device) * 2.0            # U(0, 2)
    phi = torch.rand(w.d, 8, generator=gen, device=device) * (2.0 * math.pi)
    out = torch.zeros(w.N, w.d, device=device)
    for k in range(8):                                                        # keeps memory at [N, d]
        arg = 2.0 * math.pi * (pos @ f[:, k, :].T) + phi[None, :, k]
        out += 0.5 * torch.sin(arg)
    return out


def make_head(w, tensor, b, h, call=0, device="cpu"):
    """One [N, d] bf16 tensor ('q', 'k' or 'v') of head (b, h).

    gauss: Q ~ N(0,1); K ~ N(0,1) + o_c, o_c ~ N(0, 3^2) per channel; V ~ N(0,1) + a
           N(0,1) shift per (128-token block in sequence order, channel).
    field: smooth field + N(0, 0.5^2) noise (the noise is redrawn per call, the field and
           the offsets are not), same K offsets and V block shifts.
    outliers: each channel of Q and, drawn separately, of K is an outlier channel with
           probability 0.01 (at least one per head); there every token gets + 10 * t_3.
    A list of calls returns the list of their tensors (the structure is drawn once).
    """
    tid = {"q": 0, "k": 1, "v": 2}[tensor]
    calls = list(call) if isinstance(call, (list, tuple)) else [call]
    g_struct = _gen(device, w.seed, tid, b, h, 0)           # structure: same on every call
    field = None if w.kind == "gauss" else _field(w, g_struct, device)
    offset = 3.0 * torch.randn(1, w.d, generator=g_struct, device=device) if tensor == "k" else None
    shift = None
    if tensor == "v":
        nb = (w.N + 127) // 128
        shift = torch.randn(nb, w.d, generator=g_struct, device=device).repeat_interleave(128, dim=0)[: w.N]
    mask = None
    if w.outliers and tensor in ("q", "k"):
        mask = torch.rand(w.d, generator=g_struct, device=device) < 0.01
        if not bool(mask.any()):
            mask[int(torch.randint(0, w.d, (1,), generator=g_struct, device=device))] = True
    out = []
    for c in calls:
        g_noise = _gen(device, w.seed, tid, b, h, 1, c)     # noise: redrawn per call
        x = torch.randn(w.N, w.d, generator=g_noise, device=device)
        if field is not None:
            x = field + 0.5 * x
        if offset is not None:
            x = x + offset
        if shift is not None:
            x = x + shift
        if mask is not None:
            z = torch.randn(w.N, w.d, generator=g_noise, device=device)
            chi = torch.randn(3, w.N, w.d, generator=g_noise, device=device).pow(2).sum(0) / 3.0
            x = x + mask[None, :].float() * 10.0 * z / chi.sqrt()
        out.append(x.to(torch.bfloat16))
    return out if isinstance(call, (list, tuple)) else out[0]


def make_qkv_calls(w, n_calls, device="cpu"):
    """[(Q, K, V)] for calls 0 .. n_calls-1 of the workload: what make_qkv(w, call) gives for each
    call, with the per-head structure (field, offsets, shifts, outlier channels: the same on every
    call) synthesised once instead of once per call."""
    out = [[torch.empty(w.B, w.H, w.N, w.d, dtype=torch.bfloat16, device=device) for _ in range(3)] for _ in range(n_calls)]
    for ti, tensor in enumerate(("q", "k", "v")):
        for b in range(w.B):
            for h in range(w.H):
                heads = make_head(w, tensor, b, h, list(range(n_calls)), device)
                for c in range(n_calls):
                    out[c][ti][b, h] = heads[c]
    return out


def make_qkv(w, call=0, device="cpu", heads=None):
    """Q, K, V as [B, H', N, d] bf16 where H' = len(heads) (default: all heads)."""
    heads = list(range(w.H)) if heads is None else list(heads)
    out = []
    for tensor in ("q", "k", "v"):
        t = torch.empty(w.B, len(heads), w.N, w.d, dtype=torch.bfloat16, device=device)
        for b in range(w.B):
            for i, h in enumerate(heads):
                t[b, i] = make_head(w, tensor, b, h, call, device)
        out.append(t)
    return out


# ----------------------------------------------------------------------------- permutations
def random_perm(B, H, N, seed, device="cpu"):
    g = _gen(device, seed, 77)
    p = torch.stack([torch.randperm(N, generator=g, device=device) for _ in range(B * H)])
    return p.reshape(B, H, N).to(torch.int32)
