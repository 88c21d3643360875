"""Parity at the full sizes of the benchmark configurations, in the launch configuration
bench.py times (all heads in one call, k-means permutation), on what the oracle can compute
one by one: the preprocessing of sampled heads in full, and sampled query tiles (the ragged
last one included) against all keys of those heads."""
import numpy as np
import pytest
import torch

import paper_2609_15810_b200 as vc
import vc_inputs
from paper_2609_15810_b200.binding import Params, alloc_buffers
from oracle import attention as OA
from oracle import compare as CMP

import helpers as Hh

pytestmark = pytest.mark.gpu

CASES = [("c2", 8, "kmeans"), ("c3", 8, "kmeans"), ("c3", 4, "random"), ("c4", 4, "kmeans"),
         ("c5_d64_n4096", 8, "random"), ("c5_d64_n4096", 4, "random"), ("c5_d128_n16384", 8, "kmeans"),
         ("c3", 8, "group"),          # the permutation from vc_group, as bench.py runs it
         ("c2", 8, "kmeans-int8"),    # the INT8 Q K^T arrangement
         ("c4_2heads", 8, "random"),  # the longest sequence (929 key tiles, an odd count) at 8 bits
         ("c3", 4, "group-hybrid"),   # the hybrid 4-bit arrangement (ExpCast-FP8 P over 4-bit Q, K, V)
         ("c5_d64_n4096", 4, "random-hybrid"),
         ("c4_2heads", 4, "random-hybrid"),   # 929 key tiles through the FP8 x FP4 value product
         ("n262144", 8, "random")]            # 2048 key tiles: the longest sequence tested

vc_inputs.WORKLOADS.setdefault("n262144", vc_inputs.Workload("n262144", 1, 1, 262144, 128, (64, 64, 64), (8,), 1077, "field", False))
vc_inputs.WORKLOADS.setdefault("c4_2heads", vc_inputs.Workload("c4_2heads", 1, 2, 118800, 128, (33, 45, 80), (8,), 1044, "field", True))


@pytest.mark.parametrize("name,bits,perm_kind", CASES, ids=[f"{c[0]}-{c[1]}bit-{c[2]}" for c in CASES])
def test_fullsize_sampled_parity(name, bits, perm_kind):
    w = vc_inputs.WORKLOADS[name]
    q, k, v = vc_inputs.make_qkv(w, device="cuda")
    flags = vc.VC_FLAG_ALL | (vc.VC_FLAG_INT8_QK if perm_kind.endswith("int8") else 0)
    hybrid = perm_kind.endswith("hybrid")
    p = Params.make(w.B, w.H, w.N, w.d, w.grid, bits=bits, flags=flags,
                    p_format=vc.VC_P_EXPCAST_E4M3 if hybrid else vc.VC_P_DEFAULT)
    if perm_kind.startswith("group"):
        gwork = torch.empty(vc.vc_group_workspace_bytes(p), dtype=torch.uint8, device="cuda")
        cent = torch.zeros(w.B, w.H, 64, w.d, dtype=torch.float32, device="cuda")
        perm = torch.empty(w.B, w.H, w.N, dtype=torch.int32, device="cuda")
        vc.vc_group(p, v, 64, 2, False, cent, perm, gwork)
    elif perm_kind.startswith("kmeans"):
        perm = vc_inputs.kmeans_perm_all(v, iters=2)
    else:
        perm = vc_inputs.random_perm(w.B, w.H, w.N, w.seed, device="cuda")
    quant, work = alloc_buffers(p)
    o = torch.empty(w.B, w.H, w.N, w.d, dtype=torch.bfloat16, device="cuda")
    vc.vc_attn(p, q, k, v, perm, o, quant, work)
    vc.vc_poll_status(work)
    torch.cuda.synchronize()
    got = Hh.gpu_sections(p, quant)
    nb = (w.N + 127) // 128
    tiles = sorted({0, nb // 3, (2 * nb) // 3 + 1, nb - 1})
    rows = np.concatenate([np.arange(128 * t, min(128 * (t + 1), w.N)) for t in tiles])
    for (b, h) in [(0, 0), (w.B - 1, w.H - 1)]:
        ref, cfg = Hh.oracle_prep(p, q, k, v, perm, b, h)
        stats = Hh.check_prep_head(p, got, b * w.H + h, ref, what=f"{name} b{b} h{h}")
        o_ref = OA.emulate_head(ref, cfg, rows=rows, p_format=OA.P_EXPCAST if hybrid else None)
        vmax = float(v[b, h].float().abs().max())
        m = Hh.check_output(o[b, h].float().cpu().numpy()[rows], o_ref, vmax)
        print(name, bits, (b, h), stats, m)
