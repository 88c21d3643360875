"""Parity at the full sizes of the benchmark configurations, in the launch configuration
bench.py times (all heads in one call, k-means permutation), on what the oracle can compute
one by one: the preprocessing of sampled heads in full, and sampled query tiles (the ragged
last one included) against all keys of those heads."""
import numpy as np
import pytest
import torch

import paper_2609_15810_b200 as vc
import vc_inputs
import vc_kmeans_harness
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
         ("n262144", 8, "random"),            # 2048 key tiles: the longest sequence tested
         # the rest of the mixed sweep: the longest sequences at both head dimensions and all three
         # arrangements (sampled tiles of one head keep the oracle within seconds), and the middle
         # size at 4 bits
         ("c5_d64_n65536", 8, "random"), ("c5_d64_n65536", 4, "random"), ("c5_d64_n65536", 4, "random-hybrid"),
         ("c5_d128_n65536", 8, "group"), ("c5_d128_n65536", 4, "random"), ("c5_d128_n65536", 4, "group-hybrid"),
         ("c5_d128_n16384", 4, "random"), ("c5_d64_n16384", 8, "random"), ("c5_d128_n4096", 4, "random-hybrid")]

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
        perm = vc_kmeans_harness.kmeans_perm_all(v, iters=2)
    else:
        perm = vc_inputs.random_perm(w.B, w.H, w.N, w.seed, device="cuda")
    quant, work = alloc_buffers(p)
    o = torch.empty(w.B, w.H, w.N, w.d, dtype=torch.bfloat16, device="cuda")
    vc.vc_attn(p, q, k, v, perm, o, quant, work)
    vc.vc_poll_status(work)
    torch.cuda.synchronize()
    got = Hh.gpu_sections(p, quant)
    nb = (w.N + 127) // 128
    long_case = w.N >= 65536 and w.B * w.H > 2
    tiles = sorted({0, (2 * nb) // 3 + 1, nb - 1}) if long_case else sorted({0, nb // 3, (2 * nb) // 3 + 1, nb - 1})
    rows = np.concatenate([np.arange(128 * t, min(128 * (t + 1), w.N)) for t in tiles])
    for (b, h) in ([(w.B - 1, w.H - 1)] if long_case else [(0, 0), (w.B - 1, w.H - 1)]):
        ref, cfg = Hh.oracle_prep(p, q, k, v, perm, b, h)
        stats = Hh.check_prep_head(p, got, b * w.H + h, ref, what=f"{name} b{b} h{h}")
        o_ref = OA.emulate_head(ref, cfg, rows=rows, p_format=OA.P_EXPCAST if hybrid else None)
        vmax = float(v[b, h].float().abs().max())
        o_got = o[b, h].float().cpu().numpy()[rows]
        m = Hh.check_output(o_got, o_ref, vmax)
        # what the acceptance asks to be reported beside pass / fail: how many elements are over the
        # tolerance (none may be), and how peaked the rows with the largest deviation are
        err = np.abs(o_got - o_ref).max(axis=1)
        worst = rows[np.argsort(err)[-4:]]
        qh, kh = q[b, h].float().cpu().numpy(), k[b, h].float().cpu().numpy()
        eff = []
        for r_ in worst:
            sc = OA.reference_scores(qh, kh, cfg, int(r_))
            pr = np.exp(sc - sc.max()); pr /= pr.sum()
            eff.append(float(1.0 / (pr ** 2).sum()))
        n_over = int((np.abs(o_got - o_ref) > 2e-2 * vmax).sum())
        assert n_over == 0
        print(name, bits, (b, h), stats, m, {"elements_over_tolerance": n_over, "rows_checked": len(rows),
                                            "worst_rows": worst.tolist(), "worst_rows_max_err_over_vmax": (np.sort(err)[-4:] / vmax).tolist(),
                                            "worst_rows_effective_keys": eff})
