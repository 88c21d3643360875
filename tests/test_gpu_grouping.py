"""vc_group (Sec. 3.2 "Value-guided permutation") through the C ABI against the grouping oracle.

Labels are integers decided by floating point: the CUDA path takes them from fp32 sums in its
own order, the oracle in fp64, so a token whose two nearest centroids are (almost) equally far
may legitimately land on either.  What is unique is compared exactly - the permutation must be
THE stable argsort of the labels the kernel chose, warm and cold runs must agree bit for bit,
and every label must be the oracle's wherever the oracle's margin is not tiny."""
import numpy as np
import pytest
import torch

import paper_2609_15810_b200 as vc
import vc_inputs
import vc_kmeans_harness
from paper_2609_15810_b200.binding import Params, alloc_buffers
from oracle import attention as OA
from oracle import grouping as OG

import helpers as Hh

pytestmark = pytest.mark.gpu

CASES = [  # name, B, H, N, d, grid, k
    ("n300_d64_k8", 1, 2, 300, 64, (3, 10, 10), 8),
    ("n1024_k64", 1, 2, 1024, 128, (4, 16, 16), 64),
    ("n2500_k17", 2, 2, 2500, 128, (4, 25, 25), 17),     # three chunks, the last one ragged
    ("n130_k1", 1, 1, 130, 128, (1, 10, 13), 1),
]


def _run(p, v, k, iters, warm=False, centroids=None):
    work = torch.empty(vc.vc_group_workspace_bytes(p), dtype=torch.uint8, device="cuda")
    if centroids is None:
        centroids = torch.zeros(p.B, p.H, k, p.d, dtype=torch.float32, device="cuda")
    perm = torch.empty(p.B, p.H, p.N, dtype=torch.int32, device="cuda")
    vc.vc_group(p, v, k, iters, warm, centroids, perm, work)
    torch.cuda.synchronize()
    off = vc.VC_GROUP_LABELS_OFFSET
    labels = work[off: off + p.B * p.H * p.N * 4].view(torch.int32).view(p.B, p.H, p.N).clone()
    vc.vc_poll_status(work)
    return perm, centroids, labels


def _blobby(B, H, N, d, k, seed):
    """Values with cluster structure: k centres per head plus noise, in random token order."""
    g = torch.Generator().manual_seed(seed)
    centres = torch.randn(B, H, k, d, generator=g) * 2.0
    which = torch.randint(0, k, (B, H, N), generator=g)
    v = torch.gather(centres, 2, which[..., None].expand(B, H, N, d)) + 0.5 * torch.randn(B, H, N, d, generator=g)
    return v.to(torch.bfloat16).cuda()


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_group_matches_oracle(case):
    _, B, H, N, d, grid, k = case
    v = _blobby(B, H, N, d, max(k, 2), seed=5)
    p = Params.make(B, H, N, d, grid)
    perm, cent, labels = _run(p, v, k, iters=3)
    for b in range(B):
        for h in range(H):
            x = v[b, h].float().cpu().numpy()
            lab_o, c_o, margin, _ = OG.kmeans(x, k, 3)
            lab_g = labels[b, h].cpu().numpy()
            scale = float((x * x).sum(axis=1).mean())
            clear = margin > 1e-3 * scale
            assert (lab_g[clear] == lab_o[clear]).all()
            assert (lab_g != lab_o).mean() < 0.01
            # the permutation is exactly the stable argsort of the kernel's own labels
            assert perm[b, h].cpu().numpy().tolist() == OG.stable_argsort(lab_g).tolist() or k == 1
            if k == 1:
                assert perm[b, h].cpu().numpy().tolist() == list(range(N))
            if (lab_g == lab_o).all():
                assert np.abs(cent[b, h].cpu().numpy() - c_o).max() < 1e-4 * max(1.0, np.abs(c_o).max())


def test_warm_start_continues_a_cold_run_bit_for_bit_and_runs_are_deterministic():
    B, H, N, d, grid, k = 1, 3, 3000, 128, (3, 25, 40), 32
    v = _blobby(B, H, N, d, k, seed=6)
    p = Params.make(B, H, N, d, grid)
    perm3, cent3, lab3 = _run(p, v, k, iters=3)
    perm3b, cent3b, _ = _run(p, v, k, iters=3)
    assert torch.equal(perm3, perm3b) and torch.equal(cent3, cent3b)
    _, cent2, _ = _run(p, v, k, iters=2)
    perm21, cent21, lab21 = _run(p, v, k, iters=1, warm=True, centroids=cent2.clone())
    assert torch.equal(lab21, lab3) and torch.equal(perm21, perm3) and torch.equal(cent21, cent3)


def test_group_then_attention_matches_the_oracle_with_that_permutation():
    """The permutation the kernel produces is a valid input of the hot path (config 1)."""
    w = vc_inputs.WORKLOADS["c1"]
    q, k, v = [t.cuda() for t in vc_inputs.make_qkv(w)]
    p = Params.make(w.B, w.H, w.N, w.d, w.grid, bits=8)
    perm, _, labels = _run(p, v, 8, iters=4)
    assert (torch.sort(perm.long(), dim=-1).values == torch.arange(w.N, device="cuda")).all()
    sorted_labels = torch.gather(labels.long(), 2, perm.long())
    assert (sorted_labels[..., 1:] >= sorted_labels[..., :-1]).all()
    quant, work = alloc_buffers(p)
    o = torch.empty(w.B, w.H, w.N, w.d, dtype=torch.bfloat16, device="cuda")
    vc.vc_attn(p, q, k, v, perm, o, quant, work)
    vc.vc_poll_status(work)
    vmax = float(v.float().abs().max())
    for h in range(w.H):
        bundle, cfg = Hh.oracle_prep(p, q, k, v, perm, 0, h)
        Hh.check_output(o[0, h].float().cpu().numpy(), OA.emulate_head(bundle, cfg), vmax)


def test_group_fullsize_config3_properties():
    """Wan-14B shape, field + noise values, k = 64, 4 iterations: properties that hold at any size,
    and agreement with the harness k-means (same algorithm, library matmuls, fp32)."""
    w = vc_inputs.WORKLOADS["c3"]
    v = vc_inputs.make_qkv(w, device="cuda", heads=range(3))[2]
    B, H = v.shape[0], v.shape[1]
    p = Params.make(B, H, w.N, w.d, w.grid)
    perm, cent, labels = _run(p, v, 64, iters=4)
    assert (torch.sort(perm.long(), dim=-1).values == torch.arange(w.N, device="cuda")).all()
    sl = torch.gather(labels.long(), 2, perm.long())
    assert (sl[..., 1:] >= sl[..., :-1]).all()
    same = sl[..., 1:] == sl[..., :-1]
    assert (perm[..., 1:][same] > perm[..., :-1][same]).all()          # stable inside a cluster
    for h in range(H):
        ref_perm, ref_c = vc_kmeans_harness.kmeans_perm(v[0, h], k=64, iters=4)
        x = v[0, h].float()
        obj_g = ((x - cent[0, h][labels[0, h].long()]) ** 2).sum()
        d2 = (x * x).sum(1, keepdim=True) - 2.0 * (x @ ref_c.T) + (ref_c * ref_c).sum(1)[None, :]
        obj_r = ((x - ref_c[d2.argmin(1)]) ** 2).sum()
        assert abs(float(obj_g) - float(obj_r)) < 2e-2 * float(obj_r)


def test_group_rejects_bad_arguments():
    p = Params.make(1, 1, 256, 128, (4, 8, 8))
    v = torch.zeros(1, 1, 256, 128, dtype=torch.bfloat16, device="cuda")
    work = torch.empty(vc.vc_group_workspace_bytes(p), dtype=torch.uint8, device="cuda")
    cent = torch.zeros(1, 1, 64, 128, device="cuda")
    perm = torch.empty(1, 1, 256, dtype=torch.int32, device="cuda")
    for k, iters in ((0, 1), (65, 1), (8, 0), (300, 1)):
        with pytest.raises(vc.VcError):
            vc.vc_group(p, v, k, iters, False, cent, perm, work)
