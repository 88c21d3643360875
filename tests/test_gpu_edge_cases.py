"""Edge and degenerate cases of the CUDA path against the oracle: the shortest sequences,
stage switches end to end, non-default softmax scale and ExpCast offset, and inputs that make
a scale degenerate (all-zero V, constant K, constant V)."""
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


def _params(B, H, N, d, grid, bits, **kw):
    """bits = "4-hybrid" selects the hybrid 4-bit arrangement (ExpCast-FP8 P over 4-bit Q, K, V)."""
    if bits == "4-hybrid":
        return Params.make(B, H, N, d, grid, bits=4, p_format=vc.VC_P_EXPCAST_E4M3, **kw)
    return Params.make(B, H, N, d, grid, bits=bits, **kw)


def _run(p, q, k, v, perm, softmax_scale=None, beta=None, p_format=None):
    if p_format is None and Hh.is_hybrid(p):
        p_format = OA.P_EXPCAST
    quant, work = alloc_buffers(p)
    o = torch.empty(p.B, p.H, p.N, p.d, dtype=torch.bfloat16, device="cuda")
    vc.vc_attn(p, q, k, v, perm, o, quant, work)
    vc.vc_poll_status(work)
    vmax = max(float(v.float().abs().max()), 1e-6)
    worst = None
    for b in range(p.B):
        for h in range(p.H):
            bundle, cfg = Hh.oracle_prep(p, q, k, v, perm, b, h)
            kw = {}
            if softmax_scale is not None:
                kw["softmax_scale"] = softmax_scale
            if beta is not None:
                kw["beta"] = beta
            if p_format is not None:
                kw["p_format"] = p_format
            ref = OA.emulate_head(bundle, cfg, **kw)
            got = o[b, h].float().cpu().numpy()
            assert np.isfinite(got).all()
            m = CMP.output_metrics(got, ref, vmax)
            assert m["max_err_over_vmax"] <= 2e-2, m
            if np.linalg.norm(ref) > 1e-6:
                assert m["cos"] >= 0.999, m
            worst = m
    return worst


@pytest.mark.parametrize("bits", [8, 4, "4-hybrid"])
@pytest.mark.parametrize("N,grid", [(1, (1, 1, 1)), (2, (1, 1, 2)), (17, (1, 1, 17)), (127, (1, 1, 127))])
def test_shortest_sequences(N, grid, bits):
    w = vc_inputs.Workload("t", 1, 2, N, 128, grid, (8,), 41, "gauss")
    q, k, v = [t.cuda() for t in vc_inputs.make_qkv(w)]
    _run(_params(1, 2, N, 128, grid, bits), q, k, v, None)


@pytest.mark.parametrize("flags", [0, vc.VC_FLAG_ROPE, vc.VC_FLAG_HADAMARD | vc.VC_FLAG_K_SMOOTH, vc.VC_FLAG_V_SMOOTH,
                                   vc.VC_FLAG_ALL & ~vc.VC_FLAG_V_SMOOTH])
def test_stage_switches_end_to_end(flags):
    w = vc_inputs.Workload("t", 1, 2, 600, 128, (6, 10, 10), (8,), 42, "gauss")
    q, k, v = [t.cuda() for t in vc_inputs.make_qkv(w)]
    perm = vc_inputs.random_perm(1, 2, 600, 9).cuda()
    _run(Params.make(1, 2, 600, 128, (6, 10, 10), bits=8, flags=flags), q, k, v, perm)


def test_softmax_scale_beta_and_exp_then_cast():
    w = vc_inputs.Workload("t", 1, 1, 512, 64, (8, 8, 8), (8,), 43, "gauss")
    q, k, v = [t.cuda() for t in vc_inputs.make_qkv(w)]
    _run(Params.make(1, 1, 512, 64, (8, 8, 8), bits=8, softmax_scale=0.05, beta=-0.2), q, k, v, None,
         softmax_scale=0.05, beta=-0.2)
    _run(Params.make(1, 1, 512, 64, (8, 8, 8), bits=8, p_format=vc.VC_P_EXP_E4M3, softmax_scale=0.2), q, k, v, None,
         softmax_scale=0.2, p_format=OA.P_EXP_E4M3)


@pytest.mark.parametrize("bits", [8, 4, "4-hybrid"])
def test_degenerate_scales(bits):
    w = vc_inputs.Workload("t", 1, 1, 384, 128, (6, 8, 8), (8,), 44, "gauss")
    q, k, v = [t.cuda() for t in vc_inputs.make_qkv(w)]
    p = _params(1, 1, 384, 128, (6, 8, 8), bits)
    _run(p, q, k, torch.zeros_like(v), None)                                   # all-zero V: every scale degenerate
    _run(p, q, k, torch.full_like(v, 1.5), None)                               # constant V: zero residual, mean only
    pk = _params(1, 1, 384, 128, (6, 8, 8), bits, flags=vc.VC_FLAG_ALL & ~vc.VC_FLAG_ROPE)
    _run(pk, q, torch.full_like(k, 0.75), v, None)                             # constant K: centered keys vanish
    _run(p, torch.zeros_like(q), k, v, None)                                   # zero Q: uniform attention


def test_strided_inputs_through_vc_attn():
    B, H, N, d, grid = 1, 3, 300, 128, (3, 10, 10)
    w = vc_inputs.Workload("t", B, H, N, d, grid, (8,), 45, "gauss")
    q, k, v = [t.cuda() for t in vc_inputs.make_qkv(w)]
    qs, ks, vs = [t.permute(0, 2, 1, 3).contiguous() for t in (q, k, v)]       # [B, N, H, d] storage
    ps = Params.make(B, H, N, d, grid, bits=8, stride_b=N * H * d, stride_h=d, stride_n=H * d)
    p0 = Params.make(B, H, N, d, grid, bits=8)
    outs = []
    for p, (a, b, c) in ((ps, (qs, ks, vs)), (p0, (q, k, v))):
        quant, work = alloc_buffers(p)
        o = torch.empty(B, H, N, d, dtype=torch.bfloat16, device="cuda")
        vc.vc_attn(p, a, b, c, None, o, quant, work)
        vc.vc_poll_status(work)
        outs.append(o)
    assert torch.equal(outs[0], outs[1])


@pytest.mark.parametrize("shape", [(2, 6, 300, 64, (3, 10, 10)), (1, 3, 257, 128, (1, 1, 257)), (2, 16, 200, 64, (2, 10, 10)),
                                   (1, 48, 257, 128, (1, 1, 257))],
                         ids=["12_heads_6_groups", "3_heads", "32_heads_graduated_groups", "48_heads_odd_length"])
@pytest.mark.parametrize("bits", [8, 4, "4-hybrid"])
def test_host_entry_point_equals_the_device_path(shape, bits):
    """vc_attn_host (pinned host buffers in and out, pipelined over groups of heads) gives exactly
    the output of vc_attn on the same inputs, with and without a permutation."""
    B, H, N, d, grid = shape
    w = vc_inputs.Workload("t", B, H, N, d, grid, (8,), 77, "gauss")
    q, k, v = [t.cuda() for t in vc_inputs.make_qkv(w)]
    for perm in (None, vc_inputs.random_perm(B, H, N, 3).cuda()):
        p = (Params.make(B, H, N, d, grid, bits=4, p_format=vc.VC_P_EXPCAST_E4M3) if bits == "4-hybrid"
             else Params.make(B, H, N, d, grid, bits=bits))
        quant, work = alloc_buffers(p)
        o_ref = torch.empty(B, H, N, d, dtype=torch.bfloat16, device="cuda")
        vc.vc_attn(p, q, k, v, perm, o_ref, quant, work)
        vc.vc_poll_status(work)
        hq, hk, hv = [t.cpu().pin_memory() for t in (q, k, v)]
        hperm = perm.cpu().pin_memory() if perm is not None else None
        ho = torch.zeros(B, H, N, d, dtype=torch.bfloat16).pin_memory()
        dq, dk, dv, do = [torch.zeros_like(q) for _ in range(4)]
        dperm = torch.zeros(B, H, N, dtype=torch.int32, device="cuda") if perm is not None else None
        vc.vc_attn_host(p, hq, hk, hv, hperm, ho, dq, dk, dv, dperm, do, quant, work)
        vc.vc_poll_status(work)
        assert torch.equal(ho, o_ref.cpu())


@pytest.mark.parametrize("p_format", [vc.VC_P_EXPCAST_E4M3, vc.VC_P_EXP_E4M3], ids=["expcast", "exp_then_cast"])
@pytest.mark.parametrize("shape", [(1, 2, 128, 128, (2, 8, 8)), (1, 2, 129, 128, (1, 3, 43)), (2, 1, 300, 64, (3, 10, 10)),
                                   (1, 2, 1024, 128, (4, 16, 16)), (1, 1, 2000, 128, (5, 20, 20))],
                         ids=["n128", "n129", "n300_d64", "n1024", "n2000"])
def test_8bit_kernel_variants_agree(shape, p_format):
    """The two 8-bit kernels (two query tiles per CTA, pipelined; one tile per CTA, serial) run the
    same arithmetic per key tile: each matches the oracle's emulation."""
    B, H, N, d, grid = shape
    w = vc_inputs.Workload("t", B, H, N, d, grid, (8,), 91, "gauss")
    q, k, v = [t.cuda() for t in vc_inputs.make_qkv(w)]
    perm = vc_inputs.random_perm(B, H, N, 5).cuda()
    outs = {}
    for variant in (0, 1):
        p = Params.make(B, H, N, d, grid, bits=8, p_format=p_format, kernel_variant=variant)
        quant, work = alloc_buffers(p)
        o = torch.zeros(B, H, N, d, dtype=torch.bfloat16, device="cuda")
        vc.vc_attn(p, q, k, v, perm, o, quant, work)
        vc.vc_poll_status(work)
        outs[variant] = o
    vmax = float(v.float().abs().max())
    p = Params.make(B, H, N, d, grid, bits=8, p_format=p_format)
    pf = {vc.VC_P_EXPCAST_E4M3: OA.P_EXPCAST, vc.VC_P_EXP_E4M3: OA.P_EXP_E4M3}[p_format]
    bundle, cfg = Hh.oracle_prep(p, q, k, v, perm, 0, 0)
    ref = OA.emulate_head(bundle, cfg, p_format=pf)
    for variant in (0, 1):
        Hh.check_output(outs[variant][0, 0].float().cpu().numpy(), ref, vmax)


def test_sequence_parallel_wrapper_on_one_rank_is_vc_attn():
    """The head-sharded wrapper with a single rank (no exchange) returns exactly what vc_attn does,
    with and without the permutation from vc_group."""
    from paper_2609_15810_b200 import sequence_parallel as SP
    B, H, N, d, grid = 1, 2, 640, 128, (5, 8, 16)
    w = vc_inputs.Workload("t", B, H, N, d, grid, (8,), 77, "gauss")
    q, k, v = [t.cuda() for t in vc_inputs.make_qkv(w)]
    for group_k in (0, 8):
        got = SP.vc_attn_sequence_parallel(q, k, v, grid, bits=8, group_k=group_k, group_iters=2)
        p = Params.make(B, H, N, d, grid, bits=8)
        perm = None
        if group_k:
            gwork = torch.empty(vc.vc_group_workspace_bytes(p), dtype=torch.uint8, device="cuda")
            cent = torch.zeros(B, H, group_k, d, dtype=torch.float32, device="cuda")
            perm = torch.empty(B, H, N, dtype=torch.int32, device="cuda")
            vc.vc_group(p, v, group_k, 2, False, cent, perm, gwork)
        quant, work = alloc_buffers(p)
        o = torch.empty(B, H, N, d, dtype=torch.bfloat16, device="cuda")
        vc.vc_attn(p, q, k, v, perm, o, quant, work)
        vc.vc_poll_status(work)
        assert torch.equal(got, o)


@pytest.mark.parametrize("flags", [0, vc.VC_FLAG_ROPE | vc.VC_FLAG_HADAMARD, vc.VC_FLAG_K_SMOOTH | vc.VC_FLAG_V_SMOOTH])
def test_hybrid_4bit_stage_switches_and_parameters(flags):
    """The hybrid 4-bit arrangement with stages switched off, a non-default softmax scale and
    ExpCast offset, and a bundle that is only 16-byte aligned (rejected)."""
    B, H, N, d, grid = 1, 2, 333, 128, (3, 3, 37)
    w = vc_inputs.Workload("t", B, H, N, d, grid, (4,), 91, "gauss")
    q, k, v = [t.cuda() for t in vc_inputs.make_qkv(w)]
    p = Params.make(B, H, N, d, grid, bits=4, p_format=vc.VC_P_EXPCAST_E4M3, flags=flags, softmax_scale=0.11, beta=-0.2)
    quant, work = alloc_buffers(p)
    o = torch.empty(B, H, N, d, dtype=torch.bfloat16, device="cuda")
    vc.vc_attn(p, q, k, v, None, o, quant, work)
    vc.vc_poll_status(work)
    vmax = float(v.float().abs().max())
    for h in range(H):
        bundle, cfg = Hh.oracle_prep(p, q, k, v, None, 0, h)
        ref = OA.emulate_head(bundle, cfg, p_format=OA.P_EXPCAST, softmax_scale=0.11, beta=-0.2)
        Hh.check_output(o[0, h].float().cpu().numpy(), ref, vmax)
    shifted = torch.empty(quant.numel() + 16, dtype=torch.uint8, device="cuda")[16:]
    with pytest.raises(vc.VcError):
        vc.vc_attn_fwd(p, shifted, o, work)


@pytest.mark.parametrize("bits", [8, 4, "4-hybrid"])
def test_repeated_calls_are_bitwise_identical(bits):
    """No floating-point atomics and no order that depends on timing: the bundle and the output of
    two calls on the same inputs are the same bytes (the grouping call included)."""
    B, H, N, d, grid = 1, 3, 1500, 128, (5, 15, 20)
    w = vc_inputs.Workload("t", B, H, N, d, grid, (8,), 63, "field")
    q, k, v = [t.cuda() for t in vc_inputs.make_qkv(w)]
    p = _params(B, H, N, d, grid, bits)
    outs = []
    for _ in range(2):
        gwork = torch.empty(vc.vc_group_workspace_bytes(p), dtype=torch.uint8, device="cuda")
        cent = torch.zeros(B, H, 16, d, dtype=torch.float32, device="cuda")
        perm = torch.empty(B, H, N, dtype=torch.int32, device="cuda")
        vc.vc_group(p, v, 16, 3, False, cent, perm, gwork)
        quant, work = alloc_buffers(p)
        quant.zero_()
        o = torch.empty(B, H, N, d, dtype=torch.bfloat16, device="cuda")
        vc.vc_attn(p, q, k, v, perm, o, quant, work)
        vc.vc_poll_status(work)
        outs.append((perm.clone(), cent.clone(), quant.clone(), o.clone()))
    for a, b in zip(*outs):
        assert torch.equal(a, b)
