"""Parity of the CUDA path (through the C ABI) against the CPU oracle, element by element.

Three stages so that a failure can be attributed: (1) vc_prep against the oracle's bundle;
(2) vc_attn_fwd fed the ORACLE's bundle against the oracle's emulated output; (3) vc_attn
end to end.  Tolerances (from the benchmark spec): quantized codes identical except
<= 0.1% of elements one code step apart; outputs within 2e-2 * max|V| elementwise and
cosine >= 0.999 against the emulation.
"""
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

SMALL = [  # name, B, H, N, d, grid
    ("n128", 1, 1, 128, 128, (2, 8, 8)),
    ("n129", 1, 2, 129, 128, (1, 3, 43)),
    ("n255", 2, 1, 255, 128, (3, 5, 17)),
    ("n300_d64", 1, 2, 300, 64, (3, 10, 10)),
    ("n1024", 1, 2, 1024, 128, (4, 16, 16)),
]


def _inputs(B, H, N, d, grid, seed, kind="gauss"):
    w = vc_inputs.Workload("t", B, H, N, d, grid, (8,), seed, kind)
    return [t.cuda() for t in vc_inputs.make_qkv(w)]


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("perm_kind", ["identity", "random"])
@pytest.mark.parametrize("case", SMALL, ids=[c[0] for c in SMALL])
def test_prep_matches_oracle(case, perm_kind, bits):
    _, B, H, N, d, grid = case
    q, k, v = _inputs(B, H, N, d, grid, seed=11)
    perm = None if perm_kind == "identity" else vc_inputs.random_perm(B, H, N, 5).cuda()
    p = Params.make(B, H, N, d, grid, bits=bits)
    quant, _ = Hh.run_prep(p, q, k, v, perm)
    got = Hh.gpu_sections(p, quant)
    for b in range(B):
        for h in range(H):
            ref, _ = Hh.oracle_prep(p, q, k, v, perm, b, h)
            Hh.check_prep_head(p, got, b * H + h, ref, what=f"{case[0]} b{b} h{h}")


@pytest.mark.parametrize("flags", [0, vc.VC_FLAG_ROPE, vc.VC_FLAG_HADAMARD, vc.VC_FLAG_K_SMOOTH | vc.VC_FLAG_V_SMOOTH])
def test_prep_stage_switches(flags):
    B, H, N, d, grid = 1, 2, 300, 128, (3, 10, 10)
    q, k, v = _inputs(B, H, N, d, grid, seed=12)
    p = Params.make(B, H, N, d, grid, bits=8, flags=flags)
    quant, _ = Hh.run_prep(p, q, k, v, None)
    got = Hh.gpu_sections(p, quant)
    for h in range(H):
        ref, _ = Hh.oracle_prep(p, q, k, v, None, 0, h)
        Hh.check_prep_head(p, got, h, ref, what=f"flags{flags} h{h}")


def test_prep_strided_inputs_and_head_groups():
    """[B, N, H, d] storage viewed as [B, H, N, d], preprocessed two heads at a time."""
    B, H, N, d, grid = 1, 4, 300, 128, (3, 10, 10)
    q, k, v = _inputs(B, H, N, d, grid, seed=13)
    qs, ks, vs = [t.permute(0, 2, 1, 3).contiguous() for t in (q, k, v)]          # [B, N, H, d]
    p = Params.make(B, H, N, d, grid, bits=8, stride_b=N * H * d, stride_h=d, stride_n=H * d, heads_per_pass=2)
    quant, _ = Hh.run_prep(p, qs, ks, vs, None)
    p0 = Params.make(B, H, N, d, grid, bits=8)
    quant0, _ = Hh.run_prep(p0, q, k, v, None)
    assert torch.equal(quant, quant0)


@pytest.mark.parametrize("p_format", [vc.VC_P_EXPCAST_E4M3, vc.VC_P_EXP_E4M3, vc.VC_P_EXP_POLY_E4M3, vc.VC_P_EXP_MIX_E4M3],
                         ids=["expcast", "exp_sfu", "exp_poly", "exp_mix"])
@pytest.mark.parametrize("case", SMALL, ids=[c[0] for c in SMALL])
def test_attn_fwd_on_oracle_bundle(case, p_format):
    """Stage 2: isolates the attention kernel from code flips in prep.  The polynomial forms of
    exponentiate-then-cast are held to the same oracle result as the special-function one."""
    _, B, H, N, d, grid = case
    q, k, v = _inputs(B, H, N, d, grid, seed=21)
    perm = vc_inputs.random_perm(B, H, N, 6).cuda()
    p = Params.make(B, H, N, d, grid, bits=8, p_format=p_format)
    quant, work = alloc_buffers(p)
    quant.zero_()
    bundles, refs = [], []
    fmt = OA.P_EXPCAST if p_format == vc.VC_P_EXPCAST_E4M3 else OA.P_EXP_E4M3
    for b in range(B):
        for h in range(H):
            bundle, cfg = Hh.oracle_prep(p, q, k, v, perm, b, h)
            bundles.append(bundle)
            refs.append(OA.emulate_head(bundle, cfg, p_format=fmt))
    Hh.upload_bundle(p, quant, bundles)
    o = torch.empty(B, H, N, d, dtype=torch.bfloat16, device="cuda")
    vc.vc_attn_fwd(p, quant, o, work)
    vc.vc_poll_status(work)
    vmax = float(v.float().abs().max())
    for i, ref in enumerate(refs):
        m = Hh.check_output(o.view(B * H, N, d)[i].float().cpu().numpy(), ref, vmax)
        assert m["max_err_over_vmax"] < 1e-2, m


@pytest.mark.parametrize("arrangement", ["nvfp4", "hybrid", "nvfp4_serial"])
@pytest.mark.parametrize("case", SMALL, ids=[c[0] for c in SMALL])
def test_attn_fwd_4bit_on_oracle_bundle(case, arrangement):
    """Stage 2 at 4 bits: the attention kernels fed the ORACLE's bundle (nibbles, microscales or
    power-of-two factors, outer scales uploaded through the ABI's layout), so that a difference
    in the output cannot come from a code flip in vc_prep."""
    _, B, H, N, d, grid = case
    q, k, v = _inputs(B, H, N, d, grid, seed=61)
    perm = vc_inputs.random_perm(B, H, N, 12).cuda()
    hybrid = arrangement == "hybrid"
    p = Params.make(B, H, N, d, grid, bits=4, p_format=vc.VC_P_EXPCAST_E4M3 if hybrid else vc.VC_P_DEFAULT,
                    kernel_variant=1 if arrangement == "nvfp4_serial" else 0)
    quant, work = alloc_buffers(p)
    quant.zero_()
    bundles, refs = [], []
    for b in range(B):
        for h in range(H):
            bundle, cfg = Hh.oracle_prep(p, q, k, v, perm, b, h)
            bundles.append(bundle)
            refs.append(OA.emulate_head(bundle, cfg, p_format=OA.P_EXPCAST if hybrid else None))
    Hh.upload_bundle(p, quant, bundles)
    got = Hh.gpu_sections(p, quant)                      # the upload reads back as the oracle's bundle
    assert np.array_equal(got["k_codes"][0], bundles[0]["k_codes"]) and np.array_equal(got["v_micro"][0], bundles[0]["v_micro"])
    o = torch.empty(B, H, N, d, dtype=torch.bfloat16, device="cuda")
    vc.vc_attn_fwd(p, quant, o, work)
    vc.vc_poll_status(work)
    vmax = float(v.float().abs().max())
    for i, ref in enumerate(refs):
        m = Hh.check_output(o.view(B * H, N, d)[i].float().cpu().numpy(), ref, vmax)
        assert m["max_err_over_vmax"] < 1e-2, m


@pytest.mark.parametrize("perm_kind", ["identity", "random", "kmeans"])
def test_vc_attn_end_to_end_config1(perm_kind):
    """Stage 3 on the tiny correctness configuration (B=1, H=2, N=1024, d=128, 8-bit)."""
    w = vc_inputs.WORKLOADS["c1"]
    q, k, v = [t.cuda() for t in vc_inputs.make_qkv(w)]
    perm = {"identity": None, "random": vc_inputs.random_perm(w.B, w.H, w.N, 7).cuda(),
            "kmeans": vc_kmeans_harness.kmeans_perm_all(v, k=8)}[perm_kind]
    p = Params.make(w.B, w.H, w.N, w.d, w.grid, bits=8)
    quant, work = alloc_buffers(p)
    o = torch.empty(w.B, w.H, w.N, w.d, dtype=torch.bfloat16, device="cuda")
    vc.vc_attn(p, q, k, v, perm, o, quant, work)
    vc.vc_poll_status(work)
    vmax = float(v.float().abs().max())
    for h in range(w.H):
        bundle, cfg = Hh.oracle_prep(p, q, k, v, perm, 0, h)
        ref = OA.emulate_head(bundle, cfg)
        got = o[0, h].float().cpu().numpy()
        Hh.check_output(got, ref, vmax)
        exact = OA.reference_head(q[0, h].float().cpu().numpy(), k[0, h].float().cpu().numpy(),
                                  v[0, h].float().cpu().numpy(), cfg)
        # accuracy against exact attention is reported, not gated by the tolerance above:
        # the CUDA path must simply be as close to it as the emulation is
        m0, m1 = CMP.output_metrics(got, exact, vmax), CMP.output_metrics(ref, exact, vmax)
        assert m0["cos"] > 0.999 and m0["cos"] > m1["cos"] - 1e-4, (m0, m1)
        assert m0["max_err_over_vmax"] < m1["max_err_over_vmax"] + 1e-2, (m0, m1)


@pytest.mark.parametrize("variant", [0, 1], ids=["block_scaled_fp4", "serial_bf16"])
@pytest.mark.parametrize("perm_kind", ["identity", "random"])
@pytest.mark.parametrize("case", SMALL, ids=[c[0] for c in SMALL])
def test_vc_attn_4bit_end_to_end(case, perm_kind, variant):
    """4-bit path (NVFP4 Q, K, residual and P): vc_attn against the oracle's emulation, for the
    block-scaled FP4 kernel (default) and the serial kernel that expands the operands to bf16."""
    _, B, H, N, d, grid = case
    q, k, v = _inputs(B, H, N, d, grid, seed=31)
    perm = None if perm_kind == "identity" else vc_inputs.random_perm(B, H, N, 8).cuda()
    p = Params.make(B, H, N, d, grid, bits=4, kernel_variant=variant)
    quant, work = alloc_buffers(p)
    o = torch.empty(B, H, N, d, dtype=torch.bfloat16, device="cuda")
    vc.vc_attn(p, q, k, v, perm, o, quant, work)
    vc.vc_poll_status(work)
    vmax = float(v.float().abs().max())
    for b in range(B):
        for h in range(H):
            bundle, cfg = Hh.oracle_prep(p, q, k, v, perm, b, h)
            ref = OA.emulate_head(bundle, cfg)
            Hh.check_output(o[b, h].float().cpu().numpy(), ref, vmax)


@pytest.mark.parametrize("perm_kind", ["identity", "random"])
@pytest.mark.parametrize("case", SMALL, ids=[c[0] for c in SMALL])
def test_hybrid_4bit_arrangement(case, perm_kind):
    """bits = 4 with the ExpCast-FP8 probability: NVFP4 Q^ and K^, E2M1 values under power-of-two
    factors per 32 tokens, the value product as an FP8 x FP4 block-scaled MMA.  vc_prep's value
    codes and factors against the oracle, then vc_attn end to end against its emulation."""
    _, B, H, N, d, grid = case
    q, k, v = _inputs(B, H, N, d, grid, seed=51)
    perm = None if perm_kind == "identity" else vc_inputs.random_perm(B, H, N, 10).cuda()
    p = Params.make(B, H, N, d, grid, bits=4, p_format=vc.VC_P_EXPCAST_E4M3)
    quant, work = Hh.run_prep(p, q, k, v, perm)
    got = Hh.gpu_sections(p, quant)
    o = torch.empty(B, H, N, d, dtype=torch.bfloat16, device="cuda")
    vc.vc_attn(p, q, k, v, perm, o, quant, work)
    vc.vc_poll_status(work)
    vmax = float(v.float().abs().max())
    for b in range(B):
        for h in range(H):
            bundle, cfg = Hh.oracle_prep(p, q, k, v, perm, b, h)
            assert cfg.v_format == "mxfp4"
            Hh.check_prep_head(p, got, b * H + h, bundle, what=f"hybrid head {b},{h}")
            ref = OA.emulate_head(bundle, cfg, p_format=OA.P_EXPCAST)
            Hh.check_output(o[b, h].float().cpu().numpy(), ref, vmax)


@pytest.mark.parametrize("perm_kind", ["identity", "random"])
def test_prep_with_supplied_statistics(perm_kind):
    """App. B: the statistics (K channel mean, V block means, residual maxima) can come from the
    producer of K and V; the pass then reads K and V once.  Fed the statistics vc_prep itself
    computed, the bundle is the same byte for byte; fed the ORACLE's, it matches the oracle's
    bundle within the usual tolerance."""
    B, H, N, d, grid = 2, 2, 300, 128, (3, 10, 10)
    q, k, v = _inputs(B, H, N, d, grid, seed=71)
    perm = None if perm_kind == "identity" else vc_inputs.random_perm(B, H, N, 13).cuda()
    p = Params.make(B, H, N, d, grid, bits=8)
    quant, work = Hh.run_prep(p, q, k, v, perm)
    km, vmu, vam = [t.clone() for t in vc.vc_prep_stats_view(p, quant, work)]
    quant2, work2 = alloc_buffers(p)
    quant2.zero_()
    n0 = vc.vc_launch_count()
    vc.vc_prep_with_stats(p, q, k, v, perm, km, vmu, vam, quant2, work2)
    torch.cuda.synchronize()
    n1 = vc.vc_launch_count()
    vc.vc_prep(p, q, k, v, perm, quant, work)
    assert n1 - n0 == (vc.vc_launch_count() - n1) - 2          # the two statistics launches are gone
    assert torch.equal(quant2, quant)
    # the oracle's statistics
    refs = [Hh.oracle_prep(p, q, k, v, perm, b, h)[0] for b in range(B) for h in range(H)]
    f32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()
    km_o = f32(np.stack([r["k_mean"] for r in refs]))
    vmu_o = f32(np.stack([r["v_mu"] for r in refs]))
    vam_o = f32(np.stack([np.abs(r["v_pre"]).max(axis=0) for r in refs]))
    quant2.zero_()
    vc.vc_prep_with_stats(p, q, k, v, perm, km_o, vmu_o, vam_o, quant2, work2)
    torch.cuda.synchronize()
    got = Hh.gpu_sections(p, quant2)
    for i, ref in enumerate(refs):
        Hh.check_prep_head(p, got, i, ref, what=f"supplied statistics head {i}")
    p4 = Params.make(B, H, N, d, grid, bits=4)
    q4, w4 = alloc_buffers(p4)
    with pytest.raises(vc.VcError) as e:
        vc.vc_prep_with_stats(p4, q, k, v, perm, km, vmu, vam, q4, w4)
    assert e.value.code == vc.VC_ERR_UNSUPPORTED


def test_bad_arguments_are_rejected_on_the_host():
    p = Params.make(1, 1, 128, 128, (2, 8, 8))
    quant, work = alloc_buffers(p)
    x = torch.zeros(1, 1, 128, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(vc.VcError):
        vc.vc_prep(p, None, x, x, None, quant, work)
    with pytest.raises(vc.VcError):
        vc.vc_prep(p, x.view(-1)[1:], x, x, None, quant, work)          # misaligned
    for bad in (dict(d=96), dict(N=0), dict(bits=5), dict(grid_w=9), dict(flags=64), dict(rope_dim_t=3)):
        pb = Params.make(1, 1, 128, 128, (2, 8, 8))
        for kk, vv in bad.items():
            setattr(pb, kk, vv)
        assert vc.vc_quant_bytes(pb) == 0
        with pytest.raises(vc.VcError):
            vc.vc_prep(pb, x, x, x, None, quant, work)


@pytest.mark.parametrize("perm_kind", ["identity", "random"])
@pytest.mark.parametrize("case", SMALL, ids=[c[0] for c in SMALL])
def test_int8_qk_variant(case, perm_kind):
    """VC_FLAG_INT8_QK (the INT8 Q K^T arrangement of Fig. 3): the INT8 codes and scales of vc_prep
    against the oracle, then vc_attn end to end against the oracle's emulation of that variant."""
    _, B, H, N, d, grid = case
    q, k, v = _inputs(B, H, N, d, grid, seed=41)
    perm = None if perm_kind == "identity" else vc_inputs.random_perm(B, H, N, 9).cuda()
    p = Params.make(B, H, N, d, grid, bits=8, flags=vc.VC_FLAG_ALL | vc.VC_FLAG_INT8_QK)
    quant, work = Hh.run_prep(p, q, k, v, perm)
    got = Hh.gpu_sections(p, quant)
    o = torch.empty(B, H, N, d, dtype=torch.bfloat16, device="cuda")
    vc.vc_attn(p, q, k, v, perm, o, quant, work)
    vc.vc_poll_status(work)
    vmax = float(v.float().abs().max())
    for b in range(B):
        for h in range(H):
            bundle, cfg = Hh.oracle_prep(p, q, k, v, perm, b, h)
            assert bundle["q_codes"].dtype == np.int8
            Hh.check_prep_head(p, got, b * H + h, bundle, what=f"int8 head {b},{h}")
            Hh.check_output(o[b, h].float().cpu().numpy(), OA.emulate_head(bundle, cfg), vmax)


def test_int8_qk_is_rejected_where_it_does_not_apply():
    for kw in (dict(bits=4), dict(bits=8, kernel_variant=1)):
        p = Params.make(1, 1, 256, 128, (4, 8, 8), flags=vc.VC_FLAG_ALL | vc.VC_FLAG_INT8_QK, **kw)
        assert vc.vc_quant_bytes(p) == 0
