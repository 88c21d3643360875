"""Glue between the oracle (NumPy, per head) and the CUDA library (device bundle)."""
import numpy as np
import torch

import paper_2609_15810_b200 as vc
from paper_2609_15810_b200.binding import Params, alloc_buffers, section
from oracle import attention as OA
from oracle import codecs as OC
from oracle import compare as CMP
from oracle import prep as OP


def is_hybrid(p):
    """The hybrid 4-bit arrangement: bits = 4 with the ExpCast-FP8 probability format."""
    return p.bits == 4 and p.p_format == vc.VC_P_EXPCAST_E4M3


def oracle_cfg(p, **kw):
    dims = (p.rope_dim_t, p.rope_dim_h, p.rope_dim_w)
    if is_hybrid(p):
        kw.setdefault("v_format", "mxfp4")
    return OP.PrepConfig(N=p.N, d=p.d, grid=(p.grid_t, p.grid_h, p.grid_w), bits=p.bits,
                         rope=bool(p.flags & vc.VC_FLAG_ROPE), hadamard=bool(p.flags & vc.VC_FLAG_HADAMARD),
                         k_smooth=bool(p.flags & vc.VC_FLAG_K_SMOOTH), v_smooth=bool(p.flags & vc.VC_FLAG_V_SMOOTH),
                         rope_dims=dims if any(dims) else None,
                         rope_theta=p.rope_theta if p.rope_theta else 10000.0,
                         qk_format="int8" if (p.flags & vc.VC_FLAG_INT8_QK) else "e4m3", **kw)


def oracle_prep(p, q, k, v, perm, b, h):
    """Oracle bundle of head (b, h) from the same bf16 buffers (host copies)."""
    cfg = oracle_cfg(p)
    f = lambda t: t[b, h].float().cpu().numpy()
    pm = None if perm is None else perm[b, h].cpu().numpy().astype(np.int64)
    return OP.prep_head(f(q), f(k), f(v), pm, cfg), cfg


def gpu_sections(p, quant):
    """NumPy views (host copies) of every section of the device bundle, per the ABI layout."""
    view = vc.vc_quant_view(p, quant)
    BH, d = p.B * p.H, p.d
    n_pad = 128 * ((p.N + 127) // 128)
    nb = n_pad // 128
    s = lambda name, dt=torch.uint8: section(view, name, quant, dt).cpu()
    out = {}
    if p.bits == 8:
        out["q_codes"] = s("q_codes").numpy().reshape(BH, n_pad, d)
        out["k_codes"] = s("k_codes").numpy().reshape(BH, n_pad, d)
        out["v_codes"] = s("v_codes").numpy().reshape(BH, d, n_pad).transpose(0, 2, 1)
        out["q_scale"] = s("q_scale", torch.float32).numpy().reshape(BH, nb)
        out["k_scale"] = s("k_scale", torch.float32).numpy().reshape(BH, nb)
        if p.flags & vc.VC_FLAG_INT8_QK:
            out["q_codes"], out["k_codes"] = out["q_codes"].view(np.int8), out["k_codes"].view(np.int8)
    else:
        out["q_codes"] = CMP.unpack_nibbles(s("q_codes").numpy().reshape(BH, n_pad, d // 2))
        out["k_codes"] = CMP.unpack_nibbles(s("k_codes").numpy().reshape(BH, n_pad, d // 2))
        out["v_codes"] = CMP.unpack_nibbles(s("v_codes").numpy().reshape(BH, d, n_pad // 2)).transpose(0, 2, 1)
        out["q_micro"] = s("q_micro").numpy().reshape(BH, n_pad, d // 16)
        out["k_micro"] = s("k_micro").numpy().reshape(BH, n_pad, d // 16)
        out["v_micro"] = s("v_micro").numpy().reshape(BH, d, n_pad // (32 if is_hybrid(p) else 16)).transpose(0, 2, 1)
        out["q_scale"] = s("q_scale", torch.float32).numpy().reshape(BH)
        out["k_scale"] = s("k_scale", torch.float32).numpy().reshape(BH)
    out["v_scale"] = s("v_scale", torch.float32).numpy().reshape(BH, d)
    out["v_means"] = s("v_means", torch.bfloat16).float().numpy().reshape(BH, nb, d)
    out["k_mean"] = s("k_mean", torch.float32).numpy().reshape(BH, d)
    return out


def upload_bundle(p, quant, bundles):
    """Writes the oracle's bundles (list over b*H+h) into the device bundle, in the layout the ABI
    documents: bytes at 8 bits; at 4 bits nibbles two per byte (even index low), microscale bytes
    beside them, the outer scales of Q and K in q_scale / k_scale."""
    view = vc.vc_quant_view(p, quant)
    put = lambda name, arr, dt=torch.uint8: section(view, name, quant, dt).copy_(
        torch.from_numpy(np.ascontiguousarray(arr)).view(dt).reshape(-1).to(quant.device))
    if p.bits == 8:
        put("q_codes", np.stack([b["q_codes"] for b in bundles]).view(np.uint8))
        put("k_codes", np.stack([b["k_codes"] for b in bundles]).view(np.uint8))
        put("v_codes", np.stack([b["v_codes"].T for b in bundles]))
        put("q_scale", np.stack([b["q_scale"] for b in bundles]).astype(np.float32), torch.float32)
        put("k_scale", np.stack([b["k_scale"] for b in bundles]).astype(np.float32), torch.float32)
    else:
        put("q_codes", np.stack([CMP.pack_nibbles(b["q_codes"]) for b in bundles]))
        put("k_codes", np.stack([CMP.pack_nibbles(b["k_codes"]) for b in bundles]))
        put("v_codes", np.stack([CMP.pack_nibbles(np.ascontiguousarray(b["v_codes"].T)) for b in bundles]))
        put("q_micro", np.stack([b["q_micro"] for b in bundles]))
        put("k_micro", np.stack([b["k_micro"] for b in bundles]))
        put("v_micro", np.stack([np.ascontiguousarray(b["v_micro"].T) for b in bundles]))
        put("q_scale", np.array([b["q_g"] for b in bundles], dtype=np.float32), torch.float32)
        put("k_scale", np.array([b["k_g"] for b in bundles], dtype=np.float32), torch.float32)
    put("v_scale", np.stack([b["v_scale"] for b in bundles]).astype(np.float32), torch.float32)
    put("k_mean", np.stack([b["k_mean"] for b in bundles]).astype(np.float32), torch.float32)
    means = np.stack([OC.bf16_bits(b["v_means"]) for b in bundles]).view(np.int16)
    put("v_means", means, torch.int16)


def check_prep_head(p, got, bh, ref, what=""):
    """vc_prep's sections of head bh against the oracle bundle."""
    mag = 7 if p.bits == 8 else 3
    rel = lambda a, b: float(np.max(np.abs(a - b) / np.maximum(np.abs(b), 1e-30)))
    stats = {}
    # the channel mean of K as a VECTOR: 1e-5 of its largest component.  (An fp32 sum of N values
    # of size A is off by about A 2^-24 sqrt(N), whatever the size of the mean itself, so a
    # component that happens to lie near zero cannot be held to 1e-5 of its own value.)
    assert np.abs(got["k_mean"][bh] - ref["k_mean"]).max() <= 1e-5 * max(np.abs(ref["k_mean"]).max(), 1e-30), what + " k_mean"
    if p.bits == 8:
        assert rel(got["q_scale"][bh], ref["q_scale"]) < 1e-5, what + " q_scale"
        assert rel(got["k_scale"][bh], ref["k_scale"]) < 1e-5, what + " k_scale"
        assert rel(got["v_scale"][bh], ref["v_scale"]) < 1e-5, what + " v_scale"
    else:
        assert rel(got["q_scale"][bh], ref["q_g"]) < 1e-5 and rel(got["k_scale"][bh], ref["k_g"]) < 1e-5, what
        for t in ("q", "k", "v"):
            # (the power-of-two factors of the hybrid arrangement are 8-bit magnitudes)
            stats[t + "_micro"] = CMP.assert_codes_close(got[t + "_micro"][bh], ref[t + "_micro"],
                                                         8 if t == "v" and is_hybrid(p) else 7, what=what + t + "_micro")
    for t in ("q", "k", "v"):
        if p.bits == 8 and t != "v" and (p.flags & vc.VC_FLAG_INT8_QK):
            diff = np.abs(got[t + "_codes"][bh].astype(np.int32) - ref[t + "_codes"].astype(np.int32))
            assert diff.max() <= 1 and float(np.mean(diff != 0)) <= 1e-3, what + " " + t + "_codes (int8)"
            stats[t] = float(np.mean(diff != 0))
        elif p.bits == 8:
            stats[t] = CMP.assert_codes_close(got[t + "_codes"][bh], ref[t + "_codes"], mag, what=what + " " + t + "_codes")
        else:
            # under the same microscale: codes identical except <= 0.1 % one step apart; under a
            # differing microscale (itself one step apart, counted above): compared after decoding,
            # within one element step of the larger microscale (the widest E2M1 gap is 2)
            grp = 32 if t == "v" and is_hybrid(p) else 16
            ax = 1 if t != "v" else 0
            gm, rm = got[t + "_micro"][bh], ref[t + "_micro"]
            same = np.repeat(gm == rm, grp, axis=ax)
            g, r = got[t + "_codes"][bh], ref[t + "_codes"]
            frac, dist = CMP.code_mismatch(g[same], r[same], 3)
            assert dist <= 1 and frac <= 1e-3, f"{what} {t}_codes: frac {frac:.2e} dist {dist}"
            stats[t] = frac
            if not same.all():
                dec = (lambda m: np.exp2(m.astype(np.float64) - 127.0)) if (t == "v" and is_hybrid(p)) else OC.e4m3_decode
                sg, sr = np.repeat(dec(gm), grp, axis=ax), np.repeat(dec(rm), grp, axis=ax)
                dg, dr = OC.e2m1_decode(g) * sg, OC.e2m1_decode(r) * sr
                assert np.all(np.abs(dg - dr)[~same] <= 2.0 * np.maximum(sg, sr)[~same] * (1 + 1e-9)), f"{what} {t}_codes under differing microscales"
    # block means: at most one bf16 ulp
    gm, rm = got["v_means"][bh], ref["v_means"]
    ulp = np.maximum(np.abs(rm), 1e-30) * 2.0 ** -7
    assert np.all(np.abs(gm - rm) <= ulp + 1e-30), what + " v_means"
    return stats


def run_prep(p, q, k, v, perm):
    quant, work = alloc_buffers(p)
    quant.zero_()
    vc.vc_prep(p, q, k, v, perm, quant, work)
    torch.cuda.synchronize()
    return quant, work


def check_output(o_gpu_rows, o_ref_rows, v_absmax, tol=2e-2, cos_min=0.999):
    m = CMP.output_metrics(o_gpu_rows, o_ref_rows, v_absmax)
    assert m["max_err_over_vmax"] <= tol, m
    assert m["cos"] >= cos_min, m
    return m
