"""The C-ABI library loads and exports every symbol include/vc_attn.h declares (no GPU)."""
import ctypes
import os
import re

import paper_2609_15810_b200 as vc
from paper_2609_15810_b200.binding import Params

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "vc_attn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(vc_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    lib = vc.load_library()
    names = _declared_symbols()
    assert {"vc_prep", "vc_attn_fwd", "vc_attn", "vc_quant_bytes", "vc_workspace_bytes"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_sizes_and_argument_validation_without_a_gpu():
    p = Params.make(1, 40, 32760, 128, (21, 30, 52), bits=8)
    n_pad = 32768
    qb = vc.vc_quant_bytes(p)
    assert qb >= 3 * 40 * n_pad * 128 and qb < 3 * 40 * n_pad * 128 * 1.02
    assert vc.vc_workspace_bytes(p) > 0
    p4 = Params.make(1, 40, 32760, 128, (21, 30, 52), bits=4)
    assert vc.vc_quant_bytes(p4) < 0.6 * qb
    # the hybrid 4-bit arrangement: value factors per 32 tokens instead of 16, pipelined kernel only
    ph = Params.make(1, 40, 32760, 128, (21, 30, 52), bits=4, p_format=vc.VC_P_EXPCAST_E4M3)
    assert 0 < vc.vc_quant_bytes(p4) - vc.vc_quant_bytes(ph) <= 40 * n_pad * 128 // 32 + 2048
    assert vc.vc_quant_bytes(Params.make(1, 2, 1024, 128, (4, 16, 16), bits=4, p_format=vc.VC_P_EXPCAST_E4M3, kernel_variant=1)) == 0
    assert vc.vc_quant_bytes(Params.make(1, 2, 1024, 128, (4, 16, 16), bits=4, p_format=vc.VC_P_EXP_E4M3)) == 0
    assert vc.vc_quant_bytes(Params.make(1, 2, 1024, 128, (4, 16, 16), bits=8, p_format=vc.VC_P_EXP_POLY_E4M3)) > 0
    qb0 = vc.vc_quant_bytes(Params.make(1, 2, 1024, 128, (4, 16, 16)))
    for bad in (dict(d=100), dict(N=-1), dict(bits=3), dict(grid_t=20), dict(p_format=9), dict(B=40000)):
        pb = Params.make(1, 2, 1024, 128, (4, 16, 16))
        for k, v in bad.items():
            setattr(pb, k, v)
        assert vc.vc_quant_bytes(pb) == 0 and vc.vc_workspace_bytes(pb) == 0
    assert vc.vc_status_string(0) == "ok" and "timed out" in vc.vc_status_string(5)
    assert ctypes.sizeof(Params) == 112
    # block sizes are arguments (Eq. 4's B_v, the scale blocks): 0 means 128, nothing else is implemented
    assert vc.vc_quant_bytes(Params.make(1, 2, 1024, 128, (4, 16, 16), block_q=128, block_k=128, block_v=128)) == qb0
    for name in ("block_q", "block_k", "block_v"):
        assert vc.vc_quant_bytes(Params.make(1, 2, 1024, 128, (4, 16, 16), **{name: 64})) == 0
    import ctypes as C
    lib = vc.load_library()
    pb = Params.make(1, 2, 1024, 128, (4, 16, 16), block_v=64)
    assert lib.vc_prep(C.byref(pb), 16, 16, 16, None, 16, 16, None) == vc.VC_ERR_UNSUPPORTED      # refused before any launch
    pb = Params.make(1, 2, 1024, 128, (4, 16, 16), block_v=-1)
    assert lib.vc_prep(C.byref(pb), 16, 16, 16, None, 16, 16, None) == vc.VC_ERR_INVALID_ARG
    # a row stride has to fit 32 bits in bytes (the kernels address rows with one 32 x 32 -> 64 multiply)
    pb = Params.make(1, 2, 1024, 128, (4, 16, 16), stride_n=1 << 30, stride_h=1 << 41, stride_b=1 << 43)
    assert lib.vc_prep(C.byref(pb), 16, 16, 16, None, 16, 16, None) == vc.VC_ERR_UNSUPPORTED
    assert vc.vc_quant_bytes(Params.make(1, 2, 1024, 128, (4, 16, 16), stride_n=256, stride_h=1024 * 256, stride_b=2 * 1024 * 256)) == qb0
    # the validator's bitmap is part of the workspace only when it is asked for
    pc = Params.make(1, 2, 1024, 128, (4, 16, 16), flags=vc.VC_FLAG_ALL | vc.VC_FLAG_CHECK_PERM)
    assert vc.vc_workspace_bytes(pc) > vc.vc_workspace_bytes(Params.make(1, 2, 1024, 128, (4, 16, 16)))
    assert vc.vc_launch_count() == 0


def test_grouping_schedule_matches_the_papers_worked_examples():
    """vc_group_schedule against the step lists the paper prints (tests/golden/grouping_schedule.txt)."""
    for line in open(os.path.join(ROOT, "tests", "golden", "grouping_schedule.txt")):
        if line.startswith("#") or not line.strip():
            continue
        n, steps, window = line.split()
        n, window = int(n), int(window)
        want = [int(s) for s in steps.split(",")]
        kinds = [vc.vc_group_schedule(s, n, 4) for s in range(n)]
        assert [s for s in range(n) if kinds[s] == vc.VC_GROUP_RECOMPUTE] == want
        assert all(k == vc.VC_GROUP_FROZEN for k in kinds[window:]) and vc.VC_GROUP_FROZEN not in kinds[:window]
    assert vc.vc_group_schedule(-1, 8, 4) == -1 and vc.vc_group_schedule(8, 8, 4) == -1 and vc.vc_group_schedule(0, 8, 0) == -1
