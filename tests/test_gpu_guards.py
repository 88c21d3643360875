"""Guards of the C-ABI that a correct call never meets: the validator of the permutation, the
bounded device-side waits and their status word.  Nothing here faults or hangs a GPU: a bad
permutation is clamped before it becomes an address, and a wait is made to run out on a CORRECT
run by shortening its limit through the library's test hook."""
import pytest
import torch

import paper_2609_15810_b200 as vc
import vc_inputs
from paper_2609_15810_b200.binding import Params, alloc_buffers

pytestmark = pytest.mark.gpu


def _case(bits=8, p_format=vc.VC_P_DEFAULT, flags=vc.VC_FLAG_ALL):
    w = vc_inputs.WORKLOADS["c1"]
    q, k, v = [t.cuda() for t in vc_inputs.make_qkv(w)]
    perm = vc_inputs.random_perm(w.B, w.H, w.N, 17).cuda()
    p = Params.make(w.B, w.H, w.N, w.d, w.grid, bits=bits, p_format=p_format, flags=flags)
    quant, work = alloc_buffers(p)
    o = torch.empty(w.B, w.H, w.N, w.d, dtype=torch.bfloat16, device="cuda")
    return w, p, q, k, v, perm, quant, work, o


@pytest.mark.parametrize("bits", [8, 4])
def test_permutation_validator(bits):
    """Eq. 3 needs a permutation.  An entry out of range and an entry that occurs twice are both
    reported as VC_ERR_INVALID_ARG by vc_poll_status (also after vc_attn, whose attention launch
    must not wipe what the pass recorded); the gather clamps, so the call itself is harmless."""
    w, p, q, k, v, perm, quant, work, o = _case(bits, flags=vc.VC_FLAG_ALL | vc.VC_FLAG_CHECK_PERM)
    vc.vc_attn(p, q, k, v, perm, o, quant, work)
    vc.vc_poll_status(work)                                   # a good permutation passes
    good = o.clone()
    for bad_value, where in ((w.N + 5, (0, 1, 77)), (-3, (0, 0, 0)), (1 << 30, (0, 1, w.N - 1))):
        bad = perm.clone()
        bad[where] = bad_value
        vc.vc_attn(p, q, k, v, bad, o, quant, work)
        with pytest.raises(vc.VcError) as e:
            vc.vc_poll_status(work)
        assert e.value.code == vc.VC_ERR_INVALID_ARG
    dup = perm.clone()
    dup[0, 0, 10] = dup[0, 0, 11]                             # in range, but twice
    vc.vc_prep(p, q, k, v, dup, quant, work)
    with pytest.raises(vc.VcError) as e:
        vc.vc_poll_status(work)
    assert e.value.code == vc.VC_ERR_INVALID_ARG
    vc.vc_poll_status(work)                                   # polling cleared the word
    # without the flag nothing is checked and nothing is reported, but the gather still clamps
    p2 = Params.make(w.B, w.H, w.N, w.d, w.grid, bits=bits)
    quant2, work2 = alloc_buffers(p2)
    bad = perm.clone()
    bad[0, 1, 5] = w.N + 1000
    vc.vc_attn(p2, q, k, v, bad, o, quant2, work2)
    vc.vc_poll_status(work2)
    # and the next ordinary call is what it was before
    vc.vc_attn(p, q, k, v, perm, o, quant, work)
    vc.vc_poll_status(work)
    assert torch.equal(o, good)


ARRANGEMENTS = [(8, vc.VC_P_DEFAULT, 0), (8, vc.VC_P_DEFAULT, vc.VC_FLAG_INT8_QK), (8, vc.VC_P_EXP_E4M3, 0),
                (4, vc.VC_P_DEFAULT, 0), (4, vc.VC_P_EXPCAST_E4M3, 0)]


@pytest.mark.parametrize("bits,p_format,extra", ARRANGEMENTS, ids=["fp8", "int8qk", "exp_e4m3", "nvfp4", "hybrid4"])
def test_wait_that_runs_out_is_reported_and_leaves_the_library_usable(bits, p_format, extra):
    """Every mbarrier wait of the pipelined attention kernels is bounded.  With the limit cut to
    one poll, waits run out on a correct run: the kernel records VC_ERR_TIMEOUT, waits for its
    own copies and MMAs in flight, frees its tensor memory and returns.  The very next ordinary
    call must give bit for bit what it gave before."""
    w, p, q, k, v, perm, quant, work, o = _case(bits, p_format, vc.VC_FLAG_ALL | extra)
    vc.vc_attn(p, q, k, v, perm, o, quant, work)
    vc.vc_poll_status(work)
    before = o.clone()
    try:
        vc.vc_test_set_wait_limit(1)
        vc.vc_attn_fwd(p, quant, o, work)
        with pytest.raises(vc.VcError) as e:
            vc.vc_poll_status(work)
        assert e.value.code == vc.VC_ERR_TIMEOUT
    finally:
        vc.vc_test_set_wait_limit(0)
    vc.vc_poll_status(work)                                   # cleared
    o.zero_()
    vc.vc_attn_fwd(p, quant, o, work)
    vc.vc_poll_status(work)
    assert torch.equal(o, before)


def test_grouping_wait_that_runs_out_is_reported():
    """vc_group's waits report through the status word at the start of its workspace."""
    w, p, q, k, v, perm, quant, work, o = _case()
    gwork = torch.empty(vc.vc_group_workspace_bytes(p), dtype=torch.uint8, device="cuda")
    cent = torch.zeros(w.B, w.H, 16, w.d, dtype=torch.float32, device="cuda")
    out = torch.empty(w.B, w.H, w.N, dtype=torch.int32, device="cuda")
    vc.vc_group(p, v, 16, 2, False, cent, out, gwork)
    vc.vc_poll_status(gwork)
    good = out.clone()
    assert sorted(good[0, 0].tolist()) == list(range(w.N))
    try:
        vc.vc_test_set_wait_limit(1)
        vc.vc_group(p, v, 16, 2, False, cent, out, gwork)
        with pytest.raises(vc.VcError) as e:
            vc.vc_poll_status(gwork)
        assert e.value.code == vc.VC_ERR_TIMEOUT
    finally:
        vc.vc_test_set_wait_limit(0)
    vc.vc_group(p, v, 16, 2, False, cent, out, gwork)
    vc.vc_poll_status(gwork)
    assert torch.equal(out, good)
