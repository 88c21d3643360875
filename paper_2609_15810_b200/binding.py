"""ctypes binding with the same names as the C ABI in include/vc_attn.h.

Argument marshalling only: tensors become raw device (or host) pointers, the current
PyTorch CUDA stream becomes the `stream` argument, status codes other than VC_OK raise
VcError.  Buffers are allocated by the caller (helpers below size them).
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libvc.so")

VC_P_DEFAULT, VC_P_EXPCAST_E4M3, VC_P_EXP_E4M3, VC_P_NVFP4 = 0, 1, 2, 3
VC_P_EXP_POLY_E4M3, VC_P_EXP_MIX_E4M3 = 4, 5
VC_FLAG_ROPE, VC_FLAG_HADAMARD, VC_FLAG_K_SMOOTH, VC_FLAG_V_SMOOTH, VC_FLAG_ALL = 1, 2, 4, 8, 15
VC_FLAG_INT8_QK = 16
VC_FLAG_CHECK_PERM = 32
VC_GROUP_LABELS_OFFSET = 1024
VC_OK, VC_ERR_INVALID_ARG, VC_ERR_UNSUPPORTED, VC_ERR_WORKSPACE, VC_ERR_CUDA, VC_ERR_TIMEOUT, VC_ERR_SCRATCH_LIMIT = range(7)


class VcError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {vc_status_string(code)} (status {code})")


class Params(ctypes.Structure):
    """Mirror of vc_params."""
    _fields_ = [("B", ctypes.c_int32), ("H", ctypes.c_int32), ("N", ctypes.c_int32), ("d", ctypes.c_int32),
                ("grid_t", ctypes.c_int32), ("grid_h", ctypes.c_int32), ("grid_w", ctypes.c_int32),
                ("bits", ctypes.c_int32), ("p_format", ctypes.c_int32), ("flags", ctypes.c_int32),
                ("softmax_scale", ctypes.c_float), ("beta", ctypes.c_float),
                ("rope_dim_t", ctypes.c_int32), ("rope_dim_h", ctypes.c_int32), ("rope_dim_w", ctypes.c_int32),
                ("rope_theta", ctypes.c_float),
                ("stride_b", ctypes.c_int64), ("stride_h", ctypes.c_int64), ("stride_n", ctypes.c_int64),
                ("heads_per_pass", ctypes.c_int32), ("kernel_variant", ctypes.c_int32),
                ("block_q", ctypes.c_int32), ("block_k", ctypes.c_int32), ("block_v", ctypes.c_int32)]

    @classmethod
    def make(cls, B, H, N, d, grid, bits=8, p_format=VC_P_DEFAULT, flags=VC_FLAG_ALL, **kw):
        p = cls(B=B, H=H, N=N, d=d, grid_t=grid[0], grid_h=grid[1], grid_w=grid[2], bits=bits,
                p_format=p_format, flags=flags)
        for k, v in kw.items():
            setattr(p, k, v)
        return p


class QuantView(ctypes.Structure):
    """Mirror of vc_quant_ptrs."""
    _fields_ = ([(n, ctypes.c_void_p) for n in ("q_codes", "k_codes", "v_codes", "q_scale", "k_scale", "v_scale",
                                                "v_means", "k_mean", "q_micro", "k_micro", "v_micro")] +
                [(n + "_bytes", ctypes.c_size_t) for n in ("q_codes", "k_codes", "v_codes", "q_scale", "k_scale",
                                                           "v_scale", "v_means", "k_mean", "q_micro", "k_micro",
                                                           "v_micro")])


class PrepStats(ctypes.Structure):
    """Mirror of vc_prep_stats (device pointers)."""
    _fields_ = [("k_mean", ctypes.c_void_p), ("v_block_mean", ctypes.c_void_p), ("v_amax", ctypes.c_void_p)]


_lib = None


def load_library():
    """Loads libvc.so (built in-tree); raises if it is missing -- there is no fallback."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} not found: build it with `python -m paper_2609_15810_b200.build`")
    lib = ctypes.CDLL(_LIB_PATH)
    P, vp, i32p = ctypes.POINTER(Params), ctypes.c_void_p, ctypes.c_void_p
    lib.vc_quant_bytes.restype = ctypes.c_size_t
    lib.vc_quant_bytes.argtypes = [P]
    lib.vc_workspace_bytes.restype = ctypes.c_size_t
    lib.vc_workspace_bytes.argtypes = [P]
    lib.vc_prep.restype = ctypes.c_int
    lib.vc_prep.argtypes = [P, vp, vp, vp, i32p, vp, vp, vp]
    lib.vc_prep_with_stats.restype = ctypes.c_int
    lib.vc_prep_with_stats.argtypes = [P, vp, vp, vp, i32p, ctypes.POINTER(PrepStats), vp, vp, vp]
    lib.vc_prep_stats_view.restype = ctypes.c_int
    lib.vc_prep_stats_view.argtypes = [P, vp, vp, ctypes.POINTER(PrepStats)]
    lib.vc_prep_noalloc.restype = ctypes.c_int
    lib.vc_prep_noalloc.argtypes = [P, vp, vp, vp, i32p, vp, vp]
    lib.vc_attn_fwd.restype = ctypes.c_int
    lib.vc_attn_fwd.argtypes = [P, vp, vp, vp, vp]
    lib.vc_attn.restype = ctypes.c_int
    lib.vc_attn.argtypes = [P, vp, vp, vp, i32p, vp, vp, vp, vp]
    lib.vc_attn_host.restype = ctypes.c_int
    lib.vc_attn_host.argtypes = [P] + [vp] * 13
    lib.vc_group_workspace_bytes.restype = ctypes.c_size_t
    lib.vc_group_workspace_bytes.argtypes = [P]
    lib.vc_group.restype = ctypes.c_int
    lib.vc_group.argtypes = [P, vp, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, vp, i32p, vp, vp]
    lib.vc_group_schedule.restype = ctypes.c_int32
    lib.vc_group_schedule.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.c_int32]
    lib.vc_quant_view.restype = ctypes.c_int
    lib.vc_quant_view.argtypes = [P, vp, ctypes.POINTER(QuantView)]
    lib.vc_poll_status.restype = ctypes.c_int
    lib.vc_poll_status.argtypes = [vp, vp]
    lib.vc_test_set_wait_limit.restype = None
    lib.vc_test_set_wait_limit.argtypes = [ctypes.c_uint32]
    lib.vc_test_expcast_codes.restype = ctypes.c_int
    lib.vc_test_expcast_codes.argtypes = [vp, ctypes.c_int64, ctypes.c_float, ctypes.c_float, ctypes.c_float, vp, vp]
    lib.vc_mma_peak.restype = ctypes.c_int
    lib.vc_mma_peak.argtypes = [ctypes.c_int32, ctypes.c_int32, vp, ctypes.POINTER(ctypes.c_double),
                                ctypes.POINTER(ctypes.c_double), vp]
    lib.vc_launch_count.restype = ctypes.c_uint64
    lib.vc_launch_count.argtypes = []
    lib.vc_status_string.restype = ctypes.c_char_p
    lib.vc_status_string.argtypes = [ctypes.c_int]
    _lib = lib
    return lib


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_contiguous() or t.dim() == 4, "pass strides through Params for non-packed inputs"
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def _check(code, where):
    if code != 0:
        raise VcError(code, where)


def vc_status_string(code):
    return load_library().vc_status_string(int(code)).decode()


def vc_quant_bytes(p):
    return int(load_library().vc_quant_bytes(ctypes.byref(p)))


def vc_workspace_bytes(p):
    return int(load_library().vc_workspace_bytes(ctypes.byref(p)))


def vc_prep(p, q, k, v, perm, quant, workspace):
    _check(load_library().vc_prep(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(perm), _ptr(quant),
                                  _ptr(workspace), _stream()), "vc_prep")


def vc_prep_with_stats(p, q, k, v, perm, k_mean, v_block_mean, v_amax, quant, workspace):
    """vc_prep with the statistics supplied by the caller (fp32 device tensors): no statistics launches."""
    st = PrepStats(_ptr(k_mean), _ptr(v_block_mean), _ptr(v_amax))
    _check(load_library().vc_prep_with_stats(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(perm), ctypes.byref(st),
                                             _ptr(quant), _ptr(workspace), _stream()), "vc_prep_with_stats")


def vc_prep_stats_view(p, quant, workspace):
    """(k_mean [BH, d], v_block_mean [BH, nb, d], v_amax [BH, d]) fp32 tensors aliasing where vc_prep left them."""
    st = PrepStats()
    _check(load_library().vc_prep_stats_view(ctypes.byref(p), _ptr(quant), _ptr(workspace), ctypes.byref(st)), "vc_prep_stats_view")
    BH, d, nb = p.B * p.H, p.d, (p.N + 127) // 128
    def alias(ptr, base, n):
        off = ptr - base.data_ptr()
        return base[off:off + 4 * n].view(torch.float32)
    return (alias(st.k_mean, quant, BH * d).view(BH, d), alias(st.v_block_mean, workspace, BH * nb * d).view(BH, nb, d),
            alias(st.v_amax, workspace, BH * d).view(BH, d))


def vc_prep_noalloc(p, q, k, v, perm, quant):
    """vc_prep on the library's built-in scratch array: no workspace, no allocation (size-limited)."""
    _check(load_library().vc_prep_noalloc(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(perm), _ptr(quant),
                                          _stream()), "vc_prep_noalloc")


def vc_attn_fwd(p, quant, o, workspace):
    _check(load_library().vc_attn_fwd(ctypes.byref(p), _ptr(quant), _ptr(o), _ptr(workspace), _stream()),
           "vc_attn_fwd")


def vc_attn(p, q, k, v, perm, o, quant, workspace):
    _check(load_library().vc_attn(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(perm), _ptr(o), _ptr(quant),
                                  _ptr(workspace), _stream()), "vc_attn")


def vc_attn_host(p, q_host, k_host, v_host, perm_host, o_host, q_dev, k_dev, v_dev, perm_dev, o_dev, quant,
                 workspace):
    _check(load_library().vc_attn_host(ctypes.byref(p), _ptr(q_host), _ptr(k_host), _ptr(v_host), _ptr(perm_host),
                                       _ptr(o_host), _ptr(q_dev), _ptr(k_dev), _ptr(v_dev), _ptr(perm_dev),
                                       _ptr(o_dev), _ptr(quant), _ptr(workspace), _stream()), "vc_attn_host")


def vc_group_workspace_bytes(p):
    return int(load_library().vc_group_workspace_bytes(ctypes.byref(p)))


def vc_group(p, v, k, iters, warm_start, centroids, perm, workspace):
    """k-means on the value tokens -> perm = stable argsort of the labels (centroids in/out)."""
    _check(load_library().vc_group(ctypes.byref(p), _ptr(v), int(k), int(iters), int(bool(warm_start)), _ptr(centroids),
                                   _ptr(perm), _ptr(workspace), _stream()), "vc_group")


VC_GROUP_RECOMPUTE, VC_GROUP_REUSE, VC_GROUP_FROZEN = 0, 1, 2


def vc_group_schedule(step, n_steps, reuse=4):
    """What the step-indexed grouping schedule asks for at denoising step `step` of `n_steps`."""
    return int(load_library().vc_group_schedule(int(step), int(n_steps), int(reuse)))


def vc_quant_view(p, quant):
    out = QuantView()
    _check(load_library().vc_quant_view(ctypes.byref(p), _ptr(quant), ctypes.byref(out)), "vc_quant_view")
    return out


def vc_poll_status(workspace):
    _check(load_library().vc_poll_status(_ptr(workspace), _stream()), "vc_poll_status")


def vc_test_set_wait_limit(polls):
    """Test hook: polls after which a device-side wait gives up (0 = the default)."""
    load_library().vc_test_set_wait_limit(int(polls))


def vc_test_expcast_codes(s, cs, m, beta=0.0):
    """Test hook: the ExpCast-FP8 codes of the fp32 scores `s` (CUDA tensor, numel a multiple of 4)
    under the factor cs and the running maximum m, as the attention kernels form them (uint8 tensor)."""
    assert s.dtype == torch.float32 and s.is_cuda and s.is_contiguous()
    out = torch.empty(s.numel(), dtype=torch.uint8, device=s.device)
    _check(load_library().vc_test_expcast_codes(_ptr(s), s.numel(), float(cs), float(m), float(beta), _ptr(out), _stream()),
           "vc_test_expcast_codes")
    return out.view(s.shape)


def vc_mma_peak(kind, groups=4096):
    """(TFLOP/s over the whole GPU, MAC per clock per SM) of back-to-back MMAs of one kind (8 or 4)."""
    scratch = torch.zeros(1, dtype=torch.int64, device="cuda")
    tf, mac = ctypes.c_double(0.0), ctypes.c_double(0.0)
    _check(load_library().vc_mma_peak(int(kind), int(groups), _ptr(scratch), ctypes.byref(tf), ctypes.byref(mac), _stream()),
           "vc_mma_peak")
    return tf.value, mac.value


def vc_launch_count():
    return int(load_library().vc_launch_count())


# ----------------------------------------------------------------------------- conveniences
def alloc_buffers(p, device="cuda"):
    """(quant, workspace) uint8 tensors of the sizes the library asks for."""
    qb, wb = vc_quant_bytes(p), vc_workspace_bytes(p)
    if qb == 0 or wb == 0:
        raise VcError(1, "alloc_buffers")
    return (torch.empty(qb, dtype=torch.uint8, device=device), torch.empty(wb, dtype=torch.uint8, device=device))


def section(view, name, quant, dtype=torch.uint8):
    """A tensor aliasing one section of the bundle (for tests)."""
    off = getattr(view, name) - quant.data_ptr()
    nbytes = getattr(view, name + "_bytes")
    return quant[off:off + nbytes].view(dtype)
