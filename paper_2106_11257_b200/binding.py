"""ctypes binding of libbtard.so: same names as the C ABI, argument marshalling only.

Tensors are torch tensors (device memory and streams are torch's); every step of the computation
runs in the library's kernels.  Missing library => ImportError-like failure at first use, never a
fallback.
"""
import ctypes as C
import os

import numpy as np

INIT_CALLER_V0, INIT_ZERO, INIT_MEAN, INIT_COORD_MEDIAN = 0, 1, 2, 3
ALGO_DIRECT, ALGO_GRAM, ALGO_DIRECT_COOPERATIVE = 0, 1, 2
STOP_FIXED_ITERS, STOP_EPS = 0, 1
RULE_CENTERED_CLIP, RULE_GEOMETRIC_MEDIAN, RULE_MEAN, RULE_COORD_MEDIAN = 0, 1, 2, 3
SPLIT_PAPER, SPLIT_CEIL_PAD = 0, 1
STATUS_NOT_CONVERGED, STATUS_NONFINITE_ROW = 1, 2

EXPORTS = [
    "btard_partition_layout", "btard_centered_clip_workspace", "btard_centered_clip",
    "btard_verify_projections_workspace", "btard_verify_projections", "btard_random_vector",
    "btard_aggregate_host_scratch", "btard_aggregate_host", "btard_last_cuda_error",
    "btard_kernel_launch_count", "btard_profile_enable", "btard_profile_collect",
    "btard_verify_projections_static", "btard_verification_checks", "btard_preclip_workspace",
    "btard_preclip", "btard_split_gradients", "btard_merge_partitions",
    "btard_hash_partitions_workspace", "btard_hash_partitions", "btard_centered_clip_verify",
    "btard_preclip_factors",
]

_ERRORS = {-1: "invalid argument", -2: "bad alignment", -3: "workspace too small",
           -4: "CUDA error", -5: "unsupported"}


class BtardError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        extra = ""
        if code == -4:
            extra = " (cudaError %d)" % lib().btard_last_cuda_error()
        super().__init__("%s: %s%s" % (where, _ERRORS.get(code, "error %d" % code), extra))


class CclipArgs(C.Structure):
    _fields_ = [("n_peers", C.c_int32), ("n_partitions", C.c_int32), ("row_stride", C.c_int64),
                ("part_len", C.c_void_p), ("g", C.c_void_p), ("tau", C.c_void_p),
                ("init_mode", C.c_int32), ("algo", C.c_int32), ("stop_mode", C.c_int32),
                ("max_iters", C.c_int32), ("eps", C.c_double), ("v", C.c_void_p),
                ("iters", C.c_void_p), ("last_step_norm", C.c_void_p), ("resid_norm", C.c_void_p),
                ("status", C.c_void_p), ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
                ("stream", C.c_void_p), ("rule", C.c_int32), ("tau_schedule", C.c_void_p),
                ("row_scale", C.c_void_p)]


class VerifyArgs(C.Structure):
    _fields_ = [("n_peers", C.c_int32), ("n_partitions", C.c_int32), ("row_stride", C.c_int64),
                ("part_len", C.c_void_p), ("g", C.c_void_p), ("v", C.c_void_p), ("tau", C.c_void_p),
                ("seed", C.c_uint64), ("n_z", C.c_int32), ("partition_base", C.c_int32),
                ("resid_norm_in", C.c_void_p), ("norm", C.c_void_p), ("weight", C.c_void_p),
                ("dot", C.c_void_p), ("s", C.c_void_p), ("s_sum", C.c_void_p),
                ("znorm2", C.c_void_p), ("resid_sum_norm", C.c_void_p), ("resid_sum", C.c_void_p),
                ("status", C.c_void_p), ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
                ("stream", C.c_void_p), ("row_scale", C.c_void_p)]


class HostArgs(C.Structure):
    _fields_ = [("n_peers", C.c_int32), ("n_partitions", C.c_int32), ("row_stride", C.c_int64),
                ("part_len", C.c_void_p), ("tau", C.c_void_p), ("g", C.c_void_p),
                ("init_mode", C.c_int32), ("stop_mode", C.c_int32), ("max_iters", C.c_int32),
                ("eps", C.c_double), ("seed", C.c_uint64), ("n_z", C.c_int32), ("v", C.c_void_p),
                ("iters", C.c_void_p), ("last_step_norm", C.c_void_p), ("norm", C.c_void_p),
                ("weight", C.c_void_p), ("dot", C.c_void_p), ("s", C.c_void_p),
                ("s_sum", C.c_void_p), ("znorm2", C.c_void_p), ("resid_sum_norm", C.c_void_p),
                ("status", C.c_void_p), ("device_scratch", C.c_void_p),
                ("device_scratch_bytes", C.c_size_t), ("stream", C.c_void_p),
                ("copy_stream", C.c_void_p), ("algo", C.c_int32)]


class PreclipArgs(C.Structure):
    _fields_ = [("n_peers", C.c_int32), ("n_partitions", C.c_int32), ("row_stride", C.c_int64),
                ("part_len", C.c_void_p), ("lambda_", C.c_void_p), ("g", C.c_void_p),
                ("row_norm", C.c_void_p), ("factor", C.c_void_p), ("status", C.c_void_p),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t), ("stream", C.c_void_p)]


class ChecksArgs(C.Structure):
    _fields_ = [("n_peers", C.c_int32), ("n_partitions", C.c_int32), ("n_z", C.c_int32),
                ("norm", C.c_void_p), ("norm_reported", C.c_void_p), ("s", C.c_void_p),
                ("s_reported", C.c_void_p), ("delta_max", C.c_void_p), ("rel_tol", C.c_double),
                ("abs_tol", C.c_double), ("sum_tol", C.c_double), ("norm_mismatch", C.c_void_p),
                ("s_mismatch", C.c_void_p), ("sum_violation", C.c_void_p), ("check", C.c_void_p),
                ("votes", C.c_void_p), ("check_averaging", C.c_void_p), ("stream", C.c_void_p)]


_lib = None


def library_path():
    return os.path.join(os.path.dirname(os.path.abspath(__file__)), "libbtard.so")


def lib():
    """Loads libbtard.so (built by paper_2106_11257_b200/build.py); raises if it is missing."""
    global _lib
    if _lib is None:
        path = library_path()
        if not os.path.exists(path):
            raise OSError("libbtard.so is not built: run `python -m paper_2106_11257_b200.build` "
                          "(there is no CPU fallback)")
        L = C.CDLL(path)
        L.btard_partition_layout.restype = C.c_int
        L.btard_partition_layout.argtypes = [C.c_int64, C.c_int32, C.c_int32, C.c_int32,
                                             C.c_void_p, C.c_void_p, C.POINTER(C.c_int64)]
        L.btard_centered_clip_workspace.restype = C.c_size_t
        L.btard_centered_clip_workspace.argtypes = [C.POINTER(CclipArgs)]
        L.btard_centered_clip.restype = C.c_int
        L.btard_centered_clip.argtypes = [C.POINTER(CclipArgs)]
        L.btard_verify_projections_workspace.restype = C.c_size_t
        L.btard_verify_projections_workspace.argtypes = [C.POINTER(VerifyArgs)]
        L.btard_verify_projections.restype = C.c_int
        L.btard_verify_projections.argtypes = [C.POINTER(VerifyArgs)]
        L.btard_verify_projections_static.restype = C.c_int
        L.btard_verify_projections_static.argtypes = [C.POINTER(VerifyArgs)]
        L.btard_centered_clip_verify.restype = C.c_int
        L.btard_centered_clip_verify.argtypes = [C.POINTER(CclipArgs), C.POINTER(VerifyArgs)]
        L.btard_preclip_workspace.restype = C.c_size_t
        L.btard_preclip_workspace.argtypes = [C.POINTER(PreclipArgs)]
        L.btard_preclip.restype = C.c_int
        L.btard_preclip.argtypes = [C.POINTER(PreclipArgs)]
        L.btard_preclip_factors.restype = C.c_int
        L.btard_preclip_factors.argtypes = [C.POINTER(PreclipArgs)]
        L.btard_verification_checks.restype = C.c_int
        L.btard_verification_checks.argtypes = [C.POINTER(ChecksArgs)]
        L.btard_random_vector.restype = C.c_int
        L.btard_random_vector.argtypes = [C.c_uint64, C.c_int32, C.c_int32, C.c_int64, C.c_void_p,
                                          C.c_void_p]
        L.btard_aggregate_host_scratch.restype = C.c_size_t
        L.btard_aggregate_host_scratch.argtypes = [C.POINTER(HostArgs)]
        L.btard_aggregate_host.restype = C.c_int
        L.btard_aggregate_host.argtypes = [C.POINTER(HostArgs)]
        L.btard_last_cuda_error.restype = C.c_int
        L.btard_kernel_launch_count.restype = C.c_int64
        L.btard_profile_enable.restype = None
        L.btard_profile_enable.argtypes = [C.c_int]
        L.btard_profile_collect.restype = C.c_int
        L.btard_profile_collect.argtypes = [C.c_void_p, C.c_void_p, C.c_int32]
        _lib = L
    return _lib


def kernel_launch_count():
    return int(lib().btard_kernel_launch_count())


KERNEL_KINDS = ("median", "init", "iter", "verify", "other", "gram", "coef", "combine")


def profile_enable(on):
    lib().btard_profile_enable(1 if on else 0)


def profile_collect():
    """Returns {kind: (total_ms, launches)} for the kernels timed since the last call."""
    ms = np.zeros(len(KERNEL_KINDS), dtype=np.float64)
    cnt = np.zeros(len(KERNEL_KINDS), dtype=np.int64)
    _check(lib().btard_profile_collect(ms.ctypes.data, cnt.ctypes.data, len(KERNEL_KINDS)),
           "btard_profile_collect")
    return {k: (float(ms[i]), int(cnt[i])) for i, k in enumerate(KERNEL_KINDS)}


def last_cuda_error():
    return int(lib().btard_last_cuda_error())


def _check(rc, where):
    if rc != 0:
        raise BtardError(rc, where)


def partition_layout(d, P, mode=SPLIT_PAPER, align_elems=32):
    """Host-only.  Returns (part_offset[P], part_len[P], row_stride)."""
    off = np.zeros(P, dtype=np.int64)
    ln = np.zeros(P, dtype=np.int64)
    stride = C.c_int64(0)
    _check(lib().btard_partition_layout(int(d), int(P), int(mode), int(align_elems),
                                        off.ctypes.data, ln.ctypes.data, C.byref(stride)),
           "btard_partition_layout")
    return off, ln, int(stride.value)


def _torch():
    import torch
    return torch


def _stream_ptr(stream):
    torch = _torch()
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _host_arr(x, P, dtype):
    return np.ascontiguousarray(np.broadcast_to(np.asarray(x, dtype=dtype), (P,)))


def _dev_f64(t, shape):
    """Optional device float64 tensor of the given shape -> pointer (None stays None)."""
    if t is None:
        return None
    torch = _torch()
    assert t.is_cuda and t.dtype == torch.float64 and t.is_contiguous() and tuple(t.shape) == tuple(shape), shape
    return t.data_ptr()


def centered_clip_workspace(n, P, row_stride, stop_mode=STOP_EPS, algo=ALGO_DIRECT):
    a = CclipArgs(n_peers=n, n_partitions=P, row_stride=row_stride, stop_mode=stop_mode, algo=algo)
    return int(lib().btard_centered_clip_workspace(C.byref(a)))


def centered_clip(g, tau, part_len=None, init_mode=INIT_ZERO, v=None, stop_mode=STOP_FIXED_ITERS,
                  max_iters=1, eps=0.0, algo=ALGO_DIRECT, workspace=None, out=None, stream=None,
                  rule=RULE_CENTERED_CLIP, tau_schedule=None, row_scale=None):
    """g: CUDA float32 [P][n][row_stride].  Returns dict of CUDA tensors
    (v, iters, last_step_norm, resid_norm, status).  Asynchronous on the current stream.
    tau_schedule: CUDA float64 [P][max_iters] or None; row_scale: CUDA float64 [P][n] or None."""
    torch = _torch()
    assert g.is_cuda and g.dtype == torch.float32 and g.dim() == 3 and g.is_contiguous()
    P, n, stride = g.shape
    ln = _host_arr(stride if part_len is None else part_len, P, np.int64)
    tau_h = _host_arr(tau, P, np.float64)
    dev = g.device
    if v is None:
        assert init_mode != INIT_CALLER_V0, "CALLER_V0 needs v"
        v = torch.empty((P, stride), dtype=torch.float32, device=dev)
    assert v.is_cuda and v.dtype == torch.float32 and v.is_contiguous() and v.numel() == P * stride
    o = out if out is not None else dict(
        iters=torch.empty(P, dtype=torch.int32, device=dev),
        last_step_norm=torch.empty(P, dtype=torch.float64, device=dev),
        resid_norm=torch.empty((P, n), dtype=torch.float64, device=dev),
        status=torch.empty(P, dtype=torch.int32, device=dev))
    need = centered_clip_workspace(n, P, stride, stop_mode, algo)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=dev)
    a = CclipArgs(n_peers=n, n_partitions=P, row_stride=stride, part_len=ln.ctypes.data,
                  g=g.data_ptr(), tau=tau_h.ctypes.data, init_mode=init_mode, algo=algo,
                  stop_mode=stop_mode, max_iters=max_iters, eps=eps, v=v.data_ptr(),
                  iters=o["iters"].data_ptr(), last_step_norm=o["last_step_norm"].data_ptr(),
                  resid_norm=o["resid_norm"].data_ptr(), status=o["status"].data_ptr(),
                  workspace=workspace.data_ptr(), workspace_bytes=workspace.numel(),
                  stream=_stream_ptr(stream), rule=rule,
                  tau_schedule=_dev_f64(tau_schedule, (P, max_iters)), row_scale=_dev_f64(row_scale, (P, n)))
    with torch.cuda.device(dev):
        _check(lib().btard_centered_clip(C.byref(a)), "btard_centered_clip")
    res = dict(o)
    res["v"] = v
    res["workspace"] = workspace
    return res


def verify_projections_workspace(n, P, row_stride, K):
    a = VerifyArgs(n_peers=n, n_partitions=P, row_stride=row_stride, n_z=K)
    return int(lib().btard_verify_projections_workspace(C.byref(a)))


def verify_projections(g, v, tau, seed, K=1, part_len=None, resid_norm_in=None, partition_base=0,
                       want_resid_sum=False, workspace=None, out=None, stream=None, row_scale=None):
    """Returns dict of CUDA tensors: norm, weight [P][n]; dot, s [P][n][K]; s_sum, znorm2 [P][K];
    resid_sum_norm [P]; status [P]; resid_sum [P][row_stride] if asked."""
    torch = _torch()
    assert g.is_cuda and g.dtype == torch.float32 and g.dim() == 3 and g.is_contiguous()
    P, n, stride = g.shape
    assert v.is_cuda and v.dtype == torch.float32 and v.is_contiguous() and v.numel() == P * stride
    ln = _host_arr(stride if part_len is None else part_len, P, np.int64)
    tau_h = _host_arr(tau, P, np.float64)
    dev = g.device
    f64 = dict(dtype=torch.float64, device=dev)
    o = out if out is not None else dict(
        norm=torch.empty((P, n), **f64), weight=torch.empty((P, n), **f64),
        dot=torch.empty((P, n, K), **f64), s=torch.empty((P, n, K), **f64),
        s_sum=torch.empty((P, K), **f64), znorm2=torch.empty((P, K), **f64),
        resid_sum_norm=torch.empty(P, **f64), status=torch.empty(P, dtype=torch.int32, device=dev))
    rs = None
    if want_resid_sum:
        rs = o.get("resid_sum")
        if rs is None:
            rs = torch.zeros((P, stride), dtype=torch.float32, device=dev)
    need = verify_projections_workspace(n, P, stride, K)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=dev)
    if resid_norm_in is not None:
        assert resid_norm_in.is_cuda and resid_norm_in.dtype == torch.float64 and resid_norm_in.is_contiguous()
    a = VerifyArgs(n_peers=n, n_partitions=P, row_stride=stride, part_len=ln.ctypes.data,
                   g=g.data_ptr(), v=v.data_ptr(), tau=tau_h.ctypes.data, seed=int(seed), n_z=K,
                   partition_base=partition_base,
                   resid_norm_in=resid_norm_in.data_ptr() if resid_norm_in is not None else None,
                   norm=o["norm"].data_ptr(), weight=o["weight"].data_ptr(), dot=o["dot"].data_ptr(),
                   s=o["s"].data_ptr(), s_sum=o["s_sum"].data_ptr(), znorm2=o["znorm2"].data_ptr(),
                   resid_sum_norm=o["resid_sum_norm"].data_ptr(),
                   resid_sum=rs.data_ptr() if rs is not None else None, status=o["status"].data_ptr(),
                   workspace=workspace.data_ptr(), workspace_bytes=workspace.numel(),
                   stream=_stream_ptr(stream), row_scale=_dev_f64(row_scale, (P, n)))
    with torch.cuda.device(dev):
        _check(lib().btard_verify_projections(C.byref(a)), "btard_verify_projections")
    res = dict(o)
    if rs is not None:
        res["resid_sum"] = rs
    res["workspace"] = workspace
    return res


def centered_clip_verify(g, tau, seed, K=1, part_len=None, init_mode=INIT_ZERO, v=None,
                         stop_mode=STOP_FIXED_ITERS, max_iters=1, eps=0.0, algo=ALGO_DIRECT, partition_base=0,
                         want_resid_sum=False, workspaces=None, out=None, stream=None, tau_schedule=None,
                         row_scale=None):
    """btard_centered_clip_verify: aggregation and verification in one call.  Returns (clip, verify), the
    dicts that centered_clip and verify_projections return.  workspaces / out: optional pairs to reuse."""
    torch = _torch()
    assert g.is_cuda and g.dtype == torch.float32 and g.dim() == 3 and g.is_contiguous()
    P, n, stride = g.shape
    ln = _host_arr(stride if part_len is None else part_len, P, np.int64)
    tau_h = _host_arr(tau, P, np.float64)
    dev = g.device
    if v is None:
        assert init_mode != INIT_CALLER_V0, "CALLER_V0 needs v"
        v = torch.empty((P, stride), dtype=torch.float32, device=dev)
    assert v.is_cuda and v.dtype == torch.float32 and v.is_contiguous() and v.numel() == P * stride
    f64 = dict(dtype=torch.float64, device=dev)
    oc, ov = out if out is not None else (None, None)
    if oc is None:
        oc = dict(iters=torch.empty(P, dtype=torch.int32, device=dev), last_step_norm=torch.empty(P, **f64),
                  resid_norm=torch.empty((P, n), **f64), status=torch.empty(P, dtype=torch.int32, device=dev))
    if ov is None:
        ov = dict(norm=torch.empty((P, n), **f64), weight=torch.empty((P, n), **f64),
                  dot=torch.empty((P, n, K), **f64), s=torch.empty((P, n, K), **f64),
                  s_sum=torch.empty((P, K), **f64), znorm2=torch.empty((P, K), **f64),
                  resid_sum_norm=torch.empty(P, **f64), status=torch.empty(P, dtype=torch.int32, device=dev))
    rs = None
    if want_resid_sum:
        rs = ov.get("resid_sum")
        if rs is None:
            rs = torch.zeros((P, stride), dtype=torch.float32, device=dev)
    wc, wv = workspaces if workspaces is not None else (None, None)
    if wc is None:
        wc = torch.empty(centered_clip_workspace(n, P, stride, stop_mode, algo), dtype=torch.uint8, device=dev)
    if wv is None:
        wv = torch.empty(verify_projections_workspace(n, P, stride, K), dtype=torch.uint8, device=dev)
    ca = CclipArgs(n_peers=n, n_partitions=P, row_stride=stride, part_len=ln.ctypes.data,
                   g=g.data_ptr(), tau=tau_h.ctypes.data, init_mode=init_mode, algo=algo,
                   stop_mode=stop_mode, max_iters=max_iters, eps=eps, v=v.data_ptr(),
                   iters=oc["iters"].data_ptr(), last_step_norm=oc["last_step_norm"].data_ptr(),
                   resid_norm=oc["resid_norm"].data_ptr(), status=oc["status"].data_ptr(),
                   workspace=wc.data_ptr(), workspace_bytes=wc.numel(), stream=_stream_ptr(stream),
                   rule=RULE_CENTERED_CLIP, tau_schedule=_dev_f64(tau_schedule, (P, max_iters)),
                   row_scale=_dev_f64(row_scale, (P, n)))
    va = VerifyArgs(n_peers=n, n_partitions=P, row_stride=stride, seed=int(seed), n_z=K,
                    partition_base=partition_base,
                    norm=ov["norm"].data_ptr(), weight=ov["weight"].data_ptr(), dot=ov["dot"].data_ptr(),
                    s=ov["s"].data_ptr(), s_sum=ov["s_sum"].data_ptr(), znorm2=ov["znorm2"].data_ptr(),
                    resid_sum_norm=ov["resid_sum_norm"].data_ptr(),
                    resid_sum=rs.data_ptr() if rs is not None else None, status=ov["status"].data_ptr(),
                    workspace=wv.data_ptr(), workspace_bytes=wv.numel())
    with torch.cuda.device(dev):
        _check(lib().btard_centered_clip_verify(C.byref(ca), C.byref(va)), "btard_centered_clip_verify")
    rc, rv = dict(oc), dict(ov)
    rc["v"] = v
    rc["workspace"] = wc
    if rs is not None:
        rv["resid_sum"] = rs
    rv["workspace"] = wv
    return rc, rv


def verify_projections_static(g, v, tau, seed, K=1, part_len=None, resid_norm_in=None,
                              partition_base=0, want_resid_sum=False, out=None, stream=None, row_scale=None):
    """verify_projections for callers that cannot allocate device memory: the library's built-in
    scratch array is used instead of a workspace.  Pass `out` (pre-made output tensors, same keys as
    verify_projections returns) to keep this wrapper from allocating too; calls on one GPU must not
    overlap.  Raises BtardError("workspace too small") when the problem exceeds the built-in array."""
    torch = _torch()
    assert g.is_cuda and g.dtype == torch.float32 and g.dim() == 3 and g.is_contiguous()
    P, n, stride = g.shape
    assert v.is_cuda and v.dtype == torch.float32 and v.is_contiguous() and v.numel() == P * stride
    ln = _host_arr(stride if part_len is None else part_len, P, np.int64)
    tau_h = _host_arr(tau, P, np.float64)
    dev = g.device
    f64 = dict(dtype=torch.float64, device=dev)
    o = out if out is not None else dict(
        norm=torch.empty((P, n), **f64), weight=torch.empty((P, n), **f64),
        dot=torch.empty((P, n, K), **f64), s=torch.empty((P, n, K), **f64),
        s_sum=torch.empty((P, K), **f64), znorm2=torch.empty((P, K), **f64),
        resid_sum_norm=torch.empty(P, **f64), status=torch.empty(P, dtype=torch.int32, device=dev))
    rs = o.get("resid_sum") if want_resid_sum else None
    if want_resid_sum and rs is None:
        rs = torch.zeros((P, stride), dtype=torch.float32, device=dev)
    a = VerifyArgs(n_peers=n, n_partitions=P, row_stride=stride, part_len=ln.ctypes.data,
                   g=g.data_ptr(), v=v.data_ptr(), tau=tau_h.ctypes.data, seed=int(seed), n_z=K,
                   partition_base=partition_base,
                   resid_norm_in=resid_norm_in.data_ptr() if resid_norm_in is not None else None,
                   norm=o["norm"].data_ptr(), weight=o["weight"].data_ptr(), dot=o["dot"].data_ptr(),
                   s=o["s"].data_ptr(), s_sum=o["s_sum"].data_ptr(), znorm2=o["znorm2"].data_ptr(),
                   resid_sum_norm=o["resid_sum_norm"].data_ptr(),
                   resid_sum=rs.data_ptr() if rs is not None else None, status=o["status"].data_ptr(),
                   workspace=None, workspace_bytes=0, stream=_stream_ptr(stream),
                   row_scale=_dev_f64(row_scale, (P, n)))
    with torch.cuda.device(dev):
        _check(lib().btard_verify_projections_static(C.byref(a)), "btard_verify_projections_static")
    res = dict(o)
    if rs is not None:
        res["resid_sum"] = rs
    return res


def split_gradients(grads, P, mode=SPLIT_CEIL_PAD, align_elems=32, stream=None, layout=None):
    """grads: CUDA float32 [n][d] -> (g [P][n][row_stride], part_offset, part_len).
    layout: optional (part_offset, part_len, row_stride) to use instead of btard_partition_layout's, one entry
    per slab in the order the slabs are wanted (a permutation of the parts, for instance)."""
    torch = _torch()
    assert grads.is_cuda and grads.dtype == torch.float32 and grads.dim() == 2 and grads.is_contiguous()
    n, d = grads.shape
    if layout is None:
        off, ln, stride = partition_layout(d, P, mode, align_elems)
    else:
        off = np.ascontiguousarray(layout[0], dtype=np.int64)
        ln = np.ascontiguousarray(layout[1], dtype=np.int64)
        stride = int(layout[2])
        assert off.shape == (P,) and ln.shape == (P,)
    g = torch.empty((P, n, stride), dtype=torch.float32, device=grads.device)
    table = torch.empty(16 * P, dtype=torch.uint8, device=grads.device)
    L = lib()
    L.btard_split_gradients.restype = C.c_int
    L.btard_split_gradients.argtypes = [C.c_int64, C.c_int32, C.c_int32, C.c_int64, C.c_void_p, C.c_void_p,
                                        C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    with torch.cuda.device(grads.device):
        _check(L.btard_split_gradients(d, n, P, stride, off.ctypes.data, ln.ctypes.data, grads.data_ptr(),
                                       g.data_ptr(), table.data_ptr(), _stream_ptr(stream)),
               "btard_split_gradients")
    return g, off, ln


def merge_partitions(v, d, part_offset, part_len, stream=None):
    """v: CUDA float32 [P][row_stride] -> out [d]."""
    torch = _torch()
    assert v.is_cuda and v.dtype == torch.float32 and v.dim() == 2 and v.is_contiguous()
    P, stride = v.shape
    out = torch.empty(d, dtype=torch.float32, device=v.device)
    table = torch.empty(16 * P, dtype=torch.uint8, device=v.device)
    off = np.ascontiguousarray(part_offset, dtype=np.int64)
    ln = np.ascontiguousarray(part_len, dtype=np.int64)
    L = lib()
    L.btard_merge_partitions.restype = C.c_int
    L.btard_merge_partitions.argtypes = [C.c_int64, C.c_int32, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p,
                                         C.c_void_p, C.c_void_p, C.c_void_p]
    with torch.cuda.device(v.device):
        _check(L.btard_merge_partitions(d, P, stride, off.ctypes.data, ln.ctypes.data, v.data_ptr(),
                                        out.data_ptr(), table.data_ptr(), _stream_ptr(stream)),
               "btard_merge_partitions")
    return out


def hash_partitions(x, part_len=None, stream=None):
    """Tree SHA-256 commitment of every row of a CUDA float32 tensor [P][rows][row_stride] (g) or
    [P][row_stride] (v).  Returns a CUDA uint8 tensor [P][rows][32]."""
    torch = _torch()
    if x.dim() == 2:
        x = x.unsqueeze(1)
    assert x.is_cuda and x.dtype == torch.float32 and x.dim() == 3 and x.is_contiguous()
    P, rows, stride = x.shape
    ln = _host_arr(stride if part_len is None else part_len, P, np.int64)
    L = lib()
    L.btard_hash_partitions_workspace.restype = C.c_size_t
    L.btard_hash_partitions_workspace.argtypes = [C.c_int32, C.c_int32, C.c_int64]
    L.btard_hash_partitions.restype = C.c_int
    L.btard_hash_partitions.argtypes = [C.c_int32, C.c_int32, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p,
                                        C.c_void_p, C.c_size_t, C.c_void_p]
    ws = torch.empty(int(L.btard_hash_partitions_workspace(P, rows, stride)), dtype=torch.uint8, device=x.device)
    out = torch.empty((P, rows, 32), dtype=torch.uint8, device=x.device)
    with torch.cuda.device(x.device):
        _check(L.btard_hash_partitions(P, rows, stride, ln.ctypes.data, x.data_ptr(), out.data_ptr(),
                                       ws.data_ptr(), ws.numel(), _stream_ptr(stream)), "btard_hash_partitions")
    return out


def preclip(g, lam, part_len=None, stream=None, in_place=True):
    """Per-part clipping g_i(l) <- min{1, lam/||g_i(l)||} g_i(l) of a CUDA float32 tensor
    [P][n][row_stride]: in place, or (in_place=False, btard_preclip_factors) only the norms and the
    factors, to be handed to centered_clip / verify_projections as row_scale.
    Returns dict(row_norm, factor [P][n] float64, status [P])."""
    torch = _torch()
    assert g.is_cuda and g.dtype == torch.float32 and g.dim() == 3 and g.is_contiguous()
    P, n, stride = g.shape
    ln = _host_arr(stride if part_len is None else part_len, P, np.int64)
    lam_h = _host_arr(lam, P, np.float64)
    dev = g.device
    o = dict(row_norm=torch.empty((P, n), dtype=torch.float64, device=dev),
             factor=torch.empty((P, n), dtype=torch.float64, device=dev),
             status=torch.empty(P, dtype=torch.int32, device=dev))
    a = PreclipArgs(n_peers=n, n_partitions=P, row_stride=stride, part_len=ln.ctypes.data,
                    lambda_=lam_h.ctypes.data, g=g.data_ptr(), row_norm=o["row_norm"].data_ptr(),
                    factor=o["factor"].data_ptr(), status=o["status"].data_ptr(), stream=_stream_ptr(stream))
    need = int(lib().btard_preclip_workspace(C.byref(a)))
    ws = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
    a.workspace = ws.data_ptr()
    a.workspace_bytes = ws.numel()
    with torch.cuda.device(dev):
        if in_place:
            _check(lib().btard_preclip(C.byref(a)), "btard_preclip")
        else:
            _check(lib().btard_preclip_factors(C.byref(a)), "btard_preclip_factors")
    o["workspace"] = ws
    return o


def verification_checks(norm, s, delta_max, norm_reported=None, s_reported=None, rel_tol=0.0,
                        abs_tol=0.0, sum_tol=0.0, stream=None):
    """Predicates of Verifications 1-3 on CUDA float64 tensors norm [P][n], s [P][n][K], delta_max [P].
    Returns dict of CUDA tensors: norm_mismatch, check [P][n] uint8; s_mismatch [P][n][K] uint8;
    sum_violation [P][K] uint8; votes [P] int32; check_averaging [P] uint8."""
    torch = _torch()
    P, n, K = s.shape
    dev = s.device
    for t in (norm, s, delta_max, norm_reported, s_reported):
        assert t is None or (t.is_cuda and t.dtype == torch.float64 and t.is_contiguous())
    u8 = dict(dtype=torch.uint8, device=dev)
    o = dict(norm_mismatch=torch.empty((P, n), **u8), s_mismatch=torch.empty((P, n, K), **u8),
             sum_violation=torch.empty((P, K), **u8), check=torch.empty((P, n), **u8),
             votes=torch.empty(P, dtype=torch.int32, device=dev), check_averaging=torch.empty(P, **u8))
    a = ChecksArgs(n_peers=n, n_partitions=P, n_z=K, norm=norm.data_ptr(),
                   norm_reported=norm_reported.data_ptr() if norm_reported is not None else None,
                   s=s.data_ptr(), s_reported=s_reported.data_ptr() if s_reported is not None else None,
                   delta_max=delta_max.data_ptr(), rel_tol=rel_tol, abs_tol=abs_tol, sum_tol=sum_tol,
                   norm_mismatch=o["norm_mismatch"].data_ptr(), s_mismatch=o["s_mismatch"].data_ptr(),
                   sum_violation=o["sum_violation"].data_ptr(), check=o["check"].data_ptr(),
                   votes=o["votes"].data_ptr(), check_averaging=o["check_averaging"].data_ptr(),
                   stream=_stream_ptr(stream))
    with torch.cuda.device(dev):
        _check(lib().btard_verification_checks(C.byref(a)), "btard_verification_checks")
    return o


def random_vector(seed, p, k, part_len, device="cuda", stream=None):
    """Unnormalised fp32 z_k of partition p as a CUDA tensor of part_len entries."""
    torch = _torch()
    padded = (int(part_len) + 3) // 4 * 4
    z = torch.zeros(max(padded, 4), dtype=torch.float32, device=device)
    with torch.cuda.device(z.device):
        _check(lib().btard_random_vector(int(seed), int(p), int(k), int(part_len), z.data_ptr(),
                                         _stream_ptr(stream)), "btard_random_vector")
    return z[:int(part_len)]


def aggregate_host_scratch(n, P, row_stride, K, algo=ALGO_DIRECT):
    a = HostArgs(n_peers=n, n_partitions=P, row_stride=row_stride, n_z=K, algo=algo)
    return int(lib().btard_aggregate_host_scratch(C.byref(a)))


def aggregate_host(g_host, tau, seed, K=1, part_len=None, init_mode=INIT_COORD_MEDIAN, v_host=None,
                   stop_mode=STOP_FIXED_ITERS, max_iters=1, eps=0.0, scratch=None, out=None,
                   device="cuda", stream=None, copy_stream=None, algo=ALGO_DIRECT):
    """Whole aggregation + verification from HOST tensors (ideally pinned); blocks until done.
    `copy_stream` (a second torch.cuda.Stream) lets the host-to-device copy of the next chunk of
    partitions overlap the kernels of the current one.  Returns dict of host tensors."""
    torch = _torch()
    assert not g_host.is_cuda and g_host.dtype == torch.float32 and g_host.dim() == 3 and g_host.is_contiguous()
    P, n, stride = g_host.shape
    ln = _host_arr(stride if part_len is None else part_len, P, np.int64)
    tau_h = _host_arr(tau, P, np.float64)
    pin = g_host.is_pinned()

    def host(shape, dtype):
        return torch.empty(shape, dtype=dtype, pin_memory=pin)
    o = out if out is not None else dict(
        v=v_host if v_host is not None else host((P, stride), torch.float32),
        iters=host(P, torch.int32), last_step_norm=host(P, torch.float64),
        norm=host((P, n), torch.float64), weight=host((P, n), torch.float64),
        dot=host((P, n, K), torch.float64), s=host((P, n, K), torch.float64),
        s_sum=host((P, K), torch.float64), znorm2=host((P, K), torch.float64),
        resid_sum_norm=host(P, torch.float64), status=host(P, torch.int32))
    need = aggregate_host_scratch(n, P, stride, K, algo)
    if scratch is None:
        scratch = torch.empty(need, dtype=torch.uint8, device=device)
    a = HostArgs(n_peers=n, n_partitions=P, row_stride=stride, part_len=ln.ctypes.data,
                 tau=tau_h.ctypes.data, g=g_host.data_ptr(), init_mode=init_mode,
                 stop_mode=stop_mode, max_iters=max_iters, eps=eps, seed=int(seed), n_z=K,
                 v=o["v"].data_ptr(), iters=o["iters"].data_ptr(),
                 last_step_norm=o["last_step_norm"].data_ptr(), norm=o["norm"].data_ptr(),
                 weight=o["weight"].data_ptr(), dot=o["dot"].data_ptr(), s=o["s"].data_ptr(),
                 s_sum=o["s_sum"].data_ptr(), znorm2=o["znorm2"].data_ptr(),
                 resid_sum_norm=o["resid_sum_norm"].data_ptr(), status=o["status"].data_ptr(),
                 device_scratch=scratch.data_ptr(), device_scratch_bytes=scratch.numel(),
                 stream=_stream_ptr(stream),
                 copy_stream=C.c_void_p(copy_stream.cuda_stream) if copy_stream is not None else None,
                 algo=algo)
    with torch.cuda.device(scratch.device):
        _check(lib().btard_aggregate_host(C.byref(a)), "btard_aggregate_host")
    res = dict(o)
    res["scratch"] = scratch
    return res
