"""ctypes front end of the float64 CPU oracle (test infrastructure only).

Each function marshals numpy arrays to ``btard_oracle.c`` and returns numpy
arrays; no arithmetic of the method is done in Python.
"""
import ctypes as C
import os
import subprocess
import threading

import numpy as np

INIT_CALLER, INIT_ZERO, INIT_MEAN, INIT_COORD_MEDIAN = 0, 1, 2, 3
STOP_FIXED, STOP_EPS = 0, 1
SPLIT_PAPER, SPLIT_CEIL_PAD = 0, 1
STATUS_NOT_CONVERGED, STATUS_NONFINITE_ROW = 1, 2
RULE_CENTERED_CLIP, RULE_GEOMETRIC_MEDIAN, RULE_MEAN, RULE_COORD_MEDIAN = 0, 1, 2, 3

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "btard_oracle.c")
_LIB = os.path.join(_HERE, "libbtard_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force=False):
    """Compile the oracle with gcc (no fast-math, no fp contraction)."""
    if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC):
        return _LIB
    tmp = _LIB + ".tmp%d" % os.getpid()
    cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
           "-fno-fast-math", "-Wall", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            _lib = C.CDLL(build())
            _lib.btard_oracle_max_threads.restype = C.c_int
    return _lib


def _p(a, ty):
    return a.ctypes.data_as(C.POINTER(ty)) if a is not None else None


def max_threads():
    return int(_load().btard_oracle_max_threads())


def philox4x32_10(ctr, key):
    """One Philox4x32-10 block: 4 counter words, 2 key words -> 4 output words."""
    c = np.ascontiguousarray(ctr, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    _load().btard_oracle_philox4x32_10(_p(c, C.c_uint32), _p(k, C.c_uint32), _p(out, C.c_uint32))
    return out


def random_vector(seed, p, k, part_len):
    """Unnormalised fp32 coordinates of z_k for partition p."""
    z = np.zeros(int(part_len), dtype=np.float32)
    _load().btard_oracle_random_vector(C.c_uint64(int(seed)), C.c_int32(p), C.c_int32(k),
                                       C.c_int64(int(part_len)), _p(z, C.c_float))
    return z


def partition_layout(d, P, mode=SPLIT_PAPER, align_elems=32):
    off = np.zeros(P, dtype=np.int64)
    ln = np.zeros(P, dtype=np.int64)
    stride = C.c_int64(0)
    rc = _load().btard_oracle_partition_layout(C.c_int64(int(d)), C.c_int32(P), C.c_int32(mode),
                                               C.c_int32(align_elems), _p(off, C.c_int64),
                                               _p(ln, C.c_int64), C.byref(stride))
    if rc:
        raise ValueError("partition_layout: invalid argument")
    return off, ln, int(stride.value)


def _as_g(g):
    g = np.ascontiguousarray(g, dtype=np.float32)
    if g.ndim == 2:
        g = g[None]
    assert g.ndim == 3, "g must be [P][n][stride]"
    return g


def _per_part(x, P, dtype):
    a = np.ascontiguousarray(np.broadcast_to(np.asarray(x, dtype=dtype), (P,)))
    return a


def centered_clip(g, tau, part_len=None, init_mode=INIT_ZERO, v0=None, stop_mode=STOP_FIXED,
                  max_iters=1, eps=0.0, rule=RULE_CENTERED_CLIP, tau_schedule=None, row_scale=None):
    """Batched CenteredClip.  g: [P][n][stride] fp32 (or [n][stride]).

    tau_schedule [P][max_iters]: the radius of update l (tau_l of App. D.2) instead of the constant tau.
    row_scale [P][n]: row i enters as row_scale[p][i] * g[p][i] (the clipped gradients of Alg. 9).
    Returns dict(v [P][stride] f64, resid_norm [P][n], iters [P], last_step_norm [P], status [P]).
    """
    g = _as_g(g)
    P, n, stride = g.shape
    ln = _per_part(stride if part_len is None else part_len, P, np.int64)
    tau = _per_part(tau, P, np.float64)
    if v0 is not None:
        v0 = np.ascontiguousarray(v0, dtype=np.float32).reshape(P, stride)
    if tau_schedule is not None:
        tau_schedule = np.ascontiguousarray(np.broadcast_to(np.asarray(tau_schedule, np.float64), (P, max_iters)))
    if row_scale is not None:
        row_scale = np.ascontiguousarray(np.asarray(row_scale, np.float64).reshape(P, n))
    v = np.zeros((P, stride), dtype=np.float64)
    rn = np.zeros((P, n), dtype=np.float64)
    it = np.zeros(P, dtype=np.int32)
    ls = np.zeros(P, dtype=np.float64)
    st = np.zeros(P, dtype=np.uint32)
    rc = _load().btard_oracle_aggregate_ex(
        C.c_int32(rule), _p(g, C.c_float), C.c_int32(n), C.c_int32(P), C.c_int64(stride), _p(ln, C.c_int64),
        _p(tau, C.c_double), _p(tau_schedule, C.c_double), _p(row_scale, C.c_double),
        C.c_int32(init_mode), _p(v0, C.c_float), C.c_int32(stop_mode),
        C.c_int32(max_iters), C.c_double(eps), _p(v, C.c_double), _p(rn, C.c_double),
        _p(it, C.c_int32), _p(ls, C.c_double), _p(st, C.c_uint32))
    if rc:
        raise ValueError("centered_clip: invalid argument")
    return dict(v=v, resid_norm=rn, iters=it, last_step_norm=ls, status=st)


def verify(g, v, tau, seed, K=1, part_len=None, norm_in=None, want_resid_sum=False,
           first_partition=0, row_scale=None):
    """Batched verification metadata.  v: [P][stride] fp32 (the vector a peer received).

    ``first_partition`` shifts the partition index that keys the z stream, so that a
    slab cut out of a larger tensor is verified with the z of its true position.
    """
    g = _as_g(g)
    P, n, stride = g.shape
    v = np.ascontiguousarray(v, dtype=np.float32).reshape(P, stride)
    ln = _per_part(stride if part_len is None else part_len, P, np.int64)
    tau = _per_part(tau, P, np.float64)
    if norm_in is not None:
        norm_in = np.ascontiguousarray(norm_in, dtype=np.float64).reshape(P, n)
    out = dict(norm=np.zeros((P, n)), weight=np.zeros((P, n)), dot=np.zeros((P, n, K)),
               s=np.zeros((P, n, K)), s_sum=np.zeros((P, K)), znorm2=np.zeros((P, K)),
               resid_sum_norm=np.zeros(P), status=np.zeros(P, dtype=np.uint32))
    rs = np.zeros((P, stride)) if want_resid_sum else None
    lib = _load()
    if row_scale is not None:
        row_scale = np.ascontiguousarray(np.asarray(row_scale, np.float64).reshape(P, n))
    if first_partition == 0 and row_scale is None:
        rc = lib.btard_oracle_verify(
            _p(g, C.c_float), C.c_int32(n), C.c_int32(P), C.c_int64(stride), _p(ln, C.c_int64),
            _p(v, C.c_float), _p(tau, C.c_double), C.c_uint64(int(seed)), C.c_int32(K),
            _p(norm_in, C.c_double), _p(out["norm"], C.c_double), _p(out["weight"], C.c_double),
            _p(out["dot"], C.c_double), _p(out["s"], C.c_double), _p(out["s_sum"], C.c_double),
            _p(out["znorm2"], C.c_double), _p(out["resid_sum_norm"], C.c_double),
            _p(rs, C.c_double), _p(out["status"], C.c_uint32))
        if rc:
            raise ValueError("verify: invalid argument")
    else:
        for p in range(P):
            rsn = C.c_double(0.0)
            stt = C.c_uint32(0)
            rc = lib.btard_oracle_verify_one_ex(
                _p(g[p], C.c_float), C.c_int32(n), C.c_int64(stride), C.c_int64(int(ln[p])),
                _p(v[p], C.c_float), C.c_double(float(tau[p])),
                _p(row_scale[p], C.c_double) if row_scale is not None else None, C.c_uint64(int(seed)),
                C.c_int32(first_partition + p), C.c_int32(K),
                _p(norm_in[p], C.c_double) if norm_in is not None else None,
                _p(out["norm"][p], C.c_double), _p(out["weight"][p], C.c_double),
                _p(out["dot"][p], C.c_double), _p(out["s"][p], C.c_double),
                _p(out["s_sum"][p], C.c_double), _p(out["znorm2"][p], C.c_double),
                C.byref(rsn), _p(rs[p], C.c_double) if rs is not None else None, C.byref(stt))
            if rc:
                raise ValueError("verify: invalid argument")
            out["resid_sum_norm"][p] = rsn.value
            out["status"][p] = stt.value
    if rs is not None:
        out["resid_sum"] = rs
    return out


def checks(norm, s, delta_max, norm_reported=None, s_reported=None, rel_tol=0.0, abs_tol=0.0, sum_tol=0.0):
    """Predicates of Verifications 1-3.  norm [P][n], s [P][n][K], delta_max [P] (float64)."""
    norm = np.ascontiguousarray(norm, dtype=np.float64)
    s = np.ascontiguousarray(s, dtype=np.float64)
    P, n, K = s.shape
    dm = _per_part(delta_max, P, np.float64)
    nr = None if norm_reported is None else np.ascontiguousarray(norm_reported, dtype=np.float64)
    sr = None if s_reported is None else np.ascontiguousarray(s_reported, dtype=np.float64)
    out = dict(norm_mismatch=np.zeros((P, n), np.uint8), s_mismatch=np.zeros((P, n, K), np.uint8),
               sum_violation=np.zeros((P, K), np.uint8), check=np.zeros((P, n), np.uint8),
               votes=np.zeros(P, np.int32), check_averaging=np.zeros(P, np.uint8))
    lib = _load()
    for p in range(P):
        votes = C.c_int32(0)
        ca = C.c_uint8(0)
        lib.btard_oracle_checks_one(
            C.c_int32(n), C.c_int32(K), _p(norm[p], C.c_double),
            _p(nr[p], C.c_double) if nr is not None else None, _p(s[p], C.c_double),
            _p(sr[p], C.c_double) if sr is not None else None, C.c_double(float(dm[p])),
            C.c_double(rel_tol), C.c_double(abs_tol), C.c_double(sum_tol),
            _p(out["norm_mismatch"][p], C.c_uint8), _p(out["s_mismatch"][p], C.c_uint8),
            _p(out["sum_violation"][p], C.c_uint8), _p(out["check"][p], C.c_uint8),
            C.byref(votes), C.byref(ca))
        out["votes"][p] = votes.value
        out["check_averaging"][p] = ca.value
    return out


def preclip(g, lam, part_len=None):
    """Per-part clipping.  Returns dict(g [P][n][stride] float64, row_norm, factor [P][n])."""
    g = _as_g(g)
    P, n, stride = g.shape
    ln = _per_part(stride if part_len is None else part_len, P, np.int64)
    lam = _per_part(lam, P, np.float64)
    out = np.zeros((P, n, stride), dtype=np.float64)
    norm = np.zeros((P, n))
    fac = np.zeros((P, n))
    lib = _load()
    for p in range(P):
        for i in range(n):
            nr, f = C.c_double(0.0), C.c_double(0.0)
            lib.btard_oracle_preclip_row(_p(g[p, i], C.c_float), C.c_int64(int(ln[p])),
                                         C.c_double(float(lam[p])), _p(out[p, i], C.c_double),
                                         C.byref(nr), C.byref(f))
            norm[p, i], fac[p, i] = nr.value, f.value
    return dict(g=out, row_norm=norm, factor=fac)


def sha256(data):
    """SHA-256 of a bytes object by the oracle's own implementation."""
    buf = np.frombuffer(bytes(data), dtype=np.uint8).copy() if len(data) else np.zeros(1, np.uint8)
    out = np.zeros(32, dtype=np.uint8)
    _load().btard_oracle_sha256(_p(buf, C.c_uint8), C.c_int64(len(data)), _p(out, C.c_uint8))
    return out.tobytes()


def commitment(x, part_len=None):
    """Tree SHA-256 of every row of x [P][rows][stride] (or [P][stride]): uint8 [P][rows][32]."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if x.ndim == 2:
        x = x[:, None, :]
    P, rows, stride = x.shape
    ln = _per_part(stride if part_len is None else part_len, P, np.int64)
    out = np.zeros((P, rows, 32), dtype=np.uint8)
    lib = _load()
    for p in range(P):
        for i in range(rows):
            lib.btard_oracle_commitment(_p(x[p, i], C.c_float), C.c_int64(int(ln[p])), _p(out[p, i], C.c_uint8))
    return out
