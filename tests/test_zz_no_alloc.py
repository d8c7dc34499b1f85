"""The scratch-free verification entry point against the ordinary one (run last: see file name).

btard_verify_projections_static serves callers that cannot allocate device memory, for instance a
component living in a process whose framework already reserved the whole GPU for its own pool, or a
loop that must never call cudaMalloc because the call can stall the device.  It uses an array built
into the library instead of a caller workspace, and every call on a GPU shares that array.  The test
therefore calls it twice in a row on different inputs (the second call finds the first call's leftovers
in the array) and checks both results, through the C ABI, against btard_verify_projections and against
the float64 oracle.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2106_11257_b200 as btard

pytestmark = pytest.mark.gpu
RTOL = 1e-5


def _case(seed, P, n, stride, lens):
    rng = np.random.default_rng(seed)
    g = (rng.standard_normal((P, n, stride)) * 0.05 + rng.standard_normal((P, 1, stride))).astype(np.float32)
    g[:, : n // 4] *= 30.0
    v = (g[:, n // 2:].mean(axis=1)).astype(np.float32)
    for p in range(P):
        v[p, lens[p]:] = 0.0
    return torch.from_numpy(g).cuda(), torch.from_numpy(v).cuda()


def _same(a, b, keys):
    for k in keys:
        x, y = a[k].double().cpu().numpy(), b[k].double().cpu().numpy()
        scale = np.linalg.norm(y.ravel()) + 1e-300
        if k in ("s_sum", "resid_sum_norm", "resid_sum"):       # near-zero by design: absolute scale
            scale = np.abs(b["s"].cpu().numpy()).sum() + np.abs(y).sum() + 1e-300
        assert np.linalg.norm((x - y).ravel()) <= RTOL * scale, k


KEYS = ("norm", "weight", "dot", "s", "s_sum", "znorm2", "resid_sum_norm", "status")


def test_static_scratch_matches_workspace_entry_twice_in_a_row():
    cases = [
        dict(seed=1, P=3, n=16, stride=40_000, lens=np.array([40_000, 39_999, 17]), K=3, tau=1.0),
        dict(seed=2, P=5, n=64, stride=8_192, lens=np.array([8192, 8000, 4097, 1, 0]), K=1, tau=0.5),
    ]
    for c in cases:                       # back to back: the second call reuses a dirty array
        g, v = _case(c["seed"], c["P"], c["n"], c["stride"], c["lens"])
        ref = btard.verify_projections(g, v, c["tau"], 1234, K=c["K"], part_len=c["lens"],
                                       want_resid_sum=True)
        got = btard.verify_projections_static(g, v, c["tau"], 1234, K=c["K"], part_len=c["lens"],
                                              want_resid_sum=True)
        torch.cuda.synchronize()
        _same(got, ref, KEYS + ("resid_sum",))
        # and against the float64 oracle, on the same terms as the workspace entry point's own test
        exp = oracle.verify(g.cpu().numpy(), v.cpu().numpy(), c["tau"], 1234, K=c["K"], part_len=c["lens"])
        for k in ("norm", "weight", "dot", "s"):
            x = got[k].cpu().numpy()
            for p in range(c["P"]):
                den = np.linalg.norm(exp[k][p].ravel())
                assert np.linalg.norm((x[p] - exp[k][p]).ravel()) <= RTOL * den + 1e-300, (k, p)
        assert np.allclose(got["znorm2"].cpu().numpy(), exp["znorm2"], rtol=1e-6)
        assert np.all(np.abs(got["s_sum"].cpu().numpy() - exp["s_sum"]) <= RTOL * (np.abs(exp["s"]).sum(1) + 1e-300))
        # norms handed over by the caller: the other branch of the entry point
        got2 = btard.verify_projections_static(g, v, c["tau"], 1234, K=c["K"], part_len=c["lens"],
                                               resid_norm_in=ref["norm"])
        torch.cuda.synchronize()
        _same(got2, ref, KEYS)


def test_static_scratch_refuses_what_does_not_fit():
    # 2000 partitions exceed the built-in array: a clear error, nothing is launched
    P, n, stride = 2000, 4, 64
    g = torch.zeros((P, n, stride), dtype=torch.float32, device="cuda")
    v = torch.zeros((P, stride), dtype=torch.float32, device="cuda")
    before = btard.kernel_launch_count()
    with pytest.raises(btard.BtardError) as e:
        btard.verify_projections_static(g, v, 1.0, 1, K=1)
    assert e.value.code == -3 and btard.kernel_launch_count() == before
