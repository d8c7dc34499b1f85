"""GPU-vs-oracle parity through the C ABI (run on a B200: `pytest -m gpu`).

Tolerances: bit-exact for z, layout and indices; relative L2 <= 1e-5 per partition for v, norms,
weights, dots and s in fixed-iteration mode; near-zero sums compared absolutely against the scale of
their terms; iteration counts equal or +-1 in eps mode.
"""
import numpy as np
import pytest
import torch

import oracle
import workloads
import paper_2106_11257_b200 as btard

pytestmark = pytest.mark.gpu
RTOL = 1e-5


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64).ravel()
    b = np.asarray(b, dtype=np.float64).ravel()
    den = np.linalg.norm(b)
    return np.linalg.norm(a - b) / den if den > 0 else np.linalg.norm(a)


def cpu(t):
    return t.detach().cpu().numpy()


def run_gpu_cclip(g_np, tau, lens, **kw):
    g = torch.from_numpy(np.ascontiguousarray(g_np)).cuda()
    v0 = kw.pop("v0", None)
    v = torch.from_numpy(np.ascontiguousarray(v0)).cuda().clone() if v0 is not None else None
    r = btard.centered_clip(g, tau, part_len=lens, v=v, **kw)
    torch.cuda.synchronize()
    return g, r


def check_cclip(r, ref, lens, eps_mode=False, g=None, tau=None, init=None, v0=None, rule=0, gram=False):
    """Compares one aggregation with the oracle's.  In eps mode the update counts may differ by one
    (the stop test sits on a rounding edge); the GPU result is then compared with the oracle run for
    exactly the GPU's number of updates, which needs the inputs (g, tau, init)."""
    P = ref["v"].shape[0]
    v = cpu(r["v"])
    it = cpu(r["iters"])
    for p in range(P):
        L = int(lens[p])
        refp = {k: ref[k][p] for k in ("v", "resid_norm", "last_step_norm", "iters")}
        if eps_mode:
            assert abs(int(it[p]) - int(ref["iters"][p])) <= 1, (p, it[p], ref["iters"][p])
            if it[p] != ref["iters"][p]:
                if g is None:
                    continue
                again = oracle.centered_clip(g[p], float(np.broadcast_to(tau, (P,))[p]), lens[p:p + 1], init_mode=init,
                                             v0=None if v0 is None else v0[p], max_iters=int(it[p]), rule=rule)
                refp = {k: again[k][0] for k in ("v", "resid_norm", "last_step_norm", "iters")}
        else:
            assert it[p] == ref["iters"][p]
        assert rel_l2(v[p, :L], refp["v"][:L]) <= RTOL, ("v", p)
        assert np.all(v[p, L:] == 0)
        assert rel_l2(cpu(r["resid_norm"])[p], refp["resid_norm"]) <= RTOL
        ls, lr = cpu(r["last_step_norm"])[p], refp["last_step_norm"]
        # the last step is a difference of nearly equal vectors: absolute floor from fp32 v, whose rounding
        # error goes with the size of the rows that were averaged into it (a far row counts)
        floor = 3e-7 * (1 + np.linalg.norm(refp["v"][:L]) + np.max(refp["resid_norm"], initial=0.0))
        if gram:
            # the Gram variant has the step as sqrt(d^T G d) with G from fp32 products: when the d_i are not small
            # but sum_i d_i r_i cancels (a start at the exact mean with every weight 1), what is left of the
            # square is eps_fp32 rho^2, i.e. about 2.4e-4 rho in the norm
            floor += 1e-3 * np.max(refp["resid_norm"], initial=0.0)
        assert abs(ls - lr) <= 1e-4 * lr + floor, (p, ls, lr)


# ----------------------------------------------------------------------------- z and layout
@pytest.mark.parametrize("seed,p,k,length", [(0, 0, 0, 1024), (0x1234567890ABCDEF, 3, 2, 4099),
                                             (7, 15, 7, 698373), (2 ** 64 - 1, 63, 63, 1),
                                             (5, 1, 0, 2), (5, 1, 0, 3), (5, 1, 0, 0), (9, 0, 1, 1 << 22)])
def test_random_vector_is_bit_exact(seed, p, k, length):
    z = cpu(btard.random_vector(seed, p, k, length))
    ref = oracle.random_vector(seed, p, k, length)
    assert np.array_equal(z.view(np.uint32), ref.view(np.uint32))


def test_random_vector_rare_words():
    """Exhaustive over the polynomial's inputs is too much; sweep many blocks so that every exponent
    bucket of u and both sign bits occur, still bit for bit."""
    z = cpu(btard.random_vector(123456789, 5, 3, 1 << 24))
    ref = oracle.random_vector(123456789, 5, 3, 1 << 24)
    assert np.array_equal(z.view(np.uint32), ref.view(np.uint32))


# ----------------------------------------------------------------------------- CenteredClip
def make_case(rng, P, n, stride, lens, far_rows=0, scale=0.02):
    g = (rng.standard_normal((P, n, stride)) * scale).astype(np.float32)
    g += rng.standard_normal((P, 1, stride)).astype(np.float32)          # common mean
    if far_rows:
        g[:, :far_rows] = (rng.standard_normal((P, far_rows, stride)) * 5).astype(np.float32)
    for p in range(P):
        g[p, :, lens[p]:] = 77.0                                           # garbage in the pad
    return g


@pytest.mark.parametrize("algo", [btard.ALGO_DIRECT, btard.ALGO_DIRECT_COOPERATIVE])
@pytest.mark.parametrize("n", [1, 3, 4, 7, 8, 16, 23, 64, 100, 256])
@pytest.mark.parametrize("init", [btard.INIT_ZERO, btard.INIT_MEAN, btard.INIT_COORD_MEDIAN,
                                  btard.INIT_CALLER_V0])
def test_fixed_iterations_match_oracle(n, init, algo):
    rng = np.random.default_rng(100 + n)
    P, stride = 3, 5024
    lens = np.array([5024, 4097, 0 if n % 2 else 13])
    g = make_case(rng, P, n, stride, lens, far_rows=n // 3)
    tau = np.array([0.5, 1.0, 2.0])
    v0 = None
    if init == btard.INIT_CALLER_V0:
        v0 = rng.standard_normal((P, stride)).astype(np.float32)
    ref = oracle.centered_clip(g, tau, lens, init_mode=init, v0=v0, max_iters=6)
    _, r = run_gpu_cclip(g, tau, lens, init_mode=init, v0=v0, max_iters=6, algo=algo)
    check_cclip(r, ref, lens)
    assert not (cpu(r["status"]) & 4).any()


@pytest.mark.parametrize("algo", [btard.ALGO_DIRECT, btard.ALGO_DIRECT_COOPERATIVE])
@pytest.mark.parametrize("stop", [btard.STOP_FIXED_ITERS, btard.STOP_EPS])
def test_many_tiles_per_cta_and_many_ctas(algo, stop):
    """One long partition: several CTAs, each with many tiles, plus a ragged last tile."""
    rng = np.random.default_rng(5)
    P, n, stride = 2, 16, 1_000_032
    lens = np.array([1_000_001, 999_999])
    g = make_case(rng, P, n, stride, lens, far_rows=5, scale=0.001)
    ref = oracle.centered_clip(g, 1.0, lens, init_mode=oracle.INIT_COORD_MEDIAN, max_iters=4, stop_mode=stop, eps=1e-9)
    _, r = run_gpu_cclip(g, 1.0, lens, init_mode=btard.INIT_COORD_MEDIAN, max_iters=4, algo=algo, stop_mode=stop, eps=1e-9)
    check_cclip(r, ref, lens, eps_mode=(stop == btard.STOP_EPS), g=g, tau=1.0, init=oracle.INIT_COORD_MEDIAN)


def test_config1_fixed_and_eps():
    w = workloads.make_workload(1)
    g = w.g.numpy()
    ref = oracle.centered_clip(g, w.tau, w.part_len, init_mode=oracle.INIT_COORD_MEDIAN, max_iters=50)
    _, r = run_gpu_cclip(g, w.tau, w.part_len, init_mode=btard.INIT_COORD_MEDIAN, max_iters=50)
    check_cclip(r, ref, w.part_len)
    ref = oracle.centered_clip(g, w.tau, w.part_len, init_mode=oracle.INIT_COORD_MEDIAN,
                               stop_mode=oracle.STOP_EPS, max_iters=100, eps=1e-6)
    _, r = run_gpu_cclip(g, w.tau, w.part_len, init_mode=btard.INIT_COORD_MEDIAN,
                         stop_mode=btard.STOP_EPS, max_iters=100, eps=1e-6)
    check_cclip(r, ref, w.part_len, eps_mode=True, g=g, tau=w.tau, init=oracle.INIT_COORD_MEDIAN)
    assert cpu(r["status"])[0] == ref["status"][0] == 0


@pytest.mark.parametrize("algo", [btard.ALGO_DIRECT, btard.ALGO_DIRECT_COOPERATIVE])
def test_eps_mode_counts_and_cap_flag(algo):
    rng = np.random.default_rng(6)
    P, n, stride = 4, 8, 2048
    lens = np.array([2048, 2000, 1, 1027])
    g = make_case(rng, P, n, stride, lens, far_rows=2)
    for eps, cap in [(1e-3, 200), (1e-5, 200), (1e-5, 3)]:
        ref = oracle.centered_clip(g, 0.7, lens, init_mode=oracle.INIT_MEAN, stop_mode=oracle.STOP_EPS,
                                   max_iters=cap, eps=eps)
        _, r = run_gpu_cclip(g, 0.7, lens, init_mode=btard.INIT_MEAN, stop_mode=btard.STOP_EPS,
                             max_iters=cap, eps=eps, algo=algo)
        check_cclip(r, ref, lens, eps_mode=True, g=g, tau=0.7, init=oracle.INIT_MEAN)
        same = cpu(r["iters"]) == ref["iters"]
        assert np.array_equal(cpu(r["status"])[same] & 1, ref["status"][same] & 1)
    assert len(set(ref["iters"])) >= 1


def test_special_radii():
    rng = np.random.default_rng(7)
    P, n, stride = 3, 5, 1024
    lens = np.array([1024, 1000, 999])
    g = make_case(rng, P, n, stride, lens)
    tau = np.array([np.inf, 0.0, 1e-3])
    ref = oracle.centered_clip(g, tau, lens, init_mode=oracle.INIT_ZERO, max_iters=3)
    _, r = run_gpu_cclip(g, tau, lens, init_mode=btard.INIT_ZERO, max_iters=3)
    check_cclip(r, ref, lens)
    v = cpu(r["v"])
    assert rel_l2(v[0, :1024], g[0].astype(np.float64).mean(0)) < 1e-6     # tau = inf: the mean
    assert np.all(v[1] == 0)                                               # tau = 0: never moves


@pytest.mark.parametrize("algo", [btard.ALGO_DIRECT, btard.ALGO_DIRECT_COOPERATIVE])
@pytest.mark.parametrize("stride", [1024, 40_000])
def test_non_finite_rows_take_weight_zero(algo, stride):
    rng = np.random.default_rng(8)
    P, n = 2, 6
    lens = np.array([stride, stride - 3])
    g = make_case(rng, P, n, stride, lens)
    g[0, 2, 17] = np.nan
    g[1, 4, 900] = np.inf
    g[1, 0, 3] = -np.inf
    ref = oracle.centered_clip(g, 1.0, lens, init_mode=oracle.INIT_ZERO, max_iters=4)
    _, r = run_gpu_cclip(g, 1.0, lens, init_mode=btard.INIT_ZERO, max_iters=4, algo=algo)
    v = cpu(r["v"])
    assert np.all(np.isfinite(v))
    for p in range(P):
        assert rel_l2(v[p], ref["v"][p]) <= RTOL
        assert cpu(r["status"])[p] & btard.STATUS_NONFINITE_ROW
        assert ref["status"][p] & oracle.STATUS_NONFINITE_ROW
    rn = cpu(r["resid_norm"])
    assert np.array_equal(np.isfinite(rn), np.isfinite(ref["resid_norm"]))


@pytest.mark.parametrize("n", [5, 16, 40, 64, 100])
def test_non_finite_rows_with_a_median_start(n):
    """A Byzantine row holding NaN / inf together with the coordinate-median start (the start every
    benchmark uses): the median orders NaNs at the ends, the row takes weight 0 in every update; direct,
    Gram and one-call paths."""
    rng = np.random.default_rng(80 + n)
    P, stride = 2, 4096
    lens = np.array([4096, 4001])
    g = make_case(rng, P, n, stride, lens)
    g[0, 2, 17] = np.nan
    g[0, 2, 18] = -np.nan
    g[1, n - 1, 900] = np.inf
    g[1, n - 1, 3] = -np.inf
    ref = oracle.centered_clip(g, 1.0, lens, init_mode=oracle.INIT_COORD_MEDIAN, max_iters=5)
    assert np.all(np.isfinite(ref["v"])) and (ref["status"] & oracle.STATUS_NONFINITE_ROW).all()
    for algo in (btard.ALGO_DIRECT, btard.ALGO_GRAM, btard.ALGO_DIRECT_COOPERATIVE):
        _, r = run_gpu_cclip(g, 1.0, lens, init_mode=btard.INIT_COORD_MEDIAN, max_iters=5, algo=algo)
        v = cpu(r["v"])
        assert np.all(np.isfinite(v))
        for p in range(P):
            assert rel_l2(v[p], ref["v"][p]) <= RTOL, (algo, p)
            assert cpu(r["status"])[p] & btard.STATUS_NONFINITE_ROW
        rn = cpu(r["resid_norm"])
        fin = np.isfinite(ref["resid_norm"])
        assert np.array_equal(np.isfinite(rn), fin) and rel_l2(rn[fin], ref["resid_norm"][fin]) <= RTOL
    rc, rv = btard.centered_clip_verify(torch.from_numpy(g).cuda(), 1.0, 5, K=2, part_len=lens,
                                        init_mode=btard.INIT_COORD_MEDIAN, max_iters=5, algo=btard.ALGO_GRAM)
    torch.cuda.synchronize()
    v = cpu(rc["v"])
    refv = oracle.verify(g, v, 1.0, 5, K=2, part_len=lens)
    for p in range(P):
        assert rel_l2(v[p], ref["v"][p]) <= RTOL
        assert cpu(rc["status"])[p] & btard.STATUS_NONFINITE_ROW and cpu(rv["status"])[p] & btard.STATUS_NONFINITE_ROW
        fin = np.isfinite(refv["norm"][p])
        assert np.array_equal(np.isfinite(cpu(rv["norm"])[p]), fin)
        assert np.array_equal(cpu(rv["weight"])[p] == 0.0, ~fin)
        assert rel_l2(cpu(rv["s"])[p][fin], refv["s"][p][fin]) <= RTOL
        scale = np.abs(refv["s"][p]).sum(0) + 1e-300
        assert np.all(np.abs(cpu(rv["s_sum"])[p] - refv["s_sum"][p]) <= RTOL * scale)


def test_peer_and_partition_indexing():
    """Row i / slab p of every output belongs to peer i / partition p: distinct magnitudes."""
    P, n, stride = 4, 5, 256
    g = np.zeros((P, n, stride), dtype=np.float32)
    for p in range(P):
        for i in range(n):
            g[p, i, :] = (p + 1) * 10 + i
    lens = np.full(P, stride)
    ref = oracle.centered_clip(g, np.inf, lens, init_mode=oracle.INIT_ZERO, max_iters=1)
    _, r = run_gpu_cclip(g, np.inf, lens, init_mode=btard.INIT_ZERO, max_iters=1)
    assert np.allclose(cpu(r["resid_norm"]), ref["resid_norm"], rtol=1e-6)
    assert np.allclose(cpu(r["v"]), ref["v"], rtol=1e-6)


# ----------------------------------------------------------------------------- cooperative variant
def test_cooperative_variant_eps_mode_many_items_per_cta():
    """All updates inside one cooperative kernel with grid barriers; rows long enough that every
    resident CTA holds several work items, eps stop with partitions finishing at different updates."""
    rng = np.random.default_rng(12)
    P, n, stride = 5, 16, 600_000
    lens = np.array([600_000, 599_999, 123_457, 600_000, 31])
    g = make_case(rng, P, n, stride, lens, far_rows=5, scale=0.001)
    tau = np.array([1.0, 0.5, 2.0, 1.0, 1.0])
    ref = oracle.centered_clip(g, tau, lens, init_mode=oracle.INIT_COORD_MEDIAN,
                               stop_mode=oracle.STOP_EPS, max_iters=60, eps=1e-5)
    _, r = run_gpu_cclip(g, tau, lens, init_mode=btard.INIT_COORD_MEDIAN, stop_mode=btard.STOP_EPS,
                         max_iters=60, eps=1e-5, algo=btard.ALGO_DIRECT_COOPERATIVE)
    check_cclip(r, ref, lens, eps_mode=True, g=g, tau=tau, init=oracle.INIT_COORD_MEDIAN)
    assert len(set(ref["iters"].tolist())) > 1
    assert not (cpu(r["status"]) & 4).any()


# ----------------------------------------------------------------------------- baseline aggregators
@pytest.mark.parametrize("algo", [btard.ALGO_DIRECT, btard.ALGO_DIRECT_COOPERATIVE])
@pytest.mark.parametrize("n", [3, 16, 64])
def test_geometric_median_rule_matches_oracle(n, algo):
    rng = np.random.default_rng(500 + n)
    P, stride = 3, 5024
    lens = np.array([5024, 4097, 13])
    g = make_case(rng, P, n, stride, lens, far_rows=n // 3)
    floor = np.array([1e-3, 1e-6, 0.5])
    for stop, iters, eps in ((btard.STOP_FIXED_ITERS, 8, 0.0), (btard.STOP_EPS, 200, 1e-5)):
        ref = oracle.centered_clip(g, floor, lens, init_mode=oracle.INIT_MEAN, stop_mode=stop,
                                   max_iters=iters, eps=eps, rule=oracle.RULE_GEOMETRIC_MEDIAN)
        _, r = run_gpu_cclip(g, floor, lens, init_mode=btard.INIT_MEAN, stop_mode=stop, max_iters=iters,
                             eps=eps, algo=algo, rule=btard.RULE_GEOMETRIC_MEDIAN)
        check_cclip(r, ref, lens, eps_mode=(stop == btard.STOP_EPS), g=g, tau=floor, init=oracle.INIT_MEAN,
                    rule=oracle.RULE_GEOMETRIC_MEDIAN)


@pytest.mark.parametrize("n", [1, 4, 16, 23, 64, 100])
def test_mean_and_coordinate_median_rules_match_oracle(n):
    rng = np.random.default_rng(600 + n)
    P, stride = 3, 5024
    lens = np.array([5024, 4097, 13])
    g = make_case(rng, P, n, stride, lens, far_rows=n // 3)
    for rule, orule in ((btard.RULE_MEAN, oracle.RULE_MEAN), (btard.RULE_COORD_MEDIAN, oracle.RULE_COORD_MEDIAN)):
        ref = oracle.centered_clip(g, 1.0, lens, rule=orule)
        _, r = run_gpu_cclip(g, 1.0, lens, rule=rule)
        check_cclip(r, ref, lens)
        assert (cpu(r["iters"]) == 0).all()


@pytest.mark.parametrize("n", [2, 5, 16, 32, 33, 64, 100])
def test_coordinate_median_with_special_values_is_exact(n):
    """The median kernel sorts a column as floats when its sum is not NaN and on integer keys otherwise:
    columns with infinities of one or both signs, NaNs of both signs, zeros of both signs and ties must
    come out as the oracle's, value for value (the sign of a zero aside)."""
    rng = np.random.default_rng(900 + n)
    P, stride = 2, 2048
    lens = np.array([2048, 1999])
    g = (rng.standard_normal((P, n, stride)) * 1e-2).astype(np.float32)
    for p in range(P):
        g[p, :, lens[p]:] = 0.0
    rows = rng.integers(0, n, size=(P, 64))
    for p in range(P):
        for t in range(64):
            c, r = 16 * t, rows[p, t]
            kind = t % 8
            if kind == 0: g[p, r, c] = np.inf
            elif kind == 1: g[p, r, c] = -np.inf
            elif kind == 2: g[p, r, c] = np.inf; g[p, (r + 1) % n, c] = -np.inf
            elif kind == 3: g[p, r, c] = np.nan
            elif kind == 4: g[p, r, c] = -np.nan; g[p, (r + 1) % n, c] = np.nan
            elif kind == 5: g[p, :, c] = 0.0; g[p, r, c] = -0.0
            elif kind == 6: g[p, :, c] = g[p, 0, c]
            else: g[p, : (n + 1) // 2, c] = np.inf
    scale = rng.uniform(0.5, 1.0, size=(P, n))
    scale[0, n - 1] = 0.0                                # a dropped row
    scale[1, 0] = 1.0
    for rs in (None, scale):
        ref = oracle.centered_clip(g, 1.0, lens, rule=oracle.RULE_COORD_MEDIAN, row_scale=rs)
        _, r = run_gpu_cclip(g, 1.0, lens, rule=btard.RULE_COORD_MEDIAN,
                             row_scale=None if rs is None else torch.from_numpy(rs).cuda())
        v = cpu(r["v"])
        for p in range(P):
            a, b = v[p, : lens[p]] + np.float32(0.0), ref["v"][p, : lens[p]].astype(np.float32) + np.float32(0.0)
            if rs is None:
                assert np.array_equal(a, b, equal_nan=True), (p, np.nonzero(~((a == b) | (np.isnan(a) & np.isnan(b))))[0][:8])
            else:                                        # the products f x are rounded to fp32 on the GPU only
                fin = np.isfinite(b)
                assert np.array_equal(np.isnan(a), np.isnan(b)) and np.array_equal(a[~fin & ~np.isnan(b)], b[~fin & ~np.isnan(b)])
                assert np.all(np.abs(a[fin] - b[fin]) <= 2e-7 * np.abs(b[fin]) + 5e-9), p   # values are O(1e-2): one rounding of f x


@pytest.mark.parametrize("n", [32, 64])
def test_fused_median_start_with_special_values(n):
    """32 and 64 peers, direct algorithm: the median start and the start pass are one kernel.  With tau = 0
    every weight is 0, so the aggregate stays at the start and must equal the oracle's median value for
    value, on columns with an infinity, NaNs of both signs, zeros of both signs and ties; the norms at the
    start are compared too."""
    rng = np.random.default_rng(950 + n)
    P, stride = 3, 33_024                      # more than 256 columns per thread of one CTA: several CTAs
    lens = np.array([33_024, 20_001, 77])
    g = (rng.standard_normal((P, n, stride)) * 1e-2).astype(np.float32)
    for p in range(P):
        g[p, :, lens[p]:] = 77.0
    bad_rows = [set() for _ in range(P)]
    for p in range(P):
        for t in range(min(60, lens[p] // 16)):
            c, r = 16 * t + 3, int(rng.integers(0, n))
            kind = t % 6
            if kind == 0: g[p, r, c] = np.inf; bad_rows[p].add(r)
            elif kind == 1: g[p, r, c] = -np.inf; bad_rows[p].add(r)
            elif kind == 2: g[p, r, c] = np.nan; bad_rows[p].add(r)
            elif kind == 3:
                g[p, r, c] = -np.nan; g[p, (r + 1) % n, c] = np.nan
                bad_rows[p].update((r, (r + 1) % n))
            elif kind == 4: g[p, :, c] = 0.0; g[p, r, c] = -0.0
            else: g[p, :, c] = g[p, 0, c]
    ref = oracle.centered_clip(g, 0.0, lens, init_mode=oracle.INIT_COORD_MEDIAN, max_iters=1)
    med = oracle.centered_clip(g, 1.0, lens, rule=oracle.RULE_COORD_MEDIAN)
    _, r = run_gpu_cclip(g, 0.0, lens, init_mode=btard.INIT_COORD_MEDIAN, max_iters=1, algo=btard.ALGO_DIRECT)
    v, rn = cpu(r["v"]), cpu(r["resid_norm"])
    for p in range(P):
        L = lens[p]
        a = v[p, :L] + np.float32(0.0)
        assert np.array_equal(a, med["v"][p, :L].astype(np.float32) + np.float32(0.0)), p
        assert np.array_equal(a, ref["v"][p, :L].astype(np.float32) + np.float32(0.0)), p
        fin = np.isfinite(ref["resid_norm"][p])
        assert set(np.nonzero(~fin)[0]) == bad_rows[p]
        assert np.array_equal(np.isfinite(rn[p]), fin)
        assert rel_l2(rn[p][fin], ref["resid_norm"][p][fin]) <= RTOL
        assert cpu(r["status"])[p] & btard.STATUS_NONFINITE_ROW


def test_geometric_median_rule_rejects_a_zero_floor_and_gram():
    g = torch.zeros((1, 4, 64), device="cuda")
    with pytest.raises(btard.BtardError):
        btard.centered_clip(g, 0.0, init_mode=btard.INIT_ZERO, rule=btard.RULE_GEOMETRIC_MEDIAN)
    with pytest.raises(btard.BtardError) as e:
        btard.centered_clip(g, 1.0, init_mode=btard.INIT_ZERO, rule=btard.RULE_GEOMETRIC_MEDIAN, algo=btard.ALGO_GRAM)
    assert e.value.code == -5


# ----------------------------------------------------------------------------- Split / Merge
@pytest.mark.parametrize("mode", [btard.SPLIT_PAPER, btard.SPLIT_CEIL_PAD])
@pytest.mark.parametrize("n,d,P", [(4, 1024, 1), (5, 100_003, 7), (3, 10, 4), (16, 1_000_001, 16)])
def test_split_and_merge_are_exact_copies(n, d, P, mode):
    """Split(v, n) / Merge (App. D.1): bit-exact against plain slicing with the oracle's layout."""
    rng = np.random.default_rng(d)
    grads = rng.standard_normal((n, d)).astype(np.float32)
    g, off, ln = btard.split_gradients(torch.from_numpy(grads).cuda(), P, mode=mode)
    o_off, o_ln, o_stride = oracle.partition_layout(d, P, mode, 32)
    assert np.array_equal(off, o_off) and np.array_equal(ln, o_ln) and g.shape[2] == max(o_stride, 32)
    got = cpu(g)
    for p in range(P):
        assert np.array_equal(got[p, :, :ln[p]], grads[:, off[p]:off[p] + ln[p]])
        assert np.all(got[p, :, ln[p]:] == 0)
    # aggregate with tau = inf (the mean) and merge: the average gradient, as plain All-Reduce would give
    r = btard.centered_clip(g, np.inf, part_len=ln, init_mode=btard.INIT_ZERO, max_iters=1)
    merged = cpu(btard.merge_partitions(r["v"], d, off, ln))
    assert rel_l2(merged, grads.astype(np.float64).mean(0)) < 1e-6
    v = torch.from_numpy(rng.standard_normal((P, g.shape[2])).astype(np.float32)).cuda()
    out = cpu(btard.merge_partitions(v, d, off, ln))
    for p in range(P):
        assert np.array_equal(out[off[p]:off[p] + ln[p]], cpu(v)[p, :ln[p]])


# ----------------------------------------------------------------------------- commitments
@pytest.mark.parametrize("rows,stride,lens", [(4, 1024, [1024]), (16, 100_000, [100_000, 99_973, 1]),
                                               (3, 2048, [2047, 1025, 0, 14]), (1, 698_400, [698_373, 698_367])])
def test_commitments_are_bit_exact(rows, stride, lens):
    rng = np.random.default_rng(stride + rows)
    P = len(lens)
    x = rng.standard_normal((P, rows, stride)).astype(np.float32)
    ref = oracle.commitment(x, np.array(lens))
    out = cpu(btard.hash_partitions(torch.from_numpy(x).cuda(), np.array(lens)))
    assert np.array_equal(out, ref)


def test_commitment_of_an_aggregate_changes_with_one_bit():
    v = torch.randn((2, 4096), device="cuda")
    a = cpu(btard.hash_partitions(v))
    v2 = v.clone(); v2[1, 4095] = torch.nextafter(v2[1, 4095], torch.tensor(10.0, device="cuda"))
    b = cpu(btard.hash_partitions(v2))
    assert np.array_equal(a[0], b[0]) and not np.array_equal(a[1], b[1])


# ----------------------------------------------------------------------------- Clipped-SGD pre-clip
@pytest.mark.parametrize("n,stride", [(4, 1024), (16, 100_000), (64, 5024)])
def test_preclip_matches_oracle(n, stride):
    rng = np.random.default_rng(700 + n)
    P = 3
    lens = np.array([stride, stride - 27, 13])
    g = (rng.standard_normal((P, n, stride)) * 0.01).astype(np.float32)
    g[:, ::3] *= 50.0                                              # every third peer is far too long
    g[1, 1, 7] = np.inf
    lam = np.array([1.0, 2.0, np.inf])
    ref = oracle.preclip(g, lam, part_len=lens)
    gd = torch.from_numpy(g.copy()).cuda()
    out = btard.preclip(gd, lam, part_len=lens)
    torch.cuda.synchronize()
    got = cpu(gd)
    for p in range(P):
        L = lens[p]
        fin = np.isfinite(ref["row_norm"][p])
        assert rel_l2(cpu(out["row_norm"])[p][fin], ref["row_norm"][p][fin]) <= 1e-6
        assert np.array_equal(np.isfinite(cpu(out["row_norm"])[p]), fin)
        assert rel_l2(cpu(out["factor"])[p], ref["factor"][p]) <= 1e-6
        assert rel_l2(got[p, :, :L], ref["g"][p, :, :L]) <= 1e-6
        untouched = ref["factor"][p] == 1.0
        assert np.array_equal(got[p, untouched, :L], g[p, untouched, :L])   # bit for bit
    assert cpu(out["status"])[1] & btard.STATUS_NONFINITE_ROW and np.all(got[1, 1, :lens[1]] == 0)


# ----------------------------------------------------------------------------- tau_l schedule, Clipped-SGD factors
@pytest.mark.parametrize("algo", [btard.ALGO_DIRECT, btard.ALGO_GRAM, btard.ALGO_DIRECT_COOPERATIVE])
@pytest.mark.parametrize("n", [3, 16, 23, 64, 100])
def test_tau_schedule_matches_oracle(n, algo):
    """Update l uses the radius tau_l (App. D.2): every algorithm against the oracle's scheduled run."""
    rng = np.random.default_rng(1300 + n)
    P, stride, iters = 3, 5024, 7
    lens = np.array([5024, 4097, 13])
    g = make_case(rng, P, n, stride, lens, far_rows=n // 3)
    sched = np.abs(rng.standard_normal((P, iters))) + 0.2
    sched[1, 2] = np.inf
    sched[2, 4] = 0.0
    ref = oracle.centered_clip(g, 1.0, lens, init_mode=oracle.INIT_COORD_MEDIAN, max_iters=iters, tau_schedule=sched)
    _, r = run_gpu_cclip(g, 1.0, lens, init_mode=btard.INIT_COORD_MEDIAN, max_iters=iters, algo=algo,
                         tau_schedule=torch.from_numpy(sched).cuda())
    check_cclip(r, ref, lens)


@pytest.mark.parametrize("n,K", [(4, 1), (16, 2), (16, 5), (23, 1), (64, 1), (64, 4), (100, 2)])
def test_clipped_sgd_factors_applied_on_load(n, K):
    """BTARD-Clipped-SGD (Alg. 9) without rewriting g: btard_preclip_factors, then aggregation and
    verification with row_scale, against the oracle's clip factors and its scaled aggregation; direct and
    Gram algorithms, separate calls and the one-call entry point.  One row holds an inf (factor 0)."""
    rng = np.random.default_rng(1400 + 3 * n + K)
    P, stride = 3, 20_032
    lens = np.array([20_032, 17_001, 13])
    g = make_case(rng, P, n, stride, lens, far_rows=n // 3)
    g[1, n - 1, 5] = np.inf
    lam = np.array([200.0, 150.0, 5.0])
    tau = np.array([0.5, 1.0, 2.0])
    pc = oracle.preclip(g, lam, part_len=lens)
    assert (pc["factor"] < 1).any() and (pc["factor"] == 1).any() and pc["factor"][1, n - 1] == 0
    gd = torch.from_numpy(g).cuda()
    keep = gd.clone()
    out = btard.preclip(gd, lam, part_len=lens, in_place=False)
    torch.cuda.synchronize()
    assert torch.equal(gd, keep)                                  # g untouched
    fin = np.isfinite(pc["row_norm"])
    assert rel_l2(cpu(out["row_norm"])[fin], pc["row_norm"][fin]) <= 1e-6
    assert rel_l2(cpu(out["factor"]), pc["factor"]) <= 1e-6 and cpu(out["factor"])[1, n - 1] == 0
    assert cpu(out["status"])[1] & btard.STATUS_NONFINITE_ROW
    f = out["factor"]
    refc = oracle.centered_clip(g, tau, lens, init_mode=oracle.INIT_COORD_MEDIAN, max_iters=6, row_scale=pc["factor"])
    for algo in (btard.ALGO_DIRECT, btard.ALGO_GRAM):
        if algo == btard.ALGO_GRAM and n > 128:
            continue
        r = btard.centered_clip(gd, tau, part_len=lens, init_mode=btard.INIT_COORD_MEDIAN, max_iters=6, algo=algo,
                                row_scale=f)
        torch.cuda.synchronize()
        check_cclip(r, refc, lens)
        v32 = cpu(r["v"])
        refv = oracle.verify(g, v32, tau, 21, K=K, part_len=lens, row_scale=pc["factor"], want_resid_sum=True)
        o = btard.verify_projections(gd, r["v"], tau, 21, K=K, part_len=lens, row_scale=f, want_resid_sum=True)
        torch.cuda.synchronize()
        check_verify(o, refv, K)
        rc, rv = btard.centered_clip_verify(gd, tau, 21, K=K, part_len=lens, init_mode=btard.INIT_COORD_MEDIAN,
                                            max_iters=6, algo=algo, row_scale=f)
        torch.cuda.synchronize()
        check_cclip(rc, refc, lens)
        check_verify(rv, oracle.verify(g, cpu(rc["v"]), tau, 21, K=K, part_len=lens, row_scale=pc["factor"]), K)


# ----------------------------------------------------------------------------- Gram variant
@pytest.mark.parametrize("n", [1, 3, 8, 16, 23, 64, 100, 128])
@pytest.mark.parametrize("init", [btard.INIT_MEAN, btard.INIT_COORD_MEDIAN, btard.INIT_CALLER_V0])
def test_gram_mode_matches_oracle(n, init):
    """Same iteration in coefficient space: must equal the direct oracle, cancellation included
    (a third of the rows are 100x farther than the rest)."""
    rng = np.random.default_rng(300 + n)
    P, stride = 3, 5024
    lens = np.array([5024, 4097, 13])
    g = make_case(rng, P, n, stride, lens, far_rows=n // 3)
    tau = np.array([0.5, 1.0, 2.0])
    v0 = None
    if init == btard.INIT_CALLER_V0:
        v0 = (g[:, n // 3:].mean(axis=1) + 0.01).astype(np.float32)
    ref = oracle.centered_clip(g, tau, lens, init_mode=init, v0=v0, max_iters=12)
    _, r = run_gpu_cclip(g, tau, lens, init_mode=init, v0=v0, max_iters=12, algo=btard.ALGO_GRAM)
    check_cclip(r, ref, lens)


def test_gram_mode_eps_and_long_rows():
    rng = np.random.default_rng(11)
    P, n, stride = 2, 16, 1_000_032
    lens = np.array([1_000_001, 999_999])
    g = make_case(rng, P, n, stride, lens, far_rows=5, scale=0.001)
    ref = oracle.centered_clip(g, 1.0, lens, init_mode=oracle.INIT_COORD_MEDIAN,
                               stop_mode=oracle.STOP_EPS, max_iters=300, eps=1e-6)
    _, r = run_gpu_cclip(g, 1.0, lens, init_mode=btard.INIT_COORD_MEDIAN, stop_mode=btard.STOP_EPS,
                         max_iters=300, eps=1e-6, algo=btard.ALGO_GRAM)
    check_cclip(r, ref, lens, eps_mode=True, g=g, tau=1.0, init=oracle.INIT_COORD_MEDIAN)
    assert np.array_equal(cpu(r["status"]) & 1, ref["status"] & 1)


@pytest.mark.parametrize("n", [5, 20, 64])
def test_gram_mode_on_very_short_rows(n):
    """Rows shorter than one 32-column tile (the tensor-core kernel does not take them: the fp32 kernels do)."""
    rng = np.random.default_rng(40 + n)
    P, stride = 2, 28
    lens = np.array([28, 5])
    g = make_case(rng, P, n, stride, lens, far_rows=n // 3)
    ref = oracle.centered_clip(g, 1.0, lens, init_mode=oracle.INIT_MEAN, max_iters=6)
    _, r = run_gpu_cclip(g, 1.0, lens, init_mode=btard.INIT_MEAN, max_iters=6, algo=btard.ALGO_GRAM)
    check_cclip(r, ref, lens)


def test_gram_mode_rejects_too_many_peers():
    g = torch.zeros((1, 129, 64), device="cuda")
    with pytest.raises(btard.BtardError) as e:
        btard.centered_clip(g, 1.0, init_mode=btard.INIT_ZERO, max_iters=1, algo=btard.ALGO_GRAM)
    assert e.value.code == -5


# ----------------------------------------------------------------------------- verification
def check_verify(out, ref, K):
    P, n = ref["norm"].shape
    for p in range(P):
        for key in ("norm", "weight"):
            assert rel_l2(cpu(out[key])[p], ref[key][p]) <= RTOL, (key, p)
        # Projections: relative L2 over the partition's [n][K] array, with the floor fp32 sets: <r_i, z> / |z| summed
        # in fp32 carries an error of a few eps_fp32 rho_i whatever its own size (the residuals are rounded, with row
        # factors the rows too), so an array whose directions are all nearly orthogonal to the residuals (2 peers,
        # 1 direction: one independent number) is known to 4 eps_fp32 |rho| = 5e-7 |rho|, not to 1e-5 of itself
        # (seen: 1.7e-7 |rho| on a projection of 0.012 rho, with row factors)
        wr = ref["weight"][p] * ref["norm"][p]
        for key, vec in (("dot", ref["norm"][p]), ("s", wr)):
            got, want = cpu(out[key])[p].astype(np.float64), ref[key][p]
            floor = 5e-2 * np.linalg.norm(vec) * np.sqrt(K)
            assert np.linalg.norm(got - want) <= RTOL * max(np.linalg.norm(want), floor), (key, p)
        assert np.allclose(cpu(out["znorm2"])[p], ref["znorm2"][p], rtol=1e-6)
        rscale = (ref["weight"][p] * ref["norm"][p]).sum() + 1e-300
        # |s_i| <= w_i rho_i, and the fp32 error of a projection goes with rho_i, not with the projection: a
        # direction that happens to be nearly orthogonal to every residual has sum |s_i| far below that scale.
        # s_i = w_i <r_i, z> / |z| evaluated in fp32 carries an error of about eps_fp32 w_i rho_i (1.2e-7; seen:
        # up to 2.8e-8 sum_i w_i rho_i with row factors and far rows), so the floor is 1e-7 sum_i w_i rho_i
        scale = np.maximum(np.abs(ref["s"][p]).sum(0), 1e-2 * rscale) + 1e-300
        assert np.all(np.abs(cpu(out["s_sum"])[p] - ref["s_sum"][p]) <= RTOL * scale), ("s_sum", p)
        assert abs(cpu(out["resid_sum_norm"])[p] - ref["resid_sum_norm"][p]) <= RTOL * rscale


@pytest.mark.parametrize("n,K", [(1, 1), (4, 1), (4, 2), (5, 3), (8, 2), (13, 2), (16, 8), (16, 1), (16, 2),
                                 (23, 4), (64, 4), (64, 8), (64, 11), (100, 2), (200, 5),
                                 (1, 8), (4, 8), (4, 64)])       # one row group, 8 directions: the largest z block
def test_verify_matches_oracle(n, K):
    rng = np.random.default_rng(200 + n + K)
    P, stride = 3, 5024
    lens = np.array([5024, 4097, 13])
    g = make_case(rng, P, n, stride, lens, far_rows=n // 3)
    tau = np.array([0.5, 1.0, 2.0])
    refc = oracle.centered_clip(g, tau, lens, init_mode=oracle.INIT_COORD_MEDIAN, max_iters=8)
    v32 = refc["v"].astype(np.float32)
    seed = 0xABCDEF0123 + n
    gd = torch.from_numpy(g).cuda()
    vd = torch.from_numpy(v32).cuda()
    # norms computed by the library itself
    ref = oracle.verify(g, v32, tau, seed, K=K, part_len=lens, want_resid_sum=True)
    out = btard.verify_projections(gd, vd, tau, seed, K=K, part_len=lens, want_resid_sum=True)
    torch.cuda.synchronize()
    check_verify(out, ref, K)
    for p in range(P):
        L = lens[p]
        rs = cpu(out["resid_sum"])[p]
        scale = (ref["weight"][p] * ref["norm"][p]).sum()
        assert np.linalg.norm(rs[:L] - ref["resid_sum"][p, :L]) <= RTOL * scale
    # norms handed over from the aggregation
    nin = refc["resid_norm"]
    ref2 = oracle.verify(g, v32, tau, seed, K=K, part_len=lens, norm_in=nin)
    out2 = btard.verify_projections(gd, vd, tau, seed, K=K, part_len=lens,
                                    resid_norm_in=torch.from_numpy(nin).cuda())
    torch.cuda.synchronize()
    check_verify(out2, ref2, K)


@pytest.mark.parametrize("algo", [btard.ALGO_GRAM, btard.ALGO_DIRECT])
@pytest.mark.parametrize("n,K", [(1, 1), (4, 1), (7, 2), (16, 1), (16, 2), (16, 3), (16, 8), (23, 1), (64, 2),
                                 (64, 4), (64, 11), (100, 2),
                                 (4, 3), (4, 8), (7, 8)])         # fused pass with more than 48 KB of shared memory
def test_one_call_aggregation_and_verification(n, K, algo):
    """btard_centered_clip_verify against the oracle's aggregation followed by its verification.  With the
    Gram variant the combine and verification passes are one kernel (all rows of a column in one thread
    for n <= 16 and K <= 2, row groups with a shared z block otherwise; K = 11 needs a second, plain
    launch); the direct algorithm takes the two calls back to back.  A third of the rows are 100x
    farther than the rest."""
    rng = np.random.default_rng(500 + 7 * n + K)
    P, stride = 3, 40_032                     # several CTAs per partition, many tiles, a ragged tail
    lens = np.array([40_032, 33_001, 13])
    g = make_case(rng, P, n, stride, lens, far_rows=n // 3)
    tau = np.array([0.5, 1.0, 2.0])
    seed = 0x5EED0000 + n
    refc = oracle.centered_clip(g, tau, lens, init_mode=oracle.INIT_COORD_MEDIAN, max_iters=9)
    gd = torch.from_numpy(g).cuda()
    rc, rv = btard.centered_clip_verify(gd, tau, seed, K=K, part_len=lens, init_mode=btard.INIT_COORD_MEDIAN,
                                        max_iters=9, algo=algo, partition_base=2, want_resid_sum=True)
    torch.cuda.synchronize()
    check_cclip(rc, refc, lens)
    # the oracle verifies the aggregate the GPU produced (fp32), with the norms the GPU reported
    v32 = cpu(rc["v"])
    refv = oracle.verify(g, v32, tau, seed, K=K, part_len=lens, first_partition=2, want_resid_sum=True)
    check_verify(rv, refv, K)
    for p in range(P):
        L = lens[p]
        scale = (refv["weight"][p] * refv["norm"][p]).sum()
        assert np.linalg.norm(cpu(rv["resid_sum"])[p, :L] - refv["resid_sum"][p, :L]) <= RTOL * scale
    assert np.array_equal(cpu(rc["status"]), np.zeros(P, dtype=np.int32))


@pytest.mark.parametrize("n,K", [(4, 1), (16, 2), (16, 8), (40, 4), (64, 1), (100, 2)])
def test_nan_beyond_the_partition_length_is_never_data(n, K):
    """Columns at and beyond part_len[p] are masked whatever they hold: here they hold NaN (also in the
    caller's v0 and under row factors), the lengths end inside a quad of columns, and every path must give
    the oracle's finite results: direct, cooperative, Gram, the verification and the one-call entry."""
    rng = np.random.default_rng(700 + 3 * n + K)
    P, stride = 3, 12_320
    lens = np.array([12_317, 9_002, 5])
    g = make_case(rng, P, n, stride, lens, far_rows=n // 3)
    for p in range(P):
        g[p, :, lens[p]:] = np.nan
    tau = np.array([0.5, 1.0, 2.0])
    seed = 0xABCD00 + n
    ref = oracle.centered_clip(g, tau, lens, init_mode=oracle.INIT_COORD_MEDIAN, max_iters=6)
    for algo in (btard.ALGO_DIRECT, btard.ALGO_DIRECT_COOPERATIVE, btard.ALGO_GRAM):
        _, r = run_gpu_cclip(g, tau, lens, init_mode=btard.INIT_COORD_MEDIAN, max_iters=6, algo=algo)
        assert np.all(np.isfinite(cpu(r["v"]))), algo
        check_cclip(r, ref, lens)
        assert not cpu(r["status"]).any()
    v0 = rng.standard_normal((P, stride)).astype(np.float32)
    for p in range(P):
        v0[p, lens[p]:] = np.nan
    ref0 = oracle.centered_clip(g, tau, lens, init_mode=oracle.INIT_CALLER, v0=v0, max_iters=3)
    _, r0 = run_gpu_cclip(g, tau, lens, init_mode=btard.INIT_CALLER_V0, v0=v0, max_iters=3)
    check_cclip(r0, ref0, lens)
    gd = torch.from_numpy(g).cuda()
    for algo in (btard.ALGO_GRAM, btard.ALGO_DIRECT):
        rc, rv = btard.centered_clip_verify(gd, tau, seed, K=K, part_len=lens, init_mode=btard.INIT_COORD_MEDIAN,
                                            max_iters=6, algo=algo, want_resid_sum=True)
        torch.cuda.synchronize()
        check_cclip(rc, ref, lens)
        v32 = cpu(rc["v"])
        assert np.all(np.isfinite(v32))
        refv = oracle.verify(g, v32, tau, seed, K=K, part_len=lens, want_resid_sum=True)
        check_verify(rv, refv, K)
        assert np.all(np.isfinite(cpu(rv["resid_sum"]))) and not cpu(rv["status"]).any()
    scale = rng.uniform(0.5, 1.0, size=(P, n))
    refs = oracle.centered_clip(g, tau, lens, init_mode=oracle.INIT_COORD_MEDIAN, max_iters=4, row_scale=scale)
    for algo in (btard.ALGO_DIRECT, btard.ALGO_GRAM):
        _, r = run_gpu_cclip(g, tau, lens, init_mode=btard.INIT_COORD_MEDIAN, max_iters=4, algo=algo,
                             row_scale=torch.from_numpy(scale).cuda())
        check_cclip(r, refs, lens)


@pytest.mark.parametrize("n,K", [(16, 1), (16, 8), (64, 4)])
def test_all_work_is_ordered_on_the_callers_stream(n, K):
    """The inputs become valid only late on a side stream (behind ~50 ms of other work there) and the
    outputs are read after that stream alone is synchronised: anything the library queued on another
    stream would read the zeros the buffers held before, or be read too early."""
    rng = np.random.default_rng(1300 + n + K)
    P, stride = 2, 20_000
    lens = np.array([20_000, 17_003])
    g = make_case(rng, P, n, stride, lens, far_rows=n // 3)
    tau = np.array([0.7, 1.5])
    seed = 99
    ref = oracle.centered_clip(g, tau, lens, init_mode=oracle.INIT_COORD_MEDIAN, max_iters=5)
    staged = torch.from_numpy(g).cuda()
    busy = torch.randn((4096, 4096), device="cuda")
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    for algo in (btard.ALGO_DIRECT, btard.ALGO_DIRECT_COOPERATIVE, btard.ALGO_GRAM):
        gd = torch.zeros_like(staged)
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            acc = busy
            for _ in range(40):
                acc = acc @ busy * 1e-3
            gd.copy_(staged, non_blocking=True)
            rc, rv = btard.centered_clip_verify(gd, tau, seed, K=K, part_len=lens, init_mode=btard.INIT_COORD_MEDIAN,
                                                max_iters=5, algo=algo, stream=side)
        side.synchronize()
        check_cclip(rc, ref, lens)
        refv = oracle.verify(g, cpu(rc["v"]), tau, seed, K=K, part_len=lens)
        check_verify(rv, refv, K)
    torch.cuda.synchronize()


@pytest.mark.parametrize("n,K", [(16, 2), (64, 4), (100, 1)])
def test_results_are_bitwise_reproducible(n, K):
    """Cross-CTA sums go through per-CTA slots added in a fixed order, never through floating-point
    atomics: the same call on the same inputs gives the same bits, whatever order the CTAs ran in and
    whatever an earlier call left in the workspaces."""
    rng = np.random.default_rng(1400 + n)
    P, stride = 5, 60_000                       # several CTAs per partition
    lens = np.array([60_000, 59_999, 31_000, 7, 0])
    g = torch.from_numpy(make_case(rng, P, n, stride, lens, far_rows=n // 4)).cuda()
    tau = np.array([0.5, 1.0, 2.0, 1.0, 1.0])
    for algo, stop in ((btard.ALGO_DIRECT, btard.STOP_EPS), (btard.ALGO_DIRECT_COOPERATIVE, btard.STOP_EPS),
                       (btard.ALGO_GRAM, btard.STOP_FIXED_ITERS)):
        runs = []
        ws = None
        for rep in range(3):
            rc, rv = btard.centered_clip_verify(g, tau, 4242, K=K, part_len=lens, init_mode=btard.INIT_COORD_MEDIAN,
                                                stop_mode=stop, max_iters=12, eps=1e-4, algo=algo,
                                                want_resid_sum=True, workspaces=ws)
            torch.cuda.synchronize()
            ws = (rc["workspace"], rv["workspace"])
            runs.append({**{"c_" + k: cpu(rc[k]).copy() for k in ("v", "iters", "last_step_norm", "resid_norm", "status")},
                         **{"v_" + k: cpu(rv[k]).copy() for k in ("norm", "weight", "dot", "s", "s_sum", "znorm2",
                                                                   "resid_sum_norm", "resid_sum", "status")}})
            ws[0].fill_(0xA5)                       # leftovers of another kind for the next call
            ws[1].fill_(0x5A)
        for k in runs[0]:
            for other in runs[1:]:
                assert runs[0][k].tobytes() == other[k].tobytes(), (algo, k)


@pytest.mark.parametrize("n,K", [(4, 1), (16, 3), (40, 2), (100, 1)])
def test_many_small_partitions(n, K):
    """More partitions than the per-launch batch of the partition table (128), than CTAs that fit the GPU at
    once and than SMs: P = 700 short partitions of every length from 0 to the stride."""
    rng = np.random.default_rng(1500 + n)
    P, stride = 700, 96
    lens = rng.integers(0, stride + 1, size=P)
    lens[:3] = (0, stride, 1)
    g = make_case(rng, P, n, stride, lens)       # no far rows: over <= 96 columns their projections are ill-conditioned
    tau = rng.uniform(0.3, 2.0, size=P)
    seed = 31337
    ref = oracle.centered_clip(g, tau, lens, init_mode=oracle.INIT_COORD_MEDIAN, max_iters=4)
    gd = torch.from_numpy(g).cuda()
    for algo in (btard.ALGO_DIRECT, btard.ALGO_DIRECT_COOPERATIVE, btard.ALGO_GRAM):
        rc, rv = btard.centered_clip_verify(gd, tau, seed, K=K, part_len=lens, init_mode=btard.INIT_COORD_MEDIAN,
                                            max_iters=4, algo=algo, partition_base=5)
        torch.cuda.synchronize()
        check_cclip(rc, ref, lens)
        refv = oracle.verify(g, cpu(rc["v"]), tau, seed, K=K, part_len=lens, first_partition=5)
        check_verify(rv, refv, K)


@pytest.mark.parametrize("case", list(range(32)) + [2125, 6441])   # 2125: 3 far rows with factors, 16 directions, one of
def test_random_shapes_match_oracle(case):                         # them nearly orthogonal to every residual (the s_sum
                                                                   # floor); 6441: 2 peers, 1 such direction (the dot floor)
    """Seeded random draws of everything a caller chooses: peers, partitions, row stride, ragged and empty
    lengths, radii, start, stop rule, algorithm, directions, and optionally a radius schedule and row factors."""
    rng = np.random.default_rng(7000 + case)
    n = int(rng.choice([1, 2, 3, 5, 8, 11, 16, 17, 24, 32, 33, 48, 63, 64, 65, 96, 128, 130, 200]))
    P = int(rng.integers(1, 7))
    stride = 32 * int(rng.integers(1, 260))
    lens = rng.integers(0, stride + 1, size=P)
    lens[rng.integers(0, P)] = stride
    if case % 5 == 0:
        lens[rng.integers(0, P)] = 0
    K = int(rng.choice([1, 2, 3, 4, 5, 8, 9, 16]))
    tau = rng.uniform(0.2, 3.0, size=P)
    algos = [btard.ALGO_DIRECT, btard.ALGO_DIRECT_COOPERATIVE] + ([btard.ALGO_GRAM] if n <= 128 else [])
    algo = algos[int(rng.integers(0, len(algos)))]
    init_g, init_o = [(btard.INIT_ZERO, oracle.INIT_ZERO), (btard.INIT_MEAN, oracle.INIT_MEAN),
                      (btard.INIT_COORD_MEDIAN, oracle.INIT_COORD_MEDIAN),
                      (btard.INIT_CALLER_V0, oracle.INIT_CALLER)][int(rng.integers(0, 4))]
    if algo == btard.ALGO_GRAM and init_g in (btard.INIT_ZERO, btard.INIT_CALLER_V0):
        init_g, init_o = btard.INIT_COORD_MEDIAN, oracle.INIT_COORD_MEDIAN    # the Gram variant wants a robust centre
    eps_mode = bool(rng.integers(0, 2))
    max_iters = int(rng.integers(1, 12)) if not eps_mode else 60
    g = make_case(rng, P, n, stride, lens, far_rows=int(rng.integers(0, n // 3 + 1)))
    v0 = rng.standard_normal((P, stride)).astype(np.float32) if init_g == btard.INIT_CALLER_V0 else None
    sched = rng.uniform(0.2, 3.0, size=(P, max_iters)) if (case % 3 == 0 and not eps_mode) else None
    scale = rng.uniform(0.3, 1.0, size=(P, n)) if (case % 4 == 1 and n > 1) else None
    if scale is not None:
        # The GPU rounds the products f x to fp32, the oracle keeps them in fp64: an error of 6e-8 |f x| per
        # coordinate, which is below the tolerance only relative to residuals of the size of the rows
        # themselves.  So these cases have no large common mean.
        g = (g - np.float32(0.95) * g.mean(axis=1, keepdims=True)).astype(np.float32)
        for p in range(P):
            g[p, :, lens[p]:] = 77.0
        if algo == btard.ALGO_DIRECT_COOPERATIVE:
            algo = btard.ALGO_DIRECT                       # the cooperative kernel takes no row factors
    kw_o = dict(init_mode=init_o, v0=v0, max_iters=max_iters, tau_schedule=sched, row_scale=scale)
    kw_g = dict(init_mode=init_g, max_iters=max_iters, algo=algo,
                tau_schedule=None if sched is None else torch.from_numpy(sched).cuda(),
                row_scale=None if scale is None else torch.from_numpy(scale).cuda())
    if eps_mode:
        kw_o.update(stop_mode=oracle.STOP_EPS, eps=1e-4)
        kw_g.update(stop_mode=btard.STOP_EPS, eps=1e-4)
    ref = oracle.centered_clip(g, tau, lens, **kw_o)
    gd = torch.from_numpy(g).cuda()
    vd = torch.from_numpy(v0).cuda().clone() if v0 is not None else None
    seed = 0xC0FFEE + case
    rc, rv = btard.centered_clip_verify(gd, tau, seed, K=K, part_len=lens, v=vd, partition_base=case,
                                        want_resid_sum=True, **kw_g)
    torch.cuda.synchronize()
    if eps_mode:
        it = cpu(rc["iters"])
        assert np.all(np.abs(it - ref["iters"]) <= 1), (it, ref["iters"])
        same = it == ref["iters"]
        v = cpu(rc["v"])
        for p in np.nonzero(same)[0]:
            assert rel_l2(v[p, : lens[p]], ref["v"][p, : lens[p]]) <= RTOL, ("v", p)
    else:
        check_cclip(rc, ref, lens, gram=(algo == btard.ALGO_GRAM))
    refv = oracle.verify(g, cpu(rc["v"]), tau, seed, K=K, part_len=lens, first_partition=case, want_resid_sum=True,
                         row_scale=scale)
    check_verify(rv, refv, K)
    for p in range(P):
        rscale = (refv["weight"][p] * refv["norm"][p]).sum() + 1e-300
        assert np.linalg.norm(cpu(rv["resid_sum"])[p, : lens[p]] - refv["resid_sum"][p, : lens[p]]) <= RTOL * rscale


@pytest.mark.parametrize("case", range(10))
def test_random_long_rows_match_oracle(case):
    """The same kind of draw with rows of 10 000 to 190 000 columns (several tiles and CTAs per partition, ragged
    ends inside a tile), a few fixed updates: peers, radii, start, algorithm, directions, schedule, row factors."""
    rng = np.random.default_rng(90000 + case)
    n = int(rng.choice([2, 5, 8, 12, 16, 17, 24, 32, 40, 48, 63, 64, 65, 100]))
    P = int(rng.integers(1, 4))
    stride = 32 * int(rng.integers(300, 6000))
    lens = rng.integers(stride // 2, stride + 1, size=P)
    lens[rng.integers(0, P)] = stride
    K = int(rng.choice([1, 2, 4, 5, 8]))
    tau = rng.uniform(2.0, 30.0, size=P)
    algo = [btard.ALGO_DIRECT, btard.ALGO_DIRECT_COOPERATIVE, btard.ALGO_GRAM][int(rng.integers(0, 3))]
    init_g, init_o = [(btard.INIT_MEAN, oracle.INIT_MEAN),
                      (btard.INIT_COORD_MEDIAN, oracle.INIT_COORD_MEDIAN)][int(rng.integers(0, 2))]
    max_iters = int(rng.integers(1, 6))
    g = make_case(rng, P, n, stride, lens, far_rows=int(rng.integers(0, n // 3 + 1)))
    sched = rng.uniform(2.0, 30.0, size=(P, max_iters)) if case % 3 == 0 else None
    scale = rng.uniform(0.3, 1.0, size=(P, n)) if case % 4 == 1 else None
    if scale is not None:                                  # as above: no large common mean under row factors
        g = (g - np.float32(0.95) * g.mean(axis=1, keepdims=True)).astype(np.float32)
        for p in range(P):
            g[p, :, lens[p]:] = 77.0
        if algo == btard.ALGO_DIRECT_COOPERATIVE:
            algo = btard.ALGO_DIRECT
    ref = oracle.centered_clip(g, tau, lens, init_mode=init_o, max_iters=max_iters, tau_schedule=sched, row_scale=scale)
    seed = 0xBEEF + case
    rc, rv = btard.centered_clip_verify(torch.from_numpy(g).cuda(), tau, seed, K=K, part_len=lens, partition_base=case,
                                        want_resid_sum=True, init_mode=init_g, max_iters=max_iters, algo=algo,
                                        tau_schedule=None if sched is None else torch.from_numpy(sched).cuda(),
                                        row_scale=None if scale is None else torch.from_numpy(scale).cuda())
    torch.cuda.synchronize()
    check_cclip(rc, ref, lens, gram=(algo == btard.ALGO_GRAM))
    refv = oracle.verify(g, cpu(rc["v"]), tau, seed, K=K, part_len=lens, first_partition=case, want_resid_sum=True,
                         row_scale=scale)
    check_verify(rv, refv, K)


@pytest.mark.parametrize("n,K", [(5, 1), (16, 2), (16, 3), (40, 1)])
def test_empty_partition_in_every_path(n, K):
    """A partition without coordinates (possible when d < P): v stays 0, norms and projections are
    empty sums, s is 0 and not 0/0; in the separate calls, the Gram variant and the one-call entry."""
    rng = np.random.default_rng(900 + n + K)
    P, stride = 3, 4096
    lens = np.array([4096, 0, 17])
    g = make_case(rng, P, n, stride, lens, far_rows=n // 3)
    tau = np.array([0.5, 1.0, 2.0])
    gd = torch.from_numpy(g).cuda()
    refc = oracle.centered_clip(g, tau, lens, init_mode=oracle.INIT_COORD_MEDIAN, max_iters=5)
    for algo in (btard.ALGO_DIRECT, btard.ALGO_GRAM):
        _, r = run_gpu_cclip(g, tau, lens, init_mode=btard.INIT_COORD_MEDIAN, max_iters=5, algo=algo)
        check_cclip(r, refc, lens)
        v32 = cpu(r["v"])
        refv = oracle.verify(g, v32, tau, 3, K=K, part_len=lens)
        out = btard.verify_projections(gd, r["v"], tau, 3, K=K, part_len=lens, resid_norm_in=r["resid_norm"])
        torch.cuda.synchronize()
        check_verify(out, refv, K)
        assert np.all(cpu(out["s"])[1] == 0.0) and np.all(cpu(out["znorm2"])[1] == 0.0)
        rc, rv = btard.centered_clip_verify(gd, tau, 3, K=K, part_len=lens, init_mode=btard.INIT_COORD_MEDIAN,
                                            max_iters=5, algo=algo)
        torch.cuda.synchronize()
        check_cclip(rc, refc, lens)
        check_verify(rv, oracle.verify(g, cpu(rc["v"]), tau, 3, K=K, part_len=lens), K)
        assert np.all(cpu(rv["s"])[1] == 0.0)


def test_one_call_reports_a_non_finite_row():
    rng = np.random.default_rng(77)
    P, n, stride = 2, 8, 4096
    lens = np.array([4096, 4001])
    g = make_case(rng, P, n, stride, lens)
    g[1, 3, 17] = np.inf
    rc, rv = btard.centered_clip_verify(torch.from_numpy(g).cuda(), 1.0, 5, K=1, part_len=lens,
                                        init_mode=btard.INIT_MEAN, max_iters=4, algo=btard.ALGO_GRAM)
    torch.cuda.synchronize()
    assert cpu(rc["status"])[1] & btard.STATUS_NONFINITE_ROW and not cpu(rc["status"])[0] & btard.STATUS_NONFINITE_ROW
    assert cpu(rv["status"])[1] & btard.STATUS_NONFINITE_ROW
    assert cpu(rv["weight"])[1, 3] == 0.0


def test_verify_partition_base_keys_z():
    rng = np.random.default_rng(9)
    P, n, stride, K = 2, 4, 1024, 2
    lens = np.array([1024, 1001])
    g = make_case(rng, P, n, stride, lens)
    v = np.zeros((P, stride), dtype=np.float32)
    ref = oracle.verify(g, v, 1.0, 11, K=K, part_len=lens, first_partition=5)
    out = btard.verify_projections(torch.from_numpy(g).cuda(), torch.from_numpy(v).cuda(), 1.0, 11, K=K,
                                   part_len=lens, partition_base=5)
    torch.cuda.synchronize()
    check_verify(out, ref, K)


def test_wrong_aggregate_is_exposed_on_the_gpu_too():
    """Aggregation attack (App. C): a modified v makes sum_i s_i visibly non-zero."""
    w = workloads.make_workload(1)
    g = w.g.cuda()
    r = btard.centered_clip(g, w.tau, part_len=w.part_len, init_mode=btard.INIT_COORD_MEDIAN,
                            stop_mode=btard.STOP_EPS, max_iters=500, eps=1e-7)
    good = btard.verify_projections(g, r["v"], w.tau, 0, K=4, part_len=w.part_len,
                                    resid_norm_in=r["resid_norm"])
    bad_v = r["v"] + 0.01 * torch.randn_like(r["v"])
    bad = btard.verify_projections(g, bad_v, w.tau, 0, K=4, part_len=w.part_len)
    torch.cuda.synchronize()
    sg, sb = cpu(good["s_sum"])[0], cpu(bad["s_sum"])[0]
    scale = np.abs(cpu(good["s"])[0]).sum(0)
    assert np.all(np.abs(sg) < 1e-4 * scale)
    assert np.all(np.abs(sb) > 10 * np.abs(sg))


def test_verification_checks_are_bit_exact():
    """Integer/boolean outputs: same fp64 inputs, same fp64 comparisons, identical flags."""
    rng = np.random.default_rng(15)
    P, n, K = 7, 23, 3
    norm = np.abs(rng.standard_normal((P, n))) * 2
    s = rng.standard_normal((P, n, K))
    s[:, -1, :] = -s[:, :-1, :].sum(axis=1)                       # sums to ~0 up to rounding
    nr = norm.copy(); sr = s.copy()
    nr[1, 3] *= 1 + 1e-9; nr[2, 0] = np.nan; sr[4, 5, 1] += 1e-7; sr[6, :, 0] += 0.01
    dmax = np.array([0.5, 1.0, 1.5, 2.0, np.inf, 0.0, 1.3])
    for tol in (dict(), dict(rel_tol=1e-8, abs_tol=1e-12, sum_tol=1e-9), dict(rel_tol=1e-3, sum_tol=1e-2)):
        for rep in (dict(), dict(norm_reported=nr, s_reported=sr)):
            ref = oracle.checks(norm, s, dmax, **rep, **tol)
            dev = {k: torch.from_numpy(v).cuda() for k, v in rep.items()}
            out = btard.verification_checks(torch.from_numpy(norm).cuda(), torch.from_numpy(s).cuda(),
                                            torch.from_numpy(dmax).cuda(), **dev, **tol)
            torch.cuda.synchronize()
            for key in ref:
                assert np.array_equal(cpu(out[key]), ref[key]), (key, tol, list(rep))


def test_checks_on_library_outputs_catch_a_shifted_aggregate():
    w = workloads.make_workload(1)
    g = w.g.cuda()
    r = btard.centered_clip(g, w.tau, part_len=w.part_len, init_mode=btard.INIT_COORD_MEDIAN,
                            stop_mode=btard.STOP_EPS, max_iters=500, eps=1e-7)
    good = btard.verify_projections(g, r["v"], w.tau, 0, K=2, part_len=w.part_len, resid_norm_in=r["resid_norm"])
    dmax = torch.tensor([5.0], dtype=torch.float64, device="cuda")
    ok = btard.verification_checks(good["norm"], good["s"], dmax, sum_tol=1e-4)
    bad = btard.verify_projections(g, r["v"] + 1.0, w.tau, 0, K=2, part_len=w.part_len)
    flagged = btard.verification_checks(bad["norm"], bad["s"], dmax, sum_tol=1e-4)
    torch.cuda.synchronize()
    assert not cpu(ok["sum_violation"]).any() and cpu(ok["check_averaging"])[0] == 0
    assert cpu(flagged["sum_violation"]).all() and cpu(flagged["check_averaging"])[0] == 1
    # a peer that misreports its inner product is singled out
    sr = good["s"].clone(); sr[0, 2, 1] += 0.5
    acc = btard.verification_checks(good["norm"], good["s"], dmax, s_reported=sr, rel_tol=1e-9, sum_tol=1e-4)
    torch.cuda.synchronize()
    assert cpu(acc["s_mismatch"]).sum() == 1 and cpu(acc["s_mismatch"])[0, 2, 1] == 1
    assert cpu(acc["sum_violation"])[0, 1] == 1


# ----------------------------------------------------------------------------- host-buffer path
def test_aggregate_host_matches_device_path():
    rng = np.random.default_rng(10)
    P, n, stride, K = 3, 16, 4128, 2
    lens = np.array([4128, 4100, 4001])
    g = make_case(rng, P, n, stride, lens, far_rows=4)
    gh = torch.from_numpy(g).pin_memory()
    h = btard.aggregate_host(gh, 1.0, 77, K=K, part_len=lens, init_mode=btard.INIT_COORD_MEDIAN,
                             max_iters=7)
    gd = torch.from_numpy(g).cuda()
    r = btard.centered_clip(gd, 1.0, part_len=lens, init_mode=btard.INIT_COORD_MEDIAN, max_iters=7)
    o = btard.verify_projections(gd, r["v"], 1.0, 77, K=K, part_len=lens, resid_norm_in=r["resid_norm"])
    torch.cuda.synchronize()
    assert torch.equal(h["v"], r["v"].cpu())
    for key in ("norm", "weight", "dot", "s", "s_sum", "znorm2", "resid_sum_norm"):
        assert torch.equal(h[key], o[key].cpu()), key
    assert torch.equal(h["iters"], r["iters"].cpu())
    # chunked, with the copies on a second stream: same numbers (z is keyed by the global partition)
    h2 = btard.aggregate_host(gh, 1.0, 77, K=K, part_len=lens, init_mode=btard.INIT_COORD_MEDIAN,
                              max_iters=7, copy_stream=torch.cuda.Stream())
    assert torch.equal(h2["iters"], h["iters"])
    for key in ("v", "norm", "weight", "dot", "s", "znorm2"):      # other CTA grouping: last bits may differ
        assert rel_l2(h2[key].numpy(), h[key].numpy()) <= 1e-6, key


def test_aggregate_host_gram_path_and_uneven_chunks():
    """The host-buffer call with the Gram variant, and a partition count whose chunks of P/4 need more
    workspace than the whole batch would (fewer partitions get more CTAs each): 38 partitions, K = 8."""
    rng = np.random.default_rng(21)
    P, n, stride, K = 38, 16, 8192, 8
    lens = np.full(P, stride)
    lens[-1] = 4097
    g = make_case(rng, P, n, stride, lens, far_rows=4)
    gh = torch.from_numpy(g).pin_memory()
    refc = oracle.centered_clip(g, 1.0, lens, init_mode=oracle.INIT_COORD_MEDIAN, max_iters=7)
    for algo in (btard.ALGO_DIRECT, btard.ALGO_GRAM):
        for cs in (None, torch.cuda.Stream()):
            h = btard.aggregate_host(gh, 1.0, 77, K=K, part_len=lens, init_mode=btard.INIT_COORD_MEDIAN,
                                     max_iters=7, copy_stream=cs, algo=algo)
            hc = dict(v=h["v"].cuda(), iters=h["iters"], resid_norm=h["norm"], last_step_norm=h["last_step_norm"])
            check_cclip(hc, refc, lens)
            refv = oracle.verify(g, h["v"].numpy(), 1.0, 77, K=K, part_len=lens, norm_in=h["norm"].numpy())
            check_verify(h, refv, K)
            assert not h["status"].numpy().any()
    # eps mode through the host call: the cooperative kernel per chunk, and the Gram variant
    refe = oracle.centered_clip(g, 1.0, lens, init_mode=oracle.INIT_COORD_MEDIAN, stop_mode=oracle.STOP_EPS,
                                max_iters=40, eps=1e-4)
    for algo in (btard.ALGO_DIRECT, btard.ALGO_GRAM):
        h = btard.aggregate_host(gh, 1.0, 77, K=K, part_len=lens, init_mode=btard.INIT_COORD_MEDIAN,
                                 stop_mode=btard.STOP_EPS, max_iters=40, eps=1e-4,
                                 copy_stream=torch.cuda.Stream(), algo=algo)
        hc = dict(v=h["v"].cuda(), iters=h["iters"], resid_norm=h["norm"], last_step_norm=h["last_step_norm"])
        check_cclip(hc, refe, lens, eps_mode=True, g=g, tau=1.0, init=oracle.INIT_COORD_MEDIAN)


# ----------------------------------------------------------------------------- full-size configs
_WORKLOADS = {}
_ORACLE_MEMO = {}


def _workload(cfg):
    """Full-size configurations 2-4 on the GPU, generated once per test session (5.6 GB in all)."""
    if cfg not in _WORKLOADS:
        _WORKLOADS[cfg] = workloads.make_workload(cfg, device="cuda")
    return _WORKLOADS[cfg]


def _full_config(cfg, sample, max_iters=None, stop=None, algo=None, one_call=False):
    """Runs configuration `cfg` (a number, or a workload already on the GPU) at full size in the
    benchmark's launch configuration and compares the sampled partitions with the oracle.  one_call:
    through btard_centered_clip_verify, as the benchmark does for the Gram variant."""
    w = _workload(cfg) if isinstance(cfg, int) else cfg
    stop_mode = w.stop_mode if stop is None else stop
    iters = w.max_iters if max_iters is None else max_iters
    if one_call:
        r, o = btard.centered_clip_verify(w.g, w.tau, w.zseed, K=w.K, part_len=w.part_len,
                                          init_mode=btard.INIT_COORD_MEDIAN, stop_mode=stop_mode, max_iters=iters,
                                          eps=w.eps, algo=btard.ALGO_DIRECT if algo is None else algo)
    else:
        r = btard.centered_clip(w.g, w.tau, part_len=w.part_len, init_mode=btard.INIT_COORD_MEDIAN,
                                stop_mode=stop_mode, max_iters=iters, eps=w.eps,
                                algo=btard.ALGO_DIRECT if algo is None else algo)
        o = btard.verify_projections(w.g, r["v"], w.tau, w.zseed, K=w.K, part_len=w.part_len,
                                     resid_norm_in=r["resid_norm"])
    torch.cuda.synchronize()
    sample = list(sample)
    idx = torch.tensor(sample, device=w.g.device)
    gs = cpu(w.g.index_select(0, idx))                       # the oracle runs the sampled partitions in parallel
    lens, taus = w.part_len[sample], w.tau[sample]
    key = (id(w), tuple(sample), stop_mode, iters)           # the same reference serves every algorithm
    if key not in _ORACLE_MEMO:
        _ORACLE_MEMO.clear()
        _ORACLE_MEMO[key] = oracle.centered_clip(gs, taus, lens, init_mode=oracle.INIT_COORD_MEDIAN,
                                                 stop_mode=stop_mode, max_iters=iters, eps=w.eps)
    ref = _ORACLE_MEMO[key]
    sub = {k: r[k].index_select(0, idx) for k in ("v", "iters", "resid_norm", "last_step_norm", "status")}
    check_cclip(sub, ref, lens, eps_mode=(stop_mode == btard.STOP_EPS), g=gs, tau=taus,
                init=oracle.INIT_COORD_MEDIAN)
    for s, p in enumerate(sample):                           # z is keyed by the partition's true index
        refv = oracle.verify(gs[s:s + 1], cpu(sub["v"][s:s + 1]), taus[s], w.zseed, K=w.K, part_len=lens[s:s + 1],
                             norm_in=cpu(sub["resid_norm"][s:s + 1]), first_partition=p)
        subo = {k: o[k][p:p + 1] for k in ("norm", "weight", "dot", "s", "s_sum", "znorm2",
                                          "resid_sum_norm")}
        check_verify(subo, refv, w.K)
    return w, r, o


def test_config2_full_size_all_partitions():
    _full_config(2, sample=range(16))
    # fixed-iteration parity at full size as well (eps mode may differ by one update)
    _full_config(2, sample=range(16), max_iters=10, stop=btard.STOP_FIXED_ITERS)


def test_config3_full_size_all_partitions():
    _full_config(3, sample=range(16), max_iters=10, stop=btard.STOP_FIXED_ITERS)
    _full_config(3, sample=range(16))


def test_config4_full_size_all_partitions():
    _full_config(4, sample=range(0, 64, 2))
    _full_config(4, sample=range(1, 64, 2), max_iters=5, stop=btard.STOP_FIXED_ITERS)


def test_config2_and_4_gram_mode_full_size():
    _full_config(2, sample=range(16), max_iters=20, stop=btard.STOP_FIXED_ITERS, algo=btard.ALGO_GRAM)
    _full_config(4, sample=range(0, 64, 4), algo=btard.ALGO_GRAM)


def test_gram_one_call_full_size():
    """The Gram variant through the one-call entry point (fused combine-and-verify pass) at full size."""
    _full_config(2, sample=range(16), max_iters=20, stop=btard.STOP_FIXED_ITERS, algo=btard.ALGO_GRAM, one_call=True)
    _full_config(3, sample=range(16), algo=btard.ALGO_GRAM, one_call=True)
    _full_config(4, sample=range(2, 64, 4), algo=btard.ALGO_GRAM, one_call=True)


def test_config5_full_size_sampled():
    """Config 5 at full size (64 GiB of rows): fixed 20 iterations and the Gram variant side by side
    (separate calls and the one-call entry point), four 1 GiB partitions checked against the oracle
    together with the verification pass (K = 4)."""
    _WORKLOADS.clear()
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    d = 1 << 28 if free > 90 * (1 << 30) else 1 << 26              # smaller boards: a quarter of the length
    w = workloads.make_workload(5, device="cuda", d=d)
    sample = [3, 22, 41, 60]
    _full_config(w, sample, algo=btard.ALGO_DIRECT)
    _full_config(w, sample, algo=btard.ALGO_GRAM)
    _full_config(w, sample, algo=btard.ALGO_GRAM, one_call=True)
