"""Pins for the float64 oracle: each test checks it against something the paper or the
mathematics fixes, never against the oracle itself or the CUDA path."""
import math
import os

import numpy as np
import pytest
from scipy import stats

import oracle

HERE = os.path.dirname(os.path.abspath(__file__))


def clipped_residual_sum(x, v, tau):
    """Left-hand side of the CenteredClip fixed-point equation (Sec. 3.1 eq. (1)), evaluated
    with numpy for a candidate v.  Used only to test a *result*; it is not the iteration."""
    r = x.astype(np.float64) - v[None, :]
    rho = np.linalg.norm(r, axis=1)
    w = np.where(rho <= tau, 1.0, tau / np.maximum(rho, 1e-300))
    return (w[:, None] * r).sum(0), rho, w


# ----------------------------------------------------------------------------- Philox / z
def test_philox_known_answers():
    """Published Philox4x32-10 vectors (Random123, SC'11)."""
    rows = [l.split() for l in open(os.path.join(HERE, "golden", "philox4x32_10_kat.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        w = [int(t, 16) for t in r]
        out = oracle.philox4x32_10(w[0:4], w[4:6])
        assert [int(t) for t in out] == w[6:10]


def test_philox_is_a_bijection_of_the_counter():
    """A counter-based generator permutes counters for a fixed key: distinct counters must give
    distinct blocks, and each counter word must matter."""
    base = oracle.philox4x32_10([5, 6, 7, 8], [9, 10])
    for pos in range(4):
        c = [5, 6, 7, 8]
        c[pos] += 1
        assert not np.array_equal(oracle.philox4x32_10(c, [9, 10]), base)
    assert not np.array_equal(oracle.philox4x32_10([5, 6, 7, 8], [9, 11]), base)
    assert not np.array_equal(oracle.philox4x32_10([5, 6, 7, 8], [10, 10]), base)


def _box_muller_libm(seed, p, k, length):
    """Textbook Box-Muller in float64 with libm, fed by the same Philox words and the same
    word -> uniform maps as the definition of z."""
    out = np.zeros(length)
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for q in range((length + 3) // 4):
        w = [int(t) for t in oracle.philox4x32_10([q, p, k, 0x42544152], key)]
        vals = []
        for a, b in ((w[0], w[1]), (w[2], w[3])):
            u = ((a >> 8) + 1) / 2.0 ** 24
            frac = (((b >> 6) & 0xFFFFFF) + 0.5) / 2.0 ** 24      # position inside the quadrant
            theta = (math.pi / 2) * frac
            r = math.sqrt(-2.0 * math.log(u))
            n0, n1 = r * math.cos(theta), r * math.sin(theta)
            if b & 0x80000000:
                n0 = -n0
            if b & 0x40000000:
                n1 = -n1
            vals += [n0, n1]
        for t in range(4):
            if 4 * q + t < length:
                out[4 * q + t] = vals[t]
    return out


def test_z_matches_libm_box_muller():
    """The fp32 polynomial transform is a Box-Muller: it must agree with a libm one to ~1e-5."""
    for seed, p, k in [(0, 0, 0), (0x1234567890ABCDEF, 3, 2)]:
        z = oracle.random_vector(seed, p, k, 4001)
        ref = _box_muller_libm(seed, p, k, 4001)
        assert np.max(np.abs(z - ref)) < 2e-5 * (1 + np.max(np.abs(ref)))


def test_z_is_standard_normal():
    """iid N(0,1) coordinates <=> uniform direction after normalisation (App. D.5)."""
    z = oracle.random_vector(7, 1, 0, 1 << 20).astype(np.float64)
    n = z.size
    assert abs(z.mean()) < 5 / math.sqrt(n)
    assert abs(z.var() - 1) < 5 * math.sqrt(2 / n)
    assert abs(stats.kurtosis(z)) < 5 * math.sqrt(24 / n)
    assert abs(stats.skew(z)) < 5 * math.sqrt(6 / n)
    assert stats.kstest(z[:200000], "norm").pvalue > 1e-3
    # E ||z||^2 = length
    assert abs((z ** 2).sum() / n - 1) < 5 * math.sqrt(2 / n)
    # lanes of one Philox block, and neighbouring blocks, are uncorrelated
    for lag in (1, 2, 3, 4):
        assert abs(np.mean(z[:-lag] * z[lag:])) < 5 / math.sqrt(n)


def test_z_streams_differ_by_seed_partition_and_index():
    a = oracle.random_vector(1, 0, 0, 4096).astype(np.float64)
    for args in [(2, 0, 0), (1, 1, 0), (1, 0, 1), (1 << 32 | 1, 0, 0)]:
        b = oracle.random_vector(*args, 4096).astype(np.float64)
        assert abs(np.corrcoef(a, b)[0, 1]) < 0.08


def test_z_prefix_property_and_ragged_tail():
    """Coordinate c depends on (seed, p, k, c) only, whatever the length."""
    full = oracle.random_vector(3, 2, 1, 1027)
    for ln in (0, 1, 2, 3, 5, 1024, 1026):
        assert np.array_equal(oracle.random_vector(3, 2, 1, ln), full[:ln])


# ----------------------------------------------------------------------------- Split
@pytest.mark.parametrize("d,P", [(10, 3), (11173962, 16), (17683968, 64), (1 << 28, 64), (5, 8), (7, 7)])
def test_split_paper_sizes(d, P):
    """Split(v, n): first d mod n parts ceil(d/n), the rest floor(d/n) (App. D.1)."""
    off, ln, stride = oracle.partition_layout(d, P, oracle.SPLIT_PAPER, 32)
    assert ln.sum() == d
    assert np.all(ln[: d % P] == -(-d // P)) and np.all(ln[d % P:] == d // P)
    assert np.array_equal(off, np.concatenate([[0], np.cumsum(ln)[:-1]]))
    assert stride % 32 == 0 and stride >= ln.max() and stride - ln.max() < 32


def test_split_ceil_pad_sizes():
    off, ln, stride = oracle.partition_layout(11173962, 16, oracle.SPLIT_CEIL_PAD, 32)
    assert list(ln[:15]) == [698373] * 15 and ln[15] == 11173962 - 15 * 698373 == 698367
    assert stride == 698400 and ln.sum() == 11173962
    off, ln, stride = oracle.partition_layout(5, 4, oracle.SPLIT_CEIL_PAD, 4)
    assert list(ln) == [2, 2, 1, 0] and list(off) == [0, 2, 4, 5] and stride == 4


# ----------------------------------------------------------------------------- CenteredClip
def rand_rows(rng, n, L, scale=1.0):
    return (rng.standard_normal((n, L)) * scale).astype(np.float32)


@pytest.mark.parametrize("init", [oracle.INIT_ZERO, oracle.INIT_MEAN, oracle.INIT_COORD_MEDIAN])
def test_tau_inf_gives_mean_in_one_step(init):
    """tau = inf: good peers compute an exact average (App. E; eq. (CenteredClip))."""
    rng = np.random.default_rng(0)
    x = rand_rows(rng, 7, 133, 3.0)
    r = oracle.centered_clip(x, np.inf, init_mode=init, max_iters=1)
    assert np.allclose(r["v"][0], x.astype(np.float64).mean(0), rtol=0, atol=1e-14)
    r = oracle.centered_clip(x, np.inf, init_mode=init, max_iters=5)
    assert np.allclose(r["v"][0], x.astype(np.float64).mean(0), rtol=0, atol=1e-14)


def test_all_inside_radius_gives_mean():
    """Inside the sphere of radius tau CenteredClip behaves like the mean (App. D.2)."""
    rng = np.random.default_rng(1)
    x = rand_rows(rng, 5, 64, 0.01)
    r = oracle.centered_clip(x, 1.0, init_mode=oracle.INIT_ZERO, max_iters=1)
    assert np.allclose(r["v"][0], x.astype(np.float64).mean(0), atol=1e-15)


def test_single_row_moves_by_tau_then_lands():
    """n = 1: the fixed point is the row itself; while farther than tau, v moves exactly tau
    toward it per update."""
    x = np.zeros((1, 8), dtype=np.float32)
    x[0, 0], x[0, 1] = 3.0, 4.0                                   # distance 5 from the origin
    for iters, dist in [(1, 4.0), (2, 3.0), (4, 1.0), (5, 0.0), (9, 0.0)]:
        r = oracle.centered_clip(x, 1.0, init_mode=oracle.INIT_ZERO, max_iters=iters)
        v = r["v"][0]
        assert abs(np.linalg.norm(x[0] - v) - dist) < 1e-12
        assert abs(r["resid_norm"][0, 0] - dist) < 1e-12
        if dist > 0:
            assert np.allclose(v[:2] / np.linalg.norm(v[:2]), [0.6, 0.8])
    r = oracle.centered_clip(x, 10.0, init_mode=oracle.INIT_ZERO, max_iters=1)
    assert np.array_equal(r["v"][0], x[0].astype(np.float64))


def test_one_dimensional_closed_form():
    """Two points 0 and D on a line, v0 = 0, tau < D/2: the far point always pulls with force
    tau, the near one with -v, so v_{l+1} = (v_l + tau)/2 and v_l = tau (1 - 2^-l)."""
    x = np.array([[0.0], [10.0]], dtype=np.float32)
    tau = 1.5
    for l in (1, 2, 3, 7, 20):
        r = oracle.centered_clip(x, tau, init_mode=oracle.INIT_ZERO, max_iters=l)
        assert abs(r["v"][0, 0] - tau * (1 - 2.0 ** -l)) < 1e-13
        assert abs(r["last_step_norm"][0] - tau * 2.0 ** -l) < 1e-13
        assert r["iters"][0] == l


def test_three_points_clip_weight_and_one_over_n():
    """v0 = 0, rows (3,0), (0,0.5), (-0.2,0), tau = 1: only the first is clipped (to length 1), so
    one update gives ((1,0) + (0,.5) + (-.2,0)) / 3."""
    x = np.array([[3, 0], [0, 0.5], [-0.2, 0]], dtype=np.float32)
    r = oracle.centered_clip(x, 1.0, init_mode=oracle.INIT_ZERO, max_iters=1)
    assert np.allclose(r["v"][0], [(1 - np.float32(0.2)) / 3, 0.5 / 3], atol=1e-15)


def test_tie_and_zero_residual_have_weight_one():
    """||r|| = tau and ||r|| = 0 both take weight 1 (no division)."""
    x = np.array([[1.0, 0.0], [0.0, 0.0]], dtype=np.float32)
    r = oracle.centered_clip(x, 1.0, init_mode=oracle.INIT_ZERO, max_iters=1)
    assert np.allclose(r["v"][0], [0.5, 0.0], atol=0)


def test_tau_zero_never_moves():
    rng = np.random.default_rng(2)
    x = rand_rows(rng, 4, 16)
    r = oracle.centered_clip(x, 0.0, init_mode=oracle.INIT_ZERO, max_iters=3)
    assert np.array_equal(r["v"][0], np.zeros(16))


def test_small_tau_step_is_mean_of_unit_vectors():
    """tau -> 0: each update is (tau/n) * sum of unit vectors toward the rows (geometric-median
    regime, App. D.2), hence no longer than tau."""
    rng = np.random.default_rng(3)
    x = rand_rows(rng, 6, 32, 5.0)
    tau = 1e-3
    r = oracle.centered_clip(x, tau, init_mode=oracle.INIT_ZERO, max_iters=1)
    unit = x.astype(np.float64) / np.linalg.norm(x.astype(np.float64), axis=1, keepdims=True)
    assert np.allclose(r["v"][0], tau * unit.mean(0), atol=1e-16)
    assert r["last_step_norm"][0] <= tau


def test_permutation_invariance():
    rng = np.random.default_rng(4)
    x = rand_rows(rng, 9, 77, 2.0)
    a = oracle.centered_clip(x, 1.0, init_mode=oracle.INIT_COORD_MEDIAN, max_iters=7)
    perm = rng.permutation(9)
    b = oracle.centered_clip(x[perm], 1.0, init_mode=oracle.INIT_COORD_MEDIAN, max_iters=7)
    assert np.allclose(a["v"], b["v"], atol=1e-13)
    assert np.allclose(a["resid_norm"][0][perm], b["resid_norm"][0], atol=1e-12)


def test_fixed_point_equation_holds_at_convergence():
    """At convergence sum_i (g_i - v) min{1, tau/||g_i - v||} = 0 (Sec. 3.1 eq. (1))."""
    rng = np.random.default_rng(5)
    x = rand_rows(rng, 16, 200, 0.05)
    x[:5] = rand_rows(rng, 5, 200, 30.0)                          # far rows, always clipped
    r = oracle.centered_clip(x, 1.0, init_mode=oracle.INIT_COORD_MEDIAN,
                             stop_mode=oracle.STOP_EPS, max_iters=2000, eps=1e-12)
    assert r["status"][0] == 0 and r["last_step_norm"][0] <= 1e-12
    lhs, rho, w = clipped_residual_sum(x, r["v"][0], 1.0)
    assert np.linalg.norm(lhs) < 16 * 1.01e-12
    assert np.allclose(r["resid_norm"][0], rho, rtol=1e-12)
    assert (w < 1).sum() >= 5 and (w == 1).sum() >= 1            # both branches are exercised


def test_update_equals_clipped_residual_sum_over_n():
    """sum_i Delta_i = n (v^{l+1} - v^l): consecutive oracle iterates differ by the clipped
    residual sum at the earlier one, evaluated independently."""
    rng = np.random.default_rng(6)
    x = rand_rows(rng, 8, 50, 1.0)
    a = oracle.centered_clip(x, 2.0, init_mode=oracle.INIT_ZERO, max_iters=3)
    b = oracle.centered_clip(x, 2.0, init_mode=oracle.INIT_ZERO, max_iters=4)
    lhs, _, _ = clipped_residual_sum(x, a["v"][0], 2.0)
    assert np.allclose(b["v"][0] - a["v"][0], lhs / 8, atol=1e-14)
    assert abs(b["last_step_norm"][0] - np.linalg.norm(lhs) / 8) < 1e-14


def test_byzantine_shift_bound_with_identical_honest_rows():
    """b Byzantine rows shift the output by at most tau*b/n per update (App. C, gradient
    attacks); with identical honest rows and v0 on them, ||v^I - x|| <= I tau b / n, and with
    b = 0 the point is fixed."""
    rng = np.random.default_rng(7)
    n, b, L, tau = 10, 3, 40, 0.7
    honest = rng.standard_normal(L).astype(np.float32)
    x = np.tile(honest, (n, 1))
    r = oracle.centered_clip(x, tau, init_mode=oracle.INIT_CALLER, v0=honest[None], max_iters=5)
    assert np.array_equal(r["v"][0], honest.astype(np.float64)) and r["last_step_norm"][0] == 0
    x[:b] = rand_rows(rng, b, L, 1e4)
    prev = honest.astype(np.float64)
    for I in range(1, 6):
        r = oracle.centered_clip(x, tau, init_mode=oracle.INIT_CALLER, v0=honest[None], max_iters=I)
        v = r["v"][0]
        assert np.linalg.norm(v - honest) <= I * tau * b / n + 1e-12
        assert r["last_step_norm"][0] <= tau + 1e-12
        prev = v
    # one update from the honest point is exactly (tau/n) * sum of unit vectors to the attackers
    r = oracle.centered_clip(x, tau, init_mode=oracle.INIT_CALLER, v0=honest[None], max_iters=1)
    dirs = x[:b].astype(np.float64) - honest
    dirs /= np.linalg.norm(dirs, axis=1, keepdims=True)
    assert np.allclose(r["v"][0] - honest, tau / n * dirs.sum(0), atol=1e-14)


def test_coordinate_median_start_is_the_sorted_middle():
    rng = np.random.default_rng(8)
    for n in (1, 2, 5, 8):
        x = rand_rows(rng, n, 33)
        x[0, 0] = np.inf
        if n > 2:
            x[1, 1] = -np.inf
        # tau = 0 freezes v at v0, exposing the initialiser
        r = oracle.centered_clip(x, 0.0, init_mode=oracle.INIT_COORD_MEDIAN, max_iters=1)
        assert np.array_equal(r["v"][0], np.median(x.astype(np.float64), axis=0))


def test_coordinate_median_orders_nans_at_the_ends():
    """IEEE 754 totalOrder puts -NaN below -inf and +NaN above +inf, so NaNs planted in a column never
    land in the middle while they are a minority: hand-worked columns of 5 and 4 rows."""
    pnan = np.float32(np.nan)
    nnan = np.frombuffer(np.uint32(0xFFC00000).tobytes(), dtype=np.float32)[0]
    assert not np.signbit(pnan) and np.signbit(nnan)
    cols = [([1.0, pnan, 3.0, nnan, 2.0], 2.0),            # -NaN 1 2 3 +NaN: middle is 2
            ([pnan, pnan, 1.0, 2.0, 3.0], 3.0),            # 1 2 3 +NaN +NaN: middle is 3
            ([nnan, 5.0, nnan, 4.0, 6.0], 4.0),            # -NaN -NaN 4 5 6: middle is 4
            ([nnan, -np.inf, 7.0, np.inf, pnan], 7.0),     # -NaN -inf 7 +inf +NaN
            ([nnan, 1.0, 2.0, pnan], 1.5),                 # even count: mean of the two middle values
            ([pnan, 1.0, 2.0, 4.0], 3.0)]                  # 1 2 4 +NaN: (2 + 4) / 2
    for col, want in cols:
        x = np.zeros((len(col), 8), dtype=np.float32)
        x[:, 3] = np.array(col, dtype=np.float32)
        r = oracle.centered_clip(x, 0.0, init_mode=oracle.INIT_COORD_MEDIAN, max_iters=1)
        assert r["v"][0, 3] == want, (col, r["v"][0, 3])


def test_a_nan_row_with_a_median_start_takes_weight_zero():
    """Reading of the non-finite rule together with the median start: the row that holds a NaN is left
    out of every update, so the result equals the aggregation of the other rows from the same start."""
    rng = np.random.default_rng(81)
    x = rand_rows(rng, 5, 40)
    bad = x.copy()
    bad[2, 7] = np.nan
    v0 = oracle.centered_clip(bad, 0.0, init_mode=oracle.INIT_COORD_MEDIAN, max_iters=1)["v"][0].astype(np.float32)
    a = oracle.centered_clip(bad, 0.5, init_mode=oracle.INIT_COORD_MEDIAN, max_iters=4)
    # restated with numpy on the other four rows; the divisor stays the full peer count n = 5
    keep = np.delete(x, 2, axis=0)
    v = v0.astype(np.float64)
    for _ in range(4):
        r = keep.astype(np.float64) - v
        rho = np.sqrt((r * r).sum(1))
        w = np.where(rho <= 0.5, 1.0, 0.5 / rho)
        v = v + (w[:, None] * r).sum(0) / 5.0
    assert np.allclose(a["v"][0], v, rtol=0, atol=1e-14)
    assert a["status"][0] & oracle.STATUS_NONFINITE_ROW and np.isnan(a["resid_norm"][0, 2])


def test_padding_does_not_change_the_result():
    """Zero columns past part_len are ignored: a padded run equals the unpadded run."""
    rng = np.random.default_rng(9)
    x = rand_rows(rng, 6, 45)
    xp = np.zeros((6, 64), dtype=np.float32)
    xp[:, :45] = x
    xp[:, 45:] = 99.0                                              # garbage in the pad
    a = oracle.centered_clip(x, 1.0, init_mode=oracle.INIT_MEAN, max_iters=6)
    b = oracle.centered_clip(xp, 1.0, part_len=45, init_mode=oracle.INIT_MEAN, max_iters=6)
    assert np.array_equal(a["v"][0], b["v"][0, :45]) and np.all(b["v"][0, 45:] == 0)
    assert np.array_equal(a["resid_norm"], b["resid_norm"])


def test_partitions_are_independent_and_tau_is_per_partition():
    rng = np.random.default_rng(10)
    g = rng.standard_normal((3, 5, 32)).astype(np.float32)
    tau = np.array([0.5, 1.0, np.inf])
    lens = np.array([32, 17, 30])
    r = oracle.centered_clip(g, tau, part_len=lens, init_mode=oracle.INIT_ZERO, max_iters=4)
    for p in range(3):
        one = oracle.centered_clip(g[p][:, :lens[p]].copy(), tau[p], init_mode=oracle.INIT_ZERO,
                                   max_iters=4)
        assert np.array_equal(r["v"][p, :lens[p]], one["v"][0])


def test_eps_mode_counts_updates_and_flags_the_cap():
    x = np.array([[0.0], [10.0]], dtype=np.float32)
    # steps are 1.5 * 2^-l: the first step <= 1e-3 is l = 11
    r = oracle.centered_clip(x, 1.5, init_mode=oracle.INIT_ZERO, stop_mode=oracle.STOP_EPS,
                             max_iters=100, eps=1e-3)
    assert r["iters"][0] == 11 and r["status"][0] == 0
    r = oracle.centered_clip(x, 1.5, init_mode=oracle.INIT_ZERO, stop_mode=oracle.STOP_EPS,
                             max_iters=5, eps=1e-3)
    assert r["iters"][0] == 5 and r["status"][0] & oracle.STATUS_NOT_CONVERGED


def test_non_finite_row_is_left_out():
    rng = np.random.default_rng(11)
    x = rand_rows(rng, 5, 20)
    bad = x.copy()
    bad[2, 3] = np.nan
    r = oracle.centered_clip(bad, np.inf, init_mode=oracle.INIT_ZERO, max_iters=1)
    keep = [0, 1, 3, 4]
    assert np.allclose(r["v"][0], x[keep].astype(np.float64).sum(0) / 5, atol=1e-15)
    assert r["status"][0] & oracle.STATUS_NONFINITE_ROW
    bad[2, 3] = np.inf
    r2 = oracle.centered_clip(bad, 1.0, init_mode=oracle.INIT_ZERO, max_iters=3)
    assert np.all(np.isfinite(r2["v"])) and r2["status"][0] & oracle.STATUS_NONFINITE_ROW


# ----------------------------------------------------------------------------- verification
def _converged_case(seed=12, n=12, L=301):
    rng = np.random.default_rng(seed)
    x = rand_rows(rng, n, L, 0.04)
    x[:4] = rand_rows(rng, 4, L, 20.0)
    r = oracle.centered_clip(x, 1.0, init_mode=oracle.INIT_COORD_MEDIAN, stop_mode=oracle.STOP_EPS,
                             max_iters=5000, eps=1e-13)
    return x, r


def test_projection_definitions_against_numpy():
    """norm, w, <g_i - v, z_k>, s = w * dot / ||z||, sums: recomputed with numpy from the z the
    generator emits (indexing of i, k and of the coordinate)."""
    x, r = _converged_case()
    v32 = r["v"].astype(np.float32)
    K, seed, tau = 3, 99, 1.0
    out = oracle.verify(x, v32, tau, seed, K=K, want_resid_sum=True)
    res = x.astype(np.float64) - v32[0].astype(np.float64)
    rho = np.linalg.norm(res, axis=1)
    w = np.minimum(1.0, tau / rho)
    assert np.allclose(out["norm"][0], rho, rtol=1e-13)
    assert np.allclose(out["weight"][0], w, rtol=1e-13)
    for k in range(K):
        z = oracle.random_vector(seed, 0, k, x.shape[1]).astype(np.float64)
        assert np.allclose(out["dot"][0, :, k], res @ z, rtol=1e-10, atol=1e-12)
        assert np.allclose(out["znorm2"][0, k], z @ z, rtol=1e-13)
        assert np.allclose(out["s"][0, :, k], w * (res @ z) / np.linalg.norm(z), rtol=1e-10, atol=1e-13)
        assert np.allclose(out["s_sum"][0, k], (w * (res @ z) / np.linalg.norm(z)).sum(), atol=1e-12)
    rs = (w[:, None] * res).sum(0)
    assert np.allclose(out["resid_sum"][0], rs, atol=1e-13)
    assert np.allclose(out["resid_sum_norm"][0], np.linalg.norm(rs), atol=1e-13)


def test_projection_sum_vanishes_at_the_fixed_point_and_exposes_a_wrong_v():
    """Verification 2 (App. D.5): sum_i s_i = 0 for any z when v solves the CenteredClip equation;
    a modified v (aggregation attack, App. C) makes the sum visibly non-zero."""
    x, r = _converged_case()
    v64 = r["v"][0]
    v32 = v64.astype(np.float32)
    out = oracle.verify(x, v32, 1.0, seed=5, K=4)
    scale = np.abs(out["s"][0]).sum(0)
    # v is rounded to fp32, so the equation holds to fp32 rounding of v (about 1e-7 relative)
    assert np.all(np.abs(out["s_sum"][0]) < 1e-5 * scale)
    assert out["resid_sum_norm"][0] < 1e-5 * (out["weight"][0] * out["norm"][0]).sum()
    rng = np.random.default_rng(0)
    bad = (v64 + 0.05 * rng.standard_normal(v64.size)).astype(np.float32)
    out_bad = oracle.verify(x, bad, 1.0, seed=5, K=4)
    assert np.all(np.abs(out_bad["s_sum"][0]) > 1e-3 * np.abs(out_bad["s"][0]).sum(0))
    assert out_bad["resid_sum_norm"][0] > 100 * out["resid_sum_norm"][0]


def test_projection_is_linear_in_the_clipped_residual():
    """s_i = <z, Delta_i> with Delta_i = w_i (g_i - v): scaling one unclipped row's residual by c
    scales its s by c; a clipped row's s depends on direction only."""
    rng = np.random.default_rng(13)
    L = 64
    v = np.zeros((1, L), dtype=np.float32)
    d = rng.standard_normal(L).astype(np.float32)
    d /= np.linalg.norm(d)
    x = np.stack([0.25 * d, 0.5 * d, 4 * d, 8 * d]).astype(np.float32)
    out = oracle.verify(x, v, 1.0, seed=1, K=2)
    s = out["s"][0]
    assert np.allclose(s[1], 2 * s[0], rtol=1e-6)
    assert np.allclose(s[2], s[3], rtol=1e-6) and np.allclose(s[2], 4 * s[0], rtol=1e-6)
    assert np.allclose(out["weight"][0], [1, 1, 0.25, 0.125], rtol=1e-6)


def test_reported_norms_drive_the_weights():
    x, r = _converged_case(n=6, L=50)
    v32 = r["v"].astype(np.float32)
    fake = np.full((1, 6), 4.0)
    out = oracle.verify(x, v32, 1.0, seed=1, K=1, norm_in=fake)
    assert np.allclose(out["weight"][0], 0.25) and np.allclose(out["norm"][0], 4.0)


def test_partition_index_keys_z():
    rng = np.random.default_rng(14)
    g = rng.standard_normal((3, 4, 32)).astype(np.float32)
    v = np.zeros((3, 32), dtype=np.float32)
    lens = np.array([32, 30, 7])
    full = oracle.verify(g, v, 1.0, seed=8, K=2, part_len=lens)
    sub = oracle.verify(g[1:], v[1:], 1.0, seed=8, K=2, part_len=lens[1:], first_partition=1)
    for key in ("dot", "s", "znorm2", "s_sum", "norm"):
        assert np.array_equal(full[key][1:], sub[key])
    z = oracle.random_vector(8, 2, 1, 7).astype(np.float64)
    assert np.allclose(full["dot"][2, :, 1], g[2][:, :7].astype(np.float64) @ z, rtol=1e-12)


def test_empty_partition_projects_to_zero():
    """No coordinates: the inner product <z, Delta> is the empty sum."""
    g = np.ones((2, 3, 8), dtype=np.float32)
    v = np.zeros((2, 8), dtype=np.float32)
    out = oracle.verify(g, v, 1.0, seed=1, K=2, part_len=np.array([0, 8]))
    assert np.all(out["s"][0] == 0) and np.all(out["s_sum"][0] == 0) and np.all(out["znorm2"][0] == 0)
    assert np.all(np.isfinite(out["s"]))


# ----------------------------------------------------------------------------- Verifications 1-3
def test_check_predicates_follow_alg6():
    """Alg. 6: norm_ji != ||.|| (V1), s_j^i != <z, Delta> and sum_i s_i != 0 (V2),
    check_ij = [norm > Delta_max] with CheckAveraging when more than n/2 peers vote (V3)."""
    norm = np.array([[1.0, 2.0, 5.0, 0.5, 7.0]])
    s = np.array([[[0.25], [-0.75], [0.5], [-0.125], [0.125]]])        # sums to exactly 0
    out = oracle.checks(norm, s, [1.5])
    assert out["check"].tolist() == [[0, 1, 1, 0, 1]] and out["votes"][0] == 3
    assert out["check_averaging"][0] == 1                              # 3 > 5/2
    assert out["sum_violation"][0, 0] == 0 and not out["norm_mismatch"].any() and not out["s_mismatch"].any()
    out = oracle.checks(norm, s, [2.0])                                # strict ">": 2.0 is not far
    assert out["check"].tolist() == [[0, 0, 1, 0, 1]] and out["check_averaging"][0] == 0
    out = oracle.checks(norm[:, :4], s[:, :4], [0.75])                 # n = 4: 2 votes is not > n/2
    assert out["votes"][0] == 3 and out["check_averaging"][0] == 1
    out = oracle.checks(norm[:, :4], s[:, :4], [1.5])
    assert out["votes"][0] == 2 and out["check_averaging"][0] == 0
    # a peer misreports its norm and its inner product; the broadcast sum no longer vanishes
    nr = norm.copy(); nr[0, 3] = 0.5000001
    sr = s.copy(); sr[0, 1, 0] = -0.7
    out = oracle.checks(norm, s, [1.5], norm_reported=nr, s_reported=sr)
    assert out["norm_mismatch"].tolist() == [[0, 0, 0, 1, 0]]
    assert out["s_mismatch"][0, :, 0].tolist() == [0, 1, 0, 0, 0] and out["sum_violation"][0, 0] == 1
    # tolerances: the same discrepancies pass when allowed for
    out = oracle.checks(norm, s, [1.5], norm_reported=nr, s_reported=sr, rel_tol=0.1, sum_tol=0.1)
    assert not out["norm_mismatch"].any() and not out["s_mismatch"].any() and not out["sum_violation"].any()
    # NaN reports always differ; Delta_max = inf never fires
    nr[0, 0] = np.nan
    out = oracle.checks(norm, s, [np.inf], norm_reported=nr, rel_tol=1.0)
    assert out["norm_mismatch"][0, 0] == 1 and out["votes"][0] == 0


def test_checks_flag_an_aggregation_attack_end_to_end():
    """Aggregation attack (App. C): the aggregator returns a shifted v.  Honest peers' inner products
    then do not sum to zero (V2), and if the shift is large most peers see norm > Delta_max (V3)."""
    x, r = _converged_case()
    tau = 1.0
    good = oracle.verify(x, r["v"].astype(np.float32), tau, seed=3, K=2)
    dmax = float(np.sort(good["norm"][0])[x.shape[0] // 2 - 1] * 1.5)   # most honest peers are within it
    ok = oracle.checks(good["norm"], good["s"], [dmax], sum_tol=1e-5)
    assert not ok["sum_violation"].any() and ok["check_averaging"][0] == 0
    bad_v = (r["v"] + 3.0).astype(np.float32)
    bad = oracle.verify(x, bad_v, tau, seed=3, K=2)
    flagged = oracle.checks(bad["norm"], bad["s"], [dmax], sum_tol=1e-5)
    assert flagged["sum_violation"].all() and flagged["check_averaging"][0] == 1


# ----------------------------------------------------------------------------- baseline aggregators
def test_geometric_median_closed_forms():
    """Weiszfeld's iteration: the Fermat point of an equilateral triangle is its centroid; the
    geometric median of collinear points (odd count) is the middle point; one point is itself."""
    tri = np.array([[0.0, 0.0], [4.0, 0.0], [2.0, 2.0 * math.sqrt(3.0)]], dtype=np.float32)
    r = oracle.centered_clip(tri, 1e-9, init_mode=oracle.INIT_ZERO, stop_mode=oracle.STOP_EPS,
                             max_iters=1000, eps=1e-13, rule=oracle.RULE_GEOMETRIC_MEDIAN)
    assert np.allclose(r["v"][0], tri.astype(np.float64).mean(0), atol=1e-9) and r["status"][0] == 0
    line = np.array([[-3.0, -6.0], [0.5, 1.0], [1.0, 2.0], [7.0, 14.0], [2.0, 4.0]], dtype=np.float32)
    r = oracle.centered_clip(line, 1e-12, init_mode=oracle.INIT_MEAN, stop_mode=oracle.STOP_EPS,
                             max_iters=20000, eps=1e-14, rule=oracle.RULE_GEOMETRIC_MEDIAN)
    assert np.allclose(r["v"][0], [1.0, 2.0], atol=1e-6)
    one = np.array([[3.0, -1.0, 2.0]], dtype=np.float32)
    r = oracle.centered_clip(one, 1e-6, init_mode=oracle.INIT_ZERO, max_iters=1, rule=oracle.RULE_GEOMETRIC_MEDIAN)
    assert np.allclose(r["v"][0], one[0], atol=1e-15)


def test_geometric_median_optimality_and_centered_clip_limit():
    """At the geometric median the unit vectors to the points cancel; that is also the fixed-point
    equation of CenteredClip when tau is below every distance (App. D.2: tau -> 0)."""
    rng = np.random.default_rng(21)
    x = rand_rows(rng, 9, 40, 2.0)
    r = oracle.centered_clip(x, 1e-9, init_mode=oracle.INIT_COORD_MEDIAN, stop_mode=oracle.STOP_EPS,
                             max_iters=5000, eps=1e-13, rule=oracle.RULE_GEOMETRIC_MEDIAN)
    v = r["v"][0]
    d = x.astype(np.float64) - v
    unit = d / np.linalg.norm(d, axis=1, keepdims=True)
    assert np.linalg.norm(unit.sum(0)) < 1e-9
    tau = 1e-3
    lhs, rho, w = clipped_residual_sum(x, v, tau)
    assert rho.min() > tau and np.linalg.norm(lhs) < 1e-11           # v solves the CenteredClip equation
    # one Weiszfeld step from v0, against its textbook form sum x_i/rho_i / sum 1/rho_i
    v0 = rng.standard_normal(40).astype(np.float32)
    r1 = oracle.centered_clip(x, 1e-9, init_mode=oracle.INIT_CALLER, v0=v0[None], max_iters=1,
                              rule=oracle.RULE_GEOMETRIC_MEDIAN)
    rho0 = np.linalg.norm(x.astype(np.float64) - v0, axis=1)
    assert np.allclose(r1["v"][0], (x.astype(np.float64) / rho0[:, None]).sum(0) / (1 / rho0).sum(), atol=1e-13)


def test_mean_and_coordinate_median_rules():
    rng = np.random.default_rng(22)
    g = rng.standard_normal((2, 6, 33)).astype(np.float32)
    lens = np.array([33, 20])
    for rule, fn in ((oracle.RULE_MEAN, np.mean), (oracle.RULE_COORD_MEDIAN, np.median)):
        r = oracle.centered_clip(g, 1.0, part_len=lens, rule=rule, max_iters=7)
        for p in range(2):
            ref = fn(g[p][:, :lens[p]].astype(np.float64), axis=0)
            assert np.allclose(r["v"][p, :lens[p]], ref, atol=1e-15) and r["iters"][p] == 0
            assert np.allclose(r["resid_norm"][p], np.linalg.norm(g[p][:, :lens[p]] - ref, axis=1), rtol=1e-12)


# ----------------------------------------------------------------------------- Clipped-SGD pre-clip
def test_preclip_closed_forms():
    """g~ = min{1, lambda/||g||} g (Alg. 9): short rows are untouched, long rows land on the sphere of
    radius lambda with their direction kept; lambda = inf is the identity."""
    rng = np.random.default_rng(30)
    g = rng.standard_normal((2, 4, 40)).astype(np.float32)
    g[0, 1] *= 100; g[1, 3] *= 1e-3
    lens = np.array([40, 25])
    out = oracle.preclip(g, [3.0, 3.0], part_len=lens)
    for p in range(2):
        for i in range(4):
            x = g[p, i, :lens[p]].astype(np.float64)
            nrm = np.linalg.norm(x)
            assert abs(out["row_norm"][p, i] - nrm) < 1e-12
            y = out["g"][p, i, :lens[p]]
            if nrm <= 3.0:
                assert out["factor"][p, i] == 1.0 and np.array_equal(y, x)
            else:
                assert abs(np.linalg.norm(y) - 3.0) < 1e-12 and np.allclose(y / 3.0, x / nrm, atol=1e-15)
            assert np.all(out["g"][p, i, lens[p]:] == 0)
    ident = oracle.preclip(g, np.inf, part_len=lens)
    assert np.array_equal(ident["g"][0], g[0].astype(np.float64)) and np.all(ident["factor"] == 1.0)
    bad = g.copy(); bad[0, 2, 5] = np.nan
    out = oracle.preclip(bad, 3.0, part_len=lens)
    assert out["factor"][0, 2] == 0.0 and np.all(out["g"][0, 2] == 0)


# ----------------------------------------------------------------------------- commitments
def test_sha256_against_published_answers_and_hashlib():
    """FIPS 180-4 examples ("abc", the empty message, the 448-bit message) and hashlib on messages whose
    lengths straddle every padding case."""
    import hashlib
    assert oracle.sha256(b"abc").hex() == "ba7816bf8f01cfea414140de5dae2223b00361a396177a9cb410ff61f20015ad"
    assert oracle.sha256(b"").hex() == "e3b0c44298fc1c149afbf4c8996fb92427ae41e4649b934ca495991b7852b855"
    assert oracle.sha256(b"abcdbcdecdefdefgefghfghighijhijkijkljklmklmnlmnomnopnopq").hex() == \
        "248d6a61d20638b8e5c026930c3e6039a33ce45964ff2167f6ecedd419db06c1"
    rng = np.random.default_rng(40)
    for n in (1, 3, 55, 56, 57, 63, 64, 65, 119, 120, 128, 4095, 4096, 4097, 100_000):
        m = rng.integers(0, 256, n, dtype=np.uint8).tobytes()
        assert oracle.sha256(m) == hashlib.sha256(m).digest(), n


def test_commitment_is_the_stated_tree_of_sha256():
    import hashlib
    rng = np.random.default_rng(41)
    x = rng.standard_normal((2, 3, 2600)).astype(np.float32)
    lens = np.array([2600, 1023])
    out = oracle.commitment(x, lens)
    for p in range(2):
        for i in range(3):
            raw = x[p, i, :lens[p]].tobytes()
            cat = b"".join(hashlib.sha256(raw[o:o + 4096]).digest() for o in range(0, len(raw), 4096))
            assert out[p, i].tobytes() == hashlib.sha256(cat + len(raw).to_bytes(8, "little")).digest()
    empty = oracle.commitment(x[:1, :1], np.array([0]))
    assert empty[0, 0].tobytes() == hashlib.sha256((0).to_bytes(8, "little")).digest()
    # a one-bit change anywhere, or padding content, must / must not change the commitment
    y = x.copy(); y[1, 2, 1022] = np.nextafter(y[1, 2, 1022], np.float32(10))
    z = x.copy(); z[1, 2, 1023:] = 7.0
    assert not np.array_equal(oracle.commitment(y, lens)[1, 2], out[1, 2])
    assert np.array_equal(oracle.commitment(z, lens), out)


# ----------------------------------------------------------------------------- tau_l schedule, clipped rows
def test_constant_schedule_and_unit_factors_change_nothing():
    """A schedule that repeats tau and factors of 1 must reproduce the plain call bit for bit."""
    rng = np.random.default_rng(31)
    x = np.stack([rand_rows(rng, 7, 50), rand_rows(rng, 7, 50, 4.0)])
    x[0, 1, 3] = np.inf
    tau = np.array([0.7, 2.0])
    for init in (oracle.INIT_ZERO, oracle.INIT_MEAN, oracle.INIT_COORD_MEDIAN):
        a = oracle.centered_clip(x, tau, init_mode=init, max_iters=6)
        b = oracle.centered_clip(x, tau, init_mode=init, max_iters=6, tau_schedule=np.repeat(tau[:, None], 6, 1),
                                 row_scale=np.ones((2, 7)))
        for k in ("v", "resid_norm", "last_step_norm", "iters", "status"):
            assert np.array_equal(a[k], b[k], equal_nan=True), k
    v32 = a["v"].astype(np.float32)
    p = oracle.verify(x[1:], v32[1:], 2.0, 5, K=2)
    q = oracle.verify(x[1:], v32[1:], 2.0, 5, K=2, row_scale=np.ones((1, 7)))
    for k in ("norm", "weight", "dot", "s", "s_sum", "resid_sum_norm"):
        assert np.array_equal(p[k], q[k]), k


def test_schedule_walks_a_single_row_by_tau_l():
    """n = 1, row at distance 10: while it is farther than tau_l, update l moves v by exactly tau_l toward it
    (App. D.2 with the schedule tau_l)."""
    x = np.zeros((1, 4), dtype=np.float32)
    x[0, 2] = 10.0
    sched = np.array([1.0, 2.5, 0.25, 3.0])
    for iters in range(1, 5):
        r = oracle.centered_clip(x, 99.0, init_mode=oracle.INIT_ZERO, max_iters=iters, tau_schedule=sched[:iters])
        assert abs(r["v"][0, 2] - sched[:iters].sum()) < 1e-13
        assert abs(r["last_step_norm"][0] - sched[iters - 1]) < 1e-13
    # and a radius that covers the rest lands on the row
    r = oracle.centered_clip(x, 0.0, init_mode=oracle.INIT_ZERO, max_iters=3, tau_schedule=[1.0, 2.0, 50.0])
    assert r["v"][0, 2] == 10.0


def test_two_value_schedule_by_hand():
    """Three collinear points and two updates with different radii, worked out by hand:
    x = -1, 0, 5 on a line, v0 = 0.  Update 0 with tau = 2: residuals -1, 0, 5 -> weights 1, 1, 2/5 -> step
    (-1 + 0 + 2)/3 = 1/3.  Update 1 with tau = 1/2: residuals -4/3, -1/3, 14/3 -> clipped to -1/2, -1/3, 1/2
    -> step (-1/3)/3 = -1/9.  v = 1/3 - 1/9 = 2/9."""
    x = np.zeros((3, 2), dtype=np.float32)
    x[:, 0] = [-1.0, 0.0, 5.0]
    r = oracle.centered_clip(x, 7.0, init_mode=oracle.INIT_ZERO, max_iters=2, tau_schedule=[2.0, 0.5])
    assert abs(r["v"][0, 0] - 2.0 / 9.0) < 1e-15 and r["v"][0, 1] == 0.0


def test_row_factors_equal_rescaled_rows():
    """Factors that are powers of two rescale fp32 rows exactly, so aggregating (f_i, g_i) must equal
    aggregating the rows f_i g_i written out, bit for bit; a factor of 0 reads the row as zeros even if it
    holds an inf."""
    rng = np.random.default_rng(32)
    x = rand_rows(rng, 6, 41, 3.0)
    f = np.array([1.0, 0.5, 0.25, 2.0, 0.0, 1.0])
    y = (x.astype(np.float64) * f[:, None]).astype(np.float32)
    x[4, 7] = np.inf                                               # dropped by its factor of 0
    for init in (oracle.INIT_MEAN, oracle.INIT_COORD_MEDIAN):
        a = oracle.centered_clip(x, 0.8, init_mode=init, max_iters=5, row_scale=f)
        b = oracle.centered_clip(y, 0.8, init_mode=init, max_iters=5)
        for k in ("v", "resid_norm", "last_step_norm", "status"):
            assert np.array_equal(a[k], b[k]), k
    v32 = a["v"].astype(np.float32)
    p = oracle.verify(x, v32, 0.8, 11, K=3, row_scale=f, want_resid_sum=True)
    q = oracle.verify(y, v32, 0.8, 11, K=3, want_resid_sum=True)
    for k in ("norm", "weight", "dot", "s", "s_sum", "resid_sum", "resid_sum_norm"):
        assert np.array_equal(p[k], q[k]), k


def test_clipped_sgd_aggregation_is_clip_then_aggregate():
    """Alg. 9: peers clip their parts to lambda, then ButterflyClip aggregates them.  One update from v = 0,
    restated with numpy on the clipped rows, against the oracle fed with the clip factors."""
    rng = np.random.default_rng(33)
    x = rand_rows(rng, 8, 60, 0.2)
    x[::3] *= 40.0
    lam, tau = 1.5, 0.9
    pc = oracle.preclip(x, lam)
    assert (pc["factor"] < 1).any() and (pc["factor"] == 1).any()
    gt = pc["g"][0]                                                # clipped rows, float64
    assert np.all(np.linalg.norm(gt, axis=1) <= lam * (1 + 1e-12))
    rho = np.linalg.norm(gt, axis=1)
    w = np.where(rho <= tau, 1.0, tau / rho)
    v1 = (w[:, None] * gt).sum(0) / 8
    r = oracle.centered_clip(x, tau, init_mode=oracle.INIT_ZERO, max_iters=1, row_scale=pc["factor"])
    assert np.allclose(r["v"][0], v1, rtol=0, atol=1e-15)
    assert np.allclose(r["resid_norm"][0], np.linalg.norm(gt - v1, axis=1), rtol=1e-13)
