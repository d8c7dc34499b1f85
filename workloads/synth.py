"""Seeded synthetic gradient tensors for the five benchmark configurations.

The paper's experiments aggregate real ResNet-18 / CIFAR-10 and ALBERT-large /
WikiText-103 gradients under attack (Sec. 4.1-4.2, App. I.3).  Neither dataset
nor any trained weight is available offline, so these generators stand in for
them: same number of peers, same vector length and partitioning, the same
Byzantine fractions and attack families (sign flipping, random direction, IPM,
ALIE), with honest rows drawn as a common mean plus Gaussian or Student-t noise.

Every partition is generated from its own seed (a function of the configuration
and the partition index), so a single partition of a tensor that is too large
for host memory can be regenerated alone.  Quantities the attacks define over
the whole vector (the honest norm, a unit direction) use their expected values,
sqrt(d * per-coordinate second moment) and 1/sqrt(d) scaling, so that no pass
over the other partitions is needed; the realised values differ from the exact
normalisation by O(d^-1/2).
"""
from dataclasses import dataclass, field
import math

import numpy as np
import torch

INIT_CALLER, INIT_ZERO, INIT_MEAN, INIT_COORD_MEDIAN = 0, 1, 2, 3
STOP_FIXED, STOP_EPS = 0, 1

CONFIGS = {
    # n peers, d coordinates, P partitions, honest noise, attacks [(kind, rows, param)], ...
    1: dict(n=4, d=1024, P=1, mu_std=1.0, noise=("normal", 0.1), attacks=[("signflip_mu", 1, 10.0)],
            tau=1.0, K=1, zseed=0, stop=STOP_FIXED, max_iters=50, eps=1e-6),
    2: dict(n=16, d=11_173_962, P=16, mu_std=1e-2, noise=("normal", 3e-3),
            attacks=[("random_direction", 7, 100.0)],
            tau=1.0, K=1, zseed=2, stop=STOP_EPS, max_iters=100, eps=1e-6),
    3: dict(n=16, d=11_173_962, P=16, mu_std=1e-2, noise=("normal", 3e-3),
            attacks=[("alie", 7, 1.0)],
            tau=("half_median_honest_residual",), K=8, zseed=3, stop=STOP_EPS, max_iters=100,
            eps=1e-6),
    4: dict(n=64, d=17_683_968, P=64, mu_std=1e-2, noise=("student_t", 1e-3, 4),
            attacks=[("signflip_own", 8, 4.0), ("ipm", 8, 0.5)],
            tau=1.0, K=1, zseed=4, stop=STOP_EPS, max_iters=100, eps=1e-6),
    5: dict(n=64, d=1 << 28, P=64, mu_std=1e-2, noise=("student_t", 1e-3, 3),
            attacks=[("random_direction", 11, 100.0), ("signflip_own", 10, 4.0), ("alie", 10, 1.0)],
            tau=1.0, K=4, zseed=5, stop=STOP_FIXED, max_iters=20, eps=1e-6),
}


@dataclass
class Workload:
    cfg: int
    n: int
    d: int
    P: int
    row_stride: int
    part_len: np.ndarray            # int64 [P]
    tau: np.ndarray                 # float64 [P]
    K: int
    zseed: int
    init_mode: int
    stop_mode: int
    max_iters: int
    eps: float
    byz_rows: dict                  # attack kind -> row indices
    g: torch.Tensor = None          # [P][n][row_stride] fp32 (None when only metadata is wanted)
    partitions: list = field(default_factory=list)   # indices of the partitions held in g


def layout_ceil_pad(d, P, align=32):
    """Every part holds ceil(d/P) coordinates until d runs out; rows are padded to `align`."""
    L = -(-d // P)
    lens = np.array([max(0, min(L, d - j * L)) for j in range(P)], dtype=np.int64)
    stride = -(-max(int(lens.max()), 1) // align) * align
    return lens, stride


def _rows(spec, seed):
    """Seeded choice of which peers are Byzantine, per attack kind."""
    rng = np.random.RandomState(seed)
    nb = sum(a[1] for a in spec["attacks"])
    chosen = rng.permutation(spec["n"])[:nb]
    out, at = {}, 0
    for kind, cnt, _ in spec["attacks"]:
        out[kind] = np.sort(chosen[at:at + cnt])
        at += cnt
    return out


def _noise(spec, shape, gen, device):
    kind = spec["noise"][0]
    sigma = spec["noise"][1]
    z = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
    if kind == "normal":
        return z * sigma
    nu = spec["noise"][2]
    chi2 = torch.zeros(shape, device=device, dtype=torch.float32)
    for _ in range(nu):
        chi2 += torch.randn(shape, generator=gen, device=device, dtype=torch.float32) ** 2
    t = z / torch.sqrt(chi2 / nu)
    return t * (sigma / math.sqrt(nu / (nu - 2.0)))


def make_partition(cfg, p, device="cpu", d=None, spec=None):
    """Rows of partition p: returns (g_p [n][row_stride] fp32 on `device`, tau_p, part_len_p)."""
    spec = dict(CONFIGS[cfg]) if spec is None else spec
    if d is not None:
        spec["d"] = d
    n, dd, P = spec["n"], spec["d"], spec["P"]
    lens, stride = layout_ceil_pad(dd, P)
    L = int(lens[p])
    byz = _rows(spec, 1000 + cfg)
    gen = torch.Generator(device=device)
    gen.manual_seed((1000 + cfg) * 1_000_003 + p)
    g = torch.zeros((n, stride), dtype=torch.float32, device=device)
    mu = torch.randn(L, generator=gen, device=device, dtype=torch.float32) * spec["mu_std"]
    for i in range(n):                      # every peer first gets its own honest row
        g[i, :L] = mu + _noise(spec, (L,), gen, device)
    is_byz = np.zeros(n, dtype=bool)
    for rows in byz.values():
        is_byz[rows] = True
    honest = torch.from_numpy(np.nonzero(~is_byz)[0]).to(device)
    hon = g.index_select(0, honest)[:, :L]
    hmean = hon.mean(dim=0)
    sigma = spec["noise"][1]
    honest_norm = math.sqrt(dd * (spec["mu_std"] ** 2 + sigma ** 2))
    for kind, cnt, param in spec["attacks"]:
        rows = byz[kind]
        if kind == "signflip_mu":           # the opposite of the common mean, amplified
            g[rows, :L] = -param * mu
        elif kind == "signflip_own":        # the opposite of the peer's own gradient, amplified
            g[rows, :L] = -param * g[rows, :L]
        elif kind == "random_direction":    # all attackers share one direction
            direction = torch.randn(L, generator=gen, device=device, dtype=torch.float32)
            g[rows, :L] = direction * (param * honest_norm / math.sqrt(dd))
        elif kind == "ipm":                 # inner-product manipulation
            g[rows, :L] = -param * hmean
        elif kind == "alie":                # "a little is enough": shift inside the honest spread
            g[rows, :L] = hmean - param * hon.std(dim=0)
        else:
            raise ValueError(kind)
    tau = spec["tau"]
    if isinstance(tau, tuple):
        res = torch.linalg.vector_norm((hon - hmean).double(), dim=1)
        tau = 0.5 * float(res.median())
    return g, float(tau), L


def make_workload(cfg, device="cpu", d=None, partitions=None, data=True):
    """Assemble configuration `cfg` (optionally with a smaller d, or a subset of partitions)."""
    spec = dict(CONFIGS[cfg])
    if d is not None:
        spec["d"] = d
    n, dd, P = spec["n"], spec["d"], spec["P"]
    lens, stride = layout_ceil_pad(dd, P)
    parts = list(range(P)) if partitions is None else list(partitions)
    tau = np.zeros(len(parts), dtype=np.float64)
    g = torch.zeros((len(parts), n, stride), dtype=torch.float32, device=device) if data else None
    for s, p in enumerate(parts):
        if data:
            gp, tau[s], _ = make_partition(cfg, p, device=device, spec=spec)
            g[s] = gp
            del gp
        elif not isinstance(spec["tau"], tuple):
            tau[s] = spec["tau"]
    return Workload(cfg=cfg, n=n, d=dd, P=len(parts), row_stride=stride,
                    part_len=lens[parts].copy(), tau=tau, K=spec["K"], zseed=spec["zseed"],
                    init_mode=INIT_COORD_MEDIAN, stop_mode=spec["stop"],
                    max_iters=spec["max_iters"], eps=spec["eps"], byz_rows=_rows(spec, 1000 + cfg),
                    g=g, partitions=parts)
