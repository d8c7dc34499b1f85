"""ButterflyClip (Alg. 2) through the library's kernels and NCCL on one GPU.

One GPU means one rank, so the exchanges are trivial here (their logic is tested between CPU processes in
test_butterfly_gloo.py); what this file covers is the device side of paper_2106_11257_b200/butterfly.py:
Split into a permuted send buffer, the one-call aggregation + verification of a shard keyed by
partition_base, Merge, the commitments, and the NCCL calls on CUDA tensors, all against the float64 oracle.
"""
import os

import numpy as np
import pytest
import torch

import oracle
import paper_2106_11257_b200 as btard
from paper_2106_11257_b200 import butterfly

pytestmark = pytest.mark.gpu
RTOL = 1e-5


def rel_l2(a, b):
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    den = np.linalg.norm(b)
    return np.linalg.norm(a - b) / den if den > 0 else np.linalg.norm(a)


def test_split_with_a_permuted_layout_matches_numpy():
    rng = np.random.default_rng(3)
    n, d, P = 5, 10007, 6
    x = rng.standard_normal((n, d)).astype(np.float32)
    off, ln, stride = btard.partition_layout(d, P, btard.SPLIT_CEIL_PAD)
    order = butterfly.send_order(3, 2)
    g, o2, l2 = btard.split_gradients(torch.from_numpy(x).cuda(), P, layout=(off[order], ln[order], stride))
    g = g.cpu().numpy()
    assert g.shape == (P, n, stride) and np.array_equal(o2, off[order]) and np.array_equal(l2, ln[order])
    for q, p in enumerate(order):
        assert np.array_equal(g[q, :, :ln[p]], x[:, off[p]:off[p] + ln[p]])
        assert np.all(g[q, :, ln[p]:] == 0)


@pytest.fixture
def one_rank_nccl():
    import torch.distributed as dist
    port = 29500 + (os.getpid() * 3 + 17) % 2000
    dist.init_process_group("nccl", init_method="tcp://127.0.0.1:%d" % port, rank=0, world_size=1,
                            device_id=torch.device("cuda:0"))
    yield dist
    dist.destroy_process_group()


@pytest.mark.parametrize("ppr,d,algo", [(1, 70001, btard.ALGO_DIRECT), (3, 100003, btard.ALGO_DIRECT),
                                        (4, 65536, btard.ALGO_GRAM)])
def test_one_rank_round_matches_the_oracle(one_rank_nccl, ppr, d, algo):
    rng = np.random.default_rng(11 + ppr)
    x = rng.standard_normal(d).astype(np.float32)
    tau, seed, K, iters = 30.0, 2024, 2, 3
    res = butterfly.butterfly_clip(torch.from_numpy(x).cuda(), tau, seed, K=K, parts_per_rank=ppr, commit=True,
                                   init_mode=btard.INIT_ZERO, stop_mode=btard.STOP_FIXED_ITERS, max_iters=iters,
                                   algo=algo)
    torch.cuda.synchronize()
    P = ppr
    off, ln, stride = oracle.partition_layout(d, P, oracle.SPLIT_CEIL_PAD)
    assert np.array_equal(res["part_offset"], off) and np.array_equal(res["part_len"], ln) and res["row_stride"] == stride
    g = np.zeros((P, 1, stride), dtype=np.float32)
    for p in range(P):
        g[p, 0, :ln[p]] = x[off[p]:off[p] + ln[p]]
    # one peer, start at 0, radius below the row's norm: every update moves v by tau along the row (App. D.2 update)
    c = oracle.centered_clip(g, tau, ln, init_mode=oracle.INIT_ZERO, max_iters=iters)
    v_gpu = res["v_parts"].cpu().numpy()
    for p in range(P):
        assert rel_l2(v_gpu[p, :ln[p]], c["v"][p, :ln[p]]) <= RTOL
        assert np.all(v_gpu[p, ln[p]:] == 0)
    assert np.array_equal(res["aggregate"].cpu().numpy(), np.concatenate([v_gpu[p, :ln[p]] for p in range(P)]))
    assert np.array_equal(res["clip"]["iters"].cpu().numpy(), c["iters"])
    # verification of the shard at the v the GPU produced, z keyed by the global part index
    r = oracle.verify(g, v_gpu, tau, seed, K=K, part_len=ln)
    for k in ("norm", "weight", "dot", "s", "znorm2"):
        got = res["verify"][k].cpu().numpy()
        assert got.shape == r[k].shape, k
        assert rel_l2(got, r[k]) <= RTOL, k
    # commitments: bit-exact against the oracle's SHA-256 tree, and what arrived is what was announced
    assert np.array_equal(res["commit"]["parts"].cpu().numpy(), oracle.commitment(g, ln).transpose(1, 0, 2))
    assert np.array_equal(res["commit"]["aggregates"].cpu().numpy(), oracle.commitment(v_gpu, ln)[:, 0, :])
    assert res["commit"]["parts_match"].cpu().numpy().all()
