"""The partition-sharded ButterflyClip (Alg. 2) between CPU processes: gloo ranks, no GPU.

What is checked here is the exchange logic of paper_2106_11257_b200/butterfly.py: which part goes to which
rank, the order of the slabs a rank receives, the z key of a shard (partition_base), the order in which the
aggregated parts and the scalars come back, the commitments.  The three device steps are replaced by the
float64 oracle (the product's steps need a GPU; their parity is tested in test_gpu_parity.py), and the result
of every rank must equal the oracle run on the whole [P][n][stride] tensor by one process.
"""
import os
import pickle
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SEED, K, TAU, ITERS = 77, 2, 0.7, 4


def peer_gradient(rank, d):
    rng = np.random.default_rng(1000 + rank)
    g = rng.standard_normal(d).astype(np.float32)
    if rank == 1:
        g *= 6.0                                       # one peer far from the others: its rows are clipped
    return g


class OracleSteps:
    """Stand-ins for the device steps, with the outputs (keys, shapes, dtypes) of the CUDA binding."""

    def __init__(self, oracle):
        self.o = oracle

    def split(self, grad, part_offset, part_len, row_stride):
        x = grad.numpy()
        out = np.zeros((len(part_offset), row_stride), dtype=np.float32)
        for q, (o, l) in enumerate(zip(part_offset, part_len)):
            out[q, :l] = x[o:o + l]
        return torch.from_numpy(out)

    def aggregate(self, g, tau, seed, K, part_len, partition_base, **kw):
        o = self.o
        c = o.centered_clip(g.numpy(), tau, part_len, init_mode=o.INIT_COORD_MEDIAN, max_iters=kw["max_iters"])
        v32 = c["v"].astype(np.float32)
        r = o.verify(g.numpy(), v32, tau, seed, K=K, part_len=part_len, first_partition=partition_base)
        clip = dict(v=torch.from_numpy(v32), iters=torch.from_numpy(c["iters"].astype(np.int32)),
                    last_step_norm=torch.from_numpy(c["last_step_norm"]), resid_norm=torch.from_numpy(c["resid_norm"]),
                    status=torch.from_numpy(c["status"].astype(np.int32)))
        ver = {k: torch.from_numpy(r[k].astype(np.int32) if k == "status" else r[k]) for k in
               ("norm", "weight", "dot", "s", "s_sum", "znorm2", "resid_sum_norm", "status")}
        return clip, ver

    def merge(self, v, d, part_offset, part_len):
        out = np.zeros(d, dtype=np.float32)
        for p, (o, l) in enumerate(zip(part_offset, part_len)):
            out[o:o + l] = v[p, :l].numpy()
        return torch.from_numpy(out)

    def commit(self, x, part_len):
        return torch.from_numpy(self.o.commitment(x.numpy(), part_len))


def _worker(rank, world, port, out_dir, d, ppr, tamper):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import oracle
    from paper_2106_11257_b200 import butterfly
    steps = OracleSteps(oracle)
    if tamper and rank == 0:
        # rank 0 announces the hashes of its true parts, then alters the last part before it travels
        honest_commit = steps.commit
        calls = []

        def commit(x, part_len):
            digests = honest_commit(x, part_len)
            if not calls:
                x.reshape(-1, x.shape[-1])[-1, 0] += 1.0   # x is the send buffer; its last slab is part P - 1
            calls.append(1)
            return digests
        steps.commit = commit
    res = butterfly.butterfly_clip(torch.from_numpy(peer_gradient(rank, d)), TAU, SEED, K=K, parts_per_rank=ppr,
                                   steps=steps, commit=True, max_iters=ITERS)
    keep = {"aggregate": res["aggregate"].numpy(), "v_parts": res["v_parts"].numpy(), "owned": res["owned"],
            "clip": {k: v.numpy() for k, v in res["clip"].items()},
            "verify": {k: v.numpy() for k, v in res["verify"].items()},
            "commit": {k: v.numpy() for k, v in res["commit"].items()}}
    with open(os.path.join(out_dir, "rank%d.pkl" % rank), "wb") as f:
        pickle.dump(keep, f)
    dist.barrier()
    dist.destroy_process_group()


def whole_tensor_reference(world, d, ppr):
    """The same round by one process: every peer's parts stacked as [P][n][stride], one oracle call."""
    sys.path.insert(0, ROOT)
    import oracle
    P = world * ppr
    off, ln, stride = oracle.partition_layout(d, P, oracle.SPLIT_CEIL_PAD)
    g = np.zeros((P, world, stride), dtype=np.float32)
    for i in range(world):
        x = peer_gradient(i, d)
        for p in range(P):
            g[p, i, :ln[p]] = x[off[p]:off[p] + ln[p]]
    c = oracle.centered_clip(g, TAU, ln, init_mode=oracle.INIT_COORD_MEDIAN, max_iters=ITERS)
    v32 = c["v"].astype(np.float32)
    r = oracle.verify(g, v32, TAU, SEED, K=K, part_len=ln)
    agg = np.concatenate([v32[p, :ln[p]] for p in range(P)])
    return dict(g=g, ln=ln, v=v32, clip=c, verify=r, aggregate=agg, oracle=oracle)


@pytest.mark.parametrize("world,d,ppr", [(2, 1000, 1), (2, 1003, 3), (3, 517, 2)])
def test_sharded_round_equals_the_whole_tensor(tmp_path, world, d, ppr):
    port = 29500 + (os.getpid() * 7 + world * 13 + ppr) % 2000
    mp.spawn(_worker, args=(world, port, str(tmp_path), d, ppr, False), nprocs=world, join=True)
    ref = whole_tensor_reference(world, d, ppr)
    P = world * ppr
    for rank in range(world):
        res = pickle.load(open(tmp_path / ("rank%d.pkl" % rank), "rb"))
        assert res["owned"] == list(range(rank * ppr, (rank + 1) * ppr))
        # same arithmetic on the same rows: bit for bit
        assert np.array_equal(res["aggregate"], ref["aggregate"])
        assert np.array_equal(res["v_parts"], ref["v"])
        for k in ("norm", "weight", "dot", "s", "s_sum", "znorm2", "resid_sum_norm"):
            assert res["verify"][k].shape == ref["verify"][k].shape, k
            assert np.array_equal(res["verify"][k], ref["verify"][k]), k
        assert np.array_equal(res["clip"]["iters"], ref["clip"]["iters"])
        assert np.array_equal(res["clip"]["resid_norm"], ref["clip"]["resid_norm"])
        assert np.array_equal(res["clip"]["last_step_norm"], ref["clip"]["last_step_norm"])
        # commitments: hash(g_i[j]) indexed [peer][part], hash of every aggregated part, and everything matched
        want = ref["oracle"].commitment(ref["g"], ref["ln"])                 # [P][n][32]
        assert np.array_equal(res["commit"]["parts"], want.transpose(1, 0, 2))
        assert np.array_equal(res["commit"]["aggregates"], ref["oracle"].commitment(ref["v"], ref["ln"])[:, 0, :])
        assert res["commit"]["parts_match"].shape == (ppr, world) and res["commit"]["parts_match"].all()
    # rows are clipped and no two parts have the same scalars, so a shard verified with another part's z, rows
    # or position would not have compared equal above
    assert (ref["verify"]["weight"] < 1.0).any()
    assert len({ref["verify"]["s"][p].tobytes() for p in range(P)}) == P
    assert P == len(ref["ln"])


def test_a_part_that_differs_from_its_commitment_is_flagged(tmp_path):
    world, d, ppr = 2, 640, 2
    port = 29500 + (os.getpid() * 11 + 5) % 2000
    mp.spawn(_worker, args=(world, port, str(tmp_path), d, ppr, True), nprocs=world, join=True)
    res = [pickle.load(open(tmp_path / ("rank%d.pkl" % r), "rb")) for r in range(world)]
    assert res[0]["commit"]["parts_match"].all()                   # rank 0 received honest parts
    m = res[1]["commit"]["parts_match"]                            # rank 1 owns parts 2 and 3
    assert m.shape == (2, 2)
    assert not m[1, 0] and m[0, 0] and m[:, 1].all()               # part 3 from peer 0 is the altered one


def test_send_order_and_ownership():
    sys.path.insert(0, ROOT)
    from paper_2106_11257_b200 import butterfly
    for world, ppr in [(1, 1), (2, 3), (4, 2), (8, 1)]:
        order = butterfly.send_order(world, ppr)
        assert sorted(order.tolist()) == list(range(world * ppr))
        for m in range(ppr):
            for r in range(world):
                assert order[m * world + r] == butterfly.owned_parts(r, world, ppr)[m]
