"""ButterflyClip over several GPUs (Alg. 2; verification scalars of Alg. 1 and Alg. 6).

One process per GPU, every rank a peer.  A rank splits its own gradient into P parts (App. D.1), sends
part j to the rank that aggregates it, aggregates and verifies the parts it owns with the library's
kernels, and receives everybody's aggregated parts back:

    Split  ->  all-to-all of the parts  ->  CenteredClip + verification per owned part
           ->  all-gather of the aggregated parts  ->  Merge,   all-gather of the scalars

P = parts_per_rank * world.  Rank r owns the consecutive parts r * parts_per_rank ... (r + 1) *
parts_per_rank - 1, so the gathered parts arrive in Split order and `partition_base` = the first owned part
keys z exactly as one GPU holding every part would.  The send buffer is written by the Split kernel in the
order [local part m][destination r], which makes every exchange a plain equal-split all-to-all between
contiguous buffers: the received rows are the slab tensor [parts_per_rank][n][row_stride] the kernels read,
with no repacking on either side.  Rows land in this GPU's memory first and every kernel reads local memory only.

The collectives go through torch.distributed (NCCL between GPUs).  The arithmetic is the library's: there
is no CPU implementation behind this module, and `ops` exists so that the exchange logic can be exercised
between CPU processes with stand-in steps.
"""
import numpy as np

from . import binding as B


class CudaSteps:
    """The three device steps of one rank, on the library's kernels."""

    def split(self, grad, part_offset, part_len, row_stride):
        g, _, _ = B.split_gradients(grad.reshape(1, -1), len(part_offset), layout=(part_offset, part_len, row_stride))
        return g.reshape(len(part_offset), row_stride)

    def aggregate(self, g, tau, seed, K, part_len, partition_base, **kw):
        return B.centered_clip_verify(g, tau, seed, K=K, part_len=part_len, partition_base=partition_base, **kw)

    def merge(self, v, d, part_offset, part_len):
        return B.merge_partitions(v, d, part_offset, part_len)

    def commit(self, x, part_len):
        return B.hash_partitions(x, part_len)


def owned_parts(rank, world, parts_per_rank):
    """Global indices of the parts rank `rank` aggregates."""
    return list(range(rank * parts_per_rank, (rank + 1) * parts_per_rank))


def send_order(world, parts_per_rank):
    """Part held by slab q of the send buffer [parts_per_rank][world]: slab m * world + r goes to rank r as
    its local part m, i.e. it is global part r * parts_per_rank + m."""
    return np.array([r * parts_per_rank + m for m in range(parts_per_rank) for r in range(world)], dtype=np.int64)


_VERIFY_KEYS = ("norm", "weight", "dot", "s", "s_sum", "znorm2", "resid_sum_norm", "status")
_CLIP_KEYS = ("iters", "last_step_norm", "resid_norm", "status")


def _gather_scalars(torch, dist, group, world, parts_per_rank, tables):
    """All-gather of the per-part scalars (Alg. 1: every peer broadcasts its s and norms): each rank's
    values travel as one float64 buffer (32-bit integers are exact in it) and come back with the part
    index leading, in Split order."""
    names, shapes, flat = [], [], []
    for prefix, d, keys in tables:
        for k in keys:
            t = d[k]
            names.append((prefix, k, t.dtype))
            shapes.append(tuple(t.shape[1:]))
            flat.append(t.reshape(parts_per_rank, -1).to(torch.float64))
    mine = torch.cat(flat, dim=1).contiguous()                      # [parts_per_rank][values per part]
    everyone = torch.empty((world,) + tuple(mine.shape), dtype=torch.float64, device=mine.device)
    dist.all_gather(list(everyone.unbind(0)), mine, group=group)
    everyone = everyone.reshape(world * parts_per_rank, -1)
    out, at = {}, 0
    for (prefix, k, dtype), shape in zip(names, shapes):
        width = int(np.prod(shape)) if shape else 1
        out.setdefault(prefix, {})[k] = everyone[:, at:at + width].reshape((-1,) + shape).to(dtype)
        at += width
    return out


def butterfly_clip(grad, tau, seed, K=1, parts_per_rank=1, group=None, steps=None, commit=False, **aggregation):
    """One ButterflyClip round (Alg. 2) with the verification scalars of Alg. 6 for every part.

    grad: this rank's gradient, float32 [d], on this rank's GPU.  tau: one radius or one per part [P].
    seed: the round's shared 64-bit seed (the paper draws it with its multi-party generator; here an input).
    aggregation: passed to centered_clip_verify (init_mode, stop_mode, max_iters, eps, algo, ...).
    commit: also exchange the SHA-256 commitments hash(g_i[j]) and hash(g^_j) and compare every received
    part with its sender's commitment.

    Returns a dict: `aggregate` [d] (Merge of the aggregated parts), `v_parts` [P][row_stride],
    `part_offset`, `part_len`, `row_stride`, `owned` (this rank's parts), `clip` and `verify` (the
    per-part outputs of the aggregation and of the verification, gathered from their owners, part index
    leading) and, with commit, `commit` = {parts [n][P][32], aggregates [P][32], parts_match [owned][n] bool}.
    Every rank must call it with the same d, tau, seed, K, parts_per_rank and aggregation settings."""
    import torch
    import torch.distributed as dist
    steps = steps if steps is not None else CudaSteps()
    world, rank = dist.get_world_size(group), dist.get_rank(group)
    assert grad.dim() == 1 and grad.dtype == torch.float32 and grad.is_contiguous()
    assert parts_per_rank >= 1
    d, n, P = grad.numel(), world, world * parts_per_rank
    off, ln, stride = B.partition_layout(d, P, B.SPLIT_CEIL_PAD)
    order = send_order(world, parts_per_rank)
    mine = owned_parts(rank, world, parts_per_rank)
    tau_all = np.ascontiguousarray(np.broadcast_to(np.asarray(tau, dtype=np.float64), (P,)))

    # Split, in send order; the exchange of the parts below moves local part m of every rank in one all-to-all
    send = steps.split(grad, off[order], ln[order], stride).reshape(parts_per_rank, world, stride)
    res = {"part_offset": off, "part_len": ln, "row_stride": stride, "owned": mine}
    if commit:
        # hash(g_i[j]) for every j, announced by every peer before the parts travel
        inv = np.argsort(order)
        own = steps.commit(send.reshape(P, 1, stride), ln[order]).reshape(P, 32)
        own = own[torch.as_tensor(inv, device=own.device)].contiguous()              # Split order
        announced = torch.empty((n, P, 32), dtype=torch.uint8, device=own.device)
        dist.all_gather(list(announced.unbind(0)), own, group=group)
    g = torch.empty((parts_per_rank, n, stride), dtype=torch.float32, device=grad.device)
    for m in range(parts_per_rank):
        dist.all_to_all_single(g[m], send[m], group=group)
    if commit:
        # what arrived is hashed again and compared with its sender's announcement
        arrived = steps.commit(g, ln[mine]).reshape(parts_per_rank, n, 32)
        expected = announced[:, mine[0]:mine[0] + parts_per_rank, :].permute(1, 0, 2)
        res["commit"] = {"parts": announced, "parts_match": (arrived == expected).all(dim=2)}

    clip, verify = steps.aggregate(g, tau_all[mine], seed, K, ln[mine], mine[0], **aggregation)

    # the aggregated parts go back to everybody (owners are consecutive, so they arrive in Split order)
    v_mine = clip["v"].reshape(parts_per_rank, stride)
    v_all = torch.empty((world, parts_per_rank, stride), dtype=torch.float32, device=grad.device)
    dist.all_gather(list(v_all.unbind(0)), v_mine, group=group)
    v_all = v_all.reshape(P, stride)
    res["v_parts"] = v_all
    res["aggregate"] = steps.merge(v_all, d, off, ln)
    if commit:
        agg = steps.commit(v_mine.reshape(parts_per_rank, 1, stride), ln[mine]).reshape(parts_per_rank, 32)
        agg_all = torch.empty((world, parts_per_rank, 32), dtype=torch.uint8, device=agg.device)
        dist.all_gather(list(agg_all.unbind(0)), agg.contiguous(), group=group)
        res["commit"]["aggregates"] = agg_all.reshape(P, 32)
    res.update(_gather_scalars(torch, dist, group, world, parts_per_rank,
                               [("clip", clip, _CLIP_KEYS), ("verify", verify, _VERIFY_KEYS)]))
    return res
