"""Multi-GPU plumbing: one process per GPU over torch.distributed.

The attention path shards with no collective inside it (by request, by q-head group, or by KV range), so the
only exchanges are outside the kernels: a barrier and a max-reduction for timing, and -- for KV-range
(context-parallel) sharding -- an all-gather of the fp32 partials (o, lse) that `vpp_lse_merge` combines.
Everything here works on the gloo backend too, which is how it is tested without GPUs.
"""
import os

import numpy as np
import torch
import torch.distributed as dist


def env_rank_world():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("LOCAL_RANK", "0"))


def init(backend, device=None):
    """Initialise the default process group from the torchrun environment (no-op for world size 1)."""
    rank, world, _ = env_rank_world()
    if world > 1 and not dist.is_initialized():
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=device)
        else:
            dist.init_process_group(backend)
    return rank, world


def barrier(device=None):
    if device is not None and device.type == "cuda":
        torch.cuda.synchronize(device)
    if dist.is_initialized():
        dist.barrier()
        if device is not None and device.type == "cuda":
            torch.cuda.synchronize(device)


def max_over_ranks(values, device=None):
    """Element-wise maximum of a list of floats over all ranks (identity for world size 1)."""
    if not dist.is_initialized():
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def whole_job_rate(units_per_rank, local_seconds, device=None):
    """Aggregate rate = units all ranks processed / slowest rank's time (weak scaling)."""
    world = dist.get_world_size() if dist.is_initialized() else 1
    (t_max,) = max_over_ranks([local_seconds], device)
    return world * units_per_rank / t_max


def partition_requests(prefix_lens, chunk_lens, world):
    """Longest-first greedy split of a varlen batch over `world` ranks by attention cost
    C*P + C(C+1)/2 (visible query-key pairs).  Returns a list of request-index lists, one per rank;
    every request appears exactly once, order inside a rank is ascending."""
    p = np.asarray(prefix_lens, dtype=np.int64)
    c = np.asarray(chunk_lens, dtype=np.int64)
    cost = c * p + c * (c + 1) // 2
    order = sorted(range(len(cost)), key=lambda i: (-int(cost[i]), i))
    loads = [0] * world
    parts = [[] for _ in range(world)]
    for i in order:
        r = min(range(world), key=lambda k: (loads[k], k))
        parts[r].append(i)
        loads[r] += int(cost[i])
    return [sorted(x) for x in parts]


def kv_ranges(seq_len, world, prefix_len=None):
    """Contiguous, 128-aligned KV ranges [lo, hi) of a context-parallel split of one sequence.

    With prefix_len (the tokens cached before the current chunk) no range starts beyond the prefix, which is what
    vpp_chunk_attn_partial_fwd needs (every query row must see a key of every range): the chunk's own keys stay with the
    last range.  Ranges may be empty (lo == hi) when there are more ranks than 128-key tiles; an empty range is skipped
    by its rank (its partial is lse = -inf)."""
    tiles = (seq_len + 127) // 128
    cuts = [min(seq_len, ((tiles * r) // world) * 128) for r in range(world)] + [seq_len]
    if prefix_len is not None:
        cap = (int(prefix_len) // 128) * 128
        cuts = [min(c, cap) for c in cuts[:-1]] + [seq_len]
    return [(cuts[r], cuts[r + 1]) for r in range(world)]


def all_gather_partials(o_part, lse_part):
    """All-gather per-rank partial outputs [T, Hq, Dv] and log-sum-exp [T, Hq] into [world, ...] tensors
    (the inputs of vpp_lse_merge)."""
    world = dist.get_world_size()
    o_all = [torch.empty_like(o_part) for _ in range(world)]
    l_all = [torch.empty_like(lse_part) for _ in range(world)]
    dist.all_gather(o_all, o_part.contiguous())
    dist.all_gather(l_all, lse_part.contiguous())
    return torch.stack(o_all), torch.stack(l_all)
