"""The N > 1 path on CPU: two gloo ranks exercise the plumbing bench.py and a multi-GPU caller use --
request sharding with gathered outputs, KV-range (context-parallel) sharding with all-gathered partials
merged by the log-sum-exp rule, and max-over-ranks timing.  The per-rank attention is the CPU oracle."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2608_26523_b200 import dist as D, workloads as W


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _oracle(p, rows, lo=0, hi=-1):
    return oracle.ref_chunk_attn_rows(p.q, p.k_cache, p.v_cache, p.k_cache.stride()[:3], p.v_cache.stride()[:3],
                                      None if p.block_table is None else p.block_table.numpy(), p.block_size,
                                      p.prefix_len.numpy(), p.chunk_len.numpy(), p.num_q_heads, p.num_kv_heads,
                                      p.head_dim_qk, p.head_dim_v, p.scale, rows, lo, hi)


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port), OMP_NUM_THREADS="2")
    try:
        r, w = D.init("gloo")
        assert (r, w) == (rank, world)
        P, C = [40, 0, 300, 7, 129], [9, 5, 17, 30, 3]
        prob = W.make_problem(31, P, C, 4, 2, 16, 16, block_size=8)
        rows_all = oracle.all_rows(C, 4)
        ref_o, ref_l = _oracle(prob, rows_all)

        # (1) request sharding: each rank computes its requests, outputs are gathered, nothing else is exchanged
        parts = D.partition_requests(P, C, world)
        assert sorted(sum(parts, [])) == list(range(5))
        mine = rows_all[np.isin(rows_all[:, 0], parts[rank])]
        o, l = _oracle(prob, mine)
        gathered = [None] * world
        dist.all_gather_object(gathered, (mine, o, l))
        rows_cat = np.concatenate([g[0] for g in gathered]); o_cat = np.concatenate([g[1] for g in gathered])
        order = np.lexsort((rows_cat[:, 2], rows_cat[:, 1], rows_cat[:, 0]))
        assert np.array_equal(rows_cat[order], rows_all) and np.array_equal(o_cat[order], ref_o)

        # (2) KV-range sharding of one long request: partials + all-gather + merge == unsharded
        one = W.make_problem(32, [300], [40], 4, 2, 16, 16, block_size=8)
        rows1 = oracle.all_rows([40], 4)
        full_o, full_l = _oracle(one, rows1)
        lo, hi = D.kv_ranges(340, world)[rank]
        po, pl = _oracle(one, rows1, lo, hi)
        o_all, l_all = D.all_gather_partials(torch.from_numpy(po), torch.from_numpy(pl))
        mo, ml = oracle.ref_lse_merge(o_all.numpy(), l_all.numpy())
        assert np.abs(mo - full_o).max() < 1e-12 and np.abs(ml - full_l).max() < 1e-12

        # (3) timing: the slowest rank decides
        D.barrier()
        assert D.max_over_ranks([1.0 + rank, 5.0 - rank]) == [float(world), 5.0]
        assert abs(D.whole_job_rate(100.0, 1.0 + rank) - world * 100.0 / world) < 1e-12
        q.put((rank, "ok"))
    except Exception as e:  # report instead of hanging the parent
        q.put((rank, "FAIL %r" % (e,)))
    finally:
        if dist.is_initialized():
            dist.destroy_process_group()


@pytest.mark.timeout(180)
def test_two_gloo_ranks():
    oracle.build()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = [q.get(timeout=150) for _ in procs]
    for p in procs:
        p.join(timeout=30)
    assert sorted(res) == [(0, "ok"), (1, "ok")], res


def test_partition_is_balanced_and_complete():
    L, C, P = W.cfg5_lengths()
    for world in (1, 2, 4, 8):
        parts = D.partition_requests(P, C, world)
        assert sorted(sum(parts, [])) == list(range(32))
        cost = [sum(C[i] * P[i] + C[i] * (C[i] + 1) // 2 for i in part) for part in parts]
        assert max(cost) <= sum(cost) / world + max(C[i] * P[i] + C[i] * (C[i] + 1) // 2 for i in range(32))


def test_kv_ranges_cover_the_sequence():
    for n, w in [(340, 2), (1, 4), (128, 2), (100000, 8)]:
        r = D.kv_ranges(n, w)
        assert r[0][0] == 0 and r[-1][1] == n and all(a[1] == b[0] for a, b in zip(r, r[1:]))
        assert all(lo % 128 == 0 for lo, _ in r)


def test_kv_ranges_with_a_prefix_start_inside_it():
    for seq, pre, w in [(5700, 5000, 4), (900, 130, 4), (700, 0, 2), (100000, 99000, 8)]:
        r = D.kv_ranges(seq, w, prefix_len=pre)
        assert r[0][0] == 0 and r[-1][1] == seq and all(a[1] == b[0] for a, b in zip(r, r[1:]))
        assert all(lo % 128 == 0 and lo <= pre for lo, _ in r)
