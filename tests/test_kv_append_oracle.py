"""Pins for the KV-append oracle: a hand-written placement, and the tie to the attention oracle (a cache built by
appending chunk after chunk gives the same attention as the cache built in one piece)."""
import numpy as np
import torch

import oracle
from oracle.ref_kv_append import ref_kv_append
from paper_2608_26523_b200 import workloads as W


def test_hand_written_placement():
    # 2 requests, pages of 4 slots, 1 kv-head, 2 features.  Request 0 has 3 cached tokens and appends 3 (positions
    # 3, 4, 5: slot 3 of its first page, slots 0 and 1 of its second); request 1 has 0 cached and appends 2.
    k_cache = np.zeros((5, 4, 1, 2), np.uint16)
    bt = np.array([[2, 0], [4, 1]], np.int32)
    k_new = (np.arange(5 * 2, dtype=np.uint16) + 100).reshape(5, 1, 2)
    k_out, v_out = ref_kv_append(k_cache, None, k_new, None, bt, 4, [3, 0], [3, 2])
    assert v_out is None
    want = np.zeros_like(k_cache)
    want[2, 3, 0] = [100, 101]   # request 0, position 3 -> logical page 0 = physical 2, slot 3
    want[0, 0, 0] = [102, 103]   # position 4 -> logical page 1 = physical 0, slot 0
    want[0, 1, 0] = [104, 105]
    want[4, 0, 0] = [106, 107]   # request 1, position 0 -> physical 4, slot 0
    want[4, 1, 0] = [108, 109]
    assert (k_out == want).all()


def test_contiguous_cache_and_separate_values():
    k_cache = np.full((2, 6, 2, 8), 7, np.uint16)
    v_cache = np.full((2, 6, 2, 8), 9, np.uint16)
    k_new = np.arange(3 * 2 * 8, dtype=np.uint16).reshape(3, 2, 8)
    v_new = k_new + 1000
    k_out, v_out = ref_kv_append(k_cache, v_cache, k_new, v_new, None, 0, [4, 1], [2, 1])
    assert (k_out[0, 4] == k_new[0]).all() and (k_out[0, 5] == k_new[1]).all() and (k_out[1, 1] == k_new[2]).all()
    assert (v_out[0, 5] == v_new[1]).all() and (v_out[1, 1] == v_new[2]).all()
    untouched = np.ones((2, 6), bool)
    untouched[0, 4] = untouched[0, 5] = untouched[1, 1] = False
    assert (k_out[untouched] == 7).all() and (v_out[untouched] == 9).all()
    assert (k_cache == 7).all()          # the inputs are not modified


def _bits(t):
    return t.view(torch.int16).numpy().view(np.uint16)


def test_chunk_by_chunk_append_rebuilds_the_cache_and_the_attention():
    full = W.make_problem(31, [0, 0], [150, 70], 4, 2, 128, 128, block_size=16, std=0.5)
    kb, vb = _bits(full.k_cache), _bits(full.v_cache)
    bt = full.block_table.numpy()
    # start from a cache that has nothing of these requests and append in chunks of 64 tokens
    k_run, v_run = np.array(kb, copy=True), np.array(vb, copy=True)
    lens = [150, 70]
    for r, n in enumerate(lens):
        for pos in range(n):
            k_run[bt[r, pos // 16], pos % 16] = 0xFFFF
            v_run[bt[r, pos // 16], pos % 16] = 0xFFFF
    done = [0, 0]
    while any(d < n for d, n in zip(done, lens)):
        chunk = [min(64, n - d) for d, n in zip(done, lens)]
        rows_k, rows_v = [], []
        for r in range(2):
            for pos in range(done[r], done[r] + chunk[r]):
                rows_k.append(kb[bt[r, pos // 16], pos % 16])
                rows_v.append(vb[bt[r, pos // 16], pos % 16])
        k_run, v_run = ref_kv_append(k_run, v_run, np.stack(rows_k), np.stack(rows_v), bt, 16, done, chunk)
        done = [d + c for d, c in zip(done, chunk)]
    used = np.zeros(kb.shape[:2], bool)
    for r, n in enumerate(lens):
        for pos in range(n):
            used[bt[r, pos // 16], pos % 16] = True
    assert (k_run[used] == kb[used]).all() and (v_run[used] == vb[used]).all()
    assert (k_run[~used] == kb[~used]).all()
    # the attention oracle sees the same cache either way
    rows = oracle.all_rows(full.chunk_len.numpy(), full.num_q_heads)[::37]
    ks, vs = full.k_cache.stride(), full.v_cache.stride()
    kw = dict(block_table=bt, block_size=16, prefix_len=full.prefix_len.numpy(), chunk_len=full.chunk_len.numpy(),
              num_q_heads=4, num_kv_heads=2, head_dim_qk=128, head_dim_v=128, scale=full.scale, rows=rows)
    o1, l1 = oracle.ref_chunk_attn_rows(_bits(full.q), kb, vb, ks[:3], vs[:3], **kw)
    o2, l2 = oracle.ref_chunk_attn_rows(_bits(full.q), k_run, v_run, ks[:3], vs[:3], **kw)
    assert (o1 == o2).all() and (l1 == l2).all()
