"""Pins for the sparse (index-selected) attention oracle: closed forms, special cases that reduce to the dense
oracle (separate C code), brute force with math.exp, and invariants -- never the oracle against itself or the GPU."""
import math

import numpy as np
import pytest
import torch

import oracle
from oracle.ref_sparse_attn import ref_sparse_chunk_attn
from paper_2608_26523_b200 import workloads as W


def _bits(t):
    return t.view(torch.int16).numpy().view(np.uint16)


def _problem(seed=11, prefix=(37, 0), chunk=(9, 5), hq=4, dqk=32, dv=16, bs=8):
    return W.make_problem(seed, list(prefix), list(chunk), hq, 1, dqk, dv, block_size=bs, std=0.8, v_aliases_k=True)


def _run(p, idx, tokens=None):
    return ref_sparse_chunk_attn(_bits(p.q), _bits(p.k_cache), idx, None if p.block_table is None else p.block_table.numpy(),
                                 p.block_size, p.prefix_len.numpy(), p.chunk_len.numpy(), p.head_dim_v, p.scale, tokens)


def _logical_row(p, r, pos):
    blk, slot = int(p.block_table[r, pos // p.block_size]), pos % p.block_size
    return p.k_cache[blk, slot, 0].to(torch.float64).numpy()


def _token_table(p):
    rows = []
    for r in range(p.num_reqs):
        for i in range(int(p.chunk_len[r])):
            rows.append((r, int(p.prefix_len[r]) + i))
    return rows


def test_listing_every_causal_position_is_dense_attention():
    """A list that names all positions 0..pos, in any order, must give the dense causal result (Eq. 1) -- computed by
    the dense oracle, which is separate C code pinned on its own."""
    p = _problem()
    tt = _token_table(p)
    topk = max(pos for _, pos in tt) + 4
    rng = np.random.default_rng(3)
    idx = np.full((len(tt), topk), -1, np.int32)
    for t, (_, pos) in enumerate(tt):
        idx[t, : pos + 1] = rng.permutation(pos + 1)
    out, lse = _run(p, idx)
    rows = oracle.all_rows(p.chunk_len.numpy(), p.num_q_heads)
    ref_o, ref_l = oracle.ref_chunk_attn_rows(p.q, p.k_cache, p.v_cache, p.k_cache.stride()[:3], p.v_cache.stride()[:3],
                                              p.block_table.numpy(), p.block_size, p.prefix_len.numpy(), p.chunk_len.numpy(),
                                              p.num_q_heads, 1, p.head_dim_qk, p.head_dim_v, p.scale, rows)
    np.testing.assert_allclose(out.reshape(-1, p.head_dim_v), ref_o, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(lse.reshape(-1), ref_l, rtol=1e-12, atol=1e-13)


def test_single_entry_returns_that_value_row_and_its_score():
    p = _problem()
    tt = _token_table(p)
    idx = np.full((len(tt), 3), -1, np.int32)
    picks = [pos // 2 for _, pos in tt]
    idx[:, 1] = picks
    out, lse = _run(p, idx)
    for t, (r, pos) in enumerate(tt):
        krow = _logical_row(p, r, picks[t])
        for h in range(p.num_q_heads):
            qv = p.q[t, h].to(torch.float64).numpy()
            s = p.scale * sum(float(a) * float(b) for a, b in zip(qv, krow))
            assert np.array_equal(out[t, h], krow[: p.head_dim_v])
            assert abs(lse[t, h] - s) <= 1e-12 * max(1.0, abs(s))


def test_two_entries_closed_form_and_duplicates_count_twice():
    p = _problem()
    tt = _token_table(p)
    t = len(tt) - 1
    r, pos = tt[t]
    a, b = 1, pos
    idx = np.full((len(tt), 4), -1, np.int32)
    idx[t, :2] = [a, b]
    out, lse = _run(p, idx, tokens=[t])
    ka, kb = _logical_row(p, r, a), _logical_row(p, r, b)
    for h in range(p.num_q_heads):
        qv = p.q[t, h].to(torch.float64).numpy()
        sa, sb = p.scale * float(qv @ ka), p.scale * float(qv @ kb)
        wa = 1.0 / (1.0 + math.exp(sb - sa))
        np.testing.assert_allclose(out[0, h], wa * ka[: p.head_dim_v] + (1 - wa) * kb[: p.head_dim_v], rtol=1e-12, atol=1e-14)
        assert abs(lse[0, h] - (max(sa, sb) + math.log1p(math.exp(-abs(sa - sb))))) < 1e-12
    # the same position twice: same output, lse larger by ln 2
    idx2 = np.full((len(tt), 4), -1, np.int32)
    idx2[t, :2] = [a, a]
    idx1 = np.full((len(tt), 4), -1, np.int32)
    idx1[t, 0] = a
    o2, l2 = _run(p, idx2, tokens=[t])
    o1, l1 = _run(p, idx1, tokens=[t])
    np.testing.assert_allclose(o2, o1, rtol=1e-13)
    np.testing.assert_allclose(l2, l1 + math.log(2.0), rtol=1e-13)


def test_entries_that_are_negative_or_in_the_future_are_skipped():
    p = _problem()
    tt = _token_table(p)
    rng = np.random.default_rng(5)
    base = np.full((len(tt), 6), -1, np.int32)
    noisy = np.full((len(tt), 11), -1, np.int32)
    for t, (_, pos) in enumerate(tt):
        sel = rng.choice(pos + 1, size=min(pos + 1, 6), replace=False)
        base[t, : sel.size] = sel
        row = np.concatenate([sel, [pos + 1, pos + 1000, -7, -1, 2 ** 30]])
        noisy[t, : row.size] = row[rng.permutation(row.size)]
    o1, l1 = _run(p, base)
    o2, l2 = _run(p, noisy)
    np.testing.assert_allclose(o2, o1, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(l2, l1, rtol=1e-13)
    # nothing selected at all: zero output, lse = -inf
    o0, l0 = _run(p, np.full((len(tt), 4), -1, np.int32))
    assert (o0 == 0).all() and np.isneginf(l0).all()


def test_brute_force_with_math_exp_on_a_tiny_case():
    p = _problem(seed=12, prefix=(5,), chunk=(4,), hq=2, dqk=8, dv=4, bs=4)
    tt = _token_table(p)
    idx = W.make_sparse_indices(9, [5], [4], 3)
    out, lse = _run(p, idx)
    for t, (r, pos) in enumerate(tt):
        for h in range(2):
            qv = [float(x) for x in p.q[t, h].to(torch.float64)]
            ks = [[float(x) for x in _logical_row(p, r, int(e))] for e in idx[t] if 0 <= e <= pos]
            s = [p.scale * sum(a * b for a, b in zip(qv, k)) for k in ks]
            m = max(s)
            w = [math.exp(x - m) for x in s]
            l = sum(w)
            for d in range(4):
                assert abs(out[t, h, d] - sum(wi * k[d] for wi, k in zip(w, ks)) / l) < 1e-13
            assert abs(lse[t, h] - (m + math.log(l))) < 1e-13


def test_uniform_scores_average_the_selected_values_and_paging_does_not_matter():
    # q = 0: every selected key weighs the same -> out = mean of the listed value rows, lse = ln(count)
    p = _problem(seed=13)
    p.q.zero_()
    tt = _token_table(p)
    idx = W.make_sparse_indices(21, p.prefix_len.tolist(), p.chunk_len.tolist(), 5)
    out, lse = _run(p, idx)
    for t, (r, pos) in enumerate(tt):
        sel = [int(e) for e in idx[t] if 0 <= e <= pos]
        mean = np.mean([_logical_row(p, r, e)[: p.head_dim_v] for e in sel], axis=0)
        np.testing.assert_allclose(out[t, 0], mean, rtol=1e-13, atol=1e-15)
        assert abs(lse[t, 0] - math.log(len(sel))) < 1e-13
    # the same logical cache behind another block table: identical results
    p1 = _problem(seed=14)
    perm = np.random.default_rng(2).permutation(p1.k_cache.shape[0])
    inv = np.argsort(perm)
    k2 = p1.k_cache[torch.from_numpy(perm)]
    bt2 = torch.from_numpy(inv.astype(np.int32))[p1.block_table.clamp(min=0).long()].to(torch.int32)
    idx = W.make_sparse_indices(22, p1.prefix_len.tolist(), p1.chunk_len.tolist(), 7)
    a = ref_sparse_chunk_attn(_bits(p1.q), _bits(p1.k_cache), idx, p1.block_table.numpy(), p1.block_size,
                              p1.prefix_len.numpy(), p1.chunk_len.numpy(), p1.head_dim_v, p1.scale)
    b = ref_sparse_chunk_attn(_bits(p1.q), _bits(k2), idx, bt2.numpy(), p1.block_size, p1.prefix_len.numpy(),
                              p1.chunk_len.numpy(), p1.head_dim_v, p1.scale)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


@pytest.mark.parametrize("kind", ["scattered", "clustered"])
def test_index_generator_lists_distinct_causal_positions(kind):
    prefix, chunk, topk = [300, 0], [130, 70], 64
    idx = W.make_sparse_indices(7, prefix, chunk, topk, kind=kind, group=32)
    row = 0
    for P, C in zip(prefix, chunk):
        for i in range(C):
            e = idx[row + i]
            sel = e[e >= 0]
            assert sel.size == min(topk, P + i + 1) and np.unique(sel).size == sel.size and sel.max() <= P + i
            assert (e[sel.size:] == -1).all()
            if P + i + 1 > topk:
                assert np.isin(np.arange(P + i + 1 - topk // 4, P + i + 1), sel).all()
        row += C
    assert np.array_equal(idx, W.make_sparse_indices(7, prefix, chunk, topk, kind=kind, group=32))
