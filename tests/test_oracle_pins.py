"""Pins for the fp64 CPU oracle: it is checked against what the definition and the mathematics fix
(closed forms, invariants, brute force, a library routine), never against itself or the GPU path.

Definition pinned: Eq. 1 of the paper with its causal rule ("each token attends only to itself and
preceding tokens"), applied per chunk as in the paper's chunked-prefill background section.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2608_26523_b200 import workloads as W


def bf16_bits_to_f64(t):
    return t.to(torch.float64).numpy()


def run_all(p, kv_lo=0, kv_hi=-1, rows=None):
    if rows is None:
        rows = oracle.all_rows(p.chunk_len.numpy(), p.num_q_heads)
    out, lse = oracle.ref_chunk_attn_rows(
        p.q, p.k_cache, p.v_cache, p.k_cache.stride()[:3], p.v_cache.stride()[:3],
        None if p.block_table is None else p.block_table.numpy(), p.block_size,
        p.prefix_len.numpy(), p.chunk_len.numpy(), p.num_q_heads, p.num_kv_heads,
        p.head_dim_qk, p.head_dim_v, p.scale, rows, kv_lo, kv_hi)
    return rows, out, lse


def gather_kv(p, r, g):
    """Logical [seq, D] K and V of request r, kv-head g, as float64 (test-side re-implementation of paging)."""
    n = int(p.prefix_len[r] + p.chunk_len[r])
    K = np.empty((n, p.head_dim_qk)); V = np.empty((n, p.head_dim_v))
    for j in range(n):
        if p.block_table is None:
            blk, slot = r, j
        else:
            blk, slot = int(p.block_table[r, j // p.block_size]), j % p.block_size
        K[j] = p.k_cache[blk, slot, g].to(torch.float64).numpy()
        V[j] = p.v_cache[blk, slot, g].to(torch.float64).numpy()
    return K, V


def brute_force(p):
    """Pure-Python/numpy row-by-row evaluation of the definition with math.exp."""
    G = p.num_q_heads // p.num_kv_heads
    outs, lses = [], []
    qs = 0
    for r in range(p.num_reqs):
        P, C = int(p.prefix_len[r]), int(p.chunk_len[r])
        for i in range(C):
            for h in range(p.num_q_heads):
                K, V = gather_kv(p, r, h // G)
                qv = p.q[qs + i, h].to(torch.float64).numpy()
                s = [p.scale * float(np.dot(qv, K[j])) for j in range(P + i + 1)]
                m = max(s)
                w = [math.exp(x - m) for x in s]
                l = sum(w)
                o = sum(wj * V[j] for j, wj in enumerate(w)) / l
                outs.append(o); lses.append(m + math.log(l))
        qs += C
    return np.array(outs), np.array(lses)


# ---- P5: brute force on tiny shapes -----------------------------------------------------------

@pytest.mark.parametrize("block_size", [None, 4])
def test_brute_force_tiny(block_size):
    p = W.make_problem(11, [0, 5, 2], [3, 4, 1], 4, 2, 8, 6, block_size=block_size)
    _, out, lse = run_all(p)
    bo, bl = brute_force(p)
    assert np.abs(out - bo).max() < 1e-13
    assert np.abs(lse - bl).max() < 1e-13


def test_two_key_closed_form():
    """Row 1 of a fresh chunk sees two keys: weights are sigmoid(s0 - s1) and its complement."""
    p = W.make_problem(12, [0], [2], 1, 1, 4, 3, block_size=None)
    _, out, lse = run_all(p)
    K, V = gather_kv(p, 0, 0)
    q1 = p.q[1, 0].to(torch.float64).numpy()
    s0, s1 = p.scale * q1 @ K[0], p.scale * q1 @ K[1]
    w0 = 1.0 / (1.0 + math.exp(-(s0 - s1)))
    assert np.allclose(out[1], w0 * V[0] + (1 - w0) * V[1], rtol=0, atol=1e-14)
    assert abs(lse[1] - (s1 + math.log1p(math.exp(s0 - s1)))) < 1e-13


def test_hand_evaluated_three_tokens():
    """3 tokens, d=2, numbers chosen by hand (exactly representable in bf16)."""
    q = torch.tensor([[[1.0, 0.0]], [[0.0, 2.0]], [[1.0, 1.0]]], dtype=torch.bfloat16)
    k = torch.tensor([[1.0, 0.0], [0.0, 1.0], [2.0, -1.0]], dtype=torch.bfloat16).view(1, 3, 1, 2)
    v = torch.tensor([[1.0, 2.0], [3.0, -4.0], [0.5, 8.0]], dtype=torch.bfloat16).view(1, 3, 1, 2)
    rows = np.array([[0, 0, 0], [0, 1, 0], [0, 2, 0]], dtype=np.int32)
    out, lse = oracle.ref_chunk_attn_rows(q, k, v, k.stride()[:3], v.stride()[:3], None, 3,
                                          [0], [3], 1, 1, 2, 2, 0.5, rows)
    # row 0: only key 0, s = 0.5
    assert np.array_equal(out[0], [1.0, 2.0]) and abs(lse[0] - 0.5) < 1e-15
    # row 1: s = (0, 1): weights 1/(1+e), e/(1+e)
    e = math.e
    assert np.allclose(out[1], [(1 + 3 * e) / (1 + e), (2 - 4 * e) / (1 + e)], atol=1e-14, rtol=0)
    assert abs(lse[1] - math.log(1 + e)) < 1e-14
    # row 2: s = (0.5, 0.5, 0.5): uniform weights
    assert np.allclose(out[2], [1.5, 2.0], atol=1e-14, rtol=0)
    assert abs(lse[2] - (0.5 + math.log(3))) < 1e-14


# ---- P3: single key ---------------------------------------------------------------------------

def test_single_key_returns_value_row():
    p = W.make_problem(13, [0], [5], 4, 2, 16, 16, block_size=8)
    rows = np.array([[0, 0, h] for h in range(4)], dtype=np.int32)
    _, out, lse = run_all(p, rows=rows)
    for h in range(4):
        K, V = gather_kv(p, 0, h // 2)
        assert np.array_equal(out[h], V[0])
        assert abs(lse[h] - p.scale * float(p.q[0, h].to(torch.float64).numpy() @ K[0])) < 1e-14


# ---- P2 / P6: identical keys, zero queries ----------------------------------------------------

def test_identical_keys_give_running_mean():
    p = W.make_problem(14, [7], [6], 2, 1, 8, 4, block_size=4)
    p.k_cache[:] = p.k_cache[int(p.block_table[0, 0]), 0, 0]
    _, out, lse = run_all(p)
    K, V = gather_kv(p, 0, 0)
    n = 0
    for i in range(6):
        for h in range(2):
            pos = 7 + i
            assert np.abs(out[n] - V[:pos + 1].mean(0)).max() < 1e-13
            s = p.scale * float(p.q[i, h].to(torch.float64).numpy() @ K[0])
            assert abs(lse[n] - (s + math.log(pos + 1))) < 1e-13
            n += 1


def test_zero_queries_uniform_weights():
    p = W.make_problem(15, [3], [4], 2, 2, 8, 8, block_size=None)
    p.q.zero_()
    _, out, lse = run_all(p)
    n = 0
    for i in range(4):
        for h in range(2):
            _, V = gather_kv(p, 0, h)
            assert np.abs(out[n] - V[:3 + i + 1].mean(0)).max() < 1e-13
            assert abs(lse[n] - math.log(3 + i + 1)) < 1e-13
            n += 1


# ---- P1: chunked == unchunked == explicit full causal softmax (config 1, full size) ------------

def test_cfg1_chunked_equals_unchunked_equals_dense():
    full = W.cfg1(0).extra["full"]              # P=0, C=2048
    _, out_full, lse_full = run_all(full)
    out_full = out_full.reshape(2048, 4, 128); lse_full = lse_full.reshape(2048, 4)
    for k in range(4):
        pk = W.cfg1(k)
        _, o, l = run_all(pk)
        assert np.abs(o.reshape(512, 4, 128) - out_full[512 * k:512 * (k + 1)]).max() < 1e-12
        assert np.abs(l.reshape(512, 4) - lse_full[512 * k:512 * (k + 1)]).max() < 1e-12
    # explicit dense causal softmax in numpy float64
    K = full.k_cache[0, :, 0].to(torch.float64).numpy()
    V = full.v_cache[0, :, 0].to(torch.float64).numpy()
    mask = np.tril(np.ones((2048, 2048), dtype=bool))
    for h in range(4):
        Q = full.q[:, h].to(torch.float64).numpy()
        S = np.where(mask, full.scale * (Q @ K.T), -np.inf)
        m = S.max(1, keepdims=True)
        E = np.exp(S - m)
        l = E.sum(1, keepdims=True)
        assert np.abs((E / l) @ V - out_full[:, h]).max() < 1e-12
        assert np.abs((m + np.log(l))[:, 0] - lse_full[:, h]).max() < 1e-12


# ---- P4: split + merge == unsplit ---------------------------------------------------------------

@pytest.mark.parametrize("cuts", [[0, 9, 25, 10 ** 9], [0, 0, 5, 26, 10 ** 9], [0, 24, 10 ** 9]])
def test_split_merge_equals_unsplit(cuts):
    # prefix 20, chunk 8: rows sit at positions 20..27; a cut at 24 or 26 lies beyond the causal
    # horizon of the early rows, and [0,0) is an empty segment
    p = W.make_problem(16, [20], [8], 4, 2, 16, 12, block_size=8)
    rows, out, lse = run_all(p)
    parts_o, parts_l = [], []
    for lo, hi in zip(cuts[:-1], cuts[1:]):
        _, o, l = run_all(p, kv_lo=lo, kv_hi=hi)
        parts_o.append(o); parts_l.append(l)
    assert any(np.isneginf(l).any() for l in parts_l)
    mo, ml = oracle.ref_lse_merge(np.stack(parts_o), np.stack(parts_l))
    assert np.abs(mo - out).max() < 1e-12
    assert np.abs(ml - lse).max() < 1e-12


def test_merge_closed_form_and_all_empty():
    o = np.array([[[1.0, 2.0]], [[3.0, 6.0]]])          # S=2, n=1, Dv=2
    l = np.array([[math.log(1.0)], [math.log(3.0)]])     # weights 1/4, 3/4
    mo, ml = oracle.ref_lse_merge(o, l)
    assert np.allclose(mo, [[2.5, 5.0]], atol=1e-15) and abs(ml[0] - math.log(4.0)) < 1e-15
    mo, ml = oracle.ref_lse_merge(np.ones((2, 1, 2)), np.full((2, 1), -np.inf))
    assert np.array_equal(mo, [[0.0, 0.0]]) and np.isneginf(ml[0])
    # order of the operands matters: swapping the partials but not the lse changes the answer
    mo2, _ = oracle.ref_lse_merge(o[::-1].copy(), l)
    assert np.allclose(mo2, [[1.5, 3.0]], atol=1e-15)


# ---- P7: invariants ---------------------------------------------------------------------------------

def test_invariants_shift_constant_v_causality_bounds():
    p = W.make_problem(17, [10, 0], [6, 9], 4, 2, 16, 8, block_size=4, unused_fill=float("nan"),
                       tail_fill=float("nan"))
    rows, out, lse = run_all(p)
    assert np.isfinite(out).all() and np.isfinite(lse).all()     # NaN tails / unused blocks never read
    # within [min, max] of the visible values
    G = 2
    for n, (r, i, h) in enumerate(rows):
        _, V = gather_kv(p, r, h // G)
        vis = V[: int(p.prefix_len[r]) + i + 1]
        assert (out[n] <= vis.max(0) + 1e-12).all() and (out[n] >= vis.min(0) - 1e-12).all()
    # V == 1 -> out == 1
    p1 = W.make_problem(17, [10, 0], [6, 9], 4, 2, 16, 8, block_size=4, tail_fill=None, unused_fill=None)
    p1.v_cache.fill_(1.0)
    _, o1, _ = run_all(p1)
    assert np.abs(o1 - 1.0).max() < 1e-14
    # adding a constant vector c to every key shifts lse by scale*q.c and leaves out unchanged
    p2 = W.make_problem(18, [5], [4], 2, 1, 8, 8, block_size=None)
    p2.k_cache.copy_((p2.k_cache.float().clamp(-4, 4) * 8).round() / 8)    # coarse grid: the shift stays exact
    _, oa, la = run_all(p2)
    c = torch.tensor([0.5, -1.0, 0.25, 2.0, 0.0, 1.0, -0.5, 0.125], dtype=torch.float64)
    kf = p2.k_cache.to(torch.float64) + c
    assert torch.equal(kf.to(torch.bfloat16).to(torch.float64), kf), "shift must stay exact in bf16"
    p2.k_cache.copy_(kf.to(torch.bfloat16))
    _, ob, lb = run_all(p2)
    shift = np.array([p2.scale * float(p2.q[i, h].to(torch.float64) @ c) for i in range(4) for h in range(2)])
    assert np.abs(oa - ob).max() < 1e-12 and np.abs(lb - la - shift).max() < 1e-12


def test_causality_future_keys_do_not_matter_and_prefix_permutation():
    p = W.make_problem(19, [6], [5], 2, 1, 8, 8, block_size=None)
    rows, out, lse = run_all(p)
    # change K/V at the last position: only the last row (both heads) may change
    p.k_cache[0, 10] = 3.0; p.v_cache[0, 10] = -7.0
    _, o2, l2 = run_all(p)
    assert np.array_equal(out[:-2], o2[:-2]) and np.array_equal(lse[:-2], l2[:-2])
    assert not np.array_equal(out[-2:], o2[-2:])
    # permuting (k_j, v_j) pairs inside the prefix leaves every row unchanged up to summation order
    perm = torch.tensor([3, 0, 5, 1, 4, 2])
    p.k_cache[0, :6] = p.k_cache[0, perm]; p.v_cache[0, :6] = p.v_cache[0, perm]
    _, o3, l3 = run_all(p)
    assert np.abs(o3 - o2).max() < 1e-13 and np.abs(l3 - l2).max() < 1e-13


def test_shuffled_block_table_equals_contiguous():
    kw = dict(prefix_lens=[13, 0, 40], chunk_lens=[9, 7, 3], num_q_heads=4, num_kv_heads=2,
              head_dim_qk=16, head_dim_v=16)
    pc = W.make_problem(20, block_size=None, tail_fill=None, unused_fill=None, **kw)
    pp = W.make_problem(21, block_size=8, **kw)
    # copy the logical contents of the contiguous cache into the paged one
    pp.q.copy_(pc.q)
    for r in range(3):
        for j in range(kw["prefix_lens"][r] + kw["chunk_lens"][r]):
            blk = int(pp.block_table[r, j // 8])
            pp.k_cache[blk, j % 8] = pc.k_cache[r, j]
            pp.v_cache[blk, j % 8] = pc.v_cache[r, j]
    _, oc, lc = run_all(pc)
    _, op, lp = run_all(pp)
    assert np.array_equal(oc, op) and np.array_equal(lc, lp)


def test_gqa_head_mapping_is_contiguous_groups():
    """q-heads 0..G-1 read kv-head 0, the next G read kv-head 1, ..."""
    p = W.make_problem(22, [4], [2], 6, 3, 8, 8, block_size=None)
    p.q[:] = p.q[:, :1]                           # all heads share one query vector
    _, out, _ = run_all(p)
    out = out.reshape(2, 6, 8)
    assert np.array_equal(out[:, 0], out[:, 1]) and np.array_equal(out[:, 2], out[:, 3])
    assert not np.array_equal(out[:, 1], out[:, 2]) and not np.array_equal(out[:, 3], out[:, 4])


def test_mla_aliasing_v_is_prefix_of_k_row():
    p = W.make_problem(23, [9], [4], 4, 1, 24, 16, block_size=4, std=0.5, v_aliases_k=True,
                       scale=1.0 / math.sqrt(192.0))
    assert p.v_cache.data_ptr() == p.k_cache.data_ptr() and p.v_cache.stride() == p.k_cache.stride()
    _, out, lse = run_all(p)
    bo, bl = brute_force(p)
    assert np.abs(out - bo).max() < 1e-13 and np.abs(lse - bl).max() < 1e-13


# ---- P8: library special case -------------------------------------------------------------------

@pytest.mark.parametrize("P,C,hq,hkv,dqk,dv,bs", [(0, 33, 4, 4, 32, 32, None), (50, 17, 8, 2, 64, 64, 16),
                                                  (31, 40, 4, 1, 48, 32, 8)])
def test_against_torch_sdpa_float64(P, C, hq, hkv, dqk, dv, bs):
    p = W.make_problem(24 + P, [P], [C], hq, hkv, dqk, dv, block_size=bs, v_aliases_k=(dqk != dv))
    _, out, lse = run_all(p)
    out = out.reshape(C, hq, dv)
    G = hq // hkv
    pos = torch.arange(P, P + C)[:, None]
    mask = torch.arange(P + C)[None, :] <= pos                      # explicit boolean mask
    for h in range(hq):
        K, V = gather_kv(p, 0, h // G)
        ref = torch.nn.functional.scaled_dot_product_attention(
            p.q[:, h].to(torch.float64)[None], torch.from_numpy(K)[None], torch.from_numpy(V)[None],
            attn_mask=mask[None], scale=p.scale)[0].numpy()
        assert np.abs(ref - out[:, h]).max() < 1e-10
    # lse against torch.logsumexp
    S = p.scale * (p.q[:, 0].to(torch.float64) @ torch.from_numpy(gather_kv(p, 0, 0)[0]).T)
    ref_lse = torch.logsumexp(S.masked_fill(~mask, float("-inf")), dim=1).numpy()
    assert np.abs(ref_lse - lse.reshape(C, hq)[:, 0]).max() < 1e-12


def test_bad_row_triple_is_rejected():
    p = W.make_problem(30, [2], [3], 2, 1, 8, 8, block_size=None)
    with pytest.raises(ValueError):
        run_all(p, rows=np.array([[0, 3, 0]], dtype=np.int32))
