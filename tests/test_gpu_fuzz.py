"""Randomised parity: seeded random batches (request counts, prefix and chunk lengths, head counts, page sizes, split
counts, both head-dim families) through the C ABI against the fp64 oracle, every element.  The shapes are drawn so that
short items, ragged tails, single-token rows, empty requests and diagonal-only tiles mix within one launch -- the
situations in which the kernels' rings, barrier phases and tail fix-ups wrap around each other."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_26523_b200 import workloads as W
from parity import compare, run_gpu

pytestmark = pytest.mark.gpu


def _draw(seed):
    rng = np.random.default_rng(seed)
    mla = rng.random() < 0.35
    R = int(rng.integers(1, 7))
    kinds = rng.integers(0, 6, size=R)
    prefix, chunk = [], []
    for k in kinds:
        if k == 0:                       # decode row
            prefix.append(int(rng.integers(0, 700)))
            chunk.append(1)
        elif k == 1:                     # empty request
            prefix.append(int(rng.integers(0, 300)))
            chunk.append(0)
        elif k == 2:                     # first chunk of a prompt
            prefix.append(0)
            chunk.append(int(rng.integers(1, 400)))
        else:                            # a chunk somewhere in a prompt
            prefix.append(int(rng.integers(1, 900)))
            chunk.append(int(rng.integers(2, 420)))
    if sum(chunk) == 0:
        chunk[0] = 5
    if mla:
        hq, hkv, dqk, dv = int(rng.choice([1, 2, 16, 72, 128])), 1, 576, 512
        scale, std = 1.0 / 192 ** 0.5, 0.5
    else:
        hkv = int(rng.choice([1, 2, 3]))
        hq = hkv * int(rng.choice([1, 2, 3, 4, 8]))
        dqk = dv = 128
        scale, std = None, float(rng.choice([0.5, 0.7, 1.0]))     # (the value range of the benchmark inputs: the tolerance is derived for it)
    bs = rng.choice([None, 16, 32, 64, 128, 256])
    bs = None if bs is None else int(bs)
    splits = int(rng.choice([0, 0, 1, 2, 3, 5]))
    return dict(prefix=prefix, chunk=chunk, hq=hq, hkv=hkv, dqk=dqk, dv=dv, bs=bs, splits=splits, scale=scale, std=std, mla=mla)


@pytest.mark.parametrize("seed", range(48))
def test_random_batches(seed):
    c = _draw(7000 + seed)
    prob = W.make_problem(8000 + seed, c["prefix"], c["chunk"], c["hq"], c["hkv"], c["dqk"], c["dv"], block_size=c["bs"],
                          std=c["std"], scale=c["scale"], v_aliases_k=c["mla"])
    out, lse, _ = run_gpu(prob.to("cuda"), c["splits"])
    rows = oracle.all_rows(prob.chunk_len.numpy(), prob.num_q_heads)
    print(c, compare(out, lse, prob, rows, "fuzz %d" % seed))


@pytest.mark.parametrize("seed", range(12))
def test_random_batches_of_many_items(seed):
    """Launches of several hundred to a few thousand work items (every CTA runs many, long and short ones in turn), d = 128
    and MLA: item ring, K/V ring, tail fix-ups and barrier phases across item boundaries."""
    rng = np.random.default_rng(7500 + seed)
    mla = seed % 3 == 2
    R = int(rng.integers(12, 48))
    prefix = [int(rng.integers(0, 2500)) if rng.random() < 0.8 else 0 for _ in range(R)]
    chunk = [1 if rng.random() < 0.3 else int(rng.integers(1, 330)) for _ in range(R)]
    bs = int(rng.choice([16, 64, 128]))
    if mla:
        prob = W.make_problem(8500 + seed, prefix, chunk, 32, 1, 576, 512, block_size=bs, std=0.5, scale=1.0 / 192 ** 0.5,
                              v_aliases_k=True)
    else:
        hkv = int(rng.choice([2, 4]))
        prob = W.make_problem(8500 + seed, prefix, chunk, hkv * int(rng.choice([1, 4, 8])), hkv, 128, 128, block_size=bs, std=0.7)
    out, lse, _ = run_gpu(prob.to("cuda"), int(rng.choice([0, 0, 2])))
    rows = oracle.all_rows(prob.chunk_len.numpy(), prob.num_q_heads)
    print(R, sum(chunk), bs, compare(out, lse, prob, rows, "fuzz many %d" % seed))
