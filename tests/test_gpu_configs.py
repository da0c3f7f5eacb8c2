"""Full-size parity: the benchmark configurations at their real sizes, in the launch configuration bench.py
times, compared with the CPU oracle on a deterministic sample of rows the oracle can compute one by one:
chunk ends, rows around query-tile edges and cache-block edges, random (row, head) pairs, and one random row of
every work item of the launch (query tile x pair of q-heads for the d = 128 kernel, query tile x kv-head for
the 1M-token sweep; for the absorbed-MLA kernel one row of every query tile and every head of eight rows), so
that an error tied to an item's place in the schedule cannot hide behind the sample."""
import numpy as np
import pytest
import torch

from paper_2608_26523_b200 import api, workloads as W
from parity import all_heads_of_rows, compare, run_gpu, sample_rows, tile_rows

pytestmark = pytest.mark.gpu


def check_sampled(prob_gpu, label, num_kv_splits=0, n_random=192, seed=0, per_item=None, heads_of_rows=0):
    out, lse, runner = run_gpu(prob_gpu, num_kv_splits)
    # every row of the launch must have been written (canaries were NaN)
    assert torch.isfinite(out.float()).all() and torch.isfinite(lse).all(), label
    prob_cpu = prob_gpu.to("cpu")
    rows = [sample_rows(prob_cpu, n_random=n_random, seed=seed)]
    if per_item:
        rows.append(tile_rows(prob_cpu, per=per_item, seed=seed + 1))
    if heads_of_rows:
        rows.append(all_heads_of_rows(prob_cpu, heads_of_rows, seed=seed + 2))
    rows = np.unique(np.concatenate(rows), axis=0)
    s = compare(out, lse, prob_cpu, rows, label)
    print(s)
    return s


@pytest.mark.parametrize("prefix", W.CFG2_PREFIXES)
def test_cfg2_gqa_long_context(prefix):
    # 64 query tiles x 32 pairs of q-heads = 2048 work items, one compared row in each
    s = check_sampled(W.cfg2(prefix=prefix, device="cuda"), "cfg2 P=%d" % prefix, per_item="pair")
    assert s["rows"] >= 2048


@pytest.mark.parametrize("prefix,splits", [(0, 4), (16384 * 8, 0), (16384 * 13, 4), (16384 * 34, 4), (16384 * 63, 4),
                                           (16384 * 63, 1)])
def test_cfg4_million_token_split_kv(prefix, splits):
    # 128 query tiles x 8 kv-heads, one compared row in each (the oracle needs ~0.5 GFLOP per row at 1M tokens)
    assert prefix in W.CFG4_PREFIXES
    s = check_sampled(W.cfg4(prefix=prefix, device="cuda"), "cfg4 P=%d S=%d" % (prefix, splits),
                      num_kv_splits=splits, n_random=128, per_item="kvhead")
    assert s["rows"] >= 1024


@pytest.mark.parametrize("prefix", W.CFG3_PREFIXES)
def test_cfg3_absorbed_mla(prefix):
    # one row of each of the 64 query tiles, and all 128 heads of eight rows
    s = check_sampled(W.cfg3(prefix=prefix, device="cuda"), "cfg3 P=%d" % prefix, n_random=96, per_item="tile",
                      heads_of_rows=8)
    assert s["rows"] >= 1024


def test_cfg5_mixed_varlen_batch():
    prob = W.cfg5(device="cuda")
    assert prob.total_q == 16384 and prob.num_reqs == 32
    check_sampled(prob, "cfg5", n_random=256, per_item="pair")


def test_cfg5_mixed_varlen_batch_forced_split():
    check_sampled(W.cfg5(device="cuda"), "cfg5 S=3", num_kv_splits=3, n_random=128, seed=1, per_item="kvhead")
