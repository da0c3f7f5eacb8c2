"""Full-size parity: the benchmark configurations at their real sizes, in the launch configuration bench.py
times, compared with the CPU oracle on a deterministic sample of rows the oracle can compute one by one
(chunk ends, rows around query-tile edges and cache-block edges, random (row, head) pairs)."""
import numpy as np
import pytest
import torch

from paper_2608_26523_b200 import api, workloads as W
from parity import compare, run_gpu, sample_rows

pytestmark = pytest.mark.gpu


def check_sampled(prob_gpu, label, num_kv_splits=0, n_random=192, seed=0):
    out, lse, runner = run_gpu(prob_gpu, num_kv_splits)
    # every row of the launch must have been written (canaries were NaN)
    assert torch.isfinite(out.float()).all() and torch.isfinite(lse).all(), label
    prob_cpu = prob_gpu.to("cpu")
    rows = sample_rows(prob_cpu, n_random=n_random, seed=seed)
    s = compare(out, lse, prob_cpu, rows, label)
    print(s)
    return s


@pytest.mark.parametrize("prefix", [0, 8192, 65536, 131072])
def test_cfg2_gqa_long_context(prefix):
    check_sampled(W.cfg2(prefix=prefix, device="cuda"), "cfg2 P=%d" % prefix)


@pytest.mark.parametrize("prefix,splits", [(0, 4), (16384 * 13, 4), (16384 * 63, 4), (16384 * 63, 1)])
def test_cfg4_million_token_split_kv(prefix, splits):
    check_sampled(W.cfg4(prefix=prefix, device="cuda"), "cfg4 P=%d S=%d" % (prefix, splits),
                  num_kv_splits=splits, n_random=128)


@pytest.mark.parametrize("prefix", [0, 65536, 516096])
def test_cfg3_absorbed_mla(prefix):
    check_sampled(W.cfg3(prefix=prefix, device="cuda"), "cfg3 P=%d" % prefix, n_random=96)


def test_cfg5_mixed_varlen_batch():
    prob = W.cfg5(device="cuda")
    assert prob.total_q == 16384 and prob.num_reqs == 32
    check_sampled(prob, "cfg5", n_random=256)


def test_cfg5_mixed_varlen_batch_forced_split():
    check_sampled(W.cfg5(device="cuda"), "cfg5 S=3", num_kv_splits=3, n_random=128, seed=1)
