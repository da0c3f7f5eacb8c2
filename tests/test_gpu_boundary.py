"""GPU tests of the boundary beside the attention results themselves: the bounded device wait that runs out, the
tensor-map cache, and key-range partial launches (the context-parallel building block) merged by vpp_lse_merge."""
import time

import numpy as np
import pytest
import torch

import oracle
from paper_2608_26523_b200 import api, workloads as W
from parity import compare

pytestmark = pytest.mark.gpu


def test_a_bounded_wait_that_runs_out_returns_a_timeout_status():
    """Every wait in the kernels gives up after a cycle limit, raises the CTA's abort flag and lets the launch end
    with VPP_DEV_TIMEOUT.  The hook runs that primitive on a barrier nobody arrives at (no copy or MMA in flight)."""
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    api.vpp_test_bounded_wait(status, 200_000)            # ~0.1 ms of SM clocks
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    assert int(status.item()) == 3                        # VPP_DEV_TIMEOUT
    assert dt < 0.5, "the wait must end by itself within milliseconds (took %.3f s)" % dt
    # the context is intact: an ordinary launch right after it succeeds
    prob = W.make_problem(31, [300], [200], 4, 2, 128, 128, block_size=64).to("cuda")
    runner = api.ChunkAttn(prob)
    out, lse = runner.run()
    torch.cuda.synchronize()
    assert int(runner.status.item()) == 0
    compare(out, lse, prob.to("cpu"), oracle.all_rows(prob.chunk_len.cpu().numpy(), 4), "after the timed-out wait")


@pytest.mark.parametrize("mla", [False, True])
def test_a_repeated_call_encodes_no_tensor_map(mla):
    if mla:
        prob = W.make_problem(32, [200], [130], 16, 1, 576, 512, block_size=64, std=0.5, v_aliases_k=True).to("cuda")
    else:
        prob = W.make_problem(33, [500, 0], [300, 1], 8, 2, 128, 128, block_size=128).to("cuda")
    runner = api.ChunkAttn(prob)
    runner.run()
    l0, e0 = api.vpp_tensor_map_cache_stats()
    out1 = runner.out.clone()
    for _ in range(3):
        runner.run()
    torch.cuda.synchronize()
    l1, e1 = api.vpp_tensor_map_cache_stats()
    assert l1 > l0 and e1 == e0, "a call with the same buffers and shapes must find every map in the cache"
    assert torch.equal(out1, runner.out)
    # other buffers of the same shape: new maps, and still the right result
    other = api.ChunkAttn(prob)
    out2, lse2 = other.run()
    torch.cuda.synchronize()
    l2, e2 = api.vpp_tensor_map_cache_stats()
    assert e2 >= e1
    compare(out2, lse2, prob.to("cpu"), oracle.all_rows(prob.chunk_len.cpu().numpy(), prob.num_q_heads), "cached maps")


def _partials(prob, ranges):
    runner = api.ChunkAttn(prob, num_kv_splits=1)
    T, Hq, Dv = prob.total_q, prob.num_q_heads, prob.head_dim_v
    o_parts = torch.full((len(ranges), T, Hq, Dv), float("nan"), dtype=torch.float32, device="cuda")
    lse_parts = torch.full((len(ranges), T, Hq), float("nan"), dtype=torch.float32, device="cuda")
    for s, (b, e) in enumerate(ranges):
        api.vpp_chunk_attn_partial_fwd(runner.args, b, e, o_parts[s], lse_parts[s])
        torch.cuda.synchronize()
        assert int(runner.status.item()) == 0
    return runner, o_parts, lse_parts


@pytest.mark.parametrize("case", ["gqa", "gqa_decode", "mla", "mha"])
def test_key_range_partials_merge_to_the_unsplit_result(case):
    """Two (three) key ranges that tile the cache, one partial launch each, merged by vpp_lse_merge: equal to the
    oracle's unsplit attention, every element -- the KV-range shard of a context-parallel prefix on one GPU."""
    if case == "gqa":
        prob = W.make_problem(41, [1000, 384], [300, 200], 8, 2, 128, 128, block_size=64)
        ranges = [(0, 256), (256, 384), (384, 1 << 30)]
    elif case == "gqa_decode":
        prob = W.make_problem(42, [900, 700, 640], [1, 1, 130], 16, 2, 128, 128, block_size=128)
        ranges = [(0, 512), (512, 1 << 30)]
    elif case == "mla":
        prob = W.make_problem(43, [520, 300], [200, 1], 32, 1, 576, 512, block_size=64, std=0.5, v_aliases_k=True)
        ranges = [(0, 256), (256, 1 << 30)]
    else:
        prob = W.make_problem(44, [400], [260], 3, 3, 128, 128, block_size=32)
        ranges = [(0, 128), (128, 384), (384, 1 << 30)]
    gpu = prob.to("cuda")
    runner, o_parts, lse_parts = _partials(gpu, ranges)
    assert torch.isfinite(o_parts).all() and torch.isfinite(lse_parts).all()      # every row sees a key in every range
    out = torch.full((gpu.total_q, gpu.num_q_heads, gpu.head_dim_v), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((gpu.total_q, gpu.num_q_heads), float("nan"), dtype=torch.float32, device="cuda")
    api.vpp_lse_merge(o_parts, lse_parts, out, lse)
    torch.cuda.synchronize()
    rows = oracle.all_rows(prob.chunk_len.numpy(), prob.num_q_heads)
    print(compare(out, lse, prob, rows, "partials " + case))
    # each partial by itself is the oracle's attention over that key range (kv_lo / kv_hi of the oracle)
    b, e = ranges[0]
    ref_o, ref_l = oracle.ref_chunk_attn_rows(
        prob.q, prob.k_cache, prob.v_cache, prob.k_cache.stride()[:3], prob.v_cache.stride()[:3],
        prob.block_table.numpy(), prob.block_size, prob.prefix_len.numpy(), prob.chunk_len.numpy(), prob.num_q_heads,
        prob.num_kv_heads, prob.head_dim_qk, prob.head_dim_v, prob.scale, rows, kv_lo=b, kv_hi=e)
    got = o_parts[0].cpu().numpy().astype(np.float64).reshape(ref_o.shape)
    assert np.abs(got - ref_o).max() <= 1e-2
    got_l = lse_parts[0].cpu().numpy().astype(np.float64).reshape(ref_l.shape)
    assert (np.abs(got_l - ref_l) <= 1e-5 * np.maximum(1.0, np.abs(ref_l))).all()


def test_a_key_range_beyond_a_request_prefix_is_refused_on_the_device():
    prob = W.make_problem(45, [100], [300], 4, 2, 128, 128, block_size=64).to("cuda")
    runner = api.ChunkAttn(prob, num_kv_splits=1)
    o = torch.full((300, 4, 128), 7.0, dtype=torch.float32, device="cuda")
    l = torch.full((300, 4), 7.0, dtype=torch.float32, device="cuda")
    api.vpp_chunk_attn_partial_fwd(runner.args, 128, 1 << 30, o, l)       # rows 0..27 would see no key at all
    torch.cuda.synchronize()
    assert int(runner.status.item()) == 1                                 # VPP_DEV_BAD_LENGTHS
    assert (o == 7.0).all() and (l == 7.0).all()                          # nothing written


@pytest.mark.parametrize("world", [2, 4])
@pytest.mark.parametrize("mla", [False, True])
def test_context_parallel_ranks_emulated_on_one_gpu(world, mla):
    """The KV-range split of dist.kv_ranges with the library as every rank's kernel: rank r's launch sees only its range of
    the cache, the partials are stacked as an all-gather would stack them and merged.  (One GPU: the ranks run in turn.)"""
    from paper_2608_26523_b200 import dist as D
    if mla:
        prob = W.make_problem(51, [3000], [450], 16, 1, 576, 512, block_size=64, std=0.5, v_aliases_k=True)
    else:
        prob = W.make_problem(52, [5000], [700], 8, 2, 128, 128, block_size=128)
    P, C = int(prob.prefix_len[0]), int(prob.chunk_len[0])
    ranges = [(lo, hi) for lo, hi in D.kv_ranges(P + C, world, prefix_len=P) if hi > lo]
    assert len(ranges) == world
    gpu = prob.to("cuda")
    runner, o_parts, lse_parts = _partials(gpu, ranges)
    out = torch.empty((gpu.total_q, gpu.num_q_heads, gpu.head_dim_v), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((gpu.total_q, gpu.num_q_heads), dtype=torch.float32, device="cuda")
    api.vpp_lse_merge(o_parts, lse_parts, out, lse)
    torch.cuda.synchronize()
    rows = oracle.all_rows(prob.chunk_len.numpy(), prob.num_q_heads)
    print(compare(out, lse, prob, rows, "context parallel, %d ranks" % world))
