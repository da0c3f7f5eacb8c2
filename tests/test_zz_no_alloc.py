"""The allocation-free entry point (collected last on purpose).

vpp_chunk_attn_fwd_static serves callers that may not allocate device memory -- for instance a plugin
running inside a framework's memory-planned region, or a server that gave all device memory away at
start-up: they pass inputs and outputs, and the library's built-in scratch array replaces the
workspace.  The test calls it through the C ABI twice in a row on a launch that really uses scratch
(forced split-KV: work list, per-row split counts and fp32 partials) and compares both results with the
ordinary entry point's and with the CPU oracle (every element), checks that further calls leave the device's free memory
and torch's allocator untouched, then that an oversized launch is refused cleanly.
"""
import pytest
import torch

import oracle
from paper_2608_26523_b200 import api, workloads as W
from parity import compare

pytestmark = pytest.mark.gpu


def _launch(prob, static, num_kv_splits):
    runner = api.ChunkAttn(prob, num_kv_splits=num_kv_splits)
    runner.out.fill_(float("nan"))
    runner.lse.fill_(float("nan"))
    if static:
        runner.args.workspace = None           # the static variant must not need it
        runner.args.workspace_bytes = 0
        api.vpp_chunk_attn_fwd_static(runner.args)
    else:
        api.vpp_chunk_attn_fwd(runner.args)
    torch.cuda.synchronize()
    assert int(runner.status.item()) == 0
    return runner.out.float().clone(), runner.lse.clone()


def test_static_scratch_matches_workspace_entry_point_twice():
    prob_cpu = W.make_problem(9001, [900, 0, 260], [300, 140, 77], 8, 2, 128, 128, block_size=64)
    prob = prob_cpu.to("cuda")
    rows = oracle.all_rows(prob_cpu.chunk_len.numpy(), prob_cpu.num_q_heads)
    ref_out, ref_lse = _launch(prob, static=False, num_kv_splits=3)
    assert torch.isfinite(ref_out).all()
    for call in range(2):                                    # the second call finds the first one's leftovers
        out, lse = _launch(prob, static=True, num_kv_splits=3)
        # against the definition: every element, with the tolerances of the parity suite
        compare(out, lse, prob_cpu, rows, "static entry point, call %d" % call)
        # same kernels, same work list: the results agree to the tolerance of the parity tests (they are in
        # fact identical up to the order in which equal-cost work units were listed)
        assert (out - ref_out).abs().max().item() <= 1e-2, "call %d" % call
        assert ((lse - ref_lse).abs() <= 1e-5 * ref_lse.abs().clamp(min=1)).all(), "call %d" % call
    # a different launch in between must not disturb the next one
    other = W.make_problem(9002, [64], [200], 4, 2, 128, 128, block_size=None).to("cuda")
    _launch(other, static=True, num_kv_splits=0)
    out, lse = _launch(prob, static=True, num_kv_splits=3)
    assert (out - ref_out).abs().max().item() <= 1e-2


def test_static_entry_point_allocates_nothing_after_its_first_call():
    """The first call on a device resolves the scratch array's address (and may make the runtime load that part of the
    library); from then on a call that really uses the scratch (split-KV partials) must leave the device's free memory
    and torch's allocator exactly as they were."""
    prob = W.make_problem(9005, [700], [400], 8, 2, 128, 128, block_size=64).to("cuda")
    runner = api.ChunkAttn(prob, num_kv_splits=4)
    runner.args.workspace, runner.args.workspace_bytes = None, 0
    api.vpp_chunk_attn_fwd_static(runner.args)               # first call: set-up included
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for _ in range(3):
        api.vpp_chunk_attn_fwd_static(runner.args)
    torch.cuda.synchronize()
    assert int(runner.status.item()) == 0
    free1, _ = torch.cuda.mem_get_info()
    assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == (alloc0, reserved0)
    assert free1 == free0, "device free memory changed by %d bytes across static calls" % (free0 - free1)


def test_static_scratch_refuses_oversized_launch():
    limit = api.vpp_static_scratch_bytes()
    assert limit == 32 << 20
    # 16 splits x 4096 rows x 8 heads x 129 floats = 270 MB of partials: far beyond the built-in array
    prob = W.make_problem(9003, [0], [4096], 8, 2, 128, 128, block_size=128).to("cuda")
    runner = api.ChunkAttn(prob, num_kv_splits=16)
    assert api.vpp_chunk_attn_workspace_size(runner.args) > limit
    runner.out.fill_(5.0)
    with pytest.raises(api.VppError) as ei:
        api.vpp_chunk_attn_fwd_static(runner.args)
    assert ei.value.status == api.VPP_ERR_WORKSPACE
    torch.cuda.synchronize()
    assert (runner.out == 5.0).all()                         # nothing was enqueued


def test_static_scratch_drops_the_library_chosen_split_when_its_partials_do_not_fit():
    """8192 rows x 16 q-heads at a long prefix: left to itself the library splits this launch in two (3.46 waves of work
    items otherwise), which takes 135 MB of partials; the static entry point runs it unsplit instead of refusing."""
    prob = W.make_problem(9004, [16384], [8192], 16, 2, 128, 128, block_size=128).to("cuda")
    auto = api.ChunkAttn(prob, num_kv_splits=0)
    assert api.vpp_chunk_attn_workspace_size(auto.args) > api.vpp_static_scratch_bytes()
    ref_out, ref_lse = _launch(prob, static=False, num_kv_splits=1)
    out, lse = _launch(prob, static=True, num_kv_splits=0)
    assert (out - ref_out).abs().max().item() <= 1e-2
    assert ((lse - ref_lse).abs() <= 1e-5 * ref_lse.abs().clamp(min=1)).all()
