"""GPU integration: append then attend through the C ABI, and CUDA-graph capture of one chunk step."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_26523_b200 import api, workloads as W
from parity import compare

pytestmark = pytest.mark.gpu


def test_append_then_attend_matches_the_oracle():
    """The chunk's K/V rows are cut out of a complete cache, the slots poisoned, vpp_kv_append writes them back and
    vpp_chunk_attn_fwd attends over the result: same output as the oracle on the complete cache."""
    prob_cpu = W.make_problem(4100, [700, 0, 131], [300, 129, 1], 8, 2, 128, 128, block_size=16, std=0.7)
    prob = prob_cpu.to("cuda")
    bs = 16
    rows_k, rows_v = [], []
    for r in range(3):
        P, C = int(prob_cpu.prefix_len[r]), int(prob_cpu.chunk_len[r])
        for pos in range(P, P + C):
            blk, slot = int(prob_cpu.block_table[r, pos // bs]), pos % bs
            rows_k.append(prob.k_cache[blk, slot].clone())
            rows_v.append(prob.v_cache[blk, slot].clone())
            prob.k_cache[blk, slot] = float("nan")
            prob.v_cache[blk, slot] = float("nan")
    k_new, v_new = torch.stack(rows_k), torch.stack(rows_v)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.vpp_kv_append(k_new, v_new, prob.k_cache, prob.v_cache, prob.block_table, prob.prefix_len, prob.chunk_len, bs,
                      prob.max_seq_len, status=status)
    runner = api.ChunkAttn(prob)
    out, lse = runner.run()
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and int(runner.status.item()) == 0
    rows = oracle.all_rows(prob_cpu.chunk_len.numpy(), prob_cpu.num_q_heads)
    print(compare(out, lse, prob_cpu, rows, "append + attend"))


@pytest.mark.parametrize("splits", [0, 3])
def test_one_chunk_step_replays_from_a_cuda_graph(splits):
    """Work decomposition + attention (+ merge) enqueue only stream work, so a call can be captured once and replayed
    with new contents in the same buffers."""
    prob = W.make_problem(4200, [500, 64], [200, 1], 4, 2, 128, 128, block_size=16, std=0.7).to("cuda")
    runner = api.ChunkAttn(prob, num_kv_splits=splits)
    runner.run()                                  # first call outside capture (module / attribute set-up)
    torch.cuda.synchronize()
    eager = runner.out.clone()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        side.wait_stream(torch.cuda.current_stream())
        graph.capture_begin()
        runner.run(side.cuda_stream)
        graph.capture_end()
    runner.out.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(runner.out.view(torch.int16), eager.view(torch.int16))
    # new queries in the same buffer: the replay recomputes
    prob.q.mul_(-1.0)
    graph.replay()
    torch.cuda.synchronize()
    runner2_out = runner.out.clone()
    runner.run()
    torch.cuda.synchronize()
    assert torch.equal(runner.out.view(torch.int16), runner2_out.view(torch.int16))
    assert not torch.equal(runner2_out.view(torch.int16), eager.view(torch.int16))


def _host_side(prob_cpu, prob, pipe):
    """Pinned host copies of what vpp_chunk_attn_host_fwd brings in (q and the chunk's own K/V rows, token-major), with
    those rows poisoned on the device beforehand, and pinned result buffers."""
    aliased = prob_cpu.v_cache.data_ptr() == prob_cpu.k_cache.data_ptr()
    q_host = prob_cpu.q.clone().pin_memory()
    k_new = pipe.chunk_rows(prob_cpu.k_cache).contiguous().pin_memory()
    v_new = None if aliased else pipe.chunk_rows(prob_cpu.v_cache).contiguous().pin_memory()
    pos = torch.arange(pipe.P, pipe.P + pipe.C)
    blk = prob_cpu.block_table[0, (pos // prob_cpu.block_size).long()].long().cuda()
    slot = (pos % prob_cpu.block_size).long().cuda()
    prob.k_cache[blk, slot] = float("nan")
    if not aliased:
        prob.v_cache[blk, slot] = float("nan")
    C = pipe.C
    out_host = torch.full((C, prob_cpu.num_q_heads, prob_cpu.head_dim_v), float("nan"), dtype=torch.bfloat16).pin_memory()
    lse_host = torch.full((C, prob_cpu.num_q_heads), float("nan"), dtype=torch.float32).pin_memory()
    return q_host, k_new, v_new, out_host, lse_host


def test_host_entry_point_matches_the_oracle():
    """vpp_chunk_attn_host_fwd: a chunk streamed from pinned host memory in four given slices (copies overlapping
    append + attention) gives the oracle's rows, and the chunk's K/V rows end up in the cache bit for bit."""
    prob_cpu = W.make_problem(4300, [256], [512], 8, 2, 128, 128, block_size=64, std=0.7)
    prob = prob_cpu.to("cuda")
    pipe = api.HostChunkPipeline(prob, slices=[128, 64, 192, 128])
    assert pipe.slices == [128, 64, 192, 128]
    q_host, k_new, v_new, out_host, lse_host = _host_side(prob_cpu, prob, pipe)
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    for _ in range(2):                       # a second step reuses every buffer, stream and event
        out_host.fill_(float("nan"))
        pipe.run(q_host, k_new, v_new, out_host, lse_host, stream)
        stream.synchronize()
        assert int(pipe.status.item()) == 0
        rows = oracle.all_rows(prob_cpu.chunk_len.numpy(), prob_cpu.num_q_heads)
        print(compare(out_host, lse_host, prob_cpu, rows, "host entry point"))
    live = torch.zeros(prob_cpu.k_cache.shape[:2], dtype=torch.bool)
    for pos in range(256 + 512):
        live[int(prob_cpu.block_table[0, pos // 64]), pos % 64] = True
    assert torch.equal(prob.k_cache.cpu()[live].view(torch.int16), prob_cpu.k_cache[live].view(torch.int16))
    assert torch.equal(prob.v_cache.cpu()[live].view(torch.int16), prob_cpu.v_cache[live].view(torch.int16))


@pytest.mark.parametrize("case", ["mla", "ragged", "no_lse", "unaligned_prefix"])
def test_host_entry_point_variants(case):
    """The latent (MLA) cache whose values alias the keys, a ragged chunk (one slice), a call without lse, and a prefix
    that is not a multiple of the page size (the rows are appended by the kernel, not copied page-wise)."""
    if case == "mla":
        prob_cpu = W.make_problem(4310, [320], [384], 16, 1, 576, 512, block_size=64, std=0.5, v_aliases_k=True)
    elif case == "ragged":
        prob_cpu = W.make_problem(4311, [100], [333], 8, 2, 128, 128, block_size=32, std=0.7)
    elif case == "unaligned_prefix":
        prob_cpu = W.make_problem(4313, [77], [512], 6, 2, 128, 128, block_size=16, std=0.7)
    else:
        prob_cpu = W.make_problem(4312, [128], [384], 4, 4, 128, 128, block_size=128, std=0.7)
    prob = prob_cpu.to("cuda")
    pipe = api.HostChunkPipeline(prob, want_lse=(case != "no_lse"))
    assert sum(pipe.slices) == int(prob_cpu.chunk_len[0]) and len(pipe.slices) == (1 if case == "ragged" else 3)
    q_host, k_new, v_new, out_host, lse_host = _host_side(prob_cpu, prob, pipe)
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    pipe.run(q_host, k_new, v_new, out_host, None if case == "no_lse" else lse_host, stream)
    stream.synchronize()
    assert int(pipe.status.item()) == 0
    rows = oracle.all_rows(prob_cpu.chunk_len.numpy(), prob_cpu.num_q_heads)
    print(case, pipe.slices, compare(out_host, None if case == "no_lse" else lse_host, prob_cpu, rows, "host entry point, " + case))


def test_host_entry_point_in_a_cuda_graph():
    """The whole chunk step from host memory (copies in, append, attention, copies out, three streams) captured once in a
    CUDA graph and replayed with new contents in the same pinned buffers."""
    prob_cpu = W.make_problem(4330, [256], [512], 8, 2, 128, 128, block_size=64, std=0.7)
    prob = prob_cpu.to("cuda")
    pipe = api.HostChunkPipeline(prob)
    q_host, k_new, v_new, out_host, lse_host = _host_side(prob_cpu, prob, pipe)
    warm = torch.cuda.Stream()
    warm.wait_stream(torch.cuda.current_stream())
    pipe.run(q_host, k_new, v_new, out_host, lse_host, warm)       # first call on the device: creates the copy streams
    warm.synchronize()
    eager = out_host.clone()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        side.wait_stream(torch.cuda.current_stream())
        graph.capture_begin()
        pipe.run(q_host, k_new, v_new, out_host, lse_host, side)
        graph.capture_end()
    out_host.fill_(float("nan"))
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(out_host.view(torch.int16), eager.view(torch.int16))
    # new queries in the same pinned buffer: the replay reads them
    q_host.mul_(-1.0)
    graph.replay()
    torch.cuda.synchronize()
    flipped = prob_cpu.to("cpu")
    flipped.q = -prob_cpu.q
    rows = oracle.all_rows(prob_cpu.chunk_len.numpy(), prob_cpu.num_q_heads)
    print(compare(out_host, lse_host, flipped, rows, "host entry point, graph replay"))


def test_host_entry_point_refuses_bad_arguments():
    prob = W.make_problem(4320, [256], [512], 8, 2, 128, 128, block_size=64).to("cuda")
    with pytest.raises(api.VppError):
        api.HostChunkPipeline(prob, slices=[128, 128])              # does not add up to the chunk
    pipe = api.HostChunkPipeline(prob)
    pipe.hargs.dev.workspace_bytes = 1024
    q = torch.zeros((512, 8, 128), dtype=torch.bfloat16).pin_memory()
    kv = torch.zeros((512, 2, 128), dtype=torch.bfloat16).pin_memory()
    with pytest.raises(api.VppError) as e:
        pipe.run(q, kv, kv, q.clone().pin_memory(), None)
    assert e.value.status == api.VPP_ERR_WORKSPACE


def test_sparse_attention_after_append_and_from_a_cuda_graph():
    """Latent rows of the chunk appended with vpp_kv_append (keys only: the values alias them), then index-selected
    attention over the cache, captured once in a CUDA graph and replayed; checked against the sparse oracle."""
    from oracle.ref_sparse_attn import ref_sparse_chunk_attn
    prefix, chunk = [300, 64], [90, 3]
    prob_cpu = W.make_problem(4400, prefix, chunk, 128, 1, 576, 512, block_size=64, std=0.6, v_aliases_k=True)
    idx = W.make_sparse_indices(4401, prefix, chunk, 200, kind="clustered", group=16)
    prob = prob_cpu.to("cuda")
    rows = []
    for r in range(2):
        for pos in range(prefix[r], prefix[r] + chunk[r]):
            blk, slot = int(prob_cpu.block_table[r, pos // 64]), pos % 64
            rows.append(prob.k_cache[blk, slot].clone())
            prob.k_cache[blk, slot] = float("nan")
    k_new = torch.stack(rows)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.vpp_kv_append(k_new, None, prob.k_cache, prob.v_cache, prob.block_table, prob.prefix_len, prob.chunk_len, 64,
                      prob.max_seq_len, status=st)
    sp = api.SparseAttn(prob, torch.from_numpy(idx).cuda())
    sp.run()
    torch.cuda.synchronize()
    assert int(st.item()) == 0 and int(sp.status.item()) == 0
    eager = sp.out.clone()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        side.wait_stream(torch.cuda.current_stream())
        graph.capture_begin()
        sp.run(side.cuda_stream)
        graph.capture_end()
    sp.out.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(sp.out.view(torch.int16), eager.view(torch.int16))
    bits = lambda t: t.view(torch.int16).numpy().view(np.uint16)
    ref_o, ref_l = ref_sparse_chunk_attn(bits(prob_cpu.q), bits(prob_cpu.k_cache), idx, prob_cpu.block_table.numpy(), 64,
                                         prob_cpu.prefix_len.numpy(), prob_cpu.chunk_len.numpy(), 512, prob_cpu.scale)
    assert np.abs(sp.out.float().cpu().numpy() - ref_o).max() <= 1e-2
    got_l = sp.lse.cpu().numpy().astype(np.float64)
    both = np.isfinite(ref_l)
    assert (np.isfinite(got_l) == both).all()                 # tokens without a listed key: -inf on both sides
    assert (np.abs(got_l - ref_l)[both] <= 1e-5 * np.maximum(1.0, np.abs(ref_l[both]))).all()


def test_host_entry_point_at_benchmark_size_matches_the_oracle():
    """The end-to-end leg of bench.py at its real size: the cfg 2 chunk at prefix 65536 streamed from pinned host memory in
    the planned slices, compared with the oracle on one row of every (query tile, pair of q-heads) plus the edge rows."""
    from parity import sample_rows, tile_rows
    prob = W.cfg2(prefix=65536, device="cuda")
    prob_cpu = prob.to("cpu")
    pipe = api.HostChunkPipeline(prob)
    assert pipe.slices == [1152, 5888, 1152]
    q_host, k_new, v_new, out_host, lse_host = _host_side(prob_cpu, prob, pipe)
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    pipe.run(q_host, k_new, v_new, out_host, lse_host, stream)
    stream.synchronize()
    assert int(pipe.status.item()) == 0
    assert torch.isfinite(out_host.float()).all() and torch.isfinite(lse_host).all()
    rows = np.unique(np.concatenate([sample_rows(prob_cpu, n_random=64), tile_rows(prob_cpu, per="pair", seed=3)]), axis=0)
    print(compare(out_host, lse_host, prob_cpu, rows, "host entry point, cfg2 at 65536"))
