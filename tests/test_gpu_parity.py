"""GPU parity: the CUDA library, called through its C ABI, against the fp64 CPU oracle on the same
seeded inputs, element by element."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_26523_b200 import api, workloads as W
from parity import compare, run_gpu, sample_rows

pytestmark = pytest.mark.gpu


def full_check(prob_cpu, num_kv_splits=0, label=""):
    out, lse, runner = run_gpu(prob_cpu.to("cuda"), num_kv_splits)
    rows = oracle.all_rows(prob_cpu.chunk_len.numpy(), prob_cpu.num_q_heads)
    return compare(out, lse, prob_cpu, rows, label), runner


@pytest.mark.parametrize("k", [0, 1, 2, 3])
def test_cfg1_every_element(k):
    s, _ = full_check(W.cfg1(k), label="cfg1 chunk %d" % k)
    print(s)


@pytest.mark.parametrize("splits", [1, 2, 3, 5])
def test_cfg1_forced_splits(splits):
    s, _ = full_check(W.cfg1(3), num_kv_splits=splits, label="cfg1 chunk 3 S=%d" % splits)
    print(s)


CASES = [
    # prefix_lens, chunk_lens, hq, hkv, block_size
    ([0], [1], 2, 1, None),                       # one token, one key
    ([0], [129], 4, 2, 128),                      # one row into a second query tile
    ([127], [2], 2, 2, 64),                       # straddles a KV tile edge
    ([300], [77], 4, 1, 16),                      # unaligned everything, small pages
    ([1000, 0, 17, 511], [200, 0, 300, 129], 8, 2, 32),   # varlen batch with an empty request
    ([4095], [257], 4, 4, 256),                   # pages larger than a KV tile, MHA
    ([513], [640], 4, 2, None),                   # contiguous cache, several tiles
    ([0, 0, 0], [5, 130, 1], 2, 1, 128),
]


@pytest.mark.parametrize("case", range(len(CASES)))
@pytest.mark.parametrize("splits", [0, 1, 3])
def test_adversarial_shapes(case, splits):
    P, C, hq, hkv, bs = CASES[case]
    prob = W.make_problem(1000 + case, P, C, hq, hkv, 128, 128, block_size=bs)   # NaN tails / unused blocks
    s, _ = full_check(prob, num_kv_splits=splits, label="case %d S=%d" % (case, splits))
    print(s)


MLA_CASES = [
    # prefix_lens, chunk_lens, hq, block_size      (absorbed MLA: Dqk 576, Dv 512, one shared latent kv-head)
    ([0], [1], 2, None),
    ([0], [129], 4, 64),
    ([63], [2], 2, 64),
    ([300], [77], 4, 16),
    ([1000, 0, 17, 511], [200, 0, 300, 129], 8, 32),
    ([4095], [257], 4, 256),
    ([513], [640], 4, None),
]


@pytest.mark.parametrize("case", range(len(MLA_CASES)))
@pytest.mark.parametrize("splits", [0, 1, 3])
def test_mla_adversarial_shapes(case, splits):
    P, C, hq, bs = MLA_CASES[case]
    prob = W.make_problem(2000 + case, P, C, hq, 1, 576, 512, block_size=bs, std=0.5, scale=1.0 / 192 ** 0.5,
                          v_aliases_k=True)
    s, _ = full_check(prob, num_kv_splits=splits, label="mla case %d S=%d" % (case, splits))
    print(s)


def _ramp_scores(prob, step):
    """Make the scores grow along the sequence: key p gets its last feature = p * step (for absorbed MLA that
    feature is not part of the values), every query the same feature = 1, so the
    running row maximum rises by more than the rescale threshold at every KV tile (the lazy rescale of O fires
    on each tile instead of almost never)."""
    bs = prob.k_cache.shape[1]
    for r in range(len(prob.prefix_len)):
        n = int(prob.prefix_len[r] + prob.chunk_len[r])
        pos = torch.arange(n)
        if prob.block_table is None:
            prob.k_cache[r, pos, :, -1] = (pos.float() * step).to(prob.k_cache.dtype)[:, None]
        else:
            blk = prob.block_table[r, pos // bs].long()
            prob.k_cache[blk, pos % bs, :, -1] = (pos.float() * step).to(prob.k_cache.dtype)[:, None]
    prob.q[:, :, -1] = 1.0


@pytest.mark.parametrize("family", ["gqa", "mla"])
@pytest.mark.parametrize("splits", [0, 2])
def test_running_maximum_grows_every_tile(family, splits):
    if family == "gqa":
        prob = W.make_problem(2200, [2000, 700], [300, 129], 4, 2, 128, 128, block_size=16, std=0.5)
    else:
        prob = W.make_problem(2201, [2000, 700], [300, 129], 4, 1, 576, 512, block_size=64, std=0.5,
                              scale=1.0 / 192 ** 0.5, v_aliases_k=True)
    _ramp_scores(prob, 1.0)   # scale * 128 keys * 1.0 is about 9-11 nats per tile, well above the 2^8 threshold
    s, _ = full_check(prob, num_kv_splits=splits, label="%s ramp S=%d" % (family, splits))
    print(s)


@pytest.mark.parametrize("hq,hkv", [(64, 4), (16, 8), (8, 1)])
@pytest.mark.parametrize("splits", [0, 1, 4])
def test_decode_rows_mixed_with_prefill_chunks(hq, hkv, splits):
    """Single-token requests (decode steps) batched with prefill chunks: the kernel packs the q-heads of a kv-head
    into one tile for them.  Every element against the oracle."""
    prefix = [700, 0, 1333, 128, 2047, 5, 300, 64, 1000]
    chunk = [1, 1, 1, 1, 1, 1, 200, 129, 1]
    prob = W.make_problem(2300 + hq, prefix, chunk, hq, hkv, 128, 128, block_size=16, std=0.7)
    s, _ = full_check(prob, num_kv_splits=splits, label="decode mix Hq=%d Hkv=%d S=%d" % (hq, hkv, splits))
    print(s)


@pytest.mark.parametrize("hq", [128, 16, 72])
@pytest.mark.parametrize("splits", [0, 1, 4])
def test_mla_decode_rows_mixed_with_prefill_chunks(hq, splits):
    """Absorbed MLA: single-token requests next to prefill chunks (the q-heads become the rows of the tile)."""
    prefix = [700, 0, 1333, 128, 2047, 5, 300, 64]
    chunk = [1, 1, 1, 1, 1, 1, 130, 1]
    prob = W.make_problem(2400 + hq, prefix, chunk, hq, 1, 576, 512, block_size=64, std=0.5, scale=1.0 / 192 ** 0.5,
                          v_aliases_k=True)
    s, _ = full_check(prob, num_kv_splits=splits, label="mla decode mix Hq=%d S=%d" % (hq, splits))
    print(s)


def test_mla_requires_aliased_values():
    prob = W.make_problem(2100, [10], [20], 2, 1, 576, 512, block_size=16, std=0.5, v_aliases_k=True).to("cuda")
    runner = api.ChunkAttn(prob)
    other = torch.zeros_like(prob.k_cache)
    runner.args.v_cache = other.data_ptr()
    with pytest.raises(api.VppError) as ei:
        runner.run()
    assert ei.value.status == api.VPP_ERR_UNSUPPORTED


def test_outputs_outside_the_launch_are_untouched():
    """Canary rows around out / lse keep their value."""
    prob = W.make_problem(77, [40], [100], 4, 2, 128, 128, block_size=64).to("cuda")
    big_out = torch.full((102, 4, 128), 7.0, dtype=torch.bfloat16, device="cuda")
    big_lse = torch.full((102, 4), 7.0, dtype=torch.float32, device="cuda")
    runner = api.ChunkAttn(prob)
    runner.args.out = big_out[1:].data_ptr()
    runner.args.lse = big_lse[1:].data_ptr()
    runner.run()
    torch.cuda.synchronize()
    assert (big_out[0] == 7).all() and (big_out[101] == 7).all()
    assert (big_lse[0] == 7).all() and (big_lse[101] == 7).all()
    assert torch.isfinite(big_out[1:101].float()).all()


def test_lse_merge_against_oracle():
    g = torch.Generator().manual_seed(5)
    S, T, Hq, Dv = 5, 37, 3, 128
    o = torch.randn(S, T, Hq, Dv, generator=g)
    l = torch.randn(S, T, Hq, generator=g) * 4
    l[2, 5] = float("-inf")
    l[:, 7, 1] = float("-inf")
    out = torch.empty(T, Hq, Dv, dtype=torch.bfloat16, device="cuda")
    lse = torch.empty(T, Hq, device="cuda")
    api.vpp_lse_merge(o.cuda(), l.cuda(), out, lse)
    torch.cuda.synchronize()
    ro, rl = oracle.ref_lse_merge(o.reshape(S, T * Hq, Dv).double().numpy(), l.reshape(S, T * Hq).double().numpy())
    got = out.float().cpu().numpy().reshape(T * Hq, Dv)
    assert np.abs(got - ro).max() <= 2.0 ** -8 * np.abs(ro).max() + 1e-6
    gl = lse.cpu().numpy().reshape(-1)
    fin = np.isfinite(rl)
    assert np.array_equal(np.isneginf(gl), ~fin)
    assert (np.abs(gl[fin] - rl[fin]) <= 1e-5 * np.maximum(1, np.abs(rl[fin]))).all()


def test_bad_lengths_set_device_status_and_write_nothing():
    prob = W.make_problem(78, [10], [20], 2, 1, 128, 128, block_size=16).to("cuda")
    runner = api.ChunkAttn(prob)
    runner.out.fill_(3.0)
    bad = prob.prefix_len.clone(); bad[0] = 10 ** 6            # beyond max_seq_len
    runner.args.prefix_len = bad.data_ptr()
    runner.run()
    torch.cuda.synchronize()
    assert int(runner.status.item()) == 1
    assert (runner.out == 3.0).all()


def test_many_short_requests_with_ragged_single_tiles():
    """Hundreds of work items of one ragged KV tile each: consecutive fix-ups of value rows past the end of a sequence,
    item boundaries at every tile."""
    rng = np.random.default_rng(31)
    n_req = 150
    prefix = [int(rng.integers(0, 60)) for _ in range(n_req)]
    chunk = [int(rng.integers(2, 40)) for _ in range(n_req)]
    prob_cpu = W.make_problem(6100, prefix, chunk, 8, 2, 128, 128, block_size=128, std=0.8)
    out, lse, _ = run_gpu(prob_cpu.to("cuda"))
    rows = oracle.all_rows(prob_cpu.chunk_len.numpy(), prob_cpu.num_q_heads)
    print(compare(out, lse, prob_cpu, rows, "short ragged items"))


@pytest.mark.parametrize("layout", ["head_major", "padded_rows", "k_and_v_interleaved"])
@pytest.mark.parametrize("block_size", [128, 32])
def test_cache_layouts_given_by_strides(layout, block_size):
    """The caches are described by strides, not by a fixed layout: pages stored head-major ([block][kv-head][slot][d]), rows
    padded to a larger token stride, and K and V interleaved in one allocation all give the same rows as the oracle (which
    reads the logical tensors)."""
    prob_cpu = W.make_problem(9300 + block_size, [300, 0, 77], [260, 200, 3], 8, 2, 128, 128, block_size=block_size, std=0.8)
    prob = prob_cpu.to("cuda")
    k, v = prob.k_cache, prob.v_cache                      # logical [blocks, slots, kv-heads, d]
    nb, bs, hk, d = k.shape
    if layout == "head_major":
        k2 = k.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
        v2 = v.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    elif layout == "padded_rows":
        store_k = torch.full((nb, bs, hk + 1, d), float("nan"), dtype=k.dtype, device=k.device)
        store_v = torch.full((nb, bs, hk + 1, d), float("nan"), dtype=k.dtype, device=k.device)
        store_k[:, :, :hk] = k
        store_v[:, :, :hk] = v
        k2, v2 = store_k[:, :, :hk], store_v[:, :, :hk]
    else:
        store = torch.empty((nb, bs, hk, 2, d), dtype=k.dtype, device=k.device)
        store[:, :, :, 0] = k
        store[:, :, :, 1] = v
        k2, v2 = store[:, :, :, 0], store[:, :, :, 1]
    assert torch.equal(k2.view(torch.int16), k.view(torch.int16)) and k2.stride() != k.stride()
    prob.k_cache, prob.v_cache = k2, v2
    out, lse, _ = run_gpu(prob, 0)
    rows = oracle.all_rows(prob_cpu.chunk_len.numpy(), prob_cpu.num_q_heads)
    print(layout, compare(out, lse, prob_cpu, rows, "layout " + layout))


@pytest.mark.parametrize("block_size", [64, 16])
def test_mla_latent_rows_with_a_padded_stride(block_size):
    """The absorbed-MLA cache with its 576-feature rows 640 elements apart (values still alias the first 512 features of
    the keys): both MLA kernels (pages of 64 tokens and smaller ones) read through the strides."""
    prob_cpu = W.make_problem(9400 + block_size, [333, 0], [200, 140], 16, 1, 576, 512, block_size=block_size, std=0.5,
                              v_aliases_k=True)
    prob = prob_cpu.to("cuda")
    nb, bs, hk, d = prob.k_cache.shape
    store = torch.full((nb, bs, hk, 640), float("nan"), dtype=torch.bfloat16, device="cuda")
    store[..., :576] = prob.k_cache
    prob.k_cache = store[..., :576]
    prob.v_cache = store[..., :512]
    assert prob.k_cache.stride(1) == 640 and prob.v_cache.data_ptr() == prob.k_cache.data_ptr()
    out, lse, _ = run_gpu(prob, 0)
    rows = oracle.all_rows(prob_cpu.chunk_len.numpy(), prob_cpu.num_q_heads)
    print(compare(out, lse, prob_cpu, rows, "MLA padded rows, pages of %d" % block_size))
