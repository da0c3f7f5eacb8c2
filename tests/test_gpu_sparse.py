"""GPU parity of index-selected (sparse) attention over the latent cache against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle.ref_sparse_attn import ref_sparse_chunk_attn
from paper_2608_26523_b200 import api, workloads as W
from parity import ABS_TOL, LSE_TOL, REL_L2_TOL

pytestmark = pytest.mark.gpu


def _bits(t):
    return t.view(torch.int16).numpy().view(np.uint16)


def _problem(seed, prefix, chunk, hq, bs=64, std=0.6):
    return W.make_problem(seed, list(prefix), list(chunk), hq, 1, 576, 512, block_size=bs, std=std, v_aliases_k=True)


def _check(prob_cpu, idx, tokens=None, label=""):
    prob = prob_cpu.to("cuda")
    runner = api.SparseAttn(prob, torch.from_numpy(idx).cuda())
    runner.out.fill_(float("nan"))
    runner.lse.fill_(float("nan"))
    out, lse = runner.run()
    torch.cuda.synchronize()
    assert int(runner.status.item()) == 0
    bt = None if prob_cpu.block_table is None else prob_cpu.block_table.numpy()
    ref_o, ref_l = ref_sparse_chunk_attn(_bits(prob_cpu.q), _bits(prob_cpu.k_cache), idx, bt, prob_cpu.block_size,
                                         prob_cpu.prefix_len.numpy(), prob_cpu.chunk_len.numpy(), 512, prob_cpu.scale, tokens)
    sel = slice(None) if tokens is None else torch.as_tensor(tokens)
    got_o = out.float().cpu()[sel].numpy().astype(np.float64)
    got_l = lse.cpu()[sel].numpy().astype(np.float64)
    assert np.isfinite(got_o).all(), label
    err = np.abs(got_o - ref_o)
    assert (err <= np.maximum(ABS_TOL, 2.0 ** -8 * np.abs(ref_o))).all(), "%s: max abs err %.4g" % (label, err.max())
    rel = np.linalg.norm(got_o - ref_o) / max(np.linalg.norm(ref_o), 1e-30)
    assert rel <= REL_L2_TOL, "%s: rel L2 %.4g" % (label, rel)
    fin = np.isfinite(ref_l)
    assert np.array_equal(np.isneginf(got_l), ~fin), label
    lerr = np.abs(got_l[fin] - ref_l[fin]) / np.maximum(1.0, np.abs(ref_l[fin]))
    assert lerr.size == 0 or lerr.max() <= LSE_TOL, "%s: lse rel err %.4g" % (label, lerr.max())
    return dict(max_abs=float(err.max()), rel_l2=float(rel))


@pytest.mark.parametrize("hq", [128, 64, 16, 80])
@pytest.mark.parametrize("kind", ["scattered", "clustered"])
def test_every_token_against_the_oracle(hq, kind):
    # two requests, pages of 64 tokens shuffled in the pool; lists of 256 = two KV tiles; the first request starts at
    # position 0, so its early tokens list fewer than topk positions and pad with -1
    prefix, chunk = [0, 1500], [150, 83]
    p = _problem(5100 + hq, prefix, chunk, hq)
    idx = W.make_sparse_indices(61, prefix, chunk, 256, kind=kind, group=32)
    print(_check(p, idx, label="hq%d %s" % (hq, kind)))


@pytest.mark.parametrize("topk", [1, 100, 128, 333, 2048])
def test_list_lengths_with_ragged_last_tile(topk):
    prefix, chunk = [4000], [37]
    p = _problem(5200 + topk, prefix, chunk, 128)
    idx = W.make_sparse_indices(62 + topk, prefix, chunk, topk)
    print(_check(p, idx, label="topk%d" % topk))


def test_skipped_entries_duplicates_and_tokens_without_any_entry():
    prefix, chunk = [700, 0], [70, 40]
    p = _problem(5300, prefix, chunk, 128, bs=16)
    rng = np.random.default_rng(8)
    idx = W.make_sparse_indices(63, prefix, chunk, 192)
    pos = np.concatenate([700 + np.arange(70), np.arange(40)])
    for t in range(idx.shape[0]):
        k = rng.integers(0, 192, size=40)
        idx[t, k[:10]] = pos[t] + 1 + rng.integers(0, 50, size=10)     # the future
        idx[t, k[10:20]] = -rng.integers(1, 1000, size=10)             # negative
        idx[t, k[20:30]] = 2 ** 31 - 1 - rng.integers(0, 5, size=10)   # far outside the cache
        idx[t, k[30:40]] = rng.integers(0, pos[t] + 1, size=10)        # duplicates of earlier positions
    idx[5] = -1                                                        # nothing listed
    idx[77] = pos[77] + 3                                              # only the future listed
    idx[9, :] = -1
    idx[9, 191] = 3                                                    # a single entry in the last slot
    print(_check(p, idx, label="skips"))


def test_contiguous_cache_and_wide_scores():
    prefix, chunk = [900, 300, 0], [33, 64, 5]
    p = W.make_problem(5400, prefix, chunk, 128, 1, 576, 512, block_size=None, std=0.7, scale=0.1, v_aliases_k=True)
    idx = W.make_sparse_indices(64, prefix, chunk, 384, kind="clustered", group=16)
    print(_check(p, idx, label="contiguous"))


def test_more_tokens_than_resident_pairs_and_empty_launch():
    prefix, chunk = [2048], [600]          # 600 tokens > 74 pairs: several tokens per pair, ragged last round
    p = _problem(5500, prefix, chunk, 128)
    idx = W.make_sparse_indices(65, prefix, chunk, 512, kind="clustered")
    tokens = sorted(set(np.random.default_rng(1).integers(0, 600, size=48).tolist()) | {0, 73, 74, 147, 148, 599})
    print(_check(p, idx, tokens=tokens, label="many tokens"))
    # zero tokens: nothing is launched, status stays 0
    p0 = _problem(5501, [10], [0], 128).to("cuda")
    r0 = api.SparseAttn(p0, torch.zeros((0, 128), dtype=torch.int32, device="cuda"))
    r0.run()
    torch.cuda.synchronize()
    assert int(r0.status.item()) == 0


def test_bad_lengths_write_nothing():
    p = _problem(5600, [100], [20], 128).to("cuda")
    idx = torch.from_numpy(W.make_sparse_indices(66, [100], [20], 128)).cuda()
    runner = api.SparseAttn(p, idx)
    p.chunk_len.fill_(19)                  # does not add up to total_q
    runner.out.fill_(7.0)
    runner.run()
    torch.cuda.synchronize()
    assert int(runner.status.item()) == 1
    assert (runner.out == 7.0).all()


def test_benchmark_size_launch_on_sampled_tokens():
    """The launch bench.py times (cfg 3 cache, 8192-token chunk at prefix 65536, 2048 listed keys per token, both list
    kinds), checked on sampled tokens that the oracle computes one by one."""
    prob_cpu = W.cfg3(prefix=65536)
    rng = np.random.default_rng(17)
    tokens = sorted(set(rng.integers(0, 8192, size=20).tolist()) | {0, 1, 63, 64, 4095, 8191})
    for kind in ("clustered", "scattered"):
        idx = W.make_sparse_indices_strata(W.BASE_SEED + 401, [65536], [8192], 2048, kind=kind).numpy()
        print(kind, _check(prob_cpu, idx, tokens=tokens, label="bench size " + kind))


@pytest.mark.parametrize("seed", list(range(10)))
def test_seeded_random_shapes(seed):
    """Odd head counts, list lengths, page sizes and request mixes: the tile counts, ragged tiles and barrier phases
    they produce are not the ones the hand-picked cases have."""
    rng = np.random.default_rng(9000 + seed)
    hq = int(rng.choice([1, 3, 8, 17, 40, 64, 65, 100, 127, 128]))
    topk = int(rng.integers(1, 700))
    n_req = int(rng.integers(1, 5))
    prefix = [int(rng.integers(0, 3000)) for _ in range(n_req)]
    chunk = [int(rng.integers(0, 90)) for _ in range(n_req)]
    if sum(chunk) == 0:
        chunk[0] = 5
    bs = [None, 16, 32, 64, 128][int(rng.integers(0, 5))]
    p = W.make_problem(9100 + seed, prefix, chunk, hq, 1, 576, 512, block_size=bs, std=0.6, v_aliases_k=True)
    idx = W.make_sparse_indices(9200 + seed, prefix, chunk, topk, kind=["scattered", "clustered"][seed & 1], group=16)
    holes = rng.random(idx.shape) < 0.05                      # knock out 5 % of the entries
    idx[holes] = -1
    print(dict(hq=hq, topk=topk, prefix=prefix, chunk=chunk, bs=bs), _check(p, idx, label="random %d" % seed))


def test_lists_of_every_causal_position_reproduce_the_dense_kernel():
    """With every causal position listed (shuffled), the sparse entry point and the dense chunk-attention entry point
    compute the same thing through entirely different data paths; both are held to the dense oracle."""
    import oracle
    from parity import compare
    prefix, chunk = [700, 0], [150, 200]
    p = _problem(5700, prefix, chunk, 128)
    topk = 1024
    rng = np.random.default_rng(4)
    idx = np.full((sum(chunk), topk), -1, np.int32)
    row = 0
    for P, C in zip(prefix, chunk):
        for i in range(C):
            idx[row, : P + i + 1] = rng.permutation(P + i + 1)
            row += 1
    pg = p.to("cuda")
    sp = api.SparseAttn(pg, torch.from_numpy(idx).cuda())
    o_s, l_s = sp.run()
    dn = api.ChunkAttn(pg)
    o_d, l_d = dn.run()
    torch.cuda.synchronize()
    assert int(sp.status.item()) == 0 and int(dn.status.item()) == 0
    rows = oracle.all_rows(p.chunk_len.numpy(), 128)
    print(compare(o_s, l_s, p, rows, "sparse, all positions listed"))
    print(compare(o_d, l_d, p, rows, "dense"))
    assert (o_s.float() - o_d.float()).abs().max().item() <= 1e-2
    assert (l_s - l_d).abs().max().item() <= 1e-4
