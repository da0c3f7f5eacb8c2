"""GPU parity for vpp_kv_append (bit-exact against the CPU oracle) and its device-side checks."""
import numpy as np
import pytest
import torch

from oracle.ref_kv_append import ref_kv_append
from paper_2608_26523_b200 import api, workloads as W

pytestmark = pytest.mark.gpu


def _bits(t):
    return t.cpu().view(torch.int16).numpy().view(np.uint16)


def run_case(seed, prefix, chunk, hkv, dqk, dv, block_size, alias):
    """Take a problem whose cache is complete, cut the chunk's rows out as k_new / v_new, poison their slots, append
    them back with the library and compare the whole cache (pool included) with the oracle's result."""
    prob = W.make_problem(seed, prefix, chunk, hkv * 2 if not alias else 4, hkv, dqk, dv, block_size=block_size, std=0.5,
                          v_aliases_k=alias)
    kb = _bits(prob.k_cache)
    vb = None if alias else _bits(prob.v_cache)
    bs = prob.k_cache.shape[1]
    bt = None if prob.block_table is None else prob.block_table.numpy()
    rows_k, rows_v, where = [], [], []
    for r in range(len(prefix)):
        for pos in range(prefix[r], prefix[r] + chunk[r]):
            blk, slot = (r, pos) if bt is None else (int(bt[r, pos // bs]), pos % bs)
            rows_k.append(kb[blk, slot].copy())
            if vb is not None:
                rows_v.append(vb[blk, slot].copy())
            where.append((blk, slot))
    total = len(rows_k)
    k_new = np.stack(rows_k) if total else np.zeros((0, hkv, dqk), np.uint16)
    v_new = None if alias else (np.stack(rows_v) if total else np.zeros((0, hkv, dv), np.uint16))
    k_start, v_start = kb.copy(), None if alias else vb.copy()
    for blk, slot in where:
        k_start[blk, slot] = 0x7FC1           # a NaN pattern that is not in the data
        if v_start is not None:
            v_start[blk, slot] = 0x7FC2
    want_k, want_v = ref_kv_append(k_start, v_start, k_new, v_new, bt, bs, prefix, chunk)

    dev = "cuda"
    to_t = lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).to(dev)
    k_cache = to_t(k_start)
    v_cache = k_cache[..., :dv] if alias else to_t(v_start)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    api.vpp_kv_append(to_t(k_new), None if alias else to_t(v_new), k_cache, v_cache,
                      None if bt is None else prob.block_table.to(dev), prob.prefix_len.to(dev), prob.chunk_len.to(dev),
                      bs, prob.max_seq_len, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert (_bits(k_cache) == want_k).all()
    if not alias:
        assert (_bits(v_cache) == want_v).all()
    # and the result is the complete cache again
    assert (_bits(k_cache) == kb).all()


CASES = [
    # prefix, chunk, Hkv, Dqk, Dv, block_size, v aliases k
    ([0], [1], 1, 128, 128, 16, False),
    ([37], [300], 2, 128, 128, 16, False),
    ([1000, 0, 17, 511], [200, 0, 300, 129], 2, 128, 128, 32, False),
    ([4095], [257], 4, 128, 128, 256, False),
    ([513], [640], 2, 128, 128, None, False),            # contiguous cache
    ([300, 5], [77, 130], 1, 576, 512, 64, True),         # absorbed MLA: one latent row, values alias keys
    ([0, 0, 0], [5, 130, 1], 8, 128, 128, 128, False),
]


@pytest.mark.parametrize("case", range(len(CASES)))
def test_append_matches_oracle_bit_for_bit(case):
    run_case(3000 + case, *CASES[case])


def test_many_requests():
    rng = np.random.RandomState(5)
    prefix = [int(x) for x in rng.randint(0, 40, 200)]
    chunk = [int(x) for x in rng.randint(0, 9, 200)]
    run_case(3100, prefix, chunk, 2, 128, 128, 16, False)


def test_bad_lengths_write_nothing_and_bad_block_skips_the_row():
    prob = W.make_problem(3200, [10], [20], 4, 2, 128, 128, block_size=16, std=0.5).to("cuda")
    k_new = torch.ones(20, 2, 128, dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    before = prob.k_cache.clone()
    # sum(chunk_len) != total_q
    api.vpp_kv_append(k_new, k_new, prob.k_cache, prob.v_cache, prob.block_table, prob.prefix_len, prob.chunk_len,
                      16, prob.max_seq_len, status=status, total_q=19)
    torch.cuda.synchronize()
    assert int(status.item()) == 1          # VPP_DEV_BAD_LENGTHS
    assert torch.equal(before.view(torch.int16), prob.k_cache.view(torch.int16))
    # a request that outgrows its pages
    too_long = torch.tensor([10 ** 6], dtype=torch.int32, device="cuda")
    api.vpp_kv_append(k_new, k_new, prob.k_cache, prob.v_cache, prob.block_table, too_long, prob.chunk_len,
                      16, prob.max_seq_len, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 1
    assert torch.equal(before.view(torch.int16), prob.k_cache.view(torch.int16))
    # one block-table entry out of range: its rows are skipped, the others are written
    bt = prob.block_table.clone()
    bt[0, 1] = prob.k_cache.shape[0] + 3           # logical page 1 = positions 16..31
    api.vpp_kv_append(k_new, k_new, prob.k_cache, prob.v_cache, bt, prob.prefix_len, prob.chunk_len,
                      16, prob.max_seq_len, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 2
    ok_blk = int(prob.block_table[0, 0])
    assert (prob.k_cache[ok_blk, 10:16].float() == 1).all()        # positions 10..15 landed
    bad_blk = int(prob.block_table[0, 1])
    assert torch.equal(before[bad_blk].view(torch.int16), prob.k_cache[bad_blk].view(torch.int16))


def test_host_side_argument_checks():
    prob = W.make_problem(3201, [10], [20], 4, 2, 128, 128, block_size=16).to("cuda")
    k_new = torch.ones(20, 2, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(api.VppError):
        api.vpp_kv_append(k_new[:, :, :100].contiguous(), None, prob.k_cache, prob.v_cache, prob.block_table,
                          prob.prefix_len, prob.chunk_len, 16, prob.max_seq_len)   # head dim not a multiple of 8
    with pytest.raises(api.VppError):
        api.vpp_kv_append(k_new, k_new, prob.k_cache, prob.v_cache, prob.block_table, prob.prefix_len, prob.chunk_len,
                          24, prob.max_seq_len)                                     # block size not a power of two
