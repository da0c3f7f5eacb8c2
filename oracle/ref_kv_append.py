"""CPU oracle for the paged KV-cache append -- TEST INFRASTRUCTURE ONLY.

The step before attention in a chunked prefill: the chunk's new key and value rows are written to the cache
positions [prefix_len, prefix_len + chunk_len) of their request (the paper's "Chunked Prefill Pipeline Parallelism"
section: each chunk's KV is appended to the cache that later chunks attend to).  Plain Python loops over tokens,
one element-wise copy per (token, kv-head): bit-exact byte movement, no arithmetic.

Nothing here imports or shares code with the CUDA library; only the tests and the smoke / benchmark checks call it.
"""
import numpy as np


def ref_kv_append(k_cache, v_cache, k_new, v_new, block_table, block_size, prefix_len, chunk_len):
    """Write rows into copies of the caches and return them.

    k_cache  uint16 (bf16 bits) [num_blocks, slots, Hkv, Dqk]; v_cache likewise with Dv, or None when the values are
             the leading features of the keys (absorbed MLA).
    k_new    uint16 [total_q, Hkv, Dqk], request-major packing; v_new [total_q, Hkv, Dv] or None.
    block_table int32 [R, max_blocks] or None: contiguous, request r is block r and slot = position.
    Rows of request r go to positions prefix_len[r] + i, i = 0..chunk_len[r]-1.
    """
    k_out = np.array(k_cache, copy=True)
    v_out = None if v_cache is None else np.array(v_cache, copy=True)
    row = 0
    for r in range(len(prefix_len)):
        for i in range(int(chunk_len[r])):
            p = int(prefix_len[r]) + i
            if block_table is None:
                blk, slot = r, p
            else:
                blk, slot = int(block_table[r, p // block_size]), p % block_size
            for g in range(k_new.shape[1]):
                k_out[blk, slot, g, :] = k_new[row, g, :]
                if v_out is not None:
                    v_out[blk, slot, g, :] = v_new[row, g, :]
            row += 1
    assert row == k_new.shape[0]
    return k_out, v_out
