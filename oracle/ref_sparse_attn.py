"""fp64 CPU oracle for index-selected (sparse) chunk attention over a latent cache -- TEST INFRASTRUCTURE ONLY.

The paper's third model attends with "MLA + DSA sparse attention" (its evaluation-setup section) and notes in the
"Impact of Sparse Attention" paragraph that this flattens the growth of the attention cost with the prefix.  The paper
does not define the selection; the reading taken here is the public one of that attention family: for every query
token an external indexer supplies a list of key positions, shared by all q-heads, and Eq. 1 is evaluated over the
listed keys only.  What this file fixes:

  * token t of request r sits at position pos = prefix_len[r] + i; an entry e of its list takes part iff
    0 <= e <= pos (anything else -- negative padding, a position in the future -- is skipped);
  * the list is a list, not a set: a position listed twice counts twice in the softmax;
  * keys are rows of the one latent kv-head (Dqk features); values are the first Dv features of the same row;
  * out = sum_j softmax_j(scale * q . k_j) v_j and lse = log sum_j exp(scale * q . k_j) over the entries that take
    part; a token none of whose entries takes part has out = 0 and lse = -inf.

Plain numpy in float64, one token at a time, no blocking.  Nothing here imports or shares code with the CUDA
library; only the tests, the smoke check and the benchmark's CPU-baseline leg call it.
"""
import numpy as np


def bf16_bits_to_f64(bits):
    """bf16 bit patterns (uint16) -> float64, exactly."""
    bits = np.asarray(bits)
    if bits.dtype == np.int16:
        bits = bits.view(np.uint16)
    assert bits.dtype == np.uint16
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def ref_sparse_chunk_attn(q, kv_cache, indices, block_table, block_size, prefix_len, chunk_len, head_dim_v, scale,
                          tokens=None):
    """q uint16 [T, Hq, Dqk] (bf16 bits, request-major); kv_cache uint16 [num_blocks, block_size, 1, Dqk];
    indices int32 [T, topk] key positions within the token's own request; block_table int32 [R, max_blocks] or None
    (contiguous: request r is block r, slot = position).  tokens: optional list of global token rows to evaluate
    (default all).  Returns (out [n, Hq, Dv] float64, lse [n, Hq] float64)."""
    q = np.asarray(q)
    T, Hq, Dqk = q.shape
    indices = np.asarray(indices)
    assert indices.shape[0] == T
    req_of, pos_of = np.empty(T, np.int64), np.empty(T, np.int64)
    row = 0
    for r in range(len(prefix_len)):
        for i in range(int(chunk_len[r])):
            req_of[row], pos_of[row] = r, int(prefix_len[r]) + i
            row += 1
    assert row == T
    tokens = list(range(T)) if tokens is None else [int(t) for t in tokens]
    out = np.zeros((len(tokens), Hq, head_dim_v), np.float64)
    lse = np.full((len(tokens), Hq), -np.inf, np.float64)
    cache = np.asarray(kv_cache)
    for n, t in enumerate(tokens):
        r, pos = int(req_of[t]), int(pos_of[t])
        rows = []
        for e in indices[t].tolist():
            if e < 0 or e > pos:
                continue
            if block_table is None:
                blk, slot = r, e
            else:
                blk, slot = int(block_table[r, e // block_size]), e % block_size
            rows.append(cache[blk, slot, 0, :])
        if not rows:
            continue
        k = bf16_bits_to_f64(np.stack(rows))                 # [n_sel, Dqk]
        s = scale * (bf16_bits_to_f64(q[t]) @ k.T)           # [Hq, n_sel]
        m = s.max(axis=1, keepdims=True)
        p = np.exp(s - m)
        l = p.sum(axis=1, keepdims=True)
        out[n] = (p / l) @ k[:, :head_dim_v]
        lse[n] = (m + np.log(l))[:, 0]
    return out, lse
