"""Shared helpers for the GPU parity tests: run the CUDA library and the CPU oracle on the same bytes."""
import numpy as np
import torch

import oracle
from paper_2608_26523_b200 import api

# Tolerances (bf16 inputs): max abs error <= 1e-2 -- or half a bf16 ulp of the reference where that is
# larger (|ref| >= 4) -- relative L2 <= 5e-3, lse within 1e-5 relative (absolute below |lse| = 1).
ABS_TOL = 1e-2
REL_L2_TOL = 5e-3
LSE_TOL = 1e-5


def oracle_rows(prob_cpu, rows):
    p = prob_cpu
    return oracle.ref_chunk_attn_rows(
        p.q, p.k_cache, p.v_cache, p.k_cache.stride()[:3], p.v_cache.stride()[:3],
        None if p.block_table is None else p.block_table.numpy(), p.block_size,
        p.prefix_len.numpy(), p.chunk_len.numpy(), p.num_q_heads, p.num_kv_heads,
        p.head_dim_qk, p.head_dim_v, p.scale, rows)


def packed_index(prob_cpu, rows):
    """Packed query-row index of each (request, row, head) triple."""
    c = prob_cpu.chunk_len.numpy().astype(np.int64)
    start = np.concatenate([[0], np.cumsum(c)[:-1]])
    rows = np.asarray(rows)
    return start[rows[:, 0]] + rows[:, 1], rows[:, 2]


def compare(out_gpu, lse_gpu, prob_cpu, rows, label=""):
    """Element-by-element comparison of the listed rows; returns the error summary."""
    rows = np.asarray(rows, dtype=np.int32).reshape(-1, 3)
    ref_o, ref_l = oracle_rows(prob_cpu, rows)
    ti, hi = packed_index(prob_cpu, rows)
    got_o = out_gpu.float().cpu().numpy().astype(np.float64)[ti, hi]
    got_l = lse_gpu.cpu().numpy().astype(np.float64)[ti, hi] if lse_gpu is not None else ref_l   # (None: out only)
    assert np.isfinite(got_o).all(), "%s: non-finite output" % label
    err = np.abs(got_o - ref_o)
    allowed = np.maximum(ABS_TOL, 2.0 ** -8 * np.abs(ref_o))
    max_abs = float(err.max()) if err.size else 0.0
    rel_l2 = float(np.linalg.norm(got_o - ref_o) / max(np.linalg.norm(ref_o), 1e-30)) if err.size else 0.0
    lse_err = np.abs(got_l - ref_l) / np.maximum(1.0, np.abs(ref_l))
    max_lse = float(lse_err.max()) if lse_err.size else 0.0
    summary = dict(label=label, rows=int(rows.shape[0]), max_abs=max_abs, rel_l2=rel_l2, max_lse_rel=max_lse,
                   needed_ulp_clause=bool((err > ABS_TOL).any()))
    assert (err <= allowed).all(), "%s: max abs err %.4g (worst allowed %.4g) %s" % (
        label, max_abs, float(allowed[np.unravel_index(err.argmax(), err.shape)]), summary)
    assert rel_l2 <= REL_L2_TOL, "%s: rel L2 %.4g %s" % (label, rel_l2, summary)
    assert max_lse <= LSE_TOL, "%s: lse rel err %.4g %s" % (label, max_lse, summary)
    return summary


def run_gpu(prob_gpu, num_kv_splits=0):
    runner = api.ChunkAttn(prob_gpu, num_kv_splits=num_kv_splits)
    # canaries: the library must write every row it owns and nothing else
    runner.out.fill_(float("nan"))
    runner.lse.fill_(float("nan"))
    out, lse = runner.run()
    torch.cuda.synchronize()
    st = int(runner.status.item())
    assert st == 0, "device status %d" % st
    return out, lse, runner


def sample_rows(prob_cpu, n_random=256, seed=0):
    """Deterministic row sample: chunk ends, +-1 around 128-row tile edges of the first and last query
    tile, rows whose position straddles a cache-block edge, and random (row, head) pairs."""
    rng = np.random.default_rng(seed)
    hq = prob_cpu.num_q_heads
    B = prob_cpu.block_size
    trip = []
    for r in range(prob_cpu.num_reqs):
        P, C = int(prob_cpu.prefix_len[r]), int(prob_cpu.chunk_len[r])
        if C == 0:
            continue
        cand = {0, C - 1, 1, 126, 127, 128, 129, C - 129, C - 128, C - 127, C - 2}
        for i in range(max(0, -P % B - 1), C, max(B, 1)):      # positions next to a block edge
            cand.update({i, i + 1})
            if len(cand) > 40:
                break
        for i in sorted(x for x in cand if 0 <= x < C):
            for h in {0, hq - 1, int(rng.integers(0, hq))}:
                trip.append((r, i, h))
        for _ in range(max(1, n_random // max(prob_cpu.num_reqs, 1))):
            trip.append((r, int(rng.integers(0, C)), int(rng.integers(0, hq))))
    return np.array(sorted(set(trip)), dtype=np.int32)


def tile_rows(prob_cpu, per="pair", seed=0, every=1):
    """One random (row, head) per work item of the launch: for every 128-row query tile of every request, one row
    of the tile and one head out of each head group -- "pair": each pair of q-heads (the items of the d = 128
    kernel); "kvhead": each kv-head's group; "tile": one head of all.  `every` > 1 keeps every n-th tile only."""
    rng = np.random.default_rng(seed)
    hq, hkv = prob_cpu.num_q_heads, prob_cpu.num_kv_heads
    groups = {"pair": [(h, min(h + 2, hq)) for h in range(0, hq, 2)],
              "kvhead": [(g * (hq // hkv), (g + 1) * (hq // hkv)) for g in range(hkv)],
              "tile": [(0, hq)]}[per]
    trip = []
    for r in range(prob_cpu.num_reqs):
        C = int(prob_cpu.chunk_len[r])
        for k, t0 in enumerate(range(0, C, 128)):
            if k % every:
                continue
            for lo, hi in groups:
                trip.append((r, int(rng.integers(t0, min(t0 + 128, C))), int(rng.integers(lo, hi))))
    return np.array(sorted(set(trip)), dtype=np.int32).reshape(-1, 3)


def all_heads_of_rows(prob_cpu, n_rows=8, seed=0):
    """Every q-head of n_rows random rows per request (first and last row included)."""
    rng = np.random.default_rng(seed)
    trip = []
    for r in range(prob_cpu.num_reqs):
        C = int(prob_cpu.chunk_len[r])
        if C == 0:
            continue
        rows = {0, C - 1} | {int(x) for x in rng.integers(0, C, max(n_rows - 2, 0))}
        trip += [(r, i, h) for i in sorted(rows) for h in range(prob_cpu.num_q_heads)]
    return np.array(sorted(set(trip)), dtype=np.int32).reshape(-1, 3)
