"""Seeded synthetic inputs for chunked-prefill attention.

Used by the tests (which hand the same bytes to the CPU oracle and to the CUDA
library), by the smoke check and by the benchmark.  This module holds no
attention arithmetic: it only draws random tensors, lays a KV cache out in
pages, and shuffles a block table.

The shapes follow the long-context MoE serving workloads of the paper's
evaluation (GQA and absorbed-MLA models, fixed chunk budgets of 8K-32K tokens,
prompts from 1K to 1M tokens, mixed-length batches); the value distributions
and the five named configurations are the benchmark definitions this
repository is measured on.  No dataset is involved.
"""
import math
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np
import torch

BASE_SEED = 260826523


@dataclass
class Problem:
    """One launch worth of inputs.  All tensors live on `device`."""
    q: torch.Tensor                      # bf16 [total_q, Hq, Dqk], packed request-major
    k_cache: torch.Tensor                # bf16 [num_blocks, block_size, Hkv, Dqk]
    v_cache: torch.Tensor                # bf16 [num_blocks, block_size, Hkv, Dv]; may be a view of k_cache
    block_table: Optional[torch.Tensor]  # int32 [R, max_blocks_per_req] or None (contiguous)
    prefix_len: torch.Tensor             # int32 [R]
    chunk_len: torch.Tensor              # int32 [R]
    block_size: int
    num_q_heads: int
    num_kv_heads: int
    head_dim_qk: int
    head_dim_v: int
    scale: float
    max_seq_len: int
    name: str = ""
    extra: dict = field(default_factory=dict)

    @property
    def num_reqs(self):
        return int(self.prefix_len.numel())

    @property
    def total_q(self):
        return int(self.q.shape[0])

    def pairs(self):
        """Visible (query, key) pairs per q-head: sum_r C_r*P_r + C_r(C_r+1)/2."""
        p = self.prefix_len.cpu().numpy().astype(np.int64)
        c = self.chunk_len.cpu().numpy().astype(np.int64)
        return int((c * p + c * (c + 1) // 2).sum())

    def flops(self):
        """2*(Dqk+Dv) flop per visible pair per q-head (exact causal count)."""
        return 2 * self.num_q_heads * (self.head_dim_qk + self.head_dim_v) * self.pairs()

    def with_chunk(self, prefix_len, chunk_len, q):
        """Same cache and block table, another (prefix, chunk) window and query tensor."""
        dev = self.q.device
        return Problem(q=q, k_cache=self.k_cache, v_cache=self.v_cache, block_table=self.block_table,
                       prefix_len=torch.tensor(prefix_len, dtype=torch.int32, device=dev),
                       chunk_len=torch.tensor(chunk_len, dtype=torch.int32, device=dev),
                       block_size=self.block_size, num_q_heads=self.num_q_heads,
                       num_kv_heads=self.num_kv_heads, head_dim_qk=self.head_dim_qk,
                       head_dim_v=self.head_dim_v, scale=self.scale, max_seq_len=self.max_seq_len,
                       name=self.name, extra=dict(self.extra))

    def to(self, device):
        bt = None if self.block_table is None else self.block_table.to(device)
        k = self.k_cache.to(device)
        if self.extra.get("v_aliases_k"):
            v = k[..., : self.head_dim_v]
        else:
            v = self.v_cache.to(device)
        return Problem(q=self.q.to(device), k_cache=k, v_cache=v, block_table=bt,
                       prefix_len=self.prefix_len.to(device), chunk_len=self.chunk_len.to(device),
                       block_size=self.block_size, num_q_heads=self.num_q_heads,
                       num_kv_heads=self.num_kv_heads, head_dim_qk=self.head_dim_qk,
                       head_dim_v=self.head_dim_v, scale=self.scale, max_seq_len=self.max_seq_len,
                       name=self.name, extra=dict(self.extra))


def _randn_bf16(shape, std, gen, device):
    """N(0, std) rounded to bf16, drawn in slabs so multi-GB tensors never need an fp32 copy."""
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    flat = out.view(-1)
    step = 1 << 26
    for s in range(0, flat.numel(), step):
        n = min(step, flat.numel() - s)
        x = torch.randn(n, generator=gen, device=device, dtype=torch.float32)
        if std != 1.0:
            x.mul_(std)
        flat[s:s + n] = x.to(torch.bfloat16)
    return out


def random_q(seed, total_q, num_q_heads, head_dim_qk, std=1.0, device="cpu"):
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed))
    return _randn_bf16((total_q, num_q_heads, head_dim_qk), std, gen, device)


def make_problem(seed, prefix_lens: List[int], chunk_lens: List[int], num_q_heads, num_kv_heads,
                 head_dim_qk, head_dim_v, block_size=None, std=1.0, scale=None, v_aliases_k=False,
                 pool_factor=1.25, unused_fill=float("nan"), tail_fill=float("nan"),
                 seq_lens: Optional[List[int]] = None, device="cpu", name=""):
    """Draw Q and a KV cache that holds positions [0, seq_len) of every request.

    block_size=None: contiguous cache [R, max_seq_len, Hkv, D], no block table.
    Otherwise the cache is a pool of ceil(pool_factor * needed) blocks and the
    block table is a seeded random injection of logical into physical blocks.
    Blocks no request owns are filled with `unused_fill`; slots of a request's
    last block that lie at or beyond seq_len are filled with `tail_fill`.
    seq_lens (default prefix+chunk) lets one cache serve several chunk positions.
    v_aliases_k: V is the first head_dim_v features of each K row (absorbed MLA).
    """
    R = len(prefix_lens)
    assert len(chunk_lens) == R
    if seq_lens is None:
        seq_lens = [p + c for p, c in zip(prefix_lens, chunk_lens)]
    assert all(s >= p + c for s, p, c in zip(seq_lens, prefix_lens, chunk_lens))
    if scale is None:
        scale = 1.0 / math.sqrt(head_dim_qk)
    total_q = int(sum(chunk_lens))
    max_seq = max(max(seq_lens), 1)
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed))
    rng = np.random.default_rng(int(seed))

    q = _randn_bf16((total_q, num_q_heads, head_dim_qk), std, gen, device)

    if block_size is None:
        B = max_seq
        num_blocks = R
        block_table = None
        owner_len = list(seq_lens)                  # valid slots per physical block
    else:
        B = int(block_size)
        per_req = [(s + B - 1) // B for s in seq_lens]
        needed = sum(per_req)
        num_blocks = max(int(math.ceil(pool_factor * needed)), needed, 1)
        perm = rng.permutation(num_blocks)[:needed]
        max_blocks = max(max(per_req), 1)
        bt = np.full((R, max_blocks), -1, dtype=np.int32)
        owner_len = [0] * num_blocks
        o = 0
        for r in range(R):
            for b in range(per_req[r]):
                phys = int(perm[o]); o += 1
                bt[r, b] = phys
                owner_len[phys] = min(B, seq_lens[r] - b * B)
        block_table = torch.from_numpy(bt).to(device)

    k_cache = _randn_bf16((num_blocks, B, num_kv_heads, head_dim_qk), std, gen, device)
    if v_aliases_k:
        assert head_dim_v <= head_dim_qk
        v_cache = k_cache[..., :head_dim_v]
    else:
        v_cache = _randn_bf16((num_blocks, B, num_kv_heads, head_dim_v), std, gen, device)

    # poison what must never influence a result
    valid = torch.tensor(owner_len, dtype=torch.int64, device=device)
    slot = torch.arange(B, device=device)
    for cache in ([k_cache] if v_aliases_k else [k_cache, v_cache]):
        if unused_fill is not None:
            cache[valid == 0] = unused_fill
        if tail_fill is not None:
            partial = ((valid > 0) & (valid < B)).nonzero().flatten()
            for blk in partial.tolist():
                cache[blk, int(valid[blk]):] = tail_fill
    del slot

    return Problem(q=q, k_cache=k_cache, v_cache=v_cache, block_table=block_table,
                   prefix_len=torch.tensor(prefix_lens, dtype=torch.int32, device=device),
                   chunk_len=torch.tensor(chunk_lens, dtype=torch.int32, device=device),
                   block_size=B, num_q_heads=num_q_heads, num_kv_heads=num_kv_heads,
                   head_dim_qk=head_dim_qk, head_dim_v=head_dim_v, scale=float(scale),
                   max_seq_len=max_seq, name=name,
                   extra={"v_aliases_k": bool(v_aliases_k), "seed": int(seed), "seq_lens": list(seq_lens)})


# ----------------------------------------------------------------------------------------------
# The five benchmark configurations
# ----------------------------------------------------------------------------------------------

def cfg1(chunk_index=0, device="cpu"):
    """2048 tokens as 4 chunks of 512; Hq=4, Hkv=1, d=128; N(0,1); contiguous cache."""
    assert 0 <= chunk_index < 4
    base = make_problem(BASE_SEED + 1, [0], [2048], 4, 1, 128, 128, block_size=None, device=device,
                        name="cfg1")
    # the 2048 drawn query rows are the whole prompt; chunk k takes rows [512k, 512k+512)
    qk = base.q[512 * chunk_index: 512 * (chunk_index + 1)].contiguous()
    p = base.with_chunk([512 * chunk_index], [512], qk)
    p.extra["full"] = base
    return p


CFG2_PREFIXES = [0, 8192, 32768, 65536, 131072]
CFG3_PREFIXES = [0, 65536, 262144, 516096]
CFG4_CHUNK_IDX = [0, 4, 8, 13, 17, 21, 25, 29, 34, 38, 42, 46, 50, 55, 59, 63]
CFG4_PREFIXES = [16384 * k for k in CFG4_CHUNK_IDX]


def _single_request_cache(seed, max_prefix, chunk, hq, hkv, dqk, dv, block_size, std, scale,
                          v_aliases_k, device, name, prefix):
    """One request whose cache holds max_prefix+chunk tokens; the query chunk sits at `prefix`."""
    total = max_prefix + chunk
    prob = make_problem(seed, [prefix], [chunk], hq, hkv, dqk, dv, block_size=block_size, std=std,
                        scale=scale, v_aliases_k=v_aliases_k, seq_lens=[total], device=device,
                        name=name)
    return prob


single_request_cache = _single_request_cache   # (same recipe with other shapes / page sizes: bench.py --workload pages)


def cfg2(prefix=65536, max_prefix=None, device="cpu"):
    """GQA long-context chunk: Hq=64, Hkv=4, d=128, chunk 8192, 128-token pages, shuffled table."""
    mp = prefix if max_prefix is None else max_prefix
    return _single_request_cache(BASE_SEED + 2, mp, 8192, 64, 4, 128, 128, 128, 1.0, None, False,
                                 device, "cfg2", prefix)


def cfg3(prefix=65536, max_prefix=None, device="cpu"):
    """Absorbed MLA: Hq=128 sharing one latent row of 512+64, V = first 512 features, 64-token pages.

    Values N(0, sigma=0.5); softmax scale 1/sqrt(192) (128 nope + 64 rope dims before absorption)."""
    mp = prefix if max_prefix is None else max_prefix
    return _single_request_cache(BASE_SEED + 3, mp, 8192, 128, 1, 576, 512, 64, 0.5,
                                 1.0 / math.sqrt(192.0), True, device, "cfg3", prefix)


def cfg4(prefix=1032192, max_prefix=None, device="cpu"):
    """1M-token sweep: Hq=64, Hkv=8, d=128, chunk 16384, 128-token pages."""
    mp = prefix if max_prefix is None else max_prefix
    return _single_request_cache(BASE_SEED + 4, mp, 16384, 64, 8, 128, 128, 128, 1.0, None, False,
                                 device, "cfg4", prefix)


def cfg5_lengths(seed=BASE_SEED + 5, num_reqs=32, budget=16384, lo=1024, hi=262144,
                 c_min=64, c_max=2048):
    """Seeded (total length, chunk length, prefix) triples for the mixed varlen batch.

    L_r = floor(exp(U(ln lo, ln hi))); the chunk lengths are a random composition of `budget`
    into num_reqs parts with c_min <= C_r <= min(L_r, c_max) (rejection sampled); the chunk sits
    at a uniformly random, unaligned prefix P_r in [0, L_r - C_r]."""
    rng = np.random.default_rng(int(seed))
    L = np.floor(np.exp(rng.uniform(math.log(lo), math.log(hi), size=num_reqs))).astype(np.int64)
    cap = np.minimum(L, c_max)
    spare = budget - c_min * num_reqs
    assert spare >= 0
    for _ in range(100000):
        w = rng.dirichlet(np.full(num_reqs, 2.0))
        c = c_min + np.floor(w * spare).astype(np.int64)
        short = budget - int(c.sum())
        idx = rng.permutation(num_reqs)[:short]
        c[idx] += 1
        if int(c.sum()) == budget and np.all(c <= cap):
            break
    else:
        raise RuntimeError("no admissible composition found")
    P = np.array([rng.integers(0, int(L[r] - c[r]) + 1) for r in range(num_reqs)], dtype=np.int64)
    return L.tolist(), c.tolist(), P.tolist()


def cfg5(device="cpu", scale_lengths=1.0):
    """Mixed varlen batch: 32 requests, 16384 packed query tokens, Hq=64, Hkv=8, d=128, 128-token pages.

    scale_lengths < 1 shrinks every total length (keeping the chunk composition) for CPU-sized cases."""
    L, C, P = cfg5_lengths()
    if scale_lengths != 1.0:
        P = [int(p * scale_lengths) for p in P]
    return make_problem(BASE_SEED + 5, P, C, 64, 8, 128, 128, block_size=128, device=device,
                        name="cfg5")


# ----------------------------------------------------------------------------------------------
# Index lists for index-selected (sparse) attention over the latent cache
# ----------------------------------------------------------------------------------------------

def make_sparse_indices(seed, prefix_lens, chunk_lens, topk, kind="scattered", window=None, group=64, pool_factor=1.5,
                        pad=-1):
    """Per-token lists of selected key positions, int32 [total_q, topk] (numpy), seeded.

    Stands in for the output of a learned top-k indexer (the paper's MLA + DSA model; no trained weights here).  Every
    list holds distinct causal positions (<= the token's own position); a token with fewer than topk causal positions
    lists them all and pads with `pad`.  The order inside a list is shuffled.
      kind="scattered": the `window` most recent positions (default topk/4) plus uniformly random earlier positions --
                        no two tokens share more than chance: the worst case for cache reuse.
      kind="clustered": the same window, and the earlier positions of all tokens of a group of `group` consecutive
                        tokens are drawn from one pool of pool_factor * topk random positions -- neighbouring tokens
                        select mostly the same keys, as a trained indexer's lists do.
    """
    rng = np.random.default_rng(int(seed))
    total = int(sum(chunk_lens))
    out = np.full((total, topk), pad, dtype=np.int32)
    window = topk // 4 if window is None else int(window)
    row = 0
    for P, C in zip(prefix_lens, chunk_lens):
        for g0 in range(0, C, group):
            g1 = min(C, g0 + group)
            lo_pos = P + g0                       # every token of the group may see positions <= lo_pos
            pool = None
            if kind == "clustered" and lo_pos + 1 > topk:
                n_pool = min(lo_pos + 1, int(pool_factor * topk))
                pool = rng.choice(lo_pos + 1, size=n_pool, replace=False)
            for i in range(g0, g1):
                pos = P + i
                if pos + 1 <= topk:
                    sel = np.arange(pos + 1)
                else:
                    recent = np.arange(pos + 1 - window, pos + 1)
                    n_far = topk - window
                    if pool is not None:
                        cand = pool[pool < pos + 1 - window]
                        far = cand[rng.permutation(cand.size)[:n_far]]
                    else:
                        far = np.empty(0, np.int64)
                    if far.size < n_far:          # top up with uniform picks outside what is already chosen
                        need = n_far - far.size
                        extra = rng.choice(pos + 1 - window, size=min(pos + 1 - window, need + far.size), replace=False)
                        extra = extra[~np.isin(extra, far)][:need]
                        far = np.concatenate([far, extra])
                    sel = np.concatenate([recent, far])
                sel = sel[rng.permutation(sel.size)]
                out[row + i, : sel.size] = sel
        row += C
    return out


def make_sparse_indices_strata(seed, prefix_lens, chunk_lens, topk, kind="scattered", window=None, group=64):
    """Vectorised variant of make_sparse_indices for benchmark sizes (millions of entries): int32 torch tensor
    [total_q, topk] on the CPU.  Same structure -- the `window` most recent positions plus distinct earlier ones,
    -1 padding when fewer than topk causal positions exist -- but the earlier positions are one uniform draw from each
    of topk - window equal strata of [0, pos - window], which makes them distinct without rejection.
    kind="clustered": the tokens of a group of `group` consecutive tokens use the same draws and the strata of the
    group's first token, so their earlier selections coincide."""
    gen = torch.Generator()
    gen.manual_seed(int(seed))
    window = topk // 4 if window is None else int(window)
    n_far = topk - window
    parts = []
    for P, C in zip(prefix_lens, chunk_lens):
        if C == 0:
            continue
        pos = P + torch.arange(C, dtype=torch.int64)                       # [C]
        if kind == "clustered":
            grp = torch.arange(C) // group
            u = torch.rand((int(grp.max()) + 1, n_far), generator=gen, dtype=torch.float64)[grp]
            span_pos = P + grp * group                                     # the group's first token
        else:
            u = torch.rand((C, n_far), generator=gen, dtype=torch.float64)
            span_pos = pos
        span = (span_pos + 1 - window).clamp(min=0).to(torch.float64)      # earlier positions available
        k = torch.arange(n_far, dtype=torch.float64)
        w = span[:, None] / n_far                                          # stratum k = [floor(k w), floor((k+1) w))
        lo, hi = (k[None, :] * w).floor(), ((k[None, :] + 1) * w).floor()
        far = (lo + (u * (hi - lo)).floor()).to(torch.int64)
        recent = pos[:, None] - torch.arange(window, dtype=torch.int64)[None, :]
        idx = torch.cat([recent, far], dim=1)
        # tokens with fewer than topk causal positions (or strata narrower than one position): list 0..pos, pad with -1
        short = (span_pos + 1 - window) < n_far
        if short.any():
            full = torch.arange(topk, dtype=torch.int64)[None, :].expand(int(short.sum()), topk).clone()
            full[full > pos[short][:, None]] = -1
            idx[short] = full
        parts.append(idx.to(torch.int32))
    if not parts:
        return torch.zeros((0, topk), dtype=torch.int32)
    out = torch.cat(parts, dim=0)
    perm = torch.argsort(torch.rand(out.shape, generator=gen), dim=1)      # shuffle inside each list
    return torch.gather(out, 1, perm.to(torch.int64)).contiguous()
