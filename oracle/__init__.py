"""fp64 CPU oracle for chunked-prefill attention -- TEST INFRASTRUCTURE ONLY.

Plain, slow, obviously-correct restatement of the paper's Eq. 1 with causal
masking, applied to one chunk of a chunked prefill (a query chunk attends to
the whole cached prefix plus itself).  The arithmetic lives in ``ref_attn.c``
(plain C loops in double, OpenMP over independent rows); this module only
compiles it with gcc and marshals numpy arrays through ctypes.

Nothing here imports, links or shares code with the CUDA library, and the
product library never calls into this package: only the tests, the smoke check
and the benchmark's CPU-baseline leg do.
"""
import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ref_attn.c")
_LIB = os.path.join(_HERE, "libref_attn.so")
_lock = threading.Lock()
_lib = None


def build(force=False):
    """Compile ref_attn.c into libref_attn.so next to it (gcc -O2 -fopenmp, no fast-math)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp%d" % os.getpid()
    subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
                           "-o", tmp, _SRC, "-lm"])
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            i32, i64, dbl, vp = ctypes.c_int32, ctypes.c_int64, ctypes.c_double, ctypes.c_void_p
            lib.ref_chunk_attn_rows.restype = ctypes.c_int
            lib.ref_chunk_attn_rows.argtypes = [vp, vp, vp, i64, i64, i64, i64, i64, i64,
                                                vp, i32, i32, vp, vp, i32,
                                                i32, i32, i32, i32, dbl,
                                                vp, i64, i64, i64, vp, vp]
            lib.ref_lse_merge.restype = None
            lib.ref_lse_merge.argtypes = [vp, vp, i32, i64, i32, vp, vp]
            _lib = lib
    return _lib


def num_threads():
    """Threads the OpenMP loops will use (OMP_NUM_THREADS, else all visible cores)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env.split(",")[0])
    return len(os.sched_getaffinity(0))


def _bits(a):
    """bf16 bit patterns as a C-contiguous uint16 numpy array (accepts torch bf16 CPU tensors)."""
    if hasattr(a, "detach"):  # torch tensor, without importing torch here
        import torch
        a = a.detach().cpu()
        if a.dtype == torch.bfloat16:
            a = a.view(torch.int16)
        a = a.numpy()
    a = np.asarray(a)
    if a.dtype == np.int16:
        a = a.view(np.uint16)
    if a.dtype != np.uint16:
        raise TypeError("expected bf16 bit patterns (uint16/int16) or a torch.bfloat16 tensor")
    return a


def _ptr(a):
    return ctypes.c_void_p(a.ctypes.data)


def ref_chunk_attn_rows(q, k_cache, v_cache, k_strides, v_strides, block_table, block_size,
                        prefix_len, chunk_len, num_q_heads, num_kv_heads, head_dim_qk,
                        head_dim_v, scale, rows, kv_lo=0, kv_hi=-1):
    """Attention output and log-sum-exp of selected query rows, in float64.

    q            bf16 bits, [total_q, Hq, Dqk] packed request-major.
    k_cache/v_cache  bf16 bits, any shape; addressed only through the strides.
                 They may be views of one buffer (v aliasing k for absorbed MLA):
                 pass the same array and give v_strides for it.
    k_strides/v_strides  (block_stride, token_stride, head_stride) in elements,
                 innermost (feature) stride 1.  If v_cache is a view that starts
                 inside another array, pass the view itself (its base pointer is used).
    block_table  int32 [num_reqs, max_blocks_per_req] or None (contiguous:
                 request r is block r, slot = token index).
    rows         int32 [n, 3] of (request, row in chunk, q-head).
    kv_lo,kv_hi  restrict keys to kv_lo <= j < kv_hi (kv_hi < 0: no upper limit).
    Returns (out [n, Dv] float64, lse [n] float64).
    """
    lib = _load()
    q = np.ascontiguousarray(_bits(q))
    k = _bits(k_cache)
    v = _bits(v_cache)
    prefix_len = np.ascontiguousarray(np.asarray(prefix_len, dtype=np.int32))
    chunk_len = np.ascontiguousarray(np.asarray(chunk_len, dtype=np.int32))
    rows = np.ascontiguousarray(np.asarray(rows, dtype=np.int32).reshape(-1, 3))
    n = rows.shape[0]
    if block_table is not None:
        block_table = np.ascontiguousarray(np.asarray(block_table, dtype=np.int32))
        bt_ptr, max_blocks = _ptr(block_table), block_table.shape[1]
    else:
        bt_ptr, max_blocks = ctypes.c_void_p(0), 0
    out = np.empty((n, head_dim_v), dtype=np.float64)
    lse = np.empty((n,), dtype=np.float64)
    rc = lib.ref_chunk_attn_rows(_ptr(q), _ptr(k), _ptr(v),
                                 *[int(x) for x in k_strides], *[int(x) for x in v_strides],
                                 bt_ptr, int(max_blocks), int(block_size),
                                 _ptr(prefix_len), _ptr(chunk_len), int(prefix_len.shape[0]),
                                 int(num_q_heads), int(num_kv_heads), int(head_dim_qk),
                                 int(head_dim_v), float(scale),
                                 _ptr(rows), n, int(kv_lo), int(kv_hi), _ptr(out), _ptr(lse))
    if rc != 0:
        raise ValueError("ref_chunk_attn_rows: a (request, row, head) triple is out of range")
    return out, lse


def ref_lse_merge(o_parts, lse_parts):
    """Merge partial attention results over disjoint key sets.

    o_parts [S, n, Dv], lse_parts [S, n] (float64).  Returns (out [n, Dv], lse [n]).
    """
    lib = _load()
    o_parts = np.ascontiguousarray(np.asarray(o_parts, dtype=np.float64))
    lse_parts = np.ascontiguousarray(np.asarray(lse_parts, dtype=np.float64))
    S, n, dv = o_parts.shape
    assert lse_parts.shape == (S, n)
    out = np.empty((n, dv), dtype=np.float64)
    lse = np.empty((n,), dtype=np.float64)
    lib.ref_lse_merge(_ptr(o_parts), _ptr(lse_parts), S, n, dv, _ptr(out), _ptr(lse))
    return out, lse


def all_rows(chunk_len, num_q_heads):
    """Row list covering every (request, row, head) of a launch."""
    trip = []
    for r, c in enumerate(np.asarray(chunk_len).tolist()):
        ii, hh = np.meshgrid(np.arange(c, dtype=np.int32), np.arange(num_q_heads, dtype=np.int32),
                             indexing="ij")
        trip.append(np.stack([np.full_like(ii, r), ii, hh], axis=-1).reshape(-1, 3))
    return np.concatenate(trip, axis=0) if trip else np.zeros((0, 3), np.int32)
