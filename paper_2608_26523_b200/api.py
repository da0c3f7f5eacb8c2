"""ctypes binding of the C ABI in include/vpp.h (argument marshalling only).

Every step of the attention path runs in the CUDA library; PyTorch is used for device memory and
streams.  There is no CPU fallback: if the shared library is missing or cannot be loaded, calls raise.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libvpp_chunk_attn.so")

VPP_OK = 0
VPP_ERR_INVALID_ARG = -1
VPP_ERR_UNSUPPORTED = -2
VPP_ERR_WORKSPACE = -3
VPP_ERR_CUDA = -4
VPP_ERR_TIMEOUT = -5

EXPORTS = ["vpp_chunk_attn_workspace_size", "vpp_chunk_attn_fwd", "vpp_lse_merge", "vpp_status_string",
           "vpp_last_error", "vpp_last_launch_count", "vpp_chunk_attn_fwd_static", "vpp_static_scratch_bytes",
           "vpp_static_last_error", "vpp_kv_append", "vpp_sparse_attn_workspace_size", "vpp_sparse_mla_fwd",
           "vpp_chunk_attn_partial_fwd", "vpp_tensor_map_cache_stats", "vpp_test_tensor_map_cache",
           "vpp_test_bounded_wait", "vpp_chunk_attn_host_workspace_size", "vpp_chunk_attn_host_plan",
           "vpp_chunk_attn_host_fwd", "vpp_host_last_error"]


class VppError(RuntimeError):
    def __init__(self, status, detail):
        super().__init__("vpp status %d: %s" % (status, detail))
        self.status = status


class ChunkAttnArgs(ctypes.Structure):
    _fields_ = [
        ("q", ctypes.c_void_p), ("k_cache", ctypes.c_void_p), ("v_cache", ctypes.c_void_p),
        ("k_block_stride", ctypes.c_int64), ("k_token_stride", ctypes.c_int64), ("k_head_stride", ctypes.c_int64),
        ("v_block_stride", ctypes.c_int64), ("v_token_stride", ctypes.c_int64), ("v_head_stride", ctypes.c_int64),
        ("block_table", ctypes.c_void_p), ("prefix_len", ctypes.c_void_p), ("chunk_len", ctypes.c_void_p),
        ("num_reqs", ctypes.c_int32), ("max_blocks_per_req", ctypes.c_int32), ("block_size", ctypes.c_int32),
        ("num_blocks", ctypes.c_int32), ("total_q", ctypes.c_int32), ("max_seq_len", ctypes.c_int32),
        ("num_q_heads", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32), ("head_dim_qk", ctypes.c_int32),
        ("head_dim_v", ctypes.c_int32), ("softmax_scale", ctypes.c_float), ("num_kv_splits", ctypes.c_int32),
        ("out", ctypes.c_void_p), ("lse", ctypes.c_void_p), ("workspace", ctypes.c_void_p),
        ("workspace_bytes", ctypes.c_size_t), ("status", ctypes.c_void_p),
    ]


class KvAppendArgs(ctypes.Structure):
    _fields_ = [
        ("k_new", ctypes.c_void_p), ("v_new", ctypes.c_void_p), ("k_cache", ctypes.c_void_p), ("v_cache", ctypes.c_void_p),
        ("k_block_stride", ctypes.c_int64), ("k_token_stride", ctypes.c_int64), ("k_head_stride", ctypes.c_int64),
        ("v_block_stride", ctypes.c_int64), ("v_token_stride", ctypes.c_int64), ("v_head_stride", ctypes.c_int64),
        ("block_table", ctypes.c_void_p), ("prefix_len", ctypes.c_void_p), ("chunk_len", ctypes.c_void_p),
        ("num_reqs", ctypes.c_int32), ("max_blocks_per_req", ctypes.c_int32), ("block_size", ctypes.c_int32),
        ("num_blocks", ctypes.c_int32), ("total_q", ctypes.c_int32), ("max_seq_len", ctypes.c_int32),
        ("num_kv_heads", ctypes.c_int32), ("head_dim_qk", ctypes.c_int32), ("head_dim_v", ctypes.c_int32),
        ("status", ctypes.c_void_p),
    ]


class SparseAttnArgs(ctypes.Structure):
    _fields_ = [
        ("q", ctypes.c_void_p), ("kv_cache", ctypes.c_void_p), ("kv_row_stride", ctypes.c_int64),
        ("indices", ctypes.c_void_p), ("topk", ctypes.c_int32),
        ("block_table", ctypes.c_void_p), ("prefix_len", ctypes.c_void_p), ("chunk_len", ctypes.c_void_p),
        ("num_reqs", ctypes.c_int32), ("max_blocks_per_req", ctypes.c_int32), ("block_size", ctypes.c_int32),
        ("num_blocks", ctypes.c_int32), ("total_q", ctypes.c_int32), ("max_seq_len", ctypes.c_int32),
        ("num_q_heads", ctypes.c_int32), ("softmax_scale", ctypes.c_float),
        ("out", ctypes.c_void_p), ("lse", ctypes.c_void_p), ("workspace", ctypes.c_void_p),
        ("workspace_bytes", ctypes.c_size_t), ("status", ctypes.c_void_p),
    ]


class HostChunkAttnArgs(ctypes.Structure):
    _fields_ = [
        ("q_host", ctypes.c_void_p), ("k_new_host", ctypes.c_void_p), ("v_new_host", ctypes.c_void_p),
        ("out_host", ctypes.c_void_p), ("lse_host", ctypes.c_void_p),
        ("prefix_len", ctypes.c_int32), ("chunk_len", ctypes.c_int32),
        ("slice_rows", ctypes.c_void_p), ("num_slices", ctypes.c_int32),
        ("dev", ChunkAttnArgs), ("k_new_dev", ctypes.c_void_p), ("v_new_dev", ctypes.c_void_p),
    ]


_lib = None


def load_library():
    """Load libvpp_chunk_attn.so (raises if it has not been built: there is no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("CUDA library %s is missing: run `python -m paper_2608_26523_b200.build`" % LIB_PATH)
        lib = ctypes.CDLL(LIB_PATH)
        lib.vpp_chunk_attn_workspace_size.restype = ctypes.c_size_t
        lib.vpp_chunk_attn_workspace_size.argtypes = [ctypes.POINTER(ChunkAttnArgs)]
        lib.vpp_chunk_attn_fwd.restype = ctypes.c_int
        lib.vpp_chunk_attn_fwd.argtypes = [ctypes.POINTER(ChunkAttnArgs), ctypes.c_void_p]
        lib.vpp_lse_merge.restype = ctypes.c_int
        lib.vpp_lse_merge.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32,
                                      ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p,
                                      ctypes.c_void_p]
        lib.vpp_status_string.restype = ctypes.c_char_p
        lib.vpp_status_string.argtypes = [ctypes.c_int]
        lib.vpp_last_error.restype = ctypes.c_char_p
        lib.vpp_last_launch_count.restype = ctypes.c_int32
        lib.vpp_chunk_attn_fwd_static.restype = ctypes.c_int
        lib.vpp_chunk_attn_fwd_static.argtypes = [ctypes.POINTER(ChunkAttnArgs), ctypes.c_void_p]
        lib.vpp_static_scratch_bytes.restype = ctypes.c_size_t
        lib.vpp_static_last_error.restype = ctypes.c_char_p
        lib.vpp_kv_append.restype = ctypes.c_int
        lib.vpp_kv_append.argtypes = [ctypes.POINTER(KvAppendArgs), ctypes.c_void_p]
        lib.vpp_sparse_attn_workspace_size.restype = ctypes.c_size_t
        lib.vpp_sparse_attn_workspace_size.argtypes = [ctypes.c_int32]
        lib.vpp_sparse_mla_fwd.restype = ctypes.c_int
        lib.vpp_sparse_mla_fwd.argtypes = [ctypes.POINTER(SparseAttnArgs), ctypes.c_void_p]
        lib.vpp_chunk_attn_partial_fwd.restype = ctypes.c_int
        lib.vpp_chunk_attn_partial_fwd.argtypes = [ctypes.POINTER(ChunkAttnArgs), ctypes.c_int32, ctypes.c_int32,
                                                   ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        lib.vpp_tensor_map_cache_stats.restype = None
        lib.vpp_tensor_map_cache_stats.argtypes = [ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int64)]
        lib.vpp_test_tensor_map_cache.restype = ctypes.c_int32
        lib.vpp_test_tensor_map_cache.argtypes = [ctypes.c_int32]
        lib.vpp_test_bounded_wait.restype = ctypes.c_int
        lib.vpp_test_bounded_wait.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p]
        lib.vpp_chunk_attn_host_workspace_size.restype = ctypes.c_size_t
        lib.vpp_chunk_attn_host_workspace_size.argtypes = [ctypes.POINTER(HostChunkAttnArgs)]
        lib.vpp_chunk_attn_host_plan.restype = ctypes.c_int32
        lib.vpp_chunk_attn_host_plan.argtypes = [ctypes.POINTER(HostChunkAttnArgs), ctypes.POINTER(ctypes.c_int32)]
        lib.vpp_chunk_attn_host_fwd.restype = ctypes.c_int
        lib.vpp_chunk_attn_host_fwd.argtypes = [ctypes.POINTER(HostChunkAttnArgs), ctypes.c_void_p]
        lib.vpp_host_last_error.restype = ctypes.c_char_p
        _lib = lib
    return _lib


def _check(rc):
    if rc != VPP_OK:
        lib = load_library()
        raise VppError(rc, "%s: %s" % (lib.vpp_status_string(rc).decode(), lib.vpp_last_error().decode()))


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def make_args(q, k_cache, v_cache, block_table, prefix_len, chunk_len, block_size, max_seq_len,
              softmax_scale, num_kv_splits=0, out=None, lse=None, workspace=None, status=None,
              total_q=None, head_dim_v=None):
    """Fill a vpp_chunk_attn_args from tensors.

    q [T, Hq, Dqk] bf16; k_cache/v_cache [num_blocks, block_size, Hkv, D] bf16 (any strides with a
    contiguous last dim; v may be a view of k); block_table int32 [R, max_blocks] or None.
    """
    a = ChunkAttnArgs()
    a.q, a.k_cache, a.v_cache = _ptr(q), _ptr(k_cache), _ptr(v_cache)
    ks, vs = k_cache.stride(), v_cache.stride()
    assert ks[3] == 1 and vs[3] == 1 and q.is_contiguous()
    a.k_block_stride, a.k_token_stride, a.k_head_stride = ks[0], ks[1], ks[2]
    a.v_block_stride, a.v_token_stride, a.v_head_stride = vs[0], vs[1], vs[2]
    a.block_table = _ptr(block_table)
    a.prefix_len, a.chunk_len = _ptr(prefix_len), _ptr(chunk_len)
    a.num_reqs = prefix_len.numel()
    a.max_blocks_per_req = 0 if block_table is None else block_table.shape[1]
    a.block_size = int(block_size)
    a.num_blocks = k_cache.shape[0]
    a.total_q = q.shape[0] if total_q is None else int(total_q)
    a.max_seq_len = int(max_seq_len)
    a.num_q_heads, a.num_kv_heads = q.shape[1], k_cache.shape[2]
    a.head_dim_qk = q.shape[2]
    a.head_dim_v = v_cache.shape[3] if head_dim_v is None else int(head_dim_v)
    a.softmax_scale = float(softmax_scale)
    a.num_kv_splits = int(num_kv_splits)
    a.out, a.lse = _ptr(out), _ptr(lse)
    a.workspace = _ptr(workspace)
    a.workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    a.status = _ptr(status)
    return a


def vpp_chunk_attn_workspace_size(args):
    return int(load_library().vpp_chunk_attn_workspace_size(ctypes.byref(args)))


def vpp_chunk_attn_fwd(args, stream=None):
    """Enqueue chunked-prefill attention on `stream` (default: torch's current stream)."""
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    _check(load_library().vpp_chunk_attn_fwd(ctypes.byref(args), ctypes.c_void_p(stream)))


def vpp_chunk_attn_fwd_static(args, stream=None):
    """Same as vpp_chunk_attn_fwd but with the library's built-in scratch array as workspace.

    For callers that cannot allocate device memory (the workspace fields of `args` are ignored).
    Launches needing more than vpp_static_scratch_bytes() are refused; calls sharing a device must not
    overlap on the GPU."""
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    lib = load_library()
    rc = lib.vpp_chunk_attn_fwd_static(ctypes.byref(args), ctypes.c_void_p(stream))
    if rc != VPP_OK:
        raise VppError(rc, "%s: %s" % (lib.vpp_status_string(rc).decode(), lib.vpp_static_last_error().decode()))


def vpp_chunk_attn_partial_fwd(args, kv_begin, kv_end, o_part, lse_part, stream=None):
    """Attention of the launch described by `args` over the cached keys [kv_begin, kv_end) only: writes the partial
    results o_part fp32 [T, Hq, Dv] and lse_part fp32 [T, Hq] (one slice of vpp_lse_merge's inputs)."""
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    _check(load_library().vpp_chunk_attn_partial_fwd(ctypes.byref(args), int(kv_begin), int(kv_end), _ptr(o_part),
                                                     _ptr(lse_part), ctypes.c_void_p(stream)))


def vpp_tensor_map_cache_stats():
    """(look-ups, driver encodes) of the library's tensor-map cache so far in this process."""
    a, b = ctypes.c_int64(0), ctypes.c_int64(0)
    load_library().vpp_tensor_map_cache_stats(ctypes.byref(a), ctypes.byref(b))
    return int(a.value), int(b.value)


def vpp_test_bounded_wait(status, limit_cycles, stream=None):
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    _check(load_library().vpp_test_bounded_wait(_ptr(status), int(limit_cycles), ctypes.c_void_p(stream)))


def vpp_static_scratch_bytes():
    return int(load_library().vpp_static_scratch_bytes())


def vpp_lse_merge(o_parts, lse_parts, out, lse=None, stream=None):
    """out/lse <- merge of o_parts [S,T,Hq,Dv] fp32 and lse_parts [S,T,Hq] fp32."""
    S, T, Hq, Dv = o_parts.shape
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    _check(load_library().vpp_lse_merge(_ptr(o_parts), _ptr(lse_parts), S, T, Hq, Dv, _ptr(out), _ptr(lse),
                                        ctypes.c_void_p(stream)))


def vpp_kv_append(k_new, v_new, k_cache, v_cache, block_table, prefix_len, chunk_len, block_size, max_seq_len,
                  status=None, stream=None, total_q=None):
    """Write the chunk's new K/V rows into the (paged) cache: row i of request r goes to position prefix_len[r] + i.

    k_new [T, Hkv, Dqk] bf16, v_new [T, Hkv, Dv] bf16 or None when v_cache is a view of k_cache (absorbed MLA);
    caches [num_blocks, block_size, Hkv, D] with a contiguous last dim; block_table int32 [R, max_blocks] or None."""
    a = KvAppendArgs()
    a.k_new, a.v_new, a.k_cache, a.v_cache = _ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache)
    ks = k_cache.stride()
    vs = v_cache.stride() if v_cache is not None else (0, 0, 0, 1)
    assert ks[3] == 1 and vs[3] == 1 and k_new.is_contiguous() and (v_new is None or v_new.is_contiguous())
    a.k_block_stride, a.k_token_stride, a.k_head_stride = ks[0], ks[1], ks[2]
    a.v_block_stride, a.v_token_stride, a.v_head_stride = vs[0], vs[1], vs[2]
    a.block_table, a.prefix_len, a.chunk_len = _ptr(block_table), _ptr(prefix_len), _ptr(chunk_len)
    a.num_reqs = prefix_len.numel()
    a.max_blocks_per_req = 0 if block_table is None else block_table.shape[1]
    a.block_size = int(block_size)
    a.num_blocks = k_cache.shape[0]
    a.total_q = k_new.shape[0] if total_q is None else int(total_q)
    a.max_seq_len = int(max_seq_len)
    a.num_kv_heads, a.head_dim_qk = k_new.shape[1], k_new.shape[2]
    a.head_dim_v = v_new.shape[2] if v_new is not None else (v_cache.shape[3] if v_cache is not None else k_new.shape[2])
    a.status = _ptr(status)
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    _check(load_library().vpp_kv_append(ctypes.byref(a), ctypes.c_void_p(stream)))


def vpp_sparse_attn_workspace_size(total_q):
    return int(load_library().vpp_sparse_attn_workspace_size(int(total_q)))


def vpp_sparse_mla_fwd(args, stream=None):
    """Enqueue index-selected attention over the latent cache for a filled-in SparseAttnArgs."""
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    _check(load_library().vpp_sparse_mla_fwd(ctypes.byref(args), ctypes.c_void_p(stream)))


class SparseAttn:
    """Owns out / lse / workspace / status of one sparse launch over a Problem with an absorbed-MLA latent cache.

    indices: int32 [total_q, topk] device tensor of key positions (see include/vpp.h)."""

    def __init__(self, prob, indices, want_lse=True):
        dev = prob.q.device
        assert prob.head_dim_qk == 576 and prob.head_dim_v == 512 and prob.num_kv_heads == 1
        assert indices.dtype == torch.int32 and indices.is_contiguous() and indices.shape[0] == prob.total_q
        kc = prob.k_cache
        assert kc.stride(3) == 1 and (prob.block_table is None or kc.stride(0) == kc.shape[1] * kc.stride(1))
        self.prob, self.indices = prob, indices
        self.out = torch.empty((prob.total_q, prob.num_q_heads, 512), dtype=torch.bfloat16, device=dev)
        self.lse = torch.empty((prob.total_q, prob.num_q_heads), dtype=torch.float32, device=dev) if want_lse else None
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.workspace = torch.empty(max(vpp_sparse_attn_workspace_size(prob.total_q), 256), dtype=torch.uint8, device=dev)
        a = SparseAttnArgs()
        a.q, a.kv_cache, a.kv_row_stride = _ptr(prob.q), _ptr(kc), kc.stride(1)
        a.indices, a.topk = _ptr(indices), indices.shape[1]
        a.block_table, a.prefix_len, a.chunk_len = _ptr(prob.block_table), _ptr(prob.prefix_len), _ptr(prob.chunk_len)
        a.num_reqs = prob.num_reqs
        a.max_blocks_per_req = 0 if prob.block_table is None else prob.block_table.shape[1]
        a.block_size = prob.block_size
        a.num_blocks = kc.shape[0]
        a.total_q = prob.total_q
        a.max_seq_len = prob.max_seq_len if prob.block_table is not None else kc.shape[1]
        a.num_q_heads = prob.num_q_heads
        a.softmax_scale = prob.scale
        a.out, a.lse, a.status = _ptr(self.out), _ptr(self.lse), _ptr(self.status)
        a.workspace, a.workspace_bytes = _ptr(self.workspace), self.workspace.numel()
        self.args = a

    def run(self, stream=None):
        vpp_sparse_mla_fwd(self.args, stream)
        return self.out, self.lse


def vpp_last_launch_count():
    return int(load_library().vpp_last_launch_count())


class ChunkAttn:
    """Convenience wrapper that owns out / lse / workspace / status for one Problem-shaped launch."""

    def __init__(self, prob, num_kv_splits=0, want_lse=True):
        dev = prob.q.device
        self.prob = prob
        self.out = torch.empty((prob.total_q, prob.num_q_heads, prob.head_dim_v), dtype=torch.bfloat16, device=dev)
        self.lse = torch.empty((prob.total_q, prob.num_q_heads), dtype=torch.float32, device=dev) if want_lse else None
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.args = make_args(prob.q, prob.k_cache, prob.v_cache, prob.block_table, prob.prefix_len,
                              prob.chunk_len, prob.block_size, prob.max_seq_len, prob.scale,
                              num_kv_splits=num_kv_splits, out=self.out, lse=self.lse, status=self.status,
                              head_dim_v=prob.head_dim_v)
        n = vpp_chunk_attn_workspace_size(self.args)
        self.workspace = torch.empty(max(n, 256), dtype=torch.uint8, device=dev)
        self.args.workspace = _ptr(self.workspace)
        self.args.workspace_bytes = self.workspace.numel()

    def run(self, stream=None):
        vpp_chunk_attn_fwd(self.args, stream)
        return self.out, self.lse


def vpp_chunk_attn_host_workspace_size(hargs):
    return int(load_library().vpp_chunk_attn_host_workspace_size(ctypes.byref(hargs)))


def vpp_chunk_attn_host_plan(hargs):
    rows = (ctypes.c_int32 * 16)()
    n = int(load_library().vpp_chunk_attn_host_plan(ctypes.byref(hargs), rows))
    return [int(rows[i]) for i in range(n)]


def vpp_chunk_attn_host_fwd(hargs, stream=None):
    lib = load_library()
    if stream is None:
        stream = torch.cuda.current_stream().cuda_stream
    elif hasattr(stream, "cuda_stream"):
        stream = stream.cuda_stream
    st = lib.vpp_chunk_attn_host_fwd(ctypes.byref(hargs), ctypes.c_void_p(stream))
    if st != 0:
        raise VppError(st, "%s: %s" % (lib.vpp_status_string(st).decode(), lib.vpp_host_last_error().decode()))


class HostChunkPipeline:
    """Argument holder for vpp_chunk_attn_host_fwd: one request's chunk whose query, new K/V rows and results live in
    pinned host memory.  All of the work (slicing, copies, append, attention) is the C entry point's; this class only
    owns the device staging buffers and the argument struct."""

    def __init__(self, prob, slices=None, num_kv_splits=0, want_lse=True):
        """prob: a one-request Problem on the GPU (its cache holds the prefix; the chunk's own rows are written by the
        call).  slices: None (the library plans) or a list of slice lengths in query rows."""
        assert prob.num_reqs == 1 and prob.block_table is not None
        dev = prob.q.device
        P, C = int(prob.prefix_len[0]), int(prob.chunk_len[0])
        self.prob, self.P, self.C = prob, P, C
        aliased = prob.v_cache.data_ptr() == prob.k_cache.data_ptr()
        self.q_dev = torch.empty_like(prob.q)
        self.out = torch.empty((C, prob.num_q_heads, prob.head_dim_v), dtype=torch.bfloat16, device=dev)
        self.lse = torch.empty((C, prob.num_q_heads), dtype=torch.float32, device=dev) if want_lse else None
        self.k_new_dev = torch.empty((C, prob.num_kv_heads, prob.head_dim_qk), dtype=torch.bfloat16, device=dev)
        self.v_new_dev = None if aliased else torch.empty((C, prob.num_kv_heads, prob.head_dim_v), dtype=torch.bfloat16, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        h = HostChunkAttnArgs()
        h.dev = make_args(self.q_dev, prob.k_cache, prob.v_cache, prob.block_table, prob.prefix_len, prob.chunk_len,
                          prob.block_size, prob.max_seq_len, prob.scale, num_kv_splits=num_kv_splits, out=self.out,
                          lse=self.lse, status=self.status, head_dim_v=prob.head_dim_v)
        h.prefix_len, h.chunk_len = P, C
        self._slice_rows = None
        if slices is not None:
            self._slice_rows = (ctypes.c_int32 * len(slices))(*[int(x) for x in slices])
            h.slice_rows, h.num_slices = ctypes.cast(self._slice_rows, ctypes.c_void_p), len(slices)
        h.k_new_dev = _ptr(self.k_new_dev)
        h.v_new_dev = _ptr(self.v_new_dev) if self.v_new_dev is not None else None
        self.hargs = h
        n = vpp_chunk_attn_host_workspace_size(h)
        if n == 0:
            raise VppError(-1, load_library().vpp_host_last_error().decode())
        self.workspace = torch.empty(n, dtype=torch.uint8, device=dev)
        h.dev.workspace, h.dev.workspace_bytes = _ptr(self.workspace), n
        self.slices = vpp_chunk_attn_host_plan(h)

    def chunk_rows(self, cache):
        """The chunk's own rows of a [blocks, block_size, Hkv, D] cache tensor, token-major (what k_new / v_new hold)."""
        p = self.prob
        pos = torch.arange(self.P, self.P + self.C, device=p.block_table.device)
        blk = p.block_table[0, (pos // p.block_size).long()].long()
        return cache[blk.to(cache.device), (pos % p.block_size).long().to(cache.device)]

    def run(self, q_host, k_new_host, v_new_host, out_host, lse_host, stream=None):
        """Host tensors (pinned for overlap): q [C, Hq, Dqk], k_new [C, Hkv, Dqk], v_new [C, Hkv, Dv] (None under MLA
        aliasing), out [C, Hq, Dv], lse [C, Hq] or None.  Enqueues everything; `stream` ends up waiting for the last
        device -> host copy."""
        h = self.hargs
        h.q_host, h.k_new_host = q_host.data_ptr(), k_new_host.data_ptr()
        h.v_new_host = v_new_host.data_ptr() if v_new_host is not None else None
        h.out_host = out_host.data_ptr()
        h.lse_host = lse_host.data_ptr() if lse_host is not None else None
        vpp_chunk_attn_host_fwd(h, stream)


