"""Host-side behaviour of the C ABI that needs no GPU: the library loads, exports every symbol that
include/vpp.h declares, sizes workspaces, and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest
import torch

from paper_2608_26523_b200 import api, workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2608_26523_b200 import build
    build.build()                      # nvcc cross-compiles without a GPU
    return api.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "vpp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(vpp_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert {"vpp_chunk_attn_fwd", "vpp_lse_merge", "vpp_chunk_attn_workspace_size",
            "vpp_chunk_attn_fwd_static"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert set(api.EXPORTS) == set(names)


def test_status_strings(lib):
    for code in (0, -1, -2, -3, -4, -5):
        assert lib.vpp_status_string(code).decode() != "unknown status"
    assert lib.vpp_status_string(-99).decode() == "unknown status"


def small_args(**kw):
    p = W.make_problem(5, [10], [20], kw.pop("hq", 4), kw.pop("hkv", 2), kw.pop("dqk", 128), kw.pop("dv", 128),
                       block_size=kw.pop("block_size", 16), v_aliases_k=kw.pop("alias", False))
    a = api.make_args(p.q, p.k_cache, p.v_cache, p.block_table, p.prefix_len, p.chunk_len, p.block_size,
                      p.max_seq_len, p.scale, **kw)
    a._keep = p
    return a


def test_workspace_size_grows_with_splits(lib):
    base = api.vpp_chunk_attn_workspace_size(small_args(num_kv_splits=1))
    split = api.vpp_chunk_attn_workspace_size(small_args(num_kv_splits=4))
    assert 0 < base < split
    # partials: S * T * Hq * (Dv + 1) floats
    assert split - base >= 4 * 20 * 4 * 129 * 4


def test_layout_of_args_struct_matches_header(tmp_path):
    """The ctypes mirror has the size and field offsets a C compiler gives the header's struct."""
    import subprocess
    src = tmp_path / "layout.c"
    src.write_text('#include <stdio.h>\n#include <stddef.h>\n#include "vpp.h"\n'
                   'int main(void){printf("%zu %zu %zu %zu %zu %zu\\n", sizeof(vpp_chunk_attn_args),'
                   'offsetof(vpp_chunk_attn_args, block_table), offsetof(vpp_chunk_attn_args, num_reqs),'
                   'offsetof(vpp_chunk_attn_args, softmax_scale), offsetof(vpp_chunk_attn_args, out),'
                   'offsetof(vpp_chunk_attn_args, status));return 0;}\n')
    exe = tmp_path / "layout"
    subprocess.check_call(["gcc", "-I", os.path.join(ROOT, "include"), "-o", str(exe), str(src)])
    c = [int(x) for x in subprocess.check_output([str(exe)]).split()]
    A = api.ChunkAttnArgs
    assert c == [ctypes.sizeof(A), A.block_table.offset, A.num_reqs.offset, A.softmax_scale.offset, A.out.offset,
                 A.status.offset]


def test_layout_of_append_args_matches_header(tmp_path):
    import subprocess
    src = tmp_path / "layout2.c"
    src.write_text('#include <stdio.h>\n#include <stddef.h>\n#include "vpp.h"\n'
                   'int main(void){printf("%zu %zu %zu %zu %zu\\n", sizeof(vpp_kv_append_args),'
                   'offsetof(vpp_kv_append_args, k_cache), offsetof(vpp_kv_append_args, block_table),'
                   'offsetof(vpp_kv_append_args, num_reqs), offsetof(vpp_kv_append_args, status));return 0;}\n')
    exe = tmp_path / "layout2"
    subprocess.check_call(["gcc", "-I", os.path.join(ROOT, "include"), "-o", str(exe), str(src)])
    c = [int(x) for x in subprocess.check_output([str(exe)]).split()]
    A = api.KvAppendArgs
    assert c == [ctypes.sizeof(A), A.k_cache.offset, A.block_table.offset, A.num_reqs.offset, A.status.offset]


@pytest.mark.parametrize("mutate,status", [
    (lambda a: setattr(a, "head_dim_qk", 96), api.VPP_ERR_UNSUPPORTED),
    (lambda a: setattr(a, "num_kv_heads", 3), api.VPP_ERR_INVALID_ARG),
    (lambda a: setattr(a, "softmax_scale", 0.0), api.VPP_ERR_INVALID_ARG),
    (lambda a: setattr(a, "num_kv_splits", 65), api.VPP_ERR_INVALID_ARG),
    (lambda a: setattr(a, "block_size", 24), api.VPP_ERR_UNSUPPORTED),
    (lambda a: setattr(a, "k_token_stride", 100), api.VPP_ERR_INVALID_ARG),
    (lambda a: setattr(a, "q", None), api.VPP_ERR_INVALID_ARG),
    (lambda a: setattr(a, "q", a.q + 2), api.VPP_ERR_INVALID_ARG),          # misaligned
    (lambda a: setattr(a, "workspace_bytes", 16), api.VPP_ERR_WORKSPACE),
])
def test_bad_arguments_are_rejected_before_any_launch(lib, mutate, status):
    a = small_args()
    ws = torch.zeros(1 << 20, dtype=torch.uint8)
    out = torch.zeros(20, 4, 128, dtype=torch.bfloat16)
    a.workspace, a.workspace_bytes, a.out = ws.data_ptr() + (-ws.data_ptr() % 256), 1 << 19, out.data_ptr()
    mutate(a)
    with pytest.raises(api.VppError) as ei:
        api.vpp_chunk_attn_fwd(a, stream=0)
    assert ei.value.status == status
    assert str(ei.value)


def test_mla_shape_needs_aliased_values(lib):
    a = small_args(hq=4, hkv=1, dqk=576, dv=512, alias=True)
    ws = torch.zeros(1 << 22, dtype=torch.uint8)
    out = torch.zeros(20, 4, 512, dtype=torch.bfloat16)
    a.workspace, a.workspace_bytes, a.out = ws.data_ptr() + (-ws.data_ptr() % 256), 1 << 21, out.data_ptr()
    a.v_cache = a.v_cache + 1152
    with pytest.raises(api.VppError) as ei:
        api.vpp_chunk_attn_fwd(a, stream=0)
    assert ei.value.status == api.VPP_ERR_UNSUPPORTED


def test_merge_argument_checks(lib):
    with pytest.raises(api.VppError) as ei:
        _check = lib.vpp_lse_merge(None, None, 0, 4, 4, 128, None, None, None)
        api._check(_check)
    assert ei.value.status == api.VPP_ERR_INVALID_ARG
    rc = lib.vpp_lse_merge(None, None, 65, 4, 4, 128, None, None, None)
    assert rc == api.VPP_ERR_UNSUPPORTED
    assert lib.vpp_lse_merge(None, None, 2, 0, 4, 128, None, None, None) == api.VPP_OK     # nothing to do


def test_static_entry_point_refuses_oversized_launch_on_host(lib):
    p = W.make_problem(6, [0], [4096], 8, 2, 128, 128, block_size=128)
    a = api.make_args(p.q, p.k_cache, p.v_cache, p.block_table, p.prefix_len, p.chunk_len, p.block_size,
                      p.max_seq_len, p.scale, num_kv_splits=16)
    assert api.vpp_chunk_attn_workspace_size(a) > api.vpp_static_scratch_bytes()
    with pytest.raises(api.VppError) as ei:
        api.vpp_chunk_attn_fwd_static(a, stream=0)
    assert ei.value.status == api.VPP_ERR_WORKSPACE


def test_cfg5_lengths_recipe():
    L, C, P = W.cfg5_lengths()
    assert len(L) == 32 and sum(C) == 16384
    assert all(1024 <= l <= 262144 for l in L)
    assert all(64 <= c <= min(l, 2048) for c, l in zip(C, L))
    assert all(0 <= p <= l - c for p, c, l in zip(P, C, L))
    assert W.cfg5_lengths() == (L, C, P)            # seeded


def test_flop_count_is_the_exact_causal_count():
    p = W.make_problem(7, [5, 0], [3, 2], 4, 2, 16, 8, block_size=None)
    pairs = (3 * 5 + 3 * 4 // 2) + (2 * 0 + 2 * 3 // 2)
    assert p.pairs() == pairs and p.flops() == 2 * 4 * (16 + 8) * pairs


def _host_plan_args(prefix, chunk, hq, hkv, dqk=128, dv=128, slices=None):
    h = api.HostChunkAttnArgs()
    h.dev.num_reqs, h.dev.total_q, h.dev.max_seq_len = 1, chunk, prefix + chunk
    h.dev.num_q_heads, h.dev.num_kv_heads, h.dev.head_dim_qk, h.dev.head_dim_v = hq, hkv, dqk, dv
    h.prefix_len, h.chunk_len = prefix, chunk
    if slices is not None:
        keep = (ctypes.c_int32 * len(slices))(*slices)
        h.slice_rows, h.num_slices = ctypes.cast(keep, ctypes.c_void_p), len(slices)
        h._keep = keep
    return h


def test_host_entry_point_slice_plan():
    """The planner of vpp_chunk_attn_host_fwd is host arithmetic: whole 128-row tiles that cover the chunk; ragged or
    short chunks in one slice; given slices are checked."""
    for prefix, chunk, hq, hkv in [(65536, 8192, 64, 4), (0, 8192, 64, 8), (256, 512, 8, 2), (4096, 1024, 16, 16)]:
        plan = api.vpp_chunk_attn_host_plan(_host_plan_args(prefix, chunk, hq, hkv))
        assert len(plan) == 3 and sum(plan) == chunk and all(n > 0 and n % 128 == 0 for n in plan)
    # the benchmark's chunk: first and last slice close to two full waves of work items, the middle one to ten
    assert api.vpp_chunk_attn_host_plan(_host_plan_args(65536, 8192, 64, 4)) == [1152, 5888, 1152]
    assert api.vpp_chunk_attn_host_plan(_host_plan_args(100, 333, 8, 2)) == [333]
    assert api.vpp_chunk_attn_host_plan(_host_plan_args(0, 256, 8, 2)) == [256]
    assert api.vpp_chunk_attn_host_plan(_host_plan_args(0, 512, 8, 2, slices=[100, 412])) == [100, 412]
    lib = api.load_library()
    for bad in [_host_plan_args(0, 512, 8, 2, slices=[100, 400]), _host_plan_args(0, 512, 8, 2, slices=[600, -88]),
                _host_plan_args(0, 512, 8, 3), _host_plan_args(0, 512, 8, 2, slices=[32] * 16 + [0])]:
        assert api.vpp_chunk_attn_host_plan(bad) == [] and lib.vpp_host_last_error() != b""
    bad = _host_plan_args(0, 512, 8, 2)
    bad.dev.num_reqs = 2
    assert api.vpp_chunk_attn_host_plan(bad) == [] and api.vpp_chunk_attn_host_workspace_size(bad) == 0
    bad = _host_plan_args(10, 512, 8, 2)
    bad.dev.max_seq_len = 500
    assert api.vpp_chunk_attn_host_plan(bad) == []


def test_host_entry_point_workspace_is_the_sum_of_its_slices():
    h = _host_plan_args(65536, 8192, 64, 4)
    h.dev.block_size, h.dev.max_blocks_per_req, h.dev.num_blocks = 128, 640, 640
    h.dev.k_block_stride = h.dev.v_block_stride = 128 * 4 * 128
    h.dev.k_token_stride = h.dev.v_token_stride = 4 * 128
    h.dev.k_head_stride = h.dev.v_head_stride = 128
    h.dev.softmax_scale = 0.088
    fake = ctypes.c_void_p(1 << 20)
    h.dev.q = h.dev.k_cache = h.dev.v_cache = h.dev.block_table = h.dev.prefix_len = h.dev.chunk_len = h.dev.out = fake
    total = api.vpp_chunk_attn_host_workspace_size(h)
    parts = 0
    for rows in (1152, 5888, 1152):
        a = api.ChunkAttnArgs.from_buffer_copy(h.dev)
        a.total_q = rows
        parts += (api.vpp_chunk_attn_workspace_size(a) + 255) // 256 * 256
    assert total == 256 + parts


def _fake_args(total_q, num_reqs, hq, hkv, max_seq_len, num_kv_splits):
    """Arguments with placeholder pointers: the workspace query is pure host code and never dereferences them."""
    a = api.ChunkAttnArgs()
    fake = ctypes.c_void_p(1 << 20)
    a.q = a.k_cache = a.v_cache = a.block_table = a.prefix_len = a.chunk_len = a.out = fake
    a.k_block_stride = a.v_block_stride = 128 * hkv * 128
    a.k_token_stride = a.v_token_stride = hkv * 128
    a.k_head_stride = a.v_head_stride = 128
    a.num_reqs, a.max_blocks_per_req, a.block_size, a.num_blocks = num_reqs, (max_seq_len + 127) // 128, 128, 1 << 16
    a.total_q, a.max_seq_len = total_q, max_seq_len
    a.num_q_heads, a.num_kv_heads, a.head_dim_qk, a.head_dim_v = hq, hkv, 128, 128
    a.softmax_scale = 0.088
    a.num_kv_splits = num_kv_splits
    return a


def _chosen_splits(total_q, num_reqs, hq, hkv, max_seq_len):
    auto = api.vpp_chunk_attn_workspace_size(_fake_args(total_q, num_reqs, hq, hkv, max_seq_len, 0))
    assert auto > 0
    for s in range(1, 17):
        if api.vpp_chunk_attn_workspace_size(_fake_args(total_q, num_reqs, hq, hkv, max_seq_len, s)) == auto:
            return s
    raise AssertionError("no forced split count reproduces the automatic workspace size")


def test_split_choice_fills_whole_waves(lib):
    """148 SMs assumed on a box without a GPU.  One request, d = 128: the split count whose equal work items leave the
    least idle last wave, after the measured cost of splitting (the picks below are the measured optima)."""
    if torch.cuda.is_available() and torch.cuda.get_device_properties(0).multi_processor_count != 148:
        pytest.skip("the expectations are for 148 SMs")
    assert _chosen_splits(8192, 1, 64, 4, 73728) == 1      # 2048 items: 13.8 waves
    assert _chosen_splits(8192, 1, 32, 4, 73728) == 1      # 1024 items: 6.92 waves
    assert _chosen_splits(8192, 1, 16, 2, 73728) == 2      # 512 items: 3.46 -> 6.92 waves
    assert _chosen_splits(8192, 1, 8, 1, 73728) == 4       # 256 items: 1.73 -> 6.92 waves
    assert _chosen_splits(4096, 1, 8, 1, 36864) == 1       # 128 items at a shorter prefix: splitting costs more than it saves
    # decode batches: one packed item per (token, kv-head)
    assert _chosen_splits(64, 64, 64, 8, 32769) == 2       # 512 items
    assert _chosen_splits(64, 64, 64, 4, 32769) == 4       # 256 items
    assert _chosen_splits(256, 256, 64, 8, 8193) == 1      # 2048 items
    assert _chosen_splits(32, 32, 64, 8, 8193) == 1        # 256 short items: the start-up of more units outweighs the wave


def test_tensor_map_cache_encodes_once_per_distinct_map(lib):
    """The cache logic with a stand-in for the driver's encoder: five identical look-ups, one with another extent and
    one with another base address take three encodes, and a hit returns the bytes the encoder produced."""
    assert lib.vpp_test_tensor_map_cache(5) == 3
    assert lib.vpp_test_tensor_map_cache(7) == 0          # everything is cached by now
    lookups, encodes = api.vpp_tensor_map_cache_stats()   # the library's own cache: untouched without a launch
    assert lookups >= 0 and encodes <= lookups


def test_contiguous_cache_regions_must_hold_max_seq_len_slots(lib):
    """Two requests in an unpaged cache whose regions are 40 slots apart, with max_seq_len = 64: the kernels would fetch
    key tiles up to slot 64 of the last region, past the allocation.  The call refuses on the host; nothing is launched."""
    p = W.make_problem(8, [10, 12], [20, 8], 4, 2, 128, 128, block_size=None)
    slots = p.k_cache.shape[1]
    a = api.make_args(p.q, p.k_cache, p.v_cache, None, p.prefix_len, p.chunk_len, 0, slots + 24, p.scale)
    ws = torch.zeros(1 << 20, dtype=torch.uint8)
    out = torch.zeros(28, 4, 128, dtype=torch.bfloat16)
    a.workspace, a.workspace_bytes, a.out = ws.data_ptr() + (-ws.data_ptr() % 256), 1 << 19, out.data_ptr()
    with pytest.raises(api.VppError) as ei:
        api.vpp_chunk_attn_fwd(a, stream=0)
    assert ei.value.status == api.VPP_ERR_INVALID_ARG and "max_seq_len" in str(ei.value)


def test_unsupported_head_dim_gives_the_same_status_from_both_entry_points(lib):
    a = small_args(dqk=96, dv=96)
    ws = torch.zeros(1 << 20, dtype=torch.uint8)
    out = torch.zeros(20, 4, 96, dtype=torch.bfloat16)
    a.workspace, a.workspace_bytes, a.out = ws.data_ptr() + (-ws.data_ptr() % 256), 1 << 19, out.data_ptr()
    assert api.vpp_chunk_attn_workspace_size(a) == 0
    for call in (api.vpp_chunk_attn_fwd, api.vpp_chunk_attn_fwd_static):
        with pytest.raises(api.VppError) as ei:
            call(a, stream=0)
        assert ei.value.status == api.VPP_ERR_UNSUPPORTED, call.__name__
    b = small_args()
    b.num_kv_heads = 3                                  # 4 q-heads over 3 kv-heads: invalid, not unsupported
    for call in (api.vpp_chunk_attn_fwd, api.vpp_chunk_attn_fwd_static):
        with pytest.raises(api.VppError) as ei:
            call(b, stream=0)
        assert ei.value.status == api.VPP_ERR_INVALID_ARG, call.__name__


@pytest.mark.parametrize("kv_begin,kv_end", [(-128, 128), (64, 256), (128, 128), (256, 128), (0, 200)])
def test_partial_entry_point_checks_its_key_range(lib, kv_begin, kv_end):
    p = W.make_problem(9, [600], [100], 4, 2, 128, 128, block_size=64)
    a = api.make_args(p.q, p.k_cache, p.v_cache, p.block_table, p.prefix_len, p.chunk_len, p.block_size,
                      p.max_seq_len, p.scale)
    ws = torch.zeros(1 << 20, dtype=torch.uint8)
    a.workspace, a.workspace_bytes = ws.data_ptr() + (-ws.data_ptr() % 256), 1 << 19
    o = torch.zeros(100, 4, 128, dtype=torch.float32)
    l = torch.zeros(100, 4, dtype=torch.float32)
    with pytest.raises(api.VppError) as ei:
        api.vpp_chunk_attn_partial_fwd(a, kv_begin, kv_end, o, l, stream=0)
    assert ei.value.status == api.VPP_ERR_INVALID_ARG


def test_bounded_wait_hook_checks_its_arguments(lib):
    assert lib.vpp_test_bounded_wait(None, 1000, None) == api.VPP_ERR_INVALID_ARG
    st = torch.zeros(1, dtype=torch.int32)
    assert lib.vpp_test_bounded_wait(st.data_ptr(), 0, None) == api.VPP_ERR_INVALID_ARG
    assert lib.vpp_test_bounded_wait(st.data_ptr(), 1 << 40, None) == api.VPP_ERR_INVALID_ARG


def test_cost_curve_fit_and_balance_identity_of_the_benchmark():
    """bench.py's evaluation of the paper's Eq. 2 (affine latency) and Eq. 3 (tau(k-1) + tau(k+1) = 2 tau(k)) on a measured
    curve: exact on an affine curve, and the residual of a known bend on the evenly spaced triples only."""
    import importlib.util
    spec = importlib.util.spec_from_file_location("bench", os.path.join(ROOT, "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    xs = [0, 8192, 32768, 65536, 98304, 131072]
    fit = bench.fit_cost_curve(xs, [1.0 + 2e-4 * x for x in xs])
    assert abs(fit["fit_ms"]["a"] - 1.0) < 1e-4 and abs(fit["fit_ms"]["b_per_token"] - 2e-4) < 1e-9
    assert fit["eq3_residual_max"] < 1e-9 and fit["eq3_triples"] == 4      # (0,32K,64K) (32K,64K,96K) (64K,96K,128K) (0,64K,128K)
    bent = bench.fit_cost_curve([0, 100, 200], [1.0, 2.0, 4.0])
    assert abs(bent["eq3_residual_max"] - abs(1.0 + 4.0 - 4.0) / 4.0) < 1e-4
    assert bench.fit_cost_curve([0, 100], [1.0, 2.0]) is None
    rec = bench.read_traffic_record("attn128_ws_cfg2_traffic.txt")
    assert rec["prefix"] == "131072" and float(rec["dram_bytes_read"]) > 0 and rec["kernel"] == "attn128_ws_kernel"
