"""The boundary used the way a C caller uses it: a plain C program, compiled against include/vpp.h and linked with the shared
library and the CUDA runtime only (no Python, no torch in the process), reads a problem from a file, allocates device memory
itself, calls vpp_chunk_attn_workspace_size / vpp_kv_append / vpp_chunk_attn_fwd and writes out and lse back.  The test
compares what it wrote with the CPU oracle."""
import os
import shutil
import subprocess

import numpy as np
import pytest
import torch

import oracle
from paper_2608_26523_b200 import api, workloads as W
from parity import compare

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

C_SOURCE = r'''
#include <cuda_runtime_api.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include "vpp.h"

#define CK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { fprintf(stderr, "%s: %s\n", #x, cudaGetErrorString(e_)); return 2; } } while (0)

static void* slurp(FILE* f, size_t bytes) {
    void* p = malloc(bytes ? bytes : 1);
    if (fread(p, 1, bytes, f) != bytes) { fprintf(stderr, "short read\n"); exit(3); }
    return p;
}

int main(int argc, char** argv) {
    if (argc != 3) return 1;
    FILE* f = fopen(argv[1], "rb");
    if (!f) return 1;
    int32_t h[12];   /* R, T, Hq, Hkv, D, B, num_blocks, max_blocks, max_seq, splits, chunk_rows_to_append, pad */
    if (fread(h, 4, 12, f) != 12) return 3;
    const int R = h[0], T = h[1], Hq = h[2], Hkv = h[3], D = h[4], B = h[5], NB = h[6], MB = h[7], MAXSEQ = h[8], S = h[9];
    float scale;
    if (fread(&scale, 4, 1, f) != 1) return 3;
    const size_t q_bytes = (size_t)T * Hq * D * 2, c_bytes = (size_t)NB * B * Hkv * D * 2, n_bytes = (size_t)T * Hkv * D * 2;
    void* q = slurp(f, q_bytes);
    void* kc = slurp(f, c_bytes);      /* cache WITHOUT the chunk's own rows: the program appends them */
    void* vc = slurp(f, c_bytes);
    void* kn = slurp(f, n_bytes);
    void* vn = slurp(f, n_bytes);
    int32_t* bt = (int32_t*)slurp(f, (size_t)R * MB * 4);
    int32_t* pre = (int32_t*)slurp(f, (size_t)R * 4);
    int32_t* chk = (int32_t*)slurp(f, (size_t)R * 4);
    fclose(f);

    void *dq, *dk, *dv, *dkn, *dvn, *dbt, *dpre, *dchk, *dout, *dlse, *dws, *dst;
    CK(cudaMalloc(&dq, q_bytes)); CK(cudaMalloc(&dk, c_bytes)); CK(cudaMalloc(&dv, c_bytes));
    CK(cudaMalloc(&dkn, n_bytes)); CK(cudaMalloc(&dvn, n_bytes));
    CK(cudaMalloc(&dbt, (size_t)R * MB * 4)); CK(cudaMalloc(&dpre, R * 4)); CK(cudaMalloc(&dchk, R * 4));
    CK(cudaMalloc(&dout, (size_t)T * Hq * D * 2)); CK(cudaMalloc(&dlse, (size_t)T * Hq * 4)); CK(cudaMalloc(&dst, 8));
    CK(cudaMemcpy(dq, q, q_bytes, cudaMemcpyHostToDevice)); CK(cudaMemcpy(dk, kc, c_bytes, cudaMemcpyHostToDevice));
    CK(cudaMemcpy(dv, vc, c_bytes, cudaMemcpyHostToDevice)); CK(cudaMemcpy(dkn, kn, n_bytes, cudaMemcpyHostToDevice));
    CK(cudaMemcpy(dvn, vn, n_bytes, cudaMemcpyHostToDevice)); CK(cudaMemcpy(dbt, bt, (size_t)R * MB * 4, cudaMemcpyHostToDevice));
    CK(cudaMemcpy(dpre, pre, R * 4, cudaMemcpyHostToDevice)); CK(cudaMemcpy(dchk, chk, R * 4, cudaMemcpyHostToDevice));
    cudaStream_t stream;
    CK(cudaStreamCreate(&stream));

    vpp_kv_append_args ap = {0};
    ap.k_new = dkn; ap.v_new = dvn; ap.k_cache = dk; ap.v_cache = dv;
    ap.k_block_stride = ap.v_block_stride = (int64_t)B * Hkv * D;
    ap.k_token_stride = ap.v_token_stride = (int64_t)Hkv * D;
    ap.k_head_stride = ap.v_head_stride = D;
    ap.block_table = (const int32_t*)dbt; ap.prefix_len = (const int32_t*)dpre; ap.chunk_len = (const int32_t*)dchk;
    ap.num_reqs = R; ap.max_blocks_per_req = MB; ap.block_size = B; ap.num_blocks = NB; ap.total_q = T; ap.max_seq_len = MAXSEQ;
    ap.num_kv_heads = Hkv; ap.head_dim_qk = D; ap.head_dim_v = D; ap.status = (int32_t*)dst;
    vpp_status st = vpp_kv_append(&ap, stream);
    if (st != VPP_OK) { fprintf(stderr, "append: %s: %s\n", vpp_status_string(st), vpp_last_error()); return 4; }

    vpp_chunk_attn_args a = {0};
    a.q = dq; a.k_cache = dk; a.v_cache = dv;
    a.k_block_stride = a.v_block_stride = ap.k_block_stride;
    a.k_token_stride = a.v_token_stride = ap.k_token_stride;
    a.k_head_stride = a.v_head_stride = D;
    a.block_table = (const int32_t*)dbt; a.prefix_len = (const int32_t*)dpre; a.chunk_len = (const int32_t*)dchk;
    a.num_reqs = R; a.max_blocks_per_req = MB; a.block_size = B; a.num_blocks = NB; a.total_q = T; a.max_seq_len = MAXSEQ;
    a.num_q_heads = Hq; a.num_kv_heads = Hkv; a.head_dim_qk = D; a.head_dim_v = D; a.softmax_scale = scale; a.num_kv_splits = S;
    a.out = dout; a.lse = (float*)dlse; a.status = (int32_t*)dst + 1;
    const size_t ws = vpp_chunk_attn_workspace_size(&a);
    if (ws == 0) { fprintf(stderr, "workspace query: %s\n", vpp_last_error()); return 5; }
    CK(cudaMalloc(&dws, ws));
    a.workspace = dws; a.workspace_bytes = ws;
    st = vpp_chunk_attn_fwd(&a, stream);
    if (st != VPP_OK) { fprintf(stderr, "attention: %s: %s\n", vpp_status_string(st), vpp_last_error()); return 6; }
    CK(cudaStreamSynchronize(stream));
    int32_t status[2];
    CK(cudaMemcpy(status, dst, 8, cudaMemcpyDeviceToHost));
    if (status[0] || status[1]) { fprintf(stderr, "device status %d %d\n", status[0], status[1]); return 7; }

    void* out = malloc((size_t)T * Hq * D * 2);
    float* lse = (float*)malloc((size_t)T * Hq * 4);
    CK(cudaMemcpy(out, dout, (size_t)T * Hq * D * 2, cudaMemcpyDeviceToHost));
    CK(cudaMemcpy(lse, dlse, (size_t)T * Hq * 4, cudaMemcpyDeviceToHost));
    FILE* g = fopen(argv[2], "wb");
    fwrite(out, 1, (size_t)T * Hq * D * 2, g);
    fwrite(lse, 1, (size_t)T * Hq * 4, g);
    fclose(g);
    printf("launches %d workspace %zu\n", (int)vpp_last_launch_count(), ws);
    return 0;
}
'''


C_SOURCE_HOST = r'''
#include <cuda_runtime_api.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
#include "vpp.h"

#define CK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { fprintf(stderr, "%s: %s\n", #x, cudaGetErrorString(e_)); return 2; } } while (0)

/* one request's chunk from page-locked host memory through vpp_chunk_attn_host_fwd */
int main(int argc, char** argv) {
    if (argc != 3) return 1;
    FILE* f = fopen(argv[1], "rb");
    if (!f) return 1;
    int32_t h[12];   /* P, C, Hq, Hkv, D, B, num_blocks, max_blocks, max_seq, splits */
    if (fread(h, 4, 12, f) != 12) return 3;
    const int P = h[0], C = h[1], Hq = h[2], Hkv = h[3], D = h[4], B = h[5], NB = h[6], MB = h[7], MAXSEQ = h[8], S = h[9];
    float scale;
    if (fread(&scale, 4, 1, f) != 1) return 3;
    const size_t q_bytes = (size_t)C * Hq * D * 2, n_bytes = (size_t)C * Hkv * D * 2, c_bytes = (size_t)NB * B * Hkv * D * 2;
    void *q, *kn, *vn, *out; float* lse;
    CK(cudaMallocHost(&q, q_bytes)); CK(cudaMallocHost(&kn, n_bytes)); CK(cudaMallocHost(&vn, n_bytes));
    CK(cudaMallocHost(&out, q_bytes)); CK(cudaMallocHost((void**)&lse, (size_t)C * Hq * 4));
    void* cache = malloc(2 * c_bytes);
    int32_t* bt = (int32_t*)malloc((size_t)MB * 4);
    if (fread(q, 1, q_bytes, f) != q_bytes || fread(cache, 1, 2 * c_bytes, f) != 2 * c_bytes || fread(kn, 1, n_bytes, f) != n_bytes ||
        fread(vn, 1, n_bytes, f) != n_bytes || fread(bt, 4, MB, f) != (size_t)MB) return 3;
    fclose(f);
    void *dq, *dk, *dv, *dkn, *dvn, *dbt, *dout, *dlse, *dst, *dws;
    CK(cudaMalloc(&dq, q_bytes)); CK(cudaMalloc(&dk, c_bytes)); CK(cudaMalloc(&dv, c_bytes)); CK(cudaMalloc(&dkn, n_bytes));
    CK(cudaMalloc(&dvn, n_bytes)); CK(cudaMalloc(&dbt, (size_t)MB * 4)); CK(cudaMalloc(&dout, q_bytes));
    CK(cudaMalloc(&dlse, (size_t)C * Hq * 4)); CK(cudaMalloc(&dst, 4));
    CK(cudaMemcpy(dk, cache, c_bytes, cudaMemcpyHostToDevice));
    CK(cudaMemcpy(dv, (char*)cache + c_bytes, c_bytes, cudaMemcpyHostToDevice));
    CK(cudaMemcpy(dbt, bt, (size_t)MB * 4, cudaMemcpyHostToDevice));
    cudaStream_t stream;
    CK(cudaStreamCreate(&stream));

    vpp_chunk_attn_host_args a;
    memset(&a, 0, sizeof a);
    a.q_host = q; a.k_new_host = kn; a.v_new_host = vn; a.out_host = out; a.lse_host = lse;
    a.prefix_len = P; a.chunk_len = C;
    a.dev.q = dq; a.dev.k_cache = dk; a.dev.v_cache = dv;
    a.dev.k_block_stride = a.dev.v_block_stride = (int64_t)B * Hkv * D;
    a.dev.k_token_stride = a.dev.v_token_stride = (int64_t)Hkv * D;
    a.dev.k_head_stride = a.dev.v_head_stride = D;
    a.dev.block_table = (const int32_t*)dbt;
    a.dev.num_reqs = 1; a.dev.max_blocks_per_req = MB; a.dev.block_size = B; a.dev.num_blocks = NB; a.dev.total_q = C;
    a.dev.max_seq_len = MAXSEQ; a.dev.num_q_heads = Hq; a.dev.num_kv_heads = Hkv; a.dev.head_dim_qk = D; a.dev.head_dim_v = D;
    a.dev.softmax_scale = scale; a.dev.num_kv_splits = S; a.dev.out = dout; a.dev.lse = (float*)dlse; a.dev.status = (int32_t*)dst;
    a.k_new_dev = dkn; a.v_new_dev = dvn;
    int32_t plan[VPP_HOST_MAX_SLICES];
    const int n = vpp_chunk_attn_host_plan(&a, plan);
    const size_t ws = vpp_chunk_attn_host_workspace_size(&a);
    if (n == 0 || ws == 0) { fprintf(stderr, "plan: %s\n", vpp_host_last_error()); return 5; }
    CK(cudaMalloc(&dws, ws));
    a.dev.workspace = dws; a.dev.workspace_bytes = ws;
    vpp_status st = vpp_chunk_attn_host_fwd(&a, stream);
    if (st != VPP_OK) { fprintf(stderr, "%s: %s\n", vpp_status_string(st), vpp_host_last_error()); return 6; }
    CK(cudaStreamSynchronize(stream));
    int32_t status;
    CK(cudaMemcpy(&status, dst, 4, cudaMemcpyDeviceToHost));
    if (status) { fprintf(stderr, "device status %d\n", status); return 7; }
    FILE* g = fopen(argv[2], "wb");
    fwrite(out, 1, q_bytes, g);
    fwrite(lse, 1, (size_t)C * Hq * 4, g);
    fclose(g);
    printf("slices %d:", n);
    for (int i = 0; i < n; ++i) printf(" %d", plan[i]);
    printf(" workspace %zu\n", ws);
    return 0;
}
'''


def _bits(t):
    return t.contiguous().view(torch.int16).numpy().tobytes()


@pytest.mark.parametrize("splits", [0, 3])
def test_a_plain_c_program_appends_a_chunk_and_attends(tmp_path, splits):
    gcc = shutil.which("gcc")
    cuda = "/usr/local/cuda"
    if gcc is None or not os.path.exists(os.path.join(cuda, "include", "cuda_runtime_api.h")):
        pytest.skip("no C toolchain / CUDA headers on this box")
    api.load_library()                                   # (makes sure the library has been built)
    prob = W.make_problem(7100 + splits, [700, 0, 260], [300, 140, 77], 8, 2, 128, 128, block_size=64)
    R, T = prob.num_reqs, prob.total_q
    # the chunk's own K/V rows leave the cache (NaN in their place) and travel as k_new / v_new: the C program appends them
    k_new = torch.empty((T, 2, 128), dtype=torch.bfloat16)
    v_new = torch.empty((T, 2, 128), dtype=torch.bfloat16)
    kc, vc = prob.k_cache.clone(), prob.v_cache.clone()
    row = 0
    for r in range(R):
        P, C = int(prob.prefix_len[r]), int(prob.chunk_len[r])
        for i in range(C):
            pos = P + i
            blk, slot = int(prob.block_table[r, pos // 64]), pos % 64
            k_new[row], v_new[row] = prob.k_cache[blk, slot], prob.v_cache[blk, slot]
            kc[blk, slot] = float("nan")
            vc[blk, slot] = float("nan")
            row += 1
    src, exe, fin, fout = tmp_path / "client.c", tmp_path / "client", tmp_path / "in.bin", tmp_path / "out.bin"
    src.write_text(C_SOURCE)
    lib_dir = os.path.dirname(api.LIB_PATH)
    subprocess.check_call([gcc, "-O1", "-std=c11", "-I", os.path.join(ROOT, "include"), "-I", os.path.join(cuda, "include"),
                           "-o", str(exe), str(src), "-L", lib_dir, "-l:libvpp_chunk_attn.so", "-L", os.path.join(cuda, "lib64"),
                           "-lcudart", "-Wl,-rpath," + lib_dir, "-Wl,-rpath," + os.path.join(cuda, "lib64")])
    head = np.array([R, T, 8, 2, 128, 64, kc.shape[0], prob.block_table.shape[1], prob.max_seq_len, splits, 0, 0], np.int32)
    with open(fin, "wb") as f:
        f.write(head.tobytes())
        f.write(np.float32(prob.scale).tobytes())
        for t in (prob.q, kc, vc, k_new, v_new):
            f.write(_bits(t))
        f.write(prob.block_table.numpy().astype(np.int32).tobytes())
        f.write(prob.prefix_len.numpy().astype(np.int32).tobytes())
        f.write(prob.chunk_len.numpy().astype(np.int32).tobytes())
    res = subprocess.run([str(exe), str(fin), str(fout)], capture_output=True, text=True, timeout=120)
    assert res.returncode == 0, res.stderr + res.stdout
    assert "launches" in res.stdout
    raw = np.fromfile(fout, dtype=np.uint8)
    n_out = T * 8 * 128 * 2
    out = torch.from_numpy(raw[:n_out].view(np.int16).copy()).view(torch.bfloat16).view(T, 8, 128)
    lse = torch.from_numpy(raw[n_out:].view(np.float32).copy()).view(T, 8)
    rows = oracle.all_rows(prob.chunk_len.numpy(), 8)
    print(compare(out, lse, prob, rows, "C client S=%d" % splits), res.stdout.strip())


def test_a_plain_c_program_runs_a_chunk_from_host_memory(tmp_path):
    """The host entry point from plain C: page-locked buffers from cudaMallocHost, one call, results back in host memory."""
    gcc = shutil.which("gcc")
    cuda = "/usr/local/cuda"
    if gcc is None or not os.path.exists(os.path.join(cuda, "include", "cuda_runtime_api.h")):
        pytest.skip("no C toolchain / CUDA headers on this box")
    api.load_library()
    P, C = 384, 640
    prob = W.make_problem(7200, [P], [C], 8, 2, 128, 128, block_size=64)
    pos = torch.arange(P, P + C)
    blk, slot = prob.block_table[0, (pos // 64).long()].long(), (pos % 64).long()
    k_new, v_new = prob.k_cache[blk, slot].contiguous(), prob.v_cache[blk, slot].contiguous()
    kc, vc = prob.k_cache.clone(), prob.v_cache.clone()
    kc[blk, slot] = float("nan")
    vc[blk, slot] = float("nan")
    src, exe, fin, fout = tmp_path / "host_client.c", tmp_path / "host_client", tmp_path / "in.bin", tmp_path / "out.bin"
    src.write_text(C_SOURCE_HOST)
    lib_dir = os.path.dirname(api.LIB_PATH)
    subprocess.check_call([gcc, "-O1", "-std=c11", "-I", os.path.join(ROOT, "include"), "-I", os.path.join(cuda, "include"),
                           "-o", str(exe), str(src), "-L", lib_dir, "-l:libvpp_chunk_attn.so", "-L", os.path.join(cuda, "lib64"),
                           "-lcudart", "-Wl,-rpath," + lib_dir, "-Wl,-rpath," + os.path.join(cuda, "lib64")])
    head = np.array([P, C, 8, 2, 128, 64, kc.shape[0], prob.block_table.shape[1], prob.max_seq_len, 0, 0, 0], np.int32)
    with open(fin, "wb") as f:
        f.write(head.tobytes())
        f.write(np.float32(prob.scale).tobytes())
        for t in (prob.q, kc, vc, k_new, v_new):
            f.write(_bits(t))
        f.write(prob.block_table[0].numpy().astype(np.int32).tobytes())
    res = subprocess.run([str(exe), str(fin), str(fout)], capture_output=True, text=True, timeout=120)
    assert res.returncode == 0, res.stderr + res.stdout
    assert "slices 3: 128 384 128" in res.stdout or "slices 3:" in res.stdout
    raw = np.fromfile(fout, dtype=np.uint8)
    n_out = C * 8 * 128 * 2
    out = torch.from_numpy(raw[:n_out].view(np.int16).copy()).view(torch.bfloat16).view(C, 8, 128)
    lse = torch.from_numpy(raw[n_out:].view(np.float32).copy()).view(C, 8)
    rows = oracle.all_rows(prob.chunk_len.numpy(), 8)
    print(compare(out, lse, prob, rows, "C host client"), res.stdout.strip())
