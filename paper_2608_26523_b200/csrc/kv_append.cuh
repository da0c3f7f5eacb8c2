// Paged KV-cache append: the chunk's new key / value rows go to cache positions [prefix_len, prefix_len + chunk_len)
// of their request (the step that precedes the attention of the same chunk; the paper's chunked-prefill section).
// Pure data movement, HBM-bound: every byte is read once and written once.
//
// One warp per token row.  Lane 0 finds the request of the row (binary search in the exclusive scan of chunk_len that
// every block builds in shared memory) and its page; then the lanes copy the row's (kv-head, 16-byte vector) units,
// all loads of a trip issued before the first store (up to kAppendUnroll 16-byte loads in flight per lane).
#pragma once
#include <cstdint>

namespace vpp {

constexpr int kAppendThreads = 256;
constexpr int kAppendUnroll = 4;
constexpr int kAppendMaxReqs = 8192;   // the scan of chunk_len lives in shared memory (32 KB + 4)

struct AppendParams {
    const uint4* k_new;      // [total_q, Hkv, Dqk] bf16 as 16-byte vectors
    const uint4* v_new;      // [total_q, Hkv, Dv] or null
    uint8_t* k_cache;
    uint8_t* v_cache;
    long long k_block_stride, k_token_stride, k_head_stride;   // bytes
    long long v_block_stride, v_token_stride, v_head_stride;   // bytes
    const int32_t* block_table;
    const int32_t* prefix_len;
    const int32_t* chunk_len;
    int num_reqs, max_blocks_per_req, block_shift, num_blocks;
    long long capacity;      // positions a request can hold: max_blocks_per_req * block_size (or the contiguous extent)
    int total_q, num_kv_heads;
    int k_vecs, v_vecs;      // 16-byte vectors per (token, kv-head) row of K and of V (0 when v_new is null)
    int32_t* status;
};

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__global__ void __launch_bounds__(kAppendThreads) kv_append_kernel(const AppendParams p) {
    extern __shared__ int32_t cu[];   // cu[r] = rows before request r; cu[num_reqs] = total
    __shared__ int s_bad;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) s_bad = 0;
    __syncthreads();
    if (warp == 0) {
        int carry = 0;
        for (int base = 0; base < p.num_reqs; base += 32) {
            const int r = base + lane;
            int c = 0;
            if (r < p.num_reqs) {
                c = p.chunk_len[r];
                const int pre = p.prefix_len[r];
                if (c < 0 || pre < 0 || static_cast<long long>(pre) + c > p.capacity) {
                    s_bad = 1;
                    c = 0;
                }
            }
            int x = c;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int y = __shfl_up_sync(0xffffffffu, x, o);
                if (lane >= o) x += y;
            }
            if (r < p.num_reqs) cu[r] = carry + x - c;
            carry += __shfl_sync(0xffffffffu, x, 31);
        }
        if (lane == 0) cu[p.num_reqs] = carry;
    }
    __syncthreads();
    if (s_bad || cu[p.num_reqs] != p.total_q) {
        // lengths that do not describe this launch: write nothing
        if (tid == 0 && blockIdx.x == 0 && p.status) atomicCAS(p.status, 0, 1 /* VPP_DEV_BAD_LENGTHS */);
        return;
    }
    const int units_k = p.num_kv_heads * p.k_vecs, units = units_k + p.num_kv_heads * p.v_vecs;
    const int warps_total = gridDim.x * (kAppendThreads / 32);
    for (int row = blockIdx.x * (kAppendThreads / 32) + warp; row < p.total_q; row += warps_total) {
        long long blk = 0;
        int slot = 0;
        if (lane == 0) {
            int lo = 0, hi = p.num_reqs;          // last r with cu[r] <= row
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (cu[mid] <= row) lo = mid; else hi = mid;
            }
            const int pos = p.prefix_len[lo] + (row - cu[lo]);
            if (p.block_table == nullptr) {
                blk = lo;
                slot = pos;
            } else {
                blk = p.block_table[static_cast<long long>(lo) * p.max_blocks_per_req + (pos >> p.block_shift)];
                slot = pos & ((1 << p.block_shift) - 1);
                if (blk < 0 || blk >= p.num_blocks) {
                    if (p.status) atomicCAS(p.status, 0, 2 /* VPP_DEV_BAD_BLOCK */);
                    blk = -1;
                }
            }
        }
        blk = __shfl_sync(0xffffffffu, blk, 0);
        slot = __shfl_sync(0xffffffffu, slot, 0);
        if (blk < 0) continue;   // the row's page is not valid: skip the row
        uint8_t* k_dst = p.k_cache + blk * p.k_block_stride + slot * p.k_token_stride;
        uint8_t* v_dst = p.v_cache + blk * p.v_block_stride + slot * p.v_token_stride;
        const uint4* k_src = p.k_new + static_cast<long long>(row) * units_k;
        const uint4* v_src = p.v_new + static_cast<long long>(row) * (units - units_k);
        for (int u0 = lane; u0 < units; u0 += 32 * kAppendUnroll) {
            uint4 v[kAppendUnroll];
#pragma unroll
            for (int i = 0; i < kAppendUnroll; ++i) {
                const int u = u0 + 32 * i;
                if (u < units) v[i] = ld_stream(u < units_k ? k_src + u : v_src + (u - units_k));
            }
#pragma unroll
            for (int i = 0; i < kAppendUnroll; ++i) {
                const int u = u0 + 32 * i;
                if (u >= units) continue;
                if (u < units_k) {
                    const int g = u / p.k_vecs, j = u - g * p.k_vecs;
                    *reinterpret_cast<uint4*>(k_dst + g * p.k_head_stride + j * 16) = v[i];
                } else {
                    const int w = u - units_k, g = w / p.v_vecs, j = w - g * p.v_vecs;
                    *reinterpret_cast<uint4*>(v_dst + g * p.v_head_stride + j * 16) = v[i];
                }
            }
        }
    }
}

}  // namespace vpp
