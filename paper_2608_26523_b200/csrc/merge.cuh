// Merge of split-KV partial results (fp32 normalised partial outputs + their log-sum-exp):
//   lse = ln sum_s exp(lse_s),  out = sum_s exp(lse_s - lse) * o_s
// One warp per (query row, q-head) pair, kMergePairs pairs per trip of a grid-stride loop.  Lane s holds
// the weight of split s (the log-sum-exp values of a pair are read once, by up to 32 lanes in parallel);
// the first batch of partial rows of every pair of the trip is requested before any weight is needed,
// so the two dependent round trips to memory overlap and each lane keeps kMergePairs*kMergeBatch 16-byte
// loads in flight.  HBM-bound: S*(4*Dv+4) bytes read, 2*Dv+4 written per pair.
#pragma once
#include <cstdint>
#include <cuda_bf16.h>

namespace vpp {

constexpr int kMergeThreads = 256;
constexpr int kMergeBatch = 4;   // partial rows in flight per lane and pair
constexpr int kMergePairs = 2;   // pairs per trip
constexpr int kMergeMaxSplits = 64;

// row_splits: optional int32 per query row = number of partials to merge for that row; rows with
// fewer than 2 were written in final form by the attention kernel and are skipped.
// When null, every row merges exactly num_splits partials.
__global__ void __launch_bounds__(kMergeThreads)
lse_merge_kernel(const float* __restrict__ o_parts, const float* __restrict__ lse_parts, int num_splits,
                 long long total_q, int num_q_heads, int head_dim_v, const int32_t* __restrict__ row_splits,
                 __nv_bfloat16* __restrict__ out, float* __restrict__ lse) {
    asm volatile("griddepcontrol.wait;" ::: "memory");   // partials come from the attention kernel launched just before
    const long long n_pairs = total_q * num_q_heads;
    const int lane = threadIdx.x & 31;
    const long long warps_total = static_cast<long long>(gridDim.x) * (kMergeThreads / 32);
    const long long warp_id = (static_cast<long long>(blockIdx.x) * kMergeThreads + threadIdx.x) >> 5;
    const int d_first = lane * 4;

    for (long long base = warp_id; base < n_pairs; base += warps_total * kMergePairs) {
        long long pair[kMergePairs];
        int ns[kMergePairs];
        float l0[kMergePairs], l1[kMergePairs];
        float4 v[kMergePairs][kMergeBatch];
#pragma unroll
        for (int q = 0; q < kMergePairs; ++q) {
            pair[q] = base + q * warps_total;
            ns[q] = 0;
            if (pair[q] < n_pairs) {
                ns[q] = num_splits;
                if (row_splits != nullptr) {
                    ns[q] = row_splits[pair[q] / num_q_heads];
                    if (ns[q] < 2) ns[q] = 0;  // written in final form by the attention kernel
                    if (ns[q] > num_splits) ns[q] = num_splits;
                }
            }
            l0[q] = lane < ns[q] ? __ldg(lse_parts + lane * n_pairs + pair[q]) : -INFINITY;
            l1[q] = lane + 32 < ns[q] ? __ldg(lse_parts + (lane + 32) * n_pairs + pair[q]) : -INFINITY;
            if (d_first < head_dim_v) {
#pragma unroll
                for (int b = 0; b < kMergeBatch; ++b)
                    if (b < ns[q])
                        v[q][b] = __ldcs(reinterpret_cast<const float4*>(o_parts + (b * n_pairs + pair[q]) * head_dim_v + d_first));
            }
        }
#pragma unroll
        for (int q = 0; q < kMergePairs; ++q) {
            if (ns[q] == 0) continue;  // warp-uniform
            float M = fmaxf(l0[q], l1[q]);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
            float w0 = 0.f, w1 = 0.f;
            if (M != -INFINITY) {
                w0 = (l0[q] == -INFINITY) ? 0.f : __expf(l0[q] - M);
                w1 = (l1[q] == -INFINITY) ? 0.f : __expf(l1[q] - M);
            }
            float z = w0 + w1;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
            const float inv_z = (M == -INFINITY) ? 0.f : 1.f / z;
            w0 *= inv_z;
            w1 *= inv_z;

            for (int d0 = 0; d0 < head_dim_v; d0 += 128) {  // warp-uniform trip count (shuffles inside)
                const int d = d0 + d_first;
                const bool in_range = d < head_dim_v;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int s0 = 0; s0 < ns[q]; s0 += kMergeBatch) {
                    if ((d0 > 0 || s0 > 0) && in_range) {
#pragma unroll
                        for (int b = 0; b < kMergeBatch; ++b)
                            if (s0 + b < ns[q])
                                v[q][b] = __ldcs(reinterpret_cast<const float4*>(
                                    o_parts + ((s0 + b) * n_pairs + pair[q]) * head_dim_v + d));
                    }
#pragma unroll
                    for (int b = 0; b < kMergeBatch; ++b) {
                        const int s = s0 + b;
                        const float w = __shfl_sync(0xffffffffu, s < 32 ? w0 : w1, s & 31);
                        if (s < ns[q]) {
                            acc.x = fmaf(w, v[q][b].x, acc.x);
                            acc.y = fmaf(w, v[q][b].y, acc.y);
                            acc.z = fmaf(w, v[q][b].z, acc.z);
                            acc.w = fmaf(w, v[q][b].w, acc.w);
                        }
                    }
                }
                if (in_range) {
                    __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y);
                    __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z, acc.w);
                    uint2 pk;
                    pk.x = *reinterpret_cast<uint32_t*>(&lo);
                    pk.y = *reinterpret_cast<uint32_t*>(&hi);
                    __stcs(reinterpret_cast<uint2*>(out + pair[q] * head_dim_v + d), pk);
                }
            }
            if (lse != nullptr && lane == 0) lse[pair[q]] = (M == -INFINITY) ? -INFINITY : M + __logf(z);
        }
    }
}

}  // namespace vpp
