// Merge of split-KV partial results (fp32 normalised partial outputs + their log-sum-exp):
//   lse = ln sum_s exp(lse_s),  out = sum_s exp(lse_s - lse) * o_s
// One warp per (query row, q-head); lanes stride the value dimension in float4.  HBM-bound.
#pragma once
#include <cstdint>
#include <cuda_bf16.h>

namespace vpp {

constexpr int kMergeThreads = 256;

// row_splits: optional int32 per query row = number of partials to merge for that row; rows with
// fewer than 2 were written in final form by the attention kernel and are skipped.
// When null, every row merges exactly num_splits partials.
__global__ void __launch_bounds__(kMergeThreads)
lse_merge_kernel(const float* __restrict__ o_parts, const float* __restrict__ lse_parts, int num_splits,
                 long long total_q, int num_q_heads, int head_dim_v, const int32_t* __restrict__ row_splits,
                 __nv_bfloat16* __restrict__ out, float* __restrict__ lse) {
    const long long n_pairs = total_q * num_q_heads;
    const long long pair = (static_cast<long long>(blockIdx.x) * kMergeThreads + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (pair >= n_pairs) return;
    int ns = num_splits;
    if (row_splits != nullptr) {
        ns = row_splits[pair / num_q_heads];
        if (ns < 2) return;
        if (ns > num_splits) ns = num_splits;
    }
    float M = -INFINITY;
    for (int s = 0; s < ns; ++s) M = fmaxf(M, __ldg(lse_parts + s * n_pairs + pair));
    float z = 0.f;
    if (M != -INFINITY)
        for (int s = 0; s < ns; ++s) z += __expf(__ldg(lse_parts + s * n_pairs + pair) - M);
    const float L = (M == -INFINITY) ? -INFINITY : M + __logf(z);
    const float inv_z = (M == -INFINITY) ? 0.f : 1.f / z;
    for (int d = lane * 4; d < head_dim_v; d += 128) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s = 0; s < ns; ++s) {
            const float ls = __ldg(lse_parts + s * n_pairs + pair);
            const float w = (ls == -INFINITY) ? 0.f : __expf(ls - M) * inv_z;
            const float4 v = __ldg(reinterpret_cast<const float4*>(o_parts + (s * n_pairs + pair) * head_dim_v + d));
            acc.x = fmaf(w, v.x, acc.x);
            acc.y = fmaf(w, v.y, acc.y);
            acc.z = fmaf(w, v.z, acc.z);
            acc.w = fmaf(w, v.w, acc.w);
        }
        __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y);
        __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z, acc.w);
        uint2 pk;
        pk.x = *reinterpret_cast<uint32_t*>(&lo);
        pk.y = *reinterpret_cast<uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(out + pair * head_dim_v + d) = pk;
    }
    if (lse != nullptr && lane == 0) lse[pair] = L;
}

}  // namespace vpp
