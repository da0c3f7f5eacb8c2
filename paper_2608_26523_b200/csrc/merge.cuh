// Merge of split-KV partial results (fp32 normalised partial outputs + their log-sum-exp):
//   lse = ln sum_s exp(lse_s),  out = sum_s exp(lse_s - lse) * o_s
// One warp per (query row, q-head) pair, kPairs pairs per trip of a grid-stride loop.  Lane s holds
// the weight of split s (the log-sum-exp values of a pair are read once, by up to 32 lanes in parallel);
// the first batch of partial rows of every pair of the trip is requested before any weight is needed,
// so the two dependent round trips to memory overlap and each lane keeps kPairs*kBatch 16-byte
// loads in flight -- eight in both instantiations: two pairs x four partial rows, or, for merges of two
// partials (too few rows per pair to fill the memory pipeline otherwise), four pairs x two rows.
// HBM-bound: S*(4*Dv+4) bytes read, 2*Dv+4 written per pair.
#pragma once
#include <cstdint>
#include <cuda_bf16.h>

namespace vpp {

constexpr int kMergeThreads = 256;
constexpr int kMergeMaxSplits = 64;
constexpr int kMergeSmallMax = 8;   // split counts up to this take the shuffle-free kernel

// row_splits: optional int32 per query row = number of partials to merge for that row; rows with
// fewer than 2 were written in final form by the attention kernel and are skipped.
// When null, every row merges exactly num_splits partials.
template <int kMergePairs /* pairs per trip */, int kMergeBatch /* partial rows in flight per lane and pair */>
__global__ void __launch_bounds__(kMergeThreads, 3)
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

// The same merge for at most kSMax (<= 8) partials, the case every launch of this library produces: one thread per
// 16-byte piece of an output row (consecutive threads take consecutive pieces, so a warp reads whole 512-byte runs of
// every partial), kPieces pieces per trip.  Each thread reads the few log-sum-exp values of its row itself (the lanes
// of a warp mostly share a row: one broadcast transaction) and forms the weights in registers -- no shuffles, no
// dependent chain between lanes -- and all kSMax * kPieces (= 8) partial loads of a trip are requested before the
// first is used.  head_dim_v must be a multiple of 4 and total_q * num_q_heads * head_dim_v / 4 below 2^31.
template <int kSMax, int kPieces>
__global__ void __launch_bounds__(kMergeThreads, 3)
lse_merge_small_kernel(const float* __restrict__ o_parts, const float* __restrict__ lse_parts, int num_splits,
                       long long total_q, int num_q_heads, int head_dim_v, const int32_t* __restrict__ row_splits,
                       __nv_bfloat16* __restrict__ out, float* __restrict__ lse) {
    asm volatile("griddepcontrol.wait;" ::: "memory");   // partials come from the attention kernel launched just before
    const long long n_pairs = total_q * num_q_heads;
    const uint32_t per_row = static_cast<uint32_t>(head_dim_v) >> 2;            // 16-byte pieces per output row
    const uint32_t n_pieces = static_cast<uint32_t>(n_pairs) * per_row;
    const uint32_t stride = gridDim.x * kMergeThreads;
    for (uint32_t base = blockIdx.x * kMergeThreads + threadIdx.x; base < n_pieces; base += stride * kPieces) {
        uint32_t pair[kPieces], piece[kPieces];
        int ns[kPieces];
        float l[kPieces][kSMax];
        float4 v[kPieces][kSMax];
#pragma unroll
        for (int u = 0; u < kPieces; ++u) {
            const uint32_t c = base + u * stride;
            ns[u] = 0;
            pair[u] = 0;
            piece[u] = 0;
            if (c < n_pieces) {
                pair[u] = c / per_row;
                piece[u] = c - pair[u] * per_row;
                ns[u] = num_splits;
                if (row_splits != nullptr) {
                    ns[u] = row_splits[pair[u] / static_cast<uint32_t>(num_q_heads)];
                    if (ns[u] < 2) ns[u] = 0;  // written in final form by the attention kernel
                    if (ns[u] > num_splits) ns[u] = num_splits;
                }
            }
#pragma unroll
            for (int s_ = 0; s_ < kSMax; ++s_) {
                l[u][s_] = -INFINITY;
                if (s_ < ns[u]) {
                    l[u][s_] = __ldg(lse_parts + s_ * n_pairs + pair[u]);
                    v[u][s_] = __ldcs(reinterpret_cast<const float4*>(o_parts + (s_ * n_pairs + pair[u]) * head_dim_v) + piece[u]);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kPieces; ++u) {
            if (ns[u] == 0) continue;
            float M = l[u][0];
#pragma unroll
            for (int s_ = 1; s_ < kSMax; ++s_) M = fmaxf(M, l[u][s_]);
            float w[kSMax], z = 0.f;
#pragma unroll
            for (int s_ = 0; s_ < kSMax; ++s_) {
                w[s_] = (l[u][s_] == -INFINITY) ? 0.f : __expf(l[u][s_] - M);   // (M = -inf only if every l is -inf)
                z += w[s_];
            }
            const float inv_z = (M == -INFINITY) ? 0.f : 1.f / z;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int s_ = 0; s_ < kSMax; ++s_) {
                if (s_ < ns[u]) {
                    const float ws = w[s_] * inv_z;
                    acc.x = fmaf(ws, v[u][s_].x, acc.x);
                    acc.y = fmaf(ws, v[u][s_].y, acc.y);
                    acc.z = fmaf(ws, v[u][s_].z, acc.z);
                    acc.w = fmaf(ws, v[u][s_].w, acc.w);
                }
            }
            __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y);
            __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z, acc.w);
            uint2 pk;
            pk.x = *reinterpret_cast<uint32_t*>(&lo);
            pk.y = *reinterpret_cast<uint32_t*>(&hi);
            __stcs(reinterpret_cast<uint2*>(out + static_cast<long long>(pair[u]) * head_dim_v) + piece[u], pk);
            if (lse != nullptr && piece[u] == 0) lse[pair[u]] = (M == -INFINITY) ? -INFINITY : M + __logf(z);
        }
    }
}

}  // namespace vpp
