// Straight-line (un-pipelined) chunked-prefill attention kernel for head_dim 128.
//
// One CTA of 128 threads walks work items (query tile x q-head x key-range split) handed out by an
// atomic counter.  Per KV tile: TMA gathers the K and V pages into 128B-swizzled shared memory, one
// thread issues tcgen05 MMAs for S = Q K^T into tensor memory, every thread owns one query row for the
// fp32 online softmax (the paper's Eq. 1 evaluated tile by tile), P goes back through shared or tensor
// memory and a second group of MMAs accumulates O += P V in tensor memory.
//
// This variant exists to validate the data path step by step and as the low-occupancy fallback for
// shapes the pipelined kernel does not take; it makes no attempt to overlap anything.
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace vpp {

constexpr int kSimpleThreads = 128;
constexpr int kSlabBytes = kTileM * 128;  // 128 rows x 64 bf16, 128B-swizzled
constexpr int kSimpleSmemBytes = 4 * 2 * kSlabBytes + 1024 /*align*/ + 256 /*barriers*/;

// Which (unit, kv-head, q-head) a flat work index means.  Units arrive sorted by decreasing cost; inside
// a block of kUnitBlock consecutive units the items are ordered kv-head-major so that CTAs running at
// the same time read the same K/V pages (L2 reuse), while blocks keep the longest-first order.
constexpr int kUnitBlock = 32;
__device__ __forceinline__ void decode_item(int w, int num_units, int items_per_unit, int per_kv_head, int& unit,
                                            int& slot) {
    const int blk_items = kUnitBlock * items_per_unit;
    const int ub = w / blk_items;
    const int rem = w - ub * blk_items;
    const int left = num_units - ub * kUnitBlock;
    const int nblk = left < kUnitBlock ? left : kUnitBlock;
    const int per_g = nblk * per_kv_head;
    const int g = rem / per_g;
    const int rem2 = rem - g * per_g;
    unit = ub * kUnitBlock + rem2 / per_kv_head;
    slot = g * per_kv_head + rem2 % per_kv_head;
}

template <bool kPInTmem>
__global__ void __launch_bounds__(kSimpleThreads, 1)
attn128_simple_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                      const __grid_constant__ CUtensorMap tm_v, const AttnParams p, const int kv_box_rows) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base;
    const uint32_t sK = sQ + 2 * kSlabBytes;
    const uint32_t sV = sK + 2 * kSlabBytes;
    const uint32_t sP = sV + 2 * kSlabBytes;
    const uint32_t sBar = sP + 2 * kSlabBytes;
    const uint32_t bar_q = sBar, bar_kv = sBar + 8, bar_mma = sBar + 16;
    uint8_t* gen_base = smem_raw + (smem_base - smem_u32(smem_raw));  // generic pointer to the aligned base
    volatile int* s_abort = reinterpret_cast<volatile int*>(gen_base + 8 * kSlabBytes + 64);
    volatile int* s_item = s_abort + 1;
    volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(s_abort + 2);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;

    if (tid == 0) {
        mbar_init(bar_q, 1);
        mbar_init(bar_kv, 1);
        mbar_init(bar_mma, 1);
        fence_mbar_init();
        *s_abort = 0;
        prefetch_tmap(&tm_q);
        prefetch_tmap(&tm_k);
        prefetch_tmap(&tm_v);
    }
    __syncthreads();
    if (warp == 0) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(s_tmem)), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *s_tmem;
    const uint32_t tS = tmem_base, tO = tmem_base + 128, tP = tmem_base + 256;
    const uint32_t lane_off = static_cast<uint32_t>(warp * 32) << 16;

    const int num_units = p.header_ro->num_units;
    const int G = p.num_q_heads / p.num_kv_heads;
    const int total_items = num_units * p.num_q_heads;
    constexpr uint32_t kIdescQK = idesc_bf16(128, 128, false, false);
    constexpr uint32_t kIdescPV = idesc_bf16(128, 128, false, true);

    uint32_t ph_q = 0, ph_kv = 0, ph_mma = 0;
    bool ok = true;

    while (ok) {
        if (tid == 0) *s_item = atomicAdd(&p.header->counter, 1);
        __syncthreads();
        const int item = *s_item;
        __syncthreads();
        if (item >= total_items) break;
        int ui, h;
        decode_item(item, num_units, p.num_q_heads, G, ui, h);
        const WorkUnit u = p.units[ui];
        const int g = h / G;

        if (tid == 0) {
            mbar_arrive_expect_tx(bar_q, 2 * kSlabBytes);
            tma_load_3d(sQ, &tm_q, bar_q, 0, h, u.q_row0);
            tma_load_3d(sQ + kSlabBytes, &tm_q, bar_q, 64, h, u.q_row0);
        }

        float m_run = -INFINITY, l_run = 0.f;
        const int my_pos = u.pos0 + tid;

        for (int j = u.kv_begin; j < u.kv_end && ok; ++j) {
            const int tile0 = j * kTileN;
            if (tid == 0) {
                mbar_arrive_expect_tx(bar_kv, 4 * kSlabBytes);
                for (int off = 0; off < kTileN; off += kv_box_rows) {
                    const int pos = tile0 + off;
                    int blk, slot;
                    if (p.block_table == nullptr) {
                        blk = u.req;
                        slot = pos;
                    } else if (pos < u.kv_len) {
                        blk = p.block_table[static_cast<long long>(u.req) * p.max_blocks_per_req +
                                            (pos >> p.block_shift)];
                        slot = pos & ((1 << p.block_shift) - 1);
                    } else {
                        blk = p.num_blocks;  // out of range: the copy engine fills zeros
                        slot = 0;
                    }
                    const uint32_t o = static_cast<uint32_t>(off) * 128u;
                    tma_load_4d(sK + o, &tm_k, bar_kv, 0, slot, g, blk);
                    tma_load_4d(sK + kSlabBytes + o, &tm_k, bar_kv, 64, slot, g, blk);
                    tma_load_4d(sV + o, &tm_v, bar_kv, 0, slot, g, blk);
                    tma_load_4d(sV + kSlabBytes + o, &tm_v, bar_kv, 64, slot, g, blk);
                }
            }
            if (j == u.kv_begin) {
                ok = mbar_wait(bar_q, ph_q, s_abort, 101);
                ph_q ^= 1;
            }
            ok = mbar_wait(bar_kv, ph_kv, s_abort, 102) && ok;
            ph_kv ^= 1;
            ok = __syncthreads_and(ok);
            if (!ok) break;

            // keys at or beyond kv_len do not exist: their V rows must not poison O through 0 * NaN
            if (tile0 + kTileN > u.kv_len) {
                if (tile0 + tid >= u.kv_len) {
                    uint4 z = make_uint4(0, 0, 0, 0);
                    uint4* v0 = reinterpret_cast<uint4*>(gen_base + 4 * kSlabBytes + tid * 128);
                    uint4* v1 = reinterpret_cast<uint4*>(gen_base + 5 * kSlabBytes + tid * 128);
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        v0[c] = z;
                        v1[c] = z;
                    }
                }
                fence_proxy_async_smem();
                __syncthreads();
            }

            if (tid == 0) {
                tc_fence_after();
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const uint32_t koff = (k >> 2) * kSlabBytes + (k & 3) * 32;
                    mma_ss(tS, smem_desc_sw128(sQ + koff, 16, 1024), smem_desc_sw128(sK + koff, 16, 1024), kIdescQK,
                           k > 0);
                }
                tc_commit(bar_mma);
            }
            ok = mbar_wait(bar_mma, ph_mma, s_abort, 103);
            ph_mma ^= 1;
            ok = __syncthreads_and(ok);
            if (!ok) break;
            tc_fence_after();

            // ---- online softmax, one row per thread ----
            const bool diag = (tile0 + kTileN - 1) > u.pos0;
            float mx = -INFINITY;
            uint32_t r[32];
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                tmem_ld32(tS + lane_off + c * 32, r);
                tc_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    float s = __uint_as_float(r[i]);
                    if (diag && (tile0 + c * 32 + i > my_pos)) s = -INFINITY;
                    mx = fmaxf(mx, s);
                }
            }
            const float m_new = fmaxf(m_run, mx * p.scale_log2e);
            const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
            const float alpha = ex2(m_run - m_use);
            float psum = 0.f;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                tmem_ld32(tS + lane_off + c * 32, r);
                tc_wait_ld();
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    float s0 = __uint_as_float(r[i]), s1 = __uint_as_float(r[i + 1]);
                    float p0 = ex2(fmaf(s0, p.scale_log2e, -m_use));
                    float p1 = ex2(fmaf(s1, p.scale_log2e, -m_use));
                    if (diag) {
                        if (tile0 + c * 32 + i > my_pos) p0 = 0.f;
                        if (tile0 + c * 32 + i + 1 > my_pos) p1 = 0.f;
                    }
                    psum += p0 + p1;
                    pk[i >> 1] = pack_bf16x2(p0, p1);
                }
                if constexpr (kPInTmem) {
                    tmem_st16(tP + lane_off + c * 16, pk);
                } else {
                    // K-major 128B-swizzled rows: 16-byte chunk index XOR (row & 7)
                    uint8_t* row = gen_base + 6 * kSlabBytes + (c >> 1) * kSlabBytes + tid * 128;
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        const int chunk = (c & 1) * 4 + q4;
                        *reinterpret_cast<uint4*>(row + ((chunk ^ (tid & 7)) << 4)) =
                            make_uint4(pk[4 * q4], pk[4 * q4 + 1], pk[4 * q4 + 2], pk[4 * q4 + 3]);
                    }
                }
            }
            l_run = l_run * alpha + psum;
            m_run = m_new;
            if (j > u.kv_begin) {
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    tmem_ld32(tO + lane_off + c * 32, r);
                    tc_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
                    tmem_st32(tO + lane_off + c * 32, r);
                }
            }
            if constexpr (kPInTmem) {
                tc_wait_st();
            } else {
                tc_wait_st();
                fence_proxy_async_smem();
            }
            tc_fence_before();
            __syncthreads();

            if (tid == 0) {
                tc_fence_after();
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const uint64_t bdesc = smem_desc_sw128(sV + k * 2048, kSlabBytes, 1024);
                    const uint32_t acc = (j > u.kv_begin || k > 0) ? 1u : 0u;
                    if constexpr (kPInTmem) {
                        mma_ts(tO, tP + k * 8, bdesc, kIdescPV, acc);
                    } else {
                        const uint32_t koff = (k >> 2) * kSlabBytes + (k & 3) * 32;
                        mma_ss(tO, smem_desc_sw128(sP + koff, 16, 1024), bdesc, kIdescPV, acc);
                    }
                }
                tc_commit(bar_mma);
            }
            ok = mbar_wait(bar_mma, ph_mma, s_abort, 104);
            ph_mma ^= 1;
            ok = __syncthreads_and(ok);
            if (!ok) break;
            tc_fence_after();
        }
        if (!ok) break;

        // ---- epilogue: normalise and store this thread's row ----
        {
            const float inv_l = 1.f / l_run;
            const bool valid = tid < u.rows;
            const long long row = static_cast<long long>(u.q_row0) + tid;
            uint32_t r[32];
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                tmem_ld32(tO + lane_off + c * 32, r);
                tc_wait_ld();
                if (!valid) continue;
                if (u.split < 0) {
                    uint4* dst = reinterpret_cast<uint4*>(static_cast<uint8_t*>(p.out) +
                                                          ((row * p.num_q_heads + h) * 128 + c * 32) * 2);
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        uint32_t w[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            w[e] = pack_bf16x2(__uint_as_float(r[q4 * 8 + 2 * e]) * inv_l,
                                               __uint_as_float(r[q4 * 8 + 2 * e + 1]) * inv_l);
                        dst[q4] = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                } else {
                    float4* dst = reinterpret_cast<float4*>(
                        p.o_parts + ((static_cast<long long>(u.split) * p.total_q + row) * p.num_q_heads + h) * 128 +
                        c * 32);
#pragma unroll
                    for (int q4 = 0; q4 < 8; ++q4)
                        dst[q4] = make_float4(__uint_as_float(r[q4 * 4]) * inv_l, __uint_as_float(r[q4 * 4 + 1]) * inv_l,
                                              __uint_as_float(r[q4 * 4 + 2]) * inv_l,
                                              __uint_as_float(r[q4 * 4 + 3]) * inv_l);
                }
            }
            if (valid) {
                const float lse = (m_run + log2f(l_run)) * 0.6931471805599453f;
                if (u.split < 0) {
                    if (p.lse) p.lse[row * p.num_q_heads + h] = lse;
                } else {
                    p.lse_parts[(static_cast<long long>(u.split) * p.total_q + row) * p.num_q_heads + h] = lse;
                }
            }
            tc_fence_before();
            __syncthreads();
            tc_fence_after();
        }
    }

    // ---- teardown ----
    __syncthreads();
    if (*s_abort != 0) {
        if (tid == 0 && p.status) atomicCAS(p.status, 0, 3 /* VPP_DEV_TIMEOUT */);
        // give copies that are still in flight time to land before the CTA's shared memory is released
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, 512);
}

}  // namespace vpp
