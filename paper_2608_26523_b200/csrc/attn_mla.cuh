// Chunked-prefill attention for absorbed MLA: 576-wide keys (512 latent + 64 rope features), values = the
// first 512 features of the same cache row, one shared kv-head.
//
// A 128-row query tile with a 512-wide fp32 output would fill tensor memory on its own (128 x 512 fp32 =
// all 512 columns), leaving no room for the scores.  This kernel therefore makes two passes over the keys,
// one per 256-wide half of the output, recomputing S = Q K^T in the second pass (+53 % MMA work); each
// pass is the paper's Eq. 1 evaluated KV tile by KV tile with a running maximum, exactly as in the
// head_dim-128 kernel.
//
// One CTA per SM, 6 warps:
//   warp 0      scheduler + TMA producer: Q tile (128 x 576, nine 64-column slabs, resident for both passes)
//               and, per 64-key KV tile, nine 8 KB slabs of the latent rows, each slab with its own
//               full / empty barrier so that slabs are refilled as soon as their last MMA has retired.
//   warp 1      (one thread) MMA issuer: S_b = Q K^T (M128 N64, 36 MMAs over the nine slabs) into one of two
//               score buffers, O += P V (M128 N256, four MMAs; V = four of the K slabs read as an MN-major
//               operand, P from tensor memory).  The score MMAs of tile j+1 that touch non-value slabs are
//               issued before waiting for P of tile j, so they overlap the softmax.
//   warps 2-5   softmax: one query row per thread on a 128 x 64 score tile, P written over S as bf16.
// Tensor memory: S0 (64 cols) | S1 (64) | O half (256).
#pragma once
#include "common.cuh"  // decode_item
#include "common.cuh"
#include "ptx.cuh"

namespace vpp {

constexpr int kMlaThreads = 192;
constexpr int kMlaDqk = 576, kMlaDv = 512;
constexpr int kMlaSlabs = kMlaDqk / 64;            // 9
constexpr int kMlaTileN = 64;                      // keys per KV tile
constexpr int kMlaQSlab = kTileM * 128;            // 16 KB: 128 rows x 64 bf16
constexpr int kMlaKSlab = kMlaTileN * 128;         // 8 KB: 64 keys x 64 bf16
constexpr int kMlaSmemBytes = kMlaSlabs * (kMlaQSlab + kMlaKSlab) + 1024 /*align*/ + 1024 /*barriers, ring*/;

struct MlaItem {
    WorkUnit u;
    int32_t h;
    int32_t valid;
    int32_t pad[2];
};

// Order in which the nine K slabs of a tile are consumed by the score MMAs in output-half `pass`: the five
// slabs that are not values of this pass first (they can be refilled while the softmax and the PV MMAs
// of the tile run), then the four value slabs.
__device__ __forceinline__ int mla_slab_order(int pass, int i) {
    // pass 0: 4 5 6 7 8 | 0 1 2 3      pass 1: 0 1 2 3 8 | 4 5 6 7
    if (pass == 0) return i < 5 ? 4 + i : i - 5;
    return i < 4 ? i : (i == 4 ? 8 : i - 1);
}

__global__ void __launch_bounds__(kMlaThreads, 1)
attn_mla_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_k4, const __grid_constant__ CUtensorMap tm_k5, const AttnParams p,
                const int kv_box_rows) {
    // tm_k loads one 64-column slab of kv_box_rows keys; tm_k4 / tm_k5 are rank-5 views of the same cache
    // (64 columns, keys, slab index, head, block) whose boxes cover 4 / 5 consecutive slabs of 64 keys, so
    // that a whole slab group arrives with one copy instruction (used when a KV tile lies in one page).
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gen_base = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sQ = smem_base;                              // 9 slabs of 16 KB
    const uint32_t sK = sQ + kMlaSlabs * kMlaQSlab;             // 9 slabs of 8 KB
    const uint32_t sBar = sK + kMlaSlabs * kMlaKSlab;
    const uint32_t bar_item_full = sBar + 0;     // [2]
    const uint32_t bar_item_empty = sBar + 16;   // [2]
    const uint32_t bar_q_full = sBar + 32;
    const uint32_t bar_q_empty = sBar + 40;
    const uint32_t bar_s_full = sBar + 48;       // [2]
    const uint32_t bar_p_full = sBar + 64;       // [2]
    const uint32_t bar_o_full = sBar + 80;
    const uint32_t bar_vfix = sBar + 88;
    // The nine K slabs of a tile travel as two groups: group 0 = the five slabs that are not values of the
    // current pass, group 1 = its four value slabs.
    const uint32_t bar_k_full = sBar + 128;      // [2 groups]
    const uint32_t bar_k_empty = sBar + 144;     // [2 groups]
    uint8_t* gen_bar = gen_base + kMlaSlabs * (kMlaQSlab + kMlaKSlab);
    volatile int* s_abort = reinterpret_cast<volatile int*>(gen_bar + 512);
    volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(gen_bar + 516);
    MlaItem* ring = reinterpret_cast<MlaItem*>(gen_bar + 576);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar_item_full + 8 * i, 1);
            mbar_init(bar_item_empty + 8 * i, 5);
            mbar_init(bar_s_full + 8 * i, 1);
            mbar_init(bar_p_full + 8 * i, 4);
        }
        mbar_init(bar_q_full, 1);
        mbar_init(bar_q_empty, 1);
        mbar_init(bar_o_full, 1);
        mbar_init(bar_vfix, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar_k_full + 8 * i, 1);
            mbar_init(bar_k_empty + 8 * i, 1);
        }
        fence_mbar_init();
        *s_abort = 0;
        prefetch_tmap(&tm_q);
        prefetch_tmap(&tm_k);
        prefetch_tmap(&tm_k4);
        prefetch_tmap(&tm_k5);
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

    const int num_units = p.header_ro->num_units;
    const int total_items = num_units * p.num_q_heads;

    // KV tiles (64 keys) of a unit: keys [kv_begin*128, min(kv_end*128, pos0 + rows))
    auto tile_range = [](const WorkUnit& u, int& t_lo, int& t_hi) {
        const int key_lo = u.kv_begin * kTileN;
        int key_hi = u.kv_end * kTileN;
        if (key_hi > u.pos0 + u.rows) key_hi = u.pos0 + u.rows;
        t_lo = key_lo / kMlaTileN;
        t_hi = (key_hi + kMlaTileN - 1) / kMlaTileN;
    };

    if (warp == 0) {
        // ================================ scheduler + TMA producer ================================
        uint32_t item_it = 0, q_it = 0, fill = 0;  // fill: KV tiles loaded so far (all slabs advance together)
        while (true) {
            int item = 0;
            if (lane == 0) item = atomicAdd(&p.header->counter, 1);
            item = __shfl_sync(0xffffffffu, item, 0);
            const bool have = item < total_items;
            const uint32_t slot = item_it & 1;
            bool ok = true;
            if (lane == 0) ok = mbar_wait(bar_item_empty + 8 * slot, ((item_it >> 1) & 1) ^ 1, s_abort, 501);
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            WorkUnit u{};
            int h = 0;
            if (have) {
                int ui;
                decode_item(item, num_units, p.num_q_heads, p.num_q_heads, ui, h);
                u = p.units[ui];
            }
            if (lane == 0) {
                ring[slot].u = u;
                ring[slot].h = h;
                ring[slot].valid = have ? 1 : 0;
                mbar_arrive(bar_item_full + 8 * slot);
            }
            ++item_it;
            if (!have) break;

            if (lane == 0) {
                ok = mbar_wait(bar_q_empty, (q_it & 1) ^ 1, s_abort, 502);
                if (ok) {
                    mbar_arrive_expect_tx(bar_q_full, kMlaSlabs * kMlaQSlab);
#pragma unroll
                    for (int s = 0; s < kMlaSlabs; ++s) tma_load_3d(sQ + s * kMlaQSlab, &tm_q, bar_q_full, 64 * s, h, u.q_row0);
                }
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            ++q_it;

            int t_lo, t_hi;
            tile_range(u, t_lo, t_hi);
            for (int pass = 0; pass < 2 && ok; ++pass) {
                for (int j = t_lo; j < t_hi && ok; ++j) {
                    const int tile0 = j * kMlaTileN;
                    if (kv_box_rows == kMlaTileN) {
                        if (lane == 0) {
                            // page lookup once per tile (not per slab): a dependent global load costs more than a slab's MMAs
                            int blk, slot_in;
                            if (p.block_table == nullptr) {
                                blk = u.req;
                                slot_in = tile0;
                            } else if (tile0 < u.kv_len) {
                                blk = __ldg(p.block_table + static_cast<long long>(u.req) * p.max_blocks_per_req +
                                            (tile0 >> p.block_shift));
                                slot_in = tile0 & ((1 << p.block_shift) - 1);
                            } else {
                                blk = p.num_blocks;  // out of range: the copy engine fills zeros
                                slot_in = 0;
                            }
                            if (j == t_lo) {
                                // the physical slabs change groups between passes: both groups of the previous tile
                                // must have been released before anything of this pass is loaded
                                ok = mbar_wait(bar_k_empty + 8, (fill & 1) ^ 1, s_abort, 505);
                            }
                            for (int grp = 0; grp < 2 && ok; ++grp) {
                                ok = mbar_wait(bar_k_empty + 8 * grp, (fill & 1) ^ 1, s_abort, 503);
                                if (!ok) break;
                                const uint32_t full = bar_k_full + 8 * grp;
                                const int i0 = grp == 0 ? 0 : 5, i1 = grp == 0 ? 5 : 9;
                                mbar_arrive_expect_tx(full, (i1 - i0) * kMlaKSlab);
                                // one page per tile: whole runs of consecutive slabs per instruction
                                if (grp == 1) {
                                    tma_load_5d(sK + pass * 4 * kMlaKSlab, &tm_k4, full, 0, slot_in, pass * 4, 0, blk);
                                } else if (pass == 0) {
                                    tma_load_5d(sK + 4 * kMlaKSlab, &tm_k5, full, 0, slot_in, 4, 0, blk);
                                } else {
                                    tma_load_5d(sK, &tm_k4, full, 0, slot_in, 0, 0, blk);
                                    tma_load_4d(sK + 8 * kMlaKSlab, &tm_k, full, 64 * 8, slot_in, 0, blk);
                                }
                            }
                        }
                    } else {
                        // Pages smaller than the tile: one copy per (slab, page), each issued by a lane of its own (every lane
                        // looks up the page of its copy itself) -- a single thread issuing the 18 to 36 copies of a tile one
                        // after the other is several times slower than the MMAs that consume them.
                        const int np = kMlaTileN / kv_box_rows;          // pages per tile: 2 or 4
                        const int pq = lane % np;                          // this lane's page of the tile
                        const int pos = tile0 + pq * kv_box_rows;
                        int blk, slot_in;
                        if (p.block_table == nullptr) {
                            blk = u.req;
                            slot_in = pos;
                        } else if (pos < u.kv_len) {
                            blk = __ldg(p.block_table + static_cast<long long>(u.req) * p.max_blocks_per_req + (pos >> p.block_shift));
                            slot_in = pos & ((1 << p.block_shift) - 1);
                        } else {
                            blk = p.num_blocks;  // out of range: the copy engine fills zeros
                            slot_in = 0;
                        }
                        if (j == t_lo) {
                            if (lane == 0) ok = mbar_wait(bar_k_empty + 8, (fill & 1) ^ 1, s_abort, 505);
                            ok = __shfl_sync(0xffffffffu, ok, 0);
                        }
                        for (int grp = 0; grp < 2 && ok; ++grp) {
                            const uint32_t full = bar_k_full + 8 * grp;
                            const int i0 = grp == 0 ? 0 : 5, i1 = grp == 0 ? 5 : 9;
                            if (lane == 0) {
                                ok = mbar_wait(bar_k_empty + 8 * grp, (fill & 1) ^ 1, s_abort, 503);
                                if (ok) mbar_arrive_expect_tx(full, (i1 - i0) * kMlaKSlab);
                            }
                            ok = __shfl_sync(0xffffffffu, ok, 0);
                            if (!ok) break;
                            const int i = i0 + lane / np;
                            if (i < i1) {
                                const int sl = mla_slab_order(pass, i);
                                tma_load_4d(sK + sl * kMlaKSlab + pq * kv_box_rows * 128, &tm_k, full, 64 * sl, slot_in, 0, blk);
                            }
                            __syncwarp();
                        }
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) break;
                    if (tile0 + kMlaTileN > u.kv_len) {
                        // keys at or beyond kv_len do not exist: zero their rows in the four value slabs of this
                        // pass so that 0 * garbage cannot poison O; the MMA thread waits for bar_vfix on such a tile
                        if (lane == 0) ok = mbar_wait(bar_k_full + 8, fill & 1, s_abort, 504);
                        ok = __shfl_sync(0xffffffffu, ok, 0);
                        if (!ok) break;
                        const int first = u.kv_len > tile0 ? u.kv_len - tile0 : 0;
                        const uint4 z = make_uint4(0, 0, 0, 0);
                        for (int i = 0; i < 4; ++i) {
                            uint8_t* vb = gen_base + kMlaSlabs * kMlaQSlab + (pass * 4 + i) * kMlaKSlab;
                            for (int r = first + lane; r < kMlaTileN; r += 32) {
                                uint4* a = reinterpret_cast<uint4*>(vb + r * 128);
#pragma unroll
                                for (int c = 0; c < 8; ++c) a[c] = z;
                            }
                        }
                        fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_vfix);
                    }
                    ++fill;
                }
            }
            if (!ok) break;
        }
    } else if (warp == 1 && lane == 0) {
        // ================================ MMA issuer (a single thread) ================================
        constexpr uint32_t kIdescQK = idesc_bf16(128, kMlaTileN, false, false);
        constexpr uint32_t kIdescPV = idesc_bf16(128, 256, false, true);
        constexpr uint32_t kHi = desc_hi_sw128(1024);
        const uint32_t tO = tmem_base + 128;
        const uint32_t q_lo = desc_lo_sw128(sQ, 16), k_lo = desc_lo_sw128(sK, 16);
        const uint32_t v_lo = desc_lo_sw128(sK, kMlaKSlab);
        uint32_t item_it = 0, q_it = 0, fill = 0, tc = 0, vfix_it = 0;
        // score MMAs of KV tile number `fl` (global count) for slabs order[i0..i1) of `pass`
        auto issue_qk = [&](uint32_t tS, int pass, int grp, uint32_t fl) -> bool {
            if (!mbar_wait(bar_k_full + 8 * grp, fl & 1, s_abort, 601)) return false;
            tc_fence_after();
            const int i0 = grp == 0 ? 0 : 5, i1 = grp == 0 ? 5 : 9;
            for (int i = i0; i < i1; ++i) {
                const int s = mla_slab_order(pass, i);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    mma_ss_lh(tS, q_lo + ((s * kMlaQSlab + kk * 32) >> 4), k_lo + ((s * kMlaKSlab + kk * 32) >> 4), kHi,
                              kIdescQK, (i > 0 || kk > 0) ? 1u : 0u);
            }
            return true;
        };
        while (true) {
            const uint32_t slot = item_it & 1;
            if (!mbar_wait(bar_item_full + 8 * slot, (item_it >> 1) & 1, s_abort, 602)) break;
            const WorkUnit u = ring[slot].u;
            const int valid = ring[slot].valid;
            mbar_arrive(bar_item_empty + 8 * slot);
            ++item_it;
            if (!valid) break;
            int t_lo, t_hi;
            tile_range(u, t_lo, t_hi);
            const int n = t_hi - t_lo;
            if (!mbar_wait(bar_q_full, q_it & 1, s_abort, 603)) break;
            ++q_it;
            bool ok = true;
            for (int pass = 0; pass < 2 && ok; ++pass) {
                // first tile of the pass: both groups
                ok = issue_qk(tmem_base + (tc & 1) * 64, pass, 0, fill);
                if (!ok) break;
                tc_commit(bar_k_empty);
                ok = issue_qk(tmem_base + (tc & 1) * 64, pass, 1, fill);
                if (!ok) break;
                tc_commit(bar_s_full + 8 * (tc & 1));
                if (n == 1 && pass == 1) tc_commit(bar_q_empty);
                for (int jj = 0; jj < n; ++jj) {
                    const int tile0 = (t_lo + jj) * kMlaTileN;
                    const uint32_t b = tc & 1;               // score buffer of tile jj
                    const uint32_t tS = tmem_base + b * 64;
                    const bool has_next = jj + 1 < n;
                    bool early = false;
                    if (has_next && mbar_try_wait(bar_k_full, (fill + 1) & 1)) {
                        // the non-value slabs of the next tile are already here: their score MMAs overlap the
                        // softmax of this tile (if they are not, P V of this tile must not wait for them)
                        ok = issue_qk(tmem_base + (b ^ 1) * 64, pass, 0, fill + 1);
                        if (!ok) break;
                        tc_commit(bar_k_empty);
                        early = true;
                    }
                    if (tile0 + kMlaTileN > u.kv_len) {
                        ok = mbar_wait(bar_vfix, vfix_it & 1, s_abort, 604);
                        if (!ok) break;
                        ++vfix_it;
                    }
                    ok = mbar_wait(bar_p_full + 8 * b, (tc >> 1) & 1, s_abort, 605);
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        mma_ts_lh(tO, tS + kk * 8, v_lo + ((pass * 4 * kMlaKSlab + kk * 2048) >> 4), kHi, kIdescPV,
                                  (jj > 0 || kk > 0) ? 1u : 0u);
                    tc_commit(bar_k_empty + 8);
                    ++fill;
                    ++tc;
                    if (has_next) {
                        if (!early) {
                            ok = issue_qk(tmem_base + (b ^ 1) * 64, pass, 0, fill);
                            if (!ok) break;
                            tc_commit(bar_k_empty);
                        }
                        if (!mbar_wait(bar_k_full + 8, fill & 1, s_abort, 606)) { ok = false; break; }
                        ok = issue_qk(tmem_base + (b ^ 1) * 64, pass, 1, fill);
                        if (!ok) break;
                        tc_commit(bar_s_full + 8 * (b ^ 1));
                        if (jj + 2 == n && pass == 1) tc_commit(bar_q_empty);
                    } else {
                        tc_commit(bar_o_full);
                    }
                }
            }
            if (!ok) break;
        }
    } else if (warp >= 2) {
        // ======================================= softmax =======================================
        const int row = ((warp & 3) << 5) | lane;      // TMEM lane = row of the tile
        const uint32_t lane_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tO = tmem_base + 128 + lane_off;
        uint32_t item_it = 0, tc = 0, o_it = 0;
        const float sc = p.scale_log2e;
        while (true) {
            const uint32_t slot = item_it & 1;
            if (!mbar_wait(bar_item_full + 8 * slot, (item_it >> 1) & 1, s_abort, 701)) break;
            const WorkUnit u = ring[slot].u;
            const int h = ring[slot].h;
            const int valid = ring[slot].valid;
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_item_empty + 8 * slot);
            ++item_it;
            if (!valid) break;
            int t_lo, t_hi;
            tile_range(u, t_lo, t_hi);
            const int my_pos = u.pos0 + row;
            bool ok = true;
            for (int pass = 0; pass < 2 && ok; ++pass) {
                float m_ref = -INFINITY, l_run = 0.f;
                for (int j = t_lo; j < t_hi; ++j) {
                    const int tile0 = j * kMlaTileN;
                    const uint32_t b = tc & 1;
                    const uint32_t tS = tmem_base + b * 64 + lane_off;
                    ok = mbar_wait(bar_s_full + 8 * b, (tc >> 1) & 1, s_abort, 702);
                    if (!ok) break;
                    ++tc;
                    tc_fence_after();
                    uint32_t s[64];
                    tmem_ld32(tS, reinterpret_cast<uint32_t(&)[32]>(s[0]));
                    tmem_ld32(tS + 32, reinterpret_cast<uint32_t(&)[32]>(s[32]));
                    tc_wait_ld();
                    if (tile0 + kMlaTileN - 1 > u.pos0) {  // diagonal tile
                        const int lim = my_pos - tile0;
#pragma unroll
                        for (int i = 0; i < 64; ++i)
                            if (i > lim) s[i] = 0xff800000u;  // -inf
                    }
                    float mx[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) mx[k] = __uint_as_float(s[k]);
#pragma unroll
                    for (int i = 8; i < 64; i += 8)
#pragma unroll
                        for (int k = 0; k < 8; ++k) mx[k] = fmaxf(mx[k], __uint_as_float(s[i + k]));
                    const float mxa = fmaxf(fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])),
                                            fmaxf(fmaxf(mx[4], mx[5]), fmaxf(mx[6], mx[7])));
                    const float m_new = fmaxf(mxa * sc, m_ref);
                    const bool grow = (m_new - m_ref > 8.f) || (m_ref == -INFINITY && m_new != -INFINITY);
                    if (__any_sync(0xffffffffu, grow)) {
                        const float alpha = grow ? ex2(m_ref - m_new) : 1.f;
                        if (grow) m_ref = m_new;
                        l_run *= alpha;
                        if (j > t_lo) {
                            uint32_t o[32];
#pragma unroll 1
                            for (int c = 0; c < 8; ++c) {
                                tmem_ld32(tO + c * 32, o);
                                tc_wait_ld();
#pragma unroll
                                for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                                tmem_st32(tO + c * 32, o);
                            }
                        }
                    }
                    const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
                    float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        uint32_t pk[16];
#pragma unroll
                        for (int i = 0; i < 32; i += 2) {
                            const float p0 = ex2(fmaf(__uint_as_float(s[c * 32 + i]), sc, -m_use));
                            const float p1 = ex2(fmaf(__uint_as_float(s[c * 32 + i + 1]), sc, -m_use));
                            sum0 += p0;
                            sum1 += p1;
                            pk[i >> 1] = pack_bf16x2(p0, p1);
                        }
                        tmem_st16(tS + c * 16, pk);
                    }
                    l_run += sum0 + sum1;
                    tc_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_p_full + 8 * b);
                }
                if (!ok) break;
                // ---- epilogue of this output half ----
                ok = mbar_wait(bar_o_full, o_it & 1, s_abort, 703);
                if (!ok) break;
                ++o_it;
                tc_fence_after();
                const float inv_l = 1.f / l_run;
                const bool live = row < u.rows;
                const long long grow_idx = static_cast<long long>(u.q_row0) + row;
                uint32_t r[32];
#pragma unroll 1
                for (int c = 0; c < 8; ++c) {
                    tmem_ld32(tO + c * 32, r);
                    tc_wait_ld();
                    if (!live) continue;
                    const int col0 = pass * 256 + c * 32;
                    if (u.split < 0) {
                        uint4* dst = reinterpret_cast<uint4*>(static_cast<uint8_t*>(p.out) +
                                                              ((grow_idx * p.num_q_heads + h) * kMlaDv + col0) * 2);
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
                            p.o_parts +
                            ((static_cast<long long>(u.split) * p.total_q + grow_idx) * p.num_q_heads + h) * kMlaDv + col0);
#pragma unroll
                        for (int q4 = 0; q4 < 8; ++q4)
                            dst[q4] = make_float4(__uint_as_float(r[q4 * 4]) * inv_l, __uint_as_float(r[q4 * 4 + 1]) * inv_l,
                                                  __uint_as_float(r[q4 * 4 + 2]) * inv_l,
                                                  __uint_as_float(r[q4 * 4 + 3]) * inv_l);
                    }
                }
                if (live && pass == 0) {
                    const float lse = (m_ref + log2f(l_run)) * 0.6931471805599453f;
                    if (u.split < 0) {
                        if (p.lse) p.lse[grow_idx * p.num_q_heads + h] = lse;
                    } else {
                        p.lse_parts[(static_cast<long long>(u.split) * p.total_q + grow_idx) * p.num_q_heads + h] = lse;
                    }
                }
                tc_fence_before();
            }
            if (!ok) break;
        }
    }

    // ---- teardown ----
    __syncthreads();
    if (*s_abort != 0) {
        if (tid == 0 && p.status) atomicCAS(p.status, 0, 3 /* VPP_DEV_TIMEOUT */);
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, 512);
}

}  // namespace vpp
