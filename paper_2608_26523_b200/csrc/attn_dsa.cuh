// Index-selected (sparse) chunk attention over the absorbed-MLA latent cache: every query token attends to the key
// positions an external indexer listed for it (the paper's "MLA + DSA sparse attention" model; the lists are inputs).
// Eq. 1 over the listed keys only: an entry e of token t takes part iff 0 <= e <= position of t.
//
// One work item = one query token; its q-heads (<= 128, all sharing the one latent kv-head) are the rows of the tile,
// 64 per CTA of a 2-CTA cluster, exactly as in the packed single-token items of the dense pair kernel, from which the
// MMA, softmax and barrier structure is taken.  What differs is the producer side: a KV tile is 128 listed rows that
// lie anywhere in the cache, fetched with the gather form of the tensor copy (cp.async.bulk.tensor ... tile::gather4:
// four rows of 64 columns per instruction, 128-byte swizzle applied on the way in).  A warp issues such copies one lane
// after the other at ~75-130 clk apiece, but warps issue independently, so the 272 copies of a tile are spread over ten
// producer warps, two per hand-back group, each issuing one instruction per tile.  (16-byte cp.async copies by the same
// warps were measured too: 385 TFLOP/s -- a warp keeps too few of them in flight.)
// Entries that do not take part are pointed at the token's own cache row (always present and finite) and masked out
// of the softmax through a 128-bit validity mask that warp 0 publishes per tile.  The cost per token does not depend on
// the prefix length: the flat latency curve the paper says weakens its linear-growth assumption.
#pragma once
#include <type_traits>

#include "attn_mla2.cuh"

namespace vpp {

constexpr int kDsaThreads = 512;   // 16 warps: see the role list in the kernel
constexpr int kDsaMaxReqs = 8192;
constexpr int kDsaPrepThreads = 256;

struct DsaParams {
    const int32_t* indices;       // [total_q, topk] key positions within the token's request
    int32_t topk;
    const int2* tok;              // [total_q] (request, position) of every token; request < 0: skip the token
    const int32_t* block_table;   // may be null (contiguous)
    int32_t max_blocks_per_req;
    int32_t block_shift;
    int32_t num_blocks;
    int32_t max_seq_len;          // contiguous: rows per request
    int32_t num_q_heads;
    int32_t total_q;
    float scale_log2e;
    void* out;                    // bf16 [T, Hq, 512]
    float* lse;                   // [T, Hq] or null
    int32_t* status;
};

// (request, position) of every token from the per-request lengths; lengths that do not describe the launch mark every
// token as skipped and set the status.
__global__ void __launch_bounds__(kDsaPrepThreads)
dsa_tokens_kernel(const int32_t* prefix_len, const int32_t* chunk_len, int num_reqs, int total_q, long long capacity,
                  int2* tok, int32_t* status) {
    extern __shared__ int32_t cu[];   // cu[r] = tokens before request r
    __shared__ int s_bad;
    const int tid = threadIdx.x, lane = tid & 31;
    if (tid == 0) s_bad = 0;
    __syncthreads();
    if (tid < 32) {
        int carry = 0;
        for (int base = 0; base < num_reqs; base += 32) {
            const int r = base + lane;
            int c = 0;
            if (r < num_reqs) {
                c = chunk_len[r];
                const int pre = prefix_len[r];
                if (c < 0 || pre < 0 || static_cast<long long>(pre) + c > capacity) {
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
            if (r < num_reqs) cu[r] = carry + x - c;
            carry += __shfl_sync(0xffffffffu, x, 31);
        }
        if (lane == 0) cu[num_reqs] = carry;
    }
    __syncthreads();
    const bool bad = s_bad || cu[num_reqs] != total_q;
    if (bad && tid == 0 && blockIdx.x == 0 && status) atomicCAS(status, 0, 1 /* VPP_DEV_BAD_LENGTHS */);
    for (int t = blockIdx.x * kDsaPrepThreads + tid; t < total_q; t += gridDim.x * kDsaPrepThreads) {
        if (bad) {
            tok[t] = make_int2(-1, -1);
            continue;
        }
        int lo = 0, hi = num_reqs;   // last r with cu[r] <= t
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (cu[mid] <= t) lo = mid; else hi = mid;
        }
        tok[t] = make_int2(lo, prefix_len[lo] + (t - cu[lo]));
    }
}

// Four rows of one 64-column slab into four consecutive 128-byte rows of shared memory.  The data lands in the executing
// CTA; the bytes are posted on a barrier that may live in the other CTA of the pair.  No multicast.
__device__ __forceinline__ void tma2_gather4(uint32_t dst, const CUtensorMap* m, uint32_t bar_cluster, int col, int r0,
                                             int r1, int r2, int r3) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes [%0], [%1, "
        "{%3, %4, %5, %6, %7}], [%2];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(m)), "r"(bar_cluster), "r"(col), "r"(r0), "r"(r1), "r"(r2), "r"(r3)
        : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kDsaThreads, 1)
dsa_attn_kernel(const __grid_constant__ CUtensorMap tm_qh, const __grid_constant__ CUtensorMap tm_rows, const DsaParams p) {
    // tm_qh:   (64 cols, Hq heads, 9 slabs, T tokens) box (64, 64, 9, 1) -- 64 q-heads of one token, all slabs (heads past Hq read as zero)
    // tm_rows: (576 cols, cache rows) box (64, 1), gather mode: four listed rows of one 64-column slab per copy
    // Per CTA, 16 warps: warps 0, 6, 8-11 K producers (two per hand-back group; warp 0 also Q and the validity masks),
    // warps 12-15 V producers (two per group), warp 1 / warp 7 of the leader: one thread each issuing the score and
    // the P V MMAs of the pair, warps 2-5 softmax.
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gen_base = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sQ = smem_base;
    const uint32_t sK = sQ + kMla2QBytes;
    const uint32_t sV = sK + kMla2KBytes;
    const uint32_t sP = sV + kMla2VBytes;
    const uint32_t sBar = sP + kMla2PBytes;
    const uint32_t bar_q_full = sBar + 0;
    const uint32_t bar_pv_done = sBar + 8;   // all P V MMAs of a tile done: last V group free, P free, O quiescent
    const uint32_t bar_s_full = sBar + 24;   // [2] scores of a tile done: also "last K group free" (and Q free after an item)
    const uint32_t bar_p_full = sBar + 40;   // [2] leader: 4 local + 4 remote warp arrivals
    const uint32_t bar_xchg = sBar + 80;     // row statistics exchange between the two threads of a row
    const uint32_t bar_k_full = sBar + 96;   // [kKGroups] leader: bytes of both CTAs
    const uint32_t bar_k_empty = sBar + 168; // [kKGroups - 1]
    const uint32_t bar_v_full = sBar + 312;  // [kVGroups]
    const uint32_t bar_v_empty = sBar + 344; // [kVGroups - 1]
    const uint32_t bar_mask = sBar + 376;    // [4] validity mask of a tile published (each CTA for itself)
    const uint32_t bar_mask_free = sBar + 192;  // [4] ... and read by the four softmax warps
    uint8_t* gen_bar = gen_base + kMla2QBytes + kMla2KBytes + kMla2VBytes + kMla2PBytes;
    volatile int* s_abort = reinterpret_cast<volatile int*>(gen_bar + 416);
    volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(gen_bar + 420);
    volatile uint32_t* vmask = reinterpret_cast<volatile uint32_t*>(gen_bar + 448);  // [4 tiles][4 words]
    float* xch = reinterpret_cast<float*>(gen_bar + 512);                            // [2 phases][128 lanes]

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const uint32_t rank = cluster_ctarank();
    const bool leader = rank == 0;
    if (tid == 0) {
        mbar_init(bar_q_full, 1);
        mbar_init(bar_pv_done, 1);
        mbar_init(bar_s_full, 1);
        mbar_init(bar_s_full + 8, 1);
        mbar_init(bar_p_full, 8);
        mbar_init(bar_p_full + 8, 8);
        mbar_init(bar_xchg, 128);
        for (int i = 0; i < kKGroups; ++i) {
            mbar_init(bar_k_full + 8 * i, 1);
            mbar_init(bar_k_empty + 8 * i, 1);
        }
        for (int i = 0; i < kVGroups; ++i) {
            mbar_init(bar_v_full + 8 * i, 1);
            mbar_init(bar_v_empty + 8 * i, 1);
        }
        for (int i = 0; i < 4; ++i) {
            mbar_init(bar_mask + 8 * i, 1);
            mbar_init(bar_mask_free + 8 * i, 4);
        }
        fence_mbar_init();
        *s_abort = 0;
        prefetch_tmap(&tm_qh);
        prefetch_tmap(&tm_rows);
    }
    __syncthreads();
    cluster_sync_all();  // barrier initialisation is visible to the other CTA before anything arrives remotely
    if (warp == 0) {
        tmem_alloc2(smem_u32(const_cast<uint32_t*>(s_tmem)), 512);
        tmem_relinquish2();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *s_tmem;

    const int num_pairs = gridDim.x >> 1;
    const int pair = blockIdx.x >> 1;
    const int n_tiles = (p.topk + kTileN - 1) / kTileN;   // the same for every token

    // cache row of position e of request req
    auto row_of = [&](int req, int e) -> int {
        if (p.block_table == nullptr) return req * p.max_seq_len + e;
        const int blk = __ldg(p.block_table + static_cast<long long>(req) * p.max_blocks_per_req + (e >> p.block_shift));
        if (static_cast<unsigned>(blk) >= static_cast<unsigned>(p.num_blocks)) {
            if (p.status) atomicCAS(p.status, 0, 2 /* VPP_DEV_BAD_BLOCK */);
            return 0;
        }
        return (blk << p.block_shift) + (e & ((1 << p.block_shift) - 1));
    };
    // list entries 128 j + key0 .. + 3 of token t (entries past the end of the list read as "none")
    auto load_entries = [&](int t, int j, int key0, int (&e)[4]) {
        const int k0 = j * kTileN + key0;
        const int32_t* src = p.indices + static_cast<long long>(t) * p.topk + k0;
#pragma unroll
        for (int i = 0; i < 4; ++i) e[i] = (k0 + i < p.topk) ? __ldg(src + i) : -1;
    };
    // rows to fetch for these entries (those that do not take part fetch the token's own row) and which take part
    auto rows_of = [&](int req, int pos, int self_row, const int (&e)[4], int (&r)[4]) -> uint32_t {
        uint32_t bits = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const bool v = e[i] >= 0 && e[i] <= pos;
            r[i] = v ? row_of(req, e[i]) : self_row;
            bits |= (v ? 1u : 0u) << i;
        }
        return bits;
    };

    const uint32_t pair_q_full = mapa_u32(bar_q_full, 0), pair_k_full = mapa_u32(bar_k_full, 0),
                   pair_v_full = mapa_u32(bar_v_full, 0);

    if (warp == 0 || warp == 6 || (warp >= 8 && warp <= 11)) {
        // ===================================== Q / K producers =====================================
        // A warp issues gather copies one lane after the other, ~75-130 clk apiece, but warps issue independently
        // (measured: 8 warps x 16 lanes reach one copy per 13-16 clk per SM).  So every hand-back group has warps of its
        // own and a warp issues ONE instruction per tile as soon as its group is free: K group g (slabs 3 g .. 3 g + 2 of
        // this CTA's 64 keys = 48 copies) belongs to warps kw = 2 g and 2 g + 1, which take 8 quads of four keys each;
        // lane = 8 * (slab within the group) + quad: 24 lanes.  Warp 0 also loads Q and publishes the validity mask of
        // the tile's 128 entries.
        const int kw = warp == 0 ? 0 : (warp == 6 ? 1 : warp - 6);
        const int g = kw >> 1;
        const int quad = 8 * (kw & 1) + (lane & 7), sg = lane >> 3;
        const int key0 = static_cast<int>(rank) * 64 + 4 * quad;          // first of this lane's four keys in the tile
        const uint32_t dst = sK + (g * kKG + sg) * 8192 + static_cast<uint32_t>(quad) * 512u;
        const int col = (g * kKG + sg) * 64;
        uint32_t kc = 0;
        bool ok = true;
        for (int t = pair; t < p.total_q && ok; t += num_pairs) {
            const int2 tk = __ldg(p.tok + t);
            if (tk.x < 0) continue;
            if (warp == 0) {
                // Q may be replaced once the scores of the previous item's last tile are done
                if (kc > 0) {
                    if (lane == 0) ok = mbar_wait(bar_s_full + 8 * ((kc - 1) & 1), ((kc - 1) >> 1) & 1, s_abort, 901);
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) break;
                }
                if (lane == 0 && leader) {
                    mbar_arrive_expect_tx(bar_q_full, 2 * kMla2QBytes);   // both CTAs' boxes, rows outside the tensor included
                }
                if (lane == 0) tma2_load_4d(sQ, &tm_qh, pair_q_full, 0, static_cast<int>(rank) * kMla2Rows, 0, t);
            }
            const int self_row = row_of(tk.x, tk.y);
            int e_next[4], m_next[4];
            load_entries(t, 0, key0, e_next);
            if (warp == 0) load_entries(t, 0, 4 * lane, m_next);
            for (int j = 0; j < n_tiles && ok; ++j) {
                int e[4], r[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) e[i] = e_next[i];
                if (warp == 0) {
                    // validity of the tile's 128 entries: word i holds entry 4 l + i of lane l in bit l; a ring of four
                    // slots that the softmax warps hand back after reading
                    uint32_t bits = 0;
#pragma unroll
                    for (int i = 0; i < 4; ++i) bits |= (m_next[i] >= 0 && m_next[i] <= tk.y ? 1u : 0u) << i;
                    const uint32_t w0 = __ballot_sync(0xffffffffu, bits & 1u), w1 = __ballot_sync(0xffffffffu, bits & 2u),
                                   w2 = __ballot_sync(0xffffffffu, bits & 4u), w3 = __ballot_sync(0xffffffffu, bits & 8u);
                    if (lane == 0) {
                        if (kc >= 4) ok = mbar_wait(bar_mask_free + 8 * (kc & 3), ((kc - 4) >> 2) & 1, s_abort, 904);
                        volatile uint32_t* m = vmask + (kc & 3) * 4;
                        m[0] = w0; m[1] = w1; m[2] = w2; m[3] = w3;
                        mbar_arrive(bar_mask + 8 * (kc & 3));
                    }
                    if (j + 1 < n_tiles) load_entries(t, j + 1, 4 * lane, m_next);
                }
                if (j + 1 < n_tiles) load_entries(t, j + 1, key0, e_next);
                rows_of(tk.x, tk.y, self_row, e, r);
                if (lane == 0 && ok) {
                    if (g < kKGroups - 1) ok = mbar_wait(bar_k_empty + 8 * g, (kc & 1) ^ 1, s_abort, 902);
                    else if (kc > 0) ok = mbar_wait(bar_s_full + 8 * ((kc - 1) & 1), ((kc - 1) >> 1) & 1, s_abort, 902);
                    if (ok && leader && (kw & 1) == 0) mbar_arrive_expect_tx(bar_k_full + 8 * g, 2 * kKG * 8192);
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                if (sg < kKG) tma2_gather4(dst, &tm_rows, pair_k_full + 8 * g, col, r[0], r[1], r[2], r[3]);
                ++kc;
            }
        }
    } else if (warp >= 12) {
        // ======================================= V producers =======================================
        // chunk c = (key half hf, instr i) holds value columns 256 i + 128 rank .. + 127 (two 64-column slabs) of keys
        // 64 hf .. 64 hf + 63.  Group hf = 64 copies = warps vw = 2 hf and 2 hf + 1 with 8 quads each,
        // lane = 8 * (2 i + slab) + quad: all 32 lanes, one instruction per tile.
        const int vw = warp - 12;
        const int hf = vw >> 1;
        const int quad = 8 * (vw & 1) + (lane & 7), s4 = lane >> 3;
        const int key0 = hf * 64 + 4 * quad;
        const int slab = 4 * (s4 >> 1) + 2 * static_cast<int>(rank) + (s4 & 1);
        const uint32_t dst = sV + (2 * hf + (s4 >> 1)) * kMla2VChunk + (s4 & 1) * 8192 + static_cast<uint32_t>(quad) * 512u;
        uint32_t vc = 0;
        bool ok = true;
        for (int t = pair; t < p.total_q && ok; t += num_pairs) {
            const int2 tk = __ldg(p.tok + t);
            if (tk.x < 0) continue;
            const int self_row = row_of(tk.x, tk.y);
            int e_next[4];
            load_entries(t, 0, key0, e_next);
            for (int j = 0; j < n_tiles && ok; ++j) {
                int e[4], r[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) e[i] = e_next[i];
                if (j + 1 < n_tiles) load_entries(t, j + 1, key0, e_next);
                rows_of(tk.x, tk.y, self_row, e, r);
                if (lane == 0) {
                    if (hf < kVGroups - 1) ok = mbar_wait(bar_v_empty + 8 * hf, (vc & 1) ^ 1, s_abort, 903);
                    else if (vc > 0) ok = mbar_wait(bar_pv_done, (vc - 1) & 1, s_abort, 903);
                    if (ok && leader && (vw & 1) == 0) mbar_arrive_expect_tx(bar_v_full + 8 * hf, 2 * kVG * kMla2VChunk);
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                tma2_gather4(dst, &tm_rows, pair_v_full + 8 * hf, slab * 64, r[0], r[1], r[2], r[3]);
                ++vc;
            }
        }
    } else if (warp == 1 && leader && lane == 0) {
        // ============ score MMA issuer: one thread for both CTAs of the pair (S = Q K^T) ============
        constexpr uint32_t kIdescQK = idesc_bf16(128, 128, false, false);
        constexpr uint32_t kHi = desc_hi_sw128(1024);
        const uint32_t q_lo = desc_lo_sw128(sQ, 16), k_lo = desc_lo_sw128(sK, 16);
        uint32_t q_it = 0, kc = 0;
        bool ok = true;
        auto qk_group_c = [&](auto gc, uint32_t tS, uint32_t bar_last) {
            constexpr int g = decltype(gc)::value;
#pragma unroll
            for (int s = g * kKG; s < (g + 1) * kKG; ++s) {
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    mma2_ss_lh(tS, q_lo + ((s * 8192 + kk * 32) >> 4), k_lo + ((s * 8192 + kk * 32) >> 4), kHi, kIdescQK,
                               (s > 0 || kk > 0) ? 1u : 0u);
                }
            }
            tc_commit2(g < kKGroups - 1 ? bar_k_empty + 8 * g : bar_last, 3);
        };
        static_assert(kKGroups == 3, "one call per K group");
        for (int t = pair; t < p.total_q && ok; t += num_pairs) {
            if (__ldg(p.tok + t).x < 0) continue;
            ok = mbar_wait(bar_q_full, q_it & 1, s_abort, 921);
            ++q_it;
            for (int jj = 0; jj < n_tiles && ok; ++jj) {
                const uint32_t b = kc & 1, kpar = kc & 1;
                const uint32_t tS = tmem_base + b * 64, bar_s = bar_s_full + 8 * b;
                // S[b] was last read by the softmax of two tiles ago: its P is ready <=> that read is over
                if (kc >= 2) ok = mbar_wait_cluster(bar_p_full + 8 * b, ((kc - 2) >> 1) & 1, s_abort, 920);
                if (!ok) break;
                ok = mbar_wait(bar_k_full, kpar, s_abort, 922);
                if (!ok) break;
                tc_fence_after();
                qk_group_c(std::integral_constant<int, 0>{}, tS, bar_s);
                ok = mbar_wait(bar_k_full + 8, kpar, s_abort, 922);
                if (!ok) break;
                tc_fence_after();
                qk_group_c(std::integral_constant<int, 1>{}, tS, bar_s);
                ok = mbar_wait(bar_k_full + 16, kpar, s_abort, 922);
                if (!ok) break;
                tc_fence_after();
                qk_group_c(std::integral_constant<int, 2>{}, tS, bar_s);
                ++kc;
            }
        }
    } else if (warp == 7 && leader && lane == 0) {
        // ============ P V MMA issuer: one thread for both CTAs of the pair (O += P V) ============
        constexpr uint32_t kIdescPV = idesc_bf16(128, 256, false, true);
        constexpr uint32_t kHi = desc_hi_sw128(1024);
        const uint32_t p_lo = desc_lo_sw128(sP, 16);
        const uint32_t v_lo = desc_lo_sw128(sV, 8192);  // MN-major: 64-column groups 8 KB apart
        const uint32_t tO0 = tmem_base + 128, tO1 = tmem_base + 256;
        uint32_t vc = 0;
        bool ok = true;
        auto pv_group_c = [&](auto gc, auto firstc) {
            constexpr int g = decltype(gc)::value;
            constexpr bool first_tile = decltype(firstc)::value;
#pragma unroll
            for (int c = g * kVG; c < (g + 1) * kVG; ++c) {
                const uint32_t tO = (c & 1) ? tO1 : tO0;
#pragma unroll
                for (int k4 = 0; k4 < 4; ++k4) {
                    mma2_ss_lh(tO, p_lo + (((c >> 1) * 8192 + k4 * 32) >> 4), v_lo + ((c * kMla2VChunk + k4 * 2048) >> 4),
                               kHi, kIdescPV, (!first_tile || c > 1 || k4 > 0) ? 1u : 0u);
                }
            }
            tc_commit2(g < kVGroups - 1 ? bar_v_empty + 8 * g : bar_pv_done, 3);
        };
        static_assert(kVGroups == 2, "one call per V group");
        for (int t = pair; t < p.total_q && ok; t += num_pairs) {
            if (__ldg(p.tok + t).x < 0) continue;
            for (int jj = 0; jj < n_tiles && ok; ++jj) {
                const uint32_t b = vc & 1, vpar = vc & 1;
                ok = mbar_wait_cluster(bar_p_full + 8 * b, (vc >> 1) & 1, s_abort, 926);
                if (!ok) break;
                ok = mbar_wait(bar_v_full, vpar, s_abort, 924);
                if (!ok) break;
                tc_fence_after();
                if (jj == 0) pv_group_c(std::integral_constant<int, 0>{}, std::true_type{});
                else pv_group_c(std::integral_constant<int, 0>{}, std::false_type{});
                ok = mbar_wait(bar_v_full + 8, vpar, s_abort, 924);
                if (!ok) break;
                tc_fence_after();
                if (jj == 0) pv_group_c(std::integral_constant<int, 1>{}, std::true_type{});
                else pv_group_c(std::integral_constant<int, 1>{}, std::false_type{});
                ++vc;
            }
        }
    } else if (warp >= 2 && warp <= 5) {
        // ======================================= softmax =======================================
        const int l128 = ((warp & 3) << 5) | lane;     // TMEM lane
        const int row = l128 & 63;                     // row of this CTA's 64 = q-head 64 rank + row
        const int half = l128 >> 6;                    // which 64 key columns of the tile
        const uint32_t lane_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tO0 = tmem_base + 128 + lane_off, tO1 = tmem_base + 256 + lane_off;
        uint8_t* p_row = gen_base + kMla2QBytes + kMla2KBytes + kMla2VBytes + half * 8192 + row * 128;
        uint32_t tc = 0, x_it = 0;
        const float sc = p.scale_log2e;
        const int h = static_cast<int>(rank) * kMla2Rows + row;
        auto exchange = [&](float mine, float& theirs) -> bool {
            float* buf = xch + (x_it & 1) * 128;
            buf[l128] = mine;
            mbar_arrive(bar_xchg);
            if (!mbar_wait(bar_xchg, x_it & 1, s_abort, 931)) return false;
            theirs = buf[l128 ^ 64];
            ++x_it;
            return true;
        };
        bool ok = true;
        for (int t = pair; t < p.total_q && ok; t += num_pairs) {
            if (__ldg(p.tok + t).x < 0) continue;
            float m_ref = -INFINITY, l_run = 0.f;
            for (int j = 0; j < n_tiles; ++j) {
                const uint32_t b = tc & 1;
                const uint32_t tS = tmem_base + b * 64 + lane_off;
                ok = mbar_wait(bar_s_full + 8 * b, (tc >> 1) & 1, s_abort, 932);
                if (!ok) break;
                tc_fence_after();
                uint32_t s[64];
                tmem_ld32(tS, reinterpret_cast<uint32_t(&)[32]>(s[0]));
                tmem_ld32(tS + 32, reinterpret_cast<uint32_t(&)[32]>(s[32]));
                ok = mbar_wait(bar_mask + 8 * (tc & 3), (tc >> 2) & 1, s_abort, 936);
                if (!ok) break;
                const uint32_t w0 = vmask[(tc & 3) * 4], w1 = vmask[(tc & 3) * 4 + 1], w2 = vmask[(tc & 3) * 4 + 2],
                               w3 = vmask[(tc & 3) * 4 + 3];
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_mask_free + 8 * (tc & 3));
                tc_wait_ld();
                if ((w0 & w1 & w2 & w3) != 0xffffffffu) {   // some listed entries of this tile do not take part
                    const uint32_t we[4] = {w0 >> (half * 16), w1 >> (half * 16), w2 >> (half * 16), w3 >> (half * 16)};
#pragma unroll
                    for (int i = 0; i < 64; ++i)
                        if (!((we[i & 3] >> (i >> 2)) & 1u)) s[i] = 0xff800000u;  // -inf
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
                float mxb;
                ok = exchange(mxa, mxb);
                if (!ok) break;
                const float m_new = fmaxf(fmaxf(mxa, mxb) * sc, m_ref);
                const bool grow = (m_new - m_ref > 8.f) || (m_ref == -INFINITY && m_new != -INFINITY);
                bool p_free = false;
                if (__any_sync(0xffffffffu, grow)) {
                    const float alpha = grow ? ex2(m_ref - m_new) : 1.f;
                    if (grow) m_ref = m_new;
                    l_run *= alpha;
                    if (j > 0) {
                        // O is rescaled in place: P V of the previous tile must be done
                        ok = mbar_wait(bar_pv_done, (tc - 1) & 1, s_abort, 935);
                        if (!ok) break;
                        p_free = true;
                        tc_fence_after();
                        uint32_t o[32];
#pragma unroll 1
                        for (int c = 0; c < 8; ++c) {
                            const uint32_t addr = (c < 4 ? tO0 : tO1) + (c & 3) * 32;
                            tmem_ld32(addr, o);
                            tc_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                            tmem_st32(addr, o);
                        }
                        tc_wait_st();
                    }
                }
                const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
                uint32_t pk[32];
                float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
                for (int i = 0; i < 64; i += 2) {
                    const float p0 = ex2(fmaf(__uint_as_float(s[i]), sc, -m_use));
                    const float p1 = ex2(fmaf(__uint_as_float(s[i + 1]), sc, -m_use));
                    sum0 += p0;
                    sum1 += p1;
                    pk[i >> 1] = pack_bf16x2(p0, p1);
                }
                l_run += sum0 + sum1;
                // P of the previous tile must have been consumed before its shared-memory rows are overwritten
                if (tc > 0 && !p_free) {
                    ok = mbar_wait(bar_pv_done, (tc - 1) & 1, s_abort, 933);
                    if (!ok) break;
                }
#pragma unroll
                for (int c = 0; c < 8; ++c)  // K-major 128B-swizzled row: 16-byte chunk index XOR (row & 7)
                    *reinterpret_cast<uint4*>(p_row + ((c ^ (row & 7)) << 4)) =
                        make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
                fence_proxy_async_smem();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (leader) mbar_arrive(bar_p_full + 8 * b);
                    else mbar_arrive_remote(bar_p_full + 8 * b, 0);
                }
                ++tc;
            }
            if (!ok) break;
            // ---- epilogue ----
            float l_other;
            ok = exchange(l_run, l_other);
            if (!ok) break;
            const float l_tot = l_run + l_other;
            ok = mbar_wait(bar_pv_done, (tc - 1) & 1, s_abort, 934);  // P V of the item's last tile
            if (!ok) break;
            tc_fence_after();
            const float inv_l = l_tot > 0.f ? 1.f / l_tot : 0.f;   // no entry took part: the output is zero
            const bool live = h < p.num_q_heads;
            uint32_t r[32];
#pragma unroll 1
            for (int c = 0; c < 8; ++c) {
                tmem_ld32((c < 4 ? tO0 : tO1) + (c & 3) * 32, r);
                tc_wait_ld();
                if (!live) continue;
                const int col0 = (c >> 2) * 256 + half * 128 + (c & 3) * 32;
                uint4* dst = reinterpret_cast<uint4*>(static_cast<uint8_t*>(p.out) +
                                                      ((static_cast<long long>(t) * p.num_q_heads + h) * kMlaDv + col0) * 2);
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    uint32_t w[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        w[e] = pack_bf16x2(__uint_as_float(r[q4 * 8 + 2 * e]) * inv_l, __uint_as_float(r[q4 * 8 + 2 * e + 1]) * inv_l);
                    dst[q4] = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
            if (live && half == 0 && p.lse)
                p.lse[static_cast<long long>(t) * p.num_q_heads + h] = (m_ref + log2f(l_tot)) * 0.6931471805599453f;
            tc_fence_before();
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
    cluster_sync_all();  // neither CTA frees tensor memory or exits while the other may still signal it
    if (warp == 0) tmem_dealloc2(tmem_base, 512);
}

}  // namespace vpp
