// Warp-specialised persistent chunked-prefill attention kernel for head_dim 128 (MHA / GQA / MQA).
//
// One CTA per SM, 12 warps:
//   warp 0      scheduler + TMA producer: pops work items from the global counter, publishes them in a
//               2-deep shared ring, loads the two Q tiles of the item and streams K/V pages through a
//               ring of 128B-swizzled 32 KB stages (K0 V0 K1 V1 ...), gathered through the block table.
//   warp 1      MMA issuer: tcgen05.mma  S_t = Q_t K^T  and  O_t += P_t V  for the two query tiles
//               t = 0, 1 of the item: two q-heads of one kv-head over the same 128 query tokens (even
//               group sizes) or, when a kv-head's group is odd (MHA included), two consecutive 128-row
//               tiles of ONE q-head -- either way both tiles use the same K/V stages.
//   warp 2      tensor-memory allocation.
//   warps 4-7   softmax group for tile 0: one query row per thread, fp32 online softmax on S_0 read
//               from tensor memory, P_0 written back to tensor memory as bf16 over S_0.
//   warps 8-11  the same for tile 1.
// While one group works on its S tile the tensor core runs the other tile's MMAs.
// A work unit of a single query token (a decode step batched with prefill chunks, or the one-row tail of a chunk) is
// run "packed": the G q-heads that share a kv-head become the rows of the Q tile, so its K/V is streamed once per
// kv-head instead of once per pair of q-heads.  Both tiles then use that one Q tile and split the KV tiles between
// them (even ones to tile 0, odd ones to tile 1) as two independent online softmaxes whose results softmax group 0
// merges at the end -- one softmax chain per KV tile would leave the memory system idle most of the time.
// Tensor memory: S_0 | S_1 | O_0 | O_1, 128 fp32 columns each (all 512 columns).
//
// The math per row is the paper's Eq. 1 with the causal rule, evaluated KV tile by KV tile with a
// running maximum; O is rescaled lazily (only when the maximum has grown by more than 2^8).
#pragma once
#include <type_traits>

#include "common.cuh"
#include "ptx.cuh"

namespace vpp {

constexpr int kWsThreads = 384;
// Register budget per thread after the roles split (setmaxnreg).  The launch gives every warp 168 registers (three warps
// per sub-partition); warps 0-3 (one per sub-partition: producer, MMA issuer, allocator, idle) hand back down to
// kWsRegsLow and each of the two softmax warps of a sub-partition takes kWsRegsHigh: 72 + 2 * 216 = 3 * 168.  With 216
// registers the softmax loop (128 scores of a row live at once) has no spills.
constexpr int kWsRegsLow = 72, kWsRegsHigh = 216;
static_assert(kWsRegsLow + 2 * kWsRegsHigh <= 3 * 168 && kWsRegsLow % 8 == 0 && kWsRegsHigh % 8 == 0, "register budget");
constexpr int kWsStages = 4;                  // 32 KB each
constexpr int kTileBytes = 2 * kSlabBytes;    // one 128 x 128 bf16 tile
// (the two alternating slots of the V-tail barrier cover a producer that runs at most two V tiles ahead of the MMA thread:
//  a ring of more than four stages would need more slots -- five stages failed parity on short items)
static_assert(kWsStages <= 4, "V-tail barrier slots");
constexpr int kWsSmemBytes = 2 * kTileBytes + kWsStages * kTileBytes + 1024 /*align*/ + 2048 /*barriers, ring, merge exchange*/;
constexpr float kRescaleThreshold = 8.f;      // log2 units
// 0: P is handed to the MMA thread whole; c in 1..3: the first 32*c key columns are handed over early so that
// O += P V can start on them while the rest of the exponentials are computed
// Early hand-overs of P: bit c set = the key columns up to 32 (c + 1) are handed to the MMA thread as soon as they are in
// tensor memory, so that O += P V starts on them while the rest of the exponentials are computed (0: P is handed over whole).
constexpr int kPartMask = 3;   // after 32 and after 64 columns (measured best: a hand-over after 96 columns costs more than it gains)
static_assert(kPartMask >= 0 && kPartMask < 8, "hand-overs after 32, 64 and 96 columns only");
constexpr int kPartWaitDefer = 8;             // pairs of columns of the next chunk computed before that hand-over's store is awaited (0: none)
static_assert(kPartWaitDefer >= 1 && kPartWaitDefer <= 16, "the wait sits inside the next chunk");

struct WsItem {
    WorkUnit u;
    int32_t h0;      // first of the two q-heads (packed item: first head of the kv-head's group)
    int32_t valid;   // 0: no more work
    int32_t packed;  // 1: single-token item, the rows of tile 0 are the G q-heads of one kv-head; tile 1 is unused
    int32_t pad;
};


// Merge of the two tiles' partial results of a packed item (rare path, kept out of line to spare the main loop's
// registers):  out = (a0 O_0 + a1 O_1) / (a0 l_0 + a1 l_1),  a_t = 2^(m_t - m).  O_1 sits 128 columns after O_0.
// (every argument by value: a reference to the kernel's parameter block or to the work unit would force them into
// local memory for the whole kernel)
__device__ __noinline__ void ws_packed_merge(void* out, float* lse_out, float* o_parts, float* lse_parts, int total_q,
                                             int num_q_heads, int split, int q_row0, bool second, const float* xm,
                                             uint32_t tO, int row, int tile_rows, int h, float m_ref, float l_run) {
    const float m1 = xm[row], l1 = xm[128 + row];
    const float m = fmaxf(m_ref, m1);
    const float a0 = m_ref == -INFINITY ? 0.f : ex2(m_ref - m), a1 = m1 == -INFINITY ? 0.f : ex2(m1 - m);
    const float l_tot = a0 * l_run + a1 * l1;
    const float s0 = a0 / l_tot, s1 = a1 / l_tot;
    const bool live = row < tile_rows;
    const long long grow_idx = q_row0;
    uint32_t r[16], r1[16];
#pragma unroll 1
    for (int c = 0; c < 8; ++c) {     // 16 output columns at a time (registers)
        tmem_ld16(tO + c * 16, r);
        if (second) tmem_ld16(tO + 128 + c * 16, r1);
        tc_wait_ld();
        if (!live) continue;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            float v = __uint_as_float(r[i]) * s0;
            if (second) v = fmaf(__uint_as_float(r1[i]), s1, v);
            r[i] = __float_as_uint(v);
        }
        if (split < 0) {
            uint4* dst = reinterpret_cast<uint4*>(static_cast<uint8_t*>(out) +
                                                  ((grow_idx * num_q_heads + h) * 128 + c * 16) * 2);
#pragma unroll
            for (int q4 = 0; q4 < 2; ++q4) {
                uint32_t w[4];
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    w[e] = pack_bf16x2(__uint_as_float(r[q4 * 8 + 2 * e]), __uint_as_float(r[q4 * 8 + 2 * e + 1]));
                dst[q4] = make_uint4(w[0], w[1], w[2], w[3]);
            }
        } else {
            float4* dst = reinterpret_cast<float4*>(
                o_parts +
                ((static_cast<long long>(split) * total_q + grow_idx) * num_q_heads + h) * 128 + c * 16);
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4)
                dst[q4] = make_float4(__uint_as_float(r[q4 * 4]), __uint_as_float(r[q4 * 4 + 1]),
                                      __uint_as_float(r[q4 * 4 + 2]), __uint_as_float(r[q4 * 4 + 3]));
        }
    }
    if (live) {
        const float lse = (m + log2f(l_tot)) * 0.6931471805599453f;
        if (split < 0) {
            if (lse_out) lse_out[grow_idx * num_q_heads + h] = lse;
        } else {
            lse_parts[(static_cast<long long>(split) * total_q + grow_idx) * num_q_heads + h] = lse;
        }
    }
}

template <bool kSameHead, bool kVWarp>
__global__ void __launch_bounds__(kWsThreads, 1)
attn128_ws_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                  const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_q2,
                  const __grid_constant__ CUtensorMap tm_k2, const __grid_constant__ CUtensorMap tm_v2,
                  const __grid_constant__ CUtensorMap tm_qh, const AttnParams p, const int kv_box_rows) {
    constexpr bool same_head = kSameHead;
    // same_head: an item is two consecutive 128-row query tiles of one q-head (work units of up to 256 rows) instead of
    // two q-heads over the same 128 rows -- for odd group sizes, where two q-heads need not share a kv-head.  Tile 1 then
    // starts 128 rows (and positions) after tile 0; the KV range of the unit covers tile 1, and the causal mask hides
    // from tile 0 what lies beyond its own rows.
    // tm_qh: the q tensor with a box of (64 features, G heads, 1 token): the rows of a packed item's Q tile
    // tm_q2 / tm_k2 / tm_v2 are views of the same tensors with the 128 features split into (64, 2): one box
    // of them brings both 64-column slabs of a 128-row tile, i.e. a whole tile per copy instruction.  Issuing a
    // copy costs the producer thread several hundred cycles, so fewer, larger copies matter.  tm_k / tm_v
    // (one slab of kv_box_rows keys per box) serve pages smaller than a KV tile.
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gen_base = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sQ = smem_base;                       // 2 tiles
    const uint32_t sKV = sQ + 2 * kTileBytes;            // kWsStages tiles
    const uint32_t sBar = sKV + kWsStages * kTileBytes;  // barriers
    // barrier map (8 bytes each)
    const uint32_t bar_item_full = sBar + 0;     // [2]
    const uint32_t bar_item_empty = sBar + 16;   // [2]
    const uint32_t bar_q_full = sBar + 32;
    const uint32_t bar_q_empty = sBar + 40;
    const uint32_t bar_s_full = sBar + 48;       // [2]
    const uint32_t bar_p_full = sBar + 64;       // [2]
    const uint32_t bar_o_full = sBar + 80;       // [2]
    // Two slots used alternately: the producer can fix up the V tile of the next short item before the MMA thread has
    // looked at the barrier for this one (slot k & 1 for the k-th such tile, 24 bytes apart).
    const uint32_t bar_vfix = sBar + 96;
    // [3][2] early hand-overs of P: part c (the key columns up to 32 (c + 1)) of tile t is in place.  One barrier per part:
    // the MMA thread may look at part 0 only after part 1 has arrived too, which a shared barrier could not tell apart.
    const uint32_t bar_p_part = sBar + 208;
    const uint32_t bar_kv_full = sBar + 128;     // [kWsStages]
    const uint32_t bar_kv_empty = sBar + 128 + 8 * kWsStages;
    const uint32_t bar_x1 = sBar + 128 + 16 * kWsStages;       // packed item: group 1 has published its (m, l) per row
    const uint32_t bar_x0 = sBar + 128 + 16 * kWsStages + 8;   // packed item: group 0 has merged, tile 1 may be reused
    uint8_t* gen_bar = gen_base + (2 + kWsStages) * kTileBytes;
    volatile int* s_abort = reinterpret_cast<volatile int*>(gen_bar + 512);
    volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(gen_bar + 516);
    WsItem* ring = reinterpret_cast<WsItem*>(gen_bar + 576);  // 2 x 48 bytes
    float* xm = reinterpret_cast<float*>(gen_bar + 1024);     // [2][128]: running maximum and row sum of tile 1 (packed items)

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar_item_full + 8 * i, 1);
            mbar_init(bar_item_empty + 8 * i, kVWarp ? 10 : 9);   // 8 softmax warps, the MMA thread, (the second producer)
            mbar_init(bar_s_full + 8 * i, 1);
            mbar_init(bar_p_full + 8 * i, 4);   // one arrival per softmax warp
            for (int c = 0; c < 3; ++c) mbar_init(bar_p_part + 16 * c + 8 * i, 4);
            mbar_init(bar_o_full + 8 * i, 1);
        }
        mbar_init(bar_q_full, 1);
        mbar_init(bar_q_empty, 1);
        mbar_init(bar_vfix, 1);
        mbar_init(bar_vfix + 24, 1);
        mbar_init(bar_x1, 4);
        mbar_init(bar_x0, 4);
        for (int i = 0; i < kWsStages; ++i) {
            mbar_init(bar_kv_full + 8 * i, 1);
            mbar_init(bar_kv_empty + 8 * i, 1);
        }
        fence_mbar_init();
        *s_abort = 0;
        prefetch_tmap(&tm_q);
        prefetch_tmap(&tm_k);
        prefetch_tmap(&tm_v);
        prefetch_tmap(&tm_q2);
        prefetch_tmap(&tm_k2);
        prefetch_tmap(&tm_v2);
        prefetch_tmap(&tm_qh);
    }
    __syncthreads();
    if (warp == 2) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(s_tmem)), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *s_tmem;

    pdl_wait();                  // the work list comes from the work-decomposition kernel launched just before
    pdl_launch_dependents();     // (the merge kernel, if any, waits for this grid to finish in the same way)
    const int num_units = p.header_ro->num_units;
    const int G = p.num_q_heads / p.num_kv_heads;
    // Items: (unit, pair of q-heads) for the units of several rows, then (unit, kv-head) for the single-token units at the
    // end of the list, which run packed when a kv-head's group fits a tile.
    const int num_packed = G <= kTileM ? p.header_ro->num_single : 0;
    const int num_normal = num_units - num_packed;
    const int heads_per_item = same_head ? 1 : 2;
    const int normal_items = num_normal * (p.num_q_heads / heads_per_item);
    const int total_items = normal_items + num_packed * p.num_kv_heads;

    if (warp < 4) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kWsRegsLow));
        // One K (which = 0) or V (which = 1) tile of the item into the next ring stage, by the calling warp.
        auto load_kv_tile = [&](const WorkUnit& u, int g, int tile0, int which, uint32_t kv_it, uint32_t& vfix_cnt) -> bool {
            bool ok = true;
                const uint32_t st = kv_it % kWsStages;
                const uint32_t ph = (kv_it / kWsStages) & 1;
                const uint32_t dst = sKV + st * kTileBytes;
                const uint32_t full = bar_kv_full + 8 * st;
                const CUtensorMap* tm = which == 0 ? &tm_k : &tm_v;
                const CUtensorMap* tm2 = which == 0 ? &tm_k2 : &tm_v2;
                if (lane == 0) {
                    ok = mbar_wait(bar_kv_empty + 8 * st, ph ^ 1, s_abort, 203);
                    if (ok) {
                        mbar_arrive_expect_tx(full, kTileBytes);
                        if (kv_box_rows == kTileN) {
                            int blk, slot_in;
                            if (p.block_table == nullptr) {
                                blk = u.req;
                                slot_in = tile0;
                            } else if (tile0 < u.kv_len) {
                                blk = __ldg(p.block_table + static_cast<long long>(u.req) * p.max_blocks_per_req +
                                            (tile0 >> p.block_shift));
                                slot_in = tile0 & ((1 << p.block_shift) - 1);
                            } else {
                                blk = p.num_blocks;
                                slot_in = 0;
                            }
                            tma_load_5d(dst, tm2, full, 0, slot_in, 0, g, blk);
                        }
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) return false;
                if (kv_box_rows != kTileN) {
                    // Pages smaller than a KV tile: one copy per (page, 64-column slab), each issued by a lane of its
                    // own -- every lane looks up its page itself, and a lane's copy costs the warp a third of what a
                    // single thread spends on one with its address arithmetic.  (The byte count was posted above.)
                    const int per = kTileN / kv_box_rows;             // pages per tile: 2 .. 8
                    if (lane < 2 * per) {
                        const int off = (lane >> 1) * kv_box_rows, sl = lane & 1;
                        const int pos = tile0 + off;
                        int blk, slot_in;
                        if (p.block_table == nullptr) {
                            blk = u.req;
                            slot_in = pos;
                        } else if (pos < u.kv_len) {
                            blk = __ldg(p.block_table + static_cast<long long>(u.req) * p.max_blocks_per_req +
                                        (pos >> p.block_shift));
                            slot_in = pos & ((1 << p.block_shift) - 1);
                        } else {
                            blk = p.num_blocks;  // out of range: the copy engine fills zeros
                            slot_in = 0;
                        }
                        tma_load_4d(dst + sl * kSlabBytes + static_cast<uint32_t>(off) * 128u, tm, full, sl * 64, slot_in, g, blk);
                    }
                    __syncwarp();
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) return false;
                if (which == 1 && tile0 + kTileN > u.kv_len) {
                    // Keys at or beyond kv_len do not exist; zero their V rows so that 0 * garbage
                    // cannot poison O.  The MMA warp waits for bar_vfix on such a tile.
                    if (lane == 0) ok = mbar_wait(full, ph, s_abort, 204);
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) return false;
                    uint8_t* vb = gen_base + 2 * kTileBytes + st * kTileBytes;
                    const int first = u.kv_len > tile0 ? u.kv_len - tile0 : 0;
                    const uint4 z = make_uint4(0, 0, 0, 0);
                    for (int r = first + lane; r < kTileN; r += 32) {
                        uint4* a = reinterpret_cast<uint4*>(vb + r * 128);
                        uint4* b = reinterpret_cast<uint4*>(vb + kSlabBytes + r * 128);
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            a[c] = z;
                            b[c] = z;
                        }
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_vfix + 24 * (vfix_cnt & 1));
                    ++vfix_cnt;
                }
            return true;
        };
        // kVWarp: a second producer warp (warp 2) loads the V tiles, warp 0 the K tiles.  The host chooses it for the launches
        // that are bound by how fast K/V arrives: pages smaller than a KV tile (a tile is then 4 to 16 copies per operand)
        // and batches of decode rows, which stream K/V at memory speed (+10 to 18 % with K and V requested by two warps).
        // Prefill over large pages keeps the single producer (a second one costs it 1 to 2 %).
        constexpr bool split_v = kVWarp;
        if (warp == 0) {
            // ============================ scheduler + TMA producer ============================
            uint32_t item_it = 0, q_it = 0, kv_it = 0, vfix_cnt = 0;
            while (true) {
                int item = 0;
                if (lane == 0) item = atomicAdd(&p.header->counter, 1);
                item = __shfl_sync(0xffffffffu, item, 0);
                const bool have = item < total_items;
                WorkUnit u{};
                int h0 = 0;
                bool packed = false;
                if (have && item < normal_items) {
                    int ui, hp;
                    decode_item(item, num_normal, p.num_q_heads / heads_per_item, G / heads_per_item, ui, hp);
                    u = p.units[ui];
                    h0 = heads_per_item * hp;
                } else if (have) {
                    const int k = item - normal_items;
                    u = p.units[num_normal + k / p.num_kv_heads];
                    h0 = (k % p.num_kv_heads) * G;
                    packed = true;
                }
                const uint32_t slot = item_it & 1;
                bool ok = true;
                if (lane == 0) ok = mbar_wait(bar_item_empty + 8 * slot, ((item_it >> 1) & 1) ^ 1, s_abort, 201);
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                if (lane == 0) {
                    ring[slot].u = u;
                    ring[slot].h0 = h0;
                    ring[slot].valid = have ? 1 : 0;
                    ring[slot].packed = packed ? 1 : 0;
                    mbar_arrive(bar_item_full + 8 * slot);
                }
                ++item_it;
                if (!have) break;
                const int g = h0 / G;

                if (lane == 0) {
                    ok = mbar_wait(bar_q_empty, (q_it & 1) ^ 1, s_abort, 202);
                    if (ok && packed) {
                        // rows = the G heads of this kv-head for the one token; rows G..127 keep whatever they held
                        mbar_arrive_expect_tx(bar_q_full, 2 * G * 128);
                        tma_load_3d(sQ, &tm_qh, bar_q_full, 0, h0, u.q_row0);
                        tma_load_3d(sQ + kSlabBytes, &tm_qh, bar_q_full, 64, h0, u.q_row0);
                    } else if (ok) {
                        mbar_arrive_expect_tx(bar_q_full, 2 * kTileBytes);
                        tma_load_4d(sQ, &tm_q2, bar_q_full, 0, u.q_row0, 0, h0);
                        // (rows past the end of q read as zero; rows of a following request are never stored)
                        tma_load_4d(sQ + kTileBytes, &tm_q2, bar_q_full, 0, u.q_row0 + (same_head ? kTileM : 0), 0,
                                    h0 + (same_head ? 0 : 1));
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                ++q_it;

                for (int j = u.kv_begin; j < u.kv_end && ok; ++j) {
#pragma unroll
                    for (int which = 0; which < 2; ++which) {  // 0: K, 1: V
                        if (!(split_v && which == 1)) ok = load_kv_tile(u, g, j * kTileN, which, kv_it, vfix_cnt);
                        if (!ok) break;
                        ++kv_it;
                    }
                }
                if (!ok) break;
            }
        } else if (warp == 2 && split_v) {
            // ============================ second producer: the V tiles when pages are small ============================
            // (follows the item ring like every other role)
            uint32_t item_it = 0, kv_it = 0, vfix_cnt = 0;
            while (true) {
                const uint32_t slot = item_it & 1;
                bool ok = true;
                if (lane == 0) ok = mbar_wait(bar_item_full + 8 * slot, (item_it >> 1) & 1, s_abort, 211);
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                const WorkUnit u = ring[slot].u;
                const int g = ring[slot].h0 / G;
                const int valid = ring[slot].valid;
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_item_empty + 8 * slot);
                ++item_it;
                if (!valid) break;
                for (int j = u.kv_begin; j < u.kv_end && ok; ++j) {
                    ++kv_it;                                             // (the K tile: warp 0's)
                    ok = load_kv_tile(u, g, j * kTileN, 1, kv_it, vfix_cnt);
                    ++kv_it;
                }
                if (!ok) break;
            }
        } else if (warp == 1 && lane == 0) {
            // ============================ MMA issuer (a single thread) ============================
            constexpr uint32_t kIdescQK = idesc_bf16(128, 128, false, false);
            constexpr uint32_t kIdescPV = idesc_bf16(128, 128, false, true);
            const uint32_t tS0 = tmem_base, tS1 = tmem_base + 128, tO0 = tmem_base + 256, tO1 = tmem_base + 384;
            uint32_t item_it = 0, q_it = 0, kv_it = 0, vfix_it = 0, p_it = 0, p_it1 = 0;   // P hand-offs seen per tile
            auto wait1 = [&](uint32_t bar, uint32_t parity, int where) -> bool {
                return mbar_wait(bar, parity, s_abort, where);
            };
            // Descriptors are advanced by adding constants to their low word: the single issuing thread
            // must not spend longer building operands than the tensor core spends on the MMA.
            constexpr uint32_t kHi = desc_hi_sw128(1024);
            const uint32_t q_lo0 = desc_lo_sw128(sQ, 16), q_lo1 = desc_lo_sw128(sQ + kTileBytes, 16);
            auto issue_qk = [&](uint32_t tS, uint32_t q_lo, uint32_t k_stage) {
                const uint32_t k_lo = desc_lo_sw128(k_stage, 16);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const uint32_t koff = ((k >> 2) * kSlabBytes + (k & 3) * 32) >> 4;
                    mma_ss_lh(tS, q_lo + koff, k_lo + koff, kHi, kIdescQK, k > 0);
                }
            };
            auto issue_pv = [&](uint32_t tO, uint32_t tP, uint32_t v_stage, bool first, int k0, int k1) {
                const uint32_t v_lo = desc_lo_sw128(v_stage, kSlabBytes);
#pragma unroll
                for (int k = k0; k < k1; ++k) {
                    mma_ts_lh(tO, tP + k * 8, v_lo + k * (2048 >> 4), kHi, kIdescPV, (!first || k > 0) ? 1u : 0u);
                }
            };
            // O_t += P_t V for one KV tile, following the hand-overs: every early part as soon as it is there, the rest after
            // the whole of P.  pit = hand-overs of P_t seen so far (tile visits).
            auto pv_tile = [&](int t, uint32_t tO, uint32_t tS, uint32_t v_stage, bool first, uint32_t pit, int where) -> bool {
                int k0 = 0;
#pragma unroll
                for (int c = 0; c < 3; ++c) {
                    if ((kPartMask >> c) & 1) {
                        if (!wait1(bar_p_part + 16 * c + 8 * t, pit & 1, where)) return false;
                        tc_fence_after();
                        issue_pv(tO, tS, v_stage, first, k0, 2 * (c + 1));
                        k0 = 2 * (c + 1);
                    }
                }
                if (!wait1(bar_p_full + 8 * t, pit & 1, where + 1)) return false;
                tc_fence_after();
                issue_pv(tO, tS, v_stage, first, k0, 8);
                return true;
            };
            while (true) {
                const uint32_t slot = item_it & 1;
                if (!wait1(bar_item_full + 8 * slot, (item_it >> 1) & 1, 301)) break;
                const WorkUnit u = ring[slot].u;
                const int valid = ring[slot].valid;
                const bool packed = ring[slot].packed != 0;
                mbar_arrive(bar_item_empty + 8 * slot);
                ++item_it;
                if (!valid) break;
                const int n = u.kv_end - u.kv_begin;
                if (!wait1(bar_q_full, q_it & 1, 302)) break;
                ++q_it;
                if (packed) {
                    // Packed single-token item: both tiles hold the same Q (the heads of one kv-head) and share the KV
                    // range -- tile t takes the KV tiles kv_begin + t, + t + 2, ... as an independent online softmax
                    // (its own S_t, O_t); the two partial results are merged by softmax group 0 at the end.
                    // Ring index of K(jj) is base + 2 jj, of V(jj) base + 2 jj + 1.
                    const uint32_t base = kv_it;
                    bool ok = true;
                    auto do_qk = [&](int jj) {
                        const uint32_t idx = base + 2 * jj, st = idx % kWsStages;
                        if (!wait1(bar_kv_full + 8 * st, (idx / kWsStages) & 1, 321)) return false;
                        tc_fence_after();
                        issue_qk((jj & 1) ? tS1 : tS0, q_lo0, sKV + st * kTileBytes);
                        tc_commit(bar_s_full + 8 * (jj & 1));
                        tc_commit(bar_kv_empty + 8 * st);
                        if (jj + 1 == n) tc_commit(bar_q_empty);
                        return true;
                    };
                    ok = do_qk(0);
                    if (ok && n > 1) ok = do_qk(1);
                    for (int jj = 0; jj < n && ok; ++jj) {
                        const int t = jj & 1;
                        const int tile0 = (u.kv_begin + jj) * kTileN;
                        const uint32_t idx = base + 2 * jj + 1, st = idx % kWsStages;
                        const uint32_t pit = t ? p_it1 : p_it;   // (no reference: the counters must stay in registers)
                        ok = wait1(bar_kv_full + 8 * st, (idx / kWsStages) & 1, 322);
                        if (!ok) break;
                        if (tile0 + kTileN > u.kv_len) {
                            ok = wait1(bar_vfix + 24 * (vfix_it & 1), (vfix_it >> 1) & 1, 323);
                            if (!ok) break;
                            ++vfix_it;
                        }
                        const uint32_t tO = t ? tO1 : tO0, tS = t ? tS1 : tS0;
                        ok = pv_tile(t, tO, tS, sKV + st * kTileBytes, jj < 2, pit, 324);
                        if (!ok) break;
                        tc_commit(bar_kv_empty + 8 * st);
                        if (t) ++p_it1; else ++p_it;
                        if (jj + 2 < n) ok = do_qk(jj + 2);
                        else tc_commit(bar_o_full + 8 * t);     // this tile's last KV tile
                    }
                    if (!ok) break;
                    kv_it = base + 2 * n;
                    continue;
                }
                // S_t(0) = Q_t K(0)^T
                uint32_t stK = kv_it % kWsStages;
                if (!wait1(bar_kv_full + 8 * stK, (kv_it / kWsStages) & 1, 303)) break;
                ++kv_it;
                tc_fence_after();
                if (lane == 0) {
                    issue_qk(tS0, q_lo0, sKV + stK * kTileBytes);
                    tc_commit(bar_s_full);
                    issue_qk(tS1, q_lo1, sKV + stK * kTileBytes);
                    tc_commit(bar_s_full + 8);
                    tc_commit(bar_kv_empty + 8 * stK);
                    if (n == 1) tc_commit(bar_q_empty);
                }
                bool ok = true;
                for (int jj = 0; jj < n && ok; ++jj) {
                    const int tile0 = (u.kv_begin + jj) * kTileN;
                    const uint32_t stV = kv_it % kWsStages;
                    ok = wait1(bar_kv_full + 8 * stV, (kv_it / kWsStages) & 1, 304);
                    if (!ok) break;
                    ++kv_it;
                    if (tile0 + kTileN > u.kv_len) {
                        ok = wait1(bar_vfix + 24 * (vfix_it & 1), (vfix_it >> 1) & 1, 305);
                        if (!ok) break;
                        ++vfix_it;
                    }
                    const bool has_next = jj + 1 < n;
                    stK = kv_it % kWsStages;
                    // ---- tile 0 ----
                    ok = pv_tile(0, tO0, tS0, sKV + stV * kTileBytes, jj == 0, p_it, 308);
                    if (!ok) break;
                    if (has_next) {
                        ok = wait1(bar_kv_full + 8 * stK, (kv_it / kWsStages) & 1, 307);
                        if (!ok) break;
                        tc_fence_after();
                        if (lane == 0) {
                            issue_qk(tS0, q_lo0, sKV + stK * kTileBytes);
                            tc_commit(bar_s_full);
                        }
                    } else if (lane == 0) {
                        tc_commit(bar_o_full);
                    }
                    // ---- tile 1 ----
                    ok = pv_tile(1, tO1, tS1, sKV + stV * kTileBytes, jj == 0, p_it1, 312);
                    if (!ok) break;
                    if (lane == 0) {
                        tc_commit(bar_kv_empty + 8 * stV);
                        if (has_next) {
                            issue_qk(tS1, q_lo1, sKV + stK * kTileBytes);
                            tc_commit(bar_s_full + 8);
                            tc_commit(bar_kv_empty + 8 * stK);
                            if (jj + 2 == n) tc_commit(bar_q_empty);
                        } else {
                            tc_commit(bar_o_full + 8);
                        }
                    }
                    if (has_next) ++kv_it;
                    ++p_it;
                    ++p_it1;
                }
                if (!ok) break;
            }
        }
        // warps 2 and 3 have nothing to do until teardown
    } else {
        // ===================================== softmax groups =====================================
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kWsRegsHigh));
        const int t = (warp - 4) >> 2;                 // query tile / softmax group
        const int row = ((warp & 3) << 5) | lane;      // row of the tile = TMEM lane
        const uint32_t lane_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tS = tmem_base + t * 128 + lane_off;
        const uint32_t tO = tmem_base + 256 + t * 128 + lane_off;
        const uint32_t bar_s = bar_s_full + 8 * t, bar_p = bar_p_full + 8 * t, bar_o = bar_o_full + 8 * t;
        uint32_t item_it = 0, s_it = 0, o_it = 0, x_it = 0;
        const float sc = p.scale_log2e;
        while (true) {
            const uint32_t slot = item_it & 1;
            if (!mbar_wait(bar_item_full + 8 * slot, (item_it >> 1) & 1, s_abort, 401)) break;
            const WorkUnit u = ring[slot].u;
            const bool packed = ring[slot].packed != 0;
            // packed: row r of tile 0 is q-head h0 + r; otherwise tile t is q-head h0 + t, or rows 128 t .. of q-head h0
            const int h = ring[slot].h0 + (packed ? row : (same_head ? 0 : t));
            const int row_base = (!packed && same_head) ? t * kTileM : 0;
            const int valid = ring[slot].valid;
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_item_empty + 8 * slot);
            ++item_it;
            if (!valid) break;
            // One item's softmax work.  The packed variant (single-token items) is compiled separately so that the
            // prefill path keeps the registers and the instruction count it had without it.
            auto run_item = [&](auto packed_tag) -> bool {
            constexpr bool kPacked = decltype(packed_tag)::value;
            // rows of this thread's warp that exist: a packed tile has G rows, a warp without any only keeps the
            // barriers moving
            const int tile_rows = kPacked ? G : u.rows - row_base;   // (<= 0: tile 1 of a unit of at most 128 rows is idle)
            const bool warp_idle = kPacked && (warp & 3) * 32 >= G;

            const int tile_pos0 = u.pos0 + row_base;               // position of the tile's first row
            const int my_pos = kPacked ? u.pos0 : tile_pos0 + row;
            float m_ref = -INFINITY, l_run = 0.f;
            bool ok = true;
            // a packed item: this group's tile takes every second KV tile
            for (int j = u.kv_begin + (kPacked ? t : 0); j < u.kv_end; j += kPacked ? 2 : 1) {
                const int tile0 = j * kTileN;
                ok = mbar_wait(bar_s, s_it & 1, s_abort, 402);
                if (!ok) break;
                ++s_it;
                tc_fence_after();
                if (warp_idle) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) {
#pragma unroll
                        for (int c = 0; c < 3; ++c)
                            if ((kPartMask >> c) & 1) mbar_arrive(bar_p_part + 16 * c + 8 * t);
                        mbar_arrive(bar_p);
                    }
                    continue;
                }
                uint32_t s[128];
                const bool diag = tile0 + kTileN - 1 > tile_pos0;  // keys beyond the row's position are masked
                const int lim = my_pos - tile0;                 // columns <= lim are visible
                float mx[8];
                // the second half of the row is still in flight while the first half is reduced
                tmem_ld32(tS, reinterpret_cast<uint32_t(&)[32]>(s[0]));
                tmem_ld32(tS + 32, reinterpret_cast<uint32_t(&)[32]>(s[32]));
                tc_wait_ld();
                tmem_ld32(tS + 64, reinterpret_cast<uint32_t(&)[32]>(s[64]));
                tmem_ld32(tS + 96, reinterpret_cast<uint32_t(&)[32]>(s[96]));
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    if (hh == 1) tc_wait_ld();
                    if (diag) {
#pragma unroll
                        for (int i = 0; i < 64; ++i)
                            if (hh * 64 + i > lim) s[hh * 64 + i] = 0xff800000u;  // -inf
                    }
#pragma unroll
                    for (int i = 0; i < 64; i += 16)
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            const float v0 = __uint_as_float(s[hh * 64 + i + k]), v1 = __uint_as_float(s[hh * 64 + i + 8 + k]);
                            mx[k] = (hh == 0 && i == 0) ? fmaxf(v0, v1) : fmax3(mx[k], v0, v1);
                        }
                }
                const float mxa = fmaxf(fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])),
                                        fmaxf(fmaxf(mx[4], mx[5]), fmaxf(mx[6], mx[7])));
                const float m_new = fmaxf(mxa * sc, m_ref);
                // lazy rescale: keep the old reference unless the maximum moved by more than 2^8
                // (rows beyond the tile's last one hold leftovers: they never ask for a rescale)
                const bool grow = row < tile_rows &&
                                  ((m_new - m_ref > kRescaleThreshold) || (m_ref == -INFINITY && m_new != -INFINITY));
                if (__any_sync(0xffffffffu, grow)) {
                    const float alpha = grow ? ex2(m_ref - m_new) : 1.f;  // m_ref = -inf gives 0
                    if (grow) m_ref = m_new;
                    l_run *= alpha;
                    if (j > u.kv_begin + (kPacked ? t : 0)) {   // O of this tile already holds something
                        uint32_t o[32];
#pragma unroll 1
                        for (int c = 0; c < 4; ++c) {
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
                // The wait for the early hand-over's store comes kPartWaitDefer pairs into the next chunk, so that the warp keeps
                // issuing exponentials while the store completes.
                constexpr int kDefer = kPartWaitDefer;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        const float x0 = fmaf(__uint_as_float(s[c * 32 + i]), sc, -m_use);
                        const float x1 = fmaf(__uint_as_float(s[c * 32 + i + 1]), sc, -m_use);
                        const float p0 = ex2(x0), p1 = ex2(x1);
                        sum0 += p0;
                        sum1 += p1;
                        pk[i >> 1] = pack_bf16x2(p0, p1);
                        if (c > 0 && ((kPartMask >> (c - 1)) & 1) && (i >> 1) == kDefer - 1) {
                            tc_wait_st();
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(bar_p_part + 16 * (c - 1) + 8 * t);
                        }
                    }
                    tmem_st16(tS + c * 16, pk);
                }
                l_run += sum0 + sum1;
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_p);
            }
            if (!ok) return false;

            // ---- epilogue ----
            const bool have_tiles = !kPacked || u.kv_begin + t < u.kv_end;   // (tile 1 of a one-tile packed item has none)
            if (have_tiles) {
                ok = mbar_wait(bar_o, o_it & 1, s_abort, 403);
                if (!ok) return false;
                ++o_it;
            }
            tc_fence_after();
            if (kPacked && t == 1) {
                // hand (m, l) of every row to group 0, which also reads O_1; wait until it is done with them
                xm[row] = m_ref;
                xm[128 + row] = l_run;
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_x1);
                ok = mbar_wait(bar_x0, x_it & 1, s_abort, 404);
                if (!ok) return false;
                ++x_it;
                return true;
            }
            if (kPacked) {
                // merge the two tiles' partial results:  out = (a0 O_0 + a1 O_1) / (a0 l_0 + a1 l_1),  a_t = 2^(m_t - m)
                ok = mbar_wait(bar_x1, x_it & 1, s_abort, 405);
                if (!ok) return false;
                ++x_it;
                tc_fence_after();
                ws_packed_merge(p.out, p.lse, p.o_parts, p.lse_parts, p.total_q, p.num_q_heads, u.split, u.q_row0,
                                u.kv_begin + 1 < u.kv_end /* O_1 was written at all */, xm, tO, row, tile_rows, h, m_ref, l_run);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_x0);
                return true;
            }
            {
                const float inv_l = 1.f / l_run;
                const bool live = row < tile_rows;
                const long long grow_idx = static_cast<long long>(u.q_row0) + row_base + row;
                uint32_t r[32];
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    tmem_ld32(tO + c * 32, r);
                    tc_wait_ld();
                    if (!live) continue;
                    if (u.split < 0) {
                        uint4* dst = reinterpret_cast<uint4*>(static_cast<uint8_t*>(p.out) +
                                                              ((grow_idx * p.num_q_heads + h) * 128 + c * 32) * 2);
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
                            ((static_cast<long long>(u.split) * p.total_q + grow_idx) * p.num_q_heads + h) * 128 + c * 32);
#pragma unroll
                        for (int q4 = 0; q4 < 8; ++q4)
                            dst[q4] = make_float4(__uint_as_float(r[q4 * 4]) * inv_l, __uint_as_float(r[q4 * 4 + 1]) * inv_l,
                                                  __uint_as_float(r[q4 * 4 + 2]) * inv_l,
                                                  __uint_as_float(r[q4 * 4 + 3]) * inv_l);
                    }
                }
                if (live) {
                    const float lse = (m_ref + log2f(l_run)) * 0.6931471805599453f;
                    if (u.split < 0) {
                        if (p.lse) p.lse[grow_idx * p.num_q_heads + h] = lse;
                    } else {
                        p.lse_parts[(static_cast<long long>(u.split) * p.total_q + grow_idx) * p.num_q_heads + h] = lse;
                    }
                }
            }
            tc_fence_before();
            return true;
            };
            if (!(packed ? run_item(std::true_type{}) : run_item(std::false_type{}))) break;
        }
    }

    // ---- teardown ----
    __syncthreads();
    if (*s_abort != 0) {
        if (tid == 0 && p.status) atomicCAS(p.status, 0, 3 /* VPP_DEV_TIMEOUT */);
        for (int i = 0; i < 64; ++i) __nanosleep(1000);  // let copies and MMAs in flight drain
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 2) tmem_dealloc(tmem_base, 512);
}

}  // namespace vpp
