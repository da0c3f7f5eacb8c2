// Chunked-prefill attention for absorbed MLA (576-wide keys, values = first 512 features of the same row)
// on a pair of SMs: a 2-CTA cluster issues tcgen05.mma with cta_group::2.
//
// Why a pair: a 128-row query tile with a 512-wide fp32 output fills the tensor memory of one SM, so a single
// CTA has to recompute the scores once per output half.  With cta_group::2 and M = 128 each CTA owns 64 rows,
// and an accumulator of N columns takes only N/2 tensor-memory columns per CTA (rows 0..63 of the CTA sit in
// lanes 0..63 for the first N/2 columns and in lanes 64..127 for the second N/2).  O (64 x 512) then needs 256
// columns and two score buffers 128: everything fits and every score is computed once.  The B operands are
// split between the two CTAs' shared memories -- the 128 keys of a KV tile for S = Q K^T (64 keys each), the
// 256 value columns of each P V instruction (128 each) -- so each K/V byte is fetched from L2 once per 128
// query rows without any multicast copy.
//
// Per CTA, 8 warps:
//   warp 0      one thread: Q and K producer (TMA); the warp also allocates tensor memory
//   warp 1      rank 0: the thread that issues the score MMAs of the pair and their multicast commits; rank 1: idle
//   warp 7      rank 0: the thread that issues the P V MMAs of the pair; rank 1: idle
//   warps 2-5   softmax: lane l of tensor memory holds 64 score columns of row l & 63; the two threads of a row
//               exchange their row maximum through shared memory; P goes to shared memory (K-major, 128B swizzle)
//   warp 6      V producer (TMA) and zero-fill of value rows past the end of the sequence
// Copies issued by either CTA post their bytes on the leader's barriers (cp.async.bulk.tensor with cta_group::2,
// no multicast), so the MMA thread waits on local barriers only.
//
// What bounds the loop is the single issuing thread and the tensor pipe's fixed costs, measured on a B200:
// a tcgen05.mma of this shape occupies the pipe for at least ~48 clk (N = 128) or ~67 clk (N = 256), and every
// tcgen05.commit adds a bubble of ~90 clk.  Hence few commits (five per KV tile), each doubling as several
// signals, and K / V handed back to the producers in groups (3 x 3 slabs, 2 x 32 KB) so that the copy of the
// next tile overlaps the MMAs of this one although shared memory holds only one K and one V tile.
// Pairs walk the work list round-robin (pair p takes items p, p + #pairs, ...), so the two CTAs of a pair agree
// on the item sequence without exchanging anything.
// The math per row is the paper's Eq. 1 with the causal rule, KV tile by KV tile with a running maximum.
#pragma once
#include <type_traits>

#include "common.cuh"
#include "ptx.cuh"

namespace vpp {

constexpr int kMlaDqk = 576, kMlaDv = 512;         // latent row: 512 value features + 64 rope features
constexpr int kMlaSlabs = kMlaDqk / 64;            // 9 slabs of 64 features

constexpr int kMla2Threads = 256;
constexpr int kMla2Rows = 64;                                 // query rows per CTA
constexpr int kMla2QBytes = kMlaSlabs * kMla2Rows * 128;      // 72 KB: 9 slabs x 64 rows
constexpr int kMla2KBytes = kMlaSlabs * 64 * 128;             // 72 KB: 9 slabs x 64 keys (this CTA's half of a tile)
constexpr int kMla2VBytes = 2 * 2 * 2 * 64 * 128;             // 64 KB: [key half][instr][col group][64 keys][128 B]
constexpr int kMla2PBytes = 2 * kMla2Rows * 128;              // 16 KB: 2 slabs x 64 rows
constexpr int kMla2VChunks = 4;                               // V is refilled in 16 KB chunks: (key half, instr)
constexpr int kMla2VChunk = kMla2VBytes / kMla2VChunks;
constexpr int kKG = 3;  // K slabs per hand-back group (3 groups per tile)
constexpr int kVG = 2;  // V chunks per hand-back group (2 groups per tile: key half 0, key half 1)
constexpr int kKGroups = kMlaSlabs / kKG, kVGroups = kMla2VChunks / kVG;
constexpr int kMla2SmemBytes = kMla2QBytes + kMla2KBytes + kMla2VBytes + kMla2PBytes + 1024 /*align*/ + 1536;

// ---- the pair protocol as checkable facts --------------------------------------------------------------------
// Copy boxes (elements of the tensor maps the host encodes; the host uses these constants):
constexpr int kMla2BoxCols = 64, kMla2BoxRows = 64;                       // 64 features x 64 rows / keys per slab
constexpr int kMla2QBoxBytes = kMla2BoxCols * kMla2BoxRows * kMlaSlabs * 2;   // one copy: all nine slabs of a CTA's 64 rows
constexpr int kMla2KBoxBytes = kMla2BoxCols * kMla2BoxRows * kKG * 2;         // one copy: one K hand-back group of a CTA
constexpr int kMla2VBoxSlabs = 2;                                             // one copy: one V chunk = 2 slabs x 64 keys
constexpr int kMla2VBoxBytes = kMla2BoxCols * kMla2BoxRows * kMla2VBoxSlabs * 2;
// Bytes announced on a barrier = sum of the boxes of the copies that post on it:
//   bar_q_full            2 CTAs x 1 copy  of kMla2QBoxBytes         (announced: 2 * kMla2QBytes)
//   bar_k_full[g]         2 CTAs x 1 copy  of kMla2KBoxBytes         (announced: 2 * kKG * 8192)
//   bar_v_full[g]         2 CTAs x kVG copies of kMla2VBoxBytes      (announced: 2 * kVG * kMla2VChunk);
//                         on a tile past the end of the sequence each CTA lands its own kVG copies on a barrier of its
//                         own (announced there: kVG * kMla2VChunk)
static_assert(kMla2QBoxBytes == kMla2QBytes, "Q: one copy per CTA fills the CTA's Q buffer");
static_assert(kMla2KBoxBytes == kKG * 8192, "K: a group's copy is what the producer announces per CTA");
static_assert(kMla2VBoxBytes == kMla2VChunk, "V: a chunk's copy is what the producer announces per chunk");
static_assert(kKG * kKGroups == kMlaSlabs && kVG * kVGroups == kMla2VChunks, "groups tile the K slabs / V chunks");
static_assert(2 * kMla2QBytes < (1 << 20) && 2 * kKG * 8192 < (1 << 20) && 2 * kVG * kMla2VChunk < (1 << 20),
              "a barrier's pending byte count must stay below 2^20");
// Arrivals per phase: bar_p_full = one per softmax warp of both CTAs (4 + 4); bar_xchg = every softmax thread of a CTA;
// bar_vfix = one per CTA; every other barrier has a single arrival (a producer's announce or a tcgen05.commit).
constexpr int kMla2SoftmaxWarps = 4;
constexpr int kMla2PFullArrivals = 2 * kMla2SoftmaxWarps, kMla2XchgArrivals = 32 * kMla2SoftmaxWarps;
// Which commit hands back what (all commits are multicast to both CTAs, issued by the leader's two MMA threads; a
// commit covers only the MMAs of the thread that issues it):
//   score thread, after K group g < last:  bar_k_empty[g]   -> K group g may be refilled
//   score thread, after the last K group:  bar_s_full[b]    -> scores of S[b] ready; last K group free; Q free after an item
//   P V thread,   after V group g < last:  bar_v_empty[g]   -> V group g may be refilled
//   P V thread,   after the last V group:  bar_pv_done      -> last V group free; P free; O quiescent / complete
// Tensor-memory columns of a CTA (512 allocated): S[0] 0..63, S[1] 64..127, O columns 128..255 and 256..383.
constexpr int kMla2TmemS = 0, kMla2TmemO0 = 128, kMla2TmemO1 = 256, kMla2TmemEnd = 384;
static_assert(kMla2TmemS + 2 * 64 <= kMla2TmemO0 && kMla2TmemO0 + 128 <= kMla2TmemO1 && kMla2TmemO1 + 128 <= kMla2TmemEnd &&
              kMla2TmemEnd <= 512, "tensor-memory regions do not overlap");
static_assert(kMla2SmemBytes <= 232448, "shared memory of one CTA");

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}
__device__ __forceinline__ void tmem_alloc2(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish2() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// D[tmem of both CTAs] (+)= A[smem of both] * B[smem of both]; issued by one thread of the even CTA
__device__ __forceinline__ void mma2_ss_lh(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc,
                                           uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 da, {%1, %3};\n\t"
        "mov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %4, p;\n\t}" ::"r"(d_tmem),
        "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate)
        : "memory");
}
// arrive on the barrier at the same shared-memory offset in every CTA of `mask` once all MMAs issued so far are done
__device__ __forceinline__ void tc_commit2(uint32_t bar, uint16_t mask) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
                 "h"(mask)
                 : "memory");
}
// Arrive on a barrier that lives in another CTA of the cluster.  Default semantics (release at CTA scope): the
// .release.cluster form measured ~1000 clk per arrive here.  What the arrive publishes is shared memory of the
// arriving CTA that each writer has already pushed to the async proxy with fence.proxy.async.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t local_bar, uint32_t target_rank) {
    asm volatile(
        "{\n\t.reg .b32 ra;\n\t"
        "mapa.shared::cluster.u32 ra, %0, %1;\n\t"
        "mbarrier.arrive.shared::cluster.b64 _, [ra];\n\t}" ::"r"(local_bar),
        "r"(target_rank)
        : "memory");
}
__device__ __forceinline__ uint32_t mapa_u32(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
// Tiled copies of a CTA pair: the data lands in the executing CTA's shared memory, the byte count is posted on a
// barrier that may live in the other CTA of the pair (bar_cluster is a shared::cluster address).  No multicast.
__device__ __forceinline__ void tma2_load_4d(uint32_t dst, const CUtensorMap* m, uint32_t bar_cluster, int c0, int c1,
                                             int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, "
        "%6}], [%2];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(m)), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
__device__ __forceinline__ void tma2_load_5d(uint32_t dst, const CUtensorMap* m, uint32_t bar_cluster, int c0, int c1,
                                             int c2, int c3, int c4) {
    asm volatile(
        "cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, "
        "%6, %7}], [%2];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(m)), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
        : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// bounded wait with cluster-scope acquire (the barrier may have been completed by the other CTA)
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag, int where) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    const long long t0 = clock64();
    int spins = 0;
    while (true) {
        if (mbar_try_wait_cluster(bar, parity)) return true;
        if ((++spins & 63) == 0) {
            if (*abort_flag != 0) return false;
            if (clock64() - t0 > kWaitLimitCycles) {
                atomicCAS(const_cast<int*>(abort_flag), 0, where);
                return false;
            }
        }
    }
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kMla2Threads, 1)
attn_mla2_kernel(const __grid_constant__ CUtensorMap tm_q1, const __grid_constant__ CUtensorMap tm_qh,
                 const __grid_constant__ CUtensorMap tm_k3, const __grid_constant__ CUtensorMap tm_k2,
                 const __grid_constant__ CUtensorMap tm_k1, const AttnParams p, const int kv_box_rows) {
    // tm_k1: (64 cols, keys, head, block) box (64, kv_box_rows, 1, 1) -- one page's share of one slab, for pages under 64 tokens
    //        (kv_box_rows < 64): a 64-key group then takes one copy per (slab, page), each issued by a lane of its own
    // tm_qh: (64 cols, Hq heads, 9 slabs, T rows) box (64, 64, 9, 1)      -- 64 q-heads of one token (packed items)
    // tm_q1: (64 cols, T rows, 9 slabs, Hq) box (64, 64, 9, 1)         -- 64 query rows, all nine 64-column slabs
    // tm_k3: (64 cols, keys, 9 slabs, head, block) box (64, 64, 3, 1, 1) -- 64 keys of three slabs: one K hand-back group
    // tm_k2: the same tensor, box (64, 64, 2, 1, 1)                      -- 64 keys of two slabs: one V chunk
    // One copy per group / chunk: a thread spends 100 clk and more on every copy it issues, and the data of a group
    // is wanted as soon as possible after its buffer is free (slab-by-slab copies: 1159 TFLOP/s on cfg 3 at 64K, this: 1234).
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gen_base = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t sQ = smem_base;
    const uint32_t sK = sQ + kMla2QBytes;
    const uint32_t sV = sK + kMla2KBytes;
    const uint32_t sP = sV + kMla2VBytes;
    const uint32_t sBar = sP + kMla2PBytes;
    // A tcgen05.commit costs the tensor pipe about as much as two small MMAs, so there are as few as possible: one
    // per K group, the last of which doubles as "scores ready", and one per V group, the last of which doubles as
    // "P consumed" and "O complete".  A barrier may have any number of waiters.
    const uint32_t bar_q_full = sBar + 0;
    const uint32_t bar_pv_done = sBar + 8;   // all P V MMAs of a tile done: last V group free, P free, O quiescent
    const uint32_t bar_s_full = sBar + 24;   // [2] scores of a tile done: also "last K group free" (and Q free after an item)
    const uint32_t bar_p_full = sBar + 40;   // [2] (used in the leader only: 4 local + 4 remote warp arrivals)
    const uint32_t bar_vfix = sBar + 72;     // leader: both V producers -> MMA thread (tiles past the end of a sequence)
    const uint32_t bar_xchg = sBar + 80;     // row statistics exchange between the two threads of a row
    // K and V are refilled piecewise: the copy of the next tile's group starts as soon as the MMAs that read this
    // tile's group have finished
    const uint32_t bar_k_full = sBar + 96;    // [kKGroups] leader: bytes of both CTAs
    const uint32_t bar_k_empty = sBar + 168;  // [kKGroups - 1]
    const uint32_t bar_v_full = sBar + 312;   // [kVGroups]
    const uint32_t bar_v_empty = sBar + 344;  // [kVGroups - 1]
    const uint32_t bar_v_local = sBar + 376;  // [kVGroups] rank 1: tiles past the end of the sequence land here
    uint8_t* gen_bar = gen_base + kMla2QBytes + kMla2KBytes + kMla2VBytes + kMla2PBytes;
    volatile int* s_abort = reinterpret_cast<volatile int*>(gen_bar + 416);
    volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(gen_bar + 420);
    float* xch = reinterpret_cast<float*>(gen_bar + 512);  // [2 phases][128 lanes]

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
        mbar_init(bar_p_full, kMla2PFullArrivals);
        mbar_init(bar_p_full + 8, kMla2PFullArrivals);
        mbar_init(bar_vfix, 2);     // one arrival per CTA
        mbar_init(bar_xchg, kMla2XchgArrivals);
        for (int i = 0; i < kKGroups; ++i) {
            mbar_init(bar_k_full + 8 * i, 1);
            mbar_init(bar_k_empty + 8 * i, 1);
        }
        for (int i = 0; i < kVGroups; ++i) {
            mbar_init(bar_v_full + 8 * i, 1);
            mbar_init(bar_v_empty + 8 * i, 1);
            mbar_init(bar_v_local + 8 * i, 1);
        }
        fence_mbar_init();
        *s_abort = 0;
        prefetch_tmap(&tm_q1);
        prefetch_tmap(&tm_qh);
        prefetch_tmap(&tm_k3);
        prefetch_tmap(&tm_k2);
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

    const int num_units = p.header_ro->num_units;
    const int num_pairs = gridDim.x >> 1;
    const int pair = blockIdx.x >> 1;
    // Items: (unit, q-head) for the units of several rows, then one item per single-token unit (the end of the list):
    // those run "packed" -- the q-heads are the rows of the tile (64 per CTA; they all share the one latent kv-head), so
    // the cache is streamed once per token instead of once per head.
    const int num_packed = p.num_q_heads <= 2 * kMla2Rows ? p.header_ro->num_single : 0;
    const int num_normal = num_units - num_packed;
    const int normal_items = num_normal * p.num_q_heads;
    const int total_items = normal_items + num_packed;

    // KV tiles (128 keys) of a unit: [kv_begin, min(kv_end, ceil((pos0 + rows) / 128)))
    auto tile_hi = [](const WorkUnit& u) {
        const int need = (u.pos0 + u.rows + kTileN - 1) / kTileN;
        return u.kv_end < need ? u.kv_end : need;
    };
    auto get_item = [&](int item, WorkUnit& u, int& h) -> bool {
        if (item < normal_items) {
            int ui;
            decode_item(item, num_normal, p.num_q_heads, p.num_q_heads, ui, h);
            u = p.units[ui];
        } else {
            u = p.units[num_normal + (item - normal_items)];
            h = 0;
        }
        return true;
    };
    auto is_packed = [&](const WorkUnit& u) { return num_packed > 0 && u.rows == 1; };
    // page and slot of the 64-key group that starts at position pos
    auto page_of = [&](const WorkUnit& u, int pos, int& blk, int& slot_in) {
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
    };

    // zero the value rows of keys at or beyond `first` (position within the tile) in V chunk c = (key half, instr)
    auto zero_v_rows = [&](int c, int first) {
        const int r0 = first - (c >> 1) * 64;
        const uint4 z = make_uint4(0, 0, 0, 0);
        for (int rr = (r0 > 0 ? r0 : 0) + lane; rr < 64; rr += 32) {
#pragma unroll
            for (int g = 0; g < 2; ++g) {
                uint4* a = reinterpret_cast<uint4*>(gen_base + kMla2QBytes + kMla2KBytes + c * kMla2VChunk + g * 8192 +
                                                    rr * 128);
#pragma unroll
                for (int q = 0; q < 8; ++q) a[q] = z;
            }
        }
    };

    // Copies of both CTAs post their bytes on the leader's "full" barriers (the MMA thread lives there); the leader's
    // producer announces the byte count of the pair.  Each CTA waits on its own "empty" barriers (multicast commits).
    const uint32_t pair_q_full = mapa_u32(bar_q_full, 0), pair_k_full = mapa_u32(bar_k_full, 0),
                   pair_v_full = mapa_u32(bar_v_full, 0);

    if (warp == 0) {
        // ===================================== Q / K producer =====================================
        // one thread: group g of the next tile is requested as soon as the MMAs that read group g of this tile are done
        if (kv_box_rows < 64) {
            // pages under 64 tokens: the waits and the Q copy by lane 0, the K copies of a group by 3 x (64 / page) lanes
            const int np = 64 / kv_box_rows, pq = lane % np;
            uint32_t q_it = 0, kc = 0;
            bool ok = true;
            for (int item = pair; item < total_items && ok; item += num_pairs) {
                WorkUnit u;
                int h;
                if (!get_item(item, u, h)) continue;
                if (lane == 0) {
                    if (kc > 0) ok = mbar_wait(bar_s_full + 8 * ((kc - 1) & 1), ((kc - 1) >> 1) & 1, s_abort, 801);
                    if (ok) {
                        if (leader) mbar_arrive_expect_tx(bar_q_full, 2 * kMla2QBytes);
                        if (is_packed(u))
                            tma2_load_4d(sQ, &tm_qh, pair_q_full, 0, static_cast<int>(rank) * kMla2Rows, 0, u.q_row0);
                        else
                            tma2_load_4d(sQ, &tm_q1, pair_q_full, 0, u.q_row0 + static_cast<int>(rank) * kMla2Rows, 0, h);
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                ++q_it;
                const int t_hi = tile_hi(u);
                for (int j = u.kv_begin; j < t_hi && ok; ++j) {
                    int blk, slot_in;                      // this lane's page of the CTA's 64 keys
                    page_of(u, j * kTileN + static_cast<int>(rank) * 64 + pq * kv_box_rows, blk, slot_in);
                    const uint32_t par = (kc & 1) ^ 1;
#pragma unroll 1
                    for (int g = 0; g < kKGroups; ++g) {
                        if (lane == 0) {
                            if (g < kKGroups - 1) ok = mbar_wait(bar_k_empty + 8 * g, par, s_abort, 802);
                            else if (kc > 0) ok = mbar_wait(bar_s_full + 8 * ((kc - 1) & 1), ((kc - 1) >> 1) & 1, s_abort, 802);
                            if (ok && leader) mbar_arrive_expect_tx(bar_k_full + 8 * g, 2 * kKG * 8192);
                        }
                        ok = __shfl_sync(0xffffffffu, ok, 0);
                        if (!ok) break;
                        if (lane < kKG * np) {
                            const int sl = g * kKG + lane / np;
                            tma2_load_4d(sK + sl * 8192 + pq * kv_box_rows * 128, &tm_k1, pair_k_full + 8 * g, 64 * sl, slot_in, 0, blk);
                        }
                        __syncwarp();
                    }
                    ++kc;
                }
            }
        } else if (lane == 0) {
            uint32_t q_it = 0, kc = 0, item_it = 0;
            bool ok = true;
            for (int item = pair; item < total_items && ok; item += num_pairs) {
                WorkUnit u;
                int h;
                if (!get_item(item, u, h)) continue;
                ++item_it;
                // Q may be replaced once the scores of the previous item's last tile are done
                if (kc > 0) ok = mbar_wait(bar_s_full + 8 * ((kc - 1) & 1), ((kc - 1) >> 1) & 1, s_abort, 801);
                if (!ok) break;
                if (leader) mbar_arrive_expect_tx(bar_q_full, 2 * kMla2QBytes);   // both CTAs' boxes, rows outside the tensor included
                // one copy of all nine slabs
                if (is_packed(u))   // heads 64 rank .. 64 rank + 63 of the token (heads that do not exist read as zero)
                    tma2_load_4d(sQ, &tm_qh, pair_q_full, 0, static_cast<int>(rank) * kMla2Rows, 0, u.q_row0);
                else
                    tma2_load_4d(sQ, &tm_q1, pair_q_full, 0, u.q_row0 + static_cast<int>(rank) * kMla2Rows, 0, h);
                ++q_it;
                const int t_hi = tile_hi(u);
                int blk_next = 0, slot_next = 0;
                page_of(u, u.kv_begin * kTileN + static_cast<int>(rank) * 64, blk_next, slot_next);
                for (int j = u.kv_begin; j < t_hi && ok; ++j) {
                    const int blk = blk_next, slot_in = slot_next;
                    if (j + 1 < t_hi) page_of(u, (j + 1) * kTileN + static_cast<int>(rank) * 64, blk_next, slot_next);
                    const uint32_t par = (kc & 1) ^ 1;
#pragma unroll 1
                    for (int g = 0; g < kKGroups; ++g) {
                        if (g < kKGroups - 1) ok = mbar_wait(bar_k_empty + 8 * g, par, s_abort, 802);
                        else if (kc > 0) ok = mbar_wait(bar_s_full + 8 * ((kc - 1) & 1), ((kc - 1) >> 1) & 1, s_abort, 802);
                        if (!ok) break;
                        if (leader) mbar_arrive_expect_tx(bar_k_full + 8 * g, 2 * kKG * 8192);
                        tma2_load_5d(sK + g * kKG * 8192, &tm_k3, pair_k_full + 8 * g, 0, slot_in, g * kKG, 0, blk);
                    }
                    ++kc;
                }
            }
        }
    } else if (warp == 6) {
        // ======================================= V producer =======================================
        // chunk c = (key half hf, instr i) holds value columns 256 i + 128 rank .. + 127 of keys 64 hf .. 64 hf + 63.
        // A tile that reaches past the end of the sequence is special: each CTA lands its part on a barrier of its
        // own, zeroes the value rows of the keys that do not exist (0 * garbage must not reach O) and then arrives
        // on bar_vfix, which the MMA thread waits on before it multiplies that tile.
        uint32_t vc = 0, tails = 0;
        bool ok = true;
        const uint32_t own_v_full = leader ? bar_v_full : bar_v_local;
        for (int item = pair; item < total_items && ok; item += num_pairs) {
            WorkUnit u;
            int h;
            if (!get_item(item, u, h)) continue;
            const int t_hi = tile_hi(u);
            int nb0 = 0, ns0 = 0, nb1 = 0, ns1 = 0;
            if (lane == 0) {
                page_of(u, u.kv_begin * kTileN, nb0, ns0);
                page_of(u, u.kv_begin * kTileN + 64, nb1, ns1);
            }
            for (int j = u.kv_begin; j < t_hi && ok; ++j) {
                const int tile0 = j * kTileN;
                const bool tail = tile0 + kTileN > u.kv_len;
                if (kv_box_rows < 64) {
                    // pages under 64 tokens: a group's two chunks take 2 chunks x 2 slabs x (64 / page) copies, a lane each
                    const int np = 64 / kv_box_rows, pq = lane % np;
                    const uint32_t par = (vc & 1) ^ 1;
#pragma unroll 1
                    for (int g = 0; g < kVGroups; ++g) {
                        if (lane == 0) {
                            if (g < kVGroups - 1) ok = mbar_wait(bar_v_empty + 8 * g, par, s_abort, 803);
                            else if (vc > 0) ok = mbar_wait(bar_pv_done, (vc - 1) & 1, s_abort, 803);
                            if (ok) {
                                if (tail) mbar_arrive_expect_tx(own_v_full + 8 * g, kVG * kMla2VChunk);
                                else if (leader) mbar_arrive_expect_tx(bar_v_full + 8 * g, 2 * kVG * kMla2VChunk);
                            }
                        }
                        ok = __shfl_sync(0xffffffffu, ok, 0);
                        if (!ok) break;
                        if (lane < kVG * 2 * np) {
                            const int c = g * kVG + lane / (2 * np), s2 = (lane / np) & 1;
                            const int hf = c >> 1, slab = 4 * (c & 1) + 2 * static_cast<int>(rank) + s2;
                            int blk, slot_in;
                            page_of(u, tile0 + 64 * hf + pq * kv_box_rows, blk, slot_in);
                            const uint32_t dst = sV + c * kMla2VChunk + s2 * 8192 + pq * kv_box_rows * 128;
                            if (tail) tma_load_4d(dst, &tm_k1, own_v_full + 8 * g, 64 * slab, slot_in, 0, blk);
                            else tma2_load_4d(dst, &tm_k1, pair_v_full + 8 * g, 64 * slab, slot_in, 0, blk);
                        }
                        __syncwarp();
                    }
                } else if (lane == 0) {
                    const int b0 = nb0, s0 = ns0, b1 = nb1, s1 = ns1;
                    if (j + 1 < t_hi) {
                        page_of(u, tile0 + kTileN, nb0, ns0);
                        page_of(u, tile0 + kTileN + 64, nb1, ns1);
                    }
                    const uint32_t par = (vc & 1) ^ 1;
#pragma unroll 1
                    for (int c = 0; c < kMla2VChunks; ++c) {
                        const int g = c / kVG;
                        if (c % kVG == 0) {
                            if (g < kVGroups - 1) ok = mbar_wait(bar_v_empty + 8 * g, par, s_abort, 803);
                            else if (vc > 0) ok = mbar_wait(bar_pv_done, (vc - 1) & 1, s_abort, 803);
                            if (!ok) break;
                            if (tail) mbar_arrive_expect_tx(own_v_full + 8 * g, kVG * kMla2VChunk);
                            else if (leader) mbar_arrive_expect_tx(bar_v_full + 8 * g, 2 * kVG * kMla2VChunk);
                        }
                        const int hf = c >> 1, slab0 = 4 * (c & 1) + 2 * static_cast<int>(rank);
                        const uint32_t dst = sV + c * kMla2VChunk;
                        if (tail) tma_load_5d(dst, &tm_k2, own_v_full + 8 * g, 0, hf ? s1 : s0, slab0, 0, hf ? b1 : b0);
                        else tma2_load_5d(dst, &tm_k2, pair_v_full + 8 * g, 0, hf ? s1 : s0, slab0, 0, hf ? b1 : b0);
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                if (tail) {
                    if (lane == 0) {
                        for (int g = 0; g < kMla2VChunks / kVG && ok; ++g)
                            ok = mbar_wait(own_v_full + 8 * g, leader ? (vc & 1) : (tails & 1), s_abort, 804);
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) break;
                    const int first = u.kv_len > tile0 ? u.kv_len - tile0 : 0;
                    for (int c = 0; c < kMla2VChunks; ++c)
                        if (first < (c >> 1) * 64 + 64) zero_v_rows(c, first);
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        if (leader) mbar_arrive(bar_vfix);
                        else mbar_arrive_remote(bar_vfix, 0);
                    }
                    ++tails;
                }
                ++vc;
            }
        }
    } else if (warp == 1 && leader && lane == 0) {
        // ============ score MMA issuer: one thread for both CTAs of the pair (S = Q K^T) ============
        // Two issuing threads, this one and the P V issuer in warp 7: a single thread has nothing to hide the latency of
        // its own barrier tests, commits and MMA issue behind, and the tensor pipe idled between its groups.
        constexpr uint32_t kIdescQK = idesc_bf16(128, 128, false, false);
        constexpr uint32_t kHi = desc_hi_sw128(1024);
        const uint32_t q_lo = desc_lo_sw128(sQ, 16), k_lo = desc_lo_sw128(sK, 16);
        uint32_t q_it = 0, kc = 0, item_it = 0;   // kc: score tiles issued so far (all items)
        bool ok = true;
        // Scores of K group g (kKG slabs), unrolled completely with compile-time offsets: every descriptor is a
        // loop-invariant base plus a constant.  The group goes back to the producer when its MMAs are done; the last
        // group's commit also tells the softmax warps that the scores are complete.
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
        for (int item = pair; item < total_items && ok; item += num_pairs) {
            WorkUnit u;
            int h;
            if (!get_item(item, u, h)) continue;
            const int n = tile_hi(u) - u.kv_begin;
            ++item_it;
            ok = mbar_wait(bar_q_full, q_it & 1, s_abort, 821);
            ++q_it;
            for (int jj = 0; jj < n && ok; ++jj) {
                const uint32_t b = kc & 1, kpar = kc & 1;
                const uint32_t tS = tmem_base + b * 64, bar_s = bar_s_full + 8 * b;
                // S[b] was last read by the softmax of two tiles ago: its P is ready <=> that read is over
                if (kc >= 2) ok = mbar_wait_cluster(bar_p_full + 8 * b, ((kc - 2) >> 1) & 1, s_abort, 820);
                if (!ok) break;
                ok = mbar_wait(bar_k_full, kpar, s_abort, 822);
                if (!ok) break;
                tc_fence_after();
                qk_group_c(std::integral_constant<int, 0>{}, tS, bar_s);
                ok = mbar_wait(bar_k_full + 8, kpar, s_abort, 822);
                if (!ok) break;
                tc_fence_after();
                qk_group_c(std::integral_constant<int, 1>{}, tS, bar_s);
                ok = mbar_wait(bar_k_full + 16, kpar, s_abort, 822);
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
        const uint32_t tO0 = tmem_base + kMla2TmemO0, tO1 = tmem_base + kMla2TmemO1;
        uint32_t vc = 0, vfix_it = 0, item_it = 0;   // vc: P V tiles issued so far (all items)
        bool ok = true;
        // O += P V for V group g: chunk c = (key half c >> 1, output half c & 1)
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
        for (int item = pair; item < total_items && ok; item += num_pairs) {
            WorkUnit u;
            int h;
            if (!get_item(item, u, h)) continue;
            const int n = tile_hi(u) - u.kv_begin;
            ++item_it;
            for (int jj = 0; jj < n && ok; ++jj) {
                const int tile0 = (u.kv_begin + jj) * kTileN;
                const uint32_t b = vc & 1, vpar = vc & 1;
                ok = mbar_wait_cluster(bar_p_full + 8 * b, (vc >> 1) & 1, s_abort, 826);
                if (ok && tile0 + kTileN > u.kv_len) {
                    ok = mbar_wait_cluster(bar_vfix, vfix_it & 1, s_abort, 825);
                    ++vfix_it;
                }
                if (!ok) break;
                ok = mbar_wait(bar_v_full, vpar, s_abort, 824);
                if (!ok) break;
                tc_fence_after();
                if (jj == 0) pv_group_c(std::integral_constant<int, 0>{}, std::true_type{});
                else pv_group_c(std::integral_constant<int, 0>{}, std::false_type{});
                ok = mbar_wait(bar_v_full + 8, vpar, s_abort, 824);
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
        const int row = l128 & 63;                     // row of this CTA's 64
        const int half = l128 >> 6;                    // which 64 key columns of the tile
        const uint32_t lane_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tO0 = tmem_base + kMla2TmemO0 + lane_off, tO1 = tmem_base + kMla2TmemO1 + lane_off;
        uint8_t* p_row = gen_base + kMla2QBytes + kMla2KBytes + kMla2VBytes + half * 8192 + row * 128;
        uint32_t tc = 0, x_it = 0, item_it = 0;
        const float sc = p.scale_log2e;
        auto exchange = [&](float mine, float& theirs) -> bool {
            float* buf = xch + (x_it & 1) * 128;
            buf[l128] = mine;
            mbar_arrive(bar_xchg);
            if (!mbar_wait(bar_xchg, x_it & 1, s_abort, 831)) return false;
            theirs = buf[l128 ^ 64];
            ++x_it;
            return true;
        };
        bool ok = true;
        for (int item = pair; item < total_items && ok; item += num_pairs) {
            WorkUnit u;
            int h;
            if (!get_item(item, u, h)) continue;
            const int t_hi = tile_hi(u);
            ++item_it;
            const int my_row = static_cast<int>(rank) * kMla2Rows + row;  // row of the 128-row tile
            const bool packed = is_packed(u);
            const int my_pos = packed ? u.pos0 : u.pos0 + my_row;
            if (packed) h = my_row;                                       // row r of a packed tile is q-head r
            float m_ref = -INFINITY, l_run = 0.f;
            for (int j = u.kv_begin; j < t_hi; ++j) {
                const int tile0 = j * kTileN;
                const uint32_t b = tc & 1;
                const uint32_t tS = tmem_base + b * 64 + lane_off;
                ok = mbar_wait(bar_s_full + 8 * b, (tc >> 1) & 1, s_abort, 832);
                if (!ok) break;
                tc_fence_after();
                uint32_t s[64];
                tmem_ld32(tS, reinterpret_cast<uint32_t(&)[32]>(s[0]));
                tmem_ld32(tS + 32, reinterpret_cast<uint32_t(&)[32]>(s[32]));
                tc_wait_ld();
                if (tile0 + kTileN - 1 > u.pos0) {  // diagonal tile
                    const int lim = my_pos - tile0 - half * 64;
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
                    if (j > u.kv_begin) {
                        // O is rescaled in place: P V of the previous tile (issued after this tile's scores) must be done
                        ok = mbar_wait(bar_pv_done, (tc - 1) & 1, s_abort, 835);
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
                    ok = mbar_wait(bar_pv_done, (tc - 1) & 1, s_abort, 833);
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
            ok = mbar_wait(bar_pv_done, (tc - 1) & 1, s_abort, 834);  // P V of the item's last tile
            if (!ok) break;
            tc_fence_after();
            const float inv_l = 1.f / l_tot;
            const bool live = packed ? my_row < p.num_q_heads : my_row < u.rows;
            const long long grow_idx = static_cast<long long>(u.q_row0) + (packed ? 0 : my_row);
            uint32_t r[32];
#pragma unroll 1
            for (int c = 0; c < 8; ++c) {
                tmem_ld32((c < 4 ? tO0 : tO1) + (c & 3) * 32, r);
                tc_wait_ld();
                if (!live) continue;
                const int col0 = (c >> 2) * 256 + half * 128 + (c & 3) * 32;
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
                        p.o_parts + ((static_cast<long long>(u.split) * p.total_q + grow_idx) * p.num_q_heads + h) * kMlaDv +
                        col0);
#pragma unroll
                    for (int q4 = 0; q4 < 8; ++q4)
                        dst[q4] = make_float4(__uint_as_float(r[q4 * 4]) * inv_l, __uint_as_float(r[q4 * 4 + 1]) * inv_l,
                                              __uint_as_float(r[q4 * 4 + 2]) * inv_l, __uint_as_float(r[q4 * 4 + 3]) * inv_l);
                }
            }
            if (live && half == 0) {
                const float lse = (m_ref + log2f(l_tot)) * 0.6931471805599453f;
                if (u.split < 0) {
                    if (p.lse) p.lse[grow_idx * p.num_q_heads + h] = lse;
                } else {
                    p.lse_parts[(static_cast<long long>(u.split) * p.total_q + grow_idx) * p.num_q_heads + h] = lse;
                }
            }
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
