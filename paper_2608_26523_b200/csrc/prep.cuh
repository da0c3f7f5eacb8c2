// Work decomposition: from the per-request (prefix_len, chunk_len) on the device, build the list of
// work units (query tile of 128 -- or 256 -- rows x key-range split) ordered by decreasing cost, so that the
// persistent attention kernel can hand out tiles of very unequal cost longest-first.
//
// A query tile whose first row sits at absolute position pos0 needs the KV tiles
// [0, ceil((pos0 + rows) / 128)); its cost is that count -- it grows linearly with the prefix,
// which is the per-chunk imbalance the paper's Eq. 2 models.
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace vpp {

constexpr int kPrepThreads = 1024;
constexpr int kCostBins = 2048;

struct PrepParams {
    const int32_t* prefix_len;
    const int32_t* chunk_len;
    const int32_t* block_table;  // may be null
    int32_t num_reqs;
    int32_t total_q;
    int32_t max_seq_len;
    int32_t max_blocks_per_req;
    int32_t block_shift;
    int32_t num_blocks;
    int32_t splits;      // S >= 1
    int32_t max_units;
    int32_t max_cost;    // ceil(max_seq_len / 128), >= 1
    int32_t tile_m;      // query rows per unit: 128, or 256 when a work item is two 128-row tiles of one q-head
    int32_t partial;     // 1: key-range restricted launch whose results are partial (o fp32, lse) of "split 0"
    int32_t range_begin; // first KV tile of the key range (partial launches)
    int32_t range_end;   // one past its last KV tile
    WorkHeader* header;
    WorkUnit* units;
    int32_t* row_splits;  // [total_q], only written when splits > 1
    int32_t* q_start;     // [num_reqs + 1] scratch
    int32_t* tile_start;  // [num_reqs + 1] scratch
    int32_t* status;      // may be null
};

// Exclusive scan of one value per thread over the block; returns the block total through `total`.
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_sums, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = warp_sums[lane];
        int wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int t = __shfl_up_sync(0xffffffffu, wi, o);
            if (lane >= o) wi += t;
        }
        warp_sums[lane] = wi - w;          // exclusive warp offsets
        if (lane == 31) warp_sums[32] = wi;  // block total
    }
    __syncthreads();
    const int res = warp_sums[warp] + incl - v;
    total = warp_sums[32];
    __syncthreads();
    return res;
}

// Number of key-range splits of the query tile whose first row is at absolute position pos0:
// every split must start at or before pos0 so that each row sees at least one key in each split.
__device__ __forceinline__ int tile_num_splits(int pos0, int S) {
    const int splittable = pos0 / kTileN + 1;  // KV tiles that start at or before pos0
    return S < splittable ? S : splittable;
}

__device__ __forceinline__ void split_range(int pos0, int n_tiles, int nsplit, int s, int& kb, int& ke) {
    const int splittable = pos0 / kTileN + 1;
    kb = static_cast<int>((static_cast<long long>(s) * splittable) / nsplit);
    ke = (s + 1 == nsplit) ? n_tiles : static_cast<int>((static_cast<long long>(s + 1) * splittable) / nsplit);
}

__device__ __forceinline__ int cost_bin(int cost, int max_cost) {
    long long b = (static_cast<long long>(cost) * (kCostBins - 1)) / max_cost;
    if (b > kCostBins - 1) b = kCostBins - 1;
    if (b < 0) b = 0;
    return kCostBins - 1 - static_cast<int>(b);  // bin 0 = most expensive
}

__global__ void __launch_bounds__(kPrepThreads, 1) prep_kernel(const PrepParams p) {
    __shared__ int warp_sums[33];
    __shared__ int bins[2 * kCostBins];   // [0, kCostBins): units of several rows; [kCostBins, ..): single-token units
    __shared__ int s_error;
    __shared__ int s_carry_q, s_carry_t;
    const int tid = threadIdx.x;
    pdl_launch_dependents();   // the attention kernel may set itself up (barriers, tensor memory) while this runs
    if (tid == 0) {
        s_error = 0;
        s_carry_q = 0;
        s_carry_t = 0;
    }
    for (int b = tid; b < 2 * kCostBins; b += kPrepThreads) bins[b] = 0;
    __syncthreads();

    // ---- phase 1: validate lengths, scan chunk lengths and query-tile counts over requests ----
    for (int base = 0; base < p.num_reqs; base += kPrepThreads) {
        const int r = base + tid;
        int c = 0, nt = 0;
        if (r < p.num_reqs) {
            const int P = p.prefix_len[r];
            c = p.chunk_len[r];
            // (a key range must start inside every request's prefix, so that each query row sees at least one of its keys)
            if (P < 0 || c < 0 || static_cast<long long>(P) + c > p.max_seq_len ||
                (p.partial && c > 0 && P < p.range_begin * kTileN)) {
                atomicExch(&s_error, 1 /* VPP_DEV_BAD_LENGTHS */);
                c = 0;
            }
            nt = (c + p.tile_m - 1) / p.tile_m;
        }
        int tot_q, tot_t;
        const int eq = block_exclusive_scan(c, warp_sums, tot_q);
        const int et = block_exclusive_scan(nt, warp_sums, tot_t);
        if (r < p.num_reqs) {
            p.q_start[r] = s_carry_q + eq;
            p.tile_start[r] = s_carry_t + et;
        }
        __syncthreads();
        if (tid == 0) {
            s_carry_q += tot_q;
            s_carry_t += tot_t;
        }
        __syncthreads();
    }
    const int total_tiles = s_carry_t;
    if (tid == 0) {
        p.q_start[p.num_reqs] = s_carry_q;
        p.tile_start[p.num_reqs] = s_carry_t;
        if (s_carry_q != p.total_q) s_error = 1;
    }
    __syncthreads();

    // ---- phase 1b: every block-table entry a request needs must name a real block ----
    if (s_error == 0 && p.block_table != nullptr) {
        for (int r = 0; r < p.num_reqs; ++r) {
            const int kv_len = p.prefix_len[r] + p.chunk_len[r];
            if (p.chunk_len[r] == 0) continue;
            const int nb = (kv_len + (1 << p.block_shift) - 1) >> p.block_shift;
            if (nb > p.max_blocks_per_req) {
                if (tid == 0) s_error = 2;
                continue;
            }
            for (int b = tid; b < nb; b += kPrepThreads) {
                const int e = p.block_table[static_cast<long long>(r) * p.max_blocks_per_req + b];
                if (e < 0 || e >= p.num_blocks) atomicExch(&s_error, 2 /* VPP_DEV_BAD_BLOCK */);
            }
        }
    }
    __syncthreads();
    if (s_error != 0) {
        if (tid == 0) {
            p.header->num_units = 0;
            p.header->num_single = 0;
            p.header->counter = 0;
            p.header->error = s_error;
            if (p.status) *p.status = s_error;
        }
        return;
    }

    // ---- phases 2-4: counting sort of the units by decreasing cost ----
    for (int pass = 0; pass < 2; ++pass) {
        for (int gt = tid; gt < total_tiles; gt += kPrepThreads) {
            // request of global query tile gt: last r with tile_start[r] <= gt
            int lo = 0, hi = p.num_reqs - 1;
            while (lo < hi) {
                const int mid = (lo + hi + 1) >> 1;
                if (p.tile_start[mid] <= gt) lo = mid; else hi = mid - 1;
            }
            const int r = lo;
            const int qt = gt - p.tile_start[r];
            const int P = p.prefix_len[r], C = p.chunk_len[r];
            const int row_off = qt * p.tile_m;
            const int rows = (C - row_off) < p.tile_m ? (C - row_off) : p.tile_m;
            const int pos0 = P + row_off;
            const int n_tiles = (pos0 + rows + kTileN - 1) / kTileN;
            const int nsplit = p.partial ? 1 : tile_num_splits(pos0, p.splits);
            for (int s = 0; s < nsplit; ++s) {
                int kb, ke;
                if (p.partial) {
                    kb = p.range_begin;
                    ke = n_tiles < p.range_end ? n_tiles : p.range_end;
                } else {
                    split_range(pos0, n_tiles, nsplit, s, kb, ke);
                }
                // single-token units go to the end of the list (each part ordered by decreasing cost): the attention
                // kernels may run them with the q-heads of a kv-head packed into one tile
                const int bin = cost_bin(ke - kb, p.max_cost) + (rows == 1 ? kCostBins : 0);
                if (pass == 0) {
                    atomicAdd(&bins[bin], 1);
                } else {
                    const int slot = atomicAdd(&bins[bin], 1);
                    if (slot < p.max_units) {
                        WorkUnit u;
                        u.req = r;
                        u.q_row0 = p.q_start[r] + row_off;
                        u.rows = rows;
                        u.pos0 = pos0;
                        u.kv_begin = kb;
                        u.kv_end = ke;
                        u.split = (nsplit > 1 || p.partial) ? s : -1;
                        u.kv_len = P + C;
                        p.units[slot] = u;
                    }
                }
            }
            if (pass == 1 && p.splits > 1) {
                for (int i = 0; i < rows; ++i) p.row_splits[p.q_start[r] + row_off + i] = nsplit;
            }
        }
        __syncthreads();
        if (pass == 0) {
            // exclusive scan of the bins (bin 0 = most expensive first)
            static_assert(2 * kCostBins == 4 * kPrepThreads, "four bins per thread");
            const int b0 = bins[4 * tid], b1 = bins[4 * tid + 1], b2 = bins[4 * tid + 2], b3 = bins[4 * tid + 3];
            int total;
            const int ex = block_exclusive_scan(b0 + b1 + b2 + b3, warp_sums, total);
            bins[4 * tid] = ex;
            bins[4 * tid + 1] = ex + b0;
            bins[4 * tid + 2] = ex + b0 + b1;
            bins[4 * tid + 3] = ex + b0 + b1 + b2;
            __syncthreads();
            if (tid == 0) {
                const int n = total < p.max_units ? total : p.max_units;
                const int first_single = bins[kCostBins] < n ? bins[kCostBins] : n;
                p.header->num_units = n;
                p.header->num_single = n - first_single;
                p.header->counter = 0;
                p.header->error = 0;
                if (p.status) *p.status = 0;
            }
            __syncthreads();
        }
    }
}

// The same decomposition for small launches (at most 32 requests and 32 query tiles: a short chunk, a small decode
// batch), by ONE warp: a lane per request, then a lane per query tile, scans by shuffles, no block-wide
// synchronisation, no sort -- the units of such a launch all start in the first wave of work items, so their order
// does not matter (units of several rows first, single-token units last, as the attention kernels expect).  About a
// third of the big kernel's latency, which is most of what a launch of a few work items costs.
constexpr int kPrepSmallMax = 32;

__global__ void __launch_bounds__(32, 1) prep_small_kernel(const PrepParams p) {
    __shared__ int s_P[kPrepSmallMax], s_C[kPrepSmallMax], s_q0[kPrepSmallMax + 1], s_t0[kPrepSmallMax + 1];
    const int lane = threadIdx.x;
    pdl_launch_dependents();
    // ---- requests: validate, scan chunk lengths and tile counts ----
    int P = 0, c = 0, nt = 0, bad = 0;
    if (lane < p.num_reqs) {
        P = p.prefix_len[lane];
        c = p.chunk_len[lane];
        if (P < 0 || c < 0 || static_cast<long long>(P) + c > p.max_seq_len ||
            (p.partial && c > 0 && P < p.range_begin * kTileN)) {
            bad = 1;
            c = 0;
        }
        nt = (c + p.tile_m - 1) / p.tile_m;
    }
    int iq = c, it = nt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int a = __shfl_up_sync(0xffffffffu, iq, o), b = __shfl_up_sync(0xffffffffu, it, o);
        if (lane >= o) {
            iq += a;
            it += b;
        }
    }
    const int total_q = __shfl_sync(0xffffffffu, iq, 31), total_tiles = __shfl_sync(0xffffffffu, it, 31);
    if (lane < p.num_reqs) {
        s_P[lane] = P;
        s_C[lane] = c;
        s_q0[lane] = iq - c;
        s_t0[lane] = it - nt;
        p.q_start[lane] = iq - c;
        p.tile_start[lane] = it - nt;
    }
    if (lane == 0) {
        s_t0[p.num_reqs] = total_tiles;
        p.q_start[p.num_reqs] = total_q;
        p.tile_start[p.num_reqs] = total_tiles;
    }
    int error = __any_sync(0xffffffffu, bad) || total_q != p.total_q || total_tiles > kPrepSmallMax ? 1 : 0;
    __syncwarp();
    // ---- every block-table entry a request needs must name a real block ----
    if (error == 0 && p.block_table != nullptr) {
        int bad_blk = 0;
        for (int r = 0; r < p.num_reqs; ++r) {
            if (s_C[r] == 0) continue;
            const int nb = (s_P[r] + s_C[r] + (1 << p.block_shift) - 1) >> p.block_shift;
            if (nb > p.max_blocks_per_req) {
                bad_blk = 1;
                continue;
            }
            for (int b = lane; b < nb; b += 32) {
                const int e = p.block_table[static_cast<long long>(r) * p.max_blocks_per_req + b];
                if (e < 0 || e >= p.num_blocks) bad_blk = 1;
            }
        }
        if (__any_sync(0xffffffffu, bad_blk)) error = 2;
    }
    if (error != 0) {
        if (lane == 0) {
            p.header->num_units = 0;
            p.header->num_single = 0;
            p.header->counter = 0;
            p.header->error = error;
            if (p.status) *p.status = error;
        }
        return;
    }
    // ---- a lane per query tile: its units, placed by two scans (units of several rows, then single-token units) ----
    int r = 0, rows = 0, pos0 = 0, n_tiles = 0, nsplit = 0, row_off = 0;
    if (lane < total_tiles) {
        while (s_t0[r + 1] <= lane) ++r;
        row_off = (lane - s_t0[r]) * p.tile_m;
        rows = s_C[r] - row_off < p.tile_m ? s_C[r] - row_off : p.tile_m;
        pos0 = s_P[r] + row_off;
        n_tiles = (pos0 + rows + kTileN - 1) / kTileN;
        nsplit = p.partial ? 1 : tile_num_splits(pos0, p.splits);
    }
    const bool single = rows == 1;
    int in = single ? 0 : nsplit, is = single ? nsplit : 0;
    const int mine_n = in, mine_s = is;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int a = __shfl_up_sync(0xffffffffu, in, o), b = __shfl_up_sync(0xffffffffu, is, o);
        if (lane >= o) {
            in += a;
            is += b;
        }
    }
    const int total_n = __shfl_sync(0xffffffffu, in, 31), total_s = __shfl_sync(0xffffffffu, is, 31);
    const int first = single ? total_n + is - mine_s : in - mine_n;
    for (int s = 0; s < nsplit; ++s) {
        int kb, ke;
        if (p.partial) {
            kb = p.range_begin;
            ke = n_tiles < p.range_end ? n_tiles : p.range_end;
        } else {
            split_range(pos0, n_tiles, nsplit, s, kb, ke);
        }
        if (first + s < p.max_units) {
            WorkUnit u;
            u.req = r;
            u.q_row0 = s_q0[r] + row_off;
            u.rows = rows;
            u.pos0 = pos0;
            u.kv_begin = kb;
            u.kv_end = ke;
            u.split = (nsplit > 1 || p.partial) ? s : -1;
            u.kv_len = s_P[r] + s_C[r];
            p.units[first + s] = u;
        }
    }
    if (p.splits > 1) {
        // per-row split counts, written by the whole warp tile by tile
        for (int t = 0; t < total_tiles; ++t) {
            const int t_rows = __shfl_sync(0xffffffffu, rows, t), t_ns = __shfl_sync(0xffffffffu, nsplit, t);
            const int t_q0 = __shfl_sync(0xffffffffu, lane < total_tiles ? s_q0[r] + row_off : 0, t);
            for (int i = lane; i < t_rows; i += 32) p.row_splits[t_q0 + i] = t_ns;
        }
    }
    if (lane == 0) {
        const int n = total_n + total_s < p.max_units ? total_n + total_s : p.max_units;
        const int first_single = total_n < n ? total_n : n;
        p.header->num_units = n;
        p.header->num_single = n - first_single;
        p.header->counter = 0;
        p.header->error = 0;
        if (p.status) *p.status = 0;
    }
}

}  // namespace vpp
