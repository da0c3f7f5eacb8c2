// Structures shared by the host entry points and the kernels.
#pragma once
#include <cstdint>
#include <cuda.h>

namespace vpp {

constexpr int kTileM = 128;  // query rows per MMA tile
constexpr int kTileN = 128;  // keys per KV tile

// One schedulable unit: a 128-row query tile of one request restricted to a range of KV tiles.
// The attention kernel turns (unit, head slot) pairs into work items.
struct __align__(16) WorkUnit {
    int32_t req;        // request index
    int32_t q_row0;     // first packed query row of the tile
    int32_t rows;       // valid rows in the unit (1..128; up to 256 when an item is two tiles of one q-head)
    int32_t pos0;       // absolute position of the tile's first row (prefix_len + row offset)
    int32_t kv_begin;   // first KV tile (units of kTileN keys)
    int32_t kv_end;     // one past the last KV tile
    int32_t split;      // split index of this unit, or -1 when the tile is not split (final output)
    int32_t kv_len;     // prefix_len + chunk_len of the request: keys at or beyond it do not exist
};

// Head of the workspace; written by the work-decomposition kernel.
struct WorkHeader {
    int32_t num_units;  // units in the sorted list
    int32_t counter;    // persistent-kernel work counter
    int32_t error;      // VPP_DEV_* (0 = ok); when nonzero num_units is 0
    int32_t num_single; // the last num_single units of the list are single-token units (rows == 1)
};

struct WorkspaceLayout {
    size_t header;      // WorkHeader
    size_t units;       // WorkUnit[max_units]
    size_t row_splits;  // int32[total_q]: number of partials to merge for each query row (0/1: none)
    size_t o_parts;     // float[S][total_q][Hq][Dv]
    size_t lse_parts;   // float[S][total_q][Hq]
    size_t total;
    int32_t max_units;
    int32_t splits;     // S, the uniform upper bound on splits per tile
};

struct AttnParams {
    const int32_t* block_table;   // may be null (contiguous)
    int32_t max_blocks_per_req;
    int32_t block_shift;          // log2(block_size) (paged only)
    int32_t num_blocks;
    int32_t num_q_heads;
    int32_t num_kv_heads;
    int32_t total_q;
    float scale_log2e;            // softmax_scale * log2(e)
    void* out;                    // bf16 [T, Hq, Dv]
    float* lse;                   // [T, Hq] or null
    float* o_parts;               // [S, T, Hq, Dv]
    float* lse_parts;             // [S, T, Hq]
    const WorkHeader* header_ro;
    WorkHeader* header;
    const WorkUnit* units;
    int32_t* status;              // may be null
};

constexpr int kSlabBytes = kTileM * 128;  // 128 rows x 64 bf16, 128B-swizzled

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

}  // namespace vpp
