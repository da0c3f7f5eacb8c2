// Host side of the C ABI declared in include/vpp.h: argument validation, workspace layout,
// tensor-map construction and kernel launches.  Nothing here synchronises or allocates device memory.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>

#include "../../include/vpp.h"
#include "attn_mla2.cuh"
#include "attn_dsa.cuh"
#include "attn_ws.cuh"
#include "common.cuh"
#include "kv_append.cuh"
#include "merge.cuh"
#include "prep.cuh"
#include "wait_test.cuh"

namespace {

thread_local char g_err[512] = "";
thread_local int32_t g_launches = 0;

vpp_status fail(vpp_status s, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
    return s;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---- device facts, cached per device -------------------------------------------------------------
struct DeviceInfo {
    bool ready = false;
    int sm_count = 0;
    bool attrs_set = false;
};
std::mutex g_mu;
DeviceInfo g_dev[64];

int sm_count_or_default() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        cudaGetLastError();
        return 148;
    }
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g_dev[dev].ready) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
            cudaGetLastError();
            n = 148;
        }
        g_dev[dev].sm_count = n;
        g_dev[dev].ready = true;
    }
    return g_dev[dev].sm_count;
}

// ---- tensor maps ------------------------------------------------------------------------------------
using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                              const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                              CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn get_encode() {
    static EncodeFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeFn>(p);
        else
            cudaGetLastError();
    });
    return fn;
}

// Encoded tensor maps are cached: a serving loop calls with the same buffers and shapes again and again, and seven
// to nine driver encodes per call are a visible part of a short launch.  A map depends only on (base address, rank,
// extents, strides, box), so an entry never goes stale; the cache is a small 4-way set-associative table (least recently
// used way replaced) guarded by a mutex.
struct TmapKey {
    const void* base;
    uint64_t dims[5];
    uint64_t strides[4];
    uint32_t box[5];
    uint32_t rank;
};
using RawEncodeFn = bool (*)(CUtensorMap*, const TmapKey&);

class TmapCache {
public:
    static constexpr int kSets = 64, kWays = 4;   // a call uses up to nine maps; 256 entries serve a few dozen distinct launches
    bool get(const TmapKey& key, RawEncodeFn encode, CUtensorMap* out) {
        const uint64_t h = hash(key);
        Slot* set = slots_ + (h % kSets) * kWays;
        std::lock_guard<std::mutex> lk(mu_);
        ++lookups_;
        ++clock_;
        Slot* victim = set;
        for (int w = 0; w < kWays; ++w) {
            Slot& sl = set[w];
            if (sl.valid && sl.hash == h && std::memcmp(&sl.key, &key, sizeof key) == 0) {
                sl.stamp = clock_;
                *out = sl.map;
                return true;
            }
            // the way to replace on a miss: an empty one if there is any, else the least recently used
            if (victim->valid && (!sl.valid || sl.stamp < victim->stamp)) victim = &sl;
        }
        CUtensorMap m;
        if (!encode(&m, key)) return false;
        ++encodes_;
        victim->key = key;
        victim->hash = h;
        victim->map = m;
        victim->valid = true;
        victim->stamp = clock_;
        *out = m;
        return true;
    }
    void stats(int64_t* lookups, int64_t* encodes) {
        std::lock_guard<std::mutex> lk(mu_);
        *lookups = lookups_;
        *encodes = encodes_;
    }
private:
    struct Slot {
        TmapKey key;
        uint64_t hash = 0, stamp = 0;
        CUtensorMap map;
        bool valid = false;
    };
    static uint64_t hash(const TmapKey& k) {   // FNV-1a over the key's bytes (the key is zero-initialised, padding included)
        const unsigned char* b = reinterpret_cast<const unsigned char*>(&k);
        uint64_t h = 1469598103934665603ull;
        for (size_t i = 0; i < sizeof k; ++i) h = (h ^ b[i]) * 1099511628211ull;
        return h;
    }
    std::mutex mu_;
    Slot slots_[kSets * kWays];
    int64_t lookups_ = 0, encodes_ = 0;
    uint64_t clock_ = 0;
};
TmapCache g_tmaps;

// bf16 tensor, innermost dimension contiguous, 128-byte swizzle, zero fill out of bounds.
bool encode_with_driver(CUtensorMap* m, const TmapKey& k) {
    EncodeFn enc = get_encode();
    if (!enc) return false;
    cuuint64_t gd[5], gs[4];
    cuuint32_t bx[5], es[5];
    for (uint32_t i = 0; i < k.rank; ++i) {
        gd[i] = k.dims[i];
        bx[i] = k.box[i];
        es[i] = 1;
        if (i > 0) gs[i - 1] = k.strides[i - 1];
    }
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, k.rank, const_cast<void*>(k.base), gd, gs, bx, es,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

TmapKey make_key(const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes, const uint32_t* box) {
    TmapKey k;
    std::memset(&k, 0, sizeof k);
    k.base = base;
    k.rank = static_cast<uint32_t>(rank);
    for (int i = 0; i < rank; ++i) {
        k.dims[i] = dims[i];
        k.box[i] = box[i];
        if (i > 0) k.strides[i - 1] = strides_bytes[i - 1];
    }
    return k;
}

bool make_tmap(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
               const uint32_t* box) {
    return g_tmaps.get(make_key(base, rank, dims, strides_bytes, box), encode_with_driver, m);
}

// ---- validation -------------------------------------------------------------------------------------
bool is_pow2(int x) { return x > 0 && (x & (x - 1)) == 0; }
int ilog2(int x) {
    int s = 0;
    while ((1 << s) < x) ++s;
    return s;
}

enum class Family { kGqa128, kMla576, kNone };

vpp_status validate(const vpp_chunk_attn_args* a, Family* fam) {
    if (!a) return fail(VPP_ERR_INVALID_ARG, "args is null");
    if (a->num_reqs < 0 || a->total_q < 0 || a->max_seq_len < 0)
        return fail(VPP_ERR_INVALID_ARG, "num_reqs, total_q and max_seq_len must be >= 0");
    if (a->num_q_heads <= 0 || a->num_kv_heads <= 0 || a->num_q_heads % a->num_kv_heads != 0)
        return fail(VPP_ERR_INVALID_ARG, "num_q_heads (%d) must be a positive multiple of num_kv_heads (%d)",
                    a->num_q_heads, a->num_kv_heads);
    if (!(a->softmax_scale > 0.f) || !std::isfinite(a->softmax_scale))
        return fail(VPP_ERR_INVALID_ARG, "softmax_scale must be positive and finite");
    if (a->num_kv_splits < 0 || a->num_kv_splits > 64)
        return fail(VPP_ERR_INVALID_ARG, "num_kv_splits must be in [0, 64]");
    if (a->head_dim_qk == 128 && a->head_dim_v == 128)
        *fam = Family::kGqa128;
    else if (a->head_dim_qk == 576 && a->head_dim_v == 512 && a->num_kv_heads == 1)
        *fam = Family::kMla576;
    else
        return fail(VPP_ERR_UNSUPPORTED, "no kernel for head dims (%d, %d) with %d kv heads", a->head_dim_qk,
                    a->head_dim_v, a->num_kv_heads);
    if (a->block_table != nullptr) {
        if (!is_pow2(a->block_size) || a->block_size < 16)
            return fail(VPP_ERR_UNSUPPORTED, "block_size %d: need a power of two >= 16", a->block_size);
        if (a->max_blocks_per_req <= 0 || a->num_blocks <= 0)
            return fail(VPP_ERR_INVALID_ARG, "paged cache needs max_blocks_per_req > 0 and num_blocks > 0");
    }
    return VPP_OK;
}

vpp_status validate_pointers(const vpp_chunk_attn_args* a) {
    if (a->num_reqs > 0 && (!a->prefix_len || !a->chunk_len))
        return fail(VPP_ERR_INVALID_ARG, "prefix_len / chunk_len is null");
    if (a->total_q > 0 && (!a->q || !a->out || !a->k_cache || !a->v_cache))
        return fail(VPP_ERR_INVALID_ARG, "q, k_cache, v_cache and out must be non-null");
    auto mis16 = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
    if (mis16(a->q) || mis16(a->out) || mis16(a->k_cache) || mis16(a->v_cache))
        return fail(VPP_ERR_INVALID_ARG, "q, out, k_cache and v_cache must be 16-byte aligned");
    const int64_t st[6] = {a->k_block_stride, a->k_token_stride, a->k_head_stride,
                           a->v_block_stride, a->v_token_stride, a->v_head_stride};
    for (int i = 0; i < 6; ++i)
        if (st[i] <= 0 || st[i] % 8 != 0)
            return fail(VPP_ERR_INVALID_ARG, "cache strides must be positive multiples of 8 elements");
    if (a->block_table == nullptr && a->num_reqs > 1 &&
        (a->k_block_stride < a->k_token_stride * a->max_seq_len || a->v_block_stride < a->v_token_stride * a->max_seq_len))
        return fail(VPP_ERR_INVALID_ARG,
                    "contiguous cache: every request's region must hold max_seq_len (%d) slots, but the block strides are "
                    "shorter than max_seq_len token strides", a->max_seq_len);
    return VPP_OK;
}

// Upper bound on key-range splits per query tile for this launch.
int choose_splits(const vpp_chunk_attn_args* a, int heads_per_item) {
    if (a->num_kv_splits >= 1) return a->num_kv_splits;
    const int group = a->num_q_heads / a->num_kv_heads;
    if (heads_per_item == 2 && a->total_q > 0 && a->total_q <= a->num_reqs && group <= vpp::kTileM) {
        // A decode batch of the d = 128 family: one packed item per (token, kv-head), all about max_seq_len long.  Equal
        // items fill the SMs in whole waves, so the split count is the one with the least idle last wave, charged with
        // what splitting costs (measured: partials + merge ~5 %, ~1 % per extra split, ~4 us of start-up per unit
        // against ~1.5 us per KV tile).
        const double items = static_cast<double>(a->total_q) * a->num_kv_heads;
        const double slots = sm_count_or_default();
        const double tiles = a->max_seq_len / static_cast<double>(vpp::kTileN);
        int best = 1;
        double best_cost = 0.0;
        for (int s = 1; s <= 4; ++s) {
            if (s > 1 && tiles / s < 4.0) break;   // keep at least 4 KV tiles per split
            const double waves = items * s / slots;
            double cost = std::ceil(waves) / waves;
            if (s > 1) cost *= 1.05 + 0.01 * s;
            cost *= 1.0 + (s - 1) * 4.0 / (tiles * 1.5 + 1.0);
            if (s == 1 || cost < best_cost) {
                best = s;
                best_cost = cost;
            }
        }
        return best;
    }
    if (heads_per_item == 2 && a->num_reqs == 1) {
        // One request of the d = 128 family: the work items (query tile x pair of q-heads) are about equally long, so
        // they fill the SMs in waves here too.  Measured on 8192-token chunks at 64K-128K prefixes: 512 items (3.46
        // waves) gain 7-9 % from two splits, 256 items 1.5 % from four, 128 and 1024 items are best unsplit.
        const double items = static_cast<double>((a->total_q + vpp::kTileM - 1) / vpp::kTileM) * (a->num_q_heads / 2);
        const double slots = sm_count_or_default();
        const double tiles = a->max_seq_len / static_cast<double>(vpp::kTileN);
        int best = 1;
        double best_cost = 0.0;
        for (int s = 1; s <= 8 && items > 0; ++s) {
            if (s > 1 && tiles / s < 4.0) break;   // keep at least 4 KV tiles per split
            const double waves = items * s / slots;
            double cost = std::ceil(waves) / waves;
            if (s > 1) cost *= 1.045 + 0.01 * (s - 1);                 // partials + merge
            cost *= 1.0 + (s - 1) * 4.0 / (tiles * 2.0 + 1.0);        // ~4 us of start-up per unit, ~2 us per KV tile
            if (s == 1 || cost < best_cost) {
                best = s;
                best_cost = cost;
            }
        }
        return best;
    }
    const long long tiles = (a->total_q + vpp::kTileM - 1) / vpp::kTileM + a->num_reqs;
    const long long items = tiles * (a->num_q_heads / heads_per_item);
    const int sms = sm_count_or_default();
    if (items >= 2ll * sms || items == 0) return 1;
    long long s = (2ll * sms + items - 1) / items;
    const long long by_len = (a->max_seq_len / vpp::kTileN) / 4;  // keep at least 4 KV tiles per split
    if (s > by_len) s = by_len;
    if (s > 16) s = 16;
    if (s < 1) s = 1;
    return static_cast<int>(s);
}

// The d = 128 kernel pairs two q-heads of one kv-head per work item; when a kv-head's group is odd (MHA included) an
// item is two consecutive 128-row query tiles of one q-head instead (work units of 256 rows).
bool pairs_two_heads(const vpp_chunk_attn_args* a) { return (a->num_q_heads / a->num_kv_heads) % 2 == 0; }
// The absorbed-MLA kernel runs on pairs of SMs (2-CTA clusters).
bool mla_kernel_available() { return sm_count_or_default() >= 2; }
int heads_per_item(const vpp_chunk_attn_args* a, Family fam) {
    if (fam == Family::kMla576) return 1;
    return pairs_two_heads(a) ? 2 : 1;
}

using MergeKernel = void (*)(const float*, const float*, int, long long, int, int, const int32_t*, __nv_bfloat16*, float*);
// The kernel and the grid for a merge of `splits` partials of total_q x num_q_heads rows of head_dim_v features.
MergeKernel pick_merge_kernel(int splits, long long total_q, int num_q_heads, int head_dim_v, int sms, unsigned* blocks) {
    const long long pairs = total_q * num_q_heads;
    const long long pieces = pairs * (head_dim_v / 4);
    if (splits <= vpp::kMergeSmallMax && head_dim_v % 4 == 0 && pieces < (1ll << 31)) {
        long long b = (pieces + vpp::kMergeThreads - 1) / vpp::kMergeThreads;
        if (b > 12ll * sms) b = 12ll * sms;
        *blocks = static_cast<unsigned>(b);
        if (splits <= 2) return vpp::lse_merge_small_kernel<2, 4>;
        if (splits <= 4) return vpp::lse_merge_small_kernel<4, 2>;
        return vpp::lse_merge_small_kernel<8, 1>;
    }
    long long b = (pairs * 32 + vpp::kMergeThreads - 1) / vpp::kMergeThreads;
    if (b > 8ll * sms) b = 8ll * sms;
    *blocks = static_cast<unsigned>(b);
    return vpp::lse_merge_kernel<2, 4>;
}

vpp::WorkspaceLayout layout_for(const vpp_chunk_attn_args* a, Family fam) {
    vpp::WorkspaceLayout L{};
    const int S = choose_splits(a, heads_per_item(a, fam));
    const long long tiles = (a->total_q + vpp::kTileM - 1) / vpp::kTileM + a->num_reqs;
    L.splits = S;
    L.max_units = static_cast<int32_t>(tiles * S);
    size_t off = 0;
    L.header = off;
    off = align_up(off + sizeof(vpp::WorkHeader), 256);
    L.units = off;
    off = align_up(off + sizeof(vpp::WorkUnit) * static_cast<size_t>(L.max_units > 0 ? L.max_units : 1), 256);
    L.row_splits = off;  // followed by q_start and tile_start scratch
    off = align_up(off + sizeof(int32_t) * (static_cast<size_t>(a->total_q) + 2 * (static_cast<size_t>(a->num_reqs) + 1)),
                   256);
    L.o_parts = off;
    if (S > 1)
        off = align_up(off + sizeof(float) * static_cast<size_t>(S) * a->total_q * a->num_q_heads * a->head_dim_v, 256);
    L.lse_parts = off;
    if (S > 1) off = align_up(off + sizeof(float) * static_cast<size_t>(S) * a->total_q * a->num_q_heads, 256);
    L.total = off;
    return L;
}

}  // namespace

extern "C" {

const char* vpp_status_string(vpp_status s) {
    switch (s) {
        case VPP_OK: return "ok";
        case VPP_ERR_INVALID_ARG: return "invalid argument";
        case VPP_ERR_UNSUPPORTED: return "unsupported shape";
        case VPP_ERR_WORKSPACE: return "workspace missing or too small";
        case VPP_ERR_CUDA: return "CUDA call failed";
        case VPP_ERR_TIMEOUT: return "device wait timed out";
    }
    return "unknown status";
}

const char* vpp_last_error(void) { return g_err; }
int32_t vpp_last_launch_count(void) { return g_launches; }

size_t vpp_chunk_attn_workspace_size(const vpp_chunk_attn_args* a) {
    Family fam = Family::kNone;
    if (validate(a, &fam) != VPP_OK) return 0;
    return layout_for(a, fam).total;
}

namespace {
// Key range of a partial launch, in KV tiles of kTileN keys (null: the whole causal range, final results).
struct KeyRange {
    int32_t begin_tile, end_tile;
};
vpp_status run_chunk_attn(const vpp_chunk_attn_args* a, vpp_stream_t stream_, const KeyRange* range);
}  // namespace

vpp_status vpp_chunk_attn_fwd(const vpp_chunk_attn_args* a, vpp_stream_t stream_) {
    return run_chunk_attn(a, stream_, nullptr);
}

vpp_status vpp_chunk_attn_partial_fwd(const vpp_chunk_attn_args* args, int32_t kv_begin, int32_t kv_end, float* o_part,
                                      float* lse_part, vpp_stream_t stream_) {
    g_err[0] = 0;
    if (!args) return fail(VPP_ERR_INVALID_ARG, "args is null");
    if (kv_begin < 0 || kv_end <= kv_begin) return fail(VPP_ERR_INVALID_ARG, "need 0 <= kv_begin < kv_end");
    if (kv_begin % vpp::kTileN != 0 || (kv_end % vpp::kTileN != 0 && kv_end < args->max_seq_len))
        return fail(VPP_ERR_INVALID_ARG, "kv_begin must be a multiple of %d, and so must kv_end unless it is >= max_seq_len",
                    vpp::kTileN);
    if (args->total_q > 0 && (!o_part || !lse_part)) return fail(VPP_ERR_INVALID_ARG, "o_part and lse_part must be non-null");
    vpp_chunk_attn_args b = *args;
    b.num_kv_splits = 1;       // the caller's ranges are the split
    b.out = o_part;            // (fp32 here; only checked for null and alignment)
    b.lse = lse_part;
    KeyRange r;
    r.begin_tile = kv_begin / vpp::kTileN;
    r.end_tile = static_cast<int32_t>((static_cast<int64_t>(kv_end) + vpp::kTileN - 1) / vpp::kTileN);
    return run_chunk_attn(&b, stream_, &r);
}

namespace {
vpp_status run_chunk_attn(const vpp_chunk_attn_args* a, vpp_stream_t stream_, const KeyRange* range) {
    g_err[0] = 0;
    Family fam = Family::kNone;
    vpp_status st = validate(a, &fam);
    if (st != VPP_OK) return st;
    st = validate_pointers(a);
    if (st != VPP_OK) return st;
    const vpp::WorkspaceLayout L = layout_for(a, fam);
    if (!a->workspace || a->workspace_bytes < L.total)
        return fail(VPP_ERR_WORKSPACE, "workspace: need %zu bytes, got %zu", L.total, a->workspace_bytes);
    if (reinterpret_cast<uintptr_t>(a->workspace) & 255u)
        return fail(VPP_ERR_INVALID_ARG, "workspace must be 256-byte aligned");
    if (fam == Family::kMla576 &&
        (a->v_cache != a->k_cache || a->v_block_stride != a->k_block_stride || a->v_token_stride != a->k_token_stride ||
         a->v_head_stride != a->k_head_stride))
        return fail(VPP_ERR_UNSUPPORTED,
                    "the (576, 512) kernel needs v_cache to alias k_cache with the same strides (V = first 512 features)");

    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    g_launches = 0;
    if (a->status) {
        if (cudaMemsetAsync(a->status, 0, sizeof(int32_t), stream) != cudaSuccess)
            return fail(VPP_ERR_CUDA, "memset status: %s", cudaGetErrorString(cudaGetLastError()));
    }
    if (a->total_q == 0 || a->num_reqs == 0) return VPP_OK;
    if (fam == Family::kMla576 && !mla_kernel_available())
        return fail(VPP_ERR_UNSUPPORTED, "the absorbed-MLA kernel needs clusters of two SMs");

    uint8_t* ws = static_cast<uint8_t*>(a->workspace);
    const bool paged = a->block_table != nullptr;
    const int B = paged ? a->block_size : a->max_seq_len;
    const int n_blocks = paged ? a->num_blocks : a->num_reqs;
    const int tile_n = fam == Family::kMla576 ? vpp::kMla2BoxRows : vpp::kTileN;  // keys one copy can bring (MLA: a CTA's 64 of the pair's tile)
    const int box_rows = paged ? (B < tile_n ? B : tile_n) : tile_n;

    // ---- tensor maps ----
    CUtensorMap tm_q, tm_k, tm_v;
    {
        const uint64_t d[3] = {static_cast<uint64_t>(a->head_dim_qk), static_cast<uint64_t>(a->num_q_heads),
                               static_cast<uint64_t>(a->total_q)};
        const uint64_t s[2] = {static_cast<uint64_t>(a->head_dim_qk) * 2,
                               static_cast<uint64_t>(a->head_dim_qk) * a->num_q_heads * 2};
        const uint32_t b[3] = {64, 1, static_cast<uint32_t>(vpp::kTileM)};
        if (!make_tmap(&tm_q, a->q, 3, d, s, b)) return fail(VPP_ERR_CUDA, "cuTensorMapEncodeTiled(q) failed");
    }
    {
        const uint64_t d[4] = {static_cast<uint64_t>(a->head_dim_qk), static_cast<uint64_t>(B),
                               static_cast<uint64_t>(a->num_kv_heads), static_cast<uint64_t>(n_blocks)};
        const uint64_t s[3] = {static_cast<uint64_t>(a->k_token_stride) * 2, static_cast<uint64_t>(a->k_head_stride) * 2,
                               static_cast<uint64_t>(a->k_block_stride) * 2};
        const uint32_t b[4] = {64, static_cast<uint32_t>(box_rows), 1, 1};
        if (!make_tmap(&tm_k, a->k_cache, 4, d, s, b)) return fail(VPP_ERR_CUDA, "cuTensorMapEncodeTiled(k) failed");
    }
    if (fam != Family::kMla576) {
        const uint64_t d[4] = {static_cast<uint64_t>(a->head_dim_v), static_cast<uint64_t>(B),
                               static_cast<uint64_t>(a->num_kv_heads), static_cast<uint64_t>(n_blocks)};
        const uint64_t s[3] = {static_cast<uint64_t>(a->v_token_stride) * 2, static_cast<uint64_t>(a->v_head_stride) * 2,
                               static_cast<uint64_t>(a->v_block_stride) * 2};
        const uint32_t b[4] = {64, static_cast<uint32_t>(box_rows), 1, 1};
        if (!make_tmap(&tm_v, a->v_cache, 4, d, s, b)) return fail(VPP_ERR_CUDA, "cuTensorMapEncodeTiled(v) failed");
    }

    CUtensorMap tm_q2, tm_k2, tm_v2, tm_qh;
    if (fam == Family::kGqa128) {
        // a single-token ("packed") work item takes the G q-heads of one kv-head as the rows of its Q tile
        const int G = a->num_q_heads / a->num_kv_heads;
        const uint64_t dh[3] = {static_cast<uint64_t>(a->head_dim_qk), static_cast<uint64_t>(a->num_q_heads),
                                static_cast<uint64_t>(a->total_q)};
        const uint64_t sh[2] = {static_cast<uint64_t>(a->head_dim_qk) * 2,
                                static_cast<uint64_t>(a->head_dim_qk) * a->num_q_heads * 2};
        const uint32_t bh[3] = {64, static_cast<uint32_t>(G < vpp::kTileM ? G : vpp::kTileM), 1};
        if (!make_tmap(&tm_qh, a->q, 3, dh, sh, bh)) return fail(VPP_ERR_CUDA, "cuTensorMapEncodeTiled(q heads) failed");
        // the 128 features viewed as (64, 2): a box holds both 64-column slabs of a tile
        const uint64_t dq[4] = {64, static_cast<uint64_t>(a->total_q), 2, static_cast<uint64_t>(a->num_q_heads)};
        const uint64_t sq[3] = {static_cast<uint64_t>(a->head_dim_qk) * a->num_q_heads * 2, 128,
                                static_cast<uint64_t>(a->head_dim_qk) * 2};
        const uint32_t bq[4] = {64, static_cast<uint32_t>(vpp::kTileM), 2, 1};
        if (!make_tmap(&tm_q2, a->q, 4, dq, sq, bq)) return fail(VPP_ERR_CUDA, "cuTensorMapEncodeTiled(q tiles) failed");
        const uint64_t d[5] = {64, static_cast<uint64_t>(B), 2, static_cast<uint64_t>(a->num_kv_heads),
                               static_cast<uint64_t>(n_blocks)};
        const uint64_t sk[4] = {static_cast<uint64_t>(a->k_token_stride) * 2, 128, static_cast<uint64_t>(a->k_head_stride) * 2,
                                static_cast<uint64_t>(a->k_block_stride) * 2};
        const uint64_t sv[4] = {static_cast<uint64_t>(a->v_token_stride) * 2, 128, static_cast<uint64_t>(a->v_head_stride) * 2,
                                static_cast<uint64_t>(a->v_block_stride) * 2};
        const uint32_t b5[5] = {64, static_cast<uint32_t>(box_rows), 2, 1, 1};
        if (!make_tmap(&tm_k2, a->k_cache, 5, d, sk, b5) || !make_tmap(&tm_v2, a->v_cache, 5, d, sv, b5))
            return fail(VPP_ERR_CUDA, "cuTensorMapEncodeTiled(k/v tiles) failed");
    }
    CUtensorMap tm_q9, tm_qh9, tm_k93, tm_k92;  // 64 rows of one 64-column slab per box (tm_k93 / tm_k92: of 3 / 2 slabs)
    const bool mla_pair = fam == Family::kMla576;
    if (mla_pair) {
        const uint64_t dq[4] = {64, static_cast<uint64_t>(a->total_q), static_cast<uint64_t>(vpp::kMlaSlabs),
                                static_cast<uint64_t>(a->num_q_heads)};
        const uint64_t sq[3] = {static_cast<uint64_t>(a->head_dim_qk) * a->num_q_heads * 2, 128,
                                static_cast<uint64_t>(a->head_dim_qk) * 2};
        const uint32_t bq[4] = {vpp::kMla2BoxCols, vpp::kMla2BoxRows, static_cast<uint32_t>(vpp::kMlaSlabs), 1};   // all nine slabs in one copy
        const uint64_t d[5] = {64, static_cast<uint64_t>(B), static_cast<uint64_t>(vpp::kMlaSlabs),
                               static_cast<uint64_t>(a->num_kv_heads), static_cast<uint64_t>(n_blocks)};
        const uint64_t sk[4] = {static_cast<uint64_t>(a->k_token_stride) * 2, 128, static_cast<uint64_t>(a->k_head_stride) * 2,
                                static_cast<uint64_t>(a->k_block_stride) * 2};
        // (with pages under 64 tokens the kernel copies page by page through tm_k and these two maps go unused)
        const uint32_t krows = static_cast<uint32_t>(paged && B < vpp::kMla2BoxRows ? B : vpp::kMla2BoxRows);
        const uint32_t b3[5] = {vpp::kMla2BoxCols, krows, vpp::kKG, 1, 1};               // one K hand-back group
        const uint32_t b2[5] = {vpp::kMla2BoxCols, krows, vpp::kMla2VBoxSlabs, 1, 1};    // one V chunk
        if (!make_tmap(&tm_q9, a->q, 4, dq, sq, bq) ||
            !make_tmap(&tm_k93, a->k_cache, 5, d, sk, b3) || !make_tmap(&tm_k92, a->k_cache, 5, d, sk, b2))
            return fail(VPP_ERR_CUDA, "cuTensorMapEncodeTiled(mla pair) failed");
        // packed single-token items: 64 q-heads of one token as the rows of a CTA's Q tile
        const uint64_t dh[4] = {64, static_cast<uint64_t>(a->num_q_heads), static_cast<uint64_t>(vpp::kMlaSlabs),
                                static_cast<uint64_t>(a->total_q)};
        const uint64_t sh[3] = {static_cast<uint64_t>(a->head_dim_qk) * 2, 128,
                                static_cast<uint64_t>(a->head_dim_qk) * a->num_q_heads * 2};
        const uint32_t bh[4] = {64, 64, static_cast<uint32_t>(vpp::kMlaSlabs), 1};   // heads past num_q_heads read as zero
        if (!make_tmap(&tm_qh9, a->q, 4, dh, sh, bh)) return fail(VPP_ERR_CUDA, "cuTensorMapEncodeTiled(mla q heads) failed");
    }
    // ---- work decomposition ----
    int32_t* row_splits = reinterpret_cast<int32_t*>(ws + L.row_splits);
    vpp::PrepParams pp{};
    pp.prefix_len = a->prefix_len;
    pp.chunk_len = a->chunk_len;
    pp.block_table = a->block_table;
    pp.num_reqs = a->num_reqs;
    pp.total_q = a->total_q;
    pp.max_seq_len = a->max_seq_len;
    pp.max_blocks_per_req = a->max_blocks_per_req;
    pp.block_shift = paged ? ilog2(B) : 0;
    pp.num_blocks = n_blocks;
    pp.splits = L.splits;
    pp.max_units = L.max_units;
    pp.max_cost = (a->max_seq_len + vpp::kTileN - 1) / vpp::kTileN;
    if (pp.max_cost < 1) pp.max_cost = 1;
    pp.tile_m = (fam == Family::kGqa128 && !pairs_two_heads(a)) ? 2 * vpp::kTileM : vpp::kTileM;
    pp.partial = range ? 1 : 0;
    pp.range_begin = range ? range->begin_tile : 0;
    pp.range_end = range ? range->end_tile : 0;
    pp.header = reinterpret_cast<vpp::WorkHeader*>(ws + L.header);
    pp.units = reinterpret_cast<vpp::WorkUnit*>(ws + L.units);
    pp.row_splits = row_splits;
    pp.q_start = row_splits + a->total_q;
    pp.tile_start = pp.q_start + a->num_reqs + 1;
    pp.status = a->status;
    {
        // small launches (a short chunk, a small decode batch) take the one-warp decomposition
        const long long tiles_ub = (a->total_q + pp.tile_m - 1) / pp.tile_m + a->num_reqs;
        if (a->num_reqs <= vpp::kPrepSmallMax && tiles_ub <= vpp::kPrepSmallMax)
            vpp::prep_small_kernel<<<1, 32, 0, stream>>>(pp);
        else
            vpp::prep_kernel<<<1, vpp::kPrepThreads, 0, stream>>>(pp);
    }
    ++g_launches;

    // ---- attention ----
    vpp::AttnParams ap{};
    ap.block_table = a->block_table;
    ap.max_blocks_per_req = a->max_blocks_per_req;
    ap.block_shift = pp.block_shift;
    ap.num_blocks = n_blocks;
    ap.num_q_heads = a->num_q_heads;
    ap.num_kv_heads = a->num_kv_heads;
    ap.total_q = a->total_q;
    ap.scale_log2e = a->softmax_scale * 1.4426950408889634f;
    ap.out = a->out;
    ap.lse = a->lse;
    // a partial launch writes "split 0" of the caller's buffers, which have the merge kernel's input layout
    ap.o_parts = range ? static_cast<float*>(a->out) : reinterpret_cast<float*>(ws + L.o_parts);
    ap.lse_parts = range ? a->lse : reinterpret_cast<float*>(ws + L.lse_parts);
    ap.header_ro = pp.header;
    ap.header = pp.header;
    ap.units = pp.units;
    ap.status = a->status;

    const int sms = sm_count_or_default();
    cudaError_t ce;
    if (mla_pair) {
        auto kern = vpp::attn_mla2_kernel;
        ce = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, vpp::kMla2SmemBytes);
        if (ce == cudaSuccess) kern<<<(sms / 2) * 2, vpp::kMla2Threads, vpp::kMla2SmemBytes, stream>>>(tm_q9, tm_qh9, tm_k93, tm_k92, tm_k, ap, box_rows);
    } else {
        // a second producer warp for launches bound by the arrival of K/V: pages smaller than a KV tile, batches of decode rows
        const bool v_warp = box_rows < vpp::kTileN || a->total_q <= a->num_reqs;
        auto kern = pairs_two_heads(a) ? (v_warp ? vpp::attn128_ws_kernel<false, true> : vpp::attn128_ws_kernel<false, false>)
                                       : (v_warp ? vpp::attn128_ws_kernel<true, true> : vpp::attn128_ws_kernel<true, false>);
        ce = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, vpp::kWsSmemBytes);
        if (ce == cudaSuccess) {
            // programmatic dependent launch: set-up overlaps the work-decomposition kernel (the kernel waits for it
            // before it reads the work list)
            cudaLaunchAttribute attr{};
            attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr.val.programmaticStreamSerializationAllowed = 1;
            cudaLaunchConfig_t cfg{};
            cfg.gridDim = dim3(sms);
            cfg.blockDim = dim3(vpp::kWsThreads);
            cfg.dynamicSmemBytes = vpp::kWsSmemBytes;
            cfg.stream = stream;
            cfg.attrs = &attr;
            cfg.numAttrs = 1;
            ce = cudaLaunchKernelEx(&cfg, kern, tm_q, tm_k, tm_v, tm_q2, tm_k2, tm_v2, tm_qh, ap, box_rows);
        }
    }
    if (ce != cudaSuccess) return fail(VPP_ERR_CUDA, "attention kernel attributes: %s", cudaGetErrorString(ce));
    ++g_launches;

    // ---- merge of split partials ----
    if (L.splits > 1) {
        unsigned blocks = 1;
        const MergeKernel mk = pick_merge_kernel(L.splits, a->total_q, a->num_q_heads, a->head_dim_v, sms, &blocks);
        cudaLaunchAttribute attr{};
        attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr.val.programmaticStreamSerializationAllowed = 1;
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3(blocks);
        cfg.blockDim = dim3(vpp::kMergeThreads);
        cfg.stream = stream;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        ce = cudaLaunchKernelEx(&cfg, mk, static_cast<const float*>(ap.o_parts),
                                static_cast<const float*>(ap.lse_parts), static_cast<int>(L.splits),
                                static_cast<long long>(a->total_q), static_cast<int>(a->num_q_heads),
                                static_cast<int>(a->head_dim_v), static_cast<const int32_t*>(row_splits),
                                static_cast<__nv_bfloat16*>(a->out), a->lse);
        if (ce != cudaSuccess) return fail(VPP_ERR_CUDA, "merge launch: %s", cudaGetErrorString(ce));
        ++g_launches;
    }
    ce = cudaGetLastError();
    if (ce != cudaSuccess) return fail(VPP_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(ce));
    return VPP_OK;
}
}  // namespace

vpp_status vpp_lse_merge(const float* o_parts, const float* lse_parts, int32_t num_splits, int32_t total_q,
                         int32_t num_q_heads, int32_t head_dim_v, void* out, float* lse, vpp_stream_t stream_) {
    g_err[0] = 0;
    if (num_splits <= 0 || total_q < 0 || num_q_heads <= 0 || head_dim_v <= 0)
        return fail(VPP_ERR_INVALID_ARG, "num_splits, num_q_heads, head_dim_v must be > 0 and total_q >= 0");
    if (head_dim_v % 8 != 0) return fail(VPP_ERR_UNSUPPORTED, "head_dim_v must be a multiple of 8");
    if (num_splits > vpp::kMergeMaxSplits) return fail(VPP_ERR_UNSUPPORTED, "at most %d splits", vpp::kMergeMaxSplits);
    if (total_q == 0) return VPP_OK;
    if (!o_parts || !lse_parts || !out) return fail(VPP_ERR_INVALID_ARG, "o_parts, lse_parts and out must be non-null");
    if ((reinterpret_cast<uintptr_t>(o_parts) | reinterpret_cast<uintptr_t>(out)) & 15u)
        return fail(VPP_ERR_INVALID_ARG, "o_parts and out must be 16-byte aligned");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    unsigned blocks = 1;
    const MergeKernel mk = pick_merge_kernel(num_splits, total_q, num_q_heads, head_dim_v, sm_count_or_default(), &blocks);
    mk<<<blocks, vpp::kMergeThreads, 0, stream>>>(o_parts, lse_parts, num_splits, total_q, num_q_heads, head_dim_v, nullptr,
                                                  static_cast<__nv_bfloat16*>(out), lse);
    cudaError_t ce = cudaGetLastError();
    if (ce != cudaSuccess) return fail(VPP_ERR_CUDA, "merge launch: %s", cudaGetErrorString(ce));
    return VPP_OK;
}

vpp_status vpp_kv_append(const vpp_kv_append_args* a, vpp_stream_t stream_) {
    g_err[0] = 0;
    if (!a) return fail(VPP_ERR_INVALID_ARG, "args is null");
    if (a->num_reqs < 0 || a->total_q < 0 || a->num_kv_heads <= 0 || a->head_dim_qk <= 0 || a->head_dim_v <= 0)
        return fail(VPP_ERR_INVALID_ARG, "num_reqs, total_q >= 0 and num_kv_heads, head dims > 0 required");
    if (a->head_dim_qk % 8 || a->head_dim_v % 8) return fail(VPP_ERR_UNSUPPORTED, "head dims must be multiples of 8");
    if (a->num_reqs > vpp::kAppendMaxReqs) return fail(VPP_ERR_UNSUPPORTED, "at most %d requests", vpp::kAppendMaxReqs);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (a->status && cudaMemsetAsync(a->status, 0, sizeof(int32_t), stream) != cudaSuccess)
        return fail(VPP_ERR_CUDA, "memset status: %s", cudaGetErrorString(cudaGetLastError()));
    if (a->total_q == 0 || a->num_reqs == 0) return VPP_OK;
    if (!a->k_new || !a->k_cache || !a->prefix_len || !a->chunk_len)
        return fail(VPP_ERR_INVALID_ARG, "k_new, k_cache, prefix_len and chunk_len must be non-null");
    if (a->v_new && !a->v_cache) return fail(VPP_ERR_INVALID_ARG, "v_new given without v_cache");
    int shift = 0;
    long long capacity = a->max_seq_len;
    if (a->block_table) {
        if (a->block_size < 1 || (a->block_size & (a->block_size - 1)))
            return fail(VPP_ERR_UNSUPPORTED, "block_size must be a power of two");
        if (a->max_blocks_per_req <= 0 || a->num_blocks <= 0)
            return fail(VPP_ERR_INVALID_ARG, "max_blocks_per_req and num_blocks must be > 0 with a block table");
        while ((1 << shift) < a->block_size) ++shift;
        capacity = static_cast<long long>(a->max_blocks_per_req) * a->block_size;
    } else if (a->max_seq_len <= 0) {
        return fail(VPP_ERR_INVALID_ARG, "max_seq_len must be > 0 for a contiguous cache");
    }
    const int64_t strides[6] = {a->k_block_stride, a->k_token_stride, a->k_head_stride,
                                a->v_block_stride, a->v_token_stride, a->v_head_stride};
    for (int i = 0; i < (a->v_new ? 6 : 3); ++i)
        if (strides[i] < 0 || strides[i] % 8) return fail(VPP_ERR_INVALID_ARG, "strides must be non-negative multiples of 8 elements");
    uintptr_t al = reinterpret_cast<uintptr_t>(a->k_new) | reinterpret_cast<uintptr_t>(a->k_cache);
    if (a->v_new) al |= reinterpret_cast<uintptr_t>(a->v_new) | reinterpret_cast<uintptr_t>(a->v_cache);
    if (al & 15u) return fail(VPP_ERR_INVALID_ARG, "k_new, v_new and the caches must be 16-byte aligned");

    vpp::AppendParams p{};
    p.k_new = static_cast<const uint4*>(a->k_new);
    p.v_new = static_cast<const uint4*>(a->v_new);
    p.k_cache = static_cast<uint8_t*>(a->k_cache);
    p.v_cache = static_cast<uint8_t*>(a->v_cache);
    p.k_block_stride = a->k_block_stride * 2; p.k_token_stride = a->k_token_stride * 2; p.k_head_stride = a->k_head_stride * 2;
    p.v_block_stride = a->v_block_stride * 2; p.v_token_stride = a->v_token_stride * 2; p.v_head_stride = a->v_head_stride * 2;
    p.block_table = a->block_table;
    p.prefix_len = a->prefix_len;
    p.chunk_len = a->chunk_len;
    p.num_reqs = a->num_reqs;
    p.max_blocks_per_req = a->max_blocks_per_req;
    p.block_shift = shift;
    p.num_blocks = a->num_blocks;
    p.capacity = capacity;
    p.total_q = a->total_q;
    p.num_kv_heads = a->num_kv_heads;
    p.k_vecs = a->head_dim_qk / 8;
    p.v_vecs = a->v_new ? a->head_dim_v / 8 : 0;
    p.status = a->status;
    const int rows_per_block = vpp::kAppendThreads / 32;
    long long blocks = (static_cast<long long>(a->total_q) + rows_per_block - 1) / rows_per_block;
    const long long cap = 16ll * sm_count_or_default();
    if (blocks > cap) blocks = cap;
    const size_t smem = sizeof(int32_t) * (static_cast<size_t>(a->num_reqs) + 1);
    vpp::kv_append_kernel<<<static_cast<unsigned>(blocks), vpp::kAppendThreads, smem, stream>>>(p);
    cudaError_t ce = cudaGetLastError();
    if (ce != cudaSuccess) return fail(VPP_ERR_CUDA, "append launch: %s", cudaGetErrorString(ce));
    return VPP_OK;
}

size_t vpp_sparse_attn_workspace_size(int32_t total_q) {
    return 256 + sizeof(int2) * static_cast<size_t>(total_q > 0 ? total_q : 0);
}

vpp_status vpp_sparse_mla_fwd(const vpp_sparse_attn_args* a, vpp_stream_t stream_) {
    g_err[0] = 0;
    if (!a) return fail(VPP_ERR_INVALID_ARG, "args is null");
    if (a->num_reqs < 0 || a->total_q < 0) return fail(VPP_ERR_INVALID_ARG, "num_reqs and total_q must be >= 0");
    if (a->num_q_heads <= 0 || a->num_q_heads > 2 * vpp::kMla2Rows)
        return fail(VPP_ERR_UNSUPPORTED, "num_q_heads must be in 1..%d", 2 * vpp::kMla2Rows);
    if (a->topk < 1) return fail(VPP_ERR_INVALID_ARG, "topk must be >= 1");
    if (!(a->softmax_scale > 0.f) || !std::isfinite(a->softmax_scale))
        return fail(VPP_ERR_INVALID_ARG, "softmax_scale must be positive and finite");
    if (a->num_reqs > vpp::kDsaMaxReqs) return fail(VPP_ERR_UNSUPPORTED, "at most %d requests", vpp::kDsaMaxReqs);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (a->status && cudaMemsetAsync(a->status, 0, sizeof(int32_t), stream) != cudaSuccess)
        return fail(VPP_ERR_CUDA, "memset status: %s", cudaGetErrorString(cudaGetLastError()));
    if (a->total_q == 0 || a->num_reqs == 0) return VPP_OK;
    if (!a->q || !a->kv_cache || !a->indices || !a->prefix_len || !a->chunk_len || !a->out)
        return fail(VPP_ERR_INVALID_ARG, "q, kv_cache, indices, prefix_len, chunk_len and out must be non-null");
    if ((reinterpret_cast<uintptr_t>(a->q) | reinterpret_cast<uintptr_t>(a->kv_cache) | reinterpret_cast<uintptr_t>(a->out) |
         reinterpret_cast<uintptr_t>(a->workspace)) & 15u)
        return fail(VPP_ERR_INVALID_ARG, "q, kv_cache, out and workspace must be 16-byte aligned");
    if (a->kv_row_stride < vpp::kMlaDqk || a->kv_row_stride % 8)
        return fail(VPP_ERR_INVALID_ARG, "kv_row_stride must be a multiple of 8 elements and at least %d", vpp::kMlaDqk);
    if (!a->workspace || a->workspace_bytes < vpp_sparse_attn_workspace_size(a->total_q))
        return fail(VPP_ERR_WORKSPACE, "workspace too small: %zu bytes needed", vpp_sparse_attn_workspace_size(a->total_q));
    int shift = 0;
    long long capacity, num_rows;
    if (a->block_table) {
        if (a->block_size < 1 || (a->block_size & (a->block_size - 1)))
            return fail(VPP_ERR_UNSUPPORTED, "block_size must be a power of two");
        if (a->max_blocks_per_req <= 0 || a->num_blocks <= 0)
            return fail(VPP_ERR_INVALID_ARG, "max_blocks_per_req and num_blocks must be > 0 with a block table");
        while ((1 << shift) < a->block_size) ++shift;
        capacity = static_cast<long long>(a->max_blocks_per_req) * a->block_size;
        num_rows = static_cast<long long>(a->num_blocks) * a->block_size;
    } else {
        if (a->max_seq_len <= 0) return fail(VPP_ERR_INVALID_ARG, "max_seq_len must be > 0 for a contiguous cache");
        capacity = a->max_seq_len;
        num_rows = static_cast<long long>(a->num_reqs) * a->max_seq_len;
    }
    if (num_rows >= (1ll << 31)) return fail(VPP_ERR_UNSUPPORTED, "the cache must have fewer than 2^31 rows");

    CUtensorMap tm_qh, tm_rows;
    {
        const uint64_t dh[4] = {64, static_cast<uint64_t>(a->num_q_heads), static_cast<uint64_t>(vpp::kMlaSlabs),
                                static_cast<uint64_t>(a->total_q)};
        const uint64_t sh[3] = {static_cast<uint64_t>(vpp::kMlaDqk) * 2, 128,
                                static_cast<uint64_t>(vpp::kMlaDqk) * a->num_q_heads * 2};
        const uint32_t bh[4] = {64, 64, static_cast<uint32_t>(vpp::kMlaSlabs), 1};   // heads past num_q_heads read as zero
        // gather form: a box of one row; each copy names four rows
        const uint64_t dr[2] = {static_cast<uint64_t>(vpp::kMlaDqk), static_cast<uint64_t>(num_rows)};
        const uint64_t sr[1] = {static_cast<uint64_t>(a->kv_row_stride) * 2};
        const uint32_t br[2] = {64, 1};
        if (!make_tmap(&tm_qh, a->q, 4, dh, sh, bh) || !make_tmap(&tm_rows, a->kv_cache, 2, dr, sr, br))
            return fail(VPP_ERR_CUDA, "cuTensorMapEncodeTiled(sparse mla) failed");
    }
    int2* tok = reinterpret_cast<int2*>(static_cast<uint8_t*>(a->workspace));
    const int sms = sm_count_or_default();
    {
        long long blocks = (static_cast<long long>(a->total_q) + vpp::kDsaPrepThreads - 1) / vpp::kDsaPrepThreads;
        if (blocks > 4ll * sms) blocks = 4ll * sms;
        const size_t smem = sizeof(int32_t) * (static_cast<size_t>(a->num_reqs) + 1);
        vpp::dsa_tokens_kernel<<<static_cast<unsigned>(blocks), vpp::kDsaPrepThreads, smem, stream>>>(
            a->prefix_len, a->chunk_len, a->num_reqs, a->total_q, capacity, tok, a->status);
        cudaError_t ce = cudaGetLastError();
        if (ce != cudaSuccess) return fail(VPP_ERR_CUDA, "token table launch: %s", cudaGetErrorString(ce));
    }
    vpp::DsaParams p{};
    p.indices = a->indices;
    p.topk = a->topk;
    p.tok = tok;
    p.block_table = a->block_table;
    p.max_blocks_per_req = a->max_blocks_per_req;
    p.block_shift = shift;
    p.num_blocks = a->num_blocks;
    p.max_seq_len = a->max_seq_len;
    p.num_q_heads = a->num_q_heads;
    p.total_q = a->total_q;
    p.scale_log2e = a->softmax_scale * 1.4426950408889634f;
    p.out = a->out;
    p.lse = a->lse;
    p.status = a->status;
    auto kern = vpp::dsa_attn_kernel;
    cudaError_t ce = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, vpp::kMla2SmemBytes);
    if (ce == cudaSuccess) {
        int pairs = sms / 2;
        if (pairs > a->total_q) pairs = a->total_q;
        kern<<<pairs * 2, vpp::kDsaThreads, vpp::kMla2SmemBytes, stream>>>(tm_qh, tm_rows, p);
        ce = cudaGetLastError();
    }
    if (ce != cudaSuccess) return fail(VPP_ERR_CUDA, "sparse attention launch: %s", cudaGetErrorString(ce));
    g_launches = 2;
    return VPP_OK;
}


void vpp_tensor_map_cache_stats(int64_t* lookups, int64_t* encodes) {
    int64_t l = 0, e = 0;
    g_tmaps.stats(&l, &e);
    if (lookups) *lookups = l;
    if (encodes) *encodes = e;
}

int32_t vpp_test_tensor_map_cache(int32_t repeats) {
    // the cache logic with a stand-in for the driver's encoder (pure host code)
    static TmapCache cache;
    auto fake = +[](CUtensorMap* m, const TmapKey& k) {
        std::memset(m, 0, sizeof *m);
        std::memcpy(m, &k, sizeof k < sizeof *m ? sizeof k : sizeof *m);
        return true;
    };
    const uint64_t d1[3] = {128, 8, 1000}, s1[2] = {256, 2048}, d2[3] = {128, 8, 1001};
    const uint32_t b1[3] = {64, 1, 128};
    static const char anchor[64] = {0};
    int64_t l0, e0, l1, e1;
    cache.stats(&l0, &e0);
    for (int i = 0; i < repeats; ++i) {
        CUtensorMap m, ref;
        const TmapKey k = make_key(anchor, 3, d1, s1, b1);
        if (!cache.get(k, fake, &m)) return -1;
        fake(&ref, k);
        if (std::memcmp(&m, &ref, sizeof m) != 0) return -2;     // a hit must return what the encoder produced
    }
    CUtensorMap m;
    if (!cache.get(make_key(anchor, 3, d2, s1, b1), fake, &m)) return -1;    // another extent: another map
    if (!cache.get(make_key(anchor + 16, 3, d1, s1, b1), fake, &m)) return -1;   // another base: another map
    cache.stats(&l1, &e1);
    if (l1 - l0 != repeats + 2) return -3;
    return static_cast<int32_t>(e1 - e0);
}

vpp_status vpp_test_bounded_wait(int32_t* status, int64_t limit_cycles, vpp_stream_t stream_) {
    g_err[0] = 0;
    if (!status || limit_cycles <= 0 || limit_cycles > (1ll << 31))
        return fail(VPP_ERR_INVALID_ARG, "status must be non-null and limit_cycles in (0, 2^31]");
    vpp::bounded_wait_test_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream_)>>>(status, limit_cycles);
    const cudaError_t ce = cudaGetLastError();
    if (ce != cudaSuccess) return fail(VPP_ERR_CUDA, "test kernel launch: %s", cudaGetErrorString(ce));
    return VPP_OK;
}

}  // extern "C"
