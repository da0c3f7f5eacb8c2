// vpp_chunk_attn_host_fwd: one chunk of one request whose query, new keys/values and results live in HOST memory,
// streamed through the GPU in slices (the step a pipeline stage runs per chunk in the paper's chunked-prefill
// pipeline, with the host as the source and sink of the stage's activations).
//
// The chunk's query rows are cut into slices.  Slice i's query rows and its own key/value rows go host -> device on a
// copy stream; on the caller's stream, as soon as they have landed, vpp_kv_append writes the rows into the paged
// cache and vpp_chunk_attn_fwd attends (prefix = the request's prefix plus the earlier slices, which are in the cache
// by then); the slice's output rows go device -> host on a second copy stream.  The copies of a slice overlap the
// attention of its neighbours.  Nothing here computes: every arithmetic step runs in the kernels of api.cu.
#include <cuda_runtime.h>

#include <cstdio>
#include <mutex>

#include "../../include/vpp.h"

namespace {

constexpr int kMaxSlices = VPP_HOST_MAX_SLICES;

thread_local char g_host_err[256] = "";

struct DeviceContext {
    bool ready = false;
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t ev_in[kMaxSlices] = {}, ev_done[kMaxSlices] = {}, ev_start = nullptr, ev_end = nullptr;
};
std::mutex g_mu;
DeviceContext g_ctx[64];

cudaError_t context_for_current_device(DeviceContext** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    DeviceContext& c = g_ctx[dev];
    if (!c.ready) {
        if ((e = cudaStreamCreateWithFlags(&c.s_in, cudaStreamNonBlocking)) != cudaSuccess) return e;
        if ((e = cudaStreamCreateWithFlags(&c.s_out, cudaStreamNonBlocking)) != cudaSuccess) return e;
        for (int i = 0; i < kMaxSlices; ++i) {
            if ((e = cudaEventCreateWithFlags(&c.ev_in[i], cudaEventDisableTiming)) != cudaSuccess) return e;
            if ((e = cudaEventCreateWithFlags(&c.ev_done[i], cudaEventDisableTiming)) != cudaSuccess) return e;
        }
        if ((e = cudaEventCreateWithFlags(&c.ev_start, cudaEventDisableTiming)) != cudaSuccess) return e;
        if ((e = cudaEventCreateWithFlags(&c.ev_end, cudaEventDisableTiming)) != cudaSuccess) return e;
        c.ready = true;
    }
    *out = &c;
    return cudaSuccess;
}

struct SliceScalars {
    int32_t v[2 * kMaxSlices];   // (prefix, rows) per slice
};
// The per-slice prefix_len / chunk_len arrays of the launches below (one request each), written on the device so that
// no host buffer has to outlive the call.
__global__ void slice_scalars_kernel(int32_t* dst, SliceScalars s, int n) {
    const int i = threadIdx.x;
    if (i < 2 * n) dst[i] = s.v[i];
}

vpp_status fail(vpp_status st, const char* fmt, const char* detail = "") {
    snprintf(g_host_err, sizeof g_host_err, fmt, detail);
    return st;
}

// Head of the workspace: (prefix, rows) per slice, then one status word per append and per attention launch.
constexpr size_t kScalarBytes = 256;
static_assert(4 * kMaxSlices * sizeof(int32_t) <= kScalarBytes, "slice scalars and status words");

// *status of the whole call: the first nonzero status word of its launches, in launch order.
__global__ void combine_status_kernel(const int32_t* words, int n, int32_t* status) {
    if (threadIdx.x == 0) {
        int32_t s = 0;
        for (int i = 0; i < n && s == 0; ++i) s = words[i];
        *status = s;
    }
}

size_t round_up(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }

// The launch arguments of slice [lo, hi) of the chunk.
vpp_chunk_attn_args slice_args(const vpp_chunk_attn_host_args& h, int lo, int hi, const int32_t* scalars_dev) {
    vpp_chunk_attn_args a = h.dev;
    const size_t q_row = static_cast<size_t>(a.num_q_heads) * a.head_dim_qk * 2;
    const size_t o_row = static_cast<size_t>(a.num_q_heads) * a.head_dim_v * 2;
    a.q = static_cast<const char*>(h.dev.q) + lo * q_row;
    a.out = static_cast<char*>(h.dev.out) + lo * o_row;
    a.lse = h.dev.lse ? h.dev.lse + static_cast<size_t>(lo) * a.num_q_heads : nullptr;
    a.prefix_len = scalars_dev;
    a.chunk_len = scalars_dev + 1;
    a.num_reqs = 1;
    a.total_q = hi - lo;
    return a;
}

// Slice lengths in rows.  What a step cannot overlap is the first copy in, the last copy out and, per launch, the idle
// part of its last wave of work items; three slices of whole 128-row tiles (first, middle, last) whose lengths make
// that sum smallest.  The per-tile figures are measured ones: ~2 us per KV tile of a work item, ~55 GB/s per copy.
int plan(const vpp_chunk_attn_host_args& h, int32_t* rows) {
    const vpp_chunk_attn_args& a = h.dev;
    const int chunk = h.chunk_len, step = 128, tiles = chunk / step;
    if (chunk % step || tiles < 3) {
        rows[0] = chunk;
        return 1;
    }
    int sms = 148, dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int group = a.num_q_heads / a.num_kv_heads;
    const int items_per_tile = a.head_dim_qk == 128 ? (group % 2 == 0 ? a.num_q_heads / 2 : a.num_q_heads) : a.num_q_heads;
    const double item_ms = (h.prefix_len + chunk / 2.0) / 128 * 2.0e-3;
    const double row_in = 2.0 * (a.num_q_heads * a.head_dim_qk + a.num_kv_heads * (a.head_dim_qk + a.head_dim_v));
    const double row_out = 2.0 * a.num_q_heads * a.head_dim_v + 4.0 * a.num_q_heads;
    const double in_ms = step * row_in / 55e6, out_ms = step * row_out / 55e6;
    auto idle = [&](int k) {
        const double w = static_cast<double>(k) * items_per_tile / sms;
        const double full = static_cast<double>((static_cast<long long>(k) * items_per_tile + sms - 1) / sms);
        return (full - w) * item_ms;
    };
    double best = -1;
    for (int x = 1; x < tiles - 1; ++x)
        for (int z = 1; z < tiles - x; ++z) {
            const int y = tiles - x - z;
            const double cost = x * in_ms + z * out_ms + idle(x) + idle(y) + idle(z);
            if (best < 0 || cost < best) {
                best = cost;
                rows[0] = x * step;
                rows[1] = y * step;
                rows[2] = z * step;
            }
        }
    return 3;
}

// Validates and resolves the slice lengths; returns the slice count (0: invalid, g_host_err set).
int resolve_slices(const vpp_chunk_attn_host_args* h, int32_t* rows) {
    if (!h) return fail(VPP_ERR_INVALID_ARG, "args is null"), 0;
    const vpp_chunk_attn_args& a = h->dev;
    if (a.num_reqs != 1) return fail(VPP_ERR_INVALID_ARG, "the host entry point takes one request per call (dev.num_reqs = 1)"), 0;
    if (h->chunk_len <= 0 || h->prefix_len < 0 || a.total_q != h->chunk_len)
        return fail(VPP_ERR_INVALID_ARG, "chunk_len must be positive and equal dev.total_q, prefix_len non-negative"), 0;
    if (static_cast<long long>(h->prefix_len) + h->chunk_len > a.max_seq_len)
        return fail(VPP_ERR_INVALID_ARG, "prefix_len + chunk_len exceeds dev.max_seq_len"), 0;
    if (a.num_q_heads <= 0 || a.num_kv_heads <= 0 || a.num_q_heads % a.num_kv_heads)
        return fail(VPP_ERR_INVALID_ARG, "head counts"), 0;
    if (h->num_slices < 0 || h->num_slices > kMaxSlices || (h->num_slices > 0 && !h->slice_rows))
        return fail(VPP_ERR_INVALID_ARG, "num_slices must be 0 (the library plans) or 1..VPP_HOST_MAX_SLICES with slice_rows given"), 0;
    if (h->num_slices == 0) return plan(*h, rows);
    long long sum = 0;
    for (int i = 0; i < h->num_slices; ++i) {
        if (h->slice_rows[i] <= 0) return fail(VPP_ERR_INVALID_ARG, "slice_rows must be positive"), 0;
        rows[i] = h->slice_rows[i];
        sum += rows[i];
    }
    if (sum != h->chunk_len) return fail(VPP_ERR_INVALID_ARG, "slice_rows must add up to chunk_len"), 0;
    return h->num_slices;
}

}  // namespace

extern "C" {

const char* vpp_host_last_error(void) { return g_host_err; }

int32_t vpp_chunk_attn_host_plan(const vpp_chunk_attn_host_args* args, int32_t* slice_rows_out) {
    g_host_err[0] = 0;
    int32_t rows[kMaxSlices];
    const int n = resolve_slices(args, rows);
    for (int i = 0; i < n && slice_rows_out; ++i) slice_rows_out[i] = rows[i];
    return n;
}

size_t vpp_chunk_attn_host_workspace_size(const vpp_chunk_attn_host_args* args) {
    g_host_err[0] = 0;
    int32_t rows[kMaxSlices];
    const int n = resolve_slices(args, rows);
    if (n == 0) return 0;
    size_t total = kScalarBytes;
    int lo = 0;
    for (int i = 0; i < n; ++i) {
        const vpp_chunk_attn_args a = slice_args(*args, lo, lo + rows[i], nullptr);
        const size_t need = vpp_chunk_attn_workspace_size(&a);
        if (need == 0) return fail(VPP_ERR_INVALID_ARG, "invalid or unsupported arguments: %s", vpp_last_error()), 0;
        total += round_up(need);
        lo += rows[i];
    }
    return total;
}

vpp_status vpp_chunk_attn_host_fwd(const vpp_chunk_attn_host_args* args, vpp_stream_t stream_) {
    g_host_err[0] = 0;
    int32_t rows[kMaxSlices];
    const int n = resolve_slices(args, rows);
    if (n == 0) return VPP_ERR_INVALID_ARG;
    const vpp_chunk_attn_host_args& h = *args;
    const vpp_chunk_attn_args& d = h.dev;
    const bool aliased = d.v_cache == d.k_cache;
    if (!h.q_host || !h.k_new_host || !h.out_host || !d.q || !d.out || !h.k_new_dev || !d.workspace || (!aliased && (!h.v_new_host || !h.v_new_dev)))
        return fail(VPP_ERR_INVALID_ARG, "a required host or device pointer is null");
    if (h.lse_host && !d.lse) return fail(VPP_ERR_INVALID_ARG, "lse_host needs the device staging buffer dev.lse");
    const size_t need = vpp_chunk_attn_host_workspace_size(args);
    if (need == 0) return VPP_ERR_INVALID_ARG;
    if (d.workspace_bytes < need) return fail(VPP_ERR_WORKSPACE, "workspace smaller than vpp_chunk_attn_host_workspace_size");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);

    std::lock_guard<std::mutex> lk(g_mu);   // one call at a time enqueues on a device's copy streams
    DeviceContext* c = nullptr;
    cudaError_t e = context_for_current_device(&c);
    if (e != cudaSuccess) return fail(VPP_ERR_CUDA, "copy streams: %s", cudaGetErrorString(e));

    char* ws = static_cast<char*>(d.workspace);
    int32_t* scalars = reinterpret_cast<int32_t*>(ws);
    SliceScalars sc{};
    int lo = 0;
    for (int i = 0; i < n; ++i) {
        sc.v[2 * i] = h.prefix_len + lo;
        sc.v[2 * i + 1] = rows[i];
        lo += rows[i];
    }
    slice_scalars_kernel<<<1, 2 * kMaxSlices, 0, stream>>>(scalars, sc, n);
    if ((e = cudaGetLastError()) != cudaSuccess) return fail(VPP_ERR_CUDA, "slice scalars: %s", cudaGetErrorString(e));
#define VPP_CK(x)                                                                             \
    do {                                                                                      \
        if ((e = (x)) != cudaSuccess) return fail(VPP_ERR_CUDA, #x ": %s", cudaGetErrorString(e)); \
    } while (0)
    VPP_CK(cudaEventRecord(c->ev_start, stream));
    VPP_CK(cudaStreamWaitEvent(c->s_in, c->ev_start, 0));
    VPP_CK(cudaStreamWaitEvent(c->s_out, c->ev_start, 0));

    const size_t q_row = static_cast<size_t>(d.num_q_heads) * d.head_dim_qk * 2;
    const size_t k_row = static_cast<size_t>(d.num_kv_heads) * d.head_dim_qk * 2;
    const size_t v_row = static_cast<size_t>(d.num_kv_heads) * d.head_dim_v * 2;
    const size_t o_row = static_cast<size_t>(d.num_q_heads) * d.head_dim_v * 2;
    const size_t l_row = static_cast<size_t>(d.num_q_heads) * 4;
    size_t ws_off = kScalarBytes;
    lo = 0;
    for (int i = 0; i < n; ++i) {
        const int hi = lo + rows[i];
        const size_t nrows = static_cast<size_t>(rows[i]);
        // ---- in ----
        VPP_CK(cudaMemcpyAsync(static_cast<char*>(const_cast<void*>(d.q)) + lo * q_row, static_cast<const char*>(h.q_host) + lo * q_row,
                               nrows * q_row, cudaMemcpyHostToDevice, c->s_in));
        VPP_CK(cudaMemcpyAsync(static_cast<char*>(h.k_new_dev) + lo * k_row, static_cast<const char*>(h.k_new_host) + lo * k_row,
                               nrows * k_row, cudaMemcpyHostToDevice, c->s_in));
        if (!aliased)
            VPP_CK(cudaMemcpyAsync(static_cast<char*>(h.v_new_dev) + lo * v_row, static_cast<const char*>(h.v_new_host) + lo * v_row,
                                   nrows * v_row, cudaMemcpyHostToDevice, c->s_in));
        VPP_CK(cudaEventRecord(c->ev_in[i], c->s_in));
        // ---- append + attention ----
        VPP_CK(cudaStreamWaitEvent(stream, c->ev_in[i], 0));
        vpp_chunk_attn_args a = slice_args(h, lo, hi, scalars + 2 * i);
        a.workspace = ws + ws_off;
        a.workspace_bytes = round_up(vpp_chunk_attn_workspace_size(&a));
        ws_off += a.workspace_bytes;
        vpp_kv_append_args ap{};
        ap.k_new = static_cast<const char*>(h.k_new_dev) + lo * k_row;
        ap.v_new = aliased ? nullptr : static_cast<const char*>(h.v_new_dev) + lo * v_row;
        ap.k_cache = const_cast<void*>(d.k_cache);
        ap.v_cache = const_cast<void*>(d.v_cache);
        ap.k_block_stride = d.k_block_stride; ap.k_token_stride = d.k_token_stride; ap.k_head_stride = d.k_head_stride;
        ap.v_block_stride = d.v_block_stride; ap.v_token_stride = d.v_token_stride; ap.v_head_stride = d.v_head_stride;
        ap.block_table = d.block_table;
        ap.prefix_len = a.prefix_len;
        ap.chunk_len = a.chunk_len;
        ap.num_reqs = 1;
        ap.max_blocks_per_req = d.max_blocks_per_req;
        ap.block_size = d.block_size;
        ap.num_blocks = d.num_blocks;
        ap.total_q = rows[i];
        ap.max_seq_len = d.max_seq_len;
        ap.num_kv_heads = d.num_kv_heads;
        ap.head_dim_qk = d.head_dim_qk;
        ap.head_dim_v = d.head_dim_v;
        ap.status = scalars + 2 * kMaxSlices + 2 * i;
        a.status = scalars + 2 * kMaxSlices + 2 * i + 1;
        vpp_status st = vpp_kv_append(&ap, stream);
        if (st != VPP_OK) return fail(st, "append of a slice: %s", vpp_last_error());
        st = vpp_chunk_attn_fwd(&a, stream);
        if (st != VPP_OK) return fail(st, "attention of a slice: %s", vpp_last_error());
        VPP_CK(cudaEventRecord(c->ev_done[i], stream));
        // ---- out ----
        VPP_CK(cudaStreamWaitEvent(c->s_out, c->ev_done[i], 0));
        VPP_CK(cudaMemcpyAsync(static_cast<char*>(h.out_host) + lo * o_row, static_cast<const char*>(d.out) + lo * o_row, nrows * o_row,
                               cudaMemcpyDeviceToHost, c->s_out));
        if (h.lse_host)
            VPP_CK(cudaMemcpyAsync(reinterpret_cast<char*>(h.lse_host) + lo * l_row, reinterpret_cast<const char*>(d.lse) + lo * l_row,
                                   nrows * l_row, cudaMemcpyDeviceToHost, c->s_out));
        lo = hi;
    }
    if (d.status) {
        combine_status_kernel<<<1, 32, 0, stream>>>(scalars + 2 * kMaxSlices, 2 * n, d.status);
        VPP_CK(cudaGetLastError());
    }
    VPP_CK(cudaEventRecord(c->ev_end, c->s_out));
    VPP_CK(cudaStreamWaitEvent(stream, c->ev_end, 0));
#undef VPP_CK
    return VPP_OK;
}

}  // extern "C"
