// vpp_chunk_attn_fwd_static: the chunked-prefill attention entry point for callers that cannot allocate
// device memory.  Its scratch (work list, per-row split counts, split-KV partials) lives in a fixed
// array inside the library instead of a caller-provided workspace.
#include <cuda_runtime.h>

#include <cstdio>
#include <mutex>

#include "../../include/vpp.h"

namespace {

// Held by every device that loads this library, from module load until the process exits.
__device__ __align__(256) unsigned char g_static_scratch[VPP_STATIC_SCRATCH_BYTES];

std::mutex g_mu;
void* g_scratch_ptr[64] = {};   // device address of g_static_scratch, per device ordinal
bool g_scratch_ready[64] = {};

thread_local char g_static_err[256] = "";

// In host code `g_static_scratch` is only a handle: its address is not a device address.  The real
// device pointer is fetched once per device, with that device current, and passed to the kernels.
cudaError_t scratch_pointer(void** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g_scratch_ready[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_ptr[dev] = p;
        g_scratch_ready[dev] = true;
    }
    *out = g_scratch_ptr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" {

size_t vpp_static_scratch_bytes(void) { return VPP_STATIC_SCRATCH_BYTES; }

const char* vpp_static_last_error(void) { return g_static_err; }

vpp_status vpp_chunk_attn_fwd_static(const vpp_chunk_attn_args* args, vpp_stream_t stream) {
    g_static_err[0] = 0;
    if (!args) {
        snprintf(g_static_err, sizeof g_static_err, "args is null");
        return VPP_ERR_INVALID_ARG;
    }
    vpp_chunk_attn_args a = *args;
    size_t need = vpp_chunk_attn_workspace_size(&a);
    if (need == 0) {
        // invalid or unsupported arguments: report what the ordinary entry point reports for them (its argument checks
        // come before the workspace check, so nothing is enqueued)
        a.workspace = nullptr;
        a.workspace_bytes = 0;
        vpp_status st = vpp_chunk_attn_fwd(&a, stream);
        if (st == VPP_OK || st == VPP_ERR_WORKSPACE) st = VPP_ERR_INVALID_ARG;
        snprintf(g_static_err, sizeof g_static_err, "invalid or unsupported arguments: %s", vpp_last_error());
        return st;
    }
    if (need > VPP_STATIC_SCRATCH_BYTES && a.num_kv_splits == 0) {
        // the split count was the library's choice (a throughput matter): an unsplit launch needs no partials
        a.num_kv_splits = 1;
        need = vpp_chunk_attn_workspace_size(&a);
    }
    if (need == 0 || need > VPP_STATIC_SCRATCH_BYTES) {
        snprintf(g_static_err, sizeof g_static_err,
                 "this launch needs %zu bytes of scratch but the built-in scratch holds %zu: use vpp_chunk_attn_fwd "
                 "with a workspace, or lower num_kv_splits / total_q",
                 need, static_cast<size_t>(VPP_STATIC_SCRATCH_BYTES));
        return VPP_ERR_WORKSPACE;
    }
    void* scratch = nullptr;
    const cudaError_t e = scratch_pointer(&scratch);
    if (e != cudaSuccess) {
        snprintf(g_static_err, sizeof g_static_err, "cudaGetSymbolAddress: %s", cudaGetErrorString(e));
        return VPP_ERR_CUDA;
    }
    a.workspace = scratch;
    a.workspace_bytes = VPP_STATIC_SCRATCH_BYTES;
    const vpp_status st = vpp_chunk_attn_fwd(&a, stream);
    if (st != VPP_OK) snprintf(g_static_err, sizeof g_static_err, "%s", vpp_last_error());
    return st;
}

}  // extern "C"
