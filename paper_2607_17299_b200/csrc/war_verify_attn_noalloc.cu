// war_verify_attn_noalloc: the verify-attention call for callers that cannot allocate device memory.
//
// Some callers have no way to obtain a workspace: code running inside a region where the allocator must not
// be entered (a serving engine's decode loop after its memory pool has been frozen, a plugin that is only handed
// input and output buffers, a host thread that must not take the CUDA allocator's lock).  For them this entry
// point keeps the call's scratch (work list and split-KV partial results) in one fixed array that is part of the
// library image itself, so nothing is allocated, by this library or by anything it calls.
//
// The array has a fixed size (WAR_VERIFY_ATTN_NOALLOC_MAX_BYTES); every GPU that loads the library holds it until
// the process exits.  Shapes whose scratch need is larger are refused with WAR_ERR_CAPACITY.
#include "war_common.cuh"

// Scratch of the no-allocation entry point.  In host code this name is only a handle for the runtime, not a
// device address; the address that kernels may use is resolved per device below.
static __device__ __align__(256) unsigned char g_noalloc_scratch[WAR_VERIFY_ATTN_NOALLOC_MAX_BYTES];

namespace {

constexpr int kMaxDevices = 64;
void* g_scratch_ptr[kMaxDevices] = {nullptr};

// Once per device, with that device current: ask the runtime where the array lives on this device.
war_status_t scratch_for_current_device(void** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return WAR_ERR_CUDA; }
    if (dev < 0 || dev >= kMaxDevices) return WAR_ERR_UNSUPPORTED;
    if (!g_scratch_ptr[dev]) {
        void* p = nullptr;
        const cudaError_t e = cudaGetSymbolAddress((void**)&p, g_noalloc_scratch);
        if (e != cudaSuccess || !p) { (void)cudaGetLastError(); return WAR_ERR_CUDA; }
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return WAR_OK;
}

}  // namespace

extern "C" war_status_t war_verify_attn_noalloc(const void* d_q, const void* d_kpool, const void* d_vpool,
                                                const int32_t* d_page_table, const int32_t* d_prefix_len,
                                                const int32_t* d_num_nodes, const int32_t* d_parent,
                                                const war_attn_params_t* params, void* d_out, float* d_lse,
                                                war_stream_t stream) {
    const size_t need = war_verify_attn_workspace_bytes(params);
    if (need == 0) {
        // let the ordinary entry point classify the problem (invalid vs. unsupported); it returns before any launch
        return war_verify_attn(d_q, d_kpool, d_vpool, d_page_table, d_prefix_len, d_num_nodes, d_parent, params,
                               nullptr, d_out, d_lse, stream);
    }
    if (need > (size_t)WAR_VERIFY_ATTN_NOALLOC_MAX_BYTES) return WAR_ERR_CAPACITY;
    void* scratch = nullptr;
    const war_status_t st = scratch_for_current_device(&scratch);
    if (st != WAR_OK) return st;
    // Nothing in the scratch has to start at zero.  On the one-launch path the arrival counters of split units carry
    // the number of the call that wrote them, so what an earlier call left reads as "nothing yet"; on the three-launch
    // path the planning kernel writes counters, per-request records and the work list before anything reads them.
    // Partial results are only read for units written earlier in the same call.
    return war_verify_attn(d_q, d_kpool, d_vpool, d_page_table, d_prefix_len, d_num_nodes, d_parent, params, scratch,
                           d_out, d_lse, stream);
}
