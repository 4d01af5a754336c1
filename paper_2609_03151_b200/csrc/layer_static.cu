// basp_layer_fwd_static: the three-launch layer for callers that cannot hand the library any
// scratch memory.  The head-sharded copies of Q, K, V and O live in a fixed array that is part of
// the library image on every GPU that loads it, so the call itself allocates nothing.
#include <cstdio>
#include <mutex>

#include "common.cuh"

namespace {

// Scratch of the static entry point.  It costs BASP_STATIC_SCRATCH_BYTES of device memory on every
// GPU that loads this library, from load until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[BASP_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void *g_scratch_ptr[kMaxDevices];   // device address of g_static_scratch, per device ordinal

// In host code `g_static_scratch` is only a handle for the runtime, not a device address; the
// address a kernel may use has to be asked for, once per device, with that device current.
int scratch_address(void **out) {
    int dev = -1;
    BASP_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return BASP_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_ptr[dev]) {
        void *p = nullptr;
        BASP_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
        if (!p) return BASP_ERR_CUDA;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return BASP_OK;
}

}  // namespace

extern "C" int basp_layer_fwd_static(const basp_plan *plan, const void *const *q_seq, const void *const *k_seq,
                                     const void *const *v_seq, void *const *o_seq, float *const *lse_shards,
                                     float softmax_scale, void *stream) {
    if (!plan) return BASP_ERR_NULL;
    const size_t need = basp_workspace_bytes(plan);
    if (need > (size_t)BASP_STATIC_SCRATCH_BYTES) {
        char msg[160];
        snprintf(msg, sizeof(msg), "layer needs %zu bytes of scratch, the static array holds %zu", need,
                 (size_t)BASP_STATIC_SCRATCH_BYTES);
        basp_set_cuda_error("basp_layer_fwd_static", 0, msg);
        return BASP_ERR_WORKSPACE;
    }
    void *scratch = nullptr;
    int rc = scratch_address(&scratch);
    if (rc != BASP_OK) return rc;
    // Nothing in the scratch has to start at zero: the first launch writes every head-sharded byte
    // that the later launches read, so whatever the previous call left behind is overwritten.
    return basp_layer_fwd(plan, q_seq, k_seq, v_seq, o_seq, lse_shards, scratch, BASP_STATIC_SCRATCH_BYTES,
                          softmax_scale, stream);
}
