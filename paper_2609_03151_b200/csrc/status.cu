// Device status words, error text, launch counter: the small shared state of the library.
#include <atomic>
#include <cstdio>
#include <cstring>

#include "common.cuh"

namespace {
__device__ int g_basp_status[4];              // {code, role, block, detail}; 0 = fine
thread_local char t_cuda_error[256] = "";
std::atomic<long long> g_launches{0};
}  // namespace

void basp_set_cuda_error(const char *what, int cuda_code, const char *text) {
    snprintf(t_cuda_error, sizeof(t_cuda_error), "%s: %s (%d)", what, text, cuda_code);
}

void basp_count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

// Device address of the status words on the current device (NULL on failure).
int *basp_status_device_ptr() {
    int *p = nullptr;
    cudaError_t e = cudaGetSymbolAddress((void **)&p, g_basp_status);
    if (e != cudaSuccess) {
        basp_set_cuda_error("cudaGetSymbolAddress(status)", (int)e, cudaGetErrorString(e));
        return nullptr;
    }
    return p;
}

extern "C" int basp_get_status(void *stream, int *status_out) {
    int host[4] = {0, 0, 0, 0};
    int *dev = basp_status_device_ptr();
    if (!dev) return BASP_ERR_CUDA;
    BASP_CUDA_TRY(cudaMemcpyAsync(host, dev, sizeof(host), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    BASP_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    if (status_out) memcpy(status_out, host, sizeof(host));
    return host[0] == 0 ? BASP_OK : BASP_ERR_TIMEOUT;
}

extern "C" int basp_clear_status(void *stream) {
    int *dev = basp_status_device_ptr();
    if (!dev) return BASP_ERR_CUDA;
    BASP_CUDA_TRY(cudaMemsetAsync(dev, 0, 4 * sizeof(int), (cudaStream_t)stream));
    return BASP_OK;
}

extern "C" const char *basp_strerror(int code) {
    switch (code) {
        case BASP_OK: return "ok";
        case BASP_ERR_INVALID: return "invalid plan or argument (N mod G, B > N, S mod K, head split)";
        case BASP_ERR_UNSUPPORTED: return "valid but not implemented by the kernels";
        case BASP_ERR_NULL: return "null pointer";
        case BASP_ERR_ALIGN: return "device pointer not 16-byte aligned";
        case BASP_ERR_ALIAS: return "output shard overlaps an input shard";
        case BASP_ERR_CUDA: return "CUDA call failed";
        case BASP_ERR_TIMEOUT: return "a bounded wait inside a kernel expired";
        case BASP_ERR_WORKSPACE: return "workspace too small";
        default: return "unknown error";
    }
}

extern "C" const char *basp_last_cuda_error(void) { return t_cuda_error; }

extern "C" long long basp_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }
