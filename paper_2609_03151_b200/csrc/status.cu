// Device status words, error text, launch counter: the small shared state of the library.
#include <atomic>
#include <cstdio>
#include <cstring>

#include "common.cuh"
#include "ptx.cuh"

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

namespace {
// Two warps wait on a barrier that nothing ever arrives on: warp 0 with the given (short) limit, warp 1 with the
// normal one.  Warp 0 gives up, records {code 2, role, block, detail = waited microseconds} and raises the CTA's abort
// flag; warp 1 must then leave through that flag.  Both reach the final barrier: the kernel ends by itself.
__global__ void wait_selftest_kernel(int *status, unsigned long long limit_ns) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bar, 1);
        abort_flag = 0;
        ptx::fence_mbar_init();
    }
    __syncthreads();
    const uint64_t t0 = ptx::globaltimer_ns();
    const bool ok = ptx::mbar_wait(&bar, 0, &abort_flag, 0, warp == 0 ? limit_ns : ptx::kWaitLimitNs);
    if (!ok && warp == 0 && (threadIdx.x & 31) == 0) {
        abort_flag = 1;
        if (atomicCAS(status, 0, 2) == 0) {
            status[1] = 100;
            status[2] = (int)blockIdx.x;
            status[3] = (int)((ptx::globaltimer_ns() - t0) / 1000);
        }
    }
    __syncthreads();
}
}  // namespace

extern "C" int basp_selftest_wait_timeout(unsigned int limit_us, void *stream) {
    if (limit_us == 0 || limit_us > 1000000u) return BASP_ERR_INVALID;
    int *dev = basp_status_device_ptr();
    if (!dev) return BASP_ERR_CUDA;
    wait_selftest_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(dev, (unsigned long long)limit_us * 1000ull);
    BASP_CUDA_TRY(cudaGetLastError());
    basp_count_launch(1);
    return BASP_OK;
}

extern "C" const char *basp_strerror(int code) {
    switch (code) {
        case BASP_OK: return "ok";
        case BASP_ERR_INVALID: return "invalid plan or argument (N mod G, B > N, S mod K, head split, rank range)";
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
