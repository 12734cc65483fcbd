// Process-wide pieces of the library: the device status word, error text, launch counter.
#include "common.cuh"
#include <atomic>
#include <mutex>
#include <string>

namespace csd {

static std::mutex g_mu;
static int* g_status_host = nullptr;   // mapped pinned host word
static int* g_status_dev = nullptr;    // its device alias
static thread_local std::string g_cuda_error;
static std::atomic<long long> g_launches{0};

int* status_word_device() {
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g_status_dev) {
        int* h = nullptr;
        if (cudaHostAlloc((void**)&h, sizeof(int), cudaHostAllocMapped) != cudaSuccess) {
            note_cuda(cudaGetLastError());
            return nullptr;
        }
        *h = 0;
        int* d = nullptr;
        if (cudaHostGetDevicePointer((void**)&d, h, 0) != cudaSuccess) {
            note_cuda(cudaGetLastError());
            cudaFreeHost(h);
            return nullptr;
        }
        g_status_host = h;
        g_status_dev = d;
    }
    return g_status_dev;
}

csd_status note_cuda(cudaError_t e) {
    if (e == cudaSuccess) return CSD_OK;
    g_cuda_error = cudaGetErrorString(e);
    return CSD_ERR_CUDA;
}

void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
long long launches_so_far() { return g_launches.load(std::memory_order_relaxed); }

}  // namespace csd

using namespace csd;

extern "C" const char* csd_status_string(csd_status s) {
    switch (s) {
        case CSD_OK: return "ok";
        case CSD_ERR_INVALID_ARG: return "invalid argument";
        case CSD_ERR_SHAPE: return "unsupported model shape";
        case CSD_ERR_CAPACITY: return "capacity exceeded";
        case CSD_ERR_OOM: return "out of host memory";
        case CSD_ERR_CUDA: return "CUDA runtime error";
        case CSD_ERR_BAD_TOKEN: return "token id outside the vocabulary";
        case CSD_ERR_TIMEOUT: return "bounded device loop reached its limit";
        case CSD_ERR_UNSUPPORTED: return "unsupported";
    }
    return "unknown status";
}

extern "C" const char* csd_last_cuda_error(void) { return g_cuda_error.c_str(); }

extern "C" csd_status csd_device_status(void* stream, int* code_out) {
    if (!code_out) return CSD_ERR_INVALID_ARG;
    if (!status_word_device()) return CSD_ERR_CUDA;
    CSD_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    std::lock_guard<std::mutex> lk(g_mu);
    *code_out = *(volatile int*)g_status_host;
    *(volatile int*)g_status_host = 0;
    return CSD_OK;
}
