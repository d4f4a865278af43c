// Status word, status strings.
#include "war_common.cuh"

__device__ int g_war_device_status = 0;

int* war_status_word() {
    static int* cache[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!cache[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_war_device_status) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
        cache[dev] = (int*)p;
    }
    return cache[dev];
}

extern "C" war_status_t war_device_status(war_stream_t stream, int32_t* h_status) {
    if (!h_status) return WAR_ERR_INVALID_ARG;
    int v = 0, zero = 0;
    WAR_CUDA_TRY(cudaMemcpyFromSymbolAsync(&v, g_war_device_status, sizeof(int), 0, cudaMemcpyDeviceToHost, stream));
    WAR_CUDA_TRY(cudaMemcpyToSymbolAsync(g_war_device_status, &zero, sizeof(int), 0, cudaMemcpyHostToDevice, stream));
    WAR_CUDA_TRY(cudaStreamSynchronize(stream));
    *h_status = v;
    return WAR_OK;
}

extern "C" const char* war_status_string(war_status_t s) {
    switch (s) {
        case WAR_OK: return "ok";
        case WAR_ERR_INVALID_ARG: return "invalid argument";
        case WAR_ERR_OOM: return "out of device memory";
        case WAR_ERR_CAPACITY: return "index capacity exceeded";
        case WAR_ERR_CUDA: return "CUDA runtime error";
        case WAR_ERR_TIMEOUT: return "bounded device wait expired";
        case WAR_ERR_UNSUPPORTED: return "unsupported configuration";
        case WAR_ERR_BAD_TREE: return "malformed draft tree";
        case WAR_ERR_BAD_PAGE: return "page index outside the pool";
    }
    return "unknown status";
}
