// Handle management and the device status word.
#include "lq_common.cuh"

unsigned long long lq_launches_total = 0;

extern "C" uint64_t lq_launch_count(void) { return lq_launches_total; }

extern "C" const char* lq_version(void) { return "lq 0.1 (sm_100a)"; }

extern "C" int lq_create(lq_handle** out, int device) {
    if (!out) return LQ_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return LQ_ERR_CUDA;
    LQ_CUDA_TRY(cudaSetDevice(device));
    cudaDeviceProp prop;
    LQ_CUDA_TRY(cudaGetDeviceProperties(&prop, device));
    if (prop.major != 10) return LQ_ERR_UNSUPPORTED;   // kernels are built for sm_100a only
    lq_handle* h = new lq_handle;
    h->device = device;
    h->sm_count = prop.multiProcessorCount;
    h->dstatus = nullptr;
    h->aux = nullptr;
    h->ev_fork = h->ev_next = h->ev_rest = nullptr;
    if (cudaStreamCreateWithFlags(&h->aux, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_next, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_rest, cudaEventDisableTiming) != cudaSuccess) {
        if (h->ev_rest) cudaEventDestroy(h->ev_rest);
        if (h->ev_next) cudaEventDestroy(h->ev_next);
        if (h->ev_fork) cudaEventDestroy(h->ev_fork);
        if (h->aux) cudaStreamDestroy(h->aux);
        delete h;
        return LQ_ERR_CUDA;
    }
    if (cudaMalloc(&h->dstatus, sizeof(lq_dev_status)) != cudaSuccess ||
        cudaMemset(h->dstatus, 0, sizeof(lq_dev_status)) != cudaSuccess) {
        if (h->dstatus) cudaFree(h->dstatus);
        cudaEventDestroy(h->ev_rest);
        cudaEventDestroy(h->ev_next);
        cudaEventDestroy(h->ev_fork);
        cudaStreamDestroy(h->aux);
        delete h;
        return LQ_ERR_CUDA;
    }
    *out = h;
    return LQ_OK;
}

extern "C" int lq_destroy(lq_handle* h) {
    if (!h) return LQ_ERR_INVALID_ARG;
    cudaFree(h->dstatus);
    if (h->aux) {
        cudaStreamSynchronize(h->aux);
        cudaEventDestroy(h->ev_rest);
        cudaEventDestroy(h->ev_next);
        cudaEventDestroy(h->ev_fork);
        cudaStreamDestroy(h->aux);
    }
    delete h;
    return LQ_OK;
}

extern "C" int lq_sync_status(lq_handle* h, void* stream, int32_t* status, int64_t* info) {
    if (!h || !status) return LQ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    lq_dev_status host;
    LQ_CUDA_TRY(cudaMemcpyAsync(&host, h->dstatus, sizeof(host), cudaMemcpyDeviceToHost, st));
    LQ_CUDA_TRY(cudaMemsetAsync(h->dstatus, 0, sizeof(lq_dev_status), st));
    LQ_CUDA_TRY(cudaStreamSynchronize(st));
    *status = host.code;
    if (info) *info = host.info;
    return LQ_OK;
}
