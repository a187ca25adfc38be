// Handle management and the device status word.
#include "lq_common.cuh"

#include "lq_testing.h"

std::atomic<unsigned long long> lq_launches_total{0};

extern "C" uint64_t lq_launch_count(void) { return lq_launches_total.load(std::memory_order_relaxed); }

extern "C" int lq_testing_set_wait_limit_ns(lq_handle* h, uint64_t ns) {
    if (!h) return LQ_ERR_INVALID_ARG;
    h->wait_limit_ns = ns ? ns : LQ_DEFAULT_WAIT_LIMIT_NS;
    return LQ_OK;
}

extern "C" int lq_testing_inject_stall(lq_handle* h, int32_t on) {
    if (!h) return LQ_ERR_INVALID_ARG;
    h->inject_stall = on ? 1 : 0;
    return LQ_OK;
}

extern "C" int lq_testing_set_prepare_defer_min_blocks(lq_handle* h, int32_t n_blocks) {
    if (!h) return LQ_ERR_INVALID_ARG;
    h->prep_defer_min_blocks = n_blocks < 0 ? LQ_DEFAULT_PREP_DEFER_MIN_BLOCKS : n_blocks;
    return LQ_OK;
}

extern "C" int lq_testing_set_prepare_slices_int8(lq_handle* h, int32_t on) {
    if (!h) return LQ_ERR_INVALID_ARG;
    h->prep_slices_int8 = on ? 1 : 0;
    return LQ_OK;
}

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
    h->chain = h->mid = nullptr;
    h->ev_fork = h->ev_next = h->ev_rest = h->ev_join = h->ev_next2 = h->ev_diag = h->ev_crit = nullptr;
    h->wait_limit_ns = LQ_DEFAULT_WAIT_LIMIT_NS;
    h->inject_stall = 0;
    h->prep_defer_min_blocks = LQ_DEFAULT_PREP_DEFER_MIN_BLOCKS;
    h->prep_slices_int8 = 1;
    int prio_least = 0, prio_greatest = 0;
    if (cudaDeviceGetStreamPriorityRange(&prio_least, &prio_greatest) != cudaSuccess) prio_least = prio_greatest = 0;
    if (cudaStreamCreateWithPriority(&h->aux, cudaStreamNonBlocking, prio_least) != cudaSuccess ||
        cudaStreamCreateWithPriority(&h->chain, cudaStreamNonBlocking, prio_greatest) != cudaSuccess ||
        cudaStreamCreateWithPriority(&h->mid, cudaStreamNonBlocking, prio_greatest < prio_least ? prio_greatest + 1 : prio_least) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_next2, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_diag, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_crit, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_next, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_rest, cudaEventDisableTiming) != cudaSuccess) {
        if (h->ev_rest) cudaEventDestroy(h->ev_rest);
        if (h->ev_next) cudaEventDestroy(h->ev_next);
        if (h->ev_fork) cudaEventDestroy(h->ev_fork);
        if (h->ev_join) cudaEventDestroy(h->ev_join);
        if (h->ev_next2) cudaEventDestroy(h->ev_next2);
        if (h->ev_diag) cudaEventDestroy(h->ev_diag);
        if (h->ev_crit) cudaEventDestroy(h->ev_crit);
        if (h->mid) cudaStreamDestroy(h->mid);
        if (h->chain) cudaStreamDestroy(h->chain);
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
        cudaEventDestroy(h->ev_join);
        cudaEventDestroy(h->ev_next2);
        cudaEventDestroy(h->ev_diag);
        cudaEventDestroy(h->ev_crit);
        cudaStreamDestroy(h->mid);
        cudaStreamDestroy(h->chain);
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
        cudaStreamSynchronize(h->chain);
        cudaStreamSynchronize(h->mid);
        cudaEventDestroy(h->ev_join);
        cudaEventDestroy(h->ev_next2);
        cudaEventDestroy(h->ev_diag);
        cudaEventDestroy(h->ev_crit);
        cudaStreamDestroy(h->mid);
        cudaStreamDestroy(h->chain);
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

// ---------------------------------------------------------------- peak probes ----
// Dependent-free arithmetic loops that a benchmark times to get the machine's own rate for the pipes the
// non-tensor-core stages are bound by (the roofline denominators of stages 2-4).
namespace {
constexpr int PROBE_THREADS = 256;
constexpr int PROBE_CHAINS = 8;

__global__ void __launch_bounds__(PROBE_THREADS) probe_f32_kernel(long long iters, float seed, lq_dev_status* st) {
    float a[PROBE_CHAINS];
#pragma unroll
    for (int i = 0; i < PROBE_CHAINS; ++i) a[i] = seed + static_cast<float>(threadIdx.x + i);
    const float m = 0.999999f, b = 1e-7f;
    for (long long it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < PROBE_CHAINS; ++i) a[i] = fmaf(a[i], m, b);
    }
    float s = 0.0f;
#pragma unroll
    for (int i = 0; i < PROBE_CHAINS; ++i) s += a[i];
    if (s == -1.2345f) lq_report(st, LQ_ERR_NONFINITE, -1);       // keeps the loop alive; never true
}

__global__ void __launch_bounds__(PROBE_THREADS) probe_f64_kernel(long long iters, double seed, lq_dev_status* st) {
    double a[PROBE_CHAINS];
#pragma unroll
    for (int i = 0; i < PROBE_CHAINS; ++i) a[i] = seed + static_cast<double>(threadIdx.x + i);
    const double m = 0.999999, b = 1e-7;
    for (long long it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < PROBE_CHAINS; ++i) a[i] = fma(a[i], m, b);
    }
    double s = 0.0;
#pragma unroll
    for (int i = 0; i < PROBE_CHAINS; ++i) s += a[i];
    if (s == -1.2345) lq_report(st, LQ_ERR_NONFINITE, -1);
}

// The FP64 tensor-core form stage 2 uses: one m8n8k4 product per chain and iteration (512 flops per warp).
__global__ void __launch_bounds__(PROBE_THREADS) probe_f64_mma_kernel(long long iters, double seed, lq_dev_status* st) {
    double c0[PROBE_CHAINS], c1[PROBE_CHAINS];
#pragma unroll
    for (int i = 0; i < PROBE_CHAINS; ++i) { c0[i] = seed; c1[i] = seed + i; }
    const double a = 1.0 + 1e-9 * threadIdx.x, b = 1e-9;
    for (long long it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < PROBE_CHAINS; ++i)
            asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
                         : "+d"(c0[i]), "+d"(c1[i]) : "d"(a), "d"(b));
    }
    double s = 0.0;
#pragma unroll
    for (int i = 0; i < PROBE_CHAINS; ++i) s += c0[i] + c1[i];
    if (s == -1.2345) lq_report(st, LQ_ERR_NONFINITE, -1);
}
}  // namespace

extern "C" int lq_peak_probe(lq_handle* h, void* stream, int32_t kind, int64_t iters, double* ops) {
    if (!h || !ops || iters <= 0) return LQ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int blocks = h->sm_count * 8;                                  // 2048 threads per SM
    const double threads = static_cast<double>(blocks) * PROBE_THREADS;
    switch (kind) {
        case LQ_PROBE_F32_FMA:
            probe_f32_kernel<<<blocks, PROBE_THREADS, 0, st>>>(iters, 1.0f, h->dstatus);
            *ops = threads * PROBE_CHAINS * static_cast<double>(iters);             // lane-operations (one FMA each)
            break;
        case LQ_PROBE_F64_FMA:
            probe_f64_kernel<<<blocks, PROBE_THREADS, 0, st>>>(iters, 1.0, h->dstatus);
            *ops = 2.0 * threads * PROBE_CHAINS * static_cast<double>(iters);       // flops
            break;
        case LQ_PROBE_F64_MMA:
            probe_f64_mma_kernel<<<blocks, PROBE_THREADS, 0, st>>>(iters, 1.0, h->dstatus);
            *ops = 512.0 * (threads / 32.0) * PROBE_CHAINS * static_cast<double>(iters);   // flops: 8 x 8 x 4 x 2 per warp
            break;
        default:
            return LQ_ERR_INVALID_ARG;
    }
    LQ_LAUNCH_CHECK();
    return LQ_OK;
}
