// Activation ordering (appendix "Experiment Details", paragraph "Baseline Reproduction": the option the paper switches on
// for its GPTQ baseline): the columns are taken in the order of decreasing diag(H), i.e. the input channels with the
// largest activations are quantised first.  The order is a permutation of the columns; the pass then runs unchanged
// on the permuted layer (H with rows and columns permuted, W with columns permuted) and its outputs are put back.
#include "lq_common.cuh"
#include "lq_sort.cuh"

namespace {

constexpr int ORD_MAX_C = 16384;       // the diagonal is sorted by one CTA in shared memory

// perm[k] = index of the k-th largest diagonal entry (equal entries: lower index first).
__global__ void __launch_bounds__(KS_THREADS)
act_order_kernel(const float* __restrict__ H, int c, int64_t ldh, int n, int32_t* __restrict__ perm) {
    extern __shared__ __align__(16) unsigned char ord_smem[];
    unsigned long long* keys = reinterpret_cast<unsigned long long*>(ord_smem);
    const int tid = threadIdx.x;
    for (int i = tid; i < n; i += KS_THREADS) {
        unsigned long long key = ~0ull;                              // padding sorts last
        if (i < c) {
            uint32_t u = __float_as_uint(LQ_AT(H + static_cast<int64_t>(i) * ldh + i));
            u ^= (u & 0x80000000u) ? 0xffffffffu : 0x80000000u;      // ascending in the value ...
            key = (static_cast<unsigned long long>(~u) << 32) | static_cast<uint32_t>(i);   // ... so descending here
        }
        LQ_AT(keys + ks_slot(i)) = key;
    }
    __syncthreads();
    bitonic_sort<unsigned long long>(keys, n, tid);
    for (int i = tid; i < c; i += KS_THREADS) LQ_AT(perm + i) = static_cast<int32_t>(LQ_AT(keys + ks_slot(i)) & 0xffffffffu);
}

__global__ void permute_sym_kernel(const float* __restrict__ H, int64_t c, int64_t ldh, const int32_t* __restrict__ perm,
                                   float* __restrict__ Hp, int64_t ldo) {
    const int64_t a = blockIdx.y;
    const int64_t src_row = LQ_AT(perm + a);
    for (int64_t b = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; b < c; b += (int64_t)gridDim.x * blockDim.x)
        LQ_AT(Hp + a * ldo + b) = LQ_AT(H + src_row * ldh + LQ_AT(perm + b));
}

// gather: dst[i][k] = src[i][perm[k]];  scatter: dst[i][perm[k]] = src[i][k].  Elements of 1, 2 or 4 bytes.
template <typename E, bool SCATTER>
__global__ void permute_columns_kernel(const E* __restrict__ src, int64_t r, int64_t c, int64_t lds, const int32_t* __restrict__ perm,
                                       E* __restrict__ dst, int64_t ldd) {
    for (int64_t i = blockIdx.y; i < r; i += gridDim.y)
        for (int64_t k = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; k < c; k += (int64_t)gridDim.x * blockDim.x) {
            const int64_t p = LQ_AT(perm + k);
            if (SCATTER) LQ_AT(dst + i * ldd + p) = LQ_AT(src + i * lds + k);
            else LQ_AT(dst + i * ldd + k) = LQ_AT(src + i * lds + p);
        }
}

template <bool SCATTER>
int permute_columns(lq_handle* h, void* stream, const void* src, int32_t elem_bytes, int64_t r, int64_t c, int64_t lds,
                    const int32_t* perm, void* dst, int64_t ldd) {
    if (!h || !src || !dst || !perm || r <= 0 || c <= 0 || lds < c || ldd < c || src == dst) return LQ_ERR_INVALID_ARG;
    if (elem_bytes != 1 && elem_bytes != 2 && elem_bytes != 4) return LQ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    {
        LQ_DBG_SCOPE(h, st);
        LQ_DBG_REG(src, (static_cast<size_t>(r - 1) * lds + c) * elem_bytes);
        LQ_DBG_REG(dst, (static_cast<size_t>(r - 1) * ldd + c) * elem_bytes);
        LQ_DBG_REG(perm, static_cast<size_t>(c) * sizeof(int32_t));
        LQ_DBG_COMMIT();
    }
    dim3 g(static_cast<unsigned>(lq_ceil_div(c, 256) < 64 ? lq_ceil_div(c, 256) : 64), static_cast<unsigned>(r < 65535 ? r : 65535));
    if (elem_bytes == 1)
        permute_columns_kernel<uint8_t, SCATTER><<<g, 256, 0, st>>>(static_cast<const uint8_t*>(src), r, c, lds, perm, static_cast<uint8_t*>(dst), ldd);
    else if (elem_bytes == 2)
        permute_columns_kernel<uint16_t, SCATTER><<<g, 256, 0, st>>>(static_cast<const uint16_t*>(src), r, c, lds, perm, static_cast<uint16_t*>(dst), ldd);
    else
        permute_columns_kernel<uint32_t, SCATTER><<<g, 256, 0, st>>>(static_cast<const uint32_t*>(src), r, c, lds, perm, static_cast<uint32_t*>(dst), ldd);
    LQ_LAUNCH_CHECK();
    return LQ_OK;
}

}  // namespace

extern "C" int lq_act_order(lq_handle* h, void* stream, const float* H, int64_t c, int64_t ldh, int32_t* perm) {
    if (!h || !H || !perm || c <= 0 || ldh < c) return LQ_ERR_INVALID_ARG;
    if (c > ORD_MAX_C) return LQ_ERR_UNSUPPORTED;
    int n = 64;
    while (n < c) n <<= 1;
    const size_t smem = static_cast<size_t>(n + n / 32) * sizeof(unsigned long long);
    static lq_once_per_device attr_set;
    if (attr_set.first()) {
        LQ_CUDA_TRY(cudaFuncSetAttribute(act_order_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (ORD_MAX_C + ORD_MAX_C / 32) * static_cast<int>(sizeof(unsigned long long))));
    }
    {
        LQ_DBG_SCOPE(h, static_cast<cudaStream_t>(stream));
        LQ_DBG_REG(H, (static_cast<size_t>(c - 1) * ldh + c) * sizeof(float));
        LQ_DBG_REG(perm, static_cast<size_t>(c) * sizeof(int32_t));
        LQ_DBG_COMMIT();
    }
    act_order_kernel<<<1, KS_THREADS, smem, static_cast<cudaStream_t>(stream)>>>(H, static_cast<int>(c), ldh, n, perm);
    LQ_LAUNCH_CHECK();
    return LQ_OK;
}

extern "C" int lq_permute_hessian(lq_handle* h, void* stream, const float* H, int64_t c, int64_t ldh, const int32_t* perm,
                                  float* Hp, int64_t ldhp) {
    if (!h || !H || !Hp || !perm || c <= 0 || ldh < c || ldhp < c || H == Hp) return LQ_ERR_INVALID_ARG;
    if (c > 65535) return LQ_ERR_UNSUPPORTED;
    {
        LQ_DBG_SCOPE(h, static_cast<cudaStream_t>(stream));
        LQ_DBG_REG(H, (static_cast<size_t>(c - 1) * ldh + c) * sizeof(float));
        LQ_DBG_REG(Hp, (static_cast<size_t>(c - 1) * ldhp + c) * sizeof(float));
        LQ_DBG_REG(perm, static_cast<size_t>(c) * sizeof(int32_t));
        LQ_DBG_COMMIT();
    }
    dim3 g(static_cast<unsigned>(lq_ceil_div(c, 256) < 64 ? lq_ceil_div(c, 256) : 64), static_cast<unsigned>(c));
    permute_sym_kernel<<<g, 256, 0, static_cast<cudaStream_t>(stream)>>>(H, c, ldh, perm, Hp, ldhp);
    LQ_LAUNCH_CHECK();
    return LQ_OK;
}

extern "C" int lq_gather_columns(lq_handle* h, void* stream, const void* src, int32_t elem_bytes, int64_t r, int64_t c, int64_t lds,
                                 const int32_t* perm, void* dst, int64_t ldd) {
    return permute_columns<false>(h, stream, src, elem_bytes, r, c, lds, perm, dst, ldd);
}

extern "C" int lq_scatter_columns(lq_handle* h, void* stream, const void* src, int32_t elem_bytes, int64_t r, int64_t c, int64_t lds,
                                  const int32_t* perm, void* dst, int64_t ldd) {
    return permute_columns<true>(h, stream, src, elem_bytes, r, c, lds, perm, dst, ldd);
}
