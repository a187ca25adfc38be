// Stage 1 -- Algorithm 1 line 3: H <- 2 X X^T, accumulated chunk by chunk.
// The contraction itself is lq_tc_gemm (tcgen05 + TMA); this file holds the entry points,
// the fp32 -> 3 x bf16 operand split and the upper -> lower mirror.
#include "lq_common.cuh"

namespace {

// Tokens are summed in TMEM 64 * kSegIters at a time; see lq_tc_gemm_args::seg_iters.
constexpr int kSegIters = 8;

// src: rows x cols fp32 (ld).  dst: 3 stacked bf16 matrices of rows x dst_ld (hi, mid, lo).
__global__ void split3_kernel(const float* __restrict__ src, int64_t ld, int64_t rows, int64_t cols,
                              __nv_bfloat16* __restrict__ dst, int64_t dst_ld) {
    const int64_t row = blockIdx.y;
    const float* s = src + row * ld;
    __nv_bfloat16* d0 = dst + row * dst_ld;
    __nv_bfloat16* d1 = d0 + rows * dst_ld;
    __nv_bfloat16* d2 = d1 + rows * dst_ld;
    for (int64_t j = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; j < dst_ld; j += (int64_t)gridDim.x * blockDim.x) {
        float x = j < cols ? LQ_AT(s + j) : 0.0f;
        __nv_bfloat16 a, b, c;
        lq_split3(x, a, b, c);
        LQ_AT(d0 + j) = a; LQ_AT(d1 + j) = b; LQ_AT(d2 + j) = c;
    }
}

// Token-major input (n x c, features contiguous) is brought to the feature-major form the
// contraction reads (c x ld, tokens contiguous, zero beyond n), 64 x 64 tiles through shared memory.
__global__ void __launch_bounds__(256)
transpose_bf16_kernel(const __nv_bfloat16* __restrict__ src, int64_t lds, int64_t n, int64_t c,
                      __nv_bfloat16* __restrict__ dst, int64_t ldd) {
    __shared__ unsigned short tile[64][66];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int64_t t0 = (int64_t)blockIdx.x * 64, f0 = (int64_t)blockIdx.y * 64;
    const unsigned short* s16 = reinterpret_cast<const unsigned short*>(src);
    for (int rr = ty; rr < 64; rr += 8) {
        const int64_t tok = t0 + rr, f = f0 + 2 * tx;
        unsigned short a = 0, b = 0;
        if (tok < n) {
            if (f + 1 < c) {
                const uint32_t v = LQ_AT(reinterpret_cast<const uint32_t*>(s16 + tok * lds + f));
                a = static_cast<unsigned short>(v & 0xffffu);
                b = static_cast<unsigned short>(v >> 16);
            } else if (f < c) {
                a = LQ_AT(s16 + tok * lds + f);
            }
        }
        tile[rr][2 * tx] = a;
        tile[rr][2 * tx + 1] = b;
    }
    __syncthreads();
    unsigned short* d16 = reinterpret_cast<unsigned short*>(dst);
    for (int ff = ty; ff < 64; ff += 8) {
        const int64_t f = f0 + ff, tok = t0 + 2 * tx;
        if (f < c && tok < ldd) {          // ldd is even: a pair never straddles the end of a row
            const uint32_t v = static_cast<uint32_t>(tile[2 * tx][ff]) | (static_cast<uint32_t>(tile[2 * tx + 1][ff]) << 16);
            LQ_AT(reinterpret_cast<uint32_t*>(d16 + f * ldd + tok)) = v;
        }
    }
}

// The same for fp32 input, together with the split into three bf16 terms (three stacked c x ld matrices).
__global__ void __launch_bounds__(256)
transpose_split3_kernel(const float* __restrict__ src, int64_t lds, int64_t n, int64_t c,
                        __nv_bfloat16* __restrict__ dst, int64_t ldd) {
    __shared__ float tile[32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int64_t t0 = (int64_t)blockIdx.x * 32, f0 = (int64_t)blockIdx.y * 32;
    for (int rr = ty; rr < 32; rr += 8) {
        const int64_t tok = t0 + rr, f = f0 + tx;
        tile[rr][tx] = (tok < n && f < c) ? LQ_AT(src + tok * lds + f) : 0.0f;
    }
    __syncthreads();
    for (int ff = ty; ff < 32; ff += 8) {
        const int64_t f = f0 + ff, tok = t0 + tx;
        if (f < c && tok < ldd) {
            __nv_bfloat16 a, b, cc;
            lq_split3(tile[tx][ff], a, b, cc);
            LQ_AT(dst + f * ldd + tok) = a;
            LQ_AT(dst + (c + f) * ldd + tok) = b;
            LQ_AT(dst + (2 * c + f) * ldd + tok) = cc;
        }
    }
}

// H[j][i] = H[i][j] for j > i, 32 x 32 tiles through shared memory.
__global__ void mirror_upper_kernel(float* __restrict__ H, int64_t c, int64_t ldh) {
    __shared__ float tile[32][33];
    const int bi = blockIdx.y, bj = blockIdx.x;     // source tile (rows bi, cols bj), bj >= bi
    if (bj < bi) return;
    const int tx = threadIdx.x, ty = threadIdx.y;   // 32 x 8
    for (int k = ty; k < 32; k += 8) {
        int64_t i = (int64_t)bi * 32 + k, j = (int64_t)bj * 32 + tx;
        tile[k][tx] = (i < c && j < c) ? LQ_AT(H + i * ldh + j) : 0.0f;
    }
    __syncthreads();
    for (int k = ty; k < 32; k += 8) {
        int64_t j = (int64_t)bj * 32 + k, i = (int64_t)bi * 32 + tx;   // destination H[j][i]
        if (j < c && i < c && j > i) LQ_AT(H + j * ldh + i) = tile[tx][k];
    }
}

}  // namespace

extern "C" int lq_hessian_workspace(int32_t x_dtype, int32_t layout, int64_t c, int64_t n_chunk, size_t* bytes) {
    if (!bytes || c <= 0 || n_chunk < 0) return LQ_ERR_INVALID_ARG;
    if (layout != LQ_FEATURE_MAJOR && layout != LQ_TOKEN_MAJOR) return LQ_ERR_INVALID_ARG;
    if (x_dtype != LQ_F32 && x_dtype != LQ_BF16) return LQ_ERR_INVALID_ARG;
    const int64_t ld = lq_ceil_div(n_chunk, 8) * 8;
    if (x_dtype == LQ_BF16)
        *bytes = layout == LQ_FEATURE_MAJOR ? 0 : lq_align_up(static_cast<size_t>(c) * ld * sizeof(__nv_bfloat16), 256);
    else
        *bytes = lq_align_up(static_cast<size_t>(3) * c * ld * sizeof(__nv_bfloat16), 256);
    return LQ_OK;
}

extern "C" int lq_hessian_accumulate(lq_handle* h, void* stream, const void* X, int32_t x_dtype, int32_t layout,
                                     int64_t c, int64_t n_chunk, int64_t ldx, float* H, int64_t ldh, float alpha,
                                     void* ws, size_t ws_bytes) {
    if (!h || !H || c <= 0 || n_chunk < 0 || ldh < c) return LQ_ERR_INVALID_ARG;
    if (n_chunk == 0) return LQ_OK;                  // an empty chunk adds nothing
    if (layout != LQ_FEATURE_MAJOR && layout != LQ_TOKEN_MAJOR) return LQ_ERR_INVALID_ARG;
    const bool token_major = layout == LQ_TOKEN_MAJOR;
    if (!X || ldx < (token_major ? c : n_chunk)) return LQ_ERR_INVALID_ARG;
    if (x_dtype != LQ_BF16 && x_dtype != LQ_F32) return LQ_ERR_INVALID_ARG;
    if (ldh % 4 || (reinterpret_cast<uintptr_t>(H) & 15) || (reinterpret_cast<uintptr_t>(X) & 15)) return LQ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    lq_tc_gemm_args g = {};
    g.D = H; g.ldd = ldh; g.M = c; g.N = c; g.K = n_chunk;
    g.alpha = alpha; g.accumulate = 1; g.upper_only = 1;
    g.seg_iters = kSegIters;
    size_t need = 0;
    lq_hessian_workspace(x_dtype, layout, c, n_chunk, &need);
    if (need && (!ws || ws_bytes < need)) return LQ_ERR_WORKSPACE_TOO_SMALL;
    if (need && (reinterpret_cast<uintptr_t>(ws) & 15)) return LQ_ERR_INVALID_ARG;
    const int64_t ld = lq_ceil_div(n_chunk, 8) * 8;
    __nv_bfloat16* staged = static_cast<__nv_bfloat16*>(ws);
    {
        LQ_DBG_SCOPE(h, st);
        const size_t xb = x_dtype == LQ_F32 ? 4 : 2;
        LQ_DBG_REG(X, (static_cast<size_t>((token_major ? n_chunk : c) - 1) * ldx + (token_major ? c : n_chunk)) * xb);
        LQ_DBG_REG(ws, need);
        LQ_DBG_COMMIT();
    }
    if (x_dtype == LQ_BF16) {
        if (!token_major) {
            if (ldx % 8) return LQ_ERR_INVALID_ARG;
            g.A_all = g.B_all = static_cast<const __nv_bfloat16*>(X);
            g.lda = g.ldb = ldx;
        } else {
            if (ldx % 2) return LQ_ERR_INVALID_ARG;
            dim3 grid(static_cast<unsigned>(lq_ceil_div(ld, 64)), static_cast<unsigned>(lq_ceil_div(c, 64)));
            transpose_bf16_kernel<<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(X), ldx, n_chunk, c, staged, ld);
            LQ_LAUNCH_CHECK();
            g.A_all = g.B_all = staged;
            g.lda = g.ldb = ld;
        }
        g.a_rows = g.b_rows = c;
        g.n_pass = 1;
    } else {
        if (c > 65535) return LQ_ERR_UNSUPPORTED;        // rows of the split / transpose launches ride on the second grid dimension
        if (!token_major) {
            dim3 grid(static_cast<unsigned>(lq_ceil_div(ld, 256) < 64 ? lq_ceil_div(ld, 256) : 64), static_cast<unsigned>(c));
            split3_kernel<<<grid, 256, 0, st>>>(static_cast<const float*>(X), ldx, c, n_chunk, staged, ld);
        } else {
            dim3 grid(static_cast<unsigned>(lq_ceil_div(ld, 32)), static_cast<unsigned>(lq_ceil_div(c, 32)));
            transpose_split3_kernel<<<grid, 256, 0, st>>>(static_cast<const float*>(X), ldx, n_chunk, c, staged, ld);
        }
        LQ_LAUNCH_CHECK();
        g.A_all = g.B_all = staged;
        g.a_rows = g.b_rows = 3 * c; g.lda = g.ldb = ld;
        // (hi,hi) (hi,mid) (mid,hi) (hi,lo) (lo,hi) (mid,mid): every product term above 2^-24 relative
        const int64_t ao[6] = {0, 0, c, 0, 2 * c, c};
        const int64_t bo[6] = {0, c, 0, 2 * c, 0, c};
        for (int i = 0; i < 6; ++i) { g.a_row_off[i] = ao[i]; g.b_row_off[i] = bo[i]; }
        g.n_pass = 6;
    }
    return lq_tc_gemm(h, st, g);
}

extern "C" int lq_hessian_finalize(lq_handle* h, void* stream, float* H, int64_t c, int64_t ldh) {
    if (!h || !H || c <= 0 || ldh < c) return LQ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    {
        LQ_DBG_SCOPE(h, st);
        LQ_DBG_REG(H, (static_cast<size_t>(c - 1) * ldh + c) * sizeof(float));
        LQ_DBG_COMMIT();
    }
    unsigned nb = static_cast<unsigned>(lq_ceil_div(c, 32));
    mirror_upper_kernel<<<dim3(nb, nb), dim3(32, 8), 0, st>>>(H, c, ldh);
    LQ_LAUNCH_CHECK();
    return LQ_OK;
}
