// Stage 2 -- Algorithm 1 line 4: dampen H, invert, and take the upper Cholesky factor of the
// inverse ("Scaling to Billion-Parameter LLMs Using Cholesky and Dampening").
//
// Route: with H_d = H + damp*I, factor H_d = R R^T with R upper triangular (a Cholesky
// factorisation run from the last column backwards).  Then H_d^-1 = R^-T R^-1 and, by
// uniqueness of the Cholesky factor, U = R^-1 is exactly the upper factor with
// H_d^-1 = U^T U that the column loop needs; diag(H_d^-1)_j = sum_k U[k][j]^2.
// That is one factorisation plus one triangular inversion (2/3 c^3 flops) instead of
// factor + invert + factor again.
//
// Everything is fp64 (fp32 factors of an ill-conditioned H move too many quantisation
// decisions): a blocked right-looking factorisation with 128-wide panels, the diagonal
// blocks handled by one CTA in shared memory, and all panel / trailing updates done by an
// FP64 tensor-core GEMM (mma.sync m8n8k4 f64).
#include "lq_common.cuh"

namespace {

constexpr int NB = 128;          // panel width
constexpr int DP = NB + 1;       // shared-memory pitch of the diagonal block (bank-conflict free columns)

// ------------------------------------------------------------------ set-up kernels --
// scal[0] = damp = damp_frac * mean(diag H), dead (zero) diagonal entries counted as 1.
__global__ void diag_mean_kernel(const float* __restrict__ H, int64_t c, int64_t ldh, double damp_frac,
                                 double* __restrict__ scal) {
    __shared__ double red[1024];
    double s = 0.0;
    for (int64_t i = threadIdx.x; i < c; i += blockDim.x) {
        float d = H[i * ldh + i];
        s += (d == 0.0f) ? 1.0 : static_cast<double>(d);
    }
    red[threadIdx.x] = s;
    __syncthreads();
    for (int o = blockDim.x / 2; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) scal[0] = damp_frac * red[0] / static_cast<double>(c);
}

// Zero the weight columns of dead input channels.
template <typename T>
__global__ void zero_dead_columns_kernel(const float* __restrict__ H, int64_t c, int64_t ldh, T* __restrict__ W,
                                         int64_t r, int64_t ldw) {
    const int64_t j = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (j >= c) return;
    if (H[j * ldh + j] != 0.0f) return;
    for (int64_t i = blockIdx.y; i < r; i += gridDim.y) W[i * ldw + j] = T(0.0f);
}

// A[cp x cp] (fp64): upper triangle of H plus damping; identity on the padding; the strictly
// lower part is zeroed.  Non-finite inputs are reported.
__global__ void load_damped_kernel(const float* __restrict__ H, int64_t c, int64_t ldh, const double* __restrict__ scal,
                                   double* __restrict__ A, int64_t cp, lq_dev_status* st) {
    const int64_t i = blockIdx.y;
    const double damp = scal[0];
    for (int64_t j = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; j < cp; j += (int64_t)gridDim.x * blockDim.x) {
        double v = 0.0;
        if (i < c && j < c) {
            if (j >= i) {
                float hv = H[i * ldh + j];
                if (!isfinite(hv)) lq_report(st, LQ_ERR_NONFINITE, i * c + j);
                v = static_cast<double>(hv);
                if (i == j) v = (hv == 0.0f ? 1.0 : v) + damp;
            }
        } else if (i == j) {
            v = 1.0;
        }
        A[i * cp + j] = v;
    }
}

// --------------------------------------------------------- diagonal block kernel ----
// In place on the NB x NB diagonal block at A + off: reads its upper triangle (a symmetric
// positive definite block), computes the upper R with block = R R^T, inverts it, and writes
// V = R^-1 (upper; zeros below the diagonal).  One CTA of 1024 threads.
__global__ void __launch_bounds__(1024, 1)
diag_block_kernel(double* __restrict__ A, int64_t cp, int64_t blk, int64_t c_real, lq_dev_status* st) {
    extern __shared__ double S[];          // NB x DP
    __shared__ double colbuf[2][NB];
    __shared__ double vd[NB];
    __shared__ double piv[2];              // sqrt of the current pivot and its reciprocal
    double* base = A + blk * NB * cp + blk * NB;
    const int tid = threadIdx.x;
    const int tx = tid & 31, ty = tid >> 5;      // 32 x 32
    for (int i = ty; i < NB; i += 32)
        for (int j = tx; j < NB; j += 32) S[i * DP + j] = base[(int64_t)i * cp + j];
    __syncthreads();

    // Only one thread ever does the fp64 square root / division of a step.
    auto set_pivot = [&](int j) {
        double d = S[j * DP + j];
        if (!(d > 0.0) || !isfinite(d)) {
            if (blk * NB + j < c_real) lq_report(st, LQ_ERR_NOT_POSITIVE_DEFINITE, blk * NB + j);
            d = 1.0;
        }
        const double rjj = sqrt(d);
        piv[0] = rjj;
        piv[1] = 1.0 / rjj;
    };
    if (tid == 0) set_pivot(NB - 1);
    __syncthreads();

    // R R^T factorisation, last column first.
    for (int j = NB - 1; j >= 0; --j) {
        const double rjj = piv[0], rinv = piv[1];
        if (tid < j) {
            const double v = S[tid * DP + j] * rinv;
            colbuf[0][tid] = v;
            S[tid * DP + j] = v;
        } else if (tid == j) {
            S[j * DP + j] = rjj;
        }
        __syncthreads();
        for (int i = ty; i < j; i += 32) {
            const double ci = colbuf[0][i];
            for (int k = tx; k < j; k += 32)
                if (k >= i) S[i * DP + k] -= ci * colbuf[0][k];
        }
        // the thread that just finished the next pivot entry prepares its square root
        if (j > 0 && ty == ((j - 1) & 31) && tx == ((j - 1) & 31)) set_pivot(j - 1);
        __syncthreads();
    }

    // In-place inversion of the upper-triangular R, one column at a time:
    // V[j][j] = 1/R[j][j]; V[i][j] = -V[j][j] * sum_{k=i}^{j-1} V[i][k] R[k][j]  (i < j).
    if (tid < NB) vd[tid] = 1.0 / S[tid * DP + tid];
    for (int j = 0; j < NB; ++j) {
        double* cb = colbuf[j & 1];
        if (tid < j) cb[tid] = S[tid * DP + j];
        __syncthreads();                   // column j staged; column j-1 of V complete
        const int i = tid >> 3, part = tid & 7;      // 8 threads per row
        double acc = 0.0;
        if (i < j)
            for (int k = i + part; k < j; k += 8) acc += S[i * DP + k] * cb[k];
        acc += __shfl_xor_sync(0xffffffffu, acc, 1);
        acc += __shfl_xor_sync(0xffffffffu, acc, 2);
        acc += __shfl_xor_sync(0xffffffffu, acc, 4);
        if (part == 0) {
            if (i < j) S[i * DP + j] = -vd[j] * acc;
            else if (i == j) S[j * DP + j] = vd[j];
        }
    }
    __syncthreads();

    for (int i = ty; i < NB; i += 32)
        for (int j = tx; j < NB; j += 32) base[(int64_t)i * cp + j] = (j >= i) ? S[i * DP + j] : 0.0;
}

// -------------------------------------------------------------- FP64 MMA GEMM -------
// C[M x N] = alpha * A[M x K] * op(B) + beta * C, all fp64 row-major, M and N multiples of
// 64, K a multiple of 16.  TRANS_B: B is N x K (C = A B^T); otherwise B is K x N.
// a_tri: A is block upper triangular (entries left of the 64-aligned row start are zero and
// are skipped).  c_upper: tiles strictly below the diagonal are skipped.
__device__ __forceinline__ void dmma(double& c0, double& c1, double a, double b) {
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
                 : "+d"(c0), "+d"(c1) : "d"(a), "d"(b));
}

constexpr int GT = 64;    // tile
constexpr int GK = 16;
constexpr int GKP = 20;   // padded k pitch: conflict-free fragment loads

template <bool TRANS_B>
__global__ void __launch_bounds__(128)
dgemm_kernel(const double* __restrict__ A, int64_t lda, const double* __restrict__ B, int64_t ldb,
             double* __restrict__ C, int64_t ldc, int M, int N, int K, double alpha, double beta,
             int a_tri, int c_upper) {
    const int bi = blockIdx.y, bj = blockIdx.x;
    if (c_upper && bj < bi) return;
    __shared__ double As[GT * GKP];
    __shared__ double Bs[GT * GKP];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int wm0 = (warp >> 1) * 32, wn0 = (warp & 1) * 32;
    const int m0 = bi * GT, n0 = bj * GT;

    double acc[4][4][2];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j][0] = acc[i][j][1] = 0.0;

    // global -> register staging
    const int a_row = tid >> 1, a_k = (tid & 1) * 8;
    const int bt_k = tid >> 3, bt_n = (tid & 7) * 8;     // non-transposed B: 16 x 64 tile
    double ra[8], rb[8];
    const int k_begin = a_tri ? m0 : 0;

    auto load_tile = [&](int k0) {
        const double* ap = A + (int64_t)(m0 + a_row) * lda + k0 + a_k;
#pragma unroll
        for (int u = 0; u < 8; u += 2) {
            double2 v = *reinterpret_cast<const double2*>(ap + u);
            ra[u] = v.x; ra[u + 1] = v.y;
        }
        if (TRANS_B) {
            const double* bp = B + (int64_t)(n0 + a_row) * ldb + k0 + a_k;
#pragma unroll
            for (int u = 0; u < 8; u += 2) {
                double2 v = *reinterpret_cast<const double2*>(bp + u);
                rb[u] = v.x; rb[u + 1] = v.y;
            }
        } else {
            const double* bp = B + (int64_t)(k0 + bt_k) * ldb + n0 + bt_n;
#pragma unroll
            for (int u = 0; u < 8; u += 2) {
                double2 v = *reinterpret_cast<const double2*>(bp + u);
                rb[u] = v.x; rb[u + 1] = v.y;
            }
        }
    };
    auto store_tile = [&]() {
#pragma unroll
        for (int u = 0; u < 8; ++u) As[a_row * GKP + a_k + u] = ra[u];
        if (TRANS_B) {
#pragma unroll
            for (int u = 0; u < 8; ++u) Bs[a_row * GKP + a_k + u] = rb[u];
        } else {
#pragma unroll
            for (int u = 0; u < 8; ++u) Bs[(bt_n + u) * GKP + bt_k] = rb[u];
        }
    };

    if (k_begin < K) load_tile(k_begin);
    for (int k0 = k_begin; k0 < K; k0 += GK) {
        __syncthreads();
        store_tile();
        __syncthreads();
        if (k0 + GK < K) load_tile(k0 + GK);
        const int fr = lane >> 2, fk = lane & 3;
#pragma unroll
        for (int kk = 0; kk < GK; kk += 4) {
            double a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[(wm0 + 8 * i + fr) * GKP + kk + fk];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = Bs[(wn0 + 8 * j + fr) * GKP + kk + fk];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) dmma(acc[i][j][0], acc[i][j][1], a[i], b[j]);
        }
    }

    const int cr = lane >> 2, cc = (lane & 3) * 2;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            double* cp = C + (int64_t)(m0 + wm0 + 8 * i + cr) * ldc + n0 + wn0 + 8 * j + cc;
            double2 o;
            if (beta != 0.0) {
                double2 old = *reinterpret_cast<double2*>(cp);
                o.x = alpha * acc[i][j][0] + beta * old.x;
                o.y = alpha * acc[i][j][1] + beta * old.y;
            } else {
                o.x = alpha * acc[i][j][0];
                o.y = alpha * acc[i][j][1];
            }
            *reinterpret_cast<double2*>(cp) = o;
        }
}

void dgemm(cudaStream_t st, bool trans_b, const double* A, int64_t lda, const double* B, int64_t ldb, double* C,
           int64_t ldc, int64_t M, int64_t N, int64_t K, double alpha, double beta, int a_tri, int c_upper) {
    if (M <= 0 || N <= 0) return;
    dim3 grid(static_cast<unsigned>(N / GT), static_cast<unsigned>(M / GT));
    if (trans_b)
        dgemm_kernel<true><<<grid, 128, 0, st>>>(A, lda, B, ldb, C, ldc, (int)M, (int)N, (int)K, alpha, beta, a_tri, c_upper);
    else
        dgemm_kernel<false><<<grid, 128, 0, st>>>(A, lda, B, ldb, C, ldc, (int)M, (int)N, (int)K, alpha, beta, a_tri, c_upper);
}

// copy rows x NB doubles from P (pitch NB) into A's panel (pitch cp)
__global__ void copy_panel_kernel(const double* __restrict__ P, double* __restrict__ dst, int64_t rows, int64_t cp) {
    const int64_t i = blockIdx.x;
    for (int j = threadIdx.x; j < NB; j += blockDim.x) dst[i * cp + j] = P[i * NB + j];
}

// U (fp32, c x c, upper, zeros below) and dinv[j] = sum_k U64[k][j]^2.
__global__ void finalize_u_kernel(const double* __restrict__ A, int64_t cp, int64_t c, float* __restrict__ U, int64_t ldu) {
    const int64_t i = blockIdx.y;
    for (int64_t j = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; j < c; j += (int64_t)gridDim.x * blockDim.x)
        U[i * ldu + j] = (j >= i) ? static_cast<float>(A[i * cp + j]) : 0.0f;
}
__global__ void dinv_kernel(const double* __restrict__ A, int64_t cp, int64_t c, float* __restrict__ dinv) {
    const int64_t j = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (j >= c) return;
    double s = 0.0;
    for (int64_t k = 0; k <= j; ++k) {
        double u = A[k * cp + j];
        s += u * u;
    }
    dinv[j] = static_cast<float>(s);
}

}  // namespace

extern "C" int lq_prepare_hinv_workspace(int64_t c, size_t* bytes) {
    if (!bytes || c <= 0) return LQ_ERR_INVALID_ARG;
    const size_t cp = static_cast<size_t>(lq_ceil_div(c, NB)) * NB;
    *bytes = 256 + lq_align_up(cp * cp * sizeof(double), 256) + lq_align_up(cp * NB * sizeof(double), 256);
    return LQ_OK;
}

extern "C" int lq_prepare_hinv(lq_handle* h, void* stream, const float* H, int64_t c, int64_t ldh, float damp_frac,
                               float* U, int64_t ldu, float* dinv, void* W, int32_t w_dtype, int64_t r, int64_t ldw,
                               void* ws, size_t ws_bytes) {
    if (!h || !H || !U || !dinv || c <= 0 || ldh < c || ldu < c || !(damp_frac >= 0.0f)) return LQ_ERR_INVALID_ARG;
    if (W && (r <= 0 || ldw < c || (w_dtype != LQ_F32 && w_dtype != LQ_BF16))) return LQ_ERR_INVALID_ARG;
    size_t need = 0;
    lq_prepare_hinv_workspace(c, &need);
    if (!ws || ws_bytes < need) return LQ_ERR_WORKSPACE_TOO_SMALL;
    if (reinterpret_cast<uintptr_t>(ws) & 255) return LQ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    const int64_t nblk = lq_ceil_div(c, NB);
    const int64_t cp = nblk * NB;
    char* wsp = static_cast<char*>(ws);
    double* scal = reinterpret_cast<double*>(wsp);
    double* A = reinterpret_cast<double*>(wsp + 256);
    double* P = reinterpret_cast<double*>(wsp + 256 + lq_align_up(static_cast<size_t>(cp) * cp * sizeof(double), 256));

    static bool attr_set = false;
    const int diag_smem = NB * DP * sizeof(double);
    if (!attr_set) {
        LQ_CUDA_TRY(cudaFuncSetAttribute(diag_block_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, diag_smem));
        attr_set = true;
    }

    diag_mean_kernel<<<1, 1024, 0, st>>>(H, c, ldh, static_cast<double>(damp_frac), scal);
    LQ_LAUNCH_CHECK();
    if (W) {
        dim3 g(static_cast<unsigned>(lq_ceil_div(c, 256)), static_cast<unsigned>(r < 64 ? r : 64));
        if (w_dtype == LQ_F32)
            zero_dead_columns_kernel<float><<<g, 256, 0, st>>>(H, c, ldh, static_cast<float*>(W), r, ldw);
        else
            zero_dead_columns_kernel<__nv_bfloat16><<<g, 256, 0, st>>>(H, c, ldh, static_cast<__nv_bfloat16*>(W), r, ldw);
        LQ_LAUNCH_CHECK();
    }
    {
        dim3 g(static_cast<unsigned>(lq_ceil_div(cp, 256) < 32 ? lq_ceil_div(cp, 256) : 32), static_cast<unsigned>(cp));
        load_damped_kernel<<<g, 256, 0, st>>>(H, c, ldh, scal, A, cp, h->dstatus);
        LQ_LAUNCH_CHECK();
    }

    // Phase A: A = R R^T, R upper, last block column first.  Afterwards the off-diagonal
    // blocks of A hold R and every diagonal block holds the inverse of its R block.
    for (int64_t k = nblk - 1; k >= 0; --k) {
        diag_block_kernel<<<1, 1024, diag_smem, st>>>(A, cp, k, c, h->dstatus);
        LQ_LAUNCH_CHECK();
        if (k == 0) break;
        const int64_t rows = k * NB;
        double* panel = A + k * NB;                         // rows 0..rows-1, columns of block k
        const double* Vkk = A + k * NB * cp + k * NB;
        // R[0:k, k] = A[0:k, k] * Vkk^T
        dgemm(st, true, panel, cp, Vkk, cp, P, NB, rows, NB, NB, 1.0, 0.0, 0, 0);
        LQ_LAUNCH_CHECK();
        copy_panel_kernel<<<static_cast<unsigned>(rows), 128, 0, st>>>(P, panel, rows, cp);
        LQ_LAUNCH_CHECK();
        // A[0:k, 0:k] -= R[0:k, k] R[0:k, k]^T   (upper tiles only)
        dgemm(st, true, P, NB, P, NB, A, cp, rows, rows, NB, -1.0, 1.0, 0, 1);
        LQ_LAUNCH_CHECK();
    }
    // Phase B: U = R^-1 block column by block column:
    // U[0:k, k] = -(U[0:k, 0:k] * R[0:k, k]) * Vkk,  U[k, k] = Vkk.
    for (int64_t k = 1; k < nblk; ++k) {
        const int64_t rows = k * NB;
        double* panel = A + k * NB;
        const double* Vkk = A + k * NB * cp + k * NB;
        dgemm(st, false, A, cp, panel, cp, P, NB, rows, NB, rows, 1.0, 0.0, 1, 0);
        LQ_LAUNCH_CHECK();
        dgemm(st, false, P, NB, Vkk, cp, panel, cp, rows, NB, NB, -1.0, 0.0, 0, 0);
        LQ_LAUNCH_CHECK();
    }
    {
        dim3 g(static_cast<unsigned>(lq_ceil_div(c, 256) < 32 ? lq_ceil_div(c, 256) : 32), static_cast<unsigned>(c));
        finalize_u_kernel<<<g, 256, 0, st>>>(A, cp, c, U, ldu);
        LQ_LAUNCH_CHECK();
        dinv_kernel<<<static_cast<unsigned>(lq_ceil_div(c, 128)), 128, 0, st>>>(A, cp, c, dinv);
        LQ_LAUNCH_CHECK();
    }
    return LQ_OK;
}
