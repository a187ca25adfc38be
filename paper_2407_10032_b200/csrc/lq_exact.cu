// Algorithm 2 (Appendix, "LeanQuant-Exact"): every row is quantised in its own greedy order with a
// full downdate of its own copy of the inverse Hessian (Eq. 3 for the weights, Eq. 9 for the inverse).
//
// One CTA per row, fp64 throughout (the decisions -- which weight next, which grid point -- must be
// those of a float64 evaluation).  The row's c x c inverse lives in global memory; the O(c^2)
// downdate of Eq. 9 is not applied after every step but every `nb` steps: the columns v_m taken out
// by the steps of the current batch stay in shared memory, the column that a step needs is
//     Hinv_now[:, i] = Hinv_batch_start[:, i] - sum_m v_m (v_m[i] / pivot_m),
// and a batch ends with one rank-nb update of the matrix, which cuts its memory traffic by nb.
// The diagonal, which the greedy choice reads at every step, is kept up to date separately.
#include <cstdint>

#include "lq_common.cuh"

namespace {

constexpr int EX_THREADS = 256;
constexpr int EX_WARPS = EX_THREADS / 32;
constexpr int EX_MAX_NB = 32;

// Hinv = U^T U in fp64 from the fp32 upper factor (Hinv[i][j] = sum_{k <= min(i,j)} U[k][i] U[k][j])
__global__ void __launch_bounds__(1024) utu_kernel(const float* __restrict__ U, int64_t ldu, int64_t c, double* __restrict__ Hinv) {
    __shared__ double a[32][33], b[32][33];
    const int tx = threadIdx.x, ty = threadIdx.y;
    const int64_t i0 = static_cast<int64_t>(blockIdx.y) * 32, j0 = static_cast<int64_t>(blockIdx.x) * 32;
    const int64_t kend = min(min(i0, j0) + 32, c);
    double acc = 0.0;
    for (int64_t k0 = 0; k0 < kend; k0 += 32) {
        const int64_t k = k0 + ty;
        a[ty][tx] = (k < c && i0 + tx < c) ? static_cast<double>(U[k * ldu + i0 + tx]) : 0.0;
        b[ty][tx] = (k < c && j0 + tx < c) ? static_cast<double>(U[k * ldu + j0 + tx]) : 0.0;
        __syncthreads();
#pragma unroll 8
        for (int kk = 0; kk < 32; ++kk) acc = fma(a[kk][ty], b[kk][tx], acc);
        __syncthreads();
    }
    if (i0 + ty < c && j0 + tx < c) Hinv[(i0 + ty) * c + j0 + tx] = acc;
}

template <typename T>
__device__ __forceinline__ double ex_load(const T* p);
template <>
__device__ __forceinline__ double ex_load<float>(const float* p) { return static_cast<double>(*p); }
template <>
__device__ __forceinline__ double ex_load<__nv_bfloat16>(const __nv_bfloat16* p) { return static_cast<double>(__bfloat162float(*p)); }

struct ExactArgs {
    const void* W; int64_t ldw;
    const double* Hinv0;          // c x c
    double* slots;                // gridDim.x copies of c x c
    const float* grid;            // r x K (non-uniform)
    const float* scale; const int32_t* zero; int group, n_groups;       // affine
    uint8_t* codes;
    void* what; int what_bf16; int64_t ldwh;
    double* loss_rows;            // r
    lq_dev_status* dstatus;
    size_t slot_stride;           // doubles between two copies
    int64_t r; int c; int K; int nb;
};

// Nearest grid point by the midpoint rule (the number of midpoints strictly below w), or quant_aff.
template <bool AFFINE>
__device__ __forceinline__ void ex_quant(double w, const double* __restrict__ gpts, int K, double S, double Z, int& code, double& q) {
    if (AFFINE) {
        double t = rint(w / S) + Z;
        t = fmin(fmax(t, 0.0), static_cast<double>(K - 1));
        code = static_cast<int>(t);
        q = (t - Z) * S;
    } else {
        int a = 0;
        for (int k = 0; k + 1 < K; ++k) a += (w > 0.5 * (gpts[k] + gpts[k + 1])) ? 1 : 0;
        code = a;
        q = gpts[a];
    }
}

constexpr int EX_PER = 32;      // weights per thread at most (c <= EX_THREADS * EX_PER)

template <typename T, bool AFFINE>
__global__ void __launch_bounds__(EX_THREADS, 2) exact_row_kernel(ExactArgs A) {
    extern __shared__ __align__(16) unsigned char ex_smem[];
    const int c = A.c, nb = A.nb, K = A.K;
    double* w = reinterpret_cast<double*>(ex_smem);          // c: the row, error-compensated as it goes
    double* d = w + c;                                       // c: diagonal of the current inverse
    double* V = d + c;                                       // nb x c: the columns taken out by the steps of the current batch
    double* rpiv = V + static_cast<size_t>(nb) * c;          // nb: reciprocals of their pivots
    double* arow = rpiv + EX_MAX_NB;                         // EX_WARPS x 4 x nb: row coefficients of the batch update
    double* gpts = arow + EX_WARPS * 4 * EX_MAX_NB;          // 16
    double* red_s = gpts + 16;                               // 2 x EX_WARPS (alternating between steps)
    int* red_i = reinterpret_cast<int*>(red_s + 2 * EX_WARPS);      // 2 x EX_WARPS
    int* rows = red_i + 2 * EX_WARPS;                        // c: rows still to do, ascending (for the batch update)
    unsigned char* todo = reinterpret_cast<unsigned char*>(rows + c);      // c
    __shared__ double sh_dii[2];
    __shared__ int sh_cnt[EX_WARPS];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    double* Hi = A.slots + static_cast<size_t>(blockIdx.x) * A.slot_stride;

    for (int64_t row = blockIdx.x; row < A.r; row += gridDim.x) {
        const T* wp = static_cast<const T*>(A.W) + row * A.ldw;
        for (int j = tid; j < c; j += EX_THREADS) {
            w[j] = ex_load<T>(wp + j);
            d[j] = A.Hinv0[static_cast<size_t>(j) * c + j];
            todo[j] = 1;
        }
        if (!AFFINE && tid < K) gpts[tid] = static_cast<double>(A.grid[row * K + tid]);
        {   // this row's own copy of the inverse (only its upper triangle is kept up to date below)
            const double2* src = reinterpret_cast<const double2*>(A.Hinv0);
            double2* dst = reinterpret_cast<double2*>(Hi);
            const size_t n2 = static_cast<size_t>(c) * c / 2;
            for (size_t k = tid; k < n2; k += EX_THREADS) dst[k] = src[k];
            if ((static_cast<size_t>(c) * c & 1) && tid == 0) Hi[static_cast<size_t>(c) * c - 1] = A.Hinv0[static_cast<size_t>(c) * c - 1];
        }
        __syncthreads();

        double loss = 0.0;          // kept by every thread alike
        int kb = 0;
        for (int step = 0; step < c; ++step) {
            const int par = step & 1;
            // (a) the weight with the least loss error (q - w)^2 / (2 Hinv_ii) among those still to do
            double best = INFINITY;
            int bi = 0x7fffffff;
            for (int j = tid; j < c; j += EX_THREADS) {
                if (!todo[j]) continue;
                double S = 1.0, Z = 0.0;
                if (AFFINE) {
                    const int64_t gi = row * A.n_groups + j / A.group;
                    S = static_cast<double>(A.scale[gi]);
                    Z = static_cast<double>(A.zero[gi]);
                }
                int code;
                double q;
                ex_quant<AFFINE>(w[j], gpts, K, S, Z, code, q);
                const double e = q - w[j];
                const double sc = __ddiv_rn(__dmul_rn(e, e), 2.0 * d[j]);
                if (sc < best) { best = sc; bi = j; }          // j ascends within a thread: first minimum
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const double ob = __shfl_xor_sync(0xffffffffu, best, o);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                if (ob < best || (ob == best && oi < bi)) { best = ob; bi = oi; }
            }
            if (lane == 0) { red_s[par * EX_WARPS + warp] = best; red_i[par * EX_WARPS + warp] = bi; }
            __syncthreads();
            best = red_s[par * EX_WARPS];
            bi = red_i[par * EX_WARPS];
#pragma unroll
            for (int x = 1; x < EX_WARPS; ++x) {
                const double ob = red_s[par * EX_WARPS + x];
                const int oi = red_i[par * EX_WARPS + x];
                if (ob < best || (ob == best && oi < bi)) { best = ob; bi = oi; }
            }
            if (bi == 0x7fffffff) {                             // every score was NaN: take the first weight left
                for (int j = 0; j < c; ++j) if (todo[j]) { bi = j; break; }
            }
            const int i = bi;
            // its grid point (every thread computes it: cheaper than a broadcast)
            double qi;
            int code_i;
            {
                double S = 1.0, Z = 0.0;
                if (AFFINE) {
                    const int64_t gi = row * A.n_groups + i / A.group;
                    S = static_cast<double>(A.scale[gi]);
                    Z = static_cast<double>(A.zero[gi]);
                }
                ex_quant<AFFINE>(w[i], gpts, K, S, Z, code_i, qi);
            }
            const double err = w[i] - qi;
            // (b) column i of the current inverse: the stored upper triangle as of the start of the batch, minus the
            //     batch's downdates  sum_m v_m[j] v_m[i] / pivot_m
            double vj[EX_PER];
#pragma unroll 4
            for (int t = 0; t < EX_PER; ++t) {
                const int j = tid + t * EX_THREADS;
                if (j >= c) break;
                double x = 0.0;
                if (todo[j]) {
                    x = j <= i ? Hi[static_cast<size_t>(j) * c + i] : Hi[static_cast<size_t>(i) * c + j];
                    for (int m = 0; m < kb; ++m)
                        x = fma(-(V[static_cast<size_t>(m) * c + i] * rpiv[m]), V[static_cast<size_t>(m) * c + j], x);
                }
                vj[t] = x;
                if (j == i) sh_dii[par] = x;
            }
            __syncthreads();
            // (c) quantise weight i, spread its error (Eq. 3), downdate the diagonal (Eq. 9)
            const double dii = sh_dii[par];
            loss += __ddiv_rn(__dmul_rn(err, err), 2.0 * dii);
#pragma unroll 4
            for (int t = 0; t < EX_PER; ++t) {
                const int j = tid + t * EX_THREADS;
                if (j >= c) break;
                const double x = vj[t];
                V[static_cast<size_t>(kb) * c + j] = x;
                if (j == i) {
                    w[i] = qi;
                    todo[i] = 0;
                    rpiv[kb] = 1.0 / dii;
                    A.codes[row * c + i] = static_cast<uint8_t>(code_i);
                    if (A.what) {
                        if (A.what_bf16) static_cast<__nv_bfloat16*>(A.what)[row * A.ldwh + i] = __float2bfloat16_rn(static_cast<float>(qi));
                        else static_cast<float*>(A.what)[row * A.ldwh + i] = static_cast<float>(qi);
                    }
                    if (!(dii > 0.0)) lq_report(A.dstatus, LQ_ERR_NOT_POSITIVE_DEFINITE, row * c + i);
                } else if (todo[j]) {
                    w[j] = __dsub_rn(w[j], __dmul_rn(__ddiv_rn(x, dii), err));
                    d[j] = __dsub_rn(d[j], __ddiv_rn(__dmul_rn(x, x), dii));
                }
            }
            ++kb;
            __syncthreads();
            // (d) end of a batch: Hinv[j][l] -= sum_m v_m[j] v_m[l] / pivot_m for the rows j still to do, l >= j
            if (kb == nb && step + 1 < c) {
                // ascending list of the rows still to do
                const int per = (c + EX_THREADS - 1) / EX_THREADS;
                const int j_lo = min(tid * per, c), j_hi = min(j_lo + per, c);
                int cnt = 0;
                for (int j = j_lo; j < j_hi; ++j) cnt += todo[j];
                int incl = cnt;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int y = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += y;
                }
                if (lane == 31) sh_cnt[warp] = incl;
                __syncthreads();
                int base = incl - cnt, nr = 0;
                for (int x = 0; x < EX_WARPS; ++x) {
                    if (x < warp) base += sh_cnt[x];
                    nr += sh_cnt[x];
                }
                for (int j = j_lo; j < j_hi; ++j)
                    if (todo[j]) rows[base++] = j;
                __syncthreads();
                // each warp takes four rows at a time and walks them in strips of 128 columns (four per lane),
                // starting at the strip that holds the diagonal of the first of them
                double* aw = arow + (warp * 4) * EX_MAX_NB;
                for (int p = warp * 4; p < nr; p += EX_WARPS * 4) {
                    int jr[4];
                    double* hr[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        jr[q] = rows[min(p + q, nr - 1)];
                        hr[q] = Hi + static_cast<size_t>(jr[q]) * c;
                    }
                    const int live = min(4, nr - p);
                    if (lane < kb) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) aw[q * EX_MAX_NB + lane] = V[static_cast<size_t>(lane) * c + jr[q]] * rpiv[lane];
                    }
                    {   // the first strip of the four rows this warp takes next is asked for now
                        const int pn = p + EX_WARPS * 4 + (lane >> 3);
                        if (pn < nr) {
                            const int jn = rows[pn];
                            const int ln = (rows[min(p + EX_WARPS * 4, nr - 1)] & ~127) + (lane & 7) * 16;
                            if (ln < c) asm volatile("prefetch.global.L2 [%0];" ::"l"(Hi + static_cast<size_t>(jn) * c + ln));
                        }
                    }
                    __syncwarp();
                    for (int l0 = jr[0] & ~127; l0 < c; l0 += 128) {
                        {   // the strip after the next of the four rows is asked for now (32 lines of 128 bytes, one per lane)
                            const int ln = l0 + 256 + (lane & 7) * 16;
                            if (ln < c) asm volatile("prefetch.global.L2 [%0];" ::"l"(hr[lane >> 3] + ln));
                            if (l0 == (jr[0] & ~127)) {          // and at the start of a group also the next one
                                const int l1 = l0 + 128 + (lane & 7) * 16;
                                if (l1 < c) asm volatile("prefetch.global.L2 [%0];" ::"l"(hr[lane >> 3] + l1));
                            }
                        }
                        double x[4][4];
#pragma unroll
                        for (int q = 0; q < 4; ++q)
#pragma unroll
                            for (int t = 0; t < 4; ++t) {
                                const int l = l0 + lane + 32 * t;
                                x[q][t] = (l < c && q < live) ? hr[q][l] : 0.0;
                            }
                        for (int m = 0; m < kb; ++m) {
                            const double* vm = V + static_cast<size_t>(m) * c + l0 + lane;
                            double y[4];
#pragma unroll
                            for (int t = 0; t < 4; ++t) y[t] = (l0 + lane + 32 * t < c) ? vm[32 * t] : 0.0;
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const double cq = aw[q * EX_MAX_NB + m];
#pragma unroll
                                for (int t = 0; t < 4; ++t) x[q][t] = fma(-cq, y[t], x[q][t]);
                            }
                        }
#pragma unroll
                        for (int q = 0; q < 4; ++q)
#pragma unroll
                            for (int t = 0; t < 4; ++t) {
                                const int l = l0 + lane + 32 * t;
                                if (l < c && q < live) hr[q][l] = x[q][t];
                            }
                    }
                    __syncwarp();
                }
                kb = 0;
                __syncthreads();
            }
        }
        if (tid == 0) A.loss_rows[row] = loss;
        __syncthreads();
    }
}

__global__ void exact_loss_reduce_kernel(const double* __restrict__ rows, int64_t r, double* __restrict__ out) {
    __shared__ double part[256];
    double s = 0.0;
    for (int64_t k = threadIdx.x; k < r; k += 256) s += rows[k];      // fixed order per thread, fixed tree below
    part[threadIdx.x] = s;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) part[threadIdx.x] += part[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) *out = part[0];
}

struct ExactPlan {
    int nb;
    int slots;
    size_t smem;
    size_t off_hinv, off_slots, off_loss, total;
};

size_t exact_smem(int c, int nb) {
    return static_cast<size_t>(2 + nb) * c * sizeof(double) + (EX_MAX_NB + EX_WARPS * 4 * EX_MAX_NB + 16 + 2 * EX_WARPS) * sizeof(double) +
           (2 * EX_WARPS + c) * sizeof(int) + static_cast<size_t>(c) + 16;
}

// Batch length: as long as two CTAs still fit on an SM if that leaves at least 8 steps per batch, else one CTA per SM.
int exact_plan(int64_t r, int64_t c, int sm_count, ExactPlan* P) {
    if (c > EX_THREADS * EX_PER) return LQ_ERR_UNSUPPORTED;
    int nb = 0, per_sm = 2;
    for (int cand = EX_MAX_NB; cand >= 1; --cand)
        if (exact_smem(static_cast<int>(c), cand) <= 110 * 1024) { nb = cand; break; }
    if (nb < 8) {
        per_sm = 1;
        nb = 0;
        for (int cand = EX_MAX_NB; cand >= 1; --cand)
            if (exact_smem(static_cast<int>(c), cand) <= 220 * 1024) { nb = cand; break; }
        if (nb < 1) return LQ_ERR_UNSUPPORTED;
    }
    P->nb = nb;
    P->smem = exact_smem(static_cast<int>(c), nb);
    const size_t mat = lq_align_up(static_cast<size_t>(c) * c * sizeof(double), 256);
    int64_t slots = static_cast<int64_t>(sm_count) * per_sm;
    if (slots > r) slots = r;
    const int64_t fit = static_cast<int64_t>((static_cast<size_t>(16) << 30) / mat);     // copies of the inverse: at most 16 GiB
    if (slots > fit) slots = fit < 1 ? 1 : fit;
    P->slots = static_cast<int>(slots);
    P->off_hinv = 0;
    P->off_slots = mat;
    P->off_loss = mat + static_cast<size_t>(P->slots) * mat;
    P->total = P->off_loss + lq_align_up(static_cast<size_t>(r) * sizeof(double), 256);
    return LQ_OK;
}

int check_cfg_exact(const lq_config* cfg) {
    if (!cfg) return LQ_ERR_INVALID_ARG;
    if (cfg->bits < 2 || cfg->bits > 4) return LQ_ERR_INVALID_ARG;
    if (cfg->grid_type != LQ_GRID_NONUNIFORM && cfg->grid_type != LQ_GRID_AFFINE) return LQ_ERR_INVALID_ARG;
    if (cfg->grid_type == LQ_GRID_AFFINE && cfg->group_size < 0) return LQ_ERR_INVALID_ARG;
    return LQ_OK;
}

}  // namespace

extern "C" int lq_quantize_exact_workspace(const lq_config* cfg, int64_t r, int64_t c, size_t* bytes) {
    int e = check_cfg_exact(cfg);
    if (e) return e;
    if (!bytes || r <= 0 || c <= 0) return LQ_ERR_INVALID_ARG;
    int dev = 0, sms = 0;
    LQ_CUDA_TRY(cudaGetDevice(&dev));
    LQ_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    ExactPlan P;
    e = exact_plan(r, c, sms, &P);
    if (e) return e;
    *bytes = P.total;
    return LQ_OK;
}

extern "C" int lq_quantize_exact(lq_handle* h, void* stream, const lq_config* cfg, const void* W, int32_t w_dtype, int64_t r,
                                 int64_t c, int64_t ldw, const float* U, int64_t ldu, const float* grid, const float* scale,
                                 const int32_t* zero, uint8_t* codes, void* W_hat, int32_t what_dtype, int64_t ldwh,
                                 double* loss_out, void* ws, size_t ws_bytes) {
    int e = check_cfg_exact(cfg);
    if (e) return e;
    if (!h || !W || !U || !codes || r <= 0 || c <= 0 || ldw < c || ldu < c) return LQ_ERR_INVALID_ARG;
    if (w_dtype != LQ_F32 && w_dtype != LQ_BF16) return LQ_ERR_INVALID_ARG;
    if (W_hat && (ldwh < c || (what_dtype != LQ_F32 && what_dtype != LQ_BF16))) return LQ_ERR_INVALID_ARG;
    const bool affine = cfg->grid_type == LQ_GRID_AFFINE;
    int group = 0, n_groups = 1;
    if (affine) {
        if (!scale || !zero) return LQ_ERR_INVALID_ARG;
        const int64_t g = cfg->group_size == 0 ? c : cfg->group_size;
        if (c % g) return LQ_ERR_INVALID_ARG;
        group = static_cast<int>(g);
        n_groups = static_cast<int>(c / g);
    } else if (!grid) {
        return LQ_ERR_INVALID_ARG;
    }
    ExactPlan P;
    e = exact_plan(r, c, h->sm_count, &P);
    if (e) return e;
    if (!ws || ws_bytes < P.total) return LQ_ERR_WORKSPACE_TOO_SMALL;
    if (reinterpret_cast<uintptr_t>(ws) & 255) return LQ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char* wsp = static_cast<char*>(ws);
    double* Hinv0 = reinterpret_cast<double*>(wsp + P.off_hinv);

    {
        dim3 g(static_cast<unsigned>(lq_ceil_div(c, 32)), static_cast<unsigned>(lq_ceil_div(c, 32)));
        utu_kernel<<<g, dim3(32, 32), 0, st>>>(U, ldu, c, Hinv0);
        LQ_LAUNCH_CHECK();
    }
    ExactArgs A;
    A.W = W; A.ldw = ldw;
    A.Hinv0 = Hinv0;
    A.slots = reinterpret_cast<double*>(wsp + P.off_slots);
    A.grid = grid; A.scale = scale; A.zero = zero; A.group = group > 0 ? group : 1; A.n_groups = n_groups;
    A.codes = codes;
    A.what = W_hat; A.what_bf16 = (what_dtype == LQ_BF16); A.ldwh = ldwh;
    A.loss_rows = reinterpret_cast<double*>(wsp + P.off_loss);
    A.dstatus = h->dstatus;
    A.slot_stride = lq_align_up(static_cast<size_t>(c) * c * sizeof(double), 256) / sizeof(double);
    A.r = r; A.c = static_cast<int>(c); A.K = 1 << cfg->bits; A.nb = P.nb;

#define LQ_EXACT_LAUNCH(TT, AFF)                                                                                              \
    do {                                                                                                                      \
        LQ_CUDA_TRY(cudaFuncSetAttribute(exact_row_kernel<TT, AFF>, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024)); \
        exact_row_kernel<TT, AFF><<<P.slots, EX_THREADS, P.smem, st>>>(A);                                                    \
    } while (0)
    if (w_dtype == LQ_F32) {
        if (affine) LQ_EXACT_LAUNCH(float, true); else LQ_EXACT_LAUNCH(float, false);
    } else {
        if (affine) LQ_EXACT_LAUNCH(__nv_bfloat16, true); else LQ_EXACT_LAUNCH(__nv_bfloat16, false);
    }
#undef LQ_EXACT_LAUNCH
    LQ_LAUNCH_CHECK();
    if (loss_out) {
        exact_loss_reduce_kernel<<<1, 256, 0, st>>>(A.loss_rows, r, loss_out);
        LQ_LAUNCH_CHECK();
    }
    return LQ_OK;
}
