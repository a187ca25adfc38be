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
// The two are run as ONE sweep over 128-wide block columns k = last .. 0.  R is inverted in
// place by block Gauss-Jordan elimination with the pivots taken in the same descending order,
// so that step k needs exactly what the factorisation has produced by then:
//   diag   : A[k][k] (symmetric positive definite) -> V_k = R_kk^-1            (one CTA)
//   panel  : P_i = A[i][k] V_k^T = R[i][k]  (i < k);   A[k][j] <- V_k A[k][j]  (j > k, final U)
//   update : A[i][j] -= P_i P_j^T   (i <= j < k, the Cholesky trailing update)
//            A[i][j] -= P_i A[k][j] (i < k < j, the Gauss-Jordan update)
//            A[i][k]  = -P_i V_k    (i < k)
// Every product has inner dimension 128 and all of a step's updates form one launch over the
// whole width, so the grid stays large from the first step to the last.
//
// The matrix, the diagonal blocks and the panels are fp64 (fp32 factors of an ill-conditioned H move
// too many quantisation decisions).  The updates are done in two levels over outer blocks of
// OBB = 8 block columns (1024 columns):
//   eager    : the rows and the columns of the current outer block get every step's update at once, on the
//              FP64 tensor-core MMA (mma.sync m8n8k4 f64) fed by a cp.async ring -- these are the tiles the
//              outer block's own diagonal and panel kernels read;
//   deferred : all other tiles (rows above the outer block, columns outside it) get the updates of the outer
//              block's steps in one product of inner dimension 1024 when the outer block is complete, on the
//              integer tensor cores (tcgen05 kind::i8, lq_tc_gemm).  The fp64 operands are cut into S = 5 slices of
//              balanced 8-bit integer digits below a per-row power of two; a product of two slices is a sum of
//              integers that the int32 accumulator holds exactly, the leading slice pair (s = t = 1) is kept as a
//              result of its own and the other pairs with s + t <= S + 1 are combined, least significant level first,
//              in fp32; the two results are added in fp64 and scaled back (15 integer products in all).  Worth ~39 bits
//              relative to the largest entry of a row; entries of one row of a panel differ by several bits, which is
//              why four slices are not enough (U then comes out 1e-7 to 5e-7 of its largest entry off, measured here and
//              in the CPU emulation alike; five hold it to 1e-8).  An fp32 accumulation of split floating-point
//              operands keeps ~20 bits whatever the number of terms and moves 0.1 - 0.2 % of the codes.  The same
//              slices as bf16 values on the bf16 path (exact in its fp32 accumulator per 128 of the inner dimension)
//              remain selectable for tests; the integer path runs the stage 1.2 - 1.5 x faster.
#include "lq_common.cuh"

namespace {

constexpr int NB = 128;          // block width

// ------------------------------------------------------------------ set-up kernels --
// scal[0] = damp = damp_frac * mean(diag H), dead (zero) diagonal entries counted as 1.
__global__ void diag_mean_kernel(const float* __restrict__ H, int64_t c, int64_t ldh, double damp_frac,
                                 double* __restrict__ scal) {
    __shared__ double red[1024];
    double s = 0.0;
    for (int64_t i = threadIdx.x; i < c; i += blockDim.x) {
        float d = LQ_AT(H + i * ldh + i);
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
    if (LQ_AT(H + j * ldh + j) != 0.0f) return;
    for (int64_t i = blockIdx.y; i < r; i += gridDim.y) LQ_AT(W + i * ldw + j) = T(0.0f);
}

// A[cp x cp] (fp64): upper triangle of H plus damping; identity on the padding; the strictly
// lower part is zeroed.  Non-finite inputs are reported.
__global__ void load_damped_kernel(const float* __restrict__ H, int64_t c, int64_t ldh, const double* __restrict__ scal,
                                   double* __restrict__ A, int64_t cp, lq_dev_status* st) {
    const int64_t i = blockIdx.y;
    const double damp = scal[0];
    // four entries per thread: one 16-byte read where the row of H allows it, two 16-byte writes
    const bool vec = (ldh % 4 == 0) && ((reinterpret_cast<uintptr_t>(H) & 15) == 0);
    for (int64_t j0 = 4 * (blockIdx.x * (int64_t)blockDim.x + threadIdx.x); j0 < cp; j0 += 4 * (int64_t)gridDim.x * blockDim.x) {
        double v[4] = {0.0, 0.0, 0.0, 0.0};
        if (i < c && j0 + 3 >= i && j0 < c) {
            float hv[4] = {0.0f, 0.0f, 0.0f, 0.0f};
            if (vec && j0 + 3 < c) {
                const float4 x = LQ_AT(reinterpret_cast<const float4*>(H + i * ldh + j0));
                hv[0] = x.x; hv[1] = x.y; hv[2] = x.z; hv[3] = x.w;
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (j0 + e < c) hv[e] = LQ_AT(H + i * ldh + j0 + e);
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int64_t j = j0 + e;
                if (j < c && j >= i) {
                    if (!isfinite(hv[e])) lq_report(st, LQ_ERR_NONFINITE, i * c + j);
                    v[e] = static_cast<double>(hv[e]);
                    if (i == j) v[e] = (hv[e] == 0.0f ? 1.0 : v[e]) + damp;
                }
            }
        }
        if (i >= c && i >= j0 && i < j0 + 4) v[i - j0] = 1.0;        // identity on the padding
        double2* out = reinterpret_cast<double2*>(A + i * cp + j0);  // cp is a multiple of 128
        LQ_AT(out) = make_double2(v[0], v[1]);
        LQ_AT(out + 1) = make_double2(v[2], v[3]);
    }
}

// ------------------------------------------------------------------ FP64 MMA -------
__device__ __forceinline__ void dmma(double& c0, double& c1, double a, double b) {
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
                 : "+d"(c0), "+d"(c1) : "d"(a), "d"(b));
}
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
    const uint32_t d = static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst));
    if (!LQ_DBG_OK(gsrc, 16) || !LQ_DBG_OK(smem_dst, 16)) return;       // debug build: a copy outside the registered buffers is skipped
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// Programmatic dependent launch along the serial chain: a kernel launched with launch_chained() may be placed on the
// SMs while its predecessor in the stream still runs; it calls chain_wait() before it touches anything the predecessor
// wrote (the wait returns when the predecessor has completed and its writes are visible).  chain_release() in the
// predecessor says that the successor's CTAs may be placed from now on; without it they are placed when the
// predecessor ends.  In a kernel launched the plain way both are no-ops.
__device__ __forceinline__ void chain_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void chain_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ------------------------------------------------------------ tile product, K = 128 --
// C[TM x TN] = beta * C + alpha * A[TM x 128] * op(B), all fp64 row-major, by 256 threads = 8 warps
// arranged WMW x (8 / WMW); each warp owns an (8 MI) x 32 patch as MI x 4 MMA tiles, so
// TM = 8 MI WMW and TN = 32 (8 / WMW).  NT: B is given as TN rows of K (C = A B^T), otherwise as
// K rows of TN.  K is streamed 16 at a time through a 3-stage cp.async ring; the shared-memory
// pitches make every fragment load conflict-free.  The output may alias B when the tile spans
// all of B's rows and columns that it reads (all of B has been read before the first store).
// Optional extra outputs: a plain copy (C2) and a transposed copy (Ct).
//   <4, 4, *>  128 x 64   the bulk of the updates (two CTAs per SM)
//   <2, 4, *>   64 x 64   panel and "next" tiles: short launches that sit on the critical path
//   <2, 8, *>  128 x 32   row scaling in place (a CTA owns whole columns)
constexpr int TK = 16, NST = 3;
constexpr int AP = 20;                       // pitch (doubles) of a K-major chunk row: 16 + 4
constexpr int GEMM_THREADS = 256;
constexpr int GEMM_SMEM = NST * (128 * AP + TK * (64 + 4)) * 8;     // the largest instantiation

struct TileOut {
    double* C;  int64_t ldc;
    double* C2; int64_t ldc2;     // optional copy of the result
    double* Ct; int64_t ldct;     // optional transposed copy: Ct[col * ldct + row]
};

template <int MI, int WMW, bool NT>
__device__ __forceinline__ void gemm_tile(const double* __restrict__ A, int64_t lda, const double* B, int64_t ldb,
                                          double alpha, double beta, const TileOut& o, double* smem) {
    constexpr int WNW = 8 / WMW;
    constexpr int TMR = 8 * MI * WMW, TNC = 32 * WNW;
    constexpr int BP = TNC + 4;                               // pitch of an N-major chunk row (NN form)
    constexpr int STAGE = TMR * AP + (NT ? TNC * AP : TK * BP);
    static_assert(NST * STAGE * 8 <= GEMM_SMEM, "shared memory");
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int wm = warp / WNW, wn = warp % WNW;
    const int fr = lane >> 2, fk = lane & 3;

    auto issue = [&](int kc) {
        double* as = smem + (kc % NST) * STAGE;
        double* bs = as + TMR * AP;
#pragma unroll
        for (int u = 0; u < TMR * 8 / GEMM_THREADS; ++u) {
            const int idx = tid + GEMM_THREADS * u, row = idx >> 3, seg = idx & 7;
            cp_async16(as + row * AP + seg * 2, A + (int64_t)row * lda + kc * TK + seg * 2);
        }
        if (NT) {
#pragma unroll
            for (int u = 0; u < TNC * 8 / GEMM_THREADS; ++u) {
                const int idx = tid + GEMM_THREADS * u, row = idx >> 3, seg = idx & 7;
                cp_async16(bs + row * AP + seg * 2, B + (int64_t)row * ldb + kc * TK + seg * 2);
            }
        } else {
            constexpr int SEGS = TNC / 2;                     // 16-byte pieces per row
#pragma unroll
            for (int u = 0; u < TK * SEGS / GEMM_THREADS; ++u) {
                const int idx = tid + GEMM_THREADS * u, row = idx / SEGS, seg = idx % SEGS;
                cp_async16(bs + row * BP + seg * 2, B + (int64_t)(kc * TK + row) * ldb + seg * 2);
            }
        }
    };

    double acc[MI][4][2];
#pragma unroll
    for (int i = 0; i < MI; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j][0] = acc[i][j][1] = 0.0;

    constexpr int NCHUNK = NB / TK;
    issue(0); cp_async_commit();
    issue(1); cp_async_commit();
#pragma unroll 1
    for (int kc = 0; kc < NCHUNK; ++kc) {
        cp_async_wait<NST - 2>();
        __syncthreads();
        if (kc + NST - 1 < NCHUNK) issue(kc + NST - 1);
        cp_async_commit();
        const double* as = smem + (kc % NST) * STAGE + (wm * 8 * MI + fr) * AP + fk;
        const double* bs = smem + (kc % NST) * STAGE + TMR * AP + (NT ? (wn * 32 + fr) * AP + fk : fk * BP + wn * 32 + fr);
#pragma unroll
        for (int kk = 0; kk < TK / 4; ++kk) {
            double a[MI], b[4];
#pragma unroll
            for (int i = 0; i < MI; ++i) a[i] = as[8 * i * AP + kk * 4];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = NT ? bs[8 * j * AP + kk * 4] : bs[kk * 4 * BP + 8 * j];
#pragma unroll
            for (int i = 0; i < MI; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) dmma(acc[i][j][0], acc[i][j][1], a[i], b[j]);
        }
    }
    cp_async_wait<0>();
    __syncthreads();      // every thread's copies have landed: B may now be overwritten

#pragma unroll
    for (int i = 0; i < MI; ++i) {
        const int row = wm * 8 * MI + 8 * i + fr;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int col = wn * 32 + 8 * j + 2 * fk;
            double2 v;
            v.x = alpha * acc[i][j][0];
            v.y = alpha * acc[i][j][1];
            double* cp = o.C + (int64_t)row * o.ldc + col;
            if (beta != 0.0) {
                const double2 old = LQ_AT(reinterpret_cast<const double2*>(cp));
                v.x += beta * old.x;
                v.y += beta * old.y;
            }
            LQ_AT(reinterpret_cast<double2*>(cp)) = v;
            if (o.C2) LQ_AT(reinterpret_cast<double2*>(o.C2 + (int64_t)row * o.ldc2 + col)) = v;
            if (o.Ct) {
                LQ_AT(o.Ct + (int64_t)col * o.ldct + row) = v.x;
                LQ_AT(o.Ct + (int64_t)(col + 1) * o.ldct + row) = v.y;
            }
        }
    }
}

// Step k, panel.  Blocks [0, 4k): 64 x 64 tiles of P_i = A[i][k] V_k^T (to Pbuf: this step's 128 columns of the
// outer block's panel buffer, row stride ldp; and transposed into Q's columns of block i).  Blocks [4k, 4(nblk-1)): 128 x 32 tiles of the row scaling
// A[k][j] <- V_k A[k][j] for j > k (in place: these are final entries of U) with a copy in Q's
// columns of block j.  Q is 128 x cp: the right-hand operand of the step's update for every
// block column.
__global__ void __launch_bounds__(GEMM_THREADS, 2)
panel_kernel(double* __restrict__ A, int64_t cp, int k, double* __restrict__ Pbuf, int64_t ldp, double* __restrict__ Q) {
    extern __shared__ double smem[];
    const int t = blockIdx.x >> 2, q = blockIdx.x & 3;
    chain_wait();                                       // launched behind the diagonal kernel of this step
    const double* Vk = A + (int64_t)k * NB * cp + (int64_t)k * NB;
    TileOut o = {};
    if (t < k) {
        const int i = t, mh = q >> 1, h = q & 1;
        o.C = Pbuf + ((int64_t)i * NB + mh * 64) * ldp + h * 64; o.ldc = ldp;
        o.Ct = Q + (int64_t)(h * 64) * cp + (int64_t)i * NB + mh * 64; o.ldct = cp;
        gemm_tile<2, 4, true>(A + ((int64_t)i * NB + mh * 64) * cp + (int64_t)k * NB, cp, Vk + (int64_t)(h * 64) * cp, cp, 1.0,
                              0.0, o, smem);
    } else {
        const int j = t + 1;
        double* row = A + (int64_t)k * NB * cp + (int64_t)j * NB + q * 32;
        o.C = row; o.ldc = cp;
        o.C2 = Q + (int64_t)j * NB + q * 32; o.ldc2 = cp;
        gemm_tile<2, 8, false>(Vk, cp, row, cp, 1.0, 0.0, o, smem);
    }
}

// Step k, eager update of tiles (i, j), i < k: A[i][j] -= P_i Q[:, j] (A[i][k] = -P_i V_k).  A launch covers the
// block rows i_base + blockIdx.y and the block columns j_base + (blockIdx.x >> 1) (128 x 64 tiles).  The tiles of
// block column k-1 and of block row k-1 are all that step k-1's diagonal and panel kernels read, so they can be
// updated first ("next") and the remainder ("rest") left to run beside step k-1.  With a look-ahead of two steps the
// tiles of block row and column k-2 ("next2") leave the rest as well, so that step k-1's "next" update waits for a
// short launch only and the rest of step k has two chain steps to finish:
//   part 0: every tile of the launch;  part 2: all but block row and block column k-1;
//   part 4: all but block rows and block columns k-1 and k-2;
//   part 1: next only, grid 4 nblk x 1, 64 x 64 tiles -- block tile t < k is (t, k-1), t >= k is (k-1, t);
//   part 3: next2 only, same grid -- block tile t < k-1 is (t, k-2), t >= k is (k-2, t) (tile (k-2, k-1) belongs to next);
//   part 5: next without the diagonal tile (k-1, k-1), which crit_kernel has updated already.
__global__ void __launch_bounds__(GEMM_THREADS, 2)
update_kernel(double* __restrict__ A, int64_t cp, int k, int part, int i_base, int j_base, const double* __restrict__ Pbuf,
              int64_t ldp, const double* __restrict__ Q) {
    extern __shared__ double smem[];
    int i, j, r0, c0;
    if (part == 1 || part == 3 || part == 5) {
        const int t = blockIdx.x >> 2;
        const int nx = part == 3 ? k - 2 : k - 1;         // the block row and column this launch brings up to date
        if (part == 3 && t == k - 1) return;
        if (part == 5 && t == k - 1) return;              // the diagonal tile was updated by crit_kernel
        if (t <= nx) { i = t; j = nx; } else { i = nx; j = t; }
        r0 = ((blockIdx.x >> 1) & 1) * 64;
        c0 = (blockIdx.x & 1) * 64;
    } else if (part >= 10) {
        // parts 0 and 2 of the deferred sweep in one launch (part - 10): first the block rows [i_base, k) (part 2:
        // [i_base, k-1)) over the whole width, one grid row each; then the block rows [0, i_base) over the j_base block
        // columns of the outer block, packed into grid rows of the same width
        const int o_lo = i_base, obw = j_base;
        const int nA = k - o_lo - (part == 12 ? 1 : 0);
        if (static_cast<int>(blockIdx.y) < nA) {
            i = o_lo + blockIdx.y;
            j = blockIdx.x >> 1;
            c0 = (blockIdx.x & 1) * 64;
        } else {
            const int64_t lin = static_cast<int64_t>(blockIdx.y - nA) * gridDim.x + blockIdx.x;
            i = static_cast<int>(lin / (2 * obw));
            if (i >= o_lo) return;
            const int xx = static_cast<int>(lin - static_cast<int64_t>(i) * (2 * obw));
            j = o_lo + (xx >> 1);
            c0 = (xx & 1) * 64;
        }
        if (part == 12 && (j == k - 1 || i == k - 1)) return;
        r0 = 0;
    } else {
        j = j_base + (blockIdx.x >> 1);
        i = i_base + blockIdx.y;
        if (part >= 2 && (j == k - 1 || i == k - 1)) return;
        if (part == 4 && (j == k - 2 || i == k - 2)) return;
        r0 = 0;
        c0 = (blockIdx.x & 1) * 64;
    }
    if (j < i) return;                                  // strictly lower tiles of the symmetric part
    if (part == 1) chain_release();                     // the next step's diagonal kernel may take its SM now; it waits for this launch to end
    const double* Pi = Pbuf + ((int64_t)i * NB + r0) * ldp;
    TileOut o = {};
    o.C = A + ((int64_t)i * NB + r0) * cp + (int64_t)j * NB + c0; o.ldc = cp;
    // A[i][k] = -P_i V_k;  A[i][j] -= P_i Q[:, j] otherwise
    const double* Bsrc = (j == k) ? A + (int64_t)k * NB * cp + (int64_t)k * NB + c0 : Q + (int64_t)j * NB + c0;
    const double beta = (j == k) ? 0.0 : 1.0;
    if (part == 1 || part == 3 || part == 5) gemm_tile<2, 4, false>(Pi, ldp, Bsrc, cp, -1.0, beta, o, smem);
    else gemm_tile<4, 4, false>(Pi, ldp, Bsrc, cp, -1.0, beta, o, smem);
}

// Step k, the one tile the next diagonal block waits for.  phase 0: P' = A[k-1][k] V_k^T (the panel tile of block row
// k-1, into the scratch Pc, 128 x 128); phase 1: A[k-1][k-1] -= P' P'^T.  Four CTAs of 64 x 64 each: they find free
// places on the SMs at once, where the panel and "next" launches (over a hundred CTAs) queue behind the bulk update.
// The panel launch computes the same P' again for everybody else.
__global__ void __launch_bounds__(GEMM_THREADS, 2)
crit_kernel(double* __restrict__ A, int64_t cp, int k, int phase, double* __restrict__ Pc) {
    extern __shared__ double smem[];
    chain_wait();
    const int mh = blockIdx.x >> 1, hh = blockIdx.x & 1;
    TileOut o = {};
    if (phase == 0) {
        const double* Vk = A + (int64_t)k * NB * cp + (int64_t)k * NB;
        o.C = Pc + (int64_t)(mh * 64) * NB + hh * 64; o.ldc = NB;
        gemm_tile<2, 4, true>(A + ((int64_t)(k - 1) * NB + mh * 64) * cp + (int64_t)k * NB, cp, Vk + (int64_t)(hh * 64) * cp, cp, 1.0, 0.0, o, smem);
    } else {
        o.C = A + ((int64_t)(k - 1) * NB + mh * 64) * cp + (int64_t)(k - 1) * NB + hh * 64; o.ldc = cp;
        gemm_tile<2, 4, true>(Pc + (int64_t)(mh * 64) * NB, NB, Pc + (int64_t)(hh * 64) * NB, NB, -1.0, 1.0, o, smem);
    }
}

// ------------------------------------------------ deferred update: operands as digit slices ----
// x = 2^e (d_1 2^-8 + d_2 2^-16 + ... + d_S 2^-8S) + remainder, with integer digits |d_s| <= 128 and e such that
// |x| 2^-e <= 1/2 for every entry of the row: slice s holds d_s 2^-8s as bf16 (exact).
constexpr int OBB = 8;                   // block columns per outer block
constexpr int LDP = OBB * NB;            // row stride of the panel buffer and of the slices
constexpr int NSL = 5;                   // slices
constexpr int64_t BAND = 8192;           // rows of the deferred region handled per product

__device__ __forceinline__ int exp_for(double mx) { return mx > 0.0 ? ilogb(mx) + 2 : 0; }

__device__ __forceinline__ void digits_of(double x, int e, __nv_bfloat16 (&d)[NSL]) {
    double rest = scalbn(x, 8 - e);                     // |rest| <= 128
    double w = 0.00390625;                              // 2^-8
#pragma unroll
    for (int s = 0; s < NSL; ++s) {
        const double q = rint(rest);
        d[s] = __float2bfloat16_rn(static_cast<float>(q * w));     // an integer of at most 8 bits times a power of two
        rest = (rest - q) * 256.0;
        w *= 0.00390625;
    }
}
// The same number as signed 8-bit integers for the integer tensor-core path: balanced digits in [-128, 127].  With
// that range the digits after position s can make up anything in [-128/255, 127/255] of position s, so a digit is
// chosen to leave its remainder in that interval: q = floor(rest + 128/255).  (Unsigned lower digits would be simpler,
// but their mean of 127 puts a large common component into every lower level, and the fp32 rounding of that level's
// sum then costs five bits of the result: measured, 1e-7 instead of 4e-8 on U.)
__device__ __forceinline__ void digits_of(double x, int e, uint8_t (&d)[NSL]) {
    double rest = scalbn(x, 8 - e);                     // |rest| <= 127 (exp_for8)
#pragma unroll
    for (int s = 0; s < NSL; ++s) {
        double q = s + 1 < NSL ? floor(rest + 128.0 / 255.0) : rint(rest);
        q = fmin(fmax(q, -128.0), 127.0);
        d[s] = static_cast<uint8_t>(static_cast<int8_t>(static_cast<int>(q)));
        rest = (rest - q) * 256.0;
    }
}
// Exponent for the integer digits: the leading digit must not reach 128.
__device__ __forceinline__ int exp_for8(double mx) {
    if (!(mx > 0.0)) return 0;
    int e = ilogb(mx) + 2;                              // mx 2^(8 - e) < 128
    if (scalbn(mx, 8 - e) > 127.0) ++e;
    return e;
}

// Rows [0, rows) of the panel buffer (K columns each): exponent and slices.  One CTA per row.
template <typename D>
__global__ void __launch_bounds__(256)
slice_rows_kernel(const double* __restrict__ P, int64_t ldp, int K, int* __restrict__ ex, D* __restrict__ SL,
                  int64_t slice_rows) {
    __shared__ double red[8];
    const int64_t row = blockIdx.x;
    const double* p = P + row * ldp;
    double v[4];
    double mx = 0.0;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int kx = threadIdx.x + 256 * u;
        v[u] = kx < K ? LQ_AT(p + kx) : 0.0;
        mx = fmax(mx, fabs(v[u]));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = mx;
    __syncthreads();
    mx = red[0];
#pragma unroll
    for (int w = 1; w < 8; ++w) mx = fmax(mx, red[w]);
    const int e = isfinite(mx) ? (sizeof(D) == 1 ? exp_for8(mx) : exp_for(mx)) : 0;
    if (threadIdx.x == 0) LQ_AT(ex + row) = e;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int kx = threadIdx.x + 256 * u;
        if (kx >= K) continue;
        D d[NSL];
        digits_of(isfinite(v[u]) ? v[u] : 0.0, e, d);
#pragma unroll
        for (int s = 0; s < NSL; ++s) LQ_AT(SL + (s * slice_rows + row) * LDP + kx) = d[s];
    }
}

// Exponents of the columns j >= col0 of the K rows of A that start at row0 (the final rows of U of an outer block).
__global__ void __launch_bounds__(256)
col_exp_kernel(const double* __restrict__ A, int64_t cp, int64_t row0, int K, int64_t col0, int* __restrict__ ex, int int8) {
    // 32 columns per CTA, eight threads per column (each takes every eighth row), so that a column's K loads do not queue
    // behind one another in one thread
    __shared__ double part[8][32];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int64_t j = col0 + blockIdx.x * 32LL + tx;
    double mx = 0.0;
    if (j < cp)
        for (int kx = ty; kx < K; kx += 8) mx = fmax(mx, fabs(LQ_AT(A + (row0 + kx) * cp + j)));
    part[ty][tx] = mx;
    __syncthreads();
    if (ty == 0 && j < cp) {
#pragma unroll
        for (int q = 1; q < 8; ++q) mx = fmax(mx, part[q][tx]);
        LQ_AT(ex + j) = isfinite(mx) ? (int8 ? exp_for8(mx) : exp_for(mx)) : 0;
    }
}

// Slices of those columns, transposed: SL[s][j][kx] = digit s of A[row0 + kx][j].  64 x 64 tiles through shared memory.
template <typename D>
__global__ void __launch_bounds__(256)
slice_cols_kernel(const double* __restrict__ A, int64_t cp, int64_t row0, int K, int64_t col0, const int* __restrict__ ex,
                  D* __restrict__ SL, int64_t slice_rows) {
    __shared__ double tile[64][65];
    const int64_t j0 = col0 + (int64_t)blockIdx.x * 64;
    const int k0 = blockIdx.y * 64;
    for (int idx = threadIdx.x; idx < 64 * 64; idx += 256) {
        const int a = idx >> 6, b = idx & 63;            // row k0 + a, column j0 + b
        const int64_t j = j0 + b;
        tile[a][b] = (k0 + a < K && j < cp) ? LQ_AT(A + (row0 + k0 + a) * cp + j) : 0.0;
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < 64 * 64; idx += 256) {
        const int b = idx >> 6, a = idx & 63;            // output row j0 + b, position k0 + a
        const int64_t j = j0 + b;
        if (j >= cp || k0 + a >= K) continue;
        const double x = tile[a][b];
        D d[NSL];
        digits_of(isfinite(x) ? x : 0.0, LQ_AT(ex + j), d);
#pragma unroll
        for (int s = 0; s < NSL; ++s) LQ_AT(SL + (s * slice_rows + j) * LDP + k0 + a) = d[s];
    }
}

// A[row0 + i][col0 + j] -= 2^(ex[row0 + i] + ex[col0 + j]) (Ta[i][col0 + j] + Tb[i][col0 + j]) over nrows x ncols entries;
// with `upper`, only the 128 x 128 blocks on or above the diagonal.  Two columns per thread.
__global__ void __launch_bounds__(256)
apply_kernel(double* __restrict__ A, int64_t cp, const float* __restrict__ Ta, const float* __restrict__ Tb, int64_t ldt,
             const int* __restrict__ ex, int64_t row0, int64_t nrows, int64_t col0, int64_t ncols, int upper) {
    const int64_t i = blockIdx.y;
    const int64_t row = row0 + i;
    const int er = LQ_AT(ex + row);
    for (int64_t j2 = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; 2 * j2 < ncols; j2 += (int64_t)gridDim.x * blockDim.x) {
        const int64_t col = col0 + 2 * j2;
        if (upper && col / NB < row / NB) continue;
        const float2 a = LQ_AT(reinterpret_cast<const float2*>(Ta + i * ldt + col));
        const float2 b = LQ_AT(reinterpret_cast<const float2*>(Tb + i * ldt + col));
        double2* ap = reinterpret_cast<double2*>(A + row * cp + col);
        double2 v = LQ_AT(ap);
        v.x -= scalbn(static_cast<double>(a.x) + static_cast<double>(b.x), er + LQ_AT(ex + col));
        v.y -= scalbn(static_cast<double>(a.y) + static_cast<double>(b.y), er + LQ_AT(ex + col + 1));
        LQ_AT(ap) = v;
    }
}

// --------------------------------------------------------- diagonal block kernel ----
// In place on the 128 x 128 diagonal block k of A: reads its upper triangle (symmetric positive
// definite), computes the upper R with block = R R^T and writes V = R^-1 (upper, zeros below)
// back.  One CTA of 256 threads.  The block is handled as 4 x 4 sub-blocks of
// 32 with the same sweep as the outer algorithm: warp 0 factorises and inverts a 32 x 32
// diagonal sub-block in registers (one row per lane), then all warps do the panel, update and
// scaling products with the FP64 MMA out of shared memory.
constexpr int SB = 32;
constexpr int DP = 132;          // pitch of the block in shared memory (conflict-free fragments)
constexpr int PP = 36;           // pitch of the panel buffer
constexpr int DIAG_THREADS = 256;
constexpr int DIAG_SMEM = (NB * DP + (NB - SB) * PP + 2 * SB + SB) * 8;

// 32 x 32 sub-block at S (pitch DP): upper triangle in, V = R^-1 out (upper, zeros below).
__device__ __forceinline__ void warp_factor_invert(double* S, double* colbuf, double* rinvb, int lane,
                                                   long long col_global, long long c_real, lq_dev_status* st) {
    double a[SB];
#pragma unroll
    for (int t = 0; t < SB; ++t) a[t] = (t >= lane) ? S[lane * DP + t] : 0.0;
    // R R^T factorisation, last column first; lane i holds row i.  The pivots form the one serial chain of the whole
    // stage: the entry that becomes the next pivot is updated and broadcast first, the other columns' updates follow
    // and fill the latency of that broadcast and of the next reciprocal square root.
    double d = __shfl_sync(0xffffffffu, a[SB - 1], SB - 1);
#pragma unroll
    for (int j = SB - 1; j >= 0; --j) {
        if (!(d > 0.0) || !isfinite(d)) {
            if (lane == 0 && col_global + j < c_real) lq_report(st, LQ_ERR_NOT_POSITIVE_DEFINITE, col_global + j);
            d = 1.0;
        }
        const double rinv = rsqrt(d);
        const double l = (lane < j) ? a[j] * rinv : ((lane == j) ? d * rinv : 0.0);   // R[i][j]; sqrt(d) on the diagonal
        a[j] = l;
        if (lane == j) rinvb[j] = rinv;
        double* cb = colbuf + (j & 1) * SB;
        cb[lane] = (lane < j) ? l : 0.0;
        __syncwarp();
        if (j > 0) {
            a[j - 1] = fma(-l, cb[j - 1], a[j - 1]);
            d = __shfl_sync(0xffffffffu, a[j - 1], j - 1);
        }
#pragma unroll
        for (int t = 0; t < j - 1; ++t) a[t] -= l * cb[t];            // meaningful for lane <= t
    }
    // R to shared memory (rows), then V = R^-1, lane i forming row i column by column.  Every finished entry V[i][t] is
    // pushed at once into the right-hand sides of all later columns (independent multiply-adds), so between one entry
    // and the next there is one multiply-add and the scaling -- fp64 operations take ~23 cycles each here, and summing
    // a column's terms only when its turn comes puts several of them in series.
#pragma unroll
    for (int t = 0; t < SB; ++t) S[lane * DP + t] = (t >= lane) ? a[t] : 0.0;
    __syncwarp();
    double v[SB];
#pragma unroll
    for (int j = 0; j < SB; ++j) v[j] = (lane == j) ? 1.0 : 0.0;          // right-hand sides, turned into V in place
#pragma unroll
    for (int t = 0; t < SB; ++t) {
        const double vt = (lane <= t) ? v[t] * rinvb[t] : 0.0;
        v[t] = vt;
#pragma unroll
        for (int j = t + 1; j < SB; ++j) v[j] = fma(-vt, S[t * DP + j], v[j]);
    }
    __syncwarp();
#pragma unroll
    for (int t = 0; t < SB; ++t) S[lane * DP + t] = v[t];
}

// 16 x 16 output patch, K = 32, out of shared memory.  a(r, t): left operand, row r of the patch;
// B is given either as rows of K (NT: Bt[n * ldb + t]) or as K rows (NN: Bn[t * ldb + n]).
template <bool NT>
__device__ __forceinline__ void patch16(const double* Ap, int lda, const double* Bp, int ldb, int lane, double (&acc)[2][2][2]) {
    const int fr = lane >> 2, fk = lane & 3;
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int j = 0; j < 2; ++j) acc[i][j][0] = acc[i][j][1] = 0.0;
#pragma unroll
    for (int kk = 0; kk < SB / 4; ++kk) {
        double a[2], b[2];
#pragma unroll
        for (int i = 0; i < 2; ++i) a[i] = Ap[(8 * i + fr) * lda + kk * 4 + fk];
#pragma unroll
        for (int j = 0; j < 2; ++j) b[j] = NT ? Bp[(8 * j + fr) * ldb + kk * 4 + fk] : Bp[(kk * 4 + fk) * ldb + 8 * j + fr];
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
            for (int j = 0; j < 2; ++j) dmma(acc[i][j][0], acc[i][j][1], a[i], b[j]);
    }
}

__global__ void __launch_bounds__(DIAG_THREADS, 1)
diag_block_kernel(double* __restrict__ A, int64_t cp, int64_t blk, int64_t c_real, lq_dev_status* st) {
    extern __shared__ double sm[];
    double* S = sm;                       // NB x DP
    double* Pb = S + NB * DP;             // (NB - SB) x PP
    double* colbuf = Pb + (NB - SB) * PP; // 2 x SB
    double* rinvb = colbuf + 2 * SB;      // SB
    double* base = A + blk * NB * cp + blk * NB;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int fr = lane >> 2, fk = lane & 3;
    constexpr int NW = DIAG_THREADS / 32;

    chain_wait();                                       // launched behind the previous step's "next" update
    for (int idx = tid; idx < NB * (NB / 2); idx += DIAG_THREADS) {
        const int row = idx >> 6, c2 = (idx & 63) * 2;
        cp_async16(S + row * DP + c2, base + (int64_t)row * cp + c2);
    }
    cp_async_commit();
    cp_async_wait<0>();
    __syncthreads();

#pragma unroll 1
    for (int kb = NB / SB - 1; kb >= 0; --kb) {
        const int c0 = kb * SB;
        const int right = NB - c0 - SB;               // columns to the right of this sub-block
        double* D = S + c0 * DP + c0;                 // diagonal sub-block
        if (warp == 0) warp_factor_invert(D, colbuf, rinvb, lane, blk * NB + c0, c_real, st);
        __syncthreads();
        // panel: Pb[m][q] = sum_t S[m][c0 + t] V[q][t]   (m < c0); row scaling: S[c0 + q][j] <- sum_t V[q][t] S[c0 + t][j]  (j > c0 + 32)
        {
            const int nP = (c0 / 16) * 2;
            const int nR = right / 8;
            for (int item = warp; item < nP + nR; item += NW) {
                if (item < nP) {
                    const int m0 = (item >> 1) * 16, q0 = (item & 1) * 16;
                    double acc[2][2][2];
                    patch16<true>(S + m0 * DP + c0, DP, D + q0 * DP, DP, lane, acc);
#pragma unroll
                    for (int i = 0; i < 2; ++i)
#pragma unroll
                        for (int j = 0; j < 2; ++j) {
                            double* p = Pb + (m0 + 8 * i + fr) * PP + q0 + 8 * j + 2 * fk;
                            p[0] = acc[i][j][0];
                            p[1] = acc[i][j][1];
                        }
                } else {
                    // one warp owns an 8-column strip over all 32 rows, so the in-place update is safe
                    const int j0 = c0 + SB + (item - nP) * 8;
                    double acc[4][2];
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[i][0] = acc[i][1] = 0.0;
#pragma unroll
                    for (int kk = 0; kk < SB / 4; ++kk) {
                        const double b = S[(c0 + kk * 4 + fk) * DP + j0 + fr];
#pragma unroll
                        for (int i = 0; i < 4; ++i) dmma(acc[i][0], acc[i][1], D[(8 * i + fr) * DP + kk * 4 + fk], b);
                    }
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        double* p = S + (c0 + 8 * i + fr) * DP + j0 + 2 * fk;
                        p[0] = acc[i][0];
                        p[1] = acc[i][1];
                    }
                }
            }
        }
        __syncthreads();
        // update of the rows above: 16 x 16 patches over the whole width
        {
            const int nRow = c0 / 16;
            for (int item = warp; item < nRow * 8; item += NW) {
                const int rg = item >> 3, cg = item & 7;
                const int m0 = rg * 16, n0 = cg * 16;
                double acc[2][2][2];
                double sign_old;
                if (n0 < c0) {
                    if (cg < rg) continue;                                   // symmetric part: upper patches only
                    patch16<true>(Pb + m0 * PP, PP, Pb + n0 * PP, PP, lane, acc);          // P_m P_n^T
                    sign_old = 1.0;
                } else if (n0 < c0 + SB) {
                    patch16<false>(Pb + m0 * PP, PP, D + (n0 - c0), DP, lane, acc);        // P_m V
                    sign_old = 0.0;
                } else {
                    patch16<false>(Pb + m0 * PP, PP, S + c0 * DP + n0, DP, lane, acc);     // P_m (scaled row)
                    sign_old = 1.0;
                }
#pragma unroll
                for (int i = 0; i < 2; ++i)
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        double* p = S + (m0 + 8 * i + fr) * DP + n0 + 8 * j + 2 * fk;
                        p[0] = sign_old * p[0] - acc[i][j][0];
                        p[1] = sign_old * p[1] - acc[i][j][1];
                    }
            }
        }
        __syncthreads();
    }

    chain_release();                                    // the panel kernel's CTAs may be placed while the block is written back
    for (int idx = tid; idx < NB * (NB / 2); idx += DIAG_THREADS) {
        const int row = idx >> 6, c2 = (idx & 63) * 2;
        double2 v;
        v.x = (c2 >= row) ? S[row * DP + c2] : 0.0;
        v.y = (c2 + 1 >= row) ? S[row * DP + c2 + 1] : 0.0;
        LQ_AT(reinterpret_cast<double2*>(base + (int64_t)row * cp + c2)) = v;
    }
}

// U (fp32, c x c, upper, zeros below) and dinv[j] = sum_k U64[k][j]^2.  A CTA converts 256 rows of 32
// columns and leaves the sum of squares of its piece of every column in part[row chunk][column];
// dinv_kernel adds the pieces of a column in row order (a fixed order: the result is reproducible).
constexpr int FIN_ROWS = 256;
__global__ void __launch_bounds__(256)
finalize_kernel(const double* __restrict__ A, int64_t cp, int64_t c, float* __restrict__ U, int64_t ldu,
                double* __restrict__ part) {
    __shared__ double red[8][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int64_t j = (int64_t)blockIdx.x * 32 + tx;
    const int64_t i0 = (int64_t)blockIdx.y * FIN_ROWS;
    const int64_t i1 = i0 + FIN_ROWS < c ? i0 + FIN_ROWS : c;
    double s = 0.0;
    if (j < c) {
        for (int64_t i = i0 + ty; i < i1; i += 8) {
            double u = 0.0;
            if (i <= j) {
                u = LQ_AT(A + i * cp + j);
                s = fma(u, u, s);
            }
            LQ_AT(U + i * ldu + j) = static_cast<float>(u);
        }
    }
    red[ty][tx] = s;
    __syncthreads();
    if (ty == 0 && j < c) {
        double t = 0.0;
#pragma unroll
        for (int w = 0; w < 8; ++w) t += red[w][tx];
        LQ_AT(part + (int64_t)blockIdx.y * c + j) = t;
    }
}
__global__ void dinv_kernel(const double* __restrict__ part, int64_t c, int n_chunks, float* __restrict__ dinv) {
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= c) return;
    double t = 0.0;
    for (int q = 0; q * (int64_t)FIN_ROWS <= j && q < n_chunks; ++q) t += LQ_AT(part + (int64_t)q * c + j);
    LQ_AT(dinv + j) = static_cast<float>(t);
}

// Launches a kernel of the chain so that it may be placed before its predecessor in the stream has ended (the kernel
// itself waits with chain_wait()).
template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

struct PrepLayout {
    int64_t nblk, cp, band;
    size_t scal, a, pbuf, q, ex, sl, ta, tb, total, panel_bytes;
};
PrepLayout prep_layout(int64_t c) {
    PrepLayout L;
    L.nblk = lq_ceil_div(c, NB);
    L.cp = L.nblk * NB;
    L.band = L.cp < BAND ? L.cp : BAND;
    size_t off = 0;
    L.scal = off; off += 256;
    L.a = off;    off += lq_align_up(static_cast<size_t>(L.cp) * L.cp * sizeof(double), 256);
    L.panel_bytes = lq_align_up(static_cast<size_t>(L.cp) * NB * sizeof(double), 256);
    L.pbuf = off; off += lq_align_up(static_cast<size_t>(L.cp) * LDP * sizeof(double), 256);   // the panels of one outer block
    L.q = off;    off += 4 * L.panel_bytes;            // Q of the last four steps: with a look-ahead of two steps the rest of step k+2's update may still read its Q while step k's is written
    L.ex = off;   off += lq_align_up(static_cast<size_t>(L.cp) * sizeof(int), 256);
    L.sl = off;   off += lq_align_up(static_cast<size_t>(NSL) * L.cp * LDP * sizeof(__nv_bfloat16), 256);
    L.ta = off;   off += lq_align_up(static_cast<size_t>(L.band) * L.cp * sizeof(float), 256);
    L.tb = off;   off += lq_align_up(static_cast<size_t>(L.band) * L.cp * sizeof(float), 256);
    L.total = off;
    return L;
}

// The updates that the steps of outer block [o_lo, o_hi] owe to the tiles outside its rows and columns:
//   A[i][j] -= sum_k P_i^(k) Q_j^(k)    for block rows i < o_lo and block columns j outside the outer block, j >= i,
// with Q_j^(k) = P_j^(k)^T left of the outer block (the Cholesky part) and the final row k of U right of it (the
// Gauss-Jordan part).  Both operands go through the digit slices; row bands of at most `band` rows at a time.
int deferred_update(lq_handle* h, cudaStream_t st, double* A, int64_t cp, int64_t o_lo, int64_t o_hi, const double* Pob, int* ex,
                    void* SL, float* Ta, float* Tb, int64_t band) {
    const int K = static_cast<int>((o_hi - o_lo + 1) * NB);
    const int64_t top = o_lo * NB;                     // rows [0, top) are updated
    const int64_t right0 = (o_hi + 1) * NB;            // columns [right0, cp) on the right of the outer block
    const int64_t n_right = cp - right0;
    // digits as 8-bit integers for tcgen05 kind::i8 (twice the rate of the bf16 form), or as bf16 values
    const bool i8 = h->prep_slices_int8 != 0;
    if (i8) slice_rows_kernel<uint8_t><<<static_cast<unsigned>(top), 256, 0, st>>>(Pob, LDP, K, ex, static_cast<uint8_t*>(SL), cp);
    else slice_rows_kernel<__nv_bfloat16><<<static_cast<unsigned>(top), 256, 0, st>>>(Pob, LDP, K, ex, static_cast<__nv_bfloat16*>(SL), cp);
    LQ_LAUNCH_CHECK();
    if (n_right > 0) {
        col_exp_kernel<<<static_cast<unsigned>(lq_ceil_div(n_right, 32)), 256, 0, st>>>(A, cp, top, K, right0, ex, i8 ? 1 : 0);
        LQ_LAUNCH_CHECK();
        dim3 g(static_cast<unsigned>(lq_ceil_div(n_right, 64)), static_cast<unsigned>(lq_ceil_div(K, 64)));
        if (i8) slice_cols_kernel<uint8_t><<<g, 256, 0, st>>>(A, cp, top, K, right0, ex, static_cast<uint8_t*>(SL), cp);
        else slice_cols_kernel<__nv_bfloat16><<<g, 256, 0, st>>>(A, cp, top, K, right0, ex, static_cast<__nv_bfloat16*>(SL), cp);
        LQ_LAUNCH_CHECK();
    }
    // passes: the leading pair alone (exact), then the pairs of levels s + t = NSL + 1 down to 3, least significant first
    lq_tc_gemm_args lead = {};
    lead.A_all = lead.B_all = SL;
    lead.a_rows = lead.b_rows = static_cast<int64_t>(NSL) * cp;
    lead.lda = lead.ldb = LDP;
    lead.ldd = cp;
    lead.K = K;
    lead.alpha = 1.0f;
    lead.n_pass = 1;
    lead.seg_iters = i8 ? 0 : 4;                       // bf16: 256 digit products per partial sum, far below 2^24; integers: the
                                                       // whole inner dimension in int32, at most 1024 x 2^14 = 2^24, exact in fp32 too
    lead.int8_ops = i8 ? 1 : 0;
    lead.a_signed[0] = lead.b_signed[0] = 1;           // all digits are signed
    lead.lvl_scale[0] = 1.0f / 65536.0f;               // 2^-8 2^-8 (the bf16 digits carry their power of two themselves)
    lq_tc_gemm_args tail = lead;
    tail.seg_iters = 0;
    tail.n_pass = 0;
    tail.n_lvl = 0;
    // bf16 digits: 128 of the inner dimension per segment, at most 5 x 128 x 2^14 < 2^24 per partial sum, which the fp32
    // accumulator holds exactly.  Integer digits: the int32 accumulator holds a level's sum over the whole inner
    // dimension exactly (5 x 1024 x 2^14 < 2^27), so a level is one segment; its conversion to fp32 rounds at 2^-24 of
    // a level that lies 2^-8 or more below the leading one.
    tail.chunk_kb = i8 ? 8 : 2;
    int pair_s[LQ_TC_MAX_PASS], pair_t[LQ_TC_MAX_PASS];
    for (int lvl = NSL + 1; lvl >= 3; --lvl) {
        int cnt = 0;
        for (int sdig = 1; sdig <= NSL; ++sdig) {
            const int tdig = lvl - sdig;
            if (tdig < 1 || tdig > NSL) continue;
            pair_s[tail.n_pass] = sdig - 1;
            pair_t[tail.n_pass] = tdig - 1;
            tail.a_signed[tail.n_pass] = tail.b_signed[tail.n_pass] = 1;
            ++tail.n_pass;
            ++cnt;
        }
        tail.lvl_scale[tail.n_lvl] = static_cast<float>(ldexp(1.0, -8 * lvl));
        tail.lvl_npass[tail.n_lvl++] = cnt;
    }
    for (int64_t b0 = 0; b0 < top; b0 += band) {
        const int64_t b1 = b0 + band < top ? b0 + band : top;
        for (int side = 0; side < 2; ++side) {
            // side 0: columns [b0, top) with the tiles below the diagonal left out; side 1: columns [right0, cp)
            const int64_t col0 = side == 0 ? b0 : right0;
            const int64_t ncols = side == 0 ? top - b0 : n_right;
            if (ncols <= 0) continue;
            if (i8) {
                // integer digits: one launch, the leading pair as its first level with an output of its own
                lq_tc_gemm_args g = tail;
                for (int ps = tail.n_pass; ps > 0; --ps) {
                    g.a_signed[ps] = tail.a_signed[ps - 1]; g.b_signed[ps] = tail.b_signed[ps - 1];
                    g.a_row_off[ps] = pair_s[ps - 1] * cp + b0;
                    g.b_row_off[ps] = pair_t[ps - 1] * cp + col0;
                }
                g.a_signed[0] = g.b_signed[0] = 1;
                g.a_row_off[0] = b0;
                g.b_row_off[0] = col0;
                g.n_pass = tail.n_pass + 1;
                for (int l = tail.n_lvl; l > 0; --l) { g.lvl_npass[l] = tail.lvl_npass[l - 1]; g.lvl_scale[l] = tail.lvl_scale[l - 1]; }
                g.lvl_npass[0] = 1;
                g.lvl_scale[0] = lead.lvl_scale[0];
                g.n_lvl = tail.n_lvl + 1;
                g.D_first = Ta + col0;
                g.D = Tb + col0;
                g.M = b1 - b0;
                g.N = ncols;
                g.upper_only = side == 0 ? 1 : 0;
                int rc = lq_tc_gemm(h, st, g);
                if (rc) return rc;
            } else
            for (int which = 0; which < 2; ++which) {
                lq_tc_gemm_args g = which == 0 ? lead : tail;
                g.D = (which == 0 ? Ta : Tb) + col0;
                g.M = b1 - b0;
                g.N = ncols;
                g.upper_only = side == 0 ? 1 : 0;
                for (int ps = 0; ps < g.n_pass; ++ps) {
                    const int sd = which == 0 ? 0 : pair_s[ps], td = which == 0 ? 0 : pair_t[ps];
                    g.a_row_off[ps] = sd * cp + b0;
                    g.b_row_off[ps] = td * cp + col0;
                }
                int rc = lq_tc_gemm(h, st, g);
                if (rc) return rc;
            }
            const unsigned gx = static_cast<unsigned>(lq_ceil_div(ncols / 2, 256) < 256 ? lq_ceil_div(ncols / 2, 256) : 256);
            apply_kernel<<<dim3(gx, static_cast<unsigned>(b1 - b0)), 256, 0, st>>>(A, cp, Ta, Tb, cp, ex, b0, b1 - b0, col0, ncols,
                                                                                 side == 0 ? 1 : 0);
            LQ_LAUNCH_CHECK();
        }
    }
    return LQ_OK;
}

}  // namespace

extern "C" int lq_prepare_hinv_workspace(int64_t c, size_t* bytes) {
    if (!bytes || c <= 0) return LQ_ERR_INVALID_ARG;
    *bytes = prep_layout(c).total;
    return LQ_OK;
}

extern "C" int lq_prepare_hinv(lq_handle* h, void* stream, const float* H, int64_t c, int64_t ldh, float damp_frac,
                               float* U, int64_t ldu, float* dinv, void* W, int32_t w_dtype, int64_t r, int64_t ldw,
                               void* ws, size_t ws_bytes) {
    if (!h || !H || !U || !dinv || c <= 0 || ldh < c || ldu < c || !(damp_frac >= 0.0f)) return LQ_ERR_INVALID_ARG;
    if (W && (r <= 0 || ldw < c || (w_dtype != LQ_F32 && w_dtype != LQ_BF16))) return LQ_ERR_INVALID_ARG;
    const PrepLayout L = prep_layout(c);
    if (!ws || ws_bytes < L.total) return LQ_ERR_WORKSPACE_TOO_SMALL;
    if (reinterpret_cast<uintptr_t>(ws) & 255) return LQ_ERR_INVALID_ARG;
    if (L.nblk > 32767 || L.cp > 65535) return LQ_ERR_UNSUPPORTED;   // grid.y of the set-up and update launches; room for the column sums
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    const int64_t nblk = L.nblk, cp = L.cp;
    char* wsp = static_cast<char*>(ws);
    double* scal = reinterpret_cast<double*>(wsp + L.scal);
    double* A = reinterpret_cast<double*>(wsp + L.a);

    {
        LQ_DBG_SCOPE(h, st);
        LQ_DBG_REG(H, (static_cast<size_t>(c - 1) * ldh + c) * sizeof(float));
        LQ_DBG_REG(U, (static_cast<size_t>(c - 1) * ldu + c) * sizeof(float));
        LQ_DBG_REG(dinv, static_cast<size_t>(c) * sizeof(float));
        if (W) LQ_DBG_REG(W, (static_cast<size_t>(r - 1) * ldw + c) * (w_dtype == LQ_F32 ? 4 : 2));
        LQ_DBG_REG(ws, L.total);
        LQ_DBG_COMMIT();
    }
    static lq_once_per_device attr_set;
    if (attr_set.first()) {
        LQ_CUDA_TRY(cudaFuncSetAttribute(diag_block_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, DIAG_SMEM));
        LQ_CUDA_TRY(cudaFuncSetAttribute(panel_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM));
        LQ_CUDA_TRY(cudaFuncSetAttribute(update_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM));
        LQ_CUDA_TRY(cudaFuncSetAttribute(crit_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM));
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
        dim3 g(static_cast<unsigned>(lq_ceil_div(cp, 1024) < 32 ? lq_ceil_div(cp, 1024) : 32), static_cast<unsigned>(cp));
        load_damped_kernel<<<g, 256, 0, st>>>(H, c, ldh, scal, A, cp, h->dstatus);
        LQ_LAUNCH_CHECK();
    }

    // The sweep, outer block by outer block (last first).  Inside an outer block every step updates the rows and the
    // columns of the outer block at once (the "eager" tiles).  With an auxiliary stream, step k's diagonal and panel
    // kernels and the "next" part of its update stay on the caller's stream; the rest of the eager update goes to
    // the auxiliary stream and overlaps step k-1's diagonal and panel kernels.  When the outer block is complete,
    // all other tiles get its steps' updates in one product on the bf16 tensor cores (deferred_update).
    cudaStream_t aux = h->aux;
    const bool fork = aux != nullptr && nblk > 2;
    // With the fork the sweep leaves the caller's stream: the chain goes to the handle's high-priority stream `cs`, the
    // bulk of the eager updates to the low-priority `aux`; the caller's stream joins again after the last step.
    cudaStream_t cs = fork ? h->chain : st;
    if (fork) {
        LQ_CUDA_TRY(cudaEventRecord(h->ev_fork, st));
        LQ_CUDA_TRY(cudaStreamWaitEvent(aux, h->ev_fork, 0));
        LQ_CUDA_TRY(cudaStreamWaitEvent(cs, h->ev_fork, 0));
    }
    double* Pob = reinterpret_cast<double*>(wsp + L.pbuf);
    // Small matrices are bound by the serial chain of diagonal blocks, not by the updates: they stay on the FP64 MMA
    // throughout (one outer block as wide as the matrix).
    const bool defer = nblk > OBB && nblk >= h->prep_defer_min_blocks;
    const int64_t obb = defer ? OBB : nblk;
    if (defer) LQ_CUDA_TRY(cudaMemsetAsync(wsp + L.sl, 0, static_cast<size_t>(NSL) * cp * LDP * sizeof(__nv_bfloat16), cs));
    bool rest_pending = false, next2_pending = false;
    const bool deep = fork && !defer && h->mid != nullptr;
    const int64_t n_ob = lq_ceil_div(nblk, obb);
    if (deep) {
        // Nothing deferred (o_lo = 0): look-ahead of two steps, and only what the next diagonal block waits for on the chain.
        //   chain (highest priority): diagonal kernel of step k, then crit_kernel: the panel tile of block row k-1 and the
        //                             update of tile (k-1, k-1) -- the next diagonal block;
        //   middle stream           : panel of step k (after the diagonal kernel), "next" (block row and column k-1 but for
        //                             its diagonal tile; after crit_kernel, which read the tile (k-1, k) that "next"
        //                             overwrites), "next2" (block row and column k-2; after the rest of step k+1);
        //   low-priority stream     : the rest of step k (after the panel of step k and, in stream order, the rest of step k+1).
        // crit_kernel of step k waits for "next2" of step k+1 (and with it for "next" of step k+1 and the rest of step
        // k+2), which wrote the tiles it reads and updates.
        cudaStream_t mid = h->mid;
        LQ_CUDA_TRY(cudaStreamWaitEvent(mid, h->ev_fork, 0));
        double* Pc = reinterpret_cast<double*>(wsp + L.sl);          // 128 x 128 scratch of crit_kernel (the slices' space is free here)
        for (int64_t k = nblk - 1; k >= 0; --k) {
            double* Pk = Pob + (k & 3) * NB;
            double* Qk = reinterpret_cast<double*>(wsp + L.q + (k & 3) * L.panel_bytes);
            const int ki = static_cast<int>(k);
            LQ_CUDA_TRY(launch_chained(diag_block_kernel, dim3(1), dim3(DIAG_THREADS), DIAG_SMEM, cs, A, cp, k, c, h->dstatus));
            LQ_CUDA_TRY(cudaEventRecord(h->ev_diag, cs));
            if (k > 0) {
                if (next2_pending) LQ_CUDA_TRY(cudaStreamWaitEvent(cs, h->ev_next2, 0));
                next2_pending = false;
                crit_kernel<<<4, GEMM_THREADS, GEMM_SMEM, cs>>>(A, cp, ki, 0, Pc);
                LQ_LAUNCH_CHECK();
                LQ_CUDA_TRY(launch_chained(crit_kernel, dim3(4), dim3(GEMM_THREADS), GEMM_SMEM, cs, A, cp, ki, 1, Pc));
                LQ_CUDA_TRY(cudaEventRecord(h->ev_crit, cs));
            }
            LQ_CUDA_TRY(cudaStreamWaitEvent(mid, h->ev_diag, 0));
            panel_kernel<<<static_cast<unsigned>(4 * (nblk - 1)), GEMM_THREADS, GEMM_SMEM, mid>>>(A, cp, ki, Pk, LDP, Qk);
            LQ_LAUNCH_CHECK();
            if (k == 0) {
                LQ_CUDA_TRY(cudaEventRecord(h->ev_next2, mid));
                next2_pending = true;
                break;
            }
            if (k >= 3) LQ_CUDA_TRY(cudaEventRecord(h->ev_next, mid));       // the panel of step k is complete
            LQ_CUDA_TRY(cudaStreamWaitEvent(mid, h->ev_crit, 0));
            update_kernel<<<static_cast<unsigned>(4 * nblk), GEMM_THREADS, GEMM_SMEM, mid>>>(A, cp, ki, 5, 0, 0, Pk, LDP, Qk);
            LQ_LAUNCH_CHECK();
            if (k >= 2) {
                if (rest_pending) LQ_CUDA_TRY(cudaStreamWaitEvent(mid, h->ev_rest, 0));
                update_kernel<<<static_cast<unsigned>(4 * nblk), GEMM_THREADS, GEMM_SMEM, mid>>>(A, cp, ki, 3, 0, 0, Pk, LDP, Qk);
                LQ_LAUNCH_CHECK();
            }
            LQ_CUDA_TRY(cudaEventRecord(h->ev_next2, mid));
            next2_pending = true;
            if (k >= 3) {
                LQ_CUDA_TRY(cudaStreamWaitEvent(aux, h->ev_next, 0));
                dim3 g(static_cast<unsigned>(2 * nblk), static_cast<unsigned>(k - 2));
                update_kernel<<<g, GEMM_THREADS, GEMM_SMEM, aux>>>(A, cp, ki, 4, 0, 0, Pk, LDP, Qk);
                LQ_LAUNCH_CHECK();
                LQ_CUDA_TRY(cudaEventRecord(h->ev_rest, aux));
                rest_pending = true;
            }
        }
    } else
    for (int64_t m = n_ob - 1; m >= 0; --m) {
        const int64_t o_lo = m * obb;
        const int64_t o_hi = (o_lo + obb < nblk ? o_lo + obb : nblk) - 1;
        const int obw = static_cast<int>(o_hi - o_lo + 1);
        for (int64_t k = o_hi; k >= o_lo; --k) {
            // this step's 128 columns of the panel buffer: its place in the outer block, or one of four alternating
            // slots when nothing is deferred (the updates of the two steps before may still be reading theirs)
            double* Pk = Pob + (defer ? k - o_lo : (k & 3)) * NB;
            double* Qk = reinterpret_cast<double*>(wsp + L.q + (k & 3) * L.panel_bytes);
            const int ki = static_cast<int>(k);
            LQ_CUDA_TRY(launch_chained(diag_block_kernel, dim3(1), dim3(DIAG_THREADS), DIAG_SMEM, cs, A, cp, k, c, h->dstatus));
            if (nblk > 1) {
                LQ_CUDA_TRY(launch_chained(panel_kernel, dim3(static_cast<unsigned>(4 * (nblk - 1))), dim3(GEMM_THREADS), GEMM_SMEM, cs,
                                           A, cp, ki, Pk, LDP, Qk));
            }
            if (k == 0) break;
            // eager tiles of step k: block rows [o_lo, k) over the whole width, block rows [0, o_lo) over the
            // outer block's columns
            const int rows_in = static_cast<int>(k - o_lo);
            if (!fork || k == o_lo) {
                if (rest_pending) LQ_CUDA_TRY(cudaStreamWaitEvent(cs, h->ev_rest, 0));
                rest_pending = false;
                if (rows_in > 0 || o_lo > 0) {      // both regions in one launch: one partial round of CTAs instead of two
                    const int64_t rows_b = lq_ceil_div(o_lo * 2 * obw, 2 * nblk);
                    dim3 g(static_cast<unsigned>(2 * nblk), static_cast<unsigned>(rows_in + rows_b));
                    update_kernel<<<g, GEMM_THREADS, GEMM_SMEM, cs>>>(A, cp, ki, 10, static_cast<int>(o_lo), obw, Pk, LDP, Qk);
                    LQ_LAUNCH_CHECK();
                }
                continue;
            }
            if (rest_pending) LQ_CUDA_TRY(cudaStreamWaitEvent(cs, h->ev_rest, 0));     // step k+1's rest touched the same tiles
            update_kernel<<<static_cast<unsigned>(4 * nblk), GEMM_THREADS, GEMM_SMEM, cs>>>(A, cp, ki, 1, 0, 0, Pk, LDP, Qk);
            LQ_LAUNCH_CHECK();
            rest_pending = false;
            if (rows_in > 1 || o_lo > 0) {
                LQ_CUDA_TRY(cudaEventRecord(h->ev_next, cs));
                LQ_CUDA_TRY(cudaStreamWaitEvent(aux, h->ev_next, 0));
                {                              // block row k-1 is part of "next"; both regions in one launch
                    const int64_t rows_b = lq_ceil_div(o_lo * 2 * obw, 2 * nblk);
                    dim3 g(static_cast<unsigned>(2 * nblk), static_cast<unsigned>(rows_in - 1 + rows_b));
                    update_kernel<<<g, GEMM_THREADS, GEMM_SMEM, aux>>>(A, cp, ki, 12, static_cast<int>(o_lo), obw, Pk, LDP, Qk);
                    LQ_LAUNCH_CHECK();
                }
                LQ_CUDA_TRY(cudaEventRecord(h->ev_rest, aux));
                rest_pending = true;
            }
        }
        if (o_lo > 0) {
            if (rest_pending) LQ_CUDA_TRY(cudaStreamWaitEvent(cs, h->ev_rest, 0));
            rest_pending = false;
            int rc = deferred_update(h, cs, A, cp, o_lo, o_hi, Pob, reinterpret_cast<int*>(wsp + L.ex),
                                     wsp + L.sl, reinterpret_cast<float*>(wsp + L.ta),
                                     reinterpret_cast<float*>(wsp + L.tb), L.band);
            if (rc) return rc;
        }
    }
    if (rest_pending) LQ_CUDA_TRY(cudaStreamWaitEvent(cs, h->ev_rest, 0));
    if (next2_pending) LQ_CUDA_TRY(cudaStreamWaitEvent(cs, h->ev_next2, 0));
    if (fork) {
        LQ_CUDA_TRY(cudaEventRecord(h->ev_join, cs));
        LQ_CUDA_TRY(cudaStreamWaitEvent(st, h->ev_join, 0));
    }
    {
        // the panel buffers are free now: they hold the per-chunk column sums (c / 256 x c doubles <= 2 panels for c <= 65536)
        double* part = reinterpret_cast<double*>(wsp + L.pbuf);
        const int n_chunks = static_cast<int>(lq_ceil_div(c, FIN_ROWS));
        dim3 g(static_cast<unsigned>(lq_ceil_div(c, 32)), static_cast<unsigned>(n_chunks));
        finalize_kernel<<<g, 256, 0, st>>>(A, cp, c, U, ldu, part);
        LQ_LAUNCH_CHECK();
        dinv_kernel<<<static_cast<unsigned>(lq_ceil_div(c, 256)), 256, 0, st>>>(part, c, n_chunks, dinv);
        LQ_LAUNCH_CHECK();
    }
    return LQ_OK;
}

// ------------------------------------------------------------ diagonal of the factor --
namespace {
__global__ void chol_diag_kernel(const float* __restrict__ U, int64_t c, int64_t ldu, float* __restrict__ d) {
    const int64_t j = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (j < c) LQ_AT(d + j) = LQ_AT(U + j * ldu + j);
}
}  // namespace

extern "C" int lq_chol_diag(lq_handle* h, void* stream, const float* U, int64_t c, int64_t ldu, float* d) {
    if (!h || !U || !d || c <= 0 || ldu < c) return LQ_ERR_INVALID_ARG;
    {
        LQ_DBG_SCOPE(h, static_cast<cudaStream_t>(stream));
        LQ_DBG_REG(U, (static_cast<size_t>(c - 1) * ldu + c) * sizeof(float));
        LQ_DBG_REG(d, static_cast<size_t>(c) * sizeof(float));
        LQ_DBG_COMMIT();
    }
    chol_diag_kernel<<<static_cast<unsigned>(lq_ceil_div(c, 256)), 256, 0, static_cast<cudaStream_t>(stream)>>>(U, c, ldu, d);
    LQ_LAUNCH_CHECK();
    return LQ_OK;
}
