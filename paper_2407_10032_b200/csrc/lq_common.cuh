// Shared internals of liblq: handle layout, device status word, small helpers.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include <atomic>

#include "lq.h"

struct lq_dev_status {
    int32_t code;      // first failure recorded on the device (lq_status), 0 = none
    int32_t pad;
    long long info;    // detail of that failure
};

struct lq_handle {
    int device;
    int sm_count;
    lq_dev_status* dstatus;   // device memory
    // Fork/join helpers of stage 2: the bulk of a step's update runs on `aux` while the caller's
    // stream already works on the next block column.  Null in a handle that owns no stream
    // (everything then runs on the caller's stream).
    cudaStream_t aux;
    // Stage 2's serial chain (diagonal block, panel, "next" update) runs on a stream of the highest priority, so that
    // its CTAs are placed ahead of the queued CTAs of the bulk update; `mid` (one priority level below) takes the
    // updates that the chain needs two steps later.
    cudaStream_t chain, mid;
    cudaEvent_t ev_fork, ev_next, ev_rest, ev_join, ev_next2, ev_diag, ev_crit;
    // Time limit of every bounded wait inside a kernel launched through this handle (nanoseconds).
    unsigned long long wait_limit_ns;
    // Test hook: nonzero makes the load barriers of the tensor-core contraction expect bytes that never arrive, so that
    // its bounded waits run out (see lq_testing.h).
    int inject_stall;
    // Stage 2 defers the updates of far tiles to the bf16 tensor cores when the matrix has at least this many
    // 128-column blocks; below that the whole sweep stays on the FP64 MMA (a test hook can change the threshold).
    int prep_defer_min_blocks;
    // Digit slices of the deferred updates as 8-bit integers (tcgen05 kind::i8, the default) or as bf16 values.
    int prep_slices_int8;
};
constexpr int LQ_DEFAULT_PREP_DEFER_MIN_BLOCKS = 48;
constexpr unsigned long long LQ_DEFAULT_WAIT_LIMIT_NS = 5ull * 1000ull * 1000ull * 1000ull;

// Record the first device-side failure; later ones are dropped.
__device__ __forceinline__ void lq_report(lq_dev_status* st, int code, long long info) {
    if (atomicCAS(&st->code, 0, code) == 0) st->info = info;
}

// ---- debug build with address checks (-DLQ_DEBUG_BOUNDS) ------------------------------------------------------
// Every entry point registers the byte ranges of the buffers it was given (and of its workspace) in a small device
// table before it launches anything; the kernels then take each global or shared-memory address whose index derives
// from r, c, n, a leading dimension, a group or a block offset through LQ_AT(pointer): an address inside a registered
// range (or inside the CTA's shared-memory window) is used as it is, any other one records LQ_ERR_INVALID_ARG in the
// handle's status word (info = source line << 40 | low 40 bits of the address) and the access goes to a scratch
// word instead -- nothing traps and nothing touches memory the caller did not hand over.  In a normal build LQ_AT(p)
// is *(p) and the registration macros vanish.  The tensor-core contraction needs none of this: its global accesses are
// TMA copies, which the hardware clips to the tensor map.
#ifdef LQ_DEBUG_BOUNDS
constexpr int LQ_DBG_MAX_RANGES = 24;
struct lq_dbg_table {
    unsigned long long lo[LQ_DBG_MAX_RANGES], hi[LQ_DBG_MAX_RANGES];
    int n;
    lq_dev_status* st;
};
// one table and one scratch word per translation unit (the library is built without relocatable device code)
static __device__ lq_dbg_table lq_dbg_tab;
static __device__ __align__(16) unsigned char lq_dbg_sink[64];

__device__ __forceinline__ bool lq_dbg_ok(const void* p, size_t bytes, int line) {
    const unsigned long long a = reinterpret_cast<unsigned long long>(p);
    if (__isShared(p)) {
        const unsigned off = static_cast<unsigned>(__cvta_generic_to_shared(p));
        unsigned total;
        asm("mov.u32 %0, %%total_smem_size;" : "=r"(total));
        // the CTA's own shared memory starts behind the kilobyte the system reserves at the front of the window,
        // which %total_smem_size (static + dynamic) does not count
        if (off >= 1024u && off - 1024u + bytes <= total) return true;
    } else if (__isGlobal(p)) {
        const int n = lq_dbg_tab.n;
        for (int i = 0; i < n; ++i)
            if (a >= lq_dbg_tab.lo[i] && a + bytes <= lq_dbg_tab.hi[i]) return true;
    } else {
        return true;                       // local memory: the compiler's own
    }
    if (lq_dbg_tab.st) lq_report(lq_dbg_tab.st, LQ_ERR_INVALID_ARG, (static_cast<long long>(line) << 40) | static_cast<long long>(a & 0xffffffffffull));
    return false;
}
template <typename T> __device__ __forceinline__ T* lq_dbg_at(T* p, int line) {
    return lq_dbg_ok(p, sizeof(T), line) ? p : reinterpret_cast<T*>(lq_dbg_sink);
}
#define LQ_AT(p) (*lq_dbg_at((p), __LINE__))
#define LQ_DBG_OK(p, bytes) lq_dbg_ok((p), (bytes), __LINE__)

struct lq_dbg_scope {
    lq_dbg_table t;
    cudaStream_t stream;
    lq_dbg_scope(lq_handle* h, cudaStream_t st) : stream(st) { t.n = 0; t.st = h ? h->dstatus : nullptr; }
    void reg(const void* p, size_t bytes) {
        if (!p || !bytes || t.n >= LQ_DBG_MAX_RANGES) return;
        t.lo[t.n] = reinterpret_cast<unsigned long long>(p);
        t.hi[t.n] = t.lo[t.n] + bytes;
        ++t.n;
    }
};
#define LQ_DBG_SCOPE(h, st) lq_dbg_scope lq_dbg_s((h), (st))
#define LQ_DBG_REG(p, bytes) lq_dbg_s.reg((p), (bytes))
#define LQ_DBG_COMMIT() cudaMemcpyToSymbolAsync(lq_dbg_tab, &lq_dbg_s.t, sizeof(lq_dbg_table), 0, cudaMemcpyHostToDevice, lq_dbg_s.stream)
#else
#define LQ_AT(p) (*(p))
#define LQ_DBG_OK(p, bytes) (true)
#define LQ_DBG_SCOPE(h, st) do { } while (0)
#define LQ_DBG_REG(p, bytes) do { } while (0)
#define LQ_DBG_COMMIT() do { } while (0)
#endif

#define LQ_CUDA_TRY(expr)                                   \
    do {                                                    \
        cudaError_t _e = (expr);                            \
        if (_e != cudaSuccess) return LQ_ERR_CUDA;          \
    } while (0)

// Every kernel launch of the library goes through this: it counts the launch (see
// lq_launch_count) and turns a launch failure into LQ_ERR_CUDA.
extern std::atomic<unsigned long long> lq_launches_total;
#define LQ_LAUNCH_CHECK()                                   \
    do {                                                    \
        lq_launches_total.fetch_add(1, std::memory_order_relaxed); \
        if (cudaGetLastError() != cudaSuccess) return LQ_ERR_CUDA; \
    } while (0)

// Kernel attributes (opt-in shared memory sizes) are per device: each set-up site keeps one of these and runs its
// set-up once per device of the process.  The flags are atomic; two host threads that race on the first use of a
// device may both run the set-up, which is harmless (setting an attribute twice gives the same state).
struct lq_once_per_device {
    std::atomic<bool> done[64];
    lq_once_per_device() { for (auto& d : done) d.store(false, std::memory_order_relaxed); }
    bool first() {
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return true;
        return !done[dev].exchange(true, std::memory_order_acq_rel);
    }
};

static inline size_t lq_align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static inline int64_t lq_ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// ---- bf16 tensor-core GEMM (lq_gemm_tc.cu) -------------------------------------------
// D[M x N] (fp32, row-major, ldd) (+)= alpha * sum_p A_p[M x K] * B_p[N x K]^T
// A_p and B_p are bf16, K contiguous.  The operands of all passes live in one matrix
// each: pass p reads rows [a_row_off[p], a_row_off[p] + M) of A_all and rows
// [b_row_off[p], b_row_off[p] + N) of B_all.  accumulate != 0 adds into D (a reduction
// done by the copy engine), otherwise D is overwritten.  upper_only != 0 skips the
// 128 x 256 tiles that lie strictly below the diagonal (symmetric results).
// The tensor core adds into its fp32 accumulator with truncation, so a long K is cut into
// segments whose partial sums are added to D with round-to-nearest (seg_iters).
constexpr int LQ_TC_MAX_PASS = 16;
constexpr int LQ_TC_MAX_LVL = 5;
struct lq_tc_gemm_args {
    const void* A_all; int64_t a_rows; int64_t lda;   // a_rows = total rows of A_all; bf16, or 8-bit integers with int8_ops
    const void* B_all; int64_t b_rows; int64_t ldb;
    float* D; int64_t ldd;
    int64_t M, N, K;
    int n_pass;
    int64_t a_row_off[LQ_TC_MAX_PASS];
    int64_t b_row_off[LQ_TC_MAX_PASS];
    float alpha;
    int accumulate;
    int upper_only;
    int seg_iters;   // flush the TMEM partial sum into D every seg_iters 64-wide k-steps (0 = only at the end)
    // Optional level-major order.  With n_lvl > 0 the passes are taken in n_lvl consecutive groups of lvl_npass[i]
    // passes ("levels"), and the work of a tile is ordered level by level: for each level, for each chunk of
    // chunk_kb k-steps of K, all passes of the level over that chunk form one segment (one TMEM partial sum, added to
    // the running fp32 sum with round-to-nearest).  This is what a product of fixed-point digit slices needs: the
    // digit products of one level are integers that a short segment sums exactly, and the levels -- least significant
    // first -- are then combined with one rounding each.  seg_iters is ignored.
    int n_lvl;
    int lvl_npass[LQ_TC_MAX_LVL];
    int chunk_kb;
    // 8-bit integer operands (int8_ops != 0): A_all / B_all hold bytes, pass p reads them as signed (a_signed[p] != 0)
    // or unsigned integers, the products are summed in int32 (exactly), and every partial sum is converted to fp32 and
    // multiplied by lvl_scale[level] (lvl_scale[0] without levels) as it is added to the running sum.  A k-step and
    // chunk_kb count 128 integers instead of 64 bf16.
    int int8_ops;
    int a_signed[LQ_TC_MAX_PASS], b_signed[LQ_TC_MAX_PASS];
    float lvl_scale[LQ_TC_MAX_LVL];
    // D_first != nullptr (integer operands, n_lvl >= 2, one chunk per level, accumulate == 0): the first level's scaled
    // sum is stored to D_first (same shape and leading dimension as D) and does not enter the running sum that goes to
    // D.  An exact leading level and the rounded sum of the other levels then come out of one launch.
    float* D_first;
};
int lq_tc_gemm(lq_handle* h, cudaStream_t stream, const lq_tc_gemm_args& a);

// ---- pieces of stage 3 that other stages reuse (lq_fit_grid.cu) ------------------------
// Sample weights s_j = exp(-p (ln dinv_j - mean ln dinv)) into s64 (c doubles); scal: 256 bytes of scratch.
int lq_sample_weights(lq_handle* h, cudaStream_t st, const float* dinv, int64_t c, double p, double* scal, double* s64);
// The search of Eq. 7 over r x n_groups groups of g weights starting at W (row stride ldw); s64 holds the sample
// weights of those n_groups * g columns; (S, Z) of group gi of row i goes to scale / zero [i * out_ld + gi].
int lq_affine_search(lq_handle* h, cudaStream_t st, const void* W, int32_t w_dtype, int64_t r, int64_t ldw, int64_t g,
                     int n_groups, const double* s64, int K, int T, int t_count, float* scale, int32_t* zero, int64_t out_ld);

// Split fp32 into three bf16 terms hi + mid + lo (each the bf16 rounding of what is left).
__device__ __forceinline__ void lq_split3(float x, __nv_bfloat16& hi, __nv_bfloat16& mid, __nv_bfloat16& lo) {
    hi = __float2bfloat16_rn(x);
    float r1 = x - __bfloat162float(hi);
    mid = __float2bfloat16_rn(r1);
    float r2 = r1 - __bfloat162float(mid);
    lo = __float2bfloat16_rn(r2);
}
