// Stage 3 -- the loss-error-aware grid (Section 3.2, Algorithm 1 lines 5-9).
//
// Non-uniform (Eq. 5): one weighted 1-D k-means per output row, one CTA per row, the sample
// weights s_j = dinv_j^(-p) / geometric mean shared by all rows.  The row is sorted once in
// shared memory; Lloyd iterations then work on boundaries and prefix sums (see below).
// Centroids, midpoints and cluster sums are fp64: a weight that sits next to a midpoint must
// fall on the same side as in a float64 evaluation, or the centroids drift apart by far more
// than rounding.
//
// Affine (Eq. 7): every (row, group) enumerates the candidates (t_min, t_max) over its weights
// held in shared memory and takes the arg-min (first minimum in t_min-major order) of the fp64
// losses.  Groups of up to 1024 weights: one warp per group with an fp32 pre-score (see
// affine_search_warp_kernel); longer groups: one CTA per group, all candidates in fp64.
#include <math.h>

#include <mutex>

#include "lq_common.cuh"
#include "lq_affine_warp.cuh"
#include "lq_sort.cuh"

namespace {

// threads of the long-row kernel (1024 were no faster for K = 4 and do not fit the 2 K doubles of cluster sums per thread for K = 16)
__host__ __device__ constexpr int km_threads(int) { return 512; }

// scal[1] = mean_j ln(dinv_j)
__global__ void log_mean_kernel(const float* __restrict__ dinv, int64_t c, double* __restrict__ scal, lq_dev_status* st) {
    __shared__ double red[1024];
    double s = 0.0;
    for (int64_t j = threadIdx.x; j < c; j += blockDim.x) {
        float d = LQ_AT(dinv + j);
        if (!(d > 0.0f) || !isfinite(d)) { lq_report(st, LQ_ERR_NONFINITE, j); d = 1.0f; }
        s += log(static_cast<double>(d));
    }
    red[threadIdx.x] = s;
    __syncthreads();
    for (int o = blockDim.x / 2; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) scal[1] = red[0] / static_cast<double>(c);
}

// s_j = exp(-p (ln dinv_j - mean ln dinv))
__global__ void sample_weights_kernel(const float* __restrict__ dinv, int64_t c, double p, const double* __restrict__ scal,
                                      double* __restrict__ s) {
    const int64_t j = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (j >= c) return;
    float d = LQ_AT(dinv + j);
    if (!(d > 0.0f) || !isfinite(d)) d = 1.0f;
    LQ_AT(s + j) = exp(-p * (log(static_cast<double>(d)) - scal[1]));
}

__device__ __forceinline__ float load_w(const float* p) { return LQ_AT(p); }
__device__ __forceinline__ float load_w(const __nv_bfloat16* p) { return __bfloat162float(LQ_AT(p)); }

// ---------------------------------------------------------------- sorted k-means ----
// In one dimension the members of a cluster are a contiguous range of the sorted row, so the
// row is sorted once and every Lloyd iteration reduces to K-1 boundary searches plus
// differences of prefix sums: the per-iteration cost no longer depends on the row length.
//   keys   : (order-preserving bits of w) << 32 | column index, bitonic-sorted in shared memory;
//   coarse : exclusive prefix sums of s and s*w at every 8th element, kept as double-double
//            (hi, lo) pairs so that a light cluster next to a very heavy weight (the sample
//            weights span many decades at p = 4) loses nothing to cancellation;
//   F(b)   : prefix up to element b = coarse[b / 8] plus at most 7 terms added one by one.
// Cluster k of an iteration is [ub(m_{k-1}), ub(m_k)) with ub(m) the first sorted position
// whose weight exceeds m: exactly "code = number of midpoints strictly below w".
struct dd { double hi, lo; };
// Error-free additions: written with the _rn intrinsics, which the compiler never fuses with a
// neighbouring multiplication (a fused multiply-add in place of the first sum breaks the
// error term by up to an ulp of the large operand).
__device__ __forceinline__ dd dd_add_d(dd a, double b) {
    const double s = __dadd_rn(a.hi, b);
    const double bb = __dsub_rn(s, a.hi);
    double e = __dadd_rn(__dsub_rn(a.hi, __dsub_rn(s, bb)), __dsub_rn(b, bb));
    e = __dadd_rn(e, a.lo);
    dd r;
    r.hi = __dadd_rn(s, e);
    r.lo = __dsub_rn(e, __dsub_rn(r.hi, s));
    return r;
}
__device__ __forceinline__ dd dd_add(dd a, dd b) {
    const double s = __dadd_rn(a.hi, b.hi);
    const double bb = __dsub_rn(s, a.hi);
    double e = __dadd_rn(__dsub_rn(a.hi, __dsub_rn(s, bb)), __dsub_rn(b.hi, bb));
    e = __dadd_rn(e, __dadd_rn(a.lo, b.lo));
    dd r;
    r.hi = __dadd_rn(s, e);
    r.lo = __dsub_rn(e, __dsub_rn(r.hi, s));
    return r;
}
__device__ __forceinline__ double dd_diff(dd a, dd b) {       // a - b, rounded to double
    const double nb = -b.hi;
    const double s = __dadd_rn(a.hi, nb);
    const double bb = __dsub_rn(s, a.hi);
    double e = __dadd_rn(__dsub_rn(a.hi, __dsub_rn(s, bb)), __dsub_rn(nb, bb));
    e = __dadd_rn(e, __dsub_rn(a.lo, b.lo));
    return __dadd_rn(s, e);
}
// Sort keys: the order-preserving bits of the weight above the column index.  bf16 rows fit a
// 32-bit key (16 + 16 bits), fp32 rows take 64 bits (32 + 32).
template <typename T> struct KeyOf;
template <> struct KeyOf<__nv_bfloat16> {
    typedef uint32_t type;
    static __device__ __forceinline__ type make(__nv_bfloat16 w, int i) {
        uint32_t u = __bfloat16_as_ushort(w);
        u ^= (u & 0x8000u) ? 0xffffu : 0x8000u;
        return (u << 16) | static_cast<uint32_t>(i);
    }
    static __device__ __forceinline__ type pad() { return 0xffffffffu; }
};
template <> struct KeyOf<float> {
    typedef unsigned long long type;
    static __device__ __forceinline__ type make(float w, int i) {
        uint32_t u = __float_as_uint(w);
        u ^= (u & 0x80000000u) ? 0xffffffffu : 0x80000000u;
        return (static_cast<unsigned long long>(u) << 32) | static_cast<uint32_t>(i);
    }
    static __device__ __forceinline__ type pad() { return ~0ull; }
};
__device__ __forceinline__ float key_weight(unsigned long long key) {
    uint32_t u = static_cast<uint32_t>(key >> 32);
    u ^= (u & 0x80000000u) ? 0x80000000u : 0xffffffffu;
    return __uint_as_float(u);
}
__device__ __forceinline__ float key_weight(uint32_t key) {
    uint32_t u = key >> 16;
    u ^= (u & 0x8000u) ? 0x8000u : 0xffffu;
    return __uint_as_float(u << 16);
}
__device__ __forceinline__ uint32_t key_index(unsigned long long key) { return static_cast<uint32_t>(key); }
__device__ __forceinline__ uint32_t key_index(uint32_t key) { return key & 0xffffu; }

constexpr int KS_CHUNK = 8;
constexpr int KS_MAX_N = 16384;        // rows up to this length are sorted in shared memory
struct dd2 { dd s, sw; };              // prefix of the sample weights and of s * w

template <int K, typename T>
__global__ void __launch_bounds__(KS_THREADS, 4)
kmeans_sorted_kernel(const T* __restrict__ W, int64_t ldw, int64_t r, int c, int n, const double* __restrict__ s64,
                     float* __restrict__ grid, int n_iter, int init) {
    typedef typename KeyOf<T>::type KeyT;
    extern __shared__ __align__(16) unsigned char ks_smem[];
    dd2* coarse = reinterpret_cast<dd2*>(ks_smem);            // n / 8 + 1 coarse prefixes, then the n keys (padded slots)
    KeyT* keys = reinterpret_cast<KeyT*>(coarse + (n / KS_CHUNK + 1));
    __shared__ dd2 tot[KS_THREADS];                            // per-thread totals, then their exclusive scan
    __shared__ double g[K];
    __shared__ dd2 F[K + 1];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nch = n / KS_CHUNK;
    const int cpt = nch > KS_THREADS ? nch / KS_THREADS : 1;   // chunks per thread

    for (int64_t row = blockIdx.x; row < r; row += gridDim.x) {
        const T* wp = W + row * ldw;
        for (int i = tid; i < n; i += KS_THREADS) LQ_AT(keys + ks_slot(i)) = i < c ? KeyOf<T>::make(LQ_AT(wp + i), i) : KeyOf<T>::pad();
        __syncthreads();
        bitonic_sort<KeyT>(keys, n, tid);
        // chunk totals, thread-local exclusive prefixes
        dd2 run;
        run.s.hi = run.s.lo = run.sw.hi = run.sw.lo = 0.0;
        for (int q = tid * cpt; q < (tid + 1) * cpt && q < nch; ++q) {
            LQ_AT(coarse + q) = run;
#pragma unroll
            for (int e = 0; e < KS_CHUNK; ++e) {
                const int i = q * KS_CHUNK + e;
                if (i < c) {
                    const KeyT key = LQ_AT(keys + ks_slot(i));
                    const double sv = LQ_AT(s64 + key_index(key));
                    run.s = dd_add_d(run.s, sv);                 // same order and arithmetic as F(b) below
                    run.sw = dd_add_d(run.sw, __dmul_rn(sv, static_cast<double>(key_weight(key))));
                }
            }
        }
        tot[tid] = run;
        __syncthreads();
        if (warp == 0) {       // exclusive scan of the 256 thread totals: 8 per lane, then across the warp
            dd2 loc[KS_THREADS / 32];
            dd2 acc;
            acc.s.hi = acc.s.lo = acc.sw.hi = acc.sw.lo = 0.0;
#pragma unroll
            for (int e = 0; e < KS_THREADS / 32; ++e) {
                loc[e] = acc;
                const dd2 v = tot[lane * (KS_THREADS / 32) + e];
                acc.s = dd_add(acc.s, v.s);
                acc.sw = dd_add(acc.sw, v.sw);
            }
            dd2 inc = acc;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                dd2 up;
                up.s.hi = __shfl_up_sync(0xffffffffu, inc.s.hi, o);
                up.s.lo = __shfl_up_sync(0xffffffffu, inc.s.lo, o);
                up.sw.hi = __shfl_up_sync(0xffffffffu, inc.sw.hi, o);
                up.sw.lo = __shfl_up_sync(0xffffffffu, inc.sw.lo, o);
                if (lane >= o) { inc.s = dd_add(up.s, inc.s); inc.sw = dd_add(up.sw, inc.sw); }
            }
            dd2 excl;                                           // sum of the lanes before this one
            excl.s.hi = __shfl_up_sync(0xffffffffu, inc.s.hi, 1);
            excl.s.lo = __shfl_up_sync(0xffffffffu, inc.s.lo, 1);
            excl.sw.hi = __shfl_up_sync(0xffffffffu, inc.sw.hi, 1);
            excl.sw.lo = __shfl_up_sync(0xffffffffu, inc.sw.lo, 1);
            if (lane == 0) excl.s.hi = excl.s.lo = excl.sw.hi = excl.sw.lo = 0.0;
#pragma unroll
            for (int e = 0; e < KS_THREADS / 32; ++e) {
                dd2 v;
                v.s = dd_add(excl.s, loc[e].s);
                v.sw = dd_add(excl.sw, loc[e].sw);
                tot[lane * (KS_THREADS / 32) + e] = v;
            }
            if (lane == 31) LQ_AT(coarse + nch) = inc;          // grand total
        }
        __syncthreads();
        {
            const dd2 off = tot[tid];
            for (int q = tid * cpt; q < (tid + 1) * cpt && q < nch; ++q) {
                dd2 v = LQ_AT(coarse + q);
                v.s = dd_add(off.s, v.s);
                v.sw = dd_add(off.sw, v.sw);
                LQ_AT(coarse + q) = v;
            }
        }
        __syncthreads();

        if (warp == 0) {
            const double lo = static_cast<double>(key_weight(keys[ks_slot(0)]));
            const double hi = static_cast<double>(key_weight(LQ_AT(keys + ks_slot(c - 1))));
            if (init == LQ_INIT_UNIFORM) {
                if (lane < K) g[lane] = lo + (hi - lo) * static_cast<double>(lane) / static_cast<double>(K - 1);   // Eq. 6
            } else if (lane < K) {
                // weighted quantiles: the sorted weight at the first position whose cumulative sample
                // weight reaches (k + 1/2) / K of the total
                const dd total = coarse[nch].s;
                const double target = (static_cast<double>(lane) + 0.5) / static_cast<double>(K) * (total.hi + total.lo);
                int p0 = 0, p1 = c - 1;                        // answer in [p0, p1]
                while (p0 < p1) {
                    const int mid = (p0 + p1) >> 1;
                    const int b = mid + 1;                     // cumulative weight of positions 0 .. mid
                    const int q = b / KS_CHUNK, rem = b % KS_CHUNK;
                    dd f = LQ_AT(coarse + q).s;
                    for (int e = 0; e < rem; ++e) f = dd_add_d(f, LQ_AT(s64 + key_index(LQ_AT(keys + ks_slot(q * KS_CHUNK + e)))));
                    if (f.hi + f.lo >= target) p1 = mid; else p0 = mid + 1;
                }
                g[lane] = static_cast<double>(key_weight(LQ_AT(keys + ks_slot(p0))));
            }
            if (lane == 0) {
                F[0].s.hi = F[0].s.lo = F[0].sw.hi = F[0].sw.lo = 0.0;
                F[K] = coarse[nch];
            }
            __syncwarp();
            int b_prev = -1;
            for (int it = 0; it < n_iter; ++it) {
                int b0 = 0;
                if (lane < K - 1) {
                    const double m = 0.5 * (g[lane] + g[lane + 1]);
                    int b1 = c;                                // first position whose weight exceeds m
                    while (b0 < b1) {
                        const int mid = (b0 + b1) >> 1;
                        if (static_cast<double>(key_weight(LQ_AT(keys + ks_slot(mid)))) > m) b1 = mid; else b0 = mid + 1;
                    }
                }
                // Unchanged boundaries give back the same centroids, and so would every later
                // iteration: the fixed point has been reached and the remaining iterations are skipped.
                if (__all_sync(0xffffffffu, b0 == b_prev)) break;
                b_prev = b0;
                if (lane < K - 1) {
                    const int q = b0 / KS_CHUNK, rem = b0 % KS_CHUNK;
                    dd2 f = LQ_AT(coarse + q);
                    for (int e = 0; e < rem; ++e) {
                        const KeyT key = LQ_AT(keys + ks_slot(q * KS_CHUNK + e));
                        const double sv = LQ_AT(s64 + key_index(key));
                        f.s = dd_add_d(f.s, sv);
                        f.sw = dd_add_d(f.sw, __dmul_rn(sv, static_cast<double>(key_weight(key))));
                    }
                    F[lane + 1] = f;
                }
                __syncwarp();
                if (lane < K) {
                    const double den = dd_diff(F[lane + 1].s, F[lane].s);
                    const double num = dd_diff(F[lane + 1].sw, F[lane].sw);
                    if (den > 0.0) g[lane] = num / den;         // an empty cluster keeps its centroid
                }
                __syncwarp();
            }
            if (lane < K) LQ_AT(grid + row * K + lane) = static_cast<float>(g[lane]);
        }
        __syncthreads();
    }
}

// ------------------------------------------------- rows that fit shared memory, Eq. 6 start: grouped by value ---
// A total order is more than the iterations need.  The row is grouped once into 2^14 buckets of equal width between
// its smallest and its largest weight with a counting pass: histogram, exclusive scan, scatter.  Positions inside a
// bucket keep no order.  The prefix sums of s and s*w over the positions are taken as in the sorted kernel; the prefix
// at a bucket's first position does not depend on the order inside the buckets.  The bucket index
// floor((w - lo) * scale), clamped, is monotone in w, and a boundary m takes its bucket through the same expression:
// every member of a lower bucket is < m, every member of a higher bucket is > m, and the members of that one bucket
// are compared with m one by one.  So ub(m) = first position of the bucket + its members <= m, and F(ub(m)) = the
// prefix at the bucket's first position + the terms of those members: the same assignments as the sorted kernel,
// without the sort.  The buckets are much narrower than the spacing of bf16 values around the bulk of a row, so a
// boundary's bucket is empty more often than not.
//   offs : 2^14 16-bit counters, two to a 32-bit word (a row has at most 16384 weights, so a half never carries);
//          after the scatter half b holds the position behind bucket b's last member.
constexpr int KB_BITS = 14;
constexpr int KB_BUCKETS = 1 << KB_BITS;
constexpr int KB_MIN_N = 4096;           // shorter rows are sorted: the counters' fixed cost (clearing, scan) would dominate
constexpr int KB_SERIAL_MAX = 24;        // boundary scans longer than this are shared out over the warp
__device__ __forceinline__ int value_bucket(double w, double lo, double scale) {
    const double x = __dmul_rn(__dsub_rn(w, lo), scale);
    int b = x < static_cast<double>(KB_BUCKETS - 1) ? static_cast<int>(x) : KB_BUCKETS - 1;      // x >= 0 for a member; NaN goes to the top bucket
    return b < 0 ? 0 : b;
}
__device__ __forceinline__ int offs_half(const uint32_t* offs, int b) { return static_cast<int>((offs[b >> 1] >> ((b & 1) * 16)) & 0xffffu); }

// NT threads: 256 for rows of 4096 weights (three CTAs per SM), 512 for longer ones (one or two CTAs per SM: more
// threads for the phases that all of them share).
template <int K, typename T, int NT>
__global__ void __launch_bounds__(NT, NT == 256 ? 3 : 1)
kmeans_bucket_kernel(const T* __restrict__ W, int64_t ldw, int64_t r, int c, int n, const double* __restrict__ s64,
                     float* __restrict__ grid, int n_iter) {
    typedef typename KeyOf<T>::type KeyT;
    extern __shared__ __align__(16) unsigned char ks_smem[];
    dd2* coarse = reinterpret_cast<dd2*>(ks_smem);            // n / 8 + 1 coarse prefixes, then the n keys, then the counters
    KeyT* keys = reinterpret_cast<KeyT*>(coarse + (n / KS_CHUNK + 1));
    uint32_t* offs = reinterpret_cast<uint32_t*>(ks_smem + (((n / KS_CHUNK + 1) * sizeof(dd2) + (n + n / 32) * sizeof(KeyT) + 15) & ~size_t(15)));
    __shared__ dd2 tot[NT];                            // per-thread totals, then their exclusive scan
    __shared__ double g[K];
    __shared__ dd2 F[K + 1];
    __shared__ KeyT ext[2][NT / 32];                   // per-warp smallest and largest key
    __shared__ int wsum[NT / 32];
    __shared__ double rng[2];                                  // smallest weight of the row, buckets per unit of weight
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nch = n / KS_CHUNK;
    const int cpt = nch > NT ? nch / NT : 1;   // chunks per thread
    constexpr int WPT = KB_BUCKETS / 2 / NT;           // counter words per thread in the scan

    for (int64_t row = blockIdx.x; row < r; row += gridDim.x) {
        const T* wp = W + row * ldw;
        for (int i = tid; i < KB_BUCKETS / 8; i += NT) reinterpret_cast<uint4*>(offs)[i] = make_uint4(0u, 0u, 0u, 0u);
        // smallest and largest weight of the row
        KeyT kmin = KeyOf<T>::pad(), kmax = 0;
        for (int i = tid; i < c; i += NT) {
            const KeyT key = KeyOf<T>::make(LQ_AT(wp + i), i);
            kmin = key < kmin ? key : kmin;
            kmax = key > kmax ? key : kmax;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const KeyT a = __shfl_xor_sync(0xffffffffu, kmin, o), b = __shfl_xor_sync(0xffffffffu, kmax, o);
            kmin = a < kmin ? a : kmin;
            kmax = b > kmax ? b : kmax;
        }
        if (lane == 0) { ext[0][warp] = kmin; ext[1][warp] = kmax; }
        __syncthreads();
        if (tid == 0) {
            KeyT k0 = ext[0][0], k1 = ext[1][0];
#pragma unroll
            for (int w = 1; w < NT / 32; ++w) {
                k0 = ext[0][w] < k0 ? ext[0][w] : k0;
                k1 = ext[1][w] > k1 ? ext[1][w] : k1;
            }
            const double lo = static_cast<double>(key_weight(k0)), hi = static_cast<double>(key_weight(k1));
            rng[0] = lo;
            rng[1] = hi > lo ? static_cast<double>(KB_BUCKETS) / (hi - lo) : 0.0;
            ext[0][0] = k0;
            ext[1][0] = k1;
        }
        __syncthreads();
        const double lo = rng[0], scale = rng[1];
        // histogram of the buckets
        for (int i = tid; i < c; i += NT) {
            const int b = value_bucket(static_cast<double>(key_weight(KeyOf<T>::make(LQ_AT(wp + i), i))), lo, scale);
            atomicAdd(offs + (b >> 1), (b & 1) ? 0x10000u : 1u);
        }
        __syncthreads();
        // exclusive scan of the counters: 64 buckets per thread, then across the CTA
        {
            uint32_t wv[WPT];
            int sum = 0;
#pragma unroll
            for (int e = 0; e < WPT / 4; ++e) {
                const uint4 v = reinterpret_cast<const uint4*>(offs)[tid * (WPT / 4) + e];
                wv[4 * e] = v.x; wv[4 * e + 1] = v.y; wv[4 * e + 2] = v.z; wv[4 * e + 3] = v.w;
            }
#pragma unroll
            for (int e = 0; e < WPT; ++e) sum += static_cast<int>((wv[e] & 0xffffu) + (wv[e] >> 16));
            int inc = sum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int up = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += up;
            }
            if (lane == 31) wsum[warp] = inc;
            __syncthreads();
            int run = inc - sum;
            for (int w = 0; w < warp; ++w) run += wsum[w];
#pragma unroll
            for (int e = 0; e < WPT; ++e) {
                const uint32_t lo = wv[e] & 0xffffu, hi = wv[e] >> 16;
                wv[e] = static_cast<uint32_t>(run) | (static_cast<uint32_t>(run + lo) << 16);
                run += static_cast<int>(lo + hi);
            }
#pragma unroll
            for (int e = 0; e < WPT / 4; ++e)
                reinterpret_cast<uint4*>(offs)[tid * (WPT / 4) + e] = make_uint4(wv[4 * e], wv[4 * e + 1], wv[4 * e + 2], wv[4 * e + 3]);
        }
        __syncthreads();
        // scatter: a bucket's counter hands out its positions
        for (int i = tid; i < c; i += NT) {
            const KeyT key = KeyOf<T>::make(LQ_AT(wp + i), i);
            const int b = value_bucket(static_cast<double>(key_weight(key)), lo, scale);
            const uint32_t old = atomicAdd(offs + (b >> 1), (b & 1) ? 0x10000u : 1u);
            const int pos = static_cast<int>((b & 1) ? old >> 16 : old & 0xffffu);
            LQ_AT(keys + ks_slot(pos)) = key;
        }
        __syncthreads();
        // chunk totals, thread-local exclusive prefixes (positions in bucket order).  A chunk's eight terms are loaded
        // first and summed as two chains of four (the double-double sums are exact far below the tolerance, so
        // their grouping is free).
        dd2 run;
        run.s.hi = run.s.lo = run.sw.hi = run.sw.lo = 0.0;
        for (int q = tid * cpt; q < (tid + 1) * cpt && q < nch; ++q) {
            LQ_AT(coarse + q) = run;
            double sv[KS_CHUNK], swv[KS_CHUNK];
#pragma unroll
            for (int e = 0; e < KS_CHUNK; ++e) {
                const int i = q * KS_CHUNK + e;
                sv[e] = swv[e] = 0.0;
                if (i < c) {
                    const KeyT key = LQ_AT(keys + ks_slot(i));
                    sv[e] = LQ_AT(s64 + key_index(key));
                    swv[e] = __dmul_rn(sv[e], static_cast<double>(key_weight(key)));
                }
            }
            dd2 half;
            half.s.hi = sv[KS_CHUNK / 2]; half.s.lo = 0.0; half.sw.hi = swv[KS_CHUNK / 2]; half.sw.lo = 0.0;
#pragma unroll
            for (int e = 0; e < KS_CHUNK / 2; ++e) {
                run.s = dd_add_d(run.s, sv[e]);
                run.sw = dd_add_d(run.sw, swv[e]);
                if (e > 0) {
                    half.s = dd_add_d(half.s, sv[KS_CHUNK / 2 + e]);
                    half.sw = dd_add_d(half.sw, swv[KS_CHUNK / 2 + e]);
                }
            }
            run.s = dd_add(run.s, half.s);
            run.sw = dd_add(run.sw, half.sw);
        }
        tot[tid] = run;
        __syncthreads();
        if (warp == 0) {       // exclusive scan of the 256 thread totals: 8 per lane, then across the warp
            dd2 loc[NT / 32];
            dd2 acc;
            acc.s.hi = acc.s.lo = acc.sw.hi = acc.sw.lo = 0.0;
#pragma unroll
            for (int e = 0; e < NT / 32; ++e) {
                loc[e] = acc;
                const dd2 v = tot[lane * (NT / 32) + e];
                acc.s = dd_add(acc.s, v.s);
                acc.sw = dd_add(acc.sw, v.sw);
            }
            dd2 inc = acc;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                dd2 up;
                up.s.hi = __shfl_up_sync(0xffffffffu, inc.s.hi, o);
                up.s.lo = __shfl_up_sync(0xffffffffu, inc.s.lo, o);
                up.sw.hi = __shfl_up_sync(0xffffffffu, inc.sw.hi, o);
                up.sw.lo = __shfl_up_sync(0xffffffffu, inc.sw.lo, o);
                if (lane >= o) { inc.s = dd_add(up.s, inc.s); inc.sw = dd_add(up.sw, inc.sw); }
            }
            dd2 excl;                                           // sum of the lanes before this one
            excl.s.hi = __shfl_up_sync(0xffffffffu, inc.s.hi, 1);
            excl.s.lo = __shfl_up_sync(0xffffffffu, inc.s.lo, 1);
            excl.sw.hi = __shfl_up_sync(0xffffffffu, inc.sw.hi, 1);
            excl.sw.lo = __shfl_up_sync(0xffffffffu, inc.sw.lo, 1);
            if (lane == 0) excl.s.hi = excl.s.lo = excl.sw.hi = excl.sw.lo = 0.0;
#pragma unroll
            for (int e = 0; e < NT / 32; ++e) {
                dd2 v;
                v.s = dd_add(excl.s, loc[e].s);
                v.sw = dd_add(excl.sw, loc[e].sw);
                tot[lane * (NT / 32) + e] = v;
            }
            if (lane == 31) LQ_AT(coarse + nch) = inc;          // grand total
        }
        __syncthreads();
        {
            const dd2 off = tot[tid];
            for (int q = tid * cpt; q < (tid + 1) * cpt && q < nch; ++q) {
                dd2 v = LQ_AT(coarse + q);
                v.s = dd_add(off.s, v.s);
                v.sw = dd_add(off.sw, v.sw);
                LQ_AT(coarse + q) = v;
            }
        }
        __syncthreads();

        if (warp == 0) {
            const double hi = static_cast<double>(key_weight(ext[1][0]));
            if (lane < K) g[lane] = lo + (hi - lo) * static_cast<double>(lane) / static_cast<double>(K - 1);   // Eq. 6
            if (lane == 0) {
                F[0].s.hi = F[0].s.lo = F[0].sw.hi = F[0].sw.lo = 0.0;
                F[K] = coarse[nch];
            }
            __syncwarp();
            int b_prev = -1;
            for (int it = 0; it < n_iter; ++it) {
                // boundary of lane: its bucket's members [start, end), of which cnt do not exceed m
                int start = 0, end = 0, cnt = 0;
                double m = 0.0;
                if (lane < K - 1) {
                    m = 0.5 * (g[lane] + g[lane + 1]);
                    const int B = value_bucket(m, lo, scale);
                    start = B > 0 ? offs_half(offs, B - 1) : 0;
                    end = offs_half(offs, B);
                }
                const bool wide = end - start > KB_SERIAL_MAX;
                const unsigned big = __ballot_sync(0xffffffffu, wide);
                if (!wide)
                    for (int p = start; p < end; ++p) cnt += !(static_cast<double>(key_weight(LQ_AT(keys + ks_slot(p)))) > m);
                for (unsigned todo = big; todo;) {              // a long bucket (many equal or nearly equal weights): all lanes count
                    const int src = __ffs(todo) - 1;
                    todo &= todo - 1;
                    const int ss = __shfl_sync(0xffffffffu, start, src), es = __shfl_sync(0xffffffffu, end, src);
                    const double ms = __shfl_sync(0xffffffffu, m, src);
                    int ac = 0;
                    for (int p = ss + lane; p < es; p += 32) ac += !(static_cast<double>(key_weight(LQ_AT(keys + ks_slot(p)))) > ms);
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) ac += __shfl_xor_sync(0xffffffffu, ac, o);
                    if (lane == src) cnt = ac;
                }
                const int b0 = start + cnt;                     // ub(m)
                // Unchanged boundaries give back the same centroids, and so would every later
                // iteration: the fixed point has been reached and the remaining iterations are skipped.
                if (__all_sync(0xffffffffu, b0 == b_prev)) break;
                b_prev = b0;
                // F(ub(m)).  Nearly always the bucket's members lie on one side of m (a bucket is narrower than the
                // spacing of the values around it): every position below b0 counts, and the prefix there is the nearer
                // coarse prefix plus or minus at most four terms.  A bucket with members on both sides adds its
                // members <= m to the prefix at its first position.
                const bool mixed = cnt != 0 && cnt != end - start;
                const int at = mixed ? start : b0;
                dd2 f;
                f.s.hi = f.s.lo = f.sw.hi = f.sw.lo = 0.0;
                if (lane < K - 1) {
                    const int q = at >> 3, rem = at & (KS_CHUNK - 1);
                    if (rem <= KS_CHUNK / 2) {
                        f = LQ_AT(coarse + q);
                        for (int e = 0; e < rem; ++e) {
                            const KeyT key = LQ_AT(keys + ks_slot(q * KS_CHUNK + e));
                            const double sv = LQ_AT(s64 + key_index(key));
                            f.s = dd_add_d(f.s, sv);
                            f.sw = dd_add_d(f.sw, __dmul_rn(sv, static_cast<double>(key_weight(key))));
                        }
                    } else {
                        f = LQ_AT(coarse + q + 1);
                        for (int e = rem; e < KS_CHUNK; ++e) {
                            const int i = q * KS_CHUNK + e;
                            if (i < c) {
                                const KeyT key = LQ_AT(keys + ks_slot(i));
                                const double sv = LQ_AT(s64 + key_index(key));
                                f.s = dd_add_d(f.s, -sv);
                                f.sw = dd_add_d(f.sw, -__dmul_rn(sv, static_cast<double>(key_weight(key))));
                            }
                        }
                    }
                    if (mixed && !wide) {
                        for (int p = start; p < end; ++p) {
                            const KeyT key = LQ_AT(keys + ks_slot(p));
                            const double wv = static_cast<double>(key_weight(key));
                            if (!(wv > m)) {
                                const double sv = LQ_AT(s64 + key_index(key));
                                f.s = dd_add_d(f.s, sv);
                                f.sw = dd_add_d(f.sw, __dmul_rn(sv, wv));
                            }
                        }
                    }
                }
                for (unsigned todo = __ballot_sync(0xffffffffu, mixed && wide); todo;) {      // long and mixed: all lanes sum
                    const int src = __ffs(todo) - 1;
                    todo &= todo - 1;
                    const int ss = __shfl_sync(0xffffffffu, start, src), es = __shfl_sync(0xffffffffu, end, src);
                    const double ms = __shfl_sync(0xffffffffu, m, src);
                    dd2 a;
                    a.s.hi = a.s.lo = a.sw.hi = a.sw.lo = 0.0;
                    for (int p = ss + lane; p < es; p += 32) {
                        const KeyT key = LQ_AT(keys + ks_slot(p));
                        const double wv = static_cast<double>(key_weight(key));
                        if (!(wv > ms)) {
                            const double sv = LQ_AT(s64 + key_index(key));
                            a.s = dd_add_d(a.s, sv);
                            a.sw = dd_add_d(a.sw, __dmul_rn(sv, wv));
                        }
                    }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
                        dd2 u;
                        u.s.hi = __shfl_xor_sync(0xffffffffu, a.s.hi, o);
                        u.s.lo = __shfl_xor_sync(0xffffffffu, a.s.lo, o);
                        u.sw.hi = __shfl_xor_sync(0xffffffffu, a.sw.hi, o);
                        u.sw.lo = __shfl_xor_sync(0xffffffffu, a.sw.lo, o);
                        a.s = dd_add(a.s, u.s);
                        a.sw = dd_add(a.sw, u.sw);
                    }
                    if (lane == src) {
                        f.s = dd_add(f.s, a.s);
                        f.sw = dd_add(f.sw, a.sw);
                    }
                }
                if (lane < K - 1) F[lane + 1] = f;
                __syncwarp();
                if (lane < K) {
                    const double den = dd_diff(F[lane + 1].s, F[lane].s);
                    const double num = dd_diff(F[lane + 1].sw, F[lane].sw);
                    if (den > 0.0) g[lane] = num / den;         // an empty cluster keeps its centroid
                }
                __syncwarp();
            }
            if (lane < K) LQ_AT(grid + row * K + lane) = static_cast<float>(g[lane]);
        }
        __syncthreads();
    }
}

// ------------------------------------------------- long rows: direct k-means --------
// Rows too long to sort in shared memory: the row is staged once in shared memory in its own
// type and every iteration visits every weight (compares and cluster sums in fp64).
template <int K, typename T>
__global__ void __launch_bounds__(km_threads(K))
kmeans_rows_kernel(const T* __restrict__ W, int64_t ldw, int64_t r, int64_t c, const double* __restrict__ s64,
                   float* __restrict__ grid, int n_iter) {
    constexpr int KM_THREADS = km_threads(K), KM_WARPS = KM_THREADS / 32;
    extern __shared__ unsigned char wrow_raw[];
    T* wrow = reinterpret_cast<T*>(wrow_raw);
    __shared__ double g[K];
    __shared__ double mid[K];
    __shared__ double red[KM_WARPS][2 * K];
    __shared__ float redf[2][KM_WARPS];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int64_t row = blockIdx.x; row < r; row += gridDim.x) {
        const T* wp = W + row * ldw;
        float mn = INFINITY, mx = -INFINITY;
        for (int64_t j = tid; j < c; j += KM_THREADS) {
            const T raw = LQ_AT(wp + j);
            LQ_AT(wrow + j) = raw;
            const float w = load_w(&raw);
            mn = fminf(mn, w);
            mx = fmaxf(mx, w);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        }
        if (lane == 0) { redf[0][warp] = mn; redf[1][warp] = mx; }
        __syncthreads();
        if (tid < K) {
            float a = redf[0][0], b = redf[1][0];
            for (int w = 1; w < KM_WARPS; ++w) { a = fminf(a, redf[0][w]); b = fmaxf(b, redf[1][w]); }
            const double lo = a, hi = b;
            g[tid] = lo + (hi - lo) * static_cast<double>(tid) / static_cast<double>(K - 1);   // Eq. 6
        }
        __syncthreads();

        for (int it = 0; it < n_iter; ++it) {
            if (tid < K - 1) mid[tid] = 0.5 * (g[tid] + g[tid + 1]);
            __syncthreads();
            double ns[K], nsw[K];
#pragma unroll
            for (int k = 0; k < K; ++k) ns[k] = nsw[k] = 0.0;
            for (int64_t j = tid; j < c; j += KM_THREADS) {
                const double w = static_cast<double>(load_w(wrow + j));
                const double sv = LQ_AT(s64 + j);
                int a = 0;
#pragma unroll
                for (int step = K / 2; step > 0; step >>= 1)
                    if (w > mid[a + step - 1]) a += step;          // count of midpoints below w
                const double sw = sv * w;
#pragma unroll
                for (int k = 0; k < K; ++k) {
                    ns[k] += (a == k) ? sv : 0.0;
                    nsw[k] += (a == k) ? sw : 0.0;
                }
            }
#pragma unroll
            for (int k = 0; k < K; ++k) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    ns[k] += __shfl_xor_sync(0xffffffffu, ns[k], o);
                    nsw[k] += __shfl_xor_sync(0xffffffffu, nsw[k], o);
                }
            }
            if (lane == 0) {
#pragma unroll
                for (int k = 0; k < K; ++k) { red[warp][k] = ns[k]; red[warp][K + k] = nsw[k]; }
            }
            __syncthreads();
            if (tid < K) {
                double den = 0.0, num = 0.0;
                for (int w = 0; w < KM_WARPS; ++w) { den += red[w][tid]; num += red[w][K + tid]; }
                if (den > 0.0) g[tid] = num / den;      // an empty / weightless cluster keeps its centroid
            }
            __syncthreads();
        }
        if (tid < K) LQ_AT(grid + row * K + tid) = static_cast<float>(g[tid]);
        __syncthreads();
    }
}

template <int K, typename T>
int launch_kmeans(cudaStream_t st, int sms, const T* W, int64_t ldw, int64_t r, int64_t c, const double* s64, float* grid,
                  int n_iter, int init) {
    if (c <= KS_MAX_N) {
        int n = 64;
        while (n < c) n <<= 1;
        const size_t smem = (static_cast<size_t>(n) / KS_CHUNK + 1) * sizeof(dd2) +
                            static_cast<size_t>(n + n / 32) * sizeof(typename KeyOf<T>::type);
        const size_t bsmem = ((smem + 15) & ~size_t(15)) + KB_BUCKETS * 2;
        // the start of Eq. 6 needs no order inside a bucket: the counting pass replaces the sort (where its counters fit
        // and pays: below 4096 weights the fixed cost of the 2^14 counters exceeds the sort's)
        if (init == LQ_INIT_UNIFORM && n >= KB_MIN_N && bsmem <= 216 * 1024) {
            static lq_once_per_device battr_set;
            if (battr_set.first()) {
                LQ_CUDA_TRY(cudaFuncSetAttribute(kmeans_bucket_kernel<K, T, 256>, cudaFuncAttributeMaxDynamicSharedMemorySize, 216 * 1024));
                LQ_CUDA_TRY(cudaFuncSetAttribute(kmeans_bucket_kernel<K, T, 512>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
            }
            if (n > 8192 && bsmem <= 200 * 1024) {      // one row fills an SM's shared memory: 512 threads for it
                kmeans_bucket_kernel<K, T, 512><<<static_cast<unsigned>(r < sms ? r : sms), 512, bsmem, st>>>(
                    W, ldw, r, static_cast<int>(c), n, s64, grid, n_iter);
                LQ_LAUNCH_CHECK();
                return LQ_OK;
            }
            int per_sm = static_cast<int>((228 * 1024) / (bsmem + 10 * 1024));
            per_sm = per_sm < 1 ? 1 : (per_sm > 3 ? 3 : per_sm);
            const int64_t cap = static_cast<int64_t>(sms) * per_sm;
            kmeans_bucket_kernel<K, T, 256><<<static_cast<unsigned>(r < cap ? r : cap), 256, bsmem, st>>>(
                W, ldw, r, static_cast<int>(c), n, s64, grid, n_iter);
            LQ_LAUNCH_CHECK();
            return LQ_OK;
        }
        static lq_once_per_device attr_set;
        if (attr_set.first()) {
            LQ_CUDA_TRY(cudaFuncSetAttribute(kmeans_sorted_kernel<K, T>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
        }
        int per_sm = static_cast<int>((228 * 1024) / (smem + 10 * 1024));      // static shared memory and the per-CTA reserve
        per_sm = per_sm < 1 ? 1 : (per_sm > 4 ? 4 : per_sm);                    // 64 registers x 256 threads: four CTAs per SM
        const int64_t cap = static_cast<int64_t>(sms) * per_sm;
        kmeans_sorted_kernel<K, T><<<static_cast<unsigned>(r < cap ? r : cap), KS_THREADS, smem, st>>>(
            W, ldw, r, static_cast<int>(c), n, s64, grid, n_iter, init);
    } else {
        if (init != LQ_INIT_UNIFORM) return LQ_ERR_UNSUPPORTED;     // rows this long only start from Eq. 6
        const size_t smem = static_cast<size_t>(c) * sizeof(T);
        if (smem > 200 * 1024) return LQ_ERR_UNSUPPORTED;
        static lq_once_per_device attr_set;
        if (attr_set.first()) {
            LQ_CUDA_TRY(cudaFuncSetAttribute(kmeans_rows_kernel<K, T>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
        }
        // two CTAs per SM where two rows fit the shared memory: the loop is bound by the latency of its fp64 sums
        const int64_t cap = static_cast<int64_t>(sms) * (2 * (smem + 8 * 1024) <= 227 * 1024 ? 2 : 1);
        kmeans_rows_kernel<K, T><<<static_cast<unsigned>(r < cap ? r : cap), km_threads(K), smem, st>>>(W, ldw, r, c, s64, grid, n_iter);
    }
    LQ_LAUNCH_CHECK();
    return LQ_OK;
}

// ------------------------------------------------------------------- affine search --
constexpr int AF_THREADS = 128;

template <typename T>
__global__ void __launch_bounds__(AF_THREADS)
affine_search_kernel(const T* __restrict__ W, int64_t ldw, int64_t c, int group, int n_groups,
                     const double* __restrict__ s64, int K, int Tparts, int t_count,
                     float* __restrict__ scale, int32_t* __restrict__ zero, int64_t out_ld) {
    extern __shared__ float wg[];                 // group weights
    __shared__ float redf[2][AF_THREADS / 32];
    __shared__ double best_loss[AF_THREADS / 32];
    __shared__ int best_idx[AF_THREADS / 32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t row = blockIdx.x / n_groups;
    const int gi = blockIdx.x % n_groups;
    const T* wp = W + row * ldw + (int64_t)gi * group;
    const double* sp = s64 + (int64_t)gi * group;

    float mn = INFINITY, mx = -INFINITY;
    for (int j = tid; j < group; j += AF_THREADS) {
        float w = load_w(wp + j);
        LQ_AT(wg + j) = w;
        mn = fminf(mn, w);
        mx = fmaxf(mx, w);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    if (lane == 0) { redf[0][warp] = mn; redf[1][warp] = mx; }
    __syncthreads();
    mn = redf[0][0]; mx = redf[1][0];
    for (int w = 1; w < AF_THREADS / 32; ++w) { mn = fminf(mn, redf[0][w]); mx = fmaxf(mx, redf[1][w]); }
    const double dmn = mn, dmx = mx, R = dmx - dmn;
    const double Km1 = static_cast<double>(K - 1);
    const int64_t out = row * out_ld + gi;

    if (R == 0.0) {                                // constant group
        if (tid == 0) {
            double lo = fmin(dmn, 0.0), hi = fmax(dmx, 0.0);
            double S = 1.0, Z = 0.0;
            if (hi != lo) { S = (hi - lo) / Km1; Z = -rint(lo / S); }
            LQ_AT(scale + out) = static_cast<float>(S);
            LQ_AT(zero + out) = static_cast<int32_t>(Z);
        }
        return;
    }

    const int side = t_count + 1;
    const int n_cand = side * side;
    double my_loss = INFINITY;
    int my_idx = 0x7fffffff;
    for (int cand = tid; cand < n_cand; cand += AF_THREADS) {
        const int t_min = cand / side, t_max = cand - t_min * side;
        const double lo = dmn + static_cast<double>(t_min) * R / static_cast<double>(Tparts);
        const double hi = dmx - static_cast<double>(t_max) * R / static_cast<double>(Tparts);
        const double S = (hi - lo) / Km1;
        if (!(S > 0.0)) continue;
        const double Z = -rint(lo / S);
        double loss = 0.0;
        for (int j = 0; j < group; ++j) {
            const double w = static_cast<double>(LQ_AT(wg + j));
            double q = rint(w / S) + Z;
            q = fmin(fmax(q, 0.0), Km1);
            const double d = (q - Z) * S - w;
            loss += LQ_AT(sp + j) * (d * d);
        }
        if (loss < my_loss) { my_loss = loss; my_idx = cand; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const double ol = __shfl_xor_sync(0xffffffffu, my_loss, o);
        const int oi = __shfl_xor_sync(0xffffffffu, my_idx, o);
        if (ol < my_loss || (ol == my_loss && oi < my_idx)) { my_loss = ol; my_idx = oi; }
    }
    if (lane == 0) { best_loss[warp] = my_loss; best_idx[warp] = my_idx; }
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < AF_THREADS / 32; ++w)
            if (best_loss[w] < my_loss || (best_loss[w] == my_loss && best_idx[w] < my_idx)) {
                my_loss = best_loss[w]; my_idx = best_idx[w];
            }
        double S = 1.0, Z = 0.0;
        if (my_idx != 0x7fffffff) {
            const int t_min = my_idx / side, t_max = my_idx - t_min * side;
            const double lo = dmn + static_cast<double>(t_min) * R / static_cast<double>(Tparts);
            const double hi = dmx - static_cast<double>(t_max) * R / static_cast<double>(Tparts);
            S = (hi - lo) / Km1;
            Z = -rint(lo / S);
        }
        LQ_AT(scale + out) = static_cast<float>(S);
        LQ_AT(zero + out) = static_cast<int32_t>(Z);
    }
}

// ------------------------------------------------------ affine search, warp per group --
// Groups up to AFW_MAX_GROUP weights: one warp per (row, group), lanes over the candidates
// (t_min, t_max), the group's (w, s) pairs broadcast out of shared memory.  Every candidate is
// first scored in fp32 (ten operations per weight); only the candidates whose score lies below
// aff_bar32 of the best score of the group are then evaluated in fp64 with exactly the
// arithmetic of Eq. 7, and the arg-min (first minimum in t_min-major order) is taken over
// those fp64 losses.  A candidate that is skipped has a score above that of an evaluated one
// by more than the fp32 error of both, so it cannot be the fp64 minimum: the result is that of
// the all-fp64 search.
constexpr int AFW_WARPS = 8;
constexpr int AFW_MAX_GROUP = 1024;

template <typename T>
__global__ void __launch_bounds__(AFW_WARPS * 32)
affine_search_warp_kernel(const T* __restrict__ W, int64_t ldw, int group, int n_groups, int64_t total_groups,
                          const double* __restrict__ s64, int K, int Tparts, int t_count,
                          float* __restrict__ scale, int32_t* __restrict__ zero, int64_t out_ld) {
    extern __shared__ __align__(16) unsigned char afw_smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float2* ws = reinterpret_cast<float2*>(afw_smem) + static_cast<size_t>(warp) * group;      // (w - min, s / max s)
    const int64_t gid = static_cast<int64_t>(blockIdx.x) * AFW_WARPS + warp;
    if (gid >= total_groups) return;                       // whole warps leave; no block-wide barrier below
    const int64_t row = gid / n_groups;
    const int gi = static_cast<int>(gid - row * n_groups);
    const int64_t oidx = row * out_ld + gi;
    const T* wp = W + row * ldw + static_cast<int64_t>(gi) * group;
    const double* sp = s64 + static_cast<int64_t>(gi) * group;
    double S, Z;
    lq_affine_warp_search([&](int j) { return load_w(wp + j); }, sp, group, ws, K, Tparts, t_count, lane, S, Z);
    if (lane == 0) {
        LQ_AT(scale + oidx) = static_cast<float>(S);
        LQ_AT(zero + oidx) = static_cast<int32_t>(Z);
    }
}

// ------------------------------------------- affine search over classes of candidates --
// A candidate (t_min, t_max) of Eq. 7 acts on the weights only through (S, Z).  S depends on
// u = t_min + t_max alone (up to the last bits of its fp64 evaluation), and along a line of
// constant u the ratio lo / S grows by (K - 1) / (T - u) per step of t_min, so Z = -rint(lo / S)
// keeps one integer value over a run of about (T - u) / (K - 1) consecutive candidates: at the
// paper's T = 2048 the (t + 1)^2 = 168100 candidates of the 4-bit search give only ~2400
// different grids.  This kernel scores each class (u, Z) once, in fp32, and evaluates in fp64,
// with the arithmetic of Eq. 7, only the first member (in t_min-major order) of every class whose
// score lies within 0.1 % of the best; the arg-min is the lexicographic minimum of (fp64 loss,
// candidate index) over those.  The members of a class have fp64 losses that differ by rounding
// noise only, so this is the all-candidate search up to which member of the winning class is
// named (same Z, S equal to ~1e-16).
// One CTA per group.  Requires (K - 1) / (T - 2t) < 1/2: then every integer between the Z of the
// two ends of a line is taken by some candidate on it.
constexpr int AC_MAX_U = 2048;           // lines of constant u: 2t + 1 of them
constexpr int AC_MAX_THREADS = 512;

template <typename T>
__global__ void __launch_bounds__(AC_MAX_THREADS)
affine_class_kernel(const T* __restrict__ W, int64_t ldw, int group, int n_groups, const double* __restrict__ s64, int K,
                    int Tparts, int t_count, int p_max, float* __restrict__ scale, int32_t* __restrict__ zero, int64_t out_ld,
                    lq_dev_status* __restrict__ dstatus) {
    extern __shared__ __align__(16) unsigned char ac_smem[];
    const int nu = 2 * t_count + 1;
    float2* ws = reinterpret_cast<float2*>(ac_smem);                          // (w - min, s / max s) of the group
    int* off = reinterpret_cast<int*>(ws + group);                             // nu + 1: first class of each line
    int* za = off + nu + 1;                                                    // nu: Z at the first candidate of the line
    float* score = reinterpret_cast<float*>(za + nu);                          // p_max
    int* list = reinterpret_cast<int*>(score + p_max);                         // p_max: classes to evaluate in fp64
    __shared__ double red_d[AC_MAX_THREADS / 32], red_s[AC_MAX_THREADS / 32];
    __shared__ float red_f[2][AC_MAX_THREADS / 32];
    __shared__ int red_i[AC_MAX_THREADS / 32];
    __shared__ int n_list;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nthr = blockDim.x, nwarp = nthr >> 5;
    const int64_t gid = blockIdx.x;
    const int64_t row = gid / n_groups;
    const int gi = static_cast<int>(gid - row * n_groups);
    const int64_t oidx = row * out_ld + gi;
    const T* wp = W + row * ldw + static_cast<int64_t>(gi) * group;
    const double* sp = s64 + static_cast<int64_t>(gi) * group;

    float mn = INFINITY, mx = -INFINITY;
    double smax = 0.0, ssum = 0.0;
    for (int j = tid; j < group; j += nthr) {
        const float w = load_w(wp + j);
        mn = fminf(mn, w);
        mx = fmaxf(mx, w);
        smax = fmax(smax, LQ_AT(sp + j));
        ssum += LQ_AT(sp + j);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        smax = fmax(smax, __shfl_xor_sync(0xffffffffu, smax, o));
        ssum += __shfl_xor_sync(0xffffffffu, ssum, o);
    }
    if (lane == 0) { red_f[0][warp] = mn; red_f[1][warp] = mx; red_d[warp] = smax; red_s[warp] = ssum; }
    if (tid == 0) n_list = 0;
    __syncthreads();
    ssum = 0.0;
    for (int w = 0; w < nwarp; ++w) {
        mn = fminf(mn, red_f[0][w]); mx = fmaxf(mx, red_f[1][w]); smax = fmax(smax, red_d[w]); ssum += red_s[w];
    }
    __syncthreads();                                  // the scratch is reused below
    const double sinv = smax > 0.0 ? 1.0 / smax : 1.0;
    const float sum_s = static_cast<float>(ssum * sinv);
    for (int j = tid; j < group; j += nthr) LQ_AT(ws + j) = make_float2(load_w(wp + j) - mn, static_cast<float>(LQ_AT(sp + j) * sinv));

    const double dmn = mn, dmx = mx, R = dmx - dmn;
    const double Km1 = static_cast<double>(K - 1);
    const double dT = static_cast<double>(Tparts);
    if (R == 0.0) {                                // constant group
        if (tid == 0) {
            double lo = fmin(dmn, 0.0), hi = fmax(dmx, 0.0);
            double S = 1.0, Z = 0.0;
            if (hi != lo) { S = (hi - lo) / Km1; Z = -rint(lo / S); }
            LQ_AT(scale + oidx) = static_cast<float>(S);
            LQ_AT(zero + oidx) = static_cast<int32_t>(Z);
        }
        return;
    }
    const int side = t_count + 1;
    // (S, Z) of a candidate exactly as Eq. 7 gives them; false when the candidate is void
    auto params = [&](int t_min, int t_max, double& S, double& Z) {
        const double lo = dmn + static_cast<double>(t_min) * R / dT;
        const double hi = dmx - static_cast<double>(t_max) * R / dT;
        S = (hi - lo) / Km1;
        if (!(S > 0.0)) return false;
        Z = -rint(lo / S);
        return true;
    };

    // classes per line of constant u, then their exclusive prefix sum
    for (int u = tid; u < nu; u += nthr) {
        const int a = max(0, u - t_count), b = min(t_count, u);
        double Sa, Za, Sb, Zb;
        int cnt = 0, z0 = 0;
        if (params(a, u - a, Sa, Za) && params(b, u - b, Sb, Zb) && fabs(Za) < 1e9 && fabs(Zb) < 1e9) {
            z0 = static_cast<int>(Za);
            cnt = max(z0 - static_cast<int>(Zb), 0) + 1;
        }
        LQ_AT(za + u) = z0;
        LQ_AT(off + u) = cnt;
    }
    __syncthreads();
    {
        const int per = (nu + nthr - 1) / nthr;
        const int lo_u = min(tid * per, nu), hi_u = min(lo_u + per, nu);
        int sum = 0;
        for (int u = lo_u; u < hi_u; ++u) sum += LQ_AT(off + u);
        int incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) red_i[warp] = incl;
        __syncthreads();
        int base = incl - sum;
        for (int w = 0; w < warp; ++w) base += red_i[w];
        for (int u = lo_u; u < hi_u; ++u) { const int cnt = LQ_AT(off + u); LQ_AT(off + u) = base; base += cnt; }
        if (tid == nthr - 1) LQ_AT(off + nu) = base;
    }
    __syncthreads();
    int P = LQ_AT(off + nu);
    if (P > p_max) {                                // cannot happen with the host's bound; never write past the arrays
        if (tid == 0) lq_report(dstatus, LQ_ERR_UNSUPPORTED, gid);
        P = p_max;
    }
    // line and Z of class p
    auto class_of = [&](int p, int& u, int& Z) {
        int lo_u = 0, hi_u = nu - 1;
        while (lo_u < hi_u) {                        // the last line whose first class is <= p
            const int mid = (lo_u + hi_u + 1) >> 1;
            if (LQ_AT(off + mid) <= p) lo_u = mid; else hi_u = mid - 1;
        }
        u = lo_u;
        Z = LQ_AT(za + u) - (p - LQ_AT(off + u));
    };
    const double c_s = R / (dT * Km1);               // S of line u = c_s (T - u)
    const float Km1f = static_cast<float>(K - 1);

    // fp32 score of every class
    float best32 = INFINITY;
    for (int p = tid; p < P; p += nthr) {
        int u, Zi;
        class_of(p, u, Zi);
        const AffScore as = aff_score_setup(c_s * static_cast<double>(Tparts - u), static_cast<double>(Zi), dmn, Km1);
        float sc = aff_score32(ws, group, as, Km1f);
        if (sc != sc) sc = -INFINITY;                // a NaN score is always re-examined in fp64
        LQ_AT(score + p) = sc;
        best32 = fminf(best32, sc == -INFINITY ? INFINITY : sc);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) best32 = fminf(best32, __shfl_xor_sync(0xffffffffu, best32, o));
    if (lane == 0) red_f[0][warp] = best32;
    __syncthreads();
    for (int w = 0; w < nwarp; ++w) best32 = fminf(best32, red_f[0][w]);
    const float bar32 = aff_bar32(best32, static_cast<float>(R), sum_s);
    for (int p = tid; p < P; p += nthr)
        if (LQ_AT(score + p) <= bar32) LQ_AT(list + atomicAdd(&n_list, 1)) = p;
    __syncthreads();
    const int n_eval = n_list;

    // fp64 loss of the first member of each listed class, one class per warp at a time
    double my_loss = INFINITY;
    int my_idx = 0x7fffffff;
    for (int i = warp; i < n_eval; i += nwarp) {
        int u, Zi;
        class_of(LQ_AT(list + i), u, Zi);
        const int a = max(0, u - t_count), b = min(t_count, u);
        const double Zd = static_cast<double>(Zi);
        // first t_min on the line with rint(lo / S) >= -Z, i.e. with Z(t_min) <= Z: estimate, then settle exactly
        const double S_u = c_s * static_cast<double>(Tparts - u);
        double est = ceil(((-Zd - 0.5) * S_u - dmn) * dT / R);
        int tm = static_cast<int>(fmin(fmax(est, static_cast<double>(a)), static_cast<double>(b)));
        double S, Z;
        for (int it = 0; it < 8 && tm > a; ++it) {
            if (params(tm - 1, u - tm + 1, S, Z) && Z <= Zd) --tm; else break;
        }
        for (int it = 0; it < 8 && tm < b; ++it) {
            if (params(tm, u - tm, S, Z) && Z > Zd) ++tm; else break;
        }
        if (!params(tm, u - tm, S, Z) || Z != Zd) continue;       // no candidate of the line has this Z
        double loss = 0.0;
        for (int j = lane; j < group; j += 32) {
            const double w = static_cast<double>(load_w(wp + j));
            double q = rint(w / S) + Z;
            q = fmin(fmax(q, 0.0), Km1);
            const double d = (q - Z) * S - w;
            loss += LQ_AT(sp + j) * (d * d);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) loss += __shfl_xor_sync(0xffffffffu, loss, o);
        const int idx = tm * side + (u - tm);
        if (loss < my_loss || (loss == my_loss && idx < my_idx)) { my_loss = loss; my_idx = idx; }
    }
    if (lane == 0) { red_d[warp] = my_loss; red_i[warp] = my_idx; }
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < nwarp; ++w)
            if (red_d[w] < my_loss || (red_d[w] == my_loss && red_i[w] < my_idx)) { my_loss = red_d[w]; my_idx = red_i[w]; }
        double S = 1.0, Z = 0.0;
        if (my_idx != 0x7fffffff) {
            const int t_min = my_idx / side;
            params(t_min, my_idx - t_min * side, S, Z);
        }
        LQ_AT(scale + oidx) = static_cast<float>(S);
        LQ_AT(zero + oidx) = static_cast<int32_t>(Z);
    }
}

// Whether the class kernel applies, and an upper bound of the classes of one group: a line whose lo / S spans
// a width d takes at most floor(d) + 2 integer values of Z.
bool affine_class_plan(int K, int Tparts, int t_count, int64_t g, int* p_max, size_t* smem) {
    const int nu = 2 * t_count + 1;
    if (nu > AC_MAX_U || g % 2 != 0 || Tparts - 2 * t_count <= 2 * (K - 1)) return false;
    if (static_cast<int64_t>(t_count + 1) * (t_count + 1) < 256) return false;       // few candidates: score them all
    int64_t total = 0;
    for (int u = 0; u < nu; ++u) {
        const int a = u > t_count ? u - t_count : 0, b = u < t_count ? u : t_count;
        total += static_cast<int64_t>(static_cast<double>(b - a) * (K - 1) / static_cast<double>(Tparts - u)) + 2;
    }
    const size_t bytes = static_cast<size_t>(g) * sizeof(float2) + static_cast<size_t>(2 * nu + 1) * sizeof(int) +
                         static_cast<size_t>(total) * (sizeof(float) + sizeof(int));
    if (bytes > 200 * 1024) return false;
    *p_max = static_cast<int>(total);
    *smem = bytes;
    return true;
}

int check_cfg(const lq_config* cfg) {
    if (!cfg) return LQ_ERR_INVALID_ARG;
    if (cfg->bits < 2 || cfg->bits > 4) return LQ_ERR_INVALID_ARG;
    if (cfg->grid_type != LQ_GRID_NONUNIFORM && cfg->grid_type != LQ_GRID_AFFINE) return LQ_ERR_INVALID_ARG;
    if (cfg->grid_type == LQ_GRID_NONUNIFORM && (cfg->n_iter < 0 || (cfg->init != LQ_INIT_UNIFORM && cfg->init != LQ_INIT_WEIGHTED_QUANTILE)))
        return LQ_ERR_INVALID_ARG;
    if (cfg->grid_type == LQ_GRID_AFFINE &&
        (cfg->T <= 0 || cfg->t_count < 0 || 2 * (int64_t)cfg->t_count > cfg->T || cfg->group_size < 0 || cfg->t_count > 4095))
        return LQ_ERR_INVALID_ARG;
    return LQ_OK;
}

}  // namespace

// Sample weights s_j = exp(-p (ln dinv_j - mean ln dinv)) into s64 (c doubles); scal: 256 bytes of scratch.
int lq_sample_weights(lq_handle* h, cudaStream_t st, const float* dinv, int64_t c, double p, double* scal, double* s64) {
    {
        LQ_DBG_SCOPE(h, st);
        LQ_DBG_REG(dinv, static_cast<size_t>(c) * sizeof(float));
        LQ_DBG_REG(scal, 256);
        LQ_DBG_REG(s64, static_cast<size_t>(c) * sizeof(double));
        LQ_DBG_COMMIT();
    }
    log_mean_kernel<<<1, 1024, 0, st>>>(dinv, c, scal, h->dstatus);
    LQ_LAUNCH_CHECK();
    sample_weights_kernel<<<static_cast<unsigned>(lq_ceil_div(c, 256)), 256, 0, st>>>(dinv, c, p, scal, s64);
    LQ_LAUNCH_CHECK();
    return LQ_OK;
}

// The search of Eq. 7 over r x n_groups groups of g weights starting at W (row stride ldw); s64 holds the sample
// weights of the n_groups * g columns; (S, Z) of group gi of row i goes to scale / zero [i * out_ld + gi].
int lq_affine_search(lq_handle* h, cudaStream_t st, const void* W, int32_t w_dtype, int64_t r, int64_t ldw, int64_t g,
                     int n_groups, const double* s64, int K, int T, int t_count, float* scale, int32_t* zero, int64_t out_ld) {
    {
        LQ_DBG_SCOPE(h, st);
        LQ_DBG_REG(W, (static_cast<size_t>(r - 1) * ldw + static_cast<size_t>(g) * n_groups) * (w_dtype == LQ_F32 ? 4 : 2));
        LQ_DBG_REG(s64, static_cast<size_t>(g) * n_groups * sizeof(double));
        LQ_DBG_REG(scale, (static_cast<size_t>(r - 1) * out_ld + n_groups) * sizeof(float));
        LQ_DBG_REG(zero, (static_cast<size_t>(r - 1) * out_ld + n_groups) * sizeof(int32_t));
        LQ_DBG_COMMIT();
    }
    int p_max = 0;
    size_t smem_c = 0;
    if (affine_class_plan(K, T, t_count, g, &p_max, &smem_c)) {
        static lq_once_per_device attr_c;
        if (attr_c.first()) {
            LQ_CUDA_TRY(cudaFuncSetAttribute(affine_class_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
            LQ_CUDA_TRY(cudaFuncSetAttribute(affine_class_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
        }
        const unsigned nb = static_cast<unsigned>(r * n_groups);
        const int threads = g > 8192 ? 512 : 256;
        if (w_dtype == LQ_F32)
            affine_class_kernel<float><<<nb, threads, smem_c, st>>>(static_cast<const float*>(W), ldw, (int)g, n_groups, s64, K, T,
                                                                   t_count, p_max, scale, zero, out_ld, h->dstatus);
        else
            affine_class_kernel<__nv_bfloat16><<<nb, threads, smem_c, st>>>(static_cast<const __nv_bfloat16*>(W), ldw, (int)g, n_groups,
                                                                           s64, K, T, t_count, p_max, scale, zero, out_ld, h->dstatus);
        LQ_LAUNCH_CHECK();
        return LQ_OK;
    }
    if (g <= AFW_MAX_GROUP && g % 2 == 0) {
        const int64_t total = r * n_groups;
        const size_t smem_w = static_cast<size_t>(AFW_WARPS) * g * sizeof(float2);
        static lq_once_per_device attr_w;
        if (attr_w.first()) {
            LQ_CUDA_TRY(cudaFuncSetAttribute(affine_search_warp_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, AFW_WARPS * AFW_MAX_GROUP * 8));
            LQ_CUDA_TRY(cudaFuncSetAttribute(affine_search_warp_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, AFW_WARPS * AFW_MAX_GROUP * 8));
        }
        const unsigned nb = static_cast<unsigned>(lq_ceil_div(total, AFW_WARPS));
        if (w_dtype == LQ_F32)
            affine_search_warp_kernel<float><<<nb, AFW_WARPS * 32, smem_w, st>>>(static_cast<const float*>(W), ldw, (int)g, n_groups, total,
                                                                              s64, K, T, t_count, scale, zero, out_ld);
        else
            affine_search_warp_kernel<__nv_bfloat16><<<nb, AFW_WARPS * 32, smem_w, st>>>(static_cast<const __nv_bfloat16*>(W), ldw, (int)g,
                                                                                      n_groups, total, s64, K, T, t_count, scale, zero,
                                                                                      out_ld);
        LQ_LAUNCH_CHECK();
        return LQ_OK;
    }
    const size_t smem = static_cast<size_t>(g) * sizeof(float);
    const unsigned blocks = static_cast<unsigned>(r * n_groups);
    static lq_once_per_device attr_set;
    if (attr_set.first()) {
        LQ_CUDA_TRY(cudaFuncSetAttribute(affine_search_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
        LQ_CUDA_TRY(cudaFuncSetAttribute(affine_search_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    }
    if (w_dtype == LQ_F32)
        affine_search_kernel<float><<<blocks, AF_THREADS, smem, st>>>(static_cast<const float*>(W), ldw, 0, (int)g, n_groups, s64, K, T,
                                                                       t_count, scale, zero, out_ld);
    else
        affine_search_kernel<__nv_bfloat16><<<blocks, AF_THREADS, smem, st>>>(static_cast<const __nv_bfloat16*>(W), ldw, 0, (int)g,
                                                                               n_groups, s64, K, T, t_count, scale, zero, out_ld);
    LQ_LAUNCH_CHECK();
    return LQ_OK;
}

extern "C" int lq_fit_grid_workspace(const lq_config* cfg, int64_t r, int64_t c, size_t* bytes) {
    int e = check_cfg(cfg);
    if (e) return e;
    if (!bytes || r <= 0 || c <= 0) return LQ_ERR_INVALID_ARG;
    *bytes = 256 + lq_align_up(static_cast<size_t>(c) * sizeof(double), 256);
    return LQ_OK;
}

extern "C" int lq_fit_grid(lq_handle* h, void* stream, const lq_config* cfg, const void* W, int32_t w_dtype, int64_t r,
                           int64_t c, int64_t ldw, const float* dinv, float* grid, float* scale, int32_t* zero, void* ws,
                           size_t ws_bytes) {
    int e = check_cfg(cfg);
    if (e) return e;
    if (!h || !W || !dinv || r <= 0 || c <= 0 || ldw < c) return LQ_ERR_INVALID_ARG;
    if (w_dtype != LQ_F32 && w_dtype != LQ_BF16) return LQ_ERR_INVALID_ARG;
    size_t need = 0;
    lq_fit_grid_workspace(cfg, r, c, &need);
    if (!ws || ws_bytes < need) return LQ_ERR_WORKSPACE_TOO_SMALL;
    if (reinterpret_cast<uintptr_t>(ws) & 255) return LQ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    double* scal = static_cast<double*>(ws);
    double* s64 = reinterpret_cast<double*>(static_cast<char*>(ws) + 256);

    if (cfg->grid_type == LQ_GRID_NONUNIFORM) {
        if (!grid) return LQ_ERR_INVALID_ARG;
    } else {
        if (!scale || !zero) return LQ_ERR_INVALID_ARG;
        const int64_t g = cfg->group_size == 0 ? c : cfg->group_size;
        if (c % g) return LQ_ERR_INVALID_ARG;
        if (g * sizeof(float) > 200 * 1024) return LQ_ERR_UNSUPPORTED;
        if (r * (c / g) > 0x7fffffffLL) return LQ_ERR_UNSUPPORTED;
    }

    if (cfg->grid_type == LQ_GRID_NONUNIFORM && c > KS_MAX_N) {
        // rows too long for the sorted path: what the direct path cannot do is refused before anything is enqueued
        if (cfg->init != LQ_INIT_UNIFORM) return LQ_ERR_UNSUPPORTED;
        if (static_cast<size_t>(c) * (w_dtype == LQ_F32 ? 4 : 2) > 200 * 1024) return LQ_ERR_UNSUPPORTED;
    }

    e = lq_sample_weights(h, st, dinv, c, static_cast<double>(cfg->p), scal, s64);
    if (e) return e;

    if (cfg->grid_type == LQ_GRID_NONUNIFORM) {
        {   // (after lq_sample_weights, which registered its own buffers for its two launches)
            LQ_DBG_SCOPE(h, st);
            LQ_DBG_REG(W, (static_cast<size_t>(r - 1) * ldw + c) * (w_dtype == LQ_F32 ? 4 : 2));
            LQ_DBG_REG(s64, static_cast<size_t>(c) * sizeof(double));
            LQ_DBG_REG(grid, static_cast<size_t>(r) * (size_t(1) << cfg->bits) * sizeof(float));
            LQ_DBG_COMMIT();
        }
#define LQ_KM(KK)                                                                                                     \
    (w_dtype == LQ_F32 ? launch_kmeans<KK, float>(st, h->sm_count, static_cast<const float*>(W), ldw, r, c, s64, grid, cfg->n_iter, cfg->init) \
                       : launch_kmeans<KK, __nv_bfloat16>(st, h->sm_count, static_cast<const __nv_bfloat16*>(W), ldw, r, c, s64, grid, cfg->n_iter, cfg->init))
        switch (cfg->bits) {
            case 2: return LQ_KM(4);
            case 3: return LQ_KM(8);
            default: return LQ_KM(16);
        }
#undef LQ_KM
    }

    const int64_t g = cfg->group_size == 0 ? c : cfg->group_size;
    const int n_groups = static_cast<int>(c / g);
    return lq_affine_search(h, st, W, w_dtype, r, ldw, g, n_groups, s64, 1 << cfg->bits, cfg->T, cfg->t_count, scale, zero, n_groups);
}

// ---------------------------------------------------- entry point without allocation --
// Same computation as lq_fit_grid, with the scratch in an array that is part of the library
// image instead of a caller workspace (for callers that must not allocate device memory).
namespace {

constexpr size_t kNoAllocScratchBytes = 256 + static_cast<size_t>(LQ_FIT_GRID_NOALLOC_MAX_C) * sizeof(double);
static __device__ __align__(256) unsigned char lq_noalloc_scratch[kNoAllocScratchBytes];
static __device__ __align__(256) lq_dev_status lq_noalloc_status;    // used when the caller has no handle

// In host code the two names above are only stand-ins for the device arrays; their device
// addresses are looked up once per device and kept here.
constexpr int kMaxDevices = 64;
struct NoAllocDevice {
    bool ready = false;
    void* scratch = nullptr;
    lq_dev_status* status = nullptr;
    int sm_count = 0;
};
NoAllocDevice g_noalloc[kMaxDevices];
std::mutex g_noalloc_mutex;

int noalloc_setup(int dev, NoAllocDevice& out) {
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    NoAllocDevice& d = g_noalloc[dev];
    if (!d.ready) {
        void* sp = nullptr;
        void* tp = nullptr;
        int sms = 0;
        LQ_CUDA_TRY(cudaGetSymbolAddress(&sp, lq_noalloc_scratch));
        LQ_CUDA_TRY(cudaGetSymbolAddress(&tp, lq_noalloc_status));
        LQ_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        if (!sp || !tp || sms <= 0) return LQ_ERR_CUDA;
        d.scratch = sp;
        d.status = static_cast<lq_dev_status*>(tp);
        d.sm_count = sms;
        d.ready = true;
    }
    out = d;
    return LQ_OK;
}

}  // namespace

extern "C" int lq_fit_grid_noalloc(lq_handle* h, void* stream, const lq_config* cfg, const void* W, int32_t w_dtype,
                                   int64_t r, int64_t c, int64_t ldw, const float* dinv, float* grid, float* scale,
                                   int32_t* zero) {
    int e = check_cfg(cfg);
    if (e) return e;
    if (r <= 0 || c <= 0) return LQ_ERR_INVALID_ARG;
    size_t need = 0;
    e = lq_fit_grid_workspace(cfg, r, c, &need);
    if (e) return e;
    if (c > LQ_FIT_GRID_NOALLOC_MAX_C || need > kNoAllocScratchBytes) return LQ_ERR_STATIC_SCRATCH_TOO_SMALL;
    int dev = -1;
    LQ_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return LQ_ERR_UNSUPPORTED;
    if (h && h->device != dev) return LQ_ERR_INVALID_ARG;
    NoAllocDevice d;
    e = noalloc_setup(dev, d);
    if (e) return e;
    lq_handle local;
    local.device = dev;
    local.sm_count = d.sm_count;
    local.dstatus = d.status;
    local.aux = nullptr;
    local.chain = local.mid = nullptr;
    local.ev_fork = local.ev_next = local.ev_rest = local.ev_join = local.ev_next2 = local.ev_diag = local.ev_crit = nullptr;
    local.wait_limit_ns = LQ_DEFAULT_WAIT_LIMIT_NS;
    local.inject_stall = 0;
    local.prep_defer_min_blocks = LQ_DEFAULT_PREP_DEFER_MIN_BLOCKS;
    local.prep_slices_int8 = 1;
    return lq_fit_grid(h ? h : &local, stream, cfg, W, w_dtype, r, c, ldw, dinv, grid, scale, zero, d.scratch,
                       kNoAllocScratchBytes);
}
