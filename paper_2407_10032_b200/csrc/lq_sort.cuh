// Bitonic sort of keys in shared memory by one CTA of KS_THREADS threads (used by the k-means kernel of stage 3 to sort
// a row of weights, and by the activation-order kernel to sort the diagonal of the Hessian).
#pragma once

#include <stdint.h>

// Shared-memory slot of sorted position i: one pad slot per 32, so that the strided accesses of
// the register-blocked sort spread over the banks.
__device__ __forceinline__ int ks_slot(int i) { return i + (i >> 5); }

constexpr int KS_THREADS = 256;


// Compare-exchange sub-stages of a bitonic network on 16 keys held in registers: sub-stage s
// pairs registers that differ in bit s of their number; NST sub-stages, highest bit first.
template <typename KeyT, int NST>
__device__ __forceinline__ void ce_stages(KeyT (&e)[16], bool up) {
#pragma unroll
    for (int s = NST - 1; s >= 0; --s) {
#pragma unroll
        for (int m = 0; m < 16; ++m) {
            if ((m >> s) & 1) continue;
            const KeyT a = e[m], b = e[m | (1 << s)];
            const KeyT lo = a < b ? a : b, hi = a < b ? b : a;
            e[m] = up ? lo : hi;
            e[m | (1 << s)] = up ? hi : lo;
        }
    }
}

// Ascending bitonic sort of n keys (a power of two >= 64) in shared memory.  Every pass through
// shared memory moves 16 keys per thread into registers and runs up to four sub-stages there.
template <typename KeyT>
__device__ __forceinline__ void bitonic_sort(KeyT* keys, int n, int tid) {
    const int logn = 31 - __clz(n);
    // levels k = 2, 4, 8, 16 on 16 consecutive keys
    for (int vt = tid; vt < (n >> 4); vt += KS_THREADS) {
        KeyT e[16];
#pragma unroll
        for (int m = 0; m < 16; ++m) e[m] = keys[ks_slot(16 * vt + m)];
#pragma unroll
        for (int lk = 1; lk <= 4; ++lk) {
#pragma unroll
            for (int s = lk - 1; s >= 0; --s) {
#pragma unroll
                for (int m = 0; m < 16; ++m) {
                    if ((m >> s) & 1) continue;
                    const bool up = lk < 4 ? ((m >> lk) & 1) == 0 : (vt & 1) == 0;
                    const KeyT a = e[m], b = e[m | (1 << s)];
                    const KeyT lo = a < b ? a : b, hi = a < b ? b : a;
                    e[m] = up ? lo : hi;
                    e[m | (1 << s)] = up ? hi : lo;
                }
            }
        }
#pragma unroll
        for (int m = 0; m < 16; ++m) keys[ks_slot(16 * vt + m)] = e[m];
    }
    __syncthreads();
    for (int L = 5; L <= logn; ++L) {                 // level k = 2^L: sub-stages j = 2^(L-1) .. 1
        for (int bhi = L - 1; bhi >= 0; bhi -= 4) {
            const int lo = bhi >= 3 ? bhi - 3 : 0;
            const int nst = bhi - lo + 1;
            for (int vt = tid; vt < (n >> 4); vt += KS_THREADS) {
                const int base = ((vt >> lo) << (lo + 4)) | (vt & ((1 << lo) - 1));
                // a descending block is sorted ascending on the complemented keys: one flip on the way in and one on
                // the way out instead of a direction select in every compare-exchange
                const KeyT flip = ((base >> L) & 1) == 0 ? static_cast<KeyT>(0) : ~static_cast<KeyT>(0);
                KeyT e[16];
#pragma unroll
                for (int m = 0; m < 16; ++m) e[m] = keys[ks_slot(base | (m << lo))] ^ flip;
                if (nst == 4) ce_stages<KeyT, 4>(e, true);
                else if (nst == 3) ce_stages<KeyT, 3>(e, true);
                else if (nst == 2) ce_stages<KeyT, 2>(e, true);
                else ce_stages<KeyT, 1>(e, true);
#pragma unroll
                for (int m = 0; m < 16; ++m) keys[ks_slot(base | (m << lo))] = e[m] ^ flip;
            }
            __syncthreads();
        }
    }
}

