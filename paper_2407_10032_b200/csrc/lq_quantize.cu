// Stage 4 -- Algorithm 1 lines 10-21: the block-wise column loop with error feedback.
//
// Per block of B = 128 columns:
//   in-block kernel  : one warp per output row, four block columns per lane, walks the columns
//                      in order (quantise, E = (w - q)/U_jj, w[k] -= E * U[j][k]); the
//                      128 x 128 diagonal block of U sits in shared memory.
//   trailing update  : W[:, i+B:] -= E U[i:i+B, i+B:] on the tensor cores (lq_tc_gemm), in two
//                      levels (see the host loop), fp32
//                      operands fed as three bf16 terms each (six products), accumulated into
//                      the fp32 working copy by the copy engine's reduce-add.
#include <math.h>

#include "lq_common.cuh"
#include "lq_affine_warp.cuh"

namespace {

constexpr int B = 128;      // block width of the column loop
constexpr int OB = 1024;    // outer block: the lazy update of columns beyond it waits until it is complete

template <typename T>
__global__ void to_f32_kernel(const T* __restrict__ W, int64_t ldw, int64_t c, float* __restrict__ Wc, int64_t ldc, int vec) {
    const int64_t row = blockIdx.y;
    if (vec) {      // eight weights per thread: one 16-byte (bf16) or two 16-byte (fp32) loads, two 16-byte stores
        const int64_t n8 = c / 8;
        for (int64_t j8 = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; j8 < n8; j8 += (int64_t)gridDim.x * blockDim.x) {
            float v[8];
            if (sizeof(T) == 4) {
                const float4* p = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(W) + row * ldw + 8 * j8);
                const float4 x = LQ_AT(p), y = LQ_AT(p + 1);
                v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w; v[4] = y.x; v[5] = y.y; v[6] = y.z; v[7] = y.w;
            } else {
                const uint4 x = LQ_AT(reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(W) + row * ldw + 8 * j8));
                const uint32_t u[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    v[2 * e] = __uint_as_float(u[e] << 16);
                    v[2 * e + 1] = __uint_as_float(u[e] & 0xffff0000u);
                }
            }
            float4* q = reinterpret_cast<float4*>(Wc + row * ldc + 8 * j8);
            LQ_AT(q) = make_float4(v[0], v[1], v[2], v[3]);
            LQ_AT(q + 1) = make_float4(v[4], v[5], v[6], v[7]);
        }
        // the ragged end of the row, if any
        for (int64_t j = n8 * 8 + blockIdx.x * (int64_t)blockDim.x + threadIdx.x; j < ldc; j += (int64_t)gridDim.x * blockDim.x) {
            float v = 0.0f;
            if (j < c) {
                if (sizeof(T) == 4) v = LQ_AT(reinterpret_cast<const float*>(W) + row * ldw + j);
                else v = __bfloat162float(LQ_AT(reinterpret_cast<const __nv_bfloat16*>(W) + row * ldw + j));
            }
            LQ_AT(Wc + row * ldc + j) = v;
        }
        return;
    }
    for (int64_t j = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; j < ldc; j += (int64_t)gridDim.x * blockDim.x) {
        float v = 0.0f;
        if (j < c) {
            if (sizeof(T) == 4) v = LQ_AT(reinterpret_cast<const float*>(W) + row * ldw + j);
            else v = __bfloat162float(LQ_AT(reinterpret_cast<const __nv_bfloat16*>(W) + row * ldw + j));
        }
        LQ_AT(Wc + row * ldc + j) = v;
    }
}

// UT[s][n][k] = s-th bf16 term of U[k][n]   (three stacked c x ldt matrices).  64 x 64 tiles: 16-byte reads along n,
// 16-byte writes (eight bf16) along k.
__global__ void __launch_bounds__(256)
split_transpose_kernel(const float* __restrict__ U, int64_t ldu, int64_t c, __nv_bfloat16* __restrict__ UT, int64_t ldt) {
    __shared__ float tile[64][65];
    const int64_t k0 = (int64_t)blockIdx.y * 64, n0 = (int64_t)blockIdx.x * 64;
    const int tid = threadIdx.x;
    const bool vec_in = (ldu % 4 == 0) && ((reinterpret_cast<uintptr_t>(U) & 15) == 0);
    for (int idx = tid; idx < 64 * 16; idx += 256) {
        const int a = idx >> 4, n4 = (idx & 15) * 4;
        const int64_t k = k0 + a, n = n0 + n4;
        float4 v = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        if (k < c) {
            if (vec_in && n + 3 < c) v = LQ_AT(reinterpret_cast<const float4*>(U + k * ldu + n));
            else {
                if (n < c) v.x = LQ_AT(U + k * ldu + n);
                if (n + 1 < c) v.y = LQ_AT(U + k * ldu + n + 1);
                if (n + 2 < c) v.z = LQ_AT(U + k * ldu + n + 2);
                if (n + 3 < c) v.w = LQ_AT(U + k * ldu + n + 3);
            }
        }
        tile[a][n4] = v.x; tile[a][n4 + 1] = v.y; tile[a][n4 + 2] = v.z; tile[a][n4 + 3] = v.w;
    }
    __syncthreads();
    for (int idx = tid; idx < 64 * 8; idx += 256) {
        const int a = idx >> 3, k8 = (idx & 7) * 8;        // output row n0 + a, eight consecutive k
        const int64_t n = n0 + a, k = k0 + k8;
        if (n >= c || k >= ldt) continue;
        uint32_t ph[4], pm[4], pl[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            __nv_bfloat16 h0, m0, l0, h1, m1, l1;
            lq_split3(tile[k8 + 2 * e][a], h0, m0, l0);            // rows k >= c of the tile are zero
            lq_split3(tile[k8 + 2 * e + 1][a], h1, m1, l1);
            ph[e] = static_cast<uint32_t>(__bfloat16_as_ushort(h0)) | (static_cast<uint32_t>(__bfloat16_as_ushort(h1)) << 16);
            pm[e] = static_cast<uint32_t>(__bfloat16_as_ushort(m0)) | (static_cast<uint32_t>(__bfloat16_as_ushort(m1)) << 16);
            pl[e] = static_cast<uint32_t>(__bfloat16_as_ushort(l0)) | (static_cast<uint32_t>(__bfloat16_as_ushort(l1)) << 16);
        }
        // ldt is a multiple of 8 and k a multiple of 8: the eight entries are inside the row and 16-byte aligned
        LQ_AT(reinterpret_cast<uint4*>(UT + n * ldt + k)) = make_uint4(ph[0], ph[1], ph[2], ph[3]);
        LQ_AT(reinterpret_cast<uint4*>(UT + (c + n) * ldt + k)) = make_uint4(pm[0], pm[1], pm[2], pm[3]);
        LQ_AT(reinterpret_cast<uint4*>(UT + (2 * c + n) * ldt + k)) = make_uint4(pl[0], pl[1], pl[2], pl[3]);
    }
}

struct QuantOut {
    uint8_t* codes;          // r x c
    void* what;              // r x ldwh or null
    int what_bf16;
    int64_t ldwh;
    __nv_bfloat16* esplit;   // 3 x r x e_ld: the errors of one outer block; this launch fills columns e_col ..
    int64_t e_ld;
    int e_col;
    double* loss_rows;       // r
};

// One warp per output row, lane l owning columns 4l .. 4l+3 of the block.  Column step j:
// the owning lane's weight is broadcast; the nearest grid point is found by every lane
// comparing the weight with "its" midpoint (lane k holds g_k and m_k = (g_k + g_{k+1})/2) and a
// ballot -- code = number of midpoints strictly below w -- and the grid value comes back from
// lane `code`; then E = (w - q) / U_jj and every lane feeds it into its four weights with one
// 16-byte read of row j of the block of U held in shared memory.  Entries of that row left of
// the diagonal are zero, so no lane needs a predicate.
constexpr int IB_ROWS = 2;             // rows per warp of the in-block kernel (one where groups are refitted inside it)
constexpr int IB_MAX_THREADS = 1024;   // warps (= rows) per CTA are chosen at launch so that the rows spread evenly over the SMs

// Refit of groups shorter than a block inside the loop (the lazy variant of the affine grid): what the kernel needs
// for the search of Eq. 7 when it reaches a group's first column.
struct RefitArgs {
    const double* s64;       // sample weights of all c columns
    float* scale;            // outputs, r x n_groups
    int32_t* zero;
    int T, t_count;
};

template <int K, bool AFFINE, bool REFIT, int ROWS>
__global__ void __launch_bounds__(REFIT ? IB_MAX_THREADS / 2 : IB_MAX_THREADS)
inblock_kernel(const float* __restrict__ Wc, int64_t ldc, int64_t r, int64_t c, int64_t i0, const float* __restrict__ U,
               int64_t ldu, const float* __restrict__ grid, const float* __restrict__ scale,
               const int32_t* __restrict__ zero, int group, int n_groups, QuantOut out, RefitArgs refit) {
    extern __shared__ float Us[];          // B x B block of U, then B reciprocals of its diagonal
    float* invd = Us + B * B;              // (REFIT: then per warp `group` floats and `group` float2 of search scratch)
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int bw = (c - i0) < B ? static_cast<int>(c - i0) : B;

    // The block of U goes to shared memory with asynchronous copies (plain loads for a ragged
    // last block); the row's weights and grid are fetched while those copies are in flight.
    const bool whole = bw == B && (ldu % 4 == 0);
    const int nthr = blockDim.x;
    for (int idx = tid; idx < B * B / 4; idx += nthr) {
        const int jj = idx / (B / 4), k4 = (idx % (B / 4)) * 4;
        if (whole) {
            const uint32_t dst = static_cast<uint32_t>(__cvta_generic_to_shared(Us + jj * B + k4));
            if (LQ_DBG_OK(U + (i0 + jj) * ldu + i0 + k4, 16) && LQ_DBG_OK(Us + jj * B + k4, 16))
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(U + (i0 + jj) * ldu + i0 + k4) : "memory");
        } else {
            float t[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int kk = k4 + u;
                t[u] = (jj < bw && kk < bw) ? LQ_AT(U + (i0 + jj) * ldu + i0 + kk) : (jj == kk ? 1.0f : 0.0f);
            }
            LQ_AT(reinterpret_cast<float4*>(Us + jj * B + k4)) = make_float4(t[0], t[1], t[2], t[3]);
        }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");

    // A warp carries R rows: the loads of the block of U, which every row needs, are shared between them, and their
    // dependency chains (broadcast, compare, look-up, subtract, multiply-add per column) interleave.
    constexpr int R = ROWS;
    const int64_t row0 = ((int64_t)blockIdx.x * (nthr >> 5) + warp) * R;
    bool valid[R];
    const int col0 = 4 * lane;             // first of this lane's columns inside the block
    float w[R][4];
    float gl[R], ml[R];                    // this lane's grid point and the midpoint above it
    float S_mine[R], Z_mine[R];            // affine parameters of this lane's columns
#pragma unroll
    for (int q = 0; q < R; ++q) {
        const int64_t row = row0 + q;
        valid[q] = row < r;
#pragma unroll
        for (int u = 0; u < 4; ++u) w[q][u] = 0.0f;
        if (valid[q]) {
            const float* wp = Wc + row * ldc + i0 + col0;
            if (col0 + 3 < bw) {
                const float4 v = LQ_AT(reinterpret_cast<const float4*>(wp));
                w[q][0] = v.x; w[q][1] = v.y; w[q][2] = v.z; w[q][3] = v.w;
            } else {
#pragma unroll
                for (int u = 0; u < 4; ++u) w[q][u] = (col0 + u < bw) ? LQ_AT(wp + u) : 0.0f;
            }
        }
        gl[q] = 0.0f; ml[q] = INFINITY; S_mine[q] = 1.0f; Z_mine[q] = 0.0f;
        if (!AFFINE) {
            if (valid[q] && lane < K) gl[q] = LQ_AT(grid + row * K + lane);
            const float gn = __shfl_down_sync(0xffffffffu, gl[q], 1);
            if (lane < K - 1) ml[q] = 0.5f * (gl[q] + gn);
        } else if (!REFIT && valid[q] && col0 < bw) {
            const int64_t gi = (i0 + col0) / group;
            const int64_t gidx = row * n_groups + (gi < n_groups ? gi : n_groups - 1);
            S_mine[q] = LQ_AT(scale + gidx);
            Z_mine[q] = static_cast<float>(LQ_AT(zero + gidx));
        }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    if (tid < B) LQ_AT(invd + tid) = 1.0f / LQ_AT(Us + tid * B + tid);
    __syncthreads();
    // rows of the block scaled by the reciprocal of their diagonal entry: the column loop then feeds w - q straight
    // into the other columns, and only the lane that owns a column turns it into E = (w - q) / U_jj afterwards
    for (int idx = tid; idx < B * B / 4; idx += nthr) {
        const int jj = idx / (B / 4);
        float4* p4 = reinterpret_cast<float4*>(Us) + idx;
        float4 v = LQ_AT(p4);
        const float sc = LQ_AT(invd + jj);
        v.x *= sc; v.y *= sc; v.z *= sc; v.w *= sc;
        LQ_AT(p4) = v;
    }
    __syncthreads();
    if (!valid[0]) return;                 // rows are handed out in order: without the first a warp has none

    float dkeep[R][4];
    uint32_t cpack[R];
#pragma unroll
    for (int q = 0; q < R; ++q) {
        cpack[q] = 0;
#pragma unroll
        for (int u = 0; u < 4; ++u) dkeep[q][u] = 0.0f;
    }
    const int n_owner = (bw + 3) / 4;
#pragma unroll 1
    for (int jj = 0; jj < n_owner; ++jj) {
        float S[R], Zf[R], rS[R];
#pragma unroll
        for (int q = 0; q < R; ++q) { S[q] = 1.0f; Zf[q] = 0.0f; rS[q] = 1.0f; }
        if (REFIT && (i0 + 4 * jj) % group == 0) {
            // a group starts at this column: fit its (S, Z) by Eq. 7 on the group's weights as they stand now, with the
            // errors of every earlier column already fed back (the lanes that own the group hand their weights over)
            float* wtmp = invd + B + static_cast<size_t>(warp) * 3 * group;
            float2* ws = reinterpret_cast<float2*>(wtmp + group);
            const int gln = group / 4;                       // lanes per group
            if (lane >= jj && lane < jj + gln) {
#pragma unroll
                for (int u = 0; u < 4; ++u) LQ_AT(wtmp + 4 * (lane - jj) + u) = w[0][u];
            }
            __syncwarp();
            double Sd, Zd;
            lq_affine_warp_search([&](int j) { return LQ_AT(wtmp + j); }, refit.s64 + i0 + 4 * jj, group, ws, K, refit.T, refit.t_count, lane,
                                  Sd, Zd);
            if (lane >= jj && lane < jj + gln) { S_mine[0] = static_cast<float>(Sd); Z_mine[0] = static_cast<float>(static_cast<int32_t>(Zd)); }
            if (lane == jj) {
                const int64_t gidx = row0 * n_groups + (i0 + 4 * jj) / group;
                LQ_AT(refit.scale + gidx) = static_cast<float>(Sd);
                LQ_AT(refit.zero + gidx) = static_cast<int32_t>(Zd);
            }
            __syncwarp();
        }
        if (AFFINE) {
#pragma unroll
            for (int q = 0; q < R; ++q) {
                S[q] = __shfl_sync(0xffffffffu, S_mine[q], jj);
                Zf[q] = __shfl_sync(0xffffffffu, Z_mine[q], jj);
                rS[q] = __fdiv_rn(1.0f, S[q]);     // one division per four columns; w / S below is w * (1 / S)
            }
        }
        const bool mine = lane == jj;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int j = 4 * jj + u;
            float d[R];
#pragma unroll
            for (int q = 0; q < R; ++q) {
                const float wj = __shfl_sync(0xffffffffu, w[q][u], jj);
                int code;
                float qv;
                if (AFFINE) {
                    float qi = rintf(wj * rS[q]) + Zf[q];
                    qi = fminf(fmaxf(qi, 0.0f), static_cast<float>(K - 1));
                    code = static_cast<int>(qi);
                    qv = (qi - Zf[q]) * S[q];
                } else {
                    code = __popc(__ballot_sync(0xffffffffu, wj > ml[q]));
                    qv = __shfl_sync(0xffffffffu, gl[q], code);
                }
                d[q] = wj - qv;
                if (mine) {
                    dkeep[q][u] = d[q];
                    cpack[q] |= static_cast<uint32_t>(code) << (8 * u);
                }
            }
            const float4 uv = LQ_AT(reinterpret_cast<const float4*>(Us + j * B + col0));
#pragma unroll
            for (int q = 0; q < R; ++q) {
                w[q][0] = fmaf(-d[q], uv.x, w[q][0]);
                w[q][1] = fmaf(-d[q], uv.y, w[q][1]);
                w[q][2] = fmaf(-d[q], uv.z, w[q][2]);
                w[q][3] = fmaf(-d[q], uv.w, w[q][3]);
            }
        }
    }

#pragma unroll
    for (int q = 0; q < R; ++q) {
        if (!valid[q]) continue;            // the same for the whole warp
        const int64_t row = row0 + q;
        // this lane's four columns: grid values from the codes, E from w - q, and the row's share of the loss
        float qkeep[4], ekeep[4];
        float loss = 0.0f;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int code = static_cast<int>((cpack[q] >> (8 * u)) & 0xffu);
            if (AFFINE) qkeep[u] = (static_cast<float>(code) - Z_mine[q]) * S_mine[q];
            else qkeep[u] = __shfl_sync(0xffffffffu, gl[q], code);
            ekeep[u] = (col0 + u < bw) ? dkeep[q][u] * LQ_AT(invd + col0 + u) : 0.0f;
            loss = fmaf(ekeep[u], ekeep[u], loss);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) loss += __shfl_xor_sync(0xffffffffu, loss, o);
        // outputs of this lane's four columns
        if (col0 < bw) {
            const int64_t gcol = i0 + col0;
            if (col0 + 3 < bw && (c % 4 == 0)) {
                LQ_AT(reinterpret_cast<uint32_t*>(out.codes + row * c + gcol)) = cpack[q];
            } else {
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (col0 + u < bw) LQ_AT(out.codes + row * c + gcol + u) = static_cast<uint8_t>((cpack[q] >> (8 * u)) & 0xff);
            }
            if (out.what) {
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (col0 + u < bw) {
                        if (out.what_bf16) LQ_AT(static_cast<__nv_bfloat16*>(out.what) + row * out.ldwh + gcol + u) = __float2bfloat16_rn(qkeep[u]);
                        else LQ_AT(static_cast<float*>(out.what) + row * out.ldwh + gcol + u) = qkeep[u];
                    }
            }
        }
        {
            uint32_t ph[2], pm[2], pl[2];
#pragma unroll
            for (int t = 0; t < 4; t += 2) {
                __nv_bfloat16 h0, m0, l0, h1, m1, l1;
                lq_split3(ekeep[t], h0, m0, l0);
                lq_split3(ekeep[t + 1], h1, m1, l1);
                ph[t / 2] = static_cast<uint32_t>(__bfloat16_as_ushort(h0)) | (static_cast<uint32_t>(__bfloat16_as_ushort(h1)) << 16);
                pm[t / 2] = static_cast<uint32_t>(__bfloat16_as_ushort(m0)) | (static_cast<uint32_t>(__bfloat16_as_ushort(m1)) << 16);
                pl[t / 2] = static_cast<uint32_t>(__bfloat16_as_ushort(l0)) | (static_cast<uint32_t>(__bfloat16_as_ushort(l1)) << 16);
            }
            __nv_bfloat16* e0 = out.esplit + row * out.e_ld + out.e_col + col0;
            __nv_bfloat16* e1 = e0 + r * out.e_ld;
            __nv_bfloat16* e2 = e1 + r * out.e_ld;
            LQ_AT(reinterpret_cast<uint2*>(e0)) = make_uint2(ph[0], ph[1]);
            LQ_AT(reinterpret_cast<uint2*>(e1)) = make_uint2(pm[0], pm[1]);
            LQ_AT(reinterpret_cast<uint2*>(e2)) = make_uint2(pl[0], pl[1]);
        }
        if (lane == 0) LQ_AT(out.loss_rows + row) += static_cast<double>(loss);
    }
}

// Packed output: the b-bit codes of a row as one little-endian bit stream (code j in bits
// [j b, (j + 1) b) of the row), one thread per output byte.
__global__ void pack_codes_kernel(const uint8_t* __restrict__ codes, int64_t r, int64_t c, int bits,
                                  uint8_t* __restrict__ packed, int64_t ldp) {
    const int64_t row = blockIdx.y;
    const int64_t nbytes = (c * bits + 7) / 8;
    for (int64_t b = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; b < nbytes; b += (int64_t)gridDim.x * blockDim.x) {
        const int64_t bit0 = 8 * b;
        const int64_t j0 = bit0 / bits, j1 = (bit0 + 7) / bits;
        uint32_t acc = 0;
        for (int64_t j = j0; j <= j1 && j < c; ++j) {
            const int64_t sh = j * bits - bit0;                 // position of code j relative to this byte
            const uint32_t v = LQ_AT(codes + row * c + j) & ((1u << bits) - 1u);
            acc |= sh >= 0 ? (v << sh) : (v >> (-sh));
        }
        LQ_AT(packed + row * ldp + b) = static_cast<uint8_t>(acc & 0xffu);
    }
}

__global__ void zero_doubles_kernel(double* p, int64_t n) {
    const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (i < n) LQ_AT(p + i) = 0.0;
}

// loss_out[0] = 1/2 * sum_rows loss_rows
__global__ void loss_reduce_kernel(const double* __restrict__ loss_rows, int64_t r, double* __restrict__ loss_out) {
    __shared__ double red[1024];
    double s = 0.0;
    for (int64_t i = threadIdx.x; i < r; i += blockDim.x) s += LQ_AT(loss_rows + i);
    red[threadIdx.x] = s;
    __syncthreads();
    for (int o = blockDim.x / 2; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) loss_out[0] = 0.5 * red[0];
}

struct WsLayout {
    size_t wc, ut, es, loss, total;
    int64_t ldc, ldt;
};
WsLayout ws_layout(int64_t r, int64_t c) {
    WsLayout L;
    L.ldc = lq_ceil_div(c, 4) * 4;
    L.ldt = lq_ceil_div(c, 8) * 8;
    size_t off = 0;
    L.wc = off; off += lq_align_up(static_cast<size_t>(r) * L.ldc * sizeof(float), 256);
    L.ut = off; off += lq_align_up(static_cast<size_t>(3) * c * L.ldt * sizeof(__nv_bfloat16), 256);
    L.es = off; off += lq_align_up(static_cast<size_t>(3) * r * OB * sizeof(__nv_bfloat16), 256);
    L.loss = off; off += lq_align_up(static_cast<size_t>(r) * sizeof(double), 256);
    L.total = off;
    return L;
}

int check_cfg4(const lq_config* cfg) {
    if (!cfg) return LQ_ERR_INVALID_ARG;
    if (cfg->bits < 2 || cfg->bits > 4) return LQ_ERR_INVALID_ARG;
    if (cfg->block != B) return LQ_ERR_UNSUPPORTED;
    if (cfg->grid_type != LQ_GRID_NONUNIFORM && cfg->grid_type != LQ_GRID_AFFINE) return LQ_ERR_INVALID_ARG;
    return LQ_OK;
}

template <int K, bool AFFINE, bool REFIT, int ROWS>
int launch_inblock_rows(cudaStream_t st, int sm_count, float* Wc, int64_t ldc, int64_t r, int64_t c, int64_t i0, const float* U, int64_t ldu,
                        const float* grid, const float* scale, const int32_t* zero, int group, int n_groups, const QuantOut& out,
                        const RefitArgs& refit) {
    // What matters is the largest number of rows on one SM: up to 32 rows per SM one CTA per SM takes an even share;
    // beyond that, CTAs of 16 warps fill the SMs.
    int warps = 16;
    if (r <= (REFIT ? 16 : 32) * static_cast<int64_t>(sm_count)) {
        warps = static_cast<int>(lq_ceil_div(lq_ceil_div(r, sm_count), ROWS));
        if (warps < 4) warps = 4;                  // the 128 reciprocals of the diagonal are computed by the first 128 threads
    }
    const int smem = (B * B + B) * sizeof(float) + (REFIT ? warps * 3 * group * static_cast<int>(sizeof(float)) : 0);
    static lq_once_per_device attr_set;
    if (attr_set.first()) {
        LQ_CUDA_TRY(cudaFuncSetAttribute(inblock_kernel<K, AFFINE, REFIT, ROWS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (B * B + B) * static_cast<int>(sizeof(float)) + (REFIT ? 16 * 3 * B * static_cast<int>(sizeof(float)) : 0)));
    }
    inblock_kernel<K, AFFINE, REFIT, ROWS><<<static_cast<unsigned>(lq_ceil_div(r, static_cast<int64_t>(warps) * ROWS)), warps * 32, smem, st>>>(
        Wc, ldc, r, c, i0, U, ldu, grid, scale, zero, group, n_groups, out, refit);
    LQ_LAUNCH_CHECK();
    return LQ_OK;
}
// A warp carries two rows where an SM gets enough of them to stay busy that way (measured: 2 % faster at 28 rows per
// SM, 6 % at 360, 5 % slower at 14), and one where it refits groups inside the kernel.
template <int K, bool AFFINE, bool REFIT>
int launch_inblock(cudaStream_t st, int sm_count, float* Wc, int64_t ldc, int64_t r, int64_t c, int64_t i0, const float* U, int64_t ldu,
                   const float* grid, const float* scale, const int32_t* zero, int group, int n_groups, const QuantOut& out,
                   const RefitArgs& refit) {
    if (!REFIT && r >= 24 * static_cast<int64_t>(sm_count))
        return launch_inblock_rows<K, AFFINE, REFIT, REFIT ? 1 : IB_ROWS>(st, sm_count, Wc, ldc, r, c, i0, U, ldu, grid, scale, zero, group, n_groups, out, refit);
    return launch_inblock_rows<K, AFFINE, REFIT, 1>(st, sm_count, Wc, ldc, r, c, i0, U, ldu, grid, scale, zero, group, n_groups, out, refit);
}

}  // namespace

extern "C" int lq_quantize_layer_workspace(const lq_config* cfg, int64_t r, int64_t c, size_t* bytes) {
    int e = check_cfg4(cfg);
    if (e) return e;
    if (!bytes || r <= 0 || c <= 0) return LQ_ERR_INVALID_ARG;
    *bytes = ws_layout(r, c).total;
    return LQ_OK;
}

namespace {
// Whether the (S, Z) of a group can be refitted when the column loop reaches it: by then every earlier block's errors
// must have reached all of the group's columns, which the two-level update guarantees for groups that tile a
// 1024-column outer block, for groups made of whole outer blocks, and trivially for one group per row.
bool lazy_group_ok(int64_t g, int64_t c) {
    if (g == c) return true;
    if (g < B) return g % 4 == 0 && B % g == 0;        // inside a block: refitted by the in-block kernel itself
    if (g % B) return false;
    return (g <= OB && OB % g == 0) || (g % OB == 0);
}

// dinv != nullptr selects the lazy refit: scale / zero are then outputs, filled group by group as the loop goes.
int quantize_impl(lq_handle* h, void* stream, const lq_config* cfg, const void* W, int32_t w_dtype,
                  int64_t r, int64_t c, int64_t ldw, const float* U, int64_t ldu, const float* grid,
                  float* scale, int32_t* zero, const float* dinv, uint8_t* codes, void* W_hat,
                  int32_t what_dtype, int64_t ldwh, double* loss_out, void* ws, size_t ws_bytes) {
    int e = check_cfg4(cfg);
    if (e) return e;
    if (!h || !W || !U || !codes || r <= 0 || c <= 0 || ldw < c || ldu < c) return LQ_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(U) & 15) || (reinterpret_cast<uintptr_t>(codes) & 15)) return LQ_ERR_INVALID_ARG;
    if (w_dtype != LQ_F32 && w_dtype != LQ_BF16) return LQ_ERR_INVALID_ARG;
    if (W_hat && (ldwh < c || (what_dtype != LQ_F32 && what_dtype != LQ_BF16))) return LQ_ERR_INVALID_ARG;
    const bool affine = cfg->grid_type == LQ_GRID_AFFINE;
    int group = 0, n_groups = 1;
    if (affine) {
        if (!scale || !zero) return LQ_ERR_INVALID_ARG;
        const int64_t g = cfg->group_size == 0 ? c : cfg->group_size;
        if (c % g) return LQ_ERR_INVALID_ARG;
        if (g != c && (g % 4)) return LQ_ERR_UNSUPPORTED;      // a lane's four columns share one (S, Z)
        if (g > 0x7fffffffLL) return LQ_ERR_UNSUPPORTED;
        group = static_cast<int>(g);
        n_groups = static_cast<int>(c / g);
    } else if (!grid) {
        return LQ_ERR_INVALID_ARG;
    }
    const WsLayout L = ws_layout(r, c);
    const bool lazy = dinv != nullptr;
    const size_t lazy_bytes = lazy ? 256 + lq_align_up(static_cast<size_t>(c) * sizeof(double), 256) : 0;
    if (!ws || ws_bytes < L.total + lazy_bytes) return LQ_ERR_WORKSPACE_TOO_SMALL;
    if (reinterpret_cast<uintptr_t>(ws) & 255) return LQ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char* wsp = static_cast<char*>(ws);
    double* s64 = nullptr;
    if (lazy) {
        if (!affine) return LQ_ERR_INVALID_ARG;
        if (cfg->T <= 0 || cfg->t_count < 0 || 2 * static_cast<int64_t>(cfg->t_count) > cfg->T || cfg->t_count > 4095) return LQ_ERR_INVALID_ARG;
        if (!lazy_group_ok(group, c) || static_cast<size_t>(group) * sizeof(float) > 200 * 1024) return LQ_ERR_UNSUPPORTED;
        s64 = reinterpret_cast<double*>(wsp + L.total + 256);
        e = lq_sample_weights(h, st, dinv, c, static_cast<double>(cfg->p), reinterpret_cast<double*>(wsp + L.total), s64);
        if (e) return e;
    }
    {
        LQ_DBG_SCOPE(h, st);
        const size_t wb = w_dtype == LQ_F32 ? 4 : 2;
        LQ_DBG_REG(W, (static_cast<size_t>(r - 1) * ldw + c) * wb);
        LQ_DBG_REG(U, (static_cast<size_t>(c - 1) * ldu + c) * sizeof(float));
        LQ_DBG_REG(ws, L.total + lazy_bytes);
        LQ_DBG_REG(codes, static_cast<size_t>(r) * c);
        if (W_hat) LQ_DBG_REG(W_hat, (static_cast<size_t>(r - 1) * ldwh + c) * (what_dtype == LQ_F32 ? 4 : 2));
        if (grid) LQ_DBG_REG(grid, static_cast<size_t>(r) * (size_t(1) << cfg->bits) * sizeof(float));
        if (scale) LQ_DBG_REG(scale, static_cast<size_t>(r) * n_groups * sizeof(float));
        if (zero) LQ_DBG_REG(zero, static_cast<size_t>(r) * n_groups * sizeof(int32_t));
        if (loss_out) LQ_DBG_REG(loss_out, sizeof(double));
        LQ_DBG_COMMIT();
    }
    float* Wc = reinterpret_cast<float*>(wsp + L.wc);
    __nv_bfloat16* UT = reinterpret_cast<__nv_bfloat16*>(wsp + L.ut);
    __nv_bfloat16* ES = reinterpret_cast<__nv_bfloat16*>(wsp + L.es);
    double* loss_rows = reinterpret_cast<double*>(wsp + L.loss);

    // 16-byte accesses when rows of W start on 16-byte boundaries (the working copy's always do)
    const int vec = ((reinterpret_cast<uintptr_t>(W) & 15) == 0 && (ldw * (w_dtype == LQ_F32 ? 4 : 2)) % 16 == 0) ? 1 : 0;
    for (int64_t r0 = 0; r0 < r; r0 += 65535) {          // rows in slabs: the second grid dimension holds 65535 at most
        const int64_t rr = r - r0 < 65535 ? r - r0 : 65535;
        dim3 g(static_cast<unsigned>(lq_ceil_div(L.ldc, 256) < 32 ? lq_ceil_div(L.ldc, 256) : 32), static_cast<unsigned>(rr));
        if (w_dtype == LQ_F32)
            to_f32_kernel<float><<<g, 256, 0, st>>>(static_cast<const float*>(W) + r0 * ldw, ldw, c, Wc + r0 * L.ldc, L.ldc, vec);
        else
            to_f32_kernel<__nv_bfloat16><<<g, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(W) + r0 * ldw, ldw, c, Wc + r0 * L.ldc,
                                                           L.ldc, vec);
        LQ_LAUNCH_CHECK();
    }
    if (c > B) {
        dim3 g(static_cast<unsigned>(lq_ceil_div(c, 64)), static_cast<unsigned>(lq_ceil_div(L.ldt, 64)));
        split_transpose_kernel<<<g, 256, 0, st>>>(U, ldu, c, UT, L.ldt);
        LQ_LAUNCH_CHECK();
    }
    zero_doubles_kernel<<<static_cast<unsigned>(lq_ceil_div(r, 256)), 256, 0, st>>>(loss_rows, r);
    LQ_LAUNCH_CHECK();

    QuantOut out;
    out.codes = codes;
    out.what = W_hat;
    out.what_bf16 = (what_dtype == LQ_BF16);
    out.ldwh = ldwh;
    out.esplit = ES;
    out.e_ld = OB;
    out.e_col = 0;
    out.loss_rows = loss_rows;

    for (int64_t i0 = 0; i0 < c; i0 += B) {
        int rc;
        const int64_t o0 = i0 / OB * OB;          // start of the outer block
        out.e_col = static_cast<int>(i0 - o0);
        const bool refit_inside = lazy && group < B;     // groups shorter than a block are refitted by the in-block kernel
        if (lazy && !refit_inside && i0 % group == 0) {  // (S, Z) of the group that starts here, on the columns as they stand now
            rc = lq_affine_search(h, st, Wc + i0, LQ_F32, r, L.ldc, group, 1, s64 + i0, 1 << cfg->bits, cfg->T, cfg->t_count,
                                  scale + i0 / group, zero + i0 / group, n_groups);
            if (rc) return rc;
        }
        RefitArgs refit = {};
        if (refit_inside) { refit.s64 = s64; refit.scale = scale; refit.zero = zero; refit.T = cfg->T; refit.t_count = cfg->t_count; }
#define LQ_IB(KK, AFF, RF) launch_inblock<KK, AFF, RF>(st, h->sm_count, Wc, L.ldc, r, c, i0, U, ldu, grid, scale, zero, group, n_groups, out, refit)
        if (refit_inside) {
            switch (cfg->bits) {
                case 2: rc = LQ_IB(4, true, true); break;
                case 3: rc = LQ_IB(8, true, true); break;
                default: rc = LQ_IB(16, true, true); break;
            }
        } else if (affine) {
            switch (cfg->bits) {
                case 2: rc = LQ_IB(4, true, false); break;
                case 3: rc = LQ_IB(8, true, false); break;
                default: rc = LQ_IB(16, true, false); break;
            }
        } else {
            switch (cfg->bits) {
                case 2: rc = LQ_IB(4, false, false); break;
                case 3: rc = LQ_IB(8, false, false); break;
                default: rc = LQ_IB(16, false, false); break;
            }
        }
#undef LQ_IB
        if (rc) return rc;
        // Lazy update (Algorithm 1 line 20) in two levels.  The columns that the next blocks of
        // this outer block are about to quantise get this block's errors now (K = 128); the columns
        // beyond the outer block get the errors of all its blocks in one product once it is complete
        // (K = 1024), which cuts the read-modify-write traffic on the working copy eightfold.  The
        // result is the same sum in a different order.
        const int64_t ob_end = (o0 + OB < c) ? o0 + OB : c;
        const int64_t ao[6] = {0, 0, r, 0, 2 * r, r};
        const int64_t bo[6] = {0, c, 0, 2 * c, 0, c};
        const int64_t near = ob_end - (i0 + B);
        if (near > 0) {
            lq_tc_gemm_args g = {};
            g.A_all = ES + (i0 - o0); g.a_rows = 3 * r; g.lda = OB;
            g.B_all = UT + (i0 + B) * L.ldt + i0; g.b_rows = 3 * c - (i0 + B); g.ldb = L.ldt;
            g.D = Wc + (i0 + B); g.ldd = L.ldc;
            g.M = r; g.N = near; g.K = B;
            g.n_pass = 6;
            for (int i = 0; i < 6; ++i) { g.a_row_off[i] = ao[i]; g.b_row_off[i] = bo[i]; }
            g.alpha = -1.0f; g.accumulate = 1; g.upper_only = 0;
            rc = lq_tc_gemm(h, st, g);
            if (rc) return rc;
        }
        if (i0 + B >= ob_end && ob_end < c) {
            lq_tc_gemm_args g = {};
            g.A_all = ES; g.a_rows = 3 * r; g.lda = OB;
            g.B_all = UT + ob_end * L.ldt + o0; g.b_rows = 3 * c - ob_end; g.ldb = L.ldt;
            g.D = Wc + ob_end; g.ldd = L.ldc;
            g.M = r; g.N = c - ob_end; g.K = ob_end - o0;
            g.n_pass = 6;
            for (int i = 0; i < 6; ++i) { g.a_row_off[i] = ao[i]; g.b_row_off[i] = bo[i]; }
            g.alpha = -1.0f; g.accumulate = 1; g.upper_only = 0;
            g.seg_iters = 12;          // partial sums leave the tensor core's truncating accumulator every 128 columns
            rc = lq_tc_gemm(h, st, g);
            if (rc) return rc;
        }
    }
    if (loss_out) {
        loss_reduce_kernel<<<1, 1024, 0, st>>>(loss_rows, r, loss_out);
        LQ_LAUNCH_CHECK();
    }
    return LQ_OK;
}
}  // namespace

extern "C" int lq_quantize_layer(lq_handle* h, void* stream, const lq_config* cfg, const void* W, int32_t w_dtype,
                                 int64_t r, int64_t c, int64_t ldw, const float* U, int64_t ldu, const float* grid,
                                 const float* scale, const int32_t* zero, uint8_t* codes, void* W_hat,
                                 int32_t what_dtype, int64_t ldwh, double* loss_out, void* ws, size_t ws_bytes) {
    return quantize_impl(h, stream, cfg, W, w_dtype, r, c, ldw, U, ldu, grid, const_cast<float*>(scale), const_cast<int32_t*>(zero),
                         nullptr, codes, W_hat, what_dtype, ldwh, loss_out, ws, ws_bytes);
}

extern "C" int lq_quantize_layer_lazy_workspace(const lq_config* cfg, int64_t r, int64_t c, size_t* bytes) {
    int e = lq_quantize_layer_workspace(cfg, r, c, bytes);
    if (e) return e;
    *bytes += 256 + lq_align_up(static_cast<size_t>(c) * sizeof(double), 256);
    return LQ_OK;
}

extern "C" int lq_quantize_layer_lazy(lq_handle* h, void* stream, const lq_config* cfg, const void* W, int32_t w_dtype,
                                      int64_t r, int64_t c, int64_t ldw, const float* U, int64_t ldu, const float* dinv,
                                      float* scale, int32_t* zero, uint8_t* codes, void* W_hat, int32_t what_dtype,
                                      int64_t ldwh, double* loss_out, void* ws, size_t ws_bytes) {
    if (!dinv || !cfg || cfg->grid_type != LQ_GRID_AFFINE) return LQ_ERR_INVALID_ARG;
    return quantize_impl(h, stream, cfg, W, w_dtype, r, c, ldw, U, ldu, nullptr, scale, zero, dinv, codes, W_hat, what_dtype, ldwh,
                         loss_out, ws, ws_bytes);
}

extern "C" int lq_pack_codes(lq_handle* h, void* stream, const uint8_t* codes, int64_t r, int64_t c, int32_t bits,
                             uint8_t* packed, int64_t ldp) {
    if (!h || !codes || !packed || r <= 0 || c <= 0 || bits < 1 || bits > 8) return LQ_ERR_INVALID_ARG;
    const int64_t nbytes = (c * bits + 7) / 8;
    if (ldp < nbytes) return LQ_ERR_INVALID_ARG;
    if (r > 65535) {                       // grid.y limit: rows in slabs
        for (int64_t r0 = 0; r0 < r; r0 += 65535) {
            const int64_t rr = r - r0 < 65535 ? r - r0 : 65535;
            int rc = lq_pack_codes(h, stream, codes + r0 * c, rr, c, bits, packed + r0 * ldp, ldp);
            if (rc) return rc;
        }
        return LQ_OK;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    {
        LQ_DBG_SCOPE(h, st);
        LQ_DBG_REG(codes, static_cast<size_t>(r) * c);
        LQ_DBG_REG(packed, static_cast<size_t>(r - 1) * ldp + nbytes);
        LQ_DBG_COMMIT();
    }
    dim3 g(static_cast<unsigned>(lq_ceil_div(nbytes, 256) < 64 ? lq_ceil_div(nbytes, 256) : 64), static_cast<unsigned>(r));
    pack_codes_kernel<<<g, 256, 0, st>>>(codes, r, c, bits, packed, ldp);
    LQ_LAUNCH_CHECK();
    return LQ_OK;
}
