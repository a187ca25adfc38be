// The search of Eq. 7 for one group of weights by one warp: shared between stage 3 (lq_fit_grid.cu) and the column
// loop's refit of groups shorter than a block (lq_quantize.cu).
#pragma once

#include <math.h>

#include "lq_common.cuh"

// ------------------------------------------------------- fp32 screening of candidates --
// Both searches below score a candidate (S, Z) in fp32 first and evaluate in fp64 only those whose
// score cannot be told from the best one.  With x = w - min:  w / S + Z = x / S + c0,  c0 = min / S + Z
// (both divided by K - 1 in AffScore, so that the clamp to [0, K - 1] is a saturation),
// and the error of a weight is d = q S - x - beta,  beta = min + Z S.
struct AffScore { float rS, c0, Sh, beta; };

__device__ __forceinline__ AffScore aff_score_setup(double S, double Z, double dmn, double Km1) {
    AffScore a;
    const double rS = 1.0 / S;
    a.rS = static_cast<float>(rS / Km1);                 // u / (K - 1) = x rS + c0, saturated to [0, 1] in aff_score32
    a.c0 = static_cast<float>((dmn * rS + Z) / Km1);
    a.Sh = static_cast<float>(S);
    a.beta = static_cast<float>(dmn + Z * S);
    return a;
}

// sum_j s_j d_j^2 over the (x, s) pairs of a group (group even)
__device__ __forceinline__ float aff_score32(const float2* __restrict__ ws, int group, const AffScore& a, float Km1f) {
    float a0 = 0.0f, a1 = 0.0f;
    for (int j = 0; j < group; j += 2) {
        const float4 p2 = LQ_AT(reinterpret_cast<const float4*>(ws + j));    // two (x, s) pairs
        // clamp to [0, K - 1] and round: the clamp rides on the multiply-add as a saturation of u / (K - 1) to [0, 1]
        // (a weight within rounding of a tie may take the other neighbour, which leaves its error where it was)
        const float q0 = rintf(__saturatef(fmaf(p2.x, a.rS, a.c0)) * Km1f);
        const float q1 = rintf(__saturatef(fmaf(p2.z, a.rS, a.c0)) * Km1f);
        const float d0 = fmaf(q0, a.Sh, -p2.x) - a.beta;
        const float d1 = fmaf(q1, a.Sh, -p2.z) - a.beta;
        a0 = fmaf(p2.y * d0, d0, a0);
        a1 = fmaf(p2.w * d1, d1, a1);
    }
    return a0 + a1;
}

// Scores up to this bar are re-examined in fp64.  The fp32 value of d carries an absolute error of at most
// delta = 2.2e-7 R: roundings of x, of beta and of the intermediate q S - x, each below 2^-25 of a quantity
// bounded by R or 1.5 R, plus q times the rounding of S to fp32 (q <= K - 1, S <= R / (K - 1): below 2^-24 R).
// Hence |score - loss| <= 2 delta sqrt(sum_s loss) + delta^2 sum_s (Cauchy-Schwarz); the 0.1 % on top covers the
// rounding of the sum itself.  When the loss is far above delta^2 sum_s, as it is unless a few heavy weights are
// met almost exactly, the bar is 0.1 % above the best score.  (A weight within the fp32 error of u of a rounding tie,
// ~1e-5, may be given the other neighbour: its error is then S / 2 either way, up to that 1e-5 relative.)
__device__ __forceinline__ float aff_bar32(float best, float R, float sum_s) {
    const float delta = 2.2e-7f * R;
    const float A = delta * delta * sum_s;
    const float E = 2.0f * sqrtf(A * best) + A;
    return best * 1.001f + 2.5f * E;
}


// One warp, one group.  w_at(j) gives weight j of the group as float; sp its sample weights; ws: `group` float2 slots of
// shared memory owned by this warp.  Lanes take candidates (t_min, t_max); every candidate is first scored in fp32,
// only the candidates whose score lies below aff_bar32 of the best score are then evaluated in fp64 with exactly the
// arithmetic of Eq. 7, in candidate order by the whole warp, so the arg-min (first minimum in t_min-major order) is that
// of the all-fp64 search.  On return every lane holds (S, Z).
template <typename WAt>
__device__ __forceinline__ void lq_affine_warp_search(WAt w_at, const double* __restrict__ sp, int group, float2* ws, int K,
                                                      int Tparts, int t_count, int lane, double& S_out, double& Z_out) {
    float mn = INFINITY, mx = -INFINITY;
    double smax = 0.0, ssum = 0.0;
    for (int j = lane; j < group; j += 32) {
        const float w = w_at(j);
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
    const double sinv = smax > 0.0 ? 1.0 / smax : 1.0;
    const float sum_s = static_cast<float>(ssum * sinv);
    for (int j = lane; j < group; j += 32) LQ_AT(ws + j) = make_float2(w_at(j) - mn, static_cast<float>(LQ_AT(sp + j) * sinv));
    __syncwarp();

    const double dmn = mn, dmx = mx, R = dmx - dmn;
    const double Km1 = static_cast<double>(K - 1);
    if (R == 0.0) {                                // constant group
        double lo = fmin(dmn, 0.0), hi = fmax(dmx, 0.0);
        double S = 1.0, Z = 0.0;
        if (hi != lo) { S = (hi - lo) / Km1; Z = -rint(lo / S); }
        S_out = S; Z_out = Z;
        return;
    }

    const int side = t_count + 1;
    const int n_cand = side * side;
    const float Km1f = static_cast<float>(K - 1);
    // (S, Z) of a candidate exactly as Eq. 7 gives them; false when the candidate is void
    auto params = [&](int cand, double& S, double& Z) {
        const int t_min = cand / side, t_max = cand - t_min * side;
        const double lo = dmn + static_cast<double>(t_min) * R / static_cast<double>(Tparts);
        const double hi = dmx - static_cast<double>(t_max) * R / static_cast<double>(Tparts);
        S = (hi - lo) / Km1;
        if (!(S > 0.0)) return false;
        Z = -rint(lo / S);
        return true;
    };
    auto score32 = [&](double S, double Z) { return aff_score32(ws, group, aff_score_setup(S, Z, dmn, Km1), Km1f); };
    // fp64 loss of one candidate, computed by the whole warp (lane l takes weights l, l + 32, ...)
    auto loss64 = [&](double S, double Z) {
        double loss = 0.0;
        for (int j = lane; j < group; j += 32) {
            const double w = static_cast<double>(w_at(j));
            double q = rint(w / S) + Z;
            q = fmin(fmax(q, 0.0), Km1);
            const double d = (q - Z) * S - w;
            loss += LQ_AT(sp + j) * (d * d);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) loss += __shfl_xor_sync(0xffffffffu, loss, o);
        return loss;
    };

    // pass 1: fp32 scores of all candidates and their minimum over the warp
    constexpr int KEEP = 8;                        // scores kept in registers when there are at most 32 * KEEP candidates
    const bool keep = n_cand <= 32 * KEEP;
    float sc[KEEP];
    float best32 = INFINITY;
    if (keep) {
#pragma unroll
        for (int rd = 0; rd < KEEP; ++rd) {
            const int cand = lane + 32 * rd;
            double S, Z;
            sc[rd] = (cand < n_cand && params(cand, S, Z)) ? score32(S, Z) : INFINITY;
            if (sc[rd] != sc[rd]) sc[rd] = -INFINITY;          // a NaN score is always re-examined in fp64
            best32 = fminf(best32, sc[rd] == -INFINITY ? INFINITY : sc[rd]);
        }
    } else {
        for (int cand = lane; cand < n_cand; cand += 32) {
            double S, Z;
            if (!params(cand, S, Z)) continue;
            best32 = fminf(best32, score32(S, Z));             // fminf ignores a NaN
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) best32 = fminf(best32, __shfl_xor_sync(0xffffffffu, best32, o));
    const float bar32 = aff_bar32(best32, static_cast<float>(R), sum_s);

    // pass 2: candidates whose score is below the bar are evaluated in fp64, one at a time
    // in candidate order by the whole warp, so the first minimum wins and every lane holds the result
    double my_loss = INFINITY;
    int my_idx = 0x7fffffff;
    const int rounds = (n_cand + 31) / 32;
    for (int rd = 0; rd < rounds; ++rd) {
        const int cand = lane + 32 * rd;
        bool want = false;
        if (keep) {
            float v = INFINITY;
#pragma unroll
            for (int k = 0; k < KEEP; ++k) v = (k == rd) ? sc[k] : v;
            want = cand < n_cand && v <= bar32;
        } else {
            double S, Z;
            if (cand < n_cand && params(cand, S, Z)) want = !(score32(S, Z) > bar32);      // true for a NaN score
        }
        uint32_t todo = __ballot_sync(0xffffffffu, want);
        while (todo) {
            const int src = __ffs(todo) - 1;
            todo &= todo - 1;
            double S, Z;
            if (!params(src + 32 * rd, S, Z)) continue;
            const double loss = loss64(S, Z);
            if (loss < my_loss) { my_loss = loss; my_idx = src + 32 * rd; }
        }
    }
    double S = 1.0, Z = 0.0;
    if (my_idx != 0x7fffffff) params(my_idx, S, Z);
    S_out = S; Z_out = Z;
}
