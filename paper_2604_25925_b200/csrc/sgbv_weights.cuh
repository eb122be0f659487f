// Acceptance weights of the multi-draft greedy block verifier (Eq. 2 and Eq. 3, float64) and the scan of
// Algorithm 1, shared by the finishing kernels of the one-device path and of the vocabulary-sharded path.
#pragma once

#include "sgbv_common.cuh"

namespace sgbv {

// 1 - (1-u)^K as the geometric sum u (1 + (1-u) + ... + (1-u)^(K-1)): all terms are positive, so
// a tiny u keeps its full relative accuracy, and no transcendental function is needed.
__device__ __forceinline__ double gfun(double u, int K) {
    if (u >= 1.0) return 1.0;
    if (!(u > 0.0)) return 0.0;
    const double v = 1.0 - u;
    double sum = 1.0;
    for (int j = 1; j < K; ++j) sum = fma(sum, v, 1.0);
    return u * sum;
}

__device__ __forceinline__ double clamp01(double x) {
    if (!(x > 0.0)) return 0.0;
    return x > 1.0 ? 1.0 : x;
}

// Eq. 2 from the three cached sums of the row that follows the sub-block (all divided by Zq):
//   R = sum_x q (1 - min{c p/q,1})^K,  Dp = sum_x max(c p - q, 0),  M = sum_x q (c-t)^2 Q(t).
// numerator/a   = R                                  (c >= 1)
//               = M + K (1-c)^(K-1) Dp               (c <  1, `exact`; equals R - (1-c)^K term by term)
//               = R - (1-c)^K                        (c <  1, not `exact`: only where plain_form_is_safe says so)
// denominator/a = numerator/a + g(b)/a - g(min(c,1))
static __device__ double weight_sub(double la, double lb, double R, double Dp, double M, int K, bool below_one, bool exact) {
    const double a = exp_short(la), b = exp_short(lb), c = exp_short(lb - la);
    const double gb = gfun(b, K);
    if (!(a > 0.0)) return gb > 0.0 ? 0.0 : 1.0;
    double num, extra;
    if (below_one) {  // decided on the float32 c the reduction pass used
        double pw = 1.0;
        for (int j = 1; j < K; ++j) pw *= (1.0 - c);
        num = exact ? M + (double)K * pw * Dp : fmax(R - pw * (1.0 - c), 0.0);
        extra = (K == 1) ? 0.0 : gb / a - gfun(c, K);
    } else {
        num = R;
        extra = gb / a - 1.0;
    }
    if (extra < 0.0) extra = 0.0;
    const double den = num + extra;
    if (!(den > 1e-12 * (gb / a + 1.0))) return 1.0;  // 0/0: accept, as single-draft GBV does
    return clamp01(num / den);
}

// For c < 1 the numerator of Eq. 2 over a is R - (1-c)^K, a difference of two numbers of which R carries the rounding
// of a float32 vocabulary sum (a few 1e-7 relative).  As long as (1-c)^K is at most half of R the difference loses at
// most one bit of that; beyond (p close to q on the part of the vocabulary that matters) the sums Dp and M, whose
// terms are all non-negative, are needed.
static __device__ bool plain_form_is_safe(double R, double c, int K) {
    double pw = 1.0;
    for (int j = 0; j < K; ++j) pw *= (1.0 - c);
    return pw <= 0.5 * R;
}

// Eq. 3.
static __device__ double weight_full(double la, double lb, int K) {
    const double a = exp_short(la), b = exp_short(lb);
    double c = exp_short(lb - la);
    if (!(a > 0.0) || c > 1.0) c = 1.0;
    const double den = gfun(b, K);
    if (!(den > 0.0)) return 0.0;
    return clamp01(a * gfun(c, K) / den);
}

// Algorithm 1's scan over drafts and lengths by one warp (all 32 lanes call).  pass_s[k]: bit i-1 is set when the
// trial of length i of draft k succeeds (eta < h); lcp_s[k*K+k']: longest common prefix of drafts k and k';
// sh_or: two words of shared memory.  Every lane returns the accepted length tau and the draft f (-1 if none).
static __device__ void scan_block(const unsigned long long *pass_s, const unsigned char *lcp_s, int K, int g,
                                  unsigned *sh_or, int &tau, int &f) {
    const int lane = threadIdx.x & 31;
    // The state is bit sets over the lengths 1..gamma (bit i-1 = length i): pass (shared memory, left by
    // the weights above) = the lengths whose Bernoulli trial succeeds (eta < h); rej (registers, lane l
    // owns drafts l and l + 32) = the lengths at which the draft entered H.  A draft's walk over i = tau+1..gamma does not
    // depend on its own progress (the start is fixed when the draft is entered, H only holds earlier
    // drafts), so it is evaluated for all lengths at once: the accepted length is the largest one in
    // the range whose trial passes and whose sub-block is not in H.
    auto low = [](int l) { return l >= 64 ? ~0ull : (1ull << l) - 1ull; };  // lengths 1..l
    unsigned long long rej0 = 0, rej1 = 0;
    tau = 0;
    f = -1;
    for (int k = 0; k < K; ++k) {
        const unsigned long long passk = pass_s[k];
        // common prefix of draft k with this lane's drafts; only earlier drafts can be in H
        const int l0 = (lane < k) ? lcp_s[k * K + lane] : 0;
        const int l1 = (lane + 32 < k) ? lcp_s[k * K + lane + 32] : 0;
        // lengths at which an earlier draft with the same prefix of that length entered H
        const unsigned long long mine = (rej0 & low(l0)) | (rej1 & low(l1));
        // union over the lanes, through shared memory
        if (lane == 0) sh_or[0] = sh_or[1] = 0u;
        __syncwarp();
        if ((unsigned)mine) atomicOr(&sh_or[0], (unsigned)mine);
        if ((unsigned)(mine >> 32)) atomicOr(&sh_or[1], (unsigned)(mine >> 32));
        __syncwarp();
        const unsigned long long inH = ((unsigned long long)sh_or[1] << 32) | (unsigned long long)sh_or[0];
        __syncwarp();
        const unsigned long long range = low(g) & ~low(tau);  // lengths tau+1..gamma
        const unsigned long long acc = passk & ~inH & range;
        const unsigned long long rejk = range & ~acc;
        if (acc != 0ull) {
            tau = 64 - __clzll((long long)acc);
            f = k;
        }
        if (lane == (k & 31)) {
            if (k < 32) rej0 = rejk;
            else rej1 = rejk;
        }
        if (tau == g) break;  // the whole block was accepted
    }
}

}  // namespace sgbv
