// Shared device-side definitions of the verify path: workspace layout, per-row records and the
// element arithmetic of the coupling sums (Eq. 2's vocabulary sum / Eq. 4's weights).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/sgbv.h"

namespace sgbv {

// Batches of at most this many rows: the finishing kernel (one CTA per row) leaves most SMs idle, so the next
// call's streaming kernel is allowed onto them while it runs (programmatic dependent launch across calls).
constexpr int kChainedLaunchMaxB = 16;
constexpr int kRatioWords = 256;   // ratio words at the head of the scratch: the row walk needs one per row and
                                   // only runs while every row has a cluster of its own in one wave (<= 148)
constexpr int kTile = 256;         // vocabulary elements per tile (granularity of the cached partial sums)
constexpr int kMaxK = 64;
constexpr int kMaxGamma = 64;
constexpr int kMaxV = 1 << 22;
constexpr float kLog2e = 1.4426950408889634f;

// Per (b,k,i) row pair, i < gamma.  Written by the statistics pass, read by the reduction pass
// and by the finishing kernel.
struct RowInfo {
    double Zq;      // sum_x exp((zq_x - mq)/T)
    double Zp;
    float mq;       // row maxima of the raw logits
    float mp;
    float kappa;    // c * Zq / Zp with c = b/a: ratio c*p(x)/q(x) = kappa * ep/eq in row-max units
    float c;        // c = p(x_k^i)/q(x_k^i), ratio of the joint prefix probabilities (c < 1 selects
                    // the cancellation-free numerator)
    int32_t flags;  // SGBV_STATUS_NONFINITE_LOGIT if the streaming pass found the row pair unusable
    int32_t pad_;   // 1: dpart/mpart hold this row's extra sums although only some rows have them (Workspace::have_aux = 2)
};

struct Workspace {
    RowInfo *rows;      // [B*K*gamma]
    float *part;        // [B*K*gamma][nsplit][4]: slice partials (mq, Zq, mp, Zp)   (two-pass path)
    float *wpart;       // [B*K*gamma][ntiles]: sum over the tile of eq * max(1 - kappa ep/eq, 0)^K
    float *dpart;       // [B*K*gamma][ntiles]: sum of max(kappa ep - eq, 0)               (c < 1)
    float *mpart;       // [B*K*gamma][ntiles]: sum of eq (c - t)^2 Q(t)                    (c < 1)
    double *ratio;      // [kRatioWords]: p_i(tok_i)/q_i(tok_i) of each row (row walk of the fused kernel, which
                        // only runs when B*K*gamma <= kRatioWords); every word holds a NaN pattern ("not
                        // published yet") whenever no call is in flight
    double *cut;        // [B*cpr]: c handed from the cluster that walks the head of a chain to the one that walks its tail
                        // (chain walk of the fused kernel; preset to the NaN pattern when any range cuts a chain)
    int have_aux;       // which rows with c < 1 have their two extra sums in dpart and mpart: 1 = all of them (two-sweep
                        // path, row walk of the fused kernel), 2 = those marked RowInfo::pad_ = 1 (chain walk of the fused
                        // kernel followed by auxreduce_kernel); the others take the plain form of Eq. 2's numerator
    int ratio_used;     // the streaming kernel walked rows: the finishing kernel puts the NaN pattern back
    float *bonus;       // [B][2][ntiles]: per-tile sums and maxima of the row a bonus token is drawn from
    int bonus_in_smem;  // set by the finishing kernel's launcher: those tile sums fit its shared memory
    double *h;          // [B][K][gamma]
    double *resmass;    // [B][K][gamma]
    int32_t *status;    // [B]: final per-row status, written by the finishing kernel
    int32_t *prestatus; // [B] bits set by earlier kernels with atomics (zeroed first), or NULL when the
                        // streaming pass reports through RowInfo::flags instead
    int32_t *error;     // [1]: set when a bounded device-side wait expired
};

struct Shape {
    int B, K, gamma, V;
    int cpr;      // draft chains per batch row: K for the verify step, 1 for Algorithm 2 (K is then only the exponent)
    int zq_rows;  // rows of the target tensor per chain: gamma + 1 for the verify step, 1 for Algorithm 2
    int ntiles;   // ceil(V / kTile)
    int nsplit;   // slices per row in the two-pass path
    int tiles_per_slice;
    float scale;  // log2(e) / T
    double inv_T;
};

template <typename T>
__device__ __forceinline__ float ld_logit(const T *p, size_t i);
template <>
__device__ __forceinline__ float ld_logit<float>(const float *p, size_t i) {
    return __ldg(p + i);
}
template <>
__device__ __forceinline__ float ld_logit<uint16_t>(const uint16_t *p, size_t i) {
    return __uint_as_float(((uint32_t)__ldg(p + i)) << 16);
}

// exp((z - m)/T) as 2^((z-m)*scale).
__device__ __forceinline__ float expo(float z, float m, float scale) { return exp2f((z - m) * scale); }

// One vocabulary element of the coupling sums, in row-max units (eq = exp((zq-mq)/T) etc.).
//   w  = eq * max(1 - kappa*ep/eq, 0)^K       -> sum/Zq = R_i, and w is Eq. 4's weight
//   dp = max(kappa*ep - eq, 0)                 -> sum/Zq = sum_x max(c p - q, 0)
//   m2 = eq * (c - t)^2 * Q(t), t = min(kappa*ep/eq, 1),
//        Q(t) = sum_{m=0}^{K-2} (K-1-m) (1-c)^(K-2-m) (1-t)^m
// For c < 1 the numerator of Eq. 2 over a_i equals  sum(m2)/Zq + K (1-c)^(K-1) sum(dp)/Zq,
// a sum of non-negative terms (no cancellation); for c >= 1 it equals sum(w)/Zq.
template <bool kNeedAux>
__device__ __forceinline__ void element_terms(float eq, float ep, float kappa, float c, int K, float &w,
                                              float &dp, float &m2) {
    float diff = fmaf(-kappa, ep, eq);
    float d = fmaxf(diff, 0.0f);
    float r = (eq > 0.0f) ? __fdividef(d, eq) : 0.0f;  // r = 1 - t in [0,1]
    float pw = d;
    for (int j = 1; j < K; ++j) pw *= r;
    w = pw;
    if (kNeedAux) {
        dp = fmaxf(-diff, 0.0f);
        float v = 1.0f - c;
        float acc = (K >= 2) ? 1.0f : 0.0f;
        float vj = 1.0f;
        for (int j = 1; j <= K - 2; ++j) {
            vj *= v;
            acc = fmaf(acc, r, (float)(j + 1) * vj);
        }
        float ct = c - 1.0f + r;  // c - t
        m2 = eq * ct * ct * acc;
    }
}

// 2^x in double precision: x = n + f with |f| <= 1/2, e^(f ln 2) by its Taylor series to degree 13
// (remainder below 1e-17), scaled by 2^n.  A short dependent chain, unlike the library routine's.
__device__ __forceinline__ double exp2_short(double x) {
    if (x != x) return x;
    if (x < -1100.0) return 0.0;
    if (x > 1100.0) return INFINITY;
    const double n = rint(x);
    const double t = (x - n) * 0.6931471805599453094;
    double pl = 1.0 / 6227020800.0;
    pl = fma(pl, t, 1.0 / 479001600.0);
    pl = fma(pl, t, 1.0 / 39916800.0);
    pl = fma(pl, t, 1.0 / 3628800.0);
    pl = fma(pl, t, 1.0 / 362880.0);
    pl = fma(pl, t, 1.0 / 40320.0);
    pl = fma(pl, t, 1.0 / 5040.0);
    pl = fma(pl, t, 1.0 / 720.0);
    pl = fma(pl, t, 1.0 / 120.0);
    pl = fma(pl, t, 1.0 / 24.0);
    pl = fma(pl, t, 1.0 / 6.0);
    pl = fma(pl, t, 0.5);
    pl = fma(pl, t, 1.0);
    pl = fma(pl, t, 1.0);
    // 2^n built from its bit pattern where it is a normal number, else the library's scaling
    const int ni = (int)n;
    if (ni > -1000 && ni < 1000) return pl * __longlong_as_double((long long)(ni + 1023) << 52);
    return scalbn(pl, ni);
}
// e^x through the same short chain.
__device__ __forceinline__ double exp_short(double x) { return exp2_short(x * 1.4426950408889634074); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Host-side launchers (one translation unit each).
struct Launch {
    const void *zq;
    const void *zp;
    int dtype;
    const int32_t *tok;
    const float *u;
    Shape s;
    Workspace ws;
    int32_t *out_tau;
    int32_t *out_f;
    int32_t *out_tokens;
    cudaStream_t stream;
    cudaEvent_t ev_begin = nullptr;  // optional: recorded around the dominant kernel
    cudaEvent_t ev_end = nullptr;
    bool ratio_preset = false;       // ws.ratio is known to hold the NaN pattern (the library's own scratch)
    // Algorithm 2: joint log-probabilities log q(s), log p(s) of what has been emitted so far, per chain (device
    // pointers); c starts at exp(log p(s) - log q(s)) instead of 1.  NULL for the verify step.
    const double *carry_loga = nullptr;
    const double *carry_logb = nullptr;
};

int launch_twopass(const Launch &L);  // statistics + chain + reduction, returns launches or <0
int launch_auxreduce(const Launch &L); // the extra sums of Eq. 2 for the rows that need them (behind the fused chain walk)
int launch_finish(const Launch &L);   // weights, scan, extra token
// Algorithm 2's draw per batch row from the cell sums of a gamma = 1 launch with carried logs
int launch_modify_finish(const Launch &L, const float *u, int32_t *out_token, double *out_loga, double *out_logb,
                         double *out_resmass, int32_t *out_status);
// K-SEQ / token-level verification, one CTA per batch row; tile_scratch: [B][2][ntiles] floats
int launch_kseq(const Launch &L, float *tile_scratch, double *out_rho, double *out_acc, int32_t *out_status);
// one token per row of z [s.B, s.V] from softmax(z/T) by inverse CDF; tile_scratch: [s.B][2][ntiles] floats
int launch_draw_rows(const void *z, int dtype, const float *u, const Shape &s, float *tile_scratch, int32_t *out_token,
                     double *out_logp, int32_t *out_status, cudaStream_t stream);
bool fused_supported(const Launch &L);
// single-read cluster path for steps A1-A3: launches (> 0), 0 if it declined before launching
// anything (the caller then takes the two-sweep path), or < 0
// *walked_rows: the kernel used (and consumed the preset of) ws.ratio
// *aux_apart: it left the two extra sums of the rows with c < 1 to launch_auxreduce
int launch_fused(const Launch &L, int *error_flag, bool *walked_rows, bool *aux_apart);
void fused_set_options(int cluster, int max_clusters, int walk, int poll_us, int withhold, int aux);

}  // namespace sgbv
