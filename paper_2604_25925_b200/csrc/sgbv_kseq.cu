// Comparison verifiers of Section 3 of the paper, behind the same boundary as the block verifier:
// SpecTr's position-wise K-SEQ (Section 3.2) and, as its one-draft case, token-level speculative sampling
// (Section 3.1).  They exist so that the verification cost of the methods can be compared on one machine
// (the paper's Table 2); they are written for correctness and reasonable speed, not tuned like the block
// verifier's streaming kernel.
//
// One CTA per batch row walks the positions i = 0..gamma-1 in order.  At a position the drafts that still match
// the accepted prefix ("retained", n of them) are the candidates; they share the rows of that prefix, and the
// rows of the first retained draft are read:
//   1. row maxima and normalisers of the target and draft rows (two passes over the rows, from L2);
//   2. rho in [1, n]: root of 1 - (1 - beta(rho))^n = rho beta(rho), beta(rho) = sum_x min{p(x), q(x)/rho}, by
//      bisection, one pass over the rows per step (n = 1: rho = 1);
//   3. the retained drafts are tried in order, draft k's token x is accepted if eta < min{1, q(x)/(rho p(x))};
//      the first accepted token extends the prefix, the drafts with that token stay retained;
//   4. if none is accepted: y from norm(max{q - rho p, 0}) by inverse CDF over per-tile sums, and the row is done.
// After gamma accepted positions y is drawn from the target row that follows the block.
#include "sgbv_sample.cuh"

namespace sgbv {

namespace {

constexpr int kKseqThreads = 1024;
constexpr int kBisections = 34;  // interval n 2^-34: far below float32 resolution of beta

// 1 - (1-u)^n as a geometric sum (all terms positive).
__device__ __forceinline__ double gfun_n(double u, int n) {
    if (u >= 1.0) return 1.0;
    if (!(u > 0.0)) return 0.0;
    const double v = 1.0 - u;
    double sum = 1.0;
    for (int j = 1; j < n; ++j) sum = fma(sum, v, 1.0);
    return u * sum;
}

// Sum of a double over the CTA (every thread gets it).  All threads must call.
__device__ __forceinline__ double block_sum(double v, double *sh_warp) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    v = warp_sum(v);
    __syncthreads();  // (sh_warp may still be read from the previous use)
    if (lane == 0) sh_warp[wid] = v;
    __syncthreads();
    return warp_sum(lane < nwarps ? sh_warp[lane] : 0.0);
}

template <typename T>
__global__ void __launch_bounds__(kKseqThreads)
kseq_kernel(const T *__restrict__ zq_all, const T *__restrict__ zp_all, const int32_t *__restrict__ tok_all,
            const float *__restrict__ u_all, Shape s, float *__restrict__ tile_scratch, int32_t *__restrict__ out_tau,
            int32_t *__restrict__ out_tokens, double *__restrict__ out_rho, double *__restrict__ out_acc,
            int32_t *__restrict__ out_status) {
    __shared__ SampleScratch sc;
    __shared__ int kept[kMaxK];
    __shared__ int sh_n, sh_accepted, sh_flags;
    __shared__ float sh_max[2][kSampleMaxWarps];
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int nthreads = blockDim.x, nwarps = nthreads >> 5;
    const int K = s.K, g = s.gamma, V = s.V;
    const int32_t *tok = tok_all + (size_t)b * K * g;
    const float *u = u_all + (size_t)b * (K * g + 1);
    float *tile_s = tile_scratch + (size_t)b * 2 * s.ntiles, *tile_m = tile_s + s.ntiles;

    for (int n = tid; n <= g; n += nthreads) out_tokens[(size_t)b * (g + 1) + n] = -1;
    if (out_rho)
        for (int n = tid; n < g; n += nthreads) out_rho[(size_t)b * g + n] = NAN;
    if (out_acc)
        for (int n = tid; n < K * g; n += nthreads) out_acc[(size_t)b * K * g + n] = NAN;
    if (tid == 0) {
        sh_n = K;
        sh_flags = 0;
    }
    for (int k = tid; k < K; k += nthreads) kept[k] = k;
    __syncthreads();
    bool range = false;
    for (int n = tid; n < K * g; n += nthreads) range |= tok[n] < 0 || tok[n] >= V;
    if (__syncthreads_or(range)) {
        if (tid == 0) {
            out_tau[b] = -1;
            out_status[b] = SGBV_STATUS_TOKEN_RANGE;
        }
        return;
    }

    int tau = 0, y = -1, flags = 0;
    bool stopped = false;
    for (int i = 0; i < g && !stopped; ++i) {
        const int k0 = kept[0], nk = sh_n;
        const T *zq = zq_all + (((size_t)b * K + k0) * (g + 1) + i) * V;
        const T *zp = zp_all + (((size_t)b * K + k0) * g + i) * V;
        // ---- 1. maxima (NaN / +inf detection on the way), then normalisers ---------------------------------
        float mq = -INFINITY, mp = -INFINITY;
        bool bad = false;
        for (int x = tid; x < V; x += nthreads) {
            const float a = ld_logit(zq, x), c = ld_logit(zp, x);
            bad |= (a != a) | (c != c) | (a == INFINITY) | (c == INFINITY);
            mq = fmaxf(mq, a);
            mp = fmaxf(mp, c);
        }
        mq = warp_max(mq);
        mp = warp_max(mp);
        if (lane == 0) {
            sh_max[0][wid] = mq;
            sh_max[1][wid] = mp;
        }
        bad = __syncthreads_or(bad);
        mq = warp_max(lane < nwarps ? sh_max[0][lane] : -INFINITY);
        mp = warp_max(lane < nwarps ? sh_max[1][lane] : -INFINITY);
        if (bad || !(mq > -INFINITY) || !(mp > -INFINITY)) {
            flags |= SGBV_STATUS_NONFINITE_LOGIT;
            break;
        }
        float sq = 0.0f, sp = 0.0f;
        for (int x = tid; x < V; x += nthreads) {
            sq += expo(ld_logit(zq, x), mq, s.scale);
            sp += expo(ld_logit(zp, x), mp, s.scale);
        }
        const double Zq = block_sum((double)sq, sc.warp), Zp = block_sum((double)sp, sc.warp);
        const float inv_Zq = (float)(1.0 / Zq), inv_Zp = (float)(1.0 / Zp);
        // ---- 2. rho -----------------------------------------------------------------------------------------
        double rho = 1.0;
        if (nk > 1) {
            double lo = 1.0, hi = (double)nk;
            for (int it = 0; it < kBisections; ++it) {
                const double mid = 0.5 * (lo + hi);
                const float q_scale = (float)(1.0 / (Zq * mid));
                float acc = 0.0f;
                for (int x = tid; x < V; x += nthreads) {
                    const float qx = expo(ld_logit(zq, x), mq, s.scale) * q_scale;
                    const float px = expo(ld_logit(zp, x), mp, s.scale) * inv_Zp;
                    acc += fminf(px, qx);
                }
                const double beta = block_sum((double)acc, sc.warp);
                const double f = gfun_n(beta, nk) - mid * beta;  // (the same on every thread)
                if (f > 0.0) lo = mid;
                else hi = mid;
            }
            rho = 0.5 * (lo + hi);
        }
        // ---- 3. the retained drafts, in order -----------------------------------------------------------------
        if (tid == 0) {
            if (out_rho) out_rho[(size_t)b * g + i] = rho;
            int accepted = -1;
            for (int j = 0; j < nk && accepted < 0; ++j) {
                const int k = kept[j];
                const int x = tok[k * g + i];
                const float zpx = ld_logit(zp, x);
                double acc = 1.0;
                if (zpx > -INFINITY) {
                    const double lq = ((double)ld_logit(zq, x) - (double)mq) * s.inv_T - log(Zq);
                    const double lp = ((double)zpx - (double)mp) * s.inv_T - log(Zp);
                    acc = exp(lq - lp) / rho;
                    if (!(acc < 1.0)) acc = 1.0;
                }
                if (out_acc) out_acc[((size_t)b * K + k) * g + i] = acc;
                if ((double)u[k * g + i] < acc) accepted = k;
            }
            sh_accepted = accepted;
            if (accepted >= 0) {
                const int x = tok[accepted * g + i];
                int m = 0;
                for (int j = 0; j < nk; ++j)
                    if (tok[kept[j] * g + i] == x) kept[m++] = kept[j];
                sh_n = m;
                out_tokens[(size_t)b * (g + 1) + i] = x;
            }
        }
        __syncthreads();
        if (sh_accepted >= 0) {
            tau = i + 1;
            continue;
        }
        // ---- 4. nothing accepted: y from norm(max{q - rho p, 0}) ------------------------------------------------
        const float rho_p = (float)rho * inv_Zp;
        auto wfun = [&](int x) {
            const float qx = expo(ld_logit(zq, x), mq, s.scale) * inv_Zq;
            const float px = expo(ld_logit(zp, x), mp, s.scale) * rho_p;
            return fmaxf(qx - px, 0.0f);
        };
        double wtot = 0.0;
        for (int t = wid; t < s.ntiles; t += nwarps) {  // one warp per 256-entry tile
            float acc = 0.0f;
            for (int x = t * kTile + lane; x < min(V, (t + 1) * kTile); x += 32) acc += wfun(x);
            acc = warp_sum(acc);
            if (lane == 0) tile_s[t] = acc;
            wtot += (double)acc;
        }
        const double W = block_sum(lane == 0 ? wtot : 0.0, sc.warp);
        const double us = (double)u[K * g];
        if (W > 0.0) {
            locate_tile(tile_s, nullptr, s.ntiles, us * W, false, sc.i, sc.d, sc.warp);
            const int sel = sc.i[2];
            Pick pk = pick_in_tile(sel * kTile, min(V, (sel + 1) * kTile), sc.d[0], sc.d[1], wfun, sc.warp, sc.pick);
            y = (pk.first != INT_MAX) ? pk.first : pk.last;
        } else {  // q <= rho p everywhere: the draw comes from q itself
            flags |= SGBV_STATUS_DEGENERATE_RESIDUAL;
            bool bad_row = false;
            y = draw_from_row<T>(zq, s, us, tile_s, tile_m, &sc, bad_row);
            if (bad_row) flags |= SGBV_STATUS_NONFINITE_LOGIT;
        }
        stopped = true;
    }
    if (!stopped && !(flags & SGBV_STATUS_NONFINITE_LOGIT)) {  // every position accepted: bonus token
        const T *zq = zq_all + (((size_t)b * K + kept[0]) * (g + 1) + g) * V;
        bool bad_row = false;
        y = draw_from_row<T>(zq, s, (double)u[K * g], tile_s, tile_m, &sc, bad_row);
        if (bad_row) flags |= SGBV_STATUS_NONFINITE_LOGIT;
    }
    __syncthreads();
    const bool failed = (flags & SGBV_STATUS_NONFINITE_LOGIT) != 0;
    if (failed) {
        for (int n = tid; n <= g; n += nthreads) out_tokens[(size_t)b * (g + 1) + n] = -1;
    } else if (tid == 0) {
        out_tokens[(size_t)b * (g + 1) + tau] = y;
    }
    if (tid == 0) {
        out_tau[b] = failed ? -1 : tau;
        out_status[b] = flags;
    }
}

}  // namespace

int launch_kseq(const Launch &L, float *tile_scratch, double *out_rho, double *out_acc, int32_t *out_status) {
    const Shape &s = L.s;
    if (L.dtype == SGBV_DTYPE_BF16)
        kseq_kernel<uint16_t><<<s.B, kKseqThreads, 0, L.stream>>>((const uint16_t *)L.zq, (const uint16_t *)L.zp, L.tok, L.u, s,
                                                                  tile_scratch, L.out_tau, L.out_tokens, out_rho, out_acc,
                                                                  out_status);
    else
        kseq_kernel<float><<<s.B, kKseqThreads, 0, L.stream>>>((const float *)L.zq, (const float *)L.zp, L.tok, L.u, s,
                                                               tile_scratch, L.out_tau, L.out_tokens, out_rho, out_acc,
                                                               out_status);
    if (cudaGetLastError() != cudaSuccess) return SGBV_ERR_CUDA;
    return 1;
}

}  // namespace sgbv
