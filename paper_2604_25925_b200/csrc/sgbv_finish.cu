// Finishing kernel: one CTA per batch row.
//   0. log a_i = log q(x_k^i), log b_i = log p(x_k^i) of every draft by running sums of the token
//      log-probabilities (row maxima and normalisers come from the streaming pass);
//   1. combine the cached per-tile sums of every (k,i) row into S_i and the acceptance weights
//      (Eq. 2 for proper sub-blocks, Eq. 3 for the whole block), in float64;
//   2. the scan of Algorithm 1 over drafts and positions with the pre-drawn uniforms;
//   3. the extra token: inverse CDF of Eq. 4's residual (located through the cached tile sums,
//      only one tile is recomputed) or of the target row after a full accept.
#include <limits.h>

#include "sgbv_common.cuh"

namespace sgbv {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kEpt = kTile / kThreads;  // elements per thread inside one tile
static_assert(kEpt >= 1 && kEpt * kThreads == kTile, "a tile is a whole number of elements per thread");

__device__ __forceinline__ double gfun(double u, int K) {  // 1 - (1-u)^K
    if (u >= 1.0) return 1.0;
    if (!(u > 0.0)) return 0.0;
    return -expm1((double)K * log1p(-u));
}

__device__ __forceinline__ double clamp01(double x) {
    if (!(x > 0.0)) return 0.0;
    return x > 1.0 ? 1.0 : x;
}

// Eq. 2 from the three cached sums of the row that follows the sub-block (all divided by Zq):
//   R = sum_x q (1 - min{c p/q,1})^K,  Dp = sum_x max(c p - q, 0),  M = sum_x q (c-t)^2 Q(t).
// numerator/a   = R                                  (c >= 1)
//               = M + K (1-c)^(K-1) Dp               (c <  1; equals R - (1-c)^K term by term)
// denominator/a = numerator/a + g(b)/a - g(min(c,1))
__device__ double weight_sub(double la, double lb, double R, double Dp, double M, int K, bool below_one) {
    const double a = exp(la), b = exp(lb), c = exp(lb - la);
    const double gb = gfun(b, K);
    if (!(a > 0.0)) return gb > 0.0 ? 0.0 : 1.0;
    double num, extra;
    if (below_one) {  // decided on the float32 c the reduction pass used
        double pw = 1.0;
        for (int j = 1; j < K; ++j) pw *= (1.0 - c);
        num = M + (double)K * pw * Dp;
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

// Eq. 3.
__device__ double weight_full(double la, double lb, int K) {
    const double a = exp(la), b = exp(lb);
    double c = exp(lb - la);
    if (!(a > 0.0) || c > 1.0) c = 1.0;
    const double den = gfun(b, K);
    if (!(den > 0.0)) return 0.0;
    return clamp01(a * gfun(c, K) / den);
}

struct Pick {
    int first;  // smallest index whose cumulative weight exceeds the target, INT_MAX if none
    int last;   // largest index with positive weight, -1 if none
};

// Inverse CDF inside one tile: element x0 + kEpt*tid + j has weight wfun(x). base = cumulative
// weight before the tile. All threads must call.
template <typename F>
__device__ Pick pick_in_tile(int x0, int x1, double base, double target, F wfun, double *sh_warp, int *sh_pick) {
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    float w[kEpt];
    double local = 0.0;
#pragma unroll
    for (int j = 0; j < kEpt; ++j) {
        const int x = x0 + kEpt * tid + j;
        w[j] = (x < x1) ? wfun(x) : 0.0f;
        local += (double)w[j];
    }
    double incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        double v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    if (tid == 0) {
        sh_pick[0] = INT_MAX;
        sh_pick[1] = -1;
    }
    if (lane == 31) sh_warp[wid] = incl;
    __syncthreads();
    double off = base;
    for (int k = 0; k < wid; ++k) off += sh_warp[k];
    double cum = off + incl - local;
#pragma unroll
    for (int j = 0; j < kEpt; ++j) {
        cum += (double)w[j];
        const int x = x0 + kEpt * tid + j;
        if (w[j] > 0.0f) {
            atomicMax(&sh_pick[1], x);
            if (cum > target) atomicMin(&sh_pick[0], x);
        }
    }
    __syncthreads();
    Pick p{sh_pick[0], sh_pick[1]};
    __syncthreads();
    return p;
}

// First tile whose inclusive prefix of the cached tile sums exceeds the target (sequential,
// float64, ascending: the same order as the total).  If rounding leaves none, the last tile
// with positive mass, with a base that makes the in-tile search fall back to its last
// positive element.  Results: sh_i[2] = tile, sh_d[0] = mass before it, sh_d[1] = target.
__device__ void locate_tile(const float *partials, int ntiles, double target, int *sh_i, double *sh_d) {
    double cum = 0.0, base = 0.0;
    int sel = -1, lastpos = 0;
    for (int t = 0; t < ntiles; ++t) {
        const double v = (double)partials[t];
        if (v > 0.0) lastpos = t;
        if (cum + v > target) {
            sel = t;
            base = cum;
            break;
        }
        cum += v;
    }
    if (sel < 0) {
        sel = lastpos;
        base = -INFINITY;
    }
    sh_i[2] = sel;
    sh_d[0] = base;
    sh_d[1] = target;
}

template <typename T>
__global__ void __launch_bounds__(kThreads)
finish_kernel(const T *__restrict__ zq_all, const T *__restrict__ zp_all, const int32_t *__restrict__ tok_all,
              const float *__restrict__ u_all, Shape s, Workspace ws, int32_t *__restrict__ out_tau,
              int32_t *__restrict__ out_f, int32_t *__restrict__ out_tokens) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int K = s.K, g = s.gamma, KG = K * g;
    double *h_s = reinterpret_cast<double *>(smem_raw);                       // [K*g]
    double *W_s = h_s + KG;                                                   // [K*g] sum of wpart
    double *la_s = W_s + KG;                                                  // [K*(g+1)] log q(x_k^i)
    double *lb_s = la_s + K * (g + 1);                                        // [K*(g+1)] log p(x_k^i)
    unsigned long long *rej_s = reinterpret_cast<unsigned long long *>(lb_s + K * (g + 1));  // [K]
    float *tile_s = reinterpret_cast<float *>(rej_s + K);                     // [ntiles]
    unsigned char *lcp_s = reinterpret_cast<unsigned char *>(tile_s + s.ntiles);  // [K*K]
    __shared__ double sh_warp[kWarps];
    __shared__ float sh_redf[kWarps];
    __shared__ int sh_pick[2];
    __shared__ int sh_i[4];
    __shared__ double sh_d[2];

    const int b = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int32_t *tok = tok_all + (size_t)b * KG;
    const float *u = u_all + (size_t)b * (KG + 1);
    const int status_in = ws.status[b];
    const bool lost = *ws.error != 0;  // a bounded wait expired upstream: nothing can be trusted
    const bool invalid = lost || (status_in & (SGBV_STATUS_TOKEN_RANGE | SGBV_STATUS_NONFINITE_LOGIT)) != 0;

    // ---- 0. joint prefix probabilities (logs), one thread per draft -----------------------------
    for (int k = tid; k < K; k += kThreads) {
        double la = 0.0, lb = 0.0;
        for (int i = 0; i < g; ++i) {
            la_s[k * (g + 1) + i] = la;
            lb_s[k * (g + 1) + i] = lb;
            const size_t r = ((size_t)b * K + k) * g + i;
            const RowInfo ri = ws.rows[r];
            int t = tok[k * g + i];
            if (t < 0 || t >= s.V) t = 0;  // the row is flagged and produces no output
            const float zqt = ld_logit(zq_all, (((size_t)b * K + k) * (g + 1) + i) * s.V + t);
            const float zpt = ld_logit(zp_all, r * s.V + t);
            la += ((double)zqt - (double)ri.mq) * s.inv_T - log(ri.Zq);
            lb += ((double)zpt - (double)ri.mp) * s.inv_T - log(ri.Zp);
        }
        la_s[k * (g + 1) + g] = la;
        lb_s[k * (g + 1) + g] = lb;
    }
    __syncthreads();

    // ---- 1. weights ---------------------------------------------------------------------------
    for (int n = wid; n < KG; n += kWarps) {
        const int k = n / g, i = n % g;
        const size_t r = ((size_t)b * K + k) * g + i;
        const RowInfo ri = ws.rows[r];
        const bool aux = ri.c < 1.0f;
        const float *wp = ws.wpart + r * s.ntiles, *dp = ws.dpart + r * s.ntiles, *mp = ws.mpart + r * s.ntiles;
        double sw = 0.0, sd = 0.0, sm = 0.0;
        for (int t = lane; t < s.ntiles; t += 32) {
            sw += (double)wp[t];
            if (aux) {
                sd += (double)dp[t];
                sm += (double)mp[t];
            }
        }
        sw = warp_sum(sw);
        sd = warp_sum(sd);
        sm = warp_sum(sm);
        if (lane == 0) {
            const double R = sw / ri.Zq;
            W_s[n] = sw;
            const double la = la_s[k * (g + 1) + i], lb = lb_s[k * (g + 1) + i];
            const double S = exp(la) * R;
            ws.resmass[(size_t)b * KG + n] = invalid ? NAN : S;
            if (i >= 1) {
                const double hv = weight_sub(la, lb, R, sd / ri.Zq, sm / ri.Zq, K, aux);
                h_s[k * g + i - 1] = hv;
                ws.h[(size_t)b * KG + k * g + i - 1] = invalid ? NAN : hv;
            }
        }
    }
    for (int k = tid; k < K; k += kThreads) {
        const double hv = weight_full(la_s[k * (g + 1) + g], lb_s[k * (g + 1) + g], K);
        h_s[k * g + g - 1] = hv;
        ws.h[(size_t)b * KG + k * g + g - 1] = invalid ? NAN : hv;
        rej_s[k] = 0ull;
    }
    // longest common prefix of every pair of drafts (for the membership test in H)
    for (int n = tid; n < K * K; n += kThreads) {
        const int k = n / K, kp = n % K;
        int l = 0;
        while (l < g && tok[k * g + l] == tok[kp * g + l]) ++l;
        lcp_s[n] = (unsigned char)l;
    }
    __syncthreads();

    if (invalid) {
        if (tid == 0) {
            out_tau[b] = -1;
            out_f[b] = -1;
            if (lost) ws.status[b] = status_in | SGBV_STATUS_TIMEOUT;
        }
        for (int j = tid; j <= g; j += kThreads) out_tokens[(size_t)b * (g + 1) + j] = -1;
        return;
    }

    // ---- 2. scan (Algorithm 1), warp 0 ---------------------------------------------------------
    if (wid == 0) {
        int tau = 0, f = -1;
        bool done = false;
        for (int k = 0; k < K && !done; ++k) {
            const int start = tau + 1;
            for (int i = start; i <= g; ++i) {
                const double hv = h_s[k * g + i - 1];
                const double eta = (double)u[k * g + i - 1];
                bool inH = false;  // an earlier draft with the same i-token prefix was rejected at length i
                for (int kp = lane; kp < k; kp += 32)
                    inH |= (lcp_s[k * K + kp] >= i) && ((rej_s[kp] >> (i - 1)) & 1ull);
                inH = __any_sync(0xffffffffu, inH);
                const bool accept = (eta < hv) && !inH;
                if (accept) {
                    tau = i;
                    f = k;
                    if (i == g) {
                        done = true;
                        break;
                    }
                } else if (lane == 0) {
                    rej_s[k] |= 1ull << (i - 1);
                }
                __syncwarp();
            }
        }
        if (lane == 0) {
            sh_i[0] = tau;
            sh_i[1] = f;
        }
    }
    __syncthreads();
    const int tau = sh_i[0], f = sh_i[1];
    const int kk = (tau == 0) ? 0 : f;
    const double us = (double)u[KG];

    // ---- 3. extra token -------------------------------------------------------------------------
    int y = -1;
    int flags = 0;
    const T *zq = zq_all + (((size_t)b * K + kk) * (g + 1) + tau) * s.V;
    bool from_q = (tau == g);
    if (!from_q) {
        const size_t r = ((size_t)b * K + kk) * g + tau;
        const double W = W_s[kk * g + tau];
        if (W > 0.0) {
            const float *wp = ws.wpart + r * s.ntiles;
            if (tid == 0) locate_tile(wp, s.ntiles, us * W, sh_i, sh_d);
            __syncthreads();
            const int sel = sh_i[2];
            const RowInfo ri = ws.rows[r];
            const T *zp = zp_all + (((size_t)b * K + kk) * g + tau) * s.V;
            const int x0 = sel * kTile, x1 = min(s.V, x0 + kTile);
            auto wfun = [&](int x) {
                float eq = expo(ld_logit(zq, x), ri.mq, s.scale);
                float ep = expo(ld_logit(zp, x), ri.mp, s.scale);
                float w, d0, d1;
                element_terms<false>(eq, ep, ri.kappa, ri.c, K, w, d0, d1);
                return w;
            };
            Pick p = pick_in_tile(x0, x1, sh_d[0], sh_d[1], wfun, sh_warp, sh_pick);
            y = (p.first != INT_MAX) ? p.first : p.last;
        } else {
            from_q = true;  // zero residual mass: draw from q of the same row
            flags |= SGBV_STATUS_DEGENERATE_RESIDUAL;
        }
    }
    if (from_q) {
        // softmax(zq/T) of one row, block-wide: max, per-tile sums, locate, pick
        float m = -INFINITY;
        bool bad = false;
        for (int x = tid; x < s.V; x += kThreads) {
            const float z = ld_logit(zq, x);
            bad |= (z != z) | (z == INFINITY);
            m = fmaxf(m, z);
        }
        m = warp_max(m);
        if (lane == 0) sh_redf[wid] = m;
        bad = __syncthreads_or(bad);
        m = sh_redf[0];
        for (int w = 1; w < kWarps; ++w) m = fmaxf(m, sh_redf[w]);
        if (bad || !(m > -INFINITY)) {
            flags |= SGBV_STATUS_NONFINITE_LOGIT;
        } else {
            for (int t = wid; t < s.ntiles; t += kWarps) {
                const int x0 = t * kTile, x1 = min(s.V, x0 + kTile);
                float acc = 0.0f;
                for (int x = x0 + lane; x < x1; x += 32) acc += expo(ld_logit(zq, x), m, s.scale);
                acc = warp_sum(acc);
                if (lane == 0) tile_s[t] = acc;
            }
            __syncthreads();
            if (tid == 0) {
                double W = 0.0;
                for (int t = 0; t < s.ntiles; ++t) W += (double)tile_s[t];
                locate_tile(tile_s, s.ntiles, us * W, sh_i, sh_d);
            }
            __syncthreads();
            const int sel = sh_i[2];
            const int x0 = sel * kTile, x1 = min(s.V, x0 + kTile);
            auto wfun = [&](int x) { return expo(ld_logit(zq, x), m, s.scale); };
            Pick p = pick_in_tile(x0, x1, sh_d[0], sh_d[1], wfun, sh_warp, sh_pick);
            y = (p.first != INT_MAX) ? p.first : p.last;
        }
    }

    // ---- 4. outputs ------------------------------------------------------------------------------
    const bool failed = (flags & SGBV_STATUS_NONFINITE_LOGIT) != 0;
    if (tid == 0) {
        out_tau[b] = failed ? -1 : tau;
        out_f[b] = failed ? -1 : f;
        if (flags) ws.status[b] = status_in | flags;
    }
    for (int j = tid; j <= g; j += kThreads) {
        int v = -1;
        if (!failed) {
            if (j < tau) v = tok[f * g + j];
            else if (j == tau) v = y;
        }
        out_tokens[(size_t)b * (g + 1) + j] = v;
    }
}

template <typename T>
int run(const Launch &L) {
    const Shape &s = L.s;
    const size_t KG = (size_t)s.K * s.gamma;
    const size_t smem = 2 * KG * sizeof(double) + 2 * (size_t)s.K * (s.gamma + 1) * sizeof(double) +
                        s.K * sizeof(unsigned long long) + (size_t)s.ntiles * sizeof(float) + (size_t)s.K * s.K;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(finish_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return SGBV_ERR_CUDA;
    }
    finish_kernel<T><<<s.B, kThreads, smem, L.stream>>>((const T *)L.zq, (const T *)L.zp, L.tok, L.u, s, L.ws,
                                                        L.out_tau, L.out_f, L.out_tokens);
    return cudaGetLastError() == cudaSuccess ? 1 : SGBV_ERR_CUDA;
}

}  // namespace

int launch_finish(const Launch &L) {
    return L.dtype == SGBV_DTYPE_BF16 ? run<uint16_t>(L) : run<float>(L);
}

}  // namespace sgbv
