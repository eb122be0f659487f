// Finishing kernel: one CTA of 1024 threads per batch row.
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

constexpr int kMaxThreads = 1024;  // CTA size when few batch rows leave most SMs idle (the kernel is a
constexpr int kMinThreads = 256;   // chain of memory latencies, so more warps per row help); else 512 or 256
constexpr int kMaxWarps = kMaxThreads / 32;
constexpr int kTilesInSmem = 4096;  // rows up to 2^20 entries keep the bonus row's tile sums in shared memory
constexpr int kEpt = 1;  // elements per thread inside one tile (threads beyond the tile hold none)
static_assert(kMinThreads >= kTile, "one thread per element of a tile");

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
//               = M + K (1-c)^(K-1) Dp               (c <  1; equals R - (1-c)^K term by term)
// denominator/a = numerator/a + g(b)/a - g(min(c,1))
__device__ double weight_sub(double la, double lb, double R, double Dp, double M, int K, bool below_one) {
    const double a = exp_short(la), b = exp_short(lb), c = exp_short(lb - la);
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
    const double a = exp_short(la), b = exp_short(lb);
    double c = exp_short(lb - la);
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
    // mass of the warps before this one: a butterfly over the lanes instead of a loop over the warps
    const double wv = lane < (int)(blockDim.x >> 5) ? sh_warp[lane] : 0.0;
    const double off = base + warp_sum(lane < wid ? wv : 0.0);
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

// First tile whose inclusive prefix of the tile sums exceeds the target (float64, ascending
// vocabulary order), found by the whole block: every thread owns a contiguous run of tiles, the
// runs' totals are scanned across the block, and each thread searches its own run.  If rounding
// leaves no such tile, the last tile with positive mass is taken, with a base that makes the
// in-tile search fall back to its last positive element.  scale[t] (may be NULL) multiplies tile
// t's sum.  relative: `target` is a fraction of the total of all tile sums (computed here on the
// way) instead of a mass.  All threads must call.  Results: sh_i[2] = tile, sh_d[0] = mass before it,
// sh_d[1] = target.
__device__ void locate_tile(const float *partials, const float *scale, int ntiles, double target, bool relative,
                            int *sh_i, double *sh_d, double *sh_warp) {
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int nthreads = blockDim.x;
    const int per = (ntiles + nthreads - 1) / nthreads;
    const int t0 = min(ntiles, tid * per), t1 = min(ntiles, t0 + per);
    // the thread's tile sums: the first four stay in registers for the search below
    constexpr int kKeep = 4;
    double kept[kKeep];
    double local = 0.0;
#pragma unroll
    for (int e = 0; e < kKeep; ++e) {
        const int t = t0 + e;
        kept[e] = (t < t1) ? (double)partials[t] * (scale ? (double)scale[t] : 1.0) : 0.0;
        local += kept[e];
    }
    for (int t = t0 + kKeep; t < t1; ++t) local += (double)partials[t] * (scale ? (double)scale[t] : 1.0);
    double incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    if (tid == 0) {
        sh_i[2] = INT_MAX;  // first tile that crosses the target
        sh_i[3] = -1;       // last tile with positive mass
    }
    if (lane == 31) sh_warp[wid] = incl;
    __syncthreads();
    // the warps' totals: every warp adds up those of the warps before it (and all of them) with a butterfly
    // over its lanes instead of one after the other
    const double wv = lane < (nthreads >> 5) ? sh_warp[lane] : 0.0;
    const double cum0 = incl - local + warp_sum(lane < wid ? wv : 0.0);
    if (relative) target *= warp_sum(wv);  // the target is given as a fraction of the total of all tiles
    double cum = cum0;
    int first = INT_MAX, lastpos = -1;
    double base = 0.0;
    for (int t = t0; t < t1; ++t) {
        double v;
        if (t - t0 < kKeep) {
            v = kept[0];
#pragma unroll
            for (int e = 1; e < kKeep; ++e)
                if (t - t0 == e) v = kept[e];
        } else {
            v = (double)partials[t] * (scale ? (double)scale[t] : 1.0);
        }
        if (v > 0.0) lastpos = t;
        if (first == INT_MAX && cum + v > target) {
            first = t;
            base = cum;
        }
        cum += v;
    }
    if (first != INT_MAX) atomicMin(&sh_i[2], first);
    if (lastpos >= 0) atomicMax(&sh_i[3], lastpos);
    __syncthreads();
    if (first != INT_MAX && sh_i[2] == first) sh_d[0] = base;  // exactly one thread owns that tile
    __syncthreads();
    if (tid == 0) {
        if (sh_i[2] == INT_MAX) {
            sh_i[2] = max(sh_i[3], 0);
            sh_d[0] = -INFINITY;
        }
        sh_d[1] = target;
    }
    __syncthreads();
}

// The 8 entries of a 256-entry tile that one lane takes when the row can be read in 16-byte pieces (the row starts
// on a 16-byte boundary and V is a multiple of the entries per piece, so a piece lies inside the row or past it).
template <typename T>
__device__ __forceinline__ void load_tile_pieces(const T *zq, int tile, bool in, int V, int lane, float (&z)[kTile / 32]);
template <>
__device__ __forceinline__ void load_tile_pieces<float>(const float *zq, int tile, bool in, int V, int lane,
                                                        float (&z)[kTile / 32]) {
    const float ninf = -INFINITY;
    const int xa = tile * kTile + lane * 4, xb = xa + kTile / 2;
    const float4 a = (in && xa < V) ? __ldg(reinterpret_cast<const float4 *>(zq + xa)) : make_float4(ninf, ninf, ninf, ninf);
    const float4 b = (in && xb < V) ? __ldg(reinterpret_cast<const float4 *>(zq + xb)) : make_float4(ninf, ninf, ninf, ninf);
    z[0] = a.x; z[1] = a.y; z[2] = a.z; z[3] = a.w;
    z[4] = b.x; z[5] = b.y; z[6] = b.z; z[7] = b.w;
}
template <>
__device__ __forceinline__ void load_tile_pieces<uint16_t>(const uint16_t *zq, int tile, bool in, int V, int lane,
                                                           float (&z)[kTile / 32]) {
    const uint32_t ninf2 = 0xff80ff80u;  // two bf16 -inf
    const int xa = tile * kTile + lane * 8;
    const uint4 a = (in && xa < V) ? __ldg(reinterpret_cast<const uint4 *>(zq + xa)) : make_uint4(ninf2, ninf2, ninf2, ninf2);
    z[0] = __uint_as_float(a.x << 16); z[1] = __uint_as_float(a.x & 0xffff0000u);
    z[2] = __uint_as_float(a.y << 16); z[3] = __uint_as_float(a.y & 0xffff0000u);
    z[4] = __uint_as_float(a.z << 16); z[5] = __uint_as_float(a.z & 0xffff0000u);
    z[6] = __uint_as_float(a.w << 16); z[7] = __uint_as_float(a.w & 0xffff0000u);
}

template <typename T>
__global__ void __launch_bounds__(kMaxThreads)
finish_kernel(const T *__restrict__ zq_all, const T *__restrict__ zp_all, const int32_t *__restrict__ tok_all,
              const float *__restrict__ u_all, Shape s, Workspace ws, int32_t *__restrict__ out_tau,
              int32_t *__restrict__ out_f, int32_t *__restrict__ out_tokens) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int K = s.K, g = s.gamma, KG = K * g;
    double *W_s = reinterpret_cast<double *>(smem_raw);                       // [K*g] sum of wpart
    double *D_s = W_s + KG;                                                   // [K*g] sum of dpart
    double *M_s = D_s + KG;                                                   // [K*g] sum of mpart
    double *la_s = M_s + KG;                                                  // [K*(g+1)] log q(x_k^i)
    double *lb_s = la_s + K * (g + 1);                                        // [K*(g+1)] log p(x_k^i)
    unsigned long long *pass_s = reinterpret_cast<unsigned long long *>(lb_s + K * (g + 1));  // [K] bit i-1: eta < h for length i
    int32_t *tok_s = reinterpret_cast<int32_t *>(pass_s + K);                 // [K*g] the draft tokens
    float *u_s = reinterpret_cast<float *>(tok_s + KG);                       // [K*g+1] the uniforms
    unsigned char *lcp_s = reinterpret_cast<unsigned char *>(u_s + KG + 1);   // [K*K]
    // per-tile (sum, maximum -> factor) of the target row a bonus token is drawn from: shared memory
    // when the row has few enough tiles (the launcher then reserves the space), else global scratch
    float *tile_s = ws.bonus_in_smem ? reinterpret_cast<float *>(lcp_s + ((K * K + 15) / 16) * 16)
                                               : ws.bonus + (size_t)blockIdx.x * 2 * s.ntiles;  // [ntiles]
    float *tile_m = tile_s + s.ntiles;                                        // [ntiles]
    __shared__ double sh_warp[kMaxWarps];
    __shared__ float sh_redf[kMaxWarps];
    __shared__ int sh_pick[2];
    __shared__ int sh_i[4];
    __shared__ unsigned sh_or[2];
    __shared__ int sh_flags;
    __shared__ double sh_d[2];

    // A kernel launched behind this one with programmatic stream serialisation (the next call's streaming
    // kernel) may be scheduled from now on; it waits for this grid to complete before it touches memory.
    // Only for small batches, where this grid leaves most SMs idle.
    if (s.B <= kChainedLaunchMaxB) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int b = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int nthreads = blockDim.x, nwarps = nthreads / 32;
    const int32_t *tok = tok_all + (size_t)b * KG;
    const float *u = u_all + (size_t)b * (KG + 1);
    // the uniforms are needed by the serial scan: fetch them now, with threads other than those
    // that start the token work below
    for (int n = (tid + nthreads / 2) % nthreads; n <= KG; n += nthreads) u_s[n] = u[n];
    for (int n = tid; n < KG; n += nthreads) tok_s[n] = tok[n];
    for (int k = tid; k < K; k += nthreads) pass_s[k] = 0ull;
    if (tid == 0) sh_flags = 0;
    // Everything above reads only the caller's inputs.  The kernel may have been scheduled while the
    // streaming kernel was still running (programmatic dependent launch): wait for it to complete
    // before touching the row records and cell sums.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    __syncthreads();  // the staged tokens and uniforms are read by other threads than those that fetched them
    const bool lost = *ws.error != 0;  // a bounded wait expired upstream: nothing can be trusted
    // the streaming kernel has consumed the "not published yet" pattern of this batch row's ratio words:
    // put it back, so that the next call on this scratch area need not clear them first
    if (ws.ratio_used)
        for (int n = tid; n < KG; n += nthreads)
            reinterpret_cast<unsigned long long *>(ws.ratio)[(size_t)b * KG + n] = ~0ull;
    int myflags = (tid == 0 && ws.prestatus) ? ws.prestatus[b] : 0;

    // ---- cell sums of every row (k,i), one warp per row, first warps first; the token work of step 0
    //      below starts with the LAST threads, so that for small K*gamma both run side by side ----
    for (int n = wid; n < KG; n += nwarps) {
        const int k = n / g, i = n % g;
        const size_t r = ((size_t)b * K + k) * g + i;
        const RowInfo ri = ws.rows[r];
        const bool aux = ri.c < 1.0f;
        const float *wp = ws.wpart + r * s.ntiles, *dp = ws.dpart + r * s.ntiles, *mp = ws.mpart + r * s.ntiles;
        double sw = 0.0, sd = 0.0, sm = 0.0;
        for (int t0 = 0; t0 < s.ntiles; t0 += 128) {  // four independent loads per array in flight
            float w4[4], d4[4], m4[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int t = t0 + lane + 32 * e;
                const bool in = t < s.ntiles;
                // the two extra arrays are fetched whether or not the row has them (c < 1), so that the
                // fetches do not wait for the row's record; what they hold otherwise is dropped below
                w4[e] = in ? wp[t] : 0.0f;
                d4[e] = in ? dp[t] : 0.0f;
                m4[e] = in ? mp[t] : 0.0f;
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                sw += (double)w4[e];
                sd += aux ? (double)d4[e] : 0.0;
                sm += aux ? (double)m4[e] : 0.0;
            }
        }
        sw = warp_sum(sw);
        sd = warp_sum(sd);
        sm = warp_sum(sm);
        if (lane == 0) {
            W_s[n] = sw;
            D_s[n] = sd;
            M_s[n] = sm;
        }
    }

    // ---- 0. joint prefix probabilities (logs): token log-probabilities in parallel, then one
    //         running sum per draft ------------------------------------------------------------
    const int n_first = nthreads - 1 - tid;  // this thread's first (k,i), here and in the weights below
    double inv_Zq_first = 0.0;
    bool below_first = false;
    for (int n = n_first; n < KG; n += nthreads) {
        const int k = n / g, i = n % g;
        const size_t r = ((size_t)b * K + k) * g + i;
        const RowInfo ri = ws.rows[r];
        if (n == n_first) {
            inv_Zq_first = 1.0 / ri.Zq;
            below_first = ri.c < 1.0f;
        }
        int t = tok_s[n];
        myflags |= ri.flags;
        if (t < 0 || t >= s.V) {  // the row is flagged and produces no output
            myflags |= SGBV_STATUS_TOKEN_RANGE;
            t = 0;
        }
        const float zqt = ld_logit(zq_all, (((size_t)b * K + k) * (g + 1) + i) * s.V + t);
        const float zpt = ld_logit(zp_all, r * s.V + t);
        la_s[k * (g + 1) + i + 1] = ((double)zqt - (double)ri.mq) * s.inv_T - log(ri.Zq);
        lb_s[k * (g + 1) + i + 1] = ((double)zpt - (double)ri.mp) * s.inv_T - log(ri.Zp);
    }
    // block-wide OR of the flags (rarely any), then the barrier after the loop
    if (myflags) atomicOr(&sh_flags, myflags);
    __syncthreads();
    const int status_in = sh_flags & (SGBV_STATUS_TOKEN_RANGE | SGBV_STATUS_NONFINITE_LOGIT);
    const bool invalid = lost || status_in != 0;
    // la_s/lb_s[k][i+1] now hold log q_i(x_k^i), log p_i(x_k^i); every user below adds up the terms it needs
    // itself, in the order of a running sum (at most gamma additions, and no pass and barrier of its own)
    auto prefix = [&](const double *row, int len) {
        double acc = 0.0;
        for (int j = 1; j <= len; ++j) acc += row[j];
        return acc;
    };

    // ---- 1. weights ---------------------------------------------------------------------------
    // the float64 transcendentals of Eq. 2, one thread per (k,i) so that they run side by side
    // (the thread that fetched the row's record for step 0 still has what it needs of it); each weight
    // leaves the outcome of its trial, eta < h, as one bit for the scan
    for (int n = n_first; n < KG; n += nthreads) {
        const int k = n / g, i = n % g;
        double inv_Zq = inv_Zq_first;
        bool below = below_first;
        if (n != n_first) {
            const RowInfo ri = ws.rows[((size_t)b * K + k) * g + i];
            inv_Zq = 1.0 / ri.Zq;
            below = ri.c < 1.0f;
        }
        const double R = W_s[n] * inv_Zq;
        const double la = prefix(la_s + k * (g + 1), i), lb = prefix(lb_s + k * (g + 1), i);
        const double S = exp_short(la) * R;
        ws.resmass[(size_t)b * KG + n] = invalid ? NAN : S;
        if (i >= 1) {
            const double hv = weight_sub(la, lb, R, D_s[n] * inv_Zq, M_s[n] * inv_Zq, K, below);
            if ((double)u_s[k * g + i - 1] < hv) atomicOr(&pass_s[k], 1ull << (i - 1));
            ws.h[(size_t)b * KG + k * g + i - 1] = invalid ? NAN : hv;
        }
    }
    for (int k = tid; k < K; k += nthreads) {  // the first threads, while the last ones do Eq. 2
        const double hv = weight_full(prefix(la_s + k * (g + 1), g), prefix(lb_s + k * (g + 1), g), K);
        if ((double)u_s[k * g + g - 1] < hv) atomicOr(&pass_s[k], 1ull << (g - 1));
        ws.h[(size_t)b * KG + k * g + g - 1] = invalid ? NAN : hv;
    }
    // longest common prefix of every pair of drafts (for the membership test in H)
    for (int n = (tid + nthreads / 2) % nthreads; n < K * K; n += nthreads) {
        const int k = n / K, kp = n % K;
        int l = 0;
        while (l < g && tok_s[k * g + l] == tok_s[kp * g + l]) ++l;
        lcp_s[n] = (unsigned char)l;
    }
    __syncthreads();

    if (invalid) {
        if (tid == 0) {
            out_tau[b] = -1;
            out_f[b] = -1;
            ws.status[b] = status_in | (lost ? SGBV_STATUS_TIMEOUT : 0);
        }
        for (int j = tid; j <= g; j += nthreads) out_tokens[(size_t)b * (g + 1) + j] = -1;
        return;
    }

    // ---- 2. scan (Algorithm 1), warp 0 ---------------------------------------------------------
    if (wid == 0) {
        // The state is bit sets over the lengths 1..gamma (bit i-1 = length i): pass (shared memory, left by
        // the weights above) = the lengths whose Bernoulli trial succeeds (eta < h); rej (registers, lane l
        // owns drafts l and l + 32) = the lengths at which the draft entered H.  A draft's walk over i = tau+1..gamma does not
        // depend on its own progress (the start is fixed when the draft is entered, H only holds earlier
        // drafts), so it is evaluated for all lengths at once: the accepted length is the largest one in
        // the range whose trial passes and whose sub-block is not in H.
        auto low = [](int l) { return l >= 64 ? ~0ull : (1ull << l) - 1ull; };  // lengths 1..l
        unsigned long long rej0 = 0, rej1 = 0;
        int tau = 0, f = -1;
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
        if (lane == 0) {
            sh_i[0] = tau;
            sh_i[1] = f;
        }
    }
    __syncthreads();
    const int tau = sh_i[0], f = sh_i[1];
    const int kk = (tau == 0) ? 0 : f;
    const double us = (double)u_s[KG];

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
            const RowInfo ri = ws.rows[r];  // fetched while the tile is being located
            locate_tile(wp, nullptr, s.ntiles, us * W, false, sh_i, sh_d, sh_warp);
            const int sel = sh_i[2];
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
        // softmax(zq/T) of one row in a single pass over memory: every tile's maximum and its
        // sum of exponentials relative to that maximum, then the row maximum, the factors that move
        // the tile sums to it, the tile search and the pick inside the tile
        bool bad = false;
        float m = -INFINITY;
        constexpr int kNT = 4;  // tiles a warp has in flight
        static_assert(kTile == 256, "a lane takes 8 entries of a tile");
        const bool pieces = (reinterpret_cast<uintptr_t>(zq) % 16 == 0) && (s.V % (16 / (int)sizeof(T)) == 0);
        for (int tb = wid * kNT; tb < s.ntiles; tb += nwarps * kNT) {
            float z[kNT][kTile / 32];
            if (pieces) {  // 16-byte loads
#pragma unroll
                for (int q = 0; q < kNT; ++q) load_tile_pieces<T>(zq, tb + q, tb + q < s.ntiles, s.V, lane, z[q]);
            } else {
#pragma unroll
                for (int q = 0; q < kNT; ++q)
#pragma unroll
                    for (int e = 0; e < kTile / 32; ++e) {
                        const int x = (tb + q) * kTile + lane + 32 * e;
                        z[q][e] = (tb + q < s.ntiles && x < s.V) ? ld_logit(zq, x) : -INFINITY;
                    }
            }
            // the four tiles are reduced side by side (independent shuffle chains)
            float mt[kNT], acc[kNT];
#pragma unroll
            for (int q = 0; q < kNT; ++q) {
                mt[q] = -INFINITY;
#pragma unroll
                for (int e = 0; e < kTile / 32; ++e) {
                    bad |= (z[q][e] != z[q][e]) | (z[q][e] == INFINITY);
                    mt[q] = fmaxf(mt[q], z[q][e]);
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1)
#pragma unroll
                for (int q = 0; q < kNT; ++q) mt[q] = fmaxf(mt[q], __shfl_xor_sync(0xffffffffu, mt[q], o));
#pragma unroll
            for (int q = 0; q < kNT; ++q) {
                acc[q] = 0.0f;
                if (mt[q] > -INFINITY) {
#pragma unroll
                    for (int e = 0; e < kTile / 32; ++e) acc[q] += expo(z[q][e], mt[q], s.scale);
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1)
#pragma unroll
                for (int q = 0; q < kNT; ++q) acc[q] += __shfl_xor_sync(0xffffffffu, acc[q], o);
#pragma unroll
            for (int q = 0; q < kNT; ++q) {
                if (lane == 0 && tb + q < s.ntiles) {
                    tile_s[tb + q] = acc[q];
                    tile_m[tb + q] = mt[q];
                }
                m = fmaxf(m, mt[q]);
            }
        }
        if (lane == 0) sh_redf[wid] = m;
        bad = __syncthreads_or(bad);
        m = warp_max(lane < nwarps ? sh_redf[lane] : -INFINITY);
        if (bad || !(m > -INFINITY)) {
            flags |= SGBV_STATUS_NONFINITE_LOGIT;
        } else {
            // tile_m becomes the factor exp((m_t - m)/T) of its tile
            for (int t = tid; t < s.ntiles; t += nthreads) tile_m[t] = (tile_m[t] > -INFINITY) ? expo(tile_m[t], m, s.scale) : 0.0f;
            __syncthreads();
            // the target is us times the row's total, which the tile search computes on its way
            locate_tile(tile_s, tile_m, s.ntiles, us, true, sh_i, sh_d, sh_warp);
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
        ws.status[b] = status_in | flags;
    }
    for (int j = tid; j <= g; j += nthreads) {
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
    size_t smem = 3 * KG * sizeof(double) + 2 * (size_t)s.K * (s.gamma + 1) * sizeof(double) +
                  s.K * sizeof(unsigned long long) + KG * sizeof(int32_t) + (KG + 1) * sizeof(float) +
                  ((size_t)s.K * s.K + 15) / 16 * 16;
    Workspace ws = L.ws;
    const size_t tiles = 2 * (size_t)s.ntiles * sizeof(float);
    ws.bonus_in_smem = (s.ntiles <= kTilesInSmem && smem + tiles <= 160 * 1024) ? 1 : 0;
    if (ws.bonus_in_smem) smem += tiles;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(finish_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return SGBV_ERR_CUDA;
    }
    // programmatic stream serialisation: the kernel may be scheduled before the one ahead of it in the
    // stream has finished; it waits for that kernel itself (griddepcontrol.wait) once it needs its results
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(s.B);
    // the largest CTA with which all batch rows are still resident at once (64 registers per thread: one CTA of
    // 1024 threads per SM, two of 512, four of 256)
    cfg.blockDim = dim3(s.B <= 148 ? kMaxThreads : s.B <= 296 ? 512 : kMinThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = L.stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, finish_kernel<T>, (const T *)L.zq, (const T *)L.zp, L.tok, L.u, s, ws,
                                       L.out_tau, L.out_f, L.out_tokens);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return SGBV_ERR_CUDA;
    }
    return 1;
}

}  // namespace

int launch_finish(const Launch &L) {
    return L.dtype == SGBV_DTYPE_BF16 ? run<uint16_t>(L) : run<float>(L);
}

}  // namespace sgbv
