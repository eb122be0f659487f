// Finishing kernel: one CTA of 1024 threads per batch row.
//   0. log a_i = log q(x_k^i), log b_i = log p(x_k^i) of every draft by running sums of the token
//      log-probabilities (row maxima and normalisers come from the streaming pass);
//   1. combine the cached per-tile sums of every (k,i) row into S_i and the acceptance weights
//      (Eq. 2 for proper sub-blocks, Eq. 3 for the whole block), in float64;
//   2. the scan of Algorithm 1 over drafts and positions with the pre-drawn uniforms;
//   3. the extra token: inverse CDF of Eq. 4's residual (located through the cached tile sums,
//      only one tile is recomputed) or of the target row after a full accept.
#include "sgbv_sample.cuh"
#include "sgbv_weights.cuh"

namespace sgbv {

namespace {

constexpr int kMaxThreads = 1024;  // CTA size when few batch rows leave most SMs idle (the kernel is a
constexpr int kMinThreads = 256;   // chain of memory latencies, so more warps per row help); else 512 or 256
constexpr int kMaxWarps = kMaxThreads / 32;
constexpr int kTilesInSmem = 4096;  // rows up to 2^20 entries keep the bonus row's tile sums in shared memory
static_assert(kMinThreads >= kTile, "one thread per element of a tile");

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
    // [K*g] per row (k,i) with c < 1: 1 = D_s and M_s hold its two extra sums, 0 = Eq. 2's numerator in its plain form
    unsigned char *exact_s = lcp_s + ((K * K + 15) / 16) * 16;
    // per-tile (sum, maximum -> factor) of the target row a bonus token is drawn from: shared memory
    // when the row has few enough tiles (the launcher then reserves the space), else global scratch
    float *tile_s = ws.bonus_in_smem ? reinterpret_cast<float *>(exact_s + ((KG + 15) / 16) * 16)
                                               : ws.bonus + (size_t)blockIdx.x * 2 * s.ntiles;  // [ntiles]
    float *tile_m = tile_s + s.ntiles;                                        // [ntiles]
    __shared__ SampleScratch sc;
    __shared__ unsigned sh_or[2];
    __shared__ int sh_flags;
    double *sh_warp = sc.warp;
    int *sh_pick = sc.pick, *sh_i = sc.i;
    double *sh_d = sc.d;

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
        const bool aux = ri.c < 1.0f && (ws.have_aux == 1 || ri.pad_ == 1);
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
            exact_s[n] = aux;
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
            const double hv = weight_sub(la, lb, R, D_s[n] * inv_Zq, M_s[n] * inv_Zq, K, below, exact_s[n] != 0);
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
        int tau, f;
        scan_block(pass_s, lcp_s, K, g, sh_or, tau, f);
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
        bool bad = false;
        y = draw_from_row<T>(zq, s, us, tile_s, tile_m, &sc, bad);
        if (bad) flags |= SGBV_STATUS_NONFINITE_LOGIT;
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

// Algorithm 2, one position: per batch row the token drawn from q_new by inverse CDF over the cached cell sums
// (one cell recomputed), the carried joint logs with that token appended, and the normaliser.  The streaming
// kernels ran with one chain per batch row, gamma = 1 and c = exp(log p(s) - log q(s)) carried in.
template <typename T>
__global__ void __launch_bounds__(kMaxThreads)
modify_finish_kernel(const T *__restrict__ zq_all, const T *__restrict__ zp_all, const float *__restrict__ u_all, Shape s,
                     Workspace ws, const double *carry_loga, const double *carry_logb, int32_t *__restrict__ out_token,
                     double *out_loga, double *out_logb, double *__restrict__ out_resmass, int32_t *__restrict__ out_status) {
    __shared__ SampleScratch sc;
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int nthreads = blockDim.x, nwarps = nthreads / 32;
    asm volatile("griddepcontrol.wait;" ::: "memory");  // (launched behind the streaming kernel)
    const bool lost = *ws.error != 0;
    const RowInfo ri = ws.rows[b];
    const int status_in = (ri.flags | (ws.prestatus ? ws.prestatus[b] : 0)) & SGBV_STATUS_NONFINITE_LOGIT;
    const float *wp = ws.wpart + (size_t)b * s.ntiles;
    double local = 0.0;
    for (int t = tid; t < s.ntiles; t += nthreads) local += (double)wp[t];
    local = warp_sum(local);
    if (lane == 0) sc.warp[wid] = local;
    __syncthreads();
    const double W = warp_sum(lane < nwarps ? sc.warp[lane] : 0.0);
    __syncthreads();
    const double la = carry_loga[b], lb = carry_logb[b];
    if (lost || status_in) {
        if (tid == 0) {
            out_token[b] = -1;
            out_loga[b] = NAN;
            out_logb[b] = NAN;
            if (out_resmass) out_resmass[b] = NAN;
            if (out_status) out_status[b] = status_in | (lost ? SGBV_STATUS_TIMEOUT : 0);
        }
        return;
    }
    const T *zq = zq_all + (size_t)b * s.V, *zp = zp_all + (size_t)b * s.V;
    const double us = (double)u_all[b];
    int y = -1, flags = 0;
    if (W > 0.0) {
        locate_tile(wp, nullptr, s.ntiles, us * W, false, sc.i, sc.d, sc.warp);
        const int sel = sc.i[2];
        const int x0 = sel * kTile, x1 = min(s.V, x0 + kTile);
        auto wfun = [&](int x) {
            float eq = expo(ld_logit(zq, x), ri.mq, s.scale);
            float ep = expo(ld_logit(zp, x), ri.mp, s.scale);
            float w, d0, d1;
            element_terms<false>(eq, ep, ri.kappa, ri.c, s.K, w, d0, d1);
            return w;
        };
        Pick pk = pick_in_tile(x0, x1, sc.d[0], sc.d[1], wfun, sc.warp, sc.pick);
        y = (pk.first != INT_MAX) ? pk.first : pk.last;
    } else {  // no residual mass at all: the draw comes from q(.|s) itself
        flags |= SGBV_STATUS_DEGENERATE_RESIDUAL;
        bool bad = false;
        float *tile_s = ws.bonus + (size_t)b * 2 * s.ntiles;
        y = draw_from_row<T>(zq, s, us, tile_s, tile_s + s.ntiles, &sc, bad);
        if (bad) flags |= SGBV_STATUS_NONFINITE_LOGIT;
    }
    if (tid == 0) {
        const bool failed = y < 0;
        out_token[b] = y;
        const double lq = failed ? NAN : ((double)ld_logit(zq, y) - (double)ri.mq) * s.inv_T - log(ri.Zq);
        const double lp = failed ? NAN : ((double)ld_logit(zp, y) - (double)ri.mp) * s.inv_T - log(ri.Zp);
        out_loga[b] = la + lq;
        out_logb[b] = lb + lp;
        if (out_resmass) out_resmass[b] = W / ri.Zq;
        if (out_status) out_status[b] = flags;
    }
}

template <typename T>
int run_modify(const Launch &L, const float *u, int32_t *out_token, double *out_loga, double *out_logb,
               double *out_resmass, int32_t *out_status) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(L.s.B);
    cfg.blockDim = dim3(L.s.B <= 148 ? kMaxThreads : L.s.B <= 296 ? 512 : kMinThreads);
    cfg.stream = L.stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, modify_finish_kernel<T>, (const T *)L.zq, (const T *)L.zp, u, L.s, L.ws,
                                       L.carry_loga, L.carry_logb, out_token, out_loga, out_logb, out_resmass, out_status);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return SGBV_ERR_CUDA;
    }
    return 1;
}

template <typename T>
int run(const Launch &L) {
    const Shape &s = L.s;
    const size_t KG = (size_t)s.K * s.gamma;
    size_t smem = 3 * KG * sizeof(double) + 2 * (size_t)s.K * (s.gamma + 1) * sizeof(double) +
                  s.K * sizeof(unsigned long long) + KG * sizeof(int32_t) + (KG + 1) * sizeof(float) +
                  ((size_t)s.K * s.K + 15) / 16 * 16 + (KG + 15) / 16 * 16;
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

int launch_modify_finish(const Launch &L, const float *u, int32_t *out_token, double *out_loga, double *out_logb,
                         double *out_resmass, int32_t *out_status) {
    return L.dtype == SGBV_DTYPE_BF16 ? run_modify<uint16_t>(L, u, out_token, out_loga, out_logb, out_resmass, out_status)
                                      : run_modify<float>(L, u, out_token, out_loga, out_logb, out_resmass, out_status);
}

}  // namespace sgbv
