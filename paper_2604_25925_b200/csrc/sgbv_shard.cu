// Vocabulary-sharded form of the verify step: every rank holds the logits of a contiguous range of the vocabulary
// (what a tensor-parallel LM head leaves behind) and the step runs as four local phases with three small exchanges
// between them, which the caller performs (an all-gather of the row statistics, an all-gather of the row sums, a
// max-all-reduce of the token matrix):
//   1. shard_stats_kernel    per row and shard: (max, sum of exponentials relative to it), the logit of the draft
//                            token if the shard holds it
//   2. shard_chain_kernel    every rank combines all shards' statistics into the row normalisers and the chain
//                            c_i, kappa_i (same arithmetic on every rank), then the cell sums of Eq. 2 / Eq. 4 over
//                            its shard (the reduction kernel of the two-sweep path) and their totals per row
//   3. shard_decide_kernel   every rank adds the shards' row sums in rank order, evaluates Eq. 2 / Eq. 3 and scans
//                            (Algorithm 1): identical decisions on every rank; the extra token's inverse CDF is
//                            split in rank order: the owner shard and the target inside it
//   4. shard_draw_kernel     the owner draws inside its shard and writes the global token id
// No kernel waits for another rank: the exchanges happen between launches.
#include "sgbv_sample.cuh"
#include "sgbv_weights.cuh"

namespace sgbv {

int launch_otreduce(const Launch &L);

namespace {

constexpr int kRec = 8;        // floats per statistics record: mq, sq, mp, sp, zq[token], zp[token], flags, unused
constexpr int kMaxRanks = 64;
constexpr int kThreads = 256;
constexpr size_t kAlign = 256;

size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

// Where the extra token of a batch row is drawn.
struct Plan {
    double frac;     // target inside the owner's share of the row, as a fraction of that share (>1: take the last entry)
    int32_t owner;   // rank that draws, -1 if the row produces no token
    int32_t mode;    // 0: Eq. 4's residual of row (k,i); 1: the target row (k,i) itself (bonus, or no residual mass)
    int32_t k, i;
};

struct ShardSpace {
    RowInfo *rows;   // [B*K*gamma], global normalisers
    double *ltok;    // [B*K*gamma][2]: log q_i(x_k^i), log p_i(x_k^i)
    float *wpart, *dpart, *mpart;  // [B*K*gamma][ntiles of the shard]
    float *bonus;    // [B][2][ntiles]
    Plan *plan;      // [B]
    int32_t *error;  // [1], always zero here (the reduction kernel's launcher wants one)
    size_t total;
};

ShardSpace carve(unsigned char *base, int B, int K, int gamma, int ntiles) {
    const size_t NR = (size_t)B * K * gamma;
    ShardSpace w;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        unsigned char *p = reinterpret_cast<unsigned char *>(reinterpret_cast<uintptr_t>(base) + off);
        off += align_up(bytes);
        return p;
    };
    w.rows = (RowInfo *)take(NR * sizeof(RowInfo));
    w.ltok = (double *)take(NR * 2 * sizeof(double));
    w.wpart = (float *)take(NR * ntiles * sizeof(float));
    w.dpart = (float *)take(NR * ntiles * sizeof(float));
    w.mpart = (float *)take(NR * ntiles * sizeof(float));
    w.bonus = (float *)take((size_t)B * 2 * ntiles * sizeof(float));
    w.plan = (Plan *)take((size_t)B * sizeof(Plan));
    w.error = (int32_t *)take(sizeof(int32_t));
    w.total = off;
    return w;
}

Shape shard_shape(int B, int K, int gamma, int Vs, float temperature) {
    Shape s;
    s.B = B;
    s.K = K;
    s.gamma = gamma;
    s.V = Vs;
    s.cpr = K;
    s.zq_rows = gamma + 1;
    s.ntiles = (Vs + kTile - 1) / kTile;
    const long rows = (long)B * K * gamma;
    long want = (4L * 148 + rows - 1) / rows;
    if (want < 1) want = 1;
    if (want > s.ntiles) want = s.ntiles;
    s.tiles_per_slice = (int)((s.ntiles + want - 1) / want);
    s.nsplit = (s.ntiles + s.tiles_per_slice - 1) / s.tiles_per_slice;
    s.scale = (float)((double)kLog2e / (double)temperature);
    s.inv_T = 1.0 / (double)temperature;
    return s;
}

// ---- phase 1 ----------------------------------------------------------------------------------------------------
// One CTA per row index (b,k,i), i <= gamma: the target row i and, for i < gamma, the draft row i of this shard.
template <typename T>
__global__ void __launch_bounds__(kThreads)
shard_stats_kernel(const T *__restrict__ zq_all, const T *__restrict__ zp_all, const int32_t *__restrict__ tok, Shape s,
                   int v_begin, int V_total, float *__restrict__ out) {
    const int row = blockIdx.x;  // (b*K + k)*(gamma+1) + i
    const int i = row % (s.gamma + 1), bk = row / (s.gamma + 1);
    const bool has_p = i < s.gamma;
    const T *zq = zq_all + (size_t)row * s.V;
    const T *zp = zp_all + ((size_t)bk * s.gamma + (has_p ? i : 0)) * s.V;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    __shared__ float red[4][kThreads / 32];
    float mq = -INFINITY, mp = -INFINITY;
    bool bad = false;
    for (int x = tid; x < s.V; x += kThreads) {
        const float a = ld_logit(zq, x);
        bad |= (a != a) | (a == INFINITY);
        mq = fmaxf(mq, a);
        if (has_p) {
            const float b = ld_logit(zp, x);
            bad |= (b != b) | (b == INFINITY);
            mp = fmaxf(mp, b);
        }
    }
    mq = warp_max(mq);
    mp = warp_max(mp);
    if (lane == 0) {
        red[0][wid] = mq;
        red[1][wid] = mp;
    }
    bad = __syncthreads_or(bad);
    mq = warp_max(lane < kThreads / 32 ? red[0][lane] : -INFINITY);
    mp = warp_max(lane < kThreads / 32 ? red[1][lane] : -INFINITY);
    float sq = 0.0f, sp = 0.0f;
    for (int x = tid; x < s.V; x += kThreads) {
        if (mq > -INFINITY) sq += expo(ld_logit(zq, x), mq, s.scale);
        if (has_p && mp > -INFINITY) sp += expo(ld_logit(zp, x), mp, s.scale);
    }
    sq = warp_sum(sq);
    sp = warp_sum(sp);
    if (lane == 0) {
        red[2][wid] = sq;
        red[3][wid] = sp;
    }
    __syncthreads();
    if (tid == 0) {
        float a = 0.0f, b = 0.0f;
        for (int w = 0; w < kThreads / 32; ++w) {  // fixed order
            a += red[2][w];
            b += red[3][w];
        }
        int flags = bad ? SGBV_STATUS_NONFINITE_LOGIT : 0;
        float zqt = -INFINITY, zpt = -INFINITY;
        if (has_p) {
            const int t = tok[(size_t)bk * s.gamma + i];
            if (t < 0 || t >= V_total) flags |= SGBV_STATUS_TOKEN_RANGE;
            else if (t >= v_begin && t < v_begin + s.V) {
                zqt = ld_logit(zq, t - v_begin);
                zpt = ld_logit(zp, t - v_begin);
            }
        }
        float *o = out + (size_t)row * kRec;
        o[0] = mq;
        o[1] = a;
        o[2] = has_p ? mp : -INFINITY;
        o[3] = has_p ? b : 0.0f;
        o[4] = zqt;
        o[5] = zpt;
        o[6] = (float)flags;
        o[7] = 0.0f;
    }
}

// The same records in one pass over memory, for shards whose rows can be read in 16-byte pieces: every lane keeps a
// running (max, sum relative to it) per tensor over the pieces it reads; the CTA merges them in a fixed order.
struct Running {
    float m, s;
};

__device__ __forceinline__ void running_add(Running &o, const float (&z)[kTile / 32], float scale, bool &bad) {
    float cm = z[0];
#pragma unroll
    for (int e = 0; e < kTile / 32; ++e) {
        bad |= (z[e] != z[e]) | (z[e] == INFINITY);
        cm = fmaxf(cm, z[e]);
    }
    if (cm > o.m) {  // (an empty sum stays empty: 0 * 2^-inf = 0)
        o.s *= exp2f((o.m - cm) * scale);
        o.m = cm;
    }
    if (o.m > -INFINITY) {
#pragma unroll
        for (int e = 0; e < kTile / 32; ++e) o.s += exp2f((z[e] - o.m) * scale);
    }
}

template <typename T>
__global__ void __launch_bounds__(kThreads)
shard_stats_pieces_kernel(const T *__restrict__ zq_all, const T *__restrict__ zp_all, const int32_t *__restrict__ tok,
                          Shape s, int v_begin, int V_total, float *__restrict__ out) {
    const int row = blockIdx.x;
    const int i = row % (s.gamma + 1), bk = row / (s.gamma + 1);
    const bool has_p = i < s.gamma;
    const T *zq = zq_all + (size_t)row * s.V;
    const T *zp = zp_all + ((size_t)bk * s.gamma + (has_p ? i : 0)) * s.V;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    constexpr int kW = kThreads / 32;
    __shared__ float red[4][kW];
    Running q{-INFINITY, 0.0f}, p{-INFINITY, 0.0f};
    bool bad = false;
    for (int t = wid * 2; t < s.ntiles; t += 2 * kW) {  // two cells of both tensors in flight per warp
        float a[2][kTile / 32], b[2][kTile / 32];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            load_tile_pieces<T>(zq, t + e, t + e < s.ntiles, s.V, lane, a[e]);
            load_tile_pieces<T>(zp, t + e, has_p && t + e < s.ntiles, s.V, lane, b[e]);
        }
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            running_add(q, a[e], s.scale, bad);
            running_add(p, b[e], s.scale, bad);
        }
    }
    const float mq_w = warp_max(q.m), mp_w = warp_max(p.m);
    if (lane == 0) {
        red[0][wid] = mq_w;
        red[1][wid] = mp_w;
    }
    bad = __syncthreads_or(bad);
    const float mq = warp_max(lane < kW ? red[0][lane] : -INFINITY);
    const float mp = warp_max(lane < kW ? red[1][lane] : -INFINITY);
    float sq = q.m > -INFINITY ? q.s * exp2f((q.m - mq) * s.scale) : 0.0f;
    float sp = p.m > -INFINITY ? p.s * exp2f((p.m - mp) * s.scale) : 0.0f;
    sq = warp_sum(sq);
    sp = warp_sum(sp);
    if (lane == 0) {
        red[2][wid] = sq;
        red[3][wid] = sp;
    }
    __syncthreads();
    if (tid == 0) {
        float a = 0.0f, b = 0.0f;
        for (int w = 0; w < kW; ++w) {  // fixed order
            a += red[2][w];
            b += red[3][w];
        }
        int flags = bad ? SGBV_STATUS_NONFINITE_LOGIT : 0;
        float zqt = -INFINITY, zpt = -INFINITY;
        if (has_p) {
            const int t = tok[(size_t)bk * s.gamma + i];
            if (t < 0 || t >= V_total) flags |= SGBV_STATUS_TOKEN_RANGE;
            else if (t >= v_begin && t < v_begin + s.V) {
                zqt = ld_logit(zq, t - v_begin);
                zpt = ld_logit(zp, t - v_begin);
            }
        }
        float *o = out + (size_t)row * kRec;
        o[0] = mq;
        o[1] = a;
        o[2] = has_p ? mp : -INFINITY;
        o[3] = has_p ? b : 0.0f;
        o[4] = zqt;
        o[5] = zpt;
        o[6] = (float)flags;
        o[7] = 0.0f;
    }
}

// ---- phase 2 ----------------------------------------------------------------------------------------------------
struct RowStats {
    double Zq, Zp;
    float mq, mp, zqt, zpt;
    int flags;
};

// All shards' records of one row into the row's statistics: maxima, the sums of exponentials moved to them (float64,
// rank order), the token's logits (held by exactly one shard), the flags.
__device__ RowStats combine_stats(const float *__restrict__ stats_all, int R, size_t nrows, size_t row, float scale) {
    RowStats o;
    o.mq = o.mp = o.zqt = o.zpt = -INFINITY;
    o.flags = 0;
    for (int r = 0; r < R; ++r) {
        const float *rec = stats_all + ((size_t)r * nrows + row) * kRec;
        o.mq = fmaxf(o.mq, rec[0]);
        o.mp = fmaxf(o.mp, rec[2]);
        o.zqt = fmaxf(o.zqt, rec[4]);
        o.zpt = fmaxf(o.zpt, rec[5]);
        o.flags |= (int)rec[6];
    }
    o.Zq = o.Zp = 0.0;
    for (int r = 0; r < R; ++r) {
        const float *rec = stats_all + ((size_t)r * nrows + row) * kRec;
        if (rec[0] > -INFINITY) o.Zq += (double)rec[1] * exp2((double)(rec[0] - o.mq) * (double)scale);
        if (rec[2] > -INFINITY) o.Zp += (double)rec[3] * exp2((double)(rec[2] - o.mp) * (double)scale);
    }
    return o;
}

// Normalisers, c_i and kappa_i of every row, as the one-device path computes them.  One thread per row (b,k,i)
// combines the shards' records (the costly part: one float64 exponential per shard and tensor), a CTA holds whole
// chains, and every thread then adds up the token log-probabilities before its row in the order of a running sum.
constexpr int kChainThreads = 256;
__global__ void __launch_bounds__(kChainThreads)
shard_chain_kernel(const float *__restrict__ stats_all, int R, Shape s, int chains_per_cta,
                   RowInfo *__restrict__ rows, double *__restrict__ ltok) {
    __shared__ double lq_s[kChainThreads], lp_s[kChainThreads];
    const int tid = threadIdx.x;
    const int chain = tid / s.gamma, i = tid % s.gamma;
    const int bk = blockIdx.x * chains_per_cta + chain;
    const bool mine = chain < chains_per_cta && bk < s.B * s.K;
    const size_t nrows = (size_t)s.B * s.K * (s.gamma + 1);
    RowStats st{};
    if (mine) {
        st = combine_stats(stats_all, R, nrows, (size_t)bk * (s.gamma + 1) + i, s.scale);
        lq_s[tid] = ((double)st.zqt - (double)st.mq) * s.inv_T - log(st.Zq);
        lp_s[tid] = ((double)st.zpt - (double)st.mp) * s.inv_T - log(st.Zp);
    }
    __syncthreads();
    if (!mine) return;
    double la = 0.0, lb = 0.0;
    for (int j = 0; j < i; ++j) {
        la += lq_s[chain * s.gamma + j];
        lb += lp_s[chain * s.gamma + j];
    }
    RowInfo ri;
    ri.Zq = st.Zq;
    ri.Zp = st.Zp;
    ri.mq = st.mq;
    ri.mp = st.mp;
    const double c = exp(lb - la);
    ri.c = (float)c;
    ri.kappa = (float)(c * st.Zq / st.Zp);
    ri.flags = st.flags;
    if (!(st.mq > -INFINITY) || !(st.mp > -INFINITY)) ri.flags |= SGBV_STATUS_NONFINITE_LOGIT;
    ri.pad_ = 0;
    const size_t r = (size_t)bk * s.gamma + i;
    rows[r] = ri;
    ltok[2 * r] = lq_s[tid];
    ltok[2 * r + 1] = lp_s[tid];
}

// One warp per row: the totals of the shard's cell sums (float64, fixed order).
__global__ void __launch_bounds__(kThreads)
shard_rowsums_kernel(Shape s, const RowInfo *__restrict__ rows, const float *__restrict__ wpart,
                     const float *__restrict__ dpart, const float *__restrict__ mpart, double *__restrict__ out) {
    const int lane = threadIdx.x & 31;
    const size_t r = (size_t)blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
    if (r >= (size_t)s.B * s.K * s.gamma) return;
    const bool aux = rows[r].c < 1.0f;
    double sw = 0.0, sd = 0.0, sm = 0.0;
    for (int t = lane; t < s.ntiles; t += 32) {
        sw += (double)wpart[r * s.ntiles + t];
        if (aux) {
            sd += (double)dpart[r * s.ntiles + t];
            sm += (double)mpart[r * s.ntiles + t];
        }
    }
    sw = warp_sum(sw);
    sd = warp_sum(sd);
    sm = warp_sum(sm);
    if (lane == 0) {
        out[3 * r] = sw;
        out[3 * r + 1] = sd;
        out[3 * r + 2] = sm;
    }
}

// ---- phase 3 ----------------------------------------------------------------------------------------------------
// One CTA per batch row; every rank runs it on the same gathered inputs and reaches the same decisions.
__global__ void __launch_bounds__(kThreads)
shard_decide_kernel(const int32_t *__restrict__ tok_all, const float *__restrict__ u_all, Shape s,
                    const float *__restrict__ stats_all, const double *__restrict__ sums_all, int R,
                    const RowInfo *__restrict__ rows, const double *__restrict__ ltok, Plan *__restrict__ plan,
                    int32_t *__restrict__ out_tau, int32_t *__restrict__ out_f, int32_t *__restrict__ out_tokens,
                    double *__restrict__ out_h, double *__restrict__ out_resmass, int32_t *__restrict__ out_status) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int K = s.K, g = s.gamma, KG = K * g;
    double *W_s = reinterpret_cast<double *>(smem_raw);
    double *D_s = W_s + KG;
    double *M_s = D_s + KG;
    double *la_s = M_s + KG;               // [K*(g+1)] log q_i(x_k^i) at [k][i+1]
    double *lb_s = la_s + K * (g + 1);
    unsigned long long *pass_s = reinterpret_cast<unsigned long long *>(lb_s + K * (g + 1));
    int32_t *tok_s = reinterpret_cast<int32_t *>(pass_s + K);
    float *u_s = reinterpret_cast<float *>(tok_s + KG);
    unsigned char *lcp_s = reinterpret_cast<unsigned char *>(u_s + KG + 1);
    __shared__ unsigned sh_or[2];
    __shared__ int sh_i[2];
    __shared__ int sh_flags;

    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const size_t NR = (size_t)s.B * KG;
    const int32_t *tok = tok_all + (size_t)b * KG;
    for (int n = tid; n <= KG; n += kThreads) u_s[n] = u_all[(size_t)b * (KG + 1) + n];
    for (int n = tid; n < KG; n += kThreads) tok_s[n] = tok[n];
    for (int k = tid; k < K; k += kThreads) pass_s[k] = 0ull;
    if (tid == 0) sh_flags = 0;
    __syncthreads();
    int myflags = 0;
    for (int n = tid; n < KG; n += kThreads) {
        const size_t r = (size_t)b * KG + n;
        myflags |= rows[r].flags;
        double sw = 0.0, sd = 0.0, sm = 0.0;
        for (int q = 0; q < R; ++q) {  // rank order
            const double *v = sums_all + ((size_t)q * NR + r) * 3;
            sw += v[0];
            sd += v[1];
            sm += v[2];
        }
        W_s[n] = sw;
        D_s[n] = sd;
        M_s[n] = sm;
        const int k = n / g, i = n % g;
        la_s[k * (g + 1) + i + 1] = ltok[2 * r];
        lb_s[k * (g + 1) + i + 1] = ltok[2 * r + 1];
    }
    if (myflags) atomicOr(&sh_flags, myflags);
    __syncthreads();
    const int status_in = sh_flags & (SGBV_STATUS_TOKEN_RANGE | SGBV_STATUS_NONFINITE_LOGIT);
    const bool invalid = status_in != 0;
    auto prefix = [&](const double *row, int len) {
        double acc = 0.0;
        for (int j = 1; j <= len; ++j) acc += row[j];
        return acc;
    };
    // Eq. 2 for the proper sub-blocks, Eq. 3 for the whole block; each weight leaves the outcome of its trial
    for (int n = tid; n < KG; n += kThreads) {
        const int k = n / g, i = n % g;
        const RowInfo ri = rows[(size_t)b * KG + n];
        const double inv_Zq = 1.0 / ri.Zq;
        const double Rr = W_s[n] * inv_Zq;
        const double la = prefix(la_s + k * (g + 1), i), lb = prefix(lb_s + k * (g + 1), i);
        if (out_resmass) out_resmass[(size_t)b * KG + n] = invalid ? NAN : exp_short(la) * Rr;
        if (i >= 1) {
            const double hv = weight_sub(la, lb, Rr, D_s[n] * inv_Zq, M_s[n] * inv_Zq, K, ri.c < 1.0f, true);
            if ((double)u_s[k * g + i - 1] < hv) atomicOr(&pass_s[k], 1ull << (i - 1));
            if (out_h) out_h[(size_t)b * KG + k * g + i - 1] = invalid ? NAN : hv;
        }
    }
    for (int k = tid; k < K; k += kThreads) {
        const double hv = weight_full(prefix(la_s + k * (g + 1), g), prefix(lb_s + k * (g + 1), g), K);
        if ((double)u_s[k * g + g - 1] < hv) atomicOr(&pass_s[k], 1ull << (g - 1));
        if (out_h) out_h[(size_t)b * KG + k * g + g - 1] = invalid ? NAN : hv;
    }
    for (int n = tid; n < K * K; n += kThreads) {
        const int k = n / K, kp = n % K;
        int l = 0;
        while (l < g && tok_s[k * g + l] == tok_s[kp * g + l]) ++l;
        lcp_s[n] = (unsigned char)l;
    }
    __syncthreads();
    if (wid == 0 && !invalid) {
        int tau, f;
        scan_block(pass_s, lcp_s, K, g, sh_or, tau, f);
        if (lane == 0) {
            sh_i[0] = tau;
            sh_i[1] = f;
        }
    }
    __syncthreads();
    int tau = invalid ? -1 : sh_i[0], f = invalid ? -1 : sh_i[1];
    int status = status_in;
    if (tid == 0) {
        Plan pl;
        pl.owner = -1;
        pl.mode = 0;
        pl.k = pl.i = 0;
        pl.frac = 0.0;
        if (!invalid) {
            const int kk = (tau == 0) ? 0 : f;
            const double us = (double)u_s[KG];
            const bool residual = tau < g && W_s[kk * g + tau] > 0.0;
            if (tau < g && !residual) status |= SGBV_STATUS_DEGENERATE_RESIDUAL;
            pl.mode = residual ? 0 : 1;
            pl.k = kk;
            pl.i = tau;
            // the shards' shares of the mass the token is drawn from, in vocabulary (= rank) order
            const size_t nrows = (size_t)s.B * K * (g + 1);
            const size_t qrow = ((size_t)b * K + kk) * (g + 1) + tau;
            const size_t rrow = (size_t)b * KG + kk * g + (residual ? tau : 0);
            float m = -INFINITY;
            bool bad = false;
            if (!residual)
                for (int q = 0; q < R; ++q) {
                    const float *rec = stats_all + ((size_t)q * nrows + qrow) * kRec;
                    m = fmaxf(m, rec[0]);
                    bad |= ((int)rec[6] & SGBV_STATUS_NONFINITE_LOGIT) != 0;
                }
            auto share = [&](int q) {
                if (residual) return sums_all[((size_t)q * NR + rrow) * 3];
                const float *rec = stats_all + ((size_t)q * nrows + qrow) * kRec;
                return rec[0] > -INFINITY ? (double)rec[1] * exp2((double)(rec[0] - m) * (double)s.scale) : 0.0;
            };
            double total = 0.0;
            for (int q = 0; q < R; ++q) total += share(q);
            if (bad || !(total > 0.0)) {  // the row a token would be drawn from is unusable
                status |= SGBV_STATUS_NONFINITE_LOGIT;
                tau = f = -1;
            } else {
                const double target = us * total;
                double cum = 0.0;
                int last = -1;
                for (int q = 0; q < R; ++q) {
                    const double v = share(q);
                    if (v > 0.0) last = q;
                    if (pl.owner < 0 && cum + v > target) {
                        pl.owner = q;
                        pl.frac = (target - cum) / v;
                    }
                    cum += v;
                }
                if (pl.owner < 0) {  // rounding left no crossing: the last entry with positive weight
                    pl.owner = last;
                    pl.frac = 2.0;
                }
            }
        }
        plan[b] = pl;
        out_tau[b] = tau;
        out_f[b] = f;
        if (out_status) out_status[b] = status;
        sh_i[0] = tau;
        sh_i[1] = f;
    }
    __syncthreads();
    tau = sh_i[0];
    f = sh_i[1];
    // the accepted prefix; the slot of the extra token is filled by the owner's drawing kernel and reaches the other
    // ranks through the max-all-reduce of this matrix
    for (int j = tid; j <= g; j += kThreads)
        out_tokens[(size_t)b * (g + 1) + j] = (tau > 0 && j < tau) ? tok_s[f * g + j] : -1;
}

// ---- phase 4 ----------------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(kThreads)
shard_draw_kernel(const T *__restrict__ zq_all, const T *__restrict__ zp_all, Shape s, int v_begin, int rank,
                  const RowInfo *__restrict__ rows, const float *__restrict__ wpart, float *__restrict__ bonus,
                  const Plan *__restrict__ plan, int32_t *__restrict__ tokens) {
    __shared__ SampleScratch sc;
    const int b = blockIdx.x;
    const Plan pl = plan[b];
    if (pl.owner != rank) return;
    const int K = s.K, g = s.gamma;
    const T *zq = zq_all + (((size_t)b * K + pl.k) * (g + 1) + pl.i) * s.V;
    int y = -1;
    if (pl.mode == 0) {
        const size_t r = ((size_t)b * K + pl.k) * g + pl.i;
        const RowInfo ri = rows[r];
        const T *zp = zp_all + r * s.V;
        locate_tile(wpart + r * s.ntiles, nullptr, s.ntiles, pl.frac, true, sc.i, sc.d, sc.warp);
        const int sel = sc.i[2];
        const int x0 = sel * kTile, x1 = min(s.V, x0 + kTile);
        auto wfun = [&](int x) {
            float eq = expo(ld_logit(zq, x), ri.mq, s.scale);
            float ep = expo(ld_logit(zp, x), ri.mp, s.scale);
            float w, d0, d1;
            element_terms<false>(eq, ep, ri.kappa, ri.c, K, w, d0, d1);
            return w;
        };
        const Pick p = pick_in_tile(x0, x1, sc.d[0], sc.d[1], wfun, sc.warp, sc.pick);
        y = (p.first != INT_MAX) ? p.first : p.last;
    } else {
        bool bad = false;
        float *tile_s = bonus + (size_t)b * 2 * s.ntiles;
        y = draw_from_row<T>(zq, s, pl.frac, tile_s, tile_s + s.ntiles, &sc, bad);
    }
    if (threadIdx.x == 0 && y >= 0) tokens[(size_t)b * (g + 1) + pl.i] = y + v_begin;
}

int check(int B, int K, int gamma, int Vs, int dtype) {
    if (B < 1 || K < 1 || gamma < 1 || Vs < 1 || K > kMaxK || gamma > kMaxGamma || Vs > kMaxV) return SGBV_ERR_SHAPE;
    if (dtype != SGBV_DTYPE_F32 && dtype != SGBV_DTYPE_BF16) return SGBV_ERR_SHAPE;
    if ((double)B * K * gamma > 2.0e8) return SGBV_ERR_SHAPE;
    return SGBV_OK;
}

bool good_T(float t) { return t > 0.0f && isfinite(t); }

int last_error() { return cudaGetLastError() == cudaSuccess ? SGBV_OK : SGBV_ERR_CUDA; }

}  // namespace
}  // namespace sgbv

using namespace sgbv;

extern "C" {

int sgbv_shard_workspace_bytes(int B, int K, int gamma, int shard_V, int dtype, size_t *out_bytes) {
    if (!out_bytes) return SGBV_ERR_NULL;
    int rc = check(B, K, gamma, shard_V, dtype);
    if (rc != SGBV_OK) return rc;
    *out_bytes = carve(nullptr, B, K, gamma, (shard_V + kTile - 1) / kTile).total;
    return SGBV_OK;
}

int sgbv_shard_stats(const void *target_shard, const void *draft_shard, int dtype, const int32_t *draft_tokens, int B,
                     int K, int gamma, int shard_V, int v_begin, int V, float temperature, float *out_stats,
                     void *stream) {
    if (!target_shard || !draft_shard || !draft_tokens || !out_stats) return SGBV_ERR_NULL;
    int rc = check(B, K, gamma, shard_V, dtype);
    if (rc != SGBV_OK) return rc;
    if (v_begin < 0 || V > kMaxV || (long)v_begin + shard_V > (long)V) return SGBV_ERR_SHAPE;
    if (!good_T(temperature)) return SGBV_ERR_TEMPERATURE;
    const size_t esz = dtype == SGBV_DTYPE_BF16 ? 2 : 4;
    if (((uintptr_t)target_shard % esz) || ((uintptr_t)draft_shard % esz) || ((uintptr_t)draft_tokens % 4) ||
        ((uintptr_t)out_stats % 4))
        return SGBV_ERR_ALIGN;
    const Shape s = shard_shape(B, K, gamma, shard_V, temperature);
    const unsigned grid = (unsigned)((size_t)B * K * (gamma + 1));
    cudaStream_t st = (cudaStream_t)stream;
    // rows that start on 16-byte boundaries are read in 16-byte pieces, in one pass
    const bool pieces = ((uintptr_t)target_shard % 16 == 0) && ((uintptr_t)draft_shard % 16 == 0) &&
                        (shard_V % (16 / (int)esz) == 0);
    if (dtype == SGBV_DTYPE_BF16) {
        const uint16_t *zq = (const uint16_t *)target_shard, *zp = (const uint16_t *)draft_shard;
        if (pieces) shard_stats_pieces_kernel<uint16_t><<<grid, kThreads, 0, st>>>(zq, zp, draft_tokens, s, v_begin, V, out_stats);
        else shard_stats_kernel<uint16_t><<<grid, kThreads, 0, st>>>(zq, zp, draft_tokens, s, v_begin, V, out_stats);
    } else {
        const float *zq = (const float *)target_shard, *zp = (const float *)draft_shard;
        if (pieces) shard_stats_pieces_kernel<float><<<grid, kThreads, 0, st>>>(zq, zp, draft_tokens, s, v_begin, V, out_stats);
        else shard_stats_kernel<float><<<grid, kThreads, 0, st>>>(zq, zp, draft_tokens, s, v_begin, V, out_stats);
    }
    return last_error();
}

int sgbv_shard_sums(const void *target_shard, const void *draft_shard, int dtype, int B, int K, int gamma, int shard_V,
                    float temperature, const float *stats_all, int n_ranks, void *workspace, size_t workspace_bytes,
                    double *out_sums, void *stream_) {
    if (!target_shard || !draft_shard || !stats_all || !workspace || !out_sums) return SGBV_ERR_NULL;
    int rc = check(B, K, gamma, shard_V, dtype);
    if (rc != SGBV_OK) return rc;
    if (n_ranks < 1 || n_ranks > kMaxRanks) return SGBV_ERR_SHAPE;
    if (!good_T(temperature)) return SGBV_ERR_TEMPERATURE;
    const size_t esz = dtype == SGBV_DTYPE_BF16 ? 2 : 4;
    if (((uintptr_t)target_shard % esz) || ((uintptr_t)draft_shard % esz) || ((uintptr_t)stats_all % 4) ||
        ((uintptr_t)out_sums % 8))
        return SGBV_ERR_ALIGN;
    const Shape s = shard_shape(B, K, gamma, shard_V, temperature);
    const ShardSpace w = carve((unsigned char *)workspace, B, K, gamma, s.ntiles);
    if (workspace_bytes < w.total || ((uintptr_t)workspace % kAlign)) return SGBV_ERR_WORKSPACE;
    cudaStream_t stream = (cudaStream_t)stream_;
    const int nbk = B * K, chains_per_cta = kChainThreads / gamma;  // gamma <= 64: at least four chains per CTA
    shard_chain_kernel<<<(nbk + chains_per_cta - 1) / chains_per_cta, kChainThreads, 0, stream>>>(
        stats_all, n_ranks, s, chains_per_cta, w.rows, w.ltok);
    Launch L;
    L.zq = target_shard;
    L.zp = draft_shard;
    L.dtype = dtype;
    L.tok = nullptr;
    L.u = nullptr;
    L.s = s;
    L.ws = Workspace{};
    L.ws.rows = w.rows;
    L.ws.wpart = w.wpart;
    L.ws.dpart = w.dpart;
    L.ws.mpart = w.mpart;
    L.stream = stream;
    rc = launch_otreduce(L);
    if (rc < 0) return rc;
    const size_t NR = (size_t)B * K * gamma;
    shard_rowsums_kernel<<<(unsigned)((NR + kThreads / 32 - 1) / (kThreads / 32)), kThreads, 0, stream>>>(
        s, w.rows, w.wpart, w.dpart, w.mpart, out_sums);
    return last_error();
}

int sgbv_shard_decide(const int32_t *draft_tokens, const float *uniforms, int B, int K, int gamma, int shard_V,
                      float temperature, const float *stats_all, const double *sums_all, int n_ranks, void *workspace,
                      size_t workspace_bytes, int32_t *out_accept_len, int32_t *out_draft_idx, int32_t *out_tokens,
                      double *out_h, double *out_resmass, int32_t *out_status, void *stream) {
    if (!draft_tokens || !uniforms || !stats_all || !sums_all || !workspace || !out_accept_len || !out_draft_idx ||
        !out_tokens)
        return SGBV_ERR_NULL;
    int rc = check(B, K, gamma, shard_V, SGBV_DTYPE_F32);
    if (rc != SGBV_OK) return rc;
    if (n_ranks < 1 || n_ranks > kMaxRanks) return SGBV_ERR_SHAPE;
    if (!good_T(temperature)) return SGBV_ERR_TEMPERATURE;
    if (((uintptr_t)draft_tokens % 4) || ((uintptr_t)uniforms % 4) || ((uintptr_t)stats_all % 4) ||
        ((uintptr_t)sums_all % 8) || ((uintptr_t)out_accept_len % 4) || ((uintptr_t)out_draft_idx % 4) ||
        ((uintptr_t)out_tokens % 4) || ((uintptr_t)out_h % 8) || ((uintptr_t)out_resmass % 8) ||
        ((uintptr_t)out_status % 4))
        return SGBV_ERR_ALIGN;
    const Shape s = shard_shape(B, K, gamma, shard_V, temperature);
    const ShardSpace w = carve((unsigned char *)workspace, B, K, gamma, s.ntiles);
    if (workspace_bytes < w.total || ((uintptr_t)workspace % kAlign)) return SGBV_ERR_WORKSPACE;
    const size_t KG = (size_t)K * gamma;
    const size_t smem = 3 * KG * sizeof(double) + 2 * (size_t)K * (gamma + 1) * sizeof(double) +
                        K * sizeof(unsigned long long) + KG * sizeof(int32_t) + (KG + 1) * sizeof(float) +
                        ((size_t)K * K + 15) / 16 * 16;
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(shard_decide_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return SGBV_ERR_CUDA;
    shard_decide_kernel<<<B, kThreads, smem, (cudaStream_t)stream>>>(draft_tokens, uniforms, s, stats_all, sums_all,
                                                                    n_ranks, w.rows, w.ltok, w.plan, out_accept_len,
                                                                    out_draft_idx, out_tokens, out_h, out_resmass,
                                                                    out_status);
    return last_error();
}

int sgbv_shard_draw(const void *target_shard, const void *draft_shard, int dtype, int B, int K, int gamma, int shard_V,
                    int v_begin, float temperature, int rank, void *workspace, size_t workspace_bytes,
                    int32_t *tokens, void *stream) {
    if (!target_shard || !draft_shard || !workspace || !tokens) return SGBV_ERR_NULL;
    int rc = check(B, K, gamma, shard_V, dtype);
    if (rc != SGBV_OK) return rc;
    if (rank < 0 || rank >= kMaxRanks || v_begin < 0) return SGBV_ERR_SHAPE;
    if (!good_T(temperature)) return SGBV_ERR_TEMPERATURE;
    const size_t esz = dtype == SGBV_DTYPE_BF16 ? 2 : 4;
    if (((uintptr_t)target_shard % esz) || ((uintptr_t)draft_shard % esz) || ((uintptr_t)tokens % 4)) return SGBV_ERR_ALIGN;
    const Shape s = shard_shape(B, K, gamma, shard_V, temperature);
    const ShardSpace w = carve((unsigned char *)workspace, B, K, gamma, s.ntiles);
    if (workspace_bytes < w.total || ((uintptr_t)workspace % kAlign)) return SGBV_ERR_WORKSPACE;
    if (dtype == SGBV_DTYPE_BF16)
        shard_draw_kernel<uint16_t><<<B, kThreads, 0, (cudaStream_t)stream>>>(
            (const uint16_t *)target_shard, (const uint16_t *)draft_shard, s, v_begin, rank, w.rows, w.wpart, w.bonus,
            w.plan, tokens);
    else
        shard_draw_kernel<float><<<B, kThreads, 0, (cudaStream_t)stream>>>(
            (const float *)target_shard, (const float *)draft_shard, s, v_begin, rank, w.rows, w.wpart, w.bonus, w.plan,
            tokens);
    return last_error();
}

}  // extern "C"
