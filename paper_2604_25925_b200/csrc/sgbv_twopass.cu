// Generic two-sweep path: works for any V, any alignment, either dtype.
//   sweep 1  (rowstats_kernel)  slice-wise (max, sum-exp) of every target and draft row i < gamma
//   chain    (chain_kernel)     per draft: row normalisers, c_i = p(x^i)/q(x^i), kappa_i
//   sweep 2  (otreduce_kernel)  per-tile sums of the residual weights (and of the two
//                               non-negative numerator terms when c_i < 1)
// It reads each needed logit twice, so it is the fallback, not the fast path.
#include "sgbv_sample.cuh"
#include "sgbv_weights.cuh"

namespace sgbv {

namespace {

constexpr int kThreads = 256;

template <typename T>
__global__ void __launch_bounds__(kThreads)
rowstats_kernel(const T *__restrict__ zq_all, const T *__restrict__ zp_all, Shape s, float *__restrict__ part,
                int32_t *__restrict__ status) {
    const int r = blockIdx.x / s.nsplit;  // row pair (b,k,i), i < gamma
    const int sl = blockIdx.x % s.nsplit;
    const int i = r % s.gamma;
    const int bk = r / s.gamma;
    const T *zq = zq_all + ((size_t)bk * s.zq_rows + i) * s.V;
    const T *zp = zp_all + ((size_t)bk * s.gamma + i) * s.V;
    const int x0 = sl * s.tiles_per_slice * kTile;
    const int x1 = min(s.V, x0 + s.tiles_per_slice * kTile);

    __shared__ float red[4][kThreads / 32];
    __shared__ float bcast[2];

    float mq = -INFINITY, mp = -INFINITY;
    bool bad = false;
    for (int x = x0 + threadIdx.x; x < x1; x += kThreads) {
        float a = ld_logit(zq, x), b = ld_logit(zp, x);
        bad |= (a != a) | (b != b) | (a == INFINITY) | (b == INFINITY);
        mq = fmaxf(mq, a);
        mp = fmaxf(mp, b);
    }
    mq = warp_max(mq);
    mp = warp_max(mp);
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    if (lane == 0) {
        red[0][wid] = mq;
        red[1][wid] = mp;
    }
    if (__syncthreads_or(bad) && threadIdx.x == 0) atomicOr(status + bk / s.cpr, SGBV_STATUS_NONFINITE_LOGIT);
    if (threadIdx.x == 0) {
        float a = red[0][0], b = red[1][0];
        for (int w = 1; w < kThreads / 32; ++w) {
            a = fmaxf(a, red[0][w]);
            b = fmaxf(b, red[1][w]);
        }
        bcast[0] = a;
        bcast[1] = b;
    }
    __syncthreads();
    mq = bcast[0];
    mp = bcast[1];
    float sq = 0.0f, sp = 0.0f;
    if (mq > -INFINITY || mp > -INFINITY) {
        for (int x = x0 + threadIdx.x; x < x1; x += kThreads) {
            if (mq > -INFINITY) sq += expo(ld_logit(zq, x), mq, s.scale);
            if (mp > -INFINITY) sp += expo(ld_logit(zp, x), mp, s.scale);
        }
    }
    sq = warp_sum(sq);
    sp = warp_sum(sp);
    if (lane == 0) {
        red[2][wid] = sq;
        red[3][wid] = sp;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float a = 0.0f, b = 0.0f;
        for (int w = 0; w < kThreads / 32; ++w) {
            a += red[2][w];
            b += red[3][w];
        }
        float *o = part + ((size_t)r * s.nsplit + sl) * 4;
        o[0] = mq;
        o[1] = a;
        o[2] = mp;
        o[3] = b;
    }
}

// One thread per draft chain (b,k): sequential over the gamma positions.
template <typename T>
__global__ void chain_kernel(const T *__restrict__ zq_all, const T *__restrict__ zp_all,
                             const int32_t *__restrict__ tok, Shape s, const float *__restrict__ part,
                             RowInfo *__restrict__ rows, int32_t *__restrict__ status,
                             const double *__restrict__ carry_loga, const double *__restrict__ carry_logb) {
    const int bk = blockIdx.x * blockDim.x + threadIdx.x;
    if (bk >= s.B * s.cpr) return;
    // joint log-probabilities of the prefix: 0 at the start of a draft, or what Algorithm 2 carries in
    double la = carry_loga ? carry_loga[bk] : 0.0, lb = carry_logb ? carry_logb[bk] : 0.0;
    for (int i = 0; i < s.gamma; ++i) {
        const int r = bk * s.gamma + i;
        const float *p = part + (size_t)r * s.nsplit * 4;
        float mq = -INFINITY, mp = -INFINITY;
        for (int sl = 0; sl < s.nsplit; ++sl) {
            mq = fmaxf(mq, p[sl * 4 + 0]);
            mp = fmaxf(mp, p[sl * 4 + 2]);
        }
        double Zq = 0.0, Zp = 0.0;
        for (int sl = 0; sl < s.nsplit; ++sl) {
            if (p[sl * 4 + 0] > -INFINITY) Zq += (double)p[sl * 4 + 1] * exp2((double)(p[sl * 4 + 0] - mq) * (double)s.scale);
            if (p[sl * 4 + 2] > -INFINITY) Zp += (double)p[sl * 4 + 3] * exp2((double)(p[sl * 4 + 2] - mp) * (double)s.scale);
        }
        if (!(mq > -INFINITY) || !(mp > -INFINITY)) atomicOr(status + bk / s.cpr, SGBV_STATUS_NONFINITE_LOGIT);
        RowInfo ri;
        ri.Zq = Zq;
        ri.Zp = Zp;
        ri.mq = mq;
        ri.mp = mp;
        double c = exp(lb - la);
        ri.c = (float)c;
        ri.flags = 0;
        ri.pad_ = 0;
        ri.kappa = (float)(c * Zq / Zp);
        rows[r] = ri;
        if (!tok) break;  // Algorithm 2: one position, nothing follows
        int t = tok[r];
        if (t < 0 || t >= s.V) {
            atomicOr(status + bk / s.cpr, SGBV_STATUS_TOKEN_RANGE);
            t = 0;
        }
        const float zqt = ld_logit(zq_all, ((size_t)bk * s.zq_rows + i) * s.V + t);
        const float zpt = ld_logit(zp_all, ((size_t)bk * s.gamma + i) * s.V + t);
        la += ((double)zqt - (double)mq) * s.inv_T - log(Zq);
        lb += ((double)zpt - (double)mp) * s.inv_T - log(Zp);
    }
}

// One warp per 256-element tile: lanes stride the tile, one shuffle reduction per sum.
template <typename T, bool kNeedAux, bool kStoreW = true>
__device__ __forceinline__ void reduce_tiles(const T *zq, const T *zp, const Shape &s, const RowInfo &ri, int K, int t0,
                                             int t1, float *wpart, float *dpart, float *mpart) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    for (int t = t0 + wid; t < t1; t += kThreads / 32) {
        const int x0 = t * kTile, x1 = min(s.V, x0 + kTile);
        float sw = 0.0f, sd = 0.0f, sm = 0.0f;
        for (int x = x0 + lane; x < x1; x += 32) {
            float eq = expo(ld_logit(zq, x), ri.mq, s.scale);
            float ep = expo(ld_logit(zp, x), ri.mp, s.scale);
            float w, dp = 0.0f, m2 = 0.0f;
            element_terms<kNeedAux>(eq, ep, ri.kappa, ri.c, K, w, dp, m2);
            sw += w;
            sd += dp;
            sm += m2;
        }
        sw = warp_sum(sw);
        if (kNeedAux) {
            sd = warp_sum(sd);
            sm = warp_sum(sm);
        }
        if (lane == 0) {
            if (kStoreW) wpart[t] = sw;
            dpart[t] = sd;
            mpart[t] = sm;
        }
    }
}

// The same sums for rows that can be read in 16-byte pieces: a lane takes 8 entries of a cell of each tensor, two
// cells per warp are in flight.
template <typename T, bool kNeedAux, bool kStoreW = true>
__device__ __forceinline__ void reduce_tiles_pieces(const T *zq, const T *zp, const Shape &s, const RowInfo &ri, int K,
                                                    int t0, int t1, float *wpart, float *dpart, float *mpart) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    for (int t = t0 + 2 * wid; t < t1; t += 2 * (kThreads / 32)) {
        float a[2][kTile / 32], b[2][kTile / 32];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            load_tile_pieces<T>(zq, t + e, t + e < t1, s.V, lane, a[e]);
            load_tile_pieces<T>(zp, t + e, t + e < t1, s.V, lane, b[e]);
        }
        float sw[2] = {0.0f, 0.0f}, sd[2] = {0.0f, 0.0f}, sm[2] = {0.0f, 0.0f};
#pragma unroll
        for (int e = 0; e < 2; ++e)
#pragma unroll
            for (int j = 0; j < kTile / 32; ++j) {  // entries past the row hold -inf and add nothing
                const float eq = expo(a[e][j], ri.mq, s.scale), ep = expo(b[e][j], ri.mp, s.scale);
                float w, dp = 0.0f, m2 = 0.0f;
                element_terms<kNeedAux>(eq, ep, ri.kappa, ri.c, K, w, dp, m2);
                sw[e] += w;
                sd[e] += dp;
                sm[e] += m2;
            }
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            sw[e] = warp_sum(sw[e]);
            if (kNeedAux) {
                sd[e] = warp_sum(sd[e]);
                sm[e] = warp_sum(sm[e]);
            }
            if (lane == 0 && t + e < t1) {
                if (kStoreW) wpart[t + e] = sw[e];
                dpart[t + e] = sd[e];
                mpart[t + e] = sm[e];
            }
        }
    }
}

// KT: the number of drafts as a compile-time constant (the power in Eq. 2 then unrolls, in the same order of
// multiplications as the run-time loop), or 0 for the run-time value.
template <typename T, int KT>
__global__ void __launch_bounds__(kThreads)
otreduce_kernel(const T *__restrict__ zq_all, const T *__restrict__ zp_all, Shape s,
                const RowInfo *__restrict__ rows, float *__restrict__ wpart, float *__restrict__ dpart,
                float *__restrict__ mpart) {
    const int r = blockIdx.x / s.nsplit;
    const int sl = blockIdx.x % s.nsplit;
    const int i = r % s.gamma;
    const int bk = r / s.gamma;
    const T *zq = zq_all + ((size_t)bk * s.zq_rows + i) * s.V;
    const T *zp = zp_all + ((size_t)bk * s.gamma + i) * s.V;
    const RowInfo ri = rows[r];
    const int t0 = sl * s.tiles_per_slice, t1 = min(s.ntiles, t0 + s.tiles_per_slice);
    float *wp = wpart + (size_t)r * s.ntiles, *dp = dpart + (size_t)r * s.ntiles, *mp = mpart + (size_t)r * s.ntiles;
    const int K = KT ? KT : s.K;
    const bool pieces = (reinterpret_cast<uintptr_t>(zq) % 16 == 0) && (reinterpret_cast<uintptr_t>(zp) % 16 == 0) &&
                        (s.V % (16 / (int)sizeof(T)) == 0);
    if (ri.c < 1.0f) {
        if (pieces) reduce_tiles_pieces<T, true>(zq, zp, s, ri, K, t0, t1, wp, dp, mp);
        else reduce_tiles<T, true>(zq, zp, s, ri, K, t0, t1, wp, dp, mp);
    } else {
        if (pieces) reduce_tiles_pieces<T, false>(zq, zp, s, ri, K, t0, t1, wp, dp, mp);
        else reduce_tiles<T, false>(zq, zp, s, ri, K, t0, t1, wp, dp, mp);
    }
}

// Behind a fused kernel that left the two extra sums of Eq. 2 aside (large problems), two small kernels:
//   auxflag_kernel  one warp per row: for a row with c < 1 whose numerator R - (1-c)^K would cancel in that plain form
//                   (plain_form_is_safe; R from the cell sums the fused kernel wrote), the row is put on a list and
//                   marked in its record (RowInfo::pad_ = 1) for the finishing kernel;
//   auxwork_kernel  a fixed grid shares out the listed rows in slices of kAuxSliceTiles cells and writes, per cell, the
//                   sums over max(c p - q, 0) and q (c-t)^2 Q(t) from a second read of the row pair.
// A few per cent of the rows are listed; the order of the list varies from run to run, the sums do not.
constexpr int kAuxSliceTiles = 16;

__global__ void __launch_bounds__(kThreads)
auxflag_kernel(Shape s, RowInfo *__restrict__ rows, const float *__restrict__ wpart, int *__restrict__ list) {
    const int lane = threadIdx.x & 31;
    const size_t r = (size_t)blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
    if (r >= (size_t)s.B * s.cpr * s.gamma || r % s.gamma == 0) return;  // Eq. 2 is about sub-blocks of length i >= 1
    const RowInfo ri = rows[r];
    if (!(ri.c < 1.0f) || ri.flags) return;
    double sw = 0.0;
    for (int t = lane; t < s.ntiles; t += 32) sw += (double)wpart[r * s.ntiles + t];
    sw = warp_sum(sw);
    if (plain_form_is_safe(sw / ri.Zq, (double)ri.c, s.K)) return;
    if (lane == 0) {
        list[1 + atomicAdd(list, 1)] = (int)r;  // list[0] counts
        rows[r].pad_ = 1;
    }
}

template <typename T, int KT>
__global__ void __launch_bounds__(kThreads)
auxwork_kernel(const T *__restrict__ zq_all, const T *__restrict__ zp_all, Shape s, const RowInfo *__restrict__ rows,
               const int *__restrict__ list, float *__restrict__ dpart, float *__restrict__ mpart) {
    const int K = KT ? KT : s.K;
    const int per_row = (s.ntiles + kAuxSliceTiles - 1) / kAuxSliceTiles;
    const long items = (long)list[0] * per_row;
    for (long w = blockIdx.x; w < items; w += gridDim.x) {
        const int r = list[1 + w / per_row], sl = (int)(w % per_row);
        const RowInfo ri = rows[r];
        const int bk = r / s.gamma, i = r % s.gamma;
        const T *zq = zq_all + ((size_t)bk * s.zq_rows + i) * s.V;
        const T *zp = zp_all + ((size_t)bk * s.gamma + i) * s.V;
        const int t0 = sl * kAuxSliceTiles, t1 = min(s.ntiles, t0 + kAuxSliceTiles);
        float *dp = dpart + (size_t)r * s.ntiles, *mp = mpart + (size_t)r * s.ntiles;
        const bool pieces = (reinterpret_cast<uintptr_t>(zq) % 16 == 0) && (reinterpret_cast<uintptr_t>(zp) % 16 == 0) &&
                            (s.V % (16 / (int)sizeof(T)) == 0);
        if (pieces) reduce_tiles_pieces<T, true, false>(zq, zp, s, ri, K, t0, t1, nullptr, dp, mp);
        else reduce_tiles<T, true, false>(zq, zp, s, ri, K, t0, t1, nullptr, dp, mp);
    }
}

template <typename T>
void launch_ot(const Launch &L, unsigned grid) {
    const Shape &s = L.s;
    const T *zq = (const T *)L.zq, *zp = (const T *)L.zp;
#define SGBV_OT(KT) \
    otreduce_kernel<T, KT><<<grid, kThreads, 0, L.stream>>>(zq, zp, s, L.ws.rows, L.ws.wpart, L.ws.dpart, L.ws.mpart)
    switch (s.K) {
        case 1: SGBV_OT(1); break;
        case 2: SGBV_OT(2); break;
        case 3: SGBV_OT(3); break;
        case 4: SGBV_OT(4); break;
        case 8: SGBV_OT(8); break;
        default: SGBV_OT(0); break;
    }
#undef SGBV_OT
}

template <typename T>
int run(const Launch &L) {
    const Shape &s = L.s;
    const int NR = s.B * s.cpr * s.gamma;
    const unsigned grid = (unsigned)NR * (unsigned)s.nsplit;
    const T *zq = (const T *)L.zq, *zp = (const T *)L.zp;
    rowstats_kernel<T><<<grid, kThreads, 0, L.stream>>>(zq, zp, s, L.ws.part, L.ws.status);
    const int nbk = s.B * s.cpr;
    chain_kernel<T><<<(nbk + 127) / 128, 128, 0, L.stream>>>(zq, zp, L.tok, s, L.ws.part, L.ws.rows,
                                                            L.ws.status, L.carry_loga, L.carry_logb);
    if (L.ev_begin) cudaEventRecord(L.ev_begin, L.stream);
    launch_ot<T>(L, grid);
    if (L.ev_end) cudaEventRecord(L.ev_end, L.stream);
    return cudaGetLastError() == cudaSuccess ? 3 : SGBV_ERR_CUDA;
}

template <typename T>
int run_otreduce(const Launch &L) {
    const Shape &s = L.s;
    const unsigned grid = (unsigned)(s.B * s.cpr * s.gamma) * (unsigned)s.nsplit;
    launch_ot<T>(L, grid);
    return cudaGetLastError() == cudaSuccess ? 1 : SGBV_ERR_CUDA;
}

template <typename T>
int run_auxreduce(const Launch &L) {
    const Shape &s = L.s;
    const size_t NR = (size_t)s.B * s.cpr * s.gamma;
    // the list lives where the two-sweep path keeps its slice partials (at least 16 bytes per row), unused here
    int *list = reinterpret_cast<int *>(L.ws.part);
    if (cudaMemsetAsync(list, 0, sizeof(int), L.stream) != cudaSuccess) return SGBV_ERR_CUDA;
    auxflag_kernel<<<(unsigned)((NR + kThreads / 32 - 1) / (kThreads / 32)), kThreads, 0, L.stream>>>(s, L.ws.rows, L.ws.wpart,
                                                                                                     list);
    const T *zq = (const T *)L.zq, *zp = (const T *)L.zp;
    const unsigned grid = 8 * 148;
#define SGBV_AUX(KT) \
    auxwork_kernel<T, KT><<<grid, kThreads, 0, L.stream>>>(zq, zp, s, L.ws.rows, list, L.ws.dpart, L.ws.mpart)
    switch (s.K) {
        case 1: SGBV_AUX(1); break;
        case 2: SGBV_AUX(2); break;
        case 3: SGBV_AUX(3); break;
        case 4: SGBV_AUX(4); break;
        case 8: SGBV_AUX(8); break;
        default: SGBV_AUX(0); break;
    }
#undef SGBV_AUX
    return cudaGetLastError() == cudaSuccess ? 2 : SGBV_ERR_CUDA;
}

}  // namespace

// the two extra sums of Eq. 2 for the rows that need them, behind the fused kernel's chain walk
int launch_auxreduce(const Launch &L) {
    return L.dtype == SGBV_DTYPE_BF16 ? run_auxreduce<uint16_t>(L) : run_auxreduce<float>(L);
}

// the second sweep alone, over rows whose records are already in place
int launch_otreduce(const Launch &L) {
    return L.dtype == SGBV_DTYPE_BF16 ? run_otreduce<uint16_t>(L) : run_otreduce<float>(L);
}

int launch_twopass(const Launch &L) {
    return L.dtype == SGBV_DTYPE_BF16 ? run<uint16_t>(L) : run<float>(L);
}

}  // namespace sgbv
