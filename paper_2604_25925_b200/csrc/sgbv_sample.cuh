// Inverse-CDF sampling over a vocabulary row by one CTA: the pieces shared by the finishing kernels
// (Eq. 4's residual draw, the bonus draw from the target row, Algorithm 2's draw, K-SEQ's residual).
// Summation order is fixed (ascending vocabulary index, float64 running sums), so draws are reproducible.
#pragma once

#include <limits.h>

#include "sgbv_common.cuh"

namespace sgbv {

constexpr int kSampleMaxWarps = 32;  // CTAs of up to 1024 threads
constexpr int kEpt = 1;              // elements per thread inside one tile (threads beyond the tile hold none)

// Shared-memory scratch of the routines below (one per CTA).
struct SampleScratch {
    double warp[kSampleMaxWarps];
    float redf[kSampleMaxWarps];
    int pick[2];
    int i[4];
    double d[2];
};

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
static __device__ void locate_tile(const float *partials, const float *scale, int ntiles, double target, bool relative,
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


// One token from softmax(zq/T) of a single row in one pass over memory: every tile's maximum and its sum of
// exponentials relative to that maximum, then the row maximum, the factors that move the tile sums to it, the
// tile search and the pick inside the tile.  tile_s, tile_m: ntiles floats each (shared or global scratch).
// Returns the token, or -1 with `bad` set if the row holds NaN/+inf or no finite logit; row_max_out (optional)
// receives the row maximum.  On return tile_s[t] * tile_m[t] is tile t's sum of exponentials relative to the row
// maximum.  All threads must call.
template <typename T>
__device__ int draw_from_row(const T *zq, const Shape &s, double us, float *tile_s, float *tile_m, SampleScratch *sc,
                             bool &bad_out, float *row_max_out = nullptr) {
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int nthreads = blockDim.x, nwarps = nthreads / 32;
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
    if (lane == 0) sc->redf[wid] = m;
    bad = __syncthreads_or(bad);
    m = warp_max(lane < nwarps ? sc->redf[lane] : -INFINITY);
    if (bad || !(m > -INFINITY)) {
        bad_out = true;
        return -1;
    }
    bad_out = false;
    if (row_max_out) *row_max_out = m;
    // tile_m becomes the factor exp((m_t - m)/T) of its tile
    for (int t = tid; t < s.ntiles; t += nthreads) tile_m[t] = (tile_m[t] > -INFINITY) ? expo(tile_m[t], m, s.scale) : 0.0f;
    __syncthreads();
    // the target is us times the row's total, which the tile search computes on its way
    locate_tile(tile_s, tile_m, s.ntiles, us, true, sc->i, sc->d, sc->warp);
    const int sel = sc->i[2];
    const int x0 = sel * kTile, x1 = min(s.V, x0 + kTile);
    auto wfun = [&](int x) { return expo(ld_logit(zq, x), m, s.scale); };
    Pick p = pick_in_tile(x0, x1, sc->d[0], sc->d[1], wfun, sc->warp, sc->pick);
    return (p.first != INT_MAX) ? p.first : p.last;
}

}  // namespace sgbv
