// Fused single-read path (steps A1-A3): one thread-block cluster walks one draft chain (b,k).
//
// For every position i = 0..gamma-1 of the chain the cluster
//   * streams the target row and the draft row from HBM exactly once: one elected thread issues
//     bulk asynchronous copies (cp.async.bulk + mbarrier transaction counts) of 4096-element chunks
//     into a shared-memory ring that runs ahead across rows and chains;
//   * keeps the whole row pair resident in REGISTERS (each CTA of the cluster owns a contiguous
//     slice of the vocabulary, each thread 8 elements of every chunk), so the second sweep of the
//     coupling sum never re-reads memory;
//   * reduces max and sum-exp per CTA (warp shuffles + shared memory), exchanges the CTA partials
//     through distributed shared memory with one cluster barrier per row, derives the chain
//     scalars (log a_i, log b_i, c_i, kappa_i) redundantly and identically in every CTA;
//   * runs the second sweep from registers and writes one partial sum per 256-element cell
//     (a cell is what one warp owns in one chunk: 256 contiguous vocabulary entries).
// The finishing kernel (weights, scan, extra token) consumes the cell sums.
//
// Every wait on an mbarrier is bounded; on expiry the CTA records an error flag and keeps
// executing the protocol (all cluster barriers are still reached), so a lost copy cannot hang.
#include "sgbv_common.cuh"

namespace sgbv {

namespace {

constexpr int kFThreads = 512;
constexpr int kFWarps = kFThreads / 32;
constexpr int kCell = kTile;               // 256 contiguous elements: one warp's share of a chunk
constexpr int kChunk = kFWarps * kCell;    // 4096 elements per chunk per tensor
constexpr int kLag = 1;                    // the producer refills the stage consumed kLag chunks ago
constexpr int kSpinLimit = 1 << 22;
static_assert(kTile == 256, "the fused path writes one partial sum per 256-element cell");

struct FusedParams {
    const void *zq;
    const void *zp;
    const int32_t *tok;
    Shape s;
    Workspace ws;
    int cluster;      // CTAs per cluster
    int slice_len;    // vocabulary elements per CTA (multiple of kCell)
    int stages;       // ring depth
    int nchains;      // B*K
    int *error_flag;  // set to 1 if a bounded wait expired
};

// ---- PTX wrappers ------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: returns false if the phase did not complete within the spin limit.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity) {
    for (int it = 0; it < kSpinLimit; ++it) {
        if (mbar_test(bar, parity)) return true;
        if (it > 128) __nanosleep(40);
    }
    return false;
}
__device__ __forceinline__ void bulk_load(void *dst, const void *src, uint32_t bytes, uint64_t *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float4 ld_dsmem_f4(const void *local, uint32_t rank) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(local)), "r"(rank));
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "r"(remote)
                 : "memory");
    return v;
}
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// ---- shared memory layout ------------------------------------------------------------------------
struct Control {
    uint64_t full[8];
    uint64_t empty[8];
    float4 slot[2];        // this CTA's (mq, Zq, mp, Zp), double-buffered by row parity
    float red[4][kFWarps];
    float bc[8];           // fq, kp, c, aux, eq-reference, ep-reference
    int32_t tok[kMaxGamma];
};

// Reads this lane's 8 elements of one chunk of one tensor from the ring.
template <typename T>
__device__ __forceinline__ void read_cell(const unsigned char *stage_base, int warp, int lane, float (&v)[8]);
template <>
__device__ __forceinline__ void read_cell<float>(const unsigned char *stage_base, int warp, int lane, float (&v)[8]) {
    const float4 *p = reinterpret_cast<const float4 *>(stage_base) + warp * 64 + lane;
    const float4 a = p[0], b = p[32];
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
template <>
__device__ __forceinline__ void read_cell<uint16_t>(const unsigned char *stage_base, int warp, int lane, float (&v)[8]) {
    const uint4 a = reinterpret_cast<const uint4 *>(stage_base)[warp * 32 + lane];
    v[0] = __uint_as_float(a.x << 16); v[1] = __uint_as_float(a.x & 0xffff0000u);
    v[2] = __uint_as_float(a.y << 16); v[3] = __uint_as_float(a.y & 0xffff0000u);
    v[4] = __uint_as_float(a.z << 16); v[5] = __uint_as_float(a.z & 0xffff0000u);
    v[6] = __uint_as_float(a.w << 16); v[7] = __uint_as_float(a.w & 0xffff0000u);
}
// Offset (in elements, within the 256-element cell) of this lane's e-th element.
template <typename T>
__device__ __forceinline__ int cell_offset(int lane, int e) {
    if (sizeof(T) == 4) return (e < 4) ? lane * 4 + e : 128 + lane * 4 + (e - 4);
    return lane * 8 + e;
}

// Second sweep over the register-resident row: cell sums of the residual weight and, for c < 1, of
// the two non-negative numerator terms.  eq/ep are in CTA-max units; fq rescales eq to row-max
// units and kp = kappa * fp does the same for the draft side.
template <int NCH, int KT, bool kAux>
__device__ __forceinline__ void sweep_two(const float (&eq)[NCH][8], const float (&ep)[NCH][8], float fq, float kp,
                                          float c, int K, int lane, int first_cell, int ncells_valid, int warp,
                                          float *wpart, float *dpart, float *mpart) {
    const float v1 = 1.0f - c;
#pragma unroll
    for (int j = 0; j < NCH; ++j) {
        float sw = 0.0f, sd = 0.0f, sm = 0.0f;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const float q = fq * eq[j][e];
            const float diff = fmaf(-kp, ep[j][e], q);
            const float d = fmaxf(diff, 0.0f);
            const float r = (d > 0.0f) ? __fdividef(d, q) : 0.0f;
            float pw = d;
            if (KT > 0) {
#pragma unroll
                for (int t = 1; t < KT; ++t) pw *= r;
            } else {
                for (int t = 1; t < K; ++t) pw *= r;
            }
            sw += pw;
            if (kAux) {
                sd += fmaxf(-diff, 0.0f);
                float acc = 0.0f;
                if (KT > 0) {
                    if (KT >= 2) {
                        acc = 1.0f;
                        float vj = 1.0f;
#pragma unroll
                        for (int t = 1; t <= KT - 2; ++t) {
                            vj *= v1;
                            acc = fmaf(acc, r, (float)(t + 1) * vj);
                        }
                    }
                } else if (K >= 2) {
                    acc = 1.0f;
                    float vj = 1.0f;
                    for (int t = 1; t <= K - 2; ++t) {
                        vj *= v1;
                        acc = fmaf(acc, r, (float)(t + 1) * vj);
                    }
                }
                const float ct = c - 1.0f + r;
                sm = fmaf(q * ct * ct, acc, sm);
            }
        }
        sw = warp_sum(sw);
        if (kAux) {
            sd = warp_sum(sd);
            sm = warp_sum(sm);
        }
        const int cell = j * kFWarps + warp;  // cell index inside this CTA's slice
        if (lane == 0 && cell < ncells_valid) {
            wpart[first_cell + cell] = sw;
            if (kAux) {
                dpart[first_cell + cell] = sd;
                mpart[first_cell + cell] = sm;
            }
        }
    }
}

template <int NCH, bool kAux>
__device__ __forceinline__ void sweep_two_dispatch(const float (&eq)[NCH][8], const float (&ep)[NCH][8], float fq,
                                                   float kp, float c, int K, int lane, int first_cell,
                                                   int ncells_valid, int warp, float *wpart, float *dpart,
                                                   float *mpart) {
    switch (K) {
        case 1: sweep_two<NCH, 1, kAux>(eq, ep, fq, kp, c, K, lane, first_cell, ncells_valid, warp, wpart, dpart, mpart); break;
        case 2: sweep_two<NCH, 2, kAux>(eq, ep, fq, kp, c, K, lane, first_cell, ncells_valid, warp, wpart, dpart, mpart); break;
        case 3: sweep_two<NCH, 3, kAux>(eq, ep, fq, kp, c, K, lane, first_cell, ncells_valid, warp, wpart, dpart, mpart); break;
        case 4: sweep_two<NCH, 4, kAux>(eq, ep, fq, kp, c, K, lane, first_cell, ncells_valid, warp, wpart, dpart, mpart); break;
        case 8: sweep_two<NCH, 8, kAux>(eq, ep, fq, kp, c, K, lane, first_cell, ncells_valid, warp, wpart, dpart, mpart); break;
        default: sweep_two<NCH, 0, kAux>(eq, ep, fq, kp, c, K, lane, first_cell, ncells_valid, warp, wpart, dpart, mpart); break;
    }
}

template <typename T, int NCH>
__global__ void __launch_bounds__(kFThreads, 1) fused_chain_kernel(const FusedParams p) {
    extern __shared__ __align__(1024) unsigned char smem[];
    const Shape &s = p.s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int C = p.cluster;
    const int rank = (int)cluster_ctarank();
    const int cid = blockIdx.x / C;
    const int G = gridDim.x / C;
    const int S = p.stages;
    constexpr int kStageBytes = 2 * kChunk * (int)sizeof(T);
    Control *ctl = reinterpret_cast<Control *>(smem + (size_t)S * kStageBytes);

    // this CTA's slice of the vocabulary
    const int x_begin = rank * p.slice_len;
    const int cta_len = max(0, min(s.V, x_begin + p.slice_len) - x_begin);
    const int ncells_valid = (cta_len + kCell - 1) / kCell;
    const int first_cell = x_begin / kCell;

    if (tid == 0) {
        for (int i = 0; i < S; ++i) {
            mbar_init(&ctl->full[i], 1);
            mbar_init(&ctl->empty[i], kFWarps);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    cluster_sync_all();  // every CTA of the cluster is running before any remote shared-memory access

    const int my_chains = (p.nchains - cid + G - 1) / G;
    const int loads_per_chain = s.gamma * NCH;
    const int total_loads = my_chains * loads_per_chain;
    bool timed_out = false;

    // Producer (thread 0): loads are issued in consumption order; (p_cl, p_i, p_j, p_st) describe the
    // next one: chain number within this cluster's list, position, chunk, ring stage.
    int p_cl = 0, p_i = 0, p_j = 0, p_st = 0, p_issued = 0;
    auto issue_next = [&]() {
        const size_t bk = (size_t)cid + (size_t)p_cl * G;
        const T *zq = reinterpret_cast<const T *>(p.zq) + (bk * (s.gamma + 1) + p_i) * s.V + x_begin + p_j * kChunk;
        const T *zp = reinterpret_cast<const T *>(p.zp) + (bk * s.gamma + p_i) * s.V + x_begin + p_j * kChunk;
        const int nvalid = max(0, min(kChunk, cta_len - p_j * kChunk));
        const uint32_t bytes = (uint32_t)nvalid * (uint32_t)sizeof(T);
        mbar_expect_tx(&ctl->full[p_st], 2 * bytes);
        if (bytes) {
            unsigned char *dst = smem + (size_t)p_st * kStageBytes;
            bulk_load(dst, zq, bytes, &ctl->full[p_st]);
            bulk_load(dst + kChunk * sizeof(T), zp, bytes, &ctl->full[p_st]);
        }
        ++p_issued;
        if (++p_st == S) p_st = 0;
        if (++p_j == NCH) {
            p_j = 0;
            if (++p_i == s.gamma) {
                p_i = 0;
                ++p_cl;
            }
        }
    };
    if (tid == 0) {
        const int first = total_loads < S ? total_loads : S;
        for (int k = 0; k < first; ++k) issue_next();
    }

    // consumption state (same in every thread): ring stage and phase parity of the next chunk, and of
    // the chunk consumed one step earlier (the one whose stage the producer refills)
    int st = 0, prev_st = 0, consumed = 0, rowcount = 0;
    uint32_t ph = 0, prev_ph = 0;
    for (int cl = 0; cl < my_chains; ++cl) {
        const size_t bk = (size_t)cid + (size_t)cl * G;
        const int brow = (int)(bk / s.K);
        if (tid < s.gamma) {
            int t = p.tok[bk * s.gamma + tid];
            if (t < 0 || t >= s.V) {
                if (rank == 0) atomicOr(p.ws.status + brow, SGBV_STATUS_TOKEN_RANGE);
                t = 0;
            }
            ctl->tok[tid] = t;
        }
        __syncthreads();
        double la = 0.0, lb = 0.0;  // log a_i, log b_i (meaningful in warp 0)

        for (int i = 0; i < s.gamma; ++i) {
            const size_t r = bk * s.gamma + i;
            const T *zq_row = reinterpret_cast<const T *>(p.zq) + (bk * (s.gamma + 1) + i) * s.V;
            const T *zp_row = reinterpret_cast<const T *>(p.zp) + (bk * s.gamma + i) * s.V;
            // token logits for the chain scalars: fetched now, used after the first sweep
            float zq_tok = 0.0f, zp_tok = 0.0f;
            if (warp == 0 && lane == 0) {
                const int t = ctl->tok[i];
                zq_tok = ld_logit(zq_row, t);
                zp_tok = ld_logit(zp_row, t);
            }

            // ---- first sweep, part 1: ring -> registers, running max -------------------------------
            float eq[NCH][8], ep[NCH][8];
            float mq = -INFINITY, mp = -INFINITY;
#pragma unroll
            for (int j = 0; j < NCH; ++j) {
                if (tid == 0 && consumed >= kLag && p_issued < total_loads) {
                    // refill the stage of the previous chunk once every warp has released it
                    if (!mbar_wait(&ctl->empty[prev_st], prev_ph)) timed_out = true;
                    issue_next();
                }
                if (!mbar_wait(&ctl->full[st], ph)) timed_out = true;
                const unsigned char *base = smem + (size_t)st * kStageBytes;
                const int cell = j * kFWarps + warp;
                if (cell < ncells_valid) {
                    read_cell<T>(base, warp, lane, eq[j]);
                    read_cell<T>(base + kChunk * sizeof(T), warp, lane, ep[j]);
                    const int cell_x = x_begin + cell * kCell;
                    if (cell_x + kCell > s.V) {  // the row ends inside this cell
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            if (cell_x + cell_offset<T>(lane, e) >= s.V) eq[j][e] = ep[j][e] = -INFINITY;
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < 8; ++e) eq[j][e] = ep[j][e] = -INFINITY;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctl->empty[st]);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    mq = fmaxf(mq, eq[j][e]);
                    mp = fmaxf(mp, ep[j][e]);
                }
                prev_st = st;
                prev_ph = ph;
                if (++st == S) {
                    st = 0;
                    ph ^= 1u;
                }
                ++consumed;
            }
            mq = warp_max(mq);
            mp = warp_max(mp);
            if (lane == 0) {
                ctl->red[0][warp] = mq;
                ctl->red[1][warp] = mp;
            }
            __syncthreads();
            mq = ctl->red[0][0];
            mp = ctl->red[1][0];
#pragma unroll
            for (int w = 1; w < kFWarps; ++w) {
                mq = fmaxf(mq, ctl->red[0][w]);
                mp = fmaxf(mp, ctl->red[1][w]);
            }
            // reference points for the exponentials: the CTA maxima (0 if the slice is all -inf)
            const float rq = (mq > -INFINITY) ? mq : 0.0f;
            const float rp = (mp > -INFINITY) ? mp : 0.0f;

            // ---- first sweep, part 2: exponentials in place, sums ----------------------------------
            float sq = 0.0f, sp = 0.0f;
#pragma unroll
            for (int j = 0; j < NCH; ++j) {
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    eq[j][e] = ex2((eq[j][e] - rq) * s.scale);
                    ep[j][e] = ex2((ep[j][e] - rp) * s.scale);
                    sq += eq[j][e];
                    sp += ep[j][e];
                }
            }
            sq = warp_sum(sq);
            sp = warp_sum(sp);
            if (lane == 0) {
                ctl->red[2][warp] = sq;
                ctl->red[3][warp] = sp;
            }
            __syncthreads();
            if (tid == 0) {
                float a = 0.0f, b = 0.0f;
#pragma unroll
                for (int w = 0; w < kFWarps; ++w) {
                    a += ctl->red[2][w];
                    b += ctl->red[3][w];
                }
                ctl->slot[rowcount & 1] = make_float4(mq, a, mp, b);
            }
            cluster_sync_all();

            // ---- chain scalars (warp 0 of every CTA, identical arithmetic) ---------------------------
            if (warp == 0) {
                float4 v = make_float4(-INFINITY, 0.0f, -INFINITY, 0.0f);
                if (lane < C) v = ld_dsmem_f4(&ctl->slot[rowcount & 1], (uint32_t)lane);
                const float mq_row = warp_max(v.x), mp_row = warp_max(v.z);
                double zq_part = 0.0, zp_part = 0.0;
                if (lane < C) {
                    if (v.x > -INFINITY) zq_part = (double)v.y * exp2((double)(v.x - mq_row) * (double)s.scale);
                    if (v.z > -INFINITY) zp_part = (double)v.w * exp2((double)(v.z - mp_row) * (double)s.scale);
                }
                const double Zq = warp_sum(zq_part), Zp = warp_sum(zp_part);
                if (lane == 0) {
                    const double c = exp(lb - la);
                    const double kappa = c * Zq / Zp;
                    // nonfinite logits: NaN poisons Z, +inf shows up as an infinite maximum, a row of
                    // -inf only has Z = 0
                    const bool bad = !(Zq > 0.0) || !(Zp > 0.0) || !(Zq < INFINITY) || !(Zp < INFINITY) ||
                                     !(mq_row < INFINITY) || !(mp_row < INFINITY);
                    if (rank == 0) {
                        if (bad) atomicOr(p.ws.status + brow, SGBV_STATUS_NONFINITE_LOGIT);
                        RowInfo ri;
                        ri.log_a = la;
                        ri.log_b = lb;
                        ri.Zq = Zq;
                        ri.Zp = Zp;
                        ri.mq = mq_row;
                        ri.mp = mp_row;
                        ri.kappa = (float)kappa;
                        ri.c = (float)c;
                        p.ws.rows[r] = ri;
                    }
                    const float fq = ex2((rq - mq_row) * s.scale);   // CTA units -> row units
                    const float fp = ex2((rp - mp_row) * s.scale);
                    ctl->bc[0] = fq;
                    ctl->bc[1] = (float)kappa * fp;
                    ctl->bc[2] = (float)c;
                    la += ((double)zq_tok - (double)mq_row) * s.inv_T - log(Zq);
                    lb += ((double)zp_tok - (double)mp_row) * s.inv_T - log(Zp);
                    if (i == s.gamma - 1 && rank == 0) {
                        p.ws.chain_end[2 * bk + 0] = la;
                        p.ws.chain_end[2 * bk + 1] = lb;
                    }
                }
            }
            __syncthreads();
            const float fq = ctl->bc[0], kp = ctl->bc[1], c = ctl->bc[2];

            // ---- second sweep from registers ---------------------------------------------------------
            float *wp = p.ws.wpart + r * s.ntiles, *dp = p.ws.dpart + r * s.ntiles, *mpp = p.ws.mpart + r * s.ntiles;
            if (c < 1.0f)
                sweep_two_dispatch<NCH, true>(eq, ep, fq, kp, c, s.K, lane, first_cell, ncells_valid, warp, wp, dp, mpp);
            else
                sweep_two_dispatch<NCH, false>(eq, ep, fq, kp, c, s.K, lane, first_cell, ncells_valid, warp, wp, dp, mpp);
            ++rowcount;
        }
        __syncthreads();  // ctl->tok is rewritten for the next chain
    }
    if (timed_out) atomicExch(p.error_flag, 1);
    cluster_sync_all();  // no CTA leaves while a neighbour may still read its slots
}

// ---- host side ----------------------------------------------------------------------------------------
struct Plan {
    int cluster, slice_len, nch, stages, grid_clusters;
    size_t smem;
};

int g_opt_cluster = 0;     // 0 = automatic
int g_opt_stages = 0;
int g_opt_max_clusters = 0;

template <typename T, int NCH>
int launch_nch(const Launch &L, const Plan &plan, int *error_flag) {
    auto kernel = fused_chain_kernel<T, NCH>;
    static bool attr_done[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SGBV_ERR_CUDA;
    if (!attr_done[dev]) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
            return SGBV_ERR_CUDA;
        attr_done[dev] = true;
    }
    FusedParams fp;
    fp.zq = L.zq;
    fp.zp = L.zp;
    fp.tok = L.tok;
    fp.s = L.s;
    fp.ws = L.ws;
    fp.cluster = plan.cluster;
    fp.slice_len = plan.slice_len;
    fp.stages = plan.stages;
    fp.nchains = L.s.B * L.s.K;
    fp.error_flag = error_flag;

    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kFThreads);
    cfg.dynamicSmemBytes = plan.smem;
    cfg.stream = L.stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = plan.cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;

    int clusters = plan.grid_clusters;
    if (clusters <= 0) {
        // persistent grid: as many clusters as can be co-resident (queried once per configuration)
        static int cached[9][9];  // [cluster size][stages]
        int &slot = cached[plan.cluster][plan.stages];
        if (slot == 0) {
            cfg.gridDim = dim3(plan.cluster * 148);
            int nmax = 0;
            if (cudaOccupancyMaxActiveClusters(&nmax, kernel, &cfg) != cudaSuccess || nmax < 1) {
                cudaGetLastError();
                nmax = 148 / plan.cluster;
            }
            slot = nmax;
        }
        clusters = slot;
    }
    if (clusters > fp.nchains) clusters = fp.nchains;
    cfg.gridDim = dim3(clusters * plan.cluster);
    if (L.ev_begin) cudaEventRecord(L.ev_begin, L.stream);
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, fp);
    if (L.ev_end) cudaEventRecord(L.ev_end, L.stream);
    return e == cudaSuccess ? 1 : SGBV_ERR_CUDA;
}

template <typename T>
int launch_t(const Launch &L, const Plan &plan, int *error_flag) {
    switch (plan.nch) {
        case 1: return launch_nch<T, 1>(L, plan, error_flag);
        case 2: return launch_nch<T, 2>(L, plan, error_flag);
        case 3: return launch_nch<T, 3>(L, plan, error_flag);
        case 4: return launch_nch<T, 4>(L, plan, error_flag);
        case 5: return launch_nch<T, 5>(L, plan, error_flag);
        default: return SGBV_ERR_SHAPE;
    }
}

}  // namespace

void fused_set_options(int cluster, int stages, int max_clusters) {
    g_opt_cluster = cluster;
    g_opt_stages = stages;
    g_opt_max_clusters = max_clusters;
}

// Whether the fused path can take this call: rows must be 16-byte aligned for the bulk copies and
// a CTA's slice must fit its registers (at most 5 chunks of 4096 elements, clusters of at most 8).
bool fused_supported(const Launch &L) {
    const size_t esz = L.dtype == SGBV_DTYPE_BF16 ? 2 : 4;
    if (((uintptr_t)L.zq % 16) || ((uintptr_t)L.zp % 16) || (((size_t)L.s.V * esz) % 16)) return false;
    const int cells = (L.s.V + kCell - 1) / kCell;
    return (cells + 7) / 8 * kCell <= 5 * kChunk;
}

int launch_fused(const Launch &L, int *error_flag) {
    const Shape &s = L.s;
    const size_t esz = L.dtype == SGBV_DTYPE_BF16 ? 2 : 4;
    const int cells = (s.V + kCell - 1) / kCell;
    const int nchains = s.B * s.K;
    Plan plan;
    int C = g_opt_cluster;
    if (C == 0) {
        C = 1;
        while ((cells + C - 1) / C * kCell > 5 * kChunk) C *= 2;  // smallest cluster whose slices fit
        while (C < 8 && (long)nchains * C < 148 && cells / (2 * C) >= 4) C *= 2;  // few chains: spread each wider
    }
    if (C < 1 || C > 8 || (cells + C - 1) / C * kCell > 5 * kChunk) return SGBV_ERR_SHAPE;
    plan.cluster = C;
    plan.slice_len = (cells + C - 1) / C * kCell;
    plan.nch = (plan.slice_len + kChunk - 1) / kChunk;
    const size_t stage_bytes = 2 * kChunk * esz;
    int S = g_opt_stages ? g_opt_stages : 8;
    const size_t budget = 227 * 1024 - sizeof(Control) - 1024;
    if ((size_t)S * stage_bytes > budget) S = (int)(budget / stage_bytes);
    if (S > 8) S = 8;
    if (S < 2) return SGBV_ERR_SHAPE;
    plan.stages = S;
    plan.smem = (size_t)S * stage_bytes + sizeof(Control);
    plan.grid_clusters = g_opt_max_clusters;
    return L.dtype == SGBV_DTYPE_BF16 ? launch_t<uint16_t>(L, plan, error_flag) : launch_t<float>(L, plan, error_flag);
}

}  // namespace sgbv
