// Fused single-read path (steps A1-A3): one thread-block cluster walks one draft chain (b,k).
//
// For every position i = 0..gamma-1 of the chain the cluster
//   * streams the target row and the draft row from HBM exactly once: one elected thread issues
//     bulk asynchronous copies (cp.async.bulk + mbarrier transaction counts) of 2048-element chunks
//     into a shared-memory ring that runs ahead across rows and chains;
//   * keeps the whole row pair resident in REGISTERS (each CTA of the cluster owns a contiguous
//     slice of the vocabulary, each thread 8 elements of every chunk) as exponentials relative to
//     the thread's own maximum, so the second sweep of the coupling sum never re-reads memory;
//   * exchanges per-warp (max, sum-exp) partials by PUSHING them into every CTA's shared memory
//     (distributed shared memory stores) followed by one cluster barrier per row; after the barrier
//     every warp combines the partials locally and identically, so there is no second block-wide
//     synchronisation and no remote load on the critical path;
//   * runs the second sweep from registers and writes one partial sum per 256-element cell
//     (a cell is what one warp owns in one chunk: 256 contiguous vocabulary entries).
// The joint likelihood ratio c_i = p(x^i)/q(x^i) is carried as a running product by one thread,
// which computes c_{i+1} while the other warps are already in the second sweep of row i.
// Two CTAs of 256 threads share an SM (different clusters), so one CTA's exchange latency is
// covered by the other's arithmetic.  The finishing kernel (weights, scan, extra token) consumes
// the cell sums.
//
// Every wait on an mbarrier is bounded; on expiry the CTA records an error flag and keeps
// executing the protocol (all cluster barriers are still reached), so a lost copy cannot hang.
#include "sgbv_common.cuh"

namespace sgbv {

namespace {

constexpr int kFThreads = 256;
constexpr int kFWarps = kFThreads / 32;
constexpr int kCell = kTile;               // 256 contiguous elements: one warp's share of a chunk
constexpr int kChunk = kFWarps * kCell;    // 2048 elements per chunk per tensor
constexpr int kMaxNch = 5;                 // chunks of a row slice one CTA can hold in registers
constexpr int kMaxStages = 12;
constexpr int kMaxCluster = 16;
constexpr long long kWaitLimitCycles = 2000000000ll;  // about one second of SM clock
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
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: returns false if the phase did not complete within about a second.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity) {
    if (mbar_test(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_test(bar, parity))
        if (clock64() - t0 > kWaitLimitCycles) return false;
    return true;
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
__device__ __forceinline__ void cluster_arrive() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait() {
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Store 16 bytes into the shared memory of CTA `rank` of this cluster, at the address that
// `local` has in this CTA.
__device__ __forceinline__ void st_dsmem_f4(void *local, uint32_t rank, float4 v) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(local)), "r"(rank));
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(remote), "f"(v.x), "f"(v.y), "f"(v.z),
                 "f"(v.w)
                 : "memory");
}
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float rcp(float x) {
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// ---- shared memory layout ------------------------------------------------------------------------
struct Control {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    // per-warp partials (mq, sum eq, mp, sum ep) of every CTA of the cluster, pushed by their
    // owners; double-buffered by row parity
    float4 slots[2][kMaxCluster * kFWarps];
    double c[2];           // joint likelihood ratio c_i of the current chain, by row parity
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

// r^K for r in [0,1]; KT > 0 is a compile-time K.
template <int KT>
__device__ __forceinline__ float ipow(float r, int K) {
    if (KT == 1) return 1.0f;  // callers multiply by the base themselves where K = 1 matters
    if (KT > 1) {
        float acc = (KT & 1) ? r : 1.0f, sq = r;
#pragma unroll
        for (int k = KT >> 1; k > 0; k >>= 1) {
            sq *= sq;
            if (k & 1) acc *= sq;
        }
        return acc;
    }
    float acc = 1.0f;
    for (int t = 0; t < K; ++t) acc *= r;
    return acc;
}

// Second sweep over the register-resident row.  eq/ep are exponentials relative to the THREAD's
// maxima; kt = kappa * (fp_t / fq_t) makes  c p(x)/q(x) = kt * ep/eq;  scale_w, scale_d convert the
// thread's sums to row-max units.  Per cell:
//   wpart = sum eq (1 - min{kt ep/eq, 1})^K                    (Eq. 4's weights, Eq. 2's sum)
//   dpart = sum max(kt ep - eq, 0)                             (c < 1 only)
//   mpart = sum eq (c - t)^2 Q(t)                              (c < 1 only)
template <int NCH, int KT, bool kAux>
__device__ __forceinline__ void sweep_two(const float (&eq)[NCH][8], const float (&ep)[NCH][8], float kt,
                                          float scale_w, float scale_d, float c, int K, int lane, int warp,
                                          int ncells_valid, float *wpart, float *dpart, float *mpart) {
    const float v1 = 1.0f - c;
#pragma unroll
    for (int j = 0; j < NCH; ++j) {
        const int cell = j * kFWarps + warp;  // cell index inside this CTA's slice (warp-uniform)
        if (cell >= ncells_valid) break;
        float sw = 0.0f, sd = 0.0f, sm = 0.0f;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const float q = eq[j][e];
            const float diff = fmaf(-kt, ep[j][e], q);      // q - c p, thread units
            if (KT == 1 && !kAux) {
                sw += fmaxf(diff, 0.0f);
                continue;
            }
            // r = 1 - min{c p/q, 1}; q = 0 gives -inf or NaN before the clamp, 0 after it
            const float r = fmaxf(diff * rcp(q), 0.0f);
            if (KT == 1) sw += fmaxf(diff, 0.0f);
            else sw = fmaf(q, ipow<KT>(r, K), sw);
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
                const float ct = r - v1;  // c - t with t = 1 - r
                sm = fmaf(q * ct * ct, acc, sm);
            }
        }
        sw = warp_sum(sw * scale_w);
        if (kAux) {
            sd = warp_sum(sd * scale_d);
            sm = warp_sum(sm * scale_w);
        }
        if (lane == 0) {
            wpart[cell] = sw;
            if (kAux) {
                dpart[cell] = sd;
                mpart[cell] = sm;
            }
        }
    }
}

template <int NCH, bool kAux>
__device__ __forceinline__ void sweep_two_dispatch(const float (&eq)[NCH][8], const float (&ep)[NCH][8], float kt,
                                                   float scale_w, float scale_d, float c, int K, int lane, int warp,
                                                   int ncells_valid, float *wpart, float *dpart, float *mpart) {
#define SGBV_SWEEP(KT) \
    sweep_two<NCH, KT, kAux>(eq, ep, kt, scale_w, scale_d, c, K, lane, warp, ncells_valid, wpart, dpart, mpart)
    switch (K) {
        case 1: SGBV_SWEEP(1); break;
        case 2: SGBV_SWEEP(2); break;
        case 3: SGBV_SWEEP(3); break;
        case 4: SGBV_SWEEP(4); break;
        case 8: SGBV_SWEEP(8); break;
        default: SGBV_SWEEP(0); break;
    }
#undef SGBV_SWEEP
}

template <typename T, int NCH>
__global__ void __launch_bounds__(kFThreads, 2) fused_chain_kernel(const FusedParams p) {
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
    cluster_arrive();  // every CTA of the cluster is running before any remote shared-memory access
    cluster_wait();

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
        if (tid == 0) ctl->c[rowcount & 1] = 1.0;  // c_0 = 1 (empty prefix)
        __syncthreads();

        for (int i = 0; i < s.gamma; ++i) {
            const size_t r = bk * s.gamma + i;
            const int par = rowcount & 1;
            // token logits for the chain ratio: fetched now, used after the exchange
            float zq_tok = 0.0f, zp_tok = 0.0f;
            if (tid == 0) {
                const int t = ctl->tok[i];
                zq_tok = ld_logit(reinterpret_cast<const T *>(p.zq) + (bk * (s.gamma + 1) + i) * s.V, t);
                zp_tok = ld_logit(reinterpret_cast<const T *>(p.zp) + (bk * s.gamma + i) * s.V, t);
            }

            // ---- first sweep, part 1: ring -> registers, running maxima of this thread ---------------
            float eq[NCH][8], ep[NCH][8];
            float mq = -INFINITY, mp = -INFINITY;
#pragma unroll
            for (int j = 0; j < NCH; ++j) {
                if (tid == 0 && consumed >= 1 && p_issued < total_loads) {
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
            // reference points of the exponentials: the thread's own maxima (0 if it saw only -inf)
            const bool has_q = mq > -INFINITY, has_p = mp > -INFINITY;
            const float rq = has_q ? mq : 0.0f;
            const float rp = has_p ? mp : 0.0f;

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
            // warp partials in warp-max units, pushed to every CTA of the cluster
            const float mqw = warp_max(mq), mpw = warp_max(mp);
            const float rqw = (mqw > -INFINITY) ? mqw : 0.0f, rpw = (mpw > -INFINITY) ? mpw : 0.0f;
            sq = warp_sum(has_q ? sq * ex2((rq - rqw) * s.scale) : 0.0f);
            sp = warp_sum(has_p ? sp * ex2((rp - rpw) * s.scale) : 0.0f);
            if (lane < C) st_dsmem_f4(&ctl->slots[par][rank * kFWarps + warp], (uint32_t)lane, make_float4(mqw, sq, mpw, sp));
            cluster_arrive();
            cluster_wait();

            // ---- row statistics: every warp combines all partials, in the same order ------------------
            float mq_row = -INFINITY, mp_row = -INFINITY;
            const int nslots = C * kFWarps;
            for (int e = lane; e < nslots; e += 32) {
                const float4 v = ctl->slots[par][e];
                mq_row = fmaxf(mq_row, v.x);
                mp_row = fmaxf(mp_row, v.z);
            }
            mq_row = warp_max(mq_row);
            mp_row = warp_max(mp_row);
            const float rq_row = (mq_row > -INFINITY) ? mq_row : 0.0f, rp_row = (mp_row > -INFINITY) ? mp_row : 0.0f;
            double Zq = 0.0, Zp = 0.0;
            for (int e = lane; e < nslots; e += 32) {
                const float4 v = ctl->slots[par][e];
                if (v.x > -INFINITY) Zq += (double)(v.y * ex2((v.x - rq_row) * s.scale));
                if (v.z > -INFINITY) Zp += (double)(v.w * ex2((v.z - rp_row) * s.scale));
            }
            Zq = warp_sum(Zq);
            Zp = warp_sum(Zp);
            const double cd = ctl->c[par];
            const double kappa_d = cd * Zq / Zp;
            const float c = (float)cd;

            if (tid == 0) {
                // nonfinite logits: NaN poisons Z, +inf shows up as an infinite maximum, a row of
                // -inf only has Z = 0
                const bool bad = !(Zq > 0.0) || !(Zp > 0.0) || !(Zq < INFINITY) || !(Zp < INFINITY) ||
                                 !(mq_row < INFINITY) || !(mp_row < INFINITY);
                if (rank == 0) {
                    if (bad) atomicOr(p.ws.status + brow, SGBV_STATUS_NONFINITE_LOGIT);
                    RowInfo ri;
                    ri.Zq = Zq;
                    ri.Zp = Zp;
                    ri.mq = mq_row;
                    ri.mp = mp_row;
                    ri.kappa = (float)kappa_d;
                    ri.c = c;
                    p.ws.rows[r] = ri;
                }
                // c_{i+1} = c_i p_i(tok_i)/q_i(tok_i), for the next row of this chain
                const double lp = ((double)zp_tok - (double)mp_row) * s.inv_T;
                const double lq = ((double)zq_tok - (double)mq_row) * s.inv_T;
                ctl->c[par ^ 1] = cd * exp(lp - lq) * (Zq / Zp);
            }

            // thread units -> row units
            const float fq = has_q ? ex2((rq - rq_row) * s.scale) : 0.0f;
            const float fp = has_p ? ex2((rp - rp_row) * s.scale) : 0.0f;
            float kt = (float)kappa_d * fp / fq;
            float scale_w = fq, scale_d = fq;
            if (__any_sync(0xffffffffu, !(fq > 1e-30f))) {
                // a thread whose share of the target row underflows (or nearly so, which would
                // overflow kt): its q is 0 in row units, its weights vanish, and max(c p - q, 0) = c p
                if (!(fq > 1e-30f)) {
#pragma unroll
                    for (int j = 0; j < NCH; ++j)
#pragma unroll
                        for (int e = 0; e < 8; ++e) eq[j][e] = 0.0f;
                    kt = 1.0f;
                    scale_w = 0.0f;
                    scale_d = (float)kappa_d * fp;
                }
            }

            // ---- second sweep from registers ---------------------------------------------------------
            float *wp = p.ws.wpart + r * s.ntiles + first_cell, *dp = p.ws.dpart + r * s.ntiles + first_cell,
                  *mpp = p.ws.mpart + r * s.ntiles + first_cell;
            if (c < 1.0f)
                sweep_two_dispatch<NCH, true>(eq, ep, kt, scale_w, scale_d, c, s.K, lane, warp, ncells_valid, wp, dp, mpp);
            else
                sweep_two_dispatch<NCH, false>(eq, ep, kt, scale_w, scale_d, c, s.K, lane, warp, ncells_valid, wp, dp, mpp);
            ++rowcount;
        }
        __syncthreads();  // ctl->tok and ctl->c are rewritten for the next chain
    }
    if (timed_out) atomicExch(p.error_flag, 1);
    cluster_arrive();  // no CTA leaves while a neighbour may still write into its slots
    cluster_wait();
}

// ---- host side ----------------------------------------------------------------------------------------
struct Plan {
    int cluster, slice_len, nch, stages, grid_clusters;
    size_t smem;
};

int g_opt_cluster = 0;     // 0 = automatic
int g_opt_stages = 0;
int g_opt_max_clusters = 0;

constexpr int kSmemPerSm = 228 * 1024;     // shared memory of one SM
constexpr int kSmemReserved = 1024;        // per resident CTA, taken by the system
constexpr int kCtaSlots = 2 * 148;         // resident CTAs of this kernel on the whole device

int cells_of(int V) { return (V + kCell - 1) / kCell; }
int slice_cells(int cells, int C) { return (cells + C - 1) / C; }

template <typename T, int NCH>
int launch_nch(const Launch &L, const Plan &plan, int *error_flag) {
    auto kernel = fused_chain_kernel<T, NCH>;
    static bool attr_done[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SGBV_ERR_CUDA;
    if (!attr_done[dev]) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kSmemPerSm / 2 - kSmemReserved) != cudaSuccess)
            return SGBV_ERR_CUDA;
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess)
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
        static int cached[64][kMaxCluster + 1][kMaxStages + 1];  // [device][cluster size][stages]
        int &slot = cached[dev][plan.cluster][plan.stages];
        if (slot == 0) {
            cfg.gridDim = dim3(plan.cluster * (kCtaSlots / plan.cluster));
            int nmax = 0;
            if (cudaOccupancyMaxActiveClusters(&nmax, kernel, &cfg) != cudaSuccess || nmax < 1) {
                cudaGetLastError();
                return 0;  // this cluster shape cannot be scheduled here: nothing launched
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
    if (e != cudaSuccess) {
        cudaGetLastError();
        return SGBV_ERR_CUDA;
    }
    return 1;
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
// a CTA's slice must fit its registers (at most 5 chunks of 2048 elements, clusters of at most 16).
bool fused_supported(const Launch &L) {
    const size_t esz = L.dtype == SGBV_DTYPE_BF16 ? 2 : 4;
    if (((uintptr_t)L.zq % 16) || ((uintptr_t)L.zp % 16) || (((size_t)L.s.V * esz) % 16)) return false;
    return slice_cells(cells_of(L.s.V), kMaxCluster) * kCell <= kMaxNch * kChunk;
}

int launch_fused(const Launch &L, int *error_flag) {
    const Shape &s = L.s;
    const size_t esz = L.dtype == SGBV_DTYPE_BF16 ? 2 : 4;
    const int cells = cells_of(s.V);
    const long nchains = (long)s.B * s.K;
    Plan plan;
    int C = g_opt_cluster;
    if (C == 0) {
        C = 1;
        while (slice_cells(cells, C) * kCell > kMaxNch * kChunk) C *= 2;  // smallest cluster whose slices fit
        // few chains: spread each over more CTAs while they all stay co-resident in one wave
        while (C < kMaxCluster && nchains * 2 * C <= kCtaSlots && cells / (2 * C) >= 4) C *= 2;
    }
    if (C < 1 || C > kMaxCluster || slice_cells(cells, C) * kCell > kMaxNch * kChunk) return SGBV_ERR_SHAPE;
    plan.cluster = C;
    plan.slice_len = slice_cells(cells, C) * kCell;
    plan.nch = (plan.slice_len + kChunk - 1) / kChunk;
    const size_t stage_bytes = 2 * kChunk * esz;
    int S = g_opt_stages ? g_opt_stages : kMaxStages;
    const size_t budget = kSmemPerSm / 2 - kSmemReserved - sizeof(Control);
    if ((size_t)S * stage_bytes > budget) S = (int)(budget / stage_bytes);
    if (S > kMaxStages) S = kMaxStages;
    if (S < 2) return SGBV_ERR_SHAPE;
    plan.stages = S;
    plan.smem = (size_t)S * stage_bytes + sizeof(Control);
    plan.grid_clusters = g_opt_max_clusters;
    return L.dtype == SGBV_DTYPE_BF16 ? launch_t<uint16_t>(L, plan, error_flag) : launch_t<float>(L, plan, error_flag);
}

}  // namespace sgbv
