// Fused single-read path (steps A1-A3): one thread-block cluster walks one draft chain (b,k).
//
// For every position i = 0..gamma-1 of the chain the cluster
//   * streams the target row and the draft row from HBM exactly once: bulk asynchronous copies
//     (cp.async.bulk + mbarrier transaction counts) of 2048-element chunks of both tensors into a
//     shared-memory ring that runs ahead across rows and chains.  A warp owns the 256-element
//     cells  warp, warp+8, warp+16, ...  of its CTA's slice.  There is no producer thread and no
//     "stage free" barrier: once the row's exchange (below) is complete, every warp of the CTA has
//     moved the row into registers, so its ring stages are refilled right then, by a different warp
//     for each chunk; the copies stay large (few requests to the copy engine);
//   * keeps the whole row pair resident in REGISTERS (each thread 8 elements of every cell) as
//     exponentials relative to the thread's own maximum, so the second
//     sweep of the coupling sum never re-reads memory;
//   * exchanges (max, sum-exp) partials in two levels: the warps of a CTA leave theirs in shared
//     memory and the last one to arrive combines them and PUSHES one partial per CTA into every
//     CTA's shared memory with asynchronous distributed-shared-memory stores that complete on the
//     receiver's mbarrier; a warp goes on as soon as all CTA partials of the row have landed.
//     There is no block-wide or cluster-wide barrier inside the row loop;
//   * runs the second sweep from registers and writes one partial sum per cell.
// The joint likelihood ratio c_i = p(x^i)/q(x^i) is carried as a running product by one thread per
// CTA, which computes c_{i+1} right after the statistics of row i and arms the next row's exchange
// with it, a whole row before it is needed.  Two CTAs of 256 threads share an SM (different clusters).  The finishing
// kernel (weights, scan, extra token) consumes the cell sums.
//
// Every wait on an mbarrier is bounded; on expiry the warp records an error flag and keeps
// executing the protocol, so a lost copy cannot hang the kernel.
#include "sgbv_common.cuh"

namespace sgbv {

namespace {

constexpr int kFThreads = 256;
constexpr int kFWarps = kFThreads / 32;
constexpr int kCell = kTile;               // 256 contiguous elements: one warp's share of a chunk
constexpr int kChunk = kFWarps * kCell;    // 2048 elements: one cell of every warp
constexpr int kMaxNch = 5;                 // cells per warp: what one thread can hold in registers (5 x 8 pairs)
constexpr int kMaxStages = 12;             // ring depth
constexpr int kRowBars = 16;               // "row has landed" barriers: more than the rows the ring can hold
constexpr int kMaxCluster = 16;
constexpr long long kWaitLimitCycles = 2000000000ll;  // about one second of SM clock
constexpr uint32_t kSuspendNs = 20000u;               // longest single suspension inside a wait
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
    int row_mode;     // 0: a cluster walks whole chains; 1: a cluster walks single rows (see the kernel)
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
// The same test, but the thread may be suspended for up to about `kSuspendNs` until the phase completes
// (the hardware wakes it when it does), instead of coming back at once.
__device__ __forceinline__ bool mbar_test_suspend(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(kSuspendNs)
        : "memory");
    return ok != 0;
}
// Bounded wait: returns false if the phase did not complete within about a second.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity) {
    if (mbar_test(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_test_suspend(bar, parity))
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
// Asynchronous store of 16 bytes into the shared memory of CTA `rank` of this cluster, at the
// address that `local` has in this CTA; its completion is counted (16 bytes) on the receiver's
// mbarrier that sits where `local_bar` sits here.
__device__ __forceinline__ void push_f4(void *local, uint64_t *local_bar, uint32_t rank, float4 v) {
    uint32_t dst, bar;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(dst) : "r"(smem_u32(local)), "r"(rank));
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(bar) : "r"(smem_u32(local_bar)), "r"(rank));
    asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%0], {%1,%2,%3,%4}, [%5];" ::"r"(dst),
                 "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w), "r"(bar)
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
// [ring: stages x (chunk of zq, chunk of zp)] [Control]
struct Control {
    uint64_t rowbar[kRowBars];           // by row of the walk (mod 16): "all chunks of the row have landed"
    uint64_t xbar[2];                    // by row parity: "all partials of the row (chain walk: and c_i) are here"
    uint64_t cbar[2];                    // by row parity, row walk only: "c_i is here"
    // partials (maximum of zq, sum eq, maximum of zp, sum ep), double-buffered by row parity:
    // of this CTA's warps, and of every CTA of the cluster (pushed by their owners)
    float4 wslots[2][kFWarps];
    int arrivals;                        // partials left in wslots so far, over all rows (never reset)
    float4 slots[2][kMaxCluster];
    double c[2];                         // joint likelihood ratio c_i of the current row, by row parity
};

// Reads this lane's 8 elements of one cell of one tensor from the ring.
template <typename T>
__device__ __forceinline__ void read_cell(const unsigned char *cell_base, int lane, float2 (&v)[4]);
template <>
__device__ __forceinline__ void read_cell<float>(const unsigned char *cell_base, int lane, float2 (&v)[4]) {
    const float4 *p = reinterpret_cast<const float4 *>(cell_base) + lane;
    const float4 a = p[0], b = p[32];
    v[0] = make_float2(a.x, a.y); v[1] = make_float2(a.z, a.w);
    v[2] = make_float2(b.x, b.y); v[3] = make_float2(b.z, b.w);
}
template <>
__device__ __forceinline__ void read_cell<uint16_t>(const unsigned char *cell_base, int lane, float2 (&v)[4]) {
    const uint4 a = reinterpret_cast<const uint4 *>(cell_base)[lane];
    v[0] = make_float2(__uint_as_float(a.x << 16), __uint_as_float(a.x & 0xffff0000u));
    v[1] = make_float2(__uint_as_float(a.y << 16), __uint_as_float(a.y & 0xffff0000u));
    v[2] = make_float2(__uint_as_float(a.z << 16), __uint_as_float(a.z & 0xffff0000u));
    v[3] = make_float2(__uint_as_float(a.w << 16), __uint_as_float(a.w & 0xffff0000u));
}
// Offset (in elements, within the 256-element cell) of this lane's e-th element.
template <typename T>
__device__ __forceinline__ int cell_offset(int lane, int e) {
    if (sizeof(T) == 4) return (e < 4) ? lane * 4 + e : 128 + lane * 4 + (e - 4);
    return lane * 8 + e;
}

// Maximum over the warp in one instruction (NaN inputs are passed over, as fmaxf does).
__device__ __forceinline__ float warp_max_redux(float v) {
    float r;
    asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
    return r;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
__device__ __forceinline__ float2 splat(float x) { return make_float2(x, x); }

// r^K for both halves of r, r in [0,1]; KT > 1 is a compile-time K, KT = 0 takes K at run time.
template <int KT>
__device__ __forceinline__ float2 ipow2(float2 r, int K) {
    if (KT > 1) {
        float2 acc = r, sq = r;  // acc is only read once it has been assigned
        bool have = (KT & 1) != 0;
#pragma unroll
        for (int k = KT >> 1; k > 0; k >>= 1) {
            sq = __fmul2_rn(sq, sq);
            if (k & 1) {
                acc = have ? __fmul2_rn(acc, sq) : sq;
                have = true;
            }
        }
        return acc;
    }
    float2 acc = r;
    for (int t = 1; t < K; ++t) acc = __fmul2_rn(acc, r);
    return acc;
}

// Sums N values over the 32 lanes of a warp at once ("transposed" butterfly: at every step a lane
// hands half of its values to its partner and keeps the other half).  P = N rounded up to a power
// of two (<= 16).  On return v[0] of lane l is the warp total of value number owner_index<P>(l).
template <int P>
__device__ __forceinline__ int owner_index(int lane) {
    int idx = 0;
    if (P >= 2) idx += (lane & 16) ? P / 2 : 0;
    if (P >= 4) idx += (lane & 8) ? P / 4 : 0;
    if (P >= 8) idx += (lane & 4) ? P / 8 : 0;
    if (P >= 16) idx += (lane & 2) ? P / 16 : 0;
    return idx;
}
template <int P>
__device__ __forceinline__ void warp_sum_multi(float (&v)[P], int lane) {
    int off = 16;
#pragma unroll
    for (int n = P; n > 1; n >>= 1, off >>= 1) {
        const bool upper = (lane & off) != 0;
#pragma unroll
        for (int k = 0; k < n / 2; ++k) {
            const float keep = upper ? v[k + n / 2] : v[k];
            const float send = upper ? v[k] : v[k + n / 2];
            v[k] = keep + __shfl_xor_sync(0xffffffffu, send, off);
        }
    }
    for (; off > 0; off >>= 1) v[0] += __shfl_xor_sync(0xffffffffu, v[0], off);
}

// Second sweep over the register-resident row, two vocabulary entries per instruction (f32x2).
// eq/ep are exponentials relative to the THREAD's maxima; kt = kappa * (fp_t / fq_t) makes
// c p(x)/q(x) = kt * ep/eq;  scale_w, scale_d convert the thread's sums to row-max units.
// nj = number of cells this warp holds; the output pointers address this warp's first cell, its
// cells are kFWarps apart.  Per cell:
//   wpart = sum eq (1 - min{kt ep/eq, 1})^K                    (Eq. 4's weights, Eq. 2's sum)
//   dpart = sum max(kt ep - eq, 0)                             (c < 1 only)
//   mpart = sum eq (c - t)^2 Q(t)                              (c < 1 only)
template <int NCH, int KT, bool kAux>
__device__ __forceinline__ void sweep_two(const float2 (&eq)[NCH][4], const float2 (&ep)[NCH][4], float kt,
                                          float scale_w, float scale_d, float c, int K, int lane, int nj,
                                          float *wpart, float *dpart, float *mpart) {
    constexpr int NV = kAux ? 3 * NCH : NCH;
    constexpr int P = NV <= 1 ? 1 : NV <= 2 ? 2 : NV <= 4 ? 4 : NV <= 8 ? 8 : 16;
    static_assert(NV <= 16, "at most 16 sums per thread");
    float sums[P];
#pragma unroll
    for (int k = 0; k < P; ++k) sums[k] = 0.0f;
    const float v1 = 1.0f - c;
    const float2 nkt = splat(-kt), nv1 = splat(-v1);
    // Horner coefficients of Q: (t+1) (1-c)^t, t = 1..K-2 (uniform over the row)
    float2 coef[KT > 2 ? KT - 2 : 1];
    if (kAux && KT > 2) {
        float vj = 1.0f;
#pragma unroll
        for (int t = 1; t <= KT - 2; ++t) {
            vj *= v1;
            coef[t - 1] = splat((float)(t + 1) * vj);
        }
    }
#pragma unroll
    for (int j = 0; j < NCH; ++j) {
        if (j >= nj) break;  // warp-uniform
        float2 sw = splat(0.0f), sd = splat(0.0f), sm = splat(0.0f);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 q = eq[j][e];
            const float2 diff = __ffma2_rn(nkt, ep[j][e], q);  // q - c p, thread units
            const float2 pos = make_float2(fmaxf(diff.x, 0.0f), fmaxf(diff.y, 0.0f));
            if (KT == 1) sw = __fadd2_rn(sw, pos);
            if (KT == 1 && !kAux) continue;
            // r = 1 - min{c p/q, 1}; q = 0 gives -inf or NaN before the clamp, 0 after it
            const float2 t = __fmul2_rn(diff, make_float2(rcp(q.x), rcp(q.y)));
            const float2 r = make_float2(fmaxf(t.x, 0.0f), fmaxf(t.y, 0.0f));
            if (KT != 1) sw = __ffma2_rn(q, ipow2<KT>(r, K), sw);
            if (kAux) {
                sd = __fadd2_rn(sd, make_float2(fmaxf(-diff.x, 0.0f), fmaxf(-diff.y, 0.0f)));
                float2 acc = splat(0.0f);
                if (KT > 0) {
                    if (KT >= 2) {
                        acc = splat(1.0f);
#pragma unroll
                        for (int u = 0; u < KT - 2; ++u) acc = __ffma2_rn(acc, r, coef[u]);
                    }
                } else if (K >= 2) {
                    acc = splat(1.0f);
                    float vj = 1.0f;
                    for (int u = 1; u <= K - 2; ++u) {
                        vj *= v1;
                        acc = __ffma2_rn(acc, r, splat((float)(u + 1) * vj));
                    }
                }
                const float2 ct = __fadd2_rn(r, nv1);  // c - t with t = 1 - r
                sm = __ffma2_rn(__fmul2_rn(q, __fmul2_rn(ct, ct)), acc, sm);
            }
        }
        sums[j] = (sw.x + sw.y) * scale_w;
        if (kAux) {
            sums[NCH + j] = (sd.x + sd.y) * scale_d;
            sums[2 * NCH + j] = (sm.x + sm.y) * scale_w;
        }
    }
    warp_sum_multi<P>(sums, lane);
    // the lane that owns value number idx (and has the low lane bits clear) stores it
    const int idx = owner_index<P>(lane);
    constexpr int kLowMask = P >= 16 ? 1 : P >= 8 ? 3 : P >= 4 ? 7 : P >= 2 ? 15 : 31;
    if ((lane & kLowMask) == 0 && idx < NV) {
        const int jj = kAux ? idx % NCH : idx, which = kAux ? idx / NCH : 0;
        if (jj < nj) {
            float *dst = which == 0 ? wpart : which == 1 ? dpart : mpart;
            dst[jj * kFWarps] = sums[0];
        }
    }
}

template <int NCH, bool kAux>
__device__ __forceinline__ void sweep_two_dispatch(const float2 (&eq)[NCH][4], const float2 (&ep)[NCH][4], float kt,
                                                   float scale_w, float scale_d, float c, int K, int lane, int nj,
                                                   float *wpart, float *dpart, float *mpart) {
#define SGBV_SWEEP(KT) sweep_two<NCH, KT, kAux>(eq, ep, kt, scale_w, scale_d, c, K, lane, nj, wpart, dpart, mpart)
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

// OCC = CTAs of this kernel that share an SM (2, 3 or 4): more co-resident CTAs hide more of each
// other's exchange and pipeline latency, but leave each thread fewer registers, hence fewer cells.
template <typename T, int NCH, int OCC, bool kRow>
__global__ void __launch_bounds__(kFThreads, OCC) fused_chain_kernel(const FusedParams p) {
    extern __shared__ __align__(1024) unsigned char smem[];
    const Shape &s = p.s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int C = p.cluster;
    const int rank = (int)cluster_ctarank();
    const int cid = blockIdx.x / C;
    const int G = gridDim.x / C;
    const int S = p.stages;
    constexpr int kCellBytes = kCell * (int)sizeof(T);
    constexpr int kChunkBytes = kChunk * (int)sizeof(T);
    constexpr int kStageBytes = 2 * kChunkBytes;  // one chunk of zq, then the same chunk of zp
    unsigned char *ring = smem;
    Control *ctl = reinterpret_cast<Control *>(smem + (size_t)S * kStageBytes);

    // this CTA's slice of the vocabulary, and this warp's cells in it: warp, warp + 8, ...
    const int x_begin = rank * p.slice_len;
    const int cta_len = max(0, min(s.V, x_begin + p.slice_len) - x_begin);
    const int ncells_valid = (cta_len + kCell - 1) / kCell;
    const int nj = ncells_valid > warp ? (ncells_valid - warp + kFWarps - 1) / kFWarps : 0;
    const int nchunks = (ncells_valid + kFWarps - 1) / kFWarps;  // chunks per row of this CTA
    const int first_cell = x_begin / kCell + warp;
    const int x_warp = x_begin + warp * kCell;  // first element of this warp's first cell

    if (tid == 0) {
        // one arrival (with its byte count) per chunk of the row
        for (int i = 0; i < kRowBars; ++i) mbar_init(&ctl->rowbar[i], (uint32_t)max(nchunks, 1));
        mbar_init(&ctl->xbar[0], 1);
        mbar_init(&ctl->xbar[1], 1);
        mbar_init(&ctl->cbar[0], 1);
        mbar_init(&ctl->cbar[1], 1);
        ctl->arrivals = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    cluster_arrive();  // every CTA of the cluster is running before any remote shared-memory access
    cluster_wait();

    // Small batches: this grid is itself launched with programmatic stream serialisation, so all of the above may have run while
    // the kernel ahead of it in the stream was still running (in a sequence of calls that is the previous
    // call's finishing kernel, which reads the scratch that this grid is about to write).  Nothing in global
    // memory has been touched so far; from here on that kernel has completed and its writes are visible.
    if (s.B <= kChainedLaunchMaxB) asm volatile("griddepcontrol.wait;" ::: "memory");
    // The finishing kernel is launched with programmatic stream serialisation: let it be scheduled now
    // (it waits for this grid to complete before it reads anything this grid writes).  Not in row mode:
    // there clusters wait for one another, so no CTA of this grid may find its place on an SM taken by
    // a kernel that in turn waits for this grid.
    if (!kRow) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (blockIdx.x == 0 && tid == 0) *p.error_flag = 0;  // set again only by a wait that expires (about a second later)
    // The walk of this cluster: position n = 0, 1, ... is row (bk, i).
    //   chain mode: chains cid, cid+G, ... each from i = 0 to gamma-1 (c_i is carried along the chain);
    //   row mode:   rows u = cid, cid+G, ... of the list of all rows, u = bk*gamma + i.  Used when there
    //               are few chains: all rows of a chain then run at the same time on different clusters,
    //               and c_i comes from the ratios p_j(tok_j)/q_j(tok_j) that the clusters of rows j < i
    //               publish in global memory.  A row only waits for rows earlier in the list, which are
    //               walked no later by clusters that are all resident, so every wait ends.
    // One step of the walk: bk += step_bk, i += step_i, and on i >= gamma: i -= gamma, bk += wrap_bk.
    constexpr bool row_mode = kRow;
    const int step_bk = row_mode ? G / s.gamma : 0, step_i = row_mode ? G % s.gamma : 1, wrap_bk = row_mode ? 1 : G;
    const long total_rows = (long)p.nchains * s.gamma;
    const int nrows = row_mode ? (int)((total_rows - cid + G - 1) / G)
                               : ((p.nchains - cid + G - 1) / G) * s.gamma;  // rows this cluster walks
    const int total_loads = nrows * nchunks;    // chunk pairs this CTA loads
    const uint32_t xbytes = (uint32_t)(C * sizeof(float4));  // one partial from every CTA of the cluster
    bool timed_out = false;

    // Loads are numbered in consumption order: chunk m of this CTA's walk is chunk m % nchunks of
    // row m / nchunks and lands in ring stage m % S.  issue_chunk is stateless, so any lane can issue
    // any chunk: lanes of one warp issue the chunks of a whole row side by side.  All chunks of walk
    // position `row` complete on the barrier of that row (one wait per row instead of one per chunk).
    auto issue_at = [&](size_t bkc, int pos, int jc, int stage, int row) {
        const int x0 = x_begin + jc * kChunk;  // first element of the chunk
        const T *zq = reinterpret_cast<const T *>(p.zq) + (bkc * (s.gamma + 1) + pos) * s.V + x0;
        const T *zp = reinterpret_cast<const T *>(p.zp) + (bkc * s.gamma + pos) * s.V + x0;
        const uint32_t bytes = (uint32_t)min(kChunk, cta_len - jc * kChunk) * (uint32_t)sizeof(T);
        unsigned char *dst = ring + (size_t)stage * kStageBytes;
        uint64_t *bar = &ctl->rowbar[row & (kRowBars - 1)];
        mbar_expect_tx(bar, 2 * bytes);
        bulk_load(dst, zq, bytes, bar);
        bulk_load(dst + kChunkBytes, zp, bytes, bar);
    };
    auto issue_chunk = [&](int m) {
        const int row = m / nchunks;  // position in the walk
        if (row_mode) {
            const long u = (long)cid + (long)row * G;
            issue_at((size_t)(u / s.gamma), (int)(u % s.gamma), m - row * nchunks, m % S, row);
        } else {
            const int chain = row / s.gamma;
            issue_at((size_t)cid + (size_t)chain * G, row - chain * s.gamma, m - row * nchunks, m % S, row);
        }
    };
    // Fill the ring in two goes: the first row's chunks now, so that they do not share the memory system
    // with later rows' chunks and the first row can start as early as possible; the rest of the ring once
    // the first row has landed (see the load phase of the first row).
    if (warp == 0 && lane < nchunks && lane < total_loads) issue_chunk(lane);

    // The chain thread of this CTA carries c_i and fetches the token logits one row
    // ahead: tok_next is the token of the next row of the walk.
    const bool chain_thread = tid == kFThreads - 32;  // lane 0 of the last warp; thread 0 writes the row records
    int tok_next = 0;
    if (chain_thread && nrows > 0) tok_next = p.tok[row_mode ? (size_t)cid : (size_t)cid * s.gamma];
    if (chain_thread && nrows > 0 && !row_mode) {  // the first row of the walk starts a chain: c_0 = 1
        ctl->c[0] = 1.0;
        mbar_expect_tx(&ctl->xbar[0], xbytes);
    }

    int st = 0;
    int n = 0;  // row number in this cluster's walk
    size_t bk = row_mode ? (size_t)(cid / s.gamma) : (size_t)cid;
    int i = row_mode ? cid % s.gamma : 0;
    {
        for (; n < nrows; ++n) {
            const size_t r = bk * s.gamma + i;
            const int par = n & 1;
            const uint32_t xph = (uint32_t)(n >> 1) & 1u;

            // ---- chain thread: the logits of this row's draft token, and the next row's token -----------
            float zq_tok = 0.0f, zp_tok = 0.0f;  // logits of this row's draft token
            if (chain_thread) {
                if (row_mode) mbar_expect_tx(&ctl->xbar[par], xbytes);  // the exchange does not wait for c_i here
                int t = tok_next;
                if (t < 0 || t >= s.V) t = 0;  // the finishing kernel flags the batch row
                zq_tok = ld_logit(reinterpret_cast<const T *>(p.zq) + (bk * (s.gamma + 1) + i) * s.V, t);
                zp_tok = ld_logit(reinterpret_cast<const T *>(p.zp) + (bk * s.gamma + i) * s.V, t);
                if (n + 1 < nrows) {
                    size_t bk_n = bk + step_bk;
                    int i_n = i + step_i;
                    if (i_n >= s.gamma) {
                        i_n -= s.gamma;
                        bk_n += wrap_bk;
                    }
                    tok_next = p.tok[bk_n * s.gamma + i_n];
                }
            }

            // ---- first sweep, part 1: ring -> registers, running maxima of this thread ---------------
            float2 eq[NCH][4], ep[NCH][4];  // two neighbouring vocabulary entries per register pair
            float mq = -INFINITY, mp = -INFINITY;
            if (nchunks > 0 && !mbar_wait(&ctl->rowbar[n & (kRowBars - 1)], (uint32_t)(n / kRowBars) & 1u)) timed_out = true;
            if (n == 0 && warp == 0 && lane >= nchunks && lane < S && lane < total_loads) issue_chunk(lane);  // rest of the ring
            // all loads first, so that their latencies overlap; the maxima afterwards
#pragma unroll
            for (int j = 0; j < NCH; ++j) {
                if (j < nchunks) {  // uniform over the CTA
                    if (j < nj) {  // warp-uniform
                        const unsigned char *base = ring + (size_t)st * kStageBytes + warp * kCellBytes;
                        read_cell<T>(base, lane, eq[j]);
                        read_cell<T>(base + kChunkBytes, lane, ep[j]);
                    }
                    if (++st == S) st = 0;
                }
            }
#pragma unroll
            for (int j = 0; j < NCH; ++j) {
                if (j < nj) {
                    const int cell_x = x_warp + j * kChunk;
                    if (cell_x + kCell > s.V) {  // the row ends inside this cell
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            if (cell_x + cell_offset<T>(lane, 2 * e) >= s.V) eq[j][e].x = ep[j][e].x = -INFINITY;
                            if (cell_x + cell_offset<T>(lane, 2 * e + 1) >= s.V) eq[j][e].y = ep[j][e].y = -INFINITY;
                        }
                    }
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        mq = max3(mq, eq[j][e].x, eq[j][e].y);
                        mp = max3(mp, ep[j][e].x, ep[j][e].y);
                    }
                }
            }
            // reference points of this thread's exponentials: its own maxima (0 if it saw only -inf);
            // the maximum itself maps to exactly 1, so point-mass rows stay exact
            const bool has_q = mq > -INFINITY, has_p = mp > -INFINITY;
            const float bq = has_q ? mq : 0.0f;
            const float bp = has_p ? mp : 0.0f;

            // ---- first sweep, part 2: exponentials in place, sums ----------------------------------
            float2 sq2 = splat(0.0f), sp2 = splat(0.0f);
            const float2 nbq = splat(-bq), nbp = splat(-bp), sc2 = splat(s.scale);
#pragma unroll
            for (int j = 0; j < NCH; ++j) {
                if (j < nj) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 aq = __fmul2_rn(__fadd2_rn(eq[j][e], nbq), sc2);
                        const float2 ap = __fmul2_rn(__fadd2_rn(ep[j][e], nbp), sc2);
                        eq[j][e] = make_float2(ex2(aq.x), ex2(aq.y));
                        ep[j][e] = make_float2(ex2(ap.x), ex2(ap.y));
                        sq2 = __fadd2_rn(sq2, eq[j][e]);
                        sp2 = __fadd2_rn(sp2, ep[j][e]);
                    }
                }
            }
            float sq = sq2.x + sq2.y, sp = sp2.x + sp2.y;
            // warp partials relative to the warp's maxima, pushed to every CTA
            const float bqw = warp_max_redux(has_q ? bq : -INFINITY), bpw = warp_max_redux(has_p ? bp : -INFINITY);
            const float rqw = (bqw > -INFINITY) ? bqw : 0.0f, rpw = (bpw > -INFINITY) ? bpw : 0.0f;
            sq = warp_sum(has_q ? sq * ex2((bq - rqw) * s.scale) : 0.0f);
            sp = warp_sum(has_p ? sp * ex2((bp - rpw) * s.scale) : 0.0f);
            // two-level exchange: the warp partials meet in this CTA's shared memory; the warp that
            // arrives last combines them (fixed order) and pushes ONE partial per CTA to every CTA
            bool last_warp = false;
            if (lane == 0) {
                ctl->wslots[par][warp] = make_float4(bqw, sq, bpw, sp);
                __threadfence_block();
                last_warp = atomicAdd(&ctl->arrivals, 1) + 1 == kFWarps * (n + 1);
            }
            if (__shfl_sync(0xffffffffu, last_warp, 0)) {
                __threadfence_block();
                const float4 v = lane < kFWarps ? ctl->wslots[par][lane] : make_float4(-INFINITY, 0.0f, -INFINITY, 0.0f);
                const float mqc = warp_max_redux(v.x), mpc = warp_max_redux(v.z);
                const float rqc = (mqc > -INFINITY) ? mqc : 0.0f, rpc = (mpc > -INFINITY) ? mpc : 0.0f;
                const float sqc = warp_sum(v.x > -INFINITY ? v.y * ex2((v.x - rqc) * s.scale) : 0.0f);
                const float spc = warp_sum(v.z > -INFINITY ? v.w * ex2((v.z - rpc) * s.scale) : 0.0f);
                if (lane < C)
                    push_f4(&ctl->slots[par][rank], &ctl->xbar[par], (uint32_t)lane, make_float4(mqc, sqc, mpc, spc));
            }

            // Ring refill.  Once all warps of this CTA have left their partials, all of them have turned
            // this row's ring stages into registers, and the stages can take the chunks S ahead.  Warps
            // 1, 2, ... take one chunk each, so the copy requests are issued side by side; a warp that
            // sees the condition already now does it while it would otherwise wait for the exchange,
            // the others do it after the exchange (whose completion implies the condition).
            auto do_refill = [&]() {
                const int jc = (warp + kFWarps - 1) % kFWarps;  // warp 1 -> chunk 0, ..., warp 0 -> chunk 7
                if (lane == 0 && jc < nchunks && n * nchunks + jc + S < total_loads) {
                    // chunk jc of this row sits in stage (st - nchunks + jc) mod S; the chunk that replaces it
                    // is S chunks further along the walk: a few rows on, maybe in the next chain
                    int stage = st - nchunks + jc;
                    while (stage < 0) stage += S;
                    int jc2 = jc + S, pos = i, row2 = n;
                    size_t bkc = bk;
                    while (jc2 >= nchunks) {  // one step of the walk per row
                        jc2 -= nchunks;
                        ++row2;
                        bkc += step_bk;
                        pos += step_i;
                        if (pos >= s.gamma) {
                            pos -= s.gamma;
                            bkc += wrap_bk;
                        }
                    }
                    issue_at(bkc, pos, jc2, stage, row2);
                }
            };
            bool refilled = false;
            {
                int seen = 0;
                if (lane == 0) seen = *reinterpret_cast<volatile int *>(&ctl->arrivals);
                if (__shfl_sync(0xffffffffu, seen, 0) >= kFWarps * (n + 1)) {
                    do_refill();
                    refilled = true;
                }
            }
            if (!mbar_wait(&ctl->xbar[par], xph)) timed_out = true;

            // Refill (see do_refill above) if it could not be done while waiting.
            if (!refilled) do_refill();

            // ---- row statistics: every warp combines the CTA partials, in the same order -------------
            const float4 cv = lane < C ? ctl->slots[par][lane] : make_float4(-INFINITY, 0.0f, -INFINITY, 0.0f);
            const float bq_row = warp_max_redux(cv.x), bp_row = warp_max_redux(cv.z);
            const float rq_row = (bq_row > -INFINITY) ? bq_row : 0.0f, rp_row = (bp_row > -INFINITY) ? bp_row : 0.0f;
            const float Zq = warp_sum(cv.x > -INFINITY ? cv.y * ex2((cv.x - rq_row) * s.scale) : 0.0f);
            const float Zp = warp_sum(cv.z > -INFINITY ? cv.w * ex2((cv.z - rp_row) * s.scale) : 0.0f);
            // the ratio p_i(tok_i)/q_i(tok_i) of this row (chain thread)
            auto token_ratio = [&]() {
                const double lp = ((double)zp_tok - (double)rp_row) * (double)s.scale;
                const double lq = ((double)zq_tok - (double)rq_row) * (double)s.scale;
                return exp2_short(lp - lq) * (double)(Zq / Zp);
            };
            double cd;
            if (row_mode) {
                // Publish this row's ratio for the clusters that walk the later rows of this chain.  The
                // word itself says "ready": it is preset to a NaN pattern, and a ratio is never stored as
                // NaN (a row that produces one is flagged invalid anyway).
                if (chain_thread && rank == 0 && i + 1 < s.gamma) {
                    double ratio = token_ratio();
                    if (ratio != ratio) ratio = 0.0;
                    *reinterpret_cast<volatile double *>(p.ws.ratio + r) = ratio;
                }
                // c_i = product of the published ratios of rows 0..i-1 of this chain (fixed order: a
                // butterfly over the lanes).  Those rows are walked by other clusters at about the same
                // time and publish right after their own statistics, which do not depend on c: no chain of
                // waits forms.  Every lane of the last warp polls one of them.  Bounded waits.
                if (warp == kFWarps - 1) {
                    double cprod = 1.0;
                    const size_t r0 = bk * s.gamma;
                    for (int j0 = 0; j0 < i; j0 += 32) {
                        double v = 1.0;
                        if (j0 + lane < i) {
                            const volatile double *word =
                                reinterpret_cast<const volatile double *>(p.ws.ratio + r0 + j0 + lane);
                            v = *word;
                            if (v != v) {
                                const long long t0 = clock64();
                                while ((v = *word) != v) {
                                    if (clock64() - t0 > kWaitLimitCycles) {
                                        timed_out = true;
                                        v = 0.0;
                                        break;
                                    }
                                }
                            }
                        }
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) v *= __shfl_xor_sync(0xffffffffu, v, o);
                        cprod *= v;
                    }
                    if (lane == 0) {
                        ctl->c[par] = cprod;
                        mbar_arrive(&ctl->cbar[par]);  // c_i is there
                    }
                }
                if (!mbar_wait(&ctl->cbar[par], xph)) timed_out = true;
                cd = ctl->c[par];
            } else {
                cd = ctl->c[par];
                if (chain_thread && n + 1 < nrows) {
                    // c of the next row of the walk: c_{i+1} = c_i ratio, or 1 at the start of the next
                    // chain; publishing it arms the next row's exchange
                    ctl->c[par ^ 1] = (i + 1 < s.gamma) ? cd * token_ratio() : 1.0;
                    mbar_expect_tx(&ctl->xbar[par ^ 1], xbytes);
                }
            }
            const float c = (float)cd;
            const float kappa = (float)(cd * (double)(Zq / Zp));

            if (tid == 0) {
                if (rank == 0) {
                    // nonfinite logits: NaN poisons Z, +inf shows up as an infinite maximum, a row of
                    // -inf only has Z = 0
                    const bool bad = !(Zq > 0.0f) || !(Zp > 0.0f) || !(Zq < INFINITY) || !(Zp < INFINITY) ||
                                     !(bq_row < INFINITY) || !(bp_row < INFINITY);
                    RowInfo ri;
                    ri.flags = bad ? SGBV_STATUS_NONFINITE_LOGIT : 0;
                    ri.pad_ = 0;
                    ri.Zq = (double)Zq;
                    ri.Zp = (double)Zp;
                    ri.mq = bq_row;
                    ri.mp = bp_row;
                    ri.kappa = kappa;
                    ri.c = c;
                    p.ws.rows[r] = ri;
                }
            }

            // thread units -> row units
            const float fq = has_q ? ex2((bq - rq_row) * s.scale) : 0.0f;
            const float fp = has_p ? ex2((bp - rp_row) * s.scale) : 0.0f;
            float kt = kappa * fp / fq;
            float scale_w = fq, scale_d = fq;
            if (__any_sync(0xffffffffu, !(fq > 1e-30f))) {
                // a thread whose share of the target row underflows (or nearly so, which would
                // overflow kt): its q is 0 in row units, its weights vanish, and max(c p - q, 0) = c p
                if (!(fq > 1e-30f)) {
#pragma unroll
                    for (int j = 0; j < NCH; ++j)
#pragma unroll
                        for (int e = 0; e < 4; ++e) eq[j][e] = splat(0.0f);
                    kt = 1.0f;
                    scale_w = 0.0f;
                    scale_d = kappa * fp;
                }
            }

            // ---- second sweep from registers ---------------------------------------------------------
            float *wp = p.ws.wpart + r * s.ntiles + first_cell, *dp = p.ws.dpart + r * s.ntiles + first_cell,
                  *mpp = p.ws.mpart + r * s.ntiles + first_cell;
            if (c < 1.0f)
                sweep_two_dispatch<NCH, true>(eq, ep, kt, scale_w, scale_d, c, s.K, lane, nj, wp, dp, mpp);
            else
                sweep_two_dispatch<NCH, false>(eq, ep, kt, scale_w, scale_d, c, s.K, lane, nj, wp, dp, mpp);

            // one step of the walk
            bk += step_bk;
            i += step_i;
            if (i >= s.gamma) {
                i -= s.gamma;
                bk += wrap_bk;
            }
        }
    }
    if (__any_sync(0xffffffffu, timed_out) && lane == 0) atomicExch(p.error_flag, 1);
    cluster_arrive();  // no CTA leaves while a neighbour may still write into its slots
    cluster_wait();
}

// ---- host side ----------------------------------------------------------------------------------------
struct Plan {
    int cluster, slice_len, nch, occ, stages, grid_clusters, row_mode;
    size_t smem;
};

int g_opt_cluster = 0;     // 0 = automatic
int g_opt_stages = 0;
int g_opt_max_clusters = 0;
int g_opt_occupancy = 0;
int g_opt_walk = 0;        // 0 = automatic, 1 = chains, 2 = rows

constexpr int kSmemPerSm = 228 * 1024;     // shared memory of one SM
constexpr int kSmemReserved = 1024;        // per resident CTA, taken by the system
constexpr int kSms = 148;
// cells per warp that fit the registers when OCC CTAs share an SM
int max_nch(int occ) { return occ <= 2 ? kMaxNch : occ == 3 ? 2 : 1; }

int cells_of(int V) { return (V + kCell - 1) / kCell; }
int slice_cells(int cells, int C) { return (cells + C - 1) / C; }

template <typename T, int NCH, int OCC, bool kRow>
int launch_nch(const Launch &L, const Plan &plan, int *error_flag) {
    auto kernel = fused_chain_kernel<T, NCH, OCC, kRow>;
    static bool attr_done[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SGBV_ERR_CUDA;
    if (!attr_done[dev]) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kSmemPerSm / OCC - kSmemReserved) != cudaSuccess)
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
    fp.row_mode = plan.row_mode;
    fp.error_flag = error_flag;

    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kFThreads);
    cfg.dynamicSmemBytes = plan.smem;
    cfg.stream = L.stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = plan.cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // the kernel may be scheduled before the one ahead of it in the stream has finished (it waits for it
    // itself before it touches global memory): its launch and start-up then overlap that kernel's tail
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = L.s.B <= kChainedLaunchMaxB ? 2 : 1;  // small batches only: see kChainedLaunchMaxB

    int clusters = plan.grid_clusters;
    if (clusters <= 0) {
        // persistent grid: as many clusters as can be co-resident (queried once per configuration)
        static int cached[64][kMaxCluster + 1][kMaxStages + 1];  // [device][cluster size][stages]
        int &slot = cached[dev][plan.cluster][plan.stages];
        if (slot == 0) {
            cfg.gridDim = dim3(plan.cluster * (OCC * kSms / plan.cluster));
            int nmax = 0;
            if (cudaOccupancyMaxActiveClusters(&nmax, kernel, &cfg) != cudaSuccess || nmax < 1) {
                cudaGetLastError();
                return 0;  // this cluster shape cannot be scheduled here: nothing launched
            }
            slot = nmax;
        }
        clusters = slot;
    }
    const long units = plan.row_mode ? (long)fp.nchains * L.s.gamma : (long)fp.nchains;  // what the clusters share out
    if (clusters > units) clusters = (int)units;
    if (plan.row_mode && !L.ratio_preset &&
        cudaMemsetAsync(L.ws.ratio, 0xff, (size_t)fp.nchains * L.s.gamma * sizeof(double), L.stream) != cudaSuccess)
        return SGBV_ERR_CUDA;
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
    if (plan.row_mode) {  // the row walk exists for two CTAs per SM
        if (plan.occ != 2) return SGBV_ERR_SHAPE;
        switch (plan.nch) {
            case 1: return launch_nch<T, 1, 2, true>(L, plan, error_flag);
            case 2: return launch_nch<T, 2, 2, true>(L, plan, error_flag);
            case 3: return launch_nch<T, 3, 2, true>(L, plan, error_flag);
            case 4: return launch_nch<T, 4, 2, true>(L, plan, error_flag);
            case 5: return launch_nch<T, 5, 2, true>(L, plan, error_flag);
            default: return SGBV_ERR_SHAPE;
        }
    }
    switch (plan.occ * 10 + plan.nch) {
        case 21: return launch_nch<T, 1, 2, false>(L, plan, error_flag);
        case 22: return launch_nch<T, 2, 2, false>(L, plan, error_flag);
        case 23: return launch_nch<T, 3, 2, false>(L, plan, error_flag);
        case 24: return launch_nch<T, 4, 2, false>(L, plan, error_flag);
        case 25: return launch_nch<T, 5, 2, false>(L, plan, error_flag);
        case 31: return launch_nch<T, 1, 3, false>(L, plan, error_flag);
        case 32: return launch_nch<T, 2, 3, false>(L, plan, error_flag);
        case 41: return launch_nch<T, 1, 4, false>(L, plan, error_flag);
        default: return SGBV_ERR_SHAPE;
    }
}

}  // namespace

void fused_set_options(int cluster, int stages, int max_clusters, int occupancy, int walk) {
    g_opt_walk = walk;
    g_opt_cluster = cluster;
    g_opt_stages = stages;
    g_opt_max_clusters = max_clusters;
    g_opt_occupancy = occupancy;
}

// Whether the fused path can take this call: rows must be 16-byte aligned for the bulk copies and
// a CTA's slice must fit its registers (at most 5 chunks of 2048 elements, clusters of at most 16).
bool fused_supported(const Launch &L) {
    const size_t esz = L.dtype == SGBV_DTYPE_BF16 ? 2 : 4;
    if (((uintptr_t)L.zq % 16) || ((uintptr_t)L.zp % 16) || (((size_t)L.s.V * esz) % 16)) return false;
    return slice_cells(cells_of(L.s.V), kMaxCluster) * kCell <= kMaxNch * kChunk;
}

int launch_fused(const Launch &L, int *error_flag, bool *walked_rows) {
    *walked_rows = false;
    const Shape &s = L.s;
    const size_t esz = L.dtype == SGBV_DTYPE_BF16 ? 2 : 4;
    const int cells = cells_of(s.V);
    const long nchains = (long)s.B * s.K;
    Plan plan;
    const int occ = g_opt_occupancy ? g_opt_occupancy : 2;
    const int cap = max_nch(occ) * kChunk;  // elements of a row one CTA can hold
    const long cta_slots = (long)occ * kSms;
    int C = g_opt_cluster;
    int Cmin = 1;
    while (Cmin < kMaxCluster && slice_cells(cells, Cmin) * kCell > cap) Cmin *= 2;  // smallest cluster whose slices fit
    if (C == 0) {
        C = Cmin;
        // few chains: spread each over more CTAs while they all stay co-resident in one wave
        while (C < kMaxCluster && nchains * 2 * C <= cta_slots && cells / (2 * C) >= 4) C *= 2;
    }
    // Few rows in all: when every ROW can have a cluster of its own in one wave, share out single rows
    // instead of chains (their only coupling, c_i, is looked up), so that the gamma rows of a chain run
    // side by side instead of one after the other.
    {
        const long units = nchains * s.gamma;
        int Crow = g_opt_cluster ? g_opt_cluster : Cmin;
        if (g_opt_cluster == 0)
            while (Crow < kMaxCluster && units * 2 * Crow <= cta_slots && cells / (2 * Crow) >= 4) Crow *= 2;
        plan.row_mode = occ == 2 && s.gamma > 1 && (g_opt_walk == 2 || (g_opt_walk == 0 && units * Crow <= cta_slots));
        if (plan.row_mode) C = Crow;
    }
    if (C < 1 || C > kMaxCluster || slice_cells(cells, C) * kCell > cap) return g_opt_occupancy ? SGBV_ERR_SHAPE : 0;
    plan.cluster = C;
    plan.occ = occ;
    plan.slice_len = slice_cells(cells, C) * kCell;
    plan.nch = (plan.slice_len + kChunk - 1) / kChunk;
    const size_t stage_bytes = 2 * kChunk * esz;
    int S = g_opt_stages ? g_opt_stages : kMaxStages;
    const size_t budget = kSmemPerSm / occ - kSmemReserved - sizeof(Control);
    if ((size_t)S * stage_bytes > budget) S = (int)(budget / stage_bytes);
    if (S > kMaxStages) S = kMaxStages;
    // a whole row slice is moved to registers before any of its stages is refilled, so the ring must
    // hold all chunks of a row at once
    if (S < 2 || S < plan.nch) return g_opt_stages ? SGBV_ERR_SHAPE : 0;
    plan.stages = S;
    plan.smem = (size_t)S * stage_bytes + sizeof(Control);
    plan.grid_clusters = g_opt_max_clusters;
    *walked_rows = plan.row_mode != 0;
    return L.dtype == SGBV_DTYPE_BF16 ? launch_t<uint16_t>(L, plan, error_flag) : launch_t<float>(L, plan, error_flag);
}

}  // namespace sgbv
