// Fused single-read path (steps A1-A3): one thread-block cluster walks one draft chain (b,k), one
// CTA of 32 warps per SM, the row resident in TENSOR MEMORY between the two sweeps.
//
// For every position i = 0..gamma-1 of the chain the cluster
//   * streams the target row and the draft row from HBM exactly once.  CTA r of the cluster owns a
//     contiguous slice of the vocabulary, warp w of the CTA the 256-entry cells  w, w+32, w+64, w+96
//     of that slice.  Every warp runs its own little ring of bulk asynchronous copies
//     (cp.async.bulk + mbarrier transaction counts; one cell of both tensors per slot): the warp that
//     consumes a slot refills it itself, so the load path needs no block-wide synchronisation and
//     runs ahead across rows and chains;
//   * first sweep: a thread takes 8 (target, draft) pairs of a cell, turns them into exponentials
//     relative to its own maxima of that cell (the maximum maps to exactly 1) and parks them in
//     tensor memory (tcgen05.st; each warp owns 64 of the 512 columns of its lane quarter, 256 KB per
//     SM in all = 32,768 pairs), keeping only the cell's maximum and sum in registers;
//   * exchanges (max, sum-exp) partials in two levels: the warps of a CTA leave theirs in shared
//     memory and the last one to arrive combines them and PUSHES one partial per CTA into every
//     CTA's shared memory with asynchronous distributed-shared-memory stores that complete on the
//     receiver's mbarrier; a warp goes on as soon as all CTA partials of the row have landed.
//     There is no block-wide or cluster-wide barrier inside the row loop;
//   * second sweep: reads the exponentials back from tensor memory (tcgen05.ld) and writes one
//     partial sum of the coupling terms per cell.  Shared memory is never read twice and the
//     registers hold no row data between the sweeps, which is what lets 32 warps share the SM.
// The joint likelihood ratio c_i = p(x^i)/q(x^i) is carried as a running product by one thread per
// CTA, which computes c_{i+1} right after the statistics of row i and arms the next row's exchange
// with it, a whole row before it is needed.  The finishing kernel (weights, scan, extra token)
// consumes the cell sums.
//
// Every wait on an mbarrier or on a word in global memory is bounded; on expiry the warp records
// an error flag and keeps executing the protocol, so a lost copy cannot hang the kernel, and the
// tensor memory is released on every path.
#include <algorithm>
#include <mutex>

#include "sgbv_common.cuh"

namespace sgbv {

namespace {

constexpr int kMaxWarps = 32;              // warps per CTA: 32 (64 registers each) or 16 (128 registers each)
constexpr int kCell = kTile;               // 256 contiguous entries: the unit a warp works on
constexpr int kCtasPerSm = 1;              // CTAs that share an SM (1 or 2): two are in different phases of their rows
                                           // most of the time, so that one's exponentials overlap the other's sums
constexpr int kWarps = 32;                 // warps per CTA (16 warps of 128 registers measured a third slower)
constexpr int kCtaCells = 128 / kCtasPerSm;  // cells of a row per CTA: 16 tensor-memory columns per cell in each of the 4
                                           // lane quarters, 512 columns per SM: 128 cells = 32,768 entries per SM
constexpr int kTmemCols = 512 / kCtasPerSm;  // this CTA's share of the SM's tensor memory
constexpr int kMaxCluster = 8 * kCtasPerSm;  // CTAs per cluster (beyond 8 the size is not portable, which sm_100 allows)
constexpr long long kWaitLimitCycles = 2000000000ll;  // about one second of SM clock
constexpr uint32_t kPollNs = 100u;                    // sleep between two tests of a barrier that is not ready
static_assert(kTile == 256, "the fused path writes one partial sum per 256-element cell");

struct FusedParams {
    const void *zq;
    const void *zp;
    const int32_t *tok;
    Shape s;
    Workspace ws;
    int cluster;      // CTAs per cluster
    int slice_cells;  // cells of a row per CTA (at most kCtaCells)
    int nchains;      // B*K
    const double *carry_loga, *carry_logb;  // Algorithm 2: per-chain joint logs carried in (else NULL)
    int *error_flag;  // set to 1 if a bounded wait expired
    long long poll_limit;  // cycles a poll of a published ratio may take (row walk)
    int withhold;     // failure-detection test: the first row of every chain does not publish its ratio
    int aux_here;     // rows with c < 1 get their two extra sums in this kernel (else: the kernels that follow it)
};

// ---- PTX wrappers ------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// mbarrier operations take the barrier's 32-bit shared-memory address
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: sets `gave_up` if the phase did not complete within about a second.  Between tests the
// warp sleeps, so that a waiting warp leaves the issue slots to the working ones; the clock is read only
// every 64 tests.  A thread that has given up once only tests from then on, so that the time a failing
// kernel takes stays bounded.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, uint32_t &gave_up) {
    if (mbar_test(bar, parity) || gave_up) return;
    uint32_t tests = 0;
    long long t0 = 0;
    for (;;) {
        __nanosleep(kPollNs);
        if (mbar_test(bar, parity)) return;
        if ((++tests & 63u) == 0u) {
            const long long t = clock64();
            if (t0 == 0) t0 = t;
            else if (t - t0 > kWaitLimitCycles) {
                gave_up = 1u;
                return;
            }
        }
    }
}
// One cell of both tensors into a ring slot (the draft part `half` bytes behind the target part): the lane
// with pred != 0 announces 2 x bytes on the slot's barrier and starts the two bulk copies.  Every lane
// executes the statement (no branch); the copies complete on the barrier.
__device__ __forceinline__ void issue_cell(uint32_t dst, const void *zq, const void *zp, uint32_t bytes, uint32_t bar,
                                           uint32_t pred, uint32_t half) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b32 d2, b2;\n\t"
        "setp.ne.u32 p, %5, 0;\n\t"
        "shl.b32 b2, %3, 1;\n\t"
        "add.u32 d2, %0, %6;\n\t"
        "@p mbarrier.arrive.expect_tx.shared::cta.b64 _, [%4], b2;\n\t"
        "@p cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %3, [%4];\n\t"
        "@p cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [d2], [%2], %3, [%4];\n\t}" ::"r"(dst),
        "l"(zq), "l"(zp), "r"(bytes), "r"(bar), "r"(pred), "r"(half)
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
__device__ __forceinline__ void push_f4(void *local, uint32_t local_bar, uint32_t rank, float4 v) {
    uint32_t dst, bar;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(dst) : "r"(smem_u32(local)), "r"(rank));
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(bar) : "r"(local_bar), "r"(rank));
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

// ---- tensor memory --------------------------------------------------------------------------------
// One warp allocates all columns for the CTA (the address lands in shared memory), every warp then
// reads and writes only the lanes of its own quarter (warp index mod 4) and its own columns.
__device__ __forceinline__ void tmem_alloc(uint32_t *dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// 16 consecutive columns of this thread's lane: the 8 target and the 8 draft exponentials of a cell
__device__ __forceinline__ void tmem_st_cell(uint32_t taddr, const float2 (&a)[4], const float2 (&b)[4]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
        "f"(a[0].x), "f"(a[0].y), "f"(a[1].x), "f"(a[1].y), "f"(a[2].x), "f"(a[2].y), "f"(a[3].x), "f"(a[3].y), "f"(b[0].x),
        "f"(b[0].y), "f"(b[1].x), "f"(b[1].y), "f"(b[2].x), "f"(b[2].y), "f"(b[3].x), "f"(b[3].y)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_cell(uint32_t taddr, float2 (&a)[4], float2 (&b)[4]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=f"(a[0].x), "=f"(a[0].y), "=f"(a[1].x), "=f"(a[1].y), "=f"(a[2].x), "=f"(a[2].y), "=f"(a[3].x), "=f"(a[3].y),
          "=f"(b[0].x), "=f"(b[0].y), "=f"(b[1].x), "=f"(b[1].y), "=f"(b[2].x), "=f"(b[2].y), "=f"(b[3].x), "=f"(b[3].y)
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// Waits for this thread's tensor-memory loads; the loaded registers pass through the statement, so that no
// use of them can be scheduled ahead of it.
__device__ __forceinline__ void tmem_wait_ld(float2 (&a)[4], float2 (&b)[4]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+f"(a[0].x), "+f"(a[0].y), "+f"(a[1].x), "+f"(a[1].y), "+f"(a[2].x), "+f"(a[2].y), "+f"(a[3].x), "+f"(a[3].y),
                   "+f"(b[0].x), "+f"(b[0].y), "+f"(b[1].x), "+f"(b[1].y), "+f"(b[2].x), "+f"(b[2].y), "+f"(b[3].x), "+f"(b[3].y)
                 :
                 : "memory");
}

// ---- shared memory layout ------------------------------------------------------------------------
// [rings: 32 warps x slots x (cell of zq, cell of zp)] [full barriers: 32 warps x slots] [Control]
struct Control {
    uint64_t xbar[2];                    // by row parity: "the partials of all CTAs of the cluster are here"
    // partials (maximum of zq, sum eq, maximum of zp, sum ep): of this CTA's warps, and, double-buffered by
    // row parity, of every CTA of the cluster (pushed by their owners)
    float4 wslots[kMaxWarps];
    float4 slots[2][kMaxCluster];
    float4 rs;                           // the row's scalars for the second sweep: rq, rp, kappa, c
    uint32_t tmem_base;                  // address of the allocated tensor memory
};

// Named hardware barriers of the CTA (0 is the one of __syncthreads).
__device__ __forceinline__ void bar_sync(int id, int nthreads) {
    asm volatile("barrier.cta.sync.aligned %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
__device__ __forceinline__ void bar_arrive(int id, int nthreads) {
    asm volatile("barrier.cta.arrive.aligned %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

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

// Sums P values over the 32 lanes of a warp at once ("transposed" butterfly: at every step a lane
// hands half of its values to its partner and keeps the other half).  P is a power of two (<= 8).
// On return v[0] of lane l is the warp total of value number owner_index<P>(l).
template <int P>
__device__ __forceinline__ int owner_index(int lane) {
    int idx = 0;
    if (P >= 2) idx += (lane & 16) ? P / 2 : 0;
    if (P >= 4) idx += (lane & 8) ? P / 4 : 0;
    if (P >= 8) idx += (lane & 4) ? P / 8 : 0;
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

// What the second sweep needs of a row from this thread's point of view.
struct RowScalars {
    float Fq;     // moves sums in units of this thread's row maximum of zq to row-max units (0: the thread saw no finite zq)
    float KF;     // kappa * Fp / Fq: with the cell's factor ratio it makes c p(x)/q(x) = kt * ep/eq
    float kFp;    // kappa * Fp (cells whose target share underflows)
    float c;      // c_i
};

// First sweep of one cell, first half: the lane's 8 target and 8 draft logits from the ring slot (entries past the
// end of the row read as -inf), and their maxima.
template <typename T>
__device__ __forceinline__ void first_sweep_fetch(const unsigned char *slot, int lane, bool is_tail, int tail_valid,
                                                  float2 (&eq)[4], float2 (&ep)[4], float &m1, float &m2) {
    read_cell<T>(slot, lane, eq);
    read_cell<T>(slot + kCell * (int)sizeof(T), lane, ep);
    if (is_tail) {  // the row ends inside this cell
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (cell_offset<T>(lane, 2 * e) >= tail_valid) eq[e].x = ep[e].x = -INFINITY;
            if (cell_offset<T>(lane, 2 * e + 1) >= tail_valid) eq[e].y = ep[e].y = -INFINITY;
        }
    }
    m1 = m2 = -INFINITY;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        m1 = max3(m1, eq[e].x, eq[e].y);
        m2 = max3(m2, ep[e].x, ep[e].y);
    }
}
// Second half: exponentials relative to the thread's own maxima of the cell (0 if it saw only -inf; the maximum
// itself maps to exactly 1, so point-mass rows stay exact) into tensor memory, and their sums.
__device__ __forceinline__ void first_sweep_store(uint32_t taddr_cell, float scale, float2 (&eq)[4], float2 (&ep)[4], float m1,
                                                  float m2, float &s1, float &s2) {
    const float bq = (m1 > -INFINITY) ? m1 : 0.0f;
    const float bp = (m2 > -INFINITY) ? m2 : 0.0f;
    const float2 nbq = splat(-bq), nbp = splat(-bp), sc2 = splat(scale);
    float2 sq2 = splat(0.0f), sp2 = splat(0.0f);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const float2 aq = __fmul2_rn(__fadd2_rn(eq[e], nbq), sc2);
        const float2 ap = __fmul2_rn(__fadd2_rn(ep[e], nbp), sc2);
        eq[e] = make_float2(ex2(aq.x), ex2(aq.y));
        ep[e] = make_float2(ex2(ap.x), ex2(ap.y));
        sq2 = __fadd2_rn(sq2, eq[e]);
        sp2 = __fadd2_rn(sp2, ep[e]);
    }
    tmem_st_cell(taddr_cell, eq, ep);
    s1 = sq2.x + sq2.y;
    s2 = sp2.x + sp2.y;
}

// Second sweep of one cell, read back from tensor memory, two vocabulary entries per instruction (f32x2).
// eq/ep are exponentials relative to the THREAD's maxima of the cell; fmq moves the cell's target units to the
// thread's row units, rt is the ratio of the cell's draft and target factors, so that fq = fmq Fq and
// kt = KF rt.  Returns in row-max units
//   w  = sum eq (1 - min{kt ep/eq, 1})^K                    (Eq. 4's weights, Eq. 2's sum)
//   sd = sum max(kt ep - eq, 0)                             (c < 1 only)
//   sm = sum eq (c - t)^2 Q(t)                              (c < 1 only)
// coef: Horner coefficients of Q, (t+1) (1-c)^t, t = 1..K-2.  fmp_stash: this thread's draft factor of the cell
// in shared memory, read only when its target share underflows in a row with c < 1.
template <int KT, bool kAux>
__device__ __forceinline__ void second_sweep_cell(uint32_t taddr_cell, float fmq, float rt, const RowScalars &rs, int K,
                                                  const float2 *coef, const float *fmp_stash, float &w, float &sd_out,
                                                  float &sm_out) {
    float2 eq[4], ep[4];
    tmem_ld_cell(taddr_cell, eq, ep);
    // thread units -> row units
    float scale_w = fmq * rs.Fq, scale_d = scale_w;
    float kt = rs.KF * rt;
    const float v1 = 1.0f - rs.c;
    const float2 nv1 = splat(-v1);
    tmem_wait_ld(eq, ep);
    if (kAux) {
        // A thread whose share of the target row underflows (or nearly so, which would overflow kt): its q
        // is 0 in row units, its weights vanish, and max(c p - q, 0) = c p.  Without the extra sums nothing
        // needs doing: an infinite or NaN kt gives a zero weight through the clamps below.
        const bool tiny = !(scale_w > 1e-30f);
        if (__any_sync(0xffffffffu, tiny)) {
            if (tiny) {
#pragma unroll
                for (int e = 0; e < 4; ++e) eq[e] = splat(0.0f);
                kt = 1.0f;
                scale_w = 0.0f;
                scale_d = rs.kFp * *fmp_stash;
            }
        }
    }
    const float2 nkt = splat(-kt);
    float2 sw = splat(0.0f), sd = splat(0.0f), sm = splat(0.0f);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const float2 q = eq[e];
        const float2 diff = __ffma2_rn(nkt, ep[e], q);  // q - c p, thread units
        const float2 pos = make_float2(fmaxf(diff.x, 0.0f), fmaxf(diff.y, 0.0f));
        if (KT == 1) {  // one draft: Q = 0, the second extra sum vanishes and nothing needs the ratio
            sw = __fadd2_rn(sw, pos);
            if (kAux) sd = __fadd2_rn(sd, make_float2(fmaxf(-diff.x, 0.0f), fmaxf(-diff.y, 0.0f)));
            continue;
        }
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
    w = (sw.x + sw.y) * scale_w;
    if (kAux) {
        sd_out = (sd.x + sd.y) * scale_d;
        sm_out = (sm.x + sm.y) * scale_w;
    }
}

// W warps per CTA; NS ring slots per warp (the cells per warp and row, kCtaCells / W, are a multiple of it, so
// that cell j of a row always sits in slot j % NS); KT: the number of drafts K when it has a specialised
// second sweep (1, 2, 3, 4, 8), else 0 (any K, loops).
template <typename T, bool kRow, int W, int NS, int KT>
__global__ void __launch_bounds__(W * 32, kCtasPerSm) fused_chain_kernel(const FusedParams p) {
    constexpr int kFWarps = W, kFThreads = W * 32, kCellsPerWarp = kCtaCells / W;
    static_assert(kCellsPerWarp % NS == 0, "cell j of a row must always land in slot j % NS");
    extern __shared__ __align__(1024) unsigned char smem[];
    const Shape &s = p.s;
    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);  // (tells the compiler that it is the same in all lanes)
    const int C = p.cluster;
    const int rank = (int)cluster_ctarank();
    const int cid = blockIdx.x / C;
    const int G = gridDim.x / C;
    constexpr int kHalfBytes = kCell * (int)sizeof(T);  // one tensor's cell
    constexpr int kSlotBytes = 2 * kHalfBytes;          // the cell of zq, then the same cell of zp
    constexpr int kStrideBytes = kFWarps * kHalfBytes;  // from one cell of a warp to its next, in a row
    constexpr int kRingBytes = kFWarps * NS * kSlotBytes;
    // [rings][full barriers][draft factors of every thread's cells][Control]
    const unsigned char *ring = smem + (size_t)warp * NS * kSlotBytes;
    const uint32_t ring_u32 = smem_u32(ring);
    const uint32_t full_u32 = smem_u32(smem) + (uint32_t)(kRingBytes + warp * NS * 8);
    float *fmp_stash = reinterpret_cast<float *>(smem + kRingBytes + kFWarps * NS * 8) + tid;  // [cell][thread]
    Control *ctl = reinterpret_cast<Control *>(smem + kRingBytes + kFWarps * NS * 8 + kCellsPerWarp * kFThreads * 4);
    const uint32_t xbar_u32 = smem_u32(&ctl->xbar[0]);

    // this CTA's slice of the vocabulary, and this warp's cells in it: warp, warp + W, ...
    const int cell_begin = rank * p.slice_cells;
    const int ncells_cta = max(0, min(s.ntiles, cell_begin + p.slice_cells) - cell_begin);
    const int ncw = ncells_cta > warp ? (ncells_cta - warp + kFWarps - 1) / kFWarps : 0;  // cells of this warp per row
    const int first_cell = cell_begin + warp;
    // the row's last cell may be a partial one: which of this warp's cells it is (-1: none), and its entries
    const int tail_valid = s.V - (s.ntiles - 1) * kCell;
    const int tail_j = (tail_valid < kCell && ncw > 0 && first_cell + (ncw - 1) * kFWarps == s.ntiles - 1) ? ncw - 1 : -1;

    if (tid == 0) {
        mbar_init(xbar_u32, 1);
        mbar_init(xbar_u32 + 8, 1);
    }
    if (lane == 0)
        for (int k = 0; k < NS; ++k) mbar_init(full_u32 + 8 * k, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncwarp();
    if (warp == 0) tmem_alloc(&ctl->tmem_base, kTmemCols);
    tmem_fence_before();
    __syncthreads();
    tmem_fence_after();
    // lanes of this warp's quarter, and its columns
    const uint32_t taddr = ctl->tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(warp >> 2) * (16u * kCellsPerWarp);
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
    //   chain mode: the list of all rows, u = bk*gamma + i, is cut into G contiguous ranges of equal length (+-1), one
    //               per cluster, so that the clusters finish together whatever the number of chains.  A range may
    //               begin and end inside a chain.  The cluster walks first the HEAD of the chain its range ends in
    //               (rows 0..off_hi-1 of chain_hi) and leaves the ratio c reached there in a word of global memory,
    //               then its whole chains, and last the TAIL of the chain its range begins in (rows off_lo.. of
    //               chain_lo), whose c it picks up from the word the cluster before it wrote at its very start.  The
    //               words are preset to a NaN pattern; the one wait (bounded) is for something written long before.
    //   row mode:   rows u = cid, cid+G, ... of the list.  Used when there are few rows: all rows of a chain then run
    //               at the same time on different clusters, and c_i comes from the ratios p_j(tok_j)/q_j(tok_j) that
    //               the clusters of rows j < i publish in global memory.  A row only waits for rows earlier in the
    //               list, which are walked no later by clusters that are all resident, so every wait ends.
    constexpr bool row_mode = kRow;
    const long total_rows = (long)p.nchains * s.gamma;
    const long range_lo = row_mode ? 0 : total_rows * cid / G, range_hi = row_mode ? 0 : total_rows * (cid + 1) / G;
    const int chain_lo = (int)(range_lo / s.gamma), off_lo = (int)(range_lo % s.gamma);
    const int chain_hi = (int)(range_hi / s.gamma), off_hi = (int)(range_hi % s.gamma);
    const int chain_mid = chain_lo + (off_lo > 0 ? 1 : 0);  // first whole chain of the range
    const int nrows = row_mode ? (int)((total_rows - cid + G - 1) / G) : (int)(range_hi - range_lo);  // rows this cluster walks
    // the row after (bk, i) in this cluster's walk
    auto walk_next = [&](int &bk, int &i) {
        if (row_mode) {
            bk += G / s.gamma;
            i += G % s.gamma;
            if (i >= s.gamma) {
                i -= s.gamma;
                ++bk;
            }
            return;
        }
        ++i;
        if (bk == chain_hi) {  // in the head
            if (i >= off_hi) {
                if (chain_mid < chain_hi) {
                    bk = chain_mid;
                    i = 0;
                } else {
                    bk = chain_lo;
                    i = off_lo;
                }
            }
        } else if (i >= s.gamma && !(bk == chain_lo && off_lo > 0)) {  // a whole chain is done (the tail is the last segment)
            if (bk + 1 < chain_hi) {
                ++bk;
                i = 0;
            } else {
                bk = chain_lo;
                i = off_lo;
            }
        }
    };
    const uint32_t xbytes = (uint32_t)(C * sizeof(float4));  // one partial from every CTA of the cluster
    uint32_t timed_out = 0;

    // ---- this warp's copy ring --------------------------------------------------------------------
    // Cell j of a row lands in slot j % NS.  The warp that has moved a cell from its slot to registers refills
    // the slot at once with the next cell that maps to it: cell j + NS of the same row, or, past the warp's
    // last cell, the slot's first cell of the next row of the walk.  So the schedule is fixed at compile time
    // apart from the number of cells this warp has (ncw); lane 0 starts the copies.  `pending` has bit k set
    // while a copy into slot k is under way, `phases` bit k is the parity of slot k's barrier.  A warp that has
    // given up on a wait issues no further loads and, before it leaves, waits for those in flight.
    const size_t row_bytes = (size_t)s.V * sizeof(T);
    const unsigned char *const zq_warp = reinterpret_cast<const unsigned char *>(p.zq) + (size_t)first_cell * kHalfBytes;
    const unsigned char *const zp_warp = reinterpret_cast<const unsigned char *>(p.zp) + (size_t)first_cell * kHalfBytes;
    const uint32_t is_lane0 = lane == 0 ? 1u : 0u;
    uint32_t pending = 0, phases = 0;
#define SGBV_ISSUE(QROW, PROW, JJ, SLOT)                                                                                \
    do {                                                                                                               \
        const uint32_t bytes_ = ((JJ) == tail_j) ? (uint32_t)(tail_valid * (int)sizeof(T)) : (uint32_t)kHalfBytes;      \
        issue_cell(ring_u32 + (uint32_t)((SLOT) * kSlotBytes), (QROW) + (size_t)(JJ) * kStrideBytes,                    \
                   (PROW) + (size_t)(JJ) * kStrideBytes, bytes_, full_u32 + 8u * (uint32_t)(SLOT), is_lane0, kHalfBytes); \
        pending |= 1u << (SLOT);                                                                                       \
    } while (0)
    // First sweep of cell J of the row whose cells start at (QROW, PROW); the slot is refilled from the same row
    // or, past this warp's last cell, from the row that follows (QNXT, PNXT; only if MORE).
#define SGBV_FIRST_SWEEP_CELL(J, QROW, PROW, QNXT, PNXT, MORE)                                                          \
    do {                                                                                                               \
        const int slot_ = (J) % NS; /* (a constant once the loop is unrolled) */                                       \
        if (pending & (1u << slot_)) {                                                                                 \
            mbar_wait(full_u32 + 8u * slot_, (phases >> slot_) & 1u, timed_out);                                       \
            phases ^= 1u << slot_;                                                                                     \
            pending ^= 1u << slot_;                                                                                    \
        }                                                                                                              \
        float2 eq_[4], ep_[4];                                                                                         \
        first_sweep_fetch<T>(ring + slot_ * kSlotBytes, lane, (J) == tail_j, tail_valid, eq_, ep_, mq[J], mp[J]);      \
        /* every lane holds its share of the slot in registers now: refill it */                                       \
        __syncwarp();                                                                                                  \
        if ((J) + NS < ncw) {                                                                                          \
            if (!timed_out) SGBV_ISSUE(QROW, PROW, (J) + NS, slot_);                                                   \
        } else if (MORE) {                                                                                             \
            SGBV_ISSUE(QNXT, PNXT, slot_, slot_);                                                                      \
        }                                                                                                              \
        first_sweep_store(taddr + 16u * (uint32_t)(J), s.scale, eq_, ep_, mq[J], mp[J], sq[J], sp[J]);                 \
    } while (0)

    // rows of the walk: A = the row whose second sweep runs, B = the one after it, whose first sweep runs in the
    // same loop, D = the one after B, whose cells are requested meanwhile
    int bk_a = 0, i_a = 0;  // (set when B becomes A)
    int bk_b = row_mode ? cid / s.gamma : (off_hi > 0 ? chain_hi : chain_mid);  // (a range of gamma rows or more has one of them)
    int i_b = row_mode ? cid % s.gamma : 0;
    const unsigned char *q_b = zq_warp + ((size_t)bk_b * s.zq_rows + i_b) * row_bytes;  // this warp's first cell of row B
    const unsigned char *p_b = zp_warp + ((size_t)bk_b * s.gamma + i_b) * row_bytes;
    if (nrows > 0) {
#pragma unroll
        for (int k = 0; k < NS; ++k)
            if (k < ncw) SGBV_ISSUE(q_b, p_b, k, k);
    }

    // The last warp of this CTA combines the partials, carries c_i and fetches the token logits of a row while its
    // first sweep runs (every lane the same words).
    const bool combiner = warp == kFWarps - 1;
    // c at the start of chain bk: 1, or exp(log p(s) - log q(s)) of what Algorithm 2 carries in
#define SGBV_C0(BK) (p.carry_loga ? exp_short(p.carry_logb[BK] - p.carry_loga[BK]) : 1.0)
    double c_carry = 1.0;  // chain walk: c of the row whose exchange comes next (the first row of the walk starts a chain)
    if (combiner && nrows > 0) c_carry = SGBV_C0(bk_b);

    float fmq[kCellsPerWarp], rt[kCellsPerWarp];  // row A: what the second sweep needs of every cell
    RowScalars rs;                                 // row A
    rs.Fq = rs.KF = rs.kFp = 0.0f;
    rs.c = 1.0f;
#pragma unroll
    for (int j = 0; j < kCellsPerWarp; ++j) fmq[j] = rt[j] = 0.0f;

    // n = -1: only the first sweep of row 0; n = nrows - 1: only the second sweep of the last row
    for (int n = -1; n < nrows; ++n) {
        const bool has_a = n >= 0, has_b = n + 1 < nrows;
        // row D, the one after B
        int bk_d = bk_b, i_d = i_b;
        walk_next(bk_d, i_d);
        const bool has_d = n + 2 < nrows;
        const bool more = has_d && !timed_out;
        const unsigned char *q_d = zq_warp + ((size_t)bk_d * s.zq_rows + i_d) * row_bytes;
        const unsigned char *p_d = zp_warp + ((size_t)bk_d * s.gamma + i_d) * row_bytes;
        const size_t r_a = (size_t)bk_a * s.gamma + i_a, r_b = (size_t)bk_b * s.gamma + i_b;

        // ---- combining warp: the logits of row B's draft token ------------------------------------------
        float zq_tok = 0.0f, zp_tok = 0.0f;
        const int par = (n + 1) & 1;  // of row B's exchange
        const uint32_t xph = (uint32_t)((n + 1) >> 1) & 1u;
        const uint32_t xbar = xbar_u32 + 8u * (uint32_t)par;
        if (combiner && has_b) {
            if (C > 1 && lane == 0) mbar_expect_tx(xbar, xbytes);  // row B's partials of the cluster's CTAs
            int t = p.tok ? p.tok[r_b] : 0;
            if (t < 0 || t >= s.V) t = 0;  // the finishing kernel flags the batch row
            zq_tok = ld_logit(reinterpret_cast<const T *>(p.zq) + ((size_t)bk_b * s.zq_rows + i_b) * s.V, t);
            zp_tok = ld_logit(reinterpret_cast<const T *>(p.zp) + r_b * s.V, t);
        }

        // ---- second sweep of row A from tensor memory, cell by cell, each followed by the first sweep of the
        //      same cell of row B into the columns just read: the exponentials of the one and the sums of the
        //      other keep different pipes busy --------------------------------------------------------------
        float mq[kCellsPerWarp], mp[kCellsPerWarp], sq[kCellsPerWarp], sp[kCellsPerWarp];  // row B
        float wsum[kCellsPerWarp];                                                         // row A
#pragma unroll
        for (int j = 0; j < kCellsPerWarp; ++j) {
            mq[j] = mp[j] = -INFINITY;
            sq[j] = sp[j] = wsum[j] = 0.0f;
        }
        float *wp = p.ws.wpart + r_a * s.ntiles + first_cell;
        // The common case by far has nothing to decide per cell: a warp with all its cells, rows before and after,
        // no partial cell.  Its loop body is straight-line code.
        // Rows with c < 1 may need two more sums for Eq. 2.  Small and medium problems work them out here, for all
        // such rows (p.aux_here).  Large ones leave them to two kernels that follow this one and only touch the rows
        // whose plain numerator would cancel, a few per cent: here they slow every row with c < 1, and with it the
        // whole cluster, by more than half, which is worth two more launches only when the step is long.
        const bool aux_row = p.aux_here && rs.c < 1.0f;
        const bool steady = ncw == kCellsPerWarp && has_a && more && tail_j < 0 && !aux_row;
        if (steady) {
#pragma unroll
            for (int j = 0; j < kCellsPerWarp; ++j) {
                float unused0, unused1;
                second_sweep_cell<KT, false>(taddr + 16u * (uint32_t)j, fmq[j], rt[j], rs, s.K, nullptr, nullptr, wsum[j],
                                             unused0, unused1);
                const int slot = j % NS;  // (a constant once the loop is unrolled)
                mbar_wait(full_u32 + 8u * slot, (phases >> slot) & 1u, timed_out);
                phases ^= 1u << slot;
                float2 eq_[4], ep_[4];
                first_sweep_fetch<T>(ring + slot * kSlotBytes, lane, false, tail_valid, eq_, ep_, mq[j], mp[j]);
                __syncwarp();  // every lane holds its share of the slot in registers now: refill it
                if (j + NS < kCellsPerWarp)
                    issue_cell(ring_u32 + (uint32_t)(slot * kSlotBytes), q_b + (size_t)(j + NS) * kStrideBytes,
                               p_b + (size_t)(j + NS) * kStrideBytes, kHalfBytes, full_u32 + 8u * (uint32_t)slot, is_lane0,
                               kHalfBytes);
                else
                    issue_cell(ring_u32 + (uint32_t)(slot * kSlotBytes), q_d + (size_t)slot * kStrideBytes,
                               p_d + (size_t)slot * kStrideBytes, kHalfBytes, full_u32 + 8u * (uint32_t)slot, is_lane0,
                               kHalfBytes);
                first_sweep_store(taddr + 16u * (uint32_t)j, s.scale, eq_, ep_, mq[j], mp[j], sq[j], sp[j]);
            }
        } else if (has_a && aux_row) {  // the rare kind of row: two more sums per cell
            float *dp = p.ws.dpart + r_a * s.ntiles + first_cell, *mpp = p.ws.mpart + r_a * s.ntiles + first_cell;
            float2 coef[KT > 2 ? KT - 2 : 1];
            if (KT > 2) {
                float vj = 1.0f;
#pragma unroll
                for (int t = 1; t <= KT - 2; ++t) {
                    vj *= 1.0f - rs.c;
                    coef[t - 1] = splat((float)(t + 1) * vj);
                }
            }
#pragma unroll
            for (int j = 0; j < kCellsPerWarp; ++j) {
                if (j < ncw) {  // warp-uniform
                    float aux[2];
                    second_sweep_cell<KT, true>(taddr + 16u * (uint32_t)j, fmq[j], rt[j], rs, s.K, coef,
                                                fmp_stash + j * kFThreads, wsum[j], aux[0], aux[1]);
                    warp_sum_multi<2>(aux, lane);  // the two extra sums of the cell leave right away
                    if ((lane & 15) == 0) ((lane & 16) ? mpp : dp)[j * kFWarps] = aux[0];
                    if (has_b) SGBV_FIRST_SWEEP_CELL(j, q_b, p_b, q_d, p_d, more);
                }
            }
        } else {
#pragma unroll
            for (int j = 0; j < kCellsPerWarp; ++j) {
                if (j < ncw) {  // warp-uniform
                    float unused0, unused1;
                    if (has_a)
                        second_sweep_cell<KT, false>(taddr + 16u * (uint32_t)j, fmq[j], rt[j], rs, s.K, nullptr, nullptr, wsum[j],
                                                     unused0, unused1);
                    if (has_b) SGBV_FIRST_SWEEP_CELL(j, q_b, p_b, q_d, p_d, more);
                }
            }
        }
        // row A's cell sums: summed over the warp now, stored after the exchange below (a store that is still
        // under way would hold up the memory fence of the exchange)
        const int idx = owner_index<kCellsPerWarp>(lane);  // the lane that owns value number idx stores it
        constexpr int kOwnerMask = 32 / kCellsPerWarp - 1;  // lanes that hold the same total
        const bool store_w = has_a && (lane & kOwnerMask) == 0 && idx < ncw;
        if (has_a) warp_sum_multi<kCellsPerWarp>(wsum, lane);
        if (!has_b) {
            if (store_w) wp[idx * kFWarps] = wsum[0];
            break;
        }
        timed_out = __any_sync(0xffffffffu, timed_out != 0);  // the warp gives up as one
        tmem_wait_st();

        // ---- this thread's partial of row B: cell sums moved to its maximum over the cells; what the
        //      second sweep will need of every cell: fmq[j] = cell's target units -> thread's row units,
        //      rt[j] = ratio of the cell's draft and target factors ------------------------------------
        float mqt = mq[0], mpt = mp[0];
#pragma unroll
        for (int j = 1; j < kCellsPerWarp; ++j) {
            mqt = fmaxf(mqt, mq[j]);
            mpt = fmaxf(mpt, mp[j]);
        }
        const bool has_q = mqt > -INFINITY, has_p = mpt > -INFINITY;
        const float bqt = has_q ? mqt : 0.0f, bpt = has_p ? mpt : 0.0f;
        float sqt = 0.0f, spt = 0.0f;
#pragma unroll
        for (int j = 0; j < kCellsPerWarp; ++j) {
            fmq[j] = rt[j] = 0.0f;
            if (j < ncw) {  // a cell without a finite entry has sum 0 and factor 2^-inf = 0
                const float dq = (mq[j] - bqt) * s.scale, dp = (mp[j] - bpt) * s.scale;
                const float fmp = ex2(dp);
                fmq[j] = ex2(dq);
                rt[j] = ex2(dp - dq);  // (NaN or inf where a factor is 0: those cells weigh nothing)
                sqt = fmaf(sq[j], fmq[j], sqt);
                spt = fmaf(sp[j], fmp, spt);
                fmp_stash[j * kFThreads] = fmp;
            }
        }
        // warp partials relative to the warp's maxima
        const float bqw = warp_max_redux(has_q ? bqt : -INFINITY), bpw = warp_max_redux(has_p ? bpt : -INFINITY);
        const float rqw = (bqw > -INFINITY) ? bqw : 0.0f, rpw = (bpw > -INFINITY) ? bpw : 0.0f;
        sqt = warp_sum(has_q ? sqt * ex2((bqt - rqw) * s.scale) : 0.0f);
        spt = warp_sum(has_p ? spt * ex2((bpt - rpw) * s.scale) : 0.0f);
        // Exchange.  Every warp leaves its partial in shared memory; the LAST warp of the CTA combines them,
        // trades the CTA's partial with the other CTAs of the cluster (asynchronous distributed-shared-memory
        // stores that complete on the receiver's mbarrier; it alone polls that barrier), works out the row's
        // scalars and hands them to the others.  The others wait on hardware barriers, which costs them no
        // issue slots: barrier 1 = "all partials are in", barrier 2 = "the row's scalars are in".
        // (a store to shared memory followed by an arrival on the barrier is the producer half of the hardware
        // barrier's producer/consumer pattern: the consumer that syncs on it sees the store)
        if (lane == 0) ctl->wslots[warp] = make_float4(bqw, sqt, bpw, spt);
        __syncwarp();
        float4 rowv;  // rq, rp, kappa, c
        if (!combiner) {
            bar_arrive(1, kFThreads);
            bar_sync(2, kFThreads);
            rowv = ctl->rs;  // (the barrier statement is a compiler barrier for memory)
        } else {
            bar_sync(1, kFThreads);
            const float4 v = lane < kFWarps ? ctl->wslots[lane] : make_float4(-INFINITY, 0.0f, -INFINITY, 0.0f);
            float bq_row = warp_max_redux(v.x), bp_row = warp_max_redux(v.z);
            float rq_row = (bq_row > -INFINITY) ? bq_row : 0.0f, rp_row = (bp_row > -INFINITY) ? bp_row : 0.0f;
            float Zq = warp_sum(v.x > -INFINITY ? v.y * ex2((v.x - rq_row) * s.scale) : 0.0f);
            float Zp = warp_sum(v.z > -INFINITY ? v.w * ex2((v.z - rp_row) * s.scale) : 0.0f);
            if (C > 1) {  // the same once more over the CTAs of the cluster
                if (lane < C) push_f4(&ctl->slots[par][rank], xbar, (uint32_t)lane, make_float4(bq_row, Zq, bp_row, Zp));
                mbar_wait(xbar, xph, timed_out);
                timed_out = __any_sync(0xffffffffu, timed_out != 0);
                const float4 cv = lane < C ? ctl->slots[par][lane] : make_float4(-INFINITY, 0.0f, -INFINITY, 0.0f);
                bq_row = warp_max_redux(cv.x);
                bp_row = warp_max_redux(cv.z);
                rq_row = (bq_row > -INFINITY) ? bq_row : 0.0f;
                rp_row = (bp_row > -INFINITY) ? bp_row : 0.0f;
                Zq = warp_sum(cv.x > -INFINITY ? cv.y * ex2((cv.x - rq_row) * s.scale) : 0.0f);
                Zp = warp_sum(cv.z > -INFINITY ? cv.w * ex2((cv.z - rp_row) * s.scale) : 0.0f);
            }
            // The ratio p_i(tok_i)/q_i(tok_i) of this row: a chain of float64 operations.  In the chain walk only the
            // NEXT row needs it, so it is worked out after the other warps have been released.
#define SGBV_RATIO()                                                                                                     \
    (exp2_short(((double)zp_tok - (double)rp_row) * (double)s.scale - ((double)zq_tok - (double)rq_row) * (double)s.scale) * \
     (double)(Zq / Zp))
            double cd;
            if (row_mode) {
                const double ratio = SGBV_RATIO();
                // Publish this row's ratio for the clusters that walk the later rows of this chain.  The
                // word itself says "ready": it is preset to a NaN pattern, and a ratio is never stored as
                // NaN (a row that produces one is flagged invalid anyway).
                if (lane == 0 && rank == 0 && i_b + 1 < s.gamma && !(p.withhold && i_b == 0))
                    *reinterpret_cast<volatile double *>(p.ws.ratio + r_b) = (ratio != ratio) ? 0.0 : ratio;
                // c_i = product of the published ratios of rows 0..i-1 of this chain (fixed order: a
                // butterfly over the lanes).  Those rows are walked by other clusters at about the same
                // time and publish right after their own statistics, which do not depend on c: no chain of
                // waits forms.  Every lane polls one of them.  Bounded waits.
                cd = SGBV_C0(bk_b);
                const size_t r0 = (size_t)bk_b * s.gamma;
                for (int j0 = 0; j0 < i_b; j0 += 32) {
                    double w = 1.0;
                    if (j0 + lane < i_b) {
                        const volatile double *word = reinterpret_cast<const volatile double *>(p.ws.ratio + r0 + j0 + lane);
                        w = *word;
                        if (w != w && timed_out) w = 0.0;
                        if (w != w) {
                            const long long t0 = clock64();
                            while ((w = *word) != w) {
                                if (clock64() - t0 > p.poll_limit) {
                                    timed_out = 1;
                                    w = 0.0;
                                    break;
                                }
                            }
                        }
                    }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) w *= __shfl_xor_sync(0xffffffffu, w, o);
                    cd *= w;
                }
                timed_out = __any_sync(0xffffffffu, timed_out != 0);
            } else {
                cd = c_carry;  // carried along the chain
            }
            rowv = make_float4(rq_row, rp_row, (float)(cd * (double)(Zq / Zp)), (float)cd);
            if (lane == 0) ctl->rs = rowv;
            __syncwarp();
            bar_arrive(2, kFThreads);
            // off the critical path: c of the next row of the chain walk (c_{i+1} = c_i ratio, and 1 at the start of
            // the next chain), and the row's record for the finishing kernel
            if (!row_mode) {
                const double c_next = cd * SGBV_RATIO();  // c after this row
                // the head of a chain that another cluster continues: leave c where that cluster looks for it
                if (bk_b == chain_hi && i_b == off_hi - 1 && lane == 0 && rank == 0)
                    *reinterpret_cast<volatile double *>(p.ws.cut + bk_b) = (c_next != c_next) ? 0.0 : c_next;
                if (has_d) {
                    if (i_d == 0) {
                        c_carry = SGBV_C0(bk_d);
                    } else if (bk_d == bk_b) {
                        c_carry = c_next;
                    } else {  // the tail of a chain whose head another cluster walked at its very start
                        const volatile double *word = reinterpret_cast<const volatile double *>(p.ws.cut + bk_d);
                        double w = *word;
                        if (w != w && !timed_out) {
                            const long long t0 = clock64();
                            while ((w = *word) != w)
                                if (clock64() - t0 > kWaitLimitCycles) {
                                    timed_out = 1;
                                    break;
                                }
                        }
                        c_carry = (w != w) ? 0.0 : w;
                    }
                }
            }
            if (lane == 0 && rank == 0) {
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
                ri.kappa = rowv.z;
                ri.c = rowv.w;
                p.ws.rows[r_b] = ri;
            }
#undef SGBV_RATIO
        }
        if (store_w) wp[idx * kFWarps] = wsum[0];
        // this thread's row units -> row-max units; row B becomes row A
        const float Fp = has_p ? ex2((bpt - rowv.y) * s.scale) : 0.0f;
        rs.Fq = has_q ? ex2((bqt - rowv.x) * s.scale) : 0.0f;
        // equal factors (identical rows above all) must give kappa itself: p = q everywhere then leaves an
        // exactly zero residual
        rs.KF = (Fp == rs.Fq) ? rowv.z : rowv.z * Fp * rcp(rs.Fq);
        rs.kFp = rowv.z * Fp;
        rs.c = rowv.w;
        bk_a = bk_b;
        i_a = i_b;
        bk_b = bk_d;
        i_b = i_d;
        q_b = q_d;
        p_b = p_d;
    }
    // a warp that gave up may still have copies under way: they must land before the shared memory goes
    if (timed_out) {
        uint32_t fresh = 0;
#pragma unroll
        for (int k = 0; k < NS; ++k)
            if (pending & (1u << k)) mbar_wait(full_u32 + 8u * k, (phases >> k) & 1u, fresh);
        if (lane == 0) atomicExch(p.error_flag, 1);
    }
    cluster_arrive();  // no CTA leaves while a neighbour may still write into its slots
    cluster_wait();
    tmem_fence_before();
    __syncthreads();  // every warp of this CTA is done with the tensor memory
    if (warp == 0) tmem_dealloc(ctl->tmem_base, kTmemCols);
#undef SGBV_ISSUE
#undef SGBV_FIRST_SWEEP_CELL
#undef SGBV_C0
}

// ---- host side ----------------------------------------------------------------------------------------
struct Plan {
    int cluster, slice_cells, row_mode;
};

int g_opt_cluster = 0;     // 0 = automatic
int g_opt_max_clusters = 0;
int g_opt_walk = 0;        // 0 = automatic, 1 = chains, 2 = rows
int g_opt_poll_us = 0;     // 0 = about a second
int g_opt_withhold = 0;
int g_opt_aux = 0;         // 0 = automatic, 1 = the extra sums of rows with c < 1 in the streaming kernel, 2 = in kernels of their own
constexpr double kAuxApartMinBytes = 1024.0 * 1024 * 1024;

constexpr int kSmemPerCta = (228 * 1024) / kCtasPerSm - 1024;  // largest dynamic shared memory of one CTA
constexpr int kDevices = 64;
std::mutex g_plan_mu;      // guards the options and the per-device caches below

constexpr int kCtaSlots = 148 * kCtasPerSm;  // CTAs the device holds
// ring slots per warp: half a row's cells for float32 (128 KB of copies under way per SM), all of them for bfloat16
template <typename T>
constexpr int slots_for() { return (sizeof(T) == 4 ? 2 : 4) * 32 / kWarps / kCtasPerSm; }
template <typename T>
constexpr size_t smem_bytes() {
    return (size_t)kWarps * slots_for<T>() * (2 * kCell * sizeof(T) + 8) + (size_t)(kCtaCells / kWarps) * kWarps * 32 * 4 + sizeof(Control);
}
int slice_cells_of(int cells, int C) { return (cells + C - 1) / C; }

template <typename T, bool kRow, int KT>
cudaError_t prepare(int dev) {
    static bool attr_done[kDevices];
    if (!attr_done[dev]) {
        cudaError_t e = cudaFuncSetAttribute(fused_chain_kernel<T, kRow, kWarps, slots_for<T>(), KT>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemPerCta);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(fused_chain_kernel<T, kRow, kWarps, slots_for<T>(), KT>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        if (e != cudaSuccess) return e;
        attr_done[dev] = true;
    }
    return cudaSuccess;
}

// Clusters of C CTAs of this kernel that the device runs side by side (queried once per configuration).
template <typename T, bool kRow, int KT>
int resident_clusters(int dev, int C) {
    static int cached[kDevices][kMaxCluster + 1];
    int &slot = cached[dev][C];
    if (slot == 0) {
        cudaLaunchConfig_t cfg = {};
        cfg.blockDim = dim3(kWarps * 32);
        cfg.dynamicSmemBytes = smem_bytes<T>();
        cfg.gridDim = dim3(C * (kCtaSlots / C));
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = C;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int nmax = 0;
        if (cudaOccupancyMaxActiveClusters(&nmax, fused_chain_kernel<T, kRow, kWarps, slots_for<T>(), KT>, &cfg) != cudaSuccess || nmax < 1) {
            cudaGetLastError();
            return 0;
        }
        slot = nmax;
    }
    return slot;
}

template <typename T, bool kRow, int KT>
int launch_as(const Launch &L, const Plan &plan, int *error_flag, int clusters, bool aux_here) {
    FusedParams fp;
    fp.zq = L.zq;
    fp.zp = L.zp;
    fp.tok = L.tok;
    fp.s = L.s;
    fp.ws = L.ws;
    fp.cluster = plan.cluster;
    fp.slice_cells = plan.slice_cells;
    fp.nchains = L.s.B * L.s.cpr;
    fp.carry_loga = L.carry_loga;
    fp.carry_logb = L.carry_logb;
    fp.error_flag = error_flag;
    fp.poll_limit = g_opt_poll_us > 0 ? (long long)g_opt_poll_us * 2000ll : kWaitLimitCycles;
    fp.withhold = g_opt_withhold;
    fp.aux_here = aux_here ? 1 : 0;

    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kWarps * 32);
    cfg.dynamicSmemBytes = smem_bytes<T>();
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
    cfg.gridDim = dim3(clusters * plan.cluster);
    if (!kRow && (fp.nchains % clusters) != 0 &&  // some ranges begin or end inside a chain: their hand-over words
        cudaMemsetAsync(L.ws.cut, 0xff, (size_t)fp.nchains * sizeof(double), L.stream) != cudaSuccess)
        return SGBV_ERR_CUDA;
    if (kRow && !L.ratio_preset &&
        cudaMemsetAsync(L.ws.ratio, 0xff, (size_t)fp.nchains * L.s.gamma * sizeof(double), L.stream) != cudaSuccess)
        return SGBV_ERR_CUDA;
    if (L.ev_begin) cudaEventRecord(L.ev_begin, L.stream);
    cudaError_t e = cudaLaunchKernelEx(&cfg, fused_chain_kernel<T, kRow, kWarps, slots_for<T>(), KT>, fp);
    if (L.ev_end) cudaEventRecord(L.ev_end, L.stream);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return SGBV_ERR_CUDA;
    }
    return 1;
}

// Chooses the cluster size and the walk, then launches.  Returns launches, 0 if declined, or < 0.
template <typename T, int KT>
int plan_and_launch(const Launch &L, int *error_flag, bool *walked_rows, bool *aux_apart) {
    const Shape &s = L.s;
    const int cells = s.ntiles;
    const long nchains = (long)s.B * s.cpr, units = nchains * s.gamma;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kDevices) return SGBV_ERR_CUDA;
    if (prepare<T, false, KT>(dev) != cudaSuccess || prepare<T, true, KT>(dev) != cudaSuccess) {
        cudaGetLastError();
        return SGBV_ERR_CUDA;
    }
    Plan plan;
    int Cmin = (cells + kCtaCells - 1) / kCtaCells;  // smallest cluster whose slices fit the tensor memory
    if (Cmin > kMaxCluster) return 0;
    auto fits = [&](int C) { return C >= Cmin && C <= kMaxCluster; };
    auto resident = [&](int C, bool row) {
        return row ? resident_clusters<T, true, KT>(dev, C) : resident_clusters<T, false, KT>(dev, C);
    };
    // Few units of work: spread each over more CTAs (at least half the warps keep a cell) while all of them
    // still run side by side.
    auto widen = [&](long n_units, bool row) {
        int C = Cmin;
        while (2 * C <= kMaxCluster && cells >= C * kWarps && n_units <= resident(2 * C, row)) C *= 2;
        return C;
    };
    int C = g_opt_cluster ? g_opt_cluster : widen(nchains, false);
    // Few rows in all: when every ROW can have a cluster of its own in one wave, share out single rows
    // instead of chains (their only coupling, c_i, is looked up), so that the gamma rows of a chain run
    // side by side instead of one after the other.
    const int Crow = g_opt_cluster ? g_opt_cluster : widen(units, true);
    plan.row_mode = 0;
    if (g_opt_walk == 2 && units > kRatioWords) return SGBV_ERR_SHAPE;  // one ratio word per row, and only so many
    if (s.gamma > 1 && fits(Crow) && units <= kRatioWords &&
        (g_opt_walk == 2 || (g_opt_walk == 0 && units <= resident(Crow, true)))) {
        plan.row_mode = 1;
        C = Crow;
    }
    if (!fits(C)) return g_opt_cluster ? SGBV_ERR_SHAPE : 0;
    plan.cluster = C;
    plan.slice_cells = slice_cells_of(cells, C);
    int clusters = g_opt_max_clusters > 0 ? g_opt_max_clusters : resident(C, plan.row_mode != 0);
    if (clusters < 1) return 0;  // this cluster shape cannot be scheduled here: nothing launched
    const long share = plan.row_mode ? units : nchains;  // what the clusters share out
    if (clusters > share) clusters = (int)share;
    *walked_rows = plan.row_mode != 0;
    // the extra sums of rows with c < 1: in this kernel, or for long steps (chain walk, 1 GB of logits or more) in the
    // kernels that the caller queues behind it
    const double bytes = 2.0 * (double)units * (double)s.V * (double)sizeof(T);
    // (with one draft the extra sum costs the kernel next to nothing, and most rows with c < 1 would be listed)
    const bool aux_here = plan.row_mode || g_opt_aux == 1 || (g_opt_aux == 0 && (bytes < kAuxApartMinBytes || s.K == 1));
    *aux_apart = !aux_here;
    return plan.row_mode ? launch_as<T, true, KT>(L, plan, error_flag, clusters, true)
                         : launch_as<T, false, KT>(L, plan, error_flag, clusters, aux_here);
}

}  // namespace

void fused_set_options(int cluster, int max_clusters, int walk, int poll_us, int withhold, int aux) {
    std::lock_guard<std::mutex> lock(g_plan_mu);
    g_opt_aux = aux;
    g_opt_withhold = withhold;
    g_opt_walk = walk;
    g_opt_cluster = cluster;
    g_opt_max_clusters = max_clusters;
    g_opt_poll_us = poll_us;
}

// Whether the fused path can take this call: rows must be 16-byte aligned for the bulk copies and a
// row must fit the tensor memory of a cluster (8 CTAs x 32,768 entries).
bool fused_supported(const Launch &L) {
    const size_t esz = L.dtype == SGBV_DTYPE_BF16 ? 2 : 4;
    if (((uintptr_t)L.zq % 16) || ((uintptr_t)L.zp % 16) || (((size_t)L.s.V * esz) % 16)) return false;
    return L.s.ntiles <= kMaxCluster * kCtaCells;
}

template <typename T>
int dispatch_k(const Launch &L, int *error_flag, bool *walked_rows, bool *aux_apart) {
    switch (L.s.K) {
        case 1: return plan_and_launch<T, 1>(L, error_flag, walked_rows, aux_apart);
        case 2: return plan_and_launch<T, 2>(L, error_flag, walked_rows, aux_apart);
        case 3: return plan_and_launch<T, 3>(L, error_flag, walked_rows, aux_apart);
        case 4: return plan_and_launch<T, 4>(L, error_flag, walked_rows, aux_apart);
        case 8: return plan_and_launch<T, 8>(L, error_flag, walked_rows, aux_apart);
        default: return plan_and_launch<T, 0>(L, error_flag, walked_rows, aux_apart);
    }
}

int launch_fused(const Launch &L, int *error_flag, bool *walked_rows, bool *aux_apart) {
    *walked_rows = false;
    *aux_apart = false;
    std::lock_guard<std::mutex> lock(g_plan_mu);
    return L.dtype == SGBV_DTYPE_BF16 ? dispatch_k<uint16_t>(L, error_flag, walked_rows, aux_apart)
                                      : dispatch_k<float>(L, error_flag, walked_rows, aux_apart);
}

}  // namespace sgbv
