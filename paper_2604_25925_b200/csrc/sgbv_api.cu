// C ABI of the verify step: argument checks, scratch carving, launch sequence, host-buffer form.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>

#include "sgbv_common.cuh"

namespace sgbv {

namespace {

constexpr size_t kAlign = 256;
constexpr int kMaxDevices = 64;

size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

Shape make_shape(int B, int K, int gamma, int V, float temperature) {
    Shape s;
    s.B = B;
    s.K = K;
    s.gamma = gamma;
    s.V = V;
    s.cpr = K;
    s.zq_rows = gamma + 1;
    s.ntiles = (V + kTile - 1) / kTile;
    const long rows = (long)B * K * gamma;
    long want = (4L * 148 + rows - 1) / rows;  // enough slices to fill the machine a few times over
    if (want < 1) want = 1;
    if (want > s.ntiles) want = s.ntiles;
    s.tiles_per_slice = (int)((s.ntiles + want - 1) / want);
    s.nsplit = (s.ntiles + s.tiles_per_slice - 1) / s.tiles_per_slice;
    s.scale = (float)((double)kLog2e / (double)temperature);
    s.inv_T = 1.0 / (double)temperature;
    return s;
}

struct Carve {
    size_t rows, part, wpart, dpart, mpart, ratio, cut, bonus, h, resmass, status, error, total;
};

Carve carve(const Shape &s) {
    const size_t NR = (size_t)s.B * s.cpr * s.gamma;
    Carve c;
    size_t off = 0;
    // the ratio words sit at the head, at the same place for every shape: on the library's own scratch
    // they keep their "not published yet" pattern from call to call, whatever shapes the calls have
    c.ratio = off;     off += align_up(kRatioWords * sizeof(double));
    c.rows = off;      off += align_up(NR * sizeof(RowInfo));
    c.part = off;      off += align_up(NR * s.nsplit * 4 * sizeof(float));
    c.wpart = off;     off += align_up(NR * s.ntiles * sizeof(float));
    c.dpart = off;     off += align_up(NR * s.ntiles * sizeof(float));
    c.mpart = off;     off += align_up(NR * s.ntiles * sizeof(float));
    c.cut = off;       off += align_up((size_t)s.B * s.cpr * sizeof(double));
    c.bonus = off;     off += align_up((size_t)s.B * 2 * s.ntiles * sizeof(float));
    c.h = off;         off += align_up(NR * sizeof(double));
    c.resmass = off;   off += align_up(NR * sizeof(double));
    c.status = off;    off += align_up((size_t)s.B * sizeof(int32_t));
    c.error = off;     off += align_up(sizeof(int32_t));
    c.total = off;
    return c;
}

int check_shape(int B, int K, int gamma, int V, int dtype) {
    if (B < 1 || K < 1 || gamma < 1 || V < 1 || K > kMaxK || gamma > kMaxGamma || V > kMaxV) return SGBV_ERR_SHAPE;
    if (dtype != SGBV_DTYPE_F32 && dtype != SGBV_DTYPE_BF16) return SGBV_ERR_SHAPE;
    if ((double)B * K * gamma > 2.0e8) return SGBV_ERR_SHAPE;
    return SGBV_OK;
}

// Per-device buffers owned by the library: scratch for sgbv_verify, staging for sgbv_verify_host.
struct DeviceBuffers {
    void *scratch = nullptr;
    size_t scratch_bytes = 0;
    void *stage = nullptr;
    size_t stage_bytes = 0;
    void *idx = nullptr;        // accepted-draft indices that sgbv_verify_gbv has no output for
    size_t idx_bytes = 0;
    // the ratio words at the head of the scratch may not hold the "not published yet" pattern (a call
    // failed between the kernel that consumes them and the one that puts them back)
    bool ratio_dirty = false;
};
DeviceBuffers g_buf[kMaxDevices];
std::mutex g_mu;

// Grows a per-device buffer.  preset_head: the first bytes of a new buffer get the 0xff pattern of unpublished
// ratio words before anyone uses it (the device is idle then).
int grow(void **ptr, size_t *have, size_t need, size_t preset_head = 0) {
    if (*have >= need) return SGBV_OK;
    if (*ptr) {
        if (cudaDeviceSynchronize() != cudaSuccess) return SGBV_ERR_CUDA;
        cudaFree(*ptr);
        *ptr = nullptr;
        *have = 0;
    }
    if (cudaMalloc(ptr, need) != cudaSuccess) {
        cudaGetLastError();
        *ptr = nullptr;
        return SGBV_ERR_CUDA;
    }
    if (preset_head && (cudaMemset(*ptr, 0xff, preset_head) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess)) {
        cudaGetLastError();
        cudaFree(*ptr);
        *ptr = nullptr;
        return SGBV_ERR_CUDA;
    }
    *have = need;
    return SGBV_OK;
}

thread_local int t_last_launches = 0;
thread_local const char *t_last_kernel = "none";
int g_opt_path = 0, g_opt_cluster = 0, g_opt_max_clusters = 0, g_opt_walk = 0, g_opt_poll_us = 0, g_opt_withhold = 0, g_opt_aux = 0;

// Optional timing of the dominant kernel: event pairs recorded around it, summed on request.
struct Profile {
    cudaEvent_t *begin = nullptr;
    cudaEvent_t *end = nullptr;
    int capacity = 0;
    int used = 0;
};
Profile g_prof;

int verify_device(const void *zq, const void *zp, int dtype, const int32_t *tok, const float *u, int B, int K,
                  int gamma, int V, float temperature, int32_t *out_tau, int32_t *out_f, int32_t *out_tokens,
                  void *workspace, size_t workspace_bytes, double *out_h, double *out_resmass,
                  int32_t *out_status, cudaStream_t stream) {
    if (!zq || !zp || !tok || !u || !out_tau || !out_f || !out_tokens) return SGBV_ERR_NULL;
    int rc = check_shape(B, K, gamma, V, dtype);
    if (rc != SGBV_OK) return rc;
    if (!(temperature > 0.0f) || !isfinite(temperature)) return SGBV_ERR_TEMPERATURE;
    const size_t esz = dtype == SGBV_DTYPE_BF16 ? 2 : 4;
    if (((uintptr_t)zq % esz) || ((uintptr_t)zp % esz) || ((uintptr_t)tok % 4) || ((uintptr_t)u % 4) ||
        ((uintptr_t)out_tau % 4) || ((uintptr_t)out_f % 4) || ((uintptr_t)out_tokens % 4) ||
        ((uintptr_t)out_h % 8) || ((uintptr_t)out_resmass % 8) || ((uintptr_t)out_status % 4))
        return SGBV_ERR_ALIGN;

    Launch L;
    L.s = make_shape(B, K, gamma, V, temperature);
    const Carve c = carve(L.s);
    unsigned char *base = nullptr;
    int own_dev = -1;  // >= 0: the scratch is the library's own (nobody else writes to it between calls)
    if (workspace) {
        if (workspace_bytes < c.total || ((uintptr_t)workspace % kAlign)) return SGBV_ERR_WORKSPACE;
        base = (unsigned char *)workspace;
    } else {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SGBV_ERR_CUDA;
        std::lock_guard<std::mutex> lock(g_mu);
        rc = grow(&g_buf[dev].scratch, &g_buf[dev].scratch_bytes, c.total, kRatioWords * sizeof(double));
        if (rc != SGBV_OK) return rc;
        base = (unsigned char *)g_buf[dev].scratch;
        own_dev = dev;
        // The row walk of the fused kernel needs its ratio words preset.  They sit at a fixed place, are preset
        // when the buffer is allocated, and every finishing kernel puts the pattern back after use: whatever the
        // order of eager calls and graph replays, a call finds them ready.  Only a call that failed half-way
        // leaves them in doubt; the next row walk then clears them itself.
        L.ratio_preset = !g_buf[dev].ratio_dirty;
    }
    L.ws.rows = (RowInfo *)(base + c.rows);
    L.ws.part = (float *)(base + c.part);
    L.ws.wpart = (float *)(base + c.wpart);
    L.ws.dpart = (float *)(base + c.dpart);
    L.ws.mpart = (float *)(base + c.mpart);
    L.ws.ratio = (double *)(base + c.ratio);
    L.ws.cut = (double *)(base + c.cut);
    L.ws.bonus = (float *)(base + c.bonus);
    L.ws.h = out_h ? out_h : (double *)(base + c.h);
    L.ws.resmass = out_resmass ? out_resmass : (double *)(base + c.resmass);
    L.ws.status = out_status ? out_status : (int32_t *)(base + c.status);
    L.ws.error = (int32_t *)(base + c.error);
    L.zq = zq;
    L.zp = zp;
    L.dtype = dtype;
    L.tok = tok;
    L.u = u;
    L.out_tau = out_tau;
    L.out_f = out_f;
    L.out_tokens = out_tokens;
    L.stream = stream;

    if (g_prof.used < g_prof.capacity) {
        L.ev_begin = g_prof.begin[g_prof.used];
        L.ev_end = g_prof.end[g_prof.used];
        ++g_prof.used;
    }
    // the fused kernel needs nothing cleared: it reports through the row records and zeroes the
    // error word itself; the two-sweep kernels set status bits with atomics, so those start at zero
    bool fused = g_opt_path != 1 && fused_supported(L);
    L.ws.prestatus = nullptr;
    bool walked_rows = false;
    bool aux_apart = false;
    int n1 = fused ? launch_fused(L, L.ws.error, &walked_rows, &aux_apart) : 0;
    if (n1 < 0) return n1;
    L.ws.ratio_used = (n1 > 0 && walked_rows) ? 1 : 0;
    if (n1 == 0) {
        if (g_opt_path == 2) return SGBV_ERR_SHAPE;
        fused = false;
        L.ws.prestatus = L.ws.status;
        if (cudaMemsetAsync(L.ws.status, 0, (size_t)B * sizeof(int32_t), stream) != cudaSuccess) return SGBV_ERR_CUDA;
        if (cudaMemsetAsync(L.ws.error, 0, sizeof(int32_t), stream) != cudaSuccess) return SGBV_ERR_CUDA;
        n1 = launch_twopass(L);
        if (n1 < 0) return n1;
    }
    // the extra sums of Eq. 2 for rows with c < 1: written for all such rows by the two-sweep path and, for small and
    // medium problems, by the fused kernel; for large ones it leaves them to kernels of their own, which do the few rows
    // that need them
    L.ws.have_aux = 1;
    if (fused && aux_apart) {
        const int na = launch_auxreduce(L);
        if (na < 0) return na;
        n1 += na;
        L.ws.have_aux = 2;
    }
    int n2 = launch_finish(L);
    if (own_dev >= 0 && L.ws.ratio_used) {
        // a walk that cleared the words itself is followed by a finishing kernel that puts them back: the
        // doubt ends unless that kernel was not launched, or nothing ran at all (stream capture)
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        const bool capturing = cudaStreamIsCapturing(stream, &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone;
        std::lock_guard<std::mutex> lock(g_mu);
        if (n2 < 0) g_buf[own_dev].ratio_dirty = true;
        else if (!capturing) g_buf[own_dev].ratio_dirty = false;
    }
    if (n2 < 0) return n2;
    t_last_launches = n1 + n2;
    t_last_kernel = fused ? "fused_chain_kernel" : "otreduce_kernel";
    return SGBV_OK;
}

}  // namespace
}  // namespace sgbv

using namespace sgbv;

extern "C" {

int sgbv_workspace_bytes(int B, int K, int gamma, int V, int dtype, size_t *out_bytes) {
    if (!out_bytes) return SGBV_ERR_NULL;
    int rc = check_shape(B, K, gamma, V, dtype);
    if (rc != SGBV_OK) return rc;
    *out_bytes = carve(make_shape(B, K, gamma, V, 1.0f)).total;
    return SGBV_OK;
}

int sgbv_verify(const float *target_logits, const float *draft_logits, const int32_t *draft_tokens,
                const float *uniforms, int B, int K, int gamma, int V, float temperature,
                int32_t *out_accept_len, int32_t *out_draft_idx, int32_t *out_tokens, void *stream) {
    return verify_device(target_logits, draft_logits, SGBV_DTYPE_F32, draft_tokens, uniforms, B, K, gamma, V,
                         temperature, out_accept_len, out_draft_idx, out_tokens, nullptr, 0, nullptr, nullptr,
                         nullptr, (cudaStream_t)stream);
}

int sgbv_verify_bf16(const uint16_t *target_logits, const uint16_t *draft_logits, const int32_t *draft_tokens,
                     const float *uniforms, int B, int K, int gamma, int V, float temperature,
                     int32_t *out_accept_len, int32_t *out_draft_idx, int32_t *out_tokens, void *stream) {
    return verify_device(target_logits, draft_logits, SGBV_DTYPE_BF16, draft_tokens, uniforms, B, K, gamma, V,
                         temperature, out_accept_len, out_draft_idx, out_tokens, nullptr, 0, nullptr, nullptr,
                         nullptr, (cudaStream_t)stream);
}

int sgbv_verify_ex(const void *target_logits, const void *draft_logits, int dtype, const int32_t *draft_tokens,
                   const float *uniforms, int B, int K, int gamma, int V, float temperature,
                   int32_t *out_accept_len, int32_t *out_draft_idx, int32_t *out_tokens, void *workspace,
                   size_t workspace_bytes, double *out_h, double *out_resmass, int32_t *out_status, void *stream) {
    return verify_device(target_logits, draft_logits, dtype, draft_tokens, uniforms, B, K, gamma, V, temperature,
                         out_accept_len, out_draft_idx, out_tokens, workspace, workspace_bytes, out_h,
                         out_resmass, out_status, (cudaStream_t)stream);
}

int sgbv_verify_host(const void *target_logits, const void *draft_logits, int dtype, const int32_t *draft_tokens,
                     const float *uniforms, int B, int K, int gamma, int V, float temperature,
                     int32_t *out_accept_len, int32_t *out_draft_idx, int32_t *out_tokens, int32_t *out_status,
                     void *stream_) {
    if (!target_logits || !draft_logits || !draft_tokens || !uniforms || !out_accept_len || !out_draft_idx ||
        !out_tokens)
        return SGBV_ERR_NULL;
    int rc = check_shape(B, K, gamma, V, dtype);
    if (rc != SGBV_OK) return rc;
    if (!(temperature > 0.0f) || !isfinite(temperature)) return SGBV_ERR_TEMPERATURE;
    cudaStream_t stream = (cudaStream_t)stream_;
    const size_t esz = dtype == SGBV_DTYPE_BF16 ? 2 : 4;
    const size_t n_zq = (size_t)B * K * (gamma + 1) * V * esz, n_zp = (size_t)B * K * gamma * V * esz;
    const size_t n_tok = (size_t)B * K * gamma * 4, n_u = (size_t)B * (K * gamma + 1) * 4;
    const size_t n_tau = (size_t)B * 4, n_tokens = (size_t)B * (gamma + 1) * 4;
    size_t off = 0;
    const size_t o_zq = off;     off += align_up(n_zq);
    const size_t o_zp = off;     off += align_up(n_zp);
    const size_t o_tok = off;    off += align_up(n_tok);
    const size_t o_u = off;      off += align_up(n_u);
    const size_t o_tau = off;    off += align_up(n_tau);
    const size_t o_f = off;      off += align_up(n_tau);
    const size_t o_tokens = off; off += align_up(n_tokens);
    const size_t o_status = off; off += align_up(n_tau);
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SGBV_ERR_CUDA;
    unsigned char *st = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        rc = grow(&g_buf[dev].stage, &g_buf[dev].stage_bytes, off);
        if (rc != SGBV_OK) return rc;
        st = (unsigned char *)g_buf[dev].stage;
    }
    bool ok = true;
    ok &= cudaMemcpyAsync(st + o_zq, target_logits, n_zq, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(st + o_zp, draft_logits, n_zp, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(st + o_tok, draft_tokens, n_tok, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(st + o_u, uniforms, n_u, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    if (!ok) return SGBV_ERR_CUDA;
    rc = verify_device(st + o_zq, st + o_zp, dtype, (const int32_t *)(st + o_tok), (const float *)(st + o_u), B, K,
                       gamma, V, temperature, (int32_t *)(st + o_tau), (int32_t *)(st + o_f),
                       (int32_t *)(st + o_tokens), nullptr, 0, nullptr, nullptr, (int32_t *)(st + o_status), stream);
    if (rc != SGBV_OK) return rc;
    ok &= cudaMemcpyAsync(out_accept_len, st + o_tau, n_tau, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(out_draft_idx, st + o_f, n_tau, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(out_tokens, st + o_tokens, n_tokens, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    if (out_status)
        ok &= cudaMemcpyAsync(out_status, st + o_status, n_tau, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    ok &= cudaStreamSynchronize(stream) == cudaSuccess;
    return ok ? SGBV_OK : SGBV_ERR_CUDA;
}

int sgbv_modify(const void *target_logits, const void *draft_logits, int dtype, const double *log_a, const double *log_b,
                const float *uniforms, int B, int K, int V, float temperature, int32_t *out_token, double *out_log_a,
                double *out_log_b, double *out_resmass, int32_t *out_status, void *workspace, size_t workspace_bytes,
                void *stream_) {
    if (!target_logits || !draft_logits || !log_a || !log_b || !uniforms || !out_token || !out_log_a || !out_log_b)
        return SGBV_ERR_NULL;
    int rc = check_shape(B, K, 1, V, dtype);
    if (rc != SGBV_OK) return rc;
    if (!(temperature > 0.0f) || !isfinite(temperature)) return SGBV_ERR_TEMPERATURE;
    const size_t esz = dtype == SGBV_DTYPE_BF16 ? 2 : 4;
    if (((uintptr_t)target_logits % esz) || ((uintptr_t)draft_logits % esz) || ((uintptr_t)log_a % 8) ||
        ((uintptr_t)log_b % 8) || ((uintptr_t)uniforms % 4) || ((uintptr_t)out_token % 4) || ((uintptr_t)out_log_a % 8) ||
        ((uintptr_t)out_log_b % 8) || ((uintptr_t)out_resmass % 8) || ((uintptr_t)out_status % 4))
        return SGBV_ERR_ALIGN;
    cudaStream_t stream = (cudaStream_t)stream_;
    Launch L;
    L.s = make_shape(B, K, 1, V, temperature);
    L.s.cpr = 1;      // one chain per batch row: K is only the exponent of Eq. 4's weights here
    L.s.zq_rows = 1;  // and the target tensor holds just the row of this position
    const Carve c = carve(L.s);
    unsigned char *base = nullptr;
    if (workspace) {
        if (workspace_bytes < c.total || ((uintptr_t)workspace % kAlign)) return SGBV_ERR_WORKSPACE;
        base = (unsigned char *)workspace;
    } else {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SGBV_ERR_CUDA;
        std::lock_guard<std::mutex> lock(g_mu);
        rc = grow(&g_buf[dev].scratch, &g_buf[dev].scratch_bytes, c.total, kRatioWords * sizeof(double));
        if (rc != SGBV_OK) return rc;
        base = (unsigned char *)g_buf[dev].scratch;
    }
    L.ws.rows = (RowInfo *)(base + c.rows);
    L.ws.part = (float *)(base + c.part);
    L.ws.wpart = (float *)(base + c.wpart);
    L.ws.dpart = (float *)(base + c.dpart);
    L.ws.mpart = (float *)(base + c.mpart);
    L.ws.ratio = (double *)(base + c.ratio);
    L.ws.cut = (double *)(base + c.cut);
    L.ws.ratio_used = 0;  // (a single position per chain never takes the row walk)
    L.ws.bonus = (float *)(base + c.bonus);
    L.ws.bonus_in_smem = 0;
    L.ws.h = (double *)(base + c.h);
    L.ws.resmass = (double *)(base + c.resmass);
    L.ws.status = (int32_t *)(base + c.status);
    L.ws.prestatus = nullptr;
    L.ws.error = (int32_t *)(base + c.error);
    L.zq = target_logits;
    L.zp = draft_logits;
    L.dtype = dtype;
    L.tok = nullptr;
    L.u = uniforms;
    L.out_tau = nullptr;
    L.out_f = nullptr;
    L.out_tokens = nullptr;
    L.stream = stream;
    L.carry_loga = log_a;
    L.carry_logb = log_b;
    bool fused = g_opt_path != 1 && fused_supported(L);
    bool walked_rows = false;
    bool aux_apart = false;  // (Algorithm 2 needs no extra sums: its draw only uses Eq. 4's weights)
    int n1 = fused ? launch_fused(L, L.ws.error, &walked_rows, &aux_apart) : 0;
    if (n1 < 0) return n1;
    if (n1 == 0) {
        if (g_opt_path == 2) return SGBV_ERR_SHAPE;
        fused = false;
        L.ws.prestatus = L.ws.status;
        if (cudaMemsetAsync(L.ws.status, 0, (size_t)B * sizeof(int32_t), stream) != cudaSuccess) return SGBV_ERR_CUDA;
        if (cudaMemsetAsync(L.ws.error, 0, sizeof(int32_t), stream) != cudaSuccess) return SGBV_ERR_CUDA;
        n1 = launch_twopass(L);
        if (n1 < 0) return n1;
    }
    const int n2 = launch_modify_finish(L, uniforms, out_token, out_log_a, out_log_b, out_resmass, out_status);
    if (n2 < 0) return n2;
    t_last_launches = n1 + n2;
    t_last_kernel = fused ? "fused_chain_kernel" : "otreduce_kernel";
    return SGBV_OK;
}

int sgbv_verify_kseq(const void *target_logits, const void *draft_logits, int dtype, const int32_t *draft_tokens,
                     const float *uniforms, int B, int K, int gamma, int V, float temperature, int32_t *out_accept_len,
                     int32_t *out_tokens, double *out_rho, double *out_accept_prob, int32_t *out_status, void *workspace,
                     size_t workspace_bytes, void *stream_) {
    if (!target_logits || !draft_logits || !draft_tokens || !uniforms || !out_accept_len || !out_tokens) return SGBV_ERR_NULL;
    int rc = check_shape(B, K, gamma, V, dtype);
    if (rc != SGBV_OK) return rc;
    if (!(temperature > 0.0f) || !isfinite(temperature)) return SGBV_ERR_TEMPERATURE;
    const size_t esz = dtype == SGBV_DTYPE_BF16 ? 2 : 4;
    if (((uintptr_t)target_logits % esz) || ((uintptr_t)draft_logits % esz) || ((uintptr_t)draft_tokens % 4) ||
        ((uintptr_t)uniforms % 4) || ((uintptr_t)out_accept_len % 4) || ((uintptr_t)out_tokens % 4) ||
        ((uintptr_t)out_rho % 8) || ((uintptr_t)out_accept_prob % 8) || ((uintptr_t)out_status % 4))
        return SGBV_ERR_ALIGN;
    Launch L;
    L.s = make_shape(B, K, gamma, V, temperature);
    const Carve c = carve(L.s);
    unsigned char *base = nullptr;
    if (workspace) {
        if (workspace_bytes < c.total || ((uintptr_t)workspace % kAlign)) return SGBV_ERR_WORKSPACE;
        base = (unsigned char *)workspace;
    } else {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SGBV_ERR_CUDA;
        std::lock_guard<std::mutex> lock(g_mu);
        rc = grow(&g_buf[dev].scratch, &g_buf[dev].scratch_bytes, c.total, kRatioWords * sizeof(double));
        if (rc != SGBV_OK) return rc;
        base = (unsigned char *)g_buf[dev].scratch;
    }
    L.zq = target_logits;
    L.zp = draft_logits;
    L.dtype = dtype;
    L.tok = draft_tokens;
    L.u = uniforms;
    L.out_tau = out_accept_len;
    L.out_f = nullptr;
    L.out_tokens = out_tokens;
    L.stream = (cudaStream_t)stream_;
    const int n = launch_kseq(L, (float *)(base + c.bonus), out_rho, out_accept_prob,
                              out_status ? out_status : (int32_t *)(base + c.status));
    if (n < 0) return n;
    t_last_launches = n;
    t_last_kernel = "kseq_kernel";
    return SGBV_OK;
}

int sgbv_verify_token(const void *target_logits, const void *draft_logits, int dtype, const int32_t *draft_tokens,
                      const float *uniforms, int B, int gamma, int V, float temperature, int32_t *out_accept_len,
                      int32_t *out_tokens, double *out_accept_prob, int32_t *out_status, void *workspace,
                      size_t workspace_bytes, void *stream) {
    return sgbv_verify_kseq(target_logits, draft_logits, dtype, draft_tokens, uniforms, B, 1, gamma, V, temperature,
                            out_accept_len, out_tokens, nullptr, out_accept_prob, out_status, workspace, workspace_bytes,
                            stream);
}

int sgbv_verify_gbv(const void *target_logits, const void *draft_logits, int dtype, const int32_t *draft_tokens,
                    const float *uniforms, int B, int gamma, int V, float temperature, int32_t *out_accept_len,
                    int32_t *out_tokens, double *out_accept_prob, int32_t *out_status, void *workspace,
                    size_t workspace_bytes, void *stream) {
    if (!out_accept_len) return SGBV_ERR_NULL;
    // single-draft greedy block verification is the K = 1 case of the block verifier; the accepted draft index
    // (0 or -1) lands in scratch
    int rc = check_shape(B, 1, gamma, V, dtype);
    if (rc != SGBV_OK) return rc;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SGBV_ERR_CUDA;
    int32_t *f_scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        rc = grow(&g_buf[dev].idx, &g_buf[dev].idx_bytes, (size_t)B * sizeof(int32_t));
        if (rc != SGBV_OK) return rc;
        f_scratch = (int32_t *)g_buf[dev].idx;
    }
    return verify_device(target_logits, draft_logits, dtype, draft_tokens, uniforms, B, 1, gamma, V, temperature,
                         out_accept_len, f_scratch, out_tokens, workspace, workspace_bytes, out_accept_prob, nullptr,
                         out_status, (cudaStream_t)stream);
}

int sgbv_draw_tokens(const void *logits, int dtype, const float *uniforms, int N, int V, float temperature,
                     int32_t *out_token, double *out_logprob, int32_t *out_status, void *workspace, size_t workspace_bytes,
                     void *stream) {
    if (!logits || !uniforms || !out_token) return SGBV_ERR_NULL;
    int rc = check_shape(N, 1, 1, V, dtype);
    if (rc != SGBV_OK) return rc;
    if (!(temperature > 0.0f) || !isfinite(temperature)) return SGBV_ERR_TEMPERATURE;
    const size_t esz = dtype == SGBV_DTYPE_BF16 ? 2 : 4;
    if (((uintptr_t)logits % esz) || ((uintptr_t)uniforms % 4) || ((uintptr_t)out_token % 4) || ((uintptr_t)out_logprob % 8) ||
        ((uintptr_t)out_status % 4))
        return SGBV_ERR_ALIGN;
    const Shape s = make_shape(N, 1, 1, V, temperature);
    const Carve c = carve(s);
    unsigned char *base = nullptr;
    if (workspace) {
        if (workspace_bytes < c.total || ((uintptr_t)workspace % kAlign)) return SGBV_ERR_WORKSPACE;
        base = (unsigned char *)workspace;
    } else {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SGBV_ERR_CUDA;
        std::lock_guard<std::mutex> lock(g_mu);
        rc = grow(&g_buf[dev].scratch, &g_buf[dev].scratch_bytes, c.total, kRatioWords * sizeof(double));
        if (rc != SGBV_OK) return rc;
        base = (unsigned char *)g_buf[dev].scratch;
    }
    const int n = launch_draw_rows(logits, dtype, uniforms, s, (float *)(base + c.bonus), out_token, out_logprob, out_status,
                                   (cudaStream_t)stream);
    if (n < 0) return n;
    t_last_launches = n;
    t_last_kernel = "draw_rows_kernel";
    return SGBV_OK;
}

int sgbv_last_launch_count(void) { return t_last_launches; }

const char *sgbv_last_main_kernel(void) { return t_last_kernel; }

int sgbv_set_option(const char *name, int value) {
    if (!name) return SGBV_ERR_NULL;
    if (!strcmp(name, "path")) {
        if (value < 0 || value > 2) return SGBV_ERR_SHAPE;
        g_opt_path = value;
    } else if (!strcmp(name, "cluster")) {
        if (value < 0 || value > 16) return SGBV_ERR_SHAPE;
        g_opt_cluster = value;
    } else if (!strcmp(name, "max_clusters")) {
        if (value < 0) return SGBV_ERR_SHAPE;
        g_opt_max_clusters = value;
    } else if (!strcmp(name, "walk")) {
        if (value < 0 || value > 2) return SGBV_ERR_SHAPE;
        g_opt_walk = value;
    } else if (!strcmp(name, "poll_us")) {
        if (value < 0 || value > 1000000) return SGBV_ERR_SHAPE;
        g_opt_poll_us = value;
    } else if (!strcmp(name, "withhold")) {
        if (value < 0 || value > 1) return SGBV_ERR_SHAPE;
        g_opt_withhold = value;
    } else if (!strcmp(name, "aux")) {
        if (value < 0 || value > 2) return SGBV_ERR_SHAPE;
        g_opt_aux = value;
    } else {
        return SGBV_ERR_SHAPE;
    }
    fused_set_options(g_opt_cluster, g_opt_max_clusters, g_opt_walk, g_opt_poll_us, g_opt_withhold, g_opt_aux);
    return SGBV_OK;
}

// ---- allocation-free variant ---------------------------------------------------------------------
// Scratch for sgbv_verify_static: a fixed array inside the library's device image.  Every device
// that loads the library holds these bytes until the process exits.  In host code the name below
// is only a handle for the symbol, not a device address: the kernels get the address that
// cudaGetSymbolAddress returns for the current device.
static __device__ __align__(256) unsigned char g_static_scratch[SGBV_STATIC_SCRATCH_BYTES];

namespace {
void *g_static_ptr[kMaxDevices];  // resolved once per device, under g_mu
}

int sgbv_verify_static(const void *target_logits, const void *draft_logits, int dtype, const int32_t *draft_tokens,
                       const float *uniforms, int B, int K, int gamma, int V, float temperature,
                       int32_t *out_accept_len, int32_t *out_draft_idx, int32_t *out_tokens, double *out_h,
                       double *out_resmass, int32_t *out_status, void *stream) {
    int rc = check_shape(B, K, gamma, V, dtype);
    if (rc != SGBV_OK) return rc;
    const size_t need = carve(make_shape(B, K, gamma, V, 1.0f)).total;
    if (need > (size_t)SGBV_STATIC_SCRATCH_BYTES) return SGBV_ERR_WORKSPACE;  // shape exceeds the fixed scratch
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SGBV_ERR_CUDA;
    void *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_static_ptr[dev]) {  // first call on this device: look the symbol up with this device current
            void *p = nullptr;
            if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
                cudaGetLastError();
                return SGBV_ERR_CUDA;
            }
            g_static_ptr[dev] = p;
        }
        scratch = g_static_ptr[dev];
    }
    return verify_device(target_logits, draft_logits, dtype, draft_tokens, uniforms, B, K, gamma, V, temperature,
                         out_accept_len, out_draft_idx, out_tokens, scratch, (size_t)SGBV_STATIC_SCRATCH_BYTES, out_h,
                         out_resmass, out_status, (cudaStream_t)stream);
}

int sgbv_profile_begin(int max_records) {
    if (max_records < 1 || max_records > (1 << 20) || g_prof.capacity != 0) return SGBV_ERR_SHAPE;
    g_prof.begin = (cudaEvent_t *)calloc((size_t)max_records, sizeof(cudaEvent_t));
    g_prof.end = (cudaEvent_t *)calloc((size_t)max_records, sizeof(cudaEvent_t));
    if (!g_prof.begin || !g_prof.end) return SGBV_ERR_CUDA;
    for (int i = 0; i < max_records; ++i)
        if (cudaEventCreate(&g_prof.begin[i]) != cudaSuccess || cudaEventCreate(&g_prof.end[i]) != cudaSuccess)
            return SGBV_ERR_CUDA;
    g_prof.used = 0;
    g_prof.capacity = max_records;
    return SGBV_OK;
}

int sgbv_profile_end(double *out_total_ms, int *out_records) {
    if (!out_total_ms || !out_records) return SGBV_ERR_NULL;
    if (g_prof.capacity == 0) return SGBV_ERR_SHAPE;
    double total = 0.0;
    bool ok = true;
    for (int i = 0; i < g_prof.used; ++i) {
        float ms = 0.0f;
        ok &= cudaEventSynchronize(g_prof.end[i]) == cudaSuccess;
        ok &= cudaEventElapsedTime(&ms, g_prof.begin[i], g_prof.end[i]) == cudaSuccess;
        total += ms;
    }
    for (int i = 0; i < g_prof.capacity; ++i) {
        cudaEventDestroy(g_prof.begin[i]);
        cudaEventDestroy(g_prof.end[i]);
    }
    free(g_prof.begin);
    free(g_prof.end);
    *out_total_ms = total;
    *out_records = g_prof.used;
    g_prof = Profile();
    return ok ? SGBV_OK : SGBV_ERR_CUDA;
}

const char *sgbv_status_string(int code) {
    switch (code) {
        case SGBV_OK: return "SGBV_OK";
        case SGBV_ERR_NULL: return "SGBV_ERR_NULL: a required pointer is NULL";
        case SGBV_ERR_SHAPE: return "SGBV_ERR_SHAPE: B,K,gamma,V out of range or unknown dtype";
        case SGBV_ERR_TEMPERATURE: return "SGBV_ERR_TEMPERATURE: temperature must be finite and > 0";
        case SGBV_ERR_ALIGN: return "SGBV_ERR_ALIGN: pointer not aligned to its element size";
        case SGBV_ERR_WORKSPACE: return "SGBV_ERR_WORKSPACE: workspace too small or not 256-byte aligned";
        case SGBV_ERR_CUDA: return "SGBV_ERR_CUDA: a CUDA runtime call failed";
        default: return "SGBV: unknown code";
    }
}

}  // extern "C"
