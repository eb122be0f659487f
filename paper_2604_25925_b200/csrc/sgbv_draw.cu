// Draft-token draw (Algorithm 3, the step that samples the K draft blocks): one token per logit row from
// softmax(z/T) by inverse CDF, softmax and draw fused in one pass over the row (per-tile maxima and sums, the
// tile located through them, one tile recomputed).  One CTA per row.
#include "sgbv_sample.cuh"

namespace sgbv {

namespace {

template <typename T>
__global__ void __launch_bounds__(1024)
draw_rows_kernel(const T *__restrict__ z_all, const float *__restrict__ u, Shape s, float *__restrict__ tile_scratch,
                 int32_t *__restrict__ out_token, double *__restrict__ out_logp, int32_t *__restrict__ out_status) {
    __shared__ SampleScratch sc;
    const int r = blockIdx.x;
    const T *z = z_all + (size_t)r * s.V;
    float *tile_s = tile_scratch + (size_t)r * 2 * s.ntiles;
    bool bad = false;
    float m = 0.0f;
    const int y = draw_from_row<T>(z, s, (double)u[r], tile_s, tile_s + s.ntiles, &sc, bad, &m);
    if (threadIdx.x == 0) {
        out_token[r] = y;
        if (out_status) out_status[r] = bad ? SGBV_STATUS_NONFINITE_LOGIT : 0;
    }
    if (out_logp) {
        // log softmax of the drawn token: the tile sums and factors that the draw left behind add up to the row's sum
        // of exponentials relative to its maximum
        double local = 0.0;
        if (!bad)
            for (int t = threadIdx.x; t < s.ntiles; t += blockDim.x) local += (double)tile_s[t] * (double)tile_s[s.ntiles + t];
        const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
        local = warp_sum(local);
        __syncthreads();
        if (lane == 0) sc.warp[wid] = local;
        __syncthreads();
        const double Z = warp_sum(lane < nwarps ? sc.warp[lane] : 0.0);
        if (threadIdx.x == 0) out_logp[r] = bad ? NAN : ((double)ld_logit(z, y) - (double)m) * s.inv_T - log(Z);
    }
}

}  // namespace

int launch_draw_rows(const void *z, int dtype, const float *u, const Shape &s, float *tile_scratch, int32_t *out_token,
                     double *out_logp, int32_t *out_status, cudaStream_t stream) {
    if (dtype == SGBV_DTYPE_BF16)
        draw_rows_kernel<uint16_t><<<s.B, 1024, 0, stream>>>((const uint16_t *)z, u, s, tile_scratch, out_token, out_logp,
                                                             out_status);
    else
        draw_rows_kernel<float><<<s.B, 1024, 0, stream>>>((const float *)z, u, s, tile_scratch, out_token, out_logp, out_status);
    return cudaGetLastError() == cudaSuccess ? 1 : SGBV_ERR_CUDA;
}

}  // namespace sgbv
