// Combine step: average state, row norms of the averaged sketch, median, H, trigger
// (Algorithm 1 lines 7-8; Theorem 1 for SketchFDA, Theorem 2 for LinearFDA).
// One block; fp64 accumulation in a fixed order, so the result is reproducible.
#include "fda_internal.h"

namespace {

__device__ double block_sum(double v, double *scratch)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_down_sync(0xffffffffu, v, off);
    __syncthreads();                       // scratch may still be read from the last call
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    double t = 0.0;
    if (threadIdx.x == 0)
        for (int wv = 0; wv < nwarps; ++wv) t += scratch[wv];
    return t;                              // valid in thread 0
}

__global__ void __launch_bounds__(1024, 1)
k_combine(const float *__restrict__ states, int K, int l, int m, int variant, float epsilon,
          float theta, fda_estimate *__restrict__ est)
{
    __shared__ double scratch[32];
    __shared__ double rows[FDA_MAX_ROWS];
    __shared__ double head[2];
    const size_t slen = 2 + (size_t)l * (size_t)m;
    const double inv_k = 1.0 / (double)K;

    if (threadIdx.x < 2) {                 // S-bar[0] and S-bar[1]
        double acc = 0.0;
        for (int k = 0; k < K; ++k) acc += (double)states[(size_t)k * slen + threadIdx.x];
        head[threadIdx.x] = acc / (double)K;
    }
    for (int i = 0; i < l; ++i) {          // ||row i of the averaged sketch||^2
        double part = 0.0;
        for (int c = threadIdx.x; c < m; c += blockDim.x) {
            double acc = 0.0;
            const float *col = states + 2 + (size_t)i * m + c;
#pragma unroll 4
            for (int k = 0; k < K; ++k) acc += (double)col[(size_t)k * slen];
            acc *= inv_k;
            part += acc * acc;
        }
        const double r = block_sum(part, scratch);
        if (threadIdx.x == 0) rows[i] = r;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        double est_sq;
        if (variant == FDA_VARIANT_SKETCH) {
            double srt[FDA_MAX_ROWS];
            for (int i = 0; i < l; ++i) {          // insertion sort, l <= 16
                double v = rows[i];
                int q = i;
                while (q > 0 && srt[q - 1] > v) { srt[q] = srt[q - 1]; --q; }
                srt[q] = v;
            }
            const double med = (l & 1) ? srt[l / 2] : 0.5 * (srt[l / 2 - 1] + srt[l / 2]);
            est_sq = med / (1.0 + (double)epsilon);
        } else {
            est_sq = head[1] * head[1];
        }
        const double H = head[0] - est_sq;
        est->mean_sq_norm = (float)head[0];
        est->est_sq_norm_of_mean = (float)est_sq;
        est->H = (float)H;
        est->theta = theta;
        est->trigger = (H > (double)theta) ? 1 : 0;    // decided in fp64, strict '>'
        est->l = l;
        for (int i = 0; i < FDA_MAX_ROWS; ++i) est->row_sq_norm[i] = i < l ? (float)rows[i] : 0.f;
    }
}

}  // namespace

cudaError_t fda_launch_combine(const fda_ctx *ctx, const float *states, int K, int variant,
                               float epsilon, float theta, fda_estimate *est_dev, cudaStream_t s)
{
    int threads = 32;
    while (threads < ctx->m && threads < 1024) threads <<= 1;
    k_combine<<<1, threads, 0, s>>>(states, K, ctx->l, ctx->m, variant, epsilon, theta, est_dev);
    return cudaGetLastError();
}
