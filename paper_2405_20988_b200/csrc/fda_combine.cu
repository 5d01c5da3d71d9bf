// Combine step: average state, row norms of the averaged sketch, median, H, trigger
// (Algorithm 1: the state average and the variance test; Theorem 1 for SketchFDA, Theorem 2 for LinearFDA).
//
// One block per sketch row plus one for the two scalar entries, so that the K x (2 + l*m) reads
// of a large state table are spread over several SMs; the block that finishes last (a ticket
// counter, no waiting) takes the median and writes the estimate.  fp64 accumulation in a fixed
// order, so the result is reproducible.
#include "fda_internal.h"

namespace {

constexpr int kCombineThreads = 1024;

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

// scratch (device, owned by the context): [0..1] S-bar[0..1], [2 .. 2+l) row norms; *ticket is 0
// between launches.
__global__ void __launch_bounds__(kCombineThreads, 1)
k_combine(const float *__restrict__ states, int K, int l, int m, int cw /* pow2 >= min(m, threads) */,
          int variant, float epsilon, float theta, double *scratch_out, unsigned int *ticket,
          fda_estimate *__restrict__ est)
{
    __shared__ double scratch[32];
    __shared__ double part_s[kCombineThreads];
    __shared__ bool last_s;
    const size_t slen = 2 + (size_t)l * (size_t)m;
    const double inv_k = 1.0 / (double)K;
    const int tid = threadIdx.x;
    const int i = blockIdx.x;              // sketch row; block l handles the two scalars

    if (i == l) {
        if (tid < 2) {                     // S-bar[0] and S-bar[1]
            double acc = 0.0;
            for (int k = 0; k < K; ++k) acc += (double)states[(size_t)k * slen + tid];
            scratch_out[tid] = acc * inv_k;
            __threadfence();
        }
    } else {                               // ||row i of the averaged sketch||^2
        // thread (kp, cl): workers kp, kp + ks, ... of column c0 + cl; then the ks partial sums
        // of a column are added in order
        const int ks = blockDim.x / cw, cl = tid % cw, kp = tid / cw;
        double part = 0.0;
        for (int c0 = 0; c0 < m; c0 += cw) {
            const int c = c0 + cl;
            double acc = 0.0;
            if (c < m && kp < ks) {
                const float *col = states + 2 + (size_t)i * m + c;
                int k = kp;
                for (; k + 3 * ks < K; k += 4 * ks) {
                    const float v0 = col[(size_t)k * slen], v1 = col[(size_t)(k + ks) * slen],
                                v2 = col[(size_t)(k + 2 * ks) * slen], v3 = col[(size_t)(k + 3 * ks) * slen];
                    acc += (double)v0; acc += (double)v1; acc += (double)v2; acc += (double)v3;
                }
                for (; k < K; k += ks) acc += (double)col[(size_t)k * slen];
            }
            __syncthreads();               // part_s of the previous chunk has been read
            part_s[tid] = acc;
            __syncthreads();
            if (kp == 0 && c < m) {
                double t = 0.0;
                for (int q = 0; q < ks; ++q) t += part_s[q * cw + cl];
                t *= inv_k;
                part += t * t;
            }
        }
        const double r = block_sum(part, scratch);
        if (tid == 0) scratch_out[2 + i] = r;
    }

    // ---- the last block to arrive finishes the estimate ----
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const unsigned int t = atomicAdd(ticket, 1u);
        last_s = (t == gridDim.x - 1);
    }
    __syncthreads();
    if (!last_s || tid != 0) return;
    __threadfence();
    const volatile double *res = scratch_out;
    double rows[FDA_MAX_ROWS];
    for (int r = 0; r < l; ++r) rows[r] = res[2 + r];
    const double head0 = res[0], head1 = res[1];
    double est_sq;
    if (variant == FDA_VARIANT_SKETCH) {
        double srt[FDA_MAX_ROWS];
        for (int r = 0; r < l; ++r) {              // insertion sort, l <= 16
            double v = rows[r];
            int q = r;
            while (q > 0 && srt[q - 1] > v) { srt[q] = srt[q - 1]; --q; }
            srt[q] = v;
        }
        const double med = (l & 1) ? srt[l / 2] : 0.5 * (srt[l / 2 - 1] + srt[l / 2]);
        est_sq = med / (1.0 + (double)epsilon);
    } else {
        est_sq = head1 * head1;
    }
    const double H = head0 - est_sq;
    est->mean_sq_norm = (float)head0;
    est->est_sq_norm_of_mean = (float)est_sq;
    est->H = (float)H;
    est->theta = theta;
    est->trigger = (H > (double)theta) ? 1 : 0;    // decided in fp64, strict '>'
    est->l = l;
    for (int r = 0; r < FDA_MAX_ROWS; ++r) est->row_sq_norm[r] = r < l ? (float)rows[r] : 0.f;
    *ticket = 0u;                                  // ready for the next launch on this context
}

}  // namespace

cudaError_t fda_launch_combine(const fda_ctx *ctx, const float *states, int K, int variant,
                               float epsilon, float theta, fda_estimate *est_dev, cudaStream_t s)
{
    // columns per pass: the power of two that covers m (at most the block); the other threads
    // of the block split the workers
    int cw = 32;
    while (cw < ctx->m && cw < kCombineThreads) cw <<= 1;
    int threads = cw;
    while (threads < kCombineThreads && threads / cw < (K + 7) / 8) threads <<= 1;
    k_combine<<<ctx->l + 1, threads, 0, s>>>(states, K, ctx->l, ctx->m, cw, variant, epsilon, theta,
                                            ctx->combine_scratch, ctx->combine_ticket, est_dev);
    return cudaGetLastError();
}
