// K-way model average (Section 3: the workers synchronise with an AllReduce of their models,
// the synchronisation step of Algorithm 1): w-bar = (1/K) sum_k w^(k), written to w_t0 and, when broadcasting, to every row.
// Bandwidth-bound streaming kernel; the whole launch is predicated on the trigger word of
// the device-side estimate so that no host round trip is needed between the two calls.
#include "fda_internal.h"

namespace {

constexpr int kBatch = 8;   // rows loaded before they are summed (loads in flight per thread)

// XI: also write the unnormalised direction of the global step, delta = w-bar_new - w_t0_old, to
// xi_out and the block's partial of ||delta||^2 to part (Section 3.2: xi is the normalised
// difference of the models of the last two synchronisations).
template <bool VEC, bool XI>
__global__ void __launch_bounds__(256)
k_average(float *w, int64_t row_stride, int K, int64_t d, float *__restrict__ w_t0,
          const fda_estimate *est, int broadcast, float *__restrict__ xi_out, double *__restrict__ part)
{
    if (est != nullptr && est->trigger == 0) return;
    double dsq = 0.0;
    const float inv_k = 1.0f / (float)K;
    const int64_t nthreads = (int64_t)gridDim.x * blockDim.x;
    const int64_t t0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (VEC) {
        const int64_t nq = d / 4;
        for (int64_t q = t0; q < nq; q += nthreads) {
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int k0 = 0; k0 < K; k0 += kBatch) {
                float4 v[kBatch];
#pragma unroll
                for (int b = 0; b < kBatch; ++b)
                    if (k0 + b < K)
                        v[b] = __ldcs(reinterpret_cast<const float4 *>(w + (size_t)(k0 + b) * row_stride + q * 4));
#pragma unroll
                for (int b = 0; b < kBatch; ++b)
                    if (k0 + b < K) { acc.x += v[b].x; acc.y += v[b].y; acc.z += v[b].z; acc.w += v[b].w; }
            }
            acc.x *= inv_k; acc.y *= inv_k; acc.z *= inv_k; acc.w *= inv_k;
            if (XI) {
                const float4 old = *reinterpret_cast<const float4 *>(w_t0 + q * 4);
                const float4 dl = make_float4(acc.x - old.x, acc.y - old.y, acc.z - old.z, acc.w - old.w);
                *reinterpret_cast<float4 *>(xi_out + q * 4) = dl;
                dsq += (double)(dl.x * dl.x + dl.y * dl.y + dl.z * dl.z + dl.w * dl.w);
            }
            __stcs(reinterpret_cast<float4 *>(w_t0 + q * 4), acc);
            if (broadcast)
                for (int k = 0; k < K; ++k)
                    __stcs(reinterpret_cast<float4 *>(w + (size_t)k * row_stride + q * 4), acc);
        }
    }
    // scalar path: everything when !VEC, the d % 4 tail otherwise
    const int64_t begin = VEC ? (d / 4) * 4 : 0;
    for (int64_t j = begin + t0; j < d; j += nthreads) {
        float acc = 0.f;
        for (int k = 0; k < K; ++k) acc += w[(size_t)k * row_stride + j];
        acc *= inv_k;
        if (XI) {
            const float dl = acc - w_t0[j];
            xi_out[j] = dl;
            dsq += (double)(dl * dl);
        }
        w_t0[j] = acc;
        if (broadcast)
            for (int k = 0; k < K; ++k) w[(size_t)k * row_stride + j] = acc;
    }
    if (XI) {      // block partial of ||delta||^2, fixed order
        __shared__ double red[8];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) dsq += __shfl_xor_sync(0xffffffffu, dsq, off);
        if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = dsq;
        __syncthreads();
        if (threadIdx.x == 0) {
            double t = 0.0;
            for (int wv = 0; wv < 8; ++wv) t += red[wv];
            part[blockIdx.x] = t;
        }
    }
}

// xi_out *= 1 / ||delta||  (0 when the step is zero); gated like the average itself
__global__ void __launch_bounds__(256)
k_scale_xi(float *__restrict__ xi_out, int64_t d, const double *__restrict__ part, int nparts,
           const fda_estimate *est)
{
    if (est != nullptr && est->trigger == 0) return;
    __shared__ float scale_s;
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int b = 0; b < nparts; ++b) t += part[b];
        scale_s = t > 0.0 ? (float)(1.0 / sqrt(t)) : 0.f;
    }
    __syncthreads();
    const float scale = scale_s;
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < d; j += (int64_t)gridDim.x * blockDim.x)
        xi_out[j] *= scale;
}

}  // namespace

cudaError_t fda_launch_average(const fda_ctx *ctx, float *w, int64_t row_stride, int K, int64_t d,
                               float *w_t0, float *xi_out, const fda_estimate *est_dev, uint32_t flags,
                               cudaStream_t s)
{
    const bool vec = ((((uintptr_t)w | (uintptr_t)w_t0 | (uintptr_t)xi_out) & 15u) == 0) && (row_stride % 4 == 0);
    const fda_estimate *gate = (flags & FDA_AVG_UNCONDITIONAL) ? nullptr : est_dev;
    const int broadcast = (flags & FDA_AVG_BROADCAST) ? 1 : 0;
    const int threads = 256;
    int64_t work = vec ? (d + 3) / 4 : d;
    int64_t blocks = (work + threads - 1) / threads;
    const int64_t cap = (int64_t)ctx->n_sm * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    if (xi_out) {
        if (vec) k_average<true, true><<<(unsigned)blocks, threads, 0, s>>>(w, row_stride, K, d, w_t0, gate, broadcast, xi_out, ctx->part_np);
        else     k_average<false, true><<<(unsigned)blocks, threads, 0, s>>>(w, row_stride, K, d, w_t0, gate, broadcast, xi_out, ctx->part_np);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        k_scale_xi<<<(unsigned)blocks, threads, 0, s>>>(xi_out, d, ctx->part_np, (int)blocks, gate);
        return cudaGetLastError();
    }
    if (vec) k_average<true, false><<<(unsigned)blocks, threads, 0, s>>>(w, row_stride, K, d, w_t0, gate, broadcast, nullptr, nullptr);
    else     k_average<false, false><<<(unsigned)blocks, threads, 0, s>>>(w, row_stride, K, d, w_t0, gate, broadcast, nullptr, nullptr);
    return cudaGetLastError();
}
