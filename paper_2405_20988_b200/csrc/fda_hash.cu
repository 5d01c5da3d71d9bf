// Hash-table builder and hash dump kernels.
#include "fda_hash.cuh"
#include "fda_internal.h"

namespace {

// One thread per (index, row): tab[i*tab_stride + j] = bucket | sign bit, for j < n.
__global__ void k_build_table(const uint64_t *__restrict__ coeffs, int l, uint32_t m, uint64_t magic,
                              int64_t n, int64_t tab_stride, uint16_t *__restrict__ tab)
{
    const int i = blockIdx.y;
    const uint64_t c[6] = {coeffs[6 * i + 0], coeffs[6 * i + 1], coeffs[6 * i + 2],
                           coeffs[6 * i + 3], coeffs[6 * i + 4], coeffs[6 * i + 5]};
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < n;
         j += (int64_t)gridDim.x * blockDim.x) {
        const uint32_t b = fda::bucket_of(c, (uint32_t)j, m, magic);
        const uint32_t s = fda::sign_is_negative(c, (uint32_t)j) ? FDA_TAB_SIGN_BIT : 0u;
        tab[(size_t)i * tab_stride + j] = (uint16_t)(b | s);
    }
    (void)l;
}

// 32-bit variant for the staged sketch kernel: bits 0..23 hold the cell i*m + bucket, bit 31 is
// set when the sign is -1.  The kernel's bins are bins[cell][32] floats, so one shift-and-add
// (the shift by 7 drops the sign bit) gives the address and one AND-XOR the signed value.
__global__ void k_build_table32(const uint64_t *__restrict__ coeffs, uint32_t m, uint64_t magic, int64_t n,
                                int64_t tab_stride, uint32_t *__restrict__ tab)
{
    const int i = blockIdx.y;
    const uint64_t c[6] = {coeffs[6 * i + 0], coeffs[6 * i + 1], coeffs[6 * i + 2],
                           coeffs[6 * i + 3], coeffs[6 * i + 4], coeffs[6 * i + 5]};
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < n;
         j += (int64_t)gridDim.x * blockDim.x) {
        const uint32_t b = fda::bucket_of(c, (uint32_t)j, m, magic);
        const uint32_t s = fda::sign_is_negative(c, (uint32_t)j) ? 0x80000000u : 0u;
        tab[(size_t)i * tab_stride + j] = ((uint32_t)i * m + b) | s;
    }
}

__global__ void k_debug_hash(const uint64_t *__restrict__ coeffs, uint32_t m, uint64_t magic,
                             int64_t j0, int64_t n, uint16_t *__restrict__ buckets,
                             int8_t *__restrict__ signs)
{
    const int i = blockIdx.y;
    const uint64_t c[6] = {coeffs[6 * i + 0], coeffs[6 * i + 1], coeffs[6 * i + 2],
                           coeffs[6 * i + 3], coeffs[6 * i + 4], coeffs[6 * i + 5]};
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < n;
         t += (int64_t)gridDim.x * blockDim.x) {
        const uint32_t j = (uint32_t)(j0 + t);
        buckets[(size_t)i * n + t] = (uint16_t)fda::bucket_of(c, j, m, magic);
        signs[(size_t)i * n + t] = fda::sign_is_negative(c, j) ? (int8_t)-1 : (int8_t)1;
    }
}

inline unsigned blocks_for(int64_t n, int threads, int cap)
{
    int64_t b = (n + threads - 1) / threads;
    if (b > cap) b = cap;
    if (b < 1) b = 1;
    return (unsigned)b;
}

}  // namespace

cudaError_t fda_launch_build_table(const fda_ctx *ctx, cudaStream_t s)
{
    if (ctx->l == 0) return cudaSuccess;
    const uint64_t magic = ~0ull / (uint64_t)ctx->m;
    dim3 grid(blocks_for(ctx->tab_stride, 256, ctx->n_sm * 16), (unsigned)ctx->l);
    k_build_table<<<grid, 256, 0, s>>>(ctx->coeffs_dev, ctx->l, (uint32_t)ctx->m, magic,
                                      ctx->tab_stride, ctx->tab_stride, ctx->tab);
    if (ctx->tab32) {
        dim3 grid32(blocks_for(ctx->tab32_stride, 256, ctx->n_sm * 16), (unsigned)ctx->l);
        k_build_table32<<<grid32, 256, 0, s>>>(ctx->coeffs_dev, (uint32_t)ctx->m, magic, ctx->tab32_stride,
                                              ctx->tab32_stride, ctx->tab32);
    }
    return cudaGetLastError();
}

cudaError_t fda_launch_debug_hash(const fda_ctx *ctx, int64_t j0, int64_t n, uint16_t *buckets,
                                  int8_t *signs, cudaStream_t s)
{
    const uint64_t magic = ~0ull / (uint64_t)ctx->m;
    dim3 grid(blocks_for(n, 256, ctx->n_sm * 16), (unsigned)ctx->l);
    k_debug_hash<<<grid, 256, 0, s>>>(ctx->coeffs_dev, (uint32_t)ctx->m, magic, j0, n, buckets, signs);
    return cudaGetLastError();
}
