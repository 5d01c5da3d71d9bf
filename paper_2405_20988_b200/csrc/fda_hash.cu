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

// The 16-bit hash table (bucket | sign << 15 per row and index) of the plain-load sketch kernels
// and of the mean-sketch pass: 2*l bytes per index of d_max, built by the first call that needs it
// (contexts that only ever use the list kernel never pay for it).
cudaError_t fda_ensure_table(fda_ctx *ctx, cudaStream_t s)
{
    if (ctx->l == 0 || ctx->tab) return cudaSuccess;
    uint16_t *tab = nullptr;
    cudaError_t e = cudaMalloc(&tab, sizeof(uint16_t) * (size_t)ctx->l * ctx->tab_stride);
    if (e != cudaSuccess) return e;
    const uint64_t magic = ~0ull / (uint64_t)ctx->m;
    dim3 grid(blocks_for(ctx->tab_stride, 256, ctx->n_sm * 16), (unsigned)ctx->l);
    k_build_table<<<grid, 256, 0, s>>>(ctx->coeffs_dev, ctx->l, (uint32_t)ctx->m, magic,
                                      ctx->tab_stride, ctx->tab_stride, tab);
    e = cudaGetLastError();
    if (e != cudaSuccess) { cudaFree(tab); return e; }
    ctx->tab = tab;
    return cudaSuccess;
}

cudaError_t fda_launch_debug_hash(const fda_ctx *ctx, int64_t j0, int64_t n, uint16_t *buckets,
                                  int8_t *signs, cudaStream_t s)
{
    const uint64_t magic = ~0ull / (uint64_t)ctx->m;
    dim3 grid(blocks_for(n, 256, ctx->n_sm * 16), (unsigned)ctx->l);
    k_debug_hash<<<grid, 256, 0, s>>>(ctx->coeffs_dev, (uint32_t)ctx->m, magic, j0, n, buckets, signs);
    return cudaGetLastError();
}
