// Pieces shared by the two kernels that walk the list schedule (fda_sched.cu): the per-worker
// sketch pass (fda_local_state_gather.cu) and the averaged state (fda_mean_state_gather.cu).
#ifndef FDA_LIST_KERNEL_CUH_
#define FDA_LIST_KERNEL_CUH_

#include "fda_internal.h"

namespace fda_list {

constexpr int GW = kListWorkers;
constexpr int kChunksAhead = 8;                // entry chunks (four steps each) the walkers of the averaged state load ahead (sketches below 7 rows)
constexpr int kMaxProducerWarps = 16;          // the fp64 sums in shared memory have room for that many

struct ListParams {
    const float *w, *w_t0, *xi;
    int64_t row_stride;
    int K;
    int64_t d;
    int have_xi;
    int vec;                         // 16-byte aligned inputs: the producers load 128 bits at a time
    int l, m;
    int groups, cpg;                 // block = c * groups + g
    int T, nb;                       // indices and batches per tile
    int64_t tiles;                   // tiles that hold indices below d
    int tab_bytes;                   // bytes of one item-table buffer in shared memory
    const unsigned char *sched;
    const uint64_t *sched_off;
    float *part_sk;                  // [block][cell][GW]
    double *part_np;                 // [block][GW][2]
};

template <int THREADS>
__device__ __forceinline__ void block_barrier()
{
    asm volatile("bar.sync 1, %0;" ::"n"(THREADS) : "memory");
}

// Loads and stores of the producers as volatile statements: the compiler keeps them in program
// order, so a batch's loads are issued kDepth batches before its values are used.
__device__ __forceinline__ float4 load4_stream(const float *ptr)
{
    float4 v;
    asm volatile("ld.global.cs.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(ptr));
    return v;
}
__device__ __forceinline__ float4 load4_keep(const float *ptr)
{
    float4 v;
    asm volatile("ld.global.nc.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(ptr));
    return v;
}
__device__ __forceinline__ float load1(const float *ptr, bool on)
{
    float v;
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %2, 0;\n\tmov.b32 %0, 0;\n\t@p ld.global.f32 %0, [%1];\n\t}"
                 : "=f"(v) : "l"(ptr), "r"((int)on));
    return v;
}
// four floats from ptr: one 128-bit load when `vec` (aligned, all four below the end), else the
// `n` valid ones with 32-bit loads and zeros behind them
template <bool STREAM>
__device__ __forceinline__ float4 load_quad(const float *ptr, bool vec, int n)
{
    if (vec) return STREAM ? load4_stream(ptr) : load4_keep(ptr);
    float4 v;
    v.x = load1(ptr, n > 0); v.y = load1(ptr + 1, n > 1); v.z = load1(ptr + 2, n > 2); v.w = load1(ptr + 3, n > 3);
    return v;
}
__device__ __forceinline__ uint4 load_u4(const void *ptr)
{
    uint4 v;
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(ptr));
    return v;
}
__device__ __forceinline__ unsigned long long load_u64(const void *ptr)
{
    unsigned long long v;
    asm volatile("ld.global.nc.u64 %0, [%1];" : "=l"(v) : "l"(ptr));
    return v;
}
__device__ __forceinline__ void store_row(uint32_t addr, float x, float y, float z, float w)
{
    asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "f"(x), "f"(y), "f"(z), "f"(w) : "memory");
}
__device__ __forceinline__ float comp(const float4 &v, int q) { return q == 0 ? v.x : (q == 1 ? v.y : (q == 2 ? v.z : v.w)); }

// One schedule entry: gather the row (four workers) and add it with the entry's sign.  The
// sums stay packed as fp32 pairs, the sign is a multiplication by (+-1, +-1) (exact).
__device__ __forceinline__ void gather_row(uint32_t row_off, uint32_t sign_one, uint32_t base,
                                           unsigned long long &a01, unsigned long long &a23)
{
    unsigned long long u0, u1, ss;
    asm volatile("ld.shared.v2.b64 {%0,%1}, [%2];" : "=l"(u0), "=l"(u1) : "r"(base + row_off));
    asm("mov.b64 %0, {%1,%1};" : "=l"(ss) : "r"(sign_one));
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(a01) : "l"(u0), "l"(ss));
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(a23) : "l"(u1), "l"(ss));
}
// low / high half of a 32-bit word holding two entries (bits 0..12 row, bit 15 sign)
__device__ __forceinline__ void gather_lo(uint32_t w, uint32_t base, unsigned long long &a01, unsigned long long &a23)
{
    gather_row((w & 0x1fffu) << 4, ((w << 16) & 0x80000000u) ^ 0x3f800000u, base, a01, a23);
}
__device__ __forceinline__ void gather_hi(uint32_t w, uint32_t base, unsigned long long &a01, unsigned long long &a23)
{
    gather_row((w >> 12) & 0x1fff0u, (w & 0x80000000u) ^ 0x3f800000u, base, a01, a23);
}

}  // namespace fda_list

#endif
