// Device helpers shared by the tensor-core kernels (sm_100a): packed-bf16 tile access in tensor memory, the quad
// layout of accumulator loads, tagged 64-bit words for exchanges through global memory, column reductions.
#pragma once

#include "lot_common.cuh"
#include "lot_sm100.cuh"

namespace lot {
namespace tile {

using namespace sm100;

__device__ __forceinline__ uint32_t pack_bf16(float a, float b)
{
    __nv_bfloat162 t = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&t);
}
__device__ __forceinline__ float2 unpack_bf16(uint32_t w)
{
    return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
__device__ __forceinline__ float max3(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ void st_tagged2(unsigned long long *p, float a, float b, unsigned tag)
{
    const unsigned long long w0 = ((unsigned long long)tag << 32) | __float_as_uint(a);
    const unsigned long long w1 = ((unsigned long long)tag << 32) | __float_as_uint(b);
    asm volatile("st.relaxed.gpu.global.v2.b64 [%0], {%1, %2};" ::"l"(p), "l"(w0), "l"(w1) : "memory");
}
__device__ __forceinline__ void ld_tagged2(const unsigned long long *p, unsigned long long &w0, unsigned long long &w1)
{
    asm volatile("ld.relaxed.gpu.global.v2.b64 {%0, %1}, [%2];" : "=l"(w0), "=l"(w1) : "l"(p) : "memory");
}
__device__ __forceinline__ unsigned long long ld_acquire64(const unsigned long long *p)
{
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release64(unsigned long long *p, unsigned long long v)
{
    asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait_group_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}

// Packed tile access, 16 lanes x (4 X) 32-bit columns: thread L of the warp holds, in r[2 rep + k], lane L/4 + 8 k and
// column 4 rep + L % 4 of the 16-lane block at taddr.  With two bf16 per column this is the quad layout of the
// accumulator loads below (rows in lane quads, entry pair (8 rep + 2 (L % 4), + 1)).
template <int X>
__device__ __forceinline__ void tmem_ld_pk(uint32_t taddr, uint32_t *r)
{
    if constexpr (X == 8) {
        asm volatile("tcgen05.ld.sync.aligned.16x128b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                     : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                       "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                     : "r"(taddr) : "memory");
    } else if constexpr (X == 4) {
        asm volatile("tcgen05.ld.sync.aligned.16x128b.x4.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                     : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                     : "r"(taddr) : "memory");
    } else {
        static_assert(X == 2, "repeat count");
        asm volatile("tcgen05.ld.sync.aligned.16x128b.x2.b32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(taddr) : "memory");
    }
}
template <int X>
__device__ __forceinline__ void tmem_st_pk(uint32_t taddr, const uint32_t *r)
{
    if constexpr (X == 8) {
        asm volatile("tcgen05.st.sync.aligned.16x128b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
                     ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                       "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]) : "memory");
    } else if constexpr (X == 4) {
        asm volatile("tcgen05.st.sync.aligned.16x128b.x4.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                     ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]) : "memory");
    } else {
        static_assert(X == 2, "repeat count");
        asm volatile("tcgen05.st.sync.aligned.16x128b.x2.b32 [%0], {%1, %2, %3, %4};"
                     ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
    }
}
// Accumulator load, quad layout (16 lanes x 8 X float columns): v[4 rep + k] = lane L/4 + 8 (k/2), column
// 8 rep + 2 (L % 4) + k % 2.
template <int X>
__device__ __forceinline__ void tmem_ld_acc(uint32_t taddr, float *v)
{
    uint32_t *r = reinterpret_cast<uint32_t *>(v);
    if constexpr (X == 8) {
        asm volatile("tcgen05.ld.sync.aligned.16x256b.x8.b32 "
                     "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                     "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                     : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                       "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                       "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                       "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                     : "r"(taddr) : "memory");
    } else if constexpr (X == 4) {
        asm volatile("tcgen05.ld.sync.aligned.16x256b.x4.b32 "
                     "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                     : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                       "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                     : "r"(taddr) : "memory");
    } else {
        static_assert(X == 2, "repeat count");
        asm volatile("tcgen05.ld.sync.aligned.16x256b.x2.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                     : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                     : "r"(taddr) : "memory");
    }
}

// Sum a[0..N-1] over the 8 lanes that share (lane & 3), halving the live set while it is longer than two.  Afterwards
// every lane holds in a[0], a[1] the totals of entries b, b + 1; b is returned.  For N < 16 several lanes end with the
// same pair; `owner` tells the caller which of them writes it out.
template <int N>
__device__ __forceinline__ int quad_col_reduce(float (&a)[N], int lane, bool &owner)
{
    static_assert(N == 16 || N == 8 || N == 4, "entries per thread");
    int b = 0;
    owner = true;
    if constexpr (N >= 16) {
        const bool up = (lane & 16) != 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float send = up ? a[j] : a[j + 8], keep = up ? a[j + 8] : a[j];
            a[j] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
        }
        b += up ? 8 : 0;
    } else {
#pragma unroll
        for (int j = 0; j < N; ++j) a[j] += __shfl_xor_sync(0xffffffffu, a[j], 16);
        owner = owner && (lane & 16) == 0;
    }
    if constexpr (N >= 8) {
        const bool up = (lane & 8) != 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float send = up ? a[j] : a[j + 4], keep = up ? a[j + 4] : a[j];
            a[j] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
        }
        b += up ? 4 : 0;
    } else {
#pragma unroll
        for (int j = 0; j < N; ++j) a[j] += __shfl_xor_sync(0xffffffffu, a[j], 8);
        owner = owner && (lane & 8) == 0;
    }
    {
        const bool up = (lane & 4) != 0;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const float send = up ? a[j] : a[j + 2], keep = up ? a[j + 2] : a[j];
            a[j] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
        }
        b += up ? 2 : 0;
    }
    return b;
}


} // namespace tile
} // namespace lot
