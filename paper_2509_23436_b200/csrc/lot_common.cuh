// Device helpers shared by the liblot kernels (sm_100a).
//
// Arithmetic convention of every kernel here: potentials and logits are kept in
// base-2 log units, L = C * (log2(e)/eps), G = g * (log2(e)/eps), so that the
// exponentials are single ex2 instructions.  A column sum that may span hundreds of
// orders of magnitude is carried as a pair (kappa, S) meaning S * 2^kappa.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

// Bounds-check build (-DLOT_DEBUG): every checked global access states the extent of its buffer; an access outside it
// is skipped and recorded in a per-file device word that lot_device_status reports as LOT_DEV_BOUNDS.  Never a trap.
#ifdef LOT_DEBUG
static __device__ int g_lot_bounds_flag;
#define LOT_CHECK(cond) ((cond) ? true : (atomicOr(&g_lot_bounds_flag, 1), false))
#define LOT_DEBUG_FLAG_READER(name)                                                              \
    int name()                                                                                   \
    {                                                                                            \
        int v = 0, zero = 0;                                                                     \
        if (cudaMemcpyFromSymbol(&v, g_lot_bounds_flag, sizeof(int)) != cudaSuccess) return 0;   \
        (void)cudaMemcpyToSymbol(g_lot_bounds_flag, &zero, sizeof(int));                         \
        return v;                                                                                \
    }
#else
#define LOT_CHECK(cond) true
#define LOT_DEBUG_FLAG_READER(name) \
    int name() { return 0; }
#endif

namespace lot {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ float neg_inf() { return __int_as_float(0xff800000); }

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float lg2(float x)
{
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// (k1,s1) <- (k1,s1) (+) (k2,s2) for pairs meaning s * 2^k; an empty pair is (-inf, 0).
__device__ __forceinline__ void pair_merge(float &k1, float &s1, float k2, float s2)
{
    float k = fmaxf(k1, k2);
    if (k == neg_inf()) { s1 = 0.f; return; }
    s1 = s1 * ex2(k1 - k) + s2 * ex2(k2 - k);
    k1 = k;
}

// Add one term 2^y to the pair; rescales only when y exceeds the running reference by 2^20.
__device__ __forceinline__ void pair_add(float &k, float &s, float y)
{
    float dlt = y - k;
    if (dlt > 20.f) {
        s = s * ex2(k - y) + 1.f;
        k = y;
    } else {
        s += ex2(dlt);
    }
}

template <typename T> struct Elem;
template <> struct Elem<float> {
    static __device__ __forceinline__ float load(const float *p) { return __ldg(p); }
    static __device__ __forceinline__ void store(float *p, float v) { *p = v; }
};
template <> struct Elem<__nv_bfloat16> {
    static __device__ __forceinline__ float load(const __nv_bfloat16 *p)
    {
        return __bfloat162float(*p);
    }
    static __device__ __forceinline__ void store(__nv_bfloat16 *p, float v)
    {
        *p = __float2bfloat16_rn(v);
    }
};

// 4 consecutive elements -> 4 floats (pointer 4-element aligned)
__device__ __forceinline__ void load4(const float *p, float (&o)[4])
{
    float4 t = __ldg(reinterpret_cast<const float4 *>(p));
    o[0] = t.x; o[1] = t.y; o[2] = t.z; o[3] = t.w;
}
__device__ __forceinline__ void load4(const __nv_bfloat16 *p, float (&o)[4])
{
    uint2 t = __ldg(reinterpret_cast<const uint2 *>(p));
    o[0] = __uint_as_float(t.x << 16);
    o[1] = __uint_as_float(t.x & 0xffff0000u);
    o[2] = __uint_as_float(t.y << 16);
    o[3] = __uint_as_float(t.y & 0xffff0000u);
}
__device__ __forceinline__ void store4(float *p, const float (&v)[4])
{
    *reinterpret_cast<float4 *>(p) = make_float4(v[0], v[1], v[2], v[3]);
}
__device__ __forceinline__ void store4(__nv_bfloat16 *p, const float (&v)[4])
{
    __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]);
    __nv_bfloat162 b = __floats2bfloat162_rn(v[2], v[3]);
    uint2 t;
    t.x = *reinterpret_cast<uint32_t *>(&a);
    t.y = *reinterpret_cast<uint32_t *>(&b);
    *reinterpret_cast<uint2 *>(p) = t;
}

} // namespace lot
