// The two apply stages of Eq. (4) from the stored Gibbs kernel (bf16 tensors, d = 64, 32 < r <= 64), as two
// kernels launched behind the persistent Sinkhorn kernel (lot_fused.cu) on the same stream:
//
//   apply_w_kernel    W = Gamma2 V per slice.  With K~2_jt = 2^(L_jt - max_t L_jt) stored as bf16 (workspace, L2) and
//                     w_t = 2^(G2_t - max G2):  W_t = w_t sum_j K~2_jt (v_j / s_j) / kv,  s_j = sum_t K~2_jt w_t.  The
//                     stored tile is the A operand as it is (MN-major, no rewrite); the value rows are scaled by 1/s_j
//                     and split into bf16 hi + lo in shared memory.  Every block writes the partial of its tile range.
//   apply_out_kernel  out_i = sum_t K~1_it (w1_t W'_t) / s_i,  W' = W / beta.  The stored query tile is the A operand
//                     straight from TMA; W'' = Diag(w1) W' (partials added in slot order) is the B operand, hi + lo.
//
// Neither kernel recomputes a logit or an exponential, and neither waits for another block: the kernel boundary is the
// grid barrier.  Slices whose stored kernel cannot carry the final potentials (decision word 2) were applied by the
// Sinkhorn kernel itself and are skipped here.  Four tiles are in flight per block (TMA ring, one accumulator per ring
// stage in the output kernel), so the tensor-core latency of one tile overlaps the CUDA-core work on its neighbours.
#include "lot_common.cuh"
#include "lot_internal.h"
#include "lot_sm100.cuh"
#include "lot_tile.cuh"

#include <cuda.h>
#include <string.h>

#include <mutex>

namespace lot {
namespace apply {

using namespace sm100;
using namespace tile;

constexpr int kTileRows = 128;
constexpr int kDK = 64;
constexpr int kTileBytes = kTileRows * kDK * 2;
constexpr int kStages = 4;
constexpr int kThreads = 384;          // warp 0 producer, warp 1 MMA issuer, warps 4-11 two worker quads (2, 3 idle)
constexpr int kWorkers = 256;
constexpr uint64_t kWaitNs = 1000000000ull;

struct alignas(64) ApplyParams {
    CUtensorMap tmKt;            // stored kernel [2 BH][npad][64] bf16 (side 0 queries, 1 keys), box 64 x 128 x 1
    CUtensorMap tmV, tmO;        // [BH][n][64] bf16
    const float *G;              // [2][BH][64] final pivot potentials, base-2 units
    const float *beta;           // [H][r]
    const int32_t *key_len;      // [B] or nullptr
    const int *decision;         // [2][BH]: 2 = the Sinkhorn kernel applied this slice itself (either side says so)
    float *wpart;                // [BH][maxslots][64 pivots][64 channels]
    int *status;
    int B, H, n, r, TPS, NT, ctas, maxslots;
};

__device__ __forceinline__ int range_lo(const ApplyParams &P, int cta) { return (int)(((long long)cta * P.NT) / P.ctas); }
__device__ __forceinline__ int cta_of_tile(const ApplyParams &P, int u) { return (int)((((long long)u + 1) * P.ctas - 1) / P.NT); }
__device__ __forceinline__ int key_count(const ApplyParams &P, int s)
{
    return P.key_len != nullptr ? min(max(__ldg(P.key_len + s / P.H), 0), P.n) : P.n;
}
__device__ __forceinline__ bool slice_here(const ApplyParams &P, int s)
{
    const int BH = P.B * P.H;
    return __ldcg(P.decision + s) != 2 && __ldcg(P.decision + BH + s) != 2;
}

// Bounded mbarrier wait (cold part out of line, plain arguments).
__device__ __noinline__ bool wait_slow(uint32_t b, uint32_t parity, volatile int *abort_flag, int *status)
{
    uint64_t t0 = 0;
    for (uint32_t it = 0;; ++it) {
        if (mbar_try_wait(b, parity)) return true;
        if ((it & 63u) == 63u) {
            if (*abort_flag) return false;
            const uint64_t now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitNs) break;
        }
    }
    *abort_flag = 1;
    atomicOr(status, 4 /* LOT_DEV_TIMEOUT */);
    return false;
}
struct Sync {
    uint32_t bar0;
    volatile int *abort_flag;
    int *status;
    int lane;
    __device__ __forceinline__ uint32_t bar(int id) const { return bar0 + 8u * id; }
    __device__ __forceinline__ bool wait(int id, uint32_t parity) const
    {
        const uint32_t b = bar(id);
        if (mbar_try_wait(b, parity)) return true;
        if (mbar_try_wait(b, parity)) return true;
        return wait_slow(b, parity, abort_flag, status);
    }
    __device__ __forceinline__ bool warp_wait(int id, uint32_t parity) const
    {
        return __all_sync(0xffffffffu, wait(id, parity)) != 0;
    }
    __device__ __forceinline__ void warp_arrive(int id) const
    {
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(id));
    }
};

// Weights w_t = 2^(G_t - max G) of one (slice, side) into shared memory (one warp; columns >= r get 0).
__device__ __forceinline__ void weights_to_smem(const float *G, int r, float *sW, int lane)
{
    const float g0 = lane < r ? __ldcg(G + lane) : neg_inf(), g1 = lane + 32 < r ? __ldcg(G + lane + 32) : neg_inf();
    float mx = fmaxf(g0, g1);
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
    sW[lane] = lane < r ? ex2(g0 - mx) : 0.f;
    sW[lane + 32] = lane + 32 < r ? ex2(g1 - mx) : 0.f;
}

// Row sums s = sum_t K~ w of the thread's four rows (rq + 8 j of its warp's 32) of a stored tile in shared memory
// (128-byte rows, 16-byte chunks xor row % 8): the thread reads columns 16 cq .. 16 cq + 15, the quad adds up.
__device__ __forceinline__ void tile_row_sums(const uint8_t *tileptr, int w4, int rq, int cq, const float2 (&w2)[8], float (&sr)[4])
{
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int rin = w4 * 32 + j * 8 + rq;
        const uint8_t *row = tileptr + rin * 128;
        const uint4 a = *reinterpret_cast<const uint4 *>(row + (((2 * cq) ^ (rin & 7)) * 16));
        const uint4 b = *reinterpret_cast<const uint4 *>(row + (((2 * cq + 1) ^ (rin & 7)) * 16));
        const uint32_t d[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
        float2 sa = make_float2(0.f, 0.f);
#pragma unroll
        for (int e = 0; e < 8; ++e) sa = __ffma2_rn(unpack_bf16(d[e]), w2[e], sa);
        sr[j] = sa.x + sa.y;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) sr[j] += __shfl_xor_sync(0xffffffffu, sr[j], 1);
#pragma unroll
    for (int j = 0; j < 4; ++j) sr[j] += __shfl_xor_sync(0xffffffffu, sr[j], 2);
}

// ---------------------------------------------------------------------------------------
// W = Gamma2 V
// ---------------------------------------------------------------------------------------
struct PlanW {
    static constexpr int offK = 0;                              // stored key tiles
    static constexpr int offV = offK + kStages * kTileBytes;    // value tiles, rewritten as the hi part of V / s
    static constexpr int offL = offV + kStages * kTileBytes;    // lo part
    static constexpr int offBar = offL + kStages * kTileBytes;  // 32 mbarriers
    static constexpr int offW = offBar + 32 * 8;                // float sW[64]
    static constexpr int offMisc = offW + 64 * 4;
    static constexpr int total = offMisc + 64;
};
enum BarW { wFull = 0 /* [4] */, wEmpty = 4 /* [4] */, wScaled = 8 /* [4] count 4 */, wAcc = 12 /* accumulator of a segment complete */,
            wRead = 13 /* count 8: read out */ };

__global__ void __launch_bounds__(kThreads, 1)
apply_w_kernel(const __grid_constant__ ApplyParams P)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + PlanW::offBar);
    float *sW = reinterpret_cast<float *>(smem + PlanW::offW);
    volatile int *sAbort = reinterpret_cast<volatile int *>(smem + PlanW::offMisc);
    uint32_t *sTmem = reinterpret_cast<uint32_t *>(smem + PlanW::offMisc + 4);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const Sync S{smem_u32(bars), sAbort, P.status, lane};
    if ((sbase & 1023u) != 0) { if (threadIdx.x == 0) atomicOr(P.status, 4); return; }
    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) { mbar_init(S.bar(wFull + i), 1); mbar_init(S.bar(wEmpty + i), 1); mbar_init(S.bar(wScaled + i), 4); }
        mbar_init(S.bar(wAcc), 1); mbar_init(S.bar(wRead), 8);
        *sAbort = 0;
        fence_barrier_init();
        prefetch_tensormap(&P.tmKt); prefetch_tensormap(&P.tmV);
    }
    if (warp == 1) { tmem_alloc(smem_u32(sTmem), 64); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *sTmem;
    const int BH = P.B * P.H;
    const int u0 = range_lo(P, blockIdx.x), u1 = range_lo(P, blockIdx.x + 1);
    const int s_lo = u0 < u1 ? u0 / P.TPS : 0, s_hi = u0 < u1 ? (u1 - 1) / P.TPS : -1;

    // the same enumeration in every role: slices of this block's range that are applied here, their valid key tiles
    auto seg_range = [&](int s, int &t0, int &t1, int &kv) {
        kv = key_count(P, s);
        const int vtk = (kv + kTileRows - 1) / kTileRows;
        t0 = max(u0 - s * P.TPS, 0);
        t1 = min(min(u1 - s * P.TPS, P.TPS), vtk);
        return t0 < t1 && slice_here(P, s);
    };

    if (warp == 0) {
        if (lane == 0) {
            int cnt = 0;
            bool ok = true;
            for (int s = s_lo; s <= s_hi && ok; ++s) {
                int t0, t1, kv;
                if (!seg_range(s, t0, t1, kv)) continue;
                for (int t = t0; t < t1 && ok; ++t, ++cnt) {
                    const int st = cnt % kStages;
                    if (cnt >= kStages) ok = S.wait(wEmpty + st, ((cnt / kStages) - 1) & 1);
                    if (!ok) break;
                    mbar_arrive_expect_tx(S.bar(wFull + st), 2 * kTileBytes);
                    tma_load_3d(sbase + PlanW::offK + st * kTileBytes, &P.tmKt, S.bar(wFull + st), 0, t * kTileRows, BH + s);
                    tma_load_3d(sbase + PlanW::offV + st * kTileBytes, &P.tmV, S.bar(wFull + st), 0, t * kTileRows, s);
                }
            }
        }
    } else if (warp == 1) {
        constexpr uint32_t idesc = make_idesc_bf16(64, kDK, 1, 1);
        const uint64_t dMN = make_smem_desc(sbase, kTileBytes, 1024);
        const uint32_t d_hi = (uint32_t)(dMN >> 32), d_lo = (uint32_t)dMN;
        int cnt = 0, seg = 0;
        bool ok = true;
        for (int s = s_lo; s <= s_hi && ok; ++s) {
            int t0, t1, kv;
            if (!seg_range(s, t0, t1, kv)) continue;
            if (seg > 0) ok = S.warp_wait(wRead, (seg - 1) & 1);           // the previous segment's accumulator is read out
            for (int t = t0; t < t1 && ok; ++t, ++cnt) {
                const int st = cnt % kStages;
                ok = S.warp_wait(wScaled + st, (cnt / kStages) & 1);
                if (!ok) break;
                tc_fence_after();
                const uint32_t ka = d_lo + ((PlanW::offK + st * kTileBytes) >> 4);
                const uint32_t va = d_lo + ((PlanW::offV + st * kTileBytes) >> 4), la = d_lo + ((PlanW::offL + st * kTileBytes) >> 4);
                if (elect_one()) {
#pragma unroll
                    for (int part = 0; part < 2; ++part)
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks)
                            umma_bf16(tmem, ((uint64_t)d_hi << 32) | (ka + ks * 128), ((uint64_t)d_hi << 32) | ((part ? la : va) + ks * 128),
                                      idesc, (t == t0 && part == 0 && ks == 0) ? 0u : 1u);
                    umma_commit(S.bar(wEmpty + st));
                    if (t == t1 - 1) umma_commit(S.bar(wAcc));
                }
                __syncwarp();
            }
            ++seg;
        }
    } else if (warp >= 4) {
        const int quad = (warp - 4) >> 2, w4 = warp & 3, rq = lane >> 2, cq = lane & 3, wtid = (int)threadIdx.x - 128;
        const uint32_t lane_addr = tmem + ((uint32_t)(w4 * 32) << 16);
        int cnt = 0, seg = 0;
        bool ok = true;
        for (int s = s_lo; s <= s_hi; ++s) {
            int t0, t1, kv;
            if (!seg_range(s, t0, t1, kv)) continue;
            named_bar_sync(1, kWorkers);                                   // sW of the previous segment is no longer read
            if (warp == 4) weights_to_smem(P.G + ((size_t)BH + s) * 64, P.r, sW, lane);
            named_bar_sync(1, kWorkers);
            float2 w2[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) w2[e] = *reinterpret_cast<const float2 *>(sW + 16 * cq + 2 * e);
            for (int t = t0; t < t1; ++t, ++cnt) {
                if ((cnt & 1) != quad) continue;
                const int st = cnt % kStages;
                if (ok) ok = S.warp_wait(wFull + st, (cnt / kStages) & 1);
                if (!ok) continue;
                float sr[4];
                tile_row_sums(smem + PlanW::offK + st * kTileBytes, w4, rq, cq, w2, sr);
                uint8_t *vt = smem + PlanW::offV + st * kTileBytes, *lt = smem + PlanW::offL + st * kTileBytes;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int rin = w4 * 32 + j * 8 + rq, row = t * kTileRows + rin;
                    const float u = row < kv ? __fdividef(1.f, sr[j]) : 0.f;
                    const float2 uu = make_float2(u, u);
#pragma unroll
                    for (int h2 = 0; h2 < 2; ++h2) {
                        const int off = rin * 128 + (((2 * cq + h2) ^ (rin & 7)) * 16);
                        uint4 x = *reinterpret_cast<uint4 *>(vt + off), y;
                        uint32_t *xw = reinterpret_cast<uint32_t *>(&x), *yw = reinterpret_cast<uint32_t *>(&y);
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float2 f = __fmul2_rn(unpack_bf16(xw[e]), uu);
                            __nv_bfloat162 hh = __floats2bfloat162_rn(f.x, f.y);
                            xw[e] = *reinterpret_cast<uint32_t *>(&hh);
                            yw[e] = pack_bf16(f.x - __low2float(hh), f.y - __high2float(hh));
                        }
                        *reinterpret_cast<uint4 *>(vt + off) = x;
                        *reinterpret_cast<uint4 *>(lt + off) = y;
                    }
                }
                fence_proxy_async_smem();
                S.warp_arrive(wScaled + st);
            }
            // ---- the segment's accumulator: pivot rows 16 w4 .. + 15 in the first 16 lanes of lane quarter w4; quad q takes
            // channels 32 q .. + 31; the partial leaves multiplied by the key-side weights
            if (ok) ok = S.warp_wait(wAcc, seg & 1);
            float v[16];
            if (ok) {
                tc_fence_after();
                tmem_ld_acc<4>(lane_addr + 32 * quad, v);
                tmem_wait_ld();
                tc_fence_before();
            }
            S.warp_arrive(wRead);
            if (ok) {
                const int tA = 16 * w4 + rq, tB = tA + 8;
                const float wA = sW[tA], wB = sW[tB];
                const int slot = (int)blockIdx.x - cta_of_tile(P, s * P.TPS);
                float *dst = P.wpart + ((size_t)s * P.maxslots + slot) * (64 * kDK) + 32 * quad + 2 * cq;
#pragma unroll
                for (int rep = 0; rep < 4; ++rep) {
                    *reinterpret_cast<float2 *>(dst + tA * kDK + rep * 8) = make_float2(v[rep * 4 + 0] * wA, v[rep * 4 + 1] * wA);
                    *reinterpret_cast<float2 *>(dst + tB * kDK + rep * 8) = make_float2(v[rep * 4 + 2] * wB, v[rep * 4 + 3] * wB);
                }
            }
            ++seg;
            (void)wtid;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem, 64); }
}

// ---------------------------------------------------------------------------------------
// out = K~1 W'' / s
// ---------------------------------------------------------------------------------------
struct PlanO {
    static constexpr int offK = 0;                              // stored query tiles
    static constexpr int offO = offK + kStages * kTileBytes;    // output staging
    static constexpr int offWq = offO + kStages * kTileBytes;   // two W'' operands (hi, lo: 8 KB each)
    static constexpr int offBar = offWq + 2 * kTileBytes;
    static constexpr int offW = offBar + 32 * 8;                // float sW[64]
    static constexpr int offMisc = offW + 64 * 4;
    static constexpr int total = offMisc + 64;
};
enum BarO { oFull = 0 /* [4] */, oEmpty = 4 /* [4] count 5 */, oAcc = 8 /* [4] accumulator of the stage's tile complete */,
            oRead = 12 /* [4] count 4: read out */, oWq = 16 /* [2] count 8: W'' operand written */ };

__global__ void __launch_bounds__(kThreads, 1)
apply_out_kernel(const __grid_constant__ ApplyParams P)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + PlanO::offBar);
    float *sW = reinterpret_cast<float *>(smem + PlanO::offW);
    volatile int *sAbort = reinterpret_cast<volatile int *>(smem + PlanO::offMisc);
    uint32_t *sTmem = reinterpret_cast<uint32_t *>(smem + PlanO::offMisc + 4);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const Sync S{smem_u32(bars), sAbort, P.status, lane};
    if ((sbase & 1023u) != 0) { if (threadIdx.x == 0) atomicOr(P.status, 4); return; }
    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) {
            mbar_init(S.bar(oFull + i), 1); mbar_init(S.bar(oEmpty + i), 5); mbar_init(S.bar(oAcc + i), 1); mbar_init(S.bar(oRead + i), 4);
        }
        mbar_init(S.bar(oWq), 8); mbar_init(S.bar(oWq + 1), 8);
        *sAbort = 0;
        fence_barrier_init();
        prefetch_tensormap(&P.tmKt); prefetch_tensormap(&P.tmO);
    }
    if (warp == 1) { tmem_alloc(smem_u32(sTmem), 256); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *sTmem;
    const int u0 = range_lo(P, blockIdx.x), u1 = range_lo(P, blockIdx.x + 1);
    const int s_lo = u0 < u1 ? u0 / P.TPS : 0, s_hi = u0 < u1 ? (u1 - 1) / P.TPS : -1;
    auto seg_range = [&](int s, int &t0, int &t1) {
        t0 = max(u0 - s * P.TPS, 0);
        t1 = min(u1 - s * P.TPS, P.TPS);
        return t0 < t1 && slice_here(P, s);
    };

    if (warp == 0) {
        if (lane == 0) {
            int cnt = 0;
            bool ok = true;
            for (int s = s_lo; s <= s_hi && ok; ++s) {
                int t0, t1;
                if (!seg_range(s, t0, t1)) continue;
                for (int t = t0; t < t1 && ok; ++t, ++cnt) {
                    const int st = cnt % kStages;
                    if (cnt >= kStages) ok = S.wait(oEmpty + st, ((cnt / kStages) - 1) & 1);
                    if (!ok) break;
                    mbar_arrive_expect_tx(S.bar(oFull + st), kTileBytes);
                    tma_load_3d(sbase + PlanO::offK + st * kTileBytes, &P.tmKt, S.bar(oFull + st), 0, t * kTileRows, s);
                }
            }
        }
    } else if (warp == 1) {
        constexpr uint32_t idesc = make_idesc_bf16(128, kDK, 0, 0);
        const uint64_t dK = make_smem_desc(sbase, 16, 1024);
        const uint32_t d_hi = (uint32_t)(dK >> 32), d_lo = (uint32_t)dK;
        int cnt = 0, seg = 0;
        bool ok = true;
        for (int s = s_lo; s <= s_hi && ok; ++s) {
            int t0, t1;
            if (!seg_range(s, t0, t1)) continue;
            ok = S.warp_wait(oWq + (seg & 1), (seg >> 1) & 1);
            const uint32_t wa = d_lo + ((PlanO::offWq + (seg & 1) * kTileBytes) >> 4);
            for (int t = t0; t < t1 && ok; ++t, ++cnt) {
                const int st = cnt % kStages;
                ok = S.warp_wait(oFull + st, (cnt / kStages) & 1);
                if (ok && cnt >= kStages) ok = S.warp_wait(oRead + st, ((cnt / kStages) - 1) & 1);
                if (!ok) break;
                tc_fence_after();
                const uint32_t aa = d_lo + ((PlanO::offK + st * kTileBytes) >> 4);
                if (elect_one()) {
#pragma unroll
                    for (int part = 0; part < 2; ++part)
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            umma_bf16(tmem + st * kDK, ((uint64_t)d_hi << 32) | (aa + ks * 2),
                                      ((uint64_t)d_hi << 32) | (wa + part * ((kDK * 128) >> 4) + ks * 2), idesc, (part | ks) ? 1u : 0u);
                    umma_commit(S.bar(oAcc + st));
                    umma_commit(S.bar(oEmpty + st));
                }
                __syncwarp();
            }
            ++seg;
        }
    } else if (warp >= 4) {
        const int quad = (warp - 4) >> 2, w4 = warp & 3, rq = lane >> 2, cq = lane & 3, wtid = (int)threadIdx.x - 128;
        const uint32_t lane_addr = tmem + ((uint32_t)(w4 * 32) << 16);
        const bool storer = w4 == 0 && lane == 0;
        int cnt = 0, seg = 0;
        bool ok = true;
        for (int s = s_lo; s <= s_hi; ++s) {
            int t0, t1;
            if (!seg_range(s, t0, t1)) continue;
            const int h = s % P.H, kv = key_count(P, s);
            // ---- W''^T = (Diag(w1) Diag(beta)^-1 Gamma2 V)^T of the slice as the B operand (rows = channels, 128 bytes = 64
            // pivots, 16-byte chunks xor row % 8; hi part, lo part): the partials of the blocks that hold keys of the slice,
            // added in slot order.  The operand buffer of segment seg - 2 is free: its tiles have all been read out.
            named_bar_sync(1, kWorkers);
            if (warp == 4) weights_to_smem(P.G + (size_t)s * 64, P.r, sW, lane);
            named_bar_sync(1, kWorkers);
            {
                const int vtk = (kv + kTileRows - 1) / kTileRows;
                const int c_lo = cta_of_tile(P, s * P.TPS);
                const int wslots = vtk > 0 ? cta_of_tile(P, s * P.TPS + vtk - 1) - c_lo + 1 : 0;
                const int tA = 16 * w4 + rq, tB = tA + 8;
                float acc[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) acc[e] = 0.f;
                const float *src0 = P.wpart + (size_t)s * P.maxslots * (64 * kDK) + 32 * quad + 2 * cq;
                for (int sl = 0; sl < wslots; ++sl) {
                    const float *src = src0 + (size_t)sl * (64 * kDK);
#pragma unroll
                    for (int rep = 0; rep < 4; ++rep) {
                        const float2 a = __ldcg(reinterpret_cast<const float2 *>(src + tA * kDK + rep * 8));
                        const float2 b = __ldcg(reinterpret_cast<const float2 *>(src + tB * kDK + rep * 8));
                        acc[rep * 4 + 0] += a.x; acc[rep * 4 + 1] += a.y; acc[rep * 4 + 2] += b.x; acc[rep * 4 + 3] += b.y;
                    }
                }
                const float mass = kv > 0 ? 1.f / (float)kv : 0.f;
                const float cA = tA < P.r ? sW[tA] * mass / __ldg(P.beta + h * P.r + tA) : 0.f;
                const float cB = tB < P.r ? sW[tB] * mass / __ldg(P.beta + h * P.r + tB) : 0.f;
                uint8_t *wq = smem + PlanO::offWq + (seg & 1) * kTileBytes;
#pragma unroll
                for (int rep = 0; rep < 4; ++rep)
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const int ch = 32 * quad + rep * 8 + 2 * cq + u;
#pragma unroll
                        for (int rb = 0; rb < 2; ++rb) {
                            const int t = rb ? tB : tA;
                            const float x = acc[rep * 4 + 2 * rb + u] * (rb ? cB : cA);
                            const __nv_bfloat16 hi = __float2bfloat16_rn(x);
                            const __nv_bfloat16 lo = __float2bfloat16_rn(x - __bfloat162float(hi));
                            uint8_t *dst = wq + ch * 128 + (((t >> 3) ^ (ch & 7)) * 16) + (t & 7) * 2;
                            *reinterpret_cast<__nv_bfloat16 *>(dst) = hi;
                            *reinterpret_cast<__nv_bfloat16 *>(dst + kDK * 128) = lo;
                        }
                    }
                fence_proxy_async_smem();
                S.warp_arrive(oWq + (seg & 1));
            }
            float2 w2[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) w2[e] = *reinterpret_cast<const float2 *>(sW + 16 * cq + 2 * e);
            for (int t = t0; t < t1; ++t, ++cnt) {
                if ((cnt & 1) != quad) continue;
                const int st = cnt % kStages;
                if (ok) ok = S.warp_wait(oFull + st, (cnt / kStages) & 1);
                if (!ok) continue;
                float sr[4];
                tile_row_sums(smem + PlanO::offK + st * kTileBytes, w4, rq, cq, w2, sr);
                S.warp_arrive(oEmpty + st);                     // the tile's rows are in registers
                if (ok) ok = S.warp_wait(oAcc + st, (cnt / kStages) & 1);
                if (!ok) continue;
                tc_fence_after();
                float o[2][32];
                tmem_ld_acc<8>(lane_addr + st * kDK, o[0]);
                tmem_ld_acc<8>(lane_addr + (16u << 16) + st * kDK, o[1]);
                tmem_wait_ld();
                tc_fence_before();
                S.warp_arrive(oRead + st);
                // the store that last read this stage's staging buffer (two of this quad's tiles ago) must be done with it
                if (storer) bulk_wait_group_read<1>();
                named_bar_sync(2 + quad, 128);
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int rinA = w4 * 32 + half * 16 + rq;
                    const float iA = __fdividef(1.f, sr[2 * half]), iB = __fdividef(1.f, sr[2 * half + 1]);
                    const uint32_t rowaddr = sbase + PlanO::offO + st * kTileBytes + rinA * 128 + cq * 4;
#pragma unroll
                    for (int rep = 0; rep < 8; ++rep) {
                        const uint32_t addr = rowaddr + ((rep ^ (rinA & 7)) << 4);
                        asm volatile("st.shared.b32 [%0], %1;" ::"r"(addr), "r"(pack_bf16(o[half][rep * 4 + 0] * iA, o[half][rep * 4 + 1] * iA)) : "memory");
                        asm volatile("st.shared.b32 [%0 + 1024], %1;" ::"r"(addr), "r"(pack_bf16(o[half][rep * 4 + 2] * iB, o[half][rep * 4 + 3] * iB)) : "memory");
                    }
                }
                fence_proxy_async_smem();
                named_bar_sync(2 + quad, 128);
                if (storer) {
                    tma_store_3d(&P.tmO, sbase + PlanO::offO + st * kTileBytes, 0, t * kTileRows, s);
                    bulk_commit_group();
                }
            }
            ++seg;
            (void)wtid;
        }
        if (storer) bulk_wait_group0();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem, 256); }
}

// ---------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static bool make_map(CUtensorMap *m, const void *base, long long outer, int rows)
{
    static EncodeTiledFn fn = nullptr;
    static std::mutex mu;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (fn == nullptr) {
            void *p = nullptr;
            cudaDriverEntryPointQueryResult qres;
            if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
                qres != cudaDriverEntryPointSuccess)
                return false;
            fn = reinterpret_cast<EncodeTiledFn>(p);
        }
    }
    cuuint64_t dims[3] = {64u, (cuuint64_t)rows, (cuuint64_t)outer};
    cuuint64_t strides[2] = {128u, (cuuint64_t)rows * 128u};
    cuuint32_t box[3] = {64u, 128u, 1u};
    cuuint32_t es[3] = {1u, 1u, 1u};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

} // namespace apply

size_t stored_apply_wpart_bytes(int B, int H, int n)
{
    const int TPS = (n + 127) / 128;
    const long long NT = (long long)B * H * TPS;
    const int sms = device_sm_count();
    const int ctas = NT < sms ? (int)NT : sms;
    const int maxslots = (int)(((long long)TPS * ctas) / NT) + 2;
    return (size_t)B * H * maxslots * 64 * 64 * 4;
}

cudaError_t stored_apply(const void *kt, int npad, const float *G, const float *beta, const int32_t *key_len, const int *decision,
                         const void *v, void *out, float *wpart, int *status, int B, int H, int n, int r, cudaStream_t st)
{
    using namespace apply;
    ApplyParams P;
    memset(&P, 0, sizeof(P));
    const long long BH = (long long)B * H;
    if (!make_map(&P.tmKt, kt, 2 * BH, npad) || !make_map(&P.tmV, v, BH, n) || !make_map(&P.tmO, out, BH, n)) return cudaErrorInvalidValue;
    P.G = G; P.beta = beta; P.key_len = key_len; P.decision = decision; P.wpart = wpart; P.status = status;
    P.B = B; P.H = H; P.n = n; P.r = r;
    P.TPS = (n + 127) / 128;
    P.NT = (int)(BH * P.TPS);
    const int sms = device_sm_count();
    P.ctas = P.NT < sms ? P.NT : sms;
    P.maxslots = (int)(((long long)P.TPS * P.ctas) / P.NT) + 2;
    static std::mutex mu;
    static bool attr[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!attr[dev]) {
            cudaError_t e = cudaFuncSetAttribute(apply_w_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, PlanW::total);
            if (e == cudaSuccess) e = cudaFuncSetAttribute(apply_out_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, PlanO::total);
            if (e != cudaSuccess) return e;
            attr[dev] = true;
        }
    }
    apply_w_kernel<<<P.ctas, kThreads, PlanW::total, st>>>(P);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    apply_out_kernel<<<P.ctas, kThreads, PlanO::total, st>>>(P);
    return cudaGetLastError();
}

} // namespace lot
