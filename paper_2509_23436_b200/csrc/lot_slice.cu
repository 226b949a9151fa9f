// Slice path of the LOT attention forward (Eq. (1)-(4)): one thread block per (batch, head) slice, for sequences
// short enough that a side's whole n x r logit matrix fits the block's registers (bf16 tensors, d = 64, r <= 64,
// n <= 512, 16 ceil(n/16) x rpad <= 16384).  Nothing crosses thread blocks and nothing but the inputs and the output
// touches global memory:
//   key side:   K, V -> shared memory; logits L2 = K Z^T * log2(e)/eps on the tensor cores (warp-level MMA, Z as bf16
//               hi + lo) into registers; T Sinkhorn iterations on the registers (scaling form on the float32 Gibbs
//               kernel, log domain when the potentials spread too far; row reductions inside a lane quad, column
//               sums through shared memory in a fixed order); plan rows -> shared memory as bf16 hi + lo;
//               W = Gamma2^T V on the tensor cores; W' = Diag(1/beta) W -> shared memory, bf16 hi + lo.
//   query side: Q -> shared memory; logits; iterations; out = R1 W' with the plan rows straight from the registers
//               that held the logits (an accumulator fragment is an A fragment); bf16 rows to global memory.
// Logits and Gibbs kernel are float32 in registers: no stored bf16 kernel, and no range limit (see solve).
// 512 threads; warp w owns the 16-row tiles w, w + 16; a thread holds rows g and g + 8 (g = lane / 4) of each and,
// per 8-column tile, columns 2 (lane % 4) and + 1: the accumulator layout of mma.m16n8k16.
#include "lot_common.cuh"
#include "lot_internal.h"

#include <mutex>

namespace lot {
namespace slice {

constexpr int kThreads = 512;
constexpr int kWarps = 16;
constexpr int kD = 64;
constexpr int kPitch = 144;            // bytes per 64-element bf16 row in shared memory (128 + 16: conflict-free ldmatrix)
constexpr float kTiny = 1e-30f;        // a plain column sum below this is recomputed relative to its maximum

struct SliceParams {
    const __nv_bfloat16 *q, *k, *v;
    const float *z, *beta;
    const int32_t *key_len;
    __nv_bfloat16 *out;
    float *g1_out, *g2_out;
    int *status;
    int B, H, n, r, T;
    float scale;       // log2(e)/eps
    float eps_ln2;
};

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all()
{
    asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;" ::: "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D += A (16 x 16, row) * B (16 x 8, col), bf16 operands, float accumulators
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi)
{
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&t);
}
// (hi, lo) bf16 pairs of two floats: x = hi + lo to about 2^-17
__device__ __forceinline__ void split2(float x0, float x1, uint32_t &hi, uint32_t &lo)
{
    __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
    hi = *reinterpret_cast<uint32_t *>(&h);
    lo = pack2(x0 - __low2float(h), x1 - __high2float(h));
}

template <int NT, int MT>
struct Plan {
    static constexpr int RP = 8 * NT;                      // padded pivot count
    static constexpr int RX = 256 * MT;                    // padded token count
    static constexpr int pitchP = RP * 2 + 16;             // bytes per row of a plan plane / a W' plane
    static constexpr int xBytes = RX * kPitch > 2 * RX * pitchP ? RX * kPitch : 2 * RX * pitchP;
    static constexpr int offX = 0;                         // K, then the plan planes (hi, lo), then Q
    static constexpr int offV = offX + xBytes;
    static constexpr int offZ = offV + RX * kPitch;        // Z * log2(e)/eps as bf16 hi, lo: [RP][64]
    static constexpr int offWp = offZ + 2 * RP * kPitch;   // W'^T as bf16 hi, lo: [64][RP]
    static constexpr int offWacc = offWp + 2 * kD * pitchP; // float [ksplit][RP][64], ksplit * RP = 64
    static constexpr int offRed = offWacc + 64 * kD * 4;   // float [16][64]
    static constexpr int offLam = offRed + kWarps * 64 * 4; // float [64] log2 of the column sums
    static constexpr int offLb = offLam + 64 * 4;          // float [64] log2(beta_t * valid tokens)
    static constexpr int offKap = offLb + 64 * 4;          // float [64] column maxima (robust recomputation)
    static constexpr int offG = offKap + 64 * 4;           // float [64] potentials (scaling-form iterations)
    static constexpr int offStat = offG + 64 * 4;          // uint [2][2]: max and min of the potentials, ordered encoding
    static constexpr int offFlag = offStat + 16;           // int
    static constexpr int total = offFlag + 16;
};

// One side's logits into the accumulators: L = X Zs^T for the warp's tiles.
template <int NT, int MT>
__device__ __forceinline__ void logits(float (&L)[MT][NT][4], const uint8_t *sX, const uint8_t *sZ, int warp, int lane, int ntiles)
{
    using PL = Plan<NT, MT>;
    const uint32_t xb = smem_addr(sX), zh = smem_addr(sZ), zl = zh + PL::RP * kPitch;
#pragma unroll
    for (int mi = 0; mi < MT; ++mi) {
#pragma unroll
        for (int j = 0; j < NT; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) L[mi][j][e] = 0.f;
        const int mt = warp + kWarps * mi;
        if (mt >= ntiles) continue;                                   // warp-uniform
        const int row0 = mt * 16;
#pragma unroll
        for (int ks = 0; ks < kD / 16; ++ks) {
            uint32_t a[4];
            ldsm_x4(a, xb + (row0 + (lane & 7) + ((lane >> 3) & 1) * 8) * kPitch + (ks * 16 + (lane >> 4) * 8) * 2);
#pragma unroll
            for (int jp = 0; jp < NT / 2; ++jp) {
                const uint32_t off = (jp * 16 + (lane & 7) + (lane >> 4) * 8) * kPitch + (ks * 16 + ((lane >> 3) & 1) * 8) * 2;
                uint32_t bh[4], bl[4];
                ldsm_x4(bh, zh + off);
                ldsm_x4(bl, zl + off);
                mma16816(L[mi][2 * jp], a, bh[0], bh[1]);
                mma16816(L[mi][2 * jp], a, bl[0], bl[1]);
                mma16816(L[mi][2 * jp + 1], a, bh[2], bh[3]);
                mma16816(L[mi][2 * jp + 1], a, bl[2], bl[3]);
            }
        }
    }
}

// One round of a halving reduction over the lanes that differ in `bit`: of CNT live values a lane keeps one half
// (the upper one if its bit is set), hands the other to its partner and adds what it receives; `off` follows which
// of the original values the lane ends up with.  With one value left both partners keep the sum.
template <int CNT, bool MAX>
__device__ __forceinline__ void halve(float (&v)[16], int lane, int bit, int &off)
{
    if constexpr (CNT > 1) {
        constexpr int H = CNT / 2;
        const bool up = (lane & bit) != 0;
#pragma unroll
        for (int i = 0; i < H; ++i) {
            const float give = up ? v[i] : v[i + H], keep = up ? v[i + H] : v[i];
            const float got = __shfl_xor_sync(0xffffffffu, give, bit);
            v[i] = MAX ? fmaxf(keep, got) : keep + got;
        }
        off += up ? H : 0;
    } else {
        const float got = __shfl_xor_sync(0xffffffffu, v[0], bit);
        v[0] = MAX ? fmaxf(v[0], got) : v[0] + got;
    }
}

// Sum (or maximum) of per-thread column values over the block, in a fixed order: lanes of equal lane % 4 hold the
// same columns and reduce them by halving; warp results go through sRed; thread t < 8 NT then owns column t and
// gets its total (others 0).  One __syncthreads inside; the caller orders the reuse of sRed.
template <int NT, bool MAX>
__device__ __forceinline__ float block_columns(float (&c)[NT][2], float *sRed, int warp, int lane)
{
    constexpr int NV = 2 * NT;
    float v[16];
#pragma unroll
    for (int i = 0; i < NV; ++i) v[i] = c[i >> 1][i & 1];
    int off = 0;
    halve<NV, MAX>(v, lane, 16, off);
    halve<(NV > 1 ? NV / 2 : 1), MAX>(v, lane, 8, off);
    halve<(NV > 3 ? NV / 4 : 1), MAX>(v, lane, 4, off);
    constexpr int FC = NV >= 8 ? NV / 8 : 1;
    const int q = lane & 3;
#pragma unroll
    for (int i = 0; i < FC; ++i) {
        const int idx = off + i;
        sRed[warp * 64 + 8 * (idx >> 1) + 2 * q + (idx & 1)] = v[i];
    }
    __syncthreads();
    float tot = MAX ? neg_inf() : 0.f;
    const int t = threadIdx.x;
    if (t < 8 * NT) {
#pragma unroll
        for (int w = 0; w < kWarps; ++w) tot = MAX ? fmaxf(tot, sRed[w * 64 + t]) : tot + sRed[w * 64 + t];
    }
    return tot;
}

// floats as unsigned integers of the same order (for atomicMax / atomicMin in shared memory)
__device__ __forceinline__ uint32_t enc_ord(float f)
{
    const uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float dec_ord(uint32_t u)
{
    return __uint_as_float((u & 0x80000000u) ? (u & 0x7fffffffu) : ~u);
}

// T Sinkhorn iterations and the closing token update on one side's logits (base-2 units, Eq. (1)-(2) with the token
// potential eliminated): G_t += log2(beta_t * nv) - log2 sum_i R_it, R_it = 2^(L_it + G_t - M_i) the row-stochastic
// plan, M_i the row log-sum-exp.  On return L holds R (zero rows for tokens without mass) and G the final potentials
// of the thread's columns.
// Scaling form while the potentials allow it: the logits are replaced once by the stabilised Gibbs kernel
// K~_it = 2^(L_it - max_t L_it) in float32, and an iteration is two multiply-adds per entry with the weights
// w_t = 2^(G_t - max G): s_i = sum_t K~_it w_t, column sums of K~_it / s_i.  When the potentials spread over more than
// 64 binades, or a column sum leaves float32's range, the logits are computed again and the iteration continues in
// the log domain (exact for any spread; a column sum out of range is taken relative to its column maximum).
template <int NT, int MT>
__device__ __forceinline__ void solve(float (&L)[MT][NT][4], float (&G)[NT][2], uint8_t *smem, const uint8_t *sX,
                                      const uint8_t *sZ, int warp, int lane, int ntiles, int nv, int r, int T, int *status)
{
    using PL = Plan<NT, MT>;
    float *sRed = reinterpret_cast<float *>(smem + PL::offRed);
    float *sLam = reinterpret_cast<float *>(smem + PL::offLam);
    const float *sLb = reinterpret_cast<const float *>(smem + PL::offLb);
    float *sKap = reinterpret_cast<float *>(smem + PL::offKap);
    float *sG = reinterpret_cast<float *>(smem + PL::offG);
    uint32_t *sStat = reinterpret_cast<uint32_t *>(smem + PL::offStat);   // [2][2]: max, min of G, by iteration parity
    volatile int *sFlag = reinterpret_cast<volatile int *>(smem + PL::offFlag);
    const int g = lane >> 2, q = lane & 3, tid = threadIdx.x;

    auto mask_columns = [&]() {
#pragma unroll
        for (int mi = 0; mi < MT; ++mi)
#pragma unroll
            for (int j = 0; j < NT; ++j)
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (8 * j + 2 * q + (e & 1) >= r) L[mi][j][e] = neg_inf();
    };
    mask_columns();
    // the stabilised Gibbs kernel in place of the logits
#pragma unroll
    for (int mi = 0; mi < MT; ++mi)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int row = (warp + kWarps * mi) * 16 + g + 8 * h;
            float m = neg_inf();
#pragma unroll
            for (int j = 0; j < NT; ++j) m = fmaxf(m, fmaxf(L[mi][j][2 * h], L[mi][j][2 * h + 1]));
            m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
            m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
#pragma unroll
            for (int j = 0; j < NT; ++j)
#pragma unroll
                for (int e = 0; e < 2; ++e) L[mi][j][2 * h + e] = row < nv ? ex2(L[mi][j][2 * h + e] - m) : 0.f;
        }
    if (tid < 64) sG[tid] = 0.f;
    if (tid == 0) {
        sStat[0] = enc_ord(0.f); sStat[1] = enc_ord(0.f);
        sStat[2] = 0u; sStat[3] = 0xffffffffu;
    }
    __syncthreads();

    bool fast = true;
    int it = 0;
    while (true) {
        const bool closing = it == T;
        float c[NT][2];
#pragma unroll
        for (int j = 0; j < NT; ++j) { c[j][0] = 0.f; c[j][1] = 0.f; }
        if (fast) {
            const float Gmax = dec_ord(sStat[(it & 1) * 2]), Gmin = dec_ord(sStat[(it & 1) * 2 + 1]);
            bool leave = Gmax - Gmin > 64.f;                       // block-uniform
            if (!leave) {
                float w[NT][2];
#pragma unroll
                for (int j = 0; j < NT; ++j) {
                    const float2 gg = *reinterpret_cast<const float2 *>(sG + 8 * j + 2 * q);
                    w[j][0] = 8 * j + 2 * q < r ? ex2(gg.x - Gmax) : 0.f;
                    w[j][1] = 8 * j + 2 * q + 1 < r ? ex2(gg.y - Gmax) : 0.f;
                }
#pragma unroll
                for (int mi = 0; mi < MT; ++mi)
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        float s = 0.f;
#pragma unroll
                        for (int j = 0; j < NT; ++j) {
                            s = fmaf(L[mi][j][2 * h], w[j][0], s);
                            s = fmaf(L[mi][j][2 * h + 1], w[j][1], s);
                        }
                        s += __shfl_xor_sync(0xffffffffu, s, 1);
                        s += __shfl_xor_sync(0xffffffffu, s, 2);
                        const float inv = s > 0.f ? __fdividef(1.f, s) : 0.f;
#pragma unroll
                        for (int j = 0; j < NT; ++j)
#pragma unroll
                            for (int e = 0; e < 2; ++e) {
                                if (closing) L[mi][j][2 * h + e] = L[mi][j][2 * h + e] * w[j][e] * inv;
                                else c[j][e] = fmaf(L[mi][j][2 * h + e], inv, c[j][e]);
                            }
                    }
                if (closing) break;
                const float tot = block_columns<NT, false>(c, sRed, warp, lane);
                float g_old = 0.f;
                const bool ok = tot >= kTiny;
                if (warp < 2) {                                    // threads 0..63 own the columns
                    uint32_t emax = 0u, emin = 0xffffffffu;
                    if (tid < r) {
                        g_old = sG[tid];
                        if (ok) {
                            const float gn = sLb[tid] + Gmax - lg2(tot);
                            sG[tid] = gn;
                            emax = emin = enc_ord(gn);
                            if (!isfinite(gn)) atomicOr(status, 1 /* LOT_DEV_NONFINITE */);
                        } else {
                            *sFlag = 1;
                        }
                    }
                    emax = __reduce_max_sync(0xffffffffu, emax);
                    emin = __reduce_min_sync(0xffffffffu, emin);
                    if (lane == 0) {
                        atomicMax(sStat + ((it + 1) & 1) * 2, emax);
                        atomicMin(sStat + ((it + 1) & 1) * 2 + 1, emin);
                    }
                }
                if (tid == 0) { sStat[(it & 1) * 2] = 0u; sStat[(it & 1) * 2 + 1] = 0xffffffffu; }
                __syncthreads();
                leave = *sFlag != 0;                               // a column sum out of range: redo this iteration
                if (leave) {
                    if (tid < r && ok) sG[tid] = g_old;
                    __syncthreads();
                    if (tid == 0) *sFlag = 0;
                } else {
                    ++it;
                }
            }
            if (leave) {
                fast = false;
                logits<NT, MT>(L, sX, sZ, warp, lane, ntiles);
                mask_columns();
#pragma unroll
                for (int j = 0; j < NT; ++j) {
                    const float2 gg = *reinterpret_cast<const float2 *>(sG + 8 * j + 2 * q);
                    G[j][0] = gg.x; G[j][1] = gg.y;
                }
            }
            continue;
        }

        // ---- log domain
#pragma unroll
        for (int mi = 0; mi < MT; ++mi)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int row = (warp + kWarps * mi) * 16 + g + 8 * h;
                float l[NT][2];
                float m = neg_inf();
#pragma unroll
                for (int j = 0; j < NT; ++j)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        l[j][e] = L[mi][j][2 * h + e] + G[j][e];
                        m = fmaxf(m, l[j][e]);
                    }
                m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
                m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
                float s = 0.f;
#pragma unroll
                for (int j = 0; j < NT; ++j)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        l[j][e] = ex2(l[j][e] - m);
                        s += l[j][e];
                    }
                s += __shfl_xor_sync(0xffffffffu, s, 1);
                s += __shfl_xor_sync(0xffffffffu, s, 2);
                const float inv = row < nv ? __fdividef(1.f, s) : 0.f;
#pragma unroll
                for (int j = 0; j < NT; ++j)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const float pr = l[j][e] * inv;
                        if (closing) L[mi][j][2 * h + e] = pr;
                        else c[j][e] += pr;
                    }
            }
        if (closing) break;

        float tot = block_columns<NT, false>(c, sRed, warp, lane);
        if (tid < r) {
            sLam[tid] = lg2(tot);
            if (!(tot >= kTiny)) *sFlag = 1;
        }
        __syncthreads();
        if (*sFlag) {
            // some column sum is out of float32's range: column maxima kappa_t of x_it = L_it + G_t - M_i first, then
            // the sums of 2^(x_it - kappa_t)   (block-uniform branch)
            float mx[NT][2];
#pragma unroll
            for (int j = 0; j < NT; ++j) { mx[j][0] = neg_inf(); mx[j][1] = neg_inf(); }
            float Mrow[MT][2];
#pragma unroll
            for (int mi = 0; mi < MT; ++mi)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int row = (warp + kWarps * mi) * 16 + g + 8 * h;
                    float m = neg_inf();
#pragma unroll
                    for (int j = 0; j < NT; ++j)
#pragma unroll
                        for (int e = 0; e < 2; ++e) m = fmaxf(m, L[mi][j][2 * h + e] + G[j][e]);
                    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
                    m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
                    float s = 0.f;
#pragma unroll
                    for (int j = 0; j < NT; ++j)
#pragma unroll
                        for (int e = 0; e < 2; ++e) s += ex2(L[mi][j][2 * h + e] + G[j][e] - m);
                    s += __shfl_xor_sync(0xffffffffu, s, 1);
                    s += __shfl_xor_sync(0xffffffffu, s, 2);
                    Mrow[mi][h] = row < nv ? m + lg2(s) : __int_as_float(0x7f800000);
#pragma unroll
                    for (int j = 0; j < NT; ++j)
#pragma unroll
                        for (int e = 0; e < 2; ++e) mx[j][e] = fmaxf(mx[j][e], L[mi][j][2 * h + e] + G[j][e] - Mrow[mi][h]);
                }
            const float kap = block_columns<NT, true>(mx, sRed, warp, lane);
            if (tid < 8 * NT) sKap[tid] = kap;
            __syncthreads();
#pragma unroll
            for (int j = 0; j < NT; ++j) {
                const float2 kk = *reinterpret_cast<const float2 *>(sKap + 8 * j + 2 * q);
                c[j][0] = 0.f; c[j][1] = 0.f;
#pragma unroll
                for (int mi = 0; mi < MT; ++mi)
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        if (kk.x > neg_inf()) c[j][0] += ex2(L[mi][j][2 * h] + G[j][0] - Mrow[mi][h] - kk.x);
                        if (kk.y > neg_inf()) c[j][1] += ex2(L[mi][j][2 * h + 1] + G[j][1] - Mrow[mi][h] - kk.y);
                    }
            }
            tot = block_columns<NT, false>(c, sRed, warp, lane);
            if (tid < r) sLam[tid] = sKap[tid] + lg2(tot);
            __syncthreads();
            if (tid == 0) *sFlag = 0;
        }
        bool bad = false;
#pragma unroll
        for (int j = 0; j < NT; ++j) {
            const float2 lam = *reinterpret_cast<const float2 *>(sLam + 8 * j + 2 * q);
            const float2 lb = *reinterpret_cast<const float2 *>(sLb + 8 * j + 2 * q);
            if (8 * j + 2 * q < r) { G[j][0] += lb.x - lam.x; bad |= !isfinite(G[j][0]); }
            if (8 * j + 2 * q + 1 < r) { G[j][1] += lb.y - lam.y; bad |= !isfinite(G[j][1]); }
        }
        if (bad && warp == 0 && g == 0) atomicOr(status, 1 /* LOT_DEV_NONFINITE */);
        ++it;
    }
    if (fast) {
#pragma unroll
        for (int j = 0; j < NT; ++j) {
            const float2 gg = *reinterpret_cast<const float2 *>(sG + 8 * j + 2 * q);
            G[j][0] = gg.x; G[j][1] = gg.y;
        }
    }
    __syncthreads();                                   // shared scratch is free for the next side
}

template <int NT, int MT>
__global__ void __launch_bounds__(kThreads, 1)
slice_forward_kernel(const SliceParams P)
{
    using PL = Plan<NT, MT>;
    extern __shared__ __align__(128) uint8_t smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, q = lane & 3;
    const int s = blockIdx.x, b = s / P.H, h = s % P.H;
    const int n = P.n, r = P.r;
    const int ntiles = (n + 15) / 16;
    int kv = n;
    if (P.key_len != nullptr) kv = min(max(__ldg(P.key_len + b), 0), n);
    uint8_t *sX = smem + PL::offX, *sV = smem + PL::offV, *sZ = smem + PL::offZ, *sWp = smem + PL::offWp;
    float *sWacc = reinterpret_cast<float *>(smem + PL::offWacc);
    float *sLb = reinterpret_cast<float *>(smem + PL::offLb);
    const size_t tok = (size_t)s * n * kD;

    // token rows of one tensor into a [RX][144-byte] buffer; rows beyond n are zero
    auto load_rows = [&](const __nv_bfloat16 *src, uint8_t *dst) {
        for (int idx = threadIdx.x; idx < ntiles * 16 * 8; idx += kThreads) {
            const int row = idx >> 3, ch = idx & 7;
            uint8_t *d = dst + row * kPitch + ch * 16;
            if (row < n) cp_async16(smem_addr(d), src + (size_t)row * kD + ch * 8);
            else *reinterpret_cast<uint4 *>(d) = make_uint4(0, 0, 0, 0);
        }
    };
    load_rows(P.k + tok, sX);
    load_rows(P.v + tok, sV);
    // the query rows are wanted after the key side is solved: have them in L2 by then
    for (int idx = threadIdx.x; idx < n; idx += kThreads)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(P.q + tok + (size_t)idx * kD));
    // pivots of this head, scaled to base-2 logit units, as bf16 hi + lo
    for (int idx = threadIdx.x; idx < PL::RP * (kD / 2); idx += kThreads) {
        const int t = idx / (kD / 2), c2 = (idx % (kD / 2)) * 2;
        float2 zz = make_float2(0.f, 0.f);
        if (t < r) zz = __ldg(reinterpret_cast<const float2 *>(P.z + ((size_t)h * r + t) * kD + c2));
        uint32_t hi, lo;
        split2(zz.x * P.scale, zz.y * P.scale, hi, lo);
        *reinterpret_cast<uint32_t *>(sZ + t * kPitch + c2 * 2) = hi;
        *reinterpret_cast<uint32_t *>(sZ + PL::RP * kPitch + t * kPitch + c2 * 2) = lo;
    }
    if (threadIdx.x < 64) {
        sLb[threadIdx.x] = (int)threadIdx.x < r ? lg2(__ldg(P.beta + h * r + threadIdx.x) * (float)max(kv, 1)) : 0.f;
        if (threadIdx.x == 0) *reinterpret_cast<volatile int *>(smem + PL::offFlag) = 0;
    }
    cp_async_wait_all();
    __syncthreads();

    float L[MT][NT][4];
    float G[NT][2];
    // ------------------------------------------------------------------ key side
    if (kv > 0) {
        logits<NT, MT>(L, sX, sZ, warp, lane, ntiles);
        solve<NT, MT>(L, G, smem, sX, sZ, warp, lane, ntiles, kv, r, P.T, P.status);
    } else {
        // no keys: nothing to transport; the output is zero (flagged), the key-side potentials stay at zero
#pragma unroll
        for (int mi = 0; mi < MT; ++mi)
#pragma unroll
            for (int j = 0; j < NT; ++j)
#pragma unroll
                for (int e = 0; e < 4; ++e) L[mi][j][e] = 0.f;
#pragma unroll
        for (int j = 0; j < NT; ++j) { G[j][0] = 0.f; G[j][1] = 0.f; }
        if (threadIdx.x == 0) atomicOr(P.status, 2 /* LOT_DEV_EMPTY */);
    }
    if (P.g2_out != nullptr && warp == 0 && g == 0) {
#pragma unroll
        for (int j = 0; j < NT; ++j)
#pragma unroll
            for (int e = 0; e < 2; ++e)
                if (8 * j + 2 * q + e < r) P.g2_out[(size_t)s * r + 8 * j + 2 * q + e] = G[j][e] * P.eps_ln2;
    }
    __syncthreads();                                   // every warp is done with K in sX
    // plan rows (row-stochastic; the key mass 1/kv goes into W') as bf16 hi + lo planes [token][pivot]
    {
        uint8_t *pl_hi = sX, *pl_lo = sX + PL::RX * PL::pitchP;
#pragma unroll
        for (int mi = 0; mi < MT; ++mi) {
            const int mt = warp + kWarps * mi;
            if (mt >= ntiles) continue;
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const int row = mt * 16 + g + 8 * hh;
#pragma unroll
                for (int j = 0; j < NT; ++j) {
                    uint32_t hi, lo;
                    split2(L[mi][j][2 * hh], L[mi][j][2 * hh + 1], hi, lo);
                    *reinterpret_cast<uint32_t *>(pl_hi + row * PL::pitchP + (8 * j + 2 * q) * 2) = hi;
                    *reinterpret_cast<uint32_t *>(pl_lo + row * PL::pitchP + (8 * j + 2 * q) * 2) = lo;
                }
            }
        }
    }
    __syncthreads();
    // W[t][c] = sum_j R2[j][t] v[j][c]: work item = (16 pivots, 16 channels, one share of the tokens)
    {
        constexpr int items = (PL::RP / 16) * 4, ksplit = kWarps / items;     // 4, 8 or 16 items
        const int item = warp % items, ks_id = warp / items;
        const int t0 = (item / 4) * 16, c0 = (item % 4) * 16;
        const int steps = ntiles;                                            // 16 tokens per step
        const int per = (steps + ksplit - 1) / ksplit;
        const int st0 = ks_id * per, st1 = min(st0 + per, steps);
        const uint32_t ph = smem_addr(sX), plo = ph + PL::RX * PL::pitchP, vb = smem_addr(sV);
        float acc[2][4] = {};
        const int mi4 = lane >> 3;
        for (int st = st0; st < st1; ++st) {
            const int j0 = st * 16;
            uint32_t ah[4], al[4], bv[4];
            const uint32_t aoff = (j0 + (lane & 7) + (mi4 >> 1) * 8) * PL::pitchP + (t0 + (mi4 & 1) * 8) * 2;
            ldsm_x4_t(ah, ph + aoff);
            ldsm_x4_t(al, plo + aoff);
            ldsm_x4_t(bv, vb + (j0 + (lane & 7) + (mi4 & 1) * 8) * kPitch + (c0 + (mi4 >> 1) * 8) * 2);
            mma16816(acc[0], ah, bv[0], bv[1]);
            mma16816(acc[0], al, bv[0], bv[1]);
            mma16816(acc[1], ah, bv[2], bv[3]);
            mma16816(acc[1], al, bv[2], bv[3]);
        }
        float *dst = sWacc + (size_t)ks_id * PL::RP * kD;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
            const int c = c0 + nt * 8 + 2 * q;
            *reinterpret_cast<float2 *>(dst + (t0 + g) * kD + c) = make_float2(acc[nt][0], acc[nt][1]);
            *reinterpret_cast<float2 *>(dst + (t0 + g + 8) * kD + c) = make_float2(acc[nt][2], acc[nt][3]);
        }
        __syncthreads();
        // W'^T[c][t] = W[t][c] / (kv beta_t) as bf16 hi + lo, two pivots per thread and step
        const float inv_kv = kv > 0 ? 1.f / (float)kv : 0.f;
        for (int idx = threadIdx.x; idx < kD * (PL::RP / 2); idx += kThreads) {
            const int c = idx % kD, t = (idx / kD) * 2;
            float w0 = 0.f, w1 = 0.f;
#pragma unroll
            for (int k2 = 0; k2 < ksplit; ++k2) {
                w0 += sWacc[((size_t)k2 * PL::RP + t) * kD + c];
                w1 += sWacc[((size_t)k2 * PL::RP + t + 1) * kD + c];
            }
            w0 = t < r ? w0 * inv_kv / __ldg(P.beta + h * r + t) : 0.f;
            w1 = t + 1 < r ? w1 * inv_kv / __ldg(P.beta + h * r + t + 1) : 0.f;
            uint32_t hi, lo;
            split2(w0, w1, hi, lo);
            *reinterpret_cast<uint32_t *>(sWp + c * PL::pitchP + t * 2) = hi;
            *reinterpret_cast<uint32_t *>(sWp + kD * PL::pitchP + c * PL::pitchP + t * 2) = lo;
        }
    }
    __syncthreads();                                   // plan planes consumed: sX is free for Q
    // ------------------------------------------------------------------ query side
    load_rows(P.q + tok, sX);
    if (threadIdx.x < 64) sLb[threadIdx.x] = (int)threadIdx.x < r ? lg2(__ldg(P.beta + h * r + threadIdx.x) * (float)n) : 0.f;
    cp_async_wait_all();
    __syncthreads();
    logits<NT, MT>(L, sX, sZ, warp, lane, ntiles);
    solve<NT, MT>(L, G, smem, sX, sZ, warp, lane, ntiles, n, r, P.T, P.status);
    if (P.g1_out != nullptr && warp == 0 && g == 0) {
#pragma unroll
        for (int j = 0; j < NT; ++j)
#pragma unroll
            for (int e = 0; e < 2; ++e)
                if (8 * j + 2 * q + e < r) P.g1_out[(size_t)s * r + 8 * j + 2 * q + e] = G[j][e] * P.eps_ln2;
    }
    // out[i][c] = sum_t R1[i][t] W'[t][c]: the plan rows are A fragments as they stand (hi + lo), W'^T gives B
    {
        const uint32_t wh = smem_addr(sWp), wl = wh + kD * PL::pitchP;
        __nv_bfloat16 *ob = P.out + tok;
#pragma unroll
        for (int mi = 0; mi < MT; ++mi) {
            const int mt = warp + kWarps * mi;
            if (mt >= ntiles) continue;
            float acc[kD / 8][4];
#pragma unroll
            for (int jn = 0; jn < kD / 8; ++jn)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[jn][e] = 0.f;
#pragma unroll
            for (int kk = 0; kk < NT / 2; ++kk) {
                uint32_t ah[4], al[4];
                split2(L[mi][2 * kk][0], L[mi][2 * kk][1], ah[0], al[0]);
                split2(L[mi][2 * kk][2], L[mi][2 * kk][3], ah[1], al[1]);
                split2(L[mi][2 * kk + 1][0], L[mi][2 * kk + 1][1], ah[2], al[2]);
                split2(L[mi][2 * kk + 1][2], L[mi][2 * kk + 1][3], ah[3], al[3]);
#pragma unroll
                for (int cp = 0; cp < kD / 16; ++cp) {
                    const uint32_t off = (cp * 16 + (lane & 7) + (lane >> 4) * 8) * PL::pitchP + (kk * 16 + ((lane >> 3) & 1) * 8) * 2;
                    uint32_t bh[4], bl[4];
                    ldsm_x4(bh, wh + off);
                    ldsm_x4(bl, wl + off);
                    mma16816(acc[2 * cp], ah, bh[0], bh[1]);
                    mma16816(acc[2 * cp], ah, bl[0], bl[1]);
                    mma16816(acc[2 * cp], al, bh[0], bh[1]);
                    mma16816(acc[2 * cp + 1], ah, bh[2], bh[3]);
                    mma16816(acc[2 * cp + 1], ah, bl[2], bl[3]);
                    mma16816(acc[2 * cp + 1], al, bh[2], bh[3]);
                }
            }
            const int r0 = mt * 16 + g, r1 = r0 + 8;
#pragma unroll
            for (int jn = 0; jn < kD / 8; ++jn) {
                const int c = 8 * jn + 2 * q;
                if (r0 < n) *reinterpret_cast<uint32_t *>(ob + (size_t)r0 * kD + c) = pack2(acc[jn][0], acc[jn][1]);
                if (r1 < n) *reinterpret_cast<uint32_t *>(ob + (size_t)r1 * kD + c) = pack2(acc[jn][2], acc[jn][3]);
            }
        }
    }
}

template <int NT, int MT>
cudaError_t launch(const SliceParams &P, int BH, cudaStream_t st)
{
    static std::mutex mu;
    static bool attr_set[64] = {};
    auto kern = slice_forward_kernel<NT, MT>;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!attr_set[dev]) {
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Plan<NT, MT>::total);
            if (e != cudaSuccess) return e;
            attr_set[dev] = true;
        }
    }
    kern<<<BH, kThreads, Plan<NT, MT>::total, st>>>(P);
    return cudaGetLastError();
}

} // namespace slice

bool slice_supported(int dtype, int n, int d, int r)
{
    if (dtype != 1 || d != slice::kD || r < 1 || r > 64 || n < 1 || n > 512) return false;
    const int rp = r <= 16 ? 16 : r <= 32 ? 32 : 64;
    return ((n + 15) / 16) * 16 * rp <= 16384;
}

cudaError_t slice_attention(const void *q, const void *k, const void *v, const float *z, const float *beta,
                            const int32_t *key_len, int B, int H, int n, int r, float eps, int iters, void *out,
                            float *g1_out, float *g2_out, int *status, cudaStream_t st)
{
    slice::SliceParams P{};
    P.q = static_cast<const __nv_bfloat16 *>(q); P.k = static_cast<const __nv_bfloat16 *>(k);
    P.v = static_cast<const __nv_bfloat16 *>(v); P.z = z; P.beta = beta; P.key_len = key_len;
    P.out = static_cast<__nv_bfloat16 *>(out); P.g1_out = g1_out; P.g2_out = g2_out; P.status = status;
    P.B = B; P.H = H; P.n = n; P.r = r; P.T = iters;
    P.scale = (float)(1.4426950408889634 / (double)eps);
    P.eps_ln2 = (float)((double)eps * 0.6931471805599453);
    cudaError_t e = cudaMemsetAsync(status, 0, sizeof(int), st);
    if (e != cudaSuccess) return e;
    const int BH = B * H;
    const int mt = n > 256 ? 2 : 1;
    if (r <= 16) return mt == 2 ? slice::launch<2, 2>(P, BH, st) : slice::launch<2, 1>(P, BH, st);
    if (r <= 32) return mt == 2 ? slice::launch<4, 2>(P, BH, st) : slice::launch<4, 1>(P, BH, st);
    return slice::launch<8, 1>(P, BH, st);
}

} // namespace lot
