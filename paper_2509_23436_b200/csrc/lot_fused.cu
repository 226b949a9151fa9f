// Fused tensor-core path of the LOT attention forward for bf16 tensors (sm_100a).
//
// The similarity matrices are never stored: every pass recomputes the logits of a 128-token
// tile with tcgen05.mma (bf16 tokens x pivots pre-scaled by log2(e)/eps and split into bf16
// hi + lo parts, f32 accumulation in TMEM), tokens staged by TMA.  One thread owns one token
// row of the TMEM accumulator, so the row log-sum-exp over the pivots (token update of the
// Sinkhorn iteration, Eq. (1)-(2) in scaling form) needs no cross-thread traffic, and the
// column sums over tokens (pivot update) are accumulated per thread over all tiles of a
// segment and reduced across threads once per segment.
//
// One launch per pass ("round"); a CTA owns a fixed range of tiles of both sides, split into
// segments = (slice, side).  Cross-CTA reductions are per-CTA partials merged in slot order by
// the last CTA to arrive on a ticket (no CTA ever waits for another).
//   SUM  rounds: both sides, one pivot update of G per round and (slice, side).
//   WRED round : key side, closing token update, W = Gamma2 V on tensor cores, W' = W / beta.
//   OUT  round : query side, closing token update, out = softmax-rows x W' on tensor cores.
// Warp roles: warp 0 TMA producer, warp 1 MMA issuer and TMEM owner, warps 2-9 two epilogue
// groups of 128 threads (group g takes the tiles of parity g and TMEM accumulator g).
#include "lot_common.cuh"
#include "lot_internal.h"
#include "lot_sm100.cuh"

#include <cuda.h>
#include <string.h>

namespace lot {
namespace fused {

using namespace sm100;

constexpr int kModeSum = 0, kModeWred = 1, kModeOut = 2;
constexpr int kThreads = 320;
constexpr int kEpiThreads = 256;
constexpr int kTileRows = 128;
constexpr int kPanelBytes = 128 * 128;   // 128 rows x 64 bf16 (one 128-byte-swizzled panel)
constexpr float kPlainFloor = 8.2718061e-25f;   // 2^-80: smallest column mass the plain sums may report

struct alignas(64) FusedParams {
    CUtensorMap tmQ, tmK, tmV;   // [BH][n][d] bf16, box 64 x 128 x 1
    CUtensorMap tmZ;             // [2H][RP][d] bf16 (hi, lo of scaled pivots), box 64 x RP x 1
    CUtensorMap tmW;             // [2BH][d][64] bf16 (hi, lo of W'^T), box 64 x d x 1
    const float *beta;           // [H][r]
    const int32_t *key_len;      // [B] or nullptr
    float *G;                    // [2][BH][RP] pivot potentials, base-2 units (side 0 = queries, 1 = keys)
    float *part;                 // [2][BH][maxslots][RP][2] column pairs per CTA slot
    unsigned *ticket;            // [2][BH]
    int *iter;                   // [2][BH] pivot updates done
    int *robust;                 // [2][BH] 1 = column sums carried as (kappa, S) pairs
    float *wpart;                // [BH][maxslots][128][d] per-slot W accumulators (rows 0-63 hi, 64-127 lo)
    __nv_bfloat16 *Wb;           // [BH][2][d][64] W'^T split hi/lo, pivot-contiguous
    unsigned *wticket;           // [BH]
    __nv_bfloat16 *out;          // [BH][n][d]
    float *g_nat;                // [2][BH][r] final potentials, natural-log units
    int *status;
    int B, H, n, r, T;
    int TPS;                     // tiles per slice = ceil(n / 128)
    int q;                       // tiles per CTA and side
    int maxslots;
    float eps_ln2;
};

// ---------------------------------------------------------------------------------------
// Segment enumeration: identical in every warp role of a CTA.
// ---------------------------------------------------------------------------------------
struct Seg {
    int s, side, b, h, nvalid, t0, t1, slot, nslots, robust, iter;
};

template <int MODE>
struct SegIter {
    const FusedParams &P;
    int u0, u1, s, s_end, side_idx;
    __device__ explicit SegIter(const FusedParams &p) : P(p)
    {
        const int NT = p.B * p.H * p.TPS;
        u0 = blockIdx.x * p.q;
        u1 = min(NT, u0 + p.q);
        s = u0 / p.TPS;
        s_end = (u1 - 1) / p.TPS;
        side_idx = 0;
    }
    __device__ bool next(Seg &g)
    {
        constexpr int nsides = MODE == kModeSum ? 2 : 1;
        const int BH = P.B * P.H;
        while (s <= s_end) {
            if (side_idx >= nsides) { side_idx = 0; ++s; continue; }
            const int side = MODE == kModeSum ? (side_idx == 0 ? 1 : 0) : (MODE == kModeWred ? 1 : 0);
            ++side_idx;
            g.s = s; g.side = side; g.b = s / P.H; g.h = s % P.H;
            g.nvalid = P.n;
            if (side == 1 && P.key_len != nullptr) g.nvalid = min(max(__ldg(P.key_len + g.b), 0), P.n);
            const int vt = (g.nvalid + kTileRows - 1) / kTileRows;
            g.t0 = max(u0 - s * P.TPS, 0);
            g.t1 = min(u1 - s * P.TPS, vt);
            if (g.t0 >= g.t1) continue;
            g.robust = 0; g.iter = 0;
            if (MODE == kModeSum) {
                g.iter = __ldcg(P.iter + side * BH + s);
                if (g.iter >= P.T) continue;
                g.robust = __ldcg(P.robust + side * BH + s);
            }
            const int c_lo = (s * P.TPS) / P.q, c_hi = (s * P.TPS + vt - 1) / P.q;
            g.slot = (int)blockIdx.x - c_lo;
            g.nslots = c_hi - c_lo + 1;
            return true;
        }
        return false;
    }
};

// ---------------------------------------------------------------------------------------
// Shared-memory plan
// ---------------------------------------------------------------------------------------
template <int DK, int MODE>
struct Plan {
    static constexpr int KB = DK / 64;                        // 64-column panels per token tile
    static constexpr int XS = MODE == kModeSum ? (DK == 64 ? 4 : 3) : (DK == 64 ? 3 : 2);
    static constexpr int XBYTES = KB * kPanelBytes;
    static constexpr int ZBYTES = 2 * KB * (64 * 128);        // hi, lo x panels of <= 64 pivot rows
    static constexpr int VS = MODE == kModeWred ? (DK == 64 ? 3 : 2) : 0;
    static constexpr int PBUFS = MODE == kModeSum ? 0 : (MODE == kModeWred && DK == 128 ? 1 : 2);
    static constexpr int PBYTES = MODE == kModeWred ? 2 * kPanelBytes : kPanelBytes;
    static constexpr int WBYTES = MODE == kModeOut ? 2 * DK * 128 : 0;
    static constexpr int offX = 0;
    static constexpr int offZ = offX + XS * XBYTES;
    static constexpr int offV = offZ + ZBYTES;
    static constexpr int offP = offV + VS * XBYTES;
    static constexpr int offW = offP + PBUFS * PBYTES;
    static constexpr int offBar = offW + WBYTES;              // 64 mbarriers
    static constexpr int offMisc = offBar + 64 * 8;
    static constexpr int offG = offMisc + 64;                 // float sG[2][64]
    static constexpr int offRed = offG + 2 * 64 * 4;          // float sRed[8][64][2]
    static constexpr int offKap = offRed + 8 * 64 * 2 * 4;    // float sKap[64][256]: per-thread exponents of the
    static constexpr int total = offKap + (MODE == kModeSum ? 64 * 256 * 4 : 0);   // robust (kappa, S) pairs
    static constexpr int dyn_bytes = total + 1024;            // slack for 1024-byte alignment
    static constexpr int tmem_cols = MODE == kModeSum ? 128 : (MODE == kModeWred ? 256 : (DK == 64 ? 256 : 512));
    static constexpr int colW = 128;                          // first TMEM column of the apply accumulators
};

enum BarId { bXFull = 0, bXEmpty = 4, bZFull = 8, bZEmpty = 9, bAccFull = 10, bAccEmpty = 12, bVFull = 14, bVEmpty = 18,
             bPFull = 22, bPEmpty = 24, bOFull = 26, bOEmpty = 28, bWFull = 30, bWEmpty = 31, bWqFull = 32, bWqEmpty = 33,
             bCount = 34 };

// sum-reduce acc[0..N) over the 32 lanes; afterwards lane L holds, in acc[0..N/32) (N >= 32), the
// totals of columns L*N/32 + j, or for N = 16 lane L holds column L/2 in acc[0].
template <int N>
__device__ __forceinline__ void warp_reduce_cols(float (&acc)[N], int lane)
{
    int cnt = N / 2;
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        if (cnt >= 1) {
            const bool up = (lane & off) != 0;
#pragma unroll
            for (int j = 0; j < N / 2; ++j) {
                if (j < cnt) {
                    float send = up ? acc[j] : acc[j + cnt];
                    float keep = up ? acc[j + cnt] : acc[j];
                    acc[j] = keep + __shfl_xor_sync(0xffffffffu, send, off);
                }
            }
            cnt >>= 1;
        } else {
            acc[0] += __shfl_xor_sync(0xffffffffu, acc[0], off);
        }
    }
}
// the same for (kappa, S) pairs
template <int N>
__device__ __forceinline__ void warp_reduce_pairs(float (&kap)[N], float (&S)[N], int lane)
{
    int cnt = N / 2;
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        if (cnt >= 1) {
            const bool up = (lane & off) != 0;
#pragma unroll
            for (int j = 0; j < N / 2; ++j) {
                if (j < cnt) {
                    float sk = up ? kap[j] : kap[j + cnt], ss = up ? S[j] : S[j + cnt];
                    float kk = up ? kap[j + cnt] : kap[j], ks = up ? S[j + cnt] : S[j];
                    float ok = __shfl_xor_sync(0xffffffffu, sk, off), os = __shfl_xor_sync(0xffffffffu, ss, off);
                    pair_merge(kk, ks, ok, os);
                    kap[j] = kk; S[j] = ks;
                }
            }
            cnt >>= 1;
        } else {
            float ok = __shfl_xor_sync(0xffffffffu, kap[0], off), os = __shfl_xor_sync(0xffffffffu, S[0], off);
            float kk = kap[0], ks = S[0];
            pair_merge(kk, ks, ok, os);
            kap[0] = kk; S[0] = ks;
        }
    }
}
// column held in slot j of lane `lane` after warp_reduce_*<N>
template <int N>
__device__ __forceinline__ int reduced_col(int lane, int j)
{
    return N >= 32 ? lane * (N / 32) + j : lane / 2;
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b)
{
    __nv_bfloat162 t = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&t);
}

// ---------------------------------------------------------------------------------------
// The round kernel
// ---------------------------------------------------------------------------------------
template <int DK, int RP, int MODE>
__global__ void __launch_bounds__(kThreads, 1)
fused_round_kernel(const __grid_constant__ FusedParams P)
{
    using PL = Plan<DK, MODE>;
    constexpr int KB = PL::KB;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + PL::offBar);
    volatile int *sAbort = reinterpret_cast<volatile int *>(smem + PL::offMisc);
    uint32_t *sTmem = reinterpret_cast<uint32_t *>(smem + PL::offMisc + 4);
    volatile int *sLast = reinterpret_cast<volatile int *>(smem + PL::offMisc + 8);
    volatile int *sFail = reinterpret_cast<volatile int *>(smem + PL::offMisc + 12);
    float *sG = reinterpret_cast<float *>(smem + PL::offG);
    float *sRed = reinterpret_cast<float *>(smem + PL::offRed);
    auto bar = [&](int id) { return smem_u32(bars + id); };
    // whole-warp wait with a warp-uniform verdict (every lane polls; the warp agrees on the result)
    auto wwait = [&](uint32_t b, uint32_t parity, volatile int *ab, int *st) {
        const bool r = mbar_wait(b, parity, ab, st);
        return __all_sync(0xffffffffu, r) != 0;
    };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int BH = P.B * P.H;

    if (threadIdx.x == 0) {
        for (int i = 0; i < 4; ++i) { mbar_init(bar(bXFull + i), 1); mbar_init(bar(bXEmpty + i), 1); }
        mbar_init(bar(bZFull), 1); mbar_init(bar(bZEmpty), 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(bAccFull + i), 1); mbar_init(bar(bAccEmpty + i), 4);
            mbar_init(bar(bPFull + i), 4); mbar_init(bar(bPEmpty + i), 1);
            mbar_init(bar(bOFull + i), 1); mbar_init(bar(bOEmpty + i), 4);
        }
        for (int i = 0; i < 4; ++i) { mbar_init(bar(bVFull + i), 1); mbar_init(bar(bVEmpty + i), 1); }
        mbar_init(bar(bWFull), 1); mbar_init(bar(bWEmpty), 8);
        mbar_init(bar(bWqFull), 1); mbar_init(bar(bWqEmpty), 1);
        *sAbort = 0;
        fence_barrier_init();
        prefetch_tensormap(&P.tmQ); prefetch_tensormap(&P.tmK); prefetch_tensormap(&P.tmZ);
        if (MODE == kModeWred) prefetch_tensormap(&P.tmV);
        if (MODE == kModeOut) prefetch_tensormap(&P.tmW);
    }
    if (warp == 1) { tmem_alloc(smem_u32(sTmem), PL::tmem_cols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *sTmem;

    constexpr uint32_t idesc_cost = make_idesc_bf16(128, RP, 0, 0);
    constexpr uint32_t idesc_w = make_idesc_bf16(128, DK, 1, 1);
    constexpr uint32_t idesc_o = make_idesc_bf16(128, DK, 0, 0);

    if (warp == 0) {
        // ======================= TMA producer =======================
        if (lane == 0) {
            SegIter<MODE> it(P);
            Seg g;
            int k = 0, zc = 0, prev_h = -1, segc = 0;
            bool ok = true;
            while (ok && it.next(g)) {
                if (g.h != prev_h) {
                    if (zc > 0) ok = mbar_wait(bar(bZEmpty), (zc - 1) & 1, sAbort, P.status);
                    if (!ok) break;
                    mbar_arrive_expect_tx(bar(bZFull), 2 * KB * RP * 128);
#pragma unroll
                    for (int part = 0; part < 2; ++part)
#pragma unroll
                        for (int kb = 0; kb < KB; ++kb)
                            tma_load_3d(sbase + PL::offZ + (part * KB + kb) * (64 * 128), &P.tmZ, bar(bZFull),
                                        kb * 64, 0, g.h * 2 + part);
                    ++zc; prev_h = g.h;
                }
                if (MODE == kModeOut) {
                    if (segc > 0) ok = mbar_wait(bar(bWqEmpty), (segc - 1) & 1, sAbort, P.status);
                    if (!ok) break;
                    mbar_arrive_expect_tx(bar(bWqFull), PL::WBYTES);
#pragma unroll
                    for (int part = 0; part < 2; ++part)
                        tma_load_3d(sbase + PL::offW + part * (DK * 128), &P.tmW, bar(bWqFull), 0, 0, g.s * 2 + part);
                }
                const CUtensorMap *xm = g.side ? &P.tmK : &P.tmQ;
                for (int t = g.t0; t < g.t1 && ok; ++t, ++k) {
                    const int st = k % PL::XS, ph = (k / PL::XS) & 1;
                    ok = mbar_wait(bar(bXEmpty + st), ph ^ 1, sAbort, P.status);
                    if (!ok) break;
                    mbar_arrive_expect_tx(bar(bXFull + st), PL::XBYTES);
#pragma unroll
                    for (int kb = 0; kb < KB; ++kb)
                        tma_load_3d(sbase + PL::offX + st * PL::XBYTES + kb * kPanelBytes, xm, bar(bXFull + st),
                                    kb * 64, t * kTileRows, g.s);
                    if constexpr (MODE == kModeWred) {
                        const int vs = k % PL::VS, vph = (k / PL::VS) & 1;
                        ok = mbar_wait(bar(bVEmpty + vs), vph ^ 1, sAbort, P.status);
                        if (!ok) break;
                        mbar_arrive_expect_tx(bar(bVFull + vs), PL::XBYTES);
#pragma unroll
                        for (int kb = 0; kb < KB; ++kb)
                            tma_load_3d(sbase + PL::offV + vs * PL::XBYTES + kb * kPanelBytes, &P.tmV, bar(bVFull + vs),
                                        kb * 64, t * kTileRows, g.s);
                    }
                }
                ++segc;
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ======================= MMA issuer =======================
        SegIter<MODE> it(P);
        Seg g;
        int k = 0, zc = 0, prev_h = -1, segc = 0;
        bool ok = true;
        int pend_k = -1, pend_first = 0;      // tile whose apply MMA is still to be issued

        auto issue_apply = [&](int kk, int first) {
            const int grp = kk & 1, j = kk >> 1;
            const int pb = PL::PBUFS == 2 ? grp : 0;
            const int pj = PL::PBUFS == 2 ? j : kk;
            if (ok) ok = wwait(bar(bPFull + pb), pj & 1, sAbort, P.status);
            if constexpr (MODE == kModeWred) {
                const int vs = kk % PL::VS, vph = (kk / PL::VS) & 1;
                if (ok) ok = wwait(bar(bVFull + vs), vph, sAbort, P.status);
                tc_fence_after();
                if (ok && lane == 0) {
                    const uint32_t pa = sbase + PL::offP + pb * PL::PBYTES;
                    const uint32_t va = sbase + PL::offV + vs * PL::XBYTES;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        uint64_t ad = make_smem_desc(pa + ks * 2048, kPanelBytes, 1024);
                        uint64_t bd = make_smem_desc(va + ks * 2048, kPanelBytes, 1024);
                        umma_bf16(tmem_base + PL::colW, ad, bd, idesc_w, (first && ks == 0) ? 0u : 1u);
                    }
                    umma_commit(bar(bPEmpty + pb));
                    umma_commit(bar(bVEmpty + vs));
                }
            } else {
                if (ok) ok = wwait(bar(bOEmpty + grp), (j & 1) ^ 1, sAbort, P.status);
                tc_fence_after();
                if (ok && lane == 0) {
                    const uint32_t pa = sbase + PL::offP + pb * PL::PBYTES;
#pragma unroll
                    for (int part = 0; part < 2; ++part)
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) {
                            uint64_t ad = make_smem_desc(pa + ks * 32, 16, 1024);
                            uint64_t bd = make_smem_desc(sbase + PL::offW + part * (DK * 128) + ks * 32, 16, 1024);
                            umma_bf16(tmem_base + PL::colW + grp * DK, ad, bd, idesc_o, (part | ks) ? 1u : 0u);
                        }
                    umma_commit(bar(bPEmpty + pb));
                    umma_commit(bar(bOFull + grp));
                }
            }
            __syncwarp();
        };

        while (ok && it.next(g)) {
            if (MODE != kModeSum && pend_k >= 0) { issue_apply(pend_k, pend_first); pend_k = -1; }
            if (MODE == kModeWred && segc > 0) {
                if (lane == 0) umma_commit(bar(bWFull));                      // W of the previous segment complete
                if (ok) ok = wwait(bar(bWEmpty), (segc - 1) & 1, sAbort, P.status);
            }
            if (g.h != prev_h) {
                if (zc > 0 && lane == 0) umma_commit(bar(bZEmpty));
                if (ok) ok = wwait(bar(bZFull), zc & 1, sAbort, P.status);
                ++zc; prev_h = g.h;
            }
            if (MODE == kModeOut) {
                if (segc > 0 && lane == 0) umma_commit(bar(bWqEmpty));
                if (ok) ok = wwait(bar(bWqFull), segc & 1, sAbort, P.status);
            }
            for (int t = g.t0; t < g.t1 && ok; ++t, ++k) {
                const int grp = k & 1, j = k >> 1;
                const int st = k % PL::XS, ph = (k / PL::XS) & 1;
                ok = wwait(bar(bXFull + st), ph, sAbort, P.status);
                if (ok) ok = wwait(bar(bAccEmpty + grp), (j & 1) ^ 1, sAbort, P.status);
                tc_fence_after();
                if (ok && lane == 0) {
                    const uint32_t xa = sbase + PL::offX + st * PL::XBYTES;
#pragma unroll
                    for (int part = 0; part < 2; ++part)
#pragma unroll
                        for (int kk = 0; kk < DK / 16; ++kk) {
                            const int kb = kk / 4, ko = (kk % 4) * 32;
                            uint64_t ad = make_smem_desc(xa + kb * kPanelBytes + ko, 16, 1024);
                            uint64_t bd = make_smem_desc(sbase + PL::offZ + (part * KB + kb) * (64 * 128) + ko, 16, 1024);
                            umma_bf16(tmem_base + grp * RP, ad, bd, idesc_cost, (part | kk) ? 1u : 0u);
                        }
                    umma_commit(bar(bXEmpty + st));
                    umma_commit(bar(bAccFull + grp));
                }
                __syncwarp();
                if (MODE != kModeSum) {
                    if (pend_k >= 0) issue_apply(pend_k, pend_first);
                    pend_k = k; pend_first = (t == g.t0);
                }
            }
            ++segc;
        }
        if (MODE != kModeSum && pend_k >= 0 && ok) { issue_apply(pend_k, pend_first); pend_k = -1; }
        if (MODE == kModeWred && segc > 0 && ok && lane == 0) umma_commit(bar(bWFull));
        __syncwarp();
    } else {
        // ======================= epilogue (8 warps) =======================
        const int ew = warp - 2, grp = ew >> 2, qd = warp & 3;
        const int etid = threadIdx.x - 64, gtid = etid & 127;
        const int rit = qd * 32 + lane;                                   // row inside the tile = TMEM lane
        const uint32_t lane_addr = tmem_base + ((uint32_t)(qd * 32) << 16);
        float *myG = sG + grp * 64;
        SegIter<MODE> it(P);
        Seg g;
        int k = 0, segc = 0;
        bool ok = true;

        float acc[RP];      // plain column sums, or S of the (kappa, S) pairs
        float *myKap = reinterpret_cast<float *>(smem + PL::offKap) + etid;   // kappa of column c at myKap[c * 256]

        while (it.next(g)) {
            named_bar_sync(1 + grp, 128);
            if (gtid < RP) myG[gtid] = gtid < P.r ? __ldcg(P.G + ((size_t)g.side * BH + g.s) * RP + gtid) : neg_inf();
            named_bar_sync(1 + grp, 128);
#pragma unroll
            for (int c = 0; c < RP; ++c) acc[c] = 0.f;
            if (MODE == kModeSum && g.robust) {
#pragma unroll
                for (int c = 0; c < RP; ++c) myKap[c * 256] = neg_inf();
            }

            for (int t = g.t0; t < g.t1; ++t, ++k) {
                if ((k & 1) != grp) continue;
                const int j = k >> 1;
                if (ok) ok = wwait(bar(bAccFull + grp), j & 1, sAbort, P.status);
                if (!ok) continue;
                tc_fence_after();
                const int row = t * kTileRows + rit;
                const bool valid = row < g.nvalid;
                if (MODE == kModeSum && g.robust) {
                    // ---- robust sums: three sweeps over the accumulator in 16-column chunks
                    float m = neg_inf();
#pragma unroll
                    for (int c0 = 0; c0 < RP; c0 += 16) {
                        float v[16];
                        tmem_ld16(lane_addr + grp * RP + c0, v);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 16; ++c) m = fmaxf(m, v[c] + myG[c0 + c]);
                    }
                    float s = 0.f;
#pragma unroll
                    for (int c0 = 0; c0 < RP; c0 += 16) {
                        float v[16];
                        tmem_ld16(lane_addr + grp * RP + c0, v);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 16; ++c) s += ex2(v[c] + myG[c0 + c] - m);
                    }
                    const float Mi = m + lg2(s);
#pragma unroll
                    for (int c0 = 0; c0 < RP; c0 += 16) {
                        float v[16];
                        tmem_ld16(lane_addr + grp * RP + c0, v);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 16; ++c)
                            if (valid && c0 + c < P.r) {
                                float kk = myKap[(c0 + c) * 256];
                                pair_add(kk, acc[c0 + c], (v[c] + myG[c0 + c] - m) - (Mi - m));
                                myKap[(c0 + c) * 256] = kk;
                            }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(bAccEmpty + grp));
                    continue;
                }
                float v[RP];
                tmem_ld<RP>(lane_addr + grp * RP, v);
                tmem_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(bAccEmpty + grp));
                float m = neg_inf();
#pragma unroll
                for (int c = 0; c < RP; ++c) { v[c] += myG[c]; m = fmaxf(m, v[c]); }
                float s = 0.f;
#pragma unroll
                for (int c = 0; c < RP; ++c) { v[c] = ex2(v[c] - m); s += v[c]; }
                const float inv = __fdividef(1.f, s);
                if (MODE == kModeSum) {
                    const float w = valid ? inv : 0.f;
#pragma unroll
                    for (int c = 0; c < RP; ++c) acc[c] = fmaf(v[c], w, acc[c]);
                } else {
                    // ---- write the plan tile as an MMA operand (128-byte rows, 16-byte chunks xor row%8)
                    const int pb = PL::PBUFS == 2 ? grp : 0;
                    const int pj = PL::PBUFS == 2 ? j : k;
                    ok = wwait(bar(bPEmpty + pb), (pj & 1) ^ 1, sAbort, P.status);
                    if (!ok) continue;
                    uint8_t *prow = smem + PL::offP + pb * PL::PBYTES + rit * 128;
                    const float w = MODE == kModeWred ? (valid ? inv : 0.f) : 1.f;
#pragma unroll
                    for (int c8 = 0; c8 < 8; ++c8) {
                        uint32_t hi[4], lo[4];
#pragma unroll
                        for (int e2 = 0; e2 < 4; ++e2) {
                            const int c = c8 * 8 + e2 * 2;
                            float a0 = c < RP ? v[c < RP ? c : 0] * w : 0.f;
                            float a1 = c + 1 < RP ? v[c + 1 < RP ? c + 1 : 0] * w : 0.f;
                            __nv_bfloat162 hh = __floats2bfloat162_rn(a0, a1);
                            hi[e2] = *reinterpret_cast<uint32_t *>(&hh);
                            if (MODE == kModeWred) lo[e2] = pack_bf16(a0 - __low2float(hh), a1 - __high2float(hh));
                        }
                        const int pc = (c8 ^ (rit & 7)) * 16;
                        *reinterpret_cast<uint4 *>(prow + pc) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                        if (MODE == kModeWred)
                            *reinterpret_cast<uint4 *>(prow + kPanelBytes + pc) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(bPFull + pb));
                    if (MODE == kModeOut) {
                        ok = wwait(bar(bOFull + grp), j & 1, sAbort, P.status);
                        if (!ok) continue;
                        tc_fence_after();
                        float o[DK];
                        tmem_ld<DK>(lane_addr + PL::colW + grp * DK, o);
                        tmem_wait_ld();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar(bOEmpty + grp));
                        if (row < P.n) {
                            __nv_bfloat16 *orow = P.out + ((size_t)g.s * P.n + row) * DK;
#pragma unroll
                            for (int c = 0; c < DK; c += 8) {
                                uint4 pk;
                                pk.x = pack_bf16(o[c] * inv, o[c + 1] * inv);
                                pk.y = pack_bf16(o[c + 2] * inv, o[c + 3] * inv);
                                pk.z = pack_bf16(o[c + 4] * inv, o[c + 5] * inv);
                                pk.w = pack_bf16(o[c + 6] * inv, o[c + 7] * inv);
                                *reinterpret_cast<uint4 *>(orow + c) = pk;
                            }
                        }
                    }
                }
            }

            // ------------------------------ segment end ------------------------------
            if (MODE == kModeSum) {
                constexpr int NJ = RP >= 32 ? RP / 32 : 1;
                if (g.robust) {
                    // slow path: merge the 32 lanes' pairs column by column
#pragma unroll
                    for (int c = 0; c < RP; ++c) {
                        float kk = myKap[c * 256], ss = acc[c];
#pragma unroll
                        for (int off = 16; off >= 1; off >>= 1) {
                            float ok2 = __shfl_xor_sync(0xffffffffu, kk, off), os2 = __shfl_xor_sync(0xffffffffu, ss, off);
                            pair_merge(kk, ss, ok2, os2);
                        }
                        if (lane == 0) { sRed[(ew * 64 + c) * 2] = kk; sRed[(ew * 64 + c) * 2 + 1] = ss; }
                    }
                } else {
                    warp_reduce_cols<RP>(acc, lane);
                    if (RP >= 32 || (lane & 1) == 0) {
#pragma unroll
                        for (int jx = 0; jx < NJ; ++jx) {
                            const int col = reduced_col<RP>(lane, jx);
                            sRed[(ew * 64 + col) * 2] = 0.f;
                            sRed[(ew * 64 + col) * 2 + 1] = acc[jx];
                        }
                    }
                }
                named_bar_sync(3, kEpiThreads);
                if (etid < RP) {
                    float kk = sRed[etid * 2], ss = sRed[etid * 2 + 1];
#pragma unroll
                    for (int w = 1; w < 8; ++w) {
                        if (g.robust) pair_merge(kk, ss, sRed[(w * 64 + etid) * 2], sRed[(w * 64 + etid) * 2 + 1]);
                        else ss += sRed[(w * 64 + etid) * 2 + 1];
                    }
                    float *dst = P.part + ((((size_t)g.side * BH + g.s) * P.maxslots + g.slot) * RP + etid) * 2;
                    __stcg(dst, kk);
                    __stcg(dst + 1, ss);
                    __threadfence();
                }
                named_bar_sync(3, kEpiThreads);
                if (etid == 0) {
                    __threadfence();
                    unsigned tk = atomicAdd(P.ticket + g.side * BH + g.s, 1u);
                    *sLast = (tk == (unsigned)g.nslots - 1u);
                    *sFail = 0;
                }
                named_bar_sync(3, kEpiThreads);
                if (*sLast) {
                    __threadfence();
                    float kk = g.robust ? neg_inf() : 0.f, ss = 0.f;
                    if (etid < P.r) {
                        for (int sl = 0; sl < g.nslots; ++sl) {
                            const float *src = P.part + ((((size_t)g.side * BH + g.s) * P.maxslots + sl) * RP + etid) * 2;
                            if (g.robust) pair_merge(kk, ss, __ldcg(src), __ldcg(src + 1));
                            else ss += __ldcg(src + 1);
                        }
                        if (!g.robust && !(ss >= kPlainFloor && ss <= 3.0e38f)) *sFail = 1;
                    }
                    named_bar_sync(3, kEpiThreads);
                    const int fail = *sFail;
                    if (!fail && etid < P.r) {
                        float *gp = P.G + ((size_t)g.side * BH + g.s) * RP + etid;
                        const float gn = *gp + lg2(__ldg(P.beta + g.h * P.r + etid) * (float)g.nvalid) - (kk + lg2(ss));
                        if (!isfinite(gn)) atomicOr(P.status, 1 /* LOT_DEV_NONFINITE */);
                        *gp = gn;
                        if (g.iter + 1 == P.T) P.g_nat[((size_t)g.side * BH + g.s) * P.r + etid] = gn * P.eps_ln2;
                    }
                    if (etid == 0) {
                        if (fail) P.robust[g.side * BH + g.s] = 1;
                        else P.iter[g.side * BH + g.s] = g.iter + 1;
                        P.ticket[g.side * BH + g.s] = 0u;
                    }
                }
            } else if (MODE == kModeWred) {
                // the W accumulator of this segment: every group reads half of the channels of its lanes
                if (ok) ok = wwait(bar(bWFull), segc & 1, sAbort, P.status);
                if (ok) {
                    tc_fence_after();
                    float w[DK / 2];
                    tmem_ld<DK / 2>(lane_addr + PL::colW + grp * (DK / 2), w);
                    tmem_wait_ld();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(bWEmpty));
                    float *dst = P.wpart + (((size_t)g.s * P.maxslots + g.slot) * 128 + rit) * DK + grp * (DK / 2);
#pragma unroll
                    for (int c = 0; c < DK / 2; c += 4) __stcg(reinterpret_cast<float4 *>(dst + c), make_float4(w[c], w[c + 1], w[c + 2], w[c + 3]));
                    __threadfence();
                }
                named_bar_sync(3, kEpiThreads);
                if (etid == 0) {
                    __threadfence();
                    unsigned tk = atomicAdd(P.wticket + g.s, 1u);
                    *sLast = (tk == (unsigned)g.nslots - 1u);
                }
                named_bar_sync(3, kEpiThreads);
                if (*sLast) {
                    __threadfence();
                    const float mass = g.nvalid > 0 ? 1.f / (float)g.nvalid : 0.f;
                    for (int idx = etid; idx < 64 * DK; idx += kEpiThreads) {
                        const int tt = idx / DK, c = idx % DK;
                        float sum = 0.f;
                        for (int sl = 0; sl < g.nslots; ++sl) {
                            const float *src = P.wpart + (((size_t)g.s * P.maxslots + sl) * 128) * DK + c;
                            sum += __ldcg(src + (size_t)tt * DK) + __ldcg(src + (size_t)(64 + tt) * DK);
                        }
                        float wv = tt < P.r ? sum * mass / __ldg(P.beta + g.h * P.r + tt) : 0.f;
                        __nv_bfloat16 hi = __float2bfloat16_rn(wv);
                        __nv_bfloat16 lo = __float2bfloat16_rn(wv - __bfloat162float(hi));
                        P.Wb[(((size_t)g.s * 2 + 0) * DK + c) * 64 + tt] = hi;
                        P.Wb[(((size_t)g.s * 2 + 1) * DK + c) * 64 + tt] = lo;
                    }
                    if (etid == 0) P.wticket[g.s] = 0u;
                }
            }
            ++segc;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, PL::tmem_cols);
    }
}

// ---------------------------------------------------------------------------------------
// Pivot preparation: Z' = Z * log2(e)/eps split into bf16 hi + lo, rows padded to RP with zeros.
// Also raises LOT_DEV_EMPTY for non-positive key lengths.
// ---------------------------------------------------------------------------------------
__global__ void zprep_kernel(const float *__restrict__ z, __nv_bfloat16 *__restrict__ zp, const int32_t *key_len,
                             int *status, int B, int H, int r, int RP, int d, float scale)
{
    const int total = H * RP * d;
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
        const int h = idx / (RP * d), rem = idx % (RP * d), t = rem / d, c = rem % d;
        float v = t < r ? z[((size_t)h * r + t) * d + c] * scale : 0.f;
        __nv_bfloat16 hi = __float2bfloat16_rn(v);
        __nv_bfloat16 lo = __float2bfloat16_rn(v - __bfloat162float(hi));
        zp[(((size_t)h * 2 + 0) * RP + t) * d + c] = hi;
        zp[(((size_t)h * 2 + 1) * RP + t) * d + c] = lo;
    }
    if (key_len != nullptr && blockIdx.x == 0)
        for (int b = threadIdx.x; b < B; b += blockDim.x)
            if (key_len[b] <= 0) atomicOr(status, 2 /* LOT_DEV_EMPTY */);
}

// ---------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// bf16 tensor [outer][rows][cols] (cols contiguous), box = 64 cols x box_rows rows x 1, 128-byte swizzle
static bool make_map(CUtensorMap *m, const void *base, int outer, int rows, int cols, int box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)outer};
    cuuint64_t strides[2] = {(cuuint64_t)cols * 2, (cuuint64_t)rows * cols * 2};
    cuuint32_t box[3] = {64u, (cuuint32_t)box_rows, 1u};
    cuuint32_t es[3] = {1u, 1u, 1u};
    CUresult rc = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, es,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return rc == CUDA_SUCCESS;
}

static int g_num_sms = 0;
static int num_sms()
{
    if (g_num_sms == 0) {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0)
            g_num_sms = v;
        else
            g_num_sms = 148;
    }
    return g_num_sms;
}

static inline size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }
static inline int pad_r(int r) { return r <= 16 ? 16 : (r <= 32 ? 32 : 64); }

} // namespace fused

bool fused_supported(int dtype, int d, int r)
{
    return dtype == 1 && d == 64 && r >= 1 && r <= 64;
}

void fused_geometry(int B, int H, int n, int *q, int *ctas, int *maxslots)
{
    const int TPS = (n + 127) / 128;
    const long long NT = (long long)B * H * TPS;
    const int sms = fused::num_sms();
    int qq = (int)((NT + sms - 1) / sms);
    if (qq < 1) qq = 1;
    *q = qq;
    *ctas = (int)((NT + qq - 1) / qq);
    *maxslots = (TPS - 1) / qq + 2;
}

FusedLayout fused_layout(int B, int H, int n, int d, int r)
{
    using fused::up256;
    FusedLayout L;
    const int BH = B * H, RP = fused::pad_r(r);
    int q, ctas, ms;
    fused_geometry(B, H, n, &q, &ctas, &ms);
    size_t o = 0;
    L.status = o; o += 256;
    L.G = o; o += up256((size_t)2 * BH * RP * 4);
    L.ticket = o; o += up256((size_t)2 * BH * 4);
    L.iter = o; o += up256((size_t)2 * BH * 4);
    L.robust = o; o += up256((size_t)2 * BH * 4);
    L.wticket = o; o += up256((size_t)BH * 4);
    L.gnat = o; o += up256((size_t)2 * BH * r * 4);
    L.Wb = o; o += up256((size_t)BH * 2 * d * 64 * 2);
    L.head_end = o;
    L.zprep = o; o += up256((size_t)H * 2 * RP * d * 2);
    L.part = o; o += up256((size_t)2 * BH * ms * RP * 2 * 4);
    L.wpart = o; o += up256((size_t)BH * ms * 128 * d * 4);
    L.total = o;
    return L;
}

template <int DK, int RP, int MODE>
static cudaError_t launch_round(const fused::FusedParams &P, int ctas, cudaStream_t st)
{
    using PL = fused::Plan<DK, MODE>;
    static bool attr_set = false;
    auto kern = fused::fused_round_kernel<DK, RP, MODE>;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, PL::dyn_bytes);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    kern<<<ctas, fused::kThreads, PL::dyn_bytes, st>>>(P);
    return cudaGetLastError();
}

template <int DK, int RP>
static cudaError_t run_rounds(const fused::FusedParams &P, int ctas, int iters, cudaStream_t st)
{
    cudaError_t e;
    // iters pivot updates, plus one spare round: a slice whose plain column sums underflowed in its
    // first round repeats that update with (kappa, S) pairs; every other CTA finds nothing to do.
    const int sum_rounds = iters > 0 ? iters + 1 : 0;
    for (int it = 0; it < sum_rounds; ++it)
        if ((e = launch_round<DK, RP, fused::kModeSum>(P, ctas, st)) != cudaSuccess) return e;
    if ((e = launch_round<DK, RP, fused::kModeWred>(P, ctas, st)) != cudaSuccess) return e;
    return launch_round<DK, RP, fused::kModeOut>(P, ctas, st);
}

cudaError_t fused_attention(const void *q, const void *k, const void *v, const float *z, const float *beta,
                            const int32_t *key_len, int B, int H, int n, int d, int r, float eps, int iters,
                            void *out, float *g1_out, float *g2_out, void *ws, cudaStream_t st)
{
    using namespace fused;
    const int BH = B * H, RP = pad_r(r);
    FusedLayout L = fused_layout(B, H, n, d, r);
    char *w = static_cast<char *>(ws);
    cudaError_t e;
    if ((e = cudaMemsetAsync(ws, 0, L.head_end, st)) != cudaSuccess) return e;

    FusedParams P;
    memset(&P, 0, sizeof(P));
    __nv_bfloat16 *zp = reinterpret_cast<__nv_bfloat16 *>(w + L.zprep);
    P.Wb = reinterpret_cast<__nv_bfloat16 *>(w + L.Wb);
    if (!make_map(&P.tmQ, q, BH, n, d, 128) || !make_map(&P.tmK, k, BH, n, d, 128) ||
        !make_map(&P.tmV, v, BH, n, d, 128) || !make_map(&P.tmZ, zp, 2 * H, RP, d, RP) ||
        !make_map(&P.tmW, P.Wb, 2 * BH, d, 64, d))
        return cudaErrorInvalidValue;
    P.beta = beta; P.key_len = key_len;
    P.G = reinterpret_cast<float *>(w + L.G);
    P.part = reinterpret_cast<float *>(w + L.part);
    P.ticket = reinterpret_cast<unsigned *>(w + L.ticket);
    P.iter = reinterpret_cast<int *>(w + L.iter);
    P.robust = reinterpret_cast<int *>(w + L.robust);
    P.wpart = reinterpret_cast<float *>(w + L.wpart);
    P.wticket = reinterpret_cast<unsigned *>(w + L.wticket);
    P.out = static_cast<__nv_bfloat16 *>(out);
    P.g_nat = reinterpret_cast<float *>(w + L.gnat);
    P.status = reinterpret_cast<int *>(w + L.status);
    P.B = B; P.H = H; P.n = n; P.r = r; P.T = iters;
    P.TPS = (n + 127) / 128;
    int ctas;
    fused_geometry(B, H, n, &P.q, &ctas, &P.maxslots);
    P.eps_ln2 = (float)((double)eps * 0.6931471805599453);

    const float scale = (float)(1.4426950408889634 / (double)eps);
    const int total = H * RP * d;
    zprep_kernel<<<(total + 255) / 256, 256, 0, st>>>(z, zp, key_len, P.status, B, H, r, RP, d, scale);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;

    if (RP == 16) e = run_rounds<64, 16>(P, ctas, iters, st);
    else if (RP == 32) e = run_rounds<64, 32>(P, ctas, iters, st);
    else e = run_rounds<64, 64>(P, ctas, iters, st);
    if (e != cudaSuccess) return e;

    const size_t gb = (size_t)BH * r * sizeof(float);
    if (g1_out && (e = cudaMemcpyAsync(g1_out, P.g_nat, gb, cudaMemcpyDeviceToDevice, st)) != cudaSuccess) return e;
    if (g2_out && (e = cudaMemcpyAsync(g2_out, P.g_nat + (size_t)BH * r, gb, cudaMemcpyDeviceToDevice, st)) != cudaSuccess) return e;
    return cudaSuccess;
}

int fused_launches(int iters) { return 1 + (iters > 0 ? iters + 1 : 0) + 2; }

} // namespace lot
