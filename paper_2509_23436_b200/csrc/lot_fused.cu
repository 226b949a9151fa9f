// Fused tensor-core path of the LOT attention forward for bf16 tensors (sm_100a): ONE persistent,
// cooperatively launched kernel runs every Sinkhorn pass and both apply stages.
//
// The n x r similarity matrices are never stored as such.  The first Sinkhorn pass, and every pass of
// a solve that cannot use the stored kernel (r <= 32, potentials spread over more than 64 binades, a
// column sum that underflowed), recomputes the logits of a 128-token tile with tcgen05.mma (bf16
// tokens x pivots pre-scaled by log2(e)/eps and split into bf16 hi + lo parts, f32 accumulation in
// TMEM), tokens staged by TMA.  For 32 < r <= 64 the first pass keeps 2^(L - rowmax), the stabilised
// Gibbs kernel of the scaling form of Eq. (1)-(2), as bf16 (staged in shared memory, one TMA store per
// warp and tile); the later passes stream it back and are the paper's matrix-vector scalings.  With
// the token potential eliminated the state of a solve is the pivot potential G:
//   token update : row log-sum-exp over the pivots (inside a thread quad / a thread)
//   pivot update : column sums over the tokens of the row-normalised tile, per (slice, side)
//
// Work split.  CTA c owns a fixed range of the slice-major tile list, for both sides, in every pass
// (with few slices: the same number of CTAs per slice, none spanning two); a (slice, side) range of it
// is a segment.  Pass order: T SUM passes (both sides, one pivot update each), one spare SUM pass for
// segments that had to repeat an update with (kappa, S) column pairs, the WRED pass (key side: closing
// token update, W = Gamma2 V on tensor cores) and the OUT pass (query side: closing token update,
// out = softmax-rows x W' on tensor cores, W' = W / beta).
//
// Warp roles: warp 0 TMA producer, warp 1 MMA issuer and TMEM owner, warp 2 the publisher, warp 3 the
// gatherer, warps 4-11 kGroups = 2 epilogue groups of 128 threads (two groups with 168 registers per
// thread measured faster than three with 128).  In the SUM passes the tile in ring stage st belongs to
// group st % kGroups: the epilogue waits on a stage's barrier by parity, which is only valid for a
// waiter that has seen the stage's previous fill complete.  In the apply passes the groups take turns.
// Producer and MMA issuer never depend on G, so they run ahead across pass boundaries; only the
// epilogue warps wait, per segment, for the potential of that attempt.
//
// Cross-CTA protocol (all CTAs are co-resident: cooperative launch, one CTA per SM).  The epilogue
// warps leave their column partials of a segment in shared memory and go on; the publisher warp adds
// them in warp order and writes the CTA's partial to its slot as 64-bit words that carry the attempt
// number beside the value, so a word is valid by itself and no fence or ticket is needed.  The
// gatherer warp of EVERY CTA that shares the (slice, side) polls all slots until their tags match,
// merges them in slot order (deterministic and identical in all CTAs, including the verdict that
// plain sums underflowed), updates its copy of G and hands it to its epilogue warps through shared
// memory.  W is merged the same way: every CTA writes its partial to its slot and raises a flag, and
// every CTA of the slice adds the slots itself, in slot order.  Every wait, on an mbarrier, on shared
// or on global memory, is bounded in time and raises LOT_DEV_TIMEOUT.
#include "lot_common.cuh"
#include "lot_internal.h"
#include "lot_sm100.cuh"

#include <cuda.h>
#include <string.h>
#include <mutex>
#include <type_traits>

namespace lot {
namespace fused {

using namespace sm100;

constexpr int kPhaseSum = 0, kPhaseWred = 1, kPhaseOut = 2;
constexpr int kGroups = 2;                        // epilogue groups of four warps (one per TMEM lane quarter)
constexpr int kEpiWarps = kGroups * 4;
constexpr int kWGroups = kGroups == 4 ? 4 : (kGroups >= 2 ? 2 : 1);    // groups that read the W accumulator out (64 / kWGroups columns each)
constexpr int kEpiThreads = kGroups * 128;
constexpr int kThreads = 128 + kEpiThreads;        // warps 0-3: producer, MMA issuer, publisher, gatherer; then the epilogue
constexpr int kMaxLoc = 16;                      // (slice, side) states of a CTA cached in shared memory
constexpr int kTileRows = 128;
constexpr int kDK = 64;                          // head dimension of this path
constexpr int kStageBytes = kTileRows * kDK * 2; // one token tile: 128 rows x 64 bf16, 128-byte swizzled
constexpr int kStages = 6;
constexpr int kLock = 4;                         // rows of a stored-kernel tile a thread advances in step
constexpr float kPlainFloor = 8.2718061e-25f;    // 2^-80: smallest column mass the plain sums may report

struct alignas(64) FusedParams {
    CUtensorMap tmQ, tmK, tmV;   // [BH][n][64] bf16, box 64 x 128 x 1
    CUtensorMap tmZ;             // [2H][RP][64] bf16 (hi, lo of scaled pivots), box 64 x RP x 1
    CUtensorMap tmKt;            // [2BH][npad][64] bf16 stored Gibbs kernel (r > 32 only), box 64 x 128 x 1
    CUtensorMap tmKtS;           // the same tensor with box 64 x 32 x 1: a warp's rows of a tile, for the store
    const float *beta;           // [H][r]
    const int32_t *key_len;      // [B] or nullptr
    __nv_bfloat16 *Kt;           // [2][BH][npad][64]: 2^(L_it - rowmax_i L), written by the first pass, or nullptr
    int npad;                    // TPS * 128
    float *G;                    // [2][BH][RP] pivot potentials, base-2 units (side 0 = queries, 1 = keys)
    unsigned long long *part;    // [2 attempt parities][2][BH][maxslots][RP][2] tagged words per CTA slot: (kappa, tag), (S, tag)
    int *epoch;                  // [2][BH] attempts finished (used for segments beyond the shared-memory cache)
    int *iter;                   // [2][BH] pivot updates done
    int *robust;                 // [2][BH] 1 = column sums carried as (kappa, S) pairs (sticky)
    float *wpart;                // [BH][maxslots][64 channels][64 pivots] per-slot partial of W^T = (Gamma2 V)^T
    int *wflag;                  // [BH][maxslots] 1 = that slot's partial is complete
    __nv_bfloat16 *out;          // [BH][n][64]
    float *g1_out, *g2_out;      // [BH][r] final potentials, natural-log units, or nullptr
    const unsigned *redo;        // not nullptr: run only if *redo == redo_tag (a call that repeats a resident launch)
    unsigned redo_tag;
    int ext_apply;               // 1: the apply stages run as separate kernels from the stored Gibbs kernel (lot_apply.cu);
                                 // this kernel applies only the slices whose stored kernel cannot carry the final potentials
    int *decision;               // [2][BH] per (side, slice), zero at the start: 1 = stored kernel good to the end, 2 = not
    int *status;
    int B, H, n, r, T;
    int TPS;                     // tiles per slice = ceil(n / 128)
    int q;                       // tiles per CTA and side (contiguous mapping)
    int cps;                     // > 0: aligned mapping, this many CTAs per slice, none spanning two slices
    int maxslots;
    float eps_ln2;
};

// ---------------------------------------------------------------------------------------
// Schedule: the same enumeration in every warp role of a CTA (it depends on launch constants
// and key_len only).
// ---------------------------------------------------------------------------------------
struct Seg {
    int phase, attempt, extra, s, side, b, h, nvalid, t0, t1, slot, nslots, li;
};

// Tile range [u0, u1) of a CTA in the slice-major tile list.  Aligned mapping: cps CTAs split every slice evenly, so
// that no CTA works on two slices; contiguous mapping: q tiles per CTA regardless of slice borders.
__device__ __forceinline__ void cta_range(const FusedParams &P, int cta, int &u0, int &u1)
{
    if (P.cps > 0) {
        const int s = cta / P.cps, j = cta % P.cps;
        u0 = s * P.TPS + (j * P.TPS) / P.cps;
        u1 = s * P.TPS + ((j + 1) * P.TPS) / P.cps;
    } else {
        u0 = cta * P.q;
        u1 = min(P.B * P.H * P.TPS, u0 + P.q);
    }
}
// First CTA and number of CTAs that hold valid tiles [0, vt) of slice s.
__device__ __forceinline__ void slice_slots(const FusedParams &P, int s, int vt, int &c_lo, int &nslots)
{
    if (P.cps > 0) {
        c_lo = s * P.cps;
        nslots = min(P.cps, (vt * P.cps + P.TPS - 1) / P.TPS);
    } else {
        c_lo = (s * P.TPS) / P.q;
        nslots = (s * P.TPS + vt - 1) / P.q - c_lo + 1;
    }
}

// The static part of a (slice, side) of this CTA: what does not change from pass to pass.
__device__ __forceinline__ bool seg_static(const FusedParams &P, int u0, int u1, int s_lo, int s, int side, Seg &g)
{
    g.s = s; g.side = side; g.b = s / P.H; g.h = s % P.H;
    g.li = (s - s_lo) * 2 + (side ? 0 : 1);         // index among this CTA's segments of one pass
    g.nvalid = P.n;
    if (side == 1 && P.key_len != nullptr) g.nvalid = min(max(__ldg(P.key_len + g.b), 0), P.n);
    const int vt = (g.nvalid + kTileRows - 1) / kTileRows;
    g.t0 = max(u0 - s * P.TPS, 0);
    g.t1 = min(u1 - s * P.TPS, vt);
    int c_lo;
    slice_slots(P, s, vt, c_lo, g.nslots);
    g.slot = (int)blockIdx.x - c_lo;
    return g.t0 < g.t1;
}
constexpr int kSegInts = 10;   // table entry: s, side, b, h, nvalid, t0, t1, slot, nslots, (unused)

// Enumeration of (pass, segment).  With at most kMaxLoc segments per pass the static parts come from a table in
// shared memory filled once per CTA (no integer division on the way); otherwise they are recomputed.
struct Sched {
    const FusedParams &P;
    const int *tab;
    int u0, u1, s_lo, s_hi, nloc, pass, cur;
    __device__ __forceinline__ Sched(const FusedParams &p, const int *table) : P(p), tab(table)
    {
        cta_range(p, blockIdx.x, u0, u1);
        s_lo = u0 / p.TPS;
        s_hi = (u1 - 1) / p.TPS;
        nloc = 2 * (s_hi - s_lo + 1);
        if (nloc > kMaxLoc) tab = nullptr;
        pass = p.T == 0 ? 1 : 0;       // passes 0..T-1 SUM, T spare SUM, T+1 WRED, T+2 OUT
        cur = 0;
    }
    __device__ __forceinline__ bool next(Seg &g)
    {
        for (;;) {
            if (pass > P.T + 2) return false;
            if (cur >= nloc) { cur = 0; ++pass; continue; }
            const int li = cur++;
            const int side = (li & 1) ? 0 : 1;                 // key side first
            const int phase = pass <= P.T ? kPhaseSum : (pass == P.T + 1 ? kPhaseWred : kPhaseOut);
            if ((phase == kPhaseWred && side == 0) || (phase == kPhaseOut && side == 1)) continue;
            if (tab != nullptr) {
                const int *e = tab + li * kSegInts;
                if (e[5] >= e[6]) continue;
                g.s = e[0]; g.side = e[1]; g.b = e[2]; g.h = e[3]; g.nvalid = e[4]; g.t0 = e[5]; g.t1 = e[6];
                g.slot = e[7]; g.nslots = e[8]; g.li = li;
            } else if (!seg_static(P, u0, u1, s_lo, s_lo + (li >> 1), side, g)) {
                continue;
            }
            g.phase = phase; g.attempt = pass; g.extra = (phase == kPhaseSum && pass == P.T);
            return true;
        }
    }
};

// ---------------------------------------------------------------------------------------
// Shared-memory plan
// ---------------------------------------------------------------------------------------
struct Plan {
    static constexpr int ZBYTES = 2 * (64 * 128);              // hi, lo panels of <= 64 pivot rows
    static constexpr int PBYTES = 2 * kStageBytes;             // plan tile as MMA operand: hi and lo panels
    static constexpr int WBYTES = 2 * kDK * 128;               // W'^T hi, lo
    static constexpr int offX = 0;
    static constexpr int offZ = offX + kStages * kStageBytes;  // two pivot buffers
    static constexpr int offP = offZ + 2 * ZBYTES;             // two plan buffers
    static constexpr int offW = offP + 2 * PBYTES;
    static constexpr int offBar = offW + WBYTES;               // 64 mbarriers
    static constexpr int offMisc = offBar + 64 * 8;            // abort flag, TMEM base, flags
    static constexpr int offG = offMisc + 128;                 // float sG[kGroups][64]
    static constexpr int offGc = offG + kGroups * 64 * 4;      // float sGc[kMaxLoc][64]: this CTA's copy of the potentials
    static constexpr int offState = offGc + kMaxLoc * 64 * 4;  // int sDone, sIter, sRobust, sResFirst, sResLast, sDec [kMaxLoc]
    static constexpr int offSeg = offState + 6 * kMaxLoc * 4;  // int sSeg[kMaxLoc][kSegInts]: static parts of the segments
    static constexpr int offWt = offSeg + kMaxLoc * kSegInts * 4; // float sWt[kMaxLoc][64]: weights 2^(G - max G) of the stored-kernel passes
    static constexpr int total = offWt + kMaxLoc * 64 * 4;
    // float sPart[2][kEpiWarps][64][2], the per-warp column pairs of the SUM passes, lives in the first plan buffer
    // (free until the WRED pass; the epilogue waits for the publisher's last read before it writes a plan tile)
    static constexpr int offPart = offP;
    // the second plan buffer is, in the first pass, where every epilogue warp stages its 32 rows of a stored-kernel
    // tile (4 KB, 128-byte swizzled like the tile itself) for the TMA store
    static constexpr int offKtStage = offP + PBYTES;
    static_assert(kEpiWarps * 32 * 128 <= PBYTES, "staging of the stored kernel must fit a plan buffer");
    static constexpr int dyn_bytes = total + 1024;             // slack for 1024-byte alignment
    static constexpr int tmem_cols = 512;
    static constexpr int colW = 256;                           // W accumulator (WRED): 64 columns
    static constexpr int colO = 320;                           // two output accumulators (OUT): 2 x 64 columns
};

enum BarId { bXFull = 0, bXEmpty = 8, bZFull = 16, bZEmpty = 18, bAccFull = 20, bAccEmpty = 24, bPFull = 28, bPEmpty = 30,
             bOFull = 32, bOEmpty = 34, bWFull = 36, bWEmpty = 37, bWqFull = 38, bWqEmpty = 39, bSegFull = 40, bSegEmpty = 42,
             bREmpty = 44,   // stage released by the four warps that read a stored-kernel tile (bXEmpty: by an MMA commit)
             bCount = 52 };

__device__ __forceinline__ uint32_t pack_bf16(float a, float b)
{
    __nv_bfloat162 t = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&t);
}
__device__ __forceinline__ float max3(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ int ld_acquire(const int *p)
{
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release(int *p, int v)
{
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// Bounded wait until *p >= want (one thread polls).
__device__ __forceinline__ bool poll_ge(const int *p, int want, volatile int *abort_flag, int *status)
{
    if (*abort_flag) return false;
    uint64_t t0 = 0;
    for (uint32_t it = 0;; ++it) {
        if (ld_acquire(p) >= want) return true;
        if ((it & 31u) == 31u) {
            if (*abort_flag) return false;
            const uint64_t now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitLimitNs) break;
        }
        __nanosleep(32);
    }
    *abort_flag = 1;
    atomicOr(status, 4 /* LOT_DEV_TIMEOUT */);
    return false;
}

// The same on a shared-memory word written by another warp of this CTA.
__device__ __forceinline__ bool spin_ge(volatile int *p, int want, volatile int *abort_flag, int *status)
{
    if (*abort_flag) return false;
    uint64_t t0 = 0;
    for (uint32_t it = 0;; ++it) {
        if (*p >= want) return true;
        if ((it & 255u) == 255u) {
            if (*abort_flag) return false;
            const uint64_t now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitLimitNs) break;
        }
    }
    *abort_flag = 1;
    atomicOr(status, 4 /* LOT_DEV_TIMEOUT */);
    return false;
}
__device__ __forceinline__ void st_tagged(unsigned long long *p, float a, float b, unsigned tag)
{
    const unsigned long long w0 = ((unsigned long long)tag << 32) | __float_as_uint(a);
    const unsigned long long w1 = ((unsigned long long)tag << 32) | __float_as_uint(b);
    asm volatile("st.relaxed.gpu.global.v2.b64 [%0], {%1, %2};" ::"l"(p), "l"(w0), "l"(w1) : "memory");
}
__device__ __forceinline__ void ld_tagged(const unsigned long long *p, unsigned long long &w0, unsigned long long &w1)
{
    asm volatile("ld.relaxed.gpu.global.v2.b64 {%0, %1}, [%2];" : "=l"(w0), "=l"(w1) : "l"(p) : "memory");
}

// Sum a[0..15] over the 8 lanes that share (lane & 3), halving the live set in every round (14 shuffles instead of
// 48).  Afterwards every lane holds in a[0], a[1] the totals of entries b, b + 1; b is returned.
template <int N>
__device__ __forceinline__ int quad_col_reduce16(float (&a)[N], int lane)
{
    if constexpr (N == 16) {
    {
        const bool up = (lane & 16) != 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float send = up ? a[j] : a[j + 8], keep = up ? a[j + 8] : a[j];
            a[j] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
        }
    }
    {
        const bool up = (lane & 8) != 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float send = up ? a[j] : a[j + 4], keep = up ? a[j + 4] : a[j];
            a[j] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
        }
    }
    {
        const bool up = (lane & 4) != 0;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const float send = up ? a[j] : a[j + 2], keep = up ? a[j + 2] : a[j];
            a[j] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
        }
    }
    }
    return 8 * ((lane >> 4) & 1) + 4 * ((lane >> 3) & 1) + 2 * ((lane >> 2) & 1);
}

// Quad-layout TMEM load (16 lanes x RP columns): thread L of the warp gets, in v[rep*4 + k],
// lane L/4 + 8*(k/2) and column rep*8 + 2*(L%4) + (k%2) of the 16-lane block at taddr.
template <int RP>
__device__ __forceinline__ void tmem_ld_quad(uint32_t taddr, float *v)
{
    uint32_t *r = reinterpret_cast<uint32_t *>(v);
    if constexpr (RP == 64) {
        asm volatile("tcgen05.ld.sync.aligned.16x256b.x8.b32 "
                     "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                     "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                     : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                       "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                       "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                       "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                     : "r"(taddr) : "memory");
    } else if constexpr (RP == 32) {
        asm volatile("tcgen05.ld.sync.aligned.16x256b.x4.b32 "
                     "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                     : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                       "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                     : "r"(taddr) : "memory");
    } else {
        static_assert(RP == 16, "pivot padding");
        asm volatile("tcgen05.ld.sync.aligned.16x256b.x2.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                     : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                     : "r"(taddr) : "memory");
    }
}

// ---------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------
// EXT: the variant whose apply stages may be left to the kernels of lot_apply.cu (P.ext_apply); the plain variant
// carries none of that code.
template <int RP, bool EXT>
__global__ void __launch_bounds__(kThreads, 1)
fused_forward_kernel(const __grid_constant__ FusedParams P)
{
    using PL = Plan;
    constexpr int DK = kDK;
    constexpr int NC = RP / 4;          // columns per thread in the quad layout
    if (P.redo != nullptr && *reinterpret_cast<const volatile unsigned *>(P.redo) != P.redo_tag) return;   // grid-uniform
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + PL::offBar);
    volatile int *sAbort = reinterpret_cast<volatile int *>(smem + PL::offMisc);
    uint32_t *sTmem = reinterpret_cast<uint32_t *>(smem + PL::offMisc + 4);
    float *sG = reinterpret_cast<float *>(smem + PL::offG);
    float *sPart = reinterpret_cast<float *>(smem + PL::offPart);
    float *sGc = reinterpret_cast<float *>(smem + PL::offGc);
    volatile int *sDone = reinterpret_cast<volatile int *>(smem + PL::offState);
    volatile int *sIter = sDone + kMaxLoc;
    volatile int *sRobust = sIter + kMaxLoc;
    // Attempts sResFirst[li] .. sResLast[li] of a segment read the stored Gibbs kernel (INT_MAX = not known yet).  There is
    // one such run per segment, and both ends are written before the attempt they first matter for is released, so a
    // warp that asks late about an old attempt (the MMA issuer has nothing to do in these passes) still gets that
    // attempt's answer.
    volatile int *sResFirst = sRobust + kMaxLoc;
    volatile int *sResLast = sResFirst + kMaxLoc;
    // 1 = the stored kernel of this segment serves the apply kernels, 2 = it does not (written with the last pivot update)
    volatile int *sDec = sResLast + kMaxLoc;
    volatile int *sPubDone = reinterpret_cast<volatile int *>(smem + PL::offMisc + 12);
    int *sSeg = reinterpret_cast<int *>(smem + PL::offSeg);
    // Wait until `need` attempts of local segment li (global index idx) are complete: 0 = gave up, else
    // 1 + robust flag + 2 * (the attempt reads the stored Gibbs kernel)
    auto seg_state = [&](int li, int idx, int need) -> int {
        if (li < kMaxLoc)
            return spin_ge(sDone + li, need, sAbort, P.status)
                       ? 1 + sRobust[li] + 2 * (need >= sResFirst[li] && need <= sResLast[li] ? 1 : 0) : 0;
        return poll_ge(P.epoch + idx, need, sAbort, P.status) ? 1 + __ldcg(P.robust + idx) : 0;
    };
    auto bar = [&](int id) { return smem_u32(bars + id); };
    // whole-warp wait with a warp-uniform verdict
    auto wwait = [&](uint32_t b, uint32_t parity) {
        const bool r = mbar_wait(b, parity, sAbort, P.status);
        return __all_sync(0xffffffffu, r) != 0;
    };

    // the same for two barriers whose first tries are in flight together
    auto wwait2 = [&](uint32_t b0, uint32_t p0, uint32_t b1, uint32_t p1) {
        const bool r0 = mbar_try_wait(b0, p0);
        const bool r1 = mbar_try_wait(b1, p1);
        if (__all_sync(0xffffffffu, r0 && r1)) return true;
        return wwait(b0, p0) && wwait(b1, p1);
    };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int BH = P.B * P.H;
    // With the apply stages in their own kernels: does this kernel still apply slice g.s?  Only if the stored kernel of
    // one of its sides cannot carry the final potentials.  A side of which this block holds tiles answers from shared
    // memory once its last pivot update is in; the other side's answer is polled from global memory.  (One thread.)
    // Returns 0 = gave up, 1 = skip the segment, 2 = apply it here.
    auto apply_here = [&](const Seg &g, int s_lo) -> int {
        if (!EXT || !P.ext_apply) return 2;
        int verdict = 1;
        for (int side = 0; side < 2; ++side) {
            const int li = (g.s - s_lo) * 2 + (side ? 0 : 1);
            const int *e = sSeg + li * kSegInts;
            int d;
            if (e[5] < e[6]) {
                if (!spin_ge(sIter + li, P.T, sAbort, P.status)) return 0;
                d = sDec[li];
            } else if (side == 1 && P.key_len != nullptr && __ldg(P.key_len + g.b) <= 0) {
                d = 1;                      // no keys at all: nothing updates that side; the apply kernels write the zeros
            } else {
                if (!poll_ge(P.decision + side * BH + g.s, 1, sAbort, P.status)) return 0;
                d = ld_acquire(P.decision + side * BH + g.s);
            }
            if (d == 2) verdict = 2;
        }
        return verdict;
    };

    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) { mbar_init(bar(bXFull + i), 1); mbar_init(bar(bXEmpty + i), 1); mbar_init(bar(bREmpty + i), 4); }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(bZFull + i), 1); mbar_init(bar(bZEmpty + i), 1);
            mbar_init(bar(bPFull + i), 4); mbar_init(bar(bPEmpty + i), 1);
            mbar_init(bar(bOFull + i), 1); mbar_init(bar(bOEmpty + i), 4);
        }
        for (int i = 0; i < kGroups; ++i) { mbar_init(bar(bAccFull + i), 1); mbar_init(bar(bAccEmpty + i), 4); }
        mbar_init(bar(bWFull), 1); mbar_init(bar(bWEmpty), kEpiWarps);
        mbar_init(bar(bWqFull), kEpiWarps); mbar_init(bar(bWqEmpty), 1);
        for (int i = 0; i < 2; ++i) { mbar_init(bar(bSegFull + i), kEpiWarps); mbar_init(bar(bSegEmpty + i), 1); }
        *sAbort = 0;
        *sPubDone = 0;
        fence_barrier_init();
        prefetch_tensormap(&P.tmQ); prefetch_tensormap(&P.tmK); prefetch_tensormap(&P.tmZ); prefetch_tensormap(&P.tmV);
        if (P.Kt != nullptr) { prefetch_tensormap(&P.tmKt); prefetch_tensormap(&P.tmKtS); }
    }
    if (warp == 1) { tmem_alloc(smem_u32(sTmem), PL::tmem_cols); tmem_relinquish(); }
    for (int i = threadIdx.x; i < kMaxLoc * 64; i += kThreads) sGc[i] = 0.f;
    if (threadIdx.x < 3 * kMaxLoc) sDone[threadIdx.x] = 0;
    else if (threadIdx.x < 5 * kMaxLoc) sDone[threadIdx.x] = 0x7fffffff;
    else if (threadIdx.x < 6 * kMaxLoc) sDone[threadIdx.x] = 0;
    if (threadIdx.x >= 128 && threadIdx.x < 128 + kMaxLoc) {
        // segment table: one thread per (slice, side) of this CTA
        const int li = threadIdx.x - 128;
        int u0, u1;
        cta_range(P, blockIdx.x, u0, u1);
        const int s_lo = u0 / P.TPS, s_hi = (u1 - 1) / P.TPS;
        int *e = sSeg + li * kSegInts;
        e[5] = 0; e[6] = 0;
        if (li < 2 * (s_hi - s_lo + 1)) {
            Seg g;
            seg_static(P, u0, u1, s_lo, s_lo + (li >> 1), (li & 1) ? 0 : 1, g);
            e[0] = g.s; e[1] = g.side; e[2] = g.b; e[3] = g.h; e[4] = g.nvalid; e[5] = g.t0; e[6] = g.t1;
            e[7] = g.slot; e[8] = g.nslots;
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *sTmem;

    constexpr uint32_t idesc_cost = make_idesc_bf16(128, RP, 0, 0);
    constexpr uint32_t idesc_w = make_idesc_bf16(128, DK, 1, 1);
    constexpr uint32_t idesc_o = make_idesc_bf16(128, DK, 0, 0);

    if (warp < 4) {
    if (warp == 0) {
        // ======================= TMA producer (one lane) =======================
        if (lane == 0) {
            Sched it(P, sSeg);
            Seg g;
            int kx = 0, ztag[2] = {-1, -1}, zuse[2] = {0, 0};
            bool ok = true;
            // A stage is handed back either by an MMA commit (bXEmpty) or by the readers of a stored-kernel tile
            // (bREmpty): remember per stage which one its last use ends with and how often each has happened.
            uint32_t used = 0, lastres = 0, xpar = 0, rpar = 0;     // bit st: used at all / last use was a kernel tile /
                                                                    // parity of the commit-released / reader-released uses
            auto acquire_stage = [&](int st, bool res) -> bool {
                bool w = true;
                if (used & (1u << st)) {
                    if (lastres & (1u << st)) w = mbar_wait(bar(bREmpty + st), ((rpar >> st) & 1) ^ 1, sAbort, P.status);
                    else w = mbar_wait(bar(bXEmpty + st), ((xpar >> st) & 1) ^ 1, sAbort, P.status);
                }
                used |= 1u << st;
                if (res) { lastres |= 1u << st; rpar ^= 1u << st; }
                else { lastres &= ~(1u << st); xpar ^= 1u << st; }
                return w;
            };
            while (ok && it.next(g)) {
                const int idx = g.side * BH + g.s;
                bool resident = false;
                if (g.phase == kPhaseSum && g.attempt > 0) {
                    const int go = seg_state(g.li, idx, g.attempt);
                    if (go == 0) { ok = false; break; }
                    if (g.extra && ((go - 1) & 1) == 0) continue;
                    resident = (go - 1) >> 1;
                }
                if (EXT && g.phase != kPhaseSum) {
                    const int ah = apply_here(g, it.s_lo);
                    if (ah == 0) { ok = false; break; }
                    if (ah == 1) continue;
                }
                if (resident) {
                    // tiles of the stored Gibbs kernel instead of token tiles; no pivots, no MMA
                    for (int t = g.t0; t < g.t1 && ok; ++t) {
                        const int st = kx % kStages;
                        ok = acquire_stage(st, true);
                        if (!ok) break;
                        mbar_arrive_expect_tx(bar(bXFull + st), kStageBytes);
                        tma_load_3d(sbase + PL::offX + st * kStageBytes, &P.tmKt, bar(bXFull + st), 0, t * kTileRows, idx);
                        ++kx;
                    }
                    continue;
                }
                const int zs = g.h & 1;
                if (ztag[zs] != g.h) {
                    if (zuse[zs] > 0) ok = mbar_wait(bar(bZEmpty + zs), (zuse[zs] - 1) & 1, sAbort, P.status);
                    if (!ok) break;
                    mbar_arrive_expect_tx(bar(bZFull + zs), 2 * RP * 128);
#pragma unroll
                    for (int part = 0; part < 2; ++part)
                        tma_load_3d(sbase + PL::offZ + zs * PL::ZBYTES + part * (64 * 128), &P.tmZ, bar(bZFull + zs),
                                    0, 0, g.h * 2 + part);
                    ztag[zs] = g.h; ++zuse[zs];
                }
                const CUtensorMap *xm = g.side ? &P.tmK : &P.tmQ;
                for (int t = g.t0; t < g.t1 && ok; ++t) {
                    {
                        const int st = kx % kStages;
                        ok = acquire_stage(st, false);
                        if (!ok) break;
                        mbar_arrive_expect_tx(bar(bXFull + st), kStageBytes);
                        tma_load_3d(sbase + PL::offX + st * kStageBytes, xm, bar(bXFull + st), 0, t * kTileRows, g.s);
                        ++kx;
                    }
                    if (g.phase == kPhaseWred) {
                        const int st = kx % kStages;
                        ok = acquire_stage(st, false);
                        if (!ok) break;
                        mbar_arrive_expect_tx(bar(bXFull + st), kStageBytes);
                        tma_load_3d(sbase + PL::offX + st * kStageBytes, &P.tmV, bar(bXFull + st), 0, t * kTileRows, g.s);
                        ++kx;
                    }
                }
            }
            if (!ok) {
                // give the copies still in flight a bounded time to land before the CTA exits
                const int first = kx > kStages ? kx - kStages : 0;
                for (int j = first; j < kx; ++j) {
                    const uint64_t t0 = global_timer_ns();
                    while (!mbar_try_wait(bar(bXFull + j % kStages), (j / kStages) & 1))
                        if (global_timer_ns() - t0 > kWaitLimitNs) break;
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ======================= MMA issuer =======================
        // The whole warp runs the loop with warp-uniform values (so that descriptors and addresses can stay in
        // uniform registers); one elected lane issues the tcgen05 instructions.
        Sched it(P, sSeg);
        Seg g;
        int k = 0, kx = 0, ztag[2] = {-1, -1}, zuse[2] = {0, 0}, segw = 0, sego = 0;
        int gk = 0;                           // group of the next tile of the apply passes; per-group tile-count parities
        uint32_t gpar = 0;
        int ka = 0, ko = 0;                   // tiles of the apply passes / of the OUT pass so far
        bool ok = true, w_open = false;
        // Apply MMAs are issued two tiles late, so that the logits of the following tiles are not held back by them:
        // pend_* is the older waiting tile, pnew_* the newer one.
        int pend_k = -1, pend_o = 0, pend_first = 0, pend_vs = 0, pend_phase = 0;
        int pnew_k = -1, pnew_o = 0, pnew_first = 0, pnew_vs = 0, pnew_phase = 0;
        const uint32_t tm = __shfl_sync(0xffffffffu, tmem_base, 0);
        // Descriptors differ only in the 16-byte-granular start address (low word).
        const uint64_t dK = make_smem_desc(sbase, 16, 1024);               // K-major operand, 128-byte rows
        const uint64_t dMN = make_smem_desc(sbase, kStageBytes, 1024);     // MN-major operand, panels kStageBytes apart
        const uint32_t dK_hi = (uint32_t)(dK >> 32), dK_lo = (uint32_t)dK;
        const uint32_t dMN_hi = (uint32_t)(dMN >> 32), dMN_lo = (uint32_t)dMN;
        auto desc = [](uint32_t hi, uint32_t lo) { return ((uint64_t)hi << 32) | lo; };

        auto issue_apply = [&]() {
            const int pb = pend_k & 1, pj = pend_k >> 1, ob = pend_o & 1, oj = pend_o >> 1;
            const uint32_t pa = (PL::offP + pb * PL::PBYTES) >> 4;
            if (pend_phase == kPhaseWred) {
                const int vs = pend_vs % kStages, vph = (pend_vs / kStages) & 1;
                if (ok) ok = wwait2(bar(bPFull + pb), pj & 1, bar(bXFull + vs), vph);
                tc_fence_after();
                const uint32_t va = (PL::offX + vs * kStageBytes) >> 4;
                if (ok && elect_one()) {
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
                        umma_bf16(tm + PL::colW, desc(dMN_hi, dMN_lo + pa + ks * 128),
                                  desc(dMN_hi, dMN_lo + va + ks * 128), idesc_w, (pend_first && ks == 0) ? 0u : 1u);
                    umma_commit(bar(bPEmpty + pb));
                    umma_commit(bar(bXEmpty + vs));
                }
            } else {
                if (ok) ok = wwait2(bar(bPFull + pb), pj & 1, bar(bOEmpty + ob), (oj & 1) ^ 1);
                tc_fence_after();
                if (ok && elect_one()) {
#pragma unroll
                    for (int part = 0; part < 2; ++part)
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            umma_bf16(tm + PL::colO + ob * DK, desc(dK_hi, dK_lo + pa + ks * 2),
                                      desc(dK_hi, dK_lo + ((PL::offW + part * (DK * 128)) >> 4) + ks * 2), idesc_o,
                                      (part | ks) ? 1u : 0u);
                    umma_commit(bar(bPEmpty + pb));
                    umma_commit(bar(bOFull + ob));
                }
            }
            __syncwarp();
            pend_k = pnew_k; pend_o = pnew_o; pend_first = pnew_first; pend_vs = pnew_vs; pend_phase = pnew_phase;
            pnew_k = -1;
        };

        while (ok && it.next(g)) {
            const int idx = g.side * BH + g.s;
            if (g.phase == kPhaseSum && g.attempt > 0) {
                int go = 0;
                if (lane == 0) go = seg_state(g.li, idx, g.attempt);
                go = __shfl_sync(0xffffffffu, go, 0);
                if (go == 0) { ok = false; break; }
                if (g.extra && ((go - 1) & 1) == 0) continue;
                if ((go - 1) >> 1) {                     // the epilogue reads the stored Gibbs kernel: nothing to issue
                    kx += g.t1 - g.t0;
                    k += g.t1 - g.t0;
                    // This warp has not seen the fills of this segment complete, so it may not wait on a stage barrier by
                    // parity again before they all have: wait until the segment has been gathered (every tile of it has
                    // then been read).
                    int done = 0;
                    if (lane == 0) done = seg_state(g.li, idx, g.attempt + 1);
                    done = __shfl_sync(0xffffffffu, done, 0);
                    if (done == 0) { ok = false; break; }
                    continue;
                }
            }
            if (EXT && g.phase != kPhaseSum) {
                int ah = 0;
                if (lane == 0) ah = apply_here(g, it.s_lo);
                ah = __shfl_sync(0xffffffffu, ah, 0);
                if (ah == 0) { ok = false; break; }
                if (ah == 1) continue;
            }
            while (pend_k >= 0) issue_apply();
            if (w_open) {                                                    // W of the previous WRED segment complete
                if (ok && elect_one()) umma_commit(bar(bWFull));
                __syncwarp();
                w_open = false;
            }
            if (g.phase == kPhaseWred) {
                if (segw > 0 && ok) ok = wwait(bar(bWEmpty), (segw - 1) & 1);
                ++segw;
                w_open = true;
            }
            const int zs = g.h & 1;
            if (ztag[zs] != g.h) {
                if (zuse[zs] > 0 && elect_one()) umma_commit(bar(bZEmpty + zs));
                __syncwarp();
                if (ok) ok = wwait(bar(bZFull + zs), zuse[zs] & 1);
                ztag[zs] = g.h; ++zuse[zs];
            }
            if (g.phase == kPhaseOut) {
                if (sego > 0 && elect_one()) umma_commit(bar(bWqEmpty));
                __syncwarp();
                if (ok) ok = wwait(bar(bWqFull), sego & 1);
                ++sego;
            }
            const uint32_t za = dK_lo + ((PL::offZ + zs * PL::ZBYTES) >> 4);
            for (int t = g.t0; t < g.t1 && ok; ++t, ++k) {
                // SUM passes: the group is the ring stage's (stage % kGroups), as in the stored-kernel passes, so that a
                // group has seen, through its accumulator, every earlier fill of a stage it later waits on by parity.
                // Apply passes: the groups simply take turns.
                const int grp = g.phase == kPhaseSum ? kx % kGroups : gk;
                const uint32_t gbit = (gpar >> grp) & 1;    // parity of this group's tile count
                gpar ^= 1u << grp;
                if (g.phase != kPhaseSum) gk = gk + 1 == kGroups ? 0 : gk + 1;
                const int st = kx % kStages, ph = (kx / kStages) & 1;
                ok = wwait2(bar(bXFull + st), ph, bar(bAccEmpty + grp), gbit ^ 1);
                tc_fence_after();
                const uint32_t xa = dK_lo + ((PL::offX + st * kStageBytes) >> 4);
                const uint32_t dcol = tm + grp * RP;
                if (ok && elect_one()) {
#pragma unroll
                    for (int part = 0; part < 2; ++part)
#pragma unroll
                        for (int kk = 0; kk < DK / 16; ++kk)
                            umma_bf16(dcol, desc(dK_hi, xa + kk * 2), desc(dK_hi, za + part * ((64 * 128) >> 4) + kk * 2),
                                      idesc_cost, (part | kk) ? 1u : 0u);
                    umma_commit(bar(bXEmpty + st));
                    umma_commit(bar(bAccFull + grp));
                }
                __syncwarp();
                ++kx;
                if (g.phase != kPhaseSum) {
                    const int vs = kx;
                    if (g.phase == kPhaseWred) ++kx;      // the value tile sits in the next ring stage
                    if (pnew_k >= 0) issue_apply();          // two waiting already: issue the older one
                    const int nk = ka++, no = g.phase == kPhaseOut ? ko++ : 0;
                    if (pend_k < 0) { pend_k = nk; pend_o = no; pend_first = (t == g.t0); pend_vs = vs; pend_phase = g.phase; }
                    else { pnew_k = nk; pnew_o = no; pnew_first = (t == g.t0); pnew_vs = vs; pnew_phase = g.phase; }
                }
            }
        }
        while (pend_k >= 0 && ok) issue_apply();
        if (w_open && ok && elect_one()) umma_commit(bar(bWFull));
        __syncwarp();
    } else if (warp == 2) {
        // ======================= publisher (one warp): the CTA's column partial of every SUM segment =======================
        Sched it(P, sSeg);
        Seg g;
        int segs = 0;
        bool ok = true;
        const int c0 = 2 * lane;                          // this lane's two columns (lanes with c0 >= RP idle)
        const bool mine = c0 < RP;
        while (it.next(g)) {
            if (g.phase != kPhaseSum) break;              // SUM segments come first in the schedule
            const int idx = g.side * BH + g.s, li = g.li;
            int go = 0;
            if (lane == 0) go = seg_state(li, idx, g.attempt);
            go = __shfl_sync(0xffffffffu, go, 0);
            if (go == 0) ok = false;
            if (g.extra && ((go - 1) & 1) == 0) continue;
            const int rb = (go - 1) & 1;
            const int par = segs & 1;
            if (ok) ok = wwait(bar(bSegFull + par), (segs >> 1) & 1);
            ++segs;
            if (!ok) continue;
            float k0 = rb ? neg_inf() : 0.f, s0 = 0.f, k1 = k0, s1 = 0.f;
            if (mine) {
                const float *src = sPart + ((par * kEpiWarps) * 64 + c0) * 2;
#pragma unroll
                for (int w = 0; w < kEpiWarps; ++w) {
                    const float4 pr = *reinterpret_cast<const float4 *>(src + w * 128);
                    if (rb) { pair_merge(k0, s0, pr.x, pr.y); pair_merge(k1, s1, pr.z, pr.w); }
                    else { s0 += pr.y; s1 += pr.w; }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(bSegEmpty + par));
            if (mine) {
                // two buffers by attempt parity: a CTA may publish attempt a+1 while a slower one still gathers attempt a
                unsigned long long *dst = P.part + ((((size_t)(g.attempt & 1) * 2 * BH + idx) * P.maxslots + g.slot) * RP + c0) * 2;
                st_tagged(dst, k0, s0, (unsigned)g.attempt + 1u);
                st_tagged(dst + 2, k1, s1, (unsigned)g.attempt + 1u);
            }
        }
        __syncwarp();
        if (lane == 0) { __threadfence_block(); *sPubDone = 1; }
    } else {
        // ======================= gatherer (one warp): all slots of a (slice, side) -> this CTA's copy of G =======================
        Sched it(P, sSeg);
        Seg g;
        bool ok = true;
        const int c0 = 2 * lane;
        const bool mine = c0 < RP;
        while (it.next(g)) {
            if (g.phase != kPhaseSum) break;
            const int idx = g.side * BH + g.s, li = g.li;
            const bool cached = li < kMaxLoc;
            int go = 0;
            if (lane == 0) go = seg_state(li, idx, g.attempt);
            go = __shfl_sync(0xffffffffu, go, 0);
            if (go == 0) ok = false;
            if (g.extra && ((go - 1) & 1) == 0) continue;
            if (!ok) continue;
            const int rb = (go - 1) & 1;
            const unsigned tag = (unsigned)g.attempt + 1u;
            float k0 = rb ? neg_inf() : 0.f, s0 = 0.f, k1 = k0, s1 = 0.f;
            const unsigned long long *src = P.part + ((((size_t)(g.attempt & 1) * 2 * BH + idx) * P.maxslots) * RP + c0) * 2;
            for (int p0 = 0; p0 < g.nslots && ok; p0 += 4) {
                unsigned long long w[4][4];
                uint64_t t0 = 0;
                for (uint32_t tries = 0;; ++tries) {
                    bool ready = true;
                    if (mine) {
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            if (p0 + u < g.nslots) {
                                ld_tagged(src + (size_t)(p0 + u) * RP * 2, w[u][0], w[u][1]);
                                ld_tagged(src + (size_t)(p0 + u) * RP * 2 + 2, w[u][2], w[u][3]);
                            }
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            if (p0 + u < g.nslots)
                                ready = ready && (unsigned)(w[u][0] >> 32) == tag && (unsigned)(w[u][1] >> 32) == tag &&
                                        (unsigned)(w[u][2] >> 32) == tag && (unsigned)(w[u][3] >> 32) == tag;
                    }
                    if (__all_sync(0xffffffffu, ready)) break;
                    bool giveup = *sAbort != 0;
                    if ((tries & 7u) == 7u) {
                        const uint64_t now = global_timer_ns();
                        if (t0 == 0) t0 = now;
                        else if (now - t0 > kWaitLimitNs) giveup = true;
                    }
                    if (__any_sync(0xffffffffu, giveup)) {
                        if (lane == 0) { *sAbort = 1; atomicOr(P.status, 4 /* LOT_DEV_TIMEOUT */); }
                        ok = false;
                        break;
                    }
                    __nanosleep(64);
                }
                if (!ok || !mine) continue;
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (p0 + u < g.nslots) {
                        const float a0 = __uint_as_float((unsigned)w[u][0]), b0 = __uint_as_float((unsigned)w[u][1]);
                        const float a1 = __uint_as_float((unsigned)w[u][2]), b1 = __uint_as_float((unsigned)w[u][3]);
                        if (rb) { pair_merge(k0, s0, a0, b0); pair_merge(k1, s1, a1, b1); }
                        else { s0 += b0; s1 += b1; }
                    }
            }
            if (!ok) continue;
            bool bad = false;
            if (!rb && mine) {
                if (c0 < P.r && !(s0 >= kPlainFloor && s0 <= 3.0e38f)) bad = true;
                if (c0 + 1 < P.r && !(s1 >= kPlainFloor && s1 <= 3.0e38f)) bad = true;
            }
            const int fail = __any_sync(0xffffffffu, bad);
            const int itn = cached ? sIter[li] : __ldcg(P.iter + idx);
            if (!fail && mine) {
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int col = c0 + u;
                    if (col < P.r) {
                        const float kk = u ? k1 : k0, ss = u ? s1 : s0;
                        const float gold = cached ? sGc[li * 64 + col] : __ldcg(P.G + (size_t)idx * RP + col);
                        const float gn = gold + lg2(__ldg(P.beta + g.h * P.r + col) * (float)g.nvalid) - (kk + lg2(ss));
                        if (cached) sGc[li * 64 + col] = gn;
                        else __stcg(P.G + (size_t)idx * RP + col, gn);
                        if (g.slot == 0) {
                            if (!isfinite(gn)) atomicOr(P.status, 1 /* LOT_DEV_NONFINITE */);
                            float *gdst = g.side ? P.g2_out : P.g1_out;
                            if (itn + 1 == P.T && gdst != nullptr) gdst[(size_t)g.s * P.r + col] = gn * P.eps_ln2;
                        }
                    }
                }
            }
            // the next attempt may read the stored kernel if the potentials' spread keeps 2^(G - max G) well inside
            // the float32 range (it decides how small a row sum can get)
            float gmx = neg_inf(), gmn = -neg_inf();
            if (RP == 64 && cached && !fail && mine) {
#pragma unroll
                for (int u = 0; u < 2; ++u)
                    if (c0 + u < P.r) { const float gv = sGc[li * 64 + c0 + u]; gmx = fmaxf(gmx, gv); gmn = fminf(gmn, gv); }
            }
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) {
                gmx = fmaxf(gmx, __shfl_xor_sync(0xffffffffu, gmx, off));
                gmn = fminf(gmn, __shfl_xor_sync(0xffffffffu, gmn, off));
            }
            if (EXT && P.ext_apply && !fail && itn + 1 == P.T) {
                // the last pivot update of this (slice, side): can the apply kernels work from its stored kernel?
                const int dec = (RP == 64 && cached && !rb && P.Kt != nullptr && (gmx - gmn) <= 64.f) ? 1 : 2;
                if (mine && g.slot == 0 && cached) {
                    if (c0 < P.r) __stcg(P.G + (size_t)idx * RP + c0, sGc[li * 64 + c0]);
                    if (c0 + 1 < P.r) __stcg(P.G + (size_t)idx * RP + c0 + 1, sGc[li * 64 + c0 + 1]);
                }
                if (lane == 0) {
                    if (cached) sDec[li] = dec;
                    if (g.slot == 0) { __threadfence(); st_release(P.decision + idx, dec); }
                }
            }
            const bool run_started = cached && sResFirst[li] != 0x7fffffff, run_ended = cached && sResLast[li] != 0x7fffffff;
            const int next_resident = RP == 64 && cached && !fail && !rb && !run_ended && P.Kt != nullptr && (gmx - gmn) <= 64.f;
            if (next_resident && mine) {
                // weights of the next attempt, w_t = 2^(G_t - max G), computed once here for all epilogue warps
                float *sWt = reinterpret_cast<float *>(smem + PL::offWt) + li * 64;
                sWt[c0] = c0 < P.r ? ex2(sGc[li * 64 + c0] - gmx) : 0.f;
                sWt[c0 + 1] = c0 + 1 < P.r ? ex2(sGc[li * 64 + c0 + 1] - gmx) : 0.f;
            }
            if (cached) {
                __threadfence_block();
                __syncwarp();
                if (lane == 0) {
                    if (next_resident && !run_started) sResFirst[li] = g.attempt + 1;
                    if (!next_resident && run_started && !run_ended) sResLast[li] = g.attempt;
                    if (fail) sRobust[li] = 1;
                    else sIter[li] = itn + 1;
                    __threadfence_block();
                    sDone[li] = g.attempt + 1;
                }
            } else {
                // beyond the cache the state lives in global memory; every sharing CTA writes the same values
                __threadfence();
                __syncwarp();
                if (lane == 0) {
                    if (fail) __stcg(P.robust + idx, 1);
                    __threadfence();
                    if (!fail) st_release(P.iter + idx, itn + 1);
                    st_release(P.epoch + idx, g.attempt + 1);
                }
            }
        }
    }
    } else {
        // ======================= epilogue (kGroups groups of four warps) =======================
        const int ew = warp - 4, grp = ew >> 2, w4 = ew & 3, qd = warp & 3;
        const int etid = threadIdx.x - 128, gtid = w4 * 32 + lane;
        const int rq = lane >> 2, cq = lane & 3;                          // quad layout: row and column quarter
        const int rit = qd * 32 + lane;                                   // row-per-thread layout: row inside the tile
        const uint32_t lane_addr = tmem_base + ((uint32_t)(qd * 32) << 16);
        float *myG = sG + grp * 64;
        Sched it(P, sSeg);
        Seg g;
        int k = 0;
        int gk = 0;                           // group of the next tile of the apply passes
        uint32_t mypar = 0;                   // parity of the number of tiles this group has taken
        bool ok = true;
        // The schedule lists every SUM segment before the first WRED segment: two loops, so that the state of one kind
        // of pass is not carried through the other.
        bool more = it.next(g);
        {
            int segs = 0;
            int kx = 0;                       // ring stage counter, as in the producer
            for (; more && g.phase == kPhaseSum; more = it.next(g)) {
                const int idx = g.side * BH + g.s;
                // ================= SUM: quad layout, column sums in registers =================
                // every warp waits by itself for the potential of this attempt
                const int li = g.li;
                int go = 0;
                if (lane == 0) go = seg_state(li, idx, g.attempt);
                go = __shfl_sync(0xffffffffu, go, 0);
                if (go == 0) ok = false;
                const int rb = (go - 1) & 1, resident = go > 0 ? (go - 1) >> 1 : 0;
                if (g.extra && rb == 0) continue;                       // this segment needed no repeat
                float *dstp = sPart + (((segs & 1) * kEpiWarps + ew) * 64) * 2;
                const uint32_t par_empty = ((segs >> 1) & 1) ^ 1;
                const int par = segs & 1;
                ++segs;

                if constexpr (RP == 64) {
                    if (resident) {
                        // ---- stored-kernel pass: K~_it = 2^(L_it - max_t L_it) comes back as bf16 tiles; with
                        // w_t = 2^(G_t - max G) the row sums are s_i = sum_t K~_it w_t and the column sums
                        // w_t sum_i K~_it / s_i: two FMAs per entry, no exponential, no tensor-core work.
                        // Thread = 4 rows (rq + 8 j of the warp's 32) x 16 consecutive columns (16 cq ..).
                        // column pairs are kept as float2 so that the sums run as packed two-wide FMAs
                        float2 w2[8], c2[8];
                        {
                            const float4 *wt = reinterpret_cast<const float4 *>(smem + PL::offWt + (li * 64 + cq * 16) * 4);
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const float4 w4v = wt[j];
                                w2[2 * j] = make_float2(w4v.x, w4v.y);
                                w2[2 * j + 1] = make_float2(w4v.z, w4v.w);
                                c2[2 * j] = make_float2(0.f, 0.f);
                                c2[2 * j + 1] = make_float2(0.f, 0.f);
                            }
                        }
                        // A ring stage is always read by the same group (stage % kGroups; kStages is a multiple of kGroups),
                        // whatever the segment: a parity wait on a stage's barrier is only safe for a waiter that has
                        // itself seen the stage's previous fill complete.  (With the tile's index in the segment deciding
                        // the group, a group could ask for fill f of a stage while fill f - 1, the other group's, was still
                        // in flight, and the parity of fill f - 2 answered.)
                        static_assert(kStages % kGroups == 0, "a ring stage must always fall to the same epilogue group");
                        for (int t = g.t0 + (grp - kx % kGroups + kGroups) % kGroups; t < g.t1; t += kGroups) {
                            const int kxt = kx + (t - g.t0);
                            const int stg = kxt % kStages;
                            if (ok) ok = wwait(bar(bXFull + stg), (kxt / kStages) & 1);
                            if (ok) {
                                const uint8_t *tile = smem + PL::offX + stg * kStageBytes;
#pragma unroll
                                for (int jp = 0; jp < 4; jp += kLock) {
                                    // kLock rows advance in step: every instruction has independent twins
                                    float2 kf[kLock][8], sa[kLock], sb[kLock];
                                    float sr[kLock];
#pragma unroll
                                    for (int q = 0; q < kLock; ++q) {
                                        const int rin = w4 * 32 + (jp + q) * 8 + rq;           // row inside the tile
                                        const uint4 a = *reinterpret_cast<const uint4 *>(tile + rin * 128 + (((2 * cq) ^ (rin & 7)) * 16));
                                        const uint4 b = *reinterpret_cast<const uint4 *>(tile + rin * 128 + (((2 * cq + 1) ^ (rin & 7)) * 16));
                                        const uint32_t pk[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
                                        for (int e = 0; e < 8; ++e)
                                            kf[q][e] = make_float2(__uint_as_float(pk[e] << 16), __uint_as_float(pk[e] & 0xffff0000u));
                                        sa[q] = make_float2(0.f, 0.f); sb[q] = make_float2(0.f, 0.f);
                                    }
#pragma unroll
                                    for (int e = 0; e < 8; e += 2) {
#pragma unroll
                                        for (int q = 0; q < kLock; ++q) {
                                            sa[q] = __ffma2_rn(kf[q][e], w2[e], sa[q]);
                                            sb[q] = __ffma2_rn(kf[q][e + 1], w2[e + 1], sb[q]);
                                        }
                                    }
#pragma unroll
                                    for (int q = 0; q < kLock; ++q) sr[q] = (sa[q].x + sa[q].y) + (sb[q].x + sb[q].y);
#pragma unroll
                                    for (int q = 0; q < kLock; ++q) sr[q] += __shfl_xor_sync(0xffffffffu, sr[q], 1);
#pragma unroll
                                    for (int q = 0; q < kLock; ++q) sr[q] += __shfl_xor_sync(0xffffffffu, sr[q], 2);
                                    float2 uu[kLock];
#pragma unroll
                                    for (int q = 0; q < kLock; ++q) {
                                        const int rin = w4 * 32 + (jp + q) * 8 + rq;
                                        const float u = t * kTileRows + rin < g.nvalid ? __fdividef(1.f, sr[q]) : 0.f;
                                        uu[q] = make_float2(u, u);
                                    }
#pragma unroll
                                    for (int e = 0; e < 8; ++e) {
#pragma unroll
                                        for (int q = 0; q < kLock; ++q) c2[e] = __ffma2_rn(kf[q][e], uu[q], c2[e]);
                                    }
                                }
                            }
                            // this warp has its rows in registers: one of the four releases of the stage
                            __syncwarp();
                            if (lane == 0 && ok) mbar_arrive(bar(bREmpty + stg));
                        }
                        k += g.t1 - g.t0;
                        kx += g.t1 - g.t0;
                        float c[16];
#pragma unroll
                        for (int j = 0; j < 8; ++j) { c[2 * j] = c2[j].x * w2[j].x; c[2 * j + 1] = c2[j].y * w2[j].y; }
                        const int cb = quad_col_reduce16(c, lane);
                        if (ok) ok = wwait(bar(bSegEmpty + par), par_empty);
                        *reinterpret_cast<float4 *>(dstp + (cq * 16 + cb) * 2) = make_float4(0.f, c[0], 0.f, c[1]);
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar(bSegFull + par));
                        continue;
                    }
                }
                // first pass of a solve that will run stored-kernel passes: keep 2^(L - rowmax) as bf16
                const bool store_kt = RP == 64 && P.Kt != nullptr && g.attempt == 0 && li < kMaxLoc;

                auto run = [&](auto rbtag) {
                    constexpr bool RB = decltype(rbtag)::value;
                    float Gr[NC], acc[NC], kap[RB ? NC : 1];
#pragma unroll
                    for (int ci = 0; ci < NC; ++ci) {
                        const int col = (ci >> 1) * 8 + 2 * cq + (ci & 1);
                        Gr[ci] = col < P.r ? (li < kMaxLoc ? sGc[li * 64 + col] : __ldcg(P.G + (size_t)idx * RP + col)) : neg_inf();
                        acc[ci] = 0.f;
                        if (RB) kap[ci] = neg_inf();
                    }
                    // the tile in ring stage st goes to group st % kGroups: step straight from own tile to own tile
                    const int first = (grp - kx % kGroups + kGroups) % kGroups;
                    for (int t = g.t0 + first; t < g.t1; t += kGroups) {
                        if (ok) ok = wwait(bar(bAccFull + grp), mypar);
                        mypar ^= 1u;
                        if (!ok) continue;
                        tc_fence_after();
                        if (!RB && store_kt) {
                            // the store of the previous tile must have read the staging rows before they are rewritten
                            if (lane == 0) bulk_wait_group_read0();
                            __syncwarp();
                        }
#pragma unroll
                        for (int half = 0; half < 2; ++half) {
                            float v[2 * NC];
                            tmem_ld_quad<RP>(lane_addr + ((uint32_t)(half * 16) << 16) + grp * RP, v);
                            tmem_wait_ld();
                            if (half == 1) {
                                tc_fence_before();
                                __syncwarp();
                                if (lane == 0) mbar_arrive(bar(bAccEmpty + grp));
                            }
                            const int rowA = t * kTileRows + qd * 32 + half * 16 + rq, rowB = rowA + 8;
                            float mA = neg_inf(), mB = neg_inf();
#pragma unroll
                            for (int rep = 0; rep < NC / 2; ++rep) {
                                const float2 g2 = make_float2(Gr[rep * 2], Gr[rep * 2 + 1]);
                                const float2 xa = __fadd2_rn(make_float2(v[rep * 4 + 0], v[rep * 4 + 1]), g2);
                                const float2 xb = __fadd2_rn(make_float2(v[rep * 4 + 2], v[rep * 4 + 3]), g2);
                                v[rep * 4 + 0] = xa.x; v[rep * 4 + 1] = xa.y; v[rep * 4 + 2] = xb.x; v[rep * 4 + 3] = xb.y;
                                mA = max3(mA, xa.x, xa.y);
                                mB = max3(mB, xb.x, xb.y);
                            }
                            mA = fmaxf(mA, __shfl_xor_sync(0xffffffffu, mA, 1));
                            mB = fmaxf(mB, __shfl_xor_sync(0xffffffffu, mB, 1));
                            mA = fmaxf(mA, __shfl_xor_sync(0xffffffffu, mA, 2));
                            mB = fmaxf(mB, __shfl_xor_sync(0xffffffffu, mB, 2));
                            float sA0 = 0.f, sA1 = 0.f, sB0 = 0.f, sB1 = 0.f;
                            if (!RB) {
                                // column pairs as packed two-wide operations
                                const float2 nA = make_float2(-mA, -mA), nB = make_float2(-mB, -mB);
                                float2 sA2 = make_float2(0.f, 0.f), sB2 = make_float2(0.f, 0.f);
#pragma unroll
                                for (int rep = 0; rep < NC / 2; ++rep) {
                                    const float2 xa = __fadd2_rn(make_float2(v[rep * 4 + 0], v[rep * 4 + 1]), nA);
                                    const float2 xb = __fadd2_rn(make_float2(v[rep * 4 + 2], v[rep * 4 + 3]), nB);
                                    const float2 ea = make_float2(ex2(xa.x), ex2(xa.y)), eb = make_float2(ex2(xb.x), ex2(xb.y));
                                    v[rep * 4 + 0] = ea.x; v[rep * 4 + 1] = ea.y; v[rep * 4 + 2] = eb.x; v[rep * 4 + 3] = eb.y;
                                    sA2 = __fadd2_rn(sA2, ea);
                                    sB2 = __fadd2_rn(sB2, eb);
                                }
                                sA0 = sA2.x; sA1 = sA2.y; sB0 = sB2.x; sB1 = sB2.y;
                            } else {
#pragma unroll
                                for (int rep = 0; rep < NC / 2; ++rep) {
                                    sA0 += ex2(v[rep * 4 + 0] - mA); sA1 += ex2(v[rep * 4 + 1] - mA);
                                    sB0 += ex2(v[rep * 4 + 2] - mB); sB1 += ex2(v[rep * 4 + 3] - mB);
                                }
                            }
                            if (!RB && store_kt) {
                                // G = 0 in this pass, so the exponentials are the stored kernel's entries: staged in shared
                                // memory (rows of 128 bytes, 16-byte chunks xor row % 8) and written by one TMA store per warp
                                // row A = half * 16 + rq, row B = row A + 8: both have row % 8 == rq, so one swizzled
                                // address per column block serves both (the xor is kept inside the loop on purpose: hoisted,
                                // the sixteen addresses would cost sixteen registers for the whole pass)
                                const uint32_t rowA = smem_u32(smem) + PL::offKtStage + ((threadIdx.x >> 5) - 4) * (32 * 128) +
                                                      (half * 16 + rq) * 128 + (rq << 4) + cq * 4;
#pragma unroll
                                for (int rep = 0; rep < NC / 2; ++rep) {
                                    uint32_t addr;
                                    asm volatile("xor.b32 %0, %1, %2;" : "=r"(addr) : "r"(rowA), "r"(rep << 4));
                                    asm volatile("st.shared.b32 [%0], %1;" ::"r"(addr), "r"(pack_bf16(v[rep * 4 + 0], v[rep * 4 + 1])) : "memory");
                                    asm volatile("st.shared.b32 [%0 + 1024], %1;" ::"r"(addr), "r"(pack_bf16(v[rep * 4 + 2], v[rep * 4 + 3])) : "memory");
                                }
                                if (half == 1) {
                                    fence_proxy_async_smem();
                                    __syncwarp();
                                    if (lane == 0) {
                                        tma_store_3d(&P.tmKtS, smem_u32(smem) + PL::offKtStage + ((threadIdx.x >> 5) - 4) * (32 * 128), 0, t * kTileRows + ((threadIdx.x >> 5) & 3) * 32, idx);
                                        bulk_commit_group();
                                    }
                                }
                            }
                            float sA = sA0 + sA1, sB = sB0 + sB1;
                            sA += __shfl_xor_sync(0xffffffffu, sA, 1);
                            sB += __shfl_xor_sync(0xffffffffu, sB, 1);
                            sA += __shfl_xor_sync(0xffffffffu, sA, 2);
                            sB += __shfl_xor_sync(0xffffffffu, sB, 2);
                            if (!RB) {
                                const float wA = rowA < g.nvalid ? __fdividef(1.f, sA) : 0.f;
                                const float wB = rowB < g.nvalid ? __fdividef(1.f, sB) : 0.f;
                                const float2 wA2 = make_float2(wA, wA), wB2 = make_float2(wB, wB);
#pragma unroll
                                for (int rep = 0; rep < NC / 2; ++rep) {
                                    float2 a2 = make_float2(acc[rep * 2], acc[rep * 2 + 1]);
                                    a2 = __ffma2_rn(make_float2(v[rep * 4 + 0], v[rep * 4 + 1]), wA2, a2);
                                    a2 = __ffma2_rn(make_float2(v[rep * 4 + 2], v[rep * 4 + 3]), wB2, a2);
                                    acc[rep * 2] = a2.x; acc[rep * 2 + 1] = a2.y;
                                }
                            } else {
                                // exact log2 of every normalised entry, added to (kappa, S) pairs
                                const float MA = mA + lg2(sA), MB = mB + lg2(sB);
#pragma unroll
                                for (int ci = 0; ci < NC; ++ci) {
                                    const int col = (ci >> 1) * 8 + 2 * cq + (ci & 1);
                                    if (col < P.r) {
                                        if (rowA < g.nvalid) pair_add(kap[RB ? ci : 0], acc[ci], v[(ci >> 1) * 4 + (ci & 1)] - MA);
                                        if (rowB < g.nvalid) pair_add(kap[RB ? ci : 0], acc[ci], v[(ci >> 1) * 4 + 2 + (ci & 1)] - MB);
                                    }
                                }
                            }
                        }
                    }
                    k += g.t1 - g.t0;
                    kx += g.t1 - g.t0;
                    // ---- warp partial: the 8 rows-lanes of every column quarter, left in shared memory
                    if constexpr (!RB && NC == 16) {
                        const int cb = quad_col_reduce16(acc, lane);
                        if (store_kt) {                      // the stores of this warp are complete before the segment is handed over
                            if (lane == 0) bulk_wait_group0();
                            __syncwarp();
                        }
                        if (ok) ok = wwait(bar(bSegEmpty + par), par_empty);
                        *reinterpret_cast<float4 *>(dstp + ((cb >> 1) * 8 + 2 * cq) * 2) = make_float4(0.f, acc[0], 0.f, acc[1]);
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar(bSegFull + par));
                        return;
                    }
#pragma unroll
                    for (int off = 4; off <= 16; off <<= 1) {
#pragma unroll
                        for (int ci = 0; ci < NC; ++ci) {
                            if (RB) {
                                const float ok2 = __shfl_xor_sync(0xffffffffu, kap[RB ? ci : 0], off);
                                const float os2 = __shfl_xor_sync(0xffffffffu, acc[ci], off);
                                pair_merge(kap[RB ? ci : 0], acc[ci], ok2, os2);
                            } else {
                                acc[ci] += __shfl_xor_sync(0xffffffffu, acc[ci], off);
                            }
                        }
                    }
                    if (ok) ok = wwait(bar(bSegEmpty + par), par_empty);
                    if (rq == 0) {
#pragma unroll
                        for (int ci = 0; ci < NC; ci += 2) {
                            const int col = (ci >> 1) * 8 + 2 * cq;
                            *reinterpret_cast<float4 *>(dstp + col * 2) =
                                make_float4(RB ? kap[RB ? ci : 0] : 0.f, acc[ci], RB ? kap[RB ? ci + 1 : 0] : 0.f, acc[ci + 1]);
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(bSegFull + par));
                };
                if (rb) run(std::true_type{});
                else run(std::false_type{});
            }
        }

        int ka = 0, ko = 0, segw = 0, sego = 0;
        for (; more; more = it.next(g)) {
            const int idx = g.side * BH + g.s;
            // ---- WRED / OUT: wait until the final potential (and W') of this slice is known here
            const int li = g.li;
            if (EXT) {
                int ah = 0;
                if (lane == 0) ah = apply_here(g, it.s_lo);
                ah = __shfl_sync(0xffffffffu, ah, 0);
                if (ah == 0) ok = false;
                if (ah == 1) continue;
            }
            if (gtid == 0) {
                bool w = spin_ge(sPubDone, 1, sAbort, P.status);          // plan buffers free of SUM partials
                if (w) w = li < kMaxLoc ? spin_ge(sIter + li, P.T, sAbort, P.status) : poll_ge(P.iter + idx, P.T, sAbort, P.status);
            }
            // key-side geometry of this slice: which slots hold a partial of W
            int kv = P.n, wslots = 0;
            if (g.phase == kPhaseOut) {
                if (P.key_len != nullptr) kv = min(max(__ldg(P.key_len + g.b), 0), P.n);
                if (kv > 0) {
                    int c_lo;
                    slice_slots(P, g.s, (kv + kTileRows - 1) / kTileRows, c_lo, wslots);
                }
                if (w4 == 0)
                    for (int j = lane; j < wslots; j += 32) poll_ge(P.wflag + (size_t)g.s * P.maxslots + j, 1, sAbort, P.status);
            }
            named_bar_sync(1 + grp, 128);
            if (*sAbort) ok = false;

            // ================= WRED / OUT: one thread per token row =================
            if (gtid < RP)
                myG[gtid] = gtid < P.r ? (li < kMaxLoc ? sGc[li * 64 + gtid] : __ldcg(P.G + (size_t)idx * RP + gtid)) : neg_inf();
            if (g.phase == kPhaseOut) {
                // W'^T = (Diag(beta)^-1 Gamma2 V)^T of this slice as the B operand (hi and lo parts; 128-byte rows =
                // channels, 16-byte chunks of 8 pivots xor row % 8): every CTA of the slice adds the slots' partials
                // itself, in slot order, so all of them hold the same bits
                if (sego > 0 && ok) ok = wwait(bar(bWqEmpty), (sego - 1) & 1);
                const float mass = kv > 0 ? 1.f / (float)kv : 0.f;
                for (int item = etid; item < DK * 8; item += kEpiThreads) {
                    const int c = item >> 3, tc = item & 7, t0 = tc * 8;
                    float acc8[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                    const float *src0 = P.wpart + (size_t)g.s * P.maxslots * (DK * 64) + c * 64 + t0;
                    for (int sl0 = 0; sl0 < wslots; sl0 += 8) {
                        float4 a[8], b[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            a[u] = b[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                            if (sl0 + u < wslots) {
                                const float4 *src = reinterpret_cast<const float4 *>(src0 + (size_t)(sl0 + u) * (DK * 64));
                                a[u] = __ldcg(src);
                                b[u] = __ldcg(src + 1);
                            }
                        }
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            acc8[0] += a[u].x; acc8[1] += a[u].y; acc8[2] += a[u].z; acc8[3] += a[u].w;
                            acc8[4] += b[u].x; acc8[5] += b[u].y; acc8[6] += b[u].z; acc8[7] += b[u].w;
                        }
                    }
                    uint32_t hi[4], lo[4];
#pragma unroll
                    for (int e2 = 0; e2 < 4; ++e2) {
                        float wv2[2];
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            const int t = t0 + e2 * 2 + u;
                            wv2[u] = t < P.r ? acc8[e2 * 2 + u] * (mass / __ldg(P.beta + g.h * P.r + t)) : 0.f;
                        }
                        __nv_bfloat162 hh = __floats2bfloat162_rn(wv2[0], wv2[1]);
                        hi[e2] = *reinterpret_cast<uint32_t *>(&hh);
                        lo[e2] = pack_bf16(wv2[0] - __low2float(hh), wv2[1] - __high2float(hh));
                    }
                    uint8_t *dst = smem + PL::offW + c * 128 + ((tc ^ (c & 7)) * 16);
                    *reinterpret_cast<uint4 *>(dst) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                    *reinterpret_cast<uint4 *>(dst + DK * 128) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(bWqFull));
                ++sego;
            }
            named_bar_sync(1 + grp, 128);

            // the tile loop is compiled once per pass kind, so that the other kind's work is not carried along
            auto tiles = [&](auto wtag) {
                constexpr bool WRED = decltype(wtag)::value;
            const int first = grp >= gk ? grp - gk : grp - gk + kGroups;
            for (int t = g.t0 + first; t < g.t1; t += kGroups) {
                const int kat = ka + (t - g.t0), kot = ko + (t - g.t0);
                const int pb = kat & 1, pj = kat >> 1, ob = kot & 1, oj = kot >> 1;
                if (ok) ok = wwait(bar(bAccFull + grp), mypar);
                mypar ^= 1u;
                if (!ok) continue;
                tc_fence_after();
                const int row = t * kTileRows + rit;
                const bool valid = row < g.nvalid;
                float v[RP];
                tmem_ld<RP>(lane_addr + grp * RP, v);
                tmem_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(bAccEmpty + grp));
                // four independent chains for the row maximum and the row sum
                float m4[4] = {neg_inf(), neg_inf(), neg_inf(), neg_inf()};
#pragma unroll
                for (int c = 0; c < RP; c += 8) {
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        v[c + 2 * u] += myG[c + 2 * u];
                        v[c + 2 * u + 1] += myG[c + 2 * u + 1];
                        m4[u] = max3(m4[u], v[c + 2 * u], v[c + 2 * u + 1]);
                    }
                }
                const float m = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
                float s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int c = 0; c < RP; c += 4) {
#pragma unroll
                    for (int u = 0; u < 4; ++u) { v[c + u] = ex2(v[c + u] - m); s4[u] += v[c + u]; }
                }
                const float inv = __fdividef(1.f, (s4[0] + s4[1]) + (s4[2] + s4[3]));
                // ---- write the plan tile as an MMA operand
                ok = wwait(bar(bPEmpty + pb), (pj & 1) ^ 1);
                if (!ok) continue;
                uint8_t *prow = smem + PL::offP + pb * PL::PBYTES + rit * 128;
                const float w = WRED ? (valid ? inv : 0.f) : 1.f;
#pragma unroll
                for (int c8 = 0; c8 < 8; ++c8) {
                    uint32_t hi[4], lo[4];
#pragma unroll
                    for (int e2 = 0; e2 < 4; ++e2) {
                        const int c = c8 * 8 + e2 * 2;
                        const float a0 = c < RP ? v[c < RP ? c : 0] * w : 0.f;
                        const float a1 = c + 1 < RP ? v[c + 1 < RP ? c + 1 : 0] * w : 0.f;
                        __nv_bfloat162 hh = __floats2bfloat162_rn(a0, a1);
                        hi[e2] = *reinterpret_cast<uint32_t *>(&hh);
                        lo[e2] = pack_bf16(a0 - __low2float(hh), a1 - __high2float(hh));
                    }
                    const int pc = (c8 ^ (rit & 7)) * 16;
                    *reinterpret_cast<uint4 *>(prow + pc) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                    if (WRED)
                        *reinterpret_cast<uint4 *>(prow + kStageBytes + pc) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(bPFull + pb));
                if (!WRED) {
                    ok = wwait(bar(bOFull + ob), oj & 1);
                    if (!ok) continue;
                    tc_fence_after();
                    __nv_bfloat16 *orow = P.out + ((size_t)g.s * P.n + row) * DK;
#pragma unroll
                    for (int c0 = 0; c0 < DK; c0 += 32) {
                        float o[32];
                        tmem_ld32(lane_addr + PL::colO + ob * DK + c0, o);
                        tmem_wait_ld();
                        if (c0 + 32 == DK) {
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(bar(bOEmpty + ob));
                        }
                        if (row < P.n) {
#pragma unroll
                            for (int c = 0; c < 32; c += 8) {
                                uint4 pk;
                                pk.x = pack_bf16(o[c] * inv, o[c + 1] * inv);
                                pk.y = pack_bf16(o[c + 2] * inv, o[c + 3] * inv);
                                pk.z = pack_bf16(o[c + 4] * inv, o[c + 5] * inv);
                                pk.w = pack_bf16(o[c + 6] * inv, o[c + 7] * inv);
                                *reinterpret_cast<uint4 *>(orow + c0 + c) = pk;
                            }
                        }
                    }
                }
            }
            {
                const int nt = g.t1 - g.t0;
                gk = (gk + nt) % kGroups;
                k += nt; ka += nt;
                if (!WRED) ko += nt;
            }
            };
            if (g.phase == kPhaseWred) tiles(std::true_type{});
            else tiles(std::false_type{});

            if (g.phase == kPhaseWred) {
                // ---- W accumulator of this segment: TMEM lanes 0-63 hold the pivots' rows from the hi part of the plan,
                // lanes 64-127 those from the lo part.  Warp (qd, grp < kWGroups) takes its 32 lanes x WC channels; the
                // two halves are added through shared memory (the plan buffers are idle: every apply MMA has completed)
                // and the CTA's partial goes to its slot, transposed to [channel][pivot].
                constexpr int WC = DK / kWGroups;              // channels per reading group
                float wv[WC];
                if (ok) ok = wwait(bar(bWFull), segw & 1);
                if (ok) {
                    tc_fence_after();
                    if (grp < kWGroups) {
                        tmem_ld<WC>(lane_addr + PL::colW + grp * WC, wv);
                        tmem_wait_ld();
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(bWEmpty));
                }
                ++segw;
                float *xch = reinterpret_cast<float *>(smem + PL::offP);     // [channel][pivot] float
                if (ok && grp < kWGroups && qd >= 2) {
#pragma unroll
                    for (int c = 0; c < WC; ++c) xch[(grp * WC + c) * 64 + rit - 64] = wv[c];
                }
                named_bar_sync(5, kEpiThreads);
                if (ok && grp < kWGroups && qd < 2) {
                    float *dst = P.wpart + ((size_t)g.s * P.maxslots + g.slot) * (DK * 64) + rit;
#pragma unroll
                    for (int c = 0; c < WC; ++c) __stcg(dst + (grp * WC + c) * 64, wv[c] + xch[(grp * WC + c) * 64 + rit]);
                    __threadfence();
                }
                named_bar_sync(5, kEpiThreads);
                if (etid == 0 && !*sAbort) {
                    __threadfence();
                    st_release(P.wflag + (size_t)g.s * P.maxslots + g.slot, 1);
                }
            }
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
// Also clears the part of the workspace that must start at zero (`head`, head_vecs 16-byte words; the status word
// lies before it and is cleared by block 0) and raises LOT_DEV_EMPTY for non-positive key lengths.
// ---------------------------------------------------------------------------------------
__global__ void zprep_kernel(const float *__restrict__ z, __nv_bfloat16 *__restrict__ zp, const int32_t *key_len,
                             int *status, uint4 *head, size_t head_vecs, int B, int H, int r, int RP, int d, float scale,
                             float *g1_out, float *g2_out, int T, const unsigned *redo, unsigned redo_tag)
{
    if (blockIdx.x == 0) {
        if (threadIdx.x == 0) *status = 0;
        __syncthreads();
    }
    if (redo != nullptr && *reinterpret_cast<const volatile unsigned *>(redo) != redo_tag) return;
    // potentials nobody updates: every one of a zero-iteration call, the key side of a slice without keys
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < (size_t)B * H * r; i += (size_t)gridDim.x * blockDim.x) {
        const int b = (int)(i / ((size_t)H * r));
        if (g1_out != nullptr && T == 0) g1_out[i] = 0.f;
        if (g2_out != nullptr && (T == 0 || (key_len != nullptr && key_len[b] <= 0))) g2_out[i] = 0.f;
    }
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < head_vecs; i += (size_t)gridDim.x * blockDim.x)
        head[i] = make_uint4(0u, 0u, 0u, 0u);
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

static int num_sms() { return device_sm_count(); }

static inline size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }
static inline int pad_r(int r) { return r <= 16 ? 16 : (r <= 32 ? 32 : 64); }

} // namespace fused

// The apply stages run as separate kernels when the first pass keeps the Gibbs kernel (32 < r <= 64, more than one
// iteration), every block caches the state of all its segments in shared memory, and the problem is large: measured on
// B200 at B = 1, H = 16 the three-kernel form is 6 % faster at n = 65536, even at n = 16384 and 14 % slower at n = 4096
// (two more launches), so it is taken from 4096 tiles per side on.
bool fused_ext_apply(int B, int H, int n, int r, int iters)
{
    if (fused::pad_r(r) != 64 || iters < 2) return false;
    if ((long long)B * H * ((n + 127) / 128) < 4096) return false;
    int q, ctas, ms, cps;
    fused_geometry(B, H, n, &q, &ctas, &ms, &cps);
    if (cps > 0) return true;
    const int TPS = (n + 127) / 128;
    const int slices = (q + TPS - 2) / TPS + 1;           // most slices a block of q consecutive tiles can touch
    return 2 * slices <= fused::kMaxLoc;
}

bool fused_supported(int dtype, int d, int r)
{
    return dtype == 1 && d == fused::kDK && r >= 1 && r <= 64;
}

void fused_geometry(int B, int H, int n, int *q, int *ctas, int *maxslots, int *cps)
{
    const int TPS = (n + 127) / 128;
    const long long BH = (long long)B * H, NT = BH * TPS;
    const int sms = fused::num_sms();
    // aligned mapping when whole groups of CTAs per slice fill (nearly) all SMs: every CTA then has one
    // (slice, side) per side and pass, and the CTAs of a slice stay in step
    const int c = BH <= sms ? (int)(sms / BH) : 0;
    if (c >= 1 && TPS >= c && BH * c * 100 >= 85ll * sms) {
        *cps = c;
        *q = (TPS + c - 1) / c;
        *ctas = (int)(BH * c);
        *maxslots = c;
        return;
    }
    *cps = 0;
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
    int q, ctas, ms, cps;
    fused_geometry(B, H, n, &q, &ctas, &ms, &cps);
    size_t o = 0;
    L.status = o; o += 256;
    L.G = o; o += up256((size_t)2 * BH * RP * 4);
    L.epoch = o; o += up256((size_t)2 * BH * 4);
    L.iter = o; o += up256((size_t)2 * BH * 4);
    L.robust = o; o += up256((size_t)2 * BH * 4);
    L.wflag = o; o += up256((size_t)BH * ms * 4);
    L.gnat = o; o += up256((size_t)2 * BH * r * 4);
    L.decision = o; o += up256((size_t)2 * BH * 4);
    L.part = o; o += up256((size_t)2 * 2 * BH * ms * RP * 2 * 8);
    L.head_end = o;
    L.kt = o; o += RP == 64 ? up256((size_t)2 * BH * ((n + 127) / 128) * 128 * 64 * 2) : 0;
    L.zprep = o; o += up256((size_t)H * 2 * RP * d * 2);
    L.wpart = o; o += up256((size_t)BH * ms * 64 * d * 4);
    L.wpart2 = o; o += fused_ext_apply(B, H, n, r, 2) ? up256(stored_apply_wpart_bytes(B, H, n)) : 0;
    L.total = o;
    return L;
}

template <int RP, bool EXT>
static cudaError_t launch_forward(const fused::FusedParams &P, int ctas, cudaStream_t st)
{
    // the attribute is per device: remember where it has been set
    static std::mutex mu;
    static bool attr_set[64] = {};
    auto kern = fused::fused_forward_kernel<RP, EXT>;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!attr_set[dev]) {
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, fused::Plan::dyn_bytes);
            if (e != cudaSuccess) return e;
            attr_set[dev] = true;
        }
    }
    // cooperative launch: the CTAs wait for one another, so all of them must be resident at once
    void *args[] = {const_cast<fused::FusedParams *>(&P)};
    return cudaLaunchCooperativeKernel(reinterpret_cast<void *>(kern), dim3(ctas), dim3(fused::kThreads), args,
                                       fused::Plan::dyn_bytes, st);
}

cudaError_t fused_attention(const void *q, const void *k, const void *v, const float *z, const float *beta,
                            const int32_t *key_len, int B, int H, int n, int d, int r, float eps, int iters,
                            void *out, float *g1_out, float *g2_out, void *ws, const unsigned *redo, unsigned redo_tag,
                            cudaStream_t st)
{
    using namespace fused;
    const int BH = B * H, RP = pad_r(r);
    FusedLayout L = fused_layout(B, H, n, d, r);
    char *w = static_cast<char *>(ws);
    cudaError_t e;

    FusedParams P;
    memset(&P, 0, sizeof(P));
    __nv_bfloat16 *zp = reinterpret_cast<__nv_bfloat16 *>(w + L.zprep);
    if (!make_map(&P.tmQ, q, BH, n, d, 128) || !make_map(&P.tmK, k, BH, n, d, 128) ||
        !make_map(&P.tmV, v, BH, n, d, 128) || !make_map(&P.tmZ, zp, 2 * H, RP, d, RP))
        return cudaErrorInvalidValue;
    P.npad = ((n + 127) / 128) * 128;
    P.Kt = (RP == 64 && iters > 1) ? reinterpret_cast<__nv_bfloat16 *>(w + L.kt) : nullptr;
    if (P.Kt != nullptr && (!make_map(&P.tmKt, P.Kt, 2 * BH, P.npad, 64, 128) || !make_map(&P.tmKtS, P.Kt, 2 * BH, P.npad, 64, 32)))
        return cudaErrorInvalidValue;
    P.beta = beta; P.key_len = key_len;
    P.G = reinterpret_cast<float *>(w + L.G);
    P.part = reinterpret_cast<unsigned long long *>(w + L.part);
    P.epoch = reinterpret_cast<int *>(w + L.epoch);
    P.iter = reinterpret_cast<int *>(w + L.iter);
    P.robust = reinterpret_cast<int *>(w + L.robust);
    P.wpart = reinterpret_cast<float *>(w + L.wpart);
    P.wflag = reinterpret_cast<int *>(w + L.wflag);
    P.out = static_cast<__nv_bfloat16 *>(out);
    P.g1_out = g1_out; P.g2_out = g2_out;
    P.redo = redo; P.redo_tag = redo_tag;
    P.ext_apply = fused_ext_apply(B, H, n, r, iters) && redo == nullptr ? 1 : 0;
    P.decision = reinterpret_cast<int *>(w + L.decision);
    P.status = reinterpret_cast<int *>(w + L.status);
    P.B = B; P.H = H; P.n = n; P.r = r; P.T = iters;
    P.TPS = (n + 127) / 128;
    int ctas;
    fused_geometry(B, H, n, &P.q, &ctas, &P.maxslots, &P.cps);
    P.eps_ln2 = (float)((double)eps * 0.6931471805599453);

    const float scale = (float)(1.4426950408889634 / (double)eps);
    const int total = H * RP * d;
    // the words after the 256-byte status block up to head_end must start at zero: the same kernel clears them
    const size_t head_vecs = (L.head_end - 256) / 16;
    int blocks = (int)((head_vecs + 255) / 256);
    if (blocks < (total + 255) / 256) blocks = (total + 255) / 256;
    if (blocks > 1184) blocks = 1184;
    zprep_kernel<<<blocks, 256, 0, st>>>(z, zp, key_len, P.status, reinterpret_cast<uint4 *>(w + 256), head_vecs,
                                         B, H, r, RP, d, scale, g1_out, g2_out, iters, redo, redo_tag);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;

    if (RP == 16) e = launch_forward<16, false>(P, ctas, st);
    else if (RP == 32) e = launch_forward<32, false>(P, ctas, st);
    else if (P.ext_apply) e = launch_forward<64, true>(P, ctas, st);
    else e = launch_forward<64, false>(P, ctas, st);
    if (e != cudaSuccess || !P.ext_apply) return e;
    // the apply stages from the stored kernel, for every slice the Sinkhorn kernel left to them
    return stored_apply(P.Kt, P.npad, P.G, beta, key_len, P.decision, v, out, reinterpret_cast<float *>(w + L.wpart2), P.status,
                        B, H, n, r, st);
}

int fused_launches(int B, int H, int n, int r, int iters) { return fused_ext_apply(B, H, n, r, iters) ? 4 : 2; }

} // namespace lot
