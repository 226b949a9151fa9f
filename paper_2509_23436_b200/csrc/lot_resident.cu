// Resident tensor-core path of the LOT attention forward for bf16 tensors, d = 64, r <= 64 (sm_100a): ONE
// persistent, cooperatively launched kernel in which the stabilised Gibbs kernel of the scaling form of
// Eq. (1)-(2), K~_it = 2^(L_it - max_t L_it) with L = C log2(e)/eps, stays on the SM between the Sinkhorn
// iterations.
//
//   phase X  (first pass)  token tiles (128 tokens x 64, TMA, 128-byte swizzle) -> logits by tcgen05.mma against the
//            pivots (scaled by log2(e)/eps, split into bf16 hi + lo by the thread block itself) -> one ex2 per
//            entry -> K~ as bf16: query side packed two per 32-bit TMEM column (tcgen05.st), key side written over
//            the token tile it came from, in place in shared memory.  The first pivot update comes out of the same
//            pass.
//   phase S  (passes 2..T)  the paper's matrix-vector scalings on the resident tiles: with w_t = 2^(G_t - max G),
//            s_i = sum_t K~_it w_t and c_t = sum_i K~_it / s_i: two packed FMAs per entry, no exponential, no
//            tensor-core work, no global-memory traffic except the column partials.
//   phase W  W = Gamma2 V on tensor cores straight from the resident key tiles (MN-major A operand); the value
//            rows are scaled by 1/s_j in shared memory.  The blocks of a slice add one another's partials.
//   phase O  out = K~1 (Diag(w1) W') / s_i: query tiles copied from TMEM to shared memory as the A operand, output
//            rows staged over them and written by TMA.
//
// Work split.  "Split" mode: the slice-major tile list of each side is cut into one contiguous range per thread
// block (at most two slices per block); the blocks that share a (slice, side) all-gather their column partials
// through global memory as 64-bit words that carry a call-unique tag beside the value, so nothing has to be
// cleared between calls.  "Whole" mode (short sequences): every block owns whole slices, up to two at a time
// (a "wave"), and nothing crosses blocks.  Capacity per block and wave: 14 key-side tiles (12 resident slots plus
// 2 that spill to global memory and come back into the two auxiliary buffers) and 448 TMEM columns of query-side
// tiles; problems beyond that take the streamed kernel (lot_fused.cu).
//
// The stored bf16 kernel cannot represent a problem whose potentials spread over more than 96 binades or whose
// column mass underflows; such a call raises the redo word and the streamed kernel, launched behind this one on
// the same stream, recomputes it (it returns at once when the word is not raised).
//
// Warp roles: 0 TMA producer, 1 MMA issuer and TMEM owner, 2 publisher, 3 gatherer, 4-11 two worker quads (one
// warp per TMEM lane quarter each).  Barrier discipline: every mbarrier has waiters that see each of its phases in
// order (per-quad and per-tile barriers wherever the two quads take turns), because a parity wait cannot tell
// phase f from phase f - 2; all barriers are re-initialised between the phases, so phase counts never leave a
// phase.  Every wait is bounded in time and raises LOT_DEV_TIMEOUT.
#include "lot_common.cuh"
#include "lot_internal.h"
#include "lot_sm100.cuh"
#include "lot_tile.cuh"

#include <cuda.h>
#include <string.h>

#include <atomic>
#include <mutex>

namespace lot {
namespace resident {

using namespace sm100;
using namespace tile;

constexpr int kTileRows = 128;
constexpr int kDK = 64;
constexpr int kTileBytes = kTileRows * kDK * 2;     // 16 KB: a token tile, a stored key-side tile, a value tile
constexpr int kSlots = 12;                          // resident key-side tiles
constexpr int kAux = 2;                             // auxiliary buffers: pivots / spilled tiles / value tiles / W''
constexpr int kBufs = kSlots + kAux;
constexpr int kMaxSeg = 4;                          // (slice, side) segments of a wave: two slices x two sides
constexpr int kThreads = 384;
constexpr int kWorkers = 256;
constexpr int kAccCol = 448;                        // 64 TMEM columns of accumulator behind the query-side tiles
constexpr float kPlainFloor = 8.2718061e-25f;       // 2^-80: smallest column mass the plain sums may report
// Largest spread of the pivot potentials (in binades) the stored kernel serves: with w_t = 2^(G_t - max G) >= 2^-96 a row
// sum is at least 2^-96, its reciprocal and the column sums stay far inside the float range, and an entry that matters
// for a row (within 2^-24 of the row's largest product K~ w) is at least 2^-120, which bf16 still holds.
constexpr float kMaxSpread = 96.f;

struct alignas(64) ResParams {
    CUtensorMap tmQ, tmK, tmV, tmO;  // [BH][n][64] bf16, box 64 x 128 x 1, 128-byte swizzle
    CUtensorMap tmS;                 // spilled key-side tiles [ctas * 2][128][64] bf16, same box
    const float *z;                  // [H][r][64]
    const float *beta;               // [H][r]
    const int32_t *key_len;          // [B] or nullptr
    unsigned long long *part;        // [2 pass parities][2 sides][BH][maxslots][RP] tagged words (value | tag << 32)
    float *wpart;                    // [BH][maxslots][64 pivots][64 channels] per-block partial of Gamma2 V
    unsigned long long *wflag;       // [BH][maxslots] tagged word: that partial is complete
    unsigned long long *status;      // device status word (flags | tag << 32)
    unsigned *redo;                  // == tag: the streamed kernel has to recompute this call
    float *g1_out, *g2_out;          // [BH][r] or nullptr
    int B, H, n, r, T;
    int TPS;                         // tiles per slice
    int NT;                          // tiles per side = BH * TPS
    int ctas;
    int maxslots;
    int whole;                       // 1: whole-slice mode
    int wave_slices;                 // whole mode: slices per wave (1 or 2)
    unsigned tag;                    // call-unique tag base; pass p uses tag + p + 1
    float scale;                     // log2(e) / eps
    float eps_ln2;
    unsigned long long wait_ns;      // limit of every device-side wait
    int skip_publish_cta;            // test hook: that block never publishes its first column partial (-1: none)
    unsigned long long *trace;       // profiling hook: block 0 logs (event, nanoseconds) pairs here, or nullptr
};

// ---------------------------------------------------------------------------------------
// Shared-memory plan (dynamic shared memory only; its base must be 1024-byte aligned)
// ---------------------------------------------------------------------------------------
struct SegInfo {           // one (slice, side) range of this block in the current wave
    int s, h;
    int nvalid;            // valid tokens of that side of the slice
    int t0, t1;            // tile range inside the slice (empty when t0 >= t1)
    int slot, nslots;      // this block's rank among the blocks that hold tiles of it, and their number
    int first;             // index of its first tile in this block's per-side tile numbering
    int kv;                // valid keys of the slice
    int wslot, wslots;     // rank among / number of the blocks that publish a partial of W for this slice
};
struct Misc {
    volatile int abort;
    volatile int phase;    // phase in progress (for the record a timed-out wait leaves)
    uint32_t tmem;
    int nseg;              // 2 or 4 entries of seg[] in use
    int nQ, nK;            // tiles of this wave per side
    int have_wave;
    SegInfo seg[kMaxSeg];  // order: queries of slice a, keys of a, queries of slice b, keys of b
    uint8_t worder[16];    // phase W: key tile (per-side index) processed at position k
    uint8_t wbuf[16];      // phase W: buffer of the value tile of position k
    uint8_t kbuf[2];       // phase W: buffer of spilled key tile o
    int8_t wdep[18];       // phase W: position whose MMA frees the buffer of load i (-1: free at the start)
};
struct Plan {
    static constexpr int offBuf = 0;
    static constexpr int offBar = kBufs * kTileBytes;          // 64 mbarriers
    static constexpr int offW = offBar + 64 * 8;               // float sW[kMaxSeg][64]: weights 2^(G - max G)
    static constexpr int offPart = offW + kMaxSeg * 64 * 4;    // float sPart[4][64]: column partials, one row per lane quarter
    static constexpr int offMail = offPart + 4 * 64 * 4;       // float sMail[64]: a sole owner's column sums, publisher -> gatherer
    static constexpr int offMisc = offMail + 64 * 4;
    static constexpr int total = offMisc + 256;
    static_assert(sizeof(Misc) <= 256, "misc block");
    static_assert(total <= 232448, "shared-memory plan exceeds the per-block limit");
};
// Barriers are initialised once per thread block.  Ids are grouped by arrival count, so that the phases of the kernel
// can reuse them; between phases every barrier is brought back to an even number of completed phases (see
// settle_bars), which lets every phase count its own barrier phases from zero.
enum BarId {
    // ---- all phases
    bP1 = 0,          //      (4) quad 1 left its column partials
    bP2 = 1,          //      (4) quad 0 added its own (the publisher waits)
    bPFree = 2,       //      partials consumed by the publisher
    bWReady = 3,      // [4]  weights of a segment's next pass in shared memory
    bMail = 7,        //      a sole owner's column sums are in the mailbox (the gatherer waits)
    bMailFree = 8,    //      mailbox read
    // ---- arrival count 1, one per buffer or tile
    bFull = 10,       // [14] X: buffer filled by TMA (waited on by the MMA issuer only)
    bVFull = 10,      // [14] W: value tile of position k landed (the quad of position k waits, once)
    bEmpty = 24,      // [14] X: buffer released (waited on by the producer only)
    bWDone = 24,      // [14] W: both MMAs of position k complete (the producer waits, in position order)
    // ---- arrival count 1
    bAccFull = 38,    // [2]  X: logits accumulator of a tile complete, per quad
    bKFull = 38,      // [2]  W: spilled key tile o landed
    bOFull = 38,      // [2]  O: output accumulator complete, per quad
    bSFull = 40,      // [2]  S: spilled tile o back in auxiliary buffer o
    bWFull = 40,      // [2]  W: accumulator of key segment j complete
    bHiDone = 42,     // [2]  W: the hi-part MMAs of a quad's tile have read the value buffer, per quad
    // ---- arrival count 4 (the warps of a quad)
    bAccEmpty = 46,   // [2]  X: accumulator read out, per quad
    bVHi = 46,        // [2]  W: value tile rewritten with the hi part of the scaled rows, per quad
    bAFull = 46,      // [2]  O: query tile staged as A operand, per quad
    bVLo = 48,        // [2]  W: value tile rewritten with the lo part, per quad
    bORead = 48,      // [2]  O: output accumulator read out, per quad
    // ---- arrival count 8 (all worker warps)
    bZFull = 50,      //      X: pivot operands written
    bWRead = 50,      // [2]  W: accumulator of key segment j read out
    bCount = 52
};
__host__ __device__ constexpr int bar_count(int id)
{
    return (id == bP1 || id == bP2 || (id >= 46 && id < 50)) ? 4 : ((id >= 50 && id < 52) ? 8 : 1);
}

// ---------------------------------------------------------------------------------------
// Context shared by the warp roles
// ---------------------------------------------------------------------------------------
struct Ctx {
    const ResParams &P;
    uint8_t *smem;
    uint32_t sbase;
    uint64_t *bars;
    Misc *M;
    float *sW, *sPart, *sMail;
    int warp, lane;
    __device__ __forceinline__ uint32_t bar(int id) const { return smem_u32(bars + id); }
    __device__ __forceinline__ uint8_t *buf(int b) const { return smem + Plan::offBuf + b * kTileBytes; }
    __device__ __forceinline__ uint32_t bufa(int b) const { return sbase + Plan::offBuf + b * kTileBytes; }
};

// Raise a device status flag: the word keeps the flags of the call whose tag it carries.
__device__ __noinline__ void raise_flag(const ResParams &P, unsigned flag)
{
    unsigned long long old = *reinterpret_cast<volatile unsigned long long *>(P.status);
    for (int it = 0; it < 1024; ++it) {
        const unsigned long long base = (unsigned)(old >> 32) == P.tag ? old : ((unsigned long long)P.tag << 32);
        const unsigned long long got = atomicCAS(P.status, old, base | flag);
        if (got == old) return;
        old = got;
    }
}

// Profiling hook: block 0 appends (warp << 32 | code, global timer) to the trace buffer (word 0 counts the entries, at
// most 4000).
__device__ __forceinline__ void trace(const Ctx &c, unsigned code)
{
    if (c.P.trace != nullptr && blockIdx.x == 0 && c.lane == 0) {
        const unsigned long long n = atomicAdd(c.P.trace, 1ull);
        if (n < 4000) { c.P.trace[1 + 2 * n] = ((unsigned long long)c.warp << 32) | code; c.P.trace[2 + 2 * n] = global_timer_ns(); }
    }
}

// Diagnostic record of a wait that gave up: (tag << 32) | block << 20 | phase << 16 | barrier << 8 | warp, one word per
// warp behind the status and redo words (barrier >= 100: a poll of global memory).
__device__ __noinline__ void record_timeout(const ResParams *P, volatile Misc *M, int warp, int barid)
{
    unsigned long long *info = P->status + 2 + blockIdx.x * 12 + warp;
    const unsigned long long mine = ((unsigned long long)P->tag << 32) | ((unsigned)blockIdx.x << 20) |
                                    ((unsigned)(M->phase & 15) << 16) | ((unsigned)(barid & 255) << 8) | (unsigned)warp;
    const unsigned long long old = *reinterpret_cast<volatile unsigned long long *>(info);
    if ((unsigned)(old >> 32) != P->tag) atomicCAS(info, old, mine);
}

// The timed part of a barrier wait; the cold path takes plain values so that the callers' context stays in registers.
__device__ __noinline__ bool bar_wait_slow(uint32_t b, uint32_t parity, uint32_t bar0, volatile Misc *M, const ResParams *P, int warp)
{
    uint64_t t0 = 0;
    for (uint32_t it = 0;; ++it) {
        if (mbar_try_wait(b, parity)) return true;
        if ((it & 63u) == 63u) {
            if (M->abort) return false;
            const uint64_t now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > P->wait_ns) break;
        }
    }
    M->abort = 1;
    record_timeout(P, M, warp, (int)((b - bar0) >> 3));
    raise_flag(*P, 4 /* LOT_DEV_TIMEOUT */);
    return false;
}
__device__ __forceinline__ bool bar_wait(const Ctx &c, int id, uint32_t parity)
{
    const uint32_t b = c.bar(id);
    if (mbar_try_wait(b, parity)) return true;
    if (mbar_try_wait(b, parity)) return true;
    return bar_wait_slow(b, parity, c.bar(0), c.M, &c.P, c.warp);
}
// whole-warp wait with a warp-uniform verdict
__device__ __forceinline__ bool warp_wait(const Ctx &c, int id, uint32_t parity)
{
    const bool r = bar_wait(c, id, parity);
    return __all_sync(0xffffffffu, r) != 0;
}
// lane 0 arrives for its warp, after the warp's earlier shared-memory accesses
__device__ __forceinline__ void warp_arrive(const Ctx &c, int id)
{
    __syncwarp();
    if (c.lane == 0) mbar_arrive(c.bar(id));
}

// ---------------------------------------------------------------------------------------
// Geometry
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ int range_lo(const ResParams &P, int cta) { return (int)(((long long)cta * P.NT) / P.ctas); }
// block that holds tile u of the slice-major list (split mode)
__device__ __forceinline__ int cta_of_tile(const ResParams &P, int u) { return (int)((((long long)u + 1) * P.ctas - 1) / P.NT); }

// Fill the segment table of wave `wave` (one thread).
__device__ __noinline__ void build_wave(const ResParams &P, Misc *M, int wave)
{
    const int cta = blockIdx.x;
    int s_first = 0, s_count = 0, u0 = 0, u1 = 0;
    M->have_wave = 0;
    M->nseg = 0; M->nQ = 0; M->nK = 0;
    if (P.whole) {
        const int BH = P.B * P.H;
        const int lo = (int)(((long long)cta * BH) / P.ctas), hi = (int)(((long long)(cta + 1) * BH) / P.ctas);
        s_first = lo + wave * P.wave_slices;
        if (s_first >= hi) return;
        s_count = min(P.wave_slices, hi - s_first);
    } else {
        if (wave > 0) return;
        u0 = range_lo(P, cta); u1 = range_lo(P, cta + 1);
        if (u0 >= u1) return;
        s_first = u0 / P.TPS;
        s_count = (u1 - 1) / P.TPS - s_first + 1;
    }
    M->have_wave = 1;
    int nQ = 0, nK = 0, ns = 0;
    for (int j = 0; j < s_count; ++j) {
        const int s = s_first + j, b = s / P.H, h = s % P.H;
        int kv = P.n;
        if (P.key_len != nullptr) kv = min(max(__ldg(P.key_len + b), 0), P.n);
        const int vtk = (kv + kTileRows - 1) / kTileRows;
        int t0 = 0, t1 = P.TPS;
        if (!P.whole) { t0 = max(u0 - s * P.TPS, 0); t1 = min(u1 - s * P.TPS, P.TPS); }
        const int c_lo = P.whole ? cta : cta_of_tile(P, s * P.TPS);
        int wslots = 0;
        if (vtk > 0) wslots = P.whole ? 1 : cta_of_tile(P, s * P.TPS + vtk - 1) - c_lo + 1;
        for (int side = 0; side < 2; ++side) {
            SegInfo &g = M->seg[ns++];
            g.s = s; g.h = h; g.kv = kv; g.wslots = wslots; g.wslot = cta - c_lo;
            g.nvalid = side ? kv : P.n;
            g.t0 = t0;
            g.t1 = side ? min(t1, vtk) : t1;
            if (g.t1 < g.t0) g.t1 = g.t0;
            const int vt = side ? vtk : P.TPS;
            g.slot = cta - c_lo;
            g.nslots = P.whole ? 1 : (vt > 0 ? cta_of_tile(P, s * P.TPS + vt - 1) - c_lo + 1 : 0);
            g.first = side ? nK : nQ;
            if (side) nK += g.t1 - g.t0; else nQ += g.t1 - g.t0;
        }
    }
    for (int i = ns; i < kMaxSeg; ++i) {
        SegInfo &g = M->seg[i];
        g.s = 0; g.h = 0; g.nvalid = 0; g.t0 = g.t1 = 0; g.slot = 0; g.nslots = 0; g.first = 0; g.kv = 0; g.wslot = 0; g.wslots = 0;
    }
    M->nseg = ns; M->nQ = nQ; M->nK = nK;
    // Phase W order: per key segment its resident tiles first, then its spilled ones (the spilled tiles are the first
    // nSp key tiles; they come back from global memory into buffers that have fallen free by then).
    const int nSp = max(nK - kSlots, 0);
    {
        int pos = 0;
        for (int sg = 1; sg < kMaxSeg; sg += 2) {
            const SegInfo &g = M->seg[sg];
            const int lo = g.first, hi = g.first + (g.t1 - g.t0);
            for (int kk = max(lo, nSp); kk < hi; ++kk) M->worder[pos++] = (uint8_t)kk;
            for (int kk = lo; kk < min(hi, nSp); ++kk) M->worder[pos++] = (uint8_t)kk;
        }
    }
    // Which buffer each load of phase W goes to.  Free buffers form a queue: the two auxiliary ones at the start, then,
    // as the MMA of position j completes, the buffer of its value tile and the buffer its key tile sat in.  Loads in
    // order: for position k = 0.., first the key tile itself if it was spilled, then its value tile.
    {
        uint8_t q[40]; int8_t qd[40];
        int qh = 0, qt = 0, li = 0, freed = 0;
        q[qt] = kSlots; qd[qt++] = -1;
        q[qt] = kSlots + 1; qd[qt++] = -1;
        for (int k = 0; k < nK; ++k) {
            const int kk = M->worder[k];
            for (int what = (kk < nSp ? 0 : 1); what < 2; ++what) {
                while (qh == qt) {                       // the next MMA frees its two buffers
                    const int j = freed++, kj = M->worder[j];
                    q[qt] = M->wbuf[j]; qd[qt++] = (int8_t)j;
                    q[qt] = kj < nSp ? M->kbuf[kj] : (uint8_t)(kj - nSp); qd[qt++] = (int8_t)j;
                }
                if (what == 0) M->kbuf[kk] = q[qh]; else M->wbuf[k] = q[qh];
                M->wdep[li++] = qd[qh++];
            }
        }
    }
}

// Per-side tile index -> segment and tile inside the slice.
__device__ __forceinline__ void locate(const Misc *M, int side, int idx, int &seg, int &t)
{
    const SegInfo &g0 = M->seg[side];
    const int n0 = g0.t1 - g0.t0;
    if (idx < n0) { seg = side; t = g0.t0 + idx; }
    else { seg = 2 + side; t = M->seg[2 + side].t0 + (idx - n0); }
}
// Phase X processes the query tiles first (per-side index k), then the key tiles (index k - nQ); the first
// nSp = max(nK - 12, 0) key tiles are the spilled ones.  Buffer of tile k: ring over the 12 slots for query and spilled
// tiles; a resident key tile lands in its own slot and stays there.
__device__ __forceinline__ int xbuf(const Misc *M, int k)
{
    const int nRing = M->nQ + max(M->nK - kSlots, 0);
    return k < nRing ? k % kSlots : k - nRing;
}
// buffer of key tile kk in phases S (spilled tiles in the auxiliary buffers) and W (spilled tiles in M->kbuf)
__device__ __forceinline__ int kslot(const Misc *M, int kk, bool phase_w)
{
    const int nSp = max(M->nK - kSlots, 0);
    if (kk >= nSp) return kk - nSp;
    return phase_w ? M->kbuf[kk] : kSlots + kk;
}

// ---------------------------------------------------------------------------------------
// Role: TMA producer (lane 0 of warp 0)
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void tma_tile(const Ctx &c, const CUtensorMap *map, int b, int barid, int row, int outer)
{
    mbar_arrive_expect_tx(c.bar(barid), kTileBytes);
    tma_load_3d(c.bufa(b), map, c.bar(barid), 0, row, outer);
}

__device__ __noinline__ void producer_x(const Ctx c)
{
    const ResParams &P = c.P;
    const Misc *M = c.M;
    const int nX = M->nQ + M->nK, nRing = M->nQ + max(M->nK - kSlots, 0);
    unsigned long long fills = 0, rels = 0;      // 4 bits per buffer: loads issued into it / releases of it waited for
    for (int k = 0; k < nX; ++k) {
        const int b = xbuf(M, k);
        const int f = (int)((fills >> (4 * b)) & 15ull);
        // the buffer's previous user (a query or spilled tile of the ring) must have released it
        if (f > 0) {
            if (!bar_wait(c, bEmpty + b, (f - 1) & 1)) return;
            rels += 1ull << (4 * b);
        }
        fills += 1ull << (4 * b);
        int seg, t;
        const int side = k < M->nQ ? 0 : 1;
        locate(M, side, side ? k - M->nQ : k, seg, t);
        tma_tile(c, side ? &P.tmK : &P.tmQ, b, bFull + b, t * kTileRows, M->seg[seg].s);
    }
    // every release of a ring tile must have arrived before the barriers are settled for the next phase
    for (int b = 0; b < kSlots; ++b) {
        const int ring_uses = b < nRing ? (nRing - 1 - b) / kSlots + 1 : 0;
        for (int f = (int)((rels >> (4 * b)) & 15ull); f < ring_uses; ++f)
            if (!bar_wait(c, bEmpty + b, f & 1)) return;
    }
}
__device__ __noinline__ void producer_s(const Ctx c)
{
    const Misc *M = c.M;
    const int nSp = max(M->nK - kSlots, 0);
    if (c.P.T >= 2)
        for (int o = 0; o < nSp; ++o) tma_tile(c, &c.P.tmS, kSlots + o, bSFull + o, 0, blockIdx.x * 2 + o);
    // the value tiles of phase W: asked into the L2 now, while the Sinkhorn passes need no memory traffic
    for (int k = 0; k < M->nK; ++k) {
        int seg, t;
        locate(M, 1, k, seg, t);
        asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];"
                     ::"l"(reinterpret_cast<uint64_t>(&c.P.tmV)), "r"(0), "r"(t * kTileRows), "r"(M->seg[seg].s) : "memory");
    }
}
__device__ __noinline__ void producer_w(const Ctx c)
{
    const ResParams &P = c.P;
    const Misc *M = c.M;
    const int nSp = max(M->nK - kSlots, 0);
    int li = 0, seen = 0;               // MMAs whose completion has been waited for (they complete in position order)
    for (int k = 0; k < M->nK; ++k) {
        const int kk = M->worder[k];
        int seg, t;
        locate(M, 1, kk, seg, t);
        for (int what = (kk < nSp ? 0 : 1); what < 2; ++what) {
            const int dep = M->wdep[li++];
            while (seen <= dep) { if (!bar_wait(c, bWDone + seen, 0)) return; ++seen; }
            if (what == 0) tma_tile(c, &P.tmS, M->kbuf[kk], bKFull + kk, 0, blockIdx.x * 2 + kk);
            else tma_tile(c, &P.tmV, M->wbuf[k], bVFull + k, t * kTileRows, M->seg[seg].s);
        }
    }
    // every MMA completion must have arrived before the barriers are settled for the next phase
    while (seen < M->nK) { if (!bar_wait(c, bWDone + seen, 0)) return; ++seen; }
}

// ---------------------------------------------------------------------------------------
// Role: MMA issuer (warp 1; the whole warp runs the loops with warp-uniform values, one elected lane issues)
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ uint64_t desc64(uint32_t hi, uint32_t lo) { return ((uint64_t)hi << 32) | lo; }

template <int RP>
__device__ __noinline__ void mma_x(const Ctx c)
{
    const Misc *M = c.M;
    const int nX = M->nQ + M->nK, nRing = M->nQ + max(M->nK - kSlots, 0);
    const uint32_t tm = c.M->tmem + kAccCol;
    constexpr uint32_t idesc = make_idesc_bf16(128, RP, 0, 0);
    const uint64_t dK = make_smem_desc(c.sbase, 16, 1024);
    const uint32_t d_hi = (uint32_t)(dK >> 32), d_lo = (uint32_t)dK;
    bool ok = warp_wait(c, bZFull, 0);
    unsigned long long fills = 0;
    for (int k = 0; k < nX && ok; ++k) {
        const int b = xbuf(M, k);
        const int f = (int)((fills >> (4 * b)) & 15ull);
        fills += 1ull << (4 * b);
        ok = warp_wait(c, bFull + b, f & 1);
        if (ok && k >= 1) ok = warp_wait(c, bAccEmpty + ((k - 1) & 1), ((k - 1) >> 1) & 1);
        if (!ok) break;
        tc_fence_after();
        trace(c, 0x100 + k);
        int seg, t;
        const int side = k < M->nQ ? 0 : 1;
        locate(M, side, side ? k - M->nQ : k, seg, t);
        const uint32_t xa = d_lo + ((Plan::offBuf + b * kTileBytes) >> 4);
        const uint32_t za = d_lo + ((Plan::offBuf + (kSlots + (seg >> 1)) * kTileBytes) >> 4);
        if (elect_one()) {
#pragma unroll
            for (int part = 0; part < 2; ++part)
#pragma unroll
                for (int ks = 0; ks < kDK / 16; ++ks)
                    umma_bf16(tm, desc64(d_hi, xa + ks * 2), desc64(d_hi, za + part * ((RP * 128) >> 4) + ks * 2), idesc,
                              (part | ks) ? 1u : 0u);
            umma_commit(c.bar(bAccFull + (k & 1)));
            if (k < M->nQ) umma_commit(c.bar(bEmpty + b));       // a spilled tile's buffer is released by its store
        }
        __syncwarp();
    }
    (void)nRing;
}

// The value rows reach the tensor cores scaled by 1/s_j, as a bf16 hi part and a bf16 lo part (one rounding of the
// product would cost the output three times its own bf16 rounding).  Both parts pass through the tile's one buffer:
// the hi-part MMAs of position k, the hi-part MMAs of position k + 1 (the other quad's), then the lo-part MMAs of
// position k, which its quad has written over the hi part meanwhile.
__device__ __noinline__ void mma_w(const Ctx c)
{
    const Misc *M = c.M;
    const int nSp = max(M->nK - kSlots, 0);
    const uint32_t tm = c.M->tmem + kAccCol;
    constexpr uint32_t idesc = make_idesc_bf16(64, kDK, 1, 1);
    const uint64_t dMN = make_smem_desc(c.sbase, kTileBytes, 1024);
    const uint32_t d_hi = (uint32_t)(dMN >> 32), d_lo = (uint32_t)dMN;
    const int n1 = M->seg[1].t1 - M->seg[1].t0;       // positions [0, n1) belong to the first key segment
    bool ok = true;
    int pending = -1;                                 // position whose lo part is still to be issued
    auto issue = [&](int k, bool lo_part) {
        const int kk = M->worder[k];
        const int kb = kk < nSp ? M->kbuf[kk] : kk - nSp, vb = M->wbuf[k];
        // hi and lo parts have a barrier each per quad: one barrier for both could run two phases ahead of this warp
        if (ok) ok = warp_wait(c, (lo_part ? bVLo : bVHi) + (k & 1), (k >> 1) & 1);
        if (!ok) return;
        tc_fence_after();
        const uint32_t ka = d_lo + ((Plan::offBuf + kb * kTileBytes) >> 4), va = d_lo + ((Plan::offBuf + vb * kTileBytes) >> 4);
        const bool first = !lo_part && (k == 0 || k == n1);
        if (elect_one()) {
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
                umma_bf16(tm, desc64(d_hi, ka + ks * 128), desc64(d_hi, va + ks * 128), idesc, (first && ks == 0) ? 0u : 1u);
            if (lo_part) umma_commit(c.bar(bWDone + k));
            else umma_commit(c.bar(bHiDone + (k & 1)));
        }
        __syncwarp();
    };
    for (int k = 0; k < M->nK && ok; ++k) {
        if (k == n1 && n1 > 0) {
            // segment border: finish the first key segment, and let the workers read its accumulator out
            if (pending >= 0) { issue(pending, true); pending = -1; }
            if (ok && elect_one()) umma_commit(c.bar(bWFull + 0));
            __syncwarp();
            if (ok) ok = warp_wait(c, bWRead + 0, 0);
        }
        issue(k, false);
        if (pending >= 0) issue(pending, true);
        pending = k;
    }
    if (pending >= 0) issue(pending, true);
    if (ok && M->nK > 0 && elect_one()) umma_commit(c.bar(bWFull + (n1 < M->nK ? 1 : 0)));
    __syncwarp();
}

template <int RP>
__device__ __noinline__ void mma_o(const Ctx c)
{
    const Misc *M = c.M;
    const uint32_t tm = c.M->tmem + kAccCol;
    constexpr uint32_t idesc = make_idesc_bf16(128, kDK, 0, 0);
    const uint64_t dK = make_smem_desc(c.sbase, 16, 1024);
    const uint32_t d_hi = (uint32_t)(dK >> 32), d_lo = (uint32_t)dK;
    bool ok = true;
    for (int qq = 0; qq < M->nQ && ok; ++qq) {
        const int q = qq & 1, j = qq >> 1, ab = q + 2 * (j % 3);
        ok = warp_wait(c, bAFull + q, j & 1);
        if (ok && qq >= 1) ok = warp_wait(c, bORead + ((qq - 1) & 1), ((qq - 1) >> 1) & 1);
        if (!ok) break;
        tc_fence_after();
        int seg, t;
        locate(M, 0, qq, seg, t);
        const uint32_t aa = d_lo + ((Plan::offBuf + ab * kTileBytes) >> 4);
        const uint32_t wa = d_lo + ((Plan::offBuf + (kSlots + (seg >> 1)) * kTileBytes) >> 4);
        if (elect_one()) {
#pragma unroll
            for (int part = 0; part < 2; ++part)
#pragma unroll
                for (int ks = 0; ks < RP / 16; ++ks)
                    umma_bf16(tm, desc64(d_hi, aa + ks * 2), desc64(d_hi, wa + part * ((kDK * 128) >> 4) + ks * 2), idesc,
                              (part | ks) ? 1u : 0u);
            umma_commit(c.bar(bOFull + q));
        }
        __syncwarp();
    }
}

// ---------------------------------------------------------------------------------------
// Roles: publisher (warp 2) and gatherer (warp 3).  Lane l owns pivot columns 2l and 2l + 1.
// Segment order inside a pass: queries of slice a, queries of b, keys of a, keys of b.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ int seg_at(int i) { return i == 0 ? 0 : (i == 1 ? 2 : (i == 2 ? 1 : 3)); }
__device__ __forceinline__ bool seg_active(const Misc *M, int sg) { return M->seg[sg].t1 > M->seg[sg].t0; }

__device__ __forceinline__ unsigned long long *part_slot(const ResParams &P, int RP, int pass, int side, int s, int slot)
{
    return P.part + ((((size_t)(pass & 1) * 2 + side) * (size_t)(P.B * P.H) + s) * P.maxslots + slot) * RP;
}

template <int RP>
__device__ __noinline__ void publisher(const Ctx c, int p_lo, int p_hi)
{
    const ResParams &P = c.P;
    const Misc *M = c.M;
    const int c0 = 2 * c.lane;
    const bool mine = c0 < RP;
    int nph = 0, nmail = 0;
    bool ok = true;
    for (int p = p_lo; p < p_hi; ++p)
        for (int i = 0; i < kMaxSeg; ++i) {
            const int sg = seg_at(i);
            if (!seg_active(M, sg)) continue;
            const SegInfo &g = M->seg[sg];
            if (ok) ok = warp_wait(c, bP2, nph & 1);
            ++nph;
            trace(c, 0x600 + p * 4 + sg);
            // column masses of this block's tiles: the four lane quarters' rows, times the weights of this pass
            float a0 = 0.f, a1 = 0.f;
            if (mine && ok) {
#pragma unroll
                for (int w = 0; w < 4; ++w) {
                    const float2 v = *reinterpret_cast<const float2 *>(c.sPart + w * 64 + c0);
                    a0 += v.x; a1 += v.y;
                }
                if (p > 0) { const float2 w = *reinterpret_cast<const float2 *>(c.sW + sg * 64 + c0); a0 *= w.x; a1 *= w.y; }
            }
            warp_arrive(c, bPFree);
            if (g.nslots <= 1) {
                // sole owner: straight to the gatherer through the mailbox
                if (nmail > 0 && ok) ok = warp_wait(c, bMailFree, (nmail - 1) & 1);
                ++nmail;
                if (mine) *reinterpret_cast<float2 *>(c.sMail + c0) = make_float2(a0, a1);
                warp_arrive(c, bMail);
            } else if (mine && ok && !(p == 0 && (int)blockIdx.x == P.skip_publish_cta)) {
                st_tagged2(part_slot(P, RP, p, sg & 1, g.s, g.slot) + c0, a0, a1, P.tag + (unsigned)p + 1u);
            }
        }
}

struct GatherState {
    float G[kMaxSeg][2];
};

template <int RP>
__device__ __noinline__ void gatherer(const Ctx c, GatherState &st, int p_lo, int p_hi)
{
    const ResParams &P = c.P;
    const Misc *M = c.M;
    const int c0 = 2 * c.lane;
    const bool mine = c0 < RP;
    int nph = 0;
    bool ok = true;
    for (int p = p_lo; p < p_hi; ++p)
#pragma unroll
        for (int i = 0; i < kMaxSeg; ++i) {
            const int sg = i == 0 ? 0 : (i == 1 ? 2 : (i == 2 ? 1 : 3));
            if (!seg_active(M, sg)) continue;
            const SegInfo &g = M->seg[sg];
            if (!ok) continue;
            float s0 = 0.f, s1 = 0.f;
            if (g.nslots <= 1) {
                ok = warp_wait(c, bMail, nph & 1);
                ++nph;
                if (!ok) continue;
                if (mine) { const float2 v = *reinterpret_cast<const float2 *>(c.sMail + c0); s0 = v.x; s1 = v.y; }
                warp_arrive(c, bMailFree);
            } else {
                // all slots of the (slice, side), polled until their tags match, summed in slot order
                const unsigned tag = P.tag + (unsigned)p + 1u;
                const unsigned long long *src = part_slot(P, RP, p, sg & 1, g.s, 0) + c0;
                constexpr int kBatch = 12;          // slots polled together: their loads are all in flight at once
                for (int p0 = 0; p0 < g.nslots && ok; p0 += kBatch) {
                    unsigned long long w[kBatch][2];
                    uint64_t t0 = 0;
                    for (uint32_t tries = 0;; ++tries) {
                        bool ready = true;
                        if (mine) {
#pragma unroll
                            for (int u = 0; u < kBatch; ++u)
                                if (p0 + u < g.nslots) ld_tagged2(src + (size_t)(p0 + u) * RP, w[u][0], w[u][1]);
#pragma unroll
                            for (int u = 0; u < kBatch; ++u)
                                if (p0 + u < g.nslots)
                                    ready = ready && (unsigned)(w[u][0] >> 32) == tag && (unsigned)(w[u][1] >> 32) == tag;
                        }
                        if (__all_sync(0xffffffffu, ready)) break;
                        bool giveup = c.M->abort != 0;
                        if ((tries & 7u) == 7u) {
                            const uint64_t now = global_timer_ns();
                            if (t0 == 0) t0 = now;
                            else if (now - t0 > P.wait_ns) giveup = true;
                        }
                        if (__any_sync(0xffffffffu, giveup)) {
                            if (c.lane == 0) { c.M->abort = 1; record_timeout(&P, c.M, c.warp, 100 + sg); raise_flag(P, 4 /* LOT_DEV_TIMEOUT */); }
                            ok = false;
                            break;
                        }
                        __nanosleep(32);
                    }
                    if (!ok || !mine) continue;
#pragma unroll
                    for (int u = 0; u < kBatch; ++u)
                        if (p0 + u < g.nslots) { s0 += __uint_as_float((unsigned)w[u][0]); s1 += __uint_as_float((unsigned)w[u][1]); }
                }
                if (!ok) continue;
            }
            // pivot update G_t += log2(beta_t / m) - log2(column mass), m = 1 / nvalid
            bool bad = false;
            float gmx = neg_inf(), gmn = -neg_inf();
            if (mine) {
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int col = c0 + u;
                    if (col < P.r) {
                        float ss = u ? s1 : s0;
                        if (!(ss >= kPlainFloor && ss <= 3.0e38f)) { bad = true; ss = fminf(fmaxf(ss, kPlainFloor), 3.0e38f); }
                        const float gn = st.G[i][u] + lg2(__ldg(P.beta + g.h * P.r + col) * (float)g.nvalid) - lg2(ss);
                        st.G[i][u] = gn;
                        gmx = fmaxf(gmx, gn); gmn = fminf(gmn, gn);
                        if (g.slot == 0) {
                            if (!isfinite(gn)) raise_flag(P, 1 /* LOT_DEV_NONFINITE */);
                            float *dst = (sg & 1) ? P.g2_out : P.g1_out;
                            if (p + 1 == P.T && dst != nullptr) dst[(size_t)g.s * P.r + col] = gn * P.eps_ln2;
                        }
                    }
                }
            }
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) {
                gmx = fmaxf(gmx, __shfl_xor_sync(0xffffffffu, gmx, off));
                gmn = fminf(gmn, __shfl_xor_sync(0xffffffffu, gmn, off));
            }
            // what the stored bf16 kernel cannot carry: a column mass outside the plain range, potentials spread over
            // more than kMaxSpread binades.  NaN fails the comparison too.
            if (__any_sync(0xffffffffu, bad) || !(gmx - gmn <= kMaxSpread)) {
                if (c.lane == 0) *reinterpret_cast<volatile unsigned *>(P.redo) = P.tag;
            }
            if (mine) {
                float2 w;
                w.x = c0 < P.r ? ex2(st.G[i][0] - gmx) : 0.f;
                w.y = c0 + 1 < P.r ? ex2(st.G[i][1] - gmx) : 0.f;
                *reinterpret_cast<float2 *>(c.sW + sg * 64 + c0) = w;
            }
            warp_arrive(c, bWReady + sg);
            trace(c, 0x700 + p * 4 + sg);
        }
}

// ---------------------------------------------------------------------------------------
// Role: workers (warps 4-11: quad = (warp - 4) / 4, lane quarter w4 = warp % 4)
// ---------------------------------------------------------------------------------------
struct WorkerId {
    int quad, w4, rq, cq, wtid;        // wtid: 0..255 among the workers
    uint32_t lane_addr;                // TMEM address of this warp's lane quarter, column 0
};

// Column partials of one segment: quad 1 leaves them in shared memory, quad 0 adds its own (one row per lane quarter),
// the publisher / gatherer adds the four rows.  a0, a1: this lane's totals of columns col, col + 1.
__device__ __forceinline__ bool flush_partial(const Ctx &c, const WorkerId &id, float a0, float a1, int col, bool owner,
                                              int &nflush, bool ok)
{
    float2 *dst = reinterpret_cast<float2 *>(c.sPart + id.w4 * 64 + col);
    if (id.quad == 1) {
        if (nflush > 0 && ok) ok = warp_wait(c, bPFree, (nflush - 1) & 1);
        if (owner) *dst = make_float2(a0, a1);
        warp_arrive(c, bP1);
    } else {
        if (ok) ok = warp_wait(c, bP1, nflush & 1);
        if (owner) { const float2 o = *dst; *dst = make_float2(o.x + a0, o.y + a1); }
        warp_arrive(c, bP2);
    }
    ++nflush;
    return ok;
}

// ---- phase X: pivots -> MMA operands; logits -> stabilised kernel tiles and the first column sums
template <int RP>
__device__ __noinline__ void worker_x(const Ctx c, const WorkerId id)
{
    constexpr int X = RP / 8;            // repeats of the 8-column pattern of the accumulator load
    const ResParams &P = c.P;
    const Misc *M = c.M;
    // pivots of the (one or two) heads of this wave: Z * log2(e)/eps as bf16 hi + lo, K-major, 128-byte swizzle
    {
        const int heads = M->nseg / 2;
        for (int item = id.wtid; item < heads * RP * 8; item += kWorkers) {
            const int j = item / (RP * 8), t = (item >> 3) % RP, ch = item & 7;
            float v[8];
            if (t < P.r) {
                const float4 *src = reinterpret_cast<const float4 *>(P.z + ((size_t)M->seg[2 * j].h * P.r + t) * kDK + ch * 8);
                const float4 a = __ldg(src), b = __ldg(src + 1);
                v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) v[e] = 0.f;
            }
            uint32_t hi[4], lo[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float x0 = v[2 * e] * P.scale, x1 = v[2 * e + 1] * P.scale;
                __nv_bfloat162 hh = __floats2bfloat162_rn(x0, x1);
                hi[e] = *reinterpret_cast<uint32_t *>(&hh);
                lo[e] = pack_bf16(x0 - __low2float(hh), x1 - __high2float(hh));
            }
            uint8_t *dst = c.buf(kSlots + j) + t * 128 + ((ch ^ (t & 7)) * 16);
            *reinterpret_cast<uint4 *>(dst) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
            *reinterpret_cast<uint4 *>(dst + RP * 128) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        }
        fence_proxy_async_smem();
        warp_arrive(c, bZFull);
    }
    const int nQ = M->nQ, nSp = max(M->nK - kSlots, 0);
    const bool sums = P.T > 0;
    bool ok = true;
    int nflush = 0, ntile = 0;           // ntile: tiles this quad has taken (accumulator phase of its barrier)
    bool stored = false;
    for (int i = 0; i < kMaxSeg; ++i) {
        const int sg = seg_at(i);
        if (!seg_active(M, sg)) continue;
        const SegInfo &g = M->seg[sg];
        const int side = sg & 1;
        const int k_lo = (side ? nQ : 0) + g.first, k_hi = k_lo + (g.t1 - g.t0);
        float acc[2 * X];
#pragma unroll
        for (int e = 0; e < 2 * X; ++e) acc[e] = 0.f;
        for (int k = k_lo + ((k_lo ^ id.quad) & 1); k < k_hi; k += 2) {
            const int idx = k - (side ? nQ : 0), t = g.t0 + (idx - g.first);
            const bool spill = side && idx < nSp;
            const int b = xbuf(M, k);
            if (ok) ok = warp_wait(c, bAccFull + id.quad, ntile & 1);
            ++ntile;
            if (!ok) continue;
            tc_fence_after();
            trace(c, 0x200 + k);
            // both 16-lane halves into registers, then the accumulator goes back to the MMA issuer at once
            float vv[2][4 * X];
            tmem_ld_acc<X>(id.lane_addr + kAccCol, vv[0]);
            tmem_ld_acc<X>(id.lane_addr + (16u << 16) + kAccCol, vv[1]);
            tmem_wait_ld();
            tc_fence_before();
            warp_arrive(c, bAccEmpty + id.quad);
            trace(c, 0x300 + k);
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                float (&v)[4 * X] = vv[half];
                const int rinA = id.w4 * 32 + half * 16 + id.rq;          // row inside the tile; row B = row A + 8
                const int rowA = t * kTileRows + rinA, rowB = rowA + 8;
                if (P.r < RP) {
#pragma unroll
                    for (int rep = 0; rep < X; ++rep)
#pragma unroll
                        for (int u = 0; u < 2; ++u)
                            if (rep * 8 + 2 * id.cq + u >= P.r) { v[rep * 4 + u] = neg_inf(); v[rep * 4 + 2 + u] = neg_inf(); }
                }
                float mA = neg_inf(), mB = neg_inf();
#pragma unroll
                for (int rep = 0; rep < X; ++rep) {
                    mA = max3(mA, v[rep * 4 + 0], v[rep * 4 + 1]);
                    mB = max3(mB, v[rep * 4 + 2], v[rep * 4 + 3]);
                }
                mA = fmaxf(mA, __shfl_xor_sync(0xffffffffu, mA, 1));
                mB = fmaxf(mB, __shfl_xor_sync(0xffffffffu, mB, 1));
                mA = fmaxf(mA, __shfl_xor_sync(0xffffffffu, mA, 2));
                mB = fmaxf(mB, __shfl_xor_sync(0xffffffffu, mB, 2));
                float2 sA2 = make_float2(0.f, 0.f), sB2 = make_float2(0.f, 0.f);
                uint32_t pk[2 * X];
#pragma unroll
                for (int rep = 0; rep < X; ++rep) {
                    const float2 ea = make_float2(ex2(v[rep * 4 + 0] - mA), ex2(v[rep * 4 + 1] - mA));
                    const float2 eb = make_float2(ex2(v[rep * 4 + 2] - mB), ex2(v[rep * 4 + 3] - mB));
                    v[rep * 4 + 0] = ea.x; v[rep * 4 + 1] = ea.y; v[rep * 4 + 2] = eb.x; v[rep * 4 + 3] = eb.y;
                    sA2 = __fadd2_rn(sA2, ea);
                    sB2 = __fadd2_rn(sB2, eb);
                    pk[2 * rep] = pack_bf16(ea.x, ea.y);
                    pk[2 * rep + 1] = pack_bf16(eb.x, eb.y);
                }
                // the tile's home: packed TMEM columns (queries) or the token tile's own buffer (keys)
                if (!side) {
                    tmem_st_pk<X>(id.lane_addr + ((uint32_t)(half * 16) << 16) + idx * (RP / 2), pk);
                    stored = true;
                } else {
                    const uint32_t rowaddr = c.bufa(b) + rinA * 128 + id.cq * 4;
#pragma unroll
                    for (int rep = 0; rep < X; ++rep) {
                        const uint32_t addr = rowaddr + ((rep ^ (rinA & 7)) << 4);
                        asm volatile("st.shared.b32 [%0], %1;" ::"r"(addr), "r"(pk[2 * rep]) : "memory");
                        asm volatile("st.shared.b32 [%0 + 1024], %1;" ::"r"(addr), "r"(pk[2 * rep + 1]) : "memory");
                    }
                }
                if (sums) {
                    float sA = sA2.x + sA2.y, sB = sB2.x + sB2.y;
                    sA += __shfl_xor_sync(0xffffffffu, sA, 1);
                    sB += __shfl_xor_sync(0xffffffffu, sB, 1);
                    sA += __shfl_xor_sync(0xffffffffu, sA, 2);
                    sB += __shfl_xor_sync(0xffffffffu, sB, 2);
                    const float uA = rowA < g.nvalid ? __fdividef(1.f, sA) : 0.f;
                    const float uB = rowB < g.nvalid ? __fdividef(1.f, sB) : 0.f;
                    const float2 uA2 = make_float2(uA, uA), uB2 = make_float2(uB, uB);
#pragma unroll
                    for (int rep = 0; rep < X; ++rep) {
                        float2 a2 = make_float2(acc[rep * 2], acc[rep * 2 + 1]);
                        a2 = __ffma2_rn(make_float2(v[rep * 4 + 0], v[rep * 4 + 1]), uA2, a2);
                        a2 = __ffma2_rn(make_float2(v[rep * 4 + 2], v[rep * 4 + 3]), uB2, a2);
                        acc[rep * 2] = a2.x; acc[rep * 2 + 1] = a2.y;
                    }
                }
            }
            if (spill) {
                // a spilled key tile leaves through global memory: one TMA store per tile, then its ring buffer is free
                fence_proxy_async_smem();
                named_bar_sync(2 + id.quad, 128);
                if (id.w4 == 0 && c.lane == 0) {
                    tma_store_3d(&P.tmS, c.bufa(b), 0, 0, blockIdx.x * 2 + idx);
                    bulk_commit_group();
                    bulk_wait_group_read0();
                    mbar_arrive(c.bar(bEmpty + b));
                }
            }
        }
        if (sums) {
            bool owner;
            const int eb = quad_col_reduce(acc, c.lane, owner);
            // entry pair (eb, eb + 1) of the quad layout = columns 8 (eb / 2) + 2 cq, + 1
            ok = flush_partial(c, id, acc[0], acc[1], (eb >> 1) * 8 + 2 * id.cq, owner, nflush, ok);
        }
    }
    if (stored) tmem_wait_st();
    if (id.w4 == 0 && c.lane == 0) bulk_wait_group0();        // spilled tiles have reached global memory
    fence_proxy_async_smem();                                  // key tiles written here are MMA operands in phase W
}

// ---- phase S: passes 2..T on the resident tiles
// One tile: rows rq + 8 j (j = 0..3) of this warp's 32, NW packed words (2 NW entries) per row.
//   TMEM tile: word e = columns (8 e + 2 cq, + 1).  Shared-memory tile: the thread's 4 NW bytes of the row's first
//   2 RP bytes, i.e. columns (RP / 4) cq + 2 e, + 1, read as one vector load (two for RP = 64).
template <int RP, bool TM>
__device__ __forceinline__ void load_rows(const Ctx &c, const WorkerId &id, uint32_t taddr, const uint8_t *tile,
                                          uint32_t (&d)[4][RP / 8])
{
    constexpr int NW = RP / 8;
    if constexpr (TM) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            uint32_t r[2 * NW];
            tmem_ld_pk<NW>(taddr + ((uint32_t)(half * 16) << 16), r);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < NW; ++e) { d[2 * half][e] = r[2 * e]; d[2 * half + 1][e] = r[2 * e + 1]; }
        }
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int rin = id.w4 * 32 + j * 8 + id.rq;
            const uint8_t *row = tile + rin * 128;
            if constexpr (RP == 64) {
                const uint4 a = *reinterpret_cast<const uint4 *>(row + (((2 * id.cq) ^ (rin & 7)) * 16));
                const uint4 b = *reinterpret_cast<const uint4 *>(row + (((2 * id.cq + 1) ^ (rin & 7)) * 16));
                d[j][0] = a.x; d[j][1] = a.y; d[j][2] = a.z; d[j][3] = a.w; d[j][4] = b.x; d[j][5] = b.y; d[j][6] = b.z; d[j][7] = b.w;
            } else if constexpr (RP == 32) {
                const uint4 a = *reinterpret_cast<const uint4 *>(row + ((id.cq ^ (rin & 7)) * 16));
                d[j][0] = a.x; d[j][1] = a.y; d[j][2] = a.z; d[j][3] = a.w;
            } else {
                const uint2 a = *reinterpret_cast<const uint2 *>(row + (((id.cq >> 1) ^ (rin & 7)) * 16) + (id.cq & 1) * 8);
                d[j][0] = a.x; d[j][1] = a.y;
            }
        }
    }
}
// first column of word e of this thread
template <int RP, bool TM>
__device__ __forceinline__ int word_col(const WorkerId &id, int e)
{
    return TM ? 8 * e + 2 * id.cq : (RP / 4) * id.cq + 2 * e;
}
// row sums s_j = sum_t K~_jt w_t of the thread's four rows (complete after the two quad shuffles)
template <int NW>
__device__ __forceinline__ void row_sums(const uint32_t (&d)[4][NW], const float2 (&w2)[NW], float (&sr)[4])
{
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        float2 sa = make_float2(0.f, 0.f);
#pragma unroll
        for (int e = 0; e < NW; ++e) sa = __ffma2_rn(unpack_bf16(d[j][e]), w2[e], sa);
        sr[j] = sa.x + sa.y;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) sr[j] += __shfl_xor_sync(0xffffffffu, sr[j], 1);
#pragma unroll
    for (int j = 0; j < 4; ++j) sr[j] += __shfl_xor_sync(0xffffffffu, sr[j], 2);
}

template <int RP, bool TM>
__device__ __forceinline__ bool pass_segment(const Ctx &c, const WorkerId &id, int sg, int &nflush, bool ok)
{
    constexpr int NW = RP / 8;
    const Misc *M = c.M;
    const SegInfo &g = M->seg[sg];
    const int nSp = max(M->nK - kSlots, 0);
    float2 w2[NW], c2[NW];
#pragma unroll
    for (int e = 0; e < NW; ++e) {
        w2[e] = *reinterpret_cast<const float2 *>(c.sW + sg * 64 + word_col<RP, TM>(id, e));
        c2[e] = make_float2(0.f, 0.f);
    }
    const int lo = g.first, hi = g.first + (g.t1 - g.t0);
    for (int idx = lo + ((lo ^ id.quad) & 1); idx < hi; idx += 2) {
        const int t = g.t0 + (idx - lo);
        uint32_t d[4][NW];
        if (TM) {
            load_rows<RP, true>(c, id, id.lane_addr + idx * (RP / 2), nullptr, d);
        } else {
            if (idx < nSp && ok) ok = warp_wait(c, bSFull + idx, 0);
            load_rows<RP, false>(c, id, 0, c.buf(idx < nSp ? kSlots + idx : idx - nSp), d);
        }
        float sr[4];
        row_sums<NW>(d, w2, sr);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int row = t * kTileRows + id.w4 * 32 + j * 8 + id.rq;
            const float u = row < g.nvalid ? __fdividef(1.f, sr[j]) : 0.f;
            const float2 uu = make_float2(u, u);
            // unpacked a second time on purpose: the float pairs of a whole tile would not fit the registers
#pragma unroll
            for (int e = 0; e < NW; ++e) c2[e] = __ffma2_rn(unpack_bf16(d[j][e]), uu, c2[e]);
        }
    }
    float a[2 * NW];
#pragma unroll
    for (int e = 0; e < NW; ++e) { a[2 * e] = c2[e].x; a[2 * e + 1] = c2[e].y; }
    bool owner;
    const int eb = quad_col_reduce(a, c.lane, owner);
    return flush_partial(c, id, a[0], a[1], word_col<RP, TM>(id, eb >> 1), owner, nflush, ok);
}

template <int RP>
__device__ __noinline__ void worker_s(const Ctx c, const WorkerId id)
{
    const Misc *M = c.M;
    int nflush = 0;
    bool ok = true;
    for (int p = 1; p < c.P.T; ++p)
        for (int i = 0; i < kMaxSeg; ++i) {
            const int sg = seg_at(i);
            if (!seg_active(M, sg)) continue;
            // weights of this pass: the gather of pass p - 1 (pass 0's finished before this phase began)
            trace(c, 0x400 + p * 4 + sg);
            if (p >= 2 && ok) ok = warp_wait(c, bWReady + sg, p & 1);
            trace(c, 0x500 + p * 4 + sg);
            if (sg & 1) ok = pass_segment<RP, false>(c, id, sg, nflush, ok);
            else ok = pass_segment<RP, true>(c, id, sg, nflush, ok);
        }
}

// ---- phase W: closing token update of the key side, value rows scaled by 1/s_j, W = K~2^T V' on tensor cores
template <int RP>
__device__ __noinline__ void worker_w(const Ctx c, const WorkerId id)
{
    constexpr int NW = RP / 8;
    const ResParams &P = c.P;
    const Misc *M = c.M;
    const int nSp = max(M->nK - kSlots, 0);
    const int n1 = M->seg[1].t1 - M->seg[1].t0;
    bool ok = true;
    int ntile = 0;                      // tiles this quad has taken
    for (int j = 0; j < 2; ++j) {
        const int sg = 1 + 2 * j;
        if (!seg_active(M, sg)) continue;
        const SegInfo &g = M->seg[sg];
        const int k_lo = j ? n1 : 0, k_hi = j ? M->nK : n1;
        float2 w2[NW];
#pragma unroll
        for (int e = 0; e < NW; ++e) w2[e] = *reinterpret_cast<const float2 *>(c.sW + sg * 64 + word_col<RP, false>(id, e));
        for (int k = k_lo + ((k_lo ^ id.quad) & 1); k < k_hi; k += 2) {
            const int kk = M->worder[k], t = g.t0 + (kk - g.first);
            const int kb = kk < nSp ? M->kbuf[kk] : kk - nSp, vb = M->wbuf[k];
            if (kk < nSp && ok) ok = warp_wait(c, bKFull + kk, 0);
            if (ok) ok = warp_wait(c, bVFull + k, 0);
            if (!ok) continue;
            trace(c, 0x800 + k);
            uint32_t d[4][NW];
            load_rows<RP, false>(c, id, 0, c.buf(kb), d);
            float sr[4];
            row_sums<NW>(d, w2, sr);
            // value rows times 1/s_j (0 for rows without mass): hi part in place now, lo part once the hi-part MMAs have
            // read the buffer
            uint8_t *vt = c.buf(vb);
            uint32_t lo[4][8];
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                const int rin = id.w4 * 32 + jj * 8 + id.rq, row = t * kTileRows + rin;
                const float u = row < g.nvalid ? __fdividef(1.f, sr[jj]) : 0.f;
                const float2 uu = make_float2(u, u);
#pragma unroll
                for (int h2 = 0; h2 < 2; ++h2) {
                    uint4 *p = reinterpret_cast<uint4 *>(vt + rin * 128 + (((2 * id.cq + h2) ^ (rin & 7)) * 16));
                    uint4 x = *p;
                    uint32_t *xw = reinterpret_cast<uint32_t *>(&x);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 f = __fmul2_rn(unpack_bf16(xw[e]), uu);
                        __nv_bfloat162 hh = __floats2bfloat162_rn(f.x, f.y);
                        xw[e] = *reinterpret_cast<uint32_t *>(&hh);
                        lo[jj][h2 * 4 + e] = pack_bf16(f.x - __low2float(hh), f.y - __high2float(hh));
                    }
                    *p = x;
                }
            }
            fence_proxy_async_smem();
            warp_arrive(c, bVHi + id.quad);
            if (ok) ok = warp_wait(c, bHiDone + id.quad, ntile & 1);
            ++ntile;
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                const int rin = id.w4 * 32 + jj * 8 + id.rq;
#pragma unroll
                for (int h2 = 0; h2 < 2; ++h2)
                    *reinterpret_cast<uint4 *>(vt + rin * 128 + (((2 * id.cq + h2) ^ (rin & 7)) * 16)) =
                        make_uint4(lo[jj][h2 * 4], lo[jj][h2 * 4 + 1], lo[jj][h2 * 4 + 2], lo[jj][h2 * 4 + 3]);
            }
            fence_proxy_async_smem();
            warp_arrive(c, bVLo + id.quad);
            trace(c, 0x900 + k);
        }
        // ---- this segment's accumulator: pivot rows 16 w4 .. + 15 sit in the first 16 lanes of lane quarter w4; quad q
        // takes channels 32 q .. + 31.  The partial leaves multiplied by the key-side weights w2_t.
        if (ok) ok = warp_wait(c, bWFull + j, 0);
        trace(c, 0xa00 + j);
        float v[16];
        if (ok) {
            tc_fence_after();
            tmem_ld_acc<4>(id.lane_addr + kAccCol + 32 * id.quad, v);
            tmem_wait_ld();
            tc_fence_before();
        }
        warp_arrive(c, bWRead + j);
        if (ok) {
            const int tA = 16 * id.w4 + id.rq, tB = tA + 8;
            const float wA = c.sW[sg * 64 + tA], wB = c.sW[sg * 64 + tB];
            float *dst = P.wpart + ((size_t)g.s * P.maxslots + g.wslot) * (64 * kDK) + 32 * id.quad + 2 * id.cq;
#pragma unroll
            for (int rep = 0; rep < 4; ++rep) {
                __stcg(reinterpret_cast<float2 *>(dst + tA * kDK + rep * 8), make_float2(v[rep * 4 + 0] * wA, v[rep * 4 + 1] * wA));
                __stcg(reinterpret_cast<float2 *>(dst + tB * kDK + rep * 8), make_float2(v[rep * 4 + 2] * wB, v[rep * 4 + 3] * wB));
            }
            __threadfence();
        }
        named_bar_sync(1, kWorkers);
        if (id.wtid == 0 && !c.M->abort) {
            const unsigned tag = P.tag + (unsigned)P.T + 2u;
            st_release64(P.wflag + (size_t)g.s * P.maxslots + g.wslot, ((unsigned long long)tag << 32) | (unsigned)~tag);
        }
    }
}

// ---- phase O: the blocks of a slice add up W, then out = K~1 W'' / s_i per query tile
template <int RP>
__device__ __noinline__ void worker_o(const Ctx c, const WorkerId id)
{
    constexpr int NW = RP / 8;
    const ResParams &P = c.P;
    const Misc *M = c.M;
    bool ok = true;
    // W''^T = (Diag(w1) Diag(beta)^-1 Gamma2 V)^T of each slice as the B operand: rows = channels (128 bytes = 64 pivots,
    // 16-byte chunks xor row % 8), hi part and lo part.  Every block of the slice adds the partials in slot order.
    for (int j = 0; j < 2; ++j) {
        const int sg = 2 * j;
        if (!seg_active(M, sg)) continue;
        const SegInfo &g = M->seg[sg];
        const unsigned tag = P.tag + (unsigned)P.T + 2u;
        const unsigned long long want = ((unsigned long long)tag << 32) | (unsigned)~tag;
        if (id.wtid < g.wslots) {
            const unsigned long long *f = P.wflag + (size_t)g.s * P.maxslots + id.wtid;
            uint64_t t0 = 0;
            for (uint32_t it = 0;; ++it) {
                if (ld_acquire64(f) == want) break;
                if ((it & 15u) == 15u) {
                    if (c.M->abort) break;
                    const uint64_t now = global_timer_ns();
                    if (t0 == 0) t0 = now;
                    else if (now - t0 > P.wait_ns) { c.M->abort = 1; record_timeout(&P, c.M, c.warp, 110 + j); raise_flag(P, 4 /* LOT_DEV_TIMEOUT */); break; }
                }
                __nanosleep(32);
            }
        }
        named_bar_sync(1, kWorkers);
        if (c.M->abort) ok = false;
        const int tA = 16 * id.w4 + id.rq, tB = tA + 8;
        float acc[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) acc[e] = 0.f;
        if (ok) {
            const float *src0 = P.wpart + (size_t)g.s * P.maxslots * (64 * kDK) + 32 * id.quad + 2 * id.cq;
            for (int sl = 0; sl < g.wslots; ++sl) {
                const float *src = src0 + (size_t)sl * (64 * kDK);
#pragma unroll
                for (int rep = 0; rep < 4; ++rep) {
                    const float2 a = __ldcg(reinterpret_cast<const float2 *>(src + tA * kDK + rep * 8));
                    const float2 b = __ldcg(reinterpret_cast<const float2 *>(src + tB * kDK + rep * 8));
                    acc[rep * 4 + 0] += a.x; acc[rep * 4 + 1] += a.y; acc[rep * 4 + 2] += b.x; acc[rep * 4 + 3] += b.y;
                }
            }
        }
        const float mass = g.kv > 0 ? 1.f / (float)g.kv : 0.f;
        const float cA = tA < P.r ? c.sW[sg * 64 + tA] * mass / __ldg(P.beta + g.h * P.r + tA) : 0.f;
        const float cB = tB < P.r ? c.sW[sg * 64 + tB] * mass / __ldg(P.beta + g.h * P.r + tB) : 0.f;
        uint8_t *wq = c.buf(kSlots + j);
#pragma unroll
        for (int rep = 0; rep < 4; ++rep)
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int ch = 32 * id.quad + rep * 8 + 2 * id.cq + u;
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
    }
    fence_proxy_async_smem();
    named_bar_sync(1, kWorkers);
    trace(c, 0xb00);

    const bool storer = id.w4 == 0 && c.lane == 0;
    for (int qq = id.quad; qq < M->nQ; qq += 2) {
        const int j = qq >> 1, ab = id.quad + 2 * (j % 3);
        int sg, t;
        locate(M, 0, qq, sg, t);
        const SegInfo &g = M->seg[sg];
        if (j >= 3) {
            // the store that last used this buffer (three tiles ago) must have read it
            if (storer) bulk_wait_group_read<2>();
            named_bar_sync(2 + id.quad, 128);
        }
        float2 w2[NW];
#pragma unroll
        for (int e = 0; e < NW; ++e) w2[e] = *reinterpret_cast<const float2 *>(c.sW + sg * 64 + word_col<RP, true>(id, e));
        uint32_t d[4][NW];
        load_rows<RP, true>(c, id, id.lane_addr + qq * (RP / 2), nullptr, d);
        float sr[4];
        row_sums<NW>(d, w2, sr);
        // the tile as A operand: K-major rows of 64 bf16 (only the first RP columns are read)
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
            const int rin = id.w4 * 32 + jj * 8 + id.rq;
            const uint32_t rowaddr = c.bufa(ab) + rin * 128 + id.cq * 4;
#pragma unroll
            for (int e = 0; e < NW; ++e)
                asm volatile("st.shared.b32 [%0], %1;" ::"r"(rowaddr + ((e ^ (rin & 7)) << 4)), "r"(d[jj][e]) : "memory");
        }
        fence_proxy_async_smem();
        warp_arrive(c, bAFull + id.quad);
        trace(c, 0xc00 + qq);
        if (ok) ok = warp_wait(c, bOFull + id.quad, j & 1);
        if (!ok) continue;
        tc_fence_after();
        trace(c, 0xd00 + qq);
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            float o[32];
            tmem_ld_acc<8>(id.lane_addr + ((uint32_t)(half * 16) << 16) + kAccCol, o);
            tmem_wait_ld();
            if (half == 1) {
                tc_fence_before();
                warp_arrive(c, bORead + id.quad);
            }
            const int rinA = id.w4 * 32 + half * 16 + id.rq;
            const float iA = __fdividef(1.f, sr[2 * half]), iB = __fdividef(1.f, sr[2 * half + 1]);
            const uint32_t rowaddr = c.bufa(ab) + rinA * 128 + id.cq * 4;
#pragma unroll
            for (int rep = 0; rep < 8; ++rep) {
                const uint32_t addr = rowaddr + ((rep ^ (rinA & 7)) << 4);
                asm volatile("st.shared.b32 [%0], %1;" ::"r"(addr), "r"(pack_bf16(o[rep * 4 + 0] * iA, o[rep * 4 + 1] * iA)) : "memory");
                asm volatile("st.shared.b32 [%0 + 1024], %1;" ::"r"(addr), "r"(pack_bf16(o[rep * 4 + 2] * iB, o[rep * 4 + 3] * iB)) : "memory");
            }
        }
        fence_proxy_async_smem();
        named_bar_sync(2 + id.quad, 128);
        if (storer) {
            tma_store_3d(&P.tmO, c.bufa(ab), 0, t * kTileRows, g.s);
            bulk_commit_group();
        }
    }
    if (storer) bulk_wait_group0();
}

// ---------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_inval(uint32_t bar)
{
    asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
enum { kPhaseX = 0, kPhaseS = 1, kPhaseW = 2, kPhaseO = 3 };

__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Between two phases (one thread; nobody touches a barrier meanwhile, and every barrier is between two of its phases):
// a barrier that has completed an odd number of phases gets one more full set of arrivals, so that the next phase of
// the kernel finds every barrier as after its initialisation.
__device__ __noinline__ void settle_bars(uint32_t bar0)
{
    for (int i = 0; i < bCount; ++i)
        if (mbar_test_wait(bar0 + 8 * i, 0))
            for (int a = 0; a < bar_count(i); ++a) mbar_arrive(bar0 + 8 * i);
}

template <int RP>
__global__ void __launch_bounds__(kThreads, 1)
resident_forward_kernel(const __grid_constant__ ResParams P)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    Ctx c{P, smem, smem_u32(smem), reinterpret_cast<uint64_t *>(smem + Plan::offBar),
          reinterpret_cast<Misc *>(smem + Plan::offMisc), reinterpret_cast<float *>(smem + Plan::offW),
          reinterpret_cast<float *>(smem + Plan::offPart), reinterpret_cast<float *>(smem + Plan::offMail),
          (int)(threadIdx.x >> 5), (int)(threadIdx.x & 31)};
    if ((c.sbase & 1023u) != 0) {               // the swizzled tiles need a 1024-byte aligned base: refuse, do not corrupt
        if (threadIdx.x == 0) raise_flag(P, 4 /* LOT_DEV_TIMEOUT: the call did not run */);
        return;
    }
    const int warp = c.warp;
    if (threadIdx.x == 0) {
        c.M->abort = 0;
        prefetch_tensormap(&P.tmQ); prefetch_tensormap(&P.tmK); prefetch_tensormap(&P.tmV);
        prefetch_tensormap(&P.tmO); prefetch_tensormap(&P.tmS);
    }
    if (warp == 1) { tmem_alloc(smem_u32(&c.M->tmem), 512); tmem_relinquish(); }
    WorkerId id;
    id.quad = (warp - 4) >> 2; id.w4 = warp & 3; id.rq = c.lane >> 2; id.cq = c.lane & 3;
    id.wtid = (int)threadIdx.x - 128;
    GatherState gs;

    // time stamps of this block's phases (nanoseconds of the global timer), for profiling: [block][8] behind the records
    unsigned long long *stamps = P.status + 2 + (size_t)gridDim.x * 12 + (size_t)blockIdx.x * 8;
    if (threadIdx.x == 0) stamps[0] = global_timer_ns();
    auto phase_sync = [&](int next_phase) {
        tc_fence_before();
        __syncthreads();
        if (threadIdx.x == 0) { settle_bars(c.bar(0)); c.M->phase = next_phase; if (next_phase <= kPhaseO) stamps[next_phase + 1] = global_timer_ns(); }
        __syncthreads();
        tc_fence_after();
    };

    for (int wave = 0;; ++wave) {
        if (threadIdx.x == 0) {
            build_wave(P, c.M, wave);
            if (wave == 0) {
                for (int i = 0; i < bCount; ++i) mbar_init(c.bar(i), bar_count(i));
                fence_barrier_init();
            } else {
                settle_bars(c.bar(0));
            }
            c.M->phase = kPhaseX;
            stamps[1] = global_timer_ns();
        }
        for (int i = threadIdx.x; i < kMaxSeg * 64; i += kThreads) c.sW[i] = (i & 63) < P.r ? 1.f : 0.f;
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        if (!c.M->have_wave) break;
        id.lane_addr = c.M->tmem + ((uint32_t)(id.w4 * 32) << 16);
        const Misc *M = c.M;
        if (threadIdx.x == 0) {
            // bookkeeping of the block that holds a slice's first query tile: empty key sets, potentials of a zero-iteration call
            for (int j = 0; j < M->nseg / 2; ++j) {
                const SegInfo &g = M->seg[2 * j];
                if (g.t0 != 0) continue;
                if (g.kv <= 0) raise_flag(P, 2 /* LOT_DEV_EMPTY */);
                for (int t = 0; t < P.r; ++t) {
                    if (P.T == 0 && P.g1_out != nullptr) P.g1_out[(size_t)g.s * P.r + t] = 0.f;
                    if ((P.T == 0 || g.kv <= 0) && P.g2_out != nullptr) P.g2_out[(size_t)g.s * P.r + t] = 0.f;
                }
            }
        }
#pragma unroll
        for (int i = 0; i < kMaxSeg; ++i) { gs.G[i][0] = 0.f; gs.G[i][1] = 0.f; }
        const int p1 = P.T > 0 ? 1 : 0;

        // ---------------- phase X
        if (warp == 0) { if (c.lane == 0) producer_x(c); }
        else if (warp == 1) mma_x<RP>(c);
        else if (warp == 2) publisher<RP>(c, 0, p1);
        else if (warp == 3) gatherer<RP>(c, gs, 0, p1);
        else worker_x<RP>(c, id);
        phase_sync(kPhaseS);
        // ---------------- phase S
        if (warp == 0 && c.lane == 0) producer_s(c);
        if (P.T > 1) {
            if (warp == 2) publisher<RP>(c, 1, P.T);
            else if (warp == 3) gatherer<RP>(c, gs, 1, P.T);
            else if (warp >= 4) worker_s<RP>(c, id);
        }
        phase_sync(kPhaseW);
        // ---------------- phase W
        if (warp == 0) { if (c.lane == 0) producer_w(c); }
        else if (warp == 1) mma_w(c);
        else if (warp >= 4) worker_w<RP>(c, id);
        phase_sync(kPhaseO);
        // ---------------- phase O
        if (warp == 1) mma_o<RP>(c);
        else if (warp >= 4) worker_o<RP>(c, id);
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        if (threadIdx.x == 0) stamps[5] = global_timer_ns();
    }
    if (warp == 1) tmem_dealloc(c.M->tmem, 512);
}

// ---------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn()
{
    static std::atomic<EncodeTiledFn> fn{nullptr};
    EncodeTiledFn f = fn.load();
    if (f == nullptr) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess) {
            f = reinterpret_cast<EncodeTiledFn>(p);
            fn.store(f);
        }
    }
    return f;
}

// bf16 tensor [outer][rows][64] (64 contiguous), box = 64 x 128 x 1, 128-byte swizzle
static bool make_map(CUtensorMap *m, const void *base, long long outer, int rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {64u, (cuuint64_t)rows, (cuuint64_t)outer};
    cuuint64_t strides[2] = {128u, (cuuint64_t)rows * 128u};
    cuuint32_t box[3] = {64u, 128u, 1u};
    cuuint32_t es[3] = {1u, 1u, 1u};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr int kMaxDevices = 64;
static std::mutex g_dev_mu;
static int g_sms[kMaxDevices];
static bool g_attr[kMaxDevices][3];

static int current_device()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
    return dev;
}

static inline size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }
static inline int pad_r(int r) { return r <= 16 ? 16 : (r <= 32 ? 32 : 64); }

static std::atomic<unsigned> g_tag{0x1000u};
static std::atomic<long long> g_wait_ns{1000000000ll};
static std::atomic<int> g_skip_cta{-1};
static std::atomic<unsigned long long *> g_trace{nullptr};

} // namespace resident

int device_sm_count()
{
    const int dev = resident::current_device();
    if (dev < 0) return 148;
    std::lock_guard<std::mutex> lock(resident::g_dev_mu);
    if (resident::g_sms[dev] == 0) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0) resident::g_sms[dev] = v;
        else { (void)cudaGetLastError(); return 148; }
    }
    return resident::g_sms[dev];
}

void resident_debug(int what, long long value)
{
    if (what == 1) resident::g_skip_cta.store((int)value);
    else if (what == 2) resident::g_wait_ns.store(value > 0 ? value : 1000000000ll);
    else if (what == 3) resident::g_trace.store(reinterpret_cast<unsigned long long *>(value));
}

ResidentGeom resident_geometry(int dtype, int B, int H, int n, int d, int r)
{
    using namespace resident;
    ResidentGeom G{};
    G.ok = false;
    if (dtype != 1 || d != kDK || r < 1 || r > 64 || B < 1 || H < 1 || n < 1) return G;
    const int RP = pad_r(r);
    const int cap = (kAccCol / (RP / 2)) < kBufs ? (kAccCol / (RP / 2)) : kBufs;   // tiles per side of a block and wave
    const int sms = device_sm_count();
    const long long BH = (long long)B * H;
    G.TPS = (n + kTileRows - 1) / kTileRows;
    const long long NT = BH * G.TPS;
    if (NT >= (1ll << 30)) return G;
    G.NT = (int)NT;
    const bool whole_ok = G.TPS <= cap;
    const int ctas_s = NT < sms ? (int)NT : sms;
    const int qmax = (int)((NT + ctas_s - 1) / ctas_s);
    const bool split_ok = qmax <= cap && qmax <= G.TPS;
    if (whole_ok && (2 * BH >= sms || !split_ok)) {
        G.whole = 1;
        G.ctas = BH < sms ? (int)BH : sms;
        G.wave_slices = 2 * G.TPS <= cap ? 2 : 1;
        G.maxslots = 1;
    } else if (split_ok) {
        G.whole = 0;
        G.ctas = ctas_s;
        G.wave_slices = 0;
        G.maxslots = (int)(((long long)G.TPS * G.ctas) / NT) + 2;
    } else {
        return G;
    }
    G.ok = true;
    return G;
}

ResidentLayout resident_layout(int B, int H, int n, int d, int r)
{
    using namespace resident;
    ResidentLayout L{};
    const ResidentGeom G = resident_geometry(1, B, H, n, d, r);
    const size_t BH = (size_t)B * H;
    const int RP = pad_r(r);
    size_t o = 0;
    // status word, redo word at + 8, then one record per warp of a wait that gave up, then eight time stamps per block
    L.status = o; o += up256(16 + (size_t)G.ctas * 12 * 8 + (size_t)G.ctas * 8 * 8);
    L.part = o; o += up256((size_t)2 * 2 * BH * G.maxslots * RP * 8);
    L.wflag = o; o += up256(BH * G.maxslots * 8);
    L.wpart = o; o += up256(BH * G.maxslots * 64 * kDK * 4);
    L.spill = o; o += up256((size_t)G.ctas * 2 * kTileBytes);
    L.total = o;
    return L;
}

template <int RP>
static cudaError_t launch(const resident::ResParams &P, int dev, cudaStream_t st)
{
    using namespace resident;
    auto kern = resident_forward_kernel<RP>;
    constexpr int slot = RP == 16 ? 0 : (RP == 32 ? 1 : 2);
    {
        std::lock_guard<std::mutex> lock(g_dev_mu);
        if (!g_attr[dev][slot]) {
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Plan::total);
            if (e != cudaSuccess) return e;
            g_attr[dev][slot] = true;
        }
    }
    // cooperative launch: the blocks wait for one another, so all of them must be resident at once
    void *args[] = {const_cast<ResParams *>(&P)};
    return cudaLaunchCooperativeKernel(reinterpret_cast<void *>(kern), dim3(P.ctas), dim3(kThreads), args, Plan::total, st);
}

cudaError_t resident_attention(const void *q, const void *k, const void *v, const float *z, const float *beta,
                               const int32_t *key_len, int B, int H, int n, int d, int r, float eps, int iters,
                               void *out, float *g1_out, float *g2_out, void *ws, unsigned *tag_out, cudaStream_t st)
{
    using namespace resident;
    const int dev = current_device();
    if (dev < 0) return cudaErrorInvalidDevice;
    const ResidentGeom G = resident_geometry(1, B, H, n, d, r);
    if (!G.ok) return cudaErrorInvalidValue;
    const ResidentLayout L = resident_layout(B, H, n, d, r);
    char *w = static_cast<char *>(ws);
    const long long BH = (long long)B * H;

    ResParams P;
    memset(&P, 0, sizeof(P));
    if (!make_map(&P.tmQ, q, BH, n) || !make_map(&P.tmK, k, BH, n) || !make_map(&P.tmV, v, BH, n) ||
        !make_map(&P.tmO, out, BH, n) || !make_map(&P.tmS, w + L.spill, (long long)G.ctas * 2, kTileRows))
        return cudaErrorInvalidValue;
    P.z = z; P.beta = beta; P.key_len = key_len;
    P.part = reinterpret_cast<unsigned long long *>(w + L.part);
    P.wpart = reinterpret_cast<float *>(w + L.wpart);
    P.wflag = reinterpret_cast<unsigned long long *>(w + L.wflag);
    P.status = reinterpret_cast<unsigned long long *>(w + L.status);
    P.redo = reinterpret_cast<unsigned *>(w + L.status + 8);
    P.g1_out = g1_out; P.g2_out = g2_out;
    P.B = B; P.H = H; P.n = n; P.r = r; P.T = iters;
    P.TPS = G.TPS; P.NT = G.NT; P.ctas = G.ctas; P.maxslots = G.maxslots; P.whole = G.whole; P.wave_slices = G.wave_slices;
    // tags of one call: tag + 1 .. tag + T + 2; a fresh range per call, so words left by earlier calls never match
    P.tag = g_tag.fetch_add((unsigned)iters + 8u);
    P.scale = (float)(1.4426950408889634 / (double)eps);
    P.eps_ln2 = (float)((double)eps * 0.6931471805599453);
    P.wait_ns = (unsigned long long)g_wait_ns.load();
    P.skip_publish_cta = g_skip_cta.exchange(-1);
    P.trace = g_trace.load();
    *tag_out = P.tag;

    const int RP = pad_r(r);
    if (RP == 16) return launch<16>(P, dev, st);
    if (RP == 32) return launch<32>(P, dev, st);
    return launch<64>(P, dev, st);
}

} // namespace lot
