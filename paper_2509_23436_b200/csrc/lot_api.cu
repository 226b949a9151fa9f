// The C ABI of liblot (see include/lot.h): argument validation, workspace carving and the
// launch sequence.  No arithmetic of the method lives here.
#include "../../include/lot.h"
#include "lot_internal.h"

#include <math.h>
#include <atomic>
#include <mutex>
#include <unordered_map>

namespace {

using namespace lot;

constexpr int kMaxR = 256;
constexpr int kMaxD = 256;
constexpr int kMaxDevices = 64;

inline size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }
inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_dims(int B, int H, int n, int r)
{
    if (B < 0 || H < 1 || n < 0 || r < 1) return LOT_ERR_INVALID_ARG;
    if (r > kMaxR) return LOT_ERR_UNSUPPORTED_SHAPE;
    if ((long long)B * H > 32767) return LOT_ERR_UNSUPPORTED_SHAPE;
    if ((long long)n * r >= (1ll << 31)) return LOT_ERR_UNSUPPORTED_SHAPE;
    return LOT_OK;
}

int check_d(int n, int d)
{
    if (d < 1) return LOT_ERR_INVALID_ARG;
    if (d < 8 || d > kMaxD || (d % 8) != 0) return LOT_ERR_UNSUPPORTED_SHAPE;
    if ((long long)n * d >= (1ll << 31)) return LOT_ERR_UNSUPPORTED_SHAPE;
    return LOT_OK;
}

// Workspace of one Sinkhorn problem set.  The head (status word, potentials, tickets) is one
// contiguous region cleared at the start of every call.
struct SinkLayout {
    size_t status, G, counter, head_end, gnat, part, M, total;
    int chunks, rows_per_chunk;
};

// lt = bytes of the type potentials and row log-sum-exps are held in (4 or 8).
SinkLayout sink_layout(int nprob, int n, int r, size_t base, size_t lt)
{
    SinkLayout L;
    L.chunks = pass_chunks(nprob > 0 ? nprob : 1, n > 0 ? n : 1);
    L.rows_per_chunk = (n + L.chunks - 1) / L.chunks;
    size_t o = base;
    L.status = o; o += 256;
    L.G = o; o += up256((size_t)nprob * r * lt);
    L.counter = o; o += up256((size_t)nprob * 4);
    L.head_end = o;
    L.gnat = o; o += up256((size_t)nprob * r * 4);
    L.part = o; o += up256((size_t)nprob * L.chunks * r * 2 * 4);
    L.M = o; o += up256((size_t)nprob * n * lt);
    L.total = o;
    return L;
}

struct AttnLayout {
    SinkLayout s;
    size_t counter2, cost, wpart, Wp, total;
    int achunks, arows;
};

AttnLayout attn_layout(int B, int H, int n, int d, int r, int dtype)
{
    AttnLayout A;
    const size_t lt = dtype == LOT_F32 ? 8 : 4;
    const int BH = B * H;
    // tickets of the apply stage sit right behind the status word so one memset clears all
    size_t o = 0;
    int tiles = ((r + 63) / 64) * ((d + 63) / 64) * BH;
    A.counter2 = 256;
    o = 256 + up256((size_t)tiles * 4);
    A.s = sink_layout(2 * BH, n, r, o, lt);
    A.s.status = 0; // shared status word at the very start
    o = A.s.total;
    A.cost = o; o += up256((size_t)2 * BH * n * r * lt);
    A.achunks = apply_chunks(BH > 0 ? BH : 1, n > 0 ? n : 1, r, d);
    A.arows = (n + A.achunks - 1) / A.achunks;
    A.wpart = o; o += up256((size_t)BH * A.achunks * r * d * 4);
    A.Wp = o; o += up256((size_t)BH * r * d * 4);
    A.total = o;
    return A;
}

// Workspace of lot_attention_fwd_var: the two sides have their own token counts, so each gets a Sinkhorn block.
struct VarLayout {
    SinkLayout s1, s2;
    size_t counter2, cost1, cost2, wa, wb, scores, wpart, Wp, total;
    int achunks, arows;
};

VarLayout var_layout(int B, int H, int nq, int nk, int d, int r, int dtype)
{
    VarLayout V;
    const size_t lt = dtype == LOT_F32 ? 8 : 4;
    const int BH = B * H;
    const int tiles = ((r + 63) / 64) * ((d + 63) / 64) * BH;
    V.counter2 = 256;
    size_t o = 256 + up256((size_t)tiles * 4);
    // one cleared head for both sides: status word at 0, then tickets and potentials
    V.s1 = sink_layout(BH, nq, r, o, lt);
    V.s2 = sink_layout(BH, nk, r, V.s1.total, lt);
    o = V.s2.total;
    V.cost1 = o; o += up256((size_t)BH * nq * r * lt);
    V.cost2 = o; o += up256((size_t)BH * nk * r * lt);
    V.wa = o; o += up256((size_t)BH * nq * 4);
    V.wb = o; o += up256((size_t)BH * nk * 4);
    V.scores = o; o += up256((size_t)BH * nk * 4);
    V.achunks = apply_chunks(BH > 0 ? BH : 1, nk > 0 ? nk : 1, r, d);
    V.arows = (nk + V.achunks - 1) / V.achunks;
    V.wpart = o; o += up256((size_t)BH * V.achunks * r * d * 4);
    V.Wp = o; o += up256((size_t)BH * r * d * 4);
    V.total = o;
    return V;
}

// Workspace of lot_attention_bwd: the general path's blocks plus the kept potentials of every iteration, the
// gradient with respect to the similarities and the small reduction buffers.
struct BwdLayout {
    size_t counter, counter2, hist, gamma, dbeta_acc, head_end, part, M, cost, dC, wpart, Wp, Xw, dWm, dbeta_direct, zt,
        dzpart, total;
    int chunks, rows_per_chunk, achunks, arows, dzchunks;
};

BwdLayout bwd_layout(int B, int H, int n, int d, int r, int dtype, int iters)
{
    BwdLayout L;
    const size_t lt = dtype == LOT_F32 ? 8 : 4;
    const int BH = B * H, np = 2 * BH;
    const int tiles = ((r + 63) / 64) * ((d + 63) / 64) * BH;
    L.chunks = pass_chunks(np > 0 ? np : 1, n > 0 ? n : 1);
    L.rows_per_chunk = (n + L.chunks - 1) / L.chunks;
    L.achunks = apply_chunks(BH > 0 ? BH : 1, n > 0 ? n : 1, r, d);
    L.arows = (n + L.achunks - 1) / L.achunks;
    L.dzchunks = bwd_dz_chunks(BH > 0 ? BH : 1, n > 0 ? n : 1, r, d);
    size_t o = 256;                                   // status word at 0
    L.counter = o; o += up256((size_t)np * 4);
    L.counter2 = o; o += up256((size_t)tiles * 4);
    L.hist = o; o += up256((size_t)(iters + 1) * np * r * lt);
    L.gamma = o; o += up256((size_t)np * r * lt);
    L.dbeta_acc = o; o += up256((size_t)np * r * lt);
    L.head_end = o;
    L.part = o; o += up256((size_t)np * L.chunks * r * 8);
    L.M = o; o += up256((size_t)np * n * lt);
    L.cost = o; o += up256((size_t)np * n * r * lt);
    L.dC = o; o += up256((size_t)np * n * r * lt);
    L.wpart = o; o += up256((size_t)BH * L.achunks * r * d * 4);
    L.Wp = o; o += up256((size_t)BH * r * d * 4);
    L.Xw = o; o += up256((size_t)BH * r * d * 4);
    L.dWm = o; o += up256((size_t)BH * r * d * 4);
    L.dbeta_direct = o; o += up256((size_t)BH * r * 4);
    L.zt = o; o += up256((size_t)H * r * d * 4);
    L.dzpart = o; o += up256((size_t)np * L.dzchunks * r * d * lt);
    L.total = o;
    return L;
}

template <typename T> inline T *at(void *ws, size_t off) { return reinterpret_cast<T *>(static_cast<char *>(ws) + off); }

struct Managed {
    void *ptr = nullptr;
    size_t bytes = 0;
};
Managed g_managed[kMaxDevices];
std::mutex g_managed_mu;

// Which path last ran on a workspace, and the tag of that call: the resident path keeps its status word tagged
// instead of clearing it, so reading it needs the tag (lot_device_status).
struct WsRecord {
    int path;
    unsigned tag;
    size_t fused_off;
};
std::unordered_map<const void *, WsRecord> g_ws_records;
std::mutex g_ws_mu;
void remember_ws(const void *ws, int path, unsigned tag, size_t fused_off)
{
    std::lock_guard<std::mutex> lock(g_ws_mu);
    if (g_ws_records.size() > 65536) g_ws_records.clear();
    g_ws_records[ws] = WsRecord{path, tag, fused_off};
}

enum { kPathGeneral = 0, kPathStreamed = 1, kPathResident = 2, kPathSlice = 3 };
std::atomic<int> g_force_path{-1};      // test hook: 0 picks the general path, 1 or 2 that tensor-core path wherever it can run
int choose_path(int dtype, int B, int H, int n, int d, int r)
{
    if (!fused_supported(dtype, d, r)) return kPathGeneral;
    const bool res_ok = B >= 1 && n >= 1 && resident_geometry(dtype, B, H, n, d, r).ok;
    const bool slice_ok = B >= 1 && slice_supported(dtype, n, d, r);
    const int force = g_force_path.load();
    if (force == kPathGeneral) return kPathGeneral;
    if (force == kPathStreamed) return kPathStreamed;
    if (force == kPathResident) return res_ok ? kPathResident : kPathStreamed;
    // short sequences: one thread block per slice, everything on chip, exact float32 logits
    if (slice_ok) return kPathSlice;
    // Measured on B200 (see the design notes): the resident kernel wins where the streamed one has no stored-kernel
    // passes (r <= 32, every pass recomputes logits and exponentials) and every thread block holds its whole share at
    // once (whole slices, one wave); elsewhere the streamed kernel is as fast or faster.
    if (res_ok && r <= 32) {
        const ResidentGeom G = resident_geometry(dtype, B, H, n, d, r);
        if (G.whole && (long long)B * H <= (long long)G.ctas * G.wave_slices) return kPathResident;
    }
    return kPathStreamed;
}

// Scratch of lot_sinkhorn_static: part of the library image, present on every device that loads
// it.  In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[LOT_STATIC_SCRATCH_BYTES];
void *g_static_ptr[kMaxDevices];   // device address of the array, per device (looked up once)
std::mutex g_static_mu;

} // namespace

extern "C" {

#ifdef LOT_DEBUG
int lot_version(void) { return 100 + 100000; }      // the bounds-check build answers 100100
#else
int lot_version(void) { return 100; }
#endif

const char *lot_status_string(int status)
{
    switch (status) {
    case LOT_OK: return "LOT_OK";
    case LOT_ERR_INVALID_ARG: return "LOT_ERR_INVALID_ARG: null or misaligned pointer, eps <= 0, iters < 0 or unknown dtype";
    case LOT_ERR_UNSUPPORTED_SHAPE: return "LOT_ERR_UNSUPPORTED_SHAPE: need 1 <= r <= 256, 8 <= d <= 256, d % 8 == 0, B*H <= 32767, n*r and n*d < 2^31";
    case LOT_ERR_WORKSPACE: return "LOT_ERR_WORKSPACE: workspace null, not 256-byte aligned or too small (lot_sinkhorn_static: the problem needs more than LOT_STATIC_SCRATCH_BYTES)";
    case LOT_ERR_CUDA: return "LOT_ERR_CUDA: a CUDA runtime call or kernel launch failed";
    default: return "unknown lot status";
    }
}

int lot_cost(const void *x, const float *z, int dtype, int B, int H, int n, int d, int r,
             float *cost, lot_stream_t stream)
{
    if (dtype != LOT_F32 && dtype != LOT_BF16) return LOT_ERR_INVALID_ARG;
    int st = check_dims(B, H, n, r);
    if (st != LOT_OK) return st;
    st = check_d(n, d);
    if (st != LOT_OK) return st;
    if (B == 0 || n == 0) return LOT_OK;
    if (!x || !z || !cost) return LOT_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(z) || !aligned16(cost)) return LOT_ERR_INVALID_ARG;
    cudaError_t e = launch_cost(x, z, dtype, B * H, H, n, d, r, cost, false, (cudaStream_t)stream);
    return e == cudaSuccess ? LOT_OK : LOT_ERR_CUDA;
}

size_t lot_sinkhorn_workspace_bytes(int B, int H, int n, int r)
{
    if (check_dims(B, H, n, r) != LOT_OK) return 0;
    return sink_layout(B * H, n, r, 0, 8).total;
}

int lot_sinkhorn(const float *cost, const float *beta, const int32_t *len,
                 int B, int H, int n, int r, float eps, int iters,
                 float *g, float *f, float *plan,
                 void *ws, size_t ws_bytes, lot_stream_t stream)
{
    int st = check_dims(B, H, n, r);
    if (st != LOT_OK) return st;
    if (!(eps > 0.f) || !isfinite(eps) || iters < 0) return LOT_ERR_INVALID_ARG;
    if (B == 0 || n == 0) return LOT_OK;
    if (!cost || !beta || !g) return LOT_ERR_INVALID_ARG;
    if (!aligned16(cost) || !aligned16(beta) || !aligned16(g) || !aligned16(f) || !aligned16(plan) ||
        (len && (reinterpret_cast<uintptr_t>(len) & 3u)))
        return LOT_ERR_INVALID_ARG;
    const int nprob = B * H;
    SinkLayout L = sink_layout(nprob, n, r, 0, 8);
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u) || ws_bytes < L.total) return LOT_ERR_WORKSPACE;
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemsetAsync(ws, 0, L.head_end, s) != cudaSuccess) return LOT_ERR_CUDA;

    PassArgs a{};
    a.cost = cost; a.beta = beta; a.len = len; a.len_from = 0;
    a.G = at<void>(ws, L.G); a.part = at<float>(ws, L.part); a.counter = at<unsigned>(ws, L.counter);
    a.M = at<void>(ws, L.M); a.g_out = g; a.f_out = f; a.plan_out = plan;
    a.status = at<int>(ws, L.status);
    a.nprob = nprob; a.B = B; a.H = H; a.n = n; a.r = r;
    a.chunks = L.chunks; a.rows_per_chunk = L.rows_per_chunk;
    a.mode = kModeCostF32Wide;
    a.scale_d = 1.4426950408889634 / (double)eps;
    a.eps_ln2 = (float)((double)eps * 0.6931471805599453);
    for (int it = 0; it < iters; ++it)
        if (launch_sinkhorn_pass(a, false, s) != cudaSuccess) return LOT_ERR_CUDA;
    if (launch_sinkhorn_pass(a, true, s) != cudaSuccess) return LOT_ERR_CUDA;
    return LOT_OK;
}

int lot_sinkhorn_static(const float *cost, const float *beta, const int32_t *len,
                        int B, int H, int n, int r, float eps, int iters,
                        float *g, float *f, float *plan, int32_t *status_out,
                        lot_stream_t stream)
{
    // every argument check comes first, in lot_sinkhorn's order, so that a bad call is refused before any device work
    int st = check_dims(B, H, n, r);
    if (st != LOT_OK) return st;
    if (!(eps > 0.f) || !isfinite(eps) || iters < 0) return LOT_ERR_INVALID_ARG;
    if (status_out && (reinterpret_cast<uintptr_t>(status_out) & 3u)) return LOT_ERR_INVALID_ARG;
    if (B == 0 || n == 0) return LOT_OK;
    if (!cost || !beta || !g) return LOT_ERR_INVALID_ARG;
    if (!aligned16(cost) || !aligned16(beta) || !aligned16(g) || !aligned16(f) || !aligned16(plan) ||
        (len && (reinterpret_cast<uintptr_t>(len) & 3u)))
        return LOT_ERR_INVALID_ARG;
    if (sink_layout(B * H, n, r, 0, 8).total > (size_t)LOT_STATIC_SCRATCH_BYTES) return LOT_ERR_WORKSPACE;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LOT_ERR_CUDA;
    void *ws = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_static_mu);
        if (g_static_ptr[dev] == nullptr) {
            void *p = nullptr;
            if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) {
                (void)cudaGetLastError();
                return LOT_ERR_CUDA;
            }
            g_static_ptr[dev] = p;
        }
        ws = g_static_ptr[dev];
    }
    st = lot_sinkhorn(cost, beta, len, B, H, n, r, eps, iters, g, f, plan, ws, LOT_STATIC_SCRATCH_BYTES, stream);
    if (st != LOT_OK) return st;
    if (status_out && cudaMemcpyAsync(status_out, ws, sizeof(int32_t), cudaMemcpyDeviceToDevice,
                                      (cudaStream_t)stream) != cudaSuccess)
        return LOT_ERR_CUDA;
    return LOT_OK;
}

size_t lot_workspace_bytes(int B, int H, int n, int d, int r, int dtype)
{
    if (dtype != LOT_F32 && dtype != LOT_BF16) return 0;
    if (check_dims(B, H, n, r) != LOT_OK || check_d(n, d) != LOT_OK) return 0;
    const int path = choose_path(dtype, B, H, n, d, r);
    if (path == kPathResident) return up256(resident_layout(B, H, n, d, r).total) + fused_layout(B, H, n, d, r).total;
    if (path == kPathStreamed) return fused_layout(B, H, n, d, r).total;
    if (path == kPathSlice) return 256;                              // the status word
    return attn_layout(B, H, n, d, r, dtype).total;
}

int lot_path(int dtype, int B, int H, int n, int d, int r, int iters)
{
    (void)iters;
    if (dtype != LOT_F32 && dtype != LOT_BF16) return 0;
    if (check_dims(B, H, n, r) != LOT_OK || check_d(n, d) != LOT_OK) return 0;
    return choose_path(dtype, B, H, n, d, r);
}

int lot_launch_count(int dtype, int B, int H, int n, int d, int r, int iters)
{
    if (iters < 0) return 0;
    const int path = lot_path(dtype, B, H, n, d, r, iters);
    if (path == kPathResident) return 1 + 2;                        // the two streamed kernels return at once unless asked to redo
    if (path == kPathStreamed) return fused_launches(B, H, n, r, iters);
    if (path == kPathSlice) return 1;
    return 2 + iters + 1 + 2;
}

int lot_debug_hook(int what, long long value)
{
    if (what < 1 || what > 4) return LOT_ERR_INVALID_ARG;
    if (what == 4) g_force_path.store((int)value);
    else resident_debug(what, value);
    return LOT_OK;
}

int lot_attention_fwd_ex(const void *q, const void *k, const void *v,
                         const float *z, const float *beta, const int32_t *key_len,
                         int dtype, int B, int H, int n, int d, int r, float eps, int iters,
                         void *out, float *g1_out, float *g2_out,
                         void *ws, size_t ws_bytes, lot_stream_t stream)
{
    if (dtype != LOT_F32 && dtype != LOT_BF16) return LOT_ERR_INVALID_ARG;
    int st = check_dims(B, H, n, r);
    if (st != LOT_OK) return st;
    st = check_d(n, d);
    if (st != LOT_OK) return st;
    if (!(eps > 0.f) || !isfinite(eps) || iters < 0) return LOT_ERR_INVALID_ARG;
    if (B == 0 || n == 0) return LOT_OK;
    if (!q || !k || !v || !z || !beta || !out) return LOT_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(z) || !aligned16(beta) ||
        !aligned16(out) || !aligned16(g1_out) || !aligned16(g2_out) ||
        (key_len && (reinterpret_cast<uintptr_t>(key_len) & 3u)))
        return LOT_ERR_INVALID_ARG;
    const int path = choose_path(dtype, B, H, n, d, r);
    if (path == kPathSlice) {
        if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u) || ws_bytes < 256) return LOT_ERR_WORKSPACE;
        remember_ws(ws, kPathSlice, 0, 0);
        cudaError_t e = slice_attention(q, k, v, z, beta, key_len, B, H, n, r, eps, iters, out, g1_out, g2_out,
                                        at<int>(ws, 0), (cudaStream_t)stream);
        return e == cudaSuccess ? LOT_OK : LOT_ERR_CUDA;
    }
    if (path != kPathGeneral) {
        const size_t res_bytes = path == kPathResident ? up256(resident_layout(B, H, n, d, r).total) : 0;
        const size_t need = res_bytes + fused_layout(B, H, n, d, r).total;
        if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u) || ws_bytes < need) return LOT_ERR_WORKSPACE;
        cudaStream_t s = (cudaStream_t)stream;
        unsigned tag = 0;
        const unsigned *redo = nullptr;
        if (path == kPathResident) {
            if (resident_attention(q, k, v, z, beta, key_len, B, H, n, d, r, eps, iters, out, g1_out, g2_out, ws, &tag, s) !=
                cudaSuccess) {
                (void)cudaGetLastError();
                return LOT_ERR_CUDA;
            }
            redo = at<unsigned>(ws, resident_layout(B, H, n, d, r).status + 8);
        }
        remember_ws(ws, path, tag, res_bytes);
        // behind a resident launch the streamed kernels run only if that launch asked for it (a problem outside the
        // range of the stored bf16 kernel); alone they are the path
        cudaError_t e = fused_attention(q, k, v, z, beta, key_len, B, H, n, d, r, eps, iters, out, g1_out, g2_out,
                                        at<char>(ws, res_bytes), redo, tag, s);
        return e == cudaSuccess ? LOT_OK : LOT_ERR_CUDA;
    }
    remember_ws(ws, kPathGeneral, 0, 0);
    AttnLayout A = attn_layout(B, H, n, d, r, dtype);
    const bool wide = dtype == LOT_F32;
    const size_t lt = wide ? 8 : 4;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u) || ws_bytes < A.total) return LOT_ERR_WORKSPACE;
    cudaStream_t s = (cudaStream_t)stream;
    const int BH = B * H;
    if (cudaMemsetAsync(ws, 0, A.s.head_end, s) != cudaSuccess) return LOT_ERR_CUDA;

    char *cost1 = at<char>(ws, A.cost);
    char *cost2 = cost1 + (size_t)BH * n * r * lt;
    if (launch_cost(q, z, dtype, BH, H, n, d, r, cost1, wide, s) != cudaSuccess) return LOT_ERR_CUDA;
    if (launch_cost(k, z, dtype, BH, H, n, d, r, cost2, wide, s) != cudaSuccess) return LOT_ERR_CUDA;

    PassArgs a{};
    a.cost = cost1; a.beta = beta; a.len = key_len; a.len_from = BH;
    a.G = at<void>(ws, A.s.G); a.part = at<float>(ws, A.s.part); a.counter = at<unsigned>(ws, A.s.counter);
    a.M = at<void>(ws, A.s.M); a.g_out = at<float>(ws, A.s.gnat); a.f_out = nullptr; a.plan_out = nullptr;
    a.status = at<int>(ws, 0);
    a.nprob = 2 * BH; a.B = B; a.H = H; a.n = n; a.r = r;
    a.chunks = A.s.chunks; a.rows_per_chunk = A.s.rows_per_chunk;
    a.mode = wide ? kModeWide : kModeF32;
    a.scale_d = 1.4426950408889634 / (double)eps;
    a.eps_ln2 = (float)((double)eps * 0.6931471805599453);
    for (int it = 0; it < iters; ++it)
        if (launch_sinkhorn_pass(a, false, s) != cudaSuccess) return LOT_ERR_CUDA;
    if (launch_sinkhorn_pass(a, true, s) != cudaSuccess) return LOT_ERR_CUDA;

    ApplyArgs ap{};
    ap.cost1 = cost1; ap.cost2 = cost2;
    ap.G1 = a.G; ap.G2 = static_cast<char *>(a.G) + (size_t)BH * r * lt;
    ap.M1 = a.M; ap.M2 = static_cast<char *>(a.M) + (size_t)BH * n * lt;
    ap.beta = beta; ap.key_len = key_len; ap.v = v; ap.out = out;
    ap.wpart = at<float>(ws, A.wpart); ap.Wp = at<float>(ws, A.Wp); ap.counter = at<unsigned>(ws, A.counter2);
    ap.B = B; ap.H = H; ap.n = n; ap.nk = n; ap.d = d; ap.r = r;
    ap.chunks = A.achunks; ap.rows_per_chunk = A.arows; ap.scale_d = a.scale_d;
    if (launch_apply_w(ap, dtype, s) != cudaSuccess) return LOT_ERR_CUDA;
    if (launch_apply_out(ap, dtype, s) != cudaSuccess) return LOT_ERR_CUDA;

    const size_t gb = (size_t)BH * r * sizeof(float);
    if (g1_out && cudaMemcpyAsync(g1_out, a.g_out, gb, cudaMemcpyDeviceToDevice, s) != cudaSuccess) return LOT_ERR_CUDA;
    if (g2_out && cudaMemcpyAsync(g2_out, a.g_out + (size_t)BH * r, gb, cudaMemcpyDeviceToDevice, s) != cudaSuccess)
        return LOT_ERR_CUDA;
    return LOT_OK;
}

size_t lot_var_workspace_bytes(int B, int H, int nq, int nk, int d, int r, int dtype)
{
    if (dtype != LOT_F32 && dtype != LOT_BF16) return 0;
    if (check_dims(B, H, nq, r) != LOT_OK || check_dims(B, H, nk, r) != LOT_OK) return 0;
    if (check_d(nq, d) != LOT_OK || check_d(nk, d) != LOT_OK) return 0;
    return var_layout(B, H, nq, nk, d, r, dtype).total;
}

int lot_attention_fwd_var(const void *q, const void *k, const void *v, const float *z, const float *beta,
                          const float *a, const float *b, const int32_t *key_len,
                          const float *g1_in, const float *g2_in, int cls, float cls_tau,
                          int dtype, int B, int H, int nq, int nk, int d, int r, float eps, int iters,
                          void *out, float *g1_out, float *g2_out,
                          void *ws, size_t ws_bytes, lot_stream_t stream)
{
    if (dtype != LOT_F32 && dtype != LOT_BF16) return LOT_ERR_INVALID_ARG;
    int st = check_dims(B, H, nq, r);
    if (st == LOT_OK) st = check_dims(B, H, nk, r);
    if (st == LOT_OK) st = check_d(nq, d);
    if (st == LOT_OK) st = check_d(nk, d);
    if (st != LOT_OK) return st;
    if (!(eps > 0.f) || !isfinite(eps) || iters < 0) return LOT_ERR_INVALID_ARG;
    if (cls != 0 && cls != 1) return LOT_ERR_INVALID_ARG;
    if (cls && (!(cls_tau > 0.f) || !isfinite(cls_tau) || a != nullptr || b != nullptr)) return LOT_ERR_INVALID_ARG;
    if (B == 0 || nq == 0) return LOT_OK;
    if (nk == 0) return LOT_ERR_INVALID_ARG;
    if (!q || !k || !v || !z || !beta || !out) return LOT_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(z) || !aligned16(beta) || !aligned16(out) ||
        !aligned16(g1_out) || !aligned16(g2_out) || !aligned16(g1_in) || !aligned16(g2_in) || !aligned16(a) ||
        !aligned16(b) || (key_len && (reinterpret_cast<uintptr_t>(key_len) & 3u)))
        return LOT_ERR_INVALID_ARG;
    VarLayout V = var_layout(B, H, nq, nk, d, r, dtype);
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u) || ws_bytes < V.total) return LOT_ERR_WORKSPACE;
    const bool wide = dtype == LOT_F32;
    const size_t lt = wide ? 8 : 4;
    cudaStream_t s = (cudaStream_t)stream;
    const int BH = B * H;
    remember_ws(ws, kPathGeneral, 0, 0);
    // the head (status word, tickets) starts at zero; the potentials start at the given ones
    if (cudaMemsetAsync(ws, 0, V.s1.head_end, s) != cudaSuccess) return LOT_ERR_CUDA;
    if (cudaMemsetAsync(at<char>(ws, V.s2.status), 0, V.s2.head_end - V.s2.status, s) != cudaSuccess) return LOT_ERR_CUDA;
    const double scale = 1.4426950408889634 / (double)eps;
    if (g1_in && launch_g_init(g1_in, at<void>(ws, V.s1.G), (size_t)BH * r, scale, wide, s) != cudaSuccess) return LOT_ERR_CUDA;
    if (g2_in && launch_g_init(g2_in, at<void>(ws, V.s2.G), (size_t)BH * r, scale, wide, s) != cudaSuccess) return LOT_ERR_CUDA;
    const float *wa = a, *wb = b;
    if (cls) {
        if (launch_cls_marginals(at<float>(ws, V.wa), at<float>(ws, V.wb), key_len, B, H, nq, nk, at<int>(ws, 0), s) != cudaSuccess)
            return LOT_ERR_CUDA;
        wa = at<float>(ws, V.wa);
        wb = at<float>(ws, V.wb);
    }

    char *cost1 = at<char>(ws, V.cost1), *cost2 = at<char>(ws, V.cost2);
    if (launch_cost(q, z, dtype, BH, H, nq, d, r, cost1, wide, s) != cudaSuccess) return LOT_ERR_CUDA;
    if (launch_cost(k, z, dtype, BH, H, nk, d, r, cost2, wide, s) != cudaSuccess) return LOT_ERR_CUDA;

    PassArgs pa[2] = {};
    for (int side = 0; side < 2; ++side) {
        const SinkLayout &L = side ? V.s2 : V.s1;
        PassArgs &x = pa[side];
        x = PassArgs{};
        x.cost = side ? cost2 : cost1; x.beta = beta;
        // a key length is a mask on the key side only; with explicit weights it only bounds the rows that are read
        x.len = side ? key_len : nullptr; x.len_from = 0;
        x.mass = side ? wb : wa;
        x.G = at<void>(ws, L.G); x.part = at<float>(ws, L.part); x.counter = at<unsigned>(ws, L.counter);
        x.M = at<void>(ws, L.M); x.g_out = side ? g2_out : g1_out;
        x.status = at<int>(ws, 0);
        x.nprob = BH; x.B = B; x.H = H; x.n = side ? nk : nq; x.r = r;
        x.chunks = L.chunks; x.rows_per_chunk = L.rows_per_chunk;
        x.mode = wide ? kModeWide : kModeF32;
        x.scale_d = scale;
        x.eps_ln2 = (float)((double)eps * 0.6931471805599453);
        for (int it = 0; it < iters; ++it)
            if (launch_sinkhorn_pass(x, false, s) != cudaSuccess) return LOT_ERR_CUDA;
        if (launch_sinkhorn_pass(x, true, s) != cudaSuccess) return LOT_ERR_CUDA;
    }

    ApplyArgs ap{};
    ap.cost1 = cost1; ap.cost2 = cost2;
    ap.G1 = pa[0].G; ap.G2 = pa[1].G; ap.M1 = pa[0].M; ap.M2 = pa[1].M;
    ap.beta = beta; ap.key_len = key_len; ap.mass2 = wb; ap.v = v; ap.out = out;
    ap.wpart = at<float>(ws, V.wpart); ap.Wp = at<float>(ws, V.Wp); ap.counter = at<unsigned>(ws, V.counter2);
    ap.B = B; ap.H = H; ap.n = nq; ap.nk = nk; ap.d = d; ap.r = r;
    ap.chunks = V.achunks; ap.rows_per_chunk = V.arows; ap.scale_d = scale;
    if (launch_apply_w(ap, dtype, s) != cudaSuccess) return LOT_ERR_CUDA;
    if (launch_apply_out(ap, dtype, s) != cudaSuccess) return LOT_ERR_CUDA;
    if (cls && launch_cls_row(q, k, v, key_len, dtype, B, H, nq, nk, d, cls_tau, at<float>(ws, V.scores), out, s) != cudaSuccess)
        return LOT_ERR_CUDA;
    (void)lt;
    return LOT_OK;
}

int lot_attention_fwd(const float *q, const float *k, const float *v,
                      const float *z, const float *beta,
                      int B, int H, int n, int d, int r, float eps, int iters,
                      float *out, lot_stream_t stream)
{
    int st = check_dims(B, H, n, r);
    if (st != LOT_OK) return st;
    st = check_d(n, d);
    if (st != LOT_OK) return st;
    if (B == 0 || n == 0) return LOT_OK;
    const size_t need = attn_layout(B, H, n, d, r, LOT_F32).total;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LOT_ERR_CUDA;
    void *ws = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_managed_mu);
        Managed &m = g_managed[dev];
        if (m.bytes < need) {
            if (cudaDeviceSynchronize() != cudaSuccess) return LOT_ERR_CUDA;
            if (m.ptr) cudaFree(m.ptr);
            m.ptr = nullptr; m.bytes = 0;
            if (cudaMalloc(&m.ptr, need) != cudaSuccess) { (void)cudaGetLastError(); m.ptr = nullptr; return LOT_ERR_CUDA; }
            m.bytes = need;
        }
        ws = m.ptr;
    }
    return lot_attention_fwd_ex(q, k, v, z, beta, nullptr, LOT_F32, B, H, n, d, r, eps, iters,
                                out, nullptr, nullptr, ws, need, stream);
}

int lot_device_status(const void *ws, lot_stream_t stream, int *status)
{
    if (!status) return LOT_ERR_INVALID_ARG;
    if (!ws) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LOT_ERR_CUDA;
        std::lock_guard<std::mutex> lock(g_managed_mu);
        ws = g_managed[dev].ptr;
        if (!ws) { *status = 0; return LOT_OK; }
    }
    cudaStream_t s = (cudaStream_t)stream;
    WsRecord rec{kPathGeneral, 0, 0};
    {
        std::lock_guard<std::mutex> lock(g_ws_mu);
        auto it = g_ws_records.find(ws);
        if (it != g_ws_records.end()) rec = it->second;
    }
    if (rec.path != kPathResident) {
        if (cudaMemcpyAsync(status, ws, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return LOT_ERR_CUDA;
        if (cudaStreamSynchronize(s) != cudaSuccess) return LOT_ERR_CUDA;
        if (kernels_debug_flag() | backward_debug_flag()) *status |= LOT_DEV_BOUNDS;      // bounds-check build only
        return LOT_OK;
    }
    // resident path: {flags | tag << 32, redo word} at the start, the streamed kernels' word behind the resident block
    unsigned head[4] = {0, 0, 0, 0};
    int streamed = 0;
    if (cudaMemcpyAsync(head, ws, sizeof(head), cudaMemcpyDeviceToHost, s) != cudaSuccess) return LOT_ERR_CUDA;
    if (cudaMemcpyAsync(&streamed, static_cast<const char *>(ws) + rec.fused_off, sizeof(int), cudaMemcpyDeviceToHost, s) !=
        cudaSuccess)
        return LOT_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return LOT_ERR_CUDA;
    const int mine = head[1] == rec.tag ? (int)head[0] : 0;
    // a call that was recomputed reports the recomputation's flags (and a timeout of the first attempt, if any)
    *status = head[2] == rec.tag ? (LOT_DEV_RECOMPUTED | streamed | (mine & LOT_DEV_TIMEOUT)) : (mine | streamed);
    return LOT_OK;
}

size_t lot_bwd_workspace_bytes(int B, int H, int n, int d, int r, int dtype, int iters)
{
    if (dtype != LOT_F32 && dtype != LOT_BF16) return 0;
    if (check_dims(B, H, n, r) != LOT_OK || check_d(n, d) != LOT_OK || iters < 0) return 0;
    return bwd_layout(B, H, n, d, r, dtype, iters).total;
}

int lot_attention_bwd(const void *q, const void *k, const void *v, const float *z, const float *beta,
                      const int32_t *key_len, const void *dout,
                      int dtype, int B, int H, int n, int d, int r, float eps, int iters,
                      void *dq, void *dk, void *dv, float *dz, float *dbeta,
                      void *ws, size_t ws_bytes, lot_stream_t stream)
{
    if (dtype != LOT_F32 && dtype != LOT_BF16) return LOT_ERR_INVALID_ARG;
    int st = check_dims(B, H, n, r);
    if (st != LOT_OK) return st;
    st = check_d(n, d);
    if (st != LOT_OK) return st;
    if (!(eps > 0.f) || !isfinite(eps) || iters < 0) return LOT_ERR_INVALID_ARG;
    if (!z || !beta || !dz || !dbeta) return LOT_ERR_INVALID_ARG;
    if (!aligned16(z) || !aligned16(beta) || !aligned16(dz) || !aligned16(dbeta)) return LOT_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    if (B == 0 || n == 0) {
        // no tokens: the pivots receive no gradient
        if (cudaMemsetAsync(dz, 0, (size_t)H * r * d * sizeof(float), s) != cudaSuccess) return LOT_ERR_CUDA;
        if (cudaMemsetAsync(dbeta, 0, (size_t)H * r * sizeof(float), s) != cudaSuccess) return LOT_ERR_CUDA;
        return LOT_OK;
    }
    if (!q || !k || !v || !dout || !dq || !dk || !dv) return LOT_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(dout) || !aligned16(dq) || !aligned16(dk) ||
        !aligned16(dv) || (key_len && (reinterpret_cast<uintptr_t>(key_len) & 3u)))
        return LOT_ERR_INVALID_ARG;
    const BwdLayout L = bwd_layout(B, H, n, d, r, dtype, iters);
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u) || ws_bytes < L.total) return LOT_ERR_WORKSPACE;
    remember_ws(ws, kPathGeneral, 0, 0);
    const bool wide = dtype == LOT_F32;
    const size_t lt = wide ? 8 : 4;
    const int BH = B * H, np = 2 * BH;
    const int ttype = dtype == LOT_F32 ? 0 : 1;        // tensor element type for the products
    const int ltype = wide ? 2 : 0;                    // type of the similarity-sized buffers
    if (cudaMemsetAsync(ws, 0, L.head_end, s) != cudaSuccess) return LOT_ERR_CUDA;

    // ---- the forward, keeping the potentials of every iteration
    char *cost1 = at<char>(ws, L.cost);
    char *cost2 = cost1 + (size_t)BH * n * r * lt;
    if (launch_cost(q, z, dtype, BH, H, n, d, r, cost1, wide, s) != cudaSuccess) return LOT_ERR_CUDA;
    if (launch_cost(k, z, dtype, BH, H, n, d, r, cost2, wide, s) != cudaSuccess) return LOT_ERR_CUDA;
    char *hist = at<char>(ws, L.hist);
    const size_t hstep = (size_t)np * r * lt;
    PassArgs a{};
    a.cost = cost1; a.beta = beta; a.len = key_len; a.len_from = BH;
    a.part = at<float>(ws, L.part); a.counter = at<unsigned>(ws, L.counter);
    a.M = at<void>(ws, L.M); a.status = at<int>(ws, 0);
    a.nprob = np; a.B = B; a.H = H; a.n = n; a.r = r;
    a.chunks = L.chunks; a.rows_per_chunk = L.rows_per_chunk;
    a.mode = wide ? kModeWide : kModeF32;
    a.scale_d = 1.4426950408889634 / (double)eps;
    a.eps_ln2 = (float)((double)eps * 0.6931471805599453);
    for (int it = 0; it < iters; ++it) {
        a.G = hist + (size_t)it * hstep; a.G_next = hist + (size_t)(it + 1) * hstep;
        if (launch_sinkhorn_pass(a, false, s) != cudaSuccess) return LOT_ERR_CUDA;
    }
    char *Gfin = hist + (size_t)iters * hstep;
    a.G = Gfin; a.G_next = nullptr;
    if (launch_sinkhorn_pass(a, true, s) != cudaSuccess) return LOT_ERR_CUDA;

    char *M1 = at<char>(ws, L.M), *M2 = M1 + (size_t)BH * n * lt;
    char *G1 = Gfin, *G2 = Gfin + (size_t)BH * r * lt;
    float *Wp = at<float>(ws, L.Wp), *Xw = at<float>(ws, L.Xw), *dWm = at<float>(ws, L.dWm);
    ApplyArgs ap{};
    ap.cost1 = cost1; ap.cost2 = cost2; ap.G1 = G1; ap.G2 = G2; ap.M1 = M1; ap.M2 = M2;
    ap.beta = beta; ap.key_len = key_len; ap.v = v; ap.out = nullptr;
    ap.wpart = at<float>(ws, L.wpart); ap.Wp = Wp; ap.counter = at<unsigned>(ws, L.counter2);
    ap.B = B; ap.H = H; ap.n = n; ap.nk = n; ap.d = d; ap.r = r;
    ap.chunks = L.achunks; ap.rows_per_chunk = L.arows; ap.scale_d = a.scale_d;
    if (launch_apply_w(ap, dtype, s) != cudaSuccess) return LOT_ERR_CUDA;                 // W' = Diag(1/beta) Gamma2 V

    // ---- reverse of the read-out, Eq. (4): out = R1 W'
    ApplyArgs aq = ap;                                  // R1^T dout / (n beta): the key-side kernel on the query side
    aq.cost2 = cost1; aq.G2 = G1; aq.M2 = M1; aq.key_len = nullptr; aq.v = dout; aq.Wp = Xw;
    if (launch_apply_w(aq, dtype, s) != cudaSuccess) return LOT_ERR_CUDA;
    float *dbd = at<float>(ws, L.dbeta_direct);
    if (launch_bwd_w_fix(Xw, Wp, key_len, dWm, dbd, B, H, n, d, r, s) != cudaSuccess) return LOT_ERR_CUDA;
    ApplyArgs av = ap;                                  // dV = Gamma2 dW: the query-side kernel on the key side
    av.cost1 = cost2; av.G1 = G2; av.M1 = M2; av.Wp = dWm; av.out = dv;
    if (launch_apply_out(av, dtype, s) != cudaSuccess) return LOT_ERR_CUDA;
    char *dC1 = at<char>(ws, L.dC);
    char *dC2 = dC1 + (size_t)BH * n * r * lt;
    if (launch_gemm_nt(dout, ttype, Wp, false, dC1, ltype, BH, H, n, d, r, wide, s) != cudaSuccess) return LOT_ERR_CUDA;
    if (launch_gemm_nt(v, ttype, dWm, false, dC2, ltype, BH, H, n, d, r, wide, s) != cudaSuccess) return LOT_ERR_CUDA;

    // ---- reverse of the closing token update, then of the iterations, last first
    BwdRowArgs br{};
    br.cost = cost1; br.dC = dC1; br.gamma = at<void>(ws, L.gamma); br.dbeta_acc = at<void>(ws, L.dbeta_acc);
    br.beta = beta; br.len = key_len; br.len_from = BH;
    br.part = at<void>(ws, L.part); br.counter = at<unsigned>(ws, L.counter);
    br.nprob = np; br.B = B; br.H = H; br.n = n; br.r = r;
    br.chunks = L.chunks; br.rows_per_chunk = L.rows_per_chunk;
    br.scale_d = a.scale_d; br.eps = (double)eps;
    br.Ga = Gfin; br.Gb = nullptr;
    if (launch_bwd_rows(br, true, wide, s) != cudaSuccess) return LOT_ERR_CUDA;
    for (int it = iters; it >= 1; --it) {
        br.Ga = hist + (size_t)(it - 1) * hstep; br.Gb = hist + (size_t)it * hstep;
        if (launch_bwd_rows(br, false, wide, s) != cudaSuccess) return LOT_ERR_CUDA;
    }

    // ---- C = X Z^T: dX = dC Z, dZ = dC^T X
    float *zt = at<float>(ws, L.zt);
    if (launch_transpose_z(z, zt, H, r, d, s) != cudaSuccess) return LOT_ERR_CUDA;
    if (launch_gemm_nt(dC1, ltype, zt, true, dq, ttype, BH, H, n, r, d, wide, s) != cudaSuccess) return LOT_ERR_CUDA;
    if (launch_gemm_nt(dC2, ltype, zt, true, dk, ttype, BH, H, n, r, d, wide, s) != cudaSuccess) return LOT_ERR_CUDA;
    if (launch_bwd_dz(dC1, q, k, dtype, at<void>(ws, L.dzpart), dbd, br.dbeta_acc, dz, dbeta, B, H, n, d, r, L.dzchunks, wide,
                      s) != cudaSuccess)
        return LOT_ERR_CUDA;
    return LOT_OK;
}

} // extern "C"
