// General (any supported shape, float32 or bf16 tensors) kernels of the LOT attention
// forward path: similarity matrices, Sinkhorn passes over a materialised similarity
// matrix, and the two apply stages of Eq. (4).  All arithmetic is float32 on the CUDA
// cores; cross-block reductions are per-block partials summed in a fixed order by the
// last block to arrive (no spinning, no floating-point atomics).
#include "lot_common.cuh"
#include "lot_internal.h"

namespace lot {

// ------------------------------------------------------------------------------------
// Similarity matrix C[i,t] = <x_i, z_t>  (Section "Method", dot-product similarity).
// Block = 64 tokens x 64 pivots, 256 threads, 4x4 outputs per thread, K chunks of 32.
// ------------------------------------------------------------------------------------
constexpr int kTile = 64;
constexpr int kTileK = 32;
constexpr int kPadT = kTile + 4;

template <typename T, typename AccT, typename OutT>
__global__ void __launch_bounds__(256)
cost_kernel(const T *__restrict__ x, const float *__restrict__ z, OutT *__restrict__ cost,
            int H, int n, int d, int r)
{
    __shared__ __align__(16) AccT Xs[kTileK][kPadT];
    __shared__ __align__(16) AccT Zs[kTileK][kPadT];
    const int bh = blockIdx.z, h = bh % H;
    const int i0 = blockIdx.x * kTile, t0 = blockIdx.y * kTile;
    const T *xb = x + (size_t)bh * n * d;
    const float *zb = z + (size_t)h * r * d;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    AccT acc[4][4] = {};
    for (int k0 = 0; k0 < d; k0 += kTileK) {
#pragma unroll
        for (int rep = 0; rep < 2; ++rep) {
            int idx = threadIdx.x + rep * 256;
            int row = idx / 8, k4 = (idx % 8) * 4;
            float xv[4] = {0.f, 0.f, 0.f, 0.f}, zv[4] = {0.f, 0.f, 0.f, 0.f};
            if (i0 + row < n && k0 + k4 < d && LOT_CHECK((size_t)(i0 + row) * d + k0 + k4 + 4 <= (size_t)n * d))
                load4(xb + (size_t)(i0 + row) * d + k0 + k4, xv);
            if (t0 + row < r && k0 + k4 < d && LOT_CHECK((size_t)(t0 + row) * d + k0 + k4 + 4 <= (size_t)r * d))
                load4(zb + (size_t)(t0 + row) * d + k0 + k4, zv);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                Xs[k4 + j][row] = (AccT)xv[j];
                Zs[k4 + j][row] = (AccT)zv[j];
            }
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < kTileK; ++kk) {
            AccT xr[4], zr[4];
#pragma unroll
            for (int a = 0; a < 4; ++a) { xr[a] = Xs[kk][ty * 4 + a]; zr[a] = Zs[kk][tx * 4 + a]; }
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) acc[a][b] = fma(xr[a], zr[b], acc[a][b]);
        }
        __syncthreads();
    }
    OutT *cb = cost + (size_t)bh * n * r;
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        int i = i0 + ty * 4 + a;
        if (i >= n) continue;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            int t = t0 + tx * 4 + b;
            if (t < r && LOT_CHECK((size_t)i * r + t < (size_t)n * r)) cb[(size_t)i * r + t] = (OutT)acc[a][b];
        }
    }
}

// float32 tensors: exact products accumulated in float64 (the logits C/eps amplify the
// similarity error by 1/eps); bf16 tensors: float32 accumulation.  `wide` selects a float64
// result (the attention path's internal similarity matrix for float32 tensors).
cudaError_t launch_cost(const void *x, const float *z, int dtype, int BH, int H, int n, int d, int r,
                        void *cost, bool wide, cudaStream_t st)
{
    dim3 grid((n + kTile - 1) / kTile, (r + kTile - 1) / kTile, BH);
    if (dtype == 0) {
        const float *xf = static_cast<const float *>(x);
        if (wide) cost_kernel<float, double, double><<<grid, 256, 0, st>>>(xf, z, static_cast<double *>(cost), H, n, d, r);
        else cost_kernel<float, double, float><<<grid, 256, 0, st>>>(xf, z, static_cast<float *>(cost), H, n, d, r);
    } else {
        cost_kernel<__nv_bfloat16, float, float><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16 *>(x), z,
                                                                        static_cast<float *>(cost), H, n, d, r);
    }
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------
// One Sinkhorn pass (Eq. (1)-(2), scaling form).  With the token potential eliminated,
//   token update : M_i = log2 sum_t 2^(L_it + G_t)                       (row log-sum-exp)
//   pivot update : G_t += log2(beta_t / m) - log2 sum_i 2^(L_it + G_t - M_i)
// where m = 1/n_valid is the token mass.  A row is spread over LPR adjacent lanes (4, 8 or
// 16); a lane holds NV groups of four adjacent columns, group v of lane c being columns
// 4*(v*LPR + c) .. +3, so that the lanes of a warp read consecutive 16-byte pieces of
// consecutive rows.  kRowsPerThread rows are in flight per thread.  Row reductions are
// shuffles inside the LPR lanes; column sums are carried per lane as (kappa, S) pairs and
// merged lane -> warp -> block -> grid in a fixed order.
// FINAL = closing token update: writes M (and optionally g, f, plan), no pivot update.
// ------------------------------------------------------------------------------------
constexpr int kPassWarps = 8;
constexpr int kRowsPerThread = 2;

template <typename CostT>
__device__ __forceinline__ void load_cost4(const CostT *p, bool vec, int t, int r, CostT (&c)[4]);

template <>
__device__ __forceinline__ void load_cost4<float>(const float *p, bool vec, int t, int r, float (&c)[4])
{
    if (vec) {
        const float4 v = __ldg(reinterpret_cast<const float4 *>(p));
        c[0] = v.x; c[1] = v.y; c[2] = v.z; c[3] = v.w;
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) c[j] = t + j < r ? __ldg(p + j) : 0.f;
    }
}

template <>
__device__ __forceinline__ void load_cost4<double>(const double *p, bool vec, int t, int r, double (&c)[4])
{
    if (vec) {
        const double2 v0 = __ldg(reinterpret_cast<const double2 *>(p));
        const double2 v1 = __ldg(reinterpret_cast<const double2 *>(p) + 1);
        c[0] = v0.x; c[1] = v0.y; c[2] = v1.x; c[3] = v1.y;
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) c[j] = t + j < r ? __ldg(p + j) : 0.0;
    }
}

// CostT = stored similarity type, LT = type the logits, potentials and row LSE are assembled
// in (float for bf16 tensors; double when the caller's tensors are float32, so that logits of
// magnitude ~1e3 at small eps keep an absolute accuracy well below the 1e-4 output tolerance).
template <int LPR, int NV, bool FINAL, typename CostT, typename LT>
__global__ void __launch_bounds__(kPassWarps * 32)
sinkhorn_pass_kernel(PassArgs a)
{
    __shared__ float sm_k[kPassWarps][256];
    __shared__ float sm_s[kPassWarps][256];
    __shared__ int sm_last;
    constexpr int CPL = 4 * NV;
    constexpr int RPW = 32 / LPR;                    // rows per warp and step
    constexpr int RT = kRowsPerThread;
    const int p = blockIdx.x / a.chunks, chunk = blockIdx.x % a.chunks;
    const int slice = p % (a.B * a.H), b = slice / a.H, h = slice % a.H;
    int nvalid = a.n;
    if (a.len != nullptr && p >= a.len_from) nvalid = min(max(a.len[b], 0), a.n);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int sub = lane / LPR, cl = lane % LPR;
    const int r = a.r;
    const bool vec = (r & 3) == 0;                   // rows start on 16-byte boundaries
    const CostT *C = static_cast<const CostT *>(a.cost) + (size_t)p * a.n * r;
    LT *Gp = static_cast<LT *>(a.G) + (size_t)p * r;
    LT *Mp = static_cast<LT *>(a.M) + (size_t)p * a.n;
    const LT scale = (LT)a.scale_d;
    const float *mass_p = a.mass ? a.mass + (size_t)p * a.n : nullptr;

    LT Gk[CPL];
    float kap[CPL], S[CPL];
#pragma unroll
    for (int k = 0; k < CPL; ++k) {
        const int t = ((k >> 2) * LPR + cl) * 4 + (k & 3);
        Gk[k] = t < r ? Gp[t] : (LT)neg_inf();        // columns beyond r: logit -inf, term 0
        kap[k] = neg_inf();
        S[k] = 0.f;
    }
    const int row0 = chunk * a.rows_per_chunk;
    const int row_end = min(row0 + a.rows_per_chunk, a.n);       // rows this block owns
    const int row1 = min(row_end, nvalid);                        // ... that carry mass
    const int loop_end = FINAL ? row_end : row1;
    const float log2m = -lg2((float)max(nvalid, 1));
    const float mass = 1.f / (float)max(nvalid, 1);

    for (int base = row0 + warp * (RPW * RT); base < loop_end; base += kPassWarps * RPW * RT) {
        CostT c[RT][CPL];
        float mi[RT];
        bool rv[RT];
#pragma unroll
        for (int u = 0; u < RT; ++u) {
            const int i = base + u * RPW + sub;
            mi[u] = (mass_p != nullptr && i < row1) ? __ldg(mass_p + i) : mass;
            rv[u] = i < row1 && mi[u] > 0.f;
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                const int t = (v * LPR + cl) * 4;
                CostT cc[4] = {(CostT)0, (CostT)0, (CostT)0, (CostT)0};
                if (rv[u] && t < r && LOT_CHECK((size_t)i * r + (vec ? t + 4 : t + 1) <= (size_t)a.n * r))
                    load_cost4<CostT>(C + (size_t)i * r + t, vec, t, r, cc);
#pragma unroll
                for (int j = 0; j < 4; ++j) c[u][v * 4 + j] = cc[j];
            }
        }
#pragma unroll
        for (int u = 0; u < RT; ++u) {
            const int i = base + u * RPW + sub;
            const float lmi = mass_p != nullptr ? lg2(mi[u]) : log2m;      // log2 of this token's weight
            LT l[CPL];
            LT m = (LT)neg_inf();
#pragma unroll
            for (int k = 0; k < CPL; ++k) {
                l[k] = fma((LT)c[u][k], scale, Gk[k]);
                m = fmax(m, l[k]);
            }
#pragma unroll
            for (int off = LPR / 2; off > 0; off >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, off));
            float e[CPL];
            float s = 0.f;
#pragma unroll
            for (int k = 0; k < CPL; ++k) {
                e[k] = (float)(l[k] - m);          // <= 0, exact difference of nearby logits
                s += ex2(e[k]);
            }
#pragma unroll
            for (int off = LPR / 2; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
            const float lgs = lg2(s);
            if (!FINAL) {
                if (rv[u]) {
                    const float shift = mass_p != nullptr ? lmi - lgs : -lgs;
#pragma unroll
                    for (int k = 0; k < CPL; ++k)
                        if (e[k] > neg_inf()) pair_add(kap[k], S[k], e[k] + shift);
                }
            } else if (i < row_end) {
                if (cl == 0) {
                    const LT Mi = m + (LT)lgs;
                    Mp[i] = rv[u] ? Mi : (LT)__int_as_float(0x7f800000);
                    if (a.f_out)
                        a.f_out[(size_t)p * a.n + i] = rv[u] ? (float)((LT)a.eps_ln2 * ((LT)lmi - Mi)) : neg_inf();
                }
                if (a.plan_out) {
#pragma unroll
                    for (int k = 0; k < CPL; ++k) {
                        const int t = ((k >> 2) * LPR + cl) * 4 + (k & 3);
                        if (t < r) a.plan_out[((size_t)p * a.n + i) * r + t] = rv[u] ? mi[u] * ex2(e[k] - lgs) : 0.f;
                    }
                }
            }
        }
    }
    if (FINAL) {
        if (chunk == 0 && a.g_out != nullptr && threadIdx.x < r)
            a.g_out[(size_t)p * r + threadIdx.x] = (float)(Gp[threadIdx.x] * (LT)a.eps_ln2);
        return;
    }

    // lanes of different row groups hold the same columns: merge them, then the warps
#pragma unroll
    for (int off = LPR; off < 32; off <<= 1) {
#pragma unroll
        for (int k = 0; k < CPL; ++k) {
            float k2 = __shfl_xor_sync(0xffffffffu, kap[k], off);
            float s2 = __shfl_xor_sync(0xffffffffu, S[k], off);
            pair_merge(kap[k], S[k], k2, s2);
        }
    }
    if (sub == 0) {
#pragma unroll
        for (int k = 0; k < CPL; ++k) {
            const int t = ((k >> 2) * LPR + cl) * 4 + (k & 3);
            if (t < r) {
                sm_k[warp][t] = kap[k];
                sm_s[warp][t] = S[k];
            }
        }
    }
    __syncthreads();
    const int t = threadIdx.x;
    if (t < r) {
        float kk = sm_k[0][t], ss = sm_s[0][t];
#pragma unroll
        for (int w = 1; w < kPassWarps; ++w) pair_merge(kk, ss, sm_k[w][t], sm_s[w][t]);
        float *dst = a.part + (((size_t)p * a.chunks + chunk) * r + t) * 2;
        __stcg(dst, kk);
        __stcg(dst + 1, ss);
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned ticket = atomicAdd(a.counter + p, 1u);
        sm_last = (ticket == (unsigned)a.chunks - 1u);
    }
    __syncthreads();
    if (!sm_last) return;
    __threadfence();
    if (t < r) {
        float kk = neg_inf(), ss = 0.f;
        for (int c = 0; c < a.chunks; ++c) {
            const float *src = a.part + (((size_t)p * a.chunks + c) * r + t) * 2;
            pair_merge(kk, ss, __ldcg(src), __ldcg(src + 1));
        }
        if (nvalid <= 0) {
            atomicOr(a.status, 2 /* LOT_DEV_EMPTY */);
        } else {
            LT lam = (LT)kk + (LT)lg2(ss);
            // uniform weights: the common factor 1/nvalid was left out of the column sums
            LT gn = Gp[t] + (LT)lg2(a.mass ? a.beta[h * r + t] : a.beta[h * r + t] * (float)nvalid) - lam;
            if (!isfinite((float)gn)) atomicOr(a.status, 1 /* LOT_DEV_NONFINITE */);
            (a.G_next != nullptr ? static_cast<LT *>(a.G_next) + (size_t)p * r : Gp)[t] = gn;
        }
    }
    if (threadIdx.x == 0) a.counter[p] = 0u;
}

int pass_chunks(int nprob, int n)
{
    // enough blocks for ~4 per SM over 148 SMs, at least 64 rows each
    int want = (592 + nprob - 1) / nprob;
    int most = (n + 63) / 64;
    int c = want < most ? want : most;
    return c < 1 ? 1 : c;
}

template <int LPR, int NV, typename CostT, typename LT>
static cudaError_t launch_pass_t(const PassArgs &a, bool final_pass, cudaStream_t st)
{
    dim3 grid((unsigned)(a.nprob * a.chunks));
    if (final_pass)
        sinkhorn_pass_kernel<LPR, NV, true, CostT, LT><<<grid, kPassWarps * 32, 0, st>>>(a);
    else
        sinkhorn_pass_kernel<LPR, NV, false, CostT, LT><<<grid, kPassWarps * 32, 0, st>>>(a);
    return cudaGetLastError();
}

template <typename CostT, typename LT>
static cudaError_t launch_pass_r(const PassArgs &a, bool final_pass, cudaStream_t st)
{
    const int r = a.r;
    if (r <= 16) return launch_pass_t<4, 1, CostT, LT>(a, final_pass, st);
    if (r <= 32) return launch_pass_t<4, 2, CostT, LT>(a, final_pass, st);
    if (r <= 64) return launch_pass_t<4, 4, CostT, LT>(a, final_pass, st);
    if (r <= 128) return launch_pass_t<8, 4, CostT, LT>(a, final_pass, st);
    return launch_pass_t<16, 4, CostT, LT>(a, final_pass, st);
}

cudaError_t launch_sinkhorn_pass(const PassArgs &a, bool final_pass, cudaStream_t st)
{
    switch (a.mode) {
    case kModeF32: return launch_pass_r<float, float>(a, final_pass, st);
    case kModeCostF32Wide: return launch_pass_r<float, double>(a, final_pass, st);
    default: return launch_pass_r<double, double>(a, final_pass, st);
    }
}

// ------------------------------------------------------------------------------------
// Apply, key side (Eq. (4): Y = Gamma2 V, Z' = Diag(beta)^-1 Y).
//   W'[t,c] = (1/beta_t) sum_j m 2^(L2_jt + G2_t - M2_j) v[j,c]
// Block = 64 pivots x 64 channels over one chunk of keys; the last block of a tile sums
// the chunk partials in order and scales.
// ------------------------------------------------------------------------------------
constexpr int kRowStep = 32;

int apply_chunks(int BH, int n, int r, int d)
{
    int tiles = ((r + kTile - 1) / kTile) * ((d + kTile - 1) / kTile) * BH;
    int want = (592 + tiles - 1) / tiles;
    int most = (n + 255) / 256;
    int c = want < most ? want : most;
    return c < 1 ? 1 : c;
}

template <typename T, typename LT>
__global__ void __launch_bounds__(256)
apply_w_kernel(ApplyArgs a)
{
    __shared__ __align__(16) float Ps[kRowStep][kPadT];
    __shared__ __align__(16) float Vs[kRowStep][kPadT];
    __shared__ int sm_last;
    const int bh = blockIdx.z, b = bh / a.H, h = bh % a.H;
    const int cblks = (a.d + kTile - 1) / kTile;
    const int tblk = blockIdx.y / cblks, cblk = blockIdx.y % cblks;
    const int t0 = tblk * kTile, c0 = cblk * kTile;
    const int chunk = blockIdx.x;
    const int n = a.nk, r = a.r, d = a.d;
    int nvalid = n;
    if (a.key_len != nullptr) nvalid = min(max(a.key_len[b], 0), n);
    const float *mass2 = a.mass2 ? a.mass2 + (size_t)bh * n : nullptr;
    const int row0 = chunk * a.rows_per_chunk;
    const int row1 = min(min(row0 + a.rows_per_chunk, n), nvalid);
    const LT *C = static_cast<const LT *>(a.cost2) + (size_t)bh * n * r;
    const LT *G = static_cast<const LT *>(a.G2) + (size_t)bh * r;
    const LT *M = static_cast<const LT *>(a.M2) + (size_t)bh * n;
    const LT scale = (LT)a.scale_d;
    const T *V = static_cast<const T *>(a.v) + (size_t)bh * n * d;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    float acc[4][4] = {};

    for (int j0 = row0; j0 < row1; j0 += kRowStep) {
#pragma unroll
        for (int rep = 0; rep < 8; ++rep) {
            int idx = threadIdx.x + rep * 256;
            int jj = idx / kTile, tt = idx % kTile;
            int j = j0 + jj, t = t0 + tt;
            float val = 0.f;
            if (j < row1 && t < r) {
                val = ex2((float)(fma(__ldg(C + (size_t)j * r + t), scale, __ldg(G + t)) - __ldg(M + j)));
                if (mass2 != nullptr) val *= __ldg(mass2 + j);        // a massless key has M = +inf: val is 0 already
            }
            Ps[jj][tt] = val;
        }
#pragma unroll
        for (int rep = 0; rep < 2; ++rep) {
            int idx = threadIdx.x + rep * 256;
            int jj = idx / 16, c4 = (idx % 16) * 4;
            int j = j0 + jj, c = c0 + c4;
            float vv[4] = {0.f, 0.f, 0.f, 0.f};
            if (j < row1 && c < d) load4(V + (size_t)j * d + c, vv);
            *reinterpret_cast<float4 *>(&Vs[jj][c4]) = make_float4(vv[0], vv[1], vv[2], vv[3]);
        }
        __syncthreads();
#pragma unroll
        for (int jj = 0; jj < kRowStep; ++jj) {
            float4 pa = *reinterpret_cast<const float4 *>(&Ps[jj][ty * 4]);
            float4 vb = *reinterpret_cast<const float4 *>(&Vs[jj][tx * 4]);
            float pr[4] = {pa.x, pa.y, pa.z, pa.w}, vr[4] = {vb.x, vb.y, vb.z, vb.w};
#pragma unroll
            for (int x = 0; x < 4; ++x)
#pragma unroll
                for (int y = 0; y < 4; ++y) acc[x][y] = fmaf(pr[x], vr[y], acc[x][y]);
        }
        __syncthreads();
    }
    float *wp = a.wpart + ((size_t)bh * a.chunks + chunk) * r * d;
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        int t = t0 + ty * 4 + x;
#pragma unroll
        for (int y = 0; y < 4; ++y) {
            int c = c0 + tx * 4 + y;
            if (t < r && c < d) __stcg(wp + (size_t)t * d + c, acc[x][y]);
        }
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned ticket = atomicAdd(a.counter + (size_t)bh * gridDim.y + blockIdx.y, 1u);
        sm_last = (ticket == (unsigned)a.chunks - 1u);
    }
    __syncthreads();
    if (!sm_last) return;
    __threadfence();
    const float mass = a.mass2 ? 1.f : (nvalid > 0 ? 1.f / (float)nvalid : 0.f);
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        int t = t0 + ty * 4 + x;
        if (t >= r) continue;
        const float sc = mass / a.beta[h * r + t];
#pragma unroll
        for (int y = 0; y < 4; ++y) {
            int c = c0 + tx * 4 + y;
            if (c >= d) continue;
            float sum = 0.f;
            for (int ch = 0; ch < a.chunks; ++ch)
                sum += __ldcg(a.wpart + (((size_t)bh * a.chunks + ch) * r + t) * d + c);
            a.Wp[((size_t)bh * r + t) * d + c] = sum * sc;
        }
    }
    if (threadIdx.x == 0) a.counter[(size_t)bh * gridDim.y + blockIdx.y] = 0u;
}

cudaError_t launch_apply_w(const ApplyArgs &a, int dtype, cudaStream_t st)
{
    int tblks = (a.r + kTile - 1) / kTile, cblks = (a.d + kTile - 1) / kTile;
    dim3 grid(a.chunks, tblks * cblks, a.B * a.H);
    if (dtype == 0) apply_w_kernel<float, double><<<grid, 256, 0, st>>>(a);
    else apply_w_kernel<__nv_bfloat16, float><<<grid, 256, 0, st>>>(a);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------
// Apply, query side (Eq. (4): O = Gamma1^T Z', row-stochastic scaling):
//   out[i,c] = sum_t 2^(L1_it + G1_t - M1_i) W'[t,c]
// Block = 64 queries x 64 channels, pivots in steps of 32.
// ------------------------------------------------------------------------------------
template <typename T, typename LT>
__global__ void __launch_bounds__(256)
apply_out_kernel(ApplyArgs a)
{
    __shared__ __align__(16) float Ps[kTileK][kPadT];
    __shared__ __align__(16) float Ws[kTileK][kPadT];
    const int bh = blockIdx.z;
    const int i0 = blockIdx.x * kTile, c0 = blockIdx.y * kTile;
    const int n = a.n, r = a.r, d = a.d;
    const LT *C = static_cast<const LT *>(a.cost1) + (size_t)bh * n * r;
    const LT *G = static_cast<const LT *>(a.G1) + (size_t)bh * r;
    const LT *M = static_cast<const LT *>(a.M1) + (size_t)bh * n;
    const LT scale = (LT)a.scale_d;
    const float *W = a.Wp + (size_t)bh * r * d;
    T *O = static_cast<T *>(a.out) + (size_t)bh * n * d;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    float acc[4][4] = {};
    for (int tb = 0; tb < r; tb += kTileK) {
#pragma unroll
        for (int rep = 0; rep < 8; ++rep) {
            int idx = threadIdx.x + rep * 256;
            int tt = idx % kTileK, ii = idx / kTileK;
            int i = i0 + ii, t = tb + tt;
            float val = 0.f;
            if (i < n && t < r) val = ex2((float)(fma(__ldg(C + (size_t)i * r + t), scale, __ldg(G + t)) - __ldg(M + i)));
            Ps[tt][ii] = val;
        }
#pragma unroll
        for (int rep = 0; rep < 2; ++rep) {
            int idx = threadIdx.x + rep * 256;
            int tt = idx / 16, c4 = (idx % 16) * 4;
            int t = tb + tt, c = c0 + c4;
            float4 w = make_float4(0.f, 0.f, 0.f, 0.f);
            if (t < r && c < d) w = *reinterpret_cast<const float4 *>(W + (size_t)t * d + c);
            *reinterpret_cast<float4 *>(&Ws[tt][c4]) = w;
        }
        __syncthreads();
#pragma unroll
        for (int tt = 0; tt < kTileK; ++tt) {
            float4 pa = *reinterpret_cast<const float4 *>(&Ps[tt][ty * 4]);
            float4 wb = *reinterpret_cast<const float4 *>(&Ws[tt][tx * 4]);
            float pr[4] = {pa.x, pa.y, pa.z, pa.w}, wr[4] = {wb.x, wb.y, wb.z, wb.w};
#pragma unroll
            for (int x = 0; x < 4; ++x)
#pragma unroll
                for (int y = 0; y < 4; ++y) acc[x][y] = fmaf(pr[x], wr[y], acc[x][y]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        int i = i0 + ty * 4 + x, c = c0 + tx * 4;
        if (i < n && c < d && LOT_CHECK((size_t)i * d + c + 4 <= (size_t)n * d)) store4(O + (size_t)i * d + c, acc[x]);
    }
}

cudaError_t launch_apply_out(const ApplyArgs &a, int dtype, cudaStream_t st)
{
    dim3 grid((a.n + kTile - 1) / kTile, (a.d + kTile - 1) / kTile, a.B * a.H);
    if (dtype == 0) apply_out_kernel<float, double><<<grid, 256, 0, st>>>(a);
    else apply_out_kernel<__nv_bfloat16, float><<<grid, 256, 0, st>>>(a);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------
// Forward variants: starting potentials, the weights and the softmax row of the [CLS] treatment
// ------------------------------------------------------------------------------------
template <typename LT>
__global__ void g_init_kernel(const float *__restrict__ g_in, LT *__restrict__ G, size_t count, double scale)
{
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (size_t)gridDim.x * blockDim.x)
        G[i] = g_in ? (LT)((double)g_in[i] * scale) : (LT)0;
}

cudaError_t launch_g_init(const float *g_in, void *G, size_t count, double scale, bool wide, cudaStream_t st)
{
    if (count == 0) return cudaSuccess;
    const int blocks = (int)((count + 255) / 256 < 1024 ? (count + 255) / 256 : 1024);
    if (wide) g_init_kernel<double><<<blocks, 256, 0, st>>>(g_in, static_cast<double *>(G), count, scale);
    else g_init_kernel<float><<<blocks, 256, 0, st>>>(g_in, static_cast<float *>(G), count, scale);
    return cudaGetLastError();
}

// Eq. (5) keeps the [CLS] token (index 0) out of the transport problem: zero weight for it on both sides, uniform
// weights over the other queries and over the other valid keys.
__global__ void cls_marginals_kernel(float *__restrict__ a, float *__restrict__ b, const int32_t *key_len, int H, int nq,
                                     int nk, int *status)
{
    const int bh = blockIdx.x, bb = bh / H;
    int kv = nk;
    if (key_len != nullptr) kv = min(max(key_len[bb], 0), nk);
    if (threadIdx.x == 0 && (kv <= 1 || nq <= 1)) atomicOr(status, 2 /* LOT_DEV_EMPTY */);
    const float wa = nq > 1 ? 1.f / (float)(nq - 1) : 0.f, wb = kv > 1 ? 1.f / (float)(kv - 1) : 0.f;
    for (int i = threadIdx.x; i < nq; i += blockDim.x) a[(size_t)bh * nq + i] = i == 0 ? 0.f : wa;
    for (int j = threadIdx.x; j < nk; j += blockDim.x) b[(size_t)bh * nk + j] = (j == 0 || j >= kv) ? 0.f : wb;
}

cudaError_t launch_cls_marginals(float *a, float *b, const int32_t *key_len, int B, int H, int nq, int nk, int *status,
                                 cudaStream_t st)
{
    cls_marginals_kernel<<<B * H, 256, 0, st>>>(a, b, key_len, H, nq, nk, status);
    return cudaGetLastError();
}

// One block per slice: scores tau <q_0, k_j> of the valid keys (kept in global scratch), their maximum, the
// exponentials and their sum, then one thread per channel adds up the weighted values.
template <typename T>
__global__ void __launch_bounds__(256)
cls_row_kernel(const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ v, const int32_t *key_len, int H,
               int nq, int nk, int d, float tau, float *__restrict__ scores, T *__restrict__ out)
{
    __shared__ float red[256];
    __shared__ float q0[256];
    const int bh = blockIdx.x, bb = bh / H;
    int kv = nk;
    if (key_len != nullptr) kv = min(max(key_len[bb], 0), nk);
    const T *qb = q + (size_t)bh * nq * d, *kb = k + (size_t)bh * nk * d, *vb = v + (size_t)bh * nk * d;
    float *sc = scores + (size_t)bh * nk;
    for (int c = threadIdx.x; c < d; c += blockDim.x) q0[c] = Elem<T>::load(qb + c);
    __syncthreads();
    float mx = neg_inf();
    for (int j = threadIdx.x; j < kv; j += blockDim.x) {
        float acc = 0.f;
        for (int c = 0; c < d; c += 4) {
            float kk[4];
            load4(kb + (size_t)j * d + c, kk);
            acc = fmaf(q0[c], kk[0], acc); acc = fmaf(q0[c + 1], kk[1], acc);
            acc = fmaf(q0[c + 2], kk[2], acc); acc = fmaf(q0[c + 3], kk[3], acc);
        }
        acc *= tau;
        sc[j] = acc;
        mx = fmaxf(mx, acc);
    }
    red[threadIdx.x] = mx;
    __syncthreads();
    for (int off = 128; off > 0; off >>= 1) {
        if (threadIdx.x < off) red[threadIdx.x] = fmaxf(red[threadIdx.x], red[threadIdx.x + off]);
        __syncthreads();
    }
    mx = red[0];
    __syncthreads();
    float den = 0.f;
    for (int j = threadIdx.x; j < kv; j += blockDim.x) {
        const float e = __expf(sc[j] - mx);
        sc[j] = e;
        den += e;
    }
    red[threadIdx.x] = den;
    __syncthreads();
    for (int off = 128; off > 0; off >>= 1) {
        if (threadIdx.x < off) red[threadIdx.x] += red[threadIdx.x + off];
        __syncthreads();
    }
    den = red[0];
    __threadfence_block();
    __syncthreads();
    for (int c = threadIdx.x; c < d; c += blockDim.x) {
        float acc = 0.f;
        for (int j = 0; j < kv; ++j) acc = fmaf(sc[j], Elem<T>::load(vb + (size_t)j * d + c), acc);
        Elem<T>::store(out + (size_t)bh * nq * d + c, kv > 0 ? acc / den : 0.f);
    }
}

cudaError_t launch_cls_row(const void *q, const void *k, const void *v, const int32_t *key_len, int dtype, int B, int H,
                           int nq, int nk, int d, float tau, float *scores, void *out, cudaStream_t st)
{
    if (dtype == 0)
        cls_row_kernel<float><<<B * H, 256, 0, st>>>(static_cast<const float *>(q), static_cast<const float *>(k),
                                                     static_cast<const float *>(v), key_len, H, nq, nk, d, tau, scores,
                                                     static_cast<float *>(out));
    else
        cls_row_kernel<__nv_bfloat16><<<B * H, 256, 0, st>>>(static_cast<const __nv_bfloat16 *>(q),
                                                             static_cast<const __nv_bfloat16 *>(k),
                                                             static_cast<const __nv_bfloat16 *>(v), key_len, H, nq, nk, d, tau,
                                                             scores, static_cast<__nv_bfloat16 *>(out));
    return cudaGetLastError();
}

LOT_DEBUG_FLAG_READER(kernels_debug_flag)

} // namespace lot
