// Backward of the LOT attention forward (Section "Learning": the parameters are trained by back-propagating through
// the two shared-eps Sinkhorn problems, Eq. (1)-(2), and the glued composition, Eq. (3)-(4)).  What is differentiated
// is the unrolled iteration of the forward path: g0 = 0, `iters` times (token update, pivot update), one closing
// token update, plan read-out.  The similarity matrices are materialised (general path); nothing of the forward is
// stored but the pivot potentials of every iteration, from which each reverse step recomputes its plan.
//
// Notation (natural units): R_it = softmax_t((C_it + g_t)/eps) is the row-stochastic plan for potentials g, m_i the
// token mass (1/valid count, 0 for masked keys).  Reverse of one (token update, pivot update) pair that took g to g+
// with incoming gradient gamma = d/dg+:
//     q_it   = R_it / c_t,  c_t = sum_i m_i R_it = beta_t exp((g_t - g+_t)/eps)      (column mass before the update)
//     rho_i  = sum_t q_it gamma_t
//     dC_it -= m_i (q_it gamma_t - R_it rho_i),   d/dg_t = sum_i m_i R_it rho_i,   d/dbeta_t += eps gamma_t / beta_t
// Reverse of the closing update and read-out, given dR (gradient with respect to R):
//     dy_it = R_it (dR_it - sum_t' R_it' dR_it'),  dC_it = dy_it / eps,  d/dg_t = sum_i dy_it / eps.
// All arithmetic is float for bf16 tensors and double for float32 tensors, like the forward general path; column
// sums are per-block partials added in a fixed order by the last block to arrive.
#include "lot_common.cuh"
#include "lot_internal.h"

namespace lot {

namespace {

constexpr int kBwdWarps = 8;

template <typename LT>
__device__ __forceinline__ void load_row4(const LT *p, bool vec, int t, int r, LT (&c)[4]);

template <>
__device__ __forceinline__ void load_row4<float>(const float *p, bool vec, int t, int r, float (&c)[4])
{
    if (vec) {
        const float4 v = *reinterpret_cast<const float4 *>(p);
        c[0] = v.x; c[1] = v.y; c[2] = v.z; c[3] = v.w;
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) c[j] = t + j < r ? p[j] : 0.f;
    }
}

template <>
__device__ __forceinline__ void load_row4<double>(const double *p, bool vec, int t, int r, double (&c)[4])
{
    if (vec) {
        const double2 v0 = *reinterpret_cast<const double2 *>(p);
        const double2 v1 = *(reinterpret_cast<const double2 *>(p) + 1);
        c[0] = v0.x; c[1] = v0.y; c[2] = v1.x; c[3] = v1.y;
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) c[j] = t + j < r ? p[j] : 0.0;
    }
}

template <typename LT>
__device__ __forceinline__ void store_row4(LT *p, bool vec, int t, int r, const LT (&c)[4])
{
    if (vec) {
        if (sizeof(LT) == 4) {
            *reinterpret_cast<float4 *>(p) = make_float4((float)c[0], (float)c[1], (float)c[2], (float)c[3]);
        } else {
            *reinterpret_cast<double2 *>(p) = make_double2((double)c[0], (double)c[1]);
            *(reinterpret_cast<double2 *>(p) + 1) = make_double2((double)c[2], (double)c[3]);
        }
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (t + j < r) p[j] = c[j];
    }
}

// A row is spread over LPR adjacent lanes; a lane holds NV groups of four adjacent columns, group v of lane c being
// columns 4*(v*LPR + c) .. +3 (the layout of the forward pass kernel).
template <int LPR, int NV, bool CLOSE, typename LT>
__global__ void __launch_bounds__(kBwdWarps * 32)
bwd_row_kernel(BwdRowArgs a)
{
    __shared__ LT sm_c[kBwdWarps][256];
    __shared__ int sm_last;
    constexpr int CPL = 4 * NV;
    constexpr int RPW = 32 / LPR;
    const int p = blockIdx.x / a.chunks, chunk = blockIdx.x % a.chunks;
    const int slice = p % (a.B * a.H), b = slice / a.H, h = slice % a.H;
    int nvalid = a.n;
    if (a.len != nullptr && p >= a.len_from) nvalid = min(max(a.len[b], 0), a.n);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int sub = lane / LPR, cl = lane % LPR;
    const int r = a.r;
    const bool vec = (r & 3) == 0;
    const LT *C = static_cast<const LT *>(a.cost) + (size_t)p * a.n * r;
    LT *D = static_cast<LT *>(a.dC) + (size_t)p * a.n * r;
    const LT *Ga = static_cast<const LT *>(a.Ga) + (size_t)p * r;
    LT *gam = static_cast<LT *>(a.gamma) + (size_t)p * r;
    const LT scale = (LT)a.scale_d;
    const LT inv_eps = (LT)(1.0 / a.eps);
    const LT mass = nvalid > 0 ? (LT)1 / (LT)nvalid : (LT)0;

    LT Gk[CPL], Hk[CPL], gk[CPL], col[CPL];
#pragma unroll
    for (int k = 0; k < CPL; ++k) {
        const int t = ((k >> 2) * LPR + cl) * 4 + (k & 3);
        Gk[k] = t < r ? Ga[t] : (LT)neg_inf();
        Hk[k] = (LT)0;
        gk[k] = (LT)0;
        if (!CLOSE && t < r) {
            // exponent offset of q_it = 2^(L_it + G+_t - log2 beta_t - M_i)
            Hk[k] = static_cast<const LT *>(a.Gb)[(size_t)p * r + t] - (LT)log2((double)a.beta[h * r + t]);
            gk[k] = gam[t];
        }
        col[k] = (LT)0;
    }
    const int row0 = chunk * a.rows_per_chunk;
    const int row_end = min(row0 + a.rows_per_chunk, a.n);
    const int row1 = min(row_end, nvalid);
    const int loop_end = CLOSE ? row_end : row1;       // close also zeroes the rows of masked tokens

    for (int base = row0 + warp * RPW; base < loop_end; base += kBwdWarps * RPW) {
        const int i = base + sub;
        const bool rv = i < row1;
        LT c[CPL], x[CPL];
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            const int t = (v * LPR + cl) * 4;
            LT cc[4] = {(LT)0, (LT)0, (LT)0, (LT)0}, xx[4] = {(LT)0, (LT)0, (LT)0, (LT)0};
            if (rv && t < r && LOT_CHECK((size_t)i * r + (vec ? t + 4 : t + 1) <= (size_t)a.n * r)) {
                load_row4<LT>(C + (size_t)i * r + t, vec, t, r, cc);
                load_row4<LT>(D + (size_t)i * r + t, vec, t, r, xx);
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) { c[v * 4 + j] = cc[j]; x[v * 4 + j] = xx[j]; }
        }
        LT l[CPL];
        LT m = (LT)neg_inf();
#pragma unroll
        for (int k = 0; k < CPL; ++k) {
            l[k] = fma(c[k], scale, Gk[k]);
            m = fmax(m, l[k]);
        }
#pragma unroll
        for (int off = LPR / 2; off > 0; off >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, off));
        float pk[CPL];
        float s = 0.f;
#pragma unroll
        for (int k = 0; k < CPL; ++k) {
            pk[k] = ex2((float)(l[k] - m));
            s += pk[k];
        }
#pragma unroll
        for (int off = LPR / 2; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
        const float inv_s = 1.f / s;
        LT rho = (LT)0;
        if (CLOSE) {
#pragma unroll
            for (int k = 0; k < CPL; ++k) rho += (LT)(pk[k] * inv_s) * x[k];
        } else {
            const LT Mi = m + (LT)lg2(s);
#pragma unroll
            for (int k = 0; k < CPL; ++k) {
                // c[k] is not needed any more: it takes q_it gamma_t
                const int t = ((k >> 2) * LPR + cl) * 4 + (k & 3);
                const float qv = t < r ? ex2((float)(fma(c[k], scale, Hk[k]) - Mi)) : 0.f;
                c[k] = (LT)qv * gk[k];                        // q_it gamma_t
                rho += c[k];
            }
        }
#pragma unroll
        for (int off = LPR / 2; off > 0; off >>= 1) rho += __shfl_xor_sync(0xffffffffu, rho, off);
        if (CLOSE) {
#pragma unroll
            for (int k = 0; k < CPL; ++k) {
                const LT dy = rv ? (LT)(pk[k] * inv_s) * (x[k] - rho) * inv_eps : (LT)0;
                x[k] = dy;
                col[k] += dy;
            }
        } else {
#pragma unroll
            for (int k = 0; k < CPL; ++k) {
                const LT Rr = (LT)(pk[k] * inv_s) * rho;
                if (rv) {
                    x[k] -= mass * (c[k] - Rr);
                    col[k] += mass * Rr;
                }
            }
        }
        if (i < loop_end) {
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                const int t = (v * LPR + cl) * 4;
                if (t < r && LOT_CHECK((size_t)i * r + (vec ? t + 4 : t + 1) <= (size_t)a.n * r)) {
                    LT xx[4] = {x[v * 4], x[v * 4 + 1], x[v * 4 + 2], x[v * 4 + 3]};
                    store_row4<LT>(D + (size_t)i * r + t, vec, t, r, xx);
                }
            }
        }
    }

    // lanes of different row groups hold the same columns: add them, then the warps, then the blocks
#pragma unroll
    for (int off = LPR; off < 32; off <<= 1) {
#pragma unroll
        for (int k = 0; k < CPL; ++k) col[k] += __shfl_xor_sync(0xffffffffu, col[k], off);
    }
    if (sub == 0) {
#pragma unroll
        for (int k = 0; k < CPL; ++k) {
            const int t = ((k >> 2) * LPR + cl) * 4 + (k & 3);
            if (t < r) sm_c[warp][t] = col[k];
        }
    }
    __syncthreads();
    const int t = threadIdx.x;
    LT *part = static_cast<LT *>(a.part);
    if (t < r) {
        LT sum = sm_c[0][t];
#pragma unroll
        for (int w = 1; w < kBwdWarps; ++w) sum += sm_c[w][t];
        __stcg(part + ((size_t)p * a.chunks + chunk) * r + t, sum);
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
        LT sum = (LT)0;
        for (int c = 0; c < a.chunks; ++c) sum += __ldcg(part + ((size_t)p * a.chunks + c) * r + t);
        if (!CLOSE && nvalid > 0) {
            LT *acc = static_cast<LT *>(a.dbeta_acc) + (size_t)p * r;
            acc[t] += (LT)a.eps * gam[t] / (LT)a.beta[h * r + t];
        }
        gam[t] = nvalid > 0 ? sum : (LT)0;
    }
    if (threadIdx.x == 0) a.counter[p] = 0u;
}

template <int LPR, int NV, typename LT>
cudaError_t launch_rows_t(const BwdRowArgs &a, bool close, cudaStream_t st)
{
    dim3 grid((unsigned)(a.nprob * a.chunks));
    if (close) bwd_row_kernel<LPR, NV, true, LT><<<grid, kBwdWarps * 32, 0, st>>>(a);
    else bwd_row_kernel<LPR, NV, false, LT><<<grid, kBwdWarps * 32, 0, st>>>(a);
    return cudaGetLastError();
}

template <typename LT>
cudaError_t launch_rows_r(const BwdRowArgs &a, bool close, cudaStream_t st)
{
    const int r = a.r;
    if (r <= 16) return launch_rows_t<4, 1, LT>(a, close, st);
    if (r <= 32) return launch_rows_t<4, 2, LT>(a, close, st);
    if (r <= 64) return launch_rows_t<4, 4, LT>(a, close, st);
    if (r <= 128) return launch_rows_t<8, 4, LT>(a, close, st);
    return launch_rows_t<16, 4, LT>(a, close, st);
}

// ------------------------------------------------------------------------------------
// out[s][i][j] = sum_k A[s][i][k] Bm[.][j][k]: 64 x 64 tiles, 256 threads, 4 x 4 results per thread.
// ------------------------------------------------------------------------------------
constexpr int kGT = 64, kGK = 16, kGPad = kGT + 4;

template <typename AccT, typename T> __device__ __forceinline__ AccT ld_as(T v) { return (AccT)v; }
template <typename AccT> __device__ __forceinline__ AccT ld_as(__nv_bfloat16 v) { return (AccT)__bfloat162float(v); }
template <typename OutT> struct StoreAs {
    template <typename AccT> static __device__ __forceinline__ OutT conv(AccT v) { return (OutT)v; }
};
template <> struct StoreAs<__nv_bfloat16> {
    template <typename AccT> static __device__ __forceinline__ __nv_bfloat16 conv(AccT v) { return __float2bfloat16_rn((float)v); }
};

template <typename AT, typename AccT, typename OutT>
__global__ void __launch_bounds__(256)
gemm_nt_kernel(const AT *__restrict__ A, const float *__restrict__ Bm, OutT *__restrict__ out, int H, int per_head,
               int n, int K, int J)
{
    __shared__ AccT As[kGK][kGPad];
    __shared__ AccT Bs[kGK][kGPad];
    const int s = blockIdx.z;
    const int i0 = blockIdx.x * kGT, j0 = blockIdx.y * kGT;
    const AT *Ab = A + (size_t)s * n * K;
    const float *Bb = Bm + (size_t)(per_head ? s % H : s) * J * K;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    AccT acc[4][4] = {};
    for (int k0 = 0; k0 < K; k0 += kGK) {
#pragma unroll
        for (int rep = 0; rep < 4; ++rep) {
            const int idx = threadIdx.x + rep * 256;
            const int row = idx / kGK, kk = idx % kGK;
            AccT av = (AccT)0, bv = (AccT)0;
            if (i0 + row < n && k0 + kk < K) av = ld_as<AccT>(Ab[(size_t)(i0 + row) * K + k0 + kk]);
            if (j0 + row < J && k0 + kk < K) bv = (AccT)Bb[(size_t)(j0 + row) * K + k0 + kk];
            As[kk][row] = av;
            Bs[kk][row] = bv;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < kGK; ++kk) {
            AccT ar[4], br[4];
#pragma unroll
            for (int x = 0; x < 4; ++x) { ar[x] = As[kk][ty * 4 + x]; br[x] = Bs[kk][tx * 4 + x]; }
#pragma unroll
            for (int x = 0; x < 4; ++x)
#pragma unroll
                for (int y = 0; y < 4; ++y) acc[x][y] = fma(ar[x], br[y], acc[x][y]);
        }
        __syncthreads();
    }
    OutT *ob = out + (size_t)s * n * J;
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        const int i = i0 + ty * 4 + x;
        if (i >= n) continue;
#pragma unroll
        for (int y = 0; y < 4; ++y) {
            const int j = j0 + tx * 4 + y;
            if (j < J && LOT_CHECK((size_t)i * J + j < (size_t)n * J)) ob[(size_t)i * J + j] = StoreAs<OutT>::conv(acc[x][y]);
        }
    }
}

template <typename AT, typename AccT>
cudaError_t launch_gemm_out(const void *A, const float *Bm, bool per_head, void *out, int out_type, int S, int H, int n,
                            int K, int J, cudaStream_t st)
{
    dim3 grid((n + kGT - 1) / kGT, (J + kGT - 1) / kGT, S);
    const AT *a = static_cast<const AT *>(A);
    if (out_type == 0)
        gemm_nt_kernel<AT, AccT, float><<<grid, 256, 0, st>>>(a, Bm, static_cast<float *>(out), H, per_head, n, K, J);
    else if (out_type == 1)
        gemm_nt_kernel<AT, AccT, __nv_bfloat16><<<grid, 256, 0, st>>>(a, Bm, static_cast<__nv_bfloat16 *>(out), H, per_head, n, K, J);
    else
        gemm_nt_kernel<AT, AccT, double><<<grid, 256, 0, st>>>(a, Bm, static_cast<double *>(out), H, per_head, n, K, J);
    return cudaGetLastError();
}

__global__ void bwd_w_fix_kernel(const float *__restrict__ Xw, const float *__restrict__ Wp, const int32_t *key_len,
                                 float *__restrict__ dWm, float *__restrict__ dbeta_direct, int H, int n, int d, int r)
{
    // one warp per (slice, pivot)
    const int s = blockIdx.x, b = s / H;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, warps = blockDim.x >> 5;
    int nvalid = n;
    if (key_len != nullptr) nvalid = min(max(key_len[b], 0), n);
    const float km = nvalid > 0 ? (float)n / (float)nvalid : 0.f;
    for (int t = warp; t < r; t += warps) {
        const size_t o = ((size_t)s * r + t) * d;
        float dot = 0.f;
        for (int c = lane; c < d; c += 32) {
            const float x = Xw[o + c];
            dot = fmaf(x, Wp[o + c], dot);
            dWm[o + c] = x * km;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
        if (lane == 0) dbeta_direct[(size_t)s * r + t] = -(float)n * dot;
    }
}

__global__ void transpose_z_kernel(const float *__restrict__ z, float *__restrict__ zt, int r, int d, size_t total)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const int c = (int)(idx % d);
    const int t = (int)((idx / d) % r);
    const size_t h = idx / ((size_t)r * d);
    zt[(h * d + c) * r + t] = z[idx];
}

// partial[p][chunk][t][c] = sum over the chunk's rows of dC[p][i][t] * x[p][i][c]; p = side * BH + slice
constexpr int kDzStep = 16;

template <typename T, typename LT>
__global__ void __launch_bounds__(256)
bwd_dz_part_kernel(const LT *__restrict__ dC, const T *__restrict__ q, const T *__restrict__ k, LT *__restrict__ part,
                   int BH, int n, int d, int r, int chunks, int rows_per_chunk)
{
    __shared__ LT Ds[kDzStep][kGPad];
    __shared__ LT Xs[kDzStep][kGPad];
    const int p = blockIdx.z, side = p / BH, s = p % BH;
    const int cblks = (d + kGT - 1) / kGT;
    const int t0 = (blockIdx.y / cblks) * kGT, c0 = (blockIdx.y % cblks) * kGT;
    const int chunk = blockIdx.x;
    const int row0 = chunk * rows_per_chunk, row1 = min(row0 + rows_per_chunk, n);
    const LT *Db = dC + (size_t)p * n * r;
    const T *Xb = (side ? k : q) + (size_t)s * n * d;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    LT acc[4][4] = {};
    for (int i0 = row0; i0 < row1; i0 += kDzStep) {
#pragma unroll
        for (int rep = 0; rep < 4; ++rep) {
            const int idx = threadIdx.x + rep * 256;
            const int ii = idx / kGT, cc = idx % kGT;
            const int i = i0 + ii;
            LT dv = (LT)0, xv = (LT)0;
            if (i < row1 && t0 + cc < r) dv = Db[(size_t)i * r + t0 + cc];
            if (i < row1 && c0 + cc < d) xv = ld_as<LT>(Xb[(size_t)i * d + c0 + cc]);
            Ds[ii][cc] = dv;
            Xs[ii][cc] = xv;
        }
        __syncthreads();
#pragma unroll
        for (int ii = 0; ii < kDzStep; ++ii) {
            LT dr[4], xr[4];
#pragma unroll
            for (int x = 0; x < 4; ++x) { dr[x] = Ds[ii][ty * 4 + x]; xr[x] = Xs[ii][tx * 4 + x]; }
#pragma unroll
            for (int x = 0; x < 4; ++x)
#pragma unroll
                for (int y = 0; y < 4; ++y) acc[x][y] = fma(dr[x], xr[y], acc[x][y]);
        }
        __syncthreads();
    }
    LT *pp = part + ((size_t)p * chunks + chunk) * r * d;
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        const int t = t0 + ty * 4 + x;
        if (t >= r) continue;
#pragma unroll
        for (int y = 0; y < 4; ++y) {
            const int c = c0 + tx * 4 + y;
            if (c < d && LOT_CHECK((size_t)t * d + c < (size_t)r * d)) pp[(size_t)t * d + c] = acc[x][y];
        }
    }
}

// dz[h][t][c] = sum over batch, side and chunk (in that fixed order) of the partials; dbeta likewise
template <typename LT>
__global__ void bwd_dz_merge_kernel(const LT *__restrict__ part, const float *__restrict__ dbeta_direct,
                                    const LT *__restrict__ dbeta_acc, float *__restrict__ dz, float *__restrict__ dbeta,
                                    int B, int H, int d, int r, int chunks)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t per_head = (size_t)r * d;
    const int BH = B * H;
    if (idx < (size_t)H * per_head) {
        const int h = (int)(idx / per_head);
        const size_t e = idx % per_head;
        LT sum = (LT)0;
        for (int b = 0; b < B; ++b)
            for (int side = 0; side < 2; ++side) {
                const size_t p = (size_t)side * BH + (size_t)b * H + h;
                for (int c = 0; c < chunks; ++c) sum += part[(p * chunks + c) * per_head + e];
            }
        dz[idx] = (float)sum;
    }
    if (idx < (size_t)H * r) {
        const int h = (int)(idx / r), t = (int)(idx % r);
        LT sum = (LT)0;
        for (int b = 0; b < B; ++b) {
            const size_t s = (size_t)b * H + h;
            sum += (LT)dbeta_direct[s * r + t];
            sum += dbeta_acc[s * r + t];
            sum += dbeta_acc[((size_t)BH + s) * r + t];
        }
        dbeta[idx] = (float)sum;
    }
}

} // namespace

cudaError_t launch_bwd_rows(const BwdRowArgs &a, bool close, bool wide, cudaStream_t st)
{
    return wide ? launch_rows_r<double>(a, close, st) : launch_rows_r<float>(a, close, st);
}

cudaError_t launch_gemm_nt(const void *A, int a_type, const float *Bm, bool per_head, void *out, int out_type,
                           int S, int H, int n, int K, int J, bool acc_double, cudaStream_t st)
{
    if (a_type == 0)
        return acc_double ? launch_gemm_out<float, double>(A, Bm, per_head, out, out_type, S, H, n, K, J, st)
                          : launch_gemm_out<float, float>(A, Bm, per_head, out, out_type, S, H, n, K, J, st);
    if (a_type == 1) return launch_gemm_out<__nv_bfloat16, float>(A, Bm, per_head, out, out_type, S, H, n, K, J, st);
    return launch_gemm_out<double, double>(A, Bm, per_head, out, out_type, S, H, n, K, J, st);
}

cudaError_t launch_bwd_w_fix(const float *Xw, const float *Wp, const int32_t *key_len, float *dWm, float *dbeta_direct,
                             int B, int H, int n, int d, int r, cudaStream_t st)
{
    bwd_w_fix_kernel<<<B * H, 256, 0, st>>>(Xw, Wp, key_len, dWm, dbeta_direct, H, n, d, r);
    return cudaGetLastError();
}

cudaError_t launch_transpose_z(const float *z, float *zt, int H, int r, int d, cudaStream_t st)
{
    const size_t total = (size_t)H * r * d;
    transpose_z_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(z, zt, r, d, total);
    return cudaGetLastError();
}

int bwd_dz_chunks(int BH, int n, int r, int d)
{
    const int tiles = ((r + kGT - 1) / kGT) * ((d + kGT - 1) / kGT) * 2 * BH;
    int want = (592 + tiles - 1) / tiles;
    const int most = (n + 255) / 256;
    if (want > most) want = most;
    return want < 1 ? 1 : want;
}

cudaError_t launch_bwd_dz(const void *dC, const void *q, const void *k, int dtype, void *part, const float *dbeta_direct,
                          const void *dbeta_acc, float *dz, float *dbeta, int B, int H, int n, int d, int r, int chunks,
                          bool wide, cudaStream_t st)
{
    const int BH = B * H;
    const int rows = (n + chunks - 1) / chunks;
    dim3 grid(chunks, ((r + kGT - 1) / kGT) * ((d + kGT - 1) / kGT), 2 * BH);
    if (dtype == 0)
        bwd_dz_part_kernel<float, double><<<grid, 256, 0, st>>>(static_cast<const double *>(dC), static_cast<const float *>(q),
                                                               static_cast<const float *>(k), static_cast<double *>(part),
                                                               BH, n, d, r, chunks, rows);
    else
        bwd_dz_part_kernel<__nv_bfloat16, float><<<grid, 256, 0, st>>>(
            static_cast<const float *>(dC), static_cast<const __nv_bfloat16 *>(q), static_cast<const __nv_bfloat16 *>(k),
            static_cast<float *>(part), BH, n, d, r, chunks, rows);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const size_t work = (size_t)H * r * d;
    const unsigned blocks = (unsigned)((work + 255) / 256);
    if (wide)
        bwd_dz_merge_kernel<double><<<blocks, 256, 0, st>>>(static_cast<const double *>(part), dbeta_direct,
                                                           static_cast<const double *>(dbeta_acc), dz, dbeta, B, H, d, r, chunks);
    else
        bwd_dz_merge_kernel<float><<<blocks, 256, 0, st>>>(static_cast<const float *>(part), dbeta_direct,
                                                          static_cast<const float *>(dbeta_acc), dz, dbeta, B, H, d, r, chunks);
    return cudaGetLastError();
}

LOT_DEBUG_FLAG_READER(backward_debug_flag)

} // namespace lot
