// Internal launch interface between the C ABI (lot_api.cu) and the kernels.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace lot {

// One Sinkhorn pass over a set of independent problems.  Problem p covers the slice
// s = p % (B*H) (batch s / H, head s % H); problems p >= len_from take their valid length
// from len[batch], the others use n.
// Arithmetic modes: which types the similarity matrix is stored in and the logits, pivot
// potentials G and row log-sum-exps M are assembled in.
enum { kModeF32 = 0,          // cost float, logits float            (bf16 tensors)
       kModeCostF32Wide = 1,  // cost float, logits/G/M double       (lot_sinkhorn)
       kModeWide = 2 };       // cost double, logits/G/M double      (float32 tensors)

struct PassArgs {
    const void *cost;    // [nprob][n][r] similarity matrices (float or double, see mode)
    const float *beta;   // [H][r]
    const int32_t *len;  // [B] or nullptr
    int len_from;
    const float *mass;   // [nprob][n] token weights (>= 0; zero takes the token out of the problem), or nullptr:
                         // uniform over the valid tokens
    void *G;             // [nprob][r] pivot potentials, base-2 log units (in/out; float or double)
    void *G_next;        // not nullptr: the updated potentials go here and G stays as it was (a kept history)
    float *part;         // [nprob][chunks][r][2] per-block column pairs (kappa, S)
    unsigned *counter;   // [nprob] arrival tickets, zero on entry and on exit
    void *M;             // final pass: [nprob][n] row log-sum-exp (base 2), +inf for massless rows
    float *g_out;        // final pass, optional: [nprob][r] potentials in natural-log units
    float *f_out;        // final pass, optional: [nprob][n]
    float *plan_out;     // final pass, optional: [nprob][n][r]
    int *status;
    int nprob, B, H, n, r;
    int chunks, rows_per_chunk;
    int mode;
    double scale_d;      // log2(e)/eps
    float eps_ln2;       // eps*ln(2)
};

struct ApplyArgs {
    const void *cost1;   // [BH][n][r] query-side similarities (float: bf16 tensors, double: float32)
    const void *cost2;   // [BH][n][r] key-side similarities
    const void *G1, *G2;   // [BH][r]   same type as the similarities
    const void *M1, *M2;   // [BH][n]
    const float *beta;     // [H][r]
    const int32_t *key_len;
    const float *mass2;    // [BH][nk] key weights or nullptr (uniform over the valid keys)
    const void *v;         // [BH][nk][d]
    void *out;             // [BH][n][d]
    float *wpart;          // [BH][chunks][r][d]
    float *Wp;             // [BH][r][d]  W' = Diag(beta)^-1 Gamma2 V
    unsigned *counter;     // [BH * tblks * cblks]
    int B, H, n, d, r;     // n: queries per slice
    int nk;                // keys per slice
    int chunks, rows_per_chunk;
    double scale_d;
};

// bounds-check build only (0 otherwise): reads and clears the file's record of skipped out-of-range accesses
int kernels_debug_flag();
int backward_debug_flag();

int pass_chunks(int nprob, int n);
int apply_chunks(int BH, int n, int r, int d);

cudaError_t launch_cost(const void *x, const float *z, int dtype, int BH, int H, int n, int d, int r,
                        void *cost, bool wide, cudaStream_t st);
cudaError_t launch_sinkhorn_pass(const PassArgs &a, bool final_pass, cudaStream_t st);
cudaError_t launch_apply_w(const ApplyArgs &a, int dtype, cudaStream_t st);
cudaError_t launch_apply_out(const ApplyArgs &a, int dtype, cudaStream_t st);
// starting potentials: G = g_in * scale (float or double per `wide`), zeros when g_in == nullptr
cudaError_t launch_g_init(const float *g_in, void *G, size_t count, double scale, bool wide, cudaStream_t st);
// weights of the [CLS] treatment, Eq. (5): a = (0, 1/(nq-1), ...), b = (0, 1/(kv-1), ... up to the key length, 0 ...)
cudaError_t launch_cls_marginals(float *a, float *b, const int32_t *key_len, int B, int H, int nq, int nk, int *status,
                                 cudaStream_t st);
// row 0 of every slice: softmax_j(tau <q_0, k_j>) over the valid keys, applied to v; scores: [BH][nk] scratch
cudaError_t launch_cls_row(const void *q, const void *k, const void *v, const int32_t *key_len, int dtype, int B, int H,
                           int nq, int nk, int d, float tau, float *scores, void *out, cudaStream_t st);

// ---- backward of the general path (lot_backward.cu) ----
// One reverse step over a set of Sinkhorn problems (same problem numbering as PassArgs).  close: the closing token
// update and the plan read-out; otherwise one (token update, pivot update) pair of the unrolled iteration.
struct BwdRowArgs {
    const void *cost;    // [nprob][n][r] similarities (float or double per `wide`)
    void *dC;            // [nprob][n][r] same type.  close: in = gradient with respect to the row-stochastic plan,
                         // out = gradient with respect to the similarities; otherwise updated in place
    const void *Ga;      // [nprob][r] potentials the rows are normalised with (base-2 units)
    const void *Gb;      // [nprob][r] potentials after the pivot update being reversed (not close)
    void *gamma;         // [nprob][r] gradient with respect to the potentials in natural units: written by close,
                         // read and replaced otherwise
    void *dbeta_acc;     // [nprob][r] accumulates eps * gamma / beta over the reversed pivot updates
    const float *beta;   // [H][r]
    const int32_t *len;  // [B] or nullptr
    int len_from;
    void *part;          // [nprob][chunks][r] per-block column sums
    unsigned *counter;   // [nprob] arrival tickets, zero on entry and on exit
    int nprob, B, H, n, r;
    int chunks, rows_per_chunk;
    double scale_d;      // log2(e)/eps
    double eps;
};
cudaError_t launch_bwd_rows(const BwdRowArgs &a, bool close, bool wide, cudaStream_t st);
// out[s][i][j] = sum_k A[s][i][k] * Bm[(per_head ? s % H : s)][j][k]   (A: n x K, Bm: J x K, out: n x J)
// a_type / out_type: 0 float, 1 bf16, 2 double; Bm is float
cudaError_t launch_gemm_nt(const void *A, int a_type, const float *Bm, bool per_head, void *out, int out_type,
                           int S, int H, int n, int K, int J, bool acc_double, cudaStream_t st);
// Xw = (apply_w output of the query side on dout) -> dWm = Xw * n / nvalid_b (zero without keys),
// dbeta_direct[s][t] = -n * sum_c Xw[s][t][c] * Wp[s][t][c]
cudaError_t launch_bwd_w_fix(const float *Xw, const float *Wp, const int32_t *key_len, float *dWm, float *dbeta_direct,
                             int B, int H, int n, int d, int r, cudaStream_t st);
// zt[h][c][t] = z[h][t][c]
cudaError_t launch_transpose_z(const float *z, float *zt, int H, int r, int d, cudaStream_t st);
int bwd_dz_chunks(int BH, int n, int r, int d);
// dz[h][t][c] = sum over b, side, rows of dC[side][b,h][i][t] * x_side[b,h][i][c];  dbeta[h][t] = sum over b of
// dbeta_direct + both sides' dbeta_acc.  part: [2*BH][chunks][r][d] floats or doubles per `wide`
cudaError_t launch_bwd_dz(const void *dC, const void *q, const void *k, int dtype, void *part, const float *dbeta_direct,
                          const void *dbeta_acc, float *dz, float *dbeta, int B, int H, int n, int d, int r, int chunks,
                          bool wide, cudaStream_t st);

// ---- fused tensor-core path (lot_fused.cu): bf16 tensors, d = 64, r <= 64 ----
struct FusedLayout {
    size_t status, G, epoch, iter, robust, wflag, gnat, decision, head_end, kt, zprep, part, wpart, wpart2, total;
};
bool fused_supported(int dtype, int d, int r);
void fused_geometry(int B, int H, int n, int *q, int *ctas, int *maxslots, int *cps);
FusedLayout fused_layout(int B, int H, int n, int d, int r);
// redo != nullptr: both kernels return at once unless *redo == redo_tag (the call behind a resident launch)
cudaError_t fused_attention(const void *q, const void *k, const void *v, const float *z, const float *beta,
                            const int32_t *key_len, int B, int H, int n, int d, int r, float eps, int iters,
                            void *out, float *g1_out, float *g2_out, void *ws, const unsigned *redo, unsigned redo_tag,
                            cudaStream_t st);
int fused_launches(int B, int H, int n, int r, int iters);
// true when the apply stages of a streamed call run as the two kernels of lot_apply.cu
bool fused_ext_apply(int B, int H, int n, int r, int iters);

// ---- resident tensor-core path (lot_resident.cu): bf16 tensors, d = 64, r <= 64, tiles fit one SM's TMEM + shared memory ----
struct ResidentGeom {
    bool ok;
    int ctas, whole, wave_slices, maxslots, TPS, NT;
};
struct ResidentLayout {
    size_t status, part, wflag, wpart, spill, total;
};
int device_sm_count();                       // SM count of the current device (cached per device)
ResidentGeom resident_geometry(int dtype, int B, int H, int n, int d, int r);
ResidentLayout resident_layout(int B, int H, int n, int d, int r);
cudaError_t resident_attention(const void *q, const void *k, const void *v, const float *z, const float *beta,
                               const int32_t *key_len, int B, int H, int n, int d, int r, float eps, int iters,
                               void *out, float *g1_out, float *g2_out, void *ws, unsigned *tag_out, cudaStream_t st);
void resident_debug(int what, long long value);

// ---- slice path (lot_slice.cu): bf16 tensors, d = 64, r <= 64, short sequences; one thread block per slice ----
bool slice_supported(int dtype, int n, int d, int r);
cudaError_t slice_attention(const void *q, const void *k, const void *v, const float *z, const float *beta,
                            const int32_t *key_len, int B, int H, int n, int r, float eps, int iters, void *out,
                            float *g1_out, float *g2_out, int *status, cudaStream_t st);

// ---- apply stages from the stored Gibbs kernel (lot_apply.cu), behind the streamed Sinkhorn kernel ----
size_t stored_apply_wpart_bytes(int B, int H, int n);
cudaError_t stored_apply(const void *kt, int npad, const float *G, const float *beta, const int32_t *key_len, const int *decision,
                         const void *v, void *out, float *wpart, int *status, int B, int H, int n, int r, cudaStream_t st);   // test hooks: 1 = block that skips its first publish (one call), 2 = wait limit in ns

} // namespace lot
