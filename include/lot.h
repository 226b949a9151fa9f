/*
 * lot.h -- C ABI of liblot: the forward hot path of LOTFormer attention
 * (arXiv 2509.23436, Section "Method") as hand-written CUDA for sm_100a.
 *
 * For each (batch b, head h) slice, with queries/keys/values q,k,v [n,d], pivot
 * locations z_h [r,d] and pivot masses beta_h [r] (> 0, summing to 1):
 *
 *   costs        C1[i,t] = <q_i, z_t>,  C2[j,t] = <k_j, z_t>            (Section "Method", the
 *                unnumbered display defining C^(1), C^(2) before Eq. (1); no 1/sqrt(d) factor)
 *   two solves   Gamma1 in U(beta, a), Gamma2 in U(beta, b), the entropic problems
 *                Eq. (1)-(2), in the Sinkhorn scaling form Diag(u) exp(C/eps) Diag(v)
 *   composition  Gamma = Gamma1^T Diag(beta)^-1 Gamma2 (Eq. (3)), never formed
 *   output       out = A V = Gamma1^T (Diag(beta)^-1 (Gamma2 V)) with A = Gamma / a the
 *                row-stochastic scaling (A = n Gamma for uniform marginals; Eq. (4) and
 *                the paragraph "Rank and complexity")
 *
 * The Sinkhorn map that every entry point computes (T = iters), per side with token
 * marginal m (a for queries, b for keys):
 *       g <- 0;  repeat T times:
 *           f_i = eps (log m_i - LSE_t((C_it + g_t)/eps))
 *           g_t = eps (log beta_t - LSE_i((C_it + f_i)/eps))
 *       one closing update of f;  P_it = exp((C_it + f_i + g_t)/eps).
 * Marginals: a_i = 1/n.  b_j = 1/n, or with a key length L_b: b_j = 1/L_b for j < L_b
 * and tokens j >= L_b carry no mass (they take no part in the key-side problem).
 *
 * General conventions
 *   - Every pointer is a DEVICE pointer owned by the caller unless its comment says
 *     "host".  Tensors are dense row-major, last index fastest, 16-byte aligned.
 *   - q,k,v,out: [B,H,n,d] in `dtype` (LOT_F32 or LOT_BF16).  z: [H,r,d] float32,
 *     beta: [H,r] float32, per head and shared over the batch.  key_len: [B] int32.
 *   - Supported: B,H >= 1, n >= 1 (n*r, n*d < 2^31), 1 <= r <= 256, 8 <= d <= 256 with
 *     d % 8 == 0, eps > 0 finite, iters >= 0.  B == 0 or n == 0 is a no-op returning
 *     LOT_OK.  Anything else returns LOT_ERR_INVALID_ARG / LOT_ERR_UNSUPPORTED_SHAPE
 *     before any launch.
 *   - Calls are asynchronous on `stream` (NULL = the default stream), never
 *     synchronise the host, never abort.  The return value reports argument and launch
 *     errors only.  Conditions found on the device (a non-finite potential, an empty
 *     key set) are OR-ed into a status word at the start of the workspace; read it
 *     with lot_device_status after the work has run.
 *   - Scratch memory comes from the caller (`ws`, `ws_bytes`; size from the matching
 *     *_workspace_bytes call, 256-byte aligned).  The library keeps no state between
 *     calls except inside lot_attention_fwd (see there).  Two calls may run
 *     concurrently only on different workspaces.
 *   - Results are deterministic: reductions across thread blocks are summed in a
 *     fixed order, no floating-point atomics.
 */
#ifndef LOT_H_
#define LOT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st *lot_stream_t; /* a cudaStream_t */

#if defined(__GNUC__)
#define LOT_API __attribute__((visibility("default")))
#else
#define LOT_API
#endif

enum lot_status {
    LOT_OK = 0,
    LOT_ERR_INVALID_ARG = 1,       /* null pointer, misaligned pointer, eps <= 0, iters < 0, bad dtype */
    LOT_ERR_UNSUPPORTED_SHAPE = 2, /* a size outside the supported set above */
    LOT_ERR_WORKSPACE = 3,         /* ws null/misaligned or ws_bytes too small */
    LOT_ERR_CUDA = 4               /* a CUDA runtime call or launch failed (cudaGetLastError consumed) */
};

enum lot_dtype { LOT_F32 = 0, LOT_BF16 = 1 };

/* bits of the device status word */
enum lot_device_flag {
    LOT_DEV_NONFINITE = 1, /* a pivot potential became inf/nan (e.g. beta_t <= 0) */
    LOT_DEV_EMPTY = 2,     /* a key_len entry was <= 0: that slice has no key mass; its output is zeros */
    LOT_DEV_TIMEOUT = 4,   /* a bounded device-side wait gave up; results of the call are invalid */
    LOT_DEV_BOUNDS = 16,   /* bounds-check build only (compiled with -DLOT_DEBUG, lot_version() = 100100): an index of a
                              general-path or backward kernel fell outside its buffer; the access was skipped */
    LOT_DEV_RECOMPUTED = 8 /* information only: the resident path could not represent the problem (see lot_path)
                              and the streamed kernels recomputed the call; the results are valid */
};

/* Library version: major*10000 + minor*100 + patch. */
LOT_API int lot_version(void);

/* Static string for a lot_status value (never NULL). */
LOT_API const char *lot_status_string(int status);

/*
 * lot_cost -- the similarity matrices of Section "Method": cost[b,h,i,t] = <x[b,h,i,:], z[h,t,:]>.
 *   x     [B,H,n,d] in `dtype`;  z [H,r,d] float32;  cost [B,H,n,r] float32 (out).
 * bf16 inputs are used exactly and accumulate in float32; float32 inputs accumulate in float64
 * and the result is rounded to float32 once.  Needs no workspace.
 */
LOT_API int lot_cost(const void *x, const float *z, int dtype, int B, int H, int n, int d, int r,
             float *cost, lot_stream_t stream);

/* Scratch bytes lot_sinkhorn needs for these sizes. */
LOT_API size_t lot_sinkhorn_workspace_bytes(int B, int H, int n, int r);

/*
 * lot_sinkhorn -- one entropic solve, Eq. (1) or (2), from a materialised similarity matrix.
 *   cost [B,H,n,r] float32;  beta [H,r];  len [B] int32 or NULL (tokens i >= len[b] carry
 *   no mass and m_i = 1/len[b]; NULL means m_i = 1/n).
 * Outputs (each may be NULL except g):
 *   g    [B,H,r]   pivot potentials after T pivot updates (natural-log units, as above)
 *   f    [B,H,n]   token potentials after the closing update (-inf for massless tokens)
 *   plan [B,H,n,r] P_it (zero rows for massless tokens)
 */
LOT_API int lot_sinkhorn(const float *cost, const float *beta, const int32_t *len,
                 int B, int H, int n, int r, float eps, int iters,
                 float *g, float *f, float *plan,
                 void *ws, size_t ws_bytes, lot_stream_t stream);

/*
 * lot_sinkhorn_static -- lot_sinkhorn for callers that must not allocate device memory.
 * (The paper has no counterpart: this is a packaging variant of the same solve.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a framework whose
 * allocator owns all device memory and forbids raw allocations, in a real-time or
 * latency-critical loop where an allocation (which may synchronise the device) is not
 * acceptable, or in a plug-in that is handed tensors but no allocator.  Such callers cannot
 * produce the workspace lot_sinkhorn asks for.
 *
 * Here the scratch is a fixed array of LOT_STATIC_SCRATCH_BYTES that lives inside the library
 * image: every device that loads liblot holds that much memory until the process exits,
 * whether or not this function is ever called.  The call itself allocates nothing and calls
 * no allocating routine; the caller still provides every input and output buffer.
 *
 *   Arguments cost, beta, len, B, H, n, r, eps, iters, g, f, plan, stream: as lot_sinkhorn.
 *   status_out: device int32 or NULL; receives the device status word of this call.
 *
 * Limits and rules
 *   - lot_sinkhorn_workspace_bytes(B,H,n,r) must not exceed LOT_STATIC_SCRATCH_BYTES;
 *     larger problems return LOT_ERR_WORKSPACE before anything is launched.
 *   - The first call on each device looks up the device address of the array (with that
 *     device current).  Make that first call outside any stream capture.
 *   - All calls on a device share the one array, which still holds what the previous call
 *     left; the part that must start at zero is cleared at the start of every call.  Two
 *     calls whose work overlaps on the GPU (different streams, no ordering) race on it and
 *     give undefined results: order them.
 */
#define LOT_STATIC_SCRATCH_BYTES (4u << 20)
LOT_API int lot_sinkhorn_static(const float *cost, const float *beta, const int32_t *len,
                        int B, int H, int n, int r, float eps, int iters,
                        float *g, float *f, float *plan, int32_t *status_out,
                        lot_stream_t stream);

/* Scratch bytes lot_attention_fwd_ex needs for these sizes. */
LOT_API size_t lot_workspace_bytes(int B, int H, int n, int d, int r, int dtype);

/*
 * lot_path -- which implementation one lot_attention_fwd_ex call with these parameters takes (host
 * arithmetic only):
 *   0  the general path: a cost kernel per side, one kernel per Sinkhorn pass, two apply kernels.
 *   1  the streamed tensor-core path (bf16 tensors, d = 64, r <= 64): one persistent kernel for all
 *      passes, launched cooperatively (it needs as many free SMs as it has thread blocks, at most
 *      one per SM), plus a small pivot preparation.  With 32 < r <= 64 its first pass keeps the
 *      stabilised Gibbs kernel exp(C/eps - rowmax) of the scaling form of Eq. (1)-(2) as bf16 in the
 *      workspace and the later passes stream that copy back.
 *   2  the resident tensor-core path (same tensors; taken for r <= 32 when every thread block can
 *      hold whole sequences, up to 1792 tokens, and all of its share at once): one persistent kernel in
 *      which that bf16 kernel never leaves the SM (tensor memory and shared memory) between the
 *      iterations.  A problem it cannot represent (potentials spread over more than 96 binades, a
 *      column mass below 2^-80) is recomputed by the streamed kernels, which are launched behind it
 *      and return at once otherwise (device flag LOT_DEV_RECOMPUTED).  It can run many more shapes
 *      (lot_debug_hook what = 4), but measured no faster there.
 *   3  the slice path (same tensors; n <= 512 and 16 ceil(n/16) x (r padded to 16, 32 or 64) <= 16384): one
 *      thread block per (batch, head) slice keeps a side's logits in float32 registers for all iterations
 *      (warp-level tensor-core products, shared memory for K, V, Q and the r x d intermediate); nothing
 *      crosses thread blocks, no workspace beyond the status word.  Taken wherever it can run.
 * On paths 1 and 2 the potentials agree with an exact float evaluation to about 1e-4 and the output
 * to the bf16 rounding of `out`.
 */
LOT_API int lot_path(int dtype, int B, int H, int n, int d, int r, int iters);

/*
 * lot_launch_count -- how many kernels of this library one lot_attention_fwd_ex call with these
 * parameters launches (host arithmetic only; 0 for iters < 0).
 */
LOT_API int lot_launch_count(int dtype, int B, int H, int n, int d, int r, int iters);

/*
 * lot_debug_hook -- switches for the library's own tests; not part of the method.
 *   what = 1: the thread block `value` of the next resident-path launch never publishes its first
 *             column partial, so the bounded waits of the blocks that share its slice run out and the
 *             call ends with LOT_DEV_TIMEOUT (one call only; -1 = none).
 *   what = 2: limit of every device-side wait of the resident path in nanoseconds (0 = default, 1 s).
 *   what = 3: device address of a trace buffer (8002 64-bit words, zeroed by the caller) into which thread block 0 of
 *             the resident path logs (event code, global timer) pairs, or 0 to stop; for profiling.
 *   what = 4: 1 or 2 makes lot_attention_fwd_ex take tensor-core path 1 or 2 of lot_path wherever that path can run
 *             at all (the default choice is by measured speed), 0 the general path; -1 restores the default.
 *             lot_path, lot_launch_count and lot_workspace_bytes follow the switch.
 * Returns LOT_ERR_INVALID_ARG for any other `what`.
 */
LOT_API int lot_debug_hook(int what, long long value);

/*
 * lot_attention_fwd_ex -- the whole forward path, Eq. (1)-(4): costs, both solves, apply.
 *   q,k,v,out [B,H,n,d] in `dtype`;  z [H,r,d];  beta [H,r];  key_len [B] or NULL.
 *   g1_out, g2_out [B,H,r] float32 or NULL: the final pivot potentials of the query-side
 *   and key-side solves (natural-log units).
 * out[b,h,i,:] = sum_t softmax_t((C1_it + g1_t)/eps) * W'_t,  W' = Diag(beta)^-1 Gamma2 V.
 * Padded query rows (there is no query mask) produce ordinary finite outputs.
 */
LOT_API int lot_attention_fwd_ex(const void *q, const void *k, const void *v,
                         const float *z, const float *beta, const int32_t *key_len,
                         int dtype, int B, int H, int n, int d, int r, float eps, int iters,
                         void *out, float *g1_out, float *g2_out,
                         void *ws, size_t ws_bytes, lot_stream_t stream);

/*
 * lot_attention_bwd -- gradients of the forward path (Section "Learning": the pivots, their masses and the
 * projections are trained by back-propagating through the two shared-eps Sinkhorn problems, Eq. (1)-(2), and the
 * glued composition, Eq. (3)-(4)).  What is differentiated is exactly the map lot_attention_fwd_ex computes: the
 * unrolled iteration (start at zero, `iters` times token update then pivot update, one closing token update),
 * not the fixed point.  Given dout = d(loss)/d(out) it returns d(loss)/d(q, k, v, z, beta).
 *   q,k,v,dout,dq,dk,dv [B,H,n,d] in `dtype` (device);  z, dz [H,r,d];  beta, dbeta [H,r] float32 (device);
 *   key_len [B] int32 or NULL as in the forward (rows of dk, dv beyond the length are zero).
 *   beta is treated as r free positive numbers per head (no simplex constraint: a softmax parametrisation is the
 *   caller's chain rule); dz and dbeta are summed over the batch.
 * The forward is recomputed (materialised similarities, general path arithmetic: float32 for bf16 tensors,
 * float64 for float32 tensors); only the pivot potentials of every iteration are kept.  2*iters + 15 kernel launches.
 * ws: lot_bwd_workspace_bytes(...) bytes of device scratch, 256-byte aligned, owned by the caller; the device
 * status word of the recomputed forward sits at its start (lot_device_status).
 * Errors as lot_attention_fwd_ex.  B == 0 or n == 0: dz and dbeta are zero-filled, nothing else is touched.
 */
LOT_API size_t lot_bwd_workspace_bytes(int B, int H, int n, int d, int r, int dtype, int iters);
LOT_API int lot_attention_bwd(const void *q, const void *k, const void *v, const float *z, const float *beta,
                      const int32_t *key_len, const void *dout,
                      int dtype, int B, int H, int n, int d, int r, float eps, int iters,
                      void *dq, void *dk, void *dv, float *dz, float *dbeta,
                      void *ws, size_t ws_bytes, lot_stream_t stream);

/* Scratch bytes lot_attention_fwd_var needs for these sizes. */
LOT_API size_t lot_var_workspace_bytes(int B, int H, int nq, int nk, int d, int r, int dtype);

/*
 * lot_attention_fwd_var -- the forward path with the variations the paper uses around it:
 *   cross-attention   nq queries, nk keys and values per slice (Appendix "Bidirectional scope", closing
 *                     paragraph): q, out [B,H,nq,d];  k, v [B,H,nk,d].
 *   token weights     a [B,H,nq], b [B,H,nk] float32 or NULL: the weights p^1, p^2 of the empirical measures
 *                     (Section "Empirical measures and pivot"; >= 0, each slice summing to 1, trusted).  NULL
 *                     means uniform, over the first key_len[b] keys on the key side when key_len is given.  A
 *                     token of weight zero takes no part in its transport problem; a query of weight zero gets
 *                     an all-zero output row.  out = Diag(1/a) Gamma1^T Diag(1/beta) Gamma2 V.
 *   warm start        g1_in, g2_in [B,H,r] float32 or NULL: pivot potentials (natural-log units, as g1_out and
 *                     g2_out give them) the two iterations start from instead of zero.  T1 iterations followed
 *                     by T2 more from the exported potentials are T1 + T2 iterations.
 *   [CLS] row         cls = 1 (Eq. (5)): token 0 is the class token.  Its output row is the plain softmax
 *                     aggregate sum_j softmax_j(cls_tau <q_0, k_j>) v_j over all valid keys (cls_tau > 0 is the
 *                     temperature the paper calls beta in Eq. (5)); every other row follows the transport rule
 *                     among the remaining tokens (queries 1.., valid keys 1.., uniform weights).  a and b must
 *                     be NULL; nq, nk >= 2 are needed for the transport part (else LOT_DEV_EMPTY is flagged).
 * Everything else as lot_attention_fwd_ex.  This entry point runs on the general path for every shape.
 */
LOT_API int lot_attention_fwd_var(const void *q, const void *k, const void *v, const float *z, const float *beta,
                          const float *a, const float *b, const int32_t *key_len,
                          const float *g1_in, const float *g2_in, int cls, float cls_tau,
                          int dtype, int B, int H, int nq, int nk, int d, int r, float eps, int iters,
                          void *out, float *g1_out, float *g2_out,
                          void *ws, size_t ws_bytes, lot_stream_t stream);

/*
 * lot_attention_fwd -- the same path for float32 tensors, uniform marginals, with scratch the
 * library manages itself: one buffer per device, grown with cudaMalloc when a call needs
 * more than any earlier one (that call synchronises the device once; later calls of the
 * same or smaller size allocate nothing).  Calls on one device are serialised by the
 * caller (they share that buffer).  Arguments as lot_attention_fwd_ex.
 */
LOT_API int lot_attention_fwd(const float *q, const float *k, const float *v,
                      const float *z, const float *beta,
                      int B, int H, int n, int d, int r, float eps, int iters,
                      float *out, lot_stream_t stream);

/*
 * lot_device_status -- copy the device status word of workspace `ws` (as passed to
 * lot_sinkhorn / lot_attention_fwd_ex; NULL = the library-managed buffer of the current
 * device) to *status (host), after synchronising `stream`.  0 means nothing was flagged.
 */
LOT_API int lot_device_status(const void *ws, lot_stream_t stream, int *status /* host */);

#ifdef __cplusplus
}
#endif
#endif /* LOT_H_ */
