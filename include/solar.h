/*
 * solar.h -- C ABI of the B200 (sm_100a) SVD-Attention forward pass.
 *
 * The operation is the one defined in Section 4.1 of the SOLAR paper
 * (arxiv 2603.02561): every user's history matrix H (N x d, the shared
 * key-value matrix) is replaced by its rank-r truncated SVD (Eq. 9); the left
 * factor U cancels (Eq. 10), and M candidate queries attend over the r
 * "factor tokens" sigma_i v_i^T projected by W_K / W_V (Eq. 11, Eq. 12), with
 * the softmax kept (over the r tokens).
 *
 * Conventions shared by every entry point
 *   - All tensors are dense, row-major, batch-major; "dt" is the STORAGE type of
 *     H, C, W_Q, W_K, W_V, O and US.  Arithmetic accumulates in fp32 (or wider).
 *   - Every pointer is a DEVICE pointer owned by the caller, 16-byte aligned,
 *     valid until the work queued on `stream` has finished.  The library
 *     allocates nothing and keeps no state between calls.  Inputs may be written
 *     by work queued earlier on the same stream: the first kernel of every call
 *     waits for that work to complete before it reads any caller buffer.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL =
 *     the legacy default stream) and never synchronise.
 *   - Errors the host can see (bad sizes, NULL or misaligned pointers, a
 *     workspace that is too small) are returned BEFORE anything is launched.
 *     Conditions only the device can see (Jacobi sweeps exhausted, non-finite
 *     input) are written to info[] and never trap; such a user's outputs are
 *     NaN-filled.
 *   - Supported: d in {32, 64, 128}; 1 <= r <= min(d, N, 64); N >= 1; M >= 0;
 *     B >= 0 (B == 0 or M == 0 makes the call a no-op returning SOLAR_OK).
 *     Anything else returns SOLAR_ERR_UNSUPPORTED or SOLAR_ERR_INVALID_ARG.
 *   - Two calls that share a workspace must not overlap on the GPU.
 */
#ifndef SOLAR_H_
#define SOLAR_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SOLAR_OK = 0,
  SOLAR_ERR_INVALID_ARG = 1, /* negative size, NULL / misaligned pointer, r out of range */
  SOLAR_ERR_UNSUPPORTED = 2, /* d not in {32,64,128}, r > 64, unknown dtype or flag     */
  SOLAR_ERR_WORKSPACE = 3,   /* workspace NULL or smaller than solar_workspace_bytes()   */
  SOLAR_ERR_CUDA = 4         /* a CUDA runtime call or a launch failed                  */
} solar_status_t;

typedef enum { SOLAR_F32 = 0, SOLAR_BF16 = 1 } solar_dtype_t;

/* flags of solar_svd_attention_fwd */
enum {
  SOLAR_FLAG_NO_SOFTMAX = 1 /* "SVD-Attn without Softmax" (ablation row of Table 4):
                               O = scale * Query * Key_r^T * Value_r */
};

/* bits of info[b] written by the factorization */
enum {
  SOLAR_INFO_NOT_CONVERGED = 1, /* sweep cap reached before every rotation became negligible */
  SOLAR_INFO_NONFINITE = 2,     /* H_b^T H_b contains NaN or Inf; s, V of this user are NaN  */
  SOLAR_INFO_NOT_CERTIFIED = 4, /* only with SOLAR_ROUTE_SUBSPACE / SOLAR_ROUTE_TRIDIAG: the result
                                   was written although its error bounds did not hold          */
  SOLAR_INFO_DEVICE_WAIT = 8    /* a bounded wait inside the Gram kernel (on a TMA copy or on the
                                   tensor cores) ran out; s, V of this user are NaN             */
};

/* How solar_eig_from_partials_ex reaches the top-r eigenpairs of H_b^T H_b.
 * AUTO (what solar_lowrank_factor uses): Householder tridiagonalisation of the d x d
 * matrix, the r largest eigenvalues by Sturm-count multisection, their vectors by the
 * twisted factorisation, back-transformation; accepted per user only when the residuals
 * G v - theta v against the Gram matrix itself, V^T V = I and the trace certify the r
 * pairs, else the parallel Jacobi eigensolver on the whole matrix runs for that user.
 * SUBSPACE: Algorithm 1 (randomized range finder with power iteration) applied to the
 * d x d Gram matrix, then a Rayleigh-Ritz solve, alone; users whose residual and trace
 * bounds do not certify the result are flagged in info[].  FULL: the Jacobi eigensolver for every user (Eq. 9's exact
 * truncated SVD whatever the spectrum).  TRIDIAG: the tridiagonal route alone,
 * uncertified users flagged in info[].
 *
 * The route argument may carry two more fields above the low byte (both 0 = default):
 *   bits  8..15  sweep cap of the Jacobi eigensolver (1..16; default 16): a user not
 *                converged by then gets SOLAR_INFO_NOT_CONVERGED;
 *   bits 16..23  with SUBSPACE: run exactly this many orthonormalised power steps
 *                (Algorithm 1 with n_iter = value - 1, value <= 5) instead of the adaptive
 *                count. */
enum { SOLAR_ROUTE_AUTO = 0, SOLAR_ROUTE_SUBSPACE = 1, SOLAR_ROUTE_FULL = 2, SOLAR_ROUTE_TRIDIAG = 3 };
#define SOLAR_ROUTE_WITH(route, sweep_cap, power_steps) \
  ((route) | ((sweep_cap) << 8) | ((power_steps) << 16))

const char* solar_status_string(solar_status_t st);

/* Bytes of scratch that either call below needs for these sizes (the larger of
 * the two).  Pure host arithmetic; returns 0 for unsupported sizes. */
size_t solar_workspace_bytes(int B, int M, int N, int d, int r, solar_dtype_t dt);

/*
 * Rank-r truncated SVD of every H_b (Eq. 9), without forming U.
 *
 *   H    [B,N,d] dt   (in)   history embeddings, the shared key-value matrix
 *   S    [B,r]  f32   (out)  singular values, descending
 *   V    [B,d,r] f32  (out)  right singular vectors; V[b,j,i] = component j of v_i.
 *                            Sign convention: the largest-magnitude component of
 *                            each v_i is positive (lowest index wins a tie).
 *   US   [B,N,r] dt   (out)  U*Sigma = H*V, or NULL to skip it (Eq. 10 removes U
 *                            from the forward pass; it is offered for callers
 *                            that want the left factor)
 *   info [B] int      (out)  SOLAR_INFO_* bits per user, or NULL
 *
 * Route: G_b = H_b^T H_b is accumulated in one streaming pass over H; its top-r
 * eigenpairs come from a tridiagonal reduction of the d x d matrix (Householder,
 * Sturm-count multisection, twisted factorisation) when that result can be certified
 * against G_b, else from a parallel Jacobi eigensolver on the whole matrix
 * (SOLAR_ROUTE_AUTO above); s_i = sqrt(lambda_i).  Algorithm 1 of the paper (the
 * randomized range finder) is available as SOLAR_ROUTE_SUBSPACE of
 * solar_eig_from_partials_ex.  M is accepted for a uniform signature and ignored.
 */
solar_status_t solar_lowrank_factor(int B, int M, int N, int d, int r, solar_dtype_t dt,
                                    const void* H, float* S, float* V, void* US, int* info,
                                    void* workspace, size_t workspace_bytes, void* stream);

/*
 * SVD-Attention over the factor tokens (Eq. 11, Eq. 12):
 *   Query   = C W_Q                      [M,d]
 *   Key_r   = (V Sigma)^T W_K            [r,d]
 *   Value_r = (V Sigma)^T W_V            [r,d]
 *   O       = softmax_rows(scale * Query Key_r^T) Value_r      [M,d]
 *
 *   C        [B,M,d] dt (in)   candidate embeddings
 *   S, V               (in)    as written by solar_lowrank_factor
 *   Wq,Wk,Wv [d,d] dt   (in)   shared by all users; y = x W
 *   scale               (in)   multiplies the scores (the paper prints none; 1/sqrt(d) is usual)
 *   flags               (in)   0 or SOLAR_FLAG_NO_SOFTMAX
 *   O        [B,M,d] dt (out)
 *
 * The M x r score matrix lives in registers / tensor memory only.  N is accepted
 * for a uniform signature and ignored.
 */
solar_status_t solar_svd_attention_fwd(int B, int M, int N, int d, int r, solar_dtype_t dt,
                                       const void* C, const float* S, const float* V,
                                       const void* Wq, const void* Wk, const void* Wv,
                                       float scale, unsigned flags, void* O,
                                       void* workspace, size_t workspace_bytes, void* stream);

/*
 * The whole forward pass in one call: solar_lowrank_factor followed by
 * solar_svd_attention_fwd (Eq. 9-12), with the same arguments, outputs, info bits and
 * rules, and the same bits in S, V and O.  Three launches instead of four: every user's
 * eigensolver CTA ends with that user's factor-token projections (Eq. 11), so the
 * stand-alone projection kernel and its launch disappear.  S and V are still written.
 *
 *   workspace: solar_fused_workspace_bytes() of the same sizes (the factorization's
 *   scratch followed by the attention's); contents undefined on return.
 */
size_t solar_fused_workspace_bytes(int B, int M, int N, int d, int r, solar_dtype_t dt);

solar_status_t solar_svd_attention_fused(int B, int M, int N, int d, int r, solar_dtype_t dt,
                                         const void* H, const void* C,
                                         const void* Wq, const void* Wk, const void* Wv,
                                         float scale, unsigned flags, float* S, float* V, void* O,
                                         int* info, void* workspace, size_t workspace_bytes,
                                         void* stream);

/* ------------------------------------------------------------------------- *
 * Stage-level entry points.  The two calls above are exactly
 *   solar_lowrank_factor    = solar_gram_partials ; solar_eig_from_partials [; solar_project_us]
 *   solar_svd_attention_fwd = solar_attn_prepare  ; solar_attn_apply
 * on the same workspace.  They exist so that each kernel can be timed and
 * checked on its own; argument meaning and rules are those given above.
 * ------------------------------------------------------------------------- */

/* Tuning knob, process-wide: the largest number of row slices (CTAs) a user's history is cut
 * into by the streaming passes over H (the Gram pass of Eq. 9's factorization, U Sigma = H V,
 * dH = H K); 0, the default, means no cap.  Without a cap the slicing is chosen for the latency
 * of ONE call: B * slices CTAs fill the GPU once (B = 16, N = 10240: nine slices).  A process
 * that keeps many independent calls in flight on different streams is better served by fewer,
 * longer slices (two or three): every CTA pays its fixed start-up and wind-down while holding
 * shared memory that other requests' CTAs could use, and the eigensolver adds up fewer partial
 * matrices -- measured on that shape with 30 requests in flight: 8.5 us per request at nine
 * slices, 7.9 at three, 7.8 at two, for 66 / 71 / 77 us of latency per single call.
 * A positive value is read as "this process wants throughput" by the other kernels too: the
 * candidate attention (bf16, d = 64, r <= 32, M >= 512) then runs as a few long CTAs per user
 * that overlap the candidate stream, the GEMMs and the softmax of consecutive tiles -- the same
 * bits in O -- and the eigensolver releases it a little later; together 7.6 us per request in
 * flight and about 100 us for a lone call.
 * Results agree to rounding (the partial sums are grouped differently), not bit for bit.
 * Set it before sizing workspaces: the *_workspace_bytes functions follow the current value,
 * and a call made under a higher cap than its workspace was sized for returns
 * SOLAR_ERR_WORKSPACE.  Keep it unchanged between a stage call that writes a workspace
 * (solar_gram_partials) and the stage calls that read it.  Returns the previous value.  Safe to
 * call from any thread; calls already enqueued are not affected. */
int solar_set_slice_limit(int max_slices);

/* Number of partial Gram matrices solar_gram_partials leaves per user (>= 1), and
 * the number of row slices (CTAs, status words) per user behind them (a multiple of it). */
int solar_gram_splits(int B, int N, int d, solar_dtype_t dt);
int solar_gram_slices(int B, int N, int d, solar_dtype_t dt);

/* Streaming pass over H.  Every H_b is cut into row slices (one CTA each); partial p of
 * user b is the sum of h_n h_n^T over the rows n of its group of slices (fp32), stored at
 *   ((float*)workspace)[(b*P + p)*d*d ...],  P = solar_gram_splits(),  row-major;
 * the kernel's per-slice status words follow the partials (read by
 * solar_eig_from_partials).  H_b^T H_b (the matrix whose eigenvectors are V of Eq. 9) is
 * the sum over p.  bf16 storage with d = 64 or 128 and N >= 128 runs on the tensor cores
 * (TMA tiles, tcgen05.mma, fp32 accumulation in tensor memory); other shapes use FFMA.
 * P = solar_gram_splits() divides the slice count solar_gram_slices(): the CTAs of P-th
 * parts of the slices may add up their results on chip (thread-block clusters); as built,
 * every slice leaves its own partial. */
solar_status_t solar_gram_partials(int B, int N, int d, solar_dtype_t dt, const void* H,
                                   void* workspace, size_t workspace_bytes, void* stream);

/* Sums the partial Grams in slice order and diagonalises; writes S, V, info.  The summed
 * matrices [B,d,d] fp32 are left in the workspace (behind the status words, or in place of
 * the partials where a user has only one). */
solar_status_t solar_eig_from_partials(int B, int N, int d, int r, solar_dtype_t dt,
                                       float* S, float* V, int* info,
                                       void* workspace, size_t workspace_bytes, void* stream);

/* As above with the route chosen by the caller.  route_taken (device, [B] ints, or
 * NULL) receives per user: route used (1 subspace, 2 full, 3 tridiagonal; 0 = non-finite
 * input) | power steps << 8 | Jacobi sweeps (route 3: orthogonalisation passes) << 16 |
 * reason << 24, where reason says why the first route tried was not certified: 1 no gap
 * at the cut, 2 residual too large for its gap, 4 a kept eigenvalue not positive, 8 sweep
 * cap, 16 non-finite pivot, 32 vectors of a cluster not independent, 64 trace mismatch
 * or a non-finite value. */
solar_status_t solar_eig_from_partials_ex(int B, int N, int d, int r, solar_dtype_t dt, int route,
                                          float* S, float* V, int* info, int* route_taken,
                                          void* workspace, size_t workspace_bytes, void* stream);

/* US = H V in the storage type (second pass over H). */
solar_status_t solar_project_us(int B, int N, int d, int r, solar_dtype_t dt, const void* H,
                                const float* V, void* US, void* stream);

/* Per-user factor-token projections of Eq. 11 into the workspace:
 * Value_r and the folded score operand T_b = scale * W_Q Key_r^T  (d x r). */
solar_status_t solar_attn_prepare(int B, int d, int r, solar_dtype_t dt,
                                  const float* S, const float* V,
                                  const void* Wq, const void* Wk, const void* Wv, float scale,
                                  void* workspace, size_t workspace_bytes, void* stream);

/* Scores, softmax over the r tokens, weighted sum (Eq. 12), from the workspace
 * written by solar_attn_prepare with the same B, d, r, dt. */
solar_status_t solar_attn_apply(int B, int M, int d, int r, solar_dtype_t dt, const void* C,
                                unsigned flags, void* O,
                                void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------- *
 * Backward pass of the truncated SVD with U absent from the forward pass (Eq. 13-15
 * and the appendix that derives them):
 *   dH = U [ diag(dS) + 2 Sigma sym(F o (dV^T V)) ] V^T,   U = H V Sigma^-1,
 *   F_ij = D_ij / (D_ij^2 + eps^2),  D_ij = sigma_i^2 - sigma_j^2,  eps = eps_rel * sigma_max^2
 * (eps_rel = 0 is Eq. 14 itself, with F_ij = 0 where D_ij = 0).  The Hadamard factor is
 * dV^T V, the index order for which the formula is the derivative of the forward pass
 * (the appendix's expansion of the trace has the indices transposed, which flips the sign
 * of that term).  Evaluated as one more streaming pass over H:  dH_b = H_b K_b with
 * K_b = V Sigma^-1 [.] V^T, so U is never materialised.  For r < d this is the part of
 * the gradient that acts within the kept subspace: the component of dV orthogonal to span(V)
 * and the coupling to the discarded singular pairs are left out (the bias the paper bounds
 * by |dV_orth|_F / sigma_r).  It is the exact gradient for r = d and for perturbations of
 * the form U X V^T.
 *
 *   H   [B,N,d] dt  (in)   the histories given to solar_lowrank_factor
 *   S   [B,r]  f32  (in)   singular values,  V [B,d,r] f32 (in) right singular vectors
 *   dS  [B,r]  f32  (in)   dL/dSigma,        dV [B,d,r] f32 (in) dL/dV
 *   dH  [B,N,d] dt  (out)  dL/dH; a direction with sigma_i = 0 contributes nothing
 *   workspace: at least B*d*d*4 bytes (solar_workspace_bytes() of the same sizes is enough);
 *   holds K_b [B,d,d] f32 on return.
 * Two launches on `stream`; no synchronisation; nothing is allocated.
 * ------------------------------------------------------------------------- */
solar_status_t solar_svd_backward(int B, int N, int d, int r, solar_dtype_t dt, const void* H,
                                  const float* S, const float* V, const float* dS, const float* dV,
                                  float eps_rel, void* dH, void* workspace, size_t workspace_bytes,
                                  void* stream);

/* ------------------------------------------------------------------------- *
 * Backward pass of solar_svd_attention_fwd: the chain rule through Eq. 11-12 (the
 * paper prints the SVD's gradient, Eq. 13-15, and leaves this part to calculus).
 * Given dO = dL/dO it returns the gradients with respect to every input of the
 * forward call; dS and dV then go to solar_svd_backward for dL/dH.
 *
 *   C, S, V, Wq, Wk, Wv, scale, flags: exactly as given to solar_svd_attention_fwd
 *   dO   [B,M,d] dt  (in)
 *   dC   [B,M,d] dt  (out)
 *   dWq, dWk, dWv [d,d] f32 (out)  summed over the B users (overwritten, not accumulated)
 *   dS   [B,r]   f32 (out)  dL/dSigma        dV [B,d,r] f32 (out)  dL/dV
 *   workspace: solar_backward_workspace_bytes() of the same sizes; contents undefined on
 *   return.  The scores and probabilities are recomputed from C, never stored.
 * Sums over candidates and over users run in a fixed order: the results are
 * reproducible bit for bit.  N is accepted for a uniform signature and ignored.
 * ------------------------------------------------------------------------- */
size_t solar_backward_workspace_bytes(int B, int M, int N, int d, int r, solar_dtype_t dt);

solar_status_t solar_svd_attention_bwd(int B, int M, int N, int d, int r, solar_dtype_t dt,
                                       const void* C, const float* S, const float* V,
                                       const void* Wq, const void* Wk, const void* Wv,
                                       float scale, unsigned flags, const void* dO,
                                       void* dC, float* dWq, float* dWk, float* dWv,
                                       float* dS, float* dV,
                                       void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------- *
 * Softmax attention over the N history positions, evaluated through the factors:
 *   O = softmax_rows( scale * (C W_Q W_K^T V) (U Sigma)^T ) (U Sigma) (V^T W_V)    [M,d]
 * With H = U Sigma V^T of rank <= r this equals the softmax attention of Eq. 6-7,
 * softmax(scale * Query Key^T) Value with Key = H W_K, Value = H W_V, at O(N M r)
 * instead of O(N M d): the literal sense in which the factorization of Eq. 9 is
 * lossless WITH the softmax.  It is not the paper's SVD-Attention operator (Eq. 12),
 * which removes U (Eq. 10) and normalises over the r factor tokens; it is offered
 * beside it because it needs nothing but the factors.
 *
 *   C        [B,M,d] dt (in)   candidate embeddings
 *   US       [B,N,r] dt (in)   U Sigma = H V, as written by solar_lowrank_factor
 *   V        [B,d,r] f32 (in)  right singular vectors (any sign convention: it cancels)
 *   Wq,Wk,Wv [d,d] dt   (in)   shared by all users; y = x W
 *   O        [B,M,d] dt (out)
 *   workspace: solar_workspace_bytes() of the same sizes.
 * One flash-attention style kernel per call (after the small per-user operand set-up):
 * the N x M scores live in tensor memory only.  Supported: dt = SOLAR_BF16, d in
 * {64, 128}, r in {16, 32, 64}; other shapes return SOLAR_ERR_UNSUPPORTED.
 * ------------------------------------------------------------------------- */
solar_status_t solar_factored_softmax_attention_fwd(int B, int M, int N, int d, int r, solar_dtype_t dt,
                                                    const void* C, const void* US, const float* V,
                                                    const void* Wq, const void* Wk, const void* Wv,
                                                    float scale, void* O, void* workspace,
                                                    size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------- *
 * Factorization without caller-provided scratch.  (The paper has no counterpart:
 * this is a packaging variant of solar_lowrank_factor, not another operation.)
 *
 * Some hosts of this library may not allocate device memory at all: a ranking
 * server that carves every buffer out of an arena planned at start-up and
 * forbids cudaMalloc while serving (it synchronises the device and can fail
 * when the arena already fills the GPU), or a plug-in that is handed only its
 * input and output tensors.  For them the partial-Gram scratch sits in a fixed
 * 16 MiB array compiled into the library (solar_static_scratch_bytes()); every
 * GPU that loads the library holds those 16 MiB until the process exits.
 *
 *   - Same arguments, outputs, info bits and rules as solar_lowrank_factor,
 *     minus US and the workspace.  Calls no cudaMalloc / cudaFree and no
 *     allocating library routine.
 *   - Sizes whose scratch need, solar_workspace_bytes(B, 0, N, d, r, dt) bytes,
 *     exceeds the array return SOLAR_ERR_WORKSPACE before anything is launched
 *     (the headline shape B=16, N=10240, d=64 needs 2.25 MiB).
 *   - The first call on each device looks up the array's device address (with
 *     that device current) and caches it; make that first call outside any
 *     stream capture.  The array is chosen by the CURRENT device: the device
 *     that `stream` belongs to must be current when the call is made.
 *   - All calls on a device share the one array: it keeps whatever the last call
 *     left (every slice is fully overwritten before it is read, nothing needs
 *     zeroing), and two calls that overlap on the GPU -- different streams,
 *     or a call racing solar_eig_from_partials of another -- corrupt each other.
 *     Serialise them on one stream or with events.
 * ------------------------------------------------------------------------- */
size_t solar_static_scratch_bytes(void);
solar_status_t solar_lowrank_factor_static(int B, int M, int N, int d, int r, solar_dtype_t dt,
                                           const void* H, float* S, float* V, int* info,
                                           void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SOLAR_H_ */
