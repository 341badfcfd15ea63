/*
 * laplace_nystrom.h -- C ABI of the B200 (sm_100a) library for Nystrom-approximated
 * Laplacian-kernel attention, forward and backward (LaplacianFormer, arXiv 2604.20368).
 *
 * Per (batch, head), with Q,K,V in R^{n x d}, m landmarks L in R^{m x d}, decay lambda,
 * T Newton-Schulz steps, ridge eps and a diagonal whitening scale s in R^m:
 *
 *   k(x,y) = exp(-||x - y||_1 / lambda)              Laplacian kernel (Sec. 1)
 *   L  = average pooling of K over the token grid    landmark selection (Sec. 4.2)
 *   C  = k(Q,L) [n x m]                               Eq. 8
 *   W  = k(L,L) + eps I [m x m]                       Eq. 9 and the ridge of Alg. 2
 *   R  = k(L,K) [m x n]                               the C^T factor of Alg. 1
 *   X_0 = alpha W^T, X_{k+1} = X_k (2I - W X_k)       Alg. 2, X = X_T, alpha = 1/(||W||_1 ||W||_inf)
 *   M  = R V,  Y = X M
 *   Z_il = s_l (C_il - mean_l' C_il') + 1/m           Prop. 3 / Eq. 11 with the diagonal whitening of Eq. 6
 *   O  = Z Y                                          Eq. 7 with the kernel matrix in Nystrom form
 *
 * Conventions common to every entry point
 *   - Every pointer is a DEVICE pointer unless it is the ln_problem itself (host).
 *   - The caller owns every buffer.  The library allocates no device memory and never
 *     synchronises the device: it validates arguments on the host, enqueues kernels on
 *     `stream` (a cudaStream_t passed as void*; NULL = the default stream) and returns.
 *     LN_OK means "enqueued".  The only state kept between calls is one extra stream and a
 *     few events per (device, caller stream) pair (see ln_set_overlap), created by the first bf16
 *     attention call on that pair: that call should come before any stream capture.  Calls on
 *     different streams share none of it.  Two host threads enqueueing on the SAME stream at the
 *     same time are not supported.
 *   - Tensors are contiguous, row-major, 16-byte aligned.  Outputs are fully overwritten.
 *     Inputs are never modified and must not alias outputs.
 *   - Storage type of the [.,.,.,d] tensors is `dtype` (LN_F32 or LN_BF16); all arithmetic and
 *     every on-device intermediate is fp32.
 *   - Errors: LN_ERR_ARG (NULL required pointer, non-positive size, m > n, lambda <= 0 or not
 *     finite, T < 0, eps < 0, grid inconsistent with n or m, misaligned pointer),
 *     LN_ERR_UNSUPPORTED (d not in {32, 64, 128} or m > 256 for the attention entry points),
 *     LN_ERR_WORKSPACE (ws_bytes too small), LN_ERR_CUDA (a launch failed).  Nothing is
 *     enqueued when an argument error is returned.
 */
#ifndef LAPLACE_NYSTROM_H_
#define LAPLACE_NYSTROM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { LN_OK = 0, LN_ERR_ARG = -1, LN_ERR_UNSUPPORTED = -2, LN_ERR_WORKSPACE = -3, LN_ERR_CUDA = -4,
               LN_ERR_STATIC_LIMIT = -5 } ln_status;
typedef enum { LN_F32 = 0, LN_BF16 = 1 } ln_dtype;

/* The problem statement of Alg. 1 / Alg. 2 in the paper's notation. */
typedef struct ln_problem {
  int32_t B, H, n, d, m;  /* Q,K,V,O,dO,dQ,dK,dV: [B,H,n,d];  L,dL: [B,H,m,d]                             */
  float lambda;           /* decay of the Laplacian kernel, > 0                                           */
  int32_t ns_iters;       /* T >= 0 Newton-Schulz steps (Alg. 2)                                          */
  float ridge_eps;        /* eps >= 0 added to the diagonal of k(L,L) (Alg. 2)                            */
  float ns_alpha;         /* <= 0: alpha = 1/(||W||_1 ||W||_inf);  > 0: used as given, not differentiated */
  int32_t dtype;          /* ln_dtype of the [.,.,.,d] tensors                                            */
  int32_t map_mode;       /* 0: O = C X R V;  1: injective map of Prop. 3 applied to the rows of C        */
  const float* whiten;    /* device [H,m] fp32 whitening scale s (Eq. 6), or NULL = ones; a constant      */
  int32_t lm_mode;        /* 0: landmarks L given by the caller;  1: L = adaptive average pooling of K;   */
                          /* 2: of Q (Sec. 4.2 pools the query tensor in one place): dL then returns to dQ */
                          /* 3: two landmark sets, as Alg. 1 prints them: Lq = pool(Q), Lk = pool(K),      */
                          /*    C = k(Q,Lk), W = k(Lq,Lk) + eps I (not symmetric), R = k(Lq,K); dLq, dLk   */
                          /*    return to dQ, dK.  The per-head iteration then runs on the general engine */
                          /*    (mma.sync / FFMA, not tcgen05); whiten_mode 1 is LN_ERR_UNSUPPORTED.       */
  int32_t prefix, gh, gw, mh, mw; /* lm_mode >= 1: n = prefix + gh*gw, m = mh*mw.  Bin (a,b) averages grid  */
                          /* rows floor(a*gh/mh) .. ceil((a+1)*gh/mh)-1 and columns likewise; the first   */
                          /* `prefix` tokens (class tokens) are ordinary queries/keys but are not pooled. */
  int32_t whiten_mode;    /* 0: `whiten` is a constant input (or NULL = ones).  1: batch statistics (Eq. 5-6 in     */
                          /* training mode): the forward pass estimates s_l = 1/sqrt(Var_{b,i}(C_il) + whiten_eps)  */
                          /* over the query rows of every batch element of a head inside the kernel that forms C,  */
                          /* writes it to whiten_batch and uses it; the backward pass differentiates through the   */
                          /* variance.  Needs map_mode 1, whiten == NULL.  The batch elements of a head are then    */
                          /* coupled through the statistic.                                                         */
  float whiten_eps;       /* eps of Eq. 6 (whiten_mode 1), >= 0                                                     */
  float* whiten_batch;    /* whiten_mode 1: device [H,m] fp32 written by laplace_nystrom_fwd, read by _bwd         */
  const float* lm_filter; /* NULL: landmarks are averages over their regions.  Else the depth-wise-convolution     */
                          /* selection Sec. 4.2 describes as the alternative: device fp32 [H, taps, d], 16-byte     */
                          /* aligned, taps = (gh/mh)*(gw/mw), one filter per head and channel applied with stride  */
                          /* equal to the region (tap (u,v) of a region at index u*(gw/mw)+v; no bias; all taps    */
                          /* 1/taps is average pooling).  lm_mode 1 or 2 with mh | gh and mw | gw (else            */
                          /* LN_ERR_ARG); lm_mode 3 is LN_ERR_UNSUPPORTED.  A landmark is the fp32 value nearest   */
                          /* to the exact weighted sum.                                                            */
  float* lm_filter_grad;  /* with lm_filter: device fp32 [H, taps, d], 16-byte aligned, OVERWRITTEN by             */
                          /* laplace_nystrom_bwd with the gradient of the filter, summed over the batch; required  */
                          /* by the backward entry points (LN_ERR_ARG if NULL), ignored by the forward ones        */
  int32_t solver;         /* 0: Newton-Schulz (Alg. 2), Y = X_T M.  1: conjugate gradients, the other solver of the        */
                          /* ablation (Sec. 5.3, Table 4): Y = the ns_iters-step iterate of (k(L,L) + eps I) Y = M from    */
                          /* Y_0 = 0, every column of M on its own (Hestenes-Stiefel; a column whose residual is zero or   */
                          /* whose curvature is not positive stops); ns_alpha is ignored.  The backward pass               */
                          /* differentiates the linear system the solver approximates: dM = the same ns_iters-step         */
                          /* iterate of the system with right-hand side dY, dW = -dM Y^T (the paper names the solver       */
                          /* only).  The recurrence runs in double precision, one CTA per head, for either storage dtype.  Needs the symmetric     */
                          /* matrix of one landmark set: lm_mode 3 is LN_ERR_UNSUPPORTED, and so is whiten_mode 1 (not built).  dev_status bit 0 then means a   */
                          /* non-finite entry of Y.                                                                        */
} ln_problem;

const char* ln_status_string(int status);

/*
 * Sizes of the two caller-provided buffers of the attention entry points, in bytes.
 *   saved: context handed from laplace_nystrom_fwd to laplace_nystrom_bwd (landmarks, the kernel
 *          blocks C and R, W, the Newton-Schulz iterates X_0..X_T, M, the folded Y).  Contents are
 *          defined only between a fwd and the matching bwd.
 *   ws:    scratch whose contents are undefined between calls.  `with_saved` = 1 when a saved buffer
 *          will be passed (training), 0 for inference, where the context lives in ws as well.
 * Both return 0 for an invalid problem.
 */
size_t laplace_nystrom_saved_bytes(const ln_problem* p);
size_t laplace_nystrom_workspace_bytes(const ln_problem* p, int32_t with_saved);

/*
 * Forward of the whole path (Alg. 1 + Alg. 2 + Prop. 3).
 *   Q,K,V  [B,H,n,d] dtype;  L [B,H,m,d] dtype, required iff lm_mode == 0 (else NULL);
 *   O      [B,H,n,d] dtype, overwritten;
 *   saved  NULL for inference, else laplace_nystrom_saved_bytes(p) bytes;
 *   ws     laplace_nystrom_workspace_bytes(p, saved != NULL) bytes;
 *   dev_status NULL or int32 [B*H], zeroed by the call and written by the device, per head:
 *     bit 0 = X_T has a non-finite entry (a diverged iteration, e.g. a bad ns_alpha);
 *     bit 1 = a bounded wait on the tensor cores or on a bulk copy ran out (the kernel gave up, freed its
 *             tensor memory and returned; that head's results are then undefined).  Neither traps.
 */
int laplace_nystrom_fwd(const ln_problem* p, const void* Q, const void* K, const void* V, const void* L,
                        void* O, void* saved, void* ws, size_t ws_bytes, int32_t* dev_status, void* stream);

/*
 * Backward of the whole path: the exact adjoint of what laplace_nystrom_fwd computes, including
 * the T unrolled Newton-Schulz steps and alpha's dependence on W (App. A gives the kernel
 * gradient -(1/lambda) sign(x - y) k, with sign(0) = 0).
 *   dO [B,H,n,d] dtype;  saved: the buffer the matching fwd filled;
 *   dQ,dK,dV [B,H,n,d] dtype, overwritten;
 *   dL [B,H,m,d] dtype: required when lm_mode == 0; must be NULL when lm_mode is 1, 2 or 3 (the
 *   landmark gradient is folded into dK, dQ, or both, through the pooling adjoint).
 *   ws: laplace_nystrom_workspace_bytes(p, 1) bytes.
 *   dev_status: as for laplace_nystrom_fwd (only bit 1 can be set by the backward pass).
 */
int laplace_nystrom_bwd(const ln_problem* p, const void* Q, const void* K, const void* V, const void* L,
                        const void* dO, const void* saved, void* dQ, void* dK, void* dV, void* dL,
                        void* ws, size_t ws_bytes, int32_t* dev_status, void* stream);

/*
 * One training step of the whole path for tensors that live in HOST memory (the paper has no counterpart: a
 * packaging of laplace_nystrom_fwd + laplace_nystrom_bwd, same arithmetic, same results).  Enqueues on `stream`:
 * copies of hQ, hK, hV, hdO (host, [B,H,n,d] dtype; pinned memory makes the copies asynchronous) into
 * `staging`, the forward pass, the copy of O back to hO, the backward pass, the copies of dQ, dK, dV back to
 * hdQ, hdK, hdV.  Returns once everything is enqueued; the host outputs are valid after the stream has been
 * synchronised.  lm_mode must be 1 (landmarks pooled from K), else LN_ERR_UNSUPPORTED.
 *   staging: DEVICE memory, laplace_nystrom_host_staging_bytes(p) bytes, 16-byte aligned, owned by the caller;
 *   saved, ws, dev_status: as for laplace_nystrom_fwd / _bwd (training sizes); dev_status is cleared once and
 *   collects the flags of both passes.  Every argument check of both passes is made before the first copy.
 * The copies ride on two copy streams the library keeps per (device, stream), tied to `stream` by events (Q, K, V in,
 * dO in beside the forward pass, O out beside the backward pass, the gradients out at the end); `stream` waits for the
 * last copy, so to the caller the call is still ordered on `stream`.  With ln_set_overlap(0) everything goes on `stream`
 * itself.  Several calls on several streams with their own device buffers overlap each other's copies and kernels.
 */
size_t laplace_nystrom_host_staging_bytes(const ln_problem* p);
int laplace_nystrom_fwd_bwd_host(const ln_problem* p, const void* hQ, const void* hK, const void* hV, const void* hdO,
                                 void* hO, void* hdQ, void* hdK, void* hdV, void* staging, size_t staging_bytes,
                                 void* saved, void* ws, size_t ws_bytes, int32_t* dev_status, void* stream);

/*
 * The attention block around the path (Eq. 7 and the implementation details of Sec. 5.1):
 *     Qr = rope(Q), Kr = rope(K);   O = Z(Qr, Kr) Y(Kr, V) + DWC(V).
 * rope: rotary position embedding, channel pairs (2i, 2i+1) of the token at grid position p (row-major over the
 *   gh x gw grid; the `prefix` class tokens are not rotated) turn by p * rope_base^(-2i/d); rope_base = 0 switches it
 *   off.  The rotated tensors are kept in the storage type (bf16 storage rounds them once more).
 * DWC: depth-wise ks x ks cross-correlation over the token grid, zero padded, one filter per head and channel,
 *   dwc_w device fp32 [H, d, ks, ks] (ks odd, <= 7), NULL = no convolution branch; prefix tokens receive nothing.
 *   For bf16 storage with d = 64 or 128 the branch is added inside the kernels that form O and dV, before their one
 *   rounding; otherwise it is a pass of its own over O / dV.
 * lm_mode must be 1, 2 or 3 (the grid geometry of `p` is used), else LN_ERR_UNSUPPORTED.
 *   saved: laplace_attention_block_saved_bytes bytes; ws: laplace_attention_block_workspace_bytes bytes (both
 *   passes); the other arguments as for laplace_nystrom_fwd / _bwd.  The backward returns dQ, dK, dV and, when the
 *   convolution branch is on, dWd device fp32 [H, d, ks, ks] (summed over the batch in a fixed order), else dWd = NULL.
 */
typedef struct ln_block {
  const float* dwc_w;
  int32_t dwc_ks;
  float rope_base;
} ln_block;
size_t laplace_attention_block_saved_bytes(const ln_problem* p, const ln_block* b);
size_t laplace_attention_block_workspace_bytes(const ln_problem* p, const ln_block* b);
int laplace_attention_block_fwd(const ln_problem* p, const ln_block* b, const void* Q, const void* K, const void* V, void* O,
                                void* saved, void* ws, size_t ws_bytes, int32_t* dev_status, void* stream);
int laplace_attention_block_bwd(const ln_problem* p, const ln_block* b, const void* Q, const void* K, const void* V,
                                const void* dO, const void* saved, void* dQ, void* dK, void* dV, float* dWd, void* ws,
                                size_t ws_bytes, int32_t* dev_status, void* stream);

/*
 * Newton-Schulz iterate of (W + eps I)^-1 (Alg. 2), batched over `batch` independent m x m
 * fp32 matrices.  X [batch,m,m] receives X_T.  X_hist is NULL or [batch,iters+1,m,m] and
 * receives X_0 .. X_T.  resid is NULL or [batch] and receives ||I - (W + eps I) X_T||_F.
 * alpha <= 0 selects 1/(||W||_1 ||W||_inf).  ws: ns_pinv_workspace_bytes(batch, m, iters).
 */
size_t ns_pinv_workspace_bytes(int32_t batch, int32_t m, int32_t iters);
int ns_pinv(int32_t batch, int32_t m, const float* W, int32_t iters, float ridge_eps, float alpha,
            float* X, float* X_hist, float* resid, void* ws, size_t ws_bytes, void* stream);

/*
 * Adjoint of ns_pinv: given dX = dLoss/dX_T returns dW = dLoss/dW [batch,m,m] (W before the ridge).
 * X_hist: the [batch,iters+1,m,m] history a previous ns_pinv wrote, or NULL to recompute it.
 * With alpha <= 0 the dependence of alpha on W is differentiated (arg-max ties -> lowest index).
 * ws: ns_pinv_workspace_bytes(batch, m, iters).
 */
int ns_pinv_bwd(int32_t batch, int32_t m, const float* W, int32_t iters, float ridge_eps, float alpha,
                const float* X_hist, const float* dX, float* dW, void* ws, size_t ws_bytes, void* stream);

/*
 * ns_pinv without a workspace argument, for callers that cannot allocate device memory (the paper
 * has no counterpart; this is a packaging variant of ns_pinv, same arithmetic, same results).
 * Think of a serving process whose memory pool is fully committed at start-up, or a plug-in that
 * only ever receives input and output pointers: neither can come up with the scratch ns_pinv
 * wants.  Here the scratch is a fixed array of LN_STATIC_SCRATCH_BYTES inside the library image,
 * so every GPU that loads the library gives up that much memory until the process exits.
 *   - The caller still passes W [batch,m,m] and X [batch,m,m] (and resid [batch] or NULL); there
 *     is no X_hist output.  Nothing is allocated or freed, by this call or on its behalf.
 *   - Limit: ns_pinv_workspace_bytes(batch, m, iters) must not exceed LN_STATIC_SCRATCH_BYTES
 *     (for instance batch 16, m 64, 6 iterations, or batch 2, m 256, 8 iterations); beyond it the
 *     call returns LN_ERR_STATIC_LIMIT and enqueues nothing.
 *   - The first call on each device looks up the device address of the array (with that device
 *     current); make that first call outside any stream capture.
 *   - All calls on a device share the one array.  It keeps whatever the last call left, which is
 *     harmless (every part is written before it is read), but two calls that overlap on the GPU,
 *     for example on different streams, race on it: serialise them.
 */
#define LN_STATIC_SCRATCH_BYTES (8u << 20)
size_t ns_pinv_static_scratch_bytes(void);
int ns_pinv_static(int32_t batch, int32_t m, const float* W, int32_t iters, float ridge_eps, float alpha,
                   float* X, float* resid, void* stream);

/*
 * Laplacian kernel block (Sec. 1, Eq. 8): Kout[b,i,j] = exp(-||A[b,i,:] - Bm[b,j,:]||_1 / lambda).
 * A [batch,na,d], Bm [batch,nb,d] of `dtype`; Kout [batch,na,nb] fp32; rowsum NULL or [batch,na]
 * fp32 = sum_j Kout[b,i,j].  Any d >= 1.
 */
int l1_kernel(int32_t batch, int32_t na, int32_t nb, int32_t d, const void* A, const void* Bm, int32_t dtype,
              float lambda, float* Kout, float* rowsum, void* stream);

/*
 * Adjoint of l1_kernel (App. A): with g = dKmat * Kmat / lambda,
 *   dA[b,i,:] = -sum_j g_ij sign(A_i - B_j),  dB[b,j,:] = +sum_i g_ij sign(A_i - B_j),  sign(0) = 0.
 * Kmat: the block a previous l1_kernel wrote, or NULL to recompute it.  dA, dB have `dtype` and
 * are overwritten.  ws: l1_kernel_bwd_workspace_bytes(batch, na, nb, d) bytes of scratch.
 */
size_t l1_kernel_bwd_workspace_bytes(int32_t batch, int32_t na, int32_t nb, int32_t d);
int l1_kernel_bwd(int32_t batch, int32_t na, int32_t nb, int32_t d, const void* A, const void* Bm, int32_t dtype,
                  float lambda, const float* Kmat, const float* dKmat, void* dA, void* dB,
                  void* ws, size_t ws_bytes, void* stream);

/*
 * Exact Laplacian-kernel attention, forward only (Eq. 4 and Eq. 7 with the full n x n kernel matrix G = k(Q, K), which is
 * formed tile by tile on chip and never stored): the O(n^2) reference the Nystrom path approximates; at m = n with
 * converged Newton-Schulz the path reproduces it.  For accuracy-against-m curves, not for training.
 *   map_mode 1: O_i = sum_j (G_ij - mu_i) V_j + (1/n) sum_j V_j, mu_i = mean_j G_ij (the injective map with unit whitening);
 *   map_mode 0: O = G V.
 * Q, K, V, O: [batch, n, d] of `dtype`, d in {32, 64, 128}; batch = B * heads.
 */
int laplace_exact_fwd(int32_t batch, int32_t n, int32_t d, int32_t dtype, float lambda, int32_t map_mode, const void* Q,
                      const void* K, const void* V, void* O, void* stream);

/*
 * Whitening statistics (Eq. 5 and Eq. 6): the diagonal scale s [H, m] that `whiten` takes, estimated from the
 * query-landmark kernel block C = k(Q, L) that laplace_nystrom_fwd left in `saved`.  For head h and landmark l the
 * batch of Eq. 5 is every query row of every batch element:
 *     mu_l = mean_{b,i} C_il,   sigma_l^2 = mean_{b,i} (C_il - mu_l)^2   (the 1/B form of Eq. 5),
 *     s_l  = 1 / sqrt(sigma_l^2 + eps_w)                                  (the diagonal of D^{-1/2}, Eq. 6).
 * saved: the context of a forward call on the same problem (device).  whiten_out: device [H, m] fp32, overwritten.
 * ws: device scratch of laplace_nystrom_whiten_stats_workspace_bytes(p) bytes.  Sums are taken in double in a fixed
 * order (results are reproducible).  The scale is a constant of the attention entry points (no gradient flows through
 * it), as when the paper estimates it offline.  Errors as above; eps_w < 0 or not finite is LN_ERR_ARG.
 */
size_t laplace_nystrom_whiten_stats_workspace_bytes(const ln_problem* p);
int laplace_nystrom_whiten_stats(const ln_problem* p, const void* saved, float eps_w, float* whiten_out, void* ws,
                                 size_t ws_bytes, void* stream);

/*
 * Landmark selection by average pooling of the keys over the token grid (Sec. 4.2), lm_mode 1
 * geometry of `p`.  K [B,H,n,d] dtype -> L [B,H,m,d] fp32.  The backward overwrites dK [B,H,n,d]
 * (dtype) with pool^T(dL), dL [B,H,m,d] fp32.
 */
int landmarks_pool(const ln_problem* p, const void* K, float* L, void* stream);
int landmarks_pool_bwd(const ln_problem* p, const float* dL, void* dK, void* stream);

/*
 * Where an fp32 intermediate of the forward pass lies inside `saved` (the paper has no counterpart: an inspection
 * aid, used by the parity tests to compare intermediates with the oracle's).  name: "L" landmarks [m x d],
 * "C" = k(Q,L) [n x m], "Rt" = k(K,L) [n x m], "mu" row means of C [1 x n], "W" = k(L,L) [m x m] (before the
 * ridge), "X" = X_T [m x m], "M" = R V [m x d], "Yt" folded Y [m x d], "ybar" [1 x d];
 * lm_mode 3 only: "Lq" pooled queries [m x d] ("L" is then the pooled keys, "Rt" = k(K,Lq), "W" = k(Lq,L)).
 * info[0] = offset of head 0 in floats from the start of saved, info[1] = rows, info[2] = columns,
 * info[3] = leading dimension, info[4] = floats between consecutive heads.  LN_ERR_ARG for an unknown name.
 */
int laplace_nystrom_saved_array(const ln_problem* p, const char* name, int64_t info[5]);

/*
 * Self-test of failure detection (the paper has no counterpart).  Launches one tiny kernel that waits, with the
 * library's bounded wait and a limit of `probes` polls, on a barrier nothing ever arrives on; the wait gives up and
 * the kernel ORs bit 1 into dev_status[0] (device int32, not cleared by this call) and returns normally.  Shows a
 * caller, without hanging or faulting anything, what a timed-out wait in the attention kernels looks like.
 */
int ln_selftest_wait_timeout(int32_t probes, int32_t* dev_status, void* stream);

/*
 * FP32 rate probe (the paper has no counterpart; a measurement aid).  `blocks` CTAs of 256 threads run `iters` steps of
 * eight independent dependent-chains per thread, in registers only.  mode 0: two scalar adds per chain and step;
 * 1: one packed add.f32x2; 2: the instruction mix of the sign pass of App. A as this library runs it (two saturating
 * multiply-adds, two packed multiply-adds: 6 lane-operations); 3: the mix of the l1 forward (one packed subtract, two
 * |.| accumulations: 4 lane-operations); 4: mix 2 with its scalar and packed instructions in separate runs; 5: mix 2
 * with scalar instructions only.  ln_fp32_add_probe_lane_ops returns the lane-operations of such a launch;
 * divided by its duration it is the measured counterpart of the derived FP32 peak (SMs x 128 lanes x clock), for plain
 * adds and for the two mixes the ALU-bound kernels are made of.  sink: device fp32 [1025], sink[0] is read.
 */
int ln_fp32_add_probe(int32_t blocks, int32_t iters, int32_t mode, float* sink, void* stream);
int64_t ln_fp32_add_probe_lane_ops(int32_t blocks, int32_t iters, int32_t mode);

/*
 * Profiling aid, off by default and not thread-safe (the paper has no counterpart; Sec. 4.3 only
 * reports kernel times).  Between ln_trace_begin and ln_trace_end every kernel the library
 * launches is bracketed by two CUDA events on its stream.  ln_trace_end synchronises the device,
 * writes the number of traced launches to *count and, for the first `capacity` of them, the
 * duration in milliseconds to ms[i] and a static name to names[i] (either array may be NULL).
 * These two calls create and destroy CUDA events.
 */
int ln_trace_begin(void);
int ln_trace_end(int32_t capacity, int32_t* count, float* ms, const char** names);

/*
 * Overlap of the per-head kernels with the token-sized ones (the paper has no counterpart; Alg. 1
 * fixes the data flow only).  Newton-Schulz needs nothing but W = k(L,L), and its adjoint and
 * the landmark-block gradient nothing but Z'^T dO, so laplace_nystrom_fwd / _bwd (bf16 storage)
 * enqueue them on a second stream that belongs to the library: forked from `stream` by an event
 * after the kernels they depend on, joined back into `stream` by an event before the first
 * kernel that needs their results.  Seen from the caller all work is ordered on `stream` as
 * before.  enabled = 0 keeps every launch on `stream`; the default is 1.  Returns the previous
 * setting.  While a trace is being recorded the overlap is off, so that each launch is timed
 * running alone.
 */
int ln_set_overlap(int enabled);

/*
 * Which sign pass the bf16 backward uses for the two token-sized kernel blocks (the paper has no counterpart; App. A
 * fixes the arithmetic only).  1 (default): one kernel per block forms the upstream factor g = (U Y^T) o A / lambda
 * on the tensor cores and consumes it in place.  0: the upstream factors are written to the workspace by separate
 * product kernels and read back by the sign pass (the earlier arrangement, kept for comparison).  Both give the same
 * gradients up to rounding order.  The setting is read when sizes are computed and when a call is planned: set it
 * before laplace_nystrom_workspace_bytes and keep it for the calls that use that workspace.  Returns the previous value.
 */
int ln_set_fused_sign(int enabled);

/*
 * Number of kernels this library has launched in the process so far (the paper has no counterpart; a bookkeeping aid
 * for benchmarks that report how many launches a timed region held: read it before and after).
 */
uint64_t ln_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* LAPLACE_NYSTROM_H_ */
