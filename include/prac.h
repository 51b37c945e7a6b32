/*
 * prac.h -- C ABI of the PRAC activation-compression library for NVIDIA B200 (sm_100a).
 *
 * What the library computes, per linear layer with saved input X (N tokens x d features):
 *
 *   fit        U  = orthonormal basis (d x k) of the top-k right singular subspace of X
 *                   (Section 4.2 "PAC", Section 4.3 "Construction of the Projection
 *                   Matrix", Algorithm 1 "Update Principal Subspace")
 *              Q  = Q factor, diag(R) > 0, of the thin QR of (I - U U^T) S, S_ij ~ N(0,1)
 *                   drawn from a counter-based generator keyed by (seed, draw_counter)
 *                   (Eq. "S_o = (I - Q_1 Q_1^T) S", Algorithm 1 "Update Random Subspace")
 *              c  = (d - k) / r   (Theorem "Unbiased Reconstruction of PRAC")
 *   compress   Z  = X [U | Q]                       (Algorithm 1, "Compression"; the scale
 *                                                    is kept out of the stored tensor)
 *   gradient   dW = (dY^T Z) diag(1_k, c 1_r) [U | Q]^T   (Algorithm 2 "Backward
 *                   Propagation": the ordinary dW = dY^T X~ with X~ = X P P^T of
 *                   Section 5.1, contracted without forming X~)
 *   check      X~ = Z[:, :k] U^T + c Z[:, k:] Q^T   (Algorithm 2, "Reconstruct input
 *                   approximation")
 *
 * Paper symbol -> name here:  n -> d,  r_1 -> k,  r_2 -> r,  Q_1 -> U,  Q_2 -> Q,
 * scale factor "k" -> c,  (X_1, X_2 / k) -> Z,  nabla_W -> dW.
 *
 * Conventions
 *  - All matrices are row-major with an explicit leading dimension counted in elements.
 *  - "device" pointers are CUDA device memory owned by the caller; "host" pointers are
 *    ordinary process memory.  The library never allocates or frees device memory: the
 *    basis storage and every workspace are sized by the *_bytes() queries and passed in.
 *  - Calls enqueue work on `stream` (a cudaStream_t passed as void*; NULL = default
 *    stream) and return without waiting.  Host-detectable argument errors are reported by
 *    the return code before anything is launched.  Numerical breakdown or an expired
 *    bounded wait inside a kernel is recorded in a device status word read by
 *    prac_device_status().  No call traps, aborts or throws.
 *  - dtype (prac_params.dtype) is the storage type of X, dY and Z.  PRAC_BF16 accumulates
 *    in fp32 on the tensor cores; PRAC_F32 runs fp32 FMA kernels.
 *  - Tensor-core kernels are used when the operand rows are 16-byte aligned (base pointer
 *    and leading dimension * element size multiples of 16 bytes).  A bf16 X (prac_compress,
 *    prac_fit*) or dY (prac_weight_grad*) whose base is 16-byte aligned but whose leading
 *    dimension is not a multiple of 8, e.g. a contiguous N x 5461 matrix (and likewise the dY and
 *    dX of the fused backward passes below), also runs at
 *    tensor-core speed: the rows are fetched in groups that share one offset from the 16-byte
 *    grid.  That path reads a few elements of the neighbouring rows as padding, so the
 *    matrix must hold finite numbers throughout, and its results equal those of the aligned
 *    layout up to the order of the fp32 sums.  Any other layout is served by slower kernels
 *    with identical semantics.
 *  - The CUDA context/device current at prac_basis_create() must be current in later calls.
 */
#ifndef PRAC_H_
#define PRAC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  PRAC_OK = 0,
  PRAC_EINVAL = 1,      /* bad argument (null pointer, negative size, k + r > d, ...)   */
  PRAC_EWORKSPACE = 2,  /* workspace or basis storage smaller than the query says        */
  PRAC_EALIGN = 3,      /* storage handed to the library is not 256-byte aligned         */
  PRAC_ENUMERIC = 4,    /* orthonormalisation / eigen-solver breakdown (device status)   */
  PRAC_ETIMEOUT = 5,    /* a bounded wait inside a kernel expired (device status)        */
  PRAC_ECUDA = 6,       /* a CUDA runtime or driver call failed                          */
  PRAC_ESTATE = 7       /* basis not ready: no U/Q fitted, or Q stale after a new U      */
} prac_status;

typedef enum { PRAC_BF16 = 0, PRAC_F32 = 1 } prac_dtype;

typedef struct {
  int64_t d;           /* feature dimension of X (paper: n)                               */
  int64_t k;           /* principal rank (paper: r_1), 0 <= k                             */
  int64_t r;           /* random rank (paper: r_2), 0 <= r, 1 <= k + r <= d               */
  int32_t dtype;       /* prac_dtype of X, dY, Z                                          */
  int32_t oversample;  /* extra columns p of the subspace iteration, 0 = max(32, k/4)     */
  int32_t iters;       /* subspace iterations q, 0 = default (4)                          */
  int32_t reserved;    /* must be 0                                                       */
} prac_params;

typedef struct prac_basis prac_basis; /* host handle; its device arrays live in caller memory */

/* Library version (major * 1000 + minor). */
int prac_version(void);
/* Number of CUDA kernels this library has launched so far in this process (host counter,
 * all entry points together).  Lets a caller assert that the CUDA path is what ran. */
uint64_t prac_kernel_launches(void);
/* Test hook: poll limit of the bounded grid barriers inside the cooperative kernels of the fit
 * (Cholesky factorisation, eigen-solver).  A limit of 1 makes the first CTA to reach a barrier
 * give up at once: every CTA then leaves through its normal exit and prac_device_status()
 * returns PRAC_ETIMEOUT; 0 restores the default (about 4 million polls).  Process-wide. */
void prac_debug_set_barrier_poll_limit(uint32_t polls);
/* Bounds-checking build (libprac_dbg.so, compiled with -DPRAC_DEBUG_BOUNDS; it stands in for a memory
 * checker where none can be run): the kernels that compute their own global-memory indices check
 * each one against the extent of its buffer, count the ones outside and skip those accesses.
 * Returns that count for the current device since the library was loaded (after waiting for the
 * device), -1 in the normal build, -2 if the count cannot be read. */
int64_t prac_debug_bounds_violations(void);
/* Static string for a status code. */
const char* prac_status_string(int status);

/* Device bytes a basis needs (fp32 [U|Q], its bf16 copies, status word).  0 on bad params. */
size_t prac_basis_bytes(const prac_params* params);
/* Device workspace bytes for prac_fit_basis / prac_fit_principal / prac_draw_random on an
 * input of N tokens.  0 on bad params. */
size_t prac_fit_workspace_bytes(const prac_params* params, int64_t N);
/* Device workspace bytes for prac_weight_grad with N tokens and d_out output features. */
size_t prac_grad_workspace_bytes(const prac_params* params, int64_t N, int64_t d_out);

/* Create a basis handle over `dev_mem` (device, 256-byte aligned, >= prac_basis_bytes()).
 * The memory stays owned by the caller and must outlive the handle.  Synchronous (clears the
 * storage on the default stream and waits). */
int prac_basis_create(prac_basis** out, const prac_params* params, void* dev_mem, size_t bytes);
/* Free the host handle (device memory is the caller's). */
void prac_basis_destroy(prac_basis* basis);

/* Algorithm 1 without its last line: fit U on X (device, N x d, leading dimension ldx),
 * draw S from (seed, draw_counter), build Q and c.  Equivalent to prac_fit_principal
 * followed by prac_draw_random.  ws: device workspace (256-byte aligned). */
int prac_fit_basis(prac_basis* basis, const void* X, int64_t N, int64_t ldx,
                   uint64_t seed, uint64_t draw_counter,
                   void* ws, size_t ws_bytes, void* stream);
/* Algorithm 1 "Update Principal Subspace" only (interval T_1): Gram matrix X^T X, randomized
 * subspace iteration with Cholesky-QR re-orthonormalisation, Rayleigh-Ritz.  The start
 * block is drawn from (seed, draw_counter) on a stream disjoint from the one Q uses.
 * Marks Q stale: a new Q must be drawn against the new U before compress is allowed. */
int prac_fit_principal(prac_basis* basis, const void* X, int64_t N, int64_t ldx,
                       uint64_t seed, uint64_t draw_counter,
                       void* ws, size_t ws_bytes, void* stream);
/* The update for a basis that already holds a U (the lazy-update schedule of Algorithm 1
 * refreshes U every T_1 steps on activations whose statistics move slowly, Section 5.1 "Lazy
 * update"): orthogonal iteration started from the current U, U <- orth((X^T X) U), `iters` times
 * (0 = 2), without oversampling columns and without the Rayleigh-Ritz eigen-solve.  Each iteration
 * can only raise the captured energy ||X U||_F^2 and shrinks the error a drift of the data left
 * in span(U) by lambda_{k+1} / lambda_k; it costs less than half of a cold fit.  seed and
 * draw_counter are accepted for symmetry and not used (nothing is drawn).  Arguments, workspace
 * and effects (Q becomes stale) as for prac_fit_principal.  PRAC_ESTATE if the basis has no U yet. */
int prac_refresh_principal(prac_basis* basis, const void* X, int64_t N, int64_t ldx,
                           uint64_t seed, uint64_t draw_counter, int32_t iters,
                           void* ws, size_t ws_bytes, void* stream);
/* Building blocks for a batch whose tokens are spread over several devices (data parallel, as in
 * the paper's 4-GPU "Training Efficiency" runs; the paper does not say how the subspaces are
 * shared between devices, this is one way): both the Gram matrix of Algorithm 1's principal fit and the
 * middle factor dY^T Z of the weight gradient are sums over tokens, so each rank computes its
 * part, the parts are summed by the caller's collective (the library calls none), and every rank
 * finishes from the sum.  With one seed and draw counter all ranks then hold the same U and Q.
 *   prac_gram:                C (device, d x d fp32, ldc) = X^T X of this rank's N tokens.
 *                             ws as for prac_fit_principal with the same N.
 *   prac_fit_principal_gram:  the principal fit from a given Gram matrix (not modified).
 *                             ws: prac_fit_workspace_bytes(params, 1) or more.
 *   prac_weight_grad_partial: M (device, d_out x (k+r) fp32, ldm) = dY^T Z of this rank's tokens,
 *                             unscaled.  ws: prac_grad_workspace_bytes.
 *   prac_weight_grad_finish:  dW = (M diag(1_k, c 1_r)) [U|Q]^T from a (summed) M; arguments as
 *                             prac_weight_grad.  ws: d_out * round_up(k+r, 8) * 2 bytes (bf16),
 *                             not used for fp32 storage.
 * Summing M moves d / (k+r) times fewer bytes than summing dW. */
int prac_gram(const prac_basis* basis, const void* X, int64_t N, int64_t ldx, float* C, int64_t ldc,
              void* ws, size_t ws_bytes, void* stream);
int prac_fit_principal_gram(prac_basis* basis, const float* C, int64_t ldc, uint64_t seed,
                            uint64_t draw_counter, void* ws, size_t ws_bytes, void* stream);
int prac_weight_grad_partial(const prac_basis* basis, const void* dY, int64_t lddy, int64_t d_out,
                             const void* Z, int64_t ldz, int64_t N, float* M, int64_t ldm,
                             void* ws, size_t ws_bytes, void* stream);
int prac_weight_grad_finish(const prac_basis* basis, const float* M, int64_t ldm, int64_t d_out,
                            double c_override, void* dW, int64_t lddw, int32_t dw_dtype,
                            int32_t accumulate, void* ws, size_t ws_bytes, void* stream);

/* Algorithm 1 "Update Random Subspace" only (interval T_2): S from (seed, draw_counter),
 * projected off the current U, orthonormalised with positive diagonal of R; sets c. */
int prac_draw_random(prac_basis* basis, uint64_t seed, uint64_t draw_counter,
                     void* ws, size_t ws_bytes, void* stream);
/* Install an externally computed basis (e.g. a checkpoint): U (device fp32, d x k, ldu),
 * Q (device fp32, d x r, ldq) and c.  U or Q may be NULL when k or r is 0. */
int prac_set_basis(prac_basis* basis, const float* U, int64_t ldu, const float* Q, int64_t ldq,
                   double c, void* stream);
/* Borrow the fp32 master copy P = [U | Q] (device, d x (k+r), leading dimension *ldp) and c.
 * Any out-pointer may be NULL. */
int prac_basis_get(const prac_basis* basis, const float** P, int64_t* ldp, double* c);

/* Algorithm 1 "Compression": Z (device, N x (k+r), ldz, dtype) = X (device, N x d, ldx) [U|Q]. */
int prac_compress(const prac_basis* basis, const void* X, int64_t N, int64_t ldx,
                  void* Z, int64_t ldz, void* stream);
/* Algorithm 2 forward of one linear layer, both products of X in one pass: Y (device,
 * N x d_out, ldy, dtype) = X W^T with W (device, d_out x d, ldw, dtype; the orientation of
 * nn.Linear.weight) and Z = X [U|Q] as prac_compress.  For bf16 with 16-byte aligned rows
 * this is one kernel launch that reads every row of X once for both outputs; otherwise it
 * is the two products one after the other.  Y and Z must not overlap X or each other.
 * Z may be NULL (only Y is computed): of several linears that share an input, one call
 * produces the shared Z and the others pass NULL.  Same errors as prac_compress. */
int prac_linear_forward(const prac_basis* basis, const void* X, int64_t N, int64_t ldx,
                        const void* W, int64_t ldw, int64_t d_out, void* Y, int64_t ldy,
                        void* Z, int64_t ldz, void* stream);
/* Section 5.1 "Layer-Wise Design", non-linear layers: backward of an element-wise activation
 * y = f(x) whose input x (N x d) was stored compressed.  dX (device, N x d, lddx, dtype) =
 * dY (device, N x d, lddy, dtype) * f'(X^), with X^ = Z_k U^T + c Z_r Q^T as prac_reconstruct.
 * act: PRAC_ACT_SILU (f = x sigmoid(x)) or PRAC_ACT_GELU (f = x Phi(x), erf form).
 * bf16: X^ is formed tile by tile in tensor memory and consumed there, it is never written out;
 * Z needs 16-byte aligned rows; dY and dX either have 16-byte aligned rows too, or 16-byte aligned
 * bases and leading dimensions that are equal modulo 8 (two contiguous N x d matrices of odd d),
 * with N a multiple of 8 / gcd(lddy, 8) and N, d > 128 (PRAC_EALIGN otherwise); ws may be NULL.  fp32: X^ goes
 * through ws (prac_activation_workspace_bytes, 256-byte aligned).  dX may not overlap Z or dY. */
enum { PRAC_ACT_SILU = 0, PRAC_ACT_GELU = 1 };
int prac_activation_backward(const prac_basis* basis, const void* Z, int64_t ldz,
                             const void* dY, int64_t lddy, int64_t N, int32_t act,
                             void* dX, int64_t lddx, void* ws, size_t ws_bytes, void* stream);
size_t prac_activation_workspace_bytes(const prac_params* params, int64_t N);
/* Section 5.1, non-linear layers: backward of RMSNorm y_t = gain * x_t * rstd_t whose input x
 * (N x d) was stored compressed; rstd (device, N floats: (mean_i x_ti^2 + eps)^-1/2 of the true
 * input, kept uncompressed as the paper keeps such statistics) and gain (device, d floats).
 * With X^ rebuilt from Z as prac_reconstruct:
 *   dgain_i = sum_t dY_ti X^_ti rstd_t                         (device, d floats, overwritten)
 *   dX_t    = rstd_t (gain * dY_t) - (rstd_t^3 / d) X^_t sum_i gain_i dY_ti X^_ti   (N x d, lddx, dtype)
 * bf16: two passes of the tensor-core kernel over X^ (never written out; N > 128 and d > 128,
 * PRAC_EINVAL otherwise; layouts of Z, dY, dX as for prac_activation_backward, PRAC_EALIGN otherwise) with fixed-order
 * reductions between them.  fp32: X^ goes through the workspace.  ws: prac_rmsnorm_workspace_bytes,
 * 256-byte aligned.  dX may not overlap Z or dY. */
int prac_rmsnorm_backward(const prac_basis* basis, const void* Z, int64_t ldz, const void* dY, int64_t lddy,
                          int64_t N, const float* rstd, const float* gain, void* dX, int64_t lddx,
                          float* dgain, void* ws, size_t ws_bytes, void* stream);
size_t prac_rmsnorm_workspace_bytes(const prac_params* params, int64_t N);
/* The same for LayerNorm y_t = gain * (x_t - mean_t) * rstd_t + bias (mean, rstd: device, N floats
 * each, statistics of the true input, which are kept uncompressed: Section 5.1, Layer-Wise
 * Design).  With xn_t = (X^_t - mean_t) rstd_t and a_t = gain * dY_t:
 *   dbias_i = sum_t dY_ti,   dgain_i = sum_t dY_ti xn_ti,
 *   dX_t = rstd_t [a_t - mean_i(a_t) - xn_t mean_i(a_ti xn_ti)].
 * Restrictions, workspace and errors as prac_rmsnorm_backward (prac_layernorm_workspace_bytes). */
int prac_layernorm_backward(const prac_basis* basis, const void* Z, int64_t ldz, const void* dY, int64_t lddy,
                            int64_t N, const float* mean, const float* rstd, const float* gain,
                            void* dX, int64_t lddx, float* dgain, float* dbias,
                            void* ws, size_t ws_bytes, void* stream);
size_t prac_layernorm_workspace_bytes(const prac_params* params, int64_t N);
/* Algorithm 2 backward, weight part: dW (device, d_out x d, lddw, dw_dtype) =
 * (dY^T Z) diag(1_k, c 1_r) [U|Q]^T, with dY (device, N x d_out, lddy, dtype) and
 * Z (device, N x (k+r), ldz, dtype).  c_override: NaN = use the basis' c.
 * accumulate != 0 adds into dW instead of overwriting it. */
int prac_weight_grad(const prac_basis* basis, const void* dY, int64_t lddy, int64_t d_out,
                     const void* Z, int64_t ldz, int64_t N, double c_override,
                     void* dW, int64_t lddw, int32_t dw_dtype, int32_t accumulate,
                     void* ws, size_t ws_bytes, void* stream);
/* (No counterpart in the paper: a packaging variant of prac_weight_grad.)
 * Same result as prac_weight_grad, for callers that have no device workspace to pass and
 * cannot allocate one: code that runs where cudaMalloc is not permitted or not available,
 * such as a plug-in inside a host application that owns all device memory, a latency-critical
 * loop that must not touch the allocator, or a thin C caller without a memory pool.  The
 * scratch (the bf16 matrix between the two stages and the fp32 split-K partial tiles) is a
 * fixed array of prac_static_scratch_bytes() bytes (32 MiB) in device global memory that
 * belongs to the library image: every GPU on which the library is used holds it until the
 * process exits.  The call allocates and frees nothing.
 *  - A problem that needs more scratch than the array holds (compare
 *    prac_grad_workspace_bytes() with prac_static_scratch_bytes()) is rejected with
 *    PRAC_EWORKSPACE before anything is launched.
 *  - The first call on each device looks up the array's device address (with that device
 *    current); make that first call outside any stream capture.
 *  - All calls on a device share the one array, and it keeps whatever the previous call left:
 *    nothing in it needs clearing (every scratch element is written before it is read within
 *    a call), but two calls whose kernels overlap on the GPU (different streams, or different
 *    host threads) race on it.  Serialise them on one stream.
 * Inputs, outputs and all other arguments are those of prac_weight_grad. */
size_t prac_static_scratch_bytes(void);
int prac_weight_grad_static(const prac_basis* basis, const void* dY, int64_t lddy, int64_t d_out,
                            const void* Z, int64_t ldz, int64_t N, double c_override,
                            void* dW, int64_t lddw, int32_t dw_dtype, int32_t accumulate,
                            void* stream);
/* Algorithm 2 "Reconstruct input approximation" (for checking): Xhat (device fp32,
 * N x d, ldxh) = Z[:, :k] U^T + c Z[:, k:] Q^T. */
int prac_reconstruct(const prac_basis* basis, const void* Z, int64_t ldz, int64_t N,
                     float* Xhat, int64_t ldxh, void* stream);

/* What the last principal fit on workspace `ws` (the one passed to prac_fit_basis /
 * prac_fit_principal / prac_refresh_principal with the same N) did; waits for `stream`.
 * panel_cols = columns l of the subspace-iteration panel, iterations = q; the Rayleigh-Ritz
 * eigenproblem (Section 4.3, "via SVD") is solved on the last eig_size columns of the panel, the
 * first window_first columns going into U as they are; jacobi_sweeps = sweeps the eigen-solver ran
 * (a nearly diagonal matrix, as after a warm-started refresh, needs fewer). */
typedef struct {
  int32_t panel_cols, iterations, eig_size, window_first, jacobi_sweeps, reserved[3];
} prac_fit_info;
int prac_fit_report(const prac_basis* basis, void* ws, size_t ws_bytes, int64_t N, void* stream,
                    prac_fit_info* out);

/* Wait for `stream`, read and clear the device status word of the basis (the first four bytes
 * of the basis storage; kernels set bits in it, nothing else reads it).  Returns PRAC_OK,
 * PRAC_ETIMEOUT (a bounded wait inside a kernel gave up; every kernel still left through its
 * normal exit and the basis can be fitted again), PRAC_ENUMERIC or PRAC_ECUDA.
 * PRAC_ENUMERIC means that the orthonormalisation of the fit or of the draw met a pivot that was
 * not positive and that the extra pass which then re-orthonormalises the panel broke down as
 * well (e.g. X = 0), or that the eigen-solver ran out of sweeps: the basis is not to be used.  A
 * rank-deficient X (rank below k, fewer tokens than features) is not an error: U is completed
 * to an orthonormal d x k matrix. */
int prac_device_status(prac_basis* basis, void* stream);

/* The raw generator, exposed so the stream can be checked bit for bit: out (device,
 * n uint32 words) = the word of each of the first n entries of draw (seed, draw_counter):
 * entry e takes lane e&3 of Philox4x32-10 with counter (lo(e>>2), hi(e>>2),
 * lo(draw_counter), hi(draw_counter)) and key (lo(seed), hi(seed)). */
int prac_philox_words(uint64_t seed, uint64_t draw_counter, int64_t n, uint32_t* out, void* stream);
/* S (device fp32, d x r, lds): Box-Muller on the 23-bit uniforms of those words. */
int prac_gaussian(uint64_t seed, uint64_t draw_counter, int64_t d, int64_t r,
                  float* S, int64_t lds, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* PRAC_H_ */
