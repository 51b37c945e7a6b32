// Declarations shared by the translation units of libprac (host side).
#pragma once
#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>
#include <cuda_bf16.h>

#include "../../include/prac.h"

namespace prac {

// Bits of the device status word (set by kernels, read by prac_device_status).
enum : int {
  DEV_CHOL_PIVOT = 1,      // Cholesky pivot not positive in a final pass, also after the extra pass
  DEV_JACOBI_NOCONV = 2,   // Jacobi sweeps ran out before the rotations stopped
  DEV_WAIT_EXPIRED = 4,    // a bounded wait (mbarrier, grid barrier) gave up
  DEV_CHOL_RETRY = 8       // internal: a final Cholesky-QR pass met a bad pivot; the extra pass that
                           // follows it runs only while this bit is set, and clears it
};

// Poll limit of the grid barriers of the cooperative kernels (default GRID_BARRIER_POLLS; a test
// hook lowers it to make a barrier give up).
unsigned barrier_poll_limit();

// Number of kernels this library has launched in the process (reported by
// prac_kernel_launches so callers can check that the CUDA path is the one that ran).
void count_launch(int n = 1);

inline int64_t round_up(int64_t x, int64_t m) { return (x + m - 1) / m * m; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Build flag PRAC_DEBUG_BOUNDS (a second library, libprac_dbg.so): every global-memory index of the
// kernels that address memory themselves (everything except the TMA-fed tensor-core GEMM, whose
// tensor maps clip in hardware) is checked against the extent of its buffer before the access.  An
// index outside is counted, its source line kept, and the access skipped; nothing traps.  The
// count is read with prac_debug_bounds_violations().  In the normal build the macro is `true`
// and costs nothing.
#if defined(PRAC_DEBUG_BOUNDS) && defined(__CUDACC__)
// (one counter per translation unit: the library is built without relocatable device code)
static __device__ unsigned long long g_bounds_violations;
static __device__ int g_bounds_first_line;
__device__ __forceinline__ bool dbg_in_bounds(long long idx, long long limit, int line) {
  if (idx >= 0 && idx < limit) return true;
  if (atomicAdd(&g_bounds_violations, 1ull) == 0ull) g_bounds_first_line = line;
  return false;
}
#define PRAC_IN(idx, limit) ::prac::dbg_in_bounds(static_cast<long long>(idx), static_cast<long long>(limit), __LINE__)
// Defines `long long name()`: this translation unit's count (-1 if it cannot be read).
#define PRAC_BOUNDS_READER(name)                                                                          \
  long long name() {                                                                                      \
    unsigned long long v = 0;                                                                             \
    if (cudaMemcpyFromSymbol(&v, g_bounds_violations, sizeof(v)) != cudaSuccess) return -1;               \
    return static_cast<long long>(v);                                                                     \
  }
#else
#define PRAC_IN(idx, limit) true
#define PRAC_BOUNDS_READER(name) \
  long long name() { return 0; }
#endif
long long bounds_violations_simt();
long long bounds_violations_panel();
long long bounds_violations_cholqr();
long long bounds_violations_tc();

#define PRAC_CUDA_TRY(expr)                        \
  do {                                             \
    cudaError_t e_ = (expr);                       \
    if (e_ != cudaSuccess) return PRAC_ECUDA;      \
  } while (0)

// ------------------------------------------------------------------ general (FMA) GEMM
// C[M x N] = alpha * op(A)[M x K] * op(B)[K x N] + beta * C, row-major storage:
//   trans_a == 0: A is M x K (lda >= K);  trans_a == 1: A is stored K x M (lda >= M)
//   trans_b == 0: B is K x N (ldb >= N);  trans_b == 1: B is stored N x K (ldb >= K)
// Element types: 0 = float, 1 = bf16, 2 = double.  Accumulation is in double when
// acc_double != 0, else float.  Elements of op(A) with K-index >= kscale_from are
// multiplied by kscale (used for the diag(1, c) factor).
enum ElemType : int { ET_F32 = 0, ET_BF16 = 1, ET_F64 = 2 };
struct GemmArgs {
  int64_t M, N, K;
  const void* A; int64_t lda; int type_a; int trans_a;
  const void* B; int64_t ldb; int type_b; int trans_b;
  void* C; int64_t ldc; int type_c;
  double alpha, beta;
  int acc_double;
  int64_t kscale_from; double kscale;
  const int* run_if = nullptr;   // optional: the kernel does nothing unless *run_if & run_if_mask
  int run_if_mask = 0;
};
int gemm_general(const GemmArgs& g, cudaStream_t stream);

// ------------------------------------------------------------------ tensor-core GEMMs
// Library-wide set-up of the driver entry point used to encode TMA descriptors.
int tc_init();
int tc_num_sms();

// Z-like product with both operands K-major: C[M x N] = A[M x K] * B[N x K]^T.
// A, B bf16, 16-byte aligned rows.  C bf16 or fp32 (type_c), optional accumulate (fp32 only).
// segs != nullptr: A and B rows hold several K-long pieces side by side (rows_a / rows_b elements
// wide); segment g multiplies the piece of A at column off_a[g] by the piece of B at column
// off_b[g], all into one accumulation (K a multiple of 64).
// A may have rows that are not 16-byte aligned (any leading dimension, 2-byte aligned base) when
// tc_kmajor_takes_unaligned_a(M, N) holds, the output is bf16 and there are no segments: it is then
// fetched with plain loads instead of TMA.  B and C as before.
bool tc_kmajor_takes_unaligned_a(int64_t M, int64_t N);
// C (bf16) = A * Bmn with A (M x K, K-major) whose row pitch is not a multiple of 8 elements and Bmn
// (K x N) row-major: A is fetched by TMA through one tensor map per class of rows with the same
// offset from the 16-byte grid.  tc_rowclass_fits says whether A and the shape suit it; the other
// operands need 16-byte aligned rows.  A must hold finite numbers.
bool tc_rowclass_fits(const void* A, int64_t lda, int64_t M, int64_t N);
int tc_gemm_kmajor_rowclass(const __nv_bfloat16* A, int64_t lda, const __nv_bfloat16* Bmn, int64_t ldb, int64_t M,
                            int64_t N, int64_t K, __nv_bfloat16* C, int64_t ldc, int* dev_status, cudaStream_t stream);
bool tc_tokens_takes_unaligned_a(int64_t M, int64_t N);
struct TcSegments;
int tc_gemm_kmajor(const __nv_bfloat16* A, int64_t lda, const __nv_bfloat16* B, int64_t ldb,
                   int64_t M, int64_t N, int64_t K, void* C, int64_t ldc, int type_c,
                   int accumulate, int* dev_status, cudaStream_t stream, const struct TcSegments* segs = nullptr);

// dX[M x N] (bf16) = dY[M x N] (bf16) * f'(A B^T), the product formed tile by tile and never stored;
// act: 0 = SiLU, 1 = GeLU (erf form).  A (M x K), B (N x K) bf16 K-major, rows of dY 16-byte aligned.
int tc_gemm_kmajor_act(const __nv_bfloat16* A, int64_t lda, const __nv_bfloat16* B, int64_t ldb,
                       int64_t M, int64_t N, int64_t K, const __nv_bfloat16* dY, int64_t lddy, int act,
                       __nv_bfloat16* dX, int64_t lddx, int* dev_status, cudaStream_t stream);

// RMSNorm backward over x = A B^T (M x N, never stored), dY bf16 (M x N).  pass 1 writes
// row_part[(2 nt + h) * M + t] (partial sums over column blocks of col_g[i] dY[t][i] x[t][i];
// tc_gemm_kmajor_rms_parts(N) parts) and col_part[(t / 32) * N + i] (sums over 32 rows of
// row_a[t] dY[t][i] x[t][i]); pass 2 writes dX = row_a[t] col_g[i] dY[t][i] - row_b[t] x[t][i].
int tc_gemm_kmajor_rms(int pass, const __nv_bfloat16* A, int64_t lda, const __nv_bfloat16* B, int64_t ldb,
                       int64_t M, int64_t N, int64_t K, const __nv_bfloat16* dY, int64_t lddy,
                       const float* row_a, const float* row_b, const float* col_g, float* row_part, float* col_part,
                       __nv_bfloat16* dX, int64_t lddx, int* dev_status, cudaStream_t stream,
                       float* row_part2 = nullptr, const float* row_c = nullptr);
// (LayerNorm: pass 1 with row_part2 also leaves the sums of col_g[i] dY[t][i]; pass 2 with row_c
// adds row_c[t] to row t.)
int tc_gemm_kmajor_rms_parts(int64_t N, int64_t lddy);
// 32-row blocks pass 1 writes column partials for (more than M / 32 when dY is taken by classes of rows)
int64_t tc_gemm_kmajor_rms_blocks(int64_t M, int64_t lddy);
// Whether the fused consumers take a factor dY (and output dX, may be NULL) with these row pitches:
// 16-byte aligned rows, or rows off the grid that classes of rows cover (bases aligned, same offsets, M a
// multiple of the class count)
bool tc_consumer_takes_rows(const void* dY, int64_t lddy, const void* dX, int64_t lddx, int64_t M, int64_t N);
// row_b[t] = rstd[t]^3 / d * sum_p row_part[p * M + t];  dgain[i] = sum_b col_part[b * N + i]  (fixed order)
int launch_rms_reduce(const float* row_part, int parts, const float* col_part, int64_t blocks, const float* rstd,
                      int64_t M, int64_t N, float* row_b, float* dgain, cudaStream_t stream);
// LayerNorm backward: the sums that do not need the rebuilt input (per 512-token group: sum of dY
// and of rstd mean dY, per column), the reduction after pass 1, and the fp32-storage version.
int launch_ln_colsum_partial(const __nv_bfloat16* dY, int64_t lddy, const float* mean, const float* rstd, int64_t M,
                             int64_t N, float* part_plain, float* part_w, cudaStream_t stream);
int launch_ln_reduce(const float* row_part, const float* row_part2, int parts, const float* col_part, int64_t blocks,
                     const float* part_plain, const float* part_w, int64_t groups, const float* mean, const float* rstd,
                     int64_t M, int64_t N, float* row_b, float* row_c, float* dgain, float* dbias, cudaStream_t stream);
int launch_ln_backward_f32(const float* Xh, int64_t ldxh, const float* dY, int64_t lddy, const float* mean,
                           const float* rstd, const float* gain, float* dX, int64_t lddx, float* dgain, float* dbias,
                           int64_t M, int64_t N, cudaStream_t stream);
// fp32 storage: the whole backward from a rebuilt input Xh (M x N fp32)
int launch_rms_backward_f32(const float* Xh, int64_t ldxh, const float* dY, int64_t lddy, const float* rstd,
                            const float* gain, float* dX, int64_t lddx, float* dgain, int64_t M, int64_t N,
                            cudaStream_t stream);

// Two K-major products sharing A in one launch: C1[M x N1] = A B1^T and C2[M x N2] = A B2^T,
// everything bf16; A is read once.  Needs M > 128 (CTA pairs, 256 x 256 tiles).  Returns
// PRAC_EALIGN without launching when exactly one of the outputs has 16-byte-aligned rows (the
// two store paths must not meet in one launch); the caller then runs the products in turn.
int tc_gemm_kmajor_dual(const __nv_bfloat16* A, int64_t lda, int64_t M, int64_t K,
                        const __nv_bfloat16* B1, int64_t ldb1, int64_t N1, __nv_bfloat16* C1, int64_t ldc1,
                        const __nv_bfloat16* B2, int64_t ldb2, int64_t N2, __nv_bfloat16* C2, int64_t ldc2,
                        int* dev_status, cudaStream_t stream);

// Token-reduction product with both operands stored K x (M or N) row-major:
// C[M x N] = A[K x M]^T * B[K x N], K split over CTAs, fp32 partial tiles in `ws`, then an
// ordered reduction that multiplies columns >= scale_from by `scale` and writes C as fp32
// or bf16.  symmetric != 0 (requires A == B, M == N) computes only the tiles that touch
// the upper triangle and mirrors them.
// segs != nullptr chains several products into one accumulation: segment g multiplies the K rows
// of A starting at row off_a[g] by the K rows of B starting at row off_b[g] (K a multiple of 64;
// rows_a / rows_b = rows of the stacked operands).  Used to multiply fp32 matrices held as
// stacks of bf16 pieces (hi, mid, lo) to fp32 accuracy.
constexpr int TC_MAX_SEGMENTS = 6;
struct TcSegments { int n; int64_t off_a[TC_MAX_SEGMENTS], off_b[TC_MAX_SEGMENTS]; int64_t rows_a, rows_b; };
size_t tc_gemm_tokens_ws_bytes(int64_t M, int64_t N, int64_t K, int symmetric, int nseg = 1);
// Workspace with which tc_gemm_tokens takes an A whose row pitch lda is not a multiple of 8 elements
// by classes of rows through TMA (one partial product per class); 0 when that path does not apply.
size_t tc_gemm_tokens_rowclass_ws_bytes(int64_t lda, int64_t M, int64_t N, int64_t K);
// planes != nullptr (symmetric fp32 products only): the result also, or only (C == nullptr), leaves
// as the stack of three bf16 pieces launch_split3 would make of it: piece q at base + q * rows_pad * ld,
// rows_pad x ld each (both multiples of 64, >= M), zero outside the M x M matrix.
struct TcPlanes { __nv_bfloat16* base; int64_t rows_pad, ld; };
int tc_gemm_tokens(const __nv_bfloat16* A, int64_t lda, const __nv_bfloat16* B, int64_t ldb,
                   int64_t M, int64_t N, int64_t K, void* C, int64_t ldc, int type_c,
                   int64_t scale_from, float scale, int symmetric, const TcSegments* segs,
                   void* ws, size_t ws_bytes, int* dev_status, cudaStream_t stream,
                   const TcPlanes* planes = nullptr);

// dst = src (rows x cols fp32, leading dimension lds) as a stack of three bf16 matrices
// hi | mid | lo with hi + mid + lo = src to about 2^-24: piece q occupies rows
// [q * rows_pad, q * rows_pad + rows) of dst (leading dimension ldd); rows up to rows_pad and
// columns up to ldd are zero.
int launch_split3(const float* src, int64_t lds, int64_t rows, int64_t cols, __nv_bfloat16* dst,
                  int64_t rows_pad, int64_t ldd, cudaStream_t stream);
// The same three pieces side by side in each row: dst (rows x 3 kp bf16) = [hi | mid | lo], each kp
// (a multiple of 8, >= cols) wide, zero beyond cols.
// dst (cols x 3 kp, bf16) = the transpose of scale * src (rows x cols, fp32) in three pieces per element
int launch_split3_transposed(const float* src, int64_t lds, int64_t rows, int64_t cols, float scale,
                             __nv_bfloat16* dst, int64_t kp, cudaStream_t stream);
// C (d x n, fp32) = [C +] scale * A (d x kd) * B (kd x n), fp32 operands, on the tensor cores as three
// bf16 pieces per operand (general kernel for small panels or without workspace)
size_t panel_mm3_ws_bytes(int64_t d, int64_t kd, int64_t n);
int panel_mm3(const float* A, int64_t lda, const float* B, int64_t ldb, int64_t d, int64_t kd, int64_t n, float scale,
              float* C, int64_t ldc, int accumulate, void* ws, size_t ws_bytes, int* dev_status, cudaStream_t stream);
int launch_split3_cols(const float* src, int64_t lds, int64_t rows, int64_t cols, __nv_bfloat16* dst,
                       int64_t kp, cudaStream_t stream);

// ------------------------------------------------------------------ panel / RNG kernels
int launch_philox_words(uint64_t seed, uint64_t draw_counter, int64_t n, uint32_t* out,
                        cudaStream_t stream);
int launch_gaussian(uint64_t seed, uint64_t draw_counter, int64_t d, int64_t r, float* S,
                    int64_t lds, cudaStream_t stream);

// out (m x n, leading dimension ldo, double if out_double else float) = alpha * A^T B for fp32
// A (d x m, lda) and B (d x n, ldb), accumulated in double over row slices that are summed in a
// fixed order.  symmetric != 0 (A == B, m == n) computes the upper tiles and mirrors them.
// ws >= atb_ws_bytes(m, n, d, symmetric).
size_t atb_ws_bytes(int64_t m, int64_t n, int64_t d, int symmetric);
// run_if != nullptr: both kernels return at once unless *run_if & run_if_mask (a device word).
// zero_after: up to 1 KB (a multiple of 4 bytes) that the second kernel sets to zero.
int atb_f64(const float* A, int64_t lda, const float* B, int64_t ldb, int64_t d, int64_t m, int64_t n,
            int symmetric, double alpha, void* out, int64_t ldo, int out_double, void* ws, size_t ws_bytes,
            cudaStream_t stream, const int* run_if = nullptr, int run_if_mask = 0, void* zero_after = nullptr,
            int zero_bytes = 0);

// One Cholesky-QR pass: Vout (d x n, ldout) = Vin (d x n, ldin) R^-1 with R^T R = Vin^T Vin, the
// Gram matrix accumulated and factored in double.  R has a positive diagonal.  Vout != Vin.
// A pivot that is not safely positive is replaced by a guard value and, when flag_bit != 0,
// reported in *dev_status.  run_if_mask != 0 makes the pass optional: its kernels are launched
// but do nothing unless *dev_status has one of those bits when they start (Vout is then left
// untouched).
size_t cholqr_ws_bytes(int64_t n, int64_t d);
int cholqr_pass(const float* Vin, int64_t ldin, float* Vout, int64_t ldout, int64_t d, int64_t n, void* ws,
                size_t ws_bytes, int* dev_status, int flag_bit, cudaStream_t stream, int run_if_mask = 0);
// Orthonormalises V (d x n) into Vout with one pass that reports a bad pivot as DEV_CHOL_RETRY,
// followed by the optional pass that this bit switches on: Vout -> tmp -> Vout, a bad pivot there
// raising DEV_CHOL_PIVOT; the bit is cleared at the end.  tmp: d x n floats, leading dimension n.
int cholqr_final(const float* Vin, int64_t ldin, float* Vout, int64_t ldout, float* tmp, int64_t d, int64_t n,
                 void* ws, size_t ws_bytes, int* dev_status, cudaStream_t stream);
// dst = src (fp32, rows x cols) and *status &= ~clear_bits afterwards, both only if *status & run_if_mask.
int launch_copy2d_if(const float* src, int64_t lds, float* dst, int64_t ldd, int64_t rows, int64_t cols,
                     int* status, int run_if_mask, int clear_bits, cudaStream_t stream);

// Eigenvectors of the k largest eigenvalues of the symmetric positive semi-definite ell x ell
// matrix B (double, leading dimension ldb; only (B + B^T)/2 is used), largest first, as the
// columns of Wsel (fp32, ell x k, row-major).  One-sided block Jacobi.
size_t jacobi_ws_bytes(int64_t ell);
// Waits for the stream and reads how many sweeps the last jacobi_topk on this workspace ran.
int jacobi_read_sweeps(void* ws, int64_t ell, int* sweeps, cudaStream_t stream);
int jacobi_topk(const double* B, int64_t ldb, int64_t ell, int64_t k, float* Wsel, void* ws, size_t ws_bytes,
                int* dev_status, cudaStream_t stream);

// bf16 copies of P (d x s fp32, ldp): Pb (d x s, ldpb) and its transpose PTb (s x d, ldptb).
// Pcb (same pitch as Pb) = [U | c Q]: columns from k on scaled by c.
int launch_make_bf16_copies(const float* P, int64_t ldp, int64_t d, int64_t s, int64_t k, double c,
                            __nv_bfloat16* Pcb, __nv_bfloat16* Pb, int64_t ldpb, __nv_bfloat16* PTb, int64_t ldptb,
                            cudaStream_t stream);
// dst (rows x cols bf16, leading dimension ldd a multiple of 8, 16-byte aligned base; zero from
// cols to ldd) = src (rows x cols bf16, any leading dimension and 2-byte alignment).
int launch_repack_rows_bf16(const __nv_bfloat16* src, int64_t lds, int64_t rows, int64_t cols, __nv_bfloat16* dst,
                            int64_t ldd, cudaStream_t stream);
// dst (rows x cols, ldd) = src (rows x cols, lds), fp32.
int launch_scale_to_bf16(const float* src, int64_t lds, int64_t rows, int64_t cols, int64_t from, float scale,
                         __nv_bfloat16* dst, int64_t ldd, cudaStream_t stream);
int launch_act_backward_f32(const float* Xh, int64_t ldxh, const float* dY, int64_t lddy, float* dX, int64_t lddx,
                            int64_t rows, int64_t cols, int act, cudaStream_t stream);
int launch_copy2d(const float* src, int64_t lds, float* dst, int64_t ldd, int64_t rows,
                  int64_t cols, cudaStream_t stream);

}  // namespace prac
