// Orthonormalisation of tall fp32 panels by Cholesky-QR, three launches per pass:
//   1. G = V^T V accumulated in double over slices of the rows (atb_f64_partial_kernel) and
//      summed in a fixed order (reduce_partials_kernel);
//   2. R = chol(G) and R^-1 in one cooperative kernel (chol_inv_kernel), all in double;
//   3. V_out = V_in * R^-1: on the tensor cores for panels big enough to fill their tiles (both
//      operands as three bf16 pieces, six chained cross terms: fp32 accuracy), else a general
//      fp32 GEMM.
// R has a positive diagonal, so V R^-1 is the unique thin-QR Q factor.  The same
// transposed-product kernel serves every small "tall^T x tall" product of the basis fit.
#include <cuda_runtime.h>

#include "grid_barrier.cuh"
#include "internal.h"
#include "per_device.h"

namespace prac {
namespace {

inline unsigned nblocks(long long work, int threads) {
  return static_cast<unsigned>((work + threads - 1) / threads);
}

// ------------------------------------------------------------------ Out = A^T B, double accumulation
constexpr int AT_T = 64;     // output tile
constexpr int AT_K = 16;     // rows per staging step

struct AtbArgs {
  const float* A; long long lda;   // d x m
  const float* B; long long ldb;   // d x n
  int m, n;
  long long d;
  int splits;                      // row slices
  int tiles_m, tiles_n, num_tiles;
  int symmetric;                   // A == B, m == n: only tiles reaching the upper triangle
  double* partial;                 // [splits][m][n]
  const int* run_if;               // optional: the kernel does nothing unless *run_if & run_if_mask
  int run_if_mask;
};

// Kernels of an optional pass are always launched and look at a device word to see whether
// they have anything to do (the host does not wait for the device to find out).
__device__ __forceinline__ bool pass_is_off(const int* run_if, int mask) {
  return run_if != nullptr && (*reinterpret_cast<const volatile int*>(run_if) & mask) == 0;
}

__device__ __forceinline__ void atb_tile(const AtbArgs& g, int tile, int& ti, int& tj) {
  if (!g.symmetric) { ti = tile / g.tiles_n; tj = tile % g.tiles_n; return; }
  int row = 0, rest = tile;
  while (true) {
    const int cnt = g.tiles_n - row;
    if (rest < cnt) { ti = row; tj = row + rest; return; }
    rest -= cnt;
    ++row;
  }
}

// One double-precision tensor-core product: D (8 x 8) += A (8 x 4, row-major fragment) * B (4 x 8,
// column-major fragment).  Lane L holds A[L / 4][L % 4], B[L % 4][L / 4] and D[L / 4][2 (L % 4) + {0, 1}].
__device__ __forceinline__ void dmma_884(double (&d)[2], double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
               : "+d"(d[0]), "+d"(d[1]) : "d"(a), "d"(b));
}

// A 64 x 64 output tile over one slice of the rows: 16 rows at a time are widened to double in
// shared memory (the next 16 are already on their way in registers), warp w multiplies 16 columns
// of A (w / 2) by 32 columns of B (w % 2) on the fp64 tensor cores: six fragment loads for eight
// products (the kernel waits on its shared-memory loads; 8 x 64 per warp took nine).
__global__ void __launch_bounds__(256) atb_f64_partial_kernel(const AtbArgs g) {
  __shared__ double As[AT_K][AT_T + 2];
  __shared__ double Bs[AT_K][AT_T + 2];
  if (pass_is_off(g.run_if, g.run_if_mask)) return;
  int ti, tj;
  atb_tile(g, blockIdx.x, ti, tj);
  const int split = blockIdx.y;
  const long long r0 = g.d * split / g.splits, r1 = g.d * (split + 1) / g.splits;
  const int t = threadIdx.x;
  const int warp = t >> 5, lane = t & 31, gq = lane >> 2, q4 = lane & 3;
  const int m0 = ti * AT_T, n0 = tj * AT_T;
  const int wa = (warp >> 1) * 16, wb = (warp & 1) * 32;   // this warp's columns of A and of B within the tile
  double acc[2][4][2];
#pragma unroll
  for (int h = 0; h < 2; ++h)
#pragma unroll
    for (int c = 0; c < 4; ++c) { acc[h][c][0] = 0.0; acc[h][c][1] = 0.0; }
  // staging: row lr of the chunk, columns lc, lc + 16, lc + 32, lc + 48: the 16 threads of a row write
  // 16 consecutive doubles per store (one shared-memory wavefront per row; four columns per thread
  // side by side made every store an eight-way bank conflict)
  const int lr = t >> 4, lc = t & 15;
  // two chunks of 16 rows are on their way in registers while a third is multiplied (one was not
  // enough to cover the loads' latency: the long slices of a wide panel took 2 us per chunk)
  float ra[2][4], rb[2][4];
  auto fetch = [&](long long k0, float (&fa)[4], float (&fb)[4]) {
    const long long row = k0 + lr;
    const bool in_k = row < r1;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int ca = m0 + lc + 16 * e, cb = n0 + lc + 16 * e;
      fa[e] = (in_k && ca < g.m && PRAC_IN(row * g.lda + ca, (g.d - 1) * g.lda + g.m)) ? g.A[row * g.lda + ca] : 0.f;
      fb[e] = (in_k && cb < g.n && PRAC_IN(row * g.ldb + cb, (g.d - 1) * g.ldb + g.n)) ? g.B[row * g.ldb + cb] : 0.f;
    }
  };
  fetch(r0, ra[0], rb[0]);
  fetch(r0 + AT_K, ra[1], rb[1]);
  int cur = 0;
  for (long long k0 = r0; k0 < r1; k0 += AT_K, cur ^= 1) {
    // (cur is 0, 1, 0, ...: both branches below are the same code on the two register sets)
    if (cur == 0) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        As[lr][lc + 16 * e] = static_cast<double>(ra[0][e]);
        Bs[lr][lc + 16 * e] = static_cast<double>(rb[0][e]);
      }
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        As[lr][lc + 16 * e] = static_cast<double>(ra[1][e]);
        Bs[lr][lc + 16 * e] = static_cast<double>(rb[1][e]);
      }
    }
    __syncthreads();
    if (cur == 0) fetch(k0 + 2 * AT_K, ra[0], rb[0]);
    else fetch(k0 + 2 * AT_K, ra[1], rb[1]);
#pragma unroll
    for (int kk = 0; kk < AT_K / 4; ++kk) {
      const double a0 = As[kk * 4 + q4][wa + gq], a1 = As[kk * 4 + q4][wa + 8 + gq];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const double bv = Bs[kk * 4 + q4][wb + c * 8 + gq];
        dmma_884(acc[0][c], a0, bv);
        dmma_884(acc[1][c], a1, bv);
      }
    }
    __syncthreads();
  }
  double* out = g.partial + static_cast<long long>(split) * g.m * g.n;
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int gi = m0 + wa + h * 8 + gq;
    if (gi >= g.m) continue;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int gj = n0 + wb + c * 8 + 2 * q4 + i;
        if (gj < g.n && PRAC_IN(static_cast<long long>(gi) * g.n + gj, static_cast<long long>(g.m) * g.n))
          out[static_cast<long long>(gi) * g.n + gj] = acc[h][c][i];
      }
    }
  }
}

// out[i][j] = alpha * sum_s partial[s][i][j], slices added in order.  symmetric: entries
// below the diagonal are read from their mirror image (tiles below the diagonal were
// not computed).  TOut = float or double.
template <typename TOut>
__global__ void reduce_partials_kernel(const double* __restrict__ partial, int splits, int m, int n,
                                       int symmetric, double alpha, TOut* __restrict__ out, long long ldo,
                                       const int* run_if, int run_if_mask, int* zero_words, int zero_count) {
  if (pass_is_off(run_if, run_if_mask)) return;
  // state that the next kernel on the stream expects zeroed (its grid-barrier counter)
  if (blockIdx.x == 0 && static_cast<int>(threadIdx.x) < zero_count) zero_words[threadIdx.x] = 0;
  const long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
  if (idx >= static_cast<long long>(m) * n) return;
  const int i = static_cast<int>(idx / n), j = static_cast<int>(idx % n);
  const long long src = (symmetric && i > j) ? static_cast<long long>(j) * n + i : static_cast<long long>(i) * n + j;
  // (eight loads in flight at a time: with many slices and few entries, as for the Rayleigh-Ritz
  // matrix, the kernel is a chain of loads otherwise; the slices are still added one by one, in order)
  const long long mn = static_cast<long long>(m) * n;
  double s = 0.0;
  int sp = 0;
  for (; sp + 8 <= splits; sp += 8) {
    double v[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) v[e] = partial[(sp + e) * mn + src];
#pragma unroll
    for (int e = 0; e < 8; ++e) s += v[e];
  }
  for (; sp < splits; ++sp) s += partial[sp * mn + src];
  if (PRAC_IN(static_cast<long long>(i) * ldo + j, static_cast<long long>(m - 1) * ldo + n))
    out[static_cast<long long>(i) * ldo + j] = static_cast<TOut>(alpha * s);
}

// ------------------------------------------------------------------ Cholesky + inverse, one launch
constexpr int CB = 32;       // block size of the factorisation
// Shared-memory pitch of a block, in doubles: 36 = 8 banks (mod 32) per row, so that the rows a
// tensor-core fragment load touches (four rows of eight consecutive doubles, or eight rows of four)
// fall into two wavefronts, the least a 64-bit load of a warp can take.  (33, the pitch that keeps a
// walk down a column free of conflicts, made those loads four-way conflicts: 168 -> 154 us per launch
// at 320 columns.)
constexpr int CP = CB + 4;
constexpr int CHOL_SMEM = 6 * CB * CP * 8;   // six staging blocks
// What a launch asks for: more than half of an SM's shared memory, so that no two CTAs of this
// kernel (of this or of another factorisation running beside it) land on one SM.  The kernel is a
// chain of dependent steps that issues instructions most of the time: two of its CTAs on one SM
// take nearly twice as long, and every barrier waits for the slowest.
constexpr int CHOL_SMEM_ASK = 116 * 1024;
static_assert(CHOL_SMEM_ASK >= CHOL_SMEM && 2 * CHOL_SMEM_ASK > 227 * 1024, "one CTA per SM");

struct CholArgs {
  double* G;        // n x n, symmetric on entry; its trailing blocks are updated in place
  double* R;        // n x n: the off-diagonal blocks of the upper factor (row j, columns right of j)
  double* Dinv;     // [nb][CB][CB]: inverses of the diagonal blocks of R
  double* X;        // n x n scratch: R^-1 in double
  double* diag0;    // n: the diagonal of G on entry
  float* Rinv;      // n x n output: R^-1 (upper triangular, zeros below)
  __nv_bfloat16* Rt3;  // optional, n x 3 kp: row j = column j of R^-1 as three bf16 pieces side by side
  int kp;
  long long ldr;
  int n, nb;
  int* dev_status;
  int flag_bit;
  GridBarrierState* bar;   // zeroed before the launch
  unsigned poll_limit;
  int run_if_mask;         // != 0: the kernel does nothing unless *dev_status has one of these bits
};

// Element (i, j) of the n x n matrix padded to nb*CB with the identity.
__device__ __forceinline__ double ld_pad(const double* M, int n, int i, int j) {
  return (i < n && j < n) ? __ldcg(&M[static_cast<long long>(i) * n + j]) : (i == j ? 1.0 : 0.0);
}

// C (CB x CB, shared) = products of two CB x CB blocks, all 256 threads: warp w owns the 8-row
// band w / 2 and the two 8-column tiles 2 (w % 2), 2 (w % 2) + 1 of C.
//   MODE 0:  C  = A^T * B
//   MODE 1:  C -= A^T * B
//   MODE 2:  C  = A * B
//   MODE 3:  C -= A * B
__device__ __forceinline__ void blk_mm(double (*C)[CP], const double (*A)[CP], const double (*B)[CP], int mode) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, q = lane & 3;
  const int row0 = (warp >> 1) * 8, col0 = (warp & 1) * 16;
  double acc0[2] = {0.0, 0.0}, acc1[2] = {0.0, 0.0};
#pragma unroll
  for (int ks = 0; ks < CB / 4; ++ks) {
    const double a = (mode >= 2) ? A[row0 + g][ks * 4 + q] : A[ks * 4 + q][row0 + g];
    const double b0 = B[ks * 4 + q][col0 + g];
    const double b1 = B[ks * 4 + q][col0 + 8 + g];
    dmma_884(acc0, a, b0);
    dmma_884(acc1, a, b1);
  }
  double* c0 = &C[row0 + g][col0 + 2 * q];
  double* c1 = &C[row0 + g][col0 + 8 + 2 * q];
  if (mode == 1 || mode == 3) {
    c0[0] -= acc0[0]; c0[1] -= acc0[1]; c1[0] -= acc1[0]; c1[1] -= acc1[1];
  } else {
    c0[0] = acc0[0]; c0[1] = acc0[1]; c1[0] = acc1[0]; c1[1] = acc1[1];
  }
}

__device__ __forceinline__ void blk_load(double (*S)[CP], const double* M, int n, int bi, int bj) {
  for (int idx = threadIdx.x; idx < CB * CB; idx += blockDim.x) {
    const int i = idx / CB, j = idx % CB;
    S[i][j] = ld_pad(M, n, bi * CB + i, bj * CB + j);
  }
}
__device__ __forceinline__ void blk_store(const double (*S)[CP], double* M, int n, int bi, int bj) {
  for (int idx = threadIdx.x; idx < CB * CB; idx += blockDim.x) {
    const int i = bi * CB + idx / CB, j = bj * CB + idx % CB;
    if (i < n && j < n) M[static_cast<long long>(i) * n + j] = S[idx / CB][idx % CB];
  }
}

// In shared memory: D (CB x CB, symmetric positive definite on entry, both triangles) -> I = R^-1
// (upper), where R^T R = D.  One barrier per column and no separate inversion: the elimination
// D[i][.] -= m_ij D[j][.] (m_ij = D[j][i] / pivot_j) is also applied to an identity kept in D's
// lower triangle, which turns it into the unit-lower L^-1 of D = L U; with R = diag(1/sqrt(pivot)) U
// this gives R^-1 = (L^-1)^T diag(1/sqrt(pivot)).  D is left as working storage.  A pivot that is
// not safely positive relative to the column's original squared norm is replaced by a guard value.
// Each thread keeps its four elements of D (rows warp, warp + 8, .., column lane) in registers; a row
// is written back to shared memory once, when it becomes the next pivot row.  The reciprocal of the
// pivot is a hardware approximation refined by two Newton steps (full double accuracy); the square
// roots are taken after the loop, all at once (blk_chol_inv below).
//
// The columns j in [8 P, 8 P + 8) of the block: of a thread's rows w + 8 e only those with e >= P can
// still change (the others are final), so the finished ones are left out at compile time (the column
// step is bound by the instructions it issues: 406 -> 330 cycles per column on one CTA).
template <int P>
__device__ __forceinline__ void blk_chol_columns(double (*D)[CP], const double* guard_sh, double* pv_sh, double (&cur)[4],
                                                 int* dev_status, int flag_bit, bool report) {
  const int t = threadIdx.x, w = t >> 5, l = t & 31;
#pragma unroll 1
  for (int j = 8 * P; j < 8 * P + 8; ++j) {
    double pv = D[j][j];
    const double guard = guard_sh[j];
    if (!(pv > guard)) {
      pv = guard;
      if (t == 0 && report && flag_bit && dev_status) atomicOr(dev_status, flag_bit);
    }
    if (t == 0) pv_sh[j] = pv;
    double x;
    asm("rcp.approx.ftz.f64 %0, %1;" : "=d"(x) : "d"(pv));
    x = fma(fma(-pv, x, 1.0), x, x);
    x = fma(fma(-pv, x, 1.0), x, x);
    // (all of row j is read before the next pivot row is written, and the rows' updates are free of
    // branches: a store into D between the loads, or a branch per row, kept the rows from overlapping)
    const double rowl = D[j][l];
    double dji[4];
#pragma unroll
    for (int e = P; e < 4; ++e) dji[e] = D[j][w + 8 * e];
#pragma unroll
    for (int e = P; e < 4; ++e) {
      const int i = w + 8 * e;
      const double m = dji[e] * x;
      const double upd = fma(-m, rowl, cur[e]);
      // R part, and L^-1 columns before j: updated; L^-1 column j starts here; the rest waits
      const double nv = (l >= i || l < j) ? upd : ((l == j) ? -m : cur[e]);
      cur[e] = (e > P || i > j) ? nv : cur[e];
      if (i == j + 1) D[i][l] = cur[e];                        // the next pivot row is final
    }
    __syncthreads();
  }
}

__device__ void blk_chol_inv(double (*D)[CP], double (*I)[CP], const double* diag0, int n, int j0,
                             int* dev_status, int flag_bit, bool report) {
  __shared__ double guard_sh[CB];
  __shared__ double pv_sh[CB];
  static_assert(CB == 32, "four groups of eight columns, four rows per thread");
  const int t = threadIdx.x, w = t >> 5, l = t & 31;
  if (t < CB) {
    const double d0 = (j0 + t < n) ? __ldcg(&diag0[j0 + t]) : 1.0;
    guard_sh[t] = d0 > 0.0 ? 1e-13 * d0 : 1.0;
  }
  double cur[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) cur[e] = D[w + 8 * e][l];
  __syncthreads();
  blk_chol_columns<0>(D, guard_sh, pv_sh, cur, dev_status, flag_bit, report);
  blk_chol_columns<1>(D, guard_sh, pv_sh, cur, dev_status, flag_bit, report);
  blk_chol_columns<2>(D, guard_sh, pv_sh, cur, dev_status, flag_bit, report);
  blk_chol_columns<3>(D, guard_sh, pv_sh, cur, dev_status, flag_bit, report);
  if (t < CB) pv_sh[t] = rsqrt(pv_sh[t]);
  __syncthreads();
  for (int idx = t; idx < CB * CB; idx += blockDim.x) {
    const int r = idx / CB, c = idx % CB;
    I[r][c] = (r < c) ? D[c][r] * pv_sh[c] : ((r == c) ? pv_sh[c] : 0.0);
  }
  __syncthreads();
}

__global__ void __launch_bounds__(256) chol_inv_kernel(const CholArgs a) {
  if (a.run_if_mask && pass_is_off(a.dev_status, a.run_if_mask)) return;
  extern __shared__ double chol_smem[];
  double (*S0)[CP] = reinterpret_cast<double (*)[CP]>(chol_smem);
  double (*S1)[CP] = S0 + CB;
  double (*S2)[CP] = S1 + CB;
  double (*S3)[CP] = S2 + CB;
  double (*S4)[CP] = S3 + CB;
  double (*S5)[CP] = S4 + CB;
  const int n = a.n, nb = a.nb;
  const int cta = blockIdx.x, nctas = gridDim.x;

  // Grid barriers are bounded: a CTA that gives up (or sees that another did) reports it and
  // leaves; nothing asynchronous is in flight here, so the early exit is clean.
  unsigned passed = 0;
#define CHOL_BARRIER_OR_LEAVE()                                                                        \
  do {                                                                                                 \
    if (!grid_barrier(a.bar, ++passed * static_cast<unsigned>(nctas), a.poll_limit)) {                 \
      if (threadIdx.x == 0 && cta == 0 && a.dev_status) atomicOr(a.dev_status, DEV_WAIT_EXPIRED);      \
      return;                                                                                          \
    }                                                                                                  \
  } while (0)

  for (int i = cta * blockDim.x + threadIdx.x; i < n; i += nctas * blockDim.x)
    a.diag0[i] = a.G[static_cast<long long>(i) * n + i];
  CHOL_BARRIER_OR_LEAVE();

  for (int j = 0; j < nb; ++j) {
    // Every CTA factors the diagonal block itself (no broadcast step): S0 = R_jj, S1 = R_jj^-1
    blk_load(S0, a.G, n, j, j);
    __syncthreads();
    blk_chol_inv(S0, S1, a.diag0, n, j * CB, a.dev_status, a.flag_bit, cta == 0);
    if (cta == 0) {
      // only the inverse of the diagonal block is needed later; it is also the diagonal block of X
      for (int idx = threadIdx.x; idx < CB * CB; idx += blockDim.x)
        a.Dinv[static_cast<long long>(j) * CB * CB + idx] = S1[idx / CB][idx % CB];
      blk_store(S1, a.X, n, j, j);
    }
    // Trailing tiles (p, q), j < p <= q < nb, dealt round-robin.  A tile's owner recomputes the two
    // blocks of row j of R it needs:  R_jp = R_jj^-T G_jp,  R_jq = R_jj^-T G_jq,  then
    // G_pq -= R_jp^T R_jq.  The owner of a diagonal tile also stores R_jp (into R, not over G_jp,
    // which other CTAs are still reading).
    const int rem = nb - j - 1;
    const int ntile = rem * (rem + 1) / 2;
    for (int tile = cta; tile < ntile; tile += nctas) {
      int row = 0, rest = tile;
      while (rest >= rem - row) { rest -= rem - row; ++row; }
      const int p = j + 1 + row, q = p + rest;
      __syncthreads();
      blk_load(S2, a.G, n, j, p);            // the three blocks are fetched in one round trip
      if (q != p) blk_load(S3, a.G, n, j, q);
      blk_load(S5, a.G, n, p, q);
      __syncthreads();
      blk_mm(S4, S1, S2, 0);                 // S4 = R_jj^-T G_jp = R_jp
      __syncthreads();
      if (q != p) {
        blk_mm(S2, S1, S3, 0);               // S2 = R_jq
        __syncthreads();
      }
      blk_mm(S5, S4, (q != p) ? S2 : S4, 1); // G_pq -= R_jp^T R_jq
      __syncthreads();
      blk_store(S5, a.G, n, p, q);
      if (q == p) blk_store(S4, a.R, n, j, p);
    }
    // X = R^-1 grows with the factorisation: X_pq = -(sum_{p <= c < q} X_pc R_cq) R_qq^-1, X_pp = R_pp^-1.
    // Step j adds the c = j - 1 terms (X_p,j-1 and row j - 1 of R were finished before the last
    // grid barrier) to the running sums kept in the blocks (p, q), q >= j, of X, and closes block
    // column j with R_jj^-1 (local, S1).  j (nb - j) tasks of one product each, dealt from the last
    // CTA down so that they fall on CTAs the shrinking set of trailing tiles leaves idle.
    if (j > 0) {
      const int width = nb - j, ntask = j * width;
      for (int u = nctas - 1 - cta; u < ntask; u += nctas) {
        const int p = u / width, q = j + u % width;
        __syncthreads();
        if (p == j - 1) {
          for (int idx = threadIdx.x; idx < CB * CB; idx += blockDim.x) {
            S2[idx / CB][idx % CB] = __ldcg(&a.Dinv[static_cast<long long>(p) * CB * CB + idx]);
            S0[idx / CB][idx % CB] = 0.0;
          }
        } else {
          blk_load(S2, a.X, n, p, j - 1);
          blk_load(S0, a.X, n, p, q);          // the running sum (negated)
        }
        blk_load(S3, a.R, n, j - 1, q);
        __syncthreads();
        blk_mm(S0, S2, S3, 3);                 // S0 -= X_p,j-1 R_j-1,q
        __syncthreads();
        if (q == j) {
          blk_mm(S4, S0, S1, 2);               // X_pj = S0 R_jj^-1
          __syncthreads();
          blk_store(S4, a.X, n, p, j);
        } else {
          blk_store(S0, a.X, n, p, q);
        }
      }
    }
    CHOL_BARRIER_OR_LEAVE();
  }
  // (n * n and n * kp fit 32 bits: n is a panel width, a few thousand at most; 32-bit index
  // arithmetic, the 64-bit divisions by n took longer than the copies)
  const unsigned un = static_cast<unsigned>(n), ustep = static_cast<unsigned>(nctas) * blockDim.x;
  for (unsigned idx = cta * blockDim.x + threadIdx.x; idx < un * un; idx += ustep) {
    const unsigned i = idx / un, j = idx - i * un;
    a.Rinv[static_cast<long long>(i) * a.ldr + j] = (j >= i) ? static_cast<float>(__ldcg(&a.X[idx])) : 0.f;
  }
  if (a.Rt3) {
    // the tensor-core product V R^-1 takes (R^-1)^T with K contiguous: entry (j, l) = R^-1[l][j], l <= j
    const unsigned ukp = static_cast<unsigned>(a.kp);
    for (unsigned idx = cta * blockDim.x + threadIdx.x; idx < un * ukp; idx += ustep) {
      const int j = static_cast<int>(idx / ukp), l = static_cast<int>(idx - static_cast<unsigned>(j) * ukp);
      float x = (l < n && l <= j) ? static_cast<float>(__ldcg(&a.X[static_cast<long long>(l) * n + j])) : 0.f;
      __nv_bfloat16* o = a.Rt3 + static_cast<long long>(j) * 3 * a.kp + l;
      const __nv_bfloat16 hi = __float2bfloat16_rn(x);
      x -= __bfloat162float(hi);
      const __nv_bfloat16 mid = __float2bfloat16_rn(x);
      x -= __bfloat162float(mid);
      o[0] = hi; o[a.kp] = mid; o[2 * a.kp] = __float2bfloat16_rn(x);
    }
  }
}

#undef CHOL_BARRIER_OR_LEAVE

cudaError_t chol_smem_attr() {
  static DeviceOnce done;      // the attribute belongs to the device that was current
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (done.done(dev)) return cudaSuccess;
  e = cudaFuncSetAttribute(chol_inv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, CHOL_SMEM_ASK);
  if (e == cudaSuccess) done.mark(dev);
  return e;
}

int pick_row_splits(int num_tiles, int64_t d) {
  tc_init();
  int sms = tc_num_sms();
  if (sms <= 0) sms = 148;
  int s = (2 * sms) / (num_tiles > 0 ? num_tiles : 1);
  const int64_t max_by_rows = d / 64 > 0 ? d / 64 : 1;
  if (s > max_by_rows) s = static_cast<int>(max_by_rows);
  if (s < 1) s = 1;
  if (s > 64) s = 64;
  return s;
}

}  // namespace

PRAC_BOUNDS_READER(bounds_violations_cholqr)

// ------------------------------------------------------------------ host side
namespace {
int atb_tiles(int64_t m, int64_t n, int symmetric) {
  const int tm = static_cast<int>((m + AT_T - 1) / AT_T), tn = static_cast<int>((n + AT_T - 1) / AT_T);
  return symmetric ? tn * (tn + 1) / 2 : tm * tn;
}
}  // namespace

size_t atb_ws_bytes(int64_t m, int64_t n, int64_t d, int symmetric) {
  if (m <= 0 || n <= 0 || d <= 0) return 0;
  return static_cast<size_t>(pick_row_splits(atb_tiles(m, n, symmetric), d)) * m * n * sizeof(double);
}

int atb_f64(const float* A, int64_t lda, const float* B, int64_t ldb, int64_t d, int64_t m, int64_t n,
            int symmetric, double alpha, void* out, int64_t ldo, int out_double, void* ws, size_t ws_bytes,
            cudaStream_t stream, const int* run_if, int run_if_mask, void* zero_after, int zero_bytes) {
  if (m <= 0 || n <= 0) return PRAC_OK;
  if (d <= 0 || (symmetric && (A != B || m != n))) return PRAC_EINVAL;
  AtbArgs g{};
  g.A = A; g.lda = lda; g.B = B; g.ldb = ldb;
  g.m = static_cast<int>(m); g.n = static_cast<int>(n); g.d = d;
  g.tiles_m = static_cast<int>((m + AT_T - 1) / AT_T);
  g.tiles_n = static_cast<int>((n + AT_T - 1) / AT_T);
  g.symmetric = symmetric;
  g.num_tiles = atb_tiles(m, n, symmetric);
  g.splits = pick_row_splits(g.num_tiles, d);
  const size_t need = static_cast<size_t>(g.splits) * m * n * sizeof(double);
  if (!ws || ws_bytes < need) return PRAC_EWORKSPACE;
  g.partial = static_cast<double*>(ws);
  g.run_if = run_if; g.run_if_mask = run_if_mask;
  atb_f64_partial_kernel<<<dim3(static_cast<unsigned>(g.num_tiles), static_cast<unsigned>(g.splits)), 256, 0, stream>>>(g);
  count_launch();
  if (out_double)
    reduce_partials_kernel<double><<<nblocks(m * n, 256), 256, 0, stream>>>(g.partial, g.splits, g.m, g.n, symmetric,
                                                                            alpha, static_cast<double*>(out), ldo, run_if,
                                                                            run_if_mask, static_cast<int*>(zero_after),
                                                                            zero_bytes / 4);
  else
    reduce_partials_kernel<float><<<nblocks(m * n, 256), 256, 0, stream>>>(g.partial, g.splits, g.m, g.n, symmetric,
                                                                           alpha, static_cast<float*>(out), ldo, run_if,
                                                                           run_if_mask, static_cast<int*>(zero_after),
                                                                           zero_bytes / 4);
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

// Workspace of one Cholesky-QR pass on n columns (all 256-byte aligned):
//   G n*n double | R n*n double | X n*n double | Dinv nb*CB*CB double | diag0 n double | Rinv n*n float |
//   slices of the transposed product
namespace {
// Both operands as three bf16 pieces, side by side in rows of 3 kp: the segments of the chained
// product mid*mid, lo*hi, hi*lo, mid*hi, hi*mid, hi*hi: everything down to 2^-24 of the product, the
// small cross terms first so that they add up among themselves before the leading term arrives.
TcSegments six_cross_terms(int64_t kp) {
  TcSegments segs{};
  segs.n = 6;
  const int64_t pa[6] = {1, 2, 0, 1, 0, 0}, pb[6] = {1, 0, 2, 0, 1, 0};
  for (int q = 0; q < 6; ++q) { segs.off_a[q] = pa[q] * kp; segs.off_b[q] = pb[q] * kp; }
  segs.rows_a = 3 * kp;
  segs.rows_b = 3 * kp;
  return segs;
}

struct CholWs { double* G; double* R; double* X; double* Dinv; double* diag0; float* Rinv; void* part; size_t part_bytes; size_t bytes;
                __nv_bfloat16* V3; __nv_bfloat16* Rt3; int64_t kp; bool tensor; GridBarrierState* bar; };
// V R^-1 runs on the tensor cores (operands as three bf16 pieces each, six cross terms: fp32
// accuracy) when the panel is big enough to fill their tiles.
inline bool vr_on_tensor_cores(int64_t n, int64_t d) { return d >= 256 && n >= 64; }
CholWs carve_chol(void* ws, int64_t n, int64_t d) {
  CholWs c;
  const int64_t nb = (n + CB - 1) / CB;
  size_t off = 0;
  auto take = [&](size_t b) { size_t o = off; off += (b + 255) / 256 * 256; return o; };
  const size_t oG = take(n * n * 8), oRR = take(n * n * 8), oX = take(n * n * 8), oD = take(nb * CB * CB * 8), o0 = take(n * 8);
  const size_t oR = take(n * n * 4);
  c.part_bytes = atb_ws_bytes(n, n, d, 1);
  const size_t oP = take(c.part_bytes);
  c.tensor = vr_on_tensor_cores(n, d);
  c.kp = (n + 63) / 64 * 64;
  const size_t oV3 = take(c.tensor ? static_cast<size_t>(d) * 3 * c.kp * 2 : 0);
  const size_t oR3 = take(c.tensor ? static_cast<size_t>(n) * 3 * c.kp * 2 : 0);
  const size_t oBar = take(sizeof(GridBarrierState));
  char* b = static_cast<char*>(ws);
  c.bar = reinterpret_cast<GridBarrierState*>(b + oBar);
  c.G = reinterpret_cast<double*>(b + oG); c.R = reinterpret_cast<double*>(b + oRR); c.X = reinterpret_cast<double*>(b + oX);
  c.Dinv = reinterpret_cast<double*>(b + oD); c.diag0 = reinterpret_cast<double*>(b + o0);
  c.Rinv = reinterpret_cast<float*>(b + oR); c.part = b + oP;
  c.V3 = reinterpret_cast<__nv_bfloat16*>(b + oV3); c.Rt3 = reinterpret_cast<__nv_bfloat16*>(b + oR3);
  c.bytes = off;
  return c;
}
}  // namespace

size_t cholqr_ws_bytes(int64_t n, int64_t d) { return n > 0 ? carve_chol(nullptr, n, d).bytes : 0; }

int cholqr_pass(const float* Vin, int64_t ldin, float* Vout, int64_t ldout, int64_t d, int64_t n, void* ws,
                size_t ws_bytes, int* dev_status, int flag_bit, cudaStream_t stream, int run_if_mask) {
  if (n <= 0) return PRAC_OK;
  if (d < n || Vin == Vout || n > 40000) return PRAC_EINVAL;   // (the kernel indexes n x n with 32 bits)
  if (run_if_mask && !dev_status) return PRAC_EINVAL;
  const CholWs c = carve_chol(ws, n, d);
  if (ws == nullptr || ws_bytes < c.bytes) return PRAC_EWORKSPACE;
  const int* run_if = run_if_mask ? dev_status : nullptr;
  // (the reduction kernel also zeroes the grid-barrier state of the factorisation that follows it)
  int st = atb_f64(Vin, ldin, Vin, ldin, d, n, n, 1, 1.0, c.G, n, 1, c.part, c.part_bytes, stream, run_if, run_if_mask,
                   c.bar, static_cast<int>(sizeof(GridBarrierState)));
  if (st != PRAC_OK) return st;
  CholArgs a{};
  a.G = c.G; a.R = c.R; a.Dinv = c.Dinv; a.X = c.X; a.diag0 = c.diag0; a.Rinv = c.Rinv; a.ldr = n;
  a.n = static_cast<int>(n); a.nb = static_cast<int>((n + CB - 1) / CB);
  a.dev_status = dev_status; a.flag_bit = flag_bit;
  a.bar = c.bar; a.poll_limit = barrier_poll_limit(); a.run_if_mask = run_if_mask;
  // an optional pass (run_if_mask != 0) is rare and small: it takes the general product
  const bool tensor = run_if_mask == 0 && c.tensor && tc_init() == PRAC_OK && aligned16(Vout) && (ldout % 4) == 0;
  a.Rt3 = tensor ? c.Rt3 : nullptr;
  a.kp = static_cast<int>(c.kp);
  const int rem = a.nb - 1;
  // one CTA per task of the busiest step: trailing tiles plus the products of the inverse
  int want = rem * (rem + 1) / 2;
  for (int j = 1; j < a.nb; ++j) {
    const int w = a.nb - j;
    const int tasks = (w - 1) * w / 2 + j * w;
    if (tasks > want) want = tasks;
  }
  int grid = want < 1 ? 1 : (want > 96 ? 96 : want);
  // ... and at most a quarter of the SMs, an SM each: a transformer block fits the bases of its four
  // distinct inputs side by side (four streams), and four factorisations of 45 CTAs on 148 SMs that
  // share SMs take 170-300 us each where one alone takes 130; with 37 CTAs each the block's four fits
  // take 4.66 instead of 4.96 ms, a single fit 0.05 ms more (the busiest steps deal their tiles in
  // two rounds).
  {
    const int sms = tc_num_sms();
    const int quarter = sms >= 4 ? sms / 4 : 1;
    if (grid > quarter) grid = quarter;
  }
  const int smem = CHOL_SMEM_ASK;
  void* args[] = {const_cast<CholArgs*>(&a)};
  PRAC_CUDA_TRY(chol_smem_attr());
  // cooperative launch: the grid barrier needs every CTA resident
  PRAC_CUDA_TRY(cudaLaunchCooperativeKernel(reinterpret_cast<void*>(chol_inv_kernel), dim3(grid), dim3(256), args,
                                            smem, stream));
  count_launch();
  if (tensor) {
    st = launch_split3_cols(Vin, ldin, d, n, c.V3, c.kp, stream);
    if (st != PRAC_OK) return st;
    const TcSegments segs = six_cross_terms(c.kp);
    return tc_gemm_kmajor(c.V3, 3 * c.kp, c.Rt3, 3 * c.kp, d, n, c.kp, Vout, ldout, ET_F32, 0, dev_status, stream, &segs);
  }
  GemmArgs g{};
  g.M = d; g.N = n; g.K = n;
  g.A = Vin; g.lda = ldin; g.type_a = ET_F32; g.trans_a = 0;
  g.B = c.Rinv; g.ldb = n; g.type_b = ET_F32; g.trans_b = 0;
  g.C = Vout; g.ldc = ldout; g.type_c = ET_F32;
  g.alpha = 1.0; g.beta = 0.0; g.acc_double = 0; g.kscale_from = -1; g.kscale = 1.0;
  g.run_if = run_if; g.run_if_mask = run_if_mask;
  return gemm_general(g, stream);
}

namespace {
__global__ void copy2d_if_kernel(const float* __restrict__ src, long long lds, float* __restrict__ dst, long long ldd,
                                 long long rows, long long cols, const int* status, int run_if_mask) {
  if (pass_is_off(status, run_if_mask)) return;
  // a small fixed grid striding over the matrix: the launch is almost always a no-op and should cost one
  for (long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; idx < rows * cols;
       idx += static_cast<long long>(gridDim.x) * blockDim.x) {
    const long long i = idx / cols, j = idx % cols;
    if (!PRAC_IN(i * lds + j, (rows - 1) * lds + cols) || !PRAC_IN(i * ldd + j, (rows - 1) * ldd + cols)) continue;
    dst[i * ldd + j] = src[i * lds + j];
  }
}
// Runs alone after every kernel of the optional pass has read the word.
__global__ void clear_status_bits_kernel(int* status, int clear_bits) { atomicAnd(status, ~clear_bits); }
}  // namespace

int launch_copy2d_if(const float* src, int64_t lds, float* dst, int64_t ldd, int64_t rows, int64_t cols,
                     int* status, int run_if_mask, int clear_bits, cudaStream_t stream) {
  if (!status) return PRAC_EINVAL;
  if (rows > 0 && cols > 0) {
    const unsigned want = nblocks(rows * cols, 256);
    copy2d_if_kernel<<<want < 296u ? want : 296u, 256, 0, stream>>>(src, lds, dst, ldd, rows, cols, status, run_if_mask);
    count_launch();
  }
  clear_status_bits_kernel<<<1, 1, 0, stream>>>(status, clear_bits);
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

// C (d x n, fp32) = [C +] scale * A (d x kd, fp32) * B (kd x n, fp32) to fp32 accuracy on the tensor
// cores: A row by row and B transposed are cut into three bf16 pieces each and the six leading
// cross terms are chained into one accumulator.  Panels too small for the tensor-core tiles take
// the general kernel.  Workspace: the pieces of A (d x 3 kp) and of B^T (n x 3 kp), kp = kd up to 64.
size_t panel_mm3_ws_bytes(int64_t d, int64_t kd, int64_t n) {
  const int64_t kp = (kd + 63) / 64 * 64;
  return (static_cast<size_t>(d) * 3 * kp * 2 + 255) / 256 * 256 + (static_cast<size_t>(n) * 3 * kp * 2 + 255) / 256 * 256;
}
int panel_mm3(const float* A, int64_t lda, const float* B, int64_t ldb, int64_t d, int64_t kd, int64_t n, float scale,
              float* C, int64_t ldc, int accumulate, void* ws, size_t ws_bytes, int* dev_status, cudaStream_t stream) {
  if (d <= 0 || kd <= 0 || n <= 0) return PRAC_OK;
  if (!(d >= 256 && n >= 64 && kd >= 64) || ws == nullptr || ws_bytes < panel_mm3_ws_bytes(d, kd, n)) {
    GemmArgs g{};
    g.M = d; g.N = n; g.K = kd;
    g.A = A; g.lda = lda; g.type_a = ET_F32; g.trans_a = 0;
    g.B = B; g.ldb = ldb; g.type_b = ET_F32; g.trans_b = 0;
    g.C = C; g.ldc = ldc; g.type_c = ET_F32;
    g.alpha = scale; g.beta = accumulate ? 1.0 : 0.0; g.acc_double = 0; g.kscale_from = -1; g.kscale = 1.0;
    return gemm_general(g, stream);
  }
  const int64_t kp = (kd + 63) / 64 * 64;
  __nv_bfloat16* A3 = static_cast<__nv_bfloat16*>(ws);
  __nv_bfloat16* Bt3 = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(ws) +
                                                        (static_cast<size_t>(d) * 3 * kp * 2 + 255) / 256 * 256);
  int st = launch_split3_cols(A, lda, d, kd, A3, kp, stream);
  if (st != PRAC_OK) return st;
  st = launch_split3_transposed(B, ldb, kd, n, scale, Bt3, kp, stream);
  if (st != PRAC_OK) return st;
  const TcSegments segs = six_cross_terms(kp);
  return tc_gemm_kmajor(A3, 3 * kp, Bt3, 3 * kp, d, n, kp, C, ldc, ET_F32, accumulate, dev_status, stream, &segs);
}

int cholqr_final(const float* Vin, int64_t ldin, float* Vout, int64_t ldout, float* tmp, int64_t d, int64_t n,
                 void* ws, size_t ws_bytes, int* dev_status, cudaStream_t stream) {
  if (n <= 0) return PRAC_OK;
  if (!dev_status || tmp == Vout || tmp == Vin) return PRAC_EINVAL;
  int st = cholqr_pass(Vin, ldin, Vout, ldout, d, n, ws, ws_bytes, dev_status, DEV_CHOL_RETRY, stream);
  if (st != PRAC_OK) return st;
  // A bad pivot means the panel was (numerically) rank deficient: the guarded column of Vout is
  // amplified rounding noise, a direction of its own but neither normalised nor orthogonal to
  // the rest.  One more pass orthonormalises it; only if that pass breaks down too is the
  // failure reported.
  st = cholqr_pass(Vout, ldout, tmp, n, d, n, ws, ws_bytes, dev_status, DEV_CHOL_PIVOT, stream, DEV_CHOL_RETRY);
  if (st != PRAC_OK) return st;
  return launch_copy2d_if(tmp, n, Vout, ldout, d, n, dev_status, DEV_CHOL_RETRY, DEV_CHOL_RETRY, stream);
}

}  // namespace prac
