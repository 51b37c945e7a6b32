// Small-matrix kernels of the basis fit: the counter-based Gaussian draw, the one-sided block
// Jacobi eigen-solver of the Rayleigh-Ritz step, and format conversions.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "act.cuh"
#include "grid_barrier.cuh"
#include "internal.h"
#include "per_device.h"

namespace prac {
namespace {

// ------------------------------------------------------------------ Philox4x32-10
// Salmon, Moraes, Dror, Shaw (SC'11).  One call turns a 128-bit counter and a 64-bit key
// into four 32-bit words.
__device__ __forceinline__ uint4 philox4x32_10(uint4 ctr, uint2 key) {
  constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    const uint32_t hi0 = __umulhi(M0, ctr.x), lo0 = M0 * ctr.x;
    const uint32_t hi1 = __umulhi(M1, ctr.z), lo1 = M1 * ctr.z;
    ctr = make_uint4(hi1 ^ ctr.y ^ key.x, lo1, hi0 ^ ctr.w ^ key.y, lo0);
    key.x += W0;
    key.y += W1;
  }
  return ctr;
}

__device__ __forceinline__ uint4 draw_block(uint64_t seed, uint64_t draw_counter, uint64_t blk) {
  const uint4 ctr = make_uint4(static_cast<uint32_t>(blk), static_cast<uint32_t>(blk >> 32),
                               static_cast<uint32_t>(draw_counter), static_cast<uint32_t>(draw_counter >> 32));
  const uint2 key = make_uint2(static_cast<uint32_t>(seed), static_cast<uint32_t>(seed >> 32));
  return philox4x32_10(ctr, key);
}

__global__ void philox_words_kernel(uint64_t seed, uint64_t dc, long long n, uint32_t* __restrict__ out) {
  const long long blk = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
  const long long e0 = blk * 4;
  if (e0 >= n) return;
  const uint4 w = draw_block(seed, dc, static_cast<uint64_t>(blk));
  if (e0 + 4 <= n && (reinterpret_cast<uintptr_t>(out + e0) & 15u) == 0) {
    *reinterpret_cast<uint4*>(out + e0) = w;
  } else {
    const uint32_t v[4] = {w.x, w.y, w.z, w.w};
    for (int e = 0; e < 4 && e0 + e < n; ++e)
      if (PRAC_IN(e0 + e, n)) out[e0 + e] = v[e];
  }
}

// 23-bit uniform at a cell midpoint: (2 (w >> 9) + 1) / 2^24, never 0 or 1.
__device__ __forceinline__ double word_to_uniform(uint32_t w) {
  return (2.0 * static_cast<double>(w >> 9) + 1.0) * (1.0 / 16777216.0);
}

// Box-Muller on lane pairs (0,1) and (2,3); evaluated in double, stored as float.
__global__ void gaussian_kernel(uint64_t seed, uint64_t dc, long long d, long long r,
                                float* __restrict__ S, long long lds) {
  const long long blk = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
  const long long n = d * r;
  const long long e0 = blk * 4;
  if (e0 >= n) return;
  const uint4 w = draw_block(seed, dc, static_cast<uint64_t>(blk));
  const uint32_t wa[2] = {w.x, w.z}, wb[2] = {w.y, w.w};
  float z[4];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const double rad = sqrt(-2.0 * log(word_to_uniform(wa[h])));
    double sn, cs;
    sincospi(2.0 * word_to_uniform(wb[h]), &sn, &cs);
    z[2 * h] = static_cast<float>(rad * cs);
    z[2 * h + 1] = static_cast<float>(rad * sn);
  }
  for (int e = 0; e < 4 && e0 + e < n; ++e) {
    const long long idx = e0 + e;
    if (PRAC_IN((idx / r) * lds + (idx % r), (d - 1) * lds + r)) S[(idx / r) * lds + (idx % r)] = z[e];
  }
}

// ------------------------------------------------------------------ Jacobi eigen-solver
// Dominant eigenvectors of a small symmetric positive semi-definite matrix B by one-sided
// (Hestenes) block Jacobi.  With A = B + sigma I (sigma > 0 small), plane rotations applied to the
// columns of A make them mutually orthogonal: A J = J (Lambda + sigma I).  The column norms then
// order the eigenvalues and the normalised columns are the eigenvectors, so no eigenvector
// matrix is accumulated and a null space of B comes out as an orthonormal set.  (Rotating a
// Cholesky factor of A instead was measured: it saved no sweep and cost a factorisation.)
// The columns (stored as rows of At) are grouped in blocks of b.  In one outer step the
// round-robin schedule gives each CTA a pair of blocks: it loads the 2b columns into shared
// memory, runs one full inner sweep over them (2b - 1 steps of b disjoint rotations, one warp
// per rotation) and writes them back; the CTAs then meet at a grid barrier.  One outer sweep =
// (number of blocks - 1) barriers instead of the (n - 1) of element-wise Jacobi.
constexpr int JAC_MAX_SWEEPS = 30;
struct JacobiInfo {
  GridBarrierState bar;             // zeroed before the launch
  int sweeps;
  int rotations[JAC_MAX_SWEEPS];    // rotations applied in each outer sweep
  int max_cos2[JAC_MAX_SWEEPS];     // largest squared cosine rotated away in each sweep (float bits)
};

// Pair i of step `step` of the round-robin schedule on m (even) items, as p < q.
__device__ __forceinline__ void rr_pair(int m, int step, int i, int& p, int& q) {
  int a, b;
  if (i == 0) { a = m - 1; b = step; }
  else { a = (step + i) % (m - 1); b = (step - i + (m - 1)) % (m - 1); }
  p = a < b ? a : b;
  q = a < b ? b : a;
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// At (n x n, n a multiple of 16) = symmetrised B (ell x ell, leading dimension ldb) + sigma I,
// padded with 0.5 sigma on the diagonal; sigma = 2^-15 * largest diagonal entry of B (1 if B = 0):
// above the rounding noise that B inherits from its fp32 factors (so that null directions of B
// get columns of a definite size), and harmless, since a shift moves no eigenvector.
__global__ void __launch_bounds__(256) jacobi_prepare_kernel(const double* __restrict__ B, long long ldb, int ell,
                                                             double* __restrict__ At, int n, JacobiInfo* info) {
  __shared__ double red[256];
  if (blockIdx.x == 0) {       // the solver's barrier counter and sweep records start at zero
    int* words = reinterpret_cast<int*>(info);
    for (int i = threadIdx.x; i < static_cast<int>(sizeof(JacobiInfo) / sizeof(int)); i += blockDim.x) words[i] = 0;
  }
  double m = 0.0;
  for (int i = threadIdx.x; i < ell; i += blockDim.x) m = fmax(m, fabs(B[static_cast<long long>(i) * ldb + i]));
  red[threadIdx.x] = m;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o) red[threadIdx.x] = fmax(red[threadIdx.x], red[threadIdx.x + o]);
    __syncthreads();
  }
  const double sigma = red[0] > 0.0 ? red[0] * (1.0 / 32768.0) : 1.0;
  for (long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; idx < static_cast<long long>(n) * n;
       idx += static_cast<long long>(gridDim.x) * blockDim.x) {
    const int i = static_cast<int>(idx / n), j = static_cast<int>(idx % n);
    double v = 0.0;
    if (i < ell && j < ell) {
      v = 0.5 * (B[static_cast<long long>(i) * ldb + j] + B[static_cast<long long>(j) * ldb + i]);
      if (i == j) v += sigma;
    } else if (i == j) {
      v = 0.5 * sigma;
    }
    At[idx] = v;
  }
}

// One rotation of the shared-memory columns cp, cq (length n) by one warp.  With R > 0 each lane
// keeps its R elements of both columns in registers between the dot products and the update, so
// a rotation reads and writes shared memory once; R = 0 re-reads (any n).  Returns 1 if rotated.
template <int R>
__device__ __forceinline__ int rotate_pair(double* cp, double* cq, int n, int lane, double tol, float& max_cos2) {
  double alpha = 0.0, beta = 0.0, gamma = 0.0;
  double xr[R > 0 ? R : 1], yr[R > 0 ? R : 1];
  if (R > 0) {
#pragma unroll
    for (int e = 0; e < R; ++e) {
      const int r = lane + 32 * e;
      xr[e] = r < n ? cp[r] : 0.0;
      yr[e] = r < n ? cq[r] : 0.0;
      alpha = fma(xr[e], xr[e], alpha); beta = fma(yr[e], yr[e], beta); gamma = fma(xr[e], yr[e], gamma);
    }
  } else {
    for (int r = lane; r < n; r += 32) {
      const double x = cp[r], y = cq[r];
      alpha = fma(x, x, alpha); beta = fma(y, y, beta); gamma = fma(x, y, gamma);
    }
  }
  alpha = warp_sum(alpha); beta = warp_sum(beta); gamma = warp_sum(gamma);
  if (!(gamma * gamma > tol * tol * alpha * beta)) return 0;    // warp-uniform
  max_cos2 = fmaxf(max_cos2, static_cast<float>(gamma * gamma / (alpha * beta)));
  // The angle only has to shrink the inner product, so tan is taken in fp32 (double-precision
  // divisions and square roots are slow here); cos and sin are then formed in double from that
  // tangent, which keeps the rotation orthogonal to double accuracy.
  const float zeta = static_cast<float>(beta - alpha) / (2.f * static_cast<float>(gamma));
  const float az = fabsf(zeta);
  const float t32 = (az > 1e15f) ? 0.5f / zeta : copysignf(1.f, zeta) / (az + sqrtf(1.f + az * az));
  const double t = static_cast<double>(t32);
  const double c = rsqrt(1.0 + t * t), s = c * t;
  if (R > 0) {
#pragma unroll
    for (int e = 0; e < R; ++e) {
      const int r = lane + 32 * e;
      if (r < n) { cp[r] = c * xr[e] - s * yr[e]; cq[r] = s * xr[e] + c * yr[e]; }
    }
  } else {
    for (int r = lane; r < n; r += 32) {
      const double x = cp[r], y = cq[r];
      cp[r] = c * x - s * y;
      cq[r] = s * x + c * y;
    }
  }
  return 1;
}

// blockDim = 32 * b; dynamic shared memory = 2 b n doubles; R: see rotate_pair (32 R >= n).
// A block's own column pairs are rotated in the first visit of each sweep in which the block
// takes part (a full inner sweep over the 2b columns); every other visit rotates only the b*b
// pairs that cross the two blocks (b steps of b disjoint rotations).
template <int R>
__global__ void jacobi_kernel(double* At, int n, int b, int max_sweeps, double tol, JacobiInfo* info,
                              int* dev_status, unsigned poll_limit) {
  extern __shared__ double cols[];          // [2b][n]
  const int nb = n / b;
  const int nbr = nb + (nb & 1);            // an odd count plays with a bye
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m = 2 * b;
  const unsigned nctas = gridDim.x;
  unsigned bar = 0;
  bool alive = true, converged = false;
  int sweep = 0;
  for (; alive && sweep < max_sweeps && !converged; ++sweep) {
    for (int step = 0; alive && step < nbr - 1; ++step) {
      int I, J;
      rr_pair(nbr, step, blockIdx.x, I, J);
      if (J < nb) {                          // J == nb: bye
        // each warp moves whole columns, all of a lane's loads in flight together
        for (int lc = warp; lc < m; lc += b) {
          const double* src = At + static_cast<long long>(lc < b ? I * b + lc : J * b + (lc - b)) * n;
          double* dst = cols + lc * n;
          if (R > 0) {
            double v[R > 0 ? R : 1];
#pragma unroll
            for (int e = 0; e < R; ++e) { const int r = lane + 32 * e; v[e] = r < n ? __ldcg(&src[r]) : 0.0; }
#pragma unroll
            for (int e = 0; e < R; ++e) { const int r = lane + 32 * e; if (r < n) dst[r] = v[e]; }
          } else {
            for (int r = lane; r < n; r += 32) dst[r] = __ldcg(&src[r]);
          }
        }
        __syncthreads();
        // with a bye in the schedule, the block that sat out step 0 is first seen in step 1
        bool full = (step == 0);
        if (nbr != nb && step == 1) {
          int I0, J0;
          for (int c = 0; c < nbr / 2; ++c) {
            rr_pair(nbr, 0, c, I0, J0);
            if (J0 == nb && (I0 == I || I0 == J)) full = true;
          }
        }
        int rotated = 0;
        float max_cos2 = 0.f;
        if (full) {
          for (int is = 0; is < m - 1; ++is) {
            int p, q;
            rr_pair(m, is, warp, p, q);
            rotated += rotate_pair<R>(cols + p * n, cols + q * n, n, lane, tol, max_cos2);
            __syncthreads();
          }
        } else {
          for (int is = 0; is < b; ++is) {
            const int p = warp, q = b + (warp + is) % b;
            rotated += rotate_pair<R>(cols + p * n, cols + q * n, n, lane, tol, max_cos2);
            __syncthreads();
          }
        }
        if (lane == 0 && rotated) {
          atomicAdd(&info->rotations[sweep], rotated);
          atomicMax(&info->max_cos2[sweep], __float_as_int(max_cos2));   // non-negative floats order as ints
        }
        for (int lc = warp; lc < m; lc += b) {
          double* dstg = At + static_cast<long long>(lc < b ? I * b + lc : J * b + (lc - b)) * n;
          const double* srcs = cols + lc * n;
          for (int r = lane; r < n; r += 32) dstg[r] = srcs[r];
        }
      }
      alive = grid_barrier(&info->bar, ++bar * nctas, poll_limit);
    }
    // Every CTA reads the same values after the barrier of the sweep's last step.  Convergence is
    // quadratic: once the largest cosine rotated away in a sweep is below 1e-4, what is left is
    // of the order of its square, far below the threshold, and the sweep that would only confirm
    // it is skipped.
    if (alive) {
      const int rot = *reinterpret_cast<volatile int*>(&info->rotations[sweep]);
      const float mc2 = __int_as_float(*reinterpret_cast<volatile int*>(&info->max_cos2[sweep]));
      converged = (rot == 0) || (mc2 < 1e-8f);
    }
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    info->sweeps = sweep;
    if (!alive && dev_status) atomicOr(dev_status, DEV_WAIT_EXPIRED);
    else if (!converged && dev_status) atomicOr(dev_status, DEV_JACOBI_NOCONV);
  }
}

// ------------------------------------------------------------------ block Jacobi through the Gram matrix
// One double-precision tensor-core product: D (8 x 8) += A (8 x 4, row-major fragment) * B (4 x 8,
// column-major fragment).  Lane L holds A[L / 4][L % 4], B[L % 4][L / 4] and D[L / 4][2 (L % 4) + {0, 1}].
__device__ __forceinline__ void dmma_884(double (&d)[2], double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
               : "+d"(d[0]), "+d"(d[1]) : "d"(a), "d"(b));
}

constexpr int JG_B = 8;          // columns per block
constexpr int JG_M = 2 * JG_B;   // columns a CTA holds
constexpr int JG_P = JG_M + 1;   // pitch of the small matrices

// Rotation coefficients of one column within a round: new column x = self * x + other * partner(x).
struct JgCoef { double self, other; int partner; int pad; };

// Same sweeps, visits and rotation order as jacobi_kernel, for 8-column blocks and 256 threads, but a
// visit works on the 16 x 16 Gram matrix G of its columns: G is formed once (tensor cores), each
// round's eight disjoint rotations are read off G and applied to G and to the accumulated
// rotation J (16 x 16, one element per thread), and the columns are multiplied by J once at the
// end (tensor cores).  The long vectors are touched twice per visit instead of twice per round.
// CLUSTER: the whole grid is one thread-block cluster (at most 8 CTAs) and the CTAs meet at the
// hardware cluster barrier, whose release / acquire also orders their global-memory traffic;
// every CTA runs the same number of steps and sweeps (the stopping test reads values that are
// final before the barrier it follows), so each barrier is reached by all of them.  Otherwise a
// cooperative launch with the bounded software barrier.
template <bool CLUSTER>
__global__ void __launch_bounds__(256) jacobi_gram_kernel(double* At, int n, int max_sweeps, double tol, JacobiInfo* info,
                                                          int* dev_status, unsigned poll_limit) {
  extern __shared__ double jsm[];
  const int ns = n + 4;                                   // column pitch: keeps the fragment loads off one bank
  double* cols = jsm;                                     // [16][ns]
  double (*G0)[JG_P] = reinterpret_cast<double (*)[JG_P]>(cols + JG_M * ns);
  double (*G1)[JG_P] = G0 + JG_M;
  double (*J0)[JG_P] = G1 + JG_M;
  double (*J1)[JG_P] = J0 + JG_M;
  double* part = reinterpret_cast<double*>(J1 + JG_M);    // [8 warps][3 tiles][64]
  JgCoef* coef = reinterpret_cast<JgCoef*>(part + 8 * 3 * 64);   // [16]
  __shared__ int visit_rotated;

  const int b = JG_B, m = JG_M;
  const int nb = n / b;
  const int nbr = nb + (nb & 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, q4 = lane & 3;
  const int ei = threadIdx.x >> 4, ej = threadIdx.x & 15;   // this thread's element of the 16 x 16 matrices
  const unsigned nctas = gridDim.x;
  unsigned bar = 0;
  bool alive = true, converged = false;
  int sweep = 0;
  for (; alive && sweep < max_sweeps && !converged; ++sweep) {
    for (int step = 0; alive && step < nbr - 1; ++step) {
      int I, J;
      rr_pair(nbr, step, blockIdx.x, I, J);
      if (J < nb) {
        for (int lc = warp; lc < m; lc += 8) {
          const double* src = At + static_cast<long long>(lc < b ? I * b + lc : J * b + (lc - b)) * n;
          double* dst = cols + lc * ns;
          for (int r0 = lane; r0 < n; r0 += 32 * 12) {    // up to twelve loads in flight per lane
            double v[12];
#pragma unroll
            for (int e = 0; e < 12; ++e) { const int r = r0 + 32 * e; v[e] = r < n ? __ldcg(&src[r]) : 0.0; }
#pragma unroll
            for (int e = 0; e < 12; ++e) { const int r = r0 + 32 * e; if (r < n) dst[r] = v[e]; }
          }
        }
        if (threadIdx.x == 0) visit_rotated = 0;
        __syncthreads();
        // ---- G = A^T A: each warp sums a slice of the rows, the slices are added in warp order
        {
          double t00[2] = {0.0, 0.0}, t01[2] = {0.0, 0.0}, t11[2] = {0.0, 0.0};
          const int ks_total = n / 4, kpw = (ks_total + 7) / 8;
          const int ks_end = min(ks_total, (warp + 1) * kpw);
          for (int ks = warp * kpw; ks < ks_end; ++ks) {
            const int r = ks * 4 + q4;
            const double a0 = cols[g * ns + r], a1 = cols[(8 + g) * ns + r];
            dmma_884(t00, a0, a0);
            dmma_884(t01, a0, a1);
            dmma_884(t11, a1, a1);
          }
          double* pw = part + warp * 192 + g * 8 + 2 * q4;
          pw[0] = t00[0]; pw[1] = t00[1];
          pw[64] = t01[0]; pw[65] = t01[1];
          pw[128] = t11[0]; pw[129] = t11[1];
        }
        __syncthreads();
        {
          // element (ei, ej): tile 00, 01 (or its transpose) or 11
          int tile, r, c;
          if (ei < 8 && ej < 8) { tile = 0; r = ei; c = ej; }
          else if (ei < 8) { tile = 1; r = ei; c = ej - 8; }
          else if (ej < 8) { tile = 1; r = ej; c = ei - 8; }
          else { tile = 2; r = ei - 8; c = ej - 8; }
          double sum = 0.0;
#pragma unroll
          for (int w8 = 0; w8 < 8; ++w8) sum += part[w8 * 192 + tile * 64 + r * 8 + c];
          G0[ei][ej] = sum;
          J0[ei][ej] = (ei == ej) ? 1.0 : 0.0;
        }
        __syncthreads();
        // with a bye in the schedule, the block that sat out step 0 is first seen in step 1
        bool full = (step == 0);
        if (nbr != nb && step == 1) {
          int I0, J0b;
          for (int c = 0; c < nbr / 2; ++c) {
            rr_pair(nbr, 0, c, I0, J0b);
            if (J0b == nb && (I0 == I || I0 == J)) full = true;
          }
        }
        const int rounds = full ? m - 1 : b;
        int rotated = 0;
        float max_cos2 = 0.f;
        double (*Gc)[JG_P] = G0; double (*Gn)[JG_P] = G1;
        double (*Jc)[JG_P] = J0; double (*Jn)[JG_P] = J1;
        for (int is = 0; is < rounds; ++is) {
          if (threadIdx.x < b) {
            int p, q;
            if (full) rr_pair(m, is, threadIdx.x, p, q);
            else { p = threadIdx.x; q = b + (threadIdx.x + is) % b; }
            const double alpha = Gc[p][p], beta = Gc[q][q], gamma = Gc[p][q];
            double c = 1.0, sn = 0.0;
            if (gamma * gamma > tol * tol * alpha * beta) {
              ++rotated;
              max_cos2 = fmaxf(max_cos2, static_cast<float>(gamma * gamma) / static_cast<float>(alpha * beta));
              // The angle only has to shrink the inner product, so cos and sin are taken in fp32;
              // one Newton step on their norm in double then makes the rotation orthogonal to
              // double accuracy (the fp32 pair is off the unit circle by ~1e-7, the step squares that).
              const float zeta = static_cast<float>(beta - alpha) / (2.f * static_cast<float>(gamma));
              const float az = fabsf(zeta);
              const float t32 = (az > 1e15f) ? 0.5f / zeta : copysignf(1.f, zeta) / (az + sqrtf(1.f + az * az));
              const float c32 = rsqrtf(fmaf(t32, t32, 1.f));
              c = static_cast<double>(c32);
              sn = static_cast<double>(c32 * t32);
              const double fix = fma(-0.5, fma(c, c, sn * sn), 1.5);
              c *= fix;
              sn *= fix;
            }
            // column p' = c p - s q,  column q' = s p + c q
            coef[p].self = c; coef[p].other = -sn; coef[p].partner = q;
            coef[q].self = c; coef[q].other = sn;  coef[q].partner = p;
          }
          __syncthreads();
          {
            const JgCoef ci = coef[ei], cj = coef[ej];
            const int pi = ci.partner, pj = cj.partner;
            // G <- R^T G R and J <- J R for the round's rotation R (block diagonal after permutation)
            const double row_i = fma(cj.self, Gc[ei][ej], cj.other * Gc[ei][pj]);
            const double row_p = fma(cj.self, Gc[pi][ej], cj.other * Gc[pi][pj]);
            Gn[ei][ej] = fma(ci.self, row_i, ci.other * row_p);
            Jn[ei][ej] = fma(cj.self, Jc[ei][ej], cj.other * Jc[ei][pj]);
          }
          __syncthreads();
          double (*tg)[JG_P] = Gc; Gc = Gn; Gn = tg;
          double (*tj)[JG_P] = Jc; Jc = Jn; Jn = tj;
        }
        if (threadIdx.x < b && rotated) {
          atomicAdd(&visit_rotated, rotated);
          atomicAdd(&info->rotations[sweep], rotated);
          atomicMax(&info->max_cos2[sweep], __float_as_int(max_cos2));   // non-negative floats order as ints
        }
        __syncthreads();
        if (visit_rotated) {
          // ---- columns <- columns * J, eight rows at a time; a warp reads only the rows it writes
          double b0[4], b1[4];
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) { b0[kk] = Jc[kk * 4 + q4][g]; b1[kk] = Jc[kk * 4 + q4][8 + g]; }
          for (int band = warp; band < n / 8; band += 8) {
            const int r = band * 8 + g;
            double o0[2] = {0.0, 0.0}, o1[2] = {0.0, 0.0};
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
              const double a = cols[(kk * 4 + q4) * ns + r];
              dmma_884(o0, a, b0[kk]);
              dmma_884(o1, a, b1[kk]);
            }
            cols[(2 * q4) * ns + r] = o0[0];
            cols[(2 * q4 + 1) * ns + r] = o0[1];
            cols[(8 + 2 * q4) * ns + r] = o1[0];
            cols[(8 + 2 * q4 + 1) * ns + r] = o1[1];
          }
          __syncthreads();
          for (int lc = warp; lc < m; lc += 8) {
            double* dstg = At + static_cast<long long>(lc < b ? I * b + lc : J * b + (lc - b)) * n;
            const double* srcs = cols + lc * ns;
            for (int r = lane; r < n; r += 32) dstg[r] = srcs[r];
          }
        }
      }
      if (CLUSTER) {
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
      } else {
        alive = grid_barrier(&info->bar, ++bar * nctas, poll_limit);
      }
    }
    if (alive) {
      const int rot = *reinterpret_cast<volatile int*>(&info->rotations[sweep]);
      const float mc2 = __int_as_float(*reinterpret_cast<volatile int*>(&info->max_cos2[sweep]));
      converged = (rot == 0) || (mc2 < 1e-8f);
    }
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    info->sweeps = sweep;
    if (!alive && dev_status) atomicOr(dev_status, DEV_WAIT_EXPIRED);
    else if (!converged && dev_status) atomicOr(dev_status, DEV_JACOBI_NOCONV);
  }
}

// norms[i] = || column i of A || (row i of At): the shifted eigenvalues.
__global__ void __launch_bounds__(128) jacobi_norms_kernel(const double* __restrict__ At, int n, double* __restrict__ norms) {
  __shared__ double red[4];
  const double* row = At + static_cast<long long>(blockIdx.x) * n;
  double s = 0.0;
  for (int r = threadIdx.x; r < n; r += blockDim.x) s = fma(row[r], row[r], s);
  s = warp_sum(s);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x == 0) norms[blockIdx.x] = sqrt(red[0] + red[1] + red[2] + red[3]);
}

// Rank the eigenvalues and gather the unit eigenvectors of the k largest into Wsel (ell x k,
// float), largest first; ties go to the lower index.  One CTA per eigenvalue.
__global__ void __launch_bounds__(128) select_topk_kernel(const double* __restrict__ At, const double* __restrict__ norms,
                                                          int n, int ell, int k, float* __restrict__ Wsel) {
  const int i = blockIdx.x;
  const double li = norms[i];
  __shared__ int rank_sh;
  if (threadIdx.x == 0) rank_sh = 0;
  __syncthreads();
  int cnt = 0;
  for (int j = threadIdx.x; j < n; j += blockDim.x) {
    const double lj = norms[j];
    if (lj > li || (lj == li && j < i)) ++cnt;
  }
  atomicAdd(&rank_sh, cnt);
  __syncthreads();
  const int rank = rank_sh;
  if (rank >= k) return;
  const double inv = li > 0.0 ? 1.0 / li : 0.0;
  for (int a = threadIdx.x; a < ell; a += blockDim.x)
    if (PRAC_IN(static_cast<long long>(a) * k + rank, static_cast<long long>(ell) * k))
      Wsel[static_cast<long long>(a) * k + rank] = static_cast<float>(At[static_cast<long long>(i) * n + a] * inv);
}

// Pb[i][j] = bf16(P[i][j]);  PTb[j][i] = bf16(P[i][j]); 32 x 32 tiles through shared memory.
__global__ void __launch_bounds__(256) make_bf16_copies_kernel(const float* __restrict__ P, long long ldp,
                                                               long long d, long long s,
                                                               __nv_bfloat16* __restrict__ Pb, long long ldpb,
                                                               __nv_bfloat16* __restrict__ PTb, long long ldptb,
                                                               __nv_bfloat16* __restrict__ Pcb, long long k, float c) {
  __shared__ float tile[32][33];
  const long long i0 = static_cast<long long>(blockIdx.y) * 32, j0 = static_cast<long long>(blockIdx.x) * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;  // 32 x 8
  for (int r = ty; r < 32; r += 8) {
    const long long i = i0 + r, j = j0 + tx;
    const float v = (i < d && j < s) ? P[i * ldp + j] : 0.f;
    tile[r][tx] = v;
    if (i < d && j < s && PRAC_IN(i * ldpb + j, (d - 1) * ldpb + s)) {
      Pb[i * ldpb + j] = __float2bfloat16_rn(v);
      Pcb[i * ldpb + j] = __float2bfloat16_rn(j >= k ? c * v : v);   // [U | c Q]: operand of the rebuilt input
    }
  }
  __syncthreads();
  for (int r = ty; r < 32; r += 8) {
    const long long j = j0 + r, i = i0 + tx;
    if (i < d && j < s && PRAC_IN(j * ldptb + i, (s - 1) * ldptb + d)) PTb[j * ldptb + i] = __float2bfloat16_rn(tile[tx][r]);
  }
}

// x = hi + mid + lo, each piece a bf16 (round to nearest); the remainders are exact in fp32.
// One thread per 8 consecutive elements of a destination row (ldd is a multiple of 8).
__device__ __forceinline__ void split3_one(float x, __nv_bfloat16& hi, __nv_bfloat16& mid, __nv_bfloat16& lo) {
  hi = __float2bfloat16_rn(x);
  x -= __bfloat162float(hi);
  mid = __float2bfloat16_rn(x);
  x -= __bfloat162float(mid);
  lo = __float2bfloat16_rn(x);
}
__global__ void __launch_bounds__(256) split3_kernel(const float* __restrict__ src, long long lds, long long rows,
                                                     long long cols, __nv_bfloat16* __restrict__ dst,
                                                     long long rows_pad, long long ldd) {
  const long long groups = ldd / 8;
  const long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
  if (idx >= rows_pad * groups) return;
  const long long i = idx / groups, j0 = (idx - i * groups) * 8;
  float x[8];
  const float* s = src + i * lds + j0;
  if (i < rows && j0 + 8 <= cols && (reinterpret_cast<uintptr_t>(s) & 15u) == 0) {
    const float4 a = __ldg(reinterpret_cast<const float4*>(s)), b = __ldg(reinterpret_cast<const float4*>(s) + 1);
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
  } else {
#pragma unroll
    for (int e = 0; e < 8; ++e) x[e] = (i < rows && j0 + e < cols) ? s[e] : 0.f;
  }
  __align__(16) __nv_bfloat16 hi[8], mid[8], lo[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) split3_one(x[e], hi[e], mid[e], lo[e]);
  const long long o = i * ldd + j0, plane = rows_pad * ldd;
  *reinterpret_cast<uint4*>(dst + o) = *reinterpret_cast<const uint4*>(hi);
  *reinterpret_cast<uint4*>(dst + plane + o) = *reinterpret_cast<const uint4*>(mid);
  *reinterpret_cast<uint4*>(dst + 2 * plane + o) = *reinterpret_cast<const uint4*>(lo);
}

// The transpose of scale * src (rows x cols, fp32) as three bf16 pieces side by side: dst[j][l],
// dst[j][kp + l], dst[j][2 kp + l] = leading, middle and last piece of scale * src[l][j]; l >= rows
// is filled with zeros.  (A small matrix: the K-major second operand of a panel product.)
__global__ void __launch_bounds__(256) split3_transposed_kernel(const float* __restrict__ src, long long lds, long long rows,
                                                                long long cols, float scale,
                                                                __nv_bfloat16* __restrict__ dst, long long kp) {
  const long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
  if (idx >= cols * kp) return;
  const long long j = idx / kp, l = idx - j * kp;
  float x = 0.f;
  if (l < rows && PRAC_IN(l * lds + j, (rows - 1) * lds + cols)) x = scale * src[l * lds + j];
  __nv_bfloat16 hi, mid, lo;
  split3_one(x, hi, mid, lo);
  __nv_bfloat16* o = dst + j * 3 * kp + l;
  o[0] = hi; o[kp] = mid; o[2 * kp] = lo;
}

// The three pieces of a row side by side: dst[i] = [hi_i | mid_i | lo_i], each kp wide.
__global__ void __launch_bounds__(256) split3_cols_kernel(const float* __restrict__ src, long long lds, long long rows,
                                                          long long cols, __nv_bfloat16* __restrict__ dst, long long kp) {
  const long long groups = kp / 8;
  const long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
  if (idx >= rows * groups) return;
  const long long i = idx / groups, j0 = (idx - i * groups) * 8;
  float x[8];
  const float* s = src + i * lds + j0;
  if (j0 + 8 <= cols && (reinterpret_cast<uintptr_t>(s) & 15u) == 0) {
    const float4 a = __ldg(reinterpret_cast<const float4*>(s)), b = __ldg(reinterpret_cast<const float4*>(s) + 1);
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
  } else {
#pragma unroll
    for (int e = 0; e < 8; ++e) x[e] = (j0 + e < cols) ? s[e] : 0.f;
  }
  __align__(16) __nv_bfloat16 hi[8], mid[8], lo[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) split3_one(x[e], hi[e], mid[e], lo[e]);
  __nv_bfloat16* o = dst + i * 3 * kp + j0;
  *reinterpret_cast<uint4*>(o) = *reinterpret_cast<const uint4*>(hi);
  *reinterpret_cast<uint4*>(o + kp) = *reinterpret_cast<const uint4*>(mid);
  *reinterpret_cast<uint4*>(o + 2 * kp) = *reinterpret_cast<const uint4*>(lo);
}

// dX = dY * f'(Xh), element-wise (fp32 storage).
__global__ void __launch_bounds__(256) act_backward_f32_kernel(const float* __restrict__ Xh, long long ldxh,
                                                               const float* __restrict__ dY, long long lddy,
                                                               float* __restrict__ dX, long long lddx,
                                                               long long rows, long long cols, int act) {
  const long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
  if (idx >= rows * cols) return;
  const long long i = idx / cols, j = idx % cols;
  if (!PRAC_IN(i * lddx + j, (rows - 1) * lddx + cols) || !PRAC_IN(i * lddy + j, (rows - 1) * lddy + cols) ||
      !PRAC_IN(i * ldxh + j, (rows - 1) * ldxh + cols)) return;
  dX[i * lddx + j] = dY[i * lddy + j] * act_derivative(Xh[i * ldxh + j], act);
}

// Column sums of the pass-1 partials, shared by the two reductions below: a CTA closes 32 columns.
// Thread (g, q) adds, for the four columns 4q .. 4q + 3 of the CTA's 32, the partials of the 32-row
// blocks b = g, g + 32, ... (16-byte loads when the rows of col_part allow it); the 32 subtotals
// of a column are then combined in a fixed order, so the result does not depend on timing.
// Returns the column total in the threads with g == 0 && q < 8 as four values (columns 4q + e).
__device__ __forceinline__ void column_totals(const float* __restrict__ col_part, long long blocks, long long N,
                                              long long col0, float (&sub)[32][33], float (&tot)[4]) {
  const int g = threadIdx.x >> 3, q = threadIdx.x & 7;
  const long long c = col0 + 4 * q;
  float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
  const bool vec = (N % 4 == 0) && ((reinterpret_cast<uintptr_t>(col_part) & 15u) == 0) && c + 4 <= N;
  if (vec) {
#pragma unroll 16
    for (long long b = g; b < blocks; b += 32) {
      const float4 v = __ldg(reinterpret_cast<const float4*>(col_part + b * N + c));
      a0 += v.x; a1 += v.y; a2 += v.z; a3 += v.w;
    }
  } else {
    for (long long b = g; b < blocks; b += 32) {
      const float* r = col_part + b * N;
      if (c < N) a0 += r[c];
      if (c + 1 < N) a1 += r[c + 1];
      if (c + 2 < N) a2 += r[c + 2];
      if (c + 3 < N) a3 += r[c + 3];
    }
  }
  __syncthreads();                // an earlier call's readers are done with `sub`
  sub[g][4 * q] = a0; sub[g][4 * q + 1] = a1; sub[g][4 * q + 2] = a2; sub[g][4 * q + 3] = a3;
  __syncthreads();
  tot[0] = tot[1] = tot[2] = tot[3] = 0.f;
  if (g == 0) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      float t = 0.f;
#pragma unroll 8
      for (int h = 0; h < 32; ++h) t += sub[h][4 * q + e];
      tot[e] = t;
    }
  }
}

// After pass 1 of the RMSNorm backward.  The first ceil(M / 256) CTAs close the row sums (one
// thread per token); each of the others closes 32 column sums (column_totals).
__global__ void __launch_bounds__(256) rms_reduce_kernel(const float* __restrict__ row_part, int parts,
                                                         const float* __restrict__ col_part, long long blocks,
                                                         const float* __restrict__ rstd, long long M, long long N,
                                                         float* __restrict__ row_b, float* __restrict__ dgain) {
  __shared__ float sub[32][33];
  const long long row_ctas = (M + 255) / 256;
  if (blockIdx.x < row_ctas) {
    const long long idx = blockIdx.x * 256ll + threadIdx.x;
    if (idx < M) {
      float u = 0.f;
#pragma unroll 16
      for (int p = 0; p < parts; ++p) u += row_part[static_cast<long long>(p) * M + idx];
      const float rs = rstd[idx];
      row_b[idx] = rs * rs * rs * u / static_cast<float>(N);
    }
    return;
  }
  const long long col0 = (blockIdx.x - row_ctas) * 32;
  float tot[4];
  column_totals(col_part, blocks, N, col0, sub, tot);
  if (threadIdx.x < 8) {
#pragma unroll
    for (int e = 0; e < 4; ++e)
      if (col0 + 4 * threadIdx.x + e < N) dgain[col0 + 4 * threadIdx.x + e] = tot[e];
  }
}

// LayerNorm backward, the part that does not need the rebuilt input: per column i the sums over
// 512 tokens of dY[t][i] and of rstd[t] mean[t] dY[t][i].  Grid (ceil(N / 256), ceil(M / 512)).
// Thread (g, q) takes the eight columns 8q .. 8q + 7 of the CTA's 256 (one 16-byte load per row
// when VEC: rows of dY 16-byte aligned and padded to a multiple of 8) and the rows g, g + 8, ...
// of its 512; the eight subtotals of a column are combined in order.
template <bool VEC>
__global__ void __launch_bounds__(256) ln_colsum_partial_kernel(const __nv_bfloat16* __restrict__ dY, long long lddy,
                                                                const float* __restrict__ mean, const float* __restrict__ rstd,
                                                                long long M, long long N, float* __restrict__ part_plain,
                                                                float* __restrict__ part_w) {
  __shared__ float sp[8][257], sw[8][257];
  const int g = threadIdx.x >> 5, q = threadIdx.x & 31;
  const long long c0 = blockIdx.x * 256ll + 8 * q;
  const long long r0 = blockIdx.y * 512ll, r1 = (r0 + 512 < M) ? r0 + 512 : M;
  float ap[8], aw[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) ap[e] = aw[e] = 0.f;
  if (c0 < N) {
#pragma unroll 4
    for (long long t = r0 + g; t < r1; t += 8) {
      const float wgt = __ldg(rstd + t) * __ldg(mean + t);
      const __nv_bfloat16* row = dY + t * lddy + c0;
      if (VEC) {
        // (a group of eight that straddles the last column is still inside the padded row)
        const uint4 raw = __ldg(reinterpret_cast<const uint4*>(row));
        const __nv_bfloat16* h = reinterpret_cast<const __nv_bfloat16*>(&raw);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float v = __bfloat162float(h[e]);
          ap[e] += v;
          aw[e] = fmaf(wgt, v, aw[e]);
        }
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          if (c0 + e < N && PRAC_IN(t * lddy + c0 + e, (M - 1) * lddy + N)) {
            const float v = __bfloat162float(row[e]);
            ap[e] += v;
            aw[e] = fmaf(wgt, v, aw[e]);
          }
        }
      }
    }
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) { sp[g][8 * q + e] = ap[e]; sw[g][8 * q + e] = aw[e]; }
  __syncthreads();
  const long long col = blockIdx.x * 256ll + threadIdx.x;
  if (col < N) {
    float tp = 0.f, tw = 0.f;
#pragma unroll
    for (int h = 0; h < 8; ++h) { tp += sp[h][threadIdx.x]; tw += sw[h][threadIdx.x]; }
    part_plain[blockIdx.y * N + col] = tp;
    part_w[blockIdx.y * N + col] = tw;
  }
}

// After pass 1 of the LayerNorm backward (layout as rms_reduce_kernel).  Rows: with S = sum_i a x,
// A = sum_i a (a = gain dY): u = rstd (S - mean A); row_b = rstd^2 u / N; row_c = -rstd A / N + row_b mean.
// Columns: dgain = sum of the pass-1 column partials - sum of the weighted partials; dbias = sum
// of the plain partials.
__global__ void __launch_bounds__(256) ln_reduce_kernel(const float* __restrict__ row_part, const float* __restrict__ row_part2,
                                                        int parts, const float* __restrict__ col_part, long long blocks,
                                                        const float* __restrict__ part_plain, const float* __restrict__ part_w,
                                                        long long groups, const float* __restrict__ mean,
                                                        const float* __restrict__ rstd, long long M, long long N,
                                                        float* __restrict__ row_b, float* __restrict__ row_c,
                                                        float* __restrict__ dgain, float* __restrict__ dbias) {
  __shared__ float sub[32][33];
  const long long row_ctas = (M + 255) / 256;
  if (blockIdx.x < row_ctas) {
    const long long idx = blockIdx.x * 256ll + threadIdx.x;
    if (idx < M) {
      float S = 0.f, A = 0.f;
      for (int p = 0; p < parts; ++p) {
        S += row_part[static_cast<long long>(p) * M + idx];
        A += row_part2[static_cast<long long>(p) * M + idx];
      }
      const float rs = rstd[idx], mu = mean[idx], inv = 1.f / static_cast<float>(N);
      const float u = rs * (S - mu * A);
      const float rb = rs * rs * u * inv;
      row_b[idx] = rb;
      row_c[idx] = fmaf(rb, mu, -rs * A * inv);
    }
    return;
  }
  const long long col0 = (blockIdx.x - row_ctas) * 32;
  float tot[4], tw[4], tp[4];
  column_totals(col_part, blocks, N, col0, sub, tot);
  column_totals(part_w, groups, N, col0, sub, tw);
  column_totals(part_plain, groups, N, col0, sub, tp);
  if (threadIdx.x < 8) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const long long col = col0 + 4 * threadIdx.x + e;
      if (col < N) {
        dgain[col] = tot[e] - tw[e];
        dbias[col] = tp[e];
      }
    }
  }
}

// fp32 storage, one CTA per token: A = sum a, S = sum a xn (a = gain dY, xn = (x - mean) rstd), then
// dX = rstd (a - A / N - xn S / N).
__global__ void __launch_bounds__(256) ln_rows_f32_kernel(const float* __restrict__ Xh, long long ldxh,
                                                          const float* __restrict__ dY, long long lddy,
                                                          const float* __restrict__ mean, const float* __restrict__ rstd,
                                                          const float* __restrict__ gain, float* __restrict__ dX,
                                                          long long lddx, long long N) {
  __shared__ double ra[256], rb[256];
  const long long t = blockIdx.x;
  const float* x = Xh + t * ldxh;
  const float* y = dY + t * lddy;
  const float mu = mean[t], rs = rstd[t];
  double A = 0.0, S = 0.0;
  for (long long i = threadIdx.x; i < N; i += blockDim.x) {
    const double a = static_cast<double>(gain[i]) * y[i];
    A += a;
    S += a * ((x[i] - mu) * rs);
  }
  ra[threadIdx.x] = A; rb[threadIdx.x] = S;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o) { ra[threadIdx.x] += ra[threadIdx.x + o]; rb[threadIdx.x] += rb[threadIdx.x + o]; }
    __syncthreads();
  }
  const float mA = static_cast<float>(ra[0] / static_cast<double>(N)), mS = static_cast<float>(rb[0] / static_cast<double>(N));
  for (long long i = threadIdx.x; i < N; i += blockDim.x)
    dX[t * lddx + i] = rs * (gain[i] * y[i] - mA - (x[i] - mu) * rs * mS);
}
// fp32 storage: dgain_i = sum_t dY_ti xn_ti, dbias_i = sum_t dY_ti; one thread per column, rows in order.
__global__ void __launch_bounds__(256) ln_cols_f32_kernel(const float* __restrict__ Xh, long long ldxh,
                                                          const float* __restrict__ dY, long long lddy,
                                                          const float* __restrict__ mean, const float* __restrict__ rstd,
                                                          float* __restrict__ dgain, float* __restrict__ dbias,
                                                          long long M, long long N) {
  const long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
  if (i >= N) return;
  double sg = 0.0, sb = 0.0;
  for (long long t = 0; t < M; ++t) {
    const double y = dY[t * lddy + i];
    sg += y * ((Xh[t * ldxh + i] - mean[t]) * rstd[t]);
    sb += y;
  }
  dgain[i] = static_cast<float>(sg);
  dbias[i] = static_cast<float>(sb);
}

// fp32 storage, one CTA per token: u = sum_i gain_i dY_i x_i, then dX = rstd gain dY - rstd^3 u / N x.
__global__ void __launch_bounds__(256) rms_rows_f32_kernel(const float* __restrict__ Xh, long long ldxh,
                                                           const float* __restrict__ dY, long long lddy,
                                                           const float* __restrict__ rstd, const float* __restrict__ gain,
                                                           float* __restrict__ dX, long long lddx, long long N) {
  __shared__ double red[256];
  const long long t = blockIdx.x;
  const float* x = Xh + t * ldxh;
  const float* y = dY + t * lddy;
  double u = 0.0;
  for (long long i = threadIdx.x; i < N; i += blockDim.x) u += static_cast<double>(gain[i]) * y[i] * x[i];
  red[threadIdx.x] = u;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
    __syncthreads();
  }
  const float rs = rstd[t];
  const float coef = static_cast<float>(static_cast<double>(rs) * rs * rs * red[0] / static_cast<double>(N));
  for (long long i = threadIdx.x; i < N; i += blockDim.x) dX[t * lddx + i] = rs * gain[i] * y[i] - coef * x[i];
}
// fp32 storage: dgain_i = sum_t dY_ti x_ti rstd_t, one thread per column, rows in order.
__global__ void __launch_bounds__(256) rms_cols_f32_kernel(const float* __restrict__ Xh, long long ldxh,
                                                           const float* __restrict__ dY, long long lddy,
                                                           const float* __restrict__ rstd, float* __restrict__ dgain,
                                                           long long M, long long N) {
  const long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
  if (i >= N) return;
  double sacc = 0.0;
  for (long long t = 0; t < M; ++t) sacc += static_cast<double>(dY[t * lddy + i]) * Xh[t * ldxh + i] * rstd[t];
  dgain[i] = static_cast<float>(sacc);
}

// dst (bf16) = src with columns from `from` on multiplied by scale.
__global__ void __launch_bounds__(256) scale_to_bf16_kernel(const float* __restrict__ src, long long lds,
                                                            long long rows, long long cols, long long from, float scale,
                                                            __nv_bfloat16* __restrict__ dst, long long ldd) {
  const long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
  if (idx >= rows * cols) return;
  const long long i = idx / cols, j = idx % cols;
  if (!PRAC_IN(i * lds + j, (rows - 1) * lds + cols) || !PRAC_IN(i * ldd + j, (rows - 1) * ldd + cols)) return;
  const float v = src[i * lds + j];
  dst[i * ldd + j] = __float2bfloat16_rn(j >= from ? scale * v : v);
}

__global__ void copy2d_kernel(const float* __restrict__ src, long long lds, float* __restrict__ dst,
                              long long ldd, long long rows, long long cols) {
  const long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
  if (idx >= rows * cols) return;
  const long long i = idx / cols, j = idx % cols;
  if (!PRAC_IN(i * lds + j, (rows - 1) * lds + cols) || !PRAC_IN(i * ldd + j, (rows - 1) * ldd + cols)) return;
  dst[i * ldd + j] = src[i * lds + j];
}

// dst (rows x cols bf16, leading dimension ldd: rows 16-byte aligned, zero beyond cols up to ldd)
// = src (rows x cols bf16, any leading dimension, 2-byte aligned).  One thread per 8 destination
// elements: eight 2-byte loads (coalesced across the warp), one 16-byte store.
__global__ void __launch_bounds__(256) repack_rows_bf16_kernel(const __nv_bfloat16* __restrict__ src, long long lds,
                                                               long long rows, long long cols,
                                                               __nv_bfloat16* __restrict__ dst, long long ldd) {
  const long long groups = ldd / 8;
  const long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
  if (idx >= rows * groups) return;
  const long long i = idx / groups, j0 = (idx - i * groups) * 8;
  const unsigned short* s16 = reinterpret_cast<const unsigned short*>(src + i * lds + j0);
  unsigned short v[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) v[e] = (j0 + e < cols) ? __ldg(s16 + e) : static_cast<unsigned short>(0);
  if (!PRAC_IN(i * ldd + j0 + 7, rows * ldd)) return;
  uint4 o;
  o.x = v[0] | (static_cast<uint32_t>(v[1]) << 16);
  o.y = v[2] | (static_cast<uint32_t>(v[3]) << 16);
  o.z = v[4] | (static_cast<uint32_t>(v[5]) << 16);
  o.w = v[6] | (static_cast<uint32_t>(v[7]) << 16);
  *reinterpret_cast<uint4*>(dst + i * ldd + j0) = o;
}

inline unsigned nblocks(long long work, int threads) {
  return static_cast<unsigned>((work + threads - 1) / threads);
}

}  // namespace

PRAC_BOUNDS_READER(bounds_violations_panel)

int launch_repack_rows_bf16(const __nv_bfloat16* src, int64_t lds, int64_t rows, int64_t cols, __nv_bfloat16* dst,
                            int64_t ldd, cudaStream_t stream) {
  if (rows <= 0 || cols <= 0) return PRAC_OK;
  if (ldd % 8 != 0 || ldd < cols || (reinterpret_cast<uintptr_t>(dst) & 15u) != 0) return PRAC_EALIGN;
  repack_rows_bf16_kernel<<<nblocks(rows * (ldd / 8), 256), 256, 0, stream>>>(src, lds, rows, cols, dst, ldd);
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

int launch_philox_words(uint64_t seed, uint64_t dc, int64_t n, uint32_t* out, cudaStream_t stream) {
  if (n <= 0) return PRAC_OK;
  philox_words_kernel<<<nblocks((n + 3) / 4, 256), 256, 0, stream>>>(seed, dc, n, out);
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

int launch_gaussian(uint64_t seed, uint64_t dc, int64_t d, int64_t r, float* S, int64_t lds,
                    cudaStream_t stream) {
  if (d <= 0 || r <= 0) return PRAC_OK;
  gaussian_kernel<<<nblocks((d * r + 3) / 4, 256), 256, 0, stream>>>(seed, dc, d, r, S, lds);
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

// Eigen-solver workspace: At n*n double | norms n double | info   (n = ell rounded up to 16)
namespace {
struct JacWs { double* At; double* norms; JacobiInfo* info; size_t bytes; int64_t n; };
JacWs carve_jac(void* ws, int64_t ell) {
  JacWs j;
  j.n = round_up(ell, 16);
  size_t off = 0;
  auto take = [&](size_t b) { size_t o = off; off += (b + 255) / 256 * 256; return o; };
  const size_t o1 = take(j.n * j.n * 8), o2 = take(j.n * 8), o3 = take(sizeof(JacobiInfo));
  char* b = static_cast<char*>(ws);
  j.At = reinterpret_cast<double*>(b + o1); j.norms = reinterpret_cast<double*>(b + o2);
  j.info = reinterpret_cast<JacobiInfo*>(b + o3);
  j.bytes = off;
  return j;
}
}  // namespace

size_t jacobi_ws_bytes(int64_t ell) { return ell > 0 ? carve_jac(nullptr, ell).bytes : 0; }

int jacobi_read_sweeps(void* ws, int64_t ell, int* sweeps, cudaStream_t stream) {
  if (!ws || ell <= 0 || !sweeps) return PRAC_EINVAL;
  const JacWs j = carve_jac(ws, ell);
  PRAC_CUDA_TRY(cudaStreamSynchronize(stream));
  JacobiInfo h;
  PRAC_CUDA_TRY(cudaMemcpy(&h, j.info, sizeof(JacobiInfo), cudaMemcpyDeviceToHost));
  *sweeps = h.sweeps;
  return PRAC_OK;
}

int jacobi_topk(const double* B, int64_t ldb, int64_t ell, int64_t k, float* Wsel, void* ws, size_t ws_bytes,
                int* dev_status, cudaStream_t stream) {
  if (ell <= 0 || k <= 0 || k > ell || ldb < ell) return PRAC_EINVAL;
  const JacWs j = carve_jac(ws, ell);
  if (ws == nullptr || ws_bytes < j.bytes) return PRAC_EWORKSPACE;
  const int n = static_cast<int>(j.n);
  // columns per block: as many as fit in shared memory, two blocks per CTA, at least two blocks
  // 8 columns per block = 256 threads per CTA: measured faster than 16 (more CTAs share the
  // rotations, and the 20-element register variant fits the register file)
  int bcols = 8;
  while (bcols > 4 && static_cast<size_t>(2 * bcols) * n * 8 > 200u * 1024u) bcols /= 2;
  const size_t smem = static_cast<size_t>(2 * bcols) * n * 8;
  if (smem > 200u * 1024u) return PRAC_EINVAL;
  void (*kern)(double*, int, int, int, double, JacobiInfo*, int*, unsigned) =
      n <= 32 * 12 ? jacobi_kernel<12> : (n <= 32 * 20 ? jacobi_kernel<20> : jacobi_kernel<0>);
  int sms = 0, dev = 0, per_sm = 0;
  PRAC_CUDA_TRY(cudaGetDevice(&dev));
  static DeviceOnce attr_set;      // function attributes belong to the device that was current
  if (!attr_set.done(dev)) {
    PRAC_CUDA_TRY(cudaFuncSetAttribute(jacobi_kernel<12>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    PRAC_CUDA_TRY(cudaFuncSetAttribute(jacobi_kernel<20>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    PRAC_CUDA_TRY(cudaFuncSetAttribute(jacobi_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    attr_set.mark(dev);
  }
  const int nb = n / bcols;
  const int grid = (nb + (nb & 1)) / 2;
  PRAC_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  // 8-column blocks take the Gram-matrix kernel; narrower blocks (very long columns) the plain one
  const bool gram = (bcols == JG_B);
  const size_t gram_smem = (static_cast<size_t>(JG_M) * (n + 4) + 4 * JG_M * JG_P + 8 * 3 * 64) * 8 + JG_M * sizeof(JgCoef);
  if (gram) {
    static DeviceOnce gram_attr;
    if (!gram_attr.done(dev)) {
      PRAC_CUDA_TRY(cudaFuncSetAttribute(jacobi_gram_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024));
      PRAC_CUDA_TRY(cudaFuncSetAttribute(jacobi_gram_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024));
      gram_attr.mark(dev);
    }
    PRAC_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, jacobi_gram_kernel<false>, 256, gram_smem));
  } else {
    PRAC_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, 32 * bcols, smem));
  }
  if (per_sm < 1 || grid > per_sm * sms) return PRAC_EINVAL;   // the barrier needs every CTA resident
  jacobi_prepare_kernel<<<64, 256, 0, stream>>>(B, ldb, static_cast<int>(ell), j.At, n, j.info);
  count_launch();
  double* at = j.At;
  int ni = n, bi = bcols, max_sweeps = JAC_MAX_SWEEPS;
  // a pair of columns whose cosine is below this is left alone: far below what the fp32 result keeps
  double tol = 1e-9;
  JacobiInfo* info = j.info;
  unsigned poll_limit = barrier_poll_limit();
  if (gram) {
    // Up to 16 CTAs (eigenproblems up to 256 columns: the Rayleigh-Ritz windows of k <= 512) run as
    // one cluster on the hardware barrier (more than 8 CTAs is a cluster size the device has to
    // allow and be able to place: the occupancy query below decides), unless a test has shortened
    // the software barrier's poll limit, which only that barrier can honour.
    bool as_cluster = grid <= 16 && poll_limit == GRID_BARRIER_POLLS;
    if (as_cluster && grid > 8) {
      static DeviceOnce wide_attr;
      if (!wide_attr.done(dev)) {
        if (cudaFuncSetAttribute(jacobi_gram_kernel<true>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) {
          (void)cudaGetLastError();
          as_cluster = false;
        } else {
          wide_attr.mark(dev);
        }
      }
    }
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    if (as_cluster) {
      cfg.gridDim = dim3(grid);
      cfg.blockDim = dim3(256);
      cfg.dynamicSmemBytes = gram_smem;
      cfg.stream = stream;
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = grid;
      attr[0].val.clusterDim.y = 1;
      attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr;
      cfg.numAttrs = 1;
      int clusters = 0;
      if (cudaOccupancyMaxActiveClusters(&clusters, jacobi_gram_kernel<true>, &cfg) != cudaSuccess || clusters < 1) {
        (void)cudaGetLastError();
        as_cluster = false;
      }
    }
    if (as_cluster) {
      PRAC_CUDA_TRY(cudaLaunchKernelEx(&cfg, jacobi_gram_kernel<true>, at, ni, max_sweeps, tol, info, dev_status, poll_limit));
    } else {
      void* gargs[] = {&at, &ni, &max_sweeps, &tol, &info, &dev_status, &poll_limit};
      PRAC_CUDA_TRY(cudaLaunchCooperativeKernel(reinterpret_cast<void*>(jacobi_gram_kernel<false>), dim3(grid), dim3(256),
                                                gargs, gram_smem, stream));
    }
  } else {
    void* args[] = {&at, &ni, &bi, &max_sweeps, &tol, &info, &dev_status, &poll_limit};
    PRAC_CUDA_TRY(cudaLaunchCooperativeKernel(reinterpret_cast<void*>(kern), dim3(grid), dim3(32 * bcols), args,
                                              smem, stream));
  }
  count_launch();
  jacobi_norms_kernel<<<n, 128, 0, stream>>>(j.At, n, j.norms);
  count_launch();
  select_topk_kernel<<<n, 128, 0, stream>>>(j.At, j.norms, n, static_cast<int>(ell), static_cast<int>(k), Wsel);
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

int launch_make_bf16_copies(const float* P, int64_t ldp, int64_t d, int64_t s, int64_t k, double c,
                            __nv_bfloat16* Pcb, __nv_bfloat16* Pb, int64_t ldpb,
                            __nv_bfloat16* PTb, int64_t ldptb, cudaStream_t stream) {
  dim3 grid(static_cast<unsigned>((s + 31) / 32), static_cast<unsigned>((d + 31) / 32));
  make_bf16_copies_kernel<<<grid, 256, 0, stream>>>(P, ldp, d, s, Pb, ldpb, PTb, ldptb, Pcb, k, static_cast<float>(c));
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

int launch_split3(const float* src, int64_t lds, int64_t rows, int64_t cols, __nv_bfloat16* dst,
                  int64_t rows_pad, int64_t ldd, cudaStream_t stream) {
  if (rows <= 0 || cols <= 0) return PRAC_OK;
  if (ldd % 8 != 0 || (reinterpret_cast<uintptr_t>(dst) & 15u) != 0) return PRAC_EALIGN;
  split3_kernel<<<nblocks(rows_pad * (ldd / 8), 256), 256, 0, stream>>>(src, lds, rows, cols, dst, rows_pad, ldd);
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

int launch_split3_transposed(const float* src, int64_t lds, int64_t rows, int64_t cols, float scale,
                             __nv_bfloat16* dst, int64_t kp, cudaStream_t stream) {
  if (rows <= 0 || cols <= 0) return PRAC_OK;
  if (kp < rows) return PRAC_EINVAL;
  split3_transposed_kernel<<<nblocks(cols * kp, 256), 256, 0, stream>>>(src, lds, rows, cols, scale, dst, kp);
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

int launch_split3_cols(const float* src, int64_t lds, int64_t rows, int64_t cols, __nv_bfloat16* dst, int64_t kp,
                       cudaStream_t stream) {
  if (rows <= 0 || cols <= 0) return PRAC_OK;
  if (kp % 8 != 0 || kp < cols || (reinterpret_cast<uintptr_t>(dst) & 15u) != 0) return PRAC_EALIGN;
  split3_cols_kernel<<<nblocks(rows * (kp / 8), 256), 256, 0, stream>>>(src, lds, rows, cols, dst, kp);
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

int launch_rms_reduce(const float* row_part, int parts, const float* col_part, int64_t blocks, const float* rstd,
                      int64_t M, int64_t N, float* row_b, float* dgain, cudaStream_t stream) {
  const unsigned ctas = nblocks(M, 256) + nblocks(N, 32);
  rms_reduce_kernel<<<ctas, 256, 0, stream>>>(row_part, parts, col_part, blocks, rstd, M, N, row_b, dgain);
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

int launch_ln_colsum_partial(const __nv_bfloat16* dY, int64_t lddy, const float* mean, const float* rstd, int64_t M,
                             int64_t N, float* part_plain, float* part_w, cudaStream_t stream) {
  dim3 grid(nblocks(N, 256), nblocks(M, 512));
  const bool vec = (reinterpret_cast<uintptr_t>(dY) & 15u) == 0 && lddy % 8 == 0 && lddy >= (N + 7) / 8 * 8;
  if (vec) ln_colsum_partial_kernel<true><<<grid, 256, 0, stream>>>(dY, lddy, mean, rstd, M, N, part_plain, part_w);
  else ln_colsum_partial_kernel<false><<<grid, 256, 0, stream>>>(dY, lddy, mean, rstd, M, N, part_plain, part_w);
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

int launch_ln_reduce(const float* row_part, const float* row_part2, int parts, const float* col_part, int64_t blocks,
                     const float* part_plain, const float* part_w, int64_t groups, const float* mean, const float* rstd,
                     int64_t M, int64_t N, float* row_b, float* row_c, float* dgain, float* dbias, cudaStream_t stream) {
  const unsigned ctas = nblocks(M, 256) + nblocks(N, 32);
  ln_reduce_kernel<<<ctas, 256, 0, stream>>>(row_part, row_part2, parts, col_part, blocks, part_plain, part_w, groups,
                                             mean, rstd, M, N, row_b, row_c, dgain, dbias);
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

int launch_ln_backward_f32(const float* Xh, int64_t ldxh, const float* dY, int64_t lddy, const float* mean,
                           const float* rstd, const float* gain, float* dX, int64_t lddx, float* dgain, float* dbias,
                           int64_t M, int64_t N, cudaStream_t stream) {
  ln_rows_f32_kernel<<<static_cast<unsigned>(M), 256, 0, stream>>>(Xh, ldxh, dY, lddy, mean, rstd, gain, dX, lddx, N);
  count_launch();
  ln_cols_f32_kernel<<<nblocks(N, 256), 256, 0, stream>>>(Xh, ldxh, dY, lddy, mean, rstd, dgain, dbias, M, N);
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

int launch_rms_backward_f32(const float* Xh, int64_t ldxh, const float* dY, int64_t lddy, const float* rstd,
                            const float* gain, float* dX, int64_t lddx, float* dgain, int64_t M, int64_t N,
                            cudaStream_t stream) {
  rms_rows_f32_kernel<<<static_cast<unsigned>(M), 256, 0, stream>>>(Xh, ldxh, dY, lddy, rstd, gain, dX, lddx, N);
  count_launch();
  rms_cols_f32_kernel<<<nblocks(N, 256), 256, 0, stream>>>(Xh, ldxh, dY, lddy, rstd, dgain, M, N);
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

int launch_scale_to_bf16(const float* src, int64_t lds, int64_t rows, int64_t cols, int64_t from, float scale,
                         __nv_bfloat16* dst, int64_t ldd, cudaStream_t stream) {
  if (rows <= 0 || cols <= 0) return PRAC_OK;
  scale_to_bf16_kernel<<<nblocks(rows * cols, 256), 256, 0, stream>>>(src, lds, rows, cols, from, scale, dst, ldd);
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

int launch_act_backward_f32(const float* Xh, int64_t ldxh, const float* dY, int64_t lddy, float* dX, int64_t lddx,
                            int64_t rows, int64_t cols, int act, cudaStream_t stream) {
  if (rows <= 0 || cols <= 0) return PRAC_OK;
  act_backward_f32_kernel<<<nblocks(rows * cols, 256), 256, 0, stream>>>(Xh, ldxh, dY, lddy, dX, lddx, rows, cols, act);
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

int launch_copy2d(const float* src, int64_t lds, float* dst, int64_t ldd, int64_t rows, int64_t cols,
                  cudaStream_t stream) {
  if (rows <= 0 || cols <= 0) return PRAC_OK;
  copy2d_kernel<<<nblocks(rows * cols, 256), 256, 0, stream>>>(src, lds, dst, ldd, rows, cols);
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

}  // namespace prac
