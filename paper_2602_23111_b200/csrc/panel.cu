// Small-matrix kernels of the basis fit: the counter-based Gaussian draw, the cyclic Jacobi
// eigen-solver of the Rayleigh-Ritz step, and format conversions.
#include <cooperative_groups.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "internal.h"

namespace cg = cooperative_groups;

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
    for (int e = 0; e < 4 && e0 + e < n; ++e) out[e0 + e] = v[e];
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
    S[(idx / r) * lds + (idx % r)] = z[e];
  }
}

// ------------------------------------------------------------------ Jacobi eigen-solver
// Cyclic two-sided Jacobi with round-robin pairing.  One step applies n/2 disjoint plane
// rotations J: B <- J^T B J, W <- W J.  All 2x2 blocks (rows of pair i, columns of pair j)
// are independent, so one step is one pass over B (read `cur`, write `nxt`) and one grid
// synchronisation.  Every CTA derives the same rotations from the same data, so the
// convergence decision needs no communication.
struct JacobiInfo { int final_buf; int sweeps; };

__global__ void __launch_bounds__(256) jacobi_kernel(double* B0, double* B1, double* W, int n, int max_sweeps,
                                                     double tol, JacobiInfo* info, int* dev_status) {
  cg::grid_group grid = cg::this_grid();
  extern __shared__ unsigned char jsm[];
  const int half = n / 2;
  double* sc = reinterpret_cast<double*>(jsm);
  double* ss = sc + half;
  int* sp = reinterpret_cast<int*>(ss + half);
  int* sq = sp + half;
  __shared__ int rot_count;
  __shared__ double scale_sh;

  const long long gtid = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
  const long long gthreads = static_cast<long long>(gridDim.x) * blockDim.x;

  // W = I
  for (long long idx = gtid; idx < static_cast<long long>(n) * n; idx += gthreads)
    W[idx] = (idx / n == idx % n) ? 1.0 : 0.0;
  if (threadIdx.x == 0) {
    double m = 0.0;
    for (int i = 0; i < n; ++i) m = fmax(m, fabs(__ldcg(&B0[static_cast<long long>(i) * n + i])));
    scale_sh = m;
  }
  __syncthreads();
  const double abs_floor = 1e-17 * scale_sh;
  grid.sync();

  double* cur = B0;
  double* nxt = B1;
  int buf = 0, sweep = 0;
  bool converged = false;
  for (; sweep < max_sweeps && !converged; ++sweep) {
    if (threadIdx.x == 0) rot_count = 0;
    __syncthreads();
    for (int step = 0; step < n - 1; ++step) {
      for (int i = threadIdx.x; i < half; i += blockDim.x) {
        int a, b;
        if (i == 0) { a = n - 1; b = step; }
        else { a = (step + i) % (n - 1); b = (step - i + (n - 1)) % (n - 1); }
        const int p = a < b ? a : b, q = a < b ? b : a;
        const double bpp = __ldcg(&cur[static_cast<long long>(p) * n + p]);
        const double bqq = __ldcg(&cur[static_cast<long long>(q) * n + q]);
        const double bpq = __ldcg(&cur[static_cast<long long>(p) * n + q]);
        double c = 1.0, s = 0.0;
        if (fabs(bpq) > tol * sqrt(fabs(bpp * bqq)) + abs_floor) {
          const double tau = (bqq - bpp) / (2.0 * bpq);
          const double tt = (tau >= 0.0 ? 1.0 : -1.0) / (fabs(tau) + sqrt(1.0 + tau * tau));
          c = 1.0 / sqrt(1.0 + tt * tt);
          s = tt * c;
          atomicAdd(&rot_count, 1);
        }
        sp[i] = p; sq[i] = q; sc[i] = c; ss[i] = s;
      }
      __syncthreads();
      const long long nblk = static_cast<long long>(half) * half;
      for (long long blk = gtid; blk < nblk; blk += gthreads) {
        const int i = static_cast<int>(blk / half), j = static_cast<int>(blk % half);
        const int pi = sp[i], qi = sq[i], pj = sp[j], qj = sq[j];
        const double ci = sc[i], si = ss[i], cj = sc[j], sj = ss[j];
        const double a = __ldcg(&cur[static_cast<long long>(pi) * n + pj]), b = __ldcg(&cur[static_cast<long long>(pi) * n + qj]);
        const double c = __ldcg(&cur[static_cast<long long>(qi) * n + pj]), d = __ldcg(&cur[static_cast<long long>(qi) * n + qj]);
        const double t1 = ci * a - si * c, t2 = ci * b - si * d;
        const double t3 = si * a + ci * c, t4 = si * b + ci * d;
        double o11 = t1 * cj - t2 * sj, o12 = t1 * sj + t2 * cj;
        double o21 = t3 * cj - t4 * sj, o22 = t3 * sj + t4 * cj;
        if (i == j && si != 0.0) { o12 = 0.0; o21 = 0.0; }
        nxt[static_cast<long long>(pi) * n + pj] = o11; nxt[static_cast<long long>(pi) * n + qj] = o12;
        nxt[static_cast<long long>(qi) * n + pj] = o21; nxt[static_cast<long long>(qi) * n + qj] = o22;
      }
      const long long nw = static_cast<long long>(n) * half;
      for (long long idx = gtid; idx < nw; idx += gthreads) {
        const int a = static_cast<int>(idx / half), j = static_cast<int>(idx % half);
        const int pj = sp[j], qj = sq[j];
        const double cj = sc[j], sj = ss[j];
        if (sj != 0.0) {
          const double x = __ldcg(&W[static_cast<long long>(a) * n + pj]), y = __ldcg(&W[static_cast<long long>(a) * n + qj]);
          W[static_cast<long long>(a) * n + pj] = x * cj - y * sj;
          W[static_cast<long long>(a) * n + qj] = x * sj + y * cj;
        }
      }
      grid.sync();
      double* tmp = cur; cur = nxt; nxt = tmp;
      buf ^= 1;
    }
    converged = (rot_count == 0);
    __syncthreads();
  }
  if (gtid == 0) {
    info->final_buf = buf;
    info->sweeps = sweep;
    if (!converged && dev_status) atomicOr(dev_status, DEV_JACOBI_NOCONV);
  }
}

// Rank the eigenvalues (diagonal of the final buffer) and gather the eigenvectors of the k
// largest into Wsel (n x k, float), largest first.  One CTA per eigenvalue.
__global__ void __launch_bounds__(128) select_topk_kernel(const double* __restrict__ B0, const double* __restrict__ B1,
                                                          const double* __restrict__ W, int n, int k,
                                                          const JacobiInfo* __restrict__ info,
                                                          float* __restrict__ Wsel) {
  const double* B = info->final_buf ? B1 : B0;
  const int i = blockIdx.x;
  const double li = B[static_cast<long long>(i) * n + i];
  __shared__ int rank_sh;
  if (threadIdx.x == 0) rank_sh = 0;
  __syncthreads();
  int cnt = 0;
  for (int j = threadIdx.x; j < n; j += blockDim.x) {
    const double lj = B[static_cast<long long>(j) * n + j];
    if (lj > li || (lj == li && j < i)) ++cnt;
  }
  atomicAdd(&rank_sh, cnt);
  __syncthreads();
  const int rank = rank_sh;
  if (rank >= k) return;
  for (int a = threadIdx.x; a < n; a += blockDim.x)
    Wsel[static_cast<long long>(a) * k + rank] = static_cast<float>(W[static_cast<long long>(a) * n + i]);
}

__global__ void symmetrize_kernel(double* B, int n) {
  const long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
  if (idx >= static_cast<long long>(n) * n) return;
  const int i = static_cast<int>(idx / n), j = static_cast<int>(idx % n);
  if (j > i) {
    const double v = 0.5 * (B[idx] + B[static_cast<long long>(j) * n + i]);
    B[idx] = v;
    B[static_cast<long long>(j) * n + i] = v;
  }
}

// Pb[i][j] = bf16(P[i][j]);  PTb[j][i] = bf16(P[i][j]); 32 x 32 tiles through shared memory.
__global__ void __launch_bounds__(256) make_bf16_copies_kernel(const float* __restrict__ P, long long ldp,
                                                               long long d, long long s,
                                                               __nv_bfloat16* __restrict__ Pb, long long ldpb,
                                                               __nv_bfloat16* __restrict__ PTb, long long ldptb) {
  __shared__ float tile[32][33];
  const long long i0 = static_cast<long long>(blockIdx.y) * 32, j0 = static_cast<long long>(blockIdx.x) * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;  // 32 x 8
  for (int r = ty; r < 32; r += 8) {
    const long long i = i0 + r, j = j0 + tx;
    const float v = (i < d && j < s) ? P[i * ldp + j] : 0.f;
    tile[r][tx] = v;
    if (i < d && j < s) Pb[i * ldpb + j] = __float2bfloat16_rn(v);
  }
  __syncthreads();
  for (int r = ty; r < 32; r += 8) {
    const long long j = j0 + r, i = i0 + tx;
    if (i < d && j < s) PTb[j * ldptb + i] = __float2bfloat16_rn(tile[tx][r]);
  }
}

// x = hi + mid + lo, each piece a bf16 (round to nearest); the remainders are exact in fp32.
__global__ void split3_kernel(const float* __restrict__ src, long long lds, long long rows, long long cols,
                              __nv_bfloat16* __restrict__ dst, long long rows_pad, long long ldd) {
  const long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
  if (idx >= rows_pad * ldd) return;
  const long long i = idx / ldd, j = idx % ldd;
  float x = (i < rows && j < cols) ? src[i * lds + j] : 0.f;
  const __nv_bfloat16 hi = __float2bfloat16_rn(x);
  x -= __bfloat162float(hi);
  const __nv_bfloat16 mid = __float2bfloat16_rn(x);
  x -= __bfloat162float(mid);
  const __nv_bfloat16 lo = __float2bfloat16_rn(x);
  dst[idx] = hi;
  dst[rows_pad * ldd + idx] = mid;
  dst[2 * rows_pad * ldd + idx] = lo;
}

__global__ void copy2d_kernel(const float* __restrict__ src, long long lds, float* __restrict__ dst,
                              long long ldd, long long rows, long long cols) {
  const long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
  if (idx >= rows * cols) return;
  const long long i = idx / cols, j = idx % cols;
  dst[i * ldd + j] = src[i * lds + j];
}

inline unsigned nblocks(long long work, int threads) {
  return static_cast<unsigned>((work + threads - 1) / threads);
}

}  // namespace

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

// Jacobi workspace: B1 n*n double | W n*n double | info
namespace {
struct JacWs { double* B1; double* W; JacobiInfo* info; size_t bytes; };
JacWs carve_jac(void* ws, int64_t n) {
  JacWs j;
  size_t off = 0;
  auto take = [&](size_t b) { size_t o = off; off += (b + 255) / 256 * 256; return o; };
  const size_t o1 = take(n * n * 8), o2 = take(n * n * 8), o3 = take(sizeof(JacobiInfo));
  char* b = static_cast<char*>(ws);
  j.B1 = reinterpret_cast<double*>(b + o1); j.W = reinterpret_cast<double*>(b + o2);
  j.info = reinterpret_cast<JacobiInfo*>(b + o3);
  j.bytes = off;
  return j;
}
}  // namespace

size_t jacobi_ws_bytes(int64_t n) { return n > 0 ? carve_jac(nullptr, n).bytes : 0; }

int jacobi_topk(double* B, int64_t n, int64_t k, float* Wsel, void* ws, size_t ws_bytes, int* dev_status,
                cudaStream_t stream) {
  if (n <= 0 || k <= 0 || k > n || (n & 1)) return PRAC_EINVAL;
  const JacWs j = carve_jac(ws, n);
  if (ws == nullptr || ws_bytes < j.bytes) return PRAC_EWORKSPACE;
  int dev = 0, sms = 0, per_sm = 0;
  PRAC_CUDA_TRY(cudaGetDevice(&dev));
  PRAC_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const int half = static_cast<int>(n / 2);
  const size_t smem = static_cast<size_t>(half) * (2 * sizeof(double) + 2 * sizeof(int));
  PRAC_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, jacobi_kernel, 256, smem));
  if (per_sm < 1) return PRAC_ECUDA;
  long long want = (static_cast<long long>(half) * half + 255) / 256;
  if (want < 1) want = 1;
  const int grid = static_cast<int>(want < sms ? want : sms);
  int ni = static_cast<int>(n), max_sweeps = 30;
  double tol = 1e-11;
  double* b0 = B;
  double* b1 = j.B1;
  double* w = j.W;
  JacobiInfo* info = j.info;
  void* args[] = {&b0, &b1, &w, &ni, &max_sweeps, &tol, &info, &dev_status};
  PRAC_CUDA_TRY(cudaLaunchCooperativeKernel(reinterpret_cast<void*>(jacobi_kernel), dim3(grid), dim3(256), args,
                                            smem, stream));
    count_launch();
  select_topk_kernel<<<static_cast<unsigned>(n), 128, 0, stream>>>(b0, b1, w, ni, static_cast<int>(k), info, Wsel);
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

int launch_symmetrize(double* B, int64_t n, cudaStream_t stream) {
  if (n <= 0) return PRAC_OK;
  symmetrize_kernel<<<nblocks(n * n, 256), 256, 0, stream>>>(B, static_cast<int>(n));
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

int launch_make_bf16_copies(const float* P, int64_t ldp, int64_t d, int64_t s, __nv_bfloat16* Pb, int64_t ldpb,
                            __nv_bfloat16* PTb, int64_t ldptb, cudaStream_t stream) {
  dim3 grid(static_cast<unsigned>((s + 31) / 32), static_cast<unsigned>((d + 31) / 32));
  make_bf16_copies_kernel<<<grid, 256, 0, stream>>>(P, ldp, d, s, Pb, ldpb, PTb, ldptb);
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

int launch_split3(const float* src, int64_t lds, int64_t rows, int64_t cols, __nv_bfloat16* dst,
                  int64_t rows_pad, int64_t ldd, cudaStream_t stream) {
  if (rows <= 0 || cols <= 0) return PRAC_OK;
  split3_kernel<<<nblocks(rows_pad * ldd, 256), 256, 0, stream>>>(src, lds, rows, cols, dst, rows_pad, ldd);
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
