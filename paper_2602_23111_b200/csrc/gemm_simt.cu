// General FMA GEMM: any leading dimensions and alignments, fp32 / bf16 / fp64 elements,
// fp32 or fp64 accumulation.  It serves the fp32 storage path, the small dense products
// of the basis fit (subspace iteration, projections, Cholesky updates) and any operand
// layout the TMA-fed tensor-core kernels cannot take.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "internal.h"

namespace prac {
namespace {

constexpr int TM = 64, TN = 64, TK = 16, THREADS = 256;

template <typename TAcc>
__device__ __forceinline__ TAcc load_elem(const void* base, int type, long long idx) {
  if (type == ET_F32) return static_cast<TAcc>(static_cast<const float*>(base)[idx]);
  if (type == ET_BF16) return static_cast<TAcc>(__bfloat162float(static_cast<const __nv_bfloat16*>(base)[idx]));
  return static_cast<TAcc>(static_cast<const double*>(base)[idx]);
}
template <typename TAcc>
__device__ __forceinline__ void store_elem(void* base, int type, long long idx, TAcc v) {
  if (type == ET_F32) static_cast<float*>(base)[idx] = static_cast<float>(v);
  else if (type == ET_BF16) static_cast<__nv_bfloat16*>(base)[idx] = __float2bfloat16_rn(static_cast<float>(v));
  else static_cast<double*>(base)[idx] = static_cast<double>(v);
}

struct DevGemm {
  int M, N, K;
  const void* A; long long lda; int type_a;
  const void* B; long long ldb; int type_b;
  void* C; long long ldc; int type_c;
  double alpha, beta;
  int kscale_from; double kscale;
  const int* run_if; int run_if_mask;   // optional: do nothing unless *run_if & run_if_mask
  long long ext_a, ext_b, ext_c;        // elements the three buffers span (used by the bounds-checking build)
};

template <typename TAcc, bool TRANS_A, bool TRANS_B>
__global__ void __launch_bounds__(THREADS) gemm_simt_kernel(const DevGemm g) {
  __shared__ TAcc As[TK][TM + 4];
  __shared__ TAcc Bs[TK][TN + 4];
  if (g.run_if != nullptr && (*reinterpret_cast<const volatile int*>(g.run_if) & g.run_if_mask) == 0) return;
  const int t = threadIdx.x;
  const int tx = t & 15, ty = t >> 4;
  const int m0 = blockIdx.y * TM, n0 = blockIdx.x * TN;
  TAcc acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = TAcc(0);

  for (int k0 = 0; k0 < g.K; k0 += TK) {
    // ---- A tile -> As[k][m]
    if (!TRANS_A) {
      const int i = t >> 2, kq = (t & 3) * 4;
      const int gi = m0 + i;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int gk = k0 + kq + e;
        TAcc v = TAcc(0);
        if (gi < g.M && gk < g.K && PRAC_IN(static_cast<long long>(gi) * g.lda + gk, g.ext_a)) {
          v = load_elem<TAcc>(g.A, g.type_a, static_cast<long long>(gi) * g.lda + gk);
          if (gk >= g.kscale_from) v *= static_cast<TAcc>(g.kscale);
        }
        As[kq + e][i] = v;
      }
    } else {
      const int kk = t >> 4, iq = (t & 15) * 4;
      const int gk = k0 + kk;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int gi = m0 + iq + e;
        TAcc v = TAcc(0);
        if (gi < g.M && gk < g.K && PRAC_IN(static_cast<long long>(gk) * g.lda + gi, g.ext_a)) {
          v = load_elem<TAcc>(g.A, g.type_a, static_cast<long long>(gk) * g.lda + gi);
          if (gk >= g.kscale_from) v *= static_cast<TAcc>(g.kscale);
        }
        As[kk][iq + e] = v;
      }
    }
    // ---- B tile -> Bs[k][n]
    if (!TRANS_B) {
      const int kk = t >> 4, jq = (t & 15) * 4;
      const int gk = k0 + kk;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int gj = n0 + jq + e;
        TAcc v = TAcc(0);
        if (gj < g.N && gk < g.K && PRAC_IN(static_cast<long long>(gk) * g.ldb + gj, g.ext_b))
          v = load_elem<TAcc>(g.B, g.type_b, static_cast<long long>(gk) * g.ldb + gj);
        Bs[kk][jq + e] = v;
      }
    } else {
      const int j = t >> 2, kq = (t & 3) * 4;
      const int gj = n0 + j;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int gk = k0 + kq + e;
        TAcc v = TAcc(0);
        if (gj < g.N && gk < g.K && PRAC_IN(static_cast<long long>(gj) * g.ldb + gk, g.ext_b))
          v = load_elem<TAcc>(g.B, g.type_b, static_cast<long long>(gj) * g.ldb + gk);
        Bs[kq + e][j] = v;
      }
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      TAcc a[4], b[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) { a[e] = As[kk][ty * 4 + e]; b[e] = Bs[kk][tx * 4 + e]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] += a[i] * b[j];
    }
    __syncthreads();
  }
  const TAcc alpha = static_cast<TAcc>(g.alpha), beta = static_cast<TAcc>(g.beta);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int gi = m0 + ty * 4 + i;
    if (gi >= g.M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int gj = n0 + tx * 4 + j;
      if (gj >= g.N) continue;
      const long long idx = static_cast<long long>(gi) * g.ldc + gj;
      if (!PRAC_IN(idx, g.ext_c)) continue;
      TAcc v = alpha * acc[i][j];
      if (g.beta != 0.0) v += beta * load_elem<TAcc>(g.C, g.type_c, idx);
      store_elem<TAcc>(g.C, g.type_c, idx, v);
    }
  }
}

template <typename TAcc>
void dispatch(const DevGemm& d, int ta, int tb, dim3 grid, cudaStream_t s) {
  count_launch();
  if (!ta && !tb) gemm_simt_kernel<TAcc, false, false><<<grid, THREADS, 0, s>>>(d);
  else if (!ta && tb) gemm_simt_kernel<TAcc, false, true><<<grid, THREADS, 0, s>>>(d);
  else if (ta && !tb) gemm_simt_kernel<TAcc, true, false><<<grid, THREADS, 0, s>>>(d);
  else gemm_simt_kernel<TAcc, true, true><<<grid, THREADS, 0, s>>>(d);
}

}  // namespace

PRAC_BOUNDS_READER(bounds_violations_simt)

int gemm_general(const GemmArgs& g, cudaStream_t stream) {
  if (g.M < 0 || g.N < 0 || g.K < 0) return PRAC_EINVAL;
  if (g.M == 0 || g.N == 0) return PRAC_OK;
  if (g.M > 0x7fffffff || g.N > 0x7fffffff || g.K > 0x7fffffff) return PRAC_EINVAL;
  DevGemm d;
  d.M = static_cast<int>(g.M); d.N = static_cast<int>(g.N); d.K = static_cast<int>(g.K);
  d.A = g.A; d.lda = g.lda; d.type_a = g.type_a;
  d.B = g.B; d.ldb = g.ldb; d.type_b = g.type_b;
  d.C = g.C; d.ldc = g.ldc; d.type_c = g.type_c;
  d.alpha = g.alpha; d.beta = g.beta;
  d.kscale_from = (g.kscale_from < 0 || g.kscale_from > g.K) ? d.K : static_cast<int>(g.kscale_from);
  d.kscale = g.kscale;
  d.run_if = g.run_if; d.run_if_mask = g.run_if_mask;
  // what a row-major buffer of these dimensions spans: (rows - 1) * ld + cols elements
  d.ext_a = g.trans_a ? (g.K - 1) * g.lda + g.M : (g.M - 1) * g.lda + g.K;
  d.ext_b = g.trans_b ? (g.N - 1) * g.ldb + g.K : (g.K - 1) * g.ldb + g.N;
  d.ext_c = (g.M - 1) * g.ldc + g.N;
  const long long gy = (g.M + TM - 1) / TM, gx = (g.N + TN - 1) / TN;
  if (gy > 65535) return PRAC_EINVAL;
  dim3 grid(static_cast<unsigned>(gx), static_cast<unsigned>(gy));
  if (g.acc_double) dispatch<double>(d, g.trans_a, g.trans_b, grid, stream);
  else dispatch<float>(d, g.trans_a, g.trans_b, grid, stream);
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

}  // namespace prac
