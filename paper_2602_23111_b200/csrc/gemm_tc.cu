// Tensor-core GEMMs for sm_100a: TMA-fed shared-memory pipelines, tcgen05.mma with fp32
// accumulators in tensor memory, warp-specialised persistent CTAs.
//
//   kernel<BN, MN_MAJOR=false>  C[M x N] = A[M x K] * B[N x K]^T     (compress, dW stage 2)
//   kernel<BN, MN_MAJOR=true >  C[M x N] = A[K x M]^T * B[K x N]     (dY^T Z, X^T X), split
//                               over K with fp32 partial tiles and an ordered reduction.
//
// One CTA = 6 warps: warp 0 issues TMA loads, warp 1 owns tensor memory and issues the
// MMAs, warps 2..5 drain accumulators (each warp reads the 32 TMEM lanes it may access).
// Two accumulator buffers let the epilogue of one tile overlap the MMAs of the next.
// Every mbarrier wait is bounded; a wait that gives up raises a status bit and the CTA
// leaves through the common exit that frees its tensor memory.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <mutex>

#include "internal.h"
#include "ptx.cuh"

namespace prac {
namespace {

constexpr int BM = 128;     // tile rows = TMEM lanes
constexpr int BK = 64;      // bf16 elements per pipeline stage along K (= one 128-byte swizzle row)
constexpr int UMMA_K = 16;  // K of one tcgen05.mma for 16-bit inputs
constexpr int NUM_THREADS = 192;
constexpr uint32_t WAIT_LIMIT = 1u << 22;

enum Epilogue : int { EPI_BF16 = 0, EPI_F32 = 1, EPI_PARTIAL = 2 };

template <int BN>
struct Cfg {
  static constexpr int A_BYTES = BM * BK * 2;
  static constexpr int B_BYTES = BN * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = (BN == 256) ? 4 : ((BN == 128) ? 6 : 8);
  static constexpr int TMEM_COLS = 2 * BN;  // two accumulator buffers; 128, 256 or 512
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*align*/ + 256 /*barriers*/;
};

struct TcParams {
  int M, N, K;
  int n_tiles;        // tiles along N
  int num_tiles;      // tiles to compute (all, or those touching the upper triangle)
  int splits;         // K splits (1 for the K-major kernel)
  int kblocks;        // ceil(K / BK)
  int symmetric;
  void* C;            // direct output (EPI_BF16 / EPI_F32)
  long long ldc;
  int accumulate;
  float* partial;     // EPI_PARTIAL: [splits][M_pad][N_pad]
  long long partial_ld;
  long long partial_split_stride;
  int* dev_status;
};

struct SmemCtl {
  uint64_t full[8];
  uint64_t empty[8];
  uint64_t acc_full[2];
  uint64_t acc_empty[2];
  uint32_t tmem_base;
  int abort_flag;
};

template <int BN>
__device__ __forceinline__ void tile_coords(const TcParams& p, int tile, int& mt, int& nt) {
  if (!p.symmetric) {
    mt = tile / p.n_tiles;
    nt = tile % p.n_tiles;
    return;
  }
  // Row-tile mt keeps the column tiles nt >= (mt * BM) / BN (those reaching the diagonal).
  int row = 0, rest = tile;
  while (true) {
    const int first = (row * BM) / BN;
    const int cnt = p.n_tiles - first;
    if (rest < cnt) { mt = row; nt = first + rest; return; }
    rest -= cnt;
    ++row;
  }
}

template <int BN, bool MN_MAJOR, int EPI>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
               const TcParams p) {
  using C = Cfg<BN>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  SmemCtl* ctl = reinterpret_cast<SmemCtl*>(smem + C::STAGES * C::STAGE_BYTES);
  volatile int* abort_flag = &ctl->abort_flag;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int total_items = p.num_tiles * p.splits;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) {
      ptx::mbar_init(&ctl->full[s], 1);
      ptx::mbar_init(&ctl->empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(&ctl->acc_full[b], 1);
      ptx::mbar_init(&ctl->acc_empty[b], 4);
    }
    ctl->abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::fence_proxy_async();
  }
  if (warp == 1) {
    ptx::tmem_alloc(&ctl->tmem_base, C::TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = ctl->tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (ptx::elect_one()) {
      ptx::prefetch_tensormap(&tmap_a);
      ptx::prefetch_tensormap(&tmap_b);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
        const int split = item / p.num_tiles;
        int mt, nt;
        tile_coords<BN>(p, item % p.num_tiles, mt, nt);
        const int kb0 = static_cast<int>(static_cast<long long>(split) * p.kblocks / p.splits);
        const int kb1 = static_cast<int>(static_cast<long long>(split + 1) * p.kblocks / p.splits);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!ptx::mbar_wait(&ctl->empty[stage], phase ^ 1u, abort_flag, WAIT_LIMIT)) { ok = false; break; }
          uint8_t* sa = smem + stage * C::STAGE_BYTES;
          uint8_t* sb = sa + C::A_BYTES;
          ptx::mbar_arrive_expect_tx(&ctl->full[stage], C::STAGE_BYTES);
          if (!MN_MAJOR) {
            ptx::tma_load_2d(sa, &tmap_a, &ctl->full[stage], kb * BK, mt * BM);
            ptx::tma_load_2d(sb, &tmap_b, &ctl->full[stage], kb * BK, nt * BN);
          } else {
#pragma unroll
            for (int j = 0; j < BM / 64; ++j)
              ptx::tma_load_2d(sa + j * (BK * 128), &tmap_a, &ctl->full[stage], mt * BM + 64 * j, kb * BK);
#pragma unroll
            for (int j = 0; j < BN / 64; ++j)
              ptx::tma_load_2d(sb + j * (BK * 128), &tmap_b, &ctl->full[stage], nt * BN + 64 * j, kb * BK);
          }
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (ptx::elect_one()) {
      constexpr uint32_t idesc = ptx::idesc_bf16_f32(BM, BN, MN_MAJOR, MN_MAJOR);
      int stage = 0;
      uint32_t phase = 0;
      int acc_iter = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x, ++acc_iter) {
        const int split = item / p.num_tiles;
        const int kb0 = static_cast<int>(static_cast<long long>(split) * p.kblocks / p.splits);
        const int kb1 = static_cast<int>(static_cast<long long>(split + 1) * p.kblocks / p.splits);
        const int buf = acc_iter & 1;
        const uint32_t acc_phase = (acc_iter >> 1) & 1;
        if (!ptx::mbar_wait(&ctl->acc_empty[buf], acc_phase ^ 1u, abort_flag, WAIT_LIMIT)) { ok = false; break; }
        ptx::tc_fence_after_sync();
        const uint32_t tmem_d = tmem_base + static_cast<uint32_t>(buf * BN);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!ptx::mbar_wait(&ctl->full[stage], phase, abort_flag, WAIT_LIMIT)) { ok = false; break; }
          ptx::tc_fence_after_sync();
          const uint32_t sa = ptx::smem_u32(smem + stage * C::STAGE_BYTES);
          const uint32_t sb = sa + C::A_BYTES;
#pragma unroll
          for (int kk = 0; kk < BK / UMMA_K; ++kk) {
            uint64_t da, db;
            if (!MN_MAJOR) {
              // 16 K-elements = 32 bytes further inside each 128-byte row
              da = ptx::smem_desc_sw128(sa + kk * (UMMA_K * 2), 16, 1024);
              db = ptx::smem_desc_sw128(sb + kk * (UMMA_K * 2), 16, 1024);
            } else {
              // 16 K-rows of 128 bytes further; 64-column blocks are BK*128 bytes apart
              da = ptx::smem_desc_sw128(sa + kk * (UMMA_K * 128), BK * 128, 1024);
              db = ptx::smem_desc_sw128(sb + kk * (UMMA_K * 128), BK * 128, 1024);
            }
            ptx::umma_bf16(tmem_d, da, db, idesc, (kb > kb0 || kk > 0) ? 1u : 0u);
          }
          ptx::umma_commit(&ctl->empty[stage]);  // frees the stage when these MMAs retire
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) ptx::umma_commit(&ctl->acc_full[buf]);
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    const int quarter = warp & 3;  // TMEM lanes [32*quarter, 32*quarter + 32)
    int acc_iter = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x, ++acc_iter) {
      const int split = item / p.num_tiles;
      int mt, nt;
      tile_coords<BN>(p, item % p.num_tiles, mt, nt);
      const int buf = acc_iter & 1;
      const uint32_t acc_phase = (acc_iter >> 1) & 1;
      if (!ptx::mbar_wait(&ctl->acc_full[buf], acc_phase, abort_flag, WAIT_LIMIT)) { ok = false; break; }
      ptx::tc_fence_after_sync();
      const int row = mt * BM + quarter * 32 + lane;
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                             static_cast<uint32_t>(buf * BN);
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t v[32];
        ptx::tmem_ld_32x32(taddr + c * 32, v);
        ptx::tmem_ld_wait();
        const int col0 = nt * BN + c * 32;
        if (EPI == EPI_PARTIAL) {
          float* dst = p.partial + split * p.partial_split_stride +
                       static_cast<long long>(row) * p.partial_ld + col0;
#pragma unroll
          for (int j = 0; j < 8; ++j)
            reinterpret_cast<uint4*>(dst)[j] = make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
        } else if (EPI == EPI_BF16) {
          if (row < p.M && col0 < p.N) {
            __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.C) +
                                 static_cast<long long>(row) * p.ldc + col0;
            const bool vec = (col0 + 32 <= p.N) && ((reinterpret_cast<uintptr_t>(dst) & 15u) == 0);
            if (vec) {
              uint32_t w[16];
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]));
                w[j] = *reinterpret_cast<uint32_t*>(&h);
              }
#pragma unroll
              for (int j = 0; j < 4; ++j)
                reinterpret_cast<uint4*>(dst)[j] = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (col0 + j < p.N) dst[j] = __float2bfloat16_rn(__uint_as_float(v[j]));
            }
          }
        } else {  // EPI_F32
          if (row < p.M && col0 < p.N) {
            float* dst = reinterpret_cast<float*>(p.C) + static_cast<long long>(row) * p.ldc + col0;
            const bool vec = (col0 + 32 <= p.N) && ((reinterpret_cast<uintptr_t>(dst) & 15u) == 0);
            if (vec) {
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                float4 o = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                       __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
                if (p.accumulate) {
                  const float4 old = reinterpret_cast<float4*>(dst)[j];
                  o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
                }
                reinterpret_cast<float4*>(dst)[j] = o;
              }
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (col0 + j < p.N) {
                  const float o = __uint_as_float(v[j]);
                  dst[j] = p.accumulate ? dst[j] + o : o;
                }
            }
          }
        }
      }
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&ctl->acc_empty[buf]);
    }
  }

  // ---------------------------------------------------------------- common exit
  __syncwarp();
  if (*abort_flag) {
    // Some wait gave up: report it, give copies still in flight time to land, then leave.
    if (lane == 0 && p.dev_status) atomicOr(p.dev_status, DEV_WAIT_EXPIRED);
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
}

// Ordered reduction of the K-split partial tiles: out[i][j] = scale_j * sum_s partial[s][i][j].
template <typename TOut>
__global__ void splitk_reduce_kernel(const float* __restrict__ partial, long long pld,
                                     long long pstride, int splits, int M, int N, TOut* out,
                                     long long ldo, int scale_from, float scale, int symmetric) {
  const long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
  const int ncol4 = (N + 3) / 4;
  if (idx >= static_cast<long long>(M) * ncol4) return;
  const int i = static_cast<int>(idx / ncol4);
  const int j0 = static_cast<int>(idx % ncol4) * 4;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  if (!symmetric || i <= j0) {
    const float* src = partial + static_cast<long long>(i) * pld + j0;
    for (int s = 0; s < splits; ++s) {
      const float4 t = *reinterpret_cast<const float4*>(src + s * pstride);
      acc[0] += t.x; acc[1] += t.y; acc[2] += t.z; acc[3] += t.w;
    }
  } else {
    for (int e = 0; e < 4; ++e) {
      const int j = j0 + e;
      if (j >= N) break;
      const float* src = (i <= j) ? partial + static_cast<long long>(i) * pld + j
                                  : partial + static_cast<long long>(j) * pld + i;
      float a = 0.f;
      for (int s = 0; s < splits; ++s) a += src[s * pstride];
      acc[e] = a;
    }
  }
  for (int e = 0; e < 4; ++e) {
    const int j = j0 + e;
    if (j >= N) break;
    const float v = (j >= scale_from) ? acc[e] * scale : acc[e];
    if constexpr (sizeof(TOut) == 2) out[static_cast<long long>(i) * ldo + j] = __float2bfloat16_rn(v);
    else out[static_cast<long long>(i) * ldo + j] = v;
  }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;
int g_num_sms = 0;
std::once_flag g_once;
int g_init_status = PRAC_ECUDA;

void do_init() {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || fn == nullptr) {
    return;
  }
  g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return;
  if (cudaDeviceGetAttribute(&g_num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return;
  g_init_status = PRAC_OK;
}

// bf16 matrix with `rows` rows of `inner` elements (leading dimension ld), box = 64 x box_rows.
int make_map(CUtensorMap* map, const void* base, int64_t inner, int64_t rows, int64_t ld, int box_rows) {
  cuuint64_t gdim[2] = {static_cast<cuuint64_t>(inner), static_cast<cuuint64_t>(rows)};
  cuuint64_t gstr[1] = {static_cast<cuuint64_t>(ld) * 2};
  cuuint32_t box[2] = {64u, static_cast<cuuint32_t>(box_rows)};
  cuuint32_t estr[2] = {1u, 1u};
  CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstr,
                        box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? PRAC_OK : PRAC_ECUDA;
}

template <int BN, bool MN, int EPI>
int launch(const CUtensorMap& ta, const CUtensorMap& tb, const TcParams& p, cudaStream_t stream) {
  using C = Cfg<BN>;
  auto kern = gemm_tc_kernel<BN, MN, EPI>;
  static bool attr_set = false;  // per instantiation
  if (!attr_set) {
    PRAC_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
    attr_set = true;
  }
  const int items = p.num_tiles * p.splits;
  const int grid = items < g_num_sms ? items : g_num_sms;
  kern<<<grid, NUM_THREADS, C::SMEM_BYTES, stream>>>(ta, tb, p);
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

int pick_bn(int64_t N) { return N > 128 ? 256 : (N > 64 ? 128 : 64); }

int count_tiles(int m_tiles, int n_tiles, int bn, int symmetric) {
  if (!symmetric) return m_tiles * n_tiles;
  int cnt = 0;
  for (int mt = 0; mt < m_tiles; ++mt) {
    const int first = (mt * BM) / bn;
    if (first < n_tiles) cnt += n_tiles - first;
  }
  return cnt;
}

int pick_splits(int num_tiles, int kblocks) {
  int s = g_num_sms / (num_tiles > 0 ? num_tiles : 1);
  if (s < 1) s = 1;
  const int max_by_k = kblocks / 4 > 0 ? kblocks / 4 : 1;  // at least 4 k-blocks per split
  if (s > max_by_k) s = max_by_k;
  return s;
}

}  // namespace

int tc_init() {
  std::call_once(g_once, do_init);
  return g_init_status;
}
int tc_num_sms() { return g_num_sms; }

int tc_gemm_kmajor(const __nv_bfloat16* A, int64_t lda, const __nv_bfloat16* B, int64_t ldb,
                   int64_t M, int64_t N, int64_t K, void* Cout, int64_t ldc, int type_c,
                   int accumulate, int* dev_status, cudaStream_t stream) {
  if (tc_init() != PRAC_OK) return PRAC_ECUDA;
  if (M <= 0 || N <= 0 || K <= 0) return PRAC_EINVAL;
  if (!aligned16(A) || !aligned16(B) || (lda % 8) || (ldb % 8)) return PRAC_EALIGN;
  if (type_c != ET_BF16 && type_c != ET_F32) return PRAC_EINVAL;
  const int bn = pick_bn(N);
  CUtensorMap ta, tb;
  if (make_map(&ta, A, K, M, lda, BM) != PRAC_OK) return PRAC_ECUDA;
  if (make_map(&tb, B, K, N, ldb, bn) != PRAC_OK) return PRAC_ECUDA;
  TcParams p{};
  p.M = static_cast<int>(M); p.N = static_cast<int>(N); p.K = static_cast<int>(K);
  const int m_tiles = static_cast<int>((M + BM - 1) / BM);
  p.n_tiles = static_cast<int>((N + bn - 1) / bn);
  p.num_tiles = m_tiles * p.n_tiles;
  p.splits = 1;
  p.kblocks = static_cast<int>((K + BK - 1) / BK);
  p.symmetric = 0;
  p.C = Cout; p.ldc = ldc; p.accumulate = accumulate;
  p.dev_status = dev_status;
  if (type_c == ET_BF16) {
    if (accumulate) return PRAC_EINVAL;
    if (bn == 256) return launch<256, false, EPI_BF16>(ta, tb, p, stream);
    if (bn == 128) return launch<128, false, EPI_BF16>(ta, tb, p, stream);
    return launch<64, false, EPI_BF16>(ta, tb, p, stream);
  }
  if (bn == 256) return launch<256, false, EPI_F32>(ta, tb, p, stream);
  if (bn == 128) return launch<128, false, EPI_F32>(ta, tb, p, stream);
  return launch<64, false, EPI_F32>(ta, tb, p, stream);
}

namespace {
struct TokensPlan {
  int bn, m_tiles, n_tiles, num_tiles, kblocks, splits;
  int64_t m_pad, n_pad;
};
TokensPlan plan_tokens(int64_t M, int64_t N, int64_t K, int symmetric) {
  TokensPlan t;
  t.bn = pick_bn(N);
  t.m_tiles = static_cast<int>((M + BM - 1) / BM);
  t.n_tiles = static_cast<int>((N + t.bn - 1) / t.bn);
  t.num_tiles = count_tiles(t.m_tiles, t.n_tiles, t.bn, symmetric);
  t.kblocks = static_cast<int>((K + BK - 1) / BK);
  t.splits = pick_splits(t.num_tiles, t.kblocks);
  t.m_pad = static_cast<int64_t>(t.m_tiles) * BM;
  t.n_pad = static_cast<int64_t>(t.n_tiles) * t.bn;
  return t;
}
}  // namespace

size_t tc_gemm_tokens_ws_bytes(int64_t M, int64_t N, int64_t K, int symmetric) {
  if (tc_init() != PRAC_OK) {
    // No device yet: size for the worst case the planner can choose (148 CTAs' worth of splits).
    const int bn = pick_bn(N);
    const int64_t m_pad = round_up(M, BM), n_pad = round_up(N, bn);
    const int64_t tiles = (m_pad / BM) * (n_pad / bn);
    int64_t splits = 148 / (tiles > 0 ? tiles : 1);
    if (splits < 1) splits = 1;
    return static_cast<size_t>(splits * m_pad * n_pad) * sizeof(float);
  }
  const TokensPlan t = plan_tokens(M, N, K, symmetric);
  return static_cast<size_t>(t.splits) * t.m_pad * t.n_pad * sizeof(float);
}

int tc_gemm_tokens(const __nv_bfloat16* A, int64_t lda, const __nv_bfloat16* B, int64_t ldb,
                   int64_t M, int64_t N, int64_t K, void* Cout, int64_t ldc, int type_c,
                   int64_t scale_from, float scale, int symmetric,
                   void* ws, size_t ws_bytes, int* dev_status, cudaStream_t stream) {
  if (tc_init() != PRAC_OK) return PRAC_ECUDA;
  if (M <= 0 || N <= 0 || K <= 0) return PRAC_EINVAL;
  if (!aligned16(A) || !aligned16(B) || (lda % 8) || (ldb % 8)) return PRAC_EALIGN;
  if (type_c != ET_BF16 && type_c != ET_F32) return PRAC_EINVAL;
  if (symmetric && (A != B || M != N)) return PRAC_EINVAL;
  const TokensPlan t = plan_tokens(M, N, K, symmetric);
  const size_t need = static_cast<size_t>(t.splits) * t.m_pad * t.n_pad * sizeof(float);
  if (ws == nullptr || ws_bytes < need) return PRAC_EWORKSPACE;
  CUtensorMap ta, tb;
  if (make_map(&ta, A, M, K, lda, BK) != PRAC_OK) return PRAC_ECUDA;
  if (make_map(&tb, B, N, K, ldb, BK) != PRAC_OK) return PRAC_ECUDA;
  TcParams p{};
  p.M = static_cast<int>(M); p.N = static_cast<int>(N); p.K = static_cast<int>(K);
  p.n_tiles = t.n_tiles;
  p.num_tiles = t.num_tiles;
  p.splits = t.splits;
  p.kblocks = t.kblocks;
  p.symmetric = symmetric;
  p.partial = static_cast<float*>(ws);
  p.partial_ld = t.n_pad;
  p.partial_split_stride = t.m_pad * t.n_pad;
  p.dev_status = dev_status;
  int st;
  if (t.bn == 256) st = launch<256, true, EPI_PARTIAL>(ta, tb, p, stream);
  else if (t.bn == 128) st = launch<128, true, EPI_PARTIAL>(ta, tb, p, stream);
  else st = launch<64, true, EPI_PARTIAL>(ta, tb, p, stream);
  if (st != PRAC_OK) return st;
  const long long work = static_cast<long long>(M) * ((N + 3) / 4);
  const int threads = 256;
  const unsigned blocks = static_cast<unsigned>((work + threads - 1) / threads);
  const int sf = scale_from < 0 || scale_from > N ? static_cast<int>(N) : static_cast<int>(scale_from);
  if (type_c == ET_BF16)
    splitk_reduce_kernel<__nv_bfloat16><<<blocks, threads, 0, stream>>>(
        p.partial, p.partial_ld, p.partial_split_stride, p.splits, p.M, p.N,
        static_cast<__nv_bfloat16*>(Cout), ldc, sf, scale, symmetric);
  else
    splitk_reduce_kernel<float><<<blocks, threads, 0, stream>>>(
        p.partial, p.partial_ld, p.partial_split_stride, p.splits, p.M, p.N,
        static_cast<float*>(Cout), ldc, sf, scale, symmetric);
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

}  // namespace prac
