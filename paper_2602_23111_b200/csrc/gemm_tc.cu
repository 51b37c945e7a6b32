// Tensor-core GEMMs for sm_100a: TMA-fed shared-memory pipelines, tcgen05.mma with fp32
// accumulators in tensor memory, warp-specialised persistent CTAs.
//
//   kernel<CTAS, BN, MN_MAJOR=false>  C[M x N] = A[M x K] * B[N x K]^T   (compress, dW stage 2)
//   kernel<CTAS, BN, MN_MAJOR=true >  C[M x N] = A[K x M]^T * B[K x N]   (dY^T Z, X^T X), split
//                                     over K with fp32 partial tiles and an ordered reduction.
//
// CTAS = 2 is the main path: the two CTAs of a cluster share one 256 x 256 output tile.  Each
// loads its own 128 rows of A and its own half of B, the leader CTA issues
// tcgen05.mma.cta_group::2 (M = 256) over both, and each CTA drains its own 128 accumulator
// rows.  Per k-block a CTA moves 32 KB for 2 x 128 x 256 x 64 flop, which keeps the
// L2-to-shared-memory traffic at half of what 128 x 256 single-CTA tiles need and leaves room
// for a 6- or 7-stage ring.  CTAS = 1 (128 x BN tiles, BN in {64, 128, 256}) serves narrow outputs.
// BN = 512 (CTA pairs, K-major, bf16 out) is the compress of a long input into 257..512 columns:
// one 256 x 512 tile per 256 rows, two MMAs of N = 256 per k-step on one A stage, a single
// accumulator that fills tensor memory and is handed back to the MMA warp in two halves.
//
// One CTA = 10 warps: warp 0 issues TMA loads, warp 1 owns tensor memory and issues the
// MMAs, warps 2..9 drain accumulators (a warp reaches the 32 TMEM lanes 32 (warp % 4)..., so two
// warps share each quarter of the rows and take alternate column blocks).  Two accumulator
// buffers let the epilogue of one tile overlap the MMAs of the next.  Epilogues: bf16 / fp32
// output (TMA tile stores), fp32 partial tiles, and fused consumers of the product that never
// store it (activation derivative times a factor; the two passes of the RMSNorm backward), whose
// element-wise factor arrives by TMA tile loads into the buffers the results then leave from.
// Operands whose rows are off the 16-byte grid (a contiguous bf16 matrix of odd width) go through
// TMA as classes of rows that share one offset from that grid (ClassMaps; the *_rowclass_kernel
// entry points), or, where the base pointer itself is off the grid, through loader warps with
// plain loads (A_LDG).
// Every mbarrier wait is bounded; a wait that gives up raises a status bit and the CTA
// leaves through the common exit that frees its tensor memory.  No load is multicast.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <mutex>

#include "act.cuh"
#include "internal.h"
#include "per_device.h"
#include "ptx.cuh"

namespace prac {
namespace {

constexpr int BM = 128;     // rows per CTA = TMEM lanes
constexpr int BK = 64;      // bf16 elements per pipeline stage along K (= one 128-byte swizzle row)
constexpr int UMMA_K = 16;  // K of one tcgen05.mma for 16-bit inputs
constexpr int EPI_WARPS = 8;                             // two per quarter of the accumulator's rows
constexpr int NUM_THREADS = 32 * (2 + EPI_WARPS);
// A operand whose rows are not 16-byte aligned (a contiguous bf16 matrix of odd width, e.g. 5461)
// cannot be fetched by TMA.  Such launches carry LOADER_WARPS more warps that fill A's half of
// every pipeline stage with 32-bit loads, re-aligned in registers, while B still arrives by TMA.
// The loader warps work in LOADER_GROUPS groups of LOADER_WARPS: group g fills the stages of the
// k-blocks g, g + LOADER_GROUPS, ... of the CTA's sequence, so that many k-blocks' loads are in
// flight at once, each thread holding only its 32 words of one of them.
constexpr int LOADER_WARPS = 4;         // warps that share one stage: 32 row segments each
constexpr int LOADER_GROUPS = 3;
constexpr int NUM_THREADS_LDG = NUM_THREADS + 32 * LOADER_WARPS * LOADER_GROUPS;
constexpr uint32_t WAIT_LIMIT = 1u << 22;
constexpr int MAX_STAGES = 8;
constexpr int MAX_SEG = TC_MAX_SEGMENTS;
constexpr int SMEM_LIMIT = 227 * 1024;

// EPI_SILU / EPI_GELU: bf16 output = aux (bf16, same shape as the output) * f'(accumulator)
// EPI_RMS1 / EPI_RMS2: the two passes of the RMSNorm backward over the rebuilt input (no matrix
// output in the first: row and column sums only)
enum Epilogue : int { EPI_BF16 = 0, EPI_F32 = 1, EPI_PARTIAL = 2, EPI_SILU = 3, EPI_GELU = 4, EPI_RMS1 = 5, EPI_RMS2 = 6 };
static_assert(EPI_PARTIAL == 2 && EPI_SILU == 3 && EPI_GELU == 4 && EPI_RMS1 == 5 && EPI_RMS2 == 6, "Cfg spells these out");

constexpr int STORE_BUF_BYTES = 32 * 128;               // 32 rows of 128 bytes
// A 32 x 32 transpose tile of 32-bit words lives in one such buffer: word j of row l sits at
// l * 32 + (j ^ l), so that a warp writing rows and a warp reading columns both touch 32 banks.
constexpr int XPOSE_BYTES = 32 * 32 * 4;
static_assert(XPOSE_BYTES == STORE_BUF_BYTES, "a transpose tile takes the place of one staging buffer");
#ifndef PRAC_AUX_BUFS
#define PRAC_AUX_BUFS 3          // staging buffers per epilogue warp where factors come in and results leave
#endif
#ifndef PRAC_AUX_BUFS_NOSTORE
#define PRAC_AUX_BUFS_NOSTORE 2  // the same where nothing is stored (pass 1 of the norm backward)
#endif
constexpr int MAX_AUX_BUFS = PRAC_AUX_BUFS > PRAC_AUX_BUFS_NOSTORE ? PRAC_AUX_BUFS : PRAC_AUX_BUFS_NOSTORE;
static_assert(PRAC_AUX_BUFS >= 3 && PRAC_AUX_BUFS_NOSTORE >= 2, "one block must be on its way while one is worked on");
constexpr int CTL_BYTES = 512;                          // the barriers and flags behind the staging area

template <int CTAS, int BN, int EPI>
struct Cfg {
  static constexpr int TILE_M = CTAS * BM;           // output rows per tile (per cluster)
  static constexpr int NB_LOCAL = BN / CTAS;         // rows of B this CTA loads
  static constexpr int A_BYTES = BM * BK * 2;
  static constexpr int B_BYTES = NB_LOCAL * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  // Direct epilogues stage 32-row blocks in shared memory, 4 KB buffers owned by one epilogue warp
  // each: a TMA tile store leaves from there (or a transpose tile sits there when the output rows
  // are unaligned).  One buffer per warp (and a sixth pipeline stage) where the main loop sets the
  // pace.  The activation and RMSNorm epilogues also receive their element-wise factor in these
  // buffers, by TMA tile loads that run ahead of the block being worked on; the result overwrites
  // the factor and leaves from the same buffer.  Three buffers when results are stored (one being
  // loaded, one worked on, one being read by its store), two when nothing is stored (pass 1).
  static constexpr bool ACT = (EPI == 3 || EPI == 4 || EPI == 5 || EPI == 6);
  static constexpr int AUX_BUFS = (EPI == 5) ? PRAC_AUX_BUFS_NOSTORE : (ACT ? PRAC_AUX_BUFS : 0);
  static constexpr int STORE_BUFS = ACT ? AUX_BUFS : 1;
  static constexpr int STORE_BYTES = EPI_WARPS * STORE_BUFS * STORE_BUF_BYTES;
  static constexpr int EPI_BYTES = (EPI == 2) ? 0 : STORE_BYTES;
  static constexpr int FIT = (SMEM_LIMIT - 1024 - CTL_BYTES - EPI_BYTES) / STAGE_BYTES;
  static constexpr int STAGES = FIT > MAX_STAGES ? MAX_STAGES : FIT;
  // Two accumulator buffers of BN columns (128, 256 or 512 columns of tensor memory); a 512-wide
  // tile (CTA pairs only: two MMAs of N = 256 per k-step share the A stage, which cuts the bytes
  // fetched per flop by a quarter) fills tensor memory with its single accumulator.
  static constexpr int ACC_BUFS = (BN > 256) ? 1 : 2;
  static constexpr int MMA_N = (BN > 256) ? 256 : BN;
  static constexpr int TMEM_COLS = ACC_BUFS * BN;
  static_assert(BN <= 256 || (BN == 512 && CTAS == 2), "wide tiles: 512 columns on a CTA pair");
  static constexpr int EPI_OFFSET = STAGES * STAGE_BYTES;          // 1024-byte aligned
  static constexpr int CTL_OFFSET = EPI_OFFSET + EPI_BYTES;
  static constexpr int SMEM_BYTES = CTL_OFFSET + CTL_BYTES + 1024 /*align*/;
};

struct TcParams {
  int M, N, K;
  int n_tiles;        // tiles along N
  int num_tiles;      // tiles to compute (all, or those touching the upper triangle)
  int kblocks;        // ceil(K / BK)
  int splits;         // equal pieces each tile's k-blocks are cut into (1 for the K-major kernel)
  int kb_per_seg;     // the K range is a chain of segments of this many k-blocks; segment g reads
  int seg_a[MAX_SEG]; //   A from K offset seg_a[g] and B from K offset seg_b[g] (elements).  One
  int seg_b[MAX_SEG]; //   segment at offset 0 is the ordinary product.
  int symmetric;
  void* C;            // direct output (EPI_BF16 / EPI_F32)
  long long ldc;
  int accumulate;
  int tma_store;      // output rows are 16-byte aligned: tiles leave through TMA stores
  // Two products sharing A in one launch (K-major kernel only): column tiles nt >= n_tiles1
  // belong to a second B operand and a second output, [C | C2] = A [B ; B2]^T.  n_tiles1 ==
  // n_tiles is the ordinary single product.
  int n_tiles1;
  int N2;
  void* C2;
  long long ldc2;
  int tma_store2;
  // EPI_SILU / EPI_GELU: the factor multiplied element-wise into f'(product); rows 16-byte
  // aligned and at least N rounded up to 8 long
  const __nv_bfloat16* aux;
  long long ld_aux;
  // RMSNorm backward (aux = dY, accumulator = rebuilt input x):
  //   pass 1: row_part[(2 nt + half) * M + t] = sum over the warp's columns of col_g[i] dY[t][i] x[t][i]
  //           col_part[(t / 32) * N + i]      = sum over the 32 rows of row_a[t] dY[t][i] x[t][i]
  //   pass 2: out[t][i] = row_a[t] col_g[i] dY[t][i] - row_b[t] x[t][i]
  //   LayerNorm (optional): pass 1 also leaves row_part2 = the same sums of col_g[i] dY[t][i]
  //   (without x), pass 2 adds row_c[t] to every element of row t.
  const float* row_a;
  const float* row_b;
  const float* row_c;
  const float* col_g;
  int col_g_vec;      // col_g is 16-byte aligned: gains are fetched four at a time
  float* row_part;
  float* row_part2;
  float* col_part;
  float* partial;     // EPI_PARTIAL: [split][tile][TILE_M][BN] fp32
  int* dev_status;
  // A fetched with plain loads (A_LDG kernels): the matrix as stored (K-major: a_rows = M rows of
  // a_cols = K elements; token-major: a_rows = K tokens of a_cols = M elements), rows 2-byte aligned
  const __nv_bfloat16* a_ptr;
  long long a_ld;
  int a_rows, a_cols;
  // A by row classes (A_CLS kernels): rows r = P q + j of A form class j; cls_shift[j] = (j lda) mod 8 is
  // how many elements the class's tensor map starts before its rows do; cls_count = P.
  int cls_count;
  int cls_shift[8];
  int cls_sub;        // token-major launches by classes: piece (split) = class * cls_sub + part of its tokens; else 0
};

// K-major A whose row pitch is not a multiple of 16 bytes, fetched by TMA all the same.  With
// P = 8 / gcd(lda, 8) the rows r = P q + j (fixed j) start (j lda) mod 8 elements past a 16-byte
// boundary, all by the same amount, and lie P lda elements apart, which is a multiple of 8: they are
// the rows of a tensor map whose base is that boundary.  Column c of such a map is element
// c - shift of the row, so a tile of one class is the ordinary K-major tile with K running
// `shift` ahead, and the B operand is fetched `shift` rows earlier to match: B is read MN-major
// (K x N row-major), where the K coordinate of a tile load is a row number and needs no
// alignment.  The first `shift` columns of a class hold the end of the row before, the columns
// past K the start of the row after; B reads as zero there (rows outside its extent), so these
// contribute nothing as long as A holds finite numbers.  The output rows of a class are P ldc apart.
// The token-major product A^T B (A: K tokens x M, B: K tokens x N) uses the same classes of rows
// as pieces of K: the tokens of class j give one partial product, whose row i is feature
// i - shift_j (the reduction adds the classes back with that offset); a[j] and c[j] are then the
// class's rows of A and of B.
struct ClassMaps {
  CUtensorMap a[8];
  CUtensorMap c[8];
};

struct SmemCtl {
  uint64_t full[MAX_STAGES];
  uint64_t empty[MAX_STAGES];
  uint64_t acc_full[2];
  uint64_t acc_empty[2];
  uint64_t aux_full[EPI_WARPS][MAX_AUX_BUFS];   // activation epilogues: a warp's factor block has landed
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(SmemCtl) <= CTL_BYTES, "control block");

template <int TILE_M, int BN>
__device__ __forceinline__ void tile_coords(const TcParams& p, int tile, int& mt, int& nt) {
  if (!p.symmetric) {
    mt = tile / p.n_tiles;
    nt = tile % p.n_tiles;
    return;
  }
  // Row-tile mt keeps the column tiles nt >= (mt * TILE_M) / BN (those reaching the diagonal).
  int row = 0, rest = tile;
  while (true) {
    const int first = (row * TILE_M) / BN;
    const int cnt = p.n_tiles - first;
    if (rest < cnt) { mt = row; nt = first + rest; return; }
    rest -= cnt;
    ++row;
  }
}

// The sequence of (tile, k-block range) pieces one worker (a CTA, or a CTA pair) processes;
// all three roles of a CTA walk the same sequence.  Piece number = split * num_tiles + tile,
// dealt round-robin, so the workers of one round sit on neighbouring tiles of the same
// k-range and stream the same rows of the operands through L2 together.
struct WorkIter {
  int tile, kb0, kb1, slot, split;
  int next_item, stride, total;
  __device__ __forceinline__ WorkIter(const TcParams& p, int worker, int num_workers) {
    next_item = worker; stride = num_workers; total = p.num_tiles * p.splits;
    tile = kb0 = kb1 = slot = split = 0;
  }
  __device__ __forceinline__ bool next(const TcParams& p) {
    if (next_item >= total) return false;
    split = next_item / p.num_tiles;
    tile = next_item - split * p.num_tiles;
    // (by row classes: kblocks counts one class's tokens, which cls_sub pieces share)
    const int part = p.cls_sub > 0 ? split % p.cls_sub : split;
    const int parts = p.cls_sub > 0 ? p.cls_sub : p.splits;
    kb0 = static_cast<int>(static_cast<long long>(part) * p.kblocks / parts);
    kb1 = static_cast<int>(static_cast<long long>(part + 1) * p.kblocks / parts);
    slot = next_item;
    next_item += stride;
    return true;
  }
};

// The aligned 32-bit word holding elements e, e + 1 of a row of `cols` elements (e may be -1: that
// half is never used); elements outside the row read as zero and are never fetched.
__device__ __forceinline__ uint32_t ldg_pair(const __nv_bfloat16* row, int e, int cols) {
  if (e + 1 < cols) return __ldg(reinterpret_cast<const unsigned int*>(row + e));
  if (e >= 0 && e < cols) return static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(row + e)));
  return 0u;
}

template <int CTAS, int BN, bool MN_MAJOR, int EPI, bool A_LDG, bool A_CLS>
__device__ __forceinline__ void gemm_tc_body(const CUtensorMap& tmap_a, const CUtensorMap& tmap_b, const CUtensorMap& tmap_c,
                                             const CUtensorMap& tmap_b2, const CUtensorMap& tmap_c2,
                                             const ClassMaps* cls, const CUtensorMap* cls_z, const TcParams& p) {
  static_assert(!A_CLS || (!A_LDG && CTAS == 2 && (MN_MAJOR ? EPI == EPI_PARTIAL : (EPI == EPI_BF16 || Cfg<CTAS, BN, EPI>::ACT))),
                "row classes: CTA pairs; K-major with bf16 out or a fused consumer, or token-major with partial tiles");
  constexpr bool CLS_K = A_CLS && !MN_MAJOR && EPI == EPI_BF16;   // classes of rows of a K-major A: m-tiles belong to classes
  constexpr bool CLS_T = A_CLS && MN_MAJOR;                       // classes of tokens: K pieces belong to classes
  // Fused consumers whose factor and output have rows off the 16-byte grid: m-tiles belong to
  // classes of rows as in CLS_K, but here it is the output columns that run `shift` ahead (tile
  // column c is column c - shift of the matrices), so B's rows are fetched `shift` early.  cls->a are
  // the classes of the factor, cls->c of the output, cls_z of A (Z, whose rows are aligned: plain strides).
  constexpr bool CLS_N = A_CLS && !MN_MAJOR && Cfg<CTAS, BN, EPI>::ACT;
  using C = Cfg<CTAS, BN, EPI>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  SmemCtl* ctl = reinterpret_cast<SmemCtl*>(smem + C::CTL_OFFSET);
  volatile int* abort_flag = &ctl->abort_flag;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t cta_rank = (CTAS == 2) ? ptx::cluster_ctarank() : 0u;  // 0 = leader
  const int worker = blockIdx.x / CTAS;         // tile owner: a CTA, or a cluster of two
  const int num_workers = gridDim.x / CTAS;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) {
      // with plain-load A every loader warp (of both CTAs of a pair) also reports on the leader's barrier
      ptx::mbar_init(&ctl->full[s], A_LDG ? 1 + LOADER_WARPS * CTAS : 1);   // (one group of loader warps per stage)
      ptx::mbar_init(&ctl->empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(&ctl->acc_full[b], 1);
      ptx::mbar_init(&ctl->acc_empty[b], EPI_WARPS * CTAS);
    }
    if (C::ACT) {
      for (int e = 0; e < EPI_WARPS; ++e)
        for (int b = 0; b < MAX_AUX_BUFS; ++b) ptx::mbar_init(&ctl->aux_full[e][b], 1);
    }
    ctl->abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::fence_proxy_async();
  }
  if (warp == 1) {
    if (CTAS == 2) {
      ptx::tmem_alloc_pair(&ctl->tmem_base, C::TMEM_COLS);
      ptx::tmem_relinquish_pair();
    } else {
      ptx::tmem_alloc(&ctl->tmem_base, C::TMEM_COLS);
      ptx::tmem_relinquish();
    }
  }
  ptx::tc_fence_before_sync();
  if (CTAS == 2) ptx::cluster_sync_all();   // the peer's barriers must exist before any remote arrive
  else __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = ctl->tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (both CTAs)
    if (ptx::elect_one()) {
      ptx::prefetch_tensormap(&tmap_a);
      ptx::prefetch_tensormap(&tmap_b);
      if (p.n_tiles1 < p.n_tiles) ptx::prefetch_tensormap(&tmap_b2);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      WorkIter w(p, worker, num_workers);
      while (ok && w.next(p)) {
        int mt, nt;
        tile_coords<C::TILE_M, BN>(p, w.tile, mt, nt);
        // row classes: m-tile mt is tile mt / P of class mt % P; rows are counted within the class
        const int cls_j = (CLS_K || CLS_N) ? mt % p.cls_count : (CLS_T ? w.split / p.cls_sub : 0);
        const int cls_shift = CLS_K ? p.cls_shift[cls_j] : 0;
        const int n_shift = CLS_N ? p.cls_shift[cls_j] : 0;
        const CUtensorMap* map_a = (CLS_K || CLS_T) ? &cls->a[cls_j] : (CLS_N ? &cls_z[cls_j] : &tmap_a);
        const int row_a = ((CLS_K || CLS_N) ? mt / p.cls_count : mt) * C::TILE_M + static_cast<int>(cta_rank) * BM;
        const bool second = nt >= p.n_tiles1;
        const CUtensorMap* map_b = CLS_T ? &cls->c[cls_j] : (second ? &tmap_b2 : &tmap_b);
        // this CTA's rows of B: its share of the tile's columns, or (wide tiles) of each 256-column half
        const int row_b = (second ? nt - p.n_tiles1 : nt) * BN + static_cast<int>(cta_rank) * (C::MMA_N / CTAS);
        for (int kb = w.kb0; kb < w.kb1; ++kb) {
          if (!ptx::mbar_wait(&ctl->empty[stage], phase ^ 1u, abort_flag, WAIT_LIMIT)) { ok = false; break; }
          uint8_t* sa = smem + stage * C::STAGE_BYTES;
          uint8_t* sb = sa + C::A_BYTES;
          const int seg = kb / p.kb_per_seg;
          const int k_in = (kb - seg * p.kb_per_seg) * BK;
          const int ka = p.seg_a[seg] + k_in, kbb = p.seg_b[seg] + k_in;
          constexpr int TMA_BYTES = A_LDG ? C::B_BYTES : C::STAGE_BYTES;   // what TMA brings per CTA and stage
          if (CTAS == 1) {
            ptx::mbar_arrive_expect_tx(&ctl->full[stage], TMA_BYTES);
            if (!MN_MAJOR) {
              if (!A_LDG) ptx::tma_load_2d(sa, &tmap_a, &ctl->full[stage], ka, row_a);
              ptx::tma_load_2d(sb, map_b, &ctl->full[stage], kbb, row_b);
            } else {
              if (!A_LDG) {
#pragma unroll
                for (int j = 0; j < BM / 64; ++j)
                  ptx::tma_load_2d(sa + j * (BK * 128), &tmap_a, &ctl->full[stage], row_a + 64 * j, ka);
              }
#pragma unroll
              for (int j = 0; j < C::NB_LOCAL / 64; ++j)
                ptx::tma_load_2d(sb + j * (BK * 128), map_b, &ctl->full[stage], row_b + 64 * j, kbb);
            }
          } else {
            // Both CTAs' bytes are counted on the leader's barrier: the leader announces the
            // total, each CTA's copies report there.
            if (cta_rank == 0) ptx::mbar_arrive_expect_tx(&ctl->full[stage], 2 * TMA_BYTES);
            const uint32_t bar = ptx::mapa_shared(ptx::smem_u32(&ctl->full[stage]), 0);
            if (CLS_K) {
              ptx::tma_load_2d_pair(sa, map_a, bar, ka, row_a);
#pragma unroll
              for (int j = 0; j < C::NB_LOCAL / 64; ++j) {   // B rows = K, fetched `shift` rows early (zeros outside)
                constexpr int PER_HALF = C::MMA_N / CTAS / 64;   // 64-column blocks of this CTA in one MMA's columns
                ptx::tma_load_2d_pair(sb + j * (BK * 128), map_b, bar, row_b + (j / PER_HALF) * C::MMA_N + 64 * (j % PER_HALF),
                                      kbb - cls_shift);
              }
            } else if (!MN_MAJOR) {
              if (!A_LDG) ptx::tma_load_2d_pair(sa, map_a, bar, ka, row_a);
#pragma unroll
              for (int h = 0; h < BN / C::MMA_N; ++h)    // (a wide tile: this CTA's rows of each 256-column half)
                ptx::tma_load_2d_pair(sb + h * (C::B_BYTES / (BN / C::MMA_N)), map_b, bar, kbb, row_b + h * C::MMA_N - n_shift);
            } else {
              if (!A_LDG) {
#pragma unroll
                for (int j = 0; j < BM / 64; ++j)
                  ptx::tma_load_2d_pair(sa + j * (BK * 128), map_a, bar, row_a + 64 * j, ka);
              }
#pragma unroll
              for (int j = 0; j < C::NB_LOCAL / 64; ++j)
                ptx::tma_load_2d_pair(sb + j * (BK * 128), map_b, bar, row_b + 64 * j, kbb);
            }
          }
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      // Tail: wait until every stage this CTA filled has been released, so that no MMA
      // completion can still signal this CTA's barriers after it has left.
      for (int s = 0; s < C::STAGES && ok; ++s) {
        if (!ptx::mbar_wait(&ctl->empty[stage], phase ^ 1u, abort_flag, WAIT_LIMIT)) ok = false;
        if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader CTA only)
    if (cta_rank == 0 && ptx::elect_one()) {
      constexpr uint32_t idesc = ptx::idesc_bf16_f32(C::TILE_M, C::MMA_N, MN_MAJOR, MN_MAJOR || CLS_K);
      constexpr int HALVES = BN / C::MMA_N;                        // MMAs per k-step (2 for a wide tile)
      constexpr int B_HALF = C::B_BYTES / HALVES;                  // this CTA's rows of one half
      int stage = 0;
      uint32_t phase = 0;
      int acc_iter = 0;
      bool ok = true;
      WorkIter w(p, worker, num_workers);
      for (; ok && w.next(p); ++acc_iter) {
        const int kb0 = w.kb0, kb1 = w.kb1;
        const int buf = C::ACC_BUFS == 2 ? (acc_iter & 1) : 0;
        const uint32_t acc_phase = (C::ACC_BUFS == 2 ? (acc_iter >> 1) : acc_iter) & 1;
        if (!ptx::mbar_wait(&ctl->acc_empty[buf], acc_phase ^ 1u, abort_flag, WAIT_LIMIT)) { ok = false; break; }
        ptx::tc_fence_after_sync();
        const uint32_t tmem_d = tmem_base + static_cast<uint32_t>(buf * BN);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!ptx::mbar_wait(&ctl->full[stage], phase, abort_flag, WAIT_LIMIT)) { ok = false; break; }
          ptx::tc_fence_after_sync();
          const uint32_t sa = ptx::smem_u32(smem + stage * C::STAGE_BYTES);
          const uint32_t sb = sa + C::A_BYTES;
#pragma unroll
          for (int h = 0; h < HALVES; ++h) {
            // (a wide tile: the second 256 columns have their own release, so that the first MMAs of
            // a tile overlap the draining of the second half of the tile before it)
            if (HALVES == 2 && h == 1 && kb == kb0) {
              if (!ptx::mbar_wait(&ctl->acc_empty[1], acc_phase ^ 1u, abort_flag, WAIT_LIMIT)) { ok = false; break; }
              ptx::tc_fence_after_sync();
            }
            const uint32_t sbh = sb + h * B_HALF;       // this CTA's rows of half h of B
#pragma unroll
            for (int kk = 0; kk < BK / UMMA_K; ++kk) {
              uint64_t da, db;
              if (CLS_K) {
                da = ptx::smem_desc_sw128(sa + kk * (UMMA_K * 2), 16, 1024);
                db = ptx::smem_desc_sw128(sbh + kk * (UMMA_K * 128), BK * 128, 1024);
              } else if (!MN_MAJOR) {
                // 16 K-elements = 32 bytes further inside each 128-byte row
                da = ptx::smem_desc_sw128(sa + kk * (UMMA_K * 2), 16, 1024);
                db = ptx::smem_desc_sw128(sbh + kk * (UMMA_K * 2), 16, 1024);
              } else {
                // 16 K-rows of 128 bytes further; 64-column blocks are BK*128 bytes apart
                da = ptx::smem_desc_sw128(sa + kk * (UMMA_K * 128), BK * 128, 1024);
                db = ptx::smem_desc_sw128(sbh + kk * (UMMA_K * 128), BK * 128, 1024);
              }
              const uint32_t acc = (kb > kb0 || kk > 0) ? 1u : 0u;
              if (CTAS == 2) ptx::umma_bf16_pair(tmem_d + h * C::MMA_N, da, db, idesc, acc);
              else ptx::umma_bf16(tmem_d, da, db, idesc, acc);
            }
          }
          if (!ok) break;
          // frees the stage (in both CTAs) when these MMAs retire
          if (CTAS == 2) ptx::umma_commit_pair(&ctl->empty[stage], 3);
          else ptx::umma_commit(&ctl->empty[stage]);
          if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) {
          if (CTAS == 2) ptx::umma_commit_pair(&ctl->acc_full[buf], 3);
          else ptx::umma_commit(&ctl->acc_full[buf]);
        }
      }
    }
  } else if (A_LDG && warp >= 2 + EPI_WARPS) {
    // ------------------------------------------------------------ A loaders (warps 10.., both CTAs)
    // A row segment of an operand box is 64 bf16 = 128 bytes of one matrix row, starting on a
    // 2-byte boundary only.  One warp fetches it with one 32-bit load per lane: lane l wants the
    // word holding elements 2l, 2l + 1 of the segment; when the segment is not 4-byte aligned the
    // lanes load the aligned words that straddle theirs and shift (the 33rd word of each of the
    // warp's 32 segments comes from one more load, lane j taking segment j's).  The words are
    // stored with the 128-byte swizzle the MMA descriptors expect, made visible to the async
    // proxy, and the warp reports on the leader's barrier.  All 32 + 1 loads of a warp are
    // issued before the first is used; the rows a later k-block needs are prefetched into L2.
    const int lw = (warp - (2 + EPI_WARPS)) % LOADER_WARPS;      // which quarter of the stage's rows
    const int group = (warp - (2 + EPI_WARPS)) / LOADER_WARPS;   // which k-blocks
    int stage = 0;
    uint32_t phase = 0;
    int seq = 0;                 // position in the CTA's sequence of k-blocks
    bool ok = true;
    WorkIter w(p, worker, num_workers);
    const uint32_t full_leader0 = ptx::mapa_shared(ptx::smem_u32(&ctl->full[0]), 0);
    const uintptr_t base_elems = reinterpret_cast<uintptr_t>(p.a_ptr) >> 1;
    // item r in [0, 128) of a stage: K-major: row r of the tile; token-major: token r % 64 of
    // 64-column block r / 64
    auto locate = [&](int r, int row_a, int ka, int& grow, int& gcol, int& soff, int& swz) {
      if (!MN_MAJOR) { grow = row_a + r; gcol = ka; soff = r * 128; swz = r & 7; }
      else { const int j = r >> 6, kk = r & 63; grow = ka + kk; gcol = row_a + 64 * j; soff = j * (BK * 128) + kk * 128; swz = kk & 7; }
    };
    while (ok && w.next(p)) {
      int mt, nt;
      tile_coords<C::TILE_M, BN>(p, w.tile, mt, nt);
      const int row_a = mt * C::TILE_M + static_cast<int>(cta_rank) * BM;
      for (int kb = w.kb0; kb < w.kb1; ++kb, ++seq) {
        if (seq % LOADER_GROUPS == group) {
          // L2 prefetch for the k-block this group handles after the next one (lane = segment)
          {
            const int kbp = kb + 2 * LOADER_GROUPS;
            int grow, gcol, soff, swz;
            locate(lw * 32 + lane, row_a, kbp * BK, grow, gcol, soff, swz);
            if (kbp < w.kb1 && grow < p.a_rows && gcol < p.a_cols) {
              const __nv_bfloat16* q = p.a_ptr + static_cast<long long>(grow) * p.a_ld + gcol;
              ptx::prefetch_l2(q);
              if (gcol + 63 < p.a_cols) ptx::prefetch_l2(q + 63);          // a segment may straddle two lines
            }
          }
          const int ka = kb * BK;
          int g1, c1, so1, sw1;
          locate(lw * 32 + 31, row_a, ka, g1, c1, so1, sw1);
          // interior of the matrix: every 16-byte chunk touched below lies inside its row
          const bool interior = g1 < p.a_rows && c1 + 72 <= p.a_cols;
          if (interior) {
            // Eight lanes per segment, four segments per instruction: lane j of a segment loads
            // the aligned 16-byte chunks j and j + 1 of the nine that cover it (the second load
            // hits the line its neighbour's first brings in) and shifts its own output chunk out of
            // the pair.  Two batches of sixteen segments, all loads of a batch issued before the
            // first is used.  (Taking chunk j + 1 from the neighbouring lane by shuffle instead
            // was measured slower: the shuffles cost more than the second load.)
            const int j = lane & 7, rr = lane >> 3;
            uint8_t* sa = smem + stage * C::STAGE_BYTES;
            bool waited = false;
#pragma unroll 1
            for (int half_b = 0; half_b < 2; ++half_b) {
              uint4 lo[4], hi[4];
              int soffs[4], swzs[4], mis[4];
#pragma unroll
              for (int gq = 0; gq < 4; ++gq) {
                int grow, gcol;
                locate(lw * 32 + half_b * 16 + gq * 4 + rr, row_a, ka, grow, gcol, soffs[gq], swzs[gq]);
                const uintptr_t addr = reinterpret_cast<uintptr_t>(p.a_ptr + static_cast<long long>(grow) * p.a_ld + gcol);
                mis[gq] = static_cast<int>(addr & 15u);
                const uint4* q = reinterpret_cast<const uint4*>(addr & ~static_cast<uintptr_t>(15)) + j;
                asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];"
                             : "=r"(lo[gq].x), "=r"(lo[gq].y), "=r"(lo[gq].z), "=r"(lo[gq].w) : "l"(q));
                asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];"
                             : "=r"(hi[gq].x), "=r"(hi[gq].y), "=r"(hi[gq].z), "=r"(hi[gq].w) : "l"(q + 1));
              }
              if (!waited) {    // the stage must be free before it is overwritten; the loads are in flight
                if (!ptx::mbar_wait(&ctl->empty[stage], phase ^ 1u, abort_flag, WAIT_LIMIT)) { ok = false; break; }
                waited = true;
              }
#pragma unroll
              for (int gq = 0; gq < 4; ++gq) {
                const uint32_t W[8] = {lo[gq].x, lo[gq].y, lo[gq].z, lo[gq].w, hi[gq].x, hi[gq].y, hi[gq].z, hi[gq].w};
                const int wo = mis[gq] >> 2;
                const uint32_t sh = static_cast<uint32_t>(mis[gq] & 2) << 3;       // 0 or 16 bits
                uint32_t t[6], u[5];
#pragma unroll
                for (int q = 0; q < 6; ++q) t[q] = (wo & 2) ? W[q + 2] : W[q];
#pragma unroll
                for (int q = 0; q < 5; ++q) u[q] = (wo & 1) ? t[q + 1] : t[q];
                uint4 o;
                o.x = __funnelshift_r(u[0], u[1], sh);
                o.y = __funnelshift_r(u[1], u[2], sh);
                o.z = __funnelshift_r(u[2], u[3], sh);
                o.w = __funnelshift_r(u[3], u[4], sh);
                *reinterpret_cast<uint4*>(sa + soffs[gq] + ((j ^ swzs[gq]) << 4)) = o;
              }
            }
            if (!ok) break;
          } else {
          uint32_t wv[32];
          uint32_t odd_mask = 0u, extra = 0u;
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            int grow, gcol, soff, swz;
            locate(lw * 32 + e, row_a, ka, grow, gcol, soff, swz);
            const long long off = static_cast<long long>(grow) * p.a_ld + gcol;
            const bool odd = ((base_elems + static_cast<uintptr_t>(off)) & 1u) != 0;
            odd_mask |= odd ? (1u << e) : 0u;
            wv[e] = 0u;
            if (grow < p.a_rows) {
              const __nv_bfloat16* row = p.a_ptr + static_cast<long long>(grow) * p.a_ld;
              wv[e] = ldg_pair(row, gcol + 2 * lane - (odd ? 1 : 0), p.a_cols);
            }
          }
          if (odd_mask) {       // the 33rd word of the odd segments: lane j takes segment j's
            int grow, gcol, soff, swz;
            locate(lw * 32 + lane, row_a, ka, grow, gcol, soff, swz);
            if (((odd_mask >> lane) & 1u) && grow < p.a_rows)
              extra = ldg_pair(p.a_ptr + static_cast<long long>(grow) * p.a_ld, gcol + 63, p.a_cols);
          }
          // the stage must be free before it is overwritten; the loads above are already in flight
          if (!ptx::mbar_wait(&ctl->empty[stage], phase ^ 1u, abort_flag, WAIT_LIMIT)) { ok = false; break; }
          uint8_t* sa = smem + stage * C::STAGE_BYTES;
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            int grow, gcol, soff, swz;
            locate(lw * 32 + e, row_a, ka, grow, gcol, soff, swz);
            uint32_t v = wv[e];
            if ((odd_mask >> e) & 1u) {                                   // warp-uniform
              uint32_t next = __shfl_down_sync(0xffffffffu, wv[e], 1);
              const uint32_t last = __shfl_sync(0xffffffffu, extra, e);
              if (lane == 31) next = last;
              v = __funnelshift_r(wv[e], next, 16);
            }
            *reinterpret_cast<uint32_t*>(sa + soff + ((((lane >> 2) ^ swz) << 4) | ((lane & 3) << 2))) = v;
          }
          }
          ptx::fence_proxy_async();
          __syncwarp();
          if (lane == 0) {
            const uint32_t bar = full_leader0 + static_cast<uint32_t>(stage) * 8u;
            if (CTAS == 2) ptx::mbar_arrive_cluster(bar);
            else ptx::mbar_arrive(&ctl->full[stage]);
          }
        }
        if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..9, both CTAs)
    // A warp reaches the TMEM lanes [32 (warp % 4), +32).  Two warps share each quarter of the
    // accumulator's rows and take alternate column blocks of it.
    const int quarter = warp & 3;
    const int half = (warp - 2) >> 2;      // 0 or 1
    const int ewarp = warp - 2;            // 0 .. EPI_WARPS - 1: owner of a staging area
    int acc_iter = 0;
    bool ok = true;
    constexpr bool EPI_RMS = (EPI == EPI_RMS1 || EPI == EPI_RMS2);
    constexpr bool EPI_ACT = C::ACT;
    // Activation and RMSNorm epilogues: the element-wise factor of every 32-row x 64-column block
    // this warp will work on arrives by a TMA tile load (tensor map in the tmap_c2 slot) in one of
    // the warp's staging buffers, AUX_AHEAD blocks before the warp gets to it; blocks are numbered
    // in the order the warp meets them, block i uses buffer i % NBUF.  `wf` walks the same
    // sequence of tiles as `w`, ahead of it.
    constexpr int NBUF = EPI_ACT ? C::AUX_BUFS : 1;
    constexpr int AUX_AHEAD = (EPI == EPI_RMS1) ? NBUF - 1 : NBUF - 2;
    WorkIter wf(p, worker, num_workers);
    int f_mt = 0, f_nt = 0, f_c = BN / 64;   // the block the next load is for (f_c past the end: next tile)
    bool f_more = EPI_ACT;
    int produced = 0, consumed = 0;          // loads issued / blocks taken up, this warp
    auto feed = [&]() {
      // Issue loads until AUX_AHEAD blocks beyond block `consumed` are on their way.  A buffer is
      // refilled only after the store that left from it has read it: with one store group
      // committed per block, at most one group may still be pending (that of the block just
      // finished).  Where the block did not leave by a tile store the buffer was last touched by
      // ordinary reads and writes, which the proxy fence orders before the TMA write.
      if (!EPI_ACT || !f_more || produced > consumed + AUX_AHEAD) return;
      if (EPI != EPI_RMS1 && lane == 0) ptx::bulk_wait_group_read<1>();
      ptx::fence_proxy_async();     // (the buffer may last have been a transpose tile, or only read)
      __syncwarp();
      while (produced <= consumed + AUX_AHEAD) {
        // (by classes: the columns of class j run up to N + shift_j, its rows are counted within the class)
        while (!(f_c < BN / 64 && f_nt * BN + f_c * 64 < p.N + (CLS_N ? p.cls_shift[f_mt % p.cls_count] : 0))) {
          if (!wf.next(p)) { f_more = false; return; }
          tile_coords<C::TILE_M, BN>(p, wf.tile, f_mt, f_nt);
          f_c = half;
        }
        if (lane == 0) {
          const int b = produced % NBUF;
          uint64_t* bar = &ctl->aux_full[ewarp][b];
          const CUtensorMap* map_x = CLS_N ? &cls->a[f_mt % p.cls_count] : &tmap_c2;
          ptx::mbar_arrive_expect_tx(bar, STORE_BUF_BYTES);     // rows or columns past the edge arrive as zeros
          ptx::tma_load_2d(smem + C::EPI_OFFSET + (ewarp * NBUF + b) * STORE_BUF_BYTES, map_x, bar, f_nt * BN + f_c * 64,
                           (CLS_N ? f_mt / p.cls_count : f_mt) * C::TILE_M + static_cast<int>(cta_rank) * BM + quarter * 32);
        }
        ++produced;
        f_c += 2;
      }
    };
    WorkIter w(p, worker, num_workers);
    for (; ok && w.next(p); ++acc_iter) {
      int mt, nt;
      tile_coords<C::TILE_M, BN>(p, w.tile, mt, nt);
      const int buf = C::ACC_BUFS == 2 ? (acc_iter & 1) : 0;
      const uint32_t acc_phase = (C::ACC_BUFS == 2 ? (acc_iter >> 1) : acc_iter) & 1;
      if (EPI_ACT) feed();     // before the wait for the accumulator: the factor's trip overlaps it
      // RMSNorm passes: this lane's row factors, fetched ahead of the same wait
      float rms_a = 0.f, rms_b = 0.f, rms_c = 0.f;
      if (EPI_RMS) {
        const int cj = CLS_N ? mt % p.cls_count : 0;
        const int rows = CLS_N ? (p.M - cj + p.cls_count - 1) / p.cls_count : p.M;
        const int r0 = (CLS_N ? mt / p.cls_count : mt) * C::TILE_M + static_cast<int>(cta_rank) * BM + quarter * 32;
        const int gr = CLS_N ? (r0 + lane) * p.cls_count + cj : r0 + lane;
        if (r0 + lane < rows) {
          rms_a = __ldg(p.row_a + gr);
          if (EPI == EPI_RMS2) {
            rms_b = __ldg(p.row_b + gr);
            if (p.row_c) rms_c = __ldg(p.row_c + gr);
          }
        }
      }
      if (!ptx::mbar_wait(&ctl->acc_full[buf], acc_phase, abort_flag, WAIT_LIMIT)) { ok = false; break; }
      ptx::tc_fence_after_sync();
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                             static_cast<uint32_t>(buf * BN);
      if (EPI == EPI_PARTIAL) {
        float* dst_row = p.partial + static_cast<long long>(w.slot) * (C::TILE_M * BN) +
                         (static_cast<int>(cta_rank) * BM + quarter * 32 + lane) * BN;
#pragma unroll 1
        for (int c = half; c < BN / 32; c += 2) {
          uint32_t v[32];
          ptx::tmem_ld_32x32(taddr + c * 32, v);
          ptx::tmem_ld_wait();
          float* dst = dst_row + c * 32;
#pragma unroll
          for (int j = 0; j < 8; ++j)
            reinterpret_cast<uint4*>(dst)[j] = make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
        }
      } else {
        // Each lane holds one output row.  When rows start on 16-byte boundaries the lane
        // stores its own row segment with 16-byte stores.  Otherwise a 32 x 32 block of
        // 32-bit words (fp32 values, or pairs of bf16) goes through shared memory so that
        // one store instruction writes 128 contiguous bytes of a single row.
        constexpr bool OUT_BF16 = (EPI == EPI_BF16 || EPI_ACT);   // 64-column blocks (RMS1 stores nothing)
        constexpr int ELEM = OUT_BF16 ? 2 : 4;
        const bool second = nt >= p.n_tiles1;
        void* const out_c = second ? p.C2 : p.C;
        const long long out_ld = second ? p.ldc2 : p.ldc;
        const int cls_j = (CLS_K || CLS_N) ? mt % p.cls_count : 0;
        const int n_shift = CLS_N ? p.cls_shift[cls_j] : 0;      // tile column c is column c - n_shift of dY, dX, gains
        const int out_n = (second ? p.N2 : p.N) + n_shift;
        const int out_tma = second ? p.tma_store2 : p.tma_store;
        const CUtensorMap* map_c = (CLS_K || CLS_N) ? &cls->c[cls_j] : (second ? &tmap_c2 : &tmap_c);
        // rows this tile's coordinates run over: the matrix, or the class (its tensor map clips there too)
        const int m_rows = (CLS_K || CLS_N) ? (p.M - cls_j + p.cls_count - 1) / p.cls_count : p.M;
        const int nt_out = second ? nt - p.n_tiles1 : nt;
        const bool rows_aligned = ((reinterpret_cast<uintptr_t>(out_c) & 15u) == 0) && ((out_ld * ELEM) % 16 == 0);
        const int row0 = ((CLS_K || CLS_N) ? mt / p.cls_count : mt) * C::TILE_M + static_cast<int>(cta_rank) * BM + quarter * 32;
        constexpr int COLS_PER_BLOCK = OUT_BF16 ? 64 : 32;
        // this lane's row of the matrices (by classes: row0 counts rows of the class)
        const int grow = CLS_N ? (row0 + lane) * p.cls_count + cls_j : row0 + lane;
        float rms_u = 0.f, rms_u2 = 0.f;     // pass 1 of the norm backward: this lane's running row sums
        // a wide tile: the first 256 columns of the accumulator are handed back as soon as this
        // warp has read its blocks of them
        bool first_half_held = (C::ACC_BUFS == 1);
        auto release_first_half = [&]() {
          first_half_held = false;
          ptx::tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive_cluster(ptx::mapa_shared(ptx::smem_u32(&ctl->acc_empty[0]), 0));
        };
#pragma unroll 1
        for (int c = half; c < BN / COLS_PER_BLOCK; c += 2) {
          const int col0 = nt_out * BN + c * COLS_PER_BLOCK;
          if (C::ACC_BUFS == 1 && first_half_held && c * COLS_PER_BLOCK >= C::MMA_N) release_first_half();
          if (col0 >= out_n) break;                     // warp-uniform
          // the staging buffer of this block: the warp's only one, or the one its factor is in
          uint8_t* sbuf = smem + C::EPI_OFFSET + (ewarp * C::STORE_BUFS + (EPI_ACT ? consumed % NBUF : 0)) * STORE_BUF_BYTES;
          if (EPI_ACT) {
            feed();
            if (!ptx::mbar_wait(&ctl->aux_full[ewarp][consumed % NBUF], static_cast<uint32_t>(consumed / NBUF) & 1u,
                                abort_flag, WAIT_LIMIT)) { ok = false; break; }
            ++consumed;
          }
          uint32_t v[32];
          if (OUT_BF16) {
            uint32_t lo[32], hi[32];
            ptx::tmem_ld_32x32(taddr + c * 64, lo);
            ptx::tmem_ld_32x32(taddr + c * 64 + 32, hi);
            ptx::tmem_ld_wait();
            if (EPI_ACT) {
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                // eight factors of this lane's row (the tile load's 128-byte swizzle: chunk j of row l at j ^ (l & 7))
                const uint4 aux8 = *reinterpret_cast<const uint4*>(sbuf + lane * 128 + ((j ^ (lane & 7)) << 4));
                const __nv_bfloat16* f = reinterpret_cast<const __nv_bfloat16*>(&aux8);
                uint32_t* acc = (j < 4) ? lo : hi;
                float gv[8];
                if (EPI_RMS) {
                  // eight gains of these columns (the same for every lane; zero past the last column):
                  // two 16-byte loads where the gain vector allows it
                  const int cj = col0 + 8 * j - n_shift;
                  if (!CLS_N && p.col_g_vec && cj + 8 <= out_n) {
                    const float4 g0 = __ldg(reinterpret_cast<const float4*>(p.col_g + cj));
                    const float4 g1 = __ldg(reinterpret_cast<const float4*>(p.col_g + cj) + 1);
                    gv[0] = g0.x; gv[1] = g0.y; gv[2] = g0.z; gv[3] = g0.w;
                    gv[4] = g1.x; gv[5] = g1.y; gv[6] = g1.z; gv[7] = g1.w;
                  } else {
#pragma unroll
                    for (int e = 0; e < 8; ++e) gv[e] = (cj + e >= 0 && cj + e < out_n - n_shift) ? __ldg(p.col_g + cj + e) : 0.f;
                  }
                }
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                  const int w = (j & 3) * 8 + e;
                  const float x = __uint_as_float(acc[w]);
                  float dy = __bfloat162float(f[e]);                 // zero past the last row and column
                  if (CLS_N && col0 + 8 * j + e < n_shift) dy = 0.f;   // (by classes: the end of the row before)
                  if (EPI == EPI_RMS1) {
                    const float t = dy * x;
                    rms_u = fmaf(gv[e], t, rms_u);
                    rms_u2 = fmaf(gv[e], dy, rms_u2);
                    acc[w] = __float_as_uint(rms_a * t);          // this row's term of the column sum
                  } else if (EPI == EPI_RMS2) {
                    acc[w] = __float_as_uint(fmaf(rms_a * gv[e], dy, fmaf(-rms_b, x, rms_c)));
                  } else {
                    acc[w] = __float_as_uint(dy * act_derivative_fast<EPI == EPI_SILU ? ACT_SILU : ACT_GELU>(x));
                  }
                }
              }
            }
            if (EPI == EPI_RMS1) {
              // Column sums over the warp's 32 rows, 32 columns at a time, without leaving the
              // registers: five butterfly rounds, in each of which a lane keeps the half of its
              // columns that matches one bit of its number and adds the partner lane's values of
              // the same columns; lane l ends with the sum of column l.  31 shuffles per 32 columns
              // (a transpose through shared memory cost 64 accesses and two warp barriers).
              const int rowblock = CLS_N ? cls_j * ((((p.M + p.cls_count - 1) / p.cls_count) + 31) >> 5) + (row0 >> 5) : (row0 >> 5);
#pragma unroll
              for (int hh = 0; hh < 2; ++hh) {
                float a[32];
#pragma unroll
                for (int q = 0; q < 32; ++q) a[q] = __uint_as_float(hh ? hi[q] : lo[q]);
#pragma unroll
                for (int off = 16; off >= 1; off >>= 1) {
                  const bool up = (lane & off) != 0;
#pragma unroll
                  for (int q = 0; q < off; ++q) {
                    const float send = up ? a[q] : a[q + off];
                    const float keep = up ? a[q + off] : a[q];
                    a[q] = keep + __shfl_xor_sync(0xffffffffu, send, off);
                  }
                }
                const int col = col0 + 32 * hh + lane - n_shift;
                if (col >= 0 && col < p.N && row0 < m_rows) p.col_part[static_cast<long long>(rowblock) * p.N + col] = a[0];
              }
              continue;
            }
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const __nv_bfloat162 a = __floats2bfloat162_rn(__uint_as_float(lo[2 * j]), __uint_as_float(lo[2 * j + 1]));
              const __nv_bfloat162 b = __floats2bfloat162_rn(__uint_as_float(hi[2 * j]), __uint_as_float(hi[2 * j + 1]));
              v[j] = *reinterpret_cast<const uint32_t*>(&a);
              v[16 + j] = *reinterpret_cast<const uint32_t*>(&b);
            }
          } else {
            ptx::tmem_ld_32x32(taddr + c * 32, v);
            ptx::tmem_ld_wait();
          }
          // A tile store writes whole 16-byte pieces: where the row ends inside one, the piece's other
          // bytes (row padding, the neighbouring columns of a wider buffer, or, by classes, the start of
          // the next row) would be overwritten.  The block holding such a row end, and by classes also
          // the block a row starts in (its first columns are the end of the row before), leave
          // element by element through the transpose path below.
          const bool ragged = (col0 + COLS_PER_BLOCK > out_n) &&
                              (CLS_N || (static_cast<long long>(out_n - n_shift) * ELEM) % 16 != 0);
          if (out_tma && !ragged && !(CLS_N && col0 < n_shift)) {
            // Stage the 32 x 128-byte block (row = lane) with the 128-byte swizzle of the
            // tensor map, then one lane hands it to the TMA unit, which writes whole rows and
            // clips at the matrix edge.  A plain epilogue waits until the store that last left
            // from its buffer has read it; an activation epilogue writes over the factor it has
            // just used (each lane its own row), in a buffer no store is reading (see feed()),
            // and commits one group per block, with or without a store in it.
            if (row0 < m_rows) {
              if (!EPI_ACT) {
                if (lane == 0) ptx::bulk_wait_group_read<0>();
                __syncwarp();
              }
#pragma unroll
              for (int j = 0; j < 8; ++j)
                *reinterpret_cast<uint4*>(sbuf + lane * 128 + ((j ^ (lane & 7)) << 4)) =
                    make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
              ptx::fence_proxy_async();
              __syncwarp();
              if (lane == 0) {
                if (EPI == EPI_F32 && p.accumulate) ptx::tma_reduce_add_2d(map_c, sbuf, col0, row0);
                else ptx::tma_store_2d(map_c, sbuf, col0, row0);
              }
            }
            if (lane == 0 && (EPI_ACT || row0 < m_rows)) ptx::bulk_commit_group();
            continue;
          }
          if (rows_aligned && col0 + COLS_PER_BLOCK <= out_n) {
            const int row = row0 + lane;
            if (row < p.M) {
              uint8_t* dst = reinterpret_cast<uint8_t*>(out_c) + (static_cast<long long>(row) * out_ld + col0) * ELEM;
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                uint4 o = make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                if (EPI == EPI_F32 && p.accumulate) {
                  const float4 old = reinterpret_cast<const float4*>(dst)[j];
                  o.x = __float_as_uint(__uint_as_float(o.x) + old.x);
                  o.y = __float_as_uint(__uint_as_float(o.y) + old.y);
                  o.z = __float_as_uint(__uint_as_float(o.z) + old.z);
                  o.w = __float_as_uint(__uint_as_float(o.w) + old.w);
                }
                reinterpret_cast<uint4*>(dst)[j] = o;
              }
            }
            continue;
          }
          // The transpose tile takes the place of the staging buffer, once no tile store is reading
          // it any more.  Rows and columns are those of the matrices (by classes: row0 counts rows
          // of the class, and tile column c is column c - n_shift).
          uint32_t* xp = reinterpret_cast<uint32_t*>(sbuf);
          if (lane == 0) ptx::bulk_wait_group_read<0>();
          __syncwarp();
#pragma unroll
          for (int j = 0; j < 32; ++j) xp[lane * 32 + (j ^ lane)] = v[j];
          __syncwarp();
          const int real_n = out_n - n_shift;
          if (OUT_BF16) {
            __nv_bfloat16* base = reinterpret_cast<__nv_bfloat16*>(out_c);
            const bool words = (n_shift == 0) && (col0 + 64 <= out_n) && ((out_ld & 1) == 0) &&
                               ((reinterpret_cast<uintptr_t>(base) & 3u) == 0);
            const int c0 = col0 + 2 * lane - n_shift;
#pragma unroll 4
            for (int rr = 0; rr < 32; ++rr) {
              if (row0 + rr >= m_rows) break;         // warp-uniform
              const long long row = (CLS_K || CLS_N) ? static_cast<long long>(row0 + rr) * p.cls_count + cls_j : row0 + rr;
              const uint32_t wv = xp[rr * 32 + (lane ^ rr)];
              __nv_bfloat16* dst = base + row * out_ld + c0;
              if (words) {
                *reinterpret_cast<uint32_t*>(dst) = wv;
              } else {
                const __nv_bfloat162 h = *reinterpret_cast<const __nv_bfloat162*>(&wv);
                if (c0 >= 0 && c0 < real_n) dst[0] = h.x;
                if (c0 + 1 >= 0 && c0 + 1 < real_n) dst[1] = h.y;
              }
            }
          } else {
            float* base = reinterpret_cast<float*>(out_c);
            const bool in_n = col0 + lane < out_n;
#pragma unroll 4
            for (int rr = 0; rr < 32; ++rr) {
              if (row0 + rr >= m_rows) break;         // warp-uniform
              float o = __uint_as_float(xp[rr * 32 + (lane ^ rr)]);
              float* dst = base + static_cast<long long>(row0 + rr) * out_ld + col0 + lane;
              if (in_n) {
                if (p.accumulate) o += *dst;
                *dst = o;
              }
            }
          }
          __syncwarp();
          if (EPI_ACT && out_tma && lane == 0) ptx::bulk_commit_group();   // one group per block, see feed()
        }
        if (!ok) break;
        if (C::ACC_BUFS == 1 && first_half_held) release_first_half();
        if (EPI == EPI_RMS1 && row0 + lane < m_rows) {
          p.row_part[static_cast<long long>(2 * nt + half) * p.M + grow] = rms_u;
          if (p.row_part2) p.row_part2[static_cast<long long>(2 * nt + half) * p.M + grow] = rms_u2;
        }
      }
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) {
        // the accumulator buffer is free once the four warps of every CTA of the tile are done
        // (a wide tile: this releases its second half; the first was released on the way)
        const int rel = C::ACC_BUFS == 2 ? buf : 1;
        if (CTAS == 2) ptx::mbar_arrive_cluster(ptx::mapa_shared(ptx::smem_u32(&ctl->acc_empty[rel]), 0));
        else ptx::mbar_arrive(&ctl->acc_empty[rel]);
      }
    }
    if (EPI != EPI_PARTIAL && lane == 0) ptx::bulk_wait_group<0>();   // tile stores have landed
  }

  // ---------------------------------------------------------------- common exit
  __syncwarp();
  if (*abort_flag) {
    // Some wait gave up: report it, give copies still in flight time to land, then leave.
    if (lane == 0 && p.dev_status) atomicOr(p.dev_status, DEV_WAIT_EXPIRED);
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
  }
  ptx::tc_fence_before_sync();
  // Neither CTA of a pair may leave (or free tensor memory) while the other can still
  // signal its barriers or feed MMAs from its shared memory.
  if (CTAS == 2) ptx::cluster_sync_all();
  else __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    if (CTAS == 2) ptx::tmem_dealloc_pair(tmem_base, C::TMEM_COLS);
    else ptx::tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
}

template <int CTAS, int BN, bool MN_MAJOR, int EPI, bool A_LDG = false>
__global__ void __launch_bounds__(A_LDG ? NUM_THREADS_LDG : NUM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
               const __grid_constant__ CUtensorMap tmap_c, const __grid_constant__ CUtensorMap tmap_b2,
               const __grid_constant__ CUtensorMap tmap_c2, const TcParams p) {
  gemm_tc_body<CTAS, BN, MN_MAJOR, EPI, A_LDG, false>(tmap_a, tmap_b, tmap_c, tmap_b2, tmap_c2, nullptr, nullptr, p);
}

// C (bf16) = A B with A (M x K, K-major) taken by row classes (see ClassMaps) and B (K x N) MN-major.
template <int BN>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_tc_rowclass_kernel(const __grid_constant__ ClassMaps cls, const __grid_constant__ CUtensorMap tmap_b,
                        const TcParams p) {
  gemm_tc_body<2, BN, false, EPI_BF16, false, true>(cls.a[0], tmap_b, cls.c[0], tmap_b, cls.c[0], &cls, nullptr, p);
}

// Partial tiles of A^T B with the tokens (rows of A and B) taken by classes (see ClassMaps).
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_tc_tokens_rowclass_kernel(const __grid_constant__ ClassMaps cls, const TcParams p) {
  gemm_tc_body<2, 256, true, EPI_PARTIAL, false, true>(cls.a[0], cls.c[0], cls.a[0], cls.c[0], cls.a[0], &cls, nullptr, p);
}

// The fused consumers (activation backward, the two norm-backward passes) on a factor dY and an
// output dX whose rows are off the 16-byte grid: io.a = classes of dY, io.c = classes of dX, z =
// the same classes of rows of Z.
struct ConsumerClassMaps {
  ClassMaps io;
  CUtensorMap z[8];
};
template <int EPI>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_tc_consumer_rowclass_kernel(const __grid_constant__ ConsumerClassMaps cm, const __grid_constant__ CUtensorMap tmap_b,
                                 const TcParams p) {
  gemm_tc_body<2, 256, false, EPI, false, true>(cm.z[0], tmap_b, cm.io.c[0], tmap_b, cm.io.a[0], &cm.io, cm.z, p);
}

// Position of tile (mt, nt) in the order the kernel enumerates tiles.
__device__ __forceinline__ int tile_index(int mt, int nt, int n_tiles, int tile_m, int bn, int symmetric) {
  if (!symmetric) return mt * n_tiles + nt;
  int t = 0;
  for (int row = 0; row < mt; ++row) t += n_tiles - (row * tile_m) / bn;
  return t + nt - (mt * tile_m) / bn;
}

struct ReduceParams {
  const float* partial;
  int splits, num_tiles, n_tiles, tile_m, bn;
  int M, N;
  long long ldo;
  int scale_from;
  float scale;
  int symmetric;
  // pieces made from classes of tokens (cls_sub pieces per class): row i of the output is row
  // i + cls_shift[class] of that piece's tiles; cls_sub == 0 otherwise
  int cls_sub;
  int cls_shift[8];
};

// Sum, in split order, of the partial tiles that hold output elements (i, j .. j + NV - 1).
template <int NV>
__device__ __forceinline__ void sum_pieces(const ReduceParams& r, int i, int j, float (&acc)[NV]) {
  const int nt = j / r.bn;
  const long long tile_elems = static_cast<long long>(r.tile_m) * r.bn;
#pragma unroll
  for (int e = 0; e < NV; ++e) acc[e] = 0.f;
  for (int sp = 0; sp < r.splits; ++sp) {
    const int ii = r.cls_sub > 0 ? i + r.cls_shift[sp / r.cls_sub] : i;
    const int mt = ii / r.tile_m;
    const int t = tile_index(mt, nt, r.n_tiles, r.tile_m, r.bn, r.symmetric);
    const long long off = static_cast<long long>(ii - mt * r.tile_m) * r.bn + (j - nt * r.bn);
    const float* src = r.partial + (static_cast<long long>(sp) * r.num_tiles + t) * tile_elems + off;
    if (NV == 4) {
      const float4 v = *reinterpret_cast<const float4*>(src);
      acc[0] += v.x; acc[1] += v.y; acc[2] += v.z; acc[3] += v.w;
    } else {
      acc[0] += src[0];
    }
  }
}

// Ordered reduction of the partial tiles: out[i][j] = scale_j * (sum over the pieces of the
// tile holding (i, j)), taken in split order, so the result does not depend on timing.  With
// symmetric != 0 only tiles reaching the upper triangle exist and (i, j), i > j, is read from (j, i).
template <typename TOut>
__global__ void __launch_bounds__(256) splitk_reduce_kernel(const ReduceParams r, TOut* __restrict__ out) {
  const long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
  const int ncol4 = (r.N + 3) / 4;
  if (idx >= static_cast<long long>(r.M) * ncol4) return;
  const int i = static_cast<int>(idx / ncol4);
  const int j0 = static_cast<int>(idx % ncol4) * 4;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  if (!r.symmetric || i <= j0) {
    sum_pieces<4>(r, i, j0, acc);
  } else {
    for (int e = 0; e < 4; ++e) {
      const int j = j0 + e;
      if (j >= r.N) break;
      float a[1];
      if (i <= j) sum_pieces<1>(r, i, j, a);
      else sum_pieces<1>(r, j, i, a);
      acc[e] = a[0];
    }
  }
  TOut* dst = out + static_cast<long long>(i) * r.ldo + j0;
  float v[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) v[e] = (j0 + e >= r.scale_from) ? acc[e] * r.scale : acc[e];
  if (j0 + 4 <= r.N && (reinterpret_cast<uintptr_t>(dst) & (4 * sizeof(TOut) - 1)) == 0 &&
      PRAC_IN(static_cast<long long>(i) * r.ldo + j0 + 3, static_cast<long long>(r.M - 1) * r.ldo + r.N)) {
    if constexpr (sizeof(TOut) == 2) {
      const __nv_bfloat162 lo = __floats2bfloat162_rn(v[0], v[1]), hi = __floats2bfloat162_rn(v[2], v[3]);
      uint2 o;
      o.x = *reinterpret_cast<const uint32_t*>(&lo);
      o.y = *reinterpret_cast<const uint32_t*>(&hi);
      *reinterpret_cast<uint2*>(dst) = o;
    } else {
      *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[2], v[3]);
    }
  } else {
    for (int e = 0; e < 4 && j0 + e < r.N; ++e) {
      if (!PRAC_IN(static_cast<long long>(i) * r.ldo + j0 + e, static_cast<long long>(r.M - 1) * r.ldo + r.N)) continue;
      if constexpr (sizeof(TOut) == 2) dst[e] = __float2bfloat16_rn(v[e]);
      else dst[e] = v[e];
    }
  }
}

// The same reduction for a symmetric output, by 32 x 32 blocks (bi <= bj): the block is read
// once from the partial tiles (rows coalesced), written to (bi, bj), and its transpose, through
// shared memory, to (bj, bi).  Diagonal blocks take their upper triangle for both halves, so
// the output is exactly symmetric.  Grid: (block column, block row).
template <typename TOut>
__global__ void __launch_bounds__(256) splitk_reduce_sym_kernel(const ReduceParams r, TOut* __restrict__ out) {
  __shared__ float tile[32][33];
  const int bi = static_cast<int>(blockIdx.y), bj = static_cast<int>(blockIdx.x);
  if (bi > bj) return;                       // the grid is square; pairs below the diagonal have nothing to do
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int mt = (bi * 32) / r.tile_m, nt = (bj * 32) / r.bn;
  const int t = tile_index(mt, nt, r.n_tiles, r.tile_m, r.bn, 1);
  const long long tile_elems = static_cast<long long>(r.tile_m) * r.bn;
  const float* base = r.partial + static_cast<long long>(t) * tile_elems +
                      static_cast<long long>(bi * 32 - mt * r.tile_m) * r.bn + (bj * 32 - nt * r.bn) + tx;
  const long long split_stride = static_cast<long long>(r.num_tiles) * tile_elems;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  for (int sp = 0; sp < r.splits; ++sp) {
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[e] += __ldcs(base + sp * split_stride + static_cast<long long>(ty + 8 * e) * r.bn);
  }
#pragma unroll
  for (int e = 0; e < 4; ++e) tile[ty + 8 * e][tx] = acc[e];
  __syncthreads();
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const int row = ty + 8 * e;
    const int gi = bi * 32 + row, gj = bj * 32 + tx;
    if (gi < r.M && gj < r.N) {
      float v = (bi != bj || row <= tx) ? tile[row][tx] : tile[tx][row];
      if (gj >= r.scale_from) v *= r.scale;
      if constexpr (sizeof(TOut) == 2) out[static_cast<long long>(gi) * r.ldo + gj] = __float2bfloat16_rn(v);
      else out[static_cast<long long>(gi) * r.ldo + gj] = v;
    }
    if (bi != bj) {
      const int ti = bj * 32 + row, tj = bi * 32 + tx;   // transposed block
      if (ti < r.M && tj < r.N) {
        float v = tile[tx][row];
        if (tj >= r.scale_from) v *= r.scale;
        if constexpr (sizeof(TOut) == 2) out[static_cast<long long>(ti) * r.ldo + tj] = __float2bfloat16_rn(v);
        else out[static_cast<long long>(ti) * r.ldo + tj] = v;
      }
    }
  }
}

// The same reduction for the Gram matrix of the fit, which is only ever used as a stack of three
// bf16 pieces (hi + mid + lo = value to about 2^-24; see split3_kernel): 64 x 64 blocks, 16-byte
// loads of the partial tiles, and each block written as the three pieces (and as fp32 where out is
// given) to (bi, bj) and, transposed, to (bj, bi).  The planes are rows_pad x ldp (multiples of
// 64); what lies outside the M x M matrix is written as zero, so no pass over the planes follows.
__device__ __forceinline__ void split3_store4(const float (&x)[4], __nv_bfloat16* p0, long long plane) {
  __align__(8) __nv_bfloat16 hi[4], mid[4], lo[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    float v = x[e];
    hi[e] = __float2bfloat16_rn(v);
    v -= __bfloat162float(hi[e]);
    mid[e] = __float2bfloat16_rn(v);
    v -= __bfloat162float(mid[e]);
    lo[e] = __float2bfloat16_rn(v);
  }
  *reinterpret_cast<uint2*>(p0) = *reinterpret_cast<const uint2*>(hi);
  *reinterpret_cast<uint2*>(p0 + plane) = *reinterpret_cast<const uint2*>(mid);
  *reinterpret_cast<uint2*>(p0 + 2 * plane) = *reinterpret_cast<const uint2*>(lo);
}
__global__ void __launch_bounds__(256) splitk_reduce_sym_split3_kernel(const ReduceParams r, float* __restrict__ out,
                                                                       __nv_bfloat16* __restrict__ planes,
                                                                       long long rows_pad, long long ldp) {
  __shared__ float tile[64][65];
  const int bi = static_cast<int>(blockIdx.y), bj = static_cast<int>(blockIdx.x);
  if (bi > bj) return;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;      // 16 groups of four columns, 16 rows per pass
  const int mt = (bi * 64) / r.tile_m, nt = (bj * 64) / r.bn;
  const long long tile_elems = static_cast<long long>(r.tile_m) * r.bn;
  const long long split_stride = static_cast<long long>(r.num_tiles) * tile_elems;
  // (block pairs beyond the last tile only hold padding)
  const bool inside = bi * 64 < r.M && bj * 64 < r.N;
  if (inside) {
    const int t = tile_index(mt, nt, r.n_tiles, r.tile_m, r.bn, 1);
    const float* base = r.partial + static_cast<long long>(t) * tile_elems +
                        static_cast<long long>(bi * 64 - mt * r.tile_m) * r.bn + (bj * 64 - nt * r.bn) + 4 * tx;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int row = ty + 16 * e;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int sp = 0; sp < r.splits; ++sp) {
        const float4 v = __ldcs(reinterpret_cast<const float4*>(base + sp * split_stride + static_cast<long long>(row) * r.bn));
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
      }
      tile[row][4 * tx] = acc.x; tile[row][4 * tx + 1] = acc.y; tile[row][4 * tx + 2] = acc.z; tile[row][4 * tx + 3] = acc.w;
    }
  }
  __syncthreads();
  const long long plane = rows_pad * ldp;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const int row = ty + 16 * e;
    {
      const int gi = bi * 64 + row, gj = bj * 64 + 4 * tx;
      float x[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int col = 4 * tx + q;
        // diagonal blocks take their upper triangle for both halves: the result is exactly symmetric
        const float v = (bi != bj || row <= col) ? tile[row][col] : tile[col][row];
        x[q] = (inside && gi < r.M && gj + q < r.N) ? v : 0.f;
      }
      if (out != nullptr && gi < r.M) {
#pragma unroll
        for (int q = 0; q < 4; ++q) if (gj + q < r.N) out[static_cast<long long>(gi) * r.ldo + gj + q] = x[q];
      }
      split3_store4(x, planes + static_cast<long long>(gi) * ldp + gj, plane);
    }
    if (bi != bj) {
      const int ti = bj * 64 + row, tj = bi * 64 + 4 * tx;   // transposed block
      float x[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) x[q] = (inside && ti < r.M && tj + q < r.N) ? tile[4 * tx + q][row] : 0.f;
      if (out != nullptr && ti < r.M) {
#pragma unroll
        for (int q = 0; q < 4; ++q) if (tj + q < r.N) out[static_cast<long long>(ti) * r.ldo + tj + q] = x[q];
      }
      split3_store4(x, planes + static_cast<long long>(ti) * ldp + tj, plane);
    }
  }
}

}  // namespace
PRAC_BOUNDS_READER(bounds_violations_tc)
namespace {

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;
std::once_flag g_once;
int g_init_status = PRAC_ECUDA;
DeviceValue g_sm_count;    // SM count of each device this process has used

// The driver entry point is process-wide; everything else below is looked up per device.
void do_init() {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || fn == nullptr) {
    return;
  }
  g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  g_init_status = PRAC_OK;
}

int current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return -1; }
  return dev;
}

// SM count of the current device (0 when there is none).
int num_sms() {
  const int dev = current_device();
  if (dev < 0) return 0;
  int n = g_sm_count.get(dev);
  if (n > 0) return n;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) { cudaGetLastError(); return 0; }
  g_sm_count.set(dev, n);
  return n;
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

// Number of tile owners that can be resident at once: CTAs (one per SM) or CTA pairs.
template <int CTAS, int BN, bool MN, int EPI, bool LDG = false>
int resident_workers() {
  using C = Cfg<CTAS, BN, EPI>;
  const int sms = num_sms();
  if (CTAS == 1) return sms;
  static DeviceValue cached;  // per instantiation and device
  const int dev = current_device();
  if (cached.get(dev) > 0) return cached.get(dev);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(sms / 2 * 2));
  cfg.blockDim = dim3(LDG ? NUM_THREADS_LDG : NUM_THREADS);
  cfg.dynamicSmemBytes = C::SMEM_BYTES;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, gemm_tc_kernel<CTAS, BN, MN, EPI, LDG>, &cfg) != cudaSuccess || n < 1) {
    cudaGetLastError();
    n = sms / 2;
  }
  if (n > sms / 2) n = sms / 2;
  cached.set(dev, n);
  return n;
}

// Output matrix (rows x cols, leading dimension ld, 2- or 4-byte elements) as 32-row boxes of
// 128 bytes, 128-byte swizzle.  Returns PRAC_EALIGN when its rows are not 16-byte aligned.
int make_out_map(CUtensorMap* map, void* base, int64_t cols, int64_t rows, int64_t ld, int elem_bytes) {
  if (!aligned16(base) || (ld * elem_bytes) % 16 != 0) return PRAC_EALIGN;
  cuuint64_t gdim[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  cuuint64_t gstr[1] = {static_cast<cuuint64_t>(ld) * elem_bytes};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(128 / elem_bytes), 32u};
  cuuint32_t estr[2] = {1u, 1u};
  CUresult r = g_encode(map, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                        base, gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? PRAC_OK : PRAC_ECUDA;
}

template <int CTAS, int BN, bool MN, int EPI, bool LDG = false>
int launch(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& tc, const TcParams& p_in,
           cudaStream_t stream, const CUtensorMap* tb2 = nullptr, const CUtensorMap* tc2 = nullptr) {
  TcParams p = p_in;
  if (tb2 == nullptr) { p.n_tiles1 = p.n_tiles; tb2 = &tb; tc2 = &tc; }
  using C = Cfg<CTAS, BN, EPI>;
  auto kern = gemm_tc_kernel<CTAS, BN, MN, EPI, LDG>;
  constexpr int THREADS = LDG ? NUM_THREADS_LDG : NUM_THREADS;
  static DeviceOnce attr_set;  // per instantiation; the attribute belongs to the current device
  const int dev = current_device();
  if (!attr_set.done(dev)) {
    PRAC_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
    attr_set.mark(dev);
  }
  const int items = p.num_tiles * p.splits;
  const int cap = resident_workers<CTAS, BN, MN, EPI, LDG>();
  const int workers = items < cap ? items : cap;
  if (CTAS == 1) {
    kern<<<workers, THREADS, C::SMEM_BYTES, stream>>>(ta, tb, tc, *tb2, *tc2, p);
  } else {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(2 * workers));
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = C::SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    PRAC_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, ta, tb, tc, *tb2, *tc2, p));
  }
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

// Tile shape for an output of M x N: CTA pairs with 256 x 256 tiles when the output is wide
// and tall enough to fill them, otherwise single CTAs with 128 x {64, 128, 256}.
struct Shape { int ctas, bn; };
Shape pick_shape(int64_t M, int64_t N) {
  if (N > 128 && M > 128) return {2, 256};
  return {1, N > 128 ? 256 : (N > 64 ? 128 : 64)};
}

// A bf16-out K-major product on CTA pairs whose output is 257 to 512 columns wide and whose K is
// long takes one 512-wide tile per 256 rows: every row of A is then fetched by exactly one CTA pair
// and serves two MMAs.  Measured (32768 rows, 512 columns): K = 5461 146.6 -> 140.6 us, K = 4096
// 107.2 -> 103.3 us, K = 2048 57.4 -> 58.3 us; on wider outputs, where neighbouring pairs share A's
// rows through L2 anyway, the single accumulator's drain costs more than the shared stage saves.
constexpr int64_t WIDE_MIN_K = 3072;
bool wide_tiles(int64_t M, int64_t N, int64_t K) {
  return pick_shape(M, N).ctas == 2 && N > 256 && N <= 512 && K >= WIDE_MIN_K;
}

int count_tiles(int m_tiles, int n_tiles, int tile_m, int bn, int symmetric) {
  if (!symmetric) return m_tiles * n_tiles;
  int cnt = 0;
  for (int mt = 0; mt < m_tiles; ++mt) {
    const int first = (mt * tile_m) / bn;
    if (first < n_tiles) cnt += n_tiles - first;
  }
  return cnt;
}

template <int BN>
int launch_rowclass(const ClassMaps& cm, const CUtensorMap& tb, const TcParams& p, cudaStream_t stream) {
  using C = Cfg<2, BN, EPI_BF16>;
  static DeviceOnce attr_set;
  const int dev = current_device();
  if (!attr_set.done(dev)) {
    PRAC_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_rowclass_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
    attr_set.mark(dev);
  }
  const int cap = resident_workers<2, BN, false, EPI_BF16>();   // same footprint as the plain K-major kernel
  const int workers = p.num_tiles < cap ? p.num_tiles : cap;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(2 * workers));
  cfg.blockDim = dim3(NUM_THREADS);
  cfg.dynamicSmemBytes = C::SMEM_BYTES;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  PRAC_CUDA_TRY(cudaLaunchKernelEx(&cfg, gemm_tc_rowclass_kernel<BN>, cm, tb, p));
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

}  // namespace

int tc_init() {
  std::call_once(g_once, do_init);
  return g_init_status;
}
// The plain-load A path exists for the CTA-pair kernels only (outputs taller and wider than 128).
bool tc_kmajor_takes_unaligned_a(int64_t M, int64_t N) { return pick_shape(M, N).ctas == 2; }
bool tc_tokens_takes_unaligned_a(int64_t M, int64_t N) { return pick_shape(M, N).ctas == 2; }
int tc_num_sms() { return num_sms(); }

int tc_gemm_kmajor(const __nv_bfloat16* A, int64_t lda, const __nv_bfloat16* B, int64_t ldb,
                   int64_t M, int64_t N, int64_t K, void* Cout, int64_t ldc, int type_c,
                   int accumulate, int* dev_status, cudaStream_t stream, const TcSegments* segs) {
  if (tc_init() != PRAC_OK) return PRAC_ECUDA;
  if (M <= 0 || N <= 0 || K <= 0) return PRAC_EINVAL;
  const int nseg = segs ? segs->n : 1;
  if (nseg < 1 || nseg > MAX_SEG) return PRAC_EINVAL;
  if (segs && (K % BK != 0 || segs->rows_a < K || segs->rows_b < K)) return PRAC_EINVAL;
  if (!aligned16(B) || (ldb % 8)) return PRAC_EALIGN;
  if (type_c != ET_BF16 && type_c != ET_F32) return PRAC_EINVAL;
  if (type_c == ET_BF16 && accumulate) return PRAC_EINVAL;
  Shape sh = pick_shape(M, N);
  const int tile_m = sh.ctas * BM;
  // A with rows off the 16-byte grid is fetched with plain loads (CTA-pair kernel, bf16 output)
  const bool a_ldg = !aligned16(A) || (lda % 8) != 0;
  if (a_ldg && !(tc_kmajor_takes_unaligned_a(M, N) && segs == nullptr && type_c == ET_BF16)) return PRAC_EALIGN;
  const bool wide = !a_ldg && type_c == ET_BF16 && wide_tiles(M, N, K);
  CUtensorMap ta, tb;
  // with segments the operands are rows of several K-long pieces side by side (rows_a, rows_b wide)
  // (a wide tile still fetches B in boxes of 128 rows: each CTA's share of one 256-column half)
  if (make_map(&tb, B, segs ? segs->rows_b : K, N, ldb, sh.bn / sh.ctas) != PRAC_OK) return PRAC_ECUDA;
  if (wide) sh.bn = 512;
  if (a_ldg) ta = tb;   // placeholder, never used
  else if (make_map(&ta, A, segs ? segs->rows_a : K, M, lda, BM) != PRAC_OK) return PRAC_ECUDA;
  TcParams p{};
  p.M = static_cast<int>(M); p.N = static_cast<int>(N); p.K = static_cast<int>(K);
  const int m_tiles = static_cast<int>((M + tile_m - 1) / tile_m);
  p.n_tiles = static_cast<int>((N + sh.bn - 1) / sh.bn);
  p.num_tiles = m_tiles * p.n_tiles;
  p.kb_per_seg = static_cast<int>((K + BK - 1) / BK);
  p.kblocks = p.kb_per_seg * nseg;
  p.splits = 1;
  for (int g = 0; g < nseg; ++g) {
    p.seg_a[g] = segs ? static_cast<int>(segs->off_a[g]) : 0;
    p.seg_b[g] = segs ? static_cast<int>(segs->off_b[g]) : 0;
  }
  p.symmetric = 0;
  p.C = Cout; p.ldc = ldc; p.accumulate = accumulate;
  p.dev_status = dev_status;
  CUtensorMap tc = ta;   // placeholder when the output cannot take tile stores
  const int out_st = make_out_map(&tc, Cout, N, M, ldc, type_c == ET_BF16 ? 2 : 4);
  if (out_st == PRAC_ECUDA) return PRAC_ECUDA;
  p.tma_store = (out_st == PRAC_OK) ? 1 : 0;
  if (out_st != PRAC_OK) tc = ta;
  if (a_ldg) {
    p.a_ptr = A; p.a_ld = lda; p.a_rows = p.M; p.a_cols = p.K;
    return launch<2, 256, false, EPI_BF16, true>(ta, tb, tc, p, stream);
  }
  if (type_c == ET_BF16) {
    if (wide) return launch<2, 512, false, EPI_BF16>(ta, tb, tc, p, stream);
    if (sh.ctas == 2) return launch<2, 256, false, EPI_BF16>(ta, tb, tc, p, stream);
    if (sh.bn == 256) return launch<1, 256, false, EPI_BF16>(ta, tb, tc, p, stream);
    if (sh.bn == 128) return launch<1, 128, false, EPI_BF16>(ta, tb, tc, p, stream);
    return launch<1, 64, false, EPI_BF16>(ta, tb, tc, p, stream);
  }
  if (sh.ctas == 2) return launch<2, 256, false, EPI_F32>(ta, tb, tc, p, stream);
  if (sh.bn == 256) return launch<1, 256, false, EPI_F32>(ta, tb, tc, p, stream);
  if (sh.bn == 128) return launch<1, 128, false, EPI_F32>(ta, tb, tc, p, stream);
  return launch<1, 64, false, EPI_F32>(ta, tb, tc, p, stream);
}

// C (M x N, bf16) = A (M x K, K-major, row pitch lda not a multiple of 8 elements) * Bmn (K x N,
// row-major) on the row-class kernel (see ClassMaps).  PRAC_EALIGN when the shape or the other
// operands do not fit it; the caller then takes another path.
bool tc_rowclass_fits(const void* A, int64_t lda, int64_t M, int64_t N) {
  return aligned16(A) && (lda % 8) != 0 && pick_shape(M, N).ctas == 2;
}
int tc_gemm_kmajor_rowclass(const __nv_bfloat16* A, int64_t lda, const __nv_bfloat16* Bmn, int64_t ldb,
                            int64_t M, int64_t N, int64_t K, __nv_bfloat16* Cout, int64_t ldc,
                            int* dev_status, cudaStream_t stream) {
  if (tc_init() != PRAC_OK) return PRAC_ECUDA;
  if (M <= 0 || N <= 0 || K <= 0 || lda < K) return PRAC_EINVAL;
  if (!tc_rowclass_fits(A, lda, M, N) || !aligned16(Bmn) || (ldb % 8) || !aligned16(Cout) || (ldc % 8)) return PRAC_EALIGN;
  int g = 8;                                   // gcd(lda, 8)
  while (lda % g) g >>= 1;
  const int P = 8 / g;                         // 2, 4 or 8 classes
  const bool wide = wide_tiles(M, N, K);
  const int BN2 = wide ? 512 : 256;
  const int tile_m = 2 * BM;
  ClassMaps cm;
  TcParams p{};
  int max_shift = 0;
  for (int j = 0; j < 8; ++j) {
    const int jj = j < P ? j : 0;              // unused slots repeat class 0
    const int shift = static_cast<int>((jj * lda) % 8);
    const int64_t rows = (M - jj + P - 1) / P;
    if (j < P) { p.cls_shift[j] = shift; if (shift > max_shift) max_shift = shift; }
    {
      cuuint64_t gdim[2] = {static_cast<cuuint64_t>(K + shift), static_cast<cuuint64_t>(rows > 0 ? rows : 1)};
      cuuint64_t gstr[1] = {static_cast<cuuint64_t>(P) * lda * 2};
      cuuint32_t box[2] = {64u, static_cast<cuuint32_t>(BM)};
      cuuint32_t estr[2] = {1u, 1u};
      if (g_encode(&cm.a[j], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<__nv_bfloat16*>(A + jj * lda - shift), gdim,
                   gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return PRAC_ECUDA;
    }
    {
      cuuint64_t gdim[2] = {static_cast<cuuint64_t>(N), static_cast<cuuint64_t>(rows > 0 ? rows : 1)};
      cuuint64_t gstr[1] = {static_cast<cuuint64_t>(P) * ldc * 2};
      cuuint32_t box[2] = {64u, 32u};
      cuuint32_t estr[2] = {1u, 1u};
      if (g_encode(&cm.c[j], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Cout + jj * ldc, gdim, gstr, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return PRAC_ECUDA;
    }
  }
  CUtensorMap tb;                              // rows = K, inner = N, boxes of 64 x 64
  if (make_map(&tb, Bmn, N, K, ldb, 64) != PRAC_OK) return PRAC_ECUDA;
  p.M = static_cast<int>(M); p.N = static_cast<int>(N); p.K = static_cast<int>(K);
  p.cls_count = P;
  const int64_t rows0 = (M + P - 1) / P;       // the largest class
  const int tiles_per_class = static_cast<int>((rows0 + tile_m - 1) / tile_m);
  p.n_tiles = static_cast<int>((N + BN2 - 1) / BN2);
  p.n_tiles1 = p.n_tiles;
  p.num_tiles = tiles_per_class * P * p.n_tiles;
  p.kb_per_seg = static_cast<int>((K + max_shift + BK - 1) / BK);
  p.kblocks = p.kb_per_seg;
  p.splits = 1;
  p.C = Cout; p.ldc = ldc; p.tma_store = 1;
  p.dev_status = dev_status;
  return wide ? launch_rowclass<512>(cm, tb, p, stream) : launch_rowclass<256>(cm, tb, p, stream);
}

// [C1 | C2] = A [B1 ; B2]^T in one launch: A (M x K) is streamed once for both products.
// All operands bf16 K-major, both outputs bf16.  Column tiles are dealt so that one worker
// round covers neighbouring tiles of the same rows of A.
int tc_gemm_kmajor_dual(const __nv_bfloat16* A, int64_t lda, int64_t M, int64_t K,
                        const __nv_bfloat16* B1, int64_t ldb1, int64_t N1, __nv_bfloat16* C1, int64_t ldc1,
                        const __nv_bfloat16* B2, int64_t ldb2, int64_t N2, __nv_bfloat16* C2, int64_t ldc2,
                        int* dev_status, cudaStream_t stream) {
  if (tc_init() != PRAC_OK) return PRAC_ECUDA;
  if (M <= 0 || N1 <= 0 || N2 <= 0 || K <= 0) return PRAC_EINVAL;
  if (!aligned16(B1) || !aligned16(B2) || (ldb1 % 8) || (ldb2 % 8)) return PRAC_EALIGN;
  const bool a_ldg = !aligned16(A) || (lda % 8) != 0;     // A off the 16-byte grid: plain loads
  constexpr int BN2 = 256;
  const int tile_m = 2 * BM;
  CUtensorMap ta, tb1, tb2;
  if (make_map(&tb1, B1, K, N1, ldb1, BN2 / 2) != PRAC_OK) return PRAC_ECUDA;
  if (make_map(&tb2, B2, K, N2, ldb2, BN2 / 2) != PRAC_OK) return PRAC_ECUDA;
  if (a_ldg) ta = tb1;
  else if (make_map(&ta, A, K, M, lda, BM) != PRAC_OK) return PRAC_ECUDA;
  TcParams p{};
  p.M = static_cast<int>(M); p.N = static_cast<int>(N1); p.K = static_cast<int>(K);
  const int m_tiles = static_cast<int>((M + tile_m - 1) / tile_m);
  p.n_tiles1 = static_cast<int>((N1 + BN2 - 1) / BN2);
  p.n_tiles = p.n_tiles1 + static_cast<int>((N2 + BN2 - 1) / BN2);
  p.num_tiles = m_tiles * p.n_tiles;
  p.kblocks = static_cast<int>((K + BK - 1) / BK);
  p.splits = 1;
  p.kb_per_seg = p.kblocks;
  p.symmetric = 0;
  p.C = C1; p.ldc = ldc1; p.accumulate = 0;
  p.N2 = static_cast<int>(N2); p.C2 = C2; p.ldc2 = ldc2;
  p.dev_status = dev_status;
  CUtensorMap tc1 = ta, tc2 = ta;   // placeholders when an output cannot take tile stores
  const int st1 = make_out_map(&tc1, C1, N1, M, ldc1, 2);
  const int st2 = make_out_map(&tc2, C2, N2, M, ldc2, 2);
  if (st1 == PRAC_ECUDA || st2 == PRAC_ECUDA) return PRAC_ECUDA;
  // Both outputs must leave the same way (tile stores, or the transpose path): the two paths
  // share a shared-memory region, and a tile store of one output still in flight must never
  // meet a transpose tile of the other.  The caller runs the two products in turn otherwise.
  if ((st1 == PRAC_OK) != (st2 == PRAC_OK)) return PRAC_EALIGN;
  p.tma_store = (st1 == PRAC_OK) ? 1 : 0;
  p.tma_store2 = (st2 == PRAC_OK) ? 1 : 0;
  if (st1 != PRAC_OK) tc1 = ta;
  if (st2 != PRAC_OK) tc2 = ta;
  if (a_ldg) {
    p.a_ptr = A; p.a_ld = lda; p.a_rows = p.M; p.a_cols = p.K;
    return launch<2, 256, false, EPI_BF16, true>(ta, tb1, tc1, p, stream, &tb2, &tc2);
  }
  return launch<2, 256, false, EPI_BF16>(ta, tb1, tc1, p, stream, &tb2, &tc2);
}

namespace {
// Whether the fused consumers can take dY (and dX, when there is one) with these row pitches by
// classes of rows: bases on the 16-byte grid, the same offsets in both, every class equally long.
bool consumer_classes_fit(const void* dY, int64_t lddy, const void* dX, int64_t lddx, int64_t M, int64_t N) {
  if ((lddy % 8) == 0 || !aligned16(dY) || M <= 128 || N <= 128) return false;
  if (dX != nullptr && (!aligned16(dX) || (lddx % 8) != (lddy % 8))) return false;
  int g = 8;
  while (lddy % g) g >>= 1;
  return M % (8 / g) == 0;
}
// Tensor maps, tile counts and class fields of such a launch (p.M, p.N, p.K set by the caller).
int consumer_class_setup(const __nv_bfloat16* A, int64_t lda, const __nv_bfloat16* dY, int64_t lddy, __nv_bfloat16* dX,
                         int64_t lddx, ConsumerClassMaps* cm, TcParams* p) {
  int g = 8;
  while (lddy % g) g >>= 1;
  const int P = 8 / g;
  const int64_t rows = p->M / P;
  int max_shift = 0;
  for (int j = 0; j < 8; ++j) {
    const int jj = j < P ? j : 0;
    const int shift = static_cast<int>((jj * lddy) % 8);
    if (j < P) { p->cls_shift[j] = shift; if (shift > max_shift) max_shift = shift; }
    cuuint32_t estr[2] = {1u, 1u};
    cuuint64_t gdim_io[2] = {static_cast<cuuint64_t>(p->N + shift), static_cast<cuuint64_t>(rows)};
    cuuint32_t box_io[2] = {64u, 32u};
    cuuint64_t gstr_y[1] = {static_cast<cuuint64_t>(P) * lddy * 2};
    if (g_encode(&cm->io.a[j], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<__nv_bfloat16*>(dY + jj * lddy - shift), gdim_io,
                 gstr_y, box_io, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                 CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return PRAC_ECUDA;
    if (dX != nullptr) {
      cuuint64_t gstr_x[1] = {static_cast<cuuint64_t>(P) * lddx * 2};
      if (g_encode(&cm->io.c[j], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, dX + jj * lddx - shift, gdim_io, gstr_x, box_io, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return PRAC_ECUDA;
    } else {
      cm->io.c[j] = cm->io.a[j];
    }
    cuuint64_t gdim_z[2] = {static_cast<cuuint64_t>(p->K), static_cast<cuuint64_t>(rows)};
    cuuint64_t gstr_z[1] = {static_cast<cuuint64_t>(P) * lda * 2};
    cuuint32_t box_z[2] = {64u, static_cast<cuuint32_t>(BM)};
    if (g_encode(&cm->z[j], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<__nv_bfloat16*>(A + jj * lda), gdim_z, gstr_z,
                 box_z, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                 CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return PRAC_ECUDA;
  }
  p->cls_count = P;
  const int tiles_per_class = static_cast<int>((rows + 2 * BM - 1) / (2 * BM));
  p->n_tiles = static_cast<int>((p->N + max_shift + 255) / 256);
  p->n_tiles1 = p->n_tiles;
  p->num_tiles = tiles_per_class * P * p->n_tiles;
  p->tma_store = 1;
  return PRAC_OK;
}
template <int EPI>
int launch_consumer_classes(const ConsumerClassMaps& cm, const CUtensorMap& tb, const TcParams& p, cudaStream_t stream) {
  using C = Cfg<2, 256, EPI>;
  auto kern = gemm_tc_consumer_rowclass_kernel<EPI>;
  static DeviceOnce attr_set;
  const int dev = current_device();
  if (!attr_set.done(dev)) {
    PRAC_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
    attr_set.mark(dev);
  }
  const int cap = resident_workers<2, 256, false, EPI>();      // same footprint as the aligned launch
  const int workers = p.num_tiles < cap ? p.num_tiles : cap;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(2 * workers));
  cfg.blockDim = dim3(NUM_THREADS);
  cfg.dynamicSmemBytes = C::SMEM_BYTES;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  PRAC_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, cm, tb, p));
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}
}  // namespace
bool tc_consumer_takes_rows(const void* dY, int64_t lddy, const void* dX, int64_t lddx, int64_t M, int64_t N) {
  return (aligned16(dY) && lddy % 8 == 0) || consumer_classes_fit(dY, lddy, dX, lddx, M, N);
}
int64_t tc_gemm_kmajor_rms_blocks(int64_t M, int64_t lddy) {
  int g = 8;
  while (lddy % g) g >>= 1;
  const int64_t P = 8 / g;
  return (P > 1 && M % P == 0) ? P * ((M / P + 31) / 32) : (M + 31) / 32;
}

int tc_gemm_kmajor_act(const __nv_bfloat16* A, int64_t lda, const __nv_bfloat16* B, int64_t ldb,
                       int64_t M, int64_t N, int64_t K, const __nv_bfloat16* dY, int64_t lddy, int act,
                       __nv_bfloat16* dX, int64_t lddx, int* dev_status, cudaStream_t stream) {
  if (tc_init() != PRAC_OK) return PRAC_ECUDA;
  if (M <= 0 || N <= 0 || K <= 0) return PRAC_EINVAL;
  if (act != ACT_SILU && act != ACT_GELU) return PRAC_EINVAL;
  if (!aligned16(A) || !aligned16(B) || (lda % 8) || (ldb % 8)) return PRAC_EALIGN;
  if ((lddy % 8) != 0 || (lddx % 8) != 0) {
    // dY and dX with rows off the 16-byte grid (contiguous matrices of odd width): by classes of rows
    if (!consumer_classes_fit(dY, lddy, dX, lddx, M, N)) return PRAC_EALIGN;
    ConsumerClassMaps cm;
    CUtensorMap tbc;
    if (make_map(&tbc, B, K, N, ldb, 128) != PRAC_OK) return PRAC_ECUDA;
    TcParams pc{};
    pc.M = static_cast<int>(M); pc.N = static_cast<int>(N); pc.K = static_cast<int>(K);
    const int sc = consumer_class_setup(A, lda, dY, lddy, dX, lddx, &cm, &pc);
    if (sc != PRAC_OK) return sc;
    pc.kblocks = static_cast<int>((K + BK - 1) / BK);
    pc.splits = 1;
    pc.kb_per_seg = pc.kblocks;
    pc.C = dX; pc.ldc = lddx;
    pc.aux = dY; pc.ld_aux = lddy;
    pc.dev_status = dev_status;
    return act == ACT_SILU ? launch_consumer_classes<EPI_SILU>(cm, tbc, pc, stream)
                           : launch_consumer_classes<EPI_GELU>(cm, tbc, pc, stream);
  }
  if (!aligned16(dY)) return PRAC_EALIGN;
  const Shape sh = pick_shape(M, N);
  const int tile_m = sh.ctas * BM;
  CUtensorMap ta, tb;
  if (make_map(&ta, A, K, M, lda, BM) != PRAC_OK) return PRAC_ECUDA;
  if (make_map(&tb, B, K, N, ldb, sh.bn / sh.ctas) != PRAC_OK) return PRAC_ECUDA;
  TcParams p{};
  p.M = static_cast<int>(M); p.N = static_cast<int>(N); p.K = static_cast<int>(K);
  const int m_tiles = static_cast<int>((M + tile_m - 1) / tile_m);
  p.n_tiles = static_cast<int>((N + sh.bn - 1) / sh.bn);
  p.num_tiles = m_tiles * p.n_tiles;
  p.kblocks = static_cast<int>((K + BK - 1) / BK);
  p.splits = 1;
  p.kb_per_seg = p.kblocks;
  p.C = dX; p.ldc = lddx;
  p.aux = dY; p.ld_aux = lddy;
  if (act != ACT_SILU && act != ACT_GELU) return PRAC_EINVAL;
  p.dev_status = dev_status;
  CUtensorMap tc = ta;   // placeholder when the output cannot take tile stores
  const int out_st = make_out_map(&tc, dX, N, M, lddx, 2);
  if (out_st == PRAC_ECUDA) return PRAC_ECUDA;
  p.tma_store = (out_st == PRAC_OK) ? 1 : 0;
  if (out_st != PRAC_OK) tc = ta;
  // the factor arrives in the epilogue by tile loads of 32 rows x 64 columns (tensor map in the slot
  // of the second output, which these launches do not have)
  CUtensorMap taux;
  if (make_out_map(&taux, const_cast<__nv_bfloat16*>(dY), N, M, lddy, 2) != PRAC_OK) return PRAC_ECUDA;
  p.n_tiles1 = p.n_tiles;
  if (act == ACT_SILU) {
    if (sh.ctas == 2) return launch<2, 256, false, EPI_SILU>(ta, tb, tc, p, stream, &tb, &taux);
    if (sh.bn == 256) return launch<1, 256, false, EPI_SILU>(ta, tb, tc, p, stream, &tb, &taux);
    if (sh.bn == 128) return launch<1, 128, false, EPI_SILU>(ta, tb, tc, p, stream, &tb, &taux);
    return launch<1, 64, false, EPI_SILU>(ta, tb, tc, p, stream, &tb, &taux);
  }
  if (sh.ctas == 2) return launch<2, 256, false, EPI_GELU>(ta, tb, tc, p, stream, &tb, &taux);
  if (sh.bn == 256) return launch<1, 256, false, EPI_GELU>(ta, tb, tc, p, stream, &tb, &taux);
  if (sh.bn == 128) return launch<1, 128, false, EPI_GELU>(ta, tb, tc, p, stream, &tb, &taux);
  return launch<1, 64, false, EPI_GELU>(ta, tb, tc, p, stream, &tb, &taux);
}

// The two passes of the RMSNorm backward over x = A B^T (never stored), see TcParams.  pass 1:
// row_part ((2 * n_tiles) x M) and col_part (ceil(M / 32) x N) are written, dX is not touched.
// pass 2: dX (bf16) = row_a[t] col_g[i] dY[t][i] - row_b[t] x[t][i].  CTA pairs only (M, N > 128).
int tc_gemm_kmajor_rms(int pass, const __nv_bfloat16* A, int64_t lda, const __nv_bfloat16* B, int64_t ldb,
                       int64_t M, int64_t N, int64_t K, const __nv_bfloat16* dY, int64_t lddy,
                       const float* row_a, const float* row_b, const float* col_g, float* row_part, float* col_part,
                       __nv_bfloat16* dX, int64_t lddx, int* dev_status, cudaStream_t stream,
                       float* row_part2, const float* row_c) {
  if (tc_init() != PRAC_OK) return PRAC_ECUDA;
  if (M <= 128 || N <= 128 || K <= 0 || (pass != 1 && pass != 2)) return PRAC_EINVAL;
  if (!aligned16(A) || !aligned16(B) || (lda % 8) || (ldb % 8)) return PRAC_EALIGN;
  if ((lddy % 8) != 0 || (pass == 2 && (lddx % 8) != 0)) {
    // dY (and dX) with rows off the 16-byte grid: by classes of rows
    if (!consumer_classes_fit(dY, lddy, pass == 2 ? dX : nullptr, lddx, M, N)) return PRAC_EALIGN;
    ConsumerClassMaps cm;
    CUtensorMap tbc;
    if (make_map(&tbc, B, K, N, ldb, 128) != PRAC_OK) return PRAC_ECUDA;
    TcParams pc{};
    pc.M = static_cast<int>(M); pc.N = static_cast<int>(N); pc.K = static_cast<int>(K);
    const int sc = consumer_class_setup(A, lda, dY, lddy, pass == 2 ? dX : nullptr, lddx, &cm, &pc);
    if (sc != PRAC_OK) return sc;
    pc.kblocks = static_cast<int>((K + BK - 1) / BK);
    pc.splits = 1;
    pc.kb_per_seg = pc.kblocks;
    pc.C = dX; pc.ldc = lddx;
    pc.aux = dY; pc.ld_aux = lddy;
    pc.row_a = row_a; pc.row_b = row_b; pc.col_g = col_g; pc.row_part = row_part; pc.col_part = col_part;
    pc.row_part2 = row_part2; pc.row_c = row_c;
    pc.dev_status = dev_status;
    return pass == 1 ? launch_consumer_classes<EPI_RMS1>(cm, tbc, pc, stream)
                     : launch_consumer_classes<EPI_RMS2>(cm, tbc, pc, stream);
  }
  if (!aligned16(dY)) return PRAC_EALIGN;
  constexpr int BN2 = 256;
  const int tile_m = 2 * BM;
  CUtensorMap ta, tb;
  if (make_map(&ta, A, K, M, lda, BM) != PRAC_OK) return PRAC_ECUDA;
  if (make_map(&tb, B, K, N, ldb, BN2 / 2) != PRAC_OK) return PRAC_ECUDA;
  TcParams p{};
  p.M = static_cast<int>(M); p.N = static_cast<int>(N); p.K = static_cast<int>(K);
  const int m_tiles = static_cast<int>((M + tile_m - 1) / tile_m);
  p.n_tiles = static_cast<int>((N + BN2 - 1) / BN2);
  p.num_tiles = m_tiles * p.n_tiles;
  p.kblocks = static_cast<int>((K + BK - 1) / BK);
  p.splits = 1;
  p.kb_per_seg = p.kblocks;
  p.C = dX; p.ldc = lddx;
  p.aux = dY; p.ld_aux = lddy;
  p.row_a = row_a; p.row_b = row_b; p.col_g = col_g; p.row_part = row_part; p.col_part = col_part;
  p.col_g_vec = aligned16(col_g) ? 1 : 0;
  p.row_part2 = row_part2; p.row_c = row_c;
  p.dev_status = dev_status;
  CUtensorMap tc = ta;
  CUtensorMap taux;   // dY arrives in the epilogue by tile loads (slot of the second output's map)
  if (make_out_map(&taux, const_cast<__nv_bfloat16*>(dY), N, M, lddy, 2) != PRAC_OK) return PRAC_ECUDA;
  p.n_tiles1 = p.n_tiles;
  if (pass == 1) return launch<2, 256, false, EPI_RMS1>(ta, tb, tc, p, stream, &tb, &taux);
  const int out_st = make_out_map(&tc, dX, N, M, lddx, 2);
  if (out_st == PRAC_ECUDA) return PRAC_ECUDA;
  p.tma_store = (out_st == PRAC_OK) ? 1 : 0;
  if (out_st != PRAC_OK) tc = ta;
  return launch<2, 256, false, EPI_RMS2>(ta, tb, tc, p, stream, &tb, &taux);
}
// Row partials pass 1 writes: two per column tile; by classes the columns run up to N + the largest offset.
int tc_gemm_kmajor_rms_parts(int64_t N, int64_t lddy) {
  int g = 8;
  while (lddy % g) g >>= 1;
  int max_shift = 0;
  for (int j = 0; j < 8 / g; ++j) { const int sft = static_cast<int>((j * lddy) % 8); if (sft > max_shift) max_shift = sft; }
  return 2 * static_cast<int>((N + max_shift + 255) / 256);
}

namespace {
// Plan of the token-reduction GEMM: tile shape and the number of equal K pieces per tile.
// Cost model in units of one k-block of one tile: rounds * (k-blocks per piece + fill and
// drain) + writing and re-reading one more set of fp32 partial tiles (mostly through L2).
struct TokensPlan {
  int ctas, bn, tile_m, m_tiles, n_tiles, num_tiles, kblocks, splits;
  bool ok;
  size_t ws_bytes;
};
TokensPlan plan_tokens(int64_t M, int64_t N, int64_t K, int symmetric) {   // K: whole chain
  TokensPlan t{};
  const Shape sh = pick_shape(M, N);
  t.ctas = sh.ctas;
  t.bn = sh.bn;
  t.tile_m = sh.ctas * BM;
  t.m_tiles = static_cast<int>((M + t.tile_m - 1) / t.tile_m);
  t.n_tiles = static_cast<int>((N + t.bn - 1) / t.bn);
  t.num_tiles = count_tiles(t.m_tiles, t.n_tiles, t.tile_m, t.bn, symmetric);
  t.kblocks = static_cast<int>((K + BK - 1) / BK);
  const int here = num_sms();
  const int sms = here > 0 ? here : 148;
  const int workers = sms / t.ctas > 0 ? sms / t.ctas : 1;
  // one k-block of a tile: BK/16 MMAs at 8192 flop per clock per SM, about 1.9 GHz
  const double kblock_us = 2.0 * BM * t.bn * BK / 8192.0 / 1900.0;
  const double tile_bytes = static_cast<double>(t.tile_m) * t.bn * 4.0;
  const double extra_per_split = (t.num_tiles * tile_bytes * 2.0 / 8.0e6) / kblock_us;  // 8 TB/s
  const int max_s = t.kblocks / 16 > 0 ? (t.kblocks / 16 < 64 ? t.kblocks / 16 : 64) : 1;
  double best_cost = 1e300;
  t.splits = 1;
  for (int s = 1; s <= max_s; ++s) {
    const long long items = static_cast<long long>(t.num_tiles) * s;
    const long long rounds = (items + workers - 1) / workers;
    const double cost = rounds * ((t.kblocks + s - 1) / s + 8.0) + s * extra_per_split;
    if (cost < best_cost - 1e-9) { best_cost = cost; t.splits = s; }
  }
  t.ok = static_cast<long long>(t.num_tiles) * t.splits < (1ll << 30);
  t.ws_bytes = static_cast<size_t>(t.splits) * t.num_tiles * t.tile_m * t.bn * sizeof(float);
  return t;
}
}  // namespace

// The same product with the K tokens taken by classes of rows of A (row pitch lda off the 16-byte
// grid): P classes, each cut into `sub` pieces; tiles cover M plus the largest class offset.
struct TokenClassPlan {
  int P, sub, max_shift, kblocks;
  int shift[8];
  TokensPlan t;
  bool ok;
  size_t ws_bytes;
};
TokenClassPlan plan_token_classes(int64_t lda, int64_t M, int64_t N, int64_t K) {
  TokenClassPlan c{};
  int g = 8;
  while (lda % g) g >>= 1;
  c.P = 8 / g;
  for (int j = 0; j < c.P; ++j) {
    c.shift[j] = static_cast<int>((j * lda) % 8);
    if (c.shift[j] > c.max_shift) c.max_shift = c.shift[j];
  }
  c.t = plan_tokens(M + c.max_shift, N, K, 0);
  c.sub = (c.t.splits + c.P - 1) / c.P;
  const int64_t rows0 = (K + c.P - 1) / c.P;
  c.kblocks = static_cast<int>((rows0 + BK - 1) / BK);
  if (c.sub > c.kblocks) c.sub = c.kblocks;
  c.ok = c.t.ok && c.P > 1 && c.t.ctas == 2 && c.t.bn == 256;
  c.ws_bytes = static_cast<size_t>(c.P) * c.sub * c.t.num_tiles * c.t.tile_m * c.t.bn * sizeof(float);
  return c;
}
size_t tc_gemm_tokens_rowclass_ws_bytes(int64_t lda, int64_t M, int64_t N, int64_t K) {
  if (M <= 0 || N <= 0 || K <= 0 || lda % 8 == 0) return 0;
  const TokenClassPlan c = plan_token_classes(lda, M, N, K);
  return c.ok ? c.ws_bytes : 0;
}

size_t tc_gemm_tokens_ws_bytes(int64_t M, int64_t N, int64_t K, int symmetric, int nseg) {
  tc_init();  // without a device the planner assumes 148 SMs
  if (M <= 0 || N <= 0 || K <= 0 || nseg < 1) return 0;
  return plan_tokens(M, N, round_up(K, BK) * nseg, symmetric).ws_bytes;
}

int tc_gemm_tokens(const __nv_bfloat16* A, int64_t lda, const __nv_bfloat16* B, int64_t ldb,
                   int64_t M, int64_t N, int64_t K, void* Cout, int64_t ldc, int type_c,
                   int64_t scale_from, float scale, int symmetric, const TcSegments* segs,
                   void* ws, size_t ws_bytes, int* dev_status, cudaStream_t stream, const TcPlanes* planes) {
  if (tc_init() != PRAC_OK) return PRAC_ECUDA;
  if (M <= 0 || N <= 0 || K <= 0) return PRAC_EINVAL;
  if (!aligned16(B) || (ldb % 8)) return PRAC_EALIGN;
  if (type_c != ET_BF16 && type_c != ET_F32) return PRAC_EINVAL;
  if (symmetric && (A != B || M != N)) return PRAC_EINVAL;
  if (planes && (!symmetric || type_c != ET_F32 || scale != 1.f || segs != nullptr || !planes->base || !aligned16(planes->base) ||
                 planes->rows_pad % 64 != 0 || planes->ld % 64 != 0 || planes->rows_pad < M || planes->ld < M))
    return PRAC_EINVAL;
  if (!planes && Cout == nullptr) return PRAC_EINVAL;
  const bool a_ldg = !aligned16(A) || (lda % 8) != 0;     // A off the 16-byte grid
  if (a_ldg && aligned16(A) && segs == nullptr && !symmetric) {
    // rows with the same offset from the grid go through TMA as one class, when the workspace
    // holds one partial product per class; plain loads otherwise
    const TokenClassPlan c = plan_token_classes(lda, M, N, K);
    if (c.ok && ws != nullptr && ws_bytes >= c.ws_bytes) {
      ClassMaps cm;
      for (int j = 0; j < 8; ++j) {
        const int jj = j < c.P ? j : 0;
        const int64_t rows = (K - jj + c.P - 1) / c.P;
        cuuint64_t gdim_a[2] = {static_cast<cuuint64_t>(M + c.shift[jj]), static_cast<cuuint64_t>(rows > 0 ? rows : 1)};
        cuuint64_t gstr_a[1] = {static_cast<cuuint64_t>(c.P) * lda * 2};
        cuuint64_t gdim_b[2] = {static_cast<cuuint64_t>(N), static_cast<cuuint64_t>(rows > 0 ? rows : 1)};
        cuuint64_t gstr_b[1] = {static_cast<cuuint64_t>(c.P) * ldb * 2};
        cuuint32_t box[2] = {64u, static_cast<cuuint32_t>(BK)};
        cuuint32_t estr[2] = {1u, 1u};
        if (g_encode(&cm.a[j], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<__nv_bfloat16*>(A + jj * lda - c.shift[jj]),
                     gdim_a, gstr_a, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS ||
            g_encode(&cm.c[j], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<__nv_bfloat16*>(B + jj * ldb), gdim_b,
                     gstr_b, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
          return PRAC_ECUDA;
      }
      TcParams p{};
      p.M = static_cast<int>(M); p.N = static_cast<int>(N); p.K = static_cast<int>(K);
      p.n_tiles = c.t.n_tiles; p.n_tiles1 = c.t.n_tiles;
      p.num_tiles = c.t.num_tiles;
      p.kblocks = c.kblocks;
      p.kb_per_seg = c.kblocks;
      p.splits = c.P * c.sub;
      p.cls_count = c.P;
      p.cls_sub = c.sub;
      for (int j = 0; j < c.P; ++j) p.cls_shift[j] = c.shift[j];
      p.partial = static_cast<float*>(ws);
      p.dev_status = dev_status;
      using C = Cfg<2, 256, EPI_PARTIAL>;
      static DeviceOnce attr_set;
      const int dev = current_device();
      if (!attr_set.done(dev)) {
        PRAC_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_tokens_rowclass_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           C::SMEM_BYTES));
        attr_set.mark(dev);
      }
      const int items = p.num_tiles * p.splits;
      const int cap = resident_workers<2, 256, true, EPI_PARTIAL>();   // same footprint as the plain token-major kernel
      const int workers = items < cap ? items : cap;
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(static_cast<unsigned>(2 * workers));
      cfg.blockDim = dim3(NUM_THREADS);
      cfg.dynamicSmemBytes = C::SMEM_BYTES;
      cfg.stream = stream;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr;
      cfg.numAttrs = 1;
      PRAC_CUDA_TRY(cudaLaunchKernelEx(&cfg, gemm_tc_tokens_rowclass_kernel, cm, p));
      count_launch();
      ReduceParams r{};
      r.partial = p.partial;
      r.splits = p.splits; r.num_tiles = p.num_tiles;
      r.n_tiles = c.t.n_tiles; r.tile_m = c.t.tile_m; r.bn = c.t.bn;
      r.M = p.M; r.N = p.N; r.ldo = ldc;
      r.scale_from = scale_from < 0 || scale_from > N ? static_cast<int>(N) : static_cast<int>(scale_from);
      r.scale = scale;
      r.cls_sub = c.sub;
      for (int j = 0; j < c.P; ++j) r.cls_shift[j] = c.shift[j];
      const long long work = static_cast<long long>(M) * ((N + 3) / 4);
      const unsigned blocks = static_cast<unsigned>((work + 255) / 256);
      if (type_c == ET_BF16) splitk_reduce_kernel<__nv_bfloat16><<<blocks, 256, 0, stream>>>(r, static_cast<__nv_bfloat16*>(Cout));
      else splitk_reduce_kernel<float><<<blocks, 256, 0, stream>>>(r, static_cast<float*>(Cout));
      count_launch();
      PRAC_CUDA_TRY(cudaGetLastError());
      return PRAC_OK;
    }
  }
  if (a_ldg && !(tc_tokens_takes_unaligned_a(M, N) && segs == nullptr && !symmetric)) return PRAC_EALIGN;
  const int nseg = segs ? segs->n : 1;
  if (nseg < 1 || nseg > TC_MAX_SEGMENTS) return PRAC_EINVAL;
  if (segs && (K % BK != 0 || segs->rows_a < K || segs->rows_b < K)) return PRAC_EINVAL;
  const int64_t k_chain = round_up(K, BK) * nseg;
  const TokensPlan t = plan_tokens(M, N, k_chain, symmetric);
  if (!t.ok) return PRAC_EINVAL;
  if (ws == nullptr || ws_bytes < t.ws_bytes) return PRAC_EWORKSPACE;
  CUtensorMap ta, tb;
  if (make_map(&tb, B, N, segs ? segs->rows_b : K, ldb, BK) != PRAC_OK) return PRAC_ECUDA;
  if (a_ldg) ta = tb;
  else if (make_map(&ta, A, M, segs ? segs->rows_a : K, lda, BK) != PRAC_OK) return PRAC_ECUDA;
  TcParams p{};
  p.M = static_cast<int>(M); p.N = static_cast<int>(N); p.K = static_cast<int>(K);
  p.n_tiles = t.n_tiles;
  p.num_tiles = t.num_tiles;
  p.kblocks = t.kblocks;
  p.splits = t.splits;
  p.kb_per_seg = t.kblocks / nseg;
  for (int g = 0; g < nseg; ++g) {
    p.seg_a[g] = segs ? static_cast<int>(segs->off_a[g]) : 0;
    p.seg_b[g] = segs ? static_cast<int>(segs->off_b[g]) : 0;
  }
  p.symmetric = symmetric;
  p.partial = static_cast<float*>(ws);
  p.dev_status = dev_status;
  int st;
  if (a_ldg) {
    p.a_ptr = A; p.a_ld = lda; p.a_rows = p.K; p.a_cols = p.M;
    st = launch<2, 256, true, EPI_PARTIAL, true>(ta, tb, ta, p, stream);
  } else if (t.ctas == 2) st = launch<2, 256, true, EPI_PARTIAL>(ta, tb, ta, p, stream);
  else if (t.bn == 256) st = launch<1, 256, true, EPI_PARTIAL>(ta, tb, ta, p, stream);
  else if (t.bn == 128) st = launch<1, 128, true, EPI_PARTIAL>(ta, tb, ta, p, stream);
  else st = launch<1, 64, true, EPI_PARTIAL>(ta, tb, ta, p, stream);
  if (st != PRAC_OK) return st;
  ReduceParams r{};
  r.partial = p.partial;
  r.splits = t.splits; r.num_tiles = t.num_tiles;
  r.n_tiles = t.n_tiles; r.tile_m = t.tile_m; r.bn = t.bn;
  r.M = p.M; r.N = p.N; r.ldo = ldc;
  r.scale_from = scale_from < 0 || scale_from > N ? static_cast<int>(N) : static_cast<int>(scale_from);
  r.scale = scale;
  r.symmetric = symmetric;
  const long long work = static_cast<long long>(M) * ((N + 3) / 4);
  const int threads = 256;
  const unsigned blocks = static_cast<unsigned>((work + threads - 1) / threads);
  if (planes) {
    if (t.tile_m % 64 != 0 || t.bn % 64 != 0) return PRAC_EINVAL;
    const dim3 pairs(static_cast<unsigned>(planes->ld / 64), static_cast<unsigned>(planes->rows_pad / 64));
    splitk_reduce_sym_split3_kernel<<<pairs, threads, 0, stream>>>(r, static_cast<float*>(Cout), planes->base,
                                                                    planes->rows_pad, planes->ld);
  } else if (symmetric && t.tile_m % 32 == 0 && t.bn % 32 == 0) {
    const int nblk = static_cast<int>((N + 31) / 32);
    const dim3 pairs(static_cast<unsigned>(nblk), static_cast<unsigned>(nblk));
    if (type_c == ET_BF16)
      splitk_reduce_sym_kernel<__nv_bfloat16><<<pairs, threads, 0, stream>>>(r, static_cast<__nv_bfloat16*>(Cout));
    else
      splitk_reduce_sym_kernel<float><<<pairs, threads, 0, stream>>>(r, static_cast<float*>(Cout));
  } else if (type_c == ET_BF16)
    splitk_reduce_kernel<__nv_bfloat16><<<blocks, threads, 0, stream>>>(r, static_cast<__nv_bfloat16*>(Cout));
  else
    splitk_reduce_kernel<float><<<blocks, threads, 0, stream>>>(r, static_cast<float*>(Cout));
  count_launch();
  PRAC_CUDA_TRY(cudaGetLastError());
  return PRAC_OK;
}

}  // namespace prac
