// extern "C" boundary of libprac: argument checks, storage carving, and the sequence of
// kernels behind each entry point declared in include/prac.h.
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <atomic>
#include <new>

#include "internal.h"

using namespace prac;

struct prac_basis {
  prac_params p;
  int64_t s;        // k + r
  int64_t ell;      // columns of the subspace-iteration panel (k + oversampling)
  int iters;
  char* mem;
  size_t bytes;
  int* status;      // device status word
  float* P;         // d x s fp32, [U | Q]
  __nv_bfloat16* Pb;   // d x s bf16 (row pitch ldpb): K-major operand of dW stage 2
  int64_t ldpb;
  __nv_bfloat16* Pcb;  // d x s bf16 (row pitch ldpb): [U | c Q], K-major operand of the rebuilt input
  __nv_bfloat16* PTb;  // s x d bf16 (row pitch ldptb): K-major operand of compress
  int64_t ldptb;
  double c;
  bool have_u, have_q;
  bool last_fit_eig;   // the last principal fit ended with the eigen-solve (a cold fit)
};

namespace prac {
static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(static_cast<uint64_t>(n), std::memory_order_relaxed); }
static std::atomic<unsigned> g_barrier_polls{1u << 22};
unsigned barrier_poll_limit() { return g_barrier_polls.load(std::memory_order_relaxed); }
}  // namespace prac

namespace {

constexpr uint64_t START_BLOCK_STREAM = 1ull << 63;  // draw-counter bit of the iteration's start block

struct Carver {
  size_t off = 0;
  size_t take(size_t bytes) {
    const size_t o = off;
    off += (bytes + 255) / 256 * 256;
    return o;
  }
};

bool params_ok(const prac_params* p) {
  if (!p) return false;
  if (p->d <= 0 || p->k < 0 || p->r < 0) return false;
  if (p->k + p->r < 1 || p->k + p->r > p->d) return false;
  if (p->dtype != PRAC_BF16 && p->dtype != PRAC_F32) return false;
  if (p->oversample < 0 || p->iters < 0 || p->reserved != 0) return false;
  if (p->d > (1ll << 30)) return false;
  return true;
}

int64_t panel_cols(const prac_params* p) {
  if (p->k == 0) return 0;
  const int64_t over = p->oversample > 0 ? p->oversample : (p->k / 4 > 32 ? p->k / 4 : 32);
  int64_t ell = round_up(p->k + over, 16);
  if (ell > p->d) ell = p->d;
  return ell;
}

struct BasisLayout { size_t status, P, Pb, PTb, Pcb, total; int64_t ldpb, ldptb; };
BasisLayout basis_layout(const prac_params* p) {
  BasisLayout L;
  const int64_t s = p->k + p->r;
  L.ldpb = round_up(s, 8);
  L.ldptb = round_up(p->d, 8);
  Carver c;
  L.status = c.take(256);
  L.P = c.take(static_cast<size_t>(p->d) * s * sizeof(float));
  L.Pb = c.take(static_cast<size_t>(p->d) * L.ldpb * 2);
  L.PTb = c.take(static_cast<size_t>(s) * L.ldptb * 2);
  L.Pcb = c.take(static_cast<size_t>(p->d) * L.ldpb * 2);
  L.total = c.off;
  return L;
}

// The products C * V of the subspace iteration run on the tensor cores when the problem is big
// enough to fill their tiles: C and V are held as stacks of three bf16 pieces and the six
// leading cross terms are chained into one accumulation (about fp32 accuracy).
inline bool iterate_on_tensor_cores(int64_t d, int64_t ell) { return d >= 256 && ell >= 64; }

// Rayleigh-Ritz window.  After the iteration the panel's columns are in Gram-Schmidt order: the
// leading ones already lie in the dominant subspace up to components that the iteration damps by
// (lambda_j / lambda_i)^q, and only the split between the directions near rank k is left to
// decide.  The first k - w columns of the panel are therefore taken into U as they are and the
// eigenproblem is solved on the remaining n = (ell - k) + w columns, of which the top w complete
// U.  w = min(k, ell - k): as many columns as are discarded (measured: captured energy within
// 1.5x of the loss of a Rayleigh-Ritz step over the whole panel, on an eigenproblem of 128
// instead of 320 columns at k = 256; w = k is the step over the whole panel).
struct RitzWindow { int64_t w, first, n; };
RitzWindow ritz_window(int64_t k, int64_t ell) {
  RitzWindow win;
  const int64_t m = ell - k;
  win.w = k < m ? k : (m > 0 ? m : k);
  if (win.w > k) win.w = k;
  win.first = k - win.w;
  win.n = ell - win.first;
  return win;
}

struct FitLayout { size_t C, V, Y, T2, Bj, Wsel, T, chol, jac, atb, Cs, Vs, mm, mm3, part, xpack, total; size_t mm3_bytes; int64_t ldxp; int64_t nj, wcols, kp, ldcs, ldvs; size_t chol_bytes, jac_bytes, atb_bytes, mm_bytes, part_bytes; };
FitLayout fit_layout(const prac_params* p, int64_t N) {
  FitLayout L{};
  const int64_t d = p->d, k = p->k, r = p->r, ell = panel_cols(p);
  const RitzWindow win = ritz_window(k, ell);
  L.nj = win.n;
  L.wcols = ell > r ? ell : r;       // the two panels also serve as scratch of the draw's QR
  Carver c;
  L.C = c.take(k > 0 ? static_cast<size_t>(d) * d * 4 : 0);
  L.V = c.take(static_cast<size_t>(d) * L.wcols * 4);
  L.Y = c.take(static_cast<size_t>(d) * L.wcols * 4);
  L.T2 = c.take(static_cast<size_t>(d) * L.wcols * 4);     // scratch of the optional extra orthonormalisation pass
  L.Bj = c.take(static_cast<size_t>(L.nj) * L.nj * 8);
  L.Wsel = c.take(static_cast<size_t>(L.nj) * (k > 0 ? k : 1) * 4);
  L.T = c.take(static_cast<size_t>(k > 0 ? k : 1) * (r > 0 ? r : 1) * 4);
  // the row-slice count, hence the scratch, is not monotone in the panel width: size for both
  const size_t chol_ell = cholqr_ws_bytes(ell, d), chol_r = cholqr_ws_bytes(r, d), chol_k = cholqr_ws_bytes(k, d);
  L.chol_bytes = chol_ell > chol_r ? chol_ell : chol_r;
  if (chol_k > L.chol_bytes) L.chol_bytes = chol_k;      // the warm refresh orthonormalises d x k panels
  L.chol = c.take(L.chol_bytes);
  L.jac_bytes = jacobi_ws_bytes(L.nj);
  L.jac = c.take(L.jac_bytes);
  const size_t atb_rr = atb_ws_bytes(win.n, win.n, d, 0), atb_pr = atb_ws_bytes(k, r, d, 0);
  L.atb_bytes = atb_rr > atb_pr ? atb_rr : atb_pr;
  L.atb = c.take(L.atb_bytes);
  L.kp = round_up(d, 64);
  L.ldcs = round_up(d, 64);
  L.ldvs = round_up(ell > 0 ? ell : 1, 64);
  const bool tc_iter = k > 0 && iterate_on_tensor_cores(d, ell);
  L.Cs = c.take(tc_iter ? static_cast<size_t>(3) * L.kp * L.ldcs * 2 : 0);
  L.Vs = c.take(tc_iter ? static_cast<size_t>(3) * L.kp * L.ldvs * 2 : 0);
  L.mm_bytes = 0;
  if (tc_iter) {   // the product runs on the whole panel and on the Rayleigh-Ritz window
    const size_t whole = tc_gemm_tokens_ws_bytes(d, ell, L.kp, 0, 6), part = tc_gemm_tokens_ws_bytes(d, win.n, L.kp, 0, 6);
    const size_t warm = tc_gemm_tokens_ws_bytes(d, k, L.kp, 0, 6);
    const size_t whole3 = tc_gemm_tokens_ws_bytes(d, ell, L.kp, 0, 3), warm3 = tc_gemm_tokens_ws_bytes(d, k, L.kp, 0, 3);
    const size_t whole1 = tc_gemm_tokens_ws_bytes(d, ell, L.kp, 0, 1);
    L.mm_bytes = whole > part ? whole : part;
    if (warm > L.mm_bytes) L.mm_bytes = warm;
    if (whole3 > L.mm_bytes) L.mm_bytes = whole3;
    if (warm3 > L.mm_bytes) L.mm_bytes = warm3;
    if (whole1 > L.mm_bytes) L.mm_bytes = whole1;
  }
  L.mm = c.take(L.mm_bytes);
  {  // the panel products U = Y_b W (window) and S -= U (U^T S) (draw) as three bf16 pieces per operand
    const size_t win_b = k > 0 ? panel_mm3_ws_bytes(d, win.n, win.w) : 0, draw_b = (k > 0 && r > 0) ? panel_mm3_ws_bytes(d, k, r) : 0;
    L.mm3_bytes = win_b > draw_b ? win_b : draw_b;
  }
  L.mm3 = c.take(L.mm3_bytes);
  L.part_bytes = (k > 0 && p->dtype == PRAC_BF16) ? tc_gemm_tokens_ws_bytes(d, d, N, 1) : 0;
  L.part = c.take(L.part_bytes);
  // A contiguous bf16 X whose width is not a multiple of 8 has rows off the 16-byte grid, which the
  // symmetric Gram launch (both operands by TMA) cannot read: room for an aligned copy of X
  L.ldxp = round_up(d, 64);
  L.xpack = c.take((k > 0 && p->dtype == PRAC_BF16 && d % 8 != 0) ? static_cast<size_t>(N) * L.ldxp * 2 : 0);
  L.total = c.off;
  return L;
}

struct GradLayout { size_t M, part, total; size_t part_bytes; size_t min_total; };   // min_total: without the extra room of the row-class path
GradLayout grad_layout(const prac_params* p, int64_t N, int64_t d_out) {
  GradLayout L{};
  const int64_t s = p->k + p->r;
  Carver c;
  L.M = c.take(static_cast<size_t>(d_out) * round_up(s, 8) * 4);  // fp32 (general) or bf16 (tensor) view
  L.part_bytes = p->dtype == PRAC_BF16 ? tc_gemm_tokens_ws_bytes(d_out, s, N, 0) : 0;
  L.min_total = c.off + (L.part_bytes + 255) / 256 * 256;
  if (p->dtype == PRAC_BF16 && d_out % 8 != 0) {
    // a contiguous dY of this width has rows off the 16-byte grid: room for one partial product per class of rows
    const size_t by_class = tc_gemm_tokens_rowclass_ws_bytes(d_out, d_out, s, N);
    if (by_class > L.part_bytes) L.part_bytes = by_class;
  }
  L.part = c.take(L.part_bytes);
  L.total = c.off;
  return L;
}

inline bool aligned256(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }
inline int elem_type(int dtype) { return dtype == PRAC_BF16 ? ET_BF16 : ET_F32; }
inline bool tma_ok(const void* p, int64_t ld) { return aligned16(p) && (ld % 8) == 0; }

int refresh_bf16_copies(prac_basis* b, cudaStream_t st) {
  return launch_make_bf16_copies(b->P, b->s, b->p.d, b->s, b->p.k, b->c, b->Pcb, b->Pb, b->ldpb, b->PTb, b->ldptb, st);
}

GemmArgs gemm_args(int64_t M, int64_t N, int64_t K, const void* A, int64_t lda, int ta, int tra,
                   const void* B, int64_t ldb, int tb, int trb, void* C, int64_t ldc, int tc,
                   double alpha, double beta, int acc_double) {
  GemmArgs g{};
  g.M = M; g.N = N; g.K = K;
  g.A = A; g.lda = lda; g.type_a = ta; g.trans_a = tra;
  g.B = B; g.ldb = ldb; g.type_b = tb; g.trans_b = trb;
  g.C = C; g.ldc = ldc; g.type_c = tc;
  g.alpha = alpha; g.beta = beta; g.acc_double = acc_double;
  g.kscale_from = -1; g.kscale = 1.0;
  return g;
}

// Y (d x cols, leading dimension ldy) = C V for the symmetric d x d matrix C and the d x cols
// panel V (leading dimension ldv); cols <= ell.
// Y = C V.  `terms` = 6: fp32 accuracy (every cross term of the three bf16 pieces of C and V down to
// 2^-24 of the product); 3: the leading term and the two next ones (about 2^-16), for the products of
// the subspace iteration that another product and orthonormalisation follow; 1: the leading term
// alone (2^-8), for the product with the Gaussian start block, where the error is one more random
// perturbation of a random start.
int apply_gram(const prac_basis* b, const FitLayout& L, char* w, const float* V, int64_t ldv, int64_t cols, float* Y,
               int64_t ldy, cudaStream_t st, int terms = 6) {
  const int64_t d = b->p.d;
  const float* C = reinterpret_cast<const float*>(w + L.C);
  if (!iterate_on_tensor_cores(d, b->ell))
    return gemm_general(gemm_args(d, cols, d, C, d, ET_F32, 0, V, ldv, ET_F32, 0, Y, ldy, ET_F32, 1.0, 0.0, 0), st);
  __nv_bfloat16* Cs = reinterpret_cast<__nv_bfloat16*>(w + L.Cs);
  __nv_bfloat16* Vs = reinterpret_cast<__nv_bfloat16*>(w + L.Vs);
  int sc = launch_split3(V, ldv, d, cols, Vs, L.kp, L.ldvs, st);
  if (sc != PRAC_OK) return sc;
  // (piece of C, piece of V): the three smallest cross terms first, the leading one last
  static const int pa[6] = {2, 1, 0, 1, 0, 0}, pb[6] = {0, 1, 2, 0, 1, 0};
  TcSegments segs{};
  segs.n = terms;
  for (int g = 0; g < terms; ++g) { segs.off_a[g] = pa[6 - terms + g] * L.kp; segs.off_b[g] = pb[6 - terms + g] * L.kp; }
  segs.rows_a = 3 * L.kp;
  segs.rows_b = 3 * L.kp;
  // C is symmetric, so its rows serve as the K x M operand
  return tc_gemm_tokens(Cs, L.ldcs, Vs, L.ldvs, d, cols, L.kp, Y, ldy, ET_F32, -1, 1.f, 0, &segs, w + L.mm,
                        L.mm_bytes, b->status, st);
}

}  // namespace

extern "C" {

int prac_version(void) { return 1000; }

uint64_t prac_kernel_launches(void) { return prac::g_launches.load(std::memory_order_relaxed); }

int64_t prac_debug_bounds_violations(void) {
#ifdef PRAC_DEBUG_BOUNDS
  if (cudaDeviceSynchronize() != cudaSuccess) return -2;
  const long long parts[4] = {bounds_violations_simt(), bounds_violations_panel(), bounds_violations_cholqr(),
                              bounds_violations_tc()};
  long long sum = 0;
  for (long long v : parts) {
    if (v < 0) return -2;
    sum += v;
  }
  return sum;
#else
  return -1;
#endif
}

void prac_debug_set_barrier_poll_limit(uint32_t polls) {
  prac::g_barrier_polls.store(polls == 0 ? (1u << 22) : polls, std::memory_order_relaxed);
}

const char* prac_status_string(int status) {
  switch (status) {
    case PRAC_OK: return "ok";
    case PRAC_EINVAL: return "invalid argument";
    case PRAC_EWORKSPACE: return "workspace or storage too small";
    case PRAC_EALIGN: return "storage not 256-byte aligned";
    case PRAC_ENUMERIC: return "numerical breakdown in orthonormalisation or eigen-solver";
    case PRAC_ETIMEOUT: return "bounded device wait expired";
    case PRAC_ECUDA: return "CUDA call failed";
    case PRAC_ESTATE: return "basis not ready";
    default: return "unknown status";
  }
}

size_t prac_basis_bytes(const prac_params* params) {
  if (!params_ok(params)) return 0;
  return basis_layout(params).total;
}

size_t prac_fit_workspace_bytes(const prac_params* params, int64_t N) {
  if (!params_ok(params) || N <= 0) return 0;
  return fit_layout(params, N).total;
}

size_t prac_grad_workspace_bytes(const prac_params* params, int64_t N, int64_t d_out) {
  if (!params_ok(params) || N <= 0 || d_out <= 0) return 0;
  return grad_layout(params, N, d_out).total;
}

int prac_basis_create(prac_basis** out, const prac_params* params, void* dev_mem, size_t bytes) {
  if (!out) return PRAC_EINVAL;
  *out = nullptr;
  if (!params_ok(params) || !dev_mem) return PRAC_EINVAL;
  if (!aligned256(dev_mem)) return PRAC_EALIGN;
  const BasisLayout L = basis_layout(params);
  if (bytes < L.total) return PRAC_EWORKSPACE;
  PRAC_CUDA_TRY(cudaMemset(dev_mem, 0, L.total));
  PRAC_CUDA_TRY(cudaDeviceSynchronize());
  prac_basis* b = new (std::nothrow) prac_basis();
  if (!b) return PRAC_EINVAL;
  b->p = *params;
  b->s = params->k + params->r;
  b->ell = panel_cols(params);
  b->iters = params->iters > 0 ? params->iters : 4;
  b->mem = static_cast<char*>(dev_mem);
  b->bytes = bytes;
  b->status = reinterpret_cast<int*>(b->mem + L.status);
  b->P = reinterpret_cast<float*>(b->mem + L.P);
  b->Pb = reinterpret_cast<__nv_bfloat16*>(b->mem + L.Pb);
  b->PTb = reinterpret_cast<__nv_bfloat16*>(b->mem + L.PTb);
  b->Pcb = reinterpret_cast<__nv_bfloat16*>(b->mem + L.Pcb);
  b->ldpb = L.ldpb;
  b->ldptb = L.ldptb;
  b->c = params->r > 0 ? static_cast<double>(params->d - params->k) / static_cast<double>(params->r) : 1.0;
  b->have_u = (params->k == 0);
  b->have_q = false;
  b->last_fit_eig = false;
  *out = b;
  return PRAC_OK;
}

void prac_basis_destroy(prac_basis* basis) { delete basis; }

}  // extern "C"

namespace {
// The principal fit.  warm == 0: Gaussian start block, `iters` iterations.  warm != 0: the start
// block is [current U | fresh Gaussian columns], for refreshes of a slowly moving subspace.
// Cext != nullptr: the Gram matrix is given (d x d fp32, leading dimension ldce; e.g. the sum over
// the ranks of a token-sharded batch) and X is not read.
int fit_principal_impl(prac_basis* b, const void* X, int64_t N, int64_t ldx, uint64_t seed,
                       uint64_t draw_counter, void* ws, size_t ws_bytes, void* stream, int warm, int iters,
                       const float* Cext = nullptr, int64_t ldce = 0) {
  if (!b || N <= 0) return PRAC_EINVAL;
  if (Cext ? (ldce < b->p.d) : (!X || ldx < b->p.d)) return PRAC_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t d = b->p.d, k = b->p.k, ell = b->ell;
  if (k == 0) {
    b->have_u = true;
    b->have_q = false;
    return PRAC_OK;
  }
  const FitLayout L = fit_layout(&b->p, N);
  if (!ws || ws_bytes < L.total) return PRAC_EWORKSPACE;
  if (!aligned256(ws)) return PRAC_EALIGN;
  char* w = static_cast<char*>(ws);
  float* C = reinterpret_cast<float*>(w + L.C);
  float* V = reinterpret_cast<float*>(w + L.V);
  float* Y = reinterpret_cast<float*>(w + L.Y);
  double* Bj = reinterpret_cast<double*>(w + L.Bj);
  float* Wsel = reinterpret_cast<float*>(w + L.Wsel);
  int st_code;

  // a1: Gram matrix C = X^T X (fp32).  Where the iteration runs on the tensor cores C is only ever
  // used as its three bf16 pieces, which the Gram launch's reduction then writes directly.
  const bool tc_iter = iterate_on_tensor_cores(d, ell);
  const TcPlanes gram_planes{reinterpret_cast<__nv_bfloat16*>(w + L.Cs), L.kp, L.ldcs};
  bool have_pieces = false;
  if (Cext) {
    st_code = launch_copy2d(Cext, ldce, C, d, d, d, st);
  } else if (b->p.dtype == PRAC_BF16 && tma_ok(X, ldx)) {
    st_code = tc_gemm_tokens(static_cast<const __nv_bfloat16*>(X), ldx, static_cast<const __nv_bfloat16*>(X), ldx,
                             d, d, N, tc_iter ? nullptr : C, d, ET_F32, -1, 1.f, 1, nullptr, w + L.part, L.part_bytes,
                             b->status, st, tc_iter ? &gram_planes : nullptr);
    have_pieces = tc_iter;
  } else if (b->p.dtype == PRAC_BF16 && d % 8 != 0) {
    // rows of X off the 16-byte grid: one pass copies them to aligned rows, then the same launch
    __nv_bfloat16* Xp = reinterpret_cast<__nv_bfloat16*>(w + L.xpack);
    st_code = launch_repack_rows_bf16(static_cast<const __nv_bfloat16*>(X), ldx, N, d, Xp, L.ldxp, st);
    if (st_code != PRAC_OK) return st_code;
    st_code = tc_gemm_tokens(Xp, L.ldxp, Xp, L.ldxp, d, d, N, tc_iter ? nullptr : C, d, ET_F32, -1, 1.f, 1, nullptr,
                             w + L.part, L.part_bytes, b->status, st, tc_iter ? &gram_planes : nullptr);
    have_pieces = tc_iter;
  } else {
    const int et = elem_type(b->p.dtype);
    st_code = gemm_general(gemm_args(d, d, N, X, ldx, et, 1, X, ldx, et, 0, C, d, ET_F32, 1.0, 0.0, 0), st);
  }
  if (st_code != PRAC_OK) return st_code;

  // a2: randomized subspace iteration on C.  The Gaussian start block is well conditioned as
  // it is; after each product one Cholesky-QR pass keeps the panel well conditioned (its
  // columns stay in Gram-Schmidt order), and a second pass before the Rayleigh-Ritz step makes
  // it orthonormal to fp32 accuracy.
  if (tc_iter && !have_pieces) {
    st_code = launch_split3(C, d, d, d, reinterpret_cast<__nv_bfloat16*>(w + L.Cs), L.kp, L.ldcs, st);
    if (st_code != PRAC_OK) return st_code;
  }
  if (warm) {
    // Refresh of an existing U on slowly moving activations: orthogonal iteration started from
    // the current U itself, U <- orth(C U) `iters` times, then one more pass to fp32
    // orthonormality.  No oversampling columns and no Rayleigh-Ritz step: the start is already
    // (nearly) the dominant subspace, each iteration can only raise the captured energy
    // tr(U^T C U), and the error in span(U) left by a drift of the data shrinks by
    // (lambda_{k+1} / lambda_k) per iteration wherever the spectrum has a gap.  What it saves is
    // the eigen-solve and the wider panel, i.e. most of a cold fit's latency.
    st_code = launch_copy2d(b->P, b->s, V, k, d, k, st);
    if (st_code != PRAC_OK) return st_code;
    for (int it = 0; it < iters; ++it) {
      st_code = apply_gram(b, L, w, V, k, k, Y, k, st, it + 1 < iters ? 3 : 6);
      if (st_code != PRAC_OK) return st_code;
      st_code = cholqr_pass(Y, k, V, k, d, k, w + L.chol, L.chol_bytes, b->status, 0, st);
      if (st_code != PRAC_OK) return st_code;
    }
    st_code = cholqr_final(V, k, b->P, b->s, reinterpret_cast<float*>(w + L.T2), d, k, w + L.chol, L.chol_bytes,
                           b->status, st);
    if (st_code != PRAC_OK) return st_code;
    b->last_fit_eig = false;
    b->have_u = true;
    b->have_q = false;
    if (b->p.r == 0) {
      b->c = 1.0;
      st_code = refresh_bf16_copies(b, st);
      if (st_code != PRAC_OK) return st_code;
      b->have_q = true;
    }
    return PRAC_OK;
  }
  st_code = launch_gaussian(seed, draw_counter | START_BLOCK_STREAM, d, ell, V, ell, st);
  if (st_code != PRAC_OK) return st_code;
  for (int it = 0; it < iters; ++it) {
    st_code = apply_gram(b, L, w, V, ell, ell, Y, ell, st, it + 1 < iters ? (it == 0 ? 1 : 3) : 6);
    if (st_code != PRAC_OK) return st_code;
    st_code = cholqr_pass(Y, ell, V, ell, d, ell, w + L.chol, L.chol_bytes, b->status, 0, st);
    if (st_code != PRAC_OK) return st_code;
  }
  // (a bad pivot here switches on one more pass)
  st_code = cholqr_final(V, ell, Y, ell, reinterpret_cast<float*>(w + L.T2), d, ell, w + L.chol, L.chol_bytes, b->status, st);
  if (st_code != PRAC_OK) return st_code;
  // Rayleigh-Ritz on the orthonormal panel Y, restricted to its last n columns Y_b (see
  // ritz_window): T = C Y_b (into V), B = Y_b^T T, eigenvectors W of the w largest eigenvalues of
  // B; U = [first k - w columns of Y | Y_b W]
  const RitzWindow win = ritz_window(k, ell);
  const float* Yb = Y + win.first;
  st_code = apply_gram(b, L, w, Yb, ell, win.n, V, win.n, st);
  if (st_code != PRAC_OK) return st_code;
  st_code = atb_f64(Yb, ell, V, win.n, d, win.n, win.n, 0, 1.0, Bj, win.n, 1, w + L.atb, L.atb_bytes, st);
  if (st_code != PRAC_OK) return st_code;
  st_code = jacobi_topk(Bj, win.n, win.n, win.w, Wsel, w + L.jac, L.jac_bytes, b->status, st);
  if (st_code != PRAC_OK) return st_code;
  st_code = launch_copy2d(Y, ell, b->P, b->s, d, win.first, st);
  if (st_code != PRAC_OK) return st_code;
  st_code = panel_mm3(Yb, ell, Wsel, win.w, d, win.n, win.w, 1.f, b->P + win.first, b->s, 0, w + L.mm3, L.mm3_bytes,
                      b->status, st);
  if (st_code != PRAC_OK) return st_code;

  b->last_fit_eig = true;
  b->have_u = true;
  b->have_q = false;
  if (b->p.r == 0) {
    b->c = 1.0;
    st_code = refresh_bf16_copies(b, st);
    if (st_code != PRAC_OK) return st_code;
    b->have_q = true;
  }
  return PRAC_OK;
}

}  // namespace

extern "C" {

int prac_fit_principal(prac_basis* b, const void* X, int64_t N, int64_t ldx, uint64_t seed,
                       uint64_t draw_counter, void* ws, size_t ws_bytes, void* stream) {
  if (!b) return PRAC_EINVAL;
  return fit_principal_impl(b, X, N, ldx, seed, draw_counter, ws, ws_bytes, stream, 0, b->iters);
}

int prac_refresh_principal(prac_basis* b, const void* X, int64_t N, int64_t ldx, uint64_t seed,
                           uint64_t draw_counter, int32_t iters, void* ws, size_t ws_bytes, void* stream) {
  if (!b || iters < 0) return PRAC_EINVAL;
  if (b->p.k > 0 && !b->have_u) return PRAC_ESTATE;
  return fit_principal_impl(b, X, N, ldx, seed, draw_counter, ws, ws_bytes, stream, 1, iters > 0 ? iters : 2);
}

int prac_gram(const prac_basis* b, const void* X, int64_t N, int64_t ldx, float* C, int64_t ldc,
              void* ws, size_t ws_bytes, void* stream) {
  if (!b || !X || !C || N <= 0 || ldx < b->p.d || ldc < b->p.d) return PRAC_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t d = b->p.d;
  if (b->p.dtype == PRAC_BF16 && (tma_ok(X, ldx) || d % 8 != 0)) {
    const FitLayout L = fit_layout(&b->p, N);
    if (!ws || ws_bytes < L.total) return PRAC_EWORKSPACE;
    if (!aligned256(ws)) return PRAC_EALIGN;
    char* w = static_cast<char*>(ws);
    const __nv_bfloat16* Xa = static_cast<const __nv_bfloat16*>(X);
    int64_t lda = ldx;
    if (!tma_ok(X, ldx)) {       // rows off the 16-byte grid: aligned copy first
      __nv_bfloat16* Xp = reinterpret_cast<__nv_bfloat16*>(w + L.xpack);
      const int sc = launch_repack_rows_bf16(Xa, ldx, N, d, Xp, L.ldxp, st);
      if (sc != PRAC_OK) return sc;
      Xa = Xp;
      lda = L.ldxp;
    }
    return tc_gemm_tokens(Xa, lda, Xa, lda, d, d, N, C, ldc, ET_F32, -1, 1.f, 1, nullptr, w + L.part, L.part_bytes,
                          b->status, st);
  }
  const int et = elem_type(b->p.dtype);
  return gemm_general(gemm_args(d, d, N, X, ldx, et, 1, X, ldx, et, 0, C, ldc, ET_F32, 1.0, 0.0, 0), st);
}

int prac_fit_principal_gram(prac_basis* b, const float* C, int64_t ldc, uint64_t seed, uint64_t draw_counter,
                            void* ws, size_t ws_bytes, void* stream) {
  if (!b || !C) return PRAC_EINVAL;
  return fit_principal_impl(b, nullptr, 1, 0, seed, draw_counter, ws, ws_bytes, stream, 0, b->iters, C, ldc);
}

int prac_weight_grad_partial(const prac_basis* b, const void* dY, int64_t lddy, int64_t d_out, const void* Z,
                             int64_t ldz, int64_t N, float* M, int64_t ldm, void* ws, size_t ws_bytes, void* stream) {
  if (!b || !dY || !Z || !M || N <= 0 || d_out <= 0) return PRAC_EINVAL;
  if (lddy < d_out || ldz < b->s || ldm < b->s) return PRAC_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t s = b->s;
  if (b->p.dtype == PRAC_BF16 && tma_ok(Z, ldz) && (tma_ok(dY, lddy) || tc_tokens_takes_unaligned_a(d_out, s))) {
    const GradLayout L = grad_layout(&b->p, N, d_out);
    if (!ws || ws_bytes < L.min_total) return PRAC_EWORKSPACE;
    if (!aligned256(ws)) return PRAC_EALIGN;
    char* w = static_cast<char*>(ws);
    return tc_gemm_tokens(static_cast<const __nv_bfloat16*>(dY), lddy, static_cast<const __nv_bfloat16*>(Z), ldz,
                          d_out, s, N, M, ldm, ET_F32, -1, 1.f, 0, nullptr, w + L.part,
                          ws_bytes - L.part < L.part_bytes ? ws_bytes - L.part : L.part_bytes, b->status, st);
  }
  const int et = elem_type(b->p.dtype);
  return gemm_general(gemm_args(d_out, s, N, dY, lddy, et, 1, Z, ldz, et, 0, M, ldm, ET_F32, 1.0, 0.0, 0), st);
}

int prac_weight_grad_finish(const prac_basis* b, const float* M, int64_t ldm, int64_t d_out, double c_override,
                            void* dW, int64_t lddw, int32_t dw_dtype, int32_t accumulate, void* ws, size_t ws_bytes,
                            void* stream) {
  if (!b || !M || !dW || d_out <= 0 || ldm < b->s || lddw < b->p.d) return PRAC_EINVAL;
  if (dw_dtype != PRAC_BF16 && dw_dtype != PRAC_F32) return PRAC_EINVAL;
  if (!b->have_u || !b->have_q) return PRAC_ESTATE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t d = b->p.d, k = b->p.k, s = b->s;
  const double c = std::isnan(c_override) ? b->c : c_override;
  const int out_t = dw_dtype == PRAC_BF16 ? ET_BF16 : ET_F32;
  if (b->p.dtype == PRAC_BF16 && !(accumulate && out_t == ET_BF16)) {
    // M' = M diag(1, c) rounded to bf16 (as the one-call path does), then the tensor-core stage 2
    const int64_t ldmb = round_up(s, 8);
    const size_t need = static_cast<size_t>(d_out) * ldmb * 2;
    if (!ws || ws_bytes < need) return PRAC_EWORKSPACE;
    if (!aligned256(ws)) return PRAC_EALIGN;
    __nv_bfloat16* Mb = static_cast<__nv_bfloat16*>(ws);
    const int sc = launch_scale_to_bf16(M, ldm, d_out, s, k, static_cast<float>(c), Mb, ldmb, st);
    if (sc != PRAC_OK) return sc;
    return tc_gemm_kmajor(Mb, ldmb, b->Pb, b->ldpb, d_out, d, s, dW, lddw, out_t, accumulate, b->status, st);
  }
  GemmArgs g = gemm_args(d_out, d, s, M, ldm, ET_F32, 0, b->P, s, ET_F32, 1, dW, lddw, out_t, 1.0,
                         accumulate ? 1.0 : 0.0, 0);
  g.kscale_from = k;
  g.kscale = c;
  return gemm_general(g, st);
}

int prac_draw_random(prac_basis* b, uint64_t seed, uint64_t draw_counter, void* ws, size_t ws_bytes,
                     void* stream) {
  if (!b) return PRAC_EINVAL;
  if (!b->have_u) return PRAC_ESTATE;
  if (draw_counter & START_BLOCK_STREAM) return PRAC_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t d = b->p.d, k = b->p.k, r = b->p.r, s = b->s;
  if (r == 0) {
    b->c = 1.0;
    int sc = refresh_bf16_copies(b, st);
    if (sc != PRAC_OK) return sc;
    b->have_q = true;
    return PRAC_OK;
  }
  const FitLayout L = fit_layout(&b->p, 1);
  // the token count only sizes the Gram partials, which this call does not use
  const size_t need = L.part;
  if (!ws || ws_bytes < need) return PRAC_EWORKSPACE;
  if (!aligned256(ws)) return PRAC_EALIGN;
  char* w = static_cast<char*>(ws);
  float* T = reinterpret_cast<float*>(w + L.T);
  float* S = reinterpret_cast<float*>(w + L.V);     // d x r, leading dimension r
  float* Qout = b->P + k;
  int sc = launch_gaussian(seed, draw_counter, d, r, S, r, st);
  if (sc != PRAC_OK) return sc;
  if (k > 0) {
    // S_o = (I - U U^T) S.  Where U spans a small part of the space the projection removes little of
    // S (no cancellation) and one application leaves U^T S_o at the level of U's own fp32
    // orthonormality; where k is more than an eighth of d it is applied twice.
    const int reps = (8 * k > d) ? 2 : 1;
    for (int rep = 0; rep < reps; ++rep) {
      // T = U^T S ;  S -= U T
      sc = atb_f64(b->P, s, S, r, d, k, r, 0, 1.0, T, r, 0, w + L.atb, L.atb_bytes, st);
      if (sc != PRAC_OK) return sc;
      sc = panel_mm3(b->P, s, T, r, d, k, r, -1.f, S, r, 1, w + L.mm3, L.mm3_bytes, b->status, st);
      if (sc != PRAC_OK) return sc;
    }
  }
  // Thin QR with positive diagonal: one Cholesky-QR pass.  S_o is a Gaussian block with k of its d
  // dimensions removed, condition number of a few units, and its Gram matrix is accumulated and
  // factored in double, so R is exact far beyond what the fp32 product S_o R^-1 keeps; a second
  // pass (needed where the panel is ill-conditioned, as in the subspace iteration) would change
  // Q only inside its fp32 rounding.
  sc = cholqr_final(S, r, Qout, s, reinterpret_cast<float*>(w + L.T2), d, r, w + L.chol, L.chol_bytes, b->status, st);
  if (sc != PRAC_OK) return sc;
  b->c = static_cast<double>(d - k) / static_cast<double>(r);
  sc = refresh_bf16_copies(b, st);
  if (sc != PRAC_OK) return sc;
  b->have_q = true;
  return PRAC_OK;
}

int prac_fit_basis(prac_basis* b, const void* X, int64_t N, int64_t ldx, uint64_t seed,
                   uint64_t draw_counter, void* ws, size_t ws_bytes, void* stream) {
  if (draw_counter & START_BLOCK_STREAM) return PRAC_EINVAL;
  int sc = prac_fit_principal(b, X, N, ldx, seed, draw_counter, ws, ws_bytes, stream);
  if (sc != PRAC_OK) return sc;
  return prac_draw_random(b, seed, draw_counter, ws, ws_bytes, stream);
}

int prac_set_basis(prac_basis* b, const float* U, int64_t ldu, const float* Q, int64_t ldq, double c,
                   void* stream) {
  if (!b) return PRAC_EINVAL;
  const int64_t d = b->p.d, k = b->p.k, r = b->p.r;
  if ((k > 0 && (!U || ldu < k)) || (r > 0 && (!Q || ldq < r))) return PRAC_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int sc = launch_copy2d(U, ldu, b->P, b->s, d, k, st);
  if (sc != PRAC_OK) return sc;
  sc = launch_copy2d(Q, ldq, b->P + k, b->s, d, r, st);
  if (sc != PRAC_OK) return sc;
  b->c = c;
  sc = refresh_bf16_copies(b, st);
  if (sc != PRAC_OK) return sc;
  b->have_u = b->have_q = true;
  return PRAC_OK;
}

int prac_basis_get(const prac_basis* b, const float** P, int64_t* ldp, double* c) {
  if (!b) return PRAC_EINVAL;
  if (P) *P = b->P;
  if (ldp) *ldp = b->s;
  if (c) *c = b->c;
  return PRAC_OK;
}

int prac_compress(const prac_basis* b, const void* X, int64_t N, int64_t ldx, void* Z, int64_t ldz,
                  void* stream) {
  if (!b || !X || !Z || N <= 0 || ldx < b->p.d || ldz < b->s) return PRAC_EINVAL;
  if (!b->have_u || !b->have_q) return PRAC_ESTATE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t d = b->p.d, s = b->s;
  // Rows of X off the 16-byte grid (a contiguous matrix of odd width): rows with the same offset
  // from the grid are fetched by TMA as one class (the result then differs from the aligned
  // layout's in fp32 summation order only); where that does not fit, plain loads feed the same
  // tensor-core kernel; only outputs too small for its tiles take the general path.
  if (b->p.dtype == PRAC_BF16 && !tma_ok(X, ldx) && tma_ok(Z, ldz) &&
      tc_rowclass_fits(X, ldx, N, s)) {
    return tc_gemm_kmajor_rowclass(static_cast<const __nv_bfloat16*>(X), ldx, b->Pb, b->ldpb, N, s, d,
                                   static_cast<__nv_bfloat16*>(Z), ldz, b->status, st);
  }
  if (b->p.dtype == PRAC_BF16 && (tma_ok(X, ldx) || tc_kmajor_takes_unaligned_a(N, s))) {
    return tc_gemm_kmajor(static_cast<const __nv_bfloat16*>(X), ldx, b->PTb, b->ldptb, N, s, d, Z, ldz,
                          ET_BF16, 0, b->status, st);
  }
  const int et = elem_type(b->p.dtype);
  return gemm_general(gemm_args(N, s, d, X, ldx, et, 0, b->P, s, ET_F32, 0, Z, ldz, et, 1.0, 0.0, 0), st);
}

int prac_linear_forward(const prac_basis* b, const void* X, int64_t N, int64_t ldx, const void* W, int64_t ldw,
                        int64_t d_out, void* Y, int64_t ldy, void* Z, int64_t ldz, void* stream) {
  if (!b || !X || !W || !Y || N <= 0 || d_out <= 0) return PRAC_EINVAL;
  if (ldx < b->p.d || ldw < b->p.d || ldy < d_out || (Z && ldz < b->s)) return PRAC_EINVAL;
  if (Z && (!b->have_u || !b->have_q)) return PRAC_ESTATE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t d = b->p.d, s = b->s;
  if (Z && b->p.dtype == PRAC_BF16 && tma_ok(W, ldw) && N > 128) {   // (X may have unaligned rows)
    // one launch: every row tile of X is fetched once and multiplied by W and by [U|Q]
    const int dual = tc_gemm_kmajor_dual(static_cast<const __nv_bfloat16*>(X), ldx, N, d,
                                         static_cast<const __nv_bfloat16*>(W), ldw, d_out, static_cast<__nv_bfloat16*>(Y), ldy,
                                         b->PTb, b->ldptb, s, static_cast<__nv_bfloat16*>(Z), ldz, b->status, st);
    // PRAC_EALIGN: one output has 16-byte-aligned rows and the other has not; nothing was
    // launched, the two products run in turn below
    if (dual != PRAC_EALIGN) return dual;
  }
  const int et = elem_type(b->p.dtype);
  int sc;
  if (b->p.dtype == PRAC_BF16 && tma_ok(W, ldw) && (tma_ok(X, ldx) || tc_kmajor_takes_unaligned_a(N, d_out)))
    sc = tc_gemm_kmajor(static_cast<const __nv_bfloat16*>(X), ldx, static_cast<const __nv_bfloat16*>(W), ldw, N, d_out, d,
                        Y, ldy, ET_BF16, 0, b->status, st);
  else
    sc = gemm_general(gemm_args(N, d_out, d, X, ldx, et, 0, W, ldw, et, 1, Y, ldy, et, 1.0, 0.0, 0), st);
  if (sc != PRAC_OK || !Z) return sc;
  return prac_compress(b, X, N, ldx, Z, ldz, stream);
}

int prac_weight_grad(const prac_basis* b, const void* dY, int64_t lddy, int64_t d_out, const void* Z,
                     int64_t ldz, int64_t N, double c_override, void* dW, int64_t lddw, int32_t dw_dtype,
                     int32_t accumulate, void* ws, size_t ws_bytes, void* stream) {
  if (!b || !dY || !Z || !dW || N <= 0 || d_out <= 0) return PRAC_EINVAL;
  if (lddy < d_out || ldz < b->s || lddw < b->p.d) return PRAC_EINVAL;
  if (dw_dtype != PRAC_BF16 && dw_dtype != PRAC_F32) return PRAC_EINVAL;
  if (!b->have_u || !b->have_q) return PRAC_ESTATE;
  const GradLayout L = grad_layout(&b->p, N, d_out);
  if (!ws || ws_bytes < L.min_total) return PRAC_EWORKSPACE;
  if (!aligned256(ws)) return PRAC_EALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t d = b->p.d, k = b->p.k, s = b->s;
  const double c = std::isnan(c_override) ? b->c : c_override;
  char* w = static_cast<char*>(ws);
  const int out_t = dw_dtype == PRAC_BF16 ? ET_BF16 : ET_F32;
  int sc;
  if (b->p.dtype == PRAC_BF16 && tma_ok(Z, ldz) && (tma_ok(dY, lddy) || tc_tokens_takes_unaligned_a(d_out, s))) {
    // stage 1 on tensor cores: M' = (dY^T Z) diag(1, c), rounded to bf16 for stage 2
    // (rows of dY off the 16-byte grid go through TMA by classes of rows when the workspace has the
    // room the size query reports for that, else they are fetched with plain loads)
    __nv_bfloat16* Mb = reinterpret_cast<__nv_bfloat16*>(w + L.M);
    const int64_t ldm = round_up(s, 8);
    sc = tc_gemm_tokens(static_cast<const __nv_bfloat16*>(dY), lddy, static_cast<const __nv_bfloat16*>(Z), ldz,
                        d_out, s, N, Mb, ldm, ET_BF16, k, static_cast<float>(c), 0, nullptr, w + L.part,
                        ws_bytes - L.part < L.part_bytes ? ws_bytes - L.part : L.part_bytes,
                        b->status, st);
    if (sc != PRAC_OK) return sc;
    // stage 2: dW = M' [U | Q]^T
    if (!(accumulate && out_t == ET_BF16)) {
      return tc_gemm_kmajor(Mb, ldm, b->Pb, b->ldpb, d_out, d, s, dW, lddw, out_t, accumulate, b->status, st);
    }
    return gemm_general(gemm_args(d_out, d, s, Mb, ldm, ET_BF16, 0, b->P, s, ET_F32, 1, dW, lddw, out_t, 1.0, 1.0, 0), st);
  }
  const int et = elem_type(b->p.dtype);
  float* M = reinterpret_cast<float*>(w + L.M);
  sc = gemm_general(gemm_args(d_out, s, N, dY, lddy, et, 1, Z, ldz, et, 0, M, s, ET_F32, 1.0, 0.0, 0), st);
  if (sc != PRAC_OK) return sc;
  GemmArgs g = gemm_args(d_out, d, s, M, s, ET_F32, 0, b->P, s, ET_F32, 1, dW, lddw, out_t, 1.0,
                         accumulate ? 1.0 : 0.0, 0);
  g.kscale_from = k;
  g.kscale = c;
  return gemm_general(g, st);
}

int prac_reconstruct(const prac_basis* b, const void* Z, int64_t ldz, int64_t N, float* Xhat, int64_t ldxh,
                     void* stream) {
  if (!b || !Z || !Xhat || N <= 0 || ldz < b->s || ldxh < b->p.d) return PRAC_EINVAL;
  if (!b->have_u || !b->have_q) return PRAC_ESTATE;
  GemmArgs g = gemm_args(N, b->p.d, b->s, Z, ldz, elem_type(b->p.dtype), 0, b->P, b->s, ET_F32, 1, Xhat, ldxh,
                         ET_F32, 1.0, 0.0, 0);
  g.kscale_from = b->p.k;
  g.kscale = b->c;
  return gemm_general(g, static_cast<cudaStream_t>(stream));
}

int prac_activation_backward(const prac_basis* b, const void* Z, int64_t ldz, const void* dY, int64_t lddy, int64_t N,
                             int32_t act, void* dX, int64_t lddx, void* ws, size_t ws_bytes, void* stream) {
  if (!b || !Z || !dY || !dX || N <= 0 || ldz < b->s || lddy < b->p.d || lddx < b->p.d) return PRAC_EINVAL;
  if (act != PRAC_ACT_SILU && act != PRAC_ACT_GELU) return PRAC_EINVAL;
  if (!b->have_u || !b->have_q) return PRAC_ESTATE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t d = b->p.d, s = b->s;
  if (b->p.dtype == PRAC_BF16) {
    // X^ = Z [U | cQ]^T tile by tile in tensor memory; the epilogue multiplies f'(X^) into dY
    if (!tma_ok(Z, ldz) || !tc_consumer_takes_rows(dY, lddy, dX, lddx, N, d)) return PRAC_EALIGN;
    return tc_gemm_kmajor_act(static_cast<const __nv_bfloat16*>(Z), ldz, b->Pcb, b->ldpb, N, d, s,
                              static_cast<const __nv_bfloat16*>(dY), lddy, act, static_cast<__nv_bfloat16*>(dX), lddx,
                              b->status, st);
  }
  // fp32 storage: X^ into the workspace (N x d fp32), then the element-wise step
  const size_t need = static_cast<size_t>(N) * d * sizeof(float);
  if (!ws || ws_bytes < need) return PRAC_EWORKSPACE;
  if (!aligned256(ws)) return PRAC_EALIGN;
  float* Xh = static_cast<float*>(ws);
  const int sc = prac_reconstruct(b, Z, ldz, N, Xh, d, stream);
  if (sc != PRAC_OK) return sc;
  return launch_act_backward_f32(Xh, d, static_cast<const float*>(dY), lddy, static_cast<float*>(dX), lddx, N, d, act, st);
}

size_t prac_activation_workspace_bytes(const prac_params* p, int64_t N) {
  if (!params_ok(p) || N <= 0 || p->dtype == PRAC_BF16) return 0;
  return static_cast<size_t>(N) * p->d * sizeof(float);
}

namespace {
struct RmsLayout { size_t row_part, col_part, row_b, xh, total; int parts; int64_t blocks; };
RmsLayout rms_layout(const prac_params* p, int64_t N) {
  RmsLayout L{};
  Carver c;
  if (p->dtype == PRAC_BF16) {
    L.parts = tc_gemm_kmajor_rms_parts(p->d + 7, 8);     // room for the layouts taken by classes of rows
    L.blocks = (N + 31) / 32 + 8;
    L.row_part = c.take(static_cast<size_t>(L.parts) * N * sizeof(float));
    L.col_part = c.take(static_cast<size_t>(L.blocks) * p->d * sizeof(float));
    L.row_b = c.take(static_cast<size_t>(N) * sizeof(float));
  } else {
    L.xh = c.take(static_cast<size_t>(N) * p->d * sizeof(float));
  }
  L.total = c.off;
  return L;
}
}  // namespace

size_t prac_rmsnorm_workspace_bytes(const prac_params* p, int64_t N) {
  if (!params_ok(p) || N <= 0) return 0;
  return rms_layout(p, N).total;
}

int prac_rmsnorm_backward(const prac_basis* b, const void* Z, int64_t ldz, const void* dY, int64_t lddy, int64_t N,
                          const float* rstd, const float* gain, void* dX, int64_t lddx, float* dgain,
                          void* ws, size_t ws_bytes, void* stream) {
  if (!b || !Z || !dY || !dX || !rstd || !gain || !dgain || N <= 0) return PRAC_EINVAL;
  if (ldz < b->s || lddy < b->p.d || lddx < b->p.d) return PRAC_EINVAL;
  if (!b->have_u || !b->have_q) return PRAC_ESTATE;
  const RmsLayout L = rms_layout(&b->p, N);
  if (!ws || ws_bytes < L.total) return PRAC_EWORKSPACE;
  if (!aligned256(ws)) return PRAC_EALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t d = b->p.d, s = b->s;
  char* w = static_cast<char*>(ws);
  if (b->p.dtype == PRAC_BF16) {
    if (!tma_ok(Z, ldz) || !tc_consumer_takes_rows(dY, lddy, dX, lddx, N, d)) return PRAC_EALIGN;
    if (N <= 128 || d <= 128) return PRAC_EINVAL;    // the two passes run on CTA pairs only
    const int parts = tc_gemm_kmajor_rms_parts(d, lddy);            // what pass 1 writes for this layout of dY
    const int64_t blocks = tc_gemm_kmajor_rms_blocks(N, lddy);
    float* row_part = reinterpret_cast<float*>(w + L.row_part);
    float* col_part = reinterpret_cast<float*>(w + L.col_part);
    float* row_b = reinterpret_cast<float*>(w + L.row_b);
    const __nv_bfloat16* Zb = static_cast<const __nv_bfloat16*>(Z);
    const __nv_bfloat16* dYb = static_cast<const __nv_bfloat16*>(dY);
    // pass 1 over the rebuilt input: per-token sums of gain dY x and per-feature sums of rstd dY x
    int sc = tc_gemm_kmajor_rms(1, Zb, ldz, b->Pcb, b->ldpb, N, d, s, dYb, lddy, rstd, nullptr, gain, row_part, col_part,
                                nullptr, 0, b->status, st);
    if (sc != PRAC_OK) return sc;
    sc = launch_rms_reduce(row_part, parts, col_part, blocks, rstd, N, d, row_b, dgain, st);
    if (sc != PRAC_OK) return sc;
    // pass 2: dX = rstd gain dY - (rstd^3 u / d) x
    return tc_gemm_kmajor_rms(2, Zb, ldz, b->Pcb, b->ldpb, N, d, s, dYb, lddy, rstd, row_b, gain, nullptr, nullptr,
                              static_cast<__nv_bfloat16*>(dX), lddx, b->status, st);
  }
  float* Xh = reinterpret_cast<float*>(w + L.xh);
  const int sc = prac_reconstruct(b, Z, ldz, N, Xh, d, stream);
  if (sc != PRAC_OK) return sc;
  return launch_rms_backward_f32(Xh, d, static_cast<const float*>(dY), lddy, rstd, gain, static_cast<float*>(dX), lddx,
                                 dgain, N, d, st);
}

namespace {
struct LnLayout { size_t row_part, row_part2, col_part, row_b, row_c, plain, weighted, xh, total; int parts; int64_t blocks, groups; };
LnLayout ln_layout(const prac_params* p, int64_t N) {
  LnLayout L{};
  Carver c;
  if (p->dtype == PRAC_BF16) {
    L.parts = tc_gemm_kmajor_rms_parts(p->d + 7, 8);     // room for the layouts taken by classes of rows
    L.blocks = (N + 31) / 32 + 8;
    L.groups = (N + 511) / 512;
    L.row_part = c.take(static_cast<size_t>(L.parts) * N * sizeof(float));
    L.row_part2 = c.take(static_cast<size_t>(L.parts) * N * sizeof(float));
    L.col_part = c.take(static_cast<size_t>(L.blocks) * p->d * sizeof(float));
    L.row_b = c.take(static_cast<size_t>(N) * sizeof(float));
    L.row_c = c.take(static_cast<size_t>(N) * sizeof(float));
    L.plain = c.take(static_cast<size_t>(L.groups) * p->d * sizeof(float));
    L.weighted = c.take(static_cast<size_t>(L.groups) * p->d * sizeof(float));
  } else {
    L.xh = c.take(static_cast<size_t>(N) * p->d * sizeof(float));
  }
  L.total = c.off;
  return L;
}
}  // namespace

size_t prac_layernorm_workspace_bytes(const prac_params* p, int64_t N) {
  if (!params_ok(p) || N <= 0) return 0;
  return ln_layout(p, N).total;
}

int prac_layernorm_backward(const prac_basis* b, const void* Z, int64_t ldz, const void* dY, int64_t lddy, int64_t N,
                            const float* mean, const float* rstd, const float* gain, void* dX, int64_t lddx,
                            float* dgain, float* dbias, void* ws, size_t ws_bytes, void* stream) {
  if (!b || !Z || !dY || !dX || !mean || !rstd || !gain || !dgain || !dbias || N <= 0) return PRAC_EINVAL;
  if (ldz < b->s || lddy < b->p.d || lddx < b->p.d) return PRAC_EINVAL;
  if (!b->have_u || !b->have_q) return PRAC_ESTATE;
  const LnLayout L = ln_layout(&b->p, N);
  if (!ws || ws_bytes < L.total) return PRAC_EWORKSPACE;
  if (!aligned256(ws)) return PRAC_EALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t d = b->p.d, s = b->s;
  char* w = static_cast<char*>(ws);
  if (b->p.dtype == PRAC_BF16) {
    if (!tma_ok(Z, ldz) || !tc_consumer_takes_rows(dY, lddy, dX, lddx, N, d)) return PRAC_EALIGN;
    if (N <= 128 || d <= 128) return PRAC_EINVAL;    // the two passes run on CTA pairs only
    const int parts = tc_gemm_kmajor_rms_parts(d, lddy);            // what pass 1 writes for this layout of dY
    const int64_t blocks = tc_gemm_kmajor_rms_blocks(N, lddy);
    float* row_part = reinterpret_cast<float*>(w + L.row_part);
    float* row_part2 = reinterpret_cast<float*>(w + L.row_part2);
    float* col_part = reinterpret_cast<float*>(w + L.col_part);
    float* row_b = reinterpret_cast<float*>(w + L.row_b);
    float* row_c = reinterpret_cast<float*>(w + L.row_c);
    float* plain = reinterpret_cast<float*>(w + L.plain);
    float* weighted = reinterpret_cast<float*>(w + L.weighted);
    const __nv_bfloat16* Zb = static_cast<const __nv_bfloat16*>(Z);
    const __nv_bfloat16* dYb = static_cast<const __nv_bfloat16*>(dY);
    // what does not need the rebuilt input: per-feature sums of dY and of rstd mean dY
    int sc = launch_ln_colsum_partial(dYb, lddy, mean, rstd, N, d, plain, weighted, st);
    if (sc != PRAC_OK) return sc;
    // pass 1: per-token sums of gain dY x and gain dY, per-feature sums of rstd dY x
    sc = tc_gemm_kmajor_rms(1, Zb, ldz, b->Pcb, b->ldpb, N, d, s, dYb, lddy, rstd, nullptr, gain, row_part, col_part,
                            nullptr, 0, b->status, st, row_part2, nullptr);
    if (sc != PRAC_OK) return sc;
    sc = launch_ln_reduce(row_part, row_part2, parts, col_part, blocks, plain, weighted, L.groups, mean, rstd, N, d,
                          row_b, row_c, dgain, dbias, st);
    if (sc != PRAC_OK) return sc;
    // pass 2: dX = rstd gain dY - row_b x + row_c
    return tc_gemm_kmajor_rms(2, Zb, ldz, b->Pcb, b->ldpb, N, d, s, dYb, lddy, rstd, row_b, gain, nullptr, nullptr,
                              static_cast<__nv_bfloat16*>(dX), lddx, b->status, st, nullptr, row_c);
  }
  float* Xh = reinterpret_cast<float*>(w + L.xh);
  const int sc = prac_reconstruct(b, Z, ldz, N, Xh, d, stream);
  if (sc != PRAC_OK) return sc;
  return launch_ln_backward_f32(Xh, d, static_cast<const float*>(dY), lddy, mean, rstd, gain, static_cast<float*>(dX),
                                lddx, dgain, dbias, N, d, st);
}

int prac_fit_report(const prac_basis* b, void* ws, size_t ws_bytes, int64_t N, void* stream, prac_fit_info* out) {
  if (!b || !out || N <= 0) return PRAC_EINVAL;
  std::memset(out, 0, sizeof(*out));
  out->panel_cols = static_cast<int32_t>(b->ell);
  out->iterations = b->iters;
  if (b->p.k == 0) return PRAC_OK;
  if (!b->last_fit_eig) return PRAC_OK;     // a warm refresh: no eigenproblem was solved
  const RitzWindow win = ritz_window(b->p.k, b->ell);
  out->eig_size = static_cast<int32_t>(win.n);
  out->window_first = static_cast<int32_t>(win.first);
  const FitLayout L = fit_layout(&b->p, N);
  if (!ws || ws_bytes < L.total) return PRAC_EWORKSPACE;
  int sweeps = 0;
  const int sc = jacobi_read_sweeps(static_cast<char*>(ws) + L.jac, win.n, &sweeps, static_cast<cudaStream_t>(stream));
  if (sc != PRAC_OK) return sc;
  out->jacobi_sweeps = sweeps;
  return PRAC_OK;
}

int prac_device_status(prac_basis* b, void* stream) {
  if (!b) return PRAC_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  PRAC_CUDA_TRY(cudaStreamSynchronize(st));
  int h = 0;
  PRAC_CUDA_TRY(cudaMemcpy(&h, b->status, sizeof(int), cudaMemcpyDeviceToHost));
  if (h == 0) return PRAC_OK;
  PRAC_CUDA_TRY(cudaMemset(b->status, 0, sizeof(int)));
  if (h & DEV_WAIT_EXPIRED) return PRAC_ETIMEOUT;
  return PRAC_ENUMERIC;
}

int prac_philox_words(uint64_t seed, uint64_t draw_counter, int64_t n, uint32_t* out, void* stream) {
  if (n < 0 || (n > 0 && !out)) return PRAC_EINVAL;
  return launch_philox_words(seed, draw_counter, n, out, static_cast<cudaStream_t>(stream));
}

int prac_gaussian(uint64_t seed, uint64_t draw_counter, int64_t d, int64_t r, float* S, int64_t lds,
                  void* stream) {
  if (d < 0 || r < 0 || lds < r || (d * r > 0 && !S)) return PRAC_EINVAL;
  return launch_gaussian(seed, draw_counter, d, r, S, lds, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
