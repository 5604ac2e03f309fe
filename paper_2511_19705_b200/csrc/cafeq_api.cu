// C-ABI entry points of the CafeQ optimisation path (declared in include/cafeq.h).
// Host side only validates arguments, carves the caller's workspace and enqueues kernels.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#include <atomic>
#include <mutex>
#include <vector>

#include "cafeq.h"
#include "kernels_generic.cuh"
#include "kernels_fused.cuh"
#include "kernels_bwd.cuh"
#include "kernels_gemm.cuh"
#include "kernels_dense.cuh"
#include "kernels_rtn.cuh"

namespace cafeq {

// Process-wide count of kernel launches made by this library (read by benchmarks through
// cafeq_debug_launch_count; it has no effect on any result).
static std::atomic<long long> g_launches{0};
#define CQ_LAUNCH(kernel, grid, block, smem, st, ...)       \
  do {                                                      \
    g_launches.fetch_add(1, std::memory_order_relaxed);     \
    kernel<<<grid, block, smem, st>>>(__VA_ARGS__);         \
  } while (0)

// Optional per-launch timing of selected kernels with CUDA events on the launching stream (benchmarks
// only; off unless cafeq_debug_timer_begin was called).  Kinds: 1 transform pass (shape-agnostic kernels),
// 2 sparse backward, 3 block inverse, 4 dense pair product, 5 fused tensor-core transform pass.
struct KernelTimer {
  std::vector<cudaEvent_t> a, b;
  std::vector<int> kind;
  int used = 0;
  bool on = false;
};
static KernelTimer g_kt;
static inline int kt_begin(int kind, cudaStream_t st) {
  if (!g_kt.on || g_kt.used >= (int)g_kt.a.size()) return -1;
  int i = g_kt.used++;
  g_kt.kind[i] = kind;
  cudaEventRecord(g_kt.a[i], st);
  return i;
}
static inline void kt_end(int i, cudaStream_t st) {
  if (i >= 0) cudaEventRecord(g_kt.b[i], st);
}

// ------------------------------------------------------------------------------------------------
// workspace carving
// ------------------------------------------------------------------------------------------------
struct Bump {
  char* base;
  size_t cap, used;
  bool overflow;
  Bump(void* b, size_t c) : base((char*)b), cap(c), used(0), overflow(false) {}
  // (base == nullptr: nothing is handed out, `used` still adds up -- the size queries run the same carving code)
  template <typename T>
  T* take(size_t count) {
    size_t bytes = (count * sizeof(T) + 255) & ~(size_t)255;
    if (!base || used + bytes > cap) { overflow = true; used += bytes; return nullptr; }
    T* p = (T*)(base + used);
    used += bytes;
    return p;
  }
};

static inline int grid_for(long long n, int threads = 256, int cap = 148 * 16) {
  long long b = (n + threads - 1) / threads;
  if (b < 1) b = 1;
  if (b > cap) b = cap;
  return (int)b;
}

static inline float qmax_of(int bits) { return (float)((1 << (bits - 1)) - 1); }

struct Geo {  // derived geometry of one descriptor
  int d_out, d_in, g, ng, k, r, axis, nbq, nbT;
  long long ld, n;
};

static int make_geo(const cafeq_matrix_desc* d, Geo* o, bool need_transform) {
  if (!d || d->struct_size != sizeof(cafeq_matrix_desc)) return CAFEQ_ERR_INVALID_ARG;
  if (d->d_out <= 0 || d->d_in <= 0 || d->ld < d->d_in) return CAFEQ_ERR_INVALID_ARG;
  if (d->bits < 2 || d->bits > 8) return CAFEQ_ERR_INVALID_ARG;
  if (d->group < 0 || d->tblock < 0 || d->replicas < 1) return CAFEQ_ERR_INVALID_ARG;
  if (d->taxis != CAFEQ_AXIS_IN && d->taxis != CAFEQ_AXIS_OUT) return CAFEQ_ERR_INVALID_ARG;
  if (d->compute_prec != CAFEQ_PREC_BF16) return CAFEQ_ERR_UNSUPPORTED;
  o->d_out = d->d_out;
  o->d_in = d->d_in;
  o->ld = d->ld;
  o->n = (long long)d->d_out * d->d_in;
  o->g = d->group ? d->group : d->d_in;
  if (d->d_in % o->g) return CAFEQ_ERR_INVALID_ARG;
  o->ng = d->d_in / o->g;
  o->k = d->tblock;
  o->r = d->replicas;
  o->axis = d->taxis;
  o->nbq = 0;
  o->nbT = 0;
  if (o->k > 0) {
    int dim = (o->axis == CAFEQ_AXIS_IN) ? d->d_in : d->d_out;
    if (dim % o->k) return CAFEQ_ERR_INVALID_ARG;
    o->nbq = dim / o->k;
    if (o->nbq % o->r) return CAFEQ_ERR_INVALID_ARG;
    o->nbT = o->nbq / o->r;
    if (o->k > 1024) return CAFEQ_ERR_UNSUPPORTED;
  } else if (need_transform) {
    return CAFEQ_ERR_INVALID_ARG;
  }
  return CAFEQ_OK;
}

// ------------------------------------------------------------------------------------------------
// launch helpers
// ------------------------------------------------------------------------------------------------
static void launch_gemm(cudaStream_t st, const GemmArgs& g) {
  dim3 grid((g.N + 63) / 64, (g.M + 63) / 64, g.batch);
  if (g.a_bf16 && g.b_bf16) CQ_LAUNCH((gemm_kernel<true, true>), grid, 256, 0, st, g);
  else if (g.a_bf16) CQ_LAUNCH((gemm_kernel<true, false>), grid, 256, 0, st, g);
  else if (g.b_bf16) CQ_LAUNCH((gemm_kernel<false, true>), grid, 256, 0, st, g);
  else CQ_LAUNCH((gemm_kernel<false, false>), grid, 256, 0, st, g);
}

static GemmArgs gemm_defaults(const int32_t* status) {
  GemmArgs g;
  memset(&g, 0, sizeof(g));
  g.divA = g.divB = g.divC = 1;
  g.alpha = 1.f;
  g.mode = GEMM_STORE;
  g.batch = 1;
  g.status = status;
  return g;
}

// Out = T o X along `axis`; X is bf16 (x_bf16) or fp32; T fp32 blocks [nbT,k,k]; transposed uses T^T.
static void launch_apply(cudaStream_t st, const void* X, int x_bf16, long long ldx, const Geo& G, const float* T,
                         int transposed, float* Out, long long ldo, int mode, double* sq, const int32_t* status,
                         float alpha = 1.f) {
  GemmArgs g = gemm_defaults(status);
  const int k = G.k;
  g.alpha = alpha;
  g.C = Out;
  g.mode = mode;
  g.sq = sq;
  g.batch = G.nbq;
  if (G.axis == CAFEQ_AXIS_IN) {
    g.M = G.d_out; g.N = k; g.K = k;
    g.A = X; g.a_bf16 = x_bf16; g.sAm = ldx; g.sAk = 1; g.sAb = k;
    g.B = T; g.b_bf16 = 0; g.sBb = (long long)k * k; g.divB = G.r;
    if (!transposed) { g.sBk = 1; g.sBn = k; } else { g.sBk = k; g.sBn = 1; }
    g.sCm = ldo; g.sCn = 1; g.sCb = k;
  } else {
    g.M = k; g.N = G.d_in; g.K = k;
    g.A = T; g.a_bf16 = 0; g.sAb = (long long)k * k; g.divA = G.r;
    if (!transposed) { g.sAm = k; g.sAk = 1; } else { g.sAm = 1; g.sAk = k; }
    g.B = X; g.b_bf16 = x_bf16; g.sBk = ldx; g.sBn = 1; g.sBb = (long long)k * ldx;
    g.sCm = ldo; g.sCn = 1; g.sCb = (long long)k * ldo;
  }
  int ti = kt_begin(1, st);
  launch_gemm(st, g);
  kt_end(ti, st);
}

// gT[b / r][i][j] += alpha * sum_free Gm[.., i] X[.., j]  (atomic accumulation; caller zeroes gT)
static void launch_opgrad(cudaStream_t st, const float* Gm, long long ldg, const void* X, int x_bf16, long long ldx,
                          const Geo& G, float* gT, int transpose_out, float alpha, const int32_t* status) {
  GemmArgs g = gemm_defaults(status);
  const int k = G.k;
  g.M = k; g.N = k; g.batch = G.nbq;
  g.A = Gm; g.a_bf16 = 0;
  g.B = X; g.b_bf16 = x_bf16;
  g.C = gT; g.sCb = (long long)k * k; g.divC = G.r;
  if (!transpose_out) { g.sCm = k; g.sCn = 1; } else { g.sCm = 1; g.sCn = k; }
  g.alpha = alpha;
  g.mode = GEMM_STORE | GEMM_ATOMIC;
  if (G.axis == CAFEQ_AXIS_IN) {
    g.K = G.d_out;
    g.sAm = 1; g.sAk = ldg; g.sAb = k;
    g.sBk = ldx; g.sBn = 1; g.sBb = k;
  } else {
    g.K = G.d_in;
    g.sAm = ldg; g.sAk = 1; g.sAb = (long long)k * ldg;
    g.sBk = 1; g.sBn = ldx; g.sBb = (long long)k * ldx;
  }
  launch_gemm(st, g);
}

// C[b] (op)= alpha * opA(A[b]) * opB(B[b]) for k x k blocks
static void launch_kk(cudaStream_t st, const float* A, int tA, const float* B, int tB, float* C, int nb, int k, float alpha,
                      int mode, const int32_t* status) {
  GemmArgs g = gemm_defaults(status);
  g.M = g.N = g.K = k;
  g.batch = nb;
  g.A = A; g.B = B; g.C = C;
  g.sAb = g.sBb = g.sCb = (long long)k * k;
  if (!tA) { g.sAm = k; g.sAk = 1; } else { g.sAm = 1; g.sAk = k; }
  if (!tB) { g.sBk = k; g.sBn = 1; } else { g.sBk = 1; g.sBn = k; }
  g.sCm = k; g.sCn = 1;
  g.alpha = alpha;
  g.mode = mode;
  launch_gemm(st, g);
}

static void launch_inverse(cudaStream_t st, const float* Mc, float* Minv, float* cnorm, int nb, int k, int32_t* status,
                           const double* rn_check = nullptr, double tol2 = 0.0, int* redo_flag = nullptr, int* redo_count = nullptr) {
  int threads = k * k >= 1024 ? 1024 : ((k * k + 31) / 32) * 32;
  size_t sh = (size_t)3 * k * sizeof(float);
  int ti = rn_check ? -1 : kt_begin(3, st);
  CQ_LAUNCH(block_inverse_kernel, nb, threads, sh, st, Mc, Minv, cnorm, k, status, rn_check, tol2, redo_flag, redo_count);
  kt_end(ti, st);
}

// ------------------------------------------------------------------------------------------------
// k x k algebra on the tensor cores: split-precision products and the Newton-Schulz inverse
// ------------------------------------------------------------------------------------------------
struct KkWS {  // bf16 scratch, each [nbT * k * k]
  uint16_t *Ab, *Xh[2], *Xl[2], *XTh[2], *XTl[2], *RTh, *RTl, *Ph, *Pl, *Qh, *Ql;
  double* rn;  // [NS_MAX_ITERS][nbT] squared residual norms
  int* flag;   // 1 => Newton-Schulz did not converge, the Gauss-Jordan kernel takes over
  int* redo_total;  // optional running count of blocks recomputed by elimination (never cleared by a step)
  int cur;     // which of the ping-pong split sets holds the current inverse (host bookkeeping)
  bool mn;     // the inverse was refined on row-major arrays only (whole-block products with MN-major operands): the
               // transposed splits XTh / XTl are not maintained
};
constexpr int NS_MAX_ITERS = 8;
constexpr int NS_COLD_ITERS = 6;
constexpr int NS_WARM_ITERS = 4;  // upper bound: converged blocks skip the later ones (see ns_inverse)

static bool kk_fast(int k) { return k == 64 || k == 128 || k == 256; }

static void carve_kk(Bump& b, int nbT, int k, KkWS* w) {
  const size_t kk = (size_t)nbT * k * k;
  uint16_t** all[] = {&w->Ab, &w->Xh[0], &w->Xh[1], &w->Xl[0], &w->Xl[1], &w->XTh[0], &w->XTh[1], &w->XTl[0], &w->XTl[1],
                      &w->RTh, &w->RTl, &w->Ph, &w->Pl, &w->Qh, &w->Ql};
  for (auto pp : all) *pp = b.take<uint16_t>(kk);
  w->rn = b.take<double>((size_t)NS_MAX_ITERS * nbT);
  w->flag = b.take<int>(64);
  w->redo_total = nullptr;
  w->cur = 0;
  w->mn = false;
}

// C[b] = alpha * sum_t A_t[b] B_t[b]^T + beta * C0[b] + gamma * I for nb blocks of k x k; operands bf16 [nb*k, k]
static int launch_kk_tc(cudaStream_t st, int nterms, const uint16_t* const* A, const uint16_t* const* B, int nb, int k,
                        float alpha, float beta, float gamma, const float* C0, float* C, uint16_t* Chi, uint16_t* Clo,
                        uint16_t* Cthi, uint16_t* Ctlo, double* sq, const int* run_flag, int32_t* status, int sq_stride = 1,
                        const double* gate = nullptr, double gate_tol = 0.0, int a_mn = 0, int b_mn = 0) {
  TgOperand oa[TG_MAX_TERMS], ob[TG_MAX_TERMS];
  for (int t = 0; t < nterms; ++t) {
    oa[t] = TgOperand{A[t], (long long)nb * k, k, k};
    ob[t] = TgOperand{B[t], (long long)nb * k, k, k};
  }
  TgParams p;
  memset(&p, 0, sizeof(p));
  p.M = p.N = p.K = k;
  p.batch = nb;
  p.nterms = nterms;
  p.rowsA_per_batch = p.rowsB_per_batch = k;
  p.divA = 1;
  p.a_rep_k = k;
  p.a_rep_r = 1;
  p.alpha = alpha; p.beta = beta; p.gamma = gamma;
  p.C0 = C0; p.ldc0 = k; p.sC0b = (long long)k * k;
  p.C = C; p.ldc = k; p.sCb = (long long)k * k;
  p.Chi = Chi; p.Clo = Clo; p.Cthi = Cthi; p.Ctlo = Ctlo;
  p.sq = sq; p.sq_stride = sq_stride;
  p.run_flag = run_flag;
  p.gate = gate;
  p.gate_tol = gate_tol;
  p.status = status;
  g_launches.fetch_add(1, std::memory_order_relaxed);
  if (g_tb_enable.load(std::memory_order_relaxed) && tb_supported(k, nterms)) {
    const int rc = tb_launch(st, nterms, A, B, a_mn, b_mn, (long long)nb * k, (long long)nb * k, k, p);
    if (rc != CAFEQ_ERR_UNSUPPORTED) return rc;
  }
  if (a_mn || b_mn) return CAFEQ_ERR_UNSUPPORTED;  // the tiled kernel takes K-major operands only
  return tg_launch(st, oa, ob, p);
}

__global__ void transpose_blocks_kernel(const float* __restrict__ in, float* __restrict__ out, int k, long long n) {
  const long long kk = (long long)k * k;
  for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
    const long long b = e / kk, r = e - b * kk;
    const int i = (int)(r / k), j = (int)(r - (long long)i * k);
    out[e] = in[b * kk + (long long)j * k + i];
  }
}

__global__ void zero_ns_kernel(double* rn, int n, int* flag) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) rn[i] = 0.0;
  if (i == 0) *flag = 0;
}

// c[b][t] = sum_i X[b][i][t]^2
__global__ void colnorm_kernel(const float* __restrict__ X, int k, int nb, float* __restrict__ c) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  const int b = blockIdx.y;
  if (t >= k || b >= nb) return;
  const float* Xb = X + (size_t)b * k * k;
  float s = 0.f;
  for (int i = 0; i < k; ++i) {
    const float v = Xb[(size_t)i * k + t];
    s = fmaf(v, v, s);
  }
  c[(size_t)b * k + t] = s;
}

static void launch_split(cudaStream_t st, const float* X, int k, long long n, uint16_t* hi, uint16_t* lo, uint16_t* thi,
                         uint16_t* tlo, const int* run_flag, const int32_t* status, const double* gate = nullptr,
                         double gate_tol = 0.0, int parity_iters = 0, int parity_nb = 0) {
  dim3 grid(k / 32, k / 32, (unsigned)(n / ((long long)k * k)));
  CQ_LAUNCH(split_bf16_kernel, grid, dim3(32, 8), 0, st, X, k, hi, lo, thi, tlo, run_flag, status, gate, gate_tol, parity_iters,
            parity_nb);
}

// Minv = inv(bf16(M)) by Newton-Schulz iteration X <- X + X (I - A X) on the tensor cores, from X0 = A^T
// (cold: right for the near-orthogonal transforms the method starts from) or from the caller's previous
// inverse (warm).  The last residual is checked on the device; if it is not small the Gauss-Jordan kernel
// recomputes everything.  Leaves fp32 Minv in X, its bf16 splits in w.Xh/Xl/XTh/XTl[w.cur], and c = column
// square norms of Minv (optional).
static void ns_inverse(cudaStream_t st, const float* Mc, float* X, float* cnorm, int nb, int k, bool warm, KkWS& w,
                       int32_t* status, bool prepped = false, bool splits_kept = false) {
  const long long kk = (long long)nb * k * k;
  const int iters = warm ? NS_WARM_ITERS : NS_COLD_ITERS;
  // A warm start runs up to NS_WARM_ITERS iterations, as many as the step size calls for: a block whose residual
  // ||I - A X||_F was below 1e-2 before an update (below 1e-4 after it) skips the iterations that follow (their CTAs
  // return at once).  Small steps take one or two iterations, a change of the transform by half its norm four.
  constexpr double NS_GATE2 = 1e-4;  // squared: the same bound the acceptance test below puts on the residual before the last update
  int ti = kt_begin(3, st);
  if (!prepped) {  // otherwise step_prep_kernel has cleared rn / flag and written Ab
    CQ_LAUNCH(zero_ns_kernel, (NS_MAX_ITERS * nb + 127) / 128, 128, 0, st, w.rn, NS_MAX_ITERS * nb, w.flag);
    CQ_LAUNCH(operator_to_bf16_kernel, grid_for(kk), 256, 0, st, Mc, w.Ab, k, kk, 0, status);
  }
  if (!warm) CQ_LAUNCH(transpose_blocks_kernel, grid_for(kk), 256, 0, st, Mc, X, k, kk);
  int cur = 0;
  // Block sizes with the whole-block product kernel run the iteration on row-major arrays only (MN-major operands):
  // no transposed split of X or R is written.
  const bool mn = g_tb_enable.load(std::memory_order_relaxed) && tb_supported(k, 2);
  w.mn = mn;
  // (splits_kept: the splits of X that the previous call left in set 0 are still there)
  if (!(warm && splits_kept)) {
    if (mn) launch_split(st, X, k, kk, w.Xh[cur], w.Xl[cur], nullptr, nullptr, nullptr, status);
    else launch_split(st, X, k, kk, w.Xh[cur], iters > 0 ? nullptr : w.Xl[cur], w.XTh[cur], w.XTl[cur], nullptr, status);
  }
  for (int it = 0; it < iters; ++it) {
    const double* gate = (warm && it > 0) ? w.rn + (size_t)(it - 1) * nb : nullptr;
    // R = I - A X needs X to full precision (the product cancels against I): two terms over the split of X.
    // X += X R: the correction is small and the iteration corrects its own errors, so one bf16 term is enough
    // (the error it leaves is 2^-8 |R| relative, below 4e-5 for every accepted residual).
    const uint16_t* a1[2] = {w.Ab, w.Ab};
    const uint16_t* a2[1] = {w.Xh[cur]};
    if (mn) {
      const uint16_t* b1[2] = {w.Xh[cur], w.Xl[cur]};  // X stored [l][n]
      launch_kk_tc(st, 2, a1, b1, nb, k, -1.f, 0.f, 1.f, nullptr, nullptr, w.RTh, nullptr, nullptr, nullptr, w.rn + (size_t)it * nb,
                   nullptr, status, 1, gate, NS_GATE2, 0, 1);
      const uint16_t* b2[1] = {w.RTh};                  // bf16(R), row-major here
      launch_kk_tc(st, 1, a2, b2, nb, k, 1.f, 1.f, 0.f, X, X, w.Xh[cur ^ 1], w.Xl[cur ^ 1], nullptr, nullptr, nullptr, nullptr, status,
                   1, gate, NS_GATE2, 0, 1);
    } else {
      const uint16_t* b1[2] = {w.XTh[cur], w.XTl[cur]};
      launch_kk_tc(st, 2, a1, b1, nb, k, -1.f, 0.f, 1.f, nullptr, nullptr, nullptr, nullptr, w.RTh, nullptr, w.rn + (size_t)it * nb,
                   nullptr, status, 1, gate, NS_GATE2);
      const uint16_t* b2[1] = {w.RTh};
      // (the row-major low half is only read after the last iteration, by the M^-1 path of the gradient)
      launch_kk_tc(st, 1, a2, b2, nb, k, 1.f, 1.f, 0.f, X, X, w.Xh[cur ^ 1], (it == iters - 1) ? w.Xl[cur ^ 1] : nullptr,
                   w.XTh[cur ^ 1], w.XTl[cur ^ 1], nullptr, nullptr, status, 1, gate, NS_GATE2);
    }
    cur ^= 1;
  }
  w.cur = cur;
  // accept when ||I - A X||_F before the last update was below 1e-2 (the update squares it: <= 1e-4 after); a block
  // that skipped the last iteration has a zero there and was accepted by the gate
  launch_inverse(st, Mc, X, nullptr, nb, k, status, w.rn + (size_t)(iters - 1) * nb, 1e-4, w.flag, w.redo_total);
  // final splits: written by the last iteration's epilogue, except for blocks that skipped it (and for everything
  // when the elimination recomputed a block)
  if (mn) {
    // every iteration writes both row-major splits, so a block that stopped early needs this only when its newest
    // splits are in the other set
    launch_split(st, X, k, kk, w.Xh[cur], w.Xl[cur], nullptr, nullptr, w.flag, status, (warm && iters > 1) ? w.rn : nullptr, NS_GATE2,
                 iters, nb);
  } else {
    const double* last_gate = (warm && iters > 1) ? w.rn + (size_t)(iters - 2) * nb : nullptr;
    launch_split(st, X, k, kk, w.Xh[cur], w.Xl[cur], w.XTh[cur], w.XTl[cur], w.flag, status, last_gate, NS_GATE2);
  }
  if (cnorm) {
    dim3 grid((k + 127) / 128, nb);
    CQ_LAUNCH(colnorm_kernel, grid, 128, 0, st, X, k, nb, cnorm);
  }
  kt_end(ti, st);
}

// G (op)= -X^T Gx X^T for every block, on the tensor cores with three-term bf16 splits; X = Minv with its
// splits in w[w.cur]; Gx fp32 [nb,k,k] (dL/dMinv).  G += result when accumulate, else G = result.
static void minv_path_tc(cudaStream_t st, const float* Gx, float* G, int nb, int k, bool accumulate, KkWS& w, int32_t* status) {
  const long long kk = (long long)nb * k * k;
  const int c = w.cur;
  if (w.mn) {
    // T1 = X^T Gx with both operands read from their row-major arrays: A_op[i][l] = X[l][i], B_op[j][l] = Gx[l][j]
    launch_split(st, Gx, k, kk, w.Ph, w.Pl, nullptr, nullptr, nullptr, status);
    const uint16_t* a1[3] = {w.Xh[c], w.Xl[c], w.Xh[c]};
    const uint16_t* b1[3] = {w.Ph, w.Ph, w.Pl};
    launch_kk_tc(st, 3, a1, b1, nb, k, 1.f, 0.f, 0.f, nullptr, nullptr, w.Qh, w.Ql, nullptr, nullptr, nullptr, nullptr, status, 1, nullptr,
                 0.0, 1, 1);
  } else {
    launch_split(st, Gx, k, kk, nullptr, nullptr, w.Ph, w.Pl, nullptr, status);  // Gx^T splits
    // T1 = X^T Gx : T1[i][j] = sum_l XT[i][l] * GxT[j][l]
    const uint16_t* a1[3] = {w.XTh[c], w.XTl[c], w.XTh[c]};
    const uint16_t* b1[3] = {w.Ph, w.Ph, w.Pl};
    launch_kk_tc(st, 3, a1, b1, nb, k, 1.f, 0.f, 0.f, nullptr, nullptr, w.Qh, w.Ql, nullptr, nullptr, nullptr, nullptr, status);
  }
  // G -= T1 X^T : [i][j] = sum_l T1[i][l] * X[j][l]
  const uint16_t* a2[3] = {w.Qh, w.Ql, w.Qh};
  const uint16_t* b2[3] = {w.Xh[c], w.Xh[c], w.Xl[c]};
  launch_kk_tc(st, 3, a2, b2, nb, k, -1.f, accumulate ? 1.f : 0.f, 0.f, accumulate ? G : nullptr, G, nullptr, nullptr, nullptr,
               nullptr, nullptr, nullptr, status);
}

static void launch_absmax(cudaStream_t st, const float* U, long long ld, const Geo& G, float* a, float* usel, int* idx,
                          int32_t* status) {
  long long warps = (long long)G.d_out * G.ng;
  long long blocks = (warps * 32 + 255) / 256;
  CQ_LAUNCH(absmax_kernel, (unsigned)blocks, 256, 0, st, U, ld, G.d_out, G.ng, G.g, a, usel, idx, status);
}

// gm: the (row, group) records are group-major (written by the fused pass) instead of row-major
static void launch_scatter(cudaStream_t st, const void* W, const Geo& G, const float* coef, const int* idx, float* gT,
                           int transpose_out, const int32_t* status, int gm) {
  const int k = G.k;
  int ti = kt_begin(2, st);
  // block sizes 128 / 256: a dense product on the tensor cores whose left operand holds the routed coefficients
  if (bw_supported(G.axis == CAFEQ_AXIS_IN, G.d_out, G.d_in, G.ld, k, G.g, W)) {
    BwParams bp;
    memset(&bp, 0, sizeof(bp));
    bp.d_out = G.d_out; bp.d_in = G.d_in; bp.g = G.g; bp.ng = G.ng; bp.r = G.r;
    bp.gm = gm; bp.transpose_out = transpose_out;
    bp.coef = coef; bp.idx = idx; bp.gradT = gT;
    bp.status = const_cast<int32_t*>(status);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (bw_launch(st, G.axis == CAFEQ_AXIS_IN, k, W, G.ld, bp) == CAFEQ_OK) {
      kt_end(ti, st);
      return;
    }
    g_launches.fetch_sub(1, std::memory_order_relaxed);
  }
  const bool aligned = ((uintptr_t)W % 4 == 0) && (G.ld % 2 == 0);
  const int nG = (k >= G.g) ? k / G.g : 1;  // groups of one row inside one block (g | k or k | g on this path)
  if (kk_fast(k) && G.axis == CAFEQ_AXIS_IN && (k % G.g == 0 || G.g % k == 0) && nG <= 8 && ((uintptr_t)W % 16 == 0) &&
      (G.ld % 8 == 0)) {
    // 8 strip columns per thread at least: strip 32 at k = 256 (one thread per target row), 64 otherwise
    const int strip = (k == 256) ? 32 : 64;
    const int strips = k / strip;
    int rows_per = SCB_MAXP / nG;
    if (rows_per > 2048) rows_per = 2048;
    // enough CTAs to fill the machine a few times over, but never more rows than the record buffer holds
    int want = (148 * 4 + G.nbq * strips - 1) / (G.nbq * strips);
    int rp2 = (G.d_out + want - 1) / want;
    rp2 = ((rp2 + 31) / 32) * 32;
    if (rp2 < rows_per) rows_per = rp2;
    if (rows_per < 32) rows_per = 32;
    const int splits = (G.d_out + rows_per - 1) / rows_per;
    dim3 grid(G.nbq, strips, splits);
    const size_t sh = (size_t)k * (strip + 1) * 4 + (size_t)SCB_MAXP * 6;
    {  // the attribute is per device: set it on every call (cheap)
      cudaFuncSetAttribute(scatter_in_bucket_kernel<256, 32>, cudaFuncAttributeMaxDynamicSharedMemorySize, 256 * 33 * 4 + SCB_MAXP * 6);
      cudaFuncSetAttribute(scatter_in_bucket_kernel<128, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * 65 * 4 + SCB_MAXP * 6);
      cudaFuncSetAttribute(scatter_in_bucket_kernel<64, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 65 * 4 + SCB_MAXP * 6);
    }
#define SC_INB(KV, SV)                                                                                                   \
  CQ_LAUNCH((scatter_in_bucket_kernel<KV, SV>), grid, 256, sh, st, (const uint16_t*)W, G.ld, G.d_out, G.d_in, G.g, G.r, nG, coef, \
            idx, gT, transpose_out, rows_per, status, gm)
    if (k == 64) SC_INB(64, 64);
    else if (k == 128) SC_INB(128, 64);
    else SC_INB(256, 32);
#undef SC_INB
    kt_end(ti, st);
    return;
  }
  if (k % SC2_JS == 0 && k <= 256 && aligned && G.axis == CAFEQ_AXIS_IN && (k % G.g == 0 || G.g % k == 0) &&
      (nG == 1 || nG == 2 || nG == 4)) {
    {
      cudaFuncSetAttribute(scatter_in_strip_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 256 * SC2_JS * 4);
      cudaFuncSetAttribute(scatter_in_strip_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 256 * SC2_JS * 4);
      cudaFuncSetAttribute(scatter_in_strip_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 256 * SC2_JS * 4);
    }
    const int strips = k / SC2_JS;
    int splits = (148 * 3 + G.nbq * strips - 1) / (G.nbq * strips);
    if (splits < 1) splits = 1;
    int rows_per = (G.d_out + splits - 1) / splits;
    rows_per = ((rows_per + 31) / 32) * 32;
    splits = (G.d_out + rows_per - 1) / rows_per;
    dim3 grid(G.nbq, strips, splits);
    const size_t sh = (size_t)k * SC2_JS * 4;
#define SC_IN(NGV)                                                                                                       \
  CQ_LAUNCH(scatter_in_strip_kernel<NGV>, grid, 256, sh, st, (const uint16_t*)W, G.ld, G.d_out, G.d_in, G.g, k, G.r, coef, idx, \
            gT, transpose_out, rows_per, status, gm)
    if (nG == 1) SC_IN(1);
    else if (nG == 2) SC_IN(2);
    else SC_IN(4);
#undef SC_IN
    kt_end(ti, st);
    return;
  }
  if (kk_fast(k) && G.g % 4 == 0 && G.g <= 128 && ((uintptr_t)W % 8 == 0) && (G.ld % 4 == 0) && G.axis == CAFEQ_AXIS_OUT) {
    const int strips = k / SC2_JS;
    int splits = (148 * 4 + G.nbq * strips - 1) / (G.nbq * strips);
    if (splits < 1) splits = 1;
    int per = (G.ng + splits - 1) / splits;
    splits = (G.ng + per - 1) / per;
    dim3 grid(G.nbq, strips, splits);
    const size_t sh = (size_t)2 * SC2_JS * (G.g + 4) * 2;
#define SC_OUT(KV)                                                                                                      \
  CQ_LAUNCH(scatter_out_strip_kernel<KV>, grid, 256, sh, st, (const uint16_t*)W, G.ld, G.d_out, G.d_in, G.g, G.r, coef, idx, gT, \
            transpose_out, per, status, gm)
    if (k == 64) SC_OUT(64);
    else if (k == 128) SC_OUT(128);
    else SC_OUT(256);
#undef SC_OUT
    kt_end(ti, st);
    return;
  }
  size_t sh = (size_t)k * SCATTER_JS * sizeof(float);
  if (sh > 48 * 1024) {
    cudaFuncSetAttribute(scatter_in_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh);
    cudaFuncSetAttribute(scatter_out_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh);
  }
  int strips = (k + SCATTER_JS - 1) / SCATTER_JS;
  if (G.axis == CAFEQ_AXIS_IN) {
    int want = (148 * 4) / (G.nbq * strips) + 1;
    int splits = want < 1 ? 1 : want;
    int rows_per = (G.d_out + splits - 1) / splits;
    if (rows_per < 8) rows_per = 8;
    splits = (G.d_out + rows_per - 1) / rows_per;
    dim3 grid(G.nbq, strips, splits);
    CQ_LAUNCH(scatter_in_kernel, grid, 256, sh, st, (const uint16_t*)W, G.ld, G.d_out, G.d_in, G.g, k, G.r, coef, idx, gT,
                                             transpose_out, rows_per, status, gm);
  } else {
    int want = (148 * 4) / (G.nbq * strips) + 1;
    int splits = want < 1 ? 1 : want;
    int per = (G.ng + splits - 1) / splits;
    if (per < 1) per = 1;
    splits = (G.ng + per - 1) / per;
    dim3 grid(G.nbq, strips, splits);
    CQ_LAUNCH(scatter_out_kernel, grid, 256, sh, st, (const uint16_t*)W, G.ld, G.d_out, G.d_in, G.g, k, G.r, coef, idx, gT,
                                              transpose_out, per, status, gm);
  }
  kt_end(ti, st);
}

__global__ void bf16_to_f32_kernel(const uint16_t* __restrict__ W, long long ld, int rows, int cols, float* __restrict__ U) {
  const long long n = (long long)rows * cols;
  for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
    int row = (int)(e / cols), col = (int)(e - (long long)row * cols);
    U[e] = bf16_bits_to_float(W[row * ld + col]);
  }
}

__global__ void resid_sq_kernel(float* __restrict__ R, const float* __restrict__ P, long long n, double* acc,
                                const int32_t* status) {
  if (status && *status) return;
  __shared__ double red[32];
  double local = 0.0;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    float v = R[i] - P[i];
    R[i] = v;
    local += (double)v * v;
  }
  double s = block_sum_double(local, red);
  if (threadIdx.x == 0) atomicAdd(acc, s);
}

__global__ void store_sqrt_kernel(const double* acc, float* out) { *out = (float)sqrt(*acc); }

// ------------------------------------------------------------------------------------------------
// per-matrix scratch
// ------------------------------------------------------------------------------------------------
struct MatWS {
  uint16_t *Tb, *Dbf;  // fused pass: bf16 operator blocks (applied orientation) and bf16 residual
  float *U, *D, *E;
  float *a, *usel, *coef, *cw, *agrp;
  int* idx;
};

// lean: the matrix goes through the fused tensor-core pass and nothing but the per-group records leaves it (Eq. 4 /
// LogSumExp steps without the quantised loss): no matrix-sized scratch at all.
static void carve_matrix(Bump& b, const Geo& G, MatWS* w, bool need_E, bool lean = false) {
  w->Tb = b.take<uint16_t>((size_t)(G.nbT > 0 ? G.nbT : 1) * (G.k > 0 ? G.k : 1) * (G.k > 0 ? G.k : 1));
  w->Dbf = lean ? nullptr : b.take<uint16_t>(G.n);
  w->U = lean ? nullptr : b.take<float>(G.n);
  w->D = lean ? nullptr : b.take<float>(G.n);
  w->E = (need_E && !lean) ? b.take<float>(G.n) : nullptr;
  size_t rows_ng = (size_t)G.d_out * G.ng;
  w->a = b.take<float>(rows_ng);
  w->usel = b.take<float>(rows_ng);
  w->idx = b.take<int>(rows_ng);
  w->coef = b.take<float>(rows_ng);
  w->cw = b.take<float>((size_t)(G.ng > G.d_out ? G.ng : G.d_out));
  w->agrp = b.take<float>((size_t)G.ng);
}

// One fused tensor-core pass (see kernels_fused.cuh); returns false when the shape is not covered.
static bool fused_pass(cudaStream_t st, const void* X, long long ldx, const Geo& G, const float* Top, int transposed,
                       uint16_t* Tb, BdParams p, int32_t* status, const uint16_t* Tb_ready = nullptr) {
  const int form = (G.axis == CAFEQ_AXIS_IN) ? BD_IN : BD_OUT;
  if (!bd_supported(form, G.d_out, G.d_in, ldx, G.k, G.g, X)) return false;
  const long long kk = (long long)G.nbT * G.k * G.k;
  if (Tb_ready && !transposed) Tb = const_cast<uint16_t*>(Tb_ready);  // bf16 operator already in applied orientation
  else CQ_LAUNCH(operator_to_bf16_kernel, grid_for(kk), 256, 0, st, Top, Tb, G.k, kk, transposed, status);
  p.d_out = G.d_out;
  p.d_in = G.d_in;
  p.r = G.r;
  p.status = status;
  int ti = kt_begin(5, st);
  g_launches.fetch_add(1, std::memory_order_relaxed);
  int rc = bd_launch(st, form, G.k, G.g, X, ldx, Tb, G.nbT, p);
  kt_end(ti, st);
  return rc == CAFEQ_OK;
}

// U = T o W in fp32 as one-term batched products on the tensor cores (bf16 x bf16 products are exact, fp32
// accumulation: the same arithmetic as the fused pass).  Tb: bf16 operator blocks in applied orientation
// [nbT k, k].  Output axis: the contraction runs down the rows of W, so its transpose goes through WT first.
static bool apply_tc(cudaStream_t st, const void* W, const Geo& G, const uint16_t* Tb, float* U, uint16_t* WT, int32_t* status) {
  const int k = G.k;
  if (!kk_fast(k) || ((uintptr_t)W & 15) || (G.ld % 8) || (G.d_in % 4)) return false;
  TgOperand oa[1], ob[1];
  TgParams p;
  memset(&p, 0, sizeof(p));
  p.nterms = 1; p.K = k; p.batch = G.nbq; p.alpha = 1.f;
  p.a_rep_k = k; p.a_rep_r = 1; p.divA = 1;
  p.C = U; p.ldc = G.d_in;
  p.status = status;
  if (G.axis == CAFEQ_AXIS_IN) {
    oa[0] = TgOperand{W, G.d_out, G.d_in, G.ld};
    ob[0] = TgOperand{Tb, (long long)G.nbT * k, k, k};
    p.M = G.d_out; p.N = k;
    p.rowsA_per_batch = 0; p.colsA_per_batch = k;
    p.rowsB_per_batch = k; p.divB = G.r;
    p.sCb = k;
  } else {
    if (!WT || (G.d_out % 8)) return false;
    dim3 tg((G.d_in + 31) / 32, (G.d_out + 31) / 32);
    CQ_LAUNCH(transpose_bf16_kernel, tg, dim3(32, 8), 0, st, (const uint16_t*)W, G.d_out, G.d_in, G.ld, WT);
    oa[0] = TgOperand{Tb, (long long)G.nbT * k, k, k};
    ob[0] = TgOperand{WT, G.d_in, G.d_out, G.d_out};
    p.M = k; p.N = G.d_in;
    p.rowsA_per_batch = k; p.divA = G.r;
    p.rowsB_per_batch = 0; p.colsB_per_batch = k;
    p.sCb = (long long)k * G.d_in;
  }
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return tg_launch(st, oa, ob, p) == CAFEQ_OK;
}

// U = T o W, group absmax / arg-max, and (optionally) the quantiser outputs.  Returns true when the fused
// tensor-core pass ran (then the residual is in w.Dbf as bf16 instead of w.D as fp32, and U is not stored).
static bool forward_quant(cudaStream_t st, const void* W, const Geo& G, int bits, const float* Tc, int transposed,
                          const MatWS& w, const void* offsets, int off_kind, bool want_delta, float* Uhat, int8_t* codes,
                          float* scales, int32_t* status, bool allow_fused, const BdParams* surr = nullptr,
                          const uint16_t* Tb_ready = nullptr, uint16_t* WT_scratch = nullptr) {
  if (Tc && allow_fused && off_kind == CAFEQ_OFFSETS_NONE && !Uhat) {
    BdParams p;
    memset(&p, 0, sizeof(p));
    if (surr) p = *surr;
    p.epi = EPI_ABSMAX | (want_delta ? EPI_DELTA : 0) | (codes ? EPI_CODES : 0) | (surr ? EPI_SURR : 0);
    p.qmax = qmax_of(bits);
    p.a = w.a; p.usel = w.usel; p.idx = w.idx;
    p.delta = w.Dbf; p.codes = codes; p.scales = scales;
    if (fused_pass(st, W, G.ld, G, Tc, transposed, w.Tb, p, status, Tb_ready)) return true;
  }
  if (!w.U) return false;  // lean workspace: there is no scratch for the shape-agnostic kernels (callers check first)
  bool applied = false;
  if (Tc && allow_fused) {  // (allow_fused is off when the caller asked for the shape-agnostic kernels)
    const uint16_t* Tb = (Tb_ready && !transposed) ? Tb_ready : w.Tb;
    const long long kk = (long long)G.nbT * G.k * G.k;
    if (Tb == w.Tb && kk_fast(G.k)) CQ_LAUNCH(operator_to_bf16_kernel, grid_for(kk), 256, 0, st, Tc, w.Tb, G.k, kk, transposed, status);
    applied = apply_tc(st, W, G, Tb, w.U, WT_scratch, status);
  }
  if (applied) {
  } else if (Tc) launch_apply(st, W, 1, G.ld, G, Tc, transposed, w.U, G.d_in, GEMM_STORE, nullptr, status);
  else CQ_LAUNCH(bf16_to_f32_kernel, grid_for(G.n), 256, 0, st, (const uint16_t*)W, G.ld, G.d_out, G.d_in, w.U);
  launch_absmax(st, w.U, G.d_in, G, w.a, w.usel, w.idx, status);
  if (want_delta || Uhat || codes)
    CQ_LAUNCH(quant_kernel, grid_for(G.n), 256, 0, st, w.U, G.d_in, G.d_out, G.d_in, G.g, w.a, qmax_of(bits), offsets, off_kind,
              want_delta ? w.D : nullptr, Uhat, codes, status);
  if (scales)
    CQ_LAUNCH(scales_kernel, grid_for((long long)G.d_out * G.ng), 256, 0, st, w.a, scales, (long long)G.d_out * G.ng,
              qmax_of(bits), status);
  return false;
}

}  // namespace cafeq

#include "pair_dense.cuh"

using namespace cafeq;

// ------------------------------------------------------------------------------------------------
extern "C" const char* cafeq_status_string(int s) {
  switch (s) {
    case CAFEQ_OK: return "ok";
    case CAFEQ_ERR_INVALID_ARG: return "invalid argument";
    case CAFEQ_ERR_UNSUPPORTED: return "unsupported shape or mode";
    case CAFEQ_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case CAFEQ_ERR_CUDA: return "CUDA launch failed";
    case CAFEQ_ERR_SINGULAR: return "singular transform block";
    case CAFEQ_ERR_NONFINITE: return "non-finite value";
    case CAFEQ_ERR_TIMEOUT: return "bounded device wait expired";
    case CAFEQ_ERR_TOO_LARGE: return "problem needs more scratch than the built-in buffer holds";
    default: return "unknown status";
  }
}

extern "C" int cafeq_version(void) { return 100; }

extern "C" long long cafeq_debug_launch_count(void) { return g_launches.load(); }

extern "C" int cafeq_set_overlap_mode(int overlapped) {
  if (overlapped != 0 && overlapped != 1) return CAFEQ_ERR_INVALID_ARG;
  g_tg_min_ctas.store(overlapped ? 28 : 96, std::memory_order_relaxed);
  g_bd_min_tiles.store(overlapped ? 14 : 1, std::memory_order_relaxed);
  g_bw_min_tiles.store(overlapped ? 14 : 6, std::memory_order_relaxed);
  return CAFEQ_OK;
}

extern "C" int cafeq_debug_wait_probe(unsigned long long limit_ns, int32_t* status, int* result, void* stream) {
  if (!status || !result) return CAFEQ_ERR_INVALID_ARG;
  CQ_LAUNCH(wait_probe_kernel, 1, 32, 0, (cudaStream_t)stream, (uint64_t)limit_ns, status, result);
  return cudaGetLastError() == cudaSuccess ? CAFEQ_OK : CAFEQ_ERR_CUDA;
}

extern "C" int cafeq_debug_timer_begin(int capacity) {
  if (capacity < 0 || g_kt.on) return CAFEQ_ERR_INVALID_ARG;
  g_kt.a.resize(capacity);
  g_kt.b.resize(capacity);
  g_kt.kind.assign(capacity, 0);
  for (int i = 0; i < capacity; ++i) {
    if (cudaEventCreate(&g_kt.a[i]) != cudaSuccess || cudaEventCreate(&g_kt.b[i]) != cudaSuccess) return CAFEQ_ERR_CUDA;
  }
  g_kt.used = 0;
  g_kt.on = true;
  return CAFEQ_OK;
}

extern "C" int cafeq_debug_timer_read(float* ms, int* kinds, int* count) {
  if (!g_kt.on || !ms || !kinds || !count) return CAFEQ_ERR_INVALID_ARG;
  int rc = CAFEQ_OK;
  for (int i = 0; i < g_kt.used; ++i) {
    if (cudaEventSynchronize(g_kt.b[i]) != cudaSuccess || cudaEventElapsedTime(&ms[i], g_kt.a[i], g_kt.b[i]) != cudaSuccess)
      rc = CAFEQ_ERR_CUDA;
    kinds[i] = g_kt.kind[i];
  }
  *count = g_kt.used;
  for (size_t i = 0; i < g_kt.a.size(); ++i) {
    cudaEventDestroy(g_kt.a[i]);
    cudaEventDestroy(g_kt.b[i]);
  }
  g_kt.a.clear();
  g_kt.b.clear();
  g_kt.kind.clear();
  g_kt.used = 0;
  g_kt.on = false;
  return rc;
}

static int check_ws(void* ws, size_t ws_bytes) {
  if (!ws || ((uintptr_t)ws & 255)) return CAFEQ_ERR_WORKSPACE;
  (void)ws_bytes;
  return CAFEQ_OK;
}

static int last_launch() { return cudaGetLastError() == cudaSuccess ? CAFEQ_OK : CAFEQ_ERR_CUDA; }

// ------------------------------------------------------------------------------------------------
// What cafeq_rtn needs from its workspace: nothing when the streaming kernel covers the call (no transform, group 32 /
// 64 / 128 / 256, aligned rows), the per-group records and the rounded operator when the fused tensor-core pass
// covers it, matrix-sized fp32 buffers otherwise.  W / codes may be null (a size query): aligned pointers are assumed.
static size_t rtn_scratch(const Geo& G, bool has_T, const void* W, const int8_t* codes, Bump* carve, MatWS* w, float** Tc) {
  Bump count(nullptr, 0);
  Bump& b = carve ? *carve : count;
  MatWS tmp;
  MatWS& m = w ? *w : tmp;
  if (!has_T && (G.g == 32 || G.g == 64 || G.g == 128 || G.g == 256) && !((uintptr_t)W & 15) && !(G.ld % 8) &&
      !((uintptr_t)codes & 7))
    return 0;
  const bool lean = has_T && kk_fast(G.k) &&
                    bd_supported(G.axis == CAFEQ_AXIS_IN ? BD_IN : BD_OUT, G.d_out, G.d_in, G.ld, G.k, G.g, W);
  carve_matrix(b, G, &m, false, lean);
  float* t = has_T ? b.take<float>((size_t)G.nbT * G.k * G.k) : nullptr;
  if (Tc) *Tc = t;
  return b.used;
}

extern "C" int cafeq_rtn_workspace_size(const cafeq_matrix_desc* d, int has_transform, size_t* bytes) {
  Geo G;
  int rc = make_geo(d, &G, false);
  if (rc) return rc;
  if (!bytes) return CAFEQ_ERR_INVALID_ARG;
  *bytes = rtn_scratch(G, has_transform != 0 && G.k > 0, nullptr, nullptr, nullptr, nullptr, nullptr);
  return CAFEQ_OK;
}

extern "C" int cafeq_rtn(const cafeq_matrix_desc* d, const void* W, const float* T, int8_t* codes, float* scales,
                         void* ws, size_t ws_bytes, void* stream) {
  Geo G;
  int rc = make_geo(d, &G, false);
  if (rc) return rc;
  if (!W || !codes || !scales) return CAFEQ_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const bool has_T = (T != nullptr && G.k > 0);
  if (!has_T) {
    // no transform: one streaming kernel, no scratch (the workspace may be null)
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (rtn_stream_launch(st, W, G.ld, G.d_out, G.d_in, G.g, qmax_of(d->bits), codes, scales)) return last_launch();
    g_launches.fetch_sub(1, std::memory_order_relaxed);
  }
  if ((rc = check_ws(ws, ws_bytes))) return rc;
  Bump b(ws, ws_bytes);
  MatWS w;
  float* Tc = nullptr;
  rtn_scratch(G, has_T, W, codes, &b, &w, &Tc);
  if (b.overflow) return CAFEQ_ERR_WORKSPACE;
  if (has_T) CQ_LAUNCH(round_bf16_kernel, grid_for((long long)G.nbT * G.k * G.k), 256, 0, st, T, Tc, (long long)G.nbT * G.k * G.k, nullptr);
  forward_quant(st, W, G, d->bits, Tc, d->trole == CAFEQ_APPLY_TT, w, nullptr, CAFEQ_OFFSETS_NONE, false, nullptr, codes,
                scales, nullptr, true);
  return last_launch();
}

// ------------------------------------------------------------------------------------------------
// inference side: apply a block-diagonal operator to activations, dequantise packed weights
// ------------------------------------------------------------------------------------------------
static size_t apply_scratch(const Geo& G, bool fused) {
  const size_t kk = (size_t)G.nbT * G.k * G.k;
  return 1024 + kk * 6 + (fused ? 0 : (size_t)G.n * 4 + 256);
}
static Geo apply_geo(Geo G) {
  // the store epilogue ignores the quantisation groups: any group width the pass is built for will do
  if (G.d_in % 128 == 0) { G.g = 128; G.ng = G.d_in / 128; }
  return G;
}

extern "C" int cafeq_apply_workspace_size(const cafeq_matrix_desc* d, size_t* bytes) {
  Geo G;
  int rc = make_geo(d, &G, false);
  if (rc) return rc;
  if (!bytes || G.k <= 0) return CAFEQ_ERR_INVALID_ARG;
  const Geo Ga = apply_geo(G);
  // (X itself is not known here: 16-byte aligned rows are assumed; a call whose X does not qualify returns
  // CAFEQ_ERR_WORKSPACE)
  const bool fused = bd_supported(G.axis == CAFEQ_AXIS_IN ? BD_IN : BD_OUT, Ga.d_out, Ga.d_in, Ga.ld, Ga.k, Ga.g, nullptr);
  *bytes = apply_scratch(G, fused);
  return CAFEQ_OK;
}

extern "C" int cafeq_apply_transform(const cafeq_matrix_desc* d, const void* X, const float* T, void* Y, int32_t* status, void* ws,
                                     size_t ws_bytes, void* stream) {
  Geo G;
  int rc = make_geo(d, &G, false);
  if (rc) return rc;
  if (!X || !T || !Y || G.k <= 0) return CAFEQ_ERR_INVALID_ARG;
  if ((rc = check_ws(ws, ws_bytes))) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  const long long kk = (long long)G.nbT * G.k * G.k;
  Bump b(ws, ws_bytes);
  float* Tc = b.take<float>(kk);
  uint16_t* Tb = b.take<uint16_t>(kk);
  if (b.overflow) return CAFEQ_ERR_WORKSPACE;
  // the deployed operator is the bf16 rounding of the given one (what the tensor cores apply; the pass converts it
  // itself, the shape-agnostic kernels take the rounded fp32 copy)
  const int transposed = d->trole == CAFEQ_APPLY_TT;
  {
    const Geo Ga = apply_geo(G);
    BdParams p;
    memset(&p, 0, sizeof(p));
    p.epi = EPI_STORE;
    p.delta = reinterpret_cast<uint16_t*>(Y);
    if (fused_pass(st, X, G.ld, Ga, T, transposed, Tb, p, status, nullptr)) return last_launch();
  }
  float* U = b.take<float>(G.n);
  if (b.overflow) return CAFEQ_ERR_WORKSPACE;
  CQ_LAUNCH(round_bf16_kernel, grid_for(kk), 256, 0, st, T, Tc, kk, nullptr);
  launch_apply(st, X, 1, G.ld, G, Tc, transposed, U, G.d_in, GEMM_STORE, nullptr, status);
  CQ_LAUNCH(f32_to_bf16_kernel, grid_for(G.n), 256, 0, st, U, reinterpret_cast<uint16_t*>(Y), (long long)G.n);
  return last_launch();
}

extern "C" int cafeq_dequant(const cafeq_matrix_desc* d, const uint8_t* packed, const float* scales, void* What, long long ldo,
                             void* stream) {
  Geo G;
  int rc = make_geo(d, &G, false);
  if (rc) return rc;
  if (!packed || !scales || !What || ldo < G.d_in || (G.d_in % 8)) return CAFEQ_ERR_INVALID_ARG;
  CQ_LAUNCH(dequant_kernel, grid_for(G.n / 8), 256, 0, (cudaStream_t)stream, packed, scales, reinterpret_cast<uint16_t*>(What), G.d_out,
            G.d_in, d->bits, G.g, ldo);
  return last_launch();
}

// ------------------------------------------------------------------------------------------------
// single matrix forward + backward
// ------------------------------------------------------------------------------------------------
namespace cafeq {

struct SingleWS {
  MatWS m;
  float *Mc, *Minv, *gMinv, *tmp, *c, *A;
  double* acc;
  KkWS kk;
  // tensor-core straight-through path: second bf16 term of the residual, both terms transposed, N = Minv^T Minv
  uint16_t *Dlo, *DTh, *DTl;
  float* Nf;
  bool lean;  // carved without matrix-sized scratch: only the fused surrogate path may run
  int err;    // host-side error found while enqueuing a step
};

static bool carve_single(Bump& b, const Geo& G, SingleWS* s, bool need_E, bool lean = false) {
  s->lean = lean;
  s->err = CAFEQ_OK;
  carve_matrix(b, G, &s->m, need_E, lean);
  size_t kk = (size_t)G.nbT * G.k * G.k;
  s->Mc = b.take<float>(kk);
  s->Minv = b.take<float>(kk);
  s->gMinv = b.take<float>(kk);
  s->tmp = b.take<float>(kk);
  s->c = b.take<float>((size_t)G.nbT * G.k);
  s->A = b.take<float>((size_t)G.nbT * G.k);
  s->acc = b.take<double>(8);
  carve_kk(b, G.nbT, G.k, &s->kk);
  s->Dlo = lean ? nullptr : b.take<uint16_t>(G.n);
  s->DTh = lean ? nullptr : b.take<uint16_t>(G.n);
  s->DTl = lean ? nullptr : b.take<uint16_t>(G.n);
  s->Nf = b.take<float>(kk);
  return !b.overflow;
}

// Lean workspaces: a step of Eq. 4 / LogSumExp without the quantised loss on shapes the fused pass covers leaves
// nothing matrix-sized in scratch.  (W itself is not known to the size query: 16-byte aligned rows are assumed; a
// call whose weights turn out not to qualify returns CAFEQ_ERR_WORKSPACE.)
static bool lean_single_ok(const Geo& G, const cafeq_opt_cfg* cfg, const void* W) {
  if (!cfg || cfg->loss_kind != CAFEQ_LOSS_SURROGATE || cfg->eval_every != 0) return false;
  return kk_fast(G.k) && bd_supported(G.axis == CAFEQ_AXIS_IN ? BD_IN : BD_OUT, G.d_out, G.d_in, G.ld, G.k, G.g, W);
}
// Enqueue one forward(+backward) for a single matrix; gradM may be null.  hist is an optional [2] slot.
static void single_step(cudaStream_t st, const cafeq_matrix_desc* d, const Geo& G, const void* W, const float* M,
                        float* Minv_out, const void* offsets, int off_kind, int loss_kind, float kappa, bool want_exact,
                        float* losses, float* hist, float* gradM, int32_t* status, SingleWS& s, bool force_generic,
                        bool warm = false, float* step_counter = nullptr, float* grad_offsets = nullptr) {
  const int k = G.k;
  const bool tc = kk_fast(k) && !force_generic;
  const long long kk = (long long)G.nbT * k * k;
  const float qm = qmax_of(d->bits);
  const bool ste = (loss_kind == CAFEQ_LOSS_L2_STE);
  const bool need_l2 = want_exact || ste;
  const bool want_grad = (gradM != nullptr);
  const bool in_r1 = (G.axis == CAFEQ_AXIS_IN && G.r == 1);
  // straight-through mode on the tensor cores: input axis, no rounding offsets, shapes the fused pass covers
  const bool ste_tc = ste && tc && in_r1 && off_kind == CAFEQ_OFFSETS_NONE && G.d_out % 64 == 0 &&
                      bd_supported(BD_IN, G.d_out, G.d_in, G.ld, k, G.g, W);
  if (tc) {
    PrepArgs pa;
    memset(&pa, 0, sizeof(pa));
    pa.M = M; pa.Mc = s.Mc; pa.Ab = s.kk.Ab; pa.kk = kk;
    pa.zero_f[0] = s.A; pa.zero_fn[0] = (long long)G.nbT * k;
    pa.zero_f[1] = s.m.agrp; pa.zero_fn[1] = G.ng;
    if (in_r1) { pa.zero_f[2] = s.m.cw; pa.zero_fn[2] = G.ng; }
    if (want_grad) { pa.zero_f[3] = gradM; pa.zero_fn[3] = kk; }
    pa.zero_d[0] = s.acc; pa.zero_dn[0] = 8;
    pa.zero_d[1] = s.kk.rn; pa.zero_dn[1] = NS_MAX_ITERS * G.nbT;
    pa.flag = s.kk.flag;
    pa.step_counter = step_counter;
    pa.status = status;
    CQ_LAUNCH(step_prep_kernel, grid_for(kk), 256, 0, st, pa);
    ns_inverse(st, s.Mc, s.Minv, nullptr, G.nbT, k, warm, s.kk, status, true);
    dim3 cg(k / 32, G.nbT);
    CQ_LAUNCH(colnorm_cw_kernel, cg, dim3(32, 8), 0, st, s.Minv, k, s.c, in_r1 ? s.m.cw : nullptr, G.g);
    if (!in_r1) {
      if (G.axis == CAFEQ_AXIS_IN) CQ_LAUNCH(cw_in_kernel, (G.ng + 127) / 128, 128, 0, st, s.c, G.d_in, G.g, k, G.r, s.m.cw);
      else CQ_LAUNCH(cw_out_kernel, (G.d_out + 127) / 128, 128, 0, st, s.c, G.d_out, G.g, k, G.r, s.m.cw);
    }
  } else {
    CQ_LAUNCH(zero_f64_kernel, 1, 32, 0, st, s.acc, 8);
    CQ_LAUNCH(round_bf16_kernel, grid_for(kk), 256, 0, st, M, s.Mc, kk, status);
    if (step_counter) CQ_LAUNCH(adam_tick_kernel, 1, 1, 0, st, step_counter, status);
    launch_inverse(st, s.Mc, s.Minv, s.c, G.nbT, k, status);
    if (G.axis == CAFEQ_AXIS_IN) CQ_LAUNCH(cw_in_kernel, (G.ng + 127) / 128, 128, 0, st, s.c, G.d_in, G.g, k, G.r, s.m.cw);
    else CQ_LAUNCH(cw_out_kernel, (G.d_out + 127) / 128, 128, 0, st, s.c, G.d_out, G.g, k, G.r, s.m.cw);
    CQ_LAUNCH(fill_f32_kernel, grid_for(G.nbT * k), 256, 0, st, s.A, 0.f, (long long)G.nbT * k);
    CQ_LAUNCH(fill_f32_kernel, grid_for(G.ng), 256, 0, st, s.m.agrp, 0.f, G.ng);
    if (want_grad) CQ_LAUNCH(fill_f32_kernel, grid_for(kk), 256, 0, st, gradM, 0.f, kk);
  }
  if (Minv_out && Minv_out != s.Minv) CQ_LAUNCH(copy_f32_kernel, grid_for(kk), 256, 0, st, s.Minv, Minv_out, kk);
  BdParams sp;
  memset(&sp, 0, sizeof(sp));
  sp.cw = s.m.cw;
  sp.kappa = kappa;
  sp.coef = (want_grad && !ste) ? s.m.coef : nullptr;
  sp.lossacc = s.acc + 0;
  sp.Aacc = (G.axis == CAFEQ_AXIS_IN) ? s.m.agrp : s.A;
  if (ste_tc) {
    sp.delta_lo = s.Dlo;
    sp.a_always = 1;
  }
  if (s.lean && (ste || need_l2 || !tc || force_generic || off_kind != CAFEQ_OFFSETS_NONE ||
                 !bd_supported(G.axis == CAFEQ_AXIS_IN ? BD_IN : BD_OUT, G.d_out, G.d_in, G.ld, k, G.g, W))) {
    s.err = CAFEQ_ERR_WORKSPACE;  // this mode needs the matrix-sized scratch the workspace was sized without
    return;
  }
  const bool fused = forward_quant(st, W, G, d->bits, s.Mc, 0, s.m, offsets, off_kind, need_l2, nullptr, nullptr, nullptr,
                                   status, (!ste || ste_tc) && !force_generic, &sp, tc ? s.kk.Ab : nullptr);
  if (ste_tc && fused) {
    // Nothing below needs E = Minv o Delta itself.  With Gram_B = sum_o Delta[o, B]^T Delta[o, B] (k x k per block) and
    // N = Minv^T Minv:  L2 = <N, Gram>,  dL/dMinv = 2 Minv Gram,  gDelta = 2 N o Delta (one more block-diagonal
    // apply), and the scale path needs sum_e gDelta_e Delta_e per group.  Every product runs on the tensor cores
    // with the residual as a two-term bf16 split (three-term products: fp32-grade).
    KkWS& w = s.kk;
    const int c = w.cur;
    {
      dim3 tg((G.d_in + 31) / 32, (G.d_out + 31) / 32);
      CQ_LAUNCH(transpose_bf16_kernel, tg, dim3(32, 8), 0, st, s.m.Dbf, G.d_out, G.d_in, (long long)G.d_in, s.DTh);
      CQ_LAUNCH(transpose_bf16_kernel, tg, dim3(32, 8), 0, st, s.Dlo, G.d_out, G.d_in, (long long)G.d_in, s.DTl);
    }
    {  // Gram (fp32 in s.tmp, splits in w.Ph / w.Pl): contraction over the d_out rows
      TgOperand oa[3], ob[3];
      const uint16_t* at[3] = {s.DTh, s.DTl, s.DTh};
      const uint16_t* bt[3] = {s.DTh, s.DTh, s.DTl};
      for (int t = 0; t < 3; ++t) {
        oa[t] = TgOperand{at[t], G.d_in, G.d_out, G.d_out};
        ob[t] = TgOperand{bt[t], G.d_in, G.d_out, G.d_out};
      }
      TgParams p;
      memset(&p, 0, sizeof(p));
      p.M = p.N = k; p.K = G.d_out; p.batch = G.nbT; p.nterms = 3;
      p.rowsA_per_batch = p.rowsB_per_batch = k;
      p.divA = 1; p.a_rep_k = G.d_out; p.a_rep_r = 1;
      p.alpha = 1.f;
      p.C = s.tmp; p.ldc = k; p.sCb = (long long)k * k;
      p.Chi = w.Ph; p.Clo = w.Pl;
      p.min_ctas = 148;  // a long contraction: as many CTAs as the tile shapes give
      p.status = status;
      g_launches.fetch_add(1, std::memory_order_relaxed);
      tg_launch(st, oa, ob, p);
    }
    {  // N = Minv^T Minv (fp32 in s.Nf, splits in w.Qh / w.Ql)
      if (w.mn) {  // both operands are X read transposed from its row-major splits
        const uint16_t* a1[3] = {w.Xh[c], w.Xl[c], w.Xh[c]};
        const uint16_t* b1[3] = {w.Xh[c], w.Xh[c], w.Xl[c]};
        launch_kk_tc(st, 3, a1, b1, G.nbT, k, 1.f, 0.f, 0.f, nullptr, s.Nf, w.Qh, w.Ql, nullptr, nullptr, nullptr, nullptr, status, 1,
                     nullptr, 0.0, 1, 1);
      } else {
        const uint16_t* a1[3] = {w.XTh[c], w.XTl[c], w.XTh[c]};
        const uint16_t* b1[3] = {w.XTh[c], w.XTh[c], w.XTl[c]};
        launch_kk_tc(st, 3, a1, b1, G.nbT, k, 1.f, 0.f, 0.f, nullptr, s.Nf, w.Qh, w.Ql, nullptr, nullptr, nullptr, nullptr, status);
      }
    }
    CQ_LAUNCH(dot_f32_kernel, grid_for(kk), 256, 0, st, s.Nf, s.tmp, kk, s.acc + 1);
    CQ_LAUNCH(sqsum_bf16_kernel, grid_for(G.n), 256, 0, st, (const uint16_t*)W, G.ld, G.d_out, G.d_in, s.acc + 2, status);
    CQ_LAUNCH(finalize_single_kernel, 1, 1, 0, st, s.acc, losses, hist, 1);
    if (!want_grad) return;
    {  // dL/dMinv = 2 Minv Gram (Gram is symmetric: its rows serve as the contraction-major second operand)
      const uint16_t* a2[3] = {w.Xh[c], w.Xl[c], w.Xh[c]};
      const uint16_t* b2[3] = {w.Ph, w.Ph, w.Pl};
      launch_kk_tc(st, 3, a2, b2, G.nbT, k, 2.f, 0.f, 0.f, nullptr, s.gMinv, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr,
                   status);
    }
    {  // gDelta[o, B k + j] = 2 sum_l N_B[j][l] Delta[o, B k + l]  -> s.m.D (fp32 [d_out, d_in])
      TgOperand oa[3], ob[3];
      const uint16_t* at[3] = {s.m.Dbf, s.Dlo, s.m.Dbf};
      const uint16_t* bt[3] = {w.Qh, w.Qh, w.Ql};
      for (int t = 0; t < 3; ++t) {
        oa[t] = TgOperand{at[t], G.d_out, G.d_in, G.d_in};
        ob[t] = TgOperand{bt[t], (long long)G.nbT * k, k, k};
      }
      TgParams p;
      memset(&p, 0, sizeof(p));
      p.M = G.d_out; p.N = k; p.K = k; p.batch = G.nbT; p.nterms = 3;
      p.rowsA_per_batch = 0; p.colsA_per_batch = k; p.rowsB_per_batch = k;
      p.divA = 1; p.a_rep_k = k; p.a_rep_r = 1;
      p.alpha = 2.f;
      p.C = s.m.D; p.ldc = G.d_in; p.sCb = k;  // batch b writes the columns [b k, b k + k)
      p.status = status;
      g_launches.fetch_add(1, std::memory_order_relaxed);
      tg_launch(st, oa, ob, p);
    }
    const long long nrec = (long long)G.d_out * G.ng;
    CQ_LAUNCH(ste_scale_coef_kernel, (unsigned)((nrec * 32 + 255) / 256), 256, 0, st, s.m.D, (long long)G.d_in, s.m.Dbf, s.Dlo,
              (long long)G.d_in, G.d_out, G.ng, G.g, s.m.a, s.m.usel, 1, s.m.coef, status);
    launch_scatter(st, W, G, s.m.coef, s.m.idx, gradM, 0, status, 1);
    minv_path_tc(st, s.gMinv, gradM, G.nbT, k, true, s.kk, status);
    return;
  }
  if (need_l2) {
    // E = Minv o Delta, L2 = sum E^2
    bool done = false;
    if (fused) {
      BdParams bp;
      memset(&bp, 0, sizeof(bp));
      bp.epi = EPI_SQSUM;
      bp.sqacc = s.acc + 1;
      done = fused_pass(st, s.m.Dbf, G.d_in, G, s.Minv, 0, s.m.Tb, bp, status);
    }
    if (!done)
      launch_apply(st, s.m.D, 0, G.d_in, G, s.Minv, 0, s.m.E, G.d_in, (ste ? GEMM_STORE : 0) | GEMM_SQSUM, s.acc + 1, status);
    CQ_LAUNCH(sqsum_bf16_kernel, grid_for(G.n), 256, 0, st, (const uint16_t*)W, G.ld, G.d_out, G.d_in, s.acc + 2, status);
  }
  if (!fused)
    CQ_LAUNCH(surrogate_rows_kernel, (G.d_out + 127) / 128, 128, 0, st, s.m.a, s.m.usel, G.d_out, G.ng, G.g, G.axis,
                                                                 s.m.cw, kappa, k, G.r, (want_grad && !ste) ? s.m.coef : nullptr,
                                                                 s.m.agrp, s.A, s.acc + 0, status);
  if (G.axis == CAFEQ_AXIS_IN && !in_r1)
    CQ_LAUNCH(expand_agrp_kernel, (G.d_in + 127) / 128, 128, 0, st, s.m.agrp, G.d_in, G.g, k, G.r, s.A);
  CQ_LAUNCH(finalize_single_kernel, 1, 1, 0, st, s.acc, losses, hist, need_l2 ? 1 : 0);
  if (!want_grad) return;
  if (!ste) {
    launch_scatter(st, W, G, s.m.coef, s.m.idx, gradM, 0, status, fused ? 1 : 0);
    CQ_LAUNCH(gminv_kernel, grid_for(kk), 256, 0, st, s.Minv, s.A, in_r1 ? s.m.agrp : nullptr, G.g, 2.f * kappa, k, kk, s.gMinv);
  } else {
    // gMinv = 2 * sum_free E Delta^T ; gDelta = 2 Minv^T o E (overwrites Delta) ; scale path through arg-max
    CQ_LAUNCH(fill_f32_kernel, grid_for(kk), 256, 0, st, s.gMinv, 0.f, kk);
    launch_opgrad(st, s.m.E, G.d_in, s.m.D, 0, G.d_in, G, s.gMinv, 0, 2.f, status);
    launch_apply(st, s.m.E, 0, G.d_in, G, s.Minv, 1, s.m.D, G.d_in, GEMM_STORE, nullptr, status, 2.f);
    if (grad_offsets)  // s.m.D holds d L2 / d Uhat = 2 Minv^T E
      CQ_LAUNCH(grad_offsets_kernel, grid_for(G.n), 256, 0, st, s.m.U, s.m.D, (long long)G.d_in, G.d_out, G.d_in, G.g, s.m.a, qm,
                grad_offsets, status);
    CQ_LAUNCH(ste_scale_path_kernel, (unsigned)(((long long)G.d_out * G.ng * 32 + 255) / 256), 256, 0, st, 
        s.m.U, s.m.D, G.d_in, G.d_out, G.ng, G.g, s.m.a, s.m.usel, qm, offsets, off_kind, G.d_in, s.m.coef, status);
    launch_scatter(st, W, G, s.m.coef, s.m.idx, gradM, 0, status, 0);
  }
  // gradM -= Minv^T gMinv Minv^T
  if (tc) {
    minv_path_tc(st, s.gMinv, gradM, G.nbT, k, true, s.kk, status);
  } else {
    launch_kk(st, s.Minv, 1, s.gMinv, 0, s.tmp, G.nbT, k, 1.f, GEMM_STORE, status);
    launch_kk(st, s.tmp, 0, s.Minv, 1, gradM, G.nbT, k, -1.f, GEMM_STORE | GEMM_ACCUM, status);
  }
}

}  // namespace cafeq

extern "C" int cafeq_proxy_loss_fwd_bwd(const cafeq_matrix_desc* d, const void* W, const float* M, float* Minv,
                                        const void* offsets, int offsets_kind, int loss_kind, float kappa, int flags,
                                        float* losses, float* gradM, float* grad_offsets, int32_t* status, void* ws,
                                        size_t ws_bytes, void* stream) {
  Geo G;
  int rc = make_geo(d, &G, true);
  if (rc) return rc;
  if (!W || !M || !losses) return CAFEQ_ERR_INVALID_ARG;
  // the gradient with respect to soft offsets belongs to the straight-through loss evaluated with soft offsets
  if (grad_offsets && (offsets_kind != CAFEQ_OFFSETS_SOFT_F32 || loss_kind != CAFEQ_LOSS_L2_STE || (flags & CAFEQ_FLAG_NO_GRAD)))
    return CAFEQ_ERR_INVALID_ARG;
  if (loss_kind != CAFEQ_LOSS_SURROGATE && loss_kind != CAFEQ_LOSS_L2_STE) return CAFEQ_ERR_INVALID_ARG;
  if (offsets_kind < CAFEQ_OFFSETS_NONE || offsets_kind > CAFEQ_OFFSETS_SOFT_F32) return CAFEQ_ERR_INVALID_ARG;
  if (offsets_kind != CAFEQ_OFFSETS_NONE && !offsets) return CAFEQ_ERR_INVALID_ARG;
  const bool want_grad = !(flags & CAFEQ_FLAG_NO_GRAD);
  if (want_grad && !gradM) return CAFEQ_ERR_INVALID_ARG;
  if ((rc = check_ws(ws, ws_bytes))) return rc;
  if (kappa <= 0.f) kappa = 1.f / (float)(((1 << d->bits) - 1) * ((1 << d->bits) - 1));
  cudaStream_t st = (cudaStream_t)stream;
  Bump b(ws, ws_bytes);
  SingleWS s;
  // Eq. 4 alone on a shape the tensor-core pass covers leaves nothing matrix-sized in scratch (the lean size of
  // cafeq_workspace_size with a CAFEQ_LOSS_SURROGATE configuration is enough); everything else takes the full carving
  bool lean = false;
  if (loss_kind == CAFEQ_LOSS_SURROGATE && !(flags & (CAFEQ_FLAG_EXACT_LOSS | CAFEQ_FLAG_GENERIC)) &&
      offsets_kind == CAFEQ_OFFSETS_NONE) {
    cafeq_opt_cfg c0;
    memset(&c0, 0, sizeof(c0));
    c0.loss_kind = CAFEQ_LOSS_SURROGATE;
    lean = lean_single_ok(G, &c0, W);
    if (lean) {  // a workspace that holds the full carving keeps using it
      Bump probe(nullptr, 0);
      SingleWS tmp;
      carve_single(probe, G, &tmp, true, false);
      if (probe.used <= ws_bytes) lean = false;
    }
  }
  if (!carve_single(b, G, &s, true, lean)) return CAFEQ_ERR_WORKSPACE;
  const bool warm = (flags & CAFEQ_FLAG_WARM_MINV) && Minv;
  if (warm) CQ_LAUNCH(copy_f32_kernel, grid_for((long long)G.nbT * G.k * G.k), 256, 0, st, Minv, s.Minv, (long long)G.nbT * G.k * G.k);
  single_step(st, d, G, W, M, Minv, offsets, offsets_kind, loss_kind, kappa, (flags & CAFEQ_FLAG_EXACT_LOSS) != 0, losses,
              nullptr, want_grad ? gradM : nullptr, status, s, (flags & CAFEQ_FLAG_GENERIC) != 0, warm, nullptr, grad_offsets);
  if (s.err) return s.err;
  return last_launch();
}

extern "C" int cafeq_optimize_single(const cafeq_matrix_desc* d, const void* W, float* M, float* opt_state,
                                     const cafeq_opt_cfg* cfg, float* loss_history, int32_t* status, void* ws,
                                     size_t ws_bytes, void* stream) {
  Geo G;
  int rc = make_geo(d, &G, true);
  if (rc) return rc;
  if (!W || !M || !cfg || cfg->struct_size != sizeof(cafeq_opt_cfg) || !loss_history) return CAFEQ_ERR_INVALID_ARG;
  if (cfg->steps < 0) return CAFEQ_ERR_INVALID_ARG;
  if (cfg->loss_kind != CAFEQ_LOSS_SURROGATE && cfg->loss_kind != CAFEQ_LOSS_L2_STE) return CAFEQ_ERR_INVALID_ARG;
  if (cfg->optimizer == CAFEQ_OPT_ADAM && !opt_state) return CAFEQ_ERR_INVALID_ARG;
  if (cfg->optimizer != CAFEQ_OPT_ADAM && cfg->optimizer != CAFEQ_OPT_GD) return CAFEQ_ERR_INVALID_ARG;
  if ((rc = check_ws(ws, ws_bytes))) return rc;
  float kappa = cfg->kappa;
  if (kappa <= 0.f) kappa = 1.f / (float)(((1 << d->bits) - 1) * ((1 << d->bits) - 1));
  cudaStream_t st = (cudaStream_t)stream;
  Bump b(ws, ws_bytes);
  SingleWS s;
  if (!carve_single(b, G, &s, true, lean_single_ok(G, cfg, W))) return CAFEQ_ERR_WORKSPACE;
  const long long kk = (long long)G.nbT * G.k * G.k;
  float* grad = b.take<float>(kk);
  if (b.overflow) return CAFEQ_ERR_WORKSPACE;
  // the inverse of the last step's transform lives in the optimiser state, so a resumed run refines it
  const bool resume = cfg->resume && opt_state;
  if (opt_state) s.Minv = opt_state + CAFEQ_OPT_STATE_HEADER + 2 * kk;
  for (int it = 0; it < cfg->steps; ++it) {
    bool eval = cfg->eval_every > 0 && (it % cfg->eval_every == 0);
    single_step(st, d, G, W, M, nullptr, nullptr, CAFEQ_OFFSETS_NONE, cfg->loss_kind, kappa, eval, nullptr,
                loss_history + 2 * (size_t)it, grad, status, s, false, resume || it > 0, opt_state);
    if (s.err) return s.err;
    if (cfg->optimizer == CAFEQ_OPT_GD) {
      CQ_LAUNCH(gd_update_kernel, grid_for(kk), 256, 0, st, M, grad, cfg->lr, kk, status);
    } else {
      CQ_LAUNCH(adam_update_kernel, grid_for(kk), 256, 0, st, M, grad, opt_state, cfg->lr, cfg->beta1, cfg->beta2, cfg->eps, kk,
                                                       status);
    }
  }
  return last_launch();
}

// ------------------------------------------------------------------------------------------------
// pair
// ------------------------------------------------------------------------------------------------
namespace cafeq {

static int make_pair_geo(const cafeq_matrix_desc* d1, const cafeq_matrix_desc* d2, Geo* G1, Geo* G2) {
  int rc = make_geo(d1, G1, true);
  if (rc) return rc;
  if ((rc = make_geo(d2, G2, true))) return rc;
  if (G1->axis != CAFEQ_AXIS_OUT || G2->axis != CAFEQ_AXIS_IN) return CAFEQ_ERR_INVALID_ARG;
  if (G1->k != G2->k || G1->r != 1) return CAFEQ_ERR_INVALID_ARG;
  if (G1->nbT != G2->nbT) return CAFEQ_ERR_INVALID_ARG;  // h / k operator blocks on both sides
  if (d1->bits != d2->bits) return CAFEQ_ERR_UNSUPPORTED;
  return CAFEQ_OK;
}

// Cm[x][y] = sum over blocks B of W2:  A1[(B/r)k + j][x] * A2[y][B k + j]   (A1 stored [h, d1], A2 stored [d3, r h])
static void launch_pair_product(cudaStream_t st, const void* A1, int a1_bf16, long long ld1, const void* A2, int a2_bf16,
                                long long ld2, const Geo& G1, const Geo& G2, float* Cm, const int32_t* status) {
  const int d1n = G1.d_in, d3n = G2.d_out, k = G1.k;
  GemmArgs g = gemm_defaults(status);
  g.M = d1n; g.N = d3n;
  g.A = A1; g.a_bf16 = a1_bf16; g.sAm = 1; g.sAk = ld1;
  g.B = A2; g.b_bf16 = a2_bf16; g.sBk = 1; g.sBn = ld2;
  g.C = Cm; g.sCm = d3n; g.sCn = 1; g.sCb = 0;
  if (G2.r == 1) {
    g.K = G1.d_out; g.batch = 1;
    g.mode = GEMM_STORE;
  } else {
    CQ_LAUNCH(fill_f32_kernel, grid_for((long long)d1n * d3n), 256, 0, st, Cm, 0.f, (long long)d1n * d3n);
    g.K = k; g.batch = G2.nbq;
    g.sAb = (long long)k * ld1; g.divA = G2.r;
    g.sBb = k;
    g.mode = GEMM_STORE | GEMM_ATOMIC;
  }
  launch_gemm(st, g);
}

struct PairWS {
  MatWS m1, m2;
  float *Mc, *Minv, *Minv_c, *gMinv, *tmp, *RM, *amax, *R;
  float *G1, *G2, *T1, *T2;  // Appendix D.1's weighted objective: block Grams of the two weights, G1 Mc, Minv_c G2
  double* acc;
  KkWS kk;
  DenseWS dn;
  bool dense;  // the product term runs on the tensor cores (every dimension a multiple of 64)
  uint16_t *W2T, *gVTh, *gVTl;  // [r h, d3]: transposed second factor and transposed split of its gradient
  uint16_t* W1T;                // [d1, h]: transposed first factor (its apply contracts down the rows)
  bool lean;                    // carved without matrix-sized scratch: only the fused LogSumExp path may run
  int err;
};

// Operator gradient of a block-diagonal apply as batched k x k tensor-core products with a two-term split of the
// fp32 factor: out[b][m][n] (+)= sum_l A[(b r + rep) k + m][l] * (Bh + Bl)[(b r + rep) k + n][l], summed over rep.
// A bf16 [nb r k, K] (pitch lda), Bh / Bl bf16 [nb r k, K] (pitch K).
static void opgrad_tc(cudaStream_t st, const uint16_t* A, long long lda, const uint16_t* Bh, const uint16_t* Bl, int nb, int r,
                      int k, int K, float* out, bool a_is_split_side, int32_t* status) {
  (void)a_is_split_side;
  for (int rep = 0; rep < r; ++rep) {
    TgOperand oa[2], ob[2];
    const long long rows = (long long)nb * r * k - (long long)rep * k;
    oa[0] = oa[1] = TgOperand{A + (long long)rep * k * lda, rows, K, lda};
    ob[0] = TgOperand{Bh + (long long)rep * k * K, rows, K, K};
    ob[1] = TgOperand{Bl + (long long)rep * k * K, rows, K, K};
    TgParams p;
    memset(&p, 0, sizeof(p));
    p.M = p.N = k; p.K = K; p.batch = nb; p.nterms = 2;
    p.rowsA_per_batch = p.rowsB_per_batch = r * k;
    p.divA = 1; p.a_rep_k = K; p.a_rep_r = 1;
    p.alpha = 1.f;
    p.beta = rep ? 1.f : 0.f;
    p.C0 = rep ? out : nullptr; p.ldc0 = k; p.sC0b = (long long)k * k;
    p.C = out; p.ldc = k; p.sCb = (long long)k * k;
    p.min_ctas = 148;  // long contraction, few output tiles: the narrowest tile
    p.status = status;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    tg_launch(st, oa, ob, p);
  }
}

static bool dense_ok(const Geo& G1, const Geo& G2) {
  return G1.d_out % 64 == 0 && G1.d_in % 64 == 0 && G2.d_out % 64 == 0 && G2.d_in % 64 == 0 && G1.k % 32 == 0;
}

static bool carve_pair(Bump& b, const Geo& G1, const Geo& G2, PairWS* p, bool need_R, bool lean = false) {
  p->lean = lean;
  p->err = CAFEQ_OK;
  carve_matrix(b, G1, &p->m1, true, lean);
  carve_matrix(b, G2, &p->m2, true, lean);
  size_t kk = (size_t)G1.nbT * G1.k * G1.k;
  p->Mc = b.take<float>(kk);
  p->Minv = b.take<float>(kk);
  p->Minv_c = b.take<float>(kk);
  p->gMinv = b.take<float>(kk);
  p->tmp = b.take<float>(kk);
  p->RM = b.take<float>(kk);
  p->G1 = b.take<float>(kk); p->G2 = b.take<float>(kk); p->T1 = b.take<float>(kk); p->T2 = b.take<float>(kk);
  p->amax = b.take<float>(64);
  p->acc = b.take<double>(8);
  p->R = need_R ? b.take<float>((size_t)G1.d_in * G2.d_out) : nullptr;
  carve_kk(b, G1.nbT, G1.k, &p->kk);
  p->dense = need_R && dense_ok(G1, G2);
  if (p->dense) carve_dense(b, G1.d_out, G1.d_in, G2.d_out, G2.r, G1.k, G1.ng, G2.ng, &p->dn);
  p->W2T = p->gVTh = p->gVTl = p->W1T = nullptr;
  if (p->dense) {
    p->W1T = b.take<uint16_t>(G1.n);
    p->W2T = b.take<uint16_t>(G2.n);
    p->gVTh = b.take<uint16_t>(G2.n);
    p->gVTl = b.take<uint16_t>(G2.n);
  }
  return !b.overflow;
}

static bool lean_pair_ok(const Geo& G1, const Geo& G2, const cafeq_opt_cfg* cfg, const void* W1, const void* W2) {
  if (!cfg || cfg->eval_every != 0) return false;
  if (cfg->loss_kind != CAFEQ_LOSS_LSE && cfg->loss_kind != CAFEQ_LOSS_SUMSQ && cfg->loss_kind != CAFEQ_LOSS_SUMSQ_WEIGHTED) return false;
  return kk_fast(G1.k) && bd_supported(BD_OUT, G1.d_out, G1.d_in, G1.ld, G1.k, G1.g, W1) &&
         bd_supported(BD_IN, G2.d_out, G2.d_in, G2.ld, G2.k, G2.g, W2);
}

// Block Grams of a pair's weights (constants of a run): G1[b][i][j] = sum_x W1[b k + i, x] W1[b k + j, x] and
// G2[b][i][j] = sum over the r replicas and the rows y of W2[y, (b r + rep) k + i] W2[y, (b r + rep) k + j].
static void pair_grams(cudaStream_t st, const void* W1, const Geo& G1, const void* W2, const Geo& G2, PairWS& p, const int32_t* status) {
  const int k = G1.k;
  const long long kk = (long long)G1.nbT * k * k;
  GemmArgs g = gemm_defaults(status);
  g.M = k; g.N = k; g.K = G1.d_in; g.batch = G1.nbT;
  g.A = W1; g.a_bf16 = 1; g.sAm = G1.ld; g.sAk = 1; g.sAb = (long long)k * G1.ld;
  g.B = W1; g.b_bf16 = 1; g.sBk = 1; g.sBn = G1.ld; g.sBb = (long long)k * G1.ld;
  g.C = p.G1; g.sCm = k; g.sCn = 1; g.sCb = (long long)k * k;
  g.mode = GEMM_STORE;
  launch_gemm(st, g);
  CQ_LAUNCH(fill_f32_kernel, grid_for(kk), 256, 0, st, p.G2, 0.f, kk);
  GemmArgs h = gemm_defaults(status);
  h.M = k; h.N = k; h.K = G2.d_out; h.batch = G2.nbq;
  h.A = W2; h.a_bf16 = 1; h.sAm = 1; h.sAk = G2.ld; h.sAb = k;
  h.B = W2; h.b_bf16 = 1; h.sBk = G2.ld; h.sBn = 1; h.sBb = k;
  h.C = p.G2; h.sCm = k; h.sCn = 1; h.sCb = (long long)k * k; h.divC = G2.r;
  h.mode = GEMM_STORE | GEMM_ATOMIC;
  launch_gemm(st, h);
}

// One Cayley step on the rotations (Appendix D.2's strictly orthonormal baseline): V <- beta V + g,
// A = V M^T - M V^T, M <- (I + lr/2 A)^-1 (I - lr/2 A) M, the solve by the fixed-point iteration
// Y <- M - lr/2 A (M + Y) from Y = M - lr A M (five rounds: the error falls by lr/2 ||A|| per round).
static void cayley_update(cudaStream_t st, float* M, const float* grad, float* V, float lr, float beta, int nb, int k, PairWS& p,
                          const int32_t* status) {
  const long long kk = (long long)nb * k * k;
  float *A = p.tmp, *Y = p.RM, *S = p.gMinv, *Pm = p.Minv_c;
  CQ_LAUNCH(momentum_kernel, grid_for(kk), 256, 0, st, V, beta, grad, kk, status);
  launch_kk(st, V, 0, M, 1, S, nb, k, 1.f, GEMM_STORE, status);            // V M^T
  CQ_LAUNCH(skew_blocks_kernel, grid_for(kk), 256, 0, st, S, A, k, kk);    // A = V M^T - M V^T
  launch_kk(st, A, 0, M, 0, Pm, nb, k, 1.f, GEMM_STORE, status);
  CQ_LAUNCH(lincomb_kernel, grid_for(kk), 256, 0, st, Y, M, -lr, Pm, kk, status);
  for (int it = 0; it < 5; ++it) {
    CQ_LAUNCH(lincomb_kernel, grid_for(kk), 256, 0, st, S, M, 1.f, Y, kk, status);
    launch_kk(st, A, 0, S, 0, Pm, nb, k, 1.f, GEMM_STORE, status);
    CQ_LAUNCH(lincomb_kernel, grid_for(kk), 256, 0, st, Y, M, -0.5f * lr, Pm, kk, status);
  }
  CQ_LAUNCH(copy_f32_kernel, grid_for(kk), 256, 0, st, Y, M, kk);
}

static void pair_step(cudaStream_t st, const cafeq_matrix_desc* d1, const cafeq_matrix_desc* d2, const Geo& G1, const Geo& G2,
                      const void* W1, const void* W2, const float* M, const float* P, float t, float lambda, bool want_pqe,
                      float* losses, float* hist, float* gradM, int32_t* status, PairWS& p, bool force_generic,
                      bool warm = false, float* step_counter = nullptr, bool ste = false, int objective = 0) {
  const int k = G1.k;
  const bool tc = kk_fast(k) && !force_generic;
  const long long kk = (long long)G1.nbT * k * k;
  const float sqrt_h = sqrtf((float)G1.d_out);
  if (p.lean && (ste || want_pqe || !tc || !bd_supported(BD_OUT, G1.d_out, G1.d_in, G1.ld, k, G1.g, W1) ||
                 !bd_supported(BD_IN, G2.d_out, G2.d_in, G2.ld, k, G2.g, W2))) {
    p.err = CAFEQ_ERR_WORKSPACE;  // this mode needs the matrix-sized scratch the workspace was sized without
    return;
  }
  if (tc) {
    PrepArgs pa;
    memset(&pa, 0, sizeof(pa));
    pa.M = M; pa.Mc = p.Mc; pa.Ab = p.kk.Ab; pa.kk = kk;
    pa.zero_f[0] = p.amax; pa.zero_fn[0] = 1;
    if (gradM) {
      pa.zero_f[1] = gradM; pa.zero_fn[1] = kk;
      pa.zero_f[2] = p.gMinv; pa.zero_fn[2] = kk;
    }
    pa.zero_d[0] = p.acc; pa.zero_dn[0] = 8;
    pa.zero_d[1] = p.kk.rn; pa.zero_dn[1] = NS_MAX_ITERS * G1.nbT;
    pa.flag = p.kk.flag;
    pa.step_counter = step_counter;
    pa.status = status;
    CQ_LAUNCH(step_prep_kernel, grid_for(kk), 256, 0, st, pa);
    ns_inverse(st, p.Mc, p.Minv, nullptr, G1.nbT, k, warm, p.kk, status, true);
  } else {
    CQ_LAUNCH(zero_f64_kernel, 1, 32, 0, st, p.acc, 8);
    CQ_LAUNCH(fill_f32_kernel, 1, 32, 0, st, p.amax, 0.f, 1);
    CQ_LAUNCH(round_bf16_kernel, grid_for(kk), 256, 0, st, M, p.Mc, kk, status);
    if (step_counter) CQ_LAUNCH(adam_tick_kernel, 1, 1, 0, st, step_counter, status);
    launch_inverse(st, p.Mc, p.Minv, nullptr, G1.nbT, k, status);
  }
  CQ_LAUNCH(round_bf16_kernel, grid_for(kk), 256, 0, st, p.Minv, p.Minv_c, kk, status);
  // U = M_c^T o W1 (axis OUT), V = Minv_c o W2 (axis IN); Uhat kept in the E buffers when PQE is wanted
  const bool f1 = forward_quant(st, W1, G1, d1->bits, p.Mc, 1, p.m1, nullptr, CAFEQ_OFFSETS_NONE, false, want_pqe ? p.m1.E : nullptr, nullptr,
                nullptr, status, !force_generic, nullptr, nullptr, p.W1T);
  const bool f2 = forward_quant(st, W2, G2, d2->bits, p.Minv_c, 0, p.m2, nullptr, CAFEQ_OFFSETS_NONE, false, want_pqe ? p.m2.E : nullptr,
                nullptr, nullptr, status, !force_generic, nullptr, tc ? p.kk.Xh[p.kk.cur] : nullptr);  // Xh = bf16(Minv)
  const long long n1 = (long long)G1.d_out * G1.ng, n2 = (long long)G2.d_out * G2.ng;
  CQ_LAUNCH(max2_f32_kernel, grid_for(n1 + n2), 256, 0, st, p.m1.a, n1, p.m2.a, n2, p.amax, status);
  CQ_LAUNCH(sumexp2_kernel, grid_for(n1 + n2), 256, 0, st, p.m1.a, n1, p.m2.a, n2, p.amax, t, p.acc + 0, status);
  if (objective) {
    // Appendix D.1: sums of the squared group maxima; for the weighted form also ||U||_F^2 = <G1 Mc, Mc> and
    // ||V||_F^2 = <Minv_c G2, Minv_c> from the block Grams of the weights (computed once per call)
    CQ_LAUNCH(sqsum_f32_kernel, grid_for(n1), 256, 0, st, p.m1.a, n1, p.acc + 3);
    CQ_LAUNCH(sqsum_f32_kernel, grid_for(n2), 256, 0, st, p.m2.a, n2, p.acc + 4);
    if (objective == 2) {
      launch_kk(st, p.G1, 0, p.Mc, 0, p.T1, G1.nbT, k, 1.f, GEMM_STORE, status);
      launch_kk(st, p.Minv_c, 0, p.G2, 0, p.T2, G1.nbT, k, 1.f, GEMM_STORE, status);
      CQ_LAUNCH(dot_f32_kernel, grid_for(kk), 256, 0, st, p.T1, p.Mc, kk, p.acc + 5);
      CQ_LAUNCH(dot_f32_kernel, grid_for(kk), 256, 0, st, p.T2, p.Minv_c, kk, p.acc + 6);
    }
  }
  // orthonormality penalty on the fp32 parameters: R = M M^T - I (not part of the straight-through PQE loss)
  if (ste) {
  } else if (tc) {
    // R = M M^T - I (symmetric) with its bf16 splits, ||R||_F^2, and R M for the gradient
    KkWS& w = p.kk;
    launch_split(st, M, k, kk, w.Ph, w.Pl, w.Qh, w.Ql, nullptr, status);
    const uint16_t* a1[3] = {w.Ph, w.Pl, w.Ph};
    const uint16_t* b1[3] = {w.Ph, w.Ph, w.Pl};
    launch_kk_tc(st, 3, a1, b1, G1.nbT, k, 1.f, 0.f, -1.f, nullptr, nullptr, w.RTh, w.RTl, nullptr, nullptr, p.acc + 1, nullptr,
                 status, 0);
    if (gradM && lambda != 0.f) {
      const uint16_t* a2[3] = {w.RTh, w.RTl, w.RTh};
      const uint16_t* b2[3] = {w.Qh, w.Qh, w.Ql};
      launch_kk_tc(st, 3, a2, b2, G1.nbT, k, 1.f, 0.f, 0.f, nullptr, p.RM, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr,
                   status);
    }
  } else {
    launch_kk(st, M, 0, M, 1, p.tmp, G1.nbT, k, 1.f, GEMM_STORE, status);
    CQ_LAUNCH(sub_identity_kernel, grid_for(kk), 256, 0, st, p.tmp, k, kk);
    CQ_LAUNCH(sqsum_f32_kernel, grid_for(kk), 256, 0, st, p.tmp, kk, p.acc + 1);
  }
  if (want_pqe && p.dense) {
    // Eq. 5 on the tensor cores: || Uhat_exp^T Vhat^T - P ||_F^2 with three-term bf16 splits of the dequantised values
    dense_pqe(st, p.m1.E, p.m2.E, P, p.dn, p.acc + 2, nullptr, status, ste);
  } else if (want_pqe) {
    launch_pair_product(st, p.m1.E, 0, G1.d_in, p.m2.E, 0, G2.d_in, G1, G2, p.R, status);
    CQ_LAUNCH(resid_sq_kernel, grid_for((long long)G1.d_in * G2.d_out), 256, 0, st, p.R, P, (long long)G1.d_in * G2.d_out, p.acc + 2,
                                                                             status);
  }
  CQ_LAUNCH(finalize_pair_kernel, 1, 1, 0, st, p.acc, p.amax, t, lambda, sqrt_h, losses, hist, ste ? 2 : (want_pqe ? 1 : 0), objective,
            (double)n1, (double)n2);
  if (!gradM) return;
  if (ste) {
    // Straight-through gradient of ||Uhat_exp^T Vhat^T - P||_F^2 (Eq. 5 squared): the residual R [d1, d3] and
    // its transpose are in p.dn.Ph/Pl/PTh/PTl; the quantiser passes gradients through except for its scale,
    // whose dependence on the group's arg-max entry is kept.
    DenseWS& w = p.dn;
    {  // g Vhat' [d3, h] = 2 R^T Uhat^T, then one copy per replica of every inner block
      launch_split_rect(st, p.m1.E, w.h, w.d1, w.d1, 1.f, nullptr, nullptr, nullptr, w.Awh, w.Awl, nullptr, nullptr, status);
      const uint16_t* a[3] = {w.PTh, w.PTl, w.PTh};
      const uint16_t* b[3] = {w.Awh, w.Awh, w.Awl};
      DenseOut o;
      o.C = w.X0T; o.ldc = w.h;
      launch_dense_tc(st, 3, a, b, w.d3, w.h, w.d1, 2.f, 0.f, 0.f, o, status);
      CQ_LAUNCH(expand_cols_kernel, grid_for((long long)w.d3 * w.rh), 256, 0, st, w.X0T, w.d3, w.h, w.k, w.r, 1.f, w.V);
    }
    {  // g Uhat [h, d1] = 2 fold(Vhat^T) R^T
      dim3 grid((w.d3 + 31) / 32, w.h / 32);
      CQ_LAUNCH(fold_transpose_kernel, grid, dim3(32, 8), 0, st, p.m2.E, w.d3, w.h, w.k, w.r, w.Bf);
      launch_split_rect(st, w.Bf, w.h, w.d3, w.d3, 1.f, nullptr, nullptr, nullptr, w.Yh, w.Yl, nullptr, nullptr, status);
      const uint16_t* a[3] = {w.Yh, w.Yl, w.Yh};
      const uint16_t* b[3] = {w.Ph, w.Ph, w.Pl};
      DenseOut o;
      o.C = w.U; o.ldc = w.d1;
      launch_dense_tc(st, 3, a, b, w.h, w.d1, w.d3, 2.f, 0.f, 0.f, o, status);
    }
    const long long n1w = (long long)G1.d_out * G1.ng, n2w = (long long)G2.d_out * G2.ng;
    CQ_LAUNCH(ste_scale_path_kernel, (unsigned)((n1w * 32 + 255) / 256), 256, 0, st, p.m1.U, w.U, G1.d_in, G1.d_out, G1.ng, G1.g,
              p.m1.a, p.m1.usel, qmax_of(d1->bits), nullptr, CAFEQ_OFFSETS_NONE, G1.d_in, p.m1.coef, status);
    CQ_LAUNCH(add_argmax_kernel, grid_for(n1w), 256, 0, st, w.U, G1.d_in, G1.d_out, G1.ng, G1.g, p.m1.coef, p.m1.idx, status);
    CQ_LAUNCH(ste_scale_path_kernel, (unsigned)((n2w * 32 + 255) / 256), 256, 0, st, p.m2.U, w.V, G2.d_in, G2.d_out, G2.ng, G2.g,
              p.m2.a, p.m2.usel, qmax_of(d2->bits), nullptr, CAFEQ_OFFSETS_NONE, G2.d_in, p.m2.coef, status);
    CQ_LAUNCH(add_argmax_kernel, grid_for(n2w), 256, 0, st, w.V, G2.d_in, G2.d_out, G2.ng, G2.g, p.m2.coef, p.m2.idx, status);
    if (!tc) {
      CQ_LAUNCH(fill_f32_kernel, grid_for(kk), 256, 0, st, gradM, 0.f, kk);
      CQ_LAUNCH(fill_f32_kernel, grid_for(kk), 256, 0, st, p.gMinv, 0.f, kk);
    }
    const bool og_tc = tc && ((uintptr_t)W1 % 16 == 0) && (G1.ld % 8 == 0) && ((uintptr_t)W2 % 4 == 0) && G1.r == 1;
    if (og_tc) {
      // U side (operator M^T): gradM[b][m][n] = sum_c W1[b k + m][c] gU[b k + n][c], contraction along the rows' own
      // direction: both operands as they are stored
      launch_split_rect(st, w.U, w.h, w.d1, w.d1, 1.f, nullptr, nullptr, nullptr, w.Awh, w.Awl, nullptr, nullptr, status);
      opgrad_tc(st, (const uint16_t*)W1, G1.ld, w.Awh, w.Awl, G1.nbT, 1, k, G1.d_in, gradM, false, status);
      // V side (operator Minv): gMinv[b][i][j] = sum over replicas and rows o of gV[o][.. + i] W2[o][.. + j]: the
      // contraction runs down the columns, so both factors are transposed first
      {
        dim3 tg((G2.d_in + 31) / 32, (G2.d_out + 31) / 32);
        CQ_LAUNCH(transpose_bf16_kernel, tg, dim3(32, 8), 0, st, (const uint16_t*)W2, G2.d_out, G2.d_in, G2.ld, p.W2T);
      }
      launch_split_rect(st, w.V, w.d3, w.rh, w.rh, 1.f, nullptr, nullptr, nullptr, nullptr, nullptr, p.gVTh, p.gVTl, status);
      opgrad_tc(st, p.W2T, G2.d_out, p.gVTh, p.gVTl, G1.nbT, G2.r, k, G2.d_out, p.RM, true, status);
      // (W2^T as the first factor gives the transpose: RM[b][j][i]; put it back as gMinv[b][i][j])
      CQ_LAUNCH(transpose_blocks_kernel, grid_for(kk), 256, 0, st, p.RM, p.gMinv, k, kk);
    } else {
      launch_opgrad(st, w.U, G1.d_in, W1, 1, G1.ld, G1, gradM, 1, 1.f, status);    // U side: operator M^T
      launch_opgrad(st, w.V, G2.d_in, W2, 1, G2.ld, G2, p.gMinv, 0, 1.f, status);  // V side: operator Minv
    }
    if (tc) {
      minv_path_tc(st, p.gMinv, gradM, G1.nbT, k, true, p.kk, status);
    } else {
      launch_kk(st, p.Minv, 1, p.gMinv, 0, p.RM, G1.nbT, k, 1.f, GEMM_STORE, status);
      launch_kk(st, p.RM, 0, p.Minv, 1, gradM, G1.nbT, k, -1.f, GEMM_STORE | GEMM_ACCUM, status);
    }
    return;
  }
  if (objective)
    CQ_LAUNCH(sumsq_coef2_kernel, grid_for(n1 + n2), 256, 0, st, p.m1.a, p.m1.usel, p.m1.coef, n1, p.m2.a, p.m2.usel, p.m2.coef, n2,
              p.acc, objective == 2 ? 1 : 0, status);
  else
    CQ_LAUNCH(lse_coef2_kernel, grid_for(n1 + n2), 256, 0, st, p.m1.a, p.m1.usel, p.m1.coef, n1, p.m2.a, p.m2.usel, p.m2.coef, n2,
              p.amax, t, p.acc + 0, status);
  if (!tc) {
    CQ_LAUNCH(fill_f32_kernel, grid_for(kk), 256, 0, st, gradM, 0.f, kk);
    CQ_LAUNCH(fill_f32_kernel, grid_for(kk), 256, 0, st, p.gMinv, 0.f, kk);
  }
  // U side: operator is M^T, so the block gradient is stored transposed
  launch_scatter(st, W1, G1, p.m1.coef, p.m1.idx, gradM, 1, status, f1 ? 1 : 0);
  // V side: gradient with respect to Minv, then through the inverse
  launch_scatter(st, W2, G2, p.m2.coef, p.m2.idx, p.gMinv, 0, status, f2 ? 1 : 0);
  if (objective == 2) {
    // mean(a_V^2) d||U||_F/dM = mean(a_V^2) G1 Mc / ||U||_F ; mean(a_U^2) d||V||_F/dMinv = mean(a_U^2) Minv_c G2 / ||V||_F
    CQ_LAUNCH(axpy_norm_kernel, grid_for(kk), 256, 0, st, gradM, p.T1, kk, p.acc, 4, (double)n2, 5, status);
    CQ_LAUNCH(axpy_norm_kernel, grid_for(kk), 256, 0, st, p.gMinv, p.T2, kk, p.acc, 3, (double)n1, 6, status);
  }
  if (tc) {
    minv_path_tc(st, p.gMinv, gradM, G1.nbT, k, true, p.kk, status);
  } else {
    launch_kk(st, p.Minv, 1, p.gMinv, 0, p.RM, G1.nbT, k, 1.f, GEMM_STORE, status);
    launch_kk(st, p.RM, 0, p.Minv, 1, gradM, G1.nbT, k, -1.f, GEMM_STORE | GEMM_ACCUM, status);
  }
  if (lambda != 0.f) {
    if (!tc) launch_kk(st, p.tmp, 0, M, 0, p.RM, G1.nbT, k, 1.f, GEMM_STORE, status);
    CQ_LAUNCH(orth_grad_kernel, grid_for(kk), 256, 0, st, gradM, p.RM, p.acc + 1, lambda, sqrt_h, kk);
  }
}

}  // namespace cafeq

#include "adaptive_offsets.cuh"

extern "C" int cafeq_workspace_size(const cafeq_matrix_desc* d1, const cafeq_matrix_desc* d2, const cafeq_opt_cfg* cfg,
                                    size_t* bytes) {
  if (!bytes) return CAFEQ_ERR_INVALID_ARG;
  if (cfg && cfg->struct_size != sizeof(cafeq_opt_cfg)) return CAFEQ_ERR_INVALID_ARG;
  Geo G1, G2;
  int rc = make_geo(d1, &G1, false);
  if (rc) return rc;
  // the sizes come from the carving code itself, run on a counting allocator
  Bump b(nullptr, 0);
  const size_t kk = (size_t)(G1.nbT > 0 ? G1.nbT : 1) * (G1.k > 0 ? G1.k : 1) * (G1.k > 0 ? G1.k : 1);
  if (!d2) {
    SingleWS s;
    carve_single(b, G1, &s, true, G1.k > 0 && lean_single_ok(G1, cfg, nullptr));
    b.take<float>(kk);  // gradient of the optimise loop / rounded operator of cafeq_rtn
  } else {
    if ((rc = make_geo(d2, &G2, false))) return rc;
    PairWS p;
    const bool lean = G1.k > 0 && G2.k > 0 && lean_pair_ok(G1, G2, cfg, nullptr, nullptr);
    carve_pair(b, G1, G2, &p, !lean, lean);
    b.take<float>(kk);
    if (!cfg) {  // cafeq_adaptive_round's learned-offset mode carves its own set of buffers from the same workspace
      Bump b2(nullptr, 0);
      LearnWS lw;
      carve_learn(b2, G1, G2, &lw);
      b2.take<float>(kk); b2.take<float>(kk); b2.take<float>(kk);
      if (b2.used > b.used) b.used = b2.used;
    }
  }
  *bytes = b.used + 256;
  return CAFEQ_OK;
}

extern "C" int cafeq_pair_product(const cafeq_matrix_desc* d1, const void* W1, const cafeq_matrix_desc* d2,
                                  const void* W2, float* P, void* ws, size_t ws_bytes, void* stream) {
  Geo G1, G2;
  int rc = make_pair_geo(d1, d2, &G1, &G2);
  if (rc) return rc;
  if (!W1 || !W2 || !P) return CAFEQ_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (ws && !((uintptr_t)ws & 255) && dense_ok(G1, G2)) {
    Bump b(ws, ws_bytes);
    DenseWS w;
    if (carve_dense(b, G1.d_out, G1.d_in, G2.d_out, G2.r, G1.k, G1.ng, G2.ng, &w)) {
      CQ_LAUNCH(bf16_to_f32_kernel, grid_for(G1.n), 256, 0, st, (const uint16_t*)W1, G1.ld, G1.d_out, G1.d_in, w.U);
      CQ_LAUNCH(bf16_to_f32_kernel, grid_for(G2.n), 256, 0, st, (const uint16_t*)W2, G2.ld, G2.d_out, G2.d_in, w.V);
      dense_product(st, w.U, w.V, w, P, nullptr);
      return last_launch();
    }
  }
  launch_pair_product(st, W1, 1, G1.ld, W2, 1, G2.ld, G1, G2, P, nullptr);
  return last_launch();
}

extern "C" int cafeq_pair_loss_fwd_bwd(const cafeq_matrix_desc* d1, const void* W1, const cafeq_matrix_desc* d2,
                                       const void* W2, const float* M, const float* P, int loss_kind, float lse_t,
                                       float lambda_orth, int flags, float* losses, float* gradM, int32_t* status,
                                       void* ws, size_t ws_bytes, void* stream) {
  Geo G1, G2;
  int rc = make_pair_geo(d1, d2, &G1, &G2);
  if (rc) return rc;
  if (!W1 || !W2 || !M || !losses) return CAFEQ_ERR_INVALID_ARG;
  const bool ste = loss_kind == CAFEQ_LOSS_PQE_STE;
  const int objective = loss_kind == CAFEQ_LOSS_SUMSQ ? 1 : (loss_kind == CAFEQ_LOSS_SUMSQ_WEIGHTED ? 2 : 0);
  if (!ste && !objective && loss_kind != CAFEQ_LOSS_LSE) return CAFEQ_ERR_INVALID_ARG;
  if (ste && !dense_ok(G1, G2)) return CAFEQ_ERR_UNSUPPORTED;
  if (!(lse_t > 0.f)) return CAFEQ_ERR_INVALID_ARG;
  const bool want_grad = !(flags & CAFEQ_FLAG_NO_GRAD);
  const bool want_pqe = ste || (flags & CAFEQ_FLAG_EXACT_LOSS) != 0;
  if (want_grad && !gradM) return CAFEQ_ERR_INVALID_ARG;
  if (want_pqe && !P) return CAFEQ_ERR_INVALID_ARG;
  if ((rc = check_ws(ws, ws_bytes))) return rc;
  Bump b(ws, ws_bytes);
  PairWS p;
  if (!carve_pair(b, G1, G2, &p, want_pqe)) return CAFEQ_ERR_WORKSPACE;
  if (objective == 2) pair_grams((cudaStream_t)stream, W1, G1, W2, G2, p, status);
  pair_step((cudaStream_t)stream, d1, d2, G1, G2, W1, W2, M, P, lse_t, lambda_orth, want_pqe, losses, nullptr,
            want_grad ? gradM : nullptr, status, p, (flags & CAFEQ_FLAG_GENERIC) != 0, false, nullptr, ste, objective);
  return last_launch();
}

extern "C" int cafeq_optimize_pair(const cafeq_matrix_desc* d1, const void* W1, const cafeq_matrix_desc* d2,
                                   const void* W2, float* M, float* opt_state, const float* P, const cafeq_opt_cfg* cfg,
                                   float* loss_history, int32_t* status, void* ws, size_t ws_bytes, void* stream) {
  Geo G1, G2;
  int rc = make_pair_geo(d1, d2, &G1, &G2);
  if (rc) return rc;
  if (!W1 || !W2 || !M || !cfg || cfg->struct_size != sizeof(cafeq_opt_cfg) || !loss_history) return CAFEQ_ERR_INVALID_ARG;
  const bool ste = cfg->loss_kind == CAFEQ_LOSS_PQE_STE;
  const int objective = cfg->loss_kind == CAFEQ_LOSS_SUMSQ ? 1 : (cfg->loss_kind == CAFEQ_LOSS_SUMSQ_WEIGHTED ? 2 : 0);
  if ((!ste && !objective && cfg->loss_kind != CAFEQ_LOSS_LSE) || cfg->steps < 0 || !(cfg->lse_t > 0.f)) return CAFEQ_ERR_INVALID_ARG;
  if (ste && !P) return CAFEQ_ERR_INVALID_ARG;
  if (ste && !dense_ok(G1, G2)) return CAFEQ_ERR_UNSUPPORTED;
  const bool cayley = cfg->optimizer == CAFEQ_OPT_CAYLEY;
  if ((cfg->optimizer == CAFEQ_OPT_ADAM || cayley) && !opt_state) return CAFEQ_ERR_INVALID_ARG;
  if (cfg->optimizer != CAFEQ_OPT_ADAM && cfg->optimizer != CAFEQ_OPT_GD && !cayley) return CAFEQ_ERR_INVALID_ARG;
  if ((rc = check_ws(ws, ws_bytes))) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  const bool any_pqe = ste || ((P != nullptr) && cfg->eval_every > 0);
  Bump b(ws, ws_bytes);
  PairWS p;
  if (!carve_pair(b, G1, G2, &p, any_pqe, !any_pqe && lean_pair_ok(G1, G2, cfg, W1, W2))) return CAFEQ_ERR_WORKSPACE;
  const long long kk = (long long)G1.nbT * G1.k * G1.k;
  float* grad = b.take<float>(kk);
  if (b.overflow) return CAFEQ_ERR_WORKSPACE;
  // the inverse of the last step's transform lives in the optimiser state, so a resumed run refines it
  const bool resume = cfg->resume && opt_state;
  if (opt_state) p.Minv = opt_state + CAFEQ_OPT_STATE_HEADER + 2 * kk;
  if (objective == 2) pair_grams(st, W1, G1, W2, G2, p, status);
  for (int it = 0; it < cfg->steps; ++it) {
    bool eval = ste || (any_pqe && (it % cfg->eval_every == 0));
    pair_step(st, d1, d2, G1, G2, W1, W2, M, P, cfg->lse_t, cfg->lambda_orth, eval, nullptr, loss_history + 2 * (size_t)it,
              grad, status, p, false, resume || it > 0, opt_state, ste, objective);
    if (p.err) return p.err;
    if (cayley) {
      // momentum in the state's first-moment slot
      cayley_update(st, M, grad, opt_state + CAFEQ_OPT_STATE_HEADER, cfg->lr, cfg->beta1, G1.nbT, G1.k, p, status);
    } else if (cfg->optimizer == CAFEQ_OPT_GD) {
      CQ_LAUNCH(gd_update_kernel, grid_for(kk), 256, 0, st, M, grad, cfg->lr, kk, status);
    } else {
      CQ_LAUNCH(adam_update_kernel, grid_for(kk), 256, 0, st, M, grad, opt_state, cfg->lr, cfg->beta1, cfg->beta2, cfg->eps, kk,
                                                       status);
    }
  }
  return last_launch();
}

extern "C" int cafeq_adaptive_round(const cafeq_matrix_desc* d1, const void* W1, const cafeq_matrix_desc* d2,
                                    const void* W2, const float* M, int iters, int mode, int8_t* codes1, float* scales1,
                                    int8_t* codes2, float* scales2, float* pqe_history, int32_t* status, void* ws,
                                    size_t ws_bytes, void* stream) {
  Geo G1, G2;
  int rc = make_pair_geo(d1, d2, &G1, &G2);
  if (rc) return rc;
  if (!W1 || !W2 || !codes1 || !scales1 || !codes2 || !scales2 || !pqe_history) return CAFEQ_ERR_INVALID_ARG;
  if (mode != CAFEQ_ROUND_ALG1 && mode != CAFEQ_ROUND_LEARNED_OFFSETS) return CAFEQ_ERR_INVALID_ARG;
  if (iters < 0 || iters > (mode == CAFEQ_ROUND_ALG1 ? 15 : 30)) return CAFEQ_ERR_INVALID_ARG;
  if ((rc = check_ws(ws, ws_bytes))) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  if (mode == CAFEQ_ROUND_LEARNED_OFFSETS) {
    if (iters < 1) return CAFEQ_ERR_INVALID_ARG;
    Bump b(ws, ws_bytes);
    LearnWS w;
    carve_learn(b, G1, G2, &w);
    const long long kk = (long long)G1.nbT * G1.k * G1.k;
    float* Mc = b.take<float>(kk);
    float* Minv = b.take<float>(kk);
    float* Minv_c = b.take<float>(kk);
    if (b.overflow) return CAFEQ_ERR_WORKSPACE;
    if (M) {
      CQ_LAUNCH(round_bf16_kernel, grid_for(kk), 256, 0, st, M, Mc, kk, status);
      launch_inverse(st, Mc, Minv, nullptr, G1.nbT, G1.k, status);
      CQ_LAUNCH(round_bf16_kernel, grid_for(kk), 256, 0, st, Minv, Minv_c, kk, status);
      launch_apply(st, W1, 1, G1.ld, G1, Mc, 1, w.U, G1.d_in, GEMM_STORE, nullptr, status);
      launch_apply(st, W2, 1, G2.ld, G2, Minv_c, 0, w.V, G2.d_in, GEMM_STORE, nullptr, status);
    } else {
      CQ_LAUNCH(bf16_to_f32_kernel, grid_for(G1.n), 256, 0, st, (const uint16_t*)W1, G1.ld, G1.d_out, G1.d_in, w.U);
      CQ_LAUNCH(bf16_to_f32_kernel, grid_for(G2.n), 256, 0, st, (const uint16_t*)W2, G2.ld, G2.d_out, G2.d_in, w.V);
    }
    learned_offsets_run(st, d1->bits, G1, G2, iters, codes1, scales1, codes2, scales2, pqe_history, w, status);
    return last_launch();
  }
  if (!dense_ok(G1, G2)) return CAFEQ_ERR_UNSUPPORTED;  // every dimension a multiple of 64, block a multiple of 32
  Bump b(ws, ws_bytes);
  DenseWS w;
  if (!carve_dense(b, G1.d_out, G1.d_in, G2.d_out, G2.r, G1.k, G1.ng, G2.ng, &w)) return CAFEQ_ERR_WORKSPACE;
  const long long kk = (long long)G1.nbT * G1.k * G1.k;
  float* Mc = b.take<float>(kk);
  float* Minv = b.take<float>(kk);
  float* Minv_c = b.take<float>(kk);
  if (b.overflow) return CAFEQ_ERR_WORKSPACE;
  if (M) {
    // the transformed pair U = W1 M (operator bf16(M)^T on the stored rows), V = M^-1 W2 (operator bf16(inv(bf16(M))))
    CQ_LAUNCH(round_bf16_kernel, grid_for(kk), 256, 0, st, M, Mc, kk, status);
    launch_inverse(st, Mc, Minv, nullptr, G1.nbT, G1.k, status);
    CQ_LAUNCH(round_bf16_kernel, grid_for(kk), 256, 0, st, Minv, Minv_c, kk, status);
    launch_apply(st, W1, 1, G1.ld, G1, Mc, 1, w.U, G1.d_in, GEMM_STORE, nullptr, status);
    launch_apply(st, W2, 1, G2.ld, G2, Minv_c, 0, w.V, G2.d_in, GEMM_STORE, nullptr, status);
  } else {
    CQ_LAUNCH(bf16_to_f32_kernel, grid_for(G1.n), 256, 0, st, (const uint16_t*)W1, G1.ld, G1.d_out, G1.d_in, w.U);
    CQ_LAUNCH(bf16_to_f32_kernel, grid_for(G2.n), 256, 0, st, (const uint16_t*)W2, G2.ld, G2.d_out, G2.d_in, w.V);
  }
  alg1_run(st, d1->bits, G1.g, G2.g, iters, codes1, scales1, codes2, scales2, pqe_history, w, status);
  return last_launch();
}

extern "C" int cafeq_pack(const cafeq_matrix_desc* d, const int8_t* codes, uint8_t* packed, void* stream) {
  Geo G;
  int rc = make_geo(d, &G, false);
  if (rc) return rc;
  if (!codes || !packed) return CAFEQ_ERR_INVALID_ARG;
  if (G.d_in % 8) return CAFEQ_ERR_UNSUPPORTED;
  if (G.d_in % 32 == 0 && ((uintptr_t)codes % 16) == 0 && ((uintptr_t)packed % 4) == 0 && d->bits >= 2 && d->bits <= 8) {
    cudaStream_t ps = (cudaStream_t)stream;
    const unsigned pg = grid_for(G.n / 32);
    uint32_t* pw = reinterpret_cast<uint32_t*>(packed);
    switch (d->bits) {
      case 2: CQ_LAUNCH(pack32_kernel<2>, pg, 256, 0, ps, codes, pw, G.d_out, G.d_in); break;
      case 3: CQ_LAUNCH(pack32_kernel<3>, pg, 256, 0, ps, codes, pw, G.d_out, G.d_in); break;
      case 4: CQ_LAUNCH(pack32_kernel<4>, pg, 256, 0, ps, codes, pw, G.d_out, G.d_in); break;
      case 5: CQ_LAUNCH(pack32_kernel<5>, pg, 256, 0, ps, codes, pw, G.d_out, G.d_in); break;
      case 6: CQ_LAUNCH(pack32_kernel<6>, pg, 256, 0, ps, codes, pw, G.d_out, G.d_in); break;
      case 7: CQ_LAUNCH(pack32_kernel<7>, pg, 256, 0, ps, codes, pw, G.d_out, G.d_in); break;
      default: CQ_LAUNCH(pack32_kernel<8>, pg, 256, 0, ps, codes, pw, G.d_out, G.d_in); break;
    }
    return last_launch();
  }
  CQ_LAUNCH(pack_kernel, grid_for(G.n / 8), 256, 0, (cudaStream_t)stream, codes, packed, G.d_out, G.d_in, d->bits);
  return last_launch();
}

#include "layer_step.cuh"

// ------------------------------------------------------------------------------------------------
// cafeq_rtn without a caller workspace: scratch lives in the library image
// ------------------------------------------------------------------------------------------------
// In host code the name of a __device__ array is only a handle for the runtime, not an address a kernel can
// use; the device address is looked up once per device with cudaGetSymbolAddress and cached.
static __device__ __align__(256) unsigned char g_noalloc_scratch[CAFEQ_NOALLOC_SCRATCH_BYTES];
static constexpr int kMaxDevices = 64;
static void* g_noalloc_ptr[kMaxDevices] = {};
static std::mutex g_noalloc_mu;

extern "C" int cafeq_rtn_noalloc(const cafeq_matrix_desc* d, const void* W, const float* T, int8_t* codes, float* scales,
                                 void* stream) {
  Geo Gq;
  int rc = make_geo(d, &Gq, false);
  if (rc) return rc;
  if (!W || !codes || !scales) return CAFEQ_ERR_INVALID_ARG;
  // what cafeq_rtn would carve for this very call (cafeq_rtn_workspace_size gives the same figure for aligned buffers)
  const size_t need = rtn_scratch(Gq, T != nullptr && Gq.k > 0, W, codes, nullptr, nullptr, nullptr);
  if (need > (size_t)CAFEQ_NOALLOC_SCRATCH_BYTES) return CAFEQ_ERR_TOO_LARGE;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return CAFEQ_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return CAFEQ_ERR_UNSUPPORTED;
  void* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_noalloc_mu);
    if (!g_noalloc_ptr[dev]) {
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return CAFEQ_ERR_CUDA;
      g_noalloc_ptr[dev] = p;
    }
    scratch = g_noalloc_ptr[dev];
  }
  return cafeq_rtn(d, W, T, codes, scales, scratch, (size_t)CAFEQ_NOALLOC_SCRATCH_BYTES, stream);
}
