// Host side of the dense pair algebra: the product term of Eq. 5 (PQE) and Algorithm 1 (adaptive rounding),
// built from the tensor-core product kernel with three-term bf16 splits (fp32-grade accuracy).
// Included by cafeq_api.cu (uses its launch counter, workspace carving and quantiser launch helpers).
#pragma once

#include "kernels_dense.cuh"

namespace cafeq {

// C = alpha * sum_t A_t B_t^T + beta * C0 + gamma * I  for one dense product (no batching)
struct DenseOut {
  const float* C0 = nullptr;
  long long ldc0 = 0;
  float* C = nullptr;
  long long ldc = 0;
  uint16_t *Chi = nullptr, *Clo = nullptr, *Cthi = nullptr, *Ctlo = nullptr;
  double* sq = nullptr;
  const int* run_flag = nullptr;
};

// A operands are [M, Ka] row-major (Ka = K, or K / a_rep_r when the contraction blocks of A are replicated),
// B operands [N, K] row-major; nterms pairs (A[t], B[t]).
static int launch_dense_tc(cudaStream_t st, int nterms, const uint16_t* const* A, const uint16_t* const* B, int M, int N, int K,
                           float alpha, float beta, float gamma, const DenseOut& o, int32_t* status, int a_rep_k = 0,
                           int a_rep_r = 1) {
  TgOperand oa[TG_MAX_TERMS], ob[TG_MAX_TERMS];
  const long long Ka = (a_rep_r > 1) ? K / a_rep_r : K;
  for (int t = 0; t < nterms; ++t) {
    oa[t] = TgOperand{A[t], M, Ka, Ka};
    ob[t] = TgOperand{B[t], N, K, K};
  }
  TgParams p;
  memset(&p, 0, sizeof(p));
  p.M = M; p.N = N; p.K = K;
  p.batch = 1;
  p.nterms = nterms;
  p.divA = 1;
  p.a_rep_k = a_rep_k > 0 ? a_rep_k : K;
  p.a_rep_r = a_rep_r;
  p.alpha = alpha; p.beta = beta; p.gamma = gamma;
  p.C0 = o.C0; p.ldc0 = o.ldc0;
  p.C = o.C; p.ldc = o.ldc;
  p.Chi = o.Chi; p.Clo = o.Clo; p.Cthi = o.Cthi; p.Ctlo = o.Ctlo;
  p.sq = o.sq; p.sq_stride = 0;
  p.run_flag = o.run_flag;
  p.status = status;
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return tg_launch(st, oa, ob, p);
}

static void launch_split_rect(cudaStream_t st, const float* X, int R, int C, long long ld, float scale, const double* inv_scale,
                              float* Y, float* YT, uint16_t* hi, uint16_t* lo, uint16_t* thi, uint16_t* tlo, const int32_t* status,
                              uint16_t* h3 = nullptr, uint16_t* t3 = nullptr) {
  dim3 grid((C + 31) / 32, (R + 31) / 32);
  CQ_LAUNCH(split_rect_kernel, grid, dim3(32, 8), 0, st, X, R, C, ld, scale, inv_scale, Y, YT, hi, lo, thi, tlo, status, h3, t3);
}

// The same product with both operands split three ways (x = x1 + x2 + x3, 24 significand bits): the six terms down to
// 2^-24 relative, as two launches of three terms that accumulate through the fp32 output `acc` (row-major [M, N],
// pitch N; it may be o.C).  fp32-grade accuracy: what is left is the rounding of the fp32 accumulators.
// A / B: {x1, x2, x3} in the layouts launch_dense_tc takes.
static int launch_dense_tc6(cudaStream_t st, const uint16_t* const* A, const uint16_t* const* B, int M, int N, int K, float alpha,
                            float beta, float gamma, const DenseOut& o, float* acc, int32_t* status, int a_rep_k = 0, int a_rep_r = 1) {
  const uint16_t* a1[3] = {A[0], A[1], A[0]};
  const uint16_t* b1[3] = {B[0], B[0], B[1]};
  DenseOut o1;
  o1.C0 = o.C0; o1.ldc0 = o.ldc0;
  o1.C = acc; o1.ldc = N;
  o1.run_flag = o.run_flag;
  int rc = launch_dense_tc(st, 3, a1, b1, M, N, K, alpha, beta, gamma, o1, status, a_rep_k, a_rep_r);
  if (rc) return rc;
  const uint16_t* a2[3] = {A[0], A[2], A[1]};
  const uint16_t* b2[3] = {B[2], B[0], B[1]};
  DenseOut o2 = o;
  o2.C0 = acc; o2.ldc0 = N;
  if (!o2.C) { o2.C = nullptr; }
  return launch_dense_tc(st, 3, a2, b2, M, N, K, alpha, 1.f, 0.f, o2, status, a_rep_k, a_rep_r);
}

// Scratch of the dense pair algebra for a pair with stored shapes U [h, d1], V [d3, rh]
struct DenseWS {
  int h, d1, d3, rh, k, r, D;
  float *U, *V, *Uhat, *Vhat, *P, *Bf, *X0T, *Y;
  uint16_t *Ph, *Pl, *PTh, *PTl;          // P [d1, d3] and its transpose [d3, d1]
  uint16_t *UTh, *UTl;                    // transposed splits of a [h, d1] matrix: [d1, h]
  uint16_t *Vh, *Vl;                      // splits of a [d3, rh] matrix
  uint16_t *Awh, *Awl;                    // the (wide) matrix being pseudo-inverted [m, n]
  uint16_t *Yh, *Yl, *YTh[2], *YTl[2];    // iterate Y = X^T [m, n] and its transpose [n, m]
  uint16_t *CTh, *CTl;                    // transposed residual [m, m]
  uint16_t *Oh, *Ol, *O3;                 // pseudo-inverse result in the stored shape [h, D], split three ways
  uint16_t *P3, *PT3, *UT3, *V3, *Aw3, *Y3;  // third terms of the operands that take part in six-term products
  float* Cf;                              // fp32 accumulator of a six-term product [max(m, d1, d3), ...]
  float *qa, *qusel;                      // quantiser scratch: absmax, signed arg-max value
  int* qidx;
  double* sq;                             // [DENSE_SQ] accumulators: 0..: PQE history, 32..: iteration residuals
  int* flag;
};
constexpr int DENSE_SQ = 128;
constexpr int PINV_MAX_ITERS = 56;

static bool carve_dense(Bump& b, int h, int d1, int d3, int r, int k, int ng1, int ng2, DenseWS* w) {
  const size_t rh = (size_t)r * h, D = (size_t)(d1 > d3 ? d1 : d3);
  w->h = h; w->d1 = d1; w->d3 = d3; w->rh = (int)rh; w->k = k; w->r = r; w->D = (int)D;
  const size_t nU = (size_t)h * d1, nV = (size_t)d3 * rh, nP = (size_t)d1 * d3, nY = (size_t)h * D;
  const size_t m = (size_t)h < D ? (size_t)h : D;  // smaller side of any matrix that gets pseudo-inverted
  w->U = b.take<float>(nU); w->V = b.take<float>(nV);
  w->Uhat = b.take<float>(nU); w->Vhat = b.take<float>(nV);
  w->P = b.take<float>(nP);
  w->Bf = b.take<float>((size_t)h * d3);
  w->X0T = b.take<float>((size_t)d3 * h);
  w->Y = b.take<float>(nY);
  w->Ph = b.take<uint16_t>(nP); w->Pl = b.take<uint16_t>(nP); w->PTh = b.take<uint16_t>(nP); w->PTl = b.take<uint16_t>(nP);
  w->UTh = b.take<uint16_t>(nU); w->UTl = b.take<uint16_t>(nU);
  w->Vh = b.take<uint16_t>(nV); w->Vl = b.take<uint16_t>(nV);
  w->Awh = b.take<uint16_t>(nY); w->Awl = b.take<uint16_t>(nY);
  w->Yh = b.take<uint16_t>(nY); w->Yl = b.take<uint16_t>(nY);
  for (int q = 0; q < 2; ++q) { w->YTh[q] = b.take<uint16_t>(nY); w->YTl[q] = b.take<uint16_t>(nY); }
  w->CTh = b.take<uint16_t>(m * m); w->CTl = b.take<uint16_t>(m * m);
  w->Oh = b.take<uint16_t>(nY); w->Ol = b.take<uint16_t>(nY); w->O3 = b.take<uint16_t>(nY);
  w->P3 = b.take<uint16_t>(nP); w->PT3 = b.take<uint16_t>(nP);
  w->UT3 = b.take<uint16_t>(nU); w->V3 = b.take<uint16_t>(nV);
  w->Aw3 = b.take<uint16_t>(nY); w->Y3 = b.take<uint16_t>(nY);
  w->Cf = b.take<float>(m * m > nY ? m * m : nY);
  const size_t nq = ((size_t)h * ng1 > (size_t)d3 * ng2) ? (size_t)h * ng1 : (size_t)d3 * ng2;
  w->qa = b.take<float>(nq); w->qusel = b.take<float>(nq); w->qidx = b.take<int>(nq);
  w->sq = b.take<double>(DENSE_SQ);
  w->flag = b.take<int>(64);
  return !b.overflow;
}

static size_t dense_scratch_bytes(int h, int d1, int d3, int r, int k, int ng1, int ng2) {
  Bump b(nullptr, (size_t)-1);
  DenseWS w;
  carve_dense(b, h, d1, d3, r, k, ng1, ng2, &w);
  return b.used + 4096;
}

// out (hi / lo, shape [R, C] of S) = pinv(S^T) = pinv(S)^T by the Newton-Schulz iteration X <- X + X (I - A X) on
// the wide orientation A of S ([m, n], m <= n), carried as Y = X^T so that every product has both operands
// contraction-major.  Start X0 = A^T / c with c = 1.25 x a power-iteration estimate of sigma_max(A)^2, capped by
// ||A||_F^2: the eigenvalues of A X0 lie in (0, 2) (the estimate is from below and a few percent off at most; the
// iteration converges for anything below 2), to the Moore-Penrose inverse.  Scaling by sigma_max^2 instead of the
// always-safe ||A||_F^2 saves log2(stable rank) doublings of the smallest eigenvalue.  Stops on the device when ||I - A X||_F falls below 1e-3 (the next
// update squares it) or stalls (rank-deficient A); the remaining launches then return at once.
static void pinv_rows(cudaStream_t st, const float* S, int R, int C, DenseWS& w, int32_t* status) {
  const bool wide = R <= C;
  const int m = wide ? R : C, n = wide ? C : R;
  double* fro = w.sq + 120;
  double* rs = w.sq + 32;  // residuals per iteration
  CQ_LAUNCH(zero_f64_kernel, 1, 128, 0, st, w.sq + 32, DENSE_SQ - 32);
  CQ_LAUNCH(set_int_kernel, 1, 1, 0, st, w.flag, 1);
  CQ_LAUNCH(sqsum_f32_kernel, grid_for((long long)R * C), 256, 0, st, S, (long long)R * C, fro);
  double* sig2 = w.sq + 123;
  {
    // power iteration in the (not yet used) iterate buffer: v [C], v2 [C], u [R]
    float* v = w.Y;
    float* v2 = w.Y + C;
    float* u = w.Y + 2 * (size_t)C;
    double* nrm = w.sq + 121;  // two slots, used alternately
    constexpr int ROUNDS = 8;
    const int slices = (R + 511) / 512;
    CQ_LAUNCH(pw_init_kernel, (C + 255) / 256, 256, 0, st, v, C, nrm);
    CQ_LAUNCH(fill_f32_kernel, grid_for(C), 256, 0, st, v2, 0.f, (long long)C);
    for (int it = 0; it < ROUNDS; ++it) {
      CQ_LAUNCH(pw_rows_kernel, (unsigned)(((long long)R * 32 + 255) / 256), 256, 0, st, S, v, R, C, u);
      CQ_LAUNCH(pw_cols_kernel, dim3((C + 255) / 256, slices), 256, 0, st, S, u, R, C, 512, v2);
      CQ_LAUNCH(pw_norm_kernel, 32, 256, 0, st, v2, C, nrm + (it & 1));
      CQ_LAUNCH(pw_scale_kernel, (C + 255) / 256, 256, 0, st, v, v2, C, nrm + (it & 1), nrm + ((it + 1) & 1),
                (it == ROUNDS - 1) ? sig2 : nullptr, 1.25, fro);
    }
  }
  if (wide) {
    launch_split_rect(st, S, R, C, C, 1.f, nullptr, nullptr, nullptr, w.Awh, w.Awl, nullptr, nullptr, status, w.Aw3, nullptr);
    launch_split_rect(st, S, R, C, C, 1.f, sig2, w.Y, nullptr, w.Yh, w.Yl, w.YTh[0], w.YTl[0], status);
  } else {
    launch_split_rect(st, S, R, C, C, 1.f, nullptr, nullptr, nullptr, nullptr, nullptr, w.Awh, w.Awl, status, nullptr, w.Aw3);
    launch_split_rect(st, S, R, C, C, 1.f, sig2, nullptr, w.Y, w.YTh[0], w.YTl[0], w.Yh, w.Yl, status);
  }
  int cur = 0;
  for (int it = 0; it < PINV_MAX_ITERS; ++it) {
    {  // C = I - A X, kept transposed
      const uint16_t* a[3] = {w.Awh, w.Awl, w.Awh};
      const uint16_t* bb[3] = {w.Yh, w.Yh, w.Yl};
      DenseOut o;
      o.Cthi = w.CTh; o.Ctlo = w.CTl; o.sq = rs + it; o.run_flag = w.flag;
      launch_dense_tc(st, 3, a, bb, m, m, n, -1.f, 0.f, 1.f, o, status);
    }
    {  // Y += C^T Y
      const uint16_t* a[3] = {w.CTh, w.CTl, w.CTh};
      const uint16_t* bb[3] = {w.YTh[cur], w.YTh[cur], w.YTl[cur]};
      DenseOut o;
      o.C0 = w.Y; o.ldc0 = n; o.C = w.Y; o.ldc = n;
      o.Chi = w.Yh; o.Clo = w.Yl; o.Cthi = w.YTh[cur ^ 1]; o.Ctlo = w.YTl[cur ^ 1];
      o.run_flag = w.flag;
      launch_dense_tc(st, 3, a, bb, m, n, m, 1.f, 1.f, 0.f, o, status);
    }
    CQ_LAUNCH(pinv_control_kernel, 1, 1, 0, st, rs, it, 1e-6, w.flag, m, status);
    cur ^= 1;
  }
  // The loop above stops at the accuracy of its three-term products (residual entries of a few 1e-7).  One more
  // step with the residual evaluated over three-way splits (fp32-grade) squares what is left: the quantised targets
  // of Algorithm 1 then agree with a float64 pseudo-inverse except at rounding ties.  The correction C^T Y is small,
  // three terms are enough for it.  (A rank-deficient matrix stalls where it stalled before: the step changes nothing.)
  {
    launch_split_rect(st, w.Y, m, n, n, 1.f, nullptr, nullptr, nullptr, w.Yh, w.Yl, w.YTh[0], w.YTl[0], status, w.Y3, nullptr);
    const uint16_t* a[3] = {w.Awh, w.Awl, w.Aw3};
    const uint16_t* bb[3] = {w.Yh, w.Yl, w.Y3};
    DenseOut o;
    o.Cthi = w.CTh; o.Ctlo = w.CTl;
    launch_dense_tc6(st, a, bb, m, m, n, -1.f, 0.f, 1.f, o, w.Cf, status);
    const uint16_t* a2[3] = {w.CTh, w.CTl, w.CTh};
    const uint16_t* b2[3] = {w.YTh[0], w.YTh[0], w.YTl[0]};
    DenseOut o2;
    o2.C0 = w.Y; o2.ldc0 = n; o2.C = w.Y; o2.ldc = n;
    launch_dense_tc(st, 3, a2, b2, m, n, m, 1.f, 1.f, 0.f, o2, status);
  }
  if (wide) launch_split_rect(st, w.Y, m, n, n, 1.f, nullptr, nullptr, nullptr, w.Oh, w.Ol, nullptr, nullptr, status, w.O3, nullptr);
  else launch_split_rect(st, w.Y, m, n, n, 1.f, nullptr, nullptr, nullptr, nullptr, nullptr, w.Oh, w.Ol, status, nullptr, w.O3);
}

}  // namespace cafeq

namespace cafeq {

// Group quantiser on an fp32 matrix T [rows, cols] (groups of g along the row): codes, scales, dequantised values
static void quant_matrix(cudaStream_t st, const float* T, int rows, int cols, int g, int bits, int8_t* codes, float* scales,
                         float* That, DenseWS& w, int32_t* status) {
  Geo G;
  memset(&G, 0, sizeof(G));
  G.d_out = rows; G.d_in = cols; G.g = g; G.ng = cols / g; G.ld = cols; G.n = (long long)rows * cols;
  launch_absmax(st, T, cols, G, w.qa, w.qusel, w.qidx, status);
  CQ_LAUNCH(quant_kernel, grid_for(G.n), 256, 0, st, T, (long long)cols, rows, cols, g, w.qa, qmax_of(bits), nullptr,
            CAFEQ_OFFSETS_NONE, nullptr, That, codes, status);
  if (scales)
    CQ_LAUNCH(scales_kernel, grid_for((long long)rows * G.ng), 256, 0, st, w.qa, scales, (long long)rows * G.ng, qmax_of(bits), status);
}

// P = U_exp^T V^T for stored U [h, d1], V [d3, rh] (fp32): fp32 P [d1, d3] with its splits in w.Ph/Pl/PTh/PTl
// (six terms over three-way splits: P is the reference every least-squares target of Algorithm 1 is measured
// against, so it is formed to fp32 accuracy; its own third-term splits follow for the target products)
static void dense_product(cudaStream_t st, const float* U, const float* V, DenseWS& w, float* P, int32_t* status) {
  launch_split_rect(st, U, w.h, w.d1, w.d1, 1.f, nullptr, nullptr, nullptr, nullptr, nullptr, w.UTh, w.UTl, status, nullptr, w.UT3);
  launch_split_rect(st, V, w.d3, w.rh, w.rh, 1.f, nullptr, nullptr, nullptr, w.Vh, w.Vl, nullptr, nullptr, status, w.V3, nullptr);
  const uint16_t* a[3] = {w.UTh, w.UTl, w.UT3};
  const uint16_t* b[3] = {w.Vh, w.Vl, w.V3};
  DenseOut o;
  o.C = P; o.ldc = w.d3; o.Chi = w.Ph; o.Clo = w.Pl; o.Cthi = w.PTh; o.Ctlo = w.PTl;
  launch_dense_tc6(st, a, b, w.d1, w.d3, w.rh, 1.f, 0.f, 0.f, o, P, status, w.k, w.r);
  launch_split_rect(st, P, w.d1, w.d3, w.d3, 1.f, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, status, w.P3, w.PT3);
}

// *sq += || Uhat_exp^T Vhat^T - P ||_F^2 ; optionally stores the residual R [d1, d3]
static void dense_pqe(cudaStream_t st, const float* Uhat, const float* Vhat, const float* P, DenseWS& w, double* sq, float* R,
                      int32_t* status, bool keep_splits = false) {
  launch_split_rect(st, Uhat, w.h, w.d1, w.d1, 1.f, nullptr, nullptr, nullptr, nullptr, nullptr, w.UTh, w.UTl, status);
  launch_split_rect(st, Vhat, w.d3, w.rh, w.rh, 1.f, nullptr, nullptr, nullptr, w.Vh, w.Vl, nullptr, nullptr, status);
  const uint16_t* a[3] = {w.UTh, w.UTl, w.UTh};
  const uint16_t* b[3] = {w.Vh, w.Vh, w.Vl};
  DenseOut o;
  o.C0 = P; o.ldc0 = w.d3; o.C = R; o.ldc = w.d3; o.sq = sq;
  if (keep_splits) {  // the residual and its transpose as operands of the backward products
    o.Chi = w.Ph; o.Clo = w.Pl; o.Cthi = w.PTh; o.Ctlo = w.PTl;
  }
  launch_dense_tc(st, 3, a, b, w.d1, w.d3, w.rh, 1.f, -1.f, 0.f, o, status, w.k, w.r);
}

// Algorithm 1 on the transformed pair held in w.U [h, d1], w.V [d3, rh] (fp32, stored layout with r replicas of
// every inner block on the V side).  With E the replica expansion, the V update is Q((pinv((E Uhat)^T) P)^T) =
// Q(expand(pinv(Uhat^T) P) / r) (Uhat^T of full column rank) and the U update is Q((P pinv(fold(Vhat^T)))^T),
// which is the printed algorithm when r = 1.  pqe_hist: fp32 [2 iters + 1].
static void alg1_run(cudaStream_t st, int bits, int g1, int g2, int iters, int8_t* codes1, float* scales1, int8_t* codes2,
                     float* scales2, float* pqe_hist, DenseWS& w, int32_t* status) {
  CQ_LAUNCH(zero_f64_kernel, 1, 128, 0, st, w.sq, DENSE_SQ);
  dense_product(st, w.U, w.V, w, w.P, status);
  quant_matrix(st, w.U, w.h, w.d1, g1, bits, codes1, scales1, w.Uhat, w, status);
  quant_matrix(st, w.V, w.d3, w.rh, g2, bits, codes2, scales2, w.Vhat, w, status);
  dense_pqe(st, w.Uhat, w.Vhat, w.P, w, w.sq + 0, nullptr, status);
  for (int it = 0; it < iters; ++it) {
    // V side: X0^T [d3, h] = P^T pinv(Uhat^T)^T, then expand the replicas
    pinv_rows(st, w.Uhat, w.h, w.d1, w, status);
    {
      const uint16_t* a[3] = {w.PTh, w.PTl, w.PT3};
      const uint16_t* b[3] = {w.Oh, w.Ol, w.O3};
      DenseOut o;
      o.C = w.X0T; o.ldc = w.h;
      launch_dense_tc6(st, a, b, w.d3, w.h, w.d1, 1.f, 0.f, 0.f, o, w.X0T, status);
    }
    CQ_LAUNCH(expand_cols_kernel, grid_for((long long)w.d3 * w.rh), 256, 0, st, w.X0T, w.d3, w.h, w.k, w.r, 1.f / (float)w.r, w.V);
    quant_matrix(st, w.V, w.d3, w.rh, g2, bits, codes2, scales2, w.Vhat, w, status);
    dense_pqe(st, w.Uhat, w.Vhat, w.P, w, w.sq + 2 * it + 1, nullptr, status);
    // U side: U' [h, d1] = pinv(Bf)^T P^T with Bf = fold(Vhat^T) [h, d3]
    {
      dim3 grid((w.d3 + 31) / 32, w.h / 32);
      CQ_LAUNCH(fold_transpose_kernel, grid, dim3(32, 8), 0, st, w.Vhat, w.d3, w.h, w.k, w.r, w.Bf);
    }
    pinv_rows(st, w.Bf, w.h, w.d3, w, status);
    {
      const uint16_t* a[3] = {w.Oh, w.Ol, w.O3};
      const uint16_t* b[3] = {w.Ph, w.Pl, w.P3};
      DenseOut o;
      o.C = w.U; o.ldc = w.d1;
      launch_dense_tc6(st, a, b, w.h, w.d1, w.d3, 1.f, 0.f, 0.f, o, w.U, status);
    }
    quant_matrix(st, w.U, w.h, w.d1, g1, bits, codes1, scales1, w.Uhat, w, status);
    dense_pqe(st, w.Uhat, w.Vhat, w.P, w, w.sq + 2 * it + 2, nullptr, status);
  }
  CQ_LAUNCH(sqrt_hist_kernel, 1, 128, 0, st, w.sq, pqe_hist, 2 * iters + 1);
}

}  // namespace cafeq
