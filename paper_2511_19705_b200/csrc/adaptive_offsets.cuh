// Learned rounding offsets for a coupled product (cafeq_adaptive_round, mode CAFEQ_ROUND_LEARNED_OFFSETS).
//
// The paper's adaptive rounding is Algorithm 1; this mode is the gradient-learned alternative the workload statement
// names, defined by this library: scales stay at their round-to-nearest values, codes are floor(x) + rho with soft
// offsets rho in [0, 1] started at the fractional parts (zero error).  Every iteration moves the first factor's
// offsets along d = (dL/drho) / (per-entry curvature) with an exact line search (Eq. 5 squared is quadratic in one
// factor's offsets), then the second factor's at the updated first, then pushes both towards the nearer of {0, 1}
// by a weight that grows over the run; at the end the offsets are hardened at 1/2.  Shape-agnostic: every product runs on the plain fp32 product kernel, so tiny
// matrices (for comparison with exhaustive enumeration) go through the same code as large ones.
// Included by cafeq_api.cu (uses its launch helpers and workspace carving).
#pragma once

namespace cafeq {

constexpr float LEARN_LAMBDA = 0.5f;  // final weight of the push towards {0, 1}

// rho = x - floor(x), x = fl(u / s) (the quantiser's own fp32 quotient)
__global__ void offsets_init_kernel(const float* __restrict__ U, int rows, int cols, int g, const float* __restrict__ a, float qmax,
                                    float* __restrict__ rho) {
  const int ng = cols / g;
  const long long n = (long long)rows * cols;
  for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
    const int row = (int)(e / cols), col = (int)(e - (long long)row * cols);
    const float s = __fdiv_rn(a[(long long)row * ng + col / g], qmax);
    const float x = (s > 0.f) ? __fdiv_rn(U[e], s) : 0.f;
    rho[e] = x - floorf(x);
  }
}

// Bf[B k + j][y] = sum_rep V[y][(B r + rep) k + j]   (V [d3, r h] -> Bf [h, d3]); any k
__global__ void fold_t_any_kernel(const float* __restrict__ V, int d3, int h, int k, int r, float* __restrict__ Bf) {
  const long long n = (long long)h * d3;
  for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
    const int l = (int)(e / d3), y = (int)(e - (long long)l * d3);
    const int B = l / k, j = l - B * k;
    float s = 0.f;
    for (int rep = 0; rep < r; ++rep) s += V[(long long)y * r * h + (long long)(B * r + rep) * k + j];
    Bf[e] = s;
  }
}

// out[row] = scale * sum_c X[row][c]^2, one warp per row
__global__ void row_sumsq_kernel(const float* __restrict__ X, int rows, int cols, float scale, float* __restrict__ out) {
  const long long w = (blockIdx.x * (long long)blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (w >= rows) return;
  double s = 0.0;
  for (int c = lane; c < cols; c += 32) {
    const float v = X[w * cols + c];
    s += (double)v * v;
  }
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if (lane == 0) out[w] = (float)((double)scale * s);
}

// Search direction of one factor: d = g / (s H) in offset space and s d in the space of the dequantised values, for
// the entries that have an offset (not the group's arg-max, scale > 0, curvature > 0), zero elsewhere.  H is indexed
// by the row (hrow = 1) or by the column folded over the replicas (hrow = 0: column l of [., r h] uses
// H[(l / (r k)) k + l mod k]).
__global__ void offsets_direction_kernel(const float* gX /* may be d_rho */, const float* __restrict__ U, int rows, int cols, int g,
                                         const float* __restrict__ a, float qmax, const float* __restrict__ H, int hrow, int k,
                                         int r, float* d_rho, float* __restrict__ d_val) {
  const int ng = cols / g;
  const long long n = (long long)rows * cols;
  for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
    const int row = (int)(e / cols), col = (int)(e - (long long)row * cols);
    const float av = a[(long long)row * ng + col / g];
    const float s = __fdiv_rn(av, qmax);
    float hv;
    if (hrow) hv = H[row];
    else {
      const int Bq = col / k, j = col - Bq * k;
      hv = H[(Bq / r) * k + j];
    }
    float d = 0.f;
    if (s > 0.f && hv > 0.f && fabsf(U[e]) < av) d = gX[e] / (s * hv);
    d_rho[e] = d;
    d_val[e] = s * d;
  }
}

// rho <- clip(rho - alpha d, 0, 1) with the exact line-search step alpha = <R, D> / <D, D> (0 when D = 0)
__global__ void offsets_step_kernel(float* __restrict__ rho, const float* __restrict__ d_rho, long long n, const double* __restrict__ rd,
                                    const double* __restrict__ dd) {
  const float alpha = (*dd > 0.0) ? (float)(*rd / *dd) : 0.f;
  for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x)
    rho[e] = fminf(fmaxf(rho[e] - alpha * d_rho[e], 0.f), 1.f);
}

// rho <- clip(rho + lam (2 rho - 1), 0, 1)
__global__ void offsets_push_kernel(float* __restrict__ rho, long long n, float lam) {
  for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
    const float rv = rho[e];
    rho[e] = fminf(fmaxf(rv + lam * (2.f * rv - 1.f), 0.f), 1.f);
  }
}

__global__ void harden_kernel(float* __restrict__ rho, long long n) {
  for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x)
    rho[e] = (rho[e] >= 0.5f) ? 1.f : 0.f;
}

struct LearnWS {
  float *U, *V, *Uh, *Vh, *rho1, *rho2, *P, *R, *D, *Bf, *gU, *G2, *gV, *T1, *T2, *H1, *H2;
  float *a1, *u1, *a2, *u2;
  int *i1, *i2;
  double* acc;
};

static bool carve_learn(Bump& b, const Geo& G1, const Geo& G2, LearnWS* w) {
  const size_t n1 = (size_t)G1.n, n2 = (size_t)G2.n, h = (size_t)G1.d_out, d1 = (size_t)G1.d_in, d3 = (size_t)G2.d_out;
  w->U = b.take<float>(n1); w->Uh = b.take<float>(n1); w->rho1 = b.take<float>(n1); w->gU = b.take<float>(n1);
  w->V = b.take<float>(n2); w->Vh = b.take<float>(n2); w->rho2 = b.take<float>(n2); w->gV = b.take<float>(n2);
  w->T1 = b.take<float>(n1); w->T2 = b.take<float>(n2);
  w->P = b.take<float>(d1 * d3); w->R = b.take<float>(d1 * d3); w->D = b.take<float>(d1 * d3);
  w->Bf = b.take<float>(h * d3); w->G2 = b.take<float>(d3 * h);
  w->H1 = b.take<float>(h); w->H2 = b.take<float>(h);
  w->a1 = b.take<float>((size_t)G1.d_out * G1.ng); w->u1 = b.take<float>((size_t)G1.d_out * G1.ng);
  w->i1 = b.take<int>((size_t)G1.d_out * G1.ng);
  w->a2 = b.take<float>((size_t)G2.d_out * G2.ng); w->u2 = b.take<float>((size_t)G2.d_out * G2.ng);
  w->i2 = b.take<int>((size_t)G2.d_out * G2.ng);
  w->acc = b.take<double>(64);
  return !b.overflow;
}

// C = alpha * A B on the plain fp32 kernel with explicit strides (A[m][l] at sAm, sAk; B[l][n] at sBk, sBn)
static void learn_gemm(cudaStream_t st, const float* A, long long sAm, long long sAk, const float* B, long long sBk, long long sBn,
                       float* C, int M, int N, int K, float alpha, const int32_t* status) {
  GemmArgs g = gemm_defaults(status);
  g.M = M; g.N = N; g.K = K;
  g.A = A; g.sAm = sAm; g.sAk = sAk;
  g.B = B; g.sBk = sBk; g.sBn = sBn;
  g.C = C; g.sCm = N; g.sCn = 1;
  g.alpha = alpha;
  g.mode = GEMM_STORE;
  launch_gemm(st, g);
}

// w.U / w.V hold the transformed pair (fp32, stored layouts).  pqe_hist: fp32 [iters + 2] (see cafeq.h).
static void learned_offsets_run(cudaStream_t st, int bits, const Geo& G1, const Geo& G2, int iters, int8_t* codes1, float* scales1,
                                int8_t* codes2, float* scales2, float* pqe_hist, LearnWS& w, int32_t* status) {
  const int h = G1.d_out, d1 = G1.d_in, d3 = G2.d_out, rh = G2.d_in, k = G1.k, r = G2.r;
  const float qm = qmax_of(bits);
  const long long n1 = G1.n, n2 = G2.n, np = (long long)d1 * d3;
  Geo A1 = G1, A2 = G2;  // fp32 matrices with pitch = width
  A1.ld = d1; A2.ld = rh;
  CQ_LAUNCH(zero_f64_kernel, 1, 64, 0, st, w.acc, 64);
  launch_pair_product(st, w.U, 0, d1, w.V, 0, rh, G1, G2, w.P, status);
  launch_absmax(st, w.U, d1, A1, w.a1, w.u1, w.i1, status);
  launch_absmax(st, w.V, rh, A2, w.a2, w.u2, w.i2, status);
  auto quant = [&](const void* off1, const void* off2, int kind, int8_t* c1, int8_t* c2) {
    CQ_LAUNCH(quant_kernel, grid_for(n1), 256, 0, st, w.U, (long long)d1, h, d1, G1.g, w.a1, qm, off1, kind, nullptr, w.Uh, c1, status);
    CQ_LAUNCH(quant_kernel, grid_for(n2), 256, 0, st, w.V, (long long)rh, d3, rh, G2.g, w.a2, qm, off2, kind, nullptr, w.Vh, c2, status);
  };
  auto residual = [&](double* acc) {  // R = Uh_exp^T Vh^T - P, *acc = ||R||_F^2
    launch_pair_product(st, w.Uh, 0, d1, w.Vh, 0, rh, G1, G2, w.R, status);
    CQ_LAUNCH(resid_sq_kernel, grid_for(np), 256, 0, st, w.R, w.P, np, acc, status);
  };
  // history[0]: independent round-to-nearest
  quant(nullptr, nullptr, CAFEQ_OFFSETS_NONE, nullptr, nullptr);
  residual(w.acc + 0);
  CQ_LAUNCH(offsets_init_kernel, grid_for(n1), 256, 0, st, w.U, h, d1, G1.g, w.a1, qm, w.rho1);
  CQ_LAUNCH(offsets_init_kernel, grid_for(n2), 256, 0, st, w.V, d3, rh, G2.g, w.a2, qm, w.rho2);
  const unsigned hrows = (unsigned)(((long long)h * 32 + 255) / 256);
  double* ls = w.acc + 48;  // line-search accumulators: <R, D>, <D, D>
  for (int t = 1; t <= iters; ++t) {
    quant(w.rho1, w.rho2, CAFEQ_OFFSETS_SOFT_F32, nullptr, nullptr);
    residual(w.acc + t);
    // first factor: Bf = fold(Vh^T) [h, d3], gU = 2 Bf R^T [h, d1], H1 = 2 ||Bf rows||^2, direction, line search
    CQ_LAUNCH(fold_t_any_kernel, grid_for((long long)h * d3), 256, 0, st, w.Vh, d3, h, k, r, w.Bf);
    learn_gemm(st, w.Bf, d3, 1, w.R, 1, d3, w.gU, h, d1, d3, 2.f, status);
    CQ_LAUNCH(row_sumsq_kernel, hrows, 256, 0, st, w.Bf, h, d3, 2.f, w.H1);
    CQ_LAUNCH(offsets_direction_kernel, grid_for(n1), 256, 0, st, w.gU, w.U, h, d1, G1.g, w.a1, qm, w.H1, 1, k, 1, w.gU, w.T1);
    launch_pair_product(st, w.T1, 0, d1, w.Vh, 0, rh, G1, G2, w.D, status);
    CQ_LAUNCH(zero_f64_kernel, 1, 32, 0, st, ls, 2);
    CQ_LAUNCH(dot_f32_kernel, grid_for(np), 256, 0, st, w.R, w.D, np, ls + 0);
    CQ_LAUNCH(sqsum_f32_kernel, grid_for(np), 256, 0, st, w.D, np, ls + 1);
    CQ_LAUNCH(offsets_step_kernel, grid_for(n1), 256, 0, st, w.rho1, w.gU, n1, ls + 0, ls + 1);
    // second factor at the updated first: G2 = 2 R^T Uh^T [d3, h] expanded over the replicas, H2 = 2 ||Uh rows||^2
    CQ_LAUNCH(quant_kernel, grid_for(n1), 256, 0, st, w.U, (long long)d1, h, d1, G1.g, w.a1, qm, w.rho1, CAFEQ_OFFSETS_SOFT_F32, nullptr,
              w.Uh, nullptr, status);
    residual(w.acc + 40);
    learn_gemm(st, w.R, 1, d3, w.Uh, 1, d1, w.G2, d3, h, d1, 2.f, status);
    CQ_LAUNCH(expand_cols_kernel, grid_for(n2), 256, 0, st, w.G2, d3, h, k, r, 1.f, w.gV);
    CQ_LAUNCH(row_sumsq_kernel, hrows, 256, 0, st, w.Uh, h, d1, 2.f, w.H2);
    CQ_LAUNCH(offsets_direction_kernel, grid_for(n2), 256, 0, st, w.gV, w.V, d3, rh, G2.g, w.a2, qm, w.H2, 0, k, r, w.gV, w.T2);
    launch_pair_product(st, w.Uh, 0, d1, w.T2, 0, rh, G1, G2, w.D, status);
    CQ_LAUNCH(zero_f64_kernel, 1, 32, 0, st, ls, 2);
    CQ_LAUNCH(dot_f32_kernel, grid_for(np), 256, 0, st, w.R, w.D, np, ls + 0);
    CQ_LAUNCH(sqsum_f32_kernel, grid_for(np), 256, 0, st, w.D, np, ls + 1);
    CQ_LAUNCH(offsets_step_kernel, grid_for(n2), 256, 0, st, w.rho2, w.gV, n2, ls + 0, ls + 1);
    const float lam = LEARN_LAMBDA * (float)t / (float)iters;
    CQ_LAUNCH(offsets_push_kernel, grid_for(n1), 256, 0, st, w.rho1, n1, lam);
    CQ_LAUNCH(offsets_push_kernel, grid_for(n2), 256, 0, st, w.rho2, n2, lam);
  }
  CQ_LAUNCH(harden_kernel, grid_for(n1), 256, 0, st, w.rho1, n1);
  CQ_LAUNCH(harden_kernel, grid_for(n2), 256, 0, st, w.rho2, n2);
  quant(w.rho1, w.rho2, CAFEQ_OFFSETS_SOFT_F32, codes1, codes2);
  residual(w.acc + iters + 1);
  CQ_LAUNCH(scales_kernel, grid_for((long long)h * G1.ng), 256, 0, st, w.a1, scales1, (long long)h * G1.ng, qm, status);
  CQ_LAUNCH(scales_kernel, grid_for((long long)d3 * G2.ng), 256, 0, st, w.a2, scales2, (long long)d3 * G2.ng, qm, status);
  CQ_LAUNCH(sqrt_hist_kernel, 1, 128, 0, st, w.acc, pqe_hist, iters + 2);
}

}  // namespace cafeq
