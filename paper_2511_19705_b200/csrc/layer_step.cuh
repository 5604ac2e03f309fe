// Layer-level optimisation step: every single matrix and every coupled pair of one decoder layer advanced together.
//
// The problems of a layer are independent (Section 6 treats every matrix / pair on its own), so nothing here
// changes what one step computes (Section 4.1: gradient descent on Eq. 4; Section 4.2 / Appendix D: Adam on the
// LogSumExp surrogate plus the orthonormality penalty).  What changes is how the work is launched:
//   * the k x k algebra (block inverse, M^-1 path of the gradient, M M^T - I) runs once over the concatenated
//     operator blocks of all problems instead of once per problem;
//   * the transform pass and the sparse backward take all matrices of the same form in ONE persistent launch each;
//   * the backward reads an fp16 copy of the weights made once per layer, so its routed coefficients are a single
//     fp16 term and the product is issued once (see kernels_bwd.cuh);
//   * the LogSumExp normaliser is applied when the gradient is flushed (the routed coefficients are exp(t (a - max))
//     with the sign of the arg-max entry; dividing by Z afterwards is exact algebra), which removes one pass over
//     the group records;
//   * set-up and parameter update are one kernel each for the whole layer.
// This file is included by cafeq_api.cu after the per-problem paths, whose helpers it reuses.
#pragma once

namespace cafeq {

constexpr int LY_MAX_PROBS = 8;
static std::atomic<int> g_ly_dual{1};  // both forms of a layer in one pass launch and one backward launch
constexpr int LY_MAX_MATS = 2 * LY_MAX_PROBS;

// ------------------------------------------------------------------------------------------------
// kernels
// ------------------------------------------------------------------------------------------------
struct LyPrepArgs {
  int n, k;
  int blk0[LY_MAX_PROBS + 1];       // first operator block of problem p in the concatenated arrays
  const float* M[LY_MAX_PROBS];
  float* step_counter[LY_MAX_PROBS];
  int pair_blk0;                    // first block of the pairs (they come last); total blocks when there is none
  float* Mc;
  uint16_t* Ab;
  float* Mf;                        // fp32 parameters of the pair blocks, contiguous (orthonormality penalty)
  float* grad;                      // cleared: all blocks
  float* gMinv;                     // cleared: pair blocks
  uint4* zone;                      // cleared: the per-step accumulators of every matrix and problem
  long long zone_n16;
  double* rn;
  int rn_n;
  int* flag;
  const int32_t* status;
};

__global__ void __launch_bounds__(256) layer_prep_kernel(const LyPrepArgs a) {
  if (a.status && *a.status) return;
  const long long stride = (long long)gridDim.x * blockDim.x, t0 = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  const long long kk = (long long)a.k * a.k;
  const long long total4 = (long long)a.blk0[a.n] * kk / 4;   // k is a multiple of 64 and every pointer 16-byte aligned
  const long long pair0 = (long long)a.pair_blk0 * kk;
  for (long long q = t0; q < total4; q += stride) {
    const long long e = q * 4;
    const int b = (int)(e / kk);
    int p = 0;
    while (b >= a.blk0[p + 1]) ++p;
    const float4 m = *reinterpret_cast<const float4*>(a.M[p] + (e - (long long)a.blk0[p] * kk));
    const __nv_bfloat16 h0 = __float2bfloat16_rn(m.x), h1 = __float2bfloat16_rn(m.y);
    const __nv_bfloat16 h2 = __float2bfloat16_rn(m.z), h3 = __float2bfloat16_rn(m.w);
    *reinterpret_cast<float4*>(a.Mc + e) = make_float4(__bfloat162float(h0), __bfloat162float(h1), __bfloat162float(h2), __bfloat162float(h3));
    *reinterpret_cast<uint2*>(a.Ab + e) = make_uint2((uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16),
                                                     (uint32_t)__bfloat16_as_ushort(h2) | ((uint32_t)__bfloat16_as_ushort(h3) << 16));
    *reinterpret_cast<float4*>(a.grad + e) = make_float4(0.f, 0.f, 0.f, 0.f);
    if (e >= pair0) {
      *reinterpret_cast<float4*>(a.Mf + (e - pair0)) = m;
      *reinterpret_cast<float4*>(a.gMinv + e) = make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }
  for (long long e = t0; e < a.zone_n16; e += stride) a.zone[e] = make_uint4(0u, 0u, 0u, 0u);
  for (long long e = t0; e < a.rn_n; e += stride) a.rn[e] = 0.0;
  if (t0 == 0) {
    *a.flag = 0;
    for (int p = 0; p < a.n; ++p)
      if (a.step_counter[p]) *a.step_counter[p] += 1.f;
  }
}

// Column square norms of the inverse for the single matrices' blocks (blockIdx.y = block, all singles in one launch):
// c[b][t] = sum_i Minv[b][i][t]^2 and, for an input-axis matrix with one block per operator block, the group weights
// of Eq. 4: cw[G] += sum_{t in G} c[t].
struct LyColArgs {
  int n, k;
  int blk0[LY_MAX_PROBS + 1];   // block ranges of the singles (they come first)
  float* cw[LY_MAX_PROBS];      // null: only c is written
  int g[LY_MAX_PROBS];
};

__global__ void __launch_bounds__(256) layer_colnorm_kernel(const float* __restrict__ X, float* __restrict__ c, const LyColArgs a) {
  __shared__ float part[8][33];
  const int b = blockIdx.y, t = blockIdx.x * 32 + threadIdx.x, k = a.k;
  int p = 0;
  while (b >= a.blk0[p + 1]) ++p;
  const float* Xb = X + (size_t)b * k * k;
  float s = 0.f;
  for (int i = threadIdx.y; i < k; i += 8) {
    const float v = Xb[(size_t)i * k + t];
    s = fmaf(v, v, s);
  }
  part[threadIdx.y][threadIdx.x] = s;
  __syncthreads();
  if (threadIdx.y == 0) {
    float tot = 0.f;
#pragma unroll
    for (int q = 0; q < 8; ++q) tot += part[q][threadIdx.x];
    c[(size_t)b * k + t] = tot;
    float* cw = a.cw[p];
    if (cw) {
      const int g = a.g[p];
      const int col = (b - a.blk0[p]) * k + t;  // position along the transformed axis of that matrix
      if (g >= 32) {
        for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
        if (threadIdx.x == 0) atomicAdd(&cw[col / g], tot);
      } else {
        atomicAdd(&cw[col / g], tot);
      }
    }
  }
}

// dL/dMinv of Eq. 4 for all single matrices: out[b][i][t] = scale_p * Minv[b][i][t] * A_t, A_t from the matrix's
// group sums (input axis, one block per operator block) or from its per-row sums.
struct LyGminvArgs {
  int n, k;
  int blk0[LY_MAX_PROBS + 1];
  const float* A[LY_MAX_PROBS];
  const float* Agrp[LY_MAX_PROBS];
  int g[LY_MAX_PROBS];
  float scale[LY_MAX_PROBS];
};

__global__ void __launch_bounds__(256) layer_gminv_kernel(const float* __restrict__ Minv, float* __restrict__ out, const LyGminvArgs a) {
  const long long kk = (long long)a.k * a.k;
  const long long total4 = (long long)a.blk0[a.n] * kk / 4;
  for (long long q = blockIdx.x * (long long)blockDim.x + threadIdx.x; q < total4; q += (long long)gridDim.x * blockDim.x) {
    const long long e = q * 4;
    const int b = (int)(e / kk);
    int p = 0;
    while (b >= a.blk0[p + 1]) ++p;
    const int t = (int)(e % a.k);
    const int bl = b - a.blk0[p];
    float At[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) At[j] = a.Agrp[p] ? a.Agrp[p][(bl * a.k + t + j) / a.g[p]] : a.A[p][bl * a.k + t + j];
    const float4 x = *reinterpret_cast<const float4*>(Minv + e);
    const float sc = a.scale[p];
    *reinterpret_cast<float4*>(out + e) = make_float4(sc * x.x * At[0], sc * x.y * At[1], sc * x.z * At[2], sc * x.w * At[3]);
  }
}

// LogSumExp over the group maxima of both factors of every pair (blockIdx.y = pair): unnormalised routed
// coefficients exp(t (a - max)) * sign(U at the arg-max) and Z = sum exp(t (a - max)); the maximum comes from the
// transform passes (one word per matrix).
struct LyLseArgs {
  const float* a[LY_MAX_PROBS][2];
  const float* u[LY_MAX_PROBS][2];
  float* c[LY_MAX_PROBS][2];
  long long n[LY_MAX_PROBS][2];
  const float* vmax[LY_MAX_PROBS][2];
  float t[LY_MAX_PROBS];
  double* Z[LY_MAX_PROBS];
  float* amax[LY_MAX_PROBS];
  const int32_t* status;
};

__global__ void __launch_bounds__(256) layer_lse_kernel(const LyLseArgs g) {
  if (g.status && *g.status) return;
  __shared__ double red[32];
  const int p = blockIdx.y;
  const float mx = fmaxf(*g.vmax[p][0], *g.vmax[p][1]);
  const float t = g.t[p];
  const long long n1 = g.n[p][0], n = n1 + g.n[p][1];
  double local = 0.0;
  for (long long w = blockIdx.x * (long long)blockDim.x + threadIdx.x; w < n; w += (long long)gridDim.x * blockDim.x) {
    const int s = w < n1 ? 0 : 1;
    const long long i = s ? w - n1 : w;
    const float u = g.u[p][s][i];
    const float e = expf(t * (g.a[p][s][i] - mx));
    g.c[p][s][i] = (u > 0.f) ? e : ((u < 0.f) ? -e : 0.f);
    local += (double)e;
  }
  const double sum = block_sum_double(local, red);
  if (threadIdx.x == 0) {
    atomicAdd(g.Z[p], sum);
    if (blockIdx.x == 0) *g.amax[p] = mx;
  }
}

// Losses, the orthonormality term of the gradient and the parameter update of every problem (blockIdx.y = problem).
struct LyFinishArgs {
  int k;
  int blk0[LY_MAX_PROBS + 1];
  float* M[LY_MAX_PROBS];
  float* state[LY_MAX_PROBS];
  float* hist[LY_MAX_PROBS];
  int pair[LY_MAX_PROBS], optimizer[LY_MAX_PROBS];
  float lr[LY_MAX_PROBS], b1[LY_MAX_PROBS], b2[LY_MAX_PROBS], eps[LY_MAX_PROBS];
  float lambda[LY_MAX_PROBS], t[LY_MAX_PROBS], sqrt_h[LY_MAX_PROBS];
  const double* acc[LY_MAX_PROBS];   // single: {Eq. 4}; pair: {Z}
  const float* amax[LY_MAX_PROBS];
  const double* orth_sq;             // per pair block: ||(M M^T - I)_b||_F^2, indexed from pair_blk0
  int pair_blk0;
  const float* grad;
  const float* RM;                   // (M M^T - I) M, pair blocks, indexed from pair_blk0
  const int32_t* status;
};

__global__ void __launch_bounds__(256) layer_finish_kernel(const LyFinishArgs f) {
  if (f.status && *f.status) return;
  const int p = blockIdx.y;
  const long long kk = (long long)f.k * f.k;
  const long long off = (long long)f.blk0[p] * kk, n = (long long)(f.blk0[p + 1] - f.blk0[p]) * kk;
  float orth_f = 0.f;
  double r2 = 0.0;
  if (f.pair[p]) {
    for (int b = f.blk0[p]; b < f.blk0[p + 1]; ++b) r2 += f.orth_sq[b - f.pair_blk0];
    const double nrm = sqrt(r2);
    if (f.lambda[p] != 0.f && nrm >= 1e-5 * (double)f.sqrt_h[p]) orth_f = (float)(2.0 * f.lambda[p] / (nrm * f.sqrt_h[p]));
  }
  if (blockIdx.x == 0 && threadIdx.x == 0 && f.hist[p]) {
    float loss;
    if (f.pair[p]) {
      const float lse = *f.amax[p] + (float)(log(f.acc[p][0]) / (double)f.t[p]);
      loss = lse + f.lambda[p] * (float)(sqrt(r2) / (double)f.sqrt_h[p]);
    } else {
      loss = (float)f.acc[p][0];
    }
    f.hist[p][0] = loss;
    f.hist[p][1] = nanf("");
  }
  float4* M4 = reinterpret_cast<float4*>(f.M[p]);
  const float4* g4 = reinterpret_cast<const float4*>(f.grad + off);
  const float4* RM4 = f.pair[p] ? reinterpret_cast<const float4*>(f.RM + (off - (long long)f.pair_blk0 * kk)) : nullptr;
  const float lr = f.lr[p];
  const long long n4 = n / 4;
  const bool adam = f.optimizer[p] != CAFEQ_OPT_GD;
  float b1 = 0.f, b2 = 0.f, eps = 0.f, c1 = 1.f, c2 = 1.f;
  float4 *m4 = nullptr, *v4 = nullptr;
  if (adam) {
    float* state = f.state[p];
    const float step = state[0];
    b1 = f.b1[p]; b2 = f.b2[p]; eps = f.eps[p];
    c1 = 1.f - powf(b1, step);
    c2 = 1.f - powf(b2, step);
    m4 = reinterpret_cast<float4*>(state + CAFEQ_OPT_STATE_HEADER);
    v4 = reinterpret_cast<float4*>(state + CAFEQ_OPT_STATE_HEADER + n);
  }
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n4; i += (long long)gridDim.x * blockDim.x) {
    float4 gq = g4[i];
    float gi[4] = {gq.x, gq.y, gq.z, gq.w};
    if (orth_f != 0.f) {
      const float4 r = RM4[i];
      gi[0] = fmaf(orth_f, r.x, gi[0]); gi[1] = fmaf(orth_f, r.y, gi[1]);
      gi[2] = fmaf(orth_f, r.z, gi[2]); gi[3] = fmaf(orth_f, r.w, gi[3]);
    }
    const float4 mq = M4[i];
    float mv[4] = {mq.x, mq.y, mq.z, mq.w};
    if (!adam) {
#pragma unroll
      for (int j = 0; j < 4; ++j) mv[j] = mv[j] - lr * gi[j];
    } else {
      const float4 ma = m4[i], va = v4[i];
      float mm[4] = {ma.x, ma.y, ma.z, ma.w}, vv[4] = {va.x, va.y, va.z, va.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        mm[j] = b1 * mm[j] + (1.f - b1) * gi[j];
        vv[j] = b2 * vv[j] + (1.f - b2) * gi[j] * gi[j];
        mv[j] = mv[j] - lr * (mm[j] / c1) / (sqrtf(vv[j] / c2) + eps);
      }
      m4[i] = make_float4(mm[0], mm[1], mm[2], mm[3]);
      v4[i] = make_float4(vv[0], vv[1], vv[2], vv[3]);
    }
    M4[i] = make_float4(mv[0], mv[1], mv[2], mv[3]);
  }
}

// max |w| of a bf16 matrix (bit pattern of a non-negative float, atomic integer maximum)
__global__ void __launch_bounds__(256) absmax_bf16_kernel(const uint16_t* __restrict__ W, long long ld, int rows, int cols,
                                                          float* __restrict__ out) {
  float m = 0.f;
  const int cpr = cols / 8;
  const long long nch = (long long)rows * cpr;
  for (long long c = blockIdx.x * (long long)blockDim.x + threadIdx.x; c < nch; c += (long long)gridDim.x * blockDim.x) {
    const long long row = c / cpr;
    const int cc = (int)(c - row * cpr);
    const uint4 q = __ldg(reinterpret_cast<const uint4*>(W + row * ld) + cc);
    const uint32_t w4[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int h = 0; h < 4; ++h) {
      m = fmaxf(m, fabsf(__uint_as_float(w4[h] << 16)));
      m = fmaxf(m, fabsf(__uint_as_float(w4[h] & 0xFFFF0000u)));
    }
  }
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0 && m > 0.f && m < 3.0e38f) atomicMax(reinterpret_cast<int*>(out), __float_as_int(m));
}

// fp16 copy of a bf16 matrix, scaled by the power of two that brings max |w| just below 2^14:  out = fp16(w * 2^e),
// *inv_scale = 2^-e.  bf16 carries 8 significand bits, fp16 11, so every entry down to 2^-38 of the largest is copied
// exactly; smaller ones round to the fp16 subnormal grid (absolute error below 2^-39 of the largest entry).
__global__ void __launch_bounds__(256) bf16_to_scaled_f16_kernel(const uint16_t* __restrict__ W, long long ld, int rows, int cols,
                                                                 const float* __restrict__ wmax, uint16_t* __restrict__ out,
                                                                 float* __restrict__ inv_scale) {
  const float m = *wmax;
  int e = 0;
  if (m > 0.f) {
    int ex;
    frexpf(m, &ex);
    e = 14 - ex;
    if (e > 120) e = 120;
    if (e < -120) e = -120;
  }
  const float sc = exp2f((float)e);
  if (blockIdx.x == 0 && threadIdx.x == 0) *inv_scale = exp2f((float)-e);
  const int cpr = cols / 8;
  const long long nch = (long long)rows * cpr;
  for (long long c = blockIdx.x * (long long)blockDim.x + threadIdx.x; c < nch; c += (long long)gridDim.x * blockDim.x) {
    const long long row = c / cpr;
    const int cc = (int)(c - row * cpr);
    const uint4 q = __ldg(reinterpret_cast<const uint4*>(W + row * ld) + cc);
    const uint32_t w4[4] = {q.x, q.y, q.z, q.w};
    uint32_t o4[4];
#pragma unroll
    for (int h = 0; h < 4; ++h) {
      const float lo = __uint_as_float(w4[h] << 16) * sc, hi = __uint_as_float(w4[h] & 0xFFFF0000u) * sc;
      o4[h] = (uint32_t)__half_as_ushort(__float2half_rn(lo)) | ((uint32_t)__half_as_ushort(__float2half_rn(hi)) << 16);
    }
    reinterpret_cast<uint4*>(out + row * (long long)cols)[cc] = make_uint4(o4[0], o4[1], o4[2], o4[3]);
  }
}

__global__ void set_f32_kernel(float* p, float v) { *p = v; }

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
struct LyMat {
  Geo G;
  const void* W;
  int prob, side;            // owning problem, 0 / 1 = first / second matrix of it
  int bits;
  float *a, *usel, *coef;    // per (row, group) records, group-major
  int* idx;
  float *cw, *agrp, *A;      // Eq. 4 weights and sums (cleared every step)
  float* vmax;               // maximum coefficient / group maximum of the step (cleared every step)
  float *wmax, *winv;        // fp16 copy: max |w| and 2^-e (set by the prepare call)
  uint16_t* W16;
};

struct LyProb {
  int pair;
  int m0, m1;                // matrix indices (m1 = -1 for a single)
  float *M, *state, *hist;
  cafeq_opt_cfg cfg;
  float kappa;
  int blk0, nb;
  double* acc;               // [8] cleared every step
  float* amax;
};

struct LyPlan {
  int n, nm, k, g;
  int NB, pair_blk0;
  LyProb p[LY_MAX_PROBS];
  LyMat m[LY_MAX_MATS];
  // workspace
  float *Minv, *Mc, *gMinv, *grad, *RM, *Mf, *c;
  KkWS kk;
  double* orth_sq;
  float* one;
  char* zone;
  size_t zone_bytes;
  size_t ws_used;
};

// Validates the problems, orders them (singles first, pairs last) and carves the workspace.  The layout depends only
// on the descriptors, so a prepare call and later optimise calls on the same problems see the same buffers.
static int ly_plan(const cafeq_layer_problem* probs, int n, void* ws, size_t ws_bytes, LyPlan* L) {
  if (!probs || n < 1 || n > LY_MAX_PROBS) return CAFEQ_ERR_INVALID_ARG;
  memset((void*)L, 0, sizeof(*L));
  L->n = n;
  int order[LY_MAX_PROBS], no = 0;
  for (int pass = 0; pass < 2; ++pass)
    for (int i = 0; i < n; ++i) {
      if (probs[i].struct_size != sizeof(cafeq_layer_problem)) return CAFEQ_ERR_INVALID_ARG;
      if ((probs[i].pair != 0) == (pass == 1)) order[no++] = i;
    }
  int nm = 0, NB = 0;
  L->pair_blk0 = -1;
  for (int q = 0; q < n; ++q) {
    const cafeq_layer_problem& in = probs[order[q]];
    LyProb& P = L->p[q];
    P.pair = in.pair != 0;
    P.M = in.M;
    P.state = in.opt_state;
    P.hist = in.loss_history;
    P.cfg = in.cfg;
    if (!in.W1 || !in.M || !in.loss_history || in.cfg.struct_size != sizeof(cafeq_opt_cfg)) return CAFEQ_ERR_INVALID_ARG;
    if (in.cfg.optimizer != CAFEQ_OPT_GD && in.cfg.optimizer != CAFEQ_OPT_ADAM) return CAFEQ_ERR_INVALID_ARG;
    if (in.cfg.optimizer == CAFEQ_OPT_ADAM && !in.opt_state) return CAFEQ_ERR_INVALID_ARG;
    if (((uintptr_t)in.M & 15) || ((uintptr_t)in.opt_state & 15)) return CAFEQ_ERR_UNSUPPORTED;
    if (in.cfg.eval_every != 0) return CAFEQ_ERR_UNSUPPORTED;  // the quantised losses are evaluated by the per-problem calls
    Geo G1, G2;
    int rc;
    if (P.pair) {
      if (!in.W2 || in.cfg.loss_kind != CAFEQ_LOSS_LSE || !(in.cfg.lse_t > 0.f)) return CAFEQ_ERR_INVALID_ARG;
      if ((rc = make_pair_geo(&in.d1, &in.d2, &G1, &G2))) return rc;
      if (P.pair && L->pair_blk0 < 0) L->pair_blk0 = NB;
    } else {
      if (in.cfg.loss_kind != CAFEQ_LOSS_SURROGATE) return CAFEQ_ERR_UNSUPPORTED;
      if ((rc = make_geo(&in.d1, &G1, true))) return rc;
    }
    P.kappa = in.cfg.kappa > 0.f ? in.cfg.kappa : 1.f / (float)(((1 << in.d1.bits) - 1) * ((1 << in.d1.bits) - 1));
    if (q == 0) {
      L->k = G1.k;
      L->g = G1.g;
    }
    P.blk0 = NB;
    P.nb = G1.nbT;
    NB += P.nb;
    P.m0 = nm;
    P.m1 = -1;
    for (int side = 0; side < (P.pair ? 2 : 1); ++side) {
      if (nm >= LY_MAX_MATS) return CAFEQ_ERR_UNSUPPORTED;
      LyMat& Mt = L->m[nm];
      Mt.G = side ? G2 : G1;
      Mt.W = side ? in.W2 : in.W1;
      Mt.prob = q;
      Mt.side = side;
      Mt.bits = side ? in.d2.bits : in.d1.bits;
      // every matrix goes through the tensor-core pass and the tensor-core backward with one block and group size
      if (Mt.G.k != L->k || Mt.G.g != L->g || !(L->k == 128 || L->k == 256)) return CAFEQ_ERR_UNSUPPORTED;
      const int form = Mt.G.axis == CAFEQ_AXIS_IN ? BD_IN : BD_OUT;
      if (!bd_supported(form, Mt.G.d_out, Mt.G.d_in, Mt.G.ld, Mt.G.k, Mt.G.g, Mt.W)) return CAFEQ_ERR_UNSUPPORTED;
      if (!bw_supported(Mt.G.axis == CAFEQ_AXIS_IN, Mt.G.d_out, Mt.G.d_in, Mt.G.ld, Mt.G.k, Mt.G.g, Mt.W)) return CAFEQ_ERR_UNSUPPORTED;
      if (Mt.G.d_in % 8) return CAFEQ_ERR_UNSUPPORTED;
      if (side) P.m1 = nm;
      ++nm;
    }
  }
  if (L->pair_blk0 < 0) L->pair_blk0 = NB;
  L->nm = nm;
  L->NB = NB;

  Bump b(ws, ws ? ws_bytes : 0);
  if (!ws) b.cap = 0;
  const size_t kk = (size_t)NB * L->k * L->k;
  const size_t kkP = (size_t)(NB - L->pair_blk0) * L->k * L->k;
  L->Minv = b.take<float>(kk);
  L->Mc = b.take<float>(kk);
  L->gMinv = b.take<float>(kk);
  L->grad = b.take<float>(kk);
  L->RM = b.take<float>(kkP ? kkP : 1);
  L->Mf = b.take<float>(kkP ? kkP : 1);
  L->c = b.take<float>((size_t)NB * L->k);
  carve_kk(b, NB, L->k, &L->kk);
  L->one = b.take<float>(64);
  L->kk.redo_total = reinterpret_cast<int*>(L->one ? L->one + 8 : nullptr);
  for (int i = 0; i < nm; ++i) {
    LyMat& Mt = L->m[i];
    const size_t rows_ng = (size_t)Mt.G.d_out * Mt.G.ng;
    Mt.a = b.take<float>(rows_ng);
    Mt.usel = b.take<float>(rows_ng);
    Mt.coef = b.take<float>(rows_ng);
    Mt.idx = b.take<int>(rows_ng);
    Mt.W16 = b.take<uint16_t>((size_t)Mt.G.n);
    Mt.wmax = b.take<float>(64);
    Mt.winv = Mt.wmax ? Mt.wmax + 1 : nullptr;
  }
  // everything that is cleared at the start of every step, contiguous
  const size_t zone0 = b.used;
  for (int i = 0; i < nm; ++i) {
    LyMat& Mt = L->m[i];
    Mt.cw = b.take<float>((size_t)(Mt.G.ng > Mt.G.d_out ? Mt.G.ng : Mt.G.d_out));
    Mt.agrp = b.take<float>((size_t)Mt.G.ng);
    Mt.A = b.take<float>((size_t)Mt.G.nbT * Mt.G.k);
    Mt.vmax = b.take<float>(64);
  }
  for (int q = 0; q < n; ++q) {
    L->p[q].acc = b.take<double>(8);
    L->p[q].amax = b.take<float>(64);
  }
  L->orth_sq = b.take<double>((size_t)(NB - L->pair_blk0) + 1);
  L->zone = ws ? (char*)ws + zone0 : nullptr;
  L->zone_bytes = b.used - zone0;
  L->ws_used = b.used;
  if (ws && b.overflow) return CAFEQ_ERR_WORKSPACE;
  return CAFEQ_OK;
}

// Side stream of the layer step with its fork / join events, one set per host thread and device (two threads that
// enqueue steps on the same device must not share the events), created on first use.
struct LyAux {
  cudaStream_t stream;
  cudaEvent_t fork, join;
};
static LyAux* ly_aux() {
  static thread_local LyAux slots[64];
  static thread_local bool made[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  if (!made[dev]) {
    LyAux a;
    if (cudaStreamCreateWithFlags(&a.stream, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&a.fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&a.join, cudaEventDisableTiming) != cudaSuccess)
      return nullptr;
    slots[dev] = a;
    made[dev] = true;
  }
  return &slots[dev];
}
// block sizes whose inverse refinement runs on row-major arrays (the transposed split arrays are then free)
static bool w_mn_expected(int k) { return g_tb_enable.load(std::memory_order_relaxed) && tb_supported(k, 2); }

static void ly_lists(const LyPlan& L, int axis, int transpose, int* out, int* cnt) {
  // matrices whose backward shares (axis, output orientation): singles store gradT plainly, a pair's first factor
  // (operator M^T) stores it transposed, its second factor feeds dL/dMinv plainly
  *cnt = 0;
  for (int i = 0; i < L.nm; ++i) {
    const LyMat& Mt = L.m[i];
    const int tr = (L.p[Mt.prob].pair && Mt.side == 0) ? 1 : 0;
    if (Mt.G.axis == axis && tr == transpose) out[(*cnt)++] = i;
  }
}

// One optimisation step of every problem.  hist_row: which row of each loss history this step writes.
static int ly_step(cudaStream_t st, LyPlan& L, int hist_row, int32_t* status) {
  const int k = L.k, NB = L.NB;
  const long long kk1 = (long long)k * k, kk = (long long)NB * kk1;
  const int nbP = NB - L.pair_blk0;
  const long long offP = (long long)L.pair_blk0 * kk1;
  KkWS& w = L.kk;
  {
    LyPrepArgs a;
    memset(&a, 0, sizeof(a));
    a.n = L.n; a.k = k;
    for (int q = 0; q < L.n; ++q) {
      a.blk0[q] = L.p[q].blk0;
      a.M[q] = L.p[q].M;
      a.step_counter[q] = L.p[q].state;
    }
    a.blk0[L.n] = NB;
    a.pair_blk0 = L.pair_blk0;
    a.Mc = L.Mc; a.Ab = w.Ab; a.Mf = L.Mf; a.grad = L.grad; a.gMinv = L.gMinv;
    a.zone = reinterpret_cast<uint4*>(L.zone); a.zone_n16 = (long long)(L.zone_bytes / 16);
    a.rn = w.rn; a.rn_n = NS_MAX_ITERS * NB; a.flag = w.flag;
    a.status = status;
    CQ_LAUNCH(layer_prep_kernel, grid_for(kk / 4), 256, 0, st, a);
  }
  bool any_lambda = false;
  for (int q = 0; q < L.n; ++q) any_lambda |= (L.p[q].pair && L.p[q].cfg.lambda_orth != 0.f);
  // The pair blocks' penalty chain (splits of the parameters, R = M M^T - I, R M) does not depend on the inverse:
  // it runs on a side stream beside the Newton-Schulz chain (both are chains of short, latency-bound launches that
  // leave SMs idle) and joins before the transform pass, which reads bf16(M)^T.  Event record / wait pairs only, so
  // the fork and the join are captured with the step when the caller's stream is being captured.
  LyAux* aux = (nbP > 0 && g_ly_dual.load(std::memory_order_relaxed) && w_mn_expected(k)) ? ly_aux() : nullptr;
  cudaStream_t so = st;
  if (aux) {
    if (cudaEventRecord(aux->fork, st) != cudaSuccess || cudaStreamWaitEvent(aux->stream, aux->fork, 0) != cudaSuccess) return CAFEQ_ERR_CUDA;
    so = aux->stream;
  }
  if (nbP > 0) {
    // pair blocks: splits of the fp32 parameters (the transposed high halves are bf16(M)^T, the operator of the
    // first factors' pass), R = M M^T - I with ||R_b||_F^2 per block, and R M for the penalty's gradient.
    // On the side stream R's splits live in the transposed-split arrays, which the row-major refinement leaves unused
    // (the Newton-Schulz chain writes its own residual into RTh meanwhile).
    uint16_t* Rh = (aux ? w.XTh[0] : w.RTh) + offP;
    uint16_t* Rl = (aux ? w.XTl[0] : w.RTl) + offP;
    launch_split(so, L.Mf, k, (long long)nbP * kk1, w.Ph + offP, w.Pl + offP, w.Qh + offP, w.Ql + offP, nullptr, status);
    const uint16_t* a1[3] = {w.Ph + offP, w.Pl + offP, w.Ph + offP};
    const uint16_t* b1[3] = {w.Ph + offP, w.Ph + offP, w.Pl + offP};
    launch_kk_tc(so, 3, a1, b1, nbP, k, 1.f, 0.f, -1.f, nullptr, nullptr, Rh, Rl, nullptr, nullptr, L.orth_sq, nullptr, status, 1);
    if (any_lambda) {
      const uint16_t* a2[3] = {Rh, Rl, Rh};
      const uint16_t* b2[3] = {w.Qh + offP, w.Qh + offP, w.Ql + offP};
      launch_kk_tc(so, 3, a2, b2, nbP, k, 1.f, 0.f, 0.f, nullptr, L.RM, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, status);
    }
  }
  if (aux && cudaEventRecord(aux->join, aux->stream) != cudaSuccess) return CAFEQ_ERR_CUDA;
  ns_inverse(st, L.Mc, L.Minv, nullptr, NB, k, true, w, status, true, true);
  if (aux && cudaStreamWaitEvent(st, aux->join, 0) != cudaSuccess) return CAFEQ_ERR_CUDA;
  // Eq. 4 weights of the single matrices (they own the first pair_blk0 blocks)
  if (L.pair_blk0 > 0) {
    LyColArgs ca;
    memset(&ca, 0, sizeof(ca));
    ca.k = k;
    int ns = 0;
    for (int q = 0; q < L.n; ++q) {
      const LyProb& P = L.p[q];
      if (P.pair) continue;
      const Geo& G = L.m[P.m0].G;
      ca.blk0[ns] = P.blk0;
      ca.cw[ns] = (G.axis == CAFEQ_AXIS_IN && G.r == 1) ? L.m[P.m0].cw : nullptr;
      ca.g[ns] = G.g;
      ++ns;
    }
    ca.blk0[ns] = L.pair_blk0;
    ca.n = ns;
    CQ_LAUNCH(layer_colnorm_kernel, dim3(k / 32, L.pair_blk0), dim3(32, 8), 0, st, L.Minv, L.c, ca);
    for (int q = 0; q < L.n; ++q) {
      const LyProb& P = L.p[q];
      if (P.pair) continue;
      const LyMat& Mt = L.m[P.m0];
      const Geo& G = Mt.G;
      if (G.axis == CAFEQ_AXIS_IN && G.r == 1) continue;
      if (G.axis == CAFEQ_AXIS_IN) CQ_LAUNCH(cw_in_kernel, (G.ng + 127) / 128, 128, 0, st, L.c + (size_t)P.blk0 * k, G.d_in, G.g, k, G.r, Mt.cw);
      else CQ_LAUNCH(cw_out_kernel, (G.d_out + 127) / 128, 128, 0, st, L.c + (size_t)P.blk0 * k, G.d_out, G.g, k, G.r, Mt.cw);
    }
  }
  // transform passes: all matrices of a form in one launch, and both forms in the same launch when each has
  // enough tiles for its share of the CTAs
  {
    BdSub subs[2][LY_MAX_MATS];
    int ns[2] = {0, 0};
    long long ntile[2] = {0, 0};
    for (int i = 0; i < L.nm; ++i) {
      const LyMat& Mt = L.m[i];
      const int form = (Mt.G.axis == CAFEQ_AXIS_IN) ? BD_IN : BD_OUT;
      const LyProb& P = L.p[Mt.prob];
      const long long off = (long long)P.blk0 * kk1;
      BdSub& s = subs[form][ns[form]++];
      memset(&s, 0, sizeof(s));
      s.X = Mt.W; s.ld = Mt.G.ld; s.nbT = P.nb;
      BdParams& p = s.p;
      p.d_out = Mt.G.d_out; p.d_in = Mt.G.d_in; p.r = Mt.G.r;
      p.qmax = qmax_of(Mt.bits);
      p.a = Mt.a; p.usel = Mt.usel; p.idx = Mt.idx;
      p.vmax = Mt.vmax;
      p.status = status;
      if (!P.pair) {
        s.Tb = w.Ab + off;  // the parameter itself on its axis
        p.epi = EPI_ABSMAX | EPI_SURR;
        p.cw = Mt.cw; p.kappa = P.kappa; p.coef = Mt.coef; p.lossacc = P.acc;
        p.Aacc = (Mt.G.axis == CAFEQ_AXIS_IN) ? Mt.agrp : Mt.A;
      } else {
        s.Tb = (Mt.side == 0) ? w.Qh + off : w.Xh[w.cur] + off;  // bf16(M)^T for U = W1 M, bf16(M^-1) for V = M^-1 W2
        p.epi = EPI_ABSMAX;
      }
      ntile[form] += (long long)Mt.G.n / 32768;  // tiles hold 32768 entries in both forms
    }
    const bool dual = g_ly_dual.load(std::memory_order_relaxed) && ns[0] >= 1 && ns[1] >= 1 && ns[0] <= BD_MAX_SUB &&
                      ns[1] <= BD_MAX_SUB && bd_dual_ok(k, L.g) && ntile[0] >= 148 && ntile[1] >= 148;
    if (dual) {
      int ti = kt_begin(5, st);
      g_launches.fetch_add(1, std::memory_order_relaxed);
      int rc = bd_launch_dual(st, k, L.g, subs[0], ns[0], subs[1], ns[1]);
      kt_end(ti, st);
      if (rc) return rc;
    } else {
      for (int form = 0; form < 2; ++form)
        for (int c0 = 0; c0 < ns[form]; c0 += BD_MAX_SUB) {
          const int n = (ns[form] - c0 < BD_MAX_SUB) ? ns[form] - c0 : BD_MAX_SUB;
          int ti = kt_begin(5, st);
          g_launches.fetch_add(1, std::memory_order_relaxed);
          int rc = bd_launch_many(st, form, k, L.g, subs[form] + c0, n);
          kt_end(ti, st);
          if (rc) return rc;
        }
    }
  }
  // LogSumExp of the pairs
  {
    LyLseArgs g;
    memset(&g, 0, sizeof(g));
    int np = 0;
    long long nmax = 0;
    for (int q = 0; q < L.n; ++q) {
      const LyProb& P = L.p[q];
      if (!P.pair) continue;
      for (int s = 0; s < 2; ++s) {
        const LyMat& Mt = L.m[s ? P.m1 : P.m0];
        g.a[np][s] = Mt.a; g.u[np][s] = Mt.usel; g.c[np][s] = Mt.coef;
        g.n[np][s] = (long long)Mt.G.d_out * Mt.G.ng;
        g.vmax[np][s] = Mt.vmax;
      }
      g.t[np] = P.cfg.lse_t; g.Z[np] = P.acc; g.amax[np] = P.amax;
      if (g.n[np][0] + g.n[np][1] > nmax) nmax = g.n[np][0] + g.n[np][1];
      ++np;
    }
    g.status = status;
    if (np) CQ_LAUNCH(layer_lse_kernel, dim3(grid_for(nmax, 256, 148 * 4), np), 256, 0, st, g);
  }
  // sparse backward, fp16 single-term form: all matrices of one (axis, orientation) in one launch; when the layer has
  // exactly one input-axis and one output-axis group, both in the same launch
  {
    BwSub subs[4][LY_MAX_MATS];
    int cnt[4] = {0, 0, 0, 0};
    long long ntile[4] = {0, 0, 0, 0};
    for (int axis = 0; axis < 2; ++axis)
      for (int tr = 0; tr < 2; ++tr) {
        const int c = axis * 2 + tr;
        int list[LY_MAX_MATS];
        ly_lists(L, axis, tr, list, &cnt[c]);
        for (int j = 0; j < cnt[c]; ++j) {
          const LyMat& Mt = L.m[list[j]];
          const LyProb& P = L.p[Mt.prob];
          const long long off = (long long)P.blk0 * kk1;
          BwSub& s = subs[c][j];
          memset(&s, 0, sizeof(s));
          s.W16 = Mt.W16; s.ld = Mt.G.d_in;
          BwParams& p = s.p;
          p.d_out = Mt.G.d_out; p.d_in = Mt.G.d_in; p.g = Mt.G.g; p.ng = Mt.G.ng; p.r = Mt.G.r;
          p.gm = 1;
          p.coef = Mt.coef; p.idx = Mt.idx;
          p.w_inv_scale = Mt.winv;
          p.status = status;
          if (!P.pair) {
            p.gradT = L.grad + off;
            p.coefmax = Mt.vmax;
          } else {
            p.gradT = (Mt.side == 0 ? L.grad : L.gMinv) + off;
            p.coefmax = L.one;   // the largest exp(t (a - max)) is 1
            p.out_div = P.acc;   // Z
          }
          ntile[c] += (long long)Mt.G.n / (64 * k);
        }
      }
    const int c_in0 = CAFEQ_AXIS_IN * 2, c_out0 = CAFEQ_AXIS_OUT * 2;
    int ci = -1, co = -1;
    bool dual = g_ly_dual.load(std::memory_order_relaxed) && bw_dual_ok(k);
    if (cnt[c_in0] && cnt[c_in0 + 1]) dual = false;
    if (cnt[c_out0] && cnt[c_out0 + 1]) dual = false;
    ci = cnt[c_in0] ? c_in0 : c_in0 + 1;
    co = cnt[c_out0] ? c_out0 : c_out0 + 1;
    if (!cnt[ci] || !cnt[co] || cnt[ci] > BW_MAX_SUB || cnt[co] > BW_MAX_SUB || ntile[ci] < 148 * 6 || ntile[co] < 148 * 6) dual = false;
    if (dual) {
      int ti = kt_begin(2, st);
      g_launches.fetch_add(1, std::memory_order_relaxed);
      int rc = bw_launch_dual(st, k, ci & 1, subs[ci], cnt[ci], co & 1, subs[co], cnt[co]);
      kt_end(ti, st);
      if (rc) return rc;
    } else {
      for (int c = 0; c < 4; ++c)
        for (int c0 = 0; c0 < cnt[c]; c0 += BW_MAX_SUB) {
          const int ns = (cnt[c] - c0 < BW_MAX_SUB) ? cnt[c] - c0 : BW_MAX_SUB;
          int ti = kt_begin(2, st);
          g_launches.fetch_add(1, std::memory_order_relaxed);
          int rc = bw_launch_many(st, (c >> 1) == CAFEQ_AXIS_IN, k, c & 1, 1, subs[c] + c0, ns);
          kt_end(ti, st);
          if (rc) return rc;
        }
    }
  }
  // dL/dMinv of Eq. 4 for the singles, then grad -= Minv^T (dL/dMinv) Minv^T over all blocks
  if (L.pair_blk0 > 0) {
    LyGminvArgs ga;
    memset(&ga, 0, sizeof(ga));
    ga.k = k;
    int ns = 0;
    for (int q = 0; q < L.n; ++q) {
      const LyProb& P = L.p[q];
      if (P.pair) continue;
      const LyMat& Mt = L.m[P.m0];
      const Geo& G = Mt.G;
      const bool in_r1 = (G.axis == CAFEQ_AXIS_IN && G.r == 1);
      if (G.axis == CAFEQ_AXIS_IN && !in_r1) CQ_LAUNCH(expand_agrp_kernel, (G.d_in + 127) / 128, 128, 0, st, Mt.agrp, G.d_in, G.g, k, G.r, Mt.A);
      ga.blk0[ns] = P.blk0;
      ga.A[ns] = Mt.A;
      ga.Agrp[ns] = in_r1 ? Mt.agrp : nullptr;
      ga.g[ns] = G.g;
      ga.scale[ns] = 2.f * P.kappa;
      ++ns;
    }
    ga.blk0[ns] = L.pair_blk0;
    ga.n = ns;
    CQ_LAUNCH(layer_gminv_kernel, grid_for((long long)L.pair_blk0 * kk1 / 4), 256, 0, st, L.Minv, L.gMinv, ga);
  }
  minv_path_tc(st, L.gMinv, L.grad, NB, k, true, w, status);
  {
    LyFinishArgs f;
    memset(&f, 0, sizeof(f));
    f.k = k;
    long long nmax = 0;
    for (int q = 0; q < L.n; ++q) {
      const LyProb& P = L.p[q];
      f.blk0[q] = P.blk0;
      f.M[q] = P.M; f.state[q] = P.state;
      f.hist[q] = P.hist + 2 * (size_t)hist_row;
      f.pair[q] = P.pair; f.optimizer[q] = P.cfg.optimizer;
      f.lr[q] = P.cfg.lr; f.b1[q] = P.cfg.beta1; f.b2[q] = P.cfg.beta2; f.eps[q] = P.cfg.eps;
      f.lambda[q] = P.cfg.lambda_orth; f.t[q] = P.cfg.lse_t;
      f.sqrt_h[q] = sqrtf((float)L.m[P.m0].G.d_out);
      f.acc[q] = P.acc; f.amax[q] = P.amax;
      if ((long long)P.nb * kk1 > nmax) nmax = (long long)P.nb * kk1;
    }
    f.blk0[L.n] = NB;
    f.orth_sq = L.orth_sq; f.pair_blk0 = L.pair_blk0;
    f.grad = L.grad; f.RM = L.RM;
    f.status = status;
    CQ_LAUNCH(layer_finish_kernel, dim3(grid_for(nmax / 4, 256, 148 * 4), L.n), 256, 0, st, f);
  }
  return CAFEQ_OK;
}

}  // namespace cafeq

extern "C" int cafeq_layer_workspace_size(const cafeq_layer_problem* probs, int n, size_t* bytes) {
  if (!bytes) return CAFEQ_ERR_INVALID_ARG;
  LyPlan L;
  int rc = ly_plan(probs, n, nullptr, 0, &L);
  if (rc) return rc;
  *bytes = L.ws_used + 256;
  return CAFEQ_OK;
}

extern "C" int cafeq_layer_prepare(const cafeq_layer_problem* probs, int n, int32_t* status, void* ws, size_t ws_bytes,
                                   void* stream) {
  int rc;
  if ((rc = check_ws(ws, ws_bytes))) return rc;
  LyPlan L;
  if ((rc = ly_plan(probs, n, ws, ws_bytes, &L))) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  for (int i = 0; i < L.nm; ++i) {
    LyMat& Mt = L.m[i];
    CQ_LAUNCH(fill_f32_kernel, 1, 32, 0, st, Mt.wmax, 0.f, 2);
    CQ_LAUNCH(absmax_bf16_kernel, grid_for(Mt.G.n / 8), 256, 0, st, (const uint16_t*)Mt.W, Mt.G.ld, Mt.G.d_out, Mt.G.d_in, Mt.wmax);
    CQ_LAUNCH(bf16_to_scaled_f16_kernel, grid_for(Mt.G.n / 8), 256, 0, st, (const uint16_t*)Mt.W, Mt.G.ld, Mt.G.d_out, Mt.G.d_in, Mt.wmax,
              Mt.W16, Mt.winv);
  }
  CQ_LAUNCH(fill_f32_kernel, 1, 32, 0, st, L.one, 0.f, 16);  // (also clears the running count of elimination fall-backs)
  CQ_LAUNCH(set_f32_kernel, 1, 1, 0, st, L.one, 1.f);
  // inverse of the initial transforms from scratch; every step afterwards refines the previous step's inverse
  const long long kk = (long long)L.NB * L.k * L.k;
  {
    LyPrepArgs a;
    memset(&a, 0, sizeof(a));
    a.n = L.n; a.k = L.k;
    for (int q = 0; q < L.n; ++q) {
      a.blk0[q] = L.p[q].blk0;
      a.M[q] = L.p[q].M;
    }
    a.blk0[L.n] = L.NB;
    a.pair_blk0 = L.pair_blk0;
    a.Mc = L.Mc; a.Ab = L.kk.Ab; a.Mf = L.Mf; a.grad = L.grad; a.gMinv = L.gMinv;
    a.zone = reinterpret_cast<uint4*>(L.zone); a.zone_n16 = (long long)(L.zone_bytes / 16);
    a.rn = L.kk.rn; a.rn_n = NS_MAX_ITERS * L.NB; a.flag = L.kk.flag;
    a.status = status;
    CQ_LAUNCH(layer_prep_kernel, grid_for(kk / 4), 256, 0, st, a);
  }
  ns_inverse(st, L.Mc, L.Minv, nullptr, L.NB, L.k, false, L.kk, status, true);
  return last_launch();
}

extern "C" int cafeq_optimize_layer(const cafeq_layer_problem* probs, int n, int steps, int32_t* status, void* ws,
                                    size_t ws_bytes, void* stream) {
  int rc;
  if (steps < 0) return CAFEQ_ERR_INVALID_ARG;
  if ((rc = check_ws(ws, ws_bytes))) return rc;
  LyPlan L;
  if ((rc = ly_plan(probs, n, ws, ws_bytes, &L))) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  for (int it = 0; it < steps; ++it)
    if ((rc = ly_step(st, L, it, status))) return rc;
  return last_launch();
}

extern "C" int cafeq_debug_set_layer_launch(int dual, int pass_out_pct, int bwd_out_pct) {
  if ((dual != 0 && dual != 1) || pass_out_pct > 1000 || bwd_out_pct > 1000) return CAFEQ_ERR_INVALID_ARG;
  g_ly_dual.store(dual, std::memory_order_relaxed);
  if (pass_out_pct > 0) g_dual_pass_pct.store(pass_out_pct, std::memory_order_relaxed);
  if (bwd_out_pct > 0) g_dual_bwd_pct.store(bwd_out_pct, std::memory_order_relaxed);
  return CAFEQ_OK;
}

extern "C" int cafeq_layer_debug_fallbacks(const cafeq_layer_problem* probs, int n, void* ws, size_t ws_bytes, int* count) {
  if (!count) return CAFEQ_ERR_INVALID_ARG;
  int rc;
  if ((rc = check_ws(ws, ws_bytes))) return rc;
  LyPlan L;
  if ((rc = ly_plan(probs, n, ws, ws_bytes, &L))) return rc;
  return cudaMemcpy(count, L.kk.redo_total, sizeof(int), cudaMemcpyDeviceToHost) == cudaSuccess ? CAFEQ_OK : CAFEQ_ERR_CUDA;
}
