// Shape-agnostic CUDA kernels of the CafeQ path: a strided batched GEMM with fp32 accumulation and the
// element-wise / reduction steps around it.  They cover every shape (tiny test matrices, odd block
// sizes) and serve as the on-device cross-check of the fused tensor-core kernels.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "cafeq.h"

namespace cafeq {

// ------------------------------------------------------------------------------------------------
// small helpers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) { return __uint_as_float(((uint32_t)b) << 16); }

__device__ __forceinline__ float round_to_bf16(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

__device__ __forceinline__ void raise_status(int32_t* status, int code) {
  if (status) atomicCAS(status, 0, code);
}

__device__ __forceinline__ double block_sum_double(double v, double* sh) {
  // sh: at least 32 doubles of shared memory
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) sh[w] = v;
  __syncthreads();
  int nw = (blockDim.x + 31) >> 5;
  v = (threadIdx.x < nw) ? sh[threadIdx.x] : 0.0;
  if (w == 0)
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;  // valid in thread 0
}

// ------------------------------------------------------------------------------------------------
// fill / copy / round
// ------------------------------------------------------------------------------------------------
__global__ void fill_f32_kernel(float* p, float v, long long n) {
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
    p[i] = v;
}

__global__ void zero_f64_kernel(double* p, int n) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = 0.0;
}

// out = float(bf16(in)): the operand actually fed to the transform products.
__global__ void round_bf16_kernel(const float* __restrict__ in, float* __restrict__ out, long long n,
                                  const int32_t* status) {
  if (status && *status) return;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
    out[i] = round_to_bf16(in[i]);
}

__global__ void copy_f32_kernel(const float* __restrict__ in, float* __restrict__ out, long long n) {
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
    out[i] = in[i];
}

// ------------------------------------------------------------------------------------------------
// strided batched GEMM:  C[b][m][n] (op)= alpha * sum_k A[b/divA][m][k] * B[b/divB][k][n]
// ------------------------------------------------------------------------------------------------
enum { GEMM_STORE = 1, GEMM_ACCUM = 2, GEMM_ATOMIC = 4, GEMM_SUBP = 8, GEMM_SQSUM = 16 };

struct GemmArgs {
  const void* A;
  const void* B;
  float* C;
  const float* P;  // optional matrix subtracted before the square sum / store
  double* sq;      // optional accumulator of sum(v^2)
  int M, N, K, batch;
  long long sAm, sAk, sAb;
  long long sBk, sBn, sBb;
  long long sCm, sCn, sCb;
  long long sPm, sPn, sPb;
  int a_bf16, b_bf16;
  int divA, divB, divC;
  float alpha;
  int mode;
  const int32_t* status;
};

template <bool ABF, bool BBF>
__global__ void __launch_bounds__(256) gemm_kernel(GemmArgs g) {
  if (g.status && *g.status) return;
  constexpr int BM = 64, BN = 64, BK = 16;
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];
  __shared__ double red[32];
  const int tid = threadIdx.x;
  const int b = blockIdx.z;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  const long long ab = (long long)(b / g.divA) * g.sAb, bb = (long long)(b / g.divB) * g.sBb;
  const bool a_kfast = (g.sAk == 1), b_nfast = (g.sBn == 1);
  const int ty = tid >> 4, tx = tid & 15;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (int k0 = 0; k0 < g.K; k0 += BK) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      int t = tid + q * 256;
      int m, kk;
      if (a_kfast) { kk = t & 15; m = t >> 4; } else { m = t & 63; kk = t >> 6; }
      int gm = m0 + m, gk = k0 + kk;
      float v = 0.f;
      if (gm < g.M && gk < g.K) {
        long long off = ab + gm * g.sAm + gk * g.sAk;
        v = ABF ? bf16_bits_to_float(((const uint16_t*)g.A)[off]) : ((const float*)g.A)[off];
      }
      As[kk][m] = v;
      int n;
      if (b_nfast) { n = t & 63; kk = t >> 6; } else { kk = t & 15; n = t >> 4; }
      int gn = n0 + n;
      gk = k0 + kk;
      v = 0.f;
      if (gn < g.N && gk < g.K) {
        long long off = bb + gk * g.sBk + gn * g.sBn;
        v = BBF ? bf16_bits_to_float(((const uint16_t*)g.B)[off]) : ((const float*)g.B)[off];
      }
      Bs[kk][n] = v;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[4], bv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) bv[j] = Bs[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }

  double local = 0.0;
  const long long cb = (long long)(b / g.divC) * g.sCb;
  const long long pb = (long long)b * g.sPb;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int gm = m0 + ty * 4 + i;
    if (gm >= g.M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int gn = n0 + tx * 4 + j;
      if (gn >= g.N) continue;
      float v = g.alpha * acc[i][j];
      if (g.mode & GEMM_SUBP) v -= g.P[pb + gm * g.sPm + gn * g.sPn];
      if (g.mode & GEMM_SQSUM) local += (double)v * (double)v;
      if (g.mode & GEMM_STORE) {
        float* c = g.C + cb + gm * g.sCm + gn * g.sCn;
        if (g.mode & GEMM_ATOMIC) atomicAdd(c, v);
        else if (g.mode & GEMM_ACCUM) *c += v;
        else *c = v;
      }
    }
  }
  if (g.mode & GEMM_SQSUM) {
    double s = block_sum_double(local, red);
    if (tid == 0) atomicAdd(g.sq, s);
  }
}

// ------------------------------------------------------------------------------------------------
// block inverse: Gauss-Jordan with partial pivoting, one CTA per k x k block, matrix kept in the output
// buffer (global memory, L2 resident).  Also emits the column square norms c[t] = sum_i Minv[i][t]^2.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024) block_inverse_kernel(const float* __restrict__ Min, float* __restrict__ Out,
                                                             float* __restrict__ cnorm, int k, int32_t* status,
                                                             const double* __restrict__ rn_check, double tol2, int* redo_flag,
                                                             int* redo_count = nullptr) {
  // rn_check: squared residual of an iterative inverse per block; the elimination only runs for blocks whose
  // residual is above tol2 (or not finite) and then raises redo_flag for whoever depends on the result
  if (status && *status) return;
  if (rn_check) {
    if (rn_check[blockIdx.x] <= tol2) return;
    if (threadIdx.x == 0 && redo_flag) *redo_flag = 1;
    if (threadIdx.x == 0 && redo_count) atomicAdd(redo_count, 1);  // blocks recomputed by elimination, over the run
  }
  extern __shared__ float sm[];  // prow[k], fcol[k], piv (int) [k], red
  float* prow = sm;
  float* fcol = sm + k;
  int* piv = (int*)(sm + 2 * k);
  __shared__ float rv[32];
  __shared__ int ri[32];
  __shared__ int s_r;
  __shared__ int s_bad;
  const int tid = threadIdx.x, nt = blockDim.x;
  const float* A0 = Min + (size_t)blockIdx.x * k * k;
  float* A = Out + (size_t)blockIdx.x * k * k;
  for (int e = tid; e < k * k; e += nt) A[e] = A0[e];
  if (tid == 0) s_bad = 0;
  __syncthreads();
  for (int p = 0; p < k; ++p) {
    // pivot search over rows >= p of column p
    float best = -1.f;
    int bi = p;
    for (int i = p + tid; i < k; i += nt) {
      float v = fabsf(A[(size_t)i * k + p]);
      if (v > best) { best = v; bi = i; }
    }
    for (int o = 16; o > 0; o >>= 1) {
      float ov = __shfl_xor_sync(0xffffffffu, best, o);
      int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
    }
    if ((tid & 31) == 0) { rv[tid >> 5] = best; ri[tid >> 5] = bi; }
    __syncthreads();
    if (tid < 32) {
      int nw = (nt + 31) >> 5;
      best = (tid < nw) ? rv[tid] : -1.f;
      bi = (tid < nw) ? ri[tid] : p;
      for (int o = 16; o > 0; o >>= 1) {
        float ov = __shfl_xor_sync(0xffffffffu, best, o);
        int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
      }
      if (tid == 0) {
        s_r = bi;
        piv[p] = bi;
        if (!(best > 1e-30f) || !isfinite(best)) s_bad = 1;
      }
    }
    __syncthreads();
    if (s_bad) {
      if (tid == 0) raise_status(status, CAFEQ_ERR_SINGULAR);
      return;
    }
    const int r = s_r;
    // exchange rows p and r; keep the (new) pivot row in shared memory
    for (int j = tid; j < k; j += nt) {
      float vr = A[(size_t)r * k + j], vp = A[(size_t)p * k + j];
      A[(size_t)r * k + j] = vp;
      prow[j] = vr;
    }
    __syncthreads();
    const float d = 1.0f / prow[p];
    // column p after the exchange (factors); row p itself handled separately
    for (int i = tid; i < k; i += nt) fcol[i] = (i == p) ? 0.f : A[(size_t)i * k + p];
    __syncthreads();
    for (int e = tid; e < k * k; e += nt) {
      int i = e / k, j = e - i * k;
      float sp = (j == p) ? d : prow[j] * d;
      if (i == p) {
        A[e] = sp;
      } else {
        float cur = (j == p) ? 0.f : A[e];
        A[e] = fmaf(-fcol[i], sp, cur);
      }
    }
    __syncthreads();
  }
  // undo the row exchanges as column exchanges in reverse order
  for (int p = k - 1; p >= 0; --p) {
    int r = piv[p];
    if (r != p) {
      for (int i = tid; i < k; i += nt) {
        float a = A[(size_t)i * k + p];
        A[(size_t)i * k + p] = A[(size_t)i * k + r];
        A[(size_t)i * k + r] = a;
      }
    }
    __syncthreads();
  }
  if (cnorm) {
    for (int t = tid; t < k; t += nt) {
      float s = 0.f;
      for (int i = 0; i < k; ++i) {
        float v = A[(size_t)i * k + t];
        s = fmaf(v, v, s);
      }
      cnorm[(size_t)blockIdx.x * k + t] = s;
    }
  }
}

// ------------------------------------------------------------------------------------------------
// group absmax with arg-max (lowest index on ties): one warp per (row, group)
// ------------------------------------------------------------------------------------------------
__global__ void absmax_kernel(const float* __restrict__ U, long long ld, int rows, int ng, int g,
                              float* __restrict__ a, float* __restrict__ usel, int* __restrict__ idx, int32_t* status) {
  if (status && *status) return;
  long long w = (blockIdx.x * (long long)blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  const long long total = (long long)rows * ng;
  if (w >= total) return;
  const int row = (int)(w / ng), G = (int)(w - (long long)row * ng);
  const float* p = U + row * ld + (long long)G * g;
  float best = -1.f;
  int bi = 0x7fffffff;
  bool bad = false;
  for (int e = lane; e < g; e += 32) {
    float v = fabsf(p[e]);
    if (!(v <= 3.0e38f)) bad = true;
    if (v > best) { best = v; bi = e; }
  }
  for (int o = 16; o > 0; o >>= 1) {
    float ov = __shfl_xor_sync(0xffffffffu, best, o);
    int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
  }
  if (__any_sync(0xffffffffu, bad)) {
    if (lane == 0) raise_status(status, CAFEQ_ERR_NONFINITE);
    return;
  }
  if (lane == 0) {
    a[w] = best;
    idx[w] = bi;
    usel[w] = p[bi];  // signed value at the arg-max
  }
}

__global__ void scales_kernel(const float* __restrict__ a, float* __restrict__ s, long long n, float qmax,
                              const int32_t* status) {
  if (status && *status) return;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
    s[i] = __fdiv_rn(a[i], qmax);
}

// ------------------------------------------------------------------------------------------------
// quantise: code, dequantised value, residual Delta = Uhat - U
// ------------------------------------------------------------------------------------------------
// a: the group's absmax.  With rounding offsets an entry attaining it is always coded +-qmax: its exact quotient is
// +-qmax, where floor is discontinuous and the fp32 quotient lands an ulp above or below.
__device__ __forceinline__ float quantise_one(float u, float s, float a, float qmax, float off, int off_kind) {
  float x = (s > 0.f) ? __fdiv_rn(u, s) : 0.f;
  float q = (off_kind == CAFEQ_OFFSETS_NONE) ? rintf(x) : floorf(x) + off;
  if (off_kind != CAFEQ_OFFSETS_NONE && a > 0.f && fabsf(u) >= a) q = copysignf(qmax, u);
  return fminf(fmaxf(q, -qmax), qmax);
}

__global__ void quant_kernel(const float* __restrict__ U, long long ld, int rows, int cols, int g,
                             const float* __restrict__ a, float qmax, const void* __restrict__ offsets, int off_kind,
                             float* __restrict__ Delta, float* __restrict__ Uhat, int8_t* __restrict__ codes,
                             const int32_t* status) {
  if (status && *status) return;
  const int ng = cols / g;
  const long long n = (long long)rows * cols;
  for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
    int row = (int)(e / cols), col = (int)(e - (long long)row * cols);
    float u = U[row * ld + col];
    const float av = a[(long long)row * ng + col / g];
    float s = __fdiv_rn(av, qmax);
    float off = 0.f;
    if (off_kind == CAFEQ_OFFSETS_HARD_U8) off = (float)((const uint8_t*)offsets)[e];
    else if (off_kind == CAFEQ_OFFSETS_SOFT_F32) off = ((const float*)offsets)[e];
    float q = quantise_one(u, s, av, qmax, off, off_kind);
    float uh = s * q;
    if (Delta) Delta[row * ld + col] = uh - u;
    if (Uhat) Uhat[row * ld + col] = uh;
    if (codes) codes[e] = (int8_t)q;
  }
}

// ------------------------------------------------------------------------------------------------
// surrogate (Eq. 4 per entry): weights cw, loss, arg-max coefficients, A_t
// ------------------------------------------------------------------------------------------------
// axis IN:  cw[Gc] = sum_{t in group Gc} c[t'],  t' = (B / r) * k + (t mod k), B = t / k
__global__ void cw_in_kernel(const float* __restrict__ c, int d_in, int g, int k, int r, float* __restrict__ cw) {
  int Gc = blockIdx.x * blockDim.x + threadIdx.x;
  if (Gc >= d_in / g) return;
  float s = 0.f;
  for (int e = 0; e < g; ++e) {
    int t = Gc * g + e;
    int B = t / k;
    s += c[(B / r) * k + (t - B * k)];
  }
  cw[Gc] = s;
}

// axis OUT: cw[row] = g * c[t'(row)]
__global__ void cw_out_kernel(const float* __restrict__ c, int d_out, int g, int k, int r, float* __restrict__ cw) {
  int row = blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= d_out) return;
  int B = row / k;
  cw[row] = (float)g * c[(B / r) * k + (row - B * k)];
}

// one thread per row: loss partial sum and arg-max coefficients  coef = scale * cw * a * sign(U[e*]).
// A_t accumulation: axis IN  Agrp[Gc] += a^2 (per column group, expanded later);
//                   axis OUT A[t'(row)] += g * sum_G a^2.
__global__ void surrogate_rows_kernel(const float* __restrict__ a, const float* __restrict__ usel, int rows, int ng,
                                      int g, int axis,
                                      const float* __restrict__ cw, float kappa, int k, int r, float* __restrict__ coef,
                                      float* __restrict__ Agrp, float* __restrict__ A, double* __restrict__ acc,
                                      const int32_t* status) {
  if (status && *status) return;
  __shared__ double red[32];
  int row = blockIdx.x * blockDim.x + threadIdx.x;
  double local = 0.0;
  if (row < rows) {
    float srow = 0.f;
    for (int G = 0; G < ng; ++G) {
      long long w = (long long)row * ng + G;
      float av = a[w];
      float u = usel[w];
      float sgn = (u > 0.f) ? 1.f : ((u < 0.f) ? -1.f : 0.f);
      float wgt = (axis == CAFEQ_AXIS_IN) ? cw[G] : cw[row];
      local += (double)wgt * (double)av * (double)av;
      if (coef) coef[w] = 2.f * kappa * wgt * av * sgn;
      if (axis == CAFEQ_AXIS_IN) {
        if (Agrp) atomicAdd(&Agrp[G], av * av);
      } else {
        srow += av * av;
      }
    }
    if (axis == CAFEQ_AXIS_OUT && A) {
      int B = row / k;
      atomicAdd(&A[(B / r) * k + (row - B * k)], (float)g * srow);
    }
  }
  double s = block_sum_double(local, red);
  if (threadIdx.x == 0) atomicAdd(acc, (double)kappa * s);
}

// axis IN: A[t'] += Agrp[group of t]
__global__ void expand_agrp_kernel(const float* __restrict__ Agrp, int d_in, int g, int k, int r, float* __restrict__ A) {
  int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= d_in) return;
  int B = t / k;
  atomicAdd(&A[(B / r) * k + (t - B * k)], Agrp[t / g]);
}

// gMinv[b][i][t] = scale * Minv[b][i][t] * A[b][t]
__global__ void scale_cols_kernel(const float* __restrict__ Minv, const float* __restrict__ A, float scale, int k,
                                  long long n, float* __restrict__ out) {
  for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
    long long b = e / ((long long)k * k);
    int t = (int)(e % k);
    out[e] = scale * Minv[e] * A[b * k + t];
  }
}

// ------------------------------------------------------------------------------------------------
// straight-through scale path: coef[row, G] = sign(U[e*]) / qmax * sum_{e in G} gDelta_e (q_e - U_e / s_G)
// (+ optionally, for the pair PQE loss, the direct term stays in gU and is handled by a dense product)
// ------------------------------------------------------------------------------------------------
__global__ void ste_scale_path_kernel(const float* __restrict__ U, const float* __restrict__ gD, long long ld, int rows,
                                      int ng, int g, const float* __restrict__ a, const float* __restrict__ usel, float qmax,
                                      const void* __restrict__ offsets, int off_kind, int cols, float* __restrict__ coef,
                                      const int32_t* status) {
  if (status && *status) return;
  long long w = (blockIdx.x * (long long)blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (w >= (long long)rows * ng) return;
  const int row = (int)(w / ng), G = (int)(w - (long long)row * ng);
  const float av = a[w];
  const float s = __fdiv_rn(av, qmax);
  float sum = 0.f;
  for (int e = lane; e < g; e += 32) {
    long long col = (long long)G * g + e;
    float u = U[row * ld + col];
    float off = 0.f;
    if (off_kind == CAFEQ_OFFSETS_HARD_U8) off = (float)((const uint8_t*)offsets)[(long long)row * cols + col];
    else if (off_kind == CAFEQ_OFFSETS_SOFT_F32) off = ((const float*)offsets)[(long long)row * cols + col];
    float q = quantise_one(u, s, av, qmax, off, off_kind);
    float x = (s > 0.f) ? __fdiv_rn(u, s) : 0.f;
    sum = fmaf(gD[row * ld + col], q - x, sum);
  }
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  if (lane == 0) {
    float u = usel[w];
    float sgn = (u > 0.f) ? 1.f : ((u < 0.f) ? -1.f : 0.f);
    coef[w] = sum * sgn / qmax;
  }
}

// d loss / d rho for soft rounding offsets: Uhat = s (floor(U/s) + rho) with the scale kept, so d Uhat / d rho = s and
// the gradient is s * gUhat; entries attaining their group's absmax are coded +-qmax whatever rho and get 0.
__global__ void grad_offsets_kernel(const float* __restrict__ U, const float* __restrict__ gUhat, long long ld, int rows, int cols,
                                    int g, const float* __restrict__ a, float qmax, float* __restrict__ out,
                                    const int32_t* status) {
  if (status && *status) return;
  const int ng = cols / g;
  const long long n = (long long)rows * cols;
  for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
    const int row = (int)(e / cols), col = (int)(e - (long long)row * cols);
    const float av = a[(long long)row * ng + col / g];
    const float s = __fdiv_rn(av, qmax);
    const float u = U[row * ld + col];
    out[e] = (av > 0.f && fabsf(u) >= av) ? 0.f : s * gUhat[row * ld + col];
  }
}

// ------------------------------------------------------------------------------------------------
// sparse backward: gradT[B/r][i][j] += sum over (row, group) pairs routed through their arg-max entry
//   axis IN : pair (o, G) in block B adds coef * W[o, B*k + j] to row i* = (G*g + idx) mod k
//   axis OUT: pair (B*k + i, G) adds coef * W[B*k + j, G*g + idx] to row i
// transpose_out stores into gradT[..][j][i] instead (operator applied transposed).
// One CTA owns a strip of JS columns j of one block and accumulates it in shared memory.
// ------------------------------------------------------------------------------------------------
constexpr int SCATTER_JS = 32;

__global__ void __launch_bounds__(256) scatter_in_kernel(const uint16_t* __restrict__ W, long long ld, int d_out, int d_in,
                                                         int g, int k, int r, const float* __restrict__ coef,
                                                         const int* __restrict__ idx, float* __restrict__ gradT,
                                                         int transpose_out, int rows_per_cta, const int32_t* status, int gm) {
  if (status && *status) return;
  extern __shared__ float acc[];  // [k][SCATTER_JS]
  const int B = blockIdx.x, js = blockIdx.y * SCATTER_JS;
  const int r0 = blockIdx.z * rows_per_cta, r1 = min(d_out, r0 + rows_per_cta);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nw = blockDim.x >> 5;
  for (int e = tid; e < k * SCATTER_JS; e += blockDim.x) acc[e] = 0.f;
  __syncthreads();
  const int ng = d_in / g;
  const int j = js + lane;
  // groups that intersect this block: columns [B*k, B*k + k)
  const int G0 = (B * k) / g, G1 = (B * k + k - 1) / g;
  for (int o = r0 + warp; o < r1; o += nw) {
    float w = (j < k) ? bf16_bits_to_float(W[o * ld + (long long)B * k + j]) : 0.f;
    for (int G = G0; G <= G1; ++G) {
      long long p = gm ? (long long)G * d_out + o : (long long)o * ng + G;
      int col = G * g + idx[p];          // arg-max column of the group
      if (col < B * k || col >= B * k + k) continue;  // group larger than the block: arg-max in another block
      float cf = coef[p];
      if (j < k && cf != 0.f) atomicAdd(&acc[(col - B * k) * SCATTER_JS + lane], cf * w);
    }
  }
  __syncthreads();
  float* out = gradT + (size_t)(B / r) * k * k;
  for (int e = tid; e < k * SCATTER_JS; e += blockDim.x) {
    int i = e / SCATTER_JS, jj = js + (e - i * SCATTER_JS);
    if (jj < k && acc[e] != 0.f) atomicAdd(transpose_out ? &out[(size_t)jj * k + i] : &out[(size_t)i * k + jj], acc[e]);
  }
}

__global__ void __launch_bounds__(256) scatter_out_kernel(const uint16_t* __restrict__ W, long long ld, int d_out, int d_in,
                                                          int g, int k, int r, const float* __restrict__ coef,
                                                          const int* __restrict__ idx, float* __restrict__ gradT,
                                                          int transpose_out, int groups_per_cta, const int32_t* status, int gm) {
  if (status && *status) return;
  extern __shared__ float acc[];  // [k][SCATTER_JS]
  const int B = blockIdx.x, js = blockIdx.y * SCATTER_JS;
  const int ng = d_in / g;
  const int G0 = blockIdx.z * groups_per_cta, G1 = min(ng, G0 + groups_per_cta);
  const int tid = threadIdx.x;
  for (int e = tid; e < k * SCATTER_JS; e += blockDim.x) acc[e] = 0.f;
  __syncthreads();
  // thread handles (i, jj) pairs: i over rows of the block, jj over the strip
  for (int e = tid; e < k * SCATTER_JS; e += blockDim.x) {
    int i = e / SCATTER_JS, jj = e - i * SCATTER_JS;
    int j = js + jj;
    if (j >= k) continue;
    float s = 0.f;
    long long row = (long long)B * k + i;
    for (int G = G0; G < G1; ++G) {
      long long p = gm ? (long long)G * d_out + row : row * ng + G;
      float cf = coef[p];
      if (cf != 0.f) s = fmaf(cf, bf16_bits_to_float(W[((long long)B * k + j) * ld + (long long)G * g + idx[p]]), s);
    }
    acc[e] = s;
  }
  __syncthreads();
  float* out = gradT + (size_t)(B / r) * k * k;
  for (int e = tid; e < k * SCATTER_JS; e += blockDim.x) {
    int i = e / SCATTER_JS, jj = js + (e - i * SCATTER_JS);
    if (jj < k && acc[e] != 0.f) atomicAdd(transpose_out ? &out[(size_t)jj * k + i] : &out[(size_t)i * k + jj], acc[e]);
  }
}

// ------------------------------------------------------------------------------------------------
// sparse backward, strip form (k a multiple of 64).  One CTA owns 64 columns j of one block and a share of
// the free axis, accumulates gradT[.][i][js..js+64) in shared memory and adds it to global memory once.
// ------------------------------------------------------------------------------------------------
constexpr int SC2_JS = 64;
constexpr int SC2_MAXG = 4;  // groups of one row that can fall into one block (k / g)

// axis IN: every (row o, group G) adds coef * W[o, B*k + j] to row i* = arg-max column - B*k (shared atomics:
// the target row depends on the data).  A warp takes 32 consecutive rows: each lane fetches the records
// (target row, coefficient) of one row, then the warp walks the 32 rows, broadcasting a record by shuffle and
// adding the row's 64 strip columns.  A lane owns the adjacent columns 2*lane and 2*lane+1 (one 32-bit load);
// inside the accumulator the even columns sit in the first half of a row and the odd ones in the second, so both
// atomics of a warp are bank-conflict free.  NG = groups of one row that fall into one block.
template <int NG>
__global__ void __launch_bounds__(256, 3) scatter_in_strip_kernel(const uint16_t* __restrict__ W, long long ld, int d_out,
                                                                  int d_in, int g, int k, int r, const float* __restrict__ coef,
                                                                  const int* __restrict__ idx, float* __restrict__ gradT,
                                                                  int transpose_out, int rows_per_cta, const int32_t* status, int gm) {
  if (status && *status) return;
  extern __shared__ float acc[];  // [k][64]
  const int B = blockIdx.x, js = blockIdx.y * SC2_JS;
  const int r0 = blockIdx.z * rows_per_cta, r1 = min(d_out, r0 + rows_per_cta);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int e = tid; e < k * SC2_JS; e += 256) acc[e] = 0.f;
  __syncthreads();
  const int ng = d_in / g;
  const int G0 = (B * k) / g;
  const int off = G0 * g - B * k;  // column of the first group's start relative to the block
  const uint32_t* Wp = reinterpret_cast<const uint32_t*>(W + (long long)B * k + js) + lane;
  const long long ldw = ld / 2;
  float* accl = acc + lane;
  for (int base = r0 + warp * 32; base < r1; base += 256) {
    int ii[NG];
    float cf[NG];
    {
      const int o = base + lane;
      const bool ok = o < r1;
      const int oo = ok ? o : r0;
#pragma unroll
      for (int q = 0; q < NG; ++q) {
        const long long pq = gm ? (long long)(G0 + q) * d_out + oo : (long long)oo * ng + G0 + q;
        const int ix = __ldg(idx + pq);
        const float c = __ldg(coef + pq);
        const int col = q * g + ix + off;
        const bool in = ok && (unsigned)col < (unsigned)k;
        cf[q] = in ? c : 0.f;
        ii[q] = in ? col * SC2_JS : 0;
      }
    }
#pragma unroll
    for (int c8 = 0; c8 < 32; c8 += 8) {
      uint32_t w[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int row = base + c8 + u;
        w[u] = (row < r1) ? __ldg(Wp + row * ldw) : 0u;
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const float w0 = __uint_as_float(w[u] << 16), w1 = __uint_as_float(w[u] & 0xFFFF0000u);
#pragma unroll
        for (int q = 0; q < NG; ++q) {
          const int io = __shfl_sync(0xffffffffu, ii[q], c8 + u);
          const float c = __shfl_sync(0xffffffffu, cf[q], c8 + u);
          atomicAdd(accl + io, c * w0);
          atomicAdd(accl + io + 32, c * w1);
        }
      }
    }
  }
  __syncthreads();
  float* out = gradT + (size_t)(B / r) * k * k;
  for (int e = tid; e < k * SC2_JS; e += 256) {
    const int i = e / SC2_JS, pos = e - i * SC2_JS;
    const int jj = js + ((pos < 32) ? 2 * pos : 2 * (pos - 32) + 1);
    const float v = acc[e];
    if (v != 0.f) atomicAdd(transpose_out ? &out[(size_t)jj * k + i] : &out[(size_t)i * k + jj], v);
  }
}

// axis IN, bucketed form (no floating-point atomics in shared memory): the CTA first sorts the (row, group)
// records of its row range by target row i* (a counting sort in shared memory; integer atomics only), then
// thread t owns target row t / TPB and a run of 64 / TPB strip columns with the accumulators in registers and
// walks its bucket: every record adds coef * W[row, strip] (one 128-byte row segment, read with 16-byte loads).
// The accumulators go through shared memory to a coalesced add into global memory.
// K in {64, 128, 256}; rows_per_cta * NG <= SCB_MAXP; ld % 8 == 0 and W 16-byte aligned.
constexpr int SCB_MAXP = 4096;

template <int K, int STRIP>
__global__ void __launch_bounds__(256, 2) scatter_in_bucket_kernel(const uint16_t* __restrict__ W, long long ld, int d_out,
                                                                   int d_in, int g, int r, int NG, const float* __restrict__ coef,
                                                                   const int* __restrict__ idx, float* __restrict__ gradT,
                                                                   int transpose_out, int rows_per_cta, const int32_t* status, int gm) {
  if (status && *status) return;
  constexpr int TPB = 256 / K;      // threads per bucket
  constexpr int CPT = STRIP / TPB;  // strip columns per thread
  constexpr int SP = STRIP + 1;     // padded row of the staging buffer
  constexpr int RPT = SCB_MAXP / 256;
  extern __shared__ __align__(16) uint8_t sc_smem[];
  float* stage = reinterpret_cast<float*>(sc_smem);                       // [K][STRIP + 1]
  float* rec_cf = stage + K * SP;                                         // [SCB_MAXP]
  uint16_t* rec_o = reinterpret_cast<uint16_t*>(rec_cf + SCB_MAXP);       // [SCB_MAXP]
  __shared__ int cnt[K], start[K + 1], cursor[K], wsum[8];
  const int B = blockIdx.x, js = blockIdx.y * STRIP;
  const int r0 = blockIdx.z * rows_per_cta, r1 = min(d_out, r0 + rows_per_cta);
  const int R = r1 - r0;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int ng = d_in / g;
  const int G0 = (B * K) / g;
  const int off = G0 * g - B * K;
  for (int e = tid; e < K; e += 256) cnt[e] = 0;
  __syncthreads();
  // phase A: fetch this thread's records, count per target row
  short bk[RPT];
  float cfv[RPT];
  const int np = R * NG;
#pragma unroll
  for (int u = 0; u < RPT; ++u) {
    const int e = tid + u * 256;
    bk[u] = -1;
    cfv[u] = 0.f;
    if (e < np) {
      const int row = e / NG, q = e - row * NG;
      const long long p = gm ? (long long)(G0 + q) * d_out + r0 + row : (long long)(r0 + row) * ng + G0 + q;
      const float c = __ldg(coef + p);
      const int col = q * g + __ldg(idx + p) + off;
      if ((unsigned)col < (unsigned)K && c != 0.f) {
        bk[u] = (short)col;
        cfv[u] = c;
        atomicAdd(&cnt[col], 1);
      }
    }
  }
  __syncthreads();
  // exclusive scan of cnt -> start (K <= 256: one entry per thread)
  {
    int v = (tid < K) ? cnt[tid] : 0;
    int x = v;
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, x, o);
      if (lane >= o) x += y;
    }
    if (lane == 31) wsum[warp] = x;
    __syncthreads();
    int base = 0;
    for (int w = 0; w < warp; ++w) base += wsum[w];
    if (tid < K) {
      start[tid] = base + x - v;
      cursor[tid] = base + x - v;
    }
    if (tid == K - 1) start[K] = base + x;
  }
  __syncthreads();
  // phase B: place the records
#pragma unroll
  for (int u = 0; u < RPT; ++u) {
    if (bk[u] >= 0) {
      const int pos = atomicAdd(&cursor[bk[u]], 1);
      const int e = tid + u * 256;
      rec_o[pos] = (uint16_t)(e / NG);
      rec_cf[pos] = cfv[u];
    }
  }
  __syncthreads();
  // phase C: every thread walks its bucket
  const int b = tid / TPB, part = tid - b * TPB;
  float acc[CPT];
#pragma unroll
  for (int c = 0; c < CPT; ++c) acc[c] = 0.f;
  const uint16_t* Wb = W + (long long)r0 * ld + (long long)B * K + js + part * CPT;
  const int p1 = start[b + 1];
  // the row segment of the next record is requested before the current one is accumulated (two register sets)
  constexpr int NV = CPT / 8;
  uint4 wa[NV], wb[NV];
  float cfa = 0.f, cfb = 0.f;
  auto fetch = [&](int p, uint4* w, float& cf) {
    cf = rec_cf[p];
    const uint4* src = reinterpret_cast<const uint4*>(Wb + (long long)rec_o[p] * ld);
#pragma unroll
    for (int v = 0; v < NV; ++v) w[v] = __ldg(src + v);
  };
  auto accumulate = [&](const uint4* w, float cf) {
#pragma unroll
    for (int v = 0; v < NV; ++v) {
      const uint32_t ww[4] = {w[v].x, w[v].y, w[v].z, w[v].w};
#pragma unroll
      for (int h = 0; h < 4; ++h) {
        acc[v * 8 + 2 * h] = fmaf(cf, __uint_as_float(ww[h] << 16), acc[v * 8 + 2 * h]);
        acc[v * 8 + 2 * h + 1] = fmaf(cf, __uint_as_float(ww[h] & 0xFFFF0000u), acc[v * 8 + 2 * h + 1]);
      }
    }
  };
  int p = start[b];
  if (p < p1) fetch(p, wa, cfa);
  while (p < p1) {
    if (p + 1 < p1) fetch(p + 1, wb, cfb);
    accumulate(wa, cfa);
    if (++p >= p1) break;
    if (p + 1 < p1) fetch(p + 1, wa, cfa);
    accumulate(wb, cfb);
    ++p;
  }
#pragma unroll
  for (int c = 0; c < CPT; ++c) stage[b * SP + part * CPT + c] = acc[c];
  __syncthreads();
  float* out = gradT + (size_t)(B / r) * K * K;
  for (int e = tid; e < K * STRIP; e += 256) {
    const int i = e / STRIP, c = e - i * STRIP;
    const float v = stage[i * SP + c];
    if (v != 0.f) atomicAdd(transpose_out ? &out[(size_t)(js + c) * K + i] : &out[(size_t)i * K + js + c], v);
  }
}

// axis OUT: pair (row B*k + i, group G) adds coef * W[B*k + j, G*g + idx] to gradT[i][j].  The CTA stages the
// tile W[B*k + js .. +64, G*g .. +g] in shared memory; warp w owns the rows i = w, w+8, ... of the block and a
// lane the strip columns lane and lane+32, with the K/8 x 2 accumulators in registers: every (i, j) has exactly
// one owner, so nothing is atomic until the final add to global memory.  Tiles and the (coef, idx) records of
// the next group arrive by asynchronous copies while the current group is accumulated.  g <= 128, g % 4 == 0.
__device__ __forceinline__ void cp_async8(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async4(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

template <int K>
__global__ void __launch_bounds__(256) scatter_out_strip_kernel(const uint16_t* __restrict__ W, long long ld, int d_out,
                                                                int d_in, int g, int r, const float* __restrict__ coef,
                                                                const int* __restrict__ idx, float* __restrict__ gradT,
                                                                int transpose_out, int groups_per_cta, const int32_t* status, int gm) {
  if (status && *status) return;
  constexpr int RW = K / 8;  // rows of the block per warp
  extern __shared__ __align__(16) uint16_t tiles[];  // two tiles [64][g + 4]
  __shared__ float s_cf[2][K];
  __shared__ int s_ix[2][K];
  const int tp = g + 4;
  const int B = blockIdx.x, js = blockIdx.y * SC2_JS;
  const int ng = d_in / g;
  const int Ga = blockIdx.z * groups_per_cta, Gb = min(ng, Ga + groups_per_cta);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int qg = g / 4;  // 8-byte chunks per tile row
  float a0[RW], a1[RW];
#pragma unroll
  for (int m = 0; m < RW; ++m) { a0[m] = 0.f; a1[m] = 0.f; }
  auto stage = [&](int G, int buf) {
    uint16_t* tile = tiles + (size_t)buf * SC2_JS * tp;
    const uint16_t* src = W + ((long long)B * K + js) * ld + (long long)G * g;
    for (int e = tid; e < SC2_JS * qg; e += 256) {
      const int jr = e / qg, c4 = e - jr * qg;
      cp_async8(tile + jr * tp + 4 * c4, src + jr * ld + 4 * c4);
    }
    for (int i = tid; i < K; i += 256) {
      const long long p = gm ? (long long)G * d_out + (long long)B * K + i : ((long long)B * K + i) * ng + G;
      cp_async4(&s_cf[buf][i], coef + p);
      cp_async4(&s_ix[buf][i], idx + p);
    }
    cp_async_commit();
  };
  int buf = 0;
  if (Ga < Gb) stage(Ga, 0);
  for (int G = Ga; G < Gb; ++G) {
    if (G + 1 < Gb) {
      stage(G + 1, buf ^ 1);
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    const uint16_t* t0 = tiles + (size_t)buf * SC2_JS * tp + lane * tp;
    const uint16_t* t1 = t0 + 32 * tp;
    // lane m keeps the record of this warp's m-th row
    const float cfl = (lane < RW) ? s_cf[buf][warp + 8 * lane] : 0.f;
    const int ixl = (lane < RW) ? s_ix[buf][warp + 8 * lane] : 0;
#pragma unroll
    for (int m = 0; m < RW; ++m) {
      const float cf = __shfl_sync(0xffffffffu, cfl, m);
      const int c = __shfl_sync(0xffffffffu, ixl, m);
      a0[m] = fmaf(cf, bf16_bits_to_float(t0[c]), a0[m]);
      a1[m] = fmaf(cf, bf16_bits_to_float(t1[c]), a1[m]);
    }
    __syncthreads();
    buf ^= 1;
  }
  float* out = gradT + (size_t)(B / r) * K * K;
#pragma unroll
  for (int m = 0; m < RW; ++m) {
    const int i = warp + 8 * m;
    if (!transpose_out) {
      if (a0[m] != 0.f) atomicAdd(&out[(size_t)i * K + js + lane], a0[m]);
      if (a1[m] != 0.f) atomicAdd(&out[(size_t)i * K + js + lane + 32], a1[m]);
    } else {
      if (a0[m] != 0.f) atomicAdd(&out[(size_t)(js + lane) * K + i], a0[m]);
      if (a1[m] != 0.f) atomicAdd(&out[(size_t)(js + lane + 32) * K + i], a1[m]);
    }
  }
}

// ------------------------------------------------------------------------------------------------
// step set-up in one launch: Mc = float(bf16(M)), Ab = bf16(M), every accumulator of the step cleared, the
// optimiser's step counter advanced
// ------------------------------------------------------------------------------------------------
struct PrepArgs {
  const float* M;
  float* Mc;
  uint16_t* Ab;
  long long kk;
  float* zero_f[4];      // fp32 arrays to clear
  long long zero_fn[4];
  double* zero_d[2];     // double arrays to clear
  int zero_dn[2];
  int* flag;             // cleared
  float* step_counter;   // += 1 (optimiser state), may be null
  const int32_t* status;
};

__global__ void step_prep_kernel(PrepArgs a) {
  if (a.status && *a.status) return;
  const long long stride = (long long)gridDim.x * blockDim.x, t0 = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  for (long long e = t0; e < a.kk; e += stride) {
    const __nv_bfloat16 h = __float2bfloat16_rn(a.M[e]);
    if (a.Mc) a.Mc[e] = __bfloat162float(h);
    if (a.Ab) a.Ab[e] = __bfloat16_as_ushort(h);
  }
#pragma unroll
  for (int q = 0; q < 4; ++q)
    if (a.zero_f[q])
      for (long long e = t0; e < a.zero_fn[q]; e += stride) a.zero_f[q][e] = 0.f;
#pragma unroll
  for (int q = 0; q < 2; ++q)
    if (a.zero_d[q])
      for (long long e = t0; e < a.zero_dn[q]; e += stride) a.zero_d[q][e] = 0.0;
  if (t0 == 0) {
    if (a.flag) *a.flag = 0;
    if (a.step_counter) *a.step_counter += 1.f;
  }
}

// c[b][t] = sum_i X[b][i][t]^2 for 32 columns t per CTA (grid: k/32, nb; block 32 x 8), and optionally the
// input-axis group weights cw[Gc] += sum_{t in Gc} c[t] (cw cleared by the caller; groups are runs of g columns
// of the concatenated blocks, r = 1)
__global__ void __launch_bounds__(256) colnorm_cw_kernel(const float* __restrict__ X, int k, float* __restrict__ c,
                                                         float* __restrict__ cw, int g) {
  __shared__ float part[8][33];
  const int b = blockIdx.y, t = blockIdx.x * 32 + threadIdx.x;
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
    if (c) c[(size_t)b * k + t] = tot;
    if (cw) {
      const int col = b * k + t;  // position along the transformed axis
      if (g >= 32) {
        for (int o = 16; o > 0; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
        if (threadIdx.x == 0) atomicAdd(&cw[col / g], tot);
      } else {
        atomicAdd(&cw[col / g], tot);
      }
    }
  }
}

// dL/dMinv of Eq. 4: out[b][i][t] = scale * Minv[b][i][t] * A_t; input axis with r = 1 reads A_t = Agrp[(b k + t) / g]
__global__ void gminv_kernel(const float* __restrict__ Minv, const float* __restrict__ A, const float* __restrict__ Agrp,
                             int g, float scale, int k, long long n, float* __restrict__ out) {
  for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
    const long long b = e / ((long long)k * k);
    const int t = (int)(e % k);
    const float At = Agrp ? Agrp[(b * k + t) / g] : A[b * k + t];
    out[e] = scale * Minv[e] * At;
  }
}

// ------------------------------------------------------------------------------------------------
// optimiser updates and bookkeeping
// ------------------------------------------------------------------------------------------------
__global__ void gd_update_kernel(float* __restrict__ M, const float* __restrict__ g, float lr, long long n,
                                 const int32_t* status) {
  if (status && *status) return;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
    M[i] = M[i] - lr * g[i];
}

// state = {step, m[n], v[n]}; the step counter is advanced by adam_tick_kernel before the update.
__global__ void adam_tick_kernel(float* state, const int32_t* status) {
  if (status && *status) return;
  state[0] += 1.f;
}

__global__ void adam_update_kernel(float* __restrict__ M, const float* __restrict__ g, float* __restrict__ state, float lr,
                                   float b1, float b2, float eps, long long n, const int32_t* status) {
  if (status && *status) return;
  const float step = state[0];
  const float c1 = 1.f - powf(b1, step), c2 = 1.f - powf(b2, step);
  float* m = state + CAFEQ_OPT_STATE_HEADER;
  float* v = state + CAFEQ_OPT_STATE_HEADER + n;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    float gi = g[i];
    float mi = b1 * m[i] + (1.f - b1) * gi;
    float vi = b2 * v[i] + (1.f - b2) * gi * gi;
    m[i] = mi;
    v[i] = vi;
    M[i] = M[i] - lr * (mi / c1) / (sqrtf(vi / c2) + eps);
  }
}

// ------------------------------------------------------------------------------------------------
// reductions: sum of squares of bf16 / fp32 arrays
// ------------------------------------------------------------------------------------------------
__global__ void sqsum_bf16_kernel(const uint16_t* __restrict__ W, long long ld, int rows, int cols, double* acc,
                                  const int32_t* status) {
  if (status && *status) return;
  __shared__ double red[32];
  double local = 0.0;
  if ((cols % 8) == 0 && (ld % 8) == 0 && ((uintptr_t)W % 16) == 0) {
    // eight values per 16-byte load, fp32 inside the chunk (double arithmetic is scarce), double across chunks
    const int cpr = cols / 8;
    const long long nch = (long long)rows * cpr;
    for (long long c = blockIdx.x * (long long)blockDim.x + threadIdx.x; c < nch; c += (long long)gridDim.x * blockDim.x) {
      const long long row = c / cpr;
      const int cc = (int)(c - row * cpr);
      const uint4 q = __ldg(reinterpret_cast<const uint4*>(W + row * ld) + cc);
      const uint32_t w4[4] = {q.x, q.y, q.z, q.w};
      float s = 0.f;
#pragma unroll
      for (int h = 0; h < 4; ++h) {
        const float lo = __uint_as_float(w4[h] << 16), hi = __uint_as_float(w4[h] & 0xFFFF0000u);
        s = fmaf(lo, lo, s);
        s = fmaf(hi, hi, s);
      }
      local += (double)s;
    }
  } else {
    const long long n = (long long)rows * cols;
    for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
      int row = (int)(e / cols), col = (int)(e - (long long)row * cols);
      float v = bf16_bits_to_float(W[row * ld + col]);
      local += (double)v * v;
    }
  }
  double s = block_sum_double(local, red);
  if (threadIdx.x == 0) atomicAdd(acc, s);
}

// ------------------------------------------------------------------------------------------------
// pair: LogSumExp over group maxima (two passes), orthonormality penalty
// ------------------------------------------------------------------------------------------------
__global__ void max_f32_kernel(const float* __restrict__ a, long long n, float* __restrict__ out_max,
                               const int32_t* status) {
  // a >= 0, so an integer atomicMax on the bit pattern orders correctly
  if (status && *status) return;
  float m = 0.f;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
    m = fmaxf(m, a[i]);
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0) atomicMax((int*)out_max, __float_as_int(m));
}

__global__ void sumexp_kernel(const float* __restrict__ a, long long n, const float* __restrict__ amax, float t,
                              double* __restrict__ acc, const int32_t* status) {
  if (status && *status) return;
  __shared__ double red[32];
  const float mx = *amax;
  double local = 0.0;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
    local += (double)expf(t * (a[i] - mx));
  double s = block_sum_double(local, red);
  if (threadIdx.x == 0) atomicAdd(acc, s);
}

// coef[w] = exp(t (a - max)) / Z * sign(U[arg-max])
__global__ void lse_coef_kernel(const float* __restrict__ a, const float* __restrict__ usel, long long n,
                                const float* __restrict__ amax, float t, const double* __restrict__ Z,
                                float* __restrict__ coef, const int32_t* status) {
  if (status && *status) return;
  const float mx = *amax;
  const float zinv = (float)(1.0 / *Z);
  for (long long w = blockIdx.x * (long long)blockDim.x + threadIdx.x; w < n; w += (long long)gridDim.x * blockDim.x) {
    float u = usel[w];
    float sgn = (u > 0.f) ? 1.f : ((u < 0.f) ? -1.f : 0.f);
    coef[w] = expf(t * (a[w] - mx)) * zinv * sgn;
  }
}

// two-array forms of the three LogSumExp kernels (the group maxima of U and of V in one launch each)
__global__ void max2_f32_kernel(const float* __restrict__ a1, long long n1, const float* __restrict__ a2, long long n2,
                                float* __restrict__ out_max, const int32_t* status) {
  if (status && *status) return;
  float m = 0.f;
  const long long n = n1 + n2;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
    m = fmaxf(m, i < n1 ? a1[i] : a2[i - n1]);
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0) atomicMax((int*)out_max, __float_as_int(m));
}

__global__ void sumexp2_kernel(const float* __restrict__ a1, long long n1, const float* __restrict__ a2, long long n2,
                               const float* __restrict__ amax, float t, double* __restrict__ acc, const int32_t* status) {
  if (status && *status) return;
  __shared__ double red[32];
  const float mx = *amax;
  double local = 0.0;
  const long long n = n1 + n2;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
    local += (double)expf(t * ((i < n1 ? a1[i] : a2[i - n1]) - mx));
  double s = block_sum_double(local, red);
  if (threadIdx.x == 0) atomicAdd(acc, s);
}

__global__ void lse_coef2_kernel(const float* __restrict__ a1, const float* __restrict__ u1, float* __restrict__ c1, long long n1,
                                 const float* __restrict__ a2, const float* __restrict__ u2, float* __restrict__ c2, long long n2,
                                 const float* __restrict__ amax, float t, const double* __restrict__ Z, const int32_t* status) {
  if (status && *status) return;
  const float mx = *amax;
  const float zinv = (float)(1.0 / *Z);
  const long long n = n1 + n2;
  for (long long w = blockIdx.x * (long long)blockDim.x + threadIdx.x; w < n; w += (long long)gridDim.x * blockDim.x) {
    const bool first = w < n1;
    const long long i = first ? w : w - n1;
    const float u = first ? u1[i] : u2[i];
    const float av = first ? a1[i] : a2[i];
    const float sgn = (u > 0.f) ? 1.f : ((u < 0.f) ? -1.f : 0.f);
    const float c = expf(t * (av - mx)) * zinv * sgn;
    if (first) c1[i] = c; else c2[i] = c;
  }
}

// R = M M^T - I in place on a [nb,k,k] buffer that already holds M M^T
__global__ void sub_identity_kernel(float* __restrict__ R, int k, long long n) {
  for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
    long long q = e % ((long long)k * k);
    if (q / k == q % k) R[e] -= 1.f;
  }
}

__global__ void sqsum_f32_kernel(const float* __restrict__ x, long long n, double* acc) {
  __shared__ double red[32];
  double local = 0.0;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
    local += (double)x[i] * x[i];
  double s = block_sum_double(local, red);
  if (threadIdx.x == 0) atomicAdd(acc, s);
}

// gradM += lambda * 2 (R M) / (||R||_F sqrt(h));  RM holds R M;  nothing when ||R||_F / sqrt(h) < 1e-5
// (the un-squared norm has no gradient at R = 0 and below the fp32 noise floor its direction is noise)
__global__ void orth_grad_kernel(float* __restrict__ gradM, const float* __restrict__ RM, const double* __restrict__ r2,
                                 float lambda, float sqrt_h, long long n) {
  const double nrm = sqrt(*r2);
  if (nrm < 1e-5 * (double)sqrt_h) return;
  const float f = (float)(2.0 * lambda / (nrm * sqrt_h));
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
    gradM[i] += f * RM[i];
}

// ------------------------------------------------------------------------------------------------
// finalisers: double accumulators -> the fp32 outputs of the API
// ------------------------------------------------------------------------------------------------
// single: acc = {surrogate, L2, ||W||^2}
__global__ void finalize_single_kernel(const double* acc, float* losses, float* hist /*[2] or NULL*/, int want_exact) {
  if (losses) {
    losses[0] = (float)acc[0];
    losses[1] = want_exact ? (float)acc[1] : 0.f;
    losses[2] = want_exact ? (float)acc[2] : 0.f;
    losses[3] = 0.f;
  }
  if (hist) {
    hist[0] = (float)acc[0];
    hist[1] = want_exact ? (float)acc[1] : nanf("");
  }
}

// Appendix D.1's sums of squares over the group maxima: coef = w * 2 a sign(U at the arg-max) / count, with
// w = the other factor's Frobenius norm in the weighted form (acc[5] = ||U||_F^2, acc[6] = ||V||_F^2), else 1
__global__ void sumsq_coef2_kernel(const float* __restrict__ a1, const float* __restrict__ u1, float* __restrict__ c1, long long n1,
                                   const float* __restrict__ a2, const float* __restrict__ u2, float* __restrict__ c2, long long n2,
                                   const double* __restrict__ acc, int weighted, const int32_t* status) {
  if (status && *status) return;
  const float w1 = (weighted ? (float)sqrt(acc[6]) : 1.f) * 2.f / (float)n1;
  const float w2 = (weighted ? (float)sqrt(acc[5]) : 1.f) * 2.f / (float)n2;
  const long long n = n1 + n2;
  for (long long w = blockIdx.x * (long long)blockDim.x + threadIdx.x; w < n; w += (long long)gridDim.x * blockDim.x) {
    const bool first = w < n1;
    const long long i = first ? w : w - n1;
    const float u = first ? u1[i] : u2[i];
    const float av = first ? a1[i] : a2[i];
    const float sgn = (u > 0.f) ? 1.f : ((u < 0.f) ? -1.f : 0.f);
    if (first) c1[i] = w1 * av * sgn; else c2[i] = w2 * av * sgn;
  }
}

// dst += (acc[num] / count) / sqrt(acc[den]) * src   (the dense terms of the weighted form: mean(a^2) d||X||_F)
__global__ void axpy_norm_kernel(float* __restrict__ dst, const float* __restrict__ src, long long n, const double* __restrict__ acc,
                                 int num, double count, int den, const int32_t* status) {
  if (status && *status) return;
  const double d = sqrt(acc[den]);
  const float f = d > 0.0 ? (float)(acc[num] / count / d) : 0.f;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
    dst[i] = fmaf(f, src[i], dst[i]);
}

// out = T - T^T per block (the skew part that drives a Cayley step)
__global__ void skew_blocks_kernel(const float* __restrict__ T, float* __restrict__ out, int k, long long n) {
  const long long kk = (long long)k * k;
  for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
    const long long b = e / kk, q = e - b * kk;
    const int i = (int)(q / k), j = (int)(q - (long long)i * k);
    out[e] = T[e] - T[b * kk + (long long)j * k + i];
  }
}

// out = x + alpha * y  /  x = beta * x + y
__global__ void lincomb_kernel(float* __restrict__ out, const float* __restrict__ x, float alpha, const float* __restrict__ y,
                               long long n, const int32_t* status) {
  if (status && *status) return;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
    out[i] = fmaf(alpha, y[i], x[i]);
}
__global__ void momentum_kernel(float* __restrict__ v, float beta, const float* __restrict__ g, long long n, const int32_t* status) {
  if (status && *status) return;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
    v[i] = fmaf(beta, v[i], g[i]);
}

// pair: acc = {Z, ||R_orth||^2, PQE^2, sum a_U^2, sum a_V^2, ||U||_F^2, ||V||_F^2}; amax = running max.
// objective 0: LogSumExp; 1: mean of squared maxima; 2: the norm-weighted form (counts n1, n2 of group maxima)
__global__ void finalize_pair_kernel(const double* acc, const float* amax, float t, float lambda, float sqrt_h,
                                     float* losses, float* hist, int want_pqe, int objective = 0, double n1 = 1.0,
                                     double n2 = 1.0) {
  float lse = *amax + (float)(log(acc[0]) / (double)t);
  if (objective == 1) lse = (float)(acc[3] / n1 + acc[4] / n2);
  if (objective == 2) lse = (float)(sqrt(acc[6]) * acc[3] / n1 + sqrt(acc[5]) * acc[4] / n2);
  float orth = (float)(sqrt(acc[1]) / (double)sqrt_h);
  // want_pqe == 2: the squared product error is the loss being minimised (straight-through mode)
  const float loss = (want_pqe == 2) ? (float)acc[2] : lse + lambda * orth;
  if (losses) {
    losses[0] = loss;
    losses[1] = lse;
    losses[2] = orth;
    losses[3] = want_pqe ? (float)acc[2] : 0.f;
  }
  if (hist) {
    hist[0] = loss;
    hist[1] = want_pqe ? (float)acc[2] : nanf("");
  }
}

// ------------------------------------------------------------------------------------------------
// pack: u = q + qmax, little-endian bit stream per row; one thread per output 32-bit word group
// ------------------------------------------------------------------------------------------------
__global__ void pack_kernel(const int8_t* __restrict__ codes, uint8_t* __restrict__ packed, int rows, int cols, int bits) {
  // one thread packs 8 consecutive codes into `bits` bytes
  const long long chunks_per_row = cols / 8;
  const long long n = (long long)rows * chunks_per_row;
  const int qmax = (1 << (bits - 1)) - 1;
  for (long long c = blockIdx.x * (long long)blockDim.x + threadIdx.x; c < n; c += (long long)gridDim.x * blockDim.x) {
    long long row = c / chunks_per_row, ch = c - row * chunks_per_row;
    const int8_t* src = codes + row * cols + ch * 8;
    unsigned long long v = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) v |= (unsigned long long)((unsigned)(src[i] + qmax) & ((1u << bits) - 1u)) << (bits * i);
    uint8_t* dst = packed + row * ((long long)cols * bits / 8) + ch * bits;
    for (int b = 0; b < bits; ++b) dst[b] = (uint8_t)(v >> (8 * b));
  }
}

// The inverse of pack_kernel followed by the dequantisation: out[row][c] = bf16(scale(row, c / g) * (field - qmax)),
// one thread per 8 consecutive codes (`bits` bytes of the stream); cols % 8 == 0, out row pitch ldo elements.
__global__ void __launch_bounds__(256) dequant_kernel(const uint8_t* __restrict__ packed, const float* __restrict__ scales,
                                                      uint16_t* __restrict__ out, int rows, int cols, int bits, int g, long long ldo) {
  const long long chunks_per_row = cols / 8;
  const long long n = (long long)rows * chunks_per_row;
  const int qmax = (1 << (bits - 1)) - 1;
  const unsigned mask = (1u << bits) - 1u;
  const int ng = cols / g;
  for (long long c = blockIdx.x * (long long)blockDim.x + threadIdx.x; c < n; c += (long long)gridDim.x * blockDim.x) {
    const long long row = c / chunks_per_row, ch = c - row * chunks_per_row;
    const uint8_t* src = packed + row * ((long long)cols * bits / 8) + ch * bits;
    unsigned long long v = 0;
    for (int b = 0; b < bits; ++b) v |= (unsigned long long)src[b] << (8 * b);
    uint16_t* dst = out + row * ldo + ch * 8;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int col = (int)ch * 8 + i;
      const float s = __ldg(scales + row * ng + col / g);
      const int q = (int)((v >> (bits * i)) & mask) - qmax;
      dst[i] = __bfloat16_as_ushort(__float2bfloat16_rn(s * (float)q));
    }
  }
}

__global__ void __launch_bounds__(256) f32_to_bf16_kernel(const float* __restrict__ in, uint16_t* __restrict__ out, long long n) {
  for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x)
    out[e] = __bfloat16_as_ushort(__float2bfloat16_rn(in[e]));
}

// The same stream, 32 codes per thread: 32 b-bit fields are exactly b 32-bit words, so a thread reads two 16-byte
// vectors of codes and writes whole words (cols % 32 == 0, codes 16-byte aligned, packed 4-byte aligned).
template <int BITS>
__global__ void __launch_bounds__(256) pack32_kernel(const int8_t* __restrict__ codes, uint32_t* __restrict__ packed, int rows,
                                                     int cols) {
  const long long chunks_per_row = cols / 32;
  const long long n = (long long)rows * chunks_per_row;
  constexpr int qmax = (1 << (BITS - 1)) - 1;
  constexpr uint32_t mask = (1u << BITS) - 1u;
  for (long long c = blockIdx.x * (long long)blockDim.x + threadIdx.x; c < n; c += (long long)gridDim.x * blockDim.x) {
    const uint4* src = reinterpret_cast<const uint4*>(codes) + 2 * c;  // rows are contiguous: chunk c starts at 32 c
    const uint4 q0 = __ldg(src), q1 = __ldg(src + 1);
    const uint32_t w8[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
    uint32_t out[BITS];
#pragma unroll
    for (int b = 0; b < BITS; ++b) out[b] = 0u;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      const int8_t q = (int8_t)((w8[i >> 2] >> (8 * (i & 3))) & 0xFFu);
      const uint32_t u = (uint32_t)(q + qmax) & mask;
      const int bit = BITS * i;  // compile-time after unrolling
      out[bit >> 5] |= u << (bit & 31);
      if ((bit & 31) + BITS > 32) out[(bit >> 5) + 1] |= u >> (32 - (bit & 31));
    }
    uint32_t* dst = packed + c * BITS;
#pragma unroll
    for (int b = 0; b < BITS; ++b) dst[b] = out[b];
  }
}

}  // namespace cafeq
