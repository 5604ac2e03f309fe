// Dense-matrix helpers for the pairwise product term (Eq. 5) and Algorithm 1: bf16 split / transpose of
// rectangular fp32 matrices (the operand layouts of the tensor-core product kernel), replica fold / expansion
// of the inner dimension, and the small control kernels of the iterative pseudo-inverse.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "kernels_generic.cuh"

namespace cafeq {

// X fp32 [R, C] (row pitch ld) times `scale` (or times 1 / *inv_scale when inv_scale is given) ->
// bf16 hi / lo splits, row-major [R, C] and / or transposed [C, R]; optional fp32 copy Y of the scaled values
// (row-major) and YT (transposed, holding hi + lo: used only as a starting guess).  h3 / t3: optional third term
// bf16(x - hi - lo) in row-major / transposed order (hi + lo + third carries 24 significand bits: products over the
// three-way split reach fp32 accuracy).
// One 32 x 32 tile per CTA (grid: ceil(C/32), ceil(R/32); block 32 x 8).
__global__ void __launch_bounds__(256) split_rect_kernel(const float* __restrict__ X, int R, int C, long long ld, float scale,
                                                         const double* __restrict__ inv_scale, float* __restrict__ Y,
                                                         float* __restrict__ YT, uint16_t* __restrict__ hi, uint16_t* __restrict__ lo,
                                                         uint16_t* __restrict__ thi, uint16_t* __restrict__ tlo,
                                                         const int32_t* status, uint16_t* __restrict__ h3 = nullptr,
                                                         uint16_t* __restrict__ t3 = nullptr) {
  if (status && *status) return;
  __shared__ uint32_t tile[32][33];
  __shared__ uint16_t tile3[32][34];
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  const int tx = threadIdx.x, ty = threadIdx.y;
  float sc = scale;
  if (inv_scale) sc = (float)((double)scale / fmax(*inv_scale, 1e-300));
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int r = r0 + ty + 8 * q, c = c0 + tx;
    uint32_t packed = 0;
    if (r < R && c < C) {
      const float x = sc * X[(long long)r * ld + c];
      const __nv_bfloat16 h = __float2bfloat16_rn(x);
      const __nv_bfloat16 l = __float2bfloat16_rn(x - __bfloat162float(h));
      const uint16_t hb = __bfloat16_as_ushort(h), lb = __bfloat16_as_ushort(l);
      if (Y) Y[(long long)r * C + c] = x;
      if (hi) hi[(long long)r * C + c] = hb;
      if (lo) lo[(long long)r * C + c] = lb;
      packed = (uint32_t)hb | ((uint32_t)lb << 16);
      if (h3 || t3) {
        const uint16_t b3 = __bfloat16_as_ushort(__float2bfloat16_rn((x - __bfloat162float(h)) - __bfloat162float(l)));
        if (h3) h3[(long long)r * C + c] = b3;
        tile3[ty + 8 * q][tx] = b3;
      }
    }
    tile[ty + 8 * q][tx] = packed;
  }
  __syncthreads();
  if (t3) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int c = c0 + ty + 8 * q, r = r0 + tx;
      if (r < R && c < C) t3[(long long)c * R + r] = tile3[tx][ty + 8 * q];
    }
  }
  if (thi || tlo || YT) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int c = c0 + ty + 8 * q, r = r0 + tx;
      if (r < R && c < C) {
        const uint32_t v = tile[tx][ty + 8 * q];
        if (thi) thi[(long long)c * R + r] = (uint16_t)(v & 0xFFFFu);
        if (tlo) tlo[(long long)c * R + r] = (uint16_t)(v >> 16);
        if (YT) YT[(long long)c * R + r] = __uint_as_float(v << 16) + __uint_as_float(v & 0xFFFF0000u);
      }
    }
  }
}

// bf16 [R, C] (pitch ld) -> bf16 transposed [C, R]
__global__ void __launch_bounds__(256) transpose_bf16_kernel(const uint16_t* __restrict__ X, int R, int C, long long ld,
                                                             uint16_t* __restrict__ T) {
  __shared__ uint16_t tile[32][34];
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  const int tx = threadIdx.x, ty = threadIdx.y;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int r = r0 + ty + 8 * q, c = c0 + tx;
    tile[ty + 8 * q][tx] = (r < R && c < C) ? X[(long long)r * ld + c] : (uint16_t)0;
  }
  __syncthreads();
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int c = c0 + ty + 8 * q, r = r0 + tx;
    if (r < R && c < C) T[(long long)c * R + r] = tile[tx][ty + 8 * q];
  }
}

// Bf[B*k + j][y] = sum_rep V[y][(B*r + rep)*k + j]: fold the r replicas of every block of the inner dimension
// and transpose (V fp32 [d3, r*h] -> Bf fp32 [h, d3]).  grid: ceil(d3/32), h/32 (k % 32 == 0); block 32 x 8.
__global__ void __launch_bounds__(256) fold_transpose_kernel(const float* __restrict__ V, int d3, int h, int k, int r,
                                                             float* __restrict__ Bf) {
  __shared__ float tile[32][33];
  const int y0 = blockIdx.x * 32, l0 = blockIdx.y * 32;  // l0 inside one block of k
  const int tx = threadIdx.x, ty = threadIdx.y;
  const int B = l0 / k, j0 = l0 - B * k;
  const long long ldv = (long long)r * h;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int y = y0 + ty + 8 * q;
    float s = 0.f;
    if (y < d3)
      for (int rep = 0; rep < r; ++rep) s += V[(long long)y * ldv + (long long)(B * r + rep) * k + j0 + tx];
    tile[ty + 8 * q][tx] = s;
  }
  __syncthreads();
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int l = l0 + ty + 8 * q, y = y0 + tx;
    if (y < d3) Bf[(long long)l * d3 + y] = tile[tx][ty + 8 * q];
  }
}

// V[y][(B*r + rep)*k + j] = scale * X[y][B*k + j]  (X fp32 [d3, h] -> V fp32 [d3, r*h])
__global__ void expand_cols_kernel(const float* __restrict__ X, int d3, int h, int k, int r, float scale, float* __restrict__ V) {
  const long long n = (long long)d3 * r * h;
  const float inv = scale;
  for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
    const long long y = e / ((long long)r * h);
    const int l = (int)(e - y * (long long)r * h);
    const int Bq = l / k, j = l - Bq * k;
    V[e] = inv * X[y * h + (long long)(Bq / r) * k + j];
  }
}

// iteration control of the pseudo-inverse: keep running while the newest squared residual is above tol2 and
// still falling (a rank-deficient matrix stalls at its rank defect); flag: 1 = run, 0 = skip
__global__ void pinv_control_kernel(const double* __restrict__ sq, int it, double tol2, int* flag, int m, int32_t* status) {
  if (*flag == 0) return;
  const double cur = sq[it];
  if (!(cur > tol2)) { *flag = 0; return; }
  if (it >= 1) {
    const double prev = sq[it - 1];
    // With every eigenvalue of A X in (0, 2) the residual norm falls monotonically.  A residual that is still large
    // and grows means the starting scale was too small (the estimate of the largest singular value failed):
    // stop and say so instead of iterating to infinity.
    if (cur > 1.5 * prev && cur > 1e-2 * (double)m) {
      *flag = 0;
      raise_status(status, CAFEQ_ERR_NONFINITE);
      return;
    }
  }
  if (it >= 4) {
    const double prev = sq[it - 1];
    if (cur > prev * (1.0 - 1e-7) && cur < prev * (1.0 + 1e-7)) *flag = 0;  // stalled
  }
}

__global__ void set_int_kernel(int* p, int v) { *p = v; }

// gX[row][G*g + idx[row, G]] += coef[row, G]: the scale path of the straight-through quantiser lands on the
// arg-max entry of its group (records row-major)
__global__ void add_argmax_kernel(float* __restrict__ gX, long long ld, int rows, int ng, int g, const float* __restrict__ coef,
                                  const int* __restrict__ idx, const int32_t* status) {
  if (status && *status) return;
  const long long n = (long long)rows * ng;
  for (long long w = blockIdx.x * (long long)blockDim.x + threadIdx.x; w < n; w += (long long)gridDim.x * blockDim.x) {
    const long long row = w / ng;
    const int G = (int)(w - row * ng);
    gX[row * ld + (long long)G * g + idx[w]] += coef[w];
  }
}

// Scale path of the straight-through quantiser from the residual itself: with Uhat = s q and Delta = Uhat - U the
// derivative of Uhat with respect to the scale is q - U / s = Delta / s, and s = a / qmax, so the coefficient routed
// to the group's arg-max entry is sign(U at arg-max) / qmax * sum_e gDelta_e Delta_e / s = sign * sum_e gDelta_e Delta_e / a.
// Delta comes as a two-term bf16 split (row pitch ldd); records are group-major when gm is set.  One warp per record.
__global__ void ste_scale_coef_kernel(const float* __restrict__ gD, long long ldg, const uint16_t* __restrict__ Dh,
                                      const uint16_t* __restrict__ Dl, long long ldd, int rows, int ng, int g,
                                      const float* __restrict__ a, const float* __restrict__ usel, int gm,
                                      float* __restrict__ coef, const int32_t* status) {
  if (status && *status) return;
  const long long w = (blockIdx.x * (long long)blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (w >= (long long)rows * ng) return;
  // consecutive warps take consecutive groups of one row (the rows of gD and Delta are read contiguously)
  const int row = (int)(w / ng), G = (int)(w - (long long)row * ng);
  float sum = 0.f;
  for (int e = lane; e < g; e += 32) {
    const long long col = (long long)G * g + e;
    const float d = bf16_bits_to_float(Dh[row * ldd + col]) + bf16_bits_to_float(Dl[row * ldd + col]);
    sum = fmaf(gD[row * ldg + col], d, sum);
  }
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  if (lane == 0) {
    const long long pi = gm ? (long long)G * rows + row : w;
    const float av = a[pi], u = usel[pi];
    const float sgn = (u > 0.f) ? 1.f : ((u < 0.f) ? -1.f : 0.f);
    coef[pi] = (av > 0.f) ? sgn * sum / av : 0.f;
  }
}

// acc += sum x[i] y[i]  (fp32 products summed in double; one atomic per block)
__global__ void __launch_bounds__(256) dot_f32_kernel(const float* __restrict__ x, const float* __restrict__ y, long long n,
                                                      double* acc) {
  __shared__ double red[32];
  double s = 0.0;
  for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x)
    s += (double)(x[e] * y[e]);
  s = block_sum_double(s, red);
  if (threadIdx.x == 0 && s != 0.0) atomicAdd(acc, s);
}

// Power iteration for the largest singular value of S [R, C] (fp32, row-major), used to scale the starting guess
// of the pseudo-inverse iteration.  v [C], u [R] scratch; three small kernels per round:
//   u = S v (one warp per row);  v2 = S^T u (one thread per column), nrm += |v2|^2;  v = v2 / |v2|.
// After the last round *sig2 = safety * |S^T S v| (v of unit norm): a Rayleigh-type estimate from below of sigma_max^2.
__global__ void pw_init_kernel(float* __restrict__ v, int C, double* nrm) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j < C) {
    uint32_t h = (uint32_t)j * 2654435761u;
    h ^= h >> 15;
    v[j] = ((h & 1u) ? 1.f : -1.f) * rsqrtf((float)C);  // fixed +-1 pattern of unit norm
  }
  if (j == 0) *nrm = 0.0;
}
__global__ void pw_rows_kernel(const float* __restrict__ S, const float* __restrict__ v, int R, int C, float* __restrict__ u) {
  const long long w = (blockIdx.x * (long long)blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (w >= R) return;
  float s = 0.f;
  for (int j = lane; j < C; j += 32) s = fmaf(S[w * C + j], v[j], s);
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if (lane == 0) u[w] = s;
}
// grid: (ceil(C / 256), row slices); partial sums are added atomically into v2 (zeroed by the caller)
__global__ void pw_cols_kernel(const float* __restrict__ S, const float* __restrict__ u, int R, int C, int rows_per_slice,
                               float* __restrict__ v2) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= C) return;
  const int r0 = blockIdx.y * rows_per_slice, r1 = min(R, r0 + rows_per_slice);
  float s = 0.f;
  for (int r = r0; r < r1; ++r) s = fmaf(S[(long long)r * C + j], u[r], s);
  atomicAdd(&v2[j], s);
}
__global__ void pw_norm_kernel(const float* __restrict__ v2, int C, double* nrm) {
  __shared__ double red[32];
  double s = 0.0;
  for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < C; j += gridDim.x * blockDim.x) s += (double)v2[j] * (double)v2[j];
  s = block_sum_double(s, red);
  if (threadIdx.x == 0) atomicAdd(nrm, s);
}
// v = v2 / |v2|, v2 = 0, and (last round) *sig2 = safety * |v2| bounded below by floor2; nrm is cleared for the next round
__global__ void pw_scale_kernel(float* __restrict__ v, float* __restrict__ v2, int C, double* nrm_in, double* nrm_next,
                                double* sig2, double safety, const double* fro2) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  const double n = sqrt(fmax(*nrm_in, 0.0));
  if (j < C) {
    v[j] = (n > 0.0) ? (float)((double)v2[j] / n) : v[j];
    v2[j] = 0.f;
  }
  if (j == 0) {
    *nrm_next = 0.0;
    if (sig2) {
      // never above the Frobenius bound (always safe), never below 1 / rank-ish of it (a failed estimate)
      double e = safety * n;
      const double f = *fro2;
      if (!(e > 0.0) || e > f) e = f;
      *sig2 = e;
    }
  }
}

__global__ void sqrt_hist_kernel(const double* __restrict__ sq, float* __restrict__ out, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = (float)sqrt(fmax(sq[i], 0.0));
}

}  // namespace cafeq
