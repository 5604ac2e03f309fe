// Plain round-to-nearest quantisation of a bf16 matrix (Eq. 1 in its symmetric absmax form, no transform) as one
// streaming kernel: every weight is read once (16-byte loads of 8 bf16) and one int8 code is written per weight,
// plus one fp32 scale per group -- 3 + 4/g bytes per weight, the algorithmic minimum for unpacked codes.
// A group of g = 8 * LANES consecutive weights is held by LANES neighbouring lanes; its absmax is a shuffle
// reduction over those lanes; s = absmax / qmax is an IEEE fp32 division and code = rne(fl32(w / s)): the quotient is
// first formed as w * (1 / s), which differs from the IEEE quotient by less than 2 ulp, so it rounds to the same
// integer unless it lies within (qmax + 1) * 1e-6 of a half-integer; only those (rare) chunks are redone with the
// division, which keeps every code identical to the division's while the kernel stays bandwidth-bound (eight IEEE
// divisions per chunk would make it ALU-bound).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace cafeq {

template <int LANES>
__global__ void __launch_bounds__(256) rtn_stream_kernel(const uint16_t* __restrict__ W, long long ld, int rows, int cols,
                                                         float qmax, int8_t* __restrict__ codes, float* __restrict__ scales) {
  const int cpr = cols / 8;                 // 8-weight chunks per row; a multiple of LANES
  const long long nch = (long long)rows * cpr;
  const long long stride = (long long)gridDim.x * blockDim.x;
  const long long nloop = (nch + 31) / 32 * 32;  // whole warps take part in the shuffles
  constexpr int UNR = 4;                    // chunks in flight per thread: their loads are issued before any is used
  for (long long c0 = blockIdx.x * (long long)blockDim.x + threadIdx.x; c0 < nloop; c0 += UNR * stride) {
    // codes and scales are dense, so chunk c writes codes at 8 c and (every LANES-th chunk) scale c / LANES; only the
    // weight address needs the row, and not even that when the rows are contiguous (no 64-bit division per chunk)
    uint4 q4[UNR];
    bool valid[UNR];
#pragma unroll
    for (int u = 0; u < UNR; ++u) {
      const long long c = c0 + u * stride;
      valid[u] = c < nch;
      q4[u] = make_uint4(0u, 0u, 0u, 0u);
      if (valid[u]) {
        long long woff = c;  // in 16-byte units
        if (ld != cols) {
          const long long r = c / cpr;
          woff = (r * ld) / 8 + (c - r * cpr);
        }
        q4[u] = __ldcs(reinterpret_cast<const uint4*>(W) + woff);
      }
    }
#pragma unroll
    for (int u = 0; u < UNR; ++u) {
      if (c0 + u * stride >= nloop) break;  // warp-uniform: nloop and the stride are multiples of 32
      const uint32_t w4[4] = {q4[u].x, q4[u].y, q4[u].z, q4[u].w};
      float v[8];
      float m = 0.f;
#pragma unroll
      for (int h = 0; h < 4; ++h) {
        v[2 * h] = __uint_as_float(w4[h] << 16);
        v[2 * h + 1] = __uint_as_float(w4[h] & 0xFFFF0000u);
        m = fmaxf(m, fmaxf(fabsf(v[2 * h]), fabsf(v[2 * h + 1])));
      }
#pragma unroll
      for (int o = LANES / 2; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      const float s = __fdiv_rn(m, qmax);
      const float rs = (s > 0.f) ? __frcp_rn(s) : 0.f;
      const float win = 0.5f - (qmax + 1.f) * 1.0e-6f;
      float qv[8];
      bool near_half = !(rs < 3.0e38f);  // a scale so small that its reciprocal overflows: take the division
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float x = v[e] * rs;
        qv[e] = rintf(x);
        near_half |= fabsf(x - qv[e]) > win;
      }
      if (near_half) {
#pragma unroll
        for (int e = 0; e < 8; ++e) qv[e] = (s > 0.f) ? rintf(__fdiv_rn(v[e], s)) : 0.f;
      }
      uint32_t pk[2] = {0u, 0u};
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float q = fminf(fmaxf(qv[e], -qmax), qmax);
        pk[e >> 2] |= ((uint32_t)((int)q) & 0xFFu) << (8 * (e & 3));
      }
      if (valid[u]) {
        const long long c = c0 + u * stride;
        __stcs(reinterpret_cast<uint2*>(codes) + c, make_uint2(pk[0], pk[1]));
        if ((c % LANES) == 0) scales[c / LANES] = s;
      }
    }
  }
}

// true when the streaming kernel covers the shape (then it has been launched)
static bool rtn_stream_launch(cudaStream_t st, const void* W, long long ld, int rows, int cols, int g, float qmax, int8_t* codes,
                              float* scales) {
  if (!(g == 32 || g == 64 || g == 128 || g == 256) || cols % g) return false;
  if (((uintptr_t)W & 15) || (ld % 8) || ((uintptr_t)codes & 7)) return false;
  const long long nch = (long long)rows * (cols / 8);
  long long blocks = (nch + 255) / 256;
  if (blocks > 148 * 8) blocks = 148 * 8;
  if (blocks < 1) blocks = 1;
  const uint16_t* w = (const uint16_t*)W;
  switch (g) {
    case 32: rtn_stream_kernel<4><<<(unsigned)blocks, 256, 0, st>>>(w, ld, rows, cols, qmax, codes, scales); break;
    case 64: rtn_stream_kernel<8><<<(unsigned)blocks, 256, 0, st>>>(w, ld, rows, cols, qmax, codes, scales); break;
    case 128: rtn_stream_kernel<16><<<(unsigned)blocks, 256, 0, st>>>(w, ld, rows, cols, qmax, codes, scales); break;
    default: rtn_stream_kernel<32><<<(unsigned)blocks, 256, 0, st>>>(w, ld, rows, cols, qmax, codes, scales); break;
  }
  return true;
}

}  // namespace cafeq
