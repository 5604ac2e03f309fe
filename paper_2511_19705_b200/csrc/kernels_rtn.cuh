// Plain round-to-nearest quantisation of a bf16 matrix (Eq. 1 in its symmetric absmax form, no transform) as one
// streaming kernel: every weight is read once (16-byte loads of 8 bf16) and one int8 code is written per weight,
// plus one fp32 scale per group -- 3 + 4/g bytes per weight, the algorithmic minimum for unpacked codes.
// A group of g = 32 * LG consecutive weights is held by LG neighbouring lanes, 32 weights each; its absmax is a
// shuffle reduction over those lanes; s = absmax / qmax is an IEEE fp32 division and code = rne(fl32(w / s)): the
// quotient is first formed as w * (1 / s), which differs from the IEEE quotient by less than 2 ulp, so it rounds to
// the same integer unless it lies within (qmax + 1) * 1e-6 of a half-integer; only those elements are redone with the
// division, which keeps every code identical to the division's.  The kernel was bound by
// instruction issue, not by memory (66 % of the issue slots at 25 % of the DRAM rate): the rounding therefore uses
// no conversion instruction, and the division is paid once per 32 weights.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace cafeq {

// LG = lanes per group = g / 32: every thread holds 32 weights of ONE group (four 16-byte chunks), so the scale's
// division and reciprocal are paid once per 32 weights.  Within a warp's 2 KB span lane l works on group l / LG and
// its u-th chunk is the group's chunk u * LG + l % LG: a load instruction of the warp covers whole 64-byte pieces.
template <int LG>
__global__ void __launch_bounds__(256) rtn_stream_kernel(const uint16_t* __restrict__ W, long long ld, int rows, int cols,
                                                         float qmax, int8_t* __restrict__ codes, float* __restrict__ scales) {
  constexpr int UPG = 4 * LG;               // 16-byte chunks per group
  const int cpr = cols / 8;                 // chunks per row; a multiple of UPG
  const long long nch = (long long)rows * cpr;
  const int lane = threadIdx.x & 31;
  const long long warp0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarp = ((long long)gridDim.x * blockDim.x) >> 5;
  const long long nspan = (nch + 127) / 128;  // 128 chunks (2 KB) per warp iteration
  const int gl = lane / LG, j = lane % LG;
  const float win = 0.5f - (qmax + 1.f) * 1.0e-6f;
  for (long long sp = warp0; sp < nspan; sp += nwarp) {
    const long long gbase = sp * 128 + (long long)gl * UPG;  // first chunk of this lane's group
    const bool valid = gbase < nch;                           // groups are whole: all of it or nothing
    uint4 q4[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      q4[u] = make_uint4(0u, 0u, 0u, 0u);
      if (valid) {
        const long long c = gbase + u * LG + j;
        long long woff = c;  // in 16-byte units
        if (ld != cols) {
          const long long r = c / cpr;
          woff = (r * ld) / 8 + (c - r * cpr);
        }
        q4[u] = __ldcs(reinterpret_cast<const uint4*>(W) + woff);
      }
    }
    // Group maximum on the bit patterns: |bf16| as an integer orders like the magnitude, and the integer maximum runs
    // on the full-rate integer lanes (the fp32 min / max instruction does not: it kept a quarter-rate pipe 65 % busy).
    float v[32];
    uint32_t mb = 0u;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint32_t w4[4] = {q4[u].x, q4[u].y, q4[u].z, q4[u].w};
#pragma unroll
      for (int h = 0; h < 4; ++h) {
        const uint32_t lo = w4[h] << 16, hi = w4[h] & 0xFFFF0000u;
        v[8 * u + 2 * h] = __uint_as_float(lo);
        v[8 * u + 2 * h + 1] = __uint_as_float(hi);
        mb = max(mb, max(lo & 0x7FFFFFFFu, hi & 0x7FFFFFFFu));
      }
    }
#pragma unroll
    for (int o = LG / 2; o > 0; o >>= 1) mb = max(mb, __shfl_xor_sync(0xffffffffu, mb, o));
    // (a NaN's pattern exceeds infinity's, so a group holding one has a NaN maximum and takes the exact path below)
    const float m = __uint_as_float(mb);
    const float s = __fdiv_rn(m, qmax);
    const float rs = (s > 0.f) ? __frcp_rn(s) : 0.f;
    // Fast path, no conversion instruction: t = x + 1.5 * 2^23 holds rne(x) in its low mantissa bits (the fp32 add
    // rounds to nearest even, exactly as rintf), and since 1.5 * 2^23 = 0x4B400000 has a zero low byte, the low
    // byte of t's bit pattern IS the two's-complement code.  |x| <= qmax (1 + 3 * 2^-23) < qmax + 1/2 whenever the
    // group maximum is finite, so no clamp is needed here.
    constexpr float MAGIC = 12582912.f;
    // An element whose quotient lies within the window of a half-integer takes the IEEE division, one element at a
    // time: weights on the bf16 grid hit exact halves of the group maximum often (about 0.2 % of all elements at
    // qmax = 3), so redoing a whole thread's 32 elements whenever one of them does made most warps run the slow path
    // with one or two lanes active.  all_exact: a scale whose reciprocal overflows or a non-finite maximum.
    const bool all_exact = !(rs < 3.0e38f) || !(m < 3.0e38f);
    const uint32_t winb = __float_as_uint(win);
    uint32_t pk[8];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      uint32_t tb[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float ve = v[8 * u + e];
        const float x = ve * rs;
        const float t = x + MAGIC;
        tb[e] = __float_as_uint(t);
        if (((__float_as_uint(x - (t - MAGIC)) & 0x7FFFFFFFu) > winb) || all_exact) {
          float q = (s > 0.f) ? rintf(__fdiv_rn(ve, s)) : 0.f;
          q = fminf(fmaxf(q, -qmax), qmax);
          tb[e] = (uint32_t)((int)q);
        }
      }
      pk[2 * u] = __byte_perm(__byte_perm(tb[0], tb[1], 0x0040), __byte_perm(tb[2], tb[3], 0x0040), 0x5410);
      pk[2 * u + 1] = __byte_perm(__byte_perm(tb[4], tb[5], 0x0040), __byte_perm(tb[6], tb[7], 0x0040), 0x5410);
    }
    if (valid) {
#pragma unroll
      for (int u = 0; u < 4; ++u) __stcs(reinterpret_cast<uint2*>(codes) + gbase + u * LG + j, make_uint2(pk[2 * u], pk[2 * u + 1]));
      if (j == 0) scales[gbase / UPG] = s;
    }
  }
}

// true when the streaming kernel covers the shape (then it has been launched)
static bool rtn_stream_launch(cudaStream_t st, const void* W, long long ld, int rows, int cols, int g, float qmax, int8_t* codes,
                              float* scales) {
  if (!(g == 32 || g == 64 || g == 128 || g == 256) || cols % g) return false;
  if (((uintptr_t)W & 15) || (ld % 8) || ((uintptr_t)codes & 7)) return false;
  const long long nch = (long long)rows * (cols / 8);
  long long blocks = (nch / 4 + 255) / 256;  // a thread takes four chunks
  if (blocks > 148 * 8) blocks = 148 * 8;
  if (blocks < 1) blocks = 1;
  const uint16_t* w = (const uint16_t*)W;
  switch (g) {
    case 32: rtn_stream_kernel<1><<<(unsigned)blocks, 256, 0, st>>>(w, ld, rows, cols, qmax, codes, scales); break;
    case 64: rtn_stream_kernel<2><<<(unsigned)blocks, 256, 0, st>>>(w, ld, rows, cols, qmax, codes, scales); break;
    case 128: rtn_stream_kernel<4><<<(unsigned)blocks, 256, 0, st>>>(w, ld, rows, cols, qmax, codes, scales); break;
    default: rtn_stream_kernel<8><<<(unsigned)blocks, 256, 0, st>>>(w, ld, rows, cols, qmax, codes, scales); break;
  }
  return true;
}

}  // namespace cafeq
