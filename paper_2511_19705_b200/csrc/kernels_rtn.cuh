// Plain round-to-nearest quantisation of a bf16 matrix (Eq. 1 in its symmetric absmax form, no transform) as one
// streaming kernel: every weight is read once (16-byte loads of 8 bf16) and one int8 code is written per weight,
// plus one fp32 scale per group -- 3 + 4/g bytes per weight, the algorithmic minimum for unpacked codes.
// A group of g = 8 * LANES consecutive weights is held by LANES neighbouring lanes; its absmax is a shuffle
// reduction over those lanes; s = absmax / qmax and code = rne(w / s) use IEEE fp32 division (these decide integers).
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
  const int ngr = cols / (8 * LANES);
  for (long long c = blockIdx.x * (long long)blockDim.x + threadIdx.x; c < nloop; c += stride) {
    const bool valid = c < nch;
    const long long row = valid ? c / cpr : 0;
    const int cc = valid ? (int)(c - row * cpr) : 0;
    uint4 q4 = make_uint4(0u, 0u, 0u, 0u);
    if (valid) q4 = __ldcs(reinterpret_cast<const uint4*>(W + row * ld) + cc);
    const uint32_t w4[4] = {q4.x, q4.y, q4.z, q4.w};
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
    uint32_t pk[2] = {0u, 0u};
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      float q = (s > 0.f) ? rintf(__fdiv_rn(v[e], s)) : 0.f;
      q = fminf(fmaxf(q, -qmax), qmax);
      pk[e >> 2] |= ((uint32_t)((int)q) & 0xFFu) << (8 * (e & 3));
    }
    if (valid) {
      __stcs(reinterpret_cast<uint2*>(codes + row * (long long)cols) + cc, make_uint2(pk[0], pk[1]));
      if ((cc % LANES) == 0) scales[row * ngr + cc / LANES] = s;
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
  if (blocks > 148 * 16) blocks = 148 * 16;
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
