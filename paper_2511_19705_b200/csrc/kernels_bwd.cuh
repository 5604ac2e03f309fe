// Sparse backward of the transform pass on the tensor cores (tcgen05, sm_100a).
//
// Every (row, group) record of the forward pass carries a coefficient (dLoss / d group maximum, signed) and the
// position of the group's arg-max entry.  The gradient with respect to an operator block is a sum of outer
// products routed through those entries (Section 4.1: the group maximum is the only path from the transform
// to Eq. 4; App. D: the same for the LogSumExp surrogate):
//   input axis : gradT[B][i][j] = sum_o S[o][i] W[o, B k + j],   S[o][i] = coef(o, G) where i is the arg-max column of (o, G)
//   output axis: gradT[B][i][j] = sum_c S[i][c] W[B k + j, c],   S[i][c] = coef(B k + i, G(c)) where c is its arg-max column
// i.e. a dense k x k product whose left operand has one non-zero per (row, group).  The kernel streams the weight
// tiles once with TMA, writes the few non-zeros of S as a two-term bf16 split (hi + lo: fp32-grade coefficients)
// straight into shared memory in the swizzled operand layout, and accumulates the block gradient in tensor
// memory over all tiles of the block that the CTA owns; one flush per block and CTA adds it to global memory.
// The product is issued in the orientation (S^T W or W^T S) whose accumulator rows run along the fastest index of
// the requested output layout, so that the flush is coalesced atomic adds straight from registers.
//
// F16 form: when the caller holds an fp16 copy of the weights (W * 2^e, exact for every bf16 value that matters:
// fp16 keeps 11 significand bits against bf16's 8) the coefficients are written as ONE fp16 term (relative error
// 2^-12, scaled by a power of two so that the largest lands near 2^14) and the product is issued once instead of
// twice; the flush undoes both power-of-two scales.
//
// Several matrices can share one launch (see BwMulti): the tiles of all sub-problems form one list and every
// persistent CTA takes a contiguous run of it.
#pragma once

#include <cuda_fp16.h>

#include "kernels_fused.cuh"

namespace cafeq {

struct BwParams {
  int d_out, d_in;
  int g, ng;           // group width, groups per row
  int r;               // matrix blocks per operator block
  int n_major;         // blocks (input axis: column blocks; output axis: row blocks)
  int n_minor;         // tiles per block (input axis: 64-row tiles; output axis: 64-column tiles)
  int NG;              // input axis: groups of one row examined per block, max(1, k / g)
  int gm;              // records are group-major (index = group * d_out + row) instead of row-major
  int transpose_out;   // store gradT[..][j][i]
  const float* coef;
  const int* idx;
  float* gradT;        // [n_major / r, k, k], accumulated with atomic adds (caller zeroes it)
  const float* coefmax;      // F16 form: device word holding max |coef| of this matrix (sets the coefficient scale)
  const float* w_inv_scale;  // F16 form: device word holding 2^-e of the fp16 weight copy
  const double* out_div;     // optional device word: the flushed gradient is divided by it (LogSumExp normaliser)
  int32_t* status;
};

constexpr int BW_MAX_SUB = 8;
struct BwMaps {
  CUtensorMap w[BW_MAX_SUB];
};
struct BwMulti {
  int n;
  int tile_end[BW_MAX_SUB];
  BwParams p[BW_MAX_SUB];  // all share one status word
};

enum { BW_IN = 0, BW_OUT = 1 };
constexpr int BW_THREADS = 320;  // warp 0: TMA, warp 1: MMA, warps 2-9: operand builders and flush
constexpr int BW_NSTAGE = 3;
constexpr uint32_t BW_NONE = 0xFFFFFFFFu;

template <int K, int F16>
struct BwCfg {
  static constexpr int HALVES = K / 128;
  static constexpr int TERMS = F16 ? 1 : 2;
  static constexpr int NSTAGE = F16 ? 4 : BW_NSTAGE;
  static constexpr int STAGE_BYTES = K * 64 * 2;   // weight tile: 64 contraction entries x K
  static constexpr int S_TERM_BYTES = K * 64 * 2;  // S tile: K targets x 64 contraction entries, K-major, one 16-bit term
  static constexpr int S_BUF_BYTES = TERMS * S_TERM_BYTES;
  static constexpr int TMEM_COLS = HALVES * K;     // 128 or 512
  static constexpr int SMEM = 1024 + NSTAGE * STAGE_BYTES + 2 * S_BUF_BYTES + 256;
};

// instruction descriptor for fp16 operands (format field 0), fp32 accumulation
__host__ __device__ constexpr uint32_t umma_idesc_f16(int M, int N, int a_mn_major, int b_mn_major) {
  return (1u << 4) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(M >> 4) << 24);
}

// power of two that brings max |coef| just below 2^14 (fp16 holds up to 65504); 1 when there is nothing to scale
__device__ __forceinline__ float bw_coef_scale(const float* coefmax) {
  const float m = coefmax ? __ldg(coefmax) : 0.f;
  if (!(m > 0.f) || !(m < 3.0e38f)) return 1.f;
  int e;
  frexpf(m, &e);  // m = f * 2^e, f in [0.5, 1)
  int sh = 14 - e;
  if (sh > 120) sh = 120;
  if (sh < -120) sh = -120;
  return exp2f((float)sh);
}

__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// byte offset of S[target][kk] inside one term of the S tile (128-byte rows, 16-byte chunks XOR-swizzled by the
// row index modulo 8, 128-target halves 16 KB apart)
__device__ __forceinline__ uint32_t bw_s_offset(int target, int kk) {
  const int half = target >> 7, il = target & 127;
  return (uint32_t)(half * 16384 + (il >> 3) * 1024 + (il & 7) * 128 + ((((kk >> 3) ^ (il & 7)) & 7) << 4) + (kk & 7) * 2);
}

// SWAP = 0: accumulator rows = targets i, columns = j (coalesced when the output is stored transposed);
// SWAP = 1: rows = j, columns = i (coalesced for the plain layout).
template <int FORM, int K, int SWAP, int F16>
__device__ __forceinline__ void bd_bwd_body(const BwMaps& maps, const BwMulti& mp, const int cta, const int ncta) {
  using C = BwCfg<K, F16>;
  static_assert(K == 128 || K == 256, "block size");
  int32_t* const status = mp.p[0].status;
  if (status && *status) return;
  const int total_tiles = mp.tile_end[mp.n - 1];
  const int t_begin = (int)(((long long)cta * total_tiles) / ncta);
  const int t_end = (int)(((long long)(cta + 1) * total_tiles) / ncta);
  if (t_begin >= t_end) return;
  int s_first = 0;
  while (mp.tile_end[s_first] <= t_begin) ++s_first;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sStage = smem;
  uint8_t* sS = smem + C::NSTAGE * C::STAGE_BYTES;
  uint64_t* bars = (uint64_t*)(sS + 2 * C::S_BUF_BYTES);
  // barrier slots: wfull[NSTAGE], wempty[NSTAGE], sfull[2], sempty[2], accf, acce
  const uint32_t bar_wfull = smem_u32(bars);
  const uint32_t bar_wempty = bar_wfull + 8 * C::NSTAGE;
  const uint32_t bar_sfull = bar_wempty + 8 * C::NSTAGE;
  const uint32_t bar_sempty = bar_sfull + 16;
  const uint32_t bar_accf = bar_sempty + 16;
  const uint32_t bar_acce = bar_accf + 8;
  uint32_t* tmem_slot = (uint32_t*)(bars + 2 * C::NSTAGE + 6);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    tma_prefetch_desc(&maps.w[s_first]);
    for (int s = 0; s < C::NSTAGE; ++s) {
      mbar_init(bar_wfull + 8 * s, 1);
      mbar_init(bar_wempty + 8 * s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_sfull + 8 * b, 256);
      mbar_init(bar_sempty + 8 * b, 1);
    }
    mbar_init(bar_accf, 1);
    mbar_init(bar_acce, 256);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // the S tiles start as zeros; afterwards the builders clear exactly what they wrote
  {
    uint4* z = reinterpret_cast<uint4*>(sS);
    for (int e = threadIdx.x; e < 2 * C::S_BUF_BYTES / 16; e += BW_THREADS) z[e] = make_uint4(0u, 0u, 0u, 0u);
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"((uint32_t)C::TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer: one weight tile per stage
    if (lane == 0) {
      uint32_t it = 0;
      int sub = s_first;
      for (int gt = t_begin; gt < t_end; ++gt, ++it) {
        while (gt >= mp.tile_end[sub]) ++sub;
        const int tile = gt - (sub ? mp.tile_end[sub - 1] : 0);
        const int n_minor = mp.p[sub].n_minor;
        const CUtensorMap* tmW = &maps.w[sub];
        const int major = tile / n_minor, t = tile - major * n_minor;
        const uint32_t s = it % C::NSTAGE, ph = (it / C::NSTAGE) & 1u;
        if (!mbar_wait(bar_wempty + 8 * s, ph ^ 1u, abort_flag, status)) break;
        mbar_expect_tx(bar_wfull + 8 * s, C::STAGE_BYTES);
        const uint32_t dst = smem_u32(sStage + s * C::STAGE_BYTES);
        if constexpr (FORM == BW_IN) {
          // 64 rows x K columns as K / 64 boxes of 64 x 64 (one swizzle atom of the MN-major operand each)
          for (int n = 0; n < K / 64; ++n) tma_load_2d(dst + n * 8192, tmW, major * K + n * 64, t * 64, bar_wfull + 8 * s);
        } else {
          // K rows x 64 columns: one box, K-major operand
          tma_load_2d(dst, tmW, t * 64, major * K, bar_wfull + 8 * s);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      // the weight tile is MN-major on the input axis (contraction over its rows), K-major on the output axis
      constexpr int WMN = (FORM == BW_IN) ? 1 : 0;
      constexpr uint32_t idesc = F16 ? (SWAP ? umma_idesc_f16(128, K, WMN, 0) : umma_idesc_f16(128, K, 0, WMN))
                                     : (SWAP ? umma_idesc_bf16(128, K, WMN, 0) : umma_idesc_bf16(128, K, 0, WMN));
      const uint32_t sSt_u = smem_u32(sStage), sS_u = smem_u32(sS);
      int cur_id = -1, sub = s_first;
      uint32_t run = 0, it = 0;
      bool ok = true;
      for (int gt = t_begin; gt < t_end && ok; ++gt, ++it) {
        while (gt >= mp.tile_end[sub]) ++sub;
        const int tile = gt - (sub ? mp.tile_end[sub - 1] : 0);
        const int n_minor = mp.p[sub].n_minor;
        const int id = (sub << 24) | (tile / n_minor);
        const bool first = (id != cur_id);
        if (first) {
          // the flush of the previous block must have drained the accumulators
          if (cur_id >= 0) {
            if (!mbar_wait(bar_acce, (run - 1) & 1u, abort_flag, status)) { ok = false; break; }
            tc_fence_after();
          }
          cur_id = id;
        }
        const uint32_t s = it % C::NSTAGE, ph = (it / C::NSTAGE) & 1u;
        const uint32_t b = it & 1u, sph = (it >> 1) & 1u;
        if (!mbar_wait(bar_wfull + 8 * s, ph, abort_flag, status)) { ok = false; break; }
        if (!mbar_wait(bar_sfull + 8 * b, sph, abort_flag, status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t stage = sSt_u + s * C::STAGE_BYTES;
#pragma unroll
        for (int term = 0; term < C::TERMS; ++term) {
          const uint32_t sterm = sS_u + b * C::S_BUF_BYTES + term * C::S_TERM_BYTES;
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) {
            const uint32_t acc = (first && term == 0 && ks == 0) ? 0u : 1u;
#pragma unroll
            for (int h = 0; h < C::HALVES; ++h) {
              uint64_t ad, bd;
              if constexpr (SWAP == 0) {
                ad = umma_desc_sw128(sterm + h * 16384 + ks * 32);
                bd = (FORM == BW_IN) ? umma_desc_sw128_lbo(stage + ks * 2048, 8192) : umma_desc_sw128(stage + ks * 32);
              } else {
                // half h of the weight tile: 128 of its K columns (two swizzle atoms) or 128 of its K rows
                ad = (FORM == BW_IN) ? umma_desc_sw128_lbo(stage + h * 16384 + ks * 2048, 8192)
                                     : umma_desc_sw128(stage + h * 16384 + ks * 32);
                bd = umma_desc_sw128(sterm + ks * 32);
              }
              tc_mma_bf16(tmem_base + h * K, ad, bd, idesc, acc);
            }
          }
        }
        tc_commit(bar_wempty + 8 * s);
        tc_commit(bar_sempty + 8 * b);
        // last tile of this block in this CTA's run: hand the accumulators to the flush
        bool last = (gt + 1 == t_end) || (gt + 1 >= mp.tile_end[sub]);
        if (!last) last = ((tile + 1) / n_minor != tile / n_minor);
        if (last) {
          tc_commit(bar_accf);
          ++run;
        }
      }
    }
  } else {
    // ---------------------------------------------------------------- operand builders (one record per thread and tile) and flush
    const int bt = threadIdx.x - 64;
    const int q = warp & 3, hw = (warp - 2) >> 2;
    // The record of the NEXT tile is requested one tile ahead and only its raw words are kept: nothing may depend on
    // them before the next iteration, or the thread would sit out the whole memory latency here, once per tile.
    float rawC = 0.f;     // coefficient word
    int rawI = 0;         // arg-max word
    int rawBase = -1;     // input axis: column offset of this thread's group inside the block; output axis: first
                          // column of the group minus the tile's first column; -1: no record for this thread
    int rawKK = 0;        // input axis: contraction index (row inside the tile); output axis: target row
    float rawScale = 1.f;
    auto load_rec = [&](int sub, int tile) {
      const BwParams& p = mp.p[sub];
      const int major = tile / p.n_minor, t = tile - major * p.n_minor;
      rawBase = -1;
      rawC = 0.f;
      rawI = 0;
      if constexpr (FORM == BW_IN) {
        const int rl = bt & 63, qq = bt >> 6;
        const int row = t * 64 + rl;
        const int G0 = (major * K) / p.g;
        const int G = G0 + qq;
        if (qq < p.NG && row < p.d_out && G < p.ng) {
          const long long pi = p.gm ? (long long)G * p.d_out + row : (long long)row * p.ng + G;
          rawC = __ldg(p.coef + pi);
          rawI = __ldg(p.idx + pi);
          rawBase = qq * p.g + (G0 * p.g - major * K) + (1 << 20);  // kept non-negative: the offset can be below zero
          rawKK = rl;
        }
      } else {
        if (bt < K) {
          const int row = major * K + bt;
          const int G = (t * 64) / p.g;
          const long long pi = p.gm ? (long long)G * p.d_out + row : (long long)row * p.ng + G;
          rawC = __ldg(p.coef + pi);
          rawI = __ldg(p.idx + pi);
          rawBase = G * p.g - t * 64 + (1 << 20);
          rawKK = bt;
        }
      }
      if constexpr (F16) rawScale = bw_coef_scale(p.coefmax);
    };
    // the record requested one iteration ago, decoded: coefficient, target row, contraction index (tg < 0: none)
    auto take_rec = [&](float& cf, int& tg, int& kk) {
      cf = 0.f;
      tg = -1;
      kk = 0;
      if (rawBase >= 0) {
        const int col = rawBase - (1 << 20) + rawI;
        if constexpr (FORM == BW_IN) {
          if (rawC != 0.f && (unsigned)col < (unsigned)K) { cf = rawC; tg = col; kk = rawKK; }
        } else {
          if (rawC != 0.f && (unsigned)col < 64u) { cf = rawC; tg = rawKK; kk = col; }
        }
      }
      if constexpr (F16) cf *= rawScale;
    };
    // flush of one block: accumulators -> global memory, coalesced atomic adds straight from the registers
    // (accumulator row m = this thread's lane, 32 consecutive columns n per load)
    auto flush = [&](int sub, int major, uint32_t run) -> bool {
      const BwParams& p = mp.p[sub];
      bool okw = mbar_wait(bar_accf, run & 1u, abort_flag, status);
      okw = __all_sync(0xffffffffu, okw);
      if (!okw) return false;
      tc_fence_after();
      float mul = 1.f;
      if constexpr (F16) mul = (p.w_inv_scale ? __ldg(p.w_inv_scale) : 1.f) / bw_coef_scale(p.coefmax);
      if (p.out_div) mul = (float)((double)mul / *p.out_div);
      float* out = p.gradT + (size_t)(major / p.r) * K * K;
      constexpr int CH = (K == 256) ? 8 : 2;  // 32-column chunks per thread
      const int m = ((K == 256) ? hw * 128 : 0) + q * 32 + lane;
      const int nbase = (K == 256) ? 0 : hw * 64;
      const uint32_t tcol = (K == 256) ? (uint32_t)(hw * K) : (uint32_t)(hw * 64);
      for (int ch = 0; ch < CH; ++ch) {
        float v[32];
        tc_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + tcol + ch * 32, v);
        const int n0 = nbase + ch * 32;
#pragma unroll
        for (int c = 0; c < 32; ++c)
          if (v[c] != 0.f) atomicAdd(&out[(size_t)(n0 + c) * K + m], v[c] * mul);
      }
      tc_fence_before();
      mbar_arrive(bar_acce);
      return true;
    };

    uint32_t prevA = BW_NONE, prevB = BW_NONE;  // offsets this thread wrote into S buffer 0 / 1
    int sub = s_first;
    int cur_sub = s_first, cur_major = (t_begin - (s_first ? mp.tile_end[s_first - 1] : 0)) / mp.p[s_first].n_minor;
    uint32_t run = 0, tl = 0;
    bool ok = true;
    load_rec(sub, t_begin - (sub ? mp.tile_end[sub - 1] : 0));
    for (int gt = t_begin; gt < t_end && ok; ++gt, ++tl) {
      while (gt >= mp.tile_end[sub]) ++sub;
      const int tile = gt - (sub ? mp.tile_end[sub - 1] : 0);
      const int major = tile / mp.p[sub].n_minor;
      float cf;
      int tg, kk;
      take_rec(cf, tg, kk);
      if (gt + 1 < t_end) {
        int sn = sub;
        while (gt + 1 >= mp.tile_end[sn]) ++sn;
        load_rec(sn, gt + 1 - (sn ? mp.tile_end[sn - 1] : 0));
      }
      const uint32_t b = tl & 1u, sph = (tl >> 1) & 1u;
      if (major != cur_major || sub != cur_sub) {
        if (!flush(cur_sub, cur_major, run)) { ok = false; break; }
        ++run;
        cur_major = major;
        cur_sub = sub;
      }
      ok = mbar_wait(bar_sempty + 8 * b, sph ^ 1u, abort_flag, status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      uint8_t* buf = sS + b * C::S_BUF_BYTES;
      const uint32_t prev = b ? prevB : prevA;
      if (prev != BW_NONE) {
        *reinterpret_cast<uint16_t*>(buf + prev) = 0;
        if constexpr (!F16) *reinterpret_cast<uint16_t*>(buf + C::S_TERM_BYTES + prev) = 0;
      }
      uint32_t now = BW_NONE;
      if (tg >= 0) {
        now = bw_s_offset(tg, kk);
        if constexpr (F16) {
          *reinterpret_cast<uint16_t*>(buf + now) = __half_as_ushort(__float2half_rn(cf));
        } else {
          const __nv_bfloat16 hi = __float2bfloat16_rn(cf);
          const __nv_bfloat16 lo = __float2bfloat16_rn(cf - __bfloat162float(hi));
          *reinterpret_cast<uint16_t*>(buf + now) = __bfloat16_as_ushort(hi);
          *reinterpret_cast<uint16_t*>(buf + C::S_TERM_BYTES + now) = __bfloat16_as_ushort(lo);
        }
      }
      if (b) prevB = now; else prevA = now;
      fence_proxy_async_smem();
      mbar_arrive(bar_sfull + 8 * b);
    }
    if (ok) flush(cur_sub, cur_major, run);
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::TMEM_COLS) : "memory");
  }
}

template <int FORM, int K, int SWAP, int F16>
__global__ void __launch_bounds__(BW_THREADS, 1) bd_bwd_kernel(const __grid_constant__ BwMaps maps, const __grid_constant__ BwMulti mp) {
  bd_bwd_body<FORM, K, SWAP, F16>(maps, mp, (int)blockIdx.x, (int)gridDim.x);
}

// Input-axis and output-axis matrices in one launch (fp16 single-term form): the first n_in CTAs run the input-axis
// list, the others the output-axis list.
template <int K, int SWAP_IN, int SWAP_OUT>
__global__ void __launch_bounds__(BW_THREADS, 1)
bd_bwd_dual_kernel(const __grid_constant__ BwMaps maps_in, const __grid_constant__ BwMulti mp_in,
                   const __grid_constant__ BwMaps maps_out, const __grid_constant__ BwMulti mp_out, const int n_in) {
  if ((int)blockIdx.x < n_in) bd_bwd_body<BW_IN, K, SWAP_IN, 1>(maps_in, mp_in, (int)blockIdx.x, n_in);
  else bd_bwd_body<BW_OUT, K, SWAP_OUT, 1>(maps_out, mp_out, (int)blockIdx.x - n_in, (int)gridDim.x - n_in);
}

// host side ------------------------------------------------------------------------------------------------
static bool bw_supported(int axis_in, int d_out, int d_in, long long ld, int k, int g, const void* W) {
  if (!(k == 128 || k == 256)) return false;
  if ((ld % 8) || ((uintptr_t)W & 15)) return false;
  if (axis_in) {
    if (d_in % k) return false;
    if (!(k % g == 0 || g % k == 0)) return false;
    if (k / g > 4) return false;
  } else {
    if (d_out % k || d_in % 64 || g % 64 || d_in % g) return false;
  }
  return true;
}

static std::atomic<int> g_bw_min_tiles{6};  // tiles per CTA at least (more when problems overlap: see cafeq_set_overlap_mode)

static void bw_fill_tiles(BwParams& p, int axis_in, int k) {
  if (axis_in) {
    p.n_major = p.d_in / k;
    p.n_minor = (p.d_out + 63) / 64;
    p.NG = (k >= p.g) ? k / p.g : 1;
  } else {
    p.n_major = p.d_out / k;
    p.n_minor = p.d_in / 64;
    p.NG = 1;
  }
}

template <int FORM, int K, int SWAP, int F16>
static int bw_launch_t(cudaStream_t st, const BwMaps& maps, BwMulti mp, int min_tiles) {
  using C = BwCfg<K, F16>;
  static std::atomic<unsigned long long> done{0};
  if (!opt_in_smem(bd_bwd_kernel<FORM, K, SWAP, F16>, C::SMEM, done)) return CAFEQ_ERR_CUDA;
  // one persistent CTA per SM at most; small problems use fewer CTAs so that every CTA has several tiles per
  // flush (a flush moves k * k floats whatever the number of tiles behind it)
  long long total = 0, majors = 0;
  for (int s = 0; s < mp.n; ++s) {
    bw_fill_tiles(mp.p[s], FORM == BW_IN, K);
    total += (long long)mp.p[s].n_major * mp.p[s].n_minor;
    majors += mp.p[s].n_major;
    mp.tile_end[s] = (int)total;
  }
  for (int s = mp.n; s < BW_MAX_SUB; ++s) mp.tile_end[s] = (int)total;
  long long want = total / (min_tiles > 0 ? min_tiles : 1);
  if (want < majors) want = majors;
  if (want > total) want = total;
  const int grid = want < 148 ? (int)want : 148;
  bd_bwd_kernel<FORM, K, SWAP, F16><<<grid, BW_THREADS, C::SMEM, st>>>(maps, mp);
  return CAFEQ_OK;
}

static int bw_dispatch(cudaStream_t st, int axis_in, int k, int swap, int f16, const BwMaps& maps, const BwMulti& mp, int min_tiles) {
#define BW_CASE(AX, F, KK, SW, HF) \
  if ((axis_in != 0) == (AX) && k == KK && swap == SW && f16 == HF) return bw_launch_t<F, KK, SW, HF>(st, maps, mp, min_tiles);
  BW_CASE(true, BW_IN, 128, 0, 0)
  BW_CASE(true, BW_IN, 128, 1, 0)
  BW_CASE(true, BW_IN, 256, 0, 0)
  BW_CASE(true, BW_IN, 256, 1, 0)
  BW_CASE(false, BW_OUT, 128, 0, 0)
  BW_CASE(false, BW_OUT, 128, 1, 0)
  BW_CASE(false, BW_OUT, 256, 0, 0)
  BW_CASE(false, BW_OUT, 256, 1, 0)
  BW_CASE(true, BW_IN, 128, 0, 1)
  BW_CASE(true, BW_IN, 128, 1, 1)
  BW_CASE(true, BW_IN, 256, 0, 1)
  BW_CASE(true, BW_IN, 256, 1, 1)
  BW_CASE(false, BW_OUT, 128, 0, 1)
  BW_CASE(false, BW_OUT, 128, 1, 1)
  BW_CASE(false, BW_OUT, 256, 0, 1)
  BW_CASE(false, BW_OUT, 256, 1, 1)
#undef BW_CASE
  return CAFEQ_ERR_UNSUPPORTED;
}

// W: bf16 [d_out, d_in] with pitch ld; records and gradT as in BwParams (n_major, n_minor, NG are filled here)
static int bw_launch(cudaStream_t st, int axis_in, int k, const void* W, long long ld, BwParams p) {
  BwMaps maps;
  BwMulti mp;
  memset(&mp, 0, sizeof(mp));
  if (!make_map_bf16(&maps.w[0], W, p.d_in, p.d_out, ld, axis_in ? 64 : k)) return CAFEQ_ERR_UNSUPPORTED;
  for (int s = 1; s < BW_MAX_SUB; ++s) maps.w[s] = maps.w[0];
  mp.n = 1;
  mp.p[0] = p;
  const int swap = p.transpose_out ? 0 : 1;  // accumulator rows along the fastest index of the output
  return bw_dispatch(st, axis_in, k, swap, 0, maps, mp, g_bw_min_tiles.load(std::memory_order_relaxed));
}

// One sub-problem of a multi-matrix launch; W16 is the matrix in 16-bit storage (bf16, or the scaled fp16 copy of the
// F16 form) with pitch ld.  All sub-problems of a launch share axis, block size, output orientation and form.
struct BwSub {
  const void* W16;
  long long ld;
  BwParams p;
};

static int bw_launch_many(cudaStream_t st, int axis_in, int k, int transpose_out, int f16, const BwSub* subs, int n) {
  if (n < 1 || n > BW_MAX_SUB) return CAFEQ_ERR_INVALID_ARG;
  BwMaps maps;
  BwMulti mp;
  memset(&mp, 0, sizeof(mp));
  for (int s = 0; s < n; ++s) {
    if (!make_map_bf16(&maps.w[s], subs[s].W16, subs[s].p.d_in, subs[s].p.d_out, subs[s].ld, axis_in ? 64 : k)) return CAFEQ_ERR_UNSUPPORTED;
    mp.p[s] = subs[s].p;
    mp.p[s].transpose_out = transpose_out;
  }
  for (int s = n; s < BW_MAX_SUB; ++s) maps.w[s] = maps.w[0];
  mp.n = n;
  return bw_dispatch(st, axis_in, k, transpose_out ? 0 : 1, f16, maps, mp, 6);
}

template <int K, int SWAP_IN, int SWAP_OUT>
static int bw_launch_dual_t(cudaStream_t st, const BwMaps& mi, BwMulti pi, const BwMaps& mo, BwMulti po) {
  using C = BwCfg<K, 1>;
  static std::atomic<unsigned long long> done{0};
  if (!opt_in_smem(bd_bwd_dual_kernel<K, SWAP_IN, SWAP_OUT>, C::SMEM, done)) return CAFEQ_ERR_CUDA;
  long long ti = 0, to = 0, maj_i = 0, maj_o = 0;
  for (int s = 0; s < pi.n; ++s) {
    bw_fill_tiles(pi.p[s], 1, K);
    ti += (long long)pi.p[s].n_major * pi.p[s].n_minor;
    maj_i += pi.p[s].n_major;
    pi.tile_end[s] = (int)ti;
  }
  for (int s = pi.n; s < BW_MAX_SUB; ++s) pi.tile_end[s] = (int)ti;
  for (int s = 0; s < po.n; ++s) {
    bw_fill_tiles(po.p[s], 0, K);
    to += (long long)po.p[s].n_major * po.p[s].n_minor;
    maj_o += po.p[s].n_major;
    po.tile_end[s] = (int)to;
  }
  for (int s = po.n; s < BW_MAX_SUB; ++s) po.tile_end[s] = (int)to;
  // tiles of the two forms hold the same bytes (64 x K entries)
  const int n_in = dual_split(ti, to, g_dual_bwd_pct.load(std::memory_order_relaxed));
  bd_bwd_dual_kernel<K, SWAP_IN, SWAP_OUT><<<148, BW_THREADS, C::SMEM, st>>>(mi, pi, mo, po, n_in);
  return CAFEQ_OK;
}

// fp16 single-term form only; each list holds at least 148 * 6 tiles (the caller checks with bw_dual_ok)
static bool bw_dual_ok(int k) { return k == 128 || k == 256; }
static int bw_launch_dual(cudaStream_t st, int k, int tr_in, const BwSub* in, int n_in, int tr_out, const BwSub* out, int n_out) {
  if (n_in < 1 || n_in > BW_MAX_SUB || n_out < 1 || n_out > BW_MAX_SUB || !bw_dual_ok(k)) return CAFEQ_ERR_INVALID_ARG;
  BwMaps mi, mo;
  BwMulti pi, po;
  memset(&pi, 0, sizeof(pi));
  memset(&po, 0, sizeof(po));
  for (int s = 0; s < n_in; ++s) {
    if (!make_map_bf16(&mi.w[s], in[s].W16, in[s].p.d_in, in[s].p.d_out, in[s].ld, 64)) return CAFEQ_ERR_UNSUPPORTED;
    pi.p[s] = in[s].p;
    pi.p[s].transpose_out = tr_in;
  }
  for (int s = n_in; s < BW_MAX_SUB; ++s) mi.w[s] = mi.w[0];
  for (int s = 0; s < n_out; ++s) {
    if (!make_map_bf16(&mo.w[s], out[s].W16, out[s].p.d_in, out[s].p.d_out, out[s].ld, k)) return CAFEQ_ERR_UNSUPPORTED;
    po.p[s] = out[s].p;
    po.p[s].transpose_out = tr_out;
  }
  for (int s = n_out; s < BW_MAX_SUB; ++s) mo.w[s] = mo.w[0];
  pi.n = n_in;
  po.n = n_out;
  const int si = tr_in ? 0 : 1, so = tr_out ? 0 : 1;
#define BW_DUAL(KK, SI, SO) \
  if (k == KK && si == SI && so == SO) return bw_launch_dual_t<KK, SI, SO>(st, mi, pi, mo, po);
  BW_DUAL(128, 0, 0)
  BW_DUAL(128, 0, 1)
  BW_DUAL(128, 1, 0)
  BW_DUAL(128, 1, 1)
  BW_DUAL(256, 0, 0)
  BW_DUAL(256, 0, 1)
  BW_DUAL(256, 1, 0)
  BW_DUAL(256, 1, 1)
#undef BW_DUAL
  return CAFEQ_ERR_UNSUPPORTED;
}

}  // namespace cafeq
