// Batched dense products on the 5th-generation tensor cores (sm_100a) for the k x k algebra around the
// transform (Newton-Schulz refinement of M^-1, the M^-1 path of the gradient, M M^T of the orthonormality
// penalty) and for the pairwise product term of Eq. 5 (PQE).
//
//   C[b][m][n] = alpha * sum_t sum_l A_t[b / divA][m][l] * B_t[b][n][l]  + beta * C0[b][m][n] + gamma * [m == n]
//
// Every operand is bf16, row-major with the contraction index l contiguous (both K-major), so one product is
// the "A times B-transposed" form.  fp32 precision comes from summing up to three terms over bf16 splits
// (x = hi + lo, hi = bf16(x), lo = bf16(x - hi)); the accumulator is fp32 in tensor memory.
// The epilogue can write C as fp32, as bf16 hi / lo splits in row-major and / or transposed order (the
// operand layouts the next product needs), and accumulate sum(C^2).
//
// One CTA computes one 128 x BN tile: warp 0 = TMA producer, warp 1 = MMA issuer and tensor-memory owner,
// warps 2..9 = epilogue (one accumulator row and half of the tile's columns per thread).  Every mbarrier wait is bounded.
#pragma once

#include <atomic>

#include "kernels_fused.cuh"

namespace cafeq {

constexpr int TG_EPI_PARTS = 4;                       // epilogue warps per 32-lane quarter of the accumulator
constexpr int TG_THREADS = 64 + 128 * TG_EPI_PARTS;  // warp 0: TMA, warp 1: MMA, then the epilogue warps
constexpr int TG_BK = 64;
constexpr int TG_MAX_TERMS = 3;

struct TgMaps {
  CUtensorMap a[TG_MAX_TERMS];
  CUtensorMap b[TG_MAX_TERMS];
};

struct TgParams {
  int M, N, K, batch, nterms;
  int rowsA_per_batch, rowsB_per_batch;  // row offset of batch b in the 2-D operand views (0 for a shared operand)
  int divA;                              // batch b reads A rows of batch b / divA
  int colsA_per_batch;                   // column offset of batch b in the A view (block-diagonal operands: batch b
                                         // multiplies columns [b * k, b * k + k) of a wide matrix); 0 otherwise
  int divB, colsB_per_batch;             // the same for B (divB = 0 means 1)
  int min_ctas;                          // > 0: overrides the process-wide tile-width rule for this launch
  int a_rep_k, a_rep_r;                  // replicated contraction blocks of A: chunk at l reads columns ((l / k) / r) * k + l % k
  float alpha, beta, gamma;
  const float* C0;
  long long ldc0, sC0b;
  float* C;
  long long ldc, sCb;
  uint16_t *Chi, *Clo;    // bf16 splits, row-major [batch][M][N] (ld = N)
  uint16_t *Cthi, *Ctlo;  // bf16 splits, transposed [batch][N][M] (ld = M)
  double* sq;             // sum of C^2: sq[b * sq_stride]
  int sq_stride;
  const int* run_flag;    // optional: skip the whole launch when *run_flag == 0
  const double* gate;     // optional: batch b is skipped when gate[b] <= gate_tol (its iteration has converged)
  double gate_tol;
  int32_t* status;
};

template <int BN>
struct TgCfg {
  static constexpr int A_BYTES = 128 * TG_BK * 2;
  static constexpr int B_BYTES = BN * TG_BK * 2;
  static constexpr int STAGE = A_BYTES + B_BYTES;
  static constexpr int NSTAGE = (BN <= 128) ? 6 : 4;
  static constexpr int SMEM = 1024 + NSTAGE * STAGE + 256;
  static constexpr int TMEM_COLS = (BN < 32) ? 32 : BN;
};

// One 32-column chunk of one 128-row accumulator tile: scaling, C0, identity, sum of squares and every output format.
// taddr: the tile's accumulator at this warp's lane quarter; tile: this warp's [32][36] fp32 scratch in shared memory.
__device__ __forceinline__ void tg_epilogue_chunk(const TgParams& p, const int b, const int m0, const int n0, const int ch,
                                                  const uint32_t taddr, float* tile, const int q, const int lane, double& sq) {
  const int row = m0 + q * 32 + lane;
  const bool rv = row < p.M;
  const long long cb = (long long)b * p.sCb, c0b = (long long)b * p.sC0b;
  const long long sb_mn = (long long)b * p.M * p.N;
  const bool vec_ok = ((p.N | p.ldc | p.ldc0 | p.sCb | p.sC0b | ((long long)p.M * p.N)) & 3) == 0 &&
                      (((uintptr_t)p.C | (uintptr_t)p.C0) & 15) == 0 && (((uintptr_t)p.Chi | (uintptr_t)p.Clo) & 7) == 0;
  const int rbase = m0 + q * 32;
  const int r4 = lane >> 3, c4 = (lane & 7) * 4;
  const int nb0 = n0 + ch * 32;
  if (nb0 >= p.N) return;
  float v[32];
  tc_ld32(taddr + ch * 32, v);
  const bool inner = (nb0 + 32 <= p.N) && (m0 + 128 <= p.M);  // no edge in this chunk
  // Vector path (no edge, every pitch a multiple of 4 elements, aligned bases): a lane moves 16 bytes per
  // shared-memory access (pitch 36 floats: conflict-free by quarter warps) and a warp instruction covers
  // 4 rows x 128 bytes of global memory.  In the accumulator a lane owns a ROW; global traffic wants a
  // lane per COLUMN (32 lanes on 32 rows of a power-of-two pitch serialise in the memory pipe).
  const bool vec = inner && vec_ok;
  const int ncol = nb0 + lane;
  if (p.C0) {
    if (vec) {
      float4 cv[8];
#pragma unroll
      for (int i = 0; i < 8; ++i)
        cv[i] = __ldg(reinterpret_cast<const float4*>(p.C0 + c0b + (long long)(rbase + i * 4 + r4) * p.ldc0 + nb0 + c4));
#pragma unroll
      for (int i = 0; i < 8; ++i) *reinterpret_cast<float4*>(tile + (i * 4 + r4) * 36 + c4) = cv[i];
    } else {
#pragma unroll 1
      for (int r = 0; r < 32; ++r) {
        float x = 0.f;
        if (rbase + r < p.M && ncol < p.N) x = __ldg(p.C0 + c0b + (long long)(rbase + r) * p.ldc0 + ncol);
        tile[r * 36 + lane] = x;
      }
    }
    __syncwarp();
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float4 x = *reinterpret_cast<const float4*>(tile + lane * 36 + 4 * j);
      v[4 * j] = fmaf(p.beta, x.x, p.alpha * v[4 * j]);
      v[4 * j + 1] = fmaf(p.beta, x.y, p.alpha * v[4 * j + 1]);
      v[4 * j + 2] = fmaf(p.beta, x.z, p.alpha * v[4 * j + 2]);
      v[4 * j + 3] = fmaf(p.beta, x.w, p.alpha * v[4 * j + 3]);
    }
    __syncwarp();
  } else {
#pragma unroll
    for (int e = 0; e < 32; ++e) v[e] = p.alpha * v[e];
  }
  if (p.gamma != 0.f && row >= nb0 && row < nb0 + 32) {
#pragma unroll
    for (int e = 0; e < 32; ++e)
      if (nb0 + e == row) v[e] += p.gamma;
  }
  if (p.sq) {
    const int nv = rv ? min(32, p.N - nb0) : 0;
    float sqf = 0.f;
#pragma unroll
    for (int e = 0; e < 32; ++e)
      if (e < nv) sqf = fmaf(v[e], v[e], sqf);
    sq += (double)sqf;
  }
  if (p.C || p.Chi || (p.Cthi && !(inner && (p.M & 1) == 0))) {
#pragma unroll
    for (int j = 0; j < 8; ++j)
      *reinterpret_cast<float4*>(tile + lane * 36 + 4 * j) = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
    __syncwarp();
    if (vec) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int rr = i * 4 + r4;
        const float4 x = *reinterpret_cast<const float4*>(tile + rr * 36 + c4);
        if (p.C) *reinterpret_cast<float4*>(p.C + cb + (long long)(rbase + rr) * p.ldc + nb0 + c4) = x;
        if (p.Chi) {
          const __nv_bfloat16 h0 = __float2bfloat16_rn(x.x), h1 = __float2bfloat16_rn(x.y);
          const __nv_bfloat16 h2 = __float2bfloat16_rn(x.z), h3 = __float2bfloat16_rn(x.w);
          const long long o = sb_mn + (long long)(rbase + rr) * p.N + nb0 + c4;
          *reinterpret_cast<uint2*>(p.Chi + o) =
              make_uint2((uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16),
                         (uint32_t)__bfloat16_as_ushort(h2) | ((uint32_t)__bfloat16_as_ushort(h3) << 16));
          if (p.Clo) {
            const __nv_bfloat16 l0 = __float2bfloat16_rn(x.x - __bfloat162float(h0));
            const __nv_bfloat16 l1 = __float2bfloat16_rn(x.y - __bfloat162float(h1));
            const __nv_bfloat16 l2 = __float2bfloat16_rn(x.z - __bfloat162float(h2));
            const __nv_bfloat16 l3 = __float2bfloat16_rn(x.w - __bfloat162float(h3));
            *reinterpret_cast<uint2*>(p.Clo + o) =
                make_uint2((uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16),
                           (uint32_t)__bfloat16_as_ushort(l2) | ((uint32_t)__bfloat16_as_ushort(l3) << 16));
          }
        }
      }
    } else {
      // edge chunk or odd pitches: one element per lane and row, everything guarded
#pragma unroll 1
      for (int r = 0; r < 32; ++r) {
        if (rbase + r < p.M && ncol < p.N) {
          const float x = tile[r * 36 + lane];
          if (p.C) p.C[cb + (long long)(rbase + r) * p.ldc + ncol] = x;
          if (p.Chi) {
            const __nv_bfloat16 h = __float2bfloat16_rn(x);
            const long long o = sb_mn + (long long)(rbase + r) * p.N + ncol;
            p.Chi[o] = __bfloat16_as_ushort(h);
            if (p.Clo) p.Clo[o] = __bfloat16_as_ushort(__float2bfloat16_rn(x - __bfloat162float(h)));
          }
        }
      }
    }
    if (p.Cthi && !(inner && (p.M & 1) == 0) && rv) {
      // transposed outputs on an edge: this lane's row, one column at a time (read back from its tile row)
      uint16_t* cth = p.Cthi + sb_mn + (long long)nb0 * p.M + row;
      uint16_t* ctl = p.Ctlo ? p.Ctlo + sb_mn + (long long)nb0 * p.M + row : nullptr;
#pragma unroll 1
      for (int e = 0; e < 32; ++e) {
        if (nb0 + e < p.N) {
          const float x = tile[lane * 36 + e];
          const __nv_bfloat16 h = __float2bfloat16_rn(x);
          cth[(long long)e * p.M] = __bfloat16_as_ushort(h);
          if (ctl) ctl[(long long)e * p.M] = __bfloat16_as_ushort(__float2bfloat16_rn(x - __bfloat162float(h)));
        }
      }
    }
    __syncwarp();
  }
  if (p.Cthi && inner && (p.M & 1) == 0) {
    // transposed outputs: consecutive lanes are consecutive rows = consecutive addresses.  Neighbouring
    // lanes trade one value so that every lane stores a 32-bit pair of rows: even lanes write column e,
    // odd lanes column e + 1.
    const int odd = lane & 1;
    const long long rowpair = row & ~1;
#pragma unroll
    for (int e = 0; e < 32; e += 2) {
      const __nv_bfloat16 h0 = __float2bfloat16_rn(v[e]), h1 = __float2bfloat16_rn(v[e + 1]);
      const uint32_t p0 = (uint32_t)__bfloat16_as_ushort(h0) |
                          ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v[e] - __bfloat162float(h0))) << 16);
      const uint32_t p1 = (uint32_t)__bfloat16_as_ushort(h1) |
                          ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v[e + 1] - __bfloat162float(h1))) << 16);
      const uint32_t mine = odd ? p1 : p0;                       // (hi | lo << 16) of my row in the column I store
      const uint32_t other = __shfl_xor_sync(0xffffffffu, odd ? p0 : p1, 1);  // the neighbour row's, same column
      const uint32_t lo_row = odd ? other : mine, hi_row = odd ? mine : other;  // rows (2j, 2j + 1)
      const long long o = sb_mn + (long long)(nb0 + e + odd) * p.M + rowpair;
      *reinterpret_cast<uint32_t*>(p.Cthi + o) = (lo_row & 0xFFFFu) | (hi_row << 16);
      if (p.Ctlo) *reinterpret_cast<uint32_t*>(p.Ctlo + o) = (lo_row >> 16) | (hi_row & 0xFFFF0000u);
    }
  }
}

template <int BN>
__global__ void __launch_bounds__(TG_THREADS, 1)
tc_gemm_kernel(const __grid_constant__ TgMaps maps, const TgParams p) {
  using C = TgCfg<BN>;
  if (p.status && *p.status) return;
  if (p.run_flag && *p.run_flag == 0) return;
  if (p.gate && p.gate[blockIdx.z] <= p.gate_tol) return;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = (uint64_t*)(smem + C::NSTAGE * C::STAGE);
  const uint32_t bar_full = smem_u32(bars);
  const uint32_t bar_empty = bar_full + 8 * C::NSTAGE;
  const uint32_t bar_acc = bar_empty + 8 * C::NSTAGE;
  uint32_t* tmem_slot = (uint32_t*)(bars + 2 * C::NSTAGE + 1);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = blockIdx.x * BN, m0 = blockIdx.y * 128, b = blockIdx.z;

  if (threadIdx.x < 2 * TG_MAX_TERMS) {
    const int t = threadIdx.x >> 1;
    if (t < p.nterms) tma_prefetch_desc((threadIdx.x & 1) ? &maps.b[t] : &maps.a[t]);
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < C::NSTAGE; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    mbar_init(bar_acc, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
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
  const int kchunks = p.K / TG_BK;
  const int total = kchunks * p.nterms;

  if (warp == 0) {
    if (lane == 0) {
      const int ya = (b / p.divA) * p.rowsA_per_batch + m0;
      const int bb = p.divB > 1 ? b / p.divB : b;
      const int yb = bb * p.rowsB_per_batch + n0;
      for (int it = 0; it < total; ++it) {
        const int t = it / kchunks, c = it - t * kchunks;
        const uint32_t s = it % C::NSTAGE, ph = (it / C::NSTAGE) & 1u;
        if (!mbar_wait(bar_empty + 8 * s, ph ^ 1u, abort_flag, p.status)) break;
        mbar_expect_tx(bar_full + 8 * s, C::STAGE);
        const int l0 = c * TG_BK;
        int xa = l0;
        if (p.a_rep_r > 1) xa = ((l0 / p.a_rep_k) / p.a_rep_r) * p.a_rep_k + (l0 % p.a_rep_k);
        xa += (b / p.divA) * p.colsA_per_batch;
        uint8_t* st = smem + s * C::STAGE;
        tma_load_2d(smem_u32(st), &maps.a[t], xa, ya, bar_full + 8 * s);
        tma_load_2d(smem_u32(st + C::A_BYTES), &maps.b[t], l0 + bb * p.colsB_per_batch, yb, bar_full + 8 * s);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(128, BN, 0, 0);
      bool ok = true;
      for (int it = 0; it < total && ok; ++it) {
        const uint32_t s = it % C::NSTAGE, ph = (it / C::NSTAGE) & 1u;
        if (!mbar_wait(bar_full + 8 * s, ph, abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t sa = smem_u32(smem + s * C::STAGE), sb = sa + C::A_BYTES;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          tc_mma_bf16(tmem_base, umma_desc_sw128(sa + kk * 32), umma_desc_sw128(sb + kk * 32), idesc, (it | kk) != 0 ? 1u : 0u);
        tc_commit(bar_empty + 8 * s);
      }
      if (ok) tc_commit(bar_acc);
    }
  } else {
    // a warp reads the accumulator lanes of its quarter (warp index modulo 4); the warps of one quarter share
    // its 32-column chunks round-robin: with two warps per scheduler the dependent chains of the epilogue
    // (shuffles, conversions, stores) left the issue slots empty
    const int q = warp & 3, part = (warp - 2) >> 2;
    bool ok = mbar_wait(bar_acc, 0, abort_flag, p.status);
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
      double sq = 0.0;
      float* tile = reinterpret_cast<float*>(smem + (warp - 2) * 4608);  // [32][36] per warp (stage buffers are free now)
#pragma unroll 1
      for (int ch = part; ch < BN / 32; ch += TG_EPI_PARTS) tg_epilogue_chunk(p, b, m0, n0, ch, taddr, tile, q, lane, sq);
      if (p.sq) {
        for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
        if (lane == 0 && sq != 0.0) atomicAdd(p.sq + (long long)b * p.sq_stride, sq);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::TMEM_COLS) : "memory");
  }
}

// ------------------------------------------------------------------------------------------------
// Whole-block form for the batched k x k products (k = 128 or 256): ONE CTA computes the whole k x k output of a
// block (two 128-row accumulators in tensor memory at k = 256).
//   * Every DISTINCT operand array is loaded once per contraction chunk, whatever the number of split terms that
//     reuse it (a three-term product moves 512 KB per block from L2 instead of the 1152 KB of the tiled kernel).
//   * Either side may be MN-major: A_op[m][l] read from an array stored [l][m], B_op[n][l] from one stored [l][n].
//     The iteration X <- X + X (I - A X) and the M^-1 path then run on row-major arrays only; no transposed copy
//     of anything is ever written.
//   * The epilogue moves whole 32 x 32 tiles with TMA: C0 tiles are loaded into swizzled shared memory one tile
//     ahead, results are staged in swizzled shared memory (conflict-free 16-byte accesses) and stored with
//     cp.async.bulk.tensor.  The load/store units see only those shared-memory accesses: the tiled kernel's
//     epilogue spent its time in their queue (scattered global accesses and transposes through shared memory).
// Shared memory: a ring of slots, one slot = one operand array's k (rows or columns) x 64 contraction entries;
// after the products the same memory holds the epilogue tiles (12 KB per epilogue warp).
// ------------------------------------------------------------------------------------------------
constexpr int TB_MAX_ARR = 2;  // distinct arrays per side

struct TbMaps {
  CUtensorMap a[TB_MAX_ARR];
  CUtensorMap b[TB_MAX_ARR];
  CUtensorMap c0, c;    // fp32 [nb * k, k], box 32 x 32, 128-byte swizzle
  CUtensorMap chi, clo; // bf16 [nb * k, k], box 32 x 32, 64-byte swizzle
  CUtensorMap chl;      // hi and lo as the two planes of one 3-D view (when lo lies a fixed distance after hi): one store
};
struct TbTerms {
  int na, nb;                 // distinct A / B arrays
  int nterms;
  int ta[TG_MAX_TERMS], tb[TG_MAX_TERMS];  // term t multiplies a[ta[t]] by b[tb[t]]
  int a_mn, b_mn;             // the A / B arrays are stored [l][m] / [l][n] (MN-major operands)
  int hl3d;                   // Chi and Clo are stored with one 3-D bulk copy through maps.chl
};

template <int K>
struct TbCfg {
  static constexpr int HALVES = K / 128;
  static constexpr int SLOT = K * TG_BK * 2;
  static constexpr int NSLOT = (K == 256) ? 6 : 12;  // 192 KB: the epilogue tiles of 16 warps need as much
  static constexpr int KCH = K / TG_BK;
  static constexpr int EPI_WARP_BYTES = 12288;        // two fp32 tiles (C0 prefetch / C) + hi + lo
  static constexpr int NBAR = 2 * NSLOT + 1 + 2 * 4 * TG_EPI_PARTS;
  static constexpr int SMEM = 1024 + NSLOT * SLOT + 8 * NBAR + 64;
  static constexpr int TMEM_COLS = HALVES * K;  // 128 or 512
  static_assert(NSLOT * SLOT >= 4 * TG_EPI_PARTS * EPI_WARP_BYTES, "epilogue tiles must fit in the ring");
};

__device__ __forceinline__ void fence_proxy_async_smem_tb() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(map), "r"(src), "r"(x), "r"(y)
               : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int x, int y, int z) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(map), "r"(src), "r"(x), "r"(y),
               "r"(z)
               : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// all bulk stores of this thread have finished READING shared memory
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }

template <int K>
__global__ void __launch_bounds__(TG_THREADS, 1)
tc_block_kernel(const __grid_constant__ TbMaps maps, const TbTerms tt, const TgParams p) {
  using C = TbCfg<K>;
  static_assert(K == 128 || K == 256, "block size");
  if (p.status && *p.status) return;
  if (p.run_flag && *p.run_flag == 0) return;
  const int b = blockIdx.x;
  if (p.gate && p.gate[b] <= p.gate_tol) return;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = (uint64_t*)(smem + C::NSLOT * C::SLOT);
  const uint32_t bar_full = smem_u32(bars);
  const uint32_t bar_empty = bar_full + 8 * C::NSLOT;
  const uint32_t bar_acc = bar_empty + 8 * C::NSLOT;
  const uint32_t bar_c0 = bar_acc + 8;  // two per epilogue warp
  uint32_t* tmem_slot = (uint32_t*)(bars + C::NBAR);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nu = tt.na + tt.nb;  // slots per contraction chunk

  if (threadIdx.x < 2 * TB_MAX_ARR) {
    const int u = threadIdx.x >> 1;
    if (threadIdx.x & 1) { if (u < tt.nb) tma_prefetch_desc(&maps.b[u]); }
    else if (u < tt.na) tma_prefetch_desc(&maps.a[u]);
  }
  if (threadIdx.x == 32) {
    if (p.C0) tma_prefetch_desc(&maps.c0);
    if (p.C) tma_prefetch_desc(&maps.c);
    if (tt.hl3d) tma_prefetch_desc(&maps.chl);
    else {
      if (p.Chi) tma_prefetch_desc(&maps.chi);
      if (p.Clo) tma_prefetch_desc(&maps.clo);
    }
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < C::NSLOT; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    mbar_init(bar_acc, 1);
    for (int s = 0; s < 2 * 4 * TG_EPI_PARTS; ++s) mbar_init(bar_c0 + 8 * s, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
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
    if (lane == 0) {
      const int ra = (b / p.divA) * K, rb = b * K;  // first row of this batch in the A / B arrays
      uint32_t it = 0;
      bool ok = true;
      for (int c = 0; c < C::KCH && ok; ++c)
        for (int u = 0; u < nu; ++u, ++it) {
          const uint32_t s = it % C::NSLOT, ph = (it / C::NSLOT) & 1u;
          if (!mbar_wait(bar_empty + 8 * s, ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
          mbar_expect_tx(bar_full + 8 * s, C::SLOT);
          const bool isA = u < tt.na;
          const CUtensorMap* mp = isA ? &maps.a[u] : &maps.b[u - tt.na];
          const uint32_t dst = smem_u32(smem + s * C::SLOT);
          const int r0 = isA ? ra : rb;
          if ((isA ? tt.a_mn : tt.b_mn) == 0) {
            tma_load_2d(dst, mp, c * TG_BK, r0, bar_full + 8 * s);  // K rows (m or n) x 64 contraction entries
          } else {
            // stored [l][mn]: 64 contraction rows x K columns as K / 64 boxes of 64 x 64 (one swizzle atom each)
            for (int j = 0; j < K / 64; ++j) tma_load_2d(dst + j * 8192, mp, j * 64, r0 + c * TG_BK, bar_full + 8 * s);
          }
        }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_bf16(128, K, tt.a_mn, tt.b_mn);
      bool ok = true;
      uint32_t it = 0;
      for (int c = 0; c < C::KCH && ok; ++c) {
        for (int u = 0; u < nu; ++u) {
          const uint32_t s = (it + u) % C::NSLOT, ph = ((it + u) / C::NSLOT) & 1u;
          if (!mbar_wait(bar_full + 8 * s, ph, abort_flag, p.status)) { ok = false; break; }
        }
        if (!ok) break;
        tc_fence_after();
        for (int t = 0; t < tt.nterms; ++t) {
          const uint32_t sa = smem_u32(smem + ((it + tt.ta[t]) % C::NSLOT) * C::SLOT);
          const uint32_t sb = smem_u32(smem + ((it + tt.na + tt.tb[t]) % C::NSLOT) * C::SLOT);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            const uint64_t bd = tt.b_mn ? umma_desc_sw128_lbo(sb + kk * 2048, 8192) : umma_desc_sw128(sb + kk * 32);
#pragma unroll
            for (int mh = 0; mh < C::HALVES; ++mh) {
              const uint64_t ad = tt.a_mn ? umma_desc_sw128_lbo(sa + mh * 16384 + kk * 2048, 8192)
                                          : umma_desc_sw128(sa + mh * 16384 + kk * 32);
              tc_mma_bf16(tmem_base + mh * K, ad, bd, idesc, (c | t | kk) != 0 ? 1u : 0u);
            }
          }
        }
        for (int u = 0; u < nu; ++u) tc_commit(bar_empty + 8 * ((it + u) % C::NSLOT));
        it += nu;
      }
      if (ok) tc_commit(bar_acc);
    }
  } else {
    // ---------------------------------------------------------------- epilogue: 32 x 32 tiles, TMA in and out
    const int q = warp & 3, part = (warp - 2) >> 2, ew = warp - 2;
    bool ok = mbar_wait(bar_acc, 0, abort_flag, p.status);
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      tc_fence_after();
      uint8_t* wbuf = smem + ew * C::EPI_WARP_BYTES;  // the slots are free now
      const uint32_t tC = smem_u32(wbuf), tH = tC + 8192, tL = tC + 10240;
      const uint32_t bc0 = bar_c0 + 16 * ew;
      constexpr int CPH = K / 32;                      // 32-column tiles per accumulator
      constexpr int NU = C::HALVES * CPH / TG_EPI_PARTS;  // tiles per warp
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
      const int sw = lane & 7;
      float sq4[4] = {0.f, 0.f, 0.f, 0.f};
      double sq = 0.0;
      // tile i of this warp: accumulator half mh, column tile ch; block rows mh * 128 + q * 32 .. + 32
      auto tile_of = [&](int i, int& mh, int& ch) { const int c2 = part + i * TG_EPI_PARTS; mh = c2 / CPH; ch = c2 - mh * CPH; };
      if (p.C0 && lane == 0) {
        int mh, ch;
        tile_of(0, mh, ch);
        mbar_expect_tx(bc0, 4096);
        tma_load_2d(tC, &maps.c0, ch * 32, b * K + mh * 128 + q * 32, bc0);
      }
#pragma unroll 1
      for (int i = 0; i < NU && ok; ++i) {
        int mh, ch;
        tile_of(i, mh, ch);
        const int row0 = b * K + mh * 128 + q * 32, col0 = ch * 32;
        const uint32_t tCi = tC + (uint32_t)(i & 1) * 4096;
        float v[32];
        tc_ld32(taddr + mh * K + ch * 32, v);
#pragma unroll
        for (int e = 0; e < 32; ++e) v[e] *= p.alpha;
        if (p.C0) {
          ok = mbar_wait(bc0 + 8 * (i & 1), (i >> 1) & 1u, abort_flag, p.status);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            float4 x;
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(x.x), "=f"(x.y), "=f"(x.z), "=f"(x.w)
                         : "r"(tCi + lane * 128 + ((c ^ sw) << 4)));
            v[4 * c] = fmaf(p.beta, x.x, v[4 * c]);
            v[4 * c + 1] = fmaf(p.beta, x.y, v[4 * c + 1]);
            v[4 * c + 2] = fmaf(p.beta, x.z, v[4 * c + 2]);
            v[4 * c + 3] = fmaf(p.beta, x.w, v[4 * c + 3]);
          }
        }
        if (p.gamma != 0.f && col0 == mh * 128 + q * 32) {
#pragma unroll
          for (int e = 0; e < 32; ++e)
            if (e == lane) v[e] += p.gamma;
        }
        if (p.sq) {
#pragma unroll
          for (int e = 0; e < 32; ++e) sq4[e & 3] = fmaf(v[e], v[e], sq4[e & 3]);
        }
        // Only now, with this tile's values in registers: wait until the stores of the previous tile have read their
        // shared memory (the other fp32 buffer, hi, lo), then fetch the next C0 tile into that other buffer (it is needed
        // one tile from now).
        if (lane == 0) {
          tma_store_wait_read();
          if (p.C0 && i + 1 < NU) {
            int mh2, ch2;
            tile_of(i + 1, mh2, ch2);
            const uint32_t bn = bc0 + 8 * ((i + 1) & 1);
            mbar_expect_tx(bn, 4096);
            tma_load_2d(tC + (uint32_t)((i + 1) & 1) * 4096, &maps.c0, ch2 * 32, b * K + mh2 * 128 + q * 32, bn);
          }
        }
        __syncwarp();
        if (p.C) {
#pragma unroll
          for (int c = 0; c < 8; ++c)
            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(tCi + lane * 128 + ((c ^ sw) << 4)), "f"(v[4 * c]),
                         "f"(v[4 * c + 1]), "f"(v[4 * c + 2]), "f"(v[4 * c + 3])
                         : "memory");
        }
        if (p.Chi) {
          // bf16 tiles: 64-byte rows, 16-byte chunks XOR-swizzled by (row / 2) mod 4
          const int sw2 = (lane >> 1) & 3;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint32_t h[4], l[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float x0 = v[8 * c + 2 * j], x1 = v[8 * c + 2 * j + 1];
              const __nv_bfloat16 h0 = __float2bfloat16_rn(x0), h1 = __float2bfloat16_rn(x1);
              h[j] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
              if (p.Clo) {
                const __nv_bfloat16 l0 = __float2bfloat16_rn(x0 - __bfloat162float(h0));
                const __nv_bfloat16 l1 = __float2bfloat16_rn(x1 - __bfloat162float(h1));
                l[j] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
              }
            }
            const uint32_t off = lane * 64 + ((c ^ sw2) << 4);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(tH + off), "r"(h[0]), "r"(h[1]), "r"(h[2]), "r"(h[3]) : "memory");
            if (p.Clo)
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(tL + off), "r"(l[0]), "r"(l[1]), "r"(l[2]), "r"(l[3]) : "memory");
          }
        }
        fence_proxy_async_smem_tb();
        __syncwarp();
        if (lane == 0) {
          if (p.C) tma_store_2d(&maps.c, tCi, col0, row0);
          if (tt.hl3d) {
            tma_store_3d(&maps.chl, tH, col0, row0, 0);  // the lo tile follows the hi tile in shared memory
          } else {
            if (p.Chi) tma_store_2d(&maps.chi, tH, col0, row0);
            if (p.Clo) tma_store_2d(&maps.clo, tL, col0, row0);
          }
          tma_store_commit();
        }
      }
      if (lane == 0) tma_store_wait_read();
      if (p.sq) {
        sq = (double)((sq4[0] + sq4[1]) + (sq4[2] + sq4[3]));
        for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
        if (lane == 0 && sq != 0.0) atomicAdd(p.sq + (long long)b * p.sq_stride, sq);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::TMEM_COLS) : "memory");
  }
}

// 2-D bf16 operand view for the product kernel: `rows` rows of `cols` contiguous elements.
struct TgOperand {
  const void* ptr;
  long long rows, cols, pitch;
};

template <int BN>
static int tg_launch_t(cudaStream_t st, const TgOperand* A, const TgOperand* B, TgParams p) {
  using C = TgCfg<BN>;
  static std::atomic<unsigned long long> done{0};
  if (!opt_in_smem(tc_gemm_kernel<BN>, C::SMEM, done)) return CAFEQ_ERR_CUDA;
  TgMaps maps;
  memset(&maps, 0, sizeof(maps));
  for (int t = 0; t < p.nterms; ++t) {
    if (!make_map_bf16(&maps.a[t], A[t].ptr, A[t].cols, A[t].rows, A[t].pitch, 128)) return CAFEQ_ERR_UNSUPPORTED;
    if (!make_map_bf16(&maps.b[t], B[t].ptr, B[t].cols, B[t].rows, B[t].pitch, BN)) return CAFEQ_ERR_UNSUPPORTED;
  }
  dim3 grid((p.N + BN - 1) / BN, (p.M + 127) / 128, p.batch);
  tc_gemm_kernel<BN><<<grid, TG_THREADS, C::SMEM, st>>>(maps, p);
  return CAFEQ_OK;
}

// K must be a multiple of 64; operands 16-byte aligned with pitches that are multiples of 8 elements.
// Tile-width rule of the small batched products: the widest tile that still gives at least this many CTAs.
// A CTA's life is dominated by fixed latencies and its epilogue, so narrow tiles (many CTAs) finish one product
// sooner, while wide tiles (few CTAs) cost far fewer SM-microseconds and leave room for the kernels of other
// problems running in other streams.  Default: narrow tiles (one chain alone); cafeq_set_overlap_mode changes it.
static std::atomic<int> g_tg_min_ctas{96};
static int tg_launch(cudaStream_t st, const TgOperand* A, const TgOperand* B, const TgParams& p) {
  if (p.K % TG_BK || p.nterms < 1 || p.nterms > TG_MAX_TERMS) return CAFEQ_ERR_UNSUPPORTED;
  const int min_ctas = p.min_ctas > 0 ? p.min_ctas : g_tg_min_ctas.load(std::memory_order_relaxed);
  const long long mt = (long long)p.batch * ((p.M + 127) / 128);
  if (p.N > 128 && mt * ((p.N + 255) / 256) >= min_ctas) return tg_launch_t<256>(st, A, B, p);
  if (p.N > 64 && mt * ((p.N + 127) / 128) >= min_ctas) return tg_launch_t<128>(st, A, B, p);
  if (p.N <= 64 || mt * ((p.N + 127) / 128) < min_ctas) return tg_launch_t<64>(st, A, B, p);
  return tg_launch_t<128>(st, A, B, p);
}

// General 2-D tensor map: element type and size, box, swizzle mode (inner box extent in bytes <= the swizzle span).
static bool make_map_2d(CUtensorMap* m, CUtensorMapDataType dt, int esize, const void* base, long long cols, long long rows,
                        long long pitch, int box_cols, int box_rows, CUtensorMapSwizzle swz) {
  EncodeTiledFn enc = get_encode_tiled();
  if (!enc) return false;
  if (((uintptr_t)base & 15) || ((pitch * esize) & 15)) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)pitch * esize};
  cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return enc(m, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Batched k x k products in the whole-block form: operands bf16 [nb * k, k] (A of batch b at rows (b / divA) * k);
// a_mn / b_mn: the A / B arrays hold the operand transposed ([l][m] / [l][n]).  p filled as for tg_launch with
// M = N = K = k, contiguous k x k blocks in C0 / C / Chi / Clo, no transposed outputs.  Distinct pointers among the
// terms are found here.
static std::atomic<int> g_tb_enable{1};
template <int K>
static int tb_launch_t(cudaStream_t st, const TbMaps& maps, const TbTerms& tt, const TgParams& p) {
  using C = TbCfg<K>;
  static std::atomic<unsigned long long> done{0};
  if (!opt_in_smem(tc_block_kernel<K>, C::SMEM, done)) return CAFEQ_ERR_CUDA;
  tc_block_kernel<K><<<p.batch, TG_THREADS, C::SMEM, st>>>(maps, tt, p);
  return CAFEQ_OK;
}
static bool tb_supported(int k, int nterms) { return (k == 128 || k == 256) && nterms >= 1 && nterms <= TG_MAX_TERMS; }
static int tb_launch(cudaStream_t st, int nterms, const uint16_t* const* A, const uint16_t* const* B, int a_mn, int b_mn,
                     long long rowsA, long long rowsB, int k, const TgParams& p) {
  if (p.Cthi || p.Ctlo || p.ldc != k || p.sCb != (long long)k * k || (p.C0 && (p.ldc0 != k || p.sC0b != (long long)k * k)))
    return CAFEQ_ERR_UNSUPPORTED;
  TbMaps maps;
  TbTerms tt;
  memset(&maps, 0, sizeof(maps));
  memset(&tt, 0, sizeof(tt));
  const uint16_t* ua[TB_MAX_ARR] = {nullptr, nullptr};
  const uint16_t* ub[TB_MAX_ARR] = {nullptr, nullptr};
  tt.nterms = nterms;
  tt.a_mn = a_mn ? 1 : 0;
  tt.b_mn = b_mn ? 1 : 0;
  for (int t = 0; t < nterms; ++t) {
    int ia = -1, ib = -1;
    for (int u = 0; u < tt.na; ++u) if (ua[u] == A[t]) ia = u;
    if (ia < 0) { if (tt.na == TB_MAX_ARR) return CAFEQ_ERR_UNSUPPORTED; ua[tt.na] = A[t]; ia = tt.na++; }
    for (int u = 0; u < tt.nb; ++u) if (ub[u] == B[t]) ib = u;
    if (ib < 0) { if (tt.nb == TB_MAX_ARR) return CAFEQ_ERR_UNSUPPORTED; ub[tt.nb] = B[t]; ib = tt.nb++; }
    tt.ta[t] = ia;
    tt.tb[t] = ib;
  }
  // K-major arrays: one box of k rows x 64 contraction entries; MN-major arrays: boxes of 64 x 64
  for (int u = 0; u < tt.na; ++u) if (!make_map_bf16(&maps.a[u], ua[u], k, rowsA, k, a_mn ? 64 : k)) return CAFEQ_ERR_UNSUPPORTED;
  for (int u = 0; u < tt.nb; ++u) if (!make_map_bf16(&maps.b[u], ub[u], k, rowsB, k, b_mn ? 64 : k)) return CAFEQ_ERR_UNSUPPORTED;
  for (int u = tt.na; u < TB_MAX_ARR; ++u) maps.a[u] = maps.a[0];
  for (int u = tt.nb; u < TB_MAX_ARR; ++u) maps.b[u] = maps.b[0];
  const long long rowsC = (long long)p.batch * k;
  bool okm = true;
  if (p.C0) okm = okm && make_map_2d(&maps.c0, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, p.C0, k, rowsC, k, 32, 32, CU_TENSOR_MAP_SWIZZLE_128B);
  if (p.C) okm = okm && make_map_2d(&maps.c, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, p.C, k, rowsC, k, 32, 32, CU_TENSOR_MAP_SWIZZLE_128B);
  if (p.Chi) okm = okm && make_map_2d(&maps.chi, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, p.Chi, k, rowsC, k, 32, 32, CU_TENSOR_MAP_SWIZZLE_64B);
  if (p.Clo) okm = okm && make_map_2d(&maps.clo, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, p.Clo, k, rowsC, k, 32, 32, CU_TENSOR_MAP_SWIZZLE_64B);
  if (!okm) return CAFEQ_ERR_UNSUPPORTED;
  if (p.Clo && !p.Chi) return CAFEQ_ERR_UNSUPPORTED;
  if (p.Chi && p.Clo && p.Clo > p.Chi && (((uintptr_t)p.Clo - (uintptr_t)p.Chi) & 15) == 0) {
    EncodeTiledFn enc = get_encode_tiled();
    cuuint64_t dims[3] = {(cuuint64_t)k, (cuuint64_t)rowsC, 2};
    cuuint64_t strides[2] = {(cuuint64_t)k * 2, (cuuint64_t)((uintptr_t)p.Clo - (uintptr_t)p.Chi)};
    cuuint32_t box[3] = {32, 32, 2};
    cuuint32_t estr[3] = {1, 1, 1};
    if (enc && enc(&maps.chl, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, p.Chi, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS)
      tt.hl3d = 1;
  }
  return k == 256 ? tb_launch_t<256>(st, maps, tt, p) : tb_launch_t<128>(st, maps, tt, p);
}

// fp32 blocks [nb][k][k] -> bf16 hi / lo splits in row-major and transposed order; one 32 x 32 tile per CTA
// (grid: k/32, k/32, nb; block 32 x 8), transposed outputs staged through shared memory.  k % 32 == 0.
__global__ void __launch_bounds__(256) split_bf16_kernel(const float* __restrict__ X, int k, uint16_t* __restrict__ hi,
                                                         uint16_t* __restrict__ lo, uint16_t* __restrict__ thi,
                                                         uint16_t* __restrict__ tlo, const int* run_flag, const int32_t* status,
                                                         const double* gate = nullptr, double gate_tol = 0.0,
                                                         int parity_iters = 0, int parity_nb = 0) {
  // runs for every block by default; with run_flag and / or gate: only when *run_flag != 0, or for the blocks
  // with gate[block] <= gate_tol.  parity_iters > 0: `gate` is the base of the residual table [iteration][block] of
  // a gated iteration that writes its splits alternately into two sets; the block is split again only when the
  // number of iterations it ran (iteration i runs iff the residual of iteration i - 1 exceeds gate_tol) left its
  // newest splits in the other set than parity_iters iterations would have.
  if (status && *status) return;
  if (run_flag || gate) {
    bool run = run_flag && *run_flag != 0;
    if (!run && gate) {
      if (parity_iters > 0) {
        int ran = 1;
        while (ran < parity_iters && gate[(size_t)(ran - 1) * parity_nb + blockIdx.z] > gate_tol) ++ran;
        run = ((ran ^ parity_iters) & 1) != 0;
      } else {
        run = gate[blockIdx.z] <= gate_tol;
      }
    }
    if (!run) return;
  }
  __shared__ uint32_t tile[32][33];
  const size_t base = (size_t)blockIdx.z * k * k;
  const int j0 = blockIdx.x * 32, i0 = blockIdx.y * 32;
  const int tx = threadIdx.x, ty = threadIdx.y;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int i = i0 + ty + 8 * r, j = j0 + tx;
    const float x = X[base + (size_t)i * k + j];
    const __nv_bfloat16 h = __float2bfloat16_rn(x);
    const __nv_bfloat16 l = __float2bfloat16_rn(x - __bfloat162float(h));
    const uint16_t hb = __bfloat16_as_ushort(h), lb = __bfloat16_as_ushort(l);
    if (hi) hi[base + (size_t)i * k + j] = hb;
    if (lo) lo[base + (size_t)i * k + j] = lb;
    tile[ty + 8 * r][tx] = (uint32_t)hb | ((uint32_t)lb << 16);
  }
  __syncthreads();
  if (thi || tlo) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int j = j0 + ty + 8 * r, i = i0 + tx;
      const uint32_t v = tile[tx][ty + 8 * r];
      if (thi) thi[base + (size_t)j * k + i] = (uint16_t)(v & 0xFFFFu);
      if (tlo) tlo[base + (size_t)j * k + i] = (uint16_t)(v >> 16);
    }
  }
}

}  // namespace cafeq
