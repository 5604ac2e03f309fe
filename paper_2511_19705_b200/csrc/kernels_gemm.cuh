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
    const int row = m0 + q * 32 + lane;
    bool ok = mbar_wait(bar_acc, 0, abort_flag, p.status);
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      tc_fence_after();
      const bool rv = row < p.M;
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
      double sq = 0.0;
      const long long cb = (long long)b * p.sCb, c0b = (long long)b * p.sC0b;
      const long long sb_mn = (long long)b * p.M * p.N;
      const bool vec_ok = ((p.N | p.ldc | p.ldc0 | p.sCb | p.sC0b | ((long long)p.M * p.N)) & 3) == 0 &&
                          (((uintptr_t)p.C | (uintptr_t)p.C0) & 15) == 0 && (((uintptr_t)p.Chi | (uintptr_t)p.Clo) & 7) == 0;
      // The kernel lives for microseconds and every CTA runs this code once or a few times, so its size counts
      // (instruction fetch showed up as the top stall): one rolled loop over the chunks, one unrolled copy of
      // each register <-> tile move shared by all paths, rolled loops on the edge paths.
      float* tile = reinterpret_cast<float*>(smem + (warp - 2) * 4608);  // [32][36] per warp (stage buffers are free now)
      const int rbase = m0 + q * 32;
      const int r4 = lane >> 3, c4 = (lane & 7) * 4;
#pragma unroll 1
      for (int ch = part; ch < BN / 32; ch += TG_EPI_PARTS) {
        const int nb0 = n0 + ch * 32;
        if (nb0 >= p.N) break;
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

// fp32 blocks [nb][k][k] -> bf16 hi / lo splits in row-major and transposed order; one 32 x 32 tile per CTA
// (grid: k/32, k/32, nb; block 32 x 8), transposed outputs staged through shared memory.  k % 32 == 0.
__global__ void __launch_bounds__(256) split_bf16_kernel(const float* __restrict__ X, int k, uint16_t* __restrict__ hi,
                                                         uint16_t* __restrict__ lo, uint16_t* __restrict__ thi,
                                                         uint16_t* __restrict__ tlo, const int* run_flag, const int32_t* status,
                                                         const double* gate = nullptr, double gate_tol = 0.0) {
  // runs for every block by default; with run_flag and / or gate: only when *run_flag != 0, or for the blocks
  // with gate[block] <= gate_tol
  if (status && *status) return;
  if (run_flag || gate) {
    const bool run = (run_flag && *run_flag != 0) || (gate && gate[blockIdx.z] <= gate_tol);
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
