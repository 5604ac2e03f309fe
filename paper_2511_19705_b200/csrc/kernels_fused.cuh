// Fused block-diagonal transform pass on the 5th-generation tensor cores (sm_100a):
//   U = T o X on one axis of a bf16 matrix X, accumulated in tensor memory, followed in the same kernel by
//   the per-group work the method needs on U -- absmax / arg-max (Eq. 1's scale, Eq. 4's ||.||_inf, the
//   LogSumExp maxima), round-to-nearest codes, the residual Delta = Q(U) - U, or a sum of squares.
// U never goes to HBM.  One CTA keeps its operator block(s) resident in shared memory and streams tiles of
// X through a TMA ring; accumulators are double-buffered in tensor memory so the epilogue of tile t overlaps
// the products of tile t+1.
//
// Warp roles (320 threads): warp 0 = TMA producer, warp 1 = MMA issuer (and tensor-memory owner),
// warps 2..9 = epilogue (two warps per 32-lane quarter, each owning 128 accumulator columns).
// Every wait on an mbarrier is bounded; when one runs out the kernel raises CAFEQ_ERR_TIMEOUT in the status
// word, all roles leave their loops, tensor memory is released and the kernel returns.
#pragma once

#include <atomic>
#include <mutex>
#include <string.h>

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "cafeq.h"
#include "kernels_generic.cuh"

namespace cafeq {

enum { BD_IN = 0, BD_OUT = 1 };
enum { EPI_ABSMAX = 1, EPI_DELTA = 2, EPI_CODES = 4, EPI_SQSUM = 8, EPI_SURR = 16, EPI_STORE = 32 };

struct BdParams {
  int d_out, d_in;     // shape of X
  int r;               // matrix blocks per operator block
  int n_major;         // IN: tile columns (256 d_in columns each); OUT: row blocks (k rows each)
  int n_minor;         // IN: row tiles of 128; OUT: column tiles of NC
  int ctas_per_major;
  int epi;
  float qmax;
  // per (row, group) records are stored GROUP-MAJOR: index = group * d_out + row
  float* a;            // [d_in / G, d_out] group absmax
  float* usel;         // signed value at the arg-max
  int* idx;            // arg-max position inside the group
  uint16_t* delta;     // bf16 [d_out, d_in], row stride d_in (EPI_STORE: U itself is written here instead of the residual)
  uint16_t* delta_lo;  // optional second bf16 term of the residual (delta + delta_lo carries 16 mantissa bits)
  int8_t* codes;       // [d_out, d_in]
  float* scales;       // [d_out, d_in / G]
  double* sqacc;
  // EPI_SURR: Eq. 4 evaluated per entry inside the pass
  const float* cw;     // input axis: sum of c_t over each column group [d_in / G]; output axis: G * c_t per row [d_out]
  float kappa;
  float* coef;         // [d_in / G, d_out] (group-major) backward coefficient 2 kappa cw a sign(U at arg-max); may be null
  double* lossacc;     // += kappa * sum cw a^2
  int a_always;        // write the maxima and their signed values even in EPI_SURR mode
  float* Aacc;         // input axis: [d_in / G] += a^2 per column group; output axis: [nbT * k] += G * sum_G a^2 per operator row
  float* vmax;         // optional: atomic maximum (bit pattern of a non-negative float) of |coef| when coefficients are
                       // written, of the group maxima otherwise
  int32_t* status;
};

// Several matrices in one launch (the problems of a layer are independent): the tiles of all sub-problems form one
// list, sub-problem s owning [tile_end[s-1], tile_end[s]), and every persistent CTA takes a contiguous run of it.
constexpr int BD_MAX_SUB = 8;
struct BdMaps {
  CUtensorMap x[BD_MAX_SUB];  // the matrices
  CUtensorMap t[BD_MAX_SUB];  // their operator blocks
};
struct BdMulti {
  int n;
  int tile_end[BD_MAX_SUB];
  BdParams p[BD_MAX_SUB];     // all share one status word
};

constexpr int BD_THREADS = 320;
constexpr int BD_STAGE_BYTES = 16384;  // one TMA box: 64 columns x 128 rows of bf16
constexpr int BD_STAGES_PER_TILE = 4;
constexpr uint64_t BD_WAIT_NS = 2000000000ull;

// ------------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait: false when the limit ran out here or in another role (abort flag).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                          uint64_t limit_ns = BD_WAIT_NS) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  for (uint32_t spin = 0;; ++spin) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spin & 63u) == 63u) {
      if (*abort_flag) return false;
      if (global_timer_ns() - t0 > limit_ns) {
        *abort_flag = 1;
        raise_status(status, CAFEQ_ERR_TIMEOUT);
        return false;
      }
      __nanosleep(32);
    }
  }
}

// Self-test of the bounded wait: one thread waits, with the given limit, on a barrier phase that nobody completes
// (expected: the wait gives up, raises CAFEQ_ERR_TIMEOUT and sets the abort flag), then completes that phase itself
// and waits again (expected: success).  result[0] = 1 when the first wait gave up, result[1] = 1 when the second
// succeeded.  Nothing here can block: both waits are bounded and the only arrival is the thread's own.
__global__ void wait_probe_kernel(uint64_t limit_ns, int32_t* status, int* result) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const bool first = mbar_wait(smem_u32(&bar), 0, &abort_flag, status, limit_ns);
    result[0] = first ? 0 : 1;
    abort_flag = 0;
    mbar_arrive(smem_u32(&bar));
    const bool second = mbar_wait(smem_u32(&bar), 0, &abort_flag, nullptr, 1000000000ull);
    result[1] = second ? 1 : 0;
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tc_mma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}

__device__ __forceinline__ void tc_ld32(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// The same load without the wait, and a wait that names the destination registers so that no use of them can be
// scheduled ahead of it: lets the load of the next 32 columns overlap the arithmetic on the current ones.
__device__ __forceinline__ void tc_ld32_issue(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
__device__ __forceinline__ void tc_ld_wait32(float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),
                 "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]),
                 "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]),
                 "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
               :
               : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle, rows of 128 bytes, 8-row groups 1024 bytes apart.
// K-major operands step along K by moving the start address inside the swizzled row; MN-major operands
// step along K by whole 8-row groups.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t saddr) {
  uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;              // leading byte offset (unused: one swizzle chunk along the leading dim)
  d |= (uint64_t)(1024 >> 4) << 32;    // stride byte offset: next 8-row group
  d |= (uint64_t)1 << 46;              // descriptor version of this architecture
  d |= (uint64_t)2 << 61;              // SWIZZLE_128B
  return d;
}

// Same, for an MN-major operand that spans several 64-element swizzle atoms along MN: `lbo_bytes` is the distance
// between consecutive atoms.
__device__ __forceinline__ uint64_t umma_desc_sw128_lbo(uint32_t saddr, uint32_t lbo_bytes) {
  uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

__host__ __device__ constexpr uint32_t umma_idesc_bf16(int M, int N, int a_mn_major, int b_mn_major) {
  return (1u << 4) /* fp32 accumulate */ | (1u << 7) /* A bf16 */ | (1u << 10) /* B bf16 */ |
         ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(M >> 4) << 24);
}

// ------------------------------------------------------------------------------------------------
// the kernel
// ------------------------------------------------------------------------------------------------
template <int FORM, int K, int G>
struct BdCfg {
  static constexpr int NBLK = (FORM == BD_IN) ? 256 / K : 1;          // operator blocks resident per CTA
  static constexpr int T_BYTES = NBLK * K * K * 2;
  static constexpr int KH = (K >= 128) ? K / 128 : 1;                 // OUT: 128-row halves of the block
  static constexpr int NC = 256 / KH;                                 // OUT: d_in columns per tile
  static constexpr int NCC = NC / 64;                                 // OUT: 64-column chunks per tile
  static constexpr int NSTAGE = 6;                                    // even: the output-axis form consumes stages in pairs
  static constexpr int SMEM = 1024 + T_BYTES + NSTAGE * BD_STAGE_BYTES + 256;
};

// The body takes the CTA's index and the number of CTAs that share its tile list, so that one launch can run two
// lists side by side (bd_pass_dual_kernel below).
template <int FORM, int K, int G>
__device__ __forceinline__ void bd_pass_body(const BdMaps& maps, const BdMulti& mp, const int cta, const int ncta) {
  using C = BdCfg<FORM, K, G>;
  static_assert(K == 64 || K == 128 || K == 256, "block size");
  static_assert(FORM == BD_IN || K >= 128, "output-axis form needs k >= 128");
  static_assert(G == 64 || G == 128, "group size");
  int32_t* const status = mp.p[0].status;
  if (status && *status) return;

  // persistent CTA: a contiguous run of tiles in (sub-problem, major, minor) order; the operator block is reloaded
  // when the run crosses into the next major or the next sub-problem
  const int total_tiles = mp.tile_end[mp.n - 1];
  const int t_begin = (int)(((long long)cta * total_tiles) / ncta);
  const int t_end = (int)(((long long)(cta + 1) * total_tiles) / ncta);
  if (t_begin >= t_end) return;
  int s_first = 0;
  while (mp.tile_end[s_first] <= t_begin) ++s_first;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* sT = smem;
  uint8_t* sStage = smem + C::T_BYTES;
  uint64_t* bars = (uint64_t*)(sStage + C::NSTAGE * BD_STAGE_BYTES);
  // barrier slots: full[NSTAGE], empty[NSTAGE], tfull[4] (one per 64-column chunk of the operator: the products on the
  // first stage of a new block start when a quarter of it has arrived), accf[2], acce[2], tfree
  const uint32_t bar_full = smem_u32(bars);
  const uint32_t bar_empty = bar_full + 8 * C::NSTAGE;
  const uint32_t bar_tfull = bar_empty + 8 * C::NSTAGE;
  const uint32_t bar_accf = bar_tfull + 32;
  const uint32_t bar_acce = bar_accf + 16;
  const uint32_t bar_tfree = bar_acce + 16;
  uint32_t* tmem_slot = (uint32_t*)(bars + 2 * C::NSTAGE + 9);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    tma_prefetch_desc(&maps.x[s_first]);
    tma_prefetch_desc(&maps.t[s_first]);
    for (int s = 0; s < C::NSTAGE; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int c = 0; c < 4; ++c) mbar_init(bar_tfull + 8 * c, 1);
    mbar_init(bar_tfree, 1);
    mbar_init(bar_accf, 1);
    mbar_init(bar_accf + 8, 1);
    mbar_init(bar_acce, 8);
    mbar_init(bar_acce + 8, 8);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      uint32_t it = 0, tloads = 0;
      bool ok = true;
      for (int sub = s_first; sub < mp.n && ok; ++sub) {
        const int base = sub ? mp.tile_end[sub - 1] : 0;
        if (base >= t_end) break;
        const BdParams& p = mp.p[sub];
        const CUtensorMap* tmX = &maps.x[sub];
        const CUtensorMap* tmT = &maps.t[sub];
        const int lo = (t_begin > base ? t_begin : base) - base;
        const int hi = (t_end < mp.tile_end[sub] ? t_end : mp.tile_end[sub]) - base;
        int cur_major = -1;
        for (int tile = lo; tile < hi && ok; ++tile) {
          const int major = tile / p.n_minor, t = tile - major * p.n_minor;
          if (major != cur_major) {
            // the products of the previous operator block must have finished reading it
            if (tloads > 0 && !mbar_wait(bar_tfree, (tloads - 1) & 1u, abort_flag, status)) { ok = false; break; }
            for (int bi = 0; bi < C::NBLK; ++bi) {
              const int tb = (FORM == BD_IN) ? (major * C::NBLK + bi) / p.r : major / p.r;
              for (int ci = 0; ci < K / 64; ++ci) {
                const uint32_t bq = bar_tfull + 8 * (bi * (K / 64) + ci);  // at most four chunks: NBLK * K = 256 or NBLK = 1
                mbar_expect_tx(bq, K * 128);
                tma_load_2d(smem_u32(sT + bi * K * K * 2 + ci * K * 128), tmT, ci * 64, tb * K, bq);
              }
            }
            cur_major = major;
            ++tloads;
          }
          for (int sidx = 0; sidx < BD_STAGES_PER_TILE; ++sidx, ++it) {
            const uint32_t s = it % C::NSTAGE, ph = (it / C::NSTAGE) & 1u;
            if (!mbar_wait(bar_empty + 8 * s, ph ^ 1u, abort_flag, status)) { ok = false; break; }
            mbar_expect_tx(bar_full + 8 * s, BD_STAGE_BYTES);
            int x, y;
            if constexpr (FORM == BD_IN) {
              x = major * 256 + sidx * 64;
              y = t * 128;
            } else {
              const int kh = sidx / C::NCC, nc = sidx % C::NCC;  // the chunks of one row half are consecutive stages
              x = t * C::NC + nc * 64;
              y = major * K + kh * 128;
            }
            tma_load_2d(smem_u32(sStage + s * BD_STAGE_BYTES), tmX, x, y, bar_full + 8 * s);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      bool ok = true;
      uint32_t tfulls = 0;
      constexpr uint32_t idesc_in = umma_idesc_bf16(128, K, 0, 0);
      constexpr uint32_t idesc_out = umma_idesc_bf16(128, 128, 0, 1);
      const uint32_t sT_u = smem_u32(sT), sSt_u = smem_u32(sStage);
      uint32_t it = 0, tl = 0;
      for (int sub = s_first; sub < mp.n && ok; ++sub) {
        const int base = sub ? mp.tile_end[sub - 1] : 0;
        if (base >= t_end) break;
        const int n_minor = mp.p[sub].n_minor;
        const int lo = (t_begin > base ? t_begin : base) - base;
        const int hi = (t_end < mp.tile_end[sub] ? t_end : mp.tile_end[sub]) - base;
        int cur_major = -1;
        for (int tile = lo; tile < hi && ok; ++tile, ++tl) {
          const int major = tile / n_minor;
          const bool fresh = major != cur_major;  // first tile on a newly loaded operator block
          const uint32_t tph = tfulls & 1u;
          if (fresh) {
            if constexpr (FORM == BD_OUT) {
              for (int c = 0; c < K / 64 && ok; ++c) ok = mbar_wait(bar_tfull + 8 * c, tph, abort_flag, status);
              if (!ok) break;
            }
            ++tfulls;
            cur_major = major;
          }
          const uint32_t buf = tl & 1u, aph = (tl >> 1) & 1u;
          if (!mbar_wait(bar_acce + 8 * buf, aph ^ 1u, abort_flag, status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t dbase = tmem_base + buf * 256u;
          if constexpr (FORM == BD_IN) {
            for (int sidx = 0; sidx < BD_STAGES_PER_TILE; ++sidx, ++it) {
              const uint32_t s = it % C::NSTAGE, ph = (it / C::NSTAGE) & 1u;
              if (!mbar_wait(bar_full + 8 * s, ph, abort_flag, status)) { ok = false; break; }
              // stage sidx multiplies the operator's chunk sidx
              if (fresh && !mbar_wait(bar_tfull + 8 * sidx, tph, abort_flag, status)) { ok = false; break; }
              tc_fence_after();
              const uint32_t stage = sSt_u + s * BD_STAGE_BYTES;
              const int bi = (sidx * 64) / K, ci = ((sidx * 64) % K) / 64;
#pragma unroll
              for (int kk = 0; kk < 4; ++kk) {
                const uint64_t ad = umma_desc_sw128(stage + kk * 32);
                const uint64_t bd = umma_desc_sw128(sT_u + bi * K * K * 2 + ci * K * 128 + kk * 32);
                tc_mma_bf16(dbase + bi * K, ad, bd, idesc_in, (ci | kk) != 0 ? 1u : 0u);
              }
              tc_commit(bar_empty + 8 * s);
            }
          } else {
            // two consecutive stages = two 64-column chunks of the same 128 weight rows: one N = 128 product, the
            // second swizzle atom of the MN-major operand one stage further on
            for (int sidx = 0; sidx < BD_STAGES_PER_TILE; sidx += 2, it += 2) {
              const uint32_t s = it % C::NSTAGE, ph = (it / C::NSTAGE) & 1u;
              if (!mbar_wait(bar_full + 8 * s, ph, abort_flag, status)) { ok = false; break; }
              if (!mbar_wait(bar_full + 8 * (s + 1), ph, abort_flag, status)) { ok = false; break; }
              tc_fence_after();
              const uint32_t stage = sSt_u + s * BD_STAGE_BYTES;
              const int kh = sidx / C::NCC, nc = sidx % C::NCC;
#pragma unroll
              for (int ks = 0; ks < 8; ++ks) {
                const uint64_t bd = umma_desc_sw128_lbo(stage + ks * 2048, BD_STAGE_BYTES);
#pragma unroll
                for (int mh = 0; mh < C::KH; ++mh) {
                  const uint64_t ad = umma_desc_sw128(sT_u + (kh * 2 + ks / 4) * K * 128 + mh * 128 * 128 + (ks % 4) * 32);
                  tc_mma_bf16(dbase + mh * C::NC + nc * 64, ad, bd, idesc_out, (kh | ks) != 0 ? 1u : 0u);
                }
              }
              tc_commit(bar_empty + 8 * s);
              tc_commit(bar_empty + 8 * (s + 1));
            }
          }
          if (ok) tc_commit(bar_accf + 8 * buf);
          // last tile of this operator block with more to come: signal when its products are done with the block
          if (ok && base + tile + 1 < t_end && (tile + 1 == hi || (tile + 1) / n_minor != major)) tc_commit(bar_tfree);
        }
      }
    }
  } else {
    // ---------------------------------------------------------------- epilogue
    const int q = warp & 3, hw = (warp - 2) >> 2;
    const int L = q * 32 + lane;
    uint32_t tl = 0;
    bool ok = true;
    constexpr int NG = 128 / G;
    for (int sub = s_first; sub < mp.n && ok; ++sub) {
    const int base = sub ? mp.tile_end[sub - 1] : 0;
    if (base >= t_end) break;
    const BdParams& p = mp.p[sub];
    const int lo = (t_begin > base ? t_begin : base) - base;
    const int hi = (t_end < mp.tile_end[sub] ? t_end : mp.tile_end[sub]) - base;
    double sq_local = 0.0, sur_local = 0.0;
    float srow = 0.f, vm = 0.f;
    int srow_row = -1;
    bool bad = false;
    const int ng_row = p.d_in / G;
    for (int tile = lo; tile < hi && ok; ++tile, ++tl) {
      const int major = tile / p.n_minor, t = tile - major * p.n_minor;
      const uint32_t buf = tl & 1u, aph = (tl >> 1) & 1u;
      int row, col0;
      if constexpr (FORM == BD_IN) {
        row = t * 128 + L;
        col0 = major * 256 + hw * 128;
      } else if constexpr (K == 256) {
        row = major * 256 + hw * 128 + L;
        col0 = t * 128;
      } else {
        row = major * 128 + L;
        col0 = t * 256 + hw * 128;
      }
      // Eq. 4 weights of this thread's groups, requested before the wait for the accumulator so that the
      // global-memory latency is hidden behind it
      float wgt[NG];
#pragma unroll
      for (int gi = 0; gi < NG; ++gi) wgt[gi] = 0.f;
      if ((p.epi & EPI_SURR) && row < p.d_out && col0 < p.d_in) {
#pragma unroll
        for (int gi = 0; gi < NG; ++gi) wgt[gi] = (FORM == BD_IN) ? __ldg(p.cw + col0 / G + gi) : __ldg(p.cw + row);
      }
      ok = mbar_wait(bar_accf + 8 * buf, aph, abort_flag, status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * 256u + hw * 128u;
      const bool valid = (row < p.d_out) && (col0 < p.d_in);
      float v[32];
      float best[NG], bval[NG];
      int bidx[NG];
#pragma unroll
      for (int gi = 0; gi < NG; ++gi) { best[gi] = -1.f; bval[gi] = 0.f; bidx[gi] = 0; }
      if (p.epi == EPI_STORE) {
        // the transformed matrix itself, rounded to bf16 (inference-side apply of a block-diagonal operator)
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          tc_ld32(taddr + ch * 32, v);
          uint32_t pk[16];
#pragma unroll
          for (int e = 0; e < 32; e += 2)
            pk[e >> 1] = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v[e])) |
                         ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v[e + 1])) << 16);
          if (valid) {
            uint4* dst = reinterpret_cast<uint4*>(p.delta + (long long)row * p.d_in + col0 + ch * 32);
#pragma unroll
            for (int w4 = 0; w4 < 4; ++w4) dst[w4] = make_uint4(pk[4 * w4], pk[4 * w4 + 1], pk[4 * w4 + 2], pk[4 * w4 + 3]);
          }
        }
      } else if (p.epi == EPI_SQSUM) {
        // sum of squares only (second pass of the l2 proxy)
        float sq4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          tc_ld32(taddr + ch * 32, v);
#pragma unroll
          for (int e = 0; e < 32; ++e) sq4[e & 3] = fmaf(v[e], v[e], sq4[e & 3]);
        }
        sq_local += valid ? (double)((sq4[0] + sq4[1]) + (sq4[2] + sq4[3])) : 0.0;
      } else {
        // group absmax with arg-max: four independent running candidates per group (columns e mod 4), merged at
        // the end with the lowest index winning ties; the next 32 columns are in flight while these are compared
        float v2[32];
        float bv[NG][4], nz[4] = {0.f, 0.f, 0.f, 0.f};
        int bi[NG][4];
#pragma unroll
        for (int gi = 0; gi < NG; ++gi)
#pragma unroll
          for (int c = 0; c < 4; ++c) { bv[gi][c] = 0.f; bi[gi][c] = 0; }
        tc_ld32_issue(taddr, v);
        tc_ld_wait32(v);
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          float* cur = (ch & 1) ? v2 : v;
          float* nxt = (ch & 1) ? v : v2;
          if (ch < 3) tc_ld32_issue(taddr + (ch + 1) * 32, nxt);
          const int gi = (G == 128) ? 0 : (ch >> 1);
          const int e0 = (G == 128) ? ch * 32 : (ch & 1) * 32;
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const int c = e & 3;
            if (fabsf(cur[e]) > fabsf(bv[gi][c])) { bv[gi][c] = cur[e]; bi[gi][c] = e0 + e; }
            nz[c] = fmaf(cur[e], 0.f, nz[c]);  // stays 0 unless a NaN or an infinity passes by
          }
          if (ch < 3) tc_ld_wait32(nxt);
        }
#pragma unroll
        for (int gi = 0; gi < NG; ++gi) {
          float b = bv[gi][0];
          int ix = bi[gi][0];
#pragma unroll
          for (int c = 1; c < 4; ++c) {
            const float x = bv[gi][c];
            const int jx = bi[gi][c];
            const bool take = (fabsf(x) > fabsf(b)) || (fabsf(x) == fabsf(b) && jx < ix);
            if (take) { b = x; ix = jx; }
          }
          best[gi] = fabsf(b);
          bval[gi] = b;
          bidx[gi] = ix;
        }
        if (valid && !((nz[0] + nz[1]) + (nz[2] + nz[3]) == 0.f)) bad = true;
      }
      // Without a second pass over the accumulator (codes / residual) everything still needed is in registers:
      // hand the buffer back to the tensor cores now.  The arrive has release semantics, so issuing it after the
      // global stores below would make every tile wait for those stores to land.
      const bool early_release = (p.epi & (EPI_DELTA | EPI_CODES)) == 0;
      if (early_release) {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_acce + 8 * buf);
      }
      if (p.epi & (EPI_ABSMAX | EPI_DELTA | EPI_CODES)) {
#pragma unroll
        for (int gi = 0; gi < NG; ++gi)
          if (valid && !(best[gi] <= 3.0e38f)) bad = true;
        if (valid && p.vmax && !((p.epi & EPI_SURR) && p.coef)) {
#pragma unroll
          for (int gi = 0; gi < NG; ++gi) vm = fmaxf(vm, best[gi]);
        }
        if (valid && (p.epi & EPI_ABSMAX)) {
          // with Eq. 4 evaluated right here nothing downstream reads the maxima or their signs: the backward only
          // needs (arg-max index, coefficient).  Every scattered 4-byte store is a partial-sector write at L2.
          const bool need_a = !(p.epi & EPI_SURR) || p.a_always;
#pragma unroll
          for (int gi = 0; gi < NG; ++gi) {
            // group-major records: consecutive rows of one group are contiguous, so a warp's store is one line
            const long long w = (long long)(col0 / G + gi) * p.d_out + row;
            if (need_a) {
              p.a[w] = best[gi];
              p.usel[w] = bval[gi];
            }
            p.idx[w] = bidx[gi];
          }
        }
        if (p.epi & EPI_SURR) {
          float surf = 0.f;
          if constexpr (FORM == BD_OUT) {
            // the run of tiles moved on to another row block: hand over what this thread summed for its old row
            if (valid && srow_row >= 0 && srow_row != row) {
              if (srow != 0.f) {
                const int Bq = srow_row / K;
                atomicAdd(&p.Aacc[(Bq / p.r) * K + (srow_row - Bq * K)], (float)G * srow);
              }
              srow = 0.f;
            }
          }
#pragma unroll
          for (int gi = 0; gi < NG; ++gi) {
            const int Gc = col0 / G + gi;
            const float av = valid ? best[gi] : 0.f;
            surf = fmaf(wgt[gi] * av, av, surf);
            if (valid && p.coef) {
              const float sg = (bval[gi] > 0.f) ? 1.f : ((bval[gi] < 0.f) ? -1.f : 0.f);
              const float cf = 2.f * p.kappa * wgt[gi] * av;
              p.coef[(long long)Gc * p.d_out + row] = cf * sg;
              vm = fmaxf(vm, cf);
            }
            if constexpr (FORM == BD_IN) {
              float a2 = av * av;
              for (int o = 16; o > 0; o >>= 1) a2 += __shfl_xor_sync(0xffffffffu, a2, o);
              if (lane == 0 && a2 != 0.f && col0 < p.d_in) atomicAdd(&p.Aacc[Gc], a2);
            } else {
              srow = fmaf(av, av, srow);
            }
          }
          sur_local += (double)surf;
          if (valid) srow_row = row;
        }
        if (p.epi & (EPI_DELTA | EPI_CODES)) {
          float sc[NG];
#pragma unroll
          for (int gi = 0; gi < NG; ++gi) {
            sc[gi] = __fdiv_rn(best[gi], p.qmax);
            if (valid && (p.epi & EPI_CODES)) p.scales[(long long)row * ng_row + (col0 / G + gi)] = sc[gi];
          }
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            tc_ld32(taddr + ch * 32, v);
            const float s = sc[(G == 128) ? 0 : (ch >> 1)];
            uint32_t dpk[16], lpk[16];
            uint32_t cpk[8];
            // the flags are uniform over the launch: only the outputs that were asked for are formed
            const bool want_d = (p.epi & EPI_DELTA) != 0, want_dl = want_d && p.delta_lo != nullptr;
            const bool want_c = (p.epi & EPI_CODES) != 0;
            // code = rne(fl32(u / s)).  The IEEE division is a long dependent sequence with a slow-path branch per
            // element; u * (1 / s) differs from the exact quotient by less than 1.5 ulp, and from fl32(u / s) by
            // less than 2 ulp, i.e. by less than (qmax + 1) * 2.4e-7, so it rounds to the same integer unless the
            // quotient lies within that distance of a half-integer: those (rare: the transformed values are not on a
            // coarse grid) chunks are redone with the division.
            // The rounding itself uses no conversion instruction: t = x + 1.5 * 2^23 holds rne(x) in its low mantissa
            // bits (the fp32 add rounds to nearest even, as rintf does) and, 0x4B400000 having a zero low byte, the low
            // byte of t's pattern is the two's-complement code; |x| <= qmax (1 + 3 * 2^-23), so nothing is clamped.
            float qv[32];
            uint32_t cb[32];
            {
              constexpr float MAGIC = 12582912.f;
              const float rs = (s > 0.f) ? __frcp_rn(s) : 0.f;
              const uint32_t winb = __float_as_uint(0.5f - (p.qmax + 1.f) * 1.0e-6f);
              uint32_t dmax = 0u;  // largest |x - rne(x)| of the chunk, as a bit pattern
#pragma unroll
              for (int e = 0; e < 32; ++e) {
                const float x = v[e] * rs;
                const float t = x + MAGIC;
                qv[e] = t - MAGIC;
                cb[e] = __float_as_uint(t);
                dmax = max(dmax, __float_as_uint(x - qv[e]) & 0x7FFFFFFFu);
              }
              // (also: a scale so small that its reciprocal overflows)
              if (dmax > winb || !(rs < 3.0e38f)) {
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                  float q = (s > 0.f) ? rintf(__fdiv_rn(v[e], s)) : 0.f;
                  q = fminf(fmaxf(q, -p.qmax), p.qmax);
                  qv[e] = q;
                  cb[e] = (uint32_t)((int)q);
                }
              }
            }
            if (want_d) {
#pragma unroll
              for (int e = 0; e < 32; e += 2) {
                const float d0 = s * qv[e] - v[e], d1 = s * qv[e + 1] - v[e + 1];
                const __nv_bfloat16 b0 = __float2bfloat16_rn(d0), b1 = __float2bfloat16_rn(d1);
                dpk[e >> 1] = (uint32_t)__bfloat16_as_ushort(b0) | ((uint32_t)__bfloat16_as_ushort(b1) << 16);
                if (want_dl)
                  lpk[e >> 1] = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(d0 - __bfloat162float(b0))) |
                                ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(d1 - __bfloat162float(b1))) << 16);
              }
            }
            if (want_c) {
#pragma unroll
              for (int w = 0; w < 8; ++w)
                cpk[w] = __byte_perm(__byte_perm(cb[4 * w], cb[4 * w + 1], 0x0040), __byte_perm(cb[4 * w + 2], cb[4 * w + 3], 0x0040), 0x5410);
            }
            if (valid && (p.epi & EPI_DELTA)) {
              uint4* dst = reinterpret_cast<uint4*>(p.delta + (long long)row * p.d_in + col0 + ch * 32);
#pragma unroll
              for (int w4 = 0; w4 < 4; ++w4) dst[w4] = make_uint4(dpk[4 * w4], dpk[4 * w4 + 1], dpk[4 * w4 + 2], dpk[4 * w4 + 3]);
              if (p.delta_lo) {
                uint4* dl = reinterpret_cast<uint4*>(p.delta_lo + (long long)row * p.d_in + col0 + ch * 32);
#pragma unroll
                for (int w4 = 0; w4 < 4; ++w4) dl[w4] = make_uint4(lpk[4 * w4], lpk[4 * w4 + 1], lpk[4 * w4 + 2], lpk[4 * w4 + 3]);
              }
            }
            if (valid && (p.epi & EPI_CODES)) {
              uint4* dst = reinterpret_cast<uint4*>(p.codes + (long long)row * p.d_in + col0 + ch * 32);
              dst[0] = make_uint4(cpk[0], cpk[1], cpk[2], cpk[3]);
              dst[1] = make_uint4(cpk[4], cpk[5], cpk[6], cpk[7]);
            }
          }
        }
      }
      if (!early_release) {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_acce + 8 * buf);
      }
    }
    if (p.epi & EPI_SQSUM) {
      for (int o = 16; o > 0; o >>= 1) sq_local += __shfl_xor_sync(0xffffffffu, sq_local, o);
      if (lane == 0 && sq_local != 0.0) atomicAdd(p.sqacc, sq_local);
    }
    if (p.epi & EPI_SURR) {
      for (int o = 16; o > 0; o >>= 1) sur_local += __shfl_xor_sync(0xffffffffu, sur_local, o);
      if (lane == 0 && sur_local != 0.0) atomicAdd(p.lossacc, (double)p.kappa * sur_local);
      if constexpr (FORM == BD_OUT) {
        if (srow_row >= 0 && srow != 0.f) {
          const int Bq = srow_row / K;
          atomicAdd(&p.Aacc[(Bq / p.r) * K + (srow_row - Bq * K)], (float)G * srow);
        }
      }
    }
    if (p.vmax) {
      for (int o = 16; o > 0; o >>= 1) vm = fmaxf(vm, __shfl_xor_sync(0xffffffffu, vm, o));
      if (lane == 0 && vm > 0.f) atomicMax(reinterpret_cast<int*>(p.vmax), __float_as_int(vm));
    }
    if (__any_sync(0xffffffffu, bad) && lane == 0) raise_status(status, CAFEQ_ERR_NONFINITE);
    }  // sub-problems
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

template <int FORM, int K, int G>
__global__ void __launch_bounds__(BD_THREADS, 1)
bd_pass_kernel(const __grid_constant__ BdMaps maps, const __grid_constant__ BdMulti mp) {
  bd_pass_body<FORM, K, G>(maps, mp, (int)blockIdx.x, (int)gridDim.x);
}

// Both forms in one launch: the first n_in CTAs run the input-axis list, the others the output-axis list (a layer
// has matrices of both forms; two launches pay the fixed cost of a persistent kernel -- operator load, pipeline
// fill, the tail of the slowest CTA -- twice, and the smaller list alone cannot fill the memory system).
template <int K, int G>
__global__ void __launch_bounds__(BD_THREADS, 1)
bd_pass_dual_kernel(const __grid_constant__ BdMaps maps_in, const __grid_constant__ BdMulti mp_in,
                    const __grid_constant__ BdMaps maps_out, const __grid_constant__ BdMulti mp_out, const int n_in) {
  if ((int)blockIdx.x < n_in) bd_pass_body<BD_IN, K, G>(maps_in, mp_in, (int)blockIdx.x, n_in);
  else bd_pass_body<BD_OUT, K, G>(maps_out, mp_out, (int)blockIdx.x - n_in, (int)gridDim.x - n_in);
}

// ------------------------------------------------------------------------------------------------
// host side: tensor maps and launch
// ------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_tiled() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)ptr;
  });
  return fn;
}

// 2-D bf16 tensor map: `cols` contiguous elements per row, `rows` rows, row pitch in elements, box 64 x box_rows,
// 128-byte swizzle, out-of-range elements read as zero.
static bool make_map_bf16(CUtensorMap* m, const void* base, long long cols, long long rows, long long pitch, int box_rows) {
  EncodeTiledFn enc = get_encode_tiled();
  if (!enc) return false;
  if (((uintptr_t)base & 15) || ((pitch * 2) & 15)) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)pitch * 2};
  cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Shapes the fused pass covers; everything else runs on the shape-agnostic kernels.
static bool bd_supported(int form, int d_out, int d_in, long long ld, int k, int g, const void* X) {
  if (!(g == 64 || g == 128)) return false;
  if (form == BD_IN) {
    if (!(k == 64 || k == 128 || k == 256)) return false;
    if (d_in % 256) return false;
  } else {
    if (!(k == 128 || k == 256)) return false;
    if (d_out % k || d_in % 128) return false;
  }
  if ((ld % 8) || ((uintptr_t)X & 15)) return false;
  return true;
}

static std::atomic<int> g_bd_min_tiles{1};

// opt the kernel into its dynamic shared memory once per device (the attribute is per device and per function)
template <typename KernelT>
static bool opt_in_smem(KernelT kernel, int bytes, std::atomic<unsigned long long>& done_mask) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  const unsigned long long bit = 1ull << (dev & 63);
  if (done_mask.load(std::memory_order_acquire) & bit) return true;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
  done_mask.fetch_or(bit, std::memory_order_release);
  return true;
}

// tile geometry of one sub-problem
template <int FORM, int K, int G>
static void bd_fill_tiles(BdParams& p) {
  using C = BdCfg<FORM, K, G>;
  if (FORM == BD_IN) {
    p.n_major = p.d_in / 256;
    p.n_minor = (p.d_out + 127) / 128;
  } else {
    p.n_major = p.d_out / K;
    p.n_minor = (p.d_in + C::NC - 1) / C::NC;
  }
  p.ctas_per_major = 0;
}

template <int FORM, int K, int G>
static int bd_launch_multi_t(cudaStream_t st, const BdMaps& maps, BdMulti mp, int min_tiles) {
  using C = BdCfg<FORM, K, G>;
  static std::atomic<unsigned long long> done{0};
  if (!opt_in_smem(bd_pass_kernel<FORM, K, G>, C::SMEM, done)) return CAFEQ_ERR_CUDA;
  long long total = 0;
  for (int s = 0; s < mp.n; ++s) {
    bd_fill_tiles<FORM, K, G>(mp.p[s]);
    total += (long long)mp.p[s].n_major * mp.p[s].n_minor;
    mp.tile_end[s] = (int)total;
  }
  for (int s = mp.n; s < BD_MAX_SUB; ++s) mp.tile_end[s] = (int)total;
  // one persistent CTA per SM at most; when several problems overlap in streams, small matrices take fewer CTAs
  // (at least min_tiles tiles each): the fixed cost of a CTA is spread over more tiles and the SMs left over
  // run another problem's kernel
  long long want = total / (min_tiles > 0 ? min_tiles : 1);
  if (want < 1) want = 1;
  const int grid = want < 148 ? (int)want : 148;
  bd_pass_kernel<FORM, K, G><<<grid, BD_THREADS, C::SMEM, st>>>(maps, mp);
  return CAFEQ_OK;
}

static int bd_dispatch(cudaStream_t st, int form, int k, int g, const BdMaps& maps, const BdMulti& mp, int min_tiles) {
#define BD_CASE(F, KK, GG) \
  if (form == F && k == KK && g == GG) return bd_launch_multi_t<F, KK, GG>(st, maps, mp, min_tiles);
  BD_CASE(BD_IN, 64, 64)
  BD_CASE(BD_IN, 64, 128)
  BD_CASE(BD_IN, 128, 64)
  BD_CASE(BD_IN, 128, 128)
  BD_CASE(BD_IN, 256, 64)
  BD_CASE(BD_IN, 256, 128)
  BD_CASE(BD_OUT, 128, 64)
  BD_CASE(BD_OUT, 128, 128)
  BD_CASE(BD_OUT, 256, 64)
  BD_CASE(BD_OUT, 256, 128)
#undef BD_CASE
  return CAFEQ_ERR_UNSUPPORTED;
}

// X: bf16 [d_out, d_in] with pitch ld; Tb: bf16 operator blocks [nbT * k, k] in applied orientation.
static int bd_launch(cudaStream_t st, int form, int k, int g, const void* X, long long ld, const void* Tb, int nbT, BdParams p) {
  BdMaps maps;
  BdMulti mp;
  memset(&mp, 0, sizeof(mp));
  if (!make_map_bf16(&maps.x[0], X, p.d_in, p.d_out, ld, 128)) return CAFEQ_ERR_UNSUPPORTED;
  if (!make_map_bf16(&maps.t[0], Tb, k, (long long)nbT * k, k, k)) return CAFEQ_ERR_UNSUPPORTED;
  for (int s = 1; s < BD_MAX_SUB; ++s) { maps.x[s] = maps.x[0]; maps.t[s] = maps.t[0]; }
  mp.n = 1;
  mp.p[0] = p;
  return bd_dispatch(st, form, k, g, maps, mp, g_bd_min_tiles.load(std::memory_order_relaxed));
}

// One sub-problem of a multi-matrix launch: the matrix, its operator blocks (bf16, applied orientation) and its
// epilogue parameters (d_out, d_in, r, epi, ... filled by the caller).
struct BdSub {
  const void* X;
  long long ld;
  const void* Tb;
  int nbT;
  BdParams p;
};

// Up to BD_MAX_SUB matrices of the same form, block size and group size in one persistent launch.
static int bd_launch_many(cudaStream_t st, int form, int k, int g, const BdSub* subs, int n) {
  if (n < 1 || n > BD_MAX_SUB) return CAFEQ_ERR_INVALID_ARG;
  BdMaps maps;
  BdMulti mp;
  memset(&mp, 0, sizeof(mp));
  for (int s = 0; s < n; ++s) {
    if (!make_map_bf16(&maps.x[s], subs[s].X, subs[s].p.d_in, subs[s].p.d_out, subs[s].ld, 128)) return CAFEQ_ERR_UNSUPPORTED;
    if (!make_map_bf16(&maps.t[s], subs[s].Tb, k, (long long)subs[s].nbT * k, k, k)) return CAFEQ_ERR_UNSUPPORTED;
    mp.p[s] = subs[s].p;
  }
  for (int s = n; s < BD_MAX_SUB; ++s) { maps.x[s] = maps.x[0]; maps.t[s] = maps.t[0]; }
  mp.n = n;
  return bd_dispatch(st, form, k, g, maps, mp, 1);
}

// relative cost of an output-axis tile against an input-axis tile of the same bytes (measured per-tile times of
// the two forms): sets how the CTAs of a dual launch are divided
static std::atomic<int> g_dual_pass_pct{130}, g_dual_bwd_pct{80};

static int dual_split(long long tiles_in, long long tiles_out, int out_weight_pct) {
  const double wi = (double)tiles_in, wo = (double)tiles_out * out_weight_pct / 100.0;
  int n_in = (int)(148.0 * wi / (wi + wo) + 0.5);
  if (n_in < 1) n_in = 1;
  if (n_in > 147) n_in = 147;
  return n_in;
}

template <int K, int G>
static int bd_launch_dual_t(cudaStream_t st, const BdMaps& mi, BdMulti pi, const BdMaps& mo, BdMulti po) {
  constexpr int SMEM = BdCfg<BD_IN, K, G>::SMEM > BdCfg<BD_OUT, K, G>::SMEM ? BdCfg<BD_IN, K, G>::SMEM : BdCfg<BD_OUT, K, G>::SMEM;
  static std::atomic<unsigned long long> done{0};
  if (!opt_in_smem(bd_pass_dual_kernel<K, G>, SMEM, done)) return CAFEQ_ERR_CUDA;
  long long ti = 0, to = 0;
  for (int s = 0; s < pi.n; ++s) {
    bd_fill_tiles<BD_IN, K, G>(pi.p[s]);
    ti += (long long)pi.p[s].n_major * pi.p[s].n_minor;
    pi.tile_end[s] = (int)ti;
  }
  for (int s = pi.n; s < BD_MAX_SUB; ++s) pi.tile_end[s] = (int)ti;
  for (int s = 0; s < po.n; ++s) {
    bd_fill_tiles<BD_OUT, K, G>(po.p[s]);
    to += (long long)po.p[s].n_major * po.p[s].n_minor;
    po.tile_end[s] = (int)to;
  }
  for (int s = po.n; s < BD_MAX_SUB; ++s) po.tile_end[s] = (int)to;
  const int n_in = dual_split(ti, to, g_dual_pass_pct.load(std::memory_order_relaxed));
  bd_pass_dual_kernel<K, G><<<148, BD_THREADS, SMEM, st>>>(mi, pi, mo, po, n_in);
  return CAFEQ_OK;
}

// Input-axis and output-axis matrices of one block size and group size in ONE persistent launch (both lists
// non-empty, each at least 148 tiles so that every CTA has work; otherwise the caller launches them separately).
static bool bd_dual_ok(int k, int g) { return (k == 128 || k == 256) && (g == 64 || g == 128); }
static int bd_launch_dual(cudaStream_t st, int k, int g, const BdSub* in, int n_in, const BdSub* out, int n_out) {
  if (n_in < 1 || n_in > BD_MAX_SUB || n_out < 1 || n_out > BD_MAX_SUB || !bd_dual_ok(k, g)) return CAFEQ_ERR_INVALID_ARG;
  BdMaps mi, mo;
  BdMulti pi, po;
  memset(&pi, 0, sizeof(pi));
  memset(&po, 0, sizeof(po));
  for (int s = 0; s < n_in; ++s) {
    if (!make_map_bf16(&mi.x[s], in[s].X, in[s].p.d_in, in[s].p.d_out, in[s].ld, 128)) return CAFEQ_ERR_UNSUPPORTED;
    if (!make_map_bf16(&mi.t[s], in[s].Tb, k, (long long)in[s].nbT * k, k, k)) return CAFEQ_ERR_UNSUPPORTED;
    pi.p[s] = in[s].p;
  }
  for (int s = n_in; s < BD_MAX_SUB; ++s) { mi.x[s] = mi.x[0]; mi.t[s] = mi.t[0]; }
  for (int s = 0; s < n_out; ++s) {
    if (!make_map_bf16(&mo.x[s], out[s].X, out[s].p.d_in, out[s].p.d_out, out[s].ld, 128)) return CAFEQ_ERR_UNSUPPORTED;
    if (!make_map_bf16(&mo.t[s], out[s].Tb, k, (long long)out[s].nbT * k, k, k)) return CAFEQ_ERR_UNSUPPORTED;
    po.p[s] = out[s].p;
  }
  for (int s = n_out; s < BD_MAX_SUB; ++s) { mo.x[s] = mo.x[0]; mo.t[s] = mo.t[0]; }
  pi.n = n_in;
  po.n = n_out;
#define BD_DUAL(KK, GG) \
  if (k == KK && g == GG) return bd_launch_dual_t<KK, GG>(st, mi, pi, mo, po);
  BD_DUAL(128, 64)
  BD_DUAL(128, 128)
  BD_DUAL(256, 64)
  BD_DUAL(256, 128)
#undef BD_DUAL
  return CAFEQ_ERR_UNSUPPORTED;
}

// fp32 operator blocks -> bf16 in applied orientation (transposed when the role asks for T^T)
__global__ void operator_to_bf16_kernel(const float* __restrict__ T, uint16_t* __restrict__ out, int k, long long n, int transpose,
                                        const int32_t* status) {
  if (status && *status) return;
  for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
    long long b = e / ((long long)k * k);
    int i = (int)((e / k) % k), j = (int)(e % k);
    float v = transpose ? T[b * k * k + (long long)j * k + i] : T[e];
    out[e] = __bfloat16_as_ushort(__float2bfloat16_rn(v));
  }
}

}  // namespace cafeq
