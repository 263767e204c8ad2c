// Skinny weight-streaming GEMM on the sm_100a tensor cores (tcgen05 + TMEM, operands by TMA).
//   part[seg][t][n] = sum over a K range of (Xhi[t][k] + Xlo[t][k]) * W[n][k]     (fp32 acc)
// for T <= 128 activation rows: the verification forward over one draft tree and every
// draft-model level. At these sizes the cost is the single pass over W, so the kernel is
// built around keeping every SM's share of that stream in flight:
//
//  * W [N, K] (bf16, K contiguous) is cut into tiles of 256 rows x 64 columns (32 KB, one TMA
//    box, 128-byte swizzle). The tile sits on the MMA's M axis (two M = 128 halves), the
//    activation rows on its N axis (TN = T rounded up to 16/32/64/128). Both bf16 limbs of
//    X are multiplied against the same W tile into the same TMEM accumulator, so fp32-grade
//    activations cost no extra bytes of the weight stream.
//  * The tiles x K-blocks form one linear list of units (tile-major, K inner) that is cut
//    into gridDim.x equal contiguous ranges, one per CTA (one CTA per SM). A CTA therefore
//    covers the end of one tile, some whole tiles and the start of another. A tile covered by
//    one CTA is finished straight from TMEM. Otherwise every (CTA, tile) segment writes its
//    partial sum to plane `seg` = CTA - first CTA of that tile and bumps the tile's counter;
//    the CTA that arrives last adds the planes in ascending order (so the result does not
//    depend on which CTA that is) and finishes the tile. Nobody waits for anybody.
//  * "Finishing" a tile is the fused epilogue: plain store with the RMSNorm row scale, or
//    residual add + gain + two-limb split + sum of squares for the next norm, or SwiGLU.
//  * Warp 0 issues TMA loads into a ring of stages, warp 1 issues the MMAs and releases
//    stages through tcgen05.commit, warps 2-9 run the epilogue on finished accumulators
//    (double-buffered in TMEM).
//  * The weight loads of the first ring-full do not depend on the previous kernel, so they
//    are issued BEFORE griddepcontrol.wait: launched with programmatic stream serialisation
//    the kernel streams weights while its predecessor drains.
//
// Every mbarrier wait is bounded (two seconds of %globaltimer); on expiry the kernel records
// a code in *err, lets copies in flight land, frees its TMEM and returns.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace gemm_tc {

constexpr int BM = SV_TILE_ROWS;          // weight rows per tile (two UMMA halves of 128)
constexpr int BK = 64;                    // K per stage: 128 bytes = one swizzle row
constexpr int THREADS = 320;               // warp 0 TMA, warp 1 MMA, warps 2-9 epilogue
constexpr int W_STAGE_BYTES = BM * BK * 2;
constexpr int RING_BUDGET = 164 * 1024;
constexpr int MAX_T = 128;

__host__ __device__ constexpr int tn_of(int T) { return T <= 16 ? 16 : (T <= 32 ? 32 : (T <= 64 ? 64 : 128)); }
__host__ __device__ constexpr int stage_bytes(int TN) { return W_STAGE_BYTES + 2 * TN * BK * 2; }
// The ring leaves ~60 KB of the SM's shared memory free, so that the small kernels between two
// GEMMs can be resident next to a GEMM CTA while it prefetches weights.
__host__ __device__ constexpr int stages_of(int TN) { return RING_BUDGET / stage_bytes(TN); }
__host__ __device__ constexpr int smem_bytes(int TN) { return stages_of(TN) * stage_bytes(TN) + 1024 + 256; }
// Up to 64 rows both limbs of X form ONE MMA operand (N = 2 TN: hi rows, then lo rows) and the
// two column groups are added in the epilogue; at 128 rows the limbs are two MMAs into the
// same TN columns. Either way an accumulator is acc_width(TN) TMEM columns wide.
__host__ __device__ constexpr bool merged_limbs(int TN) { return TN <= 64; }
__host__ __device__ constexpr int acc_width(int TN) { return merged_limbs(TN) ? 2 * TN : TN; }
__host__ __device__ constexpr int tmem_cols(int TN) { return 4 * acc_width(TN); }      // 128, 256, 512, 512

// tiles: 256-column tiles of the output (for SwiGLU: 128 gate + 128 up columns each).
inline SegPlan make_plan(int tiles, int K, int num_sms) {
  SegPlan p;
  p.uniform = 0;
  p.KB = (K + BK - 1) / BK;
  p.U = tiles * p.KB;
  p.G = p.U < num_sms ? p.U : num_sms;
  return p;
}
// Largest number of planes any tile needs under `p`.
inline int max_segments(const SegPlan &p) {
  int m = 1;
  for (int t = 0; t < p.U / p.KB; t++) {
    const int s = nseg_of(p, t * BM);
    if (s > m) m = s;
  }
  return m;
}

// ------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
constexpr uint64_t WAIT_LIMIT_NS = 2000000000ull;
// Bounded wait: false after WAIT_LIMIT_NS without the phase completing.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 128; i++)
      if (mbar_try_wait(bar, parity)) return true;
    if (global_ns() - t0 > WAIT_LIMIT_NS) return false;
  }
}
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *tm, int x, int y, uint32_t bar,
                                            uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(bar), "l"(pol) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *tm, int x, int y, int z,
                                            uint32_t bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%2, %3, %4}], [%5], %6;"
      ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(z), "r"(bar), "l"(pol) : "memory");
}
// Linear bulk copy global -> shared (both 16-byte aligned, size a multiple of 16).
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar,
                                          uint64_t pol) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(pol) : "memory");
}
__device__ __forceinline__ void grid_dep_wait() { pdl_wait(); }
__device__ __forceinline__ void grid_dep_launch() { pdl_launch(); }
__device__ __forceinline__ void epi_barrier() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap *tm) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(tm) : "memory");
}

__device__ __forceinline__ void tc_alloc(uint32_t smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// D[tmem] (+)= A[smem] * B[smem]^T, bf16 x bf16 -> f32, one CTA.
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// The mbarrier receives one arrival when every MMA issued so far by this thread has finished.
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 16 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major tile of 128-byte rows, 128-byte swizzle, 8-row
// groups 1024 bytes apart; the tile starts on a 1024-byte boundary (plus a K offset of
// 32 bytes per MMA step inside the swizzled row).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  return (uint64_t)((addr >> 4) & 0x3FFF) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: f32 accumulator, bf16 x bf16, both K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t instr_desc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

#define SV_ERR_WAIT_EMPTY 1
#define SV_ERR_WAIT_FULL 2
#define SV_ERR_WAIT_TMEM_EMPTY 3
#define SV_ERR_WAIT_TMEM_FULL 4

// What the CTA that finishes a tile does with the summed accumulator v[t][n].
enum EpiMode {
  EPI_PLAIN = 0,    // out[row0 + t][n] = scale_t * v
  EPI_RESID = 1,    // x[row0 + t][n] = (accumulate ? x : 0) + v;  xn = limbs(x * gain[n]);  ssq_out
  EPI_SWIGLU = 2    // hid[row0 + t][n] = limbs(silu(scale_t * gate) * (scale_t * up))
};

struct EpiArgs {
  int mode;
  int row0;              // first row of this launch within the call's row range
  int T;                 // rows of this launch (<= 128)
  int N;                 // output columns (EPI_SWIGLU: F, the width of gate and of up)
  int up_off;            // EPI_SWIGLU: row of W where the up projection starts (F)
  const bf16 *wpacked;   // weights repacked by pack_weights_kernel (one contiguous 32 KB block per
                         // (tile, K block), in unit order); NULL: strided boxes through the W map
  float *part;           // planes [max segments][T][tiles * 256] for tiles shared by several CTAs
  int *counters;         // [tiles] arrivals per shared tile; zero between launches
  // row scale of the RMSNorm in front of this GEMM: rsqrt(sum_j ssq_in[row][j] * inv_k + eps)
  const float *ssq_in;   // [rows][nt_in] partial sums of squares; NULL: scale 1
  int nt_in;
  float inv_k, eps;
  // EPI_PLAIN
  float *out;
  int ldo;
  // EPI_RESID
  float *x;              // [rows][N] residual stream
  int accumulate;
  const float *gain;     // [N] gain of the NEXT RMSNorm, folded into xn; NULL: ones
  bf16 *xn;              // two limbs, [rows][N] each
  size_t xn_plane;
  float *ssq_out;        // [rows][tiles]: sum over this tile's columns of x^2
  // EPI_SWIGLU
  bf16 *hid;             // two limbs, [rows][N] each
  size_t hid_plane;
};

__device__ __forceinline__ void store_limbs(bf16 *hi_plane, size_t plane, size_t idx, float v) {
  const bf16 hi = __float2bfloat16(v);
  hi_plane[idx] = hi;
  hi_plane[plane + idx] = __float2bfloat16(v - __bfloat162float(hi));
}

template <int TN>
__global__ void __launch_bounds__(THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
               const EpiArgs ea, const SegPlan plan, int *__restrict__ err) {
  constexpr int STAGES = stages_of(TN);
  constexpr int STAGE = stage_bytes(TN);
  constexpr bool MERGE = merged_limbs(TN);
  constexpr int AW = acc_width(TN);
  constexpr uint32_t IDESC = instr_desc(AW);
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bars = base + STAGES * STAGE;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
  auto tfull_bar = [&](int b) { return bars + 8u * (2 * STAGES + b); };
  auto tempty_bar = [&](int b) { return bars + 8u * (2 * STAGES + 2 + b); };
  const uint32_t tmem_slot = bars + 8u * (2 * STAGES + 4);
  __shared__ float s_scale[MAX_T];        // RMSNorm row scales
  __shared__ float s_red[4][MAX_T];       // per-warp sums of squares
  __shared__ int s_flag[8];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long u0 = (long long)blockIdx.x * plan.U / plan.G;
  const long long u1 = (long long)(blockIdx.x + 1) * plan.U / plan.G;
  const int n_units = (int)(u1 - u0);
  const int KB = plan.KB;
  const int T = ea.T;
  const bool swiglu = ea.mode == EPI_SWIGLU;

  const int npre = n_units < STAGES ? n_units : STAGES;
  uint64_t pol_w = 0;
  auto load_w = [&](int it) {
    const int st = it % STAGES;
    const long long u = u0 + it;
    const int tile = (int)(u / KB), kb = (int)(u % KB);
    const uint32_t sW = base + st * STAGE;
    mbar_expect_tx(full_bar(st), STAGE);
    if (ea.wpacked) {
      bulk_load(sW, ea.wpacked + (size_t)u * (BM * BK), W_STAGE_BYTES, full_bar(st), pol_w);
    } else {
      // the two 128-row halves of the tile: consecutive rows, or gate rows + up rows
      const int ya = swiglu ? tile * 128 : tile * BM;
      const int yb = swiglu ? ea.up_off + tile * 128 : tile * BM + 128;
      tma_load_2d(sW, &tmW, kb * BK, ya, full_bar(st), pol_w);
      tma_load_2d(sW + 128 * BK * 2, &tmW, kb * BK, yb, full_bar(st), pol_w);
    }
  };
  if (threadIdx.x == 0) {
    prefetch_tensormap(&tmX);
    if (!ea.wpacked) prefetch_tensormap(&tmW);
    for (int s = 0; s < STAGES; s++) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; b++) {
      mbar_init(tfull_bar(b), 1);
      mbar_init(tempty_bar(b), 8);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    grid_dep_launch();
    // the first ring-full of weights needs nothing from the previous kernel nor from the rest
    // of this CTA's set-up: get it moving at once
    pol_w = policy_evict_first();
    for (int it = 0; it < npre; it++) load_w(it);
  }
  if (warp == 1) {
    tc_alloc(tmem_slot, tmem_cols(TN));
    tc_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  uint32_t tmem_base;
  asm volatile("ld.shared.b32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0 && n_units > 0) {
      const uint64_t pol_x = policy_evict_last();
      // the activations are the previous kernel's output: wait for it only now
      grid_dep_wait();
      for (int j = 0; j < npre; j++)
        tma_load_3d(base + j * STAGE + W_STAGE_BYTES, &tmX, (int)((u0 + j) % KB) * BK, ea.row0, 0, full_bar(j),
                    pol_x);
      for (int it = npre; it < n_units; it++) {
        const int st = it % STAGES, rnd = it / STAGES;
        if (!mbar_wait(empty_bar(st), (rnd - 1) & 1)) {
          atomicExch(err, SV_ERR_WAIT_EMPTY);
          break;
        }
        load_w(it);
        tma_load_3d(base + st * STAGE + W_STAGE_BYTES, &tmX, (int)((u0 + it) % KB) * BK, ea.row0, 0,
                    full_bar(st), pol_x);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && n_units > 0) {
      int sidx = -1;                 // segment number; accumulator buffer = sidx & 1
      int prev_tile = -1;
      for (int it = 0; it < n_units; it++) {
        const int st = it % STAGES, rnd = it / STAGES;
        const long long u = u0 + it;
        const int tile = (int)(u / KB);
        const bool first = tile != prev_tile;
        prev_tile = tile;
        if (first) {
          sidx++;
          // the buffer's previous accumulator (segment sidx - 2) must have been read out
          if (sidx >= 2 && !mbar_wait(tempty_bar(sidx & 1), ((sidx >> 1) - 1) & 1)) {
            atomicExch(err, SV_ERR_WAIT_TMEM_EMPTY);
            break;
          }
        }
        const int buf = sidx & 1;
        if (!mbar_wait(full_bar(st), rnd & 1)) {
          atomicExch(err, SV_ERR_WAIT_FULL);
          break;
        }
        tc_fence_after();
        const uint32_t sW = base + st * STAGE, sX = sW + W_STAGE_BYTES;
#pragma unroll
        for (int kk = 0; kk < BK / 16; kk++) {
#pragma unroll
          for (int h = 0; h < 2; h++) {
            const uint64_t adesc = smem_desc(sW + h * (128 * BK * 2) + kk * 32);
            const uint32_t d = tmem_base + (uint32_t)((buf * 2 + h) * AW);
            if (MERGE) {
              tc_mma(d, adesc, smem_desc(sX + kk * 32), IDESC, (first && kk == 0) ? 0u : 1u);
            } else {
#pragma unroll
              for (int limb = 0; limb < 2; limb++) {
                const uint64_t bdesc = smem_desc(sX + limb * (TN * BK * 2) + kk * 32);
                tc_mma(d, adesc, bdesc, IDESC, (first && kk == 0 && limb == 0) ? 0u : 1u);
              }
            }
          }
        }
        tc_commit(empty_bar(st));
        const bool last = (it == n_units - 1) || ((int)((u + 1) / KB) != tile);
        if (last) tc_commit(tfull_bar(buf));
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..9)
    // Two warps per TMEM lane quarter; they take alternate 16-row chunks of the accumulator.
    grid_dep_wait();
    const int q = warp & 3;                       // TMEM lane quarter this warp may access
    const int wp = (warp - 2) >> 2;               // which of the quarter's two warps
    const int et = threadIdx.x - 64;              // 0..255 among the epilogue threads
    // accumulator chunk: 16 rows (TMEM columns c0..c0+15 of half hf) of this thread's column
    auto load_acc = [&](uint32_t tadr, int hf, int c0, float (&v)[16]) {
      uint32_t r0[16];
      tc_ld16(tadr + hf * AW + c0, r0);
      if (MERGE) {
        uint32_t r1[16];
        tc_ld16(tadr + hf * AW + TN + c0, r1);
        tc_wait_ld();
#pragma unroll
        for (int j = 0; j < 16; j++) v[j] = __uint_as_float(r0[j]) + __uint_as_float(r1[j]);
      } else {
        tc_wait_ld();
#pragma unroll
        for (int j = 0; j < 16; j++) v[j] = __uint_as_float(r0[j]);
      }
    };
    const int tiles = plan.U / KB;
    const int ldp = tiles * BM;                   // row pitch of a plane
    if (et < T) {
      float sc = 1.f;
      if (ea.ssq_in) {
        float ss = 0.f;
        for (int j = 0; j < ea.nt_in; j++) ss += ea.ssq_in[(size_t)(ea.row0 + et) * ea.nt_in + j];
        sc = rsqrtf(ss * ea.inv_k + ea.eps);
      }
      s_scale[et] = sc;
    }
    epi_barrier();

    int sidx = 0;
    int it = 0;
    while (it < n_units) {
      const int buf = sidx & 1;
      const long long u = u0 + it;
      const int tile = (int)(u / KB), kb0 = (int)(u % KB);
      int cnt = KB - kb0;
      if (cnt > n_units - it) cnt = n_units - it;
      // all eight warps take the same decision on the wait
      const bool mine = mbar_wait(tfull_bar(buf), (sidx >> 1) & 1);
      if (lane == 0) s_flag[warp - 2] = mine ? 1 : 0;
      epi_barrier();
      const bool ok = s_flag[0] && s_flag[1] && s_flag[2] && s_flag[3] && s_flag[4] && s_flag[5] && s_flag[6] &&
                      s_flag[7];
      epi_barrier();
      if (!ok) {
        if (et == 0) atomicExch(err, SV_ERR_WAIT_TMEM_FULL);
        break;
      }
      tc_fence_after();
      const int nseg = nseg_of(plan, tile * BM);
      const int seg = (int)blockIdx.x - owner_of(plan, (long long)tile * KB);
      // column of this thread inside the tile's plane, and in the output, for the two halves
      const int pc = tile * BM + q * 32 + lane;                       // plane column of half 0 (+128: half 1)
      const int na = swiglu ? tile * 128 + q * 32 + lane : pc;       // output column, half 0
      const int nb = swiglu ? na : pc + 128;                          // output column, half 1
      const uint32_t tadr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * 2 * AW);

      bool finish = true;
      if (nseg > 1) {
        // park this segment's partial sums, then see who is last
        float *pl = ea.part + (size_t)seg * T * ldp;
#pragma unroll 1
        for (int c0 = 16 * wp; c0 < TN; c0 += 32) {
          float ra[16], rb[16];
          load_acc(tadr, 0, c0, ra);
          load_acc(tadr, 1, c0, rb);
#pragma unroll
          for (int j = 0; j < 16; j++)
            if (c0 + j < T) {
              __stcg(pl + (size_t)(c0 + j) * ldp + pc, ra[j]);
              __stcg(pl + (size_t)(c0 + j) * ldp + pc + 128, rb[j]);
            }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty_bar(buf));
        __threadfence();
        epi_barrier();
        if (et == 0) {
          const int old = atomicAdd(ea.counters + tile, 1);
          const int lastone = (old == nseg - 1);
          if (lastone) atomicExch(ea.counters + tile, 0);
          s_flag[0] = lastone;
        }
        epi_barrier();
        finish = s_flag[0] != 0;
        epi_barrier();
        if (finish) __threadfence();
      }

      if (finish) {
        float sq[8];                 // EPI_RESID: this thread's sums of squares, 8 rows at a time
#pragma unroll 1
        for (int c0 = 16 * wp; c0 < TN; c0 += 32) {
          float va[16], vb[16];
          if (nseg > 1) {
            // planes are added in ascending order; two planes (64 independent loads per thread)
            // are in flight per round
#pragma unroll
            for (int j = 0; j < 16; j++) va[j] = vb[j] = 0.f;
            const float *pl = ea.part + (size_t)c0 * ldp + pc;
            const size_t pstride = (size_t)T * ldp;
            int sgn = 0;
#pragma unroll 1
            for (; sgn + 1 < nseg; sgn += 2) {
              float ta[16], tb[16], ua[16], ub[16];
#pragma unroll
              for (int j = 0; j < 16; j++) {
                const bool in = c0 + j < T;
                const float *p0 = pl + (size_t)sgn * pstride + (size_t)j * ldp;
                ta[j] = in ? __ldcg(p0) : 0.f;
                tb[j] = in ? __ldcg(p0 + 128) : 0.f;
                ua[j] = in ? __ldcg(p0 + pstride) : 0.f;
                ub[j] = in ? __ldcg(p0 + pstride + 128) : 0.f;
              }
#pragma unroll
              for (int j = 0; j < 16; j++) {
                va[j] = (va[j] + ta[j]) + ua[j];
                vb[j] = (vb[j] + tb[j]) + ub[j];
              }
            }
            if (sgn < nseg) {
#pragma unroll
              for (int j = 0; j < 16; j++) {
                const bool in = c0 + j < T;
                const float *p0 = pl + (size_t)sgn * pstride + (size_t)j * ldp;
                va[j] += in ? __ldcg(p0) : 0.f;
                vb[j] += in ? __ldcg(p0 + 128) : 0.f;
              }
            }
          } else {
            load_acc(tadr, 0, c0, va);
            load_acc(tadr, 1, c0, vb);
          }
          if (ea.mode == EPI_PLAIN) {
#pragma unroll
            for (int j = 0; j < 16; j++)
              if (c0 + j < T) {
                const float sc = s_scale[c0 + j];
                float *o = ea.out + (size_t)(ea.row0 + c0 + j) * ea.ldo;
                if (na < ea.N) o[na] = sc * va[j];
                if (nb < ea.N) o[nb] = sc * vb[j];
              }
          } else if (ea.mode == EPI_SWIGLU) {
#pragma unroll
            for (int j = 0; j < 16; j++)
              if (c0 + j < T && na < ea.N) {
                const float sc = s_scale[c0 + j];
                const float g = sc * va[j], up = sc * vb[j];
                store_limbs(ea.hid, ea.hid_plane, (size_t)(ea.row0 + c0 + j) * ea.N + na,
                            g / (1.f + expf(-g)) * up);
              }
          } else {
            const float ga = (ea.gain && na < ea.N) ? ea.gain[na] : 1.f;
            const float gb = (ea.gain && nb < ea.N) ? ea.gain[nb] : 1.f;
            // all residual loads of the 16 rows first: they are independent of the stores below
            float xa[16], xb[16];
#pragma unroll
            for (int j = 0; j < 16; j++) {
              const bool in = ea.accumulate && c0 + j < T;
              const size_t r = (size_t)(ea.row0 + c0 + j) * ea.N;
              xa[j] = (in && na < ea.N) ? __ldcg(ea.x + r + na) : 0.f;
              xb[j] = (in && nb < ea.N) ? __ldcg(ea.x + r + nb) : 0.f;
            }
#pragma unroll
            for (int half8 = 0; half8 < 2; half8++) {
#pragma unroll
              for (int j8 = 0; j8 < 8; j8++) {
                const int j = half8 * 8 + j8;
                float s2 = 0.f;
                if (c0 + j < T) {
                  const size_t r = (size_t)(ea.row0 + c0 + j) * ea.N;
                  if (na < ea.N) {
                    const float xv = xa[j] + va[j];
                    ea.x[r + na] = xv;
                    store_limbs(ea.xn, ea.xn_plane, r + na, xv * ga);
                    s2 += xv * xv;
                  }
                  if (nb < ea.N) {
                    const float xv = xb[j] + vb[j];
                    ea.x[r + nb] = xv;
                    store_limbs(ea.xn, ea.xn_plane, r + nb, xv * gb);
                    s2 += xv * xv;
                  }
                }
                sq[j8] = s2;
              }
#pragma unroll
              for (int j8 = 0; j8 < 8; j8++) {
                const float w = warp_sum(sq[j8]);
                if (lane == 0) s_red[q][c0 + half8 * 8 + j8] = w;
              }
            }
          }
        }
        if (nseg == 1) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(tempty_bar(buf));
        }
        if (ea.mode == EPI_RESID) {
          epi_barrier();
          if (et < T)
            ea.ssq_out[(size_t)(ea.row0 + et) * tiles + tile] =
                s_red[0][et] + s_red[1][et] + s_red[2][et] + s_red[3][et];
          epi_barrier();
        }
      }
      sidx++;
      it += cnt;
    }
  }

  if (*reinterpret_cast<volatile int *>(err) != 0) {
    // a wait gave up somewhere: give copies in flight time to land before the smem goes away
    const uint64_t t0 = global_ns();
    while (global_ns() - t0 < 200000ull) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) tc_dealloc(tmem_base, tmem_cols(TN));
}

// Repacks W [N, K] (row-major) into the order the kernel streams it: one contiguous 32 KB block
// per unit (tile, K block), tile-major, each block being the shared-memory image of a stage
// (256 rows of 64 bf16, the eight 16-byte chunks of a row XOR-swizzled by row & 7, exactly what
// a 128-byte-swizzle TMA box would have written). A CTA's share of the stream is then one
// contiguous range of HBM instead of 128-byte pieces one row pitch apart. Rows / columns past
// the matrix are zero. swiglu: tile j = gate rows j*128.. then up rows F + j*128.. (N = 2F).
__global__ void pack_weights_kernel(const bf16 *__restrict__ W, int N, int K, int tiles, int KB, int swiglu,
                                    int F, bf16 *__restrict__ out) {
  const size_t total = (size_t)tiles * KB * BM * 8;
  for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (size_t)gridDim.x * blockDim.x) {
    const int c = (int)(idx & 7), r = (int)((idx >> 3) & (BM - 1));
    const size_t unit = idx >> 11;
    const int kb = (int)(unit % KB), tile = (int)(unit / KB);
    int n;
    bool ok;
    if (swiglu) {
      n = (r < 128) ? tile * 128 + r : F + tile * 128 + (r - 128);
      ok = tile * 128 + (r & 127) < F;
    } else {
      n = tile * BM + r;
      ok = n < N;
    }
    const int k = kb * BK + c * 8;
    ok = ok && k < K;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (ok) v = *reinterpret_cast<const uint4 *>(W + (size_t)n * K + k);
    *reinterpret_cast<uint4 *>(out + unit * (BM * BK) + (size_t)r * BK + ((c ^ (r & 7)) << 3)) = v;
  }
}
inline size_t packed_elems(int tiles, int K) { return (size_t)tiles * ((K + BK - 1) / BK) * BM * BK; }

// ------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// Weight matrix [N, K] bf16, K contiguous: boxes of 128 rows x 64 columns.
inline bool make_w_map(CUtensorMap *tm, const bf16 *W, int N, int K) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)N};
  cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  cuuint32_t box[2] = {BK, 128};
  cuuint32_t es[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<bf16 *>(W), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// Activation limbs [2][rows][K] bf16 (lo limb `plane` elements after hi): boxes of
// 2 limbs x TN rows x 64 columns. Rows past `rows` read as zero.
inline bool make_x_map(CUtensorMap *tm, const bf16 *X, size_t plane, int rows, int K, int TN) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)rows, 2};
  cuuint64_t strides[2] = {(cuuint64_t)K * 2, (cuuint64_t)plane * 2};
  cuuint32_t box[3] = {BK, (cuuint32_t)TN, 2};
  cuuint32_t es[3] = {1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<bf16 *>(X), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int TN>
inline cudaError_t launch_tn(const CUtensorMap &tmW, const CUtensorMap &tmX, const EpiArgs &ea,
                             const SegPlan &plan, int *err, cudaStream_t st, bool pdl) {
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<TN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         smem_bytes(TN));
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(plan.G);
  cfg.blockDim = dim3(THREADS);
  cfg.dynamicSmemBytes = smem_bytes(TN);
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, gemm_tc_kernel<TN>, tmW, tmX, ea, plan, err);
}

// One launch over ea.T <= 128 rows; tmX must have been made with TN = tn_of(ea.T).
inline cudaError_t launch(const CUtensorMap &tmW, const CUtensorMap &tmX, const EpiArgs &ea,
                          const SegPlan &plan, int *err, cudaStream_t st, bool pdl) {
  switch (tn_of(ea.T)) {
    case 16: return launch_tn<16>(tmW, tmX, ea, plan, err, st, pdl);
    case 32: return launch_tn<32>(tmW, tmX, ea, plan, err, st, pdl);
    case 64: return launch_tn<64>(tmW, tmX, ea, plan, err, st, pdl);
    default: return launch_tn<128>(tmW, tmX, ea, plan, err, st, pdl);
  }
}

}  // namespace gemm_tc
