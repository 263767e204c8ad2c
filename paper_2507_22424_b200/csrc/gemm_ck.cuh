// Weight-streaming GEMM, one 256-column output tile per CTA or per small cluster of CTAs.
//
// A B200 SM can pull well over 100 GB/s through TMA, so ~64 streaming CTAs already saturate
// HBM: there is no need to spread a matrix over all 148 SMs. Every GEMM of the decoder is
// therefore cut into whole tiles first (LM head: 126 tiles = 126 CTAs, gate/up: 86, each
// finishing its tile straight from TMEM with the fused epilogue), and only matrices with few
// tiles are split along K as well: the S (<= 8) CTAs that share a tile form one thread-block
// cluster, CTA r streams K blocks [r KB / S, (r + 1) KB / S) through the TMA ring / tcgen05
// pipeline, drops its fp32 partial tile into its own shared memory, and after one cluster
// barrier every CTA finishes the rows t = r, r + S, ... of the tile, reading the S partials
// over DSMEM in rank order (deterministic). Nothing is parked in global memory, the epilogue
// work is spread over all CTAs, and a second cluster barrier keeps every CTA's shared memory
// alive until its peers have read it.
//
// Pipeline inside a CTA (as in gemm_tc.cuh, whose helpers are used): thread 0 issues the
// weight ring before the rest of the set-up and before griddepcontrol.wait, warp 0 keeps it
// full, warp 1 issues the MMAs (both limbs of X as one operand up to 64 rows), warps 2-9 run
// the epilogue: row scale of the preceding RMSNorm, or residual add + gain + two-limb split +
// sums of squares for the next norm, or SwiGLU.
//
// Waits on mbarriers are bounded as in gemm_tc; the cluster barriers are hardware barriers
// between co-scheduled CTAs and every path through the kernel reaches both of them.
#pragma once
#include <cooperative_groups.h>

#include "gemm_tc.cuh"

namespace gemm_ck {

using namespace gemm_tc;

constexpr int MAX_S = 8;                   // largest cluster = K slices per tile (portable limit)
constexpr long FIXED_CLOCKS = 12000;       // start, accumulator read-out and exit of a CTA (cost estimate of a launch plan)

__device__ __forceinline__ uint32_t cluster_size() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__host__ __device__ constexpr int ck_tmem_cols(int TN) { return 2 * acc_width(TN) < 32 ? 32 : 2 * acc_width(TN); }

// Quantised weights (Q8): a stage holds the int8 codes of a unit (16 KB from HBM) and its X slice;
// the bf16 image the tensor cores read is written by the epilogue warps into one of two 32 KB
// buffers in front of the ring. With half the bytes per unit the ring needs twice the units in
// flight for the same HBM rate, so it takes all the shared memory there is.
__host__ __device__ constexpr int q8_stage_bytes(int TN) { return W_STAGE_BYTES / 2 + 2 * TN * BK * 2; }
// expanded buffers: as many units as can be in expansion at once (the expansion of a unit is a
// chain of shared-memory latencies, barriers and a proxy fence of about a microsecond)
__host__ __device__ constexpr int q8_expanded(int TN) { return TN <= 32 ? 3 : 2; }
__host__ __device__ constexpr int q8_stages(int TN) {
  return (216 * 1024 - q8_expanded(TN) * W_STAGE_BYTES) / q8_stage_bytes(TN) > 8
             ? 8
             : (216 * 1024 - q8_expanded(TN) * W_STAGE_BYTES) / q8_stage_bytes(TN);
}
__host__ __device__ constexpr int q8_smem_bytes(int TN) {
  return q8_expanded(TN) * W_STAGE_BYTES + q8_stages(TN) * q8_stage_bytes(TN) + 1024 + 256;
}
// Expansion groups: one per expanded buffer (group g always writes buffer g and takes the units
// g, g + NE, ...: it waits for the MMAs of its previous unit before anything else, which also tells
// it that every earlier load has landed, so a mbarrier parity can never be read a phase late).
__host__ __device__ constexpr int q8_group_threads(int TN) { return q8_expanded(TN) == 3 ? 64 : 128; }

// EpiArgs as in gemm_tc: the mode is a template parameter. KB = K blocks per tile.
template <int TN, int MODE, bool Q8>
__global__ void __launch_bounds__(THREADS, 1)
gemm_ck_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
               const __grid_constant__ CUtensorMap tmXtail, const EpiArgs ea, const int KB,
               int *__restrict__ err) {
  constexpr int STAGES = Q8 ? q8_stages(TN) : stages_of(TN);
  constexpr int STAGE = Q8 ? q8_stage_bytes(TN) : stage_bytes(TN);
  constexpr int NE = Q8 ? q8_expanded(TN) : 1;
  constexpr uint32_t RING0 = Q8 ? NE * W_STAGE_BYTES : 0;     // Q8: the expanded weight buffers come first
  constexpr uint32_t XOFF = Q8 ? W_STAGE_BYTES / 2 : W_STAGE_BYTES;   // X slice within a stage
  constexpr int AW = acc_width(TN);
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bars = base + RING0 + STAGES * STAGE;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
  const uint32_t tfull_bar = bars + 8u * (2 * STAGES);
  const uint32_t tmem_slot = bars + 8u * (2 * STAGES + 1);
  // Q8: expanded buffer e holds the bf16 image of a unit (conv) / has been read by its MMAs (efree)
  auto conv_bar = [&](int e) { return bars + 8u * (2 * STAGES + 2 + e); };
  auto efree_bar = [&](int e) { return bars + 8u * (2 * STAGES + 2 + NE + e); };
  __shared__ int s_gflag[4];
  __shared__ float s_scale[MAX_T];
  __shared__ int s_pos[MAX_T], s_slot[MAX_T], s_ep[MAX_T];
  // RoPE factors of the CTA's rows (EPI_QKV, up to 32 rows of up to 64 pairs): fetched while the
  // MMAs run, so that the finishing loop does not wait for them row after row
  constexpr bool ROPE_SMEM = TN <= 32 && MODE == EPI_QKV && !Q8;   // (Q8: the ring takes that shared memory)
  constexpr int ROPE_ROWS = ROPE_SMEM ? 32 : 1, ROPE_HALF = ROPE_SMEM ? 64 : 1;
  __shared__ __align__(16) float2 s_rope[ROPE_ROWS * ROPE_HALF];
  __shared__ float s_red[8][MAX_T];
  __shared__ int s_flag[8];
  __shared__ float s_xv[4][2];             // EPI_TOPK: exchange between the two warps of a row group
  __shared__ int s_xi[4][2];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int S = (int)cluster_size();
  const int rank = (int)cluster_rank();
  constexpr bool swiglu = MODE == EPI_SWIGLU;
  const int tile = blockIdx.x / S;
  const int kb0 = rank * KB / S, kb1 = (rank + 1) * KB / S;
  const int n_units = kb1 - kb0;
  const long long u0 = (long long)tile * KB + kb0;
  const int tiles = gridDim.x / S;
  // rows of this CTA: the blockIdx.y-th chunk. The 128-row instantiation takes its chunk length
  // and MMA width from the launch (rows are spread evenly over the chunks of a long launch, so the
  // width is rarely the full 128); the last chunk has a tensor map with its own box.
  const int row0 = ea.row0 + (int)blockIdx.y * ea.chunk_rows;
  const int T = ea.T - (int)blockIdx.y * ea.chunk_rows < ea.chunk_rows ? ea.T - (int)blockIdx.y * ea.chunk_rows
                                                                         : ea.chunk_rows;
  const bool tail = blockIdx.y == gridDim.y - 1;
  const int tn = TN == MAX_T ? (tail ? ea.tn_tail : ea.tn_chunk) : TN;
  const CUtensorMap *xmap = (TN == MAX_T && tail) ? &tmXtail : &tmX;
  constexpr int W_LOAD_BYTES = Q8 ? W_STAGE_BYTES / 2 : W_STAGE_BYTES;   // int8 codes: half the bytes from HBM
  const uint32_t stage_tx = (uint32_t)(W_LOAD_BYTES + 2 * tn * BK * 2);
  const uint32_t idesc = instr_desc(2 * tn);

  const int npre = n_units < STAGES ? n_units : STAGES;
  uint64_t pol_w = 0;
  // test hook: the K block that is never loaded (-1: none)
  const int withheld = ea.withhold_unit - 1;
  auto load_w = [&](int it) {
    if (it == withheld) return;
    const int st = it % STAGES;
    const uint32_t sW = base + RING0 + st * STAGE;
    mbar_expect_tx(full_bar(st), stage_tx);
    if (Q8) {
      // the codes of the 256 x 64 tile; the epilogue warps expand them (below)
      bulk_load(sW, ea.wq8 + (size_t)(u0 + it) * (BM * BK), W_STAGE_BYTES / 2, full_bar(st), pol_w);
    } else if (ea.wpacked) {
      bulk_load(sW, ea.wpacked + (size_t)(u0 + it) * (BM * BK), W_STAGE_BYTES, full_bar(st), pol_w);
    } else {
      // the two 128-row halves of the tile: consecutive rows, or gate rows + up rows
      const int ya = swiglu ? tile * 128 : tile * BM;
      const int yb = swiglu ? ea.up_off + tile * 128 : tile * BM + 128;
      tma_load_2d(sW, &tmW, (kb0 + it) * BK, ya, full_bar(st), pol_w);
      tma_load_2d(sW + 128 * BK * 2, &tmW, (kb0 + it) * BK, yb, full_bar(st), pol_w);
    }
  };
  if (threadIdx.x == 0) {
    prefetch_tensormap(xmap);
    if (!ea.wpacked) prefetch_tensormap(&tmW);
    for (int s = 0; s < STAGES; s++) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), Q8 ? 2 : 1);     // Q8: the codes have been expanded AND the MMAs have read X
    }
    if (Q8)
      for (int e = 0; e < NE; e++) {
        mbar_init(conv_bar(e), 1);
        mbar_init(efree_bar(e), 1);
      }
    mbar_init(tfull_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    grid_dep_launch();
    pol_w = policy_evict_first();
    for (int it = 0; it < npre; it++) load_w(it);
  }
  if (warp == 1) {
    tc_alloc(tmem_slot, ck_tmem_cols(TN));
    tc_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  uint32_t tmem_base;
  asm volatile("ld.shared.b32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));

  // finishing-loop operands that the epilogue warps fetch while the MMAs run (part 1)
  const bool rope_staged = MODE == EPI_QKV && T <= ROPE_ROWS && (ea.dh >> 1) <= ROPE_HALF;
  // Long tiles (the 128-row instantiation): the RoPE factors of the CTA's rows are copied into the
  // idle ring behind the partial tile while the accumulator is read out (asynchronous copies, no
  // registers), so that the finishing loop has no global loads left.
  const bool rope_ring = MODE == EPI_QKV && TN == MAX_T && !Q8 && !rope_staged && n_units > 0 && (ea.dh >> 1) <= 64 &&
                         tn * BM * 4 + T * (ea.dh >> 1) * 8 <= STAGES * STAGE;
  const uint32_t rope_off = (uint32_t)(tn * BM * 4);
  float4 xpre0 = make_float4(0.f, 0.f, 0.f, 0.f), xpre1 = xpre0;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0 && n_units > 0) {
      const uint64_t pol_x = policy_evict_last();
      grid_dep_wait();
      for (int j = 0; j < npre; j++)
        if (j != withheld)
          tma_load_3d(base + RING0 + j * STAGE + XOFF, xmap, (kb0 + j) * BK, row0, 0, full_bar(j), pol_x);
      for (int it = npre; it < n_units; it++) {
        const int st = it % STAGES, rnd = it / STAGES;
        if (!mbar_wait(empty_bar(st), (rnd - 1) & 1, ea.wait_ns)) {
          atomicExch(err, SV_ERR_WAIT_EMPTY);
          break;
        }
        load_w(it);
        if (it != withheld)
          tma_load_3d(base + RING0 + st * STAGE + XOFF, xmap, (kb0 + it) * BK, row0, 0, full_bar(st), pol_x);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && n_units > 0) {
      for (int it = 0; it < n_units; it++) {
        const int st = it % STAGES, rnd = it / STAGES;
        if (!mbar_wait(Q8 ? conv_bar(it % NE) : full_bar(st), Q8 ? (it / NE) & 1 : rnd & 1, ea.wait_ns)) {
          atomicExch(err, SV_ERR_WAIT_FULL);
          break;
        }
        tc_fence_after();
        const uint32_t sW = Q8 ? base + (it % NE) * W_STAGE_BYTES : base + st * STAGE;
        const uint32_t sX = base + RING0 + st * STAGE + XOFF;
#pragma unroll
        for (int kk = 0; kk < BK / 16; kk++) {
#pragma unroll
          for (int h = 0; h < 2; h++) {
            const uint64_t adesc = smem_desc(sW + h * (128 * BK * 2) + kk * 32);
            const uint32_t d = tmem_base + (uint32_t)(h * AW);
            tc_mma(d, adesc, smem_desc(sX + kk * 32), idesc, (it == 0 && kk == 0) ? 0u : 1u);
          }
        }
        tc_commit(empty_bar(st));
        if (Q8) tc_commit(efree_bar(it % NE));
        if (it == n_units - 1) tc_commit(tfull_bar);
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ epilogue, part 1:
    // accumulator -> this CTA's partial tile P[t][256] in shared memory (the ring is idle by then)
    grid_dep_wait();
    const int q = warp & 3, wp = (warp - 2) >> 2;
    const int et = threadIdx.x - 64;
    if (et < T) {
      float sc = 1.f;
      if (ea.ssq_in) {
        float ss = 0.f;
        for (int j = 0; j < ea.nt_in; j++) ss += ea.ssq_in[(size_t)(row0 + et) * ea.nt_in + j];
        sc = rsqrtf(ss * ea.inv_k + ea.eps);
      }
      s_scale[et] = sc;
      if (MODE == EPI_QKV) {
        s_pos[et] = ea.rt.pos[row0 + et];
        s_slot[et] = ea.rt.slot[row0 + et];
        s_ep[et] = ea.rt.ep[row0 + et];
      }
    }
    // operands of the finishing loop that do not depend on this GEMM, requested now
    constexpr bool p2_swiglu = MODE == EPI_SWIGLU;
    const int p2_rg = p2_swiglu ? et >> 5 : et >> 6, p2_RG = p2_swiglu ? 8 : 4;
    const int p2_n = p2_swiglu ? tile * 128 + (et & 31) * 4 : tile * BM + (et & 63) * 4;
    const int p2_t0 = rank + p2_rg * S, p2_t1 = p2_t0 + p2_RG * S;
    if (MODE == EPI_RESID && ea.accumulate && p2_n < ea.N) {
      if (p2_t0 < T) xpre0 = *reinterpret_cast<const float4 *>(ea.x + (size_t)(row0 + p2_t0) * ea.N + p2_n);
      if (p2_t1 < T) xpre1 = *reinterpret_cast<const float4 *>(ea.x + (size_t)(row0 + p2_t1) * ea.N + p2_n);
    }
    if (rope_staged) {
      epi_barrier();                                       // s_pos is in place
      const int half = ea.dh >> 1;
      for (int i = et; i < T * half; i += 256) {
        const int t = i / half, j = i - t * half;
        s_rope[t * ROPE_HALF + j] = ea.rope_tab[(size_t)s_pos[t] * half + j];
      }
    }
    if (Q8) {
      // int8 -> bf16 expansion of every unit as it lands. NE groups of warps take the units in
      // turn (group g: units g, g + NE, ... into expanded buffer g), so that NE units are in
      // expansion at once; a thread owns every GT-th 16-byte piece of the codes (16 codes in, two
      // 16-byte chunks of a 128-byte swizzled row out).
      constexpr int GT = q8_group_threads(TN);
      const int g = et / GT, gt = et - g * GT;
      auto group_sync = [&]() { asm volatile("bar.sync %0, %1;" ::"r"(2 + g), "n"(GT) : "memory"); };
      if (g < NE) {
        for (int it = g; it < n_units; it += NE) {
          const int st = it % STAGES, rnd = it / STAGES, use = it / NE;
          if (gt == 0) {
            bool ok = true;
            if (use > 0) ok = mbar_wait(efree_bar(g), (use - 1) & 1, ea.wait_ns);   // first: see above
            if (ok) ok = mbar_wait(full_bar(st), rnd & 1, ea.wait_ns);
            s_gflag[g] = ok ? 1 : 0;
          }
          group_sync();                                    // the buffer is free, the codes are there
          if (!s_gflag[g]) {
            if (gt == 0) atomicExch(err, SV_ERR_WAIT_FULL);
            break;
          }
          const uint32_t sC = base + RING0 + st * STAGE, sE = base + g * W_STAGE_BYTES;
          // A thread takes 16-byte pieces gt, gt + GT, ... of the unit's codes (piece p = codes
          // 16 (p % 4) .. + 15 of row p / 4): consecutive lanes read consecutive shared memory, and
          // the two 16-byte chunks each piece expands to land in their swizzled places.
#pragma unroll 4
          for (int p = gt; p < BM * 4; p += GT) {
            const int r = p >> 2, q = p & 3;
            uint32_t c[4];
            asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                         : "=r"(c[0]), "=r"(c[1]), "=r"(c[2]), "=r"(c[3]) : "r"(sC + p * 16) : "memory");
#pragma unroll
            for (int h2 = 0; h2 < 2; h2++) {
              // eight codes (two words) -> eight bf16, exact (|code| <= 127), on the integer and FMA
              // pipes only: code + 128 in the low mantissa byte of 2^23, minus (2^23 + 128), gives the
              // code as fp32, whose upper half is its bf16 image
              const int ch = 2 * q + h2;
              uint32_t o[4];
#pragma unroll
              for (int h = 0; h < 2; h++) {
                const uint32_t x = c[2 * h2 + h] ^ 0x80808080u;
                const float f0 = __uint_as_float(__byte_perm(x, 0x4B000000u, 0x7650)) - 8388736.f;
                const float f1 = __uint_as_float(__byte_perm(x, 0x4B000000u, 0x7651)) - 8388736.f;
                const float f2 = __uint_as_float(__byte_perm(x, 0x4B000000u, 0x7652)) - 8388736.f;
                const float f3 = __uint_as_float(__byte_perm(x, 0x4B000000u, 0x7653)) - 8388736.f;
                o[2 * h] = __byte_perm(__float_as_uint(f0), __float_as_uint(f1), 0x7632);
                o[2 * h + 1] = __byte_perm(__float_as_uint(f2), __float_as_uint(f3), 0x7632);
              }
              asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(sE + r * 128 + ((ch ^ (r & 7)) << 4)),
                           "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]) : "memory");
            }
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> tensor-core reads
          group_sync();                                    // the whole tile is written
          if (gt == 0) {
            mbar_arrive(conv_bar(g));
            mbar_arrive(empty_bar(st));                    // the codes are no longer needed
          }
        }
      }
      epi_barrier();                                       // the groups (and the idle warps) meet again
    }
    bool have = n_units > 0;
    if (have) {
      const bool mine = mbar_wait(tfull_bar, 0, ea.wait_ns);
      if (lane == 0) s_flag[warp - 2] = mine ? 1 : 0;
      epi_barrier();
      have = s_flag[0] && s_flag[1] && s_flag[2] && s_flag[3] && s_flag[4] && s_flag[5] && s_flag[6] && s_flag[7];
      if (!have && et == 0) atomicExch(err, SV_ERR_WAIT_TMEM_FULL);
      tc_fence_after();
      if (rope_ring) {
        const int hp = ea.dh >> 2;                         // 16-byte pieces (two pairs) per row
        for (int i = et; i < T * hp; i += 256) {
          const int t = i / hp, j2 = i - t * hp;
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(base + rope_off + (uint32_t)(i * 16)),
                       "l"(ea.rope_tab + (size_t)s_pos[t] * (ea.dh >> 1) + 2 * j2) : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
      }
    }
    const uint32_t tadr = tmem_base + ((uint32_t)(q * 32) << 16);
    const int col = q * 32 + lane;                       // column within a 128-column half
#pragma unroll 1
    for (int c0 = 16 * wp; c0 < tn; c0 += 32) {
#pragma unroll 1
      for (int hf = 0; hf < 2; hf++) {
        float v[16];
        if (have) {
          uint32_t r0[16], r1[16];
          tc_ld16(tadr + hf * AW + c0, r0);
          tc_ld16(tadr + hf * AW + tn + c0, r1);
          tc_wait_ld();
#pragma unroll
          for (int j = 0; j < 16; j++) v[j] = __uint_as_float(r0[j]) + __uint_as_float(r1[j]);
        } else {
#pragma unroll
          for (int j = 0; j < 16; j++) v[j] = 0.f;
        }
#pragma unroll
        for (int j = 0; j < 16; j++)
          if (c0 + j < T) {
            const uint32_t a = base + (uint32_t)(((c0 + j) * BM + hf * 128 + col) * 4);
            asm volatile("st.shared.f32 [%0], %1;" ::"r"(a), "f"(v[j]) : "memory");
          }
      }
    }
    if (rope_ring) asm volatile("cp.async.wait_group 0;" ::: "memory");
    tc_fence_before();
  }

  // every CTA's partial tile is in place
  if (S > 1) cluster_sync_all(); else __syncthreads();
  if (warp == 0 && lane == 0 && ea.pf_w) {
    // head of the next GEMM's weight stream into L2, one request per range (its CTA c reads
    // units [tile KB + r KB / S, tile KB + (r + 1) KB / S) with tile = c / S, r = c % S).
    // Issued here, off the critical path of the epilogue warps.
    const int nct = ea.pf_tiles * ea.pf_S;
    for (int c = blockIdx.y * gridDim.x + blockIdx.x; c < nct; c += gridDim.x * gridDim.y) {
      const int ptile = c / ea.pf_S, r = c - ptile * ea.pf_S;
      const int pk0 = r * ea.pf_KB / ea.pf_S;
      int n = (r + 1) * ea.pf_KB / ea.pf_S - pk0;
      if (n > ea.pf_units) n = ea.pf_units;
      if (n > 0)
        prefetch_l2(static_cast<const char *>(ea.pf_w) + ((size_t)ptile * ea.pf_KB + pk0) * ea.pf_unit_bytes,
                    (uint32_t)(n * ea.pf_unit_bytes));
    }
  }

  if (warp >= 2) {
    // ------------------------------------------------------------------ epilogue, part 2:
    // rows rank, rank + S, ... of the tile. A thread owns four consecutive columns and every
    // RG-th of those rows (64 column groups x 4 row groups; SwiGLU, whose 128 outputs come
    // from column pairs, 32 x 8); the S partials are added in rank order. Everything this code
    // needs from global memory (residual, positions, RoPE factors) is requested BEFORE the
    // partial tiles are read, so that the latencies overlap instead of adding up.
    const int et = threadIdx.x - 64;
    const int RG = swiglu ? 8 : 4;
    const int rg = swiglu ? et >> 5 : et >> 6;
    const int c4 = swiglu ? (et & 31) * 4 : (et & 63) * 4;    // first of the four columns within the tile
    const int n = swiglu ? tile * 128 + c4 : tile * BM + c4;
    const bool col_ok = n < ea.N;                             // N % 4 == 0: all four or none
    const float *P_own = reinterpret_cast<const float *>(smem_raw + (base - smem_u32(smem_raw)));
    cooperative_groups::cluster_group cluster = cooperative_groups::this_cluster();
    float4 gain = make_float4(1.f, 1.f, 1.f, 1.f);
    if (MODE == EPI_RESID && ea.gain && col_ok) gain = *reinterpret_cast<const float4 *>(ea.gain + n);
    // QKV: which of q / k / v and which half of a head the four columns lie in
    const int which = MODE == EPI_QKV ? n / ea.hd : 2;
    const int cq = MODE == EPI_QKV ? n - which * ea.hd : 0;
    const int half = ea.dh >> 1, jq = MODE == EPI_QKV ? cq % ea.dh : 0;
    const bool lo = jq < half, rot = MODE == EPI_QKV && which < 2;
    auto partial_sum = [&](int off) {
      // (the shortcut of the unsplit case only in long tiles: it measured slower in the short ones)
      if (TN == MAX_T && S == 1) return *reinterpret_cast<const float4 *>(P_own + off);
      float4 p[MAX_S];
#pragma unroll
      for (int sl = 0; sl < MAX_S; sl++)
        if (sl < S) {
          // rank sl's copy of the same shared-memory address (mapped on the spot: an array of
          // eight mapped pointers would cost sixteen registers)
          const float *P = S == 1 ? P_own : cluster.map_shared_rank(const_cast<float *>(P_own), (unsigned)sl);
          p[sl] = *reinterpret_cast<const float4 *>(P + off);
        }
      float4 acc = p[0];
#pragma unroll
      for (int sl = 1; sl < MAX_S; sl++)
        if (sl < S) {
          acc.x += p[sl].x;
          acc.y += p[sl].y;
          acc.z += p[sl].z;
          acc.w += p[sl].w;
        }
      return acc;
    };
    // Q8: the accumulators are sums over integer codes; every output column takes the scale of its
    // weight row (the rotation partner and the up projection have theirs)
    float4 ws = make_float4(1.f, 1.f, 1.f, 1.f), ws2 = ws;
    if (Q8 && col_ok) {
      ws = *reinterpret_cast<const float4 *>(ea.wscale + n);
      if (rot) ws2 = *reinterpret_cast<const float4 *>(ea.wscale + n + (lo ? half : -half));
      if (swiglu) ws2 = *reinterpret_cast<const float4 *>(ea.wscale + ea.up_off + n);
    }
    auto scaled = [](float4 v, const float4 &w) { return make_float4(v.x * w.x, v.y * w.y, v.z * w.z, v.w * w.w); };
    // The rows are taken U at a time: first every global operand of the U rows, then their partial
    // sums, then the arithmetic and the stores, so that a long tile (prefill: up to 32 rows per
    // thread) pays the load latencies once per batch instead of once per row. Short tiles (a
    // verification step: two or three rows per thread) keep one row at a time: batching them
    // measured 2 % slower per step, the first stores leaving later.
    constexpr int U = TN == MAX_T ? 4 : 1;
    const int tstep = RG * S;
    for (int tb = rank + rg * S, iter0 = 0; tb < T; tb += U * tstep, iter0 += U) {
      float4 xo_[U], v_[U], w_[U];
#pragma unroll
      for (int u = 0; u < U; u++) {
        const int t = tb + u * tstep, iter = iter0 + u;
        // the residuals of the first two rows were fetched in part 1
        xo_[u] = iter == 0 ? xpre0 : xpre1;
        if (MODE == EPI_RESID && ea.accumulate && col_ok && iter >= 2 && t < T)
          xo_[u] = *reinterpret_cast<const float4 *>(ea.x + (size_t)(row0 + t) * ea.N + n);
      }
#pragma unroll
      for (int u = 0; u < U; u++) {
        const int t = tb + u * tstep;
        v_[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        w_[u] = v_[u];
        if (t < T) {
          v_[u] = partial_sum(t * BM + c4);
          // the partner columns of the rotation (dh / 2 away) are in the same tile; so is the up projection
          if (rot) w_[u] = partial_sum(t * BM + c4 + (lo ? half : -half));
          if (swiglu) w_[u] = partial_sum(t * BM + 128 + c4);
        }
      }
#pragma unroll
      for (int u = 0; u < U; u++) {
        const int t = tb + u * tstep;
        if (t >= T) break;
        const size_t row = (size_t)(row0 + t);
        const float sc = s_scale[t];
        const float4 xo = xo_[u];
        float4 cs01 = make_float4(0.f, 0.f, 0.f, 0.f), cs23 = cs01;
        if (rot) {
          // RoPE factors: staged in shared memory (short tiles: part 1; long tiles: the idle ring); the
          // global table is the fallback of the instantiations that have no room for them
          const int jh = lo ? jq : jq - half;
          const float2 *cs = rope_staged ? s_rope + t * ROPE_HALF + jh
                             : rope_ring ? reinterpret_cast<const float2 *>(P_own + (rope_off >> 2)) + t * half + jh
                                         : ea.rope_tab + (size_t)s_pos[t] * half + jh;
          cs01 = *reinterpret_cast<const float4 *>(cs);
          cs23 = *reinterpret_cast<const float4 *>(cs + 2);
        }
        const int slot = MODE == EPI_QKV ? s_slot[t] : 0, ep = MODE == EPI_QKV ? s_ep[t] : 0;
        float4 v = v_[u];
        if (Q8) v = scaled(v, ws);
        if (MODE == EPI_PLAIN) {
          const float4 ov = make_float4(sc * v.x, sc * v.y, sc * v.z, sc * v.w);
          if (ea.out && col_ok) *reinterpret_cast<float4 *>(ea.out + row * ea.ldo + n) = ov;
          if (ea.cand) {
            // greedy argmax, first step: the top-2 of this warp's 128 columns over [lo, hi)
            sv::Top2 b{-INFINITY, -INFINITY, 0x7fffffff};
            const float vv[4] = {ov.x, ov.y, ov.z, ov.w};
  #pragma unroll
            for (int e = 0; e < 4; e++)
              if (n + e >= ea.lo && n + e < ea.hi && n + e < ea.N) sv::top2_push(b, vv[e], n + e);
            sv::top2_warp(b);
            if (lane == 0)
              ea.cand[row * (size_t)(2 * tiles) + tile * 2 + ((et >> 5) & 1)] = make_float4(b.v1, __int_as_float(b.i1), b.v2, 0.f);
          }
        } else if (MODE == EPI_TOPK) {
          // the row's 256 scores sit in the two warps of this row group, four per thread
          const int wg = (et >> 5) & 1;
          const float xv[4] = {sc * v.x, sc * v.y, sc * v.z, sc * v.w};
          bool in[4];
  #pragma unroll
          for (int e = 0; e < 4; e++) in[e] = n + e >= ea.lo && n + e < ea.hi && n + e < ea.N;
          if (ea.out && col_ok) *reinterpret_cast<float4 *>(ea.out + row * ea.ldo + n) = make_float4(xv[0], xv[1], xv[2], xv[3]);
          auto pair_sync = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(2 + rg) : "memory"); };
          float mx = -INFINITY;
  #pragma unroll
          for (int e = 0; e < 4; e++)
            if (in[e]) mx = fmaxf(mx, xv[e]);
          mx = warp_max(mx);
          if (lane == 0) s_xv[rg][wg] = mx;
          pair_sync();
          mx = fmaxf(s_xv[rg][0], s_xv[rg][1]);
          pair_sync();
          float se = 0.f;
  #pragma unroll
          for (int e = 0; e < 4; e++)
            if (in[e]) se += expf(xv[e] - mx);
          se = warp_sum(se);
          if (lane == 0) s_xv[rg][wg] = se;
          pair_sync();
          const float lse = mx + logf(s_xv[rg][0] + s_xv[rg][1]);
          pair_sync();
          unsigned taken = 0;
          for (int k = 0; k < SV_TOPK; k++) {
            float bv = -INFINITY;
            int bi = 0x7fffffff;
  #pragma unroll
            for (int e = 0; e < 4; e++)
              if (in[e] && !((taken >> e) & 1u) && (xv[e] > bv || (xv[e] == bv && n + e < bi))) {
                bv = xv[e];
                bi = n + e;
              }
  #pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
              const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
              const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
              if (ov > bv || (ov == bv && oi < bi)) {
                bv = ov;
                bi = oi;
              }
            }
            if (lane == 0) {
              s_xv[rg][wg] = bv;
              s_xi[rg][wg] = bi;
            }
            pair_sync();
            const float v0 = s_xv[rg][0], v1 = s_xv[rg][1];
            const int i0 = s_xi[rg][0], i1 = s_xi[rg][1];
            const bool first = v0 > v1 || (v0 == v1 && i0 < i1);
            bv = first ? v0 : v1;
            bi = first ? i0 : i1;
            pair_sync();
            if (bi >= n && bi < n + 4) taken |= 1u << (bi - n);
            if ((et & 63) == 0) {
              ea.top_tok[row * SV_TOPK + k] = bi + ea.tok_offset;
              ea.top_lp[row * SV_TOPK + k] = bv - lse;
            }
          }
        } else if (MODE == EPI_QKV) {
          float4 o = make_float4(sc * v.x, sc * v.y, sc * v.z, sc * v.w);
          if (rot) {
            float4 w = w_[u];
            if (Q8) w = scaled(w, ws2);
            const float sg = lo ? -sc : sc;
            o.x = o.x * cs01.x + sg * w.x * cs01.y;
            o.y = o.y * cs01.z + sg * w.y * cs01.w;
            o.z = o.z * cs23.x + sg * w.z * cs23.y;
            o.w = o.w * cs23.z + sg * w.w * cs23.w;
          }
          if (col_ok) {
            float *dst = which == 0 ? ea.q + row * ea.hd + cq
                                    : ea.cache + (size_t)ep * ea.ep_stride +
                                          ((size_t)(which - 1) * ea.max_seq + slot) * ea.hd + cq;
            *reinterpret_cast<float4 *>(dst) = o;
          }
        } else if (swiglu) {
          float4 up = w_[u];
          if (Q8) up = scaled(up, ws2);
          if (col_ok) {
            const float gx = sc * v.x, gy = sc * v.y, gz = sc * v.z, gw = sc * v.w;
            store_limbs4(ea.hid, ea.hid_plane, row * ea.N + n,
                         make_float4(__fdividef(gx, 1.f + __expf(-gx)) * (sc * up.x),
                                     __fdividef(gy, 1.f + __expf(-gy)) * (sc * up.y),
                                     __fdividef(gz, 1.f + __expf(-gz)) * (sc * up.z),
                                     __fdividef(gw, 1.f + __expf(-gw)) * (sc * up.w)));
          }
        } else {
          float s2 = 0.f;
          if (col_ok) {
            v.x += xo.x;
            v.y += xo.y;
            v.z += xo.z;
            v.w += xo.w;
            *reinterpret_cast<float4 *>(ea.x + row * ea.N + n) = v;
            store_limbs4(ea.xn, ea.xn_plane, row * ea.N + n,
                         make_float4(v.x * gain.x, v.y * gain.y, v.z * gain.z, v.w * gain.w));
            s2 = (v.x * v.x + v.y * v.y) + (v.z * v.z + v.w * v.w);
          }
          s2 = warp_sum(s2);
          if (lane == 0) s_red[warp - 2][t] = s2;
        }
      }
    }
  }
  // This CTA has read all it needs from its peers: say so now, and wait for the peers' word only
  // before leaving (nobody leaves while a peer may still be reading its shared memory), so that
  // the barrier's latency passes behind the rest of the epilogue.
  if (S > 1) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  if (warp >= 2 && MODE == EPI_RESID) {
    const int et = threadIdx.x - 64;
    epi_barrier();
    // thread i finishes this CTA's i-th row, which row group i % 4 (two warps) handled
    const int t = rank + et * S;
    if (t < T) {
      const int w0 = 2 * (et & 3);
      ea.ssq_out[(size_t)(row0 + t) * tiles + tile] = s_red[w0][t] + s_red[w0 + 1][t];
    }
  }
  if (S > 1) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");

  if (*reinterpret_cast<volatile int *>(err) != 0) {
    const uint64_t t0 = global_ns();
    while (global_ns() - t0 < 200000ull) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) tc_dealloc(tmem_base, ck_tmem_cols(TN));
}

template <int TN, int MODE, bool Q8>
inline cudaError_t launch_tq(const CUtensorMap &tmW, const CUtensorMap &tmX, const CUtensorMap &tmXtail,
                             const EpiArgs &ea, int tiles, int KB, int S, int *err, cudaStream_t st, bool pdl) {
  // per device and cheap: set on every launch, so that every device of the process has it
  constexpr int SMEM = Q8 ? q8_smem_bytes(TN) : smem_bytes(TN);
  cudaError_t e = cudaFuncSetAttribute(gemm_ck_kernel<TN, MODE, Q8>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(tiles * S, (ea.T + ea.chunk_rows - 1) / ea.chunk_rows);
  cfg.blockDim = dim3(THREADS);
  cfg.dynamicSmemBytes = SMEM;
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = S;
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, gemm_ck_kernel<TN, MODE, Q8>, tmW, tmX, tmXtail, ea, KB, err);
}
// int8 weights (ea.wq8) take the instantiation that expands the codes in shared memory; the draft
// scoring mode never runs on quantised weights.
template <int TN, int MODE>
inline cudaError_t launch_tm(const CUtensorMap &tmW, const CUtensorMap &tmX, const CUtensorMap &tmXtail,
                             const EpiArgs &ea, int tiles, int KB, int S, int *err, cudaStream_t st, bool pdl) {
  if (ea.wq8 && MODE != EPI_TOPK) return launch_tq<TN, MODE == EPI_TOPK ? EPI_PLAIN : MODE, true>(tmW, tmX, tmXtail, ea, tiles, KB, S, err, st, pdl);
  return launch_tq<TN, MODE, false>(tmW, tmX, tmXtail, ea, tiles, KB, S, err, st, pdl);
}

// The epilogue mode is a template parameter: each instantiation carries only its own finishing
// code (the epilogue runs once per CTA from a cold instruction cache, so its size matters).
template <int TN>
inline cudaError_t launch_tn(const CUtensorMap &tmW, const CUtensorMap &tmX, const CUtensorMap &tmXtail,
                             const EpiArgs &ea, int tiles, int KB, int S, int *err, cudaStream_t st, bool pdl) {
  switch (ea.mode) {
    case EPI_PLAIN: return launch_tm<TN, EPI_PLAIN>(tmW, tmX, tmXtail, ea, tiles, KB, S, err, st, pdl);
    case EPI_RESID: return launch_tm<TN, EPI_RESID>(tmW, tmX, tmXtail, ea, tiles, KB, S, err, st, pdl);
    case EPI_SWIGLU: return launch_tm<TN, EPI_SWIGLU>(tmW, tmX, tmXtail, ea, tiles, KB, S, err, st, pdl);
    case EPI_TOPK: return launch_tm<TN, EPI_TOPK>(tmW, tmX, tmXtail, ea, tiles, KB, S, err, st, pdl);
    default: return launch_tm<TN, EPI_QKV>(tmW, tmX, tmXtail, ea, tiles, KB, S, err, st, pdl);
  }
}

// How many clusters of each size 1..MAX_S can be resident at once (index = size; 0 = unknown).
struct ClusterFit {
  int max_active[MAX_S + 1];
};
// Asks the occupancy calculator about the TN = 32 instantiation (every instantiation uses most
// of an SM's shared memory: one CTA per SM).
inline ClusterFit query_cluster_fit() {
  ClusterFit f = {};
  cudaFuncSetAttribute(gemm_ck_kernel<32, EPI_RESID, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes(32));
  for (int S = 1; S <= MAX_S; S++) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(S * 64);
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = smem_bytes(32);
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = S;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, gemm_ck_kernel<32, EPI_RESID, false>, &cfg) == cudaSuccess) f.max_active[S] = n;
  }
  cudaGetLastError();
  return f;
}
// K slices per tile for `units` (tile, row chunk) pairs of KB blocks each; every slice keeps at
// least four K blocks. When the units fit on the GPU at once: the largest cluster size whose
// `units` clusters are all resident together (a second wave would double the time). Otherwise
// (more units than SMs: prefill) clusters run in waves and a CTA's time is a fixed part (start,
// reduction, epilogue: about what 16 K blocks take) plus its K blocks, so the cost of a choice
// is waves x (16 + blocks per slice), ties to the smaller cluster.
inline int slices_for(int units, int KB, const ClusterFit &fit) {
  const int fit1 = fit.max_active[1] > 0 ? fit.max_active[1] : 148;
  int best = 1;
  if (units <= fit1) {
    for (int S = 2; S <= MAX_S; S++)
      if (fit.max_active[S] >= units && KB / S >= 4) best = S;
    return best;
  }
  long best_cost = -1;
  for (int S = 1; S <= MAX_S; S++) {
    const int fits = S == 1 ? fit1 : fit.max_active[S];
    if (fits <= 0 || (S > 1 && KB / S < 4)) continue;
    const long cost = (long)((units + fits - 1) / fits) * (16 + (KB + S - 1) / S);
    if (best_cost < 0 || cost < best_cost) {
      best_cost = cost;
      best = S;
    }
  }
  return best;
}

// How a launch over R rows is cut: up to 128 rows are one chunk of the instantiation tn_of(R)
// (between 65 and 128 rows: MMAs as wide as the rows need, to the next multiple of 8). Longer
// launches (prefill, batched verification) are tensor-bound, and what counts is how evenly the
// work fills the SMs: the rows are spread evenly over `chunks` chunks (grid y) of the 128-row
// instantiation, and chunk count and K slices are chosen together by a cost estimate in SM
// clocks: waves x (fixed part of a CTA + its K blocks x clocks per K block), where a K block of tn
// rows costs 512 + 6 tn clocks (what its 64 KB + 768 tn bytes of shared-memory traffic take at
// 128 bytes per clock; the MMAs themselves need 8 tn).
struct RowPlan {
  int chunks, chunk_rows, tn_chunk, tn_tail, S;
};
inline int ceil8(int x) { return (x + 7) / 8 * 8; }
inline RowPlan plan_rows(int R, int tiles, int KB, const ClusterFit &fit) {
  RowPlan p = {1, MAX_T, tn_of(R), tn_of(R), 1};
  if (R <= MAX_T) {
    if (R > 64) p.tn_chunk = p.tn_tail = ceil8(R);
    p.S = slices_for(tiles, KB, fit);
    return p;
  }
  const int fit1 = fit.max_active[1] > 0 ? fit.max_active[1] : 148;
  const int cmin = (R + MAX_T - 1) / MAX_T;
  long best = -1;
  for (int c = cmin; c <= cmin + 6 && c <= R; c++) {
    const int rows = ceil8((R + c - 1) / c);               // chunk starts stay multiples of 8 rows
    if (rows > MAX_T || (long)rows * (c - 1) >= R) continue;
    for (int S = 1; S <= MAX_S; S++) {
      const int fits = S == 1 ? fit1 : fit.max_active[S];
      if (fits <= 0 || (S > 1 && KB / S < 4)) continue;
      const long waves = ((long)tiles * c + fits - 1) / fits;
      const long cost = waves * (FIXED_CLOCKS + 60L * rows / S + (long)((KB + S - 1) / S) * (512 + 6 * rows));
      if (best < 0 || cost < best) {
        best = cost;
        p.chunks = c;
        p.chunk_rows = rows;
        p.S = S;
      }
    }
  }
  p.tn_chunk = p.chunk_rows;
  p.tn_tail = ceil8(R - (p.chunks - 1) * p.chunk_rows);
  return p;
}

// One launch over ea.T rows in chunks of ea.chunk_rows (grid y). tmX: the X map with box rows
// ea.tn_chunk; tmXtail: the map for the last chunk (box rows ea.tn_tail).
inline cudaError_t launch(const CUtensorMap &tmW, const CUtensorMap &tmX, const CUtensorMap &tmXtail,
                          const EpiArgs &ea, int tiles, int KB, int S, int *err, cudaStream_t st, bool pdl) {
  // (launches of several chunks always take the 128-row instantiation: it alone reads the widths from ea)
  switch (ea.T > MAX_T ? MAX_T : tn_of(ea.T)) {
    case 16: return launch_tn<16>(tmW, tmX, tmX, ea, tiles, KB, S, err, st, pdl);
    case 32: return launch_tn<32>(tmW, tmX, tmX, ea, tiles, KB, S, err, st, pdl);
    case 64: return launch_tn<64>(tmW, tmX, tmX, ea, tiles, KB, S, err, st, pdl);
    default: return launch_tn<128>(tmW, tmX, tmXtail, ea, tiles, KB, S, err, st, pdl);
  }
}

}  // namespace gemm_ck
