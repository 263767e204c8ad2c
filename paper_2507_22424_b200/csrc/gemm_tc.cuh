// Building blocks of the weight-streaming GEMM on the sm_100a tensor cores (tcgen05 + TMEM,
// operands by TMA); the kernel itself is in gemm_ck.cuh.
//   Y[t][n] = sum_k (Xhi[t][k] + Xlo[t][k]) * W[n][k]        (fp32 accumulate)
// for T <= 128 activation rows per launch: the verification forward over one draft tree, every
// draft-model level, and the prefill in launches of 128 rows. At these sizes the cost is the
// single pass over W, so everything is built around streaming W:
//
//  * W [N, K] (bf16, K contiguous) is cut into tiles of 256 rows x 64 columns (32 KB, 128-byte
//    swizzle). A tile sits on the MMA's M axis (two M = 128 halves), the activation rows on its
//    N axis (TN = T rounded up to 16/32/64/128). Both bf16 limbs of X are multiplied against
//    the same W tile (as one operand of 2 TN rows, 256 at most), so fp32-grade activations
//    cost no extra bytes of the weight stream.
//  * The library keeps its own repacked copy of every weight matrix (pack_weights_kernel):
//    one contiguous 32 KB block per (tile, K block) in streaming order, already swizzled, so
//    a CTA's share of the stream is one contiguous range of HBM fetched by plain bulk copies.
//  * The epilogue is fused (EpiArgs): plain store with the RMSNorm row scale, or residual add
//    + gain + two-limb split + sums of squares for the next norm, or SwiGLU.
//  * The first ring-full of weight loads does not depend on the previous kernel, so it is
//    issued BEFORE griddepcontrol.wait: launched with programmatic stream serialisation a GEMM
//    streams weights while its predecessor drains.
//
// Every mbarrier wait is bounded (EpiArgs::wait_ns of %globaltimer, two seconds by default); on
// expiry the kernel records a code in *err, lets copies in flight land, frees its TMEM and returns.
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
// Up to 64 rows the ring leaves ~60 KB of the SM's shared memory free, so that the small kernels
// between two GEMMs can be resident next to a GEMM CTA while it prefetches weights. At 128 rows
// (prefill) a stage is 64 KB and two of them cannot cover the load latency: the ring takes a
// third and most of the SM's shared memory.
__host__ __device__ constexpr int stages_of(int TN) { return TN > 64 ? 3 : RING_BUDGET / stage_bytes(TN); }
__host__ __device__ constexpr int smem_bytes(int TN) { return stages_of(TN) * stage_bytes(TN) + 1024 + 256; }
// Both limbs of X form ONE MMA operand (N = 2 TN: hi rows, then lo rows; 256 at most, the
// largest N of an M = 128 MMA), which reads the weight operand from shared memory once for
// both; the two column groups of the accumulator are added in the epilogue.
__host__ __device__ constexpr int acc_width(int TN) { return 2 * TN; }

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
constexpr uint64_t WAIT_LIMIT_NS = 2000000000ull;     // default limit of a device-side wait
// Bounded wait: false after limit_ns without the phase completing.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint64_t limit_ns) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 128; i++)
      if (mbar_try_wait(bar, parity)) return true;
    if (global_ns() - t0 > limit_ns) return false;
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
__device__ __forceinline__ void prefetch_l2(const void *src, uint32_t bytes) {
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void grid_dep_wait() { pdl_wait(); }
__device__ __forceinline__ void grid_dep_launch() { pdl_launch(); }
// barrier among the 256 epilogue threads (warps 2-9)
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
  EPI_PLAIN = 0,    // out[row0 + t][n] = scale_t * v (when out != NULL); with cand != NULL also the
                    // top-2 of every 128 output columns over [lo, hi): the greedy argmax (Eq. 1) is
                    // finished from those by argmax_merge_kernel, no [T, V] logits are stored
  EPI_RESID = 1,    // x[row0 + t][n] = (accumulate ? x : 0) + v;  xn = limbs(x * gain[n]);  ssq_out
  EPI_SWIGLU = 2,   // hid[row0 + t][n] = limbs(silu(scale_t * gate) * (scale_t * up))
  EPI_QKV = 3,      // scale_t * v is [q | k | v]: rotate q and k by the row's position (rotate-half
                    // pairs (i, i + dh/2)), write q and, into the row's cache slot, k and v
  EPI_TOPK = 4      // one 256-column tile (the action rows of the LM head): log-softmax over columns
                    // [lo, hi) of scale_t * v and its SV_TOPK best entries per row (Eq. 2: the draft
                    // model's candidates), finished inside the GEMM
};

struct EpiArgs {
  int mode;
  int row0;              // first row of this launch within the call's row range
  int T;                 // rows of this launch; CTAs with blockIdx.y = c take rows [chunk_rows c, chunk_rows (c + 1))
  int chunk_rows;        // rows per chunk (<= 128); launches of up to 128 rows are one chunk
  int tn_chunk, tn_tail; // X box rows = half the MMA width (multiples of 8) of the 128-row instantiation: of
                         // every chunk but the last, and of the last
  int N;                 // output columns (EPI_SWIGLU: F, the width of gate and of up)
  int up_off;            // EPI_SWIGLU: row of W where the up projection starts (F)
  unsigned long long wait_ns;   // limit of every mbarrier wait
  int withhold_unit;     // test hook (specvla_gemm_fault_test): > 0: the producer of every CTA skips its
                         // (withhold_unit - 1)-th K block, so the waits for it run out; 0: off
  const signed char *wq8;   // int8 codes of the weights in the same unit order (16 KB per unit, rows of 64
                            // codes, not swizzled), or NULL; wscale[n] = scale of weight row n
  const float *wscale;
  const bf16 *wpacked;   // weights repacked by pack_weights_kernel (one contiguous 32 KB block per
                         // (tile, K block), in unit order); NULL: strided boxes through the W map
  // L2 prefetch for the GEMM that follows: once its own loads are issued, every CTA asks for
  // the first pf_units 32 KB blocks of some of the next GEMM's per-CTA ranges, so that HBM keeps
  // working through this kernel's epilogue, the kernel boundary and the next kernel's start.
  const void *pf_w;      // packed weights (or int8 codes) of the next GEMM; NULL: no prefetch
  int pf_tiles, pf_KB, pf_S, pf_units, pf_unit_bytes;
  // row scale of the RMSNorm in front of this GEMM: rsqrt(sum_j ssq_in[row][j] * inv_k + eps)
  const float *ssq_in;   // [rows][nt_in] partial sums of squares; NULL: scale 1
  int nt_in;
  float inv_k, eps;
  // EPI_PLAIN (out may be NULL when cand is given), EPI_TOPK (out may be NULL)
  float *out;
  int ldo;
  float4 *cand;          // EPI_PLAIN: [rows][2 * tiles] (top-1 value, top-1 column as int bits, top-2 value, -)
  int lo, hi;            // EPI_PLAIN with cand / EPI_TOPK: columns that take part
  int tok_offset;        // EPI_TOPK: token id of column 0
  int *top_tok;          // EPI_TOPK: [rows][SV_TOPK]
  float *top_lp;
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
  // EPI_QKV (N = 3 * H * dh)
  RowTable rt;           // per-row position, cache slot and episode
  const float2 *rope_tab;  // [position][dh / 2] (cos, sin)
  float *q;              // [rows][H * dh]
  float *cache;          // [episode][2 (K, V)][max_seq][H * dh]
  size_t ep_stride;
  int max_seq, hd, dh;
};

__device__ __forceinline__ void store_limbs(bf16 *hi_plane, size_t plane, size_t idx, float v) {
  const bf16 hi = __float2bfloat16(v);
  hi_plane[idx] = hi;
  hi_plane[plane + idx] = __float2bfloat16(v - __bfloat162float(hi));
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
// Weight-only int8 quantisation, per output row (symmetric): scale[n] = max_k |W[n][k]| / 127 (1 for
// an all-zero row), code = round-half-even(W / scale) clipped to [-127, 127]; scale and quotient in
// IEEE float32, so that any implementation of the same rule derives the same codes. One warp per row.
__global__ void row_scale_q8_kernel(const bf16 *__restrict__ W, int N, int K, float *__restrict__ scale) {
  const int n = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (n >= N) return;
  float m = 0.f;
  for (int k = lane; k < K; k += 32) m = fmaxf(m, fabsf(__bfloat162float(W[(size_t)n * K + k])));
  m = warp_max(m);
  if (lane == 0) scale[n] = m > 0.f ? __fdiv_rn(m, 127.f) : 1.f;
}
// The codes in the GEMM's unit order: one 16 KB block per (tile, K block), 256 rows of 64 codes, rows
// and tiles as in pack_weights_kernel (swiglu: 128 gate rows, then the 128 matching up rows). Rows and
// columns past the matrix are zero.
__global__ void pack_weights_q8_kernel(const bf16 *__restrict__ W, int N, int K, int tiles, int KB, int swiglu,
                                       int F, const float *__restrict__ scale, signed char *__restrict__ out) {
  const size_t total = (size_t)tiles * KB * BM * 4;                  // 16 codes per thread step
  for (size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (size_t)gridDim.x * blockDim.x) {
    const int c = (int)(idx & 3), r = (int)((idx >> 2) & (BM - 1));
    const size_t unit = idx >> 10;
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
    const float s = ok ? scale[n] : 1.f;
    uint32_t words[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int e = 0; e < 16; e++) {
      const int k = kb * BK + c * 16 + e;
      int q = 0;
      if (ok && k < K) {
        const float t = __fdiv_rn(__bfloat162float(W[(size_t)n * K + k]), s);
        q = (int)fminf(fmaxf(rintf(t), -127.f), 127.f);
      }
      words[e >> 2] |= (uint32_t)(q & 0xff) << (8 * (e & 3));
    }
    *reinterpret_cast<uint4 *>(out + unit * (BM * BK) + (size_t)r * BK + c * 16) = make_uint4(words[0], words[1], words[2], words[3]);
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

}  // namespace gemm_tc
