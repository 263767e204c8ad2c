// Persistent forward kernel: one cooperative launch runs a whole decoder forward over up to 32
// rows (the verification of one draft tree at batch 1, an autoregressive step, one level of the
// draft model): embedding, every layer (RMSNorm + QKV + RoPE + cache append, tree-mask attention,
// O projection + residual, RMSNorm + gate/up + SwiGLU, down projection + residual), the LM head
// and the greedy argmax (Eq. 1) or the draft model's log-softmax top-k (Eq. 2).
//
// Why one kernel: at these row counts a forward is one pass over the weights (13.2 GB for the
// 7B-shaped target), and with one launch per GEMM every launch pays a start, a drain and a
// boundary during which HBM idles. Here the weight stream never stops:
//
//  * Every CTA (one per SM) owns a fixed share of every weight matrix: matrix g is U_g units of
//    32 KB (one 256-row tile x 64 K, repacked and pre-swizzled by pack_weights_kernel) and CTA c
//    streams units [c U_g / G, (c + 1) U_g / G) - contiguous in HBM, perfectly balanced, whatever
//    the matrix shape.
//  * A producer thread issues those bulk copies into a four-stage shared-memory ring, matrix
//    after matrix, with no dependency on the computation: it runs ahead of the MMAs as far as the
//    ring allows, so the first stages of the next matrix are already on the SM when its
//    activations become available.
//  * The activation operand (both bf16 limbs of up to 32 rows) is kept in global memory in the
//    same K-block-major, pre-swizzled form (8 KB per K block), written by the epilogue of the
//    phase that produces it and fetched per stage by a second loader thread once that phase is
//    complete on every CTA.
//  * A CTA's unit range covers parts of one or two (rarely more) output tiles. Each part is
//    accumulated in TMEM by tcgen05.mma (M = 128 weight rows x 2 halves, N = 64 = both limbs of 32
//    rows) and written as an fp32 partial tile to an L2-resident scratch. After a grid barrier the
//    partials of every tile are summed in CTA order (deterministic) by the epilogue warps of all
//    CTAs, which apply the fused epilogue and write the next operand; a second grid barrier
//    publishes it.
//  * Attention runs between the QKV and O phases on (head, key slice) units with the same
//    three-limb tensor-core arithmetic as attention.cuh; slices meet in global scratch.
//
// Warp roles: 0 weight producer, 1 MMA issuer, 2-9 epilogue / attention / reductions, 10 loader
// of the activation operand. Every wait (mbarrier, grid barrier) is bounded by p.wait_ns of
// %globaltimer and ends early once the status word is set; a CTA that gives up records a code,
// lets its copies land, frees its TMEM and returns. The grid barrier needs all CTAs resident:
// the kernel is launched cooperatively.
#pragma once
#include "epilogue.cuh"
#include "gemm_tc.cuh"

namespace pk {

using namespace gemm_tc;

constexpr int TN = 32;                              // activation rows (padded)
constexpr int THREADS = 352;                        // 11 warps
constexpr int EPI_THREADS = 256;                    // warps 2-9
constexpr int STAGES = 4;
constexpr int X_BLOCK_ELEMS = 2 * TN * BK;          // one K block of the operand: 2 limbs x 32 rows x 64
constexpr int X_STAGE_BYTES = X_BLOCK_ELEMS * 2;    // 8 KB
constexpr int STAGE_BYTES = W_STAGE_BYTES + X_STAGE_BYTES;
constexpr int ACC_COLS = 2 * TN;                    // accumulator columns of one 128-row half
constexpr int TMEM_COLS = 4 * ACC_COLS;             // two buffers x two halves
constexpr int PART_ELEMS = TN * BM;                 // fp32 elements of one partial tile
constexpr int MAX_SPLITS = 8;

#define SV_ERR_WAIT_GRID 5
#define SV_ERR_WAIT_XREADY 6

enum OpKind { OP_EMBED = 0, OP_GEMM = 1, OP_ATTN = 2 };
enum PostKind { POST_NONE = 0, POST_ARGMAX = 1, POST_TOPK = 2 };

// One phase of the forward. GEMM phases: out = epilogue(X W^T) with W packed [tiles][KB][32 KB].
struct Op {
  int kind, mode;              // OpKind; EpiMode for GEMM phases
  const bf16 *w;               // packed weights
  int tiles, KB;               // 256-row tiles (SwiGLU: 128 gate + 128 up rows) and K blocks per tile
  int N;                       // output columns (SwiGLU: F)
  const bf16 *xin;             // packed operand
  int use_scale;               // rows are scaled by rsqrt(mean(x^2) + eps) from the sums of squares
  int accumulate;              // EPI_RESID: x += result (else x = result)
  const float *gain;           // EPI_RESID: gain of the next RMSNorm folded into the operand written
  float *cache;                // EPI_QKV / attention: this layer's cache, [episode][2][max_seq][hd]
  size_t ep_stride;
  float *out;                  // EPI_PLAIN: [rows][ldo] logits (may be NULL); POST_ARGMAX phases write
                               // to Params::logits_out instead
  int ldo, lo, hi;             // EPI_PLAIN: argmax / top-k range over output columns
  int post;                    // PostKind after an EPI_PLAIN phase
  int tok_offset;              // POST_TOPK: token id of output column 0
};

struct Params {
  const Op *ops;
  int n_ops;
  int T;                       // rows, 1..32
  int max_seg;                 // partial tiles a CTA may produce per GEMM phase
  RowTable rt;
  const bf16 *embeds, *E;      // OP_EMBED: given rows / embedding matrix
  const float *gain0;          // gain of the first RMSNorm
  int d, hd, H, dh, max_seq;
  float eps, attn_scale;
  int nt;                      // d / 128: sums-of-squares slots per row
  float *x;                    // residual [32][d]
  float *ssq;                  // [32][nt]
  float *q;                    // [32][hd]
  bf16 *xn_pk, *ao_pk, *hid_pk;   // packed operands (K = d, hd, F)
  float *part;                 // [G][max_seg][32][256] partial tiles
  float *apart;                // [H * splits][32][dh + 4]: attention slices (output, max, sum)
  int splits;
  const float2 *rope_tab;
  float4 *cand;                // [32][2 * tiles]: (top-1 value, top-1 id, top-2 value, -) per 128 columns
  float *logits_out;           // [rows][ldo] of the POST_ARGMAX phase, or NULL
  int *greedy;                 // POST_ARGMAX
  float *margin;
  int *top_tok;                // POST_TOPK: [rows][SV_TOPK]
  float *top_lp;
  unsigned *bar;               // grid-barrier counter, zero at launch
  int *err;                    // status word
  unsigned long long wait_ns;
};

// ------------------------------------------------------------------------- small helpers
// First unit of CTA c when U units are dealt out to G CTAs (U * G < 2^31, checked by the host).
__device__ __forceinline__ int ubegin(int U, int c, int G) { return (int)((unsigned)U * (unsigned)c / (unsigned)G); }
// the CTA whose range holds unit u
__device__ __forceinline__ int uowner(int U, int u, int G) {
  int c = (int)(((unsigned)u * (unsigned)G) / (unsigned)U);
  while (c + 1 < G && ubegin(U, c + 1, G) <= u) c++;
  while (c > 0 && ubegin(U, c, G) > u) c--;
  return c;
}
__device__ __forceinline__ unsigned ld_acquire(const unsigned *p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ int ld_volatile(const int *p) {
  int v;
  asm volatile("ld.volatile.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
// Bounded mbarrier wait that also gives up once the status word is set.
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, const int *err, unsigned long long limit) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; i++)
      if (mbar_try_wait(bar, parity)) return true;
    if (ld_volatile(err) != 0 || global_ns() - t0 > limit) return false;
  }
}
__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// Offset (elements) of element (row t, column k) of the hi limb in a packed operand; the lo limb
// is TN * BK elements further. Rows are 128-byte lines whose 16-byte chunks are XOR-swizzled by
// the row, as the MMA's shared-memory descriptor expects.
__device__ __forceinline__ size_t pk_off(int t, int k) {
  return (size_t)(k >> 6) * X_BLOCK_ELEMS + (size_t)t * BK + ((((k & 63) >> 3) ^ (t & 7)) << 3) + (k & 7);
}
__device__ __forceinline__ void store_limbs4_pk(bf16 *buf, int t, int k, float4 v) {
  const float4 h = make_float4(__bfloat162float(__float2bfloat16(v.x)), __bfloat162float(__float2bfloat16(v.y)),
                               __bfloat162float(__float2bfloat16(v.z)), __bfloat162float(__float2bfloat16(v.w)));
  const size_t o = pk_off(t, k);
  store_bf16x4(buf + o, h);
  store_bf16x4(buf + o + TN * BK, make_float4(v.x - h.x, v.y - h.y, v.z - h.z, v.w - h.w));
}

using sv::top2_warp;

// Shared state of one CTA.
struct Cta {
  uint32_t ring, full, empty, tfull, tempty, xready;   // shared-memory addresses
  uint32_t tmem;
  int c, G;
};

// ------------------------------------------------------------------------- grid barrier
// All 256 epilogue threads of every CTA call this the same number of times. `epoch` counts calls.
__device__ __forceinline__ bool grid_barrier(const Params &p, int G, unsigned &epoch, int et, volatile int *s_ok) {
  // what this thread wrote is about to be read by other CTAs, partly through bulk copies (async
  // proxy). The CTA barrier orders every thread's writes before the elected thread's fence, which
  // is cumulative; its counterpart after the wait covers the reads of all threads.
  asm volatile("fence.proxy.async.global;" ::: "memory");
  epi_sync();
  if (et == 0) {
    epoch++;
    __threadfence();
    asm volatile("red.relaxed.gpu.global.add.u32 [%0], 1;" ::"l"(p.bar) : "memory");
    const unsigned target = epoch * (unsigned)G;
    bool ok = true;
    if (ld_acquire(p.bar) < target) {
      const uint64_t t0 = global_ns();
      for (;;) {
        if (ld_acquire(p.bar) >= target) break;
        if (ld_volatile(p.err) != 0 || global_ns() - t0 > p.wait_ns) {
          ok = false;
          break;
        }
      }
    }
    __threadfence();
    if (!ok) atomicCAS(p.err, 0, SV_ERR_WAIT_GRID);
    *s_ok = ok ? 1 : 0;
  }
  epi_sync();
  return *s_ok != 0;
}

// ------------------------------------------------------------------------- attention unit
// One (head, key slice) of the single row block: same arithmetic as attn::tree_attention_kernel
// (three-limb bf16 MMAs, fp32 online softmax), on the 256 epilogue threads, leaving the
// unnormalised output, the running maximum and the sum of the slice in p.apart.
template <int DH>
__device__ void attention_unit(const Params &p, const Op &op, unsigned char *smem, int tid, int h, int sp) {
  constexpr int RB = 32, KT = 32;
  constexpr int C4 = DH / 4, LD = DH + 8, LP = KT + 8, LS = KT + 4;
  constexpr int NLD = KT * C4 / EPI_THREADS, KS = DH / 16, NB = DH / 32, LO = DH + 4;
  bf16 *sQh = reinterpret_cast<bf16 *>(smem);
  bf16 *sQl = sQh + RB * LD;
  bf16 *sKh = sQl + RB * LD;
  bf16 *sKl = sKh + KT * LD;
  bf16 *sVh = sKl + KT * LD;
  bf16 *sVl = sVh + KT * LD;
  bf16 *sPh = sVl + KT * LD;
  bf16 *sPl = sPh + RB * LP;
  float *sS = reinterpret_cast<float *>(sPl + RB * LP);
  __shared__ int s_nvis[RB], s_tbase[RB], s_kmax;
  __shared__ uint32_t s_mask[RB][4];
  __shared__ float s_corr[RB], s_m[RB], s_l[RB];
  const int lane = tid & 31, warp = tid >> 5;
  const int mb = warp & 1, wq = warp >> 1;
  const int hd = p.hd, nrows = p.T;
  const int ep = p.rt.ep[0];
  const float *kbase = op.cache + (size_t)ep * op.ep_stride + (size_t)h * DH;
  const float *vbase = kbase + (size_t)p.max_seq * hd;

  float4 qv[RB * C4 / EPI_THREADS];
#pragma unroll
  for (int k = 0; k < RB * C4 / EPI_THREADS; k++) {
    const int i = tid + k * EPI_THREADS;
    const int r = i / C4, c = i % C4;
    qv[k] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (r < nrows) qv[k] = __ldcg(reinterpret_cast<const float4 *>(p.q + (size_t)r * hd + h * DH + c * 4));
  }
  epi_sync();                               // the previous unit's shared state is no longer read
  if (tid < RB) {
    int nv = 0, tb = 0, km = 0;
    uint32_t m[4] = {0, 0, 0, 0};
    if (tid < nrows) {
      nv = p.rt.nvis[tid];
      tb = p.rt.tbase[tid];
      km = nv;
#pragma unroll
      for (int w = 0; w < 4; w++) {
        m[w] = p.rt.mask[(size_t)tid * 4 + w];
        if (m[w]) km = max(km, tb + 32 * w + 32 - __clz(m[w]));
      }
    }
    s_nvis[tid] = nv;
    s_tbase[tid] = tb;
#pragma unroll
    for (int w = 0; w < 4; w++) s_mask[tid][w] = m[w];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) km = max(km, __shfl_xor_sync(0xffffffffu, km, o));
    if (tid == 0) s_kmax = min(km, p.max_seq);
  }
  epi_sync();
  const int kmax = s_kmax;
  const int tiles = (kmax + KT - 1) / KT;
  const int t0 = sp * tiles / p.splits, t1 = (sp + 1) * tiles / p.splits;

  float4 kreg[NLD], vreg[NLD];
  auto fetch = [&](int t) {
#pragma unroll
    for (int k = 0; k < NLD; k++) {
      const int i = tid + k * EPI_THREADS;
      const int slot = t * KT + i / C4, c = i % C4;
      if (slot < kmax) {
        kreg[k] = __ldcg(reinterpret_cast<const float4 *>(kbase + (size_t)slot * hd + c * 4));
        vreg[k] = __ldcg(reinterpret_cast<const float4 *>(vbase + (size_t)slot * hd + c * 4));
      } else {
        kreg[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        vreg[k] = kreg[k];
      }
    }
  };
  if (t0 < t1) fetch(t0);
#pragma unroll
  for (int k = 0; k < RB * C4 / EPI_THREADS; k++) {
    const int i = tid + k * EPI_THREADS;
    const int r = i / C4, c = i % C4;
    float4 v = qv[k];
    v.x *= p.attn_scale; v.y *= p.attn_scale; v.z *= p.attn_scale; v.w *= p.attn_scale;
    uint2 hi, lo;
    attn::split4(v, hi, lo);
    *reinterpret_cast<uint2 *>(sQh + r * LD + c * 4) = hi;
    *reinterpret_cast<uint2 *>(sQl + r * LD + c * 4) = lo;
  }
  epi_sync();
  uint32_t qh[KS][4], ql[KS][4];
  {
    const int r = 16 * mb + (lane & 15), c = (lane >> 4) * 8;
#pragma unroll
    for (int ks = 0; ks < KS; ks++) {
      attn::ldsm_x4(attn::smem_addr(sQh + r * LD + 16 * ks + c), qh[ks]);
      attn::ldsm_x4(attn::smem_addr(sQl + r * LD + 16 * ks + c), ql[ks]);
    }
  }
  float m_run = -INFINITY, l_run = 0.f;
  float acc[NB][4];
#pragma unroll
  for (int nb = 0; nb < NB; nb++)
#pragma unroll
    for (int k = 0; k < 4; k++) acc[nb][k] = 0.f;

  for (int t = t0; t < t1; t++) {
    epi_sync();
#pragma unroll
    for (int k = 0; k < NLD; k++) {
      const int i = tid + k * EPI_THREADS;
      const int j = i / C4, c = i % C4;
      uint2 hi, lo;
      attn::split4(kreg[k], hi, lo);
      *reinterpret_cast<uint2 *>(sKh + j * LD + c * 4) = hi;
      *reinterpret_cast<uint2 *>(sKl + j * LD + c * 4) = lo;
      attn::split4(vreg[k], hi, lo);
      *reinterpret_cast<uint2 *>(sVh + j * LD + c * 4) = hi;
      *reinterpret_cast<uint2 *>(sVl + j * LD + c * 4) = lo;
    }
    epi_sync();
    if (t + 1 < t1) fetch(t + 1);
    {
      float sc[4] = {0.f, 0.f, 0.f, 0.f}, sc1[4] = {0.f, 0.f, 0.f, 0.f}, sc2[4] = {0.f, 0.f, 0.f, 0.f};
      const int key = 8 * wq + (lane & 7), c = (lane >> 3) * 8;
#pragma unroll
      for (int kp = 0; kp < KS / 2; kp++) {
        uint32_t bh[4], bl[4];
        attn::ldsm_x4(attn::smem_addr(sKh + key * LD + 32 * kp + c), bh);
        attn::ldsm_x4(attn::smem_addr(sKl + key * LD + 32 * kp + c), bl);
        attn::mma_bf16(sc, qh[2 * kp], bh[0], bh[1]);
        attn::mma_bf16(sc1, qh[2 * kp], bl[0], bl[1]);
        attn::mma_bf16(sc2, ql[2 * kp], bh[0], bh[1]);
        attn::mma_bf16(sc, qh[2 * kp + 1], bh[2], bh[3]);
        attn::mma_bf16(sc1, qh[2 * kp + 1], bl[2], bl[3]);
        attn::mma_bf16(sc2, ql[2 * kp + 1], bh[2], bh[3]);
      }
#pragma unroll
      for (int k = 0; k < 4; k++) sc[k] += sc1[k] + sc2[k];
      float *dst = sS + (16 * mb + (lane >> 2)) * LS + 8 * wq + 2 * (lane & 3);
      *reinterpret_cast<float2 *>(dst) = make_float2(sc[0], sc[1]);
      *reinterpret_cast<float2 *>(dst + 8 * LS) = make_float2(sc[2], sc[3]);
    }
    epi_sync();
    {
      const int r = warp * 4 + (lane >> 3), tc = lane & 7;
      const int nv = s_nvis[r], tb = s_tbase[r];
      float sv[4];
      bool vis[4];
      float mx = -INFINITY;
#pragma unroll
      for (int j = 0; j < 4; j++) {
        const int slot = t * KT + tc + 8 * j;
        vis[j] = slot < nv;
        const int b = slot - tb;
        if (!vis[j] && b >= 0 && b < 128) vis[j] = (s_mask[r][b >> 5] >> (b & 31)) & 1u;
        sv[j] = sS[r * LS + tc + 8 * j];
        if (vis[j]) mx = fmaxf(mx, sv[j]);
      }
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
      const float mn = fmaxf(m_run, mx);
      const float corr = (mn == -INFINITY) ? 1.f : __expf(m_run - mn);
      m_run = mn;
      float ps = 0.f;
#pragma unroll
      for (int j = 0; j < 4; j++) {
        const float pv = vis[j] ? __expf(sv[j] - mn) : 0.f;
        ps += pv;
        const bf16 ph = __float2bfloat16(pv);
        sPh[r * LP + tc + 8 * j] = ph;
        sPl[r * LP + tc + 8 * j] = __float2bfloat16(pv - __bfloat162float(ph));
      }
      ps += __shfl_xor_sync(0xffffffffu, ps, 1);
      ps += __shfl_xor_sync(0xffffffffu, ps, 2);
      ps += __shfl_xor_sync(0xffffffffu, ps, 4);
      l_run = l_run * corr + ps;
      if (tc == 0) s_corr[r] = corr;
    }
    epi_sync();
    {
      const float c0 = s_corr[16 * mb + (lane >> 2)], c1 = s_corr[16 * mb + (lane >> 2) + 8];
#pragma unroll
      for (int nb = 0; nb < NB; nb++) {
        acc[nb][0] *= c0;
        acc[nb][1] *= c0;
        acc[nb][2] *= c1;
        acc[nb][3] *= c1;
      }
      const int pr = 16 * mb + (lane & 15), pc = (lane >> 4) * 8;
      const int vk = (lane & 7) + ((lane >> 3) & 1) * 8, vc = (DH / 4) * wq + (lane >> 4) * 8;
#pragma unroll
      for (int ks = 0; ks < KT / 16; ks++) {
        uint32_t ph[4], pl[4];
        attn::ldsm_x4(attn::smem_addr(sPh + pr * LP + 16 * ks + pc), ph);
        attn::ldsm_x4(attn::smem_addr(sPl + pr * LP + 16 * ks + pc), pl);
#pragma unroll
        for (int np = 0; np < NB / 2; np++) {
          uint32_t vh[4], vl[4];
          attn::ldsm_x4_trans(attn::smem_addr(sVh + (16 * ks + vk) * LD + vc + 16 * np), vh);
          attn::ldsm_x4_trans(attn::smem_addr(sVl + (16 * ks + vk) * LD + vc + 16 * np), vl);
          attn::mma_bf16(acc[2 * np], ph, vh[0], vh[1]);
          attn::mma_bf16(acc[2 * np], ph, vl[0], vl[1]);
          attn::mma_bf16(acc[2 * np], pl, vh[0], vh[1]);
          attn::mma_bf16(acc[2 * np + 1], ph, vh[2], vh[3]);
          attn::mma_bf16(acc[2 * np + 1], ph, vl[2], vl[3]);
          attn::mma_bf16(acc[2 * np + 1], pl, vh[2], vh[3]);
        }
      }
    }
  }
  if ((lane & 7) == 0) {
    s_m[warp * 4 + (lane >> 3)] = m_run;
    s_l[warp * 4 + (lane >> 3)] = l_run;
  }
  epi_sync();
  // the slice goes to global scratch: [unit][row][DH output | max | sum | -]
  float *dst = p.apart + (size_t)(h * p.splits + sp) * RB * LO;
  const int ra = 16 * mb + (lane >> 2), rb = ra + 8;
  const int cbase = (DH / 4) * wq + 2 * (lane & 3);
#pragma unroll
  for (int nb = 0; nb < NB; nb++) {
    *reinterpret_cast<float2 *>(dst + ra * LO + cbase + 8 * nb) = make_float2(acc[nb][0], acc[nb][1]);
    *reinterpret_cast<float2 *>(dst + rb * LO + cbase + 8 * nb) = make_float2(acc[nb][2], acc[nb][3]);
  }
  if (tid < RB) {
    dst[tid * LO + DH] = s_m[tid];
    dst[tid * LO + DH + 1] = s_l[tid];
  }
}

// ------------------------------------------------------------------------- finishing a GEMM phase
constexpr int MAX_G = 192;                          // CTAs the unit tables are sized for
constexpr int MAX_TILES = 512;                      // output tiles of one matrix

struct RowInfo {
  const float *scale;          // RMSNorm scale per row (shared memory)
  const int *pos, *slot, *ep;  // RoPE position, cache slot, episode per row (shared memory)
  const int *begin;            // first unit of every CTA in this phase, [G + 1] (shared memory)
  const unsigned short *cf, *cl;   // first and last CTA that hold units of each output tile (shared memory)
};

// What remains of a GEMM phase once every CTA's partial tiles are in global scratch: work items of
// one row x 128 output columns (SwiGLU: 128 gate + 128 up columns) are dealt out to the epilogue
// warps of the whole grid; a warp sums the item's partial tiles in CTA order (deterministic) and
// applies the phase's epilogue. IB items are handled together, the first NB partial tiles of each
// loaded together before anything is used (loads from L2 take a microsecond: a warp that
// waited for each in turn would need several). A tile shared by more CTAs takes further batches.
template <int MODE, int IB, int NB>
__device__ __forceinline__ void finish_phase(const Params &p, const Op &o, const RowInfo &ri, int T, int G,
                                             int gw, int GW, int lane) {
  constexpr bool SW = MODE == EPI_SWIGLU;
  constexpr int halves = SW ? 1 : 2;
  const int n_items = o.tiles * T * halves;
  const int colbase = lane * 4;
  for (int base = gw; base < n_items; base += GW * IB) {
    int jj[IB], tt[IB], hh[IB], cfs[IB], cls[IB];
    float4 a[IB][NB], b[IB][SW ? NB : 1];
    // operands that do not depend on the partial tiles: residual and gain (EPI_RESID), RoPE factors
    // (EPI_QKV), requested in the same round
    float4 ex0[IB], ex1[IB];
    // first batch of partial tiles of every item
#pragma unroll
    for (int k = 0; k < IB; k++) {
      const int item = base + k * GW;
      jj[k] = -1;
      if (item < n_items) {
        const int j = item / (T * halves);
        const int rem = item - j * (T * halves);
        jj[k] = j;
        tt[k] = rem / halves;
        hh[k] = rem - tt[k] * halves;
        cfs[k] = ri.cf[j];
        cls[k] = ri.cl[j];
        const int n = j * BM + hh[k] * 128 + colbase;
        ex0[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        ex1[k] = make_float4(1.f, 1.f, 1.f, 1.f);
        if (MODE == EPI_RESID && n < o.N) {
          if (o.accumulate) ex0[k] = __ldcg(reinterpret_cast<const float4 *>(p.x + (size_t)tt[k] * o.N + n));
          if (o.gain) ex1[k] = *reinterpret_cast<const float4 *>(o.gain + n);
        }
        if (MODE == EPI_QKV) {
          const int which = n / p.hd, jq = (n - which * p.hd) & (p.dh - 1), half = p.dh >> 1;
          if (which < 2) {
            const float2 *cs = p.rope_tab + (size_t)ri.pos[tt[k]] * half + (jq < half ? jq : jq - half);
            ex0[k] = *reinterpret_cast<const float4 *>(cs);
            ex1[k] = *reinterpret_cast<const float4 *>(cs + 2);
          }
        }
      }
#pragma unroll
      for (int i = 0; i < NB; i++) {
        a[k][i] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (SW) b[k][i] = a[k][i];
        if (jj[k] >= 0 && cfs[k] + i <= cls[k]) {
          const int cc = cfs[k] + i;
          const int cb = ri.begin[cc];
          if (cb != ri.begin[cc + 1]) {                                 // a CTA without units adds nothing
            // only the first CTA of a tile can have begun in an earlier tile
            const int seg = i == 0 ? jj[k] - cb / o.KB : 0;
            const float *src = p.part + (((size_t)cc * p.max_seg + seg) * TN + tt[k]) * BM + hh[k] * 128 + colbase;
            a[k][i] = __ldcg(reinterpret_cast<const float4 *>(src));
            if (SW) b[k][i] = __ldcg(reinterpret_cast<const float4 *>(src + 128));
          }
        }
      }
    }
#pragma unroll
    for (int k = 0; k < IB; k++) {
      if (jj[k] < 0) continue;
      const int j = jj[k], t = tt[k], hf = hh[k];
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f), v2 = v;
#pragma unroll
      for (int i = 0; i < NB; i++) {
        v.x += a[k][i].x; v.y += a[k][i].y; v.z += a[k][i].z; v.w += a[k][i].w;
        if (SW) { v2.x += b[k][i].x; v2.y += b[k][i].y; v2.z += b[k][i].z; v2.w += b[k][i].w; }
      }
      // further batches (tiles shared by more than NB CTAs)
      for (int c0 = cfs[k] + NB; c0 <= cls[k]; c0 += NB) {
        float4 e[NB], f[SW ? NB : 1];
#pragma unroll
        for (int i = 0; i < NB; i++) {
          e[i] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (SW) f[i] = e[i];
          const int cc = c0 + i;
          if (cc <= cls[k] && ri.begin[cc] != ri.begin[cc + 1]) {
            const float *src = p.part + (((size_t)cc * p.max_seg) * TN + t) * BM + hf * 128 + colbase;
            e[i] = __ldcg(reinterpret_cast<const float4 *>(src));
            if (SW) f[i] = __ldcg(reinterpret_cast<const float4 *>(src + 128));
          }
        }
#pragma unroll
        for (int i = 0; i < NB; i++) {
          v.x += e[i].x; v.y += e[i].y; v.z += e[i].z; v.w += e[i].w;
          if (SW) { v2.x += f[i].x; v2.y += f[i].y; v2.z += f[i].z; v2.w += f[i].w; }
        }
      }
      const float sc = o.use_scale ? ri.scale[t] : 1.f;
      const int col = hf * 128 + colbase;                  // first of this lane's four columns within the tile
      if (MODE == EPI_QKV) {
        const int n = j * BM + col;
        const int which = n / p.hd, cq = n - which * p.hd;
        const int half = p.dh >> 1, jq = cq & (p.dh - 1);
        const bool lo = jq < half;
        float4 ov = make_float4(sc * v.x, sc * v.y, sc * v.z, sc * v.w);
        // the rotation partner (dh / 2 columns away) sits dh / 8 lanes away in the same warp
        const int dl = p.dh >> 3;
        const float wx = __shfl_xor_sync(0xffffffffu, ov.x, dl), wy = __shfl_xor_sync(0xffffffffu, ov.y, dl);
        const float wz = __shfl_xor_sync(0xffffffffu, ov.z, dl), ww = __shfl_xor_sync(0xffffffffu, ov.w, dl);
        if (which < 2) {
          const float4 cs01 = ex0[k], cs23 = ex1[k];
          const float sg = lo ? -1.f : 1.f;
          ov.x = ov.x * cs01.x + sg * wx * cs01.y;
          ov.y = ov.y * cs01.z + sg * wy * cs01.w;
          ov.z = ov.z * cs23.x + sg * wz * cs23.y;
          ov.w = ov.w * cs23.z + sg * ww * cs23.w;
        }
        if (n < o.N) {
          float *dst = which == 0 ? p.q + (size_t)t * p.hd + cq
                                  : o.cache + (size_t)ri.ep[t] * o.ep_stride +
                                        ((size_t)(which - 1) * p.max_seq + ri.slot[t]) * p.hd + cq;
          *reinterpret_cast<float4 *>(dst) = ov;
        }
      } else if (SW) {
        const int n = j * 128 + col;
        if (n < o.N) {
          const float gx = sc * v.x, gy = sc * v.y, gz = sc * v.z, gw2 = sc * v.w;
          store_limbs4_pk(p.hid_pk, t, n,
                          make_float4(__fdividef(gx, 1.f + __expf(-gx)) * (sc * v2.x),
                                      __fdividef(gy, 1.f + __expf(-gy)) * (sc * v2.y),
                                      __fdividef(gz, 1.f + __expf(-gz)) * (sc * v2.z),
                                      __fdividef(gw2, 1.f + __expf(-gw2)) * (sc * v2.w)));
        }
      } else if (MODE == EPI_RESID) {
        const int n = j * BM + col;
        float s2 = 0.f;
        if (n < o.N) {
          float *xp = p.x + (size_t)t * o.N + n;
          const float4 xo = ex0[k], g = ex1[k];
          v.x += xo.x; v.y += xo.y; v.z += xo.z; v.w += xo.w;
          *reinterpret_cast<float4 *>(xp) = v;
          store_limbs4_pk(p.xn_pk, t, n, make_float4(v.x * g.x, v.y * g.y, v.z * g.z, v.w * g.w));
          s2 = (v.x * v.x + v.y * v.y) + (v.z * v.z + v.w * v.w);
        }
        s2 = warp_sum(s2);
        if (lane == 0 && j * 2 + hf < p.nt) p.ssq[t * p.nt + j * 2 + hf] = s2;
      } else {
        // EPI_PLAIN: logits of 128 columns; their top-2 over [lo, hi) for the argmax
        const int n = j * BM + col;
        const float4 ov = make_float4(sc * v.x, sc * v.y, sc * v.z, sc * v.w);
        float *outp = o.post == POST_ARGMAX ? p.logits_out : o.out;
        if (outp && n < o.N) *reinterpret_cast<float4 *>(outp + (size_t)t * o.ldo + n) = ov;
        if (o.post == POST_ARGMAX) {
          epi::Top2 bb{-INFINITY, -INFINITY, 0x7fffffff};
          const float vv[4] = {ov.x, ov.y, ov.z, ov.w};
#pragma unroll
          for (int e2 = 0; e2 < 4; e2++)
            if (n + e2 >= o.lo && n + e2 < o.hi) epi::top2_push(bb, vv[e2], n + e2);
          top2_warp(bb);
          if (lane == 0) p.cand[(size_t)t * (2 * o.tiles) + j * 2 + hf] = make_float4(bb.v1, __int_as_float(bb.i1), bb.v2, 0.f);
        }
      }
    }
  }
}

template <int DH> __host__ __device__ constexpr int attn_smem_bytes() {
  return (2 * (32 + 2 * 32) * (DH + 8) + 2 * 32 * (32 + 8)) * (int)sizeof(bf16) + 32 * (32 + 4) * (int)sizeof(float);
}
template <int DH> __host__ __device__ constexpr int smem_bytes() { return STAGES * STAGE_BYTES + attn_smem_bytes<DH>() + 1024 + 128; }

// ------------------------------------------------------------------------- the kernel
template <int DH>
__global__ void __launch_bounds__(THREADS, 1) forward_pk_kernel(const __grid_constant__ Params p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char *ring_ptr = smem_raw + (ring - smem_u32(smem_raw));
  unsigned char *attn_smem = ring_ptr + STAGES * STAGE_BYTES;
  const uint32_t bars = ring + STAGES * STAGE_BYTES + attn_smem_bytes<DH>();
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
  auto tfull_bar = [&](int b) { return bars + 8u * (2 * STAGES + b); };
  auto tempty_bar = [&](int b) { return bars + 8u * (2 * STAGES + 2 + b); };
  const uint32_t xready_bar = bars + 8u * (2 * STAGES + 4);
  const uint32_t tmem_slot = bars + 8u * (2 * STAGES + 5);
  __shared__ int s_ok, s_gok;              // results of bounded waits, shared by the epilogue threads
  __shared__ int s_begin[MAX_G + 1];       // first unit of every CTA in the GEMM phase being run
  __shared__ unsigned short s_cf[MAX_TILES], s_cl[MAX_TILES];   // CTAs that share each of its output tiles
  __shared__ float s_scale[TN];            // RMSNorm scale of each row for the phase being finished
  __shared__ int s_pos[TN], s_slot[TN], s_ep[TN];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int c = blockIdx.x, G = gridDim.x;
  const int T = p.T;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; s++) {
      mbar_init(full_bar(s), 2);            // weight producer + operand loader
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; b++) {
      mbar_init(tfull_bar(b), 1);
      mbar_init(tempty_bar(b), 1);
    }
    mbar_init(xready_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    tc_alloc(tmem_slot, TMEM_COLS);
    tc_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  uint32_t tmem_base;
  asm volatile("ld.shared.b32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));

  if (warp == 0) {
    // ---------------------------------------------------------------- weight producer
    if (lane == 0) {
      const uint64_t pol_w = policy_evict_first();
      uint32_t it = 0;
      bool ok = true;
      for (int oi = 0; oi < p.n_ops && ok; oi++) {
        const Op &o = p.ops[oi];
        if (o.kind != OP_GEMM) continue;
        const int U = o.tiles * o.KB;
        const int ub = ubegin(U, c, G), ue = ubegin(U, c + 1, G);
        const bf16 *w = o.w;
        for (int u = ub; u < ue; u++, it++) {
          const int st = it % STAGES;
          const uint32_t rnd = it / STAGES;
          if (rnd > 0 && !wait_bar(empty_bar(st), (rnd - 1) & 1, p.err, p.wait_ns)) {
            atomicCAS(p.err, 0, SV_ERR_WAIT_EMPTY);
            ok = false;
            break;
          }
          mbar_expect_tx(full_bar(st), W_STAGE_BYTES);
          bulk_load(ring + st * STAGE_BYTES, w + (size_t)u * (BM * BK), W_STAGE_BYTES, full_bar(st), pol_w);
        }
      }
    }
    __syncwarp();
  } else if (warp == 10) {
    // ---------------------------------------------------------------- operand loader
    if (lane == 0) {
      const uint64_t pol_x = policy_evict_last();
      uint32_t it = 0, g = 0;
      bool ok = true;
      for (int oi = 0; oi < p.n_ops && ok; oi++) {
        const Op &o = p.ops[oi];
        if (o.kind != OP_GEMM) continue;
        // the phase that writes this operand is complete on every CTA
        if (!wait_bar(xready_bar, g & 1, p.err, p.wait_ns)) {
          atomicCAS(p.err, 0, SV_ERR_WAIT_XREADY);
          break;
        }
        g++;
        asm volatile("fence.proxy.async.global;" ::: "memory");
        const int U = o.tiles * o.KB;
        const int ub = ubegin(U, c, G), ue = ubegin(U, c + 1, G);
        for (int u = ub; u < ue; u++, it++) {
          const int st = it % STAGES;
          const uint32_t rnd = it / STAGES;
          if (rnd > 0 && !wait_bar(empty_bar(st), (rnd - 1) & 1, p.err, p.wait_ns)) {
            atomicCAS(p.err, 0, SV_ERR_WAIT_EMPTY);
            ok = false;
            break;
          }
          const int kb = u % o.KB;
          mbar_expect_tx(full_bar(st), X_STAGE_BYTES);
          bulk_load(ring + st * STAGE_BYTES + W_STAGE_BYTES, o.xin + (size_t)kb * X_BLOCK_ELEMS, X_STAGE_BYTES,
                    full_bar(st), pol_x);
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc = instr_desc(ACC_COLS);
      uint32_t it = 0, segc = 0;
      bool ok = true;
      for (int oi = 0; oi < p.n_ops && ok; oi++) {
        const Op &o = p.ops[oi];
        if (o.kind != OP_GEMM) continue;
        const int U = o.tiles * o.KB;
        const int ub = ubegin(U, c, G), ue = ubegin(U, c + 1, G);
        int u = ub;
        while (u < ue && ok) {
          const int kb0 = u % o.KB;
          const int n = min(ue - u, o.KB - kb0);
          const uint32_t buf = segc & 1, use = segc >> 1;
          if (use > 0 && !wait_bar(tempty_bar(buf), (use - 1) & 1, p.err, p.wait_ns)) {
            atomicCAS(p.err, 0, SV_ERR_WAIT_TMEM_EMPTY);
            ok = false;
            break;
          }
          tc_fence_after();
          for (int i = 0; i < n; i++, it++) {
            const int st = it % STAGES;
            if (!wait_bar(full_bar(st), (it / STAGES) & 1, p.err, p.wait_ns)) {
              atomicCAS(p.err, 0, SV_ERR_WAIT_FULL);
              ok = false;
              break;
            }
            tc_fence_after();
            const uint32_t sW = ring + st * STAGE_BYTES, sX = sW + W_STAGE_BYTES;
#pragma unroll
            for (int kk = 0; kk < BK / 16; kk++) {
#pragma unroll
              for (int h = 0; h < 2; h++) {
                const uint64_t adesc = smem_desc(sW + h * (128 * BK * 2) + kk * 32);
                const uint32_t d = tmem_base + buf * (2 * ACC_COLS) + (uint32_t)(h * ACC_COLS);
                tc_mma(d, adesc, smem_desc(sX + kk * 32), idesc, (i == 0 && kk == 0) ? 0u : 1u);
              }
            }
            tc_commit(empty_bar(st));
          }
          if (!ok) break;
          tc_commit(tfull_bar(buf));
          segc++;
          u += n;
        }
      }
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------------- epilogue warps
    const int et = threadIdx.x - 64, ew = warp - 2;
    const int gw = c * 8 + ew, GW = G * 8;          // this warp among the grid's epilogue warps
    unsigned epoch = 0;
    uint32_t segc = 0;
    bool alive = true;
    if (et < TN) {
      const bool in = et < T;
      s_pos[et] = in ? p.rt.pos[et] : 0;
      s_slot[et] = in ? p.rt.slot[et] : 0;
      s_ep[et] = in ? p.rt.ep[et] : 0;
    }
    epi_sync();
    for (int oi = 0; oi < p.n_ops && alive; oi++) {
      const Op o = p.ops[oi];                        // a private copy: the fields are used after fences
      if (o.kind == OP_EMBED) {
        // x = input rows; xn = limbs(x * gain0) packed; ssq per 128 columns
        for (int item = gw; item < T * p.nt; item += GW) {
          const int t = item / p.nt, ch = item - t * p.nt;
          const int k = ch * 128 + lane * 4;
          const int tok = p.rt.tok[t];
          const bf16 *src = tok >= 0 ? p.E + (size_t)tok * p.d : p.embeds + (size_t)p.rt.src[t] * p.d;
          const float4 v = load_bf16x4(src + k);
          const float4 g = *reinterpret_cast<const float4 *>(p.gain0 + k);
          *reinterpret_cast<float4 *>(p.x + (size_t)t * p.d + k) = v;
          store_limbs4_pk(p.xn_pk, t, k, make_float4(v.x * g.x, v.y * g.y, v.z * g.z, v.w * g.w));
          const float ss = warp_sum(v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w);
          if (lane == 0) p.ssq[t * p.nt + ch] = ss;
        }
        if (!grid_barrier(p, G, epoch, et, &s_gok)) break;
        continue;
      }
      if (o.kind == OP_ATTN) {
        const int units = p.H * p.splits;
        for (int un = c; un < units; un += G) attention_unit<DH>(p, o, attn_smem, et, un / p.splits, un % p.splits);
        if (!grid_barrier(p, G, epoch, et, &s_gok)) break;
        // merge of the key slices: one warp per (row, head); the O projection's operand
        constexpr int LO = DH + 4, PER = DH / 32;
        for (int item = gw; item < T * p.H; item += GW) {
          const int t = item / p.H, h = item - t * p.H;
          float ms[MAX_SPLITS], ls[MAX_SPLITS], os[MAX_SPLITS][PER];
#pragma unroll
          for (int s2 = 0; s2 < MAX_SPLITS; s2++)
            if (s2 < p.splits) {
              const float *src = p.apart + ((size_t)(h * p.splits + s2) * 32 + t) * LO;
              ms[s2] = __ldcg(src + DH);
              ls[s2] = __ldcg(src + DH + 1);
              if (PER == 4) {
                const float4 t4 = __ldcg(reinterpret_cast<const float4 *>(src + lane * 4));
                os[s2][0] = t4.x; os[s2][1] = t4.y; os[s2][2 % PER] = t4.z; os[s2][3 % PER] = t4.w;
              } else {
                const float2 t2 = __ldcg(reinterpret_cast<const float2 *>(src + lane * 2));
                os[s2][0] = t2.x; os[s2][1] = t2.y;
              }
            }
          float M = -INFINITY;
#pragma unroll
          for (int s2 = 0; s2 < MAX_SPLITS; s2++)
            if (s2 < p.splits) M = fmaxf(M, ms[s2]);
          float L = 0.f, ov[PER];
#pragma unroll
          for (int k = 0; k < PER; k++) ov[k] = 0.f;
#pragma unroll
          for (int s2 = 0; s2 < MAX_SPLITS; s2++)
            if (s2 < p.splits) {
              const float cf = (ms[s2] == -INFINITY) ? 0.f : __expf(ms[s2] - M);
              L += ls[s2] * cf;
#pragma unroll
              for (int k = 0; k < PER; k++) ov[k] += os[s2][k] * cf;
            }
          const float inv = 1.f / L;
          const int k0 = h * DH + lane * PER;
          if (PER == 4) {
            store_limbs4_pk(p.ao_pk, t, k0, make_float4(ov[0] * inv, ov[1] * inv, ov[2 % PER] * inv, ov[3 % PER] * inv));
          } else {
            const size_t off = pk_off(t, k0);
            const __nv_bfloat162 hi = __floats2bfloat162_rn(ov[0] * inv, ov[1] * inv);
            const float2 hf = __bfloat1622float2(hi);
            *reinterpret_cast<__nv_bfloat162 *>(p.ao_pk + off) = hi;
            *reinterpret_cast<__nv_bfloat162 *>(p.ao_pk + off + TN * BK) =
                __floats2bfloat162_rn(ov[0] * inv - hf.x, ov[1] * inv - hf.y);
          }
        }
        if (!grid_barrier(p, G, epoch, et, &s_gok)) break;
        continue;
      }
      // -------------------------------------------------------------- GEMM phase
      if (et == 0) mbar_arrive(xready_bar);          // everything before this phase is complete
      // unit tables of this phase (the finishing code would otherwise divide its time away)
      const int U0 = o.tiles * o.KB;
      for (int i = et; i <= G; i += EPI_THREADS) s_begin[i] = ubegin(U0, i, G);
      for (int j = et; j < o.tiles; j += EPI_THREADS) {
        s_cf[j] = (unsigned short)uowner(U0, j * o.KB, G);
        s_cl[j] = (unsigned short)uowner(U0, (j + 1) * o.KB - 1, G);
      }
      if (o.use_scale) {
        // RMSNorm scales of the rows (their sums of squares are complete), once per CTA, while the
        // MMAs run; read after the grid barrier below
        for (int t = ew; t < T; t += 8) {
          float ss = 0.f;
          for (int i = lane; i < p.nt; i += 32) ss += __ldcg(p.ssq + t * p.nt + i);
          ss = warp_sum(ss);
          if (lane == 0) s_scale[t] = rsqrtf(ss / (float)p.d + p.eps);
        }
      }
      const int U = o.tiles * o.KB;
      const int ub = ubegin(U, c, G), ue = ubegin(U, c + 1, G);
      // part 1: each finished accumulator -> fp32 partial tile [t][256] in global scratch
      {
        int u = ub, seg = 0;
        const int q = warp & 3, wp = ew >> 2;          // TMEM lane quadrant of this warp; row group
        while (u < ue) {
          const int n = min(ue - u, o.KB - u % o.KB);
          const uint32_t buf = segc & 1, use = segc >> 1;
          if (et == 0) s_ok = wait_bar(tfull_bar(buf), use & 1, p.err, p.wait_ns) ? 1 : 0;
          epi_sync();
          if (!s_ok) {
            if (et == 0) atomicCAS(p.err, 0, SV_ERR_WAIT_TMEM_FULL);
            alive = false;
            break;
          }
          tc_fence_after();
          float *dst = p.part + ((size_t)c * p.max_seg + seg) * PART_ELEMS;
          const uint32_t tadr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * (2 * ACC_COLS);
          const int c0 = 16 * wp;
          if (c0 < T) {
#pragma unroll
            for (int hf = 0; hf < 2; hf++) {
              uint32_t r0[16], r1[16];
              tc_ld16(tadr + hf * ACC_COLS + c0, r0);
              tc_ld16(tadr + hf * ACC_COLS + TN + c0, r1);
              tc_wait_ld();
#pragma unroll
              for (int j = 0; j < 16; j++)
                if (c0 + j < T) dst[(c0 + j) * BM + hf * 128 + q * 32 + lane] = __uint_as_float(r0[j]) + __uint_as_float(r1[j]);
            }
          }
          tc_fence_before();
          epi_sync();
          if (et == 0) mbar_arrive(tempty_bar(buf));
          segc++;
          seg++;
          u += n;
        }
        if (!alive) break;
      }
      if (!grid_barrier(p, G, epoch, et, &s_gok)) break;
      // part 2: sum the partial tiles of every output tile in CTA order and finish
      const RowInfo ri{s_scale, s_pos, s_slot, s_ep, s_begin, s_cf, s_cl};
      switch (o.mode) {
        case EPI_QKV: finish_phase<EPI_QKV, 2, 6>(p, o, ri, T, G, gw, GW, lane); break;
        case EPI_SWIGLU: finish_phase<EPI_SWIGLU, 2, 3>(p, o, ri, T, G, gw, GW, lane); break;
        case EPI_RESID: finish_phase<EPI_RESID, 1, 12>(p, o, ri, T, G, gw, GW, lane); break;
        default: finish_phase<EPI_PLAIN, 3, 3>(p, o, ri, T, G, gw, GW, lane); break;
      }
      if (!grid_barrier(p, G, epoch, et, &s_gok)) break;
      if (o.post == POST_ARGMAX) {
        // one warp per row merges the per-128-column candidates (ties to the lowest id)
        for (int t = gw; t < T; t += GW) {
          epi::Top2 b{-INFINITY, -INFINITY, 0x7fffffff};
          for (int i = lane; i < 2 * o.tiles; i += 32) {
            const float4 cd = __ldcg(p.cand + (size_t)t * (2 * o.tiles) + i);
            epi::Top2 other{cd.x, cd.z, __float_as_int(cd.y)};
            epi::top2_merge(b, other);
          }
          top2_warp(b);
          if (lane == 0) {
            p.greedy[t] = b.i1;
            p.margin[t] = b.v1 - b.v2;
          }
        }
      } else if (o.post == POST_TOPK) {
        // draft scoring: log-softmax over columns [lo, hi) of the logits just written and their
        // SV_TOPK best entries (ties to the lowest id); one warp per row
        for (int t = gw; t < T; t += GW) {
          const float *lg = o.out + (size_t)t * o.ldo;
          float mx = -INFINITY;
          for (int v = o.lo + lane; v < o.hi; v += 32) mx = fmaxf(mx, __ldcg(lg + v));
          mx = warp_max(mx);
          float se = 0.f;
          for (int v = o.lo + lane; v < o.hi; v += 32) se += expf(__ldcg(lg + v) - mx);
          se = warp_sum(se);
          const float lse = mx + logf(se);
          int chosen[SV_TOPK];
          for (int k = 0; k < SV_TOPK; k++) {
            float bv = -INFINITY;
            int bi = 0x7fffffff;
            for (int v = o.lo + lane; v < o.hi; v += 32) {
              bool taken = false;
              for (int jj = 0; jj < k; jj++) taken |= (chosen[jj] == v);
              const float xv = __ldcg(lg + v);
              if (!taken && (xv > bv || (xv == bv && v < bi))) { bv = xv; bi = v; }
            }
#pragma unroll
            for (int of = 16; of > 0; of >>= 1) {
              const float ov = __shfl_xor_sync(0xffffffffu, bv, of);
              const int oi2 = __shfl_xor_sync(0xffffffffu, bi, of);
              if (ov > bv || (ov == bv && oi2 < bi)) { bv = ov; bi = oi2; }
            }
            chosen[k] = bi;
            if (lane == 0) {
              p.top_tok[t * SV_TOPK + k] = bi + o.tok_offset;
              p.top_lp[t * SV_TOPK + k] = bv - lse;
            }
          }
        }
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  if (ld_volatile(p.err) != 0) {
    // a wait gave up somewhere: let this CTA's copies in flight land before its shared memory goes
    const uint64_t t0 = global_ns();
    while (global_ns() - t0 < 200000ull) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) tc_dealloc(tmem_base, TMEM_COLS);
}

}  // namespace pk
