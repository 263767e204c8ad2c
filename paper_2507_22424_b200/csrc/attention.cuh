// Tree-mask attention (Section 3.2 / 4.1: every draft-tree row is verified in one forward,
// each conditioned on its own path). Row t attends cache slots [0, nvis[t]) plus the slots
// tbase[t] + b for every bit b of its 128-bit mask. Queries, keys and values are fp32 in
// memory; softmax and accumulation are fp32; the output is written as two bf16 limbs for the
// O-projection GEMM.
//
// One CTA handles one head, a block of up to 32 consecutive rows of ONE episode and one slice
// of that block's key range (split-KV). Keys and values go through shared memory in tiles of
// 32 slots, so a K/V row is read from L2/HBM once per row block instead of once per row; the
// next tile is fetched into registers while the current one is used.
//
// The two contractions run on the tensor cores with fp32-grade operands: every operand (q
// scaled, k, v, the softmax weights p) is split into two bf16 limbs (hi = bf16(x), lo =
// bf16(x - hi): 16 mantissa bits) when it is written to shared memory, and a product is three
// m16n8k16 MMAs (hi hi + hi lo + lo hi) accumulated in fp32. A tile goes through three phases
// separated by CTA barriers: scores (warp = 16 rows x 8 keys, q fragments kept in registers
// for the whole kernel), online softmax (warp = 4 rows, lane = key; running max and sum live
// in that warp's registers), weighted sum (warp = 16 rows x a quarter of the head dimension).
// With several key slices the CTAs of a row block form a thread-block cluster: each leaves
// (max, sum, unnormalised output) in its own shared memory, and after one cluster barrier
// every CTA merges a share of the rows, reading the slices over distributed shared memory in
// ascending order (deterministic; nothing goes through global memory).
#pragma once
#include <cooperative_groups.h>
#include "common.cuh"

namespace attn {

constexpr int RB = 32;            // rows per block
constexpr int KT = 32;            // key slots per tile
constexpr int THREADS = 256;      // 8 warps x 4 rows
constexpr int MAX_SPLITS = 8;         // key slices per row block = cluster size (8: the portable limit)
constexpr int MAX_SPLIT_CTAS = 148;   // CTAs of a launch that uses more than one key slice

struct Args {
  const float *q;          // [rows][H * DH], already rotated
  const float *cache;      // [episode][2 (K, V)][max_seq][H * DH]
  size_t ep_stride;
  int max_seq, H;
  RowTable rt;
  float scale;
  bf16 *out;               // two limbs, [rows][H * DH] each
  size_t out_plane;
  int splits;              // key slices per row block; the launch's cluster is (splits, 1, 1)
};

__host__ __device__ inline int blocks_of(const EpArgs &ea) {
  int n = 0;
  for (int i = 0; i < ea.n_ep; i++) n += (ea.nrows[i] + RB - 1) / RB;
  return n;
}
// Shared memory: bf16 limb planes of Q [RB], K [KT], V [KT] (row pitch DH + 8: rows 16-byte
// aligned and ldmatrix conflict-free), of P [RB][KT + 8], and the fp32 scores [RB][KT + 4].
template <int DH> constexpr int smem_bytes() {
  return (2 * (RB + 2 * KT) * (DH + 8) + 2 * RB * (KT + 8)) * (int)sizeof(bf16) + RB * (KT + 4) * (int)sizeof(float);
}

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// c += a (16 x 16, row) * b (16 x 8, col), bf16 operands, fp32 accumulator
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// four floats -> four hi limbs and four lo limbs, 8 bytes each
__device__ __forceinline__ void split4(const float4 v, uint2 &hi, uint2 &lo) {
  const __nv_bfloat162 h01 = __floats2bfloat162_rn(v.x, v.y), h23 = __floats2bfloat162_rn(v.z, v.w);
  const float2 f01 = __bfloat1622float2(h01), f23 = __bfloat1622float2(h23);
  const __nv_bfloat162 l01 = __floats2bfloat162_rn(v.x - f01.x, v.y - f01.y);
  const __nv_bfloat162 l23 = __floats2bfloat162_rn(v.z - f23.x, v.w - f23.y);
  hi = make_uint2(*reinterpret_cast<const uint32_t *>(&h01), *reinterpret_cast<const uint32_t *>(&h23));
  lo = make_uint2(*reinterpret_cast<const uint32_t *>(&l01), *reinterpret_cast<const uint32_t *>(&l23));
}

// SLICED: grid (row blocks x key slices, heads), cluster (slices, 1, 1): the few-row launches (a
// verification step, a draft level). Unsliced (prefill: more CTAs than SMs): grid (heads, row
// blocks), the blocks taken last to first: causal rows make the late blocks of an episode the long
// ones, and CTAs are handed out x first, so every head's longest block starts before any short one
// and the last wave is made of short blocks.
template <int DH, bool SLICED>
__global__ void __launch_bounds__(THREADS, 1)
tree_attention_kernel(const EpArgs ea, const Args a) {
  constexpr int PER = DH / 32;            // head-dim columns per lane in the slice merge
  constexpr int C4 = DH / 4;              // float4 per row
  constexpr int LD = DH + 8;              // pitch (bf16) of the Q, K, V limb planes
  constexpr int LP = KT + 8;              // pitch (bf16) of the P limb planes
  constexpr int LS = KT + 4;              // pitch (float) of the scores
  constexpr int NLD = KT * C4 / THREADS;  // float4 per thread per tile
  constexpr int KS = DH / 16;             // k steps of the score MMAs
  constexpr int NB = DH / 32;             // 8-column blocks of a warp's quarter of the head dim
  extern __shared__ __align__(16) unsigned char smem_raw[];
  bf16 *sQh = reinterpret_cast<bf16 *>(smem_raw);   // [RB][LD]
  bf16 *sQl = sQh + RB * LD;
  bf16 *sKh = sQl + RB * LD;                        // [KT][LD]
  bf16 *sKl = sKh + KT * LD;
  bf16 *sVh = sKl + KT * LD;
  bf16 *sVl = sVh + KT * LD;
  bf16 *sPh = sVl + KT * LD;                        // [RB][LP]
  bf16 *sPl = sPh + RB * LP;
  float *sS = reinterpret_cast<float *>(sPl + RB * LP);   // [RB][LS]
  __shared__ int s_nvis[RB], s_tbase[RB], s_kmax;
  __shared__ uint32_t s_mask[RB][4];
  __shared__ float s_corr[RB], s_m[RB], s_l[RB];
  // The GEMM that follows is let in only once the tile loop is over (pdl_launch below): its
  // waiting CTAs would otherwise take registers and shared memory and push this grid into waves.
  pdl_wait();

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int mb = warp & 1, wq = warp >> 1;         // 16-row block; key octet (scores) / head-dim quarter (sum)
  const int h = SLICED ? blockIdx.y : blockIdx.x, hd = a.H * DH;
  const int splits = SLICED ? a.splits : 1;
  int bid = SLICED ? (int)blockIdx.x / splits : (int)gridDim.y - 1 - (int)blockIdx.y;
  const int sp = SLICED ? (int)blockIdx.x - bid * splits : 0;
  int ei = 0;
  for (; ei < ea.n_ep; ei++) {
    const int nb = (ea.nrows[ei] + RB - 1) / RB;
    if (bid < nb) break;
    bid -= nb;
  }
  if (ei >= ea.n_ep) {
    pdl_launch();
    return;
  }
  const int row0 = ea.row0[ei] + bid * RB;
  const int nrows = min(RB, ea.nrows[ei] - bid * RB);
  const float *kbase = a.cache + (size_t)ea.eps[ei] * a.ep_stride + (size_t)h * DH;
  const float *vbase = kbase + (size_t)a.max_seq * hd;

  // the block's query rows (rows past nrows are zero): requested first, used after the metadata
  float4 qv[RB * C4 / THREADS];
#pragma unroll
  for (int k = 0; k < RB * C4 / THREADS; k++) {
    const int i = tid + k * THREADS;
    const int r = i / C4, c = i % C4;
    qv[k] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (r < nrows) qv[k] = *reinterpret_cast<const float4 *>(a.q + (size_t)(row0 + r) * hd + h * DH + c * 4);
  }
  if (tid < RB) {
    int nv = 0, tb = 0, km = 0;
    uint32_t m[4] = {0, 0, 0, 0};
    if (tid < nrows) {
      nv = a.rt.nvis[row0 + tid];
      tb = a.rt.tbase[row0 + tid];
      km = nv;
#pragma unroll
      for (int w = 0; w < 4; w++) {
        m[w] = a.rt.mask[(size_t)(row0 + tid) * 4 + w];
        if (m[w]) km = max(km, tb + 32 * w + 32 - __clz(m[w]));
      }
    }
    s_nvis[tid] = nv;
    s_tbase[tid] = tb;
#pragma unroll
    for (int w = 0; w < 4; w++) s_mask[tid][w] = m[w];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) km = max(km, __shfl_xor_sync(0xffffffffu, km, o));
    if (tid == 0) s_kmax = min(km, a.max_seq);
  }
  __syncthreads();
  const int kmax = s_kmax;
  const int tiles = (kmax + KT - 1) / KT;
  const int t0 = sp * tiles / splits, t1 = (sp + 1) * tiles / splits;

  float4 kreg[NLD], vreg[NLD];
  auto fetch = [&](int t) {
#pragma unroll
    for (int k = 0; k < NLD; k++) {
      const int i = tid + k * THREADS;
      const int slot = t * KT + i / C4, c = i % C4;
      if (slot < kmax) {
        kreg[k] = *reinterpret_cast<const float4 *>(kbase + (size_t)slot * hd + c * 4);
        vreg[k] = *reinterpret_cast<const float4 *>(vbase + (size_t)slot * hd + c * 4);
      } else {
        kreg[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        vreg[k] = kreg[k];
      }
    }
  };
  if (t0 < t1) fetch(t0);                  // in flight while the queries are split

  // the query rows, scaled, as limbs
#pragma unroll
  for (int k = 0; k < RB * C4 / THREADS; k++) {
    const int i = tid + k * THREADS;
    const int r = i / C4, c = i % C4;
    float4 v = qv[k];
    v.x *= a.scale; v.y *= a.scale; v.z *= a.scale; v.w *= a.scale;
    uint2 hi, lo;
    split4(v, hi, lo);
    *reinterpret_cast<uint2 *>(sQh + r * LD + c * 4) = hi;
    *reinterpret_cast<uint2 *>(sQl + r * LD + c * 4) = lo;
  }
  __syncthreads();

  // A fragments of this warp's 16 query rows, both limbs, for the whole kernel
  uint32_t qh[KS][4], ql[KS][4];
  {
    const int r = 16 * mb + (lane & 15), c = (lane >> 4) * 8;
#pragma unroll
    for (int ks = 0; ks < KS; ks++) {
      ldsm_x4(smem_addr(sQh + r * LD + 16 * ks + c), qh[ks]);
      ldsm_x4(smem_addr(sQl + r * LD + 16 * ks + c), ql[ks]);
    }
  }
  float m_run = -INFINITY, l_run = 0.f;   // softmax statistics of row 4 warp + lane / 8
  float acc[NB][4];                       // rows 16 mb + lane / 4 (+ 8), columns (DH / 4) wq + 8 nb + 2 (lane % 4) (+ 1)
#pragma unroll
  for (int nb = 0; nb < NB; nb++)
#pragma unroll
    for (int k = 0; k < 4; k++) acc[nb][k] = 0.f;

  for (int t = t0; t < t1; t++) {
    __syncthreads();                       // the previous tile is no longer being read
#pragma unroll
    for (int k = 0; k < NLD; k++) {
      const int i = tid + k * THREADS;
      const int j = i / C4, c = i % C4;
      uint2 hi, lo;
      split4(kreg[k], hi, lo);
      *reinterpret_cast<uint2 *>(sKh + j * LD + c * 4) = hi;
      *reinterpret_cast<uint2 *>(sKl + j * LD + c * 4) = lo;
      split4(vreg[k], hi, lo);
      *reinterpret_cast<uint2 *>(sVh + j * LD + c * 4) = hi;
      *reinterpret_cast<uint2 *>(sVl + j * LD + c * 4) = lo;
    }
    __syncthreads();
    if (t + 1 < t1) fetch(t + 1);          // in flight while this tile is used

    // ---- scores of rows 16 mb .. + 16 against keys 8 wq .. + 8
    {
      // three chains (hi hi, hi lo, lo hi) instead of one of 3 DH / 16 dependent MMAs
      float sc[4] = {0.f, 0.f, 0.f, 0.f}, sc1[4] = {0.f, 0.f, 0.f, 0.f}, sc2[4] = {0.f, 0.f, 0.f, 0.f};
      // B fragments two k steps at a time: lanes 0-7 / 8-15 address the keys' columns
      // 32 kp, 32 kp + 8 (first step), lanes 16-23 / 24-31 the columns 32 kp + 16, + 24 (second)
      const int key = 8 * wq + (lane & 7), c = (lane >> 3) * 8;
#pragma unroll
      for (int kp = 0; kp < KS / 2; kp++) {
        uint32_t bh[4], bl[4];
        ldsm_x4(smem_addr(sKh + key * LD + 32 * kp + c), bh);
        ldsm_x4(smem_addr(sKl + key * LD + 32 * kp + c), bl);
        mma_bf16(sc, qh[2 * kp], bh[0], bh[1]);
        mma_bf16(sc1, qh[2 * kp], bl[0], bl[1]);
        mma_bf16(sc2, ql[2 * kp], bh[0], bh[1]);
        mma_bf16(sc, qh[2 * kp + 1], bh[2], bh[3]);
        mma_bf16(sc1, qh[2 * kp + 1], bl[2], bl[3]);
        mma_bf16(sc2, ql[2 * kp + 1], bh[2], bh[3]);
      }
#pragma unroll
      for (int k = 0; k < 4; k++) sc[k] += sc1[k] + sc2[k];
      float *dst = sS + (16 * mb + (lane >> 2)) * LS + 8 * wq + 2 * (lane & 3);
      *reinterpret_cast<float2 *>(dst) = make_float2(sc[0], sc[1]);
      *reinterpret_cast<float2 *>(dst + 8 * LS) = make_float2(sc[2], sc[3]);
    }
    __syncthreads();
    // ---- online softmax: eight lanes per row (row 4 warp + lane / 8), a lane has the keys
    // lane % 8 + 8 j of the tile
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
        const float p = vis[j] ? __expf(sv[j] - mn) : 0.f;
        ps += p;
        const bf16 ph = __float2bfloat16(p);
        sPh[r * LP + tc + 8 * j] = ph;
        sPl[r * LP + tc + 8 * j] = __float2bfloat16(p - __bfloat162float(ph));
      }
      ps += __shfl_xor_sync(0xffffffffu, ps, 1);
      ps += __shfl_xor_sync(0xffffffffu, ps, 2);
      ps += __shfl_xor_sync(0xffffffffu, ps, 4);
      l_run = l_run * corr + ps;
      if (tc == 0) s_corr[r] = corr;
    }
    __syncthreads();
    // ---- weighted sum: rows 16 mb .. + 16, head-dim columns (DH / 4) wq .. + DH / 4
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
      // V fragments (transposed loads): lanes 0-7 / 8-15 address keys 16 ks .. + 8 / + 8 .. + 16
      // at one 8-column block, lanes 16-31 the same keys at the next block
      const int vk = (lane & 7) + ((lane >> 3) & 1) * 8, vc = (DH / 4) * wq + (lane >> 4) * 8;
#pragma unroll
      for (int ks = 0; ks < KT / 16; ks++) {
        uint32_t ph[4], pl[4];
        ldsm_x4(smem_addr(sPh + pr * LP + 16 * ks + pc), ph);
        ldsm_x4(smem_addr(sPl + pr * LP + 16 * ks + pc), pl);
#pragma unroll
        for (int np = 0; np < NB / 2; np++) {
          uint32_t vh[4], vl[4];
          ldsm_x4_trans(smem_addr(sVh + (16 * ks + vk) * LD + vc + 16 * np), vh);
          ldsm_x4_trans(smem_addr(sVl + (16 * ks + vk) * LD + vc + 16 * np), vl);
          mma_bf16(acc[2 * np], ph, vh[0], vh[1]);
          mma_bf16(acc[2 * np], ph, vl[0], vl[1]);
          mma_bf16(acc[2 * np], pl, vh[0], vh[1]);
          mma_bf16(acc[2 * np + 1], ph, vh[2], vh[3]);
          mma_bf16(acc[2 * np + 1], ph, vl[2], vl[3]);
          mma_bf16(acc[2 * np + 1], pl, vh[2], vh[3]);
        }
      }
    }
  }

  pdl_launch();
  if ((lane & 7) == 0) {
    s_m[warp * 4 + (lane >> 3)] = m_run;
    s_l[warp * 4 + (lane >> 3)] = l_run;
  }
  __syncthreads();
  const int ra = 16 * mb + (lane >> 2), rb = ra + 8;        // this thread's two rows
  const int cbase = (DH / 4) * wq + 2 * (lane & 3);          // + 8 nb: its column pairs
  if (splits == 1) {
    const float ia = 1.f / s_l[ra], ib = 1.f / s_l[rb];
#pragma unroll
    for (int nb = 0; nb < NB; nb++) {
#pragma unroll
      for (int half = 0; half < 2; half++) {
        const int r = half ? rb : ra;
        if (r >= nrows) continue;
        const float inv = half ? ib : ia;
        const float v0 = acc[nb][2 * half] * inv, v1 = acc[nb][2 * half + 1] * inv;
        const size_t idx = (size_t)(row0 + r) * hd + h * DH + cbase + 8 * nb;
        const __nv_bfloat162 hi = __floats2bfloat162_rn(v0, v1);
        const float2 hf = __bfloat1622float2(hi);
        *reinterpret_cast<__nv_bfloat162 *>(a.out + idx) = hi;
        *reinterpret_cast<__nv_bfloat162 *>(a.out + a.out_plane + idx) = __floats2bfloat162_rn(v0 - hf.x, v1 - hf.y);
      }
    }
    return;
  }

  // several key slices: leave this one in shared memory (over the query planes, which were
  // only needed for the fragments), then merge rows sp, sp + splits, ... from all slices
  constexpr int LO = DH + 4;
  float *sO = reinterpret_cast<float *>(smem_raw);          // [RB][LO]: output, then max and sum
#pragma unroll
  for (int nb = 0; nb < NB; nb++) {
    *reinterpret_cast<float2 *>(sO + ra * LO + cbase + 8 * nb) = make_float2(acc[nb][0], acc[nb][1]);
    *reinterpret_cast<float2 *>(sO + rb * LO + cbase + 8 * nb) = make_float2(acc[nb][2], acc[nb][3]);
  }
  if (tid < RB) {
    sO[tid * LO + DH] = s_m[tid];
    sO[tid * LO + DH + 1] = s_l[tid];
  }
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  cooperative_groups::cluster_group cluster = cooperative_groups::this_cluster();
  for (int r = sp + splits * warp; r < nrows; r += splits * (THREADS / 32)) {
    // every load of the row's slices is issued before any is used: one latency, not one per slice
    float ms[MAX_SPLITS], ls[MAX_SPLITS], os[MAX_SPLITS][PER];
#pragma unroll
    for (int s2 = 0; s2 < MAX_SPLITS; s2++) {
      if (s2 < splits) {
        const float *src = cluster.map_shared_rank(sO, (unsigned)s2) + r * LO;
        ms[s2] = src[DH];
        ls[s2] = src[DH + 1];
        if (PER == 4) {
          const float4 t4 = *reinterpret_cast<const float4 *>(src + lane * 4);
          os[s2][0] = t4.x; os[s2][1] = t4.y; os[s2][2 % PER] = t4.z; os[s2][3 % PER] = t4.w;
        } else {
          const float2 t2 = *reinterpret_cast<const float2 *>(src + lane * 2);
          os[s2][0] = t2.x; os[s2][1] = t2.y;
        }
      }
    }
    float M = -INFINITY;
#pragma unroll
    for (int s2 = 0; s2 < MAX_SPLITS; s2++)
      if (s2 < splits) M = fmaxf(M, ms[s2]);
    float L = 0.f, o[PER];
#pragma unroll
    for (int k = 0; k < PER; k++) o[k] = 0.f;
#pragma unroll
    for (int s2 = 0; s2 < MAX_SPLITS; s2++)
      if (s2 < splits) {
        const float c = (ms[s2] == -INFINITY) ? 0.f : __expf(ms[s2] - M);
        L += ls[s2] * c;
#pragma unroll
        for (int k = 0; k < PER; k++) o[k] += os[s2][k] * c;
      }
    const float inv = 1.f / L;
#pragma unroll
    for (int k = 0; k < PER; k++) {
      const size_t idx = (size_t)(row0 + r) * hd + h * DH + lane * PER + k;
      const float v = o[k] * inv;
      const bf16 hi = __float2bfloat16(v);
      a.out[idx] = hi;
      a.out[a.out_plane + idx] = __float2bfloat16(v - __bfloat162float(hi));
    }
  }
  // nobody leaves while a peer may still be reading its shared memory
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

}  // namespace attn
