// Tree-mask attention (Section 3.2 / 4.1: every draft-tree row is verified in one forward,
// each conditioned on its own path). Row t attends cache slots [0, nvis[t]) plus the slots
// tbase[t] + b for every bit b of its 128-bit mask. Queries, keys, values, scores, softmax
// and the weighted sum are fp32; the output is written as two bf16 limbs for the
// O-projection GEMM.
//
// One CTA handles one head, a block of up to 32 consecutive rows of ONE episode and one slice
// of that block's key range (split-KV). Keys and values go through shared memory in tiles of
// 32 slots, so a K/V row is read from L2/HBM once per row block instead of once per row; the
// next tile is fetched into registers while the current one is used.
//
// Both products run on the tensor cores as warp-level m16n8k8 TF32 MMAs with fp32-grade
// operands: every operand value x is split into hi = tf32(x) and lo = tf32(x - hi) and each
// product is the sum of lo*hi, hi*lo and hi*hi (21 mantissa bits per operand, fp32
// accumulation). For the scores the eight warps tile the 32 rows x 32 keys of a tile as
// 2 x 4 fragments of 16 x 8; the softmax statistics of a row (online softmax: running max and
// sum) are combined across the four warps that hold its keys through shared memory. For the
// weighted sum each warp owns 16 rows x (head_dim / 4) columns of the output, kept in
// registers across tiles. With several key slices each CTA parks (max, sum, unnormalised
// output) and bumps a counter; the CTA that arrives last merges the slices in ascending
// order (deterministic, nobody waits).
#pragma once
#include "common.cuh"

namespace attn {

constexpr int RB = 32;            // rows per block
constexpr int KT = 32;            // key slots per tile
constexpr int THREADS = 256;      // 8 warps x 4 rows
constexpr int MAX_SPLITS = 8;
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
  int splits;              // key slices per row block
  float *part;             // [block * H + head][split][RB][DH + 2] parked slices (splits > 1)
  int *counters;           // [block * H + head], zero between launches
};

__host__ __device__ inline int blocks_of(const EpArgs &ea) {
  int n = 0;
  for (int i = 0; i < ea.n_ep; i++) n += (ea.nrows[i] + RB - 1) / RB;
  return n;
}
// Row pitches (floats) chosen so that the MMA fragment loads hit 32 distinct banks.
template <int DH> constexpr int smem_bytes() {
  return (RB * (DH + 4) + KT * (DH + 4) + KT * (DH + 8) + RB * (KT + 4) + 8 * RB) * (int)sizeof(float);
}

__device__ __forceinline__ void tf32_split(float x, uint32_t &hi, uint32_t &lo) {
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(hi) : "f"(x));
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(lo) : "f"(x - __uint_as_float(hi)));
}
// c += a (16 x 8, row-major) * b (8 x 8, column-major), TF32 operands, fp32 accumulate.
__device__ __forceinline__ void mma_tf32(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile(
      "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}
// c += a * b with both operands carried as (hi, lo) pairs: small terms first.
__device__ __forceinline__ void mma_3x(float (&c)[4], const uint32_t (&ah)[4], const uint32_t (&al)[4],
                                       const uint32_t (&bh)[2], const uint32_t (&bl)[2]) {
  mma_tf32(c, al, bh);
  mma_tf32(c, ah, bl);
  mma_tf32(c, ah, bh);
}

template <int DH>
__global__ void __launch_bounds__(THREADS)
tree_attention_kernel(const EpArgs ea, const Args a) {
  constexpr int PER = DH / 32;            // head-dim columns per lane in the slice merge
  constexpr int C4 = DH / 4;              // float4 per row
  constexpr int LQ = DH + 4;              // pitch of sQ and sK rows
  constexpr int LV = DH + 8;              // pitch of sV rows
  constexpr int LP = KT + 4;              // pitch of sP rows
  constexpr int NLD = KT * C4 / THREADS;  // float4 per thread per tile
  constexpr int NTW = DH / 32;            // 8-column output fragments per warp
  extern __shared__ __align__(16) float smem[];
  float *sQ = smem;                       // [RB][LQ]
  float *sK = sQ + RB * LQ;               // [KT][LQ]
  float *sV = sK + KT * LQ;               // [KT][LV]
  float *sP = sV + KT * LV;               // [RB][LP]
  float *s_pm = sP + RB * LP;             // [4][RB] per-warp-column partial row maxima
  float *s_ps = s_pm + 4 * RB;            // [4][RB] ... and partial row sums
  __shared__ int s_nvis[RB], s_tbase[RB], s_kmax;
  __shared__ uint32_t s_mask[RB][4];
  __shared__ int s_last;
  pdl_launch();
  pdl_wait();

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, tg = lane & 3;          // MMA fragment coordinates
  const int mt = warp & 1, nt = warp >> 1;         // 16-row block / 8-key block (or column group)
  const int r0 = 16 * mt + g, r1 = r0 + 8;         // the two rows this thread holds values of
  const int h = blockIdx.y, hd = a.H * DH;
  int bid = blockIdx.x / a.splits;
  const int sp = blockIdx.x - bid * a.splits;
  const int gblock = bid;
  int ei = 0;
  for (; ei < ea.n_ep; ei++) {
    const int nb = (ea.nrows[ei] + RB - 1) / RB;
    if (bid < nb) break;
    bid -= nb;
  }
  if (ei >= ea.n_ep) return;
  const int row0 = ea.row0[ei] + bid * RB;
  const int nrows = min(RB, ea.nrows[ei] - bid * RB);
  const float *kbase = a.cache + (size_t)ea.eps[ei] * a.ep_stride + (size_t)h * DH;
  const float *vbase = kbase + (size_t)a.max_seq * hd;

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
  for (int i = tid; i < RB * C4; i += THREADS) {
    const int r = i / C4, c = i - r * C4;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (r < nrows) {
      v = *reinterpret_cast<const float4 *>(a.q + (size_t)(row0 + r) * hd + h * DH + c * 4);
      v.x *= a.scale; v.y *= a.scale; v.z *= a.scale; v.w *= a.scale;
    }
    *reinterpret_cast<float4 *>(sQ + r * LQ + c * 4) = v;
  }
  __syncthreads();
  const int kmax = s_kmax;
  const int tiles = (kmax + KT - 1) / KT;
  const int t0 = sp * tiles / a.splits, t1 = (sp + 1) * tiles / a.splits;

  // running softmax statistics of rows r0, r1 (identical in every thread that holds the row)
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  float o[NTW][4];                          // output fragments: rows r0 / r1, columns 32 nt + 8 j + 2 tg (+1)
#pragma unroll
  for (int j = 0; j < NTW; j++)
#pragma unroll
    for (int k = 0; k < 4; k++) o[j][k] = 0.f;
  auto visible = [&](int r, int slot) {
    bool vis = slot < s_nvis[r];
    const int b = slot - s_tbase[r];
    if (!vis && b >= 0 && b < 128) vis = (s_mask[r][b >> 5] >> (b & 31)) & 1u;
    return vis;
  };

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
  if (t0 < t1) fetch(t0);
  for (int t = t0; t < t1; t++) {
    __syncthreads();                       // the previous tile is no longer being read
#pragma unroll
    for (int k = 0; k < NLD; k++) {
      const int i = tid + k * THREADS;
      const int j = i / C4, c = i % C4;
      *reinterpret_cast<float4 *>(sK + j * LQ + c * 4) = kreg[k];
      *reinterpret_cast<float4 *>(sV + j * LV + c * 4) = vreg[k];
    }
    __syncthreads();
    if (t + 1 < t1) fetch(t + 1);          // in flight while this tile is used

    // ---- scores of rows 16 mt .. +15 against keys 8 nt .. +7 of the tile
    float sc[4] = {0.f, 0.f, 0.f, 0.f};
    {
      const float *qa = sQ + r0 * LQ + tg, *qb = sQ + r1 * LQ + tg;
      const float *kp = sK + (8 * nt + g) * LQ + tg;
#pragma unroll 4
      for (int k0 = 0; k0 < DH; k0 += 8) {
        uint32_t ah[4], al[4], bh[2], bl[2];
        tf32_split(qa[k0], ah[0], al[0]);
        tf32_split(qb[k0], ah[1], al[1]);
        tf32_split(qa[k0 + 4], ah[2], al[2]);
        tf32_split(qb[k0 + 4], ah[3], al[3]);
        tf32_split(kp[k0], bh[0], bl[0]);
        tf32_split(kp[k0 + 4], bh[1], bl[1]);
        mma_3x(sc, ah, al, bh, bl);
      }
    }
    // sc[0], sc[1]: row r0, keys 8 nt + 2 tg (+1); sc[2], sc[3]: row r1, same keys
    const int slot = t * KT + 8 * nt + 2 * tg;
    const bool v00 = visible(r0, slot), v01 = visible(r0, slot + 1);
    const bool v10 = visible(r1, slot), v11 = visible(r1, slot + 1);
    float pm0 = fmaxf(v00 ? sc[0] : -INFINITY, v01 ? sc[1] : -INFINITY);
    float pm1 = fmaxf(v10 ? sc[2] : -INFINITY, v11 ? sc[3] : -INFINITY);
    pm0 = fmaxf(pm0, __shfl_xor_sync(0xffffffffu, pm0, 1));
    pm0 = fmaxf(pm0, __shfl_xor_sync(0xffffffffu, pm0, 2));
    pm1 = fmaxf(pm1, __shfl_xor_sync(0xffffffffu, pm1, 1));
    pm1 = fmaxf(pm1, __shfl_xor_sync(0xffffffffu, pm1, 2));
    if (tg == 0) {
      s_pm[nt * RB + r0] = pm0;
      s_pm[nt * RB + r1] = pm1;
    }
    __syncthreads();
    float corr[2];
    {
      const float tm0 = fmaxf(fmaxf(s_pm[r0], s_pm[RB + r0]), fmaxf(s_pm[2 * RB + r0], s_pm[3 * RB + r0]));
      const float tm1 = fmaxf(fmaxf(s_pm[r1], s_pm[RB + r1]), fmaxf(s_pm[2 * RB + r1], s_pm[3 * RB + r1]));
      const float mn0 = fmaxf(m_run[0], tm0), mn1 = fmaxf(m_run[1], tm1);
      corr[0] = (mn0 == -INFINITY) ? 1.f : __expf(m_run[0] - mn0);
      corr[1] = (mn1 == -INFINITY) ? 1.f : __expf(m_run[1] - mn1);
      m_run[0] = mn0;
      m_run[1] = mn1;
      const float p00 = v00 ? __expf(sc[0] - mn0) : 0.f, p01 = v01 ? __expf(sc[1] - mn0) : 0.f;
      const float p10 = v10 ? __expf(sc[2] - mn1) : 0.f, p11 = v11 ? __expf(sc[3] - mn1) : 0.f;
      *reinterpret_cast<float2 *>(sP + r0 * LP + 8 * nt + 2 * tg) = make_float2(p00, p01);
      *reinterpret_cast<float2 *>(sP + r1 * LP + 8 * nt + 2 * tg) = make_float2(p10, p11);
      float ps0 = p00 + p01, ps1 = p10 + p11;
      ps0 += __shfl_xor_sync(0xffffffffu, ps0, 1);
      ps0 += __shfl_xor_sync(0xffffffffu, ps0, 2);
      ps1 += __shfl_xor_sync(0xffffffffu, ps1, 1);
      ps1 += __shfl_xor_sync(0xffffffffu, ps1, 2);
      if (tg == 0) {
        s_ps[nt * RB + r0] = ps0;
        s_ps[nt * RB + r1] = ps1;
      }
    }
    __syncthreads();
    l_run[0] = l_run[0] * corr[0] + ((s_ps[r0] + s_ps[RB + r0]) + (s_ps[2 * RB + r0] + s_ps[3 * RB + r0]));
    l_run[1] = l_run[1] * corr[1] + ((s_ps[r1] + s_ps[RB + r1]) + (s_ps[2 * RB + r1] + s_ps[3 * RB + r1]));

    // ---- weighted sum: rows 16 mt .. +15, output columns (DH / 4) nt .. of the head
#pragma unroll
    for (int j = 0; j < NTW; j++) {
      o[j][0] *= corr[0];
      o[j][1] *= corr[0];
      o[j][2] *= corr[1];
      o[j][3] *= corr[1];
    }
    {
      const float *pa = sP + r0 * LP + tg, *pb = sP + r1 * LP + tg;
#pragma unroll
      for (int k0 = 0; k0 < KT; k0 += 8) {
        uint32_t ah[4], al[4];
        tf32_split(pa[k0], ah[0], al[0]);
        tf32_split(pb[k0], ah[1], al[1]);
        tf32_split(pa[k0 + 4], ah[2], al[2]);
        tf32_split(pb[k0 + 4], ah[3], al[3]);
        const float *vp = sV + (k0 + tg) * LV + NTW * 8 * nt + g;
#pragma unroll
        for (int j = 0; j < NTW; j++) {
          uint32_t bh[2], bl[2];
          tf32_split(vp[8 * j], bh[0], bl[0]);
          tf32_split(vp[4 * LV + 8 * j], bh[1], bl[1]);
          mma_3x(o[j], ah, al, bh, bl);
        }
      }
    }
  }

  // o[j][0..1]: row r0, columns cbase + 8 j + 2 tg (+1); o[j][2..3]: row r1
  const int cbase = NTW * 8 * nt + 2 * tg;
  if (a.splits == 1) {
#pragma unroll
    for (int hh = 0; hh < 2; hh++) {
      const int r = hh ? r1 : r0;
      if (r >= nrows) continue;
      const float inv = 1.f / l_run[hh];
#pragma unroll
      for (int j = 0; j < NTW; j++)
#pragma unroll
        for (int e = 0; e < 2; e++) {
          const size_t idx = (size_t)(row0 + r) * hd + h * DH + cbase + 8 * j + e;
          const float v = o[j][2 * hh + e] * inv;
          const bf16 hi = __float2bfloat16(v);
          a.out[idx] = hi;
          a.out[a.out_plane + idx] = __float2bfloat16(v - __bfloat162float(hi));
        }
    }
    return;
  }

  // several key slices: park this one, the last arrival merges
  const int unit = gblock * a.H + h;
  float *mine = a.part + ((size_t)unit * a.splits + sp) * RB * (DH + 2);
#pragma unroll
  for (int hh = 0; hh < 2; hh++) {
    const int r = hh ? r1 : r0;
    float *dst = mine + (size_t)r * (DH + 2);
#pragma unroll
    for (int j = 0; j < NTW; j++) {
      __stcg(dst + cbase + 8 * j, o[j][2 * hh]);
      __stcg(dst + cbase + 8 * j + 1, o[j][2 * hh + 1]);
    }
    if (nt == 0 && tg == 0) {
      __stcg(dst + DH, m_run[hh]);
      __stcg(dst + DH + 1, l_run[hh]);
    }
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int old = atomicAdd(a.counters + unit, 1);
    s_last = (old == a.splits - 1);
    if (s_last) atomicExch(a.counters + unit, 0);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const float *all = a.part + (size_t)unit * a.splits * RB * (DH + 2);
#pragma unroll
  for (int rr = 0; rr < 4; rr++) {
    const int r = warp * 4 + rr;
    if (r >= nrows) continue;
    float M = -INFINITY;
    for (int s2 = 0; s2 < a.splits; s2++)
      M = fmaxf(M, __ldcg(all + ((size_t)s2 * RB + r) * (DH + 2) + DH));
    float L = 0.f, o[PER];
#pragma unroll
    for (int k = 0; k < PER; k++) o[k] = 0.f;
    for (int s2 = 0; s2 < a.splits; s2++) {
      const float *src = all + ((size_t)s2 * RB + r) * (DH + 2);
      const float ms = __ldcg(src + DH);
      const float c = (ms == -INFINITY) ? 0.f : __expf(ms - M);
      L += __ldcg(src + DH + 1) * c;
#pragma unroll
      for (int k = 0; k < PER; k++) o[k] += __ldcg(src + lane * PER + k) * c;
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
}

}  // namespace attn
