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
// All arithmetic is fp32 FMA, organised so that shared-memory traffic does not limit it:
// a warp owns four rows. For the scores a lane owns four keys of the tile (k, k + 8, k + 16,
// k + 24) and a quarter of the head dimension, with that quarter of its four query rows kept
// in registers for the whole kernel, so that a step costs four conflict-free K loads per 64
// FMAs; the quarters are added with two warp shuffles. The softmax statistics of a row
// (online softmax: running max and sum) live entirely inside its warp. For the weighted sum
// a lane owns head-dim columns and reads P four keys at a time. With several key slices each
// CTA parks (max, sum, unnormalised output) and bumps a counter; the CTA that arrives last
// merges the slices in ascending order (deterministic, nobody waits).
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
// K and V tiles (rows padded by 4 floats: conflict-free float4 reads by key) and P.
template <int DH> constexpr int smem_bytes() {
  return (2 * KT * (DH + 4) + RB * (KT + 4)) * (int)sizeof(float);
}

template <int DH>
__global__ void __launch_bounds__(THREADS, 1)
tree_attention_kernel(const EpArgs ea, const Args a) {
  constexpr int PER = DH / 32;            // head-dim columns per lane in the weighted sum
  constexpr int C4 = DH / 4;              // float4 per row
  constexpr int LK = DH + 4;              // pitch of sK and sV rows
  constexpr int LP = KT + 4;              // pitch of sP rows
  constexpr int NLD = KT * C4 / THREADS;  // float4 per thread per tile
  constexpr int DPG = DH / 4;             // head-dim elements per lane group in the scores
  constexpr int NS = DPG / 4;             // float4 steps over them
  extern __shared__ __align__(16) float smem[];
  float *sK = smem;                       // [KT][LK]
  float *sV = sK + KT * LK;               // [KT][LK]
  float *sP = sV + KT * LK;               // [RB][LP]
  __shared__ int s_nvis[RB], s_tbase[RB], s_kmax;
  __shared__ uint32_t s_mask[RB][4];
  __shared__ int s_last;
  // This kernel needs the whole register file of its SM (the query rows live in registers):
  // the GEMM that follows is let in only once the tile loop is over (pdl_launch below), not
  // at the start, or its waiting CTAs would take the registers and push this grid into waves.
  pdl_wait();

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gk = lane >> 3, tc = lane & 7;         // quarter of the head dimension / key column
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
  if (ei >= ea.n_ep) {
    pdl_launch();
    return;
  }
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
  // this lane's quarter of its warp's four query rows, scaled, for the whole kernel
  float4 qreg[4][NS];
#pragma unroll
  for (int i = 0; i < 4; i++) {
    const int r = warp * 4 + i;
#pragma unroll
    for (int s4 = 0; s4 < NS; s4++) {
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (r < nrows) {
        v = *reinterpret_cast<const float4 *>(a.q + (size_t)(row0 + r) * hd + h * DH + DPG * gk + 4 * s4);
        v.x *= a.scale; v.y *= a.scale; v.z *= a.scale; v.w *= a.scale;
      }
      qreg[i][s4] = v;
    }
  }
  __syncthreads();
  const int kmax = s_kmax;
  const int tiles = (kmax + KT - 1) / KT;
  const int t0 = sp * tiles / a.splits, t1 = (sp + 1) * tiles / a.splits;

  float m_run[4], l_run[4], acc[4][PER];
#pragma unroll
  for (int rr = 0; rr < 4; rr++) {
    m_run[rr] = -INFINITY;
    l_run[rr] = 0.f;
#pragma unroll
    for (int k = 0; k < PER; k++) acc[rr][k] = 0.f;
  }

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
      *reinterpret_cast<float4 *>(sK + j * LK + c * 4) = kreg[k];
      *reinterpret_cast<float4 *>(sV + j * LK + c * 4) = vreg[k];
    }
    __syncthreads();
    if (t + 1 < t1) fetch(t + 1);          // in flight while this tile is used

    // ---- scores: rows 4 warp + i against keys tc + 8 j, this lane's quarter of the head dim
    float sc[4][4];
#pragma unroll
    for (int i = 0; i < 4; i++)
#pragma unroll
      for (int j = 0; j < 4; j++) sc[i][j] = 0.f;
    {
      const float *kp = sK + tc * LK + DPG * gk;
#pragma unroll
      for (int s4 = 0; s4 < NS; s4++) {
        float4 kf[4];
#pragma unroll
        for (int j = 0; j < 4; j++) kf[j] = *reinterpret_cast<const float4 *>(kp + 8 * j * LK + 4 * s4);
#pragma unroll
        for (int i = 0; i < 4; i++)
#pragma unroll
          for (int j = 0; j < 4; j++)
            sc[i][j] += (qreg[i][s4].x * kf[j].x + qreg[i][s4].y * kf[j].y) +
                        (qreg[i][s4].z * kf[j].z + qreg[i][s4].w * kf[j].w);
      }
    }
    // add the four quarters: afterwards all four lane groups hold the full scores
#pragma unroll
    for (int i = 0; i < 4; i++)
#pragma unroll
      for (int j = 0; j < 4; j++) {
        sc[i][j] += __shfl_xor_sync(0xffffffffu, sc[i][j], 8);
        sc[i][j] += __shfl_xor_sync(0xffffffffu, sc[i][j], 16);
      }
    float corr[4];
#pragma unroll
    for (int i = 0; i < 4; i++) {
      const int r = warp * 4 + i;
      bool vis[4];
      float mx = -INFINITY;
#pragma unroll
      for (int j = 0; j < 4; j++) {
        const int slot = t * KT + tc + 8 * j;
        vis[j] = slot < s_nvis[r];
        const int b = slot - s_tbase[r];
        if (!vis[j] && b >= 0 && b < 128) vis[j] = (s_mask[r][b >> 5] >> (b & 31)) & 1u;
        if (vis[j]) mx = fmaxf(mx, sc[i][j]);
      }
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
      const float mn = fmaxf(m_run[i], mx);
      corr[i] = (mn == -INFINITY) ? 1.f : __expf(m_run[i] - mn);
      m_run[i] = mn;
      float ps = 0.f;
#pragma unroll
      for (int j = 0; j < 4; j++) {
        const float p = vis[j] ? __expf(sc[i][j] - mn) : 0.f;
        ps += p;
        if (gk == 0) sP[r * LP + tc + 8 * j] = p;
      }
      ps += __shfl_xor_sync(0xffffffffu, ps, 1);
      ps += __shfl_xor_sync(0xffffffffu, ps, 2);
      ps += __shfl_xor_sync(0xffffffffu, ps, 4);
      l_run[i] = l_run[i] * corr[i] + ps;
    }
    __syncwarp();
    // ---- weighted sum: lane = head-dim columns PER * lane .., same four rows, four keys a step
#pragma unroll
    for (int rr = 0; rr < 4; rr++)
#pragma unroll
      for (int k = 0; k < PER; k++) acc[rr][k] *= corr[rr];
#pragma unroll 2
    for (int j4 = 0; j4 < KT; j4 += 4) {
      float4 pf[4];
#pragma unroll
      for (int rr = 0; rr < 4; rr++) pf[rr] = *reinterpret_cast<const float4 *>(sP + (warp * 4 + rr) * LP + j4);
#pragma unroll
      for (int jj = 0; jj < 4; jj++) {
        float vv[PER];
        if (PER == 4) {
          const float4 t4 = *reinterpret_cast<const float4 *>(sV + (j4 + jj) * LK + lane * 4);
          vv[0] = t4.x; vv[1] = t4.y; vv[2 % PER] = t4.z; vv[3 % PER] = t4.w;
        } else {
          const float2 t2 = *reinterpret_cast<const float2 *>(sV + (j4 + jj) * LK + lane * 2);
          vv[0] = t2.x; vv[1] = t2.y;
        }
#pragma unroll
        for (int rr = 0; rr < 4; rr++) {
          const float p = jj == 0 ? pf[rr].x : (jj == 1 ? pf[rr].y : (jj == 2 ? pf[rr].z : pf[rr].w));
#pragma unroll
          for (int k = 0; k < PER; k++) acc[rr][k] += p * vv[k];
        }
      }
    }
    __syncwarp();
  }

  pdl_launch();
  if (a.splits == 1) {
#pragma unroll
    for (int rr = 0; rr < 4; rr++) {
      const int r = warp * 4 + rr;
      if (r >= nrows) continue;
      const float inv = 1.f / l_run[rr];
#pragma unroll
      for (int k = 0; k < PER; k++) {
        const size_t idx = (size_t)(row0 + r) * hd + h * DH + lane * PER + k;
        const float v = acc[rr][k] * inv;
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
  for (int rr = 0; rr < 4; rr++) {
    const int r = warp * 4 + rr;
    float *dst = mine + (size_t)r * (DH + 2);
#pragma unroll
    for (int k = 0; k < PER; k++) __stcg(dst + lane * PER + k, acc[rr][k]);
    if (lane == 0) {
      __stcg(dst + DH, m_run[rr]);
      __stcg(dst + DH + 1, l_run[rr]);
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
  // every load of a row's slices is issued before any is used: one latency, not one per slice
#pragma unroll
  for (int rr = 0; rr < 4; rr++) {
    const int r = warp * 4 + rr;
    if (r >= nrows) continue;
    float ms[MAX_SPLITS], ls[MAX_SPLITS], os[MAX_SPLITS][PER];
#pragma unroll
    for (int s2 = 0; s2 < MAX_SPLITS; s2++) {
      const float *src = all + ((size_t)(s2 < a.splits ? s2 : 0) * RB + r) * (DH + 2);
      ms[s2] = __ldcg(src + DH);
      ls[s2] = __ldcg(src + DH + 1);
#pragma unroll
      for (int k = 0; k < PER; k++) os[s2][k] = __ldcg(src + lane * PER + k);
    }
    float M = -INFINITY;
#pragma unroll
    for (int s2 = 0; s2 < MAX_SPLITS; s2++)
      if (s2 < a.splits) M = fmaxf(M, ms[s2]);
    float L = 0.f, o[PER];
#pragma unroll
    for (int k = 0; k < PER; k++) o[k] = 0.f;
#pragma unroll
    for (int s2 = 0; s2 < MAX_SPLITS; s2++)
      if (s2 < a.splits) {
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
}

}  // namespace attn
