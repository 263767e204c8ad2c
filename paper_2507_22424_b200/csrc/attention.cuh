// Tree-mask attention (Section 3.2 / 4.1: every draft-tree row is verified in one forward,
// each conditioned on its own path). One CTA per (head, row). Row t attends cache slots
// [0, nvis[t]) plus the slots tbase[t] + b for every bit b of its 128-bit mask. Queries,
// keys, values, scores, softmax and the weighted sum are fp32; the output is written as two
// bf16 limbs for the O-projection GEMM.
//
// Each warp walks its share of the keys with an online softmax (running max / sum), lanes
// split the head dimension; the four warps' partial results are merged in shared memory in
// warp order, so the result is deterministic.
#pragma once
#include "common.cuh"

namespace attn {

constexpr int WARPS = 4;

template <int DH>
__global__ void __launch_bounds__(WARPS * 32)
tree_attention_kernel(const float *__restrict__ q, const float *__restrict__ cache, size_t ep_stride,
                      int max_seq, int H, RowTable rt, float scale, bf16 *__restrict__ out,
                      size_t out_plane) {
  constexpr int PER = DH / 32;           // head-dim elements per lane
  const int h = blockIdx.x, t = blockIdx.y;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int hd = H * DH;
  const float *kbase = cache + (size_t)rt.ep[t] * ep_stride + (size_t)h * DH + lane * PER;
  const float *vbase = kbase + (size_t)max_seq * hd;
  const int nvis = rt.nvis[t], tbase = rt.tbase[t];

  float qv[PER];
#pragma unroll
  for (int i = 0; i < PER; i++)
    qv[i] = q[(size_t)t * hd + h * DH + lane * PER + i] * scale;

  float m = -INFINITY, l = 0.f, acc[PER];
#pragma unroll
  for (int i = 0; i < PER; i++) acc[i] = 0.f;

  auto visit = [&](int slot) {
    const float *kp = kbase + (size_t)slot * hd;
    const float *vp = vbase + (size_t)slot * hd;
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < PER; i++) s += qv[i] * kp[i];
    s = warp_sum(s);
    const float mn = fmaxf(m, s);
    const float corr = __expf(m - mn), p = __expf(s - mn);
    l = l * corr + p;
#pragma unroll
    for (int i = 0; i < PER; i++) acc[i] = acc[i] * corr + p * vp[i];
    m = mn;
  };

  for (int s = warp; s < nvis; s += WARPS) visit(s);
  // masked tree slots: warp w takes the w-th 32-bit word
  uint32_t word = rt.mask[t * 4 + warp];
  while (word) {
    int b = __ffs(word) - 1;
    word &= word - 1;
    visit(tbase + warp * 32 + b);
  }

  __shared__ float sm[WARPS], sl[WARPS], sacc[WARPS][DH];
  if (lane == 0) { sm[warp] = m; sl[warp] = l; }
#pragma unroll
  for (int i = 0; i < PER; i++) sacc[warp][lane * PER + i] = acc[i];
  __syncthreads();
  if (warp == 0) {
    float M = sm[0];
    for (int w = 1; w < WARPS; w++) M = fmaxf(M, sm[w]);
    float L = 0.f, o[PER];
#pragma unroll
    for (int i = 0; i < PER; i++) o[i] = 0.f;
    for (int w = 0; w < WARPS; w++) {
      const float c = (sm[w] == -INFINITY) ? 0.f : __expf(sm[w] - M);
      L += sl[w] * c;
#pragma unroll
      for (int i = 0; i < PER; i++) o[i] += sacc[w][lane * PER + i] * c;
    }
    const float inv = 1.f / L;
#pragma unroll
    for (int i = 0; i < PER; i++) {
      const size_t idx = (size_t)t * hd + h * DH + lane * PER + i;
      const float v = o[i] * inv;
      const bf16 hi = __float2bfloat16(v);
      out[idx] = hi;
      out[out_plane + idx] = __float2bfloat16(v - __bfloat162float(hi));
    }
  }
}

}  // namespace attn
