// Row-wise kernels around the GEMMs: input embedding, the RoPE table, greedy argmax and
// log-softmax top-k over finished logits, feature materialisation. All arithmetic is fp32.
//
// RMSNorm is split around the GEMMs: the producer of a residual row x writes the GEMM operand
// limbs(x * gain) and per-row partial sums of squares ssq[row][0..nt); the GEMM that consumes
// the operand multiplies its output rows by rsqrt(sum(ssq) / d + eps). Kernels here follow the
// same convention. A value that becomes a GEMM operand is written as two bf16 limbs (hi, lo
// with hi + lo equal to the fp32 value to 16 mantissa bits), lo limb `plane` elements after hi.
//
// Every kernel starts with pdl_launch(); pdl_wait(): it may be launched while its predecessor
// still runs and touches nothing before the predecessor has finished.
#pragma once
#include "common.cuh"

namespace epi {

constexpr int THREADS = 256;

__device__ __forceinline__ void store2(bf16 *hi_plane, size_t plane, size_t idx, float v) {
  const bf16 hi = __float2bfloat16(v);
  hi_plane[idx] = hi;
  hi_plane[plane + idx] = __float2bfloat16(v - __bfloat162float(hi));
}

__device__ __forceinline__ float block_sum(float v, float *red) {
  v = warp_sum(v);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float t = (threadIdx.x < (blockDim.x >> 5)) ? red[threadIdx.x] : 0.f;
  if (warp == 0) {
    t = warp_sum(t);
    if (lane == 0) red[0] = t;
  }
  __syncthreads();
  return red[0];
}

// RMSNorm scale of a row from its partial sums of squares.
__device__ __forceinline__ float row_scale(const float *__restrict__ ssq, int nt, size_t row, int d, float eps) {
  float ss = 0.f;
  for (int j = 0; j < nt; j++) ss += ssq[row * nt + j];
  return rsqrtf(ss / d + eps);
}

// x[t] = input row (embeds[src] or E[tok]); xn[t] = limbs(x[t] * gain); ssq[t] = (sum x^2, 0, ...).
__global__ void __launch_bounds__(THREADS)
embed_kernel(RowTable rt, const bf16 *__restrict__ embeds, const bf16 *__restrict__ E,
             const float *__restrict__ gain, int d, int nt, float *__restrict__ x,
             bf16 *__restrict__ xn, size_t plane, float *__restrict__ ssq) {
  __shared__ float red[32];
  pdl_launch();
  pdl_wait();
  const int t = blockIdx.x;
  const int tok = rt.tok[t];
  const bf16 *src = tok >= 0 ? E + (size_t)tok * d : embeds + (size_t)rt.src[t] * d;
  float ss = 0.f;
#pragma unroll 2
  for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
    const float4 v = load_bf16x4(src + i);
    const float4 g = *reinterpret_cast<const float4 *>(gain + i);
    *reinterpret_cast<float4 *>(x + (size_t)t * d + i) = v;
    store_limbs4(xn, plane, (size_t)t * d + i, make_float4(v.x * g.x, v.y * g.y, v.z * g.z, v.w * g.w));
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  ss = block_sum(ss, red);
  for (int j = threadIdx.x; j < nt; j += blockDim.x) ssq[(size_t)t * nt + j] = (j == 0) ? ss : 0.f;
}

// cos/sin table in double precision: tab[pos][j] = (cos, sin)(pos * theta^(-2j/dh)).
__global__ void rope_table_kernel(float2 *tab, int max_pos, int half, double theta) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= max_pos * half) return;
  const int pos = i / half, j = i - pos * half;
  const double ang = (double)pos * pow(theta, -(double)j / (double)half);
  tab[i] = make_float2((float)cos(ang), (float)sin(ang));
}

// dst[i] = row rows[i] of src, both limbs, and its sums of squares (e.g. the last prefix row
// of each episode, for the LM head).
__global__ void gather_rows_kernel(const bf16 *__restrict__ src, size_t src_plane,
                                   const float *__restrict__ src_ssq, int nt,
                                   const int *__restrict__ rows, int d, bf16 *__restrict__ dst,
                                   size_t dst_plane, float *__restrict__ dst_ssq) {
  pdl_launch();
  pdl_wait();
  const int r = rows[blockIdx.x];
#pragma unroll 2
  for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
    *reinterpret_cast<uint2 *>(dst + (size_t)blockIdx.x * d + i) =
        *reinterpret_cast<const uint2 *>(src + (size_t)r * d + i);
    *reinterpret_cast<uint2 *>(dst + dst_plane + (size_t)blockIdx.x * d + i) =
        *reinterpret_cast<const uint2 *>(src + src_plane + (size_t)r * d + i);
  }
  for (int j = threadIdx.x; j < nt; j += blockDim.x)
    dst_ssq[(size_t)blockIdx.x * nt + j] = src_ssq[(size_t)r * nt + j];
}

// feat[t] = x[t] * rsqrt(mean(x[t]^2) + eps) * gain: the final-norm output (the "feature").
__global__ void features_kernel(const float *__restrict__ x, const float *__restrict__ ssq, int nt,
                                const float *__restrict__ gain, float eps, int d, float *__restrict__ feat) {
  pdl_launch();
  pdl_wait();
  const int t = blockIdx.x;
  const float rs = row_scale(ssq, nt, t, d, eps);
#pragma unroll 2
  for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
    const float4 v = *reinterpret_cast<const float4 *>(x + (size_t)t * d + i);
    const float4 g = *reinterpret_cast<const float4 *>(gain + i);
    *reinterpret_cast<float4 *>(feat + (size_t)t * d + i) =
        make_float4(v.x * rs * g.x, v.y * rs * g.y, v.z * rs * g.z, v.w * rs * g.w);
  }
}

// Two-limb split of an fp32 matrix (stand-alone GEMM entry point).
__global__ void split_limbs_kernel(const float *__restrict__ x, size_t n, bf16 *__restrict__ out) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) store2(out, n, i, x[i]);
}

using sv::Top2;
using sv::top2_push;
using sv::top2_merge;
using sv::top2_warp;

// Greedy token per row from the candidates a GEMM epilogue left: cand[row][0..nc) holds the top-2
// of each 128-column group of the row's logits (value, column as int bits, second value). One
// warp per row; ties go to the lowest id; margin = top-1 minus top-2. Column c is token tok_offset + c
// (the GEMM may have covered only a slice of the vocabulary).
__global__ void __launch_bounds__(128)
argmax_merge_kernel(const float4 *__restrict__ cand, int nc, int rows, int tok_offset, int *__restrict__ greedy,
                    float *__restrict__ margin) {
  pdl_launch();
  pdl_wait();
  const int t = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (t >= rows) return;
  Top2 best{-INFINITY, -INFINITY, 0x7fffffff};
  for (int i = lane; i < nc; i += 32) {
    const float4 c = cand[(size_t)t * nc + i];
    const Top2 other{c.x, c.z, __float_as_int(c.y)};
    top2_merge(best, other);
  }
  top2_warp(best);
  if (lane == 0) {
    greedy[t] = best.i1 + tok_offset;
    margin[t] = best.v1 - best.v2;
  }
}

// Draft scoring per row of logits [T][V]: log-softmax over columns [lo, hi) and its top-K
// entries (ties to the lowest id), K = SV_TOPK. Column c stands for token tok_offset + c (the
// logits may cover only a slice of the vocabulary). Selection by K rounds of block argmax.
__global__ void __launch_bounds__(THREADS)
logsoftmax_topk_kernel(const float *__restrict__ logits, int V, int lo, int hi, int tok_offset,
                       int *__restrict__ top_tok, float *__restrict__ top_lp) {
  __shared__ float redf[32];
  __shared__ float sv[THREADS / 32];
  __shared__ int si[THREADS / 32];
  __shared__ int chosen[SV_TOPK];
  pdl_launch();
  pdl_wait();
  const int t = blockIdx.x;
  const float *lg = logits + (size_t)t * V;
  float mx = -INFINITY;
  for (int v = lo + threadIdx.x; v < hi; v += blockDim.x) mx = fmaxf(mx, lg[v]);
  mx = warp_max(mx);
  if ((threadIdx.x & 31) == 0) sv[threadIdx.x >> 5] = mx;
  __syncthreads();
  mx = sv[0];
  for (int w = 1; w < THREADS / 32; w++) mx = fmaxf(mx, sv[w]);
  float se = 0.f;
  for (int v = lo + threadIdx.x; v < hi; v += blockDim.x) se += expf(lg[v] - mx);
  se = block_sum(se, redf);
  const float lse = mx + logf(se);
  for (int k = 0; k < SV_TOPK; k++) {
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    for (int v = lo + threadIdx.x; v < hi; v += blockDim.x) {
      bool taken = false;
      for (int j = 0; j < k; j++) taken |= (chosen[j] == v);
      float x = lg[v];
      if (!taken && (x > bv || (x == bv && v < bi))) { bv = x; bi = v; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    __syncthreads();
    if ((threadIdx.x & 31) == 0) { sv[threadIdx.x >> 5] = bv; si[threadIdx.x >> 5] = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
      for (int w = 1; w < THREADS / 32; w++)
        if (sv[w] > bv || (sv[w] == bv && si[w] < bi)) { bv = sv[w]; bi = si[w]; }
      chosen[k] = bi;
      top_tok[t * SV_TOPK + k] = bi + tok_offset;
      top_lp[t * SV_TOPK + k] = bv - lse;
    }
    __syncthreads();
  }
}

}  // namespace epi
