// Row-wise kernels around the GEMMs: input embedding, split-K reduction fused with
// RMSNorm / RoPE + KV append / SwiGLU / argmax / log-softmax top-k. All arithmetic is fp32.
// A value that becomes a GEMM operand is written as two bf16 limbs (hi, lo with hi + lo equal
// to the fp32 value to 16 mantissa bits), lo limb `plane` elements after the hi limb; queries
// and cache entries stay fp32. Split-K partials are summed in ascending split order, so
// results do not depend on scheduling.
#pragma once
#include "common.cuh"

namespace epi {

constexpr int THREADS = 256;

__device__ __forceinline__ void store2(bf16 *hi_plane, size_t plane, size_t idx, float v) {
  const bf16 hi = __float2bfloat16(v);
  hi_plane[idx] = hi;
  hi_plane[plane + idx] = __float2bfloat16(v - __bfloat162float(hi));
}

// Output element (t, n) of a GEMM: its planes added in ascending order.
__device__ __forceinline__ float col_sum(const float *__restrict__ part, const SegPlan &sp, int T, int N,
                                         int t, int n) {
  const int planes = nseg_of(sp, n);
  float v = 0.f;
  for (int s = 0; s < planes; s++) v += part[((size_t)s * T + t) * N + n];
  return v;
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

// x[t] = input row (embeds[src] or E[tok]); xn[t] = limbs(rmsnorm(x[t]) * gain).
__global__ void __launch_bounds__(THREADS)
embed_norm_kernel(RowTable rt, const bf16 *__restrict__ embeds, const bf16 *__restrict__ E,
                  const float *__restrict__ gain, float eps, int d, float *__restrict__ x,
                  bf16 *__restrict__ xn, size_t plane) {
  __shared__ float red[32];
  const int t = blockIdx.x;
  const int tok = rt.tok[t];
  const bf16 *src = tok >= 0 ? E + (size_t)tok * d : embeds + (size_t)rt.src[t] * d;
  float ss = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    float v = __bfloat162float(src[i]);
    x[(size_t)t * d + i] = v;
    ss += v * v;
  }
  ss = block_sum(ss, red);
  const float rs = rsqrtf(ss / d + eps);
  for (int i = threadIdx.x; i < d; i += blockDim.x)
    store2(xn, plane, (size_t)t * d + i, x[(size_t)t * d + i] * rs * gain[i]);
}

// Residual update + next norm:  x[t] (+)= sum_s part[s][t];  then
//   gain != NULL: xn[t] = limbs(rmsnorm(x[t]) * gain), feat[t] = rmsnorm(x[t]) * gain (if feat)
//   gain == NULL: xn[t] = limbs(x[t])
__global__ void __launch_bounds__(THREADS)
residual_norm_kernel(const float *__restrict__ part, SegPlan sp, int T, int d, int accumulate,
                     const float *__restrict__ gain, float eps, float *__restrict__ x,
                     bf16 *__restrict__ xn, size_t plane, float *__restrict__ feat) {
  __shared__ float red[32];
  const int t = blockIdx.x;
  float ss = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    float v = accumulate ? x[(size_t)t * d + i] : 0.f;
    const int splits = nseg_of(sp, i);
    for (int s = 0; s < splits; s++) v += part[((size_t)s * T + t) * d + i];
    x[(size_t)t * d + i] = v;
    ss += v * v;
  }
  if (gain == nullptr) {
    for (int i = threadIdx.x; i < d; i += blockDim.x)
      store2(xn, plane, (size_t)t * d + i, x[(size_t)t * d + i]);
    return;
  }
  ss = block_sum(ss, red);
  const float rs = rsqrtf(ss / d + eps);
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    float v = x[(size_t)t * d + i] * rs * gain[i];
    store2(xn, plane, (size_t)t * d + i, v);
    if (feat) feat[(size_t)t * d + i] = v;
  }
}

// q, k, v = sum_s part[s][t][...]; rotate q and k by the row's position (rotate-half pairs
// (i, i + dh/2), angle from the precomputed table); write q and, into the row's cache slot,
// k and v, all fp32. Cache layout per episode: [2 (K, V)][max_seq][H * dh] fp32.
__global__ void __launch_bounds__(THREADS)
qkv_rope_append_kernel(const float *__restrict__ part, SegPlan sp, int T, int H, int dh,
                       RowTable rt, const float2 *__restrict__ rope_tab, float *__restrict__ q,
                       float *__restrict__ cache, size_t ep_stride, int max_seq) {
  const int t = blockIdx.x;
  const int hd = H * dh, half = dh >> 1, N = 3 * hd;
  const int pos = rt.pos[t], slot = rt.slot[t];
  float *kdst = cache + (size_t)rt.ep[t] * ep_stride + (size_t)slot * hd;
  float *vdst = kdst + (size_t)max_seq * hd;
  for (int i = threadIdx.x; i < H * half; i += blockDim.x) {
    const int h = i / half, j = i - h * half;
    const int c0 = h * dh + j, c1 = c0 + half;
    const float qlo = col_sum(part, sp, T, N, t, c0), qhi = col_sum(part, sp, T, N, t, c1);
    const float klo = col_sum(part, sp, T, N, t, hd + c0), khi = col_sum(part, sp, T, N, t, hd + c1);
    const float vlo = col_sum(part, sp, T, N, t, 2 * hd + c0), vhi = col_sum(part, sp, T, N, t, 2 * hd + c1);
    const float2 cs = rope_tab[(size_t)pos * half + j];
    q[(size_t)t * hd + c0] = qlo * cs.x - qhi * cs.y;
    q[(size_t)t * hd + c1] = qhi * cs.x + qlo * cs.y;
    kdst[c0] = klo * cs.x - khi * cs.y;
    kdst[c1] = khi * cs.x + klo * cs.y;
    vdst[c0] = vlo;
    vdst[c1] = vhi;
  }
}

// hid[t][n] = limbs( silu(g) * u ), g = sum_s part[s][t][n], u = sum_s part[s][t][F + n].
__global__ void __launch_bounds__(THREADS)
swiglu_kernel(const float *__restrict__ part, SegPlan sp, int T, int F, bf16 *__restrict__ hid,
              size_t plane) {
  const int t = blockIdx.y;
  const int n = blockIdx.x * blockDim.x + threadIdx.x;
  if (n >= F) return;
  const float g = col_sum(part, sp, T, 2 * F, t, n), u = col_sum(part, sp, T, 2 * F, t, F + n);
  store2(hid, plane, (size_t)t * F + n, g / (1.f + expf(-g)) * u);
}

// cos/sin table in double precision: tab[pos][j] = (cos, sin)(pos * theta^(-2j/dh)).
__global__ void rope_table_kernel(float2 *tab, int max_pos, int half, double theta) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= max_pos * half) return;
  const int pos = i / half, j = i - pos * half;
  const double ang = (double)pos * pow(theta, -(double)j / (double)half);
  tab[i] = make_float2((float)cos(ang), (float)sin(ang));
}

// dst[i] = row rows[i] of src, both limbs (e.g. the last prefix row of each episode).
__global__ void gather_rows_kernel(const bf16 *__restrict__ src, size_t src_plane,
                                   const int *__restrict__ rows, int d, bf16 *__restrict__ dst,
                                   size_t dst_plane) {
  const int r = rows[blockIdx.x];
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    dst[(size_t)blockIdx.x * d + i] = src[(size_t)r * d + i];
    dst[dst_plane + (size_t)blockIdx.x * d + i] = src[src_plane + (size_t)r * d + i];
  }
}

// Two-limb split of an fp32 matrix (stand-alone GEMM entry point).
__global__ void split_limbs_kernel(const float *__restrict__ x, size_t n, bf16 *__restrict__ out) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) store2(out, n, i, x[i]);
}

struct Top2 {
  float v1, v2;
  int i1;
};
__device__ __forceinline__ void top2_push(Top2 &a, float v, int i) {
  if (v > a.v1 || (v == a.v1 && i < a.i1)) {
    a.v2 = a.v1;
    a.v1 = v;
    a.i1 = i;
  } else if (v > a.v2) {
    a.v2 = v;
  }
}
__device__ __forceinline__ void top2_merge(Top2 &a, const Top2 &b) {
  if (b.v1 > a.v1 || (b.v1 == a.v1 && b.i1 < a.i1)) {
    a.v2 = fmaxf(a.v1, b.v2);
    a.v1 = b.v1;
    a.i1 = b.i1;
  } else {
    a.v2 = fmaxf(a.v2, b.v1);
  }
}

// Greedy token per row: logits = sum_s part[s][t][:]; argmax over [lo, hi) with ties to the
// lowest id; margin = top-1 minus top-2 over the same range. Optionally dumps the logits.
__global__ void __launch_bounds__(THREADS)
argmax_kernel(const float *__restrict__ part, SegPlan sp, int T, int V, int lo, int hi,
              int *__restrict__ greedy, float *__restrict__ margin, float *__restrict__ logits_out) {
  __shared__ Top2 red[THREADS / 32];
  const int t = blockIdx.x;
  Top2 best{-INFINITY, -INFINITY, 0x7fffffff};
  for (int v = threadIdx.x; v < V; v += blockDim.x) {
    const float x = col_sum(part, sp, T, V, t, v);
    if (logits_out) logits_out[(size_t)t * V + v] = x;
    if (v >= lo && v < hi) top2_push(best, x, v);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    Top2 other;
    other.v1 = __shfl_xor_sync(0xffffffffu, best.v1, o);
    other.v2 = __shfl_xor_sync(0xffffffffu, best.v2, o);
    other.i1 = __shfl_xor_sync(0xffffffffu, best.i1, o);
    top2_merge(best, other);
  }
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = best;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < THREADS / 32; w++) top2_merge(best, red[w]);
    greedy[t] = best.i1;
    margin[t] = best.v1 - best.v2;
  }
}

// Draft scoring per row: log-softmax of the logits over [lo, hi) and its top-K entries
// (ties to the lowest id), K = SV_TOPK. Selection by K rounds of block argmax.
__global__ void __launch_bounds__(THREADS)
logsoftmax_topk_kernel(const float *__restrict__ part, SegPlan sp, int T, int V, int lo, int hi,
                       float *__restrict__ scratch_logits, int *__restrict__ top_tok,
                       float *__restrict__ top_lp) {
  __shared__ float redf[32];
  __shared__ float sv[THREADS / 32];
  __shared__ int si[THREADS / 32];
  __shared__ int chosen[SV_TOPK];
  const int t = blockIdx.x;
  float *lg = scratch_logits + (size_t)t * V;
  float mx = -INFINITY;
  for (int v = lo + threadIdx.x; v < hi; v += blockDim.x) {
    const float x = col_sum(part, sp, T, V, t, v);
    lg[v] = x;
    mx = fmaxf(mx, x);
  }
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
      top_tok[t * SV_TOPK + k] = bi;
      top_lp[t * SV_TOPK + k] = bv - lse;
    }
    __syncthreads();
  }
}

}  // namespace epi
