// Skinny weight-streaming GEMM, warp-level MMA version.
//   part[z][t][n] = sum over the z-th K range of (Xhi[t][k] + Xlo[t][k]) * W[n][k]   (fp32 acc)
// W [N, K] is bf16 with K contiguous. The activations come as TWO bf16 limbs (hi = bf16(x),
// lo = bf16(x - hi)), each [T, K]: the weight stream is the cost of this kernel, so spending a
// second MMA per weight tile buys fp32-grade activations for free, which the 32-layer model
// needs to stay within 2e-2 of a float64 forward (single-limb bf16 activations drift by 0.2).
// The 128 weight rows of a CTA tile sit on the MMA's M axis, the (few) activation rows on its
// N axis, so one pass over W serves every row of the tree. K ranges (split-K) are summed by
// the consuming epilogue in fixed order. Requires K % 8 == 0 (16-byte chunks); ragged N, T
// and K tails are zero-filled.
#pragma once
#include "common.cuh"

namespace gemm_mma {

constexpr int BN = 128, BK = 64, STAGES = 4;

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gsrc, int src_bytes) {
  uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(d), "l"(gsrc), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3,
                                            const void *p) {
  uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(a));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 "
               "{%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Tile element (row, 16-byte chunk c of the 128-byte row): chunks are XOR-swizzled by row.
__device__ __forceinline__ bf16 *tile_ptr(bf16 *tile, int row, int chunk) {
  return tile + row * BK + ((chunk ^ (row & 7)) << 3);
}

template <int BT, int WARPS_T>
__global__ void __launch_bounds__(128 * WARPS_T)
gemm_kernel(const bf16 *__restrict__ X, size_t x_plane, const bf16 *__restrict__ W,
            float *__restrict__ part, int T, int N, int K, int kb_per_split) {
  constexpr int NT = 128 * WARPS_T;
  constexpr int WT = BT / WARPS_T;       // activation rows per warp
  constexpr int NTILES = WT / 8;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  bf16 *sW = reinterpret_cast<bf16 *>(smem_raw);
  bf16 *sX = sW + STAGES * BN * BK;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int warp_m = warp & 3, warp_t = warp >> 2;
  const int n0 = blockIdx.x * BN, t0 = blockIdx.y * BT;
  const int nkb = (K + BK - 1) / BK;
  const int kb0 = blockIdx.z * kb_per_split;
  const int kb1 = min(nkb, kb0 + kb_per_split);

  auto load_stage = [&](int stage, int kb) {
    bf16 *w = sW + stage * BN * BK;
    bf16 *x = sX + stage * 2 * BT * BK;
    const int k0 = kb * BK;
    for (int c = tid; c < BN * 8; c += NT) {
      int row = c >> 3, ch = c & 7;
      int n = n0 + row, k = k0 + ch * 8;
      bool ok = (n < N) && (k < K);
      const bf16 *src = W + (size_t)(ok ? n : 0) * K + (ok ? k : 0);
      cp_async16(tile_ptr(w, row, ch), src, ok ? 16 : 0);
    }
    for (int c = tid; c < 2 * BT * 8; c += NT) {
      int row = c >> 3, ch = c & 7;              // rows [0, BT): hi limb, [BT, 2BT): lo limb
      int limb = row >= BT, t = t0 + row - limb * BT, k = k0 + ch * 8;
      bool ok = (t < T) && (k < K);
      const bf16 *src = X + (size_t)limb * x_plane + (size_t)(ok ? t : 0) * K + (ok ? k : 0);
      cp_async16(tile_ptr(x, row, ch), src, ok ? 16 : 0);
    }
  };

  float acc[2][NTILES][4];
#pragma unroll
  for (int i = 0; i < 2; i++)
#pragma unroll
    for (int j = 0; j < NTILES; j++)
#pragma unroll
      for (int v = 0; v < 4; v++) acc[i][j][v] = 0.f;

  const int nk = kb1 - kb0;
  for (int s = 0; s < STAGES - 1; s++) {
    if (s < nk) load_stage(s, kb0 + s);
    cp_async_commit();
  }
  for (int it = 0; it < nk; it++) {
    cp_async_wait<STAGES - 2>();
    __syncthreads();
    int nxt = it + STAGES - 1;
    if (nxt < nk) load_stage(nxt % STAGES, kb0 + nxt);
    cp_async_commit();
    bf16 *w = sW + (it % STAGES) * BN * BK;
    bf16 *x = sX + (it % STAGES) * 2 * BT * BK;
#pragma unroll
    for (int kk = 0; kk < BK / 16; kk++) {
      uint32_t a[2][4];
#pragma unroll
      for (int mt = 0; mt < 2; mt++) {
        int row = warp_m * 32 + mt * 16 + (lane & 15);
        ldmatrix_x4(a[mt][0], a[mt][1], a[mt][2], a[mt][3], tile_ptr(w, row, kk * 2 + (lane >> 4)));
      }
#pragma unroll
      for (int limb = 0; limb < 2; limb++)
#pragma unroll
        for (int p = 0; p < NTILES / 2; p++) {
          uint32_t b0, b1, b2, b3;
          int row = limb * BT + warp_t * WT + p * 16 + ((lane >> 4) << 3) + (lane & 7);
          ldmatrix_x4(b0, b1, b2, b3, tile_ptr(x, row, kk * 2 + ((lane >> 3) & 1)));
#pragma unroll
          for (int mt = 0; mt < 2; mt++) {
            mma_bf16(acc[mt][2 * p], a[mt], b0, b1);
            mma_bf16(acc[mt][2 * p + 1], a[mt], b2, b3);
          }
        }
    }
  }
  cp_async_wait<0>();

  float *out = part + (size_t)blockIdx.z * T * N;
  const int g = lane >> 2, q = lane & 3;
#pragma unroll
  for (int mt = 0; mt < 2; mt++)
#pragma unroll
    for (int nt = 0; nt < NTILES; nt++)
#pragma unroll
      for (int v = 0; v < 4; v++) {
        int n = n0 + warp_m * 32 + mt * 16 + g + ((v >> 1) << 3);
        int t = t0 + warp_t * WT + nt * 8 + q * 2 + (v & 1);
        if (n < N && t < T) out[(size_t)t * N + n] = acc[mt][nt][v];
      }
}

template <int BT, int WARPS_T>
inline cudaError_t launch_cfg(const bf16 *X, size_t x_plane, const bf16 *W, float *part, int T, int N,
                              int K, int splits, cudaStream_t st) {
  static bool attr_set = false;
  const int smem = STAGES * (BN + 2 * BT) * BK * (int)sizeof(bf16);
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(gemm_kernel<BT, WARPS_T>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  const int nkb = (K + BK - 1) / BK;
  const int kbs = (nkb + splits - 1) / splits;
  dim3 grid((N + BN - 1) / BN, (T + BT - 1) / BT, (nkb + kbs - 1) / kbs);
  gemm_kernel<BT, WARPS_T><<<grid, 128 * WARPS_T, smem, st>>>(X, x_plane, W, part, T, N, K, kbs);
  return cudaGetLastError();
}

// Number of K ranges the launch below will use (the epilogue sums exactly this many).
inline int plan_splits(int T, int N, int K, int max_splits) {
  const int BT = T <= 32 ? 32 : (T <= 64 ? 64 : 128);
  const int tiles = ((N + BN - 1) / BN) * ((T + BT - 1) / BT);
  const int nkb = (K + BK - 1) / BK;
  int s = (2 * 148 + tiles - 1) / tiles;
  if (s > max_splits) s = max_splits;
  if (s > nkb) s = nkb;
  if (s < 1) s = 1;
  const int kbs = (nkb + s - 1) / s;
  return (nkb + kbs - 1) / kbs;
}

// X: hi limb [T, K]; the lo limb starts x_plane elements after it.
inline cudaError_t launch(const bf16 *X, size_t x_plane, const bf16 *W, float *part, int T, int N, int K,
                          int splits, cudaStream_t st) {
  if (T <= 32) return launch_cfg<32, 1>(X, x_plane, W, part, T, N, K, splits, st);
  if (T <= 64) return launch_cfg<64, 1>(X, x_plane, W, part, T, N, K, splits, st);
  return launch_cfg<128, 2>(X, x_plane, W, part, T, N, K, splits, st);
}

}  // namespace gemm_mma
