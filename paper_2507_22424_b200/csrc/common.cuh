// Shared device/host declarations of the Spec-VLA verification path (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

typedef __nv_bfloat16 bf16;

#define SV_MAX_TREE 128          // rows of one tree as it is verified, root included
#define SV_MAX_CAND 320          // nodes a dynamic tree may draft before re-ranking, root included
#define SV_MAX_DEPTH 8
#define SV_MAX_BRANCH 8
#define SV_MAX_PENDING (SV_MAX_DEPTH + 1)
#define SV_TOPK 8

// Per-row description of one forward call (structure of arrays, all on the device).
struct RowTable {
  int *tok;       // token id, or -1: the row's input comes from the embeds buffer
  int *src;       // row index into the embeds buffer (prefill) when tok < 0
  int *ep;        // episode id (selects the KV cache)
  int *pos;       // RoPE position
  int *slot;      // cache slot the row's K/V are written to
  int *nvis;      // cache slots [0, nvis) are visible to the row
  int *tbase;     // slot of bit 0 of the mask
  uint32_t *mask; // [rows][4] bit b set: slot tbase + b is visible
};

// Episode list of one call, passed to kernels by value.
#define SV_MAX_EP 64
struct EpArgs {
  int n_ep;
  int eps[SV_MAX_EP];     // episode ids
  int row0[SV_MAX_EP];    // first row of each episode in the call's row table
  int nrows[SV_MAX_EP];   // its number of rows
  int aux[SV_MAX_EP];     // call-specific
};

// Per-episode decoding state on the device.
struct EpState {
  int P;                          // committed target positions
  int Pd;                         // committed draft positions
  int root;                       // last emitted token (not yet in the target cache)
  int n_pending;                  // draft rows waiting: (feature_j, token_j) at position Pd + j
  int pending_tok[SV_MAX_PENDING];
  int pad[3];
};

// Per-episode draft tree on the device.
struct DevTree {
  int n_rows;
  int n_drows;                    // draft rows used so far (row 0 = the root's catch-up row)
  int level_begin, level_end;     // nodes of the level built last
  int sel_count;                  // nodes selected for expansion at the next level
  int sel[16];                    // ... in rank order
  int tok[SV_MAX_CAND], parent[SV_MAX_CAND], depth[SV_MAX_CAND];
  float score[SV_MAX_CAND];
  int drow[SV_MAX_CAND];          // draft row that scored the node's children (-1: none)
  int xrow[SV_MAX_CAND];          // row of the draft forward that ran the node (its output feeds its children)
  uint32_t dmask[SV_MAX_TREE][4]; // ancestors-and-self over draft rows (draft mask), by draft row
};

// Device-resident state of the chunk being generated (specvla_generate_action with the loop on the
// device): tokens emitted so far per call slot, and the statistics of specvla_stats.
#define SV_MAX_CHUNK 64
struct ChunkState {
  int n_tokens, iterations, max_iterations, pad;
  int count[SV_MAX_EP];                 // tokens emitted (not clipped)
  int tokens[SV_MAX_EP][SV_MAX_CHUNK];  // the first n_tokens of them
  int accept_len[16], pos_iterations[16], pos_accept_sum[16];   // first episode of the call
};

#define SV_TILE_ROWS 256         // output columns per GEMM tile

// Programmatic dependent launch: a kernel launched with the stream-serialisation attribute may
// start while its predecessor still runs; nothing the predecessor wrote may be touched before
// pdl_wait() returns. pdl_launch() lets the kernel after this one start likewise.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Four consecutive elements at a time (every row length here is a multiple of 8 elements and
// every buffer starts on a 1024-byte boundary, so these accesses are aligned).
__device__ __forceinline__ float4 load_bf16x4(const bf16 *p) {
  const uint2 raw = *reinterpret_cast<const uint2 *>(p);
  const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162 *>(&raw.x);
  const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162 *>(&raw.y);
  const float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
  return make_float4(fa.x, fa.y, fb.x, fb.y);
}
__device__ __forceinline__ void store_bf16x4(bf16 *p, float4 v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
  uint2 raw;
  raw.x = *reinterpret_cast<uint32_t *>(&a);
  raw.y = *reinterpret_cast<uint32_t *>(&b);
  *reinterpret_cast<uint2 *>(p) = raw;
}
// Two-limb split of four values: hi = bf16(v), lo = bf16(v - hi), lo plane `plane` elements on.
__device__ __forceinline__ void store_limbs4(bf16 *hi_plane, size_t plane, size_t idx, float4 v) {
  const float4 h = make_float4(__bfloat162float(__float2bfloat16(v.x)), __bfloat162float(__float2bfloat16(v.y)),
                               __bfloat162float(__float2bfloat16(v.z)), __bfloat162float(__float2bfloat16(v.w)));
  store_bf16x4(hi_plane + idx, h);
  store_bf16x4(hi_plane + plane + idx, make_float4(v.x - h.x, v.y - h.y, v.z - h.z, v.w - h.w));
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Running (top-1 value, its index, top-2 value) of a set of values; ties go to the lowest index.
namespace sv {
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

__device__ __forceinline__ void top2_warp(Top2 &b) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    Top2 other;
    other.v1 = __shfl_xor_sync(0xffffffffu, b.v1, o);
    other.v2 = __shfl_xor_sync(0xffffffffu, b.v2, o);
    other.i1 = __shfl_xor_sync(0xffffffffu, b.i1, o);
    top2_merge(b, other);
  }
}
}  // namespace sv
