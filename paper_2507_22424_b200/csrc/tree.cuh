// Integer bookkeeping of Spec-VLA decoding on the device: row tables, the static-size draft
// tree (Section 4.1), relaxed acceptance and longest-accepted-path selection (Eq. 4,
// Algorithm 1), KV-cache compaction and the per-episode state that links iterations.
#pragma once
#include "common.cuh"

namespace tree {

// ---------------------------------------------------------------------------------------
// The chunk loop of Algorithm 1 on the device: the first token after prefill, then after every
// iteration the m accepted draft tokens and the target's token are appended per episode; the loop
// (a CUDA-graph while node) goes on while an episode still misses tokens.
__global__ void chunk_begin_kernel(EpArgs a, ChunkState *cs, const int *__restrict__ first_tok, int n_tokens,
                                   int max_iterations) {
  pdl_launch();
  pdl_wait();
  const int i = threadIdx.x;
  if (i < a.n_ep) {
    cs->count[i] = 1;
    cs->tokens[i][0] = first_tok[i];
  }
  if (i < 16) {
    cs->accept_len[i] = 0;
    cs->pos_iterations[i] = 0;
    cs->pos_accept_sum[i] = 0;
  }
  if (i == 0) {
    cs->n_tokens = n_tokens;
    cs->iterations = 0;
    cs->max_iterations = max_iterations;
  }
}
// Arms the loop (in front of the while node): it runs only if tokens are missing.
__global__ void chunk_arm_kernel(const ChunkState *cs, cudaGraphConditionalHandle handle) {
  cudaGraphSetConditional(handle, cs->n_tokens > 1 ? 1u : 0u);
}
__global__ void chunk_append_kernel(EpArgs a, ChunkState *cs, const int *__restrict__ out_m,
                                    const int *__restrict__ out_tok, const int *__restrict__ err,
                                    cudaGraphConditionalHandle handle) {
  __shared__ int s_missing;
  pdl_launch();
  pdl_wait();
  const int i = threadIdx.x, n_tokens = cs->n_tokens;
  if (i == 0) s_missing = 0;
  __syncthreads();
  if (i < a.n_ep) {
    const int m = out_m[i];
    int c = cs->count[i];
    if (i == 0) {
      const int it = cs->iterations, pos = c - 1;
      if (it < 16) cs->accept_len[it] = m;
      if (pos >= 0 && pos < 16) {
        cs->pos_iterations[pos]++;
        cs->pos_accept_sum[pos] += m;
      }
    }
    for (int k = 0; k <= m; k++, c++)
      if (c < n_tokens) cs->tokens[i][c] = out_tok[i * (SV_MAX_DEPTH + 1) + k];
    cs->count[i] = c;
    if (c < n_tokens) atomicAdd(&s_missing, 1);
  }
  __syncthreads();
  if (i == 0) {
    const int it = ++cs->iterations;
    // a device-side wait that gave up (status word set) ends the loop as well
    cudaGraphSetConditional(handle, (s_missing > 0 && it < cs->max_iterations && err[0] == 0) ? 1u : 0u);
  }
}
// A one-row tree (the root alone) per episode: an iteration without drafting is one autoregressive step.
__global__ void root_only_tree_kernel(EpArgs a, DevTree *trees) {
  pdl_launch();
  pdl_wait();
  const int i = threadIdx.x;
  if (i >= a.n_ep) return;
  DevTree &tr = trees[a.eps[i]];
  tr.n_rows = 1;
  tr.tok[0] = -1;
  tr.parent[0] = -1;
  tr.depth[0] = 0;
  tr.score[0] = 0.f;
}


// ---------------------------------------------------------------------------------------
// Verification rows of each episode's tree: row i sits at position P + depth[i], slot P + i,
// sees the P committed slots, its ancestors and itself (the mask is computed here from the
// parents, so trees need only tok / parent / depth). One CTA per episode.
__global__ void build_verify_rows_kernel(EpArgs a, DevTree *trees, const EpState *__restrict__ st,
                                         RowTable rt) {
  pdl_launch();
  pdl_wait();
  const int e = a.eps[blockIdx.x];
  DevTree &tr = trees[e];
  const int P = st[e].P;
  for (int i = threadIdx.x; i < tr.n_rows; i += blockDim.x) {
    uint32_t m[4] = {0, 0, 0, 0};
    for (int j = i; j >= 0; j = tr.parent[j]) m[j >> 5] |= 1u << (j & 31);
    const int r = a.row0[blockIdx.x] + i;
    rt.tok[r] = (i == 0 && tr.tok[0] < 0) ? st[e].root : tr.tok[i];
    rt.src[r] = 0;
    rt.ep[r] = e;
    rt.pos[r] = P + tr.depth[i];
    rt.slot[r] = P + i;
    rt.nvis[r] = P;
    rt.tbase[r] = P;
#pragma unroll
    for (int w = 0; w < 4; w++) rt.mask[r * 4 + w] = m[w];
  }
  if (threadIdx.x == 0 && tr.tok[0] < 0) tr.tok[0] = st[e].root;
}

// RMSNorm scale of a residual row from its partial sums of squares ssq[row][0..nt).
__device__ __forceinline__ float norm_scale(const float *__restrict__ ssq, int nt, size_t row, int d, float eps) {
  float ss = 0.f;
  for (int j = 0; j < nt; j++) ss += ssq[row * nt + j];
  return rsqrtf(ss / d + eps);
}

// Draft-model input rows: xin[r] = limbs([feature ; embedding]) with the feature taken from
// row feat_src[r] of `feat` and the embedding from E[tok] (or embeds[src] when tok < 0).
// With ssq != NULL, `feat` holds residual rows and the feature is their RMSNorm
// (x * rsqrt(mean x^2 + eps) * gain), computed here.
__global__ void draft_input_kernel(RowTable rt, const int *__restrict__ feat_src,
                                   const float *__restrict__ feat, const float *__restrict__ ssq, int nt,
                                   const float *__restrict__ gain, float eps,
                                   const bf16 *__restrict__ embeds,
                                   const bf16 *__restrict__ E, int d, bf16 *__restrict__ xin, size_t plane) {
  pdl_launch();
  pdl_wait();
  const int r = blockIdx.x;
  const float *f = feat + (size_t)feat_src[r] * d;
  const float rs = ssq ? norm_scale(ssq, nt, (size_t)feat_src[r], d, eps) : 1.f;
  const int tok = rt.tok[r];
  const bf16 *e = tok >= 0 ? E + (size_t)tok * d : embeds + (size_t)rt.src[r] * d;
#pragma unroll 2
  for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
    float4 fv = *reinterpret_cast<const float4 *>(f + i);
    if (ssq) {
      const float4 g = *reinterpret_cast<const float4 *>(gain + i);
      fv = make_float4(fv.x * rs * g.x, fv.y * rs * g.y, fv.z * rs * g.z, fv.w * rs * g.w);
    }
    store_limbs4(xin, plane, (size_t)r * 2 * d + i, fv);
    *reinterpret_cast<uint2 *>(xin + (size_t)r * 2 * d + d + i) = *reinterpret_cast<const uint2 *>(e + i);
    *reinterpret_cast<uint2 *>(xin + plane + (size_t)r * 2 * d + d + i) = make_uint2(0u, 0u);
  }
}

// [feature ; embedding] row r of the draft model's input: the feature is an fp32 row (split
// into limbs here), the embedding a bf16 row of E (its lo limb is zero).
__device__ __forceinline__ void write_draft_input_row(const float *__restrict__ f, const bf16 *__restrict__ e, int d,
                                                      bf16 *__restrict__ xin, size_t plane, int r) {
#pragma unroll 2
  for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
    store_limbs4(xin, plane, (size_t)r * 2 * d + i, *reinterpret_cast<const float4 *>(f + i));
    *reinterpret_cast<uint2 *>(xin + (size_t)r * 2 * d + d + i) = *reinterpret_cast<const uint2 *>(e + i);
    *reinterpret_cast<uint2 *>(xin + plane + (size_t)r * 2 * d + d + i) = make_uint2(0u, 0u);
  }
}

// Start of a draft call, one CTA per episode: the n (feature_j, token_j) pairs pending since the
// last commit become draft rows at positions Pd + j, causal among themselves (row table and
// model input written here); Pd advances by n; a new tree is opened whose root is the episode's
// last emitted token. The call always runs a.nrows[i] >= n rows per episode, whatever n is (so that
// its launches do not depend on the accepted length, which only the device knows): the rows past
// n - 1 repeat row n - 1 exactly (same input, position, cache slot and mask: they compute and write
// the same values), and the LAST row, which is pair n - 1 either way, scores the root's children.
__global__ void __launch_bounds__(256)
catchup_input_kernel(EpArgs a, EpState *st, DevTree *trees, RowTable rt, const float *__restrict__ pend_feat,
                     const bf16 *__restrict__ E, int d, bf16 *__restrict__ xin, size_t plane) {
  __shared__ int s_n, s_tok[SV_MAX_PENDING];
  pdl_launch();
  pdl_wait();
  const int i = blockIdx.x, e = a.eps[i], rows = a.nrows[i];
  EpState &s = st[e];
  if (threadIdx.x == 0) s_n = s.n_pending;
  if (threadIdx.x < SV_MAX_PENDING) s_tok[threadIdx.x] = s.pending_tok[threadIdx.x];
  __syncthreads();
  const int n = max(1, min(s_n, rows)), Pd = s.Pd;
  __syncthreads();                                  // everybody has the old Pd
  if (threadIdx.x < rows) {
    const int j = min((int)threadIdx.x, n - 1), r = a.row0[i] + threadIdx.x;
    rt.tok[r] = s_tok[j];
    rt.src[r] = 0;
    rt.ep[r] = e;
    rt.pos[r] = Pd + j;
    rt.slot[r] = Pd + j;
    rt.nvis[r] = Pd + j + 1;
    rt.tbase[r] = 0;
    for (int w = 0; w < 4; w++) rt.mask[r * 4 + w] = 0;
  }
  if (threadIdx.x == 0) {
    s.Pd = Pd + n;
    DevTree &tr = trees[e];
    tr.n_rows = 1;
    tr.n_drows = 1;
    tr.tok[0] = s.root;
    tr.parent[0] = -1;
    tr.depth[0] = 0;
    tr.score[0] = 0.f;
    tr.drow[0] = 0;
    tr.xrow[0] = a.row0[i] + rows - 1;
    for (int w = 0; w < 4; w++) tr.dmask[0][w] = 0;
    tr.level_begin = 0;
    tr.level_end = 1;
    tr.sel_count = 1;
    tr.sel[0] = 0;
  }
  for (int j = 0; j < rows; j++) {
    const int jj = min(j, n - 1);
    write_draft_input_row(pend_feat + (size_t)(e * SV_MAX_PENDING + jj) * d, E + (size_t)s_tok[jj] * d, d, xin, plane,
                          a.row0[i] + j);
  }
}

// One level of tree growth and the next level's model input, one CTA per episode. The rows
// scored last (one per selected parent, in rank order; a.row0 = the first of them, or for the
// root the episode's last catch-up row) come with their top-K tokens and log-probabilities:
// parent sel[j] gets `branch` children (score = parent score + log-prob), numbered in creation
// order. Then the `expand_next` best new nodes (by score, ties to the lower node index: rank by
// counting) are selected, in rank order, as the next level's rows a.aux + j: token = their own,
// feature = output row x[xrow[parent]] of the forward that ran their parent, position
// Pd - 1 + level + 1, cache slot Pd - 1 + draft row, mask = the parent's ancestors and itself.
__global__ void __launch_bounds__(256)
grow_input_kernel(EpArgs a, int level, int branch, int expand_next, const int *__restrict__ top_tok,
                  const float *__restrict__ top_lp, DevTree *trees, const EpState *__restrict__ st, RowTable rt,
                  const float *__restrict__ x, const bf16 *__restrict__ E, int d, bf16 *__restrict__ xin,
                  size_t plane) {
  __shared__ int s_sel_old[16], s_sel[16], s_src[16], s_tokn[16];
  __shared__ float s_score[128];
  __shared__ int s_cnt;
  pdl_launch();
  pdl_wait();
  const int i = blockIdx.x, e = a.eps[i];
  DevTree &tr = trees[e];
  const int begin = tr.n_rows, nsel = tr.sel_count, base_dr = tr.n_drows;
  if (threadIdx.x < 16) s_sel_old[threadIdx.x] = tr.sel[threadIdx.x];
  __syncthreads();                                  // the old state has been read by everybody
  const int m = nsel * branch;                      // new nodes (at most 128)
  const int k = threadIdx.x;
  if (k < m) {
    const int j = k / branch, b = k - j * branch;
    const int p = s_sel_old[j], srow = a.row0[i] + j, n = begin + k;
    const float sc = tr.score[p] + top_lp[srow * SV_TOPK + b];
    tr.tok[n] = top_tok[srow * SV_TOPK + b];
    tr.parent[n] = p;
    tr.depth[n] = level + 1;
    tr.score[n] = sc;
    tr.drow[n] = -1;
    s_score[k] = sc;
  }
  const int cnt = expand_next < m ? expand_next : m;
  if (k == 0) {
    tr.n_rows = begin + m;
    tr.level_begin = begin;
    tr.level_end = begin + m;
    tr.sel_count = cnt;
    tr.n_drows = base_dr + cnt;
    s_cnt = cnt;
  }
  __syncthreads();
  if (k < m) {
    int rank = 0;
    for (int q = 0; q < m; q++) rank += (s_score[q] > s_score[k]) || (s_score[q] == s_score[k] && q < k);
    if (rank < cnt) s_sel[rank] = begin + k;
  }
  __syncthreads();
  if (k < cnt) {
    const int n = s_sel[k], dr = base_dr + k;
    const int p = tr.parent[n], pdr = tr.drow[p];
    const int Pd = st[e].Pd, r = a.aux[i] + k;
    tr.sel[k] = n;
    tr.drow[n] = dr;
    tr.xrow[n] = r;
    uint32_t msk[4];
    for (int w = 0; w < 4; w++) msk[w] = tr.dmask[pdr][w];
    msk[dr >> 5] |= 1u << (dr & 31);
    for (int w = 0; w < 4; w++) {
      tr.dmask[dr][w] = msk[w];
      rt.mask[r * 4 + w] = msk[w];
    }
    rt.tok[r] = tr.tok[n];
    rt.src[r] = 0;
    rt.ep[r] = e;
    rt.pos[r] = Pd - 1 + level + 1;
    rt.slot[r] = Pd - 1 + dr;              // draft row dr >= 1 -> slot Pd + (dr - 1)
    rt.nvis[r] = Pd;
    rt.tbase[r] = Pd - 1;                  // bit dr of the mask <-> slot Pd - 1 + dr
    s_src[k] = tr.xrow[p];
    s_tokn[k] = tr.tok[n];
  }
  __syncthreads();
  for (int j = 0; j < s_cnt; j++)
    write_draft_input_row(x + (size_t)s_src[j] * d, E + (size_t)s_tokn[j] * d, d, xin, plane, a.aux[i] + j);
}

// ---------------------------------------------------------------------------------------
// Dynamic draft tree (Section 4.1: the Eagle-2 strategy; Section 5.1: at most 50 nodes): once
// the last level is drafted, every node is ranked by its cumulative log-probability (ties to
// the lower node index) and only the `keep` best stay, in their creation order. A node never
// outranks its parent (log-probabilities are <= 0 and the parent has the lower index), so the
// set is closed under ancestors. One CTA per episode; ranks by counting (n <= 320).
__global__ void __launch_bounds__(SV_MAX_CAND)
rerank_keep_kernel(EpArgs a, DevTree *trees, int keep) {
  __shared__ float s_score[SV_MAX_CAND];
  __shared__ int s_tok[SV_MAX_CAND], s_parent[SV_MAX_CAND], s_depth[SV_MAX_CAND], s_new[SV_MAX_CAND];
  pdl_launch();
  pdl_wait();
  DevTree &tr = trees[a.eps[blockIdx.x]];
  const int n = tr.n_rows, i = threadIdx.x;
  if (n - 1 <= keep) return;
  if (i < n) {
    s_score[i] = tr.score[i];
    s_tok[i] = tr.tok[i];
    s_parent[i] = tr.parent[i];
    s_depth[i] = tr.depth[i];
  }
  __syncthreads();
  bool kept = false;
  if (i < n) {
    int rank = 0;
    for (int j = 1; j < n; j++) rank += (s_score[j] > s_score[i]) || (s_score[j] == s_score[i] && j < i);
    kept = (i == 0) || rank < keep;
  }
  // new index = kept nodes before this one (block-wide exclusive count through ballots)
  __shared__ int s_warp[SV_MAX_CAND / 32];
  const unsigned b = __ballot_sync(0xffffffffu, kept);
  if ((i & 31) == 0) s_warp[i >> 5] = __popc(b);
  __syncthreads();
  int before = __popc(b & ((1u << (i & 31)) - 1u));
  for (int w = 0; w < (i >> 5); w++) before += s_warp[w];
  s_new[i] = kept ? before : -1;
  __syncthreads();
  if (kept) {
    tr.tok[before] = s_tok[i];
    tr.parent[before] = i == 0 ? -1 : s_new[s_parent[i]];
    tr.depth[before] = s_depth[i];
    tr.score[before] = s_score[i];
  }
  if (i == 0) tr.n_rows = 1 + keep;
}

// ---------------------------------------------------------------------------------------
// Relaxed acceptance (Eq. 4) and longest-accepted-path selection, one warp per episode.
// Node i is accepted iff its parent is accepted and |bin(tok[i]) - bin(g[parent[i]])| <= r
// (ids outside [a0, a0 + nb) must be equal). The deepest accepted node wins, ties to the
// lowest row. Lanes own rows i, i+32, ...; acceptance spreads one tree level per round
// through ballots of the per-lane flags. Emits the m accepted draft tokens plus g[n*],
// commits the state for the next iteration and gathers the features on the path.
__global__ void __launch_bounds__(128)
accept_select_kernel(EpArgs ea, DevTree *trees, EpState *st, const int *__restrict__ greedy, int r, int a0, int nb,
                     const float *__restrict__ x, const float *__restrict__ ssq, int nt,
                     const float *__restrict__ gain, float eps, int d, float *__restrict__ pend_feat,
                     int *__restrict__ out_m, int *__restrict__ out_tok, int *__restrict__ out_path) {
  pdl_launch();
  pdl_wait();
  __shared__ int s_path[SV_MAX_DEPTH + 1], s_m;
  const int e = ea.eps[blockIdx.x];
  const int base = ea.row0[blockIdx.x];
  DevTree &tr = trees[e];
  const int n = tr.n_rows;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (warp == 0) {
    bool ok[4], a[4];
#pragma unroll
    for (int k = 0; k < 4; k++) {
      const int i = lane + 32 * k;
      ok[k] = false;
      a[k] = (i == 0);
      if (i > 0 && i < n) {
        const int dt = tr.tok[i], gt = greedy[base + tr.parent[i]];
        const bool da = dt >= a0 && dt < a0 + nb, ga = gt >= a0 && gt < a0 + nb;
        ok[k] = (da && ga) ? (abs(dt - gt) <= r) : (dt == gt);
      }
    }
    for (int round = 0; round < SV_MAX_DEPTH; round++) {
      uint32_t words[4];
#pragma unroll
      for (int k = 0; k < 4; k++) words[k] = __ballot_sync(0xffffffffu, a[k]);
#pragma unroll
      for (int k = 0; k < 4; k++) {
        const int i = lane + 32 * k;
        if (i > 0 && i < n && ok[k]) {
          const int p = tr.parent[i];
          a[k] = (words[p >> 5] >> (p & 31)) & 1u;
        }
      }
    }
    // deepest accepted node, ties to the lowest row: maximise depth * 128 + (127 - row)
    int key = -1;
#pragma unroll
    for (int k = 0; k < 4; k++) {
      const int i = lane + 32 * k;
      if (i < n && a[k]) key = max(key, tr.depth[i] * SV_MAX_TREE + (SV_MAX_TREE - 1 - i));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) key = max(key, __shfl_xor_sync(0xffffffffu, key, o));
    if (lane == 0) {
      const int best = SV_MAX_TREE - 1 - (key % SV_MAX_TREE);
      const int m = tr.depth[best];
      int j = best;
      for (int k = m; k >= 0; k--) { s_path[k] = j; j = tr.parent[j]; }
      s_m = m;
      EpState &s = st[e];
      int *ot = out_tok + blockIdx.x * (SV_MAX_DEPTH + 1);
      int *op = out_path + blockIdx.x * (SV_MAX_DEPTH + 1);
      for (int k = 0; k <= SV_MAX_DEPTH; k++) { ot[k] = -1; op[k] = -1; }
      for (int k = 1; k <= m; k++) ot[k - 1] = tr.tok[s_path[k]];
      ot[m] = greedy[base + best];
      for (int k = 0; k <= m; k++) { op[k] = s_path[k]; s.pending_tok[k] = ot[k]; }
      out_m[blockIdx.x] = m;
      s.root = ot[m];
      s.n_pending = m + 1;
      // s.P is advanced by the compaction kernel, which still needs the old value
    }
  }
  __syncthreads();
  const int m = s_m;
  // features (final-norm outputs) of the rows on the path, for the draft model's next call
  for (int k = 0; k <= m; k++) {
    const size_t row = (size_t)(base + s_path[k]);
    const float *src = x + row * d;
    const float rs = norm_scale(ssq, nt, row, d, eps);
    float *dst = pend_feat + (size_t)(e * SV_MAX_PENDING + k) * d;
    for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
      const float4 v = *reinterpret_cast<const float4 *>(src + i);
      const float4 g = *reinterpret_cast<const float4 *>(gain + i);
      *reinterpret_cast<float4 *>(dst + i) = make_float4(v.x * rs * g.x, v.y * rs * g.y, v.z * rs * g.z, v.w * rs * g.w);
    }
  }
}

// In-place KV compaction: accepted row path[j] moves from slot P + path[j] to slot P + j
// (j = 1..m) in every layer, K and V. path[j] >= j and path is increasing, so copying in
// ascending j never overwrites a source that is still needed; every 16-byte column chunk is
// handled by one thread, which keeps that order. grid = (layers * 2, episodes).
__global__ void __launch_bounds__(256)
kv_compact_kernel(EpArgs a, const EpState *__restrict__ st,
                  const int *__restrict__ out_m, const int *__restrict__ out_path,
                  float *__restrict__ cache, size_t ep_stride, size_t layer_stride, int max_seq, int hd) {
  pdl_launch();
  pdl_wait();
  const int e = a.eps[blockIdx.y];
  const int m = out_m[blockIdx.y];
  const int P = st[e].P;
  const int *path = out_path + blockIdx.y * (SV_MAX_DEPTH + 1);
  const int layer = blockIdx.x >> 1, which = blockIdx.x & 1;
  uint4 *base = reinterpret_cast<uint4 *>(cache + (size_t)e * ep_stride + (size_t)layer * layer_stride +
                                          (size_t)which * max_seq * hd);
  const int chunks = hd / 4;
  for (int j = 1; j <= m; j++) {
    const int src = P + path[j], dst = P + j;
    if (src == dst) continue;
    for (int c = threadIdx.x; c < chunks; c += blockDim.x)
      base[(size_t)dst * chunks + c] = base[(size_t)src * chunks + c];
  }
}

// P <- P + 1 + m after compaction.
__global__ void advance_state_kernel(EpArgs a, EpState *st, const int *__restrict__ out_m) {
  pdl_launch();
  pdl_wait();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < a.n_ep) st[a.eps[i]].P += 1 + out_m[i];
}

// State after prefill: P = len, Pd = len - 1, root = a_1, one pending pair (f_{P-1}, a_1).
// a.nrows = prefix lengths, a.aux = last row of each episode.
__global__ void prefill_commit_kernel(EpArgs a, EpState *st,
                                      const int *__restrict__ greedy, const float *__restrict__ x,
                                      const float *__restrict__ ssq, int nt,
                                      const float *__restrict__ gain, float eps,
                                      int d, float *__restrict__ pend_feat) {
  pdl_launch();
  pdl_wait();
  const int e = a.eps[blockIdx.x];
  if (threadIdx.x == 0) {
    EpState &s = st[e];
    s.P = a.nrows[blockIdx.x];
    s.Pd = a.nrows[blockIdx.x] - 1;
    s.root = greedy[blockIdx.x];
    s.n_pending = 1;
    s.pending_tok[0] = greedy[blockIdx.x];
  }
  const size_t row = (size_t)a.aux[blockIdx.x];
  const float *src = x + row * d;
  const float rs = norm_scale(ssq, nt, row, d, eps);
  float *dst = pend_feat + (size_t)e * SV_MAX_PENDING * d;
  for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
    const float4 v = *reinterpret_cast<const float4 *>(src + i);
    const float4 g = *reinterpret_cast<const float4 *>(gain + i);
    *reinterpret_cast<float4 *>(dst + i) = make_float4(v.x * rs * g.x, v.y * rs * g.y, v.z * rs * g.z, v.w * rs * g.w);
  }
}

}  // namespace tree
