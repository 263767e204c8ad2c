// Host side of the Spec-VLA verification library: context, workspace layout, and the
// kernel sequences behind each C-ABI entry point (see include/specvla.h).
#include "../../include/specvla.h"

#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <mutex>
#include <new>
#include <vector>

#include "attention.cuh"
#include "common.cuh"
#include "epilogue.cuh"
#include "forward_pk.cuh"
#include "gemm_ck.cuh"
#include "gemm_tc.cuh"
#include "tree.cuh"

namespace {

// A weight matrix [N, K] and its TMA map (boxes of the tensor-core GEMM).
struct WMat {
  const bf16 *p;
  int N, K;
  bool has_map;
  CUtensorMap map;
  const bf16 *packed;     // the library's repacked copy (gemm_tc::pack_weights_kernel), in the workspace
  const signed char *q8;  // quantised target: int8 codes in the same unit order (then packed is NULL)
  const float *scale;     // ... and the scale of every weight row
};
// A two-limb activation buffer [2][rows][K] and its TMA maps, one per box height 8, 16, ..., 128 rows.
struct XBuf {
  bf16 *p;
  size_t plane;
  int rows, K;
  bool has_map;
  CUtensorMap map[16];
};
inline int tn_index(int TN) { return TN / 8 - 1; }

struct LayerW {
  WMat wqkv, wo, wgu, wd;
  const float *norm1, *norm2;
};


constexpr size_t ALIGN = 1024;
constexpr size_t L2_PREFETCH_BYTES = 48u << 20;   // of the next GEMM's weights, out of 126 MB of L2

struct Carver {
  char *base;
  size_t off;
  template <typename T> T *take(size_t n) {
    off = (off + ALIGN - 1) / ALIGN * ALIGN;
    T *p = base ? reinterpret_cast<T *>(base + off) : nullptr;
    off += n * sizeof(T);
    return p;
  }
};

}  // namespace

struct specvla_ctx {
  specvla_model_desc desc;
  int hd;                       // n_heads * head_dim
  int max_lm_rows;              // rows the LM head may see in one call
  int max_draft_rows;           // rows of one draft-tree level summed over episodes
  std::vector<LayerW> layers;
  LayerW dlayer;
  const bf16 *embed;
  WMat lm_head, draft_fc;
  WMat lm_head_act;             // rows [action_base, action_base + n_bins) of the LM head (draft scoring)
  const float *final_norm;
  bool has_draft;
  int nt;                       // 256-column tiles of a d_model-wide row (sums-of-squares slots)
  bool use_pdl;                 // programmatic dependent launch between the kernels of a forward
  gemm_ck::ClusterFit fit;      // clusters of each size that can be resident at once
  bool use_l2_prefetch;         // GEMMs prefetch the head of the next GEMM's weights into L2

  // workspace carve-up (device)
  float *kv_t, *kv_d;           // target [ep][layer][2][max_seq][hd], draft [ep][2][max_seq][hd], fp32
  size_t kv_t_ep_stride, kv_t_layer_stride, kv_d_ep_stride;
  float2 *rope_tab;
  float *x, *feat, *lgs, *pend_feat, *margin, *top_lp, *q;
  float *ssq, *lm_ssq;          // per-row partial sums of squares of x / of the gathered LM-head rows
  float4 *cand;                 // [rows][2 * vocab tiles] top-2 per 128 logit columns (greedy argmax, Eq. 1)
  int cand_nc;
  bf16 *packed;                 // repacked weight matrices, one after the other
  size_t packed_elems;
  signed char *packed_q8;       // quantised target: int8 codes of its matrices, one after the other
  size_t packed_q8_bytes;
  float *wscale;                // ... and their row scales
  size_t wscale_elems;
  int lgs_rows;                 // rows of the logits buffer

  // GEMM operands, two bf16 limbs each: hi plane, then the lo plane `plane` elements later
  XBuf xn, xin, ao, hid, lm_in;
  int *err;                     // device status word written by bounded waits that gave up
  RowTable rt;
  int *feat_src, *lm_rows, *greedy, *top_tok, *out_m, *out_tok, *out_path;
  EpState *st;
  DevTree *trees;

  // persistent forward kernel (forward_pk.cuh): calls of one episode and at most 32 rows
  bool pk_ok;                   // shapes allow it and all CTAs of its grid are resident together
  bool use_pk;
  int pk_G;                     // its grid: one CTA per SM
  int pk_max_seg, pk_splits, pk_nt;
  pk::Op *pk_ops_t;             // phase list of the target forward (device)
  int pk_n_ops_t;
  float *pk_part, *pk_apart, *pk_ssq;
  bf16 *pk_xn, *pk_ao, *pk_hid;
  unsigned *pk_bar;
  unsigned long long wait_ns;   // limit of every device-side wait
  const float *last_ssq;        // sums of squares (and their slots per row) left by the last target forward
  int last_nt;

  // host side
  void *pinned;                 // pinned staging: [small results | tree staging | row tables]
  size_t pinned_bytes;
  int *pin_small;               // 4096 ints of results read back
  DevTree *pin_trees;           // max_episodes trees
  int *pin_rows;                // 11 * max_rows + SV_MAX_EP ints: row tables of the target and of the draft model
  std::vector<int> hP, hPending;  // host mirror of P and n_pending; -1 = not prefilled
  std::vector<int> hTreeRows;     // rows of the device-resident tree left by the last draft call
  int last_rows;                // rows of the last target forward
  bool feat_valid;              // ctx->feat holds the features of those rows
  long long launches;
  char cuda_err[256];
  cudaEvent_t ev[4];

  // chunk loop on the device (specvla_generate_action): draft + verify + append as the body of a
  // CUDA-graph while node, captured once per (episodes, tree shape, r) and kept
  bool use_device_loop;
  bool loop_unavailable;          // capturing or instantiating the loop graph failed once: the host runs the loop
  ChunkState *chunk;              // device
  ChunkState *pin_chunk;          // pinned copy read back after the loop, then max_episodes EpState
  cudaStream_t cap_stream;        // capture happens on a stream of the context's own
  cudaGraph_t loop_graph;
  cudaGraphExec_t loop_exec;
  std::vector<int> loop_key;      // what the kept graph was captured for
  long long loop_launches_once, loop_launches_iter;   // kernels per graph launch: outside / inside the loop

  // optional per-GEMM timing (specvla_profile): events around every GEMM launch, summed per
  // weight-matrix class when the stream is next synchronised
  int prof_mask;                        // phases timed: 1 prefill, 2 draft, 4 verify
  int phase;                            // phase of the call in flight
  std::vector<cudaEvent_t> prof_ev;     // pairs (start, stop)
  std::vector<int> prof_cls;            // class of each recorded pair
  int prof_used;
  double prof_ms[SPECVLA_PROF_CLASSES];
  long long prof_n[SPECVLA_PROF_CLASSES];
  double prof_bytes[SPECVLA_PROF_CLASSES];
};

namespace {

#define CU(call)                                                                        \
  do {                                                                                  \
    cudaError_t _e = (call);                                                            \
    if (_e != cudaSuccess) {                                                            \
      snprintf(ctx->cuda_err, sizeof(ctx->cuda_err), "%s at %s:%d", cudaGetErrorString(_e), \
               __FILE__, __LINE__);                                                     \
      return SPECVLA_ERR_CUDA;                                                          \
    }                                                                                   \
  } while (0)
#define TRY(expr)             \
  do {                        \
    int _r = (expr);          \
    if (_r != SPECVLA_OK) return _r; \
  } while (0)

bool desc_ok(const specvla_model_desc *d) {
  if (!d) return false;
  if (d->n_layers < 1 || d->d_model < 64 || d->n_heads < 1 || d->d_ffn < 8 || d->vocab < 16) return false;
  if (d->head_dim != 64 && d->head_dim != 128) return false;
  if (d->d_model % 8 || d->d_ffn % 8 || (d->n_heads * d->head_dim) % 8 || d->vocab % 4 || d->n_bins % 4) return false;
  if (d->n_bins < 1 || d->action_base < 0 || d->action_base + d->n_bins > d->vocab) return false;
  if (d->weight_bits != 0 && d->weight_bits != 8 && d->weight_bits != 16) return false;
  if (d->max_seq < 2 || d->max_episodes < 1 || d->max_episodes > SV_MAX_EP || d->max_rows < 1) return false;
  if (!(d->rms_eps > 0.f) || !(d->rope_theta > 1.f)) return false;
  return true;
}

// The persistent forward kernel needs rows of 128-column groups (sums of squares, RoPE partner
// lanes) and one of its two head sizes.
bool pk_shapes_ok(const specvla_model_desc &d) {
  const int hd = d.n_heads * d.head_dim;
  // (the unit arithmetic of the kernel is 32-bit: units of the largest matrix times CTAs)
  const long long units = (long long)((d.vocab + 255) / 256) * ((std::max(d.d_model, d.d_ffn) * 2 + 63) / 64);
  return d.d_model % 128 == 0 && hd % 128 == 0 && units * 1024 < (1ll << 31) &&
         (d.vocab + 255) / 256 <= pk::MAX_TILES && (d.d_ffn + 127) / 128 <= pk::MAX_TILES &&
         (3 * hd + 255) / 256 <= pk::MAX_TILES;
}
int sm_count() {
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1)
    n = 148;
  return n;
}
int pk_splits_for(const specvla_model_desc &d, int G) {
  int s = G / d.n_heads;
  return s < 1 ? 1 : (s > pk::MAX_SPLITS ? pk::MAX_SPLITS : s);
}
// Most output tiles any CTA's unit range touches in one GEMM phase of this model.
int pk_max_segments(const specvla_model_desc &d, int G) {
  const int hd = d.n_heads * d.head_dim;
  auto kb = [](int K) { return (K + gemm_tc::BK - 1) / gemm_tc::BK; };
  auto t256 = [](int N) { return (N + SV_TILE_ROWS - 1) / SV_TILE_ROWS; };
  const int shapes[7][2] = {{t256(3 * hd), kb(d.d_model)}, {t256(d.d_model), kb(hd)},
                            {(d.d_ffn + 127) / 128, kb(d.d_model)}, {t256(d.d_model), kb(d.d_ffn)},
                            {t256(d.vocab), kb(d.d_model)}, {t256(d.n_bins), kb(d.d_model)},
                            {t256(d.d_model), kb(2 * d.d_model)}};
  int worst = 1;
  for (auto &sh : shapes) {
    const long long U = (long long)sh[0] * sh[1];
    for (int c = 0; c < G; c++) {
      const long long b = U * c / G, e = U * (c + 1) / G;
      if (e > b) worst = std::max(worst, (int)((e - 1) / sh[1] - b / sh[1] + 1));
    }
  }
  return worst;
}

// Lays the workspace out; with base == NULL only measures it.
size_t carve(specvla_ctx *c, char *base) {
  const specvla_model_desc &d = c->desc;
  const int hd = d.n_heads * d.head_dim;
  const size_t R = d.max_rows, E = d.max_episodes;
  const size_t lm_rows = c->max_lm_rows, dr = c->max_draft_rows;
  Carver cv{base, 0};
  c->kv_t_layer_stride = (size_t)2 * d.max_seq * hd;
  c->kv_t_ep_stride = c->kv_t_layer_stride * d.n_layers;
  c->kv_d_ep_stride = (size_t)2 * d.max_seq * hd;
  c->kv_t = cv.take<float>(E * c->kv_t_ep_stride);
  c->kv_d = cv.take<float>(E * c->kv_d_ep_stride);
  c->rope_tab = cv.take<float2>((size_t)d.max_seq * (d.head_dim / 2));
  c->x = cv.take<float>(R * d.d_model);
  c->feat = cv.take<float>(R * d.d_model);
  auto limbs = [&](XBuf &b, size_t rows, size_t K) {
    b.rows = (int)rows;
    b.K = (int)K;
    b.plane = rows * K;
    b.p = cv.take<bf16>(2 * b.plane);
  };
  limbs(c->xn, R, d.d_model);
  limbs(c->xin, R, 2 * d.d_model);
  c->q = cv.take<float>(R * hd);
  limbs(c->ao, R, hd);
  limbs(c->hid, R, d.d_ffn);
  limbs(c->lm_in, E, d.d_model);                 // last prefix row of each episode (first token)
  c->nt = (d.d_model + SV_TILE_ROWS - 1) / SV_TILE_ROWS;
  c->ssq = cv.take<float>(R * c->nt);
  c->lm_ssq = cv.take<float>(E * c->nt);
  auto tiles256 = [](int N) { return (N + SV_TILE_ROWS - 1) / SV_TILE_ROWS; };
  {
    // repacked weights: every target layer, the LM head and its action rows, the draft fc and
    // the draft layer
    const size_t layer = gemm_tc::packed_elems(tiles256(3 * hd), d.d_model) +
                         gemm_tc::packed_elems(tiles256(d.d_model), hd) +
                         gemm_tc::packed_elems((d.d_ffn + 127) / 128, d.d_model) +
                         gemm_tc::packed_elems(tiles256(d.d_model), d.d_ffn);
    const size_t lm = gemm_tc::packed_elems(tiles256(d.vocab), d.d_model);
    const size_t draft = layer + gemm_tc::packed_elems(tiles256(d.n_bins), d.d_model) +
                         gemm_tc::packed_elems(tiles256(d.d_model), 2 * d.d_model);
    const bool q8 = d.weight_bits == 8;
    // quantised target: its matrices are kept as int8 codes (one byte per element) plus row scales
    c->packed_elems = draft + (q8 ? 0 : layer * (size_t)d.n_layers + lm);
    c->packed = cv.take<bf16>(c->packed_elems);
    c->packed_q8_bytes = q8 ? layer * (size_t)d.n_layers + lm : 0;
    c->packed_q8 = cv.take<signed char>(c->packed_q8_bytes);
    c->wscale_elems = q8 ? (size_t)d.n_layers * (3 * hd + 2 * d.d_model + 2 * d.d_ffn) + d.vocab : 0;
    c->wscale = cv.take<float>(c->wscale_elems);
  }
  // full-vocabulary logits are stored only for the draft model's top-k when it ranges over the
  // whole vocabulary (action_only = 0); the greedy argmax works from per-128-column candidates
  c->lgs_rows = (int)dr;
  c->lgs = cv.take<float>((size_t)c->lgs_rows * (d.action_only ? d.n_bins : d.vocab));
  c->cand_nc = 2 * tiles256(d.vocab);
  c->cand = cv.take<float4>((lm_rows > 32 ? lm_rows : 32) * (size_t)c->cand_nc);
  c->pend_feat = cv.take<float>(E * SV_MAX_PENDING * d.d_model);
  c->margin = cv.take<float>(R);
  c->top_lp = cv.take<float>(dr * SV_TOPK);
  c->rt.tok = cv.take<int>(R);
  c->rt.src = cv.take<int>(R);
  c->rt.ep = cv.take<int>(R);
  c->rt.pos = cv.take<int>(R);
  c->rt.slot = cv.take<int>(R);
  c->rt.nvis = cv.take<int>(R);
  c->rt.tbase = cv.take<int>(R);
  c->rt.mask = cv.take<uint32_t>(R * 4);
  c->feat_src = cv.take<int>(R);
  c->lm_rows = cv.take<int>(R);
  c->greedy = cv.take<int>(R);
  c->top_tok = cv.take<int>(dr * SV_TOPK);
  c->out_m = cv.take<int>(E);
  c->out_tok = cv.take<int>(E * (SV_MAX_DEPTH + 1));
  c->out_path = cv.take<int>(E * (SV_MAX_DEPTH + 1));
  c->st = cv.take<EpState>(E);
  c->trees = cv.take<DevTree>(E);
  c->err = cv.take<int>(32);
  c->chunk = cv.take<ChunkState>(1);
  // persistent forward kernel: packed operands, partial tiles, attention slices, candidates
  if (pk_shapes_ok(d) && d.weight_bits != 8) {
    const size_t G = c->pk_G;
    auto kblocks = [](int K) { return (size_t)((K + gemm_tc::BK - 1) / gemm_tc::BK); };
    c->pk_nt = d.d_model / 128;
    c->pk_splits = pk_splits_for(d, (int)G);
    c->pk_max_seg = pk_max_segments(d, (int)G);
    c->pk_xn = cv.take<bf16>(kblocks(d.d_model) * pk::X_BLOCK_ELEMS);
    c->pk_ao = cv.take<bf16>(kblocks(hd) * pk::X_BLOCK_ELEMS);
    c->pk_hid = cv.take<bf16>(kblocks(d.d_ffn) * pk::X_BLOCK_ELEMS);
    c->pk_part = cv.take<float>(G * c->pk_max_seg * pk::PART_ELEMS);
    c->pk_apart = cv.take<float>((size_t)d.n_heads * c->pk_splits * 32 * (d.head_dim + 4));
    c->pk_ssq = cv.take<float>((size_t)32 * c->pk_nt);
    c->pk_ops_t = cv.take<pk::Op>((size_t)5 * d.n_layers + 2);
    c->pk_bar = cv.take<unsigned>(32);
  }
  return (cv.off + ALIGN - 1) / ALIGN * ALIGN;
}

void derive_caps(specvla_ctx *c) {
  const specvla_model_desc &d = c->desc;
  c->hd = d.n_heads * d.head_dim;
  c->pk_G = std::min(sm_count(), (int)pk::MAX_G);
  size_t lm = (size_t)d.max_episodes * SV_MAX_TREE;
  if (lm > (size_t)d.max_rows) lm = d.max_rows;
  c->max_lm_rows = (int)lm;
  size_t dr = (size_t)d.max_episodes * 16;
  if (dr > (size_t)d.max_rows) dr = d.max_rows;
  c->max_draft_rows = (int)dr;
}

// Folds the recorded GEMM event pairs into the per-class sums. The stream must be idle.
void prof_collect(specvla_ctx *ctx) {
  for (int i = 0; i < ctx->prof_used; i++) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, ctx->prof_ev[2 * i], ctx->prof_ev[2 * i + 1]) == cudaSuccess) {
      ctx->prof_ms[ctx->prof_cls[i]] += ms;
      ctx->prof_n[ctx->prof_cls[i]]++;
    }
  }
  ctx->prof_used = 0;
}

cudaLaunchConfig_t launch_cfg(dim3 grid, dim3 block, cudaStream_t st, cudaLaunchAttribute *attr, bool pdl) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.stream = st;
  attr->id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr->val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cfg;
}
// Launch of a row-wise / tree kernel on the call's stream, allowed to overlap its predecessor.
#define LAUNCH(kernel, grid, block, ...)                                                       \
  do {                                                                                         \
    cudaLaunchAttribute _at;                                                                   \
    cudaLaunchConfig_t _cfg = launch_cfg(grid, block, st, &_at, ctx->use_pdl);                 \
    CU(cudaLaunchKernelEx(&_cfg, kernel, __VA_ARGS__));                                        \
    ctx->launches++;                                                                           \
  } while (0)

// One GEMM over R rows of A against W with the fused epilogue described by `ea` (mode and
// outputs; the row range is filled in here): one launch, 128 rows per CTA.
// next: the matrix of the GEMM that will follow (its head is prefetched into L2), or NULL.
int gemm(specvla_ctx *ctx, const XBuf &A, const WMat &W, int R, gemm_tc::EpiArgs ea, cudaStream_t st, int cls,
         const WMat *next = nullptr, bool next_swiglu = false) {
  if (!W.has_map || !A.has_map || A.K != W.K) return SPECVLA_ERR_BAD_STATE;
  const bool swiglu = ea.mode == gemm_tc::EPI_SWIGLU;
  const int tiles = swiglu ? (ea.N + 127) / 128 : (W.N + SV_TILE_ROWS - 1) / SV_TILE_ROWS;
  const int KB = (W.K + gemm_tc::BK - 1) / gemm_tc::BK;
  ea.wpacked = W.packed;
  ea.wq8 = W.q8;
  ea.wscale = W.scale;
  ea.wait_ns = ctx->wait_ns;
  ea.inv_k = 1.f / (float)W.K;
  ea.eps = ctx->desc.rms_eps;
  const bool prof = (ctx->prof_mask & ctx->phase) && 2 * (ctx->prof_used + 1) <= (int)ctx->prof_ev.size();
  if (prof) CU(cudaEventRecord(ctx->prof_ev[2 * ctx->prof_used], st));
  const gemm_ck::RowPlan plan = gemm_ck::plan_rows(R, tiles, KB, ctx->fit);
  const int chunks = plan.chunks, S = plan.S;
  ea.row0 = 0;
  ea.T = R;
  ea.chunk_rows = plan.chunk_rows;
  ea.tn_chunk = plan.tn_chunk;
  ea.tn_tail = plan.tn_tail;
  ea.pf_w = nullptr;
  if (next && (next->packed || next->q8) && ctx->use_l2_prefetch) {
    // start pulling the next matrix (up to L2_PREFETCH_BYTES of it)
    ea.pf_tiles = next_swiglu ? (next->N / 2 + 127) / 128 : (next->N + SV_TILE_ROWS - 1) / SV_TILE_ROWS;
    ea.pf_KB = (next->K + gemm_tc::BK - 1) / gemm_tc::BK;
    ea.pf_S = gemm_ck::plan_rows(R, ea.pf_tiles, ea.pf_KB, ctx->fit).S;
    ea.pf_unit_bytes = next->q8 ? gemm_tc::W_STAGE_BYTES / 2 : gemm_tc::W_STAGE_BYTES;
    const size_t per_cta = L2_PREFETCH_BYTES / ((size_t)ea.pf_tiles * ea.pf_S) / ea.pf_unit_bytes;
    ea.pf_units = per_cta < 1 ? 1 : (int)per_cta;
    ea.pf_w = next->q8 ? static_cast<const void *>(next->q8) : static_cast<const void *>(next->packed);
  }
  CU(gemm_ck::launch(W.map, A.map[tn_index(ea.tn_chunk)], A.map[tn_index(ea.tn_tail)], ea, tiles, KB, S,
                     ctx->err, st, ctx->use_pdl));
  ctx->launches++;
  if (prof) {
    CU(cudaEventRecord(ctx->prof_ev[2 * ctx->prof_used + 1], st));
    ctx->prof_cls[ctx->prof_used++] = cls;
    ctx->prof_bytes[cls] += (double)W.N * W.K * (W.q8 ? 1 : sizeof(bf16));
  }
  return SPECVLA_OK;
}

gemm_tc::EpiArgs epi_plain(float *out, int ldo, int N, const float *ssq_in, int nt_in) {
  gemm_tc::EpiArgs e = {};
  e.mode = gemm_tc::EPI_PLAIN;
  e.N = N;
  e.out = out;
  e.ldo = ldo;
  e.ssq_in = ssq_in;
  e.nt_in = nt_in;
  return e;
}
// Draft scoring fused into the (one-tile) action-row LM head: log-softmax + top-k per row.
gemm_tc::EpiArgs epi_topk(specvla_ctx *ctx, int N, int tok_offset) {
  gemm_tc::EpiArgs e = {};
  e.mode = gemm_tc::EPI_TOPK;
  e.N = N;
  e.lo = 0;
  e.hi = N;
  e.tok_offset = tok_offset;
  e.top_tok = ctx->top_tok;
  e.top_lp = ctx->top_lp;
  return e;
}
// x (+)= result; xn = limbs(x * gain) (gain may be NULL); ssq = per-tile sums of squares of x.
gemm_tc::EpiArgs epi_resid(specvla_ctx *ctx, int accumulate, const float *gain) {
  gemm_tc::EpiArgs e = {};
  e.mode = gemm_tc::EPI_RESID;
  e.N = ctx->desc.d_model;
  e.x = ctx->x;
  e.accumulate = accumulate;
  e.gain = gain;
  e.xn = ctx->xn.p;
  e.xn_plane = ctx->xn.plane;
  e.ssq_out = ctx->ssq;
  return e;
}

// Tree-mask attention over the rows of `rows` (contiguous per episode) against `cache`.
int attention(specvla_ctx *ctx, const EpArgs &rows, const float *cache, size_t ep_stride, cudaStream_t st) {
  const specvla_model_desc &d = ctx->desc;
  attn::Args a = {};
  a.q = ctx->q;
  a.cache = cache;
  a.ep_stride = ep_stride;
  a.max_seq = d.max_seq;
  a.H = d.n_heads;
  a.rt = ctx->rt;
  a.scale = 1.f / sqrtf((float)d.head_dim);
  a.out = ctx->ao.p;
  a.out_plane = ctx->ao.plane;
  const int blocks = attn::blocks_of(rows);
  if (blocks < 1) return SPECVLA_OK;
  // few row blocks: slice the key range so that the launch still covers the SMs
  const int ctas = blocks * d.n_heads;
  a.splits = 1;
  if (ctas < 96) {
    a.splits = attn::MAX_SPLIT_CTAS / ctas;
    if (a.splits > attn::MAX_SPLITS) a.splits = attn::MAX_SPLITS;
    if (a.splits < 1) a.splits = 1;
  }
  // the key slices of a row block are one cluster (they merge through distributed shared memory)
  // (unsliced: heads on x, see the kernel)
  const dim3 grid = a.splits == 1 ? dim3(d.n_heads, blocks) : dim3(blocks * a.splits, d.n_heads);
  cudaLaunchAttribute at[2];
  cudaLaunchConfig_t cfg = launch_cfg(grid, dim3(attn::THREADS), st, &at[0], ctx->use_pdl);
  at[cfg.numAttrs].id = cudaLaunchAttributeClusterDimension;
  at[cfg.numAttrs].val.clusterDim.x = a.splits;
  at[cfg.numAttrs].val.clusterDim.y = 1;
  at[cfg.numAttrs].val.clusterDim.z = 1;
  cfg.numAttrs++;
  const bool sliced = a.splits > 1;
  if (d.head_dim == 128) {
    cfg.dynamicSmemBytes = attn::smem_bytes<128>();
    CU(sliced ? cudaLaunchKernelEx(&cfg, attn::tree_attention_kernel<128, true>, rows, a)
              : cudaLaunchKernelEx(&cfg, attn::tree_attention_kernel<128, false>, rows, a));
  } else {
    cfg.dynamicSmemBytes = attn::smem_bytes<64>();
    CU(sliced ? cudaLaunchKernelEx(&cfg, attn::tree_attention_kernel<64, true>, rows, a)
              : cudaLaunchKernelEx(&cfg, attn::tree_attention_kernel<64, false>, rows, a));
  }
  ctx->launches++;
  return SPECVLA_OK;
}

// One pre-norm decoder layer over R rows. In: x (residual, fp32), xn = limbs(x * norm1 gain) and
// ssq = sums of squares of x. Out: x updated; xn = limbs(x * next_gain) (limbs(x) when next_gain
// is NULL) and ssq for the norm that follows.
// after: the matrix of the GEMM that follows this layer (next layer's QKV, the LM head), or NULL.
int run_layer(specvla_ctx *ctx, const LayerW &w, int R, const EpArgs &rows, float *cache, size_t ep_stride,
              const float *next_gain, const WMat *after, cudaStream_t st) {
  const specvla_model_desc &d = ctx->desc;
  const int hd = ctx->hd, F = d.d_ffn;
  // QKV projection; its epilogue applies the norm's row scale and RoPE and appends K, V to the cache
  gemm_tc::EpiArgs qk = {};
  qk.mode = gemm_tc::EPI_QKV;
  qk.N = 3 * hd;
  qk.ssq_in = ctx->ssq;
  qk.nt_in = ctx->nt;
  qk.rt = ctx->rt;
  qk.rope_tab = ctx->rope_tab;
  qk.q = ctx->q;
  qk.cache = cache;
  qk.ep_stride = ep_stride;
  qk.max_seq = d.max_seq;
  qk.hd = hd;
  qk.dh = d.head_dim;
  TRY(gemm(ctx, ctx->xn, w.wqkv, R, qk, st, SPECVLA_PROF_QKV, &w.wo));
  TRY(attention(ctx, rows, cache, ep_stride, st));
  TRY(gemm(ctx, ctx->ao, w.wo, R, epi_resid(ctx, 1, w.norm2), st, SPECVLA_PROF_O, &w.wgu, true));
  gemm_tc::EpiArgs sw = {};
  sw.mode = gemm_tc::EPI_SWIGLU;
  sw.N = F;
  sw.up_off = F;
  sw.ssq_in = ctx->ssq;
  sw.nt_in = ctx->nt;
  sw.hid = ctx->hid.p;
  sw.hid_plane = ctx->hid.plane;
  TRY(gemm(ctx, ctx->xn, w.wgu, R, sw, st, SPECVLA_PROF_GATE_UP, &w.wd));
  TRY(gemm(ctx, ctx->hid, w.wd, R, epi_resid(ctx, 1, next_gain), st, SPECVLA_PROF_DOWN, after));
  return SPECVLA_OK;
}

// Target model over the R rows described by ctx->rt: embedding, all layers. Leaves the residual
// in ctx->x, limbs(x * final-norm gain) in ctx->xn and the sums of squares in ctx->ssq: the
// final RMSNorm itself is applied by whoever consumes them (LM head epilogue, feature readers).
// The head matrix the greedy decoding after a target forward reads (see lm_head_greedy).
const WMat *head_after_forward(const specvla_ctx *ctx) {
  return (ctx->desc.action_only && ctx->has_draft && !ctx->lm_head.q8) ? &ctx->lm_head_act : &ctx->lm_head;
}
int target_forward(specvla_ctx *ctx, int R, const EpArgs &rows, const bf16 *embeds, cudaStream_t st) {
  const specvla_model_desc &d = ctx->desc;
  LAUNCH(epi::embed_kernel, dim3(R), dim3(epi::THREADS), ctx->rt, embeds, ctx->embed, ctx->layers[0].norm1,
         d.d_model, ctx->nt, ctx->x, ctx->xn.p, ctx->xn.plane, ctx->ssq);
  for (int l = 0; l < d.n_layers; l++) {
    const bool last = (l + 1 == d.n_layers);
    TRY(run_layer(ctx, ctx->layers[l], R, rows, ctx->kv_t + (size_t)l * ctx->kv_t_layer_stride,
                  ctx->kv_t_ep_stride, last ? ctx->final_norm : ctx->layers[l + 1].norm1,
                  last ? head_after_forward(ctx) : &ctx->layers[l + 1].wqkv, st));
  }
  ctx->last_rows = R;
  ctx->last_ssq = ctx->ssq;
  ctx->last_nt = ctx->nt;
  return SPECVLA_OK;
}

// Draft model over R rows: ctx->xin = [feature ; embedding] rows are already built.
// Leaves the layer outputs in ctx->x (fp32) and ctx->xn (limbs, un-normalised).
int draft_forward(specvla_ctx *ctx, int R, const EpArgs &rows, cudaStream_t st) {
  TRY(gemm(ctx, ctx->xin, ctx->draft_fc, R, epi_resid(ctx, 0, ctx->dlayer.norm1), st, SPECVLA_PROF_FC,
           &ctx->dlayer.wqkv));
  return run_layer(ctx, ctx->dlayer, R, rows, ctx->kv_d, ctx->kv_d_ep_stride, nullptr,
                   ctx->desc.action_only ? &ctx->lm_head_act : &ctx->lm_head, st);
}

// LM head over `rows` two-limb rows of A into ctx->lgs [rows][vocab] (draft top-k over the whole
// vocabulary). ssq != NULL: the rows are limbs(x * final gain) and get their RMSNorm scale here.
int lm_head(specvla_ctx *ctx, const XBuf &A, const float *ssq, int rows, cudaStream_t st) {
  if (rows > ctx->max_lm_rows || rows > ctx->lgs_rows || ctx->desc.action_only) return SPECVLA_ERR_CAPACITY;
  return gemm(ctx, A, ctx->lm_head, rows, epi_plain(ctx->lgs, ctx->desc.vocab, ctx->desc.vocab, ssq, ctx->nt),
              st, SPECVLA_PROF_LM_HEAD);
}

void argmax_range(const specvla_ctx *ctx, int *lo, int *hi);
// LM head + greedy argmax (Eq. 1) over `rows` rows: the GEMM's epilogue leaves the top-2 of every
// 128 logit columns, a one-warp-per-row kernel finishes greedy token and margin. The logits
// themselves are written only when logits_out is given (parity tests).
int lm_head_greedy(specvla_ctx *ctx, const XBuf &A, const float *ssq, int rows, float *logits_out, cudaStream_t st) {
  if (rows > ctx->max_lm_rows) return SPECVLA_ERR_CAPACITY;
  const specvla_model_desc &d = ctx->desc;
  // Greedy decoding over the action ids alone needs only their rows of the LM head (the copy the
  // draft scoring uses: one or a few tiles instead of the whole vocabulary), unless the caller
  // wants the logits themselves.
  const bool act_rows = d.action_only && !logits_out && ctx->has_draft && !ctx->lm_head.q8;
  const WMat &W = act_rows ? ctx->lm_head_act : ctx->lm_head;
  gemm_tc::EpiArgs e = epi_plain(logits_out, d.vocab, W.N, ssq, ctx->nt);
  e.cand = ctx->cand;
  if (act_rows) {
    e.lo = 0;
    e.hi = d.n_bins;
  } else {
    argmax_range(ctx, &e.lo, &e.hi);
  }
  TRY(gemm(ctx, A, W, rows, e, st, SPECVLA_PROF_LM_HEAD));
  const int nc = 2 * ((W.N + SV_TILE_ROWS - 1) / SV_TILE_ROWS);
  LAUNCH(epi::argmax_merge_kernel, dim3((rows + 3) / 4), dim3(128), (const float4 *)ctx->cand, nc, rows,
         act_rows ? d.action_base : 0, ctx->greedy, ctx->margin);
  return SPECVLA_OK;
}

void argmax_range(const specvla_ctx *ctx, int *lo, int *hi) {
  if (ctx->desc.action_only) {
    *lo = ctx->desc.action_base;
    *hi = ctx->desc.action_base + ctx->desc.n_bins;
  } else {
    *lo = 0;
    *hi = ctx->desc.vocab;
  }
}

// Phase list of the target forward for the persistent kernel: embedding, the layers, the LM head
// with the greedy argmax. Built on the host, kept in the workspace.
void pk_build_target_ops(specvla_ctx *ctx) {
  const specvla_model_desc &d = ctx->desc;
  const int hd = ctx->hd, F = d.d_ffn;
  auto kb = [](int K) { return (K + gemm_tc::BK - 1) / gemm_tc::BK; };
  auto t256 = [](int N) { return (N + SV_TILE_ROWS - 1) / SV_TILE_ROWS; };
  std::vector<pk::Op> ops;
  auto gemm_op = [&](int mode, const WMat &w, int tiles, int N, const bf16 *xin) {
    pk::Op o = {};
    o.kind = pk::OP_GEMM;
    o.mode = mode;
    o.w = w.packed;
    o.tiles = tiles;
    o.KB = kb(w.K);
    o.N = N;
    o.xin = xin;
    return o;
  };
  pk::Op e = {};
  e.kind = pk::OP_EMBED;
  ops.push_back(e);
  for (int l = 0; l < d.n_layers; l++) {
    const LayerW &w = ctx->layers[l];
    float *cache = ctx->kv_t + (size_t)l * ctx->kv_t_layer_stride;
    pk::Op q = gemm_op(gemm_tc::EPI_QKV, w.wqkv, t256(3 * hd), 3 * hd, ctx->pk_xn);
    q.use_scale = 1;
    q.cache = cache;
    q.ep_stride = ctx->kv_t_ep_stride;
    ops.push_back(q);
    pk::Op a = {};
    a.kind = pk::OP_ATTN;
    a.cache = cache;
    a.ep_stride = ctx->kv_t_ep_stride;
    ops.push_back(a);
    pk::Op o = gemm_op(gemm_tc::EPI_RESID, w.wo, t256(d.d_model), d.d_model, ctx->pk_ao);
    o.accumulate = 1;
    o.gain = w.norm2;
    ops.push_back(o);
    pk::Op g = gemm_op(gemm_tc::EPI_SWIGLU, w.wgu, (F + 127) / 128, F, ctx->pk_xn);
    g.use_scale = 1;
    ops.push_back(g);
    pk::Op dn = gemm_op(gemm_tc::EPI_RESID, w.wd, t256(d.d_model), d.d_model, ctx->pk_hid);
    dn.accumulate = 1;
    dn.gain = (l + 1 == d.n_layers) ? ctx->final_norm : ctx->layers[l + 1].norm1;
    ops.push_back(dn);
  }
  pk::Op lm = gemm_op(gemm_tc::EPI_PLAIN, ctx->lm_head, t256(d.vocab), d.vocab, ctx->pk_xn);
  lm.use_scale = 1;
  lm.ldo = d.vocab;
  argmax_range(ctx, &lm.lo, &lm.hi);
  lm.post = pk::POST_ARGMAX;
  ops.push_back(lm);
  ctx->pk_n_ops_t = (int)ops.size();
  cudaMemcpy(ctx->pk_ops_t, ops.data(), ops.size() * sizeof(pk::Op), cudaMemcpyHostToDevice);
}

template <int DH> bool pk_prepare_dh(specvla_ctx *ctx) {
  if (cudaFuncSetAttribute(pk::forward_pk_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           pk::smem_bytes<DH>()) != cudaSuccess)
    return false;
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, pk::forward_pk_kernel<DH>, pk::THREADS,
                                                    pk::smem_bytes<DH>()) != cudaSuccess)
    return false;
  return per_sm >= 1;
}
// Shared-memory attribute and residency check of the persistent kernel; clears its buffers (the
// padding rows and columns of the packed operands are read by the MMAs and must stay finite).
bool pk_prepare(specvla_ctx *ctx) {
  const specvla_model_desc &d = ctx->desc;
  int coop = 0, dev = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
  const bool ok = coop && (d.head_dim == 128 ? pk_prepare_dh<128>(ctx) : pk_prepare_dh<64>(ctx));
  cudaGetLastError();
  if (!ok) return false;
  auto kblocks = [](int K) { return (size_t)((K + gemm_tc::BK - 1) / gemm_tc::BK); };
  cudaMemsetAsync(ctx->pk_xn, 0, kblocks(d.d_model) * pk::X_STAGE_BYTES);
  cudaMemsetAsync(ctx->pk_ao, 0, kblocks(ctx->hd) * pk::X_STAGE_BYTES);
  cudaMemsetAsync(ctx->pk_hid, 0, kblocks(d.d_ffn) * pk::X_STAGE_BYTES);
  cudaMemsetAsync(ctx->pk_bar, 0, 32 * sizeof(unsigned));
  return true;
}

// Target forward + LM head + greedy argmax over the R <= 32 rows of one episode described by
// ctx->rt, as ONE cooperative launch. Leaves the residual in ctx->x, the sums of squares in
// ctx->pk_ssq, greedy tokens and margins in ctx->greedy / ctx->margin.
int pk_target_forward(specvla_ctx *ctx, int R, const bf16 *embeds, float *logits_out, cudaStream_t st) {
  const specvla_model_desc &d = ctx->desc;
  pk::Params p = {};
  p.ops = ctx->pk_ops_t;
  p.n_ops = ctx->pk_n_ops_t;
  p.T = R;
  p.max_seg = ctx->pk_max_seg;
  p.rt = ctx->rt;
  p.embeds = embeds;
  p.E = ctx->embed;
  p.gain0 = ctx->layers[0].norm1;
  p.d = d.d_model;
  p.hd = ctx->hd;
  p.H = d.n_heads;
  p.dh = d.head_dim;
  p.max_seq = d.max_seq;
  p.eps = d.rms_eps;
  p.attn_scale = 1.f / sqrtf((float)d.head_dim);
  p.nt = ctx->pk_nt;
  p.x = ctx->x;
  p.ssq = ctx->pk_ssq;
  p.q = ctx->q;
  p.xn_pk = ctx->pk_xn;
  p.ao_pk = ctx->pk_ao;
  p.hid_pk = ctx->pk_hid;
  p.part = ctx->pk_part;
  p.apart = ctx->pk_apart;
  p.splits = ctx->pk_splits;
  p.rope_tab = ctx->rope_tab;
  p.cand = ctx->cand;
  p.logits_out = logits_out;
  p.greedy = ctx->greedy;
  p.margin = ctx->margin;
  p.bar = ctx->pk_bar;
  p.err = ctx->err;
  p.wait_ns = ctx->wait_ns;
  CU(cudaMemsetAsync(ctx->pk_bar, 0, sizeof(unsigned), st));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(ctx->pk_G);
  cfg.blockDim = dim3(pk::THREADS);
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeCooperative;
  at[0].val.cooperative = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  if (d.head_dim == 128) {
    cfg.dynamicSmemBytes = pk::smem_bytes<128>();
    CU(cudaLaunchKernelEx(&cfg, pk::forward_pk_kernel<128>, p));
  } else {
    cfg.dynamicSmemBytes = pk::smem_bytes<64>();
    CU(cudaLaunchKernelEx(&cfg, pk::forward_pk_kernel<64>, p));
  }
  ctx->launches++;
  ctx->last_rows = R;
  ctx->last_ssq = ctx->pk_ssq;
  ctx->last_nt = ctx->pk_nt;
  return SPECVLA_OK;
}

int check_episodes(const specvla_ctx *ctx, int n_ep, const int *episodes) {
  if (!ctx || !episodes || n_ep < 1) return SPECVLA_ERR_INVALID_ARG;
  if (n_ep > ctx->desc.max_episodes) return SPECVLA_ERR_CAPACITY;
  for (int i = 0; i < n_ep; i++) {
    if (episodes[i] < 0 || episodes[i] >= ctx->desc.max_episodes) return SPECVLA_ERR_INVALID_ARG;
    for (int j = 0; j < i; j++)
      if (episodes[j] == episodes[i]) return SPECVLA_ERR_INVALID_ARG;
  }
  return SPECVLA_OK;
}

int validate_tree(const specvla_tree &t) {
  if (t.n_rows < 1 || t.n_rows > SV_MAX_TREE) return SPECVLA_ERR_BAD_TREE;
  if (!t.tokens || !t.parent || !t.depth) return SPECVLA_ERR_INVALID_ARG;
  if (t.parent[0] != -1 || t.depth[0] != 0) return SPECVLA_ERR_BAD_TREE;
  for (int i = 1; i < t.n_rows; i++) {
    const int p = t.parent[i];
    if (p < 0 || p >= i) return SPECVLA_ERR_BAD_TREE;
    if (t.depth[i] != t.depth[p] + 1 || t.depth[i] > SV_MAX_DEPTH) return SPECVLA_ERR_BAD_TREE;
  }
  return SPECVLA_OK;
}

// n_nodes: nodes drafted; n_rows_out (may be NULL): rows verified (root + nodes kept).
int validate_shape(const specvla_tree_shape *s, int *n_nodes, int *n_rows_out = nullptr) {
  if (!s || s->depth < 0 || s->depth > SV_MAX_DEPTH || s->keep < 0 || s->keep > SV_MAX_TREE - 1)
    return SPECVLA_ERR_INVALID_ARG;
  const int level_max = s->keep > 0 ? 64 : 16;            // nodes of one level
  int prev = 1, total = 0;
  for (int l = 0; l < s->depth; l++) {
    if (s->branch[l] < 1 || s->branch[l] > SV_MAX_BRANCH) return SPECVLA_ERR_INVALID_ARG;
    if (s->expand[l] < 1 || s->expand[l] > 16 || s->expand[l] > prev) return SPECVLA_ERR_INVALID_ARG;
    if (l == 0 && s->expand[0] != 1) return SPECVLA_ERR_INVALID_ARG;
    prev = s->branch[l] * s->expand[l];
    if (prev > level_max) return SPECVLA_ERR_INVALID_ARG;
    total += prev;
  }
  const int kept = (s->keep > 0 && s->keep < total) ? s->keep : total;
  if (1 + total > SV_MAX_CAND || 1 + kept > SV_MAX_TREE) return SPECVLA_ERR_INVALID_ARG;
  *n_nodes = total;
  if (n_rows_out) *n_rows_out = 1 + kept;
  return SPECVLA_OK;
}

}  // namespace

// =====================================================================================
extern "C" {

size_t specvla_workspace_bytes(const specvla_model_desc *desc) {
  if (!desc_ok(desc)) return 0;
  specvla_ctx tmp{};
  tmp.desc = *desc;
  derive_caps(&tmp);
  return carve(&tmp, nullptr);
}

int specvla_create(const specvla_model_desc *desc, const specvla_weights *tw,
                   const specvla_draft_weights *dw, void *workspace, size_t workspace_bytes,
                   specvla_ctx **out) {
  if (!out) return SPECVLA_ERR_INVALID_ARG;
  *out = nullptr;
  if (!desc_ok(desc) || !tw || !workspace) return SPECVLA_ERR_INVALID_ARG;
  if (!tw->embed || !tw->lm_head || !tw->final_norm || !tw->wqkv || !tw->wo || !tw->wgu || !tw->wd ||
      !tw->norm1 || !tw->norm2)
    return SPECVLA_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) % ALIGN) != 0) return SPECVLA_ERR_INVALID_ARG;
  int dev = 0;
  cudaDeviceProp prop;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess)
    return SPECVLA_ERR_CUDA;
  if (prop.major != 10) return SPECVLA_ERR_UNSUPPORTED_ARCH;

  specvla_ctx *ctx = new (std::nothrow) specvla_ctx();
  if (!ctx) return SPECVLA_ERR_INVALID_ARG;
  ctx->desc = *desc;
  derive_caps(ctx);
  const size_t need = carve(ctx, nullptr);
  if (workspace_bytes < need) {
    delete ctx;
    return SPECVLA_ERR_CAPACITY;
  }
  carve(ctx, static_cast<char *>(workspace));
  const int hd = ctx->hd, D = desc->d_model, F = desc->d_ffn;
  ctx->use_pdl = true;
  ctx->use_l2_prefetch = true;
  ctx->fit = gemm_ck::query_cluster_fit();
  size_t packed_used = 0, q8_used = 0, scale_used = 0;
  bool pack_ok = true;
  const bool quantise = desc->weight_bits == 8;
  // swiglu: the matrix is [gate; up] stacked ([2F, K]) and is packed as tiles of 128 + 128 rows.
  // q8: a matrix of the quantised target: row scales and int8 codes instead of the bf16 copy.
  auto wmat = [&](const void *p, int N, int K, bool swiglu = false, bool q8 = false) {
    WMat w{};
    w.p = static_cast<const bf16 *>(p);
    w.N = N;
    w.K = K;
    w.has_map = p && gemm_tc::make_w_map(&w.map, w.p, N, K);
    w.packed = nullptr;
    if (p && q8) {
      const int F = N / 2;
      const int tiles = swiglu ? (F + 127) / 128 : (N + SV_TILE_ROWS - 1) / SV_TILE_ROWS;
      const int KB = (K + gemm_tc::BK - 1) / gemm_tc::BK;
      const size_t bytes = gemm_tc::packed_elems(tiles, K);
      if (q8_used + bytes > ctx->packed_q8_bytes || scale_used + (size_t)N > ctx->wscale_elems) {
        pack_ok = false;
        return w;
      }
      float *sc = ctx->wscale + scale_used;
      signed char *dst = ctx->packed_q8 + q8_used;
      scale_used += N;
      q8_used += bytes;
      gemm_tc::row_scale_q8_kernel<<<(N + 7) / 8, 256>>>(w.p, N, K, sc);
      gemm_tc::pack_weights_q8_kernel<<<148 * 8, 256>>>(w.p, N, K, tiles, KB, swiglu ? 1 : 0, F, sc, dst);
      w.q8 = dst;
      w.scale = sc;
      return w;
    }
    if (p) {
      const int F = N / 2;
      const int tiles = swiglu ? (F + 127) / 128 : (N + SV_TILE_ROWS - 1) / SV_TILE_ROWS;
      const size_t elems = gemm_tc::packed_elems(tiles, K);
      if (packed_used + elems > ctx->packed_elems) {
        pack_ok = false;
        return w;
      }
      bf16 *dst = ctx->packed + packed_used;
      packed_used += elems;
      gemm_tc::pack_weights_kernel<<<148 * 8, 256>>>(w.p, N, K, tiles, (K + gemm_tc::BK - 1) / gemm_tc::BK,
                                                     swiglu ? 1 : 0, F, dst);
      w.packed = dst;
    }
    return w;
  };
  auto xmaps = [&](XBuf &b) {
    b.has_map = true;
    for (int i = 0; i < 16 && b.has_map; i++)
      b.has_map = gemm_tc::make_x_map(&b.map[i], b.p, b.plane, b.rows, b.K, 8 * (i + 1));
  };
  xmaps(ctx->xn);
  xmaps(ctx->xin);
  xmaps(ctx->ao);
  xmaps(ctx->hid);
  xmaps(ctx->lm_in);
  ctx->embed = static_cast<const bf16 *>(tw->embed);
  ctx->lm_head = wmat(tw->lm_head, desc->vocab, D, false, quantise);
  ctx->final_norm = tw->final_norm;
  ctx->layers.resize(desc->n_layers);
  for (int l = 0; l < desc->n_layers; l++) {
    if (!tw->wqkv[l] || !tw->wo[l] || !tw->wgu[l] || !tw->wd[l] || !tw->norm1[l] || !tw->norm2[l]) {
      delete ctx;
      return SPECVLA_ERR_INVALID_ARG;
    }
    ctx->layers[l] = LayerW{wmat(tw->wqkv[l], 3 * hd, D, false, quantise), wmat(tw->wo[l], D, hd, false, quantise),
                            wmat(tw->wgu[l], 2 * F, D, true, quantise), wmat(tw->wd[l], D, F, false, quantise),
                            tw->norm1[l], tw->norm2[l]};
  }
  ctx->has_draft = dw && dw->fc && dw->wqkv && dw->wo && dw->wgu && dw->wd && dw->norm1 && dw->norm2;
  if (ctx->has_draft) {
    // the draft only ranks action tokens when action_only is set: those rows of the LM head suffice
    ctx->lm_head_act = wmat(static_cast<const bf16 *>(tw->lm_head) + (size_t)desc->action_base * D, desc->n_bins, D);
    ctx->draft_fc = wmat(dw->fc, D, 2 * D);
    ctx->dlayer = LayerW{wmat(dw->wqkv, 3 * hd, D), wmat(dw->wo, D, hd), wmat(dw->wgu, 2 * F, D, true),
                         wmat(dw->wd, D, F), dw->norm1, dw->norm2};
  }
  ctx->wait_ns = 2000000000ull;
  ctx->last_ssq = ctx->ssq;
  ctx->last_nt = ctx->nt;
  ctx->pk_ok = false;
  ctx->use_pk = false;            // measured slower than one launch per GEMM on B200: opt-in
  if (pk_shapes_ok(*desc) && pack_ok && !quantise) {
    pk_build_target_ops(ctx);
    ctx->pk_ok = pk_prepare(ctx);
  }
  ctx->hP.assign(desc->max_episodes, -1);
  ctx->hPending.assign(desc->max_episodes, 0);
  ctx->hTreeRows.assign(desc->max_episodes, 0);
  const size_t small_b = 4096 * sizeof(int);
  const size_t trees_b = (sizeof(DevTree) * desc->max_episodes + 255) / 256 * 256;
  const size_t rows_b = ((size_t)desc->max_rows * 11 + SV_MAX_EP + 256) * sizeof(int);
  ctx->pinned_bytes = small_b + trees_b + rows_b + sizeof(ChunkState) + sizeof(EpState) * desc->max_episodes;
  ctx->cuda_err[0] = 0;
  if (cudaHostAlloc(&ctx->pinned, ctx->pinned_bytes, cudaHostAllocDefault) != cudaSuccess) {
    delete ctx;
    return SPECVLA_ERR_CUDA;
  }
  ctx->pin_small = static_cast<int *>(ctx->pinned);
  ctx->pin_trees = reinterpret_cast<DevTree *>(static_cast<char *>(ctx->pinned) + small_b);
  ctx->pin_rows = reinterpret_cast<int *>(static_cast<char *>(ctx->pinned) + small_b + trees_b);
  ctx->pin_chunk = reinterpret_cast<ChunkState *>(static_cast<char *>(ctx->pinned) + small_b + trees_b + rows_b);
  ctx->use_device_loop = true;
  ctx->loop_unavailable = false;
  ctx->cap_stream = nullptr;
  ctx->loop_graph = nullptr;
  ctx->loop_exec = nullptr;
  ctx->loop_launches_once = ctx->loop_launches_iter = 0;
  for (int i = 0; i < 4; i++) cudaEventCreate(&ctx->ev[i]);
  ctx->prof_mask = 0;
  ctx->phase = 0;
  ctx->prof_used = 0;
  for (int i = 0; i < SPECVLA_PROF_CLASSES; i++) { ctx->prof_ms[i] = 0; ctx->prof_n[i] = 0; ctx->prof_bytes[i] = 0; }
  // device-side initialisation: RoPE table, zeroed state
  const int half = desc->head_dim / 2, n = desc->max_seq * half;
  epi::rope_table_kernel<<<(n + 255) / 256, 256>>>(ctx->rope_tab, desc->max_seq, half, (double)desc->rope_theta);
  cudaMemsetAsync(ctx->st, 0, sizeof(EpState) * desc->max_episodes);
  cudaMemsetAsync(ctx->trees, 0, sizeof(DevTree) * desc->max_episodes);
  cudaMemsetAsync(ctx->err, 0, 32 * sizeof(int));
  cudaFuncSetAttribute(attn::tree_attention_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                       attn::smem_bytes<128>());
  cudaFuncSetAttribute(attn::tree_attention_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                       attn::smem_bytes<128>());
  cudaFuncSetAttribute(attn::tree_attention_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                       attn::smem_bytes<64>());
  cudaFuncSetAttribute(attn::tree_attention_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                       attn::smem_bytes<64>());
  if (cudaDeviceSynchronize() != cudaSuccess || !pack_ok) {
    cudaFreeHost(ctx->pinned);
    delete ctx;
    return pack_ok ? SPECVLA_ERR_CUDA : SPECVLA_ERR_CAPACITY;
  }
  *out = ctx;
  return SPECVLA_OK;
}

// Forgets the captured chunk loop (its launches were recorded under other settings).
static void drop_loop_graph(specvla_ctx *ctx) {
  if (ctx->loop_exec) cudaGraphExecDestroy(ctx->loop_exec);
  if (ctx->loop_graph) cudaGraphDestroy(ctx->loop_graph);
  ctx->loop_exec = nullptr;
  ctx->loop_graph = nullptr;
  ctx->loop_key.clear();
}

int specvla_destroy(specvla_ctx *ctx) {
  if (!ctx) return SPECVLA_ERR_INVALID_ARG;
  cudaDeviceSynchronize();
  drop_loop_graph(ctx);
  if (ctx->cap_stream) cudaStreamDestroy(ctx->cap_stream);
  for (int i = 0; i < 4; i++) cudaEventDestroy(ctx->ev[i]);
  for (cudaEvent_t e : ctx->prof_ev) cudaEventDestroy(e);
  cudaFreeHost(ctx->pinned);
  delete ctx;
  return SPECVLA_OK;
}

int specvla_set_option(specvla_ctx *ctx, int option, long long value) {
  if (!ctx) return SPECVLA_ERR_INVALID_ARG;
  drop_loop_graph(ctx);
  switch (option) {
    case SPECVLA_OPT_DEVICE_LOOP:
      ctx->use_device_loop = value != 0;
      ctx->loop_unavailable = false;
      break;
    case SPECVLA_OPT_PERSISTENT_FORWARD: ctx->use_pk = value != 0; break;
    case SPECVLA_OPT_DEPENDENT_LAUNCH: ctx->use_pdl = value != 0; break;
    case SPECVLA_OPT_L2_PREFETCH: ctx->use_l2_prefetch = value != 0; break;
    case SPECVLA_OPT_WAIT_LIMIT_NS:
      if (value < 1000) return SPECVLA_ERR_INVALID_ARG;
      ctx->wait_ns = (unsigned long long)value;
      break;
    default: return SPECVLA_ERR_INVALID_ARG;
  }
  return SPECVLA_OK;
}

int specvla_reset(specvla_ctx *ctx, int episode) {
  if (!ctx || episode < 0 || episode >= ctx->desc.max_episodes) return SPECVLA_ERR_INVALID_ARG;
  ctx->hP[episode] = -1;
  ctx->hPending[episode] = 0;
  return SPECVLA_OK;
}

static int prefill_enqueue(specvla_ctx *ctx, int n_ep, const int *episodes, const void *embeds,
                           const int *token_ids, const int *lens, float *logits_out, cudaStream_t st);

int specvla_prefill(specvla_ctx *ctx, int n_ep, const int *episodes, const void *embeds,
                    const int *token_ids, const int *lens, int *first_token_out, float *logits_out,
                    void *stream) {
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  TRY(prefill_enqueue(ctx, n_ep, episodes, embeds, token_ids, lens, logits_out, st));
  int *h_g = ctx->pin_small;
  CU(cudaMemcpyAsync(h_g, ctx->greedy, n_ep * sizeof(int), cudaMemcpyDeviceToHost, st));
  CU(cudaMemcpyAsync(h_g + 4000, ctx->err, sizeof(int), cudaMemcpyDeviceToHost, st));
  CU(cudaStreamSynchronize(st));
  prof_collect(ctx);
  if (h_g[4000] != 0) {
    for (int i = 0; i < n_ep; i++) ctx->hP[episodes[i]] = -1;
    return SPECVLA_ERR_TIMEOUT;
  }
  for (int i = 0; i < n_ep; i++)
    if (first_token_out) first_token_out[i] = h_g[i];
  return SPECVLA_OK;
}

// Validation, row tables and all device work of a prefill, without waiting for it. The host
// mirror is updated at once: prefix lengths do not depend on results.
static int prefill_enqueue(specvla_ctx *ctx, int n_ep, const int *episodes, const void *embeds,
                           const int *token_ids, const int *lens, float *logits_out, cudaStream_t st) {
  TRY(check_episodes(ctx, n_ep, episodes));
  if (!token_ids || !lens) return SPECVLA_ERR_INVALID_ARG;
  const specvla_model_desc &d = ctx->desc;
  EpArgs ea{};
  ea.n_ep = n_ep;
  int R = 0;
  for (int i = 0; i < n_ep; i++) {
    if (lens[i] < 1) return SPECVLA_ERR_INVALID_ARG;
    if (lens[i] + 1 > d.max_seq) return SPECVLA_ERR_CAPACITY;
    ea.eps[i] = episodes[i];
    ea.row0[i] = R;
    ea.nrows[i] = lens[i];
    R += lens[i];
    ea.aux[i] = R - 1;
  }
  if (R > d.max_rows) return SPECVLA_ERR_CAPACITY;
  for (int r = 0; r < R; r++) {
    if (token_ids[r] >= d.vocab) return SPECVLA_ERR_INVALID_ARG;
    if (token_ids[r] < 0 && !embeds) return SPECVLA_ERR_INVALID_ARG;
  }
  // row table on the host: causal rows, slot = position = index within the episode
  int *h = ctx->pin_rows;
  int *h_tok = h, *h_src = h + R, *h_ep = h + 2 * R, *h_pos = h + 3 * R, *h_nvis = h + 4 * R;
  for (int i = 0; i < n_ep; i++)
    for (int j = 0; j < lens[i]; j++) {
      const int r = ea.row0[i] + j;
      h_tok[r] = token_ids[r];
      h_src[r] = r;
      h_ep[r] = episodes[i];
      h_pos[r] = j;
      h_nvis[r] = j + 1;
    }
  const size_t rb = (size_t)R * sizeof(int);
  CU(cudaMemcpyAsync(ctx->rt.tok, h_tok, rb, cudaMemcpyHostToDevice, st));
  CU(cudaMemcpyAsync(ctx->rt.src, h_src, rb, cudaMemcpyHostToDevice, st));
  CU(cudaMemcpyAsync(ctx->rt.ep, h_ep, rb, cudaMemcpyHostToDevice, st));
  CU(cudaMemcpyAsync(ctx->rt.pos, h_pos, rb, cudaMemcpyHostToDevice, st));
  CU(cudaMemcpyAsync(ctx->rt.slot, h_pos, rb, cudaMemcpyHostToDevice, st));
  CU(cudaMemcpyAsync(ctx->rt.nvis, h_nvis, rb, cudaMemcpyHostToDevice, st));
  CU(cudaMemsetAsync(ctx->rt.tbase, 0, rb, st));
  CU(cudaMemsetAsync(ctx->rt.mask, 0, rb * 4, st));

  const bf16 *emb = static_cast<const bf16 *>(embeds);
  ctx->phase = 1;
  TRY(target_forward(ctx, R, ea, emb, st));

  // first token: LM head on each episode's last row
  int *h_last = h + 5 * R;
  for (int i = 0; i < n_ep; i++) h_last[i] = ea.aux[i];
  CU(cudaMemcpyAsync(ctx->lm_rows, h_last, n_ep * sizeof(int), cudaMemcpyHostToDevice, st));
  LAUNCH(epi::gather_rows_kernel, dim3(n_ep), dim3(256), (const bf16 *)ctx->xn.p, ctx->xn.plane,
         (const float *)ctx->ssq, ctx->nt, (const int *)ctx->lm_rows, d.d_model, ctx->lm_in.p, ctx->lm_in.plane,
         ctx->lm_ssq);
  TRY(lm_head_greedy(ctx, ctx->lm_in, ctx->lm_ssq, n_ep, logits_out, st));
  LAUNCH(tree::prefill_commit_kernel, dim3(n_ep), dim3(256), ea, ctx->st, (const int *)ctx->greedy,
         (const float *)ctx->x, (const float *)ctx->ssq, ctx->nt, ctx->final_norm, d.rms_eps, d.d_model,
         ctx->pend_feat);
  // the features of every prefix row, kept for inspection (the draft pass below reuses x)
  LAUNCH(epi::features_kernel, dim3(R), dim3(256), (const float *)ctx->x, (const float *)ctx->ssq, ctx->nt,
         ctx->final_norm, d.rms_eps, d.d_model, ctx->feat);
  ctx->feat_valid = true;

  // draft model over the shifted pairs (feature_i, input_{i+1}), i = 0 .. len-2
  if (ctx->has_draft) {
    int Rd = 0;
    // The draft model's row tables live in their own part of the pinned staging area: the copies
    // of the target's tables above may still be pending on the stream.
    int *hd = h + 5 * R + SV_MAX_EP;
    int *h_tok = hd, *h_src = hd + R, *h_ep = hd + 2 * R, *h_pos = hd + 3 * R, *h_nvis = hd + 4 * R;
    int *h_fs = hd + 5 * R;                // feature source rows
    EpArgs ed = ea;
    for (int i = 0; i < n_ep; i++) {
      ed.row0[i] = Rd;
      ed.nrows[i] = lens[i] - 1;
      for (int j = 0; j + 1 < lens[i]; j++) {
        const int r = Rd++;
        const int tr = ea.row0[i] + j;     // target row of f_j; the embedding comes from row tr+1
        h_tok[r] = token_ids[tr + 1];
        h_src[r] = tr + 1;
        h_ep[r] = episodes[i];
        h_pos[r] = j;
        h_nvis[r] = j + 1;
        h_fs[r] = tr;
      }
    }
    if (Rd > 0) {
      const size_t db = (size_t)Rd * sizeof(int);
      CU(cudaMemcpyAsync(ctx->rt.tok, h_tok, db, cudaMemcpyHostToDevice, st));
      CU(cudaMemcpyAsync(ctx->rt.src, h_src, db, cudaMemcpyHostToDevice, st));
      CU(cudaMemcpyAsync(ctx->rt.ep, h_ep, db, cudaMemcpyHostToDevice, st));
      CU(cudaMemcpyAsync(ctx->rt.pos, h_pos, db, cudaMemcpyHostToDevice, st));
      CU(cudaMemcpyAsync(ctx->rt.slot, h_pos, db, cudaMemcpyHostToDevice, st));
      CU(cudaMemcpyAsync(ctx->rt.nvis, h_nvis, db, cudaMemcpyHostToDevice, st));
      CU(cudaMemcpyAsync(ctx->feat_src, h_fs, db, cudaMemcpyHostToDevice, st));
      LAUNCH(tree::draft_input_kernel, dim3(Rd), dim3(256), ctx->rt, (const int *)ctx->feat_src,
             (const float *)ctx->feat, (const float *)nullptr, 0, (const float *)nullptr, 0.f, emb, ctx->embed,
             d.d_model, ctx->xin.p, ctx->xin.plane);
      TRY(draft_forward(ctx, Rd, ed, st));
    }
  }
  for (int i = 0; i < n_ep; i++) {
    ctx->hP[episodes[i]] = lens[i];
    ctx->hPending[episodes[i]] = 1;
    ctx->hTreeRows[episodes[i]] = 0;
  }
  return SPECVLA_OK;
}

static int draft_enqueue(specvla_ctx *ctx, const EpArgs &ea, int R, const specvla_tree_shape *shape, int n_nodes,
                         int n_tree_rows, cudaStream_t st);
static int draft_readback(specvla_ctx *ctx, int n_ep, const int *episodes, specvla_tree *trees_out, cudaStream_t st);

int specvla_draft_tree(specvla_ctx *ctx, int n_ep, const int *episodes, const specvla_tree_shape *shape,
                       specvla_tree *trees_out, void *stream) {
  TRY(check_episodes(ctx, n_ep, episodes));
  if (!ctx->has_draft) return SPECVLA_ERR_BAD_STATE;
  int n_nodes = 0, n_tree_rows = 0, n_draft_rows = 0;
  TRY(validate_shape(shape, &n_nodes, &n_tree_rows));
  for (int l = 1; l < shape->depth; l++) n_draft_rows += shape->expand[l];
  const specvla_model_desc &d = ctx->desc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  EpArgs ea{};
  ea.n_ep = n_ep;
  int R = 0;
  for (int i = 0; i < n_ep; i++) {
    const int e = episodes[i];
    if (ctx->hP[e] < 0 || ctx->hPending[e] < 1) return SPECVLA_ERR_BAD_STATE;
    // target cache: the rows verified; draft cache: one row per node expanded below the root
    if (ctx->hP[e] + n_tree_rows > d.max_seq || ctx->hP[e] + n_draft_rows > d.max_seq) return SPECVLA_ERR_CAPACITY;
    ea.eps[i] = e;
    // a fixed number of catch-up rows per episode: the pending pairs, the last one repeated (the
    // launch shapes then do not depend on the accepted length of the previous iteration)
    ea.row0[i] = R;
    ea.nrows[i] = SV_MAX_PENDING;
    R += SV_MAX_PENDING;
  }
  if (R > d.max_rows || n_ep * 16 > ctx->max_draft_rows) return SPECVLA_ERR_CAPACITY;
  TRY(draft_enqueue(ctx, ea, R, shape, n_nodes, n_tree_rows, st));
  for (int i = 0; i < n_ep; i++) {
    ctx->hPending[episodes[i]] = 0;
    ctx->hTreeRows[episodes[i]] = n_tree_rows;
  }
  return draft_readback(ctx, n_ep, episodes, trees_out, st);
}

// The device work of a draft call over the episodes of `ea` (SV_MAX_PENDING catch-up rows each):
// catch-up forward, then level by level head + tree growth + draft forward, then the re-ranking
// of a dynamic tree. Launch shapes depend only on the tree shape.
static int draft_enqueue(specvla_ctx *ctx, const EpArgs &ea, int R, const specvla_tree_shape *shape, int n_nodes,
                         int n_tree_rows, cudaStream_t st) {
  const specvla_model_desc &d = ctx->desc;
  const int n_ep = ea.n_ep;
  int lo, hi;
  argmax_range(ctx, &lo, &hi);

  ctx->phase = 2;
  // catch-up over the pending rows; the last row of each episode scores the root's children
  LAUNCH(tree::catchup_input_kernel, dim3(n_ep), dim3(256), ea, ctx->st, ctx->trees, ctx->rt,
         (const float *)ctx->pend_feat, ctx->embed, d.d_model, ctx->xin.p, ctx->xin.plane);
  TRY(draft_forward(ctx, R, ea, st));
  ctx->feat_valid = false;

  // Per level: the shared LM head over the rows just run (draft layer outputs as they are: no
  // norm, no row scale) with log-softmax + top-k, then one kernel that grows the tree and writes
  // the next level's input rows, then the draft model over those.
  int scored_rows = R;               // level 0 scores every catch-up row; only each episode's last one is used
  for (int l = 0; l < shape->depth; l++) {
    if (scored_rows > ctx->lgs_rows) return SPECVLA_ERR_CAPACITY;
    if (d.action_only && d.n_bins <= SV_TILE_ROWS) {
      // the action ids are one output tile: log-softmax and top-k are finished in the GEMM's epilogue
      TRY(gemm(ctx, ctx->xn, ctx->lm_head_act, scored_rows, epi_topk(ctx, d.n_bins, d.action_base), st,
               SPECVLA_PROF_LM_HEAD));
    } else if (d.action_only) {
      TRY(gemm(ctx, ctx->xn, ctx->lm_head_act, scored_rows,
               epi_plain(ctx->lgs, d.n_bins, d.n_bins, nullptr, ctx->nt), st, SPECVLA_PROF_LM_HEAD));
      LAUNCH(epi::logsoftmax_topk_kernel, dim3(scored_rows), dim3(epi::THREADS), (const float *)ctx->lgs, d.n_bins,
             0, d.n_bins, d.action_base, ctx->top_tok, ctx->top_lp);
    } else {
      TRY(lm_head(ctx, ctx->xn, nullptr, scored_rows, st));
      LAUNCH(epi::logsoftmax_topk_kernel, dim3(scored_rows), dim3(epi::THREADS), (const float *)ctx->lgs, d.vocab,
             lo, hi, 0, ctx->top_tok, ctx->top_lp);
    }
    const int cur = shape->expand[l];                            // parents scored per episode (level 0: the root)
    const int next = (l + 1 < shape->depth) ? shape->expand[l + 1] : 0;
    EpArgs la = ea;
    for (int i = 0; i < n_ep; i++) {
      la.row0[i] = (l == 0) ? ea.row0[i] + ea.nrows[i] - 1 : i * cur;
      la.aux[i] = i * next;
    }
    LAUNCH(tree::grow_input_kernel, dim3(n_ep), dim3(256), la, l, shape->branch[l], next, (const int *)ctx->top_tok,
           (const float *)ctx->top_lp, ctx->trees, (const EpState *)ctx->st, ctx->rt, (const float *)ctx->x,
           ctx->embed, d.d_model, ctx->xin.p, ctx->xin.plane);
    if (next == 0) break;
    const int Rn = n_ep * next;
    EpArgs ln = ea;
    for (int i = 0; i < n_ep; i++) {
      ln.row0[i] = i * next;
      ln.nrows[i] = next;
    }
    TRY(draft_forward(ctx, Rn, ln, st));
    scored_rows = Rn;
  }

  if (n_tree_rows < 1 + n_nodes)
    LAUNCH(tree::rerank_keep_kernel, dim3(n_ep), dim3(SV_MAX_CAND), ea, ctx->trees, n_tree_rows - 1);
  return SPECVLA_OK;
}

// Copies the device-resident trees of the call's episodes to the caller's host structs.
static int draft_readback(specvla_ctx *ctx, int n_ep, const int *episodes, specvla_tree *trees_out, cudaStream_t st) {
  if (trees_out) {
    DevTree *h = ctx->pin_trees;
    for (int i = 0; i < n_ep; i++)
      CU(cudaMemcpyAsync(&h[i], &ctx->trees[episodes[i]], sizeof(DevTree), cudaMemcpyDeviceToHost, st));
    CU(cudaStreamSynchronize(st));
    for (int i = 0; i < n_ep; i++) {
      specvla_tree &t = trees_out[i];
      if (!t.tokens || !t.parent || !t.depth) return SPECVLA_ERR_INVALID_ARG;
      t.n_rows = h[i].n_rows;
      for (int k = 0; k < h[i].n_rows; k++) {
        t.tokens[k] = h[i].tok[k];
        t.parent[k] = h[i].parent[k];
        t.depth[k] = h[i].depth[k];
        if (t.score) t.score[k] = h[i].score[k];
      }
    }
  }
  return SPECVLA_OK;
}

// Verification of the device-resident trees of the episodes in `ea` (rows already counted):
// forward, greedy tokens, acceptance, path selection, compaction, state update. Results stay
// on the device (out_m / out_tok / out_path); the caller reads them back.
static int verify_device_trees(specvla_ctx *ctx, const EpArgs &ea, int R, int r, float *logits_out,
                               cudaStream_t st) {
  const specvla_model_desc &d = ctx->desc;
  const int n_ep = ea.n_ep;
  ctx->phase = 4;
  LAUNCH(tree::build_verify_rows_kernel, dim3(n_ep), dim3(128), ea, ctx->trees, (const EpState *)ctx->st, ctx->rt);
  if (ctx->pk_ok && ctx->use_pk && n_ep == 1 && R <= pk::TN) {
    TRY(pk_target_forward(ctx, R, nullptr, logits_out, st));
  } else {
    TRY(target_forward(ctx, R, ea, nullptr, st));
    TRY(lm_head_greedy(ctx, ctx->xn, ctx->ssq, R, logits_out, st));
  }
  ctx->feat_valid = false;
  LAUNCH(tree::accept_select_kernel, dim3(n_ep), dim3(128), ea, ctx->trees, ctx->st, (const int *)ctx->greedy, r,
         d.action_base, d.n_bins, (const float *)ctx->x, ctx->last_ssq, ctx->last_nt, ctx->final_norm,
         d.rms_eps, d.d_model, ctx->pend_feat, ctx->out_m, ctx->out_tok, ctx->out_path);
  LAUNCH(tree::kv_compact_kernel, dim3(d.n_layers * 2, n_ep), dim3(256), ea, (const EpState *)ctx->st,
         (const int *)ctx->out_m, (const int *)ctx->out_path, ctx->kv_t, ctx->kv_t_ep_stride,
         ctx->kv_t_layer_stride, d.max_seq, ctx->hd);
  LAUNCH(tree::advance_state_kernel, dim3((n_ep + 63) / 64), dim3(64), ea, ctx->st, (const int *)ctx->out_m);
  return SPECVLA_OK;
}

// Reads m and the emitted tokens back, synchronises, and updates the host mirror.
static int finish_verify(specvla_ctx *ctx, const EpArgs &ea, int *accept_len_out, int *tokens_out,
                         cudaStream_t st) {
  const int n_ep = ea.n_ep, W = SV_MAX_DEPTH + 1;
  int *h = ctx->pin_small;
  CU(cudaMemcpyAsync(h, ctx->out_m, n_ep * sizeof(int), cudaMemcpyDeviceToHost, st));
  CU(cudaMemcpyAsync(h + SV_MAX_EP, ctx->out_tok, n_ep * W * sizeof(int), cudaMemcpyDeviceToHost, st));
  CU(cudaMemcpyAsync(h + 4000, ctx->err, sizeof(int), cudaMemcpyDeviceToHost, st));
  CU(cudaStreamSynchronize(st));
  prof_collect(ctx);
  if (h[4000] != 0) return SPECVLA_ERR_TIMEOUT;
  for (int i = 0; i < n_ep; i++) {
    const int e = ea.eps[i], m = h[i];
    if (m < 0 || m > SV_MAX_DEPTH) return SPECVLA_ERR_BAD_STATE;
    ctx->hP[e] += 1 + m;
    ctx->hPending[e] = m + 1;
    ctx->hTreeRows[e] = 0;
    if (accept_len_out) accept_len_out[i] = m;
    if (tokens_out)
      for (int k = 0; k < W; k++) tokens_out[i * W + k] = h[SV_MAX_EP + i * W + k];
  }
  return SPECVLA_OK;
}

// Validates the call's trees (caller-supplied, or the device-resident ones when trees == NULL),
// lays the episodes' rows out and uploads caller-supplied trees.
static int prepare_trees(specvla_ctx *ctx, int n_ep, const int *episodes, const specvla_tree *trees, EpArgs *ea_out,
                         int *rows_out, cudaStream_t st) {
  const specvla_model_desc &d = ctx->desc;
  EpArgs ea{};
  ea.n_ep = n_ep;
  int R = 0;
  for (int i = 0; i < n_ep; i++) {
    const int e = episodes[i];
    if (ctx->hP[e] < 0) return SPECVLA_ERR_BAD_STATE;
    int rows;
    if (trees) {
      TRY(validate_tree(trees[i]));
      rows = trees[i].n_rows;
      for (int k = 0; k < rows; k++)
        if (trees[i].tokens[k] >= d.vocab || (k > 0 && trees[i].tokens[k] < 0)) return SPECVLA_ERR_BAD_TREE;
    } else {
      rows = ctx->hTreeRows[e];
      if (rows < 1) return SPECVLA_ERR_BAD_STATE;
    }
    if (ctx->hP[e] + rows > d.max_seq) return SPECVLA_ERR_CAPACITY;
    ea.eps[i] = e;
    ea.row0[i] = R;
    ea.nrows[i] = rows;
    R += rows;
  }
  if (R > d.max_rows || R > ctx->max_lm_rows) return SPECVLA_ERR_CAPACITY;
  if (trees) {
    DevTree *h = ctx->pin_trees;
    for (int i = 0; i < n_ep; i++) {
      memset(&h[i], 0, sizeof(DevTree));
      h[i].n_rows = trees[i].n_rows;
      for (int k = 0; k < trees[i].n_rows; k++) {
        h[i].tok[k] = trees[i].tokens[k];
        h[i].parent[k] = trees[i].parent[k];
        h[i].depth[k] = trees[i].depth[k];
        h[i].score[k] = trees[i].score ? trees[i].score[k] : 0.f;
        h[i].drow[k] = -1;
      }
      CU(cudaMemcpyAsync(&ctx->trees[episodes[i]], &h[i], sizeof(DevTree), cudaMemcpyHostToDevice, st));
    }
  }
  *ea_out = ea;
  *rows_out = R;
  return SPECVLA_OK;
}

int specvla_verify_tree(specvla_ctx *ctx, int n_ep, const int *episodes, const specvla_tree *trees, int r,
                        int *accept_len_out, int *tokens_out, float *logits_out, void *stream) {
  TRY(check_episodes(ctx, n_ep, episodes));
  if (r < 0 || !accept_len_out || !tokens_out) return SPECVLA_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  EpArgs ea{};
  int R = 0;
  TRY(prepare_trees(ctx, n_ep, episodes, trees, &ea, &R, st));
  TRY(verify_device_trees(ctx, ea, R, r, logits_out, st));
  return finish_verify(ctx, ea, accept_len_out, tokens_out, st);
}

int specvla_score_tree(specvla_ctx *ctx, int n_ep, const int *episodes, const specvla_tree *trees,
                       int *greedy_out, void *stream) {
  TRY(check_episodes(ctx, n_ep, episodes));
  if (!trees || !greedy_out) return SPECVLA_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  EpArgs ea{};
  int R = 0;
  TRY(prepare_trees(ctx, n_ep, episodes, trees, &ea, &R, st));
  if (R > 4096 - 64) return SPECVLA_ERR_CAPACITY;                   // results come back through the small staging area
  ctx->phase = 4;
  LAUNCH(tree::build_verify_rows_kernel, dim3(n_ep), dim3(128), ea, ctx->trees, (const EpState *)ctx->st, ctx->rt);
  if (ctx->pk_ok && ctx->use_pk && n_ep == 1 && R <= pk::TN) {
    TRY(pk_target_forward(ctx, R, nullptr, nullptr, st));
  } else {
    TRY(target_forward(ctx, R, ea, nullptr, st));
    TRY(lm_head_greedy(ctx, ctx->xn, ctx->ssq, R, nullptr, st));
  }
  ctx->feat_valid = false;
  for (int i = 0; i < n_ep; i++) ctx->hTreeRows[episodes[i]] = ea.nrows[i];
  int *h = ctx->pin_small;
  CU(cudaMemcpyAsync(h, ctx->greedy, R * sizeof(int), cudaMemcpyDeviceToHost, st));
  CU(cudaMemcpyAsync(h + 4000, ctx->err, sizeof(int), cudaMemcpyDeviceToHost, st));
  CU(cudaStreamSynchronize(st));
  prof_collect(ctx);
  if (h[4000] != 0) return SPECVLA_ERR_TIMEOUT;
  for (int k = 0; k < R; k++) greedy_out[k] = h[k];
  return SPECVLA_OK;
}

// Row layout of a call whose episodes all bring `rows` rows.
static EpArgs uniform_rows(int n_ep, const int *episodes, int rows) {
  EpArgs ea{};
  ea.n_ep = n_ep;
  for (int i = 0; i < n_ep; i++) {
    ea.eps[i] = episodes[i];
    ea.row0[i] = i * rows;
    ea.nrows[i] = rows;
  }
  return ea;
}

// Captures the chunk loop of Algorithm 1 for these episodes, this tree shape and this r as a graph:
// a kernel that arms the loop, then a while node whose body drafts the trees, verifies them and
// appends the emitted tokens; the appending kernel decides whether the body runs again. Launch
// shapes inside the body depend only on the tree shape, everything else is read from device state.
static int build_loop_graph(specvla_ctx *ctx, int n_ep, const int *episodes, const specvla_tree_shape *shape,
                            int n_nodes, int n_tree_rows, int r) {
  drop_loop_graph(ctx);
  if (!ctx->cap_stream) CU(cudaStreamCreateWithFlags(&ctx->cap_stream, cudaStreamNonBlocking));
  cudaStream_t st = ctx->cap_stream;
  CU(cudaGraphCreate(&ctx->loop_graph, 0));
  cudaGraphConditionalHandle handle;
  CU(cudaGraphConditionalHandleCreate(&handle, ctx->loop_graph, 0, cudaGraphCondAssignDefault));
  cudaGraphNode_t arm_node, loop_node;
  {
    const ChunkState *cs = ctx->chunk;
    void *args[2] = {&cs, &handle};
    cudaKernelNodeParams kp = {};
    kp.func = (void *)tree::chunk_arm_kernel;
    kp.gridDim = dim3(1);
    kp.blockDim = dim3(1);
    kp.kernelParams = args;
    CU(cudaGraphAddKernelNode(&arm_node, ctx->loop_graph, nullptr, 0, &kp));
  }
  cudaGraphNodeParams np = {};
  np.type = cudaGraphNodeTypeConditional;
  np.conditional.handle = handle;
  np.conditional.type = cudaGraphCondTypeWhile;
  np.conditional.size = 1;
  CU(cudaGraphAddNode(&loop_node, ctx->loop_graph, &arm_node, 1, &np));
  cudaGraph_t body = np.conditional.phGraph_out[0];

  const long long before = ctx->launches;
  CU(cudaStreamBeginCaptureToGraph(st, body, nullptr, nullptr, 0, cudaStreamCaptureModeRelaxed));
  auto record = [&]() -> int {
    int rows = 1;
    if (shape->depth > 0) {
      const EpArgs ea = uniform_rows(n_ep, episodes, SV_MAX_PENDING);
      TRY(draft_enqueue(ctx, ea, n_ep * SV_MAX_PENDING, shape, n_nodes, n_tree_rows, st));
      rows = n_tree_rows;
    } else {
      const EpArgs ea = uniform_rows(n_ep, episodes, 1);
      LAUNCH(tree::root_only_tree_kernel, dim3(1), dim3(SV_MAX_EP), ea, ctx->trees);
    }
    const EpArgs ev = uniform_rows(n_ep, episodes, rows);
    TRY(verify_device_trees(ctx, ev, n_ep * rows, r, nullptr, st));
    LAUNCH(tree::chunk_append_kernel, dim3(1), dim3(SV_MAX_EP), ev, ctx->chunk, (const int *)ctx->out_m,
           (const int *)ctx->out_tok, (const int *)ctx->err, handle);
    return SPECVLA_OK;
  };
  const int rc = record();
  cudaGraph_t captured = nullptr;
  const cudaError_t ce = cudaStreamEndCapture(st, &captured);
  ctx->loop_launches_iter = ctx->launches - before;
  ctx->launches = before;
  ctx->loop_launches_once = 1;
  if (rc != SPECVLA_OK || ce != cudaSuccess) {
    cudaGetLastError();
    drop_loop_graph(ctx);
    if (rc != SPECVLA_OK) return rc;
    CU(ce);
  }
  const cudaError_t ie = cudaGraphInstantiate(&ctx->loop_exec, ctx->loop_graph, 0);
  if (ie != cudaSuccess) {
    ctx->loop_exec = nullptr;
    cudaGetLastError();
    drop_loop_graph(ctx);
    CU(ie);
  }
  return SPECVLA_OK;
}

static std::vector<int> loop_key_of(const specvla_ctx *ctx, int n_ep, const int *episodes,
                                    const specvla_tree_shape *shape, int r) {
  std::vector<int> k = {n_ep, r, shape->depth, shape->keep, (int)ctx->use_pdl, (int)ctx->use_l2_prefetch};
  for (int i = 0; i < n_ep; i++) k.push_back(episodes[i]);
  for (int l = 0; l < shape->depth; l++) {
    k.push_back(shape->branch[l]);
    k.push_back(shape->expand[l]);
  }
  return k;
}

// The chunk with its loop on the device: prefill, then ONE graph launch for all iterations, then
// one read-back of tokens, statistics and episode state.
static int generate_on_device(specvla_ctx *ctx, int n_ep, const int *episodes, const void *embeds,
                              const int *token_ids, const int *lens, const specvla_tree_shape *shape, int n_nodes,
                              int n_tree_rows, int r, int n_tokens, int *tokens_out, specvla_stats *stats,
                              cudaStream_t st) {
  float ms = 0.f;
  CU(cudaEventRecord(ctx->ev[0], st));
  TRY(prefill_enqueue(ctx, n_ep, episodes, embeds, token_ids, lens, nullptr, st));
  CU(cudaEventRecord(ctx->ev[1], st));
  ctx->phase = 4;
  const EpArgs ea = uniform_rows(n_ep, episodes, 1);
  LAUNCH(tree::chunk_begin_kernel, dim3(1), dim3(SV_MAX_EP), ea, ctx->chunk, (const int *)ctx->greedy, n_tokens,
         4 * n_tokens);
  CU(cudaGraphLaunch(ctx->loop_exec, st));
  CU(cudaEventRecord(ctx->ev[2], st));
  ChunkState *h = ctx->pin_chunk;
  EpState *hs = reinterpret_cast<EpState *>(h + 1);
  CU(cudaMemcpyAsync(h, ctx->chunk, sizeof(ChunkState), cudaMemcpyDeviceToHost, st));
  CU(cudaMemcpyAsync(hs, ctx->st, sizeof(EpState) * ctx->desc.max_episodes, cudaMemcpyDeviceToHost, st));
  CU(cudaMemcpyAsync(ctx->pin_small + 4000, ctx->err, sizeof(int), cudaMemcpyDeviceToHost, st));
  CU(cudaStreamSynchronize(st));
  ctx->launches += ctx->loop_launches_once + (long long)h->iterations * ctx->loop_launches_iter;
  ctx->feat_valid = false;
  bool complete = true;
  for (int i = 0; i < n_ep; i++) {
    const int e = episodes[i];
    ctx->hP[e] = hs[e].P;
    ctx->hPending[e] = hs[e].n_pending;
    ctx->hTreeRows[e] = 0;
    complete &= h->count[i] >= n_tokens;
  }
  if (ctx->pin_small[4000] != 0) {
    for (int i = 0; i < n_ep; i++) ctx->hP[episodes[i]] = -1;
    return SPECVLA_ERR_TIMEOUT;
  }
  if (!complete) return SPECVLA_ERR_BAD_STATE;
  for (int i = 0; i < n_ep; i++)
    for (int k = 0; k < n_tokens; k++) tokens_out[(size_t)i * n_tokens + k] = h->tokens[i][k];
  if (stats) {
    CU(cudaEventElapsedTime(&ms, ctx->ev[0], ctx->ev[1]));
    stats->ms_prefill = ms;
    CU(cudaEventElapsedTime(&ms, ctx->ev[1], ctx->ev[2]));
    stats->ms_loop = ms;
    stats->device_loop = 1;
    stats->iterations = h->iterations;
    stats->tokens_emitted = h->count[0];
    for (int k = 0; k < 16; k++) {
      stats->accept_len[k] = h->accept_len[k];
      stats->pos_iterations[k] = h->pos_iterations[k];
      stats->pos_accept_sum[k] = h->pos_accept_sum[k];
    }
  }
  return SPECVLA_OK;
}

int specvla_generate_action(specvla_ctx *ctx, int n_ep, const int *episodes, const void *embeds,
                            const int *token_ids, const int *lens, const specvla_tree_shape *shape, int r,
                            int n_tokens, int *tokens_out, float *actions_out, specvla_stats *stats,
                            void *stream) {
  TRY(check_episodes(ctx, n_ep, episodes));
  int n_nodes = 0, n_tree_rows = 0;
  TRY(validate_shape(shape, &n_nodes, &n_tree_rows));
  if (r < 0 || n_tokens < 1 || n_tokens > SV_MAX_CHUNK || !tokens_out || !lens) return SPECVLA_ERR_INVALID_ARG;
  if (shape->depth > 0 && !ctx->has_draft) return SPECVLA_ERR_BAD_STATE;
  const specvla_model_desc &d = ctx->desc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int W = SV_MAX_DEPTH + 1;
  if (stats) memset(stats, 0, sizeof(*stats));
  auto actions = [&]() {
    if (actions_out)
      for (int i = 0; i < n_ep * n_tokens; i++) {
        const int b = tokens_out[i] - d.action_base;
        actions_out[i] = (b >= 0 && b < d.n_bins) ? (-1.f + (2.f * b + 1.f) / d.n_bins) : NAN;
      }
  };

  // The loop runs on the device when its launches are the same every iteration (no depth pruning,
  // no per-GEMM timing, the per-GEMM forward) and the caches certainly hold every iteration's rows.
  bool on_device = ctx->use_device_loop && !shape->prune && ctx->prof_mask == 0 && !(ctx->pk_ok && ctx->use_pk);
  if (on_device) {
    const int rows = shape->depth > 0 ? n_tree_rows : 1;
    int draft_rows = 0;
    for (int l = 1; l < shape->depth; l++) draft_rows += shape->expand[l];
    for (int i = 0; i < n_ep; i++) {
      const int worst = lens[i] + n_tokens + shape->depth;      // committed positions never exceed this
      on_device &= lens[i] >= 1 && worst + rows <= d.max_seq && worst + draft_rows <= d.max_seq;
    }
    on_device &= n_ep * rows <= d.max_rows && n_ep * rows <= ctx->max_lm_rows &&
                 n_ep * SV_MAX_PENDING <= d.max_rows && n_ep * 16 <= ctx->max_draft_rows;
  }
  if (on_device && !ctx->loop_unavailable) {
    // the graph of this (episodes, shape, r, options) combination: captured on first use and kept. If the
    // driver refuses it, the host runs the loop from now on (specvla_stats.device_loop tells which ran).
    const std::vector<int> key = loop_key_of(ctx, n_ep, episodes, shape, r);
    if (!ctx->loop_exec || key != ctx->loop_key) {
      if (build_loop_graph(ctx, n_ep, episodes, shape, n_nodes, n_tree_rows, r) == SPECVLA_OK)
        ctx->loop_key = key;
      else {
        ctx->loop_unavailable = true;
        drop_loop_graph(ctx);
        cudaGetLastError();
      }
    }
  }
  if (on_device && !ctx->loop_unavailable) {
    TRY(generate_on_device(ctx, n_ep, episodes, embeds, token_ids, lens, shape, n_nodes, n_tree_rows, r, n_tokens,
                           tokens_out, stats, st));
    actions();
    return SPECVLA_OK;
  }

  std::vector<int> first(n_ep), count(n_ep, 0), m_out(n_ep), tok_out((size_t)n_ep * W);
  float ms = 0.f;
  CU(cudaEventRecord(ctx->ev[0], st));
  TRY(specvla_prefill(ctx, n_ep, episodes, embeds, token_ids, lens, first.data(), nullptr, stream));
  CU(cudaEventRecord(ctx->ev[1], st));
  CU(cudaEventSynchronize(ctx->ev[1]));
  CU(cudaEventElapsedTime(&ms, ctx->ev[0], ctx->ev[1]));
  if (stats) stats->ms_prefill = ms;
  for (int i = 0; i < n_ep; i++) {
    tokens_out[(size_t)i * n_tokens] = first[i];
    count[i] = 1;
  }
  int iterations = 0;
  for (;;) {
    bool done = true;
    for (int i = 0; i < n_ep; i++) done &= (count[i] >= n_tokens);
    if (done) break;
    EpArgs ea{};
    ea.n_ep = n_ep;
    int R = 0;
    CU(cudaEventRecord(ctx->ev[0], st));
    // levels to draft: all of them, or (prune) no more than the tokens still missing minus the
    // one the verification adds itself
    specvla_tree_shape now = *shape;
    if (shape->prune) {
      int missing = 0;
      for (int i = 0; i < n_ep; i++) missing = std::max(missing, n_tokens - count[i]);
      now.depth = std::min(shape->depth, missing - 1);
    }
    if (now.depth > 0) {
      TRY(specvla_draft_tree(ctx, n_ep, episodes, &now, nullptr, stream));
    } else {
      // no drafting: a one-row tree (the root) per episode = one autoregressive step
      const EpArgs one = uniform_rows(n_ep, episodes, 1);
      LAUNCH(tree::root_only_tree_kernel, dim3(1), dim3(SV_MAX_EP), one, ctx->trees);
      for (int i = 0; i < n_ep; i++) ctx->hTreeRows[episodes[i]] = 1;
    }
    CU(cudaEventRecord(ctx->ev[1], st));
    for (int i = 0; i < n_ep; i++) {
      const int e = episodes[i];
      if (ctx->hP[e] + ctx->hTreeRows[e] > d.max_seq) return SPECVLA_ERR_CAPACITY;
      ea.eps[i] = e;
      ea.row0[i] = R;
      ea.nrows[i] = ctx->hTreeRows[e];
      R += ctx->hTreeRows[e];
    }
    if (R > d.max_rows || R > ctx->max_lm_rows) return SPECVLA_ERR_CAPACITY;
    TRY(verify_device_trees(ctx, ea, R, r, nullptr, st));
    CU(cudaEventRecord(ctx->ev[2], st));
    TRY(finish_verify(ctx, ea, m_out.data(), tok_out.data(), st));
    if (stats) {
      CU(cudaEventElapsedTime(&ms, ctx->ev[0], ctx->ev[1]));
      stats->ms_draft += ms;
      CU(cudaEventElapsedTime(&ms, ctx->ev[1], ctx->ev[2]));
      stats->ms_verify += ms;
      if (iterations < 16) stats->accept_len[iterations] = m_out[0];
      const int pos = count[0] - 1;
      if (pos >= 0 && pos < 16) {
        stats->pos_iterations[pos]++;
        stats->pos_accept_sum[pos] += m_out[0];
      }
    }
    for (int i = 0; i < n_ep; i++)
      for (int k = 0; k <= m_out[i]; k++) {
        if (count[i] < n_tokens) tokens_out[(size_t)i * n_tokens + count[i]] = tok_out[(size_t)i * W + k];
        count[i]++;
      }
    iterations++;
    if (iterations > 4 * n_tokens) return SPECVLA_ERR_BAD_STATE;
  }
  if (stats) {
    stats->iterations = iterations;
    stats->tokens_emitted = count[0];
    stats->ms_loop = stats->ms_draft + stats->ms_verify;
  }
  actions();
  return SPECVLA_OK;
}

int specvla_read_buffer(specvla_ctx *ctx, int what, void *host_dst, size_t bytes, void *stream) {
  if (!ctx || !host_dst) return SPECVLA_ERR_INVALID_ARG;
  const specvla_model_desc &d = ctx->desc;
  const void *src = nullptr;
  size_t avail = 0;
  switch (what) {
    case SPECVLA_BUF_GREEDY: src = ctx->greedy; avail = (size_t)d.max_rows * sizeof(int); break;
    case SPECVLA_BUF_MARGIN: src = ctx->margin; avail = (size_t)d.max_rows * sizeof(float); break;
    case SPECVLA_BUF_FEATURES: {
      // after a verification the features exist only as residual + sums of squares
      if (!ctx->feat_valid) {
        if (ctx->last_rows < 1) return SPECVLA_ERR_BAD_STATE;
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        LAUNCH(epi::features_kernel, dim3(ctx->last_rows), dim3(256), (const float *)ctx->x,
               ctx->last_ssq, ctx->last_nt, ctx->final_norm, d.rms_eps, d.d_model, ctx->feat);
        ctx->feat_valid = true;
      }
      src = ctx->feat;
      avail = (size_t)d.max_rows * d.d_model * sizeof(float);
      break;
    }
    case SPECVLA_BUF_PATH: src = ctx->out_path; avail = (size_t)d.max_episodes * (SV_MAX_DEPTH + 1) * sizeof(int); break;
    case SPECVLA_BUF_DRAFT_TOPK_TOK: src = ctx->top_tok; avail = (size_t)ctx->max_draft_rows * SV_TOPK * sizeof(int); break;
    case SPECVLA_BUF_DRAFT_TOPK_LP: src = ctx->top_lp; avail = (size_t)ctx->max_draft_rows * SV_TOPK * sizeof(float); break;
    case SPECVLA_BUF_STATE: {
      if (bytes > (size_t)d.max_episodes * 4 * sizeof(int)) return SPECVLA_ERR_INVALID_ARG;
      cudaStream_t st = static_cast<cudaStream_t>(stream);
      CU(cudaMemcpy2DAsync(host_dst, 4 * sizeof(int), ctx->st, sizeof(EpState), 4 * sizeof(int),
                           bytes / (4 * sizeof(int)), cudaMemcpyDeviceToHost, st));
      CU(cudaStreamSynchronize(st));
      return SPECVLA_OK;
    }
    default: return SPECVLA_ERR_INVALID_ARG;
  }
  if (bytes > avail) return SPECVLA_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  CU(cudaMemcpyAsync(host_dst, src, bytes, cudaMemcpyDeviceToHost, st));
  CU(cudaStreamSynchronize(st));
  return SPECVLA_OK;
}

int specvla_read_kv(specvla_ctx *ctx, int draft, int episode, int layer, int which, int slot0, int n_slots,
                    void *host_dst, void *stream) {
  if (!ctx || !host_dst) return SPECVLA_ERR_INVALID_ARG;
  const specvla_model_desc &d = ctx->desc;
  if (episode < 0 || episode >= d.max_episodes || which < 0 || which > 1 || slot0 < 0 || n_slots < 1 ||
      slot0 + n_slots > d.max_seq)
    return SPECVLA_ERR_INVALID_ARG;
  if (draft ? (layer != 0) : (layer < 0 || layer >= d.n_layers)) return SPECVLA_ERR_INVALID_ARG;
  const float *base = draft ? ctx->kv_d + (size_t)episode * ctx->kv_d_ep_stride
                           : ctx->kv_t + (size_t)episode * ctx->kv_t_ep_stride + (size_t)layer * ctx->kv_t_layer_stride;
  base += ((size_t)which * d.max_seq + slot0) * ctx->hd;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  CU(cudaMemcpyAsync(host_dst, base, (size_t)n_slots * ctx->hd * sizeof(float), cudaMemcpyDeviceToHost, st));
  CU(cudaStreamSynchronize(st));
  return SPECVLA_OK;
}

// ------------------------------------------------------------------ stand-alone GEMM
// Resident-cluster counts per device ordinal, looked up once per device under a lock.
static std::mutex g_dev_mutex;
static gemm_ck::ClusterFit g_fit[64];
static bool g_fit_known[64];
static gemm_ck::ClusterFit cluster_fit_of_current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return gemm_ck::query_cluster_fit();
  std::lock_guard<std::mutex> lock(g_dev_mutex);
  if (!g_fit_known[dev]) {
    g_fit[dev] = gemm_ck::query_cluster_fit();
    g_fit_known[dev] = true;
  }
  return g_fit[dev];
}

// scratch layout: [status word, 1 KB | two bf16 limbs of X]
static const size_t GEMM_HDR = 1024;
static size_t gemm_limb_bytes(int T, int K) { return ((size_t)2 * T * K * sizeof(bf16) + 1023) / 1024 * 1024; }
size_t specvla_gemm_scratch_bytes(int T, int N, int K) {
  if (T < 1 || N < 4 || (N % 4) || K < 8) return 0;
  return GEMM_HDR + gemm_limb_bytes(T, K);
}

// Test hook of the next stand-alone GEMM call (specvla_gemm_fault_test): wait limit and the K
// block its producers withhold. Process-wide, consumed by one call.
static unsigned long long g_gemm_wait_ns = gemm_tc::WAIT_LIMIT_NS;
static int g_gemm_withhold = 0;

int specvla_gemm_fault_test(long long wait_limit_ns, int withhold_k_block) {
  if (wait_limit_ns < 1000 || withhold_k_block < -1) return SPECVLA_ERR_INVALID_ARG;
  g_gemm_wait_ns = (unsigned long long)wait_limit_ns;
  g_gemm_withhold = withhold_k_block + 1;
  return SPECVLA_OK;
}

size_t specvla_packed_weight_bytes(int N, int K) {
  if (N < 4 || (N % 4) || K < 8 || (K % 8)) return 0;
  return gemm_tc::packed_elems((N + SV_TILE_ROWS - 1) / SV_TILE_ROWS, K) * sizeof(bf16);
}

int specvla_pack_weights(const void *W, int N, int K, void *packed, size_t packed_bytes, void *stream) {
  if (!W || !packed || (reinterpret_cast<uintptr_t>(packed) % 1024) != 0) return SPECVLA_ERR_INVALID_ARG;
  const size_t need = specvla_packed_weight_bytes(N, K);
  if (need == 0) return SPECVLA_ERR_INVALID_ARG;
  if (packed_bytes < need) return SPECVLA_ERR_CAPACITY;
  const int tiles = (N + SV_TILE_ROWS - 1) / SV_TILE_ROWS, KB = (K + gemm_tc::BK - 1) / gemm_tc::BK;
  gemm_tc::pack_weights_kernel<<<148 * 8, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const bf16 *>(W), N, K, tiles, KB, 0, N / 2, static_cast<bf16 *>(packed));
  return cudaGetLastError() == cudaSuccess ? SPECVLA_OK : SPECVLA_ERR_CUDA;
}

// W (row-major) or Wp (repacked) is given, never both.
static int gemm_entry(const float *X, const void *W, const void *Wp, float *Y, int T, int N, int K, void *scratch,
                      size_t scratch_bytes, void *stream) {
  if (!X || (!W && !Wp) || !Y || !scratch || T < 1 || N < 4 || (N % 4) || K < 8 || (K % 8)) return SPECVLA_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(scratch) % 1024) != 0) return SPECVLA_ERR_INVALID_ARG;
  if (scratch_bytes < specvla_gemm_scratch_bytes(T, N, K)) return SPECVLA_ERR_CAPACITY;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char *base = static_cast<char *>(scratch);
  int *err = reinterpret_cast<int *>(base);
  bf16 *limbs = reinterpret_cast<bf16 *>(base + GEMM_HDR);
  const size_t nx = (size_t)T * K;
  // the status word starts at zero
  if (cudaMemsetAsync(base, 0, GEMM_HDR, st) != cudaSuccess) return SPECVLA_ERR_CUDA;
  epi::split_limbs_kernel<<<(unsigned)((nx + 255) / 256), 256, 0, st>>>(X, nx, limbs);
  CUtensorMap mw = {}, mx[2];
  if (W && !gemm_tc::make_w_map(&mw, static_cast<const bf16 *>(W), N, K)) return SPECVLA_ERR_CUDA;
  const int tiles = (N + SV_TILE_ROWS - 1) / SV_TILE_ROWS;
  const int KB = (K + gemm_tc::BK - 1) / gemm_tc::BK;
  gemm_tc::EpiArgs ea = {};
  ea.mode = gemm_tc::EPI_PLAIN;
  ea.N = N;
  ea.out = Y;
  ea.ldo = N;
  ea.wpacked = static_cast<const bf16 *>(Wp);
  ea.wait_ns = g_gemm_wait_ns;
  ea.withhold_unit = g_gemm_withhold;
  g_gemm_wait_ns = gemm_tc::WAIT_LIMIT_NS;           // the test hook holds for one call
  g_gemm_withhold = 0;
  const gemm_ck::ClusterFit fit = cluster_fit_of_current_device();
  const gemm_ck::RowPlan plan = gemm_ck::plan_rows(T, tiles, KB, fit);
  ea.row0 = 0;
  ea.T = T;
  ea.chunk_rows = plan.chunk_rows;
  ea.tn_chunk = plan.tn_chunk;
  ea.tn_tail = plan.tn_tail;
  if (!gemm_tc::make_x_map(&mx[0], limbs, nx, T, K, plan.tn_chunk) ||
      !gemm_tc::make_x_map(&mx[1], limbs, nx, T, K, plan.tn_tail))
    return SPECVLA_ERR_CUDA;
  if (gemm_ck::launch(mw, mx[0], mx[1], ea, tiles, KB, plan.S, err, st, false) != cudaSuccess)
    return SPECVLA_ERR_CUDA;
  return cudaGetLastError() == cudaSuccess ? SPECVLA_OK : SPECVLA_ERR_CUDA;
}

int specvla_gemm(const float *X, const void *W, float *Y, int T, int N, int K, void *scratch,
                 size_t scratch_bytes, void *stream) {
  if (!W) return SPECVLA_ERR_INVALID_ARG;
  return gemm_entry(X, W, nullptr, Y, T, N, K, scratch, scratch_bytes, stream);
}

int specvla_gemm_prepacked(const float *X, const void *Wpacked, float *Y, int T, int N, int K, void *scratch,
                           size_t scratch_bytes, void *stream) {
  if (!Wpacked) return SPECVLA_ERR_INVALID_ARG;
  return gemm_entry(X, nullptr, Wpacked, Y, T, N, K, scratch, scratch_bytes, stream);
}

// ------------------------------------------------------------------ GEMM without allocation
// Scratch of specvla_gemm_static: lives in the library image, one copy on every device that
// loads it, for as long as the process runs. The extra 1 KB lets the start be rounded up to
// the 1024-byte boundary specvla_gemm asks for.
static __device__ __align__(256) unsigned char g_static_scratch[SPECVLA_STATIC_SCRATCH_BYTES + 1024];
// Device address of g_static_scratch per device ordinal (0 = not looked up yet). In host code
// the symbol itself is only a stand-in; kernels must be given the address looked up here.
static void *g_static_scratch_addr[64];

int specvla_gemm_static(const float *X, const void *W, float *Y, int T, int N, int K, int wait, void *stream) {
  if (!X || !W || !Y || T < 1 || N < 4 || (N % 4) || K < 8 || (K % 8)) return SPECVLA_ERR_INVALID_ARG;
  const size_t need = specvla_gemm_scratch_bytes(T, N, K);
  if (need == 0) return SPECVLA_ERR_INVALID_ARG;
  if (need > (size_t)SPECVLA_STATIC_SCRATCH_BYTES) return SPECVLA_ERR_CAPACITY;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SPECVLA_ERR_CUDA;
  void *addr = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    if (!g_static_scratch_addr[dev]) {
      void *p = nullptr;
      if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return SPECVLA_ERR_CUDA;
      g_static_scratch_addr[dev] = p;
    }
    addr = g_static_scratch_addr[dev];
  }
  const uintptr_t base = (reinterpret_cast<uintptr_t>(addr) + 1023) & ~(uintptr_t)1023;
  void *scratch = reinterpret_cast<void *>(base);
  const int rc = specvla_gemm(X, W, Y, T, N, K, scratch, SPECVLA_STATIC_SCRATCH_BYTES, stream);
  if (rc != SPECVLA_OK || !wait) return rc;
  return specvla_gemm_status(scratch, stream);
}

int specvla_gemm_static_status(void *stream) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SPECVLA_ERR_CUDA;
  void *addr = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    addr = g_static_scratch_addr[dev];
  }
  if (!addr) return SPECVLA_ERR_BAD_STATE;            // specvla_gemm_static has not run on this device
  const uintptr_t base = (reinterpret_cast<uintptr_t>(addr) + 1023) & ~(uintptr_t)1023;
  return specvla_gemm_status(reinterpret_cast<const void *>(base), stream);
}

int specvla_gemm_status(const void *scratch, void *stream) {
  if (!scratch) return SPECVLA_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int word = 0;
  if (cudaMemcpyAsync(&word, scratch, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess)
    return SPECVLA_ERR_CUDA;
  return word == 0 ? SPECVLA_OK : SPECVLA_ERR_TIMEOUT;
}

int specvla_profile(specvla_ctx *ctx, int enable) {
  if (!ctx) return SPECVLA_ERR_INVALID_ARG;
  if (enable && ctx->prof_ev.empty()) {
    const int pairs = 1024;            // GEMM launches between two synchronisations
    ctx->prof_ev.resize(2 * pairs);
    ctx->prof_cls.resize(pairs);
    for (auto &e : ctx->prof_ev)
      if (cudaEventCreate(&e) != cudaSuccess) return SPECVLA_ERR_CUDA;
  }
  if (enable) {
    for (int i = 0; i < SPECVLA_PROF_CLASSES; i++) { ctx->prof_ms[i] = 0; ctx->prof_n[i] = 0; ctx->prof_bytes[i] = 0; }
    ctx->prof_used = 0;
  }
  ctx->prof_mask = enable & 7;
  return SPECVLA_OK;
}

int specvla_profile_read(const specvla_ctx *ctx, double *ms_out, long long *launches_out, double *bytes_out) {
  if (!ctx || !ms_out || !launches_out || !bytes_out) return SPECVLA_ERR_INVALID_ARG;
  for (int i = 0; i < SPECVLA_PROF_CLASSES; i++) {
    ms_out[i] = ctx->prof_ms[i];
    launches_out[i] = ctx->prof_n[i];
    bytes_out[i] = ctx->prof_bytes[i];
  }
  return SPECVLA_OK;
}

const char *specvla_strerror(int code) {
  switch (code) {
    case SPECVLA_OK: return "ok";
    case SPECVLA_ERR_INVALID_ARG: return "invalid argument";
    case SPECVLA_ERR_CAPACITY: return "capacity exceeded (rows, slots, episodes or workspace)";
    case SPECVLA_ERR_BAD_TREE: return "malformed draft tree";
    case SPECVLA_ERR_BAD_STATE: return "episode state does not allow this call";
    case SPECVLA_ERR_CUDA: return "CUDA error";
    case SPECVLA_ERR_TIMEOUT: return "device-side wait timed out";
    case SPECVLA_ERR_UNSUPPORTED_ARCH: return "device is not sm_100";
    default: return "unknown error";
  }
}

const char *specvla_last_cuda_error(const specvla_ctx *ctx) { return ctx ? ctx->cuda_err : ""; }
long long specvla_kernel_launches(const specvla_ctx *ctx) { return ctx ? ctx->launches : 0; }

}  // extern "C"
