/*
 * specvla.h - C ABI of the B200 (sm_100a) tree-verification path of Spec-VLA.
 *
 * The library runs the hot path of Spec-VLA decoding (Algorithm 1, Appendix B) for an
 * OpenVLA-style Llama decoder: prefill, the Eagle-style one-layer draft model M_D (Eq. 2,
 * Eq. 5), one verification forward of M_V over all draft-tree rows under a tree mask
 * (Section 3.2 / 4.1), greedy argmax (Eq. 1), relaxed acceptance (Eq. 4, Section 4.3),
 * longest-accepted-path selection and KV-cache compaction.
 *
 * Conventions
 *  - Every function returns 0 on success or a negative SPECVLA_ERR_* code; nothing throws.
 *  - "device" pointers are CUDA device memory of the current device; "host" pointers are
 *    ordinary host memory. The caller owns every buffer it passes in; the library owns
 *    only the host-side context object and a few KB of pinned staging memory.
 *  - All weights are bfloat16, row-major [out_features, in_features]; RMSNorm gains are
 *    float32. Activations are float32 between kernels and enter the bf16 tensor-core GEMMs
 *    as two bf16 limbs (hi + lo); the KV caches are float32. With single-limb bf16
 *    activations or a bf16 cache the logits of the 32-layer model drift by 0.1-0.2 from an
 *    exact forward, ten times the 2e-2 this library is held to. The workspace (KV caches, activations and the library's
 *    repacked copy of every weight matrix, about the size of the weights themselves) is one
 *    device buffer allocated by the caller, at least specvla_workspace_bytes() long, 1024-byte aligned;
 *    it must outlive the context and must not be touched while a call is in flight.
 *  - specvla_create reads every weight MATRIX once (wqkv, wo, wgu, wd, lm_head and the draft
 *    model's fc / wqkv / wo / wgu / wd) and keeps its own repacked copy in the workspace; once it has
 *    returned, those matrices may be freed or overwritten: two copies of a 7B model need not stay
 *    resident. The embedding table and the norm gain vectors are read in place by every call and
 *    must outlive the context.
 *  - Work is enqueued on `stream` (a cudaStream_t passed as void*). Calls that return
 *    values through host pointers synchronise that stream before returning.
 *  - One context per host thread; calls on one context must not overlap.
 *  - There is no CPU fallback: creation fails with SPECVLA_ERR_UNSUPPORTED_ARCH unless the
 *    current device is compute capability 10.x.
 */
#ifndef SPECVLA_H
#define SPECVLA_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SPECVLA_OK                     0
#define SPECVLA_ERR_INVALID_ARG       -1   /* NULL pointer, size out of range */
#define SPECVLA_ERR_CAPACITY          -2   /* rows / slots / episodes exceed the context's capacity */
#define SPECVLA_ERR_BAD_TREE          -3   /* parent[i] >= i, wrong depth, parent[0] != -1 ... */
#define SPECVLA_ERR_BAD_STATE         -4   /* episode not prefilled, nothing pending ... */
#define SPECVLA_ERR_CUDA              -5   /* a CUDA call failed; see specvla_last_cuda_error */
#define SPECVLA_ERR_TIMEOUT           -6   /* a bounded device-side wait gave up */
#define SPECVLA_ERR_UNSUPPORTED_ARCH  -7   /* not an sm_100 device */

#define SPECVLA_MAX_TREE_ROWS   128        /* rows of one verification tree, root included */
#define SPECVLA_MAX_DEPTH       8          /* deepest draft level */
#define SPECVLA_MAX_BRANCH      8          /* children per expanded node */

typedef struct specvla_ctx specvla_ctx;

/* Model and capacity description (Section 4.1: Llama decoder; Section 4.3: 256 action bins). */
typedef struct {
  int n_layers, d_model, n_heads, head_dim, d_ffn, vocab;
  int action_base;      /* token id of action bin 0; bins are ids action_base .. action_base+n_bins-1 */
  int n_bins;           /* 256 */
  float rms_eps;        /* 1e-6 */
  float rope_theta;     /* 1e4 */
  int max_seq;          /* KV slots per episode: committed positions + rows of the tree in flight */
  int max_episodes;     /* episodes with their own KV caches */
  int max_rows;         /* rows of one forward call summed over its episodes (prefill sets this) */
  int action_only;      /* 1: greedy argmax and draft top-k range over the action ids only */
  int weight_bits;      /* 0 or 16: the target's matrices are streamed as given (bf16). 8: quantised
                         * target (Appendix C): at creation the four matrices of every target layer and
                         * the LM head are quantised to int8, per output row, symmetric: scale =
                         * max|w| / 127 (1 for a zero row), code = round-half-even(w / scale) in
                         * [-127, 127], both in float32; the kernels stream the codes (half the bytes),
                         * expand them to bf16 in shared memory and apply the scale to the accumulator.
                         * Embedding, norms and the draft model (with the original LM-head rows it
                         * scores with) are not quantised. The paper does not specify its scheme. */
} specvla_model_desc;

/* Target (verification) model weights. Per-layer members are HOST arrays of n_layers DEVICE
 * pointers. wqkv = [Wq; Wk; Wv] stacked [3*H*dh, d]; wgu = [Wgate; Wup] stacked [2F, d]. */
typedef struct {
  const void *embed;              /* bf16 [vocab, d] */
  const void *lm_head;            /* bf16 [vocab, d] */
  const float *final_norm;        /* f32 [d] */
  const void *const *wqkv;        /* bf16 [3*H*dh, d] */
  const void *const *wo;          /* bf16 [d, H*dh] */
  const void *const *wgu;         /* bf16 [2F, d] */
  const void *const *wd;          /* bf16 [d, F] */
  const float *const *norm1;      /* f32 [d] */
  const float *const *norm2;      /* f32 [d] */
} specvla_weights;

/* Draft model M_D (Eq. 2): fc over [feature ; token embedding] + one decoder layer. It shares
 * the target's embedding and LM head. May be NULL at creation when only caller-supplied
 * trees are verified. */
typedef struct {
  const void *fc;                 /* bf16 [d, 2d] */
  const void *wqkv, *wo, *wgu, *wd;
  const float *norm1, *norm2;
} specvla_draft_weights;

/* Static-size draft tree (Section 4.1, Eagle-2 style): level l (0-based) expands the
 * expand[l] best nodes of level l-1 (expand[0] must be 1: the root) into branch[l] <= 8 children
 * each. depth = 0 means no drafting: every iteration is one plain autoregressive step. */
typedef struct {
  int depth;
  int branch[SPECVLA_MAX_DEPTH];
  int expand[SPECVLA_MAX_DEPTH];
  int prune;   /* read by specvla_generate_action only. 0: every iteration drafts `depth` levels and
                * the chunk is clipped at the end (Algorithm 1 as printed). 1: an iteration whose
                * episodes still miss at most k tokens drafts min(depth, k - 1) levels (the
                * verification adds one token itself, deeper nodes could only be clipped), and
                * none at all when k = 1. Same tokens at r = 0; at r > 0 the accepted path may be
                * another equally valid one. */
  int keep;    /* 0: every drafted node is verified (at most 16 nodes per level, 127 in all).
                * N > 0: dynamic tree (Section 4.1: the Eagle-2 strategy; Section 5.1: 50 nodes,
                * top-8): levels may hold up to 64 nodes (16 of them expanded), 319 in all; after the
                * last level the nodes are ranked by cumulative log-probability (ties to the lower
                * node index) and only the N best (N <= 127) are kept and verified. */
} specvla_tree_shape;

/* One draft tree in HOST memory. Row 0 is the root (the last emitted token, not yet in the
 * target's cache): parent[0] = -1, depth[0] = 0, parent[i] < i, depth[i] = depth[parent[i]]+1.
 * tokens[0] may be -1 to take the root token from the episode's state. score may be NULL. */
typedef struct {
  int n_rows;
  int *tokens;
  int *parent;
  int *depth;
  float *score;
} specvla_tree;

typedef struct {
  int iterations;                 /* draft+verify iterations run (max over episodes) */
  int tokens_emitted;             /* before clipping, first episode */
  int accept_len[16];             /* accepted draft tokens m of the first 16 iterations, first episode */
  float ms_prefill, ms_draft, ms_verify;   /* device time, CUDA events; draft and verify are measured
                                            * apart only when the loop runs on the host (0 otherwise) */
  /* Accepted draft tokens by the position at which an iteration starts (Table 3): an iteration
   * that begins when k + 1 tokens of the chunk exist starts at position k (0 .. n_tokens - 2).
   * Iterations counted and accepted lengths m summed per position, first episode; positions past
   * 15 go uncounted. mean = pos_accept_sum[k] / pos_iterations[k]. */
  int pos_iterations[16];
  int pos_accept_sum[16];
  float ms_loop;                  /* device time of all draft+verify iterations together */
  int device_loop;                /* 1: the iterations ran as one graph launch (SPECVLA_OPT_DEVICE_LOOP) */
} specvla_stats;

/* Bytes of device workspace a context of this description needs. 0 on invalid description. */
size_t specvla_workspace_bytes(const specvla_model_desc *desc);

/* Creates a context. `workspace` (device) is carved into KV caches and activations and
 * zero-initialised where needed on `stream`-0. draft may be NULL. */
int specvla_create(const specvla_model_desc *desc, const specvla_weights *target,
                   const specvla_draft_weights *draft, void *workspace, size_t workspace_bytes,
                   specvla_ctx **out);
int specvla_destroy(specvla_ctx *ctx);

/* Execution options of a context (each defaults to the setting measured fastest on B200; they
 * exist for A/B measurements and tests, and change no result beyond rounding order):
 *   SPECVLA_OPT_PERSISTENT_FORWARD  1: forwards of one episode and at most 32 rows (the batch-1
 *       verification step of Algorithm 1, an autoregressive step) run as ONE cooperative kernel
 *       whose weight stream continues across all GEMMs of all layers; 0 (default): one launch per
 *       GEMM. The persistent kernel needs two grid-wide barriers per GEMM at about 2 us each and
 *       measures 25 % slower than the per-GEMM path on the 7B-shaped model.
 *   SPECVLA_OPT_DEPENDENT_LAUNCH    1: kernels of the per-GEMM path are launched with programmatic
 *       stream serialisation (a GEMM streams weights while its predecessor drains).
 *   SPECVLA_OPT_L2_PREFETCH         1: a GEMM of the per-GEMM path prefetches the head of the next
 *       matrix into L2.
 *   SPECVLA_OPT_WAIT_LIMIT_NS       limit of every device-side wait of the persistent kernel in
 *       nanoseconds (default 2e9); a wait that runs out makes the call return SPECVLA_ERR_TIMEOUT.
 *   SPECVLA_OPT_DEVICE_LOOP         1 (default): specvla_generate_action runs the iterations of
 *       Algorithm 1 as ONE launch of a CUDA graph whose while node repeats draft tree, verification
 *       and the appending of the emitted tokens until the chunk is complete; the host reads tokens,
 *       statistics and episode state back once. Applies when every iteration launches the same
 *       kernels (shape.prune = 0, no per-GEMM timing, per-GEMM forward) and the caches hold
 *       prefix + n_tokens + depth + tree rows; otherwise, with 0, and when the driver refuses the
 *       graph (remembered until this option is set again), the host runs the loop and reads the
 *       accepted length back every iteration. Same tokens either way; specvla_stats.device_loop
 *       says which loop ran. */
#define SPECVLA_OPT_PERSISTENT_FORWARD 1
#define SPECVLA_OPT_DEPENDENT_LAUNCH   2
#define SPECVLA_OPT_L2_PREFETCH        3
#define SPECVLA_OPT_WAIT_LIMIT_NS      4
#define SPECVLA_OPT_DEVICE_LOOP        5
int specvla_set_option(specvla_ctx *ctx, int option, long long value);

/* Forgets an episode's state (its caches are simply overwritten by the next prefill). */
int specvla_reset(specvla_ctx *ctx, int episode);

/* Prefill (Section 4.1): causal forward of M_V over each episode's prefix, the first token
 * a_1 = greedy token of the last row (Eq. 1), and M_D over the shifted (feature_i, input_{i+1})
 * pairs to fill the draft cache.
 *   episodes   host [n_ep]        distinct episode ids in [0, max_episodes)
 *   embeds     device bf16 [sum(lens), d]  row used where token_ids[row] < 0
 *   token_ids  host [sum(lens)]   >= 0: the row is that id's embedding
 *   lens       host [n_ep]        prefix length of each episode, >= 1
 *   first_token_out  host [n_ep], may be NULL
 *   logits_out device f32 [n_ep, vocab] logits of each episode's last row, may be NULL */
int specvla_prefill(specvla_ctx *ctx, int n_ep, const int *episodes, const void *embeds,
                    const int *token_ids, const int *lens, int *first_token_out,
                    float *logits_out, void *stream);

/* Draft phase (Algorithm 1, inner loop; Eq. 2): runs M_D on the rows pending since the last
 * commit, then grows the static-size tree level by level from M_D's top-k tokens. The tree
 * stays on the device for the next specvla_verify_tree(trees = NULL).
 *   trees_out  host [n_ep], may be NULL; each entry's arrays must hold 1 + sum(branch*expand)
 *              rows; n_rows is written. */
int specvla_draft_tree(specvla_ctx *ctx, int n_ep, const int *episodes,
                       const specvla_tree_shape *shape, specvla_tree *trees_out, void *stream);

/* Verification (Algorithm 1; Eq. 3 / Eq. 4): one forward of M_V over all tree rows (row i at
 * position P + depth[i], attending the committed cache, its ancestors and itself), greedy
 * token per row, acceptance of node i when |bin(tokens[i]) - bin(g[parent[i]])| <= r and its
 * parent is accepted (ids outside the action bins must match exactly), choice of the deepest
 * accepted node (ties: lowest row), compaction of the accepted rows' K/V next to the root,
 * and set-up of the next iteration's state.
 *   trees          host [n_ep] caller-supplied trees, or NULL to verify the trees left by
 *                  specvla_draft_tree
 *   r              relaxation threshold >= 0 (0 = strict matching)
 *   accept_len_out host [n_ep]: m, the number of accepted draft tokens
 *   tokens_out     host [n_ep][SPECVLA_MAX_DEPTH+1]: the m accepted draft tokens, then the
 *                  target's token after them (m + 1 valid entries per episode)
 *   logits_out     device f32 [total rows, vocab], may be NULL (debug / parity) */
int specvla_verify_tree(specvla_ctx *ctx, int n_ep, const int *episodes,
                        const specvla_tree *trees, int r, int *accept_len_out, int *tokens_out,
                        float *logits_out, void *stream);

/* The verification forward alone (Eq. 1 over every tree row): greedy token of M_V after each row
 * of caller-supplied trees, WITHOUT acceptance, compaction or any change of the episodes' state
 * (the tree rows' K/V land in cache slots beyond the committed ones and are overwritten by the next
 * forward). For harnesses that need the target's opinion on partial trees, e.g. to plant drafts
 * around its greedy bins. The uploaded trees replace the device-resident ones.
 *   greedy_out  host [total rows], rows in call order */
int specvla_score_tree(specvla_ctx *ctx, int n_ep, const int *episodes, const specvla_tree *trees,
                       int *greedy_out, void *stream);

/* Whole chunk (Algorithm 1): prefill, then draft -> verify -> accept until every episode has
 * n_tokens tokens; the result is clipped to n_tokens. One stream synchronisation per
 * iteration (the accepted length decides termination).
 *   tokens_out   host [n_ep][n_tokens]
 *   actions_out  host [n_ep][n_tokens] bin centres in [-1, 1] (256 uniform bins), may be NULL
 *   stats        may be NULL */
int specvla_generate_action(specvla_ctx *ctx, int n_ep, const int *episodes, const void *embeds,
                            const int *token_ids, const int *lens,
                            const specvla_tree_shape *shape, int r, int n_tokens,
                            int *tokens_out, float *actions_out, specvla_stats *stats,
                            void *stream);

/* Inspection (tests, parity): copies internal results of the last call to HOST memory and
 * synchronises. `what`: */
#define SPECVLA_BUF_GREEDY      1   /* int   [rows]      greedy token per row of the last verify */
#define SPECVLA_BUF_MARGIN      2   /* float [rows]      top-1 minus top-2 logit per row */
#define SPECVLA_BUF_FEATURES    3   /* float [rows, d]   final-norm outputs of the last target forward */
#define SPECVLA_BUF_PATH        4   /* int   [n_ep][SPECVLA_MAX_DEPTH+1] accepted path rows */
#define SPECVLA_BUF_STATE       5   /* int   [max_episodes][4]: P, Pd, root, n_pending */
#define SPECVLA_BUF_DRAFT_TOPK_TOK 6 /* int   [rows][8]   top tokens of the last draft level */
#define SPECVLA_BUF_DRAFT_TOPK_LP  7 /* float [rows][8]   their log-probabilities */
int specvla_read_buffer(specvla_ctx *ctx, int what, void *host_dst, size_t bytes, void *stream);

/* Copies KV-cache rows [slot0, slot0+n_slots) of one layer to host as f32 [n_slots, H*dh].
 * which: 0 = K, 1 = V; draft: 0 = target cache, 1 = draft cache (layer must be 0). */
int specvla_read_kv(specvla_ctx *ctx, int draft, int episode, int layer, int which, int slot0,
                    int n_slots, void *host_dst, void *stream);

/* Y[T, N] (f32, device) = X[T, K] (f32, device) * W[N, K]^T (bf16, device): the library's
 * weight-streaming GEMM exposed for kernel-level parity tests and roofline measurement. As in
 * the decoder, X enters the tensor cores as two bf16 limbs (hi + lo), so the result carries
 * about 16 mantissa bits of X. K % 8 == 0, N % 4 == 0.
 * scratch: device, 1024-byte aligned, at least specvla_gemm_scratch_bytes(T, N, K) bytes (a
 * status word and the two bf16 limbs of X). */
size_t specvla_gemm_scratch_bytes(int T, int N, int K);
int specvla_gemm(const float *X, const void *W, float *Y, int T, int N, int K,
                 void *scratch, size_t scratch_bytes, void *stream);
/* The same product with W given in the library's streaming order (Section 3.1: the cost of
 * decoding is the parameter stream; the decoder keeps every matrix in this form): one contiguous,
 * pre-swizzled 32 KB block per (256-row tile, 64-column K block), read by plain bulk copies.
 * specvla_pack_weights writes that form of W [N, K] into `packed` (device, 1024-byte aligned, at
 * least specvla_packed_weight_bytes(N, K) bytes; 0 is returned for an invalid shape); pack once,
 * multiply many times. Scratch and status as for specvla_gemm. */
size_t specvla_packed_weight_bytes(int N, int K);
int specvla_pack_weights(const void *W, int N, int K, void *packed, size_t packed_bytes, void *stream);
int specvla_gemm_prepacked(const float *X, const void *Wpacked, float *Y, int T, int N, int K,
                           void *scratch, size_t scratch_bytes, void *stream);

/* Failure-handling test hook (no counterpart in the paper). Every device-side wait of the GEMM
 * is bounded; this call makes the NEXT specvla_gemm / specvla_gemm_prepacked call of the process
 * run with the given wait limit (nanoseconds, >= 1000) and has the producer of every CTA withhold
 * the K block of that index within its K range (-1: none), so that the waits for it run out: the
 * kernel records the failure in the scratch's status word, lets its copies land, frees its
 * tensor memory and returns, and specvla_gemm_status reports SPECVLA_ERR_TIMEOUT. Nothing faults
 * or hangs; the context stays usable. Both settings are cleared by that one call. */
int specvla_gemm_fault_test(long long wait_limit_ns, int withhold_k_block);

/* Synchronises `stream` and reports whether the specvla_gemm calls that used `scratch` ran
 * to completion: SPECVLA_ERR_TIMEOUT if a bounded device-side wait gave up (Y is then
 * undefined), SPECVLA_ERR_CUDA if the stream is in error, else SPECVLA_OK. */
int specvla_gemm_status(const void *scratch, void *stream);

/* specvla_gemm for callers that cannot allocate device memory: code running inside a CUDA
 * stream capture or a real-time control loop, a plug-in handed only its input and output
 * buffers, a process whose memory pool is owned by another component. (The paper has no
 * counterpart of this call; it exists for such callers only.) The scratch that specvla_gemm
 * takes from its caller is here a fixed array of SPECVLA_STATIC_SCRATCH_BYTES inside the
 * library image; every GPU that loads the library holds that much memory until the process
 * exits. X, W and Y are the caller's, exactly as for specvla_gemm.
 *  - Returns SPECVLA_ERR_CAPACITY, before touching the GPU, when
 *    specvla_gemm_scratch_bytes(T, N, K) exceeds SPECVLA_STATIC_SCRATCH_BYTES.
 *  - Calls no cudaMalloc / cudaFree or any other allocating routine.
 *  - The first call on each device looks the array's device address up (the device must be
 *    current); make that first call outside any stream capture.
 *  - All calls on a device share the one array, which still holds the previous call's
 *    contents; the call clears what it needs cleared. Two calls that may overlap on the GPU
 *    (different streams, no dependency) race on it: serialise them.
 *  - wait != 0: synchronises `stream` and returns SPECVLA_ERR_TIMEOUT if a bounded
 *    device-side wait gave up (as specvla_gemm_status); wait == 0: asynchronous (ask
 *    specvla_gemm_static_status afterwards). Inside a stream capture wait must be 0. */
#define SPECVLA_STATIC_SCRATCH_BYTES (16u << 20)
int specvla_gemm_static(const float *X, const void *W, float *Y, int T, int N, int K, int wait,
                        void *stream);
/* specvla_gemm_status for the built-in scratch of the current device: synchronises `stream`. */
int specvla_gemm_static_status(void *stream);

/* Per-GEMM device timing (measurement aid; Section 3.1 attributes the latency to the
 * parameter stream, which these GEMMs are). `phases` is a bit mask: 1 = prefill, 2 = draft,
 * 4 = verification; 0 switches timing off. While a phase is enabled, every weight-streaming
 * GEMM launch of that phase is bracketed by CUDA events on the call's stream (up to 1024
 * launches between two synchronising calls; later ones go untimed); the sums are folded in at
 * each synchronisation. Classes index the weight matrix streamed. A non-zero mask resets
 * the sums. */
#define SPECVLA_PROF_QKV      0
#define SPECVLA_PROF_O        1
#define SPECVLA_PROF_GATE_UP  2
#define SPECVLA_PROF_DOWN     3
#define SPECVLA_PROF_LM_HEAD  4
#define SPECVLA_PROF_FC       5
#define SPECVLA_PROF_CLASSES  6
int specvla_profile(specvla_ctx *ctx, int phases);
/* ms_out / launches_out / bytes_out: host arrays of SPECVLA_PROF_CLASSES entries: summed
 * device time, timed launches and weight bytes streamed (N*K*2 per launch) per class. */
int specvla_profile_read(const specvla_ctx *ctx, double *ms_out, long long *launches_out,
                         double *bytes_out);

const char *specvla_strerror(int code);
/* Text of the last CUDA error seen by this context (empty string if none). */
const char *specvla_last_cuda_error(const specvla_ctx *ctx);
/* Number of kernels launched by this context since creation (for launch accounting). */
long long specvla_kernel_launches(const specvla_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* SPECVLA_H */
