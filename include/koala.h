/*
 * koala.h -- C ABI of the draft-then-verify step of speculative decoding with K-layer draft heads
 * (KOALA, arXiv 2408.08146), for NVIDIA B200 (sm_100a).
 *
 * One iteration of the method (Section 2.2 of the paper: draft with M_d, Eq. 2; verify all drafts
 * in one forward of the target M_q, Eq. 3; accept a prefix) is
 *
 *     for p in 0..D-1:  koala_draft(ctx, p);  koala_expand_tree(ctx, p);     (EAGLE-style head)
 *     koala_draft(ctx, 0);  koala_expand_tree(ctx, 0);                        (Medusa-style heads)
 *     koala_verify(ctx, NULL);
 *     koala_accept(ctx, forced_len, out_tokens, out_len);
 *
 * Conventions
 *   - Every call returns KOALA_OK (0) or a KOALA_E_* code; nothing throws, aborts or prints.
 *     koala_last_error() gives a text for the last non-zero code of that context.
 *   - The library allocates NO device memory.  Weights, KV caches, seq_len and one workspace are
 *     DEVICE pointers owned by the caller, who keeps them alive until koala_destroy().  The
 *     koala_ctx itself is host memory owned by the library.
 *   - All work is enqueued on the CUDA stream given to koala_init() and is asynchronous; no call
 *     synchronises the stream or the device.  Arguments are validated on the host before anything
 *     is enqueued.  Device-side problems (a bounded wait that ran out) are recorded in a device
 *     status word that koala_poll() copies back.
 *   - Matrices are row-major [out][in].  "dtype" is the storage type of weights, KV caches and
 *     matrix-multiply operands (fp32 or bf16); accumulation, softmax, norms and the residual
 *     stream are fp32 in both cases.  With bf16 the activations entering a matrix multiply are
 *     kept as two bf16 values (the rounded value and its rounding residual), so only the weights
 *     and the KV cache are rounded to bf16.
 *   - KV caches are laid out [layer][B][n_heads][S_max][head_dim].
 *   - A tree has at most N nodes per sequence, node 0 the root, parent index < child index.
 *     Node u of sequence b is row b*N + u of every per-node buffer.
 */
#ifndef KOALA_H_
#define KOALA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define KOALA_OK 0
#define KOALA_E_INVALID 1     /* bad argument or configuration */
#define KOALA_E_UNSUPPORTED 2 /* valid but not implemented for this shape / dtype */
#define KOALA_E_CAPACITY 3    /* workspace too small, or S + N could exceed S_max */
#define KOALA_E_STATE 4       /* call out of order */
#define KOALA_E_CUDA 5        /* a CUDA runtime / driver call failed */
#define KOALA_E_TIMEOUT 6     /* a bounded device-side wait ran out (reported by koala_poll) */

#define KOALA_FP32 0
#define KOALA_BF16 1

#define KOALA_EAGLE 0  /* autoregressive head: Embedding -> Linear -> K x Decoder Layer -> LM Head */
#define KOALA_MEDUSA 1 /* non-autoregressive heads: K x ResBlock -> (shared) Linear             */

/* flags */
#define KOALA_F_NO_TENSOR_CORES 1u /* run every GEMM on the CUDA-core path (debugging / A-B checks) */
#define KOALA_F_NO_PDL 2u          /* launch kernels without programmatic dependent launch         */
#define KOALA_F_LAYER_KERNEL 4u    /* run each decoder layer's matrix multiplies and the row-wise steps
                                      between them in one persistent launch where that applies (bf16,
                                      at most 128 rows per forward) instead of one kernel per step;
                                      same results up to summation order, measured slower on B200    */

#define KOALA_MAX_TREE 128 /* largest N: ancestor sets are 128-bit masks */
#define KOALA_MAX_TOPK 16
#define KOALA_LAYER_TENSORS 9 /* attn_norm, wq, wk, wv, wo, ffn_norm, w_gate, w_up, w_down */

typedef struct koala_ctx koala_ctx;

typedef struct {
  uint32_t struct_size; /* sizeof(koala_config) */
  int32_t dtype;        /* KOALA_FP32 | KOALA_BF16 */
  int32_t head_kind;    /* KOALA_EAGLE | KOALA_MEDUSA */
  int32_t L, H, n_heads, head_dim, F, V; /* target: layers, hidden, heads, head dim, FFN, vocab */
  float rms_eps, rope_base;
  int32_t K;              /* draft-head layers (Section 3.1) */
  int32_t n_medusa_heads; /* MEDUSA only */
  int32_t D;              /* draft levels below the root (MEDUSA: = n_medusa_heads) */
  int32_t topk;           /* expansion width k, <= KOALA_MAX_TOPK */
  int32_t N;              /* tree nodes per sequence including the root, <= KOALA_MAX_TREE */
  int32_t B;              /* sequences per step */
  int32_t S_max;          /* KV capacity per sequence (tokens) */
  uint32_t flags;
} koala_config;

typedef struct {
  /* device pointers, dtype storage */
  const void *embed;      /* [V][H] */
  const void *lm_head;    /* [V][H] shared by the target and every draft head */
  const void *final_norm; /* [H] */
  const void *const *layer_w; /* HOST array of L*9 device pointers, order of KOALA_LAYER_TENSORS */
  const void *fc_w;           /* EAGLE: [H][2H] over [hidden ; embedding] */
  const void *fc_b;           /* EAGLE: [H] */
  const void *const *draft_layer_w; /* EAGLE: HOST array of K*9 device pointers */
  const void *const *res_w;         /* MEDUSA: HOST array of n_medusa_heads*K device pointers [H][H] */
  const void *const *res_b;         /* MEDUSA: same, [H] */
  /* MEDUSA, optional: HOST array of n_medusa_heads device pointers [V][H], the Linear that ends
   * each head in Section 3.1's drawing of the Medusa head.  NULL: every head uses lm_head. */
  const void *const *medusa_lm;
  /* MEDUSA static topology, HOST arrays of N entries (node 0: parent -1, level 0) */
  const int32_t *static_parent, *static_level, *static_rank;
} koala_weights;

typedef struct {
  void *target_k, *target_v; /* [L][B][n_heads][S_max][head_dim], dtype storage */
  void *draft_k, *draft_v;   /* EAGLE: [K][B][n_heads][S_max][head_dim]; else NULL */
  int32_t *seq_len;          /* [B] device: tokens held by the target cache; caller initialises */
  void *workspace;           /* device, 256-byte aligned */
  size_t workspace_bytes;    /* >= koala_workspace_bytes(cfg) */
} koala_state;

/* A tree supplied by the caller instead of the drafted one: prompt ingestion (a chain), plain
 * autoregressive decoding (one node), tests with planted paths.  Device arrays. */
typedef struct {
  const int32_t *tok;     /* [B][stride] */
  const int32_t *parent;  /* [B][stride], root -1, parent < child */
  const int32_t *n_nodes; /* [B], 1 <= n_nodes[b] <= n_max */
  int32_t stride;
  int32_t n_max;          /* host-known bound on n_nodes, <= N */
} koala_tree;

/* Device pointers into the workspace, for inspection and for overwriting state between calls. */
typedef struct {
  float *draft_logits;   /* [draft_rows][V] logits of the last draft pass (row order: see koala_draft) */
  float *draft_feat;     /* [B][topk][H] features predicted by the last draft pass (EAGLE) /
                            [n_medusa_heads][B][H] head features (MEDUSA) */
  int32_t *topk_tok;     /* [draft_rows][topk] */
  float *topk_logp;      /* [draft_rows][topk] natural-log probabilities */
  int32_t *cand_tok;     /* [B][pool] candidate pool of the dynamic tree */
  int32_t *cand_parent;  /* [B][pool] parent candidate id, -1 = root */
  float *cand_score;     /* [B][pool] cumulative log-probability */
  int32_t *frontier;     /* [B][topk] candidate ids expanded by the next pass */
  int32_t *tree_tok;     /* [B][N] */
  int32_t *tree_parent;  /* [B][N] */
  int32_t *tree_level;   /* [B][N] */
  float *tree_score;     /* [B][N] (dynamic trees) */
  int32_t *tree_n;       /* [B] nodes in use */
  float *verify_logits;  /* [B*N][V] */
  float *verify_hid;     /* [B*N][H] output of the target's final norm */
  int32_t *verify_tgt;   /* [B*N] greedy token after each node */
  int32_t *root_tok;     /* [B] token the next tree is rooted at */
  float *pend_hid;       /* [B][N][H] hidden states of the positions accepted last */
  int32_t *pend_tok;     /* [B][N] tokens accepted last, after the root */
  int32_t *n_pend;       /* [B] how many */
  int32_t *acc_path;     /* [B][N] node indices of the accepted path */
  int32_t pool;          /* candidates per sequence: topk + (D-1)*topk*topk */
  int32_t draft_rows;    /* rows of draft_logits currently meaningful */
} koala_buffer_table;

/* Bytes of workspace koala_init() needs for this configuration (0 if the configuration is invalid). */
size_t koala_workspace_bytes(const koala_config *cfg);

/* Section 2.2 set-up: validates shapes, carves the workspace, encodes the TMA descriptors of the
 * weight matrices.  `cuda_stream` is a cudaStream_t (NULL = the default stream).  All pointer
 * tables are copied; the device memory they point to is borrowed.  *out receives the context. */
int koala_init(const koala_config *cfg, const koala_weights *w, const koala_state *st,
               void *cuda_stream, koala_ctx **out);

/* Draft pass (Eq. 2: d_1..d_t <- M_d(x | x_<=n)).
 * EAGLE-style (Section 3.1): z = W_fc [feature ; E[token]] + b_fc, K decoder layers with the
 *   head's own KV cache, logits = LM_head(z).  Pass 0 runs over the positions accepted by the
 *   last koala_accept (hidden state at position j paired with the token at j+1; the last row
 *   pairs with root_tok) and yields one logits row per sequence (row b).  Pass p >= 1 runs over
 *   the topk frontier candidates of level p (parent's predicted feature, own token) and yields
 *   rows b*topk + i.  0 <= pass < D, in order.
 * Medusa-style (Section 3.1): head i applies K residual blocks x <- x + SiLU(W x + b) to the
 *   last accepted hidden state and the shared LM head; rows i*B + b.  pass must be 0. */
int koala_draft(koala_ctx *ctx, int pass);

/* Top-k tree expansion after koala_draft(ctx, pass): per row the k most likely tokens (ties:
 * smaller id) and their log-probabilities; dynamic trees add them to the candidate pool with
 * cumulative scores, pick the next frontier (pass < D-1) or, at pass D-1, keep the N-1 best
 * candidates and emit tree_tok / tree_parent / tree_level ordered by (level, parent, rank);
 * static trees fill node (level d, rank r) with the r-th token of head d-1. */
int koala_expand_tree(koala_ctx *ctx, int pass);

/* Verification (Eq. 3): one forward of the target over all tree nodes of all sequences.  Node u
 * sits at position S + level(u), its K/V at cache slot S + u, and attends to the S cached tokens,
 * its ancestors and itself.  Fills verify_logits, verify_hid, verify_tgt.  `tree` NULL = the
 * tree built by koala_expand_tree. */
int koala_verify(koala_ctx *ctx, const koala_tree *tree);

/* Greedy acceptance (Section 4.1: a draft token is kept only if it equals the target's greedy
 * token) of the longest matching root path, then KV compaction: the accepted nodes' K/V move to
 * slots S..S+l-1 of every target layer and seq_len += l.  out_tokens[b][0..l-1] = the path's
 * tokens after the root, then the bonus token (which becomes root_tok); out_len[b] = l
 * (1 <= l <= nodes on the longest path).  forced_len (device [B] or NULL): f > 0 makes the walk
 * step to the lowest-numbered child where no child matches, until the path has f nodes or ends.
 * out_tokens: device [B][out_stride]; out_len: device [B]; out_stride >= longest possible path. */
int koala_accept(koala_ctx *ctx, const int32_t *forced_len, int32_t *out_tokens, int32_t out_stride,
                 int32_t *out_len);

/* Speculative sampling on chain drafts (Section 2.2, the paragraph after Eq. 3; the paper's
 * non-greedy runs use temperature 1).  Only for an EAGLE-style head with topk = 1, i.e. a chain of
 * D drafted tokens; the paper gives no rule for a tree.  All random numbers are the caller's.
 *
 * koala_set_sampling(ctx, u_draft): while u_draft (DEVICE [B][D], uniforms in [0, 1)) is non-null,
 * koala_expand_tree(p) draws sequence b's level-(p+1) token from d = softmax(draft logits) with
 * u_draft[b][p] (inverse CDF in token-id order: the smallest id whose cumulative probability
 * exceeds u) instead of taking the arg-max, and keeps d.  NULL switches back to greedy drafts.
 * The array is read when the kernels run: keep it alive and unchanged until then.
 *
 * koala_accept_sampled replaces koala_accept after koala_verify(ctx, NULL) of such a chain: with
 * q_i = softmax of the target's logits at chain node i-1, drafted token i is accepted iff
 * u_accept[b][i-1] * d_i(x_i) < q_i(x_i) (probability min(1, q_i/d_i)); the first rejected
 * position is redrawn from max(0, q_f - d_f) normalised, later tokens are dropped; if all D are
 * accepted one more token is drawn from q_{D+1}.  Both draws use u_bonus[b] and the same inverse
 * CDF.  u_accept: DEVICE [B][D]; u_bonus: DEVICE [B].  Outputs, cache compaction, counters and the
 * next root as in koala_accept (the extra token takes the place of the bonus token).  A tree that
 * is not a chain sets the device status to KOALA_E_INVALID. */
int koala_set_sampling(koala_ctx *ctx, const float *u_draft);
int koala_accept_sampled(koala_ctx *ctx, const float *u_accept, const float *u_bonus, int32_t *out_tokens,
                         int32_t out_stride, int32_t *out_len);

/* Position-wise acceptance counters, accumulated by every koala_accept since koala_init or the
 * last reset (Section 4.1, metrics: the acceptance rate n-alpha, i.e. the accuracy on the n-th
 * drafted token, which the paper measures with chain drafts).  Reading used here, for any tree:
 * along the walked path, position n (n = 1 is the root's child) was offered if the walk reached
 * depth n-1 and that node has a child, and hit if the walk went on to depth n; n-alpha =
 * hits[n-1] / trials[n-1].  With chain trees this is the paper's metric.  Forced steps count as
 * hits, so reset after ingesting a prompt.  hits / trials: HOST arrays of n_max <= 128 entries;
 * the call copies on the context's stream and waits for it; reset != 0 clears the counters. */
int koala_accept_stats(koala_ctx *ctx, uint64_t *hits, uint64_t *trials, int32_t n_max, int32_t reset);


int koala_buffers(koala_ctx *ctx, koala_buffer_table *out);

/* Run-time options.  KOALA_OPT_EXPAND_MODE splits koala_expand_tree for step-by-step checks:
 * 0 = top-k then tree bookkeeping (default); 1 = top-k only (the call may be repeated);
 * 2 = tree bookkeeping only, from whatever topk_tok / topk_logp hold (e.g. values the caller wrote). */
#define KOALA_OPT_EXPAND_MODE 1
/* KOALA_OPT_TIMING: 1 = bracket every matrix-multiply and attention launch with CUDA events on the
 * context's stream (this removes the launch overlap between neighbouring kernels, so it is for
 * per-kernel measurement, not for timing whole steps) and reset the totals; 0 = off (default). */
#define KOALA_OPT_TIMING 2
int koala_set_option(koala_ctx *ctx, int option, int value);

/* Totals since KOALA_OPT_TIMING was switched on, per kernel class.  Synchronises the stream. */
#define KOALA_CLS_GEMM_TC 0   /* tensor-core (tcgen05) matrix multiplies */
#define KOALA_CLS_GEMM_SIMT 1 /* CUDA-core matrix multiplies */
#define KOALA_CLS_ATTENTION 2 /* tree-masked attention */
typedef struct {
  float ms[3];           /* summed device time between the bracketing events */
  uint64_t bytes[3];     /* algorithmic bytes: weight bytes of each multiply; K/V bytes of each attention */
  int32_t launches[3];
} koala_timing;
int koala_timing_read(koala_ctx *ctx, koala_timing *out);

/* Non-blocking: *done = 1 if everything enqueued so far has finished; *device_status = the
 * device status word as of the last finished poll copy (0 = fine, else a KOALA_E_* code). */
int koala_poll(koala_ctx *ctx, int *done, int *device_status);

const char *koala_last_error(const koala_ctx *ctx);
void koala_destroy(koala_ctx *ctx);

/* Stand-alone matrix multiply used by the steps above, exported for unit tests and kernel timing:
 * Y[M][N_out] (fp32, row stride ldy) = X[M][K_in] (bf16) * W[N_out][K_in]^T (bf16), on the
 * tensor-core path (use_tensor_cores != 0; needs K_in % 64 == 0) or the CUDA-core path.
 * `scratch` (device, >= koala_gemm_scratch_bytes) holds split-K partial sums.  On the tensor-core
 * path X (and X_lo) must be allocated with koala_gemm_x_rows(M, X_lo != NULL) rows: whole token
 * tiles (the extra rows are read, their results discarded); X, X_lo and W must be 16-byte aligned.
 * split_k 0 = automatic.  Asynchronous on `cuda_stream`. */
int koala_gemm_x_rows(int M, int has_lo);
size_t koala_gemm_scratch_bytes(int M, int N_out, int K_in);
int koala_gemm_bf16(const void *X, const void *X_lo /* optional residual of X, same shape; NULL = none */,
                    const void *W, float *Y, int ldy, int M, int N_out, int K_in,
                    void *scratch, size_t scratch_bytes, int use_tensor_cores, int split_k,
                    void *cuda_stream, int *device_status /* device int, may be NULL */);

/* The paper has no counterpart for this entry point; it is a packaging variant of koala_gemm_bf16.
 *
 * Same product, Y[M][N_out] = (X [+ X_lo]) * W^T on the tensor-core path, for callers that cannot
 * provide (or allocate) a scratch buffer: a serving loop whose device memory is fixed at start-up,
 * a plug-in that a host framework hands only inputs and outputs, code running close to the
 * device's memory limit.  The split-K partial sums go to a fixed 8 MiB array inside the library's
 * device image (koala_gemm_static_scratch_bytes(); every GPU that loads the library holds it until
 * the process exits).  Nothing is allocated or freed on the device, by this call or under it.
 *   - split_k: 1..8 = that many partial sums per output, which must fit in the array
 *     (split_k * M * N_out * 4 bytes <= 8 MiB, else KOALA_E_CAPACITY; split_k 1 needs no scratch at
 *     all and is accepted at any size); 0 = automatic: the factor the multiply would choose by
 *     itself, lowered until it fits (never an error for size); above 8: KOALA_E_INVALID.
 *     K_in % 64 == 0, X rows as koala_gemm_x_rows.
 *   - The first call on each device (with that device current) looks up the array's device address
 *     and prepares the kernel for that device.  With CUDA's lazy module loading that look-up is also
 *     the moment the 8 MiB get their device memory, so make this first call at start-up, before
 *     memory is tight, and outside any stream capture.
 *   - All calls on a device share the one array and it keeps the previous call's contents (none of
 *     which is read before it is overwritten).  Two calls whose kernels may overlap on the GPU
 *     (different streams, no ordering between them) race on it: order them on one stream or with
 *     events. */
size_t koala_gemm_static_scratch_bytes(void);
int koala_gemm_bf16_static(const void *X, const void *X_lo, const void *W, float *Y, int ldy, int M,
                           int N_out, int K_in, int split_k, void *cuda_stream,
                           int *device_status /* device int, may be NULL */);

#ifdef __cplusplus
}
#endif
#endif /* KOALA_H_ */
