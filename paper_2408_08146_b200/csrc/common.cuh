// Shared device helpers and the internal launcher interface of libkoala.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <mutex>

typedef __nv_bfloat16 bf16;

namespace koala {

// ---------------------------------------------------------------------------------------------
// scalar conversions
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }

// Programmatic dependent launch: every kernel lets its successor start early and waits for its
// predecessor before touching anything the predecessor may have written.  Both are no-ops when
// the launch did not opt in.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

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

// A matrix given as the sum of partial matrices `stride` floats apart (split-K results).
// Classic split-K: every column has `n` partials.  Stream-K (sk_ctas > 0): column c belongs to
// weight tile c / 128 (c / 256 with sk_wide), whose K-blocks were dealt to the CTAs owning units
// [tile * sk_kb, (tile + 1) * sk_kb); it has one partial per such CTA, in slots 0, 1, ...
struct SplitIn {
  const float *p;
  int n;
  size_t stride;
  int ld;
  unsigned sk_ctas, sk_units, sk_kb;
  unsigned sk_wide;        // stream-K: weight tiles of 128 << sk_wide columns
  // several matrices side by side whose widths are not whole tiles (0 = not the case): the columns
  // at which the second and third matrix start, and the tiles before them
  unsigned sk_m0, sk_m1, sk_t0, sk_t1;
  __device__ __forceinline__ int count(int c) const {
    if (sk_ctas == 0) return n;
    const unsigned sh = 7u + sk_wide, uc = (unsigned)c;
    unsigned tile = uc >> sh;
    if (sk_m0 != 0 && uc >= sk_m0) tile = uc < sk_m1 ? sk_t0 + ((uc - sk_m0) >> sh) : sk_t1 + ((uc - sk_m1) >> sh);
    const unsigned u0 = tile * sk_kb;
    const unsigned first = ((u0 + 1u) * sk_ctas - 1u) / sk_units;
    const unsigned last = ((u0 + sk_kb) * sk_ctas - 1u) / sk_units;
    return (int)(last - first) + 1;
  }
  __device__ __forceinline__ float at(int r, int c) const {
    const float *q = p + (size_t)r * ld + c;
    const int k = count(c);
    float v = q[0];
    for (int s = 1; s < k; ++s) v += q[(size_t)s * stride];
    return v;
  }
};

// Deferred RMSNorm scale of a GEMM input: the producer wrote x * gain (not normalised) and, per
// row, `n` partial sums of squares; the consumer of the GEMM's output multiplies by
// rsqrt(sum / H + eps).  n == 0: nothing pending (the input was already normalised).
struct RowScale {
  const float *sumsq;   // [rows][n]
  int n;
  float inv_h, eps;
  __device__ __forceinline__ float of(int r) const {
    if (n == 0) return 1.f;
    float s = 0.f;
    for (int i = 0; i < n; ++i) s += sumsq[(size_t)r * n + i];
    return rsqrtf(s * inv_h + eps);
  }
};

// Per-row plan of one forward over R rows (rows_per_seq consecutive rows per sequence).
struct RowPlan {
  const int32_t *pos;     // [R] RoPE position
  const int32_t *slot;    // [R] KV slot to write, -1 = row not in use
  const uint64_t *mask;   // [R][2] visibility over the slots ctx_len .. ctx_len+127
  const int32_t *ctx_len; // [B] slots 0..ctx_len-1 are visible to every row of the sequence
  const int32_t *kv_len;  // [B] slots in use after this forward's writes
  const float2 *rope;     // [R][head_dim/2] (cos, sin)
};

extern unsigned long long g_launches;   // kernels launched by the library (defined in koala_api.cu)

template <typename... KArgs, typename... Args>
static inline cudaError_t launch_k(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                   cudaStream_t stream, bool pdl, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = pdl ? 1 : 0;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  ++g_launches;
  return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

// A kernel's dynamic shared-memory limit is an attribute of the function on ONE device: raise it
// once per device the library is used on (one object per kernel, kept by its launcher).
struct SmemOptIn {
  std::mutex mu;
  size_t done[64] = {};
  cudaError_t ensure(const void *fn, size_t smem) {
    if (smem <= 48 * 1024) return cudaSuccess;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu);
    if (smem <= done[dev]) return cudaSuccess;
    e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess) done[dev] = smem;
    return e;
  }
};

// ---------------------------------------------------------------------------------------------
// launcher interface (one per kernel family); every launcher is asynchronous on `st`
// ---------------------------------------------------------------------------------------------
struct Launch {
  cudaStream_t st;
  bool pdl;
};

// A matrix-multiply operand in the storage dtype.  For bf16 `lo` holds the rounding residual of
// `hi` (operand value = hi + lo); for fp32, or when the residual is not kept, lo is null.
struct Operand {
  void *hi;
  void *lo;
};

struct GemmMats {         // up to three weight matrices sharing K_in, outputs concatenated
  const void *W[3];
  int n_out[3];
  int n;
};

// ops.cu
cudaError_t embed_norm(Launch L, int dtype, const int32_t *tok, const void *E, const void *g,
                       float *x, Operand xn, int R, int H, int V, float eps);
// mode 0: v = x + sum(P); 1: v = sum(P) + bias; 2: v = x + SiLU(sum(P) + bias).  x <- v;
// n = g ? rmsnorm(v) * g : v;  xn <- T(n) if xn;  out_f32 <- n if out_f32.
cudaError_t row_epilogue(Launch L, int dtype, int mode, float *x, SplitIn P, const void *bias,
                         const void *g, Operand xn, float *out_f32, int R, int H, float eps);
cudaError_t eagle_concat(Launch L, int dtype, const float *feat_src, const int32_t *row_src,
                         const int32_t *row_tok, const void *E, Operand cat, int R, int H, int V);
// x <- x + sum(P); xg <- T(x * g) (not normalised); sumsq[r][chunk] <- partial sums of x^2 over
// chunks of 1024 columns (chunks = ceil(H / 1024)).  H % 4 == 0.
// Residual SiLU-Linear blocks of several independent heads in one launch (Medusa-style heads):
// rows [h * rows_per_head, (h + 1) * rows_per_head) belong to head h, whose partial sums start at
// P.p = p[h] (row index local to the head) and whose bias is bias[h]:
// x <- x + SiLU(sum(P) + bias); xn <- T(x).  H % 4 == 0, at most 8 heads.
struct HeadTab {
  const void *bias[8];
  const float *p[8];
  int rows_per_head;
};
cudaError_t resblock_update(Launch L, int dtype, float *x, SplitIn P, HeadTab tab, Operand xn, int R, int H);
// x <- E[tok]; xg <- T(x * g) (not normalised); sumsq as in row_update.  H % 4 == 0.
cudaError_t embed_update(Launch L, int dtype, const int32_t *tok, const void *E, const void *g, float *x,
                         Operand xg, float *sumsq, int R, int H, int V);
cudaError_t row_update(Launch L, int dtype, float *x, SplitIn P, const void *g, Operand xg, float *sumsq,
                       int R, int H);
// q_out: rotated queries in fp32; q_pair (bf16 only, may be null): the same as a bf16 pair
cudaError_t rope_kv_write(Launch L, int dtype, SplitIn qkv, RowScale sc, RowPlan plan, float *q_out,
                          Operand q_pair, void *k_cache, void *v_cache, int R, int rows_per_seq, int n_heads,
                          int head_dim, int S_max);
cudaError_t swiglu(Launch L, int dtype, SplitIn gu, RowScale sc, Operand act, int R, int F);
cudaError_t tree_attention(Launch L, int dtype, const float *q, const void *k_cache,
                           const void *v_cache, RowPlan plan, Operand out, int R, int rows_per_seq,
                           int B, int n_heads, int head_dim, int S_max);
cudaError_t argmax_rows(Launch L, const float *logits, int32_t *out, int R, int V);
cudaError_t topk_logp(Launch L, const float *logits, int32_t *tok, float *logp, int R, int V, int k);
// dst[r] = T(src[row_src ? row_src[r] : r]); optionally dst32[r * dst32_stride] = the same row in fp32
cudaError_t cast_rows(Launch L, int dtype, const float *src, const int32_t *row_src, Operand dst,
                      float *dst32, int dst32_stride, int R, int H);
cudaError_t reduce_splits(Launch L, SplitIn P, float *Y, int ldy, int R, int ncols);

// attn_mma.cu : bf16 caches, head_dim 128, tensor cores, split over key chunks
int attn_mma_chunks(int B, int n_heads, int rows_per_seq, int S_max, int num_sms);
size_t attn_mma_scratch_floats(int rows_total, int n_heads, int chunks);
cudaError_t tree_attention_mma(Launch L, const float *q, const void *k_cache, const void *v_cache,
                               RowPlan plan, Operand out, float *scratch, int rows_per_seq, int B,
                               int n_heads, int S_max, int chunks);

// attn_tc.cu : the same on tcgen05 tensor cores, all rows of a sequence in one CTA, key chunks as a cluster;
// the queries come as the bf16 pair written by rope_kv_write ([q_rows_alloc][n_heads * 128] each)
int attn_tc_chunks(int B, int n_heads, int S_max, int num_sms);
bool attn_tc_supported(int rows_per_seq, int head_dim, int S_max);
cudaError_t tree_attention_tc(Launch L, Operand q_pair, int q_rows_alloc, const void *k_cache, const void *v_cache,
                              RowPlan plan, Operand out, int rows_per_seq, int B, int n_heads, int S_max, int chunks,
                              int *status);

// gemm_simt.cu : Y[R][sum n_out] (fp32, ld ldy) = X[R][K_in] * W^T, X and W of `dtype`
cudaError_t gemm_simt(Launch L, int dtype, Operand X, GemmMats m, int K_in, int R, float *Y,
                      int ldy);

// gemm_tc.cu : bf16 tensor-core path; writes `split` partial matrices `split_stride` apart.
int tc_init_driver(char *err, size_t errlen);   // 0 on success
bool tc_supported(const GemmMats &m, int K_in);
int tc_default_split(int n_tiles, int kblocks, int tokens);
// split >= 1: classic split-K; split == 0: automatic (stream-K where it applies).  `max_slots`
// bounds the partial matrices written; *out describes them for the consumer.
cudaError_t gemm_tc(Launch L, Operand X, int x_rows_alloc, GemmMats m, int K_in, int R,
                    float *Y, int ldy, int split, size_t split_stride, int *status, int max_slots,
                    SplitIn *out);

// layer_tc.cu : several GEMMs of a decoder layer and the row-wise steps between them in one
// persistent launch (bf16, activations as pairs, at most 128 rows, head_dim 128 for the rotary step)
constexpr int LAYER_MAX_PHASES = 4;
constexpr int LAYER_SYNC_WORDS = 2 * LAYER_MAX_PHASES + 1;   // done[], ready[] counters and the abort word
enum { LAYER_POST_NONE = 0, LAYER_POST_ROW_UPDATE = 1, LAYER_POST_SWIGLU = 2, LAYER_POST_ROPE_KV = 3 };
struct LayerPhaseJob {
  Operand X;              // [x_rows_alloc][K_in] pair
  int K_in;
  GemmMats m;             // every n_out a multiple of 128
  float *Y;               // partial sums: max_slots matrices split_stride floats apart, row stride ldy
  int ldy;
  size_t split_stride;
  int max_slots;
  int post;               // what consumes the partial sums
  RowScale sc;            // SwiGLU / rotary step: RMSNorm scale still owed by this GEMM's input
  const void *gain;       // residual update: gain of the norm that follows
  Operand out;            // residual update: x * gain [R][ncols]; SwiGLU: activations [R][ncols]; rotary: query pair
  float *sumsq;           // residual update: [R][ceil(ncols / 512)]
  int ncols;              // residual update: H; SwiGLU: F
};
struct LayerJob {
  LayerPhaseJob ph[LAYER_MAX_PHASES];
  int n_phases;
  int R, x_rows_alloc;
  float *x;               // residual stream [R][H]
  RowPlan plan;           // rotary step
  float *q_out;
  void *k_cache, *v_cache;
  int rows_per_seq, n_heads, head_dim, S_max;
};
bool layer_stream_supported(const LayerJob &job);
// sync: LAYER_SYNC_WORDS device words, zero at context start; use_count: host counters [LAYER_MAX_PHASES]
// outs (optional): how each phase's partial sums are laid out, for a consumer outside the launch
cudaError_t layer_stream(Launch L, const LayerJob &job, unsigned *sync, unsigned *use_count, int *status,
                         SplitIn *outs);

// selftest.cu : a wait that runs out on purpose, with nothing else in flight
cudaError_t selftest_timeout(Launch L, int *status, long long limit_cycles);

// tree.cu
struct TreeBufs {
  int32_t *tree_tok, *tree_parent, *tree_level, *tree_n;
  float *tree_score;
  uint64_t *tree_anc;      // [B][N][2]
  int32_t *cand_tok, *cand_parent, *cand_level, *cand_rank;
  float *cand_score;
  int32_t *frontier;       // [B][k] candidate ids
  uint64_t *front_mask;    // [B][k][2] draft-cache visibility of each frontier row
  int32_t *front_row;      // [B][pool] draft tree row of a candidate once it was a frontier row
  int32_t *topk_tok;
  float *topk_logp;
  int32_t *root_tok, *pend_tok, *n_pend, *acc_path, *acc_len, *acc_S;
  unsigned long long *alpha_hits, *alpha_trials;   // [128] position-wise acceptance counters
  float *pend_hid;
};
struct PlanBufs {
  int32_t *pos, *slot, *ctx_len, *kv_len, *row_src, *row_tok, *last_row;
  uint64_t *mask;
  float2 *rope;
};
cudaError_t tree_from_caller(Launch L, TreeBufs t, const int32_t *tok, const int32_t *parent,
                             const int32_t *n_nodes, int stride, int B, int N, int *status);
cudaError_t tree_ancestors(Launch L, TreeBufs t, int B, int N);
cudaError_t plan_verify(Launch L, TreeBufs t, PlanBufs p, const int32_t *seq_len, int B, int N,
                        int head_dim, float rope_base, int S_max, int *status);
cudaError_t plan_draft0(Launch L, TreeBufs t, PlanBufs p, const int32_t *seq_len, int B, int N,
                        int rows, int head_dim, float rope_base, int S_max, int *status);
cudaError_t plan_draft_p(Launch L, TreeBufs t, PlanBufs p, const int32_t *seq_len, int B, int k,
                         int pool, int pass, int head_dim, float rope_base, int S_max, int *status);
cudaError_t expand_dynamic(Launch L, TreeBufs t, int B, int k, int pool, int pass, int D, int N);
cudaError_t expand_static(Launch L, TreeBufs t, const int32_t *s_parent, const int32_t *s_level,
                          const int32_t *s_rank, int B, int N, int k);
cudaError_t plan_medusa(Launch L, TreeBufs t, PlanBufs p, int B, int N, int heads);
cudaError_t accept_walk(Launch L, TreeBufs t, const int32_t *verify_tgt, const float *verify_hid,
                        const int32_t *forced_len, int32_t *seq_len, int32_t *out_tokens,
                        int out_stride, int32_t *out_len, int B, int N, int H);
cudaError_t kv_compact(Launch L, int dtype, TreeBufs t, void *k_cache, void *v_cache, int L_layers,
                       int B, int N, int n_heads, int head_dim, int S_max);

// sampling.cu : speculative sampling on chain drafts (one row / one chain per sequence)
cudaError_t sample_rows(Launch L, const float *logits, const float *u, int u_stride, int u_off, int32_t *tok,
                        float *logp, float *probs, int R, int V);
cudaError_t accept_sampled(Launch L, TreeBufs t, const float *verify_logits, const float *verify_hid,
                           const float *chain_d, const float *u_accept, const float *u_bonus, int32_t *seq_len,
                           int32_t *out_tokens, int out_stride, int32_t *out_len, int B, int N, int H, int V, int D,
                           int *status);

}  // namespace koala
