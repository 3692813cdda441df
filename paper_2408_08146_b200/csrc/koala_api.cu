// C ABI of libkoala: context, workspace carving and the kernel sequence of each step.
// Host code only enqueues kernels on the caller's stream; it never synchronises.
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/koala.h"
#include "common.cuh"
#include "koala_debug.h"

using namespace koala;

namespace koala {
void tc_forget_maps();
void tc_set_tuning(int key, int value);
unsigned long long g_launches = 0;
}

namespace {

enum Phase { PH_READY = 0, PH_DRAFTED, PH_EXPANDED, PH_TREE, PH_VERIFIED };

struct LayerW {
  const void *attn_norm, *wq, *wk, *wv, *wo, *ffn_norm, *wg, *wu, *wd;
};

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

constexpr size_t GUARD_BYTES = 256;
constexpr int GUARD_PATTERN = 0xC5;

// Walks the workspace; with base == nullptr it only measures.  Every buffer is followed by a guard
// of GUARD_BYTES that nothing writes after koala_init (koala_debug_check_guards).
struct Carver {
  unsigned char *base;
  size_t off;
  std::vector<size_t> *guards;
  template <typename T> T *take(size_t count) {
    off = align_up(off, 256);
    T *p = base ? reinterpret_cast<T *>(base + off) : nullptr;
    off = align_up(off + count * sizeof(T), 256);
    if (guards) guards->push_back(off);
    off += GUARD_BYTES;
    return p;
  }
};

constexpr int MAX_SPLIT = 12;     // partial-sum matrices the workspace holds per GEMM

}  // namespace

struct koala_ctx {
  koala_config cfg;
  cudaStream_t st;
  bool pdl, use_tc;
  const void *embed, *lm_head, *final_norm, *fc_w, *fc_b;
  std::vector<LayerW> layers, draft_layers;
  std::vector<const void *> res_w, res_b, medusa_lm;
  void *tk, *tv, *dk, *dv;
  int32_t *seq_len;
  // derived sizes
  int M, Mp, pool, draft_rows_max, esz;
  size_t pcols;           // widest GEMM output
  // workspace
  float *attn_part;
  float *sumsq[2];        // per-row partial sums of squares of the two deferred RMSNorms of a layer
  unsigned *layer_sync;   // device counters of the persistent layer kernel
  unsigned layer_use[LAYER_MAX_PHASES];   // how often each counter has been used (host)
  bool stream_layers;     // decoder layers run through the persistent layer kernel where it applies
  RowScale pending;       // scale still owed by the consumer of the GEMM that reads c->xn
  int attn_chunks;
  float *x, *qbuf, *P, *verify_logits, *draft_logits, *verify_hid, *feat[2], *mx;
  Operand xn, attn_out, act, cat, lmin;
  size_t p_off;            // floats: where in P the next GEMM's partial sums go (0 except while heads are batched)
  int p_slots;             // partial matrices that fit there
  Operand qpair;           // rotated queries as a bf16 pair (bf16 configurations)
  float *chain_d;          // [B][D][V] draft distributions of a sampled chain (k = 1 configurations)
  const float *u_draft;    // device [B][D] uniforms: drafted tokens are sampled while non-null
  bool pair;              // bf16 activations kept as hi + lo
  int32_t *verify_tgt, *s_parent, *s_level, *s_rank;
  int *status;
  TreeBufs t;
  PlanBufs p;
  // host state
  Phase phase;
  int last_pass, pend_cap, draft_rows, expand_mode;
  bool last_tree_from_caller;
  int *host_status;       // pinned
  cudaEvent_t poll_ev;
  bool poll_pending;
  int last_status;
  // per-kernel timing (KOALA_OPT_TIMING)
  bool timing;
  std::vector<cudaEvent_t> ev;          // pairs: start, stop
  std::vector<int> ev_cls;              // class of each pair
  size_t ev_used;                       // pairs in use
  uint64_t t_bytes[3];
  int32_t t_launches[3];
  unsigned char *ws_base;
  std::vector<size_t> guards;    // offsets of the guard words in the workspace
  char err[256];
};

namespace {

int fail(koala_ctx *c, int code, const char *fmt, ...) {
  if (c) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(c->err, sizeof(c->err), fmt, ap);
    va_end(ap);
  }
  return code;
}

#define CU_TRY(expr)                                                                     \
  do {                                                                                   \
    cudaError_t e__ = (expr);                                                            \
    if (e__ != cudaSuccess)                                                              \
      return fail(c, KOALA_E_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e__));     \
  } while (0)

bool config_ok(const koala_config *cfg, char *why, size_t n) {
#define BAD(msg)              \
  do {                        \
    snprintf(why, n, msg);    \
    return false;             \
  } while (0)
  if (!cfg) BAD("null config");
  if (cfg->struct_size != sizeof(koala_config)) BAD("koala_config.struct_size mismatch");
  if (cfg->dtype != KOALA_FP32 && cfg->dtype != KOALA_BF16) BAD("dtype must be fp32 or bf16");
  if (cfg->head_kind != KOALA_EAGLE && cfg->head_kind != KOALA_MEDUSA) BAD("unknown head_kind");
  if (cfg->L < 1 || cfg->H < 1 || cfg->F < 1 || cfg->V < 2) BAD("non-positive model dimension");
  if (cfg->n_heads < 1 || cfg->n_heads * cfg->head_dim != cfg->H) BAD("n_heads * head_dim != H");
  if (cfg->head_dim != 64 && cfg->head_dim != 128) BAD("head_dim must be 64 or 128");
  if (cfg->K < 0 || cfg->K > 64) BAD("K out of range");
  if (cfg->topk < 1 || cfg->topk > KOALA_MAX_TOPK || cfg->topk > cfg->V) BAD("topk out of range");
  if (cfg->N < 1 || cfg->N > KOALA_MAX_TREE) BAD("N out of range");
  if (cfg->B < 1 || cfg->B > 64) BAD("B out of range");
  if (cfg->D < 1 || cfg->D > 16) BAD("D out of range");
  if (cfg->S_max < cfg->N) BAD("S_max smaller than the tree");
  if (cfg->head_kind == KOALA_MEDUSA) {
    if (cfg->n_medusa_heads < 1 || cfg->n_medusa_heads > 16) BAD("n_medusa_heads out of range");
    if (cfg->D != cfg->n_medusa_heads) BAD("MEDUSA: D must equal n_medusa_heads");
  } else {
    if ((cfg->D - 1) * cfg->topk > 128) BAD("EAGLE: (D-1)*topk must be <= 128");
  }
  if (!(cfg->rms_eps > 0.f) || !(cfg->rope_base > 1.f)) BAD("bad rms_eps / rope_base");
#undef BAD
  return true;
}

// Assigns (or measures) every workspace buffer.  Must visit the same sequence in both modes.
size_t carve(koala_ctx *c, const koala_config &cfg, unsigned char *base) {
  c->guards.clear();
  Carver w{base, 0, base ? &c->guards : nullptr};
  const int B = cfg.B, N = cfg.N, H = cfg.H, F = cfg.F, V = cfg.V, k = cfg.topk;
  const int M = B * N;
  int draft_rows = B * k;
  if (cfg.head_kind == KOALA_MEDUSA && cfg.n_medusa_heads * B > draft_rows) draft_rows = cfg.n_medusa_heads * B;
  int rows = M > draft_rows ? M : draft_rows;
  // padded row count: the tensor-core GEMM reads whole token tiles (up to 256 rows) of its input
  const int Mp = (int)align_up((size_t)rows + 16, rows > 128 ? 256 : 16);
  const int pool = cfg.head_kind == KOALA_EAGLE ? k + (cfg.D - 1) * k * k : k;
  const size_t pcols = (size_t)(3 * H > 2 * F ? 3 * H : 2 * F);
  const size_t esz = cfg.dtype == KOALA_FP32 ? 4 : 2;
  c->M = M; c->Mp = Mp; c->pool = pool; c->draft_rows_max = draft_rows; c->esz = (int)esz; c->pcols = pcols;
  c->x = w.take<float>((size_t)Mp * H);
  c->qbuf = w.take<float>((size_t)Mp * H);
  c->P = w.take<float>((size_t)MAX_SPLIT * Mp * pcols);
  c->verify_logits = w.take<float>((size_t)Mp * V);
  c->draft_logits = w.take<float>((size_t)(draft_rows + 16) * V);
  c->verify_hid = w.take<float>((size_t)Mp * H);
  c->feat[0] = w.take<float>((size_t)(B * k + 16) * H);
  c->feat[1] = w.take<float>((size_t)(B * k + 16) * H);
  c->mx = w.take<float>((size_t)Mp * H);
  const bool pair = cfg.dtype == KOALA_BF16;     // bf16 operands as value + rounding residual
  c->pair = pair;
  auto operand = [&](size_t cols) {
    Operand o;
    o.hi = w.take<unsigned char>((size_t)Mp * cols * esz);
    o.lo = pair ? (void *)w.take<unsigned char>((size_t)Mp * cols * esz) : nullptr;
    if (!base) o.lo = nullptr;
    return o;
  };
  c->xn = operand(H);
  c->attn_out = operand(H);
  c->qpair = Operand{nullptr, nullptr};
  if (cfg.dtype == KOALA_BF16) {
    c->qpair.hi = w.take<unsigned char>((size_t)Mp * H * esz);
    c->qpair.lo = w.take<unsigned char>((size_t)Mp * H * esz);
  }
  c->act = operand(F);
  c->cat = operand(2 * H);
  c->lmin = operand(H);
  c->attn_chunks = 16;     // largest chunk count any launch may choose
  c->attn_part = (cfg.dtype == KOALA_BF16 && cfg.head_dim == 128)
                     ? w.take<float>(attn_mma_scratch_floats(Mp, cfg.n_heads, c->attn_chunks))
                     : nullptr;
  c->sumsq[0] = w.take<float>((size_t)Mp * 32);
  c->sumsq[1] = w.take<float>((size_t)Mp * 32);
  c->layer_sync = w.take<unsigned>(LAYER_SYNC_WORDS);
  c->verify_tgt = w.take<int32_t>(Mp);
  c->s_parent = w.take<int32_t>(N);
  c->s_level = w.take<int32_t>(N);
  c->s_rank = w.take<int32_t>(N);
  c->status = w.take<int>(4);
  TreeBufs &t = c->t;
  t.tree_tok = w.take<int32_t>(M);
  t.tree_parent = w.take<int32_t>(M);
  t.tree_level = w.take<int32_t>(M);
  t.tree_n = w.take<int32_t>(B);
  t.tree_score = w.take<float>(M);
  t.tree_anc = w.take<uint64_t>((size_t)M * 2);
  t.cand_tok = w.take<int32_t>((size_t)B * pool);
  t.cand_parent = w.take<int32_t>((size_t)B * pool);
  t.cand_level = w.take<int32_t>((size_t)B * pool);
  t.cand_rank = w.take<int32_t>((size_t)B * pool);
  t.cand_score = w.take<float>((size_t)B * pool);
  t.frontier = w.take<int32_t>((size_t)B * k);
  t.front_mask = w.take<uint64_t>((size_t)B * k * 2);
  t.front_row = w.take<int32_t>((size_t)B * pool);
  t.topk_tok = w.take<int32_t>((size_t)draft_rows * k);
  t.topk_logp = w.take<float>((size_t)draft_rows * k);
  t.root_tok = w.take<int32_t>(B);
  t.pend_tok = w.take<int32_t>(M);
  t.n_pend = w.take<int32_t>(B);
  t.acc_path = w.take<int32_t>(M);
  t.acc_len = w.take<int32_t>(B);
  t.acc_S = w.take<int32_t>(B);
  c->chain_d = (cfg.head_kind == KOALA_EAGLE && k == 1) ? w.take<float>((size_t)B * cfg.D * V) : nullptr;
  t.alpha_hits = w.take<unsigned long long>(128);
  t.alpha_trials = w.take<unsigned long long>(128);
  t.pend_hid = w.take<float>((size_t)M * H);
  PlanBufs &p = c->p;
  p.pos = w.take<int32_t>(Mp);
  p.slot = w.take<int32_t>(Mp);
  p.ctx_len = w.take<int32_t>(B);
  p.kv_len = w.take<int32_t>(B);
  p.row_src = w.take<int32_t>(Mp);
  p.row_tok = w.take<int32_t>(Mp);
  p.last_row = w.take<int32_t>(B);
  p.mask = w.take<uint64_t>((size_t)Mp * 2);
  p.rope = w.take<float2>((size_t)Mp * (cfg.head_dim / 2));
  return align_up(w.off, 256);
}

Launch LN(koala_ctx *c) { return Launch{c->st, c->pdl}; }

size_t kv_layer_elems(const koala_config &g) {
  return (size_t)g.B * g.n_heads * g.S_max * g.head_dim;
}

constexpr size_t MAX_TIMED = 8192;

// Opens a timed bracket (returns its index, or -1 when timing is off / the pool is full).
int time_begin(koala_ctx *c, int cls, uint64_t bytes) {
  if (!c->timing || c->ev_used >= MAX_TIMED) return -1;
  if (c->ev.size() < 2 * (c->ev_used + 1)) {
    cudaEvent_t a, b;
    if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) return -1;
    c->ev.push_back(a);
    c->ev.push_back(b);
    c->ev_cls.push_back(cls);
  }
  const int i = (int)c->ev_used++;
  c->ev_cls[i] = cls;
  c->t_bytes[cls] += bytes;
  c->t_launches[cls] += 1;
  cudaEventRecord(c->ev[2 * i], c->st);
  return i;
}
void time_end(koala_ctx *c, int i) {
  if (i >= 0) cudaEventRecord(c->ev[2 * i + 1], c->st);
}

RowPlan row_plan(koala_ctx *c) {
  return RowPlan{c->p.pos, c->p.slot, c->p.mask, c->p.ctx_len, c->p.kv_len, c->p.rope};
}

// Y = X * [W...]^T as a (possibly split) fp32 result in the partial buffer, or directly into
// `direct` (ld = ld_direct) when given.
int do_gemm(koala_ctx *c, Operand X, int K_in, GemmMats m, int R, float *direct, int ld_direct,
            SplitIn *out) {
  int ncols = 0;
  for (int i = 0; i < m.n; ++i) ncols += m.n_out[i];
  float *Y = direct ? direct : c->P + c->p_off;
  const int ld = direct ? ld_direct : ncols;
  const uint64_t wbytes = (uint64_t)ncols * K_in * c->esz;
  if (c->use_tc && c->cfg.dtype == KOALA_BF16 && tc_supported(m, K_in)) {
    const size_t stride = (size_t)c->Mp * ld;
    const int tb = time_begin(c, KOALA_CLS_GEMM_TC, wbytes);
    SplitIn res;
    CU_TRY(gemm_tc(LN(c), X, c->Mp, m, K_in, R, Y, ld, direct ? 1 : 0, stride, c->status,
                   c->p_slots > 0 ? c->p_slots : MAX_SPLIT, &res));
    time_end(c, tb);
    if (out) *out = res;
  } else {
    const int tb = time_begin(c, KOALA_CLS_GEMM_SIMT, wbytes);
    CU_TRY(gemm_simt(LN(c), c->cfg.dtype, X, m, K_in, R, Y, ld));
    time_end(c, tb);
    if (out) *out = SplitIn{Y, 1, 0, ld, 0u, 0u, 0u};
  }
  return KOALA_OK;
}

#define K_TRY(expr)              \
  do {                           \
    int rc__ = (expr);           \
    if (rc__ != KOALA_OK) return rc__; \
  } while (0)

// Tree-masked attention of one layer over R rows: reads the rotated queries (fp32 and pair) and the
// cache, writes the O projection's operand pair.
int run_attention(koala_ctx *c, void *kc, void *vc, int R, int rows_per_seq) {
  const koala_config &g = c->cfg;
  const int ta = time_begin(c, KOALA_CLS_ATTENTION, 0);
  if (c->use_tc && g.dtype == KOALA_BF16 && c->qpair.lo != nullptr &&
      attn_tc_supported(rows_per_seq, g.head_dim, g.S_max)) {
    CU_TRY(tree_attention_tc(LN(c), c->qpair, c->Mp, kc, vc, row_plan(c), c->attn_out, rows_per_seq, g.B, g.n_heads,
                             g.S_max, attn_tc_chunks(g.B, g.n_heads, g.S_max, 148), c->status));
  } else if (c->use_tc && g.head_dim == 128 && c->attn_part != nullptr && rows_per_seq <= 128) {
    CU_TRY(tree_attention_mma(LN(c), c->qbuf, kc, vc, row_plan(c), c->attn_out, c->attn_part, rows_per_seq,
                              g.B, g.n_heads, g.S_max,
                              attn_mma_chunks(g.B, g.n_heads, rows_per_seq, g.S_max, 148)));
  } else {
    CU_TRY(tree_attention(LN(c), g.dtype, c->qbuf, kc, vc, row_plan(c), c->attn_out, R, rows_per_seq, g.B,
                          g.n_heads, g.head_dim, g.S_max));
  }
  time_end(c, ta);
  return KOALA_OK;
}

// One pre-norm decoder layer over R rows.  On entry x holds the residual stream and xn the
// normalised input of the attention block.  On exit x is updated and `next_xn` holds
// T(rmsnorm(x) * next_g) (or T(x) if next_g is null); `out_f32` optionally receives the same in fp32.
// One pre-norm decoder layer over R rows.  On entry x holds the residual stream and xn the input
// of the attention block: normalised, or x * gain with the scale still pending in c->pending.
// On exit x is updated; if `defer` the next layer's input is left in c->xn as x * next_g with its
// scale pending, otherwise `next_xn` holds T(rmsnorm(x) * next_g) (or T(x) if next_g is null) and
// `out_f32` optionally the same in fp32.
int run_layer(koala_ctx *c, const LayerW &w, void *kc, void *vc, int R, int rows_per_seq,
              const void *next_g, Operand next_xn, float *out_f32, bool defer) {
  const koala_config &g = c->cfg;
  const int H = g.H, F = g.F;
  const bool can_defer = (H % 4) == 0 && H <= 8192;
  const RowScale none{nullptr, 0, 0.f, 0.f};
  SplitIn s;
  GemmMats qkv{{w.wq, w.wk, w.wv}, {H, H, H}, 3};
  K_TRY(do_gemm(c, c->xn, H, qkv, R, nullptr, 0, &s));
  CU_TRY(rope_kv_write(LN(c), g.dtype, s, c->pending, row_plan(c), c->qbuf, c->qpair, kc, vc, R, rows_per_seq, g.n_heads,
                       g.head_dim, g.S_max));
  c->pending = none;
  K_TRY(run_attention(c, kc, vc, R, rows_per_seq));
  GemmMats o{{w.wo, nullptr, nullptr}, {H, 0, 0}, 1};
  K_TRY(do_gemm(c, c->attn_out, H, o, R, nullptr, 0, &s));
  RowScale ffn = none;
  if (can_defer && (s.ld % 4) == 0 && (s.stride % 4) == 0) {
    CU_TRY(row_update(LN(c), g.dtype, c->x, s, w.ffn_norm, c->xn, c->sumsq[0], R, H));
    ffn = RowScale{c->sumsq[0], (H + 1023) / 1024, 1.f / (float)H, g.rms_eps};
  } else {
    CU_TRY(row_epilogue(LN(c), g.dtype, 0, c->x, s, nullptr, w.ffn_norm, c->xn, nullptr, R, H, g.rms_eps));
  }
  GemmMats gu{{w.wg, w.wu, nullptr}, {F, F, 0}, 2};
  K_TRY(do_gemm(c, c->xn, H, gu, R, nullptr, 0, &s));
  CU_TRY(swiglu(LN(c), g.dtype, s, ffn, c->act, R, F));
  GemmMats dn{{w.wd, nullptr, nullptr}, {H, 0, 0}, 1};
  K_TRY(do_gemm(c, c->act, F, dn, R, nullptr, 0, &s));
  if (defer && can_defer && next_g != nullptr && (s.ld % 4) == 0 && (s.stride % 4) == 0) {
    CU_TRY(row_update(LN(c), g.dtype, c->x, s, next_g, c->xn, c->sumsq[1], R, H));
    c->pending = RowScale{c->sumsq[1], (H + 1023) / 1024, 1.f / (float)H, g.rms_eps};
  } else {
    CU_TRY(row_epilogue(LN(c), g.dtype, 0, c->x, s, nullptr, next_g, next_xn, out_f32, R, H, g.rms_eps));
  }
  return KOALA_OK;
}


// n_layers pre-norm decoder layers over R rows.  On entry x holds the residual stream and c->xn the
// first layer's input (normalised, or x * gain with its scale pending in c->pending).  After the
// last layer the output is rmsnorm(x) * final_g (or x if final_g is null) as an operand in
// `final_xn` and, optionally, in fp32 in `out_f32`.
// Where the persistent layer kernel applies (bf16 pairs, at most 128 rows, head_dim 128, matrices
// of whole 128-row tiles) a layer is two launches: attention, and one launch that runs
// O -> residual -> gate/up -> SwiGLU -> down -> residual -> the next layer's Q/K/V -> rotary/cache.
int run_layers(koala_ctx *c, const std::vector<LayerW> &layers, int n_layers, void *kbase, void *vbase, int R,
               int rows_per_seq, const void *final_g, Operand final_xn, float *out_f32) {
  const koala_config &g = c->cfg;
  const int H = g.H, F = g.F;
  const size_t le = kv_layer_elems(g) * c->esz;
  auto kc_of = [&](int l) { return (void *)((unsigned char *)kbase + (size_t)l * le); };
  auto vc_of = [&](int l) { return (void *)((unsigned char *)vbase + (size_t)l * le); };
  bool streamed = c->stream_layers && g.dtype == KOALA_BF16 && c->pair && g.head_dim == 128 && R <= 128 &&
                  c->qpair.lo != nullptr && n_layers > 0;
  LayerJob job;
  const size_t stride = (size_t)c->Mp * c->pcols;     // one partial-sum matrix of the widest GEMM
  auto base_job = [&]() {
    memset(&job, 0, sizeof(job));
    job.R = R;
    job.x_rows_alloc = c->Mp;
    job.x = c->x;
    job.plan = row_plan(c);
    job.q_out = c->qbuf;
    job.rows_per_seq = rows_per_seq;
    job.n_heads = g.n_heads;
    job.head_dim = g.head_dim;
    job.S_max = g.S_max;
  };
  auto phase = [&](int i, Operand X, int K_in, GemmMats m, int post) -> LayerPhaseJob & {
    LayerPhaseJob &j = job.ph[i];
    int ncols = 0;
    for (int q = 0; q < m.n; ++q) ncols += m.n_out[q];
    j.X = X; j.K_in = K_in; j.m = m; j.Y = c->P; j.ldy = ncols; j.split_stride = (size_t)c->Mp * ncols;
    j.max_slots = MAX_SPLIT; j.post = post;
    j.sc = RowScale{nullptr, 0, 0.f, 0.f};
    (void)stride;
    return j;
  };
  const int chunks = (H + 511) / 512;
  auto qkv_phase = [&](int i, const LayerW &w, RowScale sc) {
    LayerPhaseJob &j = phase(i, c->xn, H, GemmMats{{w.wq, w.wk, w.wv}, {H, H, H}, 3}, LAYER_POST_ROPE_KV);
    j.sc = sc;
    j.out = c->qpair;
  };
  auto weight_bytes = [&](const LayerJob &jb) {
    uint64_t b = 0;
    for (int i = 0; i < jb.n_phases; ++i)
      for (int q = 0; q < jb.ph[i].m.n; ++q) b += (uint64_t)jb.ph[i].m.n_out[q] * jb.ph[i].K_in * c->esz;
    return b;
  };
  if (streamed) {
    // dry run of the shapes: every launch of the sequence must be supported, else the per-kernel path
    base_job();
    qkv_phase(0, layers[0], c->pending);
    job.k_cache = kc_of(0); job.v_cache = vc_of(0);
    job.n_phases = 1;
    streamed = layer_stream_supported(job);
    if (streamed) {
      LayerPhaseJob &a = phase(0, c->attn_out, H, GemmMats{{layers[0].wo, nullptr, nullptr}, {H, 0, 0}, 1}, LAYER_POST_ROW_UPDATE);
      a.gain = layers[0].ffn_norm; a.out = c->xn; a.sumsq = c->sumsq[0]; a.ncols = H;
      LayerPhaseJob &b = phase(1, c->xn, H, GemmMats{{layers[0].wg, layers[0].wu, nullptr}, {F, F, 0}, 2}, LAYER_POST_SWIGLU);
      b.out = c->act; b.ncols = F;
      phase(2, c->act, F, GemmMats{{layers[0].wd, nullptr, nullptr}, {H, 0, 0}, 1}, LAYER_POST_NONE);
      job.n_phases = 3;
      streamed = layer_stream_supported(job);
    }
  }
  if (!streamed) {
    for (int l = 0; l < n_layers; ++l) {
      const bool last = l == n_layers - 1;
      K_TRY(run_layer(c, layers[l], kc_of(l), vc_of(l), R, rows_per_seq, last ? final_g : layers[l + 1].attn_norm,
                      last ? final_xn : c->xn, last ? out_f32 : nullptr, !last));
    }
    return KOALA_OK;
  }
  const RowScale none{nullptr, 0, 0.f, 0.f};
  const RowScale ffn_scale{c->sumsq[0], chunks, 1.f / (float)H, g.rms_eps};
  const RowScale attn_scale{c->sumsq[1], chunks, 1.f / (float)H, g.rms_eps};
  // the first layer's Q/K/V with the rotary step
  base_job();
  qkv_phase(0, layers[0], c->pending);
  job.k_cache = kc_of(0); job.v_cache = vc_of(0);
  job.n_phases = 1;
  {
    const int tb = time_begin(c, KOALA_CLS_GEMM_TC, weight_bytes(job));
    CU_TRY(layer_stream(LN(c), job, c->layer_sync, c->layer_use, c->status, nullptr));
    time_end(c, tb);
  }
  c->pending = none;
  for (int l = 0; l < n_layers; ++l) {
    const bool last = l == n_layers - 1;
    const LayerW &w = layers[l];
    K_TRY(run_attention(c, kc_of(l), vc_of(l), R, rows_per_seq));
    base_job();
    LayerPhaseJob &a = phase(0, c->attn_out, H, GemmMats{{w.wo, nullptr, nullptr}, {H, 0, 0}, 1}, LAYER_POST_ROW_UPDATE);
    a.gain = w.ffn_norm; a.out = c->xn; a.sumsq = c->sumsq[0]; a.ncols = H;
    LayerPhaseJob &b = phase(1, c->xn, H, GemmMats{{w.wg, w.wu, nullptr}, {F, F, 0}, 2}, LAYER_POST_SWIGLU);
    b.sc = ffn_scale; b.out = c->act; b.ncols = F;
    LayerPhaseJob &d = phase(2, c->act, F, GemmMats{{w.wd, nullptr, nullptr}, {H, 0, 0}, 1},
                             last ? LAYER_POST_NONE : LAYER_POST_ROW_UPDATE);
    job.n_phases = 3;
    if (!last) {
      d.gain = layers[l + 1].attn_norm; d.out = c->xn; d.sumsq = c->sumsq[1]; d.ncols = H;
      qkv_phase(3, layers[l + 1], attn_scale);
      job.k_cache = kc_of(l + 1); job.v_cache = vc_of(l + 1);
      job.n_phases = 4;
    }
    SplitIn outs[LAYER_MAX_PHASES];
    const int tb = time_begin(c, KOALA_CLS_GEMM_TC, weight_bytes(job));
    CU_TRY(layer_stream(LN(c), job, c->layer_sync, c->layer_use, c->status, outs));
    time_end(c, tb);
    if (last)
      CU_TRY(row_epilogue(LN(c), g.dtype, 0, c->x, outs[2], nullptr, final_g, final_xn, out_f32, R, H, g.rms_eps));
  }
  return KOALA_OK;
}

int draft_eagle(koala_ctx *c, int pass) {
  const koala_config &g = c->cfg;
  const int H = g.H, k = g.topk, B = g.B;
  const int rows = pass == 0 ? c->pend_cap : k;
  const int R = B * rows;
  c->pending = RowScale{nullptr, 0, 0.f, 0.f};
  const float *feat_src;
  if (pass == 0) {
    CU_TRY(plan_draft0(LN(c), c->t, c->p, c->seq_len, B, g.N, rows, g.head_dim, g.rope_base, g.S_max,
                       c->status));
    feat_src = c->t.pend_hid;
  } else {
    CU_TRY(plan_draft_p(LN(c), c->t, c->p, c->seq_len, B, k, c->pool, pass, g.head_dim, g.rope_base,
                        g.S_max, c->status));
    feat_src = c->feat[(pass - 1) & 1];
  }
  CU_TRY(eagle_concat(LN(c), g.dtype, feat_src, c->p.row_src, c->p.row_tok, c->embed, c->cat, R, H, g.V));
  SplitIn s;
  GemmMats fc{{c->fc_w, nullptr, nullptr}, {H, 0, 0}, 1};
  K_TRY(do_gemm(c, c->cat, 2 * H, fc, R, nullptr, 0, &s));
  // pass 0: the feature of every row stays in x and the last valid row is gathered afterwards;
  // pass >= 1: every row's feature goes to feat[pass & 1] and to the LM head's input.
  float *f_all = pass == 0 ? nullptr : c->feat[pass & 1];
  const Operand none{nullptr, nullptr};
  const Operand lm_all = pass == 0 ? none : c->lmin;
  if (g.K == 0) {
    CU_TRY(row_epilogue(LN(c), g.dtype, 1, c->x, s, c->fc_b, nullptr, lm_all, f_all, R, H, g.rms_eps));
  } else {
    CU_TRY(row_epilogue(LN(c), g.dtype, 1, c->x, s, c->fc_b, c->draft_layers[0].attn_norm, c->xn, nullptr,
                        R, H, g.rms_eps));
    K_TRY(run_layers(c, c->draft_layers, g.K, c->dk, c->dv, R, rows, nullptr, lm_all, f_all));
  }
  int lm_rows = R;
  if (pass == 0) {
    CU_TRY(cast_rows(LN(c), g.dtype, c->x, c->p.last_row, c->lmin, c->feat[0], k, B, H));
    lm_rows = B;
  }
  GemmMats lm{{c->lm_head, nullptr, nullptr}, {g.V, 0, 0}, 1};
  K_TRY(do_gemm(c, c->lmin, H, lm, lm_rows, c->draft_logits, g.V, nullptr));
  c->draft_rows = lm_rows;
  return KOALA_OK;
}

int draft_medusa(koala_ctx *c) {
  const koala_config &g = c->cfg;
  const int H = g.H, B = g.B, nh = g.n_medusa_heads;
  const int R = nh * B;
  CU_TRY(plan_medusa(LN(c), c->t, c->p, B, g.N, nh));
  CU_TRY(cast_rows(LN(c), g.dtype, c->t.pend_hid, c->p.row_src, c->xn, c->mx, 1, R, H));
  // The heads are independent chains.  Block j of every head is multiplied first (each head's
  // partial sums in a region of its own), then the heads' epilogues run: the weight stream of one
  // head's matrix follows the previous head's without a small kernel in between.
  const size_t region = ((size_t)MAX_SPLIT * c->Mp * c->pcols / (size_t)(nh > 0 ? nh : 1)) & ~(size_t)63;
  const int slots = (int)(region / ((size_t)c->Mp * H));
  const bool batched = nh <= 8 && slots >= 1;
  SplitIn sp[8];
  for (int j = 0; j < g.K; ++j) {
    for (int i = 0; i < nh; ++i) {
      GemmMats m{{c->res_w[(size_t)i * g.K + j], nullptr, nullptr}, {H, 0, 0}, 1};
      const size_t off = (size_t)i * B * H * c->esz;
      Operand xi{(unsigned char *)c->xn.hi + off, c->xn.lo ? (unsigned char *)c->xn.lo + off : nullptr};
      if (batched) { c->p_off = (size_t)i * region; c->p_slots = slots < MAX_SPLIT ? slots : MAX_SPLIT; }
      SplitIn s;
      const int rc = do_gemm(c, xi, H, m, B, nullptr, 0, &s);
      c->p_off = 0;
      c->p_slots = 0;
      if (rc != KOALA_OK) return rc;
      if (batched) { sp[i] = s; continue; }
      CU_TRY(row_epilogue(LN(c), g.dtype, 2, c->mx + (size_t)i * B * H, s, c->res_b[(size_t)i * g.K + j],
                          nullptr, xi, nullptr, B, H, g.rms_eps));
    }
    if (!batched) continue;
    bool same = (H % 4) == 0 && (sp[0].ld % 4) == 0 && (sp[0].stride % 4) == 0 && sp[0].sk_ctas == 0;
    for (int i = 1; i < nh; ++i) same = same && sp[i].n == sp[0].n && sp[i].stride == sp[0].stride && sp[i].ld == sp[0].ld;
    if (same) {            // one launch finishes block j of every head
      HeadTab tab;
      memset(&tab, 0, sizeof(tab));
      for (int i = 0; i < nh; ++i) { tab.bias[i] = c->res_b[(size_t)i * g.K + j]; tab.p[i] = sp[i].p; }
      tab.rows_per_head = B;
      CU_TRY(resblock_update(LN(c), g.dtype, c->mx, sp[0], tab, c->xn, R, H));
      continue;
    }
    for (int i = 0; i < nh; ++i) {
      const size_t off = (size_t)i * B * H * c->esz;
      Operand xi{(unsigned char *)c->xn.hi + off, c->xn.lo ? (unsigned char *)c->xn.lo + off : nullptr};
      CU_TRY(row_epilogue(LN(c), g.dtype, 2, c->mx + (size_t)i * B * H, sp[i], c->res_b[(size_t)i * g.K + j],
                          nullptr, xi, nullptr, B, H, g.rms_eps));
    }
  }
  if (c->medusa_lm.empty()) {
    GemmMats lm{{c->lm_head, nullptr, nullptr}, {g.V, 0, 0}, 1};
    K_TRY(do_gemm(c, c->xn, H, lm, R, c->draft_logits, g.V, nullptr));
  } else {
    // every head ends in its own Linear: one multiply per head over that head's B rows
    for (int i = 0; i < nh; ++i) {
      GemmMats lm{{c->medusa_lm[i], nullptr, nullptr}, {g.V, 0, 0}, 1};
      const size_t off = (size_t)i * B * H * c->esz;
      Operand xi{(unsigned char *)c->xn.hi + off, c->xn.lo ? (unsigned char *)c->xn.lo + off : nullptr};
      K_TRY(do_gemm(c, xi, H, lm, B, c->draft_logits + (size_t)i * B * g.V, g.V, nullptr));
    }
  }
  c->draft_rows = R;
  return KOALA_OK;
}

}  // namespace

// ------------------------------------------------------------------------------------------------
extern "C" {
#pragma GCC visibility push(default)

size_t koala_workspace_bytes(const koala_config *cfg) {
  char why[128];
  if (!config_ok(cfg, why, sizeof(why))) return 0;
  koala_ctx tmp;
  return carve(&tmp, *cfg, nullptr);
}

int koala_init(const koala_config *cfg, const koala_weights *w, const koala_state *st,
               void *cuda_stream, koala_ctx **out) {
  if (!out) return KOALA_E_INVALID;
  *out = nullptr;
  koala_ctx *c = new (std::nothrow) koala_ctx();
  if (!c) return KOALA_E_INVALID;
  *out = c;   // returned even on failure so that koala_last_error() can be read; destroy it either way
  c->err[0] = 0;
  c->host_status = nullptr;
  c->poll_ev = nullptr;
  c->poll_pending = false;
  c->last_status = 0;
  c->u_draft = nullptr;
  c->p_off = 0;
  c->p_slots = 0;
  char why[128];
  if (!config_ok(cfg, why, sizeof(why))) return fail(c, KOALA_E_INVALID, "%s", why);
  if (!w || !st) return fail(c, KOALA_E_INVALID, "null weights or state");
  c->cfg = *cfg;
  const koala_config &g = c->cfg;
  if (!w->embed || !w->lm_head || !w->final_norm || !w->layer_w)
    return fail(c, KOALA_E_INVALID, "missing target weights");
  if (!st->target_k || !st->target_v || !st->seq_len || !st->workspace)
    return fail(c, KOALA_E_INVALID, "missing state pointers");
  if (((uintptr_t)st->workspace & 255u) != 0) return fail(c, KOALA_E_INVALID, "workspace not 256-byte aligned");
  c->st = (cudaStream_t)cuda_stream;
  c->pdl = (g.flags & KOALA_F_NO_PDL) == 0;
  c->use_tc = (g.flags & KOALA_F_NO_TENSOR_CORES) == 0 && g.dtype == KOALA_BF16;
  c->embed = w->embed;
  c->lm_head = w->lm_head;
  c->final_norm = w->final_norm;
  c->fc_w = w->fc_w;
  c->fc_b = w->fc_b;
  auto fill_layers = [](std::vector<LayerW> &dst, const void *const *src, int n) {
    dst.resize(n);
    for (int l = 0; l < n; ++l) {
      const void *const *q = src + (size_t)l * KOALA_LAYER_TENSORS;
      dst[l] = LayerW{q[0], q[1], q[2], q[3], q[4], q[5], q[6], q[7], q[8]};
      for (int i = 0; i < KOALA_LAYER_TENSORS; ++i)
        if (!q[i]) return false;
    }
    return true;
  };
  if (!fill_layers(c->layers, w->layer_w, g.L)) return fail(c, KOALA_E_INVALID, "null target layer tensor");
  if (g.head_kind == KOALA_EAGLE) {
    if (!w->fc_w || !w->fc_b || (g.K > 0 && (!w->draft_layer_w || !st->draft_k || !st->draft_v)))
      return fail(c, KOALA_E_INVALID, "missing EAGLE head weights or cache");
    if (g.K > 0 && !fill_layers(c->draft_layers, w->draft_layer_w, g.K))
      return fail(c, KOALA_E_INVALID, "null draft layer tensor");
  } else {
    if (!w->static_parent || !w->static_level || !w->static_rank)
      return fail(c, KOALA_E_INVALID, "missing static tree");
    if (g.K > 0 && (!w->res_w || !w->res_b)) return fail(c, KOALA_E_INVALID, "missing Medusa blocks");
    const int n = g.n_medusa_heads * g.K;
    c->res_w.assign(w->res_w, w->res_w + n);
    c->res_b.assign(w->res_b, w->res_b + n);
    if (w->medusa_lm) {
      c->medusa_lm.assign(w->medusa_lm, w->medusa_lm + g.n_medusa_heads);
      for (const void *p : c->medusa_lm)
        if (!p) return fail(c, KOALA_E_INVALID, "null Medusa head matrix");
    }
    for (int i = 0; i < n; ++i)
      if (!c->res_w[i] || !c->res_b[i]) return fail(c, KOALA_E_INVALID, "null Medusa block tensor");
    for (int u = 0; u < g.N; ++u) {
      const int p = w->static_parent[u], lv = w->static_level[u], rk = w->static_rank[u];
      const bool ok = u == 0 ? (p == -1 && lv == 0)
                             : (p >= 0 && p < u && lv == w->static_level[p] + 1 && lv <= g.n_medusa_heads &&
                                rk >= 0 && rk < g.topk);
      if (!ok) return fail(c, KOALA_E_INVALID, "malformed static tree at node %d", u);
    }
  }
  c->tk = st->target_k; c->tv = st->target_v; c->dk = st->draft_k; c->dv = st->draft_v;
  c->seq_len = st->seq_len;
  const size_t need = carve(c, g, (unsigned char *)st->workspace);
  if (st->workspace_bytes < need)
    return fail(c, KOALA_E_CAPACITY, "workspace too small: %zu < %zu bytes", st->workspace_bytes, need);
  if (c->use_tc) {
    char e[160];
    if (tc_init_driver(e, sizeof(e)) != 0) return fail(c, KOALA_E_CUDA, "%s", e);
  }
  c->ws_base = (unsigned char *)st->workspace;
  for (size_t off : c->guards) CU_TRY(cudaMemsetAsync(c->ws_base + off, GUARD_PATTERN, GUARD_BYTES, c->st));
  // small state that must start at zero
  CU_TRY(cudaMemsetAsync(c->status, 0, 4 * sizeof(int), c->st));
  CU_TRY(cudaMemsetAsync(c->layer_sync, 0, LAYER_SYNC_WORDS * sizeof(unsigned), c->st));
  memset(c->layer_use, 0, sizeof(c->layer_use));
  c->stream_layers = c->use_tc && (g.flags & KOALA_F_LAYER_KERNEL) != 0;
  CU_TRY(cudaMemsetAsync(c->t.alpha_hits, 0, 128 * sizeof(unsigned long long), c->st));
  CU_TRY(cudaMemsetAsync(c->t.alpha_trials, 0, 128 * sizeof(unsigned long long), c->st));
  CU_TRY(cudaMemsetAsync(c->t.n_pend, 0, g.B * sizeof(int32_t), c->st));
  CU_TRY(cudaMemsetAsync(c->t.root_tok, 0, g.B * sizeof(int32_t), c->st));
  CU_TRY(cudaMemsetAsync(c->t.tree_n, 0, g.B * sizeof(int32_t), c->st));
  if (g.head_kind == KOALA_MEDUSA) {
    CU_TRY(cudaMemcpyAsync(c->s_parent, w->static_parent, g.N * sizeof(int32_t), cudaMemcpyHostToDevice, c->st));
    CU_TRY(cudaMemcpyAsync(c->s_level, w->static_level, g.N * sizeof(int32_t), cudaMemcpyHostToDevice, c->st));
    CU_TRY(cudaMemcpyAsync(c->s_rank, w->static_rank, g.N * sizeof(int32_t), cudaMemcpyHostToDevice, c->st));
    // the copies above read pageable host arrays: they are staged before the call returns
  }
  CU_TRY(cudaHostAlloc((void **)&c->host_status, sizeof(int), cudaHostAllocDefault));
  *c->host_status = 0;
  CU_TRY(cudaEventCreateWithFlags(&c->poll_ev, cudaEventDisableTiming));
  c->phase = PH_READY;
  c->last_pass = -1;
  c->pend_cap = g.N < g.D + 1 ? g.N : g.D + 1;
  c->draft_rows = 0;
  c->expand_mode = 0;
  c->pending = RowScale{nullptr, 0, 0.f, 0.f};
  c->timing = false;
  c->ev_used = 0;
  memset(c->t_bytes, 0, sizeof(c->t_bytes));
  memset(c->t_launches, 0, sizeof(c->t_launches));
  c->last_tree_from_caller = false;
  return KOALA_OK;
}

int koala_draft(koala_ctx *c, int pass) {
  if (!c) return KOALA_E_INVALID;
  const koala_config &g = c->cfg;
  if (g.head_kind == KOALA_MEDUSA) {
    if (pass != 0) return fail(c, KOALA_E_INVALID, "Medusa-style heads draft in the single pass 0");
    if (c->phase != PH_READY) return fail(c, KOALA_E_STATE, "koala_draft(0) must follow koala_init / koala_accept");
    K_TRY(draft_medusa(c));
  } else {
    if (pass < 0 || pass >= g.D) return fail(c, KOALA_E_INVALID, "pass %d outside 0..D-1", pass);
    if (pass == 0 && c->phase != PH_READY)
      return fail(c, KOALA_E_STATE, "koala_draft(0) must follow koala_init / koala_accept");
    if (pass > 0 && !(c->phase == PH_EXPANDED && c->last_pass == pass - 1))
      return fail(c, KOALA_E_STATE, "koala_draft(%d) must follow koala_expand_tree(%d)", pass, pass - 1);
    K_TRY(draft_eagle(c, pass));
  }
  c->phase = PH_DRAFTED;
  c->last_pass = pass;
  return KOALA_OK;
}

int koala_expand_tree(koala_ctx *c, int pass) {
  if (!c) return KOALA_E_INVALID;
  const koala_config &g = c->cfg;
  if (c->phase != PH_DRAFTED || c->last_pass != pass)
    return fail(c, KOALA_E_STATE, "koala_expand_tree(%d) must follow koala_draft(%d)", pass, pass);
  if (c->expand_mode != 2) {
    if (c->u_draft != nullptr && c->draft_rows == g.B) {
      // chain drafts with sampled tokens: token ~ softmax(logits), the distribution is kept
      CU_TRY(sample_rows(LN(c), c->draft_logits, c->u_draft, g.D, pass, c->t.topk_tok, c->t.topk_logp, c->chain_d,
                         g.B, g.V));
    } else {
      CU_TRY(topk_logp(LN(c), c->draft_logits, c->t.topk_tok, c->t.topk_logp, c->draft_rows, g.V, g.topk));
    }
  }
  if (c->expand_mode == 1) return KOALA_OK;
  if (g.head_kind == KOALA_MEDUSA) {
    CU_TRY(expand_static(LN(c), c->t, c->s_parent, c->s_level, c->s_rank, g.B, g.N, g.topk));
    c->phase = PH_TREE;
  } else {
    CU_TRY(expand_dynamic(LN(c), c->t, g.B, g.topk, c->pool, pass, g.D, g.N));
    c->phase = pass == g.D - 1 ? PH_TREE : PH_EXPANDED;
  }
  return KOALA_OK;
}

int koala_verify(koala_ctx *c, const koala_tree *tree) {
  if (!c) return KOALA_E_INVALID;
  const koala_config &g = c->cfg;
  if (tree) {
    if (!tree->tok || !tree->parent || !tree->n_nodes) return fail(c, KOALA_E_INVALID, "null tree arrays");
    if (tree->n_max < 1 || tree->n_max > g.N || tree->stride < tree->n_max)
      return fail(c, KOALA_E_INVALID, "tree n_max %d / stride %d out of range (N = %d)", tree->n_max,
                  tree->stride, g.N);
    CU_TRY(tree_from_caller(LN(c), c->t, tree->tok, tree->parent, tree->n_nodes, tree->stride, g.B, g.N,
                            c->status));
    c->last_tree_from_caller = true;
    c->pend_cap = tree->n_max;
  } else {
    if (c->phase != PH_TREE) return fail(c, KOALA_E_STATE, "no drafted tree: run draft/expand_tree first");
    c->last_tree_from_caller = false;
    c->pend_cap = g.N < g.D + 1 ? g.N : g.D + 1;
  }
  // a single sequence with a short caller tree (a prompt chunk, a one-node step) runs n_max rows;
  // with several sequences row b * N + u is fixed, so all B * N rows run
  const int rows = (tree && g.B == 1) ? tree->n_max : g.N;
  const int R = g.B == 1 ? rows : g.B * g.N;
  c->pending = RowScale{nullptr, 0, 0.f, 0.f};
  CU_TRY(tree_ancestors(LN(c), c->t, g.B, g.N));
  CU_TRY(plan_verify(LN(c), c->t, c->p, c->seq_len, g.B, g.N, g.head_dim, g.rope_base, g.S_max, c->status));
  if ((g.H % 4) == 0 && g.H <= 8192) {
    // the embedding rows in the deferred form: their RMSNorm scale is applied by the first layer's consumer
    CU_TRY(embed_update(LN(c), g.dtype, c->p.row_tok, c->embed, c->layers[0].attn_norm, c->x, c->xn, c->sumsq[1],
                        R, g.H, g.V));
    c->pending = RowScale{c->sumsq[1], (g.H + 1023) / 1024, 1.f / (float)g.H, g.rms_eps};
  } else {
    CU_TRY(embed_norm(LN(c), g.dtype, c->p.row_tok, c->embed, c->layers[0].attn_norm, c->x, c->xn, R, g.H, g.V,
                      g.rms_eps));
  }
  K_TRY(run_layers(c, c->layers, g.L, c->tk, c->tv, R, rows, c->final_norm, c->lmin, c->verify_hid));
  GemmMats lm{{c->lm_head, nullptr, nullptr}, {g.V, 0, 0}, 1};
  K_TRY(do_gemm(c, c->lmin, g.H, lm, R, c->verify_logits, g.V, nullptr));
  CU_TRY(argmax_rows(LN(c), c->verify_logits, c->verify_tgt, R, g.V));
  c->phase = PH_VERIFIED;
  return KOALA_OK;
}

int koala_accept(koala_ctx *c, const int32_t *forced_len, int32_t *out_tokens, int32_t out_stride,
                 int32_t *out_len) {
  if (!c) return KOALA_E_INVALID;
  const koala_config &g = c->cfg;
  if (!out_tokens || !out_len || out_stride < 1) return fail(c, KOALA_E_INVALID, "null outputs");
  if (c->phase != PH_VERIFIED) return fail(c, KOALA_E_STATE, "koala_accept must follow koala_verify");
  CU_TRY(accept_walk(LN(c), c->t, c->verify_tgt, c->verify_hid, forced_len, c->seq_len, out_tokens,
                     out_stride, out_len, g.B, g.N, g.H));
  CU_TRY(kv_compact(LN(c), g.dtype, c->t, c->tk, c->tv, g.L, g.B, g.N, g.n_heads, g.head_dim, g.S_max));
  c->phase = PH_READY;
  c->last_pass = -1;
  return KOALA_OK;
}

int koala_set_sampling(koala_ctx *c, const float *u_draft) {
  if (!c) return KOALA_E_INVALID;
  if (u_draft != nullptr && c->chain_d == nullptr)
    return fail(c, KOALA_E_INVALID, "sampled drafts need an EAGLE-style head with topk = 1 (chain drafts)");
  c->u_draft = u_draft;
  return KOALA_OK;
}

int koala_accept_sampled(koala_ctx *c, const float *u_accept, const float *u_bonus, int32_t *out_tokens,
                         int32_t out_stride, int32_t *out_len) {
  if (!c) return KOALA_E_INVALID;
  const koala_config &g = c->cfg;
  if (!u_accept || !u_bonus || !out_tokens || !out_len || out_stride < 1) return fail(c, KOALA_E_INVALID, "null arguments");
  if (c->chain_d == nullptr || c->u_draft == nullptr)
    return fail(c, KOALA_E_STATE, "koala_accept_sampled needs sampled chain drafts (koala_set_sampling)");
  if (c->phase != PH_VERIFIED || c->last_tree_from_caller)
    return fail(c, KOALA_E_STATE, "koala_accept_sampled must follow koala_verify of the drafted chain");
  CU_TRY(accept_sampled(LN(c), c->t, c->verify_logits, c->verify_hid, c->chain_d, u_accept, u_bonus, c->seq_len,
                        out_tokens, out_stride, out_len, g.B, g.N, g.H, g.V, g.D, c->status));
  CU_TRY(kv_compact(LN(c), g.dtype, c->t, c->tk, c->tv, g.L, g.B, g.N, g.n_heads, g.head_dim, g.S_max));
  c->phase = PH_READY;
  c->last_pass = -1;
  return KOALA_OK;
}

int koala_accept_stats(koala_ctx *c, uint64_t *hits, uint64_t *trials, int32_t n_max, int32_t reset) {
  if (!c) return KOALA_E_INVALID;
  if (n_max < 0 || n_max > 128 || (n_max > 0 && (!hits || !trials))) return fail(c, KOALA_E_INVALID, "bad n_max / null outputs");
  if (n_max > 0) {
    CU_TRY(cudaMemcpyAsync(hits, c->t.alpha_hits, (size_t)n_max * sizeof(uint64_t), cudaMemcpyDeviceToHost, c->st));
    CU_TRY(cudaMemcpyAsync(trials, c->t.alpha_trials, (size_t)n_max * sizeof(uint64_t), cudaMemcpyDeviceToHost, c->st));
  }
  if (reset) {
    CU_TRY(cudaMemsetAsync(c->t.alpha_hits, 0, 128 * sizeof(unsigned long long), c->st));
    CU_TRY(cudaMemsetAsync(c->t.alpha_trials, 0, 128 * sizeof(unsigned long long), c->st));
  }
  CU_TRY(cudaStreamSynchronize(c->st));
  return KOALA_OK;
}

int koala_buffers(koala_ctx *c, koala_buffer_table *o) {
  if (!c || !o) return KOALA_E_INVALID;
  memset(o, 0, sizeof(*o));
  o->draft_logits = c->draft_logits;
  o->draft_feat = c->cfg.head_kind == KOALA_MEDUSA ? c->mx : c->feat[c->last_pass >= 0 ? (c->last_pass & 1) : 0];
  o->topk_tok = c->t.topk_tok;
  o->topk_logp = c->t.topk_logp;
  o->cand_tok = c->t.cand_tok;
  o->cand_parent = c->t.cand_parent;
  o->cand_score = c->t.cand_score;
  o->frontier = c->t.frontier;
  o->tree_tok = c->t.tree_tok;
  o->tree_parent = c->t.tree_parent;
  o->tree_level = c->t.tree_level;
  o->tree_score = c->t.tree_score;
  o->tree_n = c->t.tree_n;
  o->verify_logits = c->verify_logits;
  o->verify_hid = c->verify_hid;
  o->verify_tgt = c->verify_tgt;
  o->root_tok = c->t.root_tok;
  o->pend_hid = c->t.pend_hid;
  o->pend_tok = c->t.pend_tok;
  o->n_pend = c->t.n_pend;
  o->acc_path = c->t.acc_path;
  o->pool = c->pool;
  o->draft_rows = c->draft_rows;
  return KOALA_OK;
}

int koala_set_option(koala_ctx *c, int option, int value) {
  if (!c) return KOALA_E_INVALID;
  if (option == KOALA_OPT_EXPAND_MODE && value >= 0 && value <= 2) {
    c->expand_mode = value;
    return KOALA_OK;
  }
  if (option == KOALA_OPT_TIMING && (value == 0 || value == 1)) {
    c->timing = value == 1;
    c->ev_used = 0;
    memset(c->t_bytes, 0, sizeof(c->t_bytes));
    memset(c->t_launches, 0, sizeof(c->t_launches));
    return KOALA_OK;
  }
  return fail(c, KOALA_E_INVALID, "unknown option %d / value %d", option, value);
}

int koala_timing_read(koala_ctx *c, koala_timing *out) {
  if (!c || !out) return KOALA_E_INVALID;
  memset(out, 0, sizeof(*out));
  CU_TRY(cudaStreamSynchronize(c->st));
  for (size_t i = 0; i < c->ev_used; ++i) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, c->ev[2 * i], c->ev[2 * i + 1]) == cudaSuccess) out->ms[c->ev_cls[i]] += ms;
  }
  for (int k = 0; k < 3; ++k) {
    out->bytes[k] = c->t_bytes[k];
    out->launches[k] = c->t_launches[k];
  }
  (void)cudaGetLastError();
  return KOALA_OK;
}

void koala_set_tuning(int key, int value) { koala::tc_set_tuning(key, value); }

uint64_t koala_launch_count(void) { return (uint64_t)koala::g_launches; }

int koala_selftest_timeout(koala_ctx *c, int limit_cycles) {
  if (!c) return KOALA_E_INVALID;
  if (limit_cycles < 1 || limit_cycles > 100000000) return fail(c, KOALA_E_INVALID, "limit_cycles outside 1..1e8");
  CU_TRY(koala::selftest_timeout(LN(c), c->status, (long long)limit_cycles));
  return KOALA_OK;
}

int koala_debug_check_guards(koala_ctx *c, int *n_guards, int *n_damaged) {
  if (!c || !n_guards || !n_damaged) return KOALA_E_INVALID;
  CU_TRY(cudaStreamSynchronize(c->st));
  std::vector<unsigned char> host(GUARD_BYTES);
  int bad = 0;
  for (size_t off : c->guards) {
    CU_TRY(cudaMemcpy(host.data(), c->ws_base + off, GUARD_BYTES, cudaMemcpyDeviceToHost));
    bool same = true;
    for (unsigned char v : host) same = same && v == (unsigned char)GUARD_PATTERN;
    bad += same ? 0 : 1;
  }
  *n_guards = (int)c->guards.size();
  *n_damaged = bad;
  return KOALA_OK;
}

int koala_poll(koala_ctx *c, int *done, int *device_status) {
  if (!c) return KOALA_E_INVALID;
  if (c->poll_pending && cudaEventQuery(c->poll_ev) == cudaSuccess) {
    c->last_status = *c->host_status;
    c->poll_pending = false;
  }
  if (!c->poll_pending) {
    CU_TRY(cudaMemcpyAsync(c->host_status, c->status, sizeof(int), cudaMemcpyDeviceToHost, c->st));
    CU_TRY(cudaEventRecord(c->poll_ev, c->st));
    c->poll_pending = true;
    if (cudaEventQuery(c->poll_ev) == cudaSuccess) {
      c->last_status = *c->host_status;
      c->poll_pending = false;
    }
  }
  if (done) *done = c->poll_pending ? 0 : 1;
  if (device_status) *device_status = c->last_status;
  (void)cudaGetLastError();
  return KOALA_OK;
}

const char *koala_last_error(const koala_ctx *c) { return c ? c->err : "null context"; }

void koala_destroy(koala_ctx *c) {
  if (!c) return;
  if (c->host_status) cudaFreeHost(c->host_status);
  if (c->poll_ev) cudaEventDestroy(c->poll_ev);
  for (cudaEvent_t e : c->ev) cudaEventDestroy(e);
  koala::tc_forget_maps();
  delete c;
}

int koala_gemm_x_rows(int M, int has_lo) {
  if (M < 1) return 0;
  const int tt_max = (has_lo && M <= 128) ? 128 : 256;    // as in the multiply: pairs of more than 128 tokens use 256-token tiles
  int tt = (M + 15) / 16 * 16;
  if (tt > tt_max) tt = tt_max;
  return (M + tt - 1) / tt * tt;
}

size_t koala_gemm_scratch_bytes(int M, int N_out, int K_in) {
  (void)K_in;
  if (M < 1 || N_out < 1) return 0;
  return (size_t)MAX_SPLIT * ((size_t)M + 16) * (size_t)N_out * sizeof(float);
}

int koala_gemm_bf16(const void *X, const void *X_lo, const void *W, float *Y, int ldy, int M, int N_out, int K_in,
                    void *scratch, size_t scratch_bytes, int use_tensor_cores, int split_k,
                    void *cuda_stream, int *device_status) {
  if (!X || !W || !Y || M < 1 || N_out < 1 || K_in < 1 || ldy < N_out) return KOALA_E_INVALID;
  Launch L{(cudaStream_t)cuda_stream, false};
  GemmMats m{{W, nullptr, nullptr}, {N_out, 0, 0}, 1};
  Operand Xo{const_cast<void *>(X), const_cast<void *>(X_lo)};
  if (!use_tensor_cores) return gemm_simt(L, KOALA_BF16, Xo, m, K_in, M, Y, ldy) == cudaSuccess ? KOALA_OK : KOALA_E_CUDA;
  char e[160];
  if (tc_init_driver(e, sizeof(e)) != 0) return KOALA_E_CUDA;
  if (!tc_supported(m, K_in)) return KOALA_E_UNSUPPORTED;
  if (split_k > MAX_SPLIT) split_k = MAX_SPLIT;
  if (split_k < 0) split_k = 0;
  // X must hold whole token tiles (koala_gemm_x_rows)
  const int rows_alloc = koala_gemm_x_rows(M, X_lo != nullptr);
  if (split_k == 1)
    return gemm_tc(L, Xo, rows_alloc, m, K_in, M, Y, ldy, 1, 0, device_status, 1, nullptr) == cudaSuccess
               ? KOALA_OK : KOALA_E_CUDA;
  const size_t stride = (size_t)M * N_out;
  if (!scratch || scratch_bytes < (size_t)MAX_SPLIT * stride * sizeof(float)) return KOALA_E_CAPACITY;
  SplitIn s;
  if (gemm_tc(L, Xo, rows_alloc, m, K_in, M, (float *)scratch, N_out, split_k, stride, device_status, MAX_SPLIT,
              &s) != cudaSuccess)
    return KOALA_E_CUDA;
  return reduce_splits(L, s, Y, ldy, M, N_out) == cudaSuccess ? KOALA_OK : KOALA_E_CUDA;
}

#pragma GCC visibility pop
}  // extern "C"
