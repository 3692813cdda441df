// Integer bookkeeping of the candidate tree: caller trees, ancestor masks, per-row plans of the
// forwards, dynamic / static expansion, greedy acceptance and KV compaction.
// One thread block per sequence unless stated otherwise; all of it is latency-bound.
#include "common.cuh"

namespace koala {
namespace {

constexpr int E_INVALID = 1, E_CAPACITY = 3;

__device__ __forceinline__ void set_bit(uint64_t *m, int bit) {
  if (bit < 64) m[0] |= 1ull << bit;
  else if (bit < 128) m[1] |= 1ull << (bit - 64);
}

__device__ __forceinline__ void write_rope(float2 *rope, size_t row, int pos, int head_dim,
                                           float rope_base, int lane, int nthreads) {
  const int half = head_dim >> 1;
  for (int i = lane; i < half; i += nthreads) {
    const double inv = pow((double)rope_base, -2.0 * (double)i / (double)head_dim);
    double s, c;
    sincos((double)pos * inv, &s, &c);
    rope[row * half + i] = make_float2((float)c, (float)s);
  }
}

// ------------------------------------------------------------------------------- caller tree
__global__ void tree_from_caller_kernel(TreeBufs t, const int32_t *tok,
                                        const int32_t *parent,
                                        const int32_t *n_nodes, int stride, int N,
                                        int *status) {
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x;
  int n = n_nodes[b];
  if (n < 1 || n > N) {
    if (threadIdx.x == 0 && status) atomicMax(status, E_INVALID);
    n = n < 1 ? 1 : N;
  }
  for (int u = threadIdx.x; u < N; u += blockDim.x) {
    int p = -1, tk = 0;
    if (u < n) {
      tk = tok[(size_t)b * stride + u];
      p = u == 0 ? -1 : parent[(size_t)b * stride + u];
      if (u > 0 && (p < 0 || p >= u)) {
        if (status) atomicMax(status, E_INVALID);
        p = u - 1;
      }
    }
    t.tree_tok[b * N + u] = tk;
    t.tree_parent[b * N + u] = p;
    t.tree_score[b * N + u] = 0.f;
  }
  if (threadIdx.x == 0) t.tree_n[b] = n;
  __syncthreads();
  for (int u = threadIdx.x; u < N; u += blockDim.x) {
    int lvl = 0;
    if (u < n) {
      int v = t.tree_parent[b * N + u];
      while (v >= 0 && lvl < N) {
        ++lvl;
        v = t.tree_parent[b * N + v];
      }
    }
    t.tree_level[b * N + u] = lvl;
  }
}

__global__ void tree_ancestors_kernel(TreeBufs t, int N) {
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x;
  const int n = t.tree_n[b];
  for (int u = threadIdx.x; u < N; u += blockDim.x) {
    uint64_t m[2] = {0ull, 0ull};
    if (u < n) {
      int v = u, steps = 0;
      while (v >= 0 && steps <= N) {
        set_bit(m, v);
        v = t.tree_parent[b * N + v];
        ++steps;
      }
    }
    t.tree_anc[((size_t)b * N + u) * 2] = m[0];
    t.tree_anc[((size_t)b * N + u) * 2 + 1] = m[1];
  }
}

// ------------------------------------------------------------------------------- plans
__global__ void plan_verify_kernel(TreeBufs t, PlanBufs p, const int32_t *seq_len,
                                   int N, int head_dim, float rope_base, int S_max, int *status) {
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x;
  const int S = seq_len[b];
  const int n = t.tree_n[b];
  const bool fits = S >= 0 && S + n <= S_max;
  if (!fits && threadIdx.x == 0 && status) atomicMax(status, E_CAPACITY);
  if (threadIdx.x == 0) {
    p.ctx_len[b] = fits ? S : 0;
    p.kv_len[b] = fits ? S + n : 0;
  }
  {
    const int u = blockIdx.y;
    const size_t r = (size_t)b * N + u;
    const int lvl = t.tree_level[r];
    if (threadIdx.x == 0) {
      p.pos[r] = S + lvl;
      p.slot[r] = (fits && u < n) ? S + u : -1;
      p.mask[r * 2] = t.tree_anc[r * 2];
      p.mask[r * 2 + 1] = t.tree_anc[r * 2 + 1];
      p.row_tok[r] = t.tree_tok[r];
      p.row_src[r] = (int)r;
    }
    write_rope(p.rope, r, S + lvl, head_dim, rope_base, threadIdx.x, blockDim.x);
  }
}

// Draft pass 0 (EAGLE-style): the positions accepted last, as a chain on top of the head's cache.
__global__ void plan_draft0_kernel(TreeBufs t, PlanBufs p, const int32_t *seq_len,
                                   int N, int rows, int head_dim, float rope_base, int S_max,
                                   int *status) {
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x;
  const int S = seq_len[b];
  int n = t.n_pend[b];
  bool ok = n >= 1 && n <= rows && S - n >= 0 && S <= S_max;
  if (!ok && threadIdx.x == 0 && status) atomicMax(status, E_INVALID);
  if (!ok) n = 0;
  if (threadIdx.x == 0) {
    p.ctx_len[b] = ok ? S - n : 0;
    p.kv_len[b] = ok ? S : 0;
    p.last_row[b] = b * rows + (n > 0 ? n - 1 : 0);
  }
  {
    const int i = blockIdx.y;
    const size_t r = (size_t)b * rows + i;
    const int pos = S - n + i;
    if (threadIdx.x == 0) {
      p.pos[r] = pos;
      p.slot[r] = i < n ? pos : -1;
      uint64_t m[2] = {0ull, 0ull};
      if (i < 64) m[0] = (i == 63) ? ~0ull : ((1ull << (i + 1)) - 1);
      else { m[0] = ~0ull; m[1] = (i == 127) ? ~0ull : ((1ull << (i - 63)) - 1); }
      p.mask[r * 2] = m[0];
      p.mask[r * 2 + 1] = m[1];
      p.row_tok[r] = (i < n - 1) ? t.pend_tok[b * N + i] : t.root_tok[b];
      p.row_src[r] = b * N + (i < N ? i : N - 1);
    }
    write_rope(p.rope, r, pos < 0 ? 0 : pos, head_dim, rope_base, threadIdx.x, blockDim.x);
  }
}

// Medusa-style draft: every head reads the hidden state of the last accepted position.
__global__ void plan_medusa_kernel(TreeBufs t, PlanBufs p, int B, int N, int heads) {
  pdl_launch_dependents();
  pdl_wait();
  const int i = threadIdx.x;
  if (i >= heads * B) return;
  const int b = i % B;
  int n = t.n_pend[b];
  n = n < 1 ? 1 : (n > N ? N : n);
  p.row_src[i] = b * N + n - 1;
}

// Draft pass p >= 1: the k frontier candidates of level p.
__global__ void plan_draft_p_kernel(TreeBufs t, PlanBufs p, const int32_t *seq_len,
                                    int k, int pool, int pass, int head_dim, float rope_base,
                                    int S_max, int *status) {
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x;
  const int S = seq_len[b];
  const bool fits = S >= 0 && S + pass * k <= S_max;
  if (!fits && threadIdx.x == 0 && status) atomicMax(status, E_CAPACITY);
  if (threadIdx.x == 0) {
    p.ctx_len[b] = fits ? S : 0;
    p.kv_len[b] = fits ? S + pass * k : 0;
  }
  {
    const int i = blockIdx.y;
    const size_t r = (size_t)b * k + i;
    const int pos = S + pass - 1;
    if (threadIdx.x == 0) {
      const int cid = t.frontier[b * k + i];
      const int par = t.cand_parent[(size_t)b * pool + cid];
      p.pos[r] = pos;
      p.slot[r] = fits ? S + (pass - 1) * k + i : -1;
      p.mask[r * 2] = t.front_mask[r * 2];
      p.mask[r * 2 + 1] = t.front_mask[r * 2 + 1];
      p.row_tok[r] = t.cand_tok[(size_t)b * pool + cid];
      // the parent's predicted feature: row (slot of the parent in the previous pass)
      const int pslot = par < 0 ? 0 : t.front_row[(size_t)b * pool + par] - (pass - 2) * k;
      p.row_src[r] = b * k + pslot;
    }
    write_rope(p.rope, r, pos, head_dim, rope_base, threadIdx.x, blockDim.x);
  }
}

// ------------------------------------------------------------------------------- dynamic expansion
// Shared scratch: scores and flags of the candidates being ranked.
__global__ void __launch_bounds__(1024)
expand_dynamic_kernel(TreeBufs t, int k, int pool, int pass, int D, int N) {
  extern __shared__ unsigned char smem_raw[];
  float *s_score = reinterpret_cast<float *>(smem_raw);            // [pool]
  int *s_node = reinterpret_cast<int *>(s_score + pool);           // [pool] node index or -1
  int *s_front = s_node + pool;                                    // [k] old frontier ids
  uint64_t *s_mask = reinterpret_cast<uint64_t *>(s_front + ((k + 1) & ~1));   // [k][2]
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x;
  const size_t pb = (size_t)b * pool;
  const int tid = threadIdx.x, nt = blockDim.x;
  const int kk = k * k;
  if (pass == 0) {
    for (int r = tid; r < k; r += nt) {
      t.cand_tok[pb + r] = t.topk_tok[(size_t)b * k + r];
      t.cand_parent[pb + r] = -1;
      t.cand_level[pb + r] = 1;
      t.cand_rank[pb + r] = r;
      t.cand_score[pb + r] = t.topk_logp[(size_t)b * k + r];
      t.frontier[b * k + r] = r;
      t.front_row[pb + r] = r;
      uint64_t m[2] = {0ull, 0ull};
      set_bit(m, r);
      t.front_mask[((size_t)b * k + r) * 2] = m[0];
      t.front_mask[((size_t)b * k + r) * 2 + 1] = m[1];
    }
  } else {
    const int base = k + (pass - 1) * kk;
    for (int i = tid; i < k; i += nt) {
      s_front[i] = t.frontier[b * k + i];
      s_mask[i * 2] = t.front_mask[((size_t)b * k + i) * 2];
      s_mask[i * 2 + 1] = t.front_mask[((size_t)b * k + i) * 2 + 1];
    }
    __syncthreads();
    for (int e = tid; e < kk; e += nt) {
      const int i = e / k, r = e % k;
      const int par = s_front[i];
      const float sc = t.cand_score[pb + par] + t.topk_logp[((size_t)b * k + i) * k + r];
      t.cand_tok[pb + base + e] = t.topk_tok[((size_t)b * k + i) * k + r];
      t.cand_parent[pb + base + e] = par;
      t.cand_level[pb + base + e] = pass + 1;
      t.cand_rank[pb + base + e] = r;
      t.cand_score[pb + base + e] = sc;
      s_score[e] = sc;
    }
    __syncthreads();
    if (pass < D - 1) {
      // next frontier: the k best new candidates (score descending, then pool order)
      for (int e = tid; e < kk; e += nt) {
        const float sc = s_score[e];
        int rank = 0;
        for (int f = 0; f < kk; ++f) {
          const float sf = s_score[f];
          rank += (sf > sc || (sf == sc && f < e)) ? 1 : 0;
        }
        if (rank < k) {
          const int i = e / k;
          t.frontier[b * k + rank] = base + e;
          t.front_row[pb + base + e] = pass * k + rank;
          uint64_t m[2] = {s_mask[i * 2], s_mask[i * 2 + 1]};
          set_bit(m, pass * k + rank);
          t.front_mask[((size_t)b * k + rank) * 2] = m[0];
          t.front_mask[((size_t)b * k + rank) * 2 + 1] = m[1];
        }
      }
    }
  }
  if (pass != D - 1) return;
  // ---- final selection: the N-1 best candidates of the whole pool, numbered by
  //      (level, parent's node number, rank).  Scores, parents and the per-level ordering keys are
  //      staged in shared memory once; every candidate has a thread of its own (the launcher gives
  //      this pass enough threads), so each ranking loop is one pass over shared memory.
  int *s_par = reinterpret_cast<int *>(s_mask + 2 * k);            // [pool] parent candidate id
  int *s_key = s_par + pool;                                       // [pool] parent's node number * 32 + rank, -1 = dropped
  __syncthreads();
  for (int c = tid; c < pool; c += nt) {
    s_score[c] = t.cand_score[pb + c];
    s_par[c] = t.cand_parent[pb + c];
  }
  __syncthreads();
  for (int c = tid; c < pool; c += nt) {
    const float sc = s_score[c];
    int rank = 0;
    for (int f = 0; f < pool; ++f) {
      const float sf = s_score[f];
      rank += (sf > sc || (sf == sc && f < c)) ? 1 : 0;
    }
    s_node[c] = rank < N - 1 ? -2 : -1;     // -2: kept, number pending
  }
  __syncthreads();
  __shared__ int s_base;
  if (tid == 0) {
    s_base = 1;
    t.tree_tok[b * N] = t.root_tok[b];
    t.tree_parent[b * N] = -1;
    t.tree_level[b * N] = 0;
    t.tree_score[b * N] = 0.f;
  }
  __syncthreads();
  for (int lvl = 1; lvl <= D; ++lvl) {
    const int lo = lvl == 1 ? 0 : k + (lvl - 2) * kk;
    const int hi = lvl == 1 ? k : k + (lvl - 1) * kk;
    const int base_node = s_base;
    // ordering key of every kept candidate of the level (the parents already have their numbers)
    for (int c = lo + tid; c < hi; c += nt) {
      const int par = s_par[c];
      const int rk = lvl == 1 ? c : (c - lo) % k;
      s_key[c] = s_node[c] == -2 ? (par < 0 ? 0 : s_node[par]) * 32 + rk : -1;
    }
    __syncthreads();
    int kept_here = 0;
    for (int c = lo + tid; c < hi; c += nt) {
      const int key = s_key[c];
      if (key < 0) continue;
      int before = 0;
      for (int f = lo; f < hi; ++f) {
        const int kf = s_key[f];
        before += (kf >= 0 && kf < key) ? 1 : 0;
      }
      const int node = base_node + before;
      s_node[c] = node;                     // read by the next level only (after the barrier below)
      t.tree_tok[b * N + node] = t.cand_tok[pb + c];
      t.tree_parent[b * N + node] = key >> 5;
      t.tree_level[b * N + node] = lvl;
      t.tree_score[b * N + node] = s_score[c];
      ++kept_here;
    }
    if (kept_here) atomicAdd(&s_base, kept_here);
    __syncthreads();
  }
  const int n = s_base;
  if (tid == 0) t.tree_n[b] = n;
  for (int u = n + tid; u < N; u += nt) {
    t.tree_tok[b * N + u] = 0;
    t.tree_parent[b * N + u] = -1;
    t.tree_level[b * N + u] = 0;
    t.tree_score[b * N + u] = 0.f;
  }
}

__global__ void expand_static_kernel(TreeBufs t, const int32_t *__restrict__ s_parent,
                                     const int32_t *__restrict__ s_level,
                                     const int32_t *__restrict__ s_rank, int B, int N, int k) {
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x;
  for (int u = threadIdx.x; u < N; u += blockDim.x) {
    const int lvl = s_level[u];
    t.tree_tok[b * N + u] =
        u == 0 ? t.root_tok[b] : t.topk_tok[((size_t)(lvl - 1) * B + b) * k + s_rank[u]];
    t.tree_parent[b * N + u] = s_parent[u];
    t.tree_level[b * N + u] = lvl;
    t.tree_score[b * N + u] = 0.f;
  }
  if (threadIdx.x == 0) t.tree_n[b] = N;
}

// ------------------------------------------------------------------------------- acceptance
__global__ void accept_walk_kernel(TreeBufs t, const int32_t *tgt,
                                   const float *hid,
                                   const int32_t *forced_len, int32_t *seq_len,
                                   int32_t *out_tokens, int out_stride, int32_t *out_len, int N,
                                   int H) {
  __shared__ int s_path[128];
  __shared__ int s_len;
  __shared__ int s_par[128], s_tok[128], s_tgt[128];
  __shared__ int s_last;
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x;
  const int n = t.tree_n[b] < 128 ? t.tree_n[b] : 128;
  for (int v = threadIdx.x; v < n; v += blockDim.x) {
    s_par[v] = t.tree_parent[b * N + v];
    s_tok[v] = t.tree_tok[b * N + v];
    s_tgt[v] = tgt[b * N + v];
  }
  __syncthreads();
  if (threadIdx.x < 32) {
    // warp 0 walks down from the root; its lanes look at the children of the current node together
    const int lane = threadIdx.x;
    const int f = forced_len ? forced_len[b] : 0;
    int u = 0, len = 1;
    if (lane == 0) s_path[0] = 0;
    while (true) {
      if (f > 0 && len >= f) break;
      const int want = s_tgt[u];
      int match = 0x7fffffff, first = 0x7fffffff;       // smallest matching child, smallest child
      for (int v = u + 1 + lane; v < n; v += 32) {
        if (s_par[v] != u) continue;
        first = first < v ? first : v;
        if (s_tok[v] == want) match = match < v ? match : v;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const int m2 = __shfl_xor_sync(0xffffffffu, match, o), f2 = __shfl_xor_sync(0xffffffffu, first, o);
        match = match < m2 ? match : m2;
        first = first < f2 ? first : f2;
      }
      int nxt = match != 0x7fffffff ? match : -1;
      if (nxt < 0 && f > 0 && first != 0x7fffffff) nxt = first;
      if (nxt < 0) break;
      if (lane == 0) s_path[len] = nxt;
      ++len;
      u = nxt;
    }
    if (lane == 0) { s_len = len; s_last = u; }
    // position-wise acceptance (the n-alpha metric): position n was offered if the walk reached
    // depth n-1 and that node has a child, and hit if the walk went on to depth n
    int child = 0;
    for (int v = u + 1 + lane; v < n; v += 32) child |= (s_par[v] == u);
    child = __any_sync(0xffffffffu, child);
    if (t.alpha_hits != nullptr) {
      for (int i = 1 + lane; i < len && i <= 128; i += 32) {
        atomicAdd(&t.alpha_hits[i - 1], 1ull);
        atomicAdd(&t.alpha_trials[i - 1], 1ull);
      }
      if (lane == 0 && child && len <= 128) atomicAdd(&t.alpha_trials[len - 1], 1ull);
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const int len = s_len, u = s_last;
    const int bonus = s_tgt[u];
    const int S = seq_len[b];
    s_len = len;
    for (int i = 0; i < len; ++i) {
      t.acc_path[b * N + i] = s_path[i];
      if (i >= 1) {
        const int tk = s_tok[s_path[i]];
        t.pend_tok[b * N + i - 1] = tk;
        if (i - 1 < out_stride) out_tokens[(size_t)b * out_stride + i - 1] = tk;
      }
    }
    if (len - 1 < out_stride) out_tokens[(size_t)b * out_stride + len - 1] = bonus;
    out_len[b] = len;
    t.acc_len[b] = len;
    t.acc_S[b] = S;
    t.n_pend[b] = len;
    t.root_tok[b] = bonus;
    seq_len[b] = S + len;
  }
  __syncthreads();
  const int len = s_len;
  for (int i = 0; i < len; ++i) {
    const float *src = hid + ((size_t)b * N + s_path[i]) * H;
    float *dst = t.pend_hid + ((size_t)b * N + i) * H;
    if ((H & 3) == 0) {
      for (int d = threadIdx.x; d < (H >> 2); d += blockDim.x)
        reinterpret_cast<float4 *>(dst)[d] = reinterpret_cast<const float4 *>(src)[d];
    } else {
      for (int d = threadIdx.x; d < H; d += blockDim.x) dst[d] = src[d];
    }
  }
}

// grid (layers * 2, B, n_heads), block head_dim: thread d moves column d of the accepted rows,
// in path order (path[i] >= i and increasing, so a source is never overwritten before it is read).
template <typename T>
__global__ void kv_compact_kernel(TreeBufs t, T *__restrict__ k_cache, T *__restrict__ v_cache,
                                  int B, int N, int n_heads, int head_dim, int S_max) {
  pdl_launch_dependents();
  pdl_wait();
  const int layer = blockIdx.x >> 1, b = blockIdx.y, h = blockIdx.z, d = threadIdx.x;
  T *cache = (blockIdx.x & 1) ? v_cache : k_cache;
  const int len = t.acc_len[b], S = t.acc_S[b];
  T *base = cache + ((((size_t)layer * B + b) * n_heads + h) * S_max) * head_dim;
  for (int i = 0; i < len; ++i) {
    const int p = t.acc_path[b * N + i];
    if (p == i) continue;
    if (S + p >= S_max) break;
    base[(size_t)(S + i) * head_dim + d] = base[(size_t)(S + p) * head_dim + d];
  }
}

}  // namespace

cudaError_t tree_from_caller(Launch L, TreeBufs t, const int32_t *tok, const int32_t *parent,
                             const int32_t *n_nodes, int stride, int B, int N, int *status) {
  return launch_k(tree_from_caller_kernel, dim3(B), dim3(128), 0, L.st, L.pdl, t, tok, parent,
                  n_nodes, stride, N, status);
}
cudaError_t tree_ancestors(Launch L, TreeBufs t, int B, int N) {
  return launch_k(tree_ancestors_kernel, dim3(B), dim3(128), 0, L.st, L.pdl, t, N);
}
cudaError_t plan_verify(Launch L, TreeBufs t, PlanBufs p, const int32_t *seq_len, int B, int N,
                        int head_dim, float rope_base, int S_max, int *status) {
  return launch_k(plan_verify_kernel, dim3(B, N), dim3(64), 0, L.st, L.pdl, t, p, seq_len, N, head_dim,
                  rope_base, S_max, status);
}
cudaError_t plan_draft0(Launch L, TreeBufs t, PlanBufs p, const int32_t *seq_len, int B, int N,
                        int rows, int head_dim, float rope_base, int S_max, int *status) {
  return launch_k(plan_draft0_kernel, dim3(B, rows), dim3(64), 0, L.st, L.pdl, t, p, seq_len, N, rows,
                  head_dim, rope_base, S_max, status);
}
cudaError_t plan_draft_p(Launch L, TreeBufs t, PlanBufs p, const int32_t *seq_len, int B, int k,
                         int pool, int pass, int head_dim, float rope_base, int S_max, int *status) {
  return launch_k(plan_draft_p_kernel, dim3(B, k), dim3(64), 0, L.st, L.pdl, t, p, seq_len, k, pool,
                  pass, head_dim, rope_base, S_max, status);
}
cudaError_t plan_medusa(Launch L, TreeBufs t, PlanBufs p, int B, int N, int heads) {
  return launch_k(plan_medusa_kernel, dim3(1), dim3(((heads * B + 31) / 32) * 32), 0, L.st, L.pdl, t, p,
                  B, N, heads);
}
cudaError_t expand_dynamic(Launch L, TreeBufs t, int B, int k, int pool, int pass, int D, int N) {
  const size_t smem = (size_t)pool * 16 + (size_t)((k + 1) & ~1) * 4 + (size_t)k * 16 + 16;
  // the last pass ranks the whole pool: a thread per candidate
  int threads = 256;
  if (pass == D - 1)
    while (threads < pool && threads < 1024) threads *= 2;
  return launch_k(expand_dynamic_kernel, dim3(B), dim3(threads), smem, L.st, L.pdl, t, k, pool, pass, D, N);
}
cudaError_t expand_static(Launch L, TreeBufs t, const int32_t *s_parent, const int32_t *s_level,
                          const int32_t *s_rank, int B, int N, int k) {
  return launch_k(expand_static_kernel, dim3(B), dim3(128), 0, L.st, L.pdl, t, s_parent, s_level,
                  s_rank, B, N, k);
}
cudaError_t accept_walk(Launch L, TreeBufs t, const int32_t *verify_tgt, const float *verify_hid,
                        const int32_t *forced_len, int32_t *seq_len, int32_t *out_tokens,
                        int out_stride, int32_t *out_len, int B, int N, int H) {
  return launch_k(accept_walk_kernel, dim3(B), dim3(256), 0, L.st, L.pdl, t, verify_tgt, verify_hid,
                  forced_len, seq_len, out_tokens, out_stride, out_len, N, H);
}
cudaError_t kv_compact(Launch L, int dtype, TreeBufs t, void *k_cache, void *v_cache, int L_layers,
                       int B, int N, int n_heads, int head_dim, int S_max) {
  dim3 grid(L_layers * 2, B, n_heads);
  if (dtype == 0)
    return launch_k(kv_compact_kernel<float>, grid, dim3(head_dim), 0, L.st, L.pdl, t,
                    (float *)k_cache, (float *)v_cache, B, N, n_heads, head_dim, S_max);
  return launch_k(kv_compact_kernel<bf16>, grid, dim3(head_dim), 0, L.st, L.pdl, t, (bf16 *)k_cache,
                  (bf16 *)v_cache, B, N, n_heads, head_dim, S_max);
}

}  // namespace koala
