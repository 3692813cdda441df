// Speculative sampling on chain drafts (Section 2.2 of the paper, the paragraph after Eq. 3):
// drafted tokens are DRAWN from the head's distributions d_i, token i is accepted with probability
// min(1, q_i(x_i) / d_i(x_i)), the first rejected position is redrawn from norm(max(0, q_f - d_f)),
// and if every token is accepted one more is drawn from q_{t+1}.  All random numbers are inputs
// (uniforms in [0, 1)); every draw is an inverse-CDF walk in token-id order.
//   sample_rows_kernel     one row of draft logits -> softmax d (kept), token ~ d, log d(token)
//   accept_sampled_kernel  one sequence: judges the chain, draws the extra token, commits the path
//                          (the same bookkeeping as the greedy acceptance kernel)
#include "common.cuh"

namespace koala {
namespace {

constexpr int NT = 1024;

struct Scratch {          // shared-memory scratch of a block-wide draw
  double part[NT];        // per-thread segment sums
  double base;            // sum before the owner's segment
  double target;
  int owner, result;
  float red[32];
};

__device__ __forceinline__ float block_max_f(float v, float *red) {
  v = warp_max(v);
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  __syncthreads();
  if (lane == 0) red[w] = v;
  __syncthreads();
  float r = red[lane];
  r = warp_max(r);
  return r;
}
__device__ __forceinline__ float block_sum_f(float v, float *red) {
  v = warp_sum(v);
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  __syncthreads();
  if (lane == 0) red[w] = v;
  __syncthreads();
  float r = red[lane];
  r = warp_sum(r);
  return r;
}

// Inverse-CDF draw in index order from the non-negative weights w(0..V-1): the smallest j with
// w(0) + .. + w(j) > u * total.  Thread t owns the contiguous ids [t*seg, (t+1)*seg); thread 0
// adds the 1024 segment sums in order (double) and names the segment that holds the target; that
// segment's thread walks it.  If rounding leaves no such j, the last id with a positive weight.
// Every thread of the block calls this; every thread gets the result.
template <typename F>
__device__ int block_draw(F w, int V, float u, Scratch *sc) {
  const int seg = (V + NT - 1) / NT;
  const int lo = threadIdx.x * seg, hi = lo + seg < V ? lo + seg : V;
  double local = 0.0;
  for (int j = lo; j < hi; ++j) local += (double)w(j);
  __syncthreads();
  sc->part[threadIdx.x] = local;
  __syncthreads();
  if (threadIdx.x == 0) {
    double total = 0.0;
    for (int t = 0; t < NT; ++t) total += sc->part[t];
    const double target = (double)u * total;
    double acc = 0.0;
    int owner = -1, last_pos = 0;
    for (int t = 0; t < NT; ++t) {
      if (sc->part[t] > 0.0) last_pos = t;
      if (owner < 0 && acc + sc->part[t] > target) { owner = t; sc->base = acc; }
      acc += sc->part[t];
    }
    if (owner < 0) { owner = last_pos; sc->base = -1.0; }     // rounding: take the last positive id
    sc->owner = owner;
    sc->target = target;
    sc->result = 0;
  }
  __syncthreads();
  if ((int)threadIdx.x == sc->owner) {
    int res = -1, last = lo;
    if (sc->base >= 0.0) {
      double acc = sc->base;
      for (int j = lo; j < hi; ++j) {
        const double x = (double)w(j);
        if (x > 0.0) last = j;
        acc += x;
        if (acc > sc->target) { res = j; break; }
      }
    } else {
      for (int j = lo; j < hi; ++j)
        if (w(j) > 0.f) last = j;
    }
    sc->result = res >= 0 ? res : last;
  }
  __syncthreads();
  return sc->result;
}

// grid R, block 1024, dynamic shared memory V floats.  Row r of the logits belongs to sequence r
// (chain drafts: one row per sequence); its uniform is u[r * u_stride + u_off], its distribution
// goes to probs[(r * u_stride + u_off) * V ..].
__global__ void __launch_bounds__(NT)
sample_rows_kernel(const float *logits, const float *u, int u_stride, int u_off, int32_t *tok, float *logp,
                   float *probs, int V) {
  extern __shared__ float srow[];
  __shared__ Scratch sc;
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.x;
  const float *row = logits + (size_t)r * V;
  float mx = -INFINITY;
  for (int j = threadIdx.x; j < V; j += NT) {
    srow[j] = row[j];
    mx = fmaxf(mx, srow[j]);
  }
  mx = block_max_f(mx, sc.red);
  float se = 0.f;
  for (int j = threadIdx.x; j < V; j += NT) se += expf(srow[j] - mx);
  se = block_sum_f(se, sc.red);
  float *pr = probs + ((size_t)r * u_stride + u_off) * V;
  const float inv = 1.f / se;
  for (int j = threadIdx.x; j < V; j += NT) {
    const float p = expf(srow[j] - mx) * inv;
    srow[j] = p;
    pr[j] = p;
  }
  __syncthreads();
  const int idx = block_draw([&](int j) { return srow[j]; }, V, u[(size_t)r * u_stride + u_off], &sc);
  if (threadIdx.x == 0) {
    tok[r] = idx;
    logp[r] = (row[idx] - mx) - logf(se);
  }
}

// grid B, block 1024, dynamic shared memory V floats.
__global__ void __launch_bounds__(NT)
accept_sampled_kernel(TreeBufs t, const float *verify_logits, const float *hid, const float *chain_d,
                      const float *u_accept, const float *u_bonus, int32_t *seq_len, int32_t *out_tokens,
                      int out_stride, int32_t *out_len, int N, int H, int V, int D, int *status) {
  extern __shared__ float srow[];
  __shared__ Scratch sc;
  __shared__ int s_tok[128];
  __shared__ int s_accept;
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x;
  int n = t.tree_n[b] < 128 ? t.tree_n[b] : 128;
  if (n > D + 1) n = D + 1;                       // a chain of at most D drafted tokens
  for (int v = threadIdx.x; v < n; v += NT) {
    s_tok[v] = t.tree_tok[b * N + v];
    if (t.tree_parent[b * N + v] != v - 1 && status) atomicMax(status, 1);     // not a chain: invalid input
  }
  __syncthreads();
  int a = 0;                                      // accepted drafted tokens
  int bonus = 0;
  bool done = false;
  for (int i = 1; i <= n && !done; ++i) {
    // q = softmax of the target's logits at node i - 1 (judges drafted token i, or gives the extra token)
    const float *row = verify_logits + ((size_t)b * N + i - 1) * V;
    float mx = -INFINITY;
    for (int j = threadIdx.x; j < V; j += NT) {
      srow[j] = row[j];
      mx = fmaxf(mx, srow[j]);
    }
    mx = block_max_f(mx, sc.red);
    float se = 0.f;
    for (int j = threadIdx.x; j < V; j += NT) se += expf(srow[j] - mx);
    se = block_sum_f(se, sc.red);
    const float inv = 1.f / se;
    __syncthreads();
    if (i == n) {                                 // every drafted token was accepted: draw from q_{t+1}
      bonus = block_draw([&](int j) { return expf(srow[j] - mx) * inv; }, V, u_bonus[b], &sc);
      done = true;
      break;
    }
    const float *d = chain_d + ((size_t)b * D + i - 1) * V;
    if (threadIdx.x == 0) {
      const int x = s_tok[i];
      const float q = expf(srow[x] - mx) * inv;
      s_accept = (u_accept[(size_t)b * D + i - 1] * d[x] < q) ? 1 : 0;
    }
    __syncthreads();
    if (s_accept) {
      ++a;
    } else {                                      // first rejection: redraw from norm(max(0, q - d))
      bonus = block_draw([&](int j) { return fmaxf(0.f, expf(srow[j] - mx) * inv - d[j]); }, V, u_bonus[b], &sc);
      done = true;
    }
    __syncthreads();
  }
  const int len = a + 1;
  if (threadIdx.x == 0) {
    const int S = seq_len[b];
    for (int i = 0; i < len; ++i) {
      t.acc_path[b * N + i] = i;
      if (i >= 1) {
        t.pend_tok[b * N + i - 1] = s_tok[i];
        if (i - 1 < out_stride) out_tokens[(size_t)b * out_stride + i - 1] = s_tok[i];
      }
    }
    if (len - 1 < out_stride) out_tokens[(size_t)b * out_stride + len - 1] = bonus;
    out_len[b] = len;
    t.acc_len[b] = len;
    t.acc_S[b] = S;
    t.n_pend[b] = len;
    t.root_tok[b] = bonus;
    seq_len[b] = S + len;
    if (t.alpha_hits != nullptr) {
      for (int i = 1; i < len; ++i) {
        atomicAdd(&t.alpha_hits[i - 1], 1ull);
        atomicAdd(&t.alpha_trials[i - 1], 1ull);
      }
      if (len < n) atomicAdd(&t.alpha_trials[len - 1], 1ull);
    }
  }
  for (int i = 0; i < len; ++i) {
    const float *src = hid + ((size_t)b * N + i) * H;
    float *dst = t.pend_hid + ((size_t)b * N + i) * H;
    for (int dd = threadIdx.x; dd < H; dd += NT) dst[dd] = src[dd];
  }
}

}  // namespace

cudaError_t sample_rows(Launch L, const float *logits, const float *u, int u_stride, int u_off, int32_t *tok,
                        float *logp, float *probs, int R, int V) {
  static SmemOptIn optin;
  const size_t smem = (size_t)V * sizeof(float);
  cudaError_t e = optin.ensure((const void *)sample_rows_kernel, smem);
  if (e != cudaSuccess) return e;
  return launch_k(sample_rows_kernel, dim3(R), dim3(NT), smem, L.st, L.pdl, logits, u, u_stride, u_off, tok, logp,
                  probs, V);
}

cudaError_t accept_sampled(Launch L, TreeBufs t, const float *verify_logits, const float *verify_hid,
                           const float *chain_d, const float *u_accept, const float *u_bonus, int32_t *seq_len,
                           int32_t *out_tokens, int out_stride, int32_t *out_len, int B, int N, int H, int V, int D,
                           int *status) {
  static SmemOptIn optin;
  const size_t smem = (size_t)V * sizeof(float);
  cudaError_t e = optin.ensure((const void *)accept_sampled_kernel, smem);
  if (e != cudaSuccess) return e;
  return launch_k(accept_sampled_kernel, dim3(B), dim3(NT), smem, L.st, L.pdl, t, verify_logits, verify_hid, chain_d,
                  u_accept, u_bonus, seq_len, out_tokens, out_stride, out_len, N, H, V, D, status);
}

}  // namespace koala
