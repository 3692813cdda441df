// Row-wise kernels of the decoder layers and heads: embedding gather, RMSNorm / residual
// epilogues, RoPE + KV-cache write, SwiGLU, tree-masked attention (CUDA-core version),
// arg-max and top-k with log-probabilities.  All statistics are fp32.
#include "common.cuh"

namespace koala {

namespace {

__device__ __forceinline__ float block_sum(float v, float *red) {
  v = warp_sum(v);
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  if (lane == 0) red[w] = v;
  __syncthreads();
  float t = (threadIdx.x < nw) ? red[threadIdx.x] : 0.f;
  if (w == 0) {
    t = warp_sum(t);
    if (lane == 0) red[0] = t;
  }
  __syncthreads();
  t = red[0];
  __syncthreads();
  return t;
}

__device__ __forceinline__ float silu_f(float v) { return v / (1.f + expf(-v)); }

// Stores v as a matrix-multiply operand.  bf16 operands are kept as a pair hi + lo (lo = the
// rounding residual of hi, itself rounded to bf16), which carries 16 significant bits into the
// tensor cores; fp32 operands are exact and have no lo part.
template <typename T>
__device__ __forceinline__ void store_operand(T *hi, T *lo, size_t i, float v) {
  const T h = from_f<T>(v);
  hi[i] = h;
  if (lo != nullptr) lo[i] = from_f<T>(v - to_f(h));
}

// ------------------------------------------------------------------------------- embedding + norm
template <typename T>
__global__ void embed_norm_kernel(const int32_t *tok, const T *__restrict__ E,
                                  const T *__restrict__ g, float *__restrict__ x,
                                  T *__restrict__ xn, T *__restrict__ xn_lo, int H, int V, float eps) {
  __shared__ float red[32];
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.x;
  int t = tok[r];
  t = t < 0 ? 0 : (t >= V ? V - 1 : t);
  const T *e = E + (size_t)t * H;
  float ss = 0.f;
  for (int i = threadIdx.x; i < H; i += blockDim.x) {
    const float v = to_f(e[i]);
    x[(size_t)r * H + i] = v;
    ss += v * v;
  }
  const float inv = rsqrtf(block_sum(ss, red) / (float)H + eps);
  for (int i = threadIdx.x; i < H; i += blockDim.x)
    store_operand(xn, xn_lo, (size_t)r * H + i, x[(size_t)r * H + i] * inv * to_f(g[i]));
}

// ------------------------------------------------------------------------------- row epilogue
template <typename T>
__global__ void row_epilogue_kernel(int mode, float *__restrict__ x, SplitIn P,
                                    const T *__restrict__ bias, const T *__restrict__ g,
                                    T *__restrict__ xn, T *__restrict__ xn_lo,
                                    float *__restrict__ out_f32, int H, float eps) {
  __shared__ float red[32];
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.x;
  float *xr = x + (size_t)r * H;
  float ss = 0.f;
  for (int i = threadIdx.x; i < H; i += blockDim.x) {
    float p = P.at(r, i);
    float v;
    if (mode == 0) v = xr[i] + p;
    else if (mode == 1) v = p + to_f(bias[i]);
    else v = xr[i] + silu_f(p + to_f(bias[i]));
    xr[i] = v;
    ss += v * v;
  }
  float inv = 1.f;
  if (g != nullptr) inv = rsqrtf(block_sum(ss, red) / (float)H + eps);
  for (int i = threadIdx.x; i < H; i += blockDim.x) {
    float n = xr[i];
    if (g != nullptr) n = n * inv * to_f(g[i]);
    if (xn != nullptr) store_operand(xn, xn_lo, (size_t)r * H + i, n);
    if (out_f32 != nullptr) out_f32[(size_t)r * H + i] = n;
  }
}

// Vectorised variant for H % 4 == 0: one CTA per row, every thread owns up to VPT groups of four
// consecutive columns, keeps them in registers between the two passes and issues all split-K
// partial loads of a group back to back.
// (The first eight partial loads are issued before any is used - one trip to L2 instead of one
// per partial; the additions keep the slot order.)
template <int AHEAD = 8>
__device__ __forceinline__ float4 split_sum4(const SplitIn &P, int r, int c) {
  const float *q = P.p + (size_t)r * P.ld + c;
  const int k = P.count(c);
  float4 u[AHEAD];
#pragma unroll
  for (int s = 0; s < AHEAD; ++s)
    u[s] = s < k ? *reinterpret_cast<const float4 *>(q + (size_t)s * P.stride) : make_float4(0.f, 0.f, 0.f, 0.f);
  float4 v = u[0];
#pragma unroll
  for (int s = 1; s < AHEAD; ++s) {
    if (s < k) { v.x += u[s].x; v.y += u[s].y; v.z += u[s].z; v.w += u[s].w; }
  }
  for (int s = AHEAD; s < k; ++s) {
    const float4 w = *reinterpret_cast<const float4 *>(q + (size_t)s * P.stride);
    v.x += w.x; v.y += w.y; v.z += w.z; v.w += w.w;
  }
  return v;
}
template <typename T> __device__ __forceinline__ float4 load4(const T *p);
template <> __device__ __forceinline__ float4 load4<float>(const float *p) { return *reinterpret_cast<const float4 *>(p); }
template <> __device__ __forceinline__ float4 load4<bf16>(const bf16 *p) {
  const uint2 u = *reinterpret_cast<const uint2 *>(p);
  const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&u.x));
  const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&u.y));
  return make_float4(a.x, a.y, b.x, b.y);
}
__device__ __forceinline__ void store_operand4(float *hi, float *lo, size_t i, float4 v) {
  (void)lo;
  *reinterpret_cast<float4 *>(hi + i) = v;
}
__device__ __forceinline__ void store_operand4(bf16 *hi, bf16 *lo, size_t i, float4 v) {
  const __nv_bfloat162 h0 = __floats2bfloat162_rn(v.x, v.y), h1 = __floats2bfloat162_rn(v.z, v.w);
  uint2 u;
  u.x = *reinterpret_cast<const uint32_t *>(&h0);
  u.y = *reinterpret_cast<const uint32_t *>(&h1);
  *reinterpret_cast<uint2 *>(hi + i) = u;
  if (lo != nullptr) {
    const float2 f0 = __bfloat1622float2(h0), f1 = __bfloat1622float2(h1);
    const __nv_bfloat162 l0 = __floats2bfloat162_rn(v.x - f0.x, v.y - f0.y);
    const __nv_bfloat162 l1 = __floats2bfloat162_rn(v.z - f1.x, v.w - f1.y);
    u.x = *reinterpret_cast<const uint32_t *>(&l0);
    u.y = *reinterpret_cast<const uint32_t *>(&l1);
    *reinterpret_cast<uint2 *>(lo + i) = u;
  }
}

template <typename T, int VPT>
__global__ void __launch_bounds__(1024)
row_epilogue_vec_kernel(int mode, float *__restrict__ x, SplitIn P, const T *__restrict__ bias,
                        const T *__restrict__ g, T *__restrict__ xn, T *__restrict__ xn_lo,
                        float *__restrict__ out_f32, int H, float eps) {
  __shared__ float red[32];
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.x;
  float *xr = x + (size_t)r * H;
  float4 v[VPT];
  float ss = 0.f;
#pragma unroll
  for (int k = 0; k < VPT; ++k) {
    const int c = (threadIdx.x + k * blockDim.x) * 4;
    if (c < H) {
      const float4 p = split_sum4(P, r, c);
      float4 o;
      if (mode == 0) {
        const float4 xv = *reinterpret_cast<const float4 *>(xr + c);
        o = make_float4(xv.x + p.x, xv.y + p.y, xv.z + p.z, xv.w + p.w);
      } else {
        const float4 b = load4<T>(bias + c);
        if (mode == 1) {
          o = make_float4(p.x + b.x, p.y + b.y, p.z + b.z, p.w + b.w);
        } else {
          const float4 xv = *reinterpret_cast<const float4 *>(xr + c);
          o = make_float4(xv.x + silu_f(p.x + b.x), xv.y + silu_f(p.y + b.y), xv.z + silu_f(p.z + b.z),
                          xv.w + silu_f(p.w + b.w));
        }
      }
      *reinterpret_cast<float4 *>(xr + c) = o;
      v[k] = o;
      ss += o.x * o.x + o.y * o.y + o.z * o.z + o.w * o.w;
    }
  }
  // the gains are fetched before the block-wide reduction so that their latency hides behind it
  float4 gg[VPT];
#pragma unroll
  for (int k = 0; k < VPT; ++k) {
    const int c = (threadIdx.x + k * blockDim.x) * 4;
    gg[k] = (g != nullptr && c < H) ? load4<T>(g + c) : make_float4(1.f, 1.f, 1.f, 1.f);
  }
  float inv = 1.f;
  if (g != nullptr) inv = rsqrtf(block_sum(ss, red) / (float)H + eps);
#pragma unroll
  for (int k = 0; k < VPT; ++k) {
    const int c = (threadIdx.x + k * blockDim.x) * 4;
    if (c < H) {
      float4 n = v[k];
      if (g != nullptr) {
        n = make_float4(n.x * inv * gg[k].x, n.y * inv * gg[k].y, n.z * inv * gg[k].z, n.w * inv * gg[k].w);
      }
      if (xn != nullptr) store_operand4(xn, xn_lo, (size_t)r * H + c, n);
      if (out_f32 != nullptr) *reinterpret_cast<float4 *>(out_f32 + (size_t)r * H + c) = n;
    }
  }
}

// Residual update with the RMSNorm deferred: grid (chunks of 1024 columns, rows).  Many CTAs per
// row pull the split-K partial sums; the row statistic is left as per-chunk partial sums of
// squares for the consumer of the next GEMM's output (RowScale).
template <typename T>
__global__ void __launch_bounds__(256)
row_update_kernel(float *__restrict__ x, SplitIn P, const T *__restrict__ g, T *__restrict__ xg,
                  T *__restrict__ xg_lo, float *__restrict__ sumsq, int H) {
  __shared__ float red[32];
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.y;
  const int c = (blockIdx.x * 256 + threadIdx.x) * 4;
  float ss = 0.f;
  if (c < H) {
    const float4 gg = load4<T>(g + c);
    const float4 p = split_sum4(P, r, c);
    float *xr = x + (size_t)r * H + c;
    const float4 xv = *reinterpret_cast<const float4 *>(xr);
    const float4 o = make_float4(xv.x + p.x, xv.y + p.y, xv.z + p.z, xv.w + p.w);
    *reinterpret_cast<float4 *>(xr) = o;
    ss = o.x * o.x + o.y * o.y + o.z * o.z + o.w * o.w;
    store_operand4(xg, xg_lo, (size_t)r * H + c, make_float4(o.x * gg.x, o.y * gg.y, o.z * gg.z, o.w * gg.w));
  }
  const float tot = block_sum(ss, red);
  if (threadIdx.x == 0) sumsq[(size_t)r * gridDim.x + blockIdx.x] = tot;
}

template <typename T>
__global__ void __launch_bounds__(256)
resblock_update_kernel(float *__restrict__ x, SplitIn P, HeadTab tab, T *__restrict__ xn, T *__restrict__ xn_lo, int H) {
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.y;
  const int c = (blockIdx.x * 256 + threadIdx.x) * 4;
  if (c >= H) return;
  const int head = r / tab.rows_per_head;
  P.p = tab.p[head];
  const float4 p = split_sum4(P, r - head * tab.rows_per_head, c);
  const float4 b = load4<T>(reinterpret_cast<const T *>(tab.bias[head]) + c);
  float *xr = x + (size_t)r * H + c;
  const float4 xv = *reinterpret_cast<const float4 *>(xr);
  const float4 o = make_float4(xv.x + silu_f(p.x + b.x), xv.y + silu_f(p.y + b.y), xv.z + silu_f(p.z + b.z),
                               xv.w + silu_f(p.w + b.w));
  *reinterpret_cast<float4 *>(xr) = o;
  store_operand4(xn, xn_lo, (size_t)r * H + c, o);
}

// The first rows of a forward in the same deferred form: x <- E[tok]; xg <- T(x * g) (not
// normalised); sumsq[r][chunk] <- partial sums of x^2.  grid (ceil(H / 1024), R), 256 threads.
template <typename T>
__global__ void __launch_bounds__(256)
embed_update_kernel(const int32_t *tok, const T *__restrict__ E, const T *__restrict__ g, float *__restrict__ x,
                    T *__restrict__ xg, T *__restrict__ xg_lo, float *__restrict__ sumsq, int H, int V) {
  __shared__ float red[32];
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.y;
  const int c = (blockIdx.x * 256 + threadIdx.x) * 4;
  float ss = 0.f;
  if (c < H) {
    int t = tok[r];
    t = t < 0 ? 0 : (t >= V ? V - 1 : t);
    const float4 gg = load4<T>(g + c);
    const float4 o = load4<T>(E + (size_t)t * H + c);
    *reinterpret_cast<float4 *>(x + (size_t)r * H + c) = o;
    ss = o.x * o.x + o.y * o.y + o.z * o.z + o.w * o.w;
    store_operand4(xg, xg_lo, (size_t)r * H + c, make_float4(o.x * gg.x, o.y * gg.y, o.z * gg.z, o.w * gg.w));
  }
  const float tot = block_sum(ss, red);
  if (threadIdx.x == 0) sumsq[(size_t)r * gridDim.x + blockIdx.x] = tot;
}

// ------------------------------------------------------------------------------- EAGLE fc input
template <typename T>
__global__ void eagle_concat_kernel(const float *feat_src,
                                    const int32_t *row_src,
                                    const int32_t *row_tok, const T *__restrict__ E,
                                    T *__restrict__ cat, T *__restrict__ cat_lo, int H, int V) {
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.x;
  const int src = row_src[r];
  int t = row_tok[r];
  t = t < 0 ? 0 : (t >= V ? V - 1 : t);
  const float *f = feat_src + (size_t)src * H;
  const T *e = E + (size_t)t * H;
  const size_t base = (size_t)r * 2 * H;
  for (int i = threadIdx.x; i < H; i += blockDim.x) {
    store_operand(cat, cat_lo, base + i, f[i]);
    cat[base + H + i] = e[i];
    if (cat_lo != nullptr) cat_lo[base + H + i] = from_f<T>(0.f);
  }
}

// The same with four elements per thread and the row spread over grid.y CTAs (H % 4 == 0): one
// trip to memory per thread instead of a loop of dependent ones.
template <typename T>
__global__ void eagle_concat_vec_kernel(const float *feat_src, const int32_t *row_src, const int32_t *row_tok,
                                        const T *__restrict__ E, T *__restrict__ cat, T *__restrict__ cat_lo,
                                        int H, int V) {
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.x;
  const int i = (blockIdx.y * blockDim.x + threadIdx.x) * 4;
  if (i >= H) return;
  const int src = row_src[r];
  int t = row_tok[r];
  t = t < 0 ? 0 : (t >= V ? V - 1 : t);
  const float4 f = *reinterpret_cast<const float4 *>(feat_src + (size_t)src * H + i);
  const float4 e = load4<T>(E + (size_t)t * H + i);
  const size_t base = (size_t)r * 2 * H;
  store_operand4(cat, cat_lo, base + i, f);
  store_operand4(cat, cat_lo, base + H + i, e);      // the embedding is exact in T: its residual is zero
}

template <typename T>
__global__ void cast_rows_kernel(const float *src, const int32_t *row_src,
                                 T *__restrict__ dst, T *__restrict__ dst_lo,
                                 float *__restrict__ dst32, int dst32_stride, int H) {
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.x;
  const int s = row_src ? row_src[r] : r;
  for (int i = threadIdx.x; i < H; i += blockDim.x) {
    const float v = src[(size_t)s * H + i];
    store_operand(dst, dst_lo, (size_t)r * H + i, v);
    if (dst32) dst32[(size_t)r * dst32_stride * H + i] = v;
  }
}

__global__ void reduce_splits_kernel(SplitIn P, float *__restrict__ Y, int ldy, int ncols) {
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.y;
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c < ncols) Y[(size_t)r * ldy + c] = P.at(r, c);
}

// ------------------------------------------------------------------------------- RoPE + KV write
// grid (R, n_heads), block head_dim/2: thread i rotates the pair (i, i + head_dim/2).
template <typename T>
__global__ void rope_kv_kernel(SplitIn qkv, RowScale sc, RowPlan plan, float *__restrict__ q_out,
                               bf16 *__restrict__ qp_hi, bf16 *__restrict__ qp_lo,
                               T *__restrict__ k_cache, T *__restrict__ v_cache, int rows_per_seq,
                               int n_heads, int head_dim, int S_max) {
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.x, h = blockIdx.y, i = threadIdx.x;
  const int half = head_dim >> 1, H = n_heads * head_dim;
  const int b = r / rows_per_seq;
  const int slot = plan.slot[r];
  const float2 cs = plan.rope[(size_t)r * half + i];
  const int c0 = h * head_dim + i, c1 = c0 + half;
  const float rs = sc.of(r);
  const float q0 = rs * qkv.at(r, c0), q1 = rs * qkv.at(r, c1);
  const float qr0 = q0 * cs.x - q1 * cs.y, qr1 = q1 * cs.x + q0 * cs.y;
  q_out[(size_t)r * H + c0] = qr0;
  q_out[(size_t)r * H + c1] = qr1;
  if (qp_hi != nullptr) {
    store_operand(qp_hi, qp_lo, (size_t)r * H + c0, qr0);
    store_operand(qp_hi, qp_lo, (size_t)r * H + c1, qr1);
  }
  if (slot < 0 || slot >= S_max) return;
  const float k0 = rs * qkv.at(r, H + c0), k1 = rs * qkv.at(r, H + c1);
  const float v0 = rs * qkv.at(r, 2 * H + c0), v1 = rs * qkv.at(r, 2 * H + c1);
  const size_t base = (((size_t)b * n_heads + h) * S_max + slot) * head_dim;
  k_cache[base + i] = from_f<T>(k0 * cs.x - k1 * cs.y);
  k_cache[base + i + half] = from_f<T>(k1 * cs.x + k0 * cs.y);
  v_cache[base + i] = from_f<T>(v0);
  v_cache[base + i + half] = from_f<T>(v1);
}

// One CTA per row; a thread rotates two adjacent pairs (i, i+1) and (i + half, i + half + 1) of
// one head with 8-byte loads.
__device__ __forceinline__ float2 split_sum2(const SplitIn &P, int r, int c) {
  const float *q = P.p + (size_t)r * P.ld + c;
  const int k = P.count(c);
  float2 u[4];
#pragma unroll
  for (int s = 0; s < 4; ++s)
    u[s] = s < k ? *reinterpret_cast<const float2 *>(q + (size_t)s * P.stride) : make_float2(0.f, 0.f);
  float2 v = u[0];
#pragma unroll
  for (int s = 1; s < 4; ++s) {
    if (s < k) { v.x += u[s].x; v.y += u[s].y; }
  }
  for (int s = 4; s < k; ++s) {
    const float2 w = *reinterpret_cast<const float2 *>(q + (size_t)s * P.stride);
    v.x += w.x; v.y += w.y;
  }
  return v;
}
__device__ __forceinline__ void store2(float *p, float a, float b) { *reinterpret_cast<float2 *>(p) = make_float2(a, b); }
__device__ __forceinline__ void store2(bf16 *p, float a, float b) {
  *reinterpret_cast<__nv_bfloat162 *>(p) = __floats2bfloat162_rn(a, b);
}
template <typename T>
__global__ void __launch_bounds__(1024)
rope_kv_vec_kernel(SplitIn qkv, RowScale sc, RowPlan plan, float *__restrict__ q_out, bf16 *__restrict__ qp_hi,
                   bf16 *__restrict__ qp_lo, T *__restrict__ k_cache, T *__restrict__ v_cache, int rows_per_seq,
                   int n_heads, int head_dim, int S_max) {
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.x;
  const int half = head_dim >> 1, H = n_heads * head_dim, hq = half >> 1;
  const int b = r / rows_per_seq;
  const int slot = plan.slot[r];
  const bool wr = slot >= 0 && slot < S_max;
  const float rs = sc.of(r);
  // grid.y slices the row's work so that many SMs pull the partial sums
  for (int p = blockIdx.y * blockDim.x + threadIdx.x; p < n_heads * hq; p += gridDim.y * blockDim.x) {
    const int h = p / hq, i = (p - h * hq) * 2;
    const float4 cs = *reinterpret_cast<const float4 *>(&plan.rope[(size_t)r * half + i]);   // c0 s0 c1 s1
    const int c0 = h * head_dim + i, c1 = c0 + half;
    // all partial sums of this thread are requested before the first store
    float2 qa = split_sum2(qkv, r, c0), qb = split_sum2(qkv, r, c1);
    float2 ka = split_sum2(qkv, r, H + c0), kb = split_sum2(qkv, r, H + c1);
    float2 va = split_sum2(qkv, r, 2 * H + c0), vb = split_sum2(qkv, r, 2 * H + c1);
    qa.x *= rs; qa.y *= rs; qb.x *= rs; qb.y *= rs;
    const float2 ra = make_float2(qa.x * cs.x - qb.x * cs.y, qa.y * cs.z - qb.y * cs.w);
    const float2 rb = make_float2(qb.x * cs.x + qa.x * cs.y, qb.y * cs.z + qa.y * cs.w);
    store2(q_out + (size_t)r * H + c0, ra.x, ra.y);
    store2(q_out + (size_t)r * H + c1, rb.x, rb.y);
    if (qp_hi != nullptr) {      // the same values as a bf16 pair (value + rounding residual)
      const __nv_bfloat162 ha = __floats2bfloat162_rn(ra.x, ra.y), hb = __floats2bfloat162_rn(rb.x, rb.y);
      const float2 fa = __bfloat1622float2(ha), fb = __bfloat1622float2(hb);
      *reinterpret_cast<__nv_bfloat162 *>(qp_hi + (size_t)r * H + c0) = ha;
      *reinterpret_cast<__nv_bfloat162 *>(qp_hi + (size_t)r * H + c1) = hb;
      *reinterpret_cast<__nv_bfloat162 *>(qp_lo + (size_t)r * H + c0) = __floats2bfloat162_rn(ra.x - fa.x, ra.y - fa.y);
      *reinterpret_cast<__nv_bfloat162 *>(qp_lo + (size_t)r * H + c1) = __floats2bfloat162_rn(rb.x - fb.x, rb.y - fb.y);
    }
    if (!wr) continue;
    ka.x *= rs; ka.y *= rs; kb.x *= rs; kb.y *= rs;
    va.x *= rs; va.y *= rs; vb.x *= rs; vb.y *= rs;
    const size_t base = (((size_t)b * n_heads + h) * S_max + slot) * head_dim + i;
    store2(k_cache + base, ka.x * cs.x - kb.x * cs.y, ka.y * cs.z - kb.y * cs.w);
    store2(k_cache + base + half, kb.x * cs.x + ka.x * cs.y, kb.y * cs.z + ka.y * cs.w);
    store2(v_cache + base, va.x, va.y);
    store2(v_cache + base + half, vb.x, vb.y);
  }
}

// ------------------------------------------------------------------------------- SwiGLU
template <typename T>
__global__ void swiglu_kernel(SplitIn gu, RowScale sc, T *__restrict__ act, T *__restrict__ act_lo, int F) {
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.y;
  const int f = blockIdx.x * blockDim.x + threadIdx.x;
  if (f >= F) return;
  const float rs = sc.of(r);
  store_operand(act, act_lo, (size_t)r * F + f, silu_f(rs * gu.at(r, f)) * (rs * gu.at(r, F + f)));
}

template <typename T>
__global__ void swiglu_vec_kernel(SplitIn gu, RowScale sc, T *__restrict__ act, T *__restrict__ act_lo, int F) {
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.y;
  const int f = (blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (f >= F) return;
  const float rs = sc.of(r);
  const float4 a = split_sum4<3>(gu, r, f), b = split_sum4<3>(gu, r, F + f);
  store_operand4(act, act_lo, (size_t)r * F + f,
                 make_float4(silu_f(rs * a.x) * (rs * b.x), silu_f(rs * a.y) * (rs * b.y),
                             silu_f(rs * a.z) * (rs * b.z), silu_f(rs * a.w) * (rs * b.w)));
}

// ------------------------------------------------------------------------------- tree attention
// One block = 8 query rows of one (sequence, head); one warp per query row.  Keys/values stream
// through shared memory 32 at a time; lane j scores key j, then the warp accumulates P.V with
// each lane owning DH/32 output dimensions.  Online softmax in fp32.
template <typename T, int DH>
__global__ void __launch_bounds__(256)
tree_attn_kernel(const float *q, const T *kc, const T *vc,
                 RowPlan plan, T *__restrict__ out, T *__restrict__ out_lo, int rows_per_seq,
                 int n_heads, int S_max) {
  __shared__ float Ks[32][DH + 1];
  __shared__ float Vs[32][DH];
  __shared__ float qs[8][DH];
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.z, h = blockIdx.y;
  const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int i = blockIdx.x * 8 + w;
  const int H = n_heads * DH;
  const int r = b * rows_per_seq + (i < rows_per_seq ? i : 0);
  const bool valid = (i < rows_per_seq) && (plan.slot[r] >= 0);
  const int ctx = plan.ctx_len[b], kv_len = plan.kv_len[b];
  const uint64_t m0 = plan.mask[(size_t)r * 2], m1 = plan.mask[(size_t)r * 2 + 1];
  for (int d = lane; d < DH; d += 32) qs[w][d] = valid ? q[(size_t)r * H + h * DH + d] : 0.f;
  const T *kb = kc + ((size_t)b * n_heads + h) * S_max * DH;
  const T *vb = vc + ((size_t)b * n_heads + h) * S_max * DH;
  const float scale = rsqrtf((float)DH);
  float m = -INFINITY, l = 0.f;
  float o[DH / 32];
#pragma unroll
  for (int d = 0; d < DH / 32; ++d) o[d] = 0.f;
  for (int t0 = 0; t0 < kv_len; t0 += 32) {
    __syncthreads();
    for (int e = threadIdx.x; e < 32 * DH; e += 256) {
      const int j = e / DH, d = e % DH;
      const bool in = (t0 + j) < kv_len;
      Ks[j][d] = in ? to_f(kb[(size_t)(t0 + j) * DH + d]) : 0.f;
      Vs[j][d] = in ? to_f(vb[(size_t)(t0 + j) * DH + d]) : 0.f;
    }
    __syncthreads();
    const int t = t0 + lane;
    bool vis = valid && t < kv_len;
    if (vis && t >= ctx) {
      const int rel = t - ctx;
      vis = rel < 64 ? ((m0 >> rel) & 1ull) : (rel < 128 ? ((m1 >> (rel - 64)) & 1ull) : false);
    }
    float s = 0.f;
#pragma unroll 8
    for (int d = 0; d < DH; ++d) s += qs[w][d] * Ks[lane][d];
    s = vis ? s * scale : -INFINITY;
    const float m_new = fmaxf(m, warp_max(s));
    if (m_new == -INFINITY) continue;   // nothing visible so far (uniform across the warp)
    const float p = vis ? expf(s - m_new) : 0.f;
    const float corr = (m == -INFINITY) ? 0.f : expf(m - m_new);
    l = l * corr + warp_sum(p);
    m = m_new;
#pragma unroll
    for (int d = 0; d < DH / 32; ++d) o[d] *= corr;
    for (int j = 0; j < 32; ++j) {
      const float pj = __shfl_sync(0xffffffffu, p, j);
#pragma unroll
      for (int d = 0; d < DH / 32; ++d) o[d] += pj * Vs[j][lane + 32 * d];
    }
  }
  if (i < rows_per_seq) {
    const float inv = l > 0.f ? 1.f / l : 0.f;
#pragma unroll
    for (int d = 0; d < DH / 32; ++d)
      store_operand(out, out_lo, (size_t)r * H + h * DH + lane + 32 * d, o[d] * inv);
  }
}

// ------------------------------------------------------------------------------- arg-max / top-k
struct ValIdx {
  float v;
  int i;
};
__device__ __forceinline__ ValIdx better(ValIdx a, ValIdx b) {
  return (b.v > a.v || (b.v == a.v && b.i < a.i)) ? b : a;
}
__device__ __forceinline__ ValIdx block_argmax(ValIdx x, ValIdx *red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    ValIdx y;
    y.v = __shfl_xor_sync(0xffffffffu, x.v, o);
    y.i = __shfl_xor_sync(0xffffffffu, x.i, o);
    x = better(x, y);
  }
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  if (lane == 0) red[w] = x;
  __syncthreads();
  if (w == 0) {
    ValIdx y = lane < nw ? red[lane] : ValIdx{-INFINITY, 0x7fffffff};
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      ValIdx z;
      z.v = __shfl_xor_sync(0xffffffffu, y.v, o);
      z.i = __shfl_xor_sync(0xffffffffu, y.i, o);
      y = better(y, z);
    }
    if (lane == 0) red[0] = y;
  }
  __syncthreads();
  x = red[0];
  __syncthreads();
  return x;
}

__global__ void argmax_rows_kernel(const float *logits, int32_t *__restrict__ out, int V) {
  __shared__ ValIdx red[32];
  pdl_launch_dependents();
  pdl_wait();
  const float *row = logits + (size_t)blockIdx.x * V;
  ValIdx best{-INFINITY, 0x7fffffff};
  for (int i = threadIdx.x; i < V; i += blockDim.x) best = better(best, ValIdx{row[i], i});
  best = block_argmax(best, red);
  if (threadIdx.x == 0) out[blockIdx.x] = best.i;
}

// Per row: the k largest logits (ties: smaller id) and their natural-log softmax probabilities.
// The row is staged in shared memory; each round removes the current maximum.
__global__ void topk_logp_kernel(const float *logits, int32_t *__restrict__ tok,
                                 float *__restrict__ logp, int V, int k) {
  extern __shared__ float srow[];
  __shared__ ValIdx red[32];
  __shared__ float redf[32];
  pdl_launch_dependents();
  pdl_wait();
  const float *row = logits + (size_t)blockIdx.x * V;
  ValIdx best{-INFINITY, 0x7fffffff};
  for (int i = threadIdx.x; i < V; i += blockDim.x) {
    const float v = row[i];
    srow[i] = v;
    best = better(best, ValIdx{v, i});
  }
  best = block_argmax(best, red);
  const float mx = best.v;
  float se = 0.f;
  for (int i = threadIdx.x; i < V; i += blockDim.x) se += expf(srow[i] - mx);
  const float lse = mx + logf(block_sum(se, redf));
  for (int j = 0; j < k; ++j) {
    if (j > 0) {
      best = ValIdx{-INFINITY, 0x7fffffff};
      for (int i = threadIdx.x; i < V; i += blockDim.x) best = better(best, ValIdx{srow[i], i});
      best = block_argmax(best, red);
    }
    if (threadIdx.x == 0) {
      tok[(size_t)blockIdx.x * k + j] = best.i;
      logp[(size_t)blockIdx.x * k + j] = best.v - lse;
      srow[best.i] = -INFINITY;
    }
    __syncthreads();
  }
}

__device__ __forceinline__ ValIdx warp_argmax(ValIdx x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    ValIdx y;
    y.v = __shfl_xor_sync(0xffffffffu, x.v, o);
    y.i = __shfl_xor_sync(0xffffffffu, x.i, o);
    x = better(x, y);
  }
  return x;
}

// Same result for V <= 32768 and k <= 32 with two levels instead of k passes over the row: every
// thread keeps its 32 strided elements in registers, every warp extracts the k best of its 1024
// elements with shuffles only, and warp 0 extracts the k best of the 32 * k survivors.  (The k
// best of the row are among the k best of each part; ties still go to the smaller id.)
__global__ void __launch_bounds__(1024)
topk_logp_fast_kernel(const float *logits, int32_t *__restrict__ tok, float *__restrict__ logp,
                      int V, int k) {
  __shared__ ValIdx cand[32 * 32];
  __shared__ float redf[32];
  __shared__ float s_mx;
  pdl_launch_dependents();
  pdl_wait();
  const float *row = logits + (size_t)blockIdx.x * V;
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  float vals[32];
  float mx = -INFINITY;
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    const int i = tid + 1024 * j;
    vals[j] = i < V ? row[i] : -INFINITY;
    mx = fmaxf(mx, vals[j]);
  }
  mx = warp_max(mx);
  if (lane == 0) redf[w] = mx;
  __syncthreads();
  if (w == 0) {
    const float m2 = warp_max(redf[lane]);
    if (lane == 0) s_mx = m2;
  }
  __syncthreads();
  mx = s_mx;
  float se = 0.f;
#pragma unroll
  for (int j = 0; j < 32; ++j) se += expf(vals[j] - mx);       // exp(-inf) = 0 for the padding
  const float lse = mx + logf(block_sum(se, redf));
  for (int r = 0; r < k; ++r) {
    ValIdx best{-INFINITY, 0x7fffffff};
#pragma unroll
    for (int j = 0; j < 32; ++j) best = better(best, ValIdx{vals[j], tid + 1024 * j});
    best = warp_argmax(best);
    if ((best.i & 1023) == tid) {
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (j == (best.i >> 10)) vals[j] = -INFINITY;
    }
    if (lane == 0) cand[w * k + r] = best;
  }
  __syncthreads();
  if (w == 0) {
    const int n = 32 * k;
    for (int r = 0; r < k; ++r) {
      ValIdx best{-INFINITY, 0x7fffffff};
      int at = -1;
      for (int c = lane; c < n; c += 32) {
        const ValIdx x = cand[c];
        if (x.v > best.v || (x.v == best.v && x.i < best.i)) { best = x; at = c; }
      }
      const ValIdx win = warp_argmax(best);
      if (at >= 0 && best.i == win.i) cand[at] = ValIdx{-INFINITY, 0x7fffffff};
      __syncwarp();
      if (lane == 0) {
        tok[(size_t)blockIdx.x * k + r] = win.i;
        logp[(size_t)blockIdx.x * k + r] = win.v - lse;
      }
    }
  }
}

// The same result on eight CTAs per row (a thread-block cluster): CTA p takes an eighth of the
// row - 16 strided elements per thread in registers - and extracts its k best (every warp the k
// best of its 512 elements with shuffles, warp 0 the k best of those 8 * k) together with its
// (max, sum of exponentials); after a cluster barrier CTA 0 reads the eight candidate lists and
// the eight (max, sum) pairs through distributed shared memory, takes the k best of the 8 * k
// candidates (ties still go to the smaller id) and forms the log-sum-exp.  V <= 32768, k <= 32.
constexpr int TKP = 8;            // CTAs per row
__global__ void __launch_bounds__(256)
topk_logp_cluster_kernel(const float *logits, int32_t *__restrict__ tok, float *__restrict__ logp, int V, int k) {
  // logp == nullptr: only the ids are wanted (the arg-max of a row is its top-1), no exponentials
  __shared__ ValIdx cand[8 * 32];
  __shared__ ValIdx mine[32];     // this CTA's k best, read by CTA 0
  __shared__ float s_ms[2];       // this CTA's (max, sum of exp(v - max))
  __shared__ float redf[32];
  pdl_launch_dependents();
  pdl_wait();
  const int part = blockIdx.x, r = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  const int chunk = (((V + TKP - 1) / TKP) + 255) & ~255;          // ids per CTA, a multiple of 256
  const int base = part * chunk;
  const float *row = logits + (size_t)r * V;
  float vals[16];
  float mx = -INFINITY;
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const int i = base + tid + 256 * j;
    vals[j] = (tid + 256 * j < chunk && i < V) ? row[i] : -INFINITY;
    mx = fmaxf(mx, vals[j]);
  }
  mx = warp_max(mx);
  if (lane == 0) redf[w] = mx;
  __syncthreads();
  mx = warp_max(lane < 8 ? redf[lane] : -INFINITY);
  __syncthreads();
  float se = 0.f;
  if (mx != -INFINITY && logp != nullptr) {
#pragma unroll
    for (int j = 0; j < 16; ++j) se += expf(vals[j] - mx);
  }
  se = warp_sum(se);
  if (lane == 0) redf[w] = se;
  __syncthreads();
  se = warp_sum(lane < 8 ? redf[lane] : 0.f);
  if (tid == 0) { s_ms[0] = mx; s_ms[1] = se; }
  for (int rnd = 0; rnd < k; ++rnd) {
    ValIdx best{-INFINITY, 0x7fffffff};
#pragma unroll
    for (int j = 0; j < 16; ++j) best = better(best, ValIdx{vals[j], vals[j] == -INFINITY ? 0x7fffffff : base + tid + 256 * j});
    best = warp_argmax(best);
    if (best.i != 0x7fffffff && ((best.i - base) & 255) == tid) {
#pragma unroll
      for (int j = 0; j < 16; ++j)
        if (j == ((best.i - base) >> 8)) vals[j] = -INFINITY;
    }
    if (lane == 0) cand[w * k + rnd] = best;
  }
  __syncthreads();
  if (w == 0) {
    const int n = 8 * k;
    for (int rnd = 0; rnd < k; ++rnd) {
      ValIdx best{-INFINITY, 0x7fffffff};
      int at = -1;
      for (int c = lane; c < n; c += 32) {
        const ValIdx x = cand[c];
        if (x.v > best.v || (x.v == best.v && x.i < best.i)) { best = x; at = c; }
      }
      const ValIdx win = warp_argmax(best);
      if (at >= 0 && best.i == win.i && win.i != 0x7fffffff) cand[at] = ValIdx{-INFINITY, 0x7fffffff};
      __syncwarp();
      if (lane == 0) mine[rnd] = win;
    }
  }
  __syncthreads();
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
  if (part == 0 && w == 0) {
    // lane l holds candidate l of every CTA (eight registers) and CTA (l % 8)'s (max, sum)
    const uint32_t a_mine = (uint32_t)__cvta_generic_to_shared(&mine[lane < k ? lane : 0]);
    const uint32_t a_ms = (uint32_t)__cvta_generic_to_shared(&s_ms[0]);
    ValIdx c8[TKP];
#pragma unroll
    for (int j = 0; j < TKP; ++j) {
      uint32_t ra;
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(a_mine), "r"(j));
      float v; int id;
      asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(ra) : "memory");
      asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(id) : "r"(ra + 4) : "memory");
      c8[j] = lane < k ? ValIdx{v, id} : ValIdx{-INFINITY, 0x7fffffff};
    }
    uint32_t rb;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rb) : "r"(a_ms), "r"(lane & 7));
    float mj, sj;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(mj) : "r"(rb) : "memory");
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(sj) : "r"(rb + 4) : "memory");
    const float M = warp_max(mj);
    float part_sum = (lane < 8 && mj != -INFINITY) ? sj * expf(mj - M) : 0.f;
    const float lse = M + logf(warp_sum(part_sum));
    for (int rnd = 0; rnd < k; ++rnd) {
      ValIdx best{-INFINITY, 0x7fffffff};
#pragma unroll
      for (int j = 0; j < TKP; ++j) best = better(best, c8[j]);
      const ValIdx win = warp_argmax(best);
#pragma unroll
      for (int j = 0; j < TKP; ++j)
        if (c8[j].i == win.i) c8[j] = ValIdx{-INFINITY, 0x7fffffff};
      if (lane == 0) {
        tok[(size_t)r * k + rnd] = win.i;
        if (logp != nullptr) logp[(size_t)r * k + rnd] = win.v - lse;
      }
    }
  }
  // no CTA leaves while CTA 0 may still read its shared memory
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}

}  // namespace

#define DISPATCH_T(dtype, ...)                \
  if ((dtype) == 0) {                         \
    typedef float T;                          \
    __VA_ARGS__                               \
  } else {                                    \
    typedef bf16 T;                           \
    __VA_ARGS__                               \
  }

cudaError_t embed_norm(Launch L, int dtype, const int32_t *tok, const void *E, const void *g,
                       float *x, Operand xn, int R, int H, int V, float eps) {
  DISPATCH_T(dtype, return launch_k(embed_norm_kernel<T>, dim3(R), dim3(256), 0, L.st, L.pdl, tok,
                                    (const T *)E, (const T *)g, x, (T *)xn.hi, (T *)xn.lo, H, V, eps);)
}

cudaError_t row_epilogue(Launch L, int dtype, int mode, float *x, SplitIn P, const void *bias,
                         const void *g, Operand xn, float *out_f32, int R, int H, float eps) {
  if (H % 4 == 0 && P.ld % 4 == 0 && P.stride % 4 == 0 && H <= 8192) {
    const int groups = H / 4;
    int threads = groups <= 1024 ? ((groups + 31) / 32) * 32 : (((groups + 1) / 2 + 31) / 32) * 32;
    if (groups <= 1024) {
      DISPATCH_T(dtype, return launch_k(row_epilogue_vec_kernel<T, 1>, dim3(R), dim3(threads), 0, L.st, L.pdl,
                                        mode, x, P, (const T *)bias, (const T *)g, (T *)xn.hi, (T *)xn.lo,
                                        out_f32, H, eps);)
    } else {
      DISPATCH_T(dtype, return launch_k(row_epilogue_vec_kernel<T, 2>, dim3(R), dim3(threads), 0, L.st, L.pdl,
                                        mode, x, P, (const T *)bias, (const T *)g, (T *)xn.hi, (T *)xn.lo,
                                        out_f32, H, eps);)
    }
  }
  DISPATCH_T(dtype, return launch_k(row_epilogue_kernel<T>, dim3(R), dim3(256), 0, L.st, L.pdl, mode,
                                    x, P, (const T *)bias, (const T *)g, (T *)xn.hi, (T *)xn.lo, out_f32,
                                    H, eps);)
}

cudaError_t eagle_concat(Launch L, int dtype, const float *feat_src, const int32_t *row_src,
                         const int32_t *row_tok, const void *E, Operand cat, int R, int H, int V) {
  if ((H & 3) == 0) {
    const int threads = 128;
    DISPATCH_T(dtype, return launch_k(eagle_concat_vec_kernel<T>, dim3(R, (H / 4 + threads - 1) / threads),
                                      dim3(threads), 0, L.st, L.pdl, feat_src, row_src, row_tok, (const T *)E,
                                      (T *)cat.hi, (T *)cat.lo, H, V);)
  }
  DISPATCH_T(dtype, return launch_k(eagle_concat_kernel<T>, dim3(R), dim3(256), 0, L.st, L.pdl,
                                    feat_src, row_src, row_tok, (const T *)E, (T *)cat.hi, (T *)cat.lo, H,
                                    V);)
}

cudaError_t cast_rows(Launch L, int dtype, const float *src, const int32_t *row_src, Operand dst,
                      float *dst32, int dst32_stride, int R, int H) {
  DISPATCH_T(dtype, return launch_k(cast_rows_kernel<T>, dim3(R), dim3(256), 0, L.st, L.pdl, src,
                                    row_src, (T *)dst.hi, (T *)dst.lo, dst32, dst32_stride, H);)
}

cudaError_t reduce_splits(Launch L, SplitIn P, float *Y, int ldy, int R, int ncols) {
  return launch_k(reduce_splits_kernel, dim3((ncols + 255) / 256, R), dim3(256), 0, L.st, L.pdl, P, Y,
                  ldy, ncols);
}

cudaError_t resblock_update(Launch L, int dtype, float *x, SplitIn P, HeadTab tab, Operand xn, int R, int H) {
  if (H % 4 != 0 || P.ld % 4 != 0 || P.stride % 4 != 0 || tab.rows_per_head < 1) return cudaErrorInvalidValue;
  DISPATCH_T(dtype, return launch_k(resblock_update_kernel<T>, dim3((H + 1023) / 1024, R), dim3(256), 0, L.st, L.pdl,
                                    x, P, tab, (T *)xn.hi, (T *)xn.lo, H);)
}

cudaError_t embed_update(Launch L, int dtype, const int32_t *tok, const void *E, const void *g, float *x,
                         Operand xg, float *sumsq, int R, int H, int V) {
  if (H % 4 != 0) return cudaErrorInvalidValue;
  DISPATCH_T(dtype, return launch_k(embed_update_kernel<T>, dim3((H + 1023) / 1024, R), dim3(256), 0, L.st, L.pdl,
                                    tok, (const T *)E, (const T *)g, x, (T *)xg.hi, (T *)xg.lo, sumsq, H, V);)
}

cudaError_t row_update(Launch L, int dtype, float *x, SplitIn P, const void *g, Operand xg, float *sumsq,
                       int R, int H) {
  if (H % 4 != 0 || P.ld % 4 != 0 || P.stride % 4 != 0) return cudaErrorInvalidValue;
  DISPATCH_T(dtype, return launch_k(row_update_kernel<T>, dim3((H + 1023) / 1024, R), dim3(256), 0, L.st, L.pdl,
                                    x, P, (const T *)g, (T *)xg.hi, (T *)xg.lo, sumsq, H);)
}

cudaError_t rope_kv_write(Launch L, int dtype, SplitIn qkv, RowScale sc, RowPlan plan, float *q_out,
                          Operand q_pair, void *k_cache, void *v_cache, int R, int rows_per_seq, int n_heads,
                          int head_dim, int S_max) {
  bf16 *qh = (bf16 *)q_pair.hi, *ql = (bf16 *)q_pair.lo;
  if (dtype == 0 || ql == nullptr) qh = ql = nullptr;      // the pair exists for bf16 storage only
  if (head_dim % 4 == 0 && qkv.ld % 2 == 0 && qkv.stride % 2 == 0) {
    const int work = n_heads * head_dim / 4;
    const int threads = work < 128 ? ((work + 31) / 32) * 32 : 128;
    const int slices = (work + threads - 1) / threads;
    DISPATCH_T(dtype, return launch_k(rope_kv_vec_kernel<T>, dim3(R, slices), dim3(threads), 0, L.st, L.pdl, qkv, sc, plan,
                                      q_out, qh, ql, (T *)k_cache, (T *)v_cache, rows_per_seq, n_heads, head_dim,
                                      S_max);)
  }
  DISPATCH_T(dtype, return launch_k(rope_kv_kernel<T>, dim3(R, n_heads), dim3(head_dim / 2), 0, L.st,
                                    L.pdl, qkv, sc, plan, q_out, qh, ql, (T *)k_cache, (T *)v_cache,
                                    rows_per_seq, n_heads, head_dim, S_max);)
}

cudaError_t swiglu(Launch L, int dtype, SplitIn gu, RowScale sc, Operand act, int R, int F) {
  if (F % 4 == 0 && gu.ld % 4 == 0 && gu.stride % 4 == 0) {
    DISPATCH_T(dtype, return launch_k(swiglu_vec_kernel<T>, dim3((F / 4 + 255) / 256, R), dim3(256), 0, L.st,
                                      L.pdl, gu, sc, (T *)act.hi, (T *)act.lo, F);)
  }
  DISPATCH_T(dtype, return launch_k(swiglu_kernel<T>, dim3((F + 255) / 256, R), dim3(256), 0, L.st,
                                    L.pdl, gu, sc, (T *)act.hi, (T *)act.lo, F);)
}

cudaError_t tree_attention(Launch L, int dtype, const float *q, const void *k_cache,
                           const void *v_cache, RowPlan plan, Operand out, int R, int rows_per_seq,
                           int B, int n_heads, int head_dim, int S_max) {
  (void)R;
  dim3 grid((rows_per_seq + 7) / 8, n_heads, B);
  if (head_dim == 64) {
    DISPATCH_T(dtype, return launch_k(tree_attn_kernel<T, 64>, grid, dim3(256), 0, L.st, L.pdl, q,
                                      (const T *)k_cache, (const T *)v_cache, plan, (T *)out.hi,
                                      (T *)out.lo, rows_per_seq, n_heads, S_max);)
  } else if (head_dim == 128) {
    DISPATCH_T(dtype, return launch_k(tree_attn_kernel<T, 128>, grid, dim3(256), 0, L.st, L.pdl, q,
                                      (const T *)k_cache, (const T *)v_cache, plan, (T *)out.hi,
                                      (T *)out.lo, rows_per_seq, n_heads, S_max);)
  }
  return cudaErrorInvalidValue;
}

static cudaError_t topk_cluster_launch(Launch L, const float *logits, int32_t *tok, float *logp, int R, int V, int k) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(TKP, R);
  cfg.blockDim = dim3(256);
  cfg.stream = L.st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = L.pdl ? 1 : 0;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = TKP;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  ++g_launches;
  return cudaLaunchKernelEx(&cfg, topk_logp_cluster_kernel, logits, tok, logp, V, k);
}

cudaError_t argmax_rows(Launch L, const float *logits, int32_t *out, int R, int V) {
  // the arg-max (ties: smaller id) is the top-1; wide rows go to the eight-CTA kernel
  if (V <= 32768 && V >= 4096) return topk_cluster_launch(L, logits, out, nullptr, R, V, 1);
  return launch_k(argmax_rows_kernel, dim3(R), dim3(1024), 0, L.st, L.pdl, logits, out, V);
}

cudaError_t topk_logp(Launch L, const float *logits, int32_t *tok, float *logp, int R, int V, int k) {
  if (V <= 32768 && k <= 32 && V >= 4096) return topk_cluster_launch(L, logits, tok, logp, R, V, k);
  if (V <= 32768 && k <= 32)
    return launch_k(topk_logp_fast_kernel, dim3(R), dim3(1024), 0, L.st, L.pdl, logits, tok, logp, V, k);
  const size_t smem = (size_t)V * sizeof(float);
  static SmemOptIn optin;
  {
    cudaError_t e = optin.ensure((const void *)topk_logp_kernel, smem);
    if (e != cudaSuccess) return e;
  }
  return launch_k(topk_logp_kernel, dim3(R), dim3(1024), smem, L.st, L.pdl, logits, tok, logp, V, k);
}

}  // namespace koala
