// Tree-masked flash-decode attention for bf16 caches with head_dim 128, on tensor cores.
//
// One CTA = one (key chunk, group of 16 query rows, head, sequence) with four warps that split
// every 64-key tile among themselves.  The sequence's keys are cut into `chunks` ranges of whole
// tiles from the device-side length, so the grid is fixed by host-known sizes while the work
// follows the real context length; short contexts use a single chunk and need no second kernel.
// K and V tiles stream through shared memory with cp.async (three stages,
// 16-byte vector loads, XOR-swizzled rows); scores S = Q K^T and the update O += P V run on
// mma.sync m16n8k16 with fp32 accumulators.  Q and P enter the MMAs as bf16 pairs (value +
// rounding residual), so only the cached K and V carry bf16 rounding.  The mask is: slots below
// ctx_len visible to every row; slot ctx_len + j visible to a row iff bit j of its 128-bit mask.
// Softmax is online, in fp32, in base 2; row statistics use quad shuffles.  With several chunks
// each CTA writes an unnormalised partial (O, m, l) per row and a second kernel combines the
// chunks in a fixed order; either way the output is emitted as a matrix-multiply operand pair.
#include "common.cuh"

namespace koala {
namespace {

constexpr int DH = 128;
constexpr int TILE = 64;                 // keys per shared-memory tile
constexpr int ROW_BYTES = DH * 2;        // 256
constexpr int TILE_BYTES = TILE * ROW_BYTES;
constexpr int PSTRIDE = DH + 2;          // floats per partial: O[128], m, l

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// byte offset of 16-byte chunk `ch` (0..15) of row `row` inside a swizzled tile
__device__ __forceinline__ uint32_t tile_off(int row, int ch) {
  return (uint32_t)(row * ROW_BYTES + ((ch ^ (row & 7)) << 4));
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, bool valid) {
  const int sz = valid ? 16 : 0;          // zero-fill when out of range
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float *d, const uint32_t *a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// two floats -> packed bf16x2 (hi) and the packed residuals (lo)
__device__ __forceinline__ void split_pack(float x, float y, uint32_t &hi, uint32_t &lo) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
  const float2 hf = __bfloat1622float2(h);
  const __nv_bfloat162 l = __floats2bfloat162_rn(x - hf.x, y - hf.y);
  hi = *reinterpret_cast<const uint32_t *>(&h);
  lo = *reinterpret_cast<const uint32_t *>(&l);
}

__device__ __forceinline__ bool mask_bit(uint64_t m0, uint64_t m1, int rel) {
  return rel < 64 ? ((m0 >> rel) & 1ull) : (rel < 128 ? ((m1 >> (rel - 64)) & 1ull) : false);
}

// grid (chunks, row groups of 16, n_heads * B); block = 4 warps.  All four warps serve the same
// 16 query rows; warp w takes keys [16w, 16w + 16) of every 64-key tile and keeps its own running
// (max, sum, O); the four are merged through shared memory at the end.  With chunks == 1 the CTA
// writes the normalised output operand itself; otherwise it writes an unnormalised partial.
constexpr int NST = 3;                   // cp.async stages
constexpr int MSTRIDE = DH + 4;          // floats per merged row in shared memory (keeps 16-byte alignment)

__global__ void __launch_bounds__(128)
tree_attn_mma_kernel(const float *q, const bf16 *kc, const bf16 *vc,
                     RowPlan plan, float *__restrict__ part, bf16 *__restrict__ out, bf16 *__restrict__ out_lo,
                     int rows_per_seq, int n_heads, int S_max, int chunks) {
  extern __shared__ __align__(1024) unsigned char smem[];     // [NST][K tile | V tile]
  pdl_launch_dependents();
  pdl_wait();
  const int c = blockIdx.x, rg = blockIdx.y;
  const int b = blockIdx.z / n_heads, h = blockIdx.z % n_heads;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int H = n_heads * DH;
  const int ctx = plan.ctx_len[b];
  int kv_len = plan.kv_len[b];
  kv_len = kv_len > S_max ? S_max : kv_len;
  const int n_tiles = (kv_len + TILE - 1) / TILE;
  const int tile_lo = (int)(((long long)n_tiles * c) / chunks);
  const int tile_hi = (int)(((long long)n_tiles * (c + 1)) / chunks);
  const bf16 *kb = kc + ((size_t)b * n_heads + h) * S_max * DH;
  const bf16 *vb = vc + ((size_t)b * n_heads + h) * S_max * DH;
  const uint32_t sbase = smem_addr(smem);

  auto load_tile = [&](int tile, int buf) {
    const int key0 = tile * TILE;
    const uint32_t kdst = sbase + buf * 2 * TILE_BYTES, vdst = kdst + TILE_BYTES;
#pragma unroll
    for (int e = threadIdx.x; e < TILE * 16; e += 128) {
      const int row = e >> 4, ch = e & 15;
      const bool in = key0 + row < kv_len;
      const size_t goff = (size_t)(in ? key0 + row : 0) * DH + ch * 8;
      cp_async16(kdst + tile_off(row, ch), kb + goff, in);
      cp_async16(vdst + tile_off(row, ch), vb + goff, in);
    }
  };

  const int i0 = rg * 16 + g, i1 = i0 + 8;
  const bool in0 = i0 < rows_per_seq, in1 = i1 < rows_per_seq;
  const int r0 = b * rows_per_seq + (in0 ? i0 : 0), r1 = b * rows_per_seq + (in1 ? i1 : 0);
  // every global load of the prologue is issued before the first use of any of them
  const int slot0 = plan.slot[r0], slot1 = plan.slot[r1];
  const uint64_t mk00 = plan.mask[(size_t)r0 * 2], mk01 = plan.mask[(size_t)r0 * 2 + 1];
  const uint64_t mk10 = plan.mask[(size_t)r1 * 2], mk11 = plan.mask[(size_t)r1 * 2 + 1];
  float2 qa[8][4];
  {
    const float *q0 = q + (size_t)r0 * H + h * DH, *q1 = q + (size_t)r1 * H + h * DH;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      const int col = ks * 16 + 2 * t;
      qa[ks][0] = *reinterpret_cast<const float2 *>(q0 + col);
      qa[ks][1] = *reinterpret_cast<const float2 *>(q1 + col);
      qa[ks][2] = *reinterpret_cast<const float2 *>(q0 + col + 8);
      qa[ks][3] = *reinterpret_cast<const float2 *>(q1 + col + 8);
    }
  }

#pragma unroll
  for (int sidx = 0; sidx < NST - 1; ++sidx) {
    if (tile_lo + sidx < tile_hi) load_tile(tile_lo + sidx, sidx);
    cp_async_commit();
  }

  const bool ok0 = in0 && slot0 >= 0, ok1 = in1 && slot1 >= 0;
  const uint64_t m00 = ok0 ? mk00 : 0ull, m01 = ok0 ? mk01 : 0ull;
  const uint64_t m10 = ok1 ? mk10 : 0ull, m11 = ok1 ? mk11 : 0ull;
  // Q fragments (A operand, 8 k-steps of 16), as bf16 pairs; rows not in use contribute zeros
  uint32_t qh[8][4], ql[8][4];
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const bool ok = (e & 1) ? ok1 : ok0;
      split_pack(ok ? qa[ks][e].x : 0.f, ok ? qa[ks][e].y : 0.f, qh[ks][e], ql[ks][e]);
    }
  }

  float o[16][4];
#pragma unroll
  for (int j = 0; j < 16; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }
  float mrow0 = -INFINITY, mrow1 = -INFINITY, lrow0 = 0.f, lrow1 = 0.f;
  const float sc = 0.08838834764831845f * 1.4426950408889634f;    // 1/sqrt(128) * log2(e)
  const int kw = 16 * warp;                                        // this warp's key offset inside a tile

  for (int tile = tile_lo; tile < tile_hi; ++tile) {
    const int it = tile - tile_lo;
    const int buf = it % NST;
    if (tile + NST - 1 < tile_hi) load_tile(tile + NST - 1, (it + NST - 1) % NST);
    cp_async_commit();
    cp_async_wait<NST - 1>();
    __syncthreads();
    const uint32_t kt = sbase + buf * 2 * TILE_BYTES, vt = kt + TILE_BYTES;
    const int key0 = tile * TILE + kw;
    // ---- S = Q K^T over this warp's 16 keys
    // four independent accumulation chains (key group x value/residual part of Q), interleaved
    float s[2][4], sl[2][4];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
      sl[j][0] = sl[j][1] = sl[j][2] = sl[j][3] = 0.f;
    }
#pragma unroll
    for (int kp = 0; kp < 4; ++kp) {
      uint32_t ka[4], kb2[4];
      ldmatrix_x4(kt + tile_off(kw + (lane & 7), 4 * kp + (lane >> 3)), ka[0], ka[1], ka[2], ka[3]);
      ldmatrix_x4(kt + tile_off(kw + 8 + (lane & 7), 4 * kp + (lane >> 3)), kb2[0], kb2[1], kb2[2], kb2[3]);
      mma_bf16(s[0], qh[2 * kp], ka[0], ka[1]);
      mma_bf16(sl[0], ql[2 * kp], ka[0], ka[1]);
      mma_bf16(s[1], qh[2 * kp], kb2[0], kb2[1]);
      mma_bf16(sl[1], ql[2 * kp], kb2[0], kb2[1]);
      mma_bf16(s[0], qh[2 * kp + 1], ka[2], ka[3]);
      mma_bf16(sl[0], ql[2 * kp + 1], ka[2], ka[3]);
      mma_bf16(s[1], qh[2 * kp + 1], kb2[2], kb2[3]);
      mma_bf16(sl[1], ql[2 * kp + 1], kb2[2], kb2[3]);
    }
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      s[j][0] += sl[j][0]; s[j][1] += sl[j][1]; s[j][2] += sl[j][2]; s[j][3] += sl[j][3];
    }
    // ---- mask, online softmax (base 2)
    const bool need_mask = key0 + 16 > ctx;
    float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int key = key0 + 8 * j + 2 * t + e;
        bool v0 = ok0, v1 = ok1;
        if (need_mask) {
          if (key >= kv_len) { v0 = false; v1 = false; }
          else if (key >= ctx) {
            v0 = v0 && mask_bit(m00, m01, key - ctx);
            v1 = v1 && mask_bit(m10, m11, key - ctx);
          }
        }
        s[j][e] = v0 ? s[j][e] * sc : -INFINITY;
        s[j][2 + e] = v1 ? s[j][2 + e] * sc : -INFINITY;
        mx0 = fmaxf(mx0, s[j][e]);
        mx1 = fmaxf(mx1, s[j][2 + e]);
      }
    }
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
    const float mn0 = fmaxf(mrow0, mx0), mn1 = fmaxf(mrow1, mx1);
    const float mu0 = mn0 == -INFINITY ? 0.f : mn0, mu1 = mn1 == -INFINITY ? 0.f : mn1;
    const float cr0 = exp2f(mrow0 - mu0), cr1 = exp2f(mrow1 - mu1);   // exp2(-inf) = 0
    mrow0 = mn0;
    mrow1 = mn1;
    const float p00 = exp2f(s[0][0] - mu0), p01 = exp2f(s[0][1] - mu0);
    const float p10 = exp2f(s[0][2] - mu1), p11 = exp2f(s[0][3] - mu1);
    const float p02 = exp2f(s[1][0] - mu0), p03 = exp2f(s[1][1] - mu0);
    const float p12 = exp2f(s[1][2] - mu1), p13 = exp2f(s[1][3] - mu1);
    float ps0 = p00 + p01 + p02 + p03, ps1 = p10 + p11 + p12 + p13;
    uint32_t ph[4], pl[4];             // P as A operand for one k-step of 16 keys
    split_pack(p00, p01, ph[0], pl[0]);
    split_pack(p10, p11, ph[1], pl[1]);
    split_pack(p02, p03, ph[2], pl[2]);
    split_pack(p12, p13, ph[3], pl[3]);
    ps0 += __shfl_xor_sync(0xffffffffu, ps0, 1);
    ps0 += __shfl_xor_sync(0xffffffffu, ps0, 2);
    ps1 += __shfl_xor_sync(0xffffffffu, ps1, 1);
    ps1 += __shfl_xor_sync(0xffffffffu, ps1, 2);
    lrow0 = lrow0 * cr0 + ps0;
    lrow1 = lrow1 * cr1 + ps1;
    if (cr0 != 1.f || cr1 != 1.f) {
#pragma unroll
      for (int j = 0; j < 16; ++j) { o[j][0] *= cr0; o[j][1] *= cr0; o[j][2] *= cr1; o[j][3] *= cr1; }
    }
    // ---- O += P V over this warp's 16 keys, 16 groups of 8 head dims
    // (all value-part products first, then all residual-part products: 16 independent
    //  accumulators between two uses of the same one)
    uint32_t vf[8][4];
#pragma unroll
    for (int jp = 0; jp < 8; ++jp)
      ldmatrix_x4_trans(vt + tile_off(kw + (lane & 7) + 8 * ((lane >> 3) & 1), 2 * jp + (lane >> 4)),
                        vf[jp][0], vf[jp][1], vf[jp][2], vf[jp][3]);
#pragma unroll
    for (int jp = 0; jp < 8; ++jp) {
      mma_bf16(o[2 * jp], ph, vf[jp][0], vf[jp][1]);
      mma_bf16(o[2 * jp + 1], ph, vf[jp][2], vf[jp][3]);
    }
#pragma unroll
    for (int jp = 0; jp < 8; ++jp) {
      mma_bf16(o[2 * jp], pl, vf[jp][0], vf[jp][1]);
      mma_bf16(o[2 * jp + 1], pl, vf[jp][2], vf[jp][3]);
    }
    __syncthreads();      // the buffer refilled by the next iteration's load is no longer read
  }
  cp_async_wait<0>();
  __syncthreads();
  // ---- merge the four warps through shared memory: [warp][16 rows][O 128 | m | l]
  float *ms = reinterpret_cast<float *>(smem);
  {
    float *w0 = ms + ((size_t)warp * 16 + g) * MSTRIDE, *w1 = w0 + 8 * MSTRIDE;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      *reinterpret_cast<float2 *>(w0 + 8 * j + 2 * t) = make_float2(o[j][0], o[j][1]);
      *reinterpret_cast<float2 *>(w1 + 8 * j + 2 * t) = make_float2(o[j][2], o[j][3]);
    }
    if (t == 0) { w0[DH] = mrow0; w0[DH + 1] = lrow0; w1[DH] = mrow1; w1[DH + 1] = lrow1; }
  }
  __syncthreads();
  // thread -> (row = tid / 8, 16 consecutive dims starting at (tid % 8) * 16)
  const int row = threadIdx.x >> 3, d0 = (threadIdx.x & 7) * 16;
  const int i = rg * 16 + row;
  if (i >= rows_per_seq) return;
  const int r = b * rows_per_seq + i;
  float mm = -INFINITY;
#pragma unroll
  for (int w = 0; w < 4; ++w) mm = fmaxf(mm, ms[((size_t)w * 16 + row) * MSTRIDE + DH]);
  float acc[16];
#pragma unroll
  for (int d = 0; d < 16; ++d) acc[d] = 0.f;
  float l = 0.f;
  if (mm != -INFINITY) {
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const float *src = ms + ((size_t)w * 16 + row) * MSTRIDE;
      const float mw = src[DH];
      if (mw == -INFINITY) continue;
      const float wgt = exp2f(mw - mm);
      l += wgt * src[DH + 1];
#pragma unroll
      for (int d = 0; d < 16; d += 4) {
        const float4 v = *reinterpret_cast<const float4 *>(src + d0 + d);
        acc[d] += wgt * v.x; acc[d + 1] += wgt * v.y; acc[d + 2] += wgt * v.z; acc[d + 3] += wgt * v.w;
      }
    }
  }
  if (chunks == 1) {
    const float inv = l > 0.f ? 1.f / l : 0.f;
    const size_t ob = (size_t)r * H + h * DH + d0;
#pragma unroll
    for (int d = 0; d < 16; d += 2) {
      uint32_t hi, lo;
      split_pack(acc[d] * inv, acc[d + 1] * inv, hi, lo);
      *reinterpret_cast<uint32_t *>(out + ob + d) = hi;
      if (out_lo != nullptr) *reinterpret_cast<uint32_t *>(out_lo + ob + d) = lo;
    }
  } else {
    float *p = part + (((size_t)r * n_heads + h) * chunks + c) * PSTRIDE;
#pragma unroll
    for (int d = 0; d < 16; d += 2) *reinterpret_cast<float2 *>(p + d0 + d) = make_float2(acc[d], acc[d + 1]);
    if ((threadIdx.x & 7) == 0) { p[DH] = mm; p[DH + 1] = l; }
  }
}

// One warp per (row, head): merges the chunk partials in chunk order and writes the operand pair.
__global__ void __launch_bounds__(256)
tree_attn_combine_kernel(const float *part, bf16 *__restrict__ out, bf16 *__restrict__ out_lo,
                         int R, int n_heads, int chunks) {
  pdl_launch_dependents();
  pdl_wait();
  const int pair = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (pair >= R * n_heads) return;
  const float *p = part + (size_t)pair * chunks * PSTRIDE;
  float m = -INFINITY;
  for (int c = 0; c < chunks; ++c) m = fmaxf(m, p[(size_t)c * PSTRIDE + DH]);
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  float l = 0.f;
  if (m != -INFINITY) {
    for (int c = 0; c < chunks; ++c) {
      const float mc = p[(size_t)c * PSTRIDE + DH];
      if (mc == -INFINITY) continue;
      const float w = exp2f(mc - m);
      l += w * p[(size_t)c * PSTRIDE + DH + 1];
      const float2 a = *reinterpret_cast<const float2 *>(p + (size_t)c * PSTRIDE + 4 * lane);
      const float2 bq = *reinterpret_cast<const float2 *>(p + (size_t)c * PSTRIDE + 4 * lane + 2);
      acc.x += w * a.x; acc.y += w * a.y; acc.z += w * bq.x; acc.w += w * bq.y;
    }
  }
  const float inv = l > 0.f ? 1.f / l : 0.f;
  const float v[4] = {acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv};
  const size_t o = (size_t)pair * DH + 4 * lane;      // pair = r * n_heads + h  ->  r * H + h * DH
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const bf16 hi = __float2bfloat16_rn(v[e]);
    out[o + e] = hi;
    if (out_lo != nullptr) out_lo[o + e] = __float2bfloat16_rn(v[e] - __bfloat162float(hi));
  }
}

}  // namespace

// Key chunks per (sequence, head, row group): as many as keep the CTA count within two CTAs per SM
// (96 KB of shared memory each), at least one per 2048 keys of capacity, never finer than 128 keys of
// capacity per chunk.  One chunk means one kernel (no partials, no combine).  (7B-shaped draft
// iteration, 10 rows, context 1024: 1.965 / 1.905 / 1.858 / 1.845 / 1.839 ms with 1 / 2 / 4 / 6 / 8
// chunks; 13B shape at batch 4, 160 sequence-head pairs: flat from 1 to 4, slower beyond.)
int g_attn_mma_chunks = 0;     // > 0: this many key chunks whatever the shape (A/B runs)
void attn_mma_set_chunks(int chunks) { g_attn_mma_chunks = chunks; }
int attn_mma_chunks(int B, int n_heads, int rows_per_seq, int S_max, int num_sms) {
  const int rgs = (rows_per_seq + 15) / 16;
  if (g_attn_mma_chunks > 0) {
    const int lim = S_max / 64 > 1 ? S_max / 64 : 1;
    const int f = g_attn_mma_chunks > 16 ? 16 : g_attn_mma_chunks;
    return f > lim ? lim : f;
  }
  int c = (2 * num_sms) / (rgs * B * n_heads);
  const int by_len = (S_max + 2047) / 2048;
  c = c < by_len ? by_len : c;
  const int cap = S_max / 128 > 1 ? S_max / 128 : 1;
  c = c > cap ? cap : c;
  return c < 1 ? 1 : (c > 16 ? 16 : c);
}

size_t attn_mma_scratch_floats(int rows_total, int n_heads, int chunks) {
  return (size_t)rows_total * n_heads * chunks * PSTRIDE;
}

cudaError_t tree_attention_mma(Launch L, const float *q, const void *k_cache, const void *v_cache,
                               RowPlan plan, Operand out, float *scratch, int rows_per_seq, int B,
                               int n_heads, int S_max, int chunks) {
  static SmemOptIn optin;
  const size_t smem = (size_t)NST * 2 * TILE_BYTES;
  static_assert((size_t)4 * 16 * MSTRIDE * sizeof(float) <= (size_t)NST * 2 * TILE_BYTES, "merge buffer fits");
  {
    cudaError_t e = optin.ensure((const void *)tree_attn_mma_kernel, smem);
    if (e != cudaSuccess) return e;
  }
  const int rgs = (rows_per_seq + 15) / 16;
  if (rgs < 1 || rgs > 8 || chunks < 1) return cudaErrorInvalidValue;
  cudaError_t e = launch_k(tree_attn_mma_kernel, dim3(chunks, rgs, n_heads * B), dim3(128), smem, L.st, L.pdl, q,
                           (const bf16 *)k_cache, (const bf16 *)v_cache, plan, scratch, (bf16 *)out.hi,
                           (bf16 *)out.lo, rows_per_seq, n_heads, S_max, chunks);
  if (e != cudaSuccess || chunks == 1) return e;
  const int R = B * rows_per_seq;
  return launch_k(tree_attn_combine_kernel, dim3((R * n_heads + 7) / 8), dim3(256), 0, L.st, L.pdl,
                  (const float *)scratch, (bf16 *)out.hi, (bf16 *)out.lo, R, n_heads, chunks);
}

}  // namespace koala
