// Persistent layer kernel: the weight-streaming GEMMs of a decoder layer and the row-wise work
// between them in ONE launch, so that the weight stream does not stop at the boundaries.
//
// A launch runs up to four phases.  A phase is a skinny GEMM (partial sums = X * [W0;W1;W2]^T, as in
// gemm_tc.cu: weights are the MMA's M, tokens the MMA's N, activations a bf16 value + residual
// pair) followed by the row-wise step that consumes its partial sums and produces the next
// phase's activations:
//     O projection   -> residual update, x * gain of the FFN norm (its scale is owed), sums of squares
//     gate/up        -> SwiGLU (applies the owed scale)
//     down           -> residual update, x * gain of the next layer's first norm
//     Q/K/V          -> rotary embedding, KV-cache write, queries as an operand pair
// One CTA per SM, all co-resident (cooperative launch).  Every phase's (weight tile, K-block)
// units are dealt evenly to the CTAs (stream-K: a CTA's run may cross tile boundaries; every
// run inside one tile is a "segment" with its own accumulator and partial-sum slot).
//   warp 0      weight-tile producer (TMA).  Weight tiles do not depend on anything, so they are
//               requested as soon as a ring stage is free, across phase boundaries; while the ring
//               stays full for long (the consumers stand at a boundary) further tiles are requested
//               into L2.
//   warp 2      activation-tile producer: a stage's activation tile is requested once the phase's
//               activations exist (a device-wide counter).
//   warp 1      MMA issuer (tcgen05.mma, fp32 accumulators in tensor memory, two buffers).
//   warps 4..7  epilogue: accumulator -> partial sums in global memory.
//   warps 4..31 row-wise step of the phase, after a device-wide barrier (every CTA's partial sums
//               of the phase are stored), spread over all CTAs; then a second counter tells the
//               producers that the next phase's activations are complete.
// While the CTAs wait at those two barriers and do the row-wise step, the ring keeps filling with
// the next phase's weights, so the HBM stream pauses only when the ring is full.
// Measured on B200 (7B shapes, 64 rows): the streaming phases reach 5.3-5.7 TB/s, but each of the four
// boundaries of a layer costs 8-14 us (barrier, row-wise step on one CTA per SM, second barrier), which
// is no less than a dependent kernel launch costs; the one-kernel-per-step path is the faster one, so
// this kernel is used only on request (KOALA_F_LAYER_KERNEL).
// Every wait (shared-memory barrier or device-wide counter) is bounded: on expiry the CTA raises
// the launch's abort word (which ends every other CTA's waits), records KOALA_E_TIMEOUT in *status,
// lets its copies land, drains its MMAs, frees its tensor memory and returns.
#include <cuda.h>

#include <cstring>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace koala {

bool tc_get_map(const void *ptr, int rows, int K_in, int box_rows, CUtensorMap *out);
int tc_smem_optin();
int tc_num_sms();

namespace {

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int UMMA_K = 16;
constexpr int W_STAGE_BYTES = BM * BK * 2;
constexpr int MAX_STAGES = 12;
constexpr int N_WORK = 896;                    // warps 4..31: row-wise steps (warps 4..7 also read the accumulators)
constexpr int X_WARP = 2;                      // activation-tile producer (warp 3 idles)
constexpr int THREADS = 128 + N_WORK;          // 1024: at most 64 registers per thread
constexpr int L2_AHEAD = 24;                   // weight tiles a CTA may request into L2 beyond its ring during a stall
constexpr long long STALL_CYCLES = 1500;       // a full ring for this long is a phase boundary, not the steady state
constexpr int E_TIMEOUT = 6;
constexpr int MAX_TILES = 1024;                // weight tiles per phase (count table in shared memory)
constexpr int RU_CHUNK = 512;                  // columns per residual-update item (128 threads x 4)

struct Phase {
  int n0, n1, n2;          // rows of the weight matrices (multiples of 128; unused ones 0)
  int tiles0, tiles1;      // cumulative 128-row tiles of matrix 0 and of matrices 0+1
  int kblocks;             // K_in / 64
  unsigned units;          // tiles * kblocks
  int ctas;                // CTAs sharing the units (the first `ctas` of the grid)
  float *Y;                // partial-sum matrices, split_stride floats apart
  int ldy;
  size_t split_stride;
  int post;                // LAYER_POST_*
  RowScale sc;             // scale owed by the consumer of this GEMM (SwiGLU, rotary step)
  const bf16 *gain;        // residual update: gain of the norm that follows
  bf16 *out_hi, *out_lo;   // residual update: x * gain [R][ncols]; SwiGLU: activations [R][ncols]; rotary: queries
  float *sumsq;            // residual update: [R][ceil(ncols / 512)] partial sums of squares
  int ncols;               // residual update: H; SwiGLU: F
  unsigned done_target, ready_target;   // counter values once every CTA of this launch has arrived
};

struct LayerParams {
  Phase ph[LAYER_MAX_PHASES];
  int n_phases;
  int R, bn, tt, tmem_cols, stages;
  float *x;                // residual stream [R][H]
  RowPlan plan;            // rotary step
  float *q_out;
  bf16 *k_cache, *v_cache;
  int rows_per_seq, n_heads, S_max;
  unsigned *sync;          // done[p] at [p], ready[p] at [LAYER_MAX_PHASES + p], abort word at [2 * LAYER_MAX_PHASES]
  int *status;
};

struct LayerMaps {
  CUtensorMap w[LAYER_MAX_PHASES][3];
  CUtensorMap x[LAYER_MAX_PHASES][2];
};

__device__ __forceinline__ unsigned ld_acquire(const unsigned *p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ unsigned ld_relaxed(const unsigned *p) {
  unsigned v;
  asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ bool mbar_test(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void named_bar_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ bool counter_reached(const unsigned *ctr, unsigned target) {
  return (int)(ld_acquire(ctr) - target) >= 0;
}
// One thread waits until *ctr reaches target; false if the limit ran out or the launch was aborted.
__device__ __forceinline__ bool counter_wait(const unsigned *ctr, unsigned target, const unsigned *abort_word) {
  const long long t0 = clock64();
  while (!counter_reached(ctr, target)) {
    if (ld_relaxed(abort_word) != 0u) return false;
    if (clock64() - t0 > WAIT_LIMIT_CYCLES) return false;
    __nanosleep(32);
  }
  return true;
}
// This CTA's share of a phase's units
__device__ __forceinline__ void unit_range(const Phase &ph, unsigned g, unsigned &lo, unsigned &hi) {
  if ((int)g < ph.ctas) {
    lo = (unsigned)(((unsigned long long)g * ph.units) / (unsigned)ph.ctas);
    hi = (unsigned)(((unsigned long long)(g + 1) * ph.units) / (unsigned)ph.ctas);
  } else {
    lo = hi = ph.units;
  }
}
__device__ __forceinline__ unsigned sk_owner(unsigned u, unsigned ctas, unsigned units) {
  return ((u + 1u) * ctas - 1u) / units;
}

// ----------------------------------------------------------------------------- row-wise steps
// Everything another CTA of this launch may have written is read past the L1 (ld.global.cg).
__device__ __forceinline__ float silu_f(float v) { return __fdividef(v, 1.f + __expf(-v)); }
__device__ __forceinline__ float row_scale(const RowScale &sc, int r) {
  if (sc.n == 0) return 1.f;
  float s = 0.f;
  for (int i = 0; i < sc.n; ++i) s += __ldcg(sc.sumsq + (size_t)r * sc.n + i);
  return rsqrtf(s * sc.inv_h + sc.eps);
}

// Partial sums of one phase as the row-wise steps see them: `cnt[tile]` matrices per 128-column tile.
struct Parts {
  const float *p;
  size_t stride;
  int ld;
  const unsigned char *cnt;      // shared memory: contributors per weight tile
  __device__ __forceinline__ int count(int c) const { return cnt[c >> 7]; }
};
constexpr int PA = 4;            // partial sums requested before the first is used
__device__ __forceinline__ void part_ld4(const Parts &P, int r, int c, int k, float4 *u) {
  const float *q = P.p + (size_t)r * P.ld + c;
#pragma unroll
  for (int s = 0; s < PA; ++s)
    u[s] = s < k ? __ldcg(reinterpret_cast<const float4 *>(q + (size_t)s * P.stride)) : make_float4(0.f, 0.f, 0.f, 0.f);
}
// sum in slot order (the same order whatever the number of slots requested ahead)
__device__ __forceinline__ float4 part_sum4(const Parts &P, int r, int c, int k, const float4 *u) {
  float4 v = u[0];
#pragma unroll
  for (int s = 1; s < PA; ++s) {
    if (s < k) { v.x += u[s].x; v.y += u[s].y; v.z += u[s].z; v.w += u[s].w; }
  }
  const float *q = P.p + (size_t)r * P.ld + c;
  for (int s = PA; s < k; ++s) {
    const float4 w = __ldcg(reinterpret_cast<const float4 *>(q + (size_t)s * P.stride));
    v.x += w.x; v.y += w.y; v.z += w.z; v.w += w.w;
  }
  return v;
}
__device__ __forceinline__ void part_ld2(const Parts &P, int r, int c, int k, float2 *u) {
  const float *q = P.p + (size_t)r * P.ld + c;
#pragma unroll
  for (int s = 0; s < PA; ++s)
    u[s] = s < k ? __ldcg(reinterpret_cast<const float2 *>(q + (size_t)s * P.stride)) : make_float2(0.f, 0.f);
}
__device__ __forceinline__ float2 part_sum2(const Parts &P, int r, int c, int k, const float2 *u) {
  float2 v = u[0];
#pragma unroll
  for (int s = 1; s < PA; ++s) {
    if (s < k) { v.x += u[s].x; v.y += u[s].y; }
  }
  const float *q = P.p + (size_t)r * P.ld + c;
  for (int s = PA; s < k; ++s) {
    const float2 w = __ldcg(reinterpret_cast<const float2 *>(q + (size_t)s * P.stride));
    v.x += w.x; v.y += w.y;
  }
  return v;
}
__device__ __forceinline__ float4 load4_bf16(const bf16 *p) {
  const uint2 u = *reinterpret_cast<const uint2 *>(p);
  const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&u.x));
  const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&u.y));
  return make_float4(a.x, a.y, b.x, b.y);
}
// v as a bf16 value + rounding-residual pair
__device__ __forceinline__ void store_pair4(bf16 *hi, bf16 *lo, size_t i, float4 v) {
  const __nv_bfloat162 h0 = __floats2bfloat162_rn(v.x, v.y), h1 = __floats2bfloat162_rn(v.z, v.w);
  uint2 u;
  u.x = *reinterpret_cast<const uint32_t *>(&h0);
  u.y = *reinterpret_cast<const uint32_t *>(&h1);
  *reinterpret_cast<uint2 *>(hi + i) = u;
  const float2 f0 = __bfloat1622float2(h0), f1 = __bfloat1622float2(h1);
  const __nv_bfloat162 l0 = __floats2bfloat162_rn(v.x - f0.x, v.y - f0.y);
  const __nv_bfloat162 l1 = __floats2bfloat162_rn(v.z - f1.x, v.w - f1.y);
  u.x = *reinterpret_cast<const uint32_t *>(&l0);
  u.y = *reinterpret_cast<const uint32_t *>(&l1);
  *reinterpret_cast<uint2 *>(lo + i) = u;
}

// x <- x + sum(partials); out <- pair(x * gain) (not normalised); sumsq[r][chunk] <- sum of x^2
// over the chunk's 512 columns.  An item is (row, chunk); a group of 128 workers takes an item.
__device__ void post_row_update(const LayerParams &P, const Phase &ph, const Parts &S, int wt, float *red /* [groups][4] */) {
  const int H = ph.ncols;
  const int chunks = (H + RU_CHUNK - 1) / RU_CHUNK;
  const int items = P.R * chunks;
  constexpr int GROUPS = N_WORK / 128;
  const int grp = wt >> 7, t = wt & 127, wig = t >> 5, lane = t & 31;
  const int per_round = GROUPS * (int)gridDim.x;
  const int rounds = (items + per_round - 1) / per_round;
  for (int rd = 0; rd < rounds; ++rd) {
    const int item = rd * per_round + GROUPS * (int)blockIdx.x + grp;
    float ss = 0.f;
    int r = 0, ch = 0;
    const bool live = item < items;
    if (live) {
      r = item / chunks;
      ch = item - r * chunks;
      const int c = ch * RU_CHUNK + t * 4;
      if (c < H) {
        float4 u[PA];
        const int k = S.count(c);
        part_ld4(S, r, c, k, u);
        float *xr = P.x + (size_t)r * H + c;
        const float4 xv = __ldcg(reinterpret_cast<const float4 *>(xr));
        const float4 gg = load4_bf16(ph.gain + c);
        const float4 p = part_sum4(S, r, c, k, u);
        const float4 o = make_float4(xv.x + p.x, xv.y + p.y, xv.z + p.z, xv.w + p.w);
        *reinterpret_cast<float4 *>(xr) = o;
        ss = o.x * o.x + o.y * o.y + o.z * o.z + o.w * o.w;
        store_pair4(ph.out_hi, ph.out_lo, (size_t)r * H + c, make_float4(o.x * gg.x, o.y * gg.y, o.z * gg.z, o.w * gg.w));
      }
    }
    ss = warp_sum(ss);
    if (lane == 0) red[grp * 4 + wig] = ss;
    named_bar_sync(3, N_WORK);
    if (live && t == 0) ph.sumsq[(size_t)r * chunks + ch] = (red[grp * 4] + red[grp * 4 + 1]) + (red[grp * 4 + 2] + red[grp * 4 + 3]);
    named_bar_sync(3, N_WORK);
  }
}

// act <- pair(SiLU(s * gate) * (s * up)), s = the row's owed RMSNorm scale; an item is four columns
// of one row.
__device__ void post_swiglu(const LayerParams &P, const Phase &ph, const Parts &S, int wt) {
  const int F = ph.ncols, q4 = F >> 2;
  const unsigned items = (unsigned)P.R * (unsigned)q4;
  const unsigned stride = gridDim.x * (unsigned)N_WORK;
  int r_cached = -1;
  float rs = 1.f;
  for (unsigned i = blockIdx.x * (unsigned)N_WORK + (unsigned)wt; i < items; i += stride) {
    const int r = (int)(i / (unsigned)q4), f = (int)(i - (unsigned)r * (unsigned)q4) * 4;
    float4 ua[PA], ub[PA];
    const int ka = S.count(f), kb = S.count(F + f);
    part_ld4(S, r, f, ka, ua);
    part_ld4(S, r, F + f, kb, ub);
    if (r != r_cached) { rs = row_scale(ph.sc, r); r_cached = r; }
    const float4 a = part_sum4(S, r, f, ka, ua), b = part_sum4(S, r, F + f, kb, ub);
    store_pair4(ph.out_hi, ph.out_lo, (size_t)r * F + f,
                make_float4(silu_f(rs * a.x) * (rs * b.x), silu_f(rs * a.y) * (rs * b.y),
                            silu_f(rs * a.z) * (rs * b.z), silu_f(rs * a.w) * (rs * b.w)));
  }
}

// Rotary embedding of q and k (pairs (i, i + 64) of a 128-dim head), KV-cache write at the row's
// slot, queries as fp32 and as an operand pair.  An item is two adjacent pairs of one (row, head).
__device__ void post_rope_kv(const LayerParams &P, const Phase &ph, const Parts &S, int wt) {
  constexpr int DH = 128, HALF = 64, HQ = 32;
  const int H = P.n_heads * DH;
  const int per_row = P.n_heads * HQ;
  const unsigned items = (unsigned)P.R * (unsigned)per_row;
  const unsigned stride = gridDim.x * (unsigned)N_WORK;
  int r_cached = -1, slot = -1, b = 0;
  float rs = 1.f;
  for (unsigned it = blockIdx.x * (unsigned)N_WORK + (unsigned)wt; it < items; it += stride) {
    const int r = (int)(it / (unsigned)per_row);
    const int p = (int)(it - (unsigned)r * (unsigned)per_row);
    const int h = p / HQ, i = (p - h * HQ) * 2;
    const int c0 = h * DH + i, c1 = c0 + HALF;
    // every partial sum of the item is requested before anything is used
    float2 uq0[PA], uq1[PA], uk0[PA], uk1[PA], uv0[PA], uv1[PA];
    const int kq = S.count(c0), kk = S.count(H + c0), kv = S.count(2 * H + c0);   // c0 and c1 share a tile
    part_ld2(S, r, c0, kq, uq0);
    part_ld2(S, r, c1, kq, uq1);
    part_ld2(S, r, H + c0, kk, uk0);
    part_ld2(S, r, H + c1, kk, uk1);
    part_ld2(S, r, 2 * H + c0, kv, uv0);
    part_ld2(S, r, 2 * H + c1, kv, uv1);
    const float4 cs = *reinterpret_cast<const float4 *>(&P.plan.rope[(size_t)r * HALF + i]);   // c0 s0 c1 s1
    if (r != r_cached) {
      rs = row_scale(ph.sc, r);
      slot = P.plan.slot[r];
      b = r / P.rows_per_seq;
      r_cached = r;
    }
    const bool wr = slot >= 0 && slot < P.S_max;
    float2 qa = part_sum2(S, r, c0, kq, uq0), qb = part_sum2(S, r, c1, kq, uq1);
    float2 ka = part_sum2(S, r, H + c0, kk, uk0), kb = part_sum2(S, r, H + c1, kk, uk1);
    float2 va = part_sum2(S, r, 2 * H + c0, kv, uv0), vb = part_sum2(S, r, 2 * H + c1, kv, uv1);
    qa.x *= rs; qa.y *= rs; qb.x *= rs; qb.y *= rs;
    const float2 ra = make_float2(qa.x * cs.x - qb.x * cs.y, qa.y * cs.z - qb.y * cs.w);
    const float2 rb = make_float2(qb.x * cs.x + qa.x * cs.y, qb.y * cs.z + qa.y * cs.w);
    *reinterpret_cast<float2 *>(P.q_out + (size_t)r * H + c0) = ra;
    *reinterpret_cast<float2 *>(P.q_out + (size_t)r * H + c1) = rb;
    {
      const __nv_bfloat162 ha = __floats2bfloat162_rn(ra.x, ra.y), hb = __floats2bfloat162_rn(rb.x, rb.y);
      const float2 fa = __bfloat1622float2(ha), fb = __bfloat1622float2(hb);
      *reinterpret_cast<__nv_bfloat162 *>(ph.out_hi + (size_t)r * H + c0) = ha;
      *reinterpret_cast<__nv_bfloat162 *>(ph.out_hi + (size_t)r * H + c1) = hb;
      *reinterpret_cast<__nv_bfloat162 *>(ph.out_lo + (size_t)r * H + c0) = __floats2bfloat162_rn(ra.x - fa.x, ra.y - fa.y);
      *reinterpret_cast<__nv_bfloat162 *>(ph.out_lo + (size_t)r * H + c1) = __floats2bfloat162_rn(rb.x - fb.x, rb.y - fb.y);
    }
    if (!wr) continue;
    ka.x *= rs; ka.y *= rs; kb.x *= rs; kb.y *= rs;
    va.x *= rs; va.y *= rs; vb.x *= rs; vb.y *= rs;
    const size_t base = (((size_t)b * P.n_heads + h) * P.S_max + slot) * DH + i;
    *reinterpret_cast<__nv_bfloat162 *>(P.k_cache + base) = __floats2bfloat162_rn(ka.x * cs.x - kb.x * cs.y, ka.y * cs.z - kb.y * cs.w);
    *reinterpret_cast<__nv_bfloat162 *>(P.k_cache + base + HALF) = __floats2bfloat162_rn(kb.x * cs.x + ka.x * cs.y, kb.y * cs.z + ka.y * cs.w);
    *reinterpret_cast<__nv_bfloat162 *>(P.v_cache + base) = __floats2bfloat162_rn(va.x, va.y);
    *reinterpret_cast<__nv_bfloat162 *>(P.v_cache + base + HALF) = __floats2bfloat162_rn(vb.x, vb.y);
  }
}

// ----------------------------------------------------------------------------- the kernel
__global__ void __launch_bounds__(THREADS, 1)
layer_stream_kernel(const __grid_constant__ LayerMaps M, const __grid_constant__ LayerParams P) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ uint64_t full_bar[MAX_STAGES];
  __shared__ uint64_t empty_bar[MAX_STAGES];
  __shared__ uint64_t acc_full[2];
  __shared__ uint64_t acc_empty[2];
  __shared__ uint64_t drain_bar;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int s_error;
  __shared__ int s_flag;                 // result of a device-wide wait, shared with the workers
  __shared__ float s_red[4 * (N_WORK / 128)];
  __shared__ unsigned char s_cnt[MAX_TILES];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const unsigned g = blockIdx.x;
  const uint32_t raw = smem_u32(smem_raw);
  unsigned char *tiles = smem_raw + ((1024u - (raw & 1023u)) & 1023u);
  const int x_stage_bytes = P.bn * BK * 2;
  const int stage_bytes = W_STAGE_BYTES + x_stage_bytes;
  const int NS = P.stages;
  unsigned *const done_ctr = P.sync;
  unsigned *const ready_ctr = P.sync + LAYER_MAX_PHASES;
  unsigned *const abort_word = P.sync + 2 * LAYER_MAX_PHASES;

  // this CTA's unit ranges
  unsigned u_lo[LAYER_MAX_PHASES], u_hi[LAYER_MAX_PHASES];
  int n_total = 0;
#pragma unroll
  for (int p = 0; p < LAYER_MAX_PHASES; ++p) {
    u_lo[p] = u_hi[p] = 0;
    if (p < P.n_phases) {
      unit_range(P.ph[p], g, u_lo[p], u_hi[p]);
      n_total += (int)(u_hi[p] - u_lo[p]);
    }
  }

  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&acc_full[i], 1);
      mbar_init(&acc_empty[i], 4);
    }
    mbar_init(&drain_bar, 1);
    s_error = 0;
    s_flag = 1;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&tmem_base_slot)), "r"((uint32_t)(2 * P.tmem_cols)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_acc = tmem_base_slot;

  if (warp == 0) {
    // ---------------------------------------------------------------- weight-tile producer
    if (lane == 0) {
      bool ok = true;
      int s = 0;
      uint32_t round = 0;
      // L2 prefetch cursor: unit (pf_p, pf_u) is `pf_ahead` units past the load cursor's ring
      int pf_p = 0, pf_tile = 0, pf_kb = 0, pf_ahead = 0;
      unsigned pf_u = 0;
      auto pf_enter = [&]() {          // first unit of phase pf_p (skipping phases without units)
        while (pf_p < P.n_phases && u_lo[pf_p] == u_hi[pf_p]) ++pf_p;
        if (pf_p < P.n_phases) {
          pf_u = u_lo[pf_p];
          pf_tile = (int)(pf_u / (unsigned)P.ph[pf_p].kblocks);
          pf_kb = (int)(pf_u % (unsigned)P.ph[pf_p].kblocks);
        }
      };
      auto pf_advance = [&]() {
        if (pf_p >= P.n_phases) return;
        if (++pf_kb == P.ph[pf_p].kblocks) { pf_kb = 0; ++pf_tile; }
        if (++pf_u == u_hi[pf_p]) { ++pf_p; pf_enter(); }
      };
      pf_enter();
      for (int i = 0; i < NS; ++i) pf_advance();       // the ring's own units need no prefetch
      for (int p = 0; p < P.n_phases && ok; ++p) {
        if (u_lo[p] == u_hi[p]) continue;
        const Phase &ph = P.ph[p];
        const int KB = ph.kblocks;
        int tile = (int)(u_lo[p] / (unsigned)KB), kb = (int)(u_lo[p] % (unsigned)KB);
        int mat = 0, row0 = 0;
        auto place = [&]() {
          mat = 0; row0 = tile * BM;
          if (tile >= ph.tiles1) { mat = 2; row0 = (tile - ph.tiles1) * BM; }
          else if (tile >= ph.tiles0) { mat = 1; row0 = (tile - ph.tiles0) * BM; }
        };
        place();
        for (unsigned u = u_lo[p]; u < u_hi[p]; ++u) {
          if (round > 0) {
            // Ring full.  In steady state a stage frees within a fraction of a microsecond.  A
            // longer wait means that the consumers stand at a phase boundary (device-wide barrier,
            // row-wise step): then the tiles beyond the ring are requested into L2, so that HBM keeps
            // streaming and the next phase starts from L2.
            const long long t0 = clock64();
            while (!mbar_test(&empty_bar[s], (round - 1u) & 1u)) {
              const long long waited = clock64() - t0;
              if (waited > WAIT_LIMIT_CYCLES) { ok = false; break; }
              if (waited > STALL_CYCLES && pf_ahead < L2_AHEAD && pf_p < P.n_phases) {
                const Phase &q = P.ph[pf_p];
                int pm = 0, pr = pf_tile * BM;
                if (pf_tile >= q.tiles1) { pm = 2; pr = (pf_tile - q.tiles1) * BM; }
                else if (pf_tile >= q.tiles0) { pm = 1; pr = (pf_tile - q.tiles0) * BM; }
                asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];"
                             ::"l"(&M.w[pf_p][pm]), "r"(pf_kb * BK), "r"(pr) : "memory");
                ++pf_ahead;
                pf_advance();
              }
            }
            if (!ok) break;
          }
          mbar_expect_tx(&full_bar[s], (uint32_t)stage_bytes);
          tma_load_2d(&M.w[p][mat], &full_bar[s], tiles + (size_t)s * stage_bytes, kb * BK, row0);
          if (pf_ahead > 0) --pf_ahead; else pf_advance();     // the prefetch window slides with the loads
          if (++s == NS) { s = 0; ++round; }
          if (++kb == KB) { kb = 0; ++tile; place(); }
        }
      }
      if (!ok) {
        atomicExch(&s_error, 1);
        atomicExch(abort_word, 1u);
      }
    }
  } else if (warp == X_WARP) {
    // ---------------------------------------------------------------- activation-tile producer
    if (lane == 0) {
      const int lo_off = P.tt * BK * 2;
      bool ok = true;
      int s = 0;
      uint32_t round = 0;
      for (int p = 0; p < P.n_phases && ok; ++p) {
        if (u_lo[p] == u_hi[p]) continue;
        const Phase &ph = P.ph[p];
        const int KB = ph.kblocks;
        if (p == 0) {
          pdl_wait();                    // the first phase's activations come from the kernel before this one
        } else {
          ok = counter_wait(&ready_ctr[p], ph.ready_target, abort_word);
          if (!ok) break;
          asm volatile("fence.proxy.async;" ::: "memory");     // generic-proxy writes of other CTAs -> TMA reads
        }
        int kb = (int)(u_lo[p] % (unsigned)KB);
        for (unsigned u = u_lo[p]; u < u_hi[p]; ++u) {
          if (round > 0) {
            ok = mbar_wait(&empty_bar[s], (round - 1u) & 1u);
            if (!ok) break;
          }
          unsigned char *xd = tiles + (size_t)s * stage_bytes + W_STAGE_BYTES;
          tma_load_2d(&M.x[p][0], &full_bar[s], xd, kb * BK, 0);
          tma_load_2d(&M.x[p][1], &full_bar[s], xd + lo_off, kb * BK, 0);
          if (++s == NS) { s = 0; ++round; }
          if (++kb == KB) kb = 0;
        }
      }
      if (!ok) {
        atomicExch(&s_error, 1);
        atomicExch(abort_word, 1u);
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(P.bn >> 3) << 17) |
                             ((uint32_t)(BM >> 4) << 24);
      const uint64_t desc0 = smem_desc_sw128(smem_u32(tiles));
      const uint64_t stage_step = (uint64_t)(stage_bytes >> 4), x_step = (uint64_t)(W_STAGE_BYTES >> 4);
      bool ok = true;
      int s = 0, seg = 0;
      uint32_t fpar = 0;
      for (int p = 0; p < P.n_phases && ok; ++p) {
        if (u_lo[p] == u_hi[p]) continue;
        const int KB = P.ph[p].kblocks;
        int kb = (int)(u_lo[p] % (unsigned)KB);
        bool seg_start = true;
        for (unsigned u = u_lo[p]; u < u_hi[p]; ++u) {
          const int buf = seg & 1;
          if (seg_start && seg >= 2) {
            ok = mbar_wait(&acc_empty[buf], (uint32_t)((seg >> 1) - 1) & 1u);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          }
          ok = mbar_wait(&full_bar[s], fpar);
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint64_t da = desc0 + stage_step * (uint64_t)s;
          const uint64_t db = da + x_step;
          const uint32_t dacc = tmem_acc + (uint32_t)(buf * P.tmem_cols);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k)
            umma_bf16(dacc, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, (!seg_start || k > 0) ? 1u : 0u);
          umma_commit(&empty_bar[s]);
          const bool seg_end = (kb == KB - 1) || (u + 1 == u_hi[p]);
          if (seg_end) {
            umma_commit(&acc_full[buf]);
            ++seg;
          }
          seg_start = seg_end;
          if (++kb == KB) kb = 0;
          if (++s == NS) { s = 0; fpar ^= 1u; }
        }
      }
      if (!ok) {
        atomicExch(&s_error, 1);
        atomicExch(abort_word, 1u);
      }
    }
  } else if (warp >= 4) {
    // ---------------------------------------------------------------- epilogue + row-wise steps
    const int wt = threadIdx.x - 128;             // worker index 0..895
    const bool epi = warp < 8;                    // warps 4..7 read the accumulators (one TMEM lane quarter each)
    const int quarter = warp & 3;
    bool ok = true;
    int seg = 0;
    pdl_wait();       // the partial-sum buffer may still be read, and x / the row plan written, by the kernel before
    for (int p = 0; p < P.n_phases; ++p) {
      const Phase &ph = P.ph[p];
      if (epi && ok) {
        const int KB = ph.kblocks;
        unsigned u = u_lo[p];
        while (u < u_hi[p]) {
          const int tile = (int)(u / (unsigned)KB);
          unsigned seg_hi = (unsigned)(tile + 1) * KB;
          if (seg_hi > u_hi[p]) seg_hi = u_hi[p];
          const int buf = seg & 1;
          ok = __all_sync(0xffffffffu, mbar_wait(&acc_full[buf], (uint32_t)(seg >> 1) & 1u));
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          int row0 = tile * BM, col_off = 0;
          if (tile >= ph.tiles1) { row0 = (tile - ph.tiles1) * BM; col_off = ph.n0 + ph.n1; }
          else if (tile >= ph.tiles0) { row0 = (tile - ph.tiles0) * BM; col_off = ph.n0; }
          const int slot = (int)g - (int)sk_owner((unsigned)tile * KB, (unsigned)ph.ctas, ph.units);
          const int feat = row0 + quarter * 32 + lane;
          float *Yp = ph.Y + (size_t)slot * ph.split_stride + col_off + feat;
          const uint32_t lane_base = tmem_acc + (uint32_t)(buf * P.tmem_cols) + ((uint32_t)(quarter * 32) << 16);
          for (int c0 = 0; c0 < P.tt; c0 += 16) {
            uint32_t v[16], w[16];
            tmem_ld16(lane_base + (uint32_t)c0, v);
            tmem_ld16(lane_base + (uint32_t)(P.tt + c0), w);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int t = c0 + j;
              if (t < P.R) Yp[(size_t)t * ph.ldy] = __uint_as_float(v[j]) + __uint_as_float(w[j]);
            }
          }
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          __syncwarp();
          if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&acc_empty[buf])) : "memory");
          ++seg;
          u = seg_hi;
        }
        if (!ok) {
          atomicExch(&s_error, 1);
          atomicExch(abort_word, 1u);
        }
      }
      // this CTA's partial sums of the phase are stored: tell the device
      named_bar_sync(2, N_WORK);
      if (wt == 0) {
        __threadfence();
        atomicAdd(&done_ctr[p], 1u);
      }
      if (ph.post == LAYER_POST_NONE) continue;
      // every CTA's partial sums must be there before the row-wise step reads them
      if (wt == 0) s_flag = counter_wait(&done_ctr[p], ph.done_target, abort_word) ? 1 : 0;
      named_bar_sync(2, N_WORK);
      const bool go = s_flag != 0;
      if (go) {
        // contributors per weight tile (the CTAs whose unit runs touch it): slots 0 .. cnt - 1 hold its partial sums
        const int n_tiles = ph.tiles1 + ph.n2 / BM;
        for (int t = wt; t < n_tiles; t += N_WORK) {
          const unsigned first = sk_owner((unsigned)t * ph.kblocks, (unsigned)ph.ctas, ph.units);
          const unsigned last = sk_owner((unsigned)(t + 1) * ph.kblocks - 1u, (unsigned)ph.ctas, ph.units);
          s_cnt[t] = (unsigned char)(last - first + 1u);
        }
        named_bar_sync(3, N_WORK);
        const Parts S{ph.Y, ph.split_stride, ph.ldy, s_cnt};
        if (ph.post == LAYER_POST_ROW_UPDATE) post_row_update(P, ph, S, wt, s_red);
        else if (ph.post == LAYER_POST_SWIGLU) post_swiglu(P, ph, S, wt);
        else post_rope_kv(P, ph, S, wt);
      } else {
        ok = false;
      }
      // the next phase's activations are written: after the last CTA's arrival the producers may load them
      named_bar_sync(2, N_WORK);
      if (wt == 0) {
        if (!go) {
          atomicExch(&s_error, 1);
          atomicExch(abort_word, 1u);
        }
        __threadfence();
        if (p + 1 < P.n_phases) atomicAdd(&ready_ctr[p + 1], 1u);
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    if (s_error) {
      if (lane == 0) {
        umma_commit(&drain_bar);
        (void)mbar_wait(&drain_bar, 0);
      }
      __syncwarp();
    }
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"((uint32_t)(2 * P.tmem_cols))
                 : "memory");
  }
  if (threadIdx.x == 0 && s_error && P.status) atomicMax(P.status, E_TIMEOUT);
}

SmemOptIn g_optin;

}  // namespace

// Stream-K plan of one phase: how many of the grid's CTAs share its units.  Every sharing CTA gets
// at least 8 units (so that no tile has more than `max_slots` contributors, all of them
// consecutive CTAs).  Returns 0 if even one CTA per ... cannot respect max_slots.
static int plan_ctas(int tiles, int kblocks, int grid, int max_slots, int *slots_out) {
  const long long units = (long long)tiles * kblocks;
  long long g = grid;
  if (g > units / 8) g = units / 8;
  if (g < 1) g = 1;
  auto slots_of = [&](long long gg) {
    const long long per = units / gg;
    return (int)((kblocks + per - 1) / per) + ((units % gg) || (kblocks % per) ? 1 : 0);
  };
  while (g > 1 && slots_of(g) > max_slots) --g;
  *slots_out = slots_of(g);
  return (int)g;
}

bool layer_stream_supported(const LayerJob &job) {
  if (job.n_phases < 1 || job.n_phases > LAYER_MAX_PHASES || job.R < 1 || job.R > 128) return false;
  if (tc_smem_optin() < 64 * 1024 || tc_num_sms() < 1) return false;
  for (int p = 0; p < job.n_phases; ++p) {
    const LayerPhaseJob &j = job.ph[p];
    if (j.K_in % BK != 0 || j.K_in < BK || j.X.hi == nullptr || j.X.lo == nullptr) return false;
    if (((uintptr_t)j.X.hi & 15u) || ((uintptr_t)j.X.lo & 15u)) return false;
    if (j.m.n < 1 || j.m.n > 3) return false;
    {
      long long nt = 0;
      for (int i = 0; i < j.m.n; ++i) nt += j.m.n_out[i] / BM;
      if (nt > MAX_TILES) return false;
    }
    for (int i = 0; i < j.m.n; ++i)
      if (j.m.n_out[i] < BM || (j.m.n_out[i] % BM) != 0 || ((uintptr_t)j.m.W[i] & 15u)) return false;
    if (j.post == LAYER_POST_ROW_UPDATE && (j.ncols % 4 != 0 || j.ldy % 4 != 0 || j.split_stride % 4 != 0)) return false;
    if (j.post == LAYER_POST_SWIGLU && (j.ncols % 4 != 0 || j.ldy % 4 != 0 || j.split_stride % 4 != 0)) return false;
    if (j.post == LAYER_POST_ROPE_KV && (job.head_dim != 128 || j.ldy % 2 != 0 || j.split_stride % 2 != 0)) return false;
  }
  return true;
}

cudaError_t layer_stream(Launch L, const LayerJob &job, unsigned *sync, unsigned *use_count, int *status,
                         SplitIn *outs) {
  if (!layer_stream_supported(job)) return cudaErrorInvalidValue;
  LayerMaps Mx;
  LayerParams P;
  memset(&P, 0, sizeof(P));
  const int grid = tc_num_sms();
  int tt = ((job.R + 15) / 16) * 16;
  if (tt > job.x_rows_alloc) return cudaErrorInvalidValue;
  const int bn = 2 * tt;
  int cols = 32;
  while (cols < bn) cols <<= 1;
  P.R = job.R;
  P.tt = tt;
  P.bn = bn;
  P.tmem_cols = cols;
  const int stage_bytes = W_STAGE_BYTES + bn * BK * 2;
  int stages = (tc_smem_optin() - 2048) / stage_bytes;
  if (stages > MAX_STAGES) stages = MAX_STAGES;
  if (stages < 2) return cudaErrorInvalidValue;
  P.stages = stages;
  P.n_phases = job.n_phases;
  P.x = job.x;
  P.plan = job.plan;
  P.q_out = job.q_out;
  P.k_cache = (bf16 *)job.k_cache;
  P.v_cache = (bf16 *)job.v_cache;
  P.rows_per_seq = job.rows_per_seq;
  P.n_heads = job.n_heads;
  P.S_max = job.S_max;
  P.sync = sync;
  P.status = status;
  for (int p = 0; p < job.n_phases; ++p) {
    const LayerPhaseJob &j = job.ph[p];
    Phase &ph = P.ph[p];
    ph.n0 = j.m.n_out[0];
    ph.n1 = j.m.n > 1 ? j.m.n_out[1] : 0;
    ph.n2 = j.m.n > 2 ? j.m.n_out[2] : 0;
    ph.tiles0 = ph.n0 / BM;
    ph.tiles1 = ph.tiles0 + ph.n1 / BM;
    const int tiles = ph.tiles1 + ph.n2 / BM;
    ph.kblocks = j.K_in / BK;
    ph.units = (unsigned)((long long)tiles * ph.kblocks);
    int slots = 1;
    ph.ctas = plan_ctas(tiles, ph.kblocks, grid, j.max_slots, &slots);
    if (slots > j.max_slots) return cudaErrorInvalidValue;
    ph.Y = j.Y;
    ph.ldy = j.ldy;
    ph.split_stride = j.split_stride;
    ph.post = j.post;
    ph.sc = j.sc;
    ph.gain = (const bf16 *)j.gain;
    ph.out_hi = (bf16 *)j.out.hi;
    ph.out_lo = (bf16 *)j.out.lo;
    ph.sumsq = j.sumsq;
    ph.ncols = j.ncols;
    if (outs) outs[p] = SplitIn{j.Y, slots, j.split_stride, j.ldy, (unsigned)ph.ctas, ph.units, (unsigned)ph.kblocks};
    ph.done_target = (use_count[p] + 1u) * (unsigned)grid;     // use_count advances once the launch is accepted
    ph.ready_target = ph.done_target;
    for (int i = 0; i < 3; ++i) {
      const int k = i < j.m.n ? i : 0;
      if (!tc_get_map(j.m.W[k], j.m.n_out[k], j.K_in, BM, &Mx.w[p][i])) return cudaErrorInvalidValue;
    }
    if (!tc_get_map(j.X.hi, job.x_rows_alloc, j.K_in, tt, &Mx.x[p][0])) return cudaErrorInvalidValue;
    if (!tc_get_map(j.X.lo, job.x_rows_alloc, j.K_in, tt, &Mx.x[p][1])) return cudaErrorInvalidValue;
  }
  for (int p = job.n_phases; p < LAYER_MAX_PHASES; ++p) {
    for (int i = 0; i < 3; ++i) Mx.w[p][i] = Mx.w[0][0];
    Mx.x[p][0] = Mx.x[p][1] = Mx.x[0][0];
  }
  const size_t smem = (size_t)stages * stage_bytes + 1024;
  cudaError_t e = g_optin.ensure((const void *)layer_stream_kernel, smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = L.st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = L.pdl ? 1 : 0;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  ++g_launches;
  e = cudaLaunchKernelEx(&cfg, layer_stream_kernel, Mx, P);
  if (e == cudaSuccess)
    for (int p = 0; p < job.n_phases; ++p) use_count[p] += 1u;
  return e;
}

}  // namespace koala
