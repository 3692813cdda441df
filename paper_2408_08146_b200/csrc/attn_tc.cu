// Tree-masked attention for bf16 caches with head_dim 128 on the 5th-generation tensor cores.
//
// One CTA = one (key chunk, head, sequence) and ALL query rows of that sequence (at most 128 =
// the MMA's M).  The chunk's keys are walked in tiles of 64.  Per tile:
//   S[128 x 64]  = Q K^T          tcgen05.mma, A = Q (K-major), B = K tile (K-major), fp32 in TMEM
//   P            = exp2(S*c - m)  by the thread that owns the query row's TMEM lane: tcgen05.ld,
//                                 mask, row max / sum without shuffles, P written to shared memory
//   O[128x128]  += P V            tcgen05.mma, A = P (K-major), B = V tile as stored, [key][dim],
//                                 which is the MN-major operand form; O stays in tensor memory
// O accumulates over all tiles of the chunk.  A row's exponentials are relative to a reference
// maximum that is raised only when a tile's maximum exceeds it by more than 2^8; only then is the
// row's O rescaled in tensor memory (tcgen05.ld / st), so in the common case the rows never wait
// for P V: the tensor pipe computes S of tile t+1 and P V of tile t-1 while the rows turn S of tile
// t into P (two S buffers in tensor memory, two P buffers in shared memory).  Q and P enter the
// MMAs as bf16 pairs (value + rounding residual: two accumulating MMAs), so only the cached K and V
// carry bf16 rounding.  Q (written as a pair by the rotary-embedding kernel) and the K/V tiles
// arrive by TMA with the 128-byte swizzle, K/V in a three-stage ring.
// Warps 0..3 own the rows, warp 4 lane 0 issues the copies, warp 5 lane 0 the MMAs.
// With several chunks the CTAs of one (head, sequence) form a thread-block cluster: every CTA
// pushes, into each peer's shared memory, that peer's slice of the head dimension of its
// unnormalised (O, m, l); after a cluster barrier every CTA merges its slice over the chunks in
// chunk order from its own shared memory and writes it as a matrix-multiply operand pair.  (The
// receive buffer reuses the K/V ring, so a first cluster barrier makes sure that every peer is done
// with its tiles.)
// The mask is: slots below ctx_len visible to every row; slot ctx_len + j visible to a row iff
// bit j of its 128-bit mask; slots from kv_len on invisible.
// Every wait is bounded: on expiry the kernel records a timeout in *status and returns.
#include "common.cuh"
#include "tc_ptx.cuh"

namespace koala {

bool tc_get_map(const void *ptr, int rows, int K_in, int box_rows, CUtensorMap *out);
int tc_smem_optin();
int tc_num_sms();

namespace {

constexpr int DH = 128;
constexpr int TK = 64;                       // keys per tile
constexpr int NKV = 3;                       // K/V stages
constexpr int SUB = 64 * 64 * 2;             // one [64 keys][64 dims] block: 8 KB
constexpr int QSUB = 128 * 64 * 2;           // one [128 rows][64 columns] block: 16 KB
constexpr int OFF_Q = 0;                     // Q hi (2 blocks), Q lo (2 blocks)
constexpr int OFF_KV = 4 * QSUB;             // stages of K (2 blocks) + V (2 blocks)
constexpr int KV_STAGE = 4 * SUB;
constexpr int OFF_P = OFF_KV + NKV * KV_STAGE;   // two buffers of P hi, P lo
constexpr int P_BUF = 2 * QSUB;
constexpr int SMEM_BYTES = OFF_P + 2 * P_BUF;    // 224 KB
constexpr int THREADS = 192;
constexpr int E_TIMEOUT = 6;
constexpr int TMEM_COLS = 256;               // S: 2 x 64 columns, O: 128 columns
constexpr int COL_S = 0, COL_O = 128;
constexpr float RESCALE_STEP = 8.f;          // O is rescaled only when a row's maximum grows by more than 2^8
// the chunk-merge buffer reuses the K/V ring once every CTA of the cluster is done with its tiles
static_assert(8 * 128 * (DH / 8 + 4) * 4 <= NKV * KV_STAGE && 128 * (DH + 4) * 4 <= NKV * KV_STAGE,
              "the chunk-merge buffer fits in the K/V ring");

__device__ __forceinline__ void split_pack(float x, float y, uint32_t &hi, uint32_t &lo) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(x, y);
  const float2 hf = __bfloat1622float2(h);
  const __nv_bfloat162 l = __floats2bfloat162_rn(x - hf.x, y - hf.y);
  hi = *reinterpret_cast<const uint32_t *>(&h);
  lo = *reinterpret_cast<const uint32_t *>(&l);
}
// 2^x for x <= 0 (or -inf): one MUFU instruction; results below 2^-126 flush to zero
__device__ __forceinline__ float ex2_fast(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Probabilities p in [0, 1] as a bf16 pair: hi = p truncated to bf16 (exactly representable, so
// p - hi is exact), lo = that remainder rounded to bf16.  |p - hi - lo| <= 2^-17 p.
__device__ __forceinline__ void split_pack_trunc(float x, float y, uint32_t &hi, uint32_t &lo) {
  const uint32_t xb = __float_as_uint(x) & 0xffff0000u, yb = __float_as_uint(y) & 0xffff0000u;
  hi = __byte_perm(xb, yb, 0x7632);                 // (y.hi16 << 16) | x.hi16
  const __nv_bfloat162 l = __floats2bfloat162_rn(x - __uint_as_float(xb), y - __uint_as_float(yb));
  lo = *reinterpret_cast<const uint32_t *>(&l);
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ uint32_t peer_addr(uint32_t local_addr, uint32_t rank) {
  uint32_t ra;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_addr), "r"(rank));
  return ra;
}
__device__ __forceinline__ void st_cluster_v4(uint32_t ra, float a, float b, float c, float d) {
  asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(ra), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 64-bit visibility of the keys key0 .. key0+63 for a row with tree mask (m1:m0)
__device__ __forceinline__ uint64_t tile_visibility(uint64_t m0, uint64_t m1, int key0, int ctx, int kv_len) {
  uint64_t w;
  const int shift = key0 - ctx;
  if (shift <= -64) w = ~0ull;
  else if (shift < 0) w = (m0 << (-shift)) | ((1ull << (-shift)) - 1ull);
  else if (shift == 0) w = m0;
  else if (shift < 64) w = (m0 >> shift) | (m1 << (64 - shift));
  else if (shift < 128) w = m1 >> (shift - 64);
  else w = 0ull;
  const int n_valid = kv_len - key0;
  if (n_valid <= 0) w = 0ull;
  else if (n_valid < 64) w &= (1ull << n_valid) - 1ull;
  return w;
}

struct AttnParams {
  RowPlan plan;
  bf16 *out, *out_lo;      // [R][n_heads * 128]
  int rows_per_seq, n_heads, S_max, chunks;
  int longest_first;       // 1: grid slot y / n_heads takes the sequence with that rank in descending cache length
  int *status;
};

// DUP (at most 64 query rows): the rows are loaded twice, into MMA rows r and r + 64, so that all
// four row warps work: warps 0,1 take the first 32 keys of every tile and the first 64 output
// dims of rows 0..63, warps 2,3 the other halves of the same rows (tile row maxima are exchanged
// through shared memory).  Otherwise warp w owns rows 32w .. 32w+31 entirely.
template <bool DUP>
__global__ void __launch_bounds__(THREADS, 1)
tree_attn_tc_kernel(const __grid_constant__ CUtensorMap tmQh, const __grid_constant__ CUtensorMap tmQl,
                    const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                    const AttnParams P) {
  constexpr int NC = DUP ? 32 : 64;      // score columns (keys of a tile) per thread
  constexpr int ND = DUP ? 64 : 128;     // output dims per thread
  extern __shared__ unsigned char smem_raw[];
  __shared__ uint64_t q_full, kv_full[NKV], kv_empty[NKV], s_full[2], p_full[2], pv_done[2], x_bar[2], drain_bar;
  __shared__ float xch[2][128];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int s_error;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t raw = smem_u32(smem_raw);
  unsigned char *sm = smem_raw + ((1024u - (raw & 1023u)) & 1023u);
  const uint32_t sb = smem_u32(sm);
  const int c = blockIdx.x;
  int b = blockIdx.y / P.n_heads;
  const int h = blockIdx.y % P.n_heads;
  const int H = P.n_heads * DH;
  const int n_q = (P.rows_per_seq + 31) >> 5;             // 32-row groups in use
  const int n_arrive = DUP ? 2 * n_q : n_q;               // row warps in use

  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    mbar_init(&q_full, 1);
    for (int s = 0; s < NKV; ++s) { mbar_init(&kv_full[s], 1); mbar_init(&kv_empty[s], 1); }
    mbar_init(&drain_bar, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&s_full[i], 1);
      mbar_init(&p_full[i], (uint32_t)n_arrive);
      mbar_init(&pv_done[i], 1);
      mbar_init(&x_bar[i], 2);
    }
    s_error = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmQh) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmQl) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmK) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmV) : "memory");
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&tmem_base_slot)), "r"((uint32_t)TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_slot;

  pdl_wait();                      // Q, the tree rows of K/V and the row plan come from earlier kernels
  if (P.longest_first) {
    // More CTAs than SMs: the CTAs beyond the first round start when the first ones finish, so the
    // sequences are taken longest first and the late CTAs belong to the shortest one.  Lane l holds
    // sequence l's length; its rank is the number of sequences that are longer (ties: lower index).
    const int nb = (int)gridDim.y / P.n_heads;              // <= 32 here
    const int len_l = lane < nb ? P.plan.kv_len[lane] : -1;
    int rank = 0;
    for (int j = 0; j < nb; ++j) {
      const int len_j = __shfl_sync(0xffffffffu, len_l, j);
      rank += (len_j > len_l || (len_j == len_l && j < lane)) ? 1 : 0;
    }
    const unsigned hit = __ballot_sync(0xffffffffu, lane < nb && rank == b);
    b = hit ? __ffs(hit) - 1 : b;
  }
  if (threadIdx.x == 128) {        // warp 4 lane 0: the queries do not depend on the plan
    mbar_expect_tx(&q_full, (uint32_t)(4 * QSUB));
#pragma unroll
    for (int part = 0; part < 2; ++part)
#pragma unroll
      for (int hb = 0; hb < 2; ++hb)
#pragma unroll
        for (int rh = 0; rh < 2; ++rh)
          tma_load_2d(part ? &tmQl : &tmQh, &q_full, sm + OFF_Q + (part * 2 + hb) * QSUB + rh * (QSUB / 2),
                      h * DH + 64 * hb, b * P.rows_per_seq + (DUP ? 0 : 64 * rh));
  }
  const int ctx = P.plan.ctx_len[b];
  int kv_len = P.plan.kv_len[b];
  kv_len = kv_len > P.S_max ? P.S_max : kv_len;
  const int n_tiles = (kv_len + TK - 1) / TK;
  const int tile_lo = (int)(((long long)n_tiles * c) / P.chunks);
  const int tile_hi = (int)(((long long)n_tiles * (c + 1)) / P.chunks);
  const int T = tile_hi - tile_lo;

  // row ownership of warps 0..3
  const int rq = DUP ? (warp & 1) : warp;                   // 32-row group
  const int half = DUP ? (warp >> 1) : 0;                   // which half of the keys / dims
  const int row = rq * 32 + lane;
  const bool row_warp = warp < 4 && rq < n_q;
  const bool row_in = row_warp && row < P.rows_per_seq;
  const int r_glob = b * P.rows_per_seq + (row_in ? row : 0);
  float acc[ND];
  float m_run = -INFINITY, l_run = 0.f;

  if (warp == 4) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      const int y0 = (b * P.n_heads + h) * P.S_max;
      bool ok = true;
      int issued = 0;
      for (int t = 0; t < T; ++t) {
        const int s = t % NKV;
        if (t >= NKV) {
          ok = mbar_wait(&kv_empty[s], (uint32_t)((t / NKV) - 1) & 1u);
          if (!ok) break;
        }
        mbar_expect_tx(&kv_full[s], (uint32_t)KV_STAGE);
        unsigned char *dst = sm + OFF_KV + s * KV_STAGE;
        const int y = y0 + (tile_lo + t) * TK;
        tma_load_2d(&tmK, &kv_full[s], dst, 0, y);
        tma_load_2d(&tmK, &kv_full[s], dst + SUB, 64, y);
        tma_load_2d(&tmV, &kv_full[s], dst + 2 * SUB, 0, y);
        tma_load_2d(&tmV, &kv_full[s], dst + 3 * SUB, 64, y);
        issued = t + 1;
      }
      if (!ok) {
        atomicExch(&s_error, 1);
        // let the copies already requested land before the block's memory goes away
        for (int t = issued > NKV ? issued - NKV : 0; t < issued; ++t)
          (void)mbar_wait(&kv_full[t % NKV], (uint32_t)(t / NKV) & 1u);
      }
      if (T == 0 || !ok) (void)mbar_wait(&q_full, 0);      // nobody else waits for Q then
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      // D fp32, A and B bf16; S: N = 64, both K-major; O_t: N = 128, B MN-major
      const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(TK >> 3) << 17) | ((128u >> 4) << 24);
      const uint32_t idesc_o = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(DH >> 3) << 17) |
                               ((128u >> 4) << 24);
      auto issue_s = [&](int t) -> bool {
        const int s = t % NKV;
        if (!mbar_wait(&kv_full[s], (uint32_t)(t / NKV) & 1u)) return false;
        tc_fence_after();
        const uint32_t kb = sb + OFF_KV + s * KV_STAGE;
        const uint32_t d = tmem + (uint32_t)(COL_S + (t & 1) * TK);
#pragma unroll
        for (int part = 0; part < 2; ++part) {            // Q value, then Q residual
#pragma unroll
          for (int hb = 0; hb < 2; ++hb) {                 // 64-dim block
            const uint64_t da = smem_desc_sw128(sb + OFF_Q + (part * 2 + hb) * QSUB);
            const uint64_t db = smem_desc_sw128(kb + hb * SUB);
#pragma unroll
            for (int k = 0; k < 4; ++k)
              umma_bf16(d, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc_s, (part | hb | k) ? 1u : 0u);
          }
        }
        umma_commit(&s_full[t & 1]);
        return true;
      };
      bool ok = T > 0 ? mbar_wait(&q_full, 0) : true;
      if (ok && T > 0) ok = issue_s(0);
      for (int t = 0; t < T && ok; ++t) {
        if (t + 1 < T) { ok = issue_s(t + 1); if (!ok) break; }
        ok = mbar_wait(&p_full[t & 1], (uint32_t)(t >> 1) & 1u);
        if (!ok) break;
        tc_fence_after();
        const uint32_t vb = sb + OFF_KV + (t % NKV) * KV_STAGE + 2 * SUB;
        const uint32_t pb = sb + OFF_P + (t & 1) * P_BUF;
        const uint32_t d = tmem + (uint32_t)COL_O;
#pragma unroll
        for (int part = 0; part < 2; ++part) {            // P value, then P residual
          const uint64_t da = smem_desc_sw128(pb + part * QSUB);
#pragma unroll
          for (int k = 0; k < 4; ++k) {                    // 16 keys per MMA
            const uint64_t db = smem_desc_mn_sw128(vb + k * 2048, SUB, 1024);
            umma_bf16(d, da + (uint64_t)(2 * k), db, idesc_o, (t | part | k) ? 1u : 0u);   // O accumulates over the tiles
          }
        }
        umma_commit(&kv_empty[t % NKV]);
        umma_commit(&pv_done[t & 1]);
      }
      if (!ok) atomicExch(&s_error, 1);
    }
  } else if (row_warp) {
    // ------------------------------------------------------------------ softmax rows
    // O accumulates in tensor memory over all tiles of the chunk.  A row's exponentials are taken
    // relative to a reference maximum m_run that is raised only when a tile's maximum exceeds it
    // by more than RESCALE_STEP (then the row's O and l are multiplied by 2^(old - new) in place);
    // in between the probabilities may exceed 1 (by at most 2^RESCALE_STEP), which costs nothing in
    // fp32 / bf16-pair arithmetic, and the rows never wait for P V except to reuse a P buffer.
    const int slot = P.plan.slot[r_glob];
    const bool ok_row = row_in && slot >= 0;
    const uint64_t mk0 = ok_row ? P.plan.mask[(size_t)r_glob * 2] : 0ull;
    const uint64_t mk1 = ok_row ? P.plan.mask[(size_t)r_glob * 2 + 1] : 0ull;
    const float sc = 0.08838834764831845f * 1.4426950408889634f;    // 1/sqrt(128) * log2(e)
    const uint32_t lane_sel = (uint32_t)(warp * 32) << 16;          // this warp's 32 TMEM lanes
    const uint32_t prow = (uint32_t)(row * 128);
    const uint32_t psw = (uint32_t)(row & 7);
    const uint32_t o_base = tmem + lane_sel + (uint32_t)(COL_O + ND * half);
    bool ok = true;

    for (int t = 0; t < T; ++t) {
      ok = __all_sync(0xffffffffu, mbar_wait(&s_full[t & 1], (uint32_t)(t >> 1) & 1u));   // warp-uniform
      if (!ok) break;
      tc_fence_after();
      uint32_t v[NC];
      const uint32_t base = tmem + lane_sel + (uint32_t)(COL_S + (t & 1) * TK + NC * half);
#pragma unroll
      for (int c0 = 0; c0 < NC; c0 += 16) tmem_ld16(base + (uint32_t)c0, v + c0);
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      const int key0 = (tile_lo + t) * TK;
      if (kv_len - key0 < TK) {
        // The last tile reaches past kv_len: those cache slots were never written and may hold
        // anything, NaN bit patterns included, and 0 x NaN in P V would poison every row.  Zero
        // the value rows from kv_len on (a row is 128 bytes of each 64-dim block; the swizzle
        // only permutes inside the row).  The tile has landed: S, which this warp waited for, was
        // issued after it.  Every row warp in use writes the same zeros.
        const uint32_t vb = sb + OFF_KV + (t % NKV) * KV_STAGE + 2 * SUB;
        for (int kr = kv_len - key0 + lane; kr < TK; kr += 32) {
#pragma unroll
          for (int blk = 0; blk < 2; ++blk)
#pragma unroll
            for (int q = 0; q < 8; ++q) st_shared_v4(vb + blk * SUB + kr * 128 + q * 16, 0u, 0u, 0u, 0u);
        }
      }
      uint64_t vis = ok_row ? tile_visibility(mk0, mk1, key0, ctx, kv_len) : 0ull;
      if (DUP) vis >>= 32 * half;
      float m_t = -INFINITY;
#pragma unroll
      for (int j = 0; j < NC; ++j) {
        const float s = ((vis >> j) & 1ull) ? __uint_as_float(v[j]) * sc : -INFINITY;
        v[j] = __float_as_uint(s);
        m_t = fmaxf(m_t, s);
      }
      if (DUP) {
        // the row's maximum over the whole tile: exchange with the thread that holds the other 32 keys
        // (both threads of a row then keep the same reference maximum)
        xch[t & 1][threadIdx.x] = m_t;
        __syncwarp();
        if (lane == 0) mbar_arrive(&x_bar[rq]);
        ok = __all_sync(0xffffffffu, mbar_wait(&x_bar[rq], (uint32_t)t & 1u));
        if (!ok) break;
        m_t = fmaxf(m_t, xch[t & 1][threadIdx.x ^ 64]);
      }
      // raise the reference maximum?  (the first visible key sets it; O holds nothing of this row yet then)
      float factor = 1.f;
      if (m_t > m_run + RESCALE_STEP || (m_run == -INFINITY && m_t > -INFINITY)) {
        factor = m_run == -INFINITY ? 0.f : exp2f(m_run - m_t);
        m_run = m_t;
      }
      const bool rescale = t > 0 && __any_sync(0xffffffffu, factor != 1.f);
      if (rescale) {
        // every P V issued so far must have landed before O is touched; none can be issued before
        // this warp has handed in its P of tile t
        ok = __all_sync(0xffffffffu, mbar_wait(&pv_done[(t - 1) & 1], (uint32_t)((t - 1) >> 1) & 1u));
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int c0 = 0; c0 < ND; c0 += 16) {
          uint32_t o[16];
          tmem_ld16(o_base + (uint32_t)c0, o);
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
          for (int j = 0; j < 16; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * factor);
          tmem_st16(o_base + (uint32_t)c0, o);
        }
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        l_run *= factor;
      } else if (t == 0) {
        l_run = 0.f;
      }
      // the P buffer of tile t was last read by the P V of tile t - 2
      if (t >= 2) {
        ok = __all_sync(0xffffffffu, mbar_wait(&pv_done[t & 1], (uint32_t)((t - 2) >> 1) & 1u));
        if (!ok) break;
      }
      const float mu = m_run == -INFINITY ? 0.f : m_run;
      float l_t = 0.f;
      const uint32_t pb = sb + OFF_P + (uint32_t)((t & 1) * P_BUF) + prow;
#pragma unroll
      for (int ch = 0; ch < NC / 8; ++ch) {
        uint32_t hi[4], lo[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float p0 = ex2_fast(__uint_as_float(v[ch * 8 + 2 * e]) - mu);
          const float p1 = ex2_fast(__uint_as_float(v[ch * 8 + 2 * e + 1]) - mu);
          l_t += p0 + p1;
          split_pack_trunc(p0, p1, hi[e], lo[e]);
        }
        const uint32_t off = (((uint32_t)(ch + (NC / 8) * half)) ^ psw) << 4;
        st_shared_v4(pb + off, hi[0], hi[1], hi[2], hi[3]);
        st_shared_v4(pb + QSUB + off, lo[0], lo[1], lo[2], lo[3]);
        if (DUP) {                       // the copy of this row in the upper half of the MMA's rows
          st_shared_v4(pb + 64 * 128 + off, hi[0], hi[1], hi[2], hi[3]);
          st_shared_v4(pb + QSUB + 64 * 128 + off, lo[0], lo[1], lo[2], lo[3]);
        }
      }
      l_run += l_t;
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&p_full[t & 1]);
    }
    // the chunk's unnormalised O (relative to m_run) out of tensor memory
#pragma unroll
    for (int d = 0; d < ND; ++d) acc[d] = 0.f;
    if (ok && T > 0) {
      ok = __all_sync(0xffffffffu, mbar_wait(&pv_done[(T - 1) & 1], (uint32_t)((T - 1) >> 1) & 1u));
      if (ok) {
        tc_fence_after();
#pragma unroll
        for (int c0 = 0; c0 < ND; c0 += 32) {
          uint32_t o[32];
          tmem_ld16(o_base + (uint32_t)c0, o);
          tmem_ld16(o_base + (uint32_t)(c0 + 16), o + 16);
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
          for (int j = 0; j < 32; ++j) acc[c0 + j] = __uint_as_float(o[j]);
        }
      }
    }
    if (!ok) atomicExch(&s_error, 1);
  }

  tc_fence_before();
  __syncthreads();                       // all tiles consumed
  const bool failed = s_error != 0;
  // ---- merge over the chunks.  Every CTA receives, from every chunk j (itself included), the
  // dims [c * wc, (c + 1) * wc) of all rows plus (m, l): recv[j][row][wc + 4].
  const int wc = DH / P.chunks;
  const int rs = wc + 4;                 // floats per received row: wc dims, m, l (first keys), l (other keys), pad
  constexpr int RR = DUP ? 64 : 128;     // rows per source chunk in the receive buffer
  float *recv = reinterpret_cast<float *>(sm + OFF_KV);
  if (P.chunks > 1) cluster_sync_all();  // the receive buffer reuses the K/V ring: every CTA of the cluster is done with its tiles
  if (row_in) {
    const uint32_t mine = smem_u32(recv + ((size_t)c * RR + row) * rs);
#pragma unroll
    for (int d = 0; d < ND; d += 4) {
      const int gd = ND * half + d;
      const int j = gd / wc;
      const uint32_t a = mine + (uint32_t)(gd - j * wc) * 4;
      st_cluster_v4(P.chunks > 1 ? peer_addr(a, (uint32_t)j) : a, acc[d], acc[d + 1], acc[d + 2], acc[d + 3]);
    }
    for (int j = 0; j < P.chunks; ++j) {
      const uint32_t a = mine + (uint32_t)wc * 4;
      const uint32_t ra = P.chunks > 1 ? peer_addr(a, (uint32_t)j) : a;
      if (half == 0) asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(ra), "f"(m_run), "f"(l_run) : "memory");
      else asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(ra + 8), "f"(l_run) : "memory");
      if (!DUP) asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(ra + 8), "f"(0.f) : "memory");
    }
  }
  if (P.chunks > 1) cluster_sync_all(); else __syncthreads();
  if (row_in && !failed) {
    const int ncol = DUP ? wc / 2 : wc;                    // this thread's share of the CTA's dims
    const int col0 = DUP ? half * ncol : 0;
    float mm = -INFINITY;
    for (int j = 0; j < P.chunks; ++j) mm = fmaxf(mm, recv[((size_t)j * RR + row) * rs + wc]);
    float o[ND];
#pragma unroll
    for (int d = 0; d < ND; ++d) o[d] = 0.f;
    float l = 0.f;
    if (mm != -INFINITY) {
      for (int j = 0; j < P.chunks; ++j) {
        const float *src = recv + ((size_t)j * RR + row) * rs;
        const float4 ml = *reinterpret_cast<const float4 *>(src + wc);
        if (ml.x == -INFINITY) continue;
        const float w = exp2f(ml.x - mm);
        l += w * (ml.y + ml.z);
#pragma unroll
        for (int d = 0; d < ND; d += 4) {
          if (d < ncol) {
            const float4 x = *reinterpret_cast<const float4 *>(src + col0 + d);
            o[d] += w * x.x; o[d + 1] += w * x.y; o[d + 2] += w * x.z; o[d + 3] += w * x.w;
          }
        }
      }
    }
    const float inv = l > 0.f ? 1.f / l : 0.f;
    const size_t ob = (size_t)r_glob * H + h * DH + c * wc + col0;
#pragma unroll
    for (int d = 0; d < ND; d += 8) {
      if (d < ncol) {
        uint32_t hi[4], lo[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) split_pack(o[d + 2 * e] * inv, o[d + 2 * e + 1] * inv, hi[e], lo[e]);
        *reinterpret_cast<uint4 *>(P.out + ob + d) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
        if (P.out_lo != nullptr) *reinterpret_cast<uint4 *>(P.out_lo + ob + d) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
      }
    }
  }
  if (warp == 5) {
    if (failed) {      // MMAs issued before a wait ran out may still be running: no free under them
      if (lane == 0) {
        umma_commit(&drain_bar);
        (void)mbar_wait(&drain_bar, 0);
      }
      __syncwarp();
    }
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)TMEM_COLS) : "memory");
  }
  if (threadIdx.x == 0 && failed && P.status) atomicMax(P.status, E_TIMEOUT);
}

int g_attn_tc_min_rows = 16;   // fewer query rows per sequence than this: the mma.sync kernel
int g_attn_tc_chunks = 0;      // > 0: this many key chunks whatever the shape (A/B runs)

}  // namespace

void attn_tc_set_min_rows(int rows) { g_attn_tc_min_rows = rows; }
void attn_tc_set_chunks(int chunks) { g_attn_tc_chunks = chunks; }

// Key chunks (= cluster size) per (sequence, head): the largest of 1, 2, 4, 8 that keeps the CTA
// count within the SMs (one CTA per SM is resident; measured: a second, partly filled round and the
// co-scheduling of clusters cost more than shorter CTAs gain), each chunk with at least 128 keys of
// capacity.
int attn_tc_chunks(int B, int n_heads, int S_max, int num_sms) {
  int c = 1;
  if (g_attn_tc_chunks > 0) {
    while (2 * c <= g_attn_tc_chunks && 2 * c <= 8 && 2 * c * 128 <= S_max) c *= 2;
    return c;
  }
  while (c < 8 && 2 * c * B * n_heads <= num_sms && 2 * c * 128 <= S_max) c *= 2;
  return c;
}

bool attn_tc_supported(int rows_per_seq, int head_dim, int S_max) {
  return head_dim == DH && rows_per_seq >= g_attn_tc_min_rows && rows_per_seq <= 128 &&
         tc_smem_optin() >= SMEM_BYTES + 1024 + 1280 && S_max >= 1;
}

cudaError_t tree_attention_tc(Launch L, Operand q_pair, int q_rows_alloc, const void *k_cache, const void *v_cache,
                              RowPlan plan, Operand out, int rows_per_seq, int B, int n_heads, int S_max, int chunks,
                              int *status) {
  static SmemOptIn optin_dup, optin_full;
  const size_t smem = (size_t)SMEM_BYTES + 1024;
  cudaError_t e = optin_dup.ensure((const void *)tree_attn_tc_kernel<true>, smem);
  if (e == cudaSuccess) e = optin_full.ensure((const void *)tree_attn_tc_kernel<false>, smem);
  if (e != cudaSuccess) return e;
  if (chunks != 1 && chunks != 2 && chunks != 4 && chunks != 8) return cudaErrorInvalidValue;
  if (q_pair.hi == nullptr || q_pair.lo == nullptr) return cudaErrorInvalidValue;
  const long long rows = (long long)B * n_heads * S_max;
  if (rows > 0x7fffffffLL) return cudaErrorInvalidValue;
  const int H = n_heads * DH;
  CUtensorMap tmQh, tmQl, tmK, tmV;
  if (!tc_get_map(q_pair.hi, q_rows_alloc, H, 64, &tmQh) || !tc_get_map(q_pair.lo, q_rows_alloc, H, 64, &tmQl) ||
      !tc_get_map(k_cache, (int)rows, DH, TK, &tmK) || !tc_get_map(v_cache, (int)rows, DH, TK, &tmV))
    return cudaErrorInvalidValue;
  const int longest_first = (B > 1 && B <= 32 && (long long)chunks * B * n_heads > tc_num_sms()) ? 1 : 0;
  AttnParams P{plan, (bf16 *)out.hi, (bf16 *)out.lo, rows_per_seq, n_heads, S_max, chunks, longest_first, status};
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(chunks, n_heads * B);
  cfg.blockDim = dim3(THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = L.st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = L.pdl ? 1 : 0;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = chunks;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = chunks > 1 ? 2 : 1;
  ++g_launches;
  if (rows_per_seq <= 64) return cudaLaunchKernelEx(&cfg, tree_attn_tc_kernel<true>, tmQh, tmQl, tmK, tmV, P);
  return cudaLaunchKernelEx(&cfg, tree_attn_tc_kernel<false>, tmQh, tmQl, tmK, tmV, P);
}

}  // namespace koala
