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
constexpr int NKV = 3;                       // K/V stages (four with at most 64 rows, where Q takes half the room)
constexpr int NKV_MAX = 4;
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
  int l2_ahead;            // K/V tiles requested into L2 this many tiles ahead of the ring (0 = none)
  int dry_pass;            // 1: the row warps make a dry pass over the tile loop body before the dependency wait
  int *status;
};

// DUP (at most 64 query rows): the MMA's 128 rows hold both parts of the operand pair (of Q for S,
// of P for P V), so that one pass of MMAs gives both partial products, to be added: warp w owns
// queries 16w .. 16w+15, whose value parts are MMA rows (= tensor-memory lanes) 32w .. 32w+15 and
// whose residual parts are rows 32w+16 .. 32w+31.  Lanes l and l+16 of a warp therefore hold the
// two partial scores S_v, S_r of one query: they swap halves by shuffles (no shared memory, no
// barrier), after which lane l has S = S_v + S_r for keys 0..31 of the tile and lane l+16 for keys
// 32..63; the row maximum is one more shuffle; at the end they swap halves of O_v, O_r the same
// way and write dims 0..63 and 64..127.  Otherwise warp w owns rows 32w .. 32w+31 entirely and
// the pair is two accumulating MMAs.
template <bool DUP>
__global__ void __launch_bounds__(THREADS, 1)
tree_attn_tc_kernel(const __grid_constant__ CUtensorMap tmQh, const __grid_constant__ CUtensorMap tmQl,
                    const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                    const AttnParams P) {
  constexpr int NC = DUP ? 32 : 64;      // keys of a tile per thread
  constexpr int PB = DUP ? QSUB : P_BUF; // bytes of one P buffer
  constexpr int NST = DUP ? NKV + 1 : NKV;             // K/V stages
  constexpr int OKV = DUP ? OFF_KV - KV_STAGE : OFF_KV; // the ring starts where the second half of Q would be
  extern __shared__ unsigned char smem_raw[];
  __shared__ uint64_t q_full, kv_full[NKV_MAX], kv_empty[NKV_MAX], s_full[2], p_full[2], pv_done[2], drain_bar;
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
  const int n_q = DUP ? (P.rows_per_seq + 15) >> 4 : (P.rows_per_seq + 31) >> 5;   // row warps in use (16 or 32 queries each)
  const int n_arrive = n_q;

  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    mbar_init(&q_full, 1);
    for (int s = 0; s < NST; ++s) { mbar_init(&kv_full[s], 1); mbar_init(&kv_empty[s], 1); }
    mbar_init(&drain_bar, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&s_full[i], 1);
      mbar_init(&p_full[i], (uint32_t)n_arrive);
      mbar_init(&pv_done[i], 1);
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

  // Q, the tree rows of K/V and the row plan come from earlier kernels: everything that reads them
  // comes after the dependency wait in read_plan().  The row warps call it inside their tile loop,
  // after a dry pass over the loop body (see there); the other threads here.
  int ctx = 0, kv_len = 0, tile_lo = 0, T = 0;
  auto read_plan = [&]() {
    pdl_wait();
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
    ctx = P.plan.ctx_len[b];
    kv_len = P.plan.kv_len[b];
    kv_len = kv_len > P.S_max ? P.S_max : kv_len;
    const int n_tiles = (kv_len + TK - 1) / TK;
    tile_lo = (int)(((long long)n_tiles * c) / P.chunks);
    const int tile_hi = (int)(((long long)n_tiles * (c + 1)) / P.chunks);
    T = tile_hi - tile_lo;
  };
  // row ownership of warps 0..3
  const int half = DUP ? (lane >> 4) : 0;                   // DUP: residual lane; takes the second half of the keys / dims
  const int row = DUP ? warp * 16 + (lane & 15) : warp * 32 + lane;
  const bool row_warp = warp < 4 && warp < n_q;
  const bool row_in = row_warp && row < P.rows_per_seq;
  if (!row_warp) read_plan();
  if (threadIdx.x == 128) {        // warp 4 lane 0: the queries do not depend on the plan
    if (DUP) {
      // of every 32 MMA rows the first 16 are the values of 16 queries, the other 16 their residuals
      mbar_expect_tx(&q_full, (uint32_t)(2 * QSUB));
#pragma unroll
      for (int hb = 0; hb < 2; ++hb)
#pragma unroll
        for (int g = 0; g < 4; ++g)
#pragma unroll
          for (int part = 0; part < 2; ++part)
            tma_load_2d(part ? &tmQl : &tmQh, &q_full, sm + OFF_Q + hb * QSUB + (32 * g + 16 * part) * 128,
                        h * DH + 64 * hb, b * P.rows_per_seq + 16 * g);
    } else {
      mbar_expect_tx(&q_full, (uint32_t)(4 * QSUB));
#pragma unroll
      for (int part = 0; part < 2; ++part)
#pragma unroll
        for (int hb = 0; hb < 2; ++hb)
#pragma unroll
          for (int rh = 0; rh < 2; ++rh)
            tma_load_2d(part ? &tmQl : &tmQh, &q_full, sm + OFF_Q + (part * 2 + hb) * QSUB + rh * (QSUB / 2),
                        h * DH + 64 * hb, b * P.rows_per_seq + 64 * rh);
    }
  }
  int r_glob = 0;
  float m_run = -INFINITY, l_run = 0.f;
  bool have_o = false;             // this warp's O in tensor memory is complete (warp-uniform)

  if (warp == 4) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      const int y0 = (b * P.n_heads + h) * P.S_max;
      bool ok = true;
      int issued = 0;
      auto request_l2 = [&](int t) {
        const int y = y0 + (tile_lo + t) * TK;
#pragma unroll
        for (int q = 0; q < 4; ++q)
          asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];"
                       ::"l"(q < 2 ? &tmK : &tmV), "r"(64 * (q & 1)), "r"(y) : "memory");
      };
      // the cache is streamed from HBM by one CTA with a few tiles in flight: tiles beyond the ring
      // are requested into L2 so that the ring's own loads find them there
      for (int t = NST; t < NST + P.l2_ahead && t < T; ++t) request_l2(t);
      for (int t = 0; t < T; ++t) {
        const int s = t % NST;
        if (P.l2_ahead > 0 && t + NST + P.l2_ahead < T) request_l2(t + NST + P.l2_ahead);
        if (t >= NST) {
          ok = mbar_wait(&kv_empty[s], (uint32_t)((t / NST) - 1) & 1u);
          if (!ok) break;
        }
        mbar_expect_tx(&kv_full[s], (uint32_t)KV_STAGE);
        unsigned char *dst = sm + OKV + s * KV_STAGE;
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
        for (int t = issued > NST ? issued - NST : 0; t < issued; ++t)
          (void)mbar_wait(&kv_full[t % NST], (uint32_t)(t / NST) & 1u);
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
        const int s = t % NST;
        if (!mbar_wait(&kv_full[s], (uint32_t)(t / NST) & 1u)) return false;
        tc_fence_after();
        const uint32_t kb = sb + OKV + s * KV_STAGE;
        const uint32_t d = tmem + (uint32_t)(COL_S + (t & 1) * TK);
#pragma unroll
        for (int part = 0; part < (DUP ? 1 : 2); ++part) { // Q value, then Q residual (DUP: both in one operand)
#pragma unroll
          for (int hb = 0; hb < 2; ++hb) {                 // 64-dim block
            const uint64_t da = smem_desc_sw128(sb + OFF_Q + (DUP ? hb : part * 2 + hb) * QSUB);
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
        const uint32_t vb = sb + OKV + (t % NST) * KV_STAGE + 2 * SUB;
        const uint32_t pb = sb + OFF_P + (t & 1) * PB;
        const uint32_t d = tmem + (uint32_t)COL_O;
#pragma unroll
        for (int part = 0; part < (DUP ? 1 : 2); ++part) { // P value, then P residual (DUP: both in one operand)
          const uint64_t da = smem_desc_sw128(pb + part * QSUB);
#pragma unroll
          for (int k = 0; k < 4; ++k) {                    // 16 keys per MMA
            const uint64_t db = smem_desc_mn_sw128(vb + k * 2048, SUB, 1024);
            umma_bf16(d, da + (uint64_t)(2 * k), db, idesc_o, (t | part | k) ? 1u : 0u);   // O accumulates over the tiles
          }
        }
        umma_commit(&kv_empty[t % NST]);
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
    bool ok_row = false;
    uint64_t mk0 = 0ull, mk1 = 0ull;
    const float sc = 0.08838834764831845f * 1.4426950408889634f;    // 1/sqrt(128) * log2(e)
    const uint32_t lane_sel = (uint32_t)(warp * 32) << 16;          // this warp's 32 TMEM lanes
    const uint32_t prow = (uint32_t)((DUP ? warp * 32 + (lane & 15) : row) * 128);   // this query's (value) row of the P operand
    const uint32_t psw = (uint32_t)(row & 7);
    const uint32_t o_base = tmem + lane_sel + (uint32_t)COL_O;     // all 128 dims of this thread's lane
    bool ok = true;

    // Pass t = -1 is a dry pass over the loop body, made before the dependency wait while the kernel
    // before this one still runs: no waits, no row visible (every probability is 0), nothing handed
    // to the MMA warp.  The body is some 20 KB of instructions that run a few times per launch; the
    // dry pass takes their first, slow fetch off the path between the arrival of S and the first P.
    int T_run = 1;
    for (int t = P.dry_pass ? -1 : 0; t < T_run; ++t) {
      if (t == 0) {
        read_plan();
        T_run = T;
        r_glob = b * P.rows_per_seq + (row_in ? row : 0);    // also needed by a chunk without tiles: it still merges and stores its dims
        if (T == 0) break;
        ok_row = row_in && P.plan.slot[r_glob] >= 0;
        mk0 = ok_row ? P.plan.mask[(size_t)r_glob * 2] : 0ull;
        mk1 = ok_row ? P.plan.mask[(size_t)r_glob * 2 + 1] : 0ull;
      }
      const bool live = t >= 0;
      if (live) {
        ok = __all_sync(0xffffffffu, mbar_wait(&s_full[t & 1], (uint32_t)(t >> 1) & 1u));   // warp-uniform
        if (!ok) break;
      }
      tc_fence_after();
      uint32_t v[NC];
      const uint32_t base = tmem + lane_sel + (uint32_t)(COL_S + (t & 1) * TK);
      if constexpr (DUP) {
        // this lane holds one part (value or residual) of the query's 64 raw scores: keep the part of
        // this lane's 32 keys, hand the other 32 to the query's second lane, add what it hands back
        uint32_t raw[TK];
#pragma unroll
        for (int c0 = 0; c0 < TK; c0 += 16) tmem_ld16(base + (uint32_t)c0, raw + c0);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float got = __shfl_xor_sync(0xffffffffu, __uint_as_float(half ? raw[j] : raw[32 + j]), 16);
          v[j] = __float_as_uint(__uint_as_float(half ? raw[32 + j] : raw[j]) + got);
        }
      } else {
#pragma unroll
        for (int c0 = 0; c0 < NC; c0 += 16) tmem_ld16(base + (uint32_t)c0, v + c0);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      }
      const int key0 = (tile_lo + t) * TK;
      if (kv_len - key0 < TK) {
        // The last tile reaches past kv_len: those cache slots were never written and may hold
        // anything, NaN bit patterns included, and 0 x NaN in P V would poison every row.  Zero
        // the value rows from kv_len on (a row is 128 bytes of each 64-dim block; the swizzle
        // only permutes inside the row).  The tile has landed: S, which this warp waited for, was
        // issued after it.  Every row warp in use writes the same zeros.
        const uint32_t vb = sb + OKV + (t % NST) * KV_STAGE + 2 * SUB;
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
      if (DUP) m_t = fmaxf(m_t, __shfl_xor_sync(0xffffffffu, m_t, 16));   // over all 64 keys: both lanes keep the same reference
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
#pragma unroll 1
        for (int c0 = 0; c0 < DH; c0 += 16) {          // rare: kept short
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
      const uint32_t pb = sb + OFF_P + (uint32_t)((t & 1) * PB) + prow;
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
        // the residuals: 16 rows further down in the same operand (DUP) or the second operand
        st_shared_v4(pb + (DUP ? 16 * 128 : QSUB) + off, lo[0], lo[1], lo[2], lo[3]);
      }
      l_run += l_t;
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      tc_fence_before();
      __syncwarp();
      if (live && lane == 0) mbar_arrive(&p_full[t & 1]);
    }
    // every P V of the chunk has landed in tensor memory before O is read below
    if (ok && T > 0) ok = __all_sync(0xffffffffu, mbar_wait(&pv_done[(T - 1) & 1], (uint32_t)((T - 1) >> 1) & 1u));
    have_o = ok && T > 0;
    if (!ok) atomicExch(&s_error, 1);
  }

  tc_fence_before();
  __syncthreads();                       // all tiles consumed
  const bool failed = s_error != 0;
  // ---- merge over the chunks.  Every CTA receives, from every chunk j (itself included), the
  // dims [c * wc, (c + 1) * wc) of all rows plus (m, l): recv[j][row][wc + 4].  The code from here
  // on runs once per CTA, so it is written as short loops rather than unrolled over the 128 dims.
  const int wc = DH / P.chunks;
  const int rs = wc + 4;                 // floats per received row: wc dims, m, l (first keys), l (other keys), pad
  constexpr int RR = DUP ? 64 : 128;     // rows per source chunk in the receive buffer
  float *recv = reinterpret_cast<float *>(sm + OKV);
  if (P.chunks > 1) cluster_sync_all();  // the receive buffer reuses the K/V ring: every CTA of the cluster is done with its tiles
  if (row_warp && P.chunks == 1) {
    // one chunk: nothing to merge - O out of tensor memory 16 dims at a time, normalised and stored
    tc_fence_after();
    const uint32_t o_lane = tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)COL_O;   // this thread's lane, dim 0
    float l = l_run;
    if (DUP) l += __shfl_xor_sync(0xffffffffu, l_run, 16);      // the query's other 32 keys of every tile
    const float inv = (m_run != -INFINITY && l > 0.f) ? 1.f / l : 0.f;
    const size_t ob = (size_t)r_glob * H + h * DH;
#pragma unroll 1
    for (int c0 = 0; c0 < DH; c0 += 16) {
      uint32_t o[16];
      if (have_o) {
        tmem_ld16(o_lane + (uint32_t)c0, o);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) o[j] = 0u;
      }
      if constexpr (DUP) {
        // the query's two lanes hold the two parts of the pair's product: add them; each lane stores eight dims
        float x[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const float lo8 = __uint_as_float(o[k]) + __shfl_xor_sync(0xffffffffu, __uint_as_float(o[k]), 16);
          const float hi8 = __uint_as_float(o[8 + k]) + __shfl_xor_sync(0xffffffffu, __uint_as_float(o[8 + k]), 16);
          x[k] = (half ? hi8 : lo8) * inv;
        }
        if (row_in && !failed) {
          uint32_t hi[4], lo[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) split_pack(x[2 * e], x[2 * e + 1], hi[e], lo[e]);
          const size_t at = ob + c0 + 8 * half;
          *reinterpret_cast<uint4 *>(P.out + at) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
          if (P.out_lo != nullptr) *reinterpret_cast<uint4 *>(P.out_lo + at) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        }
      } else if (row_in && !failed) {
#pragma unroll
        for (int g8 = 0; g8 < 2; ++g8) {
          uint32_t hi[4], lo[4];
#pragma unroll
          for (int e = 0; e < 4; ++e)
            split_pack(__uint_as_float(o[8 * g8 + 2 * e]) * inv, __uint_as_float(o[8 * g8 + 2 * e + 1]) * inv, hi[e], lo[e]);
          const size_t at = ob + c0 + 8 * g8;
          *reinterpret_cast<uint4 *>(P.out + at) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
          if (P.out_lo != nullptr) *reinterpret_cast<uint4 *>(P.out_lo + at) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        }
      }
    }
  } else if (row_warp) {
    // the chunk's unnormalised O (relative to m_run) out of tensor memory, 16 dims at a time, each
    // group to the CTA that merges those dims
    tc_fence_after();
    const uint32_t o_lane = tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)COL_O;   // this thread's lane, dim 0
    const uint32_t mine = smem_u32(recv + ((size_t)c * RR + row) * rs);
#pragma unroll 1
    for (int c0 = 0; c0 < DH; c0 += 16) {
      uint32_t o[16];
      if (have_o) {
        tmem_ld16(o_lane + (uint32_t)c0, o);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) o[j] = 0u;
      }
      const int j = c0 / wc;
      const uint32_t a = mine + (uint32_t)(c0 - j * wc) * 4;
      const uint32_t ra = P.chunks > 1 ? peer_addr(a, (uint32_t)j) : a;
      if constexpr (DUP) {
        // the query's two lanes hold the two parts of the pair's product: add them (both lanes get
        // the sum) and let each lane store eight of the sixteen dims
        float x[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const float lo8 = __uint_as_float(o[k]) + __shfl_xor_sync(0xffffffffu, __uint_as_float(o[k]), 16);
          const float hi8 = __uint_as_float(o[8 + k]) + __shfl_xor_sync(0xffffffffu, __uint_as_float(o[8 + k]), 16);
          x[k] = half ? hi8 : lo8;
        }
        if (row_in) {
          st_cluster_v4(ra + (uint32_t)half * 32u, x[0], x[1], x[2], x[3]);
          st_cluster_v4(ra + (uint32_t)half * 32u + 16u, x[4], x[5], x[6], x[7]);
        }
      } else if (row_in) {
#pragma unroll
        for (int k = 0; k < 16; k += 4)
          st_cluster_v4(ra + (uint32_t)k * 4u, __uint_as_float(o[k]), __uint_as_float(o[k + 1]),
                        __uint_as_float(o[k + 2]), __uint_as_float(o[k + 3]));
      }
    }
    if (row_in) {
#pragma unroll 1
      for (int j = 0; j < P.chunks; ++j) {
        const uint32_t a = mine + (uint32_t)wc * 4;
        const uint32_t ra = P.chunks > 1 ? peer_addr(a, (uint32_t)j) : a;
        if (half == 0) asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(ra), "f"(m_run), "f"(l_run) : "memory");
        else asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(ra + 8), "f"(l_run) : "memory");
        if (!DUP) asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(ra + 8), "f"(0.f) : "memory");
      }
    }
  }
  if (P.chunks > 1) cluster_sync_all(); else __syncthreads();
  if (row_in && !failed && P.chunks > 1) {
    const int ncol = DUP ? wc / 2 : wc;                    // this thread's share of the CTA's dims
    const int col0 = DUP ? half * ncol : 0;
    float mm = -INFINITY, l = 0.f;
#pragma unroll 1
    for (int j = 0; j < P.chunks; ++j) mm = fmaxf(mm, recv[((size_t)j * RR + row) * rs + wc]);
    if (mm != -INFINITY) {
#pragma unroll 1
      for (int j = 0; j < P.chunks; ++j) {
        const float4 ml = *reinterpret_cast<const float4 *>(recv + ((size_t)j * RR + row) * rs + wc);
        if (ml.x != -INFINITY) l += exp2f(ml.x - mm) * (ml.y + ml.z);
      }
    }
    const float inv = l > 0.f ? 1.f / l : 0.f;
    const size_t ob = (size_t)r_glob * H + h * DH + c * wc + col0;
#pragma unroll 1
    for (int d0 = 0; d0 < ncol; d0 += 8) {
      float o[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      if (mm != -INFINITY) {
#pragma unroll 1
        for (int j = 0; j < P.chunks; ++j) {               // in chunk order
          const float *src = recv + ((size_t)j * RR + row) * rs;
          const float mj = src[wc];
          if (mj == -INFINITY) continue;
          const float w = exp2f(mj - mm);
          const float4 x0 = *reinterpret_cast<const float4 *>(src + col0 + d0);
          const float4 x1 = *reinterpret_cast<const float4 *>(src + col0 + d0 + 4);
          o[0] += w * x0.x; o[1] += w * x0.y; o[2] += w * x0.z; o[3] += w * x0.w;
          o[4] += w * x1.x; o[5] += w * x1.y; o[6] += w * x1.z; o[7] += w * x1.w;
        }
      }
      uint32_t hi[4], lo[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) split_pack(o[2 * e] * inv, o[2 * e + 1] * inv, hi[e], lo[e]);
      *reinterpret_cast<uint4 *>(P.out + ob + d0) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
      if (P.out_lo != nullptr) *reinterpret_cast<uint4 *>(P.out_lo + ob + d0) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
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
int g_attn_tc_l2_ahead = 0;    // K/V tiles requested into L2 ahead of the ring
int g_attn_tc_dry_pass = 1;

}  // namespace

void attn_tc_set_min_rows(int rows) { g_attn_tc_min_rows = rows; }
void attn_tc_set_chunks(int chunks) { g_attn_tc_chunks = chunks; }
void attn_tc_set_l2_ahead(int tiles) { g_attn_tc_l2_ahead = tiles < 0 ? 0 : tiles; }
void attn_tc_set_dry_pass(int on) { g_attn_tc_dry_pass = on ? 1 : 0; }

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
  const int q_box = rows_per_seq <= 64 ? 16 : 64;      // rows per copy of the query operand
  if (!tc_get_map(q_pair.hi, q_rows_alloc, H, q_box, &tmQh) || !tc_get_map(q_pair.lo, q_rows_alloc, H, q_box, &tmQl) ||
      !tc_get_map(k_cache, (int)rows, DH, TK, &tmK) || !tc_get_map(v_cache, (int)rows, DH, TK, &tmV))
    return cudaErrorInvalidValue;
  const int longest_first = (B > 1 && B <= 32 && (long long)chunks * B * n_heads > tc_num_sms()) ? 1 : 0;
  AttnParams P{plan, (bf16 *)out.hi, (bf16 *)out.lo, rows_per_seq, n_heads, S_max, chunks, longest_first,
               g_attn_tc_l2_ahead, g_attn_tc_dry_pass, status};
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
