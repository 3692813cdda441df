// Weight-streaming skinny GEMM on the 5th-generation tensor cores (sm_100a):
//   Y[R][N_out] (fp32) = X[R][K_in] (bf16) * W[N_out][K_in]^T (bf16)
// with R (tokens = tree nodes x batch) small and the weight matrix read exactly once.
//
// Operands are swapped so that the weights fill the MMA's M dimension: one CTA owns 128 weight
// rows and a range of K, and issues tcgen05.mma with M = 128 (weight rows), N = token tile,
// K = 16, both operands K-major in shared memory with the 128-byte swizzle that TMA writes.
// The fp32 accumulator [128 x tokens] lives in tensor memory.  Warp 0 streams weight and
// activation tiles with TMA through a ring of shared-memory stages (mbarrier full/empty pairs),
// warp 1 issues the MMAs, four to sixteen epilogue warps read the accumulator back (tcgen05.ld,
// one step ahead of the stores) and store it.
// The weight stream does not depend on the previous kernel, so under programmatic dependent
// launch the first stages are requested before waiting for the producer of X.
// Activations may come as a pair hi + lo of bf16 matrices (lo = rounding residual of hi): the
// token tile then holds the hi rows followed by the lo rows of the same tokens (MMA N doubles),
// and the epilogue adds the two halves of the accumulator, so the product carries 16 significant
// bits of the activations at no extra weight traffic.
// More than 128 tokens as a pair: value rows and residual rows are two accumulating MMAs into the same
// accumulator columns, so a tile holds up to 256 tokens and the weights are passed over once.  With
// 256 tokens a CTA takes 256 weight rows: four MMAs per K step share the activation tile and fill two
// accumulators (all 512 tensor-memory columns); a stage is 32 KB of weights + 64 KB of activations,
// two stages, one CTA per SM.  From 113 rows up (as a pair) gemm_tc_pair_kernel takes over where it
// applies: two CTAs of a cluster as one MMA unit, see there.
// Split-K: grid.y CTAs share a weight tile and write separate partial outputs that the consumer
// kernel sums in a fixed order (deterministic).
// Every wait is bounded: on expiry the kernel records KOALA_E_TIMEOUT in *status, drains, frees
// its tensor memory and returns.
#include <cuda.h>

#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <tuple>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace koala {
namespace {

constexpr int BM = 128;             // weight rows per CTA (MMA M)
constexpr int BK = 64;              // K elements per stage: 128 bytes of bf16 = one swizzle row
constexpr int UMMA_K = 16;
constexpr int THREADS_WIDE = 576;   // most threads a launch uses: producer warp, MMA warp and sixteen epilogue
                                    // warps (256-row weight tiles); 128-row tiles launch 320 threads
constexpr int W_STAGE_BYTES = BM * BK * 2;
constexpr int E_TIMEOUT = 6;
constexpr int MAX_STAGES = 12;
constexpr int L2_AHEAD = 0;          // weight tiles (16 KB each) prefetched into L2 beyond the ring (measured: any
                                     // depth slows the small kernels that run meanwhile more than it helps)

struct TcParams {
  float *Y;
  int ldy;
  int R;              // valid tokens
  int bn;             // MMA N = rows of the activation tile in shared memory, multiple of 16, <= 256
  int tt;             // tokens per tile: bn, or bn / 2 when the activations are a hi/lo pair
  int pair;           // 1: hi/lo pair
  int ztiles;         // token tiles (classic mode; fastest-varying part of blockIdx.x)
  int tmem_cols;      // power of two >= max(32, bn), per accumulator buffer
  int nbuf;           // accumulator buffers in tensor memory (2 when they fit in 256 columns)
  int tiles0, tiles1; // weight tiles of matrix 0 and of matrices 0+1 (cumulative)
  int n0, n1, n2;     // rows of each matrix
  int kblocks;        // K_in / 64
  int split;          // classic mode: CTAs along K (grid.y)
  int sk_ctas;        // stream-K mode (> 0): the grid's CTAs share all (tile, K-block) units evenly
  unsigned sk_units;  // tiles * kblocks
  size_t split_stride;
  int stages;
  int wide;           // 1: 256 weight rows per CTA (two accumulators), N = 256, one CTA per SM
  int accp;           // 1: the pair's residual rows are a second, accumulating MMA into the same columns
                      //    (bn = tt: up to 256 tokens per tile) instead of extra columns (bn = 2 tt)
  int pf_ahead;       // weight tiles requested into L2 this many units ahead of the ring (0 = none)
  int early_w;        // how many of the first stages' weight tiles are requested before the dependency wait
  int l2_ahead;       // weight tiles prefetched into L2 beyond the ring before the dependency wait
  int epi_dry;        // 1: the epilogue warps make a dry pass over their loop body (nothing stored) at kernel start
  int *status;
};

// CTA that owns unit u when `units` units are dealt to `ctas` CTAs as [g*units/ctas, (g+1)*units/ctas)
__device__ __forceinline__ unsigned sk_owner(unsigned u, unsigned ctas, unsigned units) {
  return ((u + 1u) * ctas - 1u) / units;
}

__global__ void __launch_bounds__(THREADS_WIDE, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmW0, const __grid_constant__ CUtensorMap tmW1,
               const __grid_constant__ CUtensorMap tmW2, const __grid_constant__ CUtensorMap tmX,
               const __grid_constant__ CUtensorMap tmXlo, const TcParams P) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ uint64_t full_bar[MAX_STAGES];
  __shared__ uint64_t empty_bar[MAX_STAGES];
  __shared__ uint64_t acc_full[2];      // accumulator buffer complete (MMA -> epilogue)
  __shared__ uint64_t acc_empty[2];     // accumulator buffer drained (epilogue -> MMA)
  __shared__ uint64_t drain_bar;        // error path: every MMA issued so far has finished
  __shared__ uint32_t tmem_base_slot;
  __shared__ int s_error;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t raw = smem_u32(smem_raw);
  unsigned char *tiles = smem_raw + ((1024u - (raw & 1023u)) & 1023u);
  const int x_stage_bytes = (P.accp ? 2 : 1) * P.bn * BK * 2;
  const int w_stage_bytes = P.wide ? 2 * W_STAGE_BYTES : W_STAGE_BYTES;
  const int stage_bytes = w_stage_bytes + x_stage_bytes;   // both multiples of 1024
  const int bm = P.wide ? 2 * BM : BM;                     // weight rows per tile
  const int KB = P.kblocks;

  // this CTA's run of (tile, K-block) units, tile-major; a run may cross tile boundaries (stream-K)
  unsigned u_lo, u_hi;
  int tok0 = 0;
  if (P.sk_ctas > 0) {
    u_lo = (unsigned)(((unsigned long long)blockIdx.x * P.sk_units) / (unsigned)P.sk_ctas);
    u_hi = (unsigned)(((unsigned long long)(blockIdx.x + 1) * P.sk_units) / (unsigned)P.sk_ctas);
  } else {
    const int tile = blockIdx.x / P.ztiles;
    tok0 = (blockIdx.x % P.ztiles) * P.tt;
    u_lo = (unsigned)(tile * KB + (int)(((long long)KB * blockIdx.y) / P.split));
    u_hi = (unsigned)(tile * KB + (int)(((long long)KB * (blockIdx.y + 1)) / P.split));
  }
  const int n_units = (int)(u_hi - u_lo);

  // weight tensor map and first row of a tile
  auto tile_map = [&](int tile, int &row0) -> const CUtensorMap * {
    if (tile >= P.tiles1) { row0 = (tile - P.tiles1) * bm; return &tmW2; }
    if (tile >= P.tiles0) { row0 = (tile - P.tiles0) * bm; return &tmW1; }
    row0 = tile * bm;
    return &tmW0;
  };
  // one weight tile of a stage: 128 rows per copy
  auto load_w = [&](const CUtensorMap *tmW, uint64_t *bar, unsigned char *dst, int kb, int row0) {
    tma_load_2d(tmW, bar, dst, kb * BK, row0);
    if (P.wide) tma_load_2d(tmW, bar, dst + W_STAGE_BYTES, kb * BK, row0 + BM);
  };
  const int pre = n_units < P.stages ? n_units : P.stages;

  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    for (int s = 0; s < P.stages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&acc_full[i], 1);
      mbar_init(&acc_empty[i], (blockDim.x >> 5) - 2);   // one arrival per epilogue warp
    }
    mbar_init(&drain_bar, 1);
    s_error = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    // The weight stream starts right here, before the block-wide set-up barrier and before the
    // dependency wait: weights do not depend on the kernel before this one.  A few more of this
    // CTA's weight tiles are requested into L2 (bounded, so that all CTAs together stay well
    // inside the L2).
    int tile = (int)(u_lo / KB), kb = (int)(u_lo % KB), row0;
    const CUtensorMap *tmW = tile_map(tile, row0);
    const int early = pre < P.early_w ? pre : P.early_w;
    const int ahead = early == pre ? (n_units < pre + P.l2_ahead ? n_units : pre + P.l2_ahead) : early;
    for (int it = 0; it < ahead; ++it) {
      if (it < early) {
        mbar_expect_tx(&full_bar[it], (uint32_t)stage_bytes);
        load_w(tmW, &full_bar[it], tiles + (size_t)it * stage_bytes, kb, row0);
      } else {
        asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];"
                     ::"l"(tmW), "r"(kb * BK), "r"(row0) : "memory");
        if (P.wide)
          asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];"
                       ::"l"(tmW), "r"(kb * BK), "r"(row0 + BM) : "memory");
      }
      if (++kb == KB) { kb = 0; ++tile; tmW = tile_map(tile, row0); }
    }
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmX) : "memory");
    if (P.pair) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmXlo) : "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&tmem_base_slot)), "r"((uint32_t)(P.tmem_cols * P.nbuf * (P.wide ? 2 : 1)))
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_acc = tmem_base_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int tile, kb, row0;
      const CUtensorMap *tmW;
      pdl_wait();
      const int lo_off = P.tt * BK * 2;          // the lo rows follow the hi rows of the tile
      tile = (int)(u_lo / KB);
      kb = (int)(u_lo % KB);
      tmW = tile_map(tile, row0);
      for (int it = 0; it < pre; ++it) {
        unsigned char *xd = tiles + (size_t)it * stage_bytes + w_stage_bytes;
        if (it >= P.early_w) {
          mbar_expect_tx(&full_bar[it], (uint32_t)stage_bytes);
          load_w(tmW, &full_bar[it], tiles + (size_t)it * stage_bytes, kb, row0);
        }
        tma_load_2d(&tmX, &full_bar[it], xd, kb * BK, tok0);
        if (P.pair) tma_load_2d(&tmXlo, &full_bar[it], xd + lo_off, kb * BK, tok0);
        if (++kb == KB) { kb = 0; ++tile; tmW = tile_map(tile, row0); }
      }
      bool ok = true;
      int s = pre % P.stages;
      uint32_t ph = (uint32_t)(pre / P.stages) & 1u;
      // Optional (tuning key 14): the weight tiles of the units `pf_ahead` beyond the one being loaded are
      // requested into L2.  With the two 96 KB stages of the 256-token mode this was measured slower
      // than no lookahead (13B shapes: 18.2 against 17.7 ms per verification), so it is off.
      int pf_tile = tile, pf_kb = kb, pf_row0 = row0, pf_it = pre;
      const CUtensorMap *pf_map = tmW;
      auto pf_step = [&]() {
        if (++pf_kb == KB) { pf_kb = 0; ++pf_tile; pf_map = tile_map(pf_tile, pf_row0); }
        ++pf_it;
      };
      auto pf_request = [&]() {
        asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];"
                     ::"l"(pf_map), "r"(pf_kb * BK), "r"(pf_row0) : "memory");
        if (P.wide)
          asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];"
                       ::"l"(pf_map), "r"(pf_kb * BK), "r"(pf_row0 + BM) : "memory");
      };
      if (P.pf_ahead > 0) {
        for (int q = 0; q < P.pf_ahead && pf_it < n_units; ++q) { pf_request(); pf_step(); }
      }
      for (int it = pre; it < n_units; ++it) {
        if (P.pf_ahead > 0 && pf_it < n_units) { pf_request(); pf_step(); }
        ok = mbar_wait(&empty_bar[s], ph ^ 1u);
        if (!ok) break;
        mbar_expect_tx(&full_bar[s], (uint32_t)stage_bytes);
        unsigned char *dst = tiles + (size_t)s * stage_bytes;
        load_w(tmW, &full_bar[s], dst, kb, row0);
        tma_load_2d(&tmX, &full_bar[s], dst + w_stage_bytes, kb * BK, tok0);
        if (P.pair) tma_load_2d(&tmXlo, &full_bar[s], dst + w_stage_bytes + lo_off, kb * BK, tok0);
        if (++kb == KB) { kb = 0; ++tile; tmW = tile_map(tile, row0); }
        if (++s == P.stages) { s = 0; ph ^= 1u; }
      }
      if (!ok) {
        atomicExch(&s_error, 1);
        // let the copies already requested land before the block's memory goes away
        for (int q = 0; q < P.stages; ++q) (void)mbar_wait(&full_bar[q], 0);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      // instruction descriptor: D fp32, A and B bf16, both K-major, N = bn, M = 128
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(P.bn >> 3) << 17) |
                             ((uint32_t)(BM >> 4) << 24);
      bool ok = true;
      int seg = 0;                        // segment = run of units inside one tile
      bool seg_start = true;
      int kb = (int)(u_lo % KB), s = 0, buf = 0;
      uint32_t ph = 0;
      for (int it = 0; it < n_units; ++it) {
        if (seg_start && seg >= P.nbuf) {
          // the accumulator buffer must have been drained by the epilogue of segment seg - nbuf
          ok = mbar_wait(&acc_empty[buf], (uint32_t)((seg / P.nbuf) - 1) & 1u);
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        }
        ok = mbar_wait(&full_bar[s], ph);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t wa = smem_u32(tiles + (size_t)s * stage_bytes);
        const uint64_t da = smem_desc_sw128(wa);
        const uint64_t da2 = smem_desc_sw128(wa + W_STAGE_BYTES);      // wide: the second 128 weight rows
        const uint64_t db = smem_desc_sw128(wa + (uint32_t)w_stage_bytes);
        const uint64_t db2 = smem_desc_sw128(wa + (uint32_t)(w_stage_bytes + P.tt * BK * 2));   // accp: the residual rows
        const uint32_t dacc = tmem_acc + (uint32_t)(buf * P.tmem_cols);
#pragma unroll
        for (int k = 0; k < BK / UMMA_K; ++k) {
          // advance 32 bytes (16 bf16) inside the swizzled row: +2 in the 16-byte address field
          const uint32_t acc = (!seg_start || k > 0) ? 1u : 0u;
          umma_bf16(dacc, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, acc);
          if (P.accp) umma_bf16(dacc, da + (uint64_t)(2 * k), db2 + (uint64_t)(2 * k), idesc, 1u);
          if (P.wide) {
            umma_bf16(dacc + (uint32_t)P.tmem_cols, da2 + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, acc);
            if (P.accp) umma_bf16(dacc + (uint32_t)P.tmem_cols, da2 + (uint64_t)(2 * k), db2 + (uint64_t)(2 * k), idesc, 1u);
          }
        }
        umma_commit(&empty_bar[s]);      // stage reusable once these MMAs have read it
        const bool seg_end = (kb == KB - 1) || it == n_units - 1;
        if (seg_end) {
          umma_commit(&acc_full[buf]);   // this segment's accumulator is complete
          ++seg;
          buf = (P.nbuf == 2) ? (buf ^ 1) : 0;
        }
        seg_start = seg_end;
        if (++kb == KB) kb = 0;
        if (++s == P.stages) { s = 0; ph ^= 1u; }
      }
      if (!ok) atomicExch(&s_error, 1);
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int quarter = warp & 3;        // the 32 tensor-memory lanes this warp may read
    // with more than four epilogue warps the warps of a lane quarter share the token columns
    const int n_ch = ((int)(blockDim.x >> 5) - 2) >> 2;
    const int c_per = (((P.tt >> 4) + n_ch - 1) / n_ch) << 4;
    const int c_lo = min(((warp - 2) >> 2) * c_per, P.tt);
    const int c_hi = min(c_lo + c_per, P.tt);
    // A dry pass first: the loop body once with nothing stored and nothing waited for, while the
    // first tiles stream - the epilogue's instructions are then already fetched when the first
    // accumulator is complete.
    bool dry = P.epi_dry != 0;
    if (!dry) pdl_wait();                // the output buffer may still be read by the previous kernel
    bool ok = true;
    int seg = 0;
    unsigned u = u_lo;
    while (u < u_hi && ok) {
      const int tile = (int)(u / KB);
      unsigned seg_hi = (unsigned)(tile + 1) * KB;
      if (seg_hi > u_hi) seg_hi = u_hi;
      const int buf = seg % P.nbuf;
      if (!dry) {
        ok = mbar_wait(&acc_full[buf], (uint32_t)(seg / P.nbuf) & 1u);
        if (!ok) break;
      }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      int row0, col_off = 0, n_rows = P.n0;
      if (tile >= P.tiles1) { row0 = (tile - P.tiles1) * bm; col_off = P.n0 + P.n1; n_rows = P.n2; }
      else if (tile >= P.tiles0) { row0 = (tile - P.tiles0) * bm; col_off = P.n0; n_rows = P.n1; }
      else row0 = tile * bm;
      if (dry) n_rows = 0;
      // which partial-sum slot: classic = the split index; stream-K = rank among the tile's contributors
      int slot = blockIdx.y;
      if (P.sk_ctas > 0)
        slot = (int)blockIdx.x - (int)sk_owner((unsigned)tile * KB, (unsigned)P.sk_ctas, P.sk_units);
      for (int hw = 0; hw < (P.wide ? 2 : 1); ++hw) {      // wide: one accumulator per 128 weight rows
      const int feat = row0 + hw * BM + quarter * 32 + lane;
      float *Yp = P.Y + (size_t)slot * P.split_stride + col_off + feat;
      const uint32_t lane_base = tmem_acc + (uint32_t)((buf + hw) * P.tmem_cols) + ((uint32_t)(quarter * 32) << 16);
      // 16 token columns per step; the next step's accumulator read is in flight while this
      // step's values are stored
      // (registers of a read in flight are not touched before its wait)
      uint32_t va[16], vb[16];
      auto store16 = [&](const uint32_t (&v)[16], int c0) {
        if (feat < n_rows) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const int t = tok0 + c0 + j;
            if (t < P.R) Yp[(size_t)t * P.ldy] = __uint_as_float(v[j]);
          }
        }
      };
      if (P.pair && !P.accp) {
        // value and residual rows in separate accumulator columns: added here
        for (int c0 = c_lo; c0 < c_hi; c0 += 16) {
          tmem_ld16(lane_base + (uint32_t)c0, va);
          tmem_ld16(lane_base + (uint32_t)(P.tt + c0), vb);
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
          for (int j = 0; j < 16; ++j) va[j] = __float_as_uint(__uint_as_float(va[j]) + __uint_as_float(vb[j]));
          store16(va, c0);
        }
      } else {
        if (c_lo < c_hi) tmem_ld16(lane_base + (uint32_t)c_lo, va);
        for (int c0 = c_lo; c0 < c_hi; c0 += 32) {
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
          const bool has_b = c0 + 16 < c_hi;
          if (has_b) tmem_ld16(lane_base + (uint32_t)(c0 + 16), vb);
          store16(va, c0);
          if (has_b) {
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            if (c0 + 32 < c_hi) tmem_ld16(lane_base + (uint32_t)(c0 + 32), va);
            store16(vb, c0 + 16);
          }
        }
      }
      }
      if (dry) {                         // the same segment again, for real
        dry = false;
        pdl_wait();
        continue;
      }
      // hand the accumulator buffer back to the MMA issuer
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&acc_empty[buf])) : "memory");
      ++seg;
      u = seg_hi;
    }
    if (!ok) atomicExch(&s_error, 1);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    if (s_error) {
      // a wait ran out somewhere in the block: MMAs issued before that may still be running, and
      // tensor memory must not be freed under them
      if (lane == 0) {
        umma_commit(&drain_bar);
        (void)mbar_wait(&drain_bar, 0);
      }
      __syncwarp();
    }
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                 ::"r"(tmem_acc), "r"((uint32_t)(P.tmem_cols * P.nbuf * (P.wide ? 2 : 1)))
                 : "memory");
  }
  if (threadIdx.x == 0 && s_error && P.status) atomicMax(P.status, E_TIMEOUT);
}

// ------------------------------------------------------------------------------- CTA pairs
// More than 64 tokens as a pair of activations, two CTAs of a cluster as one MMA unit
// (cta_group::2), token tile tt = 128 or 256.  With one CTA per tile these forms are bound by what
// L2 delivers into shared memory (128 tokens: 48 KB per 128 weight rows and K block, three times the
// weight bytes; 256 tokens: 96 KB per 256 weight rows).  Here a pair of CTAs owns 512 weight rows:
// every MMA has M = 256 (128 weight rows from each CTA) and N = tt tokens, of which each CTA loads
// only its half (value rows and residual rows).  Per CTA and stage: weight rows
// [a*256 + rank*128, +128) for the accumulators a = 0, 1 (2 x 16 KB) and tokens [rank*tt/2, +tt/2)
// as value and residual rows (2 x tt/2 x 128 B): 48 KB (four stages) or 64 KB (three).  With 128
// tokens the two accumulators take 256 tensor-memory columns and there are two sets, so the
// epilogue of one segment overlaps the MMAs of the next.  Every load of both CTAs is counted on
// the even CTA's full barrier; that CTA's MMA thread issues for the pair and its commits arrive on
// the empty / accumulator barriers of both CTAs; each CTA's epilogue warps read its own 128
// accumulator lanes and arrive on the even CTA's accumulator-empty barrier.  Stream-K over the
// clusters, one cluster per SM pair.
constexpr int PAIR_THREADS = 576;
constexpr int PAIR_PART_BYTES = BM * BK * 2;          // 16 KB: 128 rows of one operand part
constexpr int PAIR_MAX_STAGES = 4;
constexpr int PAIR_ROWS = 4 * BM;                     // weight rows per cluster tile

__global__ void __launch_bounds__(PAIR_THREADS, 1)
gemm_tc_pair_kernel(const __grid_constant__ CUtensorMap tmW0, const __grid_constant__ CUtensorMap tmW1,
                    const __grid_constant__ CUtensorMap tmW2, const __grid_constant__ CUtensorMap tmX,
                    const __grid_constant__ CUtensorMap tmXlo, const TcParams P) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ uint64_t full_bar[PAIR_MAX_STAGES];    // used in the even CTA: both CTAs' loads of a stage landed
  __shared__ uint64_t empty_bar[PAIR_MAX_STAGES];   // per CTA: the pair's MMAs have read this stage
  __shared__ uint64_t acc_full[2];              // per CTA: a segment's accumulators are complete
  __shared__ uint64_t acc_empty[2];             // used in the even CTA: both CTAs' epilogues drained them
  __shared__ uint64_t drain_bar;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int s_error;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();
  const unsigned cid = blockIdx.x >> 1;                       // cluster index
  const uint32_t raw = smem_u32(smem_raw);
  unsigned char *tiles = smem_raw + ((1024u - (raw & 1023u)) & 1023u);
  const int KB = P.kblocks;
  const unsigned u_lo = (unsigned)(((unsigned long long)cid * P.sk_units) / (unsigned)P.sk_ctas);
  const unsigned u_hi = (unsigned)(((unsigned long long)(cid + 1) * P.sk_units) / (unsigned)P.sk_ctas);
  const int n_units = (int)(u_hi - u_lo);
  const int n_epi = (int)(blockDim.x >> 5) - 2;
  const int tt = P.tt;                                   // 128 or 256 tokens per tile
  const int x_part = (tt >> 1) * BK * 2;                  // this CTA's tokens, value or residual rows
  const int stage_bytes = 2 * PAIR_PART_BYTES + 2 * x_part;
  const int n_stages = P.stages;

  auto tile_map = [&](int tile, int &row0) -> const CUtensorMap * {
    if (tile >= P.tiles1) { row0 = (tile - P.tiles1) * PAIR_ROWS; return &tmW2; }
    if (tile >= P.tiles0) { row0 = (tile - P.tiles0) * PAIR_ROWS; return &tmW1; }
    row0 = tile * PAIR_ROWS;
    return &tmW0;
  };
  const int pre = n_units < n_stages ? n_units : n_stages;

  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    for (int s = 0; s < n_stages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&acc_full[i], 1);
      mbar_init(&acc_empty[i], (uint32_t)(2 * n_epi));
    }
    mbar_init(&drain_bar, 1);
    s_error = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmW0) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmX) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmXlo) : "memory");
  }
  if (warp == 1) {
    // the same warp of both CTAs allocates all 512 columns in both tensor memories
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&tmem_base_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_barrier();            // both CTAs' barriers exist before anything signals them
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_acc = tmem_base_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      uint32_t full_even[PAIR_MAX_STAGES];
      for (int s = 0; s < PAIR_MAX_STAGES; ++s) full_even[s] = cluster_addr_of(smem_u32(&full_bar[s]), 0);
      int tile = (int)(u_lo / KB), kb = (int)(u_lo % KB), row0;
      const CUtensorMap *tmW = tile_map(tile, row0);
      auto load_w = [&](int s) {
        unsigned char *dst = tiles + (size_t)s * stage_bytes;
        if (rank == 0) mbar_expect_tx(&full_bar[s], 2u * (uint32_t)stage_bytes);
        tma_load_2d_pair(tmW, full_even[s], dst, kb * BK, row0 + (int)rank * BM);
        tma_load_2d_pair(tmW, full_even[s], dst + PAIR_PART_BYTES, kb * BK, row0 + 2 * BM + (int)rank * BM);
      };
      auto load_x = [&](int s, int kbx) {
        unsigned char *dst = tiles + (size_t)s * stage_bytes + 2 * PAIR_PART_BYTES;
        tma_load_2d_pair(&tmX, full_even[s], dst, kbx * BK, (int)rank * (tt >> 1));
        tma_load_2d_pair(&tmXlo, full_even[s], dst + x_part, kbx * BK, (int)rank * (tt >> 1));
      };
      // the first stages' weights do not depend on the kernel before this one
      int kb_first[PAIR_MAX_STAGES];
      for (int it = 0; it < pre; ++it) {
        kb_first[it] = kb;
        load_w(it);
        if (++kb == KB) { kb = 0; ++tile; tmW = tile_map(tile, row0); }
      }
      pdl_wait();
      for (int it = 0; it < pre; ++it) load_x(it, kb_first[it]);
      bool ok = true;
      int s = pre % n_stages;
      uint32_t ph = (uint32_t)(pre / n_stages) & 1u;
      for (int it = pre; it < n_units; ++it) {
        ok = mbar_wait(&empty_bar[s], ph ^ 1u);
        if (!ok) break;
        load_w(s);
        load_x(s, kb);
        if (++kb == KB) { kb = 0; ++tile; tmW = tile_map(tile, row0); }
        if (++s == n_stages) { s = 0; ph ^= 1u; }
      }
      if (!ok) atomicExch(&s_error, 1);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (even CTA)
    if (lane == 0 && rank == 0) {
      // D fp32, A and B bf16, both K-major, N = tt, M = 256 over the two CTAs
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(tt >> 3) << 17) |
                             ((uint32_t)(256 >> 4) << 24);
      bool ok = true;
      int seg = 0;
      bool seg_start = true;
      int kb = (int)(u_lo % KB), s = 0, buf = 0;
      uint32_t ph = 0;
      for (int it = 0; it < n_units; ++it) {
        if (seg_start && seg >= P.nbuf) {
          ok = mbar_wait(&acc_empty[buf], (uint32_t)((seg / P.nbuf) - 1) & 1u);
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        }
        ok = mbar_wait(&full_bar[s], ph);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t wa = smem_u32(tiles + (size_t)s * stage_bytes);
        const uint64_t da0 = smem_desc_sw128(wa);
        const uint64_t da1 = smem_desc_sw128(wa + PAIR_PART_BYTES);
        const uint64_t dbh = smem_desc_sw128(wa + 2 * PAIR_PART_BYTES);
        const uint64_t dbl = smem_desc_sw128(wa + 2 * PAIR_PART_BYTES + (uint32_t)x_part);
        const uint32_t d0 = tmem_acc + (uint32_t)(buf * 2 * tt), d1 = d0 + (uint32_t)tt;
#pragma unroll
        for (int k = 0; k < BK / UMMA_K; ++k) {
          const uint32_t acc = (!seg_start || k > 0) ? 1u : 0u;
          umma2_bf16(d0, da0 + (uint64_t)(2 * k), dbh + (uint64_t)(2 * k), idesc, acc);
          umma2_bf16(d0, da0 + (uint64_t)(2 * k), dbl + (uint64_t)(2 * k), idesc, 1u);
          umma2_bf16(d1, da1 + (uint64_t)(2 * k), dbh + (uint64_t)(2 * k), idesc, acc);
          umma2_bf16(d1, da1 + (uint64_t)(2 * k), dbl + (uint64_t)(2 * k), idesc, 1u);
        }
        umma2_commit_to(&empty_bar[s], 3);
        const bool seg_end = (kb == KB - 1) || it == n_units - 1;
        if (seg_end) {
          umma2_commit_to(&acc_full[buf], 3);
          ++seg;
          buf = (P.nbuf == 2) ? (buf ^ 1) : 0;
        }
        seg_start = seg_end;
        if (++kb == KB) kb = 0;
        if (++s == n_stages) { s = 0; ph ^= 1u; }
      }
      if (!ok) atomicExch(&s_error, 1);
    }
  } else {
    // ------------------------------------------------------------------ epilogue (both CTAs)
    const int quarter = warp & 3;
    const int n_ch = n_epi >> 2;
    const int c_per = (((tt >> 4) + n_ch - 1) / n_ch) << 4;   // token columns in steps of 16
    const int c_lo = min(((warp - 2) >> 2) * c_per, tt);
    const int c_hi = min(c_lo + c_per, tt);
    const uint32_t acc_empty_even[2] = {cluster_addr_of(smem_u32(&acc_empty[0]), 0),
                                        cluster_addr_of(smem_u32(&acc_empty[1]), 0)};
    bool dry = P.epi_dry != 0;           // a dry pass over the loop body first (nothing stored, nothing waited for)
    bool ok = true;
    int seg = 0;
    unsigned u = u_lo;
    while (u < u_hi && ok) {
      const int tile = (int)(u / KB);
      unsigned seg_hi = (unsigned)(tile + 1) * KB;
      if (seg_hi > u_hi) seg_hi = u_hi;
      const int buf = seg % P.nbuf;
      if (!dry) {
        ok = mbar_wait(&acc_full[buf], (uint32_t)(seg / P.nbuf) & 1u);
        if (!ok) break;
      }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      int row0, col_off = 0, n_rows = P.n0;
      if (tile >= P.tiles1) { row0 = (tile - P.tiles1) * PAIR_ROWS; col_off = P.n0 + P.n1; n_rows = P.n2; }
      else if (tile >= P.tiles0) { row0 = (tile - P.tiles0) * PAIR_ROWS; col_off = P.n0; n_rows = P.n1; }
      else row0 = tile * PAIR_ROWS;
      if (dry) n_rows = 0;
      // partial-sum slot = rank of this cluster among the tile's contributors
      const int slot = (int)cid - (int)sk_owner((unsigned)tile * KB, (unsigned)P.sk_ctas, P.sk_units);
      for (int a = 0; a < 2; ++a) {
        const int feat = row0 + a * 2 * BM + (int)rank * BM + quarter * 32 + lane;
        float *Yp = P.Y + (size_t)slot * P.split_stride + col_off + feat;
        const uint32_t lane_base = tmem_acc + (uint32_t)((buf * 2 + a) * tt) + ((uint32_t)(quarter * 32) << 16);
        uint32_t va[16], vb[16];
        auto store16 = [&](const uint32_t (&v)[16], int c0) {
          if (feat < n_rows) {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int t = c0 + j;
              if (t < P.R) Yp[(size_t)t * P.ldy] = __uint_as_float(v[j]);
            }
          }
        };
        if (c_lo < c_hi) tmem_ld16(lane_base + (uint32_t)c_lo, va);
        for (int c0 = c_lo; c0 < c_hi; c0 += 32) {
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
          const bool has_b = c0 + 16 < c_hi;
          if (has_b) tmem_ld16(lane_base + (uint32_t)(c0 + 16), vb);
          store16(va, c0);
          if (has_b) {
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            if (c0 + 32 < c_hi) tmem_ld16(lane_base + (uint32_t)(c0 + 32), va);
            store16(vb, c0 + 16);
          }
        }
      }
      if (dry) {                         // the same segment again, for real
        dry = false;
        continue;
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(acc_empty_even[buf]);
      ++seg;
      u = seg_hi;
    }
    if (!ok) atomicExch(&s_error, 1);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1 && rank == 0 && s_error) {
    // a wait ran out: MMAs issued before that may still be running on both tensor memories
    if (lane == 0) {
      asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                   ::"r"(smem_u32(&drain_bar)) : "memory");
      (void)mbar_wait(&drain_bar, 0);
    }
    __syncwarp();
  }
  // neither CTA frees tensor memory or leaves while the other may still be signalled or read
  cluster_barrier();
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(512u) : "memory");
  }
  if (threadIdx.x == 0 && s_error && P.status) atomicMax(P.status, E_TIMEOUT);
}

// ------------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;
std::mutex g_mu;
std::map<std::tuple<const void *, int, int, int>, CUtensorMap> g_maps;   // (ptr, rows, K, box rows)
// Per-device facts and set-up: the kernel's shared-memory opt-in is an attribute of the function on
// one device, so every device the library is used on is prepared once (under g_mu).
constexpr int MAX_DEVICES = 64;
struct DevInfo {
  bool ready;
  int smem_optin, num_sms;
  int pair_clusters;    // CTA pairs of gemm_tc_pair_kernel that can be resident at once (0: not usable)
};
DevInfo g_dev[MAX_DEVICES] = {};
thread_local int t_dev = 0;          // the calling thread's current device as of its last use_current_device()
// Points the per-device facts at the calling thread's current device; false if that device was
// never prepared by tc_init_driver().
bool use_current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES || !g_dev[dev].ready) return false;
  t_dev = dev;
  return true;
}
#define g_smem_optin (g_dev[t_dev].smem_optin)
#define g_num_sms (g_dev[t_dev].num_sms)
#define g_pair_clusters (g_dev[t_dev].pair_clusters)
int g_tune_stages = 0;      // 0 = as many as fit (at most 8)
int g_tune_max_split = 0;   // 0 = default rule
int g_tune_no_streamk = 0;  // 1 = always the per-tile decomposition
int g_tune_l2_ahead = -1;   // < 0 = default
int g_tune_late_w = 0;      // 1 = weights wait for the dependency too
int g_tune_early_stages = -1; // < 0 = all stages
int g_tune_no_wave_split = 0; // 1 = several token tiles keep the one-wave rule's split factor
int g_tune_no_accp = 0;      // 1 = pairs of more than 128 tokens as two 128-token tiles with extra columns
int g_tune_epi = 0;         // 1, 2: that many epilogue warps per lane quarter for 256-row weight tiles (default 4)
int g_tune_epi_narrow = 0;  // 1, 2, 4: epilogue warps per lane quarter for 128-row weight tiles (default by token tile)
int g_tune_no_pair2 = 0;    // 1 = no CTA-pair kernel; 2 = not for 65 to 128 tokens
int g_tune_pair_min = 0;    // > 0: fewest rows for the CTA-pair kernel
int g_tune_epi_dry = 1;
int g_tune_pf = 0;           // > 0: weight tiles requested into L2 ahead of the ring in that mode
int g_tune_no_wide = 0;      // 1 = 128 weight rows per CTA also for wide token tiles
int g_tune_traffic_div = 8; // split <= K_in / (div * tokens)

bool get_map(const void *ptr, int rows, int K_in, int box_rows, CUtensorMap *out) {
  std::lock_guard<std::mutex> lock(g_mu);
  auto key = std::make_tuple(ptr, rows, K_in, box_rows);
  auto it = g_maps.find(key);
  if (it != g_maps.end()) {
    *out = it->second;
    return true;
  }
  if (!g_encode) return false;
  CUtensorMap m;
  cuuint64_t dims[2] = {(cuuint64_t)K_in, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)K_in * 2};
  cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g_encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides,
                        box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  g_maps[key] = m;
  *out = m;
  return true;
}

}  // namespace

bool tc_get_map(const void *ptr, int rows, int K_in, int box_rows, CUtensorMap *out) {
  return get_map(ptr, rows, K_in, box_rows, out);
}
int tc_smem_optin() { return use_current_device() ? g_smem_optin : 0; }
int tc_num_sms() { return use_current_device() ? g_num_sms : 0; }

// Prepares the calling thread's current device (once per device) and remembers it for the
// launchers that follow on this thread.
int tc_init_driver(char *err, size_t errlen) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) {
    snprintf(err, errlen, "no usable current device: %s", cudaGetErrorString(e));
    return 1;
  }
  std::lock_guard<std::mutex> lock(g_mu);
  t_dev = dev;
  if (g_dev[dev].ready) return 0;
  if (!g_encode) {
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
    if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || fn == nullptr) {
      snprintf(err, errlen, "cuTensorMapEncodeTiled not available: %s", cudaGetErrorString(e));
      return 1;
    }
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  }
  DevInfo d{};
  cudaDeviceGetAttribute(&d.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  cudaDeviceGetAttribute(&d.num_sms, cudaDevAttrMultiProcessorCount, dev);
  e = cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, d.smem_optin - 1024);
  if (e != cudaSuccess) {
    snprintf(err, errlen, "cannot raise the GEMM kernel's shared memory: %s", cudaGetErrorString(e));
    return 1;
  }
  // the CTA-pair kernel: shared-memory opt-in, and how many pairs fit on this device at once
  {
    const size_t smem = (size_t)3 * (2 * PAIR_PART_BYTES + 256 * BK * 2) + 1024;   // = four stages of the 128-token form
    d.pair_clusters = 0;
    if ((size_t)d.smem_optin >= smem + 1024 &&
        cudaFuncSetAttribute(gemm_tc_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) == cudaSuccess) {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(2 * (d.num_sms / 2));
      cfg.blockDim = dim3(PAIR_THREADS);
      cfg.dynamicSmemBytes = smem;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = 2;
      attr[0].val.clusterDim.y = 1;
      attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr;
      cfg.numAttrs = 1;
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, gemm_tc_pair_kernel, &cfg) == cudaSuccess && n > 0)
        d.pair_clusters = n < d.num_sms / 2 ? n : d.num_sms / 2;
      (void)cudaGetLastError();
    }
  }
  d.ready = true;
  g_dev[dev] = d;
  return 0;
}

void attn_tc_set_min_rows(int rows);
void attn_tc_set_chunks(int chunks);
void attn_tc_set_l2_ahead(int tiles);
void attn_tc_set_dry_pass(int on);
void attn_mma_set_chunks(int chunks);
void tc_set_tuning(int key, int value) {
  if (key == 9) attn_tc_set_min_rows(value);
  if (key == 12) attn_tc_set_chunks(value);
  if (key == 19) attn_tc_set_l2_ahead(value);
  if (key == 20) attn_tc_set_dry_pass(value);
  if (key == 1) g_tune_stages = value;
  if (key == 10) g_tune_no_wave_split = value;
  if (key == 11) g_tune_no_wide = value;
  if (key == 13) g_tune_no_accp = value;
  if (key == 14) g_tune_pf = value;
  if (key == 15) g_tune_epi = value;
  if (key == 16) g_tune_epi_narrow = value;
  if (key == 17) g_tune_no_pair2 = value;
  if (key == 18) g_tune_pair_min = value;
  if (key == 21) g_tune_epi_dry = value;
  if (key == 22) attn_mma_set_chunks(value);
  if (key == 2) g_tune_max_split = value;
  if (key == 3) g_tune_no_streamk = value;
  if (key == 5) g_tune_l2_ahead = value;
  if (key == 6) g_tune_late_w = value;
  if (key == 8) g_tune_early_stages = value;
  if (key == 7 && value > 0) g_tune_traffic_div = value;
}

void tc_forget_maps() {
  std::lock_guard<std::mutex> lock(g_mu);
  g_maps.clear();
}

bool tc_supported(const GemmMats &m, int K_in) {
  if (K_in % BK != 0 || K_in < BK) return false;
  for (int i = 0; i < m.n; ++i)
    if (m.n_out[i] < 1 || ((uintptr_t)m.W[i] & 15u)) return false;
  return g_encode != nullptr;
}

// Split-K factor: as many CTAs as fit in one wave of the co-resident slots (two per SM), while
// every split keeps at least 8 K-blocks and the fp32 partial sums written and re-read
// (split x tokens x 4 bytes per output) stay below about half of the weight bytes.
static int split_cap(int kblocks, int tokens) {
  int s = 8;
  const int by_k = kblocks / 8;
  const int by_traffic = (kblocks * 64) / (g_tune_traffic_div * (tokens > 0 ? tokens : 1));
  if (s > by_k) s = by_k;
  if (s > by_traffic) s = by_traffic;
  if (g_tune_max_split > 0 && s > g_tune_max_split) s = g_tune_max_split;
  return s < 1 ? 1 : s;
}

int tc_default_split(int n_tiles, int kblocks, int tokens) {
  if (!use_current_device()) return 1;
  const int slots = 2 * g_num_sms;
  int s = slots / (n_tiles > 0 ? n_tiles : 1);
  const int cap = split_cap(kblocks, tokens);
  if (s > cap) s = cap;
  return s < 1 ? 1 : s;
}

// Several token tiles (more than 128 rows as pairs): `ctas` = weight tiles x token tiles may exceed
// the co-resident slots, and then the launch runs in rounds whose last one can be nearly empty.
// The time goes as rounds(split) / split (each CTA covers K / split), so among the allowed factors
// take the one with the fewest round-lengths, but leave `split0` (the one-wave rule's choice)
// unless another is at least 10 % better.
static int wave_split(int ctas, int kblocks, int tokens, int split0, int slots) {
  const int cap = split_cap(kblocks, tokens);
  auto cost = [&](int sp) { return (double)((ctas * sp + slots - 1) / slots) / sp; };
  int best = split0 <= cap ? split0 : cap;
  if (best < 1) best = 1;
  double best_cost = cost(best);
  const double keep = 0.9 * best_cost;
  for (int sp = 1; sp <= cap; ++sp)
    if (cost(sp) < keep && cost(sp) < best_cost - 1e-9) { best = sp; best_cost = cost(sp); }
  return best;
}

// Stream-K plan: how many CTAs share the (tile, K-block) units.  At most two per SM, at least 8
// units per CTA, at most `max_slots` contributors to any tile, and the fp32 partial sums written
// and re-read stay below about half of the weight bytes.  Returns 0 when the classic per-tile
// decomposition is at least as good (one contributor per tile already fills the machine).
int tc_streamk_ctas(int n_tiles, int kblocks, int tokens, int max_slots, int *slots_out) {
  const long long units = (long long)n_tiles * kblocks;
  long long g = 2LL * g_num_sms;
  if (g > units / 8) g = units / 8;
  if (g < 1) g = 1;
  // average contributors per tile = kblocks * g / units; bound it by the traffic rule
  const long long by_traffic = (long long)(kblocks * 64) / ((long long)g_tune_traffic_div * (tokens > 0 ? tokens : 1));
  const long long avg_cap = by_traffic < 1 ? 1 : by_traffic;
  if ((long long)kblocks * g > avg_cap * units) g = avg_cap * units / kblocks;
  if (g_tune_max_split > 0 && (long long)kblocks * g > (long long)g_tune_max_split * units)
    g = (long long)g_tune_max_split * units / kblocks;
  if (g < 1) g = 1;
  auto slots_of = [&](long long gg) {
    const long long per = units / gg;                 // smallest run length
    return (int)((kblocks + per - 1) / per) + ((units % gg) || (kblocks % per) ? 1 : 0);
  };
  while (g > 1 && slots_of(g) > max_slots) --g;
  *slots_out = slots_of(g);
  return (int)g;
}

cudaError_t gemm_tc(Launch L, Operand X, int x_rows_alloc, GemmMats m, int K_in, int R,
                    float *Y, int ldy, int split, size_t split_stride, int *status, int max_slots,
                    SplitIn *out) {
  if (!use_current_device()) return cudaErrorInitializationError;
  if (!tc_supported(m, K_in) || R < 1 || ((uintptr_t)X.hi & 15u) || ((uintptr_t)X.lo & 15u))
    return cudaErrorInvalidValue;
  TcParams P;
  memset(&P, 0, sizeof(P));
  const int pair = X.lo != nullptr ? 1 : 0;
  // A pair of more than 128 tokens keeps all of a tile's tokens in one accumulator (two accumulating
  // MMAs per K step, value rows then residual rows) so that a tile holds up to 256 tokens and the
  // weights are passed over once; up to 128 tokens the residual rows are extra accumulator columns.
  const int accp = (pair && R > 128 && !g_tune_no_accp) ? 1 : 0;
  const int tt_max = (pair && !accp) ? 128 : 256;
  int tt = ((R + 15) / 16) * 16;
  if (tt > tt_max) tt = tt_max;
  if (tt > x_rows_alloc) return cudaErrorInvalidValue;
  const int bn = (pair && !accp) ? 2 * tt : tt;
  const int x_bytes = (accp ? 2 : 1) * bn * BK * 2;      // activation bytes of a stage
  const int ztiles = (R + tt - 1) / tt;
  // the last token tile may reach past R: those rows must exist (they are read, results dropped)
  if (ztiles * tt > x_rows_alloc) return cudaErrorInvalidValue;
  P.tt = tt;
  P.pair = pair;
  P.accp = accp;
  P.ztiles = ztiles;
  int cols = 32;
  while (cols < bn) cols <<= 1;
  P.Y = Y;
  P.ldy = ldy;
  P.R = R;
  P.bn = bn;
  P.tmem_cols = cols;
  // wide mode: N = 256, every matrix a whole number of 256-row tiles, room for three 64 KB stages
  // (At exactly 128 tokens, where the extra-column form also reaches N = 256, 128 weight rows per CTA with
  // two CTAs per SM measured 6-7 % faster than 256 rows with one: 7B verify 5.7 against 6.1 ms.)
  bool wide = !g_tune_no_wide && accp && bn == 256 && g_smem_optin - 2048 >= 2 * (2 * W_STAGE_BYTES + x_bytes);
  for (int i = 0; i < m.n && wide; ++i) wide = (m.n_out[i] % (2 * BM)) == 0;
  // CTA pairs (512 weight rows per cluster, each CTA loading half of the tokens): 113 to 256 tokens
  // as a pair, stream-K over the clusters that fit on the device at once.  The last tile of a
  // matrix may be ragged (rows beyond the matrix are zero-filled by the loads and not stored).
  // Measured per verification, 7B shapes: 128 rows 5.67-5.85 against 5.78-5.90 ms, 2 x 64 rows
  // 5.50-5.85 against 5.76-5.90; the 128-token tile costs more than it saves below that (100 rows
  // 5.53 against 5.43, 80 rows 5.25 against 4.48, where the one-CTA form uses an 80-token tile;
  // with 32- and 64-token tiles the pair form measured 13-15 % slower at 16 to 64 rows, where two
  // independent CTAs per SM overlap each other's start and end).
  const int pair_min_rows = g_tune_pair_min > 0 ? g_tune_pair_min : 113;
  if (pair && R >= pair_min_rows && R <= 256 && !(g_tune_no_pair2 & 1) && g_pair_clusters > 0 && split == 0 &&
      out != nullptr && max_slots >= 2 && m.n <= 3 && (R > 128 || !(g_tune_no_pair2 & 2))) {
    const int q0 = (m.n_out[0] + PAIR_ROWS - 1) / PAIR_ROWS, q1 = m.n > 1 ? (m.n_out[1] + PAIR_ROWS - 1) / PAIR_ROWS : 0,
              q2 = m.n > 2 ? (m.n_out[2] + PAIR_ROWS - 1) / PAIR_ROWS : 0;
    const int n_tiles = q0 + q1 + q2, KB = K_in / BK;
    const long long units = (long long)n_tiles * KB;
    long long g = g_pair_clusters;
    if (g > units / 8) g = units / 8;
    if (g < 1) g = 1;
    auto slots_of = [&](long long gg) {
      const long long per = units / gg;
      return (int)((KB + per - 1) / per) + ((units % gg) || (KB % per) ? 1 : 0);
    };
    while (g > 1 && slots_of(g) > max_slots) --g;
    if (slots_of(g) <= max_slots) {
      const int ptt = R > 128 ? 256 : 128;
      P.tt = ptt;
      P.bn = ptt;
      P.nbuf = ptt == 128 ? 2 : 1;
      P.stages = ptt == 128 ? 4 : 3;
      P.tiles0 = q0;
      P.tiles1 = q0 + q1;
      P.n0 = m.n_out[0];
      P.n1 = m.n > 1 ? m.n_out[1] : 0;
      P.n2 = m.n > 2 ? m.n_out[2] : 0;
      P.kblocks = KB;
      P.sk_ctas = (int)g;
      P.sk_units = (unsigned)units;
      P.split = 1;
      P.split_stride = split_stride;
      P.status = status;
      P.epi_dry = g_tune_epi_dry;
      CUtensorMap mw[3], mx, mxlo;
      for (int i = 0; i < 3; ++i) {
        const int j = i < m.n ? i : 0;
        if (!get_map(m.W[j], m.n_out[j], K_in, BM, &mw[i])) return cudaErrorInvalidValue;
      }
      if (!get_map(X.hi, x_rows_alloc, K_in, ptt / 2, &mx)) return cudaErrorInvalidValue;
      if (!get_map(X.lo, x_rows_alloc, K_in, ptt / 2, &mxlo)) return cudaErrorInvalidValue;
      SplitIn si{Y, slots_of(g), split_stride, ldy, (unsigned)g, (unsigned)units, (unsigned)KB, 2u};
      bool ragged = false;
      for (int i = 0; i + 1 < m.n; ++i) ragged = ragged || (m.n_out[i] % PAIR_ROWS) != 0;
      if (ragged) {
        si.sk_m0 = (unsigned)P.n0;
        si.sk_m1 = m.n > 2 ? (unsigned)(P.n0 + P.n1) : 0xFFFFFFFFu;
        si.sk_t0 = (unsigned)q0;
        si.sk_t1 = (unsigned)(q0 + q1);
      }
      *out = si;
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3((unsigned)(2 * g));
      cfg.blockDim = dim3(PAIR_THREADS);
      cfg.dynamicSmemBytes = (size_t)P.stages * (2 * PAIR_PART_BYTES + ptt * BK * 2) + 1024;
      cfg.stream = L.st;
      cudaLaunchAttribute attr[2];
      attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[0].val.programmaticStreamSerializationAllowed = L.pdl ? 1 : 0;
      attr[1].id = cudaLaunchAttributeClusterDimension;
      attr[1].val.clusterDim.x = 2;
      attr[1].val.clusterDim.y = 1;
      attr[1].val.clusterDim.z = 1;
      cfg.attrs = attr;
      cfg.numAttrs = 2;
      ++g_launches;
      return cudaLaunchKernelEx(&cfg, gemm_tc_pair_kernel, mw[0], mw[1], mw[2], mx, mxlo, P);
    }
    memset(&P, 0, sizeof(P));
    P.tt = tt; P.pair = pair; P.accp = accp; P.ztiles = ztiles; P.Y = Y; P.ldy = ldy; P.R = R; P.bn = bn; P.tmem_cols = cols;
  }
  const int bmw = wide ? 2 * BM : BM;
  P.wide = wide ? 1 : 0;
  const int t0 = (m.n_out[0] + bmw - 1) / bmw;
  const int t1 = m.n > 1 ? (m.n_out[1] + bmw - 1) / bmw : 0;
  const int t2 = m.n > 2 ? (m.n_out[2] + bmw - 1) / bmw : 0;
  const int n_tiles = t0 + t1 + t2;
  P.tiles0 = t0;
  P.tiles1 = t0 + t1;
  P.n0 = m.n_out[0];
  P.n1 = m.n > 1 ? m.n_out[1] : 0;
  P.n2 = m.n > 2 ? m.n_out[2] : 0;
  P.kblocks = K_in / BK;
  // stream-K (split == 0): needs a single token tile and 128-row-aligned matrices, so that a
  // column's tile (and with it the number of partial sums to add) follows from the column index
  bool sk = split == 0 && ztiles == 1 && max_slots >= 2 && out != nullptr && !g_tune_no_streamk;
  for (int i = 0; i < m.n && sk; ++i) sk = (m.n_out[i] % bmw) == 0;
  // stream-K pays off where the per-tile decomposition cannot be split further and leaves the SMs
  // unevenly loaded (more tiles than SMs, not a whole number of two-per-SM waves); elsewhere
  // classic split-K gives the same balance with fewer partial sums per tile.  With 256-row tiles
  // (one CTA per SM, tensor-bound) it is taken whenever the best split factor would leave more
  // than a tenth of the SM-rounds empty.
  int sk_ctas = 0, sk_slots = 1;
  if (sk && wide) {
    const int sp = wave_split(n_tiles, P.kblocks, R, 1, g_num_sms);
    const int ctas = n_tiles * sp, rounds = (ctas + g_num_sms - 1) / g_num_sms;
    sk = (double)ctas < 0.9 * (double)rounds * g_num_sms;
    if (sk) {
      // every CTA at least 8 K-blocks, at most max_slots contributors per tile
      const long long units = (long long)n_tiles * P.kblocks;
      long long g = g_num_sms;
      if (g > units / 8) g = units / 8;
      if (g < 1) g = 1;
      auto slots_of = [&](long long gg) {
        const long long per = units / gg;
        return (int)((P.kblocks + per - 1) / per) + ((units % gg) || (P.kblocks % per) ? 1 : 0);
      };
      while (g > 1 && slots_of(g) > max_slots) --g;
      sk_ctas = (int)g;
      sk_slots = slots_of(g);
      if (sk_ctas <= ctas) sk = false;          // the classic decomposition uses as many CTAs
    }
  } else if (sk) {
    const int classic = tc_default_split(n_tiles, P.kblocks, R);
    sk = classic == 1 && n_tiles > g_num_sms && (n_tiles % (2 * g_num_sms)) != 0;
    if (sk) {
      sk_ctas = tc_streamk_ctas(n_tiles, P.kblocks, R, max_slots, &sk_slots);
      if (sk_ctas <= n_tiles) sk = false;         // nothing to share: one CTA per tile is the same thing
    }
  }
  if (!sk) {
    sk_ctas = 0;
    if (split < 1 && wide) {
      // one CTA per SM: the factor with the fewest round-lengths over the SMs
      split = wave_split(n_tiles * ztiles, P.kblocks, R, 1, g_num_sms);
    } else if (split < 1) {
      split = tc_default_split(n_tiles, P.kblocks, R);
      if (ztiles > 1 && !g_tune_no_wave_split) split = wave_split(n_tiles * ztiles, P.kblocks, R, split, 2 * g_num_sms);
    }
    if (split > P.kblocks) split = P.kblocks;
    if (max_slots > 0 && split > max_slots) split = max_slots;
  }
  P.split = sk ? 1 : split;
  P.sk_ctas = sk_ctas;
  P.sk_units = (unsigned)((long long)n_tiles * P.kblocks);
  P.split_stride = split_stride;
  P.status = status;
  P.nbuf = (sk && 2 * cols <= 256) ? 2 : 1;
  P.epi_dry = g_tune_epi_dry;
  const int stage_bytes = (wide ? 2 : 1) * W_STAGE_BYTES + x_bytes;
  int stages = (g_smem_optin - 2048) / stage_bytes;
  if (stages > MAX_STAGES) stages = MAX_STAGES;
  if (stages > 8) stages = 8;
  // default: two CTAs per SM (each with half of the shared memory), so that one CTA's prologue and
  // epilogue overlap the other's streaming
  const int two_per_sm = (g_smem_optin / 2 - 2048) / stage_bytes;
  if (g_tune_stages == 0 && two_per_sm >= 2 && two_per_sm < stages && !wide) stages = two_per_sm;
  if (g_tune_stages > 0 && g_tune_stages < stages) stages = g_tune_stages;
  if (stages < 2) return cudaErrorInvalidValue;
  P.stages = stages;
  P.l2_ahead = g_tune_l2_ahead >= 0 ? g_tune_l2_ahead : L2_AHEAD;
  P.pf_ahead = (accp && stages < 4 && g_tune_pf > 0) ? g_tune_pf : 0;   // measured: no lookahead is fastest (13B, 256 rows)
  P.early_w = g_tune_late_w ? 0 : (g_tune_early_stages >= 0 && g_tune_early_stages < stages ? g_tune_early_stages : stages);
  CUtensorMap mw[3], mx, mxlo;
  for (int i = 0; i < 3; ++i) {
    const int j = i < m.n ? i : 0;
    if (!get_map(m.W[j], m.n_out[j], K_in, BM, &mw[i])) return cudaErrorInvalidValue;
  }
  if (!get_map(X.hi, x_rows_alloc, K_in, tt, &mx)) return cudaErrorInvalidValue;
  if (!get_map(pair ? X.lo : X.hi, x_rows_alloc, K_in, tt, &mxlo)) return cudaErrorInvalidValue;
  dim3 grid = sk ? dim3(sk_ctas, 1, 1) : dim3(n_tiles * ztiles, split, 1);
  const size_t smem = (size_t)stages * stage_bytes + 1024;
  if (out) {
    *out = SplitIn{Y, sk ? sk_slots : split, split_stride, ldy, sk ? (unsigned)sk_ctas : 0u, P.sk_units,
                   (unsigned)P.kblocks, (sk && wide) ? 1u : 0u};
  }
  // Epilogue warps per 32 accumulator lanes.  256-row tiles keep one accumulator set, so the MMAs
  // of a CTA's next tile wait for the epilogue: sixteen warps (13B-shaped verification of 256 rows:
  // 18.3 ms with four, 16.8 with eight, 16.3 with sixteen).  128-row tiles: eight warps (per 7B
  // verification, against four: 16 to 48 rows 2-3 % faster, 60 and 64 rows 1 %, 100 rows 0.8 %,
  // 80 rows 0.5 % slower; the draft passes 2 % faster).
  int groups = wide ? 4 : 2;
  const int forced = wide ? g_tune_epi : g_tune_epi_narrow;
  if (forced == 1 || forced == 2 || forced == 4) groups = forced;
  return launch_k(gemm_tc_kernel, grid, dim3(64 + 128 * groups), smem, L.st, L.pdl, mw[0], mw[1], mw[2], mx, mxlo, P);
}

}  // namespace koala
