// Causal branch of Algorithm 1 on the 5th-generation tensor cores (bf16 inputs, d_k = d_v = 128,
// 128-token tiles): tcgen05.mma with TMEM accumulators, operands staged by TMA into 128-byte-swizzled
// shared memory.
//
//   chunk_scan_tc_kernel   : D_b = K_bᵀ V_b for the chunks of one block in order, with the exclusive
//                            prefix sum carried in registers; emits S_in[b] as bf16        (steps 5-6)
//   tile_product_tc_kernel : O_b = Q_b S_in[b] + tril(Q_b K_bᵀ) V_b + Y_lr,b (step 7, Eq. "local") and the three
//                            within-chunk adjoints of the backward pass (Eq. "local-adjoint")
//
// The tile width is 128 tokens whatever chunk size the caller named: the result does not depend on the
// chunk width once the block boundary n is fixed, and the launcher requires n and T - n to be multiples of 128.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "smat_internal.h"
#include "smat_tc.cuh"

namespace {

using namespace tc;

constexpr int TILE = 128;              // tokens per tile, and d_k = d_v
constexpr int HALF = 64;               // columns per 128-byte swizzled row
constexpr int BOX_BYTES = TILE * 128;  // one TMA box: 128 rows x 128 bytes = 16 KB

// ---------------------------------------------------------------------------------------------------------------
// chunk_scan_tc_kernel: one CTA per (head, block, 64-column half of the state).
//   warp 4 lane 0 : TMA producer (K_b: two boxes, V_b[:, half]: one box) into a 3-stage ring
//   warp 5 lane 0 : MMA issuer, D_b = K_bᵀ V_b[:, half]  (M = 128 features, N = 64, K = 128 tokens) into a 4-deep TMEM ring
//   warps 0-3     : one TMEM lane (state row) per thread; keep the running sum in registers, write it as bf16
//                   (the state *before* chunk b is S_in[b]), then add D_b
// ---------------------------------------------------------------------------------------------------------------
constexpr int SCAN_STAGES = 3;
constexpr int SCAN_DBUF = 4;
constexpr int SCAN_STAGE_BYTES = 3 * BOX_BYTES;
constexpr int SCAN_SMEM = SCAN_STAGES * SCAN_STAGE_BYTES + 1024 + 256;

struct ScanParams {
  int64_t T;        // tokens per head
  int NC;           // tiles per head
  int lo[2], hi[2]; // tile ranges of the (up to two) blocks
  int reverse;      // 0: exclusive prefix sums (S_in); 1: exclusive suffix sums (the scan adjoint D̄)
  const float* lam; // gated variant: inclusive prefix sums of the log-gates, [bh][T]; the running state is multiplied by
                    // the tile's total gate before the tile's sum (of rows rescaled to the tile's end, or in reverse
                    // order to its start) is added — the same recursion in both directions
  __nv_bfloat16* Sin;  // [bh][NC][128][128]
  int* status;
};

__global__ void __launch_bounds__(192) chunk_scan_tc_kernel(const __grid_constant__ CUtensorMap tmK,
                                                            const __grid_constant__ CUtensorMap tmV,
                                                            const ScanParams prm) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SCAN_STAGES * SCAN_STAGE_BYTES);
  uint64_t* full = bars;                     // [SCAN_STAGES]
  uint64_t* empty = bars + SCAN_STAGES;      // [SCAN_STAGES]
  uint64_t* dfull = empty + SCAN_STAGES;     // [SCAN_DBUF]
  uint64_t* dempty = dfull + SCAN_DBUF;      // [SCAN_DBUF]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(dempty + SCAN_DBUF);
  volatile int* cta_abort = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int half = blockIdx.x & 1, blk = blockIdx.x >> 1;
  const int bh = blockIdx.y;
  const int lo = prm.lo[blk], hi = prm.hi[blk];
  const WaitCtx wc{cta_abort, prm.status};

  if (threadIdx.x == 0) {
    *cta_abort = 0;
    for (int s = 0; s < SCAN_STAGES; ++s) { mbar_init(full + s, 1); mbar_init(empty + s, 1); }
    for (int s = 0; s < SCAN_DBUF; ++s) { mbar_init(dfull + s, 1); mbar_init(dempty + s, 4); }
    fence_barrier_init();
  }
  if (warp == 4) tmem_alloc(tmem_slot, SCAN_DBUF * HALF);
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 4 && lane == 0) {
    prefetch_tmap(&tmK);
    prefetch_tmap(&tmV);
    for (int it = 0; it + 1 < hi - lo; ++it) {  // the last visited tile's own sum is never read
      const int b = prm.reverse ? hi - 1 - it : lo + it, s = it % SCAN_STAGES;
      if (it >= SCAN_STAGES && !mbar_wait(empty + s, ((it / SCAN_STAGES) - 1) & 1, wc)) break;
      uint8_t* st = smem + s * SCAN_STAGE_BYTES;
      const int row = (int)(bh * prm.T + (int64_t)b * TILE);
      mbar_expect_tx(full + s, SCAN_STAGE_BYTES);
      tma_load_2d(st, &tmK, 0, row, full + s);
      tma_load_2d(st + BOX_BYTES, &tmK, HALF, row, full + s);
      tma_load_2d(st + 2 * BOX_BYTES, &tmV, half * HALF, row, full + s);
    }
  } else if (warp == 5 && lane == 0) {
    constexpr uint32_t idesc = make_idesc(TILE, HALF, 1, 1);
    for (int it = 0; it + 1 < hi - lo; ++it) {
      const int s = it % SCAN_STAGES, db = it % SCAN_DBUF;
      if (!mbar_wait(full + s, (it / SCAN_STAGES) & 1, wc)) break;
      if (it >= SCAN_DBUF && !mbar_wait(dempty + db, ((it / SCAN_DBUF) - 1) & 1, wc)) break;
      fence_after_sync();
      const uint32_t sK = smem_u32(smem + s * SCAN_STAGE_BYTES);
      const uint32_t sV = sK + 2 * BOX_BYTES;
      const uint64_t dA = make_desc(sK, BOX_BYTES, 1024);  // K_b as MN-major A: two 64-feature blocks 16 KB apart
      const uint64_t dB = make_desc(sV, BOX_BYTES, 1024);
#pragma unroll
      for (int kk = 0; kk < TILE / 16; ++kk)  // 16 tokens per instruction = two 8-row groups = 2048 bytes
        mma_bf16(tmem_base + db * HALF, dA + (uint64_t)(kk * 128), dB + (uint64_t)(kk * 128), idesc, kk != 0);
      mma_commit(empty + s);
      mma_commit(dfull + db);
    }
  } else if (warp < 4) {
    const int row = warp * 32 + lane;  // state row i (TMEM lane)
    float acc[HALF];
#pragma unroll
    for (int j = 0; j < HALF; ++j) acc[j] = 0.f;
    for (int it = 0; it < hi - lo; ++it) {
      const int b = prm.reverse ? hi - 1 - it : lo + it, db = it % SCAN_DBUF;
      // state[b] = running sum before this tile (in visiting order)
      uint4* dst = reinterpret_cast<uint4*>(prm.Sin + (((int64_t)bh * prm.NC + b) * TILE + row) * TILE + half * HALF);
#pragma unroll
      for (int j16 = 0; j16 < HALF / 16; ++j16) {   // whole 32-byte sectors
        uint32_t w[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) w[e] = pack_bf16(acc[j16 * 16 + 2 * e], acc[j16 * 16 + 2 * e + 1]);
        st_global_v8(dst + 2 * j16, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]);
      }
      if (it + 1 == hi - lo) break;  // every issued MMA has been consumed: nothing is in flight at teardown
      if (!mbar_wait(dfull + db, (it / SCAN_DBUF) & 1, wc)) break;
      fence_after_sync();
      uint32_t v0[32], v1[32];
      const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + db * HALF;
      tmem_ld32(taddr, v0);
      tmem_ld32(taddr + 32, v1);
      tmem_ld_wait();
      fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(dempty + db);
      float decay = 1.f;
      if (prm.lam) {   // exp(λ_{last token of tile b} - λ_{last token before it})
        const float* lh = prm.lam + (int64_t)bh * prm.T;
        const int64_t t0 = (int64_t)b * TILE;
        decay = __expf(lh[t0 + TILE - 1] - (t0 > 0 ? lh[t0 - 1] : 0.f));
      }
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        acc[j] = fmaf(acc[j], decay, __uint_as_float(v0[j]));
        acc[32 + j] = fmaf(acc[32 + j], decay, __uint_as_float(v1[j]));
      }
    }
  }
  fence_before_sync();
  __syncthreads();
  if (warp == 4) {
    fence_after_sync();
    tmem_dealloc(tmem_base, SCAN_DBUF * HALF);
  }
}

// ---------------------------------------------------------------------------------------------------------------
// tile_product_tc_kernel: one CTA per (tile, head, 64-column half of the output) computes
//
//        Out_b = X · P3_b  +  P4_b · St_b  (+ addend rows),      X = tril(P1_b P2_bᵀ) or its transpose,
//
// which is the forward tile (Eq. "local") and each of the three within-chunk adjoints (Eq. "local-adjoint")
// together with the broadcast of the scanned state adjoint:
//        O_b  = tril(Q Kᵀ)   V  + Q  S_in      P1 = Q,  P2 = K, P3 = V,  P4 = Q  (= P1), St = S_in   as [k = i][n = j]
//        dQ_b = tril(dO Vᵀ)  K  + dO S_inᵀ     P1 = dO, P2 = V, P3 = K,  P4 = dO (= P1), St = S_inᵀ: K-major rows i
//        dK_b = tril(dO Vᵀ)ᵀ Q  + V  D̄ᵀ        P1 = dO, P2 = V, P3 = Q,  P4 = V  (= P2), St = D̄ᵀ  : K-major rows i
//        dV_b = tril(Q Kᵀ)ᵀ  dO + K  D̄         P1 = Q,  P2 = K, P3 = dO, P4 = K  (= P2), St = D̄    as [k = i][n = j]
// All operands are the natural row-major tiles; transposes are expressed through the operand-major bits of the MMA.
//   warp 4 lane 0 : TMA loads (P1, P2: two boxes each; P3[:, half]; state half), then
//        MMA1  Sc = P1 P2ᵀ                                     -> TMEM columns [0, 128)
//        MMA2  Oh = P4 · St half          (M = 128, N = 64)    -> TMEM columns [128, 192)
//        MMA3  Oh += X(ᵀ) · P3[:, half]   (X = masked, rounded Sc, written over the score operand that P4 is not)
//   warps 0-3     : one tile row per thread: mask and round the scores into the swizzled layout, later read Oh,
//                   add the long-range rows and store
// ---------------------------------------------------------------------------------------------------------------
constexpr int OUT_SMEM = 6 * BOX_BYTES + 1024 + 256 + TILE * 4;   // operands, alignment, barriers, the tile's λ (gated)

struct TileParams {
  int64_t T;
  int NC;
  int64_t add_lo, add_hi;  // rows add_lo <= t < add_hi of every head add `addend`
  const float* addend;     // [bh][T][128] fp32, or
  const __nv_bfloat16* addend16;   // the same rows in bf16 (when non-null)
  const float* lam;        // GATED: inclusive prefix sums of the log-gates [bh][T]
  __nv_bfloat16* Out;      // [bh][T][128]
  int* status;
};

// GATED (forward tile only, Lemma "Gated SMat"): the masked scores are multiplied by exp(λ_i - λ_j) before they are
// rounded, and the state product keeps an accumulator of its own so that row i can be scaled by
// exp(λ_i - λ_{last token before the tile}) when the two are added.
template <bool P4_IS_P1, bool XT, bool ST_KMAJOR, bool GATED = false>
__global__ void __launch_bounds__(160) tile_product_tc_kernel(const __grid_constant__ CUtensorMap tm1,
                                                              const __grid_constant__ CUtensorMap tm2,
                                                              const __grid_constant__ CUtensorMap tm3,
                                                              const __grid_constant__ CUtensorMap tmSt,
                                                              const TileParams prm) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* s1 = smem;                    // P1: 2 boxes (K-major, k-blocks 0 and 1)
  uint8_t* s2 = smem + 2 * BOX_BYTES;    // P2: 2 boxes
  uint8_t* s3 = smem + 4 * BOX_BYTES;    // P3 half: 1 box (MN-major B)
  uint8_t* sS = smem + 5 * BOX_BYTES;    // state half: 1 box
  uint8_t* s4 = P4_IS_P1 ? s1 : s2;      // A operand of the state product
  uint8_t* sX = P4_IS_P1 ? s2 : s1;      // the masked scores replace the other score operand
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 6 * BOX_BYTES);
  uint64_t* bar_qk = bars + 0;
  uint64_t* bar_vs = bars + 1;
  uint64_t* bar_sc = bars + 2;   // scores in TMEM
  uint64_t* bar_p = bars + 3;    // X in shared memory (one arrival per warp)
  uint64_t* bar_o = bars + 4;    // output in TMEM
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 5);
  volatile int* cta_abort = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* sLam = reinterpret_cast<float*>(smem + 6 * BOX_BYTES + 256);   // [128] λ of the tile's tokens (GATED)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int half = blockIdx.x & 1, b = blockIdx.x >> 1;
  const int bh = blockIdx.y;
  const int64_t row0 = (int64_t)bh * prm.T + (int64_t)b * TILE;
  const WaitCtx wc{cta_abort, prm.status};
  if (GATED && threadIdx.x < TILE) sLam[threadIdx.x] = prm.lam[row0 + threadIdx.x];

  if (threadIdx.x == 0) {
    *cta_abort = 0;
    mbar_init(bar_qk, 1); mbar_init(bar_vs, 1); mbar_init(bar_sc, 1); mbar_init(bar_p, 4); mbar_init(bar_o, 1);
    fence_barrier_init();
  }
  if (warp == 4) tmem_alloc(tmem_slot, 256);
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_sc = tmem_base, tmem_o = tmem_base + TILE;
  const uint32_t tmem_st = GATED ? tmem_base + TILE + HALF : tmem_o;   // accumulator of the state product

  if (warp == 4 && lane == 0) {
    mbar_expect_tx(bar_qk, 4 * BOX_BYTES);
    tma_load_2d(s1, &tm1, 0, (int)row0, bar_qk);
    tma_load_2d(s1 + BOX_BYTES, &tm1, HALF, (int)row0, bar_qk);
    tma_load_2d(s2, &tm2, 0, (int)row0, bar_qk);
    tma_load_2d(s2 + BOX_BYTES, &tm2, HALF, (int)row0, bar_qk);
    mbar_expect_tx(bar_vs, 2 * BOX_BYTES);
    tma_load_2d(s3, &tm3, half * HALF, (int)row0, bar_vs);
    const int srow = (int)(((int64_t)bh * prm.NC + b) * TILE);
    if (ST_KMAJOR) {  // rows half*64 .. +63 of the state (the output columns), all 128 columns: two 64 x 64 boxes
      tma_load_2d(sS, &tmSt, 0, srow + half * HALF, bar_vs);
      tma_load_2d(sS + BOX_BYTES / 2, &tmSt, HALF, srow + half * HALF, bar_vs);
    } else {          // columns half*64 .. +63 of the state, all 128 rows
      tma_load_2d(sS, &tmSt, half * HALF, srow, bar_vs);
    }

    constexpr uint32_t idesc_sc = make_idesc(TILE, TILE, 0, 0);
    constexpr uint32_t idesc_st = make_idesc(TILE, HALF, 0, ST_KMAJOR ? 0 : 1);
    constexpr uint32_t idesc_x = make_idesc(TILE, HALF, XT ? 1 : 0, 1);
    bool ok = mbar_wait(bar_qk, 0, wc);
    if (ok) {
      fence_after_sync();
#pragma unroll
      for (int kk = 0; kk < TILE / 16; ++kk) {  // k-block kk/4 (16 KB apart), 32 bytes per 16 k-elements inside it
        const uint64_t dA = make_desc(smem_u32(s1) + (kk >> 2) * BOX_BYTES + (kk & 3) * 32, 16, 1024);
        const uint64_t dB = make_desc(smem_u32(s2) + (kk >> 2) * BOX_BYTES + (kk & 3) * 32, 16, 1024);
        mma_bf16(tmem_sc, dA, dB, idesc_sc, kk != 0);
      }
      mma_commit(bar_sc);
      ok = mbar_wait(bar_vs, 0, wc);
    }
    if (ok) {
      fence_after_sync();
#pragma unroll
      for (int kk = 0; kk < TILE / 16; ++kk) {
        const uint64_t dA = make_desc(smem_u32(s4) + (kk >> 2) * BOX_BYTES + (kk & 3) * 32, 16, 1024);
        const uint64_t dB = ST_KMAJOR ? make_desc(smem_u32(sS) + (kk >> 2) * (BOX_BYTES / 2) + (kk & 3) * 32, 16, 1024)
                                      : make_desc(smem_u32(sS) + kk * 2048, BOX_BYTES, 1024);
        mma_bf16(tmem_st, dA, dB, idesc_st, kk != 0);
      }
      ok = mbar_wait(bar_p, 0, wc);
    }
    if (ok) {
      fence_after_sync();
#pragma unroll
      for (int kk = 0; kk < TILE / 16; ++kk) {
        // X is stored [row m][key k], two 64-key blocks.  As it is: K-major A (reduce over keys).  Transposed:
        // MN-major A (rows = reduction index m, 64-key blocks 16 KB apart, 16 rows = 2048 bytes per step).
        const uint64_t dA = XT ? make_desc(smem_u32(sX) + kk * 2048, BOX_BYTES, 1024)
                               : make_desc(smem_u32(sX) + (kk >> 2) * BOX_BYTES + (kk & 3) * 32, 16, 1024);
        const uint64_t dB = make_desc(smem_u32(s3) + kk * 2048, BOX_BYTES, 1024);
        mma_bf16(tmem_o, dA, dB, idesc_x, GATED ? (kk != 0) : 1);
      }
      mma_commit(bar_o);
    }
  } else if (warp < 4) {
    const int m = warp * 32 + lane;  // row inside the tile = TMEM lane
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    if (mbar_wait(bar_sc, 0, wc)) {
      fence_after_sync();
      const float lam_m = GATED ? sLam[m] : 0.f;
#pragma unroll
      for (int cb = 0; cb < 4; ++cb) {
        uint32_t v[32];
        tmem_ld32(tmem_sc + lane_base + cb * 32, v);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 4; ++i) {  // 16-byte chunk = 8 keys
          uint32_t pk[4];
#pragma unroll
          for (int h2 = 0; h2 < 4; ++h2) {
            const int k0 = cb * 32 + i * 8 + h2 * 2;
            float lo = (k0 <= m) ? __uint_as_float(v[i * 8 + h2 * 2]) : 0.f;
            float hi = (k0 + 1 <= m) ? __uint_as_float(v[i * 8 + h2 * 2 + 1]) : 0.f;
            if (GATED) {   // exponents of non-positive differences only: the rows above the diagonal stay zero
              if (k0 <= m) lo *= __expf(lam_m - sLam[k0]);
              if (k0 + 1 <= m) hi *= __expf(lam_m - sLam[k0 + 1]);
            }
            pk[h2] = pack_bf16(lo, hi);
          }
          const int j8 = cb * 4 + i;  // chunk index along the key dimension, 0..15
          uint8_t* dst = sX + (j8 >> 3) * BOX_BYTES + m * 128 + (((j8 & 7) ^ (m & 7)) << 4);
          *reinterpret_cast<uint4*>(dst) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
      }
      fence_proxy_async();
      fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_p);   // one arrival per warp
      if (mbar_wait(bar_o, 0, wc)) {
        fence_after_sync();
        const int64_t t = (int64_t)b * TILE + m;
        const bool add_lr = t >= prm.add_lo && t < prm.add_hi;
        float row_scale = 1.f;   // GATED: exp(λ_i - λ of the last token before the tile)
        if (GATED) row_scale = __expf(lam_m - (b > 0 ? prm.lam[row0 - 1] : 0.f));
        const float4* y4 = reinterpret_cast<const float4*>(prm.addend + ((int64_t)bh * prm.T + t) * TILE + half * HALF);
        const uint4* y16 = reinterpret_cast<const uint4*>(prm.addend16 + ((int64_t)bh * prm.T + t) * TILE + half * HALF);
        uint4* dst = reinterpret_cast<uint4*>(prm.Out + ((int64_t)bh * prm.T + t) * TILE + half * HALF);
#pragma unroll
        for (int cb = 0; cb < 2; ++cb) {
          uint32_t v[32];
          tmem_ld32(tmem_o + lane_base + cb * 32, v);
          tmem_ld_wait();
          if (GATED) {
            uint32_t vs[32];
            tmem_ld32(tmem_st + lane_base + cb * 32, vs);
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 32; ++e) v[e] = __float_as_uint(fmaf(row_scale, __uint_as_float(vs[e]), __uint_as_float(v[e])));
          }
          uint32_t w[16];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            float f[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(v[i * 8 + e]);
            if (add_lr && prm.addend16) {
              const uint4 a = __ldg(y16 + cb * 4 + i);   // 8 bf16 values
              const uint32_t yy[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                f[2 * e] += __uint_as_float(yy[e] << 16);
                f[2 * e + 1] += __uint_as_float(yy[e] & 0xffff0000u);
              }
            } else if (add_lr) {
              const float4 a = __ldg(y4 + cb * 8 + i * 2), c = __ldg(y4 + cb * 8 + i * 2 + 1);
              f[0] += a.x; f[1] += a.y; f[2] += a.z; f[3] += a.w;
              f[4] += c.x; f[5] += c.y; f[6] += c.z; f[7] += c.w;
            }
            w[4 * i] = pack_bf16(f[0], f[1]); w[4 * i + 1] = pack_bf16(f[2], f[3]);
            w[4 * i + 2] = pack_bf16(f[4], f[5]); w[4 * i + 3] = pack_bf16(f[6], f[7]);
          }
#pragma unroll
          for (int h8 = 0; h8 < 2; ++h8)   // whole 32-byte sectors
            st_global_v8(dst + cb * 4 + 2 * h8, w[8 * h8], w[8 * h8 + 1], w[8 * h8 + 2], w[8 * h8 + 3], w[8 * h8 + 4],
                         w[8 * h8 + 5], w[8 * h8 + 6], w[8 * h8 + 7]);
        }
      }
    }
  }
  fence_before_sync();
  __syncthreads();
  if (warp == 4) {
    fence_after_sync();
    tmem_dealloc(tmem_base, 256);
  }
}

// ---------------------------------------------------------------------------------------------------------------
// bwd_tile_fused_tc_kernel: the three within-chunk adjoints of one 128-token tile in ONE CTA (Eq. "local-adjoint"
// with the broadcast of the scanned state adjoint), all 128 output columns:
//        G = tril(dO Vᵀ),  A = tril(Q Kᵀ)
//        dQ = dO S_inᵀ + G K,      dK = V D̄ᵀ + Gᵀ Q,      dV = K D̄ + Aᵀ dO      (+ the long-range rows of each)
// Q, K, V, dO, S_in and D̄ of the tile are loaded once (the three separate tile kernels load 2.7 times as much) and
// the two score tiles are formed once.  Shared memory: seven 32 KB tiles (Q, K, V, dO, S_in, D̄, X); tensor memory:
// scores [0,128), dQ [128,256), dK [256,384), dV [384,512).
//   warp 4 lane 0 : TMA loads (dO, V first: the G scores need nothing else), then every MMA in order
//   warps 0-3     : one tile row per thread: mask and round G, later A, into the swizzled X tile; read the three
//                   accumulators, add the long-range rows and store
// ---------------------------------------------------------------------------------------------------------------
constexpr int FUSED_SMEM = 14 * BOX_BYTES + 1024 + 256 + TILE * 4;   // tiles, alignment, barriers, the tile's λ (gated)

struct FusedParams {
  int64_t T;
  int NC;
  int64_t n;                         // rows t >= n add lr_q to dQ; rows t < n add lr_k, lr_v to dK, dV (when non-null)
  const __nv_bfloat16 *lr_q, *lr_k, *lr_v;   // [bh][T][128] bf16
  const float* lam;                  // GATED: inclusive prefix sums of the log-gates [bh][T]
  __nv_bfloat16 *dQ, *dK, *dV;       // [bh][T][128]
  int* status;
};

// GATED (Lemma "Gated SMat", adjoint side): both score tiles are multiplied by exp(λ_i - λ_j) as they are rounded, and
// the three state products are scaled row by row in tensor memory before the score products are added to them — row i
// of dO S_inᵀ by exp(λ_i - λ_{last token before the tile}), row j of V D̄ᵀ and of K D̄ by exp(λ_{last token of the
// tile} - λ_j).  S_in and D̄ are the decayed per-tile states.
template <bool GATED>
__global__ void __launch_bounds__(160) bwd_tile_fused_tc_kernel(const __grid_constant__ CUtensorMap tmQ,
                                                                const __grid_constant__ CUtensorMap tmK,
                                                                const __grid_constant__ CUtensorMap tmV,
                                                                const __grid_constant__ CUtensorMap tmG,
                                                                const __grid_constant__ CUtensorMap tmSin,
                                                                const __grid_constant__ CUtensorMap tmDb,
                                                                const FusedParams prm) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* sQ = smem;
  uint8_t* sK = smem + 2 * BOX_BYTES;
  uint8_t* sV = smem + 4 * BOX_BYTES;
  uint8_t* sG = smem + 6 * BOX_BYTES;      // dO
  uint8_t* sS = smem + 8 * BOX_BYTES;      // S_in of the tile
  uint8_t* sD = smem + 10 * BOX_BYTES;     // D̄ of the tile
  uint8_t* sX = smem + 12 * BOX_BYTES;     // masked, rounded score tile (G, then A)
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 14 * BOX_BYTES);
  uint64_t* bar_in0 = bars + 0;   // dO, V landed
  uint64_t* bar_in1 = bars + 1;   // Q, K, S_in, D̄ landed
  uint64_t* bar_sc = bars + 2;    // a score tile is in tensor memory (two phases: G, then A)
  uint64_t* bar_p = bars + 3;     // X written (one arrival per warp; two phases)
  uint64_t* bar_x = bars + 4;     // the MMAs that read X = G have finished: dQ, dK complete, X may be overwritten
  uint64_t* bar_o = bars + 5;     // dV complete
  uint64_t* bar_st = bars + 6;    // GATED: the three state products are in tensor memory
  uint64_t* bar_sl = bars + 7;    // GATED: ... and scaled (one arrival per warp)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 8);
  volatile int* cta_abort = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* sLam = reinterpret_cast<float*>(smem + 14 * BOX_BYTES + 256);   // [128] λ of the tile's tokens (GATED)
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.x, bh = blockIdx.y;
  const int64_t row0 = (int64_t)bh * prm.T + (int64_t)b * TILE;
  const WaitCtx wc{cta_abort, prm.status};
  if (GATED && threadIdx.x < TILE) sLam[threadIdx.x] = prm.lam[row0 + threadIdx.x];
  if (threadIdx.x == 0) {
    *cta_abort = 0;
    mbar_init(bar_in0, 1); mbar_init(bar_in1, 1); mbar_init(bar_sc, 1); mbar_init(bar_p, 4); mbar_init(bar_x, 1);
    mbar_init(bar_o, 1); mbar_init(bar_st, 1); mbar_init(bar_sl, 4);
    fence_barrier_init();
  }
  if (warp == 4) tmem_alloc(tmem_slot, 512);
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tm_sc = tmem_base, tm_dq = tmem_base + TILE, tm_dk = tmem_base + 2 * TILE, tm_dv = tmem_base + 3 * TILE;

  if (warp == 4 && lane == 0) {
    auto load_tile = [&](uint8_t* dst, const CUtensorMap* map, int row, uint64_t* bar) {
      tma_load_2d(dst, map, 0, row, bar);
      tma_load_2d(dst + BOX_BYTES, map, HALF, row, bar);
    };
    mbar_expect_tx(bar_in0, 4 * BOX_BYTES);
    load_tile(sG, &tmG, (int)row0, bar_in0);
    load_tile(sV, &tmV, (int)row0, bar_in0);
    mbar_expect_tx(bar_in1, 8 * BOX_BYTES);
    load_tile(sQ, &tmQ, (int)row0, bar_in1);
    load_tile(sK, &tmK, (int)row0, bar_in1);
    const int srow = (int)(((int64_t)bh * prm.NC + b) * TILE);
    load_tile(sS, &tmSin, srow, bar_in1);
    load_tile(sD, &tmDb, srow, bar_in1);

    constexpr uint32_t id_kk = make_idesc(TILE, TILE, 0, 0);   // A K-major, B K-major
    constexpr uint32_t id_km = make_idesc(TILE, TILE, 0, 1);   // A K-major, B MN-major
    constexpr uint32_t id_mm = make_idesc(TILE, TILE, 1, 1);   // A MN-major, B MN-major
    // K-major view of a [128 rows][128 k] tile (two 64-wide k blocks 16 KB apart), K-step kk; MN-major view of a
    // [128 k rows][128 n] tile (16 rows = 2048 bytes per K-step, the two 64-wide n blocks 16 KB apart)
    auto kmaj = [](const uint8_t* t, int kk) { return make_desc(smem_u32(t) + (kk >> 2) * BOX_BYTES + (kk & 3) * 32, 16, 1024); };
    auto mnmaj = [](const uint8_t* t, int kk) { return make_desc(smem_u32(t) + kk * 2048, BOX_BYTES, 1024); };
    bool ok = mbar_wait(bar_in0, 0, wc);
    if (ok) {
      fence_after_sync();
#pragma unroll
      for (int kk = 0; kk < TILE / 16; ++kk) mma_bf16(tm_sc, kmaj(sG, kk), kmaj(sV, kk), id_kk, kk != 0);   // dO Vᵀ
      mma_commit(bar_sc);
      ok = mbar_wait(bar_in1, 0, wc);
    }
    if (ok) {
      fence_after_sync();
#pragma unroll
      for (int kk = 0; kk < TILE / 16; ++kk) mma_bf16(tm_dq, kmaj(sG, kk), kmaj(sS, kk), id_kk, kk != 0);   // dO S_inᵀ
#pragma unroll
      for (int kk = 0; kk < TILE / 16; ++kk) mma_bf16(tm_dk, kmaj(sV, kk), kmaj(sD, kk), id_kk, kk != 0);   // V D̄ᵀ
#pragma unroll
      for (int kk = 0; kk < TILE / 16; ++kk) mma_bf16(tm_dv, kmaj(sK, kk), mnmaj(sD, kk), id_km, kk != 0);  // K D̄
      if (GATED) mma_commit(bar_st);
      ok = mbar_wait(bar_p, 0, wc);          // X = G in shared memory; the G scores have left tensor memory
      if (GATED && ok) ok = mbar_wait(bar_sl, 0, wc);   // the state products carry their row factors
    }
    if (ok) {
      fence_after_sync();
#pragma unroll
      for (int kk = 0; kk < TILE / 16; ++kk) mma_bf16(tm_dq, kmaj(sX, kk), mnmaj(sK, kk), id_km, 1);        // G K
#pragma unroll
      for (int kk = 0; kk < TILE / 16; ++kk) mma_bf16(tm_dk, mnmaj(sX, kk), mnmaj(sQ, kk), id_mm, 1);       // Gᵀ Q
      mma_commit(bar_x);
#pragma unroll
      for (int kk = 0; kk < TILE / 16; ++kk) mma_bf16(tm_sc, kmaj(sQ, kk), kmaj(sK, kk), id_kk, kk != 0);   // Q Kᵀ
      mma_commit(bar_sc);
      ok = mbar_wait(bar_p, 1, wc);          // X = A
    }
    if (ok) {
      fence_after_sync();
#pragma unroll
      for (int kk = 0; kk < TILE / 16; ++kk) mma_bf16(tm_dv, mnmaj(sX, kk), mnmaj(sG, kk), id_mm, 1);       // Aᵀ dO
      mma_commit(bar_o);
    }
  } else if (warp < 4) {
    const int m = warp * 32 + lane;  // row inside the tile = TMEM lane
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    const float lam_m = GATED ? sLam[m] : 0.f;
    // masked (column <= row), rounded copy of the score tile into X, swizzled as a K-major operand
    auto stage_scores = [&]() {
#pragma unroll
      for (int cb = 0; cb < 4; ++cb) {
        uint32_t v[32];
        tmem_ld32(tm_sc + lane_base + cb * 32, v);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          uint32_t pk[4];
#pragma unroll
          for (int h2 = 0; h2 < 4; ++h2) {
            const int k0 = cb * 32 + i * 8 + h2 * 2;
            float lo = (k0 <= m) ? __uint_as_float(v[i * 8 + h2 * 2]) : 0.f;
            float hi = (k0 + 1 <= m) ? __uint_as_float(v[i * 8 + h2 * 2 + 1]) : 0.f;
            if (GATED) {   // exponents of non-positive differences only
              if (k0 <= m) lo *= __expf(lam_m - sLam[k0]);
              if (k0 + 1 <= m) hi *= __expf(lam_m - sLam[k0 + 1]);
            }
            pk[h2] = pack_bf16(lo, hi);
          }
          const int j8 = cb * 4 + i;
          uint8_t* dst = sX + (j8 >> 3) * BOX_BYTES + m * 128 + (((j8 & 7) ^ (m & 7)) << 4);
          *reinterpret_cast<uint4*>(dst) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
      }
      fence_proxy_async();
      fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_p);
    };
    // one accumulator row (128 columns) plus its long-range row, rounded and stored
    const int64_t t = (int64_t)b * TILE + m;
    auto store_row = [&](uint32_t tm_acc, const __nv_bfloat16* lr, bool add, __nv_bfloat16* out) {
      const uint4* y16 = reinterpret_cast<const uint4*>(lr + ((int64_t)bh * prm.T + t) * TILE);
      __nv_bfloat16* dst = out + ((int64_t)bh * prm.T + t) * TILE;
#pragma unroll
      for (int cb = 0; cb < 4; ++cb) {
        uint32_t v[32];
        tmem_ld32(tm_acc + lane_base + cb * 32, v);
        tmem_ld_wait();
        uint32_t w[16];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          float f[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(v[i * 8 + e]);
          if (add) {
            const uint4 a = __ldg(y16 + cb * 4 + i);
            const uint32_t yy[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              f[2 * e] += __uint_as_float(yy[e] << 16);
              f[2 * e + 1] += __uint_as_float(yy[e] & 0xffff0000u);
            }
          }
          w[4 * i] = pack_bf16(f[0], f[1]); w[4 * i + 1] = pack_bf16(f[2], f[3]);
          w[4 * i + 2] = pack_bf16(f[4], f[5]); w[4 * i + 3] = pack_bf16(f[6], f[7]);
        }
#pragma unroll
        for (int h8 = 0; h8 < 2; ++h8)
          st_global_v8(dst + cb * 32 + 16 * h8, w[8 * h8], w[8 * h8 + 1], w[8 * h8 + 2], w[8 * h8 + 3], w[8 * h8 + 4],
                       w[8 * h8 + 5], w[8 * h8 + 6], w[8 * h8 + 7]);
      }
    };
    // GATED: one accumulator's rows times this row's factor, in place
    auto scale_rows = [&](uint32_t tm_acc, float f) {
#pragma unroll
      for (int cb = 0; cb < 4; ++cb) {
        uint32_t v[32];
        tmem_ld32(tm_acc + lane_base + cb * 32, v);
        tmem_ld_wait();
#pragma unroll
        for (int e = 0; e < 32; ++e) v[e] = __float_as_uint(__uint_as_float(v[e]) * f);
        tmem_st32(tm_acc + lane_base + cb * 32, v);
      }
    };
    bool ok = mbar_wait(bar_sc, 0, wc);
    if (ok) {
      fence_after_sync();
      stage_scores();                              // X = G
      if (GATED) {
        ok = mbar_wait(bar_st, 0, wc);
        if (ok) {
          fence_after_sync();
          const float row_in = __expf(lam_m - (b > 0 ? prm.lam[row0 - 1] : 0.f));   // queries' side: from the tile's start
          const float row_out = __expf(sLam[TILE - 1] - lam_m);                       // keys' side: to the tile's end
          scale_rows(tm_dq, row_in);
          scale_rows(tm_dk, row_out);
          scale_rows(tm_dv, row_out);
          tmem_st_wait();
          fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_sl);
        }
      }
      if (ok) ok = mbar_wait(bar_sc, 1, wc);       // the A scores are in (the MMAs on G were issued before them)
    }
    if (ok) ok = mbar_wait(bar_x, 0, wc);          // ... and those MMAs have finished with X: dQ, dK are complete
    if (ok) {
      fence_after_sync();
      stage_scores();                              // X = A
      store_row(tm_dq, prm.lr_q, prm.lr_q != nullptr && t >= prm.n, prm.dQ);
      store_row(tm_dk, prm.lr_k, prm.lr_k != nullptr && t < prm.n, prm.dK);
      ok = mbar_wait(bar_o, 0, wc);
    }
    if (ok) {
      fence_after_sync();
      store_row(tm_dv, prm.lr_v, prm.lr_v != nullptr && t < prm.n, prm.dV);
    }
  }
  fence_before_sync();
  __syncthreads();
  if (warp == 4) {
    fence_after_sync();
    tmem_dealloc(tmem_base, 512);
  }
}

// ---------------------------------------------------------------------------------------------------------------
// Two-level form of the causal branch.  Each block of the sequence is cut into segments of L tiles.
//   segment_state_tc_kernel  : total[seg] = Σ_{tiles of the segment} K_bᵀ V_b, accumulated in TMEM (fp32), written once
//   (scan_kernel turns the totals into the state entering each segment: exclusive prefix sum per block, fp32)
//   segment_output_tc_kernel : one CTA per (segment, head) walks its L tiles with the running state
//                              S in TMEM:  O_b = Q_b S + tril(Q_b K_bᵀ) V_b + Y_lr,b ;  S += K_bᵀ V_b
// Against the per-tile form (chunk_scan + chunk_output) this writes and reads one fp32 state per segment instead of
// one bf16 state per tile, at the price of reading K and V a second time.
// ---------------------------------------------------------------------------------------------------------------
constexpr int SEG_STATE_STAGES = 3;
constexpr int SEG_STATE_SMEM = SEG_STATE_STAGES * 4 * BOX_BYTES + 1024 + 256;

// Segments of the two-level causal branch: block 0 (tiles0 tiles) is cut into nseg0 segments, block 1 into
// nseg - nseg0, as evenly as whole tiles allow (lengths differ by at most one tile), so that the segment count can
// be matched to the number of SMs.  Segment `seg` covers tiles [*tile0, *tile0 + *count).
struct SegCut {
  int nseg0, nseg;
  int64_t tiles0, tiles1;
};
__device__ __forceinline__ void seg_range(const SegCut& c, int seg, int64_t* tile0, int* count) {
  if (seg < c.nseg0) {
    const int64_t a = (int64_t)seg * c.tiles0 / c.nseg0, b = (int64_t)(seg + 1) * c.tiles0 / c.nseg0;
    *tile0 = a; *count = (int)(b - a);
  } else {
    const int s = seg - c.nseg0, n1 = c.nseg - c.nseg0;
    const int64_t a = (int64_t)s * c.tiles1 / n1, b = (int64_t)(s + 1) * c.tiles1 / n1;
    *tile0 = c.tiles0 + a; *count = (int)(b - a);
  }
}

struct SegStateParams {
  int64_t T;
  SegCut cut;
  int nseg;              // segments per head
  float* totals;         // [bh][nseg][128][128]
  int* status;
};

__global__ void __launch_bounds__(192) segment_state_tc_kernel(const __grid_constant__ CUtensorMap tmK,
                                                               const __grid_constant__ CUtensorMap tmV,
                                                               const SegStateParams prm) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SEG_STATE_STAGES * 4 * BOX_BYTES);
  uint64_t* full = bars;
  uint64_t* empty = bars + SEG_STATE_STAGES;
  uint64_t* done = empty + SEG_STATE_STAGES;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(done + 1);
  volatile int* cta_abort = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int seg = blockIdx.x, bh = blockIdx.y;
  // The scan is exclusive: nobody reads the total of a block's last segment (the scan loads it after its last store).
  if (seg == prm.cut.nseg0 - 1 || seg == prm.cut.nseg - 1) return;
  int64_t tile0;
  int Lc;
  seg_range(prm.cut, seg, &tile0, &Lc);
  const WaitCtx wc{cta_abort, prm.status};
  if (threadIdx.x == 0) {
    *cta_abort = 0;
    for (int s = 0; s < SEG_STATE_STAGES; ++s) { mbar_init(full + s, 1); mbar_init(empty + s, 1); }
    mbar_init(done, 1);
    fence_barrier_init();
  }
  if (warp == 4) tmem_alloc(tmem_slot, TILE);
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem_d = *tmem_slot;
  if (warp == 4 && lane == 0) {
    for (int it = 0; it < Lc; ++it) {
      const int s = it % SEG_STATE_STAGES;
      if (it >= SEG_STATE_STAGES && !mbar_wait(empty + s, ((it / SEG_STATE_STAGES) - 1) & 1, wc)) break;
      uint8_t* st = smem + s * 4 * BOX_BYTES;
      const int row = (int)((int64_t)bh * prm.T + (tile0 + it) * TILE);
      mbar_expect_tx(full + s, 4 * BOX_BYTES);
      tma_load_2d(st, &tmK, 0, row, full + s);
      tma_load_2d(st + BOX_BYTES, &tmK, HALF, row, full + s);
      tma_load_2d(st + 2 * BOX_BYTES, &tmV, 0, row, full + s);
      tma_load_2d(st + 3 * BOX_BYTES, &tmV, HALF, row, full + s);
    }
  } else if (warp == 5 && lane == 0) {
    constexpr uint32_t idesc = make_idesc(TILE, TILE, 1, 1);
    bool ok = true;
    for (int it = 0; it < Lc && ok; ++it) {
      const int s = it % SEG_STATE_STAGES;
      ok = mbar_wait(full + s, (it / SEG_STATE_STAGES) & 1, wc);
      if (!ok) break;
      fence_after_sync();
      const uint32_t sK = smem_u32(smem + s * 4 * BOX_BYTES);
      const uint64_t dA = make_desc(sK, BOX_BYTES, 1024);
      const uint64_t dB = make_desc(sK + 2 * BOX_BYTES, BOX_BYTES, 1024);
#pragma unroll
      for (int kk = 0; kk < TILE / 16; ++kk)
        mma_bf16(tmem_d, dA + (uint64_t)(kk * 128), dB + (uint64_t)(kk * 128), idesc, (it | kk) != 0);
      mma_commit(empty + s);
    }
    if (ok) mma_commit(done);
  } else if (warp < 4) {
    if (mbar_wait(done, 0, wc)) {
      fence_after_sync();
      const int i = warp * 32 + lane;
      uint4* dst = reinterpret_cast<uint4*>(prm.totals + (((int64_t)bh * prm.nseg + seg) * TILE + i) * TILE);
#pragma unroll
      for (int cb = 0; cb < 4; ++cb) {
        uint32_t v[32];
        tmem_ld32(tmem_d + ((uint32_t)(warp * 32) << 16) + cb * 32, v);
        tmem_ld_wait();
#pragma unroll
        for (int q8 = 0; q8 < 4; ++q8)   // whole 32-byte sectors
          st_global_v8(dst + cb * 8 + 2 * q8, v[8 * q8], v[8 * q8 + 1], v[8 * q8 + 2], v[8 * q8 + 3], v[8 * q8 + 4], v[8 * q8 + 5],
                       v[8 * q8 + 6], v[8 * q8 + 7]);
      }
    }
  }
  fence_before_sync();
  __syncthreads();
  if (warp == 4) {
    fence_after_sync();
    tmem_dealloc(tmem_d, TILE);
  }
}

// Shared memory of segment_output_tc_kernel: two stages of (Q, K, V: two boxes each) and one 32 KB tile that holds the
// bf16 copy of the running state while O = Q S is formed and the rounded score tile P afterwards.
constexpr int SEG_OUT_STAGE = 6 * BOX_BYTES;
constexpr int SEG_OUT_SMEM = 2 * SEG_OUT_STAGE + 2 * BOX_BYTES + 1024 + 256;

struct SegOutParams {
  int64_t T;
  SegCut cut;
  int nseg;
  const float* seg_in;   // [bh][nseg][128][128] state entering each segment
  int64_t n_lr;
  const __nv_bfloat16* ylr;   // [bh][T][128] long-range rows, bf16 (rows t >= n_lr are added)
  __nv_bfloat16* O;
  __nv_bfloat16* sin_tiles;   // optional [bh][T/128][128][128]: the bf16 state entering every tile, for a later backward
  int* status;
};

// One CTA per (segment, head), all 128 output columns.
//   warps 0-15 : each owns 32 rows x 32 columns of every TMEM tile (state, scores, output)
//   warp 16    : TMA producer (two stages);   warp 17 : MMA issuer
// TMEM columns: running state S [0,128), scores [128,256), two output accumulators [256,384) and [384,512).
// Per tile:  Sc = Q Kᵀ ;  O = Q S_bf16 ;  O += tril(Sc)_bf16 V ;  S += Kᵀ V.
constexpr int SEG_EPI_WARPS = 16;
constexpr int SEG_OUT_THREADS = 32 * (SEG_EPI_WARPS + 2);

__global__ void __launch_bounds__(SEG_OUT_THREADS) segment_output_tc_kernel(const __grid_constant__ CUtensorMap tmQ,
                                                                const __grid_constant__ CUtensorMap tmK,
                                                                const __grid_constant__ CUtensorMap tmV,
                                                                const SegOutParams prm) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* sSP = smem + 2 * SEG_OUT_STAGE;           // 128 x 128 bf16, two 64-column blocks: S_bf16, then P
  uint64_t* bars = reinterpret_cast<uint64_t*>(sSP + 2 * BOX_BYTES);
  uint64_t* full = bars;          // [2] tile operands landed
  uint64_t* empty = bars + 2;     // [2] tile operands consumed
  uint64_t* bar_s = bars + 4;     // bf16 state written (one arrival per warp)
  uint64_t* bar_sc = bars + 5;    // scores in TMEM
  uint64_t* bar_qs = bars + 6;    // O = Q S finished: the shared tile may take P
  uint64_t* bar_p = bars + 7;     // P written (one arrival per warp)
  uint64_t* bar_o = bars + 8;     // output in TMEM and state updated
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 9);
  volatile int* cta_abort = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int seg = blockIdx.x, bh = blockIdx.y;
  int64_t tile0;
  int Lc;
  seg_range(prm.cut, seg, &tile0, &Lc);
  const WaitCtx wc{cta_abort, prm.status};
  if (threadIdx.x == 0) {
    *cta_abort = 0;
    mbar_init(full, 1); mbar_init(full + 1, 1); mbar_init(empty, 1); mbar_init(empty + 1, 1);
    mbar_init(bar_s, SEG_EPI_WARPS); mbar_init(bar_sc, 1); mbar_init(bar_qs, 1); mbar_init(bar_p, SEG_EPI_WARPS);
    mbar_init(bar_o, 1);
    fence_barrier_init();
  }
  if (warp == SEG_EPI_WARPS) tmem_alloc(tmem_slot, 512);
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_s = tmem_base, tmem_sc = tmem_base + TILE, tmem_o0 = tmem_base + 2 * TILE;

  if (warp == SEG_EPI_WARPS && lane == 0) {
    for (int it = 0; it < Lc; ++it) {
      const int s = it & 1;
      if (it >= 2 && !mbar_wait(empty + s, ((it >> 1) - 1) & 1, wc)) break;
      uint8_t* st = smem + s * SEG_OUT_STAGE;
      const int row = (int)((int64_t)bh * prm.T + (tile0 + it) * TILE);
      mbar_expect_tx(full + s, SEG_OUT_STAGE);
      tma_load_2d(st, &tmQ, 0, row, full + s);
      tma_load_2d(st + BOX_BYTES, &tmQ, HALF, row, full + s);
      tma_load_2d(st + 2 * BOX_BYTES, &tmK, 0, row, full + s);
      tma_load_2d(st + 3 * BOX_BYTES, &tmK, HALF, row, full + s);
      tma_load_2d(st + 4 * BOX_BYTES, &tmV, 0, row, full + s);
      tma_load_2d(st + 5 * BOX_BYTES, &tmV, HALF, row, full + s);
    }
  } else if (warp == SEG_EPI_WARPS + 1 && lane == 0) {
    constexpr uint32_t idesc_sc = make_idesc(TILE, TILE, 0, 0);   // Q Kᵀ: both K-major
    constexpr uint32_t idesc_o = make_idesc(TILE, TILE, 0, 1);    // A K-major (Q or P), B MN-major (S or V)
    constexpr uint32_t idesc_s = make_idesc(TILE, TILE, 1, 1);    // Kᵀ V: both MN-major
    // Descriptors are built once; inside the loops only constants are added (16-byte units): this lone thread pays
    // the full latency of every instruction it issues.
    constexpr uint32_t BOX16 = BOX_BYTES >> 4;
    const uint64_t dSP_k = make_desc(smem_u32(sSP), 16, 1024);           // shared tile read K-major (P)
    const uint64_t dSP_mn = make_desc(smem_u32(sSP), BOX_BYTES, 1024);   // and MN-major (S)
    uint64_t dQ_k[2], dK_k[2], dK_mn[2], dV_mn[2];
#pragma unroll
    for (int s = 0; s < 2; ++s) {
      const uint32_t sQ = smem_u32(smem + s * SEG_OUT_STAGE);
      dQ_k[s] = make_desc(sQ, 16, 1024);
      dK_k[s] = make_desc(sQ + 2 * BOX_BYTES, 16, 1024);
      dK_mn[s] = make_desc(sQ + 2 * BOX_BYTES, BOX_BYTES, 1024);
      dV_mn[s] = make_desc(sQ + 4 * BOX_BYTES, BOX_BYTES, 1024);
    }
    for (int it = 0; it < Lc; ++it) {
      const int s = it & 1;
      const uint64_t qk = s ? dQ_k[1] : dQ_k[0], kk_ = s ? dK_k[1] : dK_k[0];
      const uint64_t kmn = s ? dK_mn[1] : dK_mn[0], vmn = s ? dV_mn[1] : dV_mn[0];
      const uint32_t tmem_o = tmem_o0 + (it & 1) * TILE;
      if (!mbar_wait(full + s, (it >> 1) & 1, wc)) break;
      fence_after_sync();
#pragma unroll
      for (int kk = 0; kk < TILE / 16; ++kk) {   // Sc = Q Kᵀ (the score tile was read out before bar_p of the last tile)
        const uint64_t off = (uint64_t)((kk >> 2) * BOX16 + (kk & 3) * 2);
        mma_bf16(tmem_sc, qk + off, kk_ + off, idesc_sc, kk != 0);
      }
      mma_commit(bar_sc);
      if (!mbar_wait(bar_s, it & 1, wc)) break;  // bf16 state in the shared tile; output buffer of tile it-2 read out
      fence_after_sync();
#pragma unroll
      for (int kk = 0; kk < TILE / 16; ++kk)     // O = Q S
        mma_bf16(tmem_o, qk + (uint64_t)((kk >> 2) * BOX16 + (kk & 3) * 2), dSP_mn + (uint64_t)(kk * 128), idesc_o, kk != 0);
      mma_commit(bar_qs);
      if (!mbar_wait(bar_p, it & 1, wc)) break;
      fence_after_sync();
#pragma unroll
      for (int kk = 0; kk < TILE / 16; ++kk)     // O += P V
        mma_bf16(tmem_o, dSP_k + (uint64_t)((kk >> 2) * BOX16 + (kk & 3) * 2), vmn + (uint64_t)(kk * 128), idesc_o, 1);
#pragma unroll
      for (int kk = 0; kk < TILE / 16; ++kk)     // S += Kᵀ V
        mma_bf16(tmem_s, kmn + (uint64_t)(kk * 128), vmn + (uint64_t)(kk * 128), idesc_s, 1);
      mma_commit(bar_o);
      mma_commit(empty + s);
    }
  } else if (warp < SEG_EPI_WARPS) {
    // Sixteen warps: warp w owns the lane quarter w % 4 (32 rows) and the column quarter w / 4 (32 columns) of every
    // TMEM tile.  The per-tile work of these threads (convert, store, publish, write out) is the critical path of
    // the kernel, so it is spread as widely as the TMEM lane rule allows.
    const int cq = warp >> 2;                        // column quarter
    const int m = (warp & 3) * 32 + lane;            // TMEM lane: state row i / query row of the tile
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t col0 = cq * 32;
    // this thread's 64 bytes (four 16-byte chunks) of its row in the 64-column block that holds its columns
    uint8_t* my_tile = sSP + (cq >> 1) * BOX_BYTES + m * 128;
    const int ch0 = (cq & 1) * 4;
    auto store_row = [&](const uint4 (&pk)[4]) {
#pragma unroll
      for (int c = 0; c < 4; ++c) *reinterpret_cast<uint4*>(my_tile + (((ch0 + c) ^ (m & 7)) << 4)) = pk[c];
    };
    // bf16 copy of this thread's 32 state columns into the shared tile (and, when a backward will want the state
    // entering tile `tile`, into the per-tile table as well: 64 bytes of row m)
    auto publish_state = [&](const uint32_t (&v)[32], int64_t tile) {
      uint4 pk[4];
#pragma unroll
      for (int c = 0; c < 4; ++c)
        pk[c] = make_uint4(pack_bf16(__uint_as_float(v[8 * c]), __uint_as_float(v[8 * c + 1])),
                           pack_bf16(__uint_as_float(v[8 * c + 2]), __uint_as_float(v[8 * c + 3])),
                           pack_bf16(__uint_as_float(v[8 * c + 4]), __uint_as_float(v[8 * c + 5])),
                           pack_bf16(__uint_as_float(v[8 * c + 6]), __uint_as_float(v[8 * c + 7])));
      store_row(pk);
      if (prm.sin_tiles) {
        __nv_bfloat16* dst = prm.sin_tiles + (((int64_t)bh * (prm.T / TILE) + tile) * TILE + m) * TILE + col0;
        st_global_v8(dst, pk[0].x, pk[0].y, pk[0].z, pk[0].w, pk[1].x, pk[1].y, pk[1].z, pk[1].w);
        st_global_v8(dst + 16, pk[2].x, pk[2].y, pk[2].z, pk[2].w, pk[3].x, pk[3].y, pk[3].z, pk[3].w);
      }
      fence_proxy_async();
      fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_s);   // one arrival per warp: 512 arrivals on one barrier serialise
    };
    {  // state entering the segment: global fp32 -> TMEM (accumulator) and the shared tile
      uint32_t v[32];
      const uint4* src = reinterpret_cast<const uint4*>(prm.seg_in + (((int64_t)bh * prm.nseg + seg) * TILE + m) * TILE + col0);
#pragma unroll
      for (int q4 = 0; q4 < 8; ++q4) {
        const uint4 a = __ldg(src + q4);
        v[4 * q4] = a.x; v[4 * q4 + 1] = a.y; v[4 * q4 + 2] = a.z; v[4 * q4 + 3] = a.w;
      }
      tmem_st32(tmem_s + lane_base + col0, v);
      tmem_st_wait();
      publish_state(v, tile0);
    }
    for (int it = 0; it < Lc; ++it) {
      // --- scores of this tile -> masked bf16 P (registers), stored once O = Q S has consumed the shared tile ---
      if (!mbar_wait(bar_sc, it & 1, wc)) break;
      fence_after_sync();
      uint4 pk[4];
      {
        uint32_t v[32];
        tmem_ld32(tmem_sc + lane_base + col0, v);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          uint32_t w[4];
#pragma unroll
          for (int h2 = 0; h2 < 4; ++h2) {
            const int k0 = (int)col0 + i * 8 + h2 * 2;
            const float lo = (k0 <= m) ? __uint_as_float(v[i * 8 + h2 * 2]) : 0.f;
            const float hi = (k0 + 1 <= m) ? __uint_as_float(v[i * 8 + h2 * 2 + 1]) : 0.f;
            w[h2] = pack_bf16(lo, hi);
          }
          pk[i] = make_uint4(w[0], w[1], w[2], w[3]);
        }
      }
      if (!mbar_wait(bar_qs, it & 1, wc)) break;
      store_row(pk);
      fence_proxy_async();
      fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_p);
      // --- long-range rows of this tile, fetched while the MMAs run ---
      const int64_t t = (tile0 + it) * TILE + m;
      const bool add_lr = t >= prm.n_lr;
      uint4 y[4];                                    // 32 bf16 values
      if (add_lr) {
        const uint4* y4 = reinterpret_cast<const uint4*>(prm.ylr + ((int64_t)bh * prm.T + t) * TILE + col0);
#pragma unroll
        for (int i = 0; i < 4; ++i) y[i] = __ldg(y4 + i);
      }
      if (!mbar_wait(bar_o, it & 1, wc)) break;
      fence_after_sync();
      if (it + 1 < Lc) {  // the state now includes this tile: publish it for the next one first (critical path)
        uint32_t v[32];
        tmem_ld32(tmem_s + lane_base + col0, v);
        tmem_ld_wait();
        publish_state(v, tile0 + it + 1);
      }
      __nv_bfloat16* dst = prm.O + ((int64_t)bh * prm.T + t) * TILE + col0;
      const uint32_t tmem_o = tmem_o0 + (it & 1) * TILE;
      uint32_t v[32];
      tmem_ld32(tmem_o + lane_base + col0, v);
      tmem_ld_wait();
      uint32_t w[16];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        float f[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(v[i * 8 + e]);
        if (add_lr) {
          const uint32_t yy[4] = {y[i].x, y[i].y, y[i].z, y[i].w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            f[2 * e] += __uint_as_float(yy[e] << 16);
            f[2 * e + 1] += __uint_as_float(yy[e] & 0xffff0000u);
          }
        }
        w[4 * i] = pack_bf16(f[0], f[1]); w[4 * i + 1] = pack_bf16(f[2], f[3]);
        w[4 * i + 2] = pack_bf16(f[4], f[5]); w[4 * i + 3] = pack_bf16(f[6], f[7]);
      }
#pragma unroll
      for (int h8 = 0; h8 < 2; ++h8)   // whole 32-byte sectors
        st_global_v8(dst + 16 * h8, w[8 * h8], w[8 * h8 + 1], w[8 * h8 + 2], w[8 * h8 + 3], w[8 * h8 + 4],
                     w[8 * h8 + 5], w[8 * h8 + 6], w[8 * h8 + 7]);
    }
  }
  fence_before_sync();
  __syncthreads();
  if (warp == SEG_EPI_WARPS) {
    fence_after_sync();
    tmem_dealloc(tmem_base, 512);
  }
}

// ---------------------------------------------------------------------------------------------------------------
// state_read_tc_kernel: typed read Y_lr[t] = q_tᵀ U_type(t) (Algorithm 1, step 4) for plans whose type table is
// kept in bf16.  Persistent CTAs (three per SM), one (type, head) item at a time:
//   warp 4 lane 0 : TMA load of the 128 x 128 bf16 state (two boxes, MN-major B operand), then the MMA
//                   Y = Q_h U_h   (M = up to 128 queries of the type, N = 128, K = 128)
//   warps 0-3     : gather the queries of the type (token stride B) into the swizzled K-major A tile with
//                   cp.async, later read the rows of Y from TMEM and scatter them to their tokens
// Types with more than 128 queries take several passes over the same state.
// ---------------------------------------------------------------------------------------------------------------
constexpr int READ_SMEM = 4 * BOX_BYTES + 1024 + 256;

struct ReadParams {
  int64_t T;             // tokens per head
  SmatGroupSpec grp;     // which tokens share a state: types (recent tokens) or profiles (distant tokens)
  int64_t groups;        // states per head
  int64_t items;         // heads * groups
  const __nv_bfloat16* X;  // [bh][T][128] rows contracted against the state
  float* out;            // [bh][T][128] fp32 rows, or
  __nv_bfloat16* out_bf16;  // bf16 rows (when non-null)
  const __nv_bfloat16* X2;  // DUAL: second set of rows, contracted against the FIRST state index of the same state,
  __nv_bfloat16* out2_bf16; // and their bf16 result rows
  int* status;
};

__device__ __forceinline__ void cp_async16_tc(uint32_t smem_addr, const void* gmem) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr), "l"(gmem) : "memory");
}

// TRANS = 0: out[t][j] = Σ_i x_t[i] St[i][j]  (state as MN-major B);  TRANS = 1: out[t][i] = Σ_j x_t[j] St[i][j]
// (the same two boxes read as a K-major B).
// One pass of state_read_tc_kernel: up to 128 tokens of one (state, head) item; states without tokens are skipped.
// Every role walks the same sequence.
struct ReadPass {
  const ReadParams* pp;
  int64_t item, stride;
  int64_t bh, cnt, k0;
  SmatTokens tk;
  __device__ ReadPass(const ReadParams& p, int64_t first, int64_t stride_) : pp(&p), item(first), stride(stride_) { load(); }
  __device__ void load() {
    k0 = 0;
    for (; item < pp->items; item += stride) {
      bh = item / pp->groups;
      tk = smat_group_tokens(pp->grp, bh, item - bh * pp->groups);
      cnt = tk.cnt;
      if (cnt > 0) break;
    }
  }
  __device__ int64_t token(int m) const { return tk.at(k0 + m); }   // position of row m of this pass
  __device__ bool valid() const { return item < pp->items; }
  __device__ bool first() const { return k0 == 0; }
  __device__ bool last() const { return k0 + TILE >= cnt; }
  __device__ int tokens() const { const int64_t left = cnt - k0; return (int)(left < TILE ? left : TILE); }
  __device__ void next() {
    if (last()) { item += stride; load(); } else k0 += TILE;
  }
};

// DUAL (with TRANS = 1): both adjoint reads of a profile's tokens from one load of the state F̄_x —
// out[t] = F̄_x x_t (rows X, e.g. dK from v) and out2[t] = F̄_xᵀ x2_t (rows X2, e.g. dV from k) — two operand tiles, two
// accumulators, bf16 results.
template <int TRANS, int DUAL = 0>
__global__ void __launch_bounds__(160) state_read_tc_kernel(const __grid_constant__ CUtensorMap tmU,
                                                            const ReadParams prm) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* sA = smem;                    // queries, K-major, two 64-column blocks
  uint8_t* sB = smem + 2 * BOX_BYTES;    // state, MN-major, two 64-column blocks
  uint8_t* sA2 = smem + 4 * BOX_BYTES;   // DUAL: the second rows
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (DUAL ? 6 : 4) * BOX_BYTES);
  uint64_t* bar_u = bars + 0;   // state landed (TMA)
  uint64_t* bar_a = bars + 1;   // queries landed (one arrival per warp)
  uint64_t* bar_d = bars + 2;   // product in TMEM
  uint64_t* bar_e = bars + 3;   // TMEM read out (4 arrivals)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 4);
  volatile int* cta_abort = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const WaitCtx wc{cta_abort, prm.status};

  if (threadIdx.x == 0) {
    *cta_abort = 0;
    mbar_init(bar_u, 1); mbar_init(bar_a, 4); mbar_init(bar_d, 1); mbar_init(bar_e, 4);
    fence_barrier_init();
  }
  if (warp == 4) tmem_alloc(tmem_slot, DUAL ? 2 * TILE : TILE);
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem_d = *tmem_slot;
  constexpr uint32_t idesc = make_idesc(TILE, TILE, 0, TRANS ? 0 : 1);
  constexpr uint32_t idesc2 = make_idesc(TILE, TILE, 0, 1);
  ReadPass cur(prm, blockIdx.x, gridDim.x);

  if (warp < 4) {
    const int tid = threadIdx.x;
    const uint32_t a_base = smem_u32(sA), a2_base = smem_u32(sA2);
    auto gather = [&](const ReadPass& ps) {
      const int kn = ps.tokens();
      for (int idx = tid; idx < kn * 16; idx += 128) {
        const int m = idx >> 4, gc = idx & 15;
        const int64_t row = (ps.bh * prm.T + ps.token(m)) * TILE + gc * 8;
        const uint32_t off = (gc >> 3) * BOX_BYTES + m * 128 + (((gc & 7) ^ (m & 7)) << 4);
        cp_async16_tc(a_base + off, prm.X + row);
        if (DUAL) cp_async16_tc(a2_base + off, prm.X2 + row);
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    uint32_t n_pass = 0;
    if (cur.valid()) gather(cur);
    while (cur.valid()) {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_a);   // one arrival per warp
      ReadPass nxt = cur;
      nxt.next();
      bool ok = mbar_wait(bar_d, n_pass & 1, wc);            // the MMAs have read the query tile; the product is in TMEM
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      if (nxt.valid()) gather(nxt);                          // the next queries travel while this product is written out
      fence_after_sync();
      const int m = warp * 32 + lane, kn = cur.tokens();
      const int64_t row = (cur.bh * prm.T + (m < kn ? cur.token(m) : 0)) * TILE;
      float4* dst = reinterpret_cast<float4*>(prm.out + row);
#pragma unroll
      for (int cbo = 0; cbo < (DUAL ? 8 : 4); ++cbo) {
        const int cb = cbo & 3;
        __nv_bfloat16* dst16 = (cbo < 4 ? prm.out_bf16 : prm.out2_bf16) + row;
        uint32_t v[32];
        tmem_ld32(tmem_d + ((uint32_t)(warp * 32) << 16) + cbo * 32, v);
        tmem_ld_wait();
        if (m < kn) {
          if (DUAL || prm.out_bf16) {
#pragma unroll
            for (int h8 = 0; h8 < 2; ++h8) {
              uint32_t w[8];
#pragma unroll
              for (int e = 0; e < 8; ++e)
                w[e] = pack_bf16(__uint_as_float(v[16 * h8 + 2 * e]), __uint_as_float(v[16 * h8 + 2 * e + 1]));
              st_global_v8(dst16 + cb * 32 + 16 * h8, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]);
            }
          } else {
#pragma unroll
            for (int i = 0; i < 4; ++i)   // whole 32-byte sectors
              st_global_v8(dst + cb * 8 + 2 * i, v[8 * i], v[8 * i + 1], v[8 * i + 2], v[8 * i + 3], v[8 * i + 4],
                           v[8 * i + 5], v[8 * i + 6], v[8 * i + 7]);
          }
        }
      }
      fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_e);
      cur = nxt;
      ++n_pass;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
  } else if (lane == 0) {
    (void)idesc2;
    auto load_state = [&](int64_t item) {
      mbar_expect_tx(bar_u, 2 * BOX_BYTES);
      const int row = (int)(item * TILE);
      tma_load_2d(sB, &tmU, 0, row, bar_u);
      tma_load_2d(sB + BOX_BYTES, &tmU, HALF, row, bar_u);
    };
    uint32_t n_item = 0, n_pass = 0;  // completed uses of bar_u and of bar_a / bar_d / bar_e
    bool ok = true;
    if (cur.valid()) load_state(cur.item);
    while (cur.valid() && ok) {
      if (cur.first()) ok = mbar_wait(bar_u, n_item & 1, wc);
      if (ok) ok = mbar_wait(bar_a, n_pass & 1, wc);
      if (ok && n_pass > 0) ok = mbar_wait(bar_e, (n_pass - 1) & 1, wc);  // previous product has been read out
      if (!ok) break;
      fence_after_sync();
#pragma unroll
      for (int kk = 0; kk < TILE / 16; ++kk) {
        const uint64_t dA = make_desc(smem_u32(sA) + (kk >> 2) * BOX_BYTES + (kk & 3) * 32, 16, 1024);
        const uint64_t dB = TRANS ? make_desc(smem_u32(sB) + (kk >> 2) * BOX_BYTES + (kk & 3) * 32, 16, 1024)
                                  : make_desc(smem_u32(sB) + kk * 2048, BOX_BYTES, 1024);
        mma_bf16(tmem_d, dA, dB, idesc, kk != 0);
      }
      if (DUAL) {
#pragma unroll
        for (int kk = 0; kk < TILE / 16; ++kk) {   // the second rows against the state as it lies (MN-major B)
          const uint64_t dA = make_desc(smem_u32(sA2) + (kk >> 2) * BOX_BYTES + (kk & 3) * 32, 16, 1024);
          const uint64_t dB = make_desc(smem_u32(sB) + kk * 2048, BOX_BYTES, 1024);
          mma_bf16(tmem_d + TILE, dA, dB, idesc2, kk != 0);
        }
      }
      mma_commit(bar_d);
      // the state tile may be overwritten (next item) only after the MMAs have read it
      ok = mbar_wait(bar_d, n_pass & 1, wc);
      const bool was_last = cur.last();
      cur.next();
      ++n_pass;
      if (was_last) {
        ++n_item;
        if (ok && cur.valid()) load_state(cur.item);          // travels while the product is written out
      }
    }
  }
  fence_before_sync();
  __syncthreads();
  if (warp == 4) {
    fence_after_sync();
    tmem_dealloc(tmem_d, DUAL ? 2 * TILE : TILE);
  }
}

// ---------------------------------------------------------------------------------------------------------------
// pool_tc_kernel: F_x = Σ_{t ≡ x (mod P), t < n} k_t v_tᵀ (Algorithm 1, step 2) for profiles shared by enough tokens to
// fill tensor-core tiles (d = 2: ~170 tokens per profile, d = 3: 12-24).  Persistent CTAs, one (profile, head) item at
// a time:
//   warps 0-3     : gather the profile's K and V rows (token stride P) into swizzled MN-major tiles with cp.async
//                   (rows up to the next multiple of 16 are zeroed), later write the 128 x 128 state from TMEM
//   warp 4 lane 0 : MMA  F_x += K_xᵀ V_x  (M = N = 128 features, K = 16 tokens per instruction), TOK tokens per pass
// OUT_BF16 = 1 stores the state as bf16 (d = 2, where the profile table is the type table and is only read as an MMA
// operand), else fp32.
// ---------------------------------------------------------------------------------------------------------------
struct PoolParams {
  int64_t T;
  SmatGroupSpec grp;       // profiles (F = Σ k vᵀ over distant tokens) or types (Ū = Σ q dOᵀ over recent tokens)
  int64_t groups;          // states per head
  int64_t items;           // heads * groups
  const __nv_bfloat16* K;  // rows giving the first state index
  const __nv_bfloat16* V;  // rows giving the second state index
  void* F;                 // [bh][groups][128][128] fp32 or bf16
  int slab_major;          // bf16 only: store as [bh][512 slabs of 32 entries][groups][32] instead (a slab of entries of
                           // every state contiguous, the order the register-resident d = 3 tabulation reads)
  int* status;
};

// One pass of pool_tc_kernel: up to TOK tokens of one (group, head) item.  Every role walks the same sequence.
template <int TOK>
struct PoolPass {
  const PoolParams* pp;
  int64_t item, stride;          // current item; items advance by the grid size
  int64_t bh, cnt, k0;
  SmatTokens tk;
  __device__ PoolPass(const PoolParams& p, int64_t first, int64_t stride_) : pp(&p), item(first), stride(stride_) { load(); }
  __device__ void load() {
    k0 = 0;
    if (item < pp->items) {
      bh = item / pp->groups;
      tk = smat_group_tokens(pp->grp, bh, item - bh * pp->groups);
      cnt = tk.cnt;
    }
  }
  __device__ int64_t token(int k) const { return tk.at(k0 + k); }   // position of row k of this pass
  __device__ bool valid() const { return item < pp->items; }
  __device__ bool first() const { return k0 == 0; }
  __device__ bool last() const { return k0 + TOK >= cnt; }
  __device__ int tokens() const { const int64_t left = cnt - k0; return (int)(left < TOK ? (left > 0 ? left : 0) : TOK); }
  __device__ void next() {
    if (last()) { item += stride; load(); } else k0 += TOK;
  }
};

template <int TOK, int OUT_BF16>
__global__ void __launch_bounds__(160) pool_tc_kernel(const PoolParams prm) {
  constexpr int OP_BYTES = 2 * TOK * 128;  // one operand: two 64-feature blocks of TOK rows x 128 bytes
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  constexpr int STAGE_LD = TILE + 4;                                     // floats per staging row (padded)
  constexpr int STAGE_BYTES = OUT_BF16 ? 0 : TILE * STAGE_LD * 4;
  uint8_t* sA = smem;
  uint8_t* sB = smem + OP_BYTES;
  float* stage = reinterpret_cast<float*>(smem + 2 * OP_BYTES);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 2 * OP_BYTES + STAGE_BYTES);
  uint64_t* bar_a = bars + 0;   // operands landed (one arrival per warp)
  uint64_t* bar_d = bars + 1;   // MMAs of the pass finished
  uint64_t* bar_e = bars + 2;   // state read out of TMEM (4 arrivals)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 3);
  volatile int* cta_abort = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const WaitCtx wc{cta_abort, prm.status};

  if (threadIdx.x == 0) {
    *cta_abort = 0;
    mbar_init(bar_a, 4); mbar_init(bar_d, 1); mbar_init(bar_e, 4);
    fence_barrier_init();
  }
  if (warp == 4) tmem_alloc(tmem_slot, TILE);
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem_d = *tmem_slot;
  constexpr uint32_t idesc = make_idesc(TILE, TILE, 1, 1);
  PoolPass<TOK> cur(prm, blockIdx.x, gridDim.x);

  if (warp < 4) {
    const int tid = threadIdx.x;
    const int i = warp * 32 + lane;  // state row = TMEM lane
    const uint32_t a_base = smem_u32(sA), b_base = smem_u32(sB);
    // 16 chunks of K and 16 of V per token; rows up to the next multiple of 16 are zeroed (a group without tokens
    // still gets one all-zero pass, so that its state is written as zeros by the same path)
    auto gather = [&](const PoolPass<TOK>& ps) {
      const int kn = ps.tokens();
      const int kpad = kn ? (kn + 15) & ~15 : 16;
      for (int idx = tid; idx < kpad * 32; idx += 128) {
        const int k = idx >> 5, w = idx & 31, gc = w & 15;
        const uint32_t dst = (w < 16 ? a_base : b_base) + (gc >> 3) * (TOK * 128) + k * 128 + (((gc & 7) ^ (k & 7)) << 4);
        if (k < kn) {
          const __nv_bfloat16* src = (w < 16 ? prm.K : prm.V) + ((ps.bh * prm.T + ps.token(k)) * TILE + gc * 8);
          cp_async16_tc(dst, src);
        } else {
          asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(dst), "r"(0u) : "memory");
        }
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    uint32_t n_pass = 0;
    if (cur.valid()) gather(cur);
    while (cur.valid()) {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_a);                     // pass published (one arrival per warp)
      PoolPass<TOK> nxt = cur;
      nxt.next();
      bool ok = mbar_wait(bar_d, n_pass & 1, wc);            // its MMAs have read the tiles (and, on the last pass, the state is complete)
      ok = __all_sync(0xffffffffu, ok);
      if (ok && nxt.valid()) gather(nxt);                    // the next tokens travel while the state is written out
      if (cur.last()) {
        if (!ok && OUT_BF16) break;
        if (ok) fence_after_sync();
        const int64_t item = cur.item;
#pragma unroll
        for (int cb = 0; cb < 4; ++cb) {
          uint32_t v[32];
          if (ok) {
            tmem_ld32(tmem_d + ((uint32_t)(warp * 32) << 16) + cb * 32, v);
            tmem_ld_wait();
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = 0u;
          }
          if (OUT_BF16) {
            __nv_bfloat16* dst = static_cast<__nv_bfloat16*>(prm.F) + (item * TILE + i) * TILE + cb * 32;
            if (prm.slab_major) {   // entries 32 (4 i + cb) .. + 31 of this state are slab 4 i + cb of its head
              const int64_t head = item / prm.groups, g = item - head * prm.groups;
              dst = static_cast<__nv_bfloat16*>(prm.F) + ((head * (TILE * TILE / 32) + (4 * i + cb)) * prm.groups + g) * 32;
            }
#pragma unroll
            for (int h8 = 0; h8 < 2; ++h8) {  // whole 32-byte sectors
              uint32_t w[8];
#pragma unroll
              for (int e = 0; e < 8; ++e)
                w[e] = pack_bf16(__uint_as_float(v[16 * h8 + 2 * e]), __uint_as_float(v[16 * h8 + 2 * e + 1]));
              st_global_v8(dst + 16 * h8, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]);
            }
          } else {  // fp32 state: through a padded staging tile so that the global writes are whole 512-byte rows
            uint4* srow = reinterpret_cast<uint4*>(stage + i * STAGE_LD + cb * 32);
#pragma unroll
            for (int q4 = 0; q4 < 8; ++q4) srow[q4] = make_uint4(v[4 * q4], v[4 * q4 + 1], v[4 * q4 + 2], v[4 * q4 + 3]);
          }
        }
        if (!OUT_BF16) {
          fence_before_sync();
          const bool bad = bar_or_128(!ok);  // the four epilogue warps meet here and agree on giving up
          float4* dst = reinterpret_cast<float4*>(static_cast<float*>(prm.F) + item * (int64_t)(TILE * TILE));
#pragma unroll 4
          for (int it = 0; it < TILE * TILE / 4 / 128; ++it) {
            const int idx = it * 128 + tid, r = idx >> 5, c4 = idx & 31;
            dst[idx] = *reinterpret_cast<const float4*>(stage + r * STAGE_LD + c4 * 4);
          }
          asm volatile("bar.sync 1, 128;" ::: "memory");  // staging tile free again
          if (bad) break;
        }
        fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_e);
      } else if (!ok) {
        break;
      }
      cur = nxt;
      ++n_pass;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
  } else if (lane == 0) {
    uint32_t n_pass = 0, n_item = 0;
    bool ok = true;
    for (; cur.valid() && ok; cur.next(), ++n_pass) {
      ok = mbar_wait(bar_a, n_pass & 1, wc);
      if (ok && cur.first() && n_item > 0) ok = mbar_wait(bar_e, (n_item - 1) & 1, wc);  // previous state has been read out
      if (!ok) break;
      fence_after_sync();
      const int kn = cur.tokens();
      const int kpad = kn ? (kn + 15) & ~15 : 16;
      const uint64_t dA = make_desc(smem_u32(sA), TOK * 128, 1024);
      const uint64_t dB = make_desc(smem_u32(sB), TOK * 128, 1024);
      for (int kk = 0; kk < kpad / 16; ++kk)
        mma_bf16(tmem_d, dA + (uint64_t)(kk * 128), dB + (uint64_t)(kk * 128), idesc, !(cur.first() && kk == 0));
      mma_commit(bar_d);
      if (cur.last()) ++n_item;
    }
  }
  fence_before_sync();
  __syncthreads();
  if (warp == 4) {
    fence_after_sync();
    tmem_dealloc(tmem_d, TILE);
  }
}

// ---- host: tensor maps ----------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn lookup_encode_fn() {
  void* p = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
      q == cudaDriverEntryPointSuccess)
    return reinterpret_cast<EncodeTiledFn>(p);
  return nullptr;
}

EncodeTiledFn encode_fn() {
  static const EncodeTiledFn fn = lookup_encode_fn();  // initialised once, thread-safe
  return fn;
}

// bf16 matrix [rows, 128] row-major, box = 64 columns x box_rows rows, 128-byte swizzle
bool make_map(CUtensorMap* map, const void* base, uint64_t rows, int box_rows = TILE) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)TILE, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)TILE * 2};
  const cuuint32_t box[2] = {(cuuint32_t)HALF, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// bf16 matrix [rows, inner] row-major; box = box_inner x box_rows; optional 128-byte swizzle (box_inner = 64 then).
bool smat_make_map_2d_bf16(CUtensorMap* map, const void* base, uint64_t inner, uint64_t rows, uint32_t box_inner,
                           uint32_t box_rows, int swizzle128) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)inner * 2};
  const cuuint32_t box[2] = {box_inner, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The library holds sm_100a code only: the current device must be compute capability 10.x, and the driver must
// export the tensor-map encoder the TMA kernels need.
bool smat_tc_available() {
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return false;
  return major == 10 && encode_fn() != nullptr;
}

cudaError_t smat_launch_chunk_scan_tc(const void* K, const void* V, void* Sin_bf16, int64_t T, int bh, int64_t n,
                                      int through, int reverse, int* status, cudaStream_t st, const float* lam) {
  CUtensorMap tmK, tmV;
  if (!make_map(&tmK, K, (uint64_t)bh * T) || !make_map(&tmV, V, (uint64_t)bh * T)) return cudaErrorInvalidValue;
  ScanParams prm;
  prm.lam = lam;
  prm.T = T; prm.NC = (int)(T / TILE);
  prm.Sin = static_cast<__nv_bfloat16*>(Sin_bf16);
  prm.status = status;
  prm.reverse = reverse;
  int blocks;
  if (through) {  // d = 1: the single state U_0 = F_0 is the carry across the boundary
    blocks = 1; prm.lo[0] = 0; prm.hi[0] = prm.NC; prm.lo[1] = prm.hi[1] = 0;
  } else {
    blocks = 2; prm.lo[0] = 0; prm.hi[0] = (int)(n / TILE); prm.lo[1] = prm.hi[0]; prm.hi[1] = prm.NC;
  }
  cudaError_t err = cudaFuncSetAttribute(chunk_scan_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SCAN_SMEM);
  if (err != cudaSuccess) return err;
  dim3 grid((unsigned)(blocks * 2), (unsigned)bh);
  chunk_scan_tc_kernel<<<grid, 192, SCAN_SMEM, st>>>(tmK, tmV, prm);
  return cudaGetLastError();
}

template <bool P4_IS_P1, bool XT, bool ST_KMAJOR, bool GATED = false>
static cudaError_t launch_tile_product(const void* P1, const void* P2, const void* P3, const void* St_bf16,
                                       const float* addend, int64_t add_lo, int64_t add_hi, void* Out, int64_t T,
                                       int bh, int* status, cudaStream_t st, int addend_bf16 = 0,
                                       const float* lam = nullptr) {
  CUtensorMap tm1, tm2, tm3, tmS;
  const int NC = (int)(T / TILE);
  if (!make_map(&tm1, P1, (uint64_t)bh * T) || !make_map(&tm2, P2, (uint64_t)bh * T) ||
      !make_map(&tm3, P3, (uint64_t)bh * T) || !make_map(&tmS, St_bf16, (uint64_t)bh * NC * TILE, ST_KMAJOR ? HALF : TILE))
    return cudaErrorInvalidValue;
  TileParams prm;
  prm.T = T; prm.NC = NC; prm.add_lo = add_lo; prm.add_hi = add_hi; prm.addend = addend;
  prm.addend16 = addend_bf16 ? reinterpret_cast<const __nv_bfloat16*>(addend) : nullptr;
  prm.lam = lam;
  prm.Out = static_cast<__nv_bfloat16*>(Out);
  prm.status = status;
  cudaError_t err = cudaFuncSetAttribute(tile_product_tc_kernel<P4_IS_P1, XT, ST_KMAJOR, GATED>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, OUT_SMEM);
  if (err != cudaSuccess) return err;
  dim3 grid((unsigned)(NC * 2), (unsigned)bh);
  tile_product_tc_kernel<P4_IS_P1, XT, ST_KMAJOR, GATED><<<grid, 160, OUT_SMEM, st>>>(tm1, tm2, tm3, tmS, prm);
  return cudaGetLastError();
}

cudaError_t smat_launch_chunk_output_tc(const void* Q, const void* K, const void* V, const void* Sin_bf16,
                                        const float* ylr, int64_t n_lr, void* O, int64_t T, int bh, int* status,
                                        cudaStream_t st, const float* lam) {
  if (lam)
    return launch_tile_product<true, false, false, true>(Q, K, V, Sin_bf16, ylr, n_lr, T, O, T, bh, status, st, 0, lam);
  return launch_tile_product<true, false, false>(Q, K, V, Sin_bf16, ylr, n_lr, T, O, T, bh, status, st);
}

// The three within-chunk adjoints (which = 0: dQ, 1: dK, 2: dV).  Sin / Dbar are the per-tile bf16 states
// (incoming state, scanned state adjoint); addend rows [add_lo, add_hi) carry the long-range contribution.
cudaError_t smat_launch_chunk_adjoint_tc(int which, const void* Q, const void* K, const void* V, const void* dO,
                                         const void* Sin_bf16, const void* Dbar_bf16, const float* addend,
                                         int64_t add_lo, int64_t add_hi, void* Out, int64_t T, int bh, int* status,
                                         cudaStream_t st, int addend_bf16) {
  if (which == 0)
    return launch_tile_product<true, false, true>(dO, V, K, Sin_bf16, addend, add_lo, add_hi, Out, T, bh, status, st, addend_bf16);
  if (which == 1)
    return launch_tile_product<false, true, true>(dO, V, Q, Dbar_bf16, addend, add_lo, add_hi, Out, T, bh, status, st, addend_bf16);
  return launch_tile_product<false, true, false>(Q, K, dO, Dbar_bf16, addend, add_lo, add_hi, Out, T, bh, status, st, addend_bf16);
}

// The three within-chunk adjoints in one launch: Sin / Dbar are the per-tile bf16 states, lr_q / lr_k / lr_v the bf16
// long-range rows (null: none; lr_q is added to rows t >= n of dQ, lr_k and lr_v to rows t < n of dK and dV).
cudaError_t smat_launch_bwd_tiles_fused_tc(const void* Q, const void* K, const void* V, const void* dO,
                                           const void* Sin_bf16, const void* Dbar_bf16, const void* lr_q, const void* lr_k,
                                           const void* lr_v, int64_t n, void* dQ, void* dK, void* dV, int64_t T, int bh,
                                           int* status, cudaStream_t st, const float* lam) {
  CUtensorMap tmQ, tmK, tmV, tmG, tmS, tmD;
  const int NC = (int)(T / TILE);
  if (!make_map(&tmQ, Q, (uint64_t)bh * T) || !make_map(&tmK, K, (uint64_t)bh * T) || !make_map(&tmV, V, (uint64_t)bh * T) ||
      !make_map(&tmG, dO, (uint64_t)bh * T) || !make_map(&tmS, Sin_bf16, (uint64_t)bh * NC * TILE) ||
      !make_map(&tmD, Dbar_bf16, (uint64_t)bh * NC * TILE))
    return cudaErrorInvalidValue;
  FusedParams prm;
  prm.T = T; prm.NC = NC; prm.n = n;
  prm.lr_q = static_cast<const __nv_bfloat16*>(lr_q);
  prm.lr_k = static_cast<const __nv_bfloat16*>(lr_k);
  prm.lr_v = static_cast<const __nv_bfloat16*>(lr_v);
  prm.dQ = static_cast<__nv_bfloat16*>(dQ); prm.dK = static_cast<__nv_bfloat16*>(dK); prm.dV = static_cast<__nv_bfloat16*>(dV);
  prm.status = status;
  prm.lam = lam;
  auto kernel = lam ? bwd_tile_fused_tc_kernel<true> : bwd_tile_fused_tc_kernel<false>;
  cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, FUSED_SMEM);
  if (err != cudaSuccess) return err;
  dim3 grid((unsigned)NC, (unsigned)bh);
  kernel<<<grid, 160, FUSED_SMEM, st>>>(tmQ, tmK, tmV, tmG, tmS, tmD, prm);
  return cudaGetLastError();
}

// Both adjoint reads of the profile states in one launch: out_t[t] = St x_t (rows Xt, the second state index
// contracted) and out_n[t] = Stᵀ x_t (rows Xn, the first one), bf16 rows; every state is loaded once.
cudaError_t smat_launch_state_read_dual_tc(const void* Xt, const void* Xn, const void* state_bf16, void* out_t_bf16,
                                           void* out_n_bf16, const SmatGroupSpec& grp, int64_t groups, int64_t T, int bh,
                                           int* status, cudaStream_t st) {
  CUtensorMap tmU;
  if (!make_map(&tmU, state_bf16, (uint64_t)bh * groups * TILE)) return cudaErrorInvalidValue;
  ReadParams prm;
  prm.T = T; prm.grp = grp; prm.groups = groups; prm.items = (int64_t)bh * groups;
  prm.X = static_cast<const __nv_bfloat16*>(Xt);
  prm.X2 = static_cast<const __nv_bfloat16*>(Xn);
  prm.out = nullptr;
  prm.out_bf16 = static_cast<__nv_bfloat16*>(out_t_bf16);
  prm.out2_bf16 = static_cast<__nv_bfloat16*>(out_n_bf16);
  prm.status = status;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int smem = READ_SMEM + 2 * BOX_BYTES;
  const int64_t grid = prm.items < 2LL * sms ? prm.items : 2LL * sms;   // 256 columns of tensor memory and 97 KB each
  cudaError_t err = cudaFuncSetAttribute(state_read_tc_kernel<1, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (err != cudaSuccess) return err;
  state_read_tc_kernel<1, 1><<<(unsigned)grid, 160, smem, st>>>(tmU, prm);
  return cudaGetLastError();
}

cudaError_t smat_launch_state_read_tc(const void* X, const void* state_bf16, float* out, void* out_bf16, int transposed,
                                      const SmatGroupSpec& grp, int64_t groups, int64_t T, int bh, int* status,
                                      cudaStream_t st) {
  CUtensorMap tmU;
  if (!make_map(&tmU, state_bf16, (uint64_t)bh * groups * TILE)) return cudaErrorInvalidValue;
  ReadParams prm;
  prm.T = T; prm.grp = grp; prm.groups = groups; prm.items = (int64_t)bh * groups;
  prm.X = static_cast<const __nv_bfloat16*>(X);
  prm.X2 = nullptr; prm.out2_bf16 = nullptr;
  prm.out = out;
  prm.out_bf16 = static_cast<__nv_bfloat16*>(out_bf16);
  prm.status = status;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int64_t grid = prm.items < 3LL * sms ? prm.items : 3LL * sms;
  cudaError_t err;
  if (transposed) {
    err = cudaFuncSetAttribute(state_read_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, READ_SMEM);
    if (err != cudaSuccess) return err;
    state_read_tc_kernel<1><<<(unsigned)grid, 160, READ_SMEM, st>>>(tmU, prm);
  } else {
    err = cudaFuncSetAttribute(state_read_tc_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, READ_SMEM);
    if (err != cudaSuccess) return err;
    state_read_tc_kernel<0><<<(unsigned)grid, 160, READ_SMEM, st>>>(tmU, prm);
  }
  return cudaGetLastError();
}

template <int TOK, int OUT_BF16>
static cudaError_t launch_pool_tc(const PoolParams& prm, cudaStream_t st) {
  const int smem = 4 * TOK * 128 + (OUT_BF16 ? 0 : TILE * (TILE + 4) * 4) + 1024 + 256;
  cudaError_t err = cudaFuncSetAttribute(pool_tc_kernel<TOK, OUT_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (err != cudaSuccess) return err;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  // each CTA holds 128 columns of tensor memory, so at most four fit an SM
  const int per_sm = smem <= 54 * 1024 ? 4 : (smem <= 72 * 1024 ? 3 : (smem <= 110 * 1024 ? 2 : 1));
  const int64_t grid = prm.items < (int64_t)per_sm * sms ? prm.items : (int64_t)per_sm * sms;
  pool_tc_kernel<TOK, OUT_BF16><<<(unsigned)grid, 160, smem, st>>>(prm);
  return cudaGetLastError();
}

cudaError_t smat_launch_pool_tc(const void* K, const void* V, void* F, int out_bf16, const SmatGroupSpec& grp,
                                int64_t groups, int64_t max_tokens, int64_t T, int bh, int* status, cudaStream_t st,
                                int slab_major) {
  PoolParams prm;
  if (slab_major && !out_bf16) return cudaErrorInvalidValue;
  prm.slab_major = slab_major;
  prm.T = T; prm.grp = grp; prm.groups = groups; prm.items = (int64_t)bh * groups;
  prm.K = static_cast<const __nv_bfloat16*>(K);
  prm.V = static_cast<const __nv_bfloat16*>(V);
  prm.F = F;
  prm.status = status;
  if (max_tokens <= 32) return out_bf16 ? launch_pool_tc<32, 1>(prm, st) : launch_pool_tc<32, 0>(prm, st);
  return out_bf16 ? launch_pool_tc<128, 1>(prm, st) : launch_pool_tc<128, 0>(prm, st);
}

// Largest segment length (tiles) that divides every block and still leaves enough CTAs to fill the machine.
int smat_segment_tiles(int64_t tiles_block0, int64_t tiles_block1, int bh) {
  for (int L = 16; L >= 2; L >>= 1) {
    if (tiles_block0 % L || (tiles_block1 && tiles_block1 % L)) continue;
    const int64_t ctas = (tiles_block0 + tiles_block1) / L * bh;
    if (ctas >= 296 || L == 2) return L;
  }
  return 1;
}

// Segment counts of the two blocks.  The output kernel runs one CTA per SM and a CTA walks its segment tile by tile,
// so the launch takes ceil(segments * heads / SMs) rounds of the longest segment: the counts are chosen to fill the
// last round (t64k with 16 heads: 37 segments of 13 or 14 tiles = 4 full rounds, where 32 segments of 16 tiles leave
// the fourth round half empty).  A segment costs about two and a half tiles besides its tiles (its state goes to memory
// and back, the pipeline fills), at most 16 tiles long and at least 2 on average.  L is the power-of-two length the
// fixed rule picks, kept unless the estimate improves on it by a few percent.
void smat_segment_counts(int64_t tiles0, int64_t tiles1, int bh, int L, int* nseg0, int* nseg1) {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const double overhead = 2.5;
  auto cost = [&](int64_t n0, int64_t n1) {
    const int64_t l0 = (tiles0 + n0 - 1) / n0, l1 = n1 ? (tiles1 + n1 - 1) / n1 : 0;
    const int64_t lmax = l0 > l1 ? l0 : l1;
    const int64_t rounds = ((n0 + n1) * bh + sms - 1) / sms;
    return (double)rounds * ((double)lmax + overhead);
  };
  int64_t best0 = tiles0 / L, best1 = tiles1 / L;
  double best = cost(best0, best1) * 0.96;
  const int64_t max0 = tiles0 / 2 > 0 ? tiles0 / 2 : 1, max1 = tiles1 / 2;
  for (int64_t n0 = 1; n0 <= max0 && n0 <= 512; ++n0) {
    if ((tiles0 + n0 - 1) / n0 > 16) continue;
    // block 1 gets the count that gives it the same longest segment, or one more segment
    const int64_t l0 = (tiles0 + n0 - 1) / n0;
    for (int64_t n1 = tiles1 ? (tiles1 + l0 - 1) / l0 : 0, k = 0; k < 2; ++k, ++n1) {
      if (tiles1 && (n1 < 1 || n1 > max1 || (tiles1 + n1 - 1) / n1 > 16)) continue;
      if (!tiles1 && k) break;
      const double c = cost(n0, n1);
      if (c < best) { best = c; best0 = n0; best1 = n1; }
    }
  }
  *nseg0 = (int)best0; *nseg1 = (int)best1;
}

cudaError_t smat_launch_segment_state_tc(const void* K, const void* V, float* totals, int64_t tiles0, int64_t tiles1,
                                         int nseg0, int nseg1, int bh, int* status, cudaStream_t st) {
  const int64_t T = (tiles0 + tiles1) * TILE;
  CUtensorMap tmK, tmV;
  if (!make_map(&tmK, K, (uint64_t)bh * T) || !make_map(&tmV, V, (uint64_t)bh * T)) return cudaErrorInvalidValue;
  SegStateParams prm;
  prm.T = T; prm.nseg = nseg0 + nseg1; prm.totals = totals; prm.status = status;
  prm.cut.nseg0 = nseg0; prm.cut.nseg = nseg0 + nseg1; prm.cut.tiles0 = tiles0; prm.cut.tiles1 = tiles1;
  cudaError_t err =
      cudaFuncSetAttribute(segment_state_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SEG_STATE_SMEM);
  if (err != cudaSuccess) return err;
  dim3 grid((unsigned)prm.nseg, (unsigned)bh);
  segment_state_tc_kernel<<<grid, 192, SEG_STATE_SMEM, st>>>(tmK, tmV, prm);
  return cudaGetLastError();
}

cudaError_t smat_launch_segment_output_tc(const void* Q, const void* K, const void* V, const float* seg_in,
                                          const void* ylr_bf16, int64_t n_lr, void* O, int64_t tiles0, int64_t tiles1,
                                          int nseg0, int nseg1, int bh, int* status, cudaStream_t st, void* sin_tiles) {
  const int64_t T = (tiles0 + tiles1) * TILE;
  CUtensorMap tmQ, tmK, tmV;
  if (!make_map(&tmQ, Q, (uint64_t)bh * T) || !make_map(&tmK, K, (uint64_t)bh * T) ||
      !make_map(&tmV, V, (uint64_t)bh * T))
    return cudaErrorInvalidValue;
  SegOutParams prm;
  prm.T = T; prm.nseg = nseg0 + nseg1; prm.seg_in = seg_in; prm.n_lr = n_lr; prm.ylr = static_cast<const __nv_bfloat16*>(ylr_bf16);
  prm.cut.nseg0 = nseg0; prm.cut.nseg = nseg0 + nseg1; prm.cut.tiles0 = tiles0; prm.cut.tiles1 = tiles1;
  prm.O = static_cast<__nv_bfloat16*>(O);
  prm.sin_tiles = static_cast<__nv_bfloat16*>(sin_tiles);
  prm.status = status;
  cudaError_t err =
      cudaFuncSetAttribute(segment_output_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SEG_OUT_SMEM);
  if (err != cudaSuccess) return err;
  dim3 grid((unsigned)prm.nseg, (unsigned)bh);
  segment_output_tc_kernel<<<grid, SEG_OUT_THREADS, SEG_OUT_SMEM, st>>>(tmQ, tmK, tmV, prm);
  return cudaGetLastError();
}
