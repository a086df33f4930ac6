// Tabulation U = C F (Algorithm 2) and its transpose F̄ = Cᵀ Ū on the tensor cores, for d = 3 and d = 4 with
// bf16 tables.
//
// The incidence matrix factors through the two-dimensional finite Radon transform over F_q x F_q,
//     (R f)(a, u) = Σ_{lo + a hi ≡ u} f(lo, hi)  for slopes a in F_q,      (R f)(∞, u) = Σ_lo f(lo, u),
// a 0/1 matrix with q^2 + q rows and q^2 columns:
//   d = 3 : U = R F, one image per state entry.
//   d = 4 : stage 1, one image per x2 :  W[a3][x2][u] = Σ_{x3} F[u - a3 x3, x2, x3],  G[x3][x2] = Σ_{x1} F[x1, x2, x3]
//           stage 2, one image per a3 :  U[(1, a2, a3), b] = Σ_{x2} W[a3][x2][b - a2 x2];
//                    the image G gives the directions (0, 1, a3) and (0, 0, 1).
// These are the sums of Algorithm 2 taken one coordinate pair at a time (same real numbers, different order).
// The transposes run the same stages backwards with Rᵀ.  R is small (q <= 23) and fixed, the images are
// independent across the r p state entries, so each stage is a product of a resident 0/1 matrix with a stream
// of images: dense enough for the tensor cores (q of every q^2 entries of a row are nonzero, and the
// 5th-generation tensor cores multiply-add about 60 times faster than the fp32 pipes add), bound by the image
// traffic.
//
// radon_tc_kernel, persistent, one CTA per SM.  An item is one image restricted to 128 consecutive state entries;
// a CTA owns up to 128 output indices (its part of R; the output indices are split evenly over `parts` CTAs that
// then share every image) and applies them to every item it is given:
//   warps 0-3      : build the CTA's part of R once and move it to tensor memory (lane = output index, one column
//                    per two operand rows), where the MMAs read it as their A operand
//   warp 16 lane 0 : TMA producer; a ring slot holds `sps` lines (fixed hi, all lo) of the image x 128 state entries
//                    (MN-major B operand, two boxes of 64 entries); the extra class travels in a slot of its own
//   warps 17, 18 (lane 0) : MMA issuers, alternating items: D[128 outputs, 128 entries] += R_slot * B_slot; up to
//                    four accumulators in flight
//   warps 0-15     : epilogue, one output index (TMEM lane) per thread and one 32-entry column chunk per warp:
//                    round to bf16 and store 64 contiguous bytes of the output row as two 32-byte sectors
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "smat_internal.h"
#include "smat_tc.cuh"

namespace {

using namespace tc;

constexpr int TILE_ROWS = 128;                    // output indices per tile (MMA M)
constexpr int EPI_WARPS = 16;
constexpr int PROD_WARP = EPI_WARPS;
constexpr int MMA_WARP = EPI_WARPS + 1;
constexpr int MMA_WARPS = 2;                      // issuing threads; they take the items alternately
constexpr int RADON_THREADS = 32 * (MMA_WARP + MMA_WARPS);
constexpr int MAX_ACC = 4;                        // accumulators in flight: what the R columns leave of 512, at most 4
constexpr int ROW_INVALID = -1;
constexpr int ROW_VERT = 1 << 30;                 // flag: row of the extra ("vertical") class

// One index space of the transform: idx = lo + q*hi, hi in [0, q]; hi == q is the extra class (a = ∞ on the
// type side).  Rows are counted inside one head.
struct RadonSide {
  int32_t count;                   // q*q, or q*q + q with the extra class
  int32_t s_lo, s_hi, s_img;       // regular rows: img*s_img + lo*s_lo + hi*s_hi
  int32_t v0, sv_lo, sv_img;       // extra class : v0 + img*sv_img + lo*sv_lo
  int32_t vert_from;               // images >= vert_from carry the extra class
  int64_t rows_per_head;
};

struct RadonParams {
  int32_t q, transpose;
  int32_t sps, sr;                 // lines (hi values) per ring slot; rows of a slot = sps*q rounded up to 16
  int32_t nreg, nslots;            // slots of regular lines per image; plus one when the input has the extra class
  int32_t parts, rows_pp;          // CTAs sharing an image, and output indices per CTA (<= 128)
  int32_t ring;                    // ring slots
  int32_t images;
  int32_t slabs_per_head;          // rp / 128
  int64_t slabs;                   // heads * slabs_per_head
  int64_t rp;
  RadonSide in, out;
  const __nv_bfloat16* src;
  __nv_bfloat16* dst;
  int* status;
};

// Lane 0 polls the barrier and the warp follows.
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* bar, uint32_t parity, const WaitCtx& w) {
  bool ok = true;
  if ((threadIdx.x & 31) == 0) ok = mbar_wait(bar, parity, w);
  return __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
}

__device__ __forceinline__ int side_row(const RadonSide& s, int idx, int q) {
  if (idx >= s.count) return ROW_INVALID;
  const int lo = idx % q, hi = idx / q;
  return hi < q ? lo * s.s_lo + hi * s.s_hi : (ROW_VERT | lo * s.sv_lo);
}

// Row of the streamed operand that holds input index (lo, line): slot line / sps, then the line's q rows.
__device__ __forceinline__ int operand_row(const RadonParams& p, int line, int lo) {
  if (line >= p.q) return p.nreg * p.sr + lo;                 // extra class: a slot of its own
  const int slot = line / p.sps;
  return slot * p.sr + (line - slot * p.sps) * p.q + lo;
}

// Marks in `row` (one bf16 per operand row, zeroed by the caller) the input indices incident with output index n.
// Forward: n = (u, a); a < q meets every line hi in lo = u - a hi, a = q (extra class) meets the whole line u.
// Transposed: n = point (lo, hi); it lies on one offset u = lo + a hi of every slope a, and on offset hi of the extra class.
__device__ __forceinline__ void mark_incident(const RadonParams& p, int n, __nv_bfloat16* row) {
  const int q = p.q, x = n % q, y = n / q;
  const __nv_bfloat16 one = __float2bfloat16(1.0f);
  if (!p.transpose) {
    if (y < q) {
      int lo = x;                                               // u - a*hi for hi = 0, 1, ...
      for (int hi = 0; hi < q; ++hi) {
        row[operand_row(p, hi, lo)] = one;
        lo -= y; if (lo < 0) lo += q;
      }
    } else {
      for (int lo = 0; lo < q; ++lo) row[operand_row(p, x, lo)] = one;
    }
  } else {
    int u = x;                                                  // lo + a*hi for a = 0, 1, ...
    for (int a = 0; a < q; ++a) {
      row[operand_row(p, a, u)] = one;
      u += y; if (u >= q) u -= q;
    }
    if (p.in.count > q * q) row[operand_row(p, q, y)] = one;
  }
}

// box of 64 state entries x q rows x sps lines (regular map) or 64 x q rows (extra-class map)
__device__ __forceinline__ void tma_load_5d(void* smem_dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                            int c4, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
      ::"r"(smem_u32(smem_dst)), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void tma_load_4d(void* smem_dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                            uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(smem_u32(smem_dst)), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(smem_u32(bar))
      : "memory");
}

// D[tmem_d] (+)= A[tmem_a] * B[desc_b]: A (128 x 16, bf16) read from tensor memory, B from shared memory.
__device__ __forceinline__ void mma_bf16_ta(uint32_t tmem_d, uint32_t tmem_a, uint64_t desc_b, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n"
      "}\n" ::"r"(tmem_d),
      "r"(tmem_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}

// The MMAs of one ring slot: STEPS K-steps of 16 operand rows.  Fully unrolled so that the lone issuing thread spends
// a handful of instructions per MMA.  A K-step reads 8 columns of R (two bf16 per column) and 16 rows of the slot.
template <int STEPS>
__device__ __forceinline__ void issue_slot(uint32_t tmem_d, uint32_t tmem_a, uint64_t dB, uint32_t idesc, bool first) {
#pragma unroll
  for (int kk = 0; kk < STEPS; ++kk)
    mma_bf16_ta(tmem_d, tmem_a + kk * 8, dB + (uint64_t)(kk * 128), idesc, !(first && kk == 0));
}
__device__ __forceinline__ void issue_slot_steps(int steps, uint32_t tmem_d, uint32_t tmem_a, uint64_t dB, uint32_t idesc,
                                                 bool first) {
  switch (steps) {
    case 1: issue_slot<1>(tmem_d, tmem_a, dB, idesc, first); break;
    case 2: issue_slot<2>(tmem_d, tmem_a, dB, idesc, first); break;
    case 3: issue_slot<3>(tmem_d, tmem_a, dB, idesc, first); break;
    case 4: issue_slot<4>(tmem_d, tmem_a, dB, idesc, first); break;
    case 5: issue_slot<5>(tmem_d, tmem_a, dB, idesc, first); break;
    case 6: issue_slot<6>(tmem_d, tmem_a, dB, idesc, first); break;
    case 7: issue_slot<7>(tmem_d, tmem_a, dB, idesc, first); break;
    default: issue_slot<8>(tmem_d, tmem_a, dB, idesc, first); break;
  }
}

__global__ void __launch_bounds__(RADON_THREADS, 1) radon_tc_kernel(const __grid_constant__ CUtensorMap tm_reg,
                                                                    const __grid_constant__ CUtensorMap tm_vert,
                                                                    const RadonParams prm) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int q = prm.q;
  const int slot_bytes = prm.sr * 256;                          // two 64-entry blocks of sr rows x 128 bytes
  const int kt = prm.nslots * prm.sr;                           // operand rows per image
  uint8_t* sRing = smem;
  int32_t* out_tab = reinterpret_cast<int32_t*>(sRing + prm.ring * slot_bytes);    // [128]
  uint64_t* bars = reinterpret_cast<uint64_t*>(out_tab + TILE_ROWS);
  uint64_t* full = bars;                    // [ring] slot filled (TMA bytes)
  uint64_t* empty = bars + prm.ring;        // [ring] slot consumed by the MMAs (arrival from the epilogue, once the item is complete)
  uint64_t* acc_full = empty + prm.ring;    // [MAX_ACC] accumulator complete
  uint64_t* acc_empty = acc_full + MAX_ACC; // [MAX_ACC] accumulator read out (one arrival per epilogue warp)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + MAX_ACC);
  volatile int* cta_abort = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const WaitCtx wc{cta_abort, prm.status};
  const int part = blockIdx.x % prm.parts;

  if (threadIdx.x == 0) {
    *cta_abort = 0;
    for (int s = 0; s < prm.ring; ++s) { mbar_init(full + s, 1); mbar_init(empty + s, 1); }
    for (int b = 0; b < MAX_ACC; ++b) { mbar_init(acc_full + b, 1); mbar_init(acc_empty + b, EPI_WARPS); }
    fence_barrier_init();
    prefetch_tmap(&tm_reg);
    prefetch_tmap(&tm_vert);
  }
  if (warp == MMA_WARP) tmem_alloc(tmem_slot, 512);
  // This CTA's part of R, built row by row in the (still unused) ring and moved to tensor memory: lane = output
  // index, one column per two operand rows.  The launcher guarantees ring * slot_bytes >= 128 * kt * 2.
  __nv_bfloat16* scratch = reinterpret_cast<__nv_bfloat16*>(sRing);
  for (int c = threadIdx.x; c < prm.ring * slot_bytes / 16; c += blockDim.x)
    reinterpret_cast<uint4*>(sRing)[c] = make_uint4(0u, 0u, 0u, 0u);
  for (int n = threadIdx.x; n < TILE_ROWS; n += blockDim.x)
    out_tab[n] = n < prm.rows_pp ? side_row(prm.out, part * prm.rows_pp + n, q) : ROW_INVALID;
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t r_cols = (uint32_t)((kt / 2 + 31) & ~31);       // columns taken by R
  const uint32_t nacc = min(MAX_ACC, (int)((512 - r_cols) / 128));
  if (warp < 4) {
    const int n = warp * 32 + lane;
    __nv_bfloat16* row = scratch + (size_t)n * kt;
    if (n < prm.rows_pp && part * prm.rows_pp + n < prm.out.count) mark_incident(prm, part * prm.rows_pp + n, row);
    __syncwarp();
    const uint32_t* roww = reinterpret_cast<const uint32_t*>(row);
    for (int c0 = 0; c0 < (int)r_cols; c0 += 32) {
      uint32_t v[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] = (c0 + i) * 2 < kt ? roww[c0 + i] : 0u;
      tmem_st32(tmem_base + ((uint32_t)(warp * 32) << 16) + c0, v);
    }
    tmem_st_wait();
  }
  __syncthreads();
  // rows no box writes must never hold NaN patterns: the ones just written are 0 or 1, which is fine
  fence_proxy_async();
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem_acc = tmem_base + r_cols;

  // items of this CTA: same part always; slab fastest, image slowest
  const uint32_t first = blockIdx.x / prm.parts, step = gridDim.x / prm.parts;
  const uint32_t slabs = (uint32_t)prm.slabs, total = slabs * (uint32_t)prm.images;   // < 2^31 (checked by the launcher)

  if (warp == PROD_WARP && lane == 0) {
    // ---- TMA producer -----------------------------------------------------------------------------------------
    // The two single-thread roles keep running slot / parity counters: a lone thread pays the full latency of every
    // instruction, so divisions by the ring size inside the loop would show in the kernel time.
    uint32_t slot = 0, par = 0;                               // ring position; parity of the empty barrier's phase to wait for
    bool first_lap = true, ok = true;
    const uint32_t reg_bytes = 2u * 128u * (uint32_t)(q * prm.sps), vert_bytes = 2u * 128u * (uint32_t)q;
    const int heads = (int)(prm.slabs / prm.slabs_per_head);
    const uint32_t sph = (uint32_t)prm.slabs_per_head;
    uint32_t img = first / slabs, slab = first - img * slabs;
    for (uint32_t it = first; it < total && ok; it += step) {
      const uint32_t head = slab / sph;
      const int e0 = (int)(slab - head * sph) * 128;
      for (int g = 0; g < prm.nslots; ++g) {
        if (!first_lap) ok = mbar_wait(empty + slot, par, wc);
        if (!ok) break;
        uint8_t* dst = sRing + slot * slot_bytes;
        if (g < prm.nreg) {   // lines hi = g*sps ..; lines past q - 1 are out of bounds and arrive as zeros
          mbar_expect_tx(full + slot, reg_bytes);
          tma_load_5d(dst, &tm_reg, e0, 0, g * prm.sps, (int)img, (int)head, full + slot);
          tma_load_5d(dst + prm.sr * 128, &tm_reg, e0 + 64, 0, g * prm.sps, (int)img, (int)head, full + slot);
        } else {              // extra class; an image without it reads past the last head: zeros
          const int h = (int)img >= prm.in.vert_from ? (int)head : heads;
          const int ci = (int)img * prm.in.sv_img;   // 0 when every image shares the rows
          mbar_expect_tx(full + slot, vert_bytes);
          tma_load_4d(dst, &tm_vert, e0, 0, ci, h, full + slot);
          tma_load_4d(dst + prm.sr * 128, &tm_vert, e0 + 64, 0, ci, h, full + slot);
        }
        if (++slot == (uint32_t)prm.ring) {
          slot = 0;
          if (first_lap) { first_lap = false; par = 0; } else par ^= 1;
        }
      }
      slab += step;
      while (slab >= slabs) { slab -= slabs; ++img; }
    }
  } else if (warp >= MMA_WARP && lane == 0) {
    // ---- MMA issuers: the two threads take the items alternately, so that the issue latency of one item (waits,
    // MMAs, commits: more than the tensor pipe needs for it) overlaps with the other thread's item ----------------
    const uint32_t me = (uint32_t)(warp - MMA_WARP);
    constexpr uint32_t idesc = make_idesc(TILE_ROWS, 128, 0, 1);   // A from tensor memory (R), B MN-major (image rows)
    const uint64_t dB0 = make_desc(smem_u32(sRing), prm.sr * 128, 1024);
    const uint32_t slot16 = (uint32_t)slot_bytes >> 4;            // descriptor address units are 16 bytes
    const uint32_t slot_cols = (uint32_t)prm.sr / 2;              // columns of R per slot
    const int steps = prm.sr / 16, nslots = prm.nslots;
    const uint32_t ring = (uint32_t)prm.ring;
    uint32_t slot = 0, par = 0;                                   // ring position and the parity its full barrier shows
    uint32_t buf = 0, apar = 0, n_item = 0;                       // accumulator; parity of its empty barrier's phase to wait for
    bool ok = true;
    if (nslots == 1) {
      // One slot per item (q <= 11): a single thread, and the leanest loop: every instruction here is on the
      // critical path of the stage.
      for (uint32_t it = first; me == 0 && it < total && ok; it += step, ++n_item) {
        if (n_item >= nacc) ok = mbar_wait(acc_empty + buf, apar, wc);
        if (!ok) break;
        ok = mbar_wait(full + slot, par, wc);
        if (!ok) break;
        fence_after_sync();
        issue_slot_steps(steps, tmem_acc + buf * 128, tmem_base, dB0 + (uint64_t)(slot * slot16), idesc, true);
        mma_commit(empty + slot);
        mma_commit(acc_full + buf);
        if (++slot == ring) { slot = 0; par ^= 1; }
        if (++buf == nacc) { buf = 0; if (n_item >= nacc) apar ^= 1; }
      }
    } else {
      uint32_t turn = 0;
      for (uint32_t it = first; it < total && ok; it += step, ++n_item) {
        const bool mine = turn == me;
        if (++turn == MMA_WARPS) turn = 0;
        if (!mine) {   // the other thread's item: step the counters over it
          for (int g = 0; g < nslots; ++g)
            if (++slot == ring) { slot = 0; par ^= 1; }
          if (++buf == nacc) { buf = 0; if (n_item >= nacc) apar ^= 1; }
          continue;
        }
        if (n_item >= nacc) ok = mbar_wait(acc_empty + buf, apar, wc);
        if (!ok) break;
        fence_after_sync();
        const uint32_t tmem_d = tmem_acc + buf * 128;
        uint32_t tmem_a = tmem_base;
        for (int g = 0; g < nslots && ok; ++g, tmem_a += slot_cols) {
          ok = mbar_wait(full + slot, par, wc);
          if (!ok) break;
          fence_after_sync();
          issue_slot_steps(steps, tmem_d, tmem_a, dB0 + (uint64_t)(slot * slot16), idesc, g == 0);
          if (++slot == ring) { slot = 0; par ^= 1; }
        }
        if (ok) mma_commit(acc_full + buf);   // the only commit of the item: the epilogue frees its slots when it sees it
        if (++buf == nacc) { buf = 0; if (n_item >= nacc) apar ^= 1; }
      }
    }
  } else if (warp < EPI_WARPS) {
    // ---- epilogue ---------------------------------------------------------------------------------------------
    // Warp w reads lane quarter w % 4 (32 output indices) and the 32-entry column chunk w / 4 of every item.
    const int qd = warp & 3, cb = warp >> 2;
    const int orow = qd * 32 + lane;                            // output index of this CTA = TMEM lane
    const uint32_t lane_base = (uint32_t)(qd * 32) << 16;
    const int tv = out_tab[orow];
    const bool active = qd * 32 < prm.rows_pp;                  // warp-uniform: some output index in these lanes
    const uint32_t sph = (uint32_t)prm.slabs_per_head;
    uint32_t buf = 0, apar = 0, eslot = 0;
    uint32_t img = first / slabs, slab = first - img * slabs;
    for (uint32_t it = first; it < total; it += step) {
      const uint32_t head = slab / sph;
      const int e0 = (int)(slab - head * sph) * 128;
      if (!mbar_wait_warp(acc_full + buf, apar, wc)) break;
      fence_after_sync();
      if (warp == 0 && prm.nslots > 1) {   // every MMA of the item has completed: its ring slots are free (a commit per slot would cost the
                         // issuing thread more than the MMAs of the slot)
        for (int g = 0; g < prm.nslots; ++g) {
          if (lane == 0) mbar_arrive(empty + eslot);
          if (++eslot == (uint32_t)prm.ring) eslot = 0;
        }
      }
      if (active) {
        uint32_t v[32];
        tmem_ld32(tmem_acc + lane_base + buf * 128 + cb * 32, v);
        tmem_ld_wait();
        const bool vert = (int)img >= prm.out.vert_from;
        if (tv != ROW_INVALID && (!(tv & ROW_VERT) || vert)) {
          const int row = (tv & ROW_VERT) ? prm.out.v0 + (int)img * prm.out.sv_img + (tv & ~ROW_VERT)
                                          : (int)img * prm.out.s_img + tv;
          __nv_bfloat16* dst = prm.dst + ((int64_t)head * prm.out.rows_per_head + row) * prm.rp + e0 + cb * 32;
#pragma unroll
          for (int h8 = 0; h8 < 2; ++h8) {   // two whole 32-byte sectors per thread
            uint32_t w[8];
#pragma unroll
            for (int i = 0; i < 8; ++i)
              w[i] = pack_bf16(__uint_as_float(v[16 * h8 + 2 * i]), __uint_as_float(v[16 * h8 + 2 * i + 1]));
            st_global_v8(dst + 16 * h8, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]);
          }
        }
      }
      fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty + buf);
      if (++buf == nacc) { buf = 0; apar ^= 1; }
      slab += step;
      while (slab >= slabs) { slab -= slabs; ++img; }
    }
  }
  fence_before_sync();
  __syncthreads();
  if (warp == MMA_WARP) {
    fence_after_sync();
    tmem_dealloc(tmem_base, 512);
  }
}

struct RadonShape {
  int sps, sr, nreg, nslots, parts, rows_pp, ring, smem;
};

// Ring slots of `sps` lines (sps*q rows, rounded up to 16), chosen for the least MMA work; the output indices are
// split evenly over `parts` CTAs of at most 128 each.  R (128 lanes x one column per two operand rows) and at least
// two accumulators of 128 columns must fit the 512 columns of tensor memory, and the ring must be able to hold the
// scratch copy of R while it is built.  Returns false when q is too large for this kernel.
bool radon_shape(int q, int in_has_extra, int count_out, RadonShape* s) {
  const int budget = 227 * 1024 - 1024 - 512 - TILE_ROWS * 4;
  if (q < 2 || q > 64) return false;
  const int parts = (count_out + TILE_ROWS - 1) / TILE_ROWS;
  if (parts > 8) return false;
  int best = 1 << 30;
  for (int sps = 1; sps <= q; ++sps) {
    const int sr = (sps * q + 15) & ~15;
    if (sr > 128) break;
    const int nreg = (q + sps - 1) / sps, nslots = nreg + (in_has_extra ? 1 : 0);
    const int r_cols = (nslots * sr / 2 + 31) & ~31;
    if (r_cols + 2 * 128 > 512) continue;
    const int slot_bytes = sr * 256;
    int ring = budget / slot_bytes;
    if (ring > 8) ring = 8;
    if (ring < 3 || ring < nslots || (nslots > 1 && ring < 2 * nslots)) continue;   // several slots per item are freed
                                                                                    // together: room for two items
    const int cost = nslots * (sr + 48);   // operand rows per image, plus a charge per slot for its hand-over
    if (cost < best) {
      best = cost;
      s->sps = sps; s->sr = sr; s->nreg = nreg; s->nslots = nslots; s->parts = parts;
      s->rows_pp = (count_out + parts - 1) / parts; s->ring = ring;
      s->smem = ring * slot_bytes + TILE_ROWS * 4 + 512 + 1024;
    }
  }
  return best != (1 << 30);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn radon_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess &&
        qr == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 rows of rp entries.  Dimensions (fastest first): entry, then `rank - 1` row indices with the given sizes and
// strides in rows; box = 64 entries x box[] rows; 128-byte swizzle; out-of-bounds reads give zeros.
bool radon_map(CUtensorMap* map, const void* base, int64_t rp, int rank, const int64_t* sizes, const int64_t* row_strides,
               const int* box) {
  EncodeTiledFn fn = radon_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[5], strides[4];
  cuuint32_t bx[5], estr[5];
  dims[0] = (cuuint64_t)rp; bx[0] = 64; estr[0] = 1;
  for (int i = 1; i < rank; ++i) {
    dims[i] = (cuuint64_t)sizes[i - 1];
    strides[i - 1] = (cuuint64_t)row_strides[i - 1] * (cuuint64_t)rp * 2;
    bx[i] = (cuuint32_t)box[i - 1];
    estr[i] = 1;
  }
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), dims, strides, bx, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

RadonSide side(int count, int s_lo, int s_hi, int s_img, int64_t rows_per_head, int v0 = 0, int sv_lo = 0,
               int sv_img = 0, int vert_from = 1 << 29) {
  RadonSide s;
  s.count = count; s.s_lo = s_lo; s.s_hi = s_hi; s.s_img = s_img; s.v0 = v0; s.sv_lo = sv_lo; s.sv_img = sv_img;
  s.vert_from = vert_from; s.rows_per_head = rows_per_head;
  return s;
}

cudaError_t launch_radon(int q, int transpose, int images, const RadonSide& in, const RadonSide& out, const void* src,
                         void* dst, int64_t rp, int bh, int* status, cudaStream_t st) {
  RadonShape sh;
  const int in_has_extra = in.count > q * q;
  if (!radon_shape(q, in_has_extra, out.count, &sh) || rp % 128 || (int64_t)bh * (rp / 128) * images >= (1LL << 31))
    return cudaErrorInvalidValue;
  RadonParams prm;
  prm.q = q; prm.transpose = transpose; prm.sps = sh.sps; prm.sr = sh.sr; prm.nreg = sh.nreg; prm.nslots = sh.nslots;
  prm.parts = sh.parts; prm.rows_pp = sh.rows_pp;
  prm.ring = sh.ring; prm.images = images; prm.slabs_per_head = (int)(rp / 128); prm.slabs = (int64_t)bh * (rp / 128);
  prm.rp = rp; prm.in = in; prm.out = out;
  prm.src = static_cast<const __nv_bfloat16*>(src);
  prm.dst = static_cast<__nv_bfloat16*>(dst);
  prm.status = status;
  // regular lines: (entry, lo, hi, image, head); a size-one dimension keeps its stride valid
  CUtensorMap tm_reg, tm_vert;
  {
    const int64_t sizes[4] = {q, q, images, bh};
    const int64_t strides[4] = {in.s_lo, in.s_hi, images > 1 ? in.s_img : in.rows_per_head, in.rows_per_head};
    const int box[4] = {q, sh.sps, 1, 1};
    if (!radon_map(&tm_reg, src, rp, 5, sizes, strides, box)) return cudaErrorInvalidValue;
  }
  if (in_has_extra) {   // extra class: (entry, lo, image, head), rows v0 + image*sv_img + lo*sv_lo
    const bool per_image = in.sv_img != 0;
    const int64_t sizes[3] = {q, per_image ? images : 1, bh};
    const int64_t strides[3] = {in.sv_lo, per_image ? in.sv_img : in.rows_per_head, in.rows_per_head};
    const int box[3] = {q, 1, 1};
    if (!radon_map(&tm_vert, static_cast<const __nv_bfloat16*>(src) + (int64_t)in.v0 * rp, rp, 4, sizes, strides, box))
      return cudaErrorInvalidValue;
    prm.in.sv_img = per_image ? 1 : 0;   // the kernel passes image * sv_img as the coordinate
  } else {
    tm_vert = tm_reg;
  }
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  int64_t ctas = (int64_t)(sms / sh.parts) * sh.parts;
  const int64_t items = prm.slabs * images * sh.parts;
  if (items < ctas) ctas = items;
  cudaError_t err = cudaFuncSetAttribute(radon_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, sh.smem);
  if (err != cudaSuccess) return err;
  radon_tc_kernel<<<(unsigned)ctas, RADON_THREADS, sh.smem, st>>>(tm_reg, tm_vert, prm);
  return cudaGetLastError();
}

}  // namespace

// 1 when the tensor-core tabulation covers this geometry (d = 3 or 4, q small enough for a resident R).
int smat_tabulate_tc_supported(const SmatGeo& geo, int64_t state_elems) {
  if (geo.D != 2 && geo.D != 3) return 0;
  if (state_elems % 128) return 0;
  const int qq = geo.q * geo.q;
  RadonShape a, b;
  return radon_encode_fn() && radon_shape(geo.q, 0, qq + geo.q, &a) && radon_shape(geo.q, 1, qq, &b) ? 1 : 0;
}

// Rows (of state_elems bf16 each, per head) of the intermediate table the d = 4 stages exchange.
int64_t smat_tabulate_tc_scratch_rows(const SmatGeo& geo) {
  return geo.D == 3 ? (int64_t)geo.q * geo.q * geo.q + (int64_t)geo.q * geo.q : 0;
}

// transpose = 0: in = F [bh][P][rp] bf16, out = U [bh][B][rp] bf16.  transpose = 1: in = Ū [bh][B][rp], out = F̄ [bh][P][rp].
// scratch: [bh][smat_tabulate_tc_scratch_rows][rp] bf16 (d = 4 only).  One launch for d = 3, two for d = 4.
cudaError_t smat_launch_tabulate_tc(const void* in, void* out, void* scratch, const SmatGeo& geo, int64_t state_elems,
                                    int bh, int transpose, int* status, cudaStream_t st, int* launches) {
  const int q = geo.q, qq = q * q, qqq = qq * q;
  *launches = 0;
  if (geo.D == 2) {
    const RadonSide pts = side(qq, 1, q, 0, geo.P);
    const RadonSide typ = side(qq + q, 1, q, 0, geo.B, qq, 1, 0, 0);
    *launches = 1;
    return transpose ? launch_radon(q, 1, 1, typ, pts, in, out, state_elems, bh, status, st)
                     : launch_radon(q, 0, 1, pts, typ, in, out, state_elems, bh, status, st);
  }
  if (geo.D != 3) return cudaErrorInvalidValue;
  const int64_t wrows = smat_tabulate_tc_scratch_rows(geo);
  const RadonSide f_side = side(qq, 1, qq, q, geo.P);                       // image x2, points (x1, x3)
  const RadonSide w1_side = side(qq + q, 1, qq, q, wrows, qqq, q, 1, 0);    // (u, a3) -> W[a3][x2][u]; extra class -> G[x3][x2]
  const RadonSide w2_side = side(qq, 1, q, qq, wrows);                      // image a3 (image q: G), points (u, x2)
  const RadonSide u_side = side(qq + q, 1, q, qq, geo.B, qqq + qq, 1, 0, q);
  cudaError_t err;
  *launches = 2;
  if (!transpose) {
    err = launch_radon(q, 0, q, f_side, w1_side, in, scratch, state_elems, bh, status, st);
    if (err != cudaSuccess) return err;
    return launch_radon(q, 0, q + 1, w2_side, u_side, scratch, out, state_elems, bh, status, st);
  }
  err = launch_radon(q, 1, q + 1, u_side, w2_side, in, scratch, state_elems, bh, status, st);
  if (err != cudaSuccess) return err;
  return launch_radon(q, 1, q, w1_side, f_side, scratch, out, state_elems, bh, status, st);
}
