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
// a CTA owns up to 128 output indices (its part of R; the output indices are split over `parts` CTAs, in whole
// lines where these fit, that then share every image) and applies them to every item it is given:
//   warps 0-3      : build the CTA's part of R once and move it to tensor memory (lane = output index, one column
//                    per two operand rows), where the MMAs read it as their A operand
//   warp 16 lane 0 : TMA producer; a ring slot holds `sps` lines (fixed hi, all lo) of the image x 128 state entries
//                    (MN-major B operand, two boxes of 64 entries); the extra class travels in a slot of its own
//   warps 17, 18 (lane 0) : MMA issuers, alternating items: D[128 outputs, 128 entries] += R_slot * B_slot; up to
//                    four accumulators in flight
//   warps 0-15     : epilogue, one output index (TMEM lane) per thread and one 32-entry column chunk per warp:
//                    round to bf16 and store 64 contiguous bytes of the output row as two 32-byte sectors
//   warps 19, 20   : q = 11 only.  q^2 + q = 132 output indices are one tile of 128 and 4 left over, all of the extra
//                    class (the sum of one line's q rows): these warps add them up from the ring slot itself, so
//                    that one CTA covers an image instead of two CTAs loading it twice
// d = 4 with q <= 11: both stages in ONE launch, slab by slab.  Stage 2 of a slab needs stage 1 of every image of the
// same slab and nothing else, so a CTA keeps the slab's W rows in a private exchange buffer (q^3 + q^2 rows of 128
// entries, rewritten for every slab, stored and loaded with the L2 evict-last priority while F and U stream with
// evict-first) and the full-size W table is never built.  The storing warps make the slab's rows visible (memory
// fence, proxy fence) and arrive on a barrier the producer waits on before the first stage-2 load.
// q = 11 also sends its output tiles off by TMA: the epilogue writes the rounded tile into the item's own ring slot
// (as large as a tile, and dead once the MMAs have read it) in the box layout, and lane 0 of warp 18 issues the tile
// stores and frees the slot; the bulk of the stores bypasses the LSU.
// The kernel exists twice: radon_tc_kernel<false> for one stage per launch with every index through the MMAs (q = 13,
// 17, 19 and the small primes), without cache hints, phase tables or ALU warps; radon_tc_kernel<true> with them.
// (The tile-store path is written for several slots per item and several parts and is compiled into both, but the
// launcher switches it on for q = 11 only: it was measured slower than the direct stores for q = 13 and 17.)
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
constexpr int ALU_WARP = MMA_WARP + MMA_WARPS;    // first of the warps that sum the leftover extra-class rows
constexpr int ALU_WARPS = 2;
constexpr int ALU_MAX_ROWS = 8;
constexpr int RADON_THREADS = 32 * (ALU_WARP + ALU_WARPS);
constexpr int MAX_ACC = 4;                        // accumulators in flight: what the R columns leave of 512, at most 4
constexpr int RADON_EXCHANGE_CTAS = 148;          // CTAs of a one-launch two-stage tabulation (one exchange slab each)
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

// One stage: input and output index spaces, and where the rows live.  A "private" table is the exchange buffer of the
// two-stage kernel: [CTA][rows_per_head][128 entries], one slab per CTA, rewritten for every slab so that it stays in L2.
struct RadonPhase {
  RadonSide in, out;
  int32_t images;
  int32_t src_private, dst_private;
  int32_t src_heads;               // extent of the source maps' last coordinate: one past it reads zeros
  int64_t dst_pitch;               // entries per row of dst
  __nv_bfloat16* dst;
};

struct RadonParams {
  int32_t q, transpose;
  int32_t sps, sr;                 // lines (hi values) per ring slot; rows of a slot = sps*q rounded up to 16
  int32_t nreg, nslots;            // slots of regular lines per image; plus one when the input has the extra class
  int32_t parts, rows_pp;          // CTAs sharing an image, and output indices per CTA (<= 128)
  int32_t alu_rows;                // output indices parts*rows_pp .. (all of the extra class) summed on the ALUs by the
                                   // last part, straight from the ring slot; 0: every index goes through the MMAs
  int32_t ring;                    // ring slots
  int32_t tma_out;                 // the output tile leaves through the item's own ring slot and TMA stores (q = 11)
  int32_t mini_bytes;              // tma_out: per slot, room for the extra-class rows of the tile (two halves); 0: the
                                   // extra-class rows of a part sit in the tile itself, after its regular lines
  int32_t lines_pp;                // tma_out: regular lines per tile (the store box; lines past q - 1 are clipped)
  int32_t nph;                     // 1, or 2: both stages of the d = 4 tabulation, slab by slab
  int32_t slabs_per_head;          // rp / 128
  int64_t slabs;                   // heads * slabs_per_head
  RadonPhase ph[2];
  int* status;
};

// The items of one CTA, in the order every role walks them.  One phase: item = (slab, image) with the slab index
// fastest over the whole grid.  Two phases: slab by slab, the images of phase 0 and then those of phase 1, whose input
// is what phase 0 wrote for the same slab.
struct ItemIter {
  uint32_t slab, img, ph, left;    // the current item, and the items left including it
  uint32_t step, slabs, nph, im0, im1;
  __device__ __forceinline__ ItemIter(const RadonParams& p, uint32_t first, uint32_t step_, uint32_t nph_) {
    step = step_; slabs = (uint32_t)p.slabs; nph = nph_;
    im0 = (uint32_t)p.ph[0].images; im1 = nph > 1 ? (uint32_t)p.ph[1].images : 0u;
    ph = 0;
    if (nph == 1) {
      const uint32_t total = slabs * im0;                       // < 2^31 (checked by the launcher)
      left = first < total ? (total - 1 - first) / step + 1 : 0;
      img = first / slabs; slab = first - img * slabs;
    } else {
      left = first < slabs ? ((slabs - 1 - first) / step + 1) * (im0 + im1) : 0;
      img = 0; slab = first;
    }
  }
  __device__ __forceinline__ void next() {
    --left;
    if (nph == 1) {
      slab += step;
      while (slab >= slabs) { slab -= slabs; ++img; }
    } else if (++img == (ph ? im1 : im0)) {
      img = 0;
      if (ph == 0) ph = 1; else { ph = 0; slab += step; }
    }
  }
  // last item of phase 0 of a slab: phase 1 may start once its output is visible
  __device__ __forceinline__ bool closes_phase0() const { return nph > 1 && ph == 0 && img + 1 == im0; }
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
    if (p.ph[0].in.count > q * q) row[operand_row(p, q, y)] = one;
  }
}

// box of 64 state entries x q rows x sps lines (regular map) or 64 x q rows (extra-class map)
__device__ __forceinline__ void tma_load_5d(void* smem_dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                            int c4, uint64_t* bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4, %5, %6}], [%7], %8;"
      ::"r"(smem_u32(smem_dst)), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(smem_u32(bar)), "l"(pol)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d(void* smem_dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                            uint64_t* bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4, %5}], [%6], %7;"
      ::"r"(smem_u32(smem_dst)), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(smem_u32(bar)), "l"(pol)
      : "memory");
}

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

// L2 eviction policies: the exchange rows of the two-stage kernel should stay in the cache (they are rewritten for
// every slab, and written back to memory only when evicted), the tables streaming past them should leave it first.
enum { POLICY_NORMAL = 0, POLICY_FIRST = 1, POLICY_LAST = 2 };
__device__ __forceinline__ uint64_t l2_policy(int kind) {
  uint64_t p;
  if (kind == POLICY_FIRST) asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  else if (kind == POLICY_LAST) asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  else asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void st_global_v8_hint(void* dst, uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3,
                                                  uint32_t w4, uint32_t w5, uint32_t w6, uint32_t w7, uint64_t pol) {
  asm volatile("st.global.L2::cache_hint.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8}, %9;" ::"l"(dst), "r"(w0),
               "r"(w1), "r"(w2), "r"(w3), "r"(w4), "r"(w5), "r"(w6), "r"(w7), "l"(pol)
               : "memory");
}
__device__ __forceinline__ void st_global_v4_hint(void* dst, uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3,
                                                  uint64_t pol) {
  asm volatile("st.global.L2::cache_hint.v4.b32 [%0], {%1, %2, %3, %4}, %5;" ::"l"(dst), "r"(w0), "r"(w1), "r"(w2),
               "r"(w3), "l"(pol)
               : "memory");
}

// Tile stores: shared memory (box layout, 128-byte swizzle) -> global, as one bulk group per item.
__device__ __forceinline__ void tma_store_5d(const CUtensorMap* map, const void* smem_src, int c0, int c1, int c2, int c3,
                                             int c4, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.5d.global.shared::cta.bulk_group.L2::cache_hint [%0, {%2, %3, %4, %5, %6}], [%1], %7;"
      ::"l"(map), "r"(smem_u32(smem_src)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "l"(pol)
      : "memory");
}
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, const void* smem_src, int c0, int c1, int c2, int c3,
                                             uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.4d.global.shared::cta.bulk_group.L2::cache_hint [%0, {%2, %3, %4, %5}], [%1], %6;"
      ::"l"(map), "r"(smem_u32(smem_src)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(pol)
      : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

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

// FEAT = false is the plain instantiation (one stage per launch, every index through the MMAs, direct stores, no cache
// hints): the single-thread roles pay for every instruction, and the prime-specific paths would cost the others time.
template <bool FEAT>
__global__ void __launch_bounds__(RADON_THREADS, 1) radon_tc_kernel(const __grid_constant__ CUtensorMap tm_reg0,
                                                                    const __grid_constant__ CUtensorMap tm_vert0,
                                                                    const __grid_constant__ CUtensorMap tm_reg1,
                                                                    const __grid_constant__ CUtensorMap tm_vert1,
                                                                    const __grid_constant__ CUtensorMap tm_oreg0,
                                                                    const __grid_constant__ CUtensorMap tm_overt0,
                                                                    const __grid_constant__ CUtensorMap tm_oreg1,
                                                                    const __grid_constant__ CUtensorMap tm_overt1,
                                                                    const RadonParams prm) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int q = prm.q;
  const int slot_bytes = prm.sr * 256;                          // two 64-entry blocks of sr rows x 128 bytes
  const int kt = prm.nslots * prm.sr;                           // operand rows per image
  uint8_t* sRing = smem;
  uint8_t* sMini = sRing + prm.ring * slot_bytes;                                  // [ring] extra-class rows (tma_out)
  int32_t* out_tab = reinterpret_cast<int32_t*>(sMini + prm.ring * prm.mini_bytes);  // [2][128]
  uint64_t* bars = reinterpret_cast<uint64_t*>(out_tab + 2 * TILE_ROWS);
  uint64_t* full = bars;                    // [ring] slot filled (TMA bytes)
  uint64_t* empty = bars + prm.ring;        // [ring] slot consumed by the MMAs (arrival from the epilogue, once the item is complete)
  uint64_t* acc_full = empty + prm.ring;    // [MAX_ACC] accumulator complete
  uint64_t* acc_empty = acc_full + MAX_ACC; // [MAX_ACC] accumulator read out (one arrival per epilogue warp)
  uint64_t* w_ready = acc_empty + MAX_ACC;  // phase 0 of the current slab written out (one arrival per storing warp)
  uint64_t* staged = w_ready + 1;           // [ring] tma_out: an item's tile is complete in its first slot (one arrival per
                                            // epilogue warp); indexed by the item count modulo the ring size
  uint64_t* alu_done = staged + prm.ring;   // [ring] tma_out: the ALU warps have read the slot and written their rows
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(alu_done + prm.ring);
  volatile int* cta_abort = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const WaitCtx wc{cta_abort, prm.status};
  const int part = blockIdx.x % prm.parts;
  const bool alu_here = FEAT && prm.alu_rows > 0 && part == prm.parts - 1;
  const bool tma_out = prm.tma_out != 0;
  const uint32_t nph = FEAT ? (uint32_t)prm.nph : 1u;

  if (threadIdx.x == 0) {
    *cta_abort = 0;
    for (int s = 0; s < prm.ring; ++s) {
      mbar_init(full + s, 1);
      mbar_init(empty + s, tma_out ? 1 : (alu_here ? 1 + ALU_WARPS : 1));   // tma_out: the storing thread frees the slot
      mbar_init(alu_done + s, ALU_WARPS);
      mbar_init(staged + s, EPI_WARPS);
    }
    for (int b = 0; b < MAX_ACC; ++b) { mbar_init(acc_full + b, 1); mbar_init(acc_empty + b, EPI_WARPS); }
    mbar_init(w_ready, tma_out ? 1 : (alu_here ? EPI_WARPS + ALU_WARPS : EPI_WARPS));

    fence_barrier_init();
    prefetch_tmap(&tm_reg0);
    prefetch_tmap(&tm_vert0);
    if (nph > 1) { prefetch_tmap(&tm_reg1); prefetch_tmap(&tm_vert1); }
  }
  if (warp == MMA_WARP) tmem_alloc(tmem_slot, 512);
  // This CTA's part of R, built row by row in the (still unused) ring and moved to tensor memory: lane = output
  // index, one column per two operand rows.  The launcher guarantees ring * slot_bytes >= 128 * kt * 2.
  __nv_bfloat16* scratch = reinterpret_cast<__nv_bfloat16*>(sRing);
  for (int c = threadIdx.x; c < prm.ring * (slot_bytes + prm.mini_bytes) / 16; c += blockDim.x)
    reinterpret_cast<uint4*>(sRing)[c] = make_uint4(0u, 0u, 0u, 0u);
  for (int n = threadIdx.x; n < TILE_ROWS; n += blockDim.x)
    for (int h = 0; h < (int)nph; ++h)
      out_tab[h * TILE_ROWS + n] = n < prm.rows_pp ? side_row(prm.ph[h].out, part * prm.rows_pp + n, q) : ROW_INVALID;
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t r_cols = (uint32_t)((kt / 2 + 31) & ~31);       // columns taken by R
  const uint32_t nacc = min(MAX_ACC, (int)((512 - r_cols) / 128));
  if (warp < 4) {
    const int n = warp * 32 + lane;
    __nv_bfloat16* row = scratch + (size_t)n * kt;
    if (n < prm.rows_pp && part * prm.rows_pp + n < prm.ph[0].out.count) mark_incident(prm, part * prm.rows_pp + n, row);
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

  // per phase: streaming tables, or the exchange rows (two-stage kernel only)
  const uint64_t pol_src0 = l2_policy(nph > 1 ? (prm.ph[0].src_private ? POLICY_LAST : POLICY_FIRST) : POLICY_NORMAL);
  const uint64_t pol_src1 = l2_policy(nph > 1 ? (prm.ph[1].src_private ? POLICY_LAST : POLICY_FIRST) : POLICY_NORMAL);
  const uint64_t pol_dst0 = l2_policy(nph > 1 ? (prm.ph[0].dst_private ? POLICY_LAST : POLICY_FIRST) : POLICY_NORMAL);
  const uint64_t pol_dst1 = l2_policy(nph > 1 ? (prm.ph[1].dst_private ? POLICY_LAST : POLICY_FIRST) : POLICY_NORMAL);
  // items of this CTA: same part always
  const uint32_t first = blockIdx.x / prm.parts, step = gridDim.x / prm.parts;
  const uint32_t sph = (uint32_t)prm.slabs_per_head;

  // ---- storing thread (tma_out): one bulk group of tile stores per item; the item's first slot, which holds the tile,
  // goes back to the producer when the stores have read it.  Lane 0 of the second MMA warp when every item is one
  // slot (that warp has no items then), else lane 0 of warp 19.
  auto store_role = [&]() {
    const uint32_t ring = (uint32_t)prm.ring;
    uint32_t slot = 0, prev_slot = 0;
    uint32_t sidx = 0, spar = 0;                                // the item's "staged" barrier (items mod ring) and its parity
    bool have_prev = false;
    const int hi0 = part * prm.lines_pp;                        // first regular line of this CTA's tiles
    const int xrow0 = q * q - part * prm.rows_pp;               // tile row of the first extra-class index
    for (ItemIter it(prm, first, step, nph); it.left; it.next()) {
      const RadonPhase& ph = FEAT ? prm.ph[it.ph] : prm.ph[0];
      const CUtensorMap* oreg = FEAT && it.ph ? &tm_oreg1 : &tm_oreg0;
      const CUtensorMap* overt = FEAT && it.ph ? &tm_overt1 : &tm_overt0;
      const uint32_t head = it.slab / sph;
      const int e0 = ph.dst_private ? 0 : (int)(it.slab - head * sph) * 128;
      const int hc = ph.dst_private ? (int)blockIdx.x : (int)head;
      const uint64_t pol = it.ph ? pol_dst1 : pol_dst0;
      if (!mbar_wait(staged + sidx, spar, wc)) break;
      if (++sidx == ring) { sidx = 0; spar ^= 1; }
      const uint8_t* tile = sRing + slot * slot_bytes;
      if (hi0 < q) {
        tma_store_5d(oreg, tile, e0, 0, hi0, (int)it.img, hc, pol);
        tma_store_5d(oreg, tile + prm.sr * 128, e0 + 64, 0, hi0, (int)it.img, hc, pol);
      }
      if (ph.out.count > q * q && xrow0 < prm.rows_pp && (int)it.img >= ph.out.vert_from) {
        const int ci = ph.out.sv_img != 0 ? (int)it.img : 0;   // the map's image stride is sv_img rows
        if (prm.mini_bytes) {
          const uint8_t* mini = sMini + slot * prm.mini_bytes;
          tma_store_4d(overt, mini, e0, 0, ci, hc, pol);
          tma_store_4d(overt, mini + prm.mini_bytes / 2, e0 + 64, 0, ci, hc, pol);
        } else {
          tma_store_4d(overt, tile + xrow0 * 128, e0, 0, ci, hc, pol);
          tma_store_4d(overt, tile + prm.sr * 128 + xrow0 * 128, e0 + 64, 0, ci, hc, pol);
        }
      }
      bulk_commit();
      if (have_prev) {
        bulk_wait_read<1>();
        mbar_arrive(empty + prev_slot);
      }
      if (it.closes_phase0()) {   // the slab's stage-1 rows are in memory before the producer loads them back
        bulk_wait_all();
        fence_proxy_async_all();
        mbar_arrive(empty + slot);
        mbar_arrive(w_ready);
        have_prev = false;
      } else {
        prev_slot = slot;
        have_prev = true;
      }
      slot += (uint32_t)prm.nslots;
      if (slot >= ring) slot -= ring;
    }
    if (have_prev) { bulk_wait_read<0>(); mbar_arrive(empty + prev_slot); }
    bulk_wait_all();
  };

  if (warp == PROD_WARP && lane == 0) {
    // ---- TMA producer -----------------------------------------------------------------------------------------
    // The two single-thread roles keep running slot / parity counters: a lone thread pays the full latency of every
    // instruction, so divisions by the ring size inside the loop would show in the kernel time.
    uint32_t slot = 0, par = 0;                               // ring position; parity of the empty barrier's phase to wait for
    uint32_t wpar = 0;                                        // parity of w_ready for the current slab
    bool first_lap = true, ok = true;
    const uint32_t reg_bytes = 2u * 128u * (uint32_t)(q * prm.sps), vert_bytes = 2u * 128u * (uint32_t)q;
    for (ItemIter it(prm, first, step, nph); it.left && ok; it.next()) {
      const RadonPhase& ph = FEAT ? prm.ph[it.ph] : prm.ph[0];
      const CUtensorMap* tm_reg = FEAT && it.ph ? &tm_reg1 : &tm_reg0;
      const CUtensorMap* tm_vert = FEAT && it.ph ? &tm_vert1 : &tm_vert0;
      const uint32_t head = it.slab / sph;
      const int e0 = ph.src_private ? 0 : (int)(it.slab - head * sph) * 128;
      const int hc = ph.src_private ? (int)blockIdx.x : (int)head;
      const uint64_t pol = it.ph ? pol_src1 : pol_src0;
      if (it.ph == 1 && it.img == 0) {   // this slab's phase 0 output is complete and visible to the copy engine
        ok = mbar_wait(w_ready, wpar, wc);
        wpar ^= 1;
        fence_proxy_async_all();
        if (!ok) break;
      }
      for (int g = 0; g < prm.nslots; ++g) {
        if (!first_lap) ok = mbar_wait(empty + slot, par, wc);
        if (!ok) break;
        uint8_t* dst = sRing + slot * slot_bytes;
        if (g < prm.nreg) {   // lines hi = g*sps ..; lines past q - 1 are out of bounds and arrive as zeros
          mbar_expect_tx(full + slot, reg_bytes);
          if (FEAT) {
            tma_load_5d(dst, tm_reg, e0, 0, g * prm.sps, (int)it.img, hc, full + slot, pol);
            tma_load_5d(dst + prm.sr * 128, tm_reg, e0 + 64, 0, g * prm.sps, (int)it.img, hc, full + slot, pol);
          } else {
            tma_load_5d(dst, tm_reg, e0, 0, g * prm.sps, (int)it.img, hc, full + slot);
            tma_load_5d(dst + prm.sr * 128, tm_reg, e0 + 64, 0, g * prm.sps, (int)it.img, hc, full + slot);
          }
        } else {              // extra class; an image without it reads past the last head: zeros
          const int h = (int)it.img >= ph.in.vert_from ? hc : ph.src_heads;
          const int ci = (int)it.img * ph.in.sv_img;   // 0 when every image shares the rows
          mbar_expect_tx(full + slot, vert_bytes);
          if (FEAT) {
            tma_load_4d(dst, tm_vert, e0, 0, ci, h, full + slot, pol);
            tma_load_4d(dst + prm.sr * 128, tm_vert, e0 + 64, 0, ci, h, full + slot, pol);
          } else {
            tma_load_4d(dst, tm_vert, e0, 0, ci, h, full + slot);
            tma_load_4d(dst + prm.sr * 128, tm_vert, e0 + 64, 0, ci, h, full + slot);
          }
        }
        if (++slot == (uint32_t)prm.ring) {
          slot = 0;
          if (first_lap) { first_lap = false; par = 0; } else par ^= 1;
        }
      }
    }
  } else if (warp >= MMA_WARP && warp < ALU_WARP && lane == 0) {
    // ---- MMA issuers: the two threads take the items alternately, so that the issue latency of one item (waits,
    // MMAs, commits: more than the tensor pipe needs for it) overlaps with the other thread's item.  Both phases
    // share R and the slot layout, so the issuers only count items. ---------------------------------------------
    const uint32_t me = (uint32_t)(warp - MMA_WARP);
    if (tma_out && me == 1 && prm.nslots == 1) store_role();
    constexpr uint32_t idesc = make_idesc(TILE_ROWS, 128, 0, 1);   // A from tensor memory (R), B MN-major (image rows)
    const uint64_t dB0 = make_desc(smem_u32(sRing), prm.sr * 128, 1024);
    const uint32_t slot16 = (uint32_t)slot_bytes >> 4;            // descriptor address units are 16 bytes
    const uint32_t slot_cols = (uint32_t)prm.sr / 2;              // columns of R per slot
    const int steps = prm.sr / 16, nslots = prm.nslots;
    const int steps_last = ((q - (prm.nreg - 1) * prm.sps) * q + 15) / 16, steps_extra = (q + 15) / 16;
    const uint32_t ring = (uint32_t)prm.ring;
    const uint32_t items = ItemIter(prm, first, step, nph).left;
    uint32_t slot = 0, par = 0;                                   // ring position and the parity its full barrier shows
    uint32_t buf = 0, apar = 0;                                   // accumulator; parity of its empty barrier's phase to wait for
    bool ok = true;
    if (nslots == 1) {
      // One slot per item (q <= 11): a single thread, and the leanest loop: every instruction here is on the
      // critical path of the stage.
      for (uint32_t n_item = 0; me == 0 && n_item < items && ok; ++n_item) {
        if (n_item >= nacc) ok = mbar_wait(acc_empty + buf, apar, wc);
        if (!ok) break;
        ok = mbar_wait(full + slot, par, wc);
        if (!ok) break;
        fence_after_sync();
        issue_slot_steps(steps, tmem_acc + buf * 128, tmem_base, dB0 + (uint64_t)(slot * slot16), idesc, true);
        if (!tma_out) mma_commit(empty + slot);   // tma_out: the storing thread frees the slot once the tile has left it
        mma_commit(acc_full + buf);
        if (++slot == ring) { slot = 0; par ^= 1; }
        if (++buf == nacc) { buf = 0; if (n_item >= nacc) apar ^= 1; }
      }
    } else {
      uint32_t turn = 0;
      for (uint32_t n_item = 0; n_item < items && ok; ++n_item) {
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
          // the last slot of regular lines and the slot of the extra class hold fewer rows than a full slot: R has
          // only zeros for the rest, so their K-steps are left out
          const int st = g + 1 < prm.nreg ? steps : (g < prm.nreg ? steps_last : steps_extra);
          issue_slot_steps(st, tmem_d, tmem_a, dB0 + (uint64_t)(slot * slot16), idesc, g == 0);
          if (++slot == ring) { slot = 0; par ^= 1; }
        }
        if (ok) mma_commit(acc_full + buf);   // the only commit of the item: the epilogue frees its slots when it sees it
        if (++buf == nacc) { buf = 0; if (n_item >= nacc) apar ^= 1; }
      }
    }
  } else if (tma_out && prm.nslots > 1 && warp == ALU_WARP) {
    if (lane == 0) store_role();
  } else if (FEAT && warp >= ALU_WARP) {
    // ---- leftover rows on the ALUs ----------------------------------------------------------------------------
    // q*q + q output indices rarely fill whole tiles of 128.  When only a few are left over, and they belong to the
    // extra class (index q*q + u = the sum of line u's q rows), these warps add the rows up from the slot itself
    // instead of a second, nearly empty tile paying for every MMA again.  A task is one leftover index and 8 state
    // entries (one 16-byte chunk of the swizzled slot); 16 neighbouring tasks store 256 contiguous bytes.
    if (alu_here) {
      const int tid_a = (warp - ALU_WARP) * 32 + lane, tasks = prm.alu_rows * 16;
      const uint32_t ring = (uint32_t)prm.ring;
      uint32_t slot = 0, par = 0;
      for (ItemIter it(prm, first, step, nph); it.left; it.next()) {
        const RadonPhase& ph = FEAT ? prm.ph[it.ph] : prm.ph[0];
        const uint32_t head = it.slab / sph;
        const int e0 = ph.dst_private ? 0 : (int)(it.slab - head * sph) * 128;
        const int64_t hrow = (int64_t)(ph.dst_private ? blockIdx.x : head) * ph.out.rows_per_head;
        if (!mbar_wait_warp(full + slot, par, wc)) break;
        if ((int)it.img >= ph.out.vert_from) {
          const uint8_t* sl = sRing + slot * slot_bytes;
          for (int task = tid_a; task < tasks; task += 32 * ALU_WARPS) {
            const int u = prm.parts * prm.rows_pp + (task >> 4) - q * q, ch = task & 15;
            const uint8_t* blk = sl + (ch >> 3) * prm.sr * 128;
            float acc[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] = 0.f;
            for (int lo = 0; lo < q; ++lo) {
              const int r = u * q + lo;                           // operand row of (line u, lo): one slot holds every line
              const uint4 w = *reinterpret_cast<const uint4*>(blk + r * 128 + (((ch & 7) ^ (r & 7)) << 4));
              acc[0] += __uint_as_float(w.x << 16); acc[1] += __uint_as_float(w.x & 0xffff0000u);
              acc[2] += __uint_as_float(w.y << 16); acc[3] += __uint_as_float(w.y & 0xffff0000u);
              acc[4] += __uint_as_float(w.z << 16); acc[5] += __uint_as_float(w.z & 0xffff0000u);
              acc[6] += __uint_as_float(w.w << 16); acc[7] += __uint_as_float(w.w & 0xffff0000u);
            }
            if (tma_out) {   // into the slot's extra-class rows, from where the storing thread sends them with the tile
              uint8_t* mrow = sMini + slot * prm.mini_bytes + (ch >> 3) * (prm.mini_bytes / 2) + u * 128;
              *reinterpret_cast<uint4*>(mrow + (((ch & 7) ^ (u & 7)) << 4)) =
                  make_uint4(pack_bf16(acc[0], acc[1]), pack_bf16(acc[2], acc[3]), pack_bf16(acc[4], acc[5]),
                             pack_bf16(acc[6], acc[7]));
            } else {
              const int row = ph.out.v0 + (int)it.img * ph.out.sv_img + u * ph.out.sv_lo;
              __nv_bfloat16* dst = ph.dst + (hrow + row) * ph.dst_pitch + e0 + ch * 8;
              st_global_v4_hint(dst, pack_bf16(acc[0], acc[1]), pack_bf16(acc[2], acc[3]), pack_bf16(acc[4], acc[5]),
                                pack_bf16(acc[6], acc[7]), it.ph ? pol_dst1 : pol_dst0);
            }
          }
        }
        if (tma_out) {
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) mbar_arrive(alu_done + slot);
          if (++slot == ring) { slot = 0; par ^= 1; }
          continue;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty + slot);
        if (it.closes_phase0()) {   // what this warp stored for the slab is ordered before the copy engine's reads
          __threadfence();
          fence_proxy_async_all();
          __syncwarp();
          if (lane == 0) mbar_arrive(w_ready);
        }
        if (++slot == ring) { slot = 0; par ^= 1; }
      }
    }
  } else if (warp < EPI_WARPS) {
    // ---- epilogue ---------------------------------------------------------------------------------------------
    // Warp w reads lane quarter w % 4 (32 output indices) and the 32-entry column chunk w / 4 of every item.
    const int qd = warp & 3, cb = warp >> 2;
    const int orow = qd * 32 + lane;                            // output index of this CTA = TMEM lane
    const uint32_t lane_base = (uint32_t)(qd * 32) << 16;
    const int tv0 = out_tab[orow], tv1 = nph > 1 ? out_tab[TILE_ROWS + orow] : ROW_INVALID;
    const bool active = qd * 32 < prm.rows_pp;                  // warp-uniform: some output index in these lanes
    uint32_t buf = 0, apar = 0, eslot = 0, epar = 0, sidx = 0;
    // tma_out: where this thread's 64 bytes go inside the slot (or inside the slot's extra rows)
    const bool st_mini = prm.mini_bytes != 0 && part * prm.rows_pp + orow >= q * q;
    const int st_idx = st_mini ? part * prm.rows_pp + orow - q * q : orow;
    const int st_off = (cb >> 1) * (st_mini ? prm.mini_bytes / 2 : prm.sr * 128) + st_idx * 128;
    for (ItemIter it(prm, first, step, nph); it.left; it.next()) {
      const RadonPhase& ph = FEAT ? prm.ph[it.ph] : prm.ph[0];
      const uint32_t head = it.slab / sph;
      const int e0 = ph.dst_private ? 0 : (int)(it.slab - head * sph) * 128;
      const int64_t hrow = (int64_t)(ph.dst_private ? blockIdx.x : head) * ph.out.rows_per_head;
      const int tv = it.ph ? tv1 : tv0;
      if (!mbar_wait_warp(acc_full + buf, apar, wc)) break;
      fence_after_sync();
      if (tma_out) {
        // The tile leaves through the item's own slot (the MMAs are done with it): every thread writes its 64 bytes
        // in the box layout of a TMA tile — regular indices into the slot (row = index), extra-class indices into
        // the slot's extra rows — and the storing thread sends the tile off.  The LSU sees 4 wavefronts per warp
        // store instead of 32, and the bulk of the traffic bypasses it.
        uint32_t v[32];
        tmem_ld32(tmem_acc + lane_base + buf * 128 + cb * 32, v);
        tmem_ld_wait();
        fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(acc_empty + buf);             // the accumulator is in registers
        if (alu_here && !mbar_wait_warp(alu_done + eslot, epar, wc)) break;   // the ALU warps have read the image
        if (prm.nslots > 1) {                                     // the item's other slots are free already
          if (warp == 0 && lane == 0)
            for (int g = 1; g < prm.nslots; ++g) {
              uint32_t sl = eslot + g; if (sl >= (uint32_t)prm.ring) sl -= (uint32_t)prm.ring;
              mbar_arrive(empty + sl);
            }
          __syncwarp();
        }
        if (tv != ROW_INVALID) {
          // regular indices and, without extra rows of their own, the extra-class indices of the part: tile row =
          // TMEM lane; with extra rows per slot (q = 11) the extra-class indices go there
          const int idx = st_idx;
          uint8_t* trow = (st_mini ? sMini + eslot * prm.mini_bytes : sRing + eslot * slot_bytes) + st_off;
#pragma unroll
          for (int j = 0; j < 4; ++j)
            *reinterpret_cast<uint4*>(trow + ((((cb & 1) * 4 + j) ^ (idx & 7)) << 4)) =
                make_uint4(pack_bf16(__uint_as_float(v[8 * j]), __uint_as_float(v[8 * j + 1])),
                           pack_bf16(__uint_as_float(v[8 * j + 2]), __uint_as_float(v[8 * j + 3])),
                           pack_bf16(__uint_as_float(v[8 * j + 4]), __uint_as_float(v[8 * j + 5])),
                           pack_bf16(__uint_as_float(v[8 * j + 6]), __uint_as_float(v[8 * j + 7])));
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(staged + sidx);   // one barrier per item in flight: at most `ring` of them
        if (++sidx == (uint32_t)prm.ring) sidx = 0;
        eslot += (uint32_t)prm.nslots;
        if (eslot >= (uint32_t)prm.ring) { eslot -= (uint32_t)prm.ring; epar ^= 1; }
        if (++buf == nacc) { buf = 0; apar ^= 1; }
        continue;
      }
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
        const bool vert = (int)it.img >= ph.out.vert_from;
        if (tv != ROW_INVALID && (!(tv & ROW_VERT) || vert)) {
          const int row = (tv & ROW_VERT) ? ph.out.v0 + (int)it.img * ph.out.sv_img + (tv & ~ROW_VERT)
                                          : (int)it.img * ph.out.s_img + tv;
          __nv_bfloat16* dst = ph.dst + (hrow + row) * ph.dst_pitch + e0 + cb * 32;
#pragma unroll
          for (int h8 = 0; h8 < 2; ++h8) {   // two whole 32-byte sectors per thread
            uint32_t w[8];
#pragma unroll
            for (int i = 0; i < 8; ++i)
              w[i] = pack_bf16(__uint_as_float(v[16 * h8 + 2 * i]), __uint_as_float(v[16 * h8 + 2 * i + 1]));
            if (FEAT)
              st_global_v8_hint(dst + 16 * h8, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7], it.ph ? pol_dst1 : pol_dst0);
            else
              st_global_v8(dst + 16 * h8, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]);
          }
        }
      }
      fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty + buf);
      if (it.closes_phase0()) {   // as for the ALU warps: the slab's phase 0 rows before the copy engine reads them
        __threadfence();
        fence_proxy_async_all();
        __syncwarp();
        if (lane == 0) mbar_arrive(w_ready);
      }
      if (++buf == nacc) { buf = 0; apar ^= 1; }
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
  int sps, sr, nreg, nslots, parts, rows_pp, alu_rows, ring, smem;
};

// Ring slots of `sps` lines (sps*q rows, rounded up to 16), chosen for the least MMA work; the output indices are
// split evenly over `parts` CTAs of at most 128 each.  R (128 lanes x one column per two operand rows) and at least
// two accumulators of 128 columns must fit the 512 columns of tensor memory, and the ring must be able to hold the
// scratch copy of R while it is built.  Returns false when q is too large for this kernel.
bool radon_shape(int q, int transpose, int in_has_extra, int count_out, RadonShape* s) {
  const int budget = 227 * 1024 - 1024 - 512 - TILE_ROWS * 8;
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
      s->rows_pp = (count_out + parts - 1) / parts; s->alu_rows = 0; s->ring = ring;
      s->smem = ring * slot_bytes + TILE_ROWS * 8 + 512 + 1024;
    }
  }
  if (best == (1 << 30)) return false;
  {   // whole lines per part where they fit: a part's tile can then leave as one box of lines
    const int lines = count_out / q, lpp = (lines + s->parts - 1) / s->parts;
    if (count_out % q == 0 && lpp * q <= TILE_ROWS) s->rows_pp = lpp * q;
  }
  // A few indices past the last full tile, all of the extra class, with every line in one slot: full tiles for the
  // MMAs and the rest on the ALUs (q = 11: 132 = 128 + 4 indices, one CTA per image instead of two).
  const int left = count_out % TILE_ROWS, whole = count_out - left;
  if (!transpose && !in_has_extra && s->nslots == 1 && s->sps >= q && whole > 0 && left > 0 && left <= ALU_MAX_ROWS &&
      whole >= q * q) {
    s->parts = whole / TILE_ROWS; s->rows_pp = TILE_ROWS; s->alu_rows = left;
  }
  return true;
}

// The shared-memory map of radon_tc_kernel for a shape, checked on the host before every launch: ring slots, the
// per-slot extra-class rows (tile stores only), the output-row table and the barrier words must be disjoint and inside
// the allocation; nothing the copy engine or a thread writes for a slot may leave the slot.
//   [0, ring * slot)                      ring slots, slot = 2 halves of sr rows x 128 bytes (1024-byte aligned: sr % 16 == 0)
//   [.., + ring * mini)                   extra-class rows per slot (two halves of mini / 2)
//   [.., + 2 * 128 * 4)                   output-row table
//   [.., + (4 ring + 2 MAX_ACC + 1) * 8 + 8)   barriers, the tensor-memory slot word, the abort flag
bool radon_layout_ok(int q, const RadonShape& sh, int ring, int mini_bytes, int tma_out, int in_has_extra, int smem) {
  const int slot = sh.sr * 256, half = sh.sr * 128;
  const int bars = (4 * ring + 2 * MAX_ACC + 1) * 8 + 8;
  bool ok = sh.sr % 16 == 0 && sh.sr <= TILE_ROWS && ring >= sh.nslots;           // the scratch copy of R: 128 rows x kt bf16
  ok = ok && sh.nslots == sh.nreg + (in_has_extra ? 1 : 0) && sh.nreg * sh.sps >= q;
  ok = ok && q * sh.sps * 128 <= half && q * 128 <= half;                         // a load box (lines or extra class) per half
  ok = ok && ((sh.nslots * sh.sr / 2 + 31) & ~31) + 2 * 128 <= 512;               // R columns and two accumulators
  ok = ok && sh.rows_pp <= TILE_ROWS && sh.parts * sh.rows_pp + sh.alu_rows >= 0;
  if (tma_out) {   // the tile is written into the item's first slot: one 128-byte row per output index of the part
    ok = ok && sh.rows_pp <= sh.sr;
    ok = ok && (mini_bytes == 0 || (mini_bytes % 2048 == 0 && mini_bytes / 2 >= q * 128));
  }
  ok = ok && 1023 + ring * (slot + mini_bytes) + 2 * TILE_ROWS * 4 + bars <= smem && smem <= 227 * 1024;
  return ok;
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

// One stage as the host states it; src / dst are whole tables [bh][rows_per_head][rp], or the private exchange buffer.
struct StageSpec {
  RadonSide in, out;
  int images;
  const void* src;
  void* dst;
  bool src_private, dst_private;
};

StageSpec stage(const RadonSide& in, const RadonSide& out, int images, const void* src, void* dst, bool src_private = false,
                bool dst_private = false) {
  StageSpec s;
  s.in = in; s.out = out; s.images = images; s.src = src; s.dst = dst; s.src_private = src_private; s.dst_private = dst_private;
  return s;
}

// nph = 1: one stage over the whole tables.  nph = 2: both stages in one launch, which must share R (the same
// direction, the same index counts) and exchange their rows through the private buffer.
cudaError_t launch_radon(int q, int transpose, int nph, const StageSpec* sp, int64_t rp, int bh, int* status,
                         cudaStream_t st) {
  RadonShape sh;
  const int in_has_extra = sp[0].in.count > q * q;
  int max_images = sp[0].images;
  if (nph == 2 && sp[1].images > max_images) max_images = sp[1].images;
  if (!radon_shape(q, transpose, in_has_extra, sp[0].out.count, &sh) || rp % 128 ||
      (int64_t)bh * (rp / 128) * max_images * 2 >= (1LL << 31))
    return cudaErrorInvalidValue;
  if (nph == 2 && (sh.parts != 1 || sp[1].in.count != sp[0].in.count || sp[1].out.count != sp[0].out.count))
    return cudaErrorInvalidValue;
  RadonParams prm;
  prm.q = q; prm.transpose = transpose; prm.sps = sh.sps; prm.sr = sh.sr; prm.nreg = sh.nreg; prm.nslots = sh.nslots;
  prm.parts = sh.parts; prm.rows_pp = sh.rows_pp; prm.alu_rows = sh.alu_rows;
  prm.ring = sh.ring; prm.nph = nph; prm.slabs_per_head = (int)(rp / 128); prm.slabs = (int64_t)bh * (rp / 128);
  prm.status = status;
  // One slot per item, as large as an output tile, one CTA per image (q = 11, forward): the tile is stored by TMA
  // from the item's own slot; every slot gets room for the q extra-class rows of its tile (two 64-entry halves).
  int smem = sh.smem;
  prm.tma_out = 0; prm.mini_bytes = 0;
  prm.lines_pp = sh.rows_pp / q < q ? sh.rows_pp / q : q;
  // (Tiles of whole lines could leave the same way for q = 13, 17 — the kernel handles several slots per item and
  // several parts — but there the tile stores were measured 1.6 to 2 times slower than the direct stores.)
  if (!transpose && sh.nslots == 1 && sh.sr == TILE_ROWS && sh.parts == 1) {
    const int mini = 2 * ((q + 7) & ~7) * 128, slot = sh.sr * 256;
    int ring = (227 * 1024 - 1024 - 512 - TILE_ROWS * 8) / (slot + mini);
    if (ring > sh.ring) ring = sh.ring;
    if (ring >= 4) {
      prm.tma_out = 1; prm.mini_bytes = mini; prm.ring = ring;
      smem = ring * (slot + mini) + TILE_ROWS * 8 + 512 + 1024;
    }
  }
  if (!radon_layout_ok(q, sh, prm.ring, prm.mini_bytes, prm.tma_out, in_has_extra, smem)) return cudaErrorInvalidConfiguration;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (nph == 2 && sms > RADON_EXCHANGE_CTAS) sms = RADON_EXCHANGE_CTAS;  // one private exchange slab per CTA was sized for
  int64_t ctas = (int64_t)(sms / sh.parts) * sh.parts;
  const int64_t items = nph == 1 ? prm.slabs * sp[0].images * sh.parts : prm.slabs;
  if (items < ctas) ctas = items;
  CUtensorMap tm_reg[2], tm_vert[2], tm_oreg[2], tm_overt[2];
  for (int i = 0; i < nph; ++i) {
    RadonPhase& ph = prm.ph[i];
    const RadonSide& in = sp[i].in;
    const int images = sp[i].images;
    const int64_t src_rp = sp[i].src_private ? 128 : rp, src_heads = sp[i].src_private ? ctas : bh;
    ph.in = in; ph.out = sp[i].out; ph.images = images;
    ph.src_private = sp[i].src_private; ph.dst_private = sp[i].dst_private;
    ph.src_heads = (int)src_heads;
    ph.dst_pitch = sp[i].dst_private ? 128 : rp;
    ph.dst = static_cast<__nv_bfloat16*>(sp[i].dst);
    {   // regular lines: (entry, lo, hi, image, head); a size-one dimension keeps its stride valid
      const int64_t sizes[4] = {q, q, images, src_heads};
      const int64_t strides[4] = {in.s_lo, in.s_hi, images > 1 ? in.s_img : in.rows_per_head, in.rows_per_head};
      const int box[4] = {q, sh.sps, 1, 1};
      if (!radon_map(&tm_reg[i], sp[i].src, src_rp, 5, sizes, strides, box)) return cudaErrorInvalidValue;
    }
    if (in_has_extra) {   // extra class: (entry, lo, image, head), rows v0 + image*sv_img + lo*sv_lo
      const bool per_image = in.sv_img != 0;
      const int64_t sizes[3] = {q, per_image ? images : 1, src_heads};
      const int64_t strides[3] = {in.sv_lo, per_image ? in.sv_img : in.rows_per_head, in.rows_per_head};
      const int box[3] = {q, 1, 1};
      if (!radon_map(&tm_vert[i], static_cast<const __nv_bfloat16*>(sp[i].src) + (int64_t)in.v0 * src_rp, src_rp, 4, sizes,
                     strides, box))
        return cudaErrorInvalidValue;
      ph.in.sv_img = per_image ? 1 : 0;   // the kernel passes image * sv_img as the coordinate
    } else {
      tm_vert[i] = tm_reg[i];
    }
    tm_oreg[i] = tm_reg[i]; tm_overt[i] = tm_reg[i];
    if (prm.tma_out) {   // the same two shapes over the output rows: boxes of q lines, and of the extra class
      const RadonSide& out = sp[i].out;
      const int64_t dst_rp = sp[i].dst_private ? 128 : rp, dst_heads = sp[i].dst_private ? ctas : bh;
      const int64_t sizes[4] = {q, q, images, dst_heads};
      const int64_t strides[4] = {out.s_lo, out.s_hi, images > 1 ? out.s_img : out.rows_per_head, out.rows_per_head};
      const int box[4] = {q, prm.lines_pp, 1, 1};
      if (!radon_map(&tm_oreg[i], sp[i].dst, dst_rp, 5, sizes, strides, box)) return cudaErrorInvalidValue;
      if (out.count > q * q) {
        const bool per_image = out.sv_img != 0;
        const int64_t vsizes[3] = {q, per_image ? images : 1, dst_heads};
        const int64_t vstrides[3] = {out.sv_lo, per_image ? out.sv_img : out.rows_per_head, out.rows_per_head};
        const int vbox[3] = {q, 1, 1};
        if (!radon_map(&tm_overt[i], static_cast<__nv_bfloat16*>(sp[i].dst) + (int64_t)out.v0 * dst_rp, dst_rp, 4, vsizes,
                       vstrides, vbox))
          return cudaErrorInvalidValue;
      }
    }
  }
  if (nph == 1) {
    prm.ph[1] = prm.ph[0]; tm_reg[1] = tm_reg[0]; tm_vert[1] = tm_vert[0]; tm_oreg[1] = tm_oreg[0]; tm_overt[1] = tm_overt[0];
  }
  const bool feat = nph > 1 || prm.alu_rows > 0;
  auto kernel = feat ? radon_tc_kernel<true> : radon_tc_kernel<false>;
  cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (err != cudaSuccess) return err;
  // the plain instantiation has no use for the two ALU warps
  kernel<<<(unsigned)ctas, feat ? RADON_THREADS : 32 * (ALU_WARP + (prm.tma_out ? 1 : 0)), smem, st>>>(tm_reg[0], tm_vert[0], tm_reg[1], tm_vert[1],
                                                                            tm_oreg[0], tm_overt[0], tm_oreg[1], tm_overt[1], prm);
  return cudaGetLastError();
}

// The two stages of d = 4 run as one launch when a CTA's exchange rows (q^3 + q^2 rows of 128 entries), times the
// CTAs of the grid, stay well inside the L2 cache, and one CTA covers every output index of an image.
bool radon_two_stage_fits(int q, int transpose) {
  RadonShape sh;
  const int qq = q * q;
  if (!radon_shape(q, transpose, transpose ? 1 : 0, transpose ? qq : qq + q, &sh) || sh.parts != 1) return false;
  return ((int64_t)qq * q + qq) * 256 * RADON_EXCHANGE_CTAS <= (64LL << 20);
}

}  // namespace

// 1 when the tensor-core tabulation covers this geometry (d = 3 or 4, q small enough for a resident R).
int smat_tabulate_tc_supported(const SmatGeo& geo, int64_t state_elems) {
  if (geo.D != 2 && geo.D != 3) return 0;
  if (state_elems % 128) return 0;
  const int qq = geo.q * geo.q;
  RadonShape a, b;
  return radon_shape(geo.q, 0, 0, qq + geo.q, &a) && radon_shape(geo.q, 1, 1, qq, &b) ? 1 : 0;
}

// Host-only: 1 when the shared-memory map of every launch shape this prime can take (both directions, with and without
// the extra class on the input, with the tile-store variant where the launcher would pick it) passes radon_layout_ok.
int smat_tabulate_tc_layout_ok(int q) {
  const int qq = q * q;
  for (int transpose = 0; transpose < 2; ++transpose)
    for (int extra = 0; extra < 2; ++extra) {
      RadonShape sh;
      const int count_out = (transpose ? !extra : extra) ? qq + q : qq;   // forward stages grow, transposed ones shrink
      for (int co : {count_out, qq, qq + q}) {
        if (!radon_shape(q, transpose, extra, co, &sh)) continue;
        if (!radon_layout_ok(q, sh, sh.ring, 0, 0, extra, sh.smem)) return 0;
        if (!transpose && sh.nslots == 1 && sh.sr == TILE_ROWS && sh.parts == 1) {
          const int mini = 2 * ((q + 7) & ~7) * 128, slot = sh.sr * 256;
          int ring = (227 * 1024 - 1024 - 512 - TILE_ROWS * 8) / (slot + mini);
          if (ring > sh.ring) ring = sh.ring;
          if (ring >= 4 && !radon_layout_ok(q, sh, ring, mini, 1, extra, ring * (slot + mini) + TILE_ROWS * 8 + 512 + 1024))
            return 0;
        }
      }
    }
  return 1;
}

// Rows (of state_elems bf16 each, per head) of the intermediate table the d = 4 stages exchange.
int64_t smat_tabulate_tc_scratch_rows(const SmatGeo& geo) {
  return geo.D == 3 ? (int64_t)geo.q * geo.q * geo.q + (int64_t)geo.q * geo.q : 0;
}

// bf16 elements of the scratch table smat_launch_tabulate_tc needs: the whole intermediate table W, or, when both
// directions run their two stages in one launch, one slab of it (128 entries per row) per CTA.
int64_t smat_tabulate_tc_scratch_elems(const SmatGeo& geo, int64_t state_elems, int bh) {
  const int64_t rows = smat_tabulate_tc_scratch_rows(geo);
  if (rows == 0) return 0;
  if (radon_two_stage_fits(geo.q, 0) && radon_two_stage_fits(geo.q, 1)) {
    int64_t ctas = (int64_t)bh * (state_elems / 128);
    if (ctas > RADON_EXCHANGE_CTAS) ctas = RADON_EXCHANGE_CTAS;
    return ctas * rows * 128;
  }
  return (int64_t)bh * rows * state_elems;
}

// transpose = 0: in = F [bh][P][rp] bf16, out = U [bh][B][rp] bf16.  transpose = 1: in = Ū [bh][B][rp], out = F̄ [bh][P][rp].
// scratch: smat_tabulate_tc_scratch_elems bf16 (d = 4 only).  One launch for d = 3; one or two for d = 4.
cudaError_t smat_launch_tabulate_tc(const void* in, void* out, void* scratch, const SmatGeo& geo, int64_t state_elems,
                                    int bh, int transpose, int* status, cudaStream_t st, int* launches) {
  const int q = geo.q, qq = q * q, qqq = qq * q;
  *launches = 0;
  if (geo.D == 2) {
    const RadonSide pts = side(qq, 1, q, 0, geo.P);
    const RadonSide typ = side(qq + q, 1, q, 0, geo.B, qq, 1, 0, 0);
    const StageSpec sp = transpose ? stage(typ, pts, 1, in, out) : stage(pts, typ, 1, in, out);
    *launches = 1;
    return launch_radon(q, transpose, 1, &sp, state_elems, bh, status, st);
  }
  if (geo.D != 3) return cudaErrorInvalidValue;
  const int64_t wrows = smat_tabulate_tc_scratch_rows(geo);
  const RadonSide f_side = side(qq, 1, qq, q, geo.P);                       // image x2, points (x1, x3)
  const RadonSide w1_side = side(qq + q, 1, qq, q, wrows, qqq, q, 1, 0);    // (u, a3) -> W[a3][x2][u]; extra class -> G[x3][x2]
  const RadonSide w2_side = side(qq, 1, q, qq, wrows);                      // image a3 (image q: G), points (u, x2)
  const RadonSide u_side = side(qq + q, 1, q, qq, geo.B, qqq + qq, 1, 0, q);
  const bool fused = radon_two_stage_fits(q, transpose);
  StageSpec sp[2];
  if (!transpose) {
    sp[0] = stage(f_side, w1_side, q, in, scratch, false, fused);
    sp[1] = stage(w2_side, u_side, q + 1, scratch, out, fused, false);
  } else {
    sp[0] = stage(u_side, w2_side, q + 1, in, scratch, false, fused);
    sp[1] = stage(w1_side, f_side, q, scratch, out, fused, false);
  }
  if (fused) {
    *launches = 1;
    return launch_radon(q, transpose, 2, sp, state_elems, bh, status, st);
  }
  *launches = 2;
  cudaError_t err = launch_radon(q, transpose, 1, &sp[0], state_elems, bh, status, st);
  if (err != cudaSuccess) return err;
  return launch_radon(q, transpose, 1, &sp[1], state_elems, bh, status, st);
}
