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
// a CTA owns `mt` tiles of 128 output indices (its part of R) and applies them to every item it is given:
//   every thread   : builds the CTA's part of R (128 mt output indices x K_pad input indices, K-major, 128-byte
//                    swizzle) and the row tables once
//   warp 16 lane 0 : TMA producer; a ring slot holds `sps` lines (fixed hi, all lo) of the image x 128 state entries
//                    (MN-major B operand, two boxes of 64 entries); the extra class travels in a slot of its own
//   warp 17 lane 0 : MMA issuer, D_t[128 outputs, 128 entries] += R_t,slot * B_slot for each tile t; up to four
//                    accumulator sets in flight in TMEM
//   warps 0-15     : epilogue, one output index (TMEM lane) per thread: round 32 entries at a time to bf16 and store
//                    them as 64 contiguous bytes of the output row
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
constexpr int RADON_THREADS = 32 * (MMA_WARP + 1);
constexpr int MAX_ACC = 4;                        // accumulator sets in flight: min(4, 512 / (128 mt))
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
  int32_t mt, parts;               // tiles of 128 output indices per CTA; CTAs sharing an image
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
// 1 when output index n and input index k are incident
__device__ __forceinline__ bool radon_entry(int q, int transpose, int n, int k) {
  const int o = transpose ? k : n, pt = transpose ? n : k;
  const int u = o % q, a = o / q, lo = pt % q, hi = pt / q;
  return a < q ? (lo + a * hi) % q == u : hi == u;
}

// Input index (lo + q*hi, hi == q for the extra class) held by row k of the streamed operand, or -1 for padding.
// Slot s < nreg holds the lines hi = s*sps .. s*sps + sps - 1, q rows each; slot nreg holds the extra class.
__device__ __forceinline__ int input_index(const RadonParams& p, int k) {
  const int slot = k / p.sr, r = k - slot * p.sr, q = p.q;
  if (slot < p.nreg) {
    const int hi = slot * p.sps + r / q;
    return (r < p.sps * q && hi < q) ? (r % q) + q * hi : -1;
  }
  return r < q ? q * q + r : -1;
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

// 32-byte store (a whole sector per thread)
__device__ __forceinline__ void st_global_v8(void* dst, const uint32_t (&w)[8]) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(w[0]), "r"(w[1]), "r"(w[2]),
               "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
               : "memory");
}

// The MMAs of one ring slot: STEPS K-steps of 16 operand rows for each of MT tiles.  Fully unrolled so that the lone
// issuing thread spends a handful of instructions per MMA.
template <int STEPS, int MT>
__device__ __forceinline__ void issue_slot(uint32_t tmem_d, uint64_t dA, uint64_t dA_tile, uint64_t dB, uint32_t idesc,
                                           bool first) {
#pragma unroll
  for (int kk = 0; kk < STEPS; ++kk) {
    const uint64_t a = dA + (uint64_t)((kk >> 2) * (TILE_ROWS * 128 >> 4) + (kk & 3) * 2);
    const uint64_t b = dB + (uint64_t)(kk * 128);
    mma_bf16(tmem_d, a, b, idesc, !(first && kk == 0));
    if (MT == 2) mma_bf16(tmem_d + 128, a + dA_tile, b, idesc, !(first && kk == 0));
  }
}
template <int MT>
__device__ __forceinline__ void issue_slot_steps(int steps, uint32_t tmem_d, uint64_t dA, uint64_t dA_tile, uint64_t dB,
                                                 uint32_t idesc, bool first) {
  switch (steps) {
    case 1: issue_slot<1, MT>(tmem_d, dA, dA_tile, dB, idesc, first); break;
    case 2: issue_slot<2, MT>(tmem_d, dA, dA_tile, dB, idesc, first); break;
    case 3: issue_slot<3, MT>(tmem_d, dA, dA_tile, dB, idesc, first); break;
    case 4: issue_slot<4, MT>(tmem_d, dA, dA_tile, dB, idesc, first); break;
    case 5: issue_slot<5, MT>(tmem_d, dA, dA_tile, dB, idesc, first); break;
    case 6: issue_slot<6, MT>(tmem_d, dA, dA_tile, dB, idesc, first); break;
    case 7: issue_slot<7, MT>(tmem_d, dA, dA_tile, dB, idesc, first); break;
    default: issue_slot<8, MT>(tmem_d, dA, dA_tile, dB, idesc, first); break;
  }
}

__global__ void __launch_bounds__(RADON_THREADS, 1) radon_tc_kernel(const __grid_constant__ CUtensorMap tm_reg,
                                                                    const __grid_constant__ CUtensorMap tm_vert,
                                                                    const RadonParams prm) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int q = prm.q;
  const int slot_bytes = prm.sr * 256;                          // two 64-entry blocks of sr rows x 128 bytes
  const int kb2 = (prm.sr + 63) / 64;                           // 64-row blocks of R per slot
  const int kblocks = prm.nslots * kb2;                         // and per tile
  const int n_cta = prm.mt * TILE_ROWS;                         // output indices of this CTA
  const int r_bytes = n_cta * kblocks * 128;                    // R part: [tile][64-index block][128 rows][128 bytes]
  uint8_t* sR = smem;
  uint8_t* sRing = smem + r_bytes;
  int32_t* out_tab = reinterpret_cast<int32_t*>(sRing + prm.ring * slot_bytes);    // [n_cta]
  uint64_t* bars = reinterpret_cast<uint64_t*>(out_tab + n_cta);
  uint64_t* full = bars;                    // [ring] slot filled (TMA bytes)
  uint64_t* empty = bars + prm.ring;        // [ring] slot consumed by the MMAs
  uint64_t* acc_full = empty + prm.ring;    // [MAX_ACC] accumulator set complete
  uint64_t* acc_empty = acc_full + MAX_ACC; // [MAX_ACC] accumulator set read out (one arrival per epilogue warp)
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
  // R part, 16 bytes (8 rows of the streamed operand) per store; per tile one run of kb2 blocks for every slot
  for (int c = threadIdx.x; c < n_cta * kblocks * 8; c += blockDim.x) {
    const int n = c % n_cta, kc = c / n_cta;                   // kc: chunk of 8 operand rows, counted in blocks of 64
    const int g = kc / (kb2 * 8), r0 = (kc - g * kb2 * 8) * 8; // slot and first row inside it
    const int nidx = part * n_cta + n;
    uint32_t w[4] = {0u, 0u, 0u, 0u};
    if (nidx < prm.out.count) {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int idx = r0 + e < prm.sr ? input_index(prm, g * prm.sr + r0 + e) : -1;
        if (idx >= 0 && idx < prm.in.count && radon_entry(q, prm.transpose, nidx, idx))
          w[e >> 1] |= 0x3F80u << ((e & 1) * 16);              // bf16 1.0
      }
    }
    const int t = n >> 7, row = n & 127;
    uint8_t* dst = sR + ((t * kblocks + (kc >> 3)) * TILE_ROWS + row) * 128 + (((kc & 7) ^ (row & 7)) << 4);
    *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
  }
  for (int n = threadIdx.x; n < n_cta; n += blockDim.x) out_tab[n] = side_row(prm.out, part * n_cta + n, q);
  for (int c = threadIdx.x; c < prm.ring * slot_bytes / 16; c += blockDim.x)
    reinterpret_cast<uint4*>(sRing)[c] = make_uint4(0u, 0u, 0u, 0u);   // rows no box writes must never hold NaN patterns
  fence_proxy_async();
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t acc_cols = prm.mt * 128;                       // TMEM columns of one accumulator set
  const uint32_t nacc = min(MAX_ACC, 512 / (int)acc_cols);

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
  } else if (warp == MMA_WARP && lane == 0) {
    // ---- MMA issuer -------------------------------------------------------------------------------------------
    constexpr uint32_t idesc = make_idesc(TILE_ROWS, 128, 0, 1);   // A K-major (R), B MN-major (image rows)
    const uint64_t dA0 = make_desc(smem_u32(sR), 16, 1024);
    const uint64_t dB0 = make_desc(smem_u32(sRing), prm.sr * 128, 1024);
    const uint32_t slot16 = (uint32_t)slot_bytes >> 4;            // descriptor address units are 16 bytes
    const uint32_t tile16 = (uint32_t)kblocks * (TILE_ROWS * 128 >> 4);
    const uint32_t slotA16 = (uint32_t)kb2 * (TILE_ROWS * 128 >> 4);
    const int steps = prm.sr / 16, nslots = prm.nslots, mt = prm.mt;
    const uint32_t ring = (uint32_t)prm.ring;
    uint32_t slot = 0, par = 0;                                   // ring position and the parity its full barrier shows
    uint32_t buf = 0, apar = 0, n_item = 0;                       // accumulator set; parity of its empty barrier's phase to wait for
    bool ok = true;
    for (uint32_t it = first; it < total && ok; it += step, ++n_item) {
      if (n_item >= nacc) ok = mbar_wait(acc_empty + buf, apar, wc);
      if (!ok) break;
      fence_after_sync();
      const uint32_t tmem_d = tmem_base + buf * acc_cols;
      uint64_t dA = dA0;
      for (int g = 0; g < nslots && ok; ++g, dA += slotA16) {
        ok = mbar_wait(full + slot, par, wc);
        if (!ok) break;
        fence_after_sync();
        const uint64_t dB = dB0 + (uint64_t)(slot * slot16);
        if (mt == 2) issue_slot_steps<2>(steps, tmem_d, dA, tile16, dB, idesc, g == 0);
        else issue_slot_steps<1>(steps, tmem_d, dA, tile16, dB, idesc, g == 0);
        mma_commit(empty + slot);
        if (++slot == ring) { slot = 0; par ^= 1; }
      }
      if (ok) mma_commit(acc_full + buf);
      if (++buf == nacc) { buf = 0; if (n_item >= nacc) apar ^= 1; }
    }
  } else if (warp < EPI_WARPS) {
    // ---- epilogue ---------------------------------------------------------------------------------------------
    // Units of work per item: (tile, 32-entry column chunk); warp w takes every fourth unit, starting at w / 4, in
    // its lane quarter w % 4.
    const int qd = warp & 3, sub = warp >> 2;
    const int orow = qd * 32 + lane;                            // output index inside a tile = TMEM lane
    const uint32_t lane_base = (uint32_t)(qd * 32) << 16;
    uint32_t n_item = 0;
    for (uint32_t it = first; it < total; it += step, ++n_item) {
      const uint32_t buf = n_item % nacc;
      const uint32_t img = it / slabs, slab = it - img * slabs;
      const uint32_t head = slab / (uint32_t)prm.slabs_per_head;
      const int e0 = (int)(slab - head * (uint32_t)prm.slabs_per_head) * 128;
      __nv_bfloat16* base = prm.dst + (int64_t)head * prm.out.rows_per_head * prm.rp + e0;
      const int reg_off = (int)img * prm.out.s_img, vert_off = prm.out.v0 + (int)img * prm.out.sv_img;
      const bool vert = (int)img >= prm.out.vert_from;
      if (!mbar_wait_warp(acc_full + buf, (n_item / nacc) & 1, wc)) break;
      fence_after_sync();
      for (int unit = sub; unit < prm.mt * 4; unit += 4) {
        const int t = unit >> 2, cb = unit & 3;
        if (part * n_cta + t * TILE_ROWS + qd * 32 >= prm.out.count) break;   // warp-uniform: no output index in these lanes
        uint32_t v[32];
        tmem_ld32(tmem_base + lane_base + buf * acc_cols + t * 128 + cb * 32, v);
        tmem_ld_wait();
        const int tv = out_tab[t * TILE_ROWS + orow];
        if (tv == ROW_INVALID || ((tv & ROW_VERT) && !vert)) continue;
        const int row = (tv & ROW_VERT) ? vert_off + (tv & ~ROW_VERT) : reg_off + tv;
        __nv_bfloat16* dst = base + (int64_t)row * prm.rp + cb * 32;
#pragma unroll
        for (int h8 = 0; h8 < 2; ++h8) {   // two whole 32-byte sectors per thread
          uint32_t w[8];
#pragma unroll
          for (int i = 0; i < 8; ++i)
            w[i] = pack_bf16(__uint_as_float(v[16 * h8 + 2 * i]), __uint_as_float(v[16 * h8 + 2 * i + 1]));
          st_global_v8(dst + 16 * h8, w);
        }
      }
      fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty + buf);
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
  int sps, sr, nreg, nslots, mt, parts, ring, smem;
};

// Ring slots of `sps` lines (sps*q rows, rounded up to 16) and the split of the output indices into tiles of 128 and
// of the tiles over CTAs (two tiles per CTA when the resident part of R then still leaves a ring of three slots,
// else one), chosen for the least MMA work.  Returns false when q is too large for this kernel.
bool radon_shape(int q, int in_has_extra, int count_out, RadonShape* s) {
  const int budget = 227 * 1024 - 1024 - 512;
  if (q < 2 || q > 64) return false;
  const int tiles = (count_out + TILE_ROWS - 1) / TILE_ROWS;
  int best = 1 << 30;
  for (int sps = 1; sps <= q; ++sps) {
    const int sr = (sps * q + 15) & ~15;
    if (sr > 128) break;
    const int nreg = (q + sps - 1) / sps, nslots = nreg + (in_has_extra ? 1 : 0);
    const int kblocks = nslots * ((sr + 63) / 64);   // R keeps a run of 64-row blocks per slot
    const int slot_bytes = sr * 256;
    for (int mt = (tiles >= 2 ? 2 : 1); mt >= 1; --mt) {
      const int r_bytes = mt * TILE_ROWS * kblocks * 128;
      const int tables = mt * TILE_ROWS * 4;
      const int left = budget - r_bytes - tables;
      if (left < 3 * slot_bytes) continue;
      int ring = left / slot_bytes;
      if (ring > 8) ring = 8;
      const int parts = (tiles + mt - 1) / mt;
      if (parts > 8) continue;
      // MMA work per image (operand rows, plus a charge per slot for its hand-over), times the CTAs that repeat it
      const int cost = nslots * (sr + 48) * parts;
      if (cost < best) {
        best = cost;
        s->sps = sps; s->sr = sr; s->nreg = nreg; s->nslots = nslots; s->mt = mt; s->parts = parts; s->ring = ring;
        s->smem = r_bytes + ring * slot_bytes + tables + 512 + 1024;
      }
      break;   // the largest feasible mt for this sps
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
  prm.mt = sh.mt; prm.parts = sh.parts;
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
