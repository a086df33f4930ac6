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
//   warps 8-15     : producers; each gathers the image rows of one ring slot at a time (64 input indices x 128 state
//                    entries, MN-major B operand) with cp.async, so up to eight slots are in flight
//   warp 16 lane 0 : MMA issuer, D_t[128 outputs, 128 entries] += R_t,slot * B_slot for each tile t; up to four
//                    accumulator sets in flight in TMEM
//   warps 0-7      : epilogue, one output index (TMEM lane) per thread: round 32 entries at a time to bf16 and store
//                    them as 64 contiguous bytes of the output row
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "smat_internal.h"
#include "smat_tc.cuh"

namespace {

using namespace tc;

constexpr int SLOT_ROWS = 64;                     // input indices per ring slot (four K-steps of 16)
constexpr int SLOT_BYTES = SLOT_ROWS * 256;       // two 64-entry blocks of 64 rows x 128 bytes
constexpr int TILE_ROWS = 128;                    // output indices per tile (MMA M)
constexpr int EPI_WARPS = 8;
constexpr int PROD_WARPS = 8;
constexpr int MMA_WARP = EPI_WARPS + PROD_WARPS;
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
  int32_t k_pad;                   // input indices rounded up to 16
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

// 16-byte copy that reads `bytes` (16 or 0) from global memory and fills the rest with zeros
__device__ __forceinline__ void cp_async16_zfill(uint32_t smem_addr, const void* gmem, int bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_addr), "l"(gmem), "r"(bytes) : "memory");
}

__global__ void __launch_bounds__(RADON_THREADS, 1) radon_tc_kernel(const RadonParams prm) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int q = prm.q;
  const int kgroups = (prm.k_pad + SLOT_ROWS - 1) / SLOT_ROWS;
  const int n_cta = prm.mt * TILE_ROWS;                         // output indices of this CTA
  const int r_bytes = n_cta * kgroups * 128;                    // R part: [tile][64-index block][128 rows][128 bytes]
  uint8_t* sR = smem;
  uint8_t* sRing = smem + r_bytes;
  int32_t* in_tab = reinterpret_cast<int32_t*>(sRing + prm.ring * SLOT_BYTES);   // [kgroups*64]
  int32_t* out_tab = in_tab + kgroups * SLOT_ROWS;                                 // [n_cta]
  uint64_t* bars = reinterpret_cast<uint64_t*>(out_tab + n_cta);
  uint64_t* full = bars;                    // [ring] slot filled (one arrival, from the warp that filled it)
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
  }
  if (warp == MMA_WARP) tmem_alloc(tmem_slot, 512);
  // R part, 16 bytes (8 input indices) per store
  for (int c = threadIdx.x; c < n_cta * kgroups * 8; c += blockDim.x) {
    const int n = c % n_cta, kc = c / n_cta;                   // kc: chunk of 8 input indices
    const int nidx = part * n_cta + n;
    uint32_t w[4] = {0u, 0u, 0u, 0u};
    if (nidx < prm.out.count) {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int k = kc * 8 + e;
        if (k < prm.in.count && radon_entry(q, prm.transpose, nidx, k)) w[e >> 1] |= 0x3F80u << ((e & 1) * 16);  // bf16 1.0
      }
    }
    const int t = n >> 7, row = n & 127;
    uint8_t* dst = sR + ((t * kgroups + (kc >> 3)) * TILE_ROWS + row) * 128 + (((kc & 7) ^ (row & 7)) << 4);
    *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
  }
  for (int k = threadIdx.x; k < kgroups * SLOT_ROWS; k += blockDim.x) in_tab[k] = side_row(prm.in, k, q);
  for (int n = threadIdx.x; n < n_cta; n += blockDim.x) out_tab[n] = side_row(prm.out, part * n_cta + n, q);
  for (int c = threadIdx.x; c < prm.ring * SLOT_BYTES / 16; c += blockDim.x)
    reinterpret_cast<uint4*>(sRing)[c] = make_uint4(0u, 0u, 0u, 0u);   // stale rows must never hold NaN patterns
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

  if (warp >= EPI_WARPS && warp < MMA_WARP) {
    // ---- producers: warp pw fills the slots of the groups with (group counter) % active == pw, one group in flight each ----
    // A warp must never be two uses of a slot ahead of the consumer (its wait names a phase parity), hence no more
    // active producer warps than ring slots.
    const int pw = warp - EPI_WARPS;
    const uint32_t active = min(PROD_WARPS, prm.ring);
    const int j = lane & 15, rl = lane >> 4;                  // 16-byte piece of a 256-byte row; row parity
    const uint32_t ring_base = smem_u32(sRing) + (j >> 3) * (SLOT_ROWS * 128);
    uint32_t gc = 0;                                          // groups of this CTA so far
    bool ok = true;
    for (uint32_t it = first; it < total && ok; it += step) {
      const uint32_t img = it / slabs, slab = it - img * slabs;
      const uint32_t head = slab / (uint32_t)prm.slabs_per_head;
      const int e0 = (int)(slab - head * (uint32_t)prm.slabs_per_head) * 128;
      const __nv_bfloat16* base = prm.src + (int64_t)head * prm.in.rows_per_head * prm.rp + e0 + j * 8;
      const int reg_off = (int)img * prm.in.s_img, vert_off = prm.in.v0 + (int)img * prm.in.sv_img;
      const bool vert = (int)img >= prm.in.vert_from;
      for (int g = 0; g < kgroups; ++g, ++gc) {
        if ((int)(gc % active) != pw) continue;
        const int slot = gc % prm.ring;
        if (gc >= (uint32_t)prm.ring) ok = mbar_wait_warp(empty + slot, ((gc / prm.ring) - 1) & 1, wc);
        if (!ok) break;
        const uint32_t sbase = ring_base + slot * SLOT_BYTES;
        const int rows = min(SLOT_ROWS, prm.k_pad - g * SLOT_ROWS);
        const int32_t* tab = in_tab + g * SLOT_ROWS;
        for (int i0 = 0; i0 < rows / 2; i0 += 8) {              // rows is a multiple of 16
          int t[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) t[u] = tab[rl + 2 * (i0 + u)];
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const int r = rl + 2 * (i0 + u);
            const bool valid = t[u] >= 0 && (!(t[u] & ROW_VERT) || vert);
            const int row = valid ? (t[u] & (ROW_VERT - 1)) + ((t[u] & ROW_VERT) ? vert_off : reg_off) : 0;
            cp_async16_zfill(sbase + r * 128 + (((j & 7) ^ (r & 7)) << 4), base + (int64_t)row * prm.rp, valid ? 16 : 0);
          }
        }
        asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;" ::: "memory");
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(full + slot);
      }
    }
  } else if (warp == MMA_WARP && lane == 0) {
    // ---- MMA issuer -------------------------------------------------------------------------------------------
    constexpr uint32_t idesc = make_idesc(TILE_ROWS, 128, 0, 1);   // A K-major (R), B MN-major (image rows)
    const uint32_t aR = smem_u32(sR), aRing = smem_u32(sRing);
    uint32_t gc = 0, n_item = 0;
    bool ok = true;
    for (uint32_t it = first; it < total && ok; it += step, ++n_item) {
      const uint32_t buf = n_item % nacc;
      if (n_item >= nacc) ok = mbar_wait(acc_empty + buf, ((n_item / nacc) - 1) & 1, wc);
      if (!ok) break;
      fence_after_sync();
      const uint32_t tmem_d = tmem_base + buf * acc_cols;
      for (int g = 0; g < kgroups && ok; ++g, ++gc) {
        const int slot = gc % prm.ring;
        ok = mbar_wait(full + slot, (gc / prm.ring) & 1, wc);
        if (!ok) break;
        fence_after_sync();
        const int steps = min(4, (prm.k_pad - g * SLOT_ROWS) / 16);
        for (int t = 0; t < prm.mt; ++t)
          for (int kk = 0; kk < steps; ++kk) {
            const uint64_t dA = make_desc(aR + (t * kgroups + g) * (TILE_ROWS * 128) + kk * 32, 16, 1024);
            const uint64_t dB = make_desc(aRing + slot * SLOT_BYTES + kk * 2048, SLOT_ROWS * 128, 1024);
            mma_bf16(tmem_d + t * 128, dA, dB, idesc, (g | kk) != 0);
          }
        mma_commit(empty + slot);
      }
      if (ok) mma_commit(acc_full + buf);
    }
  } else if (warp < EPI_WARPS) {
    // ---- epilogue ---------------------------------------------------------------------------------------------
    // Units of work per item: (tile, 32-entry column chunk); warp w takes the units of parity w / 4 in its lane
    // quarter w % 4.
    const int qd = warp & 3, half = warp >> 2;
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
      for (int unit = half; unit < prm.mt * 4; unit += 2) {
        const int t = unit >> 2, cb = unit & 3;
        if (part * n_cta + t * TILE_ROWS >= prm.out.count) break;   // uniform: the tile holds no output index
        uint32_t v[32];
        tmem_ld32(tmem_base + lane_base + buf * acc_cols + t * 128 + cb * 32, v);
        tmem_ld_wait();
        const int tv = out_tab[t * TILE_ROWS + orow];
        if (tv == ROW_INVALID || ((tv & ROW_VERT) && !vert)) continue;
        const int row = (tv & ROW_VERT) ? vert_off + (tv & ~ROW_VERT) : reg_off + tv;
        uint4* dst = reinterpret_cast<uint4*>(base + (int64_t)row * prm.rp + cb * 32);
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4)
          dst[q4] = make_uint4(pack_bf16(__uint_as_float(v[8 * q4]), __uint_as_float(v[8 * q4 + 1])),
                               pack_bf16(__uint_as_float(v[8 * q4 + 2]), __uint_as_float(v[8 * q4 + 3])),
                               pack_bf16(__uint_as_float(v[8 * q4 + 4]), __uint_as_float(v[8 * q4 + 5])),
                               pack_bf16(__uint_as_float(v[8 * q4 + 6]), __uint_as_float(v[8 * q4 + 7])));
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
  int k_pad, kgroups, mt, parts, ring, smem;
};

// Splits the output indices into tiles of 128 and the tiles over CTAs: two tiles per CTA when the resident part of R
// then still leaves a ring of six slots, else one.  Returns false when q is too large for this kernel.
bool radon_shape(int count_in, int count_out, RadonShape* s) {
  const int budget = 227 * 1024 - 1024 - 512;
  s->k_pad = (count_in + 15) & ~15;
  s->kgroups = (s->k_pad + SLOT_ROWS - 1) / SLOT_ROWS;
  const int tiles = (count_out + TILE_ROWS - 1) / TILE_ROWS;
  for (int mt = (tiles >= 2 ? 2 : 1); mt >= 1; --mt) {
    const int r_bytes = mt * TILE_ROWS * s->kgroups * 128;
    const int tables = (s->kgroups * SLOT_ROWS + mt * TILE_ROWS) * 4;
    const int left = budget - r_bytes - tables;
    const int need = mt == 2 ? 6 : 4;
    if (left < need * SLOT_BYTES) continue;
    int ring = left / SLOT_BYTES;
    if (ring > 8) ring = 8;
    s->mt = mt; s->parts = (tiles + mt - 1) / mt; s->ring = ring;
    s->smem = r_bytes + ring * SLOT_BYTES + tables + 512 + 1024;
    return s->parts <= 8;
  }
  return false;
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
  if (!radon_shape(in.count, out.count, &sh) || rp % 128 || (int64_t)bh * (rp / 128) * images >= (1LL << 31))
    return cudaErrorInvalidValue;
  RadonParams prm;
  prm.q = q; prm.transpose = transpose; prm.k_pad = sh.k_pad; prm.mt = sh.mt; prm.parts = sh.parts;
  prm.ring = sh.ring; prm.images = images; prm.slabs_per_head = (int)(rp / 128); prm.slabs = (int64_t)bh * (rp / 128);
  prm.rp = rp; prm.in = in; prm.out = out;
  prm.src = static_cast<const __nv_bfloat16*>(src);
  prm.dst = static_cast<__nv_bfloat16*>(dst);
  prm.status = status;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  int64_t ctas = (int64_t)(sms / sh.parts) * sh.parts;
  const int64_t items = prm.slabs * images * sh.parts;
  if (items < ctas) ctas = items;
  cudaError_t err = cudaFuncSetAttribute(radon_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, sh.smem);
  if (err != cudaSuccess) return err;
  radon_tc_kernel<<<(unsigned)ctas, RADON_THREADS, sh.smem, st>>>(prm);
  return cudaGetLastError();
}

}  // namespace

// 1 when the tensor-core tabulation covers this geometry (d = 3 or 4, q small enough for a resident R).
int smat_tabulate_tc_supported(const SmatGeo& geo, int64_t state_elems) {
  if (geo.D != 2 && geo.D != 3) return 0;
  if (state_elems % 128) return 0;
  const int qq = geo.q * geo.q;
  RadonShape a, b;
  return radon_shape(qq, qq + geo.q, &a) && radon_shape(qq + geo.q, qq, &b) ? 1 : 0;
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
