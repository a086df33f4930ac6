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
// of images: dense enough for the tensor cores (q of every q^2... entries of a row are nonzero, but the
// 5th-generation tensor cores add 60 times faster than the fp32 pipes), and bound by the image traffic.
//
// radon_tc_kernel, persistent, one CTA per SM:
//   every thread   : builds its part of R (N_part output indices x K_pad input indices, K-major, 128-byte swizzle)
//                    and the row tables once
//   warps 4-7      : producers; gather the image rows (64 input indices x 128 state entries per ring slot, MN-major
//                    A operand) with cp.async, up to LA slots in flight
//   warp 8 lane 0  : MMA issuer, D[128 entries, N_part] += A_slot * R_slotᵀ, accumulators double-buffered in TMEM
//   warps 0-3      : epilogue, one state entry (TMEM lane) per thread: round to bf16, transpose 32 output rows at a
//                    time through a staging tile, store whole 256-byte rows
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "smat_internal.h"
#include "smat_tc.cuh"

namespace {

using namespace tc;

constexpr int SLOT_ROWS = 64;                     // input indices per ring slot (four K-steps of 16)
constexpr int SLOT_BYTES = SLOT_ROWS * 256;       // two 64-entry blocks of 64 rows x 128 bytes
constexpr int STAGE_BYTES = 2 * 32 * 128 * 2;    // epilogue staging: two tiles of 32 output rows x 128 entries, bf16
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
  int32_t n_part, parts;           // output indices per CTA (multiple of 32, <= 256) and CTAs sharing an image
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

__device__ __forceinline__ void cp_async16(uint32_t smem_addr, const void* gmem) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr), "l"(gmem) : "memory");
}
__device__ __forceinline__ void st_zero16(uint32_t smem_addr) {
  asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(smem_addr), "r"(0u) : "memory");
}

template <int LA>
__global__ void __launch_bounds__(288, 1) radon_tc_kernel(const RadonParams prm) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int q = prm.q;
  const int kgroups = (prm.k_pad + SLOT_ROWS - 1) / SLOT_ROWS;
  const int r_bytes = prm.n_part * kgroups * 128;             // R part: kgroups blocks of n_part rows x 128 bytes
  uint8_t* sR = smem;
  uint8_t* sRing = smem + r_bytes;                            // r_bytes is a multiple of 1024 (n_part % 32 == 0)
  __nv_bfloat16* stage = reinterpret_cast<__nv_bfloat16*>(sRing + prm.ring * SLOT_BYTES);   // two [32][128] tiles
  int32_t* in_tab = reinterpret_cast<int32_t*>(sRing + prm.ring * SLOT_BYTES + STAGE_BYTES);   // [kgroups*64]
  int32_t* out_tab = in_tab + kgroups * SLOT_ROWS;                                 // [n_part]
  uint64_t* bars = reinterpret_cast<uint64_t*>(out_tab + prm.n_part);
  uint64_t* full = bars;                    // [ring] slot filled (128 arrivals)
  uint64_t* empty = bars + prm.ring;        // [ring] slot consumed by the MMAs
  uint64_t* acc_full = empty + prm.ring;    // [2] accumulator complete
  uint64_t* acc_empty = acc_full + 2;       // [2] accumulator read out (4 arrivals)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* cta_abort = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const WaitCtx wc{cta_abort, prm.status};
  const int part = blockIdx.x % prm.parts;

  if (threadIdx.x == 0) {
    *cta_abort = 0;
    for (int s = 0; s < prm.ring; ++s) { mbar_init(full + s, 128); mbar_init(empty + s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(acc_full + b, 1); mbar_init(acc_empty + b, 4); }
    fence_barrier_init();
  }
  if (warp == 8) tmem_alloc(tmem_slot, 512);
  // R part, 16 bytes (8 input indices) per store
  for (int c = threadIdx.x; c < prm.n_part * kgroups * 8; c += blockDim.x) {
    const int n = c % prm.n_part, kc = c / prm.n_part;       // kc: chunk of 8 input indices
    const int nidx = part * prm.n_part + n;
    uint32_t w[4] = {0u, 0u, 0u, 0u};
    if (nidx < prm.out.count) {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int k = kc * 8 + e;
        if (k < prm.in.count && radon_entry(q, prm.transpose, nidx, k)) w[e >> 1] |= 0x3F80u << ((e & 1) * 16);  // bf16 1.0
      }
    }
    uint8_t* dst = sR + (kc >> 3) * (prm.n_part * 128) + n * 128 + (((kc & 7) ^ (n & 7)) << 4);
    *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
  }
  for (int k = threadIdx.x; k < kgroups * SLOT_ROWS; k += blockDim.x) in_tab[k] = side_row(prm.in, k, q);
  for (int n = threadIdx.x; n < prm.n_part; n += blockDim.x) out_tab[n] = side_row(prm.out, part * prm.n_part + n, q);
  for (int c = threadIdx.x; c < prm.ring * SLOT_BYTES / 16; c += blockDim.x)
    reinterpret_cast<uint4*>(sRing)[c] = make_uint4(0u, 0u, 0u, 0u);   // stale rows must never hold NaN patterns
  fence_proxy_async();
  fence_before_sync();
  __syncthreads();
  fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  // items of this CTA: same part always; slab fastest, image slowest
  const int64_t first = blockIdx.x / prm.parts, step = gridDim.x / prm.parts;
  const int64_t total = prm.slabs * prm.images;

  if (warp >= 4 && warp < 8) {
    // ---- producers --------------------------------------------------------------------------------------------
    const int tid = threadIdx.x - 128;
    const int j = tid & 15, r0 = tid >> 4;                    // 16-byte piece of a 256-byte row; first row of eight
    const uint32_t ring_base = smem_u32(sRing);
    uint32_t gc = 0;                                          // groups issued
    uint32_t done = 0;                                        // groups published
    bool ok = true;
    for (int64_t it = first; it < total && ok; it += step) {
      const int img = (int)(it / prm.slabs);
      const int64_t slab = it - (int64_t)img * prm.slabs;
      const int64_t head = slab / prm.slabs_per_head;
      const int e0 = (int)(slab - head * prm.slabs_per_head) * 128;
      const __nv_bfloat16* base = prm.src + head * prm.in.rows_per_head * prm.rp + e0 + j * 8;
      const int reg_off = img * prm.in.s_img, vert_off = prm.in.v0 + img * prm.in.sv_img;
      const bool vert = img >= prm.in.vert_from;
      for (int g = 0; g < kgroups && ok; ++g, ++gc) {
        const int slot = gc % prm.ring;
        if (gc >= (uint32_t)prm.ring) ok = mbar_wait(empty + slot, ((gc / prm.ring) - 1) & 1, wc);
        if (!ok) break;
        const uint32_t sbase = ring_base + slot * SLOT_BYTES + (j >> 3) * (SLOT_ROWS * 128);
        const int rows = min(SLOT_ROWS, prm.k_pad - g * SLOT_ROWS);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int r = r0 + 8 * i;
          if (r < rows) {
            const int t = in_tab[g * SLOT_ROWS + r];
            const uint32_t dst = sbase + r * 128 + (((j & 7) ^ (r & 7)) << 4);
            if (t == ROW_INVALID || ((t & ROW_VERT) && !vert)) {
              st_zero16(dst);
            } else {
              const int row = (t & ROW_VERT) ? vert_off + (t & ~ROW_VERT) : reg_off + t;
              cp_async16(dst, base + (int64_t)row * prm.rp);
            }
          }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        if (gc >= (uint32_t)LA) {
          asm volatile("cp.async.wait_group %0;" ::"n"(LA) : "memory");
          fence_proxy_async();
          mbar_arrive(full + (done % prm.ring));
          ++done;
        }
      }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    fence_proxy_async();
    for (; done < gc; ++done) mbar_arrive(full + (done % prm.ring));
  } else if (warp == 8 && lane == 0) {
    // ---- MMA issuer -------------------------------------------------------------------------------------------
    const uint32_t idesc = make_idesc(128, prm.n_part, 1, 0);   // A MN-major (image rows), B K-major (R)
    const uint32_t aR = smem_u32(sR), aRing = smem_u32(sRing);
    uint32_t gc = 0, n_item = 0;
    bool ok = true;
    for (int64_t it = first; it < total && ok; it += step, ++n_item) {
      const uint32_t buf = n_item & 1;
      if (n_item >= 2) ok = mbar_wait(acc_empty + buf, ((n_item >> 1) - 1) & 1, wc);
      if (!ok) break;
      fence_after_sync();
      const uint32_t tmem_d = tmem_base + buf * 256;
      for (int g = 0; g < kgroups && ok; ++g, ++gc) {
        const int slot = gc % prm.ring;
        ok = mbar_wait(full + slot, (gc / prm.ring) & 1, wc);
        if (!ok) break;
        fence_after_sync();
        const int steps = min(4, (prm.k_pad - g * SLOT_ROWS) / 16);
        for (int kk = 0; kk < steps; ++kk) {
          const uint64_t dA = make_desc(aRing + slot * SLOT_BYTES + kk * 2048, SLOT_ROWS * 128, 1024);
          const uint64_t dB = make_desc(aR + g * (prm.n_part * 128) + kk * 32, 16, 1024);
          mma_bf16(tmem_d, dA, dB, idesc, (g | kk) != 0);
        }
        mma_commit(empty + slot);
      }
      if (ok) mma_commit(acc_full + buf);
    }
  } else if (warp < 4) {
    // ---- epilogue ---------------------------------------------------------------------------------------------
    // 32 output indices at a time: every thread drops its entry's 32 values into a [32][128] bf16 staging tile,
    // then the 128 threads write the tile out as whole 256-byte rows (16 bytes per thread and store).
    const int tid = threadIdx.x;
    const int e = tid;                                           // state entry of the slab = TMEM lane
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    uint32_t n_item = 0, n_chunk = 0;
    for (int64_t it = first; it < total; it += step, ++n_item) {
      const uint32_t buf = n_item & 1;
      const int img = (int)(it / prm.slabs);
      const int64_t slab = it - (int64_t)img * prm.slabs;
      const int64_t head = slab / prm.slabs_per_head;
      const int e0 = (int)(slab - head * prm.slabs_per_head) * 128;
      __nv_bfloat16* base = prm.dst + head * prm.out.rows_per_head * prm.rp + e0 + (tid & 15) * 8;
      const int reg_off = img * prm.out.s_img, vert_off = prm.out.v0 + img * prm.out.sv_img;
      const bool vert = img >= prm.out.vert_from;
      const bool ok = mbar_wait(acc_full + buf, (n_item >> 1) & 1, wc);
      if (bar_or_128(!ok)) break;                                // the four warps give up together
      fence_after_sync();
      for (int cb = 0; cb < prm.n_part / 32; ++cb, ++n_chunk) {
        if (part * prm.n_part + cb * 32 >= prm.out.count) break;   // uniform: nothing valid from here on
        uint32_t v[32];
        tmem_ld32(tmem_base + lane_base + buf * 256 + cb * 32, v);
        tmem_ld_wait();
        __nv_bfloat16* tile = stage + (n_chunk & 1) * (32 * 128);
#pragma unroll
        for (int i = 0; i < 32; ++i) tile[i * 128 + e] = __float2bfloat16_rn(__uint_as_float(v[i]));
        asm volatile("bar.sync 1, 128;" ::: "memory");
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          const int i = (tid >> 4) + 8 * x;
          const int t = out_tab[cb * 32 + i];
          if (t == ROW_INVALID || ((t & ROW_VERT) && !vert)) continue;
          const int row = (t & ROW_VERT) ? vert_off + (t & ~ROW_VERT) : reg_off + t;
          *reinterpret_cast<uint4*>(base + (int64_t)row * prm.rp) =
              *reinterpret_cast<const uint4*>(tile + i * 128 + (tid & 15) * 8);
        }
      }
      fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(acc_empty + buf);
    }
  }
  fence_before_sync();
  __syncthreads();
  if (warp == 8) {
    fence_after_sync();
    tmem_dealloc(tmem_base, 512);
  }
}

struct RadonShape {
  int k_pad, kgroups, n_part, parts, ring, smem;
};

// Splits the output indices over `parts` CTAs so that the resident part of R and a ring of at least four slots fit
// in shared memory.  Returns false when q is too large for this kernel.
bool radon_shape(int count_in, int count_out, RadonShape* s) {
  const int budget = 227 * 1024 - 1024 - 512;
  s->k_pad = (count_in + 15) & ~15;
  s->kgroups = (s->k_pad + SLOT_ROWS - 1) / SLOT_ROWS;
  for (int parts = 1; parts <= 6; ++parts) {
    const int per = (count_out + parts - 1) / parts;
    const int n_part = (per + 31) & ~31;
    if (n_part > 256) continue;
    const int r_bytes = n_part * s->kgroups * 128;
    const int tables = (s->kgroups * SLOT_ROWS + n_part) * 4;
    const int left = budget - r_bytes - tables - STAGE_BYTES;
    if (left < 4 * SLOT_BYTES) continue;
    int ring = left / SLOT_BYTES;
    if (ring > 8) ring = 8;
    s->n_part = n_part; s->parts = parts; s->ring = ring;
    s->smem = r_bytes + ring * SLOT_BYTES + STAGE_BYTES + tables + 512 + 1024;
    return true;
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
  if (!radon_shape(in.count, out.count, &sh) || rp % 128) return cudaErrorInvalidValue;
  RadonParams prm;
  prm.q = q; prm.transpose = transpose; prm.k_pad = sh.k_pad; prm.n_part = sh.n_part; prm.parts = sh.parts;
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
  cudaError_t err;
  if (sh.ring >= 6) {
    err = cudaFuncSetAttribute(radon_tc_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, sh.smem);
    if (err != cudaSuccess) return err;
    radon_tc_kernel<4><<<(unsigned)ctas, 288, sh.smem, st>>>(prm);
  } else {
    err = cudaFuncSetAttribute(radon_tc_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, sh.smem);
    if (err != cudaSuccess) return err;
    radon_tc_kernel<2><<<(unsigned)ctas, 288, sh.smem, st>>>(prm);
  }
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
