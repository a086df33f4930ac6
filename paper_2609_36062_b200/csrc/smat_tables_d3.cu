// Tabulation U = C F for d = 3 (Algorithm 2) with primes too large for the resident-matrix tensor-core kernel,
// on the fp32 ALUs with the sums held in registers.
//
// For d = 3 the points are (x1, x2) ∈ F_q², point index x1 + q x2, and the types are the lines
//        slope a < q :  h = a q + b,   { x1 + a x2 = b }        U_h = Σ_{x2} F[(b - a x2) mod q, x2]
//        extra class :  h = q² + b,    { x2 = b }               U_h = Σ_{x1} F[x1, b]
// Two lines share at most one point, so no partial sum is common to two of them: q³ + q² additions per state entry
// is what Algorithm 2 asks for and also the least any add-only scheme can do.  What this kernel organises is where the
// operands come from.  A thread owns ONE state entry and, for K slopes at a time, all q offsets: K q accumulators in
// registers.  It walks the q columns (fixed x2) of the slab once per K slopes; each of a column's q values is loaded from
// shared memory once and added into K accumulators, so shared-memory traffic per addition falls by K.  The adds take
// the bf16 value as it is (add.f32.bf16: fp32 accumulator + bf16 operand), so nothing is unpacked.
//
// The register index of an accumulator has to be a compile-time constant.  Slopes are therefore grouped as
// a0·{g_0 .. g_{K-1}} with fixed multipliers g_i = r^i (r a primitive root of F_q) and a0 = r^{K t} for task t: the sets
// tile F_q* when K divides q - 1.  With x2' = a0 x2 the target offset is b = x1 + g_i x2', which does not depend on a0:
// every task runs the same code and only permutes the order in which it visits the columns (x2 = x2' / a0).
// Unrolling all q columns would give a loop-free body far larger than the instruction cache (measured: five times
// slower), so the columns are taken in blocks of CB: inside a block the register of every offset is fixed, between
// blocks the K accumulator rings are turned by g_i CB places with register moves, and one block's code serves all.
// Slope 0 and the extra class form one lighter task per slab, an ordinary loop.
//
// One persistent CTA per SM, eight warps, 32 lanes = the 32 entries of a slab.  The pooling kernel stores this plan's
// profile table slab-major ([head][slab of 32 entries][point][32]), so a slab is one contiguous piece of memory: it
// arrives by bulk copies into one of two buffers, is read in place (16-bit loads, a warp reads 64 contiguous bytes),
// and the warp that finishes the last task of a slab starts the copy of the slab after next into the freed buffer.
// Warps take (slab, task) pairs from a shared counter.  Tables are bf16, sums fp32, one rounding per stored entry.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <type_traits>
#include <utility>

#include "smat_internal.h"
#include "smat_tc.cuh"

namespace {

using namespace tc;

constexpr int D3_ENTRIES = 32;       // state entries per slab = lanes of a warp
constexpr int D3_WARPS = 8;
constexpr int D3_THREADS = 32 * D3_WARPS;
constexpr int D3_OUT_ROWS = 16;      // rows of U a warp stages before it writes them as whole sectors

__host__ __device__ constexpr int cpow_mod(int base, int e, int q) {
  int r = 1;
  for (int i = 0; i < e; ++i) r = (r * base) % q;
  return r;
}
__host__ __device__ constexpr bool is_primitive_root(int r, int q) {
  int v = 1;
  for (int e = 1; e < q - 1; ++e) {
    v = (v * r) % q;
    if (v == 1) return false;
  }
  return true;
}

// Per-prime constants: K slopes per task (K | q - 1), a primitive root, and the column block CB, chosen so that one
// block's code, CB q (K + 1) instructions of 16 bytes, stays near 24 KB.
template <int Q> struct D3Cfg;
template <> struct D3Cfg<23> { static constexpr int K = 2, ROOT = 5, CB = 12; };
template <> struct D3Cfg<29> { static constexpr int K = 4, ROOT = 2, CB = 10; };
template <> struct D3Cfg<31> { static constexpr int K = 3, ROOT = 3, CB = 11; };
template <> struct D3Cfg<37> { static constexpr int K = 4, ROOT = 2, CB = 8; };

template <int Q>
struct D3Layout {
  using Cfg = D3Cfg<Q>;
  static constexpr int K = Cfg::K, CB = Cfg::CB;
  static_assert((Q - 1) % K == 0 && K <= 4, "slope groups must tile the nonzero slopes");
  static_assert(is_primitive_root(Cfg::ROOT, Q), "ROOT must generate the multiplicative group");
  static constexpr int NBLK = (Q + CB - 1) / CB;
  static constexpr int HEAVY = (Q - 1) / K;            // tasks of K nonzero slopes
  static constexpr int TASKS = HEAVY + 1;              // plus slope 0 with the extra class
  static constexpr int COL_BYTES = Q * 64;             // one column: q points x 32 entries
  static constexpr int SLAB_BYTES = Q * COL_BYTES;     // contiguous in the slab-major table
  static constexpr int OUT_BYTES = D3_OUT_ROWS * 64;
  static constexpr int OFF_OUT = 2 * SLAB_BYTES;
  static constexpr int OFF_BARS = OFF_OUT + D3_WARPS * OUT_BYTES;
  static constexpr int SMEM = OFF_BARS + 256;
  static_assert(SLAB_BYTES % 16 == 0 && SMEM <= 227 * 1024, "two slabs must fit");
};

struct D3Params {
  int64_t P, B, rp;          // profile states, type states, entries per state
  int64_t slabs;             // heads * rp / 32
  int slabs_per_head;
  const __nv_bfloat16* F;    // [bh][rp / 32][P][32]: slab-major profile table
  __nv_bfloat16* U;          // [bh][B][rp]
  int* status;
};

template <int Q, int I> constexpr int D3_MULT = cpow_mod(D3Cfg<Q>::ROOT, I, Q);

// Lane 0 polls the barrier and the warp follows.
__device__ __forceinline__ bool mbar_wait_warp_d3(uint64_t* bar, uint32_t parity, const WaitCtx& w) {
  bool ok = true;
  if ((threadIdx.x & 31) == 0) ok = mbar_wait(bar, parity, w);
  return __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
}

// bf16 value of point x1 of the column at shared address `col` (this lane's entry): OFF = x1 * 64 bytes.
template <int OFF>
__device__ __forceinline__ unsigned short d3_load(uint32_t col) {
  unsigned short h;
  asm volatile("ld.shared.u16 %0, [%1+%2];" : "=h"(h) : "r"(col), "n"(OFF));
  return h;
}
// fp32 accumulator += bf16 value.
__device__ __forceinline__ void d3_add(float& a, unsigned short h) { asm("add.rn.f32.bf16 %0, %1, %0;" : "+f"(a) : "h"(h)); }

// One value of a column, at compile-time position (x1, column j of the block), into its K accumulators.
template <int Q, int K>
__device__ __forceinline__ void d3_accumulate(float (&acc)[K * Q], unsigned short h, int x1, int j) {
  d3_add(acc[0 * Q + (x1 + D3_MULT<Q, 0> * j) % Q], h);
  if constexpr (K > 1) d3_add(acc[1 * Q + (x1 + D3_MULT<Q, 1> * j) % Q], h);
  if constexpr (K > 2) d3_add(acc[2 * Q + (x1 + D3_MULT<Q, 2> * j) % Q], h);
  if constexpr (K > 3) d3_add(acc[3 * Q + (x1 + D3_MULT<Q, 3> * j) % Q], h);
}

template <int Q, int K, int J, int X1 = 0>
__device__ __forceinline__ void d3_column(float (&acc)[K * Q], uint32_t col) {
  if constexpr (X1 < Q) {
    d3_accumulate<Q, K>(acc, d3_load<X1 * 64>(col), X1, J);
    d3_column<Q, K, J, X1 + 1>(acc, col);
  }
}

// Writes the first `rows` rows of the warp's staging tile ([row][32 entries] bf16) to global memory, sixteen rows per
// store instruction: every lane moves a whole 32-byte sector.  row_of(r) gives the type index of staged row r.
template <typename RowOf>
__device__ __forceinline__ void d3_flush(const __nv_bfloat16* stage, int rows, RowOf row_of, __nv_bfloat16* u_head,
                                         int64_t rp, int64_t e0, int lane) {
  __syncwarp();
  const int half = lane & 1;
#pragma unroll
  for (int r0 = 0; r0 < D3_OUT_ROWS; r0 += 16) {
    const int rr = r0 + (lane >> 1);
    if (rr < rows) {
      const uint4* src = reinterpret_cast<const uint4*>(stage + rr * D3_ENTRIES + half * 16);
      const uint4 a = src[0], b = src[1];
      st_global_v8(u_head + (int64_t)row_of(rr) * rp + e0 + half * 16, a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w);
    }
  }
  __syncwarp();
}

// Rows of U held in `acc` (ROWS values of this lane's entry) go out through the warp's staging tile, D3_OUT_ROWS rows
// at a time.  row_of(r) gives the type index of accumulator r.
template <int ROWS, typename RowOf>
__device__ __forceinline__ void d3_store_rows(const float (&acc)[ROWS], RowOf row_of, __nv_bfloat16* stage,
                                              __nv_bfloat16* u_head, int64_t rp, int64_t e0, int lane) {
#pragma unroll
  for (int c0 = 0; c0 < ROWS; c0 += D3_OUT_ROWS) {
#pragma unroll
    for (int r = 0; r < D3_OUT_ROWS; ++r)
      if (c0 + r < ROWS) stage[r * D3_ENTRIES + lane] = __float2bfloat16_rn(acc[c0 + r]);
    d3_flush(stage, ROWS - c0 < D3_OUT_ROWS ? ROWS - c0 : D3_OUT_ROWS, [&](int r) { return row_of(c0 + r); }, u_head, rp,
             e0, lane);
  }
}

// What a task needs to know about its slab.
struct D3Task {
  uint32_t slab;             // shared address of the slab buffer plus this lane's 2-byte entry offset
  __nv_bfloat16* stage;      // the warp's staging tile
  __nv_bfloat16* u_head;     // type table of the slab's head
  int64_t rp, e0;
  int lane;
};

// Columns j = J .. CB-1 of block `blk` (compile-time j, run-time block).
template <int Q, int K, int CB, int J = 0>
__device__ __forceinline__ void d3_block(float (&acc)[K * Q], uint32_t slab, int blk, int inv, int& x2) {
  if constexpr (J < CB) {
    if (blk * CB + J < Q) {
      d3_column<Q, K, J>(acc, slab + (uint32_t)(x2 * (Q * 64)));
      x2 += inv;
      if (x2 >= Q) x2 -= Q;
    }
    d3_block<Q, K, CB, J + 1>(acc, slab, blk, inv, x2);
  }
}

// One heavy task: the K slopes a0 g_i of one slab; the sums stay in registers until the rows are written.
// `release` is called between the last read of the slab and the stores.
template <int Q, typename Release>
__device__ __forceinline__ void d3_heavy_task(const D3Task& t, int task, Release release) {
  using L = D3Layout<Q>;
  constexpr int K = L::K, CB = L::CB, NBLK = L::NBLK;
  int a0 = 1;                                      // slopes a0 g_i; columns visited in the order x2 = x2' / a0
  for (int i = 0; i < K * task; ++i) a0 = (a0 * D3Cfg<Q>::ROOT) % Q;
  int inv = 1;
  for (int i = 0; i < Q - 2; ++i) inv = (inv * a0) % Q;
  float acc[K * Q];
#pragma unroll
  for (int i = 0; i < K * Q; ++i) acc[i] = 0.f;
  int x2 = 0;
#pragma unroll 1
  for (int blk = 0; blk < NBLK; ++blk) {
    if (blk > 0) {   // turn ring i by g_i CB places: register b now stands for offset b + g_i CB blk
#pragma unroll
      for (int i = 0; i < K; ++i) {
        const int rot = (cpow_mod(D3Cfg<Q>::ROOT, i, Q) * CB) % Q;
        float tmp[Q];
#pragma unroll
        for (int b = 0; b < Q; ++b) tmp[b] = acc[i * Q + (b + rot) % Q];
#pragma unroll
        for (int b = 0; b < Q; ++b) acc[i * Q + b] = tmp[b];
      }
    }
    d3_block<Q, K, CB>(acc, t.slab, blk, inv, x2);
  }
  __syncwarp();
  release();                                       // the slab is read; the sums are in registers
  int slope[K], turned[K];                         // register b of ring i holds offset b + g_i CB (NBLK - 1)
  slope[0] = a0;
#pragma unroll
  for (int i = 1; i < K; ++i) slope[i] = (slope[i - 1] * D3Cfg<Q>::ROOT) % Q;
#pragma unroll
  for (int i = 0; i < K; ++i) turned[i] = (cpow_mod(D3Cfg<Q>::ROOT, i, Q) * CB * (NBLK - 1)) % Q;
  d3_store_rows<K * Q>(acc, [&](int r) {
    const int i = r / Q;
    int s = slope[0], tn = turned[0];
#pragma unroll
    for (int j = 1; j < K; ++j) { s = (i == j) ? slope[j] : s; tn = (i == j) ? turned[j] : tn; }
    return s * Q + (r - i * Q + tn) % Q;
  }, t.stage, t.u_head, t.rp, t.e0, t.lane);
}

// The light task: slope 0, U[b] = Σ_{x2} F[b, x2], and the extra class, U[q² + x2] = Σ_{x1} F[x1, x2].  Neither needs
// a register index that depends on the column, so this is an ordinary loop over the columns; the extra-class sums go
// through the warp's staging tile.
template <int Q, int X1 = 0>
__device__ __forceinline__ void d3_light_column(float (&acc)[Q], float (&part)[4], uint32_t col) {
  if constexpr (X1 < Q) {
    const unsigned short h = d3_load<X1 * 64>(col);
    d3_add(acc[X1], h);
    d3_add(part[X1 & 3], h);
    d3_light_column<Q, X1 + 1>(acc, part, col);
  }
}

template <int Q, typename Release>
__device__ __forceinline__ void d3_light_task(const D3Task& t, Release release) {
  using L = D3Layout<Q>;
  float acc[Q];
#pragma unroll
  for (int i = 0; i < Q; ++i) acc[i] = 0.f;
#pragma unroll 1
  for (int x2 = 0; x2 < Q; ++x2) {
    float part[4] = {0.f, 0.f, 0.f, 0.f};
    d3_light_column<Q>(acc, part, t.slab + (uint32_t)(x2 * L::COL_BYTES));
    t.stage[(x2 & (D3_OUT_ROWS - 1)) * D3_ENTRIES + t.lane] = __float2bfloat16_rn((part[0] + part[1]) + (part[2] + part[3]));
    if ((x2 & (D3_OUT_ROWS - 1)) == D3_OUT_ROWS - 1 || x2 == Q - 1) {   // a full staging tile, or the last columns
      const int first = x2 & ~(D3_OUT_ROWS - 1);
      d3_flush(t.stage, x2 - first + 1, [&](int r) { return Q * Q + first + r; }, t.u_head, t.rp, t.e0, t.lane);
    }
  }
  __syncwarp();
  release();
  d3_store_rows<Q>(acc, [&](int r) { return r; }, t.stage, t.u_head, t.rp, t.e0, t.lane);
}

template <int Q>
__global__ void __launch_bounds__(D3_THREADS, 1) tabulate_d3_regs_kernel(const D3Params prm) {
  using L = D3Layout<Q>;
  constexpr int TASKS = L::TASKS;
  // Used directly (no manual re-alignment): 128-byte alignment is all the bulk copies need.
  extern __shared__ __align__(128) uint8_t smem[];
  uint64_t* slab_full = reinterpret_cast<uint64_t*>(smem + L::OFF_BARS);   // [2] slab landed (bulk-copy bytes)
  int* tasks_done = reinterpret_cast<int*>(slab_full + 2);                  // [2] finished tasks of the slab in a buffer
  int* task_counter = tasks_done + 2;
  volatile int* cta_abort = reinterpret_cast<volatile int*>(task_counter + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const WaitCtx wc{cta_abort, prm.status};
  // slabs of this CTA: blockIdx.x, blockIdx.x + gridDim.x, ...  (slabs are numbered head-major: the table's own order)
  const int64_t my_slabs = prm.slabs > blockIdx.x ? (prm.slabs - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
  auto start_copy = [&](int64_t ks) {   // slab ks of this CTA into buffer ks & 1; one thread calls this
    const int buf = (int)(ks & 1);
    const uint8_t* src = reinterpret_cast<const uint8_t*>(prm.F) + (blockIdx.x + ks * gridDim.x) * (int64_t)L::SLAB_BYTES;
    uint8_t* dst = smem + buf * L::SLAB_BYTES;
    mbar_expect_tx(slab_full + buf, L::SLAB_BYTES);
    constexpr int PIECE = 4 * L::COL_BYTES;
    for (int off = 0; off < L::SLAB_BYTES; off += PIECE)
      bulk_load(dst + off, src + off, off + PIECE <= L::SLAB_BYTES ? PIECE : L::SLAB_BYTES - off, slab_full + buf);
  };
  if (threadIdx.x == 0) {
    *cta_abort = 0;
    *task_counter = 0;
    tasks_done[0] = tasks_done[1] = 0;
    mbar_init(slab_full, 1);
    mbar_init(slab_full + 1, 1);
    fence_barrier_init();
    for (int64_t ks = 0; ks < 2 && ks < my_slabs; ++ks) start_copy(ks);
  }
  __syncthreads();

  D3Task t;
  t.stage = reinterpret_cast<__nv_bfloat16*>(smem + L::OFF_OUT + warp * L::OUT_BYTES);
  t.rp = prm.rp;
  t.lane = lane;
  const int64_t total = my_slabs * TASKS;
  for (;;) {
    int id = 0;
    if (lane == 0) id = atomicAdd(task_counter, 1);
    id = __shfl_sync(0xffffffffu, id, 0);
    if (id >= total) break;
    const int64_t ks = id / TASKS;
    const int task = (int)(id - ks * TASKS), buf = (int)(ks & 1);
    const int64_t slab = blockIdx.x + ks * gridDim.x;
    const int64_t head = slab / prm.slabs_per_head;
    t.e0 = (slab - head * prm.slabs_per_head) * D3_ENTRIES;
    t.u_head = prm.U + head * prm.B * prm.rp;
    t.slab = smem_u32(smem + buf * L::SLAB_BYTES) + (uint32_t)(lane * 2);
    if (!mbar_wait_warp_d3(slab_full + buf, (uint32_t)((ks >> 1) & 1), wc)) break;
    // After its last read a task counts itself done; the one that completes the slab's count owns the buffer and
    // starts the copy of the slab after next (every read of the buffer has returned its value by then).
    auto release = [&]() {
      if (lane == 0) {
        __threadfence_block();
        if (atomicAdd(tasks_done + buf, 1) == TASKS - 1) {
          tasks_done[buf] = 0;
          if (ks + 2 < my_slabs) start_copy(ks + 2);
        }
      }
    };
    if (task < L::HEAVY)
      d3_heavy_task<Q>(t, task, release);
    else
      d3_light_task<Q>(t, release);
  }
}

template <int Q>
cudaError_t launch_d3_regs(const void* in, void* out, const SmatGeo& geo, int64_t rp, int bh, int* status,
                           cudaStream_t st) {
  using L = D3Layout<Q>;
  D3Params prm;
  prm.F = static_cast<const __nv_bfloat16*>(in);
  prm.P = geo.P; prm.B = geo.B; prm.rp = rp;
  prm.slabs_per_head = (int)(rp / D3_ENTRIES);
  prm.slabs = (int64_t)bh * prm.slabs_per_head;
  prm.U = static_cast<__nv_bfloat16*>(out);
  prm.status = status;
  cudaError_t err = cudaFuncSetAttribute(tabulate_d3_regs_kernel<Q>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::SMEM);
  if (err != cudaSuccess) return err;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int64_t grid = prm.slabs < sms ? prm.slabs : sms;
  tabulate_d3_regs_kernel<Q><<<(unsigned)grid, D3_THREADS, L::SMEM, st>>>(prm);
  return cudaGetLastError();
}

}  // namespace

// 1 when the register-resident d = 3 tabulation covers this geometry.
int smat_tabulate_d3_regs_supported(const SmatGeo& geo, int64_t state_elems) {
  if (geo.D != 2 || state_elems % D3_ENTRIES) return 0;
  return geo.q == 23 || geo.q == 29 || geo.q == 31 || geo.q == 37;
}

cudaError_t smat_launch_tabulate_d3_regs(const void* in, void* out, const SmatGeo& geo, int64_t state_elems, int bh,
                                         int* status, cudaStream_t st) {
  if (!smat_tabulate_d3_regs_supported(geo, state_elems)) return cudaErrorInvalidConfiguration;
  switch (geo.q) {
    case 23: return launch_d3_regs<23>(in, out, geo, state_elems, bh, status, st);
    case 29: return launch_d3_regs<29>(in, out, geo, state_elems, bh, status, st);
    case 31: return launch_d3_regs<31>(in, out, geo, state_elems, bh, status, st);
    default: return launch_d3_regs<37>(in, out, geo, state_elems, bh, status, st);
  }
}
