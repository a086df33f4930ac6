// User-supplied routing (Sec. 3, "construction of G": the content-based assignment): the caller gives every distant
// token its profile cell and every recent token its type as integer arrays; this file turns them into the per-group
// token lists (CSR: offsets + token positions, ascending inside a group) that the pooling and routed-read kernels
// walk instead of the positional strides.  Integer work only: a counting sort per (head, kind), stable so that the
// order of the floating-point sums downstream does not depend on thread timing.
#include <cuda_runtime.h>

#include "smat_internal.h"

namespace {

constexpr int ROUTE_THREADS = 256;

// One CTA per (head, kind); kind 0: profiles of the n distant tokens, kind 1: types of the m recent tokens.
// The tokens are cut into W contiguous ranges, one per warp (W as large as shared memory allows, at most 8):
//   1. every warp histograms the keys of its range in its own row of counters (keys outside [0, G) are dropped:
//      such a token belongs to no group)
//   2. totals per group, exclusive scan -> offs[0 .. G]; row w then becomes the first slot of group g for warp w's
//      tokens: offs[g] + the counts of the warps before it
//   3. stable placement: every warp walks ITS range in order, 32 tokens at a time; lanes with equal keys find each other
//      with match.any, the lowest such lane advances the warp's cursor of the group, every lane writes its token's
//      position.  Ranges are in token order and each warp's slots follow those of the warps before it, so the list of
//      a group is ascending.
struct RouteParams {
  const int32_t* key[2];   // [bh][count]
  int32_t* list[2];        // [bh][count]
  int32_t* offs[2];        // [bh][G + 1]
  int64_t count[2], G[2], first[2];   // tokens per head, groups, position of the first token of the kind
  int warps;               // W: rows of per-warp counters in shared memory
};

__global__ void __launch_bounds__(ROUTE_THREADS) routing_lists_kernel(const RouteParams prm) {
  extern __shared__ int32_t rows[];     // [1 + W][G + 1]: row 0 totals / offsets, row 1 + w the counters of warp w
  const int kind = blockIdx.y;
  const int64_t bh = blockIdx.x, n = prm.count[kind], G = prm.G[kind], pitch = G + 1;
  const int W = prm.warps;
  const int32_t* key = prm.key[kind] + bh * n;
  int32_t* list = prm.list[kind] + bh * n;
  int32_t* offs = prm.offs[kind] + bh * pitch;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int32_t* total = rows;
  for (int64_t i = tid; i < (1 + W) * pitch; i += ROUTE_THREADS) rows[i] = 0;
  __syncthreads();
  const int64_t per = ((n + W - 1) / W + 31) & ~(int64_t)31;   // tokens per warp range, a multiple of 32
  const int64_t lo = (int64_t)warp * per, hi = lo + per < n ? lo + per : n;
  if (warp < W) {
    int32_t* mine = rows + (1 + warp) * pitch;
    for (int64_t t = lo + lane; t < hi; t += 32) {
      const int32_t k = key[t];
      if (k >= 0 && k < G) atomicAdd(&mine[k], 1);
    }
  }
  __syncthreads();
  for (int64_t g = tid; g < G; g += ROUTE_THREADS) {
    int32_t sum = 0;
    for (int w = 0; w < W; ++w) sum += rows[(1 + w) * pitch + g];
    total[g + 1] = sum;          // shifted by one: the inclusive scan below leaves the first slot of group g at index g
  }
  __syncthreads();
  __shared__ int32_t warp_sum[ROUTE_THREADS / 32];
  __shared__ int32_t carry;
  if (tid == 0) carry = 0;
  __syncthreads();
  for (int64_t base = 1; base <= G; base += ROUTE_THREADS) {
    const int64_t g = base + tid;
    int32_t x = g <= G ? total[g] : 0;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int32_t y = __shfl_up_sync(0xffffffffu, x, d);
      if (lane >= d) x += y;
    }
    if (lane == 31) warp_sum[warp] = x;
    __syncthreads();
    int32_t before = carry;
    for (int w = 0; w < warp; ++w) before += warp_sum[w];
    if (g <= G) total[g] = before + x;
    __syncthreads();
    if (tid == ROUTE_THREADS - 1) carry = before + x;
    __syncthreads();
  }
  // total[g] = tokens in groups < g (total[0] = 0): the offsets; then the per-warp first slots
  for (int64_t g = tid; g <= G; g += ROUTE_THREADS) offs[g] = total[g];
  for (int64_t g = tid; g < G; g += ROUTE_THREADS) {
    int32_t slot = total[g];
    for (int w = 0; w < W; ++w) {
      const int32_t c = rows[(1 + w) * pitch + g];
      rows[(1 + w) * pitch + g] = slot;
      slot += c;
    }
  }
  __syncthreads();
  if (warp < W) {
    int32_t* cursor = rows + (1 + warp) * pitch;
    const int64_t first = prm.first[kind];
    for (int64_t t0 = lo; t0 < hi; t0 += 32) {
      const int64_t t = t0 + lane;
      const int32_t k = t < hi ? key[t] : -1;
      const bool valid = k >= 0 && k < G;
      const unsigned peers = __match_any_sync(0xffffffffu, valid ? k : -1 - lane);
      if (valid) {
        const int leader = __ffs(peers) - 1;
        int32_t slot = 0;
        if (lane == leader) {
          slot = cursor[k];
          cursor[k] = slot + __popc(peers);
        }
        slot = __shfl_sync(peers, slot, leader) + __popc(peers & ((1u << lane) - 1));
        list[slot] = (int32_t)(first + t);
      }
      __syncwarp();
    }
  }
}

// Rows of tokens that belong to no group are never written by a routed read; whoever adds those rows afterwards must
// find zeros there.  One thread per token reads its key; the (rare) token whose key is out of range zeroes its row.
__global__ void zero_unrouted_rows_kernel(const int32_t* __restrict__ key, int64_t count, int64_t G, int64_t first,
                                          uint8_t* __restrict__ rows, int64_t T, int row_bytes, int64_t total) {
  const int64_t w = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (w >= total) return;
  const int32_t k = key[w];
  if (k >= 0 && k < G) return;
  const int64_t bh = w / count, t = first + (w - bh * count);
  uint4* dst = reinterpret_cast<uint4*>(rows + (bh * T + t) * row_bytes);
  for (int i = 0; i < row_bytes / 16; ++i) dst[i] = make_uint4(0u, 0u, 0u, 0u);
}

}  // namespace

cudaError_t smat_launch_zero_unrouted(const int32_t* key, int64_t count, int64_t G, int64_t first, void* rows, int64_t T,
                                      int row_bytes, int bh, cudaStream_t st) {
  const int64_t total = (int64_t)bh * count;
  zero_unrouted_rows_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(key, count, G, first,
                                                                               static_cast<uint8_t*>(rows), T, row_bytes, total);
  return cudaGetLastError();
}

// Largest group count the list builder handles (its cursors live in shared memory).
int64_t smat_routing_max_groups() { return 27000; }

cudaError_t smat_launch_routing_lists(const int32_t* prof, const int32_t* type, int32_t* prof_list, int32_t* prof_offs,
                                      int32_t* type_list, int32_t* type_offs, const SmatGeo& geo, int bh,
                                      cudaStream_t st) {
  RouteParams prm;
  prm.key[0] = prof; prm.list[0] = prof_list; prm.offs[0] = prof_offs; prm.count[0] = geo.n; prm.G[0] = geo.P; prm.first[0] = 0;
  prm.key[1] = type; prm.list[1] = type_list; prm.offs[1] = type_offs; prm.count[1] = geo.m; prm.G[1] = geo.B; prm.first[1] = geo.n;
  const int64_t gmax = geo.P > geo.B ? geo.P : geo.B;
  if (gmax > smat_routing_max_groups()) return cudaErrorInvalidConfiguration;
  int64_t warps = (int64_t)(220 * 1024 / sizeof(int32_t)) / (gmax + 1) - 1;
  if (warps > ROUTE_THREADS / 32) warps = ROUTE_THREADS / 32;
  if (warps < 1) warps = 1;
  prm.warps = (int)warps;
  const size_t smem = (size_t)(1 + warps) * (gmax + 1) * sizeof(int32_t);
  cudaError_t err = cudaFuncSetAttribute(routing_lists_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (err != cudaSuccess) return err;
  dim3 grid((unsigned)bh, 2);
  routing_lists_kernel<<<grid, ROUTE_THREADS, smem, st>>>(prm);
  return cudaGetLastError();
}
