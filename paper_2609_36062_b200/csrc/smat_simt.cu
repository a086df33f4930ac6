// fp32-ALU kernels of libsmat: the generic grouped GEMM (every contraction of Algorithm 1 and of the
// backward pass when no tensor-core kernel applies: fp32 inputs, odd shapes), the chunk-state scans,
// the direct form of Algorithm 2 and its transpose, and the debug mask.
#include <cuda_bf16.h>

#include "smat_internal.h"

namespace {

constexpr int TILE = 64;   // output tile edge
constexpr int KSTEP = 16;  // reduction step
constexpr int LDS = TILE + 4;

__device__ __forceinline__ float load_elem(const SmatOperand& o, int64_t off) {
  if (o.bf16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(o.ptr)[off]);
  return reinterpret_cast<const float*>(o.ptr)[off];
}

__global__ void __launch_bounds__(256) gemm_grouped_kernel(const SmatGemmArgs a) {
  const int64_t g = blockIdx.y;
  const int64_t bh = blockIdx.z;
  const SmatTokens tk = smat_group_tokens(a.grp, bh, g);
  const int64_t cnt = tk.cnt;
  const int M = a.tokM ? (int)cnt : a.M;
  const int N = a.tokN ? (int)cnt : a.N;
  const int K = a.tokK ? (int)cnt : a.K;
  const int m0 = (blockIdx.x / a.tilesN) * TILE;
  const int n0 = (blockIdx.x % a.tilesN) * TILE;
  if (m0 >= M || n0 >= N) return;

  __shared__ __align__(16) float As[KSTEP][LDS];
  __shared__ __align__(16) float Bs[KSTEP][LDS];

  const int tid = threadIdx.x;
  const int ty = tid >> 4, tx = tid & 15;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  const int64_t baseA = bh * a.A.s_bh + g * a.A.s_g;
  const int64_t baseB = bh * a.B.s_bh + g * a.B.s_g;
  const bool a_k_contig = (a.A.s1 == 1 && !a.A.tok1);
  const bool b_n_contig = (a.B.s1 == 1 && !a.B.tok1);
  const bool skip = a.tril && (n0 > m0 + TILE - 1);  // tile entirely above the diagonal

  for (int k0 = 0; k0 < K && !skip; k0 += KSTEP) {
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      const int e = tid + 256 * p;
      int mm, kk;
      if (a_k_contig) { kk = e & (KSTEP - 1); mm = e >> 4; } else { mm = e & (TILE - 1); kk = e >> 6; }
      float v = 0.f;
      if (m0 + mm < M && k0 + kk < K) {
        const int64_t x0 = a.A.tok0 ? tk.at(m0 + mm) : (int64_t)(m0 + mm);
        const int64_t x1 = a.A.tok1 ? tk.at(k0 + kk) : (int64_t)(k0 + kk);
        v = load_elem(a.A, baseA + x0 * a.A.s0 + x1 * a.A.s1);
      }
      As[kk][mm] = v;
    }
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      const int e = tid + 256 * p;
      int nn, kk;
      if (b_n_contig) { nn = e & (TILE - 1); kk = e >> 6; } else { kk = e & (KSTEP - 1); nn = e >> 4; }
      float v = 0.f;
      if (n0 + nn < N && k0 + kk < K) {
        const int64_t x0 = a.B.tok0 ? tk.at(k0 + kk) : (int64_t)(k0 + kk);
        const int64_t x1 = a.B.tok1 ? tk.at(n0 + nn) : (int64_t)(n0 + nn);
        v = load_elem(a.B, baseB + x0 * a.B.s0 + x1 * a.B.s1);
      }
      Bs[kk][nn] = v;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < KSTEP; ++kk) {
      const float4 av = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
      const float4 bv = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
      const float ar[4] = {av.x, av.y, av.z, av.w};
      const float br[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(ar[i], br[j], acc[i][j]);
    }
    __syncthreads();
  }

  const int64_t baseC = bh * a.C.s_bh + g * a.C.s_g;
  const int64_t baseI = bh * a.Cin.s_bh + g * a.Cin.s_g;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= M) continue;
    const int64_t x0 = a.C.tok0 ? tk.at(m) : (int64_t)m;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= N) continue;
      const int64_t x1 = a.C.tok1 ? tk.at(n) : (int64_t)n;
      float v = (a.tril && n > m) ? 0.f : acc[i][j];
      if (a.lam && a.tril && n <= m) {   // gated: decay between the key's and the query's position
        const float* l = a.lam + bh * a.grp.T;
        v *= __expf(l[tk.at(m)] - l[tk.at(n)]);
      }
      if (a.Cin.ptr) v += reinterpret_cast<const float*>(a.Cin.ptr)[baseI + x0 * a.Cin.s0 + x1 * a.Cin.s1];
      const int64_t off = baseC + x0 * a.C.s0 + x1 * a.C.s1;
      if (a.C.bf16)
        reinterpret_cast<__nv_bfloat16*>(const_cast<void*>(a.C.ptr))[off] = __float2bfloat16_rn(v);
      else
        reinterpret_cast<float*>(const_cast<void*>(a.C.ptr))[off] = v;
    }
  }
}

// ---- scan --------------------------------------------------------------------------------------
// Each thread owns four consecutive state entries and walks the chunks of its range in order.
// Loads are issued sixteen chunks ahead of the dependent additions.
__global__ void __launch_bounds__(256) scan_kernel(float* S, int64_t state_elems, int64_t NC, int64_t lo0, int64_t hi0,
                                                   int64_t lo1, int64_t hi1, int reverse) {
  const int64_t e4 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e4 * 4 >= state_elems) return;
  const int64_t bh = blockIdx.y;
  const int64_t lo = blockIdx.z ? lo1 : lo0, hi = blockIdx.z ? hi1 : hi0;
  float4* base = reinterpret_cast<float4*>(S + bh * NC * state_elems) + e4;
  const int64_t stride4 = state_elems / 4;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  constexpr int AHEAD = 16;
  for (int64_t s = 0; s < hi - lo; s += AHEAD) {
    float4 v[AHEAD];
#pragma unroll
    for (int u = 0; u < AHEAD; ++u) {
      const int64_t k = s + u;
      if (k < hi - lo) v[u] = base[(reverse ? hi - 1 - k : lo + k) * stride4];
    }
#pragma unroll
    for (int u = 0; u < AHEAD; ++u) {
      const int64_t k = s + u;
      if (k < hi - lo) {
        base[(reverse ? hi - 1 - k : lo + k) * stride4] = acc;
        acc.x += v[u].x; acc.y += v[u].y; acc.z += v[u].z; acc.w += v[u].w;
      }
    }
  }
}

// ---- Algorithm 2, direct form ------------------------------------------------------------------------
// The CTA copies its slab (E consecutive state entries) of all input states into shared memory, then
// every (output state, entry) pair is summed by one thread.  Offsets aᵀx are maintained by a base-q
// counter: bumping a digit q times returns the running dot product to where it started, so a carry
// needs no correction.
__global__ void __launch_bounds__(256) tabulate_alg2_kernel(const float* __restrict__ in, float* __restrict__ out,
                                                            const SmatGeo geo, int64_t state_elems, int E,
                                                            int transpose) {
  extern __shared__ __align__(16) float slab[];
  const int64_t rows_in = transpose ? geo.B : geo.P;
  const int64_t rows_out = transpose ? geo.P : geo.B;
  const int64_t bh = blockIdx.y;
  const int64_t e0 = (int64_t)blockIdx.x * E;
  const float* src = in + bh * rows_in * state_elems + e0;
  for (int64_t idx = threadIdx.x; idx < rows_in * E; idx += blockDim.x) {
    const int64_t x = idx / E;
    const int e = (int)(idx - x * E);
    slab[idx] = src[x * state_elems + e];
  }
  __syncthreads();
  float* dst = out + bh * rows_out * state_elems + e0;
  const int q = geo.q, D = geo.D;
  for (int64_t item = threadIdx.x; item < rows_out * E; item += blockDim.x) {
    const int64_t row = item / E;
    const int e = (int)(item - row * E);
    float sum = 0.f;
    if (!transpose) {
      // hyperplane `row` = (direction a, offset b): visit its q^(D-1) points
      int32_t a[SMAT_MAX_DIM];
      smat_direction(geo, row / q, a);
      const int b = (int)(row % q);
      int lead = 0;
      while (a[lead] == 0) ++lead;
      int digit[SMAT_MAX_DIM];
      for (int k = 0; k < D; ++k) digit[k] = 0;
      int s = 0;        // Σ over free coordinates of a_k x_k  (mod q)
      int64_t v = 0;    // packed index of the free coordinates
      const int64_t npts = geo.qpow[D - 1];
      for (int64_t it = 0; it < npts; ++it) {
        int xl = b - s;
        if (xl < 0) xl += q;
        sum += slab[(v + (int64_t)xl * geo.qpow[lead]) * E + e];
        for (int k = 0; k < D; ++k) {  // bump the counter over the free coordinates
          if (k == lead) continue;
          s += a[k];
          if (s >= q) s -= q;
          v += geo.qpow[k];
          if (++digit[k] < q) break;
          digit[k] = 0;
          v -= geo.qpow[k + 1];
        }
      }
    } else {
      // point `row`: one hyperplane per direction, offset aᵀx
      int x[SMAT_MAX_DIM];
      int64_t vv = row;
      for (int k = 0; k < D; ++k) { x[k] = (int)(vv % q); vv /= q; }
      for (int lead = 0; lead < D; ++lead) {
        int digit[SMAT_MAX_DIM];
        for (int k = 0; k < D; ++k) digit[k] = 0;
        int dot = x[lead];
        int64_t dir = geo.dir_group_start[lead];
        const int64_t ndir = geo.qpow[D - 1 - lead];
        for (int64_t it = 0; it < ndir; ++it, ++dir) {
          sum += slab[(dir * q + dot) * E + e];
          for (int k = lead + 1; k < D; ++k) {
            dot += x[k];
            if (dot >= q) dot -= q;
            if (++digit[k] < q) break;
            digit[k] = 0;
          }
        }
      }
    }
    dst[row * state_elems + e] = sum;
  }
}

__global__ void mask_kernel(uint8_t* mask, const SmatGeo geo) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= geo.T * geo.T) return;
  mask[idx] = (uint8_t)smat_mask_entry(geo, idx / geo.T, idx % geo.T);
}

}  // namespace

cudaError_t smat_launch_gemm(const SmatGemmArgs& a_in, int max_M, int max_N, int64_t groups, int bh, cudaStream_t st) {
  if (groups <= 0 || max_M <= 0 || max_N <= 0) return cudaSuccess;
  SmatGemmArgs a = a_in;
  a.tilesN = (max_N + TILE - 1) / TILE;
  const int tilesM = (max_M + TILE - 1) / TILE;
  dim3 grid((unsigned)(tilesM * a.tilesN), (unsigned)groups, (unsigned)bh);
  gemm_grouped_kernel<<<grid, 256, 0, st>>>(a);
  return cudaGetLastError();
}

cudaError_t smat_launch_scan(float* S, int64_t state_elems, int64_t NC, int bh, int64_t lo0, int64_t hi0, int64_t lo1,
                             int64_t hi1, int reverse, cudaStream_t st) {
  const int ranges = (hi1 > lo1) ? 2 : 1;
  dim3 grid((unsigned)((state_elems / 4 + 255) / 256), (unsigned)bh, (unsigned)ranges);
  scan_kernel<<<grid, 256, 0, st>>>(S, state_elems, NC, lo0, hi0, lo1, hi1, reverse);
  return cudaGetLastError();
}

int smat_tabulate_alg2_slab(int64_t rows_in, int64_t state_elems) {
  const int64_t budget = 200 * 1024;
  int E = 128;
  while (E >= 1 && (rows_in * E * 4 > budget || state_elems % E != 0)) E >>= 1;
  return E;
}

cudaError_t smat_launch_tabulate_alg2(const float* in, float* out, const SmatGeo& geo, int64_t state_elems, int bh,
                                      int transpose, cudaStream_t st) {
  const int64_t rows_in = transpose ? geo.B : geo.P;
  const int E = smat_tabulate_alg2_slab(rows_in, state_elems);
  if (E < 1) return cudaErrorInvalidConfiguration;
  const size_t smem = (size_t)rows_in * E * sizeof(float);
  cudaError_t err = cudaFuncSetAttribute(tabulate_alg2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (err != cudaSuccess) return err;
  dim3 grid((unsigned)(state_elems / E), (unsigned)bh);
  tabulate_alg2_kernel<<<grid, 256, smem, st>>>(in, out, geo, state_elems, E, transpose);
  return cudaGetLastError();
}

cudaError_t smat_launch_mask(uint8_t* mask, const SmatGeo& geo, cudaStream_t st) {
  const int64_t total = geo.T * geo.T;
  mask_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(mask, geo);
  return cudaGetLastError();
}
