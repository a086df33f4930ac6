// Long-range branch, tabulation U = C F (Algorithm 2) as staged exact sums for d = 3, 4, and its transpose.
// The sums run on the plain fp32 ALUs: the incidence matrix is sparse (density 1/q) and every state entry is
// an independent copy of the same integer-indexed map, so this is not a dense contraction.
#include <cuda_bf16.h>

#include "smat_internal.h"

namespace {

// two packed fp32x2 additions (one instruction per pair on sm_100)
__device__ __forceinline__ float4 add4(const float4 a, const float4 b) {
  const float2 lo = __fadd2_rn(make_float2(a.x, a.y), make_float2(b.x, b.y));
  const float2 hi = __fadd2_rn(make_float2(a.z, a.w), make_float2(b.z, b.w));
  return make_float4(lo.x, lo.y, hi.x, hi.y);
}
// One float4 of a result state, written as fp32 (16 bytes) or rounded to bf16 (8 bytes); `idx4` counts float4s.
template <int BF16>
__device__ __forceinline__ void store_out4(void* base, int64_t idx4, const float4 v) {
  if (BF16) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
    uint2 pk;
    pk.x = *reinterpret_cast<const uint32_t*>(&lo);
    pk.y = *reinterpret_cast<const uint32_t*>(&hi);
    reinterpret_cast<uint2*>(base)[idx4] = pk;
  } else {
    reinterpret_cast<float4*>(base)[idx4] = v;
  }
}
// 16-byte asynchronous copy global -> shared, bypassing registers
__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"((unsigned)__cvta_generic_to_shared(smem)), "l"(gmem)
               : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
  asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;\n" ::: "memory");
}

// ---- staged exact tabulation -------------------------------------------------------------------------------------
// U_{a,b} = Σ_{x : aᵀx = b} F_x for every normalised direction a and offset b (Algorithm 2), evaluated
// one coordinate at a time instead of one hyperplane at a time.  For D = d-1 = 3 and a = (1, a2, a3):
//     W_{a3}[u, x2]   = Σ_{x3} F[u - a3 x3, x2, x3]          (q adds for each of q^2 entries, per a3)
//     U_{a,b}         = Σ_{x2} W_{a3}[b - a2 x2, x2]         (q adds for each of q^2 (a2, b) pairs, per a3)
// which costs 2 q^4 state additions for the q^2 directions of this group instead of q^5; directions with
// a leading zero work on F summed over x1 (and x2).  The sums are the same real numbers as Algorithm 2's,
// added in a different order.  Every state entry is an independent copy of this map, so a CTA owns a slab
// of E consecutive entries, keeps F[:, slab] in shared memory and writes U[:, slab].
// Layout in shared memory: point index major, E floats per point; a thread owns one float4 of an item.
template <int D, int BF16>
__global__ void __launch_bounds__(1024, 1) tabulate_staged_kernel(const float* __restrict__ in, void* __restrict__ out,
                                                              int q, int64_t P, int64_t Bn, int64_t state_elems,
                                                              int E) {
  extern __shared__ __align__(16) float4 smem4[];
  const int L4 = E / 4;                 // float4 lanes per item
  const int NT = blockDim.x;
  const int IPP = NT / L4;              // items per pass
  const int tid = threadIdx.x;
  const int l = tid % L4, it0 = tid / L4;
  const int64_t bh = blockIdx.y;
  const int64_t e0 = (int64_t)blockIdx.x * E;
  const int qq = q * q;
  float4* Fs = smem4;                                  // [P][L4]
  const float4* src = reinterpret_cast<const float4*>(in + bh * P * state_elems + e0);
  const int64_t row4 = state_elems / 4;
  for (int64_t idx = tid; idx < P * L4; idx += NT) {
    const int64_t x = idx / L4;
    cp_async16(Fs + idx, src + x * row4 + (idx - x * L4));
  }
  cp_async_wait_all();
  __syncthreads();
  const int64_t out0 = (bh * Bn * state_elems + e0) / 4;  // first float4 of this CTA's slab in the result table
  const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);

  if (D == 2) {
    // a = (1, a2):  U[a2*q + b] = Σ_{x2} F[(b - a2 x2) mod q, x2]
    for (int item = it0; item < qq; item += IPP) {
      const int a2 = item / q, b = item - a2 * q;
      float4 acc = zero;
      int x1 = b;
#pragma unroll 4
      for (int x2 = 0; x2 < q; ++x2) {
        acc = add4(acc, Fs[(x1 + q * x2) * L4 + l]);
        x1 -= a2;
        if (x1 < 0) x1 += q;
      }
      store_out4<BF16>(out, out0 + (int64_t)item * row4 + l, acc);
    }
    // a = (0, 1):  U[q*q + b] = Σ_{x1} F[x1, b]
    for (int b = it0; b < q; b += IPP) {
      float4 acc = zero;
#pragma unroll 4
      for (int x1 = 0; x1 < q; ++x1) acc = add4(acc, Fs[(x1 + q * b) * L4 + l]);
      store_out4<BF16>(out, out0 + (int64_t)(qq + b) * row4 + l, acc);
    }
  } else {
    float4* G2 = Fs + P * L4;          // [q*q][L4]   F summed over x1, indexed x2 + q*x3
    float4* W = G2 + (int64_t)qq * L4;  // [2][q*q][L4] double-buffered W_{a3}, indexed u + q*x2
    for (int item = it0; item < qq; item += IPP) {
      float4 acc = zero;
      const float4* p = Fs + (int64_t)item * q * L4 + l;
#pragma unroll 4
      for (int x1 = 0; x1 < q; ++x1) acc = add4(acc, p[x1 * L4]);
      G2[item * L4 + l] = acc;
    }
    __syncthreads();
    // a = (0, 1, a3):  U[(q^2 + a3) q + b] = Σ_{x3} G2[(b - a3 x3) mod q, x3]
    for (int item = it0; item < qq; item += IPP) {
      const int a3 = item / q, b = item - a3 * q;
      float4 acc = zero;
      int x2 = b;
#pragma unroll 4
      for (int x3 = 0; x3 < q; ++x3) {
        acc = add4(acc, G2[(x2 + q * x3) * L4 + l]);
        x2 -= a3;
        if (x2 < 0) x2 += q;
      }
      store_out4<BF16>(out, out0 + (int64_t)(qq * q + item) * row4 + l, acc);
    }
    // a = (0, 0, 1):  U[(q^2 + q) q + b] = Σ_{x2} G2[x2, b]
    for (int b = it0; b < q; b += IPP) {
      float4 acc = zero;
#pragma unroll 4
      for (int x2 = 0; x2 < q; ++x2) acc = add4(acc, G2[(x2 + q * b) * L4 + l]);
      store_out4<BF16>(out, out0 + (int64_t)((qq + q) * q + b) * row4 + l, acc);
    }
    // a = (1, a2, a3)
    for (int a3 = 0; a3 < q; ++a3) {
      float4* Wc = W + (int64_t)(a3 & 1) * qq * L4;
      for (int item = it0; item < qq; item += IPP) {       // item = u + q*x2
        const int x2 = item / q, u = item - x2 * q;
        float4 acc = zero;
        int x1 = u;
        const float4* p = Fs + (int64_t)(q * x2) * L4 + l;
#pragma unroll 4
        for (int x3 = 0; x3 < q; ++x3) {
          acc = add4(acc, p[(x1 + qq * x3) * L4]);
          x1 -= a3;
          if (x1 < 0) x1 += q;
        }
        Wc[item * L4 + l] = acc;
      }
      __syncthreads();
      for (int item = it0; item < qq; item += IPP) {       // item = b + q*a2
        const int a2 = item / q, b = item - a2 * q;
        float4 acc = zero;
        int u = b;
#pragma unroll 4
        for (int x2 = 0; x2 < q; ++x2) {
          acc = add4(acc, Wc[(u + q * x2) * L4 + l]);
          u -= a2;
          if (u < 0) u += q;
        }
        const int64_t h = (int64_t)(a2 + q * a3) * q + b;
        store_out4<BF16>(out, out0 + h * row4 + l, acc);
      }
    }
  }
}

// ---- D = 3 with the whole q x q image of a sub-problem held in registers --------------------------------------------
// For a fixed x2 (and one state entry) the sums W_{a3}[u, x2] = Σ_{x3} F[u - a3 x3, x2, x3] over all (a3, u) are
// the finite Radon transform of the q x q image F[., x2, .]: q^2 inputs, q^2 outputs, q^3 additions.  A thread
// loads one image into registers, forms every line sum with compile-time indices (no address arithmetic, no
// shared-memory read per addition) and writes the q^2 results back over the image it read.  The second stage is
// the same transform of the image W_{a3}[., .] for a fixed a3; its results again replace the image, which leaves
// rows 0 .. q^3-1 of U in the slab, in order, ready for a coalesced copy out.
// Line sums of slope A: out[v] = Σ_y img[y][(v - A y) mod Q], stored with stride `os`.
template <int Q, int A>
struct RadonSlope {
  static __device__ __forceinline__ void run(const float (&img)[Q][Q], float* out, int os) {
    float p[Q];  // the Q sums advance together, one image row at a time: Q independent additions per step
#pragma unroll
    for (int v = 0; v < Q; ++v) p[v] = img[0][v];
#pragma unroll
    for (int y = 1; y < Q; ++y)
#pragma unroll
      for (int v = 0; v < Q; ++v) p[v] += img[y][((v - A * y) % Q + Q) % Q];
#pragma unroll
    for (int v = 0; v < Q; ++v) out[v * os] = p[v];
  }
};

// All Q slopes in turn.  The empty asm between two slopes keeps the compiler from interleaving their sums, which
// would multiply the number of live partial sums (and spill the image).
template <int Q, int A = 0>
__device__ __forceinline__ void radon_all_slopes(const float (&img)[Q][Q], float* base, int slope_stride, int os) {
  if constexpr (A < Q) {
    RadonSlope<Q, A>::run(img, base + A * slope_stride, os);
    asm volatile("" ::: "memory");
    radon_all_slopes<Q, A + 1>(img, base, slope_stride, os);
  }
}

// One in-place transform: image[y][x] at base[(x + y * SY) * E], slope a results to base[(x + a * SY) * E].
// Kept out of line so that the two transforms of the kernel get their registers allocated independently.
template <int Q, int E, int SY>
__device__ __noinline__ void radon_inplace(float* base) {
  float img[Q][Q];
#pragma unroll
  for (int y = 0; y < Q; ++y)
#pragma unroll
    for (int x = 0; x < Q; ++x) img[y][x] = base[(x + y * SY) * E];
  radon_all_slopes<Q>(img, base, SY * E, E);
}

// Register budget: 168 keeps two 192-thread CTAs per SM (q <= 11); the 7-warp CTAs of q = 13 may take 224.
// Larger fields do not fit a q x q image in the registers of one thread and use tabulate_staged_kernel.
template <int Q, int E, int BF16>
__global__ void __maxnreg__(Q <= 11 ? 168 : 224)
    tabulate_radon3_kernel(const float* __restrict__ in, void* __restrict__ out, int P, int Bn, int64_t state_elems) {
  extern __shared__ __align__(16) float4 smem4[];
  constexpr int q = Q, qq = Q * Q;
  constexpr int L4 = E / 4;
  constexpr int log2L4 = E == 32 ? 3 : 2;
  static_assert(E == 16 || E == 32, "slab width");
  const int NT = blockDim.x;
  const int IPP = NT >> log2L4;
  const int tid = threadIdx.x;
  const int l = tid & (L4 - 1), it0 = tid >> log2L4;
  const int64_t bh = blockIdx.y;
  const int64_t e0 = (int64_t)blockIdx.x * E;
  float4* Fs = smem4;
  const float4* src = reinterpret_cast<const float4*>(in + bh * P * state_elems + e0);
  const int row4 = (int)(state_elems / 4);
  for (int idx = tid; idx < P * L4; idx += NT) cp_async16(Fs + idx, src + (int64_t)(idx >> log2L4) * row4 + (idx & (L4 - 1)));
  cp_async_wait_all();
  __syncthreads();
  const int64_t out0 = (bh * Bn * state_elems + e0) / 4;  // first float4 of this CTA's slab in the result table
  const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
  // directions with a leading zero work on G2[x2, x3] = Σ_{x1} F[x1, x2, x3]
  float4* G2 = Fs + P * L4;
  for (int item = it0; item < qq; item += IPP) {
    float4 acc = zero;
    const float4* p = Fs + item * q * L4 + l;
#pragma unroll
    for (int x1 = 0; x1 < q; ++x1) acc = add4(acc, p[x1 * L4]);
    G2[item * L4 + l] = acc;
  }
  __syncthreads();
  for (int item = it0; item < qq; item += IPP) {  // a = (0, 1, a3)
    const int a3 = item / q, b = item - a3 * q;
    float4 acc = zero;
    int x2 = b;
#pragma unroll
    for (int x3 = 0; x3 < q; ++x3) {
      acc = add4(acc, G2[(x2 + q * x3) * L4 + l]);
      x2 -= a3;
      if (x2 < 0) x2 += q;
    }
    store_out4<BF16>(out, out0 + (int64_t)(qq * q + item) * row4 + l, acc);
  }
  for (int b = it0; b < q; b += IPP) {  // a = (0, 0, 1)
    float4 acc = zero;
#pragma unroll
    for (int x2 = 0; x2 < q; ++x2) acc = add4(acc, G2[(x2 + q * b) * L4 + l]);
    store_out4<BF16>(out, out0 + (int64_t)((qq + q) * q + b) * row4 + l, acc);
  }
  // a = (1, a2, a3), stage 1: thread (x2, e) transforms the image F[., x2, .] in place
  float* Ff = reinterpret_cast<float*>(Fs);
  const int e = tid & (E - 1), it = tid >> (log2L4 + 2);
  if (it < q) radon_inplace<Q, E, Q * Q>(Ff + (q * it) * E + e);  // image [x3][x1]; W_{a3}[u, x2] over F[u, x2, a3]
  __syncthreads();
  // stage 2: thread (a3, e) transforms the image W_{a3}[., .]:  U_{(1,a2,a3), b} = Σ_{x2} W_{a3}[b - a2 x2, x2];
  // slot b + q a2 + q^2 a3 is row h = (a2 + q a3) q + b of U
  if (it < q) radon_inplace<Q, E, Q>(Ff + (qq * it) * E + e);  // image [x2][u]
  __syncthreads();
  for (int idx = tid; idx < P * L4; idx += NT)  // rows 0 .. q^3-1 of U, 16-byte stores
    store_out4<BF16>(out, out0 + (int64_t)(idx >> log2L4) * row4 + (idx & (L4 - 1)), Fs[idx]);
}

// Transpose for D = 2:  F̄[x1, x2] = Σ_{a2} Ū[(1,a2), x1 + a2 x2] + Ū[(0,1), x2]
template <int BF16>
__global__ void __launch_bounds__(1024, 1) tabulate_staged_t2_kernel(const float* __restrict__ in, void* __restrict__ out,
                                                                 int q, int64_t P, int64_t Bn, int64_t state_elems,
                                                                 int E) {
  extern __shared__ __align__(16) float4 smem4[];
  const int L4 = E / 4, NT = blockDim.x, IPP = NT / L4;
  const int tid = threadIdx.x;
  const int l = tid % L4, it0 = tid / L4;
  const int64_t bh = blockIdx.y;
  const int64_t e0 = (int64_t)blockIdx.x * E;
  const int qq = q * q;
  float4* Us = smem4;  // [Bn][L4]
  const float4* src = reinterpret_cast<const float4*>(in + bh * Bn * state_elems + e0);
  const int64_t row4 = state_elems / 4;
  for (int64_t idx = tid; idx < Bn * L4; idx += NT) {
    const int64_t h = idx / L4;
    cp_async16(Us + idx, src + h * row4 + (idx - h * L4));
  }
  cp_async_wait_all();
  __syncthreads();
  const int64_t out0 = (bh * P * state_elems + e0) / 4;
  for (int item = it0; item < qq; item += IPP) {  // item = x1 + q*x2
    const int x2 = item / q, x1 = item - x2 * q;
    float4 acc = Us[(qq + x2) * L4 + l];
    int b = x1;
#pragma unroll 4
    for (int a2 = 0; a2 < q; ++a2) {
      acc = add4(acc, Us[(a2 * q + b) * L4 + l]);
      b += x2;
      if (b >= q) b -= q;
    }
    store_out4<BF16>(out, out0 + (int64_t)item * row4 + l, acc);
  }
}

template <typename K>
cudaError_t set_smem(K kernel, size_t bytes) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

}  // namespace

__global__ void widen_bf16_kernel(const __nv_bfloat16* __restrict__ src, float* __restrict__ dst, int64_t count) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count) dst[i] = __bfloat162float(src[i]);
}

// ---- launchers ------------------------------------------------------------------------------------------------------
// Shared-memory floats per slab entry the staged kernels need.
// slab width of the register-resident form for the field sizes it is compiled for (0: not available)
static int radon3_slab(int q) { return q == 5 || q == 7 ? 32 : (q == 11 || q == 13 ? 16 : 0); }
static bool radon3_q(int q) { return radon3_slab(q) != 0; }
static int64_t staged_rows(const SmatGeo& geo, int transpose) {
  const int64_t q = geo.q;
  if (geo.D == 2) return transpose ? geo.B : geo.P;
  if (geo.D == 3 && !transpose) return radon3_q(geo.q) ? geo.P + q * q : geo.P + 3 * q * q;
  return 0;
}

int smat_tabulate_staged_slab(const SmatGeo& geo, int64_t state_elems, int transpose) {
  const int64_t rows = staged_rows(geo, transpose);
  if (rows == 0) return 0;
  if (geo.D == 3 && !transpose && radon3_q(geo.q) && state_elems % 32 == 0) return radon3_slab(geo.q);
  // prefer two resident CTAs per SM (about 110 KB each) with at least 16 entries, else the largest slab that fits
  const int64_t two = 110 * 1024, one = 220 * 1024;
  for (int E = 32; E >= 16; E >>= 1)
    if (rows * E * 4 <= two && state_elems % E == 0) return E;
  for (int E = 32; E >= 4; E >>= 1)
    if (rows * E * 4 <= one && state_elems % E == 0) return E;
  return 0;
}

cudaError_t smat_launch_tabulate_staged(const float* in, void* out, const SmatGeo& geo, int64_t state_elems, int bh,
                                        int transpose, int out_bf16, cudaStream_t st) {
  if (out_bf16 && transpose && geo.D != 2) return cudaErrorInvalidValue;
  const int E = smat_tabulate_staged_slab(geo, state_elems, transpose);
  if (E < 4) return cudaErrorInvalidConfiguration;
  const size_t smem = (size_t)staged_rows(geo, transpose) * E * sizeof(float);
  dim3 grid((unsigned)(state_elems / E), (unsigned)bh);
  // threads: one (item, float4 lane) unit each, q^2 items per stage, split evenly over as few passes as possible
  const int64_t units = (int64_t)geo.q * geo.q * (E / 4);
  const int64_t passes = (units + 1023) / 1024;
  int nt = (int)(((units + passes - 1) / passes + 31) / 32 * 32);
  if (nt < 128) nt = 128;
  // d = 3 has no barrier between its sums: small CTAs, several per SM, overlap one CTA's slab load with another's sums
  if (geo.D == 2 && nt > 256) nt = 256;
  cudaError_t err;
  if (geo.D == 3 && !transpose && radon3_q(geo.q)) {
#define SMAT_RADON3(QV, EV)                                                                                      \
  if (geo.q == QV && E == EV) {                                                                                  \
    const int nr = (QV * EV + 31) / 32 * 32; /* one thread per (image, entry) */                                 \
    if (out_bf16) {                                                                                              \
      if ((err = set_smem(tabulate_radon3_kernel<QV, EV, 1>, smem)) != cudaSuccess) return err;                  \
      tabulate_radon3_kernel<QV, EV, 1><<<grid, nr, smem, st>>>(in, out, (int)geo.P, (int)geo.B, state_elems);   \
    } else {                                                                                                     \
      if ((err = set_smem(tabulate_radon3_kernel<QV, EV, 0>, smem)) != cudaSuccess) return err;                  \
      tabulate_radon3_kernel<QV, EV, 0><<<grid, nr, smem, st>>>(in, out, (int)geo.P, (int)geo.B, state_elems);   \
    }                                                                                                            \
    return cudaGetLastError();                                                                                   \
  }
    SMAT_RADON3(5, 32) SMAT_RADON3(7, 32) SMAT_RADON3(11, 16) SMAT_RADON3(13, 16)
#undef SMAT_RADON3
    return cudaErrorInvalidConfiguration;
  }
  if (geo.D == 2 && transpose) {
    if (out_bf16) {
      if ((err = set_smem(tabulate_staged_t2_kernel<1>, smem)) != cudaSuccess) return err;
      tabulate_staged_t2_kernel<1><<<grid, nt, smem, st>>>(in, out, geo.q, geo.P, geo.B, state_elems, E);
    } else {
      if ((err = set_smem(tabulate_staged_t2_kernel<0>, smem)) != cudaSuccess) return err;
      tabulate_staged_t2_kernel<0><<<grid, nt, smem, st>>>(in, out, geo.q, geo.P, geo.B, state_elems, E);
    }
  } else {
#define SMAT_STAGED(DV, BV)                                                                         \
  if (geo.D == DV && out_bf16 == BV) {                                                              \
    if ((err = set_smem(tabulate_staged_kernel<DV, BV>, smem)) != cudaSuccess) return err;          \
    tabulate_staged_kernel<DV, BV><<<grid, nt, smem, st>>>(in, out, geo.q, geo.P, geo.B, state_elems, E); \
  }
    SMAT_STAGED(2, 0) SMAT_STAGED(2, 1) SMAT_STAGED(3, 0) SMAT_STAGED(3, 1)
#undef SMAT_STAGED
  }
  return cudaGetLastError();
}

// ---- d = 3 with bf16 tables and a prime too large for the resident-matrix kernel --------------------------------
// U = R F (the two-dimensional Radon sums of Algorithm 2 for d = 3) from a bf16 profile table: the slab F[:, e0 .. e0+E)
// sits in shared memory as bf16, a thread owns 8 entries of one output row and adds in fp32.  Against the fp32 form
// this halves the shared-memory bytes per addition, which is what bounds these sums.
__global__ void __launch_bounds__(256) tabulate_d3_bf16_kernel(const __nv_bfloat16* __restrict__ in,
                                                               __nv_bfloat16* __restrict__ out, int q, int64_t P,
                                                               int64_t Bn, int64_t state_elems, int E) {
  extern __shared__ __align__(16) uint4 smem8[];            // [P][E / 8]: 8 bf16 per element
  const int L8 = E / 8, NT = blockDim.x, tid = threadIdx.x;
  const int l = tid % L8, it0 = tid / L8, IPP = NT / L8;
  const int64_t bh = blockIdx.y, e0 = (int64_t)blockIdx.x * E;
  const int qq = q * q;
  const uint4* src = reinterpret_cast<const uint4*>(in + (bh * P) * state_elems + e0);
  const int64_t row8 = state_elems / 8;
  for (int64_t idx = tid; idx < P * L8; idx += NT) {
    const int64_t x = idx / L8;
    cp_async16(smem8 + idx, src + x * row8 + (idx - x * L8));
  }
  cp_async_wait_all();
  __syncthreads();
  uint4* dst = reinterpret_cast<uint4*>(out + (bh * Bn) * state_elems + e0);
  auto add8 = [](float (&acc)[8], const uint4 w) {
    const uint32_t v[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 s = __fadd2_rn(make_float2(acc[2 * i], acc[2 * i + 1]),
                                  make_float2(__uint_as_float(v[i] << 16), __uint_as_float(v[i] & 0xffff0000u)));
      acc[2 * i] = s.x; acc[2 * i + 1] = s.y;
    }
  };
  auto store8 = [&](int64_t row, const float (&acc)[8]) {
    uint4 w;
    const __nv_bfloat162 a = __floats2bfloat162_rn(acc[0], acc[1]), b = __floats2bfloat162_rn(acc[2], acc[3]),
                         c = __floats2bfloat162_rn(acc[4], acc[5]), d = __floats2bfloat162_rn(acc[6], acc[7]);
    w.x = *reinterpret_cast<const uint32_t*>(&a); w.y = *reinterpret_cast<const uint32_t*>(&b);
    w.z = *reinterpret_cast<const uint32_t*>(&c); w.w = *reinterpret_cast<const uint32_t*>(&d);
    dst[row * row8 + l] = w;
  };
  // a = (1, a2):  U[a2*q + b] = Σ_{x2} F[(b - a2 x2) mod q, x2]
  for (int item = it0; item < qq; item += IPP) {
    const int a2 = item / q, b = item - a2 * q;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    int x1 = b;
#pragma unroll 4
    for (int x2 = 0; x2 < q; ++x2) {
      add8(acc, smem8[(x1 + q * x2) * L8 + l]);
      x1 -= a2;
      if (x1 < 0) x1 += q;
    }
    store8(item, acc);
  }
  // a = (0, 1):  U[q*q + b] = Σ_{x1} F[x1, b]
  for (int b = it0; b < q; b += IPP) {
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
    for (int x1 = 0; x1 < q; ++x1) add8(acc, smem8[(x1 + q * b) * L8 + l]);
    store8(qq + b, acc);
  }
}

// Entries per CTA slab of tabulate_d3_bf16_kernel (two CTAs per SM), or 0 when the geometry is not covered.
int smat_tabulate_d3_bf16_slab(const SmatGeo& geo, int64_t state_elems) {
  if (geo.D != 2) return 0;
  for (int E = 32; E >= 8; E >>= 1)
    if (geo.P * E * 2 <= 110 * 1024 && state_elems % E == 0) return E;
  return 0;
}

cudaError_t smat_launch_tabulate_d3_bf16(const void* in, void* out, const SmatGeo& geo, int64_t state_elems, int bh,
                                         cudaStream_t st) {
  const int E = smat_tabulate_d3_bf16_slab(geo, state_elems);
  if (!E) return cudaErrorInvalidConfiguration;
  const size_t smem = (size_t)geo.P * E * 2;
  cudaError_t err = set_smem(tabulate_d3_bf16_kernel, smem);
  if (err != cudaSuccess) return err;
  dim3 grid((unsigned)(state_elems / E), (unsigned)bh);
  tabulate_d3_bf16_kernel<<<grid, 256, smem, st>>>(static_cast<const __nv_bfloat16*>(in), static_cast<__nv_bfloat16*>(out),
                                                   geo.q, geo.P, geo.B, state_elems, E);
  return cudaGetLastError();
}

__global__ void widen_bf16_slabs_kernel(const __nv_bfloat16* __restrict__ src, float* __restrict__ dst, int64_t rows,
                                        int64_t rp, int64_t count) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;   // index into dst [heads][rows][rp]
  if (idx >= count) return;
  const int64_t e = idx % rp, row = (idx / rp) % rows, head = idx / (rp * rows);
  dst[idx] = __bfloat162float(src[((head * (rp / 32) + e / 32) * rows + row) * 32 + e % 32]);
}

cudaError_t smat_launch_widen_bf16_slabs(const void* src_bf16, float* dst, int64_t heads, int64_t rows, int64_t rp,
                                         cudaStream_t st) {
  const int64_t count = heads * rows * rp;
  widen_bf16_slabs_kernel<<<(unsigned)((count + 255) / 256), 256, 0, st>>>(static_cast<const __nv_bfloat16*>(src_bf16), dst,
                                                                           rows, rp, count);
  return cudaGetLastError();
}

cudaError_t smat_launch_widen_bf16(const void* src_bf16, float* dst, int64_t count, cudaStream_t st) {
  widen_bf16_kernel<<<(unsigned)((count + 255) / 256), 256, 0, st>>>(static_cast<const __nv_bfloat16*>(src_bf16), dst,
                                                                     count);
  return cudaGetLastError();
}
