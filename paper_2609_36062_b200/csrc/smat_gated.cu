// Small kernels of the scalar-gated variant (Sec. 3.2, Eq. "gated"; Lemma "Gated SMat"): the prefix sum λ of the
// log-gates, the rescaled copies of Q, K, V, dO that carry the query-side and key-side factors, the decayed scan of the
// chunk states and the gate gradient.  Every factor is the exponential of a difference λ_i - λ_j with j <= i, so it lies
// in (0, 1] and nothing can overflow.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "smat_internal.h"

namespace {

// Inclusive prefix (reverse = 0) or suffix (reverse = 1) sum of one row of `len` floats per head; one CTA per head.
__global__ void __launch_bounds__(1024) head_scan_kernel(const float* __restrict__ in, float* __restrict__ out, int64_t len,
                                                         int reverse) {
  __shared__ float warp_sum[32];
  __shared__ float carry;
  const int tid = threadIdx.x;
  const float* src = in + (int64_t)blockIdx.x * len;
  float* dst = out + (int64_t)blockIdx.x * len;
  if (tid == 0) carry = 0.f;
  __syncthreads();
  for (int64_t base = 0; base < len; base += 1024) {
    const int64_t k = base + tid;
    const int64_t idx = reverse ? len - 1 - k : k;
    const float v = k < len ? src[idx] : 0.f;
    float x = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const float y = __shfl_up_sync(0xffffffffu, x, d);
      if ((tid & 31) >= d) x += y;
    }
    if ((tid & 31) == 31) warp_sum[tid >> 5] = x;
    __syncthreads();
    float before = carry;
    for (int w = 0; w < (tid >> 5); ++w) before += warp_sum[w];
    if (k < len) dst[idx] = before + x;
    __syncthreads();
    if (tid == 1023) carry = before + x;
    __syncthreads();
  }
}

// Rescaled copy of token rows: out[t] = src[t] * f(t), dim values per row, in the plan's dtype.
//   mode 0 (query side of a chunk)   : f = exp(λ_t - λ_{s(t)-1}),  s(t) = first token of t's chunk (λ_{-1} = 0)
//   mode 1 (key side of a chunk)     : f = exp(λ_{e(t)} - λ_t),    e(t) = last token of t's chunk
//   mode 2 (the block boundary)      : t <  n: src = A, f = exp(λ_{n-1} - λ_t)   (key side, folded into Z_j)
//                                      t >= n: src = B, f = exp(λ_t - λ_{n-1})   (query side, on the read)
template <typename T>
__global__ void gate_scale_kernel(const T* __restrict__ A, const T* __restrict__ B, T* __restrict__ out,
                                  const float* __restrict__ lam, int mode, int64_t n, int64_t c, int64_t Tlen, int dim,
                                  int64_t rows) {
  const int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / 32;
  if (row >= rows) return;
  const int lane = threadIdx.x & 31;
  const int64_t bh = row / Tlen, t = row - bh * Tlen;
  const float* l = lam + bh * Tlen;
  float f;
  const T* src = A;
  if (mode == 0) {
    const int64_t s = t - t % c;
    f = __expf(l[t] - (s > 0 ? l[s - 1] : 0.f));
  } else if (mode == 1) {
    const int64_t e = t - t % c + c - 1;
    f = __expf(l[e] - l[t]);
  } else if (t < n) {
    f = __expf(l[n - 1] - l[t]);
  } else {
    f = __expf(l[t] - l[n - 1]);
    src = B;
  }
  if (dim % 128 == 0) {   // four consecutive elements per lane: 8-byte (bf16) or 16-byte (fp32) accesses
    for (int i = lane * 4; i < dim; i += 128) {
      __align__(16) T v[4];
      if (sizeof(T) == 2) *reinterpret_cast<uint2*>(v) = *reinterpret_cast<const uint2*>(src + row * dim + i);
      else *reinterpret_cast<uint4*>(v) = *reinterpret_cast<const uint4*>(src + row * dim + i);
#pragma unroll
      for (int k = 0; k < 4; ++k) v[k] = (T)((float)v[k] * f);
      if (sizeof(T) == 2) *reinterpret_cast<uint2*>(out + row * dim + i) = *reinterpret_cast<const uint2*>(v);
      else *reinterpret_cast<uint4*>(out + row * dim + i) = *reinterpret_cast<const uint4*>(v);
    }
    return;
  }
  for (int i = lane; i < dim; i += 32) out[row * dim + i] = (T)((float)src[row * dim + i] * f);
}

// Decayed exclusive scan of per-chunk states in place: walking the chunks of a range in order (or in reverse),
//   out[b] = running;  running = γ_b running + in[b],   γ_b = exp(λ_{e(b)} - λ_{s(b)-1}) = the product of chunk b's gates.
// Forward this is S_in (Lemma "Gated SMat": the carried state is decayed by every chunk it passes); in reverse it is the
// adjoint recursion of the same scan.
__global__ void __launch_bounds__(256) gated_scan_kernel(float* S, const float* __restrict__ lam, int64_t state_elems,
                                                         int64_t NC, int64_t c, int64_t lo0, int64_t hi0, int64_t lo1,
                                                         int64_t hi1, int reverse) {
  const int64_t e4 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e4 * 4 >= state_elems) return;
  const int64_t bh = blockIdx.y;
  const int64_t lo = blockIdx.z ? lo1 : lo0, hi = blockIdx.z ? hi1 : hi0;
  float4* base = reinterpret_cast<float4*>(S + bh * NC * state_elems) + e4;
  const float* l = lam + bh * NC * c;
  const int64_t stride4 = state_elems / 4;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int64_t k = 0; k < hi - lo; ++k) {
    const int64_t b = reverse ? hi - 1 - k : lo + k;
    const float4 v = base[b * stride4];
    base[b * stride4] = acc;
    const float g = __expf(l[b * c + c - 1] - (b > 0 ? l[b * c - 1] : 0.f));
    acc.x = g * acc.x + v.x; acc.y = g * acc.y + v.y; acc.z = g * acc.z + v.z; acc.w = g * acc.w + v.w;
  }
}

// dλ_t = q_t·dQ_t - k_t·dK_t (every edge's contribution enters once as a query and once as a key); one warp per token.
template <typename T>
__global__ void gate_dlam_kernel(const T* __restrict__ Q, const T* __restrict__ dQ, const T* __restrict__ K,
                                 const T* __restrict__ dK, float* __restrict__ dlam, int dim, int64_t rows) {
  const int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / 32;
  if (row >= rows) return;
  const int lane = threadIdx.x & 31;
  float s = 0.f;
  for (int i = lane; i < dim; i += 32)
    s += (float)Q[row * dim + i] * (float)dQ[row * dim + i] - (float)K[row * dim + i] * (float)dK[row * dim + i];
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) s += __shfl_xor_sync(0xffffffffu, s, d);
  if (lane == 0) dlam[row] = s;
}

}  // namespace

cudaError_t smat_launch_head_scan(const float* in, float* out, int64_t len, int bh, int reverse, cudaStream_t st) {
  head_scan_kernel<<<(unsigned)bh, 1024, 0, st>>>(in, out, len, reverse);
  return cudaGetLastError();
}

cudaError_t smat_launch_gate_scale(const void* A, const void* B, void* out, const float* lam, int mode, int bf16,
                                   int64_t n, int64_t c, int64_t T, int dim, int bh, cudaStream_t st) {
  const int64_t rows = (int64_t)bh * T;
  const unsigned blocks = (unsigned)((rows * 32 + 255) / 256);
  if (bf16)
    gate_scale_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(A),
                                                             static_cast<const __nv_bfloat16*>(B),
                                                             static_cast<__nv_bfloat16*>(out), lam, mode, n, c, T, dim, rows);
  else
    gate_scale_kernel<float><<<blocks, 256, 0, st>>>(static_cast<const float*>(A), static_cast<const float*>(B),
                                                     static_cast<float*>(out), lam, mode, n, c, T, dim, rows);
  return cudaGetLastError();
}

cudaError_t smat_launch_gated_scan(float* S, const float* lam, int64_t state_elems, int64_t NC, int64_t c, int bh,
                                   int64_t lo0, int64_t hi0, int64_t lo1, int64_t hi1, int reverse, cudaStream_t st) {
  const int ranges = (hi1 > lo1) ? 2 : 1;
  dim3 grid((unsigned)((state_elems / 4 + 255) / 256), (unsigned)bh, (unsigned)ranges);
  gated_scan_kernel<<<grid, 256, 0, st>>>(S, lam, state_elems, NC, c, lo0, hi0, lo1, hi1, reverse);
  return cudaGetLastError();
}

cudaError_t smat_launch_gate_dlam(const void* Q, const void* dQ, const void* K, const void* dK, float* dlam, int bf16,
                                  int dim, int64_t T, int bh, cudaStream_t st) {
  const int64_t rows = (int64_t)bh * T;
  const unsigned blocks = (unsigned)((rows * 32 + 255) / 256);
  if (bf16)
    gate_dlam_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(Q),
                                                            static_cast<const __nv_bfloat16*>(dQ),
                                                            static_cast<const __nv_bfloat16*>(K),
                                                            static_cast<const __nv_bfloat16*>(dK), dlam, dim, rows);
  else
    gate_dlam_kernel<float><<<blocks, 256, 0, st>>>(static_cast<const float*>(Q), static_cast<const float*>(dQ),
                                                    static_cast<const float*>(K), static_cast<const float*>(dK), dlam, dim,
                                                    rows);
  return cudaGetLastError();
}

// ---- normalised output (Sec. 2: augmented value v̄ = [v; 1], one final division) ------------------------------------
namespace {

// Four consecutive elements of a row, as one 8-byte (bf16) or 16-byte (fp32) access.
template <typename T>
struct Quad {
  __align__(16) T v[4];
  __device__ __forceinline__ void load(const T* src) {
    if (sizeof(T) == 2) *reinterpret_cast<uint2*>(v) = *reinterpret_cast<const uint2*>(src);
    else *reinterpret_cast<uint4*>(v) = *reinterpret_cast<const uint4*>(src);
  }
  __device__ __forceinline__ void store(T* dst) const {
    if (sizeof(T) == 2) *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(v);
    else *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(v);
  }
};

// The three row kernels below take one warp per row; rows whose length is a multiple of 128 move four elements per lane
// and access (the elementwise form was bound by its 2-byte accesses and per-element index arithmetic).

// V̄ = V with its last column set to one.
template <typename T>
__global__ void augment_value_kernel(const T* __restrict__ V, T* __restrict__ Vbar, int p, int64_t rows) {
  const int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / 32;
  if (row >= rows) return;
  const int lane = threadIdx.x & 31;
  if (p % 128 == 0) {
    for (int i = lane * 4; i < p; i += 128) {
      Quad<T> q;
      q.load(V + row * p + i);
      if (i + 4 == p) q.v[3] = (T)1.0f;
      q.store(Vbar + row * p + i);
    }
    return;
  }
  for (int i = lane; i < p; i += 32) Vbar[row * p + i] = i == p - 1 ? (T)1.0f : V[row * p + i];
}

// O = ȳ_{1:p-1} / ȳ_p, and the normaliser ȳ_p itself in the last column.  One warp per row.
template <typename T>
__global__ void normalize_rows_kernel(const T* __restrict__ Y, T* __restrict__ O, int p, int64_t rows) {
  const int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / 32;
  if (row >= rows) return;
  const int lane = threadIdx.x & 31;
  const float den = (float)Y[row * p + p - 1];
  const float inv = 1.0f / den;
  if (p % 128 == 0) {
    for (int i = lane * 4; i < p; i += 128) {
      Quad<T> q;
      q.load(Y + row * p + i);
#pragma unroll
      for (int k = 0; k < 4; ++k) q.v[k] = i + k == p - 1 ? (T)den : (T)((float)q.v[k] * inv);
      q.store(O + row * p + i);
    }
    return;
  }
  for (int i = lane; i < p; i += 32) O[row * p + i] = i == p - 1 ? (T)den : (T)((float)Y[row * p + i] * inv);
}

// Upstream of the linear pass from the upstream of the normalised output (the backward of the final division):
//   dȳ_c = dO_c / z (c < p-1),   dȳ_p = dO_p - Σ_{c<p-1} dO_c O_c / z,   z = the normaliser kept in O's last column.
template <typename T>
__global__ void normalize_adjoint_kernel(const T* __restrict__ O, const T* __restrict__ dO, T* __restrict__ dY, int p,
                                         int64_t rows) {
  const int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / 32;
  if (row >= rows) return;
  const int lane = threadIdx.x & 31;
  const float inv = 1.0f / (float)O[row * p + p - 1];
  float dot = 0.f;
  if (p % 128 == 0) {
    float last = 0.f;   // dO of the normaliser column (held by the lane that owns the row's last quad)
    for (int i = lane * 4; i < p; i += 128) {
      Quad<T> g, o;
      g.load(dO + row * p + i);
      o.load(O + row * p + i);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if (i + k == p - 1) { last = (float)g.v[k]; continue; }
        dot += (float)g.v[k] * (float)o.v[k];
        g.v[k] = (T)((float)g.v[k] * inv);
      }
      if (i + 4 != p) g.store(dY + row * p + i);
      else {   // the last quad waits for the row's dot product
#pragma unroll
        for (int k = 0; k < 3; ++k) dY[row * p + i + k] = g.v[k];
      }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, d);
    if (lane == ((p - 4) % 128) / 4) dY[row * p + p - 1] = (T)(last - dot * inv);
    return;
  }
  for (int i = lane; i < p - 1; i += 32) {
    const float g = (float)dO[row * p + i];
    dot += g * (float)O[row * p + i];
    dY[row * p + i] = (T)(g * inv);
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, d);
  if (lane == 0) dY[row * p + p - 1] = (T)((float)dO[row * p + p - 1] - dot * inv);
}

// The ones column of V̄ is a constant: its gradient is dropped.
template <typename T>
__global__ void clear_last_column_kernel(T* __restrict__ dV, int p, int64_t rows) {
  const int64_t row = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (row < rows) dV[row * p + p - 1] = (T)0.0f;
}

template <typename T>
cudaError_t normalize_step(int step, const void* a, const void* b, void* out, int p, int64_t rows, cudaStream_t st) {
  const unsigned warp_blocks = (unsigned)((rows * 32 + 255) / 256);
  if (step == 0)
    augment_value_kernel<T><<<warp_blocks, 256, 0, st>>>(static_cast<const T*>(a), static_cast<T*>(out), p, rows);
  else if (step == 1)
    normalize_rows_kernel<T><<<warp_blocks, 256, 0, st>>>(static_cast<const T*>(a), static_cast<T*>(out), p, rows);
  else if (step == 2)
    normalize_adjoint_kernel<T><<<warp_blocks, 256, 0, st>>>(static_cast<const T*>(a), static_cast<const T*>(b),
                                                             static_cast<T*>(out), p, rows);
  else
    clear_last_column_kernel<T><<<(unsigned)((rows + 255) / 256), 256, 0, st>>>(static_cast<T*>(out), p, rows);
  return cudaGetLastError();
}

}  // namespace

// step 0: out = V̄ from a = V;  1: out = O from a = ȳ;  2: out = dȳ from a = O, b = dO;  3: out (dV) last column := 0
cudaError_t smat_launch_normalize_step(int step, const void* a, const void* b, void* out, int bf16, int p, int64_t rows,
                                       cudaStream_t st) {
  return bf16 ? normalize_step<__nv_bfloat16>(step, a, b, out, p, rows, st) : normalize_step<float>(step, a, b, out, p, rows, st);
}
