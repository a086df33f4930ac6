// Cached decoding of the recent block (Sec. "Memory-efficient decoding", Theorem "Streaming decoding"):
// once the distant block has been pooled and tabulated, token t >= n is answered from B + 1 states,
//     S_t = S_{t-1} + k_t v_tᵀ ,   o_t = q_tᵀ (U_type(t) + S_t) ,
// and with scalar gates (Sec. 3.2; the table then holds the keys rescaled to the block boundary)
//     S_t = a_t S_{t-1} + k_t v_tᵀ ,   g_t = a_t g_{t-1} ,   o_t = q_tᵀ (g_t U_type(t) + S_t) ,
// O(r p) work per token and head.  One step reads S and one type state and writes S back: it is a stream over
// 3 states per head, so it runs on the plain ALUs with vectorised loads, one CTA per head.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "smat_internal.h"

namespace {

template <typename T>
__device__ __forceinline__ float to_f32(T v);
template <>
__device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T>
__device__ __forceinline__ void store_out(T* p, float v);
template <>
__device__ __forceinline__ void store_out<float>(float* p, float v) { *p = v; }
template <>
__device__ __forceinline__ void store_out<__nv_bfloat16>(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// four consecutive entries of a type state
template <typename TU>
__device__ __forceinline__ float4 load_u4(const TU* p);
template <>
__device__ __forceinline__ float4 load_u4<float>(const float* p) { return *reinterpret_cast<const float4*>(p); }
template <>
__device__ __forceinline__ float4 load_u4<__nv_bfloat16>(const __nv_bfloat16* p) {
  const uint2 w = *reinterpret_cast<const uint2*>(p);
  return make_float4(__uint_as_float(w.x << 16), __uint_as_float(w.x & 0xffff0000u), __uint_as_float(w.y << 16),
                     __uint_as_float(w.y & 0xffff0000u));
}

// One CTA per head, blockDim = 256.  Thread (i0 = tid / (p / 4), j4 = tid % (p / 4)) walks the rows i0, i0 + R, ...
// of the r x p state with its four columns, so that a warp touches whole 128-byte lines.
template <typename T, typename TU>
__global__ void __launch_bounds__(256) decode_step_kernel(const T* __restrict__ q, const T* __restrict__ k,
                                                          const T* __restrict__ v, T* __restrict__ o,
                                                          float* __restrict__ S, const TU* __restrict__ U, int64_t type,
                                                          int64_t types, int r, int p, const float* __restrict__ log_a,
                                                          float* __restrict__ log_g) {
  __shared__ float s_q[128], s_k[128], s_o[128];
  const int bh = blockIdx.x, tid = threadIdx.x;
  // gated: a = this token's gate, g = the product of the gates since the block boundary (kept as its logarithm)
  float a = 1.f, g = 1.f, lg = 0.f;
  if (log_a) { lg = log_g[bh] + log_a[bh]; a = __expf(log_a[bh]); g = __expf(lg); }
  const int cols4 = p / 4, rows_per_pass = 256 / cols4;
  const int j = (tid % cols4) * 4, i0 = tid / cols4;
  if (tid < r) { s_q[tid] = to_f32(q[(int64_t)bh * r + tid]); s_k[tid] = to_f32(k[(int64_t)bh * r + tid]); }
  if (tid < p) s_o[tid] = 0.f;
  __syncthreads();
  const T* vrow = v + (int64_t)bh * p + j;
  const float v0 = to_f32(vrow[0]), v1 = to_f32(vrow[1]), v2 = to_f32(vrow[2]), v3 = to_f32(vrow[3]);
  float* Sh = S + (int64_t)bh * r * p;
  const TU* Uh = U + ((int64_t)bh * types + type) * r * p;
  float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
  for (int i = i0; i < r; i += rows_per_pass) {
    float4 s = *reinterpret_cast<const float4*>(Sh + (int64_t)i * p + j);
    const float ki = s_k[i], qi = s_q[i];
    s.x = fmaf(ki, v0, a * s.x); s.y = fmaf(ki, v1, a * s.y); s.z = fmaf(ki, v2, a * s.z); s.w = fmaf(ki, v3, a * s.w);
    *reinterpret_cast<float4*>(Sh + (int64_t)i * p + j) = s;     // S_t = a_t S_{t-1} + k vᵀ
    const float4 u = load_u4<TU>(Uh + (int64_t)i * p + j);
    a0 = fmaf(qi, fmaf(g, u.x, s.x), a0); a1 = fmaf(qi, fmaf(g, u.y, s.y), a1);
    a2 = fmaf(qi, fmaf(g, u.z, s.z), a2); a3 = fmaf(qi, fmaf(g, u.w, s.w), a3);
  }
  atomicAdd(&s_o[j], a0); atomicAdd(&s_o[j + 1], a1); atomicAdd(&s_o[j + 2], a2); atomicAdd(&s_o[j + 3], a3);
  __syncthreads();
  if (tid < p) store_out(o + (int64_t)bh * p + tid, s_o[tid]);
  if (log_a && tid == 0) log_g[bh] = lg;   // every thread read the old value before the first barrier
}

}  // namespace

// q, k: [bh][r]; v, o: [bh][p] in the plan's input type; S: [bh][r][p] fp32; U: [bh][types][r][p] (bf16 or fp32).
// Gated step: log_a [bh] = log-gates of this token, log_g [bh] = running log of the gates since the boundary (updated).
cudaError_t smat_launch_decode_step(const void* q, const void* k, const void* v, void* o, float* S, const void* U,
                                    int u_bf16, int in_bf16, int64_t type, int64_t types, int r, int p, int bh,
                                    cudaStream_t st, const float* log_a, float* log_g) {
  if (r > 128 || p > 128 || p % 4 || 256 % (p / 4)) return cudaErrorInvalidValue;
  if (in_bf16) {
    const __nv_bfloat16 *qq = static_cast<const __nv_bfloat16*>(q), *kk = static_cast<const __nv_bfloat16*>(k),
                        *vv = static_cast<const __nv_bfloat16*>(v);
    __nv_bfloat16* oo = static_cast<__nv_bfloat16*>(o);
    if (u_bf16)
      decode_step_kernel<__nv_bfloat16, __nv_bfloat16><<<bh, 256, 0, st>>>(qq, kk, vv, oo, S, static_cast<const __nv_bfloat16*>(U),
                                                                         type, types, r, p, log_a, log_g);
    else
      decode_step_kernel<__nv_bfloat16, float><<<bh, 256, 0, st>>>(qq, kk, vv, oo, S, static_cast<const float*>(U), type,
                                                                 types, r, p, log_a, log_g);
  } else {
    if (u_bf16) return cudaErrorInvalidValue;
    decode_step_kernel<float, float><<<bh, 256, 0, st>>>(static_cast<const float*>(q), static_cast<const float*>(k),
                                                         static_cast<const float*>(v), static_cast<float*>(o), S,
                                                         static_cast<const float*>(U), type, types, r, p, log_a, log_g);
  }
  return cudaGetLastError();
}
