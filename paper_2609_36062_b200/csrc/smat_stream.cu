// HBM-streaming kernels of the long-range branch, written as persistent CTAs around bulk asynchronous
// copies (TMA, one-dimensional, no multicast):
//   pool_stream_kernel       : state[g] = Σ_{tokens of g} a_tᵀ b_t ; each finished 64 KB state leaves through a
//                              bulk store while the next group's tokens are already in flight        (Algorithm 1, step 2)
//   state_read_stream_kernel : out[t] = x_t · state[g(t)] for the few tokens of every group; states arrive through
//                              a two-deep ring of bulk loads                                          (Algorithm 1, step 4)
// Both are bound by the one pass over the table they write or read.
#include <cuda_bf16.h>

#include "smat_internal.h"
#include "smat_tc.cuh"

namespace {

using tc::smem_u32;

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }

__device__ __forceinline__ float4 fma4(float s, const float4 b, float4 a) {
  a.x = fmaf(s, b.x, a.x); a.y = fmaf(s, b.y, a.y); a.z = fmaf(s, b.z, a.z); a.w = fmaf(s, b.w, a.w);
  return a;
}
__device__ __forceinline__ float4 load4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16* p) {
  const uint2 raw = *reinterpret_cast<const uint2*>(p);
  const __nv_bfloat162 lo = *reinterpret_cast<const __nv_bfloat162*>(&raw.x);
  const __nv_bfloat162 hi = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
  return make_float4(__low2float(lo), __high2float(lo), __low2float(hi), __high2float(hi));
}

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(smem)), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void bulk_store(void* gmem, const void* smem, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gmem), "r"(smem_u32(smem)), "r"(bytes)
               : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
template <int N>
__device__ __forceinline__ void bulk_store_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_load(void* smem, const void* gmem, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(smem)),
               "l"(gmem), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}


// ---- pooling ----------------------------------------------------------------------------------------------------
template <int R, int PD, typename T>
__global__ void __launch_bounds__(256) pool_stream_kernel(const T* __restrict__ A, const T* __restrict__ Bm,
                                                          float* __restrict__ state, SmatGroupSpec grp, int64_t Tlen,
                                                          int64_t groups, int64_t items) {
  constexpr int TK = sizeof(T) == 2 ? 32 : 16;  // tokens staged per tile
  constexpr int NJ4 = PD / 4;
  constexpr int NG = 256 / NJ4;
  constexpr int NS = R / NG;
  constexpr int RC = R * (int)sizeof(T) / 16, PC = PD * (int)sizeof(T) / 16;  // 16-byte chunks per row
  extern __shared__ __align__(128) uint8_t smem_raw[];
  float* outb = reinterpret_cast<float*>(smem_raw);                  // [R*PD]
  T* a_raw = reinterpret_cast<T*>(smem_raw + R * PD * 4);            // [2][TK][R]
  T* b_raw = a_raw + 2 * TK * R;                                     // [2][TK][PD]
  const int tid = threadIdx.x;
  const int j4 = tid % NJ4, ig = tid / NJ4;

  auto prefetch = [&](int64_t item, int buf) {  // first tile of tokens of an item, raw, through cp.async
    if (item < items) {
      const int64_t bh = item / groups, g = item - bh * groups;
      const SmatTokens tk = smat_group_tokens(grp, bh, g);
      const int64_t cnt = tk.cnt;
      const int kn = (int)(cnt < TK ? cnt : TK);
      const T* Ab = A + bh * Tlen * R;
      const T* Bb = Bm + bh * Tlen * PD;
      for (int idx = tid; idx < kn * RC; idx += 256) {
        const int k = idx / RC, c = idx - k * RC;
        cp_async16(reinterpret_cast<uint8_t*>(a_raw + (buf * TK + k) * R) + c * 16,
                   reinterpret_cast<const uint8_t*>(Ab + tk.at(k) * R) + c * 16);
      }
      for (int idx = tid; idx < kn * PC; idx += 256) {
        const int k = idx / PC, c = idx - k * PC;
        cp_async16(reinterpret_cast<uint8_t*>(b_raw + (buf * TK + k) * PD) + c * 16,
                   reinterpret_cast<const uint8_t*>(Bb + tk.at(k) * PD) + c * 16);
      }
    }
    cp_async_commit();
  };

  prefetch(blockIdx.x, 0);
  int n = 0;
  for (int64_t item = blockIdx.x; item < items; item += gridDim.x, ++n) {
    const int buf = n & 1;
    prefetch(item + gridDim.x, buf ^ 1);
    cp_async_wait<1>();
    __syncthreads();
    const int64_t bh = item / groups, g = item - bh * groups;
    const SmatTokens tk = smat_group_tokens(grp, bh, g);
    const int64_t cnt = tk.cnt;
    float4 acc[NS];
#pragma unroll
    for (int s = 0; s < NS; ++s) acc[s] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int64_t k0 = 0; k0 < cnt; k0 += TK) {
      const int kn = (int)((cnt - k0) < TK ? (cnt - k0) : TK);
      if (k0 > 0) {  // groups with more than one tile of tokens: fetch the further tiles in place
        __syncthreads();
        const T* Ab = A + bh * Tlen * R;
        const T* Bb = Bm + bh * Tlen * PD;
        for (int idx = tid; idx < kn * RC; idx += 256) {
          const int k = idx / RC, c = idx - k * RC;
          cp_async16(reinterpret_cast<uint8_t*>(a_raw + (buf * TK + k) * R) + c * 16,
                     reinterpret_cast<const uint8_t*>(Ab + tk.at(k0 + k) * R) + c * 16);
        }
        for (int idx = tid; idx < kn * PC; idx += 256) {
          const int k = idx / PC, c = idx - k * PC;
          cp_async16(reinterpret_cast<uint8_t*>(b_raw + (buf * TK + k) * PD) + c * 16,
                     reinterpret_cast<const uint8_t*>(Bb + tk.at(k0 + k) * PD) + c * 16);
        }
        cp_async_commit();
        cp_async_wait<0>();
        __syncthreads();
      }
      const T* as = a_raw + buf * TK * R;
      const T* bs = b_raw + buf * TK * PD;
      for (int k = 0; k < kn; ++k) {
        const float4 b4 = load4(bs + k * PD + j4 * 4);
#pragma unroll
        for (int s = 0; s < NS; ++s) acc[s] = fma4(to_float(as[k * R + ig + s * NG]), b4, acc[s]);
      }
    }
    // the previous item's bulk store reads the same buffer: it must have finished reading (the other CTA
    // resident on this SM keeps the memory pipe busy meanwhile)
    if (tid == 0) bulk_store_wait_read<0>();
    __syncthreads();
    float* ob = outb;
#pragma unroll
    for (int s = 0; s < NS; ++s) *reinterpret_cast<float4*>(ob + (ig + s * NG) * PD + j4 * 4) = acc[s];
    tc::fence_proxy_async();
    __syncthreads();
    if (tid == 0) bulk_store(state + item * (int64_t)(R * PD), ob, R * PD * 4);
  }
  if (tid == 0) bulk_store_wait_all();
  cp_async_wait<0>();
}

// ---- routed read ----------------------------------------------------------------------------------------------------
// Two CTAs share an SM; each owns one 64 KB state buffer, so one CTA's contraction overlaps the other's bulk load.
template <int R, int PD, int TRANS, typename T>
__global__ void __launch_bounds__(256, 2) state_read_stream_kernel(const T* __restrict__ X,
                                                                   const float* __restrict__ state,
                                                                   const float* acc_in, float* acc_out,
                                                                   SmatGroupSpec grp, int64_t Tlen, int64_t groups,
                                                                   int64_t items, int* status) {
  constexpr int KT = 8;
  constexpr int NJ4 = PD / 4;
  constexpr int NG = 256 / NJ4;
  constexpr int RPG = R / NG;
  constexpr int XD = TRANS ? PD : R;
  constexpr int OD = TRANS ? R : PD;
  constexpr int RED = TRANS ? KT * R : NG * KT * PD;
  constexpr int XC = XD * (int)sizeof(T) / 16;  // 16-byte chunks per x row
  extern __shared__ __align__(128) uint8_t smem_raw[];
  float* Sb = reinterpret_cast<float*>(smem_raw);        // [R*PD]
  float* red = Sb + R * PD;                              // [RED]
  T* Xraw = reinterpret_cast<T*>(red + RED);             // [2][KT][XD] raw rows of the first KT tokens of an item
  float* Xs = reinterpret_cast<float*>(Xraw + 2 * KT * XD);  // [KT][XD]
  uint64_t* bar = reinterpret_cast<uint64_t*>(Xs + KT * XD);
  volatile int* cta_abort = reinterpret_cast<volatile int*>(bar + 1);
  const tc::WaitCtx wc{cta_abort, status};
  const int tid = threadIdx.x;
  const int j4 = tid % NJ4, ig = tid / NJ4;
  constexpr uint32_t SBYTES = R * PD * 4;

  auto prefetch_x = [&](int64_t item, int buf) {
    if (item < items) {
      const int64_t bh = item / groups, g = item - bh * groups;
      const SmatTokens tk = smat_group_tokens(grp, bh, g);
      const int64_t cnt = tk.cnt;
      const int kn = (int)(cnt < KT ? cnt : KT);
      const T* Xb = X + bh * Tlen * XD;
      for (int idx = tid; idx < kn * XC; idx += 256) {
        const int k = idx / XC, c = idx - k * XC;
        cp_async16(reinterpret_cast<uint8_t*>(Xraw + (buf * KT + k) * XD) + c * 16,
                   reinterpret_cast<const uint8_t*>(Xb + tk.at(k) * XD) + c * 16);
      }
    }
    cp_async_commit();
  };

  if (tid == 0) {
    *cta_abort = 0;
    tc::mbar_init(bar, 1);
    tc::fence_barrier_init();
    if ((int64_t)blockIdx.x < items) {
      tc::mbar_expect_tx(bar, SBYTES);
      bulk_load(Sb, state + (int64_t)blockIdx.x * (R * PD), SBYTES, bar);
    }
  }
  prefetch_x(blockIdx.x, 0);
  __syncthreads();
  int n = 0;
  for (int64_t item = blockIdx.x; item < items; item += gridDim.x, ++n) {
    const int buf = n & 1;
    const int64_t bh = item / groups, g = item - bh * groups;
    const SmatTokens tk = smat_group_tokens(grp, bh, g);
    const int64_t cnt = tk.cnt;
    const T* Xb = X + bh * Tlen * XD;
    const float4* S4 = reinterpret_cast<const float4*>(Sb);
    prefetch_x(item + gridDim.x, buf ^ 1);
    cp_async_wait<1>();
    bool ok = tc::mbar_wait(bar, n & 1, wc);
    __syncthreads();
    for (int64_t k0 = 0; k0 < cnt && ok; k0 += KT) {
      const int kn = (int)((cnt - k0) < KT ? (cnt - k0) : KT);
      for (int idx = tid; idx < KT * XD; idx += 256) {
        const int k = idx / XD, i = idx % XD;
        float v = 0.f;
        if (k < kn) v = k0 == 0 ? to_float(Xraw[(buf * KT + k) * XD + i]) : to_float(Xb[tk.at(k0 + k) * XD + i]);
        Xs[idx] = v;
      }
      __syncthreads();
      if (!TRANS) {
        float4 acc[KT];
#pragma unroll
        for (int k = 0; k < KT; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
        for (int s = 0; s < RPG; ++s) {
          const int i = ig * RPG + s;
          const float4 u = S4[i * NJ4 + j4];
#pragma unroll
          for (int k = 0; k < KT; ++k) acc[k] = fma4(Xs[k * XD + i], u, acc[k]);
        }
#pragma unroll
        for (int k = 0; k < KT; ++k) *reinterpret_cast<float4*>(red + (ig * KT + k) * PD + j4 * 4) = acc[k];
        __syncthreads();
        for (int idx = tid; idx < kn * PD; idx += 256) {
          const int k = idx / PD, j = idx % PD;
          float v = 0.f;
#pragma unroll
          for (int w = 0; w < NG; ++w) v += red[(w * KT + k) * PD + j];
          const int64_t off = (bh * Tlen + tk.at(k0 + k)) * OD + j;
          acc_out[off] = v + (acc_in ? acc_in[off] : 0.f);
        }
      } else {
#pragma unroll 2
        for (int s = 0; s < RPG; ++s) {
          const int i = ig * RPG + s;
          const float4 u = S4[i * NJ4 + j4];
          float part[KT];
#pragma unroll
          for (int k = 0; k < KT; ++k) {
            const float4 x4 = *reinterpret_cast<const float4*>(Xs + k * XD + j4 * 4);
            part[k] = u.x * x4.x + u.y * x4.y + u.z * x4.z + u.w * x4.w;
          }
#pragma unroll
          for (int off = NJ4 / 2; off > 0; off >>= 1)
#pragma unroll
            for (int k = 0; k < KT; ++k) part[k] += __shfl_xor_sync(0xffffffffu, part[k], off);
          if (j4 == 0)
#pragma unroll
            for (int k = 0; k < KT; ++k) red[k * R + i] = part[k];
        }
        __syncthreads();
        for (int idx = tid; idx < kn * R; idx += 256) {
          const int k = idx / R, i = idx % R;
          const int64_t off = (bh * Tlen + tk.at(k0 + k)) * OD + i;
          acc_out[off] = red[k * R + i] + (acc_in ? acc_in[off] : 0.f);
        }
      }
      __syncthreads();
    }
    // every thread is past its reads of the state buffer: fetch the next item's state
    if (tid == 0) {
      const int64_t nxt = item + gridDim.x;
      if (nxt < items && !*cta_abort) {
        tc::mbar_expect_tx(bar, SBYTES);
        bulk_load(Sb, state + nxt * (int64_t)(R * PD), SBYTES, bar);
      }
    }
  }
  cp_async_wait<0>();
}

template <typename K>
cudaError_t set_smem(K kernel, size_t bytes) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

int sm_count() {
  static int sms = 0;
  if (!sms) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (sms <= 0) sms = 148;
  }
  return sms;
}

template <int R, int PD, typename T>
cudaError_t launch_pool(const void* A, const void* Bm, float* state, const SmatGroupSpec& grp, int64_t Tlen,
                        int64_t groups, int bh, cudaStream_t st) {
  constexpr int TK = sizeof(T) == 2 ? 32 : 16;
  const size_t smem = R * PD * 4 + 2 * TK * (R + PD) * sizeof(T);
  cudaError_t err = set_smem(pool_stream_kernel<R, PD, T>, smem);
  if (err != cudaSuccess) return err;
  const int64_t items = groups * bh;
  const int per_sm = smem <= 110 * 1024 ? 2 : 1;
  const int64_t grid = items < (int64_t)sm_count() * per_sm ? items : (int64_t)sm_count() * per_sm;
  pool_stream_kernel<R, PD, T><<<(unsigned)grid, 256, smem, st>>>(static_cast<const T*>(A), static_cast<const T*>(Bm),
                                                                   state, grp, Tlen, groups, items);
  return cudaGetLastError();
}

template <int R, int PD, int TRANS, typename T>
cudaError_t launch_read(const void* X, const float* state, const float* acc_in, float* acc_out,
                        const SmatGroupSpec& grp, int64_t Tlen, int64_t groups, int bh, int* status, cudaStream_t st) {
  constexpr int KT = 8;
  constexpr int NG = 256 / (PD / 4);
  constexpr int XD = TRANS ? PD : R;
  const size_t smem = R * PD * 4 + (TRANS ? KT * R : NG * KT * PD) * 4 + 2 * KT * XD * sizeof(T) + KT * XD * 4 + 64;
  cudaError_t err = set_smem(state_read_stream_kernel<R, PD, TRANS, T>, smem);
  if (err != cudaSuccess) return err;
  const int64_t items = groups * bh;
  const int per_sm = smem <= 110 * 1024 ? 2 : 1;
  const int64_t grid = items < (int64_t)sm_count() * per_sm ? items : (int64_t)sm_count() * per_sm;
  state_read_stream_kernel<R, PD, TRANS, T><<<(unsigned)grid, 256, smem, st>>>(
      static_cast<const T*>(X), state, acc_in, acc_out, grp, Tlen, groups, items, status);
  return cudaGetLastError();
}

}  // namespace

cudaError_t smat_launch_pool(const void* A, const void* Bm, int bf16, float* state, const SmatGroupSpec& grp,
                             int64_t Tlen, int64_t groups, int bh, int r, int p, cudaStream_t st) {
#define SMAT_POOL(RV, PV)                                                                                       \
  if (r == RV && p == PV)                                                                                       \
    return bf16 ? launch_pool<RV, PV, __nv_bfloat16>(A, Bm, state, grp, Tlen, groups, bh, st)                   \
                : launch_pool<RV, PV, float>(A, Bm, state, grp, Tlen, groups, bh, st);
  SMAT_POOL(128, 128) SMAT_POOL(64, 64) SMAT_POOL(64, 128) SMAT_POOL(128, 64)
#undef SMAT_POOL
  return cudaErrorInvalidValue;
}

cudaError_t smat_launch_state_read(const void* X, int bf16, const float* state, int transposed, const float* acc_in,
                                   float* acc_out, const SmatGroupSpec& grp, int64_t Tlen, int64_t groups, int bh,
                                   int r, int p, int* status, cudaStream_t st) {
#define SMAT_READ(RV, PV, TV)                                                                                        \
  if (r == RV && p == PV && transposed == TV)                                                                        \
    return bf16 ? launch_read<RV, PV, TV, __nv_bfloat16>(X, state, acc_in, acc_out, grp, Tlen, groups, bh, status, st) \
                : launch_read<RV, PV, TV, float>(X, state, acc_in, acc_out, grp, Tlen, groups, bh, status, st);
  SMAT_READ(128, 128, 0) SMAT_READ(64, 64, 0) SMAT_READ(64, 128, 0) SMAT_READ(128, 64, 0)
  SMAT_READ(128, 128, 1) SMAT_READ(64, 64, 1) SMAT_READ(64, 128, 1) SMAT_READ(128, 64, 1)
#undef SMAT_READ
  return cudaErrorInvalidValue;
}
