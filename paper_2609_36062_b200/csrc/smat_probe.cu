// Two small device probes behind the C boundary, neither part of the method:
//   - a wait that is meant to run out, so that the bounded-wait error path (status word ->
//     SMAT_ERR_DEVICE_TIMEOUT) can be exercised without faulting or hanging anything;
//   - a microbenchmark of the fp32 add rate of the plain ALUs, the ceiling Algorithm 2's state
//     additions are charged against in the three-term roofline.
#include <cuda_runtime.h>

#include "../../include/smat.h"
#include "smat_internal.h"
#include "smat_tc.cuh"

namespace {

// One thread waits on an mbarrier that nobody ever arrives on, gives up after `limit` SM clock cycles,
// records that in the status word and the kernel returns normally.
__global__ void timeout_probe_kernel(int* status, long long limit) {
  __shared__ uint64_t bar;
  __shared__ int cta_abort;
  if (threadIdx.x == 0) {
    cta_abort = 0;
    tc::mbar_init(&bar, 1);
    tc::fence_barrier_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const tc::WaitCtx wc{&cta_abort, status, limit};
    tc::mbar_wait(&bar, 0, wc);
  }
  __syncthreads();
}

// Independent add chains in registers: every thread keeps CHAINS accumulators and adds a loop-invariant
// value to each, `iters` times.  PACKED selects the two-lane add (add.f32x2), else the scalar add.
constexpr int ADD_CHAINS = 32;
template <bool PACKED>
__global__ void __launch_bounds__(256) fadd_rate_kernel(float* sink, int iters, float seed) {
  float acc[ADD_CHAINS];
#pragma unroll
  for (int i = 0; i < ADD_CHAINS; ++i) acc[i] = seed * (float)(i + threadIdx.x);
  const float inc = seed + 1.0f;
  for (int it = 0; it < iters; ++it) {
    if (PACKED) {
#pragma unroll
      for (int i = 0; i < ADD_CHAINS; i += 2) {
        unsigned long long a, b;
        asm volatile("mov.b64 %0, {%1, %2};" : "=l"(a) : "f"(acc[i]), "f"(acc[i + 1]));
        asm volatile("mov.b64 %0, {%1, %1};" : "=l"(b) : "f"(inc));
        asm volatile("add.rn.f32x2 %0, %0, %1;" : "+l"(a) : "l"(b));
        asm volatile("mov.b64 {%0, %1}, %2;" : "=f"(acc[i]), "=f"(acc[i + 1]) : "l"(a));
      }
    } else {
#pragma unroll
      for (int i = 0; i < ADD_CHAINS; ++i) asm volatile("add.rn.f32 %0, %0, %1;" : "+f"(acc[i]) : "f"(inc));
    }
  }
  float total = 0.f;
#pragma unroll
  for (int i = 0; i < ADD_CHAINS; ++i) total += acc[i];
  if (total == 123.456f) sink[0] = total;  // keeps the chains alive; practically never true
}

}  // namespace

extern "C" smat_status smat_debug_timeout_probe(void* workspace, int64_t limit_cycles, void* cuda_stream) {
  if (!workspace) return SMAT_ERR_NULL;
  if (reinterpret_cast<uintptr_t>(workspace) & 255) return SMAT_ERR_ALIGN;
  if (limit_cycles < 1 || limit_cycles > 2000000000LL) return SMAT_ERR_SHAPE;
  if (!smat_tc_available()) { cudaGetLastError(); return SMAT_ERR_ARCH; }
  timeout_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(static_cast<int*>(workspace),
                                                                             (long long)limit_cycles);
  return cudaGetLastError() == cudaSuccess ? SMAT_OK : SMAT_ERR_LAUNCH;
}

extern "C" smat_status smat_measure_fadd_rate(void* scratch, int packed, double* adds_per_second, void* cuda_stream) {
  if (!scratch || !adds_per_second) return SMAT_ERR_NULL;
  if (!smat_tc_available()) { cudaGetLastError(); return SMAT_ERR_ARCH; }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int blocks = sms * 8, threads = 256, iters = 4096;
  cudaEvent_t e0, e1;
  if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return SMAT_ERR_LAUNCH;
  float best_ms = 0.f;
  bool ok = true;
  for (int rep = 0; rep < 5 && ok; ++rep) {  // first repetition warms up; the fastest of the rest counts
    cudaEventRecord(e0, st);
    if (packed)
      fadd_rate_kernel<true><<<blocks, threads, 0, st>>>(static_cast<float*>(scratch), iters, 0.0f);
    else
      fadd_rate_kernel<false><<<blocks, threads, 0, st>>>(static_cast<float*>(scratch), iters, 0.0f);
    cudaEventRecord(e1, st);
    ok = cudaEventSynchronize(e1) == cudaSuccess && cudaGetLastError() == cudaSuccess;
    float ms = 0.f;
    if (ok) cudaEventElapsedTime(&ms, e0, e1);
    if (rep > 0 && (best_ms == 0.f || ms < best_ms)) best_ms = ms;
  }
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  if (!ok || best_ms <= 0.f) return SMAT_ERR_LAUNCH;
  *adds_per_second = (double)blocks * threads * ADD_CHAINS * iters / (best_ms * 1e-3);
  return SMAT_OK;
}
