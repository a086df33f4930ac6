// Allocation-free entry point: the causal (d = 1) forward with its scratch in a static device array.
//
// Some callers have no way to hand the library a workspace: a plug-in running inside a host
// application that owns all device memory and exposes no allocator, or a service whose request path
// is forbidden to call cudaMalloc because an allocation may synchronise the device and stall every
// other stream.  For them this file keeps the scratch the causal path needs (the bf16 incoming chunk
// states S_in and a status word) in a fixed array that is part of the library image.
#include <cuda_runtime.h>

#include <mutex>

#include "../../include/smat.h"
#include "smat_internal.h"

namespace {

constexpr size_t STATIC_STATUS_BYTES = 256;
constexpr size_t STATIC_TILE_BYTES = 128 * 128 * 2;  // one bf16 state
constexpr size_t STATIC_SCRATCH_BYTES = STATIC_STATUS_BYTES + (size_t)SMAT_STATIC_MAX_TILES * STATIC_TILE_BYTES;

// Every device that loads the library holds this array until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
void* g_scratch_ptr[MAX_DEVICES] = {};
std::mutex g_setup_mutex;

// Device address of the array on the current device.  The array's name is only a host-side handle:
// the address a kernel can use comes from cudaGetSymbolAddress, asked once per device while that
// device is current.
cudaError_t scratch_for_current_device(void** out) {
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    err = cudaGetSymbolAddress(&p, g_static_scratch);
    if (err != cudaSuccess) return err;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" smat_status smat_forward_causal_static(const void* Q, const void* K, const void* V, void* O, int batch,
                                                  int heads, int64_t T, void* cuda_stream) {
  if (!Q || !K || !V || !O) return SMAT_ERR_NULL;
  if (batch < 1 || heads < 1 || T < 128 || T % 128 != 0 || (int64_t)batch * heads > 65535) return SMAT_ERR_SHAPE;
  const int64_t tiles = (int64_t)batch * heads * (T / 128);
  if (tiles > SMAT_STATIC_MAX_TILES) return SMAT_ERR_WORKSPACE;  // beyond the fixed scratch: use smat_forward
  const uintptr_t bits = reinterpret_cast<uintptr_t>(Q) | reinterpret_cast<uintptr_t>(K) |
                         reinterpret_cast<uintptr_t>(V) | reinterpret_cast<uintptr_t>(O);
  if (bits & 15) return SMAT_ERR_ALIGN;
  if (!smat_tc_available()) return SMAT_ERR_ARCH;
  void* scratch = nullptr;
  if (scratch_for_current_device(&scratch) != cudaSuccess) return SMAT_ERR_LAUNCH;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  unsigned char* base = static_cast<unsigned char*>(scratch);
  int* status = reinterpret_cast<int*>(base);
  void* sin = base + STATIC_STATUS_BYTES;
  // The array keeps whatever the previous call left.  Only the status word has to start at zero: the scan
  // writes every S_in tile of this problem before the output kernel reads it.
  if (cudaMemsetAsync(status, 0, STATIC_STATUS_BYTES, st) != cudaSuccess) return SMAT_ERR_LAUNCH;
  const int bh = batch * heads;
  if (smat_launch_chunk_scan_tc(K, V, sin, T, bh, 0, /*through=*/1, /*reverse=*/0, status, st) != cudaSuccess) return SMAT_ERR_LAUNCH;
  if (smat_launch_chunk_output_tc(Q, K, V, sin, nullptr, /*n_lr=*/T, O, T, bh, status, st) != cudaSuccess)
    return SMAT_ERR_LAUNCH;
  return SMAT_OK;
}

// Reads back the status word of the static scratch: a bounded wait that ran out inside one of the two kernels above
// is reported here, since there is no caller-owned workspace that smat_check_status could look at.
extern "C" smat_status smat_static_check_status(void* cuda_stream) {
  void* scratch = nullptr;
  if (!smat_tc_available()) { cudaGetLastError(); return SMAT_ERR_ARCH; }
  if (scratch_for_current_device(&scratch) != cudaSuccess) return SMAT_ERR_LAUNCH;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int word = 0;
  if (cudaMemcpyAsync(&word, scratch, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return SMAT_ERR_LAUNCH;
  if (cudaStreamSynchronize(st) != cudaSuccess) return SMAT_ERR_LAUNCH;
  return word == 0 ? SMAT_OK : SMAT_ERR_DEVICE_TIMEOUT;
}
