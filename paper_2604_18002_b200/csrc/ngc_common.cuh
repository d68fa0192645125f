// Shared host/device helpers of the NGC CUDA library (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <mutex>

#ifdef NGC_NVTX
#include <nvtx3/nvtx3.hpp>
#endif

#include "ngc.h"

namespace ngc {

// Last cudaError_t seen by a failing call on this host thread.
extern thread_local int g_last_cuda_error;

inline int cuda_fail(cudaError_t e) {
  g_last_cuda_error = (int)e;
  return NGC_ERR_CUDA;
}

#define NGC_CUDA_TRY(expr)                              \
  do {                                                  \
    cudaError_t _e = (expr);                            \
    if (_e != cudaSuccess) return ::ngc::cuda_fail(_e); \
  } while (0)

// Optional NVTX range around every C-ABI call (build with -DNGC_NVTX): profiler timelines and launch lists then
// name the call each kernel belongs to.  Compiles to nothing otherwise.
#ifdef NGC_NVTX
#define NGC_API_RANGE(name) ::nvtx3::scoped_range ngc_api_range_ { name }
#else
#define NGC_API_RANGE(name) do { } while (0)
#endif

// Bounds-checking build (-DNGC_DEBUG, a second library beside the normal one).  The normal build already
// validates everything that comes from the caller (kept lists, counts, lengths); this build also checks the
// indices the kernels COMPUTE from them (source and destination rows, TMA row coordinates, page-table slots,
// positions in partial and output arrays) right before use.  The first violation is recorded in the status
// word as NGC_DEV_DEBUG_BOUNDS and that access is skipped, so a wrong index shows up as a status code instead
// of as a stray read or write.  It stands in for a memory checker: the tests rerun the small parity cases on
// this build and require status 0.  Expands to `true` in the normal build.
#ifdef NGC_DEBUG
#define NGC_IN_BOUNDS(status_ptr, cond) ((cond) ? true : (::ngc::set_dev_status((status_ptr), NGC_DEV_DEBUG_BOUNDS), false))
#else
#define NGC_IN_BOUNDS(status_ptr, cond) (true)
#endif

// Check the launch that was just enqueued.
inline int launch_status() {
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? NGC_OK : cuda_fail(e);
}

__host__ __device__ inline int lists_G(int lists, int L, int Hkv) {
  return lists == NGC_LISTS_SHARED ? 1 : (lists == NGC_LISTS_PER_LAYER ? L : L * Hkv);
}
__host__ __device__ inline int list_of(int lists, int l, int h, int Hkv) {
  return lists == NGC_LISTS_SHARED ? 0 : (lists == NGC_LISTS_PER_LAYER ? l : l * Hkv + h);
}

inline int elt_bytes(int dtype) { return dtype == NGC_F32 ? 4 : 2; }

inline bool valid_cache(const ngc_cache* c) {
  return c && c->k && c->v && c->seq_off && c->lens && c->L > 0 && c->B > 0 && c->Hq > 0 && c->Hkv > 0 &&
         c->Hq % c->Hkv == 0 && (c->d == 64 || c->d == 128) && c->rows >= 0 && c->max_len >= 0 &&
         (c->dtype == NGC_F32 || c->dtype == NGC_BF16) && c->lens_lists >= 0 && c->lens_lists <= 2;
}

// Index of the length entry of strip (b, l, h): lens[B] when lens_lists == 0, else lens[B][G] of that mode.
__host__ __device__ inline int64_t len_index(int lens_lists, int L, int Hkv, int b, int l, int h) {
  return (int64_t)b * lists_G(lens_lists, L, Hkv) + list_of(lens_lists, l, h, Hkv);
}

inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

// Set-up that CUDA keeps PER DEVICE (a kernel's opt-in to more than 48 KB of dynamic shared
// memory, the address of a __device__ symbol) and that a launcher wants to do once: the first
// call made while a given device is current runs `setup` for that device, later calls on the
// same device return at once.  One instance per launcher (a function-local static).
constexpr int kMaxDevices = 64;
class PerDeviceOnce {
 public:
  // `setup` returns a cudaError_t.  Returns an ngc_status; *device (if given) gets the current device.
  template <typename F> int run(F&& setup, int* device = nullptr) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= kMaxDevices) return NGC_ERR_UNSUPPORTED;
    if (device) *device = dev;
    if (done_[dev].load(std::memory_order_acquire)) return NGC_OK;
    std::lock_guard<std::mutex> lock(mu_);
    if (done_[dev].load(std::memory_order_relaxed)) return NGC_OK;
    e = setup();
    if (e != cudaSuccess) return cuda_fail(e);
    done_[dev].store(true, std::memory_order_release);
    return NGC_OK;
  }

 private:
  std::mutex mu_;
  std::atomic<bool> done_[kMaxDevices] = {};
};

// Paged layout of a call (table == nullptr: contiguous strips addressed through seq_off).
struct PagedView { const int32_t* table; int page, pages_cap, lists; };

#ifdef __CUDACC__
// Launch with programmatic stream serialisation: the kernel may begin while
// the previous kernel of the stream drains, and waits for it on the device
// (ptx::grid_dep_wait) before touching dependent memory.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// First error wins.
__device__ __forceinline__ void set_dev_status(int32_t* st, int code) {
  if (st) atomicCAS(st, 0, code);
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
#endif

}  // namespace ngc
