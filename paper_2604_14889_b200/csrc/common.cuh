// Shared host/device helpers of the MemoSight CUDA library (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "memosight.h"

namespace ms {

// Thread-local record of the last CUDA error behind an MS_ERR_CUDA.
void set_last_cuda_error(cudaError_t e);

inline int32_t cuda_status(cudaError_t e) {
  if (e == cudaSuccess) return MS_OK;
  set_last_cuda_error(e);
  return MS_ERR_CUDA;
}

#define MS_CUDA_TRY(expr)                              \
  do {                                                 \
    cudaError_t e__ = (expr);                          \
    if (e__ != cudaSuccess) return ms::cuda_status(e__); \
  } while (0)

// Launch check: launch-configuration errors surface through cudaGetLastError.
#define MS_LAUNCH_CHECK() MS_CUDA_TRY(cudaGetLastError())

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Number of SMs of the current device (cached per device).
int32_t sm_count();

inline cudaStream_t as_stream(memosight_stream_t s) { return reinterpret_cast<cudaStream_t>(s); }

// Limit of one bounded device-side wait, in microseconds (memosight_debug_set_wait_limit_us).
unsigned int wait_limit_us();

// "Last block done" counters (done_banks.cu): the zero-initialised bank of kDoneBankWords
// counters that belongs to `key` on the current device, or nullptr when every bank is taken
// (the caller then uses its two-launch form).  A kernel must leave its counters at zero.
constexpr int kDoneBankWords = 2048;
unsigned int* done_bank(const void* key);
// Puts the bank of `key` back to zero on `st` (after a kernel gave up in mid-flight).
int32_t done_bank_clear(const void* key, cudaStream_t st);

// Programmatic dependent launch.  Every kernel of the library starts with the part of its
// set-up that touches no global memory, then waits for the grid before it in the stream
// (pdl_wait: returns once that grid has completed and its writes are visible) and at once lets
// the grid behind it start its own set-up (pdl_trigger).  Because each kernel waits before its
// first global access and before it can finish, completion is transitive along the stream.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Launches `kernel` so that it may begin while the kernel before it in `st` is still running
// (the kernel itself calls pdl_wait before it reads or writes global memory).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

constexpr int kMaxNq = 16;        // largest step block of the Predict+Verify kernels
constexpr int kMaxNqBig = 32768;  // largest block of the large-block kernel (compression pass, prefill)
constexpr int kMaxGroup = 16;     // largest H_q / H_kv
constexpr int kMaxBatch = 8192;   // sequences per attention launch

// Step-local visibility (see memosight_attn_params): key j of the block vs row i.
__host__ __device__ inline bool step_key_visible(int i, int j, int n_c, int a_i) {
  return (j == i) || (j < n_c && j < a_i);
}

// Training-time visibility among the block's own tokens (see memosight_attn_params::tok_kind).
__host__ __device__ inline bool train_key_visible(int i, int j, int kind_j, int step_i, int step_j) {
  return (j == i) ||
         (j < i && kind_j != MS_KIND_FORESIGHT && (kind_j != MS_KIND_REASON || step_j == step_i));
}

}  // namespace ms
