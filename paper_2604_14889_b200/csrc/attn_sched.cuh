// Pieces shared by the two tensor-core paths of the step attention: the flat tile
// schedule (every 128-key tile of every (sequence, KV head) unit, cut into one
// contiguous range per persistent CTA), the layout of the split-KV workspace, the
// mbarrier / TMA wrappers with bounded waits, and the tensor-map builder.
#pragma once

#include "attn_internal.cuh"

namespace ms {

constexpr int kTile = 128;                 // keys per pipeline stage
constexpr uint32_t kTimeoutMagic = 0x4D535431u;
constexpr unsigned long long kWaitLimitNs = 4000000000ull;

// ---------------------------------------------------------------- PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false if the CTA is aborting or the limit ran out (and
// then records the timeout in the workspace status word and raises the abort flag).
static __device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                            uint32_t* status) {
  const unsigned long long t0 = global_ns();
  for (uint32_t spin = 1;; ++spin) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spin & 63u) == 0) {
      if (*abort_flag) return false;
      if (global_ns() - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        atomicExch(status, kTimeoutMagic);
        return false;
      }
    }
  }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          uint32_t* status) {
  if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, abort_flag, status);
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x,
                                            int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z)
      : "memory");
}
// Tiles of sequence b: its cache tiles plus the step-local tile; 0 if the block is empty.
__device__ __forceinline__ void seq_shape(const AttnArgs& a, int b, int& L, int& n_q, int& r0) {
  r0 = a.q_off[b];
  n_q = a.q_off[b + 1] - r0;
  n_q = n_q < 0 ? 0 : (n_q > a.max_nq ? a.max_nq : n_q);
  L = a.kv_len[b];
  L = L < 0 ? 0 : (L > a.max_kv_len ? a.max_kv_len : L);
}
__device__ __forceinline__ int seq_tiles(int L, int n_q) {
  return n_q > 0 ? (L + kTile - 1) / kTile + 1 : 0;
}

// Exclusive prefix sum of seq_tiles over the batch into pre[0..B] (shared memory).
static __device__ void build_tile_prefix(const AttnArgs& a, int* pre, int* scratch) {
  const int nt = blockDim.x, tid = threadIdx.x;
  const int per = (a.B + nt - 1) / nt;
  const int lo = min(a.B, tid * per), hi = min(a.B, lo + per);
  int sum = 0;
  for (int b = lo; b < hi; ++b) {
    int L, n_q, r0;
    seq_shape(a, b, L, n_q, r0);
    sum += seq_tiles(L, n_q);
  }
  scratch[tid] = sum;
  __syncthreads();
  int base = 0;
  for (int t = 0; t < tid; ++t) base += scratch[t];
  for (int b = lo; b < hi; ++b) {
    int L, n_q, r0;
    seq_shape(a, b, L, n_q, r0);
    pre[b] = base;
    base += seq_tiles(L, n_q);
  }
  if (tid == nt - 1) pre[a.B] = base;
  __syncthreads();
}

// Layout of the workspace behind the header.
__device__ __host__ inline size_t ws_prefix_bytes() { return (static_cast<size_t>(kMaxBatch) + 64) * 4; }
__device__ __host__ inline size_t ws_slot_floats(int D, int rows_pad) {
  return static_cast<size_t>(rows_pad) * (D + 2);
}

// ---------------------------------------------------------------- host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 tensor [d2][d1][D] (D innermost), box = 64 columns x box1 x box2, 128-byte swizzle.
inline bool make_map(CUtensorMap* map, const void* base, int D, uint64_t d1, uint64_t d2,
              uint64_t stride1_elems, uint64_t stride2_elems, uint32_t box1, uint32_t box2) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {static_cast<cuuint64_t>(D), d1, d2};
  const cuuint64_t strides[2] = {stride1_elems * 2, stride2_elems * 2};
  const cuuint32_t box[3] = {64, box1, box2};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box,
            estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Log-sum-exp merge of the units that the split kernel cut across CTAs (attn_mma.cu).
int32_t launch_attn_merge(const AttnArgs& a, cudaStream_t st, int rows_pad, int n_ctas);

}  // namespace ms
