// Greedy accept (paper Sec. 2.1.1 and its footnote): row argmax of the fp32
// logits, then per sequence the longest draft prefix equal to the argmax.
//
// The logits are read exactly once (HBM-bound).  Pass 1 cuts every row into
// chunks so that small batches still fill the machine: one CTA per (chunk, row)
// streams its chunk with 16-byte loads (8 in flight per thread) and leaves one
// (value, index) candidate in the workspace.  Pass 2 uses one warp per sequence:
// each lane folds the chunk candidates of one row, then lane 0 walks the block's
// rows to count the matching prefix.  Ordering rule everywhere: a NaN beats any
// number, larger value beats smaller, equal values (and two NaNs) go to the lower
// index -- the lowest-index-of-the-maximum convention with NaN treated as maximal.
#include <limits.h>

#include <mutex>

#include "common.cuh"

namespace {

constexpr int kChunk = 8192;      // floats per (row, chunk) CTA
constexpr int kThreads = 256;

struct Cand {
  float v;
  int i;
};

__device__ __forceinline__ bool better(float v, int i, float bv, int bi) {
  const bool vn = (v != v), bn = (bv != bv);
  if (vn || bn) return vn && (!bn || i < bi);
  return (v > bv) || (v == bv && i < bi);
}

__device__ __forceinline__ void fold(Cand& best, float v, int i) {
  if (better(v, i, best.v, best.i)) {
    best.v = v;
    best.i = i;
  }
}

__device__ __forceinline__ Cand warp_best(Cand c) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, c.v, o);
    const int oi = __shfl_xor_sync(0xffffffffu, c.i, o);
    fold(c, ov, oi);
  }
  return c;
}

template <bool kVec>
__global__ void __launch_bounds__(kThreads)
argmax_chunks_kernel(const float* __restrict__ logits, int64_t ld_v, int V, int n_chunks,
                     Cand* __restrict__ part) {
  const int row = blockIdx.x / n_chunks, chunk = blockIdx.x - row * n_chunks;
  const float* __restrict__ x = logits + static_cast<int64_t>(row) * ld_v;
  const int lo = chunk * kChunk;
  const int hi = min(V, lo + kChunk);
  Cand best{-INFINITY, INT_MAX};
  if (kVec) {
    // rows are 16-byte aligned: whole float4 groups, then a scalar tail
    const int n4 = (hi - lo) >> 2;
    const float4* __restrict__ x4 = reinterpret_cast<const float4*>(x + lo);
    constexpr int kUnroll = kChunk / 4 / kThreads;   // 8
    float4 r[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int j = threadIdx.x + u * kThreads;
      if (j < n4) r[u] = __ldcs(x4 + j);
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int j = threadIdx.x + u * kThreads;
      if (j < n4) {
        const int i0 = lo + 4 * j;
        fold(best, r[u].x, i0);
        fold(best, r[u].y, i0 + 1);
        fold(best, r[u].z, i0 + 2);
        fold(best, r[u].w, i0 + 3);
      }
    }
    for (int i = lo + 4 * n4 + threadIdx.x; i < hi; i += kThreads) fold(best, x[i], i);
  } else {
    for (int i = lo + threadIdx.x; i < hi; i += kThreads) fold(best, x[i], i);
  }
  __shared__ Cand s_c[kThreads / 32];
  best = warp_best(best);
  if ((threadIdx.x & 31) == 0) s_c[threadIdx.x >> 5] = best;
  __syncthreads();
  if (threadIdx.x < 32) {
    Cand c = (threadIdx.x < kThreads / 32) ? s_c[threadIdx.x] : Cand{-INFINITY, INT_MAX};
    c = warp_best(c);
    if (threadIdx.x == 0) part[static_cast<int64_t>(row) * n_chunks + chunk] = c;
  }
}

__global__ void __launch_bounds__(128)
accept_rows_kernel(const Cand* __restrict__ part, int n_chunks, const int32_t* __restrict__ row_off,
                   int B, const int32_t* __restrict__ draft, int32_t* __restrict__ argmax_out,
                   int32_t* __restrict__ n_match, int32_t* __restrict__ n_keep) {
  const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (b >= B) return;
  const int r0 = row_off[b], r1 = row_off[b + 1];
  for (int r = r0 + lane; r < r1; r += 32) {
    Cand best{-INFINITY, INT_MAX};
    for (int c = 0; c < n_chunks; ++c) {
      const Cand p = part[static_cast<int64_t>(r) * n_chunks + c];
      fold(best, p.v, p.i);
    }
    argmax_out[r] = best.i;
  }
  __syncwarp();
  if (lane == 0) {
    int m = 0;
    for (int r = r0; r < r1; ++r) {
      const int d = draft[r];
      if (d < 0 || argmax_out[r] != d) break;
      ++m;
    }
    n_match[b] = m;
    if (n_keep) n_keep[b] = (r1 > r0) ? m + 1 : 0;   // c_0 .. c_m become permanent
  }
}

inline int chunks_of(int V) { return (V + kChunk - 1) / kChunk; }

}  // namespace

extern "C" size_t memosight_accept_workspace_bytes(int32_t total_rows, int32_t vocab) {
  if (total_rows < 0 || vocab < 1) return 0;
  const size_t n = static_cast<size_t>(total_rows) * chunks_of(vocab) * sizeof(Cand);
  return n < 256 ? 256 : n;
}

extern "C" int32_t memosight_accept(const float* logits, int64_t ld_v, int32_t vocab,
                                    const int32_t* row_off, int32_t batch, int32_t total_rows,
                                    const int32_t* draft, int32_t* argmax_out, int32_t* n_match,
                                    int32_t* n_keep, void* workspace, size_t workspace_bytes,
                                    memosight_stream_t stream) {
  if (batch < 0 || total_rows < 0 || vocab < 1 || ld_v < vocab) return MS_ERR_INVALID_ARG;
  if (batch == 0) return total_rows == 0 ? MS_OK : MS_ERR_INVALID_ARG;
  if (!row_off || !n_match) return MS_ERR_INVALID_ARG;
  if (total_rows > 0 && (!logits || !draft || !argmax_out || !workspace)) return MS_ERR_INVALID_ARG;
  if (static_cast<int64_t>(total_rows) * ((vocab + kChunk - 1) / kChunk) > 0x7fffffffLL)
    return MS_ERR_UNSUPPORTED_SHAPE;
  if (workspace_bytes < memosight_accept_workspace_bytes(total_rows, vocab))
    return MS_ERR_WORKSPACE_TOO_SMALL;
  if (reinterpret_cast<uintptr_t>(workspace) & 7u) return MS_ERR_ALIGNMENT;
  cudaStream_t st = ms::as_stream(stream);
  const int n_chunks = chunks_of(vocab);
  Cand* part = static_cast<Cand*>(workspace);
  if (total_rows > 0) {
    const dim3 grid(static_cast<unsigned>(n_chunks) * static_cast<unsigned>(total_rows));
    const bool vec = ms::aligned16(logits) && (ld_v % 4 == 0);
    if (vec)
      argmax_chunks_kernel<true><<<grid, kThreads, 0, st>>>(logits, ld_v, vocab, n_chunks, part);
    else
      argmax_chunks_kernel<false><<<grid, kThreads, 0, st>>>(logits, ld_v, vocab, n_chunks, part);
    MS_LAUNCH_CHECK();
  }
  accept_rows_kernel<<<(batch + 3) / 4, 128, 0, st>>>(part, n_chunks, row_off, batch, draft,
                                                      argmax_out, n_match, n_keep);
  MS_LAUNCH_CHECK();
  return MS_OK;
}

// ---------------------------------------------------------------------------------------------
// Accept without any allocation by anyone.
//
// Some callers cannot obtain device memory at the moment they need an accept: code that runs
// inside a memory-frozen serving loop (every byte was handed out at start-up and the allocator is
// locked), plug-ins that are given tensors but no allocator handle, or hosts where cudaMalloc
// would synchronise the device in the middle of a latency-critical step.  For them the per-chunk
// candidates of pass 1 live in a fixed array inside the library image instead of a caller
// workspace.  Every GPU that loads the library carries the array (512 KB) until the process exits.
namespace {

constexpr int kStaticMaxPartials = MS_ACCEPT_STATIC_MAX_PARTIALS;
static_assert(kStaticMaxPartials == 65536, "keep the header's limit and the array in step");

static __device__ __align__(256) unsigned char g_accept_scratch[kStaticMaxPartials * sizeof(Cand)];

// In host code `g_accept_scratch` is only a handle for the runtime, not an address a kernel may
// dereference: the device address is looked up once per device, with that device current.
int32_t static_scratch_address(Cand** out) {
  static std::mutex mu;
  static Cand* addr[64] = {nullptr};
  int dev = 0;
  MS_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return MS_ERR_UNSUPPORTED_SHAPE;
  std::lock_guard<std::mutex> lock(mu);
  if (!addr[dev]) {
    void* p = nullptr;
    MS_CUDA_TRY(cudaGetSymbolAddress(&p, g_accept_scratch));
    if (!p) return ms::cuda_status(cudaErrorInvalidSymbol);
    addr[dev] = static_cast<Cand*>(p);
  }
  *out = addr[dev];
  return MS_OK;
}

}  // namespace

extern "C" int32_t memosight_accept_static(const float* logits, int64_t ld_v, int32_t vocab,
                                           const int32_t* row_off, int32_t batch,
                                           int32_t total_rows, const int32_t* draft,
                                           int32_t* argmax_out, int32_t* n_match, int32_t* n_keep,
                                           memosight_stream_t stream) {
  if (batch < 0 || total_rows < 0 || vocab < 1 || ld_v < vocab) return MS_ERR_INVALID_ARG;
  if (batch == 0) return total_rows == 0 ? MS_OK : MS_ERR_INVALID_ARG;
  if (!row_off || !n_match) return MS_ERR_INVALID_ARG;
  if (total_rows > 0 && (!logits || !draft || !argmax_out)) return MS_ERR_INVALID_ARG;
  const int n_chunks = chunks_of(vocab);
  // the fixed array holds one candidate per (row, chunk): refuse anything larger, loudly
  if (static_cast<int64_t>(total_rows) * n_chunks > kStaticMaxPartials) return MS_ERR_UNSUPPORTED_SHAPE;
  Cand* part = nullptr;
  const int32_t rc = static_scratch_address(&part);
  if (rc != MS_OK) return rc;
  cudaStream_t st = ms::as_stream(stream);
  // Nothing in the array has to start at zero: pass 1 writes every (row, chunk) entry that pass 2
  // reads, so whatever an earlier call left behind is overwritten before it is looked at.
  if (total_rows > 0) {
    const dim3 grid(static_cast<unsigned>(n_chunks) * static_cast<unsigned>(total_rows));
    const bool vec = ms::aligned16(logits) && (ld_v % 4 == 0);
    if (vec)
      argmax_chunks_kernel<true><<<grid, kThreads, 0, st>>>(logits, ld_v, vocab, n_chunks, part);
    else
      argmax_chunks_kernel<false><<<grid, kThreads, 0, st>>>(logits, ld_v, vocab, n_chunks, part);
    MS_LAUNCH_CHECK();
  }
  accept_rows_kernel<<<(batch + 3) / 4, 128, 0, st>>>(part, n_chunks, row_off, batch, draft,
                                                      argmax_out, n_match, n_keep);
  MS_LAUNCH_CHECK();
  return MS_OK;
}
