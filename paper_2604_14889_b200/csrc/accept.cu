// Greedy accept (paper Sec. 2.1.1 and its footnote): row argmax of the fp32
// logits, then per sequence the longest draft prefix equal to the argmax.
//
// The logits are read exactly once (HBM-bound).  Pass 1 cuts every row into
// chunks of 8192 floats so that small batches still fill the machine and leaves one
// (value, index) candidate per (row, chunk) in the workspace.  Its streaming form
// (16-byte-aligned rows, vocabulary a multiple of 4) is one persistent CTA per SM:
// a producer thread keeps six 32 KB bulk copies (cp.async.bulk, global -> shared
// memory, completion on an mbarrier) in flight, six warps take a chunk each from
// the ring and reduce it with shuffles only.  Other layouts fall back to one CTA per
// (chunk, row) with plain loads.  Pass 2 folds the chunk candidates of every row and counts
// the matching prefix of every sequence.  In the streaming form it needs no launch of its own:
// when a CTA has delivered all its candidates, its threads count them on per-row counters that
// started at zero; the thread whose count completes a row folds that row, and the CTA in which
// the last row of all was completed counts the prefixes -- nobody waits for anybody.  Ordering
// rule everywhere: a NaN beats any
// number, larger value beats smaller, equal values (and two NaNs) go to the lower
// index -- the lowest-index-of-the-maximum convention with NaN treated as maximal.
#include <limits.h>

#include <mutex>

#include "attn_sched.cuh"
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

// ---- pass 1, streaming form -------------------------------------------------------------------

constexpr int kStages = 6;                       // 32 KB chunks in flight per SM
constexpr int kStreamWarps = kStages;             // warp w owns stage w: it follows that stage's barrier phase by phase
constexpr int kStreamThreads = (kStreamWarps + 1) * 32;
constexpr int kStageBytes = kChunk * 4;
constexpr int kStreamSmem = kStages * kStageBytes + 2 * kStages * 8 + 32;

// Set (to a magic word) if a wait inside the streaming kernel ever ran into its time limit; the
// candidates of the chunks that were not finished then carry index -1, which matches no draft.
static __device__ unsigned int g_accept_wait_status;

// What pass 2 needs when it runs inside pass 1.  cnt: a zeroed counter per row and, at index T,
// one for the rows that are complete (left at zero again); NULL: a second kernel does pass 2.
struct Tail {
  unsigned int* cnt;
  const int32_t* row_off;
  const int32_t* draft;
  int32_t* argmax_out;
  int32_t* n_match;
  int32_t* n_keep;
  int B, T;
};

__device__ __forceinline__ Cand load_cand(const Cand* p) {
  const int2 raw = __ldcg(reinterpret_cast<const int2*>(p));
  return Cand{__int_as_float(raw.x), raw.y};
}

// Longest prefix of the block's rows whose argmax equals the draft (no early exit, so that the
// loads of a block are independent of one another).
__device__ __forceinline__ int match_prefix(const int32_t* __restrict__ draft, const int32_t* argmax, int r0, int r1) {
  int m = 0;
  bool run = true;
  for (int r = r0; r < r1; ++r) {
    const int d = draft[r];
    const int am = __ldcg(argmax + r);
    run = run && d >= 0 && am == d;
    m += run ? 1 : 0;
  }
  return m;
}

// Pass 2 inside pass 1, run by the kStreamWarps consumer warps of a CTA once all of them have
// delivered their candidates: every thread counts one of the CTA's items on the item's row; the
// thread whose count completes a row folds that row's candidates and counts the row; the CTA in
// which the last row of all was completed counts every sequence's matching prefix.  One round of
// atomics per CTA, no per-item stall, and nobody waits for another CTA.
__device__ __forceinline__ void accept_tail(const Tail& t, const Cand* part, int n_chunks, int n_local, int n_items,
                                            volatile int* s_last) {
  const int tid = threadIdx.x, n_thr = kStreamWarps * 32;
  __threadfence();                                       // this thread's candidates are visible device-wide
  asm volatile("bar.sync 1, %0;" ::"r"(n_thr) : "memory");
  for (int k = tid; k < n_local; k += n_thr) {
    const int item = static_cast<int>(blockIdx.x) + k * static_cast<int>(gridDim.x);
    const int row = item / n_chunks;
    if (atomicAdd(t.cnt + row, 1u) + 1u != static_cast<unsigned int>(n_chunks)) continue;
    // every chunk of this row is in: fold them
    __threadfence();
    Cand best{-INFINITY, INT_MAX};
    bool bad = false;
    const Cand* pr = part + static_cast<int64_t>(row) * n_chunks;
    for (int c0 = 0; c0 < n_chunks; c0 += 8) {          // eight loads in flight, then the folds
      Cand p[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) p[u] = (c0 + u < n_chunks) ? load_cand(pr + c0 + u) : Cand{-INFINITY, INT_MAX};
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        bad |= (p[u].i < 0);                             // an unfinished chunk: the row matches no draft
        fold(best, p[u].v, p[u].i);
      }
    }
    t.argmax_out[row] = bad ? -1 : best.i;
    t.cnt[row] = 0u;
    __threadfence();
    if (atomicAdd(t.cnt + t.T, 1u) + 1u == static_cast<unsigned int>(t.T)) *s_last = 1;
  }
  asm volatile("bar.sync 1, %0;" ::"r"(n_thr) : "memory");
  if (!*s_last) return;
  // every row has its argmax: the prefix of every sequence
  __threadfence();
  for (int b = tid; b < t.B; b += n_thr) {
    const int r0 = t.row_off[b], r1 = t.row_off[b + 1];
    const int m = match_prefix(t.draft, t.argmax_out, r0, r1);
    t.n_match[b] = m;
    if (t.n_keep) t.n_keep[b] = (r1 > r0) ? m + 1 : 0;
  }
  if (tid == 0) t.cnt[t.T] = 0u;
}

__global__ void __launch_bounds__(kStreamThreads, 1)
argmax_stream_kernel(const float* __restrict__ logits, int64_t ld_v, int V, int n_chunks, int n_items,
                     Cand* __restrict__ part, const Tail tail, unsigned int wait_limit_us) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sb = ms::smem_u32(smem);
  const uint32_t bars = sb + kStages * kStageBytes;           // full[kStages], empty[kStages]
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kStages * kStageBytes + 2 * kStages * 8);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int i = 0; i < kStages; ++i) {
      ms::mbar_init(bars + 8 * i, 1);
      ms::mbar_init(bars + 8 * (kStages + i), 1);
    }
    ms::wait_ctx_init(abort_flag, wait_limit_us);
    abort_flag[4] = 0;                                   // "this CTA completed the last row"
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  ms::pdl_wait();
  ms::pdl_trigger();
  // this CTA's items: blockIdx.x, blockIdx.x + gridDim.x, ...  (item = row * n_chunks + chunk)
  const int n_local = (n_items - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) /
                      static_cast<int>(gridDim.x);
  if (warp == kStreamWarps) {
    if (lane == 0) {
      // ---- producer: one bulk copy per item into the ring
      int issued = 0;
      for (int k = 0; k < n_local; ++k) {
        const int s = k % kStages;
        if (!ms::mbar_wait(bars + 8 * (kStages + s), ((k / kStages) & 1) ^ 1, abort_flag, &g_accept_wait_status)) break;
        const int item = static_cast<int>(blockIdx.x) + k * static_cast<int>(gridDim.x);
        const int row = item / n_chunks, chunk = item - row * n_chunks;
        const int lo = chunk * kChunk;
        const uint32_t bytes = static_cast<uint32_t>(min(V, lo + kChunk) - lo) * 4u;
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the warps' reads of this stage come first
        ms::mbar_arrive_expect_tx(bars + 8 * s, bytes);
        asm volatile(
            "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
            ::"r"(sb + s * kStageBytes), "l"(logits + static_cast<int64_t>(row) * ld_v + lo), "r"(bytes),
              "r"(bars + 8 * s)
            : "memory");
        ++issued;
      }
      // copies still in flight must land before the CTA's shared memory goes away
      for (int k = issued > kStages ? issued - kStages : 0; k < issued; ++k)
        (void)ms::mbar_wait(bars + 8 * (k % kStages), (k / kStages) & 1, abort_flag, &g_accept_wait_status);
    }
    return;
  }
  // ---- consumers: warp w takes the items k = w, w + kStages, ... of this CTA (always stage w)
  for (int k = warp; k < n_local; k += kStreamWarps) {
    const int s = k % kStages;
    const int item = static_cast<int>(blockIdx.x) + k * static_cast<int>(gridDim.x);
    const int row = item / n_chunks, chunk = item - row * n_chunks;
    const int lo = chunk * kChunk;
    const int n4 = (min(V, lo + kChunk) - lo) >> 2;
    const bool ok = __all_sync(0xffffffffu, ms::mbar_wait(bars + 8 * s, (k / kStages) & 1, abort_flag,
                                                          &g_accept_wait_status));
    Cand best{-INFINITY, INT_MAX};
    if (ok) {
      const uint32_t base = sb + s * kStageBytes + lane * 16;
      auto load4 = [&](int j) -> float4 {
        float4 x;
        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];"
                     : "=f"(x.x), "=f"(x.y), "=f"(x.z), "=f"(x.w)
                     : "r"(base + static_cast<uint32_t>(j - lane) * 16));
        return x;
      };
      if (lane < n4) {
        // Branch-free main pass: four running maxima (one per float4 component, each visiting its
        // indices in increasing order, so "strictly greater" keeps the lowest index of equal
        // values), started from the lane's first group.  A NaN anywhere shows up in `mix`.
        float4 x = load4(lane);
        float bv0 = x.x, bv1 = x.y, bv2 = x.z, bv3 = x.w;
        int bi0 = lo + 4 * lane, bi1 = bi0 + 1, bi2 = bi0 + 2, bi3 = bi0 + 3;
        float mix = (x.x + x.y) + (x.z + x.w);
        bool odd = (mix != mix);
#pragma unroll 4
        for (int j = lane + 32; j < n4; j += 32) {
          x = load4(j);
          const int i0 = lo + 4 * j;
          const bool g0 = x.x > bv0, g1 = x.y > bv1, g2 = x.z > bv2, g3 = x.w > bv3;
          bv0 = g0 ? x.x : bv0;
          bi0 = g0 ? i0 : bi0;
          bv1 = g1 ? x.y : bv1;
          bi1 = g1 ? i0 + 1 : bi1;
          bv2 = g2 ? x.z : bv2;
          bi2 = g2 ? i0 + 2 : bi2;
          bv3 = g3 ? x.w : bv3;
          bi3 = g3 ? i0 + 3 : bi3;
          mix = (x.x + x.y) + (x.z + x.w);
          odd |= (mix != mix);
        }
        if (!odd) {
          best.v = bv0;
          best.i = bi0;
          fold(best, bv1, bi1);
          fold(best, bv2, bi2);
          fold(best, bv3, bi3);
        } else {
          // a NaN (or +inf next to -inf) among this lane's values: the full ordering rule, element by element
          for (int j = lane; j < n4; j += 32) {
            x = load4(j);
            const int i0 = lo + 4 * j;
            fold(best, x.x, i0);
            fold(best, x.y, i0 + 1);
            fold(best, x.z, i0 + 2);
            fold(best, x.w, i0 + 3);
          }
        }
      }
      __syncwarp();                              // every lane has read the stage
      if (lane == 0) ms::mbar_arrive(bars + 8 * (kStages + s));
      best = warp_best(best);
    } else {
      best.i = -1;
    }
    if (lane == 0) part[item] = best;
  }
  if (tail.cnt) accept_tail(tail, part, n_chunks, n_local, n_items, abort_flag + 4);
}

__global__ void __launch_bounds__(128)
accept_rows_kernel(const Cand* __restrict__ part, int n_chunks, const int32_t* __restrict__ row_off,
                   int B, const int32_t* __restrict__ draft, int32_t* __restrict__ argmax_out,
                   int32_t* __restrict__ n_match, int32_t* __restrict__ n_keep) {
  ms::pdl_wait();
  ms::pdl_trigger();
  const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (b >= B) return;
  const int r0 = row_off[b], r1 = row_off[b + 1];
  for (int r = r0 + lane; r < r1; r += 32) {
    Cand best{-INFINITY, INT_MAX};
    const Cand* __restrict__ pr = part + static_cast<int64_t>(r) * n_chunks;
    for (int c0 = 0; c0 < n_chunks; c0 += 8) {       // eight loads in flight, then the folds
      Cand p[8];
#pragma unroll
      for (int u = 0; u < 8; ++u)
        p[u] = (c0 + u < n_chunks) ? pr[c0 + u] : Cand{-INFINITY, INT_MAX};
#pragma unroll
      for (int u = 0; u < 8; ++u) fold(best, p[u].v, p[u].i);
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
constexpr int kTailMaxBatch = 2048;   // beyond it one warp counting every sequence's prefix would be the long pole

// Both passes.  The streaming form of pass 1 carries pass 2 in its tail when a counter bank is to
// be had and the problem fits it; otherwise, and for the other layouts, pass 2 is a second launch.
int32_t launch_accept(const float* logits, int64_t ld_v, int vocab, const int32_t* row_off, int batch,
                      int total_rows, const int32_t* draft, int32_t* argmax_out, int32_t* n_match,
                      int32_t* n_keep, Cand* part, cudaStream_t st) {
  const int n_chunks = chunks_of(vocab);
  const int n_items = n_chunks * total_rows;
  const bool vec = ms::aligned16(logits) && (ld_v % 4 == 0);
  Tail tail;
  tail.cnt = nullptr;
  tail.row_off = row_off; tail.draft = draft; tail.argmax_out = argmax_out;
  tail.n_match = n_match; tail.n_keep = n_keep; tail.B = batch; tail.T = total_rows;
  if (total_rows > 0) {
    if (vec && vocab % 4 == 0) {
      static bool configured[64] = {false};
      int dev = 0;
      MS_CUDA_TRY(cudaGetDevice(&dev));
      if (dev >= 0 && dev < 64 && !configured[dev]) {
        MS_CUDA_TRY(cudaFuncSetAttribute(argmax_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         kStreamSmem));
        configured[dev] = true;
      }
      const int sms = ms::sm_count();
      if (sms <= 0) return ms::cuda_status(cudaErrorNoDevice);
      if (total_rows < ms::kDoneBankWords && batch <= kTailMaxBatch) tail.cnt = ms::done_bank(part);
      MS_CUDA_TRY(ms::launch_pdl(argmax_stream_kernel, dim3(n_items < sms ? n_items : sms), dim3(kStreamThreads),
                                 kStreamSmem, st, logits, ld_v, vocab, n_chunks, n_items, part, tail,
                                 ms::wait_limit_us()));
      if (tail.cnt) return MS_OK;
    } else if (vec) {
      argmax_chunks_kernel<true><<<static_cast<unsigned>(n_items), kThreads, 0, st>>>(logits, ld_v, vocab, n_chunks, part);
      MS_LAUNCH_CHECK();
    } else {
      argmax_chunks_kernel<false><<<static_cast<unsigned>(n_items), kThreads, 0, st>>>(logits, ld_v, vocab, n_chunks, part);
      MS_LAUNCH_CHECK();
    }
  }
  MS_CUDA_TRY(ms::launch_pdl(accept_rows_kernel, dim3((batch + 3) / 4), dim3(128), 0, st,
                             static_cast<const Cand*>(part), n_chunks, row_off, batch, draft, argmax_out, n_match,
                             n_keep));
  return MS_OK;
}

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
  Cand* part = static_cast<Cand*>(workspace);
  return launch_accept(logits, ld_v, vocab, row_off, batch, total_rows, draft, argmax_out, n_match, n_keep, part, st);
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
  return launch_accept(logits, ld_v, vocab, row_off, batch, total_rows, draft, argmax_out, n_match, n_keep, part, st);
}
