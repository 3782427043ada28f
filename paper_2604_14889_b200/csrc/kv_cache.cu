// KV-cache maintenance of MemoSight inference (paper Sec. 2.1.2; Algorithm 1):
//   - compaction: once a reasoning step has been condensed into memory tokens,
//     its verbose entries are evicted and the entries behind them (memory tokens,
//     <o>, anything later) slide up, in every layer, for K and V;
//   - append: the accepted candidates of a step block join the cache.
// Both are pure bit moves with 16-byte accesses; lengths live on the device.
#include "common.cuh"

namespace {

constexpr int kMoveThreads = 256;
constexpr int kMoveUnroll = 8;   // 16-byte vectors per thread per tile -> 32 KB tiles

// What the sequences' lengths become, and the kept-index list, once every thread block of a
// compaction launch has read the old lengths.  Run by one block (256 threads).
__device__ void kv_compact_finish(int B, int32_t* __restrict__ kv_len, const int32_t* __restrict__ seg_start,
                                  const int32_t* __restrict__ seg_len) {
  for (int b = threadIdx.x; b < B; b += blockDim.x) {
    const int L = kv_len[b], s = seg_start[b], n = seg_len[b];
    if (n > 0 && s >= 0 && static_cast<int64_t>(s) + n <= L) kv_len[b] = L - n;
  }
}

// One CTA per (layer, K|V, sequence, KV head).  Source and destination overlap
// whenever more entries move than were evicted, so a tile is read completely into
// registers, the CTA synchronises, and only then is it written; tiles go in
// increasing address order.  Because the shift is towards lower addresses, the
// bytes a tile writes lie strictly below everything later tiles still have to read.
//
// The lengths change in the same launch (`done` != NULL): every block reads its sequence's old
// length first and then counts itself; the block that counts last knows that all of them have
// read, writes the new lengths of all sequences and puts the counter back to zero.  Nobody
// waits.  The (layer 0, K, head 0) block of a sequence also emits its kept-index list, from the
// old length it read.  Without a counter (`done` == NULL) a second kernel does the lengths.
__global__ void __launch_bounds__(kMoveThreads)
kv_compact_move_kernel(uint16_t* __restrict__ k_cache, uint16_t* __restrict__ v_cache,
                       int64_t layer_stride, int64_t kv_head_stride, int B, int H_kv, int D,
                       const int64_t* __restrict__ kv_off, int32_t* __restrict__ kv_len,
                       const int32_t* __restrict__ seg_start, const int32_t* __restrict__ seg_len,
                       int32_t* __restrict__ src_idx, int idx_stride, unsigned int* done) {
  __shared__ int s_shape[4];
  ms::pdl_wait();
  ms::pdl_trigger();
  int u = blockIdx.x;
  const int h = u % H_kv; u /= H_kv;
  const int b = u % B;    u /= B;
  const int is_v = u & 1; u >>= 1;
  const int layer = u;
  if (threadIdx.x == 0) {
    const int L0 = kv_len[b], s0 = seg_start[b], n0 = seg_len[b];
    s_shape[0] = L0;
    s_shape[1] = s0;
    s_shape[2] = n0;
    int last = 0;
    if (done) {
      __threadfence();   // the reads above are ordered before the count
      last = (atomicAdd(done, 1u) + 1u == gridDim.x) ? 1 : 0;
    }
    s_shape[3] = last;
  }
  __syncthreads();
  const int L = s_shape[0], s = s_shape[1], n = s_shape[2];
  if (s_shape[3]) {
    kv_compact_finish(B, kv_len, seg_start, seg_len);
    if (threadIdx.x == 0) *done = 0u;
  }
  const bool valid = (n > 0 && s >= 0 && static_cast<int64_t>(s) + n <= L);
  if (src_idx && layer == 0 && !is_v && h == 0) {
    const int shift = valid ? n : 0;
    const int new_len = L - shift;
    int32_t* row = src_idx + static_cast<int64_t>(b) * idx_stride;
    const int lim = new_len < idx_stride ? new_len : idx_stride;
    for (int j = threadIdx.x; j < lim; j += blockDim.x) row[j] = (valid && j >= s) ? j + shift : j;
  }
  if (!valid) return;                                                // nothing to do / ignored
  const int tail = L - s - n;
  if (tail == 0) return;
  uint16_t* base = (is_v ? v_cache : k_cache) + layer * layer_stride + h * kv_head_stride +
                   kv_off[b] * static_cast<int64_t>(D);
  uint4* dst = reinterpret_cast<uint4*>(base + static_cast<int64_t>(s) * D);
  const uint4* src = reinterpret_cast<const uint4*>(base + static_cast<int64_t>(s + n) * D);
  const int64_t n_vec = static_cast<int64_t>(tail) * D / 8;
  constexpr int kTile = kMoveThreads * kMoveUnroll;
  for (int64_t t0 = 0; t0 < n_vec; t0 += kTile) {
    uint4 r[kMoveUnroll];
#pragma unroll
    for (int j = 0; j < kMoveUnroll; ++j) {
      const int64_t i = t0 + threadIdx.x + j * kMoveThreads;
      if (i < n_vec) r[j] = src[i];
    }
    __syncthreads();
#pragma unroll
    for (int j = 0; j < kMoveUnroll; ++j) {
      const int64_t i = t0 + threadIdx.x + j * kMoveThreads;
      if (i < n_vec) dst[i] = r[j];
    }
  }
}

// The lengths (and, when no block of a move launch could do it, the kept-index lists) as a
// kernel of their own: one CTA per sequence.  Used when there is nothing to move, when no layer
// is given, or when no counter bank is free.
__global__ void __launch_bounds__(256)
kv_compact_finish_kernel(int B, int32_t* __restrict__ kv_len, const int32_t* __restrict__ seg_start,
                         const int32_t* __restrict__ seg_len, int32_t* __restrict__ src_idx,
                         int idx_stride) {
  ms::pdl_wait();
  ms::pdl_trigger();
  const int b = blockIdx.x;
  const int L = kv_len[b], s = seg_start[b], n = seg_len[b];
  const bool valid = (n > 0 && s >= 0 && static_cast<int64_t>(s) + n <= L);
  const int shift = valid ? n : 0;
  const int new_len = L - shift;
  if (src_idx) {
    int32_t* row = src_idx + static_cast<int64_t>(b) * idx_stride;
    const int lim = new_len < idx_stride ? new_len : idx_stride;
    for (int j = threadIdx.x; j < lim; j += blockDim.x) row[j] = (valid && j >= s) ? j + shift : j;
  }
  __syncthreads();   // every thread has read kv_len[b] before it changes
  if (threadIdx.x == 0 && valid) kv_len[b] = new_len;
}

// Eviction by keep list.  One CTA per (layer, K|V, sequence, head).  keep[j] >= j and the list
// is increasing, so entry j's source lies at or above its destination and above every earlier
// destination: tiles of 128 entries are gathered completely into registers, the CTA
// synchronises, then the tile is written, tiles in increasing order -- a written slot is never
// needed again.  The leading entries with keep[j] == j stay where they are and are skipped.
__device__ __forceinline__ int gather_clamp(int nk, int L, int idx_stride) {
  return nk < 0 ? 0 : (nk > L ? L : (nk > idx_stride ? idx_stride : nk));
}

__global__ void __launch_bounds__(kMoveThreads)
kv_gather_kernel(uint16_t* __restrict__ k_cache, uint16_t* __restrict__ v_cache, int64_t layer_stride,
                 int64_t kv_head_stride, int B, int H_kv, int D, const int64_t* __restrict__ kv_off,
                 int32_t* __restrict__ kv_len, const int32_t* __restrict__ keep_idx, int idx_stride,
                 const int32_t* __restrict__ n_keep, unsigned int* done) {
  __shared__ int s_first, s_len, s_last;
  ms::pdl_wait();
  ms::pdl_trigger();
  int u = blockIdx.x;
  const int h = u % H_kv; u /= H_kv;
  const int b = u % B;    u /= B;
  const int is_v = u & 1; u >>= 1;
  const int layer = u;
  if (threadIdx.x == 0) {
    // old length first, then the count: the block that counts last writes the new lengths
    s_len = kv_len[b];
    int last = 0;
    if (done) {
      __threadfence();
      last = (atomicAdd(done, 1u) + 1u == gridDim.x) ? 1 : 0;
    }
    s_last = last;
  }
  __syncthreads();
  const int L = s_len;
  if (s_last) {
    for (int x = threadIdx.x; x < B; x += blockDim.x) kv_len[x] = gather_clamp(n_keep[x], kv_len[x], idx_stride);
    if (threadIdx.x == 0) *done = 0u;
  }
  const int nk = gather_clamp(n_keep[b], L, idx_stride);
  const int32_t* __restrict__ keep = keep_idx + static_cast<int64_t>(b) * idx_stride;
  uint4* base = reinterpret_cast<uint4*>((is_v ? v_cache : k_cache) + layer * layer_stride +
                                         h * kv_head_stride + kv_off[b] * static_cast<int64_t>(D));
  const int vpr = D / 8;                               // 16-byte vectors per entry
  const int per_tile = (kMoveThreads * kMoveUnroll) / vpr;   // entries per tile
  // first entry that moves (uniform over the CTA)
  if (threadIdx.x == 0) s_first = nk;
  __syncthreads();
  for (int j = threadIdx.x; j < nk; j += blockDim.x)
    if (keep[j] != j) { atomicMin(&s_first, j); break; }
  __syncthreads();
  const int j0 = (s_first / per_tile) * per_tile;
  for (int e0 = j0; e0 < nk; e0 += per_tile) {
    uint4 r[kMoveUnroll];
#pragma unroll
    for (int x = 0; x < kMoveUnroll; ++x) {
      const int i = threadIdx.x + x * kMoveThreads;
      const int e = e0 + i / vpr;
      if (i < per_tile * vpr && e < nk) {
        int src = keep[e];
        src = src < 0 ? 0 : (src >= L ? L - 1 : src);          // stay inside the sequence's slots
        r[x] = base[static_cast<int64_t>(src) * vpr + i % vpr];
      }
    }
    __syncthreads();
#pragma unroll
    for (int x = 0; x < kMoveUnroll; ++x) {
      const int i = threadIdx.x + x * kMoveThreads;
      const int e = e0 + i / vpr;
      if (i < per_tile * vpr && e < nk) base[static_cast<int64_t>(e) * vpr + i % vpr] = r[x];
    }
    __syncthreads();   // r[] of every thread is stored before the next tile overwrites it; tiles stay ordered
  }
}

__global__ void kv_gather_finish_kernel(int B, int32_t* __restrict__ kv_len, const int32_t* __restrict__ n_keep,
                                        int idx_stride) {
  ms::pdl_wait();
  ms::pdl_trigger();
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  kv_len[b] = gather_clamp(n_keep[b], kv_len[b], idx_stride);
}

struct AppendArgs {
  uint16_t* k_cache;
  uint16_t* v_cache;
  int64_t kv_head_stride, n_slots;
  int B, H_kv, D;
  const int64_t* kv_off;
  int32_t* kv_len;
  const int32_t* kv_cap;
  const uint16_t* k_step;
  const uint16_t* v_step;
  const int32_t* q_off;
  const int32_t* n_cand;
  const int32_t* n_keep;
  int32_t* overflow;
};

constexpr int kAppendRows = 16;   // block rows one CTA copies

// How many rows of block b are appended behind its L entries.  The request is clamped three
// times: to the candidates of the block (a foresight row is never cached), to the sequence's
// capacity (kv_cap[b] entries, when given) and to the end of the cache tensor -- an append never
// writes outside the sequence's own slots.  `clamped` says that room, not the request, decided.
__device__ __forceinline__ int append_keep(const AppendArgs& a, int b, int L, bool& clamped) {
  const int rows = a.q_off[b + 1] - a.q_off[b];
  const int nc = a.n_cand[b];
  int keep = a.n_keep[b];
  keep = keep < 0 ? 0 : (keep > nc ? nc : keep);
  keep = keep > rows ? rows : keep;
  int64_t room = a.n_slots - a.kv_off[b] - L;
  if (a.kv_cap && a.kv_cap[b] - static_cast<int64_t>(L) < room) room = a.kv_cap[b] - static_cast<int64_t>(L);
  if (L < 0 || room < 0) room = 0;
  clamped = keep > room;
  return clamped ? static_cast<int>(room) : keep;
}

// One CTA per (sequence, run of 16 block rows): copies the K and V rows, all KV heads, of the
// candidates that are kept to the first free slots.  The lengths move in the same launch: with
// one CTA per sequence (step blocks) that CTA does it after its copies have read the old length;
// with several, every CTA reads the old length and then counts itself on `done`, and the one
// that counts last moves the lengths of all sequences (nobody waits).  bump == 0 leaves them.
__global__ void __launch_bounds__(256)
kv_append_kernel(const AppendArgs a, int bump, unsigned int* done) {
  __shared__ int s_len, s_last;
  ms::pdl_wait();
  ms::pdl_trigger();
  const int b = blockIdx.x;
  if (threadIdx.x == 0) {
    s_len = a.kv_len[b];
    int last = 0;
    if (done) {
      __threadfence();   // the read above is ordered before the count
      last = (atomicAdd(done, 1u) + 1u == gridDim.x * gridDim.y) ? 1 : 0;
    }
    s_last = last;
  }
  __syncthreads();
  const int L = s_len;
  if (s_last) {
    for (int x = threadIdx.x; x < a.B; x += blockDim.x) {
      bool clamped;
      const int Lx = a.kv_len[x];
      a.kv_len[x] = Lx + append_keep(a, x, Lx, clamped);
    }
    if (threadIdx.x == 0) *done = 0u;
  }
  bool clamped;
  const int keep = append_keep(a, b, L, clamped);
  if (clamped && a.overflow && threadIdx.x == 0 && blockIdx.y == 0) *a.overflow = 1;
  const int i_lo = blockIdx.y * kAppendRows;
  const int i_hi = min(keep, i_lo + kAppendRows);
  const int vec_per_row = a.D / 8;
  const int per_row = 2 * a.H_kv * vec_per_row;
  const int r0 = a.q_off[b];
  const int64_t slot0 = a.kv_off[b] + L;
  for (int w = threadIdx.x; w < (i_hi - i_lo) * per_row; w += blockDim.x) {
    const int i = i_lo + w / per_row, x = w % per_row;
    const int is_v = x / (a.H_kv * vec_per_row);
    const int r = x - is_v * a.H_kv * vec_per_row;
    const int h = r / vec_per_row, c = r - h * vec_per_row;
    const int64_t srow = static_cast<int64_t>(r0 + i) * a.H_kv;
    const uint4* src = reinterpret_cast<const uint4*>((is_v ? a.v_step : a.k_step) + (srow + h) * a.D) + c;
    uint4* dst = reinterpret_cast<uint4*>((is_v ? a.v_cache : a.k_cache) + h * a.kv_head_stride + (slot0 + i) * a.D) + c;
    *dst = *src;
  }
  if (bump && !done && gridDim.y == 1) {
    __syncthreads();   // every thread is past its use of the old length
    if (threadIdx.x == 0) a.kv_len[b] = L + keep;
  }
}

// The lengths as a kernel of their own (blocks of more than 16 rows when no counter bank is free).
__global__ void kv_append_bump_kernel(const AppendArgs a) {
  ms::pdl_wait();
  ms::pdl_trigger();
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= a.B) return;
  bool clamped;
  const int L = a.kv_len[b];
  a.kv_len[b] = L + append_keep(a, b, L, clamped);
}

}  // namespace

extern "C" int32_t memosight_kv_compact(void* k_cache, void* v_cache, int32_t n_layers,
                                        int64_t layer_stride, int64_t kv_head_stride, int32_t batch,
                                        int32_t n_kv_heads, int32_t head_dim, const int64_t* kv_off,
                                        int32_t* kv_len, const int32_t* seg_start,
                                        const int32_t* seg_len, int32_t* src_idx, int32_t idx_stride,
                                        int32_t max_tail, memosight_stream_t stream) {
  if (n_layers < 0 || batch < 0 || n_kv_heads < 1 || head_dim < 1 || max_tail < 0 ||
      layer_stride < 0 || kv_head_stride < 0 || idx_stride < 0)
    return MS_ERR_INVALID_ARG;
  if (head_dim % 8) return MS_ERR_UNSUPPORTED_SHAPE;
  if (batch == 0) return MS_OK;
  if (!kv_off || !kv_len || !seg_start || !seg_len) return MS_ERR_INVALID_ARG;
  if (n_layers > 0 && (!k_cache || !v_cache)) return MS_ERR_INVALID_ARG;
  if (src_idx && idx_stride == 0) return MS_ERR_INVALID_ARG;
  if (n_layers > 0 && (!ms::aligned16(k_cache) || !ms::aligned16(v_cache) || (layer_stride % 8) ||
                       (kv_head_stride % 8)))
    return MS_ERR_ALIGNMENT;
  const int64_t units = static_cast<int64_t>(n_layers) * 2 * batch * n_kv_heads;
  if (units > 0x7fffffffLL) return MS_ERR_UNSUPPORTED_SHAPE;
  cudaStream_t st = ms::as_stream(stream);
  if (units > 0 && max_tail > 0) {
    // one launch when a counter bank is to be had: the block that reads the old lengths last
    // writes the new ones
    unsigned int* done = ms::done_bank(kv_len);
    MS_CUDA_TRY(ms::launch_pdl(kv_compact_move_kernel, dim3(static_cast<unsigned>(units)), dim3(kMoveThreads), 0, st,
                               static_cast<uint16_t*>(k_cache), static_cast<uint16_t*>(v_cache), layer_stride,
                               kv_head_stride, batch, n_kv_heads, head_dim, kv_off, kv_len, seg_start, seg_len,
                               done ? src_idx : nullptr, idx_stride, done));
    if (done) return MS_OK;
  }
  MS_CUDA_TRY(ms::launch_pdl(kv_compact_finish_kernel, dim3(batch), dim3(256), 0, st, batch, kv_len, seg_start,
                             seg_len, src_idx, idx_stride));
  return MS_OK;
}

extern "C" int32_t memosight_kv_gather(void* k_cache, void* v_cache, int32_t n_layers, int64_t layer_stride,
                                       int64_t kv_head_stride, int32_t batch, int32_t n_kv_heads,
                                       int32_t head_dim, const int64_t* kv_off, int32_t* kv_len,
                                       const int32_t* keep_idx, int32_t idx_stride, const int32_t* n_keep,
                                       int32_t max_keep, memosight_stream_t stream) {
  if (n_layers < 0 || batch < 0 || n_kv_heads < 1 || head_dim < 1 || max_keep < 0 || layer_stride < 0 ||
      kv_head_stride < 0 || idx_stride < 0)
    return MS_ERR_INVALID_ARG;
  if (head_dim % 8 || head_dim * 2 > kMoveThreads * kMoveUnroll * 16) return MS_ERR_UNSUPPORTED_SHAPE;
  if (batch == 0) return MS_OK;
  if (!kv_off || !kv_len || !n_keep || (max_keep > 0 && !keep_idx)) return MS_ERR_INVALID_ARG;
  if (n_layers > 0 && (!k_cache || !v_cache)) return MS_ERR_INVALID_ARG;
  if (n_layers > 0 && (!ms::aligned16(k_cache) || !ms::aligned16(v_cache) || (layer_stride % 8) ||
                       (kv_head_stride % 8)))
    return MS_ERR_ALIGNMENT;
  const int64_t units = static_cast<int64_t>(n_layers) * 2 * batch * n_kv_heads;
  if (units > 0x7fffffffLL) return MS_ERR_UNSUPPORTED_SHAPE;
  cudaStream_t st = ms::as_stream(stream);
  if (units > 0 && max_keep > 0) {
    unsigned int* done = ms::done_bank(kv_len);
    MS_CUDA_TRY(ms::launch_pdl(kv_gather_kernel, dim3(static_cast<unsigned>(units)), dim3(kMoveThreads), 0, st,
                               static_cast<uint16_t*>(k_cache), static_cast<uint16_t*>(v_cache), layer_stride,
                               kv_head_stride, batch, n_kv_heads, head_dim, kv_off, kv_len, keep_idx, idx_stride,
                               n_keep, done));
    if (done) return MS_OK;
  }
  MS_CUDA_TRY(ms::launch_pdl(kv_gather_finish_kernel, dim3((batch + 127) / 128), dim3(128), 0, st, batch, kv_len,
                             n_keep, idx_stride));
  return MS_OK;
}

extern "C" int32_t memosight_kv_append(void* k_cache, void* v_cache, int64_t kv_head_stride, int64_t n_slots,
                                       int32_t batch, int32_t n_kv_heads, int32_t head_dim,
                                       const int64_t* kv_off, int32_t* kv_len, const int32_t* kv_cap,
                                       const void* k_step, const void* v_step, const int32_t* q_off,
                                       const int32_t* n_cand, const int32_t* n_keep, int32_t max_nq,
                                       int32_t bump_len, int32_t* overflow, memosight_stream_t stream) {
  if (batch < 0 || n_kv_heads < 1 || head_dim < 1 || max_nq < 0 || kv_head_stride < 0 || n_slots < 0)
    return MS_ERR_INVALID_ARG;
  if (head_dim % 8) return MS_ERR_UNSUPPORTED_SHAPE;
  if (max_nq > ms::kMaxNqBig || n_slots >= (1ll << 31)) return MS_ERR_UNSUPPORTED_SHAPE;
  if (batch == 0) return MS_OK;
  if (!kv_off || !kv_len || !q_off || !n_cand || !n_keep) return MS_ERR_INVALID_ARG;
  if (kv_head_stride < n_slots * head_dim) return MS_ERR_INVALID_ARG;
  if (max_nq > 0 && (!k_cache || !v_cache || !k_step || !v_step)) return MS_ERR_INVALID_ARG;
  if (max_nq > 0 && (!ms::aligned16(k_cache) || !ms::aligned16(v_cache) || !ms::aligned16(k_step) ||
                     !ms::aligned16(v_step) || (kv_head_stride % 8)))
    return MS_ERR_ALIGNMENT;
  cudaStream_t st = ms::as_stream(stream);
  AppendArgs a;
  a.k_cache = static_cast<uint16_t*>(k_cache);
  a.v_cache = static_cast<uint16_t*>(v_cache);
  a.kv_head_stride = kv_head_stride;
  a.n_slots = n_slots;
  a.B = batch; a.H_kv = n_kv_heads; a.D = head_dim;
  a.kv_off = kv_off; a.kv_len = kv_len; a.kv_cap = kv_cap;
  a.k_step = static_cast<const uint16_t*>(k_step);
  a.v_step = static_cast<const uint16_t*>(v_step);
  a.q_off = q_off; a.n_cand = n_cand; a.n_keep = n_keep;
  a.overflow = overflow;
  const int chunks = max_nq > 0 ? (max_nq + kAppendRows - 1) / kAppendRows : 1;
  if (chunks > 65535) return MS_ERR_UNSUPPORTED_SHAPE;
  unsigned int* done = (bump_len && chunks > 1) ? ms::done_bank(kv_len) : nullptr;
  if (max_nq > 0 || bump_len)
    MS_CUDA_TRY(ms::launch_pdl(kv_append_kernel, dim3(batch, chunks), dim3(256), 0, st, a,
                               static_cast<int>(bump_len != 0), done));
  if (bump_len && chunks > 1 && !done)
    MS_CUDA_TRY(ms::launch_pdl(kv_append_bump_kernel, dim3((batch + 127) / 128), dim3(128), 0, st, a));
  return MS_OK;
}
