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

// One CTA per (layer, K|V, sequence, KV head).  Source and destination overlap
// whenever more entries move than were evicted, so a tile is read completely into
// registers, the CTA synchronises, and only then is it written; tiles go in
// increasing address order.  Because the shift is towards lower addresses, the
// bytes a tile writes lie strictly below everything later tiles still have to read.
__global__ void __launch_bounds__(kMoveThreads)
kv_compact_move_kernel(uint16_t* __restrict__ k_cache, uint16_t* __restrict__ v_cache,
                       int64_t layer_stride, int64_t kv_head_stride, int B, int H_kv, int D,
                       const int64_t* __restrict__ kv_off, const int32_t* __restrict__ kv_len,
                       const int32_t* __restrict__ seg_start, const int32_t* __restrict__ seg_len) {
  int u = blockIdx.x;
  const int h = u % H_kv; u /= H_kv;
  const int b = u % B;    u /= B;
  const int is_v = u & 1; u >>= 1;
  const int layer = u;
  const int L = kv_len[b], s = seg_start[b], n = seg_len[b];
  if (n <= 0 || s < 0 || static_cast<int64_t>(s) + n > L) return;   // nothing to do / ignored
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

// One CTA per sequence, after the moves: emit the kept-index list and the new length.
__global__ void __launch_bounds__(256)
kv_compact_finish_kernel(int B, int32_t* __restrict__ kv_len, const int32_t* __restrict__ seg_start,
                         const int32_t* __restrict__ seg_len, int32_t* __restrict__ src_idx,
                         int idx_stride) {
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
__global__ void __launch_bounds__(kMoveThreads)
kv_gather_kernel(uint16_t* __restrict__ k_cache, uint16_t* __restrict__ v_cache, int64_t layer_stride,
                 int64_t kv_head_stride, int B, int H_kv, int D, const int64_t* __restrict__ kv_off,
                 const int32_t* __restrict__ kv_len, const int32_t* __restrict__ keep_idx, int idx_stride,
                 const int32_t* __restrict__ n_keep) {
  int u = blockIdx.x;
  const int h = u % H_kv; u /= H_kv;
  const int b = u % B;    u /= B;
  const int is_v = u & 1; u >>= 1;
  const int layer = u;
  const int L = kv_len[b];
  int nk = n_keep[b];
  nk = nk < 0 ? 0 : (nk > L ? L : (nk > idx_stride ? idx_stride : nk));
  const int32_t* __restrict__ keep = keep_idx + static_cast<int64_t>(b) * idx_stride;
  uint4* base = reinterpret_cast<uint4*>((is_v ? v_cache : k_cache) + layer * layer_stride +
                                         h * kv_head_stride + kv_off[b] * static_cast<int64_t>(D));
  const int vpr = D / 8;                               // 16-byte vectors per entry
  const int per_tile = (kMoveThreads * kMoveUnroll) / vpr;   // entries per tile
  // first entry that moves (uniform over the CTA)
  __shared__ int s_first;
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
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  const int L = kv_len[b];
  int nk = n_keep[b];
  nk = nk < 0 ? 0 : (nk > L ? L : (nk > idx_stride ? idx_stride : nk));
  kv_len[b] = nk;
}

// One CTA per (sequence, block row): copies that candidate's K and V rows of all
// KV heads to the first free slot + row.
__global__ void __launch_bounds__(128)
kv_append_kernel(uint16_t* __restrict__ k_cache, uint16_t* __restrict__ v_cache,
                 int64_t kv_head_stride, int H_kv, int D, const int64_t* __restrict__ kv_off,
                 const int32_t* __restrict__ kv_len, const uint16_t* __restrict__ k_step,
                 const uint16_t* __restrict__ v_step, const int32_t* __restrict__ q_off,
                 const int32_t* __restrict__ n_cand, const int32_t* __restrict__ n_keep) {
  const int b = blockIdx.x, i = blockIdx.y;
  int keep = n_keep[b];
  const int nc = n_cand[b];
  keep = keep < 0 ? 0 : (keep > nc ? nc : keep);
  if (i >= keep || q_off[b] + i >= q_off[b + 1]) return;
  const int vec_per_row = D / 8;
  const int64_t slot = kv_off[b] + kv_len[b] + i;
  const int64_t srow = static_cast<int64_t>(q_off[b] + i) * H_kv;
  for (int w = threadIdx.x; w < 2 * H_kv * vec_per_row; w += blockDim.x) {
    const int is_v = w / (H_kv * vec_per_row);
    const int r = w - is_v * H_kv * vec_per_row;
    const int h = r / vec_per_row, c = r - h * vec_per_row;
    const uint4* src = reinterpret_cast<const uint4*>((is_v ? v_step : k_step) + (srow + h) * D) + c;
    uint4* dst = reinterpret_cast<uint4*>((is_v ? v_cache : k_cache) + h * kv_head_stride + slot * D) + c;
    *dst = *src;
  }
}

__global__ void kv_append_bump_kernel(int B, int32_t* __restrict__ kv_len,
                                      const int32_t* __restrict__ q_off,
                                      const int32_t* __restrict__ n_cand,
                                      const int32_t* __restrict__ n_keep) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  int keep = n_keep[b];
  const int nc = n_cand[b], rows = q_off[b + 1] - q_off[b];
  keep = keep < 0 ? 0 : (keep > nc ? nc : keep);
  keep = keep > rows ? rows : keep;
  kv_len[b] += keep;
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
    kv_compact_move_kernel<<<static_cast<unsigned>(units), kMoveThreads, 0, st>>>(
        static_cast<uint16_t*>(k_cache), static_cast<uint16_t*>(v_cache), layer_stride,
        kv_head_stride, batch, n_kv_heads, head_dim, kv_off, kv_len, seg_start, seg_len);
    MS_LAUNCH_CHECK();
  }
  kv_compact_finish_kernel<<<batch, 256, 0, st>>>(batch, kv_len, seg_start, seg_len, src_idx,
                                                  idx_stride);
  MS_LAUNCH_CHECK();
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
    kv_gather_kernel<<<static_cast<unsigned>(units), kMoveThreads, 0, st>>>(
        static_cast<uint16_t*>(k_cache), static_cast<uint16_t*>(v_cache), layer_stride, kv_head_stride, batch,
        n_kv_heads, head_dim, kv_off, kv_len, keep_idx, idx_stride, n_keep);
    MS_LAUNCH_CHECK();
  }
  kv_gather_finish_kernel<<<(batch + 127) / 128, 128, 0, st>>>(batch, kv_len, n_keep, idx_stride);
  MS_LAUNCH_CHECK();
  return MS_OK;
}

extern "C" int32_t memosight_kv_append(void* k_cache, void* v_cache, int64_t kv_head_stride,
                                       int32_t batch, int32_t n_kv_heads, int32_t head_dim,
                                       const int64_t* kv_off, int32_t* kv_len, const void* k_step,
                                       const void* v_step, const int32_t* q_off,
                                       const int32_t* n_cand, const int32_t* n_keep, int32_t max_nq,
                                       int32_t bump_len, memosight_stream_t stream) {
  if (batch < 0 || n_kv_heads < 1 || head_dim < 1 || max_nq < 0 || kv_head_stride < 0)
    return MS_ERR_INVALID_ARG;
  if (head_dim % 8) return MS_ERR_UNSUPPORTED_SHAPE;
  if (max_nq > 65535) return MS_ERR_UNSUPPORTED_SHAPE;
  if (batch == 0) return MS_OK;
  if (!kv_off || !kv_len || !q_off || !n_cand || !n_keep) return MS_ERR_INVALID_ARG;
  if (max_nq > 0 && (!k_cache || !v_cache || !k_step || !v_step)) return MS_ERR_INVALID_ARG;
  if (max_nq > 0 && (!ms::aligned16(k_cache) || !ms::aligned16(v_cache) || !ms::aligned16(k_step) ||
                     !ms::aligned16(v_step) || (kv_head_stride % 8)))
    return MS_ERR_ALIGNMENT;
  cudaStream_t st = ms::as_stream(stream);
  if (max_nq > 0) {
    kv_append_kernel<<<dim3(batch, max_nq), 128, 0, st>>>(
        static_cast<uint16_t*>(k_cache), static_cast<uint16_t*>(v_cache), kv_head_stride, n_kv_heads,
        head_dim, kv_off, kv_len, static_cast<const uint16_t*>(k_step),
        static_cast<const uint16_t*>(v_step), q_off, n_cand, n_keep);
    MS_LAUNCH_CHECK();
  }
  if (bump_len) {
    kv_append_bump_kernel<<<(batch + 127) / 128, 128, 0, st>>>(batch, kv_len, q_off, n_cand, n_keep);
    MS_LAUNCH_CHECK();
  }
  return MS_OK;
}
