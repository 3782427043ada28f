// Entry points of the step attention: argument validation, path selection,
// workspace sizing and the device status word.
#include <math.h>
#include <stddef.h>

#include "attn_sched.cuh"

#include <atomic>
#include <mutex>

namespace {

std::atomic<int32_t> g_forced_path{MS_ATTN_PATH_AUTO};
constexpr int32_t kPathBig = 100;   // large-block tcgen05 kernel (MS_ATTN_PATH_LARGE_BLOCK when forced)

// Timing events of the calling thread (memosight_attn_debug_events).
thread_local cudaEvent_t t_ev_begin = nullptr, t_ev_end = nullptr;

struct Shape {
  int B, H_kv, G, D, max_kv_len, max_nq;
};

bool mma_shape(const Shape& s) {
  return (s.D == 64 || s.D == 128) && s.max_nq <= ms::kMaxNq && s.max_nq * s.G <= 64;
}

// Does `path` serve the shape at all?
bool path_covers(int32_t path, const Shape& s) {
  switch (path) {
    case MS_ATTN_PATH_MMA_SYNC: return mma_shape(s);
    case MS_ATTN_PATH_TCGEN05: return ms::attn_umma_supports(s.D, s.G, s.max_nq);
    case MS_ATTN_PATH_TCGEN05_KEYS: return ms::attn_umma_t_supports(s.D, s.G, s.max_nq);
    case MS_ATTN_PATH_GENERAL: return true;
    case kPathBig: return s.D == 128 && s.G <= ms::kMaxGroup && s.max_nq <= ms::kMaxNqBig;
    default: return false;
  }
}

// Workspace a path needs for the shape.  Path and size always come from this one table, so a
// kernel is never launched on a workspace that was sized for another.
size_t path_workspace(int32_t path, const Shape& s) {
  int n_ctas = ms::attn_mma_grid();
  if (n_ctas <= 0) n_ctas = 256;   // no device visible: answer for the largest part we target
  switch (path) {
    case MS_ATTN_PATH_MMA_SYNC:
    case MS_ATTN_PATH_TCGEN05:
    case MS_ATTN_PATH_TCGEN05_KEYS:
      return ms::attn_mma_workspace_bytes(s.D, (s.max_nq * s.G + 15) & ~15, n_ctas);
    case kPathBig:
      return ms::attn_umma_big_workspace_bytes(s.B, s.H_kv, s.G, s.max_nq, s.max_kv_len, n_ctas);
    default:
      return ms::kWsHeaderBytes;
  }
}

// Which kernel serves a shape when nothing is forced.  head_dim 128 with up to 64 packed rows --
// every step block of the method -- streams fastest through the keys-on-lanes tcgen05 kernel,
// whose softmax cost follows the block size; more rows or more than 16 tokens take the row-tiled
// large-block kernel; head_dim 64 stays on the mma.sync kernel up to 64 rows and on the
// rows-on-lanes tcgen05 kernel up to 128.
int32_t auto_path(const Shape& s) {
  if (ms::attn_umma_big_supports(s.D, s.G, s.max_nq)) return kPathBig;
  if (path_covers(MS_ATTN_PATH_TCGEN05_KEYS, s)) return MS_ATTN_PATH_TCGEN05_KEYS;
  if (path_covers(MS_ATTN_PATH_MMA_SYNC, s)) return MS_ATTN_PATH_MMA_SYNC;
  if (path_covers(MS_ATTN_PATH_TCGEN05, s)) return MS_ATTN_PATH_TCGEN05;
  return MS_ATTN_PATH_GENERAL;
}

// The path of one call: the forced one if it covers the shape AND the caller's workspace is large
// enough for it, else the automatic choice.
int32_t pick_path(const Shape& s, size_t workspace_bytes) {
  int32_t forced = g_forced_path.load(std::memory_order_relaxed);
  if (forced == MS_ATTN_PATH_LARGE_BLOCK) forced = kPathBig;
  if (forced != MS_ATTN_PATH_AUTO && path_covers(forced, s) && workspace_bytes >= path_workspace(forced, s))
    return forced;
  return auto_path(s);
}

// ---- tensor-map cache ----
struct MapKey {
  int rank;
  const void* base;
  uint64_t dims[4], strides[3];
  uint32_t box[4];
  bool operator==(const MapKey& o) const {
    if (rank != o.rank || base != o.base) return false;
    for (int i = 0; i < 4; ++i)
      if (dims[i] != o.dims[i] || box[i] != o.box[i]) return false;
    for (int i = 0; i < 3; ++i)
      if (strides[i] != o.strides[i]) return false;
    return true;
  }
};
constexpr int kMapCacheSize = 64;
struct MapCache {
  std::mutex mu;
  MapKey key[kMapCacheSize];
  CUtensorMap map[kMapCacheSize];
  int used = 0, next = 0;
};
MapCache g_maps;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static std::atomic<EncodeTiledFn> fn{nullptr};
  EncodeTiledFn f = fn.load(std::memory_order_acquire);
  if (!f) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess) {
      f = reinterpret_cast<EncodeTiledFn>(p);
      fn.store(f, std::memory_order_release);
    }
  }
  return f;
}

}  // namespace

namespace ms {

bool tensor_map_cached(CUtensorMap* map, int rank, const void* base, const uint64_t* dims,
                       const uint64_t* strides_bytes, const uint32_t* box) {
  if (rank < 3 || rank > 4) return false;
  MapKey k = {};
  k.rank = rank;
  k.base = base;
  for (int i = 0; i < rank; ++i) { k.dims[i] = dims[i]; k.box[i] = box[i]; }
  for (int i = 0; i + 1 < rank; ++i) k.strides[i] = strides_bytes[i];
  std::lock_guard<std::mutex> lock(g_maps.mu);
  for (int i = 0; i < g_maps.used; ++i) {
    if (g_maps.key[i] == k) {
      *map = g_maps.map[i];
      return true;
    }
  }
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t d[4], st[3];
  cuuint32_t bx[4], es[4] = {1, 1, 1, 1};
  for (int i = 0; i < rank; ++i) { d[i] = k.dims[i]; bx[i] = k.box[i]; }
  for (int i = 0; i + 1 < rank; ++i) st[i] = k.strides[i];
  if (fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, static_cast<cuuint32_t>(rank), const_cast<void*>(base), d, st, bx,
         es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  const int slot = g_maps.used < kMapCacheSize ? g_maps.used++ : (g_maps.next++ % kMapCacheSize);
  g_maps.key[slot] = k;
  g_maps.map[slot] = *map;
  return true;
}

}  // namespace ms

extern "C" int32_t memosight_attn_set_path(int32_t path) {
  if (path < MS_ATTN_PATH_AUTO || path > MS_ATTN_PATH_LARGE_BLOCK) return MS_ERR_INVALID_ARG;
  return g_forced_path.exchange(path, std::memory_order_relaxed);
}

extern "C" int32_t memosight_attn_debug_events(void* ev_split_begin, void* ev_split_end) {
  if ((ev_split_begin == nullptr) != (ev_split_end == nullptr)) return MS_ERR_INVALID_ARG;
  t_ev_begin = static_cast<cudaEvent_t>(ev_split_begin);
  t_ev_end = static_cast<cudaEvent_t>(ev_split_end);
  return MS_OK;
}

extern "C" size_t memosight_attn_workspace_bytes(int32_t batch, int32_t n_q_heads,
                                                 int32_t n_kv_heads, int32_t head_dim,
                                                 int32_t max_kv_len, int32_t max_nq) {
  if (batch < 0 || n_kv_heads < 1 || n_q_heads < 1 || n_q_heads % n_kv_heads || head_dim < 1 ||
      max_kv_len < 0 || max_nq < 1 || max_nq > ms::kMaxNqBig)
    return 0;
  const Shape s{batch, n_kv_heads, n_q_heads / n_kv_heads, head_dim, max_kv_len, max_nq};
  return path_workspace(auto_path(s), s);
}

namespace {

int32_t attn_call(const memosight_attn_params* p, const memosight_attn_layers* ly, memosight_stream_t stream) {
  // structures of callers built before the training-mask fields existed end at tok_kind
  constexpr uint32_t kOldSize = offsetof(memosight_attn_params, tok_kind);
  if (!p || (p->struct_size != sizeof(memosight_attn_params) && p->struct_size != kOldSize)) return MS_ERR_INVALID_ARG;
  if (ly && ly->struct_size != sizeof(memosight_attn_layers)) return MS_ERR_INVALID_ARG;
  const bool has_meta = p->struct_size == sizeof(memosight_attn_params);
  const uint8_t* tok_kind = has_meta ? p->tok_kind : nullptr;
  const int32_t* tok_step = has_meta ? p->tok_step : nullptr;
  if ((tok_kind == nullptr) != (tok_step == nullptr)) return MS_ERR_INVALID_ARG;
  if (p->batch < 0 || p->n_kv_heads < 1 || p->n_q_heads < 1 || p->head_dim < 1 ||
      p->max_kv_len < 0 || p->total_rows < 0 || p->n_slots < 0 || p->kv_head_stride < 0)
    return MS_ERR_INVALID_ARG;
  if (p->n_q_heads % p->n_kv_heads) return MS_ERR_INVALID_ARG;
  const int G = p->n_q_heads / p->n_kv_heads;
  if (G > ms::kMaxGroup || p->max_nq < 1 || p->max_nq > ms::kMaxNqBig || p->batch > ms::kMaxBatch ||
      p->head_dim % 32 || p->head_dim > 256 || p->n_slots >= (1ll << 31))
    return MS_ERR_UNSUPPORTED_SHAPE;
  const int n_layers = ly ? ly->n_layers : 1;
  if (n_layers < 0 || n_layers > 4096) return MS_ERR_INVALID_ARG;
  if (p->batch == 0 || p->total_rows == 0 || n_layers == 0) return MS_OK;
  if (!p->kv_off || !p->kv_len || !p->q_off || !p->n_cand || !p->q || !p->k_step || !p->v_step ||
      !p->out || !p->workspace)
    return MS_ERR_INVALID_ARG;
  if (p->max_kv_len > 0 && (!p->k_cache || !p->v_cache || p->n_slots < 1)) return MS_ERR_INVALID_ARG;
  if (p->kv_head_stride < p->n_slots * p->head_dim) return MS_ERR_INVALID_ARG;
  if (!(p->sm_scale >= 0.f) || isinf(p->sm_scale)) return MS_ERR_INVALID_ARG;
  if (!ms::aligned16(p->k_cache) || !ms::aligned16(p->v_cache) || !ms::aligned16(p->q) ||
      !ms::aligned16(p->k_step) || !ms::aligned16(p->v_step) || !ms::aligned16(p->out) ||
      (p->kv_head_stride % 8) || (reinterpret_cast<uintptr_t>(p->workspace) & 255u))
    return MS_ERR_ALIGNMENT;
  if (ly && n_layers > 1) {
    // every layer's tensors must lie behind the previous layer's and keep the 16-byte rule
    const int64_t T = p->total_rows, D = p->head_dim;
    if (ly->kv_layer_stride < static_cast<int64_t>(p->n_kv_heads) * p->kv_head_stride ||
        ly->q_layer_stride < T * p->n_q_heads * D || ly->kstep_layer_stride < T * p->n_kv_heads * D ||
        ly->out_layer_stride < T * p->n_q_heads * D || (p->lse && ly->lse_layer_stride < T * p->n_q_heads))
      return MS_ERR_INVALID_ARG;
    if ((ly->kv_layer_stride % 8) || (ly->q_layer_stride % 8) || (ly->kstep_layer_stride % 8) ||
        (ly->out_layer_stride % 8))
      return MS_ERR_ALIGNMENT;
  }
  const Shape shape{p->batch, p->n_kv_heads, G, p->head_dim, p->max_kv_len, p->max_nq};
  const size_t need = path_workspace(auto_path(shape), shape);
  if (p->workspace_bytes < need) return MS_ERR_WORKSPACE_TOO_SMALL;

  ms::AttnArgs a;
  a.B = p->batch; a.H_q = p->n_q_heads; a.H_kv = p->n_kv_heads; a.G = G; a.D = p->head_dim;
  a.T = p->total_rows;
  a.k_cache = static_cast<const __nv_bfloat16*>(p->k_cache);
  a.v_cache = static_cast<const __nv_bfloat16*>(p->v_cache);
  a.kv_head_stride = p->kv_head_stride;
  a.n_slots = p->n_slots;
  a.kv_off = p->kv_off; a.kv_len = p->kv_len; a.q_off = p->q_off; a.n_cand = p->n_cand;
  a.anchor = p->anchor;
  a.tok_kind = tok_kind;
  a.tok_step = tok_step;
  a.q = static_cast<const __nv_bfloat16*>(p->q);
  a.k_step = static_cast<const __nv_bfloat16*>(p->k_step);
  a.v_step = static_cast<const __nv_bfloat16*>(p->v_step);
  a.out = static_cast<__nv_bfloat16*>(p->out);
  a.lse = p->lse;
  const double scale = p->sm_scale > 0.f ? static_cast<double>(p->sm_scale)
                                         : 1.0 / sqrt(static_cast<double>(p->head_dim));
  a.scale_log2 = static_cast<float>(scale * 1.4426950408889634);
  a.max_kv_len = p->max_kv_len; a.max_nq = p->max_nq;
  a.workspace = p->workspace;
  a.n_layers = 1;
  a.kv_layer_stride = a.q_layer_stride = a.kstep_layer_stride = a.out_layer_stride = a.lse_layer_stride = 0;
  a.done = nullptr;
  a.wait_limit_us = ms::wait_limit_us();
  a.ev_split_begin = t_ev_begin;
  a.ev_split_end = t_ev_end;

  cudaStream_t st = ms::as_stream(stream);
  // An empty cache tensor still needs a valid address for the tile descriptors.
  int32_t path = (a.k_cache && a.v_cache && a.n_slots >= 1) ? pick_path(shape, p->workspace_bytes) : MS_ATTN_PATH_GENERAL;
  if (tok_kind && path != kPathBig) path = MS_ATTN_PATH_GENERAL;   // the step kernels know the inference rule only
  if (path == MS_ATTN_PATH_TCGEN05_KEYS) {
    // the keys-on-lanes kernel walks the stacked layers in one launch
    if (n_layers > 1) {
      a.n_layers = n_layers;
      a.kv_layer_stride = ly->kv_layer_stride; a.q_layer_stride = ly->q_layer_stride;
      a.kstep_layer_stride = ly->kstep_layer_stride; a.out_layer_stride = ly->out_layer_stride;
      a.lse_layer_stride = ly->lse_layer_stride;
    }
    return ms::launch_attn_umma_t(a, st);
  }
  // every other kernel takes the layers one launch after the other
  for (int l = 0; l < n_layers; ++l) {
    ms::AttnArgs al = a;
    if (l > 0) {
      al.k_cache = a.k_cache ? a.k_cache + l * ly->kv_layer_stride : nullptr;
      al.v_cache = a.v_cache ? a.v_cache + l * ly->kv_layer_stride : nullptr;
      al.q = a.q + l * ly->q_layer_stride;
      al.k_step = a.k_step + l * ly->kstep_layer_stride;
      al.v_step = a.v_step + l * ly->kstep_layer_stride;
      al.out = a.out + l * ly->out_layer_stride;
      al.lse = a.lse ? a.lse + l * ly->lse_layer_stride : nullptr;
    }
    int32_t rc;
    if (path == MS_ATTN_PATH_MMA_SYNC) rc = ms::launch_attn_mma(al, st);
    else if (path == MS_ATTN_PATH_TCGEN05) rc = ms::launch_attn_umma(al, st);
    else if (path == kPathBig) rc = ms::launch_attn_umma_big(al, st);
    else rc = ms::launch_attn_simt(al, st);
    if (rc != MS_OK) return rc;
  }
  return MS_OK;
}

}  // namespace

extern "C" int32_t memosight_attn_step(const memosight_attn_params* p, memosight_stream_t stream) {
  return attn_call(p, nullptr, stream);
}

extern "C" int32_t memosight_attn_step_layers(const memosight_attn_params* p, const memosight_attn_layers* layers,
                                              memosight_stream_t stream) {
  if (!layers) return MS_ERR_INVALID_ARG;
  return attn_call(p, layers, stream);
}

namespace {

// One warp waits, with the bounded wait every kernel of the library uses, on a barrier at which
// nobody ever arrives: the wait runs into its limit, records that in the status word and returns.
__global__ void wait_probe_kernel(uint32_t* status, unsigned int limit_us) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int ctx[2];
  if (threadIdx.x == 0) {
    ms::mbar_init(ms::smem_u32(&bar), 1);
    ms::wait_ctx_init(ctx, limit_us);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  (void)ms::mbar_wait(ms::smem_u32(&bar), 0, ctx, status);
}

}  // namespace

extern "C" int32_t memosight_debug_wait_timeout(void* workspace, uint32_t limit_us, memosight_stream_t stream) {
  if (!workspace || limit_us == 0 || limit_us > 1000000u) return MS_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return MS_ERR_ALIGNMENT;
  wait_probe_kernel<<<1, 32, 0, ms::as_stream(stream)>>>(static_cast<uint32_t*>(workspace), limit_us);
  MS_LAUNCH_CHECK();
  return MS_OK;
}

extern "C" int32_t memosight_attn_status(const void* workspace, memosight_stream_t stream) {
  if (!workspace) return MS_ERR_INVALID_ARG;
  cudaStream_t st = ms::as_stream(stream);
  MS_CUDA_TRY(cudaStreamSynchronize(st));
  uint32_t word = 0;
  MS_CUDA_TRY(cudaMemcpy(&word, workspace, sizeof word, cudaMemcpyDeviceToHost));
  if (word == 0x4D535431u || word == 0x4D535432u) {
    const uint32_t zero = 0;
    MS_CUDA_TRY(cudaMemcpy(const_cast<void*>(workspace), &zero, sizeof zero, cudaMemcpyHostToDevice));
    // a kernel that gave up may have left merge counters behind: put them back to zero
    const int32_t rc = ms::done_bank_clear(workspace, st);
    if (rc != MS_OK) return rc;
    MS_CUDA_TRY(cudaStreamSynchronize(st));
    return MS_ERR_DEVICE_TIMEOUT;
  }
  return MS_OK;
}
