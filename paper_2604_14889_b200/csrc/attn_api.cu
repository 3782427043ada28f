// Entry points of the step attention: argument validation, path selection,
// workspace sizing and the device status word.
#include <math.h>
#include <stddef.h>

#include "attn_internal.cuh"

#include <atomic>

namespace {

std::atomic<int32_t> g_forced_path{MS_ATTN_PATH_AUTO};
constexpr int32_t kPathBig = 100;   // large-block tcgen05 kernel (chosen by shape only)

bool mma_shape(int D, int G, int max_nq) {
  return (D == 64 || D == 128) && max_nq <= ms::kMaxNq && max_nq * G <= 64;
}

// Either tensor-core path: both use the per-CTA partial slots of the split-KV workspace.
bool fast_path_shape(int D, int G, int max_nq) {
  return mma_shape(D, G, max_nq) || ms::attn_umma_supports(D, G, max_nq);
}

// Which kernel serves a shape.  head_dim 128 with up to 64 packed rows -- every step block of
// the method -- streams fastest through the keys-on-lanes tcgen05 kernel, whose softmax cost
// follows the block size; more rows or more than 16 tokens take the row-tiled large-block
// kernel; head_dim 64 stays on the mma.sync kernel up to 64 rows and on the rows-on-lanes
// tcgen05 kernel up to 128.
int32_t pick_path(int D, int G, int max_nq) {
  const int32_t forced = g_forced_path.load(std::memory_order_relaxed);
  const bool mma_ok = mma_shape(D, G, max_nq), umma_ok = ms::attn_umma_supports(D, G, max_nq);
  const bool umma_t_ok = ms::attn_umma_t_supports(D, G, max_nq);
  if (forced == MS_ATTN_PATH_MMA_SYNC && mma_ok) return forced;
  if (forced == MS_ATTN_PATH_TCGEN05 && umma_ok) return forced;
  if (forced == MS_ATTN_PATH_TCGEN05_KEYS && umma_t_ok) return forced;
  if (forced == MS_ATTN_PATH_GENERAL) return forced;
  if (ms::attn_umma_big_supports(D, G, max_nq)) return kPathBig;
  if (umma_t_ok) return MS_ATTN_PATH_TCGEN05_KEYS;
  if (mma_ok) return MS_ATTN_PATH_MMA_SYNC;
  if (umma_ok) return MS_ATTN_PATH_TCGEN05;
  return MS_ATTN_PATH_GENERAL;
}

}  // namespace

extern "C" int32_t memosight_attn_set_path(int32_t path) {
  if (path < MS_ATTN_PATH_AUTO || path > MS_ATTN_PATH_LARGE_BLOCK) return MS_ERR_INVALID_ARG;
  return g_forced_path.exchange(path, std::memory_order_relaxed);
}

extern "C" size_t memosight_attn_workspace_bytes(int32_t batch, int32_t n_q_heads,
                                                 int32_t n_kv_heads, int32_t head_dim,
                                                 int32_t max_kv_len, int32_t max_nq) {
  if (batch < 0 || n_kv_heads < 1 || n_q_heads < 1 || n_q_heads % n_kv_heads || head_dim < 1 ||
      max_kv_len < 0 || max_nq < 1 || max_nq > ms::kMaxNqBig)
    return 0;
  const int G = n_q_heads / n_kv_heads;
  int n_ctas = ms::attn_mma_grid();
  if (n_ctas <= 0) n_ctas = 256;   // no device visible: answer for the largest part we target
  if (ms::attn_umma_big_supports(head_dim, G, max_nq))
    return ms::attn_umma_big_workspace_bytes(batch, n_kv_heads, G, max_nq, max_kv_len, n_ctas);
  if (!fast_path_shape(head_dim, G, max_nq)) return ms::kWsHeaderBytes;
  const int rows_pad = (max_nq * G + 15) & ~15;
  return ms::attn_mma_workspace_bytes(head_dim, rows_pad, n_ctas);
}

extern "C" int32_t memosight_attn_step(const memosight_attn_params* p, memosight_stream_t stream) {
  // structures of callers built before the training-mask fields existed end at tok_kind
  constexpr uint32_t kOldSize = offsetof(memosight_attn_params, tok_kind);
  if (!p || (p->struct_size != sizeof(memosight_attn_params) && p->struct_size != kOldSize)) return MS_ERR_INVALID_ARG;
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
  if (p->batch == 0 || p->total_rows == 0) return MS_OK;
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
  const size_t need = memosight_attn_workspace_bytes(p->batch, p->n_q_heads, p->n_kv_heads,
                                                     p->head_dim, p->max_kv_len, p->max_nq);
  if (need == 0) return MS_ERR_INVALID_ARG;
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
  a.ev_split_begin = static_cast<cudaEvent_t>(p->ev_split_begin);
  a.ev_split_end = static_cast<cudaEvent_t>(p->ev_split_end);

  cudaStream_t st = ms::as_stream(stream);
  // An empty cache tensor still needs a valid address for the tile descriptors.
  int32_t path = (a.k_cache && a.v_cache && a.n_slots >= 1) ? pick_path(a.D, G, a.max_nq) : MS_ATTN_PATH_GENERAL;
  if (tok_kind && path != kPathBig) path = MS_ATTN_PATH_GENERAL;   // the step kernels know the inference rule only
  // the large-block kernel on a step block, when asked for and the workspace is large enough for it
  if (g_forced_path.load(std::memory_order_relaxed) == MS_ATTN_PATH_LARGE_BLOCK && a.D == 128 && a.k_cache &&
      a.v_cache && a.n_slots >= 1 &&
      p->workspace_bytes >= ms::attn_umma_big_workspace_bytes(a.B, a.H_kv, G, a.max_nq, a.max_kv_len, ms::attn_mma_grid()))
    path = kPathBig;
  if (path == MS_ATTN_PATH_MMA_SYNC) return ms::launch_attn_mma(a, st);
  if (path == MS_ATTN_PATH_TCGEN05) return ms::launch_attn_umma(a, st);
  if (path == MS_ATTN_PATH_TCGEN05_KEYS) return ms::launch_attn_umma_t(a, st);
  if (path == kPathBig) return ms::launch_attn_umma_big(a, st);
  return ms::launch_attn_simt(a, st);
}

extern "C" int32_t memosight_attn_status(const void* workspace, memosight_stream_t stream) {
  if (!workspace) return MS_ERR_INVALID_ARG;
  MS_CUDA_TRY(cudaStreamSynchronize(ms::as_stream(stream)));
  uint32_t word = 0;
  MS_CUDA_TRY(cudaMemcpy(&word, workspace, sizeof word, cudaMemcpyDeviceToHost));
  if (word == 0x4D535431u || word == 0x4D535432u) {
    const uint32_t zero = 0;
    MS_CUDA_TRY(cudaMemcpy(const_cast<void*>(workspace), &zero, sizeof zero, cudaMemcpyHostToDevice));
    return MS_ERR_DEVICE_TIMEOUT;
  }
  return MS_OK;
}
