// One whole decode step, by default driven from host-resident step data: copies in, the
// kernels of the hot path in their order (Algorithm 1: forward pass attention,
// greedy accept, S <- S (+) A, optional UpdateCache), copies out.  Pure
// sequencing of the other entry points on the caller's stream -- except that the
// logits, by far the largest input and needed only by the accept, are copied on a
// second stream of the library's own while RoPE and the attention run, and joined
// back by an event before the accept.
#include <mutex>

#include "common.cuh"

namespace {

struct CopyLane {
  cudaStream_t stream = nullptr;
  cudaEvent_t fork = nullptr, join = nullptr;
};

// One copy stream and two events per device, created at the first call on that device.
int32_t copy_lane(CopyLane** out) {
  static std::mutex mu;
  static CopyLane lanes[64];
  int dev = 0;
  MS_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return MS_ERR_UNSUPPORTED_SHAPE;
  std::lock_guard<std::mutex> lock(mu);
  CopyLane& l = lanes[dev];
  if (!l.stream) {
    cudaStream_t s = nullptr;
    cudaEvent_t f = nullptr, j = nullptr;
    MS_CUDA_TRY(cudaStreamCreateWithFlags(&s, cudaStreamNonBlocking));
    MS_CUDA_TRY(cudaEventCreateWithFlags(&f, cudaEventDisableTiming));
    MS_CUDA_TRY(cudaEventCreateWithFlags(&j, cudaEventDisableTiming));
    l.fork = f;
    l.join = j;
    l.stream = s;
  }
  *out = &l;
  return MS_OK;
}

}  // namespace

extern "C" int32_t memosight_step_host(const memosight_step_host_params* p,
                                       memosight_stream_t stream) {
  if (!p || p->struct_size != sizeof(memosight_step_host_params)) return MS_ERR_INVALID_ARG;
  const memosight_attn_params& a = p->attn;
  if (a.struct_size != sizeof(memosight_attn_params)) return MS_ERR_INVALID_ARG;
  const int32_t T = a.total_rows, B = a.batch;
  if (T < 0 || B < 0 || a.n_q_heads < 1 || a.n_kv_heads < 1 || a.head_dim < 1 || p->vocab < 0)
    return MS_ERR_INVALID_ARG;
  if (T == 0 || B == 0) return MS_OK;
  if (!p->d_pos_id || !a.q || !a.k_step || !a.v_step || !a.out) return MS_ERR_INVALID_ARG;
  if (p->vocab > 0 && (!p->d_logits || !p->d_draft || !p->d_argmax || !p->d_n_match || !p->d_n_keep ||
                       p->ld_v < p->vocab))
    return MS_ERR_INVALID_ARG;
  cudaStream_t st = ms::as_stream(stream);
  const size_t q_bytes = static_cast<size_t>(T) * a.n_q_heads * a.head_dim * 2;
  const size_t kv_bytes = static_cast<size_t>(T) * a.n_kv_heads * a.head_dim * 2;
  // ---- host -> device: the step's inputs
  if (p->h_q) MS_CUDA_TRY(cudaMemcpyAsync(const_cast<void*>(a.q), p->h_q, q_bytes, cudaMemcpyHostToDevice, st));
  if (p->h_k_step)
    MS_CUDA_TRY(cudaMemcpyAsync(const_cast<void*>(a.k_step), p->h_k_step, kv_bytes, cudaMemcpyHostToDevice, st));
  if (p->h_v_step)
    MS_CUDA_TRY(cudaMemcpyAsync(const_cast<void*>(a.v_step), p->h_v_step, kv_bytes, cudaMemcpyHostToDevice, st));
  if (p->h_pos_id)
    MS_CUDA_TRY(cudaMemcpyAsync(p->d_pos_id, p->h_pos_id, sizeof(int32_t) * T, cudaMemcpyHostToDevice, st));
  CopyLane* lane = nullptr;
  const bool side_copy = p->vocab > 0 && (p->h_logits || p->h_draft);
  if (side_copy) {
    // the logits go their own way: behind whatever `stream` holds now (the previous step's accept
    // may still read the staging buffer), beside RoPE and the attention, back in before the accept
    const int32_t rc_lane = copy_lane(&lane);
    if (rc_lane != MS_OK) return rc_lane;
    MS_CUDA_TRY(cudaEventRecord(lane->fork, st));
    MS_CUDA_TRY(cudaStreamWaitEvent(lane->stream, lane->fork, 0));
    if (p->h_logits)
      MS_CUDA_TRY(cudaMemcpyAsync(p->d_logits, p->h_logits, sizeof(float) * static_cast<size_t>(T) * p->ld_v,
                                  cudaMemcpyHostToDevice, lane->stream));
    if (p->h_draft)
      MS_CUDA_TRY(cudaMemcpyAsync(p->d_draft, p->h_draft, sizeof(int32_t) * T, cudaMemcpyHostToDevice, lane->stream));
    MS_CUDA_TRY(cudaEventRecord(lane->join, lane->stream));
  }
  // ---- the hot path
  int32_t rc = memosight_rope_qk(const_cast<void*>(a.q), const_cast<void*>(a.k_step), p->d_pos_id, T,
                                 a.n_q_heads, a.n_kv_heads, a.head_dim, p->rope_base, nullptr,
                                 p->rope_flags, stream);
  if (rc != MS_OK) return rc;
  rc = memosight_attn_step(&a, stream);
  if (rc != MS_OK) return rc;
  if (p->vocab > 0) {
    if (side_copy) MS_CUDA_TRY(cudaStreamWaitEvent(st, lane->join, 0));
    rc = memosight_accept(p->d_logits, p->ld_v, p->vocab, a.q_off, B, T, p->d_draft, p->d_argmax,
                          p->d_n_match, p->d_n_keep, p->accept_workspace, p->accept_workspace_bytes,
                          stream);
    if (rc != MS_OK) return rc;
    rc = memosight_kv_append(const_cast<void*>(a.k_cache), const_cast<void*>(a.v_cache),
                             a.kv_head_stride, a.n_slots, B, a.n_kv_heads, a.head_dim, a.kv_off,
                             const_cast<int32_t*>(a.kv_len), p->d_kv_cap, a.k_step, a.v_step, a.q_off,
                             a.n_cand, p->d_n_keep, a.max_nq, 1, nullptr, stream);
    if (rc != MS_OK) return rc;
  }
  if (p->d_seg_start) {
    if (!p->d_seg_len) return MS_ERR_INVALID_ARG;
    rc = memosight_kv_compact(const_cast<void*>(a.k_cache), const_cast<void*>(a.v_cache), 1, 0,
                              a.kv_head_stride, B, a.n_kv_heads, a.head_dim, a.kv_off,
                              const_cast<int32_t*>(a.kv_len), p->d_seg_start, p->d_seg_len, nullptr, 0,
                              p->max_tail, stream);
    if (rc != MS_OK) return rc;
  }
  // ---- device -> host: the step's results
  if (p->h_out) MS_CUDA_TRY(cudaMemcpyAsync(p->h_out, a.out, q_bytes, cudaMemcpyDeviceToHost, st));
  if (p->vocab > 0) {
    if (p->h_argmax)
      MS_CUDA_TRY(cudaMemcpyAsync(p->h_argmax, p->d_argmax, sizeof(int32_t) * T, cudaMemcpyDeviceToHost, st));
    if (p->h_n_match)
      MS_CUDA_TRY(cudaMemcpyAsync(p->h_n_match, p->d_n_match, sizeof(int32_t) * B, cudaMemcpyDeviceToHost, st));
  }
  return MS_OK;
}
