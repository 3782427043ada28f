// Internal interface between the attention entry point and its kernels.
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace ms {

// Validated, typed copy of memosight_attn_params as the kernels take it.
struct AttnArgs {
  int B, H_q, H_kv, G, D, T;
  const __nv_bfloat16* k_cache;
  const __nv_bfloat16* v_cache;
  int64_t kv_head_stride;
  int64_t n_slots;
  const int64_t* kv_off;
  const int32_t* kv_len;
  const int32_t* q_off;
  const int32_t* n_cand;
  const int32_t* anchor;
  const uint8_t* tok_kind;    // training-time mask metadata, or NULL
  const int32_t* tok_step;
  const __nv_bfloat16* q;
  const __nv_bfloat16* k_step;
  const __nv_bfloat16* v_step;
  __nv_bfloat16* out;
  float* lse;
  float scale_log2;   // softmax scale * log2(e): scores live in the exp2 domain
  int max_kv_len, max_nq;
  void* workspace;
  // Stacked layers (keys-on-lanes kernel): layer l reads the cache at k_cache + l * kv_layer_stride
  // and the step tensors / writes the results at their pointer + l * the tensor's layer stride
  // (all in elements).  n_layers == 1 everywhere else.
  int n_layers;
  int64_t kv_layer_stride, q_layer_stride, kstep_layer_stride, out_layer_stride, lse_layer_stride;
  // Counters of the in-kernel merge (two per persistent CTA, zero between launches), or NULL:
  // the merge is then a launch of its own.
  unsigned int* done;
  unsigned int wait_limit_us;   // limit of one bounded device-side wait
  cudaEvent_t ev_split_begin, ev_split_end;   // optional timing events around the split kernel
};

// Workspace header (first 256 bytes): word 0 = device status -- a magic value when a
// bounded wait ran out, anything else means ok (the workspace need not be cleared).
constexpr size_t kWsHeaderBytes = 256;

int32_t launch_attn_simt(const AttnArgs& a, cudaStream_t st);

// Tensor-core split-KV path.  rows_pad = packed rows per KV head rounded up to 16.
size_t attn_mma_workspace_bytes(int D, int rows_pad, int n_ctas);
int32_t launch_attn_mma(const AttnArgs& a, cudaStream_t st);
int attn_mma_grid();   // persistent CTAs the split kernel launches on this device

// tcgen05 split-KV path (operands from shared memory, accumulators in tensor memory):
// up to 128 packed rows per KV head; same workspace layout and merge as the path above.
bool attn_umma_supports(int D, int G, int max_nq);
int32_t launch_attn_umma(const AttnArgs& a, cudaStream_t st);

// tcgen05 path with the tile's keys on the tensor-memory lanes (the transposed products):
// blocks of up to 64 packed rows, head_dim 128.
bool attn_umma_t_supports(int D, int G, int max_nq);
int32_t launch_attn_umma_t(const AttnArgs& a, cudaStream_t st);

// tcgen05 path for large blocks (17..256 tokens per block, head_dim 128): the block is cut
// into row tiles; own schedule, workspace size and merge kernel.
bool attn_umma_big_supports(int D, int G, int max_nq);   // the only tensor-core kernel that takes tok_kind/tok_step
size_t attn_umma_big_workspace_bytes(int B, int H_kv, int G, int max_nq, int max_kv_len, int n_ctas);
int32_t launch_attn_umma_big(const AttnArgs& a, cudaStream_t st);

}  // namespace ms
