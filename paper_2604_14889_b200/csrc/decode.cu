// Device-resident bookkeeping of MemoSight's iterative inference (paper App. A, Algorithm 1):
// what the loop around the forward passes does with tokens, positions and the cache.  The
// model itself (embeddings, projections, MLPs, LM head) is the caller's; these calls build the
// metadata its forward passes need and apply the outcome of the greedy verification, all on
// the device, so a serving loop never has to bring per-sequence state to the host.
//
//   plan            Predict+Verify block of every live sequence: the pending candidates
//                   c_0..c_{n-1} (c_0 verified, the rest drafts) followed by d foresight tokens;
//                   their token ids, position IDs (Sec. 2.1.1, Sec. 2.2) and the drafts each row
//                   has to reproduce (c_{i+1}).
//   commit          after memosight_accept: c_0..c_m (m = matching prefix) become permanent, cut
//                   after the first step delimiter or end-of-sequence token among them; the
//                   model's own prediction behind the last permanent token is the next c_0; the
//                   foresight predictions are the next drafts only if every candidate was
//                   accepted (they were conditioned on all of them).
//   plan_compress   for sequences whose step just ended: the block <m>*l, <o> with l = ceil(n/c)
//                   (AMA), the memory tokens at the centres of their groups (UPL) and <o> at the
//                   step's last position + 1 (Sec. 2.1.2, Sec. 2.2), plus the eviction request.
//   commit_compress after the block was forwarded, appended and the step evicted: the next step
//                   starts behind <o>, whose prediction is its first token.
#include "common.cuh"

namespace {

constexpr int kFlagDone = 1, kFlagCompress = 2;

struct State {
  int B, d, c, max_out, max_mem;
  int tok_f, tok_m, tok_o, tok_delim, tok_eos;
  int32_t *kv_len, *pos_next, *seg_start, *seg_n, *seg_pid0, *cand, *n_cand, *flags, *out_tok, *n_out;
};

bool unpack(const memosight_decode_state* s, State* o) {
  if (!s || s->struct_size != sizeof(memosight_decode_state)) return false;
  if (s->batch < 0 || s->d < 0 || s->d > 7 || s->c < 1 || s->max_out < 1 || s->max_mem < 1 || s->max_mem > 255)
    return false;
  if (s->batch > 0 && (!s->kv_len || !s->pos_next || !s->seg_start || !s->seg_n || !s->seg_pid0 || !s->cand ||
                       !s->n_cand || !s->flags || !s->out_tok || !s->n_out))
    return false;
  o->B = s->batch; o->d = s->d; o->c = s->c; o->max_out = s->max_out; o->max_mem = s->max_mem;
  o->tok_f = s->tok_foresight; o->tok_m = s->tok_memory; o->tok_o = s->tok_output;
  o->tok_delim = s->tok_delim; o->tok_eos = s->tok_eos;
  o->kv_len = s->kv_len; o->pos_next = s->pos_next; o->seg_start = s->seg_start; o->seg_n = s->seg_n;
  o->seg_pid0 = s->seg_pid0; o->cand = s->cand; o->n_cand = s->n_cand; o->flags = s->flags;
  o->out_tok = s->out_tok; o->n_out = s->n_out;
  return true;
}

// Exclusive prefix sum of per-sequence row counts (one CTA; B <= 8192).
__device__ void block_prefix(const int* rows_of, int B, int32_t* q_off, int* s_tmp) {
  const int nt = blockDim.x, tid = threadIdx.x;
  const int per = (B + nt - 1) / nt;
  const int lo = min(B, tid * per), hi = min(B, lo + per);
  int sum = 0;
  for (int b = lo; b < hi; ++b) sum += rows_of[b];
  s_tmp[tid] = sum;
  __syncthreads();
  int base = 0;
  for (int t = 0; t < tid; ++t) base += s_tmp[t];
  for (int b = lo; b < hi; ++b) {
    q_off[b] = base;
    base += rows_of[b];
  }
  if (tid == nt - 1) q_off[B] = base;
  __syncthreads();
}

__global__ void __launch_bounds__(256)
decode_plan_kernel(State s, int32_t* __restrict__ q_off, int32_t* __restrict__ n_cand_blk,
                   int32_t* __restrict__ row_tok, int32_t* __restrict__ pos_id, int32_t* __restrict__ draft,
                   int32_t* __restrict__ summary, int* __restrict__ rows_scratch) {
  __shared__ int s_tmp[256];
  __shared__ int s_live, s_comp;
  if (threadIdx.x == 0) { s_live = 0; s_comp = 0; }
  __syncthreads();
  for (int b = threadIdx.x; b < s.B; b += blockDim.x) {
    const int f = s.flags[b];
    const bool live = !(f & kFlagDone) && !(f & kFlagCompress);
    const int n = live ? s.n_cand[b] : 0;
    rows_scratch[b] = live ? n + s.d : 0;
    n_cand_blk[b] = n;
    if (live) atomicAdd(&s_live, 1);
    if (f & kFlagCompress) atomicAdd(&s_comp, 1);
  }
  __syncthreads();
  block_prefix(rows_scratch, s.B, q_off, s_tmp);
  for (int b = threadIdx.x; b < s.B; b += blockDim.x) {
    const int rows = rows_scratch[b];
    if (rows == 0) continue;
    const int n = rows - s.d, r0 = q_off[b], p0 = s.pos_next[b];
    for (int i = 0; i < n; ++i) {
      row_tok[r0 + i] = s.cand[b * (s.d + 1) + i];
      pos_id[r0 + i] = p0 + i;
      draft[r0 + i] = (i + 1 < n) ? s.cand[b * (s.d + 1) + i + 1] : -1;
    }
    for (int k = 0; k < s.d; ++k) {       // foresight token k+1: one position further than the last candidate, each
      row_tok[r0 + n + k] = s.tok_f;
      pos_id[r0 + n + k] = p0 + n + k;    // = (p0 + n - 1) + (k + 1)
      draft[r0 + n + k] = -1;
    }
  }
  if (threadIdx.x == 0) {
    summary[0] = q_off[s.B];
    summary[1] = s_live;
    summary[2] = s_comp;
    summary[3] = 0;
  }
}

__global__ void __launch_bounds__(128)
decode_commit_kernel(State s, const int32_t* __restrict__ q_off, const int32_t* __restrict__ argmax,
                     const int32_t* __restrict__ n_match, int32_t* __restrict__ n_keep) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= s.B) return;
  const int r0 = q_off[b], rows = q_off[b + 1] - r0;
  if (rows == 0) { n_keep[b] = 0; return; }
  const int n = rows - s.d;
  int32_t* cand = s.cand + b * (s.d + 1);
  int keep = min(n_match[b], n - 1) + 1;                 // c_0 .. c_m
  int flags = s.flags[b];
  int n_out = s.n_out[b];
  // permanent tokens, cut behind the first delimiter / end-of-sequence token or at the output budget
  int kept = 0;
  for (int i = 0; i < keep; ++i) {
    const int t = cand[i];
    if (n_out < s.max_out) s.out_tok[b * s.max_out + n_out] = t;
    ++n_out;
    ++kept;
    if (t == s.tok_eos) { flags |= kFlagDone; break; }
    if (t == s.tok_delim) { flags |= kFlagCompress; break; }
    if (n_out >= s.max_out) { flags |= kFlagDone; break; }
  }
  const bool all_accepted = (kept == n);
  n_keep[b] = kept;
  s.n_out[b] = n_out;
  s.seg_n[b] += kept;
  s.pos_next[b] += kept;
  s.flags[b] = flags;
  // next block: the model's own prediction behind the last permanent token, then (only if every
  // candidate was accepted) the foresight predictions as drafts
  cand[0] = argmax[r0 + kept - 1];
  int nc = 1;
  if (all_accepted && !(flags & (kFlagDone | kFlagCompress))) {
    for (int k = 0; k < s.d; ++k) cand[1 + k] = argmax[r0 + n + k];
    nc = 1 + s.d;
  }
  s.n_cand[b] = nc;
}

__global__ void __launch_bounds__(256)
decode_plan_compress_kernel(State s, int32_t* __restrict__ q_off, int32_t* __restrict__ n_cand_blk,
                            int32_t* __restrict__ row_tok, int32_t* __restrict__ pos_id,
                            int32_t* __restrict__ n_keep, int32_t* __restrict__ seg_start_out,
                            int32_t* __restrict__ seg_len_out, int32_t* __restrict__ summary,
                            int* __restrict__ rows_scratch) {
  __shared__ int s_tmp[256];
  __shared__ int s_comp;
  if (threadIdx.x == 0) s_comp = 0;
  __syncthreads();
  for (int b = threadIdx.x; b < s.B; b += blockDim.x) {
    const bool on = (s.flags[b] & kFlagCompress) && !(s.flags[b] & kFlagDone);
    int l = 0;
    if (on) {
      l = (s.seg_n[b] + s.c - 1) / s.c;            // AMA
      l = min(l, s.max_mem);
      atomicAdd(&s_comp, 1);
    }
    rows_scratch[b] = on ? l + 1 : 0;
    n_cand_blk[b] = on ? l + 1 : 0;
    n_keep[b] = on ? l + 1 : 0;
    seg_start_out[b] = on ? s.seg_start[b] : 0;
    seg_len_out[b] = on ? s.seg_n[b] : 0;
  }
  __syncthreads();
  block_prefix(rows_scratch, s.B, q_off, s_tmp);
  for (int b = threadIdx.x; b < s.B; b += blockDim.x) {
    const int rows = rows_scratch[b];
    if (rows == 0) continue;
    const int l = rows - 1, r0 = q_off[b], n = s.seg_n[b], rho = s.seg_pid0[b];
    for (int g = 0; g < l; ++g) {                 // UPL: centre of group g, rounded down
      const int first = g * s.c;
      const int last = min(first + s.c, n) - 1;
      row_tok[r0 + g] = s.tok_m;
      pos_id[r0 + g] = rho + ((first + last) >> 1);
    }
    row_tok[r0 + l] = s.tok_o;
    pos_id[r0 + l] = rho + n;                     // last position of the step + 1
  }
  if (threadIdx.x == 0) {
    summary[0] = q_off[s.B];
    summary[1] = 0;
    summary[2] = s_comp;
    summary[3] = 0;
  }
}

__global__ void __launch_bounds__(128)
decode_commit_compress_kernel(State s, const int32_t* __restrict__ q_off, const int32_t* __restrict__ argmax) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= s.B) return;
  const int r0 = q_off[b], rows = q_off[b + 1] - r0;
  if (rows == 0) return;
  const int n = s.seg_n[b], rho = s.seg_pid0[b];
  s.cand[b * (s.d + 1)] = argmax[r0 + rows - 1];   // <o>'s prediction opens the next step
  s.n_cand[b] = 1;
  s.pos_next[b] = rho + n + 1;                     // behind <o>
  s.seg_pid0[b] = rho + n + 1;
  s.seg_start[b] = s.kv_len[b];                    // the cache now ends with the memory tokens and <o>
  s.seg_n[b] = 0;
  s.flags[b] &= ~kFlagCompress;
}

}  // namespace

extern "C" size_t memosight_decode_scratch_bytes(int32_t batch) {
  return batch < 0 ? 0 : (static_cast<size_t>(batch) + 64) * sizeof(int32_t);
}

extern "C" int32_t memosight_decode_plan(const memosight_decode_state* st, int32_t* q_off, int32_t* n_cand_blk,
                                         int32_t* row_tok, int32_t* pos_id, int32_t* draft, int32_t* summary,
                                         void* scratch, memosight_stream_t stream) {
  State s;
  if (!unpack(st, &s)) return MS_ERR_INVALID_ARG;
  if (s.B > ms::kMaxBatch) return MS_ERR_UNSUPPORTED_SHAPE;
  if (!q_off || !summary) return MS_ERR_INVALID_ARG;
  if (s.B > 0 && (!n_cand_blk || !row_tok || !pos_id || !draft || !scratch)) return MS_ERR_INVALID_ARG;
  decode_plan_kernel<<<1, 256, 0, ms::as_stream(stream)>>>(s, q_off, n_cand_blk, row_tok, pos_id, draft, summary,
                                                           static_cast<int*>(scratch));
  MS_LAUNCH_CHECK();
  return MS_OK;
}

extern "C" int32_t memosight_decode_commit(const memosight_decode_state* st, const int32_t* q_off,
                                           const int32_t* argmax, const int32_t* n_match, int32_t* n_keep,
                                           memosight_stream_t stream) {
  State s;
  if (!unpack(st, &s)) return MS_ERR_INVALID_ARG;
  if (s.B == 0) return MS_OK;
  if (!q_off || !argmax || !n_match || !n_keep) return MS_ERR_INVALID_ARG;
  decode_commit_kernel<<<(s.B + 127) / 128, 128, 0, ms::as_stream(stream)>>>(s, q_off, argmax, n_match, n_keep);
  MS_LAUNCH_CHECK();
  return MS_OK;
}

extern "C" int32_t memosight_decode_plan_compress(const memosight_decode_state* st, int32_t* q_off,
                                                  int32_t* n_cand_blk, int32_t* row_tok, int32_t* pos_id,
                                                  int32_t* n_keep, int32_t* seg_start, int32_t* seg_len,
                                                  int32_t* summary, void* scratch, memosight_stream_t stream) {
  State s;
  if (!unpack(st, &s)) return MS_ERR_INVALID_ARG;
  if (s.B > ms::kMaxBatch) return MS_ERR_UNSUPPORTED_SHAPE;
  if (!q_off || !summary) return MS_ERR_INVALID_ARG;
  if (s.B > 0 && (!n_cand_blk || !row_tok || !pos_id || !n_keep || !seg_start || !seg_len || !scratch))
    return MS_ERR_INVALID_ARG;
  decode_plan_compress_kernel<<<1, 256, 0, ms::as_stream(stream)>>>(s, q_off, n_cand_blk, row_tok, pos_id, n_keep,
                                                                    seg_start, seg_len, summary,
                                                                    static_cast<int*>(scratch));
  MS_LAUNCH_CHECK();
  return MS_OK;
}

extern "C" int32_t memosight_decode_commit_compress(const memosight_decode_state* st, const int32_t* q_off,
                                                    const int32_t* argmax, memosight_stream_t stream) {
  State s;
  if (!unpack(st, &s)) return MS_ERR_INVALID_ARG;
  if (s.B == 0) return MS_OK;
  if (!q_off || !argmax) return MS_ERR_INVALID_ARG;
  decode_commit_compress_kernel<<<(s.B + 127) / 128, 128, 0, ms::as_stream(stream)>>>(s, q_off, argmax);
  MS_LAUNCH_CHECK();
  return MS_OK;
}
