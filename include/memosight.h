/*
 * memosight.h -- C ABI of the MemoSight per-step attention hot path (B200, sm_100a).
 *
 * MemoSight inference alternates two things (paper Sec. 2.1, Algorithm 1):
 *   - Predict+Verify steps: a small block of new tokens -- the pending candidate
 *     tokens, causal among themselves, followed by d foresight tokens that see
 *     the prefix and themselves only -- runs one forward pass against the KV
 *     cache; the greedy rule accepts the longest draft prefix that equals the
 *     model's own argmax; accepted tokens are appended to the cache;
 *   - compression: when a reasoning step ends, ceil(n/c) memory tokens and one
 *     output token are appended behind it and the step's n verbose entries are
 *     evicted from the KV cache, which therefore stays compacted.
 * This library implements the attention-side work of that loop, one call per
 * operation, as CUDA kernels.  There is no CPU fallback: every call other than
 * the host-only layout helpers fails with MS_ERR_CUDA when no device is usable.
 *
 * Conventions that hold for every call unless its comment says otherwise:
 *   - "device" pointers are device memory owned by the caller, valid until the
 *     work queued on `stream` has finished; "host" pointers are ordinary host
 *     memory read or written before the call returns.
 *   - bf16 tensors are raw 16-bit patterns (the upper half of an IEEE binary32);
 *     base pointers of bf16 tensors must be 16-byte aligned.
 *   - calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL is
 *     the default stream), never synchronise, never allocate device memory and
 *     never read device scalars on the host: ragged lengths stay on the device
 *     and the caller supplies host-side upper bounds for launch sizing.
 *   - the kernels are launched with programmatic stream serialisation: each may
 *     begin its set-up while the kernel before it in the stream drains, and waits
 *     for that kernel before it touches global memory, so stream order holds as usual.
 *   - the first call of an entry point on a device sets that device up for it
 *     (function attributes, symbol addresses): make it outside any stream capture.
 *   - return value: MS_OK or a negative MS_ERR_* code.  Arguments are validated
 *     on the host before anything is launched; a rejected call has no effect.
 *     Device code never traps; the only device-side failure (a bounded wait that
 *     ran out) is recorded in the workspace and read by memosight_attn_status().
 *   - GQA: query head h reads KV head h / (n_q_heads / n_kv_heads).
 */
#ifndef MEMOSIGHT_H_
#define MEMOSIGHT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MS_OK 0
#define MS_ERR_INVALID_ARG (-1)         /* null pointer, negative size, inconsistent sizes        */
#define MS_ERR_UNSUPPORTED_SHAPE (-2)   /* a size outside the documented limits                   */
#define MS_ERR_WORKSPACE_TOO_SMALL (-3) /* workspace_bytes below the *_workspace_bytes() answer   */
#define MS_ERR_ALIGNMENT (-4)           /* a pointer or stride breaks the 16-byte rule            */
#define MS_ERR_CUDA (-5)                /* a CUDA runtime/driver call failed; see last_cuda_error */
#define MS_ERR_DEVICE_TIMEOUT (-6)      /* a bounded device-side wait ran out (attn_status only)  */

typedef void* memosight_stream_t; /* a cudaStream_t */

#if defined(__GNUC__)
#define MS_API __attribute__((visibility("default")))
#else
#define MS_API
#endif

/* RoPE flags */
#define MS_ROPE_NEOX 0u          /* pair (i, i + D/2): rotate-half, the default                  */
#define MS_ROPE_INTERLEAVED 1u   /* pair (2i, 2i+1)                                              */
#define MS_POS_HALF_UNITS 2u     /* pos_id counts half positions (exact UPL centres)             */
/* Layout flag of memosight_upl_pids: the "w/o UPL" ablation of App. B.3 */
#define MS_LAYOUT_MONOTONE 4u    /* memory tokens take fresh, monotonically increasing PIDs behind
                                    the step (rho_first + n + g) instead of the group centres    */

/* Library version (major*10000 + minor*100 + patch). */
MS_API int32_t memosight_version(void);
/* Static, NUL-terminated description of a status code. */
MS_API const char* memosight_status_string(int32_t status);
/* The cudaError_t (as int) behind the most recent MS_ERR_CUDA of this thread, 0 if none. */
MS_API int32_t memosight_last_cuda_error(void);

/* ---- Position layout (host-only integer helpers; Sec. 2.1.2, Sec. 2.2) ------------------- */

/* Adaptive Memory Allocation: number of memory tokens for a step of n tokens at
 * compression ratio c, l = ceil(n / c).  n >= 0, c >= 1, else MS_ERR_INVALID_ARG. */
MS_API int32_t memosight_ama(int32_t n, int32_t c);

/* Uniform Position Layout: the step's n tokens hold PIDs rho_first .. rho_first+n-1
 * and are cut into l = ceil(n/c) sequential groups of c (last may be shorter);
 * memory token g gets the centre PID of group g.  A half-integer centre (even
 * group size) is rounded down, or returned exactly in half positions when flags
 * has MS_POS_HALF_UNITS (value = 2*centre).  With MS_LAYOUT_MONOTONE the groups are ignored
 * and memory token g gets rho_first + n + g.  pid_out: host, capacity cap >= l.
 * Returns l, or a negative code (MS_ERR_INVALID_ARG also when cap < l). */
MS_API int32_t memosight_upl_pids(int32_t rho_first, int32_t n, int32_t c, uint32_t flags,
                           int32_t* pid_out, int32_t cap);

/* The "w/o AMA" ablation of App. B.3: a fixed budget of l memory tokens per step whatever its
 * length n >= 1.  The step is cut into l groups as evenly as possible (group g = offsets
 * floor(g*n/l) .. floor((g+1)*n/l)-1) and memory token g takes its group's centre, rounded
 * down; a group left empty (n < l) takes the position it would start at, clamped into the
 * step.  (The paper fixes only the budget, 9; the placement is this library's reading.)
 * pid_out: host, capacity cap >= l.  Returns l or a negative code. */
MS_API int32_t memosight_budget_pids(int32_t rho_first, int32_t n, int32_t l, int32_t* pid_out, int32_t cap);

/* PID of the output token <o> that closes a step: the step's last PID plus one. */
MS_API int32_t memosight_out_pid(int32_t rho_first, int32_t n);

/* PIDs of one step block (Sec. 2.1.1; Sec. 2.2, foresight tokens): rows 0..n_c-1
 * are the candidates (p0, p0+1, ...); row n_c+k-1 is foresight token f_k, which
 * takes the PID just before its prediction target: (PID of the last regular
 * token it sees) + k.  anchor (host, [d] or NULL): how many candidates f_k sees;
 * NULL means all n_c.  pid_out: host [n_c + d].  Returns MS_OK or a code. */
MS_API int32_t memosight_step_pids(int32_t p0, int32_t n_c, int32_t d, const int32_t* anchor,
                            int32_t* pid_out);

/* ---- RoPE at token-specific position IDs (Sec. 2.1.2, UPL paragraph) --------------------- */

/* Rotates, in place, every head vector of the T new tokens by the token's own PID.
 *   q       device bf16 [T][H_q][D]   (may be NULL when H_q == 0)
 *   k       device bf16 [T][H_kv][D]  (may be NULL when H_kv == 0)
 *   pos_id  device int32 [T]
 *   inv_freq host double [D/2] or NULL; NULL means theta_i = rope_base^(-2i/D)
 * The result of every element is the fp64 rotation (fp64 angle, fp64 sine and cosine) rounded
 * to bf16 once; the kernel computes it in fp32 wherever that provably gives the same bits and in
 * fp64 for the few elements next to a rounding boundary.
 * D even, 2 <= D <= 256.  T == 0 is a no-op. */
MS_API int32_t memosight_rope_qk(void* q, void* k, const int32_t* pos_id, int32_t T, int32_t H_q,
                          int32_t H_kv, int32_t D, double rope_base, const double* inv_freq,
                          uint32_t flags, memosight_stream_t stream);

/* ---- Step attention (Sec. 2.1.1 masks; Sec. 2.3 "Attention Mask Strategy") --------------- */

/* One layer of attention of all sequences' step blocks against the compacted cache.
 * Visibility: every one of the kv_len[b] cache entries is visible to every row of
 * block b (the verbose steps were evicted; prompt, memory, output tokens and the
 * current step's accepted tokens remain).  Among the block's own n_q keys, key j
 * is visible to row i iff j == i, or j is a candidate (j < n_cand[b]) and
 * j < a_i, where a_i = i for a candidate row (causal) and a_i = anchor[row]
 * (default n_cand[b]) for a foresight row.  Foresight keys are visible to no
 * other row.  The mask is evaluated from this metadata; no matrix is built. */
typedef struct memosight_attn_params {
  uint32_t struct_size;      /* sizeof(memosight_attn_params), for ABI growth                 */
  int32_t batch;             /* B >= 0                                                         */
  int32_t n_q_heads;         /* H_q, multiple of n_kv_heads                                    */
  int32_t n_kv_heads;        /* H_kv                                                           */
  int32_t head_dim;          /* D: 64 or 128 on the tensor-core paths; any multiple of 32 up to
                                256 on the general path                                        */
  const void* k_cache;       /* device bf16, one layer: [H_kv][n_slots][D], post-RoPE          */
  const void* v_cache;       /* device bf16, same layout                                       */
  int64_t kv_head_stride;    /* elements between KV heads (>= n_slots*D, multiple of 8)        */
  int64_t n_slots;           /* slots per KV head (< 2^31)                                     */
  const int64_t* kv_off;     /* device [B]: first slot of sequence b                           */
  const int32_t* kv_len;     /* device [B]: valid entries L_b (kv_off[b]+L_b <= n_slots)       */
  int32_t max_kv_len;        /* host upper bound of kv_len[]                                   */
  int32_t max_nq;            /* host upper bound of the block sizes, 1..32768                  */
  const int32_t* q_off;      /* device [B+1]: rows of block b are q_off[b] .. q_off[b+1]-1     */
  const int32_t* n_cand;     /* device [B]: candidates in block b (the block's first rows)     */
  const int32_t* anchor;     /* device [T] or NULL; read only for foresight rows               */
  int32_t total_rows;        /* T = q_off[B] (host copy)                                       */
  float sm_scale;            /* softmax scale; 0 means 1/sqrt(D)                               */
  const void* q;             /* device bf16 [T][H_q][D], post-RoPE                             */
  const void* k_step;        /* device bf16 [T][H_kv][D], post-RoPE                            */
  const void* v_step;        /* device bf16 [T][H_kv][D]                                       */
  void* out;                 /* device bf16 [T][H_q][D]                                        */
  float* lse;                /* device fp32 [T][H_q], natural-log sum-exp, or NULL             */
  void* workspace;           /* device scratch, 256-byte aligned                               */
  size_t workspace_bytes;    /* >= memosight_attn_workspace_bytes(...)                         */
  /* Optional training-time mask (Sec. 2.3 "Attention Mask Strategy"), both or neither.  The block
   * is then an augmented sequence (Sec. 2.2) whose tokens carry a kind and a reasoning-step index;
   * among the block's own keys, key j is visible to row i iff j == i, or j < i and j is neither a
   * foresight token nor a reasoning token of another step.  n_cand and anchor are ignored.  A
   * structure that ends before these fields (an older struct_size) means "not given". */
  const uint8_t* tok_kind;   /* device [T]: MS_KIND_*                                          */
  const int32_t* tok_step;   /* device [T]: index of the token's reasoning step (prompt: any)  */
} memosight_attn_params;

#define MS_KIND_PROMPT 0
#define MS_KIND_REASON 1      /* a verbose reasoning token: visible inside its own step only    */
#define MS_KIND_FORESIGHT 2   /* visible to itself only                                          */
#define MS_KIND_MEMORY 3
#define MS_KIND_OUTPUT 4

/* Scratch size for memosight_attn_step with these bounds (0 on invalid input). */
MS_API size_t memosight_attn_workspace_bytes(int32_t batch, int32_t n_q_heads, int32_t n_kv_heads,
                                      int32_t head_dim, int32_t max_kv_len, int32_t max_nq);

/* Queues the attention of one layer (split-KV pass + log-sum-exp merge).
 * Limits: n_q_heads/n_kv_heads <= 16; max_nq <= 32768; batch <= 8192 per call.
 * Step blocks (max_nq <= 16) with max_nq * (H_q/H_kv) <= 128 and D in {64,128} take a
 * tensor-core kernel (see memosight_attn_set_path).  Larger blocks -- the compression pass
 * forwards the ceil(n/c) memory tokens and <o> of a finished step as one causal block
 * (Sec. 2.1.2, Algorithm 1), and the prefill of a prompt is one causal block against an empty
 * or partly filled cache (Algorithm 1, Prefill) -- take the large-block tcgen05 kernel when D
 * is 128; so do blocks with the training-time mask (tok_kind / tok_step) when max_nq > 16.
 * Anything else inside the limits takes the slower general kernel.  Size the workspace with the very
 * batch, head counts, max_kv_len and max_nq of the call: a large-block call needs a different
 * amount than a step-block call.
 * The workspace may be reused by the next call on the same stream; two calls
 * that overlap on the GPU need two workspaces. */
MS_API int32_t memosight_attn_step(const memosight_attn_params* params, memosight_stream_t stream);

/* The same attention for n_layers stacked layers that share the step's metadata (lengths, block
 * offsets, candidates, anchors): Algorithm 1 forwards the whole model per step and keeps one
 * cache per layer, all of the same length.  Layer l reads the cache at k_cache / v_cache +
 * l * kv_layer_stride, the step tensors at q + l * q_layer_stride and k_step / v_step +
 * l * kstep_layer_stride, and writes out + l * out_layer_stride (lse + l * lse_layer_stride);
 * strides in elements, multiples of 8, each at least the size of one layer's tensor.  Step blocks
 * of head_dim 128 with up to 64 packed rows run all layers in ONE launch of the keys-on-lanes
 * kernel (the tile list is simply layer-major; tile prefix, workspace and tensor maps are shared);
 * other shapes are issued layer by layer.  The workspace is the one memosight_attn_workspace_bytes
 * gives for a single layer.  (A model that needs layer l's output before it can form layer l+1's
 * queries calls memosight_attn_step per layer; this entry serves callers that hold every layer's
 * q / k / v at once, and measures the stacked-layer step.) */
typedef struct memosight_attn_layers {
  uint32_t struct_size;        /* sizeof(memosight_attn_layers)                               */
  int32_t n_layers;            /* >= 0; 1 behaves like memosight_attn_step                    */
  int64_t kv_layer_stride;     /* elements between consecutive layers of k_cache / v_cache    */
  int64_t q_layer_stride;      /* ... of q                                                    */
  int64_t kstep_layer_stride;  /* ... of k_step and of v_step                                 */
  int64_t out_layer_stride;    /* ... of out                                                  */
  int64_t lse_layer_stride;    /* ... of lse (ignored when lse is NULL)                       */
} memosight_attn_layers;
MS_API int32_t memosight_attn_step_layers(const memosight_attn_params* params,
                                          const memosight_attn_layers* layers, memosight_stream_t stream);

/* Diagnostic switch: which kernel memosight_attn_step uses from now on, process-wide.
 * MS_ATTN_PATH_AUTO (the default) picks by shape: head_dim 128 with up to 64 packed rows
 * (max_nq * H_q/H_kv) takes the keys-on-lanes tcgen05 kernel, more rows or blocks of more than
 * 16 tokens the row-tiled large-block kernel; head_dim 64 the mma.sync kernel (up to 64 rows)
 * or the rows-on-lanes tcgen05 kernel (up to 128); anything else the general kernel.  A forced
 * path is used only for calls whose shape it covers AND whose workspace is large enough for it
 * (a path may need more than memosight_attn_workspace_bytes answers for the automatic choice);
 * any other call falls back to the automatic choice.  Returns the previous setting, or
 * MS_ERR_INVALID_ARG.  Results of all paths agree within the tolerance of bf16 inputs with fp32
 * accumulation; the switch exists for tests and timing. */
#define MS_ATTN_PATH_AUTO 0
#define MS_ATTN_PATH_MMA_SYNC 1
#define MS_ATTN_PATH_TCGEN05 2
#define MS_ATTN_PATH_GENERAL 3
#define MS_ATTN_PATH_TCGEN05_KEYS 4   /* tcgen05 with the keys on the accumulator lanes; <= 64 rows, D 128 */
#define MS_ATTN_PATH_LARGE_BLOCK 5    /* the row-tiled tcgen05 kernel of large blocks, for any block size; D 128 */
MS_API int32_t memosight_attn_set_path(int32_t path);

/* Diagnostic: from now on the attention calls of THIS thread record the two cudaEvent_t (passed
 * as void*) on their stream right before and right after the split-KV kernel, so that a
 * benchmark can time that kernel alone; (NULL, NULL) switches it off again.  Event records
 * between the kernels keep a call from overlapping its launches, so leave it off otherwise. */
MS_API int32_t memosight_attn_debug_events(void* ev_split_begin, void* ev_split_end);

/* Synchronises `stream` and returns MS_OK, or MS_ERR_DEVICE_TIMEOUT if a kernel
 * of the last memosight_attn_step on this workspace gave up on a bounded wait
 * (its output is then undefined).  Meant for tests and debugging. */
MS_API int32_t memosight_attn_status(const void* workspace, memosight_stream_t stream);

/* Diagnostics of the bounded waits.  Every wait inside the kernels (on an mbarrier that a bulk
 * copy or a tensor-core operation completes) gives up after a limit, 4 s by default; the kernel
 * then records it, drains what it has in flight and returns (see memosight_attn_status).
 * memosight_debug_set_wait_limit_us changes that limit for the launches that follow,
 * process-wide, and returns the previous one (0 only queries).  memosight_debug_wait_timeout
 * queues a one-warp kernel that waits, with a limit of limit_us (at most one second), on a
 * barrier at which nobody arrives: the wait runs out, the kernel returns, and
 * memosight_attn_status(workspace) then reports MS_ERR_DEVICE_TIMEOUT once -- the whole failure
 * path exercised without anything failing.  workspace: device, 256-byte aligned, >= 256 bytes. */
MS_API uint32_t memosight_debug_set_wait_limit_us(uint32_t limit_us);
/* Several calls finish their work in the tail of their main kernel (the merge of cut attention
 * units, pass 2 of the accept, the new lengths of append / compaction / keep-list eviction): the
 * block that finishes last does it, which it learns from a counter in a fixed array inside the
 * library (128 banks of counters, handed out per buffer address; 1 MB on every GPU that loads the
 * library).  A call that gets no bank uses its two-launch form instead, with the same result.
 * memosight_debug_set_bank_limit caps the number of banks handed out from now on (0: every call
 * takes the two-launch form; buffers that already own a bank below the cap keep it) and returns
 * the previous cap; a negative value only queries.  For tests of the two-launch forms. */
MS_API int32_t memosight_debug_set_bank_limit(int32_t n_banks);
MS_API int32_t memosight_debug_wait_timeout(void* workspace, uint32_t limit_us, memosight_stream_t stream);

/* ---- KV compaction and append (Sec. 2.1.2; Algorithm 1: UpdateCache, S <- S (+) A) ------- */

/* Evicts one verbose step per sequence from every layer's K and V cache, in place:
 * entries seg_start[b] .. seg_start[b]+seg_len[b]-1 are dropped and everything
 * behind them (the memory tokens and <o> appended after the step, and anything
 * later) moves up, order and bits preserved:  new = old[0:s) ++ old[s+n:L).
 *   k_cache, v_cache  device bf16 [n_layers][H_kv][n_slots][D]; layer_stride and
 *                     kv_head_stride in elements (multiples of 8)
 *   kv_off            device int64 [B]
 *   kv_len            device int32 [B], in/out: becomes L - n
 *   seg_start,seg_len device int32 [B]; seg_len[b] == 0 skips sequence b; a segment
 *                     that does not fit in [0, L) is ignored (sequence untouched)
 *   src_idx           device int32 [B][idx_stride] or NULL: old index of each new
 *                     entry (first L-n values of row b are written)
 *   max_tail          host upper bound of L - s - n (entries that move)
 * D*2 bytes must be a multiple of 16. */
MS_API int32_t memosight_kv_compact(void* k_cache, void* v_cache, int32_t n_layers, int64_t layer_stride,
                             int64_t kv_head_stride, int32_t batch, int32_t n_kv_heads,
                             int32_t head_dim, const int64_t* kv_off, int32_t* kv_len,
                             const int32_t* seg_start, const int32_t* seg_len, int32_t* src_idx,
                             int32_t idx_stride, int32_t max_tail, memosight_stream_t stream);

/* Eviction by an arbitrary keep list, in place, every layer, K and V:
 *     new = [old[keep_idx[b][0]], old[keep_idx[b][1]], ...],  kv_len[b] = n_keep[b].
 * MemoSight's own eviction is the special case "everything but the finished step"
 * (memosight_kv_compact, which also emits that list); the eviction policies the paper compares
 * with (heavy-hitter and separator-based, Sec. 4) keep other subsets through the same operation.
 *   keep_idx  device int32 [B][idx_stride]: strictly increasing old indices, all < kv_len[b]
 *   n_keep    device int32 [B], 0 <= n_keep[b] <= min(kv_len[b], idx_stride)
 *   max_keep  host upper bound of n_keep[]
 * A row whose list is not strictly increasing or leaves [0, kv_len) is undefined behaviour
 * within the sequence's own slots (nothing outside them is read or written).  Other arguments
 * as for memosight_kv_compact. */
MS_API int32_t memosight_kv_gather(void* k_cache, void* v_cache, int32_t n_layers, int64_t layer_stride,
                            int64_t kv_head_stride, int32_t batch, int32_t n_kv_heads, int32_t head_dim,
                            const int64_t* kv_off, int32_t* kv_len, const int32_t* keep_idx,
                            int32_t idx_stride, const int32_t* n_keep, int32_t max_keep,
                            memosight_stream_t stream);

/* Appends the accepted candidates of each block to one layer's cache: the first
 * n_keep[b] rows of block b in k_step/v_step go to slots kv_len[b] .. of sequence
 * b.  n_keep[b] is clamped to [0, n_cand[b]]: a foresight row is never cached
 * (no later token may attend to it, Sec. 2.3).  It is clamped to the room the sequence has,
 * too: to kv_cap[b] - kv_len[b] when kv_cap is given, and always to the end of the cache tensor
 * (n_slots - kv_off[b] - kv_len[b]), so an append never writes into another sequence's slots or
 * behind the tensor; when room, not the request, decided, *overflow is set to 1 (the caller
 * clears it).  kv_len[b] += (what was appended) iff bump_len != 0 (pass it on the last layer; the
 * clamps depend on kv_len, so every layer of a step appends the same rows).
 *   k_cache, v_cache device bf16 [H_kv][n_slots][D]; k_step, v_step device bf16 [T][H_kv][D]
 *   kv_cap   device int32 [B] or NULL: most entries sequence b may hold
 *   overflow device int32 [1] or NULL
 *   max_nq   host bound of the block sizes */
MS_API int32_t memosight_kv_append(void* k_cache, void* v_cache, int64_t kv_head_stride, int64_t n_slots,
                            int32_t batch, int32_t n_kv_heads, int32_t head_dim, const int64_t* kv_off,
                            int32_t* kv_len, const int32_t* kv_cap, const void* k_step, const void* v_step,
                            const int32_t* q_off, const int32_t* n_cand, const int32_t* n_keep,
                            int32_t max_nq, int32_t bump_len, int32_t* overflow, memosight_stream_t stream);

/* ---- Greedy accept (Sec. 2.1.1 and its footnote) ----------------------------------------- */

/* Scratch size for memosight_accept (0 on invalid input). */
MS_API size_t memosight_accept_workspace_bytes(int32_t total_rows, int32_t vocab);

/* Row argmax of fp32 logits and, per sequence, the length of the longest draft
 * prefix that equals the argmax row by row.
 *   logits     device fp32 [T][ld_v] (ld_v >= V; 16-byte aligned rows read faster)
 *   row_off    device int32 [B+1]; rows of sequence b: row_off[b] .. row_off[b+1]-1
 *   draft      device int32 [T]: the token row r's prediction must equal, or -1
 *              where nothing is to be verified (last candidate row, foresight rows)
 *   argmax_out device int32 [T]: lowest index of the row maximum; a NaN counts as
 *              larger than any number and the first NaN wins
 *   n_match    device int32 [B]: largest m with draft >= 0 and argmax == draft on
 *              the block's rows 0..m-1
 *   n_keep     device int32 [B] or NULL: n_match + 1 (0 for an empty block), the
 *              number of candidates that become permanent -- what kv_append takes
 * Row convention: row i of a block holds candidate c_i and predicts the token
 * after it, so draft[i] = c_{i+1}; tokens c_0..c_{n_match} become permanent and
 * argmax_out[row n_match] is the next token.
 * Every wait inside the kernels is bounded; should one ever run out (a device
 * fault), the rows concerned get argmax_out = -1, which matches no draft. */
MS_API int32_t memosight_accept(const float* logits, int64_t ld_v, int32_t vocab, const int32_t* row_off,
                         int32_t batch, int32_t total_rows, const int32_t* draft,
                         int32_t* argmax_out, int32_t* n_match, int32_t* n_keep, void* workspace,
                         size_t workspace_bytes, memosight_stream_t stream);

/* Same result as memosight_accept, for callers that cannot allocate.  (The paper has no
 * counterpart to this call; it exists for deployment reasons only.)
 *
 * Who needs it: a serving loop whose device memory was carved up at start-up and whose allocator
 * is frozen while requests are in flight, a plug-in that receives tensors but no allocator, or
 * any place where a cudaMalloc would stall the device in the middle of a decode step.  Such a
 * caller has no workspace to hand over, so the per-chunk candidates of the argmax live in a fixed
 * 512 KB array that is part of the library image: every GPU that loads the library holds it until
 * the process exits.  The call itself allocates nothing -- no cudaMalloc/cudaFree, no allocating
 * library routine -- and takes the same inputs and outputs as memosight_accept, minus the
 * workspace.
 *
 * Limit: total_rows * ceil(vocab / 8192) <= MS_ACCEPT_STATIC_MAX_PARTIALS, e.g. 3449 rows at a
 * vocabulary of 151 936.  Larger problems return MS_ERR_UNSUPPORTED_SHAPE and launch nothing;
 * use memosight_accept with a caller workspace for those.
 *
 * First call on a device: the array's device address is looked up (cudaGetSymbolAddress, with
 * that device current) and remembered; make this first call outside any stream capture.
 *
 * Sharing: all calls on a device use the one array, which keeps whatever the previous call left.
 * That is harmless for sequential calls (every entry that is read is written first by the same
 * call; nothing relies on zeros), but two calls whose kernels overlap on the GPU -- different
 * streams, or graphs replayed concurrently -- race on it and both results are then undefined. */
#define MS_ACCEPT_STATIC_MAX_PARTIALS 65536
MS_API int32_t memosight_accept_static(const float* logits, int64_t ld_v, int32_t vocab,
                                       const int32_t* row_off, int32_t batch, int32_t total_rows,
                                       const int32_t* draft, int32_t* argmax_out, int32_t* n_match,
                                       int32_t* n_keep, memosight_stream_t stream);

/* ---- Bookkeeping of the iterative inference loop (App. A, Algorithm 1) --------------------- */

/* Per-sequence decoding state, all of it in device memory owned by the caller.  The calls
 * below only read and update it with kernels on `stream`; nothing is copied to the host.
 * A sequence starts with cand[b][0] = its first token (verified by the prefill), n_cand = 1,
 * pos_next = that token's position ID, seg_start = kv_len (the reasoning step starts behind
 * the prompt), seg_n = 0, seg_pid0 = pos_next, flags = 0, n_out = 0. */
typedef struct memosight_decode_state {
  uint32_t struct_size;   /* sizeof(memosight_decode_state)                                     */
  int32_t batch;          /* B                                                                   */
  int32_t d;              /* foresight tokens per block, 0..7 (a block has at most 2d+1 rows)    */
  int32_t c;              /* compression ratio of AMA: l = ceil(n / c)                           */
  int32_t max_out;        /* capacity of out_tok per sequence; reaching it ends the sequence     */
  int32_t max_mem;        /* upper bound of l, 1..255 (longer steps get max_mem memory tokens)   */
  int32_t tok_foresight, tok_memory, tok_output;   /* ids of <f>, <m>, <o>                       */
  int32_t tok_delim, tok_eos;                      /* step delimiter (<e>) and end of sequence   */
  int32_t* kv_len;        /* [B] cache lengths: the array the cache calls update                 */
  int32_t* pos_next;      /* [B] position ID of cand[b][0]                                       */
  int32_t* seg_start;     /* [B] cache index of the current reasoning step's first entry         */
  int32_t* seg_n;         /* [B] entries of the current step in the cache so far                 */
  int32_t* seg_pid0;      /* [B] position ID of the current step's first token                   */
  int32_t* cand;          /* [B][d+1] pending candidates: c_0 verified, the others are drafts    */
  int32_t* n_cand;        /* [B] 1..d+1                                                          */
  int32_t* flags;         /* [B] bit 0: finished; bit 1: step ended, compression pending         */
  int32_t* out_tok;       /* [B][max_out] the permanent tokens in order                          */
  int32_t* n_out;         /* [B] tokens made permanent so far (may exceed max_out by the last block) */
} memosight_decode_state;

/* Device scratch needed by the two plan calls. */
MS_API size_t memosight_decode_scratch_bytes(int32_t batch);

/* Builds the Predict+Verify block of every live sequence (not finished, no compression
 * pending): rows c_0..c_{n-1} then d foresight tokens (Sec. 2.1.1).
 *   q_off [B+1], n_cand_blk [B]   as memosight_attn_params wants them (empty block = skipped)
 *   row_tok [T], pos_id [T]       token id to embed and position ID of every row
 *   draft [T]                     what memosight_accept has to find: c_{i+1}, or -1
 *   summary [4]                   {rows in total, live sequences, sequences waiting for
 *                                 compression, 0}: the one thing a host loop reads back
 * Arrays are device memory sized for T = B * (2d+1) rows. */
MS_API int32_t memosight_decode_plan(const memosight_decode_state* state, int32_t* q_off, int32_t* n_cand_blk,
                              int32_t* row_tok, int32_t* pos_id, int32_t* draft, int32_t* summary,
                              void* scratch, memosight_stream_t stream);

/* Applies the greedy verification (argmax, n_match from memosight_accept on this block):
 * c_0..c_m become permanent (m = matching prefix), cut behind the first delimiter or
 * end-of-sequence token among them (which sets the flag) or at the output budget; n_keep[b]
 * says how many, for memosight_kv_append.  The prediction behind the last permanent token is
 * the next c_0; if every candidate was accepted and the step goes on, the d foresight
 * predictions are the next drafts, otherwise they are dropped (they were conditioned on all
 * candidates).  Does not touch kv_len: the append does. */
MS_API int32_t memosight_decode_commit(const memosight_decode_state* state, const int32_t* q_off,
                                const int32_t* argmax, const int32_t* n_match, int32_t* n_keep,
                                memosight_stream_t stream);

/* Builds the compression block of every sequence whose step has ended (Sec. 2.1.2):
 * l = ceil(seg_n / c) memory tokens at the centres of their groups (UPL, rounded down) and <o> at
 * the step's last position + 1, all candidates (causal).  n_keep [B] = l + 1 for the append;
 * seg_start / seg_len [B] are the eviction request for memosight_kv_compact (0 = skip).
 * Arrays sized for T = B * (max_mem + 1) rows.  summary as above. */
MS_API int32_t memosight_decode_plan_compress(const memosight_decode_state* state, int32_t* q_off,
                                       int32_t* n_cand_blk, int32_t* row_tok, int32_t* pos_id,
                                       int32_t* n_keep, int32_t* seg_start, int32_t* seg_len,
                                       int32_t* summary, void* scratch, memosight_stream_t stream);

/* After the compression block was forwarded, appended and the step evicted (kv_len final):
 * the next step starts behind <o>, whose prediction (argmax of the block's last row) is its
 * first token; clears the pending flag. */
MS_API int32_t memosight_decode_commit_compress(const memosight_decode_state* state, const int32_t* q_off,
                                         const int32_t* argmax, memosight_stream_t stream);

/* ---- One whole step with the step's inputs and results in host memory -------------------- */

/* The KV cache is device-resident state (it is what the method keeps compacted);
 * everything a step consumes or produces besides it may live on the host.  This
 * call copies the step's inputs from host memory (pinned memory makes the copies
 * asynchronous), runs RoPE -> step attention -> greedy accept -> append of the
 * accepted candidates (-> optional compaction) on `stream`, and copies the results
 * back.  All device pointers are caller-owned staging buffers of the stated sizes.
 * The logits are copied on a stream of the library's own (created, with two
 * events, at the first call on a device) beside RoPE and the attention, and joined
 * into `stream` before the accept; calls for one device share that stream and the
 * events, so issue them one after the other, not from several threads at once,
 * and make the first call on a device outside any stream capture.
 * The call returns after queueing; synchronise `stream` before reading h_*.
 * Any h_* pointer may be NULL: that tensor is then taken from (or left in) its device staging
 * buffer and not copied.  With all of them NULL the call is the whole device-resident step --
 * RoPE, attention, accept, append, compaction -- queued by one call into the library. */
typedef struct memosight_step_host_params {
  uint32_t struct_size;          /* sizeof(memosight_step_host_params)                         */
  memosight_attn_params attn;    /* device-side description of the step: q, k_step, v_step, out,
                                    lse are the device staging buffers the host data goes
                                    through; k_cache/v_cache/kv_len are updated by the append  */
  const void* h_q;               /* host bf16 [T][H_q][D], before RoPE                         */
  const void* h_k_step;          /* host bf16 [T][H_kv][D], before RoPE                        */
  const void* h_v_step;          /* host bf16 [T][H_kv][D]                                     */
  const int32_t* h_pos_id;       /* host [T] position IDs of the block rows                    */
  int32_t* d_pos_id;             /* device [T] staging                                         */
  double rope_base;              /* theta_i = rope_base^(-2i/D)                                */
  uint32_t rope_flags;           /* MS_ROPE_* | MS_POS_*                                       */
  int32_t vocab;                 /* V; 0 skips accept and append                               */
  const float* h_logits;         /* host fp32 [T][ld_v]                                        */
  int64_t ld_v;
  float* d_logits;               /* device [T][ld_v] staging                                   */
  const int32_t* h_draft;        /* host [T]                                                   */
  int32_t* d_draft;              /* device [T] staging                                         */
  int32_t* d_argmax;             /* device [T]                                                 */
  int32_t* d_n_match;            /* device [B]                                                 */
  int32_t* d_n_keep;             /* device [B]                                                 */
  void* accept_workspace;        /* device, memosight_accept_workspace_bytes(T, V)             */
  size_t accept_workspace_bytes;
  const int32_t* d_seg_start;    /* device [B] or NULL: compaction request after the append    */
  const int32_t* d_seg_len;      /* device [B] (0 = skip sequence) when d_seg_start != NULL    */
  int32_t max_tail;              /* host bound of the entries a compaction moves               */
  const int32_t* d_kv_cap;       /* device [B] or NULL: capacity of each sequence (kv_append)  */
  void* h_out;                   /* host bf16 [T][H_q][D]                                      */
  int32_t* h_argmax;             /* host [T] or NULL                                           */
  int32_t* h_n_match;            /* host [B] or NULL                                           */
} memosight_step_host_params;

MS_API int32_t memosight_step_host(const memosight_step_host_params* params,
                                   memosight_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* MEMOSIGHT_H_ */
