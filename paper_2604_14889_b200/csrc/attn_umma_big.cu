// tcgen05 attention for large blocks (17..32768 new tokens per sequence), head_dim 128.
//
// MemoSight's compression pass (paper Sec. 2.1.2; Algorithm 1, the forward over the l memory
// tokens and <o> appended behind a finished reasoning step) is the same masked attention as
// a Predict+Verify step -- whole compacted cache visible, the block's own tokens causal -- but
// with up to ceil(512/3)+1 = 172 tokens in the block, i.e. several hundred packed rows per KV
// head.  The prefill of a prompt (Algorithm 1, Prefill) is the same call with a longer block and
// an empty cache.  The block is cut into row tiles of floor(128/G) tokens (<= 128 packed rows); a work
// unit is (sequence, KV head, row tile) and streams the whole cache plus the step-local key
// tiles up to its own last token (later keys are invisible to all of its rows).
//
// Rows on the TMEM lanes: S = Q K^T (128 x 128 per tile, Q and K from 128-byte-swizzled shared
// memory filled by TMA) and O += P V (P read from tensor memory, V from shared memory) on
// tcgen05.mma.  The softmax is the limit in this compute-heavy regime, so two warpgroups share
// every tile: warpgroup g takes key columns [64g, 64g+64) of the scores, writes its P (bf16, two
// keys per column) over the first half of those same columns once it holds the scores in
// registers, and owns an output accumulator of its own -- keys 0..63 of every tile accumulate
// into O_0, keys 64..127 into O_1 -- with its own row references and row sums.  The two groups
// therefore never have to agree inside an item; at its end they fold (m_g, l_g, O_g) through
// shared memory and group g writes output columns [64g, 64g+64).  A row's reference is the exact
// maximum of its group's columns in the item's first tile and only moves when a score exceeds it
// by about 2^48 (seen in the tile's row sum).  Tensor memory: S0 | S1 | O_0 | O_1 = 512 columns.
// The whole issuing warp walks the schedule, so that addresses and descriptors are uniform
// across it, and one elected lane issues: 8 products then issue in ~400 cycles (~620 when a
// single thread computed them).
// Schedule: work items dealt round-robin to the persistent CTAs so that the row tiles of one K/V
// chunk run side by side (see below); every wait is bounded (status word in the workspace, as in
// the other paths).
#include "attn_umma_common.cuh"

namespace ms {
namespace {

constexpr int kBWg = 2;                           // softmax warpgroups: each takes 128 / kBWg key columns of a tile
constexpr int kBCw = kTile / kBWg;
constexpr int kBThreads = 128 + 128 * kBWg;       // warp 0: TMA, warp 1: MMA issue, warps 4..: softmax warpgroups
constexpr int kBD = 128;
static_assert(kBCw % 32 == 0 && kBD / kBWg == kBCw, "a warpgroup's score and output columns are whole 32-column loads");
constexpr uint32_t kBCols = 512;  // S0 | S1 | O of key columns 0..63 | O of key columns 64..127
constexpr uint32_t kBColS = 0, kBColO = 256;      // accumulator of softmax warpgroup g at kBColO + g * kBD
static_assert(kBWg == 2 && kBColO + kBWg * kBD <= kBCols, "one output accumulator per softmax warpgroup");
constexpr float kBGrowSum = 281474976710656.f;   // 2^48: a partial row sum this large moves the reference
constexpr int kBKv = 6;                           // K/V buffers in the ring: three tiles in flight
constexpr int kBKvBytes = kTile * kBD * 2;        // 32 KB
constexpr uint32_t kBHalf = kTile * 128;          // bytes between 64-column halves of a tile
constexpr int kBQBytes = 2 * kBHalf;
constexpr int kBOffQ = 0, kBOffKv = kBQBytes;
constexpr int kBOffMisc = kBOffKv + kBKv * kBKvBytes;
// misc: barriers | scalars | mx[kBWg][128] | lpart[kBWg][128]
constexpr int kBMiscScalars = 256, kBMiscMx = 512, kBMiscL = kBMiscMx + kBWg * kTile * 4;
constexpr int kBMiscBytes = kBMiscL + kBWg * kTile * 4;
constexpr int kBSmem = kBOffMisc + kBMiscBytes;
static_assert(kBSmem <= 227 * 1024, "shared memory budget");

enum : int {
  kBbKvFull = 0, kBbKvEmpty = kBKv, kBbQFull = 2 * kBKv, kBbQEmpty, kBbPFull, kBbAll = kBbPFull + 2, kBbDrain,
  kBbCount
};
static_assert(kBbCount * 8 <= kBMiscScalars, "barriers overflow their slot");

// ---------------------------------------------------------------- schedule
//
// Work items are (sequence, KV head, chunk of the unit's tiles, row tile), enumerated in that
// order with the row tile fastest, and dealt to the persistent CTAs round-robin: at any moment
// neighbouring CTAs work on the row tiles of the same K/V chunk, so a K/V tile that several row
// tiles need is fetched from HBM once and found in L2 by the others.  A unit's tiles (cache tiles,
// then the step-local key tiles up to the row tile's last token) are cut into `nsplit` chunks only
// when there are too few units to fill the machine; a chunked unit leaves one (m, l, O) partial per
// chunk for attn_big_merge_kernel.  With more units than CTAs only the units of the last, partial
// round are cut (big_tail below).

struct BigSeq {
  int L, n_q, r0, n_c, cache_tiles, n_rt;
  long long slot_off;
};
__device__ __forceinline__ int big_step_tiles(const BigSeq& s, int rt, int tpt) {
  const int last = min(s.n_q, (rt + 1) * tpt);           // keys up to the tile's last token
  return (last + kTile - 1) / kTile;
}
__device__ __forceinline__ void big_seq(const AttnArgs& a, int b, int tpt, BigSeq& s) {
  seq_shape(a, b, s.L, s.n_q, s.r0);
  int n_c = a.n_cand[b];
  s.n_c = n_c < 0 ? 0 : (n_c > s.n_q ? s.n_q : n_c);
  s.slot_off = a.kv_off[b];
  s.cache_tiles = (s.L + kTile - 1) / kTile;
  s.n_rt = (s.n_q + tpt - 1) / tpt;
}

// pre[0..B]: exclusive prefix sum of the sequences' row-tile counts (one CTA).
__global__ void __launch_bounds__(256)
attn_big_plan_kernel(const AttnArgs a, int tpt, int* __restrict__ pre) {
  __shared__ int scratch[256];
  const int nt = blockDim.x, tid = threadIdx.x;
  const int per = (a.B + nt - 1) / nt;
  const int lo = min(a.B, tid * per), hi = min(a.B, lo + per);
  int sum = 0;
  for (int b = lo; b < hi; ++b) {
    BigSeq s;
    big_seq(a, b, tpt, s);
    sum += s.n_rt;
  }
  scratch[tid] = sum;
  __syncthreads();
  int base = 0;
  for (int t = 0; t < tid; ++t) base += scratch[t];
  for (int b = lo; b < hi; ++b) {
    BigSeq s;
    big_seq(a, b, tpt, s);
    pre[b] = base;
    base += s.n_rt;
  }
  if (tid == nt - 1) pre[a.B] = base;
}

// Whole units dealt round-robin leave the last round ragged: 512 units on 148 CTAs are three full
// rounds and 68 units more, and the launch lasts four units while the average CTA has 3.46.  When
// units are not chunked anyway, the units of that last, partial round are cut into `split` chunks
// each (as many as fit the grid once more), so that the round costs 1 / split of a unit: units
// [0, u0) stay whole, unit u0 + t / split, chunk t % split is item u0 + t, and its partial goes to
// slot t (at most one per CTA) for attn_big_tail_merge_kernel.  Both kernels derive (u0, split)
// from the unit count with this function.
constexpr int kBMaxTailSplit = 8;
__device__ __forceinline__ void big_tail(int units, int n_ctas, int nsplit, int& u0, int& split) {
  u0 = units;
  split = 1;
  if (nsplit != 1 || units <= n_ctas) return;
  const int rem = units % n_ctas;
  if (rem == 0 || n_ctas / rem < 2) return;
  split = min(n_ctas / rem, kBMaxTailSplit);
  u0 = units - rem;
}

struct BigWalk {
  BigSeq s;
  int b, h, rt, ti, ti_lo, ti_hi, tpt;
  int item, n_items, nsplit;
  int tail_u0, tail_split, item_slot;
  int it, piece_idx, piece_j, slot;
  bool first, last, done;
  int step_idx, nvalid;     // step_idx < 0: cache tile
};
// Moves to this CTA's next non-empty item (items are visited with stride gridDim.x).
__device__ __forceinline__ void bwalk_advance(const AttnArgs& a, BigWalk& w, const int* __restrict__ pre) {
  for (;;) {
    w.item += static_cast<int>(gridDim.x);
    if (w.item >= w.n_items) { w.done = true; return; }
    // index in the (sequence, head, chunk, row tile) order; a unit of the cut last round comes with its own chunk
    int idx = w.item, tail_chunk = -1;
    if (w.item >= w.tail_u0) {
      const int t = w.item - w.tail_u0;
      idx = w.tail_u0 + t / w.tail_split;
      tail_chunk = t - (t / w.tail_split) * w.tail_split;
    }
    const int per_rt = a.H_kv * w.nsplit;                 // items per row tile of a sequence
    int lo = 0, hi = a.B;
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (static_cast<long long>(pre[mid]) * per_rt <= idx) lo = mid; else hi = mid;
    }
    w.b = lo;
    big_seq(a, lo, w.tpt, w.s);
    if (w.s.n_rt == 0) continue;                          // cannot happen for a valid index; stay safe
    int j = idx - pre[lo] * per_rt;
    const int per_head = w.nsplit * w.s.n_rt;
    w.h = j / per_head;
    j -= w.h * per_head;
    int chunk = j / w.s.n_rt, n_chunks = w.nsplit;
    w.rt = j - chunk * w.s.n_rt;
    w.item_slot = (w.nsplit == 1) ? -1 : w.item;
    if (tail_chunk >= 0) {
      chunk = tail_chunk;
      n_chunks = w.tail_split;
      w.item_slot = w.item - w.tail_u0;
    }
    const int tiles_u = w.s.cache_tiles + big_step_tiles(w.s, w.rt, w.tpt);
    w.ti_lo = static_cast<int>(static_cast<long long>(tiles_u) * chunk / n_chunks);
    w.ti_hi = static_cast<int>(static_cast<long long>(tiles_u) * (chunk + 1) / n_chunks);
    if (w.ti_lo < w.ti_hi) break;
  }
  w.ti = w.ti_lo;
}
__device__ __forceinline__ void bwalk_init(const AttnArgs& a, BigWalk& w, int tpt, int nsplit, const int* pre) {
  w.tpt = tpt;
  w.nsplit = nsplit;
  {
    const int units = pre[a.B] * a.H_kv;
    big_tail(units, static_cast<int>(gridDim.x), nsplit, w.tail_u0, w.tail_split);
    w.n_items = (nsplit == 1) ? w.tail_u0 + (units - w.tail_u0) * w.tail_split : units * nsplit;
    if (nsplit != 1) w.tail_u0 = w.n_items;             // no item is a tail item
  }
  w.item_slot = -1;
  w.item = static_cast<int>(blockIdx.x) - static_cast<int>(gridDim.x);
  w.it = 0;
  w.piece_idx = -1;
  w.piece_j = 0;
  w.slot = 0;
  w.done = false;
  bwalk_advance(a, w, pre);
}
__device__ __forceinline__ void bwalk_tile(BigWalk& w) {
  w.first = (w.ti == w.ti_lo);
  if (w.first) {
    w.slot = w.item_slot;
    w.piece_idx += 1;
    w.piece_j = 0;
  }
  w.step_idx = w.ti - w.s.cache_tiles;
  w.last = (w.ti == w.ti_hi - 1);
  w.nvalid = w.step_idx >= 0 ? min(kTile, w.s.n_q - w.step_idx * kTile) : min(kTile, w.s.L - w.ti * kTile);
}
__device__ __forceinline__ void bwalk_next(const AttnArgs& a, BigWalk& w, const int* __restrict__ pre) {
  w.piece_j += 1;
  w.it += 1;
  if (++w.ti == w.ti_hi) bwalk_advance(a, w, pre);
}

// Number of leading step-local key tiles of an item that need no mask: every key of such a tile is a
// candidate that precedes every token of the row tile, and all its rows are candidates (default
// anchors, no training-time mask) -- the tiles left of the diagonal of a prefill or compression block.
__device__ __forceinline__ int big_plain_step_tiles(const AttnArgs& a, const BigSeq& s, int rt, int tpt) {
  const int tok0 = rt * tpt, tok_end = min(s.n_q, tok0 + tpt);
  return (!a.tok_kind && !a.anchor && tok_end <= s.n_c) ? tok0 / kTile : 0;
}

__device__ __host__ inline size_t big_slot_floats() { return static_cast<size_t>(kTile) * (kBD + 2); }

// The warpgroup's 64 score columns of one row, from tensor memory into v[]; with kMasked the
// invisible keys (past the valid length; on a step-local tile by the (n_cand, anchor) rule)
// become -inf.
// (With meta_kind the step-local rule is the training-time one: kind/step of key token j at
// meta_kind[j] / meta_step[j], the row's own step in anc.)
template <bool kMasked>
__device__ __forceinline__ void big_load_scores(uint32_t s_addr, float (&v)[kBCw], int col0, int nv, bool is_step,
                                                int tok, int key0, int n_c, int anc,
                                                const uint8_t* __restrict__ meta_kind = nullptr,
                                                const int32_t* __restrict__ meta_step = nullptr) {
  uint32_t raw[kBCw / 32][32];
#pragma unroll
  for (int c = 0; c < kBCw / 32; ++c) tmem_ld32(s_addr + c * 32, raw[c]);
#pragma unroll
  for (int c = 0; c < kBCw / 32; ++c) tmem_ld_wait(raw[c]);
#pragma unroll
  for (int e = 0; e < kBCw; ++e) {
    float s = __uint_as_float(raw[e >> 5][e & 31]);
    if (kMasked) {
      bool vis = col0 + e < nv;
      if (is_step && vis) {
        const int j = key0 + e;
        vis = meta_kind ? train_key_visible(tok, j, __ldg(meta_kind + j), anc, __ldg(meta_step + j))
                        : step_key_visible(tok, j, n_c, anc);
      }
      s = vis ? s : -INFINITY;
    }
    v[e] = s;
  }
}
// The same when the visible keys of the row are a prefix of the warpgroup's columns (a ragged cache
// tile; a causal tile of a block whose rows are all candidates): columns from `limit` on become -inf.
__device__ __forceinline__ void big_load_scores_prefix(uint32_t s_addr, float (&v)[kBCw], int limit) {
  uint32_t raw[kBCw / 32][32];
#pragma unroll
  for (int c = 0; c < kBCw / 32; ++c) tmem_ld32(s_addr + c * 32, raw[c]);
#pragma unroll
  for (int c = 0; c < kBCw / 32; ++c) tmem_ld_wait(raw[c]);
#pragma unroll
  for (int e = 0; e < kBCw; ++e) v[e] = (e < limit) ? __uint_as_float(raw[e >> 5][e & 31]) : -INFINITY;
}
__device__ __forceinline__ float max_cols(const float (&v)[kBCw]) {
  float m[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) m[j] = v[j];
#pragma unroll
  for (int j = 8; j < kBCw; ++j) m[j & 7] = fmaxf(m[j & 7], v[j]);
  return fmaxf(fmaxf(fmaxf(m[0], m[1]), fmaxf(m[2], m[3])), fmaxf(fmaxf(m[4], m[5]), fmaxf(m[6], m[7])));
}

// mbarrier.arrive under a predicate, without a branch.
__device__ __forceinline__ void mbar_arrive_if(bool pred, uint32_t bar) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %1, 0;\n\t@p mbarrier.arrive.shared::cta.b64 _, [%0];\n\t}"
               ::"r"(bar), "r"(static_cast<uint32_t>(pred))
               : "memory");
}

// ---------------------------------------------------------------- kernel

__global__ void __launch_bounds__(kBThreads, 1)
attn_umma_big_kernel(const AttnArgs a, const __grid_constant__ CUtensorMap map_k,
                     const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_ks,
                     const __grid_constant__ CUtensorMap map_vs, const __grid_constant__ CUtensorMap map_q,
                     int tpt, int nsplit) {
  constexpr int D = kBD, HALVES = 2, KSTEPS = D / 16;
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sb = smem_u32(smem);
  const uint32_t bars = sb + kBOffMisc;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kBOffMisc + kBMiscScalars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kBOffMisc + kBMiscScalars + 8);
  float* s_mx = reinterpret_cast<float*>(smem + kBOffMisc + kBMiscMx);      // [kBWg][128]
  float* s_lp = reinterpret_cast<float*>(smem + kBOffMisc + kBMiscL);       // [kBWg][128]
  uint32_t* status = reinterpret_cast<uint32_t*>(a.workspace);
  int* ws_pre = reinterpret_cast<int*>(reinterpret_cast<uint8_t*>(a.workspace) + kWsHeaderBytes);
  float* ws_slots = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(a.workspace) + kWsHeaderBytes +
                                             ws_prefix_bytes());
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (sb & 1023u) {
    if (threadIdx.x == 0) atomicExch(status, kTimeoutMagic + 1);
    return;
  }
  const int rows_box = tpt * a.G;

  // ---- schedule: this CTA's items, and how many tiles they hold ----
  const int* __restrict__ pre = ws_pre;
  BigWalk w0;
  bwalk_init(a, w0, tpt, nsplit, pre);
  int n_iter = 0;
  {
    BigWalk wc = w0;
    while (!wc.done) {
      n_iter += wc.ti_hi - wc.ti_lo;
      bwalk_advance(a, wc, pre);
    }
  }
  if (threadIdx.x == 0) {
    for (int i = 0; i < kBKv; ++i) {
      mbar_init(bars + 8 * (kBbKvFull + i), 1);
      mbar_init(bars + 8 * (kBbKvEmpty + i), 1);
    }
    mbar_init(bars + 8 * kBbQFull, 1);
    mbar_init(bars + 8 * kBbQEmpty, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(bars + 8 * (kBbPFull + i), 4 * kBWg);
    }
    mbar_init(bars + 8 * kBbAll, 4 * kBWg);
    mbar_init(bars + 8 * kBbDrain, 1);
    wait_ctx_init(abort_flag, a.wait_limit_us);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(tmem_slot)), "r"(kBCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0 && lane == 0 && n_iter > 0) {
    // =========================== TMA producer ===========================
    BigWalk w = w0;
    bool ok = true;
    int uses = 0, pieces = 0;
    RingPos rp;
    rp.init(0, kBKv);
    while (w.it < n_iter) {
      // ---- the item's tiles behind its first: K and V of tile after tile, no walker
      if (w.ti > w.ti_lo) {
        const int ct = w.s.cache_tiles, n_run = w.ti_hi - w.ti;
        const int n_cache = max(0, min(ct, w.ti_hi) - w.ti);
        auto ring_slot = [&](uint32_t& dst, uint32_t& bar) -> bool {
          const int buf = rp.buf;
          if (!mbar_wait(bars + 8 * (kBbKvEmpty + buf), rp.par ^ 1u, abort_flag, status)) return false;
          rp.step(1);
          fence_async_smem();
          dst = sb + kBOffKv + buf * kBKvBytes;
          bar = bars + 8 * (kBbKvFull + buf);
          mbar_arrive_expect_tx(bar, static_cast<uint32_t>(kBKvBytes));
          ++uses;
          return true;
        };
        int y = static_cast<int>(w.s.slot_off) + w.ti * kTile;
        for (int k = 0; k < 2 * n_cache; ++k) {                 // cache tiles
          uint32_t dst, bar;
          if (!ring_slot(dst, bar)) { ok = false; break; }
          const CUtensorMap* map = (k & 1) ? &map_v : &map_k;
          tma_load_3d(dst, map, bar, 0, y, w.h);
          tma_load_3d(dst + kBHalf, map, bar, 64, y, w.h);
          y += (k & 1) * kTile;
        }
        if (!ok) break;
        int z = w.s.r0 + (w.ti + n_cache - ct) * kTile;
        for (int k = 0; k < 2 * (n_run - n_cache); ++k) {       // the block's own key tiles
          uint32_t dst, bar;
          if (!ring_slot(dst, bar)) { ok = false; break; }
          const CUtensorMap* map = (k & 1) ? &map_vs : &map_ks;
          tma_load_3d(dst, map, bar, 0, w.h, z);
          tma_load_3d(dst + kBHalf, map, bar, 64, w.h, z);
          z += (k & 1) * kTile;
        }
        if (!ok) break;
        w.ti += n_run - 1;            // bwalk_next moves past the item's last tile and on to the next item
        w.it += n_run - 1;
        w.piece_j += n_run - 1;
        bwalk_next(a, w, pre);
        continue;
      }
      bwalk_tile(w);
      if (w.first) {
        // one Q buffer: every Q K^T of the previous unit must have read it
        if (!mbar_wait(bars + 8 * kBbQEmpty, (w.piece_idx & 1) ^ 1, abort_flag, status)) { ok = false; break; }
        fence_async_smem();
        const uint32_t bar = bars + 8 * kBbQFull;
        mbar_arrive_expect_tx(bar, static_cast<uint32_t>(HALVES * rows_box * 128));
#pragma unroll
        for (int hf = 0; hf < HALVES; ++hf)
          tma_load_3d(sb + kBOffQ + hf * kBHalf, &map_q, bar, hf * 64, w.h * a.G, w.s.r0 + w.rt * tpt);
        ++pieces;
      }
#pragma unroll 1
      for (int kv = 0; kv < 2; ++kv) {
        const int buf = rp.buf;
        if (!mbar_wait(bars + 8 * (kBbKvEmpty + buf), rp.par ^ 1u, abort_flag, status)) { ok = false; break; }
        rp.step(1);
        fence_async_smem();
        const uint32_t dst = sb + kBOffKv + buf * kBKvBytes;
        const uint32_t bar = bars + 8 * (kBbKvFull + buf);
        mbar_arrive_expect_tx(bar, static_cast<uint32_t>(kBKvBytes));
        if (w.step_idx >= 0) {
          const int z = w.s.r0 + w.step_idx * kTile;
#pragma unroll
          for (int hf = 0; hf < HALVES; ++hf)
            tma_load_3d(dst + hf * kBHalf, kv ? &map_vs : &map_ks, bar, hf * 64, w.h, z);
        } else {
          const int y = static_cast<int>(w.s.slot_off) + w.ti * kTile;
#pragma unroll
          for (int hf = 0; hf < HALVES; ++hf)
            tma_load_3d(dst + hf * kBHalf, kv ? &map_v : &map_k, bar, hf * 64, y, w.h);
        }
        ++uses;
      }
      if (!ok) break;
      bwalk_next(a, w, pre);
    }
    for (int u = uses > kBKv ? uses - kBKv : 0; u < uses; ++u)
      (void)mbar_wait(bars + 8 * (kBbKvFull + u % kBKv), (u / kBKv) & 1, abort_flag, status);
    if (pieces > 0) (void)mbar_wait(bars + 8 * kBbQFull, (pieces - 1) & 1, abort_flag, status);
  } else if (warp == 1 && n_iter > 0) {
    // =========================== MMA issuer ===========================
    // The whole warp walks the schedule in step, so that addresses and descriptors are the same in
    // every lane; one elected lane (always the same one) issues the tensor-core instructions.
    const uint32_t idesc_qk = instr_desc(kTile, 0), idesc_pv = instr_desc(D, 1);
    const uint32_t q_lo = desc_lo(sb + kBOffQ, 16), k_lo0 = desc_lo(sb + kBOffKv, 16);
    const uint32_t v_lo0 = desc_lo(sb + kBOffKv, kBHalf);
    BigWalk wq = w0, wp = w0;
    RingPos rk, rv;
    rk.init(0, kBKv);
    rv.init(1, kBKv);
    bool ok = true;
    auto mwait = [&](uint32_t bar, uint32_t parity) -> bool {
      return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag, status));
    };
    // Keys 0..63 of a tile accumulate into the first output accumulator, keys 64..127 into the
    // second: each softmax warpgroup then owns the running reference of its own accumulator and
    // the two never have to agree inside an item.  The second accumulator is first written by the
    // item's first tile with more than 64 valid keys.
    bool o1_live = false;
    // P of 16 keys = 8 columns of tensor memory: warpgroup g left its 64 keys in the first 32 of its
    // 64 score columns
    auto issue_pv = [&](const uint32_t p_col, const uint32_t v_lo, const int j, const uint32_t acc) {
      umma_bf16_ts_lo_elect(tmem + kBColO + (j >> 2) * kBD, p_col + (j >> 2) * kBCw + (j & 3) * 8,
                      v_lo + j * (2048 >> 4), idesc_pv, acc);
    };
    auto issue_qk = [&]() -> bool {
      bwalk_tile(wq);
      const int it = wq.it;
      if ((wq.first && !mwait(bars + 8 * kBbQFull, wq.piece_idx & 1)) ||
          !mwait(bars + 8 * (kBbKvFull + rk.buf), rk.par))
        return false;
      tc_fence_after();
      const uint32_t k_lo = k_lo0 + rk.buf * (kBKvBytes >> 4);
      const uint32_t d_s = tmem + kBColS + (it & 1) * kTile;
#pragma unroll
      for (int ks = 0; ks < KSTEPS; ++ks) {
        const uint32_t off = (ks >> 2) * (kBHalf >> 4) + (ks & 3) * 2;
        umma_bf16_lo_elect(d_s, q_lo + off, k_lo + off, idesc_qk, ks > 0);
      }
      umma_commit_elect(bars + 8 * (kBbKvEmpty + rk.buf));
      if (wq.last) umma_commit_elect(bars + 8 * kBbQEmpty);
      rk.step(2);
      bwalk_next(a, wq, pre);
      return true;
    };
    ok = issue_qk();
    while (ok && wp.it < n_iter) {
      // ---- a run of plain tiles needs neither walker: S of a tile that is neither the first nor the
      //      last of its item, O += P V of a tile with all 128 keys valid that is not the first
      if (wq.item == wp.item && wp.ti > wp.ti_lo && wq.it == wp.it + 1) {
        const int ct = wp.s.cache_tiles;
        const int p_stop = wp.ti < ct ? wp.s.L / kTile : ct + wp.s.n_q / kTile;   // tiles with all 128 keys valid
        int n_run = min(wq.ti_hi - 1 - wq.ti, p_stop - wp.ti);
        int it = wp.it;
        for (; n_run > 0; --n_run, ++it) {
          // S(it + 1)
          if (!mwait(bars + 8 * (kBbKvFull + rk.buf), rk.par)) { ok = false; break; }
          tc_fence_after();
          {
            const uint32_t k_lo = k_lo0 + rk.buf * (kBKvBytes >> 4);
            const uint32_t d_s = tmem + kBColS + ((it + 1) & 1) * kTile;
#pragma unroll
            for (int ks = 0; ks < KSTEPS; ++ks) {
              const uint32_t off = (ks >> 2) * (kBHalf >> 4) + (ks & 3) * 2;
              umma_bf16_lo_elect(d_s, q_lo + off, k_lo + off, idesc_qk, ks > 0);
            }
            umma_commit_elect(bars + 8 * (kBbKvEmpty + rk.buf));
            rk.step(2);
          }
          // O += P V (it)
          if (!mwait(bars + 8 * (kBbPFull + (it & 1)), (it >> 1) & 1) ||
              !mwait(bars + 8 * (kBbKvFull + rv.buf), rv.par)) {
            ok = false;
            break;
          }
          tc_fence_after();
          {
            const uint32_t p_lo = tmem + kBColS + (it & 1) * kTile;
            const uint32_t v_lo = v_lo0 + rv.buf * (kBKvBytes >> 4);
            const uint32_t acc1 = o1_live ? 1u : 0u;
#pragma unroll
            for (int j = 0; j < kTile / 16; ++j) issue_pv(p_lo, v_lo, j, j == 4 ? acc1 : 1u);
            o1_live = true;
            umma_commit_elect(bars + 8 * (kBbKvEmpty + rv.buf));
            rv.step(2);
          }
        }
        if (!ok) break;
        const int done = it - wp.it;
        wq.ti += done;
        wq.it += done;
        wq.piece_j += done;
        wp.ti += done;
        wp.it += done;
        wp.piece_j += done;
      }
      if (wq.it < n_iter && !issue_qk()) { ok = false; break; }
      bwalk_tile(wp);
      const int it = wp.it;
      if (!mwait(bars + 8 * (kBbPFull + (it & 1)), (it >> 1) & 1) ||
          !mwait(bars + 8 * (kBbKvFull + rv.buf), rv.par)) {
        ok = false;
        break;
      }
      tc_fence_after();
      const uint32_t p_lo = tmem + kBColS + (it & 1) * kTile;
      const uint32_t v_lo = v_lo0 + rv.buf * (kBKvBytes >> 4);
      const int ksteps = (wp.nvalid + 15) >> 4;
      const uint32_t acc0 = wp.first ? 0u : 1u;
      if (wp.first) o1_live = false;
      const uint32_t acc1 = o1_live ? 1u : 0u;
      if (ksteps == kTile / 16) {
#pragma unroll
        for (int j = 0; j < kTile / 16; ++j) issue_pv(p_lo, v_lo, j, j == 0 ? acc0 : (j == 4 ? acc1 : 1u));
      } else {
#pragma unroll 1
        for (int j = 0; j < ksteps; ++j) issue_pv(p_lo, v_lo, j, j == 0 ? acc0 : (j == 4 ? acc1 : 1u));
      }
      if (ksteps > 4) o1_live = true;
      umma_commit_elect(bars + 8 * (kBbKvEmpty + rv.buf));
      rv.step(2);
      bwalk_next(a, wp, pre);
    }
    if (!ok) {
      umma_commit_elect(bars + 8 * kBbDrain);
      const unsigned long long t_begin = global_ns();
      while (!mbar_try_wait(bars + 8 * kBbDrain, 0) && global_ns() - t_begin < wait_limit_ns(abort_flag)) {
      }
    }
  } else if (warp >= 4 && n_iter > 0) {
    // ====== softmax warps: thread = packed row; warpgroup g = key columns [kBCw*g, kBCw*(g+1)) of every tile, with
    //        an output accumulator and a running reference of its own.  Inside an item the two groups
    //        never talk; at its end they fold their halves and group g writes output columns
    //        [kBCw*g, kBCw*(g+1)) ======
    const int wg = (warp - 4) >> 2, quad = (warp - 4) & 3;
    const int r = quad * 32 + lane;
    const uint32_t lane_addr = tmem + (static_cast<uint32_t>(quad * 32) << 16);
    BigWalk w = w0;
    float m_ref = 0.f, l_part = 0.f;
    bool unref = false;     // the row has not seen a visible key among this group's columns in this item: no reference yet
    bool o1_live = false;   // the second accumulator has been written in this item (a tile with more than 64 valid keys)
    int tok = 0, anc = 0, rows = 0;
    bool row_ok = false;
    bool warp_live = true;    // some row of this warp's 32 exists in the item's row tile
    uint32_t all_phase = 0;
    bool ok = true;
    auto wait_all = [&](uint32_t bar, uint32_t parity) -> bool {
      return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag, status));
    };
    // "S(it) is complete" and "O += P V of tile it is complete" need no barriers of their own: the
    // commits that release the tile's K buffer (ring use 2 it) and V buffer (use 2 it + 1) are those
    // events.  A waiter is never two phases behind: the buffer's next use belongs to tile
    // it + kBKv / 2, whose S needs the P of every tile before it handed over and whose PV needs its own.
    auto wait_released = [&](int use) -> bool {
      return wait_all(bars + 8 * (kBbKvEmpty + use % kBKv), (use / kBKv) & 1);
    };
    auto wait_s_full = [&](int it) -> bool { return wait_released(2 * it); };
    auto wait_pv_done = [&](int it) -> bool { return wait_released(2 * it + 1); };
    // bounded barrier of all softmax warps (also publishes their shared-memory writes)
    auto sync_all = [&]() -> bool {
      __syncwarp();
      mbar_arrive_if(lane == 0, bars + 8 * kBbAll);
      const bool good = wait_all(bars + 8 * kBbAll, all_phase & 1);
      ++all_phase;
      return good;
    };
    // One tile from the scores in tensor memory to P handed over (S(it) is complete; the P buffer is
    // free with it: the commit behind S(it) tracks every earlier tcgen05 operation of the issuing
    // thread, O += P V of tile it - 2 among them).  `masked`: ragged or step-local tile.
    auto tile_body = [&](const bool masked, const bool opens_item, const int nv, const bool is_step,
                         const int step_idx, const int it) -> bool {
      const int pb = it & 1;
      tc_fence_after();
      if (masked && (nv & 15)) {
        // V rows past the valid keys hold foreign or stale bytes; P is 0 there but 0 * NaN is NaN
        const int use = 2 * it + 1, buf = use % kBKv;
        if (!wait_all(bars + 8 * (kBbKvFull + buf), (use / kBKv) & 1)) return false;
        const uint32_t va = sb + kBOffKv + buf * kBKvBytes;
        const int n_rows = ((nv + 15) & ~15) - nv;
        for (int x = wg * kTile + r; x < n_rows * HALVES * 8; x += kBWg * kTile) {
          const int rr = nv + x / (HALVES * 8), cc = x % (HALVES * 8);
          const uint32_t addr = va + (cc >> 3) * kBHalf + rr * 128 + ((cc & 7) << 4);
          asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(addr), "r"(0u) : "memory");
        }
      }
      if (!warp_live) {
        // A warp whose 32 rows all lie past the end of a short last row tile (44 of 128 rows in the
        // last tile of a 171-token block at G = 4) has nothing to exponentiate: what its rows of P
        // and O hold is never stored, and rows do not mix.  It only keeps in step -- it has waited
        // for the scores like the others and arrives like them -- and leaves the special-function
        // unit to the warps that have rows.
        if (opens_item) {
          unref = true;
          l_part = 0.f;
          o1_live = false;
        }
        if (nv > kBCw) o1_live = true;
        if (masked && (nv & 15)) fence_async_smem();
        tc_fence_before();
        __syncwarp();
        mbar_arrive_if(lane == 0, bars + 8 * (kBbPFull + pb));
        return true;
      }
      // this warpgroup's score columns of the row; invisible keys become -inf
      const uint32_t s_addr = lane_addr + kBColS + pb * kTile + wg * kBCw;
      const int key0 = (is_step ? step_idx * kTile : 0) + wg * kBCw;   // step-local index of column 0
      float v[kBCw];
      if (masked) {
        // causal block of candidates only (prefill, compression): row `tok` sees the keys up to itself
        const bool causal = !a.tok_kind && !a.anchor && min(w.s.n_q, (w.rt + 1) * tpt) <= w.s.n_c;
        if (!is_step || causal)
          big_load_scores_prefix(s_addr, v, (is_step ? min(nv, tok - step_idx * kTile + 1) : nv) - wg * kBCw);
        else
          big_load_scores<true>(s_addr, v, wg * kBCw, nv, is_step, tok, key0, w.s.n_c, anc,
                                a.tok_kind ? a.tok_kind + w.s.r0 : nullptr, a.tok_kind ? a.tok_step + w.s.r0 : nullptr);
      } else
        big_load_scores<false>(s_addr, v, 0, kTile, false, 0, 0, 0, 0);
      if (opens_item) {
        // new item: reference = exact maximum of the first tile over this group's columns
        const float m = max_cols(v);
        // A row that sees no key there (a chunk that starts right of the row's causal limit, a
        // foresight row with anchor 0, a training-mask row behind other steps' tokens, the right
        // half of a diagonal tile) stays without a reference: the first later tile with a visible
        // key sets it through the branch below, whatever the size of its scores (a placeholder of
        // 0 would flush strongly negative rows to a zero sum).
        unref = (m == -INFINITY);
        m_ref = unref ? 0.f : m * a.scale_log2;
        l_part = 0.f;
        o1_live = false;
      }
      // p = 2^(s*scale - m_ref) as bf16 over the first half of this thread's own score columns (all
      // 64 scores are in registers by now), two keys per column; the row's partial sum over this
      // group's keys
      auto p_pass = [&]() -> float {
        // scale-and-shift and the running sums two values per instruction (packed fp32 pairs)
        const f32x2_t scale2 = pack_f32x2(a.scale_log2, a.scale_log2), nm2 = pack_f32x2(-m_ref, -m_ref);
        f32x2_t ls[2] = {pack_f32x2(0.f, 0.f), pack_f32x2(0.f, 0.f)};
  #pragma unroll
        for (int c = 0; c < kBCw / 16; ++c) {
          uint32_t pk[8];
  #pragma unroll
          for (int e = 0; e < 16; e += 2) {
            float x0, x1;
            unpack_f32x2(fma_f32x2(pack_f32x2(v[c * 16 + e], v[c * 16 + e + 1]), scale2, nm2), x0, x1);
            const float p0 = ex2(x0), p1 = ex2(x1);
            ls[(e >> 1) & 1] = add_f32x2(ls[(e >> 1) & 1], pack_f32x2(p0, p1));
            pk[e >> 1] = pack2(p0, p1);
          }
          tmem_st8(s_addr + c * 8, pk);
        }
        float s0, s1, s2, s3;
        unpack_f32x2(ls[0], s0, s1);
        unpack_f32x2(ls[1], s2, s3);
        return (s0 + s1) + (s2 + s3);
      };
      float tsum = p_pass();
      // A score that outgrew the row reference by ~2^48 shows in the sum (so do inf and NaN).  The
      // reference belongs to this thread alone -- its 64 key columns, its accumulator -- so the
      // decision is the thread's own; only the tensor-memory accesses need the whole warp.
      bool regrow = row_ok && !opens_item && !(tsum < kBGrowSum);
      if (unref && row_ok && !opens_item) regrow = max_cols(v) > -INFINITY;   // the row's first visible key here: set its reference
      if (__any_sync(0xffffffffu, regrow)) {
        // ---- rare: move row references up; rescale this group's accumulator and sums ----
        float alpha = 1.f;
        if (regrow) {
          const float m = max_cols(v) * a.scale_log2;
          // (a row without a reference has accumulated nothing: its O and sum are zero and stay so)
          const float m_new = unref ? m : fmaxf(m_ref, m);
          alpha = unref ? 1.f : ex2(m_ref - m_new);
          unref = false;
          m_ref = m_new;
          l_part *= alpha;
        }
        if (wg == 0 || o1_live) {
          if (!wait_pv_done(it - 1)) return false;
          tc_fence_after();
  #pragma unroll 1
          for (int c = 0; c < kBD / 32; ++c) {
            uint32_t o[32];
            tmem_ld32(lane_addr + kBColO + wg * kBD + c * 32, o);
            tmem_ld_wait(o);
  #pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tmem_st32(lane_addr + kBColO + wg * kBD + c * 32, o);
          }
          asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        }
        // every lane again: the stores to tensor memory are warp-wide instructions (a lane whose
        // reference stayed writes the same values as before)
        __syncwarp();
        tsum = p_pass();
      }
      if (nv > kBCw) o1_live = true;
      l_part += tsum;
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      if (masked && (nv & 15)) fence_async_smem();     // the cleared V rows, for the tensor core
      tc_fence_before();
      __syncwarp();
      mbar_arrive_if(lane == 0, bars + 8 * (kBbPFull + pb));
      return true;
    };
    while (ok && w.it < n_iter) {
      // ---- a run of plain tiles -- full cache tiles and step-local tiles left of the diagonal that
      //      neither open nor close the item -- needs none of the walker nor a mask: most tiles of a
      //      long cache or a long block go through this loop
      if (w.ti > w.ti_lo) {
        const int ct = w.s.cache_tiles;
        const int stop = min(w.ti_hi - 1, w.ti < ct ? w.s.L / kTile : ct + big_plain_step_tiles(a, w.s, w.rt, tpt));
        while (w.ti < stop) {
          const int it = w.it;
          if (!wait_s_full(it) ||
              !tile_body(false, false, kTile, false, 0, it)) {
            ok = false;
            break;
          }
          ++w.ti;
          ++w.it;
          ++w.piece_j;
        }
        if (!ok) break;
      }
      bwalk_tile(w);
      const int it = w.it;
      if (w.first) {
        const int tok0 = w.rt * tpt;
        rows = (min(w.s.n_q, tok0 + tpt) - tok0) * a.G;
        row_ok = r < rows;
        warp_live = quad * 32 < rows;
        if (row_ok) {
          const int i = tok0 + r / a.G;
          tok = i;
          anc = a.tok_kind ? a.tok_step[w.s.r0 + i]            // training-time mask: the row's own step
                           : ((i < w.s.n_c) ? i : (a.anchor ? a.anchor[w.s.r0 + i] : w.s.n_c));
        } else {
          tok = 1 << 20;
          anc = 0;
        }
      }
      if (!wait_s_full(it)) { ok = false; break; }
      {
        const int nv = w.nvalid;
        const bool is_step = w.step_idx >= 0;
        const bool masked = is_step ? (w.step_idx >= big_plain_step_tiles(a, w.s, w.rt, tpt)) : (nv < kTile);
        if (!tile_body(masked, w.piece_j == 0, nv, is_step, w.step_idx, it)) { ok = false; break; }
      }

      if (w.last) {
        // ---- end of the item: the unit, or this chunk of it.  Fold the two groups' halves:
        //      (m_g, l_g, O_g) relative to M = max m_g; a group that saw no key counts as m = -inf
        s_mx[wg * kTile + r] = (unref || !(wg == 0 || o1_live)) ? -INFINITY : m_ref;
        s_lp[wg * kTile + r] = l_part;
        if (!sync_all()) { ok = false; break; }
        const float m0 = s_mx[r], m1 = s_mx[kTile + r];
        const float m_row = fmaxf(m0, m1);
        const float w0 = (m0 == -INFINITY) ? 0.f : ex2(m0 - m_row);
        const float w1 = (m1 == -INFINITY) ? 0.f : ex2(m1 - m_row);
        const float l_row = s_lp[r] * w0 + s_lp[kTile + r] * w1;
        if (!wait_pv_done(it)) { ok = false; break; }
        tc_fence_after();
        const int i = tok, g = r % a.G;
        const int64_t orow = static_cast<int64_t>(w.s.r0 + (row_ok ? i : 0)) * a.H_q + w.h * a.G + g;
        float* slot = ws_slots + static_cast<size_t>(w.slot < 0 ? 0 : w.slot) * big_slot_floats();
        const float inv = (w.slot < 0) ? 1.f / l_row : 1.f;     // a partial stays unnormalised, relative to m_row
        const float f0 = w0 * inv, f1 = w1 * inv;
#pragma unroll 1
        for (int c = 0; c < (warp_live ? kBCw / 32 : 0); ++c) {
          uint32_t o[32];
          tmem_ld32(lane_addr + kBColO + wg * kBCw + c * 32, o);
          tmem_ld_wait(o);
#pragma unroll
          for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * f0);
          if (o1_live) {
            uint32_t o1[32];
            tmem_ld32(lane_addr + kBColO + kBD + wg * kBCw + c * 32, o1);
            tmem_ld_wait(o1);
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(fmaf(__uint_as_float(o1[e]), f1, __uint_as_float(o[e])));
          }
          if (row_ok && w.slot < 0) {
            uint4* op = reinterpret_cast<uint4*>(a.out + orow * D + wg * kBCw + c * 32);
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
              uint4 u;
              u.x = pack2(__uint_as_float(o[8 * q4 + 0]), __uint_as_float(o[8 * q4 + 1]));
              u.y = pack2(__uint_as_float(o[8 * q4 + 2]), __uint_as_float(o[8 * q4 + 3]));
              u.z = pack2(__uint_as_float(o[8 * q4 + 4]), __uint_as_float(o[8 * q4 + 5]));
              u.w = pack2(__uint_as_float(o[8 * q4 + 6]), __uint_as_float(o[8 * q4 + 7]));
              op[q4] = u;
            }
          } else if (row_ok) {
            uint4* sp = reinterpret_cast<uint4*>(slot + static_cast<size_t>(r) * D + wg * kBCw + c * 32);
#pragma unroll
            for (int q4 = 0; q4 < 8; ++q4) sp[q4] = make_uint4(o[4 * q4], o[4 * q4 + 1], o[4 * q4 + 2], o[4 * q4 + 3]);
          }
        }
        if (row_ok && wg == 0) {
          if (w.slot < 0) {
            if (a.lse) a.lse[orow] = (m_row + log2f(l_row)) * 0.69314718055994531f;
          } else {
            // a row that saw no key in this chunk leaves m = -inf, l = 0 and a zero O: the merge skips it
            float* sm = slot + static_cast<size_t>(kTile) * D;
            sm[r] = m_row;
            sm[kTile + r] = l_row;
          }
        }
        tc_fence_before();   // the reads of O are ordered before the next item's first PV product
        if (!sync_all()) { ok = false; break; }   // s_mx and s_lp are rewritten at the end of the next item
      }
      bwalk_next(a, w, pre);
    }
  }

  // ---- teardown: every thread arrives here, on success and on abort ----
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kBCols) : "memory");
  }
}

// The partials of one (sequence, KV head, row tile) unit folded into its output rows; one warp per
// packed row folds the chunks' (m, l) with shuffles and accumulates its output columns.  Chunk k's
// partial is slot slot0 + k * slot_stride; a chunk without tiles has none.
__device__ __forceinline__ void big_merge_unit(const AttnArgs& a, const BigSeq& s, int h, int rt, int tpt, int n_chunks,
                                               long long slot0, long long slot_stride,
                                               const float* __restrict__ ws_slots) {
  constexpr int D = kBD, E = D / 32;
  const int tiles_u = s.cache_tiles + big_step_tiles(s, rt, tpt);
  const int tok0 = rt * tpt;
  const int rows = (min(s.n_q, tok0 + tpt) - tok0) * a.G;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const size_t slot_floats = big_slot_floats();
  for (int r = warp; r < rows; r += 4) {
    float M = -INFINITY;
    if (lane < n_chunks) {
      const bool has = static_cast<long long>(tiles_u) * lane / n_chunks < static_cast<long long>(tiles_u) * (lane + 1) / n_chunks;
      if (has) M = ws_slots[(slot0 + static_cast<long long>(lane) * slot_stride) * slot_floats + static_cast<size_t>(kTile) * D + r];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    float Lsum = 0.f, acc[E];
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = 0.f;
    for (int k = 0; k < n_chunks; ++k) {
      if (static_cast<long long>(tiles_u) * k / n_chunks >= static_cast<long long>(tiles_u) * (k + 1) / n_chunks) continue;
      const float* sp = ws_slots + (slot0 + static_cast<long long>(k) * slot_stride) * slot_floats;
      const float m = sp[static_cast<size_t>(kTile) * D + r];
      const float l = sp[static_cast<size_t>(kTile) * D + kTile + r];
      const float wgt = (m == -INFINITY) ? 0.f : exp2f(m - M);
      Lsum += l * wgt;
      const float* po = sp + static_cast<size_t>(r) * D + lane * E;
#pragma unroll
      for (int e = 0; e < E; ++e) acc[e] += wgt * po[e];
    }
    const int i = tok0 + r / a.G, g = r % a.G;
    const int64_t orow = static_cast<int64_t>(s.r0 + i) * a.H_q + h * a.G + g;
    const float inv = 1.f / Lsum;
    __nv_bfloat16* op = a.out + orow * D + lane * E;
#pragma unroll
    for (int e = 0; e < E; e += 2) *reinterpret_cast<uint32_t*>(op + e) = pack2(acc[e] * inv, acc[e + 1] * inv);
    if (a.lse && lane == 0) a.lse[orow] = (M + log2f(Lsum)) * 0.69314718055994531f;
  }
}

// One CTA per (sequence, KV head, row tile) unit of a chunked launch.
__global__ void __launch_bounds__(128)
attn_big_merge_kernel(const AttnArgs a, int tpt, int max_rt, int nsplit) {
  int u = blockIdx.x;
  const int rt = u % max_rt; u /= max_rt;
  const int h = u % a.H_kv;
  const int b = u / a.H_kv;
  const int* pre = reinterpret_cast<const int*>(reinterpret_cast<const uint8_t*>(a.workspace) + kWsHeaderBytes);
  const float* ws_slots = reinterpret_cast<const float*>(
      reinterpret_cast<const uint8_t*>(a.workspace) + kWsHeaderBytes + ws_prefix_bytes());
  BigSeq s;
  big_seq(a, b, tpt, s);
  if (rt >= s.n_rt) return;
  // slot of chunk k = its item index
  const long long item0 = static_cast<long long>(pre[b]) * a.H_kv * nsplit +
                          static_cast<long long>(h) * nsplit * s.n_rt + rt;
  big_merge_unit(a, s, h, rt, tpt, nsplit, item0, s.n_rt, ws_slots);
}

// One CTA per unit of the cut last round of an unchunked launch (see big_tail); n_ctas is the grid
// of the attention kernel that wrote the partials.
__global__ void __launch_bounds__(128)
attn_big_tail_merge_kernel(const AttnArgs a, int tpt, int n_ctas) {
  const int* pre = reinterpret_cast<const int*>(reinterpret_cast<const uint8_t*>(a.workspace) + kWsHeaderBytes);
  const float* ws_slots = reinterpret_cast<const float*>(
      reinterpret_cast<const uint8_t*>(a.workspace) + kWsHeaderBytes + ws_prefix_bytes());
  const int units = pre[a.B] * a.H_kv;
  int u0, split;
  big_tail(units, n_ctas, 1, u0, split);
  const int u = u0 + static_cast<int>(blockIdx.x);
  if (split == 1 || u >= units) return;
  int lo = 0, hi = a.B;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (static_cast<long long>(pre[mid]) * a.H_kv <= u) lo = mid; else hi = mid;
  }
  BigSeq s;
  big_seq(a, lo, tpt, s);
  if (s.n_rt == 0) return;
  const int j = u - pre[lo] * a.H_kv;
  const int h = j / s.n_rt, rt = j - h * s.n_rt;
  big_merge_unit(a, s, h, rt, tpt, split, static_cast<long long>(blockIdx.x) * split, 1, ws_slots);
}

// Chunks per unit, from a small cost model in units of one tile's time: items are dealt
// round-robin and take about the same time, so a launch lasts ceil(items / CTAs) rounds of
// (tiles per item + a fixed start-up/epilogue cost); chunked launches also pay for writing and
// merging one partial per item.  Chunking is chosen only when it wins clearly.
int big_nsplit(int B, int H_kv, int max_rt, int n_ctas, int max_kv_len) {
  const long long units = static_cast<long long>(B) * H_kv * max_rt;
  if (units == 0) return 1;
  const double tiles = max_kv_len / kTile + 2.0;
  int best = 1;
  double best_cost = 0.0;
  for (int ns = 1; ns <= 16; ++ns) {
    if (ns > 1 && tiles / ns < 8.0) break;
    const long long items = units * ns;
    const long long rounds = (items + n_ctas - 1) / n_ctas;
    const double cost = rounds * (tiles / ns + 4.0) + (ns > 1 ? 0.015 * items : 0.0);
    if (ns == 1 || cost < 0.92 * best_cost) { best = ns; best_cost = cost; }
  }
  return best;
}

}  // namespace

// Large blocks, and step blocks with more than 64 packed rows (where two softmax warpgroups per
// tile beat the one of the rows-on-lanes step kernel: 5.9 against 4.2 TB/s at 128 rows).
bool attn_umma_big_supports(int D, int G, int max_nq) {
  return D == kBD && G >= 1 && G <= kMaxGroup && max_nq <= kMaxNqBig && (max_nq > kMaxNq || G * max_nq > 64);
}

size_t attn_umma_big_workspace_bytes(int B, int H_kv, int G, int max_nq, int max_kv_len, int n_ctas) {
  const int tpt = kTile / G, max_rt = (max_nq + tpt - 1) / tpt;
  const int nsplit = big_nsplit(B, H_kv, max_rt, n_ctas, max_kv_len);
  // chunked launch: one partial per item; otherwise at most one per CTA for the cut last round
  const size_t slots = nsplit > 1 ? static_cast<size_t>(B) * H_kv * max_rt * nsplit : static_cast<size_t>(n_ctas);
  return kWsHeaderBytes + ws_prefix_bytes() + slots * big_slot_floats() * sizeof(float);
}

int32_t launch_attn_umma_big(const AttnArgs& a, cudaStream_t st) {
  if (a.B == 0 || a.T == 0) return MS_OK;
  if (a.D != kBD || a.G > kMaxGroup || a.max_nq > kMaxNqBig) return MS_ERR_UNSUPPORTED_SHAPE;
  const int tpt = kTile / a.G;                   // tokens per row tile
  const int max_rt = (a.max_nq + tpt - 1) / tpt;
  const int grid = attn_mma_grid();
  if (grid <= 0) return cuda_status(cudaErrorNoDevice);
  const int nsplit = big_nsplit(a.B, a.H_kv, max_rt, grid, a.max_kv_len);
  if (static_cast<long long>(a.B) * a.H_kv * max_rt * nsplit > 0x7fffffffLL) return MS_ERR_UNSUPPORTED_SHAPE;
  CUtensorMap mk, mv, mks, mvs, mq;
  const bool ok =
      make_map(&mk, a.k_cache, a.D, static_cast<uint64_t>(a.n_slots), a.H_kv, a.D, a.kv_head_stride, kTile, 1) &&
      make_map(&mv, a.v_cache, a.D, static_cast<uint64_t>(a.n_slots), a.H_kv, a.D, a.kv_head_stride, kTile, 1) &&
      make_map(&mks, a.k_step, a.D, a.H_kv, a.T, a.D, static_cast<uint64_t>(a.H_kv) * a.D, 1, kTile) &&
      make_map(&mvs, a.v_step, a.D, a.H_kv, a.T, a.D, static_cast<uint64_t>(a.H_kv) * a.D, 1, kTile) &&
      make_map(&mq, a.q, a.D, a.H_q, a.T, a.D, static_cast<uint64_t>(a.H_q) * a.D, a.G, tpt);
  if (!ok) return cuda_status(cudaErrorInvalidValue);
  static bool configured[64] = {false};
  int dev = 0;
  MS_CUDA_TRY(cudaGetDevice(&dev));
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    MS_CUDA_TRY(cudaFuncSetAttribute(attn_umma_big_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kBSmem));
    configured[dev] = true;
  }
  int* pre = reinterpret_cast<int*>(reinterpret_cast<uint8_t*>(a.workspace) + kWsHeaderBytes);
  attn_big_plan_kernel<<<1, 256, 0, st>>>(a, tpt, pre);
  MS_LAUNCH_CHECK();
  if (a.ev_split_begin) MS_CUDA_TRY(cudaEventRecord(a.ev_split_begin, st));
  attn_umma_big_kernel<<<grid, kBThreads, kBSmem, st>>>(a, mk, mv, mks, mvs, mq, tpt, nsplit);
  MS_LAUNCH_CHECK();
  if (a.ev_split_end) MS_CUDA_TRY(cudaEventRecord(a.ev_split_end, st));
  if (nsplit > 1) {
    const long long units = static_cast<long long>(a.B) * a.H_kv * max_rt;
    attn_big_merge_kernel<<<static_cast<unsigned>(units), 128, 0, st>>>(a, tpt, max_rt, nsplit);
    MS_LAUNCH_CHECK();
  } else if (static_cast<long long>(a.B) * a.H_kv * max_rt > grid) {
    // more units than CTAs are possible: the last round may have been cut (the kernel decides from
    // the actual block sizes; CTAs of this grid beyond the cut units return at once)
    attn_big_tail_merge_kernel<<<grid, 128, 0, st>>>(a, tpt, grid);
    MS_LAUNCH_CHECK();
  }
  return MS_OK;
}

}  // namespace ms
