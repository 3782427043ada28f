// Keys-on-lanes tcgen05 split-KV path of the MemoSight step attention (sm_100a).
//
// The step block of MemoSight (paper Sec. 2.1.1) is small -- n_q*G = 8..64 packed
// query rows per KV head -- while a K/V tile is 128 keys.  Putting the query rows
// on the 128 rows of the MMA tile would leave most tensor-memory lanes (and with
// them most of the four SM sub-partitions, each of which can only reach its own
// 32 lanes) idle in the softmax.  This kernel therefore computes the transposed
// problem, the tile's 128 keys on the lanes:
//     S^T[key][row] = K_tile (A, K-major)   x  Q^T (B = Q, K-major)      N = rows padded to 16
//     O^T[d][row]  += V_tile^T (A, MN-major) x  P^T (B, MN-major)         M = D = 128
// so that every softmax thread owns one key of the tile and touches only as many
// score columns as there are query rows: the softmax cost follows the block size
// and all four sub-partitions work on every tile.  The mask is then a per-thread
// predicate (key index against the valid length; the (n_cand, anchor) rule on the
// step-local tile).
//
// Row statistics need the keys of all lanes:
//   * the reference maximum m_ref[row] is the exact row maximum of the unit's first
//     tile (redux.sync.max per warp, combined through shared memory); later tiles
//     are exponentiated against it unchanged.  Any shift is exact for a softmax as
//     long as nothing overflows, so m_ref only moves when a score exceeds it by
//     more than 2^48: the four softmax warps agree on that each tile through one
//     mbarrier round, and then rescale O^T and the partial sums together (rare).
//   * the row sums stay per thread (one partial per key lane and row) and are
//     reduced across lanes once, at the end of the unit.
// Roles, pipeline, schedule, workspace format and bounded waits are those of the
// rows-on-lanes kernel (attn_umma.cu); head_dim is 128.
#include "attn_umma_common.cuh"

namespace ms {
namespace {

constexpr int kTThreads = 384;   // warp 0: TMA, warp 1: MMA issue, 4-7 and 8-11: the two softmax warpgroups
constexpr float kGrowLimit = 48.f;
constexpr int kTMaxKv = 8;
constexpr int kPBytes = kTile * 128;            // P^T tile: 128 keys x 64 columns of bf16
constexpr int kKvBytes = kTile * 128 * 2;       // K or V tile, D = 128
constexpr uint32_t kHalfStrideT = kTile * 128;  // bytes between the 64-column halves of a K/V tile

enum : int {
  kTbKvFull = 0, kTbKvEmpty = kTMaxKv, kTbQFull = 2 * kTMaxKv, kTbQEmpty = kTbQFull + 2,
  kTbSFull = kTbQEmpty + 2, kTbPFull = kTbSFull + 2, kTbPvDone = kTbPFull + 2, kTbWg = kTbPvDone + 2,
  kTbDrain = kTbWg + 2, kTbCount = kTbDrain + 1
};
// misc region behind the ring: barriers | scalars | m_ref[64] | red[2 warpgroups][4 warps][32 rows]
constexpr int kMiscScalars = 256, kMiscMref = 512, kMiscRed = 768, kMiscBytes = 2048;
static_assert(kTbCount * 8 <= kMiscScalars, "barriers overflow their slot");

struct TLayout {
  int rows_box;      // rows one Q box holds: G * max_nq
  int q_half, q_bytes, n_kv;
  int off_q, off_p, off_kv, off_misc, total;
};

// Sum of v[j] over the 32 lanes for 32 rows at once: lane L ends up with the total of row L.
__device__ __forceinline__ float warp_sum_32rows(float (&t)[32], int lane) {
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) {
    const bool up = (lane & o) != 0;
#pragma unroll
    for (int i = 0; i < o; ++i) {
      const float send = up ? t[i] : t[i + o];
      const float keep = up ? t[i + o] : t[i];
      t[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
    }
  }
  return t[0];
}

template <int NP>
__global__ void __launch_bounds__(kTThreads, 1)
attn_umma_t_kernel(const AttnArgs a, const __grid_constant__ CUtensorMap map_k,
                   const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_ks,
                   const __grid_constant__ CUtensorMap map_vs, const __grid_constant__ CUtensorMap map_q,
                   int rows_pad, const TLayout lay) {
  constexpr int D = 128, HALVES = 2, KSTEPS_QK = D / 16;
  constexpr int CW = NP / 2;                        // rows (score columns) per softmax warpgroup
  // the separate loop of plain tiles in the softmax warps: with 32 rows per warpgroup the second copy
  // of the tile body pushes the register allocation into spills, which costs more than the walker
  constexpr bool kPlainSoftmax = NP < 64;
  constexpr uint32_t kCols = NP <= 16 ? 64 : (NP <= 32 ? 128 : 256);   // S^T x2 and O^T, a power of two
  constexpr uint32_t kColO = 2 * NP;
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sb = smem_u32(smem);
  const uint32_t bars = sb + lay.off_misc;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + lay.off_misc + kMiscScalars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + lay.off_misc + kMiscScalars + 8);
  volatile int* grow_flags = reinterpret_cast<volatile int*>(smem + lay.off_misc + kMiscScalars + 16);
  float* s_mref = reinterpret_cast<float*>(smem + lay.off_misc + kMiscMref);
  float* s_red = reinterpret_cast<float*>(smem + lay.off_misc + kMiscRed);
  uint32_t* status = reinterpret_cast<uint32_t*>(a.workspace);
  int* ws_pre = reinterpret_cast<int*>(reinterpret_cast<uint8_t*>(a.workspace) + kWsHeaderBytes);
  float* ws_slots = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(a.workspace) + kWsHeaderBytes +
                                             ws_prefix_bytes());
  volatile int* last_flags = reinterpret_cast<volatile int*>(smem + lay.off_misc + kMiscScalars + 24);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (sb & 1023u) {
    pdl_wait();
    if (threadIdx.x == 0) atomicExch(status, kTimeoutMagic + 1);
    return;
  }

  // ---- set-up that touches no global memory: barriers, tensor memory ----
  if (threadIdx.x == 0) {
    for (int i = 0; i < kTMaxKv; ++i) {
      mbar_init(bars + 8 * (kTbKvFull + i), 1);
      mbar_init(bars + 8 * (kTbKvEmpty + i), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bars + 8 * (kTbQFull + i), 1);
      mbar_init(bars + 8 * (kTbQEmpty + i), 1);
      mbar_init(bars + 8 * (kTbSFull + i), 1);
      mbar_init(bars + 8 * (kTbPFull + i), 8);
      mbar_init(bars + 8 * (kTbPvDone + i), 1);
    }
    mbar_init(bars + 8 * kTbWg, 4);
    mbar_init(bars + 8 * (kTbWg + 1), 4);
    mbar_init(bars + 8 * kTbDrain, 1);
    wait_ctx_init(abort_flag, a.wait_limit_us);
    grow_flags[0] = 0;
    grow_flags[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(tmem_slot)), "r"(kCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // Rows of the Q buffers past the box are never loaded; as B rows they only feed the padded
  // score columns, which must stay finite: clear them once.
  {
    const int pad_rows = NP - lay.rows_box;
    for (int x = threadIdx.x; x < pad_rows * 2 * HALVES * 8; x += blockDim.x) {
      const int c = x & 7, rest = x >> 3;
      const int rr = lay.rows_box + rest % pad_rows, buf_half = rest / pad_rows;   // 0..3
      const uint32_t addr = sb + lay.off_q + (buf_half >> 1) * lay.q_bytes + (buf_half & 1) * lay.q_half +
                            rr * 128 + (c << 4);
      asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(addr), "r"(0u) : "memory");
    }
    fence_async_smem();
  }
  // ---- from here on global memory is read: the grid before this one must have finished ----
  pdl_wait();
  pdl_trigger();

  // ---- schedule (the prefix lives where the K/V ring will be) ----
  int* s_pre = reinterpret_cast<int*>(smem + lay.off_kv);
  int* s_scratch = s_pre + a.B + 1;
  build_tile_prefix(a, s_pre, s_scratch);
  const long long per_layer = static_cast<long long>(s_pre[a.B]) * a.H_kv;
  const long long n_tiles = per_layer * a.n_layers;
  const long long t0 = n_tiles * blockIdx.x / gridDim.x;
  const long long t1 = n_tiles * (blockIdx.x + 1) / gridDim.x;
  const int n_iter = static_cast<int>(t1 - t0);
  if (blockIdx.x == 0 && !a.done) {
    for (int i = threadIdx.x; i <= a.B; i += blockDim.x) ws_pre[i] = s_pre[i];
  }
  Walk w0;
  w0.n_iter = 0;
  if (n_iter > 0) {
    const int layer0 = static_cast<int>(t0 / per_layer);
    const long long rem = t0 - layer0 * per_layer;
    int lo = 0, hi = a.B;
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (static_cast<long long>(s_pre[mid]) * a.H_kv <= rem) lo = mid; else hi = mid;
    }
    walk_init(a, w0, lo, rem - static_cast<long long>(s_pre[lo]) * a.H_kv, n_iter, layer0);
  }
  tc_fence_before();
  __syncthreads();   // the prefix has been consumed; barriers, tensor memory and the Q padding are ready
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0 && lane == 0 && n_iter > 0) {
    // =========================== TMA producer ===========================
    Walk w = w0;
    bool ok = true;
    int uses = 0, pieces = 0;
    RingPos rp;
    rp.init(0, lay.n_kv);
    while (w.it < n_iter) {
      walk_tile(a, w);
      if (w.first) {
        const int qb = w.piece_idx & 1;
        if (!mbar_wait(bars + 8 * (kTbQEmpty + qb), ((w.piece_idx >> 1) & 1) ^ 1, abort_flag, status)) {
          ok = false;
          break;
        }
        fence_async_smem();
        const uint32_t bar = bars + 8 * (kTbQFull + qb);
        mbar_arrive_expect_tx(bar, static_cast<uint32_t>(HALVES * lay.rows_box * 128));
#pragma unroll
        for (int hf = 0; hf < HALVES; ++hf)
          tma_load_4d(sb + lay.off_q + qb * lay.q_bytes + hf * lay.q_half, &map_q, bar, hf * 64, w.h * a.G,
                      w.r0, w.layer);
        ++pieces;
      }
#pragma unroll 1
      for (int kv = 0; kv < 2; ++kv) {
        const int buf = rp.buf;
        if (!mbar_wait(bars + 8 * (kTbKvEmpty + buf), rp.par ^ 1u, abort_flag, status)) {
          ok = false;
          break;
        }
        rp.step(1);
        fence_async_smem();
        const uint32_t dst = sb + lay.off_kv + buf * kKvBytes;
        const uint32_t bar = bars + 8 * (kTbKvFull + buf);
        if (w.is_step) {
          mbar_arrive_expect_tx(bar, static_cast<uint32_t>(HALVES * kMaxNq * 128));
#pragma unroll
          for (int hf = 0; hf < HALVES; ++hf)
            tma_load_4d(dst + hf * kHalfStrideT, kv ? &map_vs : &map_ks, bar, hf * 64, w.h, w.r0, w.layer);
        } else {
          mbar_arrive_expect_tx(bar, static_cast<uint32_t>(kKvBytes));
          const int y = static_cast<int>(w.slot_off) + w.ti * kTile;
#pragma unroll
          for (int hf = 0; hf < HALVES; ++hf)
            tma_load_4d(dst + hf * kHalfStrideT, kv ? &map_v : &map_k, bar, hf * 64, y, w.h, w.layer);
        }
        ++uses;
      }
      if (!ok) break;
      walk_next(a, w);
    }
    // Drain: every copy issued here must have landed before the CTA may exit.
    for (int u = uses > lay.n_kv ? uses - lay.n_kv : 0; u < uses; ++u)
      (void)mbar_wait(bars + 8 * (kTbKvFull + u % lay.n_kv), (u / lay.n_kv) & 1, abort_flag, status);
    for (int p = pieces > 2 ? pieces - 2 : 0; p < pieces; ++p)
      (void)mbar_wait(bars + 8 * (kTbQFull + (p & 1)), (p >> 1) & 1, abort_flag, status);
  } else if (warp == 1 && n_iter > 0) {
    // =========================== MMA issuer ===========================
    // The whole warp walks the schedule in step, so that addresses and descriptors are the same in
    // every lane; one elected lane (always the same one) issues the tensor-core instructions.
    auto mwait = [&](uint32_t bar, uint32_t parity) -> bool {
      return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag, status));
    };
    // S^T = K Q^T: A = K tile (K-major), B = Q (K-major).  O^T += V^T P^T: A = V tile transposed
    // (MN-major), B = P^T (MN-major).  Q K^T runs one tile ahead of the PV product, so the tensor
    // pipe has the scores of tile t+1 ready while the softmax of tile t is in flight.  The
    // descriptors differ from MMA to MMA only by a constant in their low word.
    const uint32_t idesc_qk = instr_desc(NP, 0, 0), idesc_pv = instr_desc(NP, 1, 1);
    const uint32_t q_lo0 = desc_lo(sb + lay.off_q, 16), k_lo0 = desc_lo(sb + lay.off_kv, 16);
    const uint32_t p_lo0 = desc_lo(sb + lay.off_p, kHalfStrideT), v_lo0 = desc_lo(sb + lay.off_kv, kHalfStrideT);
    Walk wq = w0, wp = w0;
    RingPos rk, rv;
    rk.init(0, lay.n_kv);
    rv.init(1, lay.n_kv);
    bool ok = true;
    auto issue_qk = [&]() -> bool {
      walk_tile(a, wq);
      const int it = wq.it, qb = wq.piece_idx & 1;
      if ((wq.first && !mwait(bars + 8 * (kTbQFull + qb), (wq.piece_idx >> 1) & 1)) ||
          !mwait(bars + 8 * (kTbKvFull + rk.buf), rk.par))
        return false;
      tc_fence_after();
      const uint32_t q_lo = q_lo0 + qb * (lay.q_bytes >> 4);
      const uint32_t k_lo = k_lo0 + rk.buf * (kKvBytes >> 4);
      const uint32_t d_s = tmem + (it & 1) * NP;
#pragma unroll
      for (int ks = 0; ks < KSTEPS_QK; ++ks)
        umma_bf16_lo_elect(d_s, k_lo + (ks >> 2) * (kHalfStrideT >> 4) + (ks & 3) * 2,
                     q_lo + (ks >> 2) * (NP * 128 >> 4) + (ks & 3) * 2, idesc_qk, ks > 0);
      umma_commit_elect(bars + 8 * (kTbKvEmpty + rk.buf));
      umma_commit_elect(bars + 8 * (kTbSFull + (it & 1)));
      if (wq.last) umma_commit_elect(bars + 8 * (kTbQEmpty + qb));
      rk.step(2);
      walk_next(a, wq);
      return true;
    };
    ok = issue_qk();
    while (ok && wp.it < n_iter) {
      // ---- a run of plain tiles needs neither walker.  S^T of a tile that neither opens nor closes
      //      its piece is the same eight MMAs whatever the tile holds; O^T += V^T P^T of a full cache
      //      tile that does not open its piece is eight accumulating MMAs.  Nearly every tile of a
      //      long cache goes through this loop, whose only branches are the waits and the back edge.
      if (wq.open && wp.open && wq.it == wp.it + 1) {
        int n_run = min(min(wq.tiles_b - 1 - wq.ti, n_iter - 1 - wq.it), wp.L / kTile - wp.ti);
        const uint32_t q_lo = q_lo0 + (wq.piece_idx & 1) * (lay.q_bytes >> 4);
        int it = wp.it;
        for (; n_run > 0; --n_run, ++it) {
          // S^T(it + 1)
          if (!mwait(bars + 8 * (kTbKvFull + rk.buf), rk.par)) { ok = false; break; }
          tc_fence_after();
          {
            const uint32_t k_lo = k_lo0 + rk.buf * (kKvBytes >> 4);
            const uint32_t d_s = tmem + ((it + 1) & 1) * NP;
#pragma unroll
            for (int ks = 0; ks < KSTEPS_QK; ++ks)
              umma_bf16_lo_elect(d_s, k_lo + (ks >> 2) * (kHalfStrideT >> 4) + (ks & 3) * 2,
                           q_lo + (ks >> 2) * (NP * 128 >> 4) + (ks & 3) * 2, idesc_qk, ks > 0);
            umma_commit_elect(bars + 8 * (kTbKvEmpty + rk.buf));
            umma_commit_elect(bars + 8 * (kTbSFull + ((it + 1) & 1)));
            rk.step(2);
          }
          // O^T += V^T P^T (it)
          if (!mwait(bars + 8 * (kTbPFull + (it & 1)), (it >> 1) & 1) ||
              !mwait(bars + 8 * (kTbKvFull + rv.buf), rv.par)) {
            ok = false;
            break;
          }
          tc_fence_after();
          {
            const uint32_t p_lo = p_lo0 + (it & 1) * (kPBytes >> 4);
            const uint32_t v_lo = v_lo0 + rv.buf * (kKvBytes >> 4);
#pragma unroll
            for (int j = 0; j < kTile / 16; ++j)
              umma_bf16_lo_elect(tmem + kColO, v_lo + j * (2048 >> 4), p_lo + j * (2048 >> 4), idesc_pv, 1u);
            umma_commit_elect(bars + 8 * (kTbKvEmpty + rv.buf));
            umma_commit_elect(bars + 8 * (kTbPvDone + (it & 1)));
            rv.step(2);
          }
        }
        if (!ok) break;
        const int done = it - wp.it;
        wq.ti += done; wq.it += done; wq.piece_j += done;
        wp.ti += done; wp.it += done; wp.piece_j += done;
        if (wp.it >= n_iter) break;
      }
      // score buffer (it+1)&1 is free: the P^T of tile it-1 was waited for in the previous round
      if (wq.it < n_iter && !issue_qk()) { ok = false; break; }
      walk_tile(a, wp);
      const int it = wp.it;
      if (!mwait(bars + 8 * (kTbPFull + (it & 1)), (it >> 1) & 1) ||
          !mwait(bars + 8 * (kTbKvFull + rv.buf), rv.par)) {
        ok = false;
        break;
      }
      tc_fence_after();
      const uint32_t p_lo = p_lo0 + (it & 1) * (kPBytes >> 4);
      const uint32_t v_lo = v_lo0 + rv.buf * (kKvBytes >> 4);
      const int ksteps = wp.is_step ? 1 : (wp.nvalid + 15) >> 4;
      const uint32_t acc0 = wp.first ? 0u : 1u;
      if (ksteps == kTile / 16) {
#pragma unroll
        for (int j = 0; j < kTile / 16; ++j)
          umma_bf16_lo_elect(tmem + kColO, v_lo + j * (2048 >> 4), p_lo + j * (2048 >> 4), idesc_pv, j == 0 ? acc0 : 1u);
      } else {
#pragma unroll 1
        for (int j = 0; j < ksteps; ++j)
          umma_bf16_lo_elect(tmem + kColO, v_lo + j * (2048 >> 4), p_lo + j * (2048 >> 4), idesc_pv, j == 0 ? acc0 : 1u);
      }
      umma_commit_elect(bars + 8 * (kTbKvEmpty + rv.buf));
      umma_commit_elect(bars + 8 * (kTbPvDone + (it & 1)));
      rv.step(2);
      walk_next(a, wp);
    }
    if (!ok) {
      // aborting: let the tensor pipe run dry before tensor memory is released
      umma_commit_elect(bars + 8 * kTbDrain);
      const unsigned long long t_begin = global_ns();
      while (!mbar_try_wait(bars + 8 * kTbDrain, 0) && global_ns() - t_begin < wait_limit_ns(abort_flag)) {
      }
    }
  } else if (warp >= 4 && n_iter > 0) {
    // ============ softmax warps: thread = key of the tile; warpgroup = half of the rows ============
    // Rows (score columns) are independent of one another, so the two warpgroups never talk:
    // each has its own references, partial sums, agreement barrier and share of every P^T row.
    const int wg = (warp - 4) >> 2, quad = (warp - 4) & 3;
    const int t = quad * 32 + lane;                        // key index in the tile = TMEM lane
    const int c0 = wg * CW;                                // first row (score column) of this warpgroup
    const uint32_t lane_addr = tmem + (static_cast<uint32_t>(quad * 32) << 16);
    const uint32_t tx = t & 7;
    float* red_w = s_red + (wg * 4 + quad) * 32;
    const float* red_g = s_red + wg * 128;                 // this warpgroup's four slices
    float* mref_g = s_mref + c0;
    volatile int* grow_flag = grow_flags + wg;
    const uint32_t bar_wg = bars + 8 * (kTbWg + wg);
    Walk w = w0;
    float lsum[CW];
    uint32_t wg_phase = 0;
    int plain_left = 0;        // plain tiles ahead in the current run (used where the tile body exists once)
    bool ok = true;
    auto wait_all = [&](uint32_t bar, uint32_t parity) -> bool {
      return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag, status));
    };
    // bounded barrier of the warpgroup's four warps (also publishes their shared-memory writes)
    auto wg_sync = [&]() -> bool {
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_wg);
      const bool good = wait_all(bar_wg, wg_phase & 1);
      ++wg_phase;
      return good;
    };
    // scores of this key against the warpgroup's rows; invisible pairs become -inf
    auto load_scores = [&](float (&v)[CW], uint32_t s_addr, int nv, bool is_step) {
      uint32_t raw[CW];
#pragma unroll
      for (int c = 0; c < CW / 8; ++c) tmem_ld8(s_addr + c * 8, raw + c * 8);
#pragma unroll
      for (int c = 0; c < CW / 8; ++c) tmem_ld_wait8(raw + c * 8);
      const bool key_ok = t < nv;
      if (!is_step) {
#pragma unroll
        for (int j = 0; j < CW; ++j) v[j] = key_ok ? __uint_as_float(raw[j]) : -INFINITY;
      } else {
        int i = c0 / a.G, g = c0 - i * a.G;
#pragma unroll
        for (int j = 0; j < CW; ++j) {
          bool vis = false;
          if (key_ok && i < w.n_q) {
            const int anc = (i < w.n_c) ? i : (a.anchor ? a.anchor[w.r0 + i] : w.n_c);
            vis = step_key_visible(i, t, w.n_c, anc);
          }
          v[j] = vis ? __uint_as_float(raw[j]) : -INFINITY;
          if (++g == a.G) { g = 0; ++i; }
        }
      }
    };
    // exact maximum over the tile's keys of every row -> red[warp][row]
    auto reduce_row_max = [&](const float (&v)[CW]) {
      float keep = -INFINITY;
#pragma unroll
      for (int j = 0; j < CW; ++j) {
        const float r = warp_max_f32(v[j]);
        if (lane == j) keep = r;
      }
      red_w[lane] = keep;
    };
    auto red_max4 = [&](int j) -> float {
      return fmaxf(fmaxf(red_g[j], red_g[32 + j]), fmaxf(red_g[64 + j], red_g[96 + j]));
    };
    // x = s * scale - m_ref (log2 units); returns the largest x of this thread
    auto shift_scores = [&](float (&v)[CW]) -> float {
      float tmaxx = -INFINITY;
#pragma unroll
      for (int j4 = 0; j4 < CW / 4; ++j4) {
        const float4 m4 = *reinterpret_cast<const float4*>(mref_g + 4 * j4);
        v[4 * j4 + 0] = fmaf(v[4 * j4 + 0], a.scale_log2, -m4.x);
        v[4 * j4 + 1] = fmaf(v[4 * j4 + 1], a.scale_log2, -m4.y);
        v[4 * j4 + 2] = fmaf(v[4 * j4 + 2], a.scale_log2, -m4.z);
        v[4 * j4 + 3] = fmaf(v[4 * j4 + 3], a.scale_log2, -m4.w);
        tmaxx = fmaxf(tmaxx, fmaxf(fmaxf(v[4 * j4], v[4 * j4 + 1]), fmaxf(v[4 * j4 + 2], v[4 * j4 + 3])));
      }
      return tmaxx;
    };
    // ---- rare: move the references up, rescale O^T and the partial sums, redo x ----
    auto regrow = [&](float (&v)[CW], int it, uint32_t s_addr, int nv, bool is_step) -> bool {
      load_scores(v, s_addr, nv, is_step);
      reduce_row_max(v);
      if (!wg_sync()) return false;
      float alpha[CW];
#pragma unroll
      for (int j = 0; j < CW; ++j) {
        const float m = red_max4(j);
        const float m_old = mref_g[j];
        const float m_new = (m == -INFINITY) ? m_old : fmaxf(m_old, m * a.scale_log2);
        alpha[j] = ex2(m_old - m_new);
        lsum[j] *= alpha[j];
        v[j] = fmaf(v[j], a.scale_log2, -m_new);
      }
      if (!wg_sync()) return false;          // everyone has read the old references
      if (t < CW) {
        const float m = red_max4(t);
        if (m != -INFINITY) mref_g[t] = fmaxf(mref_g[t], m * a.scale_log2);
      }
      // all PV products issued so far are complete before O^T is touched
      if (!wait_all(bars + 8 * (kTbPvDone + ((it - 1) & 1)), ((it - 1) >> 1) & 1)) return false;
      tc_fence_after();
      {
        uint32_t o[CW];
#pragma unroll
        for (int c = 0; c < CW / 8; ++c) tmem_ld8(lane_addr + kColO + c0 + c * 8, o + c * 8);
#pragma unroll
        for (int c = 0; c < CW / 8; ++c) tmem_ld_wait8(o + c * 8);
#pragma unroll
        for (int j = 0; j < CW; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * alpha[j]);
#pragma unroll
        for (int c = 0; c < CW / 8; ++c) tmem_st8(lane_addr + kColO + c0 + c * 8, o + c * 8);
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      }
      return wg_sync();                      // new references visible to later tiles
    };
    // p = 2^x as bf16 into this key's row of the P^T tile; partial row sums stay in registers
    auto emit_p = [&](const float (&v)[CW], int pb) {
      const uint32_t p_row = sb + lay.off_p + pb * kPBytes + t * 128;
#pragma unroll
      for (int c = 0; c < CW / 8; ++c) {
        float p[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          p[e] = ex2(v[c * 8 + e]);
          lsum[c * 8 + e] += p[e];
        }
        const uint32_t addr = p_row + (((c0 / 8 + c) ^ tx) << 4);
        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(pack2(p[0], p[1])),
                     "r"(pack2(p[2], p[3])), "r"(pack2(p[4], p[5])), "r"(pack2(p[6], p[7]))
                     : "memory");
      }
    };
    // hands the P^T rows of this warp to the MMA thread
    auto publish_p = [&](int pb) {
      fence_async_smem();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bars + 8 * (kTbPFull + pb));
    };
    while (ok && w.it < n_iter) {
      // ---- a run of plain tiles: full cache tiles that neither open nor close the piece need no
      //      walker, no mask and none of the unit's begin / end work
      if (kPlainSoftmax && w.open) {
        int n_run = min(w.L / kTile - w.ti, n_iter - 1 - w.it);
        for (; n_run > 0; --n_run) {
          const int it = w.it, pb = it & 1;
          // (the commit behind these scores also covers O^T += V^T P^T of tile it - 2: its P^T buffer is free)
          if (!wait_all(bars + 8 * (kTbSFull + pb), (it >> 1) & 1)) { ok = false; break; }
          tc_fence_after();
          const uint32_t s_addr = lane_addr + pb * NP + c0;
          float v[CW];
          {
            uint32_t raw[CW];
#pragma unroll
            for (int c = 0; c < CW / 8; ++c) tmem_ld8(s_addr + c * 8, raw + c * 8);
#pragma unroll
            for (int c = 0; c < CW / 8; ++c) tmem_ld_wait8(raw + c * 8);
#pragma unroll
            for (int j = 0; j < CW; ++j) v[j] = __uint_as_float(raw[j]);
          }
          const float tmaxx = shift_scores(v);
          if (__any_sync(0xffffffffu, tmaxx > kGrowLimit) && lane == 0) *grow_flag = it + 1;
          if (!wg_sync()) { ok = false; break; }
          if (*grow_flag == it + 1 && !regrow(v, it, s_addr, kTile, false)) { ok = false; break; }
          emit_p(v, pb);
          publish_p(pb);
          ++w.ti;
          ++w.it;
          ++w.piece_j;
        }
        if (!ok) break;
      }
      // Without the separate loop above, a plain tile at least skips the schedule walker: the same
      // tile body runs with the facts of a full cache tile in the middle of its piece.
      bool plain = false;
      if (!kPlainSoftmax) {
        if (plain_left <= 0 && w.open) plain_left = min(w.L / kTile - w.ti, n_iter - 1 - w.it);
        plain = plain_left > 0;
      }
      if (!plain) walk_tile(a, w);
      const int it = w.it, pb = it & 1;
      if (!wait_all(bars + 8 * (kTbSFull + pb), (it >> 1) & 1)) { ok = false; break; }
      tc_fence_after();
      const int nv = plain ? kTile : w.nvalid;
      const bool is_step = plain ? false : w.is_step;
      const bool opens = plain ? false : (w.piece_j == 0);
      const bool closes = plain ? false : w.last;
      const uint32_t s_addr = lane_addr + pb * NP + c0;
      float v[CW];
      load_scores(v, s_addr, nv, is_step);

      if (opens) {
        // new unit: the reference maximum of each row is the exact maximum of this first tile
        reduce_row_max(v);
        if (!wg_sync()) { ok = false; break; }
        if (t < CW) {
          const float m = red_max4(t);
          mref_g[t] = (m == -INFINITY) ? 0.f : m * a.scale_log2;
        }
        if (!wg_sync()) { ok = false; break; }
#pragma unroll
        for (int j = 0; j < CW; ++j) lsum[j] = 0.f;
      }

      const float tmaxx = shift_scores(v);
      if (!opens) {
        // the four warps agree on whether any score outgrew its reference (tile index as the token);
        // a piece's first tile set the references from its own scores and cannot outgrow them
        if (__any_sync(0xffffffffu, tmaxx > kGrowLimit) && lane == 0) *grow_flag = it + 1;
        if (!wg_sync()) { ok = false; break; }
        if (*grow_flag == it + 1 && !regrow(v, it, s_addr, nv, is_step)) { ok = false; break; }
      }
      emit_p(v, pb);
      if (is_step || nv < kTile) {
        // V rows past the valid keys hold foreign or stale bytes; their P is 0 but 0 * NaN is NaN:
        // clear the rows of the last 16-key step that the PV product still reads.  Done behind the
        // exponentials, so that the wait for the V tile (which lands after the K tile) overlaps them,
        // and before P^T is handed over, so that the product sees the cleared rows.
        const int use = 2 * it + 1, buf = use % lay.n_kv;
        if (!wait_all(bars + 8 * (kTbKvFull + buf), (use / lay.n_kv) & 1)) { ok = false; break; }
        const uint32_t va = sb + lay.off_kv + buf * kKvBytes;
        const int n_rows = ((nv + 15) & ~15) - nv;
        for (int x = wg * 128 + t; x < n_rows * HALVES * 8; x += 256) {
          const int rr = nv + x / (HALVES * 8), cc = x % (HALVES * 8);
          const uint32_t addr = va + (cc >> 3) * kHalfStrideT + rr * 128 + ((cc & 7) << 4);
          asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(addr), "r"(0u) : "memory");
        }
      }
      publish_p(pb);
      if (plain) {
        ++w.ti;
        ++w.it;
        ++w.piece_j;
        --plain_left;
        continue;
      }

      if (closes) {
        // ---- end of the unit (or of this CTA's part of it) ----
        // row sums: over the 32 lanes of each warp, then over the four warps
        {
          float tsum[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) tsum[i] = (i < CW) ? lsum[i < CW ? i : 0] : 0.f;
          red_w[lane] = warp_sum_32rows(tsum, lane);
        }
        if (!wg_sync()) { ok = false; break; }
        const int rows = w.n_q * a.G;
        float l_row[CW];
#pragma unroll
        for (int j = 0; j < CW; ++j) l_row[j] = (red_g[j] + red_g[32 + j]) + (red_g[64 + j] + red_g[96 + j]);
        // thread t < CW also owns the statistics of row c0 + t (written once, outside the row loop below,
        // where a per-row "if (t == j)" made one warp walk 32 divergent branches)
        const float m_mine = (t < CW) ? mref_g[t] : 0.f;
        const float l_mine = (t < CW) ? (red_g[t] + red_g[32 + t]) + (red_g[64 + t] + red_g[96 + t]) : 1.f;
        if (!wg_sync()) { ok = false; break; }          // red and m_ref may be reused from here on
        if (!wait_all(bars + 8 * (kTbPvDone + pb), (it >> 1) & 1)) { ok = false; break; }
        tc_fence_after();
        uint32_t o[CW];
#pragma unroll
        for (int c = 0; c < CW / 8; ++c) tmem_ld8(lane_addr + kColO + c0 + c * 8, o + c * 8);
#pragma unroll
        for (int c = 0; c < CW / 8; ++c) tmem_ld_wait8(o + c * 8);
        // thread t holds element d = t of every row
        __nv_bfloat16* out_l = a.out + w.layer * a.out_layer_stride;
        float* lse_l = a.lse ? a.lse + w.layer * a.lse_layer_stride : nullptr;
        if (w.slot < 0) {
          const int i0 = c0 / a.G;
          int g = c0 - i0 * a.G;
          int64_t orow = static_cast<int64_t>(w.r0 + i0) * a.H_q + w.h * a.G + g;
          const int64_t next_token = a.H_q - a.G + 1;      // from the last head of a token's group to the first of the next
#pragma unroll
          for (int j = 0; j < CW; ++j) {
            if (c0 + j < rows) {
              out_l[orow * D + t] = __float2bfloat16_rn(__uint_as_float(o[j]) * __frcp_rn(l_row[j]));
            }
            if (++g == a.G) { g = 0; orow += next_token; } else { ++orow; }
          }
          if (lse_l && t < CW && c0 + t < rows) {
            const int r = c0 + t, i = r / a.G;
            lse_l[static_cast<int64_t>(w.r0 + i) * a.H_q + w.h * a.G + (r - i * a.G)] =
                (m_mine + log2f(l_mine)) * 0.69314718055994531f;
          }
        } else {
          float* slot = ws_slots + static_cast<size_t>(w.slot) * ws_slot_floats(D, rows_pad);
          float* sm = slot + static_cast<size_t>(rows_pad) * D;
#pragma unroll
          for (int j = 0; j < CW; ++j) {
            if (c0 + j < rows) {
              slot[static_cast<size_t>(c0 + j) * D + t] = __uint_as_float(o[j]);
            }
          }
          if (t < CW && c0 + t < rows) {
            sm[c0 + t] = m_mine;
            sm[rows_pad + c0 + t] = l_mine;
          }
          if (a.done) {
            // The unit is cut across CTAs.  Each warpgroup of each of its CTAs counts itself once its
            // half of the partial rows is out; the one that counts last merges that half (nobody waits).
            __threadfence();
            if (!wg_sync()) { ok = false; break; }
            CutUnit cu;
            const long long u0 = t0 + w.it - w.ti;
            cut_unit(n_tiles, static_cast<int>(gridDim.x), u0, u0 + w.tiles_b, cu);
            if (t == 0) {
              unsigned int* cnt = a.done + 2 * cu.c_lo + wg;
              const bool is_last = atomicAdd(cnt, 1u) + 1u == static_cast<unsigned int>(cut_pieces(cu));
              if (is_last) *cnt = 0u;
              last_flags[wg] = is_last ? 1 : 0;
            }
            if (!wg_sync()) { ok = false; break; }
            if (last_flags[wg]) {
              __threadfence();
              for (int j = quad; j < CW && c0 + j < rows; j += 4) {
                const int r = c0 + j, i = r / a.G, g = r - i * a.G;
                const int64_t orow = static_cast<int64_t>(w.r0 + i) * a.H_q + w.h * a.G + g;
                merge_row<D>(ws_slots, rows_pad, cu, r, lane, out_l + orow * D, lse_l ? lse_l + orow : nullptr);
              }
            }
          }
        }
        tc_fence_before();   // the reads of O^T are ordered before the next unit's first PV product
      }
      walk_next(a, w);
    }
  }

  // ---- teardown: every thread arrives here, on success and on abort ----
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kCols) : "memory");
  }
}

bool plan_t_layout(int np, int rows_box, TLayout* lay) {
  lay->rows_box = rows_box;
  lay->q_half = np * 128;
  lay->q_bytes = 2 * lay->q_half;
  const int fixed = 2 * lay->q_bytes + 2 * kPBytes + kMiscBytes;
  int n_kv = (227 * 1024 - fixed) / kKvBytes;
  if (n_kv > kTMaxKv) n_kv = kTMaxKv;
  if (n_kv < 3) return false;
  lay->n_kv = n_kv;
  lay->off_q = 0;
  lay->off_p = 2 * lay->q_bytes;
  lay->off_kv = lay->off_p + 2 * kPBytes;
  lay->off_misc = lay->off_kv + n_kv * kKvBytes;
  lay->total = lay->off_misc + kMiscBytes;
  return true;
}

template <int NP>
int32_t launch_t(const AttnArgs& a, cudaStream_t st, int rows_pad, int grid, const TLayout& lay,
                 const CUtensorMap& mk, const CUtensorMap& mv, const CUtensorMap& mks, const CUtensorMap& mvs,
                 const CUtensorMap& mq) {
  static bool configured[64] = {false};
  int dev = 0;
  MS_CUDA_TRY(cudaGetDevice(&dev));
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    MS_CUDA_TRY(cudaFuncSetAttribute(attn_umma_t_kernel<NP>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     227 * 1024));
    configured[dev] = true;
  }
  if (a.ev_split_begin) MS_CUDA_TRY(cudaEventRecord(a.ev_split_begin, st));
  MS_CUDA_TRY(launch_pdl(attn_umma_t_kernel<NP>, dim3(grid), dim3(kTThreads), static_cast<size_t>(lay.total), st, a,
                         mk, mv, mks, mvs, mq, rows_pad, lay));
  if (a.ev_split_end) MS_CUDA_TRY(cudaEventRecord(a.ev_split_end, st));
  return MS_OK;
}

}  // namespace

bool attn_umma_t_supports(int D, int G, int max_nq) { return D == 128 && max_nq <= kMaxNq && G * max_nq <= 64; }

int32_t launch_attn_umma_t(const AttnArgs& a_in, cudaStream_t st) {
  AttnArgs a = a_in;
  if (a.B == 0 || a.T == 0 || a.n_layers == 0) return MS_OK;
  const int rows = a.max_nq * a.G;
  const int rows_pad = (rows + 15) & ~15;
  TLayout lay;
  if (!attn_umma_t_supports(a.D, a.G, a.max_nq) || !plan_t_layout(rows_pad, rows, &lay))
    return MS_ERR_UNSUPPORTED_SHAPE;
  if (static_cast<int>((a.B + 1 + kTThreads / 32) * sizeof(int)) > lay.n_kv * kKvBytes) return MS_ERR_UNSUPPORTED_SHAPE;
  const int grid = attn_mma_grid();
  if (grid <= 0) return cuda_status(cudaErrorNoDevice);
  // Where the merge runs.  With at least two units per CTA a unit is cut into two or three pieces
  // and the warpgroup that delivers the last of them merges it on the spot (counters: two per
  // CTA).  With few units -- a small batch -- every unit is cut across many CTAs, and merging a
  // unit inside one CTA would leave the rest of the machine idle meanwhile: the merge is then a
  // launch of its own, one warp per (unit, row), behind this kernel.
  const long long units = static_cast<long long>(a.n_layers) * a.B * a.H_kv;
  a.done = (units >= 2ll * grid && 2 * grid <= kDoneBankWords) ? done_bank(a.workspace) : nullptr;
  // one descriptor per tensor covers every layer (the layer is the outermost coordinate)
  const uint64_t nl = static_cast<uint64_t>(a.n_layers);
  const uint64_t kv_ls = nl > 1 ? a.kv_layer_stride : static_cast<uint64_t>(a.H_kv) * a.kv_head_stride;
  const uint64_t q_ls = nl > 1 ? a.q_layer_stride : static_cast<uint64_t>(a.T) * a.H_q * a.D;
  const uint64_t ks_ls = nl > 1 ? a.kstep_layer_stride : static_cast<uint64_t>(a.T) * a.H_kv * a.D;
  CUtensorMap mk, mv, mks, mvs, mq;
  const bool ok =
      make_map4(&mk, a.k_cache, a.D, static_cast<uint64_t>(a.n_slots), a.H_kv, nl, a.D, a.kv_head_stride, kv_ls, kTile, 1) &&
      make_map4(&mv, a.v_cache, a.D, static_cast<uint64_t>(a.n_slots), a.H_kv, nl, a.D, a.kv_head_stride, kv_ls, kTile, 1) &&
      make_map4(&mks, a.k_step, a.D, a.H_kv, a.T, nl, a.D, static_cast<uint64_t>(a.H_kv) * a.D, ks_ls, 1, kMaxNq) &&
      make_map4(&mvs, a.v_step, a.D, a.H_kv, a.T, nl, a.D, static_cast<uint64_t>(a.H_kv) * a.D, ks_ls, 1, kMaxNq) &&
      make_map4(&mq, a.q, a.D, a.H_q, a.T, nl, a.D, static_cast<uint64_t>(a.H_q) * a.D, q_ls, a.G, a.max_nq);
  if (!ok) return cuda_status(cudaErrorInvalidValue);
  int32_t rc;
  switch (rows_pad) {
    case 16: rc = launch_t<16>(a, st, rows_pad, grid, lay, mk, mv, mks, mvs, mq); break;
    case 32: rc = launch_t<32>(a, st, rows_pad, grid, lay, mk, mv, mks, mvs, mq); break;
    case 48: rc = launch_t<48>(a, st, rows_pad, grid, lay, mk, mv, mks, mvs, mq); break;
    default: rc = launch_t<64>(a, st, rows_pad, grid, lay, mk, mv, mks, mvs, mq); break;
  }
  if (rc != MS_OK || a.done) return rc;
  return launch_attn_merge(a, st, rows_pad, grid);
}

}  // namespace ms
