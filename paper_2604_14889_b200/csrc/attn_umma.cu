// tcgen05 split-KV path of the MemoSight step attention (sm_100a).
//
// Same computation and the same flat tile schedule as the mma.sync path (paper
// Sec. 2.1.1, Sec. 2.3: the packed n_q*G query rows of a step block against the
// whole compacted cache plus the visible step-local keys), but the two
// contractions run on the 5th-generation tensor cores with both operands read
// straight from shared memory, so a K/V byte crosses shared memory once however
// many query rows there are.  Up to 128 packed rows per KV head.
//
// One persistent CTA per SM, 8 warps:
//   warp 0     TMA producer: Q tile of each unit, then K and V tiles of the flat
//              list into a ring of separately released buffers.
//   warp 1     MMA issuer (one thread): S = Q K^T into one of two TMEM score
//              buffers, and O (+)= P V into the TMEM output accumulator; it runs
//              one tile ahead with Q K^T so the tensor pipe works on tile t+1
//              while the softmax of tile t is in flight.  Completion is reported
//              by tcgen05.commit onto mbarriers (buffer release, S ready, PV done).
//   warps 4-7  softmax: thread = packed row (TMEM lane).  Scores come in with
//              tcgen05.ld, the probabilities go to shared memory as the bf16 A
//              operand of the PV product (128-byte swizzled, K-major).  The
//              running maximum is applied lazily: P is formed against the
//              reference maximum of the unit and O is rescaled (tcgen05.ld/st)
//              only when a tile exceeds it by more than 2^8, which keeps the
//              accumulator out of the per-tile critical path.  At the end of a
//              unit the same threads read O from TMEM, normalise and write
//              `out`, or the (m, l, O) partial when the unit continues in
//              another CTA.
// Rows of the 128-row MMA tile beyond the block's packed rows are never written
// by anyone and never read back: rows of A only influence their own row of D.
// Every wait is bounded; on expiry the kernel records it in the workspace status
// word, all roles leave their loops, in-flight copies and MMAs are drained and
// tensor memory is released before the CTA exits.
#include "attn_umma_common.cuh"

namespace ms {
namespace {

constexpr int kUThreads = 256;
constexpr uint32_t kTmemCols = 512;     // S0 | S1 | O, rounded to a power of two
constexpr uint32_t kColS = 0, kColO = 256;
constexpr float kRescaleSlack = 8.f;    // log2 units a tile may exceed the reference max by
constexpr int kMaxKvBufs = 12;

// Barrier slots (8 bytes each) behind lay.off_bar.
enum : int {
  kBarKvFull = 0, kBarKvEmpty = kMaxKvBufs, kBarQFull = 2 * kMaxKvBufs, kBarQEmpty = kBarQFull + 2,
  kBarSFull = kBarQEmpty + 2, kBarPFull = kBarSFull + 2, kBarPvDone = kBarPFull + 2,
  kBarDrain = kBarPvDone + 2, kBarCount = kBarDrain + 1
};

struct UmmaLayout {
  int rows_box;            // rows one Q box holds: G * max_nq
  int q_half, q_bytes;     // one 64-column half / one whole Q buffer
  int p_half, p_bytes;     // one 64-key half / one whole P buffer
  int kv_bytes, n_kv;      // one K or V tile; buffers in the ring
  int off_q, off_p, off_kv, off_bar, total;
};

// ---------------------------------------------------------------- softmax pieces

// One pass over the valid score columns of this thread's row.
//   kWrite = false: row maximum only.
//   kWrite = true : p = 2^(s*scale - m_use) -> bf16 into the P buffer, row sum; also the maximum.
//   row_ok        : this thread's row exists (only those rows are stored).
//   kMask         : the tile is ragged or step-local: columns >= nv are invisible, and on the
//                   step-local tile the (n_cand, anchor) rule applies per row.
template <bool kWrite, bool kMask>
__device__ __forceinline__ void softmax_pass(uint32_t s_addr, int nv, bool is_step, int tok, int n_c, int anc,
                                             float scale, float m_use, bool row_ok, uint32_t p_row,
                                             uint32_t p_half, uint32_t rx, float& tmax, float& tsum) {
  tmax = -INFINITY;
  tsum = 0.f;
  const int nv16 = (nv + 15) & ~15;
  const int n_chunks = kMask ? (nv + 31) >> 5 : kTile / 32;
#pragma unroll 1
  for (int c = 0; c < n_chunks; ++c) {
    uint32_t r[32];
    tmem_ld32(s_addr + c * 32, r);
    tmem_ld_wait(r);
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      float p[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        float s = __uint_as_float(r[g * 8 + e]);
        if (kMask) {
          const int col = c * 32 + g * 8 + e;
          bool vis = col < nv;
          if (is_step) vis = vis && step_key_visible(tok, col, n_c, anc);
          s = vis ? s : -INFINITY;
        }
        tmax = fmaxf(tmax, s);
        if (kWrite) {
          p[e] = ex2(fmaf(s, scale, -m_use));
          tsum += p[e];
        }
      }
      if (kWrite) {
        const int cc = c * 4 + g;                  // 16-byte group of the 128-key row
        // rows past the block's packed rows have no place in the P buffer
        if (row_ok && (!kMask || cc * 8 < nv16)) {
          const uint32_t addr = p_row + (cc >> 3) * p_half + (((cc & 7) ^ rx) << 4);
          asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(pack2(p[0], p[1])),
                       "r"(pack2(p[2], p[3])), "r"(pack2(p[4], p[5])), "r"(pack2(p[6], p[7]))
                       : "memory");
        }
      }
    }
  }
}

// ---------------------------------------------------------------- kernel

template <int D>
__global__ void __launch_bounds__(kUThreads, 1)
attn_umma_kernel(const AttnArgs a, const __grid_constant__ CUtensorMap map_k,
                 const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_ks,
                 const __grid_constant__ CUtensorMap map_vs, const __grid_constant__ CUtensorMap map_q,
                 int rows_pad, const UmmaLayout lay) {
  constexpr int HALVES = D / 64;
  constexpr int KSTEPS_QK = D / 16;
  constexpr uint32_t kHalfStride = kTile * 128;          // bytes between the 64-column halves of a K/V tile
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sb = smem_u32(smem);
  const uint32_t bars = sb + lay.off_bar;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + lay.off_bar + kBarCount * 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + lay.off_bar + kBarCount * 8 + 8);
  uint32_t* status = reinterpret_cast<uint32_t*>(a.workspace);
  int* ws_pre = reinterpret_cast<int*>(reinterpret_cast<uint8_t*>(a.workspace) + kWsHeaderBytes);
  float* ws_slots = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(a.workspace) + kWsHeaderBytes +
                                             ws_prefix_bytes());
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (sb & 1023u) {   // the swizzled layouts need a 1024-byte aligned base
    if (threadIdx.x == 0) atomicExch(status, kTimeoutMagic + 1);
    return;
  }

  // ---- schedule (the buffers are still unused: the prefix lives in their place) ----
  int* s_pre = reinterpret_cast<int*>(smem);
  int* s_scratch = s_pre + a.B + 1;
  build_tile_prefix(a, s_pre, s_scratch);
  const long long n_tiles = static_cast<long long>(s_pre[a.B]) * a.H_kv;
  const long long t0 = n_tiles * blockIdx.x / gridDim.x;
  const long long t1 = n_tiles * (blockIdx.x + 1) / gridDim.x;
  const int n_iter = static_cast<int>(t1 - t0);
  if (blockIdx.x == 0) {
    for (int i = threadIdx.x; i <= a.B; i += blockDim.x) ws_pre[i] = s_pre[i];
  }
  Walk w0;
  w0.n_iter = 0;
  if (n_iter > 0) {
    int lo = 0, hi = a.B;
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (static_cast<long long>(s_pre[mid]) * a.H_kv <= t0) lo = mid; else hi = mid;
    }
    walk_init(a, w0, lo, t0 - static_cast<long long>(s_pre[lo]) * a.H_kv, n_iter);
  }
  if (threadIdx.x == 0) {
    for (int i = 0; i < kMaxKvBufs; ++i) {
      mbar_init(bars + 8 * (kBarKvFull + i), 1);
      mbar_init(bars + 8 * (kBarKvEmpty + i), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bars + 8 * (kBarQFull + i), 1);
      mbar_init(bars + 8 * (kBarQEmpty + i), 1);
      mbar_init(bars + 8 * (kBarSFull + i), 1);
      mbar_init(bars + 8 * (kBarPFull + i), 4);
      mbar_init(bars + 8 * (kBarPvDone + i), 1);
    }
    mbar_init(bars + 8 * kBarDrain, 1);
    wait_ctx_init(abort_flag, a.wait_limit_us);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();   // the prefix has been consumed
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(tmem_slot)), "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0 && lane == 0 && n_iter > 0) {
    // =========================== TMA producer ===========================
    Walk w = w0;
    bool ok = true;
    int uses = 0;                      // K/V buffer fills issued
    int pieces = 0;                    // Q fills issued
    RingPos rp;
    rp.init(0, lay.n_kv);
    while (w.it < n_iter) {
      walk_tile(a, w);
      if (w.first) {
        const int qb = w.piece_idx & 1;
        if (!mbar_wait(bars + 8 * (kBarQEmpty + qb), ((w.piece_idx >> 1) & 1) ^ 1, abort_flag, status)) {
          ok = false;
          break;
        }
        fence_async_smem();
        const uint32_t bar = bars + 8 * (kBarQFull + qb);
        mbar_arrive_expect_tx(bar, static_cast<uint32_t>(HALVES * lay.rows_box * 128));
#pragma unroll
        for (int hf = 0; hf < HALVES; ++hf)
          tma_load_3d(sb + lay.off_q + qb * lay.q_bytes + hf * lay.q_half, &map_q, bar, hf * 64, w.h * a.G,
                      w.r0);
        ++pieces;
      }
#pragma unroll 1
      for (int kv = 0; kv < 2; ++kv) {
        const int buf = rp.buf;
        if (!mbar_wait(bars + 8 * (kBarKvEmpty + buf), rp.par ^ 1u, abort_flag, status)) {
          ok = false;
          break;
        }
        rp.step(1);
        fence_async_smem();
        const uint32_t dst = sb + lay.off_kv + buf * lay.kv_bytes;
        const uint32_t bar = bars + 8 * (kBarKvFull + buf);
        if (w.is_step) {
          mbar_arrive_expect_tx(bar, static_cast<uint32_t>(HALVES * kMaxNq * 128));
#pragma unroll
          for (int hf = 0; hf < HALVES; ++hf)
            tma_load_3d(dst + hf * kHalfStride, kv ? &map_vs : &map_ks, bar, hf * 64, w.h, w.r0);
        } else {
          mbar_arrive_expect_tx(bar, static_cast<uint32_t>(lay.kv_bytes));
          const int y = static_cast<int>(w.slot_off) + w.ti * kTile;
#pragma unroll
          for (int hf = 0; hf < HALVES; ++hf)
            tma_load_3d(dst + hf * kHalfStride, kv ? &map_v : &map_k, bar, hf * 64, y, w.h);
        }
        ++uses;
      }
      if (!ok) break;
      walk_next(a, w);
    }
    // Drain: every copy issued here must have landed before the CTA may exit.
    for (int u = uses > lay.n_kv ? uses - lay.n_kv : 0; u < uses; ++u)
      (void)mbar_wait(bars + 8 * (kBarKvFull + u % lay.n_kv), (u / lay.n_kv) & 1, abort_flag, status);
    for (int p = pieces > 2 ? pieces - 2 : 0; p < pieces; ++p)
      (void)mbar_wait(bars + 8 * (kBarQFull + (p & 1)), (p >> 1) & 1, abort_flag, status);
  } else if (warp == 1 && lane == 0 && n_iter > 0) {
    // =========================== MMA issuer ===========================
    // The descriptors of consecutive MMAs differ only by a constant in their low word.
    const uint32_t idesc_qk = instr_desc(kTile, 0), idesc_qk_step = instr_desc(kMaxNq, 0);
    const uint32_t idesc_pv = instr_desc(D, 1);
    const uint32_t q_lo0 = desc_lo(sb + lay.off_q, 16), k_lo0 = desc_lo(sb + lay.off_kv, 16);
    const uint32_t p_lo0 = desc_lo(sb + lay.off_p, 16), v_lo0 = desc_lo(sb + lay.off_kv, kHalfStride);
    Walk wq = w0, wp = w0;
    RingPos rk, rv;
    rk.init(0, lay.n_kv);
    rv.init(1, lay.n_kv);
    bool ok = true;
    auto issue_qk = [&]() -> bool {
      walk_tile(a, wq);
      const int it = wq.it, qb = wq.piece_idx & 1;
      if ((wq.first && !mbar_wait(bars + 8 * (kBarQFull + qb), (wq.piece_idx >> 1) & 1, abort_flag, status)) ||
          !mbar_wait(bars + 8 * (kBarKvFull + rk.buf), rk.par, abort_flag, status))
        return false;
      tc_fence_after();
      const uint32_t q_lo = q_lo0 + qb * (lay.q_bytes >> 4), q_half = lay.q_half >> 4;
      const uint32_t k_lo = k_lo0 + rk.buf * (lay.kv_bytes >> 4);
      const uint32_t d_s = tmem + kColS + (it & 1) * kTile;
      const uint32_t idesc = wq.is_step ? idesc_qk_step : idesc_qk;
#pragma unroll
      for (int ks = 0; ks < KSTEPS_QK; ++ks)
        umma_bf16_lo(d_s, q_lo + (ks >> 2) * q_half + (ks & 3) * 2,
                     k_lo + (ks >> 2) * (kHalfStride >> 4) + (ks & 3) * 2, idesc, ks > 0);
      umma_commit(bars + 8 * (kBarKvEmpty + rk.buf));
      umma_commit(bars + 8 * (kBarSFull + (it & 1)));
      if (wq.last) umma_commit(bars + 8 * (kBarQEmpty + qb));
      rk.step(2);
      walk_next(a, wq);
      return true;
    };
    ok = issue_qk();
    while (ok && wp.it < n_iter) {
      if (wq.it < n_iter && !issue_qk()) { ok = false; break; }
      walk_tile(a, wp);
      const int it = wp.it;
      if (!mbar_wait(bars + 8 * (kBarPFull + (it & 1)), (it >> 1) & 1, abort_flag, status) ||
          !mbar_wait(bars + 8 * (kBarKvFull + rv.buf), rv.par, abort_flag, status)) {
        ok = false;
        break;
      }
      tc_fence_after();
      const uint32_t p_lo = p_lo0 + (it & 1) * (lay.p_bytes >> 4), p_half = lay.p_half >> 4;
      const uint32_t v_lo = v_lo0 + rv.buf * (lay.kv_bytes >> 4);
      const int ksteps = wp.is_step ? 1 : (wp.nvalid + 15) >> 4;
      const uint32_t acc0 = wp.first ? 0u : 1u;
      if (ksteps == kTile / 16) {
#pragma unroll
        for (int j = 0; j < kTile / 16; ++j)
          umma_bf16_lo(tmem + kColO, p_lo + (j >> 2) * p_half + (j & 3) * 2, v_lo + j * (2048 >> 4), idesc_pv,
                       j == 0 ? acc0 : 1u);
      } else {
#pragma unroll 1
        for (int j = 0; j < ksteps; ++j)
          umma_bf16_lo(tmem + kColO, p_lo + (j >> 2) * p_half + (j & 3) * 2, v_lo + j * (2048 >> 4), idesc_pv,
                       j == 0 ? acc0 : 1u);
      }
      umma_commit(bars + 8 * (kBarKvEmpty + rv.buf));
      umma_commit(bars + 8 * (kBarPvDone + (it & 1)));
      rv.step(2);
      walk_next(a, wp);
    }
    if (!ok) {
      // aborting: let the tensor pipe run dry before tensor memory is released
      umma_commit(bars + 8 * kBarDrain);
      const unsigned long long t_begin = global_ns();
      while (!mbar_try_wait(bars + 8 * kBarDrain, 0) && global_ns() - t_begin < wait_limit_ns(abort_flag)) {
      }
    }
  } else if (warp >= 4 && n_iter > 0) {
    // =========================== softmax warps ===========================
    const int quad = warp - 4;
    const int r = quad * 32 + lane;                       // packed row = TMEM lane
    const uint32_t lane_addr = tmem + (static_cast<uint32_t>(quad * 32) << 16);
    const uint32_t rx = r & 7;
    Walk w = w0;
    float m_ref = 0.f, l_run = 0.f;
    int tok = 0, anc = 0, rows = 0;
    bool row_ok = false, warp_on = false;
    bool ok = true;
    auto wait_all = [&](uint32_t bar, uint32_t parity) -> bool {
      return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag, status));
    };
    while (ok && w.it < n_iter) {
      walk_tile(a, w);
      const int it = w.it, pb = it & 1;
      if (w.first) {
        rows = w.n_q * a.G;
        row_ok = r < rows;
        warp_on = quad * 32 < rows;
        if (row_ok) {
          const int i = r / a.G;
          tok = i;
          anc = (i < w.n_c) ? i : (a.anchor ? a.anchor[w.r0 + i] : w.n_c);
        } else {
          tok = 1 << 20;
          anc = 0;
        }
        m_ref = 0.f;
        l_run = 0.f;
      }
      if (!wait_all(bars + 8 * (kBarSFull + pb), (it >> 1) & 1)) { ok = false; break; }
      // the PV product that read this P buffer two tiles ago is complete
      if (it >= 2 && !wait_all(bars + 8 * (kBarPvDone + pb), ((it >> 1) - 1) & 1)) { ok = false; break; }
      tc_fence_after();
      const int nv = w.nvalid;
      const bool masked = w.is_step || nv < kTile;
      if (masked) {
        // V rows past the valid keys hold foreign or stale bytes; P is 0 there but 0 * NaN is NaN:
        // clear the rows of the last 16-key step that the PV product still reads
        const int use = 2 * it + 1, buf = use % lay.n_kv;
        if (!wait_all(bars + 8 * (kBarKvFull + buf), (use / lay.n_kv) & 1)) { ok = false; break; }
        const uint32_t va = sb + lay.off_kv + buf * lay.kv_bytes;
        const int n_rows = ((nv + 15) & ~15) - nv;
        for (int x = threadIdx.x - 128; x < n_rows * HALVES * 8; x += 128) {
          const int rr = nv + x / (HALVES * 8), cc = x % (HALVES * 8);
          const uint32_t addr = va + (cc >> 3) * kHalfStride + rr * 128 + ((cc & 7) << 4);
          asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(addr), "r"(0u) : "memory");
        }
      }
      if (warp_on) {
        const uint32_t p_row = sb + lay.off_p + pb * lay.p_bytes + r * 128;
        const uint32_t s_addr = lane_addr + kColS + pb * kTile;
        float tmax, tsum;
        if (w.piece_j == 0) {
          if (masked) {
            softmax_pass<false, true>(s_addr, nv, w.is_step, tok, w.n_c, anc, a.scale_log2, 0.f, row_ok, p_row,
                                      lay.p_half, rx, tmax, tsum);
            m_ref = (tmax == -INFINITY) ? 0.f : tmax * a.scale_log2;
            softmax_pass<true, true>(s_addr, nv, w.is_step, tok, w.n_c, anc, a.scale_log2, m_ref, row_ok, p_row,
                                     lay.p_half, rx, tmax, tsum);
          } else {
            softmax_pass<false, false>(s_addr, nv, false, tok, w.n_c, anc, a.scale_log2, 0.f, row_ok, p_row,
                                       lay.p_half, rx, tmax, tsum);
            m_ref = (tmax == -INFINITY) ? 0.f : tmax * a.scale_log2;
            softmax_pass<true, false>(s_addr, nv, false, tok, w.n_c, anc, a.scale_log2, m_ref, row_ok, p_row,
                                      lay.p_half, rx, tmax, tsum);
          }
          l_run = tsum;
        } else {
          if (masked)
            softmax_pass<true, true>(s_addr, nv, w.is_step, tok, w.n_c, anc, a.scale_log2, m_ref, row_ok, p_row,
                                     lay.p_half, rx, tmax, tsum);
          else
            softmax_pass<true, false>(s_addr, nv, false, tok, w.n_c, anc, a.scale_log2, m_ref, row_ok, p_row,
                                      lay.p_half, rx, tmax, tsum);
          const float m_new = tmax * a.scale_log2;
          const bool grow = row_ok && (m_new > m_ref + kRescaleSlack);
          if (__any_sync(0xffffffffu, grow)) {
            // rare: a tile outgrew the reference maximum; rescale O and l, redo this tile's P
            const float m2 = (row_ok && m_new > m_ref) ? m_new : m_ref;
            const float alpha = ex2(m_ref - m2);
            if (!wait_all(bars + 8 * (kBarPvDone + ((it - 1) & 1)), ((it - 1) >> 1) & 1)) { ok = false; break; }
            tc_fence_after();
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
              uint32_t o[32];
              tmem_ld32(lane_addr + kColO + c * 32, o);
              tmem_ld_wait(o);
#pragma unroll
              for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
              tmem_st32(lane_addr + kColO + c * 32, o);
            }
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            l_run *= alpha;
            m_ref = m2;
            if (masked)
              softmax_pass<true, true>(s_addr, nv, w.is_step, tok, w.n_c, anc, a.scale_log2, m_ref, row_ok, p_row,
                                       lay.p_half, rx, tmax, tsum);
            else
              softmax_pass<true, false>(s_addr, nv, false, tok, w.n_c, anc, a.scale_log2, m_ref, row_ok, p_row,
                                        lay.p_half, rx, tmax, tsum);
          }
          l_run += tsum;
        }
      }
      // P (and the cleared V rows) were written through the generic proxy; the MMA reads them
      // through the async proxy
      fence_async_smem();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bars + 8 * (kBarPFull + pb));

      if (w.last) {
        // ---- end of the unit (or of this CTA's part of it) ----
        if (!wait_all(bars + 8 * (kBarPvDone + pb), (it >> 1) & 1)) { ok = false; break; }
        tc_fence_after();
        if (warp_on) {
          const int i = r / a.G, g = r - i * a.G;
          const int64_t orow = static_cast<int64_t>(w.r0 + i) * a.H_q + w.h * a.G + g;
          if (w.slot < 0) {
            const float inv = 1.f / l_run;
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
              uint32_t o[32];
              tmem_ld32(lane_addr + kColO + c * 32, o);
              tmem_ld_wait(o);
              if (row_ok) {
                uint4* op = reinterpret_cast<uint4*>(a.out + orow * D + c * 32);
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                  uint4 u;
                  u.x = pack2(__uint_as_float(o[8 * v + 0]) * inv, __uint_as_float(o[8 * v + 1]) * inv);
                  u.y = pack2(__uint_as_float(o[8 * v + 2]) * inv, __uint_as_float(o[8 * v + 3]) * inv);
                  u.z = pack2(__uint_as_float(o[8 * v + 4]) * inv, __uint_as_float(o[8 * v + 5]) * inv);
                  u.w = pack2(__uint_as_float(o[8 * v + 6]) * inv, __uint_as_float(o[8 * v + 7]) * inv);
                  op[v] = u;
                }
              }
            }
            if (row_ok && a.lse) a.lse[orow] = (m_ref + log2f(l_run)) * 0.69314718055994531f;
          } else {
            float* slot = ws_slots + static_cast<size_t>(w.slot) * ws_slot_floats(D, rows_pad);
            float* sm = slot + static_cast<size_t>(rows_pad) * D;
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
              uint32_t o[32];
              tmem_ld32(lane_addr + kColO + c * 32, o);
              tmem_ld_wait(o);
              if (row_ok) {
                uint4* sp = reinterpret_cast<uint4*>(slot + static_cast<size_t>(r) * D + c * 32);
#pragma unroll
                for (int v = 0; v < 8; ++v) sp[v] = make_uint4(o[4 * v], o[4 * v + 1], o[4 * v + 2], o[4 * v + 3]);
              }
            }
            if (row_ok) {
              sm[r] = m_ref;
              sm[rows_pad + r] = l_run;
            }
          }
        }
        tc_fence_before();   // the reads of O are ordered before the next unit's first PV product
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
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols)
                 : "memory");
  }
}

bool plan_layout(int D, int rows, int rows_box, UmmaLayout* lay) {
  const int halves = D / 64;
  lay->rows_box = rows_box;
  lay->q_half = ((rows_box + 7) & ~7) * 128;
  lay->q_bytes = halves * lay->q_half;
  lay->p_half = ((rows + 7) & ~7) * 128;
  lay->p_bytes = 2 * lay->p_half;
  lay->kv_bytes = kTile * D * 2;
  const int fixed = 2 * lay->q_bytes + 2 * lay->p_bytes;
  const int bar_bytes = 1024;
  const int budget = 227 * 1024 - bar_bytes - fixed;
  int n_kv = budget / lay->kv_bytes;
  if (n_kv > kMaxKvBufs) n_kv = kMaxKvBufs;
  if (n_kv < 3) return false;
  lay->n_kv = n_kv;
  lay->off_q = 0;
  lay->off_p = lay->off_q + 2 * lay->q_bytes;
  lay->off_kv = lay->off_p + 2 * lay->p_bytes;
  lay->off_bar = lay->off_kv + n_kv * lay->kv_bytes;
  lay->total = lay->off_bar + bar_bytes;
  // the 128-row MMA reads 16 KB from each half of an A operand; the ring behind the Q and P
  // buffers keeps those reads inside the allocation
  return n_kv * lay->kv_bytes >= 2 * 16384 + 16384;
}

template <int D>
int32_t launch_umma(const AttnArgs& a, cudaStream_t st, int rows_pad, int grid, const UmmaLayout& lay,
                    const CUtensorMap& mk, const CUtensorMap& mv, const CUtensorMap& mks,
                    const CUtensorMap& mvs, const CUtensorMap& mq) {
  static int configured[64] = {0};
  int dev = 0;
  MS_CUDA_TRY(cudaGetDevice(&dev));
  if (dev >= 0 && dev < 64 && configured[dev] < lay.total) {
    MS_CUDA_TRY(cudaFuncSetAttribute(attn_umma_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     227 * 1024));
    configured[dev] = 227 * 1024;
  }
  if (a.ev_split_begin) MS_CUDA_TRY(cudaEventRecord(a.ev_split_begin, st));
  attn_umma_kernel<D><<<grid, kUThreads, lay.total, st>>>(a, mk, mv, mks, mvs, mq, rows_pad, lay);
  MS_LAUNCH_CHECK();
  if (a.ev_split_end) MS_CUDA_TRY(cudaEventRecord(a.ev_split_end, st));
  return MS_OK;
}

}  // namespace

bool attn_umma_supports(int D, int G, int max_nq) {
  UmmaLayout lay;
  return (D == 64 || D == 128) && max_nq <= kMaxNq && G * max_nq <= 128 && plan_layout(D, G * max_nq, G * max_nq, &lay);
}

int32_t launch_attn_umma(const AttnArgs& a, cudaStream_t st) {
  if (a.B == 0 || a.T == 0) return MS_OK;
  const int rows = a.max_nq * a.G;
  const int rows_pad = (rows + 15) & ~15;
  UmmaLayout lay;
  if (!plan_layout(a.D, rows, rows, &lay)) return MS_ERR_UNSUPPORTED_SHAPE;
  // the prefix of tile counts is built in the (still unused) buffers
  if (static_cast<int>((a.B + 1 + kUThreads) * sizeof(int)) > lay.off_bar) return MS_ERR_UNSUPPORTED_SHAPE;
  const int grid = attn_mma_grid();
  if (grid <= 0) return cuda_status(cudaErrorNoDevice);
  CUtensorMap mk, mv, mks, mvs, mq;
  const bool ok =
      make_map(&mk, a.k_cache, a.D, static_cast<uint64_t>(a.n_slots), a.H_kv, a.D, a.kv_head_stride, kTile, 1) &&
      make_map(&mv, a.v_cache, a.D, static_cast<uint64_t>(a.n_slots), a.H_kv, a.D, a.kv_head_stride, kTile, 1) &&
      make_map(&mks, a.k_step, a.D, a.H_kv, a.T, a.D, static_cast<uint64_t>(a.H_kv) * a.D, 1, kMaxNq) &&
      make_map(&mvs, a.v_step, a.D, a.H_kv, a.T, a.D, static_cast<uint64_t>(a.H_kv) * a.D, 1, kMaxNq) &&
      make_map(&mq, a.q, a.D, a.H_q, a.T, a.D, static_cast<uint64_t>(a.H_q) * a.D, a.G, a.max_nq);
  if (!ok) return cuda_status(cudaErrorInvalidValue);
  const int32_t rc = a.D == 128 ? launch_umma<128>(a, st, rows_pad, grid, lay, mk, mv, mks, mvs, mq)
                                : launch_umma<64>(a, st, rows_pad, grid, lay, mk, mv, mks, mvs, mq);
  if (rc != MS_OK) return rc;
  return launch_attn_merge(a, st, rows_pad, grid);
}

}  // namespace ms
