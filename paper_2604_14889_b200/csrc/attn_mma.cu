// Tensor-core split-KV path of the MemoSight step attention (sm_100a).
//
// What it computes (paper Sec. 2.1.1, Sec. 2.3): for every sequence b and KV head,
// the n_q*G packed query rows of the step block (n_q tokens x G query heads of
// the group) attend to all L_b entries of the compacted cache plus the visible
// step-local keys; softmax in fp32, bf16 inputs, fp32 accumulation.
//
// How it is laid out on the machine:
//   * The work is the flat list of 128-key tiles of all (sequence, KV head) units
//     (each unit = ceil(L_b/128) cache tiles + one tile holding the block's own
//     keys).  The list is cut into one contiguous, equally long range per CTA
//     (one persistent CTA per SM), so the load balance is exact whatever the
//     lengths are, and a unit that lies inside one CTA's range needs no merge.
//   * Inside a CTA one producer warp walks the range and issues TMA tile loads
//     (cp.async.bulk.tensor, 128-byte swizzle) of K and V into a ring of shared
//     memory stages guarded by full/empty mbarriers; it runs ahead of the math
//     across unit boundaries, so HBM requests never drain between units.
//   * Eight consumer warps = MB row blocks (16 packed rows each) x KS key slices.
//     A warp owns one slice of every tile: S = Q K^T and O += P V with
//     mma.sync.m16n8k16 (bf16 in, fp32 out; operands via ldmatrix), its own
//     online-softmax state, no per-tile synchronisation with other warps.  At the
//     end of a unit (or of the CTA's part of it) the slices are combined through
//     shared memory with a log-sum-exp tree.
//   * A unit finished inside one CTA is normalised and written to `out`
//     directly; otherwise (m, l, O) goes to one of the CTA's two partial slots
//     and attn_merge_kernel combines the pieces (warp-shuffle log-sum-exp).
//   * The mask costs nothing in the streaming loop: cache tiles only need the
//     length bound of the last tile; the (n_cand, anchor) rule is evaluated on
//     the single step-local tile.
// Every mbarrier wait is bounded (wall-clock limit); on expiry the kernel records
// it in the workspace status word, drains its own copies and returns.
#include "attn_sched.cuh"

namespace ms {
namespace {

constexpr int kConsumerWarps = 8;
constexpr int kThreads = (kConsumerWarps + 1) * 32;
enum : int { kFlagFirst = 1, kFlagLast = 2, kFlagStep = 4 };

struct TileMeta {
  int b, kvh, nvalid, flags, rows, n_c, r0, slot;   // slot < 0: unit is whole, write `out`
};

template <int D, int MB>
struct Cfg {
  static constexpr int KS = kConsumerWarps / MB;        // key slices
  static constexpr int NKW = kTile / KS;                // keys per warp per tile
  static constexpr int SUB = NKW < 32 ? NKW : 32;       // keys per softmax step
  static constexpr int NSUB = NKW / SUB;
  static constexpr int HALVES = D / 64;                 // 128-byte column groups per row
  static constexpr int KBYTES = kTile * D * 2;
  static constexpr int STAGE_BYTES = 2 * KBYTES;
  static constexpr int STAGES = (196608 / STAGE_BYTES) > 6 ? 6 : (196608 / STAGE_BYTES);
  static constexpr int OREGS = D / 2;                   // fp32 accumulators per thread
  static constexpr int MERGE_SLOTS = MB * KS / 2;
  static constexpr int MERGE_O_BYTES = MERGE_SLOTS * OREGS * 32 * 4;
  static constexpr int MERGE_ML_BYTES = MERGE_SLOTS * 4 * 32 * 4;
  static constexpr int OFF_MERGE_O = STAGES * STAGE_BYTES;
  static constexpr int OFF_MERGE_ML = OFF_MERGE_O + MERGE_O_BYTES;
  static constexpr int OFF_META = OFF_MERGE_ML + MERGE_ML_BYTES;
  static constexpr int OFF_BARS = OFF_META + STAGES * 32;           // full[], empty[], merge
  static constexpr int OFF_ABORT = OFF_BARS + (2 * STAGES + 1) * 8;
  static constexpr int SMEM_BYTES = OFF_ABORT + 16;
};

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                        uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                              uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// ---------------------------------------------------------------- split kernel

template <int D, int MB>
__global__ void __launch_bounds__(kThreads, 1)
attn_split_kernel(const AttnArgs a, const __grid_constant__ CUtensorMap map_k,
                  const __grid_constant__ CUtensorMap map_v,
                  const __grid_constant__ CUtensorMap map_ks,
                  const __grid_constant__ CUtensorMap map_vs, int rows_pad) {
  using C = Cfg<D, MB>;
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t smem_base = smem_u32(smem);
  TileMeta* meta = reinterpret_cast<TileMeta*>(smem + C::OFF_META);
  const uint32_t bar_full = smem_base + C::OFF_BARS;
  const uint32_t bar_empty = bar_full + C::STAGES * 8;
  const uint32_t bar_merge = bar_empty + C::STAGES * 8;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + C::OFF_ABORT);
  uint32_t* status = reinterpret_cast<uint32_t*>(a.workspace);
  int* ws_pre = reinterpret_cast<int*>(reinterpret_cast<uint8_t*>(a.workspace) + kWsHeaderBytes);
  float* ws_slots = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(a.workspace) +
                                             kWsHeaderBytes + ws_prefix_bytes());

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (smem_base & 1023u) {   // the swizzled tile layout needs a 1024-byte aligned base
    if (threadIdx.x == 0) atomicExch(status, kTimeoutMagic + 1);
    return;
  }

  // ---- schedule: prefix of tile counts (stage memory is still unused) ----
  int* s_pre = reinterpret_cast<int*>(smem);
  int* s_scratch = s_pre + a.B + 1;
  build_tile_prefix(a, s_pre, s_scratch);
  const long long n_tiles = static_cast<long long>(s_pre[a.B]) * a.H_kv;
  const long long t0 = n_tiles * blockIdx.x / gridDim.x;
  const long long t1 = n_tiles * (blockIdx.x + 1) / gridDim.x;
  if (blockIdx.x == 0) {
    for (int i = threadIdx.x; i <= a.B; i += blockDim.x) ws_pre[i] = s_pre[i];
  }
  // first unit of this CTA: largest b with H_kv * pre[b] <= t0
  int b0 = 0;
  if (t0 < t1) {
    int lo = 0, hi = a.B;
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (static_cast<long long>(s_pre[mid]) * a.H_kv <= t0) lo = mid; else hi = mid;
    }
    b0 = lo;
  }
  const long long unit_base0 = static_cast<long long>(s_pre[b0]) * a.H_kv;
  if (threadIdx.x == 0) {
    for (int s = 0; s < C::STAGES; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, kConsumerWarps);
    }
    mbar_init(bar_merge, kConsumerWarps);
    wait_ctx_init(abort_flag, a.wait_limit_us);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();   // prefix consumed, barriers initialised: stage memory may now be filled
  if (t0 >= t1) return;
  const int n_iter = static_cast<int>(t1 - t0);

  if (warp == kConsumerWarps) {
    // =========================== producer warp ===========================
    if (lane != 0) return;
    int b = b0, L, n_q, r0;
    seq_shape(a, b, L, n_q, r0);
    int tiles_b = seq_tiles(L, n_q);
    long long rel = t0 - unit_base0;             // tile offset inside sequence b's H_kv units
    int h = static_cast<int>(rel / tiles_b);
    int ti = static_cast<int>(rel - static_cast<long long>(h) * tiles_b);
    int n_c = a.n_cand[b];
    n_c = n_c < 0 ? 0 : (n_c > n_q ? n_q : n_c);
    long long slot_off = a.kv_off[b];
    int piece_slot = 0;
    bool piece_open = false;
    bool ok = true;
    int it = 0;
    for (; it < n_iter; ++it) {
      const int s = it % C::STAGES;
      const uint32_t ph = (it / C::STAGES) & 1;
      if (!mbar_wait(bar_empty + 8 * s, ph ^ 1, abort_flag, status)) { ok = false; break; }
      const int left = n_iter - it;               // tiles this CTA still has to issue
      int flags = 0;
      if (!piece_open) {
        flags |= kFlagFirst;
        const bool whole = (ti == 0) && (left >= tiles_b);
        piece_slot = whole ? -1 : 2 * static_cast<int>(blockIdx.x) + (it == 0 ? 0 : 1);
        piece_open = true;
      }
      const bool is_step = (ti == tiles_b - 1);
      if (is_step) flags |= kFlagStep;
      if (is_step || left == 1) flags |= kFlagLast;
      TileMeta m;
      m.b = b; m.kvh = h; m.flags = flags; m.rows = n_q * a.G; m.n_c = n_c; m.r0 = r0;
      m.slot = piece_slot;
      m.nvalid = is_step ? n_q : min(kTile, L - ti * kTile);
      meta[s] = m;
      const uint32_t dst = smem_base + s * C::STAGE_BYTES;
      const uint32_t bar = bar_full + 8 * s;
      // order earlier generic-proxy writes to this stage (zero fill) before the async-proxy writes
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      if (is_step) {
        mbar_arrive_expect_tx(bar, 2u * C::HALVES * 16 * 128);
#pragma unroll
        for (int hf = 0; hf < C::HALVES; ++hf) {
          tma_load_3d(dst + hf * (kTile * 128), &map_ks, bar, hf * 64, h, r0);
          tma_load_3d(dst + C::KBYTES + hf * (kTile * 128), &map_vs, bar, hf * 64, h, r0);
        }
      } else {
        mbar_arrive_expect_tx(bar, C::STAGE_BYTES);
        const int y = static_cast<int>(slot_off) + ti * kTile;
#pragma unroll
        for (int hf = 0; hf < C::HALVES; ++hf) {
          tma_load_3d(dst + hf * (kTile * 128), &map_k, bar, hf * 64, y, h);
          tma_load_3d(dst + C::KBYTES + hf * (kTile * 128), &map_v, bar, hf * 64, y, h);
        }
      }
      // advance to the next tile of the flat list
      if (flags & kFlagLast) piece_open = false;
      if (++ti == tiles_b) {
        ti = 0;
        if (++h == a.H_kv) {
          h = 0;
          if (it + 1 < n_iter) {
            do {
              ++b;
              seq_shape(a, b, L, n_q, r0);
              tiles_b = seq_tiles(L, n_q);
            } while (tiles_b == 0 && b + 1 < a.B);
            n_c = a.n_cand[b];
            n_c = n_c < 0 ? 0 : (n_c > n_q ? n_q : n_c);
            slot_off = a.kv_off[b];
          }
        }
      }
    }
    // Drain: every copy this warp issued must have landed before the CTA may exit.
    const int issued = ok ? n_iter : it;
    const int first = issued > C::STAGES ? issued - C::STAGES : 0;
    for (int j = first; j < issued; ++j)
      (void)mbar_wait(bar_full + 8 * (j % C::STAGES), (j / C::STAGES) & 1, abort_flag, status);
    return;
  }

  // ============================= consumer warps =============================
  const int mb = warp / C::KS, ks = warp % C::KS;
  const int quad = lane >> 2, qlane = lane & 3;
  const int row_lo = mb * 16 + quad;            // this thread's two packed rows: row_lo, row_lo + 8
  uint32_t qf[D / 16][4];
  float o[D / 8][4];
  float m_run[2], l_run[2];
  int tok[2], anc[2];                            // step-local token index / visible candidates
  uint32_t merge_phase = 0;

  for (int it = 0; it < n_iter; ++it) {
    const int s = it % C::STAGES;
    const uint32_t ph = (it / C::STAGES) & 1;
    if (!mbar_wait(bar_full + 8 * s, ph, abort_flag, status)) return;
    const TileMeta mt = meta[s];
    const uint32_t k_base = smem_base + s * C::STAGE_BYTES;
    const uint32_t v_base = k_base + C::KBYTES;

    if (mt.flags & kFlagFirst) {
      // new unit (or new part of one): load this row block's Q fragments, reset the state
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const int r = row_lo + 8 * hh;
        const __nv_bfloat16* qp = nullptr;
        tok[hh] = 1 << 20;                       // padded row: sees no step-local key
        anc[hh] = 0;
        if (r < mt.rows) {
          const int i = r / a.G, g = r - i * a.G;
          qp = a.q + (static_cast<int64_t>(mt.r0 + i) * a.H_q + mt.kvh * a.G + g) * D;
          tok[hh] = i;
          anc[hh] = (i < mt.n_c) ? i : (a.anchor ? a.anchor[mt.r0 + i] : mt.n_c);
        }
#pragma unroll
        for (int kb = 0; kb < D / 16; ++kb) {
          const int col = kb * 16 + 2 * qlane;
          qf[kb][hh] = qp ? __ldg(reinterpret_cast<const uint32_t*>(qp + col)) : 0u;
          qf[kb][2 + hh] = qp ? __ldg(reinterpret_cast<const uint32_t*>(qp + col + 8)) : 0u;
        }
      }
#pragma unroll
      for (int nb = 0; nb < D / 8; ++nb) { o[nb][0] = o[nb][1] = o[nb][2] = o[nb][3] = 0.f; }
      m_run[0] = m_run[1] = -INFINITY;
      l_run[0] = l_run[1] = 0.f;
    }

    const int my_valid = min(C::NKW, mt.nvalid - ks * C::NKW);   // valid keys in this warp's slice
#pragma unroll
    for (int sub = 0; sub < C::NSUB; ++sub) {
      const int nv = min(C::SUB, my_valid - sub * C::SUB);
      if (nv <= 0) break;
      const int key_base = ks * C::NKW + sub * C::SUB;          // row of the tile
      const bool ragged = (nv < C::SUB);
      if (ragged) {
        // rows past the valid keys hold foreign or stale bytes: P is 0 there, but 0 * NaN is
        // NaN, so clear this warp's view of those V rows before the PV product
        const int n_rows = C::SUB - nv;
        for (int w = lane; w < n_rows * C::HALVES * 8; w += 32) {
          const int rr = key_base + nv + w / (C::HALVES * 8);
          const int cc = w % (C::HALVES * 8);
          const uint32_t addr = v_base + (cc >> 3) * (kTile * 128) + rr * 128 + ((cc & 7) << 4);
          asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(addr), "r"(0u) : "memory");
        }
        __syncwarp();
      }
      // ---- S = Q K^T for SUB keys ----
      float sc[C::SUB / 8][4];
#pragma unroll
      for (int nb = 0; nb < C::SUB / 8; ++nb) {
        sc[nb][0] = sc[nb][1] = sc[nb][2] = sc[nb][3] = 0.f;
        const int krow = key_base + nb * 8 + (lane & 7);
#pragma unroll
        for (int q4 = 0; q4 < D / 32; ++q4) {
          const int chunk = q4 * 4 + (lane >> 3);
          const uint32_t addr = k_base + (chunk >> 3) * (kTile * 128) + krow * 128 +
                                (((chunk & 7) ^ (krow & 7)) << 4);
          uint32_t b0, b1, b2, b3;
          ldsm_x4(addr, b0, b1, b2, b3);
          mma_bf16(sc[nb], qf[2 * q4], b0, b1);
          mma_bf16(sc[nb], qf[2 * q4 + 1], b2, b3);
        }
      }
      // ---- mask (length bound; step-local visibility) ----
      if (ragged || (mt.flags & kFlagStep)) {
        const bool step = (mt.flags & kFlagStep) != 0;
#pragma unroll
        for (int nb = 0; nb < C::SUB / 8; ++nb) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int j = nb * 8 + 2 * qlane + (e & 1);   // key index inside this softmax step
            const int hh = e >> 1;
            bool vis = j < nv;
            if (step) vis = vis && step_key_visible(tok[hh], key_base + j, mt.n_c, anc[hh]);
            if (!vis) sc[nb][e] = -INFINITY;
          }
        }
      }
      // ---- online softmax (exp2 domain) ----
      float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
      for (int nb = 0; nb < C::SUB / 8; ++nb) {
        mx[0] = fmaxf(mx[0], fmaxf(sc[nb][0], sc[nb][1]));
        mx[1] = fmaxf(mx[1], fmaxf(sc[nb][2], sc[nb][3]));
      }
      float alpha[2], msub[2];
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        mx[hh] = fmaxf(mx[hh], __shfl_xor_sync(0xffffffffu, mx[hh], 1));
        mx[hh] = fmaxf(mx[hh], __shfl_xor_sync(0xffffffffu, mx[hh], 2));
        const float m_new = fmaxf(m_run[hh], mx[hh] * a.scale_log2);
        msub[hh] = (m_new == -INFINITY) ? 0.f : m_new;
        alpha[hh] = exp2f(m_run[hh] - msub[hh]);
        m_run[hh] = m_new;
      }
      uint32_t pf[C::SUB / 16][4];
      float psum[2] = {0.f, 0.f};
#pragma unroll
      for (int nb = 0; nb < C::SUB / 8; ++nb) {
        const float p0 = exp2f(sc[nb][0] * a.scale_log2 - msub[0]);
        const float p1 = exp2f(sc[nb][1] * a.scale_log2 - msub[0]);
        const float p2 = exp2f(sc[nb][2] * a.scale_log2 - msub[1]);
        const float p3 = exp2f(sc[nb][3] * a.scale_log2 - msub[1]);
        psum[0] += p0 + p1;
        psum[1] += p2 + p3;
        pf[nb >> 1][(nb & 1) * 2 + 0] = pack_bf16(p0, p1);
        pf[nb >> 1][(nb & 1) * 2 + 1] = pack_bf16(p2, p3);
      }
      l_run[0] = l_run[0] * alpha[0] + psum[0];
      l_run[1] = l_run[1] * alpha[1] + psum[1];
#pragma unroll
      for (int nb = 0; nb < D / 8; ++nb) {
        o[nb][0] *= alpha[0]; o[nb][1] *= alpha[0];
        o[nb][2] *= alpha[1]; o[nb][3] *= alpha[1];
      }
      // ---- O += P V ----
#pragma unroll
      for (int kb = 0; kb < C::SUB / 16; ++kb) {
        const int vrow = key_base + kb * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
        for (int dn = 0; dn < D / 8; dn += 2) {
          const int chunk = dn + (lane >> 4);
          const uint32_t addr = v_base + (chunk >> 3) * (kTile * 128) + vrow * 128 +
                                (((chunk & 7) ^ (vrow & 7)) << 4);
          uint32_t b0, b1, b2, b3;
          ldsm_x4_trans(addr, b0, b1, b2, b3);
          mma_bf16(o[dn], pf[kb], b0, b1);
          mma_bf16(o[dn + 1], pf[kb], b2, b3);
        }
      }
    }
    // this warp is done with the stage
    if (my_valid > 0 && my_valid < C::NKW) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncwarp();
    if (lane == 0) mbar_arrive(bar_empty + 8 * s);

    if (!(mt.flags & kFlagLast)) continue;

    // ---- end of the unit (or of this CTA's part of it): combine the key slices ----
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      l_run[hh] += __shfl_xor_sync(0xffffffffu, l_run[hh], 1);
      l_run[hh] += __shfl_xor_sync(0xffffffffu, l_run[hh], 2);
    }
    float* mo = reinterpret_cast<float*>(smem + C::OFF_MERGE_O);
    float* mml = reinterpret_cast<float*>(smem + C::OFF_MERGE_ML);
#pragma unroll
    for (int stride = C::KS / 2; stride >= 1; stride >>= 1) {
      if (ks >= stride && ks < 2 * stride) {
        const int slot = mb * (C::KS / 2) + (ks - stride);
        float* po = mo + static_cast<size_t>(slot) * C::OREGS * 32;
#pragma unroll
        for (int nb = 0; nb < D / 8; ++nb)
#pragma unroll
          for (int e = 0; e < 4; ++e) po[(nb * 4 + e) * 32 + lane] = o[nb][e];
        float* pm = mml + slot * 128;
        pm[lane] = m_run[0]; pm[32 + lane] = m_run[1];
        pm[64 + lane] = l_run[0]; pm[96 + lane] = l_run[1];
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_merge);
      if (!mbar_wait(bar_merge, merge_phase, abort_flag, status)) return;
      merge_phase ^= 1;
      if (ks < stride) {
        const int slot = mb * (C::KS / 2) + ks;
        const float* po = mo + static_cast<size_t>(slot) * C::OREGS * 32;
        const float* pm = mml + slot * 128;
        float fa[2], fb[2];
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          const float m2 = pm[hh * 32 + lane], l2 = pm[64 + hh * 32 + lane];
          const float mm = fmaxf(m_run[hh], m2);
          const float ms_ = (mm == -INFINITY) ? 0.f : mm;
          fa[hh] = exp2f(m_run[hh] - ms_);
          fb[hh] = exp2f(m2 - ms_);
          l_run[hh] = l_run[hh] * fa[hh] + l2 * fb[hh];
          m_run[hh] = mm;
        }
#pragma unroll
        for (int nb = 0; nb < D / 8; ++nb)
#pragma unroll
          for (int e = 0; e < 4; ++e)
            o[nb][e] = o[nb][e] * fa[e >> 1] + po[(nb * 4 + e) * 32 + lane] * fb[e >> 1];
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_merge);
      if (!mbar_wait(bar_merge, merge_phase, abort_flag, status)) return;
      merge_phase ^= 1;
    }
    if (ks != 0) continue;

    // ---- slice 0 holds the unit's (m, l, O): write it out ----
    if (mt.slot < 0) {
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const int r = row_lo + 8 * hh;
        if (r >= mt.rows) continue;
        const int i = r / a.G, g = r - i * a.G;
        const int64_t orow = static_cast<int64_t>(mt.r0 + i) * a.H_q + mt.kvh * a.G + g;
        const float inv = 1.f / l_run[hh];
        __nv_bfloat16* op = a.out + orow * D;
#pragma unroll
        for (int nb = 0; nb < D / 8; ++nb)
          *reinterpret_cast<uint32_t*>(op + nb * 8 + 2 * qlane) =
              pack_bf16(o[nb][2 * hh] * inv, o[nb][2 * hh + 1] * inv);
        if (a.lse && qlane == 0) a.lse[orow] = (m_run[hh] + log2f(l_run[hh])) * 0.69314718055994531f;
      }
    } else {
      float* slot = ws_slots + static_cast<size_t>(mt.slot) * ws_slot_floats(D, rows_pad);
      float* sm = slot + static_cast<size_t>(rows_pad) * D;
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const int r = row_lo + 8 * hh;
        if (r >= mt.rows) continue;
#pragma unroll
        for (int nb = 0; nb < D / 8; ++nb)
          *reinterpret_cast<float2*>(slot + static_cast<size_t>(r) * D + nb * 8 + 2 * qlane) =
              make_float2(o[nb][2 * hh], o[nb][2 * hh + 1]);
        if (qlane == 0) {
          sm[r] = m_run[hh];
          sm[rows_pad + r] = l_run[hh];
        }
      }
    }
  }
}

// ---------------------------------------------------------------- merge kernel

// The merge as a launch of its own (used when the split kernel does not merge in its tail): one
// CTA per (layer, sequence, KV head) unit and group of four packed rows, one warp per packed row
// (merge_row).  Units that lie inside one CTA of the split kernel were written by it: nothing to do.
template <int D>
__global__ void __launch_bounds__(128)
attn_merge_kernel(const AttnArgs a, int rows_pad, int n_ctas) {
  pdl_wait();
  pdl_trigger();
  const int units_per_layer = a.B * a.H_kv;
  const int layer = blockIdx.x / units_per_layer, bh = blockIdx.x - layer * units_per_layer;
  const int b = bh / a.H_kv, h = bh - b * a.H_kv;
  const int* ws_pre = reinterpret_cast<const int*>(reinterpret_cast<const uint8_t*>(a.workspace) +
                                                   kWsHeaderBytes);
  const float* ws_slots = reinterpret_cast<const float*>(
      reinterpret_cast<const uint8_t*>(a.workspace) + kWsHeaderBytes + ws_prefix_bytes());
  const int tiles_b = ws_pre[b + 1] - ws_pre[b];
  if (tiles_b == 0) return;
  const long long per_layer = static_cast<long long>(ws_pre[a.B]) * a.H_kv;
  const long long u0 = layer * per_layer + static_cast<long long>(ws_pre[b]) * a.H_kv +
                       static_cast<long long>(h) * tiles_b;
  CutUnit cu;
  if (!cut_unit(per_layer * a.n_layers, n_ctas, u0, u0 + tiles_b, cu)) return;   // whole unit inside one CTA
  int L, n_q, r0;
  seq_shape(a, b, L, n_q, r0);
  const int rows = n_q * a.G;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int r = blockIdx.y * 4 + warp;           // this warp's packed row
  if (r >= rows) return;
  const int i = r / a.G, g = r - i * a.G;
  const int64_t orow = static_cast<int64_t>(r0 + i) * a.H_q + h * a.G + g;
  merge_row<D>(ws_slots, rows_pad, cu, r, lane, a.out + layer * a.out_layer_stride + orow * D,
               a.lse ? a.lse + layer * a.lse_layer_stride + orow : nullptr);
}

// ---------------------------------------------------------------- host side

template <int D, int MB>
int32_t launch_split(const AttnArgs& a, cudaStream_t st, int rows_pad, int grid,
                     const CUtensorMap& mk, const CUtensorMap& mv, const CUtensorMap& mks,
                     const CUtensorMap& mvs) {
  using C = Cfg<D, MB>;
  static bool configured[64] = {false};
  int dev = 0;
  MS_CUDA_TRY(cudaGetDevice(&dev));
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    MS_CUDA_TRY(cudaFuncSetAttribute(attn_split_kernel<D, MB>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES));
    configured[dev] = true;
  }
  if (a.ev_split_begin) MS_CUDA_TRY(cudaEventRecord(a.ev_split_begin, st));
  attn_split_kernel<D, MB><<<grid, kThreads, C::SMEM_BYTES, st>>>(a, mk, mv, mks, mvs, rows_pad);
  MS_LAUNCH_CHECK();
  if (a.ev_split_end) MS_CUDA_TRY(cudaEventRecord(a.ev_split_end, st));
  return MS_OK;
}

}  // namespace

int attn_mma_grid() { return sm_count(); }

size_t attn_mma_workspace_bytes(int D, int rows_pad, int n_ctas) {
  return kWsHeaderBytes + ws_prefix_bytes() +
         static_cast<size_t>(2) * n_ctas * ws_slot_floats(D, rows_pad) * sizeof(float);
}

int32_t launch_attn_mma(const AttnArgs& a, cudaStream_t st) {
  if (a.B == 0 || a.T == 0) return MS_OK;
  const int rows = a.max_nq * a.G;
  const int rows_pad = (rows + 15) & ~15;
  const int mb = rows_pad <= 16 ? 1 : (rows_pad <= 32 ? 2 : 4);
  const int grid = attn_mma_grid();
  if (grid <= 0) return cuda_status(cudaErrorNoDevice);
  CUtensorMap mk, mv, mks, mvs;
  const bool ok =
      make_map(&mk, a.k_cache, a.D, static_cast<uint64_t>(a.n_slots), a.H_kv, a.D, a.kv_head_stride, kTile, 1) &&
      make_map(&mv, a.v_cache, a.D, static_cast<uint64_t>(a.n_slots), a.H_kv, a.D, a.kv_head_stride, kTile, 1) &&
      make_map(&mks, a.k_step, a.D, a.H_kv, a.T, a.D, static_cast<uint64_t>(a.H_kv) * a.D, 1, kMaxNq) &&
      make_map(&mvs, a.v_step, a.D, a.H_kv, a.T, a.D, static_cast<uint64_t>(a.H_kv) * a.D, 1, kMaxNq);
  if (!ok) return cuda_status(cudaErrorInvalidValue);
  int32_t rc;
  if (a.D == 128) {
    rc = mb == 1 ? launch_split<128, 1>(a, st, rows_pad, grid, mk, mv, mks, mvs)
       : mb == 2 ? launch_split<128, 2>(a, st, rows_pad, grid, mk, mv, mks, mvs)
                 : launch_split<128, 4>(a, st, rows_pad, grid, mk, mv, mks, mvs);
  } else {
    rc = mb == 1 ? launch_split<64, 1>(a, st, rows_pad, grid, mk, mv, mks, mvs)
       : mb == 2 ? launch_split<64, 2>(a, st, rows_pad, grid, mk, mv, mks, mvs)
                 : launch_split<64, 4>(a, st, rows_pad, grid, mk, mv, mks, mvs);
  }
  if (rc != MS_OK) return rc;
  return launch_attn_merge(a, st, rows_pad, grid);
}

int32_t launch_attn_merge(const AttnArgs& a, cudaStream_t st, int rows_pad, int n_ctas) {
  const dim3 grid(static_cast<unsigned>(a.n_layers * a.B * a.H_kv), static_cast<unsigned>((rows_pad + 3) / 4));
  if (a.D == 128)
    MS_CUDA_TRY(launch_pdl(attn_merge_kernel<128>, grid, dim3(128), 0, st, a, rows_pad, n_ctas));
  else
    MS_CUDA_TRY(launch_pdl(attn_merge_kernel<64>, grid, dim3(128), 0, st, a, rows_pad, n_ctas));
  return MS_OK;
}

}  // namespace ms
