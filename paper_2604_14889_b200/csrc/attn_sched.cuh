// Pieces shared by the two tensor-core paths of the step attention: the flat tile
// schedule (every 128-key tile of every (sequence, KV head) unit, cut into one
// contiguous range per persistent CTA), the layout of the split-KV workspace, the
// mbarrier / TMA wrappers with bounded waits, and the tensor-map builder.
#pragma once

#include "attn_internal.cuh"

namespace ms {

constexpr int kTile = 128;                 // keys per pipeline stage
constexpr uint32_t kTimeoutMagic = 0x4D535431u;
constexpr unsigned int kWaitLimitDefaultUs = 4000000u;   // 4 s: far beyond anything but a dead device

// Every bounded wait of a CTA shares two shared-memory words: [0] the abort flag, [1] the limit of
// one wait in microseconds (a launch parameter, see wait_limit_us()).
__device__ __forceinline__ void wait_ctx_init(volatile int* ctx, unsigned int limit_us) {
  ctx[0] = 0;
  ctx[1] = static_cast<int>(limit_us);
}
__device__ __forceinline__ unsigned long long wait_limit_ns(volatile int* ctx) {
  return static_cast<unsigned long long>(static_cast<unsigned int>(ctx[1])) * 1000ull;
}

// ---------------------------------------------------------------- PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false if the CTA is aborting or the limit ran out (and
// then records the timeout in the workspace status word and raises the abort flag).
static __device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                            uint32_t* status) {
  const unsigned long long t0 = global_ns(), limit = wait_limit_ns(abort_flag);
  for (uint32_t spin = 1;; ++spin) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spin & 63u) == 0) {
      if (*abort_flag) return false;
      if (global_ns() - t0 > limit) {
        *abort_flag = 1;
        atomicExch(status, kTimeoutMagic);
        return false;
      }
    }
  }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          uint32_t* status) {
  if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, abort_flag, status);
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x,
                                            int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x,
                                            int y, int z, int w) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z), "r"(w)
      : "memory");
}
// Tiles of sequence b: its cache tiles plus the step-local tile; 0 if the block is empty.
__device__ __forceinline__ void seq_shape(const AttnArgs& a, int b, int& L, int& n_q, int& r0) {
  r0 = a.q_off[b];
  n_q = a.q_off[b + 1] - r0;
  n_q = n_q < 0 ? 0 : (n_q > a.max_nq ? a.max_nq : n_q);
  L = a.kv_len[b];
  L = L < 0 ? 0 : (L > a.max_kv_len ? a.max_kv_len : L);
}
__device__ __forceinline__ int seq_tiles(int L, int n_q) {
  return n_q > 0 ? (L + kTile - 1) / kTile + 1 : 0;
}

// Exclusive prefix sum of seq_tiles over the batch into pre[0..B] (shared memory).  Every thread
// takes a contiguous run of sequences; the runs are scanned with warp shuffles and one
// shared-memory slot per warp (scratch: at least blockDim.x / 32 ints).
static __device__ void build_tile_prefix(const AttnArgs& a, int* pre, int* scratch) {
  const int nt = blockDim.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int per = (a.B + nt - 1) / nt;
  const int lo = min(a.B, tid * per), hi = min(a.B, lo + per);
  int sum = 0;
  for (int b = lo; b < hi; ++b) {
    int L, n_q, r0;
    seq_shape(a, b, L, n_q, r0);
    sum += seq_tiles(L, n_q);
  }
  int incl = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int up = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += up;
  }
  if (lane == 31) scratch[warp] = incl;
  __syncthreads();
  int base = incl - sum;
  for (int w = 0; w < warp; ++w) base += scratch[w];
  for (int b = lo; b < hi; ++b) {
    int L, n_q, r0;
    seq_shape(a, b, L, n_q, r0);
    pre[b] = base;
    base += seq_tiles(L, n_q);
  }
  if (tid == nt - 1) pre[a.B] = base;
  __syncthreads();
}

// Layout of the workspace behind the header.
__device__ __host__ inline size_t ws_prefix_bytes() { return (static_cast<size_t>(kMaxBatch) + 64) * 4; }
__device__ __host__ inline size_t ws_slot_floats(int D, int rows_pad) {
  return static_cast<size_t>(rows_pad) * (D + 2);
}

// ---------------------------------------------------------------- host side

// Tiled bf16 tensor map with 128-byte swizzle over a tensor of `rank` dimensions (innermost
// first: dims[0] = head_dim), box[0] = 64 columns.  Encoded maps are kept in a small cache keyed
// by every argument, so that a decoding loop that calls with the same buffers encodes nothing
// (attn_api.cu).
bool tensor_map_cached(CUtensorMap* map, int rank, const void* base, const uint64_t* dims,
                       const uint64_t* strides_bytes, const uint32_t* box);

// bf16 tensor [d2][d1][D] (D innermost), box = 64 columns x box1 x box2, 128-byte swizzle.
inline bool make_map(CUtensorMap* map, const void* base, int D, uint64_t d1, uint64_t d2,
              uint64_t stride1_elems, uint64_t stride2_elems, uint32_t box1, uint32_t box2) {
  const uint64_t dims[3] = {static_cast<uint64_t>(D), d1, d2};
  const uint64_t strides[2] = {stride1_elems * 2, stride2_elems * 2};
  const uint32_t box[3] = {64, box1, box2};
  return tensor_map_cached(map, 3, base, dims, strides, box);
}

// bf16 tensor [d3][d2][d1][D], box = 64 columns x box1 x box2 x 1.
inline bool make_map4(CUtensorMap* map, const void* base, int D, uint64_t d1, uint64_t d2, uint64_t d3,
               uint64_t stride1_elems, uint64_t stride2_elems, uint64_t stride3_elems, uint32_t box1,
               uint32_t box2) {
  const uint64_t dims[4] = {static_cast<uint64_t>(D), d1, d2, d3};
  const uint64_t strides[3] = {stride1_elems * 2, stride2_elems * 2, stride3_elems * 2};
  const uint32_t box[4] = {64, box1, box2, 1};
  return tensor_map_cached(map, 4, base, dims, strides, box);
}

// ---------------------------------------------------------------- merge of a cut unit

// A unit (sequence, KV head[, layer]) is the range [u0, u1) of the flat tile list; persistent CTA
// i owns the tiles [n_tiles * i / n_ctas, n_tiles * (i + 1) / n_ctas).  A unit that spans more
// than one CTA leaves one partial (m, l, O) per CTA: in the CTA's slot 0 when the CTA's range
// starts inside the unit (or with it), in slot 1 otherwise.
struct CutUnit {
  long long n_tiles, u0, u1;
  int n_ctas, c_lo, c_hi;
};
__device__ __forceinline__ bool cut_unit(long long n_tiles, int n_ctas, long long u0, long long u1, CutUnit& cu) {
  cu.n_tiles = n_tiles; cu.u0 = u0; cu.u1 = u1; cu.n_ctas = n_ctas;
  cu.c_lo = static_cast<int>(((u0 + 1) * n_ctas - 1) / n_tiles);
  cu.c_hi = static_cast<int>((u1 * n_ctas - 1) / n_tiles);
  return cu.c_lo != cu.c_hi;
}
// Number of partials a cut unit leaves: every CTA of c_lo..c_hi that has tiles (with fewer tiles
// than CTAs, a CTA holds one tile or none).
__device__ __forceinline__ int cut_pieces(const CutUnit& cu) {
  return cu.n_tiles >= cu.n_ctas ? cu.c_hi - cu.c_lo + 1 : static_cast<int>(cu.u1 - cu.u0);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// One warp merges packed row r of a cut unit: the lanes look up one partial each -- its slot and
// (m, l) -- and fold those with shuffles into the row's maximum and normaliser; then every lane
// accumulates its D/32 output columns over the partials (eight loads in flight), whose slots and
// weights go round by shuffle.  The partials are read past L1 (another SM wrote them).
template <int D>
__device__ __forceinline__ void merge_row(const float* ws_slots, int rows_pad, const CutUnit& cu, int r, int lane,
                                          __nv_bfloat16* out_row, float* lse_out) {
  constexpr int E = D / 32;
  const size_t slot_floats = ws_slot_floats(D, rows_pad);
  float M = -INFINITY, Lsum = 0.f, acc[E];
#pragma unroll
  for (int e = 0; e < E; ++e) acc[e] = 0.f;
  for (int c0 = cu.c_lo; c0 <= cu.c_hi; c0 += 32) {
    const int c = c0 + lane;
    int slot = -1;
    float m = -INFINITY, l = 0.f;
    if (c <= cu.c_hi) {
      const long long s0 = cu.n_tiles * c / cu.n_ctas, s1 = cu.n_tiles * (c + 1) / cu.n_ctas;
      if (s1 > s0) {                             // a CTA with tiles
        slot = 2 * c + ((s0 >= cu.u0) ? 0 : 1);
        const float* sp = ws_slots + slot * slot_floats + static_cast<size_t>(rows_pad) * D;
        m = __ldcg(sp + r);
        l = __ldcg(sp + rows_pad + r);
      }
    }
    float gm = m;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) gm = fmaxf(gm, __shfl_xor_sync(0xffffffffu, gm, o));
    const float M_new = fmaxf(M, gm);
    const float rescale = (M == -INFINITY) ? 0.f : exp2f(M - M_new);
    float w = (m == -INFINITY) ? 0.f : exp2f(m - M_new);
    if (slot < 0) w = 0.f;
    float lw = l * w;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) lw += __shfl_xor_sync(0xffffffffu, lw, o);
    Lsum = Lsum * rescale + lw;
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] *= rescale;
    M = M_new;
    const int cnt = min(32, cu.c_hi - c0 + 1);
    for (int k0 = 0; k0 < cnt; k0 += 8) {
      float x[8][E], wk[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int sk = __shfl_sync(0xffffffffu, slot, (k0 + u) & 31);
        wk[u] = __shfl_sync(0xffffffffu, w, (k0 + u) & 31);
        if (k0 + u >= cnt || sk < 0) wk[u] = 0.f;
        const float* po = ws_slots + (sk < 0 ? 0 : sk) * slot_floats + static_cast<size_t>(r) * D + lane * E;
        if (wk[u] != 0.f) {
          if (E == 4) {
            const float4 v = __ldcg(reinterpret_cast<const float4*>(po));
            x[u][0] = v.x; x[u][1] = v.y; x[u][E - 2] = v.z; x[u][E - 1] = v.w;
          } else {
            const float2 v = __ldcg(reinterpret_cast<const float2*>(po));
            x[u][0] = v.x; x[u][1] = v.y;
          }
        } else {
#pragma unroll
          for (int e = 0; e < E; ++e) x[u][e] = 0.f;
        }
      }
#pragma unroll
      for (int u = 0; u < 8; ++u)
#pragma unroll
        for (int e = 0; e < E; ++e) acc[e] = fmaf(wk[u], x[u][e], acc[e]);
    }
  }
  const float inv = 1.f / Lsum;
#pragma unroll
  for (int e = 0; e < E; e += 2)
    *reinterpret_cast<uint32_t*>(out_row + lane * E + e) = pack_bf16x2(acc[e] * inv, acc[e + 1] * inv);
  if (lse_out && lane == 0) *lse_out = (M + log2f(Lsum)) * 0.69314718055994531f;
}

// Log-sum-exp merge of the units that the split kernel cut across CTAs (attn_mma.cu).
int32_t launch_attn_merge(const AttnArgs& a, cudaStream_t st, int rows_pad, int n_ctas);

}  // namespace ms
