// General (slow) path of the step attention: plain fp32 ALU code for shapes the
// tensor-core path does not cover (head_dim other than 64/128, or more than 64
// packed rows per KV head).  One CTA per (query head, block row); its warps take
// keys round-robin, each lane owns D/32 contiguous elements of the head vector,
// every warp keeps an online-softmax state and the warps are merged at the end.
// Same visibility rule as the fast path: whole cache visible, step-local keys by
// the (n_cand, anchor) metadata.
#include "attn_internal.cuh"

namespace ms {
namespace {

constexpr int kWarps = 4;
constexpr int kMaxE = 8;   // D <= 256

__global__ void __launch_bounds__(kWarps * 32)
attn_simt_kernel(AttnArgs a) {
  const int t = blockIdx.x, hq = blockIdx.y;       // rows on grid.x: no 65535 limit on the block rows
  const int D = a.D, E = D >> 5;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // sequence of this row: largest b with q_off[b] <= t
  int lo = 0, hi = a.B;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (a.q_off[mid] <= t) lo = mid; else hi = mid;
  }
  const int b = lo;
  // block size and cache length are clamped to the host's bounds, as on the tensor-core paths
  const int r0 = a.q_off[b];
  int n_q = a.q_off[b + 1] - r0;
  n_q = n_q < 0 ? 0 : (n_q > a.max_nq ? a.max_nq : n_q);
  if (t < r0 || t >= r0 + n_q) return;
  int n_c = a.n_cand[b];
  n_c = n_c < 0 ? 0 : (n_c > n_q ? n_q : n_c);
  const int i = t - r0;
  const int a_i = (i < n_c) ? i : (a.anchor ? a.anchor[t] : n_c);
  int L = a.kv_len[b];
  L = L < 0 ? 0 : (L > a.max_kv_len ? a.max_kv_len : L);
  const int kvh = hq / a.G;
  const __nv_bfloat16* Kc = a.k_cache + kvh * a.kv_head_stride + a.kv_off[b] * static_cast<int64_t>(D);
  const __nv_bfloat16* Vc = a.v_cache + kvh * a.kv_head_stride + a.kv_off[b] * static_cast<int64_t>(D);

  float qv[kMaxE];
  const __nv_bfloat16* qp = a.q + (static_cast<int64_t>(t) * a.H_q + hq) * D + lane * E;
  for (int e = 0; e < kMaxE; ++e) qv[e] = (e < E) ? __bfloat162float(qp[e]) * a.scale_log2 : 0.f;

  float m = -INFINITY, l = 0.f, acc[kMaxE];
  for (int e = 0; e < kMaxE; ++e) acc[e] = 0.f;
  for (int j = warp; j < L + n_q; j += kWarps) {
    const __nv_bfloat16 *kp, *vp;
    if (j < L) {
      kp = Kc + static_cast<int64_t>(j) * D;
      vp = Vc + static_cast<int64_t>(j) * D;
    } else {
      const int jj = j - L;
      const bool vis = a.tok_kind ? train_key_visible(i, jj, a.tok_kind[r0 + jj], a.tok_step[t], a.tok_step[r0 + jj])
                                  : step_key_visible(i, jj, n_c, a_i);
      if (!vis) continue;                                  // warp-uniform
      kp = a.k_step + (static_cast<int64_t>(r0 + jj) * a.H_kv + kvh) * D;
      vp = a.v_step + (static_cast<int64_t>(r0 + jj) * a.H_kv + kvh) * D;
    }
    float s = 0.f;
    for (int e = 0; e < E; ++e) s += qv[e] * __bfloat162float(kp[lane * E + e]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    const float m_new = fmaxf(m, s);
    const float alpha = exp2f(m - m_new);     // m = -inf at first: exp2(-inf) = 0
    const float p = exp2f(s - m_new);
    l = l * alpha + p;
    for (int e = 0; e < E; ++e) acc[e] = acc[e] * alpha + p * __bfloat162float(vp[lane * E + e]);
    m = m_new;
  }
  // merge the warps (every row sees at least its own key, so some warp has l > 0)
  __shared__ float s_m[kWarps], s_l[kWarps];
  __shared__ float s_acc[kWarps][32 * kMaxE];
  if (lane == 0) { s_m[warp] = m; s_l[warp] = l; }
  for (int e = 0; e < E; ++e) s_acc[warp][lane * E + e] = acc[e];
  __syncthreads();
  if (warp == 0) {
    float M = -INFINITY;
    for (int w = 0; w < kWarps; ++w) M = fmaxf(M, s_m[w]);
    float Lsum = 0.f, o[kMaxE];
    for (int e = 0; e < kMaxE; ++e) o[e] = 0.f;
    for (int w = 0; w < kWarps; ++w) {
      const float f = (s_m[w] == -INFINITY) ? 0.f : exp2f(s_m[w] - M);
      Lsum += s_l[w] * f;
      for (int e = 0; e < E; ++e) o[e] += s_acc[w][lane * E + e] * f;
    }
    const float inv = 1.f / Lsum;
    __nv_bfloat16* op = a.out + (static_cast<int64_t>(t) * a.H_q + hq) * D + lane * E;
    for (int e = 0; e < E; ++e) op[e] = __float2bfloat16_rn(o[e] * inv);
    if (a.lse && lane == 0)
      a.lse[static_cast<int64_t>(t) * a.H_q + hq] = (M + log2f(Lsum)) * 0.69314718055994531f;
  }
}

}  // namespace

int32_t launch_attn_simt(const AttnArgs& a, cudaStream_t st) {
  if (a.T == 0) return MS_OK;
  attn_simt_kernel<<<dim3(a.T, a.H_q), kWarps * 32, 0, st>>>(a);
  MS_LAUNCH_CHECK();
  return MS_OK;
}

}  // namespace ms
