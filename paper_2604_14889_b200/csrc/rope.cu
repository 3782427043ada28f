// RoPE applied in place to the step block's Q and K at token-specific position
// IDs (paper Sec. 2.1.2: the position layouts of memory and foresight tokens act
// through RoPE, so each new token is rotated by its own PID, not by its cache slot).
//
// One CTA per (token, run of heads).  The D/2 angles of the token are evaluated in fp64
// (sincos of pos * theta_i) and kept in shared memory as fp64 and fp32.  The result of
// every element is the fp64 rotation rounded to bf16 once -- but it is computed in fp32
// whenever that provably gives the same bits: the fp32 value carries an error bound, and
// if both ends of the bound round to the same bf16 number, so does the exact value
// (rounding is monotonic).  Only the few elements that sit next to a rounding boundary
// (about one in a thousand) are redone in fp64.
#include <math.h>

#include "common.cuh"

namespace {

constexpr int kMaxHalf = 128;  // D <= 256

struct FreqTable {
  double f[kMaxHalf];
};

__device__ __forceinline__ uint16_t f64_to_bf16_bits(double x) {
  // One rounding fp64 -> bf16 (round to nearest even).  Going through fp32
  // would round twice; instead round the fp64 significand directly: bf16 keeps
  // 8 significant bits, i.e. drops the low 45 bits of the 53-bit significand.
  if (x != x) return 0x7FC0;
  const double ax = fabs(x);
  if (ax >= 3.3961775292304601e38) {            // >= max bf16 + half ulp: overflow to inf
    return static_cast<uint16_t>((x < 0 ? 0x8000u : 0u) | 0x7F80u);
  }
  if (ax < 1.1754943508222875e-38) {            // below the smallest normal: fixed spacing 2^-133
    const double q = rint(ax * 0x1p133);         // exact scaling, RNE
    const uint32_t m = static_cast<uint32_t>(q); // 0 .. 128 (128 = smallest normal)
    return static_cast<uint16_t>((x < 0 ? 0x8000u : 0u) | m);
  }
  uint64_t b = static_cast<uint64_t>(__double_as_longlong(ax));
  const uint64_t drop = 45;
  const uint64_t half = 1ull << (drop - 1);
  const uint64_t rem = b & ((1ull << drop) - 1);
  b >>= drop;                                     // exponent(11) | top 7 mantissa bits
  if (rem > half || (rem == half && (b & 1))) b += 1;   // carries into the exponent correctly
  const int32_t e = static_cast<int32_t>(b >> 7) - 1023 + 127;   // rebias
  const uint32_t out = (static_cast<uint32_t>(e) << 7) | static_cast<uint32_t>(b & 0x7F);
  return static_cast<uint16_t>((x < 0 ? 0x8000u : 0u) | out);
}

// a*c - b*s (sign = -1) or a*c + b*s (sign = +1), a and b exact bf16 values, rounded to bf16 once.
__device__ __forceinline__ uint16_t rot_elem(float a, float b, float c32, float s32, double c64, double s64,
                                             float sign) {
  const float bs = b * s32;
  const float r = fmaf(a, c32, sign * bs);
  // |r - exact| <= (|a c| + |b s|) * 3 * 2^-24 (two rounded constants, one rounded product, one
  // rounded sum) + denormal slack; 5 * 2^-24 leaves room for the rounding of the bound itself
  const float e = (fabsf(a * c32) + fabsf(bs)) * 2.98e-7f + 1e-44f;
  const __nv_bfloat16 lo = __float2bfloat16_rn(r - e), hi = __float2bfloat16_rn(r + e);
  const uint16_t lo_b = *reinterpret_cast<const uint16_t*>(&lo), hi_b = *reinterpret_cast<const uint16_t*>(&hi);
  if (lo_b == hi_b && r == r) return lo_b;
  const double ad = static_cast<double>(a), bd = static_cast<double>(b);
  return f64_to_bf16_bits(sign < 0.f ? ad * c64 - bd * s64 : ad * c64 + bd * s64);
}

__device__ __forceinline__ float bf16_bits_to_f32(uint16_t h) {
  return __uint_as_float(static_cast<uint32_t>(h) << 16);
}

constexpr int kRopeThreads = 128;

__global__ void __launch_bounds__(kRopeThreads)
rope_qk_kernel(uint16_t* __restrict__ q, uint16_t* __restrict__ k, const int32_t* __restrict__ pos_id,
               int H_q, int H_kv, int D, int heads_per_cta, uint32_t flags, bool vec_ok, FreqTable freq) {
  __shared__ double s_cos[kMaxHalf];
  __shared__ double s_sin[kMaxHalf];
  __shared__ float s_cos32[kMaxHalf];
  __shared__ float s_sin32[kMaxHalf];
  ms::pdl_wait();
  ms::pdl_trigger();
  const int t = blockIdx.x;
  const int half = D >> 1;
  double p = static_cast<double>(pos_id[t]);
  if (flags & MS_POS_HALF_UNITS) p *= 0.5;
  for (int i = threadIdx.x; i < half; i += blockDim.x) {
    double s, c;
    sincos(p * freq.f[i], &s, &c);
    s_cos[i] = c;
    s_sin[i] = s;
    s_cos32[i] = static_cast<float>(c);
    s_sin32[i] = static_cast<float>(s);
  }
  __syncthreads();
  const bool interleaved = (flags & MS_ROPE_INTERLEAVED) != 0;
  const int n_heads = H_q + H_kv;
  const int h_lo = blockIdx.y * heads_per_cta;
  const int n_mine = min(heads_per_cta, n_heads - h_lo);
  if (vec_ok && (half & 7) == 0) {
    // 16-byte accesses: a work item is 8 consecutive pair indices of one head (rotate-half: 8
    // elements of each half) or 4 of them (interleaved: 8 consecutive elements)
    const int per_head = interleaved ? half / 4 : half / 8;
    for (int w = threadIdx.x; w < n_mine * per_head; w += blockDim.x) {
      const int hh = w / per_head, c = w - hh * per_head, h = h_lo + hh;
      uint16_t* v = (h < H_q) ? q + (static_cast<int64_t>(t) * H_q + h) * D
                              : k + (static_cast<int64_t>(t) * H_kv + (h - H_q)) * D;
      if (interleaved) {
        uint4* pv = reinterpret_cast<uint4*>(v + 8 * c);
        uint4 x = *pv;
        uint16_t* e = reinterpret_cast<uint16_t*>(&x);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int i = 4 * c + j;
          const float a = bf16_bits_to_f32(e[2 * j]), b = bf16_bits_to_f32(e[2 * j + 1]);
          e[2 * j] = rot_elem(a, b, s_cos32[i], s_sin32[i], s_cos[i], s_sin[i], -1.f);
          e[2 * j + 1] = rot_elem(b, a, s_cos32[i], s_sin32[i], s_cos[i], s_sin[i], 1.f);
        }
        *pv = x;
      } else {
        uint4* pa = reinterpret_cast<uint4*>(v + 8 * c);
        uint4* pb = reinterpret_cast<uint4*>(v + half + 8 * c);
        uint4 xa = *pa, xb = *pb;
        uint16_t* ea = reinterpret_cast<uint16_t*>(&xa);
        uint16_t* eb = reinterpret_cast<uint16_t*>(&xb);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int i = 8 * c + j;
          const float a = bf16_bits_to_f32(ea[j]), b = bf16_bits_to_f32(eb[j]);
          ea[j] = rot_elem(a, b, s_cos32[i], s_sin32[i], s_cos[i], s_sin[i], -1.f);
          eb[j] = rot_elem(b, a, s_cos32[i], s_sin32[i], s_cos[i], s_sin[i], 1.f);
        }
        *pa = xa;
        *pb = xb;
      }
    }
    return;
  }
  for (int w = threadIdx.x; w < n_mine * half; w += blockDim.x) {
    const int hh = w / half, i = w - hh * half, h = h_lo + hh;
    uint16_t* v = (h < H_q) ? q + (static_cast<int64_t>(t) * H_q + h) * D
                            : k + (static_cast<int64_t>(t) * H_kv + (h - H_q)) * D;
    const int ia = interleaved ? 2 * i : i;
    const int ib = interleaved ? 2 * i + 1 : i + half;
    const float a = bf16_bits_to_f32(v[ia]), b = bf16_bits_to_f32(v[ib]);
    v[ia] = rot_elem(a, b, s_cos32[i], s_sin32[i], s_cos[i], s_sin[i], -1.f);
    v[ib] = rot_elem(b, a, s_cos32[i], s_sin32[i], s_cos[i], s_sin[i], 1.f);
  }
}

}  // namespace

extern "C" int32_t memosight_rope_qk(void* q, void* k, const int32_t* pos_id, int32_t T, int32_t H_q,
                                     int32_t H_kv, int32_t D, double rope_base,
                                     const double* inv_freq, uint32_t flags,
                                     memosight_stream_t stream) {
  if (T < 0 || H_q < 0 || H_kv < 0) return MS_ERR_INVALID_ARG;
  if (D < 2 || (D & 1) || D > 2 * kMaxHalf) return MS_ERR_UNSUPPORTED_SHAPE;
  if (flags & ~(MS_ROPE_INTERLEAVED | MS_POS_HALF_UNITS)) return MS_ERR_INVALID_ARG;
  if (T == 0 || H_q + H_kv == 0) return MS_OK;
  if (!pos_id || (H_q > 0 && !q) || (H_kv > 0 && !k)) return MS_ERR_INVALID_ARG;
  if (!inv_freq && !(rope_base > 0.0)) return MS_ERR_INVALID_ARG;
  FreqTable freq;
  for (int i = 0; i < D / 2; ++i)
    freq.f[i] = inv_freq ? inv_freq[i] : pow(rope_base, -2.0 * static_cast<double>(i) / D);
  for (int i = D / 2; i < kMaxHalf; ++i) freq.f[i] = 0.0;
  const bool vec_ok = ms::aligned16(q) && ms::aligned16(k);   // NULL (no heads of that kind) counts as aligned
  // few tokens: spread each token's heads over several CTAs (latency); many: one CTA per token, so
  // that the fp64 angles are evaluated once
  const int n_heads = H_q + H_kv;
  const int heads_per_cta = T >= 2048 ? n_heads : (n_heads < 8 ? n_heads : 8);
  const int chunks = (n_heads + heads_per_cta - 1) / heads_per_cta;
  if (chunks > 65535) return MS_ERR_UNSUPPORTED_SHAPE;
  MS_CUDA_TRY(ms::launch_pdl(rope_qk_kernel, dim3(T, chunks), dim3(kRopeThreads), 0, ms::as_stream(stream),
                             static_cast<uint16_t*>(q), static_cast<uint16_t*>(k), pos_id, H_q, H_kv, D,
                             heads_per_cta, flags, vec_ok, freq));
  return MS_OK;
}
