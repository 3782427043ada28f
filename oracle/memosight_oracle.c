/*
 * MemoSight hot-path ORACLE -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, fp64 CPU statement of what the per-step hot path of MemoSight
 * inference computes: position layout (AMA, UPL, <o> and foresight position
 * IDs), RoPE at token-specific position IDs, the masked GQA attention of one
 * Predict+Verify step block over a compacted KV cache, the KV-compaction
 * gather, the append of accepted tokens and the greedy accept rule.
 *
 * Only the tests, the smoke check and the benchmark's cpu_baseline /
 * --impl reference legs may build, load or call this file.  It shares no code
 * with the CUDA path and must never be imported by it.
 *
 * Every function cites the passage of the paper it follows.  There is no
 * blocking, fusion or reordering here: attention is the textbook definition
 * (scores, max, exp, sum, weighted sum) over the set of keys the paper's mask
 * rules make visible; everything else takes the algorithm's steps in the
 * paper's order.  The only concession to wall-clock time is an OpenMP
 * "parallel for" over independent (sequence, query head) units.
 *
 * Parity pins: every function below is pinned by tests/test_oracle_*.py
 * (paper examples, closed forms, brute-force dense masked softmax, library
 * routines).  Still unpinned by anything the paper prints: the rounding of a
 * UPL centre that falls between two integers (only an odd-sized example is
 * given) -- "parity unpinned" for that single choice; see ms_oracle_upl_pids.
 *
 * bf16 tensors travel as uint16_t bit patterns and are widened exactly.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define MS_ORACLE_OK 0
#define MS_ORACLE_BAD_ARG (-1)

/* ------------------------------------------------------------------------ */
/* bf16 <-> fp64                                                             */
/* ------------------------------------------------------------------------ */

/* bf16 is the upper half of an IEEE binary32: widening is exact. */
static double bf16_to_f64(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

/* fp64 -> bf16, one rounding, round-to-nearest-even.  bf16 keeps 8 significant
 * bits (1 implicit + 7 stored) and binary32's exponent range, so the spacing of
 * representable values around |x| = 1.f * 2^E is 2^(E-7), with E clamped at
 * -126 (subnormals).  |x| / spacing is exact (power of two), nearbyint() rounds
 * half to even in the default rounding mode. */
static uint16_t f64_to_bf16(double x) {
  float f;
  if (isnan(x) || isinf(x) || x == 0.0) {
    f = (float)x;
  } else {
    int e2;
    (void)frexp(fabs(x), &e2); /* |x| = m * 2^e2, m in [0.5, 1) */
    int E = e2 - 1;
    if (E < -126) E = -126;
    double spacing = ldexp(1.0, E - 7);
    double r = nearbyint(fabs(x) / spacing) * spacing;
    f = (float)(x < 0 ? -r : r); /* exact, or overflows to inf as it should */
  }
  uint32_t u;
  memcpy(&u, &f, sizeof u);
  if (isnan(x)) u |= 0x00400000u; /* keep it a NaN after truncation */
  return (uint16_t)(u >> 16);
}

void ms_oracle_f64_to_bf16(const double* x, uint16_t* out, int64_t n) {
  for (int64_t i = 0; i < n; ++i) out[i] = f64_to_bf16(x[i]);
}

void ms_oracle_bf16_to_f64(const uint16_t* x, double* out, int64_t n) {
  for (int64_t i = 0; i < n; ++i) out[i] = bf16_to_f64(x[i]);
}

/* ------------------------------------------------------------------------ */
/* Position layout (integer)                                                 */
/* ------------------------------------------------------------------------ */

/* Adaptive Memory Allocation (Sec. 2.1.2; Algorithm 1, Phase 2): a reasoning
 * step of n tokens gets l = ceil(n / c) memory tokens. */
int32_t ms_oracle_ama(int32_t n, int32_t c) {
  if (n < 0 || c < 1) return MS_ORACLE_BAD_ARG;
  int32_t l = 0;
  while ((int64_t)l * c < n) ++l; /* smallest l with l*c >= n */
  return l;
}

/* Uniform Position Layout (Sec. 2.1.2 and its footnote; Sec. 2.2 "Position ID
 * Assignment", memory tokens).  The step's n tokens hold consecutive position
 * IDs rho_first .. rho_first+n-1.  They are cut into l = ceil(n/c) sequential
 * groups of c tokens (the last may be shorter); memory token g gets the centre
 * position of group g.
 *
 * The centre of a group spanning offsets lo..hi is (lo+hi)/2.  The paper's only
 * example (span 1..3, c = 3 -> 2) has an integer centre; for an even-sized
 * group the centre is a half-integer and the paper does not say which way it
 * goes.  Reading taken here: round down (floor); with half_units != 0 the exact
 * centre is returned in units of 1/2 position instead (2*rho_first + lo + hi).
 * Returns l, or a negative code. */
int32_t ms_oracle_upl_pids(int32_t rho_first, int32_t n, int32_t c,
                           int32_t half_units, int32_t* pid_out) {
  int32_t l = ms_oracle_ama(n, c);
  if (l < 0) return l;
  for (int32_t g = 0; g < l; ++g) {
    int32_t lo = g * c;
    int32_t hi = (g + 1) * c;
    if (hi > n) hi = n;
    hi -= 1; /* last offset inside the group */
    if (half_units)
      pid_out[g] = 2 * rho_first + lo + hi;
    else
      pid_out[g] = rho_first + (lo + hi) / 2; /* lo+hi >= 0: this is floor */
  }
  return l;
}

/* Ablation "w/o UPL" (App. B.3): memory tokens take monotonically increasing
 * new position IDs right after the step's last token. */
int32_t ms_oracle_monotone_pids(int32_t rho_first, int32_t n, int32_t c,
                                int32_t* pid_out) {
  int32_t l = ms_oracle_ama(n, c);
  if (l < 0) return l;
  for (int32_t g = 0; g < l; ++g) pid_out[g] = rho_first + n + g;
  return l;
}

/* Ablation "w/o AMA" (App. B.3): a fixed budget of l memory tokens per step whatever its
 * length n.  The paper does not say where they sit; reading taken here: the step is cut
 * into l groups as evenly as possible, group g = offsets floor(g*n/l) .. floor((g+1)*n/l)-1,
 * and memory token g takes its group's centre (floor), exactly as UPL does for its groups;
 * a group left empty (n < l) takes the position it would start at, clamped into the step.
 * Parity unpinned beyond the invariants.  Returns l, or a negative code. */
int32_t ms_oracle_budget_pids(int32_t rho_first, int32_t n, int32_t l, int32_t* pid_out) {
  if (n < 1 || l < 1) return MS_ORACLE_BAD_ARG;
  for (int32_t g = 0; g < l; ++g) {
    int64_t lo = (int64_t)g * n / l, hi = (int64_t)(g + 1) * n / l - 1;
    if (hi < lo) hi = lo;                /* empty group */
    if (lo > n - 1) lo = n - 1;
    if (hi > n - 1) hi = n - 1;
    pid_out[g] = rho_first + (int32_t)((lo + hi) / 2);
  }
  return l;
}

/* Output token <o> (Sec. 2.2 "Position ID Assignment"): PID of the step's last
 * reasoning token plus one, so reasoning and output tokens are consecutive. */
int32_t ms_oracle_out_pid(int32_t rho_first, int32_t n) {
  return rho_first + n - 1 + 1;
}

/* Position IDs of one step block (Sec. 2.1.1; Sec. 2.2 foresight tokens).
 * Rows 0..n_c-1 are the pending candidate (regular) tokens: consecutive PIDs
 * p0, p0+1, ...  Rows n_c..n_c+d-1 are foresight tokens f_1..f_d: f_k takes
 * the PID immediately preceding its prediction target.  If the last regular
 * token f_k can see has PID p, f_k predicts the token at p+k+1 and so gets PID
 * p+k (the paper's example: after the prefix r_1 r_2 the foresight token holding
 * PID 3 is the one whose target is r_4; in the training layout the <f> placed
 * before r_t with offset d' holds rho_{t+d'-1}).  anchor[k-1] = number of
 * candidates f_k sees (NULL: all n_c), hence p = p0 + anchor - 1. */
void ms_oracle_step_pids(int32_t p0, int32_t n_c, int32_t d,
                         const int32_t* anchor, int32_t* pid_out) {
  for (int32_t i = 0; i < n_c; ++i) pid_out[i] = p0 + i;
  for (int32_t k = 1; k <= d; ++k) {
    int32_t a = anchor ? anchor[k - 1] : n_c;
    int32_t p_last_seen = p0 + a - 1;
    pid_out[n_c + k - 1] = p_last_seen + k;
  }
}

/* ------------------------------------------------------------------------ */
/* RoPE at token-specific position IDs (Sec. 2.1.2, UPL paragraph: RoPE is    */
/* the positional mechanism; the rotation itself is Su et al.'s definition)  */
/* ------------------------------------------------------------------------ */

#define MS_ORACLE_ROPE_INTERLEAVED 1u
#define MS_ORACLE_POS_HALF_UNITS 2u

/* x: bf16 [T][H][D], rotated in place.  Frequency i (0 <= i < D/2) is
 * theta_i = base^(-2i/D) unless inv_freq supplies it.  Pairing: rotate-half
 * (i, i+D/2) by default, interleaved (2i, 2i+1) with the flag.  The rotated
 * value is rounded to bf16 once. */
int32_t ms_oracle_rope(uint16_t* x, const int32_t* pos_id, int32_t T, int32_t H,
                       int32_t D, double rope_base, const double* inv_freq,
                       uint32_t flags) {
  if (T < 0 || H < 1 || D < 2 || (D & 1)) return MS_ORACLE_BAD_ARG;
  int32_t half = D / 2;
  for (int32_t t = 0; t < T; ++t) {
    double p = (double)pos_id[t];
    if (flags & MS_ORACLE_POS_HALF_UNITS) p *= 0.5;
    for (int32_t h = 0; h < H; ++h) {
      uint16_t* v = x + ((int64_t)t * H + h) * D;
      for (int32_t i = 0; i < half; ++i) {
        double theta = inv_freq ? inv_freq[i]
                                : pow(rope_base, -2.0 * (double)i / (double)D);
        double c = cos(p * theta), s = sin(p * theta);
        int32_t ia = (flags & MS_ORACLE_ROPE_INTERLEAVED) ? 2 * i : i;
        int32_t ib = (flags & MS_ORACLE_ROPE_INTERLEAVED) ? 2 * i + 1 : i + half;
        double a = bf16_to_f64(v[ia]), b = bf16_to_f64(v[ib]);
        v[ia] = f64_to_bf16(a * c - b * s);
        v[ib] = f64_to_bf16(b * c + a * s);
      }
    }
  }
  return MS_ORACLE_OK;
}

/* ------------------------------------------------------------------------ */
/* Mask of a step block (Sec. 2.1.1; Sec. 2.3 "Attention Mask Strategy")     */
/* ------------------------------------------------------------------------ */

/* Is step-local key j visible to step-local query i?
 *  - candidates (regular tokens) are causal among themselves;
 *  - a foresight token sees preceding regular tokens (the first a_i candidates,
 *    a_i = n_c by default) and itself;
 *  - a foresight token's key is visible to nobody else (Sec. 2.3 hides its
 *    hidden state from every later token).
 * Every entry of the compacted cache is visible to every row: the verbose
 * steps were evicted, what remains is prompt, memory and output tokens and the
 * current step's accepted prefix (Fig. 2 caption; Sec. 2.3 compression rule). */
int32_t ms_oracle_visible(int32_t i, int32_t j, int32_t n_c, int32_t a_i) {
  if (j == i) return 1;
  if (j >= n_c) return 0;          /* another token's foresight key */
  if (i < n_c) return j < i;       /* candidate: causal */
  return j < a_i;                  /* foresight: the candidates it follows */
}

/* Training-time mask over an augmented sequence (Sec. 2.3 "Attention Mask Strategy"): every
 * token of the block carries a kind and the index of its reasoning step.  Key j of the block
 * is visible to query i of the block iff it is the query itself, or it comes before the query
 * and is not a foresight token (whose hidden state is masked from all later tokens) and is
 * not a verbose reasoning token of another step (for previous steps only the prompt, memory
 * and output tokens stay visible; inside the current step attention is causal). */
#define MS_KIND_PROMPT 0
#define MS_KIND_REASON 1
#define MS_KIND_FORESIGHT 2
#define MS_KIND_MEMORY 3
#define MS_KIND_OUTPUT 4
int32_t ms_oracle_visible_train(int32_t i, int32_t j, int32_t kind_j, int32_t step_i, int32_t step_j) {
  if (j == i) return 1;
  if (j > i) return 0;
  if (kind_j == MS_KIND_FORESIGHT) return 0;
  if (kind_j == MS_KIND_REASON) return step_j == step_i;
  return 1;
}

/* ------------------------------------------------------------------------ */
/* Step attention (definition of masked softmax attention, GQA)              */
/* ------------------------------------------------------------------------ */

/* One layer.  Cache K,V: bf16 [H_kv][slots][D], kv_head_stride elements
 * between heads; sequence b owns slots kv_off[b] .. kv_off[b]+kv_len[b]-1.
 * Step block of sequence b: rows q_off[b] .. q_off[b+1]-1 of q [T][H_q][D],
 * k_step/v_step [T][H_kv][D]; the first n_cand[b] rows are candidates, the
 * rest foresight tokens.  anchor[T] (or NULL): for a foresight row the number
 * of candidates it sees; ignored for candidate rows.
 * Query head h reads KV head h / (H_q/H_kv).
 * out fp64 [T][H_q][D], lse fp64 [T][H_q] (natural log), either may be NULL. */
static int32_t local_visible(int32_t i, int32_t j, int32_t n_c, int32_t a_i, int32_t r0,
                             const uint8_t* tok_kind, const int32_t* tok_step) {
  if (tok_kind) return ms_oracle_visible_train(i, j, tok_kind[r0 + j], tok_step[r0 + i], tok_step[r0 + j]);
  return ms_oracle_visible(i, j, n_c, a_i);
}

/* tok_kind / tok_step [T] (both or neither): when given, the block's own keys follow the
 * training-time rule above instead of the (n_cand, anchor) rule. */
int32_t ms_oracle_attn_block(int32_t B, int32_t H_q, int32_t H_kv, int32_t D,
                             const uint16_t* k_cache, const uint16_t* v_cache,
                             int64_t kv_head_stride, const int64_t* kv_off,
                             const int32_t* kv_len, const int32_t* q_off,
                             const int32_t* n_cand, const int32_t* anchor,
                             const uint8_t* tok_kind, const int32_t* tok_step,
                             const uint16_t* q, const uint16_t* k_step,
                             const uint16_t* v_step, double sm_scale,
                             double* out, double* lse) {
  if (B < 0 || H_kv < 1 || H_q < 1 || H_q % H_kv || D < 1) return MS_ORACLE_BAD_ARG;
  const int32_t G = H_q / H_kv;
  int32_t bad = 0;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
  for (int32_t b = 0; b < B; ++b) {
    for (int32_t h = 0; h < H_q; ++h) {
      const int32_t kvh = h / G;
      const int32_t L = kv_len[b];
      const int32_t r0 = q_off[b], n_q = q_off[b + 1] - q_off[b];
      const int32_t n_c = n_cand[b];
      const uint16_t* Kc = k_cache + kvh * kv_head_stride + kv_off[b] * (int64_t)D;
      const uint16_t* Vc = v_cache + kvh * kv_head_stride + kv_off[b] * (int64_t)D;
      double* s = (double*)malloc(sizeof(double) * (size_t)(L + n_q + 1));
      if (!s) { bad = 1; continue; }
      for (int32_t i = 0; i < n_q; ++i) {
        const uint16_t* qv = q + ((int64_t)(r0 + i) * H_q + h) * D;
        const int32_t a_i = (i < n_c) ? i : (anchor ? anchor[r0 + i] : n_c);
        /* scores over the visible set: all L cache keys, then step-local keys */
        double m = -INFINITY;
        for (int32_t j = 0; j < L + n_q; ++j) {
          const uint16_t* kv;
          if (j < L) {
            kv = Kc + (int64_t)j * D;
          } else {
            if (!local_visible(i, j - L, n_c, a_i, r0, tok_kind, tok_step)) { s[j] = -INFINITY; continue; }
            kv = k_step + ((int64_t)(r0 + j - L) * H_kv + kvh) * D;
          }
          double dot = 0.0;
          for (int32_t e = 0; e < D; ++e) dot += bf16_to_f64(qv[e]) * bf16_to_f64(kv[e]);
          s[j] = sm_scale * dot;
          if (s[j] > m) m = s[j];
        }
        /* softmax weights; a hidden key keeps weight exactly 0 */
        double denom = 0.0;
        for (int32_t j = 0; j < L + n_q; ++j) {
          int32_t hidden = (j >= L) && !local_visible(i, j - L, n_c, a_i, r0, tok_kind, tok_step);
          s[j] = hidden ? 0.0 : exp(s[j] - m);
          denom += s[j];
        }
        if (out) {
          double* o = out + ((int64_t)(r0 + i) * H_q + h) * D;
          for (int32_t e = 0; e < D; ++e) o[e] = 0.0;
          for (int32_t j = 0; j < L + n_q; ++j) {
            if ((j >= L) && !local_visible(i, j - L, n_c, a_i, r0, tok_kind, tok_step)) continue;
            const uint16_t* vv = (j < L) ? Vc + (int64_t)j * D
                                         : v_step + ((int64_t)(r0 + j - L) * H_kv + kvh) * D;
            for (int32_t e = 0; e < D; ++e) o[e] += s[j] * bf16_to_f64(vv[e]);
          }
          for (int32_t e = 0; e < D; ++e) o[e] /= denom;
        }
        if (lse) lse[(int64_t)(r0 + i) * H_q + h] = m + log(denom);
      }
      free(s);
    }
  }
  return bad ? MS_ORACLE_BAD_ARG : MS_ORACLE_OK;
}

/* The step block of inference: the (n_cand, anchor) rule for the block's own keys. */
int32_t ms_oracle_attn_step(int32_t B, int32_t H_q, int32_t H_kv, int32_t D,
                            const uint16_t* k_cache, const uint16_t* v_cache,
                            int64_t kv_head_stride, const int64_t* kv_off,
                            const int32_t* kv_len, const int32_t* q_off,
                            const int32_t* n_cand, const int32_t* anchor,
                            const uint16_t* q, const uint16_t* k_step,
                            const uint16_t* v_step, double sm_scale,
                            double* out, double* lse) {
  return ms_oracle_attn_block(B, H_q, H_kv, D, k_cache, v_cache, kv_head_stride, kv_off, kv_len, q_off,
                              n_cand, anchor, NULL, NULL, q, k_step, v_step, sm_scale, out, lse);
}

/* ------------------------------------------------------------------------ */
/* KV compaction (Sec. 2.1.2: once a step is compressed its regular tokens    */
/* leave the KV cache; Algorithm 1, UpdateCache)                             */
/* ------------------------------------------------------------------------ */

/* Cache K,V: bf16 [n_layers][H_kv][slots][D].  For each sequence b with
 * seg_len[b] > 0, the entries seg_start[b] .. seg_start[b]+seg_len[b]-1 (the
 * verbose step) are dropped; everything behind them (the memory tokens and <o>
 * appended after the step, and anything later) moves up, order preserved:
 *     new = old[0 : s) ++ old[s+n : L)
 * src_idx[b][j] (optional, row pitch idx_stride) is the old index of new entry
 * j; kv_len[b] becomes L - n.  Payload bits are copied unchanged, in every
 * layer, for K and V. */
int32_t ms_oracle_kv_compact(uint16_t* k_cache, uint16_t* v_cache, int32_t n_layers,
                             int64_t layer_stride, int64_t kv_head_stride, int32_t B,
                             int32_t H_kv, int32_t D, const int64_t* kv_off,
                             int32_t* kv_len, const int32_t* seg_start,
                             const int32_t* seg_len, int32_t* src_idx,
                             int32_t idx_stride) {
  for (int32_t b = 0; b < B; ++b) {
    const int32_t L = kv_len[b], s = seg_start[b], n = seg_len[b];
    if (n < 0 || s < 0 || (int64_t)s + n > L) return MS_ORACLE_BAD_ARG;
    const int32_t newL = L - n;
    int32_t* keep = (int32_t*)malloc(sizeof(int32_t) * (size_t)(newL + 1));
    int32_t cnt = 0;
    for (int32_t j = 0; j < L; ++j)
      if (j < s || j >= s + n) keep[cnt++] = j;
    uint16_t* tmp = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)(newL + 1) * D);
    for (int32_t layer = 0; layer < n_layers; ++layer)
      for (int32_t kv = 0; kv < 2; ++kv)
        for (int32_t h = 0; h < H_kv; ++h) {
          uint16_t* base = (kv ? v_cache : k_cache) + layer * layer_stride +
                           h * kv_head_stride + kv_off[b] * (int64_t)D;
          for (int32_t j = 0; j < newL; ++j)
            memcpy(tmp + (int64_t)j * D, base + (int64_t)keep[j] * D, sizeof(uint16_t) * D);
          memcpy(base, tmp, sizeof(uint16_t) * (size_t)newL * D);
        }
    if (src_idx)
      for (int32_t j = 0; j < newL; ++j) src_idx[(int64_t)b * idx_stride + j] = keep[j];
    kv_len[b] = newL;
    free(tmp);
    free(keep);
  }
  return MS_ORACLE_OK;
}

/* Eviction by an arbitrary keep list (the comparison systems of Sec. 4 -- heavy-hitter and
 * separator-based eviction -- keep a different subset of the cache than MemoSight does, but
 * the cache operation is the same): new = [old[keep[0]], old[keep[1]], ...], kv_len = n_keep.
 * keep[b] must be strictly increasing and inside [0, L).  All layers, K and V, bits unchanged. */
int32_t ms_oracle_kv_gather(uint16_t* k_cache, uint16_t* v_cache, int32_t n_layers,
                            int64_t layer_stride, int64_t kv_head_stride, int32_t B,
                            int32_t H_kv, int32_t D, const int64_t* kv_off, int32_t* kv_len,
                            const int32_t* keep_idx, int32_t idx_stride, const int32_t* n_keep) {
  for (int32_t b = 0; b < B; ++b) {
    const int32_t L = kv_len[b], nk = n_keep[b];
    const int32_t* keep = keep_idx + (int64_t)b * idx_stride;
    if (nk < 0 || nk > L || nk > idx_stride) return MS_ORACLE_BAD_ARG;
    for (int32_t j = 0; j < nk; ++j)
      if (keep[j] < 0 || keep[j] >= L || (j > 0 && keep[j] <= keep[j - 1])) return MS_ORACLE_BAD_ARG;
    uint16_t* tmp = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)(nk + 1) * D);
    for (int32_t layer = 0; layer < n_layers; ++layer)
      for (int32_t kv = 0; kv < 2; ++kv)
        for (int32_t h = 0; h < H_kv; ++h) {
          uint16_t* base = (kv ? v_cache : k_cache) + layer * layer_stride +
                           h * kv_head_stride + kv_off[b] * (int64_t)D;
          for (int32_t j = 0; j < nk; ++j)
            memcpy(tmp + (int64_t)j * D, base + (int64_t)keep[j] * D, sizeof(uint16_t) * D);
          memcpy(base, tmp, sizeof(uint16_t) * (size_t)nk * D);
        }
    kv_len[b] = nk;
    free(tmp);
  }
  return MS_ORACLE_OK;
}

/* Append accepted tokens (Algorithm 1: S <- S (+) A).  One layer's cache
 * [H_kv][slots][D]: the first n_keep[b] candidate rows of the step buffers go
 * to slots kv_len[b] ..; foresight rows are never cached (Sec. 2.3: no later
 * token may attend to a foresight token).  kv_len is bumped iff bump. */
int32_t ms_oracle_kv_append(uint16_t* k_cache, uint16_t* v_cache, int64_t kv_head_stride,
                            int32_t B, int32_t H_kv, int32_t D, const int64_t* kv_off,
                            int32_t* kv_len, const uint16_t* k_step,
                            const uint16_t* v_step, const int32_t* q_off,
                            const int32_t* n_cand, const int32_t* n_keep, int32_t bump) {
  for (int32_t b = 0; b < B; ++b) {
    if (n_keep[b] < 0 || n_keep[b] > n_cand[b]) return MS_ORACLE_BAD_ARG;
    for (int32_t i = 0; i < n_keep[b]; ++i)
      for (int32_t h = 0; h < H_kv; ++h) {
        int64_t dst = h * kv_head_stride + (kv_off[b] + kv_len[b] + i) * (int64_t)D;
        int64_t src = ((int64_t)(q_off[b] + i) * H_kv + h) * D;
        memcpy(k_cache + dst, k_step + src, sizeof(uint16_t) * D);
        memcpy(v_cache + dst, v_step + src, sizeof(uint16_t) * D);
      }
  }
  if (bump)
    for (int32_t b = 0; b < B; ++b) kv_len[b] += n_keep[b];
  return MS_ORACLE_OK;
}

/* ------------------------------------------------------------------------ */
/* Greedy accept (Sec. 2.1.1 and its footnote: the accepted tokens are the    */
/* longest draft prefix that equals the model's own argmax row by row)       */
/* ------------------------------------------------------------------------ */

/* logits fp32 [T][ld_v], V used columns.  argmax = lowest index of the row
 * maximum; a NaN counts as larger than everything and the first NaN wins (the
 * numpy.argmax convention).  Rows row_off[b] .. row_off[b+1]-1 belong to
 * sequence b; draft[r] is the token that row r's prediction must equal for the
 * draft to be accepted, or -1 where nothing is to be verified.  n_match[b] =
 * the largest m such that rows 0..m-1 of the block all have draft >= 0 and
 * argmax == draft. */
int32_t ms_oracle_accept(const float* logits, int64_t ld_v, int32_t V,
                         const int32_t* row_off, int32_t B, const int32_t* draft,
                         int32_t* argmax_out, int32_t* n_match) {
  if (V < 1 || ld_v < V) return MS_ORACLE_BAD_ARG;
  const int32_t T = row_off[B];
#pragma omp parallel for schedule(static)
  for (int32_t r = 0; r < T; ++r) {
    const float* row = logits + (int64_t)r * ld_v;
    int32_t best = 0;
    for (int32_t v = 1; v < V; ++v) {
      if (isnan(row[best])) break;
      if (isnan(row[v]) || row[v] > row[best]) best = v;
    }
    argmax_out[r] = best;
  }
  for (int32_t b = 0; b < B; ++b) {
    int32_t m = 0;
    for (int32_t r = row_off[b]; r < row_off[b + 1]; ++r) {
      if (draft[r] < 0 || argmax_out[r] != draft[r]) break;
      ++m;
    }
    n_match[b] = m;
  }
  return MS_ORACLE_OK;
}

/* Number of OpenMP threads the parallel loops above will use. */
#ifdef _OPENMP
#include <omp.h>
int32_t ms_oracle_threads(void) { return omp_get_max_threads(); }
#else
int32_t ms_oracle_threads(void) { return 1; }
#endif
