/*
 * CPU oracle for ReLU-kernel linear attention -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 statement of what the paper's linear-attention path
 * computes, written from the equations.  It exists so that the CUDA kernels
 * can be checked element by element; it shares no code, header, table or
 * helper with them and must never be called from the product path.  Only the
 * tests, the smoke check and the benchmark's cpu_baseline / reference legs
 * may load this library.
 *
 * What is computed, per (batch b, head h), with phi = ReLU and head dim d:
 *
 *   Bidirectional form (Eq. 2 with the rotary factors dropped, as the text
 *   after Eq. 3 does):
 *       S[i][j] = sum_n phi(k_n)[i] * v_n[j]        (d x d)
 *       z[i]    = sum_n phi(k_n)[i]                 (d)
 *       o_n[j]  = sum_i phi(q_n)[i] S[i][j] / (sum_i phi(q_n)[i] z[i] + eps)
 *
 *   Quadratic ("brute") form of the same thing, the plain definition:
 *       w[n][m] = sum_i phi(q_n)[i] phi(k_m)[i]
 *       o_n[j]  = sum_m w[n][m] v_m[j] / (sum_m w[n][m] + eps)
 *   with an optional block mask: token m is visible to token n iff
 *   floor(m / T_b) <= floor(n / T_b)  (full attention inside a block of
 *   frames, causal across blocks -- the mask Sec. 3.2 describes).
 *
 *   Cached block-by-block generation (Eq. 3, Algorithm 1's cache update):
 *   the cache is the running pair (sum S, sum phi(K)^T); a step adds the
 *   block's own (S_blk, z_blk) and then applies the block's queries to it.
 *
 *   Eq. 2 with its rotary factors (right-hand form): RoPE after the ReLU in the
 *   numerator only, plain denominator; linear and quadratic forms (see the
 *   functions oracle_rope_*).  The paper fixes neither how features are paired
 *   nor the angles: pairs are adjacent features and the rotations are inputs.
 *
 * Readings taken where the paper is silent:
 *   - eps is added once to the denominator after the dot product;
 *   - a query whose phi(q).z is zero yields 0/(0+eps) = 0, never NaN;
 *   - "D" in the O(D^2) cache size is the per-head dimension d;
 *   - a block attends to itself (commit, then apply).
 *
 * Pins (tests/test_oracle_pins.py): closed forms (constant V, N = 1, one-hot
 * features = segment mean), an exact rational worked example, brute-force
 * equality of the linear, quadratic, masked and stepped forms, invariances
 * (positive scaling, permutation, sign of negative entries), convexity; for
 * the rotary forms the closed form sum_m cos(theta_n - theta_m) v_m / (count
 * + eps) at d = 2, over all tokens and over the tokens a block may see, for
 * the one-shot, the masked brute-force and the cached-step functions alike;
 * and a mutation test showing that planted mistakes fail those pins.  No
 * function here is unpinned.
 *
 * Tensor layout: element (b, n, h, e) of Q/K/V/O lives at
 *   b*stride_b + n*stride_n + h*stride_h + e   (strides in elements).
 * Input element types: 0 = bfloat16 bit patterns (uint16), 1 = float32,
 * 2 = float64.  All arithmetic and all outputs are fp64.
 * State layout: S[b][h][i][j] (i = key feature, j = value feature), z[b][h][i].
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
  int64_t B, N, H, d;
  int64_t stride_b, stride_n, stride_h; /* elements */
  int32_t dtype;                        /* 0 bf16 bits, 1 f32, 2 f64 */
} oracle_shape;

static inline double load_elem(const void* base, int32_t dtype, int64_t idx) {
  if (dtype == 0) {
    /* bfloat16 is the top 16 bits of an IEEE float32 */
    uint32_t u = (uint32_t)((const uint16_t*)base)[idx] << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
  }
  if (dtype == 1) return (double)((const float*)base)[idx];
  return ((const double*)base)[idx];
}

static inline double relu(double x) { return x > 0.0 ? x : 0.0; }

static inline int64_t at(const oracle_shape* s, int64_t b, int64_t n, int64_t h) {
  return b * s->stride_b + n * s->stride_n + h * s->stride_h;
}

/* S += sum_n phi(k_n)^T v_n ; z += sum_n phi(k_n), tokens n in [n0, n1).  Eq. 2 / Eq. 3 state. */
static void accumulate_state(const oracle_shape* s, const void* k, const void* v, int64_t b, int64_t h,
                             int64_t n0, int64_t n1, double* S, double* z) {
  const int64_t d = s->d;
  for (int64_t n = n0; n < n1; ++n) {
    const int64_t base = at(s, b, n, h);
    for (int64_t i = 0; i < d; ++i) {
      const double kp = relu(load_elem(k, s->dtype, base + i));
      if (kp == 0.0) continue; /* adds exactly zero */
      z[i] += kp;
      double* Srow = S + i * d;
      for (int64_t j = 0; j < d; ++j) Srow[j] += kp * load_elem(v, s->dtype, base + j);
    }
  }
}

/* o_n = phi(q_n) S / (phi(q_n).z + eps) for one token.  Eq. 2. */
static void apply_token(const oracle_shape* s, const void* q, int64_t b, int64_t n, int64_t h, const double* S,
                        const double* z, double eps, double* o_row) {
  const int64_t d = s->d;
  const int64_t base = at(s, b, n, h);
  double den = 0.0;
  for (int64_t j = 0; j < d; ++j) o_row[j] = 0.0;
  for (int64_t i = 0; i < d; ++i) {
    const double qp = relu(load_elem(q, s->dtype, base + i));
    den += qp * z[i];
    const double* Srow = S + i * d;
    for (int64_t j = 0; j < d; ++j) o_row[j] += qp * Srow[j];
  }
  den += eps;
  for (int64_t j = 0; j < d; ++j) o_row[j] /= den;
}

/* State of the whole sequence.  S: [B,H,d,d], z: [B,H,d], both overwritten. */
void oracle_state(const oracle_shape* s, const void* k, const void* v, double* S, double* z) {
  const int64_t d = s->d, BH = s->B * s->H;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t u = 0; u < BH; ++u) {
    const int64_t b = u / s->H, h = u % s->H;
    double* Su = S + u * d * d;
    double* zu = z + u * d;
    memset(Su, 0, sizeof(double) * d * d);
    memset(zu, 0, sizeof(double) * d);
    accumulate_state(s, k, v, b, h, 0, s->N, Su, zu);
  }
}

/* Apply given state to the query rows rows[0..n_rows) (token indices) of every (b,h).
 * o: [B, n_rows, H, d] dense fp64. */
void oracle_apply_rows(const oracle_shape* s, const void* q, const double* S, const double* z, double eps,
                       const int64_t* rows, int64_t n_rows, double* o) {
  const int64_t d = s->d, BH = s->B * s->H;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t u = 0; u < BH; ++u) {
    const int64_t b = u / s->H, h = u % s->H;
    for (int64_t r = 0; r < n_rows; ++r)
      apply_token(s, q, b, rows[r], h, S + u * d * d, z + u * d, eps, o + ((b * n_rows + r) * s->H + h) * d);
  }
}

/* Bidirectional linear attention, linear form.  o: [B,N,H,d] dense fp64. */
void oracle_linattn_forward(const oracle_shape* s, const void* q, const void* k, const void* v, double eps,
                            double* o) {
  const int64_t d = s->d, BH = s->B * s->H;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t u = 0; u < BH; ++u) {
    const int64_t b = u / s->H, h = u % s->H;
    double* S = (double*)calloc((size_t)(d * d + d), sizeof(double));
    double* z = S + d * d;
    accumulate_state(s, k, v, b, h, 0, s->N, S, z);
    for (int64_t n = 0; n < s->N; ++n) apply_token(s, q, b, n, h, S, z, eps, o + ((b * s->N + n) * s->H + h) * d);
    free(S);
  }
}

/* Quadratic form, with optional block mask (T_b <= 0: no mask).  O(N^2 d): tiny inputs only. */
void oracle_quadratic(const oracle_shape* s, const void* q, const void* k, const void* v, double eps, int64_t T_b,
                      double* o) {
  const int64_t d = s->d, BH = s->B * s->H;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t u = 0; u < BH; ++u) {
    const int64_t b = u / s->H, h = u % s->H;
    for (int64_t n = 0; n < s->N; ++n) {
      double* o_row = o + ((b * s->N + n) * s->H + h) * d;
      const int64_t qb = at(s, b, n, h);
      double wsum = 0.0;
      for (int64_t j = 0; j < d; ++j) o_row[j] = 0.0;
      for (int64_t m = 0; m < s->N; ++m) {
        if (T_b > 0 && (m / T_b) > (n / T_b)) continue; /* later block: not visible */
        const int64_t kb = at(s, b, m, h);
        double w = 0.0;
        for (int64_t i = 0; i < d; ++i)
          w += relu(load_elem(q, s->dtype, qb + i)) * relu(load_elem(k, s->dtype, kb + i));
        wsum += w;
        for (int64_t j = 0; j < d; ++j) o_row[j] += w * load_elem(v, s->dtype, kb + j);
      }
      wsum += eps;
      for (int64_t j = 0; j < d; ++j) o_row[j] /= wsum;
    }
  }
}

/* One cached step (Eq. 3; Algorithm 1's "update cache" followed by the read):
 * cache (S,z) += state of this block; o_blk = apply(q_blk, cache).
 * s->N is the number of tokens in the block.  S: [B,H,d,d], z: [B,H,d] updated in place.
 * o may be NULL (absorb the block only). */
void oracle_block_step(const oracle_shape* s, const void* q, const void* k, const void* v, double eps, double* S,
                       double* z, double* o) {
  const int64_t d = s->d, BH = s->B * s->H;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t u = 0; u < BH; ++u) {
    const int64_t b = u / s->H, h = u % s->H;
    accumulate_state(s, k, v, b, h, 0, s->N, S + u * d * d, z + u * d);
    if (o)
      for (int64_t n = 0; n < s->N; ++n)
        apply_token(s, q, b, n, h, S + u * d * d, z + u * d, eps, o + ((b * s->N + n) * s->H + h) * d);
  }
}

/* One-shot block-causal attention in prefix form: for each block, the state of all tokens of
 * blocks <= it, applied to the block's queries.  Equals oracle_quadratic with the mask. */
void oracle_block_masked(const oracle_shape* s, const void* q, const void* k, const void* v, double eps, int64_t T_b,
                         double* o) {
  const int64_t d = s->d, BH = s->B * s->H;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t u = 0; u < BH; ++u) {
    const int64_t b = u / s->H, h = u % s->H;
    double* S = (double*)calloc((size_t)(d * d + d), sizeof(double));
    double* z = S + d * d;
    for (int64_t n0 = 0; n0 < s->N; n0 += T_b) {
      const int64_t n1 = n0 + T_b < s->N ? n0 + T_b : s->N;
      accumulate_state(s, k, v, b, h, n0, n1, S, z);
      for (int64_t n = n0; n < n1; ++n) apply_token(s, q, b, n, h, S, z, eps, o + ((b * s->N + n) * s->H + h) * d);
    }
    free(S);
  }
}

/* ---- Eq. 2 with the rotary factors (its right-hand form) ----
 *
 *   o_n = RoPE_n(phi(q_n)) ( sum_m RoPE_m(phi(k_m))^T v_m ) / ( phi(q_n) . sum_m phi(k_m) + eps )
 *
 * The rotation is applied AFTER the ReLU and only in the numerator; the denominator uses the plain
 * features, so it stays non-negative (Sec. 3.1).  RoPE_n rotates the feature pair (2p, 2p+1) of token n by
 * an angle given through its cosine and sine: (a, b) -> (a c - b s, a s + b c), c = cs[n][p], s = sn[n][p]
 * (tables [N][d/2], shared by all batch entries and heads).  How the angles depend on the token's
 * (t, h, w) position is the caller's business: the paper does not give its 3D split or base frequency. */
static void rope_features(const oracle_shape* s, const void* x, int64_t base, const double* cs, const double* sn,
                          int64_t n, double* plain, double* rot) {
  const int64_t d = s->d, half = d / 2;
  for (int64_t i = 0; i < d; ++i) plain[i] = relu(load_elem(x, s->dtype, base + i));
  for (int64_t p = 0; p < half; ++p) {
    const double c = cs[n * half + p], t = sn[n * half + p];
    rot[2 * p] = plain[2 * p] * c - plain[2 * p + 1] * t;
    rot[2 * p + 1] = plain[2 * p] * t + plain[2 * p + 1] * c;
  }
  if (d & 1) rot[d - 1] = plain[d - 1]; /* an unpaired last feature is not rotated */
}

/* Linear form: S from the rotated keys, z from the plain keys; numerator from the rotated query, denominator
 * from the plain query.  o: [B,N,H,d] dense fp64. */
void oracle_rope_forward(const oracle_shape* s, const void* q, const void* k, const void* v, const double* cs,
                         const double* sn, double eps, double* o) {
  const int64_t d = s->d, BH = s->B * s->H;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t u = 0; u < BH; ++u) {
    const int64_t b = u / s->H, h = u % s->H;
    double* S = (double*)calloc((size_t)(d * d + 3 * d), sizeof(double));
    double* z = S + d * d;
    double* plain = z + d;
    double* rot = plain + d;
    for (int64_t n = 0; n < s->N; ++n) {
      const int64_t base = at(s, b, n, h);
      rope_features(s, k, base, cs, sn, n, plain, rot);
      for (int64_t i = 0; i < d; ++i) {
        z[i] += plain[i];
        for (int64_t j = 0; j < d; ++j) S[i * d + j] += rot[i] * load_elem(v, s->dtype, base + j);
      }
    }
    for (int64_t n = 0; n < s->N; ++n) {
      double* o_row = o + ((b * s->N + n) * s->H + h) * d;
      rope_features(s, q, at(s, b, n, h), cs, sn, n, plain, rot);
      double den = 0.0;
      for (int64_t j = 0; j < d; ++j) o_row[j] = 0.0;
      for (int64_t i = 0; i < d; ++i) {
        den += plain[i] * z[i];
        for (int64_t j = 0; j < d; ++j) o_row[j] += rot[i] * S[i * d + j];
      }
      den += eps;
      for (int64_t j = 0; j < d; ++j) o_row[j] /= den;
    }
    free(S);
  }
}

/* Quadratic form of the same: w_num[n][m] = RoPE_n(phi(q_n)) . RoPE_m(phi(k_m)), w_den[n][m] = phi(q_n) . phi(k_m),
 * o_n = sum_m w_num[n][m] v_m / (sum_m w_den[n][m] + eps), over the tokens m that n may see (all of them, or
 * with T_b > 0 those of its own and earlier blocks).  O(N^2 d): tiny inputs only. */
void oracle_rope_quadratic(const oracle_shape* s, const void* q, const void* k, const void* v, const double* cs,
                           const double* sn, double eps, int64_t T_b, double* o) {
  const int64_t d = s->d, BH = s->B * s->H;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t u = 0; u < BH; ++u) {
    const int64_t b = u / s->H, h = u % s->H;
    double* buf = (double*)calloc((size_t)(4 * d), sizeof(double));
    double *qp = buf, *qr = buf + d, *kp = buf + 2 * d, *kr = buf + 3 * d;
    for (int64_t n = 0; n < s->N; ++n) {
      double* o_row = o + ((b * s->N + n) * s->H + h) * d;
      rope_features(s, q, at(s, b, n, h), cs, sn, n, qp, qr);
      double wden = 0.0;
      for (int64_t j = 0; j < d; ++j) o_row[j] = 0.0;
      for (int64_t m = 0; m < s->N; ++m) {
        if (T_b > 0 && (m / T_b) > (n / T_b)) continue; /* later block: not visible (T_b <= 0: no mask) */
        const int64_t kb = at(s, b, m, h);
        rope_features(s, k, kb, cs, sn, m, kp, kr);
        double wn = 0.0;
        for (int64_t i = 0; i < d; ++i) { wn += qr[i] * kr[i]; wden += qp[i] * kp[i]; }
        for (int64_t j = 0; j < d; ++j) o_row[j] += wn * load_elem(v, s->dtype, kb + j);
      }
      wden += eps;
      for (int64_t j = 0; j < d; ++j) o_row[j] /= wden;
    }
    free(buf);
  }
}

/* One block of the block-causal form with rotary factors (Eq. 3's running sums applied to Eq. 2's right-hand
 * form): the cache (S, z) of one (b, h) holds (sum of RoPE(phi(k))^T v, sum of phi(k)); the block's tokens
 * [n0, n1) are added to it, then the block's queries are applied to it (rotated for the numerator, plain for
 * the denominator).  Token n of the tensors uses row n of the tables.  o may be NULL (commit only). */
static void rope_block(const oracle_shape* s, const void* q, const void* k, const void* v, const double* cs,
                       const double* sn, int64_t b, int64_t h, int64_t n0, int64_t n1, double eps, double* S,
                       double* z, double* plain, double* rot, double* o) {
  const int64_t d = s->d;
  for (int64_t n = n0; n < n1; ++n) { /* commit the block ... */
    const int64_t base = at(s, b, n, h);
    rope_features(s, k, base, cs, sn, n, plain, rot);
    for (int64_t i = 0; i < d; ++i) {
      z[i] += plain[i];
      for (int64_t j = 0; j < d; ++j) S[i * d + j] += rot[i] * load_elem(v, s->dtype, base + j);
    }
  }
  if (!o) return;
  for (int64_t n = n0; n < n1; ++n) { /* ... then read it */
    double* o_row = o + ((b * s->N + n) * s->H + h) * d;
    rope_features(s, q, at(s, b, n, h), cs, sn, n, plain, rot);
    double den = 0.0;
    for (int64_t j = 0; j < d; ++j) o_row[j] = 0.0;
    for (int64_t i = 0; i < d; ++i) {
      den += plain[i] * z[i];
      for (int64_t j = 0; j < d; ++j) o_row[j] += rot[i] * S[i * d + j];
    }
    den += eps;
    for (int64_t j = 0; j < d; ++j) o_row[j] /= den;
  }
}

/* Block-causal form with rotary factors over a whole sequence, block by block from an empty cache.
 * o: [B,N,H,d] dense fp64. */
void oracle_rope_block_masked(const oracle_shape* s, const void* q, const void* k, const void* v, const double* cs,
                              const double* sn, double eps, int64_t T_b, double* o) {
  const int64_t d = s->d, BH = s->B * s->H;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t u = 0; u < BH; ++u) {
    const int64_t b = u / s->H, h = u % s->H;
    double* S = (double*)calloc((size_t)(d * d + 3 * d), sizeof(double));
    double* z = S + d * d;
    for (int64_t n0 = 0; n0 < s->N; n0 += T_b) {
      const int64_t n1 = n0 + T_b < s->N ? n0 + T_b : s->N;
      rope_block(s, q, k, v, cs, sn, b, h, n0, n1, eps, S, z, z + d, z + 2 * d, o);
    }
    free(S);
  }
}

/* One cached step with rotary factors on a caller-held cache: S [B,H,d,d], z [B,H,d] are updated in place
 * (Algorithm 1's cache update), o [B,N,H,d] gets the block's outputs (NULL: commit only).  The tensors hold
 * the block alone (N = its tokens) and cs, sn are the table rows of those tokens.  A read-only denoising step
 * is this function run on a copy of the cache. */
void oracle_rope_block_step(const oracle_shape* s, const void* q, const void* k, const void* v, const double* cs,
                            const double* sn, double eps, double* S, double* z, double* o) {
  const int64_t d = s->d, BH = s->B * s->H;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t u = 0; u < BH; ++u) {
    double* tmp = (double*)calloc((size_t)(2 * d), sizeof(double));
    rope_block(s, q, k, v, cs, sn, u / s->H, u % s->H, 0, s->N, eps, S + u * d * d, z + u * d, tmp, tmp + d, o);
    free(tmp);
  }
}

/* Bytes of the fp64 cache this oracle keeps for a stream: depends on (B,H,d) only (Table 1). */
int64_t oracle_cache_bytes(int64_t B, int64_t H, int64_t d) { return B * H * (d * d + d) * (int64_t)sizeof(double); }
