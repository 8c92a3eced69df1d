/*
 * CPU oracle for the SparSP single-device hot path (TEST INFRASTRUCTURE ONLY).
 *
 * This file is the slow, plain definition that the CUDA kernels are checked against.  It shares no
 * code, table or helper with the CUDA path and must never be linked into it.  Only the test-suite,
 * the smoke check and the benchmark's CPU-baseline legs may call it.
 *
 * What each function follows:
 *   oracle_pool           mean-pooled query / key tiles ("masks materialised from pooled query and
 *                         key tiles", Section 4.2, Sparse KV Selection); fp32, ascending-token sum.
 *   oracle_scores         pooled-Q x pooled-K^T per head; fp32 fused-multiply-add chain.
 *   oracle_scores_f64     the same contraction in fp64 (near-tie audit only).
 *   oracle_topk_mask      block mask M[h,i,j] (Section 4.1, Design Overview), selection = top-k per query block
 *                         with lowest-index tie-break; text blocks always kept.
 *   oracle_demand         receiver demand D[r,h,p] (Section 4.1, Eq. "receiver-demand"), exchange volume V_r
 *                         (Eq. "sparse-exchange-volume"), head-preserving Boolean demand
 *                         (Section 5.2), locally derived per-head offsets (Section 5.2).
 *   oracle_pack           row-major (head, block) packing, one contiguous segment per
 *                         (consumer, producer) pair (Sections 5.2 and 6).
 *   oracle_attn_rows      softmax(QK^T/sqrt(d))V (Eq. "attention") restricted to kept blocks,
 *                         fp64 accumulation.
 *   oracle_attn_dense_masked   the same, written as a full N-wide row with -inf on masked keys.
 *
 * Pool and score are computed in fp32 in one fixed order because their result decides an integer
 * (which blocks are kept): the CUDA kernels take the decision in the same precision and order.
 * Everything downstream of the mask is either integer/byte work (exact) or fp64 (attention).
 *
 * Layouts are dense and canonical: X[h][n][c] bf16 stored as uint16_t; mask[h][i][w] uint32 words
 * with KV block j at bit (j & 31) of word (j >> 5).
 *
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -fopenmp -shared -fPIC (see oracle/build.py).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static inline float bf16_to_f32(uint16_t v) {
  uint32_t u = ((uint32_t)v) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return f;
}

static inline int64_t ceil_div64(int64_t a, int64_t b) { return (a + b - 1) / b; }

/* ------------------------------------------------------------------------------------------------
 * Step 1a.  pooled[h][i][c] = (sum over the valid tokens of block i, ascending, fp32) / n_i.
 * n_i = min(b, N - i*b).  One IEEE fp32 division per output.
 * ---------------------------------------------------------------------------------------------- */
void oracle_pool(const uint16_t* x, int64_t H, int64_t N, int64_t d, int64_t b, float* pooled) {
  const int64_t NB = ceil_div64(N, b);
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t h = 0; h < H; ++h) {
    for (int64_t i = 0; i < NB; ++i) {
      const int64_t t0 = i * b;
      const int64_t n_i = (N - t0 < b) ? (N - t0) : b;
      for (int64_t c = 0; c < d; ++c) {
        float sum = 0.0f;
        for (int64_t t = 0; t < n_i; ++t) {
          sum = sum + bf16_to_f32(x[(h * N + t0 + t) * d + c]);
        }
        pooled[(h * NB + i) * d + c] = sum / (float)n_i;
      }
    }
  }
}

/* ------------------------------------------------------------------------------------------------
 * Step 1b.  S[h][i][j] = sum_c pQ[h][i][c] * pK[h][j][c], as acc = fmaf(q_c, k_c, acc) from
 * acc = 0 with c ascending.  No 1/sqrt(d) and no softmax: both are monotone per row.
 * ---------------------------------------------------------------------------------------------- */
void oracle_scores(const float* pq, const float* pk, int64_t H, int64_t NB, int64_t d,
                   float* scores) {
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t h = 0; h < H; ++h) {
    for (int64_t i = 0; i < NB; ++i) {
      const float* q = pq + (h * NB + i) * d;
      for (int64_t j = 0; j < NB; ++j) {
        const float* k = pk + (h * NB + j) * d;
        float acc = 0.0f;
        for (int64_t c = 0; c < d; ++c) acc = fmaf(q[c], k[c], acc);
        scores[(h * NB + i) * NB + j] = acc;
      }
    }
  }
}

void oracle_scores_f64(const float* pq, const float* pk, int64_t H, int64_t NB, int64_t d,
                       double* scores) {
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t h = 0; h < H; ++h) {
    for (int64_t i = 0; i < NB; ++i) {
      const float* q = pq + (h * NB + i) * d;
      for (int64_t j = 0; j < NB; ++j) {
        const float* k = pk + (h * NB + j) * d;
        double acc = 0.0;
        for (int64_t c = 0; c < d; ++c) acc += (double)q[c] * (double)k[c];
        scores[(h * NB + i) * NB + j] = acc;
      }
    }
  }
}

/* ------------------------------------------------------------------------------------------------
 * Step 1c.  Per (h, i): order the candidate KV blocks (those with is_text[j] == 0) by score
 * descending, index ascending on equal scores (IEEE comparison, so -0 == +0), keep the first k;
 * then keep every text block.  Emits bit words, the ascending kept list and its length.
 * kv_list has `kept_cap` slots per row (unused slots = -1); it may be NULL, as may kv_count.
 * ---------------------------------------------------------------------------------------------- */
typedef struct {
  float s;
  int32_t j;
} cand_t;

static int cand_cmp(const void* a, const void* b) {
  const cand_t* x = (const cand_t*)a;
  const cand_t* y = (const cand_t*)b;
  if (x->s > y->s) return -1;
  if (x->s < y->s) return 1;
  return (x->j > y->j) - (x->j < y->j);
}

void oracle_topk_mask(const float* scores, const uint8_t* is_text, int64_t H, int64_t NB, int64_t k,
                      uint32_t* mask, int32_t* kv_list, int64_t kept_cap, int32_t* kv_count) {
  const int64_t Wd = ceil_div64(NB, 32);
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t h = 0; h < H; ++h) {
    for (int64_t i = 0; i < NB; ++i) {
      cand_t* cand = (cand_t*)malloc((size_t)NB * sizeof(cand_t));
      int64_t nc = 0;
      for (int64_t j = 0; j < NB; ++j) {
        if (!is_text[j]) {
          cand[nc].s = scores[(h * NB + i) * NB + j];
          cand[nc].j = (int32_t)j;
          ++nc;
        }
      }
      qsort(cand, (size_t)nc, sizeof(cand_t), cand_cmp);
      uint32_t* row = mask + (h * NB + i) * Wd;
      for (int64_t w = 0; w < Wd; ++w) row[w] = 0u;
      const int64_t keep = (k < nc) ? k : nc;
      for (int64_t t = 0; t < keep; ++t) row[cand[t].j >> 5] |= 1u << (cand[t].j & 31);
      for (int64_t j = 0; j < NB; ++j)
        if (is_text[j]) row[j >> 5] |= 1u << (j & 31);
      int64_t cnt = 0;
      for (int64_t j = 0; j < NB; ++j) {
        if ((row[j >> 5] >> (j & 31)) & 1u) {
          if (kv_list && cnt < kept_cap) kv_list[(h * NB + i) * kept_cap + cnt] = (int32_t)j;
          ++cnt;
        }
      }
      if (kv_list)
        for (int64_t t = cnt; t < kept_cap; ++t) kv_list[(h * NB + i) * kept_cap + t] = -1;
      if (kv_count) kv_count[h * NB + i] = (int32_t)cnt;
      free(cand);
    }
  }
}

/* ------------------------------------------------------------------------------------------------
 * Step 1c, CDF-threshold mode (Section 8.1: keep the key blocks with the highest scores until their
 * cumulative attention mass reaches the threshold tau).  Per (h, i), over the candidate KV blocks
 * (is_text[j] == 0):   p_j = exp(scale * (S_j - max S)),  Z = sum p_j,  keep the smallest set
 * { j : S_j >= v } (v one of the row's scores) whose mass reaches tau * Z; blocks with equal scores
 * are kept or dropped together; every text block is kept.  A floating-point sum would make the kept
 * set depend on the order of its additions, so the mass is counted in integers, where any order gives
 * the same sum:
 *   x_j  = (S_j - max S) * (scale * log2 e)        fp32: one subtraction, one multiplication
 *   p_j  = exp2c(x_j)                              fp32, below
 *   w_j  = floor(p_j * 2^26)                       an integer <= 2^26 + 8 (the scaling is exact)
 *   Z    = sum w_j,  mass(v) = sum of w_j over { j : S_j >= v }      exact integer sums
 *   kept: the largest v with  mass(v) >= ceil(tau * Z),  the product taken once in fp64 (Z < 2^37 is exact
 *   there, tau is the caller's fp32 value)
 * Dropping what lies below 2^-26 of a term changes the mass (>= 1: the largest term is 1) by less than
 * NB * 2^-26 <= 1.6e-5, the size of the rounding error of an fp32 sum of as many terms.
 * exp2c(x): x clamped below at -125; i = nearest integer (ties to even); f = x - i; degree-5 Horner
 * polynomial in f with fused multiply-adds; i added into the exponent field.
 * ---------------------------------------------------------------------------------------------- */
static float oracle_exp2c(float x) {
  if (x < -125.0f) x = -125.0f;
  const float fi = rintf(x);
  const float f = x - fi;
  float p = 0.0013400432653725147f;
  p = fmaf(p, f, 0.009676037356257439f);
  p = fmaf(p, f, 0.05550327152013779f);
  p = fmaf(p, f, 0.2402210682630539f);
  p = fmaf(p, f, 0.6931471824645996f);
  p = fmaf(p, f, 1.0000001192092896f);
  int32_t bits;
  memcpy(&bits, &p, 4);
  bits += (int32_t)fi * (1 << 23);
  memcpy(&p, &bits, 4);
  return p;
}

void oracle_exp2c_array(const float* x, int64_t n, float* y) {
  for (int64_t t = 0; t < n; ++t) y[t] = oracle_exp2c(x[t]);
}

/* sum of w[j] over the candidates j with take[j] != 0 */
static uint64_t mass_of(const uint32_t* w, const uint8_t* take, int64_t n) {
  uint64_t acc = 0;
  for (int64_t j = 0; j < n; ++j)
    if (take[j]) acc += w[j];
  return acc;
}

void oracle_cdf_mask(const float* scores, const uint8_t* is_text, int64_t H, int64_t NB, float tau,
                     float scale, uint32_t* mask, int32_t* kv_count) {
  const int64_t Wd = ceil_div64(NB, 32);
  const float c = scale * 1.4426950408889634f;
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t h = 0; h < H; ++h) {
    for (int64_t i = 0; i < NB; ++i) {
      const float* srow = scores + (h * NB + i) * NB;
      uint32_t* w = (uint32_t*)malloc((size_t)NB * sizeof(uint32_t));
      uint8_t* take = (uint8_t*)malloc((size_t)NB);
      cand_t* cand = (cand_t*)malloc((size_t)NB * sizeof(cand_t));
      int64_t nc = 0;
      float mx = -INFINITY;
      for (int64_t j = 0; j < NB; ++j)
        if (!is_text[j] && srow[j] > mx) mx = srow[j];
      for (int64_t j = 0; j < NB; ++j) {
        w[j] = 0u;
        take[j] = 0;
        if (!is_text[j]) {
          w[j] = (uint32_t)(oracle_exp2c((srow[j] - mx) * c) * 67108864.0f);
          take[j] = 1;
          cand[nc].s = srow[j];
          cand[nc].j = (int32_t)j;
          ++nc;
        }
      }
      const uint64_t theta = (uint64_t)ceil((double)tau * (double)mass_of(w, take, NB));
      qsort(cand, (size_t)nc, sizeof(cand_t), cand_cmp);
      /* grow the set one group of equal scores at a time, highest first */
      for (int64_t j = 0; j < NB; ++j) take[j] = 0;
      int64_t t = 0;
      while (t < nc) {
        const float v = cand[t].s;
        while (t < nc && cand[t].s == v) take[cand[t++].j] = 1;
        if (mass_of(w, take, NB) >= theta) break;
      }
      uint32_t* row = mask + (h * NB + i) * Wd;
      for (int64_t w = 0; w < Wd; ++w) row[w] = 0u;
      int64_t cnt = 0;
      for (int64_t j = 0; j < NB; ++j) {
        if (take[j] || is_text[j]) {
          row[j >> 5] |= 1u << (j & 31);
          ++cnt;
        }
      }
      if (kv_count) kv_count[h * NB + i] = (int32_t)cnt;
      free(w);
      free(take);
      free(cand);
    }
  }
}

/* ------------------------------------------------------------------------------------------------
 * Step 2a/2b.  With Q_r = { i : rank_of_block[i] = r } and P(j) = rank_of_block[j]:
 *   U[r][h]       = OR over i in Q_r of M[h][i]                       (bit words)
 *   D[r][h][p]    = U[r][h] AND own[p]          own[p] = { j : P(j) = p }
 *   cnt[r][p][h]  = |D[r][h][p]|                (p == r kept: local reuse, not in the volume)
 *   V_r           = 2*b*d*w * sum_h sum_{p != r} cnt[r][p][h]
 *   seg_off[r][p][h] = entry index, inside consumer r's buffer, of the first block of
 *                  (producer p, head h), in pack order: p ascending (p == r skipped unless
 *                  include_local), then h ascending.   total[r] = entries in r's buffer.
 * ---------------------------------------------------------------------------------------------- */
void oracle_demand(const uint32_t* mask, const int32_t* rank_of_block, int64_t H, int64_t NB,
                   int64_t P, int64_t b, int64_t d, int64_t w_bytes, int include_local,
                   uint32_t* U, int32_t* cnt, int64_t* seg_off, int64_t* total, int64_t* volume) {
  const int64_t Wd = ceil_div64(NB, 32);
  uint32_t* own = (uint32_t*)calloc((size_t)(P * Wd), sizeof(uint32_t));
  for (int64_t j = 0; j < NB; ++j) own[rank_of_block[j] * Wd + (j >> 5)] |= 1u << (j & 31);
  memset(U, 0, (size_t)(P * H * Wd) * sizeof(uint32_t));
  for (int64_t h = 0; h < H; ++h)
    for (int64_t i = 0; i < NB; ++i) {
      const int64_t r = rank_of_block[i];
      for (int64_t w = 0; w < Wd; ++w) U[(r * H + h) * Wd + w] |= mask[(h * NB + i) * Wd + w];
    }
  for (int64_t r = 0; r < P; ++r) {
    int64_t cursor = 0, remote = 0;
    for (int64_t p = 0; p < P; ++p) {
      for (int64_t h = 0; h < H; ++h) {
        int64_t c = 0;
        for (int64_t w = 0; w < Wd; ++w)
          c += __builtin_popcount(U[(r * H + h) * Wd + w] & own[p * Wd + w]);
        cnt[(r * P + p) * H + h] = (int32_t)c;
        seg_off[(r * P + p) * H + h] = cursor;
        if (p != r) remote += c;
        if (p != r || include_local) cursor += c;
      }
    }
    total[r] = cursor;
    volume[r] = 2 * b * d * w_bytes * remote;
  }
  free(own);
}

/* ------------------------------------------------------------------------------------------------
 * Step 2c.  Consumer r's buffer starts at byte dst_base[r].  For p ascending (p != r unless
 * include_local), h ascending, j ascending in D[r][h][p]: append the b x d K tile of (h, j), then
 * the b x d V tile.  Token rows at or beyond N are written as zeros, so every entry is 2*b*d*2 bytes.
 * ---------------------------------------------------------------------------------------------- */
void oracle_pack(const uint16_t* K, const uint16_t* V, const uint32_t* U,
                 const int32_t* rank_of_block, int64_t H, int64_t N, int64_t d, int64_t b,
                 int64_t P, int include_local, const int64_t* dst_base, uint8_t* packed) {
  const int64_t NB = ceil_div64(N, b);
  const int64_t Wd = ceil_div64(NB, 32);
  const int64_t tile_bytes = b * d * 2;
#pragma omp parallel for schedule(dynamic)
  for (int64_t r = 0; r < P; ++r) {
    uint8_t* out = packed + dst_base[r];
    for (int64_t p = 0; p < P; ++p) {
      if (p == r && !include_local) continue;
      for (int64_t h = 0; h < H; ++h) {
        for (int64_t j = 0; j < NB; ++j) {
          if (rank_of_block[j] != p) continue;
          if (!((U[(r * H + h) * Wd + (j >> 5)] >> (j & 31)) & 1u)) continue;
          const int64_t t0 = j * b;
          const int64_t n_j = (N - t0 < b) ? (N - t0) : b;
          memcpy(out, K + (h * N + t0) * d, (size_t)(n_j * d * 2));
          memset(out + n_j * d * 2, 0, (size_t)(tile_bytes - n_j * d * 2));
          out += tile_bytes;
          memcpy(out, V + (h * N + t0) * d, (size_t)(n_j * d * 2));
          memset(out + n_j * d * 2, 0, (size_t)(tile_bytes - n_j * d * 2));
          out += tile_bytes;
        }
      }
    }
  }
}

/* ------------------------------------------------------------------------------------------------
 * Step 3.  For each listed (head h, query block i) and each of its valid query tokens q:
 *   s_t = (sum_c Q[q][c] K[t][c]) * scale     for every token t < N whose block is kept in
 *                                             row (h, i);   masked keys contribute nothing
 *   m = max_t s_t ;  p_t = exp(s_t - m) ;  O[q][:] = sum_t p_t V[t][:] / sum_t p_t
 *   lse[q] = m + log(sum_t p_t)
 * fp64 throughout; output rows are written densely: out[u][row][c] with `b` rows reserved per
 * listed unit u (rows beyond the block's valid count stay zero).
 * ---------------------------------------------------------------------------------------------- */
void oracle_attn_rows(const uint16_t* Q, const uint16_t* K, const uint16_t* V, const uint32_t* mask,
                      int64_t H, int64_t N, int64_t d, int64_t b, double scale,
                      const int32_t* unit_head, const int32_t* unit_block, int64_t n_units,
                      float* out, float* lse) {
  const int64_t NB = ceil_div64(N, b);
  const int64_t Wd = ceil_div64(NB, 32);
  (void)H;
#pragma omp parallel for schedule(dynamic)
  for (int64_t u = 0; u < n_units; ++u) {
    const int64_t h = unit_head[u], i = unit_block[u];
    const uint32_t* row = mask + (h * NB + i) * Wd;
    double* s = (double*)malloc((size_t)N * sizeof(double));
    double* acc = (double*)malloc((size_t)d * sizeof(double));
    const int64_t q0 = i * b;
    const int64_t n_i = (N - q0 < b) ? (N - q0) : b;
    for (int64_t r = 0; r < b; ++r) {
      float* o = out + (u * b + r) * d;
      for (int64_t c = 0; c < d; ++c) o[c] = 0.0f;
      if (lse) lse[u * b + r] = 0.0f;
      if (r >= n_i) continue;
      const uint16_t* q = Q + (h * N + q0 + r) * d;
      double m = -INFINITY;
      for (int64_t j = 0; j < NB; ++j) {
        if (!((row[j >> 5] >> (j & 31)) & 1u)) continue;
        const int64_t t1 = ((j + 1) * b < N) ? (j + 1) * b : N;
        for (int64_t t = j * b; t < t1; ++t) {
          const uint16_t* k = K + (h * N + t) * d;
          double dot = 0.0;
          for (int64_t c = 0; c < d; ++c) dot += (double)bf16_to_f32(q[c]) * (double)bf16_to_f32(k[c]);
          s[t] = dot * scale;
          if (s[t] > m) m = s[t];
        }
      }
      double denom = 0.0;
      for (int64_t c = 0; c < d; ++c) acc[c] = 0.0;
      for (int64_t j = 0; j < NB; ++j) {
        if (!((row[j >> 5] >> (j & 31)) & 1u)) continue;
        const int64_t t1 = ((j + 1) * b < N) ? (j + 1) * b : N;
        for (int64_t t = j * b; t < t1; ++t) {
          const double p = exp(s[t] - m);
          denom += p;
          const uint16_t* v = V + (h * N + t) * d;
          for (int64_t c = 0; c < d; ++c) acc[c] += p * (double)bf16_to_f32(v[c]);
        }
      }
      if (denom == 0.0) { /* no kept key (only possible for hop-restricted masks): zero row, lse = -inf */
        if (lse) lse[u * b + r] = -INFINITY;
        continue;
      }
      for (int64_t c = 0; c < d; ++c) o[c] = (float)(acc[c] / denom);
      if (lse) lse[u * b + r] = (float)(m + log(denom));
    }
    free(s);
    free(acc);
  }
}

/* The textbook form for tiny inputs: every query token gets a full N-wide logit row in which the
 * keys of masked blocks are -inf; softmax over the row; weighted sum of V.  Also returns the softmax
 * weights' row sums (should be 1) so the "rows sum to one" property can be asserted.
 * out[h][n][c] fp32, rowsum[h][n]. */
void oracle_attn_dense_masked(const uint16_t* Q, const uint16_t* K, const uint16_t* V,
                              const uint32_t* mask, int64_t H, int64_t N, int64_t d, int64_t b,
                              double scale, float* out, double* rowsum) {
  const int64_t NB = ceil_div64(N, b);
  const int64_t Wd = ceil_div64(NB, 32);
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t h = 0; h < H; ++h) {
    for (int64_t qi = 0; qi < N; ++qi) {
      double* s = (double*)malloc((size_t)N * sizeof(double));
      double* pr = (double*)malloc((size_t)N * sizeof(double));
      const int64_t i = qi / b;
      const uint32_t* row = mask + (h * NB + i) * Wd;
      const uint16_t* q = Q + (h * N + qi) * d;
      double m = -INFINITY;
      for (int64_t t = 0; t < N; ++t) {
        const int64_t j = t / b;
        if ((row[j >> 5] >> (j & 31)) & 1u) {
          const uint16_t* k = K + (h * N + t) * d;
          double dot = 0.0;
          for (int64_t c = 0; c < d; ++c) dot += (double)bf16_to_f32(q[c]) * (double)bf16_to_f32(k[c]);
          s[t] = dot * scale;
        } else {
          s[t] = -INFINITY;
        }
        if (s[t] > m) m = s[t];
      }
      double denom = 0.0;
      for (int64_t t = 0; t < N; ++t) {
        pr[t] = exp(s[t] - m);
        denom += pr[t];
      }
      double rs = 0.0;
      for (int64_t t = 0; t < N; ++t) {
        pr[t] /= denom;
        rs += pr[t];
      }
      if (rowsum) rowsum[h * N + qi] = rs;
      for (int64_t c = 0; c < d; ++c) {
        double a = 0.0;
        for (int64_t t = 0; t < N; ++t) a += pr[t] * (double)bf16_to_f32(V[(h * N + t) * d + c]);
        out[(h * N + qi) * d + c] = (float)a;
      }
      free(s);
      free(pr);
    }
  }
}

/* ------------------------------------------------------------------------------------------------
 * Merging partial attention results (ring-attention style, Section 2.3 / Section 7: per-hop partial
 * outputs are combined by online softmax).  For two partial results over DISJOINT key sets, each
 * normalised by its own sum and carrying lse = log(sum of exp of its scaled logits):
 *   lse = log(exp(lse_a) + exp(lse_b));  O = O_a * exp(lse_a - lse) + O_b * exp(lse_b - lse)
 * An empty part has lse = -inf and weight 0.  fp64 throughout.  rows x d.
 * ---------------------------------------------------------------------------------------------- */
void oracle_attn_merge(const float* oa, const float* la, const float* ob, const float* lb, int64_t rows,
                       int64_t d, float* out, float* lse) {
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < rows; ++r) {
    const double a = la[r], b = lb[r];
    const double m = a > b ? a : b;
    if (m == -INFINITY) {
      for (int64_t c = 0; c < d; ++c) out[r * d + c] = 0.0f;
      lse[r] = -INFINITY;
      continue;
    }
    const double ea = exp(a - m), eb = exp(b - m);
    const double tot = ea + eb;
    for (int64_t c = 0; c < d; ++c)
      out[r * d + c] = (float)(((double)oa[r * d + c] * ea + (double)ob[r * d + c] * eb) / tot);
    lse[r] = (float)(m + log(tot));
  }
}

int oracle_num_threads(void) {
#ifdef _OPENMP
  extern int omp_get_max_threads(void);
  return omp_get_max_threads();
#else
  return 1;
#endif
}
