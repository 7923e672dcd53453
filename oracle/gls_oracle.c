/*
 * gls_oracle.c -- plain CPU oracle for Gumbel-max list sampling (GLS).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, literal, fp64 restatement of what the CUDA
 * library computes.  It shares no code, header, table or constant generator with the CUDA path
 * and must never be called from it; only the tests, the smoke check and the benchmark's
 * cpu-baseline leg load it.
 *
 * What it follows (arXiv 2506.05632):
 *   - Sec. 3 / Algorithm 1:  S_i^(k) = -ln U_i^(k);  X^(k) = argmin_i S_i^(k)/p_i;
 *                            Y = argmin_i min_k S_i^(k)/q_i;  accept iff Y in {X^(k)}.
 *   - Sec. 4 / Algorithm 2:  per position j the same races with U_i^(j,k), the active set S,
 *                            early stop when S is empty, bonus token Y_{L+1}.
 *   - Appendix B:            min over all k instead of k in S (strong drafter invariance).
 *   - Sec. 5.1 / Appendix C: encoder index Y, message M = l_Y, decoder indices X^(k) restricted
 *                            to candidates with l_i = M, over (importance) weights; with the
 *                            Gaussian model of Sec. 5.2 / Appendix D.3 also the weights themselves,
 *                            the decoder outputs and the MMSE reconstruction.
 *
 * Races are evaluated in the log domain, argmin_i S_i/p_i = argmax_i (ln p_i - ln S_i), with
 * ln p_i = logit_i / T - lse and lse = ln sum_i exp(logit_i / T) computed by the two-pass
 * max-subtracted formula in fp64.  Ties: lowest token index, then lowest k.
 *
 * Readings where the paper is silent (each also listed in the design notes of the repository):
 *   - The uniforms come from Philox4x32 (Salmon et al., SC'11) keyed by the seed with counter
 *     (token block, k | domain << 16, position id, sequence id); see gls_uniform() below.
 *   - U is taken in the open interval: v = (integer + 0.5) * 2^-32 or 2^-48, U = 1 - v,
 *     S = -ln U = -log1p(-v).
 *   - noise_spec 4 builds each group of 16 exponentials from its minimum (an exact sampler of
 *     16 i.i.d. Exp(1) values; see exp_noise_group_min() below).
 *   - NaN and +inf logits are excluded (they cannot define a probability); -inf is a masked token.
 *
 * Pins (tests/test_oracle_*.py): a second pure-Python Philox, inversion of the Philox round,
 * uniformity / exponentiality tests, Proposition 1 marginals by chi-square, the list matching
 * lemma (Theorem 1) as a lower bound, the exact acceptance probability by quadrature on small
 * alphabets, the K = 1 closed form, p = q always accepts, one-hot p, the exact joint used in the
 * proof of Theorem 1, an independent linear-domain brute force on V <= 8, Algorithm 2 on toy
 * Markov chains, and the compression special cases.
 * Numbers in the paper's experiment tables need datasets and model weights that are not
 * available: parity with those tables is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define GLSO_F32 0
#define GLSO_BF16 1
#define GLSO_F64 2 /* rows the oracle computes itself (Gaussian importance log-weights) */
#define GLSO_NOISE_SHARED_ACROSS_K 1u
#define GLSO_COMBINE_ALL 1u
#define GLSO_NO_BONUS 2u
#define GLSO_MAX_K 64

/* ------------------------------------------------------------------------------------------ */
/* Philox4x32-R, written from the published algorithm: per round                              */
/*   (c0,c1,c2,c3) <- (hi(M1*c2) ^ c1 ^ k0, lo(M1*c2), hi(M0*c0) ^ c3 ^ k1, lo(M0*c0))          */
/* and the key is bumped by the Weyl constants between rounds.                                 */
/* ------------------------------------------------------------------------------------------ */
void glso_philox4x32(const uint32_t ctr[4], const uint32_t key[2], int rounds, uint32_t out[4]) {
  const uint64_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
  const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int r = 0; r < rounds; ++r) {
    if (r > 0) {
      k0 += W0;
      k1 += W1;
    }
    uint64_t p0 = M0 * (uint64_t)c0;
    uint64_t p1 = M1 * (uint64_t)c2;
    uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    uint32_t n1 = (uint32_t)p1;
    uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    uint32_t n3 = (uint32_t)p0;
    c0 = n0;
    c1 = n1;
    c2 = n2;
    c3 = n3;
  }
  out[0] = c0;
  out[1] = c1;
  out[2] = c2;
  out[3] = c3;
}

typedef struct {
  uint64_t seed;
  int rounds;       /* Philox rounds (10 by default) */
  int spec;         /* 1, 2, 3 or 4 */
  uint32_t domain;  /* 0 decoding, 1 compression */
  uint32_t seq, pos, k;
} glso_key_t;

/* The uniform v in (0,1) of token i under the given key: Algorithm 1's U_i^(k) is 1 - v. */
double glso_exp_noise(const glso_key_t* nk, int64_t i);
double glso_uniform(const glso_key_t* nk, int64_t i) {
  if (nk->spec == 4) return -expm1(-glso_exp_noise(nk, i)); /* derived: v = 1 - exp(-S) */
  uint32_t key[2] = {(uint32_t)(nk->seed & 0xffffffffu), (uint32_t)(nk->seed >> 32)};
  uint32_t out[4];
  if (nk->spec == 1) {
    uint32_t ctr[4] = {(uint32_t)(i >> 2), nk->k | (nk->domain << 16), nk->pos, nk->seq};
    glso_philox4x32(ctr, key, nk->rounds, out);
    uint32_t w = out[i & 3];
    return ((double)w + 0.5) * 0x1p-32;
  } else if (nk->spec == 3) {
    /* 8 coarse bits (16 tokens per generator call) + 40 refinement bits (2 tokens per call) */
    uint32_t cc[4] = {(uint32_t)(i >> 4), nk->k | (nk->domain << 16), nk->pos, nk->seq};
    glso_philox4x32(cc, key, nk->rounds, out);
    uint32_t h = (out[(i & 15) >> 2] >> (8 * (i & 3))) & 0xffu;
    uint32_t cr[4] = {(uint32_t)(i >> 1), nk->k | ((nk->domain + 2u) << 16), nk->pos, nk->seq};
    glso_philox4x32(cr, key, nk->rounds, out);
    uint64_t x = ((uint64_t)(out[2 * (i & 1) + 1] & 0xffu) << 32) | out[2 * (i & 1)];
    /* h * 2^40 + x + 0.5 < 2^48 + 1: exact in fp64 */
    return ((double)h * 1099511627776.0 + (double)x + 0.5) * 0x1p-48;
  } else {
    uint32_t cc[4] = {(uint32_t)(i >> 3), nk->k | (nk->domain << 16), nk->pos, nk->seq};
    glso_philox4x32(cc, key, nk->rounds, out);
    uint32_t h = (out[(i & 7) >> 1] >> (16 * (i & 1))) & 0xffffu;
    uint32_t cr[4] = {(uint32_t)(i >> 2), nk->k | ((nk->domain + 2u) << 16), nk->pos, nk->seq};
    glso_philox4x32(cr, key, nk->rounds, out);
    uint32_t r = out[i & 3];
    /* h * 2^32 + r + 0.5 < 2^48 + 1: exact in fp64 */
    return ((double)h * 4294967296.0 + (double)r + 0.5) * 0x1p-48;
  }
}

/*
 * noise_spec 4: the 16 exponentials of tokens 16g .. 16g+15 ("group" g) are built from their
 * minimum.  If E_0..E_15 are i.i.d. Exp(1), then M = min_t E_t ~ Exp(16), its position is uniform
 * on 0..15 and independent of M, and the other fifteen, less M, are again i.i.d. Exp(1) and
 * independent of both (memorylessness; Renyi's representation of exponential order statistics).
 * Read backwards this is a sampler of 16 i.i.d. Exp(1) variables, i.e. of Sec. 3's S_i = -ln U_i:
 *     M   = -log1p(-v0) / 16,   v0 = (w * 2^16 + r + 0.5) * 2^-48
 *     S_i = M                   if (i mod 16) == loc
 *     S_i = M + (-log1p(-v_i))  otherwise,  v_i = (u_i + 0.5) * 2^-32
 * with, for the stream (seed, seq, pos, k, domain):
 *     w   = word (g >> 5) & 3 of Philox(counter ((g >> 7) << 5 | (g & 31), k | domain << 16, pos, seq))
 *           (128 consecutive groups share 32 generator calls, group g and g + 32 the same call)
 *     r   = low 16 bits, loc = bits 16..19 of word 0 of Philox((g, k | (domain + 2) << 16, pos, seq))
 *     u_i = word i & 3 of Philox((i >> 2, k | (domain + 4) << 16, pos, seq)).
 * A sweep that knows w alone already knows S_i >= M >= w * 2^-36 for all 16 tokens of the group.
 */
static double exp_noise_group_min(const glso_key_t* nk, int64_t i) {
  uint32_t key[2] = {(uint32_t)(nk->seed & 0xffffffffu), (uint32_t)(nk->seed >> 32)};
  uint32_t out[4];
  const int64_t g = i >> 4;
  uint32_t cc[4] = {(uint32_t)(((g >> 7) << 5) | (g & 31)), nk->k | (nk->domain << 16), nk->pos, nk->seq};
  glso_philox4x32(cc, key, nk->rounds, out);
  const uint32_t w = out[(g >> 5) & 3];
  uint32_t cr[4] = {(uint32_t)g, nk->k | ((nk->domain + 2u) << 16), nk->pos, nk->seq};
  glso_philox4x32(cr, key, nk->rounds, out);
  const uint32_t r = out[0] & 0xffffu;
  const int loc = (int)((out[0] >> 16) & 15u);
  /* w * 2^16 + r + 0.5 < 2^48 + 1: exact in fp64 */
  const double v0 = ((double)w * 65536.0 + (double)r + 0.5) * 0x1p-48;
  const double M = -log1p(-v0) / 16.0;
  if ((int)(i & 15) == loc) return M;
  uint32_t ct[4] = {(uint32_t)(i >> 2), nk->k | ((nk->domain + 4u) << 16), nk->pos, nk->seq};
  glso_philox4x32(ct, key, nk->rounds, out);
  const double vi = ((double)out[i & 3] + 0.5) * 0x1p-32;
  return M + (-log1p(-vi));
}

/* S = -ln U = -log1p(-v) ~ Exp(1)  (Sec. 3, "S_i^(k) = -ln U_i^(k)") */
double glso_exp_noise(const glso_key_t* nk, int64_t i) {
  if (nk->spec == 4) return exp_noise_group_min(nk, i);
  return -log1p(-glso_uniform(nk, i));
}

/* Flat wrappers for the Python side (ctypes cannot pass the struct by value portably). */
double glso_uniform_flat(uint64_t seed, int rounds, int spec, uint32_t domain, uint32_t seq,
                         uint32_t pos, uint32_t k, int64_t i) {
  glso_key_t nk = {seed, rounds, spec, domain, seq, pos, k};
  return glso_uniform(&nk, i);
}
double glso_exp_noise_flat(uint64_t seed, int rounds, int spec, uint32_t domain, uint32_t seq,
                           uint32_t pos, uint32_t k, int64_t i) {
  glso_key_t nk = {seed, rounds, spec, domain, seq, pos, k};
  return glso_exp_noise(&nk, i);
}
void glso_exp_noise_row(uint64_t seed, int rounds, int spec, uint32_t domain, uint32_t seq,
                        uint32_t pos, uint32_t k, int64_t V, double* out) {
  glso_key_t nk = {seed, rounds, spec, domain, seq, pos, k};
  for (int64_t i = 0; i < V; ++i) out[i] = glso_exp_noise(&nk, i);
}

/* out[B,K,V]: noise of sequences seq_base..seq_base+B-1, drafts 0..K-1, at one position */
void glso_exp_noise_batch(uint64_t seed, int rounds, int spec, uint32_t domain, uint32_t seq_base,
                          int B, uint32_t pos, int K, int64_t V, double* out) {
  for (int b = 0; b < B; ++b)
    for (int k = 0; k < K; ++k) {
      glso_key_t nk = {seed, rounds, spec, domain, seq_base + (uint32_t)b, pos, (uint32_t)k};
      for (int64_t i = 0; i < V; ++i) out[((int64_t)b * K + k) * V + i] = glso_exp_noise(&nk, i);
    }
}

/* ------------------------------------------------------------------------------------------ */
/* Element access                                                                              */
/* ------------------------------------------------------------------------------------------ */
static double load_elem(const void* base, int dtype, int64_t idx) {
  if (dtype == GLSO_F32) return (double)((const float*)base)[idx];
  if (dtype == GLSO_F64) return ((const double*)base)[idx];
  uint32_t bits = (uint32_t)((const uint16_t*)base)[idx] << 16; /* bf16 = top half of an fp32 */
  float f;
  memcpy(&f, &bits, 4);
  return (double)f;
}

/* scaled logit a_i = logit_i / T; excluded tokens (NaN, +inf, wrong bin) become -inf */
static double scaled_logit(const void* row, int dtype, int64_t i, double inv_temp,
                           const uint8_t* bins, int msg) {
  double x = load_elem(row, dtype, i);
  if (isnan(x) || x == INFINITY) return -INFINITY;
  if (bins && (int)bins[i] != msg) return -INFINITY;
  return x * inv_temp;
}

/* lse = ln sum_i exp(a_i), two passes, fp64; -inf if no token has support */
static double row_lse(const void* row, int dtype, int64_t V, double inv_temp, const uint8_t* bins,
                      int msg) {
  double m = -INFINITY;
  for (int64_t i = 0; i < V; ++i) {
    double a = scaled_logit(row, dtype, i, inv_temp, bins, msg);
    if (a > m) m = a;
  }
  if (m == -INFINITY) return -INFINITY;
  double s = 0.0;
  for (int64_t i = 0; i < V; ++i) {
    double a = scaled_logit(row, dtype, i, inv_temp, bins, msg);
    s += exp(a - m);
  }
  return m + log(s);
}
double glso_row_lse(const void* row, int dtype, int64_t V, double inv_temp) {
  return row_lse(row, dtype, V, inv_temp, NULL, 0);
}

/* Running result of one race: best candidate and best candidate with a different token. */
typedef struct {
  double s1;
  int64_t i1;
  int k1;
  double s2; /* best score among candidates whose token differs from i1 (-inf if none) */
  int64_t i2;
} race_t;

static void race_init(race_t* r) {
  r->s1 = -INFINITY;
  r->i1 = -1;
  r->k1 = -1;
  r->s2 = -INFINITY;
  r->i2 = -1;
}

/* order: score descending, then token ascending, then k ascending */
static int better(double s, int64_t i, int k, double s1, int64_t i1, int k1) {
  if (i1 < 0) return 1;
  if (s != s1) return s > s1;
  if (i != i1) return i < i1;
  return k < k1;
}

static void race_offer(race_t* r, double s, int64_t i, int k) {
  if (s == -INFINITY || isnan(s)) return; /* no support */
  if (better(s, i, k, r->s1, r->i1, r->k1)) {
    if (r->i1 >= 0 && i != r->i1) { /* old leader becomes the best "other" token */
      if (r->i2 < 0 || r->s1 > r->s2 || (r->s1 == r->s2 && r->i1 < r->i2)) {
        r->s2 = r->s1;
        r->i2 = r->i1;
      }
    }
    r->s1 = s;
    r->i1 = i;
    r->k1 = k;
  } else if (i != r->i1) {
    if (r->i2 < 0 || s > r->s2 || (s == r->s2 && i < r->i2)) {
      r->s2 = s;
      r->i2 = i;
    }
  }
}

/*
 * Offer every token of one row under noise stream k to the race:
 *     score(i) = a_i - norm - ln S_i^(k),   a_i = logit_i / T
 * norm = 0 gives the draft-side score; norm = lse gives ln(q_i / S_i).
 */
static void race_row(race_t* r, const void* row, int dtype, int64_t V, double inv_temp,
                     double norm, const glso_key_t* nk, const uint8_t* bins, int msg, int k_label) {
  for (int64_t i = 0; i < V; ++i) {
    double a = scaled_logit(row, dtype, i, inv_temp, bins, msg);
    if (a == -INFINITY) continue;
    double S = glso_exp_noise(nk, i);
    double s = (a - norm) - log(S);
    race_offer(r, s, i, k_label);
  }
}

static double gap_of(const race_t* r) {
  if (r->i1 < 0) return NAN;
  if (r->i2 < 0) return INFINITY;
  return r->s1 - r->s2;
}

typedef struct {
  uint64_t seed;
  uint32_t seq_base;
  const uint32_t* seq_ids; /* host array [B] or NULL */
  uint32_t pos_base;
  uint32_t noise_spec; /* 1, 2, 3 or 4 */
  uint32_t rounds;
  uint32_t flags;
} glso_noise_t;

static glso_key_t make_key(const glso_noise_t* nz, uint32_t domain, int b, int j, int k) {
  glso_key_t nk;
  nk.seed = nz->seed;
  nk.rounds = nz->rounds ? (int)nz->rounds : 10;
  nk.spec = nz->noise_spec ? (int)nz->noise_spec : 4;
  nk.domain = domain;
  nk.seq = nz->seq_ids ? nz->seq_ids[b] : nz->seq_base + (uint32_t)b;
  nk.pos = nz->pos_base + (uint32_t)j;
  nk.k = (nz->flags & GLSO_NOISE_SHARED_ACROSS_K) ? 0u : (uint32_t)k;
  return nk;
}

static const void* row_ptr(const void* data, int dtype, int64_t sb, int64_t sk, int64_t sj, int b,
                           int k, int j) {
  int64_t off = sb * b + sk * k + sj * j;
  return (const char*)data + off * (dtype == GLSO_F32 ? 4 : dtype == GLSO_F64 ? 8 : 2);
}

/* ------------------------------------------------------------------------------------------ */
/* Draft side: Algorithm 2 draft loop (and Algorithm 1, third step) for every (b,k,j).         */
/*   tokens[B,K,J], scores[B,K,J] (unnormalised a - ln S), gaps[B,K,J] (top-2, different token) */
/* ------------------------------------------------------------------------------------------ */
int glso_draft_sample(const void* logits, int dtype, int64_t sb, int64_t sk, int64_t sj, int B,
                      int K, int J, int64_t V, float inv_temp, const float* inv_temp_per_draft,
                      const glso_noise_t* nz, int32_t* tokens, double* scores, double* gaps) {
  if (!logits || !nz || !tokens || B <= 0 || K <= 0 || K > GLSO_MAX_K || J <= 0 || V <= 0)
    return 1;
  int64_t R = (int64_t)B * K * J;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t r = 0; r < R; ++r) {
    int j = (int)(r % J), k = (int)((r / J) % K), b = (int)(r / ((int64_t)J * K));
    double it = (double)(inv_temp_per_draft ? inv_temp_per_draft[k] : inv_temp);
    glso_key_t nk = make_key(nz, 0u, b, j, k);
    race_t rc;
    race_init(&rc);
    race_row(&rc, row_ptr(logits, dtype, sb, sk, sj, b, k, j), dtype, V, it, 0.0, &nk, NULL, 0, k);
    tokens[r] = (int32_t)rc.i1;
    if (scores) scores[r] = rc.i1 >= 0 ? rc.s1 : NAN;
    if (gaps) gaps[r] = gap_of(&rc);
  }
  return 0;
}

/* ------------------------------------------------------------------------------------------ */
/* Target side + verification: Algorithm 2, verification phase (active set to the end).         */
/*   tokens[B,J] (-1 beyond tau), tau[B], accept[B,K,L], scores[B,J], gaps[B,J],                 */
/*   row_lse[B,K,J] (NaN for rows the algorithm never evaluates)                                 */
/*   J = L + 1, or L with GLSO_NO_BONUS.                                                         */
/* ------------------------------------------------------------------------------------------ */
int glso_target_sample_verify(const void* logits, int dtype, int64_t sb, int64_t sk, int64_t sj,
                              int B, int K, int L, int64_t V, float inv_temp,
                              const int32_t* draft_tokens, const glso_noise_t* nz, uint32_t flags,
                              int32_t* tokens, int32_t* tau, uint8_t* accept, double* scores,
                              double* gaps, double* row_lse_out) {
  if (!logits || !nz || !tokens || !tau || B <= 0 || K <= 0 || K > GLSO_MAX_K || L < 0 || V <= 0)
    return 1;
  if (L > 0 && (!draft_tokens || !accept)) return 1;
  const int bonus = !(flags & GLSO_NO_BONUS);
  const int J = L + (bonus ? 1 : 0);
  if (J <= 0) return 1;
  const double it = (double)inv_temp;
#pragma omp parallel for schedule(dynamic, 1)
  for (int b = 0; b < B; ++b) {
    int active[GLSO_MAX_K];
    for (int k = 0; k < K; ++k) active[k] = 1;
    for (int j = 0; j < J; ++j) {
      tokens[(int64_t)b * J + j] = -1;
      if (scores) scores[(int64_t)b * J + j] = 0.0;
      if (gaps) gaps[(int64_t)b * J + j] = NAN;
    }
    if (row_lse_out)
      for (int64_t t = 0; t < (int64_t)K * J; ++t) row_lse_out[(int64_t)b * K * J + t] = NAN;
    for (int64_t t = 0; t < (int64_t)K * L; ++t) accept[(int64_t)b * K * L + t] = 0;
    int n_out = 0;
    for (int j = 0; j < J; ++j) {
      race_t rc;
      race_init(&rc);
      if (flags & GLSO_COMBINE_ALL) {
        /* Appendix B: Y_j = argmin_i min_{1<=k<=K} S_i^(j,k) / M_b(i | Y_{1:j-1}, c).  The target
         * distribution of the accepted prefix is the row of any draft that is still active (they
         * share the prefix Y_{1:j-1}); take the lowest such k.  All K noise streams enter. */
        int kref = -1;
        for (int k = 0; k < K && kref < 0; ++k)
          if (active[k]) kref = k;
        const void* row = row_ptr(logits, dtype, sb, sk, sj, b, kref, j);
        double lse = row_lse(row, dtype, V, it, NULL, 0);
        if (row_lse_out) row_lse_out[((int64_t)b * K + kref) * J + j] = lse;
        if (lse != -INFINITY)
          for (int k = 0; k < K; ++k) {
            glso_key_t nk = make_key(nz, 0u, b, j, k);
            race_row(&rc, row, dtype, V, it, lse, &nk, NULL, 0, k);
          }
      } else {
        /* Y_j = argmin_i min_{k in S} S_i^(j,k) / q_i^(j,k) */
        for (int k = 0; k < K; ++k) {
          if (!active[k]) continue;
          const void* row = row_ptr(logits, dtype, sb, sk, sj, b, k, j);
          double lse = row_lse(row, dtype, V, it, NULL, 0);
          if (row_lse_out) row_lse_out[((int64_t)b * K + k) * J + j] = lse;
          if (lse == -INFINITY) continue;
          glso_key_t nk = make_key(nz, 0u, b, j, k);
          race_row(&rc, row, dtype, V, it, lse, &nk, NULL, 0, k);
        }
      }
      tokens[(int64_t)b * J + j] = (int32_t)rc.i1;
      if (scores) scores[(int64_t)b * J + j] = rc.i1 >= 0 ? rc.s1 : NAN;
      if (gaps) gaps[(int64_t)b * J + j] = gap_of(&rc);
      n_out = j + 1;
      if (j == L) break; /* that was the bonus token */
      /* prune: a draft stays active only if its token equals Y_j */
      int any = 0;
      for (int k = 0; k < K; ++k) {
        int ok = active[k] && draft_tokens[((int64_t)b * K + k) * L + j] == (int32_t)rc.i1 &&
                 rc.i1 >= 0;
        accept[((int64_t)b * K + k) * L + j] = (uint8_t)ok;
        active[k] = ok;
        any |= ok;
      }
      if (!any) break; /* S is empty: return Y_1..Y_j */
    }
    tau[b] = n_out;
  }
  return 0;
}

/* ------------------------------------------------------------------------------------------ */
/* Compression: Sec. 5.1 encoder / decoder selection over (importance) log-weights.            */
/*   enc_logw [B,N] (stride enc_sb), dec_logw [B,K,N] (strides dec_sb, dec_sk) or NULL,        */
/*   bins NULL or uint8 [N] (bins_sb = 0) / [B,N].                                              */
/*   enc_index[B], message[B], dec_index[B,K], match[B], scores[B,1+K], gaps[B,1+K]             */
/* ------------------------------------------------------------------------------------------ */
int glso_compress_select(const void* enc_logw, int enc_dtype, int64_t enc_sb, const void* dec_logw,
                         int dec_dtype, int64_t dec_sb, int64_t dec_sk, const uint8_t* bins,
                         int64_t bins_sb, int B, int K, int64_t N, const glso_noise_t* nz,
                         int32_t* enc_index, uint8_t* message, int32_t* dec_index, uint8_t* match,
                         double* scores, double* gaps) {
  if (!enc_logw || !nz || !enc_index || !message || B <= 0 || K <= 0 || K > GLSO_MAX_K || N <= 0)
    return 1;
  if (dec_logw && (!dec_index || !match)) return 1;
#pragma omp parallel for schedule(dynamic, 1)
  for (int b = 0; b < B; ++b) {
    const uint8_t* lab = bins ? bins + bins_sb * b : NULL;
    /* encoder: Y = argmin_i min_k S_i^(k) / lambda_q,i */
    const void* erow = row_ptr(enc_logw, enc_dtype, enc_sb, 0, 0, b, 0, 0);
    double lse = row_lse(erow, enc_dtype, N, 1.0, NULL, 0);
    race_t rc;
    race_init(&rc);
    if (lse != -INFINITY) {
      for (int k = 0; k < K; ++k) {
        glso_key_t nk = make_key(nz, 1u, b, 0, k);
        race_row(&rc, erow, enc_dtype, N, 1.0, lse, &nk, NULL, 0, k);
      }
    }
    enc_index[b] = (int32_t)rc.i1;
    int msg = (lab && rc.i1 >= 0) ? (int)lab[rc.i1] : 0;
    message[b] = (uint8_t)msg; /* M = l_Y */
    if (scores) scores[(int64_t)b * (1 + K)] = rc.i1 >= 0 ? rc.s1 : NAN;
    if (gaps) gaps[(int64_t)b * (1 + K)] = gap_of(&rc);
    if (!dec_logw) continue;
    /* decoder k: X^(k) = argmin over candidates with l_i = M of S_i^(k) / lambda_p,i^(k) */
    int hit = 0;
    for (int k = 0; k < K; ++k) {
      const void* drow = row_ptr(dec_logw, dec_dtype, dec_sb, dec_sk, 0, b, k, 0);
      glso_key_t nk = make_key(nz, 1u, b, 0, k);
      race_t rd;
      race_init(&rd);
      race_row(&rd, drow, dec_dtype, N, 1.0, 0.0, &nk, lab, msg, k);
      dec_index[(int64_t)b * K + k] = (int32_t)rd.i1;
      if (scores) scores[(int64_t)b * (1 + K) + 1 + k] = rd.i1 >= 0 ? rd.s1 : NAN;
      if (gaps) gaps[(int64_t)b * (1 + K) + 1 + k] = gap_of(&rd);
      if (rd.i1 >= 0 && rd.i1 == rc.i1) hit = 1;
    }
    match[b] = (uint8_t)hit;
  }
  return 0;
}

/* ------------------------------------------------------------------------------------------ */
/* Compression from the source: Appendix C (importance sampling) with the Gaussian model of     */
/* Sec. 5.2 / Appendix D.3, applied per dimension to D-dimensional vectors.                     */
/*   candidates u_i (i < N, D floats each) drawn by the caller from the proposal N(0, s2_prior) */
/*   source a_b, side information t_bk = a_b + zeta                                             */
/*   encoder log-weight  ln p_{W|A}(u_i | a_b) - ln prop(u_i),  p_{W|A}(.|a) = N(a, s2_eta)     */
/*   decoder log-weight  ln p_{W|T}(u_i | t_bk) - ln prop(u_i),                                 */
/*                       p_{W|T}(.|t) = N(t / s2_T, s2_W - 1 / s2_T), s2_T = 1 + s2_zeta,       */
/*                       s2_W = 1 + s2_eta                                                      */
/*   (additive terms common to a row are dropped: they cannot change an argmin and cancel in    */
/*   the normalised score; the factor L_max of Appendix C's decoder weight is such a term)      */
/* then the selection of Sec. 5.1 on these weights, the decoder outputs W_k = u_{X^(k)}, the    */
/* MMSE reconstruction g(w, t) = (s2_zeta w + s2_eta t) / (s2_eta + s2_zeta + s2_eta s2_zeta)   */
/* and its squared error per dimension.                                                          */
/*   logw_out: NULL or [B, 1 + K, N] doubles (the weights as computed, for the pins)            */
/*   recon [B,K,D], sqerr [B,K] (mean over the D dimensions); the rest as glso_compress_select  */
/* ------------------------------------------------------------------------------------------ */
static void gaussian_logw_row(const float* u, int64_t N, int D, const double* mean, double var,
                              double s2_prior, double* out) {
  for (int64_t i = 0; i < N; ++i) {
    double acc = 0.0;
    for (int d = 0; d < D; ++d) {
      double x = (double)u[i * D + d];
      double diff = x - mean[d];
      acc += -(diff * diff) / (2.0 * var) + (x * x) / (2.0 * s2_prior);
    }
    out[i] = acc;
  }
}

int glso_compress_gaussian(const float* u, const float* a, const float* t, const uint8_t* bins,
                           int64_t bins_sb, int B, int K, int64_t N, int D, double s2_eta,
                           double s2_zeta, double s2_prior, const glso_noise_t* nz,
                           int32_t* enc_index, uint8_t* message, int32_t* dec_index,
                           uint8_t* match, double* scores, double* gaps, double* recon,
                           double* sqerr, double* logw_out) {
  if (!u || !a || !t || !nz || !enc_index || !message || !dec_index || !match || B <= 0 ||
      K <= 0 || K > GLSO_MAX_K || N <= 0 || D <= 0 || D > 64)
    return 1;
  if (!(s2_eta > 0.0) || !(s2_zeta > 0.0) || !(s2_prior > 0.0)) return 1;
  const double s2T = 1.0 + s2_zeta, s2W = 1.0 + s2_eta;
  const double var_dec = s2W - 1.0 / s2T;
  const double denom = s2_eta + s2_zeta + s2_eta * s2_zeta;
  int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (int b = 0; b < B; ++b) {
    double* w = (double*)malloc(sizeof(double) * (size_t)N);
    if (!w) {
      failed = 1;
      continue;
    }
    double mean[64];
    const uint8_t* lab = bins ? bins + bins_sb * b : NULL;
    /* encoder: Y = argmin_i min_k S_i^(k) / lambda_q,i */
    for (int d = 0; d < D; ++d) mean[d] = (double)a[(int64_t)b * D + d];
    gaussian_logw_row(u, N, D, mean, s2_eta, s2_prior, w);
    if (logw_out) memcpy(logw_out + (int64_t)b * (1 + K) * N, w, sizeof(double) * (size_t)N);
    double lse = row_lse(w, GLSO_F64, N, 1.0, NULL, 0);
    race_t rc;
    race_init(&rc);
    if (lse != -INFINITY)
      for (int k = 0; k < K; ++k) {
        glso_key_t nk = make_key(nz, 1u, b, 0, k);
        race_row(&rc, w, GLSO_F64, N, 1.0, lse, &nk, NULL, 0, k);
      }
    enc_index[b] = (int32_t)rc.i1;
    int msg = (lab && rc.i1 >= 0) ? (int)lab[rc.i1] : 0;
    message[b] = (uint8_t)msg;
    if (scores) scores[(int64_t)b * (1 + K)] = rc.i1 >= 0 ? rc.s1 : NAN;
    if (gaps) gaps[(int64_t)b * (1 + K)] = gap_of(&rc);
    /* decoder k: X^(k) over the candidates labelled M, W_k = u_{X^(k)}, reconstruction g(W_k, t_k) */
    int hit = 0;
    for (int k = 0; k < K; ++k) {
      const float* tk = t + ((int64_t)b * K + k) * D;
      for (int d = 0; d < D; ++d) mean[d] = (double)tk[d] / s2T;
      gaussian_logw_row(u, N, D, mean, var_dec, s2_prior, w);
      if (logw_out)
        memcpy(logw_out + ((int64_t)b * (1 + K) + 1 + k) * N, w, sizeof(double) * (size_t)N);
      glso_key_t nk = make_key(nz, 1u, b, 0, k);
      race_t rd;
      race_init(&rd);
      race_row(&rd, w, GLSO_F64, N, 1.0, 0.0, &nk, lab, msg, k);
      dec_index[(int64_t)b * K + k] = (int32_t)rd.i1;
      if (scores) scores[(int64_t)b * (1 + K) + 1 + k] = rd.i1 >= 0 ? rd.s1 : NAN;
      if (gaps) gaps[(int64_t)b * (1 + K) + 1 + k] = gap_of(&rd);
      if (rd.i1 >= 0 && rd.i1 == rc.i1) hit = 1;
      double se = 0.0;
      for (int d = 0; d < D; ++d) {
        double g = NAN;
        if (rd.i1 >= 0) {
          double wk = (double)u[rd.i1 * D + d];
          g = (s2_zeta * wk + s2_eta * (double)tk[d]) / denom;
          double e = g - (double)a[(int64_t)b * D + d];
          se += e * e;
        }
        if (recon) recon[((int64_t)b * K + k) * D + d] = g;
      }
      if (sqerr) sqerr[(int64_t)b * K + k] = rd.i1 >= 0 ? se / D : NAN;
    }
    match[b] = (uint8_t)hit;
    free(w);
  }
  return failed;
}

void glso_set_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}
int glso_max_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}
