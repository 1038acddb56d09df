/*
 * ISD-step oracle: a plain, slow, fp64 CPU statement of what one introspective
 * strided decoding (ISD) step computes.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT PRODUCT CODE.  Only the test-suite, the smoke
 * check and the benchmark's CPU-baseline leg may call it.  It shares no source,
 * header, table or helper with the CUDA library and must never be reached from
 * the product path.
 *
 * What it follows (paper: "Introspective Diffusion Language Models"):
 *   - Algorithm 1 (one ISD iteration): stride, introspect, adaptive accept,
 *     residual resample, bonus token, KV commit.
 *   - Sec. 3.2 "Adaptive stride via p/q acceptance": accept with probability
 *     min(1, p/q); on rejection resample from normalize(max(0, p - q)) and drop
 *     everything after; all accepted => bonus token from the final anchor.
 *   - Sec. 3.1 "Causal training with logit shift": strict causal mask (key i is
 *     visible to query j iff i <= j); the row at position i predicts token i+1;
 *     clean rows give the anchor law p, [MASK] rows give the proposal law q.
 *   - Sec. 3.3 (1),(2): a step is an "extend" of 2N-1 rows against a paged KV
 *     cache; after verification rejected and [MASK] positions are trimmed.
 *   - Appendix "TPF and Compute Overhead Analysis": NP step / P step renewal
 *     process (a step after a rejection has nothing to introspect).
 *   - Sec. 4.3 relaxed acceptance: the ratio is multiplied by (1 + tau).
 *
 * Every function states the arithmetic in the order the paper gives it; there is
 * no blocking, fusion or reordering.  All floating point is fp64; bf16/fp32
 * inputs are widened exactly.
 *
 * Pins (tests/test_oracle_*.py, run without a GPU): Philox known-answer values
 * and uniformity; log-sum-exp against scipy; accept rule closed forms
 * (p == q always accepted, p(x) = 0 never accepted, lattice counts);
 * chi-square of residual / bonus / finalised-token laws on tiny vocabularies;
 * brute-force enumeration of P(a >= j); the paper's TPF closed form (Eq. 3) on
 * free-running chains; the worked example of the step-by-step figure;
 * attention against torch's fp64 scaled_dot_product_attention, closed forms for
 * the causal limit and for paging/GQA mapping; allocator conservation and a
 * dictionary model of the page allocator.  No function here is "parity unpinned".
 *
 * Block layout per slot (rows of the 2N-1 wide query block):
 *   row 0                      anchor: last finalised token (has no KV yet)
 *   rows 1 .. n_ver            proposals under verification
 *   rows n_ver+1 .. n_ver+N-1  [MASK] rows that propose
 *   rows q_len .. Q-1          padding, ignored       (q_len = n_ver + N)
 * Row r sits at sequence position ctx_len + r.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_ST_POOL_EXHAUSTED 1u
#define ORC_ST_SLOT_CAPACITY 2u
#define ORC_ST_BAD_TOKEN_ID 4u
#define ORC_ST_BAD_PAGE_ID 8u
#define ORC_ST_NONFINITE_LOGIT 16u
#define ORC_ST_EMPTY_RESIDUAL 32u

#define ORC_TAG_ACCEPT 0u   /* uniform of the accept test, position j          */
#define ORC_TAG_FINAL 1u    /* Gumbel noise of the resampled / bonus token     */
#define ORC_TAG_PROPOSE 2u  /* Gumbel noise of proposal m                      */

static int g_threads = 1;
void orc_set_threads(int n) { g_threads = n < 1 ? 1 : n; }
int orc_get_threads(void) { return g_threads; }
int orc_max_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ------------------------------------------------------------------------- */
/* Random numbers: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11).  The     */
/* paper only says "draw r ~ Uniform(0,1)" (Algorithm 1) and names Gumbel-max  */
/* sampling (Sec. 3.3 (3)); the counter layout below is this build's reading.  */
/* ------------------------------------------------------------------------- */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    if (round > 0) {
      k0 += 0x9E3779B9u;
      k1 += 0xBB67AE85u;
    }
    uint64_t prod0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
    uint64_t prod1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
    uint32_t hi0 = (uint32_t)(prod0 >> 32), lo0 = (uint32_t)prod0;
    uint32_t hi1 = (uint32_t)(prod1 >> 32), lo1 = (uint32_t)prod1;
    uint32_t n0 = hi1 ^ c1 ^ k0;
    uint32_t n1 = lo1;
    uint32_t n2 = hi0 ^ c3 ^ k1;
    uint32_t n3 = lo0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* counter = (lane, step, slot, tag<<16 | position); key = (seed lo, seed hi) */
static uint32_t draw_word(uint64_t seed, uint32_t step, uint32_t slot, uint32_t tag,
                          uint32_t position, uint32_t vocab_index) {
  uint32_t ctr[4] = {vocab_index >> 2, step, slot, (tag << 16) | position};
  uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  uint32_t out[4];
  orc_philox4x32_10(ctr, key, out);
  return out[vocab_index & 3u];
}

/* Uniform on the lattice {0, 1, ..., 2^24-1} * 2^-24, i.e. in [0, 1). */
double orc_uniform(uint64_t seed, uint32_t step, uint32_t slot, uint32_t position) {
  uint32_t w = draw_word(seed, step, slot, ORC_TAG_ACCEPT, position, 0);
  return (double)(w >> 8) * 0x1p-24;
}

/* Standard Gumbel variate for vocabulary index i: u' in (0,1), g = -ln(-ln u'). */
double orc_gumbel(uint64_t seed, uint32_t step, uint32_t slot, uint32_t tag, uint32_t position,
                  uint32_t vocab_index) {
  uint32_t w = draw_word(seed, step, slot, tag, position, vocab_index);
  double u = ((double)(w >> 8) + 0.5) * 0x1p-24;
  return -log(-log(u));
}

/* ------------------------------------------------------------------------- */
/* Input widening                                                             */
/* ------------------------------------------------------------------------- */
static inline double bf16_to_f64(uint16_t h) {
  uint32_t w = (uint32_t)h << 16;
  float f;
  memcpy(&f, &w, sizeof f);
  return (double)f;
}

/* logits_dtype: 0 = fp32, 1 = bf16 */
static inline double logit_at(const void* base, int dtype, size_t idx) {
  if (dtype == 0) return (double)((const float*)base)[idx];
  return bf16_to_f64(((const uint16_t*)base)[idx]);
}

/* Scaled row (logit * invT) into a double buffer; returns 1 if a NaN or +inf
 * was seen (-inf is a legal "probability zero" logit). */
static int load_row(const void* base, int dtype, size_t row_offset, int V, double invT, double* dst) {
  int bad = 0;
  for (int i = 0; i < V; ++i) {
    double x = logit_at(base, dtype, row_offset + (size_t)i) * invT;
    if (isnan(x) || (isinf(x) && x > 0)) bad = 1;
    dst[i] = x;
  }
  return bad;
}

/* log sum_i exp(row_i), with the maximum subtracted first. */
double orc_logsumexp(const double* row, int V) {
  double m = -INFINITY;
  for (int i = 0; i < V; ++i)
    if (row[i] > m) m = row[i];
  if (isinf(m) && m < 0) return -INFINITY;
  double s = 0.0;
  for (int i = 0; i < V; ++i) s += exp(row[i] - m);
  return m + log(s);
}

/* Top-k / top-p filtered law of a scaled row (the serving configuration of the paper's appendix:
 * temperature, then top-k, then top-p on what top-k kept).  In place: entries outside the support
 * become -inf, so that softmax(row) afterwards IS the filtered, renormalised law and every routine
 * below (log-sum-exp, Gumbel-max, residual) applies unchanged.
 *   1. S_k = the top_k entries in the order (value descending, index ascending);
 *   2. w_i = exp(row_i - max) over S_k in that order, Z = sum w_i;
 *   3. the support is the shortest prefix of S_k whose cumulated w reaches top_p * Z
 *      (all of S_k when it is never reached, e.g. top_p = 1 with rounding).
 * top_k <= 0 leaves the row alone.  NaN entries are never selected. */
void orc_filter_row(double* row, int V, int top_k, double top_p) {
  if (top_k <= 0) return;
  if (top_k > V) top_k = V;
  int* sel = (int*)malloc(sizeof(int) * (size_t)top_k);
  char* taken = (char*)calloc((size_t)V, 1);
  if (!sel || !taken) { free(sel); free(taken); return; }
  int n = 0;
  for (int r = 0; r < top_k; ++r) {  /* selection, one maximum at a time */
    int best = -1;
    for (int i = 0; i < V; ++i) {
      if (taken[i] || isnan(row[i])) continue;
      if (best < 0 || row[i] > row[best]) best = i;  /* strict >: the lowest index wins ties */
    }
    if (best < 0) break;
    taken[best] = 1;
    sel[n++] = best;
  }
  int keep = n;
  if (n > 0 && !(isinf(row[sel[0]]) && row[sel[0]] < 0)) {
    const double m = row[sel[0]];
    double Z = 0.0;
    for (int r = 0; r < n; ++r) Z += exp(row[sel[r]] - m);
    double cum = 0.0;
    for (int r = 0; r < n; ++r) {
      cum += exp(row[sel[r]] - m);
      if (cum >= top_p * Z) { keep = r + 1; break; }
    }
  }
  memset(taken, 0, (size_t)V);
  for (int r = 0; r < keep; ++r) taken[sel[r]] = 1;
  for (int i = 0; i < V; ++i)
    if (!taken[i] && !isnan(row[i])) row[i] = -INFINITY;
  free(sel);
  free(taken);
}

/* argmax_i (score_i) with the lowest index winning ties; also reports the gap
 * between the best and the second-best score (for "fragile sample" reporting). */
typedef struct {
  int idx;
  double best, second;
} top2_t;

static inline void top2_init(top2_t* t) {
  t->idx = -1;
  t->best = -INFINITY;
  t->second = -INFINITY;
}
static inline void top2_push(top2_t* t, int i, double s) {
  if (t->idx < 0 || s > t->best) {
    if (t->idx >= 0) t->second = t->best;
    t->best = s;
    t->idx = i;
  } else if (s > t->second) {
    t->second = s;
  }
}

/* Gumbel-max sample of softmax(row): argmax_i(row_i + g_i).  Elements with
 * row_i = -inf have probability zero and never win. */
static int sample_row(const double* row, int V, uint64_t seed, uint32_t step, uint32_t slot,
                      uint32_t tag, uint32_t position, double* margin) {
  top2_t t;
  top2_init(&t);
  for (int i = 0; i < V; ++i) {
    if (isinf(row[i]) && row[i] < 0) continue;
    top2_push(&t, i, row[i] + orc_gumbel(seed, step, slot, tag, position, (uint32_t)i));
  }
  if (margin) *margin = t.best - t.second;
  return t.idx;
}

static int argmax_row(const double* row, int V, double* margin) {
  top2_t t;
  top2_init(&t);
  for (int i = 0; i < V; ++i) top2_push(&t, i, row[i]);
  if (margin) *margin = t.best - t.second;
  return t.idx;
}

/* ------------------------------------------------------------------------- */
/* Verify + propose for one slot  (Algorithm 1, "Introspection with adaptive   */
/* stride" loop, bonus-token branch, and the "Stride" loop for the new masks).  */
/* ------------------------------------------------------------------------- */
typedef struct {
  int B, N, V, logits_dtype, q_mode, propose_mode;
  double invT, tau;
  uint64_t seed;
  uint32_t step;
  const int32_t* n_ver;
  const uint8_t* active;
  const int32_t* block_tok; /* [B, Q]; rows 1..n_ver hold the proposals */
  const int32_t* q_row0;    /* [B] first proposal-law row inside q_prev for the slot */
  const void* logits_cur;   /* [B, Q, V] */
  const void* q_prev;       /* [B, Q, V] previous step's logits (its MASK rows are the q rows) */
  int8_t* accept;           /* [B, N-1]  1 accepted, 0 first rejection, -1 not evaluated */
  double* alpha;            /* [B, N-1]  min(1, (1+tau) p/q) where evaluated, else NaN */
  double* u_draw;           /* [B, N-1]  the uniform used, else NaN */
  int32_t* accept_len;      /* [B] a */
  int32_t* n_emit;          /* [B] a + 1 */
  int32_t* repl_tok;        /* [B] y: resampled or bonus token */
  int32_t* out_tok;         /* [B, N] finalised tokens, -1 padded */
  int32_t* new_prop_tok;    /* [B, N-1] */
  double* new_q_stats;      /* [B, N-1, 2] = {LSE(row), row[x^]} */
  double* final_margin;     /* [B] top-2 gap of y's score */
  double* prop_margin;      /* [B, N-1] top-2 gap of each proposal's score */
  uint32_t* slot_status;    /* [B] OR-ed status bits */
  int top_k;                /* 0 = unfiltered laws */
  double top_p;
} verify_args;

static void verify_slot(const verify_args* A, int b, double* lp, double* lq) {
  const int N = A->N, V = A->V, Q = 2 * N - 1, NP = N - 1;
  const int nv = A->n_ver[b];
  int8_t* accept = A->accept + (size_t)b * NP;
  double* alpha = A->alpha + (size_t)b * NP;
  double* u_draw = A->u_draw + (size_t)b * NP;
  for (int j = 0; j < NP; ++j) {
    accept[j] = -1;
    alpha[j] = NAN;
    u_draw[j] = NAN;
    A->new_prop_tok[(size_t)b * NP + j] = -1;
    A->new_q_stats[((size_t)b * NP + j) * 2 + 0] = NAN;
    A->new_q_stats[((size_t)b * NP + j) * 2 + 1] = NAN;
    A->prop_margin[(size_t)b * NP + j] = NAN;
  }
  for (int j = 0; j < N; ++j) A->out_tok[(size_t)b * N + j] = -1;
  A->accept_len[b] = 0;
  A->n_emit[b] = 0;
  A->repl_tok[b] = -1;
  A->final_margin[b] = NAN;
  if (!A->active[b]) return;
  if (nv < 0 || nv > NP) {
    A->slot_status[b] |= ORC_ST_SLOT_CAPACITY;
    return;
  }
  const size_t cur_base = (size_t)b * Q * V;
  uint32_t status = 0;

  /* Introspection: proposal j (row j of the block) is judged by the anchor law
   * p_j read from row j-1 of this step's logits (logit shift) against the law
   * q_j it was drawn from (the previous step's MASK row). */
  int a = nv;   /* accepted-prefix length if nothing is rejected */
  int y = -1;
  double y_margin = NAN;
  for (int j = 1; j <= nv; ++j) {
    const int x = A->block_tok[(size_t)b * Q + j];
    if (x < 0 || x >= V) {
      status |= ORC_ST_BAD_TOKEN_ID;
      a = -1;
      break;
    }
    if (load_row(A->logits_cur, A->logits_dtype, cur_base + (size_t)(j - 1) * V, V, A->invT, lp))
      status |= ORC_ST_NONFINITE_LOGIT;
    orc_filter_row(lp, V, A->top_k, A->top_p);
    const double lse_p = orc_logsumexp(lp, V);
    double lse_q = 0.0, logq_x = 0.0;
    if (A->q_mode == 0) {
      const size_t qoff = ((size_t)b * Q + (size_t)(A->q_row0[b] + j - 1)) * V;
      if (load_row(A->q_prev, A->logits_dtype, qoff, V, A->invT, lq)) status |= ORC_ST_NONFINITE_LOGIT;
      orc_filter_row(lq, V, A->top_k, A->top_p);
      lse_q = orc_logsumexp(lq, V);
      logq_x = lq[x] - lse_q;
    }
    const double logp_x = lp[x] - lse_p;
    const double rho = exp(logp_x - logq_x);          /* p_j(x) / q_j(x) */
    double al = (1.0 + A->tau) * rho;                  /* relaxed acceptance */
    if (al > 1.0) al = 1.0;
    if (isnan(al)) al = 0.0;
    const double u = orc_uniform(A->seed, A->step, (uint32_t)b, (uint32_t)j);
    alpha[j - 1] = al;
    u_draw[j - 1] = u;
    if (u < al) {
      accept[j - 1] = 1;
      continue;
    }
    /* First rejection: resample from normalize(max(0, p - q)) by Gumbel-max
     * over ln(residual); everything after position j is discarded. */
    accept[j - 1] = 0;
    a = j - 1;
    top2_t t;
    top2_init(&t);
    for (int i = 0; i < V; ++i) {
      const double pi = exp(lp[i] - lse_p);
      const double qi = (A->q_mode == 0) ? exp(lq[i] - lse_q) : (i == x ? 1.0 : 0.0);
      const double r = pi - qi;
      if (!(r > 0.0)) continue;
      top2_push(&t, i, log(r) + orc_gumbel(A->seed, A->step, (uint32_t)b, ORC_TAG_FINAL, (uint32_t)j, (uint32_t)i));
    }
    if (t.idx < 0) {
      /* residual numerically empty: fall back to p with the same noise */
      status |= ORC_ST_EMPTY_RESIDUAL;
      y = sample_row(lp, V, A->seed, A->step, (uint32_t)b, ORC_TAG_FINAL, (uint32_t)j, &y_margin);
    } else {
      y = t.idx;
      y_margin = t.best - t.second;
    }
    break;
  }
  if (a < 0) {
    A->slot_status[b] |= status;
    return;
  }
  if (a == nv) {
    /* Nothing rejected (or nothing to verify): the row of the last clean token
     * gives the next token's anchor law; sample it (bonus token; in an NP step
     * this is the quality-guaranteed AR token). */
    if (load_row(A->logits_cur, A->logits_dtype, cur_base + (size_t)nv * V, V, A->invT, lp))
      status |= ORC_ST_NONFINITE_LOGIT;
    orc_filter_row(lp, V, A->top_k, A->top_p);
    y = sample_row(lp, V, A->seed, A->step, (uint32_t)b, ORC_TAG_FINAL, (uint32_t)(nv + 1), &y_margin);
  }
  A->accept_len[b] = a;
  A->n_emit[b] = a + 1;
  A->repl_tok[b] = y;
  A->final_margin[b] = y_margin;
  for (int j = 1; j <= a; ++j) A->out_tok[(size_t)b * N + (j - 1)] = A->block_tok[(size_t)b * Q + j];
  A->out_tok[(size_t)b * N + a] = y;

  /* Stride: each MASK row proposes the token after its position.  After a rejection "all subsequent tokens are
   * discarded; the next step becomes a pure stride with no tokens to introspect" (Sec. 3.2, adaptive stride): the
   * MASK rows were conditioned on the discarded tokens, so no proposals are made from them and the outputs keep
   * their defaults (-1 / NaN).  The rows are still checked for non-finite logits. */
  for (int m = 1; m <= NP; ++m) {
    if (load_row(A->logits_cur, A->logits_dtype, cur_base + (size_t)(nv + m) * V, V, A->invT, lp))
      status |= ORC_ST_NONFINITE_LOGIT;
    if (a != nv) continue;
    orc_filter_row(lp, V, A->top_k, A->top_p);
    double margin;
    int xh;
    if (A->propose_mode == 0)
      xh = sample_row(lp, V, A->seed, A->step, (uint32_t)b, ORC_TAG_PROPOSE, (uint32_t)m, &margin);
    else
      xh = argmax_row(lp, V, &margin);
    A->new_prop_tok[(size_t)b * NP + (m - 1)] = xh;
    A->prop_margin[(size_t)b * NP + (m - 1)] = margin;
    A->new_q_stats[((size_t)b * NP + (m - 1)) * 2 + 0] = orc_logsumexp(lp, V);
    A->new_q_stats[((size_t)b * NP + (m - 1)) * 2 + 1] = xh >= 0 ? lp[xh] : NAN;
  }
  A->slot_status[b] |= status;
}

/* The same with every law (anchor p, proposal q, bonus, MASK rows) filtered by top-k then top-p first. */
int orc_verify_filtered(int top_k, double top_p, int B, int N, int V, int logits_dtype, int q_mode, int propose_mode, double invT,
               double tau, uint64_t seed, uint32_t step, const int32_t* n_ver, const uint8_t* active,
               const int32_t* block_tok, const int32_t* q_row0, const void* logits_cur,
               const void* q_prev, int8_t* accept, double* alpha, double* u_draw, int32_t* accept_len,
               int32_t* n_emit, int32_t* repl_tok, int32_t* out_tok, int32_t* new_prop_tok,
               double* new_q_stats, double* final_margin, double* prop_margin, uint32_t* slot_status) {
  if (B < 0 || N < 1 || V < 1) return -1;
  verify_args A = {B, N, V, logits_dtype, q_mode, propose_mode, invT, tau, seed, step, n_ver, active,
                   block_tok, q_row0, logits_cur, q_prev, accept, alpha, u_draw, accept_len, n_emit,
                   repl_tok, out_tok, new_prop_tok, new_q_stats, final_margin, prop_margin, slot_status,
                   top_k, top_p};
  int fail = 0;
#pragma omp parallel num_threads(g_threads)
  {
    double* lp = (double*)malloc(sizeof(double) * (size_t)V);
    double* lq = (double*)malloc(sizeof(double) * (size_t)V);
    if (!lp || !lq) {
#pragma omp atomic write
      fail = 1;
    } else {
#pragma omp for schedule(dynamic, 1)
      for (int b = 0; b < B; ++b) verify_slot(&A, b, lp, lq);
    }
    free(lp);
    free(lq);
  }
  return fail ? -2 : 0;
}

int orc_verify(int B, int N, int V, int logits_dtype, int q_mode, int propose_mode, double invT,
               double tau, uint64_t seed, uint32_t step, const int32_t* n_ver, const uint8_t* active,
               const int32_t* block_tok, const int32_t* q_row0, const void* logits_cur,
               const void* q_prev, int8_t* accept, double* alpha, double* u_draw, int32_t* accept_len,
               int32_t* n_emit, int32_t* repl_tok, int32_t* out_tok, int32_t* new_prop_tok,
               double* new_q_stats, double* final_margin, double* prop_margin, uint32_t* slot_status) {
  return orc_verify_filtered(0, 1.0, B, N, V, logits_dtype, q_mode, propose_mode, invT, tau, seed, step, n_ver, active,
                             block_tok, q_row0, logits_cur, q_prev, accept, alpha, u_draw, accept_len, n_emit,
                             repl_tok, out_tok, new_prop_tok, new_q_stats, final_margin, prop_margin, slot_status);
}

/* ------------------------------------------------------------------------- */
/* Attention (plain definition): strict causal softmax attention of the block  */
/* rows against the slot's paged KV followed by the block's own rows            */
/* (Sec. 3.1: key i visible to query j iff i <= j; Sec. 3.3 (1): extend of      */
/* 2N-1 rows against the paged cache).  GQA: query head h reads KV head h / G.  */
/* Also appends the block's K/V rows to the slot's pages.                      */
/* ------------------------------------------------------------------------- */
int orc_attn(int B, int Q, int Hq, int Hkv, int D, int page_size, int max_pages, int num_pages,
             double sm_scale, const int32_t* ctx_len, const int32_t* q_len, const uint8_t* active,
             const int32_t* page_table, const uint16_t* q, const uint16_t* k_new,
             const uint16_t* v_new, uint16_t* k_pool, uint16_t* v_pool, double* out, double* lse,
             uint32_t* slot_status) {
  if (Hkv < 1 || Hq % Hkv != 0) return -1;
  const int G = Hq / Hkv;
#pragma omp parallel for schedule(dynamic, 1) num_threads(g_threads)
  for (int b = 0; b < B; ++b) {
    if (!active[b]) continue;
    const int ctx = ctx_len[b], ql = q_len[b];
    if (ctx < 0 || ql < 0 || ql > Q || (ctx + ql + page_size - 1) / page_size > max_pages) {
      slot_status[b] |= ORC_ST_SLOT_CAPACITY;
      continue;
    }
    int bad_page = 0;
    for (int pg = 0; pg < (ctx + ql + page_size - 1) / page_size; ++pg) {
      int id = page_table[(size_t)b * max_pages + pg];
      if (id < 0 || id >= num_pages) bad_page = 1;
    }
    if (bad_page) {
      slot_status[b] |= ORC_ST_BAD_PAGE_ID;
      continue;
    }
    double* s = (double*)malloc(sizeof(double) * (size_t)(ctx + ql));
    for (int r = 0; r < ql; ++r) {
      for (int h = 0; h < Hq; ++h) {
        const int g = h / G;
        const uint16_t* qv = q + (((size_t)b * Q + r) * Hq + h) * D;
        const int nkeys = ctx + r + 1; /* keys 0 .. ctx + r */
        double m = -INFINITY;
        for (int j = 0; j < nkeys; ++j) {
          const uint16_t* kv;
          if (j < ctx) {
            const int page = page_table[(size_t)b * max_pages + j / page_size];
            kv = k_pool + (((size_t)page * Hkv + g) * page_size + (j % page_size)) * D;
          } else {
            kv = k_new + (((size_t)b * Q + (j - ctx)) * Hkv + g) * D;
          }
          double dot = 0.0;
          for (int d = 0; d < D; ++d) dot += bf16_to_f64(qv[d]) * bf16_to_f64(kv[d]);
          s[j] = sm_scale * dot;
          if (s[j] > m) m = s[j];
        }
        double denom = 0.0;
        for (int j = 0; j < nkeys; ++j) {
          s[j] = exp(s[j] - m);
          denom += s[j];
        }
        double* o = out + (((size_t)b * Q + r) * Hq + h) * D;
        for (int d = 0; d < D; ++d) o[d] = 0.0;
        for (int j = 0; j < nkeys; ++j) {
          const uint16_t* vv;
          if (j < ctx) {
            const int page = page_table[(size_t)b * max_pages + j / page_size];
            vv = v_pool + (((size_t)page * Hkv + g) * page_size + (j % page_size)) * D;
          } else {
            vv = v_new + (((size_t)b * Q + (j - ctx)) * Hkv + g) * D;
          }
          const double w = s[j] / denom;
          for (int d = 0; d < D; ++d) o[d] += w * bf16_to_f64(vv[d]);
        }
        if (lse) lse[((size_t)b * Q + r) * Hq + h] = m + log(denom);
      }
    }
    free(s);
    /* K/V append: rows 0..q_len-1 of the block land at positions ctx..ctx+q_len-1 */
    for (int r = 0; r < ql; ++r) {
      const int pos = ctx + r;
      const int page = page_table[(size_t)b * max_pages + pos / page_size];
      for (int g = 0; g < Hkv; ++g) {
        const size_t dst = (((size_t)page * Hkv + g) * page_size + (pos % page_size)) * D;
        const size_t src = (((size_t)b * Q + r) * Hkv + g) * D;
        memcpy(k_pool + dst, k_new + src, sizeof(uint16_t) * (size_t)D);
        memcpy(v_pool + dst, v_new + src, sizeof(uint16_t) * (size_t)D);
      }
    }
  }
  return 0;
}

/* ------------------------------------------------------------------------- */
/* Commit / rollback (Algorithm 1 last line; Sec. 3.3 (2) trim-and-commit;     */
/* appendix renewal process).  KV of the anchor and of the a accepted rows is   */
/* kept (a logical prefix, so dropping the rest is a truncation of ctx_len);    */
/* proposals made this step stay valid only if nothing was rejected.            */
/* Pages: a slot always owns ceil((ctx_len + Q) / page_size) pages; the ones it */
/* lacks after the commit are popped from the top of the free stack, slots in   */
/* ascending order, logical pages in ascending order.                           */
/* ------------------------------------------------------------------------- */
int orc_commit(int B, int N, int page_size, int max_pages, int mask_token, int32_t* ctx_len,
               int32_t* n_ver, int32_t* block_tok, int32_t* q_row0, double* q_stats,
               int32_t* page_table, int32_t* free_stack, int32_t* free_top, const uint8_t* active,
               uint32_t* slot_status, const int32_t* accept_len, const int32_t* repl_tok,
               const int32_t* new_prop_tok, const double* new_q_stats) {
  const int Q = 2 * N - 1, NP = N - 1;
  const int top0 = free_top[0];
  int requested = 0; /* pages requested by the slots before this one (served or not) */
  int popped = 0;    /* pages actually handed out */
  for (int b = 0; b < B; ++b) {
    if (!active[b]) continue;
    /* a slot with an error bit keeps its state so that the caller can recover */
    if ((slot_status[b] & ~ORC_ST_EMPTY_RESIDUAL) != 0) continue;
    const int a = accept_len[b];
    const int nv = n_ver[b];
    const int ctx_new = ctx_len[b] + a + 1; /* anchor + accepted proposals gain KV */
    const int have = (ctx_len[b] + Q + page_size - 1) / page_size;
    const int want = (ctx_new + Q + page_size - 1) / page_size;
    const int need = want - have;
    if (want > max_pages) {
      slot_status[b] |= ORC_ST_SLOT_CAPACITY;
      continue;
    }
    if (need > 0) {
      /* requests are served in slot order while they fit; once one does not fit
       * every later request fails too, so the served ones are a prefix */
      if (requested + need > top0) {
        slot_status[b] |= ORC_ST_POOL_EXHAUSTED;
        requested += need;
        continue;
      }
      for (int i = 0; i < need; ++i)
        page_table[(size_t)b * max_pages + have + i] = free_stack[top0 - 1 - (requested + i)];
      requested += need;
      popped += need;
    }
    ctx_len[b] = ctx_new;
    const int all_accepted = (a == nv);
    /* proposals made this step follow the bonus token only if nothing was
     * rejected; otherwise the next step is a pure stride (NP step) */
    n_ver[b] = all_accepted ? NP : 0;
    q_row0[b] = nv + 1; /* row of this step's first MASK row inside its logits buffer */
    block_tok[(size_t)b * Q + 0] = repl_tok[b];
    for (int m = 1; m <= NP; ++m) {
      block_tok[(size_t)b * Q + m] = all_accepted ? new_prop_tok[(size_t)b * NP + (m - 1)] : mask_token;
      if (!all_accepted) continue; /* no proposals were made: the statistics of the old ones stay (unused) */
      q_stats[((size_t)b * NP + (m - 1)) * 2 + 0] = new_q_stats[((size_t)b * NP + (m - 1)) * 2 + 0];
      q_stats[((size_t)b * NP + (m - 1)) * 2 + 1] = new_q_stats[((size_t)b * NP + (m - 1)) * 2 + 1];
    }
    for (int m = N; m < Q; ++m) block_tok[(size_t)b * Q + m] = mask_token;
  }
  free_top[0] = top0 - popped;
  return 0;
}

/* Return a finished slot's pages to the free stack (off the hot path): pages of
 * the listed slots are pushed in slot-list order, logical pages ascending. */
int orc_release(int B, int N, int page_size, int max_pages, int32_t* ctx_len, int32_t* n_ver,
                int32_t* page_table, int32_t* free_stack, int32_t* free_top, uint8_t* active,
                const int32_t* slots, int n_slots) {
  const int Q = 2 * N - 1;
  for (int s = 0; s < n_slots; ++s) {
    const int b = slots[s];
    if (b < 0 || b >= B || !active[b]) continue;
    const int have = (ctx_len[b] + Q + page_size - 1) / page_size;
    for (int i = 0; i < have; ++i) {
      free_stack[free_top[0]++] = page_table[(size_t)b * max_pages + i];
      page_table[(size_t)b * max_pages + i] = -1;
    }
    active[b] = 0;
    ctx_len[b] = 0;
    n_ver[b] = 0;
  }
  return 0;
}
