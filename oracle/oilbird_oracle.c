/*
 * Oilbird semantic-pool retrieval: the CPU oracle.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  Only the tests, the smoke
 * check and the benchmark's CPU-baseline leg may call it.  It shares no code,
 * header, table or helper with the CUDA library and never touches a GPU.
 *
 * What it computes is the plain definition of the semantic draft source's
 * lookup (paper Section 4, paragraphs "(i) Store" and "(ii) Retrieve"):
 *
 *   store     Eq. 1: one record (x_i, h_i) per committed generated position,
 *             the state kept L2-normalised in half precision (bf16 here, the
 *             precision the paper's models run in), grouped into traces.
 *   score     Algorithm 1's scoring line: the cosine of the query state with the
 *             state of every stored position; nothing is approximated.
 *   top-k     Eq. 2: E_t = arg top-k s_i.  Written here as a FULL sort of all
 *             positions by (score descending, position ascending) followed by
 *             taking the first k.  No heap, no selection, no blocking.
 *   firing    Eq. 2 and the matching test of Algorithm 1: theta gates on the best
 *             neighbour only, it is not a filter inside the top-k.
 *   depth     Eq. 3: D(s) = 48 if s >= 0.90; 8 if s >= 0.82; 0 otherwise
 *             (tier table passed in), or a fixed span length (the batched
 *             harness of the appendix copies fixed-length spans).
 *   copy      Eq. 3: gamma_i = x_{i+2 : i+1+D(s_i)}, i.e. D tokens starting
 *             two positions after the neighbour ("offset"), read out of the
 *             trace that holds i and never past that trace's end.
 *
 * Arithmetic: double precision throughout, with exactly the roundings the
 * stored format forces: a key (and the query) is x * (1/||x||) computed in
 * double, rounded once to float and once more to bf16 (round to nearest
 * even); a score is the double-precision sum, in index order, of the exact
 * products of two bf16 vectors, rounded once to float.
 *
 * Every function below is pinned by tests/test_oracle_*.py against closed
 * forms (+-1 Hamming pools), the constants the paper prints, brute force on
 * tiny pools and an independent numpy restatement; nothing is "parity
 * unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------ bf16 -- */

/* bf16 is the upper half of an IEEE-754 binary32. */
float oracle_bf16_to_f32(uint16_t b) {
  uint32_t u = ((uint32_t)b) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return f;
}

/* Round to nearest, ties to even, on the 16 discarded bits. */
uint16_t oracle_f32_to_bf16(float f) {
  uint32_t u;
  memcpy(&u, &f, sizeof u);
  if ((u & 0x7f800000u) == 0x7f800000u && (u & 0x007fffffu) != 0u) {
    return (uint16_t)((u >> 16) | 0x0040u); /* NaN stays NaN (quiet) */
  }
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7fffu + lsb;
  return (uint16_t)(u >> 16);
}

/* ------------------------------------------------------------------ pool -- */

typedef struct {
  int32_t d;
  int64_t n, cap;           /* rows stored / allocated                        */
  uint16_t *key;            /* [n][d] normalised bf16 keys (Eq. 1)            */
  int32_t *tok;             /* [n]    token x_i                               */
  int32_t *trace_id;        /* [n]    which trace holds row i                 */
  int32_t n_traces, cap_traces;
  int64_t *trace_start;     /* [n_traces] first row                           */
  int64_t *trace_end;       /* [n_traces] one past the last row               */
  uint64_t *trace_tag;      /* [n_traces] prompt tag for same-prompt skipping */
  int64_t degenerate_rows;  /* rows stored as zero (zero or non-finite input) */
} oracle_pool;

oracle_pool *oracle_pool_create(int32_t d) {
  if (d <= 0) return NULL;
  oracle_pool *p = (oracle_pool *)calloc(1, sizeof *p);
  if (p) p->d = d;
  return p;
}

void oracle_pool_destroy(oracle_pool *p) {
  if (!p) return;
  free(p->key); free(p->tok); free(p->trace_id);
  free(p->trace_start); free(p->trace_end); free(p->trace_tag);
  free(p);
}

void oracle_pool_reset(oracle_pool *p) {
  p->n = 0; p->n_traces = 0; p->degenerate_rows = 0;
}

int64_t oracle_pool_size(const oracle_pool *p) { return p->n; }
int32_t oracle_pool_num_traces(const oracle_pool *p) { return p->n_traces; }
int64_t oracle_pool_degenerate_rows(const oracle_pool *p) { return p->degenerate_rows; }
const uint16_t *oracle_pool_keys(const oracle_pool *p) { return p->key; }
const int32_t *oracle_pool_tokens(const oracle_pool *p) { return p->tok; }
const int32_t *oracle_pool_trace_ids(const oracle_pool *p) { return p->trace_id; }
const int64_t *oracle_pool_trace_starts(const oracle_pool *p) { return p->trace_start; }
const int64_t *oracle_pool_trace_ends(const oracle_pool *p) { return p->trace_end; }
const uint64_t *oracle_pool_trace_tags(const oracle_pool *p) { return p->trace_tag; }

/*
 * L2-normalise one bf16 vector into bf16 (Section 4 (i): states are stored
 * normalised, in 16-bit precision).  Returns 1 if the input was usable, 0 if it was
 * all zero or held a NaN/Inf, in which case the output is all zero.
 */
int oracle_normalize_bf16(int32_t d, const uint16_t *x, uint16_t *out) {
  double ss = 0.0;
  int finite = 1;
  for (int32_t j = 0; j < d; ++j) {
    double v = (double)oracle_bf16_to_f32(x[j]);
    if (!isfinite(v)) finite = 0;
    ss += v * v;
  }
  double nrm = sqrt(ss);
  int ok = finite && nrm > 0.0 && isfinite(nrm);
  double inv = ok ? 1.0 / nrm : 0.0;
  for (int32_t j = 0; j < d; ++j) {
    if (!ok) { out[j] = 0; continue; }
    double v = (double)oracle_bf16_to_f32(x[j]);
    out[j] = oracle_f32_to_bf16((float)(v * inv));
  }
  return ok;
}

static int grow_rows(oracle_pool *p, int64_t need) {
  if (need <= p->cap) return 0;
  int64_t cap = p->cap ? p->cap : 1024;
  while (cap < need) cap *= 2;
  uint16_t *k = (uint16_t *)realloc(p->key, (size_t)cap * (size_t)p->d * sizeof(uint16_t));
  if (!k) return -1;
  p->key = k;
  int32_t *t = (int32_t *)realloc(p->tok, (size_t)cap * sizeof(int32_t));
  if (!t) return -1;
  p->tok = t;
  int32_t *r = (int32_t *)realloc(p->trace_id, (size_t)cap * sizeof(int32_t));
  if (!r) return -1;
  p->trace_id = r;
  p->cap = cap;
  return 0;
}

static int grow_traces(oracle_pool *p) {
  if (p->n_traces < p->cap_traces) return 0;
  int32_t cap = p->cap_traces ? p->cap_traces * 2 : 64;
  int64_t *s = (int64_t *)realloc(p->trace_start, (size_t)cap * sizeof(int64_t));
  if (!s) return -1;
  p->trace_start = s;
  int64_t *e = (int64_t *)realloc(p->trace_end, (size_t)cap * sizeof(int64_t));
  if (!e) return -1;
  p->trace_end = e;
  uint64_t *g = (uint64_t *)realloc(p->trace_tag, (size_t)cap * sizeof(uint64_t));
  if (!g) return -1;
  p->trace_tag = g;
  p->cap_traces = cap;
  return 0;
}

/*
 * Store (Eq. 1; Algorithm 1's last line): append n records.  new_trace != 0
 * opens a trace carrying `tag`; otherwise the rows extend the newest trace
 * (the tag argument is then ignored).  The very first append always opens a
 * trace.  Returns 0, or -1 when memory runs out.
 */
int oracle_pool_append(oracle_pool *p, const uint16_t *states, const int32_t *tokens,
                       int64_t n, uint64_t tag, int new_trace) {
  if (n < 0) return -1;
  if (n == 0 && !new_trace) return 0;
  if (grow_rows(p, p->n + n)) return -1;
  if (new_trace || p->n_traces == 0) {
    if (grow_traces(p)) return -1;
    p->trace_start[p->n_traces] = p->n;
    p->trace_end[p->n_traces] = p->n;
    p->trace_tag[p->n_traces] = tag;
    p->n_traces += 1;
  }
  int32_t tr = p->n_traces - 1;
  int64_t bad = 0;
#pragma omp parallel for schedule(static) reduction(+ : bad)
  for (int64_t r = 0; r < n; ++r) {   /* rows are independent */
    int64_t row = p->n + r;
    int ok = oracle_normalize_bf16(p->d, states + (size_t)r * p->d, p->key + (size_t)row * p->d);
    if (!ok) bad += 1;
    p->tok[row] = tokens[r];
    p->trace_id[row] = tr;
  }
  p->degenerate_rows += bad;
  p->n += n;
  p->trace_end[tr] = p->n;
  return 0;
}

/* --------------------------------------------------------------- scoring -- */

/*
 * Algorithm 1: s_i = cos(h_t, h_i) for every stored i.  The query is
 * normalised and rounded to bf16 exactly as a key is, so the cosine of the
 * two stored-format unit vectors is their dot product.  Rows of a trace whose
 * tag equals a non-zero exclude_tag score -inf (Section 4 (i): a request never
 * retrieves from a stored trace that has its own prompt).
 * Returns 1 if the query was usable; otherwise every score is -inf and 0 is
 * returned.
 */
int oracle_scores(const oracle_pool *p, const uint16_t *q_raw, uint64_t exclude_tag,
                  float *scores) {
  const int32_t d = p->d;
  uint16_t *qn = (uint16_t *)malloc((size_t)d * sizeof(uint16_t));
  double *qd = (double *)malloc((size_t)d * sizeof(double));
  int finite = 1;
  for (int32_t j = 0; j < d; ++j)
    if (!isfinite(oracle_bf16_to_f32(q_raw[j]))) finite = 0;
  oracle_normalize_bf16(d, q_raw, qn); /* an all-zero query is legal: scores 0 */
  for (int32_t j = 0; j < d; ++j) qd[j] = (double)oracle_bf16_to_f32(qn[j]);
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < p->n; ++i) {
    if (!finite) { scores[i] = -INFINITY; continue; }
    if (exclude_tag != 0 && p->trace_tag[p->trace_id[i]] == exclude_tag) {
      scores[i] = -INFINITY;
      continue;
    }
    const uint16_t *kr = p->key + (size_t)i * d;
    double acc = 0.0;
    for (int32_t j = 0; j < d; ++j) acc += qd[j] * (double)oracle_bf16_to_f32(kr[j]);
    scores[i] = (float)acc;
  }
  free(qn); free(qd);
  return finite;
}

typedef struct { float s; int64_t i; } scored_row;

/* Order of Eq. 2 plus the tie rule: higher score first, lower position first. */
static int cmp_scored(const void *a, const void *b) {
  const scored_row *x = (const scored_row *)a, *y = (const scored_row *)b;
  if (x->s > y->s) return -1;
  if (x->s < y->s) return 1;
  if (x->i < y->i) return -1;
  if (x->i > y->i) return 1;
  return 0;
}

/* Eq. 3's D(s): the first tier (tested in the order given) whose floor s reaches. */
int32_t oracle_depth(float s, int32_t n_tiers, const float *tier_thr, const int32_t *tier_depth) {
  for (int32_t t = 0; t < n_tiers; ++t)
    if (s >= tier_thr[t]) return tier_depth[t];
  return 0;
}

/*
 * Eq. 3's copy for one neighbour: up to `dep` tokens starting `offset` after
 * row idx, clipped at the end of the trace holding idx and at L; the rest of
 * the L slots are filled with -1.  Returns the number of tokens copied.
 */
int32_t oracle_gather_one(const oracle_pool *p, int64_t idx, int32_t dep, int32_t offset,
                          int32_t L, int32_t *out) {
  for (int32_t t = 0; t < L; ++t) out[t] = -1;
  if (idx < 0 || idx >= p->n) return 0;
  int64_t start = idx + offset;
  int64_t end = p->trace_end[p->trace_id[idx]];
  int64_t len = end - start;
  if (len > dep) len = dep;
  if (len > L) len = L;
  if (len < 0) len = 0;
  for (int64_t t = 0; t < len; ++t) out[t] = p->tok[start + t];
  return (int32_t)len;
}

/*
 * One retrieval (Algorithm 1's score / top-k / firing / depth / copy lines)
 * for nq queries.  depth_mode 0 = fixed span of L tokens, 1 = tiered D(s).
 * Outputs (host, caller-owned): idx[nq][k] (-1 where fewer than k rows have a
 * finite score), score[nq][k] (-inf there), fired[nq], cont_len[nq][k],
 * cont_tok[nq][k][L] padded with -1.  all_scores, if not NULL, receives the
 * nq x N score matrix.  Returns 0, or -1 when memory runs out.
 */
int oracle_pool_query(const oracle_pool *p, const uint16_t *q_raw, int32_t nq, int32_t k,
                      float theta, int32_t offset, int32_t depth_mode, int32_t L,
                      int32_t n_tiers, const float *tier_thr, const int32_t *tier_depth,
                      const uint64_t *exclude_tag, int64_t *idx, float *score, int32_t *fired,
                      int32_t *cont_len, int32_t *cont_tok, float *all_scores) {
  const int64_t N = p->n;
  float *s = (float *)malloc((size_t)(N > 0 ? N : 1) * sizeof(float));
  scored_row *order = (scored_row *)malloc((size_t)(N > 0 ? N : 1) * sizeof(scored_row));
  if (!s || !order) { free(s); free(order); return -1; }
  for (int32_t q = 0; q < nq; ++q) {
    oracle_scores(p, q_raw + (size_t)q * p->d, exclude_tag ? exclude_tag[q] : 0, s);
    if (all_scores) memcpy(all_scores + (size_t)q * N, s, (size_t)N * sizeof(float));
    for (int64_t i = 0; i < N; ++i) { order[i].s = s[i]; order[i].i = i; }
    qsort(order, (size_t)N, sizeof(scored_row), cmp_scored);
    for (int32_t j = 0; j < k; ++j) {
      int have = j < N && order[j].s > -INFINITY;
      idx[(size_t)q * k + j] = have ? order[j].i : -1;
      score[(size_t)q * k + j] = have ? order[j].s : -INFINITY;
    }
    int f = (k > 0 && idx[(size_t)q * k] >= 0 && score[(size_t)q * k] >= theta) ? 1 : 0;
    fired[q] = f;
    for (int32_t j = 0; j < k; ++j) {
      int64_t i = idx[(size_t)q * k + j];
      int32_t dep = 0;
      if (f && i >= 0)
        dep = depth_mode == 0 ? L
                              : oracle_depth(score[(size_t)q * k + j], n_tiers, tier_thr, tier_depth);
      cont_len[(size_t)q * k + j] =
          oracle_gather_one(p, i, dep, offset, L, cont_tok + ((size_t)q * k + j) * L);
    }
  }
  free(s); free(order);
  return 0;
}

int32_t oracle_num_threads(void) {
#ifdef _OPENMP
  return (int32_t)omp_get_max_threads();
#else
  return 1;
#endif
}
