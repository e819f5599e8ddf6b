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
 * unpinned".  The 8-bit store (E4M3 section) is pinned against PyTorch's own
 * float8_e4m3fn conversions, the format's constants, a closed form and the
 * quantiser's error bound (tests/test_oracle_q8_pins.py).
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

/* ------------------------------------------------------------------ e4m3 -- */
/*
 * 8-bit keys for the bounded store (the paper's Limitations section names
 * quantisation of the store as future work and fixes no format; the format
 * here is this build's reading and is listed with the other readings).
 *
 * E4M3: 1 sign, 4 exponent (bias 7), 3 mantissa bits, no infinities.
 *   exponent field e in 1..15:  (-1)^s * 2^(e-7) * (1 + m/8)
 *   e == 0 (subnormal):         (-1)^s * 2^-6 * (m/8)
 * Codes 0x7f and 0xff are NaN and are never produced; the largest finite
 * magnitude is code 0x7e = 448.
 */
double oracle_e4m3_decode(uint8_t c) {
  int s = c >> 7, e = (c >> 3) & 15, m = c & 7;
  double v = e ? ldexp(1.0 + m / 8.0, e - 7) : ldexp(m / 8.0, -6);
  if (e == 15 && m == 7) v = NAN;
  return s ? -v : v;
}

/*
 * Nearest E4M3 value, ties to the even code, magnitudes above 448 saturate
 * to 448.  Done by search over the 127 finite magnitudes: plain, not fast.
 */
uint8_t oracle_e4m3_encode(double x) {
  uint8_t sign = signbit(x) ? 0x80 : 0;
  double a = fabs(x);
  if (!(a == a)) return 0;                 /* NaN input: stored as zero        */
  if (a >= 448.0) return (uint8_t)(sign | 0x7e);
  uint8_t best = 0;
  double best_err = a;                     /* code 0 (value 0)                 */
  for (int c = 1; c <= 0x7e; ++c) {
    double err = fabs(oracle_e4m3_decode((uint8_t)c) - a);
    /* codes increase with magnitude, so an equal error is the upper neighbour */
    if (err < best_err || (err == best_err && (c & 1) == 0)) { best = (uint8_t)c; best_err = err; }
  }
  return (uint8_t)(sign | best);
}

/*
 * Quantise one raw bf16 state into E4M3 codes with one fp32 scale per row:
 *   v_j   = x_j / ||x||                      (double)
 *   scale = fp32( max_j |v_j| / 448 )
 *   c_j   = e4m3( v_j / scale )
 * so that v_j ~ scale * decode(c_j) and the largest entry maps to +-448.  A row
 * that is all zero or holds a NaN/Inf is stored as zero codes with scale 0.
 * Returns 1 if the row was usable.
 */
int oracle_quantize_e4m3(int32_t d, const uint16_t *x, uint8_t *codes, float *scale) {
  double ss = 0.0, amax = 0.0;
  int finite = 1;
  for (int32_t j = 0; j < d; ++j) {
    double v = (double)oracle_bf16_to_f32(x[j]);
    if (!isfinite(v)) finite = 0;
    ss += v * v;
    if (fabs(v) > amax) amax = fabs(v);
  }
  double nrm = sqrt(ss);
  int ok = finite && nrm > 0.0 && isfinite(nrm);
  if (!ok) {
    for (int32_t j = 0; j < d; ++j) codes[j] = 0;
    *scale = 0.0f;
    return 0;
  }
  double inv = 1.0 / nrm;
  float sc = (float)(amax * inv / 448.0);
  for (int32_t j = 0; j < d; ++j) {
    double v = (double)oracle_bf16_to_f32(x[j]) * inv;
    codes[j] = oracle_e4m3_encode(v / (double)sc);
  }
  *scale = sc;
  return 1;
}

/* ------------------------------------------------------------------ pool -- */

typedef struct {
  int32_t d;
  int32_t fmt;              /* 0: bf16 keys; 1: E4M3 codes + one scale per row */
  uint8_t *code;            /* fmt 1: [n][d]                                   */
  float *scale;             /* fmt 1: [n]                                      */
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

/* The same store with 8-bit keys (see the E4M3 section above). */
oracle_pool *oracle_pool_create_e4m3(int32_t d) {
  oracle_pool *p = oracle_pool_create(d);
  if (p) p->fmt = 1;
  return p;
}
const uint8_t *oracle_pool_codes(const oracle_pool *p) { return p->code; }
const float *oracle_pool_scales(const oracle_pool *p) { return p->scale; }

void oracle_pool_destroy(oracle_pool *p) {
  if (!p) return;
  free(p->key); free(p->code); free(p->scale); free(p->tok); free(p->trace_id);
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
  if (p->fmt == 0) {
    uint16_t *k = (uint16_t *)realloc(p->key, (size_t)cap * (size_t)p->d * sizeof(uint16_t));
    if (!k) return -1;
    p->key = k;
  } else {
    uint8_t *c = (uint8_t *)realloc(p->code, (size_t)cap * (size_t)p->d);
    if (!c) return -1;
    p->code = c;
    float *sc = (float *)realloc(p->scale, (size_t)cap * sizeof(float));
    if (!sc) return -1;
    p->scale = sc;
  }
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
    int ok = p->fmt == 0
                 ? oracle_normalize_bf16(p->d, states + (size_t)r * p->d, p->key + (size_t)row * p->d)
                 : oracle_quantize_e4m3(p->d, states + (size_t)r * p->d,
                                        p->code + (size_t)row * p->d, p->scale + row);
    if (!ok) bad += 1;
    p->tok[row] = tokens[r];
    p->trace_id[row] = tr;
  }
  p->degenerate_rows += bad;
  p->n += n;
  p->trace_end[tr] = p->n;
  return 0;
}

/*
 * Eviction for a bounded store (the paper's Limitations section names eviction as one way
 * to keep the store bounded and defines no policy; this build's reading: oldest first, by
 * whole traces).  The first n_traces traces and their rows are dropped; what remains is
 * exactly the pool that would have been built from the remaining traces alone: rows and
 * traces are renumbered from zero, order kept.  Returns the number of rows dropped.
 */
int64_t oracle_pool_evict_oldest(oracle_pool *p, int32_t n_traces) {
  if (n_traces <= 0) return 0;
  if (n_traces > p->n_traces) n_traces = p->n_traces;
  if (n_traces == 0) return 0;
  const int64_t drop = p->trace_end[n_traces - 1];
  const int64_t live = p->n - drop;
  const int32_t d = p->d;
  for (int64_t i = 0; i < live; ++i) {
    if (p->fmt == 0) {
      for (int32_t j = 0; j < d; ++j) p->key[(size_t)i * d + j] = p->key[(size_t)(i + drop) * d + j];
    } else {
      for (int32_t j = 0; j < d; ++j) p->code[(size_t)i * d + j] = p->code[(size_t)(i + drop) * d + j];
      p->scale[i] = p->scale[i + drop];
    }
    p->tok[i] = p->tok[i + drop];
    p->trace_id[i] = p->trace_id[i + drop] - n_traces;
  }
  for (int32_t t = 0; t + n_traces < p->n_traces; ++t) {
    p->trace_start[t] = p->trace_start[t + n_traces] - drop;
    p->trace_end[t] = p->trace_end[t + n_traces] - drop;
    p->trace_tag[t] = p->trace_tag[t + n_traces];
  }
  p->n_traces -= n_traces;
  p->n = live;
  return drop;
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
    double acc = 0.0;
    if (p->fmt == 0) {
      const uint16_t *kr = p->key + (size_t)i * d;
      for (int32_t j = 0; j < d; ++j) acc += qd[j] * (double)oracle_bf16_to_f32(kr[j]);
    } else {
      /* 8-bit keys: the query stays bf16; the row's scale multiplies the exact sum */
      const uint8_t *cr = p->code + (size_t)i * d;
      for (int32_t j = 0; j < d; ++j) acc += qd[j] * oracle_e4m3_decode(cr[j]);
      acc *= (double)p->scale[i];
    }
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
 * The granularity ablation's other arm (Section 6, "Retrieval granularity"): the copy depth is
 * assigned by the neighbour's rank instead of its similarity.  The paper names the arm and
 * gives no schedule; reading: neighbour j (best first, j from 0) copies tier_depth[j] tokens
 * for j < n_tiers, and tier_depth[n_tiers - 1] from there on (the paper's table {48, 8}: the
 * best neighbour copies 48 tokens, every other one 8).  No tier: nothing is copied.
 */
int32_t oracle_depth_by_rank(int32_t j, int32_t n_tiers, const int32_t *tier_depth) {
  if (n_tiers <= 0 || j < 0) return 0;
  return tier_depth[j < n_tiers ? j : n_tiers - 1];
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
 * for nq queries.  depth_mode 0 = fixed span of L tokens, 1 = tiered D(s), 2 = by rank.
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
            : depth_mode == 2 ? oracle_depth_by_rank(j, n_tiers, tier_depth)
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

/* ============================================================ recycled pool == */
/*
 * Rejected-branch store (paper Section 4 "(i b) Recycling"; Algorithm 1's
 * recycled-pool line).  A record is keyed by the hidden state in front of a
 * rejected draft token together with that token (the "anchor"), and its value
 * is the short continuation the model endorsed from there (up to six tokens in
 * the paper).  Records live in a ring buffer: once it is full the oldest record
 * is overwritten.  A lookup with the current state and the current anchor token
 * returns at most m records whose anchor token is equal and whose cosine with the
 * query reaches a floor (paper: at most 4, floor 0.8), best first; equal scores
 * list the lower slot first.  Unlike theta of the trace store, the floor here is
 * a filter on every record (the algorithm line states both conditions per record).
 * Same arithmetic as the trace store: keys and query normalised to bf16, score =
 * double-precision dot product rounded once to float.  Written as the plain
 * definition: every slot is visited, all qualifying records are fully sorted.
 */
typedef struct {
  int32_t d, max_rollout;
  int64_t cap, total;        /* slots; records ever appended              */
  uint16_t *key;             /* [cap][d]                                  */
  int32_t *anchor;           /* [cap]                                     */
  int32_t *rollout;          /* [cap][max_rollout], padded with -1        */
} oracle_ring;

oracle_ring *oracle_ring_create(int32_t d, int64_t cap, int32_t max_rollout) {
  if (d <= 0 || cap <= 0 || max_rollout <= 0) return NULL;
  oracle_ring *r = (oracle_ring *)calloc(1, sizeof *r);
  if (!r) return NULL;
  r->d = d; r->cap = cap; r->max_rollout = max_rollout;
  r->key = (uint16_t *)calloc((size_t)cap * d, sizeof(uint16_t));
  r->anchor = (int32_t *)calloc((size_t)cap, sizeof(int32_t));
  r->rollout = (int32_t *)calloc((size_t)cap * max_rollout, sizeof(int32_t));
  if (!r->key || !r->anchor || !r->rollout) {
    free(r->key); free(r->anchor); free(r->rollout); free(r);
    return NULL;
  }
  return r;
}

void oracle_ring_destroy(oracle_ring *r) {
  if (!r) return;
  free(r->key); free(r->anchor); free(r->rollout); free(r);
}

void oracle_ring_reset(oracle_ring *r) { r->total = 0; }
int64_t oracle_ring_size(const oracle_ring *r) { return r->total < r->cap ? r->total : r->cap; }
int64_t oracle_ring_total(const oracle_ring *r) { return r->total; }
const uint16_t *oracle_ring_keys(const oracle_ring *r) { return r->key; }
const int32_t *oracle_ring_anchors(const oracle_ring *r) { return r->anchor; }
const int32_t *oracle_ring_rollouts(const oracle_ring *r) { return r->rollout; }

/* Append n records in order; record i goes to slot (total + i) mod cap. */
void oracle_ring_append(oracle_ring *r, const uint16_t *states, const int32_t *anchors,
                        const int32_t *rollouts, int64_t n) {
  for (int64_t i = 0; i < n; ++i) {
    int64_t slot = (r->total + i) % r->cap;
    oracle_normalize_bf16(r->d, states + (size_t)i * r->d, r->key + (size_t)slot * r->d);
    r->anchor[slot] = anchors[i];
    for (int32_t t = 0; t < r->max_rollout; ++t)
      r->rollout[(size_t)slot * r->max_rollout + t] = rollouts[(size_t)i * r->max_rollout + t];
  }
  r->total += n;
}

/*
 * Lookup for nq (state, anchor) pairs.  Outputs: slot[nq][m] (-1 padded),
 * score[nq][m] (-inf padded), count[nq], rollout[nq][m][max_rollout] (-1 padded),
 * rollout_len[nq][m] (tokens before the first negative entry).
 */
int oracle_ring_query(const oracle_ring *r, const uint16_t *q_raw, const int32_t *q_anchor,
                      int32_t nq, int32_t m, float floor_s, int64_t *slot, float *score,
                      int32_t *count, int32_t *rollout, int32_t *rollout_len) {
  const int64_t n = oracle_ring_size(r);
  const int32_t d = r->d, R = r->max_rollout;
  scored_row *cand = (scored_row *)malloc((size_t)(n > 0 ? n : 1) * sizeof(scored_row));
  uint16_t *qn = (uint16_t *)malloc((size_t)d * sizeof(uint16_t));
  if (!cand || !qn) { free(cand); free(qn); return -1; }
  for (int32_t q = 0; q < nq; ++q) {
    int finite = 1;
    for (int32_t j = 0; j < d; ++j)
      if (!isfinite(oracle_bf16_to_f32(q_raw[(size_t)q * d + j]))) finite = 0;
    oracle_normalize_bf16(d, q_raw + (size_t)q * d, qn);
    int64_t nc = 0;
    for (int64_t i = 0; i < n && finite; ++i) {
      if (r->anchor[i] != q_anchor[q]) continue;          /* anchor token must be equal */
      double acc = 0.0;
      for (int32_t j = 0; j < d; ++j)
        acc += (double)oracle_bf16_to_f32(qn[j]) * (double)oracle_bf16_to_f32(r->key[(size_t)i * d + j]);
      float s = (float)acc;
      if (s >= floor_s) { cand[nc].s = s; cand[nc].i = i; ++nc; }   /* cosine floor */
    }
    qsort(cand, (size_t)nc, sizeof(scored_row), cmp_scored);
    count[q] = (int32_t)(nc < m ? nc : m);
    for (int32_t j = 0; j < m; ++j) {
      int have = j < nc;
      slot[(size_t)q * m + j] = have ? cand[j].i : -1;
      score[(size_t)q * m + j] = have ? cand[j].s : -INFINITY;
      int32_t len = 0, open = 1;
      for (int32_t t = 0; t < R; ++t) {
        int32_t tok = have ? r->rollout[(size_t)cand[j].i * R + t] : -1;
        if (tok < 0) open = 0;
        if (open) ++len;
        rollout[((size_t)q * m + j) * R + t] = open ? tok : -1;
      }
      rollout_len[(size_t)q * m + j] = len;
    }
  }
  free(cand); free(qn);
  return 0;
}
