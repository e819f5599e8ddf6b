/*
 * The C-ABI from plain C: no Python, no torch.  Builds a tiny pool whose scores are known
 * in closed form (rows and query with entries +-1: s = 1 - 2*Hamming/d exactly in bf16), runs
 * append -> query -> gather through include/oilbird.h with cudaMalloc'ed buffers, and checks
 * neighbours, scores, the firing rule and the continuation (Eq. 1-3).  Prints "ok" and
 * returns 0 on success.
 */
#include <cuda_runtime.h>
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "oilbird.h"

#define CHECK(x) do { int rc_ = (x); if (rc_ != 0) { fprintf(stderr, "%s -> %d (%s) %s\n", #x, rc_, \
    oilbird_strerror(rc_), oilbird_last_cuda_error()); return 1; } } while (0)
#define CU(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { fprintf(stderr, "%s -> %s\n", #x, \
    cudaGetErrorString(e_)); return 1; } } while (0)

enum { D = 256, N = 300, K = 4, L = 3 };
static const uint16_t P1 = 0x3f80, M1 = 0xbf80;      /* +1.0 and -1.0 as bf16 */

int main(void) {
  static uint16_t rows[N][D], q[D];
  static int32_t toks[N];
  /* row i differs from the all-ones query in h(i) leading entries */
  int h[N];
  for (int i = 0; i < N; ++i) {
    h[i] = 40 + (i * 7) % 90;
    toks[i] = 1000 + i;
  }
  h[17] = 0; h[211] = 2; h[5] = 2; h[198] = 3;         /* best: 17; then a tie 5 < 211; then 198 */
  for (int i = 0; i < N; ++i)
    for (int j = 0; j < D; ++j) rows[i][j] = j < h[i] ? M1 : P1;
  for (int j = 0; j < D; ++j) q[j] = P1;

  oilbird_pool_config cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.d = D; cfg.capacity_rows = N; cfg.max_nq = 1; cfg.max_k = K; cfg.device = 0;
  oilbird_pool_t* pool = NULL;
  CHECK(oilbird_pool_create(&pool, &cfg));

  void *d_rows, *d_q; int32_t* d_tok;
  CU(cudaMalloc(&d_rows, sizeof rows)); CU(cudaMalloc(&d_q, sizeof q)); CU(cudaMalloc((void**)&d_tok, sizeof toks));
  CU(cudaMemcpy(d_rows, rows, sizeof rows, cudaMemcpyHostToDevice));
  CU(cudaMemcpy(d_q, q, sizeof q, cudaMemcpyHostToDevice));
  CU(cudaMemcpy(d_tok, toks, sizeof toks, cudaMemcpyHostToDevice));
  /* two traces: rows [0,200) and [200,300) */
  CHECK(oilbird_pool_append(pool, d_rows, d_tok, 200, 11, OILBIRD_NEW_TRACE, NULL));
  CHECK(oilbird_pool_append(pool, (uint16_t*)d_rows + 200 * D, d_tok + 200, 100, 12, OILBIRD_NEW_TRACE, NULL));
  if (oilbird_pool_size(pool) != N || oilbird_pool_num_traces(pool) != 2) return 2;

  oilbird_query_params pr;
  oilbird_query_params_default(&pr);
  pr.k = K; pr.depth_mode = OILBIRD_DEPTH_FIXED; pr.cont_len = L;      /* theta 0.8, offset 2 */
  oilbird_query_out out;
  CU(cudaMalloc((void**)&out.idx, K * 4)); CU(cudaMalloc((void**)&out.score, K * 4));
  CU(cudaMalloc((void**)&out.fired, 4)); CU(cudaMalloc((void**)&out.cont_len, K * 4));
  CU(cudaMalloc((void**)&out.cont_tok, K * L * 4));
  for (int path = OILBIRD_PATH_GEMV; path <= OILBIRD_PATH_TENSOR; ++path) {
    pr.path = path;
    CHECK(oilbird_pool_query(pool, d_q, 1, &pr, &out, NULL));
    oilbird_pool_stats st;
    CHECK(oilbird_pool_status(pool, &st, NULL));
    int32_t idx[K], fired, clen[K], ctok[K][L]; float score[K];
    CU(cudaMemcpy(idx, out.idx, sizeof idx, cudaMemcpyDeviceToHost));
    CU(cudaMemcpy(score, out.score, sizeof score, cudaMemcpyDeviceToHost));
    CU(cudaMemcpy(&fired, out.fired, 4, cudaMemcpyDeviceToHost));
    CU(cudaMemcpy(clen, out.cont_len, sizeof clen, cudaMemcpyDeviceToHost));
    CU(cudaMemcpy(ctok, out.cont_tok, sizeof ctok, cudaMemcpyDeviceToHost));
    const int want_idx[K] = {17, 5, 211, 198};
    const int want_h[K] = {0, 2, 2, 3};
    const int want_len[K] = {L, L, L, 0};          /* row 198 + 2 is the end of its trace */
    for (int j = 0; j < K; ++j) {
      if (idx[j] != want_idx[j]) { fprintf(stderr, "path %d: idx[%d] = %d\n", path, j, idx[j]); return 3; }
      if (score[j] != 1.0f - 2.0f * want_h[j] / D) { fprintf(stderr, "score[%d] = %g\n", j, score[j]); return 4; }
    }
    if (fired != 1) return 5;
    /* row 17: tokens of rows 19, 20, 21, and so on; never past the end of the trace */
    for (int j = 0; j < K; ++j) {
      if (clen[j] != want_len[j]) return 6;
      for (int t = 0; t < L; ++t)
        if (ctok[j][t] != (t < want_len[j] ? 1000 + want_idx[j] + 2 + t : -1)) return 7;
    }
  }
  /* a stored row asked for again is its own best neighbour (row 198 is unique) */
  CHECK(oilbird_pool_query(pool, (uint16_t*)d_rows + 198 * D, 1, &pr, &out, NULL));
  int32_t idx0, clen0;
  CU(cudaMemcpy(&idx0, out.idx, 4, cudaMemcpyDeviceToHost));
  CU(cudaMemcpy(&clen0, out.cont_len, 4, cudaMemcpyDeviceToHost));
  if (idx0 != 198 || clen0 != 0) { fprintf(stderr, "self: idx %d len %d\n", idx0, clen0); return 8; }
  /* host steps in two halves, two in flight: plain host arrays in, plain host arrays out */
  {
    static int32_t h_idx[2][K], h_fired[2], h_len[2][K], h_tok[2][K][L];
    static float h_score[2][K];
    oilbird_query_out ho[2];
    for (int s = 0; s < 2; ++s) {
      ho[s].idx = h_idx[s]; ho[s].score = h_score[s]; ho[s].fired = &h_fired[s];
      ho[s].cont_len = h_len[s]; ho[s].cont_tok = &h_tok[s][0][0];
    }
    pr.path = OILBIRD_PATH_AUTO;
    CHECK(oilbird_pool_step_host_begin(pool, NULL, NULL, 0, 0, 0, q, 1, &pr, 0, NULL));
    CHECK(oilbird_pool_step_host_begin(pool, NULL, NULL, 0, 0, 0, rows[198], 1, &pr, 1, NULL));
    if (oilbird_pool_step_host_begin(pool, NULL, NULL, 0, 0, 0, q, 1, &pr, 0, NULL) != OILBIRD_EINVAL) return 12;
    CHECK(oilbird_pool_step_host_end(pool, 1, &ho[1]));
    CHECK(oilbird_pool_step_host_end(pool, 0, &ho[0]));
    if (oilbird_pool_step_host_end(pool, 0, &ho[0]) != OILBIRD_EINVAL) return 13;
    if (h_idx[0][0] != 17 || h_idx[0][1] != 5 || h_fired[0] != 1 || h_tok[0][0][0] != 1000 + 19) return 14;
    if (h_idx[1][0] != 198 || h_len[1][0] != 0) return 15;
  }
  /* misaligned input is refused, nothing is appended */
  if (oilbird_pool_reset(pool, NULL) != 0) return 9;
  if (oilbird_pool_append(pool, (char*)d_rows + 2, d_tok, 1, 1, OILBIRD_NEW_TRACE, NULL) != OILBIRD_EINVAL) return 10;
  if (oilbird_pool_size(pool) != 0) return 11;
  CHECK(oilbird_pool_destroy(pool));
  printf("ok\n");
  return 0;
}
