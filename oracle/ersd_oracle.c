/*
 * ersd_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, fp64 CPU statement of exponential-race speculative decoding
 * (ERSD).  Only the test-suite, the smoke check and the benchmark's CPU
 * baseline may call it; the CUDA library never does and shares no source
 * with it.
 *
 * What the paper fixes and this file writes out:
 *   - Section 3 ("Exponential Races"): every token i of the alphabet gets an
 *     independent e_i ~ Exp(1); the winner argmin_i e_i / p_i is a sample of P.
 *     Using the SAME e for the draft law Q and the target law P couples the
 *     two winners.
 *   - Algorithm 2 (simple ERSD, k = 1) and its sequence extension (Section 3,
 *     paragraph after Algorithm 2's description): one race per drafted
 *     position, accept in order until the first disagreement, then emit the
 *     target winner of that position.
 *   - Algorithm 5 (tree ERSD, Appendix A): child number r of a node is the
 *     r-th arrival of that node's race under Q; verification walks down while
 *     the P-winner of the current node's race is one of its children.
 *
 * What the paper leaves open and this build fixes (the readings are listed
 * in the design notes): p = softmax(logit / T); the race is evaluated in log
 * form key_i = ln e_i - logit_i / T (same argmin, no softmax); the e_i come
 * from Philox4x32-10 (Salmon et al., SC'11) keyed by the sequence's 64-bit
 * seed with counter (i >> 2, position, sequence id, 0), token i taking
 * output word i & 3, mapped by w = (x + 0.5) 2^-32, e = -log1p(-w); exact
 * key ties go to the lowest token id; NaN logits count as -inf; a row with no
 * token of positive probability yields token -1; T == 0 means greedy
 * (key = -logit, no randomness).
 *
 * Parity pins live in tests/test_oracle_*.py.  Unpinned: the joint law of
 * (draft winner, target winner) off the diagonal (the paper gives no closed
 * form for it) -- "parity unpinned" for that joint law only; its marginals
 * and its diagonal are pinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_F32 0
#define ORACLE_BF16 1

/* ------------------------------------------------------------------ */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw 2011), written from the   */
/* published round function: two 32x32->64 products, a word shuffle    */
/* with the key xored in, Weyl key schedule.                           */
/* ------------------------------------------------------------------ */
void ersd_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2],
                               uint32_t out[4]) {
  const uint64_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
  const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    uint64_t p0 = M0 * (uint64_t)c0;
    uint64_t p1 = M1 * (uint64_t)c2;
    uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
    uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
    uint32_t n0 = hi1 ^ c1 ^ k0;
    uint32_t n1 = lo1;
    uint32_t n2 = hi0 ^ c3 ^ k1;
    uint32_t n3 = lo0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += W0; k1 += W1;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* 32 random bits -> Exp(1) by inversion of the CDF 1 - exp(-e) at the
 * mid-point uniform w = (x + 1/2) / 2^32 in (0, 1).  (Section 3: e_i ~ Exp(1);
 * the generator is this build's choice.) */
double ersd_oracle_exp_variate(uint32_t x) {
  double w = ((double)x + 0.5) * (1.0 / 4294967296.0);
  return -log1p(-w);
}

/* The 32-bit word that belongs to token i in the race of (seed, seq, pos). */
uint32_t ersd_oracle_token_word(uint64_t seed, uint32_t seq_id,
                                uint32_t position, uint32_t i) {
  uint32_t ctr[4] = {i >> 2, position, seq_id, 0u};
  uint32_t key[2] = {(uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)};
  uint32_t out[4];
  ersd_oracle_philox4x32_10(ctr, key, out);
  return out[i & 3u];
}

static double logit_at(const void* row, int dtype, int64_t i) {
  double z;
  if (dtype == ORACLE_BF16) {
    uint32_t bits = (uint32_t)((const uint16_t*)row)[i] << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    z = (double)f;
  } else {
    z = (double)((const float*)row)[i];
  }
  if (isnan(z)) z = -INFINITY;
  return z;
}

/* Race keys of one logit row, log form:  key_i = ln e_i - z_i / T.
 * Since ln(e_i / p_i) = ln e_i - z_i/T + ln Z with Z free of i, the ordering
 * of the keys is the ordering of the arrival times e_i / p_i (Section 3). */
void ersd_oracle_row_keys(const void* row, int dtype, int V, double T,
                          uint64_t seed, uint32_t seq_id, uint32_t position,
                          double* keys) {
  for (int i = 0; i < V; ++i) {
    double z = logit_at(row, dtype, i);
    if (T == 0.0) {
      keys[i] = -z;
    } else {
      double e = ersd_oracle_exp_variate(
          ersd_oracle_token_word(seed, seq_id, position, (uint32_t)i));
      keys[i] = log(e) - z / T;
    }
  }
}

/* Arrival times in the paper's own form, t_i = e_i / p_i with
 * p = softmax(z / T) (max subtracted).  Tokens with p_i == 0 never arrive
 * (t_i = +inf).  Only meaningful for T > 0 and rows without +inf logits. */
void ersd_oracle_row_times_def(const void* row, int dtype, int V, double T,
                               uint64_t seed, uint32_t seq_id,
                               uint32_t position, double* times) {
  double zmax = -INFINITY, Z = 0.0;
  for (int i = 0; i < V; ++i) {
    double s = logit_at(row, dtype, i) / T;
    if (s > zmax) zmax = s;
  }
  for (int i = 0; i < V; ++i) Z += exp(logit_at(row, dtype, i) / T - zmax);
  for (int i = 0; i < V; ++i) {
    double p = exp(logit_at(row, dtype, i) / T - zmax) / Z;
    double e = ersd_oracle_exp_variate(
        ersd_oracle_token_word(seed, seq_id, position, (uint32_t)i));
    times[i] = (p > 0.0) ? e / p : INFINITY;
  }
}

/* The first c arrivals of a race given its keys (or times): ascending key,
 * equal keys by ascending token id; tokens whose key is +inf never arrive.
 * tok[r] = -1 and key[r] = +inf when fewer than r+1 tokens arrive.  key has
 * c + 1 slots: the last one is the key of the next arrival after the c-th,
 * which is what a near-tie check of the c-th arrival needs. */
void ersd_oracle_first_arrivals(const double* keys, int V, int c, int32_t* tok,
                                double* key) {
  double last_key = -INFINITY;
  int32_t last_idx = -1;
  int have_last = 0;
  for (int r = 0; r <= c; ++r) {
    double best = INFINITY;
    int32_t best_idx = -1;
    for (int i = 0; i < V; ++i) {
      double ki = keys[i];
      if (!(ki < INFINITY)) continue;
      if (have_last) {
        /* only tokens strictly after the previous arrival in (key, id) order */
        if (ki < last_key || (ki == last_key && i <= last_idx)) continue;
      }
      if (best_idx < 0 || ki < best) {
        best = ki;
        best_idx = i;
      }
    }
    if (r < c) tok[r] = best_idx;
    key[r] = (best_idx >= 0) ? best : INFINITY;
    if (best_idx < 0) {
      for (int q = r + 1; q <= c; ++q) {
        if (q < c) tok[q] = -1;
        key[q] = INFINITY;
      }
      return;
    }
    last_key = best;
    last_idx = best_idx;
    have_last = 1;
  }
}

static double temp_of(float T, const float* temps, int64_t sb, int64_t sr,
                      int b, int r) {
  return temps ? (double)temps[(int64_t)b * sb + (int64_t)r * sr] : (double)T;
}

static const void* row_ptr(const void* base, int dtype, int64_t off_elems) {
  size_t es = (dtype == ORACLE_BF16) ? 2u : 4u;
  return (const char*)base + (size_t)off_elems * es;
}

/* Race sampling: for every (b, r) the first c arrivals of the race of
 * position pos_offsets[b] + r under the law of logits[b, r, :].
 * out_tok [B, R, c], out_key [B, R, c + 1] (see first_arrivals).
 * Strides are in elements and may be 0 (the same row for every b or r). */
void ersd_oracle_race_sample(const void* logits, int dtype, int64_t stride_b,
                             int64_t stride_r, const uint64_t* seeds,
                             const uint32_t* seq_ids,
                             const uint32_t* pos_offsets, int B, int R, int V,
                             float T, const float* temps, int64_t temp_sb,
                             int64_t temp_sr, int c, int32_t* out_tok,
                             double* out_key) {
  int64_t units = (int64_t)B * R;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t u = 0; u < units; ++u) {
    int b = (int)(u / R), r = (int)(u % R);
    double* keys = (double*)malloc(sizeof(double) * (size_t)(V > 0 ? V : 1));
    uint32_t seq = seq_ids ? seq_ids[b] : (uint32_t)b;
    uint32_t pos = (pos_offsets ? pos_offsets[b] : 0u) + (uint32_t)r;
    const void* row = row_ptr(logits, dtype, b * stride_b + r * stride_r);
    ersd_oracle_row_keys(row, dtype, V, temp_of(T, temps, temp_sb, temp_sr, b, r),
                         seeds[b], seq, pos, keys);
    ersd_oracle_first_arrivals(keys, V, c, out_tok + u * c,
                               out_key + u * (c + 1));
    free(keys);
  }
}

/* Same, with the paper's t = e / softmax form (small V only). */
void ersd_oracle_race_sample_def(const void* logits, int dtype,
                                 int64_t stride_b, int64_t stride_r,
                                 const uint64_t* seeds, int B, int R, int V,
                                 float T, int c, int32_t* out_tok,
                                 double* out_time) {
  int64_t units = (int64_t)B * R;
  for (int64_t u = 0; u < units; ++u) {
    int b = (int)(u / R), r = (int)(u % R);
    double* t = (double*)malloc(sizeof(double) * (size_t)(V > 0 ? V : 1));
    const void* row = row_ptr(logits, dtype, b * stride_b + r * stride_r);
    ersd_oracle_row_times_def(row, dtype, V, (double)T, seeds[b], (uint32_t)b,
                              (uint32_t)r, t);
    ersd_oracle_first_arrivals(t, V, c, out_tok + u * c, out_time + u * (c + 1));
    free(t);
  }
}

/* Sequence ERSD (Algorithm 2 extended to k drafted positions).
 *   draft_tok[b, j]  = winner of race (b, j) under the draft row j,   j < k
 *   target_tok[b, j] = winner of the SAME race under the target row j, j <= k
 *   L = first j < k with draft_tok != target_tok (or a missing winner), else k
 *   out_tokens[b, 0..L] = target_tok[b, 0..L], the rest -1; accept_len[b] = L.
 * draft_key / target_key hold (winner key, runner-up key) per row. */
void ersd_oracle_verify(const void* target, const void* draft, int dtype,
                        int64_t ld_target, int64_t ld_draft,
                        const uint64_t* seeds, const uint32_t* seq_ids,
                        const uint32_t* pos_offsets, int B, int k, int V,
                        float T, const float* temps, int64_t temp_sb,
                        int64_t temp_sr, int32_t* out_tokens,
                        int32_t* out_accept_len, int32_t* draft_tok,
                        int32_t* target_tok, double* draft_key,
                        double* target_key) {
  int rows = k + 1;
  int64_t units = (int64_t)B * rows;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t u = 0; u < units; ++u) {
    int b = (int)(u / rows), j = (int)(u % rows);
    double* keys = (double*)malloc(sizeof(double) * (size_t)(V > 0 ? V : 1));
    uint32_t seq = seq_ids ? seq_ids[b] : (uint32_t)b;
    uint32_t pos = (pos_offsets ? pos_offsets[b] : 0u) + (uint32_t)j;
    double Tj = temp_of(T, temps, temp_sb, temp_sr, b, j);
    const void* prow =
        row_ptr(target, dtype, ((int64_t)b * rows + j) * ld_target);
    ersd_oracle_row_keys(prow, dtype, V, Tj, seeds[b], seq, pos, keys);
    ersd_oracle_first_arrivals(keys, V, 1, target_tok + u, target_key + 2 * u);
    if (j < k) {
      int64_t d = (int64_t)b * k + j;
      const void* qrow = row_ptr(draft, dtype, d * ld_draft);
      ersd_oracle_row_keys(qrow, dtype, V, Tj, seeds[b], seq, pos, keys);
      ersd_oracle_first_arrivals(keys, V, 1, draft_tok + d, draft_key + 2 * d);
    }
    free(keys);
  }
  for (int b = 0; b < B; ++b) {
    const int32_t* tt = target_tok + (int64_t)b * rows;
    const int32_t* dt = draft_tok + (int64_t)b * k;
    int L = 0;
    while (L < k && tt[L] >= 0 && dt[L] == tt[L]) ++L;
    for (int j = 0; j < rows; ++j)
      out_tokens[(int64_t)b * rows + j] = (j <= L) ? tt[j] : -1;
    out_accept_len[b] = L;
  }
}

/* Tree ERSD (Algorithm 5).  Nodes 0..N, node 0 the root, parent[n] < n.
 * Siblings are ordered by node id; the sibling of rank r (0-based) carries
 * the (r+1)-th arrival of its parent's race under the parent's draft row.
 * Node n's race is the race of position pos_offsets[b] + n.
 *   arrivals[b, n, 0..max_c)  first #children(n) arrivals under draft row n
 *   target_tok[b, n]          winner of node n's race under target row n
 * Walk: cur = root; emit target_tok[cur]; move to the child whose drafted
 * token equals it; stop when there is none.
 *   out_tokens [B, D+1], out_path [B, D+1] (node ids, -1 padded),
 *   out_accept_len[b] = number of drafted tokens accepted (emitted - 1).
 * arrival_key [B, N+1, max_c + 1], target_key [B, N+1, 2]. */
void ersd_oracle_verify_tree(const void* target, const void* draft, int dtype,
                             int64_t ld_target, int64_t ld_draft,
                             const int32_t* parent, const uint64_t* seeds,
                             const uint32_t* seq_ids,
                             const uint32_t* pos_offsets, int B, int N, int V,
                             float T, const float* temps, int64_t temp_sb,
                             int64_t temp_sr, int D, int max_c,
                             int32_t* out_tokens, int32_t* out_accept_len,
                             int32_t* out_path, int32_t* arrivals,
                             int32_t* target_tok, double* arrival_key,
                             double* target_key) {
  int nodes = N + 1;
  int* nchild = (int*)calloc((size_t)nodes, sizeof(int));
  int* rank = (int*)calloc((size_t)nodes, sizeof(int));
  for (int n = 1; n < nodes; ++n) rank[n] = nchild[parent[n]]++;
  int64_t units = (int64_t)B * nodes;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t u = 0; u < units; ++u) {
    int b = (int)(u / nodes), n = (int)(u % nodes);
    double* keys = (double*)malloc(sizeof(double) * (size_t)(V > 0 ? V : 1));
    uint32_t seq = seq_ids ? seq_ids[b] : (uint32_t)b;
    uint32_t pos = (pos_offsets ? pos_offsets[b] : 0u) + (uint32_t)n;
    double Tn = temp_of(T, temps, temp_sb, temp_sr, b, n);
    const void* prow = row_ptr(target, dtype, u * ld_target);
    ersd_oracle_row_keys(prow, dtype, V, Tn, seeds[b], seq, pos, keys);
    ersd_oracle_first_arrivals(keys, V, 1, target_tok + u, target_key + 2 * u);
    int32_t* arr = arrivals + u * max_c;
    double* akey = arrival_key + u * (max_c + 1);
    for (int r = 0; r < max_c; ++r) arr[r] = -1;
    for (int r = 0; r <= max_c; ++r) akey[r] = INFINITY;
    if (nchild[n] > 0) { /* leaves have no draft row (never read) */
      const void* qrow = row_ptr(draft, dtype, u * ld_draft);
      ersd_oracle_row_keys(qrow, dtype, V, Tn, seeds[b], seq, pos, keys);
      int32_t* tmp_tok = (int32_t*)malloc(sizeof(int32_t) * (size_t)nchild[n]);
      double* tmp_key = (double*)malloc(sizeof(double) * (size_t)(nchild[n] + 1));
      ersd_oracle_first_arrivals(keys, V, nchild[n], tmp_tok, tmp_key);
      for (int r = 0; r < nchild[n]; ++r) arr[r] = tmp_tok[r];
      for (int r = 0; r <= nchild[n]; ++r) akey[r] = tmp_key[r];
      free(tmp_tok);
      free(tmp_key);
    }
    free(keys);
  }
  for (int b = 0; b < B; ++b) {
    int32_t* y = out_tokens + (int64_t)b * (D + 1);
    int32_t* path = out_path + (int64_t)b * (D + 1);
    for (int d = 0; d <= D; ++d) { y[d] = -1; path[d] = -1; }
    int cur = 0, depth = 0;
    for (;;) {
      int32_t w = target_tok[(int64_t)b * nodes + cur];
      y[depth] = w;
      path[depth] = cur;
      int next = -1;
      if (w >= 0) {
        for (int m = cur + 1; m < nodes; ++m) {
          if (parent[m] != cur) continue;
          if (arrivals[((int64_t)b * nodes + cur) * max_c + rank[m]] == w) {
            next = m;
            break;
          }
        }
      }
      if (next < 0) break;
      cur = next;
      ++depth;
    }
    out_accept_len[b] = depth;
  }
  free(nchild);
  free(rank);
}

int ersd_oracle_max_threads(void) {
#ifdef _OPENMP
  extern int omp_get_max_threads(void);
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ================================================================== */
/* Greedy speculative decoding (GSD): Algorithm 1 (Section 2) and its  */
/* tree form, Algorithm 4 (Appendix A).  The comparison verifier of    */
/* the paper: a ratio test per drafted token and, on rejection, a      */
/* sample of the residual law max(P - Q, 0) / sum.                      */
/*                                                                      */
/* What the paper leaves open and this build fixes: the uniform of a    */
/* ratio test is word 0 of Philox4x32-10 with counter (child rank,      */
/* node or position, sequence id, 1), u = (x + 1/2) 2^-32; the token    */
/* that ends the call (residual sample, or the sample of the last       */
/* target row when everything was accepted) is the winner of an         */
/* exponential race (exact by Section 3) whose variables come from      */
/* counter (i >> 2, node or position, sequence id, 2) -- streams        */
/* separate from the one that drafting uses (last counter word 0), as   */
/* Algorithm 1 needs the residual sample independent of the draft.      */
/* Algorithm 4 is garbled in two places (the tested token is typeset    */
/* without its child index, and an empty loop follows the inner while): */
/* the reading taken is the one of Section 2's text -- at each vertex    */
/* the children are tried in order, each rejection replaces the target  */
/* law by its normalised residual against the current draft law and     */
/* removes the rejected token from the draft law (sampling without      */
/* replacement), an acceptance moves to that child.                     */
/* ================================================================== */

static double gsd_uniform(uint64_t seed, uint32_t seq_id, uint32_t node, uint32_t rank) {
  uint32_t ctr[4] = {rank, node, seq_id, 1u};
  uint32_t key[2] = {(uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)};
  uint32_t out[4];
  ersd_oracle_philox4x32_10(ctr, key, out);
  return ((double)out[0] + 0.5) * (1.0 / 4294967296.0);
}

double ersd_oracle_gsd_uniform(uint64_t seed, uint32_t seq_id, uint32_t node, uint32_t rank) {
  return gsd_uniform(seed, seq_id, node, rank);
}

static double gsd_race_variate(uint64_t seed, uint32_t seq_id, uint32_t node, uint32_t i) {
  uint32_t ctr[4] = {i >> 2, node, seq_id, 2u};
  uint32_t key[2] = {(uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)};
  uint32_t out[4];
  ersd_oracle_philox4x32_10(ctr, key, out);
  return ersd_oracle_exp_variate(out[i & 3u]);
}

/* p = softmax(z / T) in double precision, maximum subtracted. */
static void softmax_row(const void* row, int dtype, int V, double T, double* p) {
  double zmax = -INFINITY, Z = 0.0;
  for (int i = 0; i < V; ++i) {
    double s = logit_at(row, dtype, i) / T;
    if (s > zmax) zmax = s;
  }
  for (int i = 0; i < V; ++i) {
    p[i] = exp(logit_at(row, dtype, i) / T - zmax);
    Z += p[i];
  }
  for (int i = 0; i < V; ++i) p[i] /= Z;
}

/* Winner of the exponential race over non-negative weights w (argmin e_i / w_i over w_i > 0,
 * ties to the lowest id), with the GSD race stream of `node`; -1 if no weight is positive.
 * times[0], times[1] receive the winner's and the runner-up's arrival time. */
static int32_t gsd_race(const double* w, int V, uint64_t seed, uint32_t seq_id, uint32_t node,
                        double* times) {
  double best = INFINITY, second = INFINITY;
  int32_t arg = -1;
  for (int i = 0; i < V; ++i) {
    if (!(w[i] > 0.0)) continue;
    double t = gsd_race_variate(seed, seq_id, node, (uint32_t)i) / w[i];
    if (t < best) {
      second = best;
      best = t;
      arg = i;
    } else if (t < second) {
      second = t;
    }
  }
  if (times) {
    times[0] = best;
    times[1] = second;
  }
  return arg;
}

/* Sequence GSD (Algorithm 1, applied position by position as Section 2 describes: drafted
 * tokens are verified in order until the first rejection).
 *   draft_tok[b, j]   the token drafted at position j (a sample of draft row j, made earlier)
 *   accept position j iff P_j(x) / Q_j(x) > u_j; at the first rejection emit a sample of
 *   max(P_j - Q_j, 0) / sum and stop; after k acceptances emit a sample of target row k.
 *   out_tokens [B, k+1] (-1 padded), out_accept_len [B];
 *   ratio, unif [B, k]: the tested ratio and uniform of every position that was tested (NaN
 *   elsewhere); last_times [B, 2]: arrival times of the final race's winner and runner-up. */
void ersd_oracle_gsd_verify(const void* target, const void* draft, const int32_t* draft_tok,
                            int dtype, const uint64_t* seeds, const uint32_t* seq_ids,
                            const uint32_t* pos_offsets, int B, int k, int V, float T,
                            const float* temps, int64_t temp_sb, int64_t temp_sr,
                            int32_t* out_tokens, int32_t* out_accept_len, double* ratio,
                            double* unif, double* last_times) {
  int rows = k + 1;
#pragma omp parallel for schedule(dynamic, 1)
  for (int b = 0; b < B; ++b) {
    double* p = (double*)malloc(sizeof(double) * (size_t)V);
    double* q = (double*)malloc(sizeof(double) * (size_t)V);
    uint32_t seq = seq_ids ? seq_ids[b] : (uint32_t)b;
    uint32_t pos0 = pos_offsets ? pos_offsets[b] : 0u;
    int32_t* y = out_tokens + (int64_t)b * rows;
    for (int j = 0; j < rows; ++j) y[j] = -1;
    for (int j = 0; j < k; ++j) {
      ratio[(int64_t)b * k + j] = NAN;
      unif[(int64_t)b * k + j] = NAN;
    }
    int L = 0, done = 0;
    for (int j = 0; j < k && !done; ++j) {
      double Tj = temp_of(T, temps, temp_sb, temp_sr, b, j);
      softmax_row(row_ptr(target, dtype, ((int64_t)b * rows + j) * V), dtype, V, Tj, p);
      softmax_row(row_ptr(draft, dtype, ((int64_t)b * k + j) * V), dtype, V, Tj, q);
      int32_t x = draft_tok[(int64_t)b * k + j];
      double u = gsd_uniform(seeds[b], seq, pos0 + (uint32_t)j, 0u);
      double r = (x >= 0 && x < V) ? p[x] / q[x] : 0.0; /* 0/0: a token neither law can emit is rejected */
      if (!(r == r)) r = 0.0;
      ratio[(int64_t)b * k + j] = r;
      unif[(int64_t)b * k + j] = u;
      if (r > u) {
        y[j] = x;
        ++L;
      } else {
        for (int i = 0; i < V; ++i) p[i] = (p[i] > q[i]) ? p[i] - q[i] : 0.0; /* residual, unnormalised: the race is scale free */
        y[j] = gsd_race(p, V, seeds[b], seq, pos0 + (uint32_t)j, last_times + 2 * (int64_t)b);
        done = 1;
      }
    }
    if (!done) {
      double Tk = temp_of(T, temps, temp_sb, temp_sr, b, k);
      softmax_row(row_ptr(target, dtype, ((int64_t)b * rows + k) * V), dtype, V, Tk, p);
      y[k] = gsd_race(p, V, seeds[b], seq, pos0 + (uint32_t)k, last_times + 2 * (int64_t)b);
    }
    out_accept_len[b] = L;
    free(p);
    free(q);
  }
}

/* Tree GSD (Algorithm 4).  Nodes 0..N, node 0 the root, parent[n] < n, siblings ordered by node
 * id; draft_tok[b, n] is the token drafted at node n (node 0: unused), siblings drafted without
 * replacement from their parent's draft row.  Walk from the root: try the current node's
 * children in order -- child of rank i is accepted iff P_t(x) / Q_d(x) > u(node, i), where after
 * every rejection P_t <- max(P_t - Q_d, 0) / sum and Q_d <- Q_d with the rejected token removed,
 * renormalised -- move to an accepted child; when no child is accepted (or there is none) emit
 * a sample of the current P_t and stop.
 *   out_tokens [B, D+1] (-1 padded), out_accept_len [B], out_path [B, D+1] (node ids). */
void ersd_oracle_gsd_verify_tree(const void* target, const void* draft, const int32_t* draft_tok,
                                 int dtype, const int32_t* parent, const uint64_t* seeds,
                                 const uint32_t* seq_ids, const uint32_t* pos_offsets, int B, int N,
                                 int V, float T, const float* temps, int64_t temp_sb,
                                 int64_t temp_sr, int D, int32_t* out_tokens,
                                 int32_t* out_accept_len, int32_t* out_path, double* last_times) {
  int nodes = N + 1;
#pragma omp parallel for schedule(dynamic, 1)
  for (int b = 0; b < B; ++b) {
    double* p = (double*)malloc(sizeof(double) * (size_t)V);
    double* q = (double*)malloc(sizeof(double) * (size_t)V);
    uint32_t seq = seq_ids ? seq_ids[b] : (uint32_t)b;
    uint32_t pos0 = pos_offsets ? pos_offsets[b] : 0u;
    int32_t* y = out_tokens + (int64_t)b * (D + 1);
    int32_t* path = out_path + (int64_t)b * (D + 1);
    for (int d = 0; d <= D; ++d) {
      y[d] = -1;
      path[d] = -1;
    }
    int cur = 0, depth = 0;
    for (;;) {
      double Tn = temp_of(T, temps, temp_sb, temp_sr, b, cur);
      softmax_row(row_ptr(target, dtype, ((int64_t)b * nodes + cur) * V), dtype, V, Tn, p);
      int have_q = 0, next = -1;
      uint32_t rank = 0;
      for (int m = cur + 1; m < nodes && next < 0; ++m) {
        if (parent[m] != cur) continue;
        if (!have_q) {
          softmax_row(row_ptr(draft, dtype, ((int64_t)b * nodes + cur) * V), dtype, V, Tn, q);
          have_q = 1;
        }
        int32_t x = draft_tok[(int64_t)b * nodes + m];
        double u = gsd_uniform(seeds[b], seq, pos0 + (uint32_t)cur, rank);
        double r = (x >= 0 && x < V) ? p[x] / q[x] : 0.0;
        if (!(r == r)) r = 0.0;
        if (r > u) {
          next = m;
          y[depth] = x;
        } else {
          double sp = 0.0, sq = 0.0;
          for (int i = 0; i < V; ++i) {
            p[i] = (p[i] > q[i]) ? p[i] - q[i] : 0.0;
            sp += p[i];
          }
          if (sp > 0.0)
            for (int i = 0; i < V; ++i) p[i] /= sp;
          if (x >= 0 && x < V) q[x] = 0.0;
          for (int i = 0; i < V; ++i) sq += q[i];
          if (sq > 0.0)
            for (int i = 0; i < V; ++i) q[i] /= sq;
        }
        ++rank;
      }
      path[depth] = cur;
      if (next < 0) {
        y[depth] = gsd_race(p, V, seeds[b], seq, pos0 + (uint32_t)cur, last_times + 2 * (int64_t)b);
        break;
      }
      cur = next;
      ++depth;
    }
    out_accept_len[b] = depth;
    free(p);
    free(q);
  }
}
