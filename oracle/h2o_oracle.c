/*
 * H2O (Heavy-Hitter Oracle) eviction policy — plain fp64 CPU oracle.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, by-the-definition restatement
 * of the method that the CUDA path is checked against.  It shares no code with
 * the CUDA path and must never be called from it.  Only the tests, the smoke
 * check and the benchmark's CPU-baseline leg may use it.
 *
 * What it follows (paper section / algorithm):
 *   - Attention of token i over a kept set S: o_i = D_i^{-1} exp(Q_i K_S^T),
 *     evicted tokens absent from numerator and normaliser (Definition 2.2, "generative
 *     process with eviction policy"; Appendix D.5 "approximate version").
 *   - With S = [i] this is ordinary causal attention (Definition 2.2, last bullet;
 *     Appendix D "generative process with full knowledge").
 *   - Accumulated score o~_i = o~_{i-1} + o_i and victim
 *     u = argmax_v F_score(G_i \ {v}), F_score(T) = h(sum_{s in T} o~_s)
 *     (Algorithm 2, formal version of Algorithm 1).  For increasing h the argmax is
 *     the candidate with the smallest accumulated score; the tests brute-force the
 *     literal argmax to pin that.
 *   - Budget split into heavy hitters and the most recent tokens; prefill keeps
 *     K heavy + K recent (all if the prompt is shorter); eviction is skipped
 *     while the cache is not full (Appendix A, system details and pseudocode).
 *
 * Readings taken where the paper leaves a choice:
 *   - token t attends to the kept set plus itself, then one entry is evicted;
 *   - scores are accumulated at every step, also while the cache is filling, and
 *     the prompt's column sums are carried into decoding;
 *   - after step t the protected window is positions t-r+1..t, so eviction
 *     candidates are the entries with pos <= t - r;
 *   - total order for eviction: smaller accumulated score first, equal scores
 *     broken by lower token position;
 *   - logits are multiplied by an explicit softmax scale c.
 *
 * Parity pins: every function here is pinned by tests/test_oracle_pins.py
 * (closed forms for uniform attention, brute force of the literal argmax, textbook
 * causal / sliding-window attention as special cases, explicit column sums).
 * The paper prints no worked numeric example, so no stored golden values exist.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* <a, b> over d elements, inputs widened to double, summed in index order. */
static double dot_fd(const float* a, const float* b, long d) {
  double s = 0.0;
  for (long c = 0; c < d; ++c) s += (double)a[c] * (double)b[c];
  return s;
}

int h2o_oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/*
 * Sparse attention patterns combined with the heavy hitters (the table of Section 5.1 that lists the strided
 * and fixed Sparse Transformer patterns with and without H2).  The paper reports the combination but gives no
 * formula; the reading taken here: the cache keeps exactly what it keeps without a pattern (k heavy hitters by
 * accumulated score, the r most recent positions); the pattern decides which entries of the RECENT region a
 * query attends.  For the query at position t and a key at position p:
 *   p == t          : attended (the token itself);
 *   p <= t - r      : attended (older than the window: a heavy hitter, or the candidate that has just left it);
 *   t - r < p < t   : attended iff the pattern allows (p, t):
 *       kind 1, strided(l, w): t - p < w (local) or (t - p) mod l == 0 (every l-th position back);
 *       kind 2, fixed(l, c)  : floor(p / l) == floor(t / l) (same block) or p mod l >= l - c (summary columns).
 * An entry that is not attended is absent from numerator and normaliser of that row and receives no score from
 * it.  "Without H2" is k = 0.  kind 0 = no pattern (everything in the window attended).
 */
static int g_mask_kind = 0;
static long g_mask_a = 1, g_mask_b = 1;
int h2o_oracle_set_mask(int kind, long a, long b) {
  if (kind < 0 || kind > 2) return -1;
  if (kind != 0 && (a < 1 || b < 0)) return -1;
  if (kind == 2 && b > a) return -1;
  g_mask_kind = kind;
  g_mask_a = a;
  g_mask_b = b;
  return 0;
}
static int attended(long p, long t, long r) {
  if (p == t || p <= t - r || g_mask_kind == 0) return 1;
  if (g_mask_kind == 1) return (t - p) < g_mask_b || (t - p) % g_mask_a == 0;
  return p / g_mask_a == t / g_mask_a || p % g_mask_a >= g_mask_a - g_mask_b;
}

/*
 * "Top-K" attention combined with the heavy hitters (appendix "Enhancing the Top-K baseline": each query keeps
 * only its largest attention logits; the paper reports it with and without H2 and gives no rule for the
 * combination).  Reading: in a decode step the query attends, of everything it would otherwise attend (the kept
 * entries the sparse pattern allows, and itself), only the m entries with the largest scaled logits — equal
 * logits: the higher position first; the others get probability 0 and no score from that step.  The cache policy
 * is unchanged.  m = 0 switches it off; the prompt rows of the one-shot prefill stay dense.
 */
static long g_topk = 0;
int h2o_oracle_set_topk(long m) {
  if (m < 0) return -1;
  g_topk = m;
  return 0;
}
typedef struct {
  double s;
  long pos, idx;
} logit_t;
static int logit_cmp(const void* a, const void* b) { /* strongest first: larger logit, then higher position */
  const logit_t* x = (const logit_t*)a;
  const logit_t* y = (const logit_t*)b;
  if (x->s != y->s) return x->s > y->s ? -1 : 1;
  if (x->pos != y->pos) return x->pos > y->pos ? -1 : 1;
  return 0;
}

/*
 * Causal softmax attention of one (sequence, head) and the column sums of its
 * probability matrix.
 *   Q, K, V : n rows of d floats, consecutive rows `stride_q` (Q) and `stride` (K, V) floats apart.
 *   c       : softmax scale.
 *   O       : [n][d]  O_i = sum_{j<=i} P[i][j] V_j
 *   rowmax, rowsum : [n]  m_i = max_j s_ij,  l_i = sum_j exp(s_ij - m_i)
 *   acc0    : [n]     acc0[j] = sum_{i>=j} P[i][j]   (summed for increasing i)
 *   P_out   : optional [n][n] (NULL to skip), zero above the diagonal.
 * P[i][j] = exp(s_ij - m_i) / l_i with s_ij = c <Q_i, K_j>, j <= i.
 * With a sparse pattern set (h2o_oracle_set_mask) row i leaves out the keys j of its recent window
 * (i - r < j < i, r = `window`) that the pattern does not allow: P[i][j] = 0 there.
 */
int h2o_oracle_causal_attention_colsum(const float* Q, const float* K, const float* V, long n, long d, long stride_q,
                                       long stride, double c, long window, double* O, double* rowmax, double* rowsum,
                                       double* acc0, double* P_out) {
  if (n < 0 || d <= 0 || stride < d || stride_q < d) return -1;
  int failed = 0;
#pragma omp parallel
  {
    double* e = (double*)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
    if (!e) {
#pragma omp atomic write
      failed = 1;
    }
#pragma omp for schedule(dynamic, 4)
    for (long i = 0; i < n; ++i) {
      if (!e) continue;
      const float* qi = Q + i * stride_q;
      double m = -INFINITY;
      for (long j = 0; j <= i; ++j) {
        if (!attended(j, i, window)) continue;
        e[j] = c * dot_fd(qi, K + j * stride, d);
        if (e[j] > m) m = e[j];
      }
      double l = 0.0;
      for (long j = 0; j <= i; ++j) {
        e[j] = attended(j, i, window) ? exp(e[j] - m) : 0.0;
        l += e[j];
      }
      rowmax[i] = m;
      rowsum[i] = l;
      double* oi = O + i * d;
      for (long x = 0; x < d; ++x) oi[x] = 0.0;
      for (long j = 0; j <= i; ++j) {
        const double p = e[j] / l;
        const float* vj = V + j * stride;
        for (long x = 0; x < d; ++x) oi[x] += p * (double)vj[x];
        if (P_out) P_out[i * n + j] = p;
      }
      if (P_out)
        for (long j = i + 1; j < n; ++j) P_out[i * n + j] = 0.0;
    }
    free(e);
    /* Column sums straight from the definition: the same s_ij, m_i and l_i again. */
#pragma omp for schedule(dynamic, 4)
    for (long j = 0; j < n; ++j) {
      const float* kj = K + j * stride;
      double a = 0.0;
      for (long i = j; i < n; ++i) {
        if (!attended(j, i, window)) continue;
        const double s = c * dot_fd(Q + i * stride_q, kj, d);
        a += exp(s - rowmax[i]) / rowsum[i];
      }
      acc0[j] = a;
    }
  }
  return failed ? -2 : 0;
}

/*
 * Score variant (Section "Discussions and Limitations", paragraph on previous attempts): the authors also
 * ranked by the AVERAGED attention score, i.e. the accumulated score divided by the number of attention
 * rows that contributed to it.  A key at position p has been attended by the queries p .. tnow, so
 *   rank score = acc / (tnow - p + 1)        (mode 1)
 *   rank score = acc                         (mode 0, Algorithm 2 as printed)
 * The accumulated score itself is stored unchanged in both modes.
 */
static int g_score_mode = 0;
int h2o_oracle_set_score_mode(int mode) {
  if (mode != 0 && mode != 1) return -1;
  g_score_mode = mode;
  return 0;
}
static double rank_score(double acc, long pos, long tnow) {
  return g_score_mode == 1 ? acc / (double)(tnow - pos + 1) : acc;
}

/*
 * F_score(S) = sum over the kept keys of h(accumulated score) (Definition of the score function and the
 * remark on h: identity in Algorithm 1/2, sqrt(z + 1) and log(z + 1) as concave choices).  Reporting
 * only: for increasing h the victim, the key whose removal keeps F_score largest, is the same.
 *   hkind 0: h(z) = z, 1: sqrt(z + 1), 2: log(z + 1)
 */
double h2o_oracle_fscore(const double* acc, long m, int hkind) {
  double f = 0.0;
  for (long j = 0; j < m; ++j) f += hkind == 1 ? sqrt(acc[j] + 1.0) : hkind == 2 ? log(acc[j] + 1.0) : acc[j];
  return f;
}

/* Eviction order: x before y iff score_x < score_y, or equal and pos_x < pos_y. */
static int precedes(double acc_x, long pos_x, double acc_y, long pos_y) {
  if (acc_x < acc_y) return 1;
  if (acc_x > acc_y) return 0;
  return pos_x < pos_y;
}

static double rel_gap(double a, double b) {
  const double m = fmax(fabs(a), fabs(b));
  return m > 0.0 ? fabs(a - b) / m : 0.0;
}

typedef struct {
  double acc;
  long pos;
} scored_t;

static int scored_cmp(const void* a, const void* b) {
  const scored_t* x = (const scored_t*)a;
  const scored_t* y = (const scored_t*)b;
  if (precedes(x->acc, x->pos, y->acc, y->pos)) return -1;
  if (precedes(y->acc, y->pos, x->acc, x->pos)) return 1;
  return 0;
}

/*
 * One-shot selection after the prompt (Appendix A: "K heavy hitters and K recent
 * tokens if the prompt has length >= 2K, otherwise all").
 *   acc0 [n], heavy budget k, recent window r.
 *   kept : out, ascending positions, min(n, k + r) of them; returns that count.
 *   boundary : out [2] = accumulated score of the weakest kept heavy hitter and of
 *              the strongest dropped candidate (NaN where there is none).
 * Heavy hitters are the k largest of positions [0, n - r) under the eviction order.
 */
long h2o_oracle_select(const double* acc0, long n, long k, long r, int32_t* kept, double* boundary) {
  boundary[0] = boundary[1] = NAN;
  if (n <= k + r) {
    for (long j = 0; j < n; ++j) kept[j] = (int32_t)j;
    return n;
  }
  const long nc = n - r; /* candidates 0..nc-1, nc > k */
  scored_t* c = (scored_t*)malloc(sizeof(scored_t) * (size_t)nc);
  if (!c) return -1;
  for (long j = 0; j < nc; ++j) {
    c[j].acc = rank_score(acc0[j], j, n - 1); /* the last prompt token is the latest query */
    c[j].pos = j;
  }
  qsort(c, (size_t)nc, sizeof(scored_t), scored_cmp); /* weakest first */
  char* keep = (char*)calloc((size_t)n, 1);
  if (!keep) {
    free(c);
    return -1;
  }
  for (long x = nc - k; x < nc; ++x) keep[c[x].pos] = 1;
  for (long j = nc; j < n; ++j) keep[j] = 1;
  if (k > 0) boundary[0] = c[nc - k].acc;
  boundary[1] = c[nc - k - 1].acc;
  long m = 0;
  for (long j = 0; j < n; ++j)
    if (keep[j]) kept[m++] = (int32_t)j;
  free(keep);
  free(c);
  return m;
}

/*
 * One decoding step for `units` independent (sequence, head) caches
 * (Algorithm 2 body: scores over G = S u {t}, accumulate, evict one).
 *
 * State, per unit u, in rows of capacity `cap` (>= k+r+1) entries:
 *   cnt[u], t[u], pos[u][cap], acc[u][cap], Kc[u][cap][d], Vc[u][cap][d]
 * Entry order carries no meaning; only `pos` does.
 * Inputs: q [units][group][d], knew, vnew [units][d]; kbud, rwin [units]; scale c.
 * group: query heads that share one unit's keys and values (grouped-query attention; 1 = every head has its own).
 *        The paper evicts per head and has no such sharing; the nearest text is its comparison with a method that
 *        accumulates scores across heads.  Reading: each query head of the group attends the shared entries with its
 *        own softmax, and a key's accumulated score grows by the SUM of the probabilities the group's heads gave it;
 *        out is [units][group][d].
 * hint  : optional [units]; a decision made elsewhere for this step (-1 none,
 *         >= 0 evicted position, -2 = no hint).  The oracle always computes its own
 *         victim first.  If the hint names a different candidate whose accumulated
 *         score is within `tie_rel` (relative) of the oracle's minimum, the hint is
 *         applied instead so that later steps stay comparable, and status = 1.
 *         Any other disagreement is status = 2 and the oracle's own choice is applied.
 * Outputs: out [units][d]; evicted [units] = oracle's own decision (-1 none);
 *          status [units]; gap [units] = relative gap between the two smallest
 *          candidate scores (inf when fewer than two); p_out optional [units][cap]
 *          = probabilities of the entries in state order, the new token last; tgap optional [units] = with
 *          "Top-K" attention on, the relative gap between the weakest kept and the strongest dropped logit
 *          (inf when nothing was dropped).
 */
int h2o_oracle_decode_step(long units, long group, long d, long cap, const int32_t* kbud, const int32_t* rwin, int32_t* t,
                           int32_t* cnt, int32_t* pos, double* acc, double* Kc, double* Vc, const float* q,
                           const float* knew, const float* vnew, double c, const int32_t* hint, double tie_rel,
                           double* out, int32_t* evicted, int32_t* status, double* gap, double* p_out, double* tgap) {
  int bad = 0;
#pragma omp parallel for schedule(dynamic, 8)
  for (long u = 0; u < units; ++u) {
    const long B = (long)kbud[u] + (long)rwin[u];
    const long r = rwin[u];
    long m = cnt[u];
    int32_t* up = pos + u * cap;
    double* ua = acc + u * cap;
    double* uk = Kc + u * cap * d;
    double* uv = Vc + u * cap * d;
    if (m + 1 > cap || m > B) {
#pragma omp atomic write
      bad = 1;
      continue;
    }
    const long tt = t[u];
    /* G = S u {t}: append the new token with zero accumulated score. */
    up[m] = (int32_t)tt;
    ua[m] = 0.0;
    for (long x = 0; x < d; ++x) {
      uk[m * d + x] = (double)knew[u * d + x];
      uv[m * d + x] = (double)vnew[u * d + x];
    }
    m += 1;
    /* scores, softmax, output: once per query head of the unit's group (one without grouped-query attention);
     * every query head adds its probabilities to the shared keys' accumulated scores */
    if (tgap) tgap[u] = INFINITY;
    double* e = (double*)malloc(sizeof(double) * (size_t)m);
    char* att = (char*)malloc((size_t)m);
    for (long g = 0; g < group; ++g) {
    const float* qg = q + (u * group + g) * d;
    long natt = 0;
    for (long j = 0; j < m; ++j) {
      att[j] = (char)attended(up[j], tt, r); /* 0: left out by the sparse pattern (none by default) */
      if (!att[j]) continue;
      double s = 0.0;
      for (long x = 0; x < d; ++x) s += (double)qg[x] * uk[j * d + x];
      e[j] = c * s;
      natt += 1;
    }
    if (g_topk > 0 && natt > g_topk) { /* keep the g_topk strongest logits only */
      logit_t* lg = (logit_t*)malloc(sizeof(logit_t) * (size_t)natt);
      long n2 = 0;
      for (long j = 0; j < m; ++j)
        if (att[j]) {
          lg[n2].s = e[j];
          lg[n2].pos = up[j];
          lg[n2].idx = j;
          n2 += 1;
        }
      qsort(lg, (size_t)natt, sizeof(logit_t), logit_cmp);
      for (long x = g_topk; x < natt; ++x) att[lg[x].idx] = 0;
      if (tgap) tgap[u] = fmin(tgap[u], rel_gap(lg[g_topk - 1].s, lg[g_topk].s)); /* weakest kept against strongest dropped */
      free(lg);
    }
    double mx = -INFINITY;
    for (long j = 0; j < m; ++j)
      if (att[j] && e[j] > mx) mx = e[j];
    double l = 0.0;
    for (long j = 0; j < m; ++j) {
      e[j] = att[j] ? exp(e[j] - mx) : 0.0;
      l += e[j];
    }
    double* o = out + (u * group + g) * d;
    for (long x = 0; x < d; ++x) o[x] = 0.0;
    for (long j = 0; j < m; ++j) {
      const double p = e[j] / l;
      for (long x = 0; x < d; ++x) o[x] += p * uv[j * d + x];
      ua[j] += p; /* accumulate */
      if (p_out) p_out[u * cap + j] = g == 0 ? p : p_out[u * cap + j] + p; /* (summed over the group) */
    }
    } /* query heads of the group */
    free(att);
    free(e);
    /* eviction */
    evicted[u] = -1;
    status[u] = 0;
    gap[u] = INFINITY;
    long victim = -1;
    if (m > B) {
      long second = -1;
      for (long j = 0; j < m; ++j) {
        if ((long)up[j] > tt - r) continue; /* protected recent window */
        if (victim < 0 || precedes(rank_score(ua[j], up[j], tt), up[j], rank_score(ua[victim], up[victim], tt), up[victim])) {
          second = victim;
          victim = j;
        } else if (second < 0 ||
                   precedes(rank_score(ua[j], up[j], tt), up[j], rank_score(ua[second], up[second], tt), up[second])) {
          second = j;
        }
      }
      if (victim < 0) { /* cannot happen with distinct positions < t; flagged, not hidden */
#pragma omp atomic write
        bad = 1;
        continue;
      }
      if (second >= 0) gap[u] = rel_gap(rank_score(ua[victim], up[victim], tt), rank_score(ua[second], up[second], tt));
      evicted[u] = up[victim];
      if (hint && hint[u] != -2 && hint[u] != evicted[u]) {
        long alt = -1;
        for (long j = 0; j < m; ++j)
          if (up[j] == hint[u] && (long)up[j] <= tt - r) alt = j;
        if (alt >= 0 && rel_gap(rank_score(ua[alt], up[alt], tt), rank_score(ua[victim], up[victim], tt)) < tie_rel) {
          status[u] = 1;
          victim = alt;
        } else {
          status[u] = 2;
        }
      }
      /* S = G \ {u}: close the gap, keeping the remaining order */
      for (long j = victim; j + 1 < m; ++j) {
        up[j] = up[j + 1];
        ua[j] = ua[j + 1];
        memcpy(uk + j * d, uk + (j + 1) * d, sizeof(double) * (size_t)d);
        memcpy(uv + j * d, uv + (j + 1) * d, sizeof(double) * (size_t)d);
      }
      m -= 1;
    } else if (hint && hint[u] != -2 && hint[u] != -1) {
      status[u] = 2;
    }
    cnt[u] = (int32_t)m;
    t[u] = (int32_t)(tt + 1);
  }
  return bad ? -1 : 0;
}
