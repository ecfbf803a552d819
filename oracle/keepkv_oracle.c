/*
 * KeepKV CPU oracle  --  TEST INFRASTRUCTURE, NOT PART OF THE PRODUCT PATH.
 *
 * A plain, slow, single-purpose restatement of what the KeepKV hot path computes
 * (Electoral-Votes attention, EMA score tracking, budgeted selection, cosine
 * matching, Zero Inference-Perturbation merge).  It exists so that the CUDA
 * library can be checked element by element against something a reader can
 * compare with the paper by eye.  It shares no code with the CUDA path, and only
 * the tests, the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * All floating-point work is fp64 on inputs that are exactly representable
 * (bf16 keys/values, fp32 votes/scores), except the two places where a floating
 * point number decides an integer:
 *   - the selection key kappa is compared as an fp32 value,
 *   - the cosine similarity that picks a merge target is a fixed fp32 recipe
 *     (sequential fmaf chain), so that CPU and GPU can take the same decision.
 *
 * One "unit" is one (sequence, kv-head) pair; every function works on one unit,
 * the *_batch wrappers loop over units with OpenMP.
 *
 * Notation follows the paper: d head dim, k_i/v_i cache rows, p_i Electoral Votes,
 * s_i = exp(q.k_i/sqrt(d)) the unnormalised score (Eq. 3), lambda_i = ln of the
 * EMA estimate of s_i (Eq. 8), G query heads sharing one kv head.
 *
 * Parity unpinned (the paper prints nothing that fixes them; they are readings
 * fixed by this oracle): the GQA score reduction (mean over the group),
 * first-observation initialisation of the EMA, the sink/recent/heavy split of the
 * selection, the gamma guard, the ascending order of the compacted cache, and the pairing
 * rule of the prefill merge-first policy (earlier entry is the target, a target is never a member).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
  int32_t G;                /* query heads per kv head                              */
  int32_t d;                /* head dimension                                       */
  int32_t n_sink;           /* always-kept first entries (App. B.3)                 */
  int32_t n_recent;         /* always-kept last entries  (App. B.3)                 */
  int32_t storage_faithful; /* 1: round K,V to bf16 and votes/lscore to fp32 on write */
  int32_t pad_;
  double sm_scale;          /* 1/sqrt(d), Eq. 3                                     */
  double ema_alpha;         /* alpha of Eq. 8                                       */
  double merge_threshold;   /* T of Algorithm 1, arg-max and threshold step; -inf merges always          */
  double gamma_min;         /* guard on the key rescale factor: merge iff           */
  double gamma_max;         /*   gamma_min < gamma <= gamma_max and |lambda_bar|>=1e-6 */
} okv_params;

typedef struct {
  int32_t n_retained, n_evicted, n_merged, n_below_T, n_guard_groups, n_groups, max_group, pad_;
} okv_stats;

/* ---------------------------------------------------------------- rounding */

/* Round-to-nearest-even of a double to the bf16 grid (8 significant bits,
 * fp32 exponent range), done directly from fp64 so there is no double rounding. */
double okv_round_bf16(double x) {
  if (x == 0.0 || isnan(x) || isinf(x)) return x;
  int e;
  double m = frexp(x, &e);          /* x = m * 2^e, 0.5 <= |m| < 1 */
  int shift = 8;                    /* 8 significant bits          */
  if (e - 8 < -133) shift = e + 133;/* subnormal bf16: fixed ulp 2^-133 */
  double r;
  if (shift <= 0) {
    r = ldexp(nearbyint(ldexp(x, 133)), -133);
  } else {
    r = ldexp(nearbyint(ldexp(m, shift)), e - shift);
  }
  if (fabs(r) >= ldexp(1.0, 128)) r = copysign(INFINITY, x);
  return r;
}

double okv_round_fp32(double x) { return (double)(float)x; }

static double store_kv(const okv_params *P, double x) { return P->storage_faithful ? okv_round_bf16(x) : x; }
static double store_f32(const okv_params *P, double x) { return P->storage_faithful ? okv_round_fp32(x) : x; }

static double logaddexp(double a, double b) {
  if (a == -INFINITY) return b;
  if (b == -INFINITY) return a;
  double m = a > b ? a : b;
  return m + log(exp(a - m) + exp(b - m));
}

/* ------------------------------------------------ Eq. 3 / Eq. 6: attention */

/* logit l_{g,i} = sm_scale * sum_j q_{g,j} k_{i,j}   (exponent of Eq. 3) */
void okv_logits(const okv_params *P, int32_t len, const double *q, const double *K, double *ell) {
  for (int g = 0; g < P->G; ++g)
    for (int i = 0; i < len; ++i) {
      double acc = 0.0;
      for (int j = 0; j < P->d; ++j) acc += q[g * P->d + j] * K[(size_t)i * P->d + j];
      ell[(size_t)g * len + i] = P->sm_scale * acc;
    }
}

/* Electoral-Votes attention, Eq. 6:  o_g = sum_i p_i s_{g,i} v_i / sum_i p_i s_{g,i}.
 * Written as a two-pass softmax over x_i = l_{g,i} + ln p_i.  lse_g = ln sum_i p_i s_{g,i}.
 * len == 0 gives a zero output and lse = -inf. */
void okv_decode(const okv_params *P, int32_t len, const double *q, const double *K, const double *V,
                const double *votes, double *out, double *lse) {
  const int G = P->G, d = P->d;
  double *ell = (double *)malloc(sizeof(double) * (size_t)G * (len > 0 ? len : 1));
  okv_logits(P, len, q, K, ell);
  for (int g = 0; g < G; ++g) {
    double M = -INFINITY;
    for (int i = 0; i < len; ++i) {
      double x = ell[(size_t)g * len + i] + log(votes[i]);
      if (x > M) M = x;
    }
    double den = 0.0;
    for (int j = 0; j < d; ++j) out[g * d + j] = 0.0;
    for (int i = 0; i < len; ++i) {
      double w = exp(ell[(size_t)g * len + i] + log(votes[i]) - M);
      den += w;
      for (int j = 0; j < d; ++j) out[g * d + j] += w * V[(size_t)i * d + j];
    }
    for (int j = 0; j < d; ++j) out[g * d + j] = len > 0 ? out[g * d + j] / den : 0.0;
    if (lse) lse[g] = len > 0 ? M + log(den) : -INFINITY;
  }
  free(ell);
}

/* --------------------------------------------------- Eq. 8: EMA of scores */

/* Score a kv head receives at this step: the mean over its G query heads of the
 * raw exponential scores, kept as a logarithm:  sigma_i = ln((1/G) sum_g exp l_{g,i}).
 * Recursive case of Eq. 8 in the log domain:
 *   lscore_i <- ln( alpha * exp(lscore_i) + (1-alpha) * exp(sigma_i) ),
 * an entry that has never been scored (lscore = -inf) takes sigma_i itself: the first
 * observed score initialises the state.  That equals Eq. 8's bias-corrected estimate
 * S / (1 - alpha^n), counted from the entry's first observation, at n = 1 only; from the
 * second observation on this is the plain recursion (0.9 s_1 + 0.1 s_2 at alpha = 0.9),
 * not the corrected form ((0.9 s_1 + s_2) / 1.9).  A reading, not the printed formula;
 * alpha = 0 gives lscore_i = sigma_i. */
void okv_score_update(const okv_params *P, int32_t len, const double *q, const double *K, double *lscore) {
  const int G = P->G;
  double *ell = (double *)malloc(sizeof(double) * (size_t)G * (len > 0 ? len : 1));
  okv_logits(P, len, q, K, ell);
  for (int i = 0; i < len; ++i) {
    double M = -INFINITY;
    for (int g = 0; g < G; ++g)
      if (ell[(size_t)g * len + i] > M) M = ell[(size_t)g * len + i];
    double s = 0.0;
    for (int g = 0; g < G; ++g) s += exp(ell[(size_t)g * len + i] - M);
    double sigma = M + log(s) - log((double)G);
    double r;
    if (lscore[i] == -INFINITY || P->ema_alpha == 0.0)
      r = sigma;
    else
      r = logaddexp(log(P->ema_alpha) + lscore[i], log(1.0 - P->ema_alpha) + sigma);
    lscore[i] = store_f32(P, r);
  }
  free(ell);
}

/* ---------------------------------- Eq. 8, first case: windowed initialisation */

/* Score estimate at the end of prefill (t = L in Eq. 8) from the last W = w + 1 prompt queries.
 * q is [W][G][d], oldest query first; query k sits at prompt position pos_k = len - W + k and, the
 * prompt being causal, has a score only for entries i <= pos_k (queries with pos_k < 0 do not
 * exist).  With weights omega_k = alpha^(W-1-k) -- the (1 - alpha) alpha^(t-k) of Eq. 8 up to the
 * common factor --
 *   s_hat_i = sum_{k visible} omega_k s_i^k / sum_{k visible} omega_k ,
 *   s_i^k   = (1/G) sum_g exp(sm_scale * q_{k,g} . k_i)        (group mean as in okv_score_update),
 * i.e. the bias correction divides by the weight actually accumulated, which for an entry seen by
 * the whole window is the printed 1 - alpha^(w+1).  alpha = 0 keeps the last query only.
 * lscore_i = ln s_hat_i overwrites whatever the entry held. */
void okv_prefill_scores(const okv_params *P, int32_t len, int32_t W, const double *q, const double *K,
                        double *lscore) {
  const int G = P->G, d = P->d;
  for (int i = 0; i < len; ++i) {
    /* log-sum-exp over the visible (k, g) pairs of  ln omega_k + l_{k,g,i} */
    double M = -INFINITY, wsum = 0.0;
    for (int pass = 0; pass < 2; ++pass) {
      double acc = 0.0;
      for (int k = 0; k < W; ++k) {
        const int pos = len - W + k;
        if (pos < 0 || i > pos) continue;
        double lw;
        if (P->ema_alpha == 0.0) {
          if (k != W - 1) continue;
          lw = 0.0;
        } else {
          lw = (double)(W - 1 - k) * log(P->ema_alpha);
        }
        if (pass == 0) wsum += exp(lw);
        for (int g = 0; g < G; ++g) {
          double dot = 0.0;
          for (int j = 0; j < d; ++j) dot += q[((size_t)k * G + g) * d + j] * K[(size_t)i * d + j];
          const double x = lw + P->sm_scale * dot;
          if (pass == 0) { if (x > M) M = x; }
          else acc += exp(x - M);
        }
      }
      if (pass == 1) lscore[i] = store_f32(P, M + log(acc) - log(wsum) - log((double)G));
    }
  }
}

/* ------------------------------------------------------------- selection */

/* Selection key: the entry's whole attention mass p_i * s_hat_i, as a logarithm,
 * evaluated in fp64 and rounded once to fp32; the comparison is on fp32 values. */
void okv_kappa(int32_t len, const double *votes, const double *lscore, float *kappa) {
  for (int i = 0; i < len; ++i) kappa[i] = (float)(log(votes[i]) + lscore[i]);
}

/* Retained set K_c = first n_sink  U  last n_recent  U  the (budget - sinks - recent)
 * largest kappa among the rest; equal kappa: lower index wins.  Output ascending.
 * If the budget cannot hold sinks + recent, the recent window shrinks first.
 * Returns the number retained (= min(len, budget)). */
int32_t okv_select(int32_t len, const float *kappa, int32_t budget, int32_t n_sink, int32_t n_recent,
                   int32_t *ret_idx) {
  if (budget < 0) budget = 0;
  if (budget >= len) {
    for (int i = 0; i < len; ++i) ret_idx[i] = i;
    return len;
  }
  if (n_sink > budget) n_sink = budget;
  if (n_recent > budget - n_sink) n_recent = budget - n_sink;
  /* budget < len from here on, so sinks and recent window cannot overlap */
  int lo = n_sink, hi = len - n_recent; /* candidates for heavy hitters: [lo, hi) */
  int n_heavy = budget - n_sink - n_recent;
  unsigned char *keep = (unsigned char *)calloc((size_t)len, 1);
  for (int i = 0; i < lo; ++i) keep[i] = 1;
  for (int i = hi; i < len; ++i) keep[i] = 1;
  /* pick the best remaining candidate n_heavy times; the strict '>' keeps the lowest index on ties */
  for (int r = 0; r < n_heavy; ++r) {
    int best = -1;
    for (int i = lo; i < hi; ++i) {
      if (keep[i]) continue;
      if (best < 0 || kappa[i] > kappa[best]) best = i;
    }
    keep[best] = 1;
  }
  int n = 0;
  for (int i = 0; i < len; ++i)
    if (keep[i]) ret_idx[n++] = i;
  free(keep);
  return n;
}

/* Same result as okv_select, by sorting (used for the large benchmark shapes where the
 * quadratic loop above is too slow); a test checks the two against each other. */
typedef struct { float k; int32_t i; } okv_ki;
static int cmp_ki(const void *a, const void *b) {
  const okv_ki *x = (const okv_ki *)a, *y = (const okv_ki *)b;
  if (x->k > y->k) return -1;
  if (x->k < y->k) return 1;
  return x->i < y->i ? -1 : (x->i > y->i ? 1 : 0);
}
int32_t okv_select_sorted(int32_t len, const float *kappa, int32_t budget, int32_t n_sink, int32_t n_recent,
                          int32_t *ret_idx) {
  if (budget < 0) budget = 0;
  if (budget >= len) {
    for (int i = 0; i < len; ++i) ret_idx[i] = i;
    return len;
  }
  if (n_sink > budget) n_sink = budget;
  if (n_recent > budget - n_sink) n_recent = budget - n_sink;
  int lo = n_sink, hi = len - n_recent, n_heavy = budget - n_sink - n_recent;
  okv_ki *a = (okv_ki *)malloc(sizeof(okv_ki) * (size_t)(hi - lo + 1));
  for (int i = lo; i < hi; ++i) { a[i - lo].k = kappa[i]; a[i - lo].i = i; }
  qsort(a, (size_t)(hi - lo), sizeof(okv_ki), cmp_ki);
  unsigned char *keep = (unsigned char *)calloc((size_t)len, 1);
  for (int i = 0; i < lo; ++i) keep[i] = 1;
  for (int i = hi; i < len; ++i) keep[i] = 1;
  for (int r = 0; r < n_heavy; ++r) keep[a[r].i] = 1;
  int n = 0;
  for (int i = 0; i < len; ++i)
    if (keep[i]) ret_idx[n++] = i;
  free(keep);
  free(a);
  return n;
}

/* -------------------------------------------- Algorithm 1, similarity and arg-max steps: match */

/* The fixed fp32 recipe for cosine similarity: sequential fused multiply-adds
 * from 0.0f over j = 0..d-1 for the dot product and both squared norms, then
 * dot / (sqrtf(n_e) * sqrtf(n_c)) with IEEE operations. */
static float dot_chain(const double *a, const double *b, int d) {
  float acc = 0.0f;
  for (int j = 0; j < d; ++j) acc = fmaf((float)a[j], (float)b[j], acc);
  return acc;
}
float okv_cosine(const double *ke, const double *kc, int d) {
  float dot = dot_chain(ke, kc, d);
  float ne = dot_chain(ke, ke, d);
  float nc = dot_chain(kc, kc, d);
  return dot / (sqrtf(ne) * sqrtf(nc));
}

/* For each entry e outside the retained set: target(e) = argmax over retained c of
 * cos(k_e, k_c), equal values -> lowest c; merge only if the maximum exceeds T.
 * target[i]: slot in the compacted cache (position of c in ret_idx), -1 = evicted
 * without merge, -2 = i is itself retained.  umax[i] = the winning cosine
 * (-inf where no retained key exists, 0 for retained entries).
 * second[i] (may be NULL): the runner-up cosine, for tie diagnostics. */
void okv_match(const okv_params *P, int32_t len, const double *K, int32_t n_ret, const int32_t *ret_idx,
               int32_t *target, float *umax, float *second) {
  const int d = P->d;
  const float T = (float)P->merge_threshold;
  float *nrm = (float *)malloc(sizeof(float) * (size_t)(len > 0 ? len : 1));
  for (int i = 0; i < len; ++i) nrm[i] = sqrtf(dot_chain(K + (size_t)i * d, K + (size_t)i * d, d));
  int r = 0;
  for (int e = 0; e < len; ++e) {
    if (r < n_ret && ret_idx[r] == e) { target[e] = -2; umax[e] = 0.0f; if (second) second[e] = 0.0f; ++r; continue; }
    float best = -INFINITY, sec = -INFINITY;
    int bi = -1;
    for (int c = 0; c < n_ret; ++c) {
      int ci = ret_idx[c];
      float u = dot_chain(K + (size_t)e * d, K + (size_t)ci * d, d) / (nrm[e] * nrm[ci]);
      if (u > best) { sec = best; best = u; bi = c; }
      else if (u > sec) sec = u;
    }
    umax[e] = best;
    if (second) second[e] = sec;
    target[e] = (bi >= 0 && best > T) ? bi : -1;
  }
  free(nrm);
}

/* ------------------------------- Eq. 7 / Eq. (A.3) with s_hat: ZIP merge */

/* One many-to-one merge of the group K'_e = members (the target c included) given
 * by idx[0..n).  With w_i = p_i * s_hat_i (s_hat_i = exp(lambda_i)):
 *   v_r = sum w_i v_i / sum w_i
 *   k_r = (sum w_i k_i) * ln(sum w_i / sum p_i) / (sum w_i ln s_hat_i)
 *   p_r = sum p_i ,  p_r * s_hat_r = sum w_i  =>  lambda_r = ln(sum w_i / sum p_i)
 * evaluated through omega_i = w_i / sum w (a softmax over a_i = ln p_i + lambda_i):
 *   k_r = gamma * sum omega_i k_i,  gamma = L / lambda_bar,
 *   L = LSE(a) - ln(sum p),  lambda_bar = sum omega_i lambda_i.
 * Returns gamma; kr, vr are length d. */
double okv_merge_group(int d, int n, const int32_t *idx, const double *K, const double *V, const double *votes,
                       const double *lscore, double *kr, double *vr, double *pr, double *lr,
                       double *lambda_bar_out) {
  double M = -INFINITY;
  for (int t = 0; t < n; ++t) {
    double a = log(votes[idx[t]]) + lscore[idx[t]];
    if (a > M) M = a;
  }
  double Z = 0.0, Psum = 0.0;
  for (int t = 0; t < n; ++t) {
    Z += exp(log(votes[idx[t]]) + lscore[idx[t]] - M);
    Psum += votes[idx[t]];
  }
  double Lam = M + log(Z);
  double L = Lam - log(Psum);
  double lbar = 0.0;
  for (int j = 0; j < d; ++j) { kr[j] = 0.0; vr[j] = 0.0; }
  for (int t = 0; t < n; ++t) {
    int i = idx[t];
    double om = exp(log(votes[i]) + lscore[i] - Lam);
    lbar += om * lscore[i];
    for (int j = 0; j < d; ++j) {
      kr[j] += om * K[(size_t)i * d + j];
      vr[j] += om * V[(size_t)i * d + j];
    }
  }
  double gamma = L / lbar;
  for (int j = 0; j < d; ++j) kr[j] *= gamma;
  *pr = Psum;
  *lr = L;
  if (lambda_bar_out) *lambda_bar_out = lbar;
  return gamma;
}

/* ---------------------------------------- Algorithm 1 end to end: compress */

/* src arrays hold len entries; dst arrays receive n_ret = min(len, budget) entries in
 * ascending original index.  ret_idx[n_ret], target[len] (as in okv_match), gammas
 * [n_ret] (NaN where the slot had no group) are outputs; any of target/gammas/stats
 * may be NULL.  use_sorted_select picks the sort-based selection.  Returns n_ret. */
/* select_key: NULL, or len importance scores supplied by the caller that replace kappa in the
 * selection only (Section 3.4, "no specific constraints on ... token selection strategies"; Section
 * 4.5 combines the merge with H2O's and PyramidInfer's selections): the retained and evicted sets
 * come from the given scores, the merging pairs and the merge itself are unchanged. */
int32_t okv_compress_keyed(const okv_params *P, int32_t len, int32_t budget, const double *K, const double *V,
                           const double *votes, const double *lscore, const float *select_key, double *dK,
                           double *dV, double *dvotes, double *dlscore, int32_t *ret_idx, int32_t *target_out,
                           double *gammas, okv_stats *stats, int32_t use_sorted_select);

int32_t okv_compress(const okv_params *P, int32_t len, int32_t budget, const double *K, const double *V,
                     const double *votes, const double *lscore, double *dK, double *dV, double *dvotes,
                     double *dlscore, int32_t *ret_idx, int32_t *target_out, double *gammas, okv_stats *stats,
                     int32_t use_sorted_select) {
  return okv_compress_keyed(P, len, budget, K, V, votes, lscore, NULL, dK, dV, dvotes, dlscore, ret_idx, target_out,
                            gammas, stats, use_sorted_select);
}

int32_t okv_compress_keyed(const okv_params *P, int32_t len, int32_t budget, const double *K, const double *V,
                           const double *votes, const double *lscore, const float *select_key, double *dK,
                           double *dV, double *dvotes, double *dlscore, int32_t *ret_idx, int32_t *target_out,
                           double *gammas, okv_stats *stats, int32_t use_sorted_select) {
  const int d = P->d;
  const int L1 = len > 0 ? len : 1;
  float *kappa = (float *)malloc(sizeof(float) * (size_t)L1);
  int32_t *target = (int32_t *)malloc(sizeof(int32_t) * (size_t)L1);
  float *umax = (float *)malloc(sizeof(float) * (size_t)L1);
  if (select_key) {
    for (int i = 0; i < len; ++i) kappa[i] = select_key[i];
  } else {
    okv_kappa(len, votes, lscore, kappa);
  }
  int32_t n_ret = use_sorted_select ? okv_select_sorted(len, kappa, budget, P->n_sink, P->n_recent, ret_idx)
                                    : okv_select(len, kappa, budget, P->n_sink, P->n_recent, ret_idx);
  okv_match(P, len, K, n_ret, ret_idx, target, umax, NULL);

  okv_stats st;
  memset(&st, 0, sizeof st);
  st.n_retained = n_ret;
  st.n_evicted = len - n_ret;
  for (int e = 0; e < len; ++e)
    if (target[e] == -1) st.n_below_T++;

  int32_t *members = (int32_t *)malloc(sizeof(int32_t) * (size_t)(L1 + 1));
  double *kr = (double *)malloc(sizeof(double) * (size_t)d);
  double *vr = (double *)malloc(sizeof(double) * (size_t)d);
  for (int c = 0; c < n_ret; ++c) {
    int ci = ret_idx[c];
    /* group of slot c: evicted entries that chose c, ascending, plus c itself in index order */
    int n = 0;
    for (int e = 0; e < len; ++e)
      if (e == ci || target[e] == c) members[n++] = e;
    if (gammas) gammas[c] = NAN;
    int merged = 0;
    if (n > 1) {
      st.n_groups++;
      double pr, lr, lbar;
      double gamma = okv_merge_group(d, n, members, K, V, votes, lscore, kr, vr, &pr, &lr, &lbar);
      if (gammas) gammas[c] = gamma;
      if (gamma > P->gamma_min && gamma <= P->gamma_max && fabs(lbar) >= 1e-6) {
        for (int j = 0; j < d; ++j) {
          dK[(size_t)c * d + j] = store_kv(P, kr[j]);
          dV[(size_t)c * d + j] = store_kv(P, vr[j]);
        }
        dvotes[c] = store_f32(P, pr);
        dlscore[c] = store_f32(P, lr);
        merged = 1;
        st.n_merged += n - 1;
        if (n - 1 > st.max_group) st.max_group = n - 1;
      } else {
        /* guard fired: the members are evicted after all, the target stays as it was */
        st.n_guard_groups++;
        for (int t = 0; t < n; ++t)
          if (members[t] != ci) target[members[t]] = -1;
      }
    }
    if (!merged) {
      for (int j = 0; j < d; ++j) {
        dK[(size_t)c * d + j] = K[(size_t)ci * d + j];
        dV[(size_t)c * d + j] = V[(size_t)ci * d + j];
      }
      dvotes[c] = votes[ci];
      dlscore[c] = lscore[ci];
    }
  }
  if (target_out) memcpy(target_out, target, sizeof(int32_t) * (size_t)len);
  if (stats) *stats = st;
  free(kappa); free(target); free(umax); free(members); free(kr); free(vr);
  return n_ret;
}

/* ---------------------------------------- Algorithm 1 in place (periodic mode, Section 1) */

/* The compression of Algorithm 1 on a cache whose rows are NOT in token order, done in place: "discard (k_e, v_e),
 * (k_c, v_c) and insert (k_r, v_r)" taken literally -- a merged entry replaces its target where it sits, an evicted
 * entry leaves a hole, nothing else moves except what must so that the valid entries end up in rows [0, n_ret).
 * pos[i] is the token position of row i (distinct per unit); it takes over what row order means elsewhere:
 *   - sinks: the n_sink smallest positions; recent window: the n_recent largest positions (if the budget cannot hold
 *     both, the recent window shrinks first, as in okv_select);
 *   - heavy hitters: the largest kappa among the rest, equal kappa -> lower ROW;
 *   - match: highest cosine over the retained rows, equal cosines -> lower ROW; merge iff above T;
 *   - merge: Eq. (A.3) over the target and its members (members in ascending row order, the target first is
 *     immaterial: the formula is symmetric), guard as in okv_compress; the result overwrites the target's row and
 *     keeps the target's position;
 *   - placement: n_ret = min(len, budget).  Retained rows below n_ret stay.  The retained rows at or above n_ret, in
 *     ascending row order, move into the rows below n_ret that were evicted, in ascending row order.
 * Arrays are modified in place (capacity >= len rows); moved_from[r] (n_ret entries, may be NULL) receives the row
 * each final row came from; target [len] as in okv_compress but in ROW numbers before the placement (-1 evicted
 * without merge, -2 retained); gammas [len] per row (NaN where the row had no group).  Returns n_ret.
 * What is fixed by the paper here is only that retained entries are untouched unless merged; the tie rules by row
 * and the placement rule are this oracle's (parity unpinned). */
int32_t okv_compress_inplace(const okv_params *P, int32_t len, int32_t budget, double *K, double *V, double *votes,
                             double *lscore, int32_t *pos, int32_t *moved_from, int32_t *target_out, double *gammas,
                             okv_stats *stats) {
  const int d = P->d;
  const int L1 = len > 0 ? len : 1;
  if (budget < 0) budget = 0;
  const int n_ret = len < budget ? len : budget;
  unsigned char *keep = (unsigned char *)calloc((size_t)L1, 1);
  int32_t *target = (int32_t *)malloc(sizeof(int32_t) * (size_t)L1);
  okv_stats st;
  memset(&st, 0, sizeof st);
  if (budget >= len) {
    for (int i = 0; i < len; ++i) keep[i] = 1;
  } else {
    int n_sink = P->n_sink, n_recent = P->n_recent;
    if (n_sink > budget) n_sink = budget;
    if (n_recent > budget - n_sink) n_recent = budget - n_sink;
    /* rank of every row by position */
    for (int i = 0; i < len; ++i) {
      int before = 0;
      for (int j = 0; j < len; ++j) before += pos[j] < pos[i] ? 1 : 0;
      if (before < n_sink || before >= len - n_recent) keep[i] = 1;
    }
    float *kappa = (float *)malloc(sizeof(float) * (size_t)L1);
    okv_kappa(len, votes, lscore, kappa);
    const int n_heavy = budget - n_sink - n_recent;
    for (int r = 0; r < n_heavy; ++r) {   /* the strict '>' keeps the lowest row on ties */
      int best = -1;
      for (int i = 0; i < len; ++i) {
        if (keep[i]) continue;
        if (best < 0 || kappa[i] > kappa[best]) best = i;
      }
      keep[best] = 1;
    }
    free(kappa);
  }
  /* match: every evicted row against every retained row */
  const float T = (float)P->merge_threshold;
  float *nrm = (float *)malloc(sizeof(float) * (size_t)L1);
  for (int i = 0; i < len; ++i) nrm[i] = sqrtf(dot_chain(K + (size_t)i * d, K + (size_t)i * d, d));
  for (int e = 0; e < len; ++e) {
    if (keep[e]) { target[e] = -2; continue; }
    float best = -INFINITY;
    int bi = -1;
    for (int c = 0; c < len; ++c) {
      if (!keep[c]) continue;
      float u = dot_chain(K + (size_t)e * d, K + (size_t)c * d, d) / (nrm[e] * nrm[c]);
      if (u > best) { best = u; bi = c; }
    }
    target[e] = (bi >= 0 && best > T) ? bi : -1;
    if (target[e] == -1) st.n_below_T++;
  }
  free(nrm);
  st.n_retained = n_ret;
  st.n_evicted = len - n_ret;
  /* merge: results are computed from the untouched inputs, then written */
  int32_t *members = (int32_t *)malloc(sizeof(int32_t) * (size_t)(L1 + 1));
  double *newK = (double *)malloc(sizeof(double) * (size_t)L1 * d), *newV = (double *)malloc(sizeof(double) * (size_t)L1 * d);
  double *newp = (double *)malloc(sizeof(double) * (size_t)L1), *newl = (double *)malloc(sizeof(double) * (size_t)L1);
  unsigned char *rewritten = (unsigned char *)calloc((size_t)L1, 1);
  for (int c = 0; c < len; ++c) {
    if (gammas) gammas[c] = NAN;
    if (!keep[c]) continue;
    int n = 0;
    for (int e = 0; e < len; ++e)
      if (e == c || target[e] == c) members[n++] = e;
    if (n > 1) {
      st.n_groups++;
      double pr, lr, lbar;
      double gamma = okv_merge_group(d, n, members, K, V, votes, lscore, newK + (size_t)c * d, newV + (size_t)c * d, &pr,
                                     &lr, &lbar);
      if (gammas) gammas[c] = gamma;
      if (gamma > P->gamma_min && gamma <= P->gamma_max && fabs(lbar) >= 1e-6) {
        for (int j = 0; j < d; ++j) {
          newK[(size_t)c * d + j] = store_kv(P, newK[(size_t)c * d + j]);
          newV[(size_t)c * d + j] = store_kv(P, newV[(size_t)c * d + j]);
        }
        newp[c] = store_f32(P, pr);
        newl[c] = store_f32(P, lr);
        rewritten[c] = 1;
        st.n_merged += n - 1;
        if (n - 1 > st.max_group) st.max_group = n - 1;
      } else {
        st.n_guard_groups++;
        for (int t = 0; t < n; ++t)
          if (members[t] != c) target[members[t]] = -1;
      }
    }
  }
  for (int c = 0; c < len; ++c)
    if (rewritten[c]) {
      memcpy(K + (size_t)c * d, newK + (size_t)c * d, sizeof(double) * (size_t)d);
      memcpy(V + (size_t)c * d, newV + (size_t)c * d, sizeof(double) * (size_t)d);
      votes[c] = newp[c];
      lscore[c] = newl[c];
    }
  /* placement */
  if (moved_from)
    for (int r = 0; r < n_ret; ++r) moved_from[r] = r;
  int hole = 0;
  for (int m = n_ret; m < len; ++m) {
    if (!keep[m]) continue;
    while (keep[hole]) ++hole;   /* as many holes below n_ret as retained rows above it */
    memcpy(K + (size_t)hole * d, K + (size_t)m * d, sizeof(double) * (size_t)d);
    memcpy(V + (size_t)hole * d, V + (size_t)m * d, sizeof(double) * (size_t)d);
    votes[hole] = votes[m];
    lscore[hole] = lscore[m];
    pos[hole] = pos[m];
    if (moved_from) moved_from[hole] = m;
    ++hole;
  }
  if (target_out) memcpy(target_out, target, sizeof(int32_t) * (size_t)len);
  if (stats) *stats = st;
  free(keep); free(target); free(members); free(newK); free(newV); free(newp); free(newl); free(rewritten);
  return n_ret;
}

/* --------------------------- Section 3.4 / App. B.3: prefill "merge first, then evict" */

/* The prefill merge policy of Section 3.4 (App. B, Table 3): before any eviction, entries whose keys are similar
 * enough are merged with each other; the eviction strategy is applied afterwards (okv_compress with
 * merge_threshold = +inf evicts without merging).  The paper states the idea only; this is the reading:
 *   1. every entry e looks for its most similar OTHER entry, c(e) = argmax_{i != e} cos(k_e, k_i) (the fixed fp32
 *      cosine of okv_cosine, equal values -> lowest i), U_e the maximum;
 *   2. e wants to merge iff U_e > T and c(e) < e: of two entries the earlier one is the target, so a mutual pair
 *      merges the later into the earlier;
 *   3. no entry is both target and member: if c(e) itself wants to merge (into a still earlier entry), e stays as it
 *      is.  The members of a target c form its group K'_e (with c) and are merged by Eq. (A.3) with the score
 *      estimates, exactly as in okv_compress, including the guard on the rescale factor: a group the guard rejects
 *      loses its members, the target stays as it was (the outcome of the guard everywhere in this oracle);
 *   4. the result holds every entry that is not a member, in ascending original order; nothing else is evicted.
 * Outputs as okv_compress: dst arrays (n_ret rows), ret_idx [n_ret], target [len] (slot of the target for a
 * member, -1 for a member whose group the guard rejected, -2 for an entry that is kept), gammas [n_ret], stats
 * (n_evicted counts the members, n_below_T stays 0).  Returns n_ret. */
int32_t okv_merge_similar(const okv_params *P, int32_t len, const double *K, const double *V, const double *votes,
                          const double *lscore, double *dK, double *dV, double *dvotes, double *dlscore,
                          int32_t *ret_idx, int32_t *target_out, double *gammas, okv_stats *stats) {
  const int d = P->d;
  const int L1 = len > 0 ? len : 1;
  const float T = (float)P->merge_threshold;
  float *nrm = (float *)malloc(sizeof(float) * (size_t)L1);
  int32_t *partner = (int32_t *)malloc(sizeof(int32_t) * (size_t)L1);
  unsigned char *wants = (unsigned char *)calloc((size_t)L1, 1), *member = (unsigned char *)calloc((size_t)L1, 1);
  int32_t *slot_of = (int32_t *)malloc(sizeof(int32_t) * (size_t)L1);
  int32_t *target = (int32_t *)malloc(sizeof(int32_t) * (size_t)L1);
  for (int i = 0; i < len; ++i) nrm[i] = sqrtf(dot_chain(K + (size_t)i * d, K + (size_t)i * d, d));
  /* 1, 2: the most similar other entry */
  for (int e = 0; e < len; ++e) {
    float best = -INFINITY;
    int bi = -1;
    for (int i = 0; i < len; ++i) {
      if (i == e) continue;
      float u = dot_chain(K + (size_t)e * d, K + (size_t)i * d, d) / (nrm[e] * nrm[i]);
      if (u > best) { best = u; bi = i; }
    }
    partner[e] = bi;
    wants[e] = (bi >= 0 && best > T && bi < e) ? 1 : 0;
  }
  /* 3: a target must stay */
  for (int e = 0; e < len; ++e) member[e] = (wants[e] && !wants[partner[e]]) ? 1 : 0;
  /* 4: kept entries, ascending */
  int n_ret = 0;
  for (int i = 0; i < len; ++i) {
    slot_of[i] = -1;
    if (!member[i]) { slot_of[i] = n_ret; ret_idx[n_ret++] = i; }
  }
  for (int e = 0; e < len; ++e) target[e] = member[e] ? slot_of[partner[e]] : -2;

  okv_stats st;
  memset(&st, 0, sizeof st);
  st.n_retained = n_ret;
  st.n_evicted = len - n_ret;
  int32_t *members = (int32_t *)malloc(sizeof(int32_t) * (size_t)(L1 + 1));
  double *kr = (double *)malloc(sizeof(double) * (size_t)d);
  double *vr = (double *)malloc(sizeof(double) * (size_t)d);
  for (int c = 0; c < n_ret; ++c) {
    int ci = ret_idx[c];
    int n = 0;
    for (int e = 0; e < len; ++e)
      if (e == ci || target[e] == c) members[n++] = e;
    if (gammas) gammas[c] = NAN;
    int merged = 0;
    if (n > 1) {
      st.n_groups++;
      double pr, lr, lbar;
      double gamma = okv_merge_group(d, n, members, K, V, votes, lscore, kr, vr, &pr, &lr, &lbar);
      if (gammas) gammas[c] = gamma;
      if (gamma > P->gamma_min && gamma <= P->gamma_max && fabs(lbar) >= 1e-6) {
        for (int j = 0; j < d; ++j) {
          dK[(size_t)c * d + j] = store_kv(P, kr[j]);
          dV[(size_t)c * d + j] = store_kv(P, vr[j]);
        }
        dvotes[c] = store_f32(P, pr);
        dlscore[c] = store_f32(P, lr);
        merged = 1;
        st.n_merged += n - 1;
        if (n - 1 > st.max_group) st.max_group = n - 1;
      } else {
        st.n_guard_groups++;
        for (int t = 0; t < n; ++t)
          if (members[t] != ci) target[members[t]] = -1;
      }
    }
    if (!merged) {
      for (int j = 0; j < d; ++j) {
        dK[(size_t)c * d + j] = K[(size_t)ci * d + j];
        dV[(size_t)c * d + j] = V[(size_t)ci * d + j];
      }
      dvotes[c] = votes[ci];
      dlscore[c] = lscore[ci];
    }
  }
  if (target_out) memcpy(target_out, target, sizeof(int32_t) * (size_t)len);
  if (stats) *stats = st;
  free(nrm); free(partner); free(wants); free(member); free(slot_of); free(target); free(members); free(kr); free(vr);
  return n_ret;
}

/* ----------------------------------------------------- Eq. 2: append */

/* K_t = [K_{t-1}, k_t], V_t = [V_{t-1}, v_t]; the new entry starts with one vote and
 * no score history.  Returns the new length. */
int32_t okv_append(int d, int32_t len, double *K, double *V, double *votes, double *lscore, const double *k_new,
                   const double *v_new) {
  for (int j = 0; j < d; ++j) {
    K[(size_t)len * d + j] = k_new[j];
    V[(size_t)len * d + j] = v_new[j];
  }
  votes[len] = 1.0;
  lscore[len] = -INFINITY;
  return len + 1;
}

/* ------------------------------------------------------- batch wrappers */
/* U units laid out back to back with a stride of n_cap entries; lens[u] valid entries.
 * q is [U][G][d], out [U][G][d].  Used by the benchmark's CPU-baseline leg. */

void okv_decode_batch(const okv_params *P, int32_t U, int32_t n_cap, const int32_t *lens, const double *q,
                      const double *K, const double *V, const double *votes, double *lscore, int32_t update_scores,
                      double *out, double *lse) {
  const int G = P->G, d = P->d;
#pragma omp parallel for schedule(dynamic, 1)
  for (int u = 0; u < U; ++u) {
    const double *Ku = K + (size_t)u * n_cap * d, *Vu = V + (size_t)u * n_cap * d;
    okv_decode(P, lens[u], q + (size_t)u * G * d, Ku, Vu, votes + (size_t)u * n_cap, out + (size_t)u * G * d,
               lse ? lse + (size_t)u * G : NULL);
    if (update_scores) okv_score_update(P, lens[u], q + (size_t)u * G * d, Ku, lscore + (size_t)u * n_cap);
  }
}

void okv_compress_batch(const okv_params *P, int32_t U, int32_t n_cap, const int32_t *lens, const int32_t *budgets,
                        const double *K, const double *V, const double *votes, const double *lscore, double *dK,
                        double *dV, double *dvotes, double *dlscore, int32_t *ret_idx, int32_t *target,
                        int32_t *new_lens, okv_stats *stats) {
  const int d = P->d;
#pragma omp parallel for schedule(dynamic, 1)
  for (int u = 0; u < U; ++u) {
    size_t o = (size_t)u * n_cap;
    new_lens[u] = okv_compress(P, lens[u], budgets[u], K + o * d, V + o * d, votes + o, lscore + o, dK + o * d,
                               dV + o * d, dvotes + o, dlscore + o, ret_idx + o, target ? target + o : NULL, NULL,
                               stats ? stats + u : NULL, 1);
  }
}

int32_t okv_num_threads(void) {
  int n = 1;
#ifdef _OPENMP
#pragma omp parallel
  {
#pragma omp master
    n = omp_get_num_threads();
  }
#endif
  return n;
}
