/*
 * CPU fp64 oracle for delta-rule linear-attention prefill (GDN and KDA).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA library is checked against.  It shares no code with the CUDA path and
 * must never be called from it: only tests, the smoke check and the bench's
 * CPU-baseline leg may load it.
 *
 * What it computes (paper Section 2.1, "Architecture of Linear-Attention
 * Hybrids": a fixed-size recurrent state per head is updated from the previous
 * state with K_t and V_t, then the output is formed from Q_t and the UPDATED
 * state).  The paper names the recurrence but prints no equation; the form
 * below is the gated delta rule, one token at a time, per V-head:
 *
 *     h      : d_k x d_v state (row = key channel, column = value channel)
 *     GDN    : h <- exp(g_t) * h                       (scalar gate per head)
 *     KDA    : h[c,:] <- exp(g_t[c]) * h[c,:]          (gate per key channel)
 *     r      = h^T k_t                                 (prediction, after decay)
 *     h      <- h + beta_t * k_t (v_t - r)^T           (delta-rule write)
 *     o_t    = scale * h^T q_t                         (post-update state)
 *
 * In the S = h^T notation this is
 *     GDN  S_t = alpha_t S_{t-1} (I - beta_t k_t k_t^T) + beta_t v_t k_t^T
 *     KDA  S_t = S_{t-1} Diag(alpha_t) (I - beta_t k_t k_t^T) + beta_t v_t k_t^T
 * with alpha = exp(g), o_t = scale * S_t q_t.
 *
 * There is no chunking, blocking, fusion or reordering here: the chunkwise
 * method (paper Section 2.1, "Chunkwise Map-Reduce-Map Execution", operators
 * #1-#6) reaches the same result faster; this is the result it has to reach.
 *
 * Parity pins for this file (tests/test_oracle_pins.py): hand-worked two-token
 * examples, the single-token closed form, the frozen-state case beta=0, the
 * small-beta limit that reduces to a causal prefix sum, orthogonal keys, the
 * retrieval identity (beta=1, q=k), split/resume, head/sequence/column
 * independence, the norm bound, and equality with an independently written
 * chunkwise fp64 evaluation.  The grouped-value head mapping (V-head j uses
 * QK-head j / (HV/HK)) is not in the paper; it is pinned only by the
 * equality with an explicitly expanded run.
 *
 * Inputs are float (bf16- or fp32-valued numbers are exact in float); all
 * arithmetic and both outputs are double.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
  int32_t variant;        /* 0 = GDN (scalar gate), 1 = KDA (gate per key channel) */
  int32_t num_seqs;       /* N                                                   */
  int32_t num_qk_heads;   /* HK                                                  */
  int32_t num_v_heads;    /* HV, multiple of HK                                  */
  int32_t d_k, d_v;
  double scale;
  const int64_t* cu_seqlens; /* [N+1], cu[0] = 0, tokens of sequence n are [cu[n], cu[n+1]) */
  const float* q;         /* [T, HK, d_k]                                        */
  const float* k;         /* [T, HK, d_k]                                        */
  const float* v;         /* [T, HV, d_v]                                        */
  const float* g;         /* GDN [T, HV]; KDA [T, HV, d_k]                       */
  const float* beta;      /* [T, HV]                                             */
  const float* h0;        /* [N, HV, d_k, d_v] or NULL (zeros)                   */
  double* o;              /* [T, HV, d_v]                                        */
  double* hT;             /* [N, HV, d_k, d_v] or NULL                           */
  const int32_t* pairs;   /* optional [num_pairs][2] = (sequence, V-head) to compute; NULL = all */
  int32_t num_pairs;
} ha_la_oracle_args;

/* One (sequence, V-head): the recurrence above, token by token. */
static void oracle_one(const ha_la_oracle_args* a, int n, int j, double* h, double* r)
{
  const int dk = a->d_k, dv = a->d_v, HK = a->num_qk_heads, HV = a->num_v_heads;
  const int jq = j / (HV / HK);
  const int64_t t0 = a->cu_seqlens[n], t1 = a->cu_seqlens[n + 1];

  if (a->h0) {
    const float* src = a->h0 + ((size_t)n * HV + j) * dk * dv;
    for (int i = 0; i < dk * dv; ++i) h[i] = (double)src[i];
  } else {
    for (int i = 0; i < dk * dv; ++i) h[i] = 0.0;
  }

  for (int64_t t = t0; t < t1; ++t) {
    const float* qt = a->q + ((size_t)t * HK + jq) * dk;
    const float* kt = a->k + ((size_t)t * HK + jq) * dk;
    const float* vt = a->v + ((size_t)t * HV + j) * dv;
    const double bt = (double)a->beta[(size_t)t * HV + j];

    /* decay */
    if (a->variant == 0) {
      const double al = exp((double)a->g[(size_t)t * HV + j]);
      for (int i = 0; i < dk * dv; ++i) h[i] *= al;
    } else {
      const float* gt = a->g + ((size_t)t * HV + j) * dk;
      for (int c = 0; c < dk; ++c) {
        const double al = exp((double)gt[c]);
        for (int x = 0; x < dv; ++x) h[c * dv + x] *= al;
      }
    }
    /* r = h^T k */
    for (int x = 0; x < dv; ++x) r[x] = 0.0;
    for (int c = 0; c < dk; ++c) {
      const double kc = (double)kt[c];
      for (int x = 0; x < dv; ++x) r[x] += h[c * dv + x] * kc;
    }
    /* h += beta k (v - r)^T */
    for (int x = 0; x < dv; ++x) r[x] = bt * ((double)vt[x] - r[x]);
    for (int c = 0; c < dk; ++c) {
      const double kc = (double)kt[c];
      for (int x = 0; x < dv; ++x) h[c * dv + x] += kc * r[x];
    }
    /* o = scale h^T q */
    double* ot = a->o + ((size_t)t * HV + j) * dv;
    for (int x = 0; x < dv; ++x) ot[x] = 0.0;
    for (int c = 0; c < dk; ++c) {
      const double qc = (double)qt[c];
      for (int x = 0; x < dv; ++x) ot[x] += h[c * dv + x] * qc;
    }
    for (int x = 0; x < dv; ++x) ot[x] *= a->scale;
  }

  if (a->hT) {
    double* dst = a->hT + ((size_t)n * HV + j) * dk * dv;
    memcpy(dst, h, sizeof(double) * (size_t)dk * dv);
  }
}

/* Returns 0 on success, 1 on a bad argument, 2 when out of memory.
 * num_threads <= 0 means "all cores".  *threads_used gets the team size. */
int ha_la_oracle(const ha_la_oracle_args* a, int num_threads, int* threads_used)
{
  if (!a || !a->cu_seqlens || !a->q || !a->k || !a->v || !a->g || !a->beta || !a->o) return 1;
  if (a->num_seqs < 0 || a->d_k <= 0 || a->d_v <= 0 || a->num_qk_heads <= 0) return 1;
  if (a->num_v_heads <= 0 || a->num_v_heads % a->num_qk_heads != 0) return 1;
  if (a->variant != 0 && a->variant != 1) return 1;
  for (int n = 0; n < a->num_seqs; ++n)
    if (a->cu_seqlens[n + 1] < a->cu_seqlens[n]) return 1;

  const int HV = a->num_v_heads;
  const long total = a->pairs ? (long)a->num_pairs : (long)a->num_seqs * HV;
  if (a->pairs)
    for (long w = 0; w < total; ++w)
      if (a->pairs[2 * w] < 0 || a->pairs[2 * w] >= a->num_seqs ||
          a->pairs[2 * w + 1] < 0 || a->pairs[2 * w + 1] >= HV) return 1;
  int used = 1, oom = 0;
#ifdef _OPENMP
  if (num_threads <= 0) num_threads = omp_get_num_procs();
  if (num_threads > total && total > 0) num_threads = (int)total;
  if (num_threads < 1) num_threads = 1;
#pragma omp parallel num_threads(num_threads)
#endif
  {
    double* h = (double*)malloc(sizeof(double) * (size_t)a->d_k * a->d_v);
    double* r = (double*)malloc(sizeof(double) * (size_t)a->d_v);
#ifdef _OPENMP
#pragma omp single
    used = omp_get_num_threads();
#endif
    if (!h || !r) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
      oom = 1;
    }
#ifdef _OPENMP
#pragma omp barrier
#pragma omp for schedule(dynamic, 1)
#endif
    for (long w = 0; w < total; ++w) {
      if (oom) continue;
      int n, j;
      if (a->pairs) { n = a->pairs[2 * w]; j = a->pairs[2 * w + 1]; }
      else          { n = (int)(w / HV);   j = (int)(w % HV); }
      oracle_one(a, n, j, h, r);
    }
    free(h);
    free(r);
  }
  if (threads_used) *threads_used = used;
  return oom ? 2 : 0;
}

int ha_la_oracle_abi_version(void) { return 1; }
