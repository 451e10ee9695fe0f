/*
 * CPU oracle for the path-composed MoE FFN layer (PCoMoE).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what
 * the layer computes, written from the paper's equations.  It shares no code,
 * header, table or helper with the CUDA library, and the CUDA library never
 * calls it.  Only tests, the smoke check and the benchmark's CPU-baseline leg
 * may load it.
 *
 * Precision: path scores are formed in fp32 with three separately rounded
 * operations (they decide integers, and the CUDA path decides them in fp32
 * too).  Everything else (path weights, dot products, SiLU, the weighted sum)
 * is evaluated in fp64 from the fp32 (or bf16, upcast exactly) input values.
 *
 * Parity pins (see tests): worked example by hand from the score / TopK
 * equations; reduction to a textbook top-k SwiGLU MoE; identical-expert
 * closed form; K=1; brute force over the dense n x n path grid; invariants.
 * The outputs y on the five benchmark layers have no printed value in the
 * paper: there the parity is pinned only through that chain.
 * Router logits: a hand-computed case, unit-row weights, a library matrix product and
 * the folded-weight identity.  Residual hand-over: hand cases around a bf16 rounding
 * tie and an independent conversion.  Mask from bias / tightening step: closed cases,
 * a numpy sort, nestedness along a schedule.  Target grouping with projection-side
 * reuse: a hand example, sorted keys, the one-sixth count of Sec. 3.2 and a numpy
 * evaluation of the layer over the merged rows.
 *
 * No blocking, fusion or reordering beyond what each equation states; OpenMP
 * is used only across tokens, which are independent.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_ERR_ARG 1
#define ORACLE_ERR_MEM 2

/* weight storage types */
#define ORACLE_W_F32 0
#define ORACLE_W_BF16 1

int pcomoe_oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ---------------------------------------------------------------------------
 * Active set A = {(i,j) | m_ij = 1}  (Sec. 4.3, "Compositional Path Routing"),
 * listed in row-major order of the flat id p = i*n + j.  Returns |A|.
 * ------------------------------------------------------------------------- */
int32_t pcomoe_oracle_active_set(int32_t n, const uint8_t *M, const float *B, int32_t *act_src,
                                 int32_t *act_tgt, float *act_bias) {
  int32_t cnt = 0;
  for (int32_t i = 0; i < n; ++i)
    for (int32_t j = 0; j < n; ++j)
      if (M[(size_t)i * n + j]) {
        if (act_src) act_src[cnt] = i;
        if (act_tgt) act_tgt[cnt] = j;
        if (act_bias) act_bias[cnt] = B[(size_t)i * n + j];
        ++cnt;
      }
  return cnt;
}

typedef struct {
  float s;
  int32_t flat;
} cand_t;

/* total order of TopK: score descending, then flat id ascending */
static int cand_cmp(const void *pa, const void *pb) {
  const cand_t *a = (const cand_t *)pa, *b = (const cand_t *)pb;
  if (a->s > b->s) return -1;
  if (a->s < b->s) return 1;
  return (a->flat > b->flat) - (a->flat < b->flat);
}

/* ---------------------------------------------------------------------------
 * Path routing.
 *   score  s_ij = g_base,i + b_ij + lambda * g_tgt,j          (Sec. 4.2, score equation)
 *   Pi(h)  = TopK over (i,j) in A of s_ij                      (Sec. 4.3, TopK equation)
 *   beta   = softmax of the scores over the K selected paths (norm_topk = 1), or
 *            softmax over the whole active set gathered at the selected paths
 *            (norm_topk = 0; inactive paths are masked out before gating, Sec. 4.2),
 *            times routed_scale.
 * z = g_base [T,n], u = g_tgt [T,n] (pass z again when there is one router).
 * Outputs are rank ordered: src, tgt [T,K] int32; w [T,K] fp32; score [T,K] fp32 (optional).
 * The paper assumes finite routing signals.  Reading for the rest: a path whose score is NaN or infinite
 * (a router that masks an expert with a -inf logit, an overflow) is not eligible for that token - the same
 * thing the mask does to a path, "prior to gating" (Sec. 4.2) - and a token left with fewer than K eligible
 * paths gets src = tgt = -1 and weight 0 in the ranks it cannot fill.
 * ------------------------------------------------------------------------- */
int pcomoe_oracle_route(int32_t T, int32_t n, int32_t K, const float *z, const float *u,
                        const uint8_t *M, const float *B, float lambda, int32_t norm_topk,
                        float routed_scale, int32_t *src, int32_t *tgt, float *w, float *score) {
  if (T < 0 || n <= 0 || K <= 0 || K > n) return ORACLE_ERR_ARG;
  for (int32_t i = 0; i < n; ++i)
    if (!M[(size_t)i * n + i]) return ORACLE_ERR_ARG; /* m_ii = 1 is required */
  int err = ORACLE_OK;
#pragma omp parallel
  {
    cand_t *c = (cand_t *)malloc(sizeof(cand_t) * (size_t)n * n);
    if (!c) {
#pragma omp atomic write
      err = ORACLE_ERR_MEM;
    }
#pragma omp for schedule(static)
    for (int32_t t = 0; t < T; ++t) {
      if (!c) continue;
      int32_t cnt = 0;
      for (int32_t i = 0; i < n; ++i)
        for (int32_t j = 0; j < n; ++j) {
          if (!M[(size_t)i * n + j]) continue;
          float a = z[(size_t)t * n + i] + B[(size_t)i * n + j]; /* rounded */
          float b = lambda * u[(size_t)t * n + j];               /* rounded */
          float s = a + b;                                       /* rounded */
          s = s + 0.0f;                                          /* -0 -> +0 */
          if (!isfinite(s)) continue; /* a NaN or infinite score takes the path out of this token's active set */
          c[cnt].s = s;
          c[cnt].flat = i * n + j;
          ++cnt;
        }
      qsort(c, (size_t)cnt, sizeof(cand_t), cand_cmp);
      const int32_t live = cnt < K ? cnt : K; /* fewer than K finite scores: the remaining ranks stay empty */
      for (int32_t k = live; k < K; ++k) {
        src[(size_t)t * K + k] = -1;
        tgt[(size_t)t * K + k] = -1;
        w[(size_t)t * K + k] = 0.0f;
        if (score) score[(size_t)t * K + k] = -INFINITY;
      }
      if (live == 0) continue;
      double s0 = (double)c[0].s;
      double den = 0.0;
      int32_t lim = norm_topk ? live : cnt;
      for (int32_t a = 0; a < lim; ++a) den += exp((double)c[a].s - s0);
      for (int32_t k = 0; k < live; ++k) {
        src[(size_t)t * K + k] = c[k].flat / n;
        tgt[(size_t)t * K + k] = c[k].flat % n;
        double beta = exp((double)c[k].s - s0) / den * (double)routed_scale;
        w[(size_t)t * K + k] = (float)beta;
        if (score) score[(size_t)t * K + k] = c[k].s;
      }
    }
    free(c);
  }
  return err;
}

/* ---------------------------------------------------------------------------
 * Source grouping and target grouping (Sec. 4.3, "Source-Grouped Compute Reuse":
 * S(h) = unique selected sources, T_i(h) = their targets).
 *   slot (t,k) is "first" iff no k' < k has the same source          (dedup = 1)
 *   stage-1 rows: for i ascending, for t ascending: token t if i in S(t)
 *   stage-2 rows: for j ascending, for flat path id q = t*K+k ascending: q if tgt = j
 * dedup = 0: every path is its own stage-1 slot and stage-1 rows run over flat path ids.
 * s1_token must hold T*K entries (R1 <= T*K are written).  Returns R1 in *R1_out.
 * ------------------------------------------------------------------------- */
int pcomoe_oracle_groups(int32_t T, int32_t n, int32_t K, int32_t dedup, const int32_t *src,
                         const int32_t *tgt, const float *w, int32_t *s1_offsets, int32_t *s1_token,
                         int32_t *path_s1row, int32_t *s2_offsets, int32_t *s2_path,
                         int32_t *s2_s1row, int32_t *s2_token, float *s2_w, int32_t *R1_out) {
  if (T < 0 || n <= 0 || K <= 0) return ORACLE_ERR_ARG;
  int32_t row = 0;
  for (int32_t i = 0; i < n; ++i) {
    s1_offsets[i] = row;
    for (int32_t t = 0; t < T; ++t) {
      if (dedup) {
        int member = 0;
        for (int32_t k = 0; k < K; ++k)
          if (src[(size_t)t * K + k] == i) member = 1;
        if (!member) continue;
        for (int32_t k = 0; k < K; ++k)
          if (src[(size_t)t * K + k] == i) path_s1row[(size_t)t * K + k] = row;
        s1_token[row++] = t;
      } else {
        for (int32_t k = 0; k < K; ++k)
          if (src[(size_t)t * K + k] == i) {
            path_s1row[(size_t)t * K + k] = row;
            s1_token[row++] = t;
          }
      }
    }
  }
  s1_offsets[n] = row;
  *R1_out = row;

  int32_t r2 = 0;
  for (int32_t j = 0; j < n; ++j) {
    s2_offsets[j] = r2;
    for (int32_t q = 0; q < T * K; ++q)
      if (tgt[q] == j) {
        s2_path[r2] = q;
        s2_s1row[r2] = path_s1row[q];
        s2_token[r2] = q / K;
        s2_w[r2] = w[q];
        ++r2;
      }
  }
  s2_offsets[n] = r2;
  return ORACLE_OK;
}

/* ---------------------------------------------------------------------------
 * Target grouping with projection-side reuse.  D_j is linear, so for one token
 *   sum_{i in paths with target j} beta_ij D_j(U_i(h)) = D_j( sum_i beta_ij U_i(h) )
 * (Sec. 3.2 counts what reusing the projection side would save; Sec. 4.1 defines D_j(a) = W_down a).
 * A stage-2 row is then a unique (token, target):
 *   path (t,k) is "primary" iff no k' < k of the token has the same target; the others join their primary's row
 *   stage-2 rows: for j ascending, for primary paths q = t*K+k ascending with tgt = j
 *   s2_w   = the path's weight when the row has one contributor, 1 when it has several (the weights then
 *            scale the contributions that are summed into the row)
 *   s2_cnt = contributors of the row;  path_s2row[q] = the row path q feeds
 * path_s1row comes from pcomoe_oracle_groups.  Arrays hold T*K entries; R2 rows are written.
 * ------------------------------------------------------------------------- */
int pcomoe_oracle_groups_target_reuse(int32_t T, int32_t n, int32_t K, const int32_t *tgt, const float *w,
                                      const int32_t *path_s1row, int32_t *s2_offsets, int32_t *s2_path,
                                      int32_t *s2_s1row, int32_t *s2_token, float *s2_w, int32_t *s2_cnt,
                                      int32_t *path_s2row, int32_t *R2_out) {
  if (T < 0 || n <= 0 || K <= 0) return ORACLE_ERR_ARG;
  int32_t r2 = 0;
  for (int32_t j = 0; j < n; ++j) {
    s2_offsets[j] = r2;
    for (int32_t t = 0; t < T; ++t) {
      int32_t first = -1, cnt = 0;
      for (int32_t k = 0; k < K; ++k)
        if (tgt[(size_t)t * K + k] == j) {
          if (first < 0) first = k;
          ++cnt;
        }
      if (first < 0) continue;
      const int32_t q = t * K + first;
      s2_path[r2] = q;
      s2_s1row[r2] = path_s1row[q];
      s2_token[r2] = t;
      s2_w[r2] = cnt == 1 ? w[q] : 1.0f;
      s2_cnt[r2] = cnt;
      for (int32_t k = 0; k < K; ++k)
        if (tgt[(size_t)t * K + k] == j) path_s2row[(size_t)t * K + k] = r2;
      ++r2;
    }
  }
  s2_offsets[n] = r2;
  *R2_out = r2;
  return ORACLE_OK;
}

/* exact upcast of a bf16 bit pattern */
static inline float bf16_bits_to_f32(uint16_t b) {
  uint32_t u = (uint32_t)b << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}

/* fp64 dot product in index order; the weight row is fp32 or bf16 bits */
static double dot_row(const void *W, size_t row_off, const double *x, int32_t len, int wdtype) {
  double acc = 0.0;
  if (wdtype == ORACLE_W_F32) {
    const float *p = (const float *)W + row_off;
    for (int32_t i = 0; i < len; ++i) acc += (double)p[i] * x[i];
  } else {
    const uint16_t *p = (const uint16_t *)W + row_off;
    for (int32_t i = 0; i < len; ++i) acc += (double)bf16_bits_to_f32(p[i]) * x[i];
  }
  return acc;
}

static inline double silu(double g) { return g / (1.0 + exp(-g)); }

/* U_e(h) = SiLU(W_gate h) (.) (W_up h)   (Sec. 4.1, expansion-side operator) */
static void expansion(const void *Wg, const void *Wu, size_t base, int32_t F, int32_t H,
                      const double *h, double *a, int wdtype) {
  for (int32_t f = 0; f < F; ++f) {
    double g = dot_row(Wg, base + (size_t)f * H, h, H, wdtype);
    double v = dot_row(Wu, base + (size_t)f * H, h, H, wdtype);
    a[f] = silu(g) * v;
  }
}

/* ---------------------------------------------------------------------------
 * Layer output for the listed tokens:
 *   y = sum over the token's selected paths of beta_ij * D_j(U_i(h))   (Sec. 4.1, layer output)
 * summed in rank order; D_j(a) = W_down^(j) a.  dedup = 1 evaluates each distinct
 * source's U_i(h) once and reuses it (Sec. 4.3, source-grouped output) - the same values in
 * the same order, so both settings give identical bits.  A shared expert (F_sh > 0) is a
 * dense SwiGLU FFN added with weight 1 after the routed sum.
 * h [T,H] fp32; weights [n,F,H],[n,F,H],[n,H,F] (+ shared [F_sh,H],[F_sh,H],[H,F_sh]) in
 * wdtype; src,tgt,w [T,K]; tokens[n_tok] lists the token ids to evaluate (NULL = 0..n_tok-1);
 * y [n_tok,H] fp64.
 * ------------------------------------------------------------------------- */
int pcomoe_oracle_ffn(int32_t T, int32_t H, int32_t F, int32_t n, int32_t K, int32_t F_sh,
                      const float *h, const void *Wg, const void *Wu, const void *Wd,
                      const void *Wsg, const void *Wsu, const void *Wsd, int32_t wdtype,
                      const int32_t *src, const int32_t *tgt, const float *w, int32_t dedup,
                      const int32_t *tokens, int32_t n_tok, double *y) {
  if (T < 0 || H <= 0 || F <= 0 || n <= 0 || K <= 0 || n_tok < 0) return ORACLE_ERR_ARG;
  int err = ORACLE_OK;
#pragma omp parallel
  {
    double *hd = (double *)malloc(sizeof(double) * (size_t)H);
    double *a = (double *)malloc(sizeof(double) * (size_t)F * (size_t)K);
    double *ash = F_sh > 0 ? (double *)malloc(sizeof(double) * (size_t)F_sh) : NULL;
    int ok = hd && a && (F_sh == 0 || ash);
    if (!ok) {
#pragma omp atomic write
      err = ORACLE_ERR_MEM;
    }
#pragma omp for schedule(dynamic, 1)
    for (int32_t it = 0; it < n_tok; ++it) {
      if (!ok) continue;
      int32_t t = tokens ? tokens[it] : it;
      if (t < 0 || t >= T) {
#pragma omp atomic write
        err = ORACLE_ERR_ARG;
        continue;
      }
      for (int32_t c = 0; c < H; ++c) hd[c] = (double)h[(size_t)t * H + c];
      double *yt = y + (size_t)it * H;
      for (int32_t c = 0; c < H; ++c) yt[c] = 0.0;
      for (int32_t k = 0; k < K; ++k) {
        int32_t i = src[(size_t)t * K + k], j = tgt[(size_t)t * K + k];
        double beta = (double)w[(size_t)t * K + k];
        double *ak = a + (size_t)k * F;
        int32_t reuse = -1;
        if (dedup)
          for (int32_t k2 = 0; k2 < k; ++k2)
            if (src[(size_t)t * K + k2] == i) {
              reuse = k2;
              break;
            }
        if (reuse >= 0)
          memcpy(ak, a + (size_t)reuse * F, sizeof(double) * (size_t)F);
        else
          expansion(Wg, Wu, (size_t)i * F * H, F, H, hd, ak, wdtype);
        for (int32_t c = 0; c < H; ++c)
          yt[c] += beta * dot_row(Wd, ((size_t)j * H + c) * F, ak, F, wdtype);
      }
      if (F_sh > 0) {
        expansion(Wsg, Wsu, 0, F_sh, H, hd, ash, wdtype);
        for (int32_t c = 0; c < H; ++c) yt[c] += dot_row(Wsd, (size_t)c * F_sh, ash, F_sh, wdtype);
      }
    }
    free(hd);
    free(a);
    free(ash);
  }
  return err;
}

/* ---------------------------------------------------------------------------
 * The same layer evaluated stage by stage over the group arrays
 * (Sec. 4.3, source-grouped output formula): stage 1 fills one row of U per
 * (token, source) slot, stage 2 walks the target groups and adds
 * s2_w * W_down^(j) U[s2_s1row] into y[s2_token].  Used to check that the group arrays mean what
 * they should; summation order differs from pcomoe_oracle_ffn, so values agree to rounding only.
 * y [T,H] fp64, all tokens.  No shared expert here.
 * ------------------------------------------------------------------------- */
int pcomoe_oracle_ffn_grouped(int32_t T, int32_t H, int32_t F, int32_t n, const float *h,
                              const void *Wg, const void *Wu, const void *Wd, int32_t wdtype,
                              const int32_t *s1_offsets, const int32_t *s1_token,
                              const int32_t *s2_offsets, const int32_t *s2_s1row,
                              const int32_t *s2_token, const float *s2_w, double *y) {
  int32_t R1 = s1_offsets[n];
  double *U = (double *)malloc(sizeof(double) * (size_t)(R1 > 0 ? R1 : 1) * F);
  double *hd = (double *)malloc(sizeof(double) * (size_t)H);
  if (!U || !hd) {
    free(U);
    free(hd);
    return ORACLE_ERR_MEM;
  }
  for (int32_t i = 0; i < n; ++i)
    for (int32_t r = s1_offsets[i]; r < s1_offsets[i + 1]; ++r) {
      int32_t t = s1_token[r];
      for (int32_t c = 0; c < H; ++c) hd[c] = (double)h[(size_t)t * H + c];
      expansion(Wg, Wu, (size_t)i * F * H, F, H, hd, U + (size_t)r * F, wdtype);
    }
  for (size_t x = 0; x < (size_t)T * H; ++x) y[x] = 0.0;
  for (int32_t j = 0; j < n; ++j)
    for (int32_t q = s2_offsets[j]; q < s2_offsets[j + 1]; ++q) {
      double *yt = y + (size_t)s2_token[q] * H;
      const double *a = U + (size_t)s2_s1row[q] * F;
      for (int32_t c = 0; c < H; ++c)
        yt[c] += (double)s2_w[q] * dot_row(Wd, ((size_t)j * H + c) * F, a, F, wdtype);
    }
  free(U);
  free(hd);
  return ORACLE_OK;
}

/* ---------------------------------------------------------------------------
 * Mask from bias (Sec. 4.2: the bias is converted into an active mask with m_ii = 1 that filters low-value
 * off-diagonal routes; the criterion is not given - reading: keep the `keep` off-diagonal pairs with the
 * largest bias, ties to the smaller flat id).  Selection by repeated arg-max: plain and slow.
 * ------------------------------------------------------------------------- */
int pcomoe_oracle_mask_from_bias(int32_t n, const float *B, int64_t keep, uint8_t *M) {
  if (n <= 0 || keep < 0 || keep > (int64_t)n * (n - 1)) return ORACLE_ERR_ARG;
  for (int32_t i = 0; i < n * n; ++i) M[i] = 0;
  for (int32_t i = 0; i < n; ++i) M[(size_t)i * n + i] = 1;
  for (int64_t r = 0; r < keep; ++r) {
    int32_t best = -1;
    for (int32_t p = 0; p < n * n; ++p) {
      if (p / n == p % n || M[p]) continue;
      if (best < 0 || B[p] > B[best]) best = p;
    }
    M[best] = 1;
  }
  return ORACLE_OK;
}

/* ---------------------------------------------------------------------------
 * Router in front of the path gate (Sec. 3.1: the router turns the hidden state into routing scores;
 * Sec. 4.2 names them the base routing signal g_base(h), and g_tgt(h) when a second head is given):
 *   logits[t,e] = sum_k h[t,k] * W_r[e,k]
 * plus, when a low-rank gate adaptation is attached (Sec. 5.1: rank-16 LoRA on the gate),
 *   logits[t,e] += scale * sum_q B_l[e,q] * (sum_k A_l[q,k] * h[t,k]).
 * h [T,H] fp32; W_r [n,H] and A_l [r,H] in wdtype; B_l [n,r] fp32; logits [T,n] fp64.  r = 0: no adaptation.
 * The paper gives no precision for the router: everything here is fp64 from the stored values.
 * ------------------------------------------------------------------------- */
int pcomoe_oracle_router_logits(int32_t T, int32_t H, int32_t n, int32_t r, const float *h, const void *Wr,
                                const void *Al, const float *Bl, double scale, int32_t wdtype,
                                double *logits) {
  if (T < 0 || H <= 0 || n <= 0 || r < 0 || !h || !Wr || !logits) return ORACLE_ERR_ARG;
  if (r > 0 && (!Al || !Bl)) return ORACLE_ERR_ARG;
  if (wdtype != ORACLE_W_F32 && wdtype != ORACLE_W_BF16) return ORACLE_ERR_ARG;
#pragma omp parallel for schedule(static)
  for (int32_t t = 0; t < T; ++t) {
    double *x = (double *)malloc(sizeof(double) * (size_t)(H + (r > 0 ? r : 1)));
    double *low = x + H;
    for (int32_t k = 0; k < H; ++k) x[k] = (double)h[(size_t)t * H + k];
    for (int32_t q = 0; q < r; ++q) low[q] = dot_row(Al, (size_t)q * H, x, H, wdtype);
    for (int32_t e = 0; e < n; ++e) {
      double v = dot_row(Wr, (size_t)e * H, x, H, wdtype);
      double d = 0.0;
      for (int32_t q = 0; q < r; ++q) d += (double)Bl[(size_t)e * r + q] * low[q];
      logits[(size_t)t * n + e] = v + scale * d;
    }
    free(x);
  }
  return ORACLE_OK;
}

/* ---------------------------------------------------------------------------
 * One step of the progressive tightening (Sec. 4.2: the sparsity criterion is tightened at training intervals
 * and the active path set only contracts; the diagonal always stays).  Reading: of the off-diagonal pairs
 * active in M_prev, the `keep` with the largest current bias stay active (ties to the smaller flat id); a pair
 * that was dropped earlier never returns.  Repeated arg-max, plain and slow.
 * ------------------------------------------------------------------------- */
int pcomoe_oracle_mask_tighten(int32_t n, const float *B, const uint8_t *M_prev, int64_t keep, uint8_t *M) {
  if (n <= 0 || keep < 0) return ORACLE_ERR_ARG;
  int64_t active = 0;
  for (int32_t p = 0; p < n * n; ++p)
    if (p / n != p % n && M_prev[p]) ++active;
  if (keep > active) return ORACLE_ERR_ARG;
  for (int32_t p = 0; p < n * n; ++p) M[p] = 0;
  for (int32_t i = 0; i < n; ++i) M[(size_t)i * n + i] = 1;
  for (int64_t r = 0; r < keep; ++r) {
    int32_t best = -1;
    for (int32_t p = 0; p < n * n; ++p) {
      if (p / n == p % n || !M_prev[p] || M[p]) continue;
      if (best < 0 || B[p] > B[best]) best = p;
    }
    M[best] = 1;
  }
  return ORACLE_OK;
}

/* ---------------------------------------------------------------------------
 * Residual stream between layers of a multi-layer loop: h_out = round(h_in + y).  The result is the next
 * layer's stored input (a quantised code when the storage type is bf16), so the precision of the decision is
 * fixed here as the CUDA path fixes it: one fp32 addition, then round-to-nearest-even to bf16 (wdtype = bf16;
 * the bf16 values travel as bit patterns) or the fp32 sum itself (wdtype = fp32).  The paper does not write
 * this step out; it is the usual residual connection around the block whose output is y (Sec. 4.1).
 * ------------------------------------------------------------------------- */
static uint16_t f32_to_bf16_rne(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x40u); /* NaN stays NaN */
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7fffu + lsb;
  return (uint16_t)(u >> 16);
}

int pcomoe_oracle_residual_cast(int64_t count, const void *h_in, const float *y, void *h_out, int32_t wdtype) {
  if (count < 0 || !h_in || !y || !h_out) return ORACLE_ERR_ARG;
  if (wdtype == ORACLE_W_F32) {
    const float *a = (const float *)h_in;
    float *o = (float *)h_out;
    for (int64_t i = 0; i < count; ++i) {
      volatile float s = a[i] + y[i];
      o[i] = s;
    }
  } else if (wdtype == ORACLE_W_BF16) {
    const uint16_t *a = (const uint16_t *)h_in;
    uint16_t *o = (uint16_t *)h_out;
    for (int64_t i = 0; i < count; ++i) {
      volatile float s = bf16_bits_to_f32(a[i]) + y[i];
      o[i] = f32_to_bf16_rne(s);
    }
  } else {
    return ORACLE_ERR_ARG;
  }
  return ORACLE_OK;
}
