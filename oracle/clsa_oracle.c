/*
 * CPU oracle for the CLSA decoding hot path. TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 restatement of what the path computes, written from the paper's
 * equations and sharing no code with the CUDA library:
 *
 *   index scores   I = Q_idx K_idx^T            (Eq. 3, first half; single indexer head, Eq. 2 text)
 *   routing index  S_t = TopK(I_t, k)           (Eq. 3, second half)
 *   sparse attn    O_t^(l) = Attn(Q_t^(l), K_{S_t}, V_{S_t})      (Eq. 4)
 *   dense attn     O^(l) = Attn(Q^(l), K, V)    (Eq. 1) -- an independent routine used only to
 *                                               check the k >= n limit of Eq. 4
 *   decode step    one S_t, reused by every cross-decoder layer   (Sec. 2.1, closing paragraph)
 *   projections    Q_idx = H W^Q_idx, K_idx = H W^K_idx  (Eq. 2) for the newest tokens, and the
 *                  append of their K_idx / K / V rows to the shared caches (the step before Eq. 3)
 *
 * These results are plain definitions (a matrix product, an exact selection, a softmax-weighted
 * mean over a subset), so each function is that definition written out with no blocking, fusion
 * or reordering. Inputs are bf16 bit patterns (uint16); bf16 -> double is exact; every sum runs
 * in double in index order.
 *
 * Readings where the paper is silent (all listed in the design notes of the repository):
 *   - scores are the bare dot product (no scale, no activation);
 *   - ties in TopK go to the lower token index, scores compare by value (-0.0 == +0.0);
 *   - fewer than k visible tokens: all of them are selected (k is stated as a maximum);
 *   - decode: every cached token is visible; causal chunk: query t of T sees s <= n - T + t;
 *   - Attn is scaled dot-product attention with an explicit sm_scale, no positional rotation
 *     (NoPE in global attention), GQA with contiguous groups: KV head = query head / group size;
 *   - the shared K and V rows are linear maps of the same hidden state, K = H W^K, V = H W^V
 *     (the paper only says the cache corresponds to H); no normalisation is applied here;
 *   - projected values are stored as bf16, rounded to nearest-even once from the exact sum.
 *
 * Only tests, the smoke check and the bench's CPU-baseline leg may call this file.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
  int32_t num_seqs;      /* B */
  int32_t q_per_seq;     /* T */
  int32_t num_q_heads;   /* Hq */
  int32_t num_kv_heads;  /* Hkv */
  int32_t head_dim;      /* D */
  int32_t idx_dim;       /* d_idx */
  int32_t top_k;         /* k */
  int32_t causal;
  double sm_scale;
  const int64_t* seq_start; /* [B] first cache row of each sequence */
  const int32_t* seq_len;   /* [B] valid tokens, including the T query tokens */
  const uint16_t* k_cache;  /* bf16 [rows][Hkv][D] with the strides below (elements) */
  const uint16_t* v_cache;
  int64_t kv_token_stride, kv_head_stride;
  const uint16_t* idx_k_cache; /* bf16 [rows][d_idx] */
  int64_t idx_token_stride;
  /* optional paging: position s of sequence b lives in block block_table[b][s / block_size] */
  const int32_t* block_table; /* [B][max_blocks_per_seq] or NULL (contiguous sequences) */
  int32_t block_size, max_blocks_per_seq;
} oracle_problem;

static double bf16_to_double(uint16_t h) {
  uint32_t u = ((uint32_t)h) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

/* cache row that holds position s of sequence b */
static int64_t cache_row(const oracle_problem* p, int b, int64_t s) {
  if (p->block_table == NULL) return p->seq_start[b] + s;
  const int64_t block = p->block_table[(int64_t)b * p->max_blocks_per_seq + s / p->block_size];
  return block * p->block_size + s % p->block_size;
}

/* number of cached tokens query t of sequence b may attend to */
static int64_t visible_tokens(const oracle_problem* p, int b, int t) {
  int64_t n = p->seq_len[b];
  return p->causal ? n - p->q_per_seq + t + 1 : n;
}

int64_t oracle_visible(const oracle_problem* p, int32_t b, int32_t t) { return visible_tokens(p, b, t); }

/* Eq. 3 (scores): I[b,t,s] = sum_j q_idx[b,t,j] * K_idx[seq_start[b]+s, j], s < visible.
 * scores is [B][T][score_stride] doubles; entries at s >= visible are left untouched. */
void oracle_index_scores(const oracle_problem* p, const uint16_t* q_idx, double* scores, int64_t score_stride) {
  const int B = p->num_seqs, T = p->q_per_seq, d = p->idx_dim;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
  for (int b = 0; b < B; ++b) {
    for (int t = 0; t < T; ++t) {
      const uint16_t* q = q_idx + ((int64_t)b * T + t) * d;
      double* out = scores + ((int64_t)b * T + t) * score_stride;
      const int64_t v = visible_tokens(p, b, t);
      for (int64_t s = 0; s < v; ++s) {
        const uint16_t* key = p->idx_k_cache + cache_row(p, b, s) * p->idx_token_stride;
        double acc = 0.0;
        for (int j = 0; j < d; ++j) acc += bf16_to_double(q[j]) * bf16_to_double(key[j]);
        out[s] = acc;
      }
    }
  }
}

/* ------------------------------------------------------------------------------------------
 * Eq. 3 (TopK), selector 1: full sort of the positions by (score descending, position ascending).
 * qsort is not stable, but the comparator is a strict total order, so the result is unique.
 * idx_out has k entries; entries >= count are -1. */
static const double* g_sort_scores; /* per-thread pointer used by the comparator */
#pragma omp threadprivate(g_sort_scores)

static int cmp_desc_then_index(const void* a, const void* b) {
  const int32_t ia = *(const int32_t*)a, ib = *(const int32_t*)b;
  const double sa = g_sort_scores[ia], sb = g_sort_scores[ib];
  if (sa > sb) return -1;
  if (sa < sb) return 1;
  return (ia > ib) - (ia < ib);
}

void oracle_topk_row_sort(const double* scores, int64_t visible, int32_t k, int32_t* idx_out, int32_t* count_out) {
  int32_t* order = (int32_t*)malloc(sizeof(int32_t) * (size_t)(visible > 0 ? visible : 1));
  for (int64_t s = 0; s < visible; ++s) order[s] = (int32_t)s;
  g_sort_scores = scores;
  qsort(order, (size_t)visible, sizeof(int32_t), cmp_desc_then_index);
  const int32_t c = (int32_t)(visible < k ? visible : k);
  for (int32_t i = 0; i < c; ++i) idx_out[i] = order[i];
  for (int32_t i = c; i < k; ++i) idx_out[i] = -1;
  *count_out = c;
  free(order);
}

/* Selector 2, written independently: find the k-th best (score, position) pair by repeated
 * three-way partitioning, then emit everything strictly better plus the pivot class. Used to
 * cross-check selector 1 and as the timed CPU selection. Output order: ascending position. */
static int better(double sa, int32_t ia, double sb, int32_t ib) { /* a ranks strictly before b */
  return sa > sb || (sa == sb && ia < ib);
}

void oracle_topk_row_select(const double* scores, int64_t visible, int32_t k, int32_t* idx_out, int32_t* count_out) {
  const int32_t c = (int32_t)(visible < k ? visible : k);
  *count_out = c;
  for (int32_t i = c; i < k; ++i) idx_out[i] = -1;
  if (c == 0) return;
  int32_t* cand = (int32_t*)malloc(sizeof(int32_t) * (size_t)visible);
  int32_t* tmp = (int32_t*)malloc(sizeof(int32_t) * (size_t)visible);
  int64_t m = visible;
  for (int64_t s = 0; s < visible; ++s) cand[s] = (int32_t)s;
  int32_t need = c;       /* how many more to take from cand[0..m) */
  double thr_s = 0.0;     /* the c-th best pair once found */
  int32_t thr_i = -1;
  uint64_t rng = 0x9E3779B97F4A7C15ull;
  while (1) {
    rng = rng * 6364136223846793005ull + 1442695040888963407ull;
    const int32_t piv = cand[(int64_t)((rng >> 33) % (uint64_t)m)];
    const double ps = scores[piv];
    int64_t nb = 0, nw = 0; /* better-than-pivot go to the front of tmp, worse to the back */
    for (int64_t i = 0; i < m; ++i) {
      const int32_t x = cand[i];
      if (x == piv) continue;
      if (better(scores[x], x, ps, piv)) tmp[nb++] = x; else tmp[m - 1 - nw++] = x;
    }
    if (nb == need - 1) { thr_s = ps; thr_i = piv; break; }
    if (nb >= need) { memcpy(cand, tmp, sizeof(int32_t) * (size_t)nb); m = nb; }
    else { need -= (int32_t)(nb + 1); memcpy(cand, tmp + (m - nw), sizeof(int32_t) * (size_t)nw); m = nw; }
  }
  int32_t w = 0;
  for (int64_t s = 0; s < visible; ++s)
    if (!better(thr_s, thr_i, scores[s], (int32_t)s)) idx_out[w++] = (int32_t)s; /* s ranks at or before the threshold pair */
  free(cand);
  free(tmp);
}

/* TopK for every (sequence, query token). selector: 0 = full sort, 1 = partition select. */
void oracle_topk(const oracle_problem* p, const double* scores, int64_t score_stride, int32_t selector,
                 int32_t* idx, int32_t* count) {
  const int B = p->num_seqs, T = p->q_per_seq, k = p->top_k;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
  for (int b = 0; b < B; ++b)
    for (int t = 0; t < T; ++t) {
      const int64_t r = (int64_t)b * T + t;
      if (selector == 0) oracle_topk_row_sort(scores + r * score_stride, visible_tokens(p, b, t), k, idx + r * k, count + r);
      else oracle_topk_row_select(scores + r * score_stride, visible_tokens(p, b, t), k, idx + r * k, count + r);
    }
}

/* ------------------------------------------------------------------------------------------
 * Eq. 4: for each sequence b, query t, head h (KV head g = h / (Hq/Hkv)):
 *   z_s = sm_scale * sum_d Q[b,t,h,d] K[seq_start[b]+s, g, d]   for s in S_{b,t}
 *   m = max z_s; w_s = exp(z_s - m); O[d] = sum_s w_s V[.., g, d] / sum_s w_s; lse = m + log sum_s w_s
 * q is one layer's queries, bf16 [B][T][Hq][D]; out is double [B][T][Hq][D]; lse double [B][T][Hq] or NULL.
 * A row with count 0 yields O = 0 and lse = -inf. */
void oracle_sparse_attn(const oracle_problem* p, const uint16_t* q, const int32_t* idx, const int32_t* count,
                        double* out, double* lse) {
  const int B = p->num_seqs, T = p->q_per_seq, Hq = p->num_q_heads, D = p->head_dim, k = p->top_k;
  const int G = Hq / p->num_kv_heads;
#pragma omp parallel for collapse(3) schedule(dynamic, 1)
  for (int b = 0; b < B; ++b)
    for (int t = 0; t < T; ++t)
      for (int h = 0; h < Hq; ++h) {
        const int64_t r = (int64_t)b * T + t;
        const int32_t c = count[r];
        const int32_t* sel = idx + r * k;
        const uint16_t* qv = q + (r * Hq + h) * D;
        const int g = h / G;
        double* o = out + (r * Hq + h) * D;
        for (int d = 0; d < D; ++d) o[d] = 0.0;
        if (c <= 0) { if (lse) lse[r * Hq + h] = -INFINITY; continue; }
        double* z = (double*)malloc(sizeof(double) * (size_t)c);
        double m = -INFINITY;
        for (int32_t i = 0; i < c; ++i) {
          const uint16_t* kr = p->k_cache + cache_row(p, b, sel[i]) * p->kv_token_stride + g * p->kv_head_stride;
          double acc = 0.0;
          for (int d = 0; d < D; ++d) acc += bf16_to_double(qv[d]) * bf16_to_double(kr[d]);
          z[i] = p->sm_scale * acc;
          if (z[i] > m) m = z[i];
        }
        double denom = 0.0;
        for (int32_t i = 0; i < c; ++i) {
          const double w = exp(z[i] - m);
          const uint16_t* vr = p->v_cache + cache_row(p, b, sel[i]) * p->kv_token_stride + g * p->kv_head_stride;
          denom += w;
          for (int d = 0; d < D; ++d) o[d] += w * bf16_to_double(vr[d]);
        }
        for (int d = 0; d < D; ++d) o[d] /= denom;
        if (lse) lse[r * Hq + h] = m + log(denom);
        free(z);
      }
}

/* Eq. 1 restricted to the visible prefix: the same softmax-weighted mean, but looping directly
 * over cache rows s = 0..visible-1 with no index array and a two-pass softmax written separately
 * from the routine above. Used only for the "k >= n reduces to dense attention" check. */
void oracle_dense_attn(const oracle_problem* p, const uint16_t* q, double* out, double* lse) {
  const int B = p->num_seqs, T = p->q_per_seq, Hq = p->num_q_heads, D = p->head_dim;
  const int G = Hq / p->num_kv_heads;
  for (int b = 0; b < B; ++b)
    for (int t = 0; t < T; ++t) {
      const int64_t v = visible_tokens(p, b, t);
      for (int h = 0; h < Hq; ++h) {
        const int64_t r = ((int64_t)b * T + t) * Hq + h;
        const uint16_t* qv = q + r * D;
        const int64_t head_off = (int64_t)(h / G) * p->kv_head_stride;
        double* logits = (double*)malloc(sizeof(double) * (size_t)(v > 0 ? v : 1));
        double top = -INFINITY;
        for (int64_t s = 0; s < v; ++s) {
          const uint16_t* kr = p->k_cache + cache_row(p, b, s) * p->kv_token_stride + head_off;
          double dot = 0.0;
          for (int d = 0; d < D; ++d) dot += bf16_to_double(kr[d]) * bf16_to_double(qv[d]);
          logits[s] = dot * p->sm_scale;
          if (logits[s] > top) top = logits[s];
        }
        double total = 0.0;
        for (int64_t s = 0; s < v; ++s) { logits[s] = exp(logits[s] - top); total += logits[s]; }
        for (int d = 0; d < D; ++d) {
          double acc = 0.0;
          for (int64_t s = 0; s < v; ++s)
            acc += (logits[s] / total) *
                   bf16_to_double(p->v_cache[cache_row(p, b, s) * p->kv_token_stride + head_off + d]);
          out[r * D + d] = acc;
        }
        if (lse) lse[r] = v > 0 ? top + log(total) : -INFINITY;
        free(logits);
      }
    }
}

/* One decode step (Sec. 2.1): scores and TopK once, then the SAME idx/count arrays feed all
 * L layers. q_layers is bf16 [L][B][T][Hq][D]; out is double [L][B][T][Hq][D]; lse [L][B][T][Hq] or NULL.
 * scores_scratch is [B][T][score_stride] doubles. */
void oracle_decode_step(const oracle_problem* p, int32_t num_layers, const uint16_t* q_idx, const uint16_t* q_layers,
                        double* scores_scratch, int64_t score_stride, int32_t* idx, int32_t* count,
                        double* out, double* lse) {
  oracle_index_scores(p, q_idx, scores_scratch, score_stride);
  oracle_topk(p, scores_scratch, score_stride, 0, idx, count);
  const int64_t per_layer = (int64_t)p->num_seqs * p->q_per_seq * p->num_q_heads;
  for (int32_t l = 0; l < num_layers; ++l)
    oracle_sparse_attn(p, q_layers + l * per_layer * p->head_dim, idx, count, out + l * per_layer * p->head_dim,
                       lse ? lse + l * per_layer : NULL);
}

/* ------------------------------------------------------------------------------------------
 * Eq. 2 and the cache append. Weights are stored one output feature per row: w is bf16
 * [n_out][d_model], so y[m][o] = sum_j h[m][j] * w[o][j]  (y = h W with W = w^T). */
void oracle_linear(const uint16_t* h, const uint16_t* w, int64_t rows, int64_t n_out, int64_t d_model, double* y) {
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < rows; ++m)
    for (int64_t o = 0; o < n_out; ++o) {
      double acc = 0.0;
      for (int64_t j = 0; j < d_model; ++j) acc += bf16_to_double(h[m * d_model + j]) * bf16_to_double(w[o * d_model + j]);
      y[m * n_out + o] = acc;
    }
}

/* Nearest bf16 (8 significant bits, exponent range of binary32), ties to the even significand, rounded
 * ONCE from the double (going through binary32 first would round twice). */
uint16_t oracle_bf16_from_double(double x) {
  if (isnan(x)) return 0x7FC0;
  const uint16_t sign = signbit(x) ? 0x8000 : 0;
  double a = fabs(x), r;
  if (a == 0.0) return sign;
  if (isinf(a)) return sign | 0x7F80;
  int e;
  (void)frexp(a, &e);                         /* a = m * 2^e, m in [0.5, 1) */
  if (e - 1 < -126) r = ldexp(nearbyint(ldexp(a, 133)), -133);   /* subnormal grid: multiples of 2^-133 */
  else r = ldexp(nearbyint(ldexp(a, 8 - e)), e - 8);             /* 8 significant bits; nearbyint = ties-to-even */
  if (r >= ldexp(1.0, 128)) return sign | 0x7F80;
  const float f = (float)r;                   /* exact: r is a bf16 number */
  uint32_t u;
  memcpy(&u, &f, sizeof u);
  return sign | (uint16_t)(u >> 16);
}

void oracle_round_bf16(const double* x, int64_t n, uint16_t* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = oracle_bf16_from_double(x[i]);
}

/* For query token t of sequence b (position s = n_b - T + t, the sequence's newest tokens), with
 * h bf16 [B][T][d_model]:
 *   q_idx_out[b][t][:]            = bf16(h W^Q_idx)                        (Eq. 2)
 *   K_idx cache row of (b, s)     = bf16(h W^K_idx)                        (Eq. 2)
 *   K / V cache rows of (b, s)    = bf16(h W^K), bf16(h W^V), laid out [Hkv][D]   (skipped when w_k is NULL)
 * The caches of `p` are written in place; no other row is touched. */
void oracle_project_append(const oracle_problem* p, int32_t d_model, const uint16_t* h, const uint16_t* w_q_idx,
                           const uint16_t* w_k_idx, const uint16_t* w_k, const uint16_t* w_v, uint16_t* q_idx_out) {
  const int B = p->num_seqs, T = p->q_per_seq, d = p->idx_dim, Hkv = p->num_kv_heads, D = p->head_dim;
  double* y = (double*)malloc(sizeof(double) * (size_t)(Hkv * D > d ? Hkv * D : d));
  for (int b = 0; b < B; ++b)
    for (int t = 0; t < T; ++t) {
      const uint16_t* hv = h + ((int64_t)b * T + t) * d_model;
      const int64_t row = cache_row(p, b, (int64_t)p->seq_len[b] - T + t);
      oracle_linear(hv, w_q_idx, 1, d, d_model, y);
      oracle_round_bf16(y, d, q_idx_out + ((int64_t)b * T + t) * d);
      oracle_linear(hv, w_k_idx, 1, d, d_model, y);
      oracle_round_bf16(y, d, (uint16_t*)p->idx_k_cache + row * p->idx_token_stride);
      if (w_k == NULL) continue;
      oracle_linear(hv, w_k, 1, (int64_t)Hkv * D, d_model, y);
      for (int g = 0; g < Hkv; ++g)
        oracle_round_bf16(y + (int64_t)g * D, D, (uint16_t*)p->k_cache + row * p->kv_token_stride + g * p->kv_head_stride);
      oracle_linear(hv, w_v, 1, (int64_t)Hkv * D, d_model, y);
      for (int g = 0; g < Hkv; ++g)
        oracle_round_bf16(y + (int64_t)g * D, D, (uint16_t*)p->v_cache + row * p->kv_token_stride + g * p->kv_head_stride);
    }
  free(y);
}

int32_t oracle_num_threads(void) {
#ifdef _OPENMP
  extern int omp_get_max_threads(void);
  return omp_get_max_threads();
#else
  return 1;
#endif
}
