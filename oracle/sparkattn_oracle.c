/*
 * CPU oracle for the block-sparse attention path.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the plain, slow, obviously-correct statement of what the path
 * computes.  Only tests, the smoke check and the benchmark's CPU-baseline leg
 * may call it; the product (the CUDA library) never does, and the two share no
 * code.  Build: gcc -O2 -fopenmp -ffp-contract=off -shared -fPIC (no fast-math).
 *
 * Parity status: every function below is pinned by tests that do not re-use
 * its own formula (dense library attention, closed forms, exact rational
 * arithmetic, brute-force nearest-value search, a library FP8 cast).
 *
 *   ATT-0  oracle_attention   exact softmax attention restricted to the kept
 *                             query-block x key-block pairs, fp64
 *                             (paper Sec. 2 "Block sparsity" + the dense
 *                             attention formula there; Sec. 4.1, sparse branch
 *                             O_s = A_M(Q,K,V)).
 *   SEL-1  oracle_select      pooled-block scores + top-k (Sec. 2 lists kinds of
 *                             selectors, top-k over per-block scores among
 *                             them, but fixes no rule; the rule used
 *                             here is spelled out step by step below).
 *   QNT-1  oracle_quant_fp8   per-(head, token-block) absmax scale + E4M3
 *                             round-to-nearest-even encode (Sec. 4.3 names FP8
 *                             E4M3 with scale-and-cast in one pass);
 *          oracle_quant_fp8_per_token   the same with one scale per token.
 *   CMP-0  oracle_comp_state / oracle_comp_apply   low-rank compensation branch and
 *                             token-wise gate fusion (Sec. 4.1), fp64.
 *   WIN-0  frame_tokens / window arguments of oracle_attention and oracle_select:
 *                             the causal window of the auto-regressive extension
 *                             (Sec. 1, the auto-regressive extension: the attention
 *                             may be limited to a causal window;
 *                             no formula is given).  Reading: tokens come in frames of
 *                             F = frame_tokens; key j counts for query i iff
 *                             j / F lies in (i / F - window, i / F].  Selection only
 *                             ranks the key blocks that hold such a key for some row
 *                             of the query block.
 *   ORD-0  block_valid argument of oracle_attention, oracle_pool and oracle_select: tokens
 *                             stored in bricks padded to whole blocks (block b holds
 *                             block_valid[b] tokens followed by padding rows).  The paper
 *                             only says that blocks are contiguous (Sec. 2) and fixes no
 *                             token order; reading: padding rows are not keys, do not
 *                             enter the pooled means, and their query rows are not
 *                             evaluated.  The brick order itself is index arithmetic in
 *                             the Python front-end.
 *
 * OpenMP only distributes independent work items (one (head, query block) or
 * one (head, block) each); inside an item everything is a scalar loop in the
 * order written.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ---------- exact widening of the storage formats ---------- */

static inline float bf16_to_f32(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}

/* OCP FP8 E4M3 (the "FN" flavour): 1 sign, 4 exponent (bias 7), 3 mantissa
 * bits; no infinities; S.1111.111 is NaN; exponent field 0 is subnormal
 * (m * 2^-9).  Written from the bit-field definition. */
double oracle_e4m3_decode(uint8_t c) {
  int s = c >> 7, e = (c >> 3) & 0xF, m = c & 7;
  double v;
  if (e == 15 && m == 7) return NAN;
  if (e == 0) v = ldexp((double)m, -9);
  else v = ldexp(1.0 + (double)m / 8.0, e - 7);
  return s ? -v : v;
}

/* Round-to-nearest (ties to even mantissa), saturating to +-448, sign kept on
 * zero and on underflow.  y is an fp32 value; all steps below are exact in
 * fp64 except rint(), which is the one rounding the format asks for. */
uint8_t oracle_e4m3_encode(float y) {
  uint32_t bits;
  memcpy(&bits, &y, 4);
  uint8_t sign = (uint8_t)((bits >> 31) << 7);
  if (isnan(y)) return (uint8_t)(sign | 0x7F);
  double a = fabs((double)y);
  if (a >= 448.0) return (uint8_t)(sign | 0x7E);
  if (a < ldexp(1.0, -6)) {
    /* subnormal grid k * 2^-9, k = 0..8 (k = 8 is the smallest normal, code 0x08) */
    int k = (int)rint(ldexp(a, 9));
    return (uint8_t)(sign | k);
  }
  int e;
  double f = frexp(a, &e); /* a = f * 2^e, f in [0.5, 1) */
  e -= 1;                  /* a = (2f) * 2^e, 2f in [1, 2) */
  int q = (int)rint((2.0 * f - 1.0) * 8.0); /* 0..8 */
  if (q == 8) { q = 0; e += 1; }
  int code = ((e + 7) << 3) | q;
  if (code > 0x7E) code = 0x7E;
  return (uint8_t)(sign | code);
}

/* element (h, n, c) of a [H][N][d] tensor stored as bf16 (dtype 0) or as E4M3
 * codes with one fp32 scale per (h, n / blk) (dtype 1), widened exactly. */
static inline double load_elem(const void* x, const float* scale, int dtype, int64_t N, int d, int blk,
                               int64_t nb, int64_t h, int64_t n, int c) {
  int64_t off = (h * N + n) * d + c;
  if (dtype == 0) return (double)bf16_to_f32(((const uint16_t*)x)[off]);
  return oracle_e4m3_decode(((const uint8_t*)x)[off]) * (double)scale[h * nb + n / blk];
}

/* ---------- ATT-0 ---------- */
/*
 * For query token i of head h, with qb = i / blk and the kept list
 * L = kept_idx[h, qb, 0 .. kept_cnt[h, qb]):
 *     J   = { j < N : j / blk in L }
 *     s_j = scale * sum_c q[i,c] k[j,c]
 *     p_j = exp(s_j - max_J s) ;  l = sum_J p_j
 *     o   = (sum_J p_j v[j,:]) / l ;  lse = max_J s + ln l
 * An empty J gives o = 0 and lse = -inf.
 *
 * items: n_items pairs (h, qb) to evaluate; out [n_items][blk][d] and
 * lse [n_items][blk] (rows of a ragged tail block beyond N are left at 0).
 * H-major tensors: q,k,v are [H][N][d]; kept_idx [H][nb][kmax]; kept_cnt [H][nb].
 */
int oracle_attention(int dtype, const void* q, const void* k, const void* v, const float* q_scale,
                     const float* k_scale, const float* v_scale, int H, int N, int d, int blk,
                     const int32_t* kept_idx, const int32_t* kept_cnt, int kmax, double scale,
                     const int32_t* items, int n_items, int frame_tokens, int window,
                     const int32_t* block_valid /* [nb] or NULL */, double* out, double* lse) {
  const int64_t nb = ((int64_t)N + blk - 1) / blk;
  if (scale == 0.0) scale = 1.0 / sqrt((double)d);
  int bad = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (int it = 0; it < n_items; ++it) {
    const int h = items[2 * it], qb = items[2 * it + 1];
    const int cnt = kept_cnt[(int64_t)h * nb + qb];
    const int32_t* list = kept_idx + ((int64_t)h * nb + qb) * kmax;
    double* s = (double*)malloc(sizeof(double) * (size_t)(cnt > 0 ? cnt : 1) * blk);
    int64_t* key = (int64_t*)malloc(sizeof(int64_t) * (size_t)(cnt > 0 ? cnt : 1) * blk);
    double* qrow = (double*)malloc(sizeof(double) * d);
    for (int r = 0; r < blk; ++r) {
      const int64_t i = (int64_t)qb * blk + r;
      double* o = out + ((int64_t)it * blk + r) * d;
      for (int c = 0; c < d; ++c) o[c] = 0.0;
      lse[(int64_t)it * blk + r] = 0.0;
      if (i >= N) continue;
      if (block_valid && r >= block_valid[qb]) continue;       /* ORD-0: a padding row */
      for (int c = 0; c < d; ++c) qrow[c] = load_elem(q, q_scale, dtype, N, d, blk, nb, h, i, c);
      int64_t nk = 0;
      double m = -INFINITY;
      for (int t = 0; t < cnt; ++t) {
        const int64_t kb = list[t];
        if (kb < 0 || kb >= nb) { bad = 1; continue; }
        const int64_t jend = kb * blk + (block_valid ? block_valid[kb] : blk);    /* ORD-0: padding rows are not keys */
        for (int64_t j = kb * blk; j < jend && j < N; ++j) {
          /* causal window over frames (WIN-0): key frame in (query frame - window, query frame] */
          if (frame_tokens > 0) {
            const int64_t fi = i / frame_tokens, fj = j / frame_tokens;
            if (fj > fi || fj <= fi - window) continue;
          }
          double acc = 0.0;
          for (int c = 0; c < d; ++c) acc += qrow[c] * load_elem(k, k_scale, dtype, N, d, blk, nb, h, j, c);
          s[nk] = scale * acc;
          key[nk] = j;
          if (s[nk] > m) m = s[nk];
          ++nk;
        }
      }
      if (nk == 0) { lse[(int64_t)it * blk + r] = -INFINITY; continue; }
      double l = 0.0;
      for (int64_t a = 0; a < nk; ++a) {
        const double p = exp(s[a] - m);
        l += p;
        for (int c = 0; c < d; ++c) o[c] += p * load_elem(v, v_scale, dtype, N, d, blk, nb, h, key[a], c);
      }
      for (int c = 0; c < d; ++c) o[c] /= l;
      lse[(int64_t)it * blk + r] = m + log(l);
    }
    free(s); free(key); free(qrow);
  }
  return bad ? -1 : 0;
}

/* ---------- SEL-1 ---------- */
/*
 * Step 1  pooled sum, fp32, tokens in ascending order:
 *             sum[c] = 0 ; for t in block (valid tokens only): sum[c] = sum[c] + x[t,c]
 * Step 2  pooled mean: p[c] = sum[c] / (float)n_valid          (IEEE fp32 divide)
 * Step 3  score(i,j): a = 0 ; for c ascending: a = fmaf(pq[i,c], pk[j,c], a)
 * Step 4  keep the topk key blocks that come first under
 *             (score descending, then block index ascending)
 * Step 5  write the kept indices in ascending index order.
 * The 1/sqrt(d) factor is omitted: it does not change the ranking.
 */
void oracle_pool(const uint16_t* x, int H, int N, int d, int blk, const int32_t* block_valid /* [nb] or NULL */,
                 float* pooled /* [H][nb][d] */) {
  const int64_t nb = ((int64_t)N + blk - 1) / blk;
#pragma omp parallel for schedule(static)
  for (int64_t hb = 0; hb < (int64_t)H * nb; ++hb) {
    const int64_t h = hb / nb, b = hb % nb;
    int64_t t0 = b * blk, t1 = (t0 + blk < N) ? t0 + blk : N;
    if (block_valid && t0 + block_valid[b] < t1) t1 = t0 + block_valid[b];      /* ORD-0: valid tokens only */
    for (int c = 0; c < d; ++c) {
      float sum = 0.0f;
      for (int64_t t = t0; t < t1; ++t) sum = sum + bf16_to_f32(x[(h * N + t) * d + c]);
      pooled[hb * d + c] = sum / (float)(t1 - t0);
    }
  }
}

typedef struct { float s; int32_t j; } scored_t;
static int scored_cmp(const void* a, const void* b) {
  const scored_t* x = (const scored_t*)a; const scored_t* y = (const scored_t*)b;
  if (x->s > y->s) return -1;
  if (x->s < y->s) return 1;
  return (x->j > y->j) - (x->j < y->j);
}
static int dcmp(const void* x, const void* y) {
  double u = *(const double*)x, v = *(const double*)y;
  return (u > v) - (u < v);
}
static int int_cmp(const void* a, const void* b) {
  int32_t x = *(const int32_t*)a, y = *(const int32_t*)b;
  return (x > y) - (x < y);
}

/* scores_out (optional, may be NULL): [H][nb][nb] fp32 scores, for inspection in tests. */
int oracle_select(const uint16_t* q, const uint16_t* k, int H, int N, int d, int blk, int topk,
                  int frame_tokens, int window, const int32_t* block_valid /* [nb] or NULL */,
                  int32_t* kept_idx /* [H][nb][topk] */, int32_t* kept_cnt /* [H][nb] or NULL */,
                  float* scores_out) {
  const int64_t nb = ((int64_t)N + blk - 1) / blk;
  if (topk < 1 || topk > nb) return -1;
  float* pq = (float*)malloc(sizeof(float) * (size_t)H * nb * d);
  float* pk = (float*)malloc(sizeof(float) * (size_t)H * nb * d);
  oracle_pool(q, H, N, d, blk, block_valid, pq);
  oracle_pool(k, H, N, d, blk, block_valid, pk);
#pragma omp parallel for schedule(static)
  for (int64_t hi = 0; hi < (int64_t)H * nb; ++hi) {
    const int64_t h = hi / nb;
    scored_t* sc = (scored_t*)malloc(sizeof(scored_t) * nb);
    for (int64_t j = 0; j < nb; ++j) {
      float a = 0.0f;
      for (int c = 0; c < d; ++c) a = fmaf(pq[hi * d + c], pk[(h * nb + j) * d + c], a);
      sc[j].s = a;
      sc[j].j = (int32_t)j;
      if (scores_out) scores_out[hi * nb + j] = a;
    }
    /* WIN-0: with a causal window only the key blocks that hold at least one key some row of the
     * query block may attend to are candidates: a contiguous run [jlo, jhi] of block indices. */
    int64_t jlo = 0, jhi = nb - 1;
    if (frame_tokens > 0) {
      const int64_t qb = hi % nb;
      const int64_t r0 = qb * blk, r1 = ((qb + 1) * blk < N ? (qb + 1) * blk : N) - 1;
      int64_t f0 = r0 / frame_tokens - window + 1;
      if (f0 < 0) f0 = 0;
      int64_t kend = (r1 / frame_tokens + 1) * frame_tokens;
      if (kend > N) kend = N;
      jlo = f0 * frame_tokens / blk;
      jhi = (kend - 1) / blk;
    }
    const int64_t ncand = jhi - jlo + 1;
    qsort(sc + jlo, ncand, sizeof(scored_t), scored_cmp);
    const int cnt = topk < ncand ? topk : (int)ncand;
    int32_t* dst = kept_idx + hi * topk;
    for (int t = 0; t < cnt; ++t) dst[t] = sc[jlo + t].j;
    qsort(dst, cnt, sizeof(int32_t), int_cmp);
    for (int t = cnt; t < topk; ++t) dst[t] = -1;     /* unused tail of the list */
    if (kept_cnt) kept_cnt[hi] = cnt;
    free(sc);
  }
  free(pq); free(pk);
  return 0;
}

/* Diagnostic: the same rule evaluated in fp64 (pooled means and scores in
 * double).  Returns the number of (head, query-block) rows whose fp64 kept set
 * differs from `kept_idx`, and through min_rel_gap the smallest relative gap
 * between the topk-th and (topk+1)-th fp64 scores over all rows. */
int64_t oracle_select_f64_diff(const uint16_t* q, const uint16_t* k, int H, int N, int d, int blk, int topk,
                               const int32_t* kept_idx, double* min_rel_gap) {
  const int64_t nb = ((int64_t)N + blk - 1) / blk;
  double* pq = (double*)malloc(sizeof(double) * (size_t)H * nb * d);
  double* pk = (double*)malloc(sizeof(double) * (size_t)H * nb * d);
  for (int w = 0; w < 2; ++w) {
    const uint16_t* x = w ? k : q; double* p = w ? pk : pq;
    for (int64_t hb = 0; hb < (int64_t)H * nb; ++hb) {
      const int64_t h = hb / nb, b = hb % nb;
      const int64_t t0 = b * blk, t1 = (t0 + blk < N) ? t0 + blk : N;
      for (int c = 0; c < d; ++c) {
        double sum = 0.0;
        for (int64_t t = t0; t < t1; ++t) sum += (double)bf16_to_f32(x[(h * N + t) * d + c]);
        p[hb * d + c] = sum / (double)(t1 - t0);
      }
    }
  }
  int64_t ndiff = 0; double gap = INFINITY;
  double* s = (double*)malloc(sizeof(double) * nb);
  double* srt = (double*)malloc(sizeof(double) * nb);
  for (int64_t hi = 0; hi < (int64_t)H * nb; ++hi) {
    const int64_t h = hi / nb;
    for (int64_t j = 0; j < nb; ++j) {
      double a = 0.0;
      for (int c = 0; c < d; ++c) a += pq[hi * d + c] * pk[(h * nb + j) * d + c];
      s[j] = a; srt[j] = a;
    }
    /* sort the negated copy ascending = scores descending */
    for (int64_t a = 0; a < nb; ++a) srt[a] = -srt[a];
    qsort(srt, nb, sizeof(double), dcmp);
    const double kth = -srt[topk - 1];
    if (topk < nb) {
      const double nxt = -srt[topk];
      const double g = (kth - nxt) / (fabs(kth) > 1e-300 ? fabs(kth) : 1e-300);
      if (g < gap) gap = g;
    }
    /* kept set under fp64: all j with s[j] > kth, plus lowest-index ties */
    int differs = 0, ngreater = 0;
    for (int64_t j = 0; j < nb; ++j) ngreater += (s[j] > kth);
    int ties_allowed = topk - ngreater;
    const int32_t* list = kept_idx + hi * topk;
    int t = 0;
    for (int64_t j = 0; j < nb; ++j) {
      int keep = 0;
      if (s[j] > kth) keep = 1;
      else if (s[j] == kth && ties_allowed > 0) { keep = 1; --ties_allowed; }
      int listed = (t < topk && list[t] == j);
      if (listed) ++t;
      if (keep != listed) differs = 1;
    }
    ndiff += differs;
  }
  free(s); free(srt); free(pq); free(pk);
  if (min_rel_gap) *min_rel_gap = gap;
  return ndiff;
}

/* ---------- QNT-1 ---------- */
/*
 * Per (head, token block) over the valid tokens x d channels:
 *   amax  = max |x|                       (exact)
 *   amax  = max(amax, 1e-12f)
 *   scale = amax / 448.0f ; inv = 448.0f / amax      (IEEE fp32 divides)
 *   code  = e4m3_rne_satfinite( (float)x * inv )     (one fp32 multiply, then the encode)
 * Dequantised value = decode(code) * scale.
 */
void oracle_quant_fp8(const uint16_t* x, int H, int N, int d, int blk, uint8_t* codes /* [H][N][d] */,
                      float* scales /* [H][nb] */) {
  const int64_t nb = ((int64_t)N + blk - 1) / blk;
#pragma omp parallel for schedule(static)
  for (int64_t hb = 0; hb < (int64_t)H * nb; ++hb) {
    const int64_t h = hb / nb, b = hb % nb;
    const int64_t t0 = b * blk, t1 = (t0 + blk < N) ? t0 + blk : N;
    float amax = 0.0f;
    for (int64_t t = t0; t < t1; ++t)
      for (int c = 0; c < d; ++c) {
        float a = fabsf(bf16_to_f32(x[(h * N + t) * d + c]));
        if (a > amax) amax = a;
      }
    if (amax < 1e-12f) amax = 1e-12f;
    const float scale = amax / 448.0f;
    const float inv = 448.0f / amax;
    scales[hb] = scale;
    for (int64_t t = t0; t < t1; ++t)
      for (int c = 0; c < d; ++c) {
        const float y = bf16_to_f32(x[(h * N + t) * d + c]) * inv;
        codes[(h * N + t) * d + c] = oracle_e4m3_encode(y);
      }
  }
}

/* Per-token variant (the granularity the paper's Sec. 4.3 states for activations: one dynamic
 * scale per token): the same QNT-1 steps with the block replaced by a single token row. */
void oracle_quant_fp8_per_token(const uint16_t* x, int H, int N, int d, uint8_t* codes /* [H][N][d] */,
                                float* scales /* [H][N] */) {
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < (int64_t)H * N; ++r) {
    float amax = 0.0f;
    for (int c = 0; c < d; ++c) {
      float a = fabsf(bf16_to_f32(x[r * d + c]));
      if (a > amax) amax = a;
    }
    if (amax < 1e-12f) amax = 1e-12f;
    const float scale = amax / 448.0f;
    const float inv = 448.0f / amax;
    scales[r] = scale;
    for (int c = 0; c < d; ++c) codes[r * d + c] = oracle_e4m3_encode(bf16_to_f32(x[r * d + c]) * inv);
  }
}

/* ---------- CMP-0: low-rank compensation branch and gate (paper Sec. 4.1) ---------- */
/*
 * For head h, token i at grid position (t, y, x) (raster order n = (t*Hg + y)*Wg + x):
 *   u      = P x                      P is [r][d] (P_q for queries, P_k for keys), x the token's q or k row
 *   a_m    = pos_{axis[m]}(i) * freq[m]                      m = 0 .. r/2-1   (rank-truncated 3-D RoPE)
 *   z      = silu(u) ,  silu(s) = s / (1 + exp(-s))
 *   x~[2m]   = z[2m] cos a_m - z[2m+1] sin a_m
 *   x~[2m+1] = z[2m] sin a_m + z[2m+1] cos a_m
 *   C      = sum_j k~_j v_j^T                                 [r][d] per head
 *   y_i    = q~_i^T C ;  O_lr,i = y_i / sqrt(mean_c y_i[c]^2 + eps)          (RMSNorm, no learned weight)
 *   r_i    = sqrt(mean_c O_s[i,c]^2)                          (RMS of the sparse-branch output row)
 *   O_i    = O_s,i + g_i * r_i * O_lr,i
 * Everything in fp64 from the stored bf16 inputs; nothing is rounded in between.
 */
static void comp_feature(const uint16_t* xrow, const uint16_t* P /* [r][d] */, int d, int r, const int32_t* axis,
                         const float* freq, const int pos[3], double* outv /* [r] */) {
  for (int a = 0; a < r; ++a) {
    double u = 0.0;
    for (int c = 0; c < d; ++c) u += (double)bf16_to_f32(P[a * d + c]) * (double)bf16_to_f32(xrow[c]);
    outv[a] = u / (1.0 + exp(-u));
  }
  for (int m = 0; m < r / 2; ++m) {
    const double ang = (double)pos[axis[m]] * (double)freq[m];
    const double cs = cos(ang), sn = sin(ang);
    const double z0 = outv[2 * m], z1 = outv[2 * m + 1];
    outv[2 * m] = z0 * cs - z1 * sn;
    outv[2 * m + 1] = z0 * sn + z1 * cs;
  }
}

/* state [H][r][d] fp64 ; k, v [H][N][d] bf16 ; pk [H][r][d] bf16 ; grid = (T, Hg, Wg) with T*Hg*Wg == N */
void oracle_comp_state(const uint16_t* k, const uint16_t* v, const uint16_t* pk, int H, int N, int d, int r,
                       const int32_t* grid, const int32_t* axis, const float* freq, double* state) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int h = 0; h < H; ++h) {
    double* C = state + (int64_t)h * r * d;
    double* kt = (double*)malloc(sizeof(double) * r);
    for (int64_t e = 0; e < (int64_t)r * d; ++e) C[e] = 0.0;
    for (int64_t j = 0; j < N; ++j) {
      const int pos[3] = {(int)(j / ((int64_t)grid[1] * grid[2])), (int)((j / grid[2]) % grid[1]), (int)(j % grid[2])};
      comp_feature(k + ((int64_t)h * N + j) * d, pk + (int64_t)h * r * d, d, r, axis, freq, pos, kt);
      for (int a = 0; a < r; ++a)
        for (int c = 0; c < d; ++c) C[a * d + c] += kt[a] * (double)bf16_to_f32(v[((int64_t)h * N + j) * d + c]);
    }
    free(kt);
  }
}

/* out [n_rows][d] fp64 for the listed (h, token) pairs ; o_sparse [H][N][d] bf16 ; gate [H][N] fp32 */
void oracle_comp_apply(const uint16_t* q, const uint16_t* pq, const double* state, const float* gate,
                       const uint16_t* o_sparse, int H, int N, int d, int r, const int32_t* grid,
                       const int32_t* axis, const float* freq, double eps, const int32_t* rows, int n_rows,
                       double* out) {
  (void)H;
#pragma omp parallel for schedule(static)
  for (int it = 0; it < n_rows; ++it) {
    const int h = rows[2 * it];
    const int64_t i = rows[2 * it + 1];
    const int pos[3] = {(int)(i / ((int64_t)grid[1] * grid[2])), (int)((i / grid[2]) % grid[1]), (int)(i % grid[2])};
    double* qt = (double*)malloc(sizeof(double) * r);
    double* y = (double*)malloc(sizeof(double) * d);
    comp_feature(q + ((int64_t)h * N + i) * d, pq + (int64_t)h * r * d, d, r, axis, freq, pos, qt);
    const double* C = state + (int64_t)h * r * d;
    double ss = 0.0, so = 0.0;
    for (int c = 0; c < d; ++c) {
      double acc = 0.0;
      for (int a = 0; a < r; ++a) acc += qt[a] * C[a * d + c];
      y[c] = acc;
      ss += acc * acc;
      const double os = (double)bf16_to_f32(o_sparse[((int64_t)h * N + i) * d + c]);
      so += os * os;
    }
    const double inv = 1.0 / sqrt(ss / d + eps);
    const double ri = sqrt(so / d);
    const double g = (double)gate[(int64_t)h * N + i];
    for (int c = 0; c < d; ++c)
      out[(int64_t)it * d + c] = (double)bf16_to_f32(o_sparse[((int64_t)h * N + i) * d + c]) + g * ri * y[c] * inv;
    free(qt); free(y);
  }
}

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}
