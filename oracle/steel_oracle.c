/*
 * CPU oracle for block-sparse fused attention.  TEST INFRASTRUCTURE ONLY: it is used by
 * the tests, by the smoke check and by the benchmark's CPU-baseline leg.  It is slow and
 * plain on purpose and shares no code with the CUDA path.
 *
 * What it computes (all arithmetic in fp64; inputs are bf16 bit patterns widened exactly):
 *
 *   steel_oracle_rows       Eq. 1 of the paper written out row by row with an explicit
 *                           dense mask row M (0 where a key is visible, -inf elsewhere):
 *                           O_i = softmax(scale * q_i K^T + M_i) V, LSE_i = ln sum_j
 *                           exp(scale * q_i.k_j + M_ij).  `scale` generalises 1/sqrt(d).
 *   steel_oracle_alg1_block the streaming form that Algorithm 1 of the paper describes, for one
 *                           query block: each row carries a running maximum, a running sum
 *                           and a rescaled accumulator through the key blocks, and only
 *                           blocks that are not fully masked are visited (Sec. "The STEEL
 *                           Pipeline", the three mask cases).  Used to pin that skipping
 *                           tiles gives the dense masked result.
 *   steel_oracle_classify   the three mask cases for one tile, by brute force over every
 *                           (query, key) pair of the tile.
 *
 * Mask predicate (the paper names causal and windowed masks; bitmap, GQA and the
 * S_q != S_kv alignment are this library's reading):
 *   allowed(h,i,j) = (!CAUSAL || j <= i + (S_kv - S_q))
 *                 && (!WINDOW || (i + (S_kv - S_q)) - j < W)
 *                 && (!BITMAP || bit[h][i / B_q][j / B_kv])
 * A query row with no visible key returns O = 0 and LSE = -inf.
 *
 * Parity pins (tests/test_oracle_pins.py): brute-force dense softmax on tiny inputs, rows
 * of P summing to 1 and vanishing where masked, closed forms (Q = 0, one visible key,
 * constant V), shift / scale / permutation invariances, GQA = repeated MHA, the library
 * routine torch scaled_dot_product_attention in fp64, and Algorithm 1 = Eq. 1.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_MASK_CAUSAL 1u
#define ORACLE_MASK_WINDOW 2u
#define ORACLE_MASK_BITMAP 4u

typedef struct {
  int32_t batch, heads_q, heads_kv, seq_q, seq_kv, head_dim;
  double scale;
  uint32_t flags;
  int32_t block_q, block_kv;
  int64_t window;
  const uint32_t *bitmap; /* [heads_q][T_q][ceil(T_kv/32)], bit (J & 31) of word J >> 5 */
} oracle_problem_t;

static double bf16_to_f64(uint16_t bits) {
  uint32_t w = (uint32_t)bits << 16;
  float f;
  memcpy(&f, &w, sizeof f);
  return (double)f;
}

static int ceil_div(int a, int b) { return (a + b - 1) / b; }

/* The mask predicate: is key j visible to query i of query head h? */
static int allowed(const oracle_problem_t *p, int h, int64_t i, int64_t j) {
  int64_t ipos = i + ((int64_t)p->seq_kv - (int64_t)p->seq_q);
  if ((p->flags & ORACLE_MASK_CAUSAL) && !(j <= ipos)) return 0;
  if ((p->flags & ORACLE_MASK_WINDOW) && !(ipos - j < p->window)) return 0;
  if (p->flags & ORACLE_MASK_BITMAP) {
    int t_q = ceil_div(p->seq_q, p->block_q), t_kv = ceil_div(p->seq_kv, p->block_kv);
    int words = ceil_div(t_kv, 32);
    int64_t I = i / p->block_q, J = j / p->block_kv;
    uint32_t word = p->bitmap[((int64_t)h * t_q + I) * words + (J >> 5)];
    if (!((word >> (J & 31)) & 1u)) return 0;
  }
  return 1;
}

int steel_oracle_allowed(const oracle_problem_t *p, int h, int64_t i, int64_t j) {
  return allowed(p, h, i, j);
}

/* Tile (I, J) of head h: 0 = fully masked (skipped), 1 = unmasked, 2 = partially masked. */
int steel_oracle_classify(const oracle_problem_t *p, int h, int I, int J) {
  int64_t i0 = (int64_t)I * p->block_q, j0 = (int64_t)J * p->block_kv;
  int64_t i1 = i0 + p->block_q, j1 = j0 + p->block_kv;
  if (i1 > p->seq_q) i1 = p->seq_q;
  if (j1 > p->seq_kv) j1 = p->seq_kv;
  int64_t visible = 0, total = (i1 - i0) * (j1 - j0);
  for (int64_t i = i0; i < i1; ++i)
    for (int64_t j = j0; j < j1; ++j) visible += allowed(p, h, i, j);
  if (visible == 0) return 0;
  return visible == total ? 1 : 2;
}

/* Kept and partial tile counts of every head, by brute force.  counts[2*h] = kept,
 * counts[2*h+1] = partial. */
void steel_oracle_count_tiles(const oracle_problem_t *p, int64_t *counts) {
  int t_q = ceil_div(p->seq_q, p->block_q), t_kv = ceil_div(p->seq_kv, p->block_kv);
#pragma omp parallel for schedule(dynamic)
  for (int h = 0; h < p->heads_q; ++h) {
    int64_t kept = 0, partial = 0;
    for (int I = 0; I < t_q; ++I)
      for (int J = 0; J < t_kv; ++J) {
        int c = steel_oracle_classify(p, h, I, J);
        kept += c != 0;
        partial += c == 2;
      }
    counts[2 * h] = kept;
    counts[2 * h + 1] = partial;
  }
}

/*
 * Eq. 1 for a list of rows.  rows[3*r + {0,1,2}] = (b, h, i).  Outputs: o[r][d], lse[r];
 * probs (optional, may be NULL) receives the full probability row P[r][seq_kv].
 */
void steel_oracle_rows(const oracle_problem_t *p, const uint16_t *q, const uint16_t *k,
                       const uint16_t *v, const int64_t *rows, int64_t n_rows, double *o,
                       double *lse, double *probs) {
  const int d = p->head_dim;
  const int64_t skv = p->seq_kv, sq = p->seq_q;
  const int group = p->heads_q / p->heads_kv;
#pragma omp parallel
  {
    double *a = (double *)malloc(sizeof(double) * (size_t)skv);
    double *qi = (double *)malloc(sizeof(double) * (size_t)d);
#pragma omp for schedule(dynamic, 1)
    for (int64_t r = 0; r < n_rows; ++r) {
      const int64_t b = rows[3 * r], h = rows[3 * r + 1], i = rows[3 * r + 2];
      const int64_t g = h / group;
      const uint16_t *qrow = q + ((b * p->heads_q + h) * sq + i) * d;
      const uint16_t *kbase = k + (b * p->heads_kv + g) * skv * d;
      const uint16_t *vbase = v + (b * p->heads_kv + g) * skv * d;
      double *orow = o + r * d;
      for (int c = 0; c < d; ++c) qi[c] = bf16_to_f64(qrow[c]);
      /* scores plus the explicit dense mask row */
      double mx = -INFINITY;
      for (int64_t j = 0; j < skv; ++j) {
        double s = 0.0;
        const uint16_t *krow = kbase + j * d;
        for (int c = 0; c < d; ++c) s += qi[c] * bf16_to_f64(krow[c]);
        double m_ij = allowed(p, (int)h, i, j) ? 0.0 : -INFINITY;
        a[j] = p->scale * s + m_ij;
        if (a[j] > mx) mx = a[j];
      }
      for (int c = 0; c < d; ++c) orow[c] = 0.0;
      if (mx == -INFINITY) { /* no visible key */
        lse[r] = -INFINITY;
        if (probs) for (int64_t j = 0; j < skv; ++j) probs[r * skv + j] = 0.0;
        continue;
      }
      double sum = 0.0;
      for (int64_t j = 0; j < skv; ++j) sum += exp(a[j] - mx);
      const double l = mx + log(sum);
      lse[r] = l;
      for (int64_t j = 0; j < skv; ++j) {
        double pj = exp(a[j] - l);
        if (probs) probs[r * skv + j] = pj;
        if (pj == 0.0) continue;
        const uint16_t *vrow = vbase + j * d;
        for (int c = 0; c < d; ++c) orow[c] += pj * bf16_to_f64(vrow[c]);
      }
    }
    free(a);
    free(qi);
  }
}

/*
 * Tile-skipping streaming softmax for query block I of (b, h): the check that Algorithm 1 (tiles,
 * running maximum, running sum, rescaled accumulator, skipped tiles) reproduces Eq. 1.  Written
 * row by row: each query row carries its own state (top = largest score seen, mass = sum of
 * 2^(score - top), acc = sum of 2^(score - top) * V) through the key blocks that the mask keeps.
 * Readings of the paper used here: the new maximum replaces the old one after the sum is updated;
 * the accumulator is rescaled and added to, not overwritten; the state starts at top = -inf,
 * mass = 0, acc = 0; scores carry the factor log2(e) and the exponent is base 2; while a row has
 * seen no visible key it adds nothing and rescales by 1.  A key block with no visible element for
 * the whole query block is skipped; any other block is masked element by element.
 * Outputs: o[B_q][d], lse[B_q] (natural log); returns the number of key blocks executed.
 */
int64_t steel_oracle_alg1_block(const oracle_problem_t *p, const uint16_t *q,
                                const uint16_t *k, const uint16_t *v, int b, int h, int I,
                                double *o, double *lse) {
  const int d = p->head_dim, bq = p->block_q, bkv = p->block_kv;
  const int64_t skv = p->seq_kv, sq = p->seq_q;
  const int group = p->heads_q / p->heads_kv, g = h / group;
  const int t_kv = ceil_div(p->seq_kv, bkv);
  const double log2e = 1.4426950408889634074, ln2 = 0.69314718055994530942;
  const uint16_t *qbase = q + (((int64_t)b * p->heads_q + h) * sq) * d;
  const uint16_t *kbase = k + (((int64_t)b * p->heads_kv + g) * skv) * d;
  const uint16_t *vbase = v + (((int64_t)b * p->heads_kv + g) * skv) * d;
  const int64_t i0 = (int64_t)I * bq;
  const int rows = (int)((i0 + bq <= sq) ? bq : sq - i0);

  /* which key blocks survive the skip rule, decided once for the whole query block */
  unsigned char *keep = (unsigned char *)malloc((size_t)t_kv);
  int64_t executed = 0;
  for (int J = 0; J < t_kv; ++J) {
    keep[J] = steel_oracle_classify(p, h, I, J) != 0;
    executed += keep[J];
  }

  double *score = (double *)malloc(sizeof(double) * (size_t)bkv);
  for (int r = 0; r < rows; ++r) {
    const int64_t i = i0 + r;
    double *acc = o + (int64_t)r * d;
    double top = -INFINITY, mass = 0.0;
    for (int c = 0; c < d; ++c) acc[c] = 0.0;
    for (int J = 0; J < t_kv; ++J) {
      if (!keep[J]) continue;
      const int64_t j0 = (int64_t)J * bkv;
      const int cols = (int)((j0 + bkv <= skv) ? bkv : skv - j0);
      /* scaled, masked scores of this row against the block, and their maximum */
      double block_top = -INFINITY;
      for (int cj = 0; cj < cols; ++cj) {
        double s = 0.0;
        for (int c = 0; c < d; ++c)
          s += bf16_to_f64(qbase[i * d + c]) * bf16_to_f64(kbase[(j0 + cj) * d + c]);
        s *= p->scale * log2e;
        if (!allowed(p, h, i, j0 + cj)) s = -INFINITY;
        score[cj] = s;
        if (s > block_top) block_top = s;
      }
      const double new_top = block_top > top ? block_top : top;
      const int blind = new_top == -INFINITY; /* nothing visible so far */
      /* move the state to the new maximum, then add this block's weights */
      const double shrink = blind ? 1.0 : exp2(top - new_top);
      double block_mass = 0.0;
      for (int c = 0; c < d; ++c) acc[c] *= shrink;
      for (int cj = 0; cj < cols; ++cj) {
        const double w = blind ? 0.0 : exp2(score[cj] - new_top);
        block_mass += w;
        if (w == 0.0) continue;
        for (int c = 0; c < d; ++c) acc[c] += w * bf16_to_f64(vbase[(j0 + cj) * d + c]);
      }
      mass = shrink * mass + block_mass;
      top = new_top;
    }
    if (mass == 0.0) {
      lse[r] = -INFINITY;
      for (int c = 0; c < d; ++c) acc[c] = 0.0;
    } else {
      for (int c = 0; c < d; ++c) acc[c] /= mass;
      lse[r] = ln2 * (top + log2(mass));
    }
  }
  free(score);
  free(keep);
  return executed;
}

/* Algorithm 1 over a list of (b, h, I) query blocks, one thread per block. */
void steel_oracle_alg1_blocks(const oracle_problem_t *p, const uint16_t *q, const uint16_t *k,
                              const uint16_t *v, const int64_t *blocks, int64_t n_blocks,
                              double *o, double *lse, int64_t *executed) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t n = 0; n < n_blocks; ++n) {
    executed[n] = steel_oracle_alg1_block(
        p, q, k, v, (int)blocks[3 * n], (int)blocks[3 * n + 1], (int)blocks[3 * n + 2],
        o + n * (int64_t)p->block_q * p->head_dim, lse + n * (int64_t)p->block_q);
  }
}

int steel_oracle_max_threads(void) {
#ifdef _OPENMP
  extern int omp_get_max_threads(void);
  return omp_get_max_threads();
#else
  return 1;
#endif
}
