/*
 * CPU oracle for policy-gated block-sparse joint attention  --  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 restatement of what the hot path computes.  It exists so that the
 * CUDA kernels can be checked against something written independently of them; it shares
 * no code, header, table or constant with the CUDA path and must never be called from it.
 *
 * What is followed.  The paper (Sec. 3.2, "Level-3: Sparse-Attention") replaces the
 * self-attention block of a DiT layer by a sparse attention whose sparsity level is picked
 * per time step by the policy head P^sparse (Sec. 3.3 c): action 0 is full attention, larger
 * actions are progressively sparser, and the head is inactive when the cache is reused).
 * The paper does not define the sparsity rule itself; the rule restated here is the one this
 * project fixes:  64-token blocks on the joint (text first, then image) sequence, mean-pooled
 * Q/K block scores, and per (image, head, query-block row) a top-k selection at the policy's
 * keep ratio, with text blocks and the diagonal block always kept.
 *
 * Parity status: every function below is pinned by definition-level tests (brute-force dense
 * attention at keep ratio 1, convexity, permutation invariance, count identity, closed forms,
 * subset enumeration).  The paper prints no mask, score or output value for this path, so
 * against the paper itself the whole path is "parity unpinned".
 *
 * Inputs are bf16 bit patterns (uint16_t); bf16 -> fp64 is exact.  All arithmetic is fp64.
 * OpenMP only spreads independent rows over cores.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define BLOCK 64

static double bf16_to_f64(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Step 1-2: block mean pooling of one [N, D] bf16 matrix (one image, one head).
 * pooled[i, :] = mean over the valid tokens of block i (the tail block divides by its own
 * token count, not by 64). */
void oracle_block_pool(const uint16_t *x, int N, int D, double *pooled /* [nb, D] */) {
    int nb = (N + BLOCK - 1) / BLOCK;
    for (int i = 0; i < nb; ++i) {
        int lo = i * BLOCK, hi = lo + BLOCK < N ? lo + BLOCK : N;
        for (int d = 0; d < D; ++d) {
            double acc = 0.0;
            for (int n = lo; n < hi; ++n) acc += bf16_to_f64(x[(size_t)n * D + d]);
            pooled[(size_t)i * D + d] = acc / (double)(hi - lo);
        }
    }
}

/* Step 3: block scores S[i, j] = pooledQ[i, :] . pooledK[j, :]  (no softmax scale). */
void oracle_block_scores(const double *pq, const double *pk, int nb, int D, double *S /* [nb, nb] */) {
    for (int i = 0; i < nb; ++i)
        for (int j = 0; j < nb; ++j) {
            double acc = 0.0;
            for (int d = 0; d < D; ++d) acc += pq[(size_t)i * D + d] * pk[(size_t)j * D + d];
            S[(size_t)i * nb + j] = acc;
        }
}

/* Number of free candidates kept at a keep ratio: ceil(ratio * n_free - 1e-6), clamped. */
int oracle_keep_count(double ratio, int n_free) {
    double x = ceil(ratio * (double)n_free - 1e-6);
    int k = (int)x;
    if (k < 0) k = 0;
    if (k > n_free) k = n_free;
    return k;
}

/* Steps 4-5: block mask of one (image, head).
 *   forced(i)  = { j : j < n_text_blocks }  u  { i };   all blocks when i < n_text_blocks
 *   free(i)    = the other blocks;  keep the k = keep_count(ratio, |free(i)|) best of them,
 *                ordered by (score descending, index ascending).
 * mask[i*nb + j] = 1 when query block i attends key block j.
 * gap[i] = score of the last kept free candidate minus score of the best dropped one
 *          (+inf when nothing is dropped or nothing free is kept): a small gap marks a near tie. */
void oracle_select_mask(const double *S, int nb, int n_text_blocks, double ratio,
                        uint8_t *mask /* [nb, nb] */, double *gap /* [nb] or NULL */) {
    int *cand = (int *)malloc(sizeof(int) * (size_t)(nb > 0 ? nb : 1));
    for (int i = 0; i < nb; ++i) {
        uint8_t *row = mask + (size_t)i * nb;
        memset(row, 0, (size_t)nb);
        int nc = 0;
        for (int j = 0; j < nb; ++j) {
            int forced = (j < n_text_blocks) || (j == i) || (i < n_text_blocks);
            if (forced) row[j] = 1; else cand[nc++] = j;
        }
        int k = oracle_keep_count(ratio, nc);
        /* insertion sort of the candidates by (score desc, index asc); nc is at most a few hundred */
        for (int a = 1; a < nc; ++a) {
            int c = cand[a];
            double sc = S[(size_t)i * nb + c];
            int b = a - 1;
            while (b >= 0) {
                double sb = S[(size_t)i * nb + cand[b]];
                if (sb > sc || (sb == sc && cand[b] < c)) break;
                cand[b + 1] = cand[b];
                --b;
            }
            cand[b + 1] = c;
        }
        for (int a = 0; a < k; ++a) row[cand[a]] = 1;
        if (gap) {
            if (k > 0 && k < nc) gap[i] = S[(size_t)i * nb + cand[k - 1]] - S[(size_t)i * nb + cand[k]];
            else gap[i] = INFINITY;
        }
    }
    free(cand);
}

/* Cumulative-mass variant of steps 4-5 (Sec. 3.2: the sparse candidates are thresholds, not
 * counts; the paper leaves the rule to the sparse-attention method it plugs in, so this is the
 * plain "smallest set of the best blocks that holds a share tau of the row's mass" rule).
 * Forced blocks as above.  For the free candidates of row i, in the order (score descending,
 * index ascending):
 *     w_c   = exp(scale * (S[i, c] - max over the free candidates of S[i, .]))
 *     k     = the smallest count whose first k weights sum to at least tau * (sum of all w);
 *             all of them when tau >= 1, none when there is no candidate
 * and the first k candidates are kept.
 * k_out[i]  = k (0 for text rows: they are dense and have no free candidate).
 * margin[i] = distance of the deciding comparison from equality, relative to the total mass:
 *             min(cum_k - target, target - cum_{k-1}) / total (+inf when tau >= 1 or no candidate).
 * gap[i]    = as in oracle_select_mask: score of the last kept minus the best dropped candidate. */
void oracle_select_mask_mass(const double *S, int nb, int n_text_blocks, double tau, double scale,
                             uint8_t *mask /* [nb, nb] */, double *gap /* [nb] or NULL */,
                             int32_t *k_out /* [nb] or NULL */, double *margin /* [nb] or NULL */) {
    int *cand = (int *)malloc(sizeof(int) * (size_t)(nb > 0 ? nb : 1));
    double *w = (double *)malloc(sizeof(double) * (size_t)(nb > 0 ? nb : 1));
    for (int i = 0; i < nb; ++i) {
        uint8_t *row = mask + (size_t)i * nb;
        const double *Si = S + (size_t)i * nb;
        memset(row, 0, (size_t)nb);
        int nc = 0;
        for (int j = 0; j < nb; ++j) {
            int forced = (j < n_text_blocks) || (j == i) || (i < n_text_blocks);
            if (forced) row[j] = 1; else cand[nc++] = j;
        }
        for (int a = 1; a < nc; ++a) {              /* order: score descending, index ascending */
            int c = cand[a];
            int b = a - 1;
            while (b >= 0 && !(Si[cand[b]] > Si[c] || (Si[cand[b]] == Si[c] && cand[b] < c))) {
                cand[b + 1] = cand[b];
                --b;
            }
            cand[b + 1] = c;
        }
        int k = nc;
        double mg = INFINITY;
        if (nc > 0 && tau < 1.0) {
            double total = 0.0;
            for (int a = 0; a < nc; ++a) {
                w[a] = exp(scale * (Si[cand[a]] - Si[cand[0]]));
                total += w[a];
            }
            double target = tau * total, cum = 0.0;
            k = nc;                                  /* rounding may leave the full sum a hair short of the target */
            for (int a = 0; a < nc; ++a) {
                double before = cum;
                cum += w[a];
                if (cum >= target) {
                    double lo = target - before, hi = cum - target;
                    k = a + 1;
                    mg = (lo < hi ? lo : hi) / total;
                    break;
                }
            }
        }
        for (int a = 0; a < k; ++a) row[cand[a]] = 1;
        if (k_out) k_out[i] = k;
        if (margin) margin[i] = mg;
        if (gap) gap[i] = (k > 0 && k < nc) ? Si[cand[k - 1]] - Si[cand[k]] : INFINITY;
    }
    free(cand);
    free(w);
}

/* Step 6: masked softmax attention of one (image, head) for query blocks [qb_lo, qb_hi).
 * For a query token n in block i, the keys are the valid tokens m of every block j with
 * mask[i, j] != 0;   z_m = scale * q_n . k_m;   p = softmax(z) over exactly those keys;
 * out[n, :] = sum_m p_m v_m.   Rows of query blocks outside the range are left untouched.
 * A row with no kept key gets zeros. */
void oracle_masked_attention(const uint16_t *q, const uint16_t *k, const uint16_t *v, int N, int D,
                             const uint8_t *mask /* [nb, nb] */, double scale, int qb_lo, int qb_hi,
                             double *out /* [N, D] */) {
    int nb = (N + BLOCK - 1) / BLOCK;
    double *kd = (double *)malloc(sizeof(double) * (size_t)N * D);
    double *vd = (double *)malloc(sizeof(double) * (size_t)N * D);
    for (size_t e = 0; e < (size_t)N * D; ++e) { kd[e] = bf16_to_f64(k[e]); vd[e] = bf16_to_f64(v[e]); }
    if (qb_lo < 0) qb_lo = 0;
    if (qb_hi > nb) qb_hi = nb;
    int n_lo = qb_lo * BLOCK, n_hi = qb_hi * BLOCK < N ? qb_hi * BLOCK : N;
#pragma omp parallel
    {
        double *z = (double *)malloc(sizeof(double) * (size_t)N);
        double *qd = (double *)malloc(sizeof(double) * (size_t)D);
#pragma omp for schedule(dynamic, 8)
        for (int n = n_lo; n < n_hi; ++n) {
            int i = n / BLOCK;
            const uint8_t *row = mask + (size_t)i * nb;
            for (int d = 0; d < D; ++d) qd[d] = bf16_to_f64(q[(size_t)n * D + d]);
            double zmax = -INFINITY;
            for (int j = 0; j < nb; ++j) {
                if (!row[j]) continue;
                int lo = j * BLOCK, hi = lo + BLOCK < N ? lo + BLOCK : N;
                for (int m = lo; m < hi; ++m) {
                    double acc = 0.0;
                    const double *km = kd + (size_t)m * D;
#pragma omp simd reduction(+ : acc)
                    for (int d = 0; d < D; ++d) acc += qd[d] * km[d];
                    z[m] = scale * acc;
                    if (z[m] > zmax) zmax = z[m];
                }
            }
            double *o = out + (size_t)n * D;
            for (int d = 0; d < D; ++d) o[d] = 0.0;
            double denom = 0.0;
            for (int j = 0; j < nb; ++j) {
                if (!row[j]) continue;
                int lo = j * BLOCK, hi = lo + BLOCK < N ? lo + BLOCK : N;
                for (int m = lo; m < hi; ++m) {
                    double p = exp(z[m] - zmax);
                    denom += p;
                    const double *vm = vd + (size_t)m * D;
                    for (int d = 0; d < D; ++d) o[d] += p * vm[d];
                }
            }
            if (denom > 0.0)
                for (int d = 0; d < D; ++d) o[d] /= denom;
        }
        free(z);
        free(qd);
    }
    free(kd);
    free(vd);
}

/* Softmax weights of one query token (for the convexity pin): w[m] for every token m,
 * zero for keys that are not kept. */
void oracle_attention_weights(const uint16_t *q, const uint16_t *k, int N, int D, const uint8_t *mask,
                              double scale, int n, double *w /* [N] */) {
    int nb = (N + BLOCK - 1) / BLOCK;
    int i = n / BLOCK;
    const uint8_t *row = mask + (size_t)i * nb;
    double zmax = -INFINITY;
    for (int m = 0; m < N; ++m) w[m] = 0.0;
    for (int m = 0; m < N; ++m) {
        if (!row[m / BLOCK]) continue;
        double acc = 0.0;
        for (int d = 0; d < D; ++d) acc += bf16_to_f64(q[(size_t)n * D + d]) * bf16_to_f64(k[(size_t)m * D + d]);
        w[m] = scale * acc;
        if (w[m] > zmax) zmax = w[m];
    }
    double denom = 0.0;
    for (int m = 0; m < N; ++m) {
        if (!row[m / BLOCK]) continue;
        w[m] = exp(w[m] - zmax);
        denom += w[m];
    }
    for (int m = 0; m < N; ++m) w[m] = row[m / BLOCK] ? w[m] / denom : 0.0;
}

int oracle_num_threads(void) {
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp single
        n = omp_get_num_threads();
    }
#endif
    return n;
}

/* ------------------------------------------------------------------------------------------
 * Q/K producer with the block pooling folded in (the step in front of the attention of an MMDiT
 * block: per-head RMS normalisation of the projected queries / keys with a learned gain, then
 * the rotary position embedding; the paper takes both from its base models and does not restate
 * them).  For one [N, D] bf16 matrix (one image, one head), token n:
 *     r      = 1 / sqrt(mean_d x[n, d]^2 + eps)
 *     y[d]   = x[n, d] * r * gain[d]
 *     z[2i]  = y[2i] cos(n, i) - y[2i+1] sin(n, i),   z[2i+1] = y[2i] sin(n, i) + y[2i+1] cos(n, i)
 * with rot[n][i] = (cos, sin) given as fp32 numbers (NULL: no rotation); out = z rounded once
 * to bf16, ties to even.  The block means the scoring pass needs are the means of the ROUNDED
 * values, i.e. oracle_block_pool of `out`.  Arithmetic in fp64. */
static uint16_t f64_to_bf16(double v) {
    /* direct round-to-nearest-even of the 52-bit mantissa to 7 bits (no detour through fp32) */
    uint64_t u;
    memcpy(&u, &v, sizeof u);
    uint16_t sign = (uint16_t)((u >> 63) << 15);
    uint64_t mag = u & 0x7fffffffffffffffULL;
    if (mag == 0) return sign;
    mag += ((1ULL << 44) - 1) + ((mag >> 45) & 1);
    int64_t e = (int64_t)(mag >> 52) - 1023 + 127;            /* exponent after a possible carry */
    if (e <= 0) return sign;                                  /* below the bf16 normal range: zero */
    if (e >= 255) return (uint16_t)(sign | 0x7f80);           /* infinity */
    return (uint16_t)(sign | ((uint16_t)e << 7) | (uint16_t)((mag >> 45) & 0x7f));
}

void oracle_qk_prepare(const uint16_t *x, int N, int D, const float *gain /* [D] */,
                       const float *rot /* [N, D/2, 2] or NULL */, double eps, uint16_t *out /* [N, D] */) {
    double *y = (double *)malloc(sizeof(double) * (size_t)D);
    for (int n = 0; n < N; ++n) {
        double ss = 0.0;
        for (int d = 0; d < D; ++d) { double v = bf16_to_f64(x[(size_t)n * D + d]); ss += v * v; }
        double r = 1.0 / sqrt(ss / (double)D + eps);
        for (int d = 0; d < D; ++d) y[d] = bf16_to_f64(x[(size_t)n * D + d]) * r * (double)gain[d];
        for (int i = 0; i < D / 2; ++i) {
            double c = 1.0, s = 0.0;
            if (rot) { c = (double)rot[((size_t)n * (D / 2) + i) * 2]; s = (double)rot[((size_t)n * (D / 2) + i) * 2 + 1]; }
            out[(size_t)n * D + 2 * i] = f64_to_bf16(y[2 * i] * c - y[2 * i + 1] * s);
            out[(size_t)n * D + 2 * i + 1] = f64_to_bf16(y[2 * i] * s + y[2 * i + 1] * c);
        }
    }
    free(y);
}
