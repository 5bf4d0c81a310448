/*
 * mpipe_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, fp64 CPU statement of what the encoder hot path computes:
 * block-diagonal (per-image) multi-head softmax self-attention over a packed
 * token sequence, its exact gradient, and the row scatter that places encoder
 * tokens into the LLM input sequence.  The paper relocates this computation
 * (the encoder forward into the warm-up bubble, the encoder backward -- only
 * when the encoder is trainable, Lemma 1 -- into the cool-down, and the
 * Replicated->Sharded "Gather" seam of Table 2 in front of the first LLM
 * stage) but never writes its formulas: a "ViT-style encoder" (Section 2) is
 * read as standard bidirectional scaled-dot-product attention, one image per
 * segment, no interaction across segments.
 *
 * Everything is the textbook definition evaluated row by row: exact softmax
 * with the row maximum subtracted, no tiling, no online softmax, no
 * recomputation tricks.  Only tests, the smoke check and the CPU-baseline leg
 * of the benchmark may call into this file.  It shares no code with the CUDA
 * library.
 *
 * Layouts: q, k, v, dout are fp64 arrays in [T, H, D] order, contiguous (the
 * Python wrapper widens bf16 bit patterns to fp64, which is exact).  Outputs
 * are fp64 and never rounded.  cu[s]..cu[s+1] are the
 * packed rows of segment s.  "scale" is the same float the GPU receives,
 * promoted to double.
 *
 * Parity pins (tests/test_oracle_*.py): dense masked brute force, a library
 * fp64 autograd cross-check, central finite differences, closed forms
 * (Q = 0, equal keys, constant V, n = 1) and invariances.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    const double *q, *k, *v, *dout;
    int64_t T;
    int H, D;
    const int32_t *cu;
    int n_seg;
    double scale;
} ctx_t;

static inline const double *row_ptr(const ctx_t *c, const double *base, int64_t tok, int h) {
    return base + ((size_t)tok * (size_t)c->H + (size_t)h) * (size_t)c->D;
}

/* s_j = scale * <Q_i, K_j> for every key j of the segment [a, b). */
static void score_row(const ctx_t *c, int h, int64_t i, int64_t a, int64_t b, double *s) {
    const double *qi = row_ptr(c, c->q, i, h);
    for (int64_t j = a; j < b; ++j) {
        const double *kj = row_ptr(c, c->k, j, h);
        double acc = 0.0;
        for (int d = 0; d < c->D; ++d) acc += qi[d] * kj[d];
        s[j - a] = c->scale * acc;
    }
}

/* Forward for one query row: O_i = sum_j P_ij V_j, LSE_i = m + ln sum_j exp(s_j - m).
 * On return s[] holds P_ij. */
static void fwd_row(const ctx_t *c, int h, int64_t i, int64_t a, int64_t b, double *s,
                    double *o_out, double *lse_out) {
    score_row(c, h, i, a, b, s);
    const int64_t n = b - a;
    double m = s[0];
    for (int64_t j = 1; j < n; ++j) if (s[j] > m) m = s[j];
    double l = 0.0;
    for (int64_t j = 0; j < n; ++j) { s[j] = exp(s[j] - m); l += s[j]; }
    for (int d = 0; d < c->D; ++d) o_out[d] = 0.0;
    for (int64_t j = 0; j < n; ++j) {
        s[j] /= l;
        const double *vj = row_ptr(c, c->v, a + j, h);
        for (int d = 0; d < c->D; ++d) o_out[d] += s[j] * vj[d];
    }
    *lse_out = m + log(l);
}

static int find_seg(const ctx_t *c, int64_t tok) {
    for (int s = 0; s < c->n_seg; ++s)
        if (tok >= c->cu[s] && tok < c->cu[s + 1]) return s;
    return -1;
}

static int64_t max_seg_len(const ctx_t *c) {
    int64_t m = 1;
    for (int s = 0; s < c->n_seg; ++s) {
        int64_t n = (int64_t)c->cu[s + 1] - c->cu[s];
        if (n > m) m = n;
    }
    return m;
}

/* ------------------------------------------------------------------------ */
/* Full forward.  O: [T,H,D] fp64, LSE: [H,T] fp64.                         */
/* ------------------------------------------------------------------------ */
int mo_attn_fwd(const double *q, const double *k, const double *v, int64_t T, int H, int D,
                const int32_t *cu, int n_seg, float scale, double *O, double *LSE) {
    ctx_t c = {q, k, v, NULL, T, H, D, cu, n_seg, (double)scale};
    const int64_t nmax = max_seg_len(&c);
    for (int s = 0; s < n_seg; ++s) {
        const int64_t a = cu[s], b = cu[s + 1];
        if (b <= a) continue;
        for (int h = 0; h < H; ++h) {
#pragma omp parallel
            {
                double *sc = (double *)malloc(sizeof(double) * (size_t)nmax);
#pragma omp for schedule(dynamic, 8)
                for (int64_t i = a; i < b; ++i)
                    fwd_row(&c, h, i, a, b, sc, O + ((size_t)i * H + h) * D, LSE + (size_t)h * T + i);
                free(sc);
            }
        }
    }
    return 0;
}

/* Forward for a list of (token row, head) pairs.  O_rows: [n_pairs, D], LSE_rows: [n_pairs]. */
int mo_attn_fwd_rows(const double *q, const double *k, const double *v, int64_t T, int H, int D,
                     const int32_t *cu, int n_seg, float scale, const int64_t *rows,
                     const int32_t *heads, int64_t n_pairs, double *O_rows, double *LSE_rows) {
    ctx_t c = {q, k, v, NULL, T, H, D, cu, n_seg, (double)scale};
    const int64_t nmax = max_seg_len(&c);
    int bad = 0;
#pragma omp parallel
    {
        double *sc = (double *)malloc(sizeof(double) * (size_t)nmax);
#pragma omp for schedule(dynamic, 1)
        for (int64_t p = 0; p < n_pairs; ++p) {
            const int s = find_seg(&c, rows[p]);
            if (s < 0) { bad = 1; continue; }
            fwd_row(&c, heads[p], rows[p], cu[s], cu[s + 1], sc, O_rows + (size_t)p * D, LSE_rows + p);
        }
        free(sc);
    }
    return bad;
}

/* ------------------------------------------------------------------------ */
/* Backward pieces.  lse and delta are per-row values of one (segment, head) */
/* ------------------------------------------------------------------------ */

/* LSE_i and Delta_i = sum_d dO_id * O_id (with the exact, unrounded O) for one row. */
static void lse_delta_row(const ctx_t *c, int h, int64_t i, int64_t a, int64_t b, double *sc,
                          double *otmp, double *lse, double *delta) {
    fwd_row(c, h, i, a, b, sc, otmp, lse);
    const double *doi = row_ptr(c, c->dout, i, h);
    double acc = 0.0;
    for (int d = 0; d < c->D; ++d) acc += doi[d] * otmp[d];
    *delta = acc;
}

/* dQ_i = scale * sum_j dS_ij K_j,  dS_ij = P_ij (dP_ij - Delta_i),  dP_ij = <dO_i, V_j>,
 * P_ij = exp(s_ij - LSE_i). */
static void dq_row(const ctx_t *c, int h, int64_t i, int64_t a, int64_t b, double *sc, double lse,
                   double delta, double *dq_out) {
    score_row(c, h, i, a, b, sc);
    const double *doi = row_ptr(c, c->dout, i, h);
    for (int d = 0; d < c->D; ++d) dq_out[d] = 0.0;
    for (int64_t j = a; j < b; ++j) {
        const double p = exp(sc[j - a] - lse);
        const double *vj = row_ptr(c, c->v, j, h);
        const double *kj = row_ptr(c, c->k, j, h);
        double dp = 0.0;
        for (int d = 0; d < c->D; ++d) dp += doi[d] * vj[d];
        const double ds = p * (dp - delta);
        for (int d = 0; d < c->D; ++d) dq_out[d] += ds * kj[d];
    }
    for (int d = 0; d < c->D; ++d) dq_out[d] *= c->scale;
}

/* dV_j = sum_i P_ij dO_i,  dK_j = scale * sum_i dS_ij Q_i  for one key row j. */
static void dkv_row(const ctx_t *c, int h, int64_t j, int64_t a, int64_t b, const double *lse,
                    const double *delta, double *dk_out, double *dv_out) {
    const double *kj = row_ptr(c, c->k, j, h);
    const double *vj = row_ptr(c, c->v, j, h);
    for (int d = 0; d < c->D; ++d) { dk_out[d] = 0.0; dv_out[d] = 0.0; }
    for (int64_t i = a; i < b; ++i) {
        const double *qi = row_ptr(c, c->q, i, h);
        const double *doi = row_ptr(c, c->dout, i, h);
        double s = 0.0, dp = 0.0;
        for (int d = 0; d < c->D; ++d) {
            s += qi[d] * kj[d];
            dp += doi[d] * vj[d];
        }
        const double p = exp(c->scale * s - lse[i - a]);
        const double ds = p * (dp - delta[i - a]);
        for (int d = 0; d < c->D; ++d) {
            dv_out[d] += p * doi[d];
            dk_out[d] += ds * qi[d];
        }
    }
    for (int d = 0; d < c->D; ++d) dk_out[d] *= c->scale;
}

/* Per-row LSE and Delta of one (segment, head); arrays of length n = b - a. */
static void seg_head_stats(const ctx_t *c, int h, int64_t a, int64_t b, double *lse, double *delta) {
    const int64_t n = b - a;
#pragma omp parallel
    {
        double *sc = (double *)malloc(sizeof(double) * (size_t)n);
        double *ot = (double *)malloc(sizeof(double) * (size_t)c->D);
#pragma omp for schedule(dynamic, 8)
        for (int64_t i = a; i < b; ++i) lse_delta_row(c, h, i, a, b, sc, ot, lse + (i - a), delta + (i - a));
        free(sc);
        free(ot);
    }
}

/* Full backward.  dQ, dK, dV: [T,H,D] fp64. */
int mo_attn_bwd(const double *dout, const double *q, const double *k, const double *v,
                int64_t T, int H, int D, const int32_t *cu, int n_seg, float scale, double *dQ,
                double *dK, double *dV) {
    ctx_t c = {q, k, v, dout, T, H, D, cu, n_seg, (double)scale};
    const int64_t nmax = max_seg_len(&c);
    double *lse = (double *)malloc(sizeof(double) * (size_t)nmax);
    double *delta = (double *)malloc(sizeof(double) * (size_t)nmax);
    for (int s = 0; s < n_seg; ++s) {
        const int64_t a = cu[s], b = cu[s + 1];
        if (b <= a) continue;
        for (int h = 0; h < H; ++h) {
            seg_head_stats(&c, h, a, b, lse, delta);
#pragma omp parallel
            {
                double *sc = (double *)malloc(sizeof(double) * (size_t)(b - a));
#pragma omp for schedule(dynamic, 8)
                for (int64_t i = a; i < b; ++i)
                    dq_row(&c, h, i, a, b, sc, lse[i - a], delta[i - a], dQ + ((size_t)i * H + h) * D);
#pragma omp for schedule(dynamic, 8)
                for (int64_t j = a; j < b; ++j)
                    dkv_row(&c, h, j, a, b, lse, delta, dK + ((size_t)j * H + h) * D,
                            dV + ((size_t)j * H + h) * D);
                free(sc);
            }
        }
    }
    free(lse);
    free(delta);
    return 0;
}

/* dQ for a list of (token row, head) pairs: each needs only its own row. dQ_rows: [n_pairs, D]. */
int mo_attn_bwd_dq_rows(const double *dout, const double *q, const double *k, const double *v,
                        int64_t T, int H, int D, const int32_t *cu, int n_seg, float scale,
                        const int64_t *rows, const int32_t *heads, int64_t n_pairs, double *dQ_rows) {
    ctx_t c = {q, k, v, dout, T, H, D, cu, n_seg, (double)scale};
    const int64_t nmax = max_seg_len(&c);
    int bad = 0;
#pragma omp parallel
    {
        double *sc = (double *)malloc(sizeof(double) * (size_t)nmax);
        double *ot = (double *)malloc(sizeof(double) * (size_t)D);
#pragma omp for schedule(dynamic, 1)
        for (int64_t p = 0; p < n_pairs; ++p) {
            const int s = find_seg(&c, rows[p]);
            if (s < 0) { bad = 1; continue; }
            double lse, delta;
            lse_delta_row(&c, heads[p], rows[p], cu[s], cu[s + 1], sc, ot, &lse, &delta);
            dq_row(&c, heads[p], rows[p], cu[s], cu[s + 1], sc, lse, delta, dQ_rows + (size_t)p * D);
        }
        free(sc);
        free(ot);
    }
    return bad;
}

/* dK, dV for a list of key rows of ONE (segment, head): the column sums need LSE and Delta of every
 * query row of that segment, which are computed first.  dK_rows, dV_rows: [n_rows, D]. */
int mo_attn_bwd_dkv_rows(const double *dout, const double *q, const double *k, const double *v,
                         int64_t T, int H, int D, const int32_t *cu, int n_seg, float scale, int seg,
                         int head, const int64_t *rows, int64_t n_rows, double *dK_rows, double *dV_rows) {
    ctx_t c = {q, k, v, dout, T, H, D, cu, n_seg, (double)scale};
    if (seg < 0 || seg >= n_seg) return 1;
    const int64_t a = cu[seg], b = cu[seg + 1];
    if (b <= a) return 1;
    for (int64_t p = 0; p < n_rows; ++p) if (rows[p] < a || rows[p] >= b) return 1;
    double *lse = (double *)malloc(sizeof(double) * (size_t)(b - a));
    double *delta = (double *)malloc(sizeof(double) * (size_t)(b - a));
    seg_head_stats(&c, head, a, b, lse, delta);
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t p = 0; p < n_rows; ++p)
        dkv_row(&c, head, rows[p], a, b, lse, delta, dK_rows + (size_t)p * D, dV_rows + (size_t)p * D);
    free(lse);
    free(delta);
    return 0;
}

/* ------------------------------------------------------------------------ */
/* Merge: the local placement of the Gather seam.  out starts as a copy of   */
/* the LLM embedding rows; encoder token i replaces row pos[i].  16-bit words.*/
/* ------------------------------------------------------------------------ */
int mo_merge_tokens(const uint16_t *enc, const uint16_t *emb_in, uint16_t *out, const int32_t *pos,
                    int64_t n_enc, int64_t n_llm, int64_t hidden) {
    memcpy(out, emb_in, sizeof(uint16_t) * (size_t)n_llm * (size_t)hidden);
    int bad = 0;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n_enc; ++i) {
        if (pos[i] < 0 || pos[i] >= n_llm) { bad = 1; continue; }
        memcpy(out + (size_t)pos[i] * hidden, enc + (size_t)i * hidden, sizeof(uint16_t) * (size_t)hidden);
    }
    return bad;
}

/* Reverse seam (only when the encoder is trainable, Lemma 1 gate (i)): d_enc[i,:] = d_emb[pos[i],:]. */
int mo_merge_tokens_bwd(const uint16_t *d_emb, uint16_t *d_enc, const int32_t *pos, int64_t n_enc,
                        int64_t n_llm, int64_t hidden) {
    int bad = 0;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n_enc; ++i) {
        if (pos[i] < 0 || pos[i] >= n_llm) { bad = 1; continue; }
        memcpy(d_enc + (size_t)i * hidden, d_emb + (size_t)pos[i] * hidden, sizeof(uint16_t) * (size_t)hidden);
    }
    return bad;
}
