/*
 * vorta_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, fp64 CPU statement of what VORTA's routed attention computes:
 * full 3D attention (Eq. 2), 3D sliding tile attention (Algorithm 1 of
 * Appendix A.1), and core-set attention = unpool . attn . pool with bucketed
 * core-set selection (Section 3.2 and the paragraph on it in Appendix
 * A.1).  It exists so that the CUDA library can be checked against
 * something written straight from the paper.  It shares no code with the CUDA
 * path and is only used by the tests, by the smoke check and by the benchmark's
 * CPU-baseline leg.
 *
 * Conventions (the paper leaves them open; both sides use the same reading):
 *   - tokens are 0-based and frame-major: i = (t*H + h)*W + w  (Section 2:
 *     the frames x height x width latent is flattened into one sequence);
 *   - scores are scaled by `scale` (the caller passes 1/sqrt(d));
 *   - a video axis with fewer tiles than the window spans is unrestricted;
 *   - the similarity of bucketed core-set selection is the cosine;
 *   - keep(n) = max(1, floor(r*n + 1/2)) tokens survive in a bucket of n tokens;
 *   - by default pruned tokens are NOT merged into the centre: they only receive
 *     the centre's output row at unpool time; the optional merge is the plain mean;
 *   - joint sequences of MMDiT models (video tokens followed by Lt text tokens; the
 *     paper runs HunyuanVideo, Section 4, but does not say how its branches treat the
 *     text tokens): a text key is visible to every query, a text query sees every
 *     key, and core-set selection prunes video tokens only.
 *
 * Pinned by tests/test_oracle_pins.py against: brute-force dense attention with
 * explicit masks built a different way (numpy), torch's fp64
 * scaled_dot_product_attention, the values the paper prints (window 18x27x24 =
 * 11664 keys, 50% core-set -> 25% cost, the 3x3 bucket of Fig. 2), and the
 * invariants (window >= grid == full, ratio 1 == full, constant buckets == full,
 * softmax rows sum to 1).
 * Parity unpinned (the paper fixes none of these; they are readings): cosine as
 * the similarity, the centre of an even-extent bucket, the rounding of r*n on
 * partial buckets, the tie-break, the order of the index list, the 1/sqrt(d)
 * scale.
 *
 * All matrices are row-major double.  One call handles one (batch, head).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define VO_API __attribute__((visibility("default")))

/* ------------------------------------------------------------------------- */
/* Geometry                                                                   */
/* ------------------------------------------------------------------------- */

/* token id -> (t, h, w) for a video of size v = (F, H, W), frame-major */
static void token_coord(int64_t i, const int32_t v[3], int32_t c[3])
{
    c[2] = (int32_t)(i % v[2]);
    c[1] = (int32_t)((i / v[2]) % v[1]);
    c[0] = (int32_t)(i / ((int64_t)v[2] * v[1]));
}

/* Algorithm 1, first step: the 3D tile a token lies in (per-axis floor division). */
static void tile_of_token(int64_t i, const int32_t v[3], const int32_t t[3], int32_t q[3])
{
    int32_t c[3];
    token_coord(i, v, c);
    for (int a = 0; a < 3; ++a) q[a] = c[a] / t[a];
}

static int32_t tiles_on_axis(const int32_t v[3], const int32_t t[3], int a)
{
    return (v[a] + t[a] - 1) / t[a]; /* the last tile may be partial */
}

/*
 * Algorithm 1, second step: every query of a window takes the window's centre
 * tile as its own, i.e. the query's tile id is moved inward so that a
 * window of w tiles centred on it stays inside the tile grid.  restricted[a]
 * is 0 when the grid has no more tiles on that axis than the window spans; the
 * window test is then skipped for the axis.
 */
static void window_centre_tile(const int32_t q[3], const int32_t v[3], const int32_t t[3],
                                 const int32_t w[3], int32_t c[3], int restricted[3])
{
    for (int a = 0; a < 3; ++a) {
        int32_t nt = tiles_on_axis(v, t, a);
        int32_t half = w[a] / 2;
        if (nt > 2 * half + 1) {
            int32_t lo = half, hi = nt - 1 - half;
            c[a] = q[a] < lo ? lo : (q[a] > hi ? hi : q[a]);
            restricted[a] = 1;
        } else {
            c[a] = q[a];
            restricted[a] = 0;
        }
    }
}

/* Algorithm 1, third step: per axis, the centre tile and the key tile are at most half a window apart. */
static int window_test(const int32_t c[3], const int32_t k[3], const int32_t w[3],
                       const int restricted[3])
{
    int m = 1;
    for (int a = 0; a < 3; ++a) {
        if (!restricted[a]) continue;
        m = m && (abs(c[a] - k[a]) <= w[a] / 2);
    }
    return m;
}

/* m[i, j] of Algorithm 1 for one (query token, key token) pair. */
static int sta_mask_pair(int64_t i, int64_t j, const int32_t v[3], const int32_t t[3],
                         const int32_t w[3])
{
    int32_t q[3], k[3], c[3];
    int restricted[3];
    tile_of_token(i, v, t, q);
    tile_of_token(j, v, t, k);
    window_centre_tile(q, v, t, w, c, restricted);
    return window_test(c, k, w, restricted);
}

/* Algorithm 1 as printed: the full L x L boolean mask by the double loop. */
VO_API int vo_sta_token_mask(const int32_t v[3], const int32_t t[3], const int32_t w[3],
                             uint8_t *M)
{
    int64_t L = (int64_t)v[0] * v[1] * v[2];
    for (int64_t i = 0; i < L; ++i)
        for (int64_t j = 0; j < L; ++j)
            M[i * L + j] = (uint8_t)sta_mask_pair(i, j, v, t, w);
    return 0;
}

/*
 * The same test between tiles: BM[qt, kt] with qt = (q_T*nt_H + q_H)*nt_W + q_W.
 * Algorithm 1 only looks at tile ids, so the mask is constant on tile pairs.
 */
VO_API int vo_sta_block_mask(const int32_t v[3], const int32_t t[3], const int32_t w[3],
                             uint8_t *BM)
{
    int32_t nt[3];
    for (int a = 0; a < 3; ++a) nt[a] = tiles_on_axis(v, t, a);
    int64_t n = (int64_t)nt[0] * nt[1] * nt[2];
    for (int64_t qt = 0; qt < n; ++qt) {
        int32_t q[3] = {(int32_t)(qt / ((int64_t)nt[1] * nt[2])), (int32_t)((qt / nt[2]) % nt[1]),
                        (int32_t)(qt % nt[2])};
        int32_t c[3];
        int restricted[3];
        window_centre_tile(q, v, t, w, c, restricted);
        for (int64_t kt = 0; kt < n; ++kt) {
            int32_t k[3] = {(int32_t)(kt / ((int64_t)nt[1] * nt[2])),
                            (int32_t)((kt / nt[2]) % nt[1]), (int32_t)(kt % nt[2])};
            BM[qt * n + kt] = (uint8_t)window_test(c, k, w, restricted);
        }
    }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Attention of one query row over a list of keys (Eq. 2, one row)            */
/* ------------------------------------------------------------------------- */

/*
 * o = softmax_j(scale * <q, K[keys[j]]>) . V[keys[j]]; keys == NULL means
 * 0..nk-1.  s is scratch of nk doubles; on return it holds the probabilities.
 */
static void attend_row(const double *q, const double *K, const double *V, int32_t d,
                       const int64_t *keys, int64_t nk, double scale, double *o, double *s)
{
    double m = -INFINITY;
    for (int64_t jj = 0; jj < nk; ++jj) {
        const double *k = K + (keys ? keys[jj] : jj) * d;
        double acc = 0.0;
#pragma omp simd reduction(+ : acc)
        for (int32_t c = 0; c < d; ++c) acc += q[c] * k[c];
        s[jj] = scale * acc;
        if (s[jj] > m) m = s[jj];
    }
    double z = 0.0;
    for (int64_t jj = 0; jj < nk; ++jj) {
        s[jj] = exp(s[jj] - m);
        z += s[jj];
    }
    for (int32_t c = 0; c < d; ++c) o[c] = 0.0;
    for (int64_t jj = 0; jj < nk; ++jj) {
        const double *vv = V + (keys ? keys[jj] : jj) * d;
        double p = s[jj] / z;
        s[jj] = p;
        for (int32_t c = 0; c < d; ++c) o[c] += p * vv[c];
    }
}

/*
 * Full attention (Eq. 2) for the query rows q_rows[0..nq) (NULL = rows 0..nq-1)
 * over all L keys.  O is [nq, d].  P, if not NULL, receives the [nq, L]
 * probabilities.
 */
VO_API int vo_attn_full(int64_t L, int32_t d, const double *Q, const double *K, const double *V,
                        double scale, int64_t nq, const int64_t *q_rows, double *O, double *P)
{
    int err = 0;
#pragma omp parallel
    {
        double *s = (double *)malloc(sizeof(double) * (size_t)(L > 0 ? L : 1));
        if (!s) {
#pragma omp atomic write
            err = 1;
        }
#pragma omp barrier
        if (!err) {
#pragma omp for schedule(dynamic, 4)
            for (int64_t r = 0; r < nq; ++r) {
                int64_t i = q_rows ? q_rows[r] : r;
                attend_row(Q + i * d, K, V, d, NULL, L, scale, O + r * d, s);
                if (P) memcpy(P + r * L, s, sizeof(double) * (size_t)L);
            }
        }
        free(s);
    }
    return err;
}

/*
 * Sliding tile attention: Eq. 2 with scores outside Algorithm 1's mask removed.
 * For each query row the mask row is evaluated pair by pair, exactly as the
 * double loop of Algorithm 1 does, and the row attends to the keys it keeps.
 *
 * Joint sequence: Q, K, V hold the L = T*H*W video tokens followed by Lt text
 * tokens.  A video query keeps the video keys of Algorithm 1's mask and every
 * text key; a text query keeps every key.  P, if not NULL, is [nq, L + Lt].
 */
VO_API int vo_attn_sliding_joint(const int32_t v[3], const int32_t t[3], const int32_t w[3], int64_t Lt,
                                 int32_t d, const double *Q, const double *K, const double *V, double scale,
                                 int64_t nq, const int64_t *q_rows, double *O, double *P)
{
    int64_t L = (int64_t)v[0] * v[1] * v[2];
    int64_t Ltot = L + Lt;
    int err = 0;
#pragma omp parallel
    {
        double *s = (double *)malloc(sizeof(double) * (size_t)Ltot);
        int64_t *keys = (int64_t *)malloc(sizeof(int64_t) * (size_t)Ltot);
        if (!s || !keys) {
#pragma omp atomic write
            err = 1;
        }
#pragma omp barrier
        if (!err) {
#pragma omp for schedule(dynamic, 4)
            for (int64_t r = 0; r < nq; ++r) {
                int64_t i = q_rows ? q_rows[r] : r;
                int64_t nk = 0;
                for (int64_t j = 0; j < L; ++j)
                    if (i >= L || sta_mask_pair(i, j, v, t, w)) keys[nk++] = j;
                for (int64_t j = L; j < Ltot; ++j) keys[nk++] = j;
                attend_row(Q + i * d, K, V, d, keys, nk, scale, O + r * d, s);
                if (P) {
                    double *prow = P + r * Ltot;
                    for (int64_t j = 0; j < Ltot; ++j) prow[j] = 0.0;
                    for (int64_t jj = 0; jj < nk; ++jj) prow[keys[jj]] = s[jj];
                }
            }
        }
        free(s);
        free(keys);
    }
    return err;
}

VO_API int vo_attn_sliding(const int32_t v[3], const int32_t t[3], const int32_t w[3], int32_t d,
                           const double *Q, const double *K, const double *V, double scale,
                           int64_t nq, const int64_t *q_rows, double *O, double *P)
{
    return vo_attn_sliding_joint(v, t, w, 0, d, Q, K, V, scale, nq, q_rows, O, P);
}

/* ------------------------------------------------------------------------- */
/* Bucketed core-set selection (Section 3.2; Appendix A.1)                    */
/* ------------------------------------------------------------------------- */

static int64_t keep_count(int64_t n, double r)
{
    int64_t k = (int64_t)floor(r * (double)n + 0.5);
    return k < 1 ? 1 : k;
}

/* Number of core-set tokens; depends on the geometry only. */
VO_API int64_t vo_coreset_len(const int32_t v[3], const int32_t b[3], double r)
{
    int64_t Lc = 0;
    for (int32_t bt = 0; bt * b[0] < v[0]; ++bt)
        for (int32_t bh = 0; bh * b[1] < v[1]; ++bh)
            for (int32_t bw = 0; bw * b[2] < v[2]; ++bw) {
                int64_t n = 1;
                int32_t id[3] = {bt, bh, bw};
                for (int a = 0; a < 3; ++a) {
                    int32_t e = v[a] - b[a] * id[a];
                    n *= (e < b[a] ? e : b[a]);
                }
                Lc += keep_count(n, r);
            }
    return Lc;
}

typedef struct {
    double s;
    int32_t local;
} scored_t;

/* most similar first; equal scores: lower local index first */
static int by_similarity_desc(const void *pa, const void *pb)
{
    const scored_t *a = (const scored_t *)pa, *b = (const scored_t *)pb;
    if (a->s > b->s) return -1;
    if (a->s < b->s) return 1;
    return (a->local > b->local) - (a->local < b->local);
}

/*
 * pool(): for every bucket of size b = (t, h, w) (edge buckets are cut by the
 * grid), compare the centre token with every other token of the bucket, prune
 * the k = n - keep(n) most similar ones, keep the rest.
 *
 *   X         [L, dx] features the similarity is taken on
 *   core_idx  [Lc]    kept token ids, bucket by bucket (raster order of buckets);
 *                     inside a bucket the centre comes first, then the other
 *                     kept tokens in raster order
 *   src_slot  [L]     for every token the position in core_idx of the token
 *                     whose attention output it receives at unpool time: its own
 *                     if kept, its bucket's centre if pruned
 *   min_gap   if not NULL: the smallest score difference, over all buckets,
 *             between the last pruned and the first surviving token (how close
 *             the selection came to a tie); +inf if nothing was pruned
 * Returns Lc.
 */
VO_API int64_t vo_coreset_select(const int32_t v[3], const int32_t b[3], double r, const double *X,
                                 int32_t dx, int32_t *core_idx, int32_t *src_slot, double *min_gap)
{
    int64_t Lc = 0;
    double gap = INFINITY;
    int64_t cap = (int64_t)b[0] * b[1] * b[2];
    int64_t *tok = (int64_t *)malloc(sizeof(int64_t) * (size_t)cap);
    scored_t *sc = (scored_t *)malloc(sizeof(scored_t) * (size_t)cap);
    uint8_t *pruned = (uint8_t *)malloc((size_t)cap);
    if (!tok || !sc || !pruned) return -1;

    for (int32_t bt = 0; bt * b[0] < v[0]; ++bt)
        for (int32_t bh = 0; bh * b[1] < v[1]; ++bh)
            for (int32_t bw = 0; bw * b[2] < v[2]; ++bw) {
                int32_t id[3] = {bt, bh, bw}, e[3];
                for (int a = 0; a < 3; ++a) {
                    e[a] = v[a] - b[a] * id[a];
                    if (e[a] > b[a]) e[a] = b[a];
                }
                /* the bucket's tokens in raster order of their local coordinates */
                int64_t n = 0;
                for (int32_t lt = 0; lt < e[0]; ++lt)
                    for (int32_t lh = 0; lh < e[1]; ++lh)
                        for (int32_t lw = 0; lw < e[2]; ++lw)
                            tok[n++] = ((int64_t)(bt * b[0] + lt) * v[1] + (bh * b[1] + lh)) * v[2] +
                                       (bw * b[2] + lw);
                /* the designated centre token (token '5' of the 3x3 example) */
                int32_t centre = ((e[0] / 2) * e[1] + (e[1] / 2)) * e[2] + (e[2] / 2);
                const double *xc = X + tok[centre] * dx;
                double nc = 0.0;
                for (int32_t c = 0; c < dx; ++c) nc += xc[c] * xc[c];
                nc = sqrt(nc);
                /* similarity between the centre and each neighbouring token */
                int64_t m = 0;
                for (int64_t l = 0; l < n; ++l) {
                    if (l == centre) continue;
                    const double *xj = X + tok[l] * dx;
                    double dot = 0.0, nj = 0.0;
                    for (int32_t c = 0; c < dx; ++c) {
                        dot += xc[c] * xj[c];
                        nj += xj[c] * xj[c];
                    }
                    nj = sqrt(nj);
                    sc[m].s = (nc == 0.0 || nj == 0.0) ? 0.0 : dot / (nc * nj);
                    sc[m].local = (int32_t)l;
                    ++m;
                }
                /* tokens with the top-k highest similarity to the centre are pruned */
                int64_t keep = keep_count(n, r);
                int64_t k = n - keep;
                qsort(sc, (size_t)m, sizeof(scored_t), by_similarity_desc);
                memset(pruned, 0, (size_t)n);
                for (int64_t a = 0; a < k; ++a) pruned[sc[a].local] = 1;
                if (k > 0 && k < m) {
                    double g = sc[k - 1].s - sc[k].s;
                    if (g < gap) gap = g;
                }
                /* the bucket's segment of the index list */
                int64_t seg = Lc;
                core_idx[Lc] = (int32_t)tok[centre];
                src_slot[tok[centre]] = (int32_t)Lc;
                ++Lc;
                for (int64_t l = 0; l < n; ++l) {
                    if (l == centre) continue;
                    if (pruned[l]) {
                        src_slot[tok[l]] = (int32_t)seg; /* receives the centre's output */
                    } else {
                        core_idx[Lc] = (int32_t)tok[l];
                        src_slot[tok[l]] = (int32_t)Lc;
                        ++Lc;
                    }
                }
            }
    if (min_gap) *min_gap = gap;
    free(tok);
    free(sc);
    free(pruned);
    return Lc;
}

/*
 * Core-set attention = unpool . attn . pool for the tokens q_rows[0..nq)
 * (NULL = all L tokens, nq = L): select on X, gather the core-set rows of Q, K
 * and V, run Eq. 2 on the shorter sequence, and hand every token the output row
 * of the slot src_slot names.  core_idx [Lc] and src_slot [L] are returned too.
 * O is [nq, d].  Returns Lc, or -1 on allocation failure.
 */
/*
 * merge != 0: the pruned tokens' information is merged into the centre (Section 3.2 says so in
 * one clause and does not give the operator -- the
 * reading here is the plain mean): the centre's rows of Q, K and V in the compact sequences
 * become the mean over the centre and the tokens pruned from its bucket.  With a bucket
 * that keeps one token this is average pooling (the AP variants of Section 4.2).
 */
/*
 * Joint sequence (Lt text tokens after the L video tokens in Q, K, V; X holds at least
 * the L video rows): selection runs on the video tokens only, every text token is kept.
 * The compact sequences are the Lc kept video tokens followed by the Lt text tokens; a
 * text query row i >= L reads compact row Lc + (i - L).  Returns Lc (video tokens kept).
 */
VO_API int64_t vo_attn_coreset_joint(const int32_t v[3], const int32_t b[3], double r, int64_t Lt, int32_t d,
                                     const double *Q, const double *K, const double *V, const double *X,
                                     int32_t dx, double scale, int64_t nq, const int64_t *q_rows,
                                     double *O, int32_t *core_idx, int32_t *src_slot, int merge)
{
    int64_t L = (int64_t)v[0] * v[1] * v[2];
    int64_t Lv = vo_coreset_select(v, b, r, X, dx, core_idx, src_slot, NULL);
    if (Lv < 0) return -1;
    int64_t Lc = Lv + Lt; /* rows of the compact sequences */

    /* pool: the compact sequences */
    double *Qc = (double *)malloc(sizeof(double) * (size_t)(Lc * d));
    double *Kc = (double *)malloc(sizeof(double) * (size_t)(Lc * d));
    double *Vc = (double *)malloc(sizeof(double) * (size_t)(Lc * d));
    int64_t *members = (int64_t *)malloc(sizeof(int64_t) * (size_t)Lc);
    if (!Qc || !members) return -1;
    /* which slots are needed, and where their output goes */
    int64_t *slot_of_row = (int64_t *)malloc(sizeof(int64_t) * (size_t)nq);
    int64_t *need = (int64_t *)malloc(sizeof(int64_t) * (size_t)Lc); /* slot -> dense id or -1 */
    if (!Kc || !Vc || !slot_of_row || !need) return -1;
    for (int64_t s = 0; s < Lc; ++s) {
        int64_t src = s < Lv ? (int64_t)core_idx[s] : L + (s - Lv); /* kept video token, or text token */
        memcpy(Qc + s * d, Q + src * d, sizeof(double) * (size_t)d);
        memcpy(Kc + s * d, K + src * d, sizeof(double) * (size_t)d);
        memcpy(Vc + s * d, V + src * d, sizeof(double) * (size_t)d);
        need[s] = -1;
        members[s] = 1;
    }
    if (merge) {
        /* add every pruned token's rows to its centre's slot, then divide by the head count */
        for (int64_t i = 0; i < L; ++i) {
            int64_t s = src_slot[i];
            if (core_idx[s] == i) continue; /* kept: it is its own slot */
            for (int32_t c = 0; c < d; ++c) {
                Qc[s * d + c] += Q[i * d + c];
                Kc[s * d + c] += K[i * d + c];
                Vc[s * d + c] += V[i * d + c];
            }
            members[s] += 1;
        }
        for (int64_t s = 0; s < Lv; ++s)
            if (members[s] > 1)
                for (int32_t c = 0; c < d; ++c) {
                    Qc[s * d + c] /= (double)members[s];
                    Kc[s * d + c] /= (double)members[s];
                    Vc[s * d + c] /= (double)members[s];
                }
    }
    int64_t n_need = 0;
    for (int64_t rr = 0; rr < nq; ++rr) {
        int64_t i = q_rows ? q_rows[rr] : rr;
        if (i < 0 || i >= L + Lt) return -1;
        int64_t s = i < L ? (int64_t)src_slot[i] : Lv + (i - L);
        if (need[s] < 0) need[s] = n_need++;
        slot_of_row[rr] = s;
    }
    int64_t *slots = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n_need > 0 ? n_need : 1));
    double *Oc = (double *)malloc(sizeof(double) * (size_t)((n_need > 0 ? n_need : 1) * d));
    if (!slots || !Oc) return -1;
    for (int64_t s = 0; s < Lc; ++s)
        if (need[s] >= 0) slots[need[s]] = s;

    /* attn on the core-set: queries and keys are both reduced */
    int err = 0;
#pragma omp parallel
    {
        double *sbuf = (double *)malloc(sizeof(double) * (size_t)Lc);
        if (!sbuf) {
#pragma omp atomic write
            err = 1;
        }
#pragma omp barrier
        if (!err) {
#pragma omp for schedule(dynamic, 4)
            for (int64_t u = 0; u < n_need; ++u) {
                const double *q = Qc + slots[u] * d;
                attend_row(q, Kc, Vc, d, NULL, Lc, scale, Oc + u * d, sbuf);
            }
        }
        free(sbuf);
    }
    /* unpool: scatter the centre's (or the token's own) output row back */
    for (int64_t rr = 0; rr < nq; ++rr)
        memcpy(O + rr * d, Oc + need[slot_of_row[rr]] * d, sizeof(double) * (size_t)d);

    free(Qc);
    free(Kc);
    free(Vc);
    free(members);
    free(slot_of_row);
    free(need);
    free(slots);
    free(Oc);
    return err ? -1 : Lv;
}

VO_API int64_t vo_attn_coreset_ex(const int32_t v[3], const int32_t b[3], double r, int32_t d,
                                  const double *Q, const double *K, const double *V, const double *X,
                                  int32_t dx, double scale, int64_t nq, const int64_t *q_rows,
                                  double *O, int32_t *core_idx, int32_t *src_slot, int merge)
{
    return vo_attn_coreset_joint(v, b, r, 0, d, Q, K, V, X, dx, scale, nq, q_rows, O, core_idx, src_slot, merge);
}

VO_API int64_t vo_attn_coreset(const int32_t v[3], const int32_t b[3], double r, int32_t d,
                               const double *Q, const double *K, const double *V, const double *X,
                               int32_t dx, double scale, int64_t nq, const int64_t *q_rows,
                               double *O, int32_t *core_idx, int32_t *src_slot)
{
    return vo_attn_coreset_ex(v, b, r, d, Q, K, V, X, dx, scale, nq, q_rows, O, core_idx, src_slot, 0);
}

VO_API int vo_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
