/*
 * CPU oracle for Stream mask estimation (Algorithm 2) and masked block attention (Eq. 2).
 *
 * TEST INFRASTRUCTURE ONLY. This file is the slow, plain definition the CUDA library is
 * checked against. It shares no code with the CUDA path and must never be called from it;
 * only the tests, the smoke check and the benchmark's CPU-baseline leg may load it.
 *
 * It walks Algorithm 2 in the paper's order and notation (f, l, m, B, omega, r, s, I), one
 * query block at a time, with no blocking, fusion or reordering. Floating point: every dot
 * product is accumulated in fp64 over the head dimension and rounded once to fp32; scores are
 * compared as fp32. Readings taken where the printed algorithm is silent or inconsistent:
 *   - log in n_it is base 2 ("refines the search space by half", Section 3);
 *   - initial node j runs over 0..k-1 and node bounds are in key-BLOCK units, so the k nodes
 *     tile [0, N_k) exactly (the printed j = 1..k with T/k overruns the array);
 *   - a node (f : l) with inclusive l splits at m = floor((f+l)/2) into (f : m) and (m+1 : l);
 *     the printed (f : m-1), (m : l) never shrinks a two-block node;
 *   - an empty branch has omega = 0, hence score -inf;
 *   - "top-k" orders by higher fp32 score, then lower branch index h; the survivors become the
 *     next nodes in ascending h;
 *   - k counts key blocks (row width k), not k / b_k;
 *   - the constant r of the input list is unused, as in the printed body;
 *   - "variable k" (named in the paper as future work, never defined): each query block runs
 *     the unchanged algorithm with a k of its own (so_build_mask_rows_var, so_k_schedule).
 * Pins (tests, CPU only): hand-worked example, brute-force block scores on integer inputs,
 * single-level == exact top-k, count/causality/ordering invariants, full mask == dense causal
 * softmax attention (checked against a library routine), an independently structured recursive
 * simulation on tiny inputs. The index readings above are this build's; no value printed in the
 * paper pins them ("parity unpinned" for the readings themselves, pinned for everything else).
 *
 * Layout: Q is [batch, n_q_heads, T, d], K and V are [batch, n_kv_heads, T, d], contiguous,
 * fp32 or bf16 (raw uint16 bit patterns). Query head h reads kv head h / (n_q_heads/n_kv_heads).
 * A "row" is one (batch, q head, query block); rows are addressed by
 * row_id = (b * n_q_heads + h) * ceil(T / b_q) + q.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int32_t batch, n_q_heads, n_kv_heads;
    int64_t T;
    int32_t d, block_q, block_k, k_top, causal;
    int32_t dtype; /* 0 = fp32, 1 = bf16 */
} so_problem;

/* flags for so_build_mask_rows */
#define SO_SCORE_CACHE 1 /* remember s(q, r) per row instead of recomputing it; same values */

static double load_elem(const void *base, int64_t idx, int dtype) {
    if (dtype == 0) return (double)((const float *)base)[idx];
    uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
    float f;
    memcpy(&f, &bits, 4);
    return (double)f;
}

static int64_t gcd64(int64_t a, int64_t b) { while (b) { int64_t t = a % b; a = b; b = t; } return a; }

/* Algorithm 2, first lines: padded length T_p = ceil(T / lcm(b_q, b_k)) * lcm. */
static int64_t padded_len(const so_problem *p) {
    int64_t l = (int64_t)p->block_q / gcd64(p->block_q, p->block_k) * p->block_k;
    return (p->T + l - 1) / l * l;
}

/* C after padding: 1 iff both tokens are inside the original T and (if causal) key <= query. */
static int valid_pair(const so_problem *p, int64_t tq, int64_t tk) {
    if (tq >= p->T || tk >= p->T) return 0;
    return !p->causal || tk <= tq;
}

/* C^blk[q, r] = max over the b_q x b_k cell of C: written out as the max itself. */
static int c_blk(const so_problem *p, int64_t q, int64_t r) {
    for (int64_t m = 0; m < p->block_q; ++m)
        for (int64_t n = 0; n < p->block_k; ++n)
            if (valid_pair(p, q * p->block_q + m, r * p->block_k + n)) return 1;
    return 0;
}

int64_t so_num_query_blocks(const so_problem *p) { return (p->T + p->block_q - 1) / p->block_q; }
int64_t so_num_rows(const so_problem *p) { return (int64_t)p->batch * p->n_q_heads * so_num_query_blocks(p); }
int so_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Q[q, m, :] (or K[r, n, :]) of the padded, blocked view as fp64; padding rows are zero. */
static void block_rows(const so_problem *p, const void *X, int64_t head_row, int64_t blk, int64_t bsz, double *dst) {
    const int64_t d = p->d;
    for (int64_t m = 0; m < bsz; ++m) {
        int64_t t = blk * bsz + m;
        for (int64_t c = 0; c < d; ++c)
            dst[m * d + c] = t < p->T ? load_elem(X, (head_row * p->T + t) * d + c, p->dtype) : 0.0;
    }
}

/* s = max over (m, n) with C = 1 of Q[q,m,:] . K[r,n,:]  (Algorithm 2 scoring line; Eq. 4 with
 * the mask). Each dot product is summed in fp64 (the compiler may keep several fp64 partial sums)
 * and rounded once to fp32. Returns -inf if no pair is allowed. */
static float tile_score(const so_problem *p, const void *Q, const void *K, int64_t b, int64_t h,
                        int64_t q, int64_t r) {
    int64_t g = h / (p->n_q_heads / p->n_kv_heads);
    const int64_t d = p->d;
    double *Qt = malloc(sizeof(double) * (size_t)(p->block_q * d));
    double *Kt = malloc(sizeof(double) * (size_t)(p->block_k * d));
    if (!Qt || !Kt) { free(Qt); free(Kt); return NAN; }
    block_rows(p, Q, b * p->n_q_heads + h, q, p->block_q, Qt);
    block_rows(p, K, b * p->n_kv_heads + g, r, p->block_k, Kt);
    float best = -INFINITY;
    for (int64_t m = 0; m < p->block_q; ++m)
        for (int64_t n = 0; n < p->block_k; ++n) {
            if (!valid_pair(p, q * p->block_q + m, r * p->block_k + n)) continue;
            const double *u = Qt + m * d, *v = Kt + n * d;
            double acc = 0.0;
#pragma omp simd reduction(+ : acc)
            for (int64_t c = 0; c < d; ++c) acc += u[c] * v[c];
            float s = (float)acc; /* one rounding to fp32 */
            if (s > best) best = s;
        }
    free(Qt); free(Kt);
    return best;
}

/* Public single-tile score, used by the brute-force pins. */
float so_tile_score(const so_problem *p, const void *Q, const void *K, int64_t b, int64_t h, int64_t q, int64_t r) {
    return tile_score(p, Q, K, b, h, q, r);
}

typedef struct { float s; int32_t h; } ranked;

/* total order of the top-k step: higher score first, then lower branch index */
static int ranked_cmp(const void *a, const void *b) {
    const ranked *x = (const ranked *)a, *y = (const ranked *)b;
    if (x->s > y->s) return -1;
    if (x->s < y->s) return 1;
    return (x->h > y->h) - (x->h < y->h);
}

static int index_cmp(const void *a, const void *b) {
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

/* One query block of Algorithm 2. mask_row/score_row have k entries (ascending block index,
 * then -1 / -inf padding). Returns 0, or -1 on allocation failure. */
static int stream_row_seen(const so_problem *p, const void *Q, const void *K, int64_t b, int64_t h, int64_t q,
                           int n_it_override, int flags, int32_t *mask_row, float *score_row, float *min_gap,
                           int64_t *tiles, unsigned char *seen_shared);

static int stream_row(const so_problem *p, const void *Q, const void *K, int64_t b, int64_t h, int64_t q,
                      int n_it_override, int flags, int32_t *mask_row, float *score_row, float *min_gap,
                      int64_t *tiles) {
    return stream_row_seen(p, Q, K, b, h, q, n_it_override, flags, mask_row, score_row, min_gap, tiles, NULL);
}

/* seen_shared: NULL, or N_k flags owned by the caller that say which representatives of this row
 * were already scored by an earlier run (another k); *tiles then counts only the new ones. The
 * scores themselves are always computed here: sharing changes the count, never a value. */
static int stream_row_seen(const so_problem *p, const void *Q, const void *K, int64_t b, int64_t h, int64_t q,
                           int n_it_override, int flags, int32_t *mask_row, float *score_row, float *min_gap,
                           int64_t *tiles, unsigned char *seen_shared) {
    const int64_t k = p->k_top;
    const int64_t N_k = padded_len(p) / p->block_k;
    int n_it = 0;
    while (((int64_t)1 << n_it) < N_k) ++n_it; /* n_it = ceil(log2(T_p / b_k)) */
    if (n_it_override >= 0) n_it = n_it_override;

    int64_t *f = malloc(sizeof(int64_t) * k), *l = malloc(sizeof(int64_t) * k);
    int64_t *Bf = malloc(sizeof(int64_t) * 2 * k), *Bl = malloc(sizeof(int64_t) * 2 * k);
    float *s = malloc(sizeof(float) * 2 * k);
    ranked *order = malloc(sizeof(ranked) * 2 * k);
    int32_t *t = malloc(sizeof(int32_t) * k);
    unsigned char *seen = calloc((size_t)N_k, 1); /* reps this run has scored */
    unsigned char *Cblk = malloc((size_t)N_k);    /* row q of C^blk */
    float *cache = malloc(sizeof(float) * (size_t)N_k);
    if (!f || !l || !Bf || !Bl || !s || !order || !t || !seen || !cache || !Cblk) return -1;
    for (int64_t r = 0; r < N_k; ++r) Cblk[r] = (unsigned char)c_blk(p, q, r);
    float gap_min = INFINITY;
    int64_t n_tiles = 0;

    /* initial k nodes tiling [0, N_k) */
    for (int64_t j = 0; j < k; ++j) {
        f[j] = (j * N_k) / k;
        l[j] = ((j + 1) * N_k) / k - 1;
    }
    for (int i = 1; i <= n_it; ++i) {
        for (int64_t j = 0; j < k; ++j) { /* split */
            if (l[j] < f[j]) { /* empty node: both branches empty */
                Bf[2 * j] = Bf[2 * j + 1] = 0;
                Bl[2 * j] = Bl[2 * j + 1] = -1;
                continue;
            }
            int64_t m = (f[j] + l[j]) / 2;
            Bf[2 * j] = f[j];         Bl[2 * j] = m;
            Bf[2 * j + 1] = m + 1;    Bl[2 * j + 1] = l[j];
        }
        for (int64_t hh = 0; hh < 2 * k; ++hh) { /* score the 2k branches */
            int omega = 0;
            for (int64_t r = Bf[hh]; r <= Bl[hh]; ++r) if (Cblk[r]) omega = 1;
            if (!omega) { s[hh] = -INFINITY; continue; }
            int64_t r = Bf[hh];
            while (!Cblk[r]) ++r; /* first valid block of the branch */
            if (!seen[r]) {
                seen[r] = 1; cache[r] = NAN;
                if (!seen_shared) ++n_tiles;
                else if (!seen_shared[r]) { seen_shared[r] = 1; ++n_tiles; }
            }
            if ((flags & SO_SCORE_CACHE) && !isnan(cache[r])) s[hh] = cache[r];
            else s[hh] = cache[r] = tile_score(p, Q, K, b, h, q, r);
        }
        for (int64_t hh = 0; hh < 2 * k; ++hh) { order[hh].s = s[hh]; order[hh].h = (int32_t)hh; }
        qsort(order, (size_t)(2 * k), sizeof(ranked), ranked_cmp);
        { /* relative gap between the k-th and (k+1)-th candidate */
            float a = order[k - 1].s, c = order[k].s;
            if (isfinite(a) && isfinite(c)) {
                float den = fmaxf(fabsf(a), fabsf(c));
                float gap = den > 0.f ? (a - c) / den : 0.f;
                if (gap < gap_min) gap_min = gap;
            }
        }
        for (int64_t j = 0; j < k; ++j) t[j] = order[j].h;
        qsort(t, (size_t)k, sizeof(int32_t), index_cmp); /* survivors in ascending h */
        for (int64_t j = 0; j < k; ++j) { f[j] = Bf[t[j]]; l[j] = Bl[t[j]]; }
    }
    /* I[q, j] = first valid block of final node j, else empty */
    int64_t cnt = 0;
    for (int64_t j = 0; j < k; ++j)
        for (int64_t r = f[j]; r <= l[j]; ++r)
            if (Cblk[r]) { t[cnt++] = (int32_t)r; break; }
    qsort(t, (size_t)cnt, sizeof(int32_t), index_cmp);
    for (int64_t j = 0; j < k; ++j) {
        mask_row[j] = j < cnt ? t[j] : -1;
        if (score_row) score_row[j] = j < cnt ? tile_score(p, Q, K, b, h, q, t[j]) : -INFINITY;
    }
    if (min_gap) *min_gap = gap_min;
    if (tiles) *tiles = n_tiles;
    free(f); free(l); free(Bf); free(Bl); free(s); free(order); free(t); free(seen); free(cache); free(Cblk);
    return 0;
}

static int check_problem(const so_problem *p) {
    if (!p || p->batch < 1 || p->n_q_heads < 1 || p->n_kv_heads < 1 || p->n_q_heads % p->n_kv_heads) return -2;
    if (p->T < 1 || p->d < 1 || p->block_q < 1 || p->block_k < 1 || p->k_top < 1) return -2;
    if (p->dtype != 0 && p->dtype != 1) return -2;
    return 0;
}

/*
 * Algorithm 2 for the listed rows (rows == NULL: rows 0..n_rows-1).
 *   mask_out  [n_rows, k]  0-based key-block indices, strictly ascending, -1 padded
 *   score_out [n_rows, k]  optional: block score of each kept block (-inf padded)
 *   min_gap_out [n_rows]   optional: smallest relative gap between the k-th and (k+1)-th
 *                          candidate over all iterations (+inf if never both finite)
 *   tiles_out [n_rows]     optional: number of distinct representative blocks scored
 *   n_it_override          -1 = the paper's n_it; otherwise run exactly that many iterations
 */
int so_build_mask_rows(const so_problem *p, const void *Q, const void *K, const int64_t *rows, int64_t n_rows,
                       int32_t *mask_out, float *score_out, float *min_gap_out, int64_t *tiles_out,
                       int n_it_override, int flags) {
    int rc = check_problem(p);
    if (rc) return rc;
    const int64_t Nq = so_num_query_blocks(p), total = so_num_rows(p);
    int err = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < n_rows; ++i) {
        int64_t id = rows ? rows[i] : i;
        if (id < 0 || id >= total) { err = -3; continue; }
        int64_t q = id % Nq, h = (id / Nq) % p->n_q_heads, b = id / Nq / p->n_q_heads;
        if (stream_row(p, Q, K, b, h, q, n_it_override, flags, mask_out + i * p->k_top,
                       score_out ? score_out + i * p->k_top : NULL, min_gap_out ? min_gap_out + i : NULL,
                       tiles_out ? tiles_out + i : NULL))
            err = -1;
    }
    return err;
}

/*
 * Algorithm 2 with a sparsity constant of its own for every query block (the "variable k" the
 * paper's discussion of needle depth and its fourth limitation name as the remedy for the
 * stronger pruning of late rows; the paper leaves it undefined, so this is a reading): row
 * (b, h, q) is the unchanged algorithm run with k = k_row[q], clamped to 1 .. k_top. Rows are
 * k_top wide: the row's k entries, then -1 / -inf padding. Other arguments as above.
 */
int so_build_mask_rows_var(const so_problem *p, const void *Q, const void *K, const int32_t *k_row,
                           const int64_t *rows, int64_t n_rows, int32_t *mask_out, float *score_out,
                           float *min_gap_out, int64_t *tiles_out, int flags) {
    int rc = check_problem(p);
    if (rc) return rc;
    if (!k_row) return -2;
    const int64_t Nq = so_num_query_blocks(p), total = so_num_rows(p);
    int err = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < n_rows; ++i) {
        int64_t id = rows ? rows[i] : i;
        if (id < 0 || id >= total) { err = -3; continue; }
        int64_t q = id % Nq, h = (id / Nq) % p->n_q_heads, b = id / Nq / p->n_q_heads;
        so_problem pq = *p; /* the same problem with this row's k */
        pq.k_top = k_row[q] < 1 ? 1 : (k_row[q] > p->k_top ? p->k_top : k_row[q]);
        int32_t *m = malloc(sizeof(int32_t) * pq.k_top);
        float *sc = score_out ? malloc(sizeof(float) * pq.k_top) : NULL;
        if (!m || (score_out && !sc)) { err = -1; free(m); free(sc); continue; }
        if (stream_row(&pq, Q, K, b, h, q, -1, flags, m, sc, min_gap_out ? min_gap_out + i : NULL,
                       tiles_out ? tiles_out + i : NULL))
            err = -1;
        for (int64_t j = 0; j < p->k_top; ++j) {
            mask_out[i * p->k_top + j] = j < pq.k_top ? m[j] : -1;
            if (score_out) score_out[i * p->k_top + j] = j < pq.k_top ? sc[j] : -INFINITY;
        }
        free(m); free(sc);
    }
    return err;
}

/*
 * Algorithm 2 for several sparsity constants at once (the search over k of Section 3 and the
 * k_success / k_fail comparison of Section 4.2 need the masks of the same inputs for more than
 * one k). Mask i is the unchanged algorithm with k = k_list[i] (1 .. k_top); a block's score
 * does not depend on k, so an implementation may score each (row, block) tile once for all k.
 *   mask_out  [n_k, n_rows, k_top], score_out likewise (optional), min_gap_out [n_k, n_rows]
 *   tiles_out [n_rows]  optional: distinct representative blocks scored over ALL k of the row
 */
int so_build_mask_rows_multi(const so_problem *p, const void *Q, const void *K, int32_t n_k, const int32_t *k_list,
                             const int64_t *rows, int64_t n_rows, int32_t *mask_out, float *score_out,
                             float *min_gap_out, int64_t *tiles_out, int flags) {
    int rc = check_problem(p);
    if (rc) return rc;
    if (!k_list || n_k < 1) return -2;
    for (int32_t i = 0; i < n_k; ++i) if (k_list[i] < 1 || k_list[i] > p->k_top) return -2;
    const int64_t Nq = so_num_query_blocks(p), total = so_num_rows(p), N_k = padded_len(p) / p->block_k;
    int err = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < n_rows; ++i) {
        int64_t id = rows ? rows[i] : i;
        if (id < 0 || id >= total) { err = -3; continue; }
        int64_t q = id % Nq, h = (id / Nq) % p->n_q_heads, b = id / Nq / p->n_q_heads;
        unsigned char *seen = calloc((size_t)N_k, 1);
        int32_t *m = malloc(sizeof(int32_t) * p->k_top);
        float *sc = malloc(sizeof(float) * p->k_top);
        if (!seen || !m || !sc) { err = -1; free(seen); free(m); free(sc); continue; }
        int64_t n_tiles = 0;
        for (int32_t j = 0; j < n_k; ++j) {
            so_problem pk = *p;
            pk.k_top = k_list[j];
            int64_t fresh = 0;
            int64_t o = ((int64_t)j * n_rows + i);
            if (stream_row_seen(&pk, Q, K, b, h, q, -1, flags, m, sc, min_gap_out ? min_gap_out + o : NULL, &fresh, seen))
                err = -1;
            n_tiles += fresh;
            for (int64_t c = 0; c < p->k_top; ++c) {
                mask_out[o * p->k_top + c] = c < pk.k_top ? m[c] : -1;
                if (score_out) score_out[o * p->k_top + c] = c < pk.k_top ? sc[c] : -INFINITY;
            }
        }
        if (tiles_out) tiles_out[i] = n_tiles;
        free(seen); free(m); free(sc);
    }
    return err;
}

/*
 * A schedule for k_row: the effective-sparsity formula of the needle-depth experiment,
 * k = floor(1 + (n - 1) s), applied to each query block with n = the number of key blocks that
 * row may look at (the paper applies it once with n = T / b_q; taking the row's own count is
 * what makes the pruning ratio the same from the top to the bottom of a causal pattern).
 * Clamped to 1 .. k_top. k_row_out has ceil(T / b_q) entries.
 */
int so_k_schedule(const so_problem *p, double s, int32_t *k_row_out) {
    int rc = check_problem(p);
    if (rc) return rc;
    if (!(s > 0.0 && s < 1.0)) return -2;
    const int64_t Nq = so_num_query_blocks(p), N_k = padded_len(p) / p->block_k;
    for (int64_t q = 0; q < Nq; ++q) {
        int64_t n = 0;
        for (int64_t r = 0; r < N_k; ++r) n += c_blk(p, q, r);
        int64_t k = (int64_t)floor(1.0 + (double)(n - 1) * s);
        k_row_out[q] = (int32_t)(k < 1 ? 1 : (k > p->k_top ? p->k_top : k));
    }
    return 0;
}

/*
 * The effective-sparsity formula of Section 4.2 as it is printed, applied once to the whole
 * context: k = floor(1 + (T / b_q - 1) s) with T / b_q the real quotient, kept inside k's range
 * 1 .. floor(T / b_q) (Section 3), and never below 1. Returns k, or a negative code.
 */
int64_t so_effective_k(int64_t T, int64_t block_q, double s) {
    if (T < 1 || block_q < 1 || !(s >= 0.0 && s <= 1.0)) return -2;
    const double n = (double)T / (double)block_q;
    int64_t k = (int64_t)floor(1.0 + (n - 1.0) * s);
    const int64_t k_max = T / block_q;
    if (k > k_max) k = k_max;
    if (k < 1) k = 1;
    return k;
}

/*
 * Eq. 2 on block masks: for every query token of each listed row, softmax over the keys of the
 * row's selected blocks that C allows, then the weighted sum of V, all in fp64.
 *   mask [n_rows, k]  as produced above; out [n_rows, b_q, d] fp64; tokens beyond T or with no
 *   allowed key give zeros.
 */
int so_sparse_attention_rows(const so_problem *p, const void *Q, const void *K, const void *V,
                             const int64_t *rows, int64_t n_rows, const int32_t *mask, double scale,
                             double *out) {
    int rc = check_problem(p);
    if (rc) return rc;
    const int64_t Nq = so_num_query_blocks(p), total = so_num_rows(p), d = p->d;
    int err = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < n_rows; ++i) {
        int64_t id = rows ? rows[i] : i;
        if (id < 0 || id >= total) { err = -3; continue; }
        int64_t q = id % Nq, h = (id / Nq) % p->n_q_heads, b = id / Nq / p->n_q_heads;
        int64_t g = h / (p->n_q_heads / p->n_kv_heads);
        const int32_t *row = mask + i * p->k_top;
        int64_t max_keys = (int64_t)p->k_top * p->block_k;
        double *logit = malloc(sizeof(double) * (size_t)max_keys);
        int64_t *key = malloc(sizeof(int64_t) * (size_t)max_keys);
        if (!logit || !key) { err = -1; free(logit); free(key); continue; }
        for (int64_t m = 0; m < p->block_q; ++m) {
            int64_t tq = q * p->block_q + m;
            double *o = out + (i * p->block_q + m) * d;
            for (int64_t c = 0; c < d; ++c) o[c] = 0.0;
            int64_t nk = 0;
            double mx = -INFINITY;
            for (int64_t j = 0; j < p->k_top; ++j) {
                if (row[j] < 0) continue;
                for (int64_t n = 0; n < p->block_k; ++n) {
                    int64_t tk = (int64_t)row[j] * p->block_k + n;
                    if (!valid_pair(p, tq, tk)) continue;
                    int64_t qo = ((b * p->n_q_heads + h) * p->T + tq) * d;
                    int64_t ko = ((b * p->n_kv_heads + g) * p->T + tk) * d;
                    double acc = 0.0;
                    for (int64_t c = 0; c < d; ++c) acc += load_elem(Q, qo + c, p->dtype) * load_elem(K, ko + c, p->dtype);
                    logit[nk] = scale * acc;
                    key[nk] = tk;
                    if (logit[nk] > mx) mx = logit[nk];
                    ++nk;
                }
            }
            if (nk == 0) continue;
            double den = 0.0;
            for (int64_t x = 0; x < nk; ++x) { logit[x] = exp(logit[x] - mx); den += logit[x]; }
            for (int64_t x = 0; x < nk; ++x) {
                int64_t vo = ((b * p->n_kv_heads + g) * p->T + key[x]) * d;
                double w = logit[x] / den;
                for (int64_t c = 0; c < d; ++c) o[c] += w * load_elem(V, vo + c, p->dtype);
            }
        }
        free(logit); free(key);
    }
    return err;
}

/*
 * Vertical attention scores of a block mask and their kurtosis (Section 4.1: receiver heads are
 * the heads whose vertical scores have high kurtosis, i.e. a few key blocks take most of the
 * attention of the later queries).
 *   mask   [batch * n_q_heads * n_query_blocks, k]  as produced by so_build_mask_rows for all rows
 *   score  same shape or NULL: weight of each kept block (NULL: every kept block counts 1)
 *   vertical_out [batch * n_q_heads, n_key_blocks]  v[h, r] = sum over query blocks q and slots j
 *                                                   with mask[h, q, j] == r of the weight
 *   kurtosis_out [batch * n_q_heads]  m4 / m2^2 of v[h, :] (central moments over the n_key_blocks
 *                                     columns, not excess); 0 when the scores are all equal
 * Everything in fp64, in index order. n_key_blocks = ceil(T / b_k).
 */
int so_vertical_scores(const so_problem *p, const int32_t *mask, const float *score, double *vertical_out,
                       double *kurtosis_out) {
    int rc = check_problem(p);
    if (rc) return rc;
    const int64_t Nq = so_num_query_blocks(p), Nk = (p->T + p->block_k - 1) / p->block_k;
    const int64_t heads = (int64_t)p->batch * p->n_q_heads;
    for (int64_t h = 0; h < heads; ++h) {
        double *v = vertical_out + h * Nk;
        for (int64_t r = 0; r < Nk; ++r) v[r] = 0.0;
        for (int64_t q = 0; q < Nq; ++q)
            for (int64_t j = 0; j < p->k_top; ++j) {
                int64_t at = (h * Nq + q) * p->k_top + j;
                int32_t r = mask[at];
                if (r < 0) continue;
                if (r >= Nk) return -4;
                v[r] += score ? (double)score[at] : 1.0;
            }
        if (kurtosis_out) {
            double mean = 0.0, m2 = 0.0, m4 = 0.0;
            for (int64_t r = 0; r < Nk; ++r) mean += v[r];
            mean /= (double)Nk;
            for (int64_t r = 0; r < Nk; ++r) {
                double dlt = v[r] - mean;
                m2 += dlt * dlt;
                m4 += dlt * dlt * dlt * dlt;
            }
            m2 /= (double)Nk;
            m4 /= (double)Nk;
            kurtosis_out[h] = m2 > 0.0 ? m4 / (m2 * m2) : 0.0;
        }
    }
    return 0;
}

/*
 * Mask subtraction (Section 4.2, "Exploring Information Flow": the masks found with a smaller k
 * are subtracted from those found with a larger k, and what is left - weighted by the larger
 * mask's block scores - are the connections that only the larger budget keeps).
 *   mask_a [n_rows, k_a], score_a same shape or NULL; mask_b [n_rows, k_b]
 *   diff_out [n_rows, k_a]: the entries of row a (in their order) that are >= 0 and do not occur
 *   in row b, then -1 padding; diff_score_out (if score_a): their scores, then -inf padding.
 */
int so_mask_difference(int64_t n_rows, int32_t k_a, const int32_t *mask_a, const float *score_a, int32_t k_b,
                       const int32_t *mask_b, int32_t *diff_out, float *diff_score_out) {
    if (n_rows < 0 || k_a < 1 || k_b < 1 || !mask_a || !mask_b || !diff_out) return -2;
    for (int64_t i = 0; i < n_rows; ++i) {
        const int32_t *a = mask_a + i * k_a, *b = mask_b + i * k_b;
        int32_t n = 0;
        for (int32_t j = 0; j < k_a; ++j) {
            if (a[j] < 0) continue;
            int found = 0;
            for (int32_t u = 0; u < k_b; ++u) if (b[u] == a[j]) found = 1;
            if (found) continue;
            diff_out[i * k_a + n] = a[j];
            if (score_a && diff_score_out) diff_score_out[i * k_a + n] = score_a[i * k_a + j];
            ++n;
        }
        for (; n < k_a; ++n) {
            diff_out[i * k_a + n] = -1;
            if (score_a && diff_score_out) diff_score_out[i * k_a + n] = -INFINITY;
        }
    }
    return 0;
}
