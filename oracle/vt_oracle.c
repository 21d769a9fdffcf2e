/*
 * CPU oracle for the VocabTrim hot path.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, obviously-correct restatement of what the trimmed-vocabulary drafter head and
 * the vocabulary build compute.  It shares no code, header, table or constant with the CUDA
 * library; only tests, the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * Floating point is fp64 throughout (the paper fixes no precision); bf16 inputs are decoded
 * exactly.  Each function states the passage of the paper it follows.  Where the paper is
 * silent (tie rules, clamping of uniforms, order of the map) the reading is noted inline.
 *
 * Parity pins: every function here is pinned by CPU tests against closed forms, invariants,
 * library special cases and brute force.  The paper prints no worked numeric example for the
 * head or the vocabulary build, so parity with *paper-printed values* is unpinned there; parity
 * with the definitions is pinned.  The speed-up formula of the Python face is pinned to the
 * (block efficiency, speed-up) pairs the paper's Table 1 prints.
 *
 * Threading: the only parallel construct is an OpenMP "parallel for" over independent
 * vocabulary rows in orc_logits (each dot product is still summed in index order by one
 * thread).  Everything else is single-threaded.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* bf16 is the upper half of an IEEE fp32 word: decoding is exact. */
static double bf16_to_double(uint16_t b) {
    uint32_t w = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

void orc_decode_bf16(const uint16_t *x, int64_t n, double *out) {
    for (int64_t i = 0; i < n; ++i) out[i] = bf16_to_double(x[i]);
}

int orc_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void orc_set_threads(int t) {
#ifdef _OPENMP
    if (t > 0) omp_set_num_threads(t);
#else
    (void)t;
#endif
}

/*
 * Algorithm 1 (Count Token Frequencies): start from a zero counter vector c over the
 * vocabulary and add one for every token of the calibration stream.  Tokenisation is outside
 * the path: the stream is already ids.  Reading for ids outside [0,V): skipped and counted in
 * *n_bad (the algorithm assumes valid ids).  If accumulate != 0 the counts are added to what
 * `counts` already holds (chunked corpora).
 */
void orc_histogram(const int32_t *ids, int64_t n, int32_t V, uint64_t *counts, int accumulate,
                   uint64_t *n_bad) {
    if (!accumulate)
        for (int32_t v = 0; v < V; ++v) counts[v] = 0;
    uint64_t bad = 0;
    for (int64_t i = 0; i < n; ++i) {
        int32_t t = ids[i];
        if (t >= 0 && t < V)
            counts[t] += 1;
        else
            bad += 1;
    }
    if (n_bad) *n_bad = bad;
}

/*
 * Eq. 1, first line: V_trim = V[Top-K(c, k)].  Reading: the K ids with the largest counts,
 * listed in rank order (most frequent first); equal counts are ordered by ascending id, so ids
 * that never occurred fill the tail in id order when fewer than K ids were seen.
 * Written as the definition: a full sort of all V (count, id) pairs.
 * map[j] = id of rank j (j < K); inv_map[v] = j if map[j] == v, else -1.
 */
typedef struct {
    uint64_t count;
    int32_t id;
} orc_pair;

static int orc_pair_cmp(const void *a, const void *b) {
    const orc_pair *x = (const orc_pair *)a, *y = (const orc_pair *)b;
    if (x->count != y->count) return (x->count > y->count) ? -1 : 1; /* count descending */
    if (x->id != y->id) return (x->id < y->id) ? -1 : 1;             /* id ascending   */
    return 0;
}

int orc_select_topk(const uint64_t *counts, int32_t V, int32_t K, int32_t *map,
                    int32_t *inv_map) {
    if (V <= 0 || K <= 0 || K > V) return 1;
    orc_pair *p = (orc_pair *)malloc(sizeof(orc_pair) * (size_t)V);
    if (!p) return 2;
    for (int32_t v = 0; v < V; ++v) {
        p[v].count = counts[v];
        p[v].id = v;
    }
    qsort(p, (size_t)V, sizeof(orc_pair), orc_pair_cmp);
    for (int32_t v = 0; v < V; ++v) inv_map[v] = -1;
    for (int32_t j = 0; j < K; ++j) {
        map[j] = p[j].id;
        inv_map[p[j].id] = j;
    }
    free(p);
    return 0;
}

/*
 * Selection variants the Method section names next to Top-K: "Top-P" and "minimum frequency of
 * tokens".  Both cut the same ranking (count descending, id ascending) at a data-dependent K:
 *   Top-P:        the smallest K whose K most frequent ids hold at least ceil(p * total) of all
 *                 counted tokens (p in (0,1]; total = sum of counts);
 *   min frequency: K = number of ids with count >= min_count.
 * Readings where the paper is silent: the target is ceil(p*total) evaluated in fp64; K is never
 * below 1 (an empty vocabulary is useless).  map receives the FULL ranking [V]; inv_map is -1
 * for ranks >= K.  Returns K, or -1 on invalid arguments.
 */
static int32_t orc_cut_ranking(const uint64_t *counts, int32_t V, int32_t K, const orc_pair *p,
                               int32_t *map, int32_t *inv_map) {
    (void)counts;
    if (K < 1) K = 1;
    if (K > V) K = V;
    for (int32_t j = 0; j < V; ++j) {
        map[j] = p[j].id;
        inv_map[p[j].id] = j < K ? j : -1;
    }
    return K;
}

static orc_pair *orc_rank_all(const uint64_t *counts, int32_t V) {
    orc_pair *p = (orc_pair *)malloc(sizeof(orc_pair) * (size_t)V);
    if (!p) return NULL;
    for (int32_t v = 0; v < V; ++v) {
        p[v].count = counts[v];
        p[v].id = v;
    }
    qsort(p, (size_t)V, sizeof(orc_pair), orc_pair_cmp);
    return p;
}

int32_t orc_select_topp(const uint64_t *counts, int32_t V, double pfrac, int32_t *map,
                        int32_t *inv_map) {
    if (V <= 0 || !(pfrac > 0.0) || pfrac > 1.0) return -1;
    orc_pair *p = orc_rank_all(counts, V);
    if (!p) return -1;
    uint64_t total = 0;
    for (int32_t v = 0; v < V; ++v) total += counts[v];
    const double target = ceil(pfrac * (double)total);
    uint64_t cum = 0;
    int32_t K = V;
    for (int32_t j = 0; j < V; ++j) {
        cum += p[j].count;
        if ((double)cum >= target) { K = j + 1; break; }
    }
    K = orc_cut_ranking(counts, V, K, p, map, inv_map);
    free(p);
    return K;
}

int32_t orc_select_minfreq(const uint64_t *counts, int32_t V, uint64_t min_count, int32_t *map,
                           int32_t *inv_map) {
    if (V <= 0) return -1;
    orc_pair *p = orc_rank_all(counts, V);
    if (!p) return -1;
    int32_t K = 0;
    for (int32_t v = 0; v < V; ++v) K += counts[v] >= min_count;
    K = orc_cut_ranking(counts, V, K, p, map, inv_map);
    free(p);
    return K;
}

/* Eq. 1, second line: W_trim = W[Top-K(c,k), :] -- a row gather, bit copy of bf16 words. */
void orc_trim_head(const uint16_t *W_full, const int32_t *map, int32_t K, int32_t d,
                   uint16_t *W_trim) {
    for (int32_t j = 0; j < K; ++j)
        for (int32_t i = 0; i < d; ++i)
            W_trim[(int64_t)j * d + i] = W_full[(int64_t)map[j] * d + i];
}

/*
 * Algorithm 2, the drafter forward with the trimmed head, head part only: the LM head is
 * a linear projection without bias, logit[b][j] = sum_i h[b][i] * W[j][i], summed in index
 * order in fp64 on exactly-decoded bf16 operands.  logits is [B,K] row-major.
 */
void orc_logits(const uint16_t *h, const uint16_t *W, int32_t B, int32_t K, int32_t d,
                double *logits) {
    double *hd = (double *)malloc(sizeof(double) * (size_t)B * (size_t)d);
    for (int64_t i = 0; i < (int64_t)B * d; ++i) hd[i] = bf16_to_double(h[i]);
#pragma omp parallel for schedule(static)
    for (int32_t j = 0; j < K; ++j) {
        const uint16_t *w = W + (int64_t)j * d;
        for (int32_t b = 0; b < B; ++b) {
            const double *hb = hd + (int64_t)b * d;
            double acc = 0.0;
            for (int32_t i = 0; i < d; ++i) acc += hb[i] * bf16_to_double(w[i]);
            logits[(int64_t)b * K + j] = acc;
        }
    }
    free(hd);
}

/*
 * Temperature softmax of one row: z = logit / T, m = max z, lse = m + log sum exp(z - m),
 * logp = z - lse.  Writes z[K] and returns lse.
 */
double orc_softmax_row(const double *logit, int32_t K, double T, double *z) {
    double m = -INFINITY;
    for (int32_t j = 0; j < K; ++j) {
        z[j] = logit[j] / T;
        if (z[j] > m) m = z[j];
    }
    double s = 0.0;
    for (int32_t j = 0; j < K; ++j) s += exp(z[j] - m);
    return m + log(s);
}

/*
 * Top-k candidates of one row for tree drafting (the paper's trees take the top-K tokens per
 * node): full sort of the indices by (z descending, index ascending), keep the first `topk`.
 */
typedef struct {
    double z;
    int32_t j;
} orc_zj;

static int orc_zj_cmp(const void *a, const void *b) {
    const orc_zj *x = (const orc_zj *)a, *y = (const orc_zj *)b;
    if (x->z != y->z) return (x->z > y->z) ? -1 : 1;
    if (x->j != y->j) return (x->j < y->j) ? -1 : 1;
    return 0;
}

void orc_topk_row(const double *z, int32_t K, int32_t topk, int32_t *idx) {
    orc_zj *p = (orc_zj *)malloc(sizeof(orc_zj) * (size_t)K);
    for (int32_t j = 0; j < K; ++j) {
        p[j].z = z[j];
        p[j].j = j;
    }
    qsort(p, (size_t)K, sizeof(orc_zj), orc_zj_cmp);
    for (int32_t r = 0; r < topk; ++r) idx[r] = p[r].j;
    free(p);
}

/*
 * Gumbel-max draw of one row from caller-supplied uniforms: u' = clamp(u, 2^-24, 1 - 2^-24)
 * taken in fp32, g = -log(-log u') in fp64, result = argmax_j (z_j + g_j), first maximal index
 * on ties.  score[K] (optional) receives z + g.
 */
int32_t orc_gumbel_row(const double *z, const float *u, int32_t K, double *score) {
    const float lo = 0x1p-24f, hi = 1.0f - 0x1p-24f;
    int32_t best = 0;
    double best_s = -INFINITY;
    for (int32_t j = 0; j < K; ++j) {
        float uc = u[j];
        if (uc < lo) uc = lo;
        if (uc > hi) uc = hi;
        double g = -log(-log((double)uc));
        double sc = z[j] + g;
        if (score) score[j] = sc;
        if (sc > best_s) {
            best_s = sc;
            best = j;
        }
    }
    return best;
}

/*
 * Algorithm 2 (drafter forward over the trimmed head, then the index mapping), head part: projection, temperature softmax, top-k candidates, Gumbel
 * draw, then the index mapper T_{d->t}: every reported trimmed index j becomes map[j]
 * (map == NULL means the identity, i.e. the untrimmed head).
 *
 * Output layout, per row b (row length 1 + topk):
 *   out_ids[b][0]      sampled id (the greedy id when uniforms == NULL)
 *   out_ids[b][1 + r]  r-th best candidate, r = 0 is the greedy argmax
 *   out_logprobs[b][c] log softmax(logits / T_b) of the id in the same column
 * out_trim (optional, same shape) receives the trimmed indices before the remap.
 * z_out [B,K], lse_out [B] and score_out [B,K] (z + g; only when uniforms != NULL) are optional.
 */
int orc_draft_head(const uint16_t *h, const uint16_t *W_trim, const int32_t *map, int32_t B,
                   int32_t K, int32_t d, const float *temp, int32_t topk,
                   const float *uniforms, int32_t *out_ids, double *out_logprobs,
                   int32_t *out_trim, double *logits_out, double *z_out, double *lse_out,
                   double *score_out) {
    if (B <= 0 || K <= 0 || d <= 0 || topk <= 0 || topk > K) return 1;
    double *logits = logits_out ? logits_out : (double *)malloc(sizeof(double) * (size_t)B * K);
    double *z = (double *)malloc(sizeof(double) * (size_t)K);
    int32_t *cand = (int32_t *)malloc(sizeof(int32_t) * (size_t)topk);
    orc_logits(h, W_trim, B, K, d, logits);
    const int32_t row = 1 + topk;
    for (int32_t b = 0; b < B; ++b) {
        double T = (double)temp[b];
        double lse = orc_softmax_row(logits + (int64_t)b * K, K, T, z);
        if (z_out) memcpy(z_out + (int64_t)b * K, z, sizeof(double) * (size_t)K);
        if (lse_out) lse_out[b] = lse;
        orc_topk_row(z, K, topk, cand);
        int32_t sampled = cand[0];
        if (uniforms)
            sampled = orc_gumbel_row(z, uniforms + (int64_t)b * K, K,
                                     score_out ? score_out + (int64_t)b * K : NULL);
        int32_t *oi = out_ids + (int64_t)b * row;
        double *ol = out_logprobs + (int64_t)b * row;
        int32_t *ot = out_trim ? out_trim + (int64_t)b * row : NULL;
        for (int32_t c = 0; c < row; ++c) {
            int32_t j = (c == 0) ? sampled : cand[c - 1];
            if (ot) ot[c] = j;
            oi[c] = map ? map[j] : j;
            ol[c] = z[j] - lse;
        }
    }
    free(cand);
    free(z);
    if (!logits_out) free(logits);
    return 0;
}

/*
 * Greedy verification of one drafted block (Experiments section: the target decodes greedily and a
 * draft token is accepted only when it equals the target's token; Algorithm 2's accept loop).
 *   token[i]   drafted id of node i, already a full-vocabulary id (after the index mapper);
 *   parent[i]  index of node i's parent, -1 for a child of the last committed token; a node whose
 *              parent is not in [-1, i) can never be reached.  parent == NULL means a chain
 *              (parent[i] = i - 1);
 *   target[0]  the target's greedy token after the committed prefix, target[i + 1] the one after
 *              the path ending in node i.
 * Walk from the committed prefix: at the current node the target's token decides; the child that
 * carries exactly this token (the lowest-indexed one, should several) is accepted and becomes the
 * current node; with no such child the block ends.  The target's token at the last accepted node
 * is emitted after the accepted ones, so a block yields n + 1 tokens, at most depth + 1.
 * Returns n; path[0..n) = accepted node indices, emitted[0..n] = the tokens of the block.
 */
int32_t orc_verify_greedy(const int32_t *token, const int32_t *parent, const int32_t *target,
                          int32_t N, int32_t *path, int32_t *emitted) {
    int32_t cur = -1, n = 0;
    for (;;) {
        const int32_t want = target[cur + 1];
        int32_t next = -1;
        for (int32_t i = cur + 1; i < N && next < 0; ++i) {
            const int32_t par = parent ? parent[i] : i - 1;
            if (par == cur && token[i] == want) next = i;
        }
        if (next < 0) break;
        path[n] = next;
        emitted[n] = token[next];
        ++n;
        cur = next;
    }
    emitted[n] = target[cur + 1];
    return n;
}
