/*
 * CPU oracle for the random-walk + skip-gram-with-negative-sampling (SGNS)
 * path of GraphScale-style node-embedding training.
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is a plain, slow, single-threaded
 * restatement of what the path computes, in fp64 for every floating-point
 * quantity, written so that it can be checked against the definitions by eye.
 * It shares no code, header, table or helper with the CUDA library and must
 * never be called from the product path.
 *
 * What the paper fixes (Section 2.2 "Node embedding training", Section 3.2
 * "Node Embedding Training", Section 4 "Configuration"):
 *   - DeepWalk = random walks from every node fed to skip-gram; node2vec = the
 *     same with a biased second-order walk (Section 2.2);
 *   - training uses skip-gram with negative sampling (Section 2.2);
 *   - a mini-batch of B source nodes touches at most B x walk_len nodes,
 *     sources included, so walk_len counts NODES (Section 3.2);
 *   - updates of a mini-batch are written as increments, and trainers may race
 *     on the same rows, Hogwild style (Section 3.2 "Synchronization").
 * Everything the paper leaves open (RNG, index mapping, negative distribution,
 * masking, gradient scaling) is a reading; each function below states the
 * reading it implements.
 *
 * Parity pins (see tests, "not gpu"): Philox known answers; walks follow
 * edges; degree-proportional stationarity; node2vec closed-form transition
 * weights; pair-count identity; alias-table mass identity; finite-difference
 * gradients; closed form of the first step from zero output vectors;
 * pair-order independence of the synchronous step; for the variants (window
 * shrinking, sub-sampling, start shuffle, Adam): window range, symmetry and
 * uniformity, exact keep thresholds at f = 4t and 16t with binomial retention
 * counts, bijectivity and uniformity of the shuffle, torch's Adam and
 * SparseAdam.
 * gso_sgns_seq_from_lists (sequential per-pair SGD, the reference point for
 * the racy Hogwild mode) has no exact counterpart on the GPU: parity unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------
 * Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as
 * easy as 1, 2, 3", SC'11).  Ten rounds; each round multiplies two counter
 * words by fixed odd constants, mixes high halves with the other two words
 * and the key, and the key is bumped by Weyl constants between rounds.
 * ---------------------------------------------------------------------- */
void gso_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Stream tags: which consumer of random words a counter belongs to. */
enum { TAG_UNIFORM_WALK = 1, TAG_NODE2VEC = 2, TAG_NEGATIVE = 3, TAG_INIT = 4,
       TAG_WINDOW = 5, TAG_SUBSAMPLE = 6, TAG_SHUFFLE = 7, TAG_ROUND_SYNC = 8, TAG_ROUND_LOCKFREE = 9 };

/* Keying shared (as a published convention, not as code) with the GPU path:
 * key = 64-bit seed; counter = (id low, id high, step, tag<<24 | sub). */
static void draw4(uint64_t seed, uint64_t id, uint32_t step, uint32_t tag, uint32_t sub,
                  uint32_t out[4])
{
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t ctr[4] = { (uint32_t)id, (uint32_t)(id >> 32), step, (tag << 24) | sub };
    gso_philox4x32_10(ctr, key, out);
}

/* Map a 32-bit word to [0, n) by multiply-high (bias <= n / 2^32, no rejection). */
static uint64_t scale32(uint32_t r, uint64_t n)
{
    return ((uint64_t)r * n) >> 32;
}

/* ------------------------------------------------------------------------
 * Uniform (DeepWalk) walks.  Section 2.2: every node is the source of walks.
 * walk[0] = start; each transition picks a uniformly random out-neighbour.
 * A node without out-neighbours ends the walk; the remaining entries are -1.
 * starts == NULL means start node = walk id mod n_nodes.
 * Returns the number of transitions taken over all walks.
 * ---------------------------------------------------------------------- */
int64_t gso_uniform_walks(int64_t n_nodes, const int64_t *off, const int32_t *col,
                          const int32_t *starts, int64_t n_walks, int64_t walk_id_base,
                          int32_t L, uint64_t seed, int32_t *walks)
{
    int64_t steps = 0;
    for (int64_t i = 0; i < n_walks; ++i) {
        uint64_t id = (uint64_t)(walk_id_base + i);
        int32_t *W = walks + i * (int64_t)L;
        int32_t cur = starts ? starts[i] : (int32_t)(id % (uint64_t)n_nodes);
        W[0] = cur;
        int32_t t = 0;
        for (; t + 1 < L; ++t) {
            int64_t deg = off[cur + 1] - off[cur];
            if (deg == 0) break;
            uint32_t r[4];
            draw4(seed, id, (uint32_t)t, TAG_UNIFORM_WALK, 0, r);
            cur = col[off[cur] + (int64_t)scale32(r[0], (uint64_t)deg)];
            W[t + 1] = cur;
            ++steps;
        }
        for (int32_t s = t + 1; s < L; ++s) W[s] = -1;
    }
    return steps;
}

/* ------------------------------------------------------------------------
 * node2vec second-order walks (Grover & Leskovec, KDD'16; named in Section
 * 2.2).  Unnormalised weight of candidate x after the move prev -> cur:
 *   1/p if x == prev;  1 if x is a neighbour of prev;  1/q otherwise.
 * Sampled by rejection: propose x uniformly from adj(cur), accept with
 * probability weight / max(1/p, 1, 1/q).  Acceptance compares a 32-bit word
 * with an integer threshold T[class] = floor(weight/max * 2^32).
 * ---------------------------------------------------------------------- */
void gso_node2vec_thresholds(double p, double q, uint64_t T[3])
{
    double a_prev = 1.0 / p, a_near = 1.0, a_far = 1.0 / q;
    double m = a_prev;
    if (a_near > m) m = a_near;
    if (a_far > m) m = a_far;
    double a[3] = { a_prev, a_near, a_far };
    for (int c = 0; c < 3; ++c) {
        double v = floor(a[c] / m * 4294967296.0);
        if (v > 4294967296.0) v = 4294967296.0;
        T[c] = (uint64_t)v;
    }
}

/* membership test in a strictly increasing adjacency list */
static int is_neighbour(const int64_t *off, const int32_t *col, int32_t u, int32_t x)
{
    int64_t lo = off[u], hi = off[u + 1];
    while (lo < hi) {
        int64_t mid = lo + (hi - lo) / 2;
        if (col[mid] < x) lo = mid + 1; else hi = mid;
    }
    return lo < off[u + 1] && col[lo] == x;
}

int64_t gso_node2vec_walks(int64_t n_nodes, const int64_t *off, const int32_t *col,
                           const int32_t *starts, int64_t n_walks, int64_t walk_id_base,
                           int32_t L, uint64_t seed, double p, double q, int32_t max_rounds,
                           int32_t *walks, int64_t *cap_hits)
{
    uint64_t T[3];
    gso_node2vec_thresholds(p, q, T);
    int64_t steps = 0, caps = 0;
    for (int64_t i = 0; i < n_walks; ++i) {
        uint64_t id = (uint64_t)(walk_id_base + i);
        int32_t *W = walks + i * (int64_t)L;
        int32_t cur = starts ? starts[i] : (int32_t)(id % (uint64_t)n_nodes);
        int32_t prev = -1;
        W[0] = cur;
        int32_t t = 0;
        for (; t + 1 < L; ++t) {
            int64_t deg = off[cur + 1] - off[cur];
            if (deg == 0) break;
            int32_t nxt = -1;
            if (t == 0) {
                /* no predecessor yet: plain uniform choice */
                uint32_t r[4];
                draw4(seed, id, 0u, TAG_NODE2VEC, 0, r);
                nxt = col[off[cur] + (int64_t)scale32(r[0], (uint64_t)deg)];
            } else {
                int accepted = 0;
                for (int32_t s = 0; s < max_rounds && !accepted; ++s) {
                    uint32_t r[4];
                    draw4(seed, id, (uint32_t)t, TAG_NODE2VEC, (uint32_t)s, r);
                    int32_t x = col[off[cur] + (int64_t)scale32(r[0], (uint64_t)deg)];
                    int cls = (x == prev) ? 0 : (is_neighbour(off, col, prev, x) ? 1 : 2);
                    nxt = x;
                    if ((uint64_t)r[1] < T[cls]) accepted = 1;
                }
                if (!accepted) ++caps;   /* keeps the last proposal */
            }
            prev = cur;
            cur = nxt;
            W[t + 1] = cur;
            ++steps;
        }
        for (int32_t s = t + 1; s < L; ++s) W[s] = -1;
    }
    if (cap_hits) *cap_hits = caps;
    return steps;
}

/* ------------------------------------------------------------------------
 * Window expansion and negative draws.
 * For position i of a walk and every j with 0 < |i-j| <= w inside the walk,
 * both entries present: pair (center = W[i], context = W[j]) in slot
 * sigma = j - i + w - (j > i), 0 <= sigma < 2w.  (Fixed window; Section 4
 * gives only "window-size".)
 * For each pair, K negatives from the alias table (thr, alias) over n_alias
 * nodes: word pair (a, b) -> cell jj = mulhi(a, n_alias); keep jj if
 * b < thr[jj] else alias[jj].  Negatives 2m and 2m+1 use words (0,1) and
 * (2,3) of the Philox block with step = i*2w + sigma, sub = m.
 *
 * forward_only != 0 keeps only the pairs with j > i.
 * shrink != 0 draws a window per center position, as word2vec does (Mikolov
 * et al. 2013 describe the effect as giving nearer words more weight): position
 * i of walk `id` uses w_i = 1 + mulhi(word 0 of the block with step = i,
 * TAG_WINDOW, sub 0; w), uniform on 1..w, and keeps the pairs with
 * |i-j| <= w_i.  Slots and the keying of the negatives are those of the full
 * window, so a kept pair has the same negatives with or without shrinking.
 * Output lists are laid out by slot: entry e = (walk*L + i)*2w + sigma;
 * centers[e] = contexts[e] = -1 and negs[e*K..] = -1 where no pair exists.
 * Returns the number of pairs.
 * ---------------------------------------------------------------------- */
int64_t gso_expand_lists(const int32_t *walks, int64_t n_walks, int64_t walk_id_base,
                         int32_t L, int32_t w, int32_t K,
                         const uint32_t *thr, const int32_t *alias, int64_t n_alias,
                         uint64_t seed, int32_t forward_only, int32_t shrink,
                         int32_t *centers, int32_t *contexts, int32_t *negs)
{
    int64_t n_pairs = 0;
    const int32_t S = 2 * w;
    for (int64_t a = 0; a < n_walks; ++a) {
        const int32_t *W = walks + a * (int64_t)L;
        uint64_t id = (uint64_t)(walk_id_base + a);
        for (int32_t i = 0; i < L; ++i) {
            int32_t w_i = w;
            if (shrink) {
                uint32_t r[4];
                draw4(seed, id, (uint32_t)i, TAG_WINDOW, 0, r);
                w_i = 1 + (int32_t)scale32(r[0], (uint64_t)w);
            }
            for (int32_t sg = 0; sg < S; ++sg) {
                int64_t e = (a * (int64_t)L + i) * S + sg;
                /* invert sigma = j - i + w - (j > i) */
                int32_t j = (sg < w) ? (i - w + sg) : (i - w + sg + 1);
                int ok = (W[i] >= 0) && (j >= 0) && (j < L) && (W[j] >= 0);
                /* forward_only: only contexts that come later in the walk.  With walks of two
                 * nodes and w = 1 this is the edge sampling of LINE (Section 3.2: a source, one
                 * positive and num_neg negatives per source node). */
                if (forward_only && j < i) ok = 0;
                if (j - i > w_i || i - j > w_i) ok = 0;
                centers[e] = ok ? W[i] : -1;
                contexts[e] = ok ? W[j] : -1;
                for (int32_t k = 0; k < K; ++k) negs[e * K + k] = -1;
                if (!ok) continue;
                ++n_pairs;
                for (int32_t m = 0; 2 * m < K; ++m) {
                    uint32_t r[4];
                    draw4(seed, id, (uint32_t)(i * S + sg), TAG_NEGATIVE, (uint32_t)m, r);
                    for (int h = 0; h < 2 && 2 * m + h < K; ++h) {
                        uint32_t ra = r[2 * h], rb = r[2 * h + 1];
                        int64_t jj = (int64_t)scale32(ra, (uint64_t)n_alias);
                        negs[e * K + 2 * m + h] = (rb < thr[jj]) ? (int32_t)jj : alias[jj];
                    }
                }
            }
        }
    }
    return n_pairs;
}

/* ------------------------------------------------------------------------
 * Alias table (Walker / Vose) for p(v) proportional to weight(v)^power;
 * zero-weight entries get probability zero.  Cells are processed through
 * two first-in-first-out queues filled in increasing node order, so the
 * table is a deterministic function of the weights.
 * thr[v] = floor(keep_probability * 2^32) capped at 2^32 - 1; a cell whose
 * keep probability is one aliases to itself, which makes the cap harmless.
 * Returns 0, or -1 when no weight is positive / allocation fails.
 * ---------------------------------------------------------------------- */
int gso_build_alias(const double *weights, int64_t n, double power,
                    uint32_t *thr, int32_t *alias)
{
    double *s = (double *)malloc(sizeof(double) * (size_t)n);
    int64_t *small = (int64_t *)malloc(sizeof(int64_t) * (size_t)n);
    int64_t *large = (int64_t *)malloc(sizeof(int64_t) * (size_t)n);
    if (!s || !small || !large) { free(s); free(small); free(large); return -1; }
    double total = 0.0;
    for (int64_t v = 0; v < n; ++v) {
        s[v] = weights[v] > 0.0 ? pow(weights[v], power) : 0.0;
        total += s[v];
    }
    if (!(total > 0.0)) { free(s); free(small); free(large); return -1; }
    int64_t sh = 0, st = 0, lh = 0, lt = 0;   /* queue heads and tails */
    for (int64_t v = 0; v < n; ++v) {
        s[v] = s[v] * (double)n / total;
        if (s[v] < 1.0) small[st++] = v; else large[lt++] = v;
    }
    for (int64_t v = 0; v < n; ++v) { thr[v] = 0xFFFFFFFFu; alias[v] = (int32_t)v; }
    while (sh < st && lh < lt) {
        int64_t l = small[sh++];
        int64_t g = large[lh];
        double keep = floor(s[l] * 4294967296.0);
        thr[l] = keep >= 4294967295.0 ? 0xFFFFFFFFu : (uint32_t)keep;
        alias[l] = (int32_t)g;
        s[g] = (s[g] + s[l]) - 1.0;
        if (s[g] < 1.0) { ++lh; small[st++] = g; }
    }
    /* whatever is left keeps its whole cell (thr = max, alias = self) */
    free(s); free(small); free(large);
    return 0;
}

/* ------------------------------------------------------------------------
 * Table initialisation: input vectors uniform in [-0.5/d, 0.5/d), output
 * vectors zero (the word2vec convention).  Entry (row, j) uses word j%4 of
 * the Philox block (id = row, step = j/4, TAG_INIT): u = (word>>8) * 2^-24,
 * value = (u - 0.5)/d.  Fills rows rows[0..n_rows) of a compact table.
 * ---------------------------------------------------------------------- */
void gso_init_rows(const int64_t *rows, int64_t n_rows, int32_t d, uint64_t seed, double *U)
{
    for (int64_t a = 0; a < n_rows; ++a) {
        for (int32_t j = 0; j < d; ++j) {
            uint32_t r[4];
            draw4(seed, (uint64_t)rows[a], (uint32_t)(j / 4), TAG_INIT, 0, r);
            double u = (double)(r[j % 4] >> 8) * (1.0 / 16777216.0);
            U[a * (int64_t)d + j] = (u - 0.5) / (double)d;
        }
    }
}

/* ------------------------------------------------------------------------
 * SGNS objective for one pair (c, o) with negatives n_1..n_K:
 *   loss = softplus(-<U_c,V_o>) + sum_k softplus(<U_c,V_nk>)
 * (Mikolov et al. 2013, the skip-gram objective with negative sampling named in Section
 * 2.2).  A negative equal to the pair's context is masked: no loss term and
 * no gradient.
 * ---------------------------------------------------------------------- */
static double softplus(double x)
{
    return (x > 0.0 ? x : 0.0) + log1p(exp(-fabs(x)));
}
static double sigmoid(double x)
{
    return 1.0 / (1.0 + exp(-x));
}
static double dot(const double *a, const double *b, int32_t d)
{
    double s = 0.0;
    for (int32_t j = 0; j < d; ++j) s += a[j] * b[j];
    return s;
}

/* Loss of a list of pairs at fixed tables (used for finite differences). */
double gso_sgns_loss_from_lists(const double *U, const double *V, int32_t d,
                                int64_t n_slots, int32_t K,
                                const int32_t *centers, const int32_t *contexts,
                                const int32_t *negs)
{
    double loss = 0.0;
    for (int64_t e = 0; e < n_slots; ++e) {
        if (centers[e] < 0) continue;
        const double *u = U + (int64_t)centers[e] * d;
        loss += softplus(-dot(u, V + (int64_t)contexts[e] * d, d));
        for (int32_t k = 0; k < K; ++k) {
            int32_t nk = negs[e * K + k];
            if (nk < 0 || nk == contexts[e]) continue;
            loss += softplus(dot(u, V + (int64_t)nk * d, d));
        }
    }
    return loss;
}

/* ------------------------------------------------------------------------
 * Deterministic synchronous mini-batch step (Section 3.2: gradients of the
 * mini-batch are computed from the embeddings fetched at the start of the
 * iteration and written back as increments, with a barrier after the write).
 * All gradients use the tables as they are on entry; the increments of every
 * pair are summed (not averaged) and applied once:
 *   g_o = sigmoid(f_o) - 1, g_k = sigmoid(f_k)
 *   GU[c] += g_o V_o + sum_k g_k V_nk ;  GV[o] += g_o U_c ;  GV[nk] += g_k U_c
 *   U -= lr GU ; V -= lr GV
 * order == NULL visits slots 0..n_slots-1; otherwise in the given order (the
 * result must not depend on it beyond rounding).
 * Row indices in the lists address rows of U and V directly (the caller may
 * have remapped node ids to a compact table; masking compares the indices,
 * which a one-to-one remap preserves).
 * ---------------------------------------------------------------------- */
int gso_sgns_det_from_lists(double *U, double *V, int64_t n_rows, int32_t d,
                            int64_t n_slots, int32_t K,
                            const int32_t *centers, const int32_t *contexts,
                            const int32_t *negs, const int64_t *order,
                            double lr, double *loss_sum, int64_t *pair_count)
{
    double *GU = (double *)calloc((size_t)(n_rows * d), sizeof(double));
    double *GV = (double *)calloc((size_t)(n_rows * d), sizeof(double));
    if (!GU || !GV) { free(GU); free(GV); return -1; }
    double loss = 0.0;
    int64_t pairs = 0;
    for (int64_t a = 0; a < n_slots; ++a) {
        int64_t e = order ? order[a] : a;
        if (centers[e] < 0) continue;
        int64_t c = centers[e], o = contexts[e];
        const double *u = U + c * d;
        ++pairs;
        {
            const double *v = V + o * d;
            double f = dot(u, v, d);
            double g = sigmoid(f) - 1.0;
            loss += softplus(-f);
            for (int32_t j = 0; j < d; ++j) {
                GU[c * d + j] += g * v[j];
                GV[o * d + j] += g * u[j];
            }
        }
        for (int32_t k = 0; k < K; ++k) {
            int64_t nk = negs[e * K + k];
            if (nk < 0 || nk == o) continue;
            const double *v = V + nk * d;
            double f = dot(u, v, d);
            double g = sigmoid(f);
            loss += softplus(f);
            for (int32_t j = 0; j < d; ++j) {
                GU[c * d + j] += g * v[j];
                GV[nk * d + j] += g * u[j];
            }
        }
    }
    for (int64_t x = 0; x < n_rows * d; ++x) {
        U[x] -= lr * GU[x];
        V[x] -= lr * GV[x];
    }
    free(GU); free(GV);
    if (loss_sum) *loss_sum = loss;
    if (pair_count) *pair_count = pairs;
    return 0;
}

/* ------------------------------------------------------------------------
 * Summed gradients of a mini-batch at fixed tables: the GU, GV of the
 * synchronous step above, returned instead of applied (both arrays are
 * n_rows x d and are overwritten).  Used by the momentum update below.
 * ---------------------------------------------------------------------- */
int gso_sgns_grad_from_lists(const double *U, const double *V, int64_t n_rows, int32_t d,
                             int64_t n_slots, int32_t K,
                             const int32_t *centers, const int32_t *contexts,
                             const int32_t *negs, double *GU, double *GV,
                             double *loss_sum, int64_t *pair_count)
{
    memset(GU, 0, sizeof(double) * (size_t)(n_rows * d));
    memset(GV, 0, sizeof(double) * (size_t)(n_rows * d));
    double loss = 0.0;
    int64_t pairs = 0;
    for (int64_t e = 0; e < n_slots; ++e) {
        if (centers[e] < 0) continue;
        int64_t c = centers[e], o = contexts[e];
        const double *u = U + c * d;
        ++pairs;
        for (int32_t k = -1; k < K; ++k) {
            int64_t t = (k < 0) ? o : negs[e * K + k];
            if (k >= 0 && (t < 0 || t == o)) continue;
            const double *v = V + t * d;
            double f = dot(u, v, d);
            double g = (k < 0) ? sigmoid(f) - 1.0 : sigmoid(f);
            loss += (k < 0) ? softplus(-f) : softplus(f);
            for (int32_t j = 0; j < d; ++j) {
                GU[c * d + j] += g * v[j];
                GV[t * d + j] += g * u[j];
            }
        }
    }
    if (loss_sum) *loss_sum = loss;
    if (pair_count) *pair_count = pairs;
    return 0;
}

/* ------------------------------------------------------------------------
 * SGD with momentum as the paper's storage applies it (Section 3.2, the
 * description of the momentum update): per iteration, over the WHOLE table,
 *   momentum <- mu * momentum            (mult)
 *   momentum[rows of the batch] += grad  (put)
 *   model    <- model - lr * momentum    (mult_add)
 * x, m, g are arrays of n values (a table flattened); g is zero outside the
 * batch's rows.
 * ---------------------------------------------------------------------- */
void gso_momentum_update(double *x, double *m, const double *g, int64_t n, double lr, double mu)
{
    for (int64_t i = 0; i < n; ++i) m[i] = mu * m[i];
    for (int64_t i = 0; i < n; ++i) m[i] += g[i];
    for (int64_t i = 0; i < n; ++i) x[i] -= lr * m[i];
}

/* ------------------------------------------------------------------------
 * Sequential per-pair SGD (each pair sees all earlier updates): the
 * race-free limit of the lock-free mode of Section 3.2 "Synchronization".
 * For each center position the center row is held fixed while its pairs
 * update the output rows, and the accumulated center gradient is applied
 * after the position's last pair (the word2vec order).  Slots must be laid
 * out position-major as gso_expand_lists writes them, S slots per position.
 * parity unpinned: the GPU's lock-free mode is racy by design.
 * ---------------------------------------------------------------------- */
int gso_sgns_seq_from_lists(double *U, double *V, int32_t d,
                            int64_t n_slots, int32_t S, int32_t K,
                            const int32_t *centers, const int32_t *contexts,
                            const int32_t *negs, double lr,
                            double *loss_sum, int64_t *pair_count)
{
    double *acc = (double *)malloc(sizeof(double) * (size_t)d);
    if (!acc) return -1;
    double loss = 0.0;
    int64_t pairs = 0;
    for (int64_t base = 0; base < n_slots; base += S) {
        int64_t c = -1;
        for (int32_t j = 0; j < d; ++j) acc[j] = 0.0;
        for (int32_t sg = 0; sg < S && base + sg < n_slots; ++sg) {
            int64_t e = base + sg;
            if (centers[e] < 0) continue;
            c = centers[e];
            const double *u = U + c * d;
            int64_t o = contexts[e];
            ++pairs;
            for (int32_t k = -1; k < K; ++k) {
                int64_t t = (k < 0) ? o : negs[e * K + k];
                if (k >= 0 && (t < 0 || t == o)) continue;
                double *v = V + t * d;
                double f = dot(u, v, d);
                double g = (k < 0) ? sigmoid(f) - 1.0 : sigmoid(f);
                loss += (k < 0) ? softplus(-f) : softplus(f);
                for (int32_t j = 0; j < d; ++j) {
                    acc[j] += g * v[j];
                    v[j] -= lr * g * u[j];
                }
            }
        }
        if (c >= 0)
            for (int32_t j = 0; j < d; ++j) U[c * d + j] -= lr * acc[j];
    }
    free(acc);
    if (loss_sum) *loss_sum = loss;
    if (pair_count) *pair_count = pairs;
    return 0;
}

/* ------------------------------------------------------------------------
 * Half-precision table storage (the paper's production tables are fp16,
 * Section 4.2): values are stored as IEEE binary16, read back exactly, all
 * arithmetic is done in full precision, and every written value is rounded
 * to the nearest binary16 (ties to even).
 * ---------------------------------------------------------------------- */
static double rn16(double x)
{
    return (double)(_Float16)x;
}

void gso_round_f16(double *x, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) x[i] = rn16(x[i]);
}

/* bfloat16: sign, 8 exponent bits (those of binary32), 7 fraction bits, i.e. 8 significant
 * bits.  One rounding of the fp64 value to the nearest such number, ties to even: the value is
 * scaled so that its 8 significant bits are the integer part, rounded with the current
 * (to-nearest-even) mode and scaled back.  Below 2^-126 the spacing stays 2^-133 (subnormals);
 * values beyond the largest finite bfloat16 round to infinity. */
static double rnb16(double x)
{
    if (x == 0.0 || isnan(x) || isinf(x)) return x;
    int e;
    frexp(x, &e);                        /* |x| = m * 2^e, 0.5 <= m < 1 */
    int q = e - 8;                       /* spacing 2^q keeps 8 significant bits */
    if (q < -133) q = -133;
    double r = ldexp(nearbyint(ldexp(x, -q)), q);
    if (fabs(r) > 3.3895313892515355e38) r = (r > 0.0) ? INFINITY : -INFINITY;   /* (2 - 2^-7) * 2^127 */
    return r;
}

void gso_round_bf16(double *x, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) x[i] = rnb16(x[i]);
}

/* ------------------------------------------------------------------------
 * Stochastic rounding to a 16-bit format (Section 4.2 of the paper keeps its production tables in
 * 16 bits; with round-to-nearest an increment below half a unit in the last place is lost every
 * time, with stochastic rounding it survives in expectation).
 *
 * The decision is taken on the fp32 value xf = float(x).  Let lo and hi be the neighbours of |xf|
 * in the format (lo towards zero; fmt 0: binary16, 11 significant bits, spacing never below
 * 2^-24; fmt 1: bfloat16, 8 significant bits, spacing never below 2^-133), frac = (|xf| - lo) /
 * (hi - lo) in [0, 1) and thr = floor(frac * 2^16).  The result is hi when the 16-bit dither u16
 * is below thr, else lo, with the sign of xf; a value that is representable never moves; a
 * magnitude beyond the largest finite value of the format, or a step up from it, gives that
 * largest value (no infinities are produced).
 * ---------------------------------------------------------------------- */
static double sr16(double x, int fmt, uint32_t u16)
{
    const float xf = (float)x;
    if (xf == 0.0f || isnan(xf)) return (double)xf;
    const int p = fmt ? 8 : 11;
    const int qmin = fmt ? -133 : -24;
    const double maxv = fmt ? 3.3895313892515355e38 : 65504.0;
    const double ax = fabs((double)xf);
    double r;
    if (ax >= maxv) {
        r = maxv;
    } else {
        int e;
        frexp(ax, &e);                       /* ax = m * 2^e, 0.5 <= m < 1 */
        int q = e - p;                       /* spacing 2^q keeps p significant bits */
        if (q < qmin) q = qmin;
        const double scaled = ldexp(ax, -q); /* exact */
        const double lo = floor(scaled);
        const uint32_t thr = (uint32_t)floor((scaled - lo) * 65536.0);
        r = ldexp(lo + (u16 < thr ? 1.0 : 0.0), q);
        if (r > maxv) r = maxv;
    }
    return xf < 0.0f ? -r : r;
}

void gso_round_sr(double *x, int64_t n, int fmt, const uint32_t *u16)
{
    for (int64_t i = 0; i < n; ++i) x[i] = sr16(x[i], fmt, u16[i] & 0xFFFFu);
}

/* The dither of column j of one row-write event.  An event has one Philox block r[0..3]; the
 * 16-bit dithers of its columns come from a cheap mix of those words (the finalizer of
 * MurmurHash3, a bijection of 32-bit words, so distinct inputs give distinct outputs): columns
 * 2k and 2k+1 take the upper and lower half of
 *   mix(r[k & 3] ^ 0x9E3779B9 * (k / 4 + 1) ^ 0x85EBCA77 * salt),
 * `salt` telling apart the rows that share an event (lock-free mode). */
static uint32_t mix32(uint32_t h)
{
    h ^= h >> 16; h *= 0x85EBCA6Bu; h ^= h >> 13; h *= 0xC2B2AE35u; h ^= h >> 16;
    return h;
}

static uint32_t dither16(const uint32_t r[4], uint32_t salt, int32_t j)
{
    const uint32_t k = (uint32_t)j >> 1;
    const uint32_t h = mix32(r[k & 3u] ^ (0x9E3779B9u * ((k >> 2) + 1u)) ^ (0x85EBCA77u * salt));
    return (j & 1) ? (h & 0xFFFFu) : (h >> 16);
}

void gso_dither16(const uint32_t r[4], uint32_t salt, int32_t d, uint32_t *out)
{
    for (int32_t j = 0; j < d; ++j) out[j] = dither16(r, salt, j);
}

/* Event of the synchronous mode: row `row` of table `table` (0 input, 1 output) written by the
 * step whose first walk id is walk_id_base: block (id = row | table << 32, step = low word of
 * walk_id_base, TAG_ROUND_SYNC, sub = bits 32..55 of walk_id_base), salt 0. */
static void sync_round_event(uint64_t seed, int64_t row, uint32_t table, int64_t walk_id_base, uint32_t r[4])
{
    draw4(seed, (uint64_t)row | ((uint64_t)table << 32), (uint32_t)((uint64_t)walk_id_base & 0xFFFFFFFFu),
          TAG_ROUND_SYNC, (uint32_t)(((uint64_t)walk_id_base >> 32) & 0xFFFFFFu), r);
}

/* Rounds every value of X[n_rows][d] stochastically as the synchronous step writes it (a value
 * that is representable already - every value of a row the step did not touch - stays). */
void gso_round_sr_rows(double *X, int64_t n_rows, int32_t d, int fmt, uint64_t seed, uint32_t table,
                       int64_t walk_id_base)
{
    for (int64_t row = 0; row < n_rows; ++row) {
        uint32_t r[4];
        sync_round_event(seed, row, table, walk_id_base, r);
        for (int32_t j = 0; j < d; ++j)
            X[row * d + j] = sr16(X[row * d + j], fmt, dither16(r, 0u, j));
    }
}

/* Sequential per-pair SGD as gso_sgns_seq_from_lists, on tables whose values are kept in a
 * 16-bit format (fmt 0: binary16, 1: bfloat16): each updated output row and each updated center
 * row is rounded when written. */
typedef struct {          /* stochastic write-back of the lock-free schedule (NULL: to nearest) */
    uint64_t seed;
    int64_t walk_id_base;
    int32_t L;            /* walk length: slot e belongs to position e / S, walk (e / S) / L */
} sr_keys;

static int sgns_seq_rounded(double *U, double *V, int32_t d, int64_t n_slots, int32_t S, int32_t K,
                            const int32_t *centers, const int32_t *contexts, const int32_t *negs,
                            double lr, int fmt, const sr_keys *sr, int red, double *loss_sum, int64_t *pair_count);

int gso_sgns_seq_f16_from_lists(double *U, double *V, int32_t d,
                                int64_t n_slots, int32_t S, int32_t K,
                                const int32_t *centers, const int32_t *contexts,
                                const int32_t *negs, double lr,
                                double *loss_sum, int64_t *pair_count)
{
    return sgns_seq_rounded(U, V, d, n_slots, S, K, centers, contexts, negs, lr, 0, NULL, 0, loss_sum, pair_count);
}

int gso_sgns_seq_bf16_from_lists(double *U, double *V, int32_t d,
                                 int64_t n_slots, int32_t S, int32_t K,
                                 const int32_t *centers, const int32_t *contexts,
                                 const int32_t *negs, double lr,
                                 double *loss_sum, int64_t *pair_count)
{
    return sgns_seq_rounded(U, V, d, n_slots, S, K, centers, contexts, negs, lr, 1, NULL, 0, loss_sum, pair_count);
}

/* Same with stochastic write-back.  Event of the lock-free mode: the rows written while position
 * i of walk `id` is worked on share the block (id, step = i, TAG_ROUND_LOCKFREE, sub 0); a target
 * row takes salt = 1 + its index in the position's target list (slot * (1 + K) for the context of
 * a slot, + 1 + k for its negative k), the center row salt 0x10000. */
int gso_sgns_seq_sr_from_lists(double *U, double *V, int32_t d, int64_t n_slots, int32_t S, int32_t K,
                               const int32_t *centers, const int32_t *contexts, const int32_t *negs,
                               double lr, int fmt, uint64_t seed, int64_t walk_id_base, int32_t L,
                               double *loss_sum, int64_t *pair_count)
{
    sr_keys sr = { seed, walk_id_base, L };
    return sgns_seq_rounded(U, V, d, n_slots, S, K, centers, contexts, negs, lr, fmt, &sr, 0, loss_sum, pair_count);
}

/* Same order of pairs, but the tables are changed the way Section 3.2 describes the exchange
 * between trainer and storage: the trainer sends an INCREMENT and the storage adds it.  With a
 * 16-bit table both the increment and the sum exist in the table's format only: the increment is
 * rounded to the format (nearest even), the addition of the two 16-bit values is exact and its
 * result is rounded to the format once more.  fmt 0: binary16, 1: bfloat16. */
int gso_sgns_seq_add16_from_lists(double *U, double *V, int32_t d, int64_t n_slots, int32_t S, int32_t K,
                                  const int32_t *centers, const int32_t *contexts, const int32_t *negs,
                                  double lr, int fmt, double *loss_sum, int64_t *pair_count)
{
    return sgns_seq_rounded(U, V, d, n_slots, S, K, centers, contexts, negs, lr, fmt, NULL, 1, loss_sum, pair_count);
}

static int sgns_seq_rounded(double *U, double *V, int32_t d, int64_t n_slots, int32_t S, int32_t K,
                            const int32_t *centers, const int32_t *contexts, const int32_t *negs,
                            double lr, int fmt, const sr_keys *sr, int red, double *loss_sum, int64_t *pair_count)
{
    double *acc = (double *)malloc(sizeof(double) * (size_t)d);
    if (!acc) return -1;
    double loss = 0.0;
    int64_t pairs = 0;
    for (int64_t base = 0; base < n_slots; base += S) {
        int64_t c = -1;
        uint32_t ev[4] = { 0, 0, 0, 0 };
        if (sr) {
            const int64_t pos = base / S;
            draw4(sr->seed, (uint64_t)(sr->walk_id_base + pos / sr->L), (uint32_t)(pos % sr->L),
                  TAG_ROUND_LOCKFREE, 0, ev);
        }
        for (int32_t j = 0; j < d; ++j) acc[j] = 0.0;
        for (int32_t sg = 0; sg < S && base + sg < n_slots; ++sg) {
            int64_t e = base + sg;
            if (centers[e] < 0) continue;
            c = centers[e];
            const double *u = U + c * d;
            int64_t o = contexts[e];
            ++pairs;
            for (int32_t k = -1; k < K; ++k) {
                int64_t t = (k < 0) ? o : negs[e * K + k];
                if (k >= 0 && (t < 0 || t == o)) continue;
                double *v = V + t * d;
                double f = dot(u, v, d);
                double g = (k < 0) ? sigmoid(f) - 1.0 : sigmoid(f);
                loss += (k < 0) ? softplus(-f) : softplus(f);
                const uint32_t salt = 1u + (uint32_t)(sg * (1 + K) + (k + 1));
                for (int32_t j = 0; j < d; ++j) {
                    acc[j] += g * v[j];
                    if (red) {                       /* increment in the format, then the sum in the format */
                        const double inc = fmt ? rnb16(-lr * g * u[j]) : rn16(-lr * g * u[j]);
                        v[j] = fmt ? rnb16(v[j] + inc) : rn16(v[j] + inc);
                        continue;
                    }
                    const double nv = v[j] - lr * g * u[j];
                    v[j] = sr ? sr16(nv, fmt, dither16(ev, salt, j)) : (fmt ? rnb16(nv) : rn16(nv));
                }
            }
        }
        if (c >= 0)
            for (int32_t j = 0; j < d; ++j) {
                if (red) {
                    const double inc = fmt ? rnb16(-lr * acc[j]) : rn16(-lr * acc[j]);
                    U[c * d + j] = fmt ? rnb16(U[c * d + j] + inc) : rn16(U[c * d + j] + inc);
                    continue;
                }
                double nv = U[c * d + j] - lr * acc[j];
                U[c * d + j] = sr ? sr16(nv, fmt, dither16(ev, 0x10000u, j)) : (fmt ? rnb16(nv) : rn16(nv));
            }
    }
    free(acc);
    if (loss_sum) *loss_sum = loss;
    if (pair_count) *pair_count = pairs;
    return 0;
}

/* ------------------------------------------------------------------------
 * Sub-sampling of frequent nodes (Mikolov et al. 2013, "Distributed
 * representations of words and phrases", Section 2.3): an occurrence of a
 * node whose relative frequency f exceeds t is discarded with probability
 * 1 - sqrt(t / f).  keep(v) = min(1, sqrt(t / f(v))), f(v) = weight(v) / sum.
 * thr[v] = floor(keep * 2^32), or 0xFFFFFFFF when keep >= 1 ("always").
 * Returns 0, or -1 when no weight is positive.
 * ---------------------------------------------------------------------- */
int gso_keep_thresholds(const double *weights, int64_t n, double t, uint32_t *thr)
{
    double total = 0.0;
    for (int64_t v = 0; v < n; ++v) total += weights[v] > 0.0 ? weights[v] : 0.0;
    if (!(total > 0.0)) return -1;
    for (int64_t v = 0; v < n; ++v) {
        thr[v] = 0xFFFFFFFFu;
        if (!(weights[v] > 0.0)) continue;
        double f = weights[v] / total;
        double keep = sqrt(t / f);
        if (keep < 1.0) {
            double x = floor(keep * 4294967296.0);
            thr[v] = x >= 4294967295.0 ? 0xFFFFFFFFu : (uint32_t)x;
        }
    }
    return 0;
}

/* Entry t of walk `id` (node v = W[t] >= 0) is kept iff thr[v] == 0xFFFFFFFF or
 * word 0 of the block (id, step = t, TAG_SUBSAMPLE, sub 0) is below thr[v].  The
 * kept entries are moved to the front in their order (the window then spans
 * the discarded occurrences, as in word2vec) and the rest of the row is -1.
 * Returns the number of kept entries. */
int64_t gso_subsample_walks(const int32_t *walks, int64_t n_walks, int64_t walk_id_base,
                            int32_t L, const uint32_t *thr, uint64_t seed, int32_t *out)
{
    int64_t kept = 0;
    for (int64_t a = 0; a < n_walks; ++a) {
        const int32_t *W = walks + a * (int64_t)L;
        int32_t *O = out + a * (int64_t)L;
        uint64_t id = (uint64_t)(walk_id_base + a);
        int32_t n = 0;
        for (int32_t t = 0; t < L; ++t) {
            int32_t v = W[t];
            if (v < 0) continue;
            int keep = 1;
            if (thr[v] != 0xFFFFFFFFu) {
                uint32_t r[4];
                draw4(seed, id, (uint32_t)t, TAG_SUBSAMPLE, 0, r);
                keep = r[0] < thr[v];
            }
            if (keep) O[n++] = v;
        }
        kept += n;
        for (; n < L; ++n) O[n] = -1;
    }
    return kept;
}

/* ------------------------------------------------------------------------
 * Start-node shuffle: a keyed bijection of [0, n) per (seed, epoch), so that
 * the walks of an epoch start from the nodes in a different order each time.
 * Balanced Feistel network of four rounds on 2k bits (4^k >= n, k minimal,
 * k >= 1) whose round function is word 0 of the Philox block
 * (id = right half | epoch << 32, step = round, TAG_SHUFFLE, sub 0) masked to
 * k bits; values that land outside [0, n) are fed through the network again
 * (cycle walking; a Feistel network is a bijection of its domain, so this
 * restricts it to a bijection of [0, n)).
 * ---------------------------------------------------------------------- */
static uint64_t feistel_once(uint64_t x, int k, uint64_t seed, uint32_t epoch)
{
    uint64_t mask = ((uint64_t)1 << k) - 1;
    uint64_t left = x >> k, right = x & mask;
    for (uint32_t round = 0; round < 4; ++round) {
        uint32_t r[4];
        draw4(seed, right | ((uint64_t)epoch << 32), round, TAG_SHUFFLE, 0, r);
        uint64_t f = (uint64_t)r[0] & mask;
        uint64_t nl = right, nr = left ^ f;
        left = nl; right = nr;
    }
    return (left << k) | right;
}

int64_t gso_shuffle_node(int64_t v, int64_t n, uint64_t seed, uint32_t epoch)
{
    int k = 1;
    while (((uint64_t)1 << (2 * k)) < (uint64_t)n) ++k;
    uint64_t y = (uint64_t)v;
    do { y = feistel_once(y, k, seed, epoch); } while (y >= (uint64_t)n);
    return (int64_t)y;
}

/* starts[i] = shuffle(node (walk_id_first + i) mod n) */
void gso_shuffled_starts(int64_t n, uint64_t seed, uint32_t epoch, int64_t walk_id_first,
                         int64_t count, int32_t *starts)
{
    for (int64_t i = 0; i < count; ++i)
        starts[i] = (int32_t)gso_shuffle_node((walk_id_first + i) % n, n, seed, epoch);
}

/* ------------------------------------------------------------------------
 * Adam (Kingma & Ba 2015, Algorithm 1), which the paper names beside SGD with
 * momentum as an optimizer kept inside the storage (Section 3.2).  Applied to
 * the rows of the mini-batch only (rows outside it keep their values and
 * their moments, as a sparse-gradient Adam does); `step` counts iterations
 * from 1 and is the same for every row:
 *   m <- b1 m + (1-b1) g ;  v <- b2 v + (1-b2) g^2
 *   x <- x - lr * (m / (1-b1^step)) / (sqrt(v / (1-b2^step)) + eps)
 * rows[0..n_rows) are the distinct touched rows of a table of width d; g is
 * the dense gradient table (only the touched rows are read).
 * ---------------------------------------------------------------------- */
void gso_adam_rows(double *x, double *m, double *v, const double *g, int32_t d,
                   const int64_t *rows, int64_t n_rows, double lr, double b1, double b2,
                   double eps, int64_t step)
{
    double c1 = 1.0 - pow(b1, (double)step);
    double c2 = 1.0 - pow(b2, (double)step);
    for (int64_t a = 0; a < n_rows; ++a) {
        for (int32_t j = 0; j < d; ++j) {
            int64_t e = rows[a] * d + j;
            m[e] = b1 * m[e] + (1.0 - b1) * g[e];
            v[e] = b2 * v[e] + (1.0 - b2) * g[e] * g[e];
            double mhat = m[e] / c1;
            double vhat = v[e] / c2;
            x[e] -= lr * mhat / (sqrt(vhat) + eps);
        }
    }
}
