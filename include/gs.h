/*
 * gs.h - C ABI of the B200 random-walk + SGNS library.
 *
 * The library implements, on one GPU, the data-parallel hot path of
 * unsupervised node-embedding training as GraphScale runs it (paper Section
 * 2.2 "Node embedding training" and Section 3.2 "Node Embedding Training"):
 * random walks over a CSR graph (DeepWalk: uniform; node2vec: second-order
 * biased) and the skip-gram-with-negative-sampling (SGNS) update of an input
 * and an output embedding table, either as a synchronous mini-batch step
 * whose result does not depend on thread scheduling, or lock-free (Section
 * 3.2 "Synchronization": trainers write increments to the same rows without
 * locking).
 *
 * Conventions
 *  - Pointers named d_* are DEVICE pointers, h_* are HOST pointers.  Every
 *    buffer is allocated and freed by the caller; the library borrows it for
 *    the duration of the call (a graph handle borrows the CSR arrays until
 *    gs_graph_free).  The library allocates only its own scratch memory
 *    (cached per device, released by gs_release_workspace).  That scratch is
 *    per DEVICE, not per stream: SGNS calls on one device must be ordered
 *    after one another (same stream, or events between streams); two that
 *    overlap on the GPU would share grouping buffers and the walk ticket.
 *  - `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *    Calls enqueue work on it and return without waiting unless stated.
 *  - Every function returns a gs_status; nothing throws, aborts or traps.
 *    gs_last_error() gives a thread-local description of the last failure.
 *  - Random numbers are Philox4x32-10 blocks with key = seed and counter =
 *    (id low, id high, step, tag << 24 | sub): a result depends on
 *    (seed, walk id, position), never on launch shape or batching.
 *      tag 1 uniform walk : id = walk id, step = transition index t
 *      tag 2 node2vec     : id = walk id, step = t, sub = rejection round
 *      tag 3 negatives    : id = walk id, step = i * 2w + slot, sub = m
 *      tag 4 table init   : id = row, step = column / 4
 *      tag 5 window draw  : id = walk id, step = position i
 *      tag 6 sub-sampling : id = walk id, step = position t
 *      tag 7 start shuffle: id = right half | epoch << 32, step = Feistel round
 *      tag 8, 9 dithers of the stochastic write-back (GS_ROUND_STOCHASTIC)
 *  - A 32-bit word r is mapped to [0, n) as (r * n) >> 32.
 */
#ifndef GS_H
#define GS_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define GS_API __attribute__((visibility("default")))
#else
#define GS_API
#endif

typedef int32_t gs_status;
#define GS_OK                 0
#define GS_ERR_INVALID_ARG   (-1)  /* null pointer, negative size, bad enum          */
#define GS_ERR_BAD_CSR       (-2)  /* offsets not monotone / column out of range     */
#define GS_ERR_UNSORTED_ADJ  (-3)  /* a row is not strictly increasing               */
#define GS_ERR_CUDA          (-4)  /* a CUDA call failed; text in gs_last_error()    */
#define GS_ERR_OOM           (-5)  /* scratch allocation failed                      */
#define GS_ERR_UNSUPPORTED   (-6)  /* shape outside the supported range              */

/* Thread-local, library-owned, NUL-terminated; valid until the next call. */
GS_API const char *gs_last_error(void);

/* ---------------------------------------------------------------- graph */
typedef struct gs_graph gs_graph;

#define GS_VALIDATE        1u   /* check offsets and column range on the device    */
#define GS_REQUIRE_SORTED  2u   /* additionally require strictly increasing rows   */
#define GS_BUILD_WALK_INDEX 4u  /* build the per-entry walk index (implies GS_VALIDATE) */
#define GS_BUILD_EDGE_SET  8u   /* build the hashed edge set for node2vec (implies GS_VALIDATE) */

/*
 * Wraps a CSR graph that already lives in device memory (the whole topology
 * stays resident next to the sampler, as each trainer keeps it in Section 3.1).
 *   d_offsets : n_nodes+1 entries, int64 if offsets_are_64bit else int32
 *   d_cols    : n_edges int32 neighbour ids
 * With GS_VALIDATE the call checks offsets[0] = 0, offsets[n] = n_edges,
 * monotone offsets and 0 <= col < n_nodes, records the maximum degree, and
 * WAITS for the result (one small device-to-host read).  node2vec needs
 * GS_REQUIRE_SORTED rows.  On error *out is NULL; GS_ERR_BAD_CSR /
 * GS_ERR_UNSORTED_ADJ name the first offending row in gs_last_error().
 * With GS_BUILD_WALK_INDEX the handle also owns 16 bytes of device memory per
 * CSR entry (allocated here, freed by gs_graph_free; GS_ERR_OOM if it does not
 * fit): entry e records cols[e] with that node's degree and offset, so that a
 * uniform-walk transition needs one random read instead of two.  Walks are
 * identical with or without the index.
 * With GS_BUILD_EDGE_SET the handle also owns a hash table of all CSR entries
 * (8 bytes per slot, 2 to 4 slots per entry; GS_ERR_OOM if it does not fit):
 * node2vec then decides "is x a neighbour of prev" with one or two reads instead
 * of a binary search over the row of prev.  Walks are identical with or without it.
 */
GS_API gs_status gs_graph_load_csr(int64_t n_nodes, int64_t n_edges,
                            const void *d_offsets, int32_t offsets_are_64bit,
                            const int32_t *d_cols, uint32_t flags,
                            void *stream, gs_graph **out);

/* Releases the resident topology of gs_graph_load_csr (Section 3.1 keeps it for the lifetime
 * of a trainer): frees the handle and the walk index and edge set it owns, waiting for the
 * device if there are any; the CSR arrays stay the caller's.  NULL is allowed. */
GS_API void gs_graph_free(gs_graph *g);

/* Sizes of the resident graph G = (V, E) of Section 2.2: |V|, the number of CSR entries, the
 * largest out-degree (-1 if the graph was loaded without GS_VALIDATE) and whether the rows
 * were verified strictly increasing.  Output pointers may be NULL. */
GS_API gs_status gs_graph_info(const gs_graph *g, int64_t *n_nodes, int64_t *n_edges,
                        int64_t *max_degree, int32_t *rows_sorted);

/* ---------------------------------------------------------------- alias table */
/*
 * HOST function.  Builds the alias table of p(v) ~ h_weights[v]^power (the
 * word2vec unigram^0.75 negative distribution when weights are node
 * frequencies or degrees; the paper only says that negatives are sampled,
 * Section 3.2).  Zero weights get probability zero.  Entry v of h_table_out
 * packs thr (low 32 bits) and alias (high 32 bits): a draw with words (a, b)
 * picks cell j = (a * n) >> 32 and returns j if b < thr[j], else alias[j].
 * The caller uploads the table.  Deterministic: small and large cells are
 * paired through two first-in-first-out queues filled in increasing v.
 * Errors: GS_ERR_INVALID_ARG (null, n <= 0, n >= 2^31, no positive weight,
 * negative or non-finite weight), GS_ERR_OOM.
 */
GS_API gs_status gs_build_alias(const double *h_weights, int64_t n, double power,
                         uint64_t *h_table_out);

/* ---------------------------------------------------------------- tables */
/*
 * Fills d_w_in[n_nodes][dim] with (u - 0.5)/dim, u = (word >> 8) * 2^-24 drawn
 * with tag 4, and d_w_out[n_nodes][dim] with zeros (either may be NULL to
 * skip it).  Row-major fp32, rows contiguous.
 */
GS_API gs_status gs_init_embeddings(float *d_w_in, float *d_w_out, int64_t n_nodes,
                             int32_t dim, uint64_t seed, void *stream);

/* ---------------------------------------------------------------- walks */
/*
 * DeepWalk walks (Section 2.2: every node is the source of random walks).
 *   d_starts     : n_walks start nodes, or NULL for start = walk id mod n_nodes;
 *                  a start outside [0, n_nodes) gives a walk of -1 entries
 *   walk id      : walk_id_base + index; selects the random stream
 *   walk_len     : number of NODES per walk (Section 3.2 counts a batch as
 *                  B x walk_len nodes, sources included); >= 1
 *   d_walks_out  : [n_walks][walk_len] int32, walk-major.  A walk that reaches
 *                  a node without out-edges stops; remaining entries are -1.
 *   d_steps      : if not NULL, the number of transitions taken is ADDED to it.
 * Transition t: next = cols[off[cur] + ((word0 * deg) >> 32)], tag 1.
 */
GS_API gs_status gs_random_walks(const gs_graph *g, const int32_t *d_starts,
                          int64_t n_walks, int64_t walk_id_base, int32_t walk_len,
                          uint64_t seed, int32_t *d_walks_out,
                          uint64_t *d_steps, void *stream);

/*
 * node2vec walks (Section 2.2: a biased walk that trades breadth-first
 * against depth-first exploration; Grover & Leskovec 2016).  After
 * the move prev -> cur, neighbour x of cur has weight 1/p if x = prev, 1 if x
 * is a neighbour of prev, 1/q otherwise.  Sampled by rejection with tag 2:
 * round s proposes x = cols[off[cur] + ((word0 * deg) >> 32)] and accepts iff
 * word1 < floor(weight / max(1/p, 1, 1/q) * 2^32).  The first transition is
 * uniform (round 0, word 0).  If max_rounds rounds reject, the last proposal
 * is taken and *d_cap_hits (nullable) is incremented.  Needs a graph loaded
 * with GS_REQUIRE_SORTED (GS_ERR_UNSORTED_ADJ otherwise); p, q > 0;
 * 1 <= max_rounds <= 65536.
 */
GS_API gs_status gs_node2vec_walks(const gs_graph *g, const int32_t *d_starts,
                            int64_t n_walks, int64_t walk_id_base, int32_t walk_len,
                            uint64_t seed, double p, double q, int32_t max_rounds,
                            int32_t *d_walks_out, uint64_t *d_steps,
                            uint64_t *d_cap_hits, void *stream);

/* ---------------------------------------------------------------- SGNS */
#define GS_DETERMINISTIC  0   /* synchronous mini-batch step, bitwise reproducible */
#define GS_HOGWILD        1   /* lock-free: plain loads and stores, rows may race   */
#define GS_HOGWILD_RED    2   /* lock-free: increments sent as reductions (no lost  */
                              /* updates, gradients may still be stale)             */
#define GS_PAIRS_FORWARD_ONLY 0x100  /* OR into `mode`: keep only pairs whose context comes  */
                                     /* LATER in the walk.  Walks of two nodes with window 1 */
                                     /* then give one (source, neighbour) pair per source    */
                                     /* with n_neg negatives: the batch shape of LINE        */
                                     /* (Section 3.2: B x (2 + num_neg) nodes).              */
#define GS_WINDOW_SHRINK      0x200   /* OR into `mode`: position i of a walk uses the window   */
                                     /* w_i = 1 + ((word0 * window) >> 32), uniform on        */
                                     /* 1..window (tag 5), and keeps the pairs with           */
                                     /* |i-j| <= w_i: word2vec's shrinking window, which      */
                                     /* weights near contexts more.  Slots and the keying of  */
                                     /* the negatives stay those of the full window.  (The    */
                                     /* paper's runs use a fixed window, Section 4.)          */

#define GS_ROUND_STOCHASTIC   0x400   /* OR into `mode`, 16-bit tables only (gs_sgns_step_f16 / _bf16, and  */
                                     /* gs_sgns_epoch with such tables): written values are rounded to    */
                                     /* one of their two neighbours in the table's format, upwards in      */
                                     /* magnitude with probability (|x| - lo) / (hi - lo) taken to 16     */
                                     /* bits, instead of to the nearest.  An increment below half a unit  */
                                     /* in the last place then survives in expectation.  (Section 4.2:    */
                                     /* the production tables are 16-bit; the rounding is this library's.) */
                                     /* Dithers: tag 8 (synchronous: block keyed by row | table << 32,    */
                                     /* step = low word of walk_id_base, sub = its bits 32..55) or tag 9  */
                                     /* (lock-free: block keyed by walk id, step = position; a target row */
                                     /* takes salt 1 + its index in the position's target list, the       */
                                     /* center row 0x10000); columns 2k, 2k+1 take the halves of          */
                                     /* mix(word[k & 3] ^ 0x9E3779B9 (k/4 + 1) ^ 0x85EBCA77 salt).        */
                                     /* GS_ERR_UNSUPPORTED with fp32 tables.                              */

/*
 * One SGNS update over a batch of walks: skip-gram with negative sampling on
 * the nodes of random walks (Section 2.2), run as the paper's training
 * iteration - fetch the rows of the batch, compute the loss and its gradients,
 * write the increments back (Section 3.2 "Node Embedding Training"; the two
 * update disciplines are those of Section 3.2 "Synchronization").
 *
 * Pairs: for position i of a walk and j with 0 < |i-j| <= window inside the
 * walk, both entries >= 0: center = walk[i], context = walk[j], slot
 * sigma = j - i + window - (j > i) in [0, 2*window).
 * Negatives: n_neg draws per pair from d_alias (n_nodes packed entries, see
 * gs_build_alias), tag 3, block m gives draws 2m and 2m+1 from words (0,1)
 * and (2,3).  A negative equal to the pair's context is masked (no term).
 * Objective per pair: softplus(-<u_c, v_o>) + sum_k softplus(<u_c, v_nk>),
 * u rows of d_w_in, v rows of d_w_out; g = sigmoid(f) - label.
 *
 * GS_DETERMINISTIC: every gradient uses the tables as they are on entry;
 * increments are grouped by destination row, summed in a fixed order without
 * atomics and applied once: U -= lr * GU, V -= lr * GV (sum over pairs, not
 * mean).  Two runs give identical bits.  Scratch grows with
 * n_walks * walk_len * 2 * window * (1 + n_neg) (about 20 + dim/16 bytes per slot);
 * GS_ERR_UNSUPPORTED beyond 2^30 slots.
 * GS_HOGWILD / GS_HOGWILD_RED: one warp per walk runs positions in order;
 * per position the center row is read once, every target row is read,
 * updated from the current center row and written back at once, and the
 * center row receives its accumulated increment after the last pair.
 * Results depend on scheduling.  Target rows are handled a chunk at a time
 * (6 to 24 rows, all loaded before any is stored): with GS_HOGWILD a row that
 * occurs more than once in a chunk keeps the increment of its last occurrence
 * only, like a row that two warps update at the same moment (adding the
 * occurrences up instead was measured and lowers the loss no further);
 * GS_HOGWILD_RED adds every increment.
 *
 *   d_w_in, d_w_out : [n_nodes][dim] fp32 row-major, 16-byte aligned,
 *                     dim in {32, 64, 128, 256}
 *   d_walks         : [n_walks][walk_len] int32 (as written by the walk calls); an
 *                     entry outside [0, n_nodes) counts as absent, like -1
 *   d_loss_sum      : the batch's summed loss is ADDED (nullable)
 *   d_pair_count    : the number of pairs is ADDED (nullable)
 *   d_pairs_dump    : nullable; [n_walks][walk_len][2*window][2] int32
 *                     (center, context) or (-1,-1) where no pair exists
 *   d_negs_dump     : nullable; [n_walks][walk_len][2*window][n_neg] int32, the
 *                     drawn ids (masked ones included), -1 where no pair exists
 * Limits: 1 <= window <= 32, 0 <= n_neg <= 32, 1 <= walk_len <= 1024,
 * 2*window*(1+n_neg) <= 512.
 */
GS_API gs_status gs_sgns_step(float *d_w_in, float *d_w_out, int64_t n_nodes, int32_t dim,
                       const int32_t *d_walks, int64_t n_walks, int64_t walk_id_base,
                       int32_t walk_len, int32_t window, int32_t n_neg,
                       const uint64_t *d_alias, float lr, uint64_t seed, int32_t mode,
                       double *d_loss_sum, int64_t *d_pair_count,
                       int32_t *d_pairs_dump, int32_t *d_negs_dump, void *stream);

/*
 * gs_sgns_step with GS_DETERMINISTIC for callers that must not allocate device
 * memory: code running where cudaMalloc is forbidden or unsafe - inside a
 * region whose memory budget is already fully handed out, in a real-time loop
 * that cannot take the implicit device synchronisation of an allocation, or
 * under a host framework that owns the allocator and forbids foreign calls to
 * it.  (The paper has no counterpart; this is a convenience of this library.)
 *
 * Same arguments, arithmetic, launch order and result bits as gs_sgns_step in
 * deterministic mode (without the dump arrays), but the grouping scratch comes
 * from a fixed 32 MiB array that is part of the library image: every GPU that
 * loads the library carries those 32 MiB until the process ends.  The call
 * performs no cudaMalloc / cudaFree and calls no allocating routine.
 *
 * Limit: the batch must need at most 32 MiB of scratch,
 *   slots = n_walks * walk_len * (P + 1), P = 2*window*(1+n_neg) rounded up to a power of two
 *   bytes ~ (25 + dim/16) * slots + n_walks * walk_len * (4*dim + 16)  (+ < 1 % for the sort)
 * e.g. up to about 300 walks of length 40 with window 5, 5 negatives, dim 128.
 * Larger batches are rejected with GS_ERR_UNSUPPORTED and a message that
 * states the bytes needed; nothing is launched in that case.
 *
 * The first call on each device looks up the array's device address (one
 * cudaGetSymbolAddress with that device current).  With lazy module loading
 * that lookup, and the first launch of each kernel, is also what makes the
 * driver load this library's device code and set aside the 32 MiB, which may
 * allocate and synchronise inside the driver: make one call per device during
 * set-up, outside any stream capture, before entering the region that must
 * not allocate.  All calls on a device share the one array and
 * it keeps whatever the previous call left: every pass overwrites what it
 * later reads, so stale contents are harmless, but two calls whose kernels
 * overlap on the GPU (different streams, no ordering between them) race on
 * the array and corrupt each other - order them.
 */
GS_API gs_status gs_sgns_step_static(float *d_w_in, float *d_w_out, int64_t n_nodes, int32_t dim,
                                     const int32_t *d_walks, int64_t n_walks,
                                     int64_t walk_id_base, int32_t walk_len, int32_t window,
                                     int32_t n_neg, const uint64_t *d_alias, float lr,
                                     uint64_t seed, double *d_loss_sum, int64_t *d_pair_count,
                                     void *stream);

/*
 * Synchronous mini-batch step with SGD momentum (Section 3.2, the momentum
 * update carried out inside the storage: multiply the momentum matrix by the
 * momentum value, add the batch's gradients to its rows, subtract lr times
 * the momentum from the model).  Defined densely, for EVERY row per iteration,
 *   m <- momentum * m ;  m[rows of the batch] += grad ;  w <- w - lr * m
 * but applied sparsely: a row that a batch does not touch is brought up to
 * date only when a later batch reads it (k missed iterations:
 * w -= lr m (mu + ... + mu^k), m *= mu^k), which is the same arithmetic up to
 * rounding as long as lr and momentum are THE SAME IN EVERY CALL of a run.
 *   d_m_in, d_m_out       : momentum tables, same shape as the embedding tables,
 *                           zero before the first iteration
 *   d_last_in, d_last_out : int32[n_nodes], iteration up to which each row is
 *                           current; zero before the first iteration
 *   iteration             : 0, 1, 2, ... one per call; gradients as in
 *                           gs_sgns_step(GS_DETERMINISTIC) (same pairs, draws,
 *                           summation order, no floating-point atomics)
 * Between calls only rows with d_last == iteration are current; call
 * gs_momentum_flush on each table before reading the tables elsewhere.
 * 0 <= momentum < 1.  Scratch as for the deterministic step.
 */
GS_API gs_status gs_sgns_step_momentum(float *d_w_in, float *d_w_out, float *d_m_in, float *d_m_out,
                                       int32_t *d_last_in, int32_t *d_last_out, int64_t n_nodes,
                                       int32_t dim, const int32_t *d_walks, int64_t n_walks,
                                       int64_t walk_id_base, int32_t walk_len, int32_t window,
                                       int32_t n_neg, const uint64_t *d_alias, float lr,
                                       float momentum, int32_t iteration, uint64_t seed,
                                       double *d_loss_sum, int64_t *d_pair_count, void *stream);

/*
 * Brings every row of one table (and its momentum) up to `iteration`, i.e. to
 * the state the dense definition above has after `iteration` iterations, and
 * stamps d_last.  One pass over the table.
 */
GS_API gs_status gs_momentum_flush(float *d_w, float *d_m, int32_t *d_last, int64_t n_rows,
                                   int32_t dim, float lr, float momentum, int32_t iteration,
                                   void *stream);

/*
 * Half-precision table storage (the paper's production tables are fp16: 1e9 x
 * 128 values in 256 GB, Section 4.2).  d_w_in / d_w_out hold IEEE half values,
 * [n_nodes][dim] row-major, dim in {64, 128, 256}.  Every row is widened to
 * fp32 when read, all arithmetic is as in gs_sgns_step, and a written row is
 * rounded to nearest-even half (or stochastically, GS_ROUND_STOCHASTIC).  Row
 * traffic halves; to nearest, increments far below half a unit in the last
 * place of the stored value are lost.
 * Modes: GS_DETERMINISTIC (bitwise reproducible), GS_HOGWILD, and
 * GS_HOGWILD_RED: there every change is sent as an INCREMENT rounded to the
 * table's format and the reduction unit adds it in that format (a second
 * rounding to nearest; Section 3.2: trainers send increments, the storage adds
 * them), so no update is lost to a race; GS_ROUND_STOCHASTIC cannot be combined
 * with it (GS_ERR_UNSUPPORTED).  Other arguments as gs_sgns_step.
 * gs_init_embeddings_f16 writes the start values of gs_init_embeddings rounded
 * to half.
 */
GS_API gs_status gs_init_embeddings_f16(void *d_w_in, void *d_w_out, int64_t n_nodes,
                                        int32_t dim, uint64_t seed, void *stream);
GS_API gs_status gs_sgns_step_f16(void *d_w_in, void *d_w_out, int64_t n_nodes, int32_t dim,
                                  const int32_t *d_walks, int64_t n_walks, int64_t walk_id_base,
                                  int32_t walk_len, int32_t window, int32_t n_neg,
                                  const uint64_t *d_alias, float lr, uint64_t seed, int32_t mode,
                                  double *d_loss_sum, int64_t *d_pair_count,
                                  int32_t *d_pairs_dump, int32_t *d_negs_dump, void *stream);

/*
 * The same with bfloat16 storage (sign, the 8 exponent bits of fp32, 7 fraction bits): the other
 * 16-bit format in use for embedding tables; the range of fp32 at 8 significant bits, where IEEE
 * half has 11 bits and a narrow range.  The paper's tables are fp16 (Section 4.2); this variant is
 * offered beside it.  d_w_in / d_w_out hold bfloat16 values, dim in {64, 128, 256}; rows are
 * widened to fp32 when read, arithmetic as in gs_sgns_step, written rows rounded to nearest even.
 * With 8 significant bits an increment below 2^-9 of the stored value is lost, so plain SGD stalls
 * earlier than with half tables.  Modes as gs_sgns_step_f16.
 */
GS_API gs_status gs_init_embeddings_bf16(void *d_w_in, void *d_w_out, int64_t n_nodes,
                                         int32_t dim, uint64_t seed, void *stream);
GS_API gs_status gs_sgns_step_bf16(void *d_w_in, void *d_w_out, int64_t n_nodes, int32_t dim,
                                   const int32_t *d_walks, int64_t n_walks, int64_t walk_id_base,
                                   int32_t walk_len, int32_t window, int32_t n_neg,
                                   const uint64_t *d_alias, float lr, uint64_t seed, int32_t mode,
                                   double *d_loss_sum, int64_t *d_pair_count,
                                   int32_t *d_pairs_dump, int32_t *d_negs_dump, void *stream);

/*
 * Synchronous mini-batch step with Adam (Kingma & Ba 2015, Algorithm 1), the second optimizer
 * the paper keeps inside its storage (Section 3.2).  Gradients as in
 * gs_sgns_step(GS_DETERMINISTIC); only the rows of the batch move (the rows that occur as a
 * center, a context or an unmasked negative), as a sparse-gradient Adam does: a row outside the
 * batch keeps its value and its moments.  For every value of a touched row with summed
 * gradient g:
 *   m <- beta1 m + (1-beta1) g ;  v <- beta2 v + (1-beta2) g^2
 *   x <- x - lr * (m / (1-beta1^step)) / (sqrt(v / (1-beta2^step)) + eps)
 *   d_m_*, d_v_* : first and second moments, shape of the tables, zero before step 1
 *   step         : 1, 2, 3, ... one per call, the same for every row
 *   pair_mode    : 0, or GS_PAIRS_FORWARD_ONLY / GS_WINDOW_SHRINK OR-ed together
 * 0 <= beta1, beta2 < 1, eps > 0.  Bitwise reproducible; scratch as for the deterministic step.
 */
GS_API gs_status gs_sgns_step_adam(float *d_w_in, float *d_w_out, float *d_m_in, float *d_v_in,
                                   float *d_m_out, float *d_v_out, int64_t n_nodes, int32_t dim,
                                   const int32_t *d_walks, int64_t n_walks, int64_t walk_id_base,
                                   int32_t walk_len, int32_t window, int32_t n_neg,
                                   const uint64_t *d_alias, float lr, float beta1, float beta2,
                                   float eps, int64_t step, uint64_t seed, int32_t pair_mode,
                                   double *d_loss_sum, int64_t *d_pair_count, void *stream);

/* ---------------------------------------------------------------- corpus variants */
/*
 * Sub-sampling of frequent nodes, as word2vec thins frequent words (Mikolov et al. 2013,
 * Section 2.3; the paper's pipeline has no such step): an occurrence of node v is kept with
 * probability min(1, sqrt(t / f(v))), f(v) = h_weights[v] / sum of weights.
 * HOST function: h_thr_out[v] = floor(keep * 2^32), or 0xFFFFFFFF for "always" (keep >= 1 or
 * zero weight).  Errors: GS_ERR_INVALID_ARG (null, n <= 0, t <= 0, negative or non-finite
 * weight, no positive weight).  The caller uploads the thresholds.
 */
GS_API gs_status gs_build_keep_thresholds(const double *h_weights, int64_t n, double t,
                                          uint32_t *h_thr_out);

/*
 * Applies the thresholds to walks: entry t of walk id (node v >= 0) stays iff
 * d_keep_thr[v] == 0xFFFFFFFF or word 0 of the block (tag 6, step t) is below d_keep_thr[v].
 * Kept entries move to the front of the walk in their order, the rest of the row becomes -1,
 * so the windows of gs_sgns_step then span the dropped occurrences.  d_walks_out may be
 * d_walks (in place).  d_kept (nullable): the number of kept entries is ADDED.
 * d_keep_thr has n_nodes entries; an entry of d_walks outside [0, n_nodes) is dropped.
 */
GS_API gs_status gs_subsample_walks(const int32_t *d_walks, int64_t n_walks, int64_t walk_id_base,
                                    int32_t walk_len, const uint32_t *d_keep_thr, int64_t n_nodes,
                                    uint64_t seed, int32_t *d_walks_out, uint64_t *d_kept,
                                    void *stream);

/*
 * Start nodes in shuffled order: d_starts_out[i] = P((walk_id_first + i) mod n_nodes), where P
 * is a bijection of [0, n_nodes) chosen by (seed, epoch), so that consecutive walk ids (and
 * with them the mini-batches) start from nodes spread over the graph and every epoch uses a
 * different order.  P is a four-round balanced Feistel network on 2k bits, 4^k >= n_nodes with
 * k minimal, round function = word 0 of the Philox block (tag 7) masked to k bits; results
 * outside [0, n_nodes) are passed through the network again.  Pass the result as d_starts to
 * the walk calls.  (The paper does not say in which order the sources are visited.)
 */
GS_API gs_status gs_shuffled_starts(int64_t n_nodes, uint64_t seed, uint32_t epoch,
                                    int64_t walk_id_first, int64_t count, int32_t *d_starts_out,
                                    void *stream);

#define GS_WALK_UNIFORM   0
#define GS_WALK_NODE2VEC  1
#define GS_TABLE_F32      0
#define GS_TABLE_F16      1   /* tables of IEEE half, see gs_sgns_step_f16      */
#define GS_TABLE_BF16     2   /* tables of bfloat16, see gs_sgns_step_bf16      */
#define GS_LR_CONSTANT    0
#define GS_LR_LINEAR      1   /* lr_b = lr0 * max(1 - b / total_batches, 1e-4) */
#define GS_OPT_SGD        0
#define GS_OPT_MOMENTUM   1
#define GS_OPT_ADAM       2

typedef struct gs_sgns_config {
    int32_t dim;
    int32_t walks_per_node;   /* walk ids are rep * n_nodes + v, start node v   */
    int32_t walk_len;
    int32_t window;
    int32_t n_neg;
    int32_t walk_kind;        /* GS_WALK_*                                       */
    int32_t lr_schedule;      /* GS_LR_*                                         */
    int32_t mode;             /* GS_DETERMINISTIC | GS_HOGWILD | GS_HOGWILD_RED, */
                              /* optionally OR-ed with GS_PAIRS_FORWARD_ONLY,    */
                              /* GS_WINDOW_SHRINK                                */
    int32_t max_rounds;       /* node2vec rejection cap                          */
    int32_t table_dtype;      /* GS_TABLE_F32 (0), GS_TABLE_F16 or GS_TABLE_BF16 */
    double  p, q;             /* node2vec parameters                             */
    double  lr0;
    int64_t batch_walks;      /* walks per mini-batch (512 in the paper's runs)  */
    int64_t first_batch;      /* resume point; batches are numbered over the     */
    int64_t num_batches;      /* whole epoch; <= 0 means "to the end"            */
    uint64_t seed;
    const uint32_t *d_keep_thr; /* device, n_nodes thresholds of gs_build_keep_thresholds: */
                              /* walks are sub-sampled before the update; NULL = off      */
    int32_t shuffle_starts;   /* != 0: walk id a starts at the gs_shuffled_starts image  */
    uint32_t epoch;           /* of a mod n_nodes for this epoch instead of at a mod n   */
    /* Optimizer of the synchronous mode (Section 3.2 keeps SGD with momentum and Adam inside the
     * storage; its large run uses momentum 0.9).  GS_OPT_SGD: plain steps, the fields below are
     * ignored.  GS_OPT_MOMENTUM: every batch is one gs_sgns_step_momentum with iteration =
     * iteration_base + batch index; needs GS_LR_CONSTANT, fp32 tables, no pair flags; rows are
     * brought up to date lazily, so call gs_momentum_flush(iteration = iteration_base + index of
     * the last batch + 1) before reading the tables elsewhere; iteration_base + the index after
     * the last batch of the call must stay below 2^31 - 1 (GS_ERR_INVALID_ARG otherwise: the
     * per-row stamps are 32-bit).  GS_OPT_ADAM: every batch is one
     * gs_sgns_step_adam with step = iteration_base + batch index + 1; fp32 tables. */
    int32_t optimizer;        /* GS_OPT_*                                                */
    float   momentum;         /* GS_OPT_MOMENTUM: momentum value; GS_OPT_ADAM: beta1     */
    float   beta2, eps;       /* GS_OPT_ADAM                                             */
    int64_t iteration_base;   /* iterations done before batch 0 of this epoch            */
    float  *d_m_in, *d_m_out; /* momentum tables / first moments, shape of the tables    */
    float  *d_v_in, *d_v_out; /* GS_OPT_ADAM: second moments                             */
    int32_t *d_last_in, *d_last_out;   /* GS_OPT_MOMENTUM: per-row iteration stamps      */
} gs_sgns_config;

typedef struct gs_epoch_stats {
    double  loss_sum;         /* sum of per-pair losses, each at its batch start */
    int64_t pairs;
    int64_t steps;            /* walk transitions taken                          */
    int64_t cap_hits;         /* node2vec rejection cap hits                     */
    int64_t batches;
    int64_t masked_negs;      /* negatives dropped because they equal their context */
                              /* (counted with GS_OPT_SGD only)                      */
    float   ms_walk;          /* device time of the walk kernels                 */
    float   ms_sgns;          /* device time of the SGNS kernels on the caller's stream */
    float   ms_total;
    float   ms_prepare;       /* synchronous mode: device time of the table-independent */
                              /* part of the step (targets, sort) on the walk stream    */
    int64_t refused_ids;      /* see gs_refused_ids: what this call added to the counter */
} gs_epoch_stats;

/*
 * One pass (or a range of mini-batches of one pass) over all walks: for batch
 * b = walk ids [b*batch_walks, (b+1)*batch_walks): generate the walks, then
 * one gs_sgns_step with lr_b (the paper's loop: sample, fetch rows, compute,
 * write back, barrier - Section 3.2).  Walk generation of batch b+1 overlaps
 * the SGNS step of batch b on a second stream; in the synchronous mode that
 * stream also lists and sorts the contributions of batch b+1, which needs no
 * table (results are the same as with one gs_sgns_step per batch).  WAITS for
 * completion and fills *h_out (host struct).  Epoch defaults of the paper: batch 512.
 */
GS_API gs_status gs_sgns_epoch(const gs_graph *g, const uint64_t *d_alias,
                        void *d_w_in, void *d_w_out, const gs_sgns_config *cfg,
                        gs_epoch_stats *h_out, void *stream);

/*
 * Sticky per-device count of ids that the kernels refused (the paper has no counterpart: its
 * storage is addressed with node ids that the partitioner made, Section 3.1).  The library never
 * dereferences an id it has not range-checked; a start node passed in d_starts, a walk entry other
 * than -1, or an alias-table cell that lies outside [0, n_nodes) is treated as absent - and
 * counted here, so that a corrupt input does not pass unnoticed as "fewer pairs".  Counted by
 * gs_random_walks / gs_node2vec_walks (explicit start nodes), by every gs_sgns_step* call except
 * gs_sgns_step_static, and by gs_sgns_epoch (which also reports its own share in
 * gs_epoch_stats.refused_ids).  Reads the counter of the current device into *h_count after the
 * work queued on `stream` so far, clears it if clear != 0, and WAITS.  gs_release_workspace
 * also clears it.
 */
GS_API gs_status gs_refused_ids(uint64_t *h_count, int32_t clear, void *stream);

/* Frees the cached scratch memory of the current device (waits for the device). */
GS_API gs_status gs_release_workspace(void);

/*
 * Which node2vec kernel runs (Section 2.2 names node2vec; the sampler is this library's).
 * 0 (default): one lane per walk, rejection rounds and transitions flattened into one loop, so
 * a lane that has accepted starts its next transition without waiting for its warp.  1, 2, 4,
 * 8, 32: the generic kernel with that many lanes cooperating on a walk - lane k of a group
 * evaluates rejection round base + k and the first accepted round wins; it also serves walk
 * lengths that are not a multiple of 4 and unaligned outputs whatever the setting.  Walks do
 * not depend on this setting.  Other values: GS_ERR_INVALID_ARG.
 */
GS_API gs_status gs_tune_node2vec_group(int32_t lanes);

#ifdef __cplusplus
}
#endif
#endif /* GS_H */
