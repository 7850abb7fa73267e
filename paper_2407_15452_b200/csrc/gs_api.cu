// C ABI entry points (see include/gs.h): argument checks, the graph handle,
// the host-side alias-table builder, the cached scratch memory and the epoch
// driver.  Kernels live in gs_walks.cu, gs_sgns.cu and gs_sort.cu.
#include <math.h>
#include <stdarg.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>
#include <new>
#include <vector>

#include "gs_common.cuh"

namespace gs {

// ---- implemented in the kernel files ------------------------------------------
gs_status validate_csr(const gs_graph *g, bool check_sorted, cudaStream_t st, int64_t *bad_row,
                       int64_t *unsorted_row, int64_t *max_degree, bool *ends_bad);
gs_status build_walk_index(const gs_graph *g, int4 *rec, cudaStream_t st);
gs_status build_edge_hash(const gs_graph *g, unsigned long long *table, unsigned long long mask,
                          cudaStream_t st);
gs_status init_embeddings(float *w_in, float *w_out, int64_t n, int32_t dim, uint64_t seed,
                          cudaStream_t st);
gs_status launch_uniform_walks(const gs_graph *g, const int32_t *starts, int64_t n_walks,
                               int64_t base, int32_t L, uint64_t seed, int32_t *walks,
                               unsigned long long *steps, unsigned long long *refused, cudaStream_t st);
gs_status launch_node2vec_walks(const gs_graph *g, const int32_t *starts, int64_t n_walks,
                                int64_t base, int32_t L, uint64_t seed, double p, double q,
                                int32_t max_rounds, int group, int32_t *walks,
                                unsigned long long *steps, unsigned long long *caps,
                                unsigned long long *refused, cudaStream_t st);
gs_status sgns_step(float *w_in, float *w_out, int64_t n_nodes, int32_t dim, const int32_t *walks,
                    int64_t n_walks, int64_t walk_id_base, int32_t L, int32_t w, int32_t K,
                    const uint64_t *alias, float lr, uint64_t seed, int32_t mode, double *loss,
                    int64_t *pairs, int32_t *dump_pairs, int32_t *dump_negs, cudaStream_t st,
                    unsigned long long *masked = nullptr, int prepared = -1);

gs_status sgns_step_f16(void *w_in, void *w_out, int64_t n_nodes, int32_t dim, const int32_t *walks,
                        int64_t n_walks, int64_t walk_id_base, int32_t L, int32_t w, int32_t K,
                        const uint64_t *alias, float lr, uint64_t seed, int32_t mode, double *loss,
                        int64_t *pairs, int32_t *dump_pairs, int32_t *dump_negs, cudaStream_t st,
                        unsigned long long *masked = nullptr, int prepared = -1);
gs_status init_embeddings_f16(void *w_in, void *w_out, int64_t n, int32_t dim, uint64_t seed,
                              cudaStream_t st);
gs_status init_embeddings_bf16(void *w_in, void *w_out, int64_t n, int32_t dim, uint64_t seed,
                               cudaStream_t st);
gs_status sgns_step_bf16(void *w_in, void *w_out, int64_t n_nodes, int32_t dim, const int32_t *walks,
                         int64_t n_walks, int64_t walk_id_base, int32_t L, int32_t w, int32_t K,
                         const uint64_t *alias, float lr, uint64_t seed, int32_t mode, double *loss,
                         int64_t *pairs, int32_t *dump_pairs, int32_t *dump_negs, cudaStream_t st,
                         unsigned long long *masked = nullptr, int prepared = -1);
gs_status sgns_step_momentum(float *w_in, float *w_out, float *m_in, float *m_out, int32_t *last_in,
                             int32_t *last_out, int64_t n_nodes, int32_t dim, const int32_t *walks,
                             int64_t n_walks, int64_t walk_id_base, int32_t L, int32_t w, int32_t K,
                             const uint64_t *alias, float lr, float mu, int32_t iter, uint64_t seed,
                             double *loss, int64_t *pairs, cudaStream_t st, int prepared = -1);
gs_status sgns_prepare_sync(int64_t n_nodes, int32_t dim, const int32_t *walks, int64_t n_walks,
                            int64_t walk_id_base, int32_t L, int32_t w, int32_t K, const uint64_t *alias,
                            uint64_t seed, int32_t pair_mode, int set, cudaStream_t st);
gs_status momentum_flush(float *w, float *m, int32_t *last, int64_t n_rows, int32_t dim, float lr,
                         float mu, int32_t iter, cudaStream_t st);
gs_status sgns_step_adam(float *w_in, float *w_out, float *m_in, float *v_in, float *m_out,
                         float *v_out, int64_t n_nodes, int32_t dim, const int32_t *walks,
                         int64_t n_walks, int64_t walk_id_base, int32_t L, int32_t w, int32_t K,
                         const uint64_t *alias, float lr, float b1, float b2, float eps, int64_t step,
                         uint64_t seed, int32_t pair_mode, double *loss, int64_t *pairs, cudaStream_t st,
                         int prepared = -1);
gs_status launch_subsample_walks(const int32_t *walks, int64_t n_walks, int64_t base, int32_t L,
                                 const uint32_t *keep_thr, int64_t n_nodes, uint64_t seed, int32_t *out,
                                 unsigned long long *kept, cudaStream_t st);
gs_status launch_shuffled_starts(int64_t n_nodes, uint64_t seed, uint32_t epoch, int64_t first,
                                 int64_t count, int32_t *starts, cudaStream_t st);

// ---- errors ----------------------------------------------------------------------
static thread_local char g_err[512] = "";

void set_error(const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

gs_status cuda_fail(cudaError_t e, const char *what)
{
    set_error("CUDA error %d (%s) in %s", (int)e, cudaGetErrorString(e), what);
    return GS_ERR_CUDA;
}

static gs_status invalid(const char *msg)
{
    set_error("invalid argument: %s", msg);
    return GS_ERR_INVALID_ARG;
}

// ---- per-device state ----------------------------------------------------------------
struct DeviceState {
    void *ws[WS_SLOTS] = {};
    size_t ws_bytes[WS_SLOTS] = {};
    int sms = 0;
};
static std::mutex g_mu;
static DeviceState g_dev[64];

static DeviceState *current_state()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    return &g_dev[dev];
}

int sm_count()
{
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceState *d = current_state();
    if (!d) return 148;
    if (d->sms == 0) {
        int dev = 0, n = 0;
        cudaGetDevice(&dev);
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            n = 148;
        d->sms = n;
    }
    return d->sms;
}

gs_status workspace_get(int slot, size_t bytes, void **out)
{
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceState *d = current_state();
    if (!d) { set_error("no current CUDA device"); return GS_ERR_CUDA; }
    if (d->ws_bytes[slot] < bytes) {
        if (d->ws[slot]) {
            cudaError_t e = cudaFree(d->ws[slot]);       // waits for work that may still use it
            d->ws[slot] = nullptr;
            d->ws_bytes[slot] = 0;
            if (e != cudaSuccess) return cuda_fail(e, "cudaFree(scratch)");
        }
        size_t want = bytes + bytes / 4;                  // head room against regrowth
        want = (want + 255) & ~(size_t)255;
        void *p = nullptr;
        cudaError_t e = cudaMalloc(&p, want);
        if (e != cudaSuccess) {
            cudaGetLastError();
            set_error("scratch allocation of %zu bytes failed: %s", want, cudaGetErrorString(e));
            return GS_ERR_OOM;
        }
        if (slot == WS_COUNTERS && (e = cudaMemset(p, 0, want)) != cudaSuccess) {   // counters start at zero
            cudaFree(p);
            return cuda_fail(e, "cudaMemset(counters)");
        }
        d->ws[slot] = p;
        d->ws_bytes[slot] = want;
    }
    *out = d->ws[slot];
    return GS_OK;
}

unsigned long long *refused_counter()
{
    void *ws = nullptr;
    if (workspace_get(WS_COUNTERS, 256, &ws) != GS_OK) return nullptr;
    return (unsigned long long *)((char *)ws + 160);
}

static bool dim_ok(int32_t dim) { return dim == 32 || dim == 64 || dim == 128 || dim == 256; }

}  // namespace gs

using namespace gs;

extern "C" {

const char *gs_last_error(void) { return g_err; }

gs_status gs_refused_ids(uint64_t *h_count, int32_t clear, void *stream)
{
    if (!h_count) return invalid("h_count is NULL");
    unsigned long long *ctr = refused_counter();
    if (!ctr) return GS_ERR_OOM;
    cudaStream_t st = (cudaStream_t)stream;
    unsigned long long v = 0;
    GS_CUDA_TRY(cudaMemcpyAsync(&v, ctr, sizeof(v), cudaMemcpyDeviceToHost, st));
    if (clear) GS_CUDA_TRY(cudaMemsetAsync(ctr, 0, sizeof(v), st));
    GS_CUDA_TRY(cudaStreamSynchronize(st));
    *h_count = (uint64_t)v;
    return GS_OK;
}

gs_status gs_release_workspace(void)
{
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceState *d = current_state();
    if (!d) return GS_OK;
    for (int s = 0; s < WS_SLOTS; ++s) {
        if (d->ws[s]) {
            cudaError_t e = cudaFree(d->ws[s]);
            d->ws[s] = nullptr;
            d->ws_bytes[s] = 0;
            if (e != cudaSuccess) return cuda_fail(e, "cudaFree(scratch)");
        }
    }
    return GS_OK;
}

// ------------------------------------------------------------------ graph
gs_status gs_graph_load_csr(int64_t n_nodes, int64_t n_edges, const void *d_offsets,
                            int32_t offsets_are_64bit, const int32_t *d_cols, uint32_t flags,
                            void *stream, gs_graph **out)
{
    if (!out) return invalid("out is NULL");
    *out = nullptr;
    if (n_nodes <= 0 || n_nodes >= ((int64_t)1 << 31)) return invalid("n_nodes must be in [1, 2^31)");
    if (n_edges < 0) return invalid("n_edges < 0");
    if (!d_offsets) return invalid("d_offsets is NULL");
    if (n_edges > 0 && !d_cols) return invalid("d_cols is NULL");
    if (!offsets_are_64bit && n_edges >= ((int64_t)1 << 31))
        return invalid("int32 offsets cannot address 2^31 or more edges");
    if (flags & ~(GS_VALIDATE | GS_REQUIRE_SORTED | GS_BUILD_WALK_INDEX | GS_BUILD_EDGE_SET)) return invalid("unknown flag");
    if (flags & (GS_BUILD_WALK_INDEX | GS_BUILD_EDGE_SET)) flags |= GS_VALIDATE;   // built from checked data
    gs_graph *g = new (std::nothrow) gs_graph;
    if (!g) { set_error("out of host memory"); return GS_ERR_OOM; }
    g->n_nodes = n_nodes;
    g->n_edges = n_edges;
    g->d_offsets = d_offsets;
    g->d_cols = d_cols;
    g->offsets64 = offsets_are_64bit ? 1 : 0;
    g->sorted = 0;
    g->max_degree = -1;
    g->device = 0;
    g->d_edge_rec = nullptr;
    g->d_edge_hash = nullptr;
    g->hash_mask = 0;
    cudaGetDevice(&g->device);
    if (flags & (GS_VALIDATE | GS_REQUIRE_SORTED)) {
        int64_t bad = -1, unsorted = -1, maxdeg = 0;
        bool ends_bad = false;
        const bool want_sorted = (flags & GS_REQUIRE_SORTED) != 0;
        gs_status s = validate_csr(g, want_sorted, (cudaStream_t)stream, &bad, &unsorted, &maxdeg,
                                   &ends_bad);
        if (s != GS_OK) { delete g; return s; }
        if (ends_bad) {
            delete g;
            set_error("bad CSR: offsets[0] must be 0 and offsets[n_nodes] must equal n_edges");
            return GS_ERR_BAD_CSR;
        }
        if (bad >= 0) {
            delete g;
            set_error("bad CSR: row %lld has decreasing/out-of-range offsets or a column outside [0, n_nodes)",
                      (long long)bad);
            return GS_ERR_BAD_CSR;
        }
        if (unsorted >= 0) {
            delete g;
            set_error("row %lld is not strictly increasing", (long long)unsorted);
            return GS_ERR_UNSORTED_ADJ;
        }
        g->max_degree = maxdeg;
        g->sorted = want_sorted ? 1 : 0;
    }
    if ((flags & GS_BUILD_WALK_INDEX) && n_edges > 0) {
        void *rec = nullptr;
        cudaError_t e = cudaMalloc(&rec, sizeof(int4) * (size_t)n_edges);
        if (e != cudaSuccess) {
            cudaGetLastError();
            delete g;
            set_error("walk index of %lld x 16 bytes could not be allocated: %s", (long long)n_edges,
                      cudaGetErrorString(e));
            return GS_ERR_OOM;
        }
        g->d_edge_rec = (int4 *)rec;
        gs_status s = build_walk_index(g, g->d_edge_rec, (cudaStream_t)stream);
        if (s != GS_OK) { cudaFree(rec); delete g; return s; }
    }
    if ((flags & GS_BUILD_EDGE_SET) && n_edges > 0) {
        unsigned long long cap = 1024;
        while (cap < 2ull * (unsigned long long)n_edges) cap <<= 1;      // at most half full
        void *tab = nullptr;
        cudaError_t e = cudaMalloc(&tab, sizeof(unsigned long long) * (size_t)cap);
        if (e != cudaSuccess) {
            cudaGetLastError();
            if (g->d_edge_rec) cudaFree(g->d_edge_rec);
            delete g;
            set_error("edge set of %llu x 8 bytes could not be allocated: %s", cap, cudaGetErrorString(e));
            return GS_ERR_OOM;
        }
        g->d_edge_hash = (unsigned long long *)tab;
        g->hash_mask = cap - 1;
        gs_status s = build_edge_hash(g, g->d_edge_hash, g->hash_mask, (cudaStream_t)stream);
        if (s != GS_OK) { cudaFree(tab); if (g->d_edge_rec) cudaFree(g->d_edge_rec); delete g; return s; }
    }
    *out = g;
    return GS_OK;
}

void gs_graph_free(gs_graph *g)
{
    if (!g) return;
    if (g->d_edge_hash) cudaFree(g->d_edge_hash);
    if (g->d_edge_rec) cudaFree(g->d_edge_rec);          // waits for kernels that may still read it
    delete g;
}

gs_status gs_graph_info(const gs_graph *g, int64_t *n_nodes, int64_t *n_edges, int64_t *max_degree,
                        int32_t *rows_sorted)
{
    if (!g) return invalid("graph is NULL");
    if (n_nodes) *n_nodes = g->n_nodes;
    if (n_edges) *n_edges = g->n_edges;
    if (max_degree) *max_degree = g->max_degree;
    if (rows_sorted) *rows_sorted = g->sorted;
    return GS_OK;
}

// ------------------------------------------------------------------ alias table (host)
gs_status gs_build_alias(const double *h_weights, int64_t n, double power, uint64_t *h_table_out)
{
    if (!h_weights || !h_table_out) return invalid("null pointer");
    if (n <= 0 || n >= ((int64_t)1 << 31)) return invalid("n must be in [1, 2^31)");
    std::vector<double> mass;
    std::vector<int64_t> lo_q, hi_q;
    try {
        mass.resize((size_t)n);
        lo_q.resize((size_t)n);
        hi_q.resize((size_t)n);
    } catch (const std::bad_alloc &) {
        set_error("out of host memory building the alias table");
        return GS_ERR_OOM;
    }
    double total = 0.0;
    for (int64_t v = 0; v < n; ++v) {
        const double x = h_weights[v];
        if (!(x >= 0.0) || !isfinite(x)) return invalid("weights must be finite and >= 0");
        mass[v] = x > 0.0 ? pow(x, power) : 0.0;
        total += mass[v];
    }
    if (!(total > 0.0)) return invalid("no positive weight");
    // cells scaled so that the average cell holds mass 1; under-full cells queue in lo_q,
    // the others in hi_q, both in increasing node order
    int64_t lo_head = 0, lo_tail = 0, hi_head = 0, hi_tail = 0;
    for (int64_t v = 0; v < n; ++v) {
        mass[v] = mass[v] * (double)n / total;
        if (mass[v] < 1.0) lo_q[lo_tail++] = v; else hi_q[hi_tail++] = v;
        h_table_out[v] = ((uint64_t)(uint32_t)v << 32) | 0xFFFFFFFFull;   // keep whole cell
    }
    while (lo_head < lo_tail && hi_head < hi_tail) {
        const int64_t under = lo_q[lo_head++];
        const int64_t donor = hi_q[hi_head];
        const double keep = floor(mass[under] * 4294967296.0);
        const uint32_t thr = keep >= 4294967295.0 ? 0xFFFFFFFFu : (uint32_t)keep;
        h_table_out[under] = ((uint64_t)(uint32_t)donor << 32) | (uint64_t)thr;
        mass[donor] = (mass[donor] + mass[under]) - 1.0;
        if (mass[donor] < 1.0) { ++hi_head; lo_q[lo_tail++] = donor; }
    }
    return GS_OK;
}

// ------------------------------------------------------------------ tables
gs_status gs_init_embeddings(float *d_w_in, float *d_w_out, int64_t n_nodes, int32_t dim,
                             uint64_t seed, void *stream)
{
    if (n_nodes < 0) return invalid("n_nodes < 0");
    if (!dim_ok(dim)) { set_error("dim %d not supported (32, 64, 128, 256)", dim); return GS_ERR_UNSUPPORTED; }
    return init_embeddings(d_w_in, d_w_out, n_nodes, dim, seed, (cudaStream_t)stream);
}

// ------------------------------------------------------------------ walks
static gs_status check_walk_args(const gs_graph *g, int64_t n_walks, int64_t base, int32_t L,
                                 const int32_t *out)
{
    if (!g) return invalid("graph is NULL");
    if (n_walks < 0 || base < 0) return invalid("negative n_walks or walk_id_base");
    if (L < 1 || L > 1024) { set_error("walk_len %d outside [1, 1024]", L); return GS_ERR_UNSUPPORTED; }
    if (n_walks > 0 && !out) return invalid("d_walks_out is NULL");
    return GS_OK;
}

gs_status gs_random_walks(const gs_graph *g, const int32_t *d_starts, int64_t n_walks,
                          int64_t walk_id_base, int32_t walk_len, uint64_t seed,
                          int32_t *d_walks_out, uint64_t *d_steps, void *stream)
{
    gs_status s = check_walk_args(g, n_walks, walk_id_base, walk_len, d_walks_out);
    if (s != GS_OK) return s;
    return launch_uniform_walks(g, d_starts, n_walks, walk_id_base, walk_len, seed, d_walks_out,
                                (unsigned long long *)d_steps, d_starts ? refused_counter() : nullptr,
                                (cudaStream_t)stream);
}

static int g_n2v_group = 0;   // node2vec kernel: 0 = one lane per walk, flattened loop (the default)

gs_status gs_node2vec_walks(const gs_graph *g, const int32_t *d_starts, int64_t n_walks,
                            int64_t walk_id_base, int32_t walk_len, uint64_t seed, double p,
                            double q, int32_t max_rounds, int32_t *d_walks_out, uint64_t *d_steps,
                            uint64_t *d_cap_hits, void *stream)
{
    gs_status s = check_walk_args(g, n_walks, walk_id_base, walk_len, d_walks_out);
    if (s != GS_OK) return s;
    if (!(p > 0.0) || !(q > 0.0) || !isfinite(p) || !isfinite(q)) return invalid("p and q must be positive");
    if (max_rounds < 1 || max_rounds > 65536) return invalid("max_rounds outside [1, 65536]");
    if (!g->sorted) {
        set_error("node2vec needs a graph loaded with GS_REQUIRE_SORTED");
        return GS_ERR_UNSORTED_ADJ;
    }
    return launch_node2vec_walks(g, d_starts, n_walks, walk_id_base, walk_len, seed, p, q,
                                 max_rounds, g_n2v_group, d_walks_out,
                                 (unsigned long long *)d_steps, (unsigned long long *)d_cap_hits,
                                 d_starts ? refused_counter() : nullptr, (cudaStream_t)stream);
}

// Which node2vec kernel runs: 0 the flattened one-lane kernel, 1..32 the generic kernel with that
// many lanes per walk.  Results do not depend on it.
gs_status gs_tune_node2vec_group(int32_t lanes)
{
    if (lanes != 0 && lanes != 1 && lanes != 2 && lanes != 4 && lanes != 8 && lanes != 32)
        return invalid("lanes per walk must be 0 (one lane, flattened loop), 1, 2, 4, 8 or 32");
    g_n2v_group = lanes;
    return GS_OK;
}

// ------------------------------------------------------------------ SGNS
static gs_status check_sgns_shape(int32_t dim, int32_t L, int32_t w, int32_t K, int32_t mode)
{
    if (!dim_ok(dim)) { set_error("dim %d not supported (32, 64, 128, 256)", dim); return GS_ERR_UNSUPPORTED; }
    if (L < 1 || L > 1024) { set_error("walk_len %d outside [1, 1024]", L); return GS_ERR_UNSUPPORTED; }
    if (w < 1 || w > 32) { set_error("window %d outside [1, 32]", w); return GS_ERR_UNSUPPORTED; }
    if (K < 0 || K > 32) { set_error("n_neg %d outside [0, 32]", K); return GS_ERR_UNSUPPORTED; }
    if (2 * w * (1 + K) > 512) { set_error("2*window*(1+n_neg) = %d exceeds 512", 2 * w * (1 + K)); return GS_ERR_UNSUPPORTED; }
    const int32_t base_mode = mode & ~(GS_PAIRS_FORWARD_ONLY | GS_WINDOW_SHRINK | GS_ROUND_STOCHASTIC);
    if (base_mode != GS_DETERMINISTIC && base_mode != GS_HOGWILD && base_mode != GS_HOGWILD_RED)
        return invalid("unknown mode");
    return GS_OK;
}

gs_status gs_sgns_step(float *d_w_in, float *d_w_out, int64_t n_nodes, int32_t dim,
                       const int32_t *d_walks, int64_t n_walks, int64_t walk_id_base,
                       int32_t walk_len, int32_t window, int32_t n_neg, const uint64_t *d_alias,
                       float lr, uint64_t seed, int32_t mode, double *d_loss_sum,
                       int64_t *d_pair_count, int32_t *d_pairs_dump, int32_t *d_negs_dump,
                       void *stream)
{
    if (!d_w_in || !d_w_out) return invalid("table pointer is NULL");
    if (n_nodes <= 0 || n_nodes >= ((int64_t)1 << 31)) return invalid("n_nodes must be in [1, 2^31)");
    if (n_walks < 0 || walk_id_base < 0) return invalid("negative n_walks or walk_id_base");
    if (n_walks > 0 && !d_walks) return invalid("d_walks is NULL");
    gs_status s = check_sgns_shape(dim, walk_len, window, n_neg, mode);
    if (s != GS_OK) return s;
    if (n_neg > 0 && !d_alias) return invalid("d_alias is NULL");
    if (((uintptr_t)d_w_in | (uintptr_t)d_w_out) & 15) return invalid("tables must be 16-byte aligned");
    return sgns_step(d_w_in, d_w_out, n_nodes, dim, d_walks, n_walks, walk_id_base, walk_len,
                     window, n_neg, d_alias, lr, seed, mode, d_loss_sum, d_pair_count,
                     d_pairs_dump, d_negs_dump, (cudaStream_t)stream);
}

// ------------------------------------------------------------------ 16-bit tables
static bool dim_ok_f16(int32_t dim) { return dim == 64 || dim == 128 || dim == 256; }

static gs_status init_embeddings_16(bool bf16, void *d_w_in, void *d_w_out, int64_t n_nodes, int32_t dim,
                                    uint64_t seed, void *stream)
{
    if (n_nodes < 0) return invalid("n_nodes < 0");
    if (!dim_ok_f16(dim)) { set_error("dim %d not supported with 16-bit tables (64, 128, 256)", dim); return GS_ERR_UNSUPPORTED; }
    return bf16 ? init_embeddings_bf16(d_w_in, d_w_out, n_nodes, dim, seed, (cudaStream_t)stream)
                : init_embeddings_f16(d_w_in, d_w_out, n_nodes, dim, seed, (cudaStream_t)stream);
}

static gs_status sgns_step_16(bool bf16, void *d_w_in, void *d_w_out, int64_t n_nodes, int32_t dim,
                              const int32_t *d_walks, int64_t n_walks, int64_t walk_id_base,
                              int32_t walk_len, int32_t window, int32_t n_neg, const uint64_t *d_alias,
                              float lr, uint64_t seed, int32_t mode, double *d_loss_sum,
                              int64_t *d_pair_count, int32_t *d_pairs_dump, int32_t *d_negs_dump,
                              void *stream)
{
    if (!d_w_in || !d_w_out) return invalid("table pointer is NULL");
    if (n_nodes <= 0 || n_nodes >= ((int64_t)1 << 31)) return invalid("n_nodes must be in [1, 2^31)");
    if (n_walks < 0 || walk_id_base < 0) return invalid("negative n_walks or walk_id_base");
    if (n_walks > 0 && !d_walks) return invalid("d_walks is NULL");
    if (!dim_ok_f16(dim)) { set_error("dim %d not supported with 16-bit tables (64, 128, 256)", dim); return GS_ERR_UNSUPPORTED; }
    gs_status s = check_sgns_shape(128, walk_len, window, n_neg, mode);
    if (s != GS_OK) return s;
    if (n_neg > 0 && !d_alias) return invalid("d_alias is NULL");
    if (((uintptr_t)d_w_in | (uintptr_t)d_w_out) & 15) return invalid("tables must be 16-byte aligned");
    return bf16 ? sgns_step_bf16(d_w_in, d_w_out, n_nodes, dim, d_walks, n_walks, walk_id_base, walk_len,
                                 window, n_neg, d_alias, lr, seed, mode, d_loss_sum, d_pair_count,
                                 d_pairs_dump, d_negs_dump, (cudaStream_t)stream)
                : sgns_step_f16(d_w_in, d_w_out, n_nodes, dim, d_walks, n_walks, walk_id_base, walk_len,
                                window, n_neg, d_alias, lr, seed, mode, d_loss_sum, d_pair_count,
                                d_pairs_dump, d_negs_dump, (cudaStream_t)stream);
}

gs_status gs_init_embeddings_f16(void *d_w_in, void *d_w_out, int64_t n_nodes, int32_t dim,
                                 uint64_t seed, void *stream)
{
    return init_embeddings_16(false, d_w_in, d_w_out, n_nodes, dim, seed, stream);
}

gs_status gs_init_embeddings_bf16(void *d_w_in, void *d_w_out, int64_t n_nodes, int32_t dim,
                                  uint64_t seed, void *stream)
{
    return init_embeddings_16(true, d_w_in, d_w_out, n_nodes, dim, seed, stream);
}

gs_status gs_sgns_step_f16(void *d_w_in, void *d_w_out, int64_t n_nodes, int32_t dim,
                           const int32_t *d_walks, int64_t n_walks, int64_t walk_id_base,
                           int32_t walk_len, int32_t window, int32_t n_neg, const uint64_t *d_alias,
                           float lr, uint64_t seed, int32_t mode, double *d_loss_sum,
                           int64_t *d_pair_count, int32_t *d_pairs_dump, int32_t *d_negs_dump,
                           void *stream)
{
    return sgns_step_16(false, d_w_in, d_w_out, n_nodes, dim, d_walks, n_walks, walk_id_base, walk_len, window,
                        n_neg, d_alias, lr, seed, mode, d_loss_sum, d_pair_count, d_pairs_dump, d_negs_dump,
                        stream);
}

gs_status gs_sgns_step_bf16(void *d_w_in, void *d_w_out, int64_t n_nodes, int32_t dim,
                            const int32_t *d_walks, int64_t n_walks, int64_t walk_id_base,
                            int32_t walk_len, int32_t window, int32_t n_neg, const uint64_t *d_alias,
                            float lr, uint64_t seed, int32_t mode, double *d_loss_sum,
                            int64_t *d_pair_count, int32_t *d_pairs_dump, int32_t *d_negs_dump,
                            void *stream)
{
    return sgns_step_16(true, d_w_in, d_w_out, n_nodes, dim, d_walks, n_walks, walk_id_base, walk_len, window,
                        n_neg, d_alias, lr, seed, mode, d_loss_sum, d_pair_count, d_pairs_dump, d_negs_dump,
                        stream);
}

// ------------------------------------------------------------------ momentum
gs_status gs_sgns_step_momentum(float *d_w_in, float *d_w_out, float *d_m_in, float *d_m_out,
                                int32_t *d_last_in, int32_t *d_last_out, int64_t n_nodes,
                                int32_t dim, const int32_t *d_walks, int64_t n_walks,
                                int64_t walk_id_base, int32_t walk_len, int32_t window, int32_t n_neg,
                                const uint64_t *d_alias, float lr, float momentum, int32_t iteration,
                                uint64_t seed, double *d_loss_sum, int64_t *d_pair_count, void *stream)
{
    if (!d_w_in || !d_w_out || !d_m_in || !d_m_out || !d_last_in || !d_last_out)
        return invalid("table, momentum or stamp pointer is NULL");
    if (n_nodes <= 0 || n_nodes >= ((int64_t)1 << 31)) return invalid("n_nodes must be in [1, 2^31)");
    if (n_walks < 0 || walk_id_base < 0) return invalid("negative n_walks or walk_id_base");
    if (n_walks > 0 && !d_walks) return invalid("d_walks is NULL");
    if (!(momentum >= 0.f) || !(momentum < 1.f)) return invalid("momentum must be in [0, 1)");
    if (iteration < 0 || iteration == 0x7FFFFFFF) return invalid("iteration must be in [0, 2^31 - 1)");
    gs_status s = check_sgns_shape(dim, walk_len, window, n_neg, GS_DETERMINISTIC);
    if (s != GS_OK) return s;
    if (n_neg > 0 && !d_alias) return invalid("d_alias is NULL");
    if (((uintptr_t)d_w_in | (uintptr_t)d_w_out | (uintptr_t)d_m_in | (uintptr_t)d_m_out) & 15)
        return invalid("tables must be 16-byte aligned");
    return sgns_step_momentum(d_w_in, d_w_out, d_m_in, d_m_out, d_last_in, d_last_out, n_nodes, dim,
                              d_walks, n_walks, walk_id_base, walk_len, window, n_neg, d_alias, lr,
                              momentum, iteration, seed, d_loss_sum, d_pair_count, (cudaStream_t)stream);
}

gs_status gs_momentum_flush(float *d_w, float *d_m, int32_t *d_last, int64_t n_rows, int32_t dim,
                            float lr, float momentum, int32_t iteration, void *stream)
{
    if (!d_w || !d_m || !d_last) return invalid("null pointer");
    if (n_rows < 0) return invalid("n_rows < 0");
    if (!dim_ok(dim)) { set_error("dim %d not supported (32, 64, 128, 256)", dim); return GS_ERR_UNSUPPORTED; }
    if (!(momentum >= 0.f) || !(momentum < 1.f)) return invalid("momentum must be in [0, 1)");
    if (iteration < 0) return invalid("iteration < 0");
    return momentum_flush(d_w, d_m, d_last, n_rows, dim, lr, momentum, iteration, (cudaStream_t)stream);
}

// ------------------------------------------------------------------ Adam
gs_status gs_sgns_step_adam(float *d_w_in, float *d_w_out, float *d_m_in, float *d_v_in,
                            float *d_m_out, float *d_v_out, int64_t n_nodes, int32_t dim,
                            const int32_t *d_walks, int64_t n_walks, int64_t walk_id_base,
                            int32_t walk_len, int32_t window, int32_t n_neg, const uint64_t *d_alias,
                            float lr, float beta1, float beta2, float eps, int64_t step, uint64_t seed,
                            int32_t pair_mode, double *d_loss_sum, int64_t *d_pair_count, void *stream)
{
    if (!d_w_in || !d_w_out || !d_m_in || !d_v_in || !d_m_out || !d_v_out)
        return invalid("table or moment pointer is NULL");
    if (n_nodes <= 0 || n_nodes >= ((int64_t)1 << 31)) return invalid("n_nodes must be in [1, 2^31)");
    if (n_walks < 0 || walk_id_base < 0) return invalid("negative n_walks or walk_id_base");
    if (n_walks > 0 && !d_walks) return invalid("d_walks is NULL");
    if (!(beta1 >= 0.f) || !(beta1 < 1.f) || !(beta2 >= 0.f) || !(beta2 < 1.f))
        return invalid("beta1 and beta2 must be in [0, 1)");
    if (!(eps > 0.f)) return invalid("eps must be positive");
    if (step < 1) return invalid("step counts from 1");
    if (pair_mode & ~(GS_PAIRS_FORWARD_ONLY | GS_WINDOW_SHRINK)) return invalid("unknown pair_mode flag");
    gs_status s = check_sgns_shape(dim, walk_len, window, n_neg, GS_DETERMINISTIC);
    if (s != GS_OK) return s;
    if (n_neg > 0 && !d_alias) return invalid("d_alias is NULL");
    if (((uintptr_t)d_w_in | (uintptr_t)d_w_out | (uintptr_t)d_m_in | (uintptr_t)d_m_out |
         (uintptr_t)d_v_in | (uintptr_t)d_v_out) & 15)
        return invalid("tables must be 16-byte aligned");
    return sgns_step_adam(d_w_in, d_w_out, d_m_in, d_v_in, d_m_out, d_v_out, n_nodes, dim, d_walks,
                          n_walks, walk_id_base, walk_len, window, n_neg, d_alias, lr, beta1, beta2,
                          eps, step, seed, pair_mode, d_loss_sum, d_pair_count, (cudaStream_t)stream);
}

// ------------------------------------------------------------------ corpus variants
gs_status gs_build_keep_thresholds(const double *h_weights, int64_t n, double t, uint32_t *h_thr_out)
{
    if (!h_weights || !h_thr_out) return invalid("null pointer");
    if (n <= 0) return invalid("n must be positive");
    if (!(t > 0.0) || !isfinite(t)) return invalid("t must be positive");
    double sum = 0.0;
    for (int64_t v = 0; v < n; ++v) {
        const double x = h_weights[v];
        if (!(x >= 0.0) || !isfinite(x)) return invalid("weights must be finite and >= 0");
        sum += x;
    }
    if (!(sum > 0.0)) return invalid("no positive weight");
    for (int64_t v = 0; v < n; ++v) {
        uint32_t thr = 0xFFFFFFFFu;                       // always kept
        if (h_weights[v] > 0.0) {
            const double freq = h_weights[v] / sum;
            const double keep = sqrt(t / freq);
            if (keep < 1.0) {
                const double scaled = floor(keep * 4294967296.0);
                if (scaled < 4294967295.0) thr = (uint32_t)scaled;
            }
        }
        h_thr_out[v] = thr;
    }
    return GS_OK;
}

gs_status gs_subsample_walks(const int32_t *d_walks, int64_t n_walks, int64_t walk_id_base,
                             int32_t walk_len, const uint32_t *d_keep_thr, int64_t n_nodes,
                             uint64_t seed, int32_t *d_walks_out, uint64_t *d_kept, void *stream)
{
    if (n_walks < 0 || walk_id_base < 0) return invalid("negative n_walks or walk_id_base");
    if (n_nodes <= 0 || n_nodes >= ((int64_t)1 << 31)) return invalid("n_nodes must be in [1, 2^31)");
    if (walk_len < 1 || walk_len > 1024) { set_error("walk_len %d outside [1, 1024]", walk_len); return GS_ERR_UNSUPPORTED; }
    if (n_walks > 0 && (!d_walks || !d_walks_out || !d_keep_thr)) return invalid("null pointer");
    return launch_subsample_walks(d_walks, n_walks, walk_id_base, walk_len, d_keep_thr, n_nodes, seed,
                                  d_walks_out, (unsigned long long *)d_kept, (cudaStream_t)stream);
}

gs_status gs_shuffled_starts(int64_t n_nodes, uint64_t seed, uint32_t epoch, int64_t walk_id_first,
                             int64_t count, int32_t *d_starts_out, void *stream)
{
    if (n_nodes <= 0 || n_nodes >= ((int64_t)1 << 31)) return invalid("n_nodes must be in [1, 2^31)");
    if (walk_id_first < 0 || count < 0) return invalid("negative walk_id_first or count");
    if (count > 0 && !d_starts_out) return invalid("d_starts_out is NULL");
    return launch_shuffled_starts(n_nodes, seed, epoch, walk_id_first, count, d_starts_out,
                                  (cudaStream_t)stream);
}

// ------------------------------------------------------------------ epoch driver
struct EpochCounters {
    double loss;
    long long pairs;
    unsigned long long steps;
    unsigned long long caps;
    unsigned long long masked;
};

namespace {
// A small ring of event pairs that accumulates device time of one kind of work.
struct TimerRing {
    static const int N = 8;
    cudaEvent_t beg[N], end[N];
    bool used[N];
    int next = 0;
    double total_ms = 0.0;
    bool ok = false;
    bool init()
    {
        for (int i = 0; i < N; ++i) {
            used[i] = false;
            if (cudaEventCreate(&beg[i]) != cudaSuccess || cudaEventCreate(&end[i]) != cudaSuccess)
                return false;
        }
        ok = true;
        return true;
    }
    void collect(int i)
    {
        if (!used[i]) return;
        float ms = 0.f;
        if (cudaEventSynchronize(end[i]) == cudaSuccess &&
            cudaEventElapsedTime(&ms, beg[i], end[i]) == cudaSuccess)
            total_ms += ms;
        used[i] = false;
    }
    int start(cudaStream_t st)
    {
        const int i = next;
        next = (next + 1) % N;
        collect(i);
        cudaEventRecord(beg[i], st);
        return i;
    }
    void stop(int i, cudaStream_t st) { cudaEventRecord(end[i], st); used[i] = true; }
    void finish() { for (int i = 0; i < N; ++i) collect(i); }
    void destroy()
    {
        if (!ok) return;
        for (int i = 0; i < N; ++i) { cudaEventDestroy(beg[i]); cudaEventDestroy(end[i]); }
    }
};
}  // namespace

gs_status gs_sgns_epoch(const gs_graph *g, const uint64_t *d_alias, void *d_w_in, void *d_w_out,
                        const gs_sgns_config *cfg, gs_epoch_stats *h_out, void *stream)
{
    if (!g || !cfg || !h_out) return invalid("null pointer");
    if (!d_w_in || !d_w_out) return invalid("table pointer is NULL");
    if (cfg->table_dtype != GS_TABLE_F32 && cfg->table_dtype != GS_TABLE_F16 &&
        cfg->table_dtype != GS_TABLE_BF16)
        return invalid("unknown table_dtype");
    const bool f16 = cfg->table_dtype != GS_TABLE_F32;         // a 16-bit storage format
    const bool bf16 = cfg->table_dtype == GS_TABLE_BF16;
    if (f16 && !dim_ok_f16(cfg->dim)) { set_error("dim %d not supported with 16-bit tables (64, 128, 256)", cfg->dim); return GS_ERR_UNSUPPORTED; }
    gs_status s = check_sgns_shape(f16 ? 128 : cfg->dim, cfg->walk_len, cfg->window, cfg->n_neg, cfg->mode);
    if (s != GS_OK) return s;
    if (cfg->n_neg > 0 && !d_alias) return invalid("d_alias is NULL");
    if ((cfg->mode & GS_ROUND_STOCHASTIC) && !f16) { set_error("GS_ROUND_STOCHASTIC applies to 16-bit tables"); return GS_ERR_UNSUPPORTED; }
    if (cfg->walks_per_node < 1 || cfg->batch_walks < 1) return invalid("walks_per_node and batch_walks must be >= 1");
    if (cfg->walk_kind != GS_WALK_UNIFORM && cfg->walk_kind != GS_WALK_NODE2VEC) return invalid("unknown walk_kind");
    if (cfg->lr_schedule != GS_LR_CONSTANT && cfg->lr_schedule != GS_LR_LINEAR) return invalid("unknown lr_schedule");
    if (cfg->first_batch < 0) return invalid("first_batch < 0");
    if (cfg->walk_kind == GS_WALK_NODE2VEC) {
        if (!g->sorted) { set_error("node2vec needs a graph loaded with GS_REQUIRE_SORTED"); return GS_ERR_UNSORTED_ADJ; }
        if (!(cfg->p > 0.0) || !(cfg->q > 0.0)) return invalid("p and q must be positive");
        if (cfg->max_rounds < 1 || cfg->max_rounds > 65536) return invalid("max_rounds outside [1, 65536]");
    }
    if (cfg->optimizer != GS_OPT_SGD) {
        if (cfg->optimizer != GS_OPT_MOMENTUM && cfg->optimizer != GS_OPT_ADAM) return invalid("unknown optimizer");
        if (f16) { set_error("momentum and Adam need fp32 tables"); return GS_ERR_UNSUPPORTED; }
        if ((cfg->mode & 0xFF) != GS_DETERMINISTIC) return invalid("momentum and Adam run in the synchronous mode only");
        if (cfg->iteration_base < 0 || cfg->iteration_base > 0x7FFFFFF0) return invalid("iteration_base outside [0, 2^31 - 16)");
        if (!cfg->d_m_in || !cfg->d_m_out) return invalid("moment tables are NULL");
        if (cfg->optimizer == GS_OPT_MOMENTUM) {
            if (cfg->lr_schedule != GS_LR_CONSTANT) return invalid("momentum needs a constant learning rate");
            if (cfg->mode != GS_DETERMINISTIC) return invalid("momentum takes no pair flags");
            if (!cfg->d_last_in || !cfg->d_last_out) return invalid("iteration stamps are NULL");
            if (!(cfg->momentum >= 0.f) || !(cfg->momentum < 1.f)) return invalid("momentum must be in [0, 1)");
        } else {
            if (!cfg->d_v_in || !cfg->d_v_out) return invalid("second-moment tables are NULL");
            if (!(cfg->momentum >= 0.f) || !(cfg->momentum < 1.f) || !(cfg->beta2 >= 0.f) || !(cfg->beta2 < 1.f))
                return invalid("beta1 and beta2 must be in [0, 1)");
            if (!(cfg->eps > 0.f)) return invalid("eps must be positive");
        }
    }
    memset(h_out, 0, sizeof(*h_out));
    const int64_t total_walks = g->n_nodes * (int64_t)cfg->walks_per_node;
    const int64_t nb_total = (total_walks + cfg->batch_walks - 1) / cfg->batch_walks;
    int64_t b_end = cfg->num_batches > 0 ? cfg->first_batch + cfg->num_batches : nb_total;
    if (b_end > nb_total) b_end = nb_total;
    if (cfg->first_batch >= b_end) return GS_OK;
    // momentum stamps and the iteration argument are 32-bit: the last batch's iteration + 1 must fit
    if (cfg->optimizer == GS_OPT_MOMENTUM && cfg->iteration_base + b_end > (int64_t)0x7FFFFFFE) {
        set_error("invalid argument: iteration_base + last batch = %lld exceeds 2^31 - 2; start a new "
                  "run of iterations (flush the momentum first)", (long long)(cfg->iteration_base + b_end));
        return GS_ERR_INVALID_ARG;
    }

    // The walk sampler (with the table-independent part of the synchronous step) runs on a stream
    // of the highest priority, the updates on the caller's.  The sampler's work for batch b+1 is
    // the shorter chain and batch b+1 cannot start without it, so where blocks of both are waiting
    // for an SM the sampler's go first (measured on the 1M-node workload, synchronous mode:
    // 0.43 ms per batch against 0.46 with equal priorities and 0.49 the other way round).
    cudaStream_t s_sgns = (cudaStream_t)stream;
    cudaStream_t s_walk = nullptr;
    cudaEvent_t ev_walk[2] = { nullptr, nullptr }, ev_sgns[2] = { nullptr, nullptr };
    cudaEvent_t ev_begin = nullptr, ev_end = nullptr;
    TimerRing t_walk, t_sgns, t_prep;
    const bool sync_mode = (cfg->mode & 0xFF) == GS_DETERMINISTIC;
    gs_status rc = GS_OK;
    int32_t *wbuf[2] = { nullptr, nullptr };
    int32_t *sbuf[2] = { nullptr, nullptr };
    EpochCounters *ctr = nullptr;
    EpochCounters host_ctr;
    memset(&host_ctr, 0, sizeof(host_ctr));
    unsigned long long refused_before = 0, refused_after = 0;
    unsigned long long *refused_ctr = nullptr;

#define EP_TRY(expr)                                                   \
    do {                                                               \
        cudaError_t _e = (expr);                                       \
        if (_e != cudaSuccess) { rc = cuda_fail(_e, #expr); goto done; } \
    } while (0)
#define EP_CALL(expr)                                                  \
    do { rc = (expr); if (rc != GS_OK) goto done; } while (0)

    {
        const size_t wbytes = sizeof(int32_t) * (size_t)cfg->batch_walks * (size_t)cfg->walk_len;
        void *p = nullptr;
        EP_CALL(workspace_get(WS_WALKS0, wbytes, &p)); wbuf[0] = (int32_t *)p;
        EP_CALL(workspace_get(WS_WALKS1, wbytes, &p)); wbuf[1] = (int32_t *)p;
        EP_CALL(workspace_get(WS_COUNTERS, 256, &p)); ctr = (EpochCounters *)p;
        if (cfg->shuffle_starts) {                       // start nodes of the two batches in flight
            EP_CALL(workspace_get(WS_STARTS, 2 * sizeof(int32_t) * (size_t)cfg->batch_walks, &p));
            sbuf[0] = (int32_t *)p;
            sbuf[1] = sbuf[0] + cfg->batch_walks;
        }
    }
    {
        int least = 0, greatest = 0;
        EP_TRY(cudaDeviceGetStreamPriorityRange(&least, &greatest));
        EP_TRY(cudaStreamCreateWithPriority(&s_walk, cudaStreamNonBlocking, greatest));
    }
    for (int i = 0; i < 2; ++i) {
        EP_TRY(cudaEventCreateWithFlags(&ev_walk[i], cudaEventDisableTiming));
        EP_TRY(cudaEventCreateWithFlags(&ev_sgns[i], cudaEventDisableTiming));
    }
    EP_TRY(cudaEventCreate(&ev_begin));
    EP_TRY(cudaEventCreate(&ev_end));
    if (!t_walk.init() || !t_sgns.init() || !t_prep.init()) { rc = cuda_fail(cudaGetLastError(), "cudaEventCreate"); goto done; }

    EP_TRY(cudaMemsetAsync(ctr, 0, sizeof(EpochCounters), s_sgns));
    refused_ctr = refused_counter();
    if (refused_ctr)
        EP_TRY(cudaMemcpyAsync(&refused_before, refused_ctr, sizeof(refused_before), cudaMemcpyDeviceToHost, s_sgns));
    EP_TRY(cudaEventRecord(ev_begin, s_sgns));
    EP_TRY(cudaStreamWaitEvent(s_walk, ev_begin, 0));        // the walk stream starts after prior work

    for (int64_t b = cfg->first_batch; b < b_end; ++b) {
        const int buf = (int)((b - cfg->first_batch) & 1);
        const int64_t base = b * cfg->batch_walks;
        const int64_t n = (base + cfg->batch_walks <= total_walks) ? cfg->batch_walks : total_walks - base;
        // this walk buffer was last read by the SGNS step two batches ago
        if (b - cfg->first_batch >= 2) EP_TRY(cudaStreamWaitEvent(s_walk, ev_sgns[buf], 0));
        {
            const int tk = t_walk.start(s_walk);
            const int32_t *starts = nullptr;
            if (cfg->shuffle_starts) {
                EP_CALL(launch_shuffled_starts(g->n_nodes, cfg->seed, cfg->epoch, base, n, sbuf[buf], s_walk));
                starts = sbuf[buf];
            }
            if (cfg->walk_kind == GS_WALK_UNIFORM)
                EP_CALL(launch_uniform_walks(g, starts, n, base, cfg->walk_len, cfg->seed, wbuf[buf],
                                             &ctr->steps, nullptr, s_walk));
            else
                EP_CALL(launch_node2vec_walks(g, starts, n, base, cfg->walk_len, cfg->seed, cfg->p,
                                              cfg->q, cfg->max_rounds, g_n2v_group, wbuf[buf],
                                              &ctr->steps, &ctr->caps, nullptr, s_walk));
            if (cfg->d_keep_thr)
                EP_CALL(launch_subsample_walks(wbuf[buf], n, base, cfg->walk_len, cfg->d_keep_thr,
                                               g->n_nodes, cfg->seed, wbuf[buf], nullptr, s_walk));
            t_walk.stop(tk, s_walk);
        }
        // Synchronous mode: the targets of the batch and their sorted keys do not depend on the
        // tables, so they are produced here, on the walk stream, into scratch set `buf`, while the
        // update of the batch before this one still runs on the other stream.
        const int prepared = sync_mode ? buf : -1;
        if (sync_mode) {
            const int tk = t_prep.start(s_walk);
            EP_CALL(sgns_prepare_sync(g->n_nodes, cfg->dim, wbuf[buf], n, base, cfg->walk_len, cfg->window,
                                      cfg->n_neg, d_alias, cfg->seed, cfg->mode & ~0xFF, buf, s_walk));
            t_prep.stop(tk, s_walk);
        }
        EP_TRY(cudaEventRecord(ev_walk[buf], s_walk));
        EP_TRY(cudaStreamWaitEvent(s_sgns, ev_walk[buf], 0));
        {
            double lr = cfg->lr0;
            if (cfg->lr_schedule == GS_LR_LINEAR) {
                double f = 1.0 - (double)b / (double)nb_total;
                lr = cfg->lr0 * (f > 1e-4 ? f : 1e-4);
            }
            const int tk = t_sgns.start(s_sgns);
            if (cfg->optimizer == GS_OPT_MOMENTUM)
                EP_CALL(sgns_step_momentum((float *)d_w_in, (float *)d_w_out, cfg->d_m_in, cfg->d_m_out,
                                           cfg->d_last_in, cfg->d_last_out, g->n_nodes, cfg->dim, wbuf[buf],
                                           n, base, cfg->walk_len, cfg->window, cfg->n_neg, d_alias,
                                           (float)lr, cfg->momentum, (int32_t)(cfg->iteration_base + b),
                                           cfg->seed, &ctr->loss, (int64_t *)&ctr->pairs, s_sgns, prepared));
            else if (cfg->optimizer == GS_OPT_ADAM)
                EP_CALL(sgns_step_adam((float *)d_w_in, (float *)d_w_out, cfg->d_m_in, cfg->d_v_in,
                                       cfg->d_m_out, cfg->d_v_out, g->n_nodes, cfg->dim, wbuf[buf], n, base,
                                       cfg->walk_len, cfg->window, cfg->n_neg, d_alias, (float)lr,
                                       cfg->momentum, cfg->beta2, cfg->eps, cfg->iteration_base + b + 1,
                                       cfg->seed, cfg->mode & ~0xFF, &ctr->loss, (int64_t *)&ctr->pairs,
                                       s_sgns, prepared));
            else if (bf16)
                EP_CALL(sgns_step_bf16(d_w_in, d_w_out, g->n_nodes, cfg->dim, wbuf[buf], n, base,
                                       cfg->walk_len, cfg->window, cfg->n_neg, d_alias, (float)lr,
                                       cfg->seed, cfg->mode, &ctr->loss, (int64_t *)&ctr->pairs, nullptr,
                                       nullptr, s_sgns, &ctr->masked, prepared));
            else if (f16)
                EP_CALL(sgns_step_f16(d_w_in, d_w_out, g->n_nodes, cfg->dim, wbuf[buf], n, base,
                                      cfg->walk_len, cfg->window, cfg->n_neg, d_alias, (float)lr,
                                      cfg->seed, cfg->mode, &ctr->loss, (int64_t *)&ctr->pairs, nullptr,
                                      nullptr, s_sgns, &ctr->masked, prepared));
            else
                EP_CALL(sgns_step((float *)d_w_in, (float *)d_w_out, g->n_nodes, cfg->dim, wbuf[buf], n,
                                  base, cfg->walk_len, cfg->window, cfg->n_neg, d_alias, (float)lr,
                                  cfg->seed, cfg->mode, &ctr->loss, (int64_t *)&ctr->pairs, nullptr,
                                  nullptr, s_sgns, &ctr->masked, prepared));
            t_sgns.stop(tk, s_sgns);
        }
        EP_TRY(cudaEventRecord(ev_sgns[buf], s_sgns));
        ++h_out->batches;
    }
    EP_TRY(cudaEventRecord(ev_end, s_sgns));
    EP_TRY(cudaMemcpyAsync(&host_ctr, ctr, sizeof(host_ctr), cudaMemcpyDeviceToHost, s_sgns));
    if (refused_ctr)
        EP_TRY(cudaMemcpyAsync(&refused_after, refused_ctr, sizeof(refused_after), cudaMemcpyDeviceToHost, s_sgns));
    EP_TRY(cudaStreamSynchronize(s_sgns));
    EP_TRY(cudaStreamSynchronize(s_walk));
    t_walk.finish();
    t_sgns.finish();
    t_prep.finish();
    h_out->loss_sum = host_ctr.loss;
    h_out->pairs = (int64_t)host_ctr.pairs;
    h_out->steps = (int64_t)host_ctr.steps;
    h_out->cap_hits = (int64_t)host_ctr.caps;
    h_out->masked_negs = (int64_t)host_ctr.masked;
    h_out->ms_walk = (float)t_walk.total_ms;
    h_out->ms_sgns = (float)t_sgns.total_ms;
    h_out->ms_prepare = (float)t_prep.total_ms;
    h_out->refused_ids = (int64_t)(refused_after - refused_before);
    EP_TRY(cudaEventElapsedTime(&h_out->ms_total, ev_begin, ev_end));

done:
    if (rc != GS_OK) {                       // let queued work drain before buffers are reused
        if (s_walk) cudaStreamSynchronize(s_walk);
        cudaStreamSynchronize(s_sgns);
    }
    t_walk.destroy();
    t_sgns.destroy();
    t_prep.destroy();
    for (int i = 0; i < 2; ++i) {
        if (ev_walk[i]) cudaEventDestroy(ev_walk[i]);
        if (ev_sgns[i]) cudaEventDestroy(ev_sgns[i]);
    }
    if (ev_begin) cudaEventDestroy(ev_begin);
    if (ev_end) cudaEventDestroy(ev_end);
    if (s_walk) cudaStreamDestroy(s_walk);
#undef EP_TRY
#undef EP_CALL
    return rc;
}

}  // extern "C"
