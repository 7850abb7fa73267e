// Graph validation, table initialisation, the two walk samplers and their optional indexes.
//
// Walks are chains of dependent random reads, so throughput comes from the number of walks in
// flight, not from per-walk parallelism: both samplers run one walk per THREAD.  The walk index
// makes a uniform transition one random 16-byte read; the node2vec sampler flattens rejection
// rounds and transitions into one loop and answers its neighbour test from a hashed edge set.
// The kernel that gives G lanes to a walk (speculative rejection rounds, first accepted round
// wins) serves odd walk lengths and unaligned outputs, and any walk when gs_tune_node2vec_group
// asks for it.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "gs_common.cuh"

namespace gs {

// ------------------------------------------------------------------ validation
struct CsrReport {
    unsigned long long bad_row;        // first row with broken offsets / column range
    unsigned long long unsorted_row;   // first row that is not strictly increasing
    unsigned long long max_degree;
    unsigned long long ends_bad;       // offsets[0] != 0 or offsets[n] != n_edges
};

template <typename OffT>
__global__ void __launch_bounds__(256)
validate_csr_kernel(const OffT *__restrict__ off, const int32_t *__restrict__ col,
                    int64_t n_nodes, int64_t n_edges, int check_sorted, CsrReport *rep)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    unsigned long long local_max = 0;
    for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < n_nodes; v += stride) {
        const int64_t o0 = (int64_t)off[v], o1 = (int64_t)off[v + 1];
        if (v == 0 && o0 != 0) atomicExch(&rep->ends_bad, 1ull);
        if (v == n_nodes - 1 && o1 != n_edges) atomicExch(&rep->ends_bad, 1ull);
        if (o0 < 0 || o1 < o0 || o1 > n_edges) {
            atomicMin(&rep->bad_row, (unsigned long long)v);
            continue;                                   // never index cols with a broken range
        }
        const unsigned long long deg = (unsigned long long)(o1 - o0);
        local_max = deg > local_max ? deg : local_max;
        int32_t last = -1;
        bool range_ok = true, sorted_ok = true;
        for (int64_t e = o0; e < o1; ++e) {
            const int32_t c = col[e];
            range_ok &= (c >= 0) && ((int64_t)c < n_nodes);
            sorted_ok &= c > last;
            last = c;
        }
        if (!range_ok) atomicMin(&rep->bad_row, (unsigned long long)v);
        if (check_sorted && !sorted_ok) atomicMin(&rep->unsorted_row, (unsigned long long)v);
    }
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(0xffffffffu, local_max, o);
        local_max = other > local_max ? other : local_max;
    }
    if ((threadIdx.x & 31) == 0 && local_max) atomicMax(&rep->max_degree, local_max);
}

gs_status validate_csr(const gs_graph *g, bool check_sorted, cudaStream_t st,
                       int64_t *bad_row, int64_t *unsorted_row, int64_t *max_degree, bool *ends_bad)
{
    void *ws = nullptr;
    gs_status s = workspace_get(WS_COUNTERS, 256, &ws);
    if (s != GS_OK) return s;
    CsrReport *rep = (CsrReport *)ws;
    CsrReport init = { ~0ull, ~0ull, 0ull, 0ull };
    GS_CUDA_TRY(cudaMemcpyAsync(rep, &init, sizeof(init), cudaMemcpyHostToDevice, st));
    if (g->n_nodes > 0) {
        const int threads = 256;
        int64_t blocks = (g->n_nodes + threads - 1) / threads;
        const int64_t cap = (int64_t)sm_count() * 64;
        if (blocks > cap) blocks = cap;
        if (g->offsets64)
            validate_csr_kernel<int64_t><<<(unsigned)blocks, threads, 0, st>>>(
                (const int64_t *)g->d_offsets, g->d_cols, g->n_nodes, g->n_edges, check_sorted, rep);
        else
            validate_csr_kernel<int32_t><<<(unsigned)blocks, threads, 0, st>>>(
                (const int32_t *)g->d_offsets, g->d_cols, g->n_nodes, g->n_edges, check_sorted, rep);
        GS_CUDA_TRY(cudaGetLastError());
    }
    CsrReport h;
    GS_CUDA_TRY(cudaMemcpyAsync(&h, rep, sizeof(h), cudaMemcpyDeviceToHost, st));
    GS_CUDA_TRY(cudaStreamSynchronize(st));
    *bad_row = h.bad_row == ~0ull ? -1 : (int64_t)h.bad_row;
    *unsorted_row = h.unsorted_row == ~0ull ? -1 : (int64_t)h.unsorted_row;
    *max_degree = (int64_t)h.max_degree;
    *ends_bad = h.ends_bad != 0;
    return GS_OK;
}

// ------------------------------------------------------------------ table init
// Four start values of a row: (u - 0.5) / dim with u = (word >> 8) * 2^-24, stored in the table's
// type (16-bit formats: rounded to nearest even).
__device__ __forceinline__ void store_quad(float *w, int64_t x, float a, float b, float c, float d)
{
    reinterpret_cast<float4 *>(w)[x] = make_float4(a, b, c, d);
}
__device__ __forceinline__ void store_quad(__half *w, int64_t x, float a, float b, float c, float d)
{
    __half2 *p = reinterpret_cast<__half2 *>(w) + 2 * x;
    p[0] = __floats2half2_rn(a, b);
    p[1] = __floats2half2_rn(c, d);
}
__device__ __forceinline__ void store_quad(__nv_bfloat16 *w, int64_t x, float a, float b, float c, float d)
{
    __nv_bfloat162 *p = reinterpret_cast<__nv_bfloat162 *>(w) + 2 * x;
    p[0] = __floats2bfloat162_rn(a, b);
    p[1] = __floats2bfloat162_rn(c, d);
}

template <typename T>
__global__ void __launch_bounds__(256)
init_rows_kernel(T *__restrict__ w, int64_t n_rows, int32_t dim, uint64_t seed)
{
    const int32_t quads = dim >> 2;
    const int64_t total = n_rows * quads;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const float inv_d = 1.0f / (float)dim;             // dim is a power of two here: exact
    for (int64_t x = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; x < total; x += stride) {
        const int64_t row = x / quads;
        const uint32_t qd = (uint32_t)(x - row * quads);
        const uint4 r = draw(seed, (uint64_t)row, qd, TAG_INIT, 0);
        store_quad(w, x, ((float)(r.x >> 8) * (1.0f / 16777216.0f) - 0.5f) * inv_d,
                   ((float)(r.y >> 8) * (1.0f / 16777216.0f) - 0.5f) * inv_d,
                   ((float)(r.z >> 8) * (1.0f / 16777216.0f) - 0.5f) * inv_d,
                   ((float)(r.w >> 8) * (1.0f / 16777216.0f) - 0.5f) * inv_d);
    }
}

template <typename T>
static gs_status init_tables(T *w_in, T *w_out, int64_t n, int32_t dim, uint64_t seed, cudaStream_t st)
{
    if (w_in && n > 0) {
        const int64_t total = n * (dim >> 2);
        int64_t blocks = (total + 255) / 256;
        const int64_t cap = (int64_t)sm_count() * 32;
        if (blocks > cap) blocks = cap;
        init_rows_kernel<T><<<(unsigned)blocks, 256, 0, st>>>(w_in, n, dim, seed);
        GS_CUDA_TRY(cudaGetLastError());
    }
    if (w_out && n > 0)
        GS_CUDA_TRY(cudaMemsetAsync(w_out, 0, sizeof(T) * (size_t)n * (size_t)dim, st));
    return GS_OK;
}

gs_status init_embeddings(float *w_in, float *w_out, int64_t n, int32_t dim, uint64_t seed,
                          cudaStream_t st)
{
    return init_tables<float>(w_in, w_out, n, dim, seed, st);
}

gs_status init_embeddings_f16(void *w_in, void *w_out, int64_t n, int32_t dim, uint64_t seed,
                              cudaStream_t st)
{
    return init_tables<__half>((__half *)w_in, (__half *)w_out, n, dim, seed, st);
}

gs_status init_embeddings_bf16(void *w_in, void *w_out, int64_t n, int32_t dim, uint64_t seed,
                               cudaStream_t st)
{
    return init_tables<__nv_bfloat16>((__nv_bfloat16 *)w_in, (__nv_bfloat16 *)w_out, n, dim, seed, st);
}

// ------------------------------------------------------------------ uniform walks
// One walk per thread.  Per transition: two adjacent offsets, one Philox block,
// one column read, one 4-byte store into the walk-major output.
template <typename OffT>
__global__ void __launch_bounds__(256)
uniform_walk_kernel(const OffT *__restrict__ off, const int32_t *__restrict__ col,
                    const int32_t *__restrict__ starts, int64_t n_nodes, int64_t n_walks,
                    int64_t walk_id_base, int32_t L, uint64_t seed,
                    int32_t *__restrict__ walks, unsigned long long *steps_out,
                    unsigned long long *refused_out)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    unsigned int my_steps = 0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_walks; i += stride) {
        const uint64_t id = (uint64_t)(walk_id_base + i);
        int32_t cur = starts ? __ldg(starts + i) : (int32_t)(id % (uint64_t)n_nodes);
        const bool bad = (uint64_t)(uint32_t)cur >= (uint64_t)n_nodes;   // start outside the graph: empty walk
        if (bad && refused_out) atomicAdd(refused_out, 1ull);
        int32_t *W = walks + i * (int64_t)L;
        W[0] = bad ? -1 : cur;
        int32_t t = 0;
        for (; !bad && t + 1 < L; ++t) {
            const int64_t o0 = ld_random(off + cur), o1 = ld_random(off + cur + 1);
            const uint32_t deg = (uint32_t)(o1 - o0);
            if (deg == 0) break;
            const uint4 r = draw(seed, id, (uint32_t)t, TAG_UNIFORM, 0);
            cur = ld_random(col + o0 + (int64_t)__umulhi(r.x, deg));
            W[t + 1] = cur;
            ++my_steps;
        }
        for (int32_t s = t + 1; s < L; ++s) W[s] = -1;
    }
    if (steps_out) {
        for (int o = 16; o > 0; o >>= 1) my_steps += __shfl_xor_sync(0xffffffffu, my_steps, o);
        if ((threadIdx.x & 31) == 0 && my_steps) atomicAdd(steps_out, (unsigned long long)my_steps);
    }
}

// Same walks, stored 32 bytes at a time: entries are collected four per int4 and two int4
// leave together, so the output reaches L2 as whole sectors instead of 4-byte fragments
// (fragments that are evicted before their sector is complete cost a DRAM read to fill and a
// second write).  Needs L % 4 == 0 and a 16-byte aligned output.
template <typename OffT>
__global__ void __launch_bounds__(256, 6)
uniform_walk_vec_kernel(const OffT *__restrict__ off, const int32_t *__restrict__ col,
                        const int32_t *__restrict__ starts, int64_t n_nodes, int64_t n_walks,
                        int64_t walk_id_base, int32_t L, uint64_t seed,
                        int32_t *__restrict__ walks, unsigned long long *steps_out,
                    unsigned long long *refused_out)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int quads = L >> 2;
    unsigned int my_steps = 0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_walks; i += stride) {
        const uint64_t id = (uint64_t)(walk_id_base + i);
        int32_t cur = starts ? __ldg(starts + i) : (int32_t)(id % (uint64_t)n_nodes);
        bool alive = (uint64_t)(uint32_t)cur < (uint64_t)n_nodes;        // start outside the graph: empty walk
        if (!alive && refused_out) atomicAdd(refused_out, 1ull);
        int4 *W4 = reinterpret_cast<int4 *>(walks + i * (int64_t)L);
        int4 pend = make_int4(0, 0, 0, 0);
        for (int q = 0; q < quads; ++q) {
            int32_t v[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int e = 4 * q + k;                 // entry index; entry 0 is the start node
                if (e > 0 && alive) {
                    const int64_t o0 = ld_random(off + cur), o1 = ld_random(off + cur + 1);
                    const uint32_t deg = (uint32_t)(o1 - o0);
                    if (deg == 0) {
                        alive = false;
                    } else {
                        const uint4 r = draw(seed, id, (uint32_t)(e - 1), TAG_UNIFORM, 0);
                        cur = ld_random(col + o0 + (int64_t)__umulhi(r.x, deg));
                        ++my_steps;
                    }
                }
                v[k] = alive ? cur : -1;
            }
            const int4 now = make_int4(v[0], v[1], v[2], v[3]);
            if (q & 1) { W4[q - 1] = pend; W4[q] = now; }
            else if (q == quads - 1) W4[q] = now;
            else pend = now;
        }
    }
    if (steps_out) {
        for (int o = 16; o > 0; o >>= 1) my_steps += __shfl_xor_sync(0xffffffffu, my_steps, o);
        if ((threadIdx.x & 31) == 0 && my_steps) atomicAdd(steps_out, (unsigned long long)my_steps);
    }
}

// ------------------------------------------------------------------ walk index
// Record of CSR entry e: the neighbour c = cols[e] together with c's own degree and offset.
// With it a transition reads ONE random 16-byte record (pick a record in the current node's
// range; it already says where the next node's range is) instead of an offset pair and then a
// column: half the random DRAM accesses per transition, paid for with 16 bytes per entry.
template <typename OffT>
__global__ void __launch_bounds__(256)
build_walk_index_kernel(const OffT *__restrict__ off, const int32_t *__restrict__ col,
                        int64_t n_edges, int4 *__restrict__ rec)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n_edges; e += stride) {
        const int32_t c = col[e];
        const int64_t o0 = ld_random(off + c), o1 = ld_random(off + c + 1);
        rec[e] = make_int4(c, (int32_t)(uint32_t)(o1 - o0), (int32_t)(uint32_t)o0,
                           (int32_t)(uint32_t)((uint64_t)o0 >> 32));
    }
}

gs_status build_walk_index(const gs_graph *g, int4 *rec, cudaStream_t st)
{
    if (g->n_edges == 0) return GS_OK;
    int64_t blocks = (g->n_edges + 255) / 256;
    const int64_t cap = (int64_t)sm_count() * 64;
    if (blocks > cap) blocks = cap;
    if (g->offsets64)
        build_walk_index_kernel<int64_t><<<(unsigned)blocks, 256, 0, st>>>(
            (const int64_t *)g->d_offsets, g->d_cols, g->n_edges, rec);
    else
        build_walk_index_kernel<int32_t><<<(unsigned)blocks, 256, 0, st>>>(
            (const int32_t *)g->d_offsets, g->d_cols, g->n_edges, rec);
    GS_CUDA_TRY(cudaGetLastError());
    return GS_OK;
}

// Uniform walks over the index: one record read per transition, sector-wide stores.
template <typename OffT>
__global__ void __launch_bounds__(256, 6)
uniform_walk_index_kernel(const OffT *__restrict__ off, const int4 *__restrict__ rec,
                          const int32_t *__restrict__ starts, int64_t n_nodes, int64_t n_walks,
                          int64_t walk_id_base, int32_t L, uint64_t seed,
                          int32_t *__restrict__ walks, unsigned long long *steps_out,
                    unsigned long long *refused_out)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int quads = L >> 2;
    unsigned int my_steps = 0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_walks; i += stride) {
        const uint64_t id = (uint64_t)(walk_id_base + i);
        int32_t cur = starts ? __ldg(starts + i) : (int32_t)(id % (uint64_t)n_nodes);
        bool alive = (uint64_t)(uint32_t)cur < (uint64_t)n_nodes;        // start outside the graph: empty walk
        if (!alive && refused_out) atomicAdd(refused_out, 1ull);
        int64_t o0 = 0;
        uint32_t deg = 0;
        if (alive) {
            o0 = ld_random(off + cur);
            deg = (uint32_t)((int64_t)ld_random(off + cur + 1) - o0);
        }
        int4 *W4 = reinterpret_cast<int4 *>(walks + i * (int64_t)L);
        int4 pend = make_int4(0, 0, 0, 0);
        for (int q = 0; q < quads; ++q) {
            int32_t v[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int e = 4 * q + k;
                if (e > 0 && alive) {
                    if (deg == 0) {
                        alive = false;
                    } else {
                        const uint4 r = draw(seed, id, (uint32_t)(e - 1), TAG_UNIFORM, 0);
                        const int4 x = ld_random(rec + o0 + (int64_t)__umulhi(r.x, deg));
                        cur = x.x;
                        deg = (uint32_t)x.y;
                        o0 = (int64_t)(((uint64_t)(uint32_t)x.w << 32) | (uint32_t)x.z);
                        ++my_steps;
                    }
                }
                v[k] = alive ? cur : -1;
            }
            const int4 now = make_int4(v[0], v[1], v[2], v[3]);
            if (q & 1) { W4[q - 1] = pend; W4[q] = now; }
            else if (q == quads - 1) W4[q] = now;
            else pend = now;
        }
    }
    if (steps_out) {
        for (int o = 16; o > 0; o >>= 1) my_steps += __shfl_xor_sync(0xffffffffu, my_steps, o);
        if ((threadIdx.x & 31) == 0 && my_steps) atomicAdd(steps_out, (unsigned long long)my_steps);
    }
}

gs_status launch_uniform_walks(const gs_graph *g, const int32_t *starts, int64_t n_walks,
                               int64_t base, int32_t L, uint64_t seed, int32_t *walks,
                               unsigned long long *steps, unsigned long long *refused, cudaStream_t st)
{
    if (n_walks == 0) return GS_OK;
    const int threads = 256;
    int64_t blocks = (n_walks + threads - 1) / threads;
    const int64_t cap = (int64_t)sm_count() * 8 * 16;
    if (blocks > cap) blocks = cap;
    const bool vec = (L % 4 == 0) && (((uintptr_t)walks & 15) == 0);
#define GS_UW(KERNEL, T)                                                                        \
    KERNEL<T><<<(unsigned)blocks, threads, 0, st>>>((const T *)g->d_offsets, g->d_cols, starts, \
                                                    g->n_nodes, n_walks, base, L, seed, walks, steps, \
                                                    refused)
    if (vec && g->d_edge_rec) {
        if (g->offsets64)
            uniform_walk_index_kernel<int64_t><<<(unsigned)blocks, threads, 0, st>>>(
                (const int64_t *)g->d_offsets, g->d_edge_rec, starts, g->n_nodes, n_walks, base, L,
                seed, walks, steps, refused);
        else
            uniform_walk_index_kernel<int32_t><<<(unsigned)blocks, threads, 0, st>>>(
                (const int32_t *)g->d_offsets, g->d_edge_rec, starts, g->n_nodes, n_walks, base, L,
                seed, walks, steps, refused);
    } else if (g->offsets64) { if (vec) GS_UW(uniform_walk_vec_kernel, int64_t); else GS_UW(uniform_walk_kernel, int64_t); }
    else { if (vec) GS_UW(uniform_walk_vec_kernel, int32_t); else GS_UW(uniform_walk_kernel, int32_t); }
#undef GS_UW
    GS_CUDA_TRY(cudaGetLastError());
    return GS_OK;
}

// ------------------------------------------------------------------ node2vec walks
struct N2VThresholds {
    unsigned long long t_prev, t_near, t_far;   // floor(weight / max weight * 2^32), <= 2^32
};

// x in cols[lo, hi) ?  (strictly increasing row, at most 32 halvings of a < 2^32 range)
__device__ __forceinline__ bool row_contains(const int32_t *__restrict__ col, int64_t lo,
                                             int64_t hi, int32_t x)
{
    const int64_t end = hi;
    while (lo < hi) {
        const int64_t mid = lo + ((hi - lo) >> 1);
        if (ld_random(col + mid) < x) lo = mid + 1; else hi = mid;
    }
    return lo < end && ld_random(col + lo) == x;
}

// ------------------------------------------------------------------ edge set
// "Is x a neighbour of prev" by binary search costs about log2(deg(prev)) dependent random reads,
// and the walk sampler is bound by the number of such reads.  The optional edge set answers it
// with one or two: every CSR entry (u, v) is stored as the key u << 32 | v in an open-addressing
// table (linear probing, at most half full, 8 bytes per slot, so the probes of one lookup fall in
// one 64-byte granule most of the time).  Built once per graph, read-only afterwards.
constexpr unsigned long long EDGE_EMPTY = 0xFFFFFFFFFFFFFFFFull;

__device__ __forceinline__ unsigned long long edge_mix(unsigned long long x)
{
    x ^= x >> 33; x *= 0xff51afd7ed558ccdull; x ^= x >> 33; x *= 0xc4ceb9fe1a85ec53ull; x ^= x >> 33;
    return x;
}

// One warp per row; lanes take the row's entries 32 at a time.
template <typename OffT>
__global__ void __launch_bounds__(256)
build_edge_hash_kernel(const OffT *__restrict__ off, const int32_t *__restrict__ col, int64_t n_nodes,
                       unsigned long long *table, unsigned long long mask)
{
    const int lane = threadIdx.x & 31;
    const int64_t n_warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    for (int64_t u = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); u < n_nodes; u += n_warps) {
        const int64_t b = (int64_t)off[u], e = (int64_t)off[u + 1];
        for (int64_t x = b + lane; x < e; x += 32) {
            const unsigned long long key = ((unsigned long long)u << 32) | (unsigned int)col[x];
            unsigned long long slot = edge_mix(key) & mask;
            for (unsigned long long n = 0; n <= mask; ++n) {          // the table is at most half full
                const unsigned long long old = atomicCAS(table + slot, EDGE_EMPTY, key);
                if (old == EDGE_EMPTY || old == key) break;
                slot = (slot + 1) & mask;
            }
        }
    }
}

__device__ __forceinline__ bool edge_set_contains(const unsigned long long *__restrict__ table,
                                                  unsigned long long mask, int32_t u, int32_t v)
{
    const unsigned long long key = ((unsigned long long)(unsigned int)u << 32) | (unsigned int)v;
    unsigned long long slot = edge_mix(key) & mask;
    for (unsigned long long n = 0; n <= mask; ++n) {
        const unsigned long long k = ld_random(reinterpret_cast<const uint64_t *>(table) + slot);
        if (k == key) return true;
        if (k == EDGE_EMPTY) return false;
        slot = (slot + 1) & mask;
    }
    return false;
}

gs_status build_edge_hash(const gs_graph *g, unsigned long long *table, unsigned long long mask,
                          cudaStream_t st)
{
    GS_CUDA_TRY(cudaMemsetAsync(table, 0xFF, sizeof(unsigned long long) * (size_t)(mask + 1), st));
    int64_t blocks = (g->n_nodes + 7) / 8;
    const int64_t cap = (int64_t)sm_count() * 64;
    if (blocks > cap) blocks = cap;
    if (g->offsets64)
        build_edge_hash_kernel<int64_t><<<(unsigned)blocks, 256, 0, st>>>(
            (const int64_t *)g->d_offsets, g->d_cols, g->n_nodes, table, mask);
    else
        build_edge_hash_kernel<int32_t><<<(unsigned)blocks, 256, 0, st>>>(
            (const int32_t *)g->d_offsets, g->d_cols, g->n_nodes, table, mask);
    GS_CUDA_TRY(cudaGetLastError());
    return GS_OK;
}

// G lanes per walk; lane k of a group evaluates rejection round base + k.
template <typename OffT, int G>
__global__ void __launch_bounds__(256)
node2vec_walk_kernel(const OffT *__restrict__ off, const int32_t *__restrict__ col,
                     const int32_t *__restrict__ starts, int64_t n_nodes, int64_t n_walks,
                     int64_t walk_id_base, int32_t L, uint64_t seed, N2VThresholds T,
                     int32_t max_rounds, int32_t *__restrict__ walks,
                     unsigned long long *steps_out, unsigned long long *caps_out,
                     unsigned long long *refused_out)
{
    const int lane = threadIdx.x & 31;
    const int sub = lane % G;                       // round offset inside the group
    const unsigned gmask = (G == 32) ? 0xffffffffu : (((1u << G) - 1u) << (lane - sub));
    const int64_t groups_per_grid = (int64_t)gridDim.x * (blockDim.x / G);
    const unsigned long long t_lo = T.t_near < T.t_far ? T.t_near : T.t_far;
    const unsigned long long t_hi = T.t_near < T.t_far ? T.t_far : T.t_near;
    unsigned int my_steps = 0, my_caps = 0;

    // n_walks is rounded up per warp so that every lane of a warp runs the same number of
    // outer iterations (the group ballots below need their whole group present).
    for (int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G; i < n_walks;
         i += groups_per_grid) {
        const uint64_t id = (uint64_t)(walk_id_base + i);
        int32_t cur = starts ? __ldg(starts + i) : (int32_t)(id % (uint64_t)n_nodes);
        int32_t prev = -1;
        int64_t p0 = 0, p1 = 0;                     // adjacency range of prev
        int32_t *W = walks + i * (int64_t)L;
        const bool bad = (uint64_t)(uint32_t)cur >= (uint64_t)n_nodes;   // same for the whole group
        if (sub == 0 && bad && refused_out) atomicAdd(refused_out, 1ull);
        if (sub == 0) W[0] = bad ? -1 : cur;
        int32_t t = 0;
        for (; !bad && t + 1 < L; ++t) {
            const int64_t o0 = ld_random(off + cur), o1 = ld_random(off + cur + 1);
            const uint32_t deg = (uint32_t)(o1 - o0);
            if (deg == 0) break;
            int32_t nxt;
            if (t == 0) {
                const uint4 r = draw(seed, id, 0u, TAG_NODE2VEC, 0);
                nxt = ld_random(col + o0 + (int64_t)__umulhi(r.x, deg));
            } else {
                nxt = -1;
                for (int32_t rbase = 0;; rbase += G) {
                    const int32_t s = rbase + sub;
                    const bool live = s < max_rounds;
                    int32_t x = -1;
                    bool acc = false;
                    if (live) {
                        const uint4 r = draw(seed, id, (uint32_t)t, TAG_NODE2VEC, (uint32_t)s);
                        x = ld_random(col + o0 + (int64_t)__umulhi(r.x, deg));
                        const unsigned long long r1 = r.y;
                        if (x == prev) acc = r1 < T.t_prev;
                        else if (r1 < t_lo) acc = true;          // accepted in either class
                        else if (r1 >= t_hi) acc = false;        // rejected in either class
                        else acc = r1 < (row_contains(col, p0, p1, x) ? T.t_near : T.t_far);
                    }
                    const unsigned votes = __ballot_sync(gmask, acc) & gmask;
                    if (votes) {
                        nxt = __shfl_sync(gmask, x, __ffs(votes) - 1);
                        break;
                    }
                    if (rbase + G >= max_rounds) {               // cap: keep the last proposal
                        const int last_lane = (lane - sub) + (max_rounds - 1 - rbase);
                        nxt = __shfl_sync(gmask, x, last_lane);
                        if (sub == 0) ++my_caps;
                        break;
                    }
                }
            }
            prev = cur; p0 = o0; p1 = o1;
            cur = nxt;
            if (sub == 0) { W[t + 1] = cur; ++my_steps; }
        }
        if (sub == 0)
            for (int32_t s = t + 1; s < L; ++s) W[s] = -1;
    }
    if (steps_out && my_steps) atomicAdd(steps_out, (unsigned long long)my_steps);
    if (caps_out && my_caps) atomicAdd(caps_out, (unsigned long long)my_caps);
}

// One walk per thread (walks in flight matter more than lanes per walk), with the rejection rounds
// and the transitions of a walk flattened into ONE loop: every trip of the loop is one round of
// whatever transition the lane is at.  With nested loops a lane that has accepted waits until the
// slowest lane of its warp has (the number of rounds is geometric, so the slowest of 32 needs
// about three times the mean); here it starts its next transition at once, and the memory system
// sees a request from every lane on every trip.  The state carries the adjacency range of the
// current and of the previous node, so a round costs one random read (the proposal) plus, when
// the draw falls between the two class thresholds, one membership test of adj(prev).  With the
// walk index the proposal's record already holds the next node's range.  Finished entries
// collect in shared memory, eight per thread, and leave as two 16-byte stores.  Needs
// L % 4 == 0 and a 16-byte aligned output.
template <typename OffT, bool INDEX, bool HASH>
__global__ void __launch_bounds__(256, 4)
node2vec_flat_kernel(const OffT *__restrict__ off, const int32_t *__restrict__ col,
                     const int4 *__restrict__ rec, const unsigned long long *__restrict__ edge_set,
                     unsigned long long edge_mask, const int32_t *__restrict__ starts,
                     int64_t n_nodes, int64_t n_walks, int64_t walk_id_base, int32_t L,
                     uint64_t seed, N2VThresholds T, int32_t max_rounds,
                     int32_t *__restrict__ walks, unsigned long long *steps_out,
                     unsigned long long *caps_out, unsigned long long *refused_out)
{
    __shared__ int32_t buf[8][256];                        // buf[j][thread]: conflict-free
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const unsigned long long t_lo = T.t_near < T.t_far ? T.t_near : T.t_far;
    const unsigned long long t_hi = T.t_near < T.t_far ? T.t_far : T.t_near;
    const int tx = threadIdx.x;
    unsigned int my_steps = 0, my_caps = 0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_walks; i += stride) {
        const uint64_t id = (uint64_t)(walk_id_base + i);
        int32_t cur = starts ? __ldg(starts + i) : (int32_t)(id % (uint64_t)n_nodes);
        bool alive = (uint64_t)(uint32_t)cur < (uint64_t)n_nodes;        // start outside the graph: empty walk
        if (!alive && refused_out) atomicAdd(refused_out, 1ull);
        int64_t o0 = 0;
        uint32_t deg = 0;
        if (alive) {
            o0 = ld_random(off + cur);
            deg = (uint32_t)((int64_t)ld_random(off + cur + 1) - o0);
        }
        int32_t prev = -1;
        int64_t p0 = 0, p1 = 0;
        int4 *W4 = reinterpret_cast<int4 *>(walks + i * (int64_t)L);
        buf[0][tx] = alive ? cur : -1;
        int32_t e = 1;                                     // next entry to produce
        int32_t sr = 0;                                    // rejection round of the transition into entry e
        while (e < L) {
            int32_t out = -1;                              // entry e once it is decided
            bool done = !alive || deg == 0;                // dead end: the rest of the walk is -1
            if (done) {
                alive = false;
            } else {
                const uint4 r = draw(seed, id, (uint32_t)(e - 1), TAG_NODE2VEC, (uint32_t)sr);
                const int64_t at = o0 + (int64_t)__umulhi(r.x, deg);
                int32_t x;
                uint32_t xdeg = 0;
                int64_t xoff = 0;
                if (INDEX) {
                    const int4 rc = ld_random(rec + at);
                    x = rc.x;
                    xdeg = (uint32_t)rc.y;
                    xoff = (int64_t)(((uint64_t)(uint32_t)rc.w << 32) | (uint32_t)rc.z);
                } else {
                    x = ld_random(col + at);
                }
                const unsigned long long r1 = r.y;
                bool acc;
                if (e == 1) acc = true;                    // first transition: uniform
                else if (x == prev) acc = r1 < T.t_prev;
                else if (r1 < t_lo) acc = true;
                else if (r1 >= t_hi) acc = false;
                else {
                    const bool near = HASH ? edge_set_contains(edge_set, edge_mask, prev, x)
                                           : row_contains(col, p0, p1, x);
                    acc = r1 < (near ? T.t_near : T.t_far);
                }
                const bool last = sr + 1 >= (e == 1 ? 1 : max_rounds);
                if (acc || last) {
                    if (!acc) ++my_caps;                   // cap reached: keep the last proposal
                    prev = cur; p0 = o0; p1 = o0 + deg;
                    cur = x;
                    if (INDEX) { o0 = xoff; deg = xdeg; }
                    else { o0 = ld_random(off + cur); deg = (uint32_t)((int64_t)ld_random(off + cur + 1) - o0); }
                    ++my_steps;
                    out = cur;
                    done = true;
                    sr = 0;
                } else {
                    ++sr;
                }
            }
            if (done) {
                buf[e & 7][tx] = out;
                ++e;
                if ((e & 7) == 0) {                        // entries [e - 8, e) are complete
                    W4[(e >> 2) - 2] = make_int4(buf[0][tx], buf[1][tx], buf[2][tx], buf[3][tx]);
                    W4[(e >> 2) - 1] = make_int4(buf[4][tx], buf[5][tx], buf[6][tx], buf[7][tx]);
                }
            }
        }
        if (L & 4)                                         // L = 8m + 4: the last four entries
            W4[(L >> 2) - 1] = make_int4(buf[0][tx], buf[1][tx], buf[2][tx], buf[3][tx]);
    }
    for (int o = 16; o > 0; o >>= 1) {
        my_steps += __shfl_xor_sync(0xffffffffu, my_steps, o);
        my_caps += __shfl_xor_sync(0xffffffffu, my_caps, o);
    }
    if ((threadIdx.x & 31) == 0) {
        if (steps_out && my_steps) atomicAdd(steps_out, (unsigned long long)my_steps);
        if (caps_out && my_caps) atomicAdd(caps_out, (unsigned long long)my_caps);
    }
}

void node2vec_thresholds(double p, double q, N2VThresholds *T)
{
    const double a[3] = { 1.0 / p, 1.0, 1.0 / q };
    double m = a[0];
    for (int c = 1; c < 3; ++c) m = a[c] > m ? a[c] : m;
    unsigned long long out[3];
    for (int c = 0; c < 3; ++c) {
        double v = floor(a[c] / m * 4294967296.0);
        if (v > 4294967296.0) v = 4294967296.0;
        out[c] = (unsigned long long)v;
    }
    T->t_prev = out[0]; T->t_near = out[1]; T->t_far = out[2];
}

template <typename OffT, int G>
static void launch_n2v(const gs_graph *g, const int32_t *starts, int64_t n_walks, int64_t base,
                       int32_t L, uint64_t seed, const N2VThresholds &T, int32_t max_rounds,
                       int32_t *walks, unsigned long long *steps, unsigned long long *caps,
                       unsigned long long *refused, cudaStream_t st)
{
    const int threads = 256;
    const int64_t per_block = threads / G;
    int64_t blocks = (n_walks + per_block - 1) / per_block;
    const int64_t cap = (int64_t)sm_count() * 8 * 16;
    if (blocks > cap) blocks = cap;
    node2vec_walk_kernel<OffT, G><<<(unsigned)blocks, threads, 0, st>>>(
        (const OffT *)g->d_offsets, g->d_cols, starts, g->n_nodes, n_walks, base, L, seed, T,
        max_rounds, walks, steps, caps, refused);
}

gs_status launch_node2vec_walks(const gs_graph *g, const int32_t *starts, int64_t n_walks,
                                int64_t base, int32_t L, uint64_t seed, double p, double q,
                                int32_t max_rounds, int group, int32_t *walks,
                                unsigned long long *steps, unsigned long long *caps,
                                unsigned long long *refused, cudaStream_t st)
{
    if (n_walks == 0) return GS_OK;
    N2VThresholds T;
    node2vec_thresholds(p, q, &T);
    if (group == 0 && L % 4 == 0 && (((uintptr_t)walks & 15) == 0)) {
        const int threads = 256;
        int64_t blocks = (n_walks + threads - 1) / threads;
        const int64_t cap = (int64_t)sm_count() * 8 * 16;
        if (blocks > cap) blocks = cap;
#define GS_N2T(T_, IDX, HSH)                                                                      \
        node2vec_flat_kernel<T_, IDX, HSH><<<(unsigned)blocks, threads, 0, st>>>(                   \
            (const T_ *)g->d_offsets, g->d_cols, g->d_edge_rec, g->d_edge_hash, g->hash_mask,      \
            starts, g->n_nodes, n_walks, base, L, seed, T, max_rounds, walks, steps, caps, refused)
#define GS_N2T_H(T_, IDX) do { if (g->d_edge_hash) GS_N2T(T_, IDX, true); else GS_N2T(T_, IDX, false); } while (0)
        if (g->offsets64) { if (g->d_edge_rec) GS_N2T_H(int64_t, true); else GS_N2T_H(int64_t, false); }
        else { if (g->d_edge_rec) GS_N2T_H(int32_t, true); else GS_N2T_H(int32_t, false); }
#undef GS_N2T_H
#undef GS_N2T
        GS_CUDA_TRY(cudaGetLastError());
        return GS_OK;
    }
    if (group == 0) group = 1;                 // odd walk length or unaligned output: generic kernel
#define GS_N2V(GG)                                                                              \
    do {                                                                                        \
        if (g->offsets64) launch_n2v<int64_t, GG>(g, starts, n_walks, base, L, seed, T,         \
                                                  max_rounds, walks, steps, caps, refused, st); \
        else launch_n2v<int32_t, GG>(g, starts, n_walks, base, L, seed, T, max_rounds, walks,   \
                                     steps, caps, refused, st);                                 \
    } while (0)
    switch (group) {
        case 1: GS_N2V(1); break;
        case 2: GS_N2V(2); break;
        case 8: GS_N2V(8); break;
        case 32: GS_N2V(32); break;
        default: GS_N2V(4); break;
    }
#undef GS_N2V
    GS_CUDA_TRY(cudaGetLastError());
    return GS_OK;
}

}  // namespace gs
