// Shared device/host helpers of the CUDA library: status plumbing, the Philox
// block function and the counter layout that gs.h documents.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "gs.h"

namespace gs {

// ---- error plumbing ------------------------------------------------------
void set_error(const char *fmt, ...);
gs_status cuda_fail(cudaError_t e, const char *what);

#define GS_CUDA_TRY(expr)                                              \
    do {                                                               \
        cudaError_t _e = (expr);                                       \
        if (_e != cudaSuccess) return ::gs::cuda_fail(_e, #expr);      \
    } while (0)

// ---- per-device scratch (grow-only, cached) --------------------------------
// Returns a 256-byte aligned scratch block of at least `bytes` for slot `slot`
// (independent blocks so that kernels on different streams do not share one).
gs_status workspace_get(int slot, size_t bytes, void **out);
enum { WS_WALKS0 = 0, WS_WALKS1 = 1, WS_SGNS = 2, WS_COUNTERS = 3, WS_STARTS = 4, WS_SGNS1 = 5, WS_SLOTS = 6 };

int sm_count();

// Device counter of the current device to which kernels add the ids they refused (start nodes,
// walk entries, alias cells outside [0, n_nodes)); nullptr if it cannot be had.  Lives in the
// WS_COUNTERS block (bytes 0..127: epoch counters, 128: walk ticket, 160: this counter).
unsigned long long *refused_counter();

// ---- graph handle --------------------------------------------------------------
}  // namespace gs

struct gs_graph {
    int64_t n_nodes;
    int64_t n_edges;
    const void *d_offsets;
    const int32_t *d_cols;
    int32_t offsets64;
    int32_t sorted;       // rows verified strictly increasing
    int64_t max_degree;   // -1 when not validated
    int device;
    int4 *d_edge_rec;     // optional walk index, library-owned: {neighbour, its degree, its offset}
    unsigned long long *d_edge_hash;   // optional edge set, library-owned: open-addressing table of
    unsigned long long hash_mask;      // keys (row << 32 | column), capacity hash_mask + 1 (power of two)
};

namespace gs {

// ---- Philox4x32-10 ---------------------------------------------------------------
enum : uint32_t { TAG_UNIFORM = 1, TAG_NODE2VEC = 2, TAG_NEGATIVE = 3, TAG_INIT = 4,
                  TAG_WINDOW = 5, TAG_SUBSAMPLE = 6, TAG_SHUFFLE = 7, TAG_ROUND_SYNC = 8,
                  TAG_ROUND_LOCKFREE = 9 };

__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c.x);
        const uint32_t lo0 = 0xD2511F53u * c.x;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z);
        const uint32_t lo1 = 0xCD9E8D57u * c.z;
        c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
        k.x += 0x9E3779B9u;
        k.y += 0xBB67AE85u;
    }
    return c;
}

// counter = (id low, id high, step, tag << 24 | sub), key = seed
__device__ __forceinline__ uint4 draw(uint64_t seed, uint64_t id, uint32_t step,
                                      uint32_t tag, uint32_t sub)
{
    return philox4x32_10(make_uint4((uint32_t)id, (uint32_t)(id >> 32), step, (tag << 24) | sub),
                         make_uint2((uint32_t)seed, (uint32_t)(seed >> 32)));
}

// Read-only loads for isolated random accesses (a CSR offset, a column, an alias cell).
// By default a miss pulls a whole 128-byte line out of DRAM; the 64-byte prefetch-size hint
// halves that for data whose neighbours will not be used.  The line still allocates in L1, so
// the second offset of a pair hits there.
__device__ __forceinline__ int32_t ld_random(const int32_t *p)
{
    int32_t v;
    asm("ld.global.nc.L2::64B.s32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ int64_t ld_random(const int64_t *p)
{
    long long v;
    asm("ld.global.nc.L2::64B.s64 %0, [%1];" : "=l"(v) : "l"(p));
    return (int64_t)v;
}
__device__ __forceinline__ int4 ld_random(const int4 *p)
{
    int4 v;
    asm("ld.global.nc.L2::64B.v4.s32 {%0, %1, %2, %3}, [%4];"
        : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ uint64_t ld_random(const uint64_t *p)
{
    unsigned long long v;
    asm("ld.global.nc.L2::64B.u64 %0, [%1];" : "=l"(v) : "l"(p));
    return (uint64_t)v;
}

}  // namespace gs
