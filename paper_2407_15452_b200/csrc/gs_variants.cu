// Walk-corpus variants that sit between walk generation and the SGNS update:
// sub-sampling of frequent nodes (Mikolov et al. 2013, Section 2.3) and the
// keyed start-node shuffle.  Both are pure functions of (seed, walk id,
// position) like the rest of the path, so batching does not change them.
#include "gs_common.cuh"

namespace gs {

// One warp per walk.  Lane l looks at entries 32c + l of the walk, decides keep/drop, and the
// kept entries of a chunk are written behind those of the earlier chunks (ballot + prefix
// count).  The write position never passes the read position, and a chunk is read completely
// before it is written, so `out` may be the same buffer as `walks`.
__global__ void __launch_bounds__(256)
subsample_walks_kernel(const int32_t *walks, int64_t n_walks, int64_t walk_id_base, int32_t L,
                       const uint32_t *__restrict__ keep_thr, uint32_t n_nodes, uint64_t seed,
                       int32_t *out, unsigned long long *kept_out)
{
    const int lane = threadIdx.x & 31;
    const int64_t n_warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    unsigned long long kept_total = 0;
    for (int64_t a = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); a < n_walks;
         a += n_warps) {
        const uint64_t id = (uint64_t)(walk_id_base + a);
        const int32_t *W = walks + a * (int64_t)L;
        int32_t *O = out + a * (int64_t)L;
        int n = 0;
        for (int t0 = 0; t0 < L; t0 += 32) {
            const int t = t0 + lane;
            const int32_t v = t < L ? W[t] : -1;
            bool keep = (uint32_t)v < n_nodes;              // -1 and ids without a threshold are dropped
            if (keep) {
                const uint32_t thr = ld_random(reinterpret_cast<const int32_t *>(keep_thr) + v);
                if (thr != 0xFFFFFFFFu)
                    keep = draw(seed, id, (uint32_t)t, TAG_SUBSAMPLE, 0).x < thr;
            }
            const unsigned m = __ballot_sync(0xffffffffu, keep);
            __syncwarp();                                   // the chunk is read; now it may be overwritten
            if (keep) O[n + __popc(m & ((1u << lane) - 1u))] = v;
            n += __popc(m);
        }
        __syncwarp();
        for (int t = n + lane; t < L; t += 32) O[t] = -1;
        __syncwarp();
        kept_total += (unsigned long long)n;
    }
    if (lane == 0 && kept_out && kept_total) atomicAdd(kept_out, kept_total);
}

gs_status launch_subsample_walks(const int32_t *walks, int64_t n_walks, int64_t base, int32_t L,
                                 const uint32_t *keep_thr, int64_t n_nodes, uint64_t seed, int32_t *out,
                                 unsigned long long *kept, cudaStream_t st)
{
    if (n_walks == 0) return GS_OK;
    int64_t blocks = (n_walks + 7) / 8;
    const int64_t cap = (int64_t)sm_count() * 8 * 4;
    if (blocks > cap) blocks = cap;
    subsample_walks_kernel<<<(unsigned)blocks, 256, 0, st>>>(walks, n_walks, base, L, keep_thr,
                                                           (uint32_t)n_nodes, seed, out, kept);
    GS_CUDA_TRY(cudaGetLastError());
    return GS_OK;
}

// Four-round balanced Feistel network on 2k bits; the round function is word 0 of the Philox
// block (id = right half | epoch << 32, step = round, TAG_SHUFFLE) masked to k bits.
__device__ __forceinline__ uint64_t feistel4(uint64_t x, int k, uint64_t seed, uint32_t epoch)
{
    const uint64_t mask = (1ull << k) - 1ull;
    uint64_t left = x >> k, right = x & mask;
#pragma unroll
    for (uint32_t round = 0; round < 4; ++round) {
        const uint64_t f = (uint64_t)draw(seed, right | ((uint64_t)epoch << 32), round, TAG_SHUFFLE, 0).x & mask;
        const uint64_t nr = left ^ f;
        left = right;
        right = nr;
    }
    return (left << k) | right;
}

// One thread per walk id.  Values outside [0, n) go through the network again: a permutation
// of the 4^k values restricted this way is a permutation of [0, n), and since 4^k < 4n the
// expected number of passes is below 4.
__global__ void __launch_bounds__(256)
shuffled_starts_kernel(int64_t n_nodes, int k, uint64_t seed, uint32_t epoch, int64_t first,
                       int64_t count, int32_t *__restrict__ starts)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += stride) {
        uint64_t y = (uint64_t)((first + i) % n_nodes);
        do { y = feistel4(y, k, seed, epoch); } while (y >= (uint64_t)n_nodes);
        starts[i] = (int32_t)y;
    }
}

gs_status launch_shuffled_starts(int64_t n_nodes, uint64_t seed, uint32_t epoch, int64_t first,
                                 int64_t count, int32_t *starts, cudaStream_t st)
{
    if (count == 0) return GS_OK;
    int k = 1;
    while ((1ull << (2 * k)) < (uint64_t)n_nodes) ++k;
    int64_t blocks = (count + 255) / 256;
    const int64_t cap = (int64_t)sm_count() * 16;
    if (blocks > cap) blocks = cap;
    shuffled_starts_kernel<<<(unsigned)blocks, 256, 0, st>>>(n_nodes, k, seed, epoch, first, count, starts);
    GS_CUDA_TRY(cudaGetLastError());
    return GS_OK;
}

}  // namespace gs
