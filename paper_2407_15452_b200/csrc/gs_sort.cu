// Stable least-significant-digit radix sort of (key, value) pairs, at most 8 bits per
// pass.  It groups the gradient contributions of a synchronous SGNS step by
// destination row while keeping contributions of one row in index order, which
// is what makes the summation order (and so the result bits) fixed.
//
// Per pass: (1) per-tile digit histograms, (2) per digit an exclusive scan over
// the tiles (256 blocks) plus the digit totals, (3) a scatter in which each warp ranks its
// items round by round with match_any, so that equal digits keep their order.
#include "gs_common.cuh"

namespace gs {

constexpr int SORT_THREADS = 256;
constexpr int SORT_ITEMS = 8;
constexpr int SORT_TILE = SORT_THREADS * SORT_ITEMS;   // 2048 keys per block
constexpr int RADIX = 256;

__global__ void __launch_bounds__(SORT_THREADS)
sort_hist_kernel(const uint32_t *__restrict__ keys, uint32_t n, int shift, uint32_t mask,
                 uint32_t n_tiles, uint32_t *__restrict__ counts)
{
    __shared__ uint32_t h[RADIX];
    h[threadIdx.x] = 0;
    __syncthreads();
    const uint32_t base = blockIdx.x * SORT_TILE;
#pragma unroll
    for (int r = 0; r < SORT_ITEMS; ++r) {
        const uint32_t i = base + r * SORT_THREADS + threadIdx.x;
        if (i < n) atomicAdd(&h[(keys[i] >> shift) & mask], 1u);
    }
    __syncthreads();
    counts[threadIdx.x * n_tiles + blockIdx.x] = h[threadIdx.x];
}

// Block d turns the per-tile counts of digit d into exclusive prefixes over the tiles and
// leaves the digit's total in totals[d].  (The prefix over digits is taken by the scatter
// kernel itself, from the 256 totals.)
__global__ void __launch_bounds__(256)
sort_scan_kernel(uint32_t *__restrict__ counts, uint32_t n_tiles, uint32_t *__restrict__ totals)
{
    __shared__ uint32_t warp_sum[8];
    __shared__ uint32_t carry_s;
    uint32_t *c = counts + (size_t)blockIdx.x * n_tiles;
    const int lane = threadIdx.x & 31, wi = threadIdx.x >> 5;
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    for (uint32_t base = 0; base < n_tiles; base += 256) {
        const uint32_t i = base + threadIdx.x;
        const uint32_t v = i < n_tiles ? c[i] : 0u;
        uint32_t incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31) warp_sum[wi] = incl;
        __syncthreads();
        uint32_t before = carry_s;
        for (int k = 0; k < wi; ++k) before += warp_sum[k];
        if (i < n_tiles) c[i] = before + incl - v;
        __syncthreads();
        if (threadIdx.x == 255) carry_s = before + incl;
        __syncthreads();
    }
    if (threadIdx.x == 0) totals[blockIdx.x] = carry_s;
}

template <bool IOTA>
__global__ void __launch_bounds__(SORT_THREADS)
sort_scatter_kernel(const uint32_t *__restrict__ keys_in, const uint32_t *__restrict__ vals_in,
                    uint32_t *__restrict__ keys_out, uint32_t *__restrict__ vals_out, uint32_t n,
                    int shift, uint32_t mask, uint32_t n_tiles, const uint32_t *__restrict__ offsets,
                    const uint32_t *__restrict__ totals)
{
    constexpr int WARPS = SORT_THREADS / 32;
    __shared__ uint32_t cnt[WARPS][RADIX];
    __shared__ uint32_t digit_base[RADIX];
    {   // exclusive prefix of the 256 digit totals (thread d owns digit d)
        const uint32_t t = totals[threadIdx.x];
        uint32_t incl = t;
        const int ln = threadIdx.x & 31;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t u = __shfl_up_sync(0xffffffffu, incl, o);
            if (ln >= o) incl += u;
        }
        digit_base[threadIdx.x] = incl - t;                // prefix inside the warp's 32 digits
        if (ln == 31) cnt[0][threadIdx.x >> 5] = incl;     // warp totals, parked in cnt for a moment
        __syncthreads();
        uint32_t before = 0;
        for (int k = 0; k < (int)(threadIdx.x >> 5); ++k) before += cnt[0][k];
        __syncthreads();
        digit_base[threadIdx.x] += before;
    }
    const int lane = threadIdx.x & 31, wi = threadIdx.x >> 5;
    for (int x = threadIdx.x; x < WARPS * RADIX; x += SORT_THREADS) (&cnt[0][0])[x] = 0;
    __syncthreads();

    // warp wi owns the contiguous run [base, base + 32 * SORT_ITEMS), visited in index order
    const uint32_t base = blockIdx.x * SORT_TILE + wi * (32 * SORT_ITEMS);
    uint32_t key[SORT_ITEMS], val[SORT_ITEMS], loc[SORT_ITEMS];
#pragma unroll
    for (int r = 0; r < SORT_ITEMS; ++r) {
        const uint32_t i = base + r * 32 + lane;
        const bool ok = i < n;
        key[r] = ok ? keys_in[i] : 0u;
        val[r] = ok ? (IOTA ? i : vals_in[i]) : 0u;
        const uint32_t d = ok ? ((key[r] >> shift) & mask) : RADIX;   // RADIX = absent
        const unsigned peers = __match_any_sync(0xffffffffu, d);
        const int leader = __ffs(peers) - 1;
        uint32_t before = 0;
        if (ok && lane == leader) {
            before = cnt[wi][d];
            cnt[wi][d] = before + __popc(peers);
        }
        before = __shfl_sync(0xffffffffu, before, leader);
        loc[r] = before + __popc(peers & ((1u << lane) - 1u));
        __syncwarp();
    }
    __syncthreads();
    {   // digit threadIdx.x: turn per-warp counts into start positions in the output
        const int d = threadIdx.x;
        uint32_t run = digit_base[d] + offsets[d * n_tiles + blockIdx.x];
#pragma unroll
        for (int k = 0; k < WARPS; ++k) {
            const uint32_t c = cnt[k][d];
            cnt[k][d] = run;
            run += c;
        }
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < SORT_ITEMS; ++r) {
        const uint32_t i = base + r * 32 + lane;
        if (i < n) {
            const uint32_t dst = cnt[wi][(key[r] >> shift) & mask] + loc[r];
            keys_out[dst] = key[r];
            vals_out[dst] = val[r];
        }
    }
}

size_t sort_counts_bytes(uint32_t n)
{
    const uint32_t n_tiles = (n + SORT_TILE - 1) / SORT_TILE;
    return sizeof(uint32_t) * ((size_t)RADIX * (n_tiles ? n_tiles : 1) + RADIX);   // + digit totals
}

// Digit widths of the passes: ceil(bits / 8) passes of equal width (21-bit keys sort as 7 + 7 + 7,
// not 8 + 8 + 5: the same number of passes with a smaller scatter fan-out in each).
static int digit_width(int bits)
{
    const int passes = (bits + 7) / 8;
    return passes ? (bits + passes - 1) / passes : 8;
}

// Sorts n pairs by the low `bits` bits of the key.  The first pass reads keys_src, which is left
// untouched, and takes value i for item i (there is no input value array); the passes then
// alternate between buffers B and C.  On return *keys_sorted / *vals_sorted point at whichever of
// B / C holds the result.  Returns launches made.
int radix_sort_pairs(const uint32_t *keys_src, uint32_t *keysB, uint32_t *valsB, uint32_t *keysC,
                     uint32_t *valsC, uint32_t n, int bits, uint32_t *counts, cudaStream_t st,
                     uint32_t **keys_sorted, uint32_t **vals_sorted)
{
    const uint32_t n_tiles = (n + SORT_TILE - 1) / SORT_TILE;
    const uint32_t *kin = keys_src, *vin = nullptr;
    uint32_t *kout = keysB, *vout = valsB;
    uint32_t *totals = counts + (size_t)RADIX * (n_tiles ? n_tiles : 1);
    int launches = 0;
    bool first = true;
    if (bits < 1) bits = 1;                                  // at least one pass: the result lives in B
    const int width = digit_width(bits);
    for (int shift = 0; shift < bits && n > 0; shift += width) {
        const uint32_t mask = (1u << width) - 1u;
        sort_hist_kernel<<<n_tiles, SORT_THREADS, 0, st>>>(kin, n, shift, mask, n_tiles, counts);
        sort_scan_kernel<<<RADIX, 256, 0, st>>>(counts, n_tiles, totals);
        if (first)
            sort_scatter_kernel<true><<<n_tiles, SORT_THREADS, 0, st>>>(kin, vin, kout, vout, n,
                                                                        shift, mask, n_tiles, counts, totals);
        else
            sort_scatter_kernel<false><<<n_tiles, SORT_THREADS, 0, st>>>(kin, vin, kout, vout, n,
                                                                         shift, mask, n_tiles, counts, totals);
        launches += 3;
        kin = kout;
        vin = vout;
        kout = kout == keysB ? keysC : keysB;
        vout = vout == valsB ? valsC : valsB;
        first = false;
    }
    *keys_sorted = const_cast<uint32_t *>(kin);
    *vals_sorted = const_cast<uint32_t *>(vin);
    return launches;
}

}  // namespace gs
