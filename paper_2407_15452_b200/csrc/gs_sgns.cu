// Skip-gram-with-negative-sampling update kernels.
//
// A row of an embedding table is dim fp32 values, always moved with 16-byte
// accesses: a whole warp holds one row of dim 256, half a warp one of dim 128,
// a quarter one of dim 64 or 32 (so one warp-wide access moves 1, 2 or 4 rows),
// and the lanes of a row read or write it as contiguous 16-byte pieces.  Dot products are
// butterfly shuffles.  The path is bound by row traffic in HBM/L2, not by
// arithmetic, so there is no tensor-core work here.
//
// Lock-free mode: one warp per walk, positions in order.  For each position
// the center row sits in registers, the targets of all its pairs (context +
// negatives, slot by slot) are listed in shared memory, and the list is
// consumed in chunks of TCH rows whose loads are all in flight together.
//
// Synchronous mode, in two parts.  Part A needs no table: one warp per position lists
// the targets of its pairs and emits one (destination row, contribution index) key per
// target, and the keys are radix-sorted.  Part B reads the entry tables: one warp per
// position computes the coefficients g and the center-row gradient; then the sorted
// contributions are walked run by run, each run summed in index order and its row
// written once.  No result depends on the order in which anything executes: a sum is
// formed by one warp in a fixed order, and every value of a table receives exactly one
// addition per step.  Because part A does not touch the tables, the epoch driver runs
// it for batch b+1 on a second stream while batch b is in part B.
#include <mutex>
#include <type_traits>

#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "gs_common.cuh"

namespace gs {

int radix_sort_pairs(const uint32_t *keys_src, uint32_t *keysB, uint32_t *valsB, uint32_t *keysC,
                     uint32_t *valsC, uint32_t n, int bits, uint32_t *counts, cudaStream_t st,
                     uint32_t **keys_sorted, uint32_t **vals_sorted);
size_t sort_counts_bytes(uint32_t n);

constexpr int HOGWILD_PF_DIST = 2;   // chunks between a prefetch and the loads that use it
constexpr int TCH = 6;            // target rows in flight per row group (3 for half rows, see run_hogwild)
constexpr int SGNS_WARPS = 4;     // warps per block

// ---------------------------------------------------------------- row vectors
template <int FPL> struct Row { float v[FPL]; };

template <int FPL>
__device__ __forceinline__ Row<FPL> row_load(const float *__restrict__ tab, int64_t r, int lane)
{
    Row<FPL> out;
    const float *p = tab + r * (int64_t)(FPL * 32);
    if constexpr (FPL == 1) {
        out.v[0] = p[lane];
    } else if constexpr (FPL == 2) {
        const float2 t = reinterpret_cast<const float2 *>(p)[lane];
        out.v[0] = t.x; out.v[1] = t.y;
    } else {
#pragma unroll
        for (int q = 0; q < FPL / 4; ++q) {
            const float4 t = reinterpret_cast<const float4 *>(p)[q * 32 + lane];
            out.v[4 * q] = t.x; out.v[4 * q + 1] = t.y; out.v[4 * q + 2] = t.z; out.v[4 * q + 3] = t.w;
        }
    }
    return out;
}

template <int FPL>
__device__ __forceinline__ void row_store(float *__restrict__ tab, int64_t r, int lane,
                                          const Row<FPL> &x)
{
    float *p = tab + r * (int64_t)(FPL * 32);
    if constexpr (FPL == 1) {
        p[lane] = x.v[0];
    } else if constexpr (FPL == 2) {
        reinterpret_cast<float2 *>(p)[lane] = make_float2(x.v[0], x.v[1]);
    } else {
#pragma unroll
        for (int q = 0; q < FPL / 4; ++q)
            reinterpret_cast<float4 *>(p)[q * 32 + lane] =
                make_float4(x.v[4 * q], x.v[4 * q + 1], x.v[4 * q + 2], x.v[4 * q + 3]);
    }
}

// The same whole-warp row access for tables stored as IEEE half (arithmetic stays fp32).  A lane
// holds the same COLUMNS as in the fp32 layout above (4 consecutive columns per access q, at
// (q * 32 + lane) * 4), so fp32 scratch rows and half table rows can be combined lane by lane.
template <int FPL>
__device__ __forceinline__ Row<FPL> row_load(const __half *__restrict__ tab, int64_t r, int lane)
{
    Row<FPL> out;
    const __half *p = tab + r * (int64_t)(FPL * 32);
    if constexpr (FPL == 2) {
        const float2 f = __half22float2(reinterpret_cast<const __half2 *>(p)[lane]);
        out.v[0] = f.x; out.v[1] = f.y;
    } else {
        static_assert(FPL % 4 == 0, "half tables need dim 64, 128 or 256");
#pragma unroll
        for (int q = 0; q < FPL / 4; ++q) {
            const uint2 t = reinterpret_cast<const uint2 *>(p)[q * 32 + lane];
            const __half2 *h = reinterpret_cast<const __half2 *>(&t);
            const float2 a = __half22float2(h[0]), b = __half22float2(h[1]);
            out.v[4 * q] = a.x; out.v[4 * q + 1] = a.y; out.v[4 * q + 2] = b.x; out.v[4 * q + 3] = b.y;
        }
    }
    return out;
}

template <int FPL>
__device__ __forceinline__ void row_store(__half *__restrict__ tab, int64_t r, int lane, const Row<FPL> &x)
{
    __half *p = tab + r * (int64_t)(FPL * 32);
    if constexpr (FPL == 2) {
        reinterpret_cast<__half2 *>(p)[lane] = __floats2half2_rn(x.v[0], x.v[1]);
    } else {
#pragma unroll
        for (int q = 0; q < FPL / 4; ++q) {
            uint2 t;
            __half2 *h = reinterpret_cast<__half2 *>(&t);
            h[0] = __floats2half2_rn(x.v[4 * q], x.v[4 * q + 1]);
            h[1] = __floats2half2_rn(x.v[4 * q + 2], x.v[4 * q + 3]);
            reinterpret_cast<uint2 *>(p)[q * 32 + lane] = t;
        }
    }
}

// ... and for tables stored as bfloat16.
template <int FPL>
__device__ __forceinline__ Row<FPL> row_load(const __nv_bfloat16 *__restrict__ tab, int64_t r, int lane)
{
    Row<FPL> out;
    const __nv_bfloat16 *p = tab + r * (int64_t)(FPL * 32);
    if constexpr (FPL == 2) {
        const float2 f = __bfloat1622float2(reinterpret_cast<const __nv_bfloat162 *>(p)[lane]);
        out.v[0] = f.x; out.v[1] = f.y;
    } else {
        static_assert(FPL % 4 == 0, "bfloat16 tables need dim 64, 128 or 256");
#pragma unroll
        for (int q = 0; q < FPL / 4; ++q) {
            const uint2 t = reinterpret_cast<const uint2 *>(p)[q * 32 + lane];
            const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&t);
            const float2 a = __bfloat1622float2(h[0]), b = __bfloat1622float2(h[1]);
            out.v[4 * q] = a.x; out.v[4 * q + 1] = a.y; out.v[4 * q + 2] = b.x; out.v[4 * q + 3] = b.y;
        }
    }
    return out;
}

template <int FPL>
__device__ __forceinline__ void row_store(__nv_bfloat16 *__restrict__ tab, int64_t r, int lane, const Row<FPL> &x)
{
    __nv_bfloat16 *p = tab + r * (int64_t)(FPL * 32);
    if constexpr (FPL == 2) {
        reinterpret_cast<__nv_bfloat162 *>(p)[lane] = __floats2bfloat162_rn(x.v[0], x.v[1]);
    } else {
#pragma unroll
        for (int q = 0; q < FPL / 4; ++q) {
            uint2 t;
            __nv_bfloat162 *h = reinterpret_cast<__nv_bfloat162 *>(&t);
            h[0] = __floats2bfloat162_rn(x.v[4 * q], x.v[4 * q + 1]);
            h[1] = __floats2bfloat162_rn(x.v[4 * q + 2], x.v[4 * q + 3]);
            reinterpret_cast<uint2 *>(p)[q * 32 + lane] = t;
        }
    }
}

template <int FPL>
__device__ __forceinline__ float row_dot(const Row<FPL> &a, const Row<FPL> &b)
{
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < FPL; ++j) s = fmaf(a.v[j], b.v[j], s);
    return s;
}

__device__ __forceinline__ float warp_sum(float s)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    return s;                       // identical bits on every lane (commutative pairs)
}

// sigmoid(z) and softplus(z) = log(1 + e^z) from one exponential, stable for either sign
__device__ __forceinline__ void sigmoid_softplus(float z, float &sig, float &sp)
{
    const float e = expf(-fabsf(z));
    const float r = 1.0f / (1.0f + e);
    sig = z >= 0.f ? r : e * r;
    sp = fmaxf(z, 0.f) + log1pf(e);
}

__device__ __forceinline__ double warp_sum_double(double s)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    return s;
}

// ---------------------------------------------------------------- rows held by part of a warp
// For dim < 128 a full warp per row would move only 128 or 256 bytes per instruction, and the
// per-row instruction cost - not bytes - would set the pace.  There a row is held by LPR = 16
// or 8 lanes and one warp-wide access moves NG = 2 or 4 different rows.
// T is the storage type of the table (float, or IEEE half with fp32 arithmetic): a lane always
// moves 16 bytes per access, i.e. 4 floats or 8 halves.
template <int DIM, typename T = float, bool NARROW = false> struct RowGeom {
    static constexpr int PER16 = 16 / (int)sizeof(T);       // values per 16-byte access
    static constexpr int BYTES = DIM * (int)sizeof(T);
    // lanes per row: 16 bytes per lane for half tables and for fp32 rows of 128 bytes; fp32 rows
    // of 256 and 512 bytes give a lane 32 bytes (8 and 16 lanes per row, 4 and 2 rows per
    // warp-wide access), which halves the per-row instruction overhead: measured +5 % on the
    // dim-64 workload and +4 % / +10 % on the 50M-node / 1M-node dim-128 workloads.  16-bit rows
    // of 256 bytes run 2 to 10 % slower that way (16 values per lane cost resident warps).
    // NARROW keeps 16 bytes per lane for those rows too: with few targets per position (LINE: one
    // pair per walk) wide chunks stay half empty and the narrow layout is 20 % faster.
    static constexpr int LPR = !NARROW && sizeof(T) == 4 && (BYTES == 256 || BYTES == 512)
                                   ? BYTES / 32 : (BYTES / 16 >= 32 ? 32 : BYTES / 16);
    static constexpr int FPL = DIM / LPR;                   // values per lane
    static constexpr int NG = 32 / LPR;                     // rows per warp-wide access
};

__device__ __forceinline__ void unpack16(const uint4 &t, float *v)
{
    v[0] = __uint_as_float(t.x); v[1] = __uint_as_float(t.y);
    v[2] = __uint_as_float(t.z); v[3] = __uint_as_float(t.w);
}
__device__ __forceinline__ uint4 pack16(const float *v, const float *)
{
    return make_uint4(__float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]),
                      __float_as_uint(v[3]));
}
__device__ __forceinline__ void unpack16h(const uint4 &t, float *v)
{
    const __half2 *h = reinterpret_cast<const __half2 *>(&t);
#pragma unroll
    for (int j = 0; j < 4; ++j) { const float2 f = __half22float2(h[j]); v[2 * j] = f.x; v[2 * j + 1] = f.y; }
}
__device__ __forceinline__ void unpack16b(const uint4 &t, float *v)
{
    const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&t);
#pragma unroll
    for (int j = 0; j < 4; ++j) { const float2 f = __bfloat1622float2(h[j]); v[2 * j] = f.x; v[2 * j + 1] = f.y; }
}
__device__ __forceinline__ uint4 pack16(const float *v, const __nv_bfloat16 *)
{
    uint4 t;
    __nv_bfloat162 *h = reinterpret_cast<__nv_bfloat162 *>(&t);
#pragma unroll
    for (int j = 0; j < 4; ++j) h[j] = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);   // round to nearest even
    return t;
}
__device__ __forceinline__ uint4 pack16(const float *v, const __half *)
{
    uint4 t;
    __half2 *h = reinterpret_cast<__half2 *>(&t);
#pragma unroll
    for (int j = 0; j < 4; ++j) h[j] = __floats2half2_rn(v[2 * j], v[2 * j + 1]);   // round to nearest even
    return t;
}

// Lane `sub` of a row group holds, for access q, the PER16 columns starting at
// (q * LPR + sub) * PER16.
template <int DIM, typename T, bool NARROW = false>
__device__ __forceinline__ Row<RowGeom<DIM, T, NARROW>::FPL> grow_load(const T *__restrict__ tab, int64_t r, int sub)
{
    using G = RowGeom<DIM, T, NARROW>;
    Row<G::FPL> out;
    const uint4 *p = reinterpret_cast<const uint4 *>(tab + r * (int64_t)DIM);
#pragma unroll
    for (int q = 0; q < G::FPL / G::PER16; ++q) {
        const uint4 t = p[q * G::LPR + sub];
        if constexpr (sizeof(T) == 4) unpack16(t, out.v + G::PER16 * q);
        else if constexpr (std::is_same<T, __half>::value) unpack16h(t, out.v + G::PER16 * q);
        else unpack16b(t, out.v + G::PER16 * q);
    }
    return out;
}

template <int DIM, typename T, bool NARROW = false>
__device__ __forceinline__ void grow_store(T *__restrict__ tab, int64_t r, int sub,
                                           const Row<RowGeom<DIM, T, NARROW>::FPL> &x)
{
    using G = RowGeom<DIM, T, NARROW>;
    uint4 *p = reinterpret_cast<uint4 *>(tab + r * (int64_t)DIM);
#pragma unroll
    for (int q = 0; q < G::FPL / G::PER16; ++q)
        p[q * G::LPR + sub] = pack16(x.v + G::PER16 * q, (const T *)nullptr);
}

// ---------------------------------------------------------------- stochastic write-back (16-bit tables)
// A value is rounded to one of its two neighbours in the table's format, upwards (in magnitude)
// with probability (|x| - lo) / (hi - lo) taken to 16 bits: up iff the 16-bit dither is below
// floor(frac * 2^16).  Representable values never move; nothing becomes infinite (a magnitude
// beyond the largest finite value, or a step up from it, gives the largest finite value).
// Both formats use the same carry: with frac held as an integer in the low bits of a word whose upper
// bits are the neighbour towards zero, "dither < frac" is the carry of frac + (all ones - dither)
// into the upper bits, so one addition both decides and rounds (a carry into the exponent is the
// step to the next binade).  The value is clamped to the largest finite value first.
__device__ __forceinline__ uint32_t sr_bits(float x, uint32_t u16, const __nv_bfloat16 *)
{
    // bfloat16 is the upper half of the fp32 pattern: the dropped 16 bits ARE frac * 2^16
    const float big = __uint_as_float(0x7F7F0000u);                 // largest finite bfloat16
    const uint32_t bits = __float_as_uint(fminf(fmaxf(x, -big), big));
    return (bits + (u16 ^ 0xFFFFu)) >> 16;
}
__device__ __forceinline__ uint32_t sr_bits(float x, uint32_t u16, const __half *)
{
    const float ax = fminf(fabsf(x), 65504.0f);
    const uint32_t abits = __float_as_uint(ax);
    const uint32_t sign = (__float_as_uint(x) >> 16) & 0x8000u;
    // normal range of binary16 (|x| >= 2^-14): 13 fraction bits are dropped, so they are
    // frac * 2^13 and the dither's upper 13 bits decide; the upper bits, exponent re-biased, are the
    // neighbour towards zero
    const uint32_t h_normal = ((abits + ((u16 >> 3) ^ 0x1FFFu)) >> 13) - 0x1C000u;
    // below 2^-14 the spacing is 2^-24: |x| * 2^40, truncated, holds the neighbour in its upper
    // and frac * 2^16 in its lower 16 bits (the product is exact)
    const uint32_t fixed = __float2uint_rz(ax * 1099511627776.0f);
    const uint32_t h_small = (fixed + (u16 ^ 0xFFFFu)) >> 16;
    return sign | (abits >= 0x38800000u ? h_normal : h_small);
}

__device__ __forceinline__ uint32_t mix32(uint32_t h)
{
    h ^= h >> 16; h *= 0x85EBCA6Bu; h ^= h >> 13; h *= 0xC2B2AE35u; h ^= h >> 16;
    return h;
}

// Dithers of columns 2k (upper half of the result) and 2k + 1 (lower half) of a row-write event
// with Philox block ev; salt_term = 0x85EBCA77 * salt tells apart the rows that share an event.
__device__ __forceinline__ uint32_t dither_pair(const uint4 &ev, uint32_t salt_term, uint32_t k)
{
    const uint32_t sel = k & 3u;
    const uint32_t w = sel == 0 ? ev.x : sel == 1 ? ev.y : sel == 2 ? ev.z : ev.w;
    return mix32(w ^ (0x9E3779B9u * ((k >> 2) + 1u)) ^ salt_term);
}

// Two consecutive columns 2k, 2k + 1 rounded stochastically and packed (low half: column 2k).
template <typename T>
__device__ __forceinline__ uint32_t sr_pack2(float a, float b, const uint4 &ev, uint32_t salt_term, uint32_t k)
{
    const uint32_t h = dither_pair(ev, salt_term, k);
    return sr_bits(a, h >> 16, (const T *)nullptr) | (sr_bits(b, h & 0xFFFFu, (const T *)nullptr) << 16);
}

// grow_store with stochastic rounding (16-bit tables): lane `sub` holds, for access q, the 8
// columns from (q * LPR + sub) * 8.
template <int DIM, typename T, bool NARROW = false>
__device__ __forceinline__ void grow_store_sr(T *__restrict__ tab, int64_t r, int sub,
                                              const Row<RowGeom<DIM, T, NARROW>::FPL> &x, const uint4 &ev,
                                              uint32_t salt_term)
{
    using G = RowGeom<DIM, T, NARROW>;
    static_assert(sizeof(T) == 2, "stochastic write-back is for 16-bit tables");
    uint4 *p = reinterpret_cast<uint4 *>(tab + r * (int64_t)DIM);
#pragma unroll
    for (int q = 0; q < G::FPL / G::PER16; ++q) {
        const uint32_t k0 = (uint32_t)(q * G::LPR + sub) * 4u;     // first column pair of this access
        const float *v = x.v + G::PER16 * q;
        uint4 t;
        t.x = sr_pack2<T>(v[0], v[1], ev, salt_term, k0);
        t.y = sr_pack2<T>(v[2], v[3], ev, salt_term, k0 + 1);
        t.z = sr_pack2<T>(v[4], v[5], ev, salt_term, k0 + 2);
        t.w = sr_pack2<T>(v[6], v[7], ev, salt_term, k0 + 3);
        p[q * G::LPR + sub] = t;
    }
}

// row_store (whole warp per row) with stochastic rounding: lane holds, for piece q, the 4 columns
// from (q * 32 + lane) * 4 (FPL = 2: columns 2 lane and 2 lane + 1).
template <int FPL, typename T>
__device__ __forceinline__ void row_store_sr(T *__restrict__ tab, int64_t r, int lane, const Row<FPL> &x,
                                             const uint4 &ev)
{
    static_assert(sizeof(T) == 2, "stochastic write-back is for 16-bit tables");
    T *p = tab + r * (int64_t)(FPL * 32);
    if constexpr (FPL == 2) {
        reinterpret_cast<uint32_t *>(p)[lane] = sr_pack2<T>(x.v[0], x.v[1], ev, 0u, (uint32_t)lane);
    } else {
#pragma unroll
        for (int q = 0; q < FPL / 4; ++q) {
            const uint32_t k0 = (uint32_t)(q * 32 + lane) * 2u;
            uint2 t;
            t.x = sr_pack2<T>(x.v[4 * q], x.v[4 * q + 1], ev, 0u, k0);
            t.y = sr_pack2<T>(x.v[4 * q + 2], x.v[4 * q + 3], ev, 0u, k0 + 1);
            reinterpret_cast<uint2 *>(p)[q * 32 + lane] = t;
        }
    }
}

// row += x as reductions.  fp32 tables: 16 bytes of fp32 increments per instruction.  16-bit
// tables: the increment is rounded to the table's format (nearest even) and the reduction unit
// adds it there in that format (one more rounding), 16 bytes = 8 values per instruction.
__device__ __forceinline__ void red_add_16bytes(__half *p, const uint4 &v)
{
    asm volatile("red.global.add.noftz.v4.f16x2 [%0], {%1, %2, %3, %4};"
                 :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void red_add_16bytes(__nv_bfloat16 *p, const uint4 &v)
{
    asm volatile("red.global.add.noftz.v4.bf16x2 [%0], {%1, %2, %3, %4};"
                 :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
template <int DIM, bool NARROW, typename T>
__device__ __forceinline__ void grow_red_add(T *__restrict__ tab, int64_t r, int sub,
                                             const Row<RowGeom<DIM, T, NARROW>::FPL> &x)
{
    using G = RowGeom<DIM, T, NARROW>;
    if constexpr (sizeof(T) == 4) {
        float4 *p = reinterpret_cast<float4 *>(tab + r * (int64_t)DIM);
#pragma unroll
        for (int q = 0; q < G::FPL / 4; ++q)
            atomicAdd(p + q * G::LPR + sub,
                      make_float4(x.v[4 * q], x.v[4 * q + 1], x.v[4 * q + 2], x.v[4 * q + 3]));
    } else {
        T *p = tab + r * (int64_t)DIM;
#pragma unroll
        for (int q = 0; q < G::FPL / G::PER16; ++q)
            red_add_16bytes(p + (q * G::LPR + sub) * G::PER16, pack16(x.v + G::PER16 * q, (const T *)nullptr));
    }
}

// Sums of N values over the LPR lanes of a row group in about half the shuffles of N separate
// butterflies.  While more than one value is left, a step pairs the values up and a lane keeps,
// of each pair, the one its lane bit selects (odd index: bit set) and sends the other; a value
// without a partner is added the plain way.  In the end every lane holds the complete sum of ONE
// value, f[0]: lane `sub` that of value group_value<LPR, N>(sub).  Value k is complete on lane
// group_owner<LPR, N>(k) and on the lanes that differ from it in bits no pairing of k used.
template <int O, int CNT, int N>
__device__ __forceinline__ void group_reduce_step(float (&f)[N], int sub)
{
    if constexpr (O >= 1) {
        if constexpr (CNT > 1) {
            const bool up = (sub & O) != 0;
#pragma unroll
            for (int i = 0; i < CNT / 2; ++i) {
                const float send = up ? f[2 * i] : f[2 * i + 1];
                const float keep = up ? f[2 * i + 1] : f[2 * i];
                f[i] = keep + __shfl_xor_sync(0xffffffffu, send, O);
            }
            if constexpr ((CNT & 1) != 0)
                f[CNT / 2] = f[CNT - 1] + __shfl_xor_sync(0xffffffffu, f[CNT - 1], O);
        } else {
            f[0] += __shfl_xor_sync(0xffffffffu, f[0], O);
        }
        group_reduce_step<O / 2, (CNT + 1) / 2, N>(f, sub);
    }
}

template <int LPR, int N>
__device__ __forceinline__ float group_reduce(float (&f)[N], int sub)
{
    static_assert(N <= LPR, "a row group sums at most as many values as it has lanes");
    group_reduce_step<LPR / 2, N, N>(f, sub);
    return f[0];
}

// lane bits that the pairings on the way of value k used (mask) and their values on the lanes
// that end up with value k (owner)
template <int LPR, int N>
__host__ __device__ constexpr int group_owner(int k, bool want_mask = false)
{
    int own = 0, mask = 0, cnt = N, slot = k;
    for (int o = LPR / 2; o >= 1 && cnt > 1; o >>= 1) {
        if ((slot | 1) < cnt) {                      // this value has a partner at this step
            mask |= o;
            if (slot & 1) own |= o;
        }
        slot >>= 1;
        cnt = (cnt + 1) / 2;
    }
    return want_mask ? mask : own;
}

template <int LPR, int N>
__device__ __forceinline__ int group_value(int sub)
{
    int k = 0;
#pragma unroll
    for (int q = 1; q < N; ++q)
        if ((sub & group_owner<LPR, N>(q, true)) == group_owner<LPR, N>(q)) k = q;
    return k;
}

// add up the per-group copies of a row held by the NG = 32 / LPR groups of a warp
template <int LPR, int FPL>
__device__ __forceinline__ void sum_over_groups(Row<FPL> &x)
{
#pragma unroll
    for (int o = LPR; o < 32; o <<= 1) {
#pragma unroll
        for (int j = 0; j < FPL; ++j) x.v[j] += __shfl_xor_sync(0xffffffffu, x.v[j], o);
    }
}

__device__ __forceinline__ void prefetch_l2(const void *p)
{
    asm volatile("prefetch.global.L2 [%0];" :: "l"(p));
}

// ---------------------------------------------------------------- target list of one position
// Slot layout: tgt[s * (1 + K) + 0] = context of slot s with bit 31 set (TARGET_IS_CONTEXT; node ids
// stay below 2^31 - 1, so no entry collides with -1), tgt[s * (1 + K) + 1 + k] = negative k;
// -1 where the pair does not exist or the negative equals the context (masked).
// W points at the walk (global or shared), c = W[i] >= 0.  Returns, identical on every lane, the
// number of pairs in bits 0..7, the number of masked negatives in bits 8..19 and, from bit 20, the
// number of ids that were refused: walk entries other than -1 and alias cells that name no row
// of the tables (they are treated as absent).  dump_* (nullable) are this position's rows of the
// dump arrays.
// flags & PAIR_FWD keeps only contexts that come later in the walk (edge sampling of LINE);
// flags & PAIR_SHRINK draws the window of this position, w_i = 1 + mulhi(word, w) uniform on
// 1..w (word2vec's shrinking window), and keeps the contexts within w_i.  Slots and the keying
// of the negatives stay those of the full window.
enum { PAIR_FWD = 1, PAIR_SHRINK = 2 };
constexpr uint32_t TARGET_IS_CONTEXT = 0x80000000u;

__device__ __forceinline__ int build_targets(const int32_t *W, int32_t L, int32_t i, int32_t w,
                                             int32_t K, uint64_t seed, uint64_t id,
                                             const uint64_t *__restrict__ alias, uint32_t n_alias,
                                             int32_t c, int32_t *tgt, int lane,
                                             int32_t *dump_pairs, int32_t *dump_negs, int flags)
{
    const int S = 2 * w, T1 = 1 + K;
    const bool fwd = (flags & PAIR_FWD) != 0;
    int w_i = w;
    if (flags & PAIR_SHRINK) w_i = 1 + (int)__umulhi(draw(seed, id, (uint32_t)i, TAG_WINDOW, 0).x, (uint32_t)w);
    const int hp = K > 0 ? (K + 1) / 2 : 1;          // Philox blocks per slot (>= 1 work item)
    int pairs = 0, masked = 0, refused = 0;
    __syncwarp();                                    // earlier readers of tgt are done
    for (int it0 = 0; it0 < S * hp; it0 += 32) {
        const int it = it0 + lane;
        bool valid = false, hid0 = false, hid1 = false;
        int bad = 0;                                 // ids this lane refused
        if (it < S * hp) {
            const int s = it / hp, m = it - s * hp;
            const int j = i - w + s + (s >= w ? 1 : 0);
            const bool in_window = j - i <= w_i && i - j <= w_i && !(fwd && s < w);   // fwd: only j > i
            int32_t ctx = (j >= 0 && j < L && in_window) ? W[j] : -1;
            if ((uint32_t)ctx >= n_alias) {                // absent, or not a node of the tables
                if (ctx != -1 && m == 0) bad = 1;
                ctx = -1;
            }
            valid = ctx >= 0;
            if (m == 0) {
                tgt[s * T1] = valid ? (int32_t)((uint32_t)ctx | TARGET_IS_CONTEXT) : -1;
                if (dump_pairs) {
                    dump_pairs[2 * s] = valid ? c : -1;
                    dump_pairs[2 * s + 1] = ctx;
                }
            }
            if (K > 0) {
                int32_t n0 = -1, n1 = -1;
                const bool two = 2 * m + 1 < K;
                if (valid) {
                    const uint4 r = draw(seed, id, (uint32_t)(i * S + s), TAG_NEGATIVE, (uint32_t)m);
                    const uint32_t j0 = __umulhi(r.x, n_alias);
                    const uint64_t e0 = ld_random(alias + j0);
                    n0 = r.y < (uint32_t)e0 ? (int32_t)j0 : (int32_t)(e0 >> 32);
                    if ((uint32_t)n0 >= n_alias) { n0 = -1; ++bad; }   // a table entry that names no node
                    if (two) {
                        const uint32_t j1 = __umulhi(r.z, n_alias);
                        const uint64_t e1 = ld_random(alias + j1);
                        n1 = r.w < (uint32_t)e1 ? (int32_t)j1 : (int32_t)(e1 >> 32);
                        if ((uint32_t)n1 >= n_alias) { n1 = -1; ++bad; }
                    }
                }
                if (dump_negs) {
                    dump_negs[s * K + 2 * m] = n0;
                    if (two) dump_negs[s * K + 2 * m + 1] = n1;
                }
                hid0 = valid && n0 == ctx;
                hid1 = valid && two && n1 == ctx;
                tgt[s * T1 + 1 + 2 * m] = (n0 == ctx) ? -1 : n0;
                if (two) tgt[s * T1 + 2 + 2 * m] = (n1 == ctx) ? -1 : n1;
            }
            valid = valid && m == 0;
        }
        pairs += __popc(__ballot_sync(0xffffffffu, valid));
        masked += __popc(__ballot_sync(0xffffffffu, hid0)) + __popc(__ballot_sync(0xffffffffu, hid1));
        if (__any_sync(0xffffffffu, bad != 0)) {           // rare: a corrupt walk buffer or alias table
            for (int o = 16; o > 0; o >>= 1) bad += __shfl_xor_sync(0xffffffffu, bad, o);
            refused += bad;
        }
    }
    __syncwarp();
    return pairs | (masked << 8) | (refused << 20);
}

__device__ __forceinline__ void dump_empty_position(int32_t S, int32_t K, int lane,
                                                    int32_t *dump_pairs, int32_t *dump_negs)
{
    if (dump_pairs) for (int x = lane; x < 2 * S; x += 32) dump_pairs[x] = -1;
    if (dump_negs) for (int x = lane; x < S * K; x += 32) dump_negs[x] = -1;
}

// Closes the gaps of a target list in place, keeping the order: afterwards tgt[0 .. n) are the
// entries other than -1 (returned: n, identical on every lane).  orig (nullable) receives the
// index each kept entry had in the slot layout.
__device__ __forceinline__ int compact_targets(int32_t *tgt, int SL, int lane, int32_t *orig)
{
    const unsigned below = (1u << lane) - 1u;
    int n = 0;
    for (int x0 = 0; x0 < SL; x0 += 32) {
        const int x = x0 + lane;
        const int32_t v = x < SL ? tgt[x] : -1;
        // every lane has read its entry before any lane writes: the ballot needs all of them, and
        // the writes go to places at or below the ones just read
        const unsigned m = __ballot_sync(0xffffffffu, v != -1);
        if (v != -1) {
            const int at = n + __popc(m & below);
            tgt[at] = v;
            if (orig) orig[at] = x;
        }
        n += __popc(m);
    }
    __syncwarp();
    return n;
}

// ---------------------------------------------------------------- lock-free kernel
// walks covered by one ticket of the lock-free kernel (host and device agree on the buffer size)
__host__ __device__ __forceinline__ int hogwild_walks_per_ticket(int L) { return L <= 16 ? 32 / L : 1; }

template <int DIM, typename T, bool RED, int MINB, int TC, bool NARROW, bool SR = false>
__global__ void __launch_bounds__(SGNS_WARPS * 32, MINB)
sgns_hogwild_kernel(T *__restrict__ w_in, T *__restrict__ w_out,
                    const int32_t *__restrict__ walks, int64_t n_walks, int64_t walk_id_base,
                    int32_t L, int32_t w, int32_t K, const uint64_t *__restrict__ alias,
                    uint32_t n_alias, float lr, uint64_t seed, double *loss_out,
                    unsigned long long *pairs_out, int32_t *dump_pairs, int32_t *dump_negs,
                    unsigned long long *ticket, int fwd, unsigned long long *masked_out,
                    unsigned long long *refused_out)
{
    using G = RowGeom<DIM, T, NARROW>;
    constexpr int FPL = G::FPL, LPR = G::LPR, NG = G::NG;
    constexpr int CH = TC * NG;                          // targets per chunk
    // 16-bit tables: few bytes are in flight per warp (CH rows of 128 to 512 bytes), so the rows of
    // a later chunk are asked into L2 ahead of time, one 128-byte line per lane
    constexpr int LINES = G::BYTES >= 128 ? G::BYTES / 128 : 1;
    constexpr int PF_LINES = (sizeof(T) == 2 && CH * LINES <= 32) ? CH * LINES : 0;
    extern __shared__ int32_t smem[];
    const int lane = threadIdx.x & 31, wi = threadIdx.x >> 5;
    const int grp = lane / LPR, sub = lane % LPR;
    const int S = 2 * w, SL = S * (1 + K);
    // Walks differ in length (dead ends), so warps draw walks from a shared ticket counter
    // instead of taking a fixed share.  A ticket covers `wpt` consecutive walks: one for ordinary
    // walks, up to 16 when walks are short (LINE: two nodes), so that the round trips of the
    // ticket and of the walk entries are paid once per 32 entries and not once per pair.
    const int wpt = hogwild_walks_per_ticket(L);
    // of every chunk this lane evaluates target my_k of its group, list entry base + my_off; the
    // lanes that hold the same sum evaluate it too, and one of them (my_owner) counts its loss
    const int my_k = group_value<LPR, TC>(sub);
    const int my_off = my_k * NG + grp;
    const bool my_owner = sub == (sub & group_owner<LPR, TC>(my_k, true));
    int32_t *Wbuf = smem + wi * (wpt * L + (SR ? 2 : 1) * SL);   // SR: + the slot index of every list entry
    int32_t *tgt = Wbuf + wpt * L;
    double loss_acc = 0.0;
    unsigned long long pair_acc = 0, masked_acc = 0, refused_acc = 0;

    for (;;) {
        unsigned long long tk = 0;
        if (lane == 0) tk = atomicAdd(ticket, (unsigned long long)wpt);
        const int64_t a0 = (int64_t)__shfl_sync(0xffffffffu, tk, 0);
        if (a0 >= n_walks) break;
        const int nw = n_walks - a0 < wpt ? (int)(n_walks - a0) : wpt;
        __syncwarp();
        for (int x = lane; x < nw * L; x += 32) Wbuf[x] = walks[a0 * L + x];
        __syncwarp();
      for (int wq = 0; wq < nw; ++wq) {
        const int64_t a = a0 + wq;
        const int32_t *W = Wbuf + wq * L;
        const uint64_t id = (uint64_t)(walk_id_base + a);
        for (int32_t i = 0; i < L; ++i) {
            const int32_t c = W[i];
            int32_t *dp = dump_pairs ? dump_pairs + ((a * L + i) * S) * 2 : nullptr;
            int32_t *dn = dump_negs ? dump_negs + ((a * L + i) * S) * (int64_t)K : nullptr;
            if ((uint32_t)c >= n_alias) {                 // -1 or no such row
                if (c != -1) ++refused_acc;
                dump_empty_position(S, K, lane, dp, dn);
                continue;
            }
            const int packed = build_targets(W, L, i, w, K, seed, id, alias, n_alias, c, tgt, lane,
                                             dp, dn, fwd);
            const int pairs = packed & 0xFF;
            masked_acc += (unsigned long long)((packed >> 8) & 0xFFF);
            refused_acc += (unsigned long long)((unsigned)packed >> 20);
            if (pairs == 0) continue;
            pair_acc += (unsigned long long)pairs;
            // the list without its gaps: chunks are full but for the last one
            const int n_tgt = compact_targets(tgt, SL, lane, SR ? tgt + SL : nullptr);
            // stochastic write-back: the rows written while this position is worked on share one
            // Philox block; a target takes salt 1 + its index in the slot layout, the center row 0x10000
            uint4 ev = make_uint4(0u, 0u, 0u, 0u);
            if (SR) ev = draw(seed, id, (uint32_t)i, TAG_ROUND_LOCKFREE, 0);
            const Row<FPL> u = grow_load<DIM, T, NARROW>(w_in, c, sub);     // every group holds the center row
            Row<FPL> acc;                                        // this group's share of its gradient
#pragma unroll
            for (int j = 0; j < FPL; ++j) acc.v[j] = 0.f;
            // The loss term of a target is softplus(z) = max(z, 0) + log(1 + e^-|z|) with z = -f for
            // a context and f for a negative.  A lane adds up the first part and multiplies the
            // second parts (each in [1, 2]); the logarithm is taken once per position.
            float sp_lin = 0.f, sp_prod = 1.f;
            // the rows of a later chunk on their way into L2 while the ones before it are worked
            // on: lane l asks for line l of the chunk's CH rows
            auto prefetch_chunk = [&](int first) {
                const int e = first + lane / LINES;
                if (lane < PF_LINES && e < n_tgt) {
                    const int64_t idn = (int64_t)((uint32_t)tgt[e] & ~TARGET_IS_CONTEXT);
                    prefetch_l2((const char *)(w_out + idn * DIM) + (lane % LINES) * 128);
                }
            };
            if constexpr (PF_LINES > 0) {
#pragma unroll
                for (int d = 1; d < HOGWILD_PF_DIST; ++d) prefetch_chunk(d * CH);
            }
            for (int base = 0; base < n_tgt; base += CH) {
                // target k of group grp is list entry base + k * NG + grp (-1: past the end)
                int32_t ids[TC];
#pragma unroll
                for (int k = 0; k < TC; ++k) {
                    const int t = base + k * NG + grp;
                    ids[k] = t < n_tgt ? tgt[t] : -1;
                }
                Row<FPL> rows[TC];
                float f[TC];
#pragma unroll
                for (int k = 0; k < TC; ++k)
                    if (ids[k] != -1)
                        rows[k] = grow_load<DIM, T, NARROW>(w_out, (int64_t)((uint32_t)ids[k] & ~TARGET_IS_CONTEXT), sub);
                if constexpr (PF_LINES > 0) prefetch_chunk(base + HOGWILD_PF_DIST * CH);
#pragma unroll
                for (int k = 0; k < TC; ++k) f[k] = ids[k] != -1 ? row_dot<FPL>(u, rows[k]) : 0.f;
                // the dot products of the chunk, reduced together: this lane ends up with that of
                // target my_k of its group and evaluates its coefficient.  For a context
                // (label 1) g = sigmoid(f) - 1 = -sigmoid(-f), for a negative sigmoid(f).
                const float fs = group_reduce<LPR, TC>(f, sub);
                const int my_t = base + my_off;
                const int32_t my_e = my_t < n_tgt ? tgt[my_t] : -1;
                const bool ctx = my_e < 0;               // bit 31 (an absent entry's g is not used)
                const float z = ctx ? -fs : fs;
                const float e = __expf(-fabsf(z));
                const float r = __fdividef(1.0f, 1.0f + e);
                const float sig = z >= 0.f ? r : e * r;
                const float my_g = ctx ? -sig : sig;
                if (my_owner && my_e != -1) {
                    sp_lin += fmaxf(z, 0.f);
                    sp_prod *= 1.0f + e;
                }
#pragma unroll
                for (int k = 0; k < TC; ++k) {
                    const float g = __shfl_sync(0xffffffffu, my_g, grp * LPR + group_owner<LPR, TC>(k));
                    if (ids[k] != -1) {
                        const int64_t row = (int64_t)((uint32_t)ids[k] & ~TARGET_IS_CONTEXT);
                        const float step = -lr * g;
                        Row<FPL> delta;
#pragma unroll
                        for (int j = 0; j < FPL; ++j) {
                            acc.v[j] = fmaf(g, rows[k].v[j], acc.v[j]);
                            delta.v[j] = step * u.v[j];
                            rows[k].v[j] += delta.v[j];
                        }
                        if (RED) grow_red_add<DIM, NARROW>(w_out, row, sub, delta);
                        else if constexpr (SR)
                            grow_store_sr<DIM, T, NARROW>(w_out, row, sub, rows[k], ev,
                                                          0x85EBCA77u * (uint32_t)(tgt[SL + base + k * NG + grp] + 1));
                        else grow_store<DIM, T, NARROW>(w_out, row, sub, rows[k]);
                    }
                }
                if (sp_prod > 1e30f) { sp_lin += logf(sp_prod); sp_prod = 1.f; }
            }
            const float loss = sp_lin + logf(sp_prod);   // this lane's share of the position's loss
            // center row: add the accumulated increment to the row as it is now
            sum_over_groups<LPR, FPL>(acc);
            Row<FPL> delta;
#pragma unroll
            for (int j = 0; j < FPL; ++j) delta.v[j] = -lr * acc.v[j];
            if (RED) {
                if (grp == 0) grow_red_add<DIM, NARROW>(w_in, c, sub, delta);
            } else {
                Row<FPL> now = grow_load<DIM, T, NARROW>(w_in, c, sub);
#pragma unroll
                for (int j = 0; j < FPL; ++j) now.v[j] += delta.v[j];
                if constexpr (SR) {
                    if (grp == 0) grow_store_sr<DIM, T, NARROW>(w_in, c, sub, now, ev, 0x85EBCA77u * 0x10000u);
                } else if (grp == 0) grow_store<DIM, T, NARROW>(w_in, c, sub, now);
            }
            loss_acc += (double)loss;
        }
      }
    }
    loss_acc = warp_sum_double(loss_acc);
    if (lane == 0) {
        if (loss_out && pair_acc) atomicAdd(loss_out, loss_acc);
        if (pairs_out && pair_acc) atomicAdd(pairs_out, pair_acc);
        if (masked_out && masked_acc) atomicAdd(masked_out, masked_acc);
        if (refused_out && refused_acc) atomicAdd(refused_out, refused_acc);
    }
}

// ---------------------------------------------------------------- synchronous mode
// Part A: one warp per position, no table is read.  The targets of a position are written as a
// dense list - its contexts first, then its unmasked negatives, each in slot order - into a
// segment of SLP = 2^shift >= SL entries: keys[pos << shift + k] = destination row of w_out for
// k < n_all, `invalid` = 2 n_nodes behind them (*n_out counts the valid ones of the whole batch:
// that is where the center keys begin once sorted).  Per position: tinfo[pos] = n_ctx | n_all << 16,
// keys[n_slots + pos] = n_nodes + center (or `invalid` when the position forms no pair) and
// pairs_pos[pos] = pairs | masked negatives << 8 | refused ids << 20.  (A power-of-two stride
// turns "which position does contribution idx belong to" into a shift in the apply passes.)
__global__ void __launch_bounds__(SGNS_WARPS * 32)
sgns_targets_kernel(const int32_t *__restrict__ walks, int64_t n_pos, int64_t walk_id_base, int32_t L,
                    int32_t w, int32_t K, const uint64_t *__restrict__ alias, uint32_t n_alias,
                    uint32_t n_nodes, uint64_t seed, int32_t shift, uint32_t *__restrict__ keys,
                    uint32_t *__restrict__ tinfo, int32_t *__restrict__ pairs_pos,
                    uint32_t *__restrict__ n_out, int32_t *dump_pairs, int32_t *dump_negs, int fwd)
{
    extern __shared__ int32_t smem[];
    const int lane = threadIdx.x & 31, wi = threadIdx.x >> 5;
    const int S = 2 * w, T1 = 1 + K, SL = S * T1, SLP = 1 << shift;
    int32_t *tgt = smem + wi * SL;
    const uint32_t invalid = 2u * n_nodes;
    const int64_t n_slots = n_pos << shift;
    const int64_t n_warps = (int64_t)gridDim.x * SGNS_WARPS;
    const unsigned below = (1u << lane) - 1u;
    for (int64_t pos = (int64_t)blockIdx.x * SGNS_WARPS + wi; pos < n_pos; pos += n_warps) {
        const int64_t a = pos / L;
        const int32_t i = (int32_t)(pos - a * L);
        const int32_t *W = walks + a * L;
        const int32_t c = W[i];
        int32_t *dp = dump_pairs ? dump_pairs + (pos * S) * 2 : nullptr;
        int32_t *dn = dump_negs ? dump_negs + (pos * S) * (int64_t)K : nullptr;
        uint32_t *kp = keys + (pos << shift);
        int packed = 0;
        __syncwarp();
        if ((uint32_t)c < n_nodes) {                   // -1, or an id outside the tables: no pairs
            packed = build_targets(W, L, i, w, K, seed, (uint64_t)(walk_id_base + a), alias, n_alias,
                                   c, tgt, lane, dp, dn, fwd);
        } else {
            if (c != -1) packed = 1 << 20;             // one refused id
            dump_empty_position(S, K, lane, dp, dn);
        }
        int n_ctx = 0, n_all = 0;
        if ((packed & 0xFF) != 0) {
#pragma unroll 1
            for (int pass = 0; pass < 2; ++pass) {     // contexts, then negatives
                for (int x0 = 0; x0 < SL; x0 += 32) {
                    const int x = x0 + lane;
                    const int32_t v = x < SL ? tgt[x] : -1;
                    const bool take = v != -1 && ((v < 0) == (pass == 0));   // bit 31: a context
                    const unsigned m = __ballot_sync(0xffffffffu, take);
                    if (take) kp[n_all + __popc(m & below)] = (uint32_t)v & ~TARGET_IS_CONTEXT;
                    n_all += __popc(m);
                }
                if (pass == 0) n_ctx = n_all;
            }
        }
        for (int x = n_all + lane; x < SLP; x += 32) kp[x] = invalid;
        if (lane == 0) {
            keys[n_slots + pos] = n_ctx > 0 ? n_nodes + (uint32_t)c : invalid;
            tinfo[pos] = (uint32_t)n_ctx | ((uint32_t)n_all << 16);
            pairs_pos[pos] = packed;
            if (n_all) atomicAdd(n_out, (uint32_t)n_all);   // integer: the total does not depend on order
        }
    }
}

// row += x where nobody else adds to the row during this launch: one reduction per value, so the
// result does not depend on timing, and the row never has to travel to the SM.
template <int FPL>
__device__ __forceinline__ void row_red_add(float *__restrict__ tab, int64_t r, int lane, const Row<FPL> &x)
{
    float *p = tab + r * (int64_t)(FPL * 32);
    if constexpr (FPL == 1) {
        atomicAdd(p + lane, x.v[0]);
    } else if constexpr (FPL == 2) {
        atomicAdd(reinterpret_cast<float2 *>(p) + lane, make_float2(x.v[0], x.v[1]));
    } else {
#pragma unroll
        for (int q = 0; q < FPL / 4; ++q)
            atomicAdd(reinterpret_cast<float4 *>(p) + q * 32 + lane,
                      make_float4(x.v[4 * q], x.v[4 * q + 1], x.v[4 * q + 2], x.v[4 * q + 3]));
    }
}

// Part A, last launch: output rows that receive exactly ONE contribution in this batch (a run of
// length one in the sorted keys; half of the rows, a quarter of the contributions on a graph of
// 10^6 nodes).  No other contribution reads or changes such a row, so the coefficient pass, which
// has the center row in registers, can add its increment at once and the apply pass can skip it:
// single[idx] = 1 for the coefficient pass, and bit 31 of the sorted contribution index for the
// apply pass (indices stay below 2^30).
constexpr uint32_t SINGLE_RUN = 0x80000000u;
// The shortcut pays where most runs have one entry, i.e. where the tables have many more rows than
// a batch has list entries (measured with 1.3e6 entries per batch: 5 % slower at 1e6 rows, 9 % slower
// at 2e6, 13 % faster at 5e6, 14 % faster at 5e7); the step marks them from this ratio of rows
// per list entry on.
constexpr int64_t SINGLE_MIN_NODES_PER_ENTRY = 3;

__global__ void __launch_bounds__(256)
sgns_mark_single_kernel(const uint32_t *__restrict__ keys, uint32_t *__restrict__ vals, uint32_t n_keys,
                        uint32_t n_nodes, uint8_t *__restrict__ single)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < (int64_t)n_keys; i += stride) {
        const uint32_t key = keys[i];
        if (key >= n_nodes) continue;                    // a center key or an empty slot
        const bool alone = (i == 0 || keys[i - 1] != key) && (i + 1 >= (int64_t)n_keys || keys[i + 1] != key);
        const uint32_t idx = vals[i];
        single[idx] = alone ? 1 : 0;
        if (alone) vals[i] = idx | SINGLE_RUN;
    }
}

// Sums of G rows at once.  v[q] is this lane's partial sum of row q.  The first log2(G) butterfly
// steps exchange half of the values each (a lane keeps the rows whose index bit equals its lane
// bit), the remaining steps add the one value left.  Afterwards the lanes whose index shares the
// top log2(G) bits, r = lane >> (5 - log2 G), all hold the complete sum of row r.
template <int G>
__device__ __forceinline__ float reduce_rows(float (&v)[G], int lane)
{
    int off = 16;
#pragma unroll
    for (int h = G / 2; h >= 1; h >>= 1, off >>= 1) {
        const bool upper = (lane & off) != 0;
#pragma unroll
        for (int j = 0; j < h; ++j) {
            const float send = upper ? v[j] : v[j + h];
            const float keep = upper ? v[j + h] : v[j];
            v[j] = keep + __shfl_xor_sync(0xffffffffu, send, off);
        }
    }
    float s = v[0];
    for (; off >= 1; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    return s;
}

// Part B, coefficients: one warp per position, a whole warp per row (a lane holds DIM / 32
// values), G target rows in flight.  Reads the dense target list that part A wrote; writes g per
// list entry, the center-row gradient GU[pos] = sum g * v and the position's loss.  The kernel is
// kept light - its pace is set by how many row reads are in flight and by instruction issue, not
// by arithmetic: the dot products of G rows are reduced together; the sigmoid, which the
// gradient needs at once, is evaluated per group of G rows on all lanes; the softplus of the
// loss is put off until every lane holds the argument of one entry (32 entries per evaluation);
// while a group is worked on, the rows of the next one are already on their way into L2.
// SINGLE (fp32 tables, plain SGD): an output row that receives only this contribution in the
// batch gets its increment -lr g u here, as one reduction per value (nobody else reads or changes
// the row in this batch, so the step stays synchronous and its bits do not depend on timing).
template <int DIM, typename T, bool SINGLE>
__global__ void __launch_bounds__(256, (DIM <= 64 ? 4 : 3))
sgns_coef_kernel(const T *__restrict__ w_in, T *w_out, int64_t n_pos, int32_t shift,
                 uint32_t n_nodes, const uint32_t *__restrict__ keys, const uint32_t *__restrict__ tinfo,
                 float *__restrict__ gbuf, float *__restrict__ GU, double *__restrict__ loss_pos,
                 const uint8_t *__restrict__ single, float lr)
{
    constexpr int FPL = DIM / 32;
    constexpr int G = FPL <= 4 ? 8 : 4;                 // rows in flight
    constexpr int SH = FPL <= 4 ? 2 : 3;                // lanes [r << SH, (r + 1) << SH) hold the sum of row r
    constexpr int QUAD = 1 << SH;                       // = 32 / G, also the groups per 32 entries
    constexpr int ROW_BYTES = DIM * (int)sizeof(T);
    const int lane = threadIdx.x & 31;
    const int64_t n_warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int64_t n_slots = n_pos << shift;
    for (int64_t pos = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); pos < n_pos;
         pos += n_warps) {
        const uint32_t info = tinfo[pos];
        const int n_ctx = (int)(info & 0xFFFFu), n = (int)(info >> 16);
        float loss = 0.f;
        if (n > 0) {                                    // the position forms pairs (same on every lane)
            const uint32_t *kp = keys + (pos << shift);
            float *gp = gbuf + (pos << shift);
            uint32_t id = lane < n ? kp[lane] : 0u;     // entries [k0, k0 + 32) of the list, one per lane
            const uint8_t *alone_p = single + (pos << shift);
            uint32_t alone = 0u;                        // ... and whether the entry is its row's only one
            if constexpr (SINGLE) alone = lane < n ? alone_p[lane] : 0u;
            const Row<FPL> u = row_load<FPL>(w_in, (int64_t)(keys[n_slots + pos] - n_nodes), lane);
            auto add_at_once = [&](uint32_t row, float g) {
                Row<FPL> d;
#pragma unroll
                for (int j = 0; j < FPL; ++j) d.v[j] = -lr * (g * u.v[j]);
                if constexpr (sizeof(T) == 4) row_red_add<FPL>(w_out, (int64_t)row, lane, d);
            };
            Row<FPL> acc;
#pragma unroll
            for (int j = 0; j < FPL; ++j) acc.v[j] = 0.f;
            // the first group's rows: one 128-byte line per lane, as far as the rows go
            {
                const uint32_t id0 = __shfl_sync(0xffffffffu, id, (lane * 128 / ROW_BYTES) & 31);
                if (lane * 128 < G * ROW_BYTES && lane * 128 / ROW_BYTES < n)
                    prefetch_l2((const char *)(w_out + (int64_t)id0 * DIM) + lane * 128 % ROW_BYTES);
            }
            for (int k0 = 0; k0 < n; k0 += 32) {
                const uint32_t id_next = k0 + 32 + lane < n ? kp[k0 + 32 + lane] : 0u;
                uint32_t alone_next = 0u;
                if constexpr (SINGLE) alone_next = k0 + 32 + lane < n ? alone_p[k0 + 32 + lane] : 0u;
                const unsigned alone_mask = __ballot_sync(0xffffffffu, alone != 0u);
                float my_z = 0.f;                       // softplus argument of the entry this lane keeps
                bool my_has = false;
                const int m = n - k0 < 32 ? n - k0 : 32;  // entries of this stretch
                int g0 = 0;
#pragma unroll 1
                for (; g0 + G <= m; g0 += G) {            // full groups of G rows
                    Row<FPL> rows[G];
                    float f[G];
#pragma unroll
                    for (int q = 0; q < G; ++q)
                        rows[q] = row_load<FPL>(w_out, (int64_t)__shfl_sync(0xffffffffu, id, g0 + q), lane);
                    {   // next group's rows towards L2: lane l asks for line l of the group's G rows
                        const int e = g0 + G + lane * 128 / ROW_BYTES;         // entry within [k0, k0 + 64)
                        const uint32_t idn = g0 + 2 * G <= 32 ? __shfl_sync(0xffffffffu, id, e & 31)
                                                              : __shfl_sync(0xffffffffu, id_next, e & 31);
                        if (lane * 128 < G * ROW_BYTES && k0 + e < n)
                            prefetch_l2((const char *)(w_out + (int64_t)idn * DIM) + lane * 128 % ROW_BYTES);
                    }
#pragma unroll
                    for (int q = 0; q < G; ++q) f[q] = row_dot<FPL>(u, rows[q]);
                    const float fr = reduce_rows<G>(f, lane);
                    const int kk = k0 + g0 + (lane >> SH);   // the entry whose sum this lane holds
                    const bool is_ctx = kk < n_ctx;     // contexts come first in the list
                    const float z = is_ctx ? -fr : fr;  // term: softplus(z); g = +-sigmoid(z)
                    const float e = expf(-fabsf(z));
                    const float rr = 1.0f / (1.0f + e);
                    const float sig = z >= 0.f ? rr : e * rr;
                    const float g = is_ctx ? -sig : sig;
                    if ((lane & (QUAD - 1)) == ((g0 / G) & (QUAD - 1))) { my_z = z; my_has = true; }
                    if ((lane & (QUAD - 1)) == 0) gp[kk] = g;
#pragma unroll
                    for (int q = 0; q < G; ++q) {
                        const float gq = __shfl_sync(0xffffffffu, g, q << SH);
#pragma unroll
                        for (int j = 0; j < FPL; ++j) acc.v[j] = fmaf(gq, rows[q].v[j], acc.v[j]);
                        if constexpr (SINGLE) {
                            if ((alone_mask >> (g0 + q)) & 1u) add_at_once(__shfl_sync(0xffffffffu, id, g0 + q), gq);
                        }
                    }
                }
#pragma unroll 1
                for (; g0 < m; ++g0) {                    // the last few entries of the list, one at a time
                    const Row<FPL> row = row_load<FPL>(w_out, (int64_t)__shfl_sync(0xffffffffu, id, g0), lane);
                    const float fr = warp_sum(row_dot<FPL>(u, row));
                    const bool is_ctx = k0 + g0 < n_ctx;
                    float sig, sp;
                    sigmoid_softplus(is_ctx ? -fr : fr, sig, sp);
                    const float g = is_ctx ? -sig : sig;
                    if (lane == 0) { gp[k0 + g0] = g; loss += sp; }
#pragma unroll
                    for (int j = 0; j < FPL; ++j) acc.v[j] = fmaf(g, row.v[j], acc.v[j]);
                    if constexpr (SINGLE) {
                        if ((alone_mask >> g0) & 1u) add_at_once(__shfl_sync(0xffffffffu, id, g0), g);
                    }
                }
                if (my_has) loss += fmaxf(my_z, 0.f) + log1pf(expf(-fabsf(my_z)));
                id = id_next;
                alone = alone_next;
            }
            row_store<FPL>(GU, pos, lane, acc);         // fp32 scratch, natural column order
        }
        loss = warp_sum(loss);                          // lane-local shares, fixed butterfly order
        if (lane == 0) loss_pos[pos] = (double)loss;
    }
}

// Optional momentum state of a table (m == nullptr: plain SGD).  With momentum the write of a
// row is  m <- mu m + grad ; row <- row - lr m ; last[row] <- next_iter  (Section 3.2: mult, put,
// mult_add, restricted to the rows of the batch; the other rows are brought up to date lazily by
// momentum_catchup before they are read again).
//
// With v != nullptr the state is Adam's instead (Kingma & Ba 2015, Algorithm 1; Section 3.2 names
// Adam next to SGD with momentum): m and v are the first and second moments, mu is beta1, and
// only the rows of the batch move (no catch-up: a row outside the batch keeps row, m and v):
//   m <- b1 m + (1-b1) g ; v <- b2 v + (1-b2) g^2 ; row <- row - lr (m/c1) / (sqrt(v/c2) + eps)
// with c1 = 1 - b1^step, c2 = 1 - b2^step computed on the host.
struct MomState {
    float *m;
    int32_t *last;
    float mu;
    int32_t next_iter;
    float *v;
    float b2, eps;
    double c1, c2;
    // stochastic write-back of a 16-bit table in the synchronous mode (sr != 0): the event of row r
    // is the block (r | sr_table << 32, sr_step, TAG_ROUND_SYNC, sr_sub), key sr_seed
    uint32_t sr, sr_table, sr_step, sr_sub;
    uint64_t sr_seed;
};

template <int FPL, typename T>
__device__ __forceinline__ void write_updated_row(T *__restrict__ tab, int64_t r, int lane,
                                                  Row<FPL> &row, const double (&acc)[FPL], float lr,
                                                  const MomState &ms)
{
    if (ms.v) {
        // fp32 arithmetic on the fp64 gradient sum rounded once: the moments are stored in fp32
        // anyway, and double-precision square roots and divisions would cost more than the rows.
        Row<FPL> m = row_load<FPL>(ms.m, r, lane);
        Row<FPL> v = row_load<FPL>(ms.v, r, lane);
        const float b1 = ms.mu, b2 = ms.b2, inv_c1 = (float)(1.0 / ms.c1), inv_c2 = (float)(1.0 / ms.c2);
#pragma unroll
        for (int j = 0; j < FPL; ++j) {
            const float g = (float)acc[j];
            m.v[j] = fmaf(b1, m.v[j], (1.0f - b1) * g);
            v.v[j] = fmaf(b2, v.v[j], (1.0f - b2) * (g * g));
            row.v[j] -= lr * (m.v[j] * inv_c1) / (sqrtf(v.v[j] * inv_c2) + ms.eps);
        }
        row_store<FPL>(ms.m, r, lane, m);
        row_store<FPL>(ms.v, r, lane, v);
    } else if (ms.m) {
        Row<FPL> m = row_load<FPL>(ms.m, r, lane);
#pragma unroll
        for (int j = 0; j < FPL; ++j) {
            const double mm = (double)ms.mu * (double)m.v[j] + acc[j];
            m.v[j] = (float)mm;
            row.v[j] = (float)((double)row.v[j] - (double)lr * mm);
        }
        row_store<FPL>(ms.m, r, lane, m);
        if (lane == 0) ms.last[r] = ms.next_iter;
    } else {
#pragma unroll
        for (int j = 0; j < FPL; ++j) row.v[j] = (float)((double)row.v[j] - (double)lr * acc[j]);
    }
    if constexpr (sizeof(T) == 2) {
        if (ms.sr) {
            const uint4 ev = draw(ms.sr_seed, (uint64_t)r | ((uint64_t)ms.sr_table << 32), ms.sr_step,
                                  TAG_ROUND_SYNC, ms.sr_sub);
            row_store_sr<FPL, T>(tab, r, lane, row, ev);
            return;
        }
    }
    row_store<FPL>(tab, r, lane, row);
}

// A row last written at iteration `last` and read at iteration `iter` missed k = iter - last
// dense updates without gradient:  row -= lr m (mu + ... + mu^k),  m *= mu^k.
__device__ __forceinline__ void catchup_factors(float mu, int k, double &f_row, double &f_m)
{
    f_m = pow((double)mu, (double)k);
    f_row = (double)mu * (1.0 - f_m) / (1.0 - (double)mu);
}

// One warp per 32 sorted keys: every run head is a distinct row the batch is about to read.
template <int FPL>
__global__ void __launch_bounds__(256)
momentum_catchup_kernel(float *__restrict__ w_in, float *__restrict__ w_out, MomState ms_in,
                        MomState ms_out, const uint32_t *__restrict__ keys, uint32_t n_keys,
                        uint32_t n_nodes, float lr, int32_t iter)
{
    const int lane = threadIdx.x & 31;
    const int64_t n_warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int64_t n_chunks = ((int64_t)n_keys + 31) >> 5;
    for (int64_t ch = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); ch < n_chunks;
         ch += n_warps) {
        const int64_t i = ch * 32 + lane;
        const uint32_t key = i < n_keys ? keys[i] : 0xFFFFFFFFu;
        const bool head = i < n_keys && key < 2u * n_nodes && (i == 0 || keys[i - 1] != key);
        const bool is_out = key < n_nodes;
        const uint32_t r = is_out ? key : key - n_nodes;
        int k = 0;
        if (head) {
            int32_t *lp = (is_out ? ms_out.last : ms_in.last) + r;
            k = iter - *lp;
            if (k > 0) *lp = iter;
        }
        unsigned todo = __ballot_sync(0xffffffffu, head && k > 0);
        while (todo) {
            const int l = __ffs(todo) - 1;
            todo &= todo - 1;
            const uint32_t rr = __shfl_sync(0xffffffffu, r, l);
            const int kk = __shfl_sync(0xffffffffu, k, l);
            const bool out = __shfl_sync(0xffffffffu, (int)is_out, l) != 0;
            float *tab = out ? w_out : w_in;
            float *mt = out ? ms_out.m : ms_in.m;
            double f_row, f_m;
            catchup_factors(ms_out.mu, kk, f_row, f_m);
            Row<FPL> row = row_load<FPL>(tab, rr, lane);
            Row<FPL> m = row_load<FPL>(mt, rr, lane);
#pragma unroll
            for (int j = 0; j < FPL; ++j) {
                row.v[j] = (float)((double)row.v[j] - (double)lr * f_row * (double)m.v[j]);
                m.v[j] = (float)(f_m * (double)m.v[j]);
            }
            row_store<FPL>(tab, rr, lane, row);
            row_store<FPL>(mt, rr, lane, m);
        }
    }
}

// Dense catch-up of a whole table (end of training, or before the table is read elsewhere).
__global__ void __launch_bounds__(256)
momentum_flush_kernel(float *__restrict__ w, float *__restrict__ m, int32_t *__restrict__ last,
                      int64_t n_rows, int32_t dim, float lr, float mu, int32_t iter)
{
    const int32_t quads = dim >> 2;
    const int64_t total = n_rows * quads;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t x = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; x < total; x += stride) {
        const int64_t row = x / quads;
        const int k = iter - last[row];
        if (k <= 0) continue;
        double f_row, f_m;
        catchup_factors(mu, k, f_row, f_m);
        float4 a = reinterpret_cast<float4 *>(w)[x], b = reinterpret_cast<float4 *>(m)[x];
        a.x = (float)((double)a.x - (double)lr * f_row * (double)b.x); b.x = (float)(f_m * (double)b.x);
        a.y = (float)((double)a.y - (double)lr * f_row * (double)b.y); b.y = (float)(f_m * (double)b.y);
        a.z = (float)((double)a.z - (double)lr * f_row * (double)b.z); b.z = (float)(f_m * (double)b.z);
        a.w = (float)((double)a.w - (double)lr * f_row * (double)b.w); b.w = (float)(f_m * (double)b.w);
        reinterpret_cast<float4 *>(w)[x] = a;
        reinterpret_cast<float4 *>(m)[x] = b;
    }
}

__global__ void __launch_bounds__(256)
momentum_stamp_kernel(int32_t *__restrict__ last, int64_t n_rows, int32_t iter)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t x = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; x < n_rows; x += stride)
        if (last[x] < iter) last[x] = iter;
}

// Passes 3 and 4 walk the sorted keys in chunks of 32: lane l looks at key 32*chunk + l and
// flags it if it starts a run of equal keys; the warp then sums each flagged run in index order
// (fp64 accumulators: a hub row can collect 10^5 terms) and writes the row once.  The metadata
// of 32 contributions is fetched by the 32 lanes at once and the rows 8 (or 4) at a time.
//
// Pass 3, keys below n_nodes: v_row -= lr * sum_j g_j * u_center(j).
// Runs are cut at every multiple of RUN_CUT sorted positions so that no warp sums more than
// RUN_CUT rows in a chain (a hub row of a 512-walk batch collects thousands).  A run that lies
// inside one block of RUN_CUT positions is finished here.  Otherwise its first piece leaves a
// partial sum in tail_part[block], each later piece in lead_part[block], and
// the last launch of the step (finish_cut_runs) adds the pieces in block order and writes the row.
constexpr int RUN_CUT = 256;

template <int FPL, typename T>
__global__ void __launch_bounds__(256, 2)
sgns_apply_out_kernel(const T *__restrict__ w_in, T *__restrict__ w_out,
                      const int32_t *__restrict__ walks, const uint32_t *__restrict__ keys,
                      const uint32_t *__restrict__ vals, const float *__restrict__ gbuf,
                      uint32_t n_keys, uint32_t n_nodes, int32_t shift, float lr,
                      double *__restrict__ lead_part, double *__restrict__ tail_part, MomState ms)
{
    // One warp per block of RUN_CUT sorted positions.  The 32 lanes fetch the metadata of 32
    // contributions at once; rows are then fetched G at a time - the center row of every
    // contribution and, where a run starts, the output row it will update - so that a block
    // full of one-element runs costs a few memory round trips, not one per run.
    constexpr int G = FPL <= 4 ? 8 : 4;
    const int lane = threadIdx.x & 31;
    const int64_t n_warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int64_t n_blocks = ((int64_t)n_keys + RUN_CUT - 1) / RUN_CUT;
    for (int64_t b = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); b < n_blocks;
         b += n_warps) {
        const int64_t base = b * RUN_CUT;
        const int64_t end = base + RUN_CUT < (int64_t)n_keys ? base + RUN_CUT : (int64_t)n_keys;
        uint32_t carry_key = base > 0 ? keys[base - 1] : 0xFFFFFFFFu;     // key before the block
        bool have = false, lead = false;         // a run is open / it started before this block
        uint32_t cur_key = 0;
        Row<FPL> cur_v;
        double acc[FPL];
#pragma unroll
        for (int j = 0; j < FPL; ++j) { acc[j] = 0.0; cur_v.v[j] = 0.f; }
        if (carry_key < n_nodes && keys[base] == carry_key) { have = true; lead = true; cur_key = carry_key; }

        auto close_run = [&](bool goes_on) {
            double *part = nullptr;
            if (lead) part = lead_part;
            else if (goes_on) part = tail_part;
            if (part) {
                double *dst = part + b * (int64_t)(FPL * 32);
#pragma unroll
                for (int j = 0; j < FPL; ++j) dst[j * 32 + lane] = acc[j];
            } else {
                write_updated_row<FPL, T>(w_out, cur_key, lane, cur_v, acc, lr, ms);
            }
        };

        // The metadata of a chunk of 32 contributions is a chain of two dependent reads (sorted key
        // and contribution index, then coefficient and center node).  It is fetched two chunks
        // ahead (first link) and one chunk ahead (second link), so that the rows of the current
        // chunk never wait for it.
        auto link1 = [&](int64_t i, uint32_t &key, uint32_t &idx) {
            key = i < end ? keys[i] : 0xFFFFFFFFu;
            idx = i < end ? vals[i] & ~SINGLE_RUN : 0u;    // this pass treats one-entry runs like the others
        };
        auto link2 = [&](uint32_t key, uint32_t idx, float &g, int32_t &c) {
            g = 0.f;
            c = 0;
            if (key < n_nodes) {
                g = gbuf[idx];
                c = walks[idx >> shift];                   // contribution idx belongs to position idx >> shift
            }
        };
        uint32_t my_key, key1, idx0, idx1;
        float g;
        int32_t c;
        link1(base + lane, my_key, idx0);
        link1(base + 32 + lane, key1, idx1);
        link2(my_key, idx0, g, c);
        for (int64_t s0 = base; s0 < end; s0 += 32) {
            uint32_t key2, idx2;
            link1(s0 + 64 + lane, key2, idx2);                        // two chunks ahead
            float g1;
            int32_t c1;
            link2(key1, idx1, g1, c1);                                // one chunk ahead
            const bool usable = my_key < n_nodes;                     // sorted: usable lanes are a prefix
            uint32_t before = __shfl_up_sync(0xffffffffu, my_key, 1);
            if (lane == 0) before = carry_key;
            carry_key = __shfl_sync(0xffffffffu, my_key, 31);
            const unsigned hmask = __ballot_sync(0xffffffffu, usable && my_key != before);
            const int n = __popc(__ballot_sync(0xffffffffu, usable));
            for (int q0 = 0; q0 < n; q0 += G) {
                Row<FPL> ru[G], rv[G];
#pragma unroll
                for (int q = 0; q < G; ++q) {
                    const int32_t cq = __shfl_sync(0xffffffffu, c, (q0 + q) & 31);
                    const uint32_t kq = __shfl_sync(0xffffffffu, my_key, (q0 + q) & 31);
                    if (q0 + q < n) {
                        ru[q] = row_load<FPL>(w_in, cq, lane);
                        if ((hmask >> (q0 + q)) & 1u) rv[q] = row_load<FPL>(w_out, kq, lane);
                    }
                }
#pragma unroll
                for (int q = 0; q < G; ++q) {
                    const float gq = __shfl_sync(0xffffffffu, g, (q0 + q) & 31);
                    const uint32_t kq = __shfl_sync(0xffffffffu, my_key, (q0 + q) & 31);
                    if (q0 + q < n) {
                        if ((hmask >> (q0 + q)) & 1u) {               // a run starts here
                            if (have) close_run(false);
                            have = true;
                            lead = false;
                            cur_key = kq;
                            cur_v = rv[q];
#pragma unroll
                            for (int j = 0; j < FPL; ++j) acc[j] = 0.0;
                        }
#pragma unroll
                        for (int j = 0; j < FPL; ++j) acc[j] += (double)(gq * ru[q].v[j]);
                    }
                }
            }
            if (n < 32) break;                                        // the rest is not ours
            my_key = key1; g = g1; c = c1;
            key1 = key2; idx1 = idx2;
        }
        if (have) close_run(end < (int64_t)n_keys && keys[end] == cur_key);
    }
}

// Pass 3 for fp32 tables and plain SGD.  Same walk over the sorted contributions as
// sgns_apply_out_kernel (one warp per block of RUN_CUT positions, runs cut at block boundaries
// and finished by the last launch of the step), made light so that many warps are resident:
//  - a run is summed in fp32, in index order, by the warp that owns its block: at most RUN_CUT
//    terms; the pieces of a longer run are added up in fp64 by the fix-up;
//  - the output row is not read: the finished sum goes out as ONE reduction per value,
//    row += -lr * sum.  Every row is owned by exactly one run, so this is the only addition the
//    row receives in the step and the result bits do not depend on scheduling.
// (Prefetching the next group's center rows into L1 while a group is added was measured and did
// not pay: 0.491 against 0.484 ms per batch.)
// MARKED: part A marked the runs of one entry and the coefficient pass has added them already.
template <int FPL, bool MARKED>
__global__ void __launch_bounds__(256, (FPL <= 2 ? 4 : 3))
sgns_apply_out_sgd_kernel(const float *__restrict__ w_in, float *__restrict__ w_out,
                          const int32_t *__restrict__ walks, const uint32_t *__restrict__ keys,
                          const uint32_t *__restrict__ vals, const float *__restrict__ gbuf,
                          uint32_t n_keys, uint32_t n_nodes, int32_t shift, float lr,
                          double *__restrict__ lead_part, double *__restrict__ tail_part)
{
    constexpr int G = FPL <= 4 ? 8 : 4;
    const int lane = threadIdx.x & 31;
    const int64_t n_warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int64_t n_blocks = ((int64_t)n_keys + RUN_CUT - 1) / RUN_CUT;
    for (int64_t b = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); b < n_blocks;
         b += n_warps) {
        const int64_t base = b * RUN_CUT;
        const int64_t end = base + RUN_CUT < (int64_t)n_keys ? base + RUN_CUT : (int64_t)n_keys;
        uint32_t carry_key = base > 0 ? keys[base - 1] : 0xFFFFFFFFu;     // key before the block
        bool have = false, lead = false;                 // a run is open / it began before this block
        uint32_t cur_key = 0;
        Row<FPL> acc;
#pragma unroll
        for (int j = 0; j < FPL; ++j) acc.v[j] = 0.f;
        if (carry_key < n_nodes && keys[base] == carry_key) { have = true; lead = true; cur_key = carry_key; }

        auto store_part = [&](double *part) {
            double *dst = part + b * (int64_t)(FPL * 32);
#pragma unroll
            for (int j = 0; j < FPL; ++j) dst[j * 32 + lane] = (double)acc.v[j];
        };
        auto close_inner = [&]() {                       // the run ends inside the block
            if (lead) {
                store_part(lead_part);
            } else {
                Row<FPL> d;
#pragma unroll
                for (int j = 0; j < FPL; ++j) d.v[j] = -lr * acc.v[j];
                row_red_add<FPL>(w_out, (int64_t)cur_key, lane, d);
            }
        };

        // metadata of a chunk: sorted key and contribution index, then coefficient and center node
        // (two dependent reads), fetched two chunks / one chunk ahead of the rows that need them
        auto link1 = [&](int64_t i, uint32_t &key, uint32_t &idx) {
            key = i < end ? keys[i] : 0xFFFFFFFFu;
            idx = i < end ? vals[i] : 0u;
        };
        // (a run of one entry, marked in bit 31 of its index, was added by the coefficient pass:
        // nothing of it is fetched here)
        auto link2 = [&](uint32_t key, uint32_t idx, float &g, int32_t &c) {
            g = 0.f;
            c = 0;
            if (key < n_nodes && !(MARKED && (idx & SINGLE_RUN))) {
                g = gbuf[idx];
                c = walks[idx >> shift];                  // contribution idx belongs to position idx >> shift
            }
        };
        uint32_t my_key, key1, idx0, idx1;
        float g;
        int32_t c;
        link1(base + lane, my_key, idx0);
        link1(base + 32 + lane, key1, idx1);
        link2(my_key, idx0, g, c);
        for (int64_t s0 = base; s0 < end; s0 += 32) {
            uint32_t key2, idx2;
            link1(s0 + 64 + lane, key2, idx2);
            float g1;
            int32_t c1;
            link2(key1, idx1, g1, c1);
            const bool usable = my_key < n_nodes;                     // sorted: usable lanes are a prefix
            uint32_t before = __shfl_up_sync(0xffffffffu, my_key, 1);
            if (lane == 0) before = carry_key;
            carry_key = __shfl_sync(0xffffffffu, my_key, 31);
            const unsigned hmask = __ballot_sync(0xffffffffu, usable && my_key != before);
            unsigned smask = 0u;                                      // runs of one entry, done already
            if constexpr (MARKED) smask = __ballot_sync(0xffffffffu, usable && (idx0 & SINGLE_RUN) != 0u);
            const int n = __popc(__ballot_sync(0xffffffffu, usable));
            // G contributions at a time: their center rows are loaded together, then added in
            // index order; where the head mask has a bit the run before ends and a new one starts
            auto add_one = [&](int i, float gq, const Row<FPL> &row) {
                if ((hmask >> i) & 1u) {                              // a run starts here (same on every lane)
                    if (have) close_inner();
                    if constexpr (MARKED) {
                        have = false;
                        if ((smask >> i) & 1u) return;                // ... and is over: done by the coefficient pass
                    }
                    have = true;
                    lead = false;
                    cur_key = __shfl_sync(0xffffffffu, my_key, i);
#pragma unroll
                    for (int j = 0; j < FPL; ++j) acc.v[j] = 0.f;
                }
#pragma unroll
                for (int j = 0; j < FPL; ++j) acc.v[j] = fmaf(gq, row.v[j], acc.v[j]);
            };
            int q0 = 0;
#pragma unroll 1
            for (; q0 + G <= n; q0 += G) {
                if constexpr (MARKED) {
                    if (((smask >> q0) & ((1u << G) - 1u)) == (1u << G) - 1u) {   // G one-entry runs in a row
                        if (have) close_inner();
                        have = false;
                        continue;
                    }
                }
                Row<FPL> ru[G];
#pragma unroll
                for (int q = 0; q < G; ++q)
                    if (!MARKED || !((smask >> (q0 + q)) & 1u))
                        ru[q] = row_load<FPL>(w_in, (int64_t)__shfl_sync(0xffffffffu, c, q0 + q), lane);
#pragma unroll
                for (int q = 0; q < G; ++q) add_one(q0 + q, __shfl_sync(0xffffffffu, g, q0 + q), ru[q]);
            }
#pragma unroll 1
            for (; q0 < n; ++q0) {                                    // only where the output-row keys end
                Row<FPL> r1;
                if (!MARKED || !((smask >> q0) & 1u))
                    r1 = row_load<FPL>(w_in, (int64_t)__shfl_sync(0xffffffffu, c, q0), lane);
                add_one(q0, __shfl_sync(0xffffffffu, g, q0), r1);
            }
            if (n < 32) break;                                        // the rest is not ours
            my_key = key1; g = g1; c = c1;
            if constexpr (MARKED) idx0 = idx1;
            key1 = key2; idx1 = idx2;
        }
        if (have) {
            const bool goes_on = end < (int64_t)n_keys && keys[end] == cur_key;
            if (goes_on && !lead) store_part(tail_part);              // first piece of a cut run
            else close_inner();                                       // (a middle piece is a lead piece)
        }
    }
}

// The last launch of a step does three independent jobs at once, by block role, instead of three
// small launches one after another (each of them too small to fill the device):
//   blocks [0, in_blocks)                      pass 4: the input rows of the centers,
//   blocks [in_blocks, in_blocks + fix_blocks) the output rows whose runs were cut at block boundaries,
//   the last block                             the fixed-order sums of losses and counters.
//
// Cut runs: one warp per block of RUN_CUT sorted positions: if a run starts in the block and
// continues past its end, add its pieces (tail of this block, then the leading pieces of the
// following blocks while they carry the same key) and write the row.
template <int FPL, typename T>
__device__ __forceinline__ void finish_cut_runs(int64_t warp, int64_t n_warps, T *__restrict__ w_out,
                                                const uint32_t *__restrict__ keys, uint32_t n_keys,
                                                uint32_t n_nodes, float lr,
                                                const double *__restrict__ lead_part,
                                                const double *__restrict__ tail_part, const MomState &ms)
{
    const int lane = threadIdx.x & 31;
    const int64_t n_blocks = ((int64_t)n_keys + RUN_CUT - 1) / RUN_CUT;
    for (int64_t b = warp; b + 1 < n_blocks; b += n_warps) {
        const int64_t last = (b + 1) * RUN_CUT - 1;                  // last position of block b
        const uint32_t key = keys[last];
        if (key >= n_nodes || keys[last + 1] != key) continue;       // nothing crosses this boundary
        if (keys[b * RUN_CUT] == key && b > 0 && keys[b * RUN_CUT - 1] == key) continue;   // run started earlier
        double acc[FPL];
        const double *t = tail_part + b * (int64_t)(FPL * 32);
#pragma unroll
        for (int j = 0; j < FPL; ++j) acc[j] = t[j * 32 + lane];
        for (int64_t nb = b + 1; nb < n_blocks && keys[nb * RUN_CUT] == key; ++nb) {
            const double *l = lead_part + nb * (int64_t)(FPL * 32);
#pragma unroll
            for (int j = 0; j < FPL; ++j) acc[j] += l[j * 32 + lane];
        }
        Row<FPL> row = row_load<FPL>(w_out, key, lane);
        write_updated_row<FPL, T>(w_out, key, lane, row, acc, lr, ms);
    }
}

// Pass 4, keys in [n_nodes, 2 n_nodes): u_row -= lr * sum of the positions' GU rows.
// The center keys sort behind every output-row key and before the invalid ones, so they form one
// stretch of at most n_pos sorted positions, and it starts at position *n_out: part A counted
// the output-row keys it wrote.  Every warp takes ONE position of the stretch: if a run of equal
// keys starts there, the warp sums the run's GU rows in index order and writes the row.
template <int FPL, typename T>
__device__ __forceinline__ void finish_input_rows(int64_t warp, int64_t n_warps, T *__restrict__ w_in,
                                                  const float *__restrict__ GU,
                                                  const uint32_t *__restrict__ keys,
                                                  const uint32_t *__restrict__ vals, uint32_t n_keys,
                                                  uint32_t n_nodes, uint32_t n_slots, uint32_t n_pos,
                                                  int64_t first, float lr, const MomState &ms)
{
    constexpr int U = FPL <= 4 ? 8 : 4;
    const int lane = threadIdx.x & 31;
    for (int64_t wi = warp; wi < (int64_t)n_pos; wi += n_warps) {
        const int64_t i = first + wi;
        if (i >= (int64_t)n_keys) break;
        const uint32_t key = keys[i];
        if (key >= 2u * n_nodes) break;                              // the invalid keys come last
        if (wi > 0 && keys[i - 1] == key) continue;                  // inside a run: its head does the work
        double acc[FPL];
#pragma unroll
        for (int j = 0; j < FPL; ++j) acc[j] = 0.0;
        for (int64_t y0 = i;; y0 += 32) {
            const int64_t y = y0 + lane;
            const bool in = y < n_keys && keys[y] == key;
            const int cnt = __popc(__ballot_sync(0xffffffffu, in));
            const uint32_t pos = in ? vals[y] - n_slots : 0u;
            for (int q0 = 0; q0 < cnt; q0 += U) {
                Row<FPL> r[U];
#pragma unroll
                for (int q = 0; q < U; ++q) {
                    const uint32_t pq = __shfl_sync(0xffffffffu, pos, (q0 + q) & 31);
                    if (q0 + q < cnt) r[q] = row_load<FPL>(GU, (int64_t)pq, lane);
                }
#pragma unroll
                for (int q = 0; q < U; ++q)
                    if (q0 + q < cnt) {
#pragma unroll
                        for (int j = 0; j < FPL; ++j) acc[j] += (double)r[q].v[j];
                    }
            }
            if (cnt < 32) break;
        }
        const int64_t c = (int64_t)(key - n_nodes);
        Row<FPL> row = row_load<FPL>(w_in, c, lane);
        write_updated_row<FPL, T>(w_in, c, lane, row, acc, lr, ms);
    }
}

// Pass 4 for fp32 tables and plain SGD: one warp per 32 sorted center positions.  The lanes fetch
// the metadata of the 32 positions at once and the GU rows G at a time; a run (the positions of
// one center node) is summed in index order by the warp whose chunk holds its first position -
// reading on past the chunk's end in the rare case that the run does - and goes out as one
// reduction per value, row += -lr * sum, the only addition that row receives in the step.
template <int FPL>
__device__ __forceinline__ void finish_input_rows_sgd(int64_t warp, int64_t n_warps, float *__restrict__ w_in,
                                                      const float *__restrict__ GU,
                                                      const uint32_t *__restrict__ keys,
                                                      const uint32_t *__restrict__ vals, uint32_t n_keys,
                                                      uint32_t n_nodes, uint32_t n_slots, uint32_t n_pos,
                                                      int64_t first, float lr)
{
    constexpr int G = FPL <= 4 ? 8 : 4;
    const int lane = threadIdx.x & 31;
    const int64_t n_chunks = ((int64_t)n_pos + 31) / 32;
    for (int64_t ch = warp; ch < n_chunks; ch += n_warps) {
        const int64_t i0 = first + ch * 32;
        if (i0 >= (int64_t)n_keys) break;
        const int64_t i = i0 + lane;
        const uint32_t key = i < (int64_t)n_keys ? keys[i] : 0xFFFFFFFFu;
        const bool usable = key >= n_nodes && key < 2u * n_nodes;    // sorted: usable lanes are a prefix
        const uint32_t pos = usable ? vals[i] - n_slots : 0u;
        uint32_t before = __shfl_up_sync(0xffffffffu, key, 1);
        if (lane == 0) before = i0 > 0 ? keys[i0 - 1] : 0xFFFFFFFFu;
        const unsigned hmask = __ballot_sync(0xffffffffu, usable && key != before);
        const int n = __popc(__ballot_sync(0xffffffffu, usable));
        if (hmask == 0) { if (n < 32) break; else continue; }        // no run starts in this chunk
        bool have = false;
        uint32_t cur_key = 0;
        Row<FPL> acc;
#pragma unroll
        for (int j = 0; j < FPL; ++j) acc.v[j] = 0.f;
        auto close = [&]() {
            Row<FPL> d;
#pragma unroll
            for (int j = 0; j < FPL; ++j) d.v[j] = -lr * acc.v[j];
            row_red_add<FPL>(w_in, (int64_t)(cur_key - n_nodes), lane, d);
        };
        auto add_one = [&](int q, const Row<FPL> &row) {
            if ((hmask >> q) & 1u) {
                if (have) close();
                have = true;
                cur_key = __shfl_sync(0xffffffffu, key, q);
#pragma unroll
                for (int j = 0; j < FPL; ++j) acc.v[j] = 0.f;
            }
#pragma unroll
            for (int j = 0; j < FPL; ++j) acc.v[j] += row.v[j];
        };
        int q0 = __ffs(hmask) - 1;                                    // entries before it belong to an earlier run
#pragma unroll 1
        for (; q0 + G <= n; q0 += G) {
            Row<FPL> r[G];
#pragma unroll
            for (int q = 0; q < G; ++q)
                r[q] = row_load<FPL>(GU, (int64_t)__shfl_sync(0xffffffffu, pos, q0 + q), lane);
#pragma unroll
            for (int q = 0; q < G; ++q) add_one(q0 + q, r[q]);
        }
#pragma unroll 1
        for (; q0 < n; ++q0) {
            const Row<FPL> r1 = row_load<FPL>(GU, (int64_t)__shfl_sync(0xffffffffu, pos, q0), lane);
            add_one(q0, r1);
        }
        if (n == 32) {                                                // the last run may go on past the chunk
            for (int64_t y = i0 + 32; y < (int64_t)n_keys && keys[y] == cur_key; ++y) {
                const Row<FPL> r1 = row_load<FPL>(GU, (int64_t)(vals[y] - n_slots), lane);
#pragma unroll
                for (int j = 0; j < FPL; ++j) acc.v[j] += r1.v[j];
            }
        }
        close();
        if (n < 32) break;
    }
}

// Fixed-order reduction of the per-position losses and counters by one block of 256 threads:
// thread t adds positions t, t + 256, ... in that order, then a binary tree over the threads.
__device__ __forceinline__ void finish_sums(const double *__restrict__ loss_pos,
                                            const int32_t *__restrict__ pairs_pos, int64_t n_pos,
                                            double *loss_out, long long *pairs_out,
                                            unsigned long long *masked_out, unsigned long long *refused_out)
{
    __shared__ double sl[256];
    __shared__ long long sp[256], sm[256];
    __shared__ unsigned int sr[256];
    double l = 0.0;
    long long p = 0, m = 0;
    unsigned int r = 0;
    for (int64_t x = threadIdx.x; x < n_pos; x += 256) {
        const int32_t packed = pairs_pos[x];             // pairs | masked negatives << 8 | refused ids << 20
        l += loss_pos[x];
        p += packed & 0xFF;
        m += (packed >> 8) & 0xFFF;
        r += (unsigned)packed >> 20;
    }
    sl[threadIdx.x] = l;
    sp[threadIdx.x] = p;
    sm[threadIdx.x] = m;
    sr[threadIdx.x] = r;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) {
            sl[threadIdx.x] += sl[threadIdx.x + o];
            sp[threadIdx.x] += sp[threadIdx.x + o];
            sm[threadIdx.x] += sm[threadIdx.x + o];
            sr[threadIdx.x] += sr[threadIdx.x + o];
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        if (loss_out) *loss_out += sl[0];
        if (pairs_out) *pairs_out += sp[0];
        if (masked_out) *masked_out += (unsigned long long)sm[0];
        if (refused_out && sr[0]) atomicAdd(refused_out, (unsigned long long)sr[0]);
    }
}

struct FinishArgs {
    const uint32_t *keys, *vals, *n_out;
    const float *GU;
    const double *lead_part, *tail_part, *loss_pos;
    const int32_t *pairs_pos;
    uint32_t n_keys, n_nodes, n_slots, n_pos;
    float lr;
    int in_blocks, fix_blocks;
    int light;                    // fp32 tables and plain SGD: input rows by reductions
    double *loss_out;
    long long *pairs_out;
    unsigned long long *masked_out, *refused_out;
};

template <int FPL, typename T>
__global__ void __launch_bounds__(256)
sgns_finish_kernel(T *__restrict__ w_in, T *__restrict__ w_out, FinishArgs fa, MomState ms_in, MomState ms_out)
{
    const int wpb = blockDim.x >> 5;
    const int b = (int)blockIdx.x;
    if (b < fa.in_blocks) {
        const int64_t warp = (int64_t)b * wpb + (threadIdx.x >> 5), n_warps = (int64_t)fa.in_blocks * wpb;
        if constexpr (std::is_same<T, float>::value) {
            if (fa.light) {
                finish_input_rows_sgd<FPL>(warp, n_warps, w_in, fa.GU, fa.keys, fa.vals, fa.n_keys, fa.n_nodes,
                                           fa.n_slots, fa.n_pos, (int64_t)*fa.n_out, fa.lr);
                return;
            }
        }
        finish_input_rows<FPL, T>(warp, n_warps, w_in, fa.GU, fa.keys, fa.vals, fa.n_keys, fa.n_nodes,
                                  fa.n_slots, fa.n_pos, (int64_t)*fa.n_out, fa.lr, ms_in);
    } else if (b < fa.in_blocks + fa.fix_blocks) {
        finish_cut_runs<FPL, T>((int64_t)(b - fa.in_blocks) * wpb + (threadIdx.x >> 5),
                                (int64_t)fa.fix_blocks * wpb, w_out, fa.keys, fa.n_keys, fa.n_nodes, fa.lr,
                                fa.lead_part, fa.tail_part, ms_out);
    } else {
        finish_sums(fa.loss_pos, fa.pairs_pos, (int64_t)fa.n_pos, fa.loss_out, fa.pairs_out, fa.masked_out,
                    fa.refused_out);
    }
}

// ---------------------------------------------------------------- host side
struct SgnsArgs {
    void *w_in, *w_out;           // tables of float or __half, as the caller of run_* says
    int64_t n_nodes;
    int32_t dim;
    const int32_t *walks;
    int64_t n_walks, walk_id_base;
    int32_t L, w, K;
    const uint64_t *alias;
    float lr;
    uint64_t seed;
    double *loss;
    int64_t *pairs;
    int32_t *dump_pairs, *dump_negs;
    int fwd;                      // PAIR_* flags of build_targets
    unsigned long long *masked;   // nullable: masked negatives are ADDED
    int prepared;                 // >= 0: scratch set in which part A of this batch already ran
    unsigned long long *refused;  // nullable: ids treated as absent because they name no row are ADDED
    int sr;                       // 16-bit tables: stochastic write-back instead of round to nearest
};

static int bit_length(uint64_t x) { int b = 0; while (x) { ++b; x >>= 1; } return b; }

template <int DIM, typename T, bool RED, int MINB, int TC = TCH, bool NARROW = false, bool SR = false>
static gs_status run_hogwild_b(const SgnsArgs &a, cudaStream_t st)
{
    const int SL = 2 * a.w * (1 + a.K);
    const size_t smem = sizeof(int32_t) * (size_t)SGNS_WARPS * (size_t)(hogwild_walks_per_ticket(a.L) * a.L + (SR ? 2 : 1) * SL);
    auto kern = sgns_hogwild_kernel<DIM, T, RED, MINB, TC, NARROW, SR>;
    if (smem > 48 * 1024)
        GS_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    int per_sm = 0;
    GS_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, SGNS_WARPS * 32, smem));
    if (per_sm < 1) per_sm = 1;
    int64_t blocks = (a.n_walks + SGNS_WARPS - 1) / SGNS_WARPS;
    const int64_t cap = (int64_t)sm_count() * per_sm;
    if (blocks > cap) blocks = cap;
    void *ws = nullptr;
    gs_status ws_s = workspace_get(WS_COUNTERS, 256, &ws);
    if (ws_s != GS_OK) return ws_s;
    unsigned long long *ticket = (unsigned long long *)((char *)ws + 128);   // bytes 0..127: other counters
    GS_CUDA_TRY(cudaMemsetAsync(ticket, 0, sizeof(unsigned long long), st));
    kern<<<(unsigned)blocks, SGNS_WARPS * 32, smem, st>>>(
        (T *)a.w_in, (T *)a.w_out, a.walks, a.n_walks, a.walk_id_base, a.L, a.w, a.K, a.alias,
        (uint32_t)a.n_nodes, a.lr, a.seed, a.loss, (unsigned long long *)a.pairs, a.dump_pairs,
        a.dump_negs, ticket, a.fwd, a.masked, a.refused);
    GS_CUDA_TRY(cudaGetLastError());
    return GS_OK;
}

// Resident blocks per SM asked of the compiler: 5 blocks of 4 warps (96 registers per thread)
// measured best when a lane holds 4 values of a row; 8 values per lane need the registers.
template <int DIM, typename T, bool RED>
static gs_status run_hogwild(const SgnsArgs &a, cudaStream_t st)
{
    if constexpr (sizeof(T) == 2) {
        if (a.sr && !RED)                   // stochastic write-back: the dithers need registers
            return run_hogwild_b<DIM, T, false, 5, 3, false, true>(a, st);
    }
    if constexpr (sizeof(T) == 2)            // 16-bit rows: 3 rows per group in flight, 5 blocks of 96 registers
        return run_hogwild_b<DIM, T, RED, 5, 3>(a, st);
    else {
        // few targets per position (fewer than two wide chunks): 16 bytes per lane, one chunk
        // of TCH rows per row group, so that chunks are full
        using W = RowGeom<DIM, T, false>;
        using N = RowGeom<DIM, T, true>;
        if (W::LPR != N::LPR && 2 * a.w * (1 + a.K) < 2 * TCH * W::NG)
            return run_hogwild_b<DIM, T, RED, (N::FPL <= 4 ? 5 : 4), TCH, true>(a, st);
        return run_hogwild_b<DIM, T, RED, (W::FPL <= 4 ? 5 : 4), TCH>(a, st);
    }
}

static size_t align_up(size_t x) { return (x + 255) & ~(size_t)255; }

// Momentum state handed in by gs_sgns_step_momentum (nullptr for the plain step).
struct MomHost {
    float *m_in, *m_out;
    int32_t *last_in, *last_out;
    float mu;
    int32_t iter;
    // Adam (gs_sgns_step_adam): second moments, beta2, eps and the 1-based step; mu is beta1
    float *v_in, *v_out;
    float b2, eps;
    int64_t step;
};

// Scratch of one synchronous step.  By default it comes from the growing per-device cache, which
// holds two sets so that part A of one batch can run while part B of the batch before it is
// still reading its own; a caller that must not allocate hands in a fixed block instead
// (gs_sgns_step_static), and a batch that does not fit it is refused.
struct FixedScratch {
    unsigned char *ptr;
    size_t bytes;
};

struct SyncScratch {
    uint32_t *keys;               // part A: destination row per slot, then one center key per position
    uint32_t *keysB, *valsB, *keysC, *valsC, *counts;   // sort buffers
    uint32_t *ks, *vs;            // where the sorted keys / contribution indices end up (B or C)
    float *gbuf, *GU;
    double *loss_pos;
    int32_t *pairs_pos;
    uint32_t *tinfo;              // per position: contexts | all targets << 16 of its dense list
    uint32_t *n_out;              // output-row keys of the batch (one counter)
    uint8_t *single;              // per list entry: the only contribution to its output row in this batch
    bool mark;                    // one-entry runs are marked (and added by the coefficient pass)
    double *lead_part, *tail_part;
    int64_t n_pos, n_slots, n_keys, n_cut;
    int SL, shift, bits;          // a position's list occupies 2^shift >= SL entries
};

// Lays the arrays of one step out in `base` (nullptr: sizes only).  Returns the bytes needed.
static size_t sync_layout(const SgnsArgs &a, unsigned char *base, SyncScratch *out)
{
    SyncScratch s;
    s.SL = 2 * a.w * (1 + a.K);
    s.shift = bit_length((uint64_t)s.SL - 1);            // smallest power of two >= SL
    s.n_pos = a.n_walks * a.L;
    s.n_slots = s.n_pos << s.shift;
    s.n_keys = s.n_slots + s.n_pos;
    s.n_cut = (s.n_keys + RUN_CUT - 1) / RUN_CUT;
    s.bits = bit_length(2ull * (uint64_t)a.n_nodes);
    s.mark = (int64_t)a.n_nodes >= SINGLE_MIN_NODES_PER_ENTRY * s.n_slots;
    const size_t b_keys = align_up(sizeof(uint32_t) * (size_t)s.n_keys);
    const size_t b_g = align_up(sizeof(float) * (size_t)s.n_slots);
    const size_t b_gu = align_up(sizeof(float) * (size_t)s.n_pos * a.dim);
    const size_t b_loss = align_up(sizeof(double) * (size_t)s.n_pos);
    const size_t b_pairs = align_up(sizeof(int32_t) * (size_t)s.n_pos);
    const size_t b_cnt = align_up(sort_counts_bytes((uint32_t)s.n_keys));
    const size_t b_part = align_up(sizeof(double) * (size_t)s.n_cut * a.dim);
    const size_t b_single = align_up((size_t)s.n_slots);
    unsigned char *p = base;
    s.keys = (uint32_t *)p; p += b_keys;
    s.keysB = (uint32_t *)p; p += b_keys;
    s.valsB = (uint32_t *)p; p += b_keys;
    s.keysC = (uint32_t *)p; p += b_keys;
    s.valsC = (uint32_t *)p; p += b_keys;
    s.gbuf = (float *)p; p += b_g;
    s.GU = (float *)p; p += b_gu;
    s.loss_pos = (double *)p; p += b_loss;
    s.pairs_pos = (int32_t *)p; p += b_pairs;
    s.tinfo = (uint32_t *)p; p += b_pairs;
    s.n_out = (uint32_t *)p; p += 256;
    s.counts = (uint32_t *)p; p += b_cnt;
    s.single = (uint8_t *)p; p += b_single;
    s.lead_part = (double *)p; p += b_part;
    s.tail_part = (double *)p; p += b_part;
    // the sort alternates B, C, B, ...: an odd number of passes ends in B
    const int passes = (s.bits + 7) / 8;
    s.ks = (passes & 1) ? s.keysB : s.keysC;
    s.vs = (passes & 1) ? s.valsB : s.valsC;
    if (out) *out = s;
    return (size_t)(p - base);
}

// Finds the scratch of set `set` (0 or 1) of the current device, or the caller's fixed block.
static gs_status sync_scratch(const SgnsArgs &a, int set, const FixedScratch *fixed, SyncScratch *out)
{
    SyncScratch probe;
    const size_t need = sync_layout(a, nullptr, &probe);
    if (probe.n_keys > ((int64_t)1 << 30)) {
        set_error("deterministic step: %lld slots exceed 2^30; use smaller batches", (long long)probe.n_keys);
        return GS_ERR_UNSUPPORTED;
    }
    void *ws = nullptr;
    if (fixed) {
        if (need > fixed->bytes) {
            set_error("gs_sgns_step_static: this batch needs %zu bytes of scratch, the fixed array has %zu; "
                      "pass fewer walks per call or use gs_sgns_step", need, fixed->bytes);
            return GS_ERR_UNSUPPORTED;
        }
        // Every byte that is read is written first by the pass before it (keys and pair counts
        // by the targets pass for all slots; digit counts by the histogram pass for all tiles;
        // the marks of one-entry runs by the marking pass for every list entry that exists;
        // g, GU and losses by the coefficient pass wherever the apply passes read them; the
        // partial sums of cut runs by the apply pass before the fix-up pass reads exactly
        // those), so nothing left over from an earlier call can leak in.
        ws = fixed->ptr;
    } else {
        gs_status s = workspace_get(set ? WS_SGNS1 : WS_SGNS, need, &ws);
        if (s != GS_OK) return s;
    }
    sync_layout(a, (unsigned char *)ws, out);
    return GS_OK;
}

// Part A of the synchronous step (no table is read): targets and keys of every slot, sorted.
static gs_status sync_prepare(const SgnsArgs &a, int set, const FixedScratch *fixed, cudaStream_t st)
{
    SyncScratch sc;
    gs_status s = sync_scratch(a, set, fixed, &sc);
    if (s != GS_OK) return s;
    const size_t smem = sizeof(int32_t) * (size_t)SGNS_WARPS * sc.SL;
    int64_t blocks = (sc.n_pos + SGNS_WARPS - 1) / SGNS_WARPS;
    if (blocks > (int64_t)sm_count() * 16) blocks = (int64_t)sm_count() * 16;
    GS_CUDA_TRY(cudaMemsetAsync(sc.n_out, 0, sizeof(uint32_t), st));
    sgns_targets_kernel<<<(unsigned)blocks, SGNS_WARPS * 32, smem, st>>>(
        a.walks, sc.n_pos, a.walk_id_base, a.L, a.w, a.K, a.alias, (uint32_t)a.n_nodes,
        (uint32_t)a.n_nodes, a.seed, sc.shift, sc.keys, sc.tinfo, sc.pairs_pos, sc.n_out, a.dump_pairs,
        a.dump_negs, a.fwd);
    GS_CUDA_TRY(cudaGetLastError());
    uint32_t *ks = nullptr, *vs = nullptr;
    radix_sort_pairs(sc.keys, sc.keysB, sc.valsB, sc.keysC, sc.valsC, (uint32_t)sc.n_keys, sc.bits,
                     sc.counts, st, &ks, &vs);
    GS_CUDA_TRY(cudaGetLastError());
    if (ks != sc.ks || vs != sc.vs) { set_error("internal: sort result buffer mismatch"); return GS_ERR_CUDA; }
    if (sc.mark) {
        int64_t mb = (sc.n_keys + 255) / 256;
        if (mb > (int64_t)sm_count() * 16) mb = (int64_t)sm_count() * 16;
        sgns_mark_single_kernel<<<(unsigned)mb, 256, 0, st>>>(sc.ks, sc.vs, (uint32_t)sc.n_keys,
                                                              (uint32_t)a.n_nodes, sc.single);
        GS_CUDA_TRY(cudaGetLastError());
    }
    return GS_OK;
}

// Part B: coefficients from the entry tables, then the apply passes over the sorted contributions.
template <int DIM, typename T>
static gs_status sync_update(const SgnsArgs &a, int set, const FixedScratch *fixed, cudaStream_t st,
                             const MomHost *mom)
{
    T *w_in = (T *)a.w_in, *w_out = (T *)a.w_out;
    constexpr int FPL = DIM / 32;                        // the passes use a whole warp per row
    MomState ms_in = { nullptr, nullptr, 0.f, 0 }, ms_out = { nullptr, nullptr, 0.f, 0 };
    const bool adam = mom && mom->v_in;
    if (adam) {
        const double c1 = 1.0 - pow((double)mom->mu, (double)mom->step);
        const double c2 = 1.0 - pow((double)mom->b2, (double)mom->step);
        ms_in = MomState{ mom->m_in, nullptr, mom->mu, 0, mom->v_in, mom->b2, mom->eps, c1, c2 };
        ms_out = MomState{ mom->m_out, nullptr, mom->mu, 0, mom->v_out, mom->b2, mom->eps, c1, c2 };
    } else if (mom) {
        ms_in = MomState{ mom->m_in, mom->last_in, mom->mu, mom->iter + 1 };
        ms_out = MomState{ mom->m_out, mom->last_out, mom->mu, mom->iter + 1 };
    }
    if (a.sr) {
        for (MomState *ms : { &ms_in, &ms_out }) {
            ms->sr = 1;
            ms->sr_table = ms == &ms_out ? 1u : 0u;
            ms->sr_step = (uint32_t)((uint64_t)a.walk_id_base & 0xFFFFFFFFu);
            ms->sr_sub = (uint32_t)(((uint64_t)a.walk_id_base >> 32) & 0xFFFFFFu);
            ms->sr_seed = a.seed;
        }
    }
    SyncScratch sc;
    gs_status s = sync_scratch(a, set, fixed, &sc);
    if (s != GS_OK) return s;
    const int64_t cap = (int64_t)sm_count() * 8 * 8;
    if (mom && !adam) {
        // lazy momentum: bring every row the batch touches up to iteration `iter` before it is read
        int64_t cb = (sc.n_keys + 255) / 256;
        if (cb > (int64_t)sm_count() * 64) cb = (int64_t)sm_count() * 64;
        if constexpr (sizeof(T) == 4)
            momentum_catchup_kernel<FPL><<<(unsigned)cb, 256, 0, st>>>(
                w_in, w_out, ms_in, ms_out, sc.ks, (uint32_t)sc.n_keys, (uint32_t)a.n_nodes, a.lr, mom->iter);
        GS_CUDA_TRY(cudaGetLastError());
    }
    {
        int64_t blocks = (sc.n_pos + 7) / 8;             // one warp per position
        if (blocks > cap) blocks = cap;
        bool light = false;
        if constexpr (sizeof(T) == 4) light = !mom;      // fp32 tables, plain SGD
        if (light && sc.mark) {
            if constexpr (sizeof(T) == 4)
                sgns_coef_kernel<DIM, T, true><<<(unsigned)blocks, 256, 0, st>>>(
                    w_in, w_out, sc.n_pos, sc.shift, (uint32_t)a.n_nodes, sc.keys, sc.tinfo, sc.gbuf, sc.GU,
                    sc.loss_pos, sc.single, a.lr);
        } else {
            sgns_coef_kernel<DIM, T, false><<<(unsigned)blocks, 256, 0, st>>>(
                w_in, w_out, sc.n_pos, sc.shift, (uint32_t)a.n_nodes, sc.keys, sc.tinfo, sc.gbuf, sc.GU,
                sc.loss_pos, sc.single, a.lr);
        }
        GS_CUDA_TRY(cudaGetLastError());
    }
    {
        const unsigned out_blocks = (unsigned)((sc.n_cut + 7) / 8);
        bool light = false;
        if constexpr (sizeof(T) == 4) light = !mom;      // fp32 tables, plain SGD
        if (light) {
            if constexpr (sizeof(T) == 4) {
                if (sc.mark)
                    sgns_apply_out_sgd_kernel<FPL, true><<<out_blocks, 256, 0, st>>>(
                        w_in, w_out, a.walks, sc.ks, sc.vs, sc.gbuf, (uint32_t)sc.n_keys, (uint32_t)a.n_nodes,
                        sc.shift, a.lr, sc.lead_part, sc.tail_part);
                else
                    sgns_apply_out_sgd_kernel<FPL, false><<<out_blocks, 256, 0, st>>>(
                        w_in, w_out, a.walks, sc.ks, sc.vs, sc.gbuf, (uint32_t)sc.n_keys, (uint32_t)a.n_nodes,
                        sc.shift, a.lr, sc.lead_part, sc.tail_part);
            }
        } else {
            sgns_apply_out_kernel<FPL, T><<<out_blocks, 256, 0, st>>>(
                w_in, w_out, a.walks, sc.ks, sc.vs, sc.gbuf, (uint32_t)sc.n_keys, (uint32_t)a.n_nodes, sc.shift,
                a.lr, sc.lead_part, sc.tail_part, ms_out);
        }
        GS_CUDA_TRY(cudaGetLastError());
    }
    {
        // last launch: input rows, cut runs of output rows, sums - independent jobs, by block role
        bool light = false;
        if constexpr (sizeof(T) == 4) light = !mom;      // fp32 tables, plain SGD
        // input rows: one warp per center position, or (light) per 32 sorted center positions
        int64_t in_blocks = light ? (sc.n_pos + 255) / 256 : (sc.n_pos + 7) / 8;
        if (in_blocks > cap) in_blocks = cap;
        int64_t fix_blocks = sc.n_cut > 1 ? (sc.n_cut + 7) / 8 : 0;
        if (fix_blocks > cap) fix_blocks = cap;
        const bool sums = a.loss || a.pairs || a.masked || a.refused;
        FinishArgs fa = { sc.ks, sc.vs, sc.n_out, sc.GU, sc.lead_part, sc.tail_part, sc.loss_pos, sc.pairs_pos,
                          (uint32_t)sc.n_keys, (uint32_t)a.n_nodes, (uint32_t)sc.n_slots, (uint32_t)sc.n_pos,
                          a.lr, (int)in_blocks, (int)fix_blocks, light ? 1 : 0, a.loss, (long long *)a.pairs,
                          a.masked, a.refused };
        sgns_finish_kernel<FPL, T><<<(unsigned)(in_blocks + fix_blocks + (sums ? 1 : 0)), 256, 0, st>>>(
            w_in, w_out, fa, ms_in, ms_out);
        GS_CUDA_TRY(cudaGetLastError());
    }
    return GS_OK;
}

// One synchronous step.  a.prepared >= 0: part A of this batch has already run into that scratch
// set (gs_sgns_epoch does that on its walk stream); otherwise both parts run here, in order.
template <int DIM, typename T>
static gs_status run_deterministic(const SgnsArgs &a, cudaStream_t st, const MomHost *mom = nullptr,
                                   const FixedScratch *fixed = nullptr)
{
    int set = a.prepared;
    if (set < 0) {
        set = 0;
        gs_status s = sync_prepare(a, set, fixed, st);
        if (s != GS_OK) return s;
    }
    return sync_update<DIM, T>(a, set, fixed, st, mom);
}

static int pair_flags_of(int32_t mode)
{
    return ((mode & GS_PAIRS_FORWARD_ONLY) ? PAIR_FWD : 0) | ((mode & GS_WINDOW_SHRINK) ? PAIR_SHRINK : 0);
}

template <int DIM, typename T>
static gs_status run_mode(const SgnsArgs &a, int mode, cudaStream_t st)
{
    if (mode == GS_DETERMINISTIC) return run_deterministic<DIM, T>(a, st);
    if (mode == GS_HOGWILD) return run_hogwild<DIM, T, false>(a, st);
    if (a.sr) {                     // the reduction unit rounds to nearest
        set_error("GS_ROUND_STOCHASTIC is not available with GS_HOGWILD_RED");
        return GS_ERR_UNSUPPORTED;
    }
    return run_hogwild<DIM, T, true>(a, st);
}

// One step on tables of type T (float, or a 16-bit format with fp32 arithmetic and write-back
// rounded to nearest even).
template <typename T>
static gs_status step_on_tables(void *w_in, void *w_out, int64_t n_nodes, int32_t dim, const int32_t *walks,
                                int64_t n_walks, int64_t walk_id_base, int32_t L, int32_t w, int32_t K,
                                const uint64_t *alias, float lr, uint64_t seed, int32_t mode, double *loss,
                                int64_t *pairs, int32_t *dump_pairs, int32_t *dump_negs, cudaStream_t st,
                                unsigned long long *masked, int prepared)
{
    if (n_walks == 0) return GS_OK;
    SgnsArgs a = { w_in, w_out, n_nodes, dim, walks, n_walks, walk_id_base, L, w, K, alias, lr,
                   seed, loss, pairs, dump_pairs, dump_negs, pair_flags_of(mode), masked, prepared, refused_counter(),
                   (mode & GS_ROUND_STOCHASTIC) ? 1 : 0 };
    if (a.sr && sizeof(T) != 2) {
        set_error("GS_ROUND_STOCHASTIC applies to 16-bit tables");
        return GS_ERR_UNSUPPORTED;
    }
    mode &= ~(GS_PAIRS_FORWARD_ONLY | GS_WINDOW_SHRINK | GS_ROUND_STOCHASTIC);
    switch (dim) {
        case 32:
            if constexpr (sizeof(T) == 4) return run_mode<32, T>(a, mode, st);
            break;
        case 64: return run_mode<64, T>(a, mode, st);
        case 128: return run_mode<128, T>(a, mode, st);
        case 256: return run_mode<256, T>(a, mode, st);
        default: break;
    }
    set_error(sizeof(T) == 4 ? "dim %d not supported (32, 64, 128, 256)"
                             : "dim %d not supported with 16-bit tables (64, 128, 256)", dim);
    return GS_ERR_UNSUPPORTED;
}

gs_status sgns_step(float *w_in, float *w_out, int64_t n_nodes, int32_t dim, const int32_t *walks,
                    int64_t n_walks, int64_t walk_id_base, int32_t L, int32_t w, int32_t K,
                    const uint64_t *alias, float lr, uint64_t seed, int32_t mode, double *loss,
                    int64_t *pairs, int32_t *dump_pairs, int32_t *dump_negs, cudaStream_t st,
                    unsigned long long *masked, int prepared)
{
    return step_on_tables<float>(w_in, w_out, n_nodes, dim, walks, n_walks, walk_id_base, L, w, K, alias, lr,
                                 seed, mode, loss, pairs, dump_pairs, dump_negs, st, masked, prepared);
}

gs_status sgns_step_f16(void *w_in, void *w_out, int64_t n_nodes, int32_t dim, const int32_t *walks,
                        int64_t n_walks, int64_t walk_id_base, int32_t L, int32_t w, int32_t K,
                        const uint64_t *alias, float lr, uint64_t seed, int32_t mode, double *loss,
                        int64_t *pairs, int32_t *dump_pairs, int32_t *dump_negs, cudaStream_t st,
                        unsigned long long *masked, int prepared)
{
    return step_on_tables<__half>(w_in, w_out, n_nodes, dim, walks, n_walks, walk_id_base, L, w, K, alias, lr,
                                  seed, mode, loss, pairs, dump_pairs, dump_negs, st, masked, prepared);
}

gs_status sgns_step_bf16(void *w_in, void *w_out, int64_t n_nodes, int32_t dim, const int32_t *walks,
                         int64_t n_walks, int64_t walk_id_base, int32_t L, int32_t w, int32_t K,
                         const uint64_t *alias, float lr, uint64_t seed, int32_t mode, double *loss,
                         int64_t *pairs, int32_t *dump_pairs, int32_t *dump_negs, cudaStream_t st,
                         unsigned long long *masked, int prepared)
{
    return step_on_tables<__nv_bfloat16>(w_in, w_out, n_nodes, dim, walks, n_walks, walk_id_base, L, w, K,
                                         alias, lr, seed, mode, loss, pairs, dump_pairs, dump_negs, st,
                                         masked, prepared);
}

gs_status sgns_step_momentum(float *w_in, float *w_out, float *m_in, float *m_out, int32_t *last_in,
                             int32_t *last_out, int64_t n_nodes, int32_t dim, const int32_t *walks,
                             int64_t n_walks, int64_t walk_id_base, int32_t L, int32_t w, int32_t K,
                             const uint64_t *alias, float lr, float mu, int32_t iter, uint64_t seed,
                             double *loss, int64_t *pairs, cudaStream_t st, int prepared)
{
    if (n_walks == 0) return GS_OK;
    SgnsArgs a = { w_in, w_out, n_nodes, dim, walks, n_walks, walk_id_base, L, w, K, alias, lr,
                   seed, loss, pairs, nullptr, nullptr, 0, nullptr, prepared, refused_counter(), 0 };
    MomHost mom = { m_in, m_out, last_in, last_out, mu, iter, nullptr, nullptr, 0.f, 0.f, 0 };
    switch (dim) {
        case 32: return run_deterministic<32, float>(a, st, &mom);
        case 64: return run_deterministic<64, float>(a, st, &mom);
        case 128: return run_deterministic<128, float>(a, st, &mom);
        case 256: return run_deterministic<256, float>(a, st, &mom);
        default:
            set_error("dim %d not supported (32, 64, 128, 256)", dim);
            return GS_ERR_UNSUPPORTED;
    }
}

gs_status sgns_step_adam(float *w_in, float *w_out, float *m_in, float *v_in, float *m_out,
                         float *v_out, int64_t n_nodes, int32_t dim, const int32_t *walks,
                         int64_t n_walks, int64_t walk_id_base, int32_t L, int32_t w, int32_t K,
                         const uint64_t *alias, float lr, float b1, float b2, float eps, int64_t step,
                         uint64_t seed, int32_t pair_mode, double *loss, int64_t *pairs, cudaStream_t st,
                         int prepared)
{
    if (n_walks == 0) return GS_OK;
    SgnsArgs a = { w_in, w_out, n_nodes, dim, walks, n_walks, walk_id_base, L, w, K, alias, lr,
                   seed, loss, pairs, nullptr, nullptr, pair_flags_of(pair_mode), nullptr, prepared, refused_counter(), 0 };
    MomHost mom = { m_in, m_out, nullptr, nullptr, b1, 0, v_in, v_out, b2, eps, step };
    switch (dim) {
        case 32: return run_deterministic<32, float>(a, st, &mom);
        case 64: return run_deterministic<64, float>(a, st, &mom);
        case 128: return run_deterministic<128, float>(a, st, &mom);
        case 256: return run_deterministic<256, float>(a, st, &mom);
        default:
            set_error("dim %d not supported (32, 64, 128, 256)", dim);
            return GS_ERR_UNSUPPORTED;
    }
}

// Part A of the synchronous step for the epoch driver: lists and sorts the contributions of a
// batch into scratch set `set` (0 or 1) without reading a table, so that it can run on another
// stream while the batch before it is still being applied.  The step functions above then take
// prepared = set.
gs_status sgns_prepare_sync(int64_t n_nodes, int32_t dim, const int32_t *walks, int64_t n_walks,
                            int64_t walk_id_base, int32_t L, int32_t w, int32_t K, const uint64_t *alias,
                            uint64_t seed, int32_t pair_mode, int set, cudaStream_t st)
{
    if (n_walks == 0) return GS_OK;
    SgnsArgs a = { nullptr, nullptr, n_nodes, dim, walks, n_walks, walk_id_base, L, w, K, alias, 0.f,
                   seed, nullptr, nullptr, nullptr, nullptr, pair_flags_of(pair_mode), nullptr, -1, nullptr, 0 };
    return sync_prepare(a, set, nullptr, st);
}

gs_status momentum_flush(float *w, float *m, int32_t *last, int64_t n_rows, int32_t dim, float lr,
                         float mu, int32_t iter, cudaStream_t st)
{
    if (n_rows == 0) return GS_OK;
    const int64_t total = n_rows * (dim >> 2);
    int64_t blocks = (total + 255) / 256;
    const int64_t cap = (int64_t)sm_count() * 32;
    if (blocks > cap) blocks = cap;
    momentum_flush_kernel<<<(unsigned)blocks, 256, 0, st>>>(w, m, last, n_rows, dim, lr, mu, iter);
    GS_CUDA_TRY(cudaGetLastError());
    int64_t b2 = (n_rows + 255) / 256;
    if (b2 > cap) b2 = cap;
    momentum_stamp_kernel<<<(unsigned)b2, 256, 0, st>>>(last, n_rows, iter);   // once every value is done
    GS_CUDA_TRY(cudaGetLastError());
    return GS_OK;
}

}  // namespace gs


// ---------------------------------------------------------------- fixed-scratch variant
// Scratch of gs_sgns_step_static: part of the library image, so every GPU that loads the
// library holds these bytes until the process exits.  Host code must not hand the symbol
// itself to a kernel (on the host it is only a stand-in); it asks the runtime for the device
// address once per device and passes that.
#define GS_STATIC_SCRATCH_BYTES (32u << 20)
static __device__ __align__(256) unsigned char g_static_scratch[GS_STATIC_SCRATCH_BYTES];

namespace gs {

static std::mutex g_static_mu;
static unsigned char *g_static_ptr[64] = { nullptr };

static gs_status static_scratch_address(unsigned char **out)
{
    int dev = 0;
    GS_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) { set_error("device index %d not supported", dev); return GS_ERR_UNSUPPORTED; }
    std::lock_guard<std::mutex> lk(g_static_mu);
    if (!g_static_ptr[dev]) {
        void *p = nullptr;
        GS_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
        g_static_ptr[dev] = (unsigned char *)p;
    }
    *out = g_static_ptr[dev];
    return GS_OK;
}

}  // namespace gs

extern "C" gs_status gs_sgns_step_static(float *d_w_in, float *d_w_out, int64_t n_nodes, int32_t dim,
                                         const int32_t *d_walks, int64_t n_walks,
                                         int64_t walk_id_base, int32_t walk_len, int32_t window,
                                         int32_t n_neg, const uint64_t *d_alias, float lr,
                                         uint64_t seed, double *d_loss_sum, int64_t *d_pair_count,
                                         void *stream)
{
    using namespace gs;
    if (!d_w_in || !d_w_out) { set_error("invalid argument: table pointer is NULL"); return GS_ERR_INVALID_ARG; }
    if (n_nodes <= 0 || n_nodes >= ((int64_t)1 << 31)) { set_error("invalid argument: n_nodes must be in [1, 2^31)"); return GS_ERR_INVALID_ARG; }
    if (n_walks < 0 || walk_id_base < 0) { set_error("invalid argument: negative n_walks or walk_id_base"); return GS_ERR_INVALID_ARG; }
    if (n_walks > 0 && !d_walks) { set_error("invalid argument: d_walks is NULL"); return GS_ERR_INVALID_ARG; }
    if (n_neg > 0 && !d_alias) { set_error("invalid argument: d_alias is NULL"); return GS_ERR_INVALID_ARG; }
    if (((uintptr_t)d_w_in | (uintptr_t)d_w_out) & 15) { set_error("invalid argument: tables must be 16-byte aligned"); return GS_ERR_INVALID_ARG; }
    if (walk_len < 1 || walk_len > 1024 || window < 1 || window > 32 || n_neg < 0 || n_neg > 32 ||
        2 * window * (1 + n_neg) > 512) {
        set_error("gs_sgns_step_static: walk_len/window/n_neg outside the range gs_sgns_step accepts");
        return GS_ERR_UNSUPPORTED;
    }
    if (n_walks == 0) return GS_OK;
    unsigned char *scratch = nullptr;
    gs_status s = static_scratch_address(&scratch);
    if (s != GS_OK) return s;
    SgnsArgs a = { d_w_in, d_w_out, n_nodes, dim, d_walks, n_walks, walk_id_base, walk_len, window,
                   n_neg, d_alias, lr, seed, d_loss_sum, d_pair_count, nullptr, nullptr, 0, nullptr, -1,
                   nullptr /* this entry point touches no library-owned memory but its array */, 0 };
    cudaStream_t st = (cudaStream_t)stream;
    const FixedScratch fixed = { scratch, (size_t)GS_STATIC_SCRATCH_BYTES };
    switch (dim) {
        case 32: return run_deterministic<32, float>(a, st, nullptr, &fixed);
        case 64: return run_deterministic<64, float>(a, st, nullptr, &fixed);
        case 128: return run_deterministic<128, float>(a, st, nullptr, &fixed);
        case 256: return run_deterministic<256, float>(a, st, nullptr, &fixed);
        default:
            set_error("dim %d not supported (32, 64, 128, 256)", dim);
            return GS_ERR_UNSUPPORTED;
    }
}
