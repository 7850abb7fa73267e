// Measurement aid of bench.py, not part of the library: the rate of INDEPENDENT random 16-byte
// reads over a buffer, issued with the load instruction the walk kernels use (read-only path,
// 64-byte L2 fetch hint).  A walk transition over the walk index is one such read that depends on
// the one before it, so the rate found here is the ceiling for transitions per second of any
// sampler that needs one isolated DRAM access per transition.
//
//   int bench_probe_random_reads(const void *d_records, int64_t n_records, int64_t n_reads,
//                                int64_t *h_reads_done, float *h_ms_out, void *stream)
//
// d_records: device buffer of n_records 16-byte records (contents do not matter).  n_reads is
// rounded up to a multiple of 65,536 (*h_reads_done).  The kernel runs twice; the second run is
// timed with events on `stream` (*h_ms_out).  Waits for completion.  Returns 0, or a cudaError_t.
//
// A second probe gives the ceiling of the update kernels' access pattern: rows of 256 or 512
// bytes of a table, visited at random, each read and written back (16 bytes per lane, the rows of
// a warp's chunk in flight together), with nothing computed in between.
//
//   int bench_probe_row_updates(void *d_table, int64_t n_rows, int32_t row_bytes, const int32_t *d_ids,
//                               int64_t n_visits, int32_t rows_in_flight, int32_t blocks_per_sm,
//                               int32_t write_back, float *h_ms_out, void *stream)
//
// d_table: n_rows rows of row_bytes (256 or 512) bytes, 16-byte aligned; its contents change when
// write_back != 0.  d_ids: n_visits row ids in [0, n_rows) (checked on the device: others are
// skipped).  rows_in_flight: 3 or 6 accesses of a warp in flight (6 or 12 rows of 256 bytes, 3 or
// 6 of 512).  One warm-up launch, one timed one.
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

__device__ __forceinline__ uint64_t mix64(uint64_t x)
{
    x ^= x >> 33; x *= 0xff51afd7ed558ccdull; x ^= x >> 33; x *= 0xc4ceb9fe1a85ec53ull; x ^= x >> 33;
    return x;
}

__device__ __forceinline__ int4 ld_isolated(const int4 *p)
{
    int4 v;
    asm volatile("ld.global.nc.L2::64B.v4.s32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__global__ void __launch_bounds__(256)
random_read_kernel(const int4 *__restrict__ rec, uint64_t n_rec, int iters, unsigned long long *sink)
{
    uint64_t s = mix64((uint64_t)blockIdx.x * blockDim.x + threadIdx.x + 1);
    int acc = 0;
    for (int it = 0; it < iters; it += 4) {
        int4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) { s = mix64(s + u + 1); v[u] = ld_isolated(rec + (s % n_rec)); }
#pragma unroll
        for (int u = 0; u < 4; ++u) acc += v[u].x;
    }
    if (acc == 0x7fffffff) atomicAdd(sink, 1ull);           // keeps the loads alive
}

// LPR lanes per row (16 bytes per lane), G accesses in flight per warp: G * 32 / LPR rows
template <int LPR, int G>
__global__ void __launch_bounds__(128)
row_update_kernel(uint4 *tab, int64_t n_rows, const int32_t *__restrict__ ids, int64_t n, int write_back,
                  unsigned long long *sink)
{
    constexpr int NG = 32 / LPR, CH = G * NG;
    const int lane = threadIdx.x & 31, grp = lane / LPR, sub = lane % LPR;
    const int64_t warp = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5), nw = (int64_t)gridDim.x * 4;
    uint32_t acc = 0;
    for (int64_t i = warp * CH; i < n; i += nw * CH) {
        uint4 r[G];
        int64_t id[G];
#pragma unroll
        for (int q = 0; q < G; ++q) {
            const int64_t e = i + q * NG + grp;
            id[q] = e < n ? (int64_t)ids[e] : -1;
            if (id[q] >= n_rows) id[q] = -1;
        }
#pragma unroll
        for (int q = 0; q < G; ++q)
            if (id[q] >= 0) r[q] = tab[id[q] * LPR + sub];
#pragma unroll
        for (int q = 0; q < G; ++q)
            if (id[q] >= 0) {
                acc += r[q].x;
                if (write_back) { r[q].x += 1u; r[q].y ^= 3u; tab[id[q] * LPR + sub] = r[q]; }
            }
    }
    if (acc == 0x7fffffffu) atomicAdd(sink, 1ull);           // keeps the loads alive
}

}  // namespace

extern "C" __attribute__((visibility("default")))
int bench_probe_row_updates(void *d_table, int64_t n_rows, int32_t row_bytes, const int32_t *d_ids,
                            int64_t n_visits, int32_t rows_in_flight, int32_t blocks_per_sm,
                            int32_t write_back, float *h_ms_out, void *stream)
{
    if (!d_table || !d_ids || !h_ms_out || n_rows < 1 || n_visits < 1 || ((uintptr_t)d_table & 15) ||
        (row_bytes != 256 && row_bytes != 512) || (rows_in_flight != 3 && rows_in_flight != 6) ||
        blocks_per_sm < 1 || blocks_per_sm > 16)
        return (int)cudaErrorInvalidValue;
    cudaStream_t st = (cudaStream_t)stream;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return (int)e;
    unsigned long long *sink = nullptr;
    e = cudaMalloc(&sink, sizeof(*sink));
    if (e != cudaSuccess) return (int)e;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    e = cudaMemsetAsync(sink, 0, sizeof(*sink), st);
    if (e == cudaSuccess) e = cudaEventCreate(&e0);
    if (e == cudaSuccess) e = cudaEventCreate(&e1);
    if (e == cudaSuccess) {
        const unsigned blocks = (unsigned)(sms * blocks_per_sm);
        for (int run = 0; run < 2; ++run) {
            if (run == 1) cudaEventRecord(e0, st);
            uint4 *t = (uint4 *)d_table;
            if (row_bytes == 256 && rows_in_flight == 3) row_update_kernel<16, 3><<<blocks, 128, 0, st>>>(t, n_rows, d_ids, n_visits, write_back, sink);
            else if (row_bytes == 256) row_update_kernel<16, 6><<<blocks, 128, 0, st>>>(t, n_rows, d_ids, n_visits, write_back, sink);
            else if (rows_in_flight == 3) row_update_kernel<32, 3><<<blocks, 128, 0, st>>>(t, n_rows, d_ids, n_visits, write_back, sink);
            else row_update_kernel<32, 6><<<blocks, 128, 0, st>>>(t, n_rows, d_ids, n_visits, write_back, sink);
        }
        cudaEventRecord(e1, st);
        e = cudaEventSynchronize(e1);
        if (e == cudaSuccess) e = cudaEventElapsedTime(h_ms_out, e0, e1);
        if (e == cudaSuccess) e = cudaGetLastError();
    }
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    cudaFree(sink);
    return (int)e;
}

extern "C" __attribute__((visibility("default")))
int bench_probe_random_reads(const void *d_records, int64_t n_records, int64_t n_reads,
                             int64_t *h_reads_done, float *h_ms_out, void *stream)
{
    if (!d_records || !h_reads_done || !h_ms_out || n_records < 1 || n_reads < 1 ||
        n_reads > ((int64_t)1 << 36) || ((uintptr_t)d_records & 15))
        return (int)cudaErrorInvalidValue;
    cudaStream_t st = (cudaStream_t)stream;
    const int iters = 256;
    const int64_t per_block = 256 * (int64_t)iters;
    const int64_t blocks = (n_reads + per_block - 1) / per_block;
    *h_reads_done = blocks * per_block;
    unsigned long long *sink = nullptr;
    cudaError_t e = cudaMalloc(&sink, sizeof(*sink));
    if (e != cudaSuccess) return (int)e;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    e = cudaMemsetAsync(sink, 0, sizeof(*sink), st);
    if (e == cudaSuccess) e = cudaEventCreate(&e0);
    if (e == cudaSuccess) e = cudaEventCreate(&e1);
    if (e == cudaSuccess) {
        random_read_kernel<<<(unsigned)blocks, 256, 0, st>>>((const int4 *)d_records, (uint64_t)n_records, iters, sink);
        cudaEventRecord(e0, st);
        random_read_kernel<<<(unsigned)blocks, 256, 0, st>>>((const int4 *)d_records, (uint64_t)n_records, iters, sink);
        cudaEventRecord(e1, st);
        e = cudaEventSynchronize(e1);
        if (e == cudaSuccess) e = cudaEventElapsedTime(h_ms_out, e0, e1);
    }
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    cudaFree(sink);
    return (int)e;
}
