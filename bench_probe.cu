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

}  // namespace

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
