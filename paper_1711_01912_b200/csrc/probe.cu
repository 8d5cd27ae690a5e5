// Diagnostic: the rate at which the SMs can gather row segments from L2 / DRAM.
//
// The step-synchronous record passes read, per relaxation, one 8-byte level and one id byte of the neighbour's row for
// every candidate: whole row segments of 1 KiB per warp, rows picked by the graph.  This kernel issues the same access
// pattern without any arithmetic -- every warp reads pseudo-random 1 KiB rows of a buffer, 16 bytes per lane and
// instruction, contiguous across the lanes -- and reports the bytes per second.  On B200 the figure does not depend
// on whether the buffer fits L2, which makes it the ceiling of those passes rather than the DRAM bandwidth.
#include "common.cuh"

namespace tfps {

namespace {

__device__ __forceinline__ unsigned mix32(unsigned x)
{
    x ^= x >> 16; x *= 0x7feb352dU; x ^= x >> 15; x *= 0x846ca68bU; x ^= x >> 16;
    return x;
}

// buf holds `rows` rows of 64 uint4 (1 KiB); every warp reads `iters` rows, `INFLIGHT` at a time
template <int INFLIGHT>
__global__ void __launch_bounds__(128) gather_probe_kernel(const uint4* __restrict__ buf, unsigned rows, int iters, unsigned* sink)
{
    const unsigned warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    unsigned acc = 0;
    for (int it = 0; it < iters; it += INFLIGHT) {
        uint4 a[INFLIGHT][2];
#pragma unroll
        for (int q = 0; q < INFLIGHT; ++q) {
            const unsigned r = mix32(warp * 7919u + (unsigned)(it + q) * 104729u) % rows;
            const uint4* p = buf + (size_t)r * 64 + lane;
            a[q][0] = __ldcg(p);        // bytes [16 * lane, +16) of the row's first half
            a[q][1] = __ldcg(p + 32);   // the same lanes' share of the second half
        }
#pragma unroll
        for (int q = 0; q < INFLIGHT; ++q) acc += a[q][0].x + a[q][0].w + a[q][1].y + a[q][1].z;
    }
    if (acc == 0x12345u) *sink = acc;   // keeps the loads alive
}

// The same with the pass' writes: row r of the buffer is WRITTEN once (1 KiB, by the warp r mod warps, rows in
// ascending order per warp) after `reads` rows picked pseudo-randomly among the `window` rows before it have been read;
// what is written depends on what was read, as in the pass.  The buffer is far larger than L2, the window is not.
// LAYOUT 0: a lane's two 16-byte pieces of a row are 512 bytes apart (every load instruction covers 512 contiguous
// bytes), read past L1; LAYOUT 1: a lane reads 32 contiguous bytes as two loads through L1 (the chained record pass'
// layout: every load instruction touches 32 sectors and uses half of each).
template <int LAYOUT>
__global__ void __launch_bounds__(128)
wavefront_probe_kernel(uint4* buf, unsigned rows, unsigned window, int reads)
{
    const unsigned warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    const unsigned warps = (gridDim.x * blockDim.x) >> 5;
    const unsigned at = LAYOUT == 0 ? lane : 2 * lane, next = LAYOUT == 0 ? 32 : 1;
    for (unsigned r = warp; r < rows; r += warps) {
        uint4 acc0 = make_uint4(r, 0u, 0u, 0u), acc1 = acc0;
        for (int q = 0; q < reads; ++q) {
            const unsigned back = 1u + mix32(r * 31u + (unsigned)q * 104729u) % window;
            if (back > r) continue;
            const uint4* p = buf + (size_t)(r - back) * 64 + at;
            uint4 a, b;
            if (LAYOUT == 0) { a = __ldcg(p); b = __ldcg(p + next); }
            else { a = p[0]; b = p[next]; }
            acc0.x += a.x; acc0.y ^= a.y; acc0.z += a.z; acc0.w ^= a.w;
            acc1.x += b.x; acc1.y ^= b.y; acc1.z += b.z; acc1.w ^= b.w;
        }
        uint4* o = buf + (size_t)r * 64 + at;
        o[0] = acc0;
        o[next] = acc1;
    }
}

}  // namespace

}  // namespace tfps

extern "C" int tfps_probe_wavefront_bandwidth(size_t total_bytes, size_t window_bytes, int reads, int layout, double* gbytes_per_s)
{
    using namespace tfps;
    if (!gbytes_per_s || total_bytes < 1024 || window_bytes < 1024 || reads < 0 || reads > 64 || layout < 0 || layout > 1)
        return TFPS_ERR_INVALID_ARG;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return TFPS_ERR_CUDA;
    void* buf = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    int rc = TFPS_ERR_CUDA;
    const unsigned rows = (unsigned)std::min<size_t>(total_bytes / 1024, 0x7fffffffu);
    const unsigned window = (unsigned)std::max<size_t>(1, std::min<size_t>(window_bytes / 1024, rows));
    const int grid = sms * 8, threads = 128;
    float ms = 0.f;
    if (cudaMalloc(&buf, (size_t)rows * 1024) != cudaSuccess) goto done;
    if (cudaMemset(buf, 1, (size_t)rows * 1024) != cudaSuccess) goto done;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) goto done;
    for (int rep = 0; rep < 3; ++rep) {   // the last repetition is the one reported
        if (cudaEventRecord(e0) != cudaSuccess) goto done;
        if (layout == 0) wavefront_probe_kernel<0><<<grid, threads>>>(static_cast<uint4*>(buf), rows, window, reads);
        else wavefront_probe_kernel<1><<<grid, threads>>>(static_cast<uint4*>(buf), rows, window, reads);
        if (cudaEventRecord(e1) != cudaSuccess || cudaEventSynchronize(e1) != cudaSuccess) goto done;
    }
    count_launches(3);
    if (cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess || ms <= 0.f) goto done;
    *gbytes_per_s = (double)rows * 1024.0 * (reads + 1) / (ms * 1e-3) / 1e9;
    rc = TFPS_OK;
done:
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    if (buf) cudaFree(buf);
    return rc;
}

extern "C" int tfps_probe_gather_bandwidth(size_t working_set_bytes, int rows_per_warp, double* gbytes_per_s)
{
    using namespace tfps;
    if (!gbytes_per_s || working_set_bytes < 1024 || rows_per_warp < 1) return TFPS_ERR_INVALID_ARG;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return TFPS_ERR_CUDA;
    void* buf = nullptr;
    unsigned* sink = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    int rc = TFPS_ERR_CUDA;
    const unsigned rows = (unsigned)std::min<size_t>(working_set_bytes / 1024, 0x7fffffffu);
    const int iters = (rows_per_warp + 1) / 2 * 2;
    const int grid = sms * 8, threads = 128;
    float ms = 0.f;
    if (cudaMalloc(&buf, (size_t)rows * 1024) != cudaSuccess) goto done;
    if (cudaMalloc(&sink, sizeof(unsigned)) != cudaSuccess) goto done;
    if (cudaMemset(buf, 1, (size_t)rows * 1024) != cudaSuccess) goto done;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) goto done;
    for (int rep = 0; rep < 3; ++rep) {   // the last repetition is the one reported
        if (cudaEventRecord(e0) != cudaSuccess) goto done;
        gather_probe_kernel<2><<<grid, threads>>>(static_cast<const uint4*>(buf), rows, iters, sink);
        if (cudaEventRecord(e1) != cudaSuccess || cudaEventSynchronize(e1) != cudaSuccess) goto done;
    }
    count_launches(3);
    if (cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess || ms <= 0.f) goto done;
    *gbytes_per_s = (double)grid * (threads / 32) * iters * 1024.0 / (ms * 1e-3) / 1e9;
    rc = TFPS_OK;
done:
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    if (buf) cudaFree(buf);
    if (sink) cudaFree(sink);
    return rc;
}
