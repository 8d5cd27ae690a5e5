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

}  // namespace

}  // namespace tfps

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
