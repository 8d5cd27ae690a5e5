// Level-synchronous pass on host-packed vertex records (k <= 16): the variant for graphs whose window does not fit
// shared memory at a useful block width (long edges), where neighbour levels have to come from L2 / DRAM.
//
// One launch per topological level, chained with programmatic dependent launch.  A block takes ONE work item (a
// vertex, or a run of the edges of a vertex with many edges) and LEVREC_WARPS * 128 candidates: it copies the
// vertex' record into shared memory once (its runtimes on every device; per edge the neighbour, the transfer time
// for every distinct bandwidth and, forward, the neighbour's runtimes on every device), then every warp relaxes its
// own 128 candidates: the neighbour's id and level come from global memory (two edges in flight), the class of the
// link from a 16 x 16 byte table, transfer time and neighbour runtime from the record.  No division, no per-edge
// table, one block barrier.  Partial items meet in the output row (zeroed beforehand) through 64-bit atomic maxima.
//   forward:  tlevel(v) = max over in-edges  of tlevel(u) + rt(u, p(u)) + w(u -> v)        (0 for sources)
//   backward: blevel(v) = rt(v, p(v)) + max over out-edges of w(v -> x) + blevel(x)         (Eq. 12)
#include "common.cuh"

namespace tfps {

namespace {

constexpr int LEVREC_WARPS = 4;
// Edges in flight per thread and resident blocks per SM.  Most vertices have one or two edges, so registers are
// better spent on more resident warps than on deeper batches: forward (the edge entry also carries the neighbour's
// runtimes) two edges and 32 warps, backward one edge and 48 warps measured best, in blocks of four warps (config 5,
// forward / backward: 37.5 / 30.3 ms with four edges in flight and 24 warps in blocks of eight, 28.9 / 20.5 ms with
// these depths in blocks of eight, 28.1 / 19.9 ms in blocks of four, 28.9 / 22.0 ms in blocks of two).
template <bool FWD> struct LevRecShape { static constexpr int EB = FWD ? 2 : 1, BLOCKS = FWD ? 8 : 12; };

__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// record of a vertex (16-byte aligned, a multiple of 16 bytes):
//   int4 {vertex, edges, 0, 0}; int rt[16]; then per edge estride bytes:
//   {int neighbour, int pad, long long W[0..ncls] (W[0] = 0), forward only: int rtu[16]}
// item (two int4): {vertex | partial << 31, record offset / 16, first edge within the record, end edge} and the
// neighbours of its first four edges: everything a block needs to start the record copy, the read of its own ids
// and the reads of the first neighbours' ids at once
template <bool FWD>
__global__ void __launch_bounds__(LEVREC_WARPS * 32, LevRecShape<FWD>::BLOCKS)
pass_levrec_kernel(LevRecArgs a, int item0, int count)
{
    constexpr int LEVREC_EB = LevRecShape<FWD>::EB;
    extern __shared__ __align__(16) unsigned char s_rec[];   // header, runtimes and the item's edges
    __shared__ __align__(16) unsigned long long s_rows[2 * LEAN64_K_MAX];   // byte [pv][pu] = 8 * class of the link
    grid_launch_dependents();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool live = *a.status == 0;
    if (tid < 2 * LEAN64_K_MAX) s_rows[tid] = a.rows16[tid];
    const long long j0 = ((long long)blockIdx.x * LEVREC_WARPS + warp) * 128 + lane * 4;
    const long long rem = a.P - j0;
    const int nvalid = rem >= 4 ? 4 : (rem > 0 ? (int)rem : 0);
    const long long jl = nvalid > 0 ? j0 : 0;   // idle lanes read (and drop) column 0
    const long long ldp = a.ldp;
    const int estride = a.estride, wbytes = a.wbytes;
    bool waited = false;

    for (int i = blockIdx.y; i < count && live; i += gridDim.y) {
        const int4 it = __ldg(a.items + 2 * (item0 + i));
        const int4 nb4 = __ldg(a.items + 2 * (item0 + i) + 1);
        const int deg = it.w - it.z;
        const int v = it.x & 0x7fffffff;
        const unsigned char* rec = a.blob + 16ll * (unsigned)it.y;
        // own ids: requested before the record arrives
        const unsigned ids = *reinterpret_cast<const unsigned*>(a.part + (long long)v * ldp + jl) & 0x0f0f0f0fu;
        // ids of the first neighbours: their vertices come with the item, not with the record
        long long off[LEVREC_EB];
        unsigned pu[LEVREC_EB];
        {
            const int nbv[4] = {nb4.x, nb4.y, nb4.z, nb4.w};
#pragma unroll
            for (int q = 0; q < LEVREC_EB; ++q) {
                if (q < deg) {
                    off[q] = (long long)nbv[q] * ldp + jl;
                    pu[q] = *reinterpret_cast<const unsigned*>(a.part + off[q]) & 0x0f0f0f0fu;
                }
            }
        }
        if (i != (int)blockIdx.y) __syncthreads();   // the previous item's record is no longer read
        // header + runtimes (80 bytes), then the item's edges (estride is a multiple of 8)
        for (int q = tid; q < 5; q += LEVREC_WARPS * 32) reinterpret_cast<uint4*>(s_rec)[q] = __ldg(reinterpret_cast<const uint4*>(rec) + q);
        {
            const unsigned long long* src = reinterpret_cast<const unsigned long long*>(rec + 80 + (size_t)it.z * estride);
            unsigned long long* dst = reinterpret_cast<unsigned long long*>(s_rec + 80);
            for (int q = tid; q < deg * (estride >> 3); q += LEVREC_WARPS * 32) dst[q] = __ldg(src + q);
        }
        __syncthreads();
        const int* rtv = reinterpret_cast<const int*>(s_rec + 16);
        const unsigned char* edges = s_rec + 80;
        const unsigned char* row[4];
        long long best[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            row[c] = reinterpret_cast<const unsigned char*>(s_rows) + 16 * ((ids >> (8 * c)) & 0xfu);
            best[c] = 0;
        }
        for (int b0 = 0; b0 < deg; b0 += LEVREC_EB) {
            const int nb = deg - b0 < LEVREC_EB ? deg - b0 : LEVREC_EB;
#pragma unroll
            for (int q = 0; q < LEVREC_EB; ++q) {
                if (b0 > 0 && q < nb) {
                    off[q] = (long long)*reinterpret_cast<const int*>(edges + (size_t)(b0 + q) * estride) * ldp + jl;
                    pu[q] = *reinterpret_cast<const unsigned*>(a.part + off[q]) & 0x0f0f0f0fu;
                }
            }
            if (!waited) { grid_dependency_wait(); waited = true; }   // neighbour levels are the previous launches' output
            longlong2 lu[LEVREC_EB][2];
#pragma unroll
            for (int q = 0; q < LEVREC_EB; ++q) {
                if (q < nb) {
                    const longlong2* p = reinterpret_cast<const longlong2*>(a.lev + off[q]);
                    lu[q][0] = p[0];
                    lu[q][1] = p[1];
                }
            }
#pragma unroll
            for (int q = 0; q < LEVREC_EB; ++q) {
                if (q < nb) {
                    const unsigned char* e = edges + (size_t)(b0 + q) * estride;
                    const long long l4[4] = {lu[q][0].x, lu[q][0].y, lu[q][1].x, lu[q][1].y};
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const unsigned d = (pu[q] >> (8 * c)) & 0xfu;                  // neighbour's device
                        long long val = l4[c] + *reinterpret_cast<const long long*>(e + 8 + row[c][d]);
                        if (FWD) val += *reinterpret_cast<const int*>(e + 8 + wbytes + 4 * d);   // finish time of the neighbour
                        best[c] = val > best[c] ? val : best[c];
                    }
                }
            }
        }
        if (!FWD) {
#pragma unroll
            for (int c = 0; c < 4; ++c) best[c] += rtv[(ids >> (8 * c)) & 0xfu];
        }
        if (!waited) { grid_dependency_wait(); waited = true; }
        long long* out = a.lev + (long long)v * ldp + j0;
        if (it.x < 0) {   // partial item
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (c < nvalid) atomicMax(out + c, best[c]);
        } else if (nvalid == 4) {
            reinterpret_cast<longlong2*>(out)[0] = make_longlong2(best[0], best[1]);
            reinterpret_cast<longlong2*>(out)[1] = make_longlong2(best[2], best[3]);
        } else {
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if (c < nvalid) out[c] = best[c];
        }
    }
    if (!waited) grid_dependency_wait();
}

template <bool FWD>
cudaError_t levrec_impl(const LevRecArgs& a, const std::vector<long long>& ip, int num_levels, cudaStream_t st)
{
    const size_t smem = (size_t)a.rec_max;
    cudaError_t e = cudaFuncSetAttribute(pass_levrec_kernel<FWD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const unsigned gx = (unsigned)((a.P + LEVREC_WARPS * 128 - 1) / (LEVREC_WARPS * 128));
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    for (int step = 0; step < num_levels; ++step) {
        const int l = FWD ? step : num_levels - 1 - step;
        const int item0 = (int)ip[l];
        const int count = (int)(ip[l + 1] - ip[l]);
        unsigned gy = (unsigned)count;
        if (gy > 65535u) gy = 65535u;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(gx, gy);
        cfg.blockDim = dim3(LEVREC_WARPS * 32);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cfg.attrs = attr;
        cfg.numAttrs = step == 0 ? 0 : 1;   // the first level follows ordinary stream order
        e = cudaLaunchKernelEx(&cfg, pass_levrec_kernel<FWD>, a, item0, count);
        if (e != cudaSuccess) return e;
    }
    count_launches(num_levels);
    return cudaGetLastError();
}

}  // namespace

// item_ptr_host: work items of every level (same items as the tile kernel's, edges relative to the vertex' first)
cudaError_t launch_pass_levrec(const LevRecArgs& a, bool fwd, const std::vector<long long>& item_ptr_host, int num_levels,
                               cudaStream_t st)
{
    if (num_levels <= 0) return cudaSuccess;
    return fwd ? levrec_impl<true>(a, item_ptr_host, num_levels, st) : levrec_impl<false>(a, item_ptr_host, num_levels, st);
}

}  // namespace tfps
