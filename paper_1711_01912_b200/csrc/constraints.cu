// Placement constraints of the candidates (Section 2): collocation constraints (Eq. 3: listed pairs of vertices must
// share a device) and device constraints (Eq. 4: listed (vertex, device) pairs must hold).  Every listed pair is one
// requirement; the kernel counts, per candidate, the requirements that do not hold.
//
// Thread = 4 contiguous candidates (one 32-bit load per id row), block = 128 threads = 512 candidates, grid.y over
// chunks of the constraint lists; the indices of a constraint are the same for the whole block (broadcast loads), the
// id rows are read as coalesced 128-byte segments per warp.  Counts are merged with integer atomic adds.
#include "common.cuh"

namespace tfps {

namespace {

constexpr int CONS_CHUNK = 256;   // constraints per block

__global__ void __launch_bounds__(128)
constraints_kernel(long long P, long long ldp, const uint8_t* __restrict__ part, int npairs, const int* __restrict__ pair_a,
                   const int* __restrict__ pair_b, int ndev, const int* __restrict__ dc_v, const int* __restrict__ dc_d,
                   int* coll_viol, int* dev_viol, const int* status)
{
    if (*status != 0) return;
    const long long j0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (j0 >= P) return;   // ldp is a multiple of 16: a word that starts below P lies inside the row
    const int i0 = blockIdx.y * CONS_CHUNK;
    int cc[4] = {0, 0, 0, 0}, cd[4] = {0, 0, 0, 0};
    if (coll_viol != nullptr) {
        const int i1 = i0 + CONS_CHUNK < npairs ? i0 + CONS_CHUNK : npairs;
        for (int i = i0; i < i1; ++i) {
            const unsigned x = __ldg(reinterpret_cast<const unsigned*>(part + (long long)__ldg(pair_a + i) * ldp + j0)) ^
                               __ldg(reinterpret_cast<const unsigned*>(part + (long long)__ldg(pair_b + i) * ldp + j0));
#pragma unroll
            for (int c = 0; c < 4; ++c) cc[c] += ((x >> (8 * c)) & 0xffu) != 0u;
        }
    }
    if (dev_viol != nullptr) {
        const int i1 = i0 + CONS_CHUNK < ndev ? i0 + CONS_CHUNK : ndev;
        for (int i = i0; i < i1; ++i) {
            const unsigned x = __ldg(reinterpret_cast<const unsigned*>(part + (long long)__ldg(dc_v + i) * ldp + j0));
            const unsigned d = (unsigned)__ldg(dc_d + i);
#pragma unroll
            for (int c = 0; c < 4; ++c) cd[c] += ((x >> (8 * c)) & 0xffu) != d;
        }
    }
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        if (j0 + c < P) {
            if (coll_viol != nullptr && cc[c] != 0) atomicAdd(coll_viol + j0 + c, cc[c]);
            if (dev_viol != nullptr && cd[c] != 0) atomicAdd(dev_viol + j0 + c, cd[c]);
        }
    }
}

}  // namespace

cudaError_t launch_constraints(long long P, long long ldp, const uint8_t* part, int npairs, const int* pair_a, const int* pair_b,
                               int ndev, const int* dc_v, const int* dc_d, int* coll_viol, int* dev_viol, const int* status,
                               cudaStream_t st)
{
    cudaError_t e;
    if (coll_viol && (e = cudaMemsetAsync(coll_viol, 0, sizeof(int) * (size_t)P, st)) != cudaSuccess) return e;
    if (dev_viol && (e = cudaMemsetAsync(dev_viol, 0, sizeof(int) * (size_t)P, st)) != cudaSuccess) return e;
    const int most = std::max(coll_viol ? npairs : 0, dev_viol ? ndev : 0);
    if (most <= 0) return cudaSuccess;
    const dim3 grid((unsigned)((P + 511) / 512), (unsigned)((most + CONS_CHUNK - 1) / CONS_CHUNK));
    constraints_kernel<<<grid, 128, 0, st>>>(P, ldp, part, npairs, pair_a, pair_b, ndev, dc_v, dc_d, coll_viol, dev_viol, status);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace tfps

// ---- critical vertices (Section 3.2) --------------------------------------------------------------------------------
// mask[v][j] = 1 where vertex v lies on a longest source-to-sink path of candidate j: tlevel + blevel == cp.  Thread =
// 2 candidates (16-byte level loads), a block row per vertex; 17 bytes move per vertex-candidate, nothing is reused.
namespace tfps {

namespace {

__global__ void __launch_bounds__(256)
critical_mask_kernel(long long n, long long P, long long ldp, const long long* __restrict__ tlevel,
                     const long long* __restrict__ blevel, const long long* __restrict__ cp, uint8_t* __restrict__ mask)
{
    const long long j0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * 2;
    if (j0 >= P) return;   // ldp is even: the pair of a column below P lies inside the row
    const bool two = j0 + 1 < P;
    const long long c0 = cp[j0], c1 = two ? cp[j0 + 1] : 0;
    for (long long v = blockIdx.y; v < n; v += gridDim.y) {
        const longlong2 t = *reinterpret_cast<const longlong2*>(tlevel + v * ldp + j0);
        const longlong2 b = *reinterpret_cast<const longlong2*>(blevel + v * ldp + j0);
        uint8_t* m = mask + v * ldp + j0;
        if (two) *reinterpret_cast<unsigned short*>(m) = (unsigned short)((t.x + b.x == c0 ? 1u : 0u) | (t.y + b.y == c1 ? 0x100u : 0u));
        else *m = t.x + b.x == c0 ? 1 : 0;
    }
}

}  // namespace

cudaError_t launch_critical_mask(long long n, long long P, long long ldp, const long long* tlevel, const long long* blevel,
                                 const long long* cp, uint8_t* mask, cudaStream_t st)
{
    if (n <= 0 || P <= 0) return cudaSuccess;
    const dim3 grid((unsigned)((P + 511) / 512), (unsigned)std::min<long long>(n, 65535));
    critical_mask_kernel<<<grid, 256, 0, st>>>(n, P, ldp, tlevel, blevel, cp, mask);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace tfps
