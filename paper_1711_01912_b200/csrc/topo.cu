// Topological structure on the GPU: Kahn frontier (cooperative, one grid sync
// per level), canonical (level, id) ordering by a bitonic sort of unique keys,
// level-ordered adjacency, scaled numerators.  A vertex becomes schedulable
// when data on all incoming edges is available (paper, Section 2).
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace tfps {

namespace {

constexpr unsigned FULL = 0xffffffffu;

// All 32 lanes of the warp must call this together.  Lanes with pred append
// `value` behind *counter with a single atomic per warp.
__device__ __forceinline__ void warp_append(bool pred, int value, int* queue, long long base, int* counter)
{
    unsigned mask = __ballot_sync(FULL, pred);
    if (mask == 0) return;
    int lane = threadIdx.x & 31;
    int leader = __ffs(mask) - 1;
    int off = 0;
    if (lane == leader) off = atomicAdd(counter, __popc(mask));
    off = __shfl_sync(FULL, off, leader);
    if (pred) queue[base + off + __popc(mask & ((1u << lane) - 1u))] = value;
}

// level_cnt[l] counts the vertices found for level l (zeroed by the host, one
// counter per level so no counter is ever reused).  result[0] = number of
// levels, result[1] = vertices emitted (n iff the graph is acyclic).
__global__ void __launch_bounds__(256)
kahn_kernel(int n, const long long* __restrict__ in_ptr, const long long* __restrict__ out_ptr,
            const int* __restrict__ out_dst, int* indeg, int* level, int* queue,
            long long* level_ptr, int* level_cnt, long long* result)
{
    cg::grid_group grid = cg::this_grid();
    const int lane = threadIdx.x & 31;
    const long long nthreads = (long long)gridDim.x * blockDim.x;
    const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long warp_base = tid - lane;

    for (long long b = warp_base; b < n; b += nthreads) {
        long long v = b + lane;
        bool src = false;
        if (v < n) {
            int d = (int)(in_ptr[v + 1] - in_ptr[v]);
            indeg[v] = d;
            if (d == 0) { src = true; level[v] = 0; }
        }
        warp_append(src, (int)v, queue, 0, &level_cnt[0]);
    }
    grid.sync();

    long long head = 0;
    long long end = *((volatile int*)&level_cnt[0]);
    int lvl = 0;
    while (end > head) {
        int* cnt = &level_cnt[lvl + 1];
        for (long long b = head + warp_base; b < end; b += nthreads) {
            long long i = b + lane;
            long long e = 0, e_end = 0;
            if (i < end) {
                int u = queue[i];
                e = out_ptr[u];
                e_end = out_ptr[u + 1];
            }
            while (__any_sync(FULL, e < e_end)) {
                bool hit = false;
                int x = 0;
                if (e < e_end) {
                    x = out_dst[e];
                    if (atomicSub(&indeg[x], 1) == 1) { hit = true; level[x] = lvl + 1; }
                    ++e;
                }
                warp_append(hit, x, queue, end, cnt);
            }
        }
        grid.sync();
        int found = *((volatile int*)cnt);
        if (tid == 0) level_ptr[lvl + 1] = end;
        head = end;
        end += found;
        ++lvl;
    }
    if (tid == 0) {
        level_ptr[0] = 0;
        result[0] = lvl;
        result[1] = end;
    }
}

// ---- canonical order: sort unique keys (level << 32 | vertex) --------------
__global__ void make_keys(int n, int npad, const int* __restrict__ level, unsigned long long* keys)
{
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= npad) return;
    keys[i] = i < n ? (((unsigned long long)(unsigned)level[i] << 32) | (unsigned)i) : ~0ull;
}

constexpr int SORT_TILE = 1024;  // elements per block in the shared-memory stages

__device__ __forceinline__ void cmp_swap(unsigned long long& a, unsigned long long& b, bool asc)
{
    if ((a > b) == asc) { unsigned long long t = a; a = b; b = t; }
}

// Runs, inside each tile of SORT_TILE keys, the merge stages j = j_start..1 of
// bitonic phase k; with k_first <= k_last it runs whole phases k_first..k_last
// (used for the phases that fit a tile).
__global__ void __launch_bounds__(SORT_TILE / 2)
bitonic_local(unsigned long long* keys, int k_first, int k_last, int j_start)
{
    __shared__ unsigned long long s[SORT_TILE];
    const int base = blockIdx.x * SORT_TILE;
    const int t = threadIdx.x;
    s[t] = keys[base + t];
    s[t + SORT_TILE / 2] = keys[base + t + SORT_TILE / 2];
    __syncthreads();
    for (int k = k_first; k <= k_last; k <<= 1) {
        int j0 = (k_first == k_last) ? j_start : (k >> 1);
        for (int j = j0; j > 0; j >>= 1) {
            int i = ((t & ~(j - 1)) << 1) | (t & (j - 1));  // lower index of the pair
            bool asc = (((base + i) & k) == 0);
            cmp_swap(s[i], s[i | j], asc);
            __syncthreads();
        }
    }
    keys[base + t] = s[t];
    keys[base + t + SORT_TILE / 2] = s[t + SORT_TILE / 2];
}

__global__ void bitonic_global(unsigned long long* keys, int npad, int k, int j)
{
    int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= npad / 2) return;
    int i = ((t & ~(j - 1)) << 1) | (t & (j - 1));
    bool asc = ((i & k) == 0);
    unsigned long long a = keys[i], b = keys[i | j];
    if ((a > b) == asc) { keys[i] = b; keys[i | j] = a; }
}

__global__ void keys_to_order(int n, const unsigned long long* __restrict__ keys, int* order)
{
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) order[i] = (int)(unsigned)(keys[i] & 0xffffffffu);
}

// ---- level-ordered adjacency ------------------------------------------------
// eptr[0..n] = exclusive prefix sum of the degrees taken in position order.
// One block; the tile loop carries the running total.
__global__ void __launch_bounds__(1024)
degree_scan(int n, const int* __restrict__ order, const long long* __restrict__ ptr, int* eptr)
{
    __shared__ int warp_sums[32];
    __shared__ int carry;
    const int t = threadIdx.x, lane = t & 31, w = t >> 5;
    if (t == 0) carry = 0;
    __syncthreads();
    for (int base = 0; base < n; base += 1024) {
        int i = base + t;
        int d = 0;
        if (i < n) { int v = order[i]; d = (int)(ptr[v + 1] - ptr[v]); }
        int x = d;
        for (int o = 1; o < 32; o <<= 1) { int y = __shfl_up_sync(FULL, x, o); if (lane >= o) x += y; }
        if (lane == 31) warp_sums[w] = x;
        __syncthreads();
        if (w == 0) {
            int s = warp_sums[lane];
            for (int o = 1; o < 32; o <<= 1) { int y = __shfl_up_sync(FULL, s, o); if (lane >= o) s += y; }
            warp_sums[lane] = s;
        }
        __syncthreads();
        int excl = carry + (w ? warp_sums[w - 1] : 0) + x - d;
        if (i < n) eptr[i] = excl;
        __syncthreads();
        if (t == 1023) carry = excl + d;
        __syncthreads();
    }
    if (t == 0) eptr[n] = carry;
}

// one warp per position copies the vertex's CSR row behind eptr[i]
__global__ void fill_adj(int n, const int* __restrict__ order, const long long* __restrict__ ptr,
                         const int* __restrict__ idx, const long long* __restrict__ t,
                         const int* __restrict__ eptr, int* nbr, long long* tperm)
{
    long long gw = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int lane = threadIdx.x & 31;
    if (gw >= n) return;
    int v = order[gw];
    long long s = ptr[v];
    int d = (int)(ptr[v + 1] - s);
    int o = eptr[gw];
    for (int j = lane; j < d; j += 32) {
        nbr[o + j] = idx[s + j];
        tperm[o + j] = t[s + j];
    }
}

__global__ void sink_flags_kernel(int n, const int* __restrict__ order, const long long* __restrict__ out_ptr, uint8_t* flag)
{
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) { int v = order[i]; flag[i] = out_ptr[v + 1] == out_ptr[v] ? 1 : 0; }
}

__global__ void vertf_kernel(int n, const int* __restrict__ order, const uint8_t* __restrict__ sink_flag, int* vertf)
{
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) vertf[i] = order[i] | (sink_flag[i] ? (int)0x80000000 : 0);
}

__device__ __forceinline__ unsigned long long numerator(long long a)
{
    return a == 0 ? NUM_ZERO : ((unsigned long long)(a - 1) << 2);
}

__global__ void numerators_vertex(int n, long long S, const int* __restrict__ order, const int* __restrict__ c,
                                  unsigned long long* xvert)
{
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) xvert[i] = numerator((long long)c[order[i]] * S);
}

__global__ void numerators_edge(int m, long long S, const long long* __restrict__ t, const int* __restrict__ nbr,
                                const int* __restrict__ c, unsigned long long* xw, unsigned long long* xnbr)
{
    int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= m) return;
    xw[e] = numerator(t[e] * S);
    if (xnbr) xnbr[e] = numerator((long long)c[nbr[e]] * S);
}

__global__ void default_mem_kernel(int n, const long long* __restrict__ out_ptr, const long long* __restrict__ out_t,
                                   long long* mem)
{
    int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= n) return;
    long long acc = 0;
    for (long long e = out_ptr[v]; e < out_ptr[v + 1]; ++e) acc += out_t[e];
    mem[v] = acc;
}

inline int cdiv(long long a, long long b) { return (int)((a + b - 1) / b); }

}  // namespace

cudaError_t launch_kahn(int n, const long long* in_ptr, const long long* out_ptr, const int* out_dst,
                        int* indeg, int* level, int* queue, long long* level_ptr_dev, int* level_cnt,
                        long long* result, int sm_count, cudaStream_t st)
{
    int per_sm = 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kahn_kernel, 256, 0);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) return cudaErrorLaunchOutOfResources;
    long long want = (long long)n / 8192 + 1;
    long long cap = (long long)per_sm * sm_count;
    int blocks = (int)(want < cap ? want : cap);
    if (blocks > sm_count) blocks = sm_count;
    if (blocks < 1) blocks = 1;
    void* args[] = {&n, &in_ptr, &out_ptr, &out_dst, &indeg, &level, &queue, &level_ptr_dev, &level_cnt, &result};
    count_launches(1);
    return cudaLaunchCooperativeKernel((void*)kahn_kernel, dim3(blocks), dim3(256), args, 0, st);
}

cudaError_t launch_sort_order(int n, const int* level, unsigned long long* keys, int npad, int* order, cudaStream_t st)
{
    long long launches = 3;
    make_keys<<<cdiv(npad, 256), 256, 0, st>>>(n, npad, level, keys);
    int tiles = npad / SORT_TILE;  // npad is a power of two >= SORT_TILE
    int k_local_max = SORT_TILE;
    bitonic_local<<<tiles, SORT_TILE / 2, 0, st>>>(keys, 2, k_local_max, 0);
    for (int k = SORT_TILE * 2; k <= npad; k <<= 1) {
        for (int j = k >> 1; j >= SORT_TILE; j >>= 1) {
            bitonic_global<<<cdiv(npad / 2, 256), 256, 0, st>>>(keys, npad, k, j);
            ++launches;
        }
        bitonic_local<<<tiles, SORT_TILE / 2, 0, st>>>(keys, k, k, SORT_TILE / 2);
        ++launches;
    }
    keys_to_order<<<cdiv(n, 256), 256, 0, st>>>(n, keys, order);
    count_launches(launches);
    return cudaGetLastError();
}

cudaError_t launch_build_adj(int n, const int* order, const long long* ptr, const int* idx, const long long* t,
                             int* eptr, int* nbr, long long* tperm, cudaStream_t st)
{
    degree_scan<<<1, 1024, 0, st>>>(n, order, ptr, eptr);
    fill_adj<<<cdiv((long long)n * 32, 256), 256, 0, st>>>(n, order, ptr, idx, t, eptr, nbr, tperm);
    count_launches(2);
    return cudaGetLastError();
}

cudaError_t launch_sink_flags(int n, const int* order, const long long* out_ptr, uint8_t* flag, cudaStream_t st)
{
    if (n > 0) { sink_flags_kernel<<<cdiv(n, 256), 256, 0, st>>>(n, order, out_ptr, flag); count_launches(1); }
    return cudaGetLastError();
}

cudaError_t launch_vertf(int n, const int* order, const uint8_t* sink_flag, int* vertf, cudaStream_t st)
{
    if (n > 0) { vertf_kernel<<<cdiv(n, 256), 256, 0, st>>>(n, order, sink_flag, vertf); count_launches(1); }
    return cudaGetLastError();
}

cudaError_t launch_numerators(int n, int m, long long S, const int* order, const int* c,
                              const int* nbr_f, const long long* t_f, const int* nbr_b, const long long* t_b,
                              unsigned long long* xvert, unsigned long long* xw_f, unsigned long long* xnbr_f,
                              unsigned long long* xw_b, cudaStream_t st)
{
    if (n > 0) { numerators_vertex<<<cdiv(n, 256), 256, 0, st>>>(n, S, order, c, xvert); count_launches(1); }
    if (m > 0) {
        count_launches(2);
        numerators_edge<<<cdiv(m, 256), 256, 0, st>>>(m, S, t_f, nbr_f, c, xw_f, xnbr_f);
        numerators_edge<<<cdiv(m, 256), 256, 0, st>>>(m, S, t_b, nbr_b, c, xw_b, nullptr);
    }
    return cudaGetLastError();
}

cudaError_t launch_default_mem(int n, const long long* out_ptr, const long long* out_t, long long* mem, cudaStream_t st)
{
    if (n > 0) { default_mem_kernel<<<cdiv(n, 256), 256, 0, st>>>(n, out_ptr, out_t, mem); count_launches(1); }
    return cudaGetLastError();
}

namespace {

__global__ void pos_of_kernel(int n, const int* __restrict__ order, int* pos_of)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) pos_of[order[i]] = i;
}

// the longest in-edge in level positions: one thread per position walks its in-edges
__global__ void maxspan_kernel(int n, const int* __restrict__ pos_of, const int* __restrict__ eptr_f,
                               const int* __restrict__ nbr_f, int* maxspan)
{
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= n) return;
    int mx = 0;
    for (int q = eptr_f[p]; q < eptr_f[p + 1]; ++q) {
        const int s = p - pos_of[nbr_f[q]];
        mx = s > mx ? s : mx;
    }
    if (mx > 0) atomicMax(maxspan, mx);
}

}  // namespace

// pos_of[v] = level position of vertex v; *maxspan (zeroed by the caller) = largest pos(v) - pos(u) over all edges u -> v
cudaError_t launch_positions(int n, const int* order, int* pos_of, const int* nbr_f, const int* eptr_f, int* maxspan,
                             cudaStream_t st)
{
    if (n <= 0) return cudaSuccess;
    pos_of_kernel<<<cdiv(n, 256), 256, 0, st>>>(n, order, pos_of);
    maxspan_kernel<<<cdiv(n, 256), 256, 0, st>>>(n, pos_of, eptr_f, nbr_f, maxspan);
    count_launches(2);
    return cudaGetLastError();
}

}  // namespace tfps
