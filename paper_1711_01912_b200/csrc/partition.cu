// Rank-driven partitioners (Section 3.2): vertex ranks (Eq. 5, Eq. 6), the critical path of the Critical Path strategy
// (Section 3.2.2, steps 1-4), Batch Split (Section 3.2.1) and Critical Path partitioning (Eq. 7).
//
// The ranks are one launch per topological level and direction (a vertex per thread, its in- or out-edges from the
// caller's CSR); they are computed once per graph, not per candidate.  Batch Split sorts vertex ids by (total rank
// descending, id ascending) with a bitonic network on an index array and then places the vertices one after the other;
// placing is sequential by definition (the feasibility of a device depends on what was placed before), so it is one
// warp whose lanes are the devices: a ballot finds the fastest feasible one.  The Critical Path partitioner walks the
// path backwards with one warp (lanes scan a vertex' predecessors), places the path, and then places the other
// vertices with a warp-wide arg-min of Eq. 7 over the devices.  Vertex data of 32 consecutive turns is fetched by the
// 32 lanes at once and handed round by shuffles, so the sequential loops do not wait for memory every turn.
#include "common.cuh"

namespace tfps {

namespace {

constexpr int PART_THREADS = 256;

// Eq. 6 (IN = true: rank over predecessors, sources first) or Eq. 5 (IN = false: over successors, sinks first) for the
// vertices order[q0 .. q1) of one level
__global__ void __launch_bounds__(PART_THREADS)
rank_level_kernel(int q0, int q1, const int* __restrict__ order, const long long* __restrict__ ptr,
                  const int* __restrict__ idx, const int* __restrict__ c, long long* rank)
{
    const int q = q0 + (int)(blockIdx.x * blockDim.x + threadIdx.x);
    if (q >= q1) return;
    const int v = order[q];
    long long best = 0;
    for (long long e = ptr[v]; e < ptr[v + 1]; ++e) {
        const long long r = rank[idx[e]];
        best = r > best ? r : best;
    }
    rank[v] = best + c[v];
}

__global__ void __launch_bounds__(PART_THREADS)
total_rank_kernel(int n, const long long* __restrict__ up, const long long* __restrict__ down, long long* total)
{
    const int v = (int)(blockIdx.x * blockDim.x + threadIdx.x);
    if (v < n) total[v] = up[v] + down[v];
}

}  // namespace

// down (Eq. 6) and up (Eq. 5) of every vertex; level_ptr: host copy of the level boundaries
cudaError_t launch_ranks(int n, const std::vector<long long>& level_ptr, const int* order, const long long* in_ptr,
                         const int* in_src, const long long* out_ptr, const int* out_dst, const int* c, long long* up,
                         long long* down, long long* total, cudaStream_t st)
{
    const int L = (int)level_ptr.size() - 1;
    int launches = 0;
    for (int l = 0; l < L; ++l) {
        const int q0 = (int)level_ptr[l], q1 = (int)level_ptr[l + 1];
        if (q1 > q0) {
            rank_level_kernel<<<(q1 - q0 + PART_THREADS - 1) / PART_THREADS, PART_THREADS, 0, st>>>(q0, q1, order, in_ptr, in_src, c, down);
            ++launches;
        }
    }
    for (int l = L - 1; l >= 0; --l) {
        const int q0 = (int)level_ptr[l], q1 = (int)level_ptr[l + 1];
        if (q1 > q0) {
            rank_level_kernel<<<(q1 - q0 + PART_THREADS - 1) / PART_THREADS, PART_THREADS, 0, st>>>(q0, q1, order, out_ptr, out_dst, c, up);
            ++launches;
        }
    }
    if (n > 0 && total) {
        total_rank_kernel<<<(n + PART_THREADS - 1) / PART_THREADS, PART_THREADS, 0, st>>>(n, up, down, total);
        ++launches;
    }
    count_launches(launches);
    return cudaGetLastError();
}

namespace {

// ---- critical path (Section 3.2.2, steps 1-4) ----------------------------------------------------------------------
// best[0] = largest downward rank of a sink, then best[1] = smallest id among the sinks that have it
__global__ void __launch_bounds__(PART_THREADS)
cp_sink_rank_kernel(int n, const long long* __restrict__ out_ptr, const long long* __restrict__ down, long long* best)
{
    const int v = (int)(blockIdx.x * blockDim.x + threadIdx.x);
    if (v < n && out_ptr[v + 1] == out_ptr[v]) atomicMax(best, down[v]);
}
__global__ void __launch_bounds__(PART_THREADS)
cp_sink_id_kernel(int n, const long long* __restrict__ out_ptr, const long long* __restrict__ down, long long* best)
{
    const int v = (int)(blockIdx.x * blockDim.x + threadIdx.x);
    if (v < n && out_ptr[v + 1] == out_ptr[v] && down[v] == best[0]) atomicMin(best + 1, (long long)v);
}

// one warp: from the chosen sink backwards along predecessors of largest downward rank (equal: smallest id); the path
// is written sink first into path[0 .. len) and turned round by the kernel after this one
__global__ void __launch_bounds__(32)
cp_walk_kernel(int n, const long long* __restrict__ in_ptr, const int* __restrict__ in_src,
               const long long* __restrict__ down, const long long* __restrict__ best, int* path, long long* len)
{
    const int lane = threadIdx.x;
    int v = (int)best[1];
    int cnt = 0;
    while (cnt < n) {
        if (lane == 0) path[cnt] = v;
        ++cnt;
        const long long e0 = in_ptr[v], e1 = in_ptr[v + 1];
        if (e1 == e0) break;
        long long bd = -1;
        int bu = 0x7fffffff;
        for (long long e = e0 + lane; e < e1; e += 32) {
            const int u = in_src[e];
            const long long d = down[u];
            if (d > bd || (d == bd && u < bu)) { bd = d; bu = u; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const long long od = __shfl_xor_sync(0xffffffffu, bd, o);
            const int ou = __shfl_xor_sync(0xffffffffu, bu, o);
            if (od > bd || (od == bd && ou < bu)) { bd = od; bu = ou; }
        }
        v = bu;
    }
    if (lane == 0) *len = cnt;
}
__global__ void __launch_bounds__(PART_THREADS)
reverse_kernel(int* path, const long long* __restrict__ len)
{
    const long long cnt = *len;
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < cnt / 2) {
        const int a = path[i], b = path[cnt - 1 - i];
        path[i] = b;
        path[cnt - 1 - i] = a;
    }
}

}  // namespace

// scratch: three int64 {largest sink rank, chosen sink, path length}; the length is left in scratch[2]
cudaError_t launch_critical_path(int n, const long long* in_ptr, const int* in_src, const long long* out_ptr,
                                 const long long* down, int* path, long long* scratch, cudaStream_t st)
{
    const long long init[3] = {-1, 0x7fffffffffffffffLL, 0};
    cudaError_t e = cudaMemcpyAsync(scratch, init, sizeof(init), cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess || n <= 0) return e;
    const int blocks = (n + PART_THREADS - 1) / PART_THREADS;
    cp_sink_rank_kernel<<<blocks, PART_THREADS, 0, st>>>(n, out_ptr, down, scratch);
    cp_sink_id_kernel<<<blocks, PART_THREADS, 0, st>>>(n, out_ptr, down, scratch);
    cp_walk_kernel<<<1, 32, 0, st>>>(n, in_ptr, in_src, down, scratch, path, scratch + 2);
    reverse_kernel<<<blocks, PART_THREADS, 0, st>>>(path, scratch + 2);   // at most n / 2 swaps
    count_launches(4);
    return cudaGetLastError();
}

namespace {

// ---- Batch Split (Section 3.2.1) -----------------------------------------------------------------------------------
// idx[i] = i for i < n, -1 (sorts last) for the padding up to a power of two
__global__ void __launch_bounds__(PART_THREADS)
iota_kernel(int n, int npad, int* idx)
{
    const int i = (int)(blockIdx.x * blockDim.x + threadIdx.x);
    if (i < npad) idx[i] = i < n ? i : -1;
}
// a comes before b: larger total rank first, equal ranks by ascending id, padding last
__device__ __forceinline__ bool rank_before(int a, int b, const long long* __restrict__ total)
{
    if (b < 0) return a >= 0;
    if (a < 0) return false;
    const long long ta = total[a], tb = total[b];
    return ta > tb || (ta == tb && a < b);
}
// one compare-exchange stage (k, j) of the bitonic network on the index array
__global__ void __launch_bounds__(PART_THREADS)
bitonic_index_kernel(int npad, int k, int j, const long long* __restrict__ total, int* idx)
{
    const int i = (int)(blockIdx.x * blockDim.x + threadIdx.x);
    const int p = i ^ j;
    if (i >= npad || p <= i) return;
    const int a = idx[i], b = idx[p];
    const bool up = (i & k) == 0;   // this stretch is sorted into "comes first" order
    if (up ? rank_before(b, a, total) : rank_before(a, b, total)) {
        idx[i] = b;
        idx[p] = a;
    }
}

// One warp places the vertices in sorted order.  ord[q] = q-th fastest device; lane q (and q + 32) answers for device
// ord[q]: feasible if its memory use stays below its capacity with the vertex on it (Eq. 2), and the first feasible
// lane in speed order wins.  used[] lives in registers: lane q holds the use of ord[q] and ord[q + 32].
__global__ void __launch_bounds__(32)
batch_place_kernel(int n, int k, const int* __restrict__ idx, const long long* __restrict__ mem,
                   const int* __restrict__ ord, const long long* __restrict__ cap, uint8_t* part, long long* unplaced)
{
    const int lane = threadIdx.x;
    const int d0 = lane < k ? ord[lane] : -1, d1 = lane + 32 < k ? ord[lane + 32] : -1;
    const long long c0 = d0 >= 0 ? cap[d0] : 0, c1 = d1 >= 0 ? cap[d1] : 0;
    long long u0 = 0, u1 = 0, bad = 0;
    const int fastest = ord[0];
    for (int base = 0; base < n; base += 32) {
        // the 32 lanes fetch the next 32 turns at once
        const int mine = base + lane < n ? idx[base + lane] : 0;
        const long long mymem = base + lane < n ? mem[mine] : 0;
        const int turns = n - base < 32 ? n - base : 32;
        for (int t = 0; t < turns; ++t) {
            const int v = __shfl_sync(0xffffffffu, mine, t);
            const long long mv = __shfl_sync(0xffffffffu, mymem, t);
            const bool f0 = d0 >= 0 && u0 + mv < c0, f1 = d1 >= 0 && u1 + mv < c1;
            const unsigned b0 = __ballot_sync(0xffffffffu, f0), b1 = __ballot_sync(0xffffffffu, f1);
            int q;   // position in speed order of the chosen device
            if (b0) q = __ffs(b0) - 1;
            else if (b1) q = 32 + __ffs(b1) - 1;
            else { q = 0; ++bad; }
            if (q == lane) u0 += mv;
            if (q == lane + 32) u1 += mv;
            const int dq = q < 32 ? __shfl_sync(0xffffffffu, d0, q) : __shfl_sync(0xffffffffu, d1, q - 32);
            if (lane == 0) part[v] = (uint8_t)(b0 | b1 ? dq : fastest);
        }
    }
    if (lane == 0) *unplaced = bad;
}

}  // namespace

// idx: int [npad] scratch (npad = n rounded up to a power of two); ord: device ids from the fastest to the slowest
cudaError_t launch_batch_split(int n, int npad, int k, const long long* total, const long long* mem, const int* ord,
                               const long long* cap, int* idx, uint8_t* part, long long* unplaced, cudaStream_t st)
{
    if (n <= 0) return cudaMemsetAsync(unplaced, 0, sizeof(long long), st);
    const int blocks = (npad + PART_THREADS - 1) / PART_THREADS;
    int launches = 2;
    iota_kernel<<<blocks, PART_THREADS, 0, st>>>(n, npad, idx);
    for (int kk = 2; kk <= npad; kk <<= 1)
        for (int j = kk >> 1; j > 0; j >>= 1) {
            bitonic_index_kernel<<<blocks, PART_THREADS, 0, st>>>(npad, kk, j, total, idx);
            ++launches;
        }
    batch_place_kernel<<<1, 32, 0, st>>>(n, k, idx, mem, ord, cap, part, unplaced);
    count_launches(launches);
    return cudaGetLastError();
}

namespace {

// ---- Critical Path partitioning (Section 3.2.2, Eq. 7) -------------------------------------------------------------
__global__ void __launch_bounds__(PART_THREADS)
mark_path_kernel(long long len, const int* __restrict__ path, uint8_t* on_path)
{
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < len) on_path[path[i]] = 1;
}

__device__ __forceinline__ long long ceil_div_ll(long long a, long long b) { return (a + b - 1) / b; }

// One warp; lane q answers for devices q and q + 32 (by index here: Eq. 7 breaks ties by the lower index), the speed
// order ord[] is only needed for the path.  used / load of a lane's two devices live in its registers.
__global__ void __launch_bounds__(32)
cp_place_kernel(int n, int k, long long S, const int* __restrict__ path, long long len, const uint8_t* __restrict__ on_path,
                const int* __restrict__ c, const long long* __restrict__ mem, const int* __restrict__ speed,
                const int* __restrict__ ord, const long long* __restrict__ cap, uint8_t* part, long long* unplaced)
{
    const int lane = threadIdx.x;
    const bool h0 = lane < k, h1 = lane + 32 < k;
    const long long s0 = h0 ? speed[lane] : 1, s1 = h1 ? speed[lane + 32] : 1;
    const long long c0 = h0 ? cap[lane] : 0, c1 = h1 ? cap[lane + 32] : 0;
    long long u0 = 0, u1 = 0, l0 = 0, l1 = 0, bad = 0;
    // place vertex v (cost cv, memory mv) on device d
    auto put = [&](int v, int d, long long cv, long long mv) {
        if (d == lane) { u0 += mv; l0 += ceil_div_ll(cv * S, s0); }
        if (d == lane + 32) { u1 += mv; l1 += ceil_div_ll(cv * S, s1); }
        if (lane == 0) part[v] = (uint8_t)d;
    };
    // the path: the fastest device that holds all of it, else vertex by vertex the fastest device with room
    long long path_mem = 0;
    for (long long i = lane; i < len; i += 32) path_mem += mem[path[i]];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) path_mem += __shfl_xor_sync(0xffffffffu, path_mem, o);
    int whole = -1;
    for (int q = 0; q < k && whole < 0; ++q) {
        const int d = ord[q];
        if (path_mem < cap[d]) whole = d;
    }
    for (long long i = 0; i < len; ++i) {
        const int v = path[i];
        const long long mv = mem[v], cv = c[v];
        int chosen = whole;
        if (chosen < 0) {
            const bool f0 = h0 && u0 + mv < c0, f1 = h1 && u1 + mv < c1;
            const unsigned long long feas = (unsigned long long)__ballot_sync(0xffffffffu, f0) |
                                            (unsigned long long)__ballot_sync(0xffffffffu, f1) << 32;   // bit d = device d has room
            for (int q = 0; q < k && chosen < 0; ++q)
                if ((feas >> ord[q]) & 1ull) chosen = ord[q];
            if (chosen < 0) { chosen = ord[0]; ++bad; }
        }
        put(v, chosen, cv, mv);
    }
    // the other vertices in ascending id: arg-min over the feasible devices of load + execution time (Eq. 7)
    const long long BIG = 0x7fffffffffffffffLL;
    for (int base = 0; base < n; base += 32) {
        const int mine = base + lane;
        const bool live = mine < n;
        const long long mymem = live ? mem[mine] : 0;
        const int myc = live ? c[mine] : 0;
        const int skip = live ? on_path[mine] : 1;
        const int turns = n - base < 32 ? n - base : 32;
        for (int t = 0; t < turns; ++t) {
            if (__shfl_sync(0xffffffffu, skip, t)) continue;
            const int v = base + t;
            const long long mv = __shfl_sync(0xffffffffu, mymem, t);
            const long long cv = __shfl_sync(0xffffffffu, myc, t);
            const long long t0 = h0 ? l0 + ceil_div_ll(cv * S, s0) : BIG, t1 = h1 ? l1 + ceil_div_ll(cv * S, s1) : BIG;
            const bool f0 = h0 && u0 + mv < c0, f1 = h1 && u1 + mv < c1;
            const bool any = __any_sync(0xffffffffu, f0 || f1);
            if (!any) ++bad;
            // without a feasible device the rule is applied to all devices
            long long bs = (f0 || (!any && h0)) ? t0 : BIG;
            int bd = lane;
            const long long alt = (f1 || (!any && h1)) ? t1 : BIG;
            if (alt < bs) { bs = alt; bd = lane + 32; }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const long long os = __shfl_xor_sync(0xffffffffu, bs, o);
                const int od = __shfl_xor_sync(0xffffffffu, bd, o);
                if (os < bs || (os == bs && od < bd)) { bs = os; bd = od; }
            }
            put(v, bd, cv, mv);
        }
    }
    if (lane == 0) *unplaced = bad;
}

}  // namespace

// on_path: uint8 [n] scratch; speed: int [k] device speeds; ord: devices from the fastest to the slowest
cudaError_t launch_cp_partition(int n, int k, long long S, const int* path, long long len, const int* c, const long long* mem,
                                const int* speed, const int* ord, const long long* cap, uint8_t* on_path, uint8_t* part,
                                long long* unplaced, cudaStream_t st)
{
    if (n <= 0) return cudaMemsetAsync(unplaced, 0, sizeof(long long), st);
    cudaError_t e = cudaMemsetAsync(on_path, 0, (size_t)n, st);
    if (e != cudaSuccess) return e;
    int launches = 1;
    if (len > 0) {
        mark_path_kernel<<<(unsigned)((len + PART_THREADS - 1) / PART_THREADS), PART_THREADS, 0, st>>>(len, path, on_path);
        ++launches;
    }
    cp_place_kernel<<<1, 32, 0, st>>>(n, k, S, path, len, on_path, c, mem, speed, ord, cap, part, unplaced);
    count_launches(launches);
    return cudaGetLastError();
}

}  // namespace tfps
