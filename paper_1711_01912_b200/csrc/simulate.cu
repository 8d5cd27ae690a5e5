// Batched list-scheduling simulation (Section 4, criteria 1-6; the event-based simulation of Section 5): every
// candidate partition is simulated on its own, one warp per candidate.
//
// A device executes its vertices one at a time without interruption; a vertex is executable once every predecessor
// has finished and its tensor has arrived (ready = max over in-edges of finish + transfer time, transfers do not
// queue); an idle device with an executable vertex starts one at once: FIFO takes the one that became executable first,
// PCT the one with the largest path computation time (Eq. 12, the blevel matrix of tfps_eval_batch), MSR the one with
// the largest successor rank (Eq. 13, computed from the out-edges when the device decides); equal keys go to the
// smaller vertex id.  Events are taken in time order: at a time T every execution that ends at T is completed,
// then every idle device starts its best executable vertex, and the two steps repeat at T while executions of zero
// length keep ending.
//
// The simulation of one candidate is sequential in time, so the parallelism is across candidates (a warp each) and,
// inside a warp, across the entries of a device's pending list (the lanes scan it for the best executable vertex and
// for the earliest future one) and across the out-edges of a finishing vertex.  Per candidate the warp keeps, in its
// own slice of a scratch buffer, ready[v] (int64), the number of unfinished predecessors left[v] and the pending
// lists (one array of n vertex ids cut into per-device regions by a counting pass); the per-device state (region,
// fill, running vertex, end of its execution) lives in the warp's shared memory.
#include "common.cuh"

namespace tfps {

namespace {

constexpr int SIM_WARPS = 4;   // warps (candidates in flight) per block

struct SimDev {                // per warp
    int first[64], count[64], run[64];
    long long busy[64];
};

__device__ __forceinline__ long long ceil_div_pos(long long a, long long b) { return (a + b - 1) / b; }

// lexicographic minimum of (a, b, at) over the warp
__device__ __forceinline__ void warp_min3(long long& a, int& b, int& at)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const long long oa = __shfl_xor_sync(0xffffffffu, a, o);
        const int ob = __shfl_xor_sync(0xffffffffu, b, o);
        const int oat = __shfl_xor_sync(0xffffffffu, at, o);
        if (oa < a || (oa == a && ob < b)) { a = oa; b = ob; at = oat; }
    }
}

struct SimArgs {
    int n, k;
    long long P, ldp, S;
    const uint8_t* part;          // [n][ldp]
    const long long* in_ptr;      // caller's CSR
    const long long* out_ptr;
    const int* out_dst;
    const long long* out_t;
    const int* c;
    const int* speed;             // [k]
    const long long* B;           // [k][k] row = source device
    int policy;                   // 0 FIFO, 1 PCT, 2 MSR
    long long w_alpha, w_beta, w_gamma, w_delta;   // MSR weights (Eq. 13)
    const long long* prio;        // [n][ldp] (PCT)
    long long* start;             // [n][ldp] or null
    long long* makespan;          // [P]
    long long* ready;             // scratch [warps][n]
    int* left;                    // scratch [warps][n]
    int* list;                    // scratch [warps][n]
    int* status;
};

__global__ void __launch_bounds__(SIM_WARPS * 32)
simulate_kernel(const SimArgs a)
{
    __shared__ SimDev s_dev[SIM_WARPS];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gw = (int)blockIdx.x * SIM_WARPS + warp, GW = (int)gridDim.x * SIM_WARPS;
    SimDev& D = s_dev[warp];
    const int n = a.n, k = a.k;
    long long* const ready = a.ready + (size_t)gw * n;
    int* const left = a.left + (size_t)gw * n;
    int* const list = a.list + (size_t)gw * n;
    const long long BIG = 0x7fffffffffffffffLL;

    for (long long j = gw; j < a.P; j += GW) {
        const uint8_t* const pj = a.part + j;
        // regions of the pending lists: how many vertices every device has
        for (int d = lane; d < 64; d += 32) { D.count[d] = 0; D.run[d] = -1; D.busy[d] = 0; }
        __syncwarp();
        bool bad_id = false;
        for (int v = lane; v < n; v += 32) {
            const int d = pj[(size_t)v * a.ldp];
            if (d >= k) { bad_id = true; continue; }
            atomicAdd(&D.count[d], 1);
            ready[v] = 0;
            left[v] = (int)(a.in_ptr[v + 1] - a.in_ptr[v]);
        }
        if (__any_sync(0xffffffffu, bad_id)) {   // ids beyond k: the candidate is not simulated
            if (lane == 0) { atomicCAS(a.status, 0, (int)TFPS_ERR_BAD_PARTITION); a.makespan[j] = -1; }
            __syncwarp();
            continue;
        }
        __syncwarp();
        if (lane == 0) {
            int acc = 0;
            for (int d = 0; d < k; ++d) { D.first[d] = acc; acc += D.count[d]; D.count[d] = 0; }
        }
        __syncwarp();
        for (int v = lane; v < n; v += 32) {
            if (left[v] == 0) {
                const int d = pj[(size_t)v * a.ldp];
                list[D.first[d] + atomicAdd(&D.count[d], 1)] = v;
            }
        }
        __syncwarp();
        long long T = 0, last = 0;
        int done = 0;
        bool stuck = false;
        while (done < n) {
            // every idle device that has pending vertices looks for its best executable one (lane d answers for the
            // devices d and d + 32; only the devices that have something to decide are visited)
            long long next = BIG;
            // MSR looks at which devices execute nothing as this step begins (Eq. 13: idle successors' devices)
            const unsigned long long idle_then =
                (unsigned long long)__ballot_sync(0xffffffffu, lane < k && D.run[lane] < 0) |
                (unsigned long long)__ballot_sync(0xffffffffu, lane + 32 < k && D.run[lane + 32] < 0) << 32;
            const unsigned want0 = __ballot_sync(0xffffffffu, lane < k && D.run[lane] < 0 && D.count[lane] > 0);
            const unsigned want1 = __ballot_sync(0xffffffffu, lane + 32 < k && D.run[lane + 32] < 0 && D.count[lane + 32] > 0);
            for (int half = 0; half < 2; ++half) {
                unsigned want = half ? want1 : want0;
                while (want) {
                    const int d = 32 * half + __ffs(want) - 1;
                    want &= want - 1;
                    const int cnt = D.count[d], f = D.first[d];
                    long long key = BIG, soon = BIG;
                    int id = 0x7fffffff, at = -1;
                    for (int i = lane; i < cnt; i += 32) {
                        const int v = __ldcg(list + f + i);
                        const long long r = __ldcg(ready + v);   // updated by atomics: read where they are performed
                        if (r > T) { soon = r < soon ? r : soon; continue; }
                        long long kv;
                        if (a.policy == 0) {
                            kv = r;
                        } else if (a.policy == 1) {
                            kv = -a.prio[(size_t)v * a.ldp + j];
                        } else {   // Eq. 13, summed over the out-edges
                            long long sc = 0;
                            for (long long e = a.out_ptr[v]; e < a.out_ptr[v + 1]; ++e) {
                                const int x = a.out_dst[e];
                                const int dx = pj[(size_t)x * a.ldp];
                                const bool single = a.in_ptr[x + 1] - a.in_ptr[x] == 1;
                                sc += a.w_alpha + (dx != d ? a.w_beta : 0) + (single ? a.w_gamma : 0) +
                                      (single && ((idle_then >> dx) & 1ull) ? a.w_delta : 0);
                            }
                            kv = -sc;
                        }
                        if (kv < key || (kv == key && v < id)) { key = kv; id = v; at = i; }
                    }
                    warp_min3(key, id, at);
                    if (at < 0) {   // nothing executable yet: the device idles until its earliest vertex is
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) {
                            const long long os = __shfl_xor_sync(0xffffffffu, soon, o);
                            soon = os < soon ? os : soon;
                        }
                        next = soon < next ? soon : next;
                        continue;
                    }
                    const int v = id;
                    const long long fin = T + ceil_div_pos((long long)a.c[v] * a.S, a.speed[d]);
                    if (lane == 0) {
                        list[f + at] = __ldcg(list + f + cnt - 1);
                        D.count[d] = cnt - 1;
                        D.run[d] = v;
                        D.busy[d] = fin;
                        if (a.start) a.start[(size_t)v * a.ldp + j] = T;
                    }
                }
            }
            __syncwarp();
            {   // the earliest end of a running execution
                long long mine = lane < k && D.run[lane] >= 0 ? D.busy[lane] : BIG;
                const long long other = lane + 32 < k && D.run[lane + 32] >= 0 ? D.busy[lane + 32] : BIG;
                mine = other < mine ? other : mine;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    const long long om = __shfl_xor_sync(0xffffffffu, mine, o);
                    mine = om < mine ? om : mine;
                }
                next = mine < next ? mine : next;
            }
            if (next == BIG) { stuck = true; break; }   // nothing runs and nothing is pending (cannot happen on a DAG)
            T = next;
            // executions that end at T
            const unsigned end0 = __ballot_sync(0xffffffffu, lane < k && D.run[lane] >= 0 && D.busy[lane] == T);
            const unsigned end1 = __ballot_sync(0xffffffffu, lane + 32 < k && D.run[lane + 32] >= 0 && D.busy[lane + 32] == T);
            for (int half = 0; half < 2; ++half) {
                unsigned ends = half ? end1 : end0;
                while (ends) {
                    const int d = 32 * half + __ffs(ends) - 1;
                    ends &= ends - 1;
                    const int u = D.run[d];
                    __syncwarp();
                    if (lane == 0) D.run[d] = -1;
                    ++done;
                    last = T;
                    const long long e0 = a.out_ptr[u], e1 = a.out_ptr[u + 1];
                    for (long long e = e0 + lane; e < e1; e += 32) {
                        const int x = a.out_dst[e];
                        const int dx = pj[(size_t)x * a.ldp];
                        const long long w = dx == d ? 0 : ceil_div_pos(a.out_t[e] * a.S, a.B[(size_t)d * k + dx]);
                        atomicMax(&ready[x], T + w);
                        __threadfence_block();
                        if (atomicSub(&left[x], 1) == 1) list[D.first[dx] + atomicAdd(&D.count[dx], 1)] = x;
                    }
                    __syncwarp();
                }
            }
        }
        if (lane == 0) {
            a.makespan[j] = stuck ? -1 : last;
            if (stuck) atomicCAS(a.status, 0, (int)TFPS_ERR_CYCLE);
        }
        __syncwarp();
    }
}

}  // namespace

// scratch: ready int64 [warps][n], left int [warps][n], list int [warps][n] for warps = blocks * 4
cudaError_t launch_simulate(int n, int k, long long P, long long ldp, long long S, const uint8_t* part,
                            const long long* in_ptr, const long long* out_ptr, const int* out_dst, const long long* out_t,
                            const int* c, const int* speed, const long long* B, int policy, const long long* prio,
                            const long long* msr_w, long long* start, long long* makespan, int blocks, long long* ready,
                            int* left, int* list, int* status, cudaStream_t st)
{
    SimArgs a;
    a.w_alpha = msr_w[0]; a.w_beta = msr_w[1]; a.w_gamma = msr_w[2]; a.w_delta = msr_w[3];
    a.n = n; a.k = k; a.P = P; a.ldp = ldp; a.S = S; a.part = part;
    a.in_ptr = in_ptr; a.out_ptr = out_ptr; a.out_dst = out_dst; a.out_t = out_t; a.c = c; a.speed = speed; a.B = B;
    a.policy = policy; a.prio = prio; a.start = start; a.makespan = makespan;
    a.ready = ready; a.left = left; a.list = list; a.status = status;
    simulate_kernel<<<blocks, SIM_WARPS * 32, 0, st>>>(a);
    count_launches(1);
    return cudaGetLastError();
}

int simulate_warps_per_block() { return SIM_WARPS; }

}  // namespace tfps
