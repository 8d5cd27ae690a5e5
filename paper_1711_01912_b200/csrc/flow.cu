// Dataflow form of the record pass (levrec.cu): one persistent launch per pass and NO grid-wide dependency at all.
//
// The work items of a pass are listed in an order in which every item follows the items of the vertices it reads (step
// after step).  The candidates are cut into tiles of 128; a warp owns one tile and walks every S-th item of the list in
// list order (S = warps / tiles item streams), so at any time the grid works on S consecutive items.  Instead of
// waiting for "the whole step before", an item waits for exactly the rows it reads: every vertex has a word of ready
// bits, one per tile, which the warp that has written the vertex' row segment sets (after a fence), and which the
// readers of that segment test.  Most dependencies reach back further than the S items in flight and are found
// resolved; a warp requests the descriptor three items ahead and, two items ahead, the record (cp.async into its own
// ring in shared memory), the ids of the item and of its first two neighbours and the ready words of its first four
// neighbours, and looks at none of them before the item in between is done -- so that the level loads of the next
// item and the fetches for the one after it are in flight while the running item's stores drain (one fence per item,
// which all of them share).
// A vertex cut into partial items (more than the split limit of edges) is ready when the last of them has added its
// maxima (atomicMax) to the zeroed row: a counter per (vertex, tile) finds the last one.
// Progress: the earliest unfinished (item, tile) belongs to a warp that has finished everything before it in its own
// stream, so that warp is working on it, and all it reads is earlier in the list and therefore published -- provided
// every warp of the grid is resident, which the cooperative launch guarantees, and a warp publishes an item before it
// waits for the next.  Every wait is bounded all the same (LevRecArgs::wait_limit polls; TFPS_ERR_TIMEOUT).
// Requirements (host-checked): k <= 16, no separate neighbour runtimes, items of at most eight edges with entries of at
// most 64 bytes, at most 32 tiles (P <= 4,096), ldp >= 128.
#include "common.cuh"
#include "ptx.cuh"

namespace tfps {

namespace {

constexpr int FL_WARPS = 4;
constexpr int FL_MINB = 7;                   // resident blocks per SM asked of the compiler
constexpr int FL_TW = 128;                   // candidates of a tile: four per lane, columns 64 h + 2 lane, + 1 (h = 0, 1)
constexpr int FL_TILES = 32;                 // ready bits per vertex
constexpr int FL_HDR = 16 + 4 * 16;          // record header and runtimes
constexpr int FL_EDGES = 8, FL_ESTRIDE = 64;
constexpr int FL_REC = FL_HDR + FL_EDGES * FL_ESTRIDE + 16;   // 608 bytes: one staged item
constexpr int FL_WARP_SMEM = 128 + 4 * FL_REC;                 // four descriptors, four records

__device__ __forceinline__ unsigned ld_relaxed_gpu(const unsigned* p)
{
    unsigned v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_or_gpu(unsigned* p, unsigned v)
{
    asm volatile("red.relaxed.gpu.global.or.b32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// what a warp fetches ahead of an item's turn, as loaded (nothing here is looked at before the item before it is done)
struct FlowAhead {
    unsigned short own[2], na[2], nb[2];   // ids of the item's row and of its first two neighbours' rows
    unsigned f0, f1, f2, f3;               // ready words of its first four neighbours
};

template <bool FWD>
__global__ void __launch_bounds__(FL_WARPS * 32, FL_MINB)
pass_flow_kernel(const __grid_constant__ LevRecArgs a)
{
    extern __shared__ __align__(16) unsigned char dsm[];   // [warp]{descriptor ring, record ring}
    __shared__ __align__(16) unsigned char s_cls[256];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int i = tid; i < 64; i += FL_WARPS * 32) reinterpret_cast<unsigned*>(s_cls)[i] = __ldg(reinterpret_cast<const unsigned*>(a.cls) + i);
    __syncthreads();   // the only block-wide barrier: from here on every warp is on its own
    if (*reinterpret_cast<volatile int*>(a.status) != 0) return;

    const int P = (int)a.P, ldp = (int)a.ldp;
    const unsigned ldp32 = (unsigned)ldp, ldp8 = (unsigned)ldp * 8u;
    const int tiles = (P + FL_TW - 1) / FL_TW;
    const int gw = (int)blockIdx.x * FL_WARPS + warp;
    const int S = ((int)gridDim.x * FL_WARPS) / tiles;   // item streams
    if (gw >= S * tiles) return;
    const int tile = gw % tiles;                          // the warps of a block work on the same items
    const int col = tile * FL_TW + FL_TW > ldp ? ldp - FL_TW : tile * FL_TW;
    const bool whole = col + FL_TW <= P;
    const unsigned bit = 1u << tile;
    const int nI = a.num_items;
    const int estride = a.estride;
    const int limit = a.wait_limit;
    unsigned* const flags = a.flags;
    const uint8_t* const partc = a.part + col + 2 * lane;
    long long* const levc = a.lev + col + 2 * lane;
    unsigned char* const wsm = dsm + (size_t)warp * FL_WARP_SMEM;
    const unsigned wsm_s = smem_u32(wsm);

    // Item number t of this warp is item gw / tiles + t * S of the list; its descriptor is staged in ring slot t & 3,
    // its record in record slot t & 3.
    auto desc = [&](int slot, int4& it, int4& nb) {
        const int4* d = reinterpret_cast<const int4*>(wsm + 32 * slot);
        it = d[0];
        nb = d[1];
    };
    auto issue_desc = [&](int i, int slot) {
        if (i < nI && lane < 2) cp_async16_ca(wsm_s + 32u * slot + 16u * lane, a.items + 2 * (size_t)i + lane);
    };
    auto issue_rec = [&](const int4& it, int slot) {   // header, runtimes and the item's edge entries
        const unsigned char* rec = a.blob + 16ll * (unsigned)it.y;
        const int first = it.z * estride, chunks = FL_HDR / 16 + (it.w - it.z) * (estride >> 4);
        const unsigned dst = wsm_s + 128u + (unsigned)slot * FL_REC;
        for (int c = lane; c < chunks; c += 32)
            cp_async16_ca(dst + 16u * c, rec + 16 * c + (c < FL_HDR / 16 ? 0 : first));
    };
    // ids of the lane's four candidates in row v, as loaded (two columns per load) ...
    auto ids_raw = [&](unsigned v, unsigned short (&r)[2]) {
        const uint8_t* p = ptr_mad(partc, v, ldp32);
        r[0] = __ldg(reinterpret_cast<const unsigned short*>(p));
        r[1] = __ldg(reinterpret_cast<const unsigned short*>(p + 64));
    };
    // ... and packed: byte c = candidate column 64 (c / 2) + 2 lane + (c & 1)
    auto ids_pack = [&](const unsigned short (&r)[2]) -> unsigned { return ((unsigned)r[0] | (unsigned)r[1] << 16) & 0x0f0f0f0fu; };
    auto fetch_ahead = [&](const int4& it, const int4& nb, FlowAhead& h) {
        const int deg = it.w - it.z;
        ids_raw((unsigned)(it.x & 0x7fffffff), h.own);
        h.f0 = h.f1 = h.f2 = h.f3 = bit;
        h.na[0] = h.na[1] = h.nb[0] = h.nb[1] = 0;
        if (deg > 0) { ids_raw((unsigned)nb.x, h.na); h.f0 = ld_relaxed_gpu(flags + nb.x); }
        if (deg > 1) { ids_raw((unsigned)nb.y, h.nb); h.f1 = ld_relaxed_gpu(flags + nb.y); }
        if (deg > 2) h.f2 = ld_relaxed_gpu(flags + nb.z);
        if (deg > 3) h.f3 = ld_relaxed_gpu(flags + nb.w);
    };
    // bounded wait for vertex u's segment of this tile; false when the wait has run out (or another warp's has)
    auto wait_ready = [&](int u) -> bool {
        bool ready = false;
#pragma unroll 1
        for (int spin = 0; !ready && spin < limit; ++spin) {
            ready = (ld_acquire_gpu(flags + u) & bit) != 0u;
            if (!ready && (spin & 63) == 63 && *reinterpret_cast<volatile int*>(a.status) != 0) break;
        }
        return ready;
    };
    auto wait_first_four = [&](const int4& it, const int4& nb) -> bool {
        const int deg = it.w - it.z;
        if (deg > 0 && !wait_ready(nb.x)) return false;
        if (deg > 1 && !wait_ready(nb.y)) return false;
        if (deg > 2 && !wait_ready(nb.z)) return false;
        if (deg > 3 && !wait_ready(nb.w)) return false;
        return true;
    };
    longlong2 la[2], lb[2];   // levels of the first two neighbours of the item whose turn is next
    auto load_levels = [&](const int4& it, const int4& nb) {
        const int deg = it.w - it.z;
        if (deg > 0) {
            const long long* p = ptr_mad(levc, (unsigned)nb.x, ldp8);
            la[0] = __ldcg(reinterpret_cast<const longlong2*>(p));
            la[1] = __ldcg(reinterpret_cast<const longlong2*>(p + 64));
        }
        if (deg > 1) {
            const long long* p = ptr_mad(levc, (unsigned)nb.y, ldp8);
            lb[0] = __ldcg(reinterpret_cast<const longlong2*>(p));
            lb[1] = __ldcg(reinterpret_cast<const longlong2*>(p + 64));
        }
    };
    auto give_up = [&]() {
        if (lane == 0) atomicCAS(a.status, 0, (int)TFPS_ERR_TIMEOUT);
        cp_async_wait<0>();
    };

    int i0 = gw / tiles;   // the running item; i0 + S, i0 + 2 S follow
    if (i0 >= nI) return;
    unsigned ids0 = 0u, pa0 = 0u, pb0 = 0u;
    FlowAhead ahead;       // of the item after the running one
    {   // the first two items: everything on the spot
        issue_desc(i0, 0);
        issue_desc(i0 + S, 1);
        issue_desc(i0 + 2 * S, 2);
        cp_async_commit();
        cp_async_wait<0>();
        __syncwarp();
        int4 it, nb;
        desc(0, it, nb);
        issue_rec(it, 0);
        fetch_ahead(it, nb, ahead);
        ids0 = ids_pack(ahead.own);
        pa0 = ids_pack(ahead.na);
        pb0 = ids_pack(ahead.nb);
        if (!wait_first_four(it, nb)) { give_up(); return; }
        load_levels(it, nb);
        if (i0 + S < nI) {
            int4 it1, nb1;
            desc(1, it1, nb1);
            issue_rec(it1, 1);
            fetch_ahead(it1, nb1, ahead);
        }
        cp_async_commit();
        __threadfence();   // ready words read above, levels read below
    }
    int slot = 0;
    for (; i0 < nI; i0 += S, slot = (slot + 1) & 3) {
        cp_async_wait<0>();   // this item's record (requested two items ago) and the descriptor two items ahead have landed
        __syncwarp();
        int4 it0, nb0;
        desc(slot, it0, nb0);
        const int deg = it0.w - it0.z;
        const unsigned v = (unsigned)(it0.x & 0x7fffffff);
        const unsigned char* rec = wsm + 128 + slot * FL_REC;
        const unsigned char* edges = rec + FL_HDR;
        long long best[4] = {0, 0, 0, 0};
        auto relax = [&](int e, unsigned pu, const longlong2 (&l)[2]) {
            const unsigned char* ee = edges + e * estride + 8;
            const unsigned x = (pu << 4) | ids0;   // byte c = pu_c * 16 + pv_c
            const long long l4[4] = {l[0].x, l[0].y, l[1].x, l[1].y};
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const unsigned comb = s_cls[(x >> (8 * c)) & 0xffu];
                const long long val = l4[c] + *reinterpret_cast<const long long*>(ee + 8u * comb);
                best[c] = val > best[c] ? val : best[c];
            }
        };
        if (deg > 0) relax(0, pa0, la);
        if (deg > 1) relax(1, pb0, lb);
        bool lost = false;
#pragma unroll 1
        for (int e = 2; e < deg; e += 2) {   // further edges, two at a time: ids and levels requested only now
            const bool two = e + 1 < deg;
            const int u0 = e == 2 ? nb0.z : *reinterpret_cast<const int*>(edges + e * estride);
            const int u1 = !two ? u0 : e == 2 ? nb0.w : *reinterpret_cast<const int*>(edges + (e + 1) * estride);
            if (e >= 4 && (!wait_ready(u0) || !wait_ready(u1))) { lost = true; break; }
            const long long* p0 = ptr_mad(levc, (unsigned)u0, ldp8);
            const long long* p1 = ptr_mad(levc, (unsigned)u1, ldp8);
            longlong2 l0[2], l1[2];
            l0[0] = __ldcg(reinterpret_cast<const longlong2*>(p0));
            l0[1] = __ldcg(reinterpret_cast<const longlong2*>(p0 + 64));
            l1[0] = __ldcg(reinterpret_cast<const longlong2*>(p1));
            l1[1] = __ldcg(reinterpret_cast<const longlong2*>(p1 + 64));
            unsigned short r0[2], r1[2];
            ids_raw((unsigned)u0, r0);
            ids_raw((unsigned)u1, r1);
            relax(e, ids_pack(r0), l0);
            if (two) relax(e + 1, ids_pack(r1), l1);
        }
        if (lost) { give_up(); return; }   // warp-uniform: every lane polls the same words
        if (!FWD) {
            const int* rtv = reinterpret_cast<const int*>(rec + 16);
#pragma unroll
            for (int c = 0; c < 4; ++c) best[c] += rtv[(ids0 >> (8 * c)) & 0xfu];
        }
        long long* out = ptr_mad(levc, v, ldp8);
        const bool partial = it0.x < 0;
        if (whole && !partial) {
            *reinterpret_cast<longlong2*>(out) = make_longlong2(best[0], best[1]);
            *reinterpret_cast<longlong2*>(out + 64) = make_longlong2(best[2], best[3]);
        } else {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int cc = col + 64 * (c >> 1) + 2 * lane + (c & 1);
                if (cc < P) {
                    if (partial) atomicMax(out + 64 * (c >> 1) + (c & 1), best[c]);   // meets the vertex' other items in the zeroed row
                    else out[64 * (c >> 1) + (c & 1)] = best[c];
                }
            }
        }
        // the next item: what was fetched for it one item ago is looked at now; if the rows it reads were ready then
        // (their ready words were read before the previous item's fence), its levels are requested before this item's
        // fence, so that the fence and the loads wait together
        const int i1 = i0 + S, slot1 = (slot + 1) & 3;
        const bool more = i1 < nI;
        int4 it1 = make_int4(0, 0, 0, 0), nb1 = it1;
        ids0 = ids_pack(ahead.own);
        pa0 = ids_pack(ahead.na);
        pb0 = ids_pack(ahead.nb);
        const bool ok1 = (ahead.f0 & ahead.f1 & ahead.f2 & ahead.f3 & bit) != 0u;
        if (more) {
            desc(slot1, it1, nb1);
            if (ok1) load_levels(it1, nb1);
        }
        // two items ahead: record, ids and ready words are requested now and looked at after the next item's turn; the
        // descriptor three items ahead is requested as well
        if (i1 + S < nI) {
            int4 it2, nb2;
            desc((slot + 2) & 3, it2, nb2);
            issue_rec(it2, (slot + 2) & 3);
            fetch_ahead(it2, nb2, ahead);
        }
        issue_desc(i1 + 2 * S, (slot + 3) & 3);
        cp_async_commit();
        // publish: every lane's stores, then the ready bit
        __threadfence();
        __syncwarp();
        if (lane == 0) {
            if (!partial) {
                red_or_gpu(flags + v, bit);
            } else {   // the last of the vertex' items to get here publishes the row
                const int2 aux = __ldg(a.item_aux + i0);
                const int old = atomicAdd(a.part_cnt + (size_t)aux.x * FL_TILES + tile, 1);
                if (old == aux.y - 1) {
                    __threadfence();
                    red_or_gpu(flags + v, bit);
                }
            }
        }
        if (more && !ok1) {   // only now (this item is published) may the warp wait
            if (!wait_first_four(it1, nb1)) { give_up(); return; }
            load_levels(it1, nb1);
        }
    }
    cp_async_wait<0>();
}

template <bool FWD>
cudaError_t flow_launch(const LevRecArgs& a, int sm_count, cudaStream_t st)
{
    auto kernel = pass_flow_kernel<FWD>;
    const size_t smem = (size_t)FL_WARPS * FL_WARP_SMEM;
    int per_sm = 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, FL_WARPS * 32, smem);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) return cudaErrorLaunchOutOfResources;
    if (a.blocks_per_sm > 0 && a.blocks_per_sm < per_sm) per_sm = a.blocks_per_sm;
    const int blocks = per_sm * sm_count;   // all resident (cooperative launch): at least 32 warps, one per tile
    e = cudaMemsetAsync(a.flags, 0, sizeof(unsigned) * (size_t)a.num_vertices, st);
    if (e != cudaSuccess) return e;
    if (a.num_heavy > 0) {
        e = cudaMemsetAsync(a.part_cnt, 0, sizeof(int) * FL_TILES * (size_t)a.num_heavy, st);
        if (e != cudaSuccess) return e;
    }
    LevRecArgs args = a;
    void* params[] = {&args};
    e = cudaLaunchCooperativeKernel((const void*)kernel, dim3((unsigned)blocks), dim3(FL_WARPS * 32), params, smem, st);
    if (e != cudaSuccess) return e;
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace

bool flow_applies(const LevRecArgs& a)
{
    return a.kp == 16 && !a.rtu && a.estride <= FL_ESTRIDE && a.rec_max <= FL_HDR + FL_EDGES * FL_ESTRIDE && a.flags != nullptr &&
           a.item_aux != nullptr && a.P <= FL_TILES * FL_TW && a.ldp >= FL_TW && a.ldp < (1LL << 28) && a.num_steps > 0;
}

cudaError_t launch_pass_flow(const LevRecArgs& a, bool fwd, int sm_count, cudaStream_t st)
{
    return fwd ? flow_launch<true>(a, sm_count, st) : flow_launch<false>(a, sm_count, st);
}

}  // namespace tfps
