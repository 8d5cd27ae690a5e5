// Persistent step-synchronous pass on host-packed vertex records (k <= 64): the variant for graphs whose window does
// not fit shared memory at a useful block width (long edges), where neighbour levels come from L2.
//
// One cooperative launch per pass.  The vertices are cut into steps (topological levels, or runs of consecutive
// vertices of the caller's numbering when that is a topological order with shorter edges): all vertices of a step
// are independent, and a vertex' neighbours lie in earlier steps.  The candidate columns of a walk over the steps are
// split into G phases; EVERY block works on every phase in turn: it evaluates its share of (step s, phase 0), signals
// a counter of that phase in global memory, goes on with (s, phase 1) ... and only then waits for all blocks to have
// signalled (s, phase 0) before it starts (s + 1, phase 0).  The latency of the grid-wide barrier of one phase is
// hidden behind the work of the others.  The cooperative launch guarantees that all blocks are resident, and every
// wait is bounded.  A walk covers G * tiles_per_phase tiles of 128 candidates, narrow enough for the rows still in
// use to stay in L2; then the next walk starts.
//
// A warp owns one tile of every phase (4 candidates per lane) and every nil-th work item of a step.  A work item is
// a vertex, or a run of at most `split` edges of a vertex with many edges (partial items meet in the output row,
// zeroed beforehand, through 64-bit atomic maxima).  The item's record -- per edge the neighbour and the edge cost for
// every combination of link class and speed class of the neighbour's device -- is copied into the warp's own
// shared-memory ring by cp.async two units ahead; neighbour ids and levels are read from global memory (levels with
// ld.global.cg: they are written during the launch) one edge pair ahead of their use.  No division, no per-edge
// table, no block barrier inside a phase.
//   forward:  tlevel(v) = max over in-edges  of tlevel(u) + rt(u, p(u)) + w(u -> v)        (0 for sources)
//   backward: blevel(v) = rt(v, p(v)) + max over out-edges of w(v -> x) + blevel(x)         (Eq. 12)
#include "common.cuh"
#include "ptx.cuh"

namespace tfps {

namespace {

// record of a vertex (16-byte aligned, a multiple of 16 bytes):
//   int4 {vertex, edges, 0, 0}; int rt[KP]; then per edge `estride` bytes (a multiple of 16):
//   {int neighbour, int pad, long long V[ncomb], RTU only: int rtu[KP]}
//   V[comb]: backward comb = class of the link (0 = same device), V = transfer time;
//            forward  comb = class * speed classes + speed class of the neighbour's device, V = transfer time + the
//            neighbour's runtime on such a device; RTU form (too many combinations): comb = class, V = transfer
//            time, and rtu[d] = the neighbour's runtime on device d is added separately.
// cls[pu * KP + pv] = comb of a neighbour on device pu and a vertex on device pv.
// item (two int4): {vertex | partial << 31, record offset / 16, first edge within the record, end edge} and the
// neighbours of the item's first four edges (the chained kernel starts their loads before the record has arrived)
//
// A lane holds 2 * CG candidates of its warp's tile (tile width TW = 64 * CG): columns {2 * lane, 2 * lane + 1} of
// each of the CG 64-column groups, so that every 16-byte level access of a warp is one contiguous 512-byte access.
// The last tile of a row is shifted left to end at ldp (it overlaps its neighbour and recomputes a few columns to
// the same values), so all tiles are whole and the groups of a lane lie at constant offsets.
//
// A warp's software pipeline, by distance from the edge being relaxed:
//   AHEAD + 1 units  the item descriptor is loaded;
//   AHEAD units      the record and the vertex' own id row are requested (cp.async into a ring of AHEAD + 1 buffers,
//                    with a note {vertex | flag, edges} beside them);
//   2 edges          (same phase of the same step only) the neighbour's ids and levels are loaded into one of three
//                    register slots.
constexpr int STEPREC_AHEAD = 4;
constexpr int STEPREC_RING = STEPREC_AHEAD + 1;
constexpr int STEPREC_NOTE = 16;
constexpr int STEPREC_DEPTH = 3;   // edge-turns copied ahead

template <int KP> struct StepRecIdx;
template <> struct StepRecIdx<16> {
    // four candidates at once: byte c = pu_c * 16 + pv_c
    static __device__ __forceinline__ unsigned combine(unsigned pu, unsigned ids) { return (pu << 4) | ids; }
    static __device__ __forceinline__ unsigned index(unsigned x, unsigned, unsigned, int c) { return (x >> (8 * c)) & 0xffu; }
};
template <> struct StepRecIdx<64> {
    static __device__ __forceinline__ unsigned combine(unsigned pu, unsigned) { return pu; }
    static __device__ __forceinline__ unsigned index(unsigned, unsigned pu, unsigned ids, int c)
    {
        return ((pu >> (8 * c)) & 0x3fu) * 64u + ((ids >> (8 * c)) & 0x3fu);
    }
};

// named barriers of a block: DONE + g -- the workers have written their rows of the running step in phase g (workers
// arrive, the control warp waits); READY + g -- every block has signalled the previous step in phase g (the control
// warp arrives, workers wait)
constexpr int STEPREC_BAR_DONE = 1, STEPREC_BAR_READY = 1 + STEPREC_GROUPS_MAX;
static_assert(STEPREC_BAR_READY + STEPREC_GROUPS_MAX <= 16, "sixteen named barriers per block");
__device__ __forceinline__ void named_bar_sync(int id, int threads) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory"); }
__device__ __forceinline__ void named_bar_arrive(int id, int threads) { asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(threads) : "memory"); }

// NW worker warps and one control warp per block.
template <bool FWD, bool RTU, int KP, int CG, int NW, int MINB>
__global__ void __launch_bounds__((NW + 1) * 32, MINB)
pass_steprec_kernel(const __grid_constant__ LevRecArgs a)
{
    constexpr int TW = 64 * CG;              // tile width in candidates
    constexpr int NC = 2 * CG;               // candidates per lane
    constexpr int NWORD = (CG + 1) / 2;      // id words per lane
    constexpr unsigned IDMASK = 0x01010101u * (unsigned)(KP - 1);
    constexpr int HDR = 16 + 4 * KP;
    constexpr int NOTE = STEPREC_NOTE, RING = STEPREC_RING, AHEAD = STEPREC_AHEAD, DEPTH = STEPREC_DEPTH;
    __shared__ __align__(16) unsigned char s_cls[KP * KP];
    __shared__ volatile int s_lost;          // a wait of the control warp ran out: the block only keeps its barriers going
    extern __shared__ __align__(16) unsigned char dsm[];
    const int tid = threadIdx.x, lane = tid & 31;
    // warp-uniform values are broadcast from lane 0, so that the compiler keeps them (and the control flow that depends
    // on them) on the uniform path
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
    constexpr int NT = (NW + 1) * 32;
    if (*a.status != 0) return;
    for (int i = tid; i < KP * KP / 4; i += NT) reinterpret_cast<unsigned*>(s_cls)[i] = __ldg(reinterpret_cast<const unsigned*>(a.cls) + i);
    if (tid == 0) s_lost = 0;
    __syncthreads();
    const int G = a.groups;                  // phases of a walk
    const int tpg = a.tiles_per_group;       // tiles of a phase
    const int gw = (int)blockIdx.x * NW + warp;
    const unsigned nblocks = gridDim.x;
    const int num_steps = a.num_steps;
    const int tiles = (int)((a.P + 64 * CG - 1) / (64 * CG));    // padding columns of a tile are read, never written

    if (warp == NW) {
        // ---- control warp: turns "all workers of this block are done with (step, phase)" into a signal to the grid,
        // and "all blocks have signalled (step, phase)" into the go-ahead for this block's workers
        unsigned signals = 0;   // signals given to every phase counter so far
        bool lost = false;
        for (int tile_base = 0; tile_base < tiles; tile_base += G * tpg) {
            for (int g = 0; g < G; ++g) named_bar_arrive(STEPREC_BAR_READY + g, NT);   // step 0 reads no rows of this walk
            for (int step = 0; step < num_steps; ++step) {
                for (int g = 0; g < G; ++g) {
                    named_bar_sync(STEPREC_BAR_DONE + g, NT);
                    if (step + 1 == num_steps) continue;   // nobody reads the last step's rows
                    if (lane == 0 && !lost) {
                        unsigned* ctr = a.bar + 32 * g;
                        __threadfence();
                        atomicAdd(ctr, 1u);
                        const unsigned target = (signals + 1u) * nblocks;   // the counter only grows: compare modulo 2^32
                        lost = true;
#pragma unroll 1
                        for (int spin = 0; lost && spin < a.wait_limit; ++spin) lost = (int)(ld_acquire_gpu(ctr) - target) < 0;
                        if (lost) {
                            atomicCAS(a.status, 0, (int)TFPS_ERR_TIMEOUT);
                            s_lost = 1;
                        }
                    }
                    lost = __shfl_sync(0xffffffffu, (int)lost, 0) != 0;
                    named_bar_arrive(STEPREC_BAR_READY + g, NT);
                }
                ++signals;
            }
            --signals;   // the last step of a walk is not signalled
        }
        return;
    }
    const int ldp = (int)a.ldp;                     // the host keeps ldp below 2^28
    const unsigned ldp32 = (unsigned)ldp, ldp8 = (unsigned)ldp * 8u;
    const int estride = a.estride;
    const int P = (int)a.P;
    const int R = a.tiles_per_run;                  // tiles a unit spans
    const int rpp = (tpg + R - 1) / R;              // runs of a phase
    const int nil = (int)(gridDim.x * NW) / rpp;    // item lanes
    const int il = gw / rpp, wr = gw % rpp;         // this warp's item lane and its run within a phase
    const bool spare = il >= nil;                   // warps beyond a whole number of item lanes only take part in the barriers
    const unsigned bufsz = (unsigned)a.rec_max + NOTE;        // a record buffer: note {vertex | flag, edges}, record
    constexpr unsigned SLOTSZ = TW * 10 + 16;                 // an edge slot: levels, neighbour ids, own ids, commit number
    unsigned char* const wbuf = dsm + (size_t)warp * (RING * bufsz + DEPTH * SLOTSZ);
    unsigned char* const wslot = wbuf + RING * bufsz;
    const unsigned wbuf_s = smem_u32(wbuf), wslot_s = smem_u32(wslot);

    // first column of a tile: the last one is shifted left so that it ends at ldp (CG > 1 needs ldp >= TW)
    auto tile_col = [&](int t) { const int c = t * TW; return (CG > 1 && c + TW > ldp) ? ldp - TW : c; };
    // items are dealt to the lanes in alternating direction (they are sorted by edge count within a step): a lane
    // that gets a second item of a step gets a light one when its first was heavy.  Returns the item of round j, or
    // a value >= i1 when the lane has none; the valid rounds of a lane form a prefix.
    auto item_of = [&](int i0, int j) { return (j & 1) ? i0 + (j + 1) * nil - 1 - il : i0 + j * nil + il; };
    int ncommit = 0;   // cp.async groups this thread has committed; a group has landed once at most ncommit - its number are pending
    auto wait_for = [&](int number) {
        const int pending = ncommit - number;
        if (pending >= 8) cp_async_wait<8>();
        else if (pending >= 4) cp_async_wait<4>();
        else if (pending >= 2) cp_async_wait<2>();
        else if (pending == 1) cp_async_wait<1>();
        else cp_async_wait<0>();
    };

    for (int tile_base = 0; tile_base < tiles; tile_base += G * tpg) {
        // tiles of this warp's run in every phase (0: none)
        int rcount[STEPREC_GROUPS_MAX];
#pragma unroll
        for (int g = 0; g < STEPREC_GROUPS_MAX; ++g) {
            const int t0 = tile_base + g * tpg + wr * R;
            int cnt = tpg - wr * R < R ? tpg - wr * R : R;
            if (t0 + cnt > tiles) cnt = tiles - t0;
            rcount[g] = (g < G && !spare && cnt > 0) ? cnt : 0;
        }
        auto rcount_of = [&](int g) {
            int v = 0;
#pragma unroll
            for (int q = 0; q < STEPREC_GROUPS_MAX; ++q) v = q == g ? rcount[q] : v;
            return v;
        };
        // ---- front of the pipeline: iterator over this warp's units (step, phase, round)
        int f_step = 0, f_g = 0, f_j = 0, f_i0 = 0, f_i1 = 0;
        auto f_load_step = [&]() {
            if (f_step < num_steps) {
                f_i0 = __shfl_sync(0xffffffffu, __ldg(a.step_ptr + f_step), 0);
                f_i1 = __shfl_sync(0xffffffffu, __ldg(a.step_ptr + f_step + 1), 0);
            }
        };
        auto f_settle = [&]() {   // move to the next (step, phase) in which this warp has a unit
            while (f_step < num_steps && (item_of(f_i0, f_j) >= f_i1 || rcount_of(f_g) == 0)) {
                if (++f_g == G) { f_g = 0; ++f_step; f_load_step(); }
                f_j = 0;
            }
        };
        {
            bool any = false;
#pragma unroll
            for (int g = 0; g < STEPREC_GROUPS_MAX; ++g) any = any || rcount[g] > 0;
            if (!any) f_step = num_steps;
        }
        f_load_step();
        f_settle();
        // descriptor of the front unit as loaded (lane 0's copy is broadcast when the unit is requested, a unit later,
        // so that the load's latency is not waited for here); end edge -1: none
        int4 dA = make_int4(0, 0, 0, -1);
        auto front_fetch = [&]() {
            if (f_step < num_steps) {
                dA = __ldg(a.items + 2 * item_of(f_i0, f_j));
                ++f_j;
                f_settle();
            } else {
                dA.w = -1;
            }
        };
        unsigned ring_b = 0;
        auto request = [&]() {   // record and note of the unit dA describes
            ++ncommit;
            dA = make_int4(__shfl_sync(0xffffffffu, dA.x, 0), __shfl_sync(0xffffffffu, dA.y, 0), __shfl_sync(0xffffffffu, dA.z, 0),
                           __shfl_sync(0xffffffffu, dA.w, 0));
            if (dA.w >= 0) {
                const unsigned dst = wbuf_s + ring_b * bufsz;
                const unsigned char* rec = a.blob + 16ll * (unsigned)dA.y;
                const int deg = dA.w - dA.z;
                constexpr int NH = HDR / 16;
                const int ne = deg * (estride >> 4);
                const unsigned char* esrc = rec + HDR + (size_t)dA.z * estride - 16 * NH;
                for (int q = lane; q < NH + ne; q += 32) cp_async16_ca(dst + NOTE + 16u * (unsigned)q, (q < NH ? rec : esrc) + 16 * q);
                if (lane == 0) sts128(dst, (unsigned)dA.x, (unsigned)deg, (unsigned)ncommit, 0u);
            }
            cp_async_commit();
            ring_b = ring_b == RING - 1 ? 0 : ring_b + 1;
        };
        for (int q = 0; q < AHEAD; ++q) { front_fetch(); request(); }
        front_fetch();
        unsigned ring_c = 0;   // buffer of the next unit to be evaluated

        for (int step = 0; step < num_steps; ++step) {
            const int i0 = __shfl_sync(0xffffffffu, __ldg(a.step_ptr + step), 0), i1 = __shfl_sync(0xffffffffu, __ldg(a.step_ptr + step + 1), 0);
            int K = 0;   // this warp's units in every phase it has tiles in
            while (item_of(i0, K) < i1) ++K;
            for (int g = 0; g < G; ++g) {
                // ---- rows of step - 1 in this phase are complete (every block has signalled them)
                named_bar_sync(STEPREC_BAR_READY + g, NT);
                const int Rn = rcount_of(g);
                if (Rn > 0 && K > 0 && __shfl_sync(0xffffffffu, s_lost, 0) == 0) {
                    const int t0 = tile_base + g * tpg + wr * R;
                    // the edge sequence of this warp's units in this phase-step: (unit j, tile r, edge e), visited twice:
                    // by the copies into the slot ring, DEPTH edges ahead, and by the relaxation
                    struct Cursor { int j, r, e, deg, v, col; unsigned ring, slot; const unsigned char* buf; };
                    auto open = [&](Cursor& c, bool wait) {
                        c.buf = wbuf + c.ring * bufsz;
                        const int4 note = *reinterpret_cast<const int4*>(c.buf);   // written by a plain store: readable at once
                        c.v = __shfl_sync(0xffffffffu, note.x, 0);
                        c.deg = __shfl_sync(0xffffffffu, note.y, 0);
                        if (wait) {   // the record itself has landed
                            wait_for(__shfl_sync(0xffffffffu, note.z, 0));
                            __syncwarp();
                        }
                        c.e = 0;
                        c.r = 0;
                        c.col = tile_col(t0);
                    };
                    auto advance = [&](Cursor& c, bool wait) {
                        c.slot = c.slot == DEPTH - 1 ? 0 : c.slot + 1;
                        if (++c.e < c.deg) return;
                        c.e = 0;
                        if (++c.r < Rn) { c.col = tile_col(t0 + c.r); return; }
                        ++c.j;
                        c.ring = c.ring == RING - 1 ? 0 : c.ring + 1;
                        if (c.j < K) open(c, wait);
                    };
                    // copies of one edge-turn into its slot: neighbour levels and ids, own ids at the first edge of a tile
                    auto issue = [&](const Cursor& c) {
                        const unsigned dst = wslot_s + c.slot * SLOTSZ;
                        ++ncommit;
                        if (lane == 0) sts32(dst + TW * 10, (unsigned)ncommit);
                        const uint8_t* own = ptr_mad(a.part + c.col, (unsigned)(c.v & 0x7fffffff), ldp32);
                        if (c.e == 0 && lane < TW / 16 && (CG > 1 || c.col + 16 * lane < ldp)) cp_async16_ca(dst + TW * 9 + 16u * lane, own + 16 * lane);
                        if (c.e < c.deg) {
                            const unsigned nbr = __shfl_sync(0xffffffffu, *reinterpret_cast<const unsigned*>(c.buf + NOTE + HDR + (size_t)c.e * estride), 0);
                            const uint8_t* pr = ptr_mad(a.part + c.col, nbr, ldp32);
                            const long long* lr = ptr_mad(a.lev + c.col + 2 * lane, nbr, ldp8);
                            if (lane < TW / 16 && (CG > 1 || c.col + 16 * lane < ldp)) cp_async16_ca(dst + TW * 8 + 16u * lane, pr + 16 * lane);
                            if (CG > 1 || c.col + 2 * lane < ldp) {
#pragma unroll
                                for (int q = 0; q < CG; ++q) cp_async16_ca(dst + 512u * q + 16u * lane, lr + 64 * q);
                            }
                        }
                        cp_async_commit();
                    };
                    Cursor C{0, 0, 0, 0, 0, 0, ring_c, 0, nullptr}, L{0, 0, 0, 0, 0, 0, ring_c, 0, nullptr};
                    open(L, true);
                    open(C, false);
                    for (int q = 0; q < DEPTH && L.j < K; ++q) {
                        issue(L);
                        advance(L, true);
                    }
                    __syncwarp();   // the slots' commit numbers are written by lane 0
                    long long best[NC];
                    unsigned ids[NWORD];
                    do {
                        const unsigned char* slot = wslot + C.slot * SLOTSZ;
                        const unsigned char* cbuf = C.buf;
                        wait_for(__shfl_sync(0xffffffffu, *reinterpret_cast<const int*>(slot + TW * 10), 0));
                        __syncwarp();
                        if (C.e == 0) {
                            if (C.r == 0) {   // a new unit: run the front
                                request();        // the unit AHEAD units on
                                front_fetch();    // the descriptor after it
                            }
                            // a new tile: the vertex' own ids, maxima from zero
                            const unsigned char* idl = slot + TW * 9 + 2 * lane;
#pragma unroll
                            for (int w = 0; w < NWORD; ++w)
                                ids[w] = ((unsigned)*reinterpret_cast<const unsigned short*>(idl + 128 * w) |
                                          (2 * w + 1 < CG ? (unsigned)*reinterpret_cast<const unsigned short*>(idl + 128 * w + 64) << 16 : 0u)) & IDMASK;
#pragma unroll
                            for (int c = 0; c < NC; ++c) best[c] = 0;
                        }
                        if (C.e < C.deg) {
                            const unsigned char* e = cbuf + NOTE + HDR + (size_t)C.e * estride;
                            const unsigned char* pul = slot + TW * 8 + 2 * lane;
#pragma unroll
                            for (int w = 0; w < NWORD; ++w) {
                                const unsigned pu = ((unsigned)*reinterpret_cast<const unsigned short*>(pul + 128 * w) |
                                                     (2 * w + 1 < CG ? (unsigned)*reinterpret_cast<const unsigned short*>(pul + 128 * w + 64) << 16 : 0u)) & IDMASK;
                                const unsigned x = StepRecIdx<KP>::combine(pu, ids[w]);
#pragma unroll
                                for (int c = 0; c < 4; ++c) {
                                    if (4 * w + c < NC) {
                                        const unsigned comb = s_cls[StepRecIdx<KP>::index(x, pu, ids[w], c)];
                                        const long long lv = *reinterpret_cast<const long long*>(slot + 512 * (2 * w + c / 2) + 16 * lane + 8 * (c & 1));
                                        long long val = lv + *reinterpret_cast<const long long*>(e + 8 + 8u * comb);
                                        if (RTU) val += *reinterpret_cast<const int*>(e + 8 + a.wbytes + 4 * ((pu >> (8 * c)) & 0xffu));
                                        best[4 * w + c] = val > best[4 * w + c] ? val : best[4 * w + c];
                                    }
                                }
                            }
                        }
                        const bool tile_done = C.e + 1 >= C.deg;
                        if (tile_done) {
                            if (!FWD) {
                                const int* rtv = reinterpret_cast<const int*>(cbuf + NOTE + 16);
#pragma unroll
                                for (int c = 0; c < NC; ++c) best[c] += rtv[(ids[c / 4] >> (8 * (c & 3))) & 0xffu];
                            }
                            long long* out = ptr_mad(a.lev + C.col + 2 * lane, (unsigned)(C.v & 0x7fffffff), ldp8);
                            if (C.col + TW <= P) {   // all columns of the tile are candidates
#pragma unroll
                                for (int q = 0; q < CG; ++q) {
                                    if (C.v < 0) {   // partial item
                                        atomicMax(out + 64 * q, best[2 * q]);
                                        atomicMax(out + 64 * q + 1, best[2 * q + 1]);
                                    } else {
                                        *reinterpret_cast<longlong2*>(out + 64 * q) = make_longlong2(best[2 * q], best[2 * q + 1]);
                                    }
                                }
                            } else {
#pragma unroll
                                for (int q = 0; q < CG; ++q) {
                                    const int c0 = C.col + 64 * q + 2 * lane;
                                    const int nv = P - c0 >= 2 ? 2 : (P > c0 ? 1 : 0);
                                    if (C.v < 0) {
                                        if (nv > 0) atomicMax(out + 64 * q, best[2 * q]);
                                        if (nv > 1) atomicMax(out + 64 * q + 1, best[2 * q + 1]);
                                    } else if (nv == 2) {
                                        *reinterpret_cast<longlong2*>(out + 64 * q) = make_longlong2(best[2 * q], best[2 * q + 1]);
                                    } else if (nv == 1) {
                                        out[64 * q] = best[2 * q];
                                    }
                                }
                            }
                        }
                        __syncwarp();   // the slot (and, after a unit's last tile, its record buffer) is rewritten below
                        advance(C, false);
                        if (L.j < K) {
                            issue(L);
                            advance(L, true);
                        }
                    } while (C.j < K);
                    ring_c = C.ring;
                }
                // ---- this warp's rows of (step, phase g) are written
                named_bar_arrive(STEPREC_BAR_DONE + g, NT);
            }
        }
        cp_async_wait<0>();
        __syncwarp();
    }
}

template <bool FWD, bool RTU, int KP, int CG, int NW, int MINB>
cudaError_t steprec_launch(LevRecArgs a, int sm_count, cudaStream_t st)
{
    auto kernel = pass_steprec_kernel<FWD, RTU, KP, CG, NW, MINB>;
    constexpr int TW = 64 * CG;
    const int R = std::max(1, std::min(a.tiles_per_run, 8));
    const size_t smem = (size_t)NW * (STEPREC_RING * ((size_t)a.rec_max + STEPREC_NOTE) + STEPREC_DEPTH * ((size_t)TW * 10 + 16));
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, (NW + 1) * 32, smem);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) return cudaErrorLaunchOutOfResources;
    if (a.blocks_per_sm > 0 && a.blocks_per_sm < per_sm) per_sm = a.blocks_per_sm;
    const long long tiles = (a.P + TW - 1) / TW;
    // phases and tiles per phase: no more than there are tiles
    int G = std::max(1, std::min(a.groups, (int)STEPREC_GROUPS_MAX));
    if (G > tiles) G = (int)tiles;
    const long long tpg = std::min<long long>(std::max(1, a.tiles_per_group), (tiles + G - 1) / G);
    // item lanes: as many as the machine holds, but no more than the widest step has items (a barrier costs more
    // the more blocks take part in it); whole blocks
    const long long warps_max = (long long)per_sm * sm_count * NW;
    const long long rpp = (tpg + R - 1) / R;   // runs of a phase: a warp takes one run of every item of its lane
    long long lanes = std::max<long long>(1, std::min<long long>(warps_max / rpp, std::max(1, a.max_step_items)));
    long long blocks = (lanes * rpp + NW - 1) / NW;
    if (blocks > (long long)per_sm * sm_count) blocks = (long long)per_sm * sm_count;
    if (blocks * NW < rpp) return cudaErrorLaunchOutOfResources;   // a phase wider than the machine
    a.groups = G;
    a.tiles_per_group = (int)tpg;
    a.tiles_per_run = R;
    e = cudaMemsetAsync(a.bar, 0, 128 * (size_t)STEPREC_GROUPS_MAX, st);
    if (e != cudaSuccess) return e;
    void* params[] = {&a};
    e = cudaLaunchCooperativeKernel((const void*)kernel, dim3((unsigned)blocks), dim3((NW + 1) * 32), params, smem, st);
    if (e != cudaSuccess) return e;
    count_launches(1);
    return cudaGetLastError();
}

// tile width by the matrix width (a tile must fit a row), block shape by the record size; a block is NW worker
// warps and the control warp (8 warps: two blocks of 128 registers per thread, or three of 80, fill an SM)
template <bool FWD, bool RTU, int KP>
cudaError_t steprec_shape(const LevRecArgs& a, int sm_count, cudaStream_t st)
{
    const bool big = a.rec_max > 1024;   // many devices or bandwidth classes: fewer warps per block so that the rings fit
    if (a.ldp >= 256 && !big && KP == 16 && a.shape < 2) {
        if (a.shape == 1) return steprec_launch<FWD, RTU, 16, 4, 7, 3>(a, sm_count, st);   // 21 workers, 80 registers
        return steprec_launch<FWD, RTU, 16, 4, 7, 2>(a, sm_count, st);                       // 14 workers, 128 registers
    }
    if (a.ldp >= 128) {
        if (big) return steprec_launch<FWD, RTU, KP, 2, 3, 4>(a, sm_count, st);
        if (a.shape == 3 && KP == 16) return steprec_launch<FWD, RTU, 16, 2, 7, 4>(a, sm_count, st);   // 28 workers, 64 registers
        return steprec_launch<FWD, RTU, KP, 2, 7, 3>(a, sm_count, st);                       // 21 workers, 80 registers
    }
    if (big) return steprec_launch<FWD, RTU, KP, 1, 3, 4>(a, sm_count, st);
    return steprec_launch<FWD, RTU, KP, 1, 7, 3>(a, sm_count, st);
}

// ---- the same pass as one launch per step --------------------------------------------------------------------------
// For wide batches, where a step has enough blocks to fill the machine: a block takes ONE work item and CHAIN_WARPS *
// 128 candidates (4 candidates per lane), stages the item's record in shared memory and relaxes its edges
// with plain (L1-allocating) loads, so that rows many items of a step share -- the rows of hub vertices -- are served
// by L1.  The launches of a pass are chained with programmatic dependent launch: a block reads what does not depend
// on the previous step (item, record, own ids) before it waits for it.
constexpr int CHAIN_WARPS = 4;

template <bool FWD, bool RTU, int KP, int EB, int MINB>
__global__ void __launch_bounds__(CHAIN_WARPS * 32, MINB)
pass_stepchain_kernel(const __grid_constant__ LevRecArgs a, int item0, int count)
{
    extern __shared__ __align__(16) unsigned char s_rec[];   // header, runtimes and the item's edges
    __shared__ __align__(16) unsigned char s_cls[KP * KP];
    constexpr unsigned IDMASK = 0x01010101u * (unsigned)(KP - 1);
    constexpr int HDR = 16 + 4 * KP;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool live = *a.status == 0;
    for (int i = tid; i < KP * KP / 4; i += CHAIN_WARPS * 32) reinterpret_cast<unsigned*>(s_cls)[i] = __ldg(reinterpret_cast<const unsigned*>(a.cls) + i);
    // a lane's four candidates are contiguous (one 32-bit id load, two 16-byte level loads whose second half is served
    // by L1; splitting a lane's candidates so that every load is contiguous across the warp measured the same)
    const long long j0 = ((long long)blockIdx.x * CHAIN_WARPS + warp) * 128 + lane * 4;
    const long long rem = a.P - j0;
    const int nvalid = rem >= 4 ? 4 : (rem > 0 ? (int)rem : 0);
    const long long jl = nvalid > 0 ? j0 : 0;   // idle lanes read (and drop) columns 0..3
    const long long ldp = a.ldp;
    const int estride = a.estride;
    bool waited = false;

    for (int i = blockIdx.y; i < count && live; i += gridDim.y) {
        const int4 it = __ldg(a.items + 2 * (item0 + i));
        const int4 nb4 = __ldg(a.items + 2 * (item0 + i) + 1);   // neighbours of the item's first four edges
        const int deg = it.w - it.z;
        const int v = it.x & 0x7fffffff;
        const unsigned char* rec = a.blob + 16ll * (unsigned)it.y;
        // own ids and the ids of the first neighbours: requested before the record arrives
        const unsigned ids = __ldg(reinterpret_cast<const unsigned*>(a.part + (long long)v * ldp + jl)) & IDMASK;
        long long off[EB];
        unsigned pu[EB];
        {
            const int nbv[4] = {nb4.x, nb4.y, nb4.z, nb4.w};
#pragma unroll
            for (int q = 0; q < EB; ++q) {
                if (q < deg) {
                    off[q] = (long long)nbv[q] * ldp + jl;
                    pu[q] = __ldg(reinterpret_cast<const unsigned*>(a.part + off[q])) & IDMASK;
                }
            }
        }
        if (i != (int)blockIdx.y) __syncthreads();   // the previous item's record is no longer read
        for (int q = tid; q < HDR / 16; q += CHAIN_WARPS * 32) reinterpret_cast<uint4*>(s_rec)[q] = __ldg(reinterpret_cast<const uint4*>(rec) + q);
        {
            const uint4* src = reinterpret_cast<const uint4*>(rec + HDR + (size_t)it.z * estride);
            uint4* dst = reinterpret_cast<uint4*>(s_rec + HDR);
            for (int q = tid; q < deg * (estride >> 4); q += CHAIN_WARPS * 32) dst[q] = __ldg(src + q);
        }
        __syncthreads();
        const int* rtv = reinterpret_cast<const int*>(s_rec + 16);
        const unsigned char* edges = s_rec + HDR;
        long long best[4] = {0, 0, 0, 0};
        for (int b0 = 0; b0 < deg; b0 += EB) {
            const int nb = deg - b0 < EB ? deg - b0 : EB;
#pragma unroll
            for (int q = 0; q < EB; ++q) {
                if (b0 > 0 && q < nb) {
                    off[q] = (long long)*reinterpret_cast<const int*>(edges + (size_t)(b0 + q) * estride) * ldp + jl;
                    pu[q] = __ldg(reinterpret_cast<const unsigned*>(a.part + off[q])) & IDMASK;
                }
            }
            if (!waited) { asm volatile("griddepcontrol.wait;" ::: "memory"); waited = true; }   // neighbour levels are the previous launches' output
            longlong2 lu[EB][2];
#pragma unroll
            for (int q = 0; q < EB; ++q) {
                if (q < nb) {
                    const longlong2* p = reinterpret_cast<const longlong2*>(a.lev + off[q]);
                    lu[q][0] = p[0];
                    lu[q][1] = p[1];
                }
            }
#pragma unroll
            for (int q = 0; q < EB; ++q) {
                if (q < nb) {
                    const unsigned char* e = edges + (size_t)(b0 + q) * estride;
                    const long long l4[4] = {lu[q][0].x, lu[q][0].y, lu[q][1].x, lu[q][1].y};
                    const unsigned x = StepRecIdx<KP>::combine(pu[q], ids);
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const unsigned comb = s_cls[StepRecIdx<KP>::index(x, pu[q], ids, c)];
                        long long val = l4[c] + *reinterpret_cast<const long long*>(e + 8 + 8u * comb);
                        if (RTU) val += *reinterpret_cast<const int*>(e + 8 + a.wbytes + 4 * ((pu[q] >> (8 * c)) & 0xffu));
                        best[c] = val > best[c] ? val : best[c];
                    }
                }
            }
        }
        if (!FWD) {
#pragma unroll
            for (int c = 0; c < 4; ++c) best[c] += rtv[(ids >> (8 * c)) & 0xffu];
        }
        if (!waited) { asm volatile("griddepcontrol.wait;" ::: "memory"); waited = true; }
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
    if (!waited) asm volatile("griddepcontrol.wait;" ::: "memory");
}

template <bool FWD, bool RTU, int KP, int EB, int MINB>
cudaError_t stepchain_launch(const LevRecArgs& a, const std::vector<int>& sp, cudaStream_t st)
{
    auto kernel = pass_stepchain_kernel<FWD, RTU, KP, EB, MINB>;
    const size_t smem = (size_t)a.rec_max;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const unsigned gx = (unsigned)((a.P + CHAIN_WARPS * 128 - 1) / (CHAIN_WARPS * 128));
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    const int steps = (int)sp.size() - 1;
    for (int step = 0; step < steps; ++step) {
        const int item0 = sp[step], count = sp[step + 1] - sp[step];
        if (count <= 0) continue;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(gx, (unsigned)std::min(count, 65535));
        cfg.blockDim = dim3(CHAIN_WARPS * 32);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cfg.attrs = attr;
        cfg.numAttrs = step == 0 ? 0 : 1;   // the first step follows ordinary stream order
        e = cudaLaunchKernelEx(&cfg, kernel, a, item0, count);
        if (e != cudaSuccess) return e;
    }
    count_launches(steps);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_pass_steprec(const LevRecArgs& a, bool fwd, int sm_count, cudaStream_t st)
{
    if (a.num_steps <= 0) return cudaSuccess;
    if (!fwd) return a.kp == 16 ? steprec_shape<false, false, 16>(a, sm_count, st) : steprec_shape<false, false, 64>(a, sm_count, st);
    if (a.rtu) return a.kp == 16 ? steprec_shape<true, true, 16>(a, sm_count, st) : steprec_shape<true, true, 64>(a, sm_count, st);
    return a.kp == 16 ? steprec_shape<true, false, 16>(a, sm_count, st) : steprec_shape<true, false, 64>(a, sm_count, st);
}

// one launch per step, chained (step_ptr_host: first item of every step)
cudaError_t launch_pass_stepchain(const LevRecArgs& a, bool fwd, const std::vector<int>& step_ptr_host, cudaStream_t st)
{
    if (a.num_steps <= 0) return cudaSuccess;
    // edges in flight per thread and resident blocks per SM: forward two edges and 32 warps, backward one edge and 48
    // (config 5, P = 4,096: 27.3 / 21.3 ms; forward with 40 warps 31.6, with four edges and 24 warps 36.9; backward
    // with 40 warps 21.0, with two edges and 32 warps 24.2)
    if (!fwd) return a.kp == 16 ? stepchain_launch<false, false, 16, 1, 12>(a, step_ptr_host, st) : stepchain_launch<false, false, 64, 1, 10>(a, step_ptr_host, st);
    if (a.rtu) return a.kp == 16 ? stepchain_launch<true, true, 16, 2, 8>(a, step_ptr_host, st) : stepchain_launch<true, true, 64, 2, 8>(a, step_ptr_host, st);
    return a.kp == 16 ? stepchain_launch<true, false, 16, 2, 8>(a, step_ptr_host, st) : stepchain_launch<true, false, 64, 2, 8>(a, step_ptr_host, st);
}

}  // namespace tfps
