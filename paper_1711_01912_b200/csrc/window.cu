// Windowed candidate-sliced pass.  Like the sliced pass, one block owns 32*CPT
// candidates and walks the whole graph chunk by chunk with one block barrier
// per chunk.  In addition the block keeps the levels and ids of the last R
// positions of ITS OWN candidates in a shared-memory ring: a neighbour that lies
// within the window is read from shared memory, so the dependent chain of a
// vertex never leaves the SM and the neighbour never touches L2; only the
// compulsory traffic (one id read, one level write per vertex-candidate)
// reaches global memory.  Neighbours outside the window are read from global
// memory as in the sliced pass.  Edge costs come from the precomputed value
// array V (see WindowPlan): one shuffle per candidate replaces the per-edge
// table build.  Adjacency, edge values and the id rows of coming chunks are
// staged with cp.async one to two chunks ahead.
#include "common.cuh"

namespace tfps {

namespace {

// ---- TMA bulk copies completing on an mbarrier ---------------------------------------------
__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_init_fence() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_expect_tx(unsigned bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// global -> shared bulk copy; both addresses 16-byte aligned, bytes a multiple of 16
__device__ __forceinline__ void bulk_g2s(unsigned dst, const void* src, unsigned bytes, unsigned bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned bar, unsigned parity)
{
    unsigned ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// 16-byte asynchronous copy through the load/store path, and the hook that makes an mbarrier count the
// completion of all cp.async issued so far by this thread as one (pre-counted) arrival
__device__ __forceinline__ void cp_async16(unsigned dst, const void* g)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(g) : "memory");
}
__device__ __forceinline__ void cp_async_arrive_on(unsigned bar)
{
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
// Bounded wait: gives up after WAIT_LIMIT polls (each poll itself blocks for a hardware-defined time slice).
constexpr int WAIT_LIMIT = 1 << 20;
__device__ __forceinline__ bool mbar_wait(unsigned bar, unsigned parity)
{
    for (int i = 0; i < WAIT_LIMIT; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

template <int CPT> struct IdWords { static constexpr int N = (CPT + 3) / 4; };

template <int CPT>
__device__ __forceinline__ void load_ids(const uint8_t* p, unsigned (&w)[IdWords<CPT>::N])
{
    if constexpr (CPT == 1) w[0] = *p;
    else if constexpr (CPT == 2) w[0] = *reinterpret_cast<const unsigned short*>(p);
    else w[0] = *reinterpret_cast<const unsigned*>(p);
}
template <int CPT>
__device__ __forceinline__ void store_ids(uint8_t* p, const unsigned (&w)[IdWords<CPT>::N])
{
    if constexpr (CPT == 1) *p = (uint8_t)w[0];
    else if constexpr (CPT == 2) *reinterpret_cast<unsigned short*>(p) = (unsigned short)w[0];
    else *reinterpret_cast<unsigned*>(p) = w[0];
}
template <int CPT>
__device__ __forceinline__ unsigned id_at(const unsigned (&w)[IdWords<CPT>::N], int c)
{
    return (w[c >> 2] >> (8 * (c & 3))) & 0xffu;
}
template <int CPT>
__device__ __forceinline__ void load_levels(const long long* p, long long (&out)[CPT])
{
    if constexpr (CPT == 1) {
        out[0] = *p;
    } else {
#pragma unroll
        for (int i = 0; i < CPT; i += 2) {
            longlong2 v = *reinterpret_cast<const longlong2*>(p + i);
            out[i] = v.x;
            out[i + 1] = v.y;
        }
    }
}
template <int CPT>
__device__ __forceinline__ void store_levels(long long* p, const long long (&v)[CPT])
{
    if constexpr (CPT == 1) {
        *p = v[0];
    } else {
#pragma unroll
        for (int i = 0; i < CPT; i += 2) *reinterpret_cast<longlong2*>(p + i) = make_longlong2(v[i], v[i + 1]);
    }
}

// Shared-memory carve-up (all offsets multiples of 16 bytes).  Rings: chunk heads (2*depth+1 slots: a head
// must have landed before the id rows of its chunk can be requested), chunk bodies and id rows (depth+1 each).
struct Carve {
    size_t bars, rt, cls2, cp, head, head_stride, body, body_stride, ids, ids_stride, win_lev, win_id, total;
};

__host__ __device__ inline size_t up16(size_t x) { return (x + 15) & ~(size_t)15; }

__host__ __device__ inline Carve carve(int k, int R, int cpt, int warps, int lsize, int max_v, int head_max, int body_max,
                                       int depth)
{
    Carve c;
    const size_t slice = 32 * (size_t)cpt;
    size_t o = 0;
    c.bars = o; o += up16(8 * (size_t)(3 * depth + 2) + 16);   // mbarriers, abort flag, two vertex counters, chunks-done counter
    c.rt = o; o += up16(sizeof(DivConst) * (size_t)k);
    c.cls2 = o; o += up16((size_t)k * k);
    c.cp = o;   // the staging rings double as the reduction buffer of the CP maxima after the last chunk
    c.head = o; c.head_stride = up16((size_t)head_max); o += (size_t)(2 * depth + 1) * c.head_stride;
    c.body = o; c.body_stride = up16((size_t)body_max); o += (size_t)(depth + 1) * c.body_stride;
    c.ids = o; c.ids_stride = up16((size_t)max_v * slice); o += (size_t)(depth + 1) * c.ids_stride;
    if (o < c.cp + sizeof(long long) * (size_t)warps * slice) o = up16(c.cp + sizeof(long long) * (size_t)warps * slice);
    c.win_lev = o; o += up16((size_t)lsize * (size_t)R * slice);
    c.win_id = o; o += up16((size_t)R * slice);
    c.total = o;
    return c;
}

// 32-bit shared-state-space load (address from __cvta_generic_to_shared)
__device__ __forceinline__ unsigned lds_u32(unsigned a) { unsigned v; asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a)); return v; }

// window rows through typed shared-memory pointers (vector width = CPT levels)
template <int CPT> __device__ __forceinline__ void load_win(const long long* p, long long (&out)[CPT]) { load_levels<CPT>(p, out); }
template <int CPT> __device__ __forceinline__ void store_win(long long* p, const long long (&v)[CPT]) { store_levels<CPT>(p, v); }
template <int CPT> __device__ __forceinline__ void load_win(const int* p, int (&out)[CPT])
{
    if constexpr (CPT == 1) out[0] = *p;
    else if constexpr (CPT == 2) { const int2 v = *reinterpret_cast<const int2*>(p); out[0] = v.x; out[1] = v.y; }
    else { const int4 v = *reinterpret_cast<const int4*>(p); out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w; }
}
template <int CPT> __device__ __forceinline__ void store_win(int* p, const int (&v)[CPT])
{
    if constexpr (CPT == 1) *p = v[0];
    else if constexpr (CPT == 2) *reinterpret_cast<int2*>(p) = make_int2(v[0], v[1]);
    else *reinterpret_cast<int4*>(p) = make_int4(v[0], v[1], v[2], v[3]);
}
// best = max(best, lu + w)
__device__ __forceinline__ long long add_max(long long lu, long long w, long long best) { const long long v = lu + w; return v > best ? v : best; }
__device__ __forceinline__ int add_max(int lu, int w, int best) { return __viaddmax_s32(lu, w, best); }

// Byte offsets of the shared-memory regions, computed on the host and passed as a kernel parameter.
struct WinLayout {
    unsigned bars, rt, cls2, cp, head, head_stride, body, body_stride, ids, ids_stride, win_lev, win_id;
    int depth;
};

// MODE 0: general.  MODE 1 (ALL_STAGED): every chunk's adjacency fits the staging buffers (no vertex with more
// than CHUNK_E edges).  MODE 2: additionally every neighbour lies inside the window, so the loop carries neither
// the distance test nor the global-memory path.
// The last warp is the producer: it runs its own loop, issuing the copies for the chunk `depth` ahead (heads
// 2*depth ahead) as soon as the consumers report the ring slot free, and never joins the consumers' per-chunk
// barrier (a named barrier over the consumer warps only), so its latency stays off their critical path.
template <int CPT, bool FWD, int MODE, typename LT>
__global__ void __launch_bounds__(1024)
pass_window_kernel(PassArgs a, WindowPlan wp, WinLayout L)
{
    extern __shared__ __align__(16) unsigned char smem[];
    constexpr int SLICE = 32 * CPT;
    constexpr bool ALL_STAGED = MODE >= 1;
    constexpr bool FULL_WINDOW = MODE == 2;
    constexpr unsigned LS = sizeof(LT);   // bytes of a level inside the block: 4 when every path length fits int32
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, wpb = blockDim.x >> 5;
    const int ncons = wpb - 1;                 // consumer warps 0..ncons-1
    const bool producer = warp == ncons;
    const int k = a.tab.k;
    const int ncomb = wp.ncomb;
    const int R = wp.R;              // power of two (or 0)
    const int rmask = R - 1;
    const int hit_span = R - CHUNK_V;  // a neighbour at most this many positions away is still in the ring
    const bool need_nbr = hit_span < wp.maxspan;   // some neighbours are read from global memory
    const unsigned sbase = (unsigned)__cvta_generic_to_shared(smem);
    DivConst* s_rt = reinterpret_cast<DivConst*>(smem + L.rt);
    long long* s_cp = reinterpret_cast<long long*>(smem + L.cp);
    volatile int* s_abort = reinterpret_cast<volatile int*>(smem + L.bars + 8 * (3 * L.depth + 2));
    // vertices of a chunk are handed out dynamically (degrees differ): one counter per chunk parity
    int* s_next = reinterpret_cast<int*>(smem + L.bars + 8 * (3 * L.depth + 2) + 4);
    // number of chunks the consumers have finished: tells the producer which ring slots are free again
    volatile int* s_done = reinterpret_cast<volatile int*>(smem + L.bars + 8 * (3 * L.depth + 2) + 12);
    if (*a.status != 0) return;
    const int D = L.depth, NB = 2 * D + 1, NS = D + 1;
    const unsigned head_bar0 = sbase + L.bars, stage_bar0 = head_bar0 + 8u * NB;
    if (threadIdx.x == 0) {
        for (int j = 0; j < NB; ++j) mbar_init(head_bar0 + 8u * j, 1);
        // a stage completes on the body's bulk copy (one arrival with its byte count) plus one arrival per
        // producer lane once that lane's id-row copies have landed
        for (int j = 0; j < NS; ++j) mbar_init(stage_bar0 + 8u * j, 33);
        *s_abort = 0;
        s_next[0] = 0;
        s_next[1] = 0;
        *s_done = 0;
        mbar_init_fence();
    }
    for (int i = threadIdx.x; i < k; i += blockDim.x) s_rt[i] = a.tab.rt_div[i];
    for (int i = threadIdx.x; i < k * k; i += blockDim.x) smem[L.cls2 + i] = wp.cls2[i];
    __syncthreads();

    const long long slice0 = (long long)blockIdx.x * SLICE;
    const long long j0 = slice0 + (long long)lane * CPT;
    const long long rem = a.P - j0;
    const int nvalid = rem >= CPT ? CPT : (rem > 0 ? (int)rem : 0);
    const int lane_col = nvalid > 0 ? lane * CPT : 0;      // idle lanes shadow the slice's first lane
    const long long jl = slice0 + lane_col;
    const unsigned idmask = nvalid >= 4 ? 0xffffffffu : (nvalid > 0 ? ((1u << (8 * nvalid)) - 1u) : 0u);
    const long long ldp = a.ldp;
    const unsigned slice_bytes = (unsigned)((ldp - slice0) < SLICE ? (ldp - slice0) : SLICE);  // multiple of 16
    const bool want_cp = a.cp != nullptr;
    long long cpmax[CPT];
#pragma unroll
    for (int c = 0; c < CPT; ++c) cpmax[c] = 0;
    LT* win_lev_lane = reinterpret_cast<LT*>(smem + L.win_lev) + lane * CPT;
    uint8_t* win_id_lane = smem + L.win_id + lane * CPT;
    const unsigned char* s_cls2 = smem + L.cls2;
    const int num_chunks = wp.num_chunks;
    const int4* desc = reinterpret_cast<const int4*>(wp.desc);
    const unsigned char* blob = reinterpret_cast<const unsigned char*>(wp.blob);

    auto fail_wait = [&]() {
        atomicCAS(a.status, 0, (int)TFPS_ERR_TIMEOUT);
        *s_abort = 1;
    };
    // ---- producer side -------------------------------------------------------------------------
    // Descriptors of the coming chunks are fetched 32 at a time (one per lane) and handed out by shuffles, so
    // the producer does not pay a global-memory round trip per chunk.
    auto load_desc = [&](int first, int4& d0, int4& d1) {   // lane l gets the descriptor of chunk first+l
        const int j = first + lane;
        d0 = make_int4(0, 0, 0, 0); d1 = d0;
        if (j < num_chunks) {
            const int idx = FWD ? j : num_chunks - 1 - j;
            d0 = desc[2 * idx];
            d1 = desc[2 * idx + 1];
        }
    };
    auto bcast = [&](const int4& v, int src) {
        return make_int4(__shfl_sync(0xffffffffu, v.x, src), __shfl_sync(0xffffffffu, v.y, src),
                         __shfl_sync(0xffffffffu, v.z, src), __shfl_sync(0xffffffffu, v.w, src));
    };
    auto issue_head = [&](const int4& d, int slot) {   // chunk -> head ring slot (needs d.x, d.y)
        if (lane == 0) {
            const unsigned bar = head_bar0 + 8u * slot;
            mbar_expect_tx(bar, (unsigned)d.y);
            bulk_g2s(sbase + L.head + (unsigned)slot * L.head_stride, blob + 16ll * (unsigned)d.x, (unsigned)d.y, bar);
        }
    };
    auto issue_stage = [&](const int4& d0, const int4& d1, int slot, int hslot, unsigned hpar) {   // body + id rows
        // warp-uniform outcome: the lanes below meet at a __syncwarp
        if (!__all_sync(0xffffffffu, mbar_wait(head_bar0 + 8u * hslot, hpar))) { fail_wait(); return; }
        const int cnt = d1.y;
        const unsigned body_bytes = (unsigned)((need_nbr || !ALL_STAGED) ? d0.w : d1.x);
        const unsigned bar = stage_bar0 + 8u * slot;
        if (lane == 0) {
            mbar_expect_tx(bar, body_bytes);
            bulk_g2s(sbase + L.body + (unsigned)slot * L.body_stride, blob + 16ll * (unsigned)d0.z, body_bytes, bar);
        }
        // id rows: short scattered pieces, cheaper as 16-byte cp.async than as one bulk copy each
        const unsigned vertf_s = sbase + L.head + (unsigned)hslot * L.head_stride + 16u;
        const unsigned ids_s = sbase + L.ids + (unsigned)slot * L.ids_stride;
        const int sh = slice_bytes >= 128u ? 3 : (slice_bytes >= 64u ? 2 : (slice_bytes >= 32u ? 1 : 0));
        const int per_row = (int)(slice_bytes >> 4);
        if ((per_row & (per_row - 1)) == 0) {
            for (int i = lane; i < (cnt << sh); i += 32) {
                const int r = i >> sh, q = i & (per_row - 1);
                const int v = (int)lds_u32(vertf_s + 4u * r) & 0x7fffffff;
                cp_async16(ids_s + (unsigned)(r * SLICE + 16 * q), a.part + (long long)v * ldp + slice0 + 16 * q);
            }
        } else {
            for (int i = lane; i < cnt * per_row; i += 32) {
                const int r = i / per_row, q = i - r * per_row;
                const int v = (int)lds_u32(vertf_s + 4u * r) & 0x7fffffff;
                cp_async16(ids_s + (unsigned)(r * SLICE + 16 * q), a.part + (long long)v * ldp + slice0 + 16 * q);
            }
        }
        cp_async_arrive_on(bar);
    };

    // register batches of descriptors: hq* for head issue (chunk ci+2D), sq* for stage issue (chunk ci+D)
    int4 hq0, hq1, sq0, sq1;
    int hq_first = 0, sq_first = 0;
    hq0 = hq1 = sq0 = sq1 = make_int4(0, 0, 0, 0);
    // ring positions: chunk ci (consumers), ci+D (producer: stage), ci+2D (producer: head)
    int hs = 0, ss = 0;
    unsigned sp = 0;
    if (producer) {
        load_desc(0, hq0, hq1);
        sq0 = hq0; sq1 = hq1;
        for (int j = 0; j < 2 * D && j < num_chunks; ++j) issue_head(bcast(hq0, j), j);       // 2D <= 16 < 32
        for (int j = 0; j < D && j < num_chunks; ++j) issue_stage(bcast(sq0, j), bcast(sq1, j), j, j, 0u);
        int hsD = D % NB, ssD = D % NS, hs2D = (2 * D) % NB;
        unsigned hpD = (unsigned)((D / NB) & 1);
        for (int ci = 0; ci < num_chunks && !*s_abort; ++ci) {
            // head(ci+2D) and stage(ci+D) overwrite the ring slots of chunk ci-1: wait until it is finished
            bool freed = ci == 0;
            for (int spin = 0; !freed && spin < WAIT_LIMIT; ++spin) {
                freed = *s_done >= ci || *s_abort;
            }
            if (!freed) { fail_wait(); break; }
            if (ci + 2 * D < num_chunks) {
                if (ci + 2 * D >= hq_first + 32) { hq_first += 32; load_desc(hq_first, hq0, hq1); }
                const int src = ci + 2 * D - hq_first;
                issue_head(make_int4(__shfl_sync(0xffffffffu, hq0.x, src), __shfl_sync(0xffffffffu, hq0.y, src), 0, 0), hs2D);
            }
            if (ci + D < num_chunks) {
                if (ci + D >= sq_first + 32) { sq_first += 32; load_desc(sq_first, sq0, sq1); }
                const int src = ci + D - sq_first;
                const int4 b0 = make_int4(0, 0, __shfl_sync(0xffffffffu, sq0.z, src), __shfl_sync(0xffffffffu, sq0.w, src));
                const int4 b1 = make_int4(__shfl_sync(0xffffffffu, sq1.x, src), __shfl_sync(0xffffffffu, sq1.y, src), 0, 0);
                issue_stage(b0, b1, ssD, hsD, hpD);
            }
            if (++hsD == NB) { hsD = 0; hpD ^= 1u; }
            if (++ssD == NS) ssD = 0;
            if (++hs2D == NB) hs2D = 0;
        }
    }

    for (int ci = 0; ci < num_chunks && !producer; ++ci) {
        // A stage is armed only after the producer has seen its head land, so seeing the stage complete
        // orders this thread after the head's arrival as well: one wait per chunk.
        if (!mbar_wait(stage_bar0 + 8u * ss, sp)) {
            fail_wait();
        } else {
            const unsigned char* head_p = smem + L.head + (unsigned)hs * L.head_stride;
            const int4 hdr = *reinterpret_cast<const int4*>(head_p);
            const int p0 = hdr.x, cnt = hdr.y, e0 = hdr.z, es = hdr.w;  // es: staged edges, -1: edges stay in global memory
            const bool staged = ALL_STAGED || es >= 0;
            const unsigned esz = es > 0 ? (unsigned)es : 0u;
            const int* vertf_p = reinterpret_cast<const int*>(head_p + 16);
            const unsigned char* body_p = smem + L.body + (unsigned)ss * L.body_stride;
            const int* eoff_p = reinterpret_cast<const int*>(body_p);
            const unsigned char* xvert_b = body_p + (((unsigned)(cnt + 1) * 4u + 15u) & ~15u);
            const unsigned long long* xvert_p = reinterpret_cast<const unsigned long long*>(xvert_b);
            const unsigned char* npos_b = xvert_b + (((unsigned)cnt * 8u + 15u) & ~15u);
            const int* npos_p = reinterpret_cast<const int*>(npos_b);
            const unsigned char* V_b = npos_b + ((esz * 4u + 15u) & ~15u);
            const LT* V_p = reinterpret_cast<const LT*>(V_b);
            const int* nbr_p = reinterpret_cast<const int*>(V_b + ((esz * (unsigned)ncomb * LS + 15u) & ~15u));
            const unsigned char* idrow_p = smem + L.ids + (unsigned)ss * L.ids_stride + (unsigned)lane_col;

            int* next_ctr = s_next + (ci & 1);
            if (threadIdx.x == 0) s_next[(ci + 1) & 1] = 0;   // last used by chunk ci-1, whose warps all passed the barrier
            const bool dynamic = cnt > ncons * wp.static_rounds;   // few vertices per warp: a fixed assignment is cheaper than the counter
            for (int round = 0;; ++round) {
                int i = warp + round * ncons;
                if (dynamic) {
                    if (lane == 0) i = atomicAdd(next_ctr, 1);
                    i = __shfl_sync(0xffffffffu, i, 0);
                }
                if (i >= cnt) break;
                const int vf = vertf_p[i];
                const int v = vf & 0x7fffffff;
                const int pos = p0 + i;
                unsigned pvw[IdWords<CPT>::N];
                load_ids<CPT>(idrow_p + i * SLICE, pvw);
                const unsigned pv = pvw[0] & idmask;
                const unsigned char* cls_v[CPT];   // &cls2[0*k + idv]
#pragma unroll
                for (int c = 0; c < CPT; ++c) cls_v[c] = s_cls2 + ((pv >> (8 * c)) & 0xffu);
                LT best[CPT];
#pragma unroll
                for (int c = 0; c < CPT; ++c) best[c] = 0;
                const int ea_abs = eoff_p[i], eb_abs = eoff_p[i + 1];
                if (staged) {
                    const int ea = ea_abs - e0, eb = eb_abs - e0;
                    for (int e = ea; e < eb; ++e) {
                        const int np = npos_p[e];
                        const int span = FWD ? pos - np : np - pos;
                        LT lu[CPT];
                        unsigned pu;
                        if (FULL_WINDOW || span <= hit_span) {
                            const int slot = np & rmask;
                            load_win<CPT>(win_lev_lane + slot * SLICE, lu);
                            unsigned w[IdWords<CPT>::N];
                            load_ids<CPT>(win_id_lane + slot * SLICE, w);
                            pu = w[0];
                        } else {
                            const long long off = (long long)nbr_p[e] * ldp + jl;
                            long long lg[CPT];
                            load_levels<CPT>(a.lev + off, lg);
#pragma unroll
                            for (int c = 0; c < CPT; ++c) lu[c] = (LT)lg[c];
                            unsigned w[IdWords<CPT>::N];
                            load_ids<CPT>(a.part + off, w);
                            pu = w[0] & idmask;
                        }
                        const LT* vrow = V_p + e * ncomb;
#pragma unroll
                        for (int c = 0; c < CPT; ++c) {
                            const unsigned cls = cls_v[c][((pu >> (8 * c)) & 0xffu) * (unsigned)k];
                            best[c] = add_max(lu[c], vrow[cls], best[c]);
                        }
                    }
                } else {
                    // a vertex whose adjacency did not fit the staging buffers: everything from global memory
                    for (int e = ea_abs; e < eb_abs; ++e) {
                        const int np = wp.npos[e];
                        const int span = FWD ? pos - np : np - pos;
                        LT lu[CPT];
                        unsigned pu;
                        if (span <= hit_span) {
                            const int slot = np & rmask;
                            load_win<CPT>(win_lev_lane + slot * SLICE, lu);
                            unsigned w[IdWords<CPT>::N];
                            load_ids<CPT>(win_id_lane + slot * SLICE, w);
                            pu = w[0];
                        } else {
                            const long long off = (long long)a.adj.nbr[e] * ldp + jl;
                            long long lg[CPT];
                            load_levels<CPT>(a.lev + off, lg);
#pragma unroll
                            for (int c = 0; c < CPT; ++c) lu[c] = (LT)lg[c];
                            unsigned w[IdWords<CPT>::N];
                            load_ids<CPT>(a.part + off, w);
                            pu = w[0] & idmask;
                        }
                        const LT* vrow = reinterpret_cast<const LT*>(wp.V) + (long long)e * ncomb;
#pragma unroll
                        for (int c = 0; c < CPT; ++c) {
                            const unsigned cls = cls_v[c][((pu >> (8 * c)) & 0xffu) * (unsigned)k];
                            best[c] = add_max(lu[c], vrow[cls], best[c]);
                        }
                    }
                }
                const bool is_cp = want_cp && (FWD ? (vf < 0) : (pos < wp.src_end));
                if ((!FWD && ea_abs == eb_abs) || is_cp) {
                    const unsigned long long Xv = xvert_p[i];
                    if (!FWD && ea_abs == eb_abs) {  // sink: blevel = own runtime
#pragma unroll
                        for (int c = 0; c < CPT; ++c)
                            best[c] = Xv != NUM_ZERO ? (LT)ceil_quot(Xv, s_rt[(pv >> (8 * c)) & 0xffu]) : (LT)0;
                    }
                    if (is_cp) {
#pragma unroll
                        for (int c = 0; c < CPT; ++c) {
                            long long fin = (long long)best[c];
                            if (FWD && Xv != NUM_ZERO) fin += ceil_quot(Xv, s_rt[(pv >> (8 * c)) & 0xffu]);
                            cpmax[c] = fin > cpmax[c] ? fin : cpmax[c];
                        }
                    }
                }
                // results: global memory (the output) and the window
                long long* gout = a.lev + (long long)v * ldp + jl;
                long long wide[CPT];
#pragma unroll
                for (int c = 0; c < CPT; ++c) wide[c] = (long long)best[c];
                if (nvalid >= CPT) store_levels<CPT>(gout, wide);
                else {
#pragma unroll
                    for (int c = 0; c < CPT; ++c)
                        if (c < nvalid) gout[c] = wide[c];
                }
                if (R > 0) {
                    const int slot = pos & rmask;
                    store_win<CPT>(win_lev_lane + slot * SLICE, best);
                    pvw[0] = pv;
                    store_ids<CPT>(win_id_lane + slot * SLICE, pvw);
                }
            }
        }
        // consumers only: results of this chunk are in the window, its ring slots are free again
        asm volatile("bar.sync 1, %0;" ::"r"(ncons * 32) : "memory");
        if (threadIdx.x == 0) {
            __threadfence_block();
            *s_done = ci + 1;
        }
        if (*s_abort) break;
        if (++hs == NB) hs = 0;
        if (++ss == NS) { ss = 0; sp ^= 1u; }
    }
    __syncthreads();   // producer and consumers meet again
    if (*s_abort) {
        // copies that were already requested may still be landing in this block's shared memory: give them
        // a bounded time before the block (and its shared memory) goes away
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
        return;
    }

    if (want_cp) {
#pragma unroll
        for (int c = 0; c < CPT; ++c) s_cp[((size_t)warp * 32 + lane) * CPT + c] = cpmax[c];
        __syncthreads();
    }
    if (want_cp && warp == 0) {
#pragma unroll
        for (int c = 0; c < CPT; ++c) {
            long long m = cpmax[c];
            for (int w = 1; w < wpb; ++w) {
                long long o = s_cp[((size_t)w * 32 + lane) * CPT + c];
                m = o > m ? o : m;
            }
            if (c < nvalid) a.cp[j0 + c] = m;
        }
    }
}

// Packs one chunk's record.  head: int4 {p0, cnt, e0, staged edges or -1}, vertf[cnt].
// body: eoff[cnt+1], xvert[cnt], npos[es], V[es*ncomb] (lsize bytes each), nbr[es]; every array padded to 16 bytes.
__global__ void pack_chunks_kernel(const int4* __restrict__ chunks, const int4* __restrict__ desc,
                                   const int* __restrict__ vertf, const int* __restrict__ eptr,
                                   const unsigned long long* __restrict__ xvert, const int* __restrict__ npos,
                                   const int* __restrict__ nbr, const void* __restrict__ V, int ncomb, int lsize,
                                   unsigned char* blob)
{
    const int4 ch = chunks[blockIdx.x];
    const int4 d0 = desc[2 * blockIdx.x];
    const int p0 = ch.x, cnt = ch.y, e0 = ch.z, ecnt = ch.w;
    const int es = ecnt <= CHUNK_E ? ecnt : -1;
    const unsigned esz = es > 0 ? (unsigned)es : 0u;
    unsigned char* head = blob + 16ll * (unsigned)d0.x;
    unsigned char* body = blob + 16ll * (unsigned)d0.z;
    if (threadIdx.x == 0) *reinterpret_cast<int4*>(head) = make_int4(p0, cnt, e0, es);
    int* o_vertf = reinterpret_cast<int*>(head + 16);
    int* o_eoff = reinterpret_cast<int*>(body);
    unsigned long long* o_xvert = reinterpret_cast<unsigned long long*>(body + (((unsigned)(cnt + 1) * 4u + 15u) & ~15u));
    unsigned char* p_npos = reinterpret_cast<unsigned char*>(o_xvert) + (((unsigned)cnt * 8u + 15u) & ~15u);
    int* o_npos = reinterpret_cast<int*>(p_npos);
    unsigned char* p_V = p_npos + ((esz * 4u + 15u) & ~15u);
    unsigned char* p_nbr = p_V + ((esz * (unsigned)ncomb * (unsigned)lsize + 15u) & ~15u);
    int* o_nbr = reinterpret_cast<int*>(p_nbr);
    for (int i = threadIdx.x; i < cnt; i += blockDim.x) { o_vertf[i] = vertf[p0 + i]; o_xvert[i] = xvert[p0 + i]; }
    for (int i = threadIdx.x; i <= cnt; i += blockDim.x) o_eoff[i] = eptr[p0 + i];
    for (int i = threadIdx.x; i < (int)esz; i += blockDim.x) { o_npos[i] = npos[e0 + i]; o_nbr[i] = nbr[e0 + i]; }
    const int words = (int)esz * ncomb * (lsize / 4);
    const int* src = reinterpret_cast<const int*>(reinterpret_cast<const unsigned char*>(V) + (long long)e0 * ncomb * lsize);
    int* dst = reinterpret_cast<int*>(p_V);
    for (int i = threadIdx.x; i < words; i += blockDim.x) dst[i] = src[i];
}

// ---- set-up kernels ---------------------------------------------------------------------
__global__ void edge_values_kernel(int n, const int* __restrict__ eptr, const unsigned long long* __restrict__ xw,
                                   const unsigned long long* __restrict__ xnbr, const unsigned long long* __restrict__ xvert,
                                   const CombDiv* __restrict__ comb, int ncomb, long long* V, int* V32)
{
    const long long gw = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (gw >= n || lane >= ncomb) return;
    const CombDiv cd = comb[lane];
    const int e0 = eptr[gw], e1 = eptr[gw + 1];
    for (int e = e0; e < e1; ++e) {
        const unsigned long long X = xw[e];
        const unsigned long long Xr = xnbr ? xnbr[e] : xvert[gw];
        long long t = 0;
        if (cd.w.pad == 0 && X != NUM_ZERO) t = ceil_quot(X, cd.w);
        if (Xr != NUM_ZERO) t += ceil_quot(Xr, cd.s);
        V[(long long)e * ncomb + lane] = t;
        if (V32) V32[(long long)e * ncomb + lane] = (int)t;
    }
}

__global__ void pos_of_kernel(int n, const int* __restrict__ order, int* pos_of)
{
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) pos_of[order[i]] = i;
}

// neighbour positions of both directions; the largest forward span |pos(v) - pos(u)| over all edges
__global__ void npos_kernel(int n, const int* __restrict__ pos_of, const int* __restrict__ eptr_f,
                            const int* __restrict__ nbr_f, const int* __restrict__ nbr_b, int m, int* npos_f,
                            int* npos_b, int* maxspan)
{
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e < m) {
        npos_f[e] = pos_of[nbr_f[e]];
        npos_b[e] = pos_of[nbr_b[e]];
    }
    // spans: one thread per position walks its in-edges
    if (e < n) {
        int mx = 0;
        for (int q = eptr_f[e]; q < eptr_f[e + 1]; ++q) {
            const int s = e - pos_of[nbr_f[q]];
            mx = s > mx ? s : mx;
        }
        if (mx > 0) atomicMax(maxspan, mx);
    }
}

inline unsigned cdivu(long long a, long long b) { return (unsigned)((a + b - 1) / b); }

template <int CPT, bool FWD, int MODE, typename LT>
cudaError_t window_impl(const PassArgs& a, const WindowPlan& plan, int warps, cudaStream_t st)
{
    const Carve c = carve(a.tab.k, plan.R, CPT, warps, (int)sizeof(LT), plan.max_v, plan.head_max, plan.body_max, plan.depth);
    WinLayout L;
    L.bars = (unsigned)c.bars; L.rt = (unsigned)c.rt; L.cls2 = (unsigned)c.cls2; L.cp = (unsigned)c.cp;
    L.head = (unsigned)c.head; L.head_stride = (unsigned)c.head_stride;
    L.body = (unsigned)c.body; L.body_stride = (unsigned)c.body_stride;
    L.ids = (unsigned)c.ids; L.ids_stride = (unsigned)c.ids_stride;
    L.win_lev = (unsigned)c.win_lev; L.win_id = (unsigned)c.win_id;
    L.depth = plan.depth;
    cudaError_t e = cudaFuncSetAttribute(pass_window_kernel<CPT, FWD, MODE, LT>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c.total);
    if (e != cudaSuccess) return e;
    pass_window_kernel<CPT, FWD, MODE, LT><<<cdivu(a.P, 32 * CPT), warps * 32, c.total, st>>>(a, plan, L);
    count_launches(1);
    return cudaGetLastError();
}

template <int CPT, typename LT>
cudaError_t window_dispatch(const PassArgs& a, bool fwd, const WindowPlan& plan, int warps, cudaStream_t st)
{
    if (plan.all_staged && plan.R - CHUNK_V >= plan.maxspan)
        return fwd ? window_impl<CPT, true, 2, LT>(a, plan, warps, st) : window_impl<CPT, false, 2, LT>(a, plan, warps, st);
    if (plan.all_staged)
        return fwd ? window_impl<CPT, true, 1, LT>(a, plan, warps, st) : window_impl<CPT, false, 1, LT>(a, plan, warps, st);
    return fwd ? window_impl<CPT, true, 0, LT>(a, plan, warps, st) : window_impl<CPT, false, 0, LT>(a, plan, warps, st);
}

}  // namespace

size_t window_smem_bytes(int k, int R, int cpt, int warps, int level_bytes, int max_v, int head_max, int body_max, int depth)
{
    return carve(k, R, cpt, warps, level_bytes, max_v, head_max, body_max, depth).total;
}

cudaError_t launch_pack_chunks(int num_chunks, const int* chunks, const int* desc, const int* vertf, const int* eptr,
                               const unsigned long long* xvert, const int* npos, const int* nbr, const void* V, int ncomb,
                               int lsize, unsigned char* blob, cudaStream_t st)
{
    if (num_chunks <= 0) return cudaSuccess;
    pack_chunks_kernel<<<num_chunks, 128, 0, st>>>(reinterpret_cast<const int4*>(chunks), reinterpret_cast<const int4*>(desc),
                                                   vertf, eptr, xvert, npos, nbr, V, ncomb, lsize, blob);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_pass_window(const PassArgs& a, bool fwd, const WindowPlan& plan, int cpt, int warps, cudaStream_t st)
{
    if (plan.num_chunks <= 0) return cudaSuccess;
    if (plan.level_bytes == 4) {
        if (cpt == 4) return window_dispatch<4, int>(a, fwd, plan, warps, st);
        if (cpt == 2) return window_dispatch<2, int>(a, fwd, plan, warps, st);
        return window_dispatch<1, int>(a, fwd, plan, warps, st);
    }
    if (cpt == 4) return window_dispatch<4, long long>(a, fwd, plan, warps, st);
    if (cpt == 2) return window_dispatch<2, long long>(a, fwd, plan, warps, st);
    return window_dispatch<1, long long>(a, fwd, plan, warps, st);
}

cudaError_t launch_edge_values(int n, const int* eptr, const unsigned long long* xw, const unsigned long long* xnbr,
                               const unsigned long long* xvert, const CombDiv* comb, int ncomb, long long* V, int* V32,
                               cudaStream_t st)
{
    if (n <= 0) return cudaSuccess;
    edge_values_kernel<<<cdivu((long long)n * 32, 256), 256, 0, st>>>(n, eptr, xw, xnbr, xvert, comb, ncomb, V, V32);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_positions(int n, int m, const int* order, int* pos_of, const int* nbr_f, const int* nbr_b,
                             const int* eptr_f, int* npos_f, int* npos_b, int* maxspan, cudaStream_t st)
{
    if (n <= 0) return cudaSuccess;
    pos_of_kernel<<<cdivu(n, 256), 256, 0, st>>>(n, order, pos_of);
    const int work = n > m ? n : m;
    npos_kernel<<<cdivu(work, 256), 256, 0, st>>>(n, pos_of, eptr_f, nbr_f, nbr_b, m, npos_f, npos_b, maxspan);
    count_launches(2);
    return cudaGetLastError();
}

}  // namespace tfps
