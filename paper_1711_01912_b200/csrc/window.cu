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

constexpr unsigned FULL = 0xffffffffu;

__device__ __forceinline__ void cp_async4(void* smem, const void* g)
{
    unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(s), "l"(g));
}
__device__ __forceinline__ void cp_async8(void* smem, const void* g)
{
    unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(s), "l"(g));
}
__device__ __forceinline__ void cp_async16(void* smem, const void* g)
{
    unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s), "l"(g));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

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

struct HeadBuf {                 // per-vertex metadata of a chunk
    unsigned long long xvert[CHUNK_V];
    int vertf[CHUNK_V];
    int eoff[CHUNK_V + 4];
};

// shared-memory carve-up (all offsets multiples of 16 bytes)
struct Carve {
    size_t head, edge_nbr, edge_npos, edge_V, ids, rt, cls2, cp, win_lev, win_id, total;
    size_t edge_stride, ids_stride;
};

__host__ __device__ inline size_t up16(size_t x) { return (x + 15) & ~(size_t)15; }

__host__ __device__ inline Carve carve(int k, int ncomb, int R, int cpt, int warps, int lsize)
{
    Carve c;
    const size_t slice = 32 * (size_t)cpt;
    size_t o = 0;
    c.head = o; o += 3 * up16(sizeof(HeadBuf));
    c.edge_nbr = o;
    c.edge_npos = c.edge_nbr + up16(sizeof(int) * CHUNK_E) + 16;
    c.edge_V = c.edge_npos + up16(sizeof(int) * CHUNK_E) + 16;
    c.edge_stride = (c.edge_V - c.edge_nbr) + up16((size_t)lsize * CHUNK_E * (size_t)ncomb) + 16;
    o += 2 * c.edge_stride;
    c.ids = o; c.ids_stride = up16(CHUNK_V * slice); o += 2 * c.ids_stride;
    c.rt = o; o += up16(sizeof(DivConst) * (size_t)k);
    c.cls2 = o; o += up16((size_t)k * k);
    c.cp = c.ids;  // the id staging area doubles as the reduction buffer of the CP maxima after the last chunk
    (void)warps;
    c.win_lev = o; o += up16((size_t)lsize * (size_t)R * slice);
    c.win_id = o; o += up16((size_t)R * slice);
    c.total = o;
    return c;
}

// 32-bit shared-state-space accessors (addresses from __cvta_generic_to_shared)
__device__ __forceinline__ unsigned lds_u8(unsigned a) { unsigned v; asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(a)); return v; }
__device__ __forceinline__ unsigned lds_u16(unsigned a) { unsigned v; asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(a)); return v; }
__device__ __forceinline__ unsigned lds_u32(unsigned a) { unsigned v; asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a)); return v; }
__device__ __forceinline__ long long lds_s64(unsigned a) { long long v; asm volatile("ld.shared.s64 %0, [%1];" : "=l"(v) : "r"(a)); return v; }
__device__ __forceinline__ void lds_v2s64(unsigned a, long long& x, long long& y) { asm volatile("ld.shared.v2.s64 {%0,%1}, [%2];" : "=l"(x), "=l"(y) : "r"(a)); }
__device__ __forceinline__ void sts_s64(unsigned a, long long v) { asm volatile("st.shared.s64 [%0], %1;" ::"r"(a), "l"(v) : "memory"); }
__device__ __forceinline__ void sts_v2s64(unsigned a, long long x, long long y) { asm volatile("st.shared.v2.s64 [%0], {%1,%2};" ::"r"(a), "l"(x), "l"(y) : "memory"); }
__device__ __forceinline__ void sts_u8(unsigned a, unsigned v) { asm volatile("st.shared.u8 [%0], %1;" ::"r"(a), "r"(v) : "memory"); }
__device__ __forceinline__ void sts_u16(unsigned a, unsigned v) { asm volatile("st.shared.u16 [%0], %1;" ::"r"(a), "r"(v) : "memory"); }
__device__ __forceinline__ void sts_u32(unsigned a, unsigned v) { asm volatile("st.shared.u32 [%0], %1;" ::"r"(a), "r"(v) : "memory"); }

template <int CPT> __device__ __forceinline__ unsigned lds_ids(unsigned a)
{
    if constexpr (CPT == 1) return lds_u8(a);
    else if constexpr (CPT == 2) return lds_u16(a);
    else return lds_u32(a);
}
template <int CPT> __device__ __forceinline__ void sts_ids(unsigned a, unsigned v)
{
    if constexpr (CPT == 1) sts_u8(a, v);
    else if constexpr (CPT == 2) sts_u16(a, v);
    else sts_u32(a, v);
}
template <int CPT> __device__ __forceinline__ void lds_levels(unsigned a, long long (&out)[CPT])
{
    if constexpr (CPT == 1) out[0] = lds_s64(a);
    else {
#pragma unroll
        for (int i = 0; i < CPT; i += 2) lds_v2s64(a + 8 * i, out[i], out[i + 1]);
    }
}
template <int CPT> __device__ __forceinline__ void sts_levels(unsigned a, const long long (&v)[CPT])
{
    if constexpr (CPT == 1) sts_s64(a, v[0]);
    else {
#pragma unroll
        for (int i = 0; i < CPT; i += 2) sts_v2s64(a + 8 * i, v[i], v[i + 1]);
    }
}
// 32-bit level mode
template <int CPT> __device__ __forceinline__ void lds_levels(unsigned a, int (&out)[CPT])
{
    if constexpr (CPT == 1) out[0] = (int)lds_u32(a);
    else if constexpr (CPT == 2) asm volatile("ld.shared.v2.s32 {%0,%1}, [%2];" : "=r"(out[0]), "=r"(out[1]) : "r"(a));
    else asm volatile("ld.shared.v4.s32 {%0,%1,%2,%3}, [%4];" : "=r"(out[0]), "=r"(out[1]), "=r"(out[2]), "=r"(out[3]) : "r"(a));
}
template <int CPT> __device__ __forceinline__ void sts_levels(unsigned a, const int (&v)[CPT])
{
    if constexpr (CPT == 1) sts_u32(a, (unsigned)v[0]);
    else if constexpr (CPT == 2) asm volatile("st.shared.v2.s32 [%0], {%1,%2};" ::"r"(a), "r"(v[0]), "r"(v[1]) : "memory");
    else asm volatile("st.shared.v4.s32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]) : "memory");
}
__device__ __forceinline__ long long lds_level1(unsigned a, long long) { return lds_s64(a); }
__device__ __forceinline__ int lds_level1(unsigned a, int) { return (int)lds_u32(a); }
// best = max(best, lu + w)
__device__ __forceinline__ long long add_max(long long lu, long long w, long long best) { const long long v = lu + w; return v > best ? v : best; }
__device__ __forceinline__ int add_max(int lu, int w, int best) { return __viaddmax_s32(lu, w, best); }

// Copies `bytes` (a multiple of 4) from 4-byte aligned global memory into the staging area `dst_area`, keeping
// the source's offset inside its 16-byte line so that the body moves as 16-byte cp.async; returns that offset.
__device__ __forceinline__ unsigned stage_bytes(unsigned char* dst_area, const void* src, int bytes)
{
    const unsigned mis = (unsigned)((unsigned long long)src & 15ull);
    unsigned char* dst = dst_area + mis;
    const unsigned char* s = reinterpret_cast<const unsigned char*>(src);
    int head = (int)((16u - mis) & 15u);
    if (head > bytes) head = bytes;
    const int body = (bytes - head) & ~15;
    const int tail = bytes - head - body;
    for (int i = threadIdx.x * 16; i < body; i += blockDim.x * 16) cp_async16(dst + head + i, s + head + i);
    const int t4 = threadIdx.x * 4;
    if (t4 < head) cp_async4(dst + t4, s + t4);
    if (t4 < tail) cp_async4(dst + head + body + t4, s + head + body + t4);
    return mis;
}

// Byte offsets of the shared-memory regions, computed on the host and passed as a kernel parameter.
struct WinLayout {
    unsigned head, head_stride;
    unsigned edge_nbr, edge_npos, edge_V, edge_stride;
    unsigned ids, ids_stride;
    unsigned rt, cls2, cp, win_lev, win_id;
};

// ALL_STAGED: every chunk's adjacency fits the staging buffers (no vertex with more than CHUNK_E edges).
template <int CPT, bool FWD, bool ALL_STAGED, typename LT>
__global__ void __launch_bounds__(1024)
pass_window_kernel(PassArgs a, WindowPlan wp, WinLayout L)
{
    extern __shared__ __align__(16) unsigned char smem[];
    constexpr int SLICE = 32 * CPT;
    constexpr unsigned LS = sizeof(LT);   // bytes of a level inside the block: 4 when every path length fits int32
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, wpb = blockDim.x >> 5;
    const int k = a.tab.k;
    const int ncomb = wp.ncomb;
    const int R = wp.R;              // power of two (or 0)
    const int rmask = R - 1;
    const int hit_span = R - CHUNK_V;  // a neighbour at most this many positions away is still in the ring
    const unsigned sbase = (unsigned)__cvta_generic_to_shared(smem);
    DivConst* s_rt = reinterpret_cast<DivConst*>(smem + L.rt);
    long long* s_cp = reinterpret_cast<long long*>(smem + L.cp);
    if (*a.status != 0) return;
    for (int i = threadIdx.x; i < k; i += blockDim.x) s_rt[i] = a.tab.rt_div[i];
    for (int i = threadIdx.x; i < k * k; i += blockDim.x) smem[L.cls2 + i] = wp.cls2[i];

    const long long slice0 = (long long)blockIdx.x * SLICE;
    const long long j0 = slice0 + (long long)lane * CPT;
    const long long rem = a.P - j0;
    const int nvalid = rem >= CPT ? CPT : (rem > 0 ? (int)rem : 0);
    const int lane_col = nvalid > 0 ? lane * CPT : 0;      // idle lanes shadow the slice's first lane
    const long long jl = slice0 + lane_col;
    const unsigned idmask = nvalid >= 4 ? 0xffffffffu : (nvalid > 0 ? ((1u << (8 * nvalid)) - 1u) : 0u);
    const long long ldp = a.ldp;
    const int slice_bytes = (int)((ldp - slice0) < SLICE ? (ldp - slice0) : SLICE);
    const bool want_cp = a.cp != nullptr;
    long long cpmax[CPT];
#pragma unroll
    for (int c = 0; c < CPT; ++c) cpmax[c] = 0;
    // per-lane shared addresses
    const unsigned win_lev_lane = sbase + L.win_lev + LS * (unsigned)(lane * CPT);
    const unsigned win_id_lane = sbase + L.win_id + (unsigned)(lane * CPT);
    const unsigned cls2_s = sbase + L.cls2;

    const int4* chunks = reinterpret_cast<const int4*>(wp.chunks);
    const int num_chunks = wp.num_chunks;
    auto entry = [&](int ci) { return chunks[FWD ? ci : num_chunks - 1 - ci]; };
    auto stage_head = [&](int4 ent, int slot) {
        HeadBuf& h = *reinterpret_cast<HeadBuf*>(smem + L.head + (unsigned)slot * L.head_stride);
        const int p0 = ent.x, cnt = ent.y;
        for (int i = threadIdx.x; i < cnt; i += blockDim.x) {
            cp_async4(&h.vertf[i], wp.vertf + p0 + i);
            cp_async8(&h.xvert[i], a.adj.xvert + p0 + i);
        }
        for (int i = threadIdx.x; i <= cnt; i += blockDim.x) cp_async4(&h.eoff[i], a.adj.eptr + p0 + i);
    };
    // returns the byte offsets at which the staged npos / nbr / V arrays start inside their areas
    auto stage_edges = [&](int4 ent, int slot, unsigned (&mis)[3]) {
        const int e0 = ent.z, ecnt = ent.w;
        mis[0] = mis[1] = mis[2] = 0;
        if (!ALL_STAGED && ecnt > CHUNK_E) return;  // read from global memory instead
        unsigned char* base = smem + (unsigned)slot * L.edge_stride;
        mis[0] = stage_bytes(base + L.edge_npos, wp.npos + e0, ecnt * 4);
        if (hit_span < wp.maxspan || !ALL_STAGED)  // neighbour ids are only needed for window misses
            mis[1] = stage_bytes(base + L.edge_nbr, a.adj.nbr + e0, ecnt * 4);
        const unsigned char* Vg = reinterpret_cast<const unsigned char*>(wp.V) + (long long)e0 * ncomb * (long long)LS;
        mis[2] = stage_bytes(base + L.edge_V, Vg, ecnt * ncomb * (int)LS);
    };
    auto stage_ids = [&](int4 ent, int head_slot, int slot) {
        const HeadBuf& h = *reinterpret_cast<const HeadBuf*>(smem + L.head + (unsigned)head_slot * L.head_stride);
        const int cnt = ent.y;
        uint8_t* dst = smem + L.ids + (unsigned)slot * L.ids_stride;
        const int per_row = slice_bytes >> 4;  // ldp and slice0 are multiples of 16
        for (int i = threadIdx.x; i < cnt * per_row; i += blockDim.x) {
            const int r = i / per_row, q = i - r * per_row;
            const int v = h.vertf[r] & 0x7fffffff;
            cp_async16(dst + r * SLICE + 16 * q, a.part + (long long)v * ldp + slice0 + 16 * q);
        }
    };

    int4 cur = entry(0);
    int4 nxt = num_chunks > 1 ? entry(1) : cur;
    int4 nxt2 = num_chunks > 2 ? entry(2) : cur;
    unsigned mis_cur[3], mis_nxt[3] = {0, 0, 0};
    stage_head(cur, 0);
    if (num_chunks > 1) stage_head(nxt, 1);
    stage_edges(cur, 0, mis_cur);
    cp_async_commit();
    cp_async_wait_all();
    __syncthreads();
    stage_ids(cur, 0, 0);
    cp_async_commit();
    cp_async_wait_all();
    __syncthreads();

    int hslot = 0;  // ci % 3
    for (int ci = 0; ci < num_chunks; ++ci) {
        const int hs1 = hslot == 2 ? 0 : hslot + 1;
        const int hs2 = hs1 == 2 ? 0 : hs1 + 1;
        int4 nxt3 = nxt2;
        if (ci + 1 < num_chunks) {
            stage_ids(nxt, hs1, (ci + 1) & 1);
            stage_edges(nxt, (ci + 1) & 1, mis_nxt);
            if (ci + 2 < num_chunks) {
                stage_head(nxt2, hs2);
                if (ci + 3 < num_chunks) nxt3 = entry(ci + 3);
            }
            cp_async_commit();
        }
        const unsigned head_s = sbase + L.head + (unsigned)hslot * L.head_stride;
        const unsigned xvert_s = head_s;                                   // HeadBuf::xvert
        const unsigned vertf_s = head_s + 8u * CHUNK_V;                    // HeadBuf::vertf
        const unsigned eoff_s = vertf_s + 4u * CHUNK_V;                    // HeadBuf::eoff
        const int p0 = cur.x, cnt = cur.y, e0 = cur.z;
        const bool staged = ALL_STAGED || cur.w <= CHUNK_E;
        const unsigned ebase_s = sbase + (unsigned)(ci & 1) * L.edge_stride;
        const unsigned npos_s = ebase_s + L.edge_npos + mis_cur[0];
        const unsigned nbr_s = ebase_s + L.edge_nbr + mis_cur[1];
        const unsigned V_s = ebase_s + L.edge_V + mis_cur[2];
        const unsigned idrow_lane = sbase + L.ids + (unsigned)(ci & 1) * L.ids_stride + (unsigned)lane_col;

        for (int i = warp; i < cnt; i += wpb) {
            const int vf = (int)lds_u32(vertf_s + 4u * i);
            const int v = vf & 0x7fffffff;
            const int pos = p0 + i;
            const unsigned pv = lds_ids<CPT>(idrow_lane + (unsigned)(i * SLICE)) & idmask;
            unsigned cls_v[CPT];   // shared address of cls2[0*k + idv]
#pragma unroll
            for (int c = 0; c < CPT; ++c) cls_v[c] = cls2_s + ((pv >> (8 * c)) & 0xffu);
            LT best[CPT];
#pragma unroll
            for (int c = 0; c < CPT; ++c) best[c] = 0;
            const int ea_abs = (int)lds_u32(eoff_s + 4u * i), eb_abs = (int)lds_u32(eoff_s + 4u * i + 4u);
            if (staged) {
                const int ea = ea_abs - e0, eb = eb_abs - e0;
                for (int e = ea; e < eb; ++e) {
                    const int np = (int)lds_u32(npos_s + 4u * e);
                    const int span = FWD ? pos - np : np - pos;
                    LT lu[CPT];
                    unsigned pu;
                    if (span <= hit_span) {
                        const unsigned slot = (unsigned)(np & rmask);
                        lds_levels<CPT>(win_lev_lane + slot * (LS * SLICE), lu);
                        pu = lds_ids<CPT>(win_id_lane + slot * (unsigned)SLICE);
                    } else {
                        const long long off = (long long)(int)lds_u32(nbr_s + 4u * e) * ldp + jl;
                        long long lg[CPT];
                        load_levels<CPT>(a.lev + off, lg);
#pragma unroll
                        for (int c = 0; c < CPT; ++c) lu[c] = (LT)lg[c];
                        unsigned w[IdWords<CPT>::N];
                        load_ids<CPT>(a.part + off, w);
                        pu = w[0] & idmask;
                    }
                    const unsigned vrow = V_s + LS * (unsigned)(e * ncomb);
#pragma unroll
                    for (int c = 0; c < CPT; ++c) {
                        const unsigned cls = lds_u8(cls_v[c] + ((pu >> (8 * c)) & 0xffu) * (unsigned)k);
                        best[c] = add_max(lu[c], lds_level1(vrow + LS * cls, LT()), best[c]);
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
                        const unsigned slot = (unsigned)(np & rmask);
                        lds_levels<CPT>(win_lev_lane + slot * (LS * SLICE), lu);
                        pu = lds_ids<CPT>(win_id_lane + slot * (unsigned)SLICE);
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
                        const unsigned cls = lds_u8(cls_v[c] + ((pu >> (8 * c)) & 0xffu) * (unsigned)k);
                        best[c] = add_max(lu[c], vrow[cls], best[c]);
                    }
                }
            }
            const bool is_cp = want_cp && (FWD ? (vf < 0) : (pos < wp.src_end));
            if ((!FWD && ea_abs == eb_abs) || is_cp) {
                const unsigned long long Xv = (unsigned long long)lds_s64(xvert_s + 8u * i);
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
                const unsigned slot = (unsigned)(pos & rmask);
                sts_levels<CPT>(win_lev_lane + slot * (LS * SLICE), best);
                sts_ids<CPT>(win_id_lane + slot * (unsigned)SLICE, pv);
            }
        }
        cp_async_wait_all();
        __syncthreads();
        cur = nxt; nxt = nxt2; nxt2 = nxt3;
        mis_cur[0] = mis_nxt[0]; mis_cur[1] = mis_nxt[1]; mis_cur[2] = mis_nxt[2];
        hslot = hs1;
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

template <int CPT, bool FWD, bool ALL_STAGED, typename LT>
cudaError_t window_impl(const PassArgs& a, const WindowPlan& plan, int warps, cudaStream_t st)
{
    const Carve c = carve(a.tab.k, plan.ncomb, plan.R, CPT, warps, (int)sizeof(LT));
    WinLayout L;
    L.head = (unsigned)c.head; L.head_stride = (unsigned)up16(sizeof(HeadBuf));
    L.edge_nbr = (unsigned)c.edge_nbr; L.edge_npos = (unsigned)c.edge_npos; L.edge_V = (unsigned)c.edge_V;
    L.edge_stride = (unsigned)c.edge_stride;
    L.ids = (unsigned)c.ids; L.ids_stride = (unsigned)c.ids_stride;
    L.rt = (unsigned)c.rt; L.cls2 = (unsigned)c.cls2; L.cp = (unsigned)c.cp;
    L.win_lev = (unsigned)c.win_lev; L.win_id = (unsigned)c.win_id;
    cudaError_t e = cudaFuncSetAttribute(pass_window_kernel<CPT, FWD, ALL_STAGED, LT>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c.total);
    if (e != cudaSuccess) return e;
    pass_window_kernel<CPT, FWD, ALL_STAGED, LT><<<cdivu(a.P, 32 * CPT), warps * 32, c.total, st>>>(a, plan, L);
    count_launches(1);
    return cudaGetLastError();
}

template <int CPT, typename LT>
cudaError_t window_dispatch(const PassArgs& a, bool fwd, const WindowPlan& plan, int warps, cudaStream_t st)
{
    if (plan.all_staged)
        return fwd ? window_impl<CPT, true, true, LT>(a, plan, warps, st) : window_impl<CPT, false, true, LT>(a, plan, warps, st);
    return fwd ? window_impl<CPT, true, false, LT>(a, plan, warps, st) : window_impl<CPT, false, false, LT>(a, plan, warps, st);
}

}  // namespace

size_t window_smem_bytes(int k, int ncomb, int R, int cpt, int warps, int level_bytes)
{
    return carve(k, ncomb, R, cpt, warps, level_bytes).total;
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
