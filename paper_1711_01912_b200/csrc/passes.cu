// Forward (tlevel) and backward (blevel = PCT, Eq. 12) longest-path passes over
// the vertex-major [n][ldp] candidate layout, critical-path reduction, per-
// device load / memory reduction, id validation and the uint8 transpose.
//
// Lane = candidate(s): a warp covers 32*CPT contiguous candidates of one
// vertex, so every neighbour-level read is one contiguous 256*CPT-byte row
// segment and every id read a contiguous 32*CPT-byte one.
#include <cstdlib>

#include "common.cuh"

namespace tfps {

namespace {

// ---- small vector helpers ----------------------------------------------------
constexpr unsigned FULL = 0xffffffffu;

template <int CPT> struct IdWords { static constexpr int N = (CPT + 3) / 4; };

// CPT partition ids (one byte each) starting at p, packed little-endian into 32-bit words
template <int CPT>
__device__ __forceinline__ void load_ids(const uint8_t* p, unsigned (&w)[IdWords<CPT>::N])
{
    if constexpr (CPT == 1) w[0] = *p;
    else if constexpr (CPT == 2) w[0] = *reinterpret_cast<const unsigned short*>(p);
    else if constexpr (CPT == 4) w[0] = *reinterpret_cast<const unsigned*>(p);
    else {
        static_assert(CPT == 8, "CPT must be 1, 2, 4 or 8");
        const uint2 v = *reinterpret_cast<const uint2*>(p);
        w[0] = v.x;
        w[1] = v.y;
    }
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
__device__ __forceinline__ void store_levels(long long* p, const long long (&v)[CPT], int nvalid)
{
    if (nvalid >= CPT) {
        if constexpr (CPT == 1) {
            *p = v[0];
        } else {
#pragma unroll
            for (int i = 0; i < CPT; i += 2) *reinterpret_cast<longlong2*>(p + i) = make_longlong2(v[i], v[i + 1]);
        }
    } else {
#pragma unroll
        for (int i = 0; i < CPT; ++i)
            if (i < nvalid) p[i] = v[i];
    }
}

__device__ __forceinline__ long long shfl64(long long v, int src)
{
    int lo = __shfl_sync(FULL, (int)(unsigned)(unsigned long long)v, src);
    int hi = __shfl_sync(FULL, (int)((unsigned long long)v >> 32), src);
    return (long long)(((unsigned long long)(unsigned)hi << 32) | (unsigned)lo);
}

// Shared-memory copy of the division constants: [k*k] pair table then [k] speed table.
__device__ __forceinline__ void stage_tables(const DevTables& tab, DivConst* s_w, DivConst* s_rt)
{
    const int k = tab.k;
    for (int i = threadIdx.x; i < k * k; i += blockDim.x) s_w[i] = tab.w_div[i];
    for (int i = threadIdx.x; i < k; i += blockDim.x) s_rt[i] = tab.rt_div[i];
    __syncthreads();
}

// Per-lane candidate bookkeeping shared by the pass kernels.
template <int CPT>
struct LaneCtx {
    long long jl;                         // (always in-bounds) first column the lane loads from
    int nvalid;                           // how many of the lane's CPT candidates are real
    unsigned maskw[IdWords<CPT>::N];      // zeroes the ids of padding candidates
};

template <int CPT>
__device__ __forceinline__ LaneCtx<CPT> lane_setup(long long slice0, long long P, int lane)
{
    LaneCtx<CPT> lc;
    const long long j0 = slice0 + (long long)lane * CPT;
    const long long rem = P - j0;
    lc.nvalid = rem >= CPT ? CPT : (rem > 0 ? (int)rem : 0);
    lc.jl = lc.nvalid > 0 ? j0 : slice0;  // idle lanes shadow the slice's first lane and never store
#pragma unroll
    for (int w = 0; w < IdWords<CPT>::N; ++w) {
        const int nv = lc.nvalid - 4 * w;  // valid bytes in this word
        lc.maskw[w] = nv >= 4 ? 0xffffffffu : (nv > 0 ? ((1u << (8 * nv)) - 1u) : 0u);
    }
    return lc;
}

template <int CPT>
__device__ __forceinline__ void load_ids_masked(const uint8_t* p, const LaneCtx<CPT>& lc, unsigned (&w)[IdWords<CPT>::N])
{
    load_ids<CPT>(p, w);
#pragma unroll
    for (int i = 0; i < IdWords<CPT>::N; ++i) w[i] &= lc.maskw[i];
}

// ---- one vertex, 32*CPT candidates --------------------------------------------
// Where the adjacency of the vertex being relaxed comes from: global memory
// (level-synchronous kernel, oversized chunks) or the staged copy in shared memory.
struct VertexMeta {
    int v;                             // vertex id
    int e0, e1;                        // edge range, as indices into the three arrays below
    const int* nbr;                    // neighbour vertex ids
    const unsigned long long* xw;      // transfer numerators
    const unsigned long long* xnbr;    // neighbour runtime numerators (forward only)
    unsigned long long xvert;          // own runtime numerator
};

// Direct form: every relaxation divides on its own (any k).
// FWD: best = max over in-edges of tlevel(u) + rt(u) + w(u->v); writes tlevel(v).
// BWD: best = max over out-edges of blevel(x) + w(v->x); writes blevel(v) = best + rt(v).
// cpmax accumulates tlevel+rt over sinks (FWD) or blevel over sources (BWD).
template <int CPT, bool FWD>
__device__ __forceinline__ void relax_vertex(const PassArgs& a, const DivConst* __restrict__ s_w,
                                             const DivConst* __restrict__ s_rt, const VertexMeta& vm,
                                             const LaneCtx<CPT>& lc, bool cp_vertex, long long* cpmax)
{
    const int k = a.tab.k;
    const int v = vm.v;
    const int e0 = vm.e0;
    const int e1 = vm.e1;
    const long long ldp = a.ldp;
    unsigned pv[IdWords<CPT>::N];
    load_ids_masked<CPT>(a.part + (long long)v * ldp + lc.jl, lc, pv);

    long long best[CPT];
#pragma unroll
    for (int c = 0; c < CPT; ++c) best[c] = 0;

    constexpr int UNR = (CPT >= 4) ? 2 : 4;
    for (int e = e0; e < e1; e += UNR) {
        long long lu[UNR][CPT];
        unsigned pu[UNR][IdWords<CPT>::N];
        unsigned long long X[UNR], Xn[UNR];
#pragma unroll
        for (int q = 0; q < UNR; ++q) {
            if (e + q < e1) {
                const int u = vm.nbr[e + q];
                X[q] = vm.xw[e + q];
                if (FWD) Xn[q] = vm.xnbr[e + q];
                const long long off = (long long)u * ldp + lc.jl;
                load_ids_masked<CPT>(a.part + off, lc, pu[q]);
                load_levels<CPT>(a.lev + off, lu[q]);
            }
        }
#pragma unroll
        for (int q = 0; q < UNR; ++q) {
            if (e + q < e1) {
#pragma unroll
                for (int c = 0; c < CPT; ++c) {
                    const unsigned idu = id_at<CPT>(pu[q], c);
                    const unsigned idv = id_at<CPT>(pv, c);
                    long long val = lu[q][c];
                    if (X[q] != NUM_ZERO) {
                        const DivConst dc = s_w[FWD ? idu * k + idv : idv * k + idu];
                        const long long w = ceil_quot(X[q], dc);
                        val += (idu != idv) ? w : 0;
                    }
                    if (FWD) {
                        if (Xn[q] != NUM_ZERO) val += ceil_quot(Xn[q], s_rt[idu]);
                    }
                    best[c] = val > best[c] ? val : best[c];
                }
            }
        }
    }

    const unsigned long long Xv = vm.xvert;
    if (!FWD) {
#pragma unroll
        for (int c = 0; c < CPT; ++c)
            if (Xv != NUM_ZERO) best[c] += ceil_quot(Xv, s_rt[id_at<CPT>(pv, c)]);
    }
    store_levels<CPT>(a.lev + (long long)v * ldp + lc.jl, best, lc.nvalid);
    if (cp_vertex) {
#pragma unroll
        for (int c = 0; c < CPT; ++c) {
            long long fin = best[c];
            if (FWD && Xv != NUM_ZERO) fin += ceil_quot(Xv, s_rt[id_at<CPT>(pv, c)]);
            cpmax[c] = fin > cpmax[c] ? fin : cpmax[c];
        }
    }
}

// Table form (k <= TABLE_K_MAX).  The cost of an edge depends on the candidate
// only through the pair (device of the neighbour nb, device of the vertex vv),
// so the warp first fills a k*k table for the edge,
//   FWD: T[nb*k+vv] = rt(u on nb) + w(nb -> vv),   BWD: T[nb*k+vv] = rt(v on vv) + w(vv -> nb),
// one entry per lane and pass, and every candidate then needs a single
// shared-memory lookup instead of two 64-bit divisions.  The neighbour's ids
// and levels are requested before the table is built, so the build overlaps
// their latency.
struct TableCtx {
    const DivConst* s_pair;         // [npass*32] pair divisors of this direction (+ dev | diag << 8)
    const DivConst* s_rt;           // [k] speed divisors
    const unsigned short* s_sel;    // [npass*32] class selectors, valid when use_cls
    long long* T;                   // this warp's table, npass*32 entries
    DivConst my_cls;                // class divisor of this lane, valid when use_cls
    int npass;
    int use_cls;
    int ncls_w;
};

template <bool FWD>
__device__ __forceinline__ void build_edge_table(const TableCtx& tc, unsigned long long X, unsigned long long Xr, int lane)
{
    __syncwarp();  // lookups of the previous edge are done
    if (tc.use_cls) {
        // one division per distinct bandwidth / speed value, spread to the entries by shuffles
        const unsigned long long num = lane < tc.ncls_w ? X : Xr;
        const long long val = num != NUM_ZERO ? ceil_quot(num, tc.my_cls) : 0;
        for (int p = 0; p < tc.npass; ++p) {
            const int i = lane + 32 * p;
            const unsigned sel = tc.s_sel[i];
            const unsigned cw = sel & 0xffu;
            long long w = shfl64(val, (int)(cw & 31u));
            const long long r = shfl64(val, (int)(sel >> 8));
            if (cw == 255u) w = 0;
            tc.T[i] = w + r;
        }
    } else {
        for (int p = 0; p < tc.npass; ++p) {
            const int i = lane + 32 * p;
            const DivConst dc = tc.s_pair[i];
            long long t = 0;
            if (X != NUM_ZERO && (dc.pad & 256u) == 0) t = ceil_quot(X, dc);
            if (Xr != NUM_ZERO) t += ceil_quot(Xr, tc.s_rt[dc.pad & 0xffu]);
            tc.T[i] = t;
        }
    }
    __syncwarp();
}

template <int CPT, bool FWD>
__device__ __forceinline__ void relax_vertex_table(const PassArgs& a, const TableCtx& tc, const VertexMeta& vm,
                                                   const LaneCtx<CPT>& lc, int lane, bool cp_vertex, long long* cpmax)
{
    const int k = a.tab.k;
    const int v = vm.v;
    const long long ldp = a.ldp;
    unsigned pv[IdWords<CPT>::N];
    load_ids_masked<CPT>(a.part + (long long)v * ldp + lc.jl, lc, pv);
    const unsigned long long Xv = vm.xvert;

    long long best[CPT];
#pragma unroll
    for (int c = 0; c < CPT; ++c) best[c] = 0;

    for (int e = vm.e0; e < vm.e1; ++e) {
        const int u = vm.nbr[e];
        const unsigned long long X = vm.xw[e];
        const unsigned long long Xr = FWD ? vm.xnbr[e] : Xv;
        const long long off = (long long)u * ldp + lc.jl;
        unsigned pu[IdWords<CPT>::N];
        long long lu[CPT];
        load_ids_masked<CPT>(a.part + off, lc, pu);
        load_levels<CPT>(a.lev + off, lu);
        build_edge_table<FWD>(tc, X, Xr, lane);
#pragma unroll
        for (int c = 0; c < CPT; ++c) {
            const unsigned idx = id_at<CPT>(pu, c) * k + id_at<CPT>(pv, c);
            const long long val = lu[c] + tc.T[idx];
            best[c] = val > best[c] ? val : best[c];
        }
    }

    if (!FWD && vm.e0 == vm.e1) {  // sink: blevel = own runtime
#pragma unroll
        for (int c = 0; c < CPT; ++c)
            if (Xv != NUM_ZERO) best[c] = ceil_quot(Xv, tc.s_rt[id_at<CPT>(pv, c)]);
    }
    store_levels<CPT>(a.lev + (long long)v * ldp + lc.jl, best, lc.nvalid);
    if (cp_vertex) {
#pragma unroll
        for (int c = 0; c < CPT; ++c) {
            long long fin = best[c];
            if (FWD && Xv != NUM_ZERO) fin += ceil_quot(Xv, tc.s_rt[id_at<CPT>(pv, c)]);
            cpmax[c] = fin > cpmax[c] ? fin : cpmax[c];
        }
    }
}

__device__ __forceinline__ VertexMeta global_meta(const LevelAdj& adj, int pos)
{
    VertexMeta vm;
    vm.v = adj.vert[pos];
    vm.e0 = adj.eptr[pos];
    vm.e1 = adj.eptr[pos + 1];
    vm.nbr = adj.nbr;
    vm.xw = adj.xw;
    vm.xnbr = adj.xnbr;
    vm.xvert = adj.xvert[pos];
    return vm;
}

// ---- level-synchronous variant: one launch per level ----------------------------
template <int CPT, bool FWD>
__global__ void __launch_bounds__(128)
pass_level_kernel(PassArgs a, int pos0, int count)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    DivConst* s_w = reinterpret_cast<DivConst*>(smem_raw);
    DivConst* s_rt = s_w + a.tab.k * a.tab.k;
    if (*a.status != 0) return;
    stage_tables(a.tab, s_w, s_rt);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, wpb = blockDim.x >> 5;
    const long long slice0 = (long long)blockIdx.x * 32 * CPT;
    const LaneCtx<CPT> lc = lane_setup<CPT>(slice0, a.P, lane);
    long long unused[CPT];
#pragma unroll
    for (int c = 0; c < CPT; ++c) unused[c] = 0;
    for (int i = blockIdx.y * wpb + warp; i < count; i += gridDim.y * wpb)
        relax_vertex<CPT, FWD>(a, s_w, s_rt, global_meta(a.adj, pos0 + i), lc, false, unused);
}

// ---- candidate-sliced persistent variant ---------------------------------------------
// One block owns 32*CPT candidates and walks the whole graph chunk by chunk; a
// chunk is a run of at most CHUNK_V positions / CHUNK_E edges inside one level
// (table built on the host).  Candidates are independent, so no block ever
// waits for another one; the block's warps share the vertices of a chunk and
// meet at one block barrier per chunk.  The adjacency of the NEXT chunk is
// copied into shared memory with cp.async while the current one is processed,
// so a warp's dependent global-memory chain per vertex is a single hop
// (neighbour ids and levels).
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
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

struct ChunkBuf {
    unsigned long long xvert[CHUNK_V];
    unsigned long long xw[CHUNK_E];
    unsigned long long xnbr[CHUNK_E];
    int vertf[CHUNK_V];
    int eoff[CHUNK_V + 4];
    int nbr[CHUNK_E];
};

template <bool FWD>
__device__ __forceinline__ void stage_chunk(const PassArgs& a, const int* __restrict__ vertf, int4 ent, ChunkBuf& b)
{
    const int p0 = ent.x, cnt = ent.y, e0 = ent.z, ecnt = ent.w;
    for (int i = threadIdx.x; i < cnt; i += blockDim.x) {
        cp_async4(&b.vertf[i], vertf + p0 + i);
        cp_async8(&b.xvert[i], a.adj.xvert + p0 + i);
    }
    for (int i = threadIdx.x; i <= cnt; i += blockDim.x) cp_async4(&b.eoff[i], a.adj.eptr + p0 + i);
    if (ecnt <= CHUNK_E) {
        for (int i = threadIdx.x; i < ecnt; i += blockDim.x) {
            cp_async4(&b.nbr[i], a.adj.nbr + e0 + i);
            cp_async8(&b.xw[i], a.adj.xw + e0 + i);
            if (FWD) cp_async8(&b.xnbr[i], a.adj.xnbr + e0 + i);
        }
    }
}

// shared-memory bytes of the sliced kernel besides the two chunk buffers
__host__ __device__ inline size_t sliced_tail_smem(int k, int npass, int warps, int cpt, bool table)
{
    size_t b = sizeof(DivConst) * (size_t)k;                       // s_rt
    b += sizeof(long long) * (size_t)warps * 32 * cpt;             // s_cp
    if (table) {
        b += sizeof(DivConst) * (size_t)npass * 32;                // s_pair
        b += sizeof(long long) * (size_t)warps * npass * 32;       // per-warp tables
        b += sizeof(unsigned short) * (size_t)npass * 32;          // s_sel
    } else {
        b += sizeof(DivConst) * (size_t)k * k;                     // s_w
    }
    return b;
}

// largest block the sliced kernel may be launched with (bounds its registers per thread)
template <int CPT, bool TABLE> struct SlicedBounds { static constexpr int THREADS = (TABLE && CPT <= 4) ? 1024 : 256; };

template <int CPT, bool FWD, bool TABLE>
__global__ void __launch_bounds__(SlicedBounds<CPT, TABLE>::THREADS)
pass_sliced_kernel(PassArgs a, const int* __restrict__ vertf, const int4* __restrict__ chunks, int num_chunks, int src_end)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, wpb = blockDim.x >> 5;
    const int k = a.tab.k;
    const int npass = a.tab.npass;
    ChunkBuf* bufs = reinterpret_cast<ChunkBuf*>(smem_raw);
    DivConst* s_rt = reinterpret_cast<DivConst*>(bufs + 2);
    long long* s_cp = reinterpret_cast<long long*>(s_rt + k);  // [warps][32*CPT]
    unsigned char* tail = reinterpret_cast<unsigned char*>(s_cp + (size_t)wpb * 32 * CPT);
    DivConst* s_w = reinterpret_cast<DivConst*>(tail);      // direct: [k*k]; table: pair table [npass*32]
    if (*a.status != 0) return;

    TableCtx tc;
    if (TABLE) {
        long long* s_T = reinterpret_cast<long long*>(s_w + npass * 32);
        unsigned short* s_sel = reinterpret_cast<unsigned short*>(s_T + (size_t)wpb * npass * 32);
        const DivConst* pair = FWD ? a.tab.pair_f : a.tab.pair_b;
        const unsigned short* sel = FWD ? a.tab.sel_f : a.tab.sel_b;
        for (int i = threadIdx.x; i < npass * 32; i += blockDim.x) { s_w[i] = pair[i]; s_sel[i] = sel[i]; }
        tc.s_pair = s_w;
        tc.s_rt = s_rt;
        tc.s_sel = s_sel;
        tc.T = s_T + (size_t)warp * npass * 32;
        tc.my_cls = a.tab.cls_div[lane];
        tc.npass = npass;
        tc.use_cls = a.tab.use_cls;
        tc.ncls_w = a.tab.ncls_w;
    } else {
        for (int i = threadIdx.x; i < k * k; i += blockDim.x) s_w[i] = a.tab.w_div[i];
    }
    for (int i = threadIdx.x; i < k; i += blockDim.x) s_rt[i] = a.tab.rt_div[i];

    const long long slice0 = (long long)blockIdx.x * 32 * CPT;
    const LaneCtx<CPT> lc = lane_setup<CPT>(slice0, a.P, lane);
    const bool want_cp = a.cp != nullptr;
    long long* cpmax = s_cp + ((size_t)warp * 32 + lane) * CPT;   // this lane's running maxima
#pragma unroll
    for (int c = 0; c < CPT; ++c) cpmax[c] = 0;

    // chunk ci of this pass is table entry ci (forward) or num_chunks-1-ci (backward)
    auto entry = [&](int ci) { return chunks[FWD ? ci : num_chunks - 1 - ci]; };
    int4 cur = entry(0);
    int4 nxt = num_chunks > 1 ? entry(1) : cur;
    stage_chunk<FWD>(a, vertf, cur, bufs[0]);
    cp_async_commit();
    cp_async_wait_all();
    __syncthreads();
    for (int ci = 0; ci < num_chunks; ++ci) {
        ChunkBuf& b = bufs[ci & 1];
        int4 nxt2 = nxt;
        if (ci + 1 < num_chunks) {
            stage_chunk<FWD>(a, vertf, nxt, bufs[(ci + 1) & 1]);
            cp_async_commit();
            if (ci + 2 < num_chunks) nxt2 = entry(ci + 2);
        }
        const int p0 = cur.x, cnt = cur.y, e0 = cur.z;
        const bool staged = cur.w <= CHUNK_E;
        for (int i = warp; i < cnt; i += wpb) {
            VertexMeta vm;
            const int vf = b.vertf[i];
            vm.v = vf & 0x7fffffff;
            vm.xvert = b.xvert[i];
            // a vertex whose adjacency did not fit the chunk buffer is read from global memory
            const int ebase = staged ? e0 : 0;
            vm.e0 = b.eoff[i] - ebase;
            vm.e1 = b.eoff[i + 1] - ebase;
            vm.nbr = staged ? b.nbr : a.adj.nbr;
            vm.xw = staged ? b.xw : a.adj.xw;
            vm.xnbr = staged ? b.xnbr : a.adj.xnbr;
            bool cpv = false;
            if (want_cp) cpv = FWD ? (vf < 0) : (p0 + i < src_end);
            if (TABLE) relax_vertex_table<CPT, FWD>(a, tc, vm, lc, lane, cpv, cpmax);
            else relax_vertex<CPT, FWD>(a, s_w, s_rt, vm, lc, cpv, cpmax);
        }
        cp_async_wait_all();
        __syncthreads();
        cur = nxt;
        nxt = nxt2;
    }

    if (want_cp && warp == 0) {
#pragma unroll
        for (int c = 0; c < CPT; ++c) {
            long long m = cpmax[c];
            for (int w = 1; w < wpb; ++w) {
                long long o = s_cp[((size_t)w * 32 + lane) * CPT + c];
                m = o > m ? o : m;
            }
            if (c < lc.nvalid) a.cp[slice0 + (long long)lane * CPT + c] = m;
        }
    }
}

// ---- critical-path length for the level-synchronous variant -----------------------
// cp[j] = max over the listed positions of lev (+ rt when reducing tlevel).  cp is
// zeroed by the host; partial maxima are merged with atomicMax (order independent).
template <bool FROM_TLEVEL>
__global__ void __launch_bounds__(128)
cp_reduce_kernel(PassArgs a, const int* __restrict__ list, int list_len, int per_block)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    DivConst* s_rt = reinterpret_cast<DivConst*>(smem_raw);
    if (*a.status != 0) return;
    for (int i = threadIdx.x; i < a.tab.k; i += blockDim.x) s_rt[i] = a.tab.rt_div[i];
    __syncthreads();
    const long long j = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= a.P) return;
    int i0 = blockIdx.y * per_block;
    int i1 = i0 + per_block < list_len ? i0 + per_block : list_len;
    long long m = 0;
    for (int i = i0; i < i1; ++i) {
        const int pos = list ? list[i] : i;
        const int v = a.adj.vert[pos];
        long long val = a.lev[(long long)v * a.ldp + j];
        if (FROM_TLEVEL) {
            const unsigned long long Xv = a.adj.xvert[pos];
            const unsigned id = a.part[(long long)v * a.ldp + j];
            if (Xv != NUM_ZERO) val += ceil_quot(Xv, s_rt[id]);
        }
        m = val > m ? val : m;
    }
    atomicMax(&a.cp[j], m);
}

// ---- per-device load and memory ----------------------------------------------------------
// Thread = 4 candidates; a block keeps [k][candidates] accumulators for load
// and memory in shared memory (each thread touches only its own columns, so no
// shared-memory atomics), walks a chunk of vertices and merges into global
// memory with 64-bit atomic adds (integer, order independent).  Doubles as the
// id validator: an id >= k raises BAD_PARTITION and is counted on device 0.
template <int C>   // candidates per thread: 1, 2 or 4
__global__ void loads_kernel(int n, long long P, long long ldp, const uint8_t* __restrict__ part,
                             const int* __restrict__ vert, const unsigned long long* __restrict__ xvert,
                             const long long* __restrict__ mem, DevTables tab, long long* load,
                             long long* memload, int* status, int validate, int rows_per_block)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int k = tab.k;
    const int nthr = blockDim.x;  // accumulators are laid out [device][c][thread]: conflict-free columns
    DivConst* s_rt = reinterpret_cast<DivConst*>(smem_raw);
    long long* acc_l = reinterpret_cast<long long*>(s_rt + k);
    long long* acc_m = acc_l + (size_t)k * nthr * C;
    for (int i = threadIdx.x; i < k; i += blockDim.x) s_rt[i] = tab.rt_div[i];
    for (int i = threadIdx.x; i < k * nthr * C; i += blockDim.x) { acc_l[i] = 0; acc_m[i] = 0; }
    __syncthreads();

    const long long slice0 = (long long)blockIdx.x * nthr * C;
    const long long j0 = slice0 + (long long)threadIdx.x * C;
    const long long rem = P - j0;
    const int nvalid = rem >= C ? C : (rem > 0 ? (int)rem : 0);
    const long long jl = nvalid > 0 ? j0 : slice0;  // idle lanes keep the warp's shuffles company
    const int lane = threadIdx.x & 31;
    const int r0 = blockIdx.y * rows_per_block;
    const int r1 = r0 + rows_per_block < n ? r0 + rows_per_block : n;
    bool bad = false;
    constexpr int RB = 4;  // rows in flight
    for (int pos = r0; pos < r1; pos += RB) {
        unsigned long long Xv[RB];
        long long mv[RB];
        unsigned packed[RB];
#pragma unroll
        for (int q = 0; q < RB; ++q) {
            if (pos + q < r1) {
                const int v = vert[pos + q];
                Xv[q] = xvert[pos + q];
                mv[q] = mem[v];
                const uint8_t* p = part + (long long)v * ldp + jl;
                if constexpr (C == 1) packed[q] = *p;
                else if constexpr (C == 2) packed[q] = *reinterpret_cast<const unsigned short*>(p);
                else packed[q] = *reinterpret_cast<const unsigned*>(p);
            }
        }
#pragma unroll
        for (int q = 0; q < RB; ++q) {
            if (pos + q < r1) {
                // runtime of this vertex on device `lane` (and lane+32): one division per device, not per candidate
                long long row_lo = 0, row_hi = 0;
                if (Xv[q] != NUM_ZERO) {
                    if (lane < k) row_lo = ceil_quot(Xv[q], s_rt[lane]);
                    if (k > 32 && lane + 32 < k) row_hi = ceil_quot(Xv[q], s_rt[lane + 32]);
                }
#pragma unroll
                for (int c = 0; c < C; ++c) {
                    unsigned id = (packed[q] >> (8 * c)) & 0xffu;
                    if (c >= nvalid) id = 0;
                    if (id >= (unsigned)k) { bad = true; id = 0; }
                    long long rt = shfl64(row_lo, (int)(id & 31u));
                    if (k > 32) {
                        const long long hi = shfl64(row_hi, (int)(id & 31u));
                        rt = id >= 32u ? hi : rt;
                    }
                    if (c < nvalid) {
                        acc_l[(id * C + c) * nthr + threadIdx.x] += rt;
                        acc_m[(id * C + c) * nthr + threadIdx.x] += mv[q];
                    }
                }
            }
        }
    }
    if (bad && validate) atomicCAS(status, 0, (int)TFPS_ERR_BAD_PARTITION);
    for (int d = 0; d < k; ++d) {
#pragma unroll
        for (int c = 0; c < C; ++c) {
            if (c < nvalid) {
                if (load) atomicAdd(reinterpret_cast<unsigned long long*>(load + d * ldp + j0 + c),
                                    (unsigned long long)acc_l[(d * C + c) * nthr + threadIdx.x]);
                if (memload) atomicAdd(reinterpret_cast<unsigned long long*>(memload + d * ldp + j0 + c),
                                       (unsigned long long)acc_m[(d * C + c) * nthr + threadIdx.x]);
            }
        }
    }
}

// id check alone (no load outputs wanted): 16 ids per thread
__global__ void validate_kernel(long long n, long long P, long long ldp, const uint8_t* __restrict__ part, int k,
                                int* status)
{
    const long long vecs_per_row = (P + 15) / 16;
    const long long total = n * vecs_per_row;
    bool bad = false;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const long long v = i / vecs_per_row;
        const long long j = (i - v * vecs_per_row) * 16;
        const uint4 q = *reinterpret_cast<const uint4*>(part + v * ldp + j);
        const unsigned w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int b = 0; b < 16; ++b) {
            const unsigned id = (w[b >> 2] >> (8 * (b & 3))) & 0xffu;
            if (j + b < P && id >= (unsigned)k) bad = true;
        }
    }
    if (bad) atomicCAS(status, 0, (int)TFPS_ERR_BAD_PARTITION);
}

__global__ void viol_kernel(long long P, long long ldp, int k, const long long* __restrict__ memload,
                            const long long* __restrict__ cap, unsigned long long* viol, const int* status)
{
    if (*status != 0) return;
    const long long j = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= P) return;
    unsigned long long bits = 0;
    for (int d = 0; d < k; ++d)
        if (memload[d * ldp + j] >= cap[d]) bits |= 1ull << d;
    viol[j] = bits;
}

// ---- [P][n] -> [n][ldp] byte transpose ------------------------------------------------------
__global__ void __launch_bounds__(256)
transpose_u8_kernel(const uint8_t* __restrict__ src, uint8_t* __restrict__ dst, long long P, long long n, long long ldp)
{
    __shared__ uint8_t tile[64][65];
    const long long v0 = (long long)blockIdx.x * 64;  // along n (contiguous in src)
    const long long j0 = (long long)blockIdx.y * 64;  // along P (contiguous in dst)
    const int tx = threadIdx.x & 63, ty = threadIdx.x >> 6;
    for (int r = ty; r < 64; r += 4) {
        const long long j = j0 + r, v = v0 + tx;
        if (j < P && v < n) tile[r][tx] = src[j * n + v];
    }
    __syncthreads();
    for (int r = ty; r < 64; r += 4) {
        const long long v = v0 + r, j = j0 + tx;
        if (v < n && j < P) dst[v * ldp + j] = tile[tx][r];
    }
}

inline unsigned cdivu(long long a, long long b) { return (unsigned)((a + b - 1) / b); }

size_t table_smem(int k) { return sizeof(DivConst) * (size_t)(k * k + k); }

template <typename K>
cudaError_t allow_smem(K kernel, size_t bytes)
{
    if (bytes <= 48 * 1024) return cudaSuccess;
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

}  // namespace

int pick_cpt(long long P)
{
    return P >= 64 * 148 ? 2 : 1;
}

template <int CPT, bool FWD>
static cudaError_t level_sync_impl(const PassArgs& a, const std::vector<long long>& lp, cudaStream_t st)
{
    const size_t smem = table_smem(a.tab.k);
    cudaError_t e = allow_smem(pass_level_kernel<CPT, FWD>, smem);
    if (e != cudaSuccess) return e;
    const unsigned gx = cdivu(a.P, 32 * CPT);
    const int L = a.num_levels;
    for (int step = 0; step < L; ++step) {
        const int l = FWD ? step : L - 1 - step;
        const int pos0 = (int)lp[l];
        const int count = (int)(lp[l + 1] - lp[l]);
        unsigned gy = cdivu(count, 4);
        if (gy > 65535u) gy = 65535u;
        pass_level_kernel<CPT, FWD><<<dim3(gx, gy), 128, smem, st>>>(a, pos0, count);
    }
    count_launches(L);
    return cudaGetLastError();
}

__global__ void zero_rows_kernel(const int* __restrict__ rows, long long P, long long ldp, long long* lev)
{
    const long long j = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (j < P) lev[(long long)rows[blockIdx.y] * ldp + j] = 0;
}

// lp: level pointers over positions, or over work items when the pass has them
cudaError_t launch_zero_rows(const int* rows, int count, long long P, long long ldp, long long* lev, cudaStream_t st)
{
    if (count <= 0 || P <= 0) return cudaSuccess;
    for (int r0 = 0; r0 < count; r0 += 65535) {
        const int c = count - r0 < 65535 ? count - r0 : 65535;
        zero_rows_kernel<<<dim3(cdivu(P, 256), (unsigned)c), 256, 0, st>>>(rows + r0, P, ldp, lev);
    }
    count_launches((count + 65534) / 65535);
    return cudaGetLastError();
}

cudaError_t launch_pass_level_sync(const PassArgs& a, bool fwd, const std::vector<long long>& lp, cudaStream_t st)
{
    const int cpt = pick_cpt(a.P);
    if (cpt == 2) return fwd ? level_sync_impl<2, true>(a, lp, st) : level_sync_impl<2, false>(a, lp, st);
    return fwd ? level_sync_impl<1, true>(a, lp, st) : level_sync_impl<1, false>(a, lp, st);
}

template <int CPT, bool FWD, bool TABLE>
static cudaError_t sliced_impl(const PassArgs& a, const SlicedPlan& plan, int warps, cudaStream_t st)
{
    if (warps * 32 > SlicedBounds<CPT, TABLE>::THREADS) warps = SlicedBounds<CPT, TABLE>::THREADS / 32;
    const size_t smem = 2 * sizeof(ChunkBuf) + sliced_tail_smem(a.tab.k, a.tab.npass, warps, CPT, TABLE);
    cudaError_t e = allow_smem(pass_sliced_kernel<CPT, FWD, TABLE>, smem);
    if (e != cudaSuccess) return e;
    const unsigned gx = cdivu(a.P, 32 * CPT);
    pass_sliced_kernel<CPT, FWD, TABLE><<<gx, warps * 32, smem, st>>>(
        a, plan.vertf, reinterpret_cast<const int4*>(plan.chunks), plan.num_chunks, plan.src_end);
    count_launches(1);
    return cudaGetLastError();
}

template <int CPT>
static cudaError_t sliced_dispatch(const PassArgs& a, bool fwd, bool table, const SlicedPlan& plan, int warps, cudaStream_t st)
{
    if (table) return fwd ? sliced_impl<CPT, true, true>(a, plan, warps, st) : sliced_impl<CPT, false, true>(a, plan, warps, st);
    return fwd ? sliced_impl<CPT, true, false>(a, plan, warps, st) : sliced_impl<CPT, false, false>(a, plan, warps, st);
}

cudaError_t launch_pass_sliced(const PassArgs& a, bool fwd, const SlicedPlan& plan, int cpt, int warps, bool table,
                               cudaStream_t st)
{
    if (plan.num_chunks <= 0) return cudaSuccess;
    if (a.tab.npass <= 0) table = false;
    if (cpt == 8) return sliced_dispatch<8>(a, fwd, table, plan, warps, st);
    if (cpt == 4) return sliced_dispatch<4>(a, fwd, table, plan, warps, st);
    if (cpt == 2) return sliced_dispatch<2>(a, fwd, table, plan, warps, st);
    return sliced_dispatch<1>(a, fwd, table, plan, warps, st);
}

cudaError_t launch_cp_reduce(const PassArgs& a, bool from_tlevel, const int* list, int list_len, cudaStream_t st)
{
    if (list_len <= 0) return cudaSuccess;
    const size_t smem = sizeof(DivConst) * (size_t)a.tab.k;
    const unsigned gx = cdivu(a.P, 128);
    int per_block = 256;
    unsigned gy = cdivu(list_len, per_block);
    if (gy > 65535u) { per_block = (int)cdivu(list_len, 65535); gy = cdivu(list_len, per_block); }
    count_launches(1);
    if (from_tlevel)
        cp_reduce_kernel<true><<<dim3(gx, gy), 128, smem, st>>>(a, list, list_len, per_block);
    else
        cp_reduce_kernel<false><<<dim3(gx, gy), 128, smem, st>>>(a, list, list_len, per_block);
    return cudaGetLastError();
}

template <int C>
static cudaError_t loads_impl(int n, long long P, long long ldp, const uint8_t* part, const int* vert,
                              const unsigned long long* xvert, const long long* mem, DevTables tab, long long* load,
                              long long* memload, int* status, bool validate, int sm_count, cudaStream_t st)
{
    const int k = tab.k;
    // threads per block sized so that 2*k*(C*threads) int64 accumulators fit in shared memory
    int threads = 64;
    while (threads > 32 && sizeof(DivConst) * k + (size_t)2 * k * threads * C * 8 > 96 * 1024) threads >>= 1;
    const size_t smem = sizeof(DivConst) * k + (size_t)2 * k * threads * C * 8;
    cudaError_t e = allow_smem(loads_kernel<C>, smem);
    if (e != cudaSuccess) return e;
    const unsigned gx = cdivu(P, threads * C);
    int per_sm = 64;
    if (const char* ov = getenv("TFPS_LOADS_BLOCKS_PER_SM")) { const int q = atoi(ov); if (q >= 1 && q <= 64) per_sm = q; }
    long long want_blocks = (long long)sm_count * per_sm;
    long long gy = (want_blocks + gx - 1) / gx;
    if (gy < 1) gy = 1;
    if (gy > n) gy = n;
    if (gy > 65535) gy = 65535;
    int rows = (int)((n + gy - 1) / gy);
    gy = (n + rows - 1) / rows;
    count_launches(1);
    loads_kernel<C><<<dim3(gx, (unsigned)gy), threads, smem, st>>>(n, P, ldp, part, vert, xvert, mem, tab, load, memload,
                                                                   status, validate ? 1 : 0, rows);
    return cudaGetLastError();
}

cudaError_t launch_loads(int n, long long P, long long ldp, const uint8_t* part, const int* vert,
                         const unsigned long long* xvert, const long long* mem, DevTables tab, long long* load,
                         long long* memload, int* status, bool validate, int sm_count, cudaStream_t st)
{
    int c = 2;  // two candidates per thread: best balance of shared-memory footprint (occupancy) and per-row work
    if (const char* ov = getenv("TFPS_LOADS_CPT")) c = atoi(ov);   // tuning override
    if (c == 1) return loads_impl<1>(n, P, ldp, part, vert, xvert, mem, tab, load, memload, status, validate, sm_count, st);
    if (c == 2) return loads_impl<2>(n, P, ldp, part, vert, xvert, mem, tab, load, memload, status, validate, sm_count, st);
    return loads_impl<4>(n, P, ldp, part, vert, xvert, mem, tab, load, memload, status, validate, sm_count, st);
}

cudaError_t launch_validate(long long n, long long P, long long ldp, const uint8_t* part, int k, int* status,
                            int sm_count, cudaStream_t st)
{
    validate_kernel<<<sm_count * 8, 256, 0, st>>>(n, P, ldp, part, k, status);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_viol(long long P, long long ldp, int k, const long long* memload, const long long* cap,
                        unsigned long long* viol, const int* status, cudaStream_t st)
{
    viol_kernel<<<cdivu(P, 256), 256, 0, st>>>(P, ldp, k, memload, cap, viol, status);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_transpose_u8(const uint8_t* src, uint8_t* dst, long long P, long long n, long long ldp, cudaStream_t st)
{
    dim3 grid(cdivu(n, 64), cdivu(P, 64));
    transpose_u8_kernel<<<grid, 256, 0, st>>>(src, dst, P, n, ldp);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace tfps
