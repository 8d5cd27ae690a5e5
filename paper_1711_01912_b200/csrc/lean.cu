// Lean windowed candidate-sliced pass.
//
// Same idea as the windowed pass (one block owns 32*CPT candidates, walks the whole graph chunk by chunk and
// keeps the levels of the last R positions of its own candidates in a shared-memory ring, so only the
// compulsory traffic -- one id read and one level write per vertex-candidate -- reaches global memory), cut
// down to the instructions the recurrences need:
//   * the host packs one record per chunk (LeanPlan): vertices in processing order (highest degree first, dealt
//     round-robin to the warps, so a fixed assignment is balanced), per-vertex runtimes for every device, and
//     per-edge transfer times for every distinct bandwidth;
//   * the window keeps finish times tlevel+rt (forward) or bottom levels (backward, Eq. 12), so a relaxation
//     only adds the transfer term: one byte permute maps the neighbour's device id to the offset of the right
//     transfer time inside the edge record, one shared-memory load fetches it, one add-max folds it in;
//   * all shared-memory traffic uses 32-bit shared-window addresses;
//   * every warp consumes; the copies of the chunk `depth` ahead (one bulk copy for the record, 16-byte
//     cp.async pieces for the id rows) are issued by all threads right after the chunk barrier, from chunk
//     descriptors and vertex ids prefetched into registers one chunk earlier.
// Requirements (checked by the host): every path length fits int32, k <= 8, at most 30 distinct off-diagonal
// bandwidths, the whole window fits in shared memory beside the stage slots.
#include "common.cuh"

namespace tfps {

namespace {

__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned lds32(unsigned a)
{
    unsigned v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ unsigned lds32_off4(unsigned a)   // word at a + 4
{
    unsigned v;
    asm volatile("ld.shared.u32 %0, [%1+4];" : "=r"(v) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ unsigned lds32_off16(unsigned a)   // word at a + 16
{
    unsigned v;
    asm volatile("ld.shared.u32 %0, [%1+16];" : "=r"(v) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ uint2 lds64(unsigned a)
{
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ uint4 lds128(unsigned a)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ unsigned lds_u16(unsigned a)
{
    unsigned short v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ unsigned lds_u8(unsigned a)
{
    unsigned v;
    asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ void sts32(unsigned a, unsigned v) { asm volatile("st.shared.u32 [%0], %1;" ::"r"(a), "r"(v) : "memory"); }
__device__ __forceinline__ void sts64(unsigned a, unsigned x, unsigned y)
{
    asm volatile("st.shared.v2.u32 [%0], {%1, %2};" ::"r"(a), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void sts128(unsigned a, unsigned x, unsigned y, unsigned z, unsigned w)
{
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ void sts_u16(unsigned a, unsigned v) { asm volatile("st.shared.u16 [%0], %1;" ::"r"(a), "h"((unsigned short)v) : "memory"); }
__device__ __forceinline__ void sts_u8(unsigned a, unsigned v) { asm volatile("st.shared.u8 [%0], %1;" ::"r"(a), "r"(v) : "memory"); }

// byte permute: result byte i = byte (sel nibble i & 7) of {b, a}; nibble bit 3 replicates that byte's sign bit instead
__device__ __forceinline__ unsigned prmt(unsigned a, unsigned b, unsigned sel)
{
    unsigned d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

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
__device__ __forceinline__ void cp_async16(unsigned dst, const void* g)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(g) : "memory");
}
// one (pre-counted) arrival on the mbarrier once every cp.async this thread has issued so far has landed
__device__ __forceinline__ void cp_async_arrive_on(unsigned bar)
{
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
// Bounded wait: gives up after WAIT_LIMIT polls (each poll blocks for a hardware-defined time slice at most).
constexpr int WAIT_LIMIT = 1 << 20;
__device__ __forceinline__ bool mbar_wait(unsigned bar, unsigned parity)
{
    for (int i = 0; i < WAIT_LIMIT; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

__device__ __forceinline__ void stg_cs_v2(long long* p, long long x, long long y)
{
    asm volatile("st.global.cs.v2.u64 [%0], {%1, %2};" ::"l"(p), "l"(x), "l"(y) : "memory");
}
__device__ __forceinline__ void stg_cs(long long* p, long long x) { asm volatile("st.global.cs.u64 [%0], %1;" ::"l"(p), "l"(x) : "memory"); }

template <int CPT> __device__ __forceinline__ unsigned ld_ids(unsigned a)
{
    if constexpr (CPT == 1) return lds_u8(a);
    else if constexpr (CPT == 2) return lds_u16(a);
    else return lds32(a);
}
template <int CPT> __device__ __forceinline__ void st_ids(unsigned a, unsigned v)
{
    if constexpr (CPT == 1) sts_u8(a, v);
    else if constexpr (CPT == 2) sts_u16(a, v);
    else sts32(a, v);
}
template <int CPT> __device__ __forceinline__ void ld_lev(unsigned a, int (&l)[CPT])
{
    if constexpr (CPT == 1) l[0] = (int)lds32(a);
    else if constexpr (CPT == 2) { const uint2 v = lds64(a); l[0] = (int)v.x; l[1] = (int)v.y; }
    else { const uint4 v = lds128(a); l[0] = (int)v.x; l[1] = (int)v.y; l[2] = (int)v.z; l[3] = (int)v.w; }
}
template <int CPT> __device__ __forceinline__ void st_lev(unsigned a, const int (&l)[CPT])
{
    if constexpr (CPT == 1) sts32(a, (unsigned)l[0]);
    else if constexpr (CPT == 2) sts64(a, (unsigned)l[0], (unsigned)l[1]);
    else sts128(a, (unsigned)l[0], (unsigned)l[1], (unsigned)l[2], (unsigned)l[3]);
}

template <int CPT, bool FWD>
__global__ void __launch_bounds__(1024, 1) pass_lean_kernel(const LeanArgs a)
{
    extern __shared__ __align__(16) unsigned char dsm[];   // [stage slots][window]
    __shared__ __align__(16) unsigned long long s_rows[LEAN_K_MAX];
    __shared__ __align__(8) unsigned long long s_bar[LEAN_DEPTH_MAX];
    __shared__ int s_abort;
    constexpr int SLICE = 32 * CPT;        // candidates of the block = bytes of an id row
    constexpr unsigned LEVB = SLICE * 4;   // a window row: SLICE levels, then SLICE id bytes
    constexpr unsigned ROWB = SLICE * 5;
    constexpr int PR = 2 * CPT;            // 16-byte pieces of an id row
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nthreads = blockDim.x, nwarps = nthreads >> 5;
    if (*a.status != 0) return;
    const int D = a.depth;
    const int nc = a.plan.num_chunks;
    const unsigned stage0 = smem_u32(dsm), win0 = stage0 + a.stage_bytes;
    const unsigned rows_s = smem_u32(s_rows), bar0 = smem_u32(s_bar);
    volatile int* abort_p = &s_abort;
    if (tid < LEAN_K_MAX) s_rows[tid] = a.plan.rows[tid];
    if (tid == 0) {
        // a stage completes on the record's bulk copy (one arrival carrying the byte count) plus one arrival
        // per thread once that thread's id-row pieces have landed
        for (int j = 0; j < D; ++j) mbar_init(bar0 + 8u * j, (unsigned)nthreads + 1u);
        s_abort = 0;
        mbar_init_fence();
    }
    __syncthreads();

    const long long slice0 = (long long)blockIdx.x * SLICE;
    const long long j0 = slice0 + (long long)lane * CPT;
    const long long rem = a.P - j0;
    const int nvalid = rem >= CPT ? CPT : (rem > 0 ? (int)rem : 0);
    const long long ldp = a.ldp;
    const unsigned slice_bytes = (unsigned)((ldp - slice0) < SLICE ? (ldp - slice0) : SLICE);   // multiple of 16
    const unsigned win_lev_lane = win0 + (unsigned)(lane * CPT * 4);
    const unsigned id_delta = LEVB - (unsigned)(3 * lane * CPT);   // id bytes of a lane relative to its levels
    const int vstride = a.plan.vstride, estride = a.plan.estride;
    const unsigned rec_max = (unsigned)a.plan.rec_max;
    const int4* __restrict__ desc = a.plan.desc;
    const int* __restrict__ vlist = a.plan.vlist;
    const unsigned char* __restrict__ blob = a.plan.blob;
    const uint8_t* __restrict__ part0 = a.part + slice0;
    long long* __restrict__ out_lane = a.lev + j0;
    const unsigned ldp8 = (unsigned)(ldp * 8);
    int cpmax[CPT];
#pragma unroll
    for (int c = 0; c < CPT; ++c) cpmax[c] = 0;

    // copies of one chunk into a stage slot: d = its descriptor, v[s] = vertex of the id row this thread fetches
    auto issue = [&](const int4& d, const int (&v)[2], unsigned slotb, unsigned bar) {
        if (d.y == 0) return;   // past the last chunk
        if (tid == 0) {
            mbar_expect_tx(bar, (unsigned)d.y);
            bulk_g2s(slotb, blob + 16ll * (unsigned)d.x, (unsigned)d.y, bar);
        }
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            const int p = tid + s * nthreads;
            const int r = p / PR, q = p % PR;
            if (r < d.z && (unsigned)(16 * q) < slice_bytes)
                cp_async16(slotb + rec_max + (unsigned)(r * SLICE + 16 * q), part0 + (long long)v[s] * ldp + 16 * q);
        }
        cp_async_arrive_on(bar);
    };
    auto fetch_v = [&](const int4& d, int (&v)[2]) {
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            const int r = (tid + s * nthreads) / PR;
            v[s] = r < d.z ? __ldg(vlist + d.w + r) : 0;
        }
    };

    for (int j = 0; j < D; ++j) {   // chunks 0..D-1 (descriptors past the end are zero)
        const int4 d = __ldg(desc + j);
        int v[2];
        fetch_v(d, v);
        issue(d, v, stage0 + (unsigned)j * a.slot_stride, bar0 + 8u * j);
    }
    int4 dC = __ldg(desc + D);   // the chunk issued after chunk 0 is done
    int slot = 0;
    unsigned par = 0;
    for (int ci = 0; ci < nc; ++ci) {
        // prefetch for the issue at the end of this iteration (chunk ci+D) and of the next one
        const int4 dN = __ldg(desc + ci + D + 1);
        int vA[2];
        fetch_v(dC, vA);
        const unsigned slotb = stage0 + (unsigned)slot * a.slot_stride;
        const unsigned bar = bar0 + 8u * slot;
        if (!mbar_wait(bar, par)) {
            atomicCAS(a.status, 0, (int)TFPS_ERR_TIMEOUT);
            *abort_p = 1;
        } else {
            const uint4 hdr = lds128(slotb);
            const int cnt = (int)hdr.x;
            const unsigned vbase = slotb + 16u, ebase = slotb + hdr.y;
            const unsigned idrow = slotb + rec_max + (unsigned)(lane * CPT);
            for (int i = warp; i < cnt; i += nwarps) {
                const unsigned vr = vbase + (unsigned)(i * vstride);
                const uint4 rec = lds128(vr);   // {v | flag, window slot, first edge byte, end edge byte}
                const unsigned ids = ld_ids<CPT>(idrow + (unsigned)(i * SLICE));
                unsigned rlo[CPT], rhi[CPT];
                int rt[CPT], best[CPT];
#pragma unroll
                for (int c = 0; c < CPT; ++c) {
                    // 8 * own device id (masked to the table size, so a bad id cannot leave the tables)
                    const unsigned pv8 = (c == 0 ? (ids << 3) : (ids >> (8 * c - 3))) & 0x38u;
                    const uint2 row = lds64(rows_s + pv8);
                    rlo[c] = row.x;
                    rhi[c] = row.y;
                    rt[c] = (int)lds32_off16(vr + (pv8 >> 1));
                    best[c] = 0;
                }
                for (unsigned ea = ebase + rec.z, ee = ebase + rec.w; ea < ee; ea += (unsigned)estride) {
                    const unsigned ns = lds32(ea);
                    const unsigned la = win_lev_lane + ns * ROWB;
                    int lu[CPT];
                    ld_lev<CPT>(la, lu);
                    const unsigned pu = ld_ids<CPT>(la + id_delta);   // bytes 0x80 | device id
#pragma unroll
                    for (int c = 0; c < CPT; ++c) {
                        // selector 0x888(8|pu): byte 0 <- rows[pv][pu], bytes 1..3 <- 0 (sign of a byte below 0x80)
                        const unsigned sel = prmt(pu, 0x88888888u, 0x4440u + (unsigned)c);
                        const unsigned off = prmt(rlo[c], rhi[c], sel);
                        const int w = (int)lds32_off4(ea + off);
                        best[c] = __viaddmax_s32(lu[c], w, best[c]);
                    }
                }
                int fin[CPT];
#pragma unroll
                for (int c = 0; c < CPT; ++c) fin[c] = best[c] + rt[c];
                if ((int)rec.x < 0) {
#pragma unroll
                    for (int c = 0; c < CPT; ++c) cpmax[c] = max(cpmax[c], fin[c]);
                }
                // results: global memory (start time forward, bottom level backward) and the window
                long long* gout = out_lane + (unsigned long long)(rec.x & 0x7fffffffu) * ldp;
                if (nvalid == CPT) {
                    if constexpr (CPT == 1) stg_cs(gout, (long long)(FWD ? best[0] : fin[0]));
                    else {
#pragma unroll
                        for (int c = 0; c < CPT; c += 2)
                            stg_cs_v2(gout + c, (long long)(FWD ? best[c] : fin[c]), (long long)(FWD ? best[c + 1] : fin[c + 1]));
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < CPT; ++c)
                        if (c < nvalid) stg_cs(gout + c, (long long)(FWD ? best[c] : fin[c]));
                }
                const unsigned lo = win_lev_lane + rec.y * ROWB;
                st_lev<CPT>(lo, fin);
                st_ids<CPT>(lo + id_delta, (ids & 0x07070707u) | 0x80808080u);
            }
        }
        __syncthreads();   // chunk ci is in the window; its stage slot is free again
        if (*abort_p) break;
        issue(dC, vA, slotb, bar);
        dC = dN;
        if (++slot == D) { slot = 0; par ^= 1u; }
    }
    __syncthreads();
    if (*abort_p) {
        // copies already requested may still be landing in this block's shared memory: give them a bounded
        // time before the block (and its shared memory) goes away
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
        return;
    }
    if (a.cp != nullptr) {
        // maxima of the warps through the (now idle) stage area
        const unsigned red = stage0 + (unsigned)((warp * 32 + lane) * CPT * 4);
#pragma unroll
        for (int c = 0; c < CPT; ++c) sts32(red + 4u * c, (unsigned)cpmax[c]);
        __syncthreads();
        if (warp == 0) {
#pragma unroll
            for (int c = 0; c < CPT; ++c) {
                int m = cpmax[c];
                for (int w = 1; w < nwarps; ++w) m = max(m, (int)lds32(stage0 + (unsigned)(((w * 32 + lane) * CPT + c) * 4)));
                if (c < nvalid) a.cp[j0 + c] = (long long)m;
            }
        }
    }
    (void)ldp8;
}

template <int CPT>
cudaError_t lean_impl(const LeanArgs& a, bool fwd, int warps, size_t smem, cudaStream_t st)
{
    const unsigned grid = (unsigned)((a.P + 32 * CPT - 1) / (32 * CPT));
    cudaError_t e;
    if (fwd) {
        e = cudaFuncSetAttribute(pass_lean_kernel<CPT, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        pass_lean_kernel<CPT, true><<<grid, warps * 32, smem, st>>>(a);
    } else {
        e = cudaFuncSetAttribute(pass_lean_kernel<CPT, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        pass_lean_kernel<CPT, false><<<grid, warps * 32, smem, st>>>(a);
    }
    count_launches(1);
    return cudaGetLastError();
}

inline size_t up16(size_t x) { return (x + 15) & ~(size_t)15; }

}  // namespace

size_t lean_smem_bytes(const LeanPlan& plan, int cpt, int warps, int depth, unsigned* slot_stride, unsigned* stage_bytes)
{
    const size_t slice = 32 * (size_t)cpt;
    const size_t slot = (size_t)plan.rec_max + up16((size_t)plan.max_v * slice);
    size_t stage = (size_t)depth * slot;
    const size_t red = (size_t)warps * slice * 4;   // CP reduction buffer after the last chunk
    if (stage < red) stage = up16(red);
    if (slot_stride) *slot_stride = (unsigned)slot;
    if (stage_bytes) *stage_bytes = (unsigned)stage;
    return stage + (size_t)plan.R * slice * 5;
}

cudaError_t launch_pass_lean(const LeanArgs& a, bool fwd, int cpt, int warps, size_t smem, cudaStream_t st)
{
    if (a.plan.num_chunks <= 0) return cudaSuccess;
    if (cpt == 4) return lean_impl<4>(a, fwd, warps, smem, st);
    if (cpt == 2) return lean_impl<2>(a, fwd, warps, smem, st);
    return lean_impl<1>(a, fwd, warps, smem, st);
}

}  // namespace tfps
