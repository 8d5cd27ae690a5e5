// Lean windowed candidate-sliced pass.
//
// Same idea as the windowed pass (one block owns a slice of 16 to 128 candidates, walks the whole graph chunk by chunk and
// keeps the levels of the last R positions of its own candidates in a shared-memory ring, so only the
// compulsory traffic -- one id read and one level write per vertex-candidate -- reaches global memory), cut
// down to the instructions the recurrences need:
//   * the host packs records of one or more consecutive chunks (LeanPlan; narrow levels share a record, with a
//     block barrier between its chunks): vertices in processing order (highest degree first, dealt
//     to the vertex groups in alternating direction, so a fixed assignment is balanced), per-vertex runtimes for
//     every device, and per-edge transfer times for every distinct bandwidth;
//   * the window keeps finish times tlevel+rt (forward) or bottom levels (backward, Eq. 12), so a relaxation
//     only adds the transfer term: one byte permute maps the neighbour's device id to the offset of the right
//     transfer time inside the edge record, one shared-memory load fetches it, one add-max folds it in;
//   * all shared-memory traffic uses 32-bit shared-window addresses;
//   * every warp consumes; the copies of the record `depth` ahead (one bulk copy for the record, 16-byte
//     cp.async pieces for the id rows) are issued by all threads right after the record's last barrier; the descriptor
//     comes from the header of the current record, the vertex ids of the id rows are requested at the top of
//     the record and first touched after that barrier.
// Requirements (checked by the host): every path length fits int32, k <= 8, at most 30 distinct off-diagonal
// bandwidths, the whole window fits in shared memory beside the stage slots.
#include "common.cuh"
#include "ptx.cuh"

namespace tfps {

namespace {

// streaming stores of non-negative 32-bit levels widened to int64 (the high words are zero)
template <int OFF> __device__ __forceinline__ void stg_cs_v2(long long* p, int x, int y)
{
    asm volatile("{\n\t.reg .b64 a, b;\n\tcvt.u64.u32 a, %1;\n\tcvt.u64.u32 b, %2;\n\tst.global.cs.v2.u64 [%0+%3], {a, b};\n\t}"
                 ::"l"(p), "r"(x), "r"(y), "n"(OFF) : "memory");
}
__device__ __forceinline__ void stg_cs(long long* p, int x)
{
    asm volatile("{\n\t.reg .b64 a;\n\tcvt.u64.u32 a, %1;\n\tst.global.cs.u64 [%0], a;\n\t}" ::"l"(p), "r"(x) : "memory");
}
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

// CPT candidates per lane, VPW vertices per warp: a vertex is handled by 32/VPW lanes, so a block owns
// SLICE = 32/VPW*CPT candidates.  Several vertices per warp cut the instructions per vertex-candidate (the
// bookkeeping of a vertex and of an edge is paid once per warp instruction, whatever the number of vertices its
// lanes serve); the lanes of different vertices simply diverge when the degrees differ, and the host deals
// vertices of similar degree to the same warp.  MAXT = largest block size of the instantiation (512 threads may
// use 128 registers each, 1024 threads 64).
template <int CPT, int VPW, bool FWD, int MAXT>
__global__ void __launch_bounds__(MAXT, 1) pass_lean_kernel(const __grid_constant__ LeanArgs a)
{
    extern __shared__ __align__(16) unsigned char dsm[];   // [stage slots][window]
    __shared__ __align__(16) unsigned long long s_rows[LEAN_K_MAX];
    __shared__ __align__(8) unsigned long long s_bar[LEAN_DEPTH_MAX];
    __shared__ int s_cp[128];   // CP maxima of the block's candidates
    constexpr int LPV = 32 / VPW;          // lanes per vertex
    constexpr int SLICE = LPV * CPT;       // candidates of the block = bytes of an id row
    constexpr unsigned LEVB = SLICE * 4;   // a window row: SLICE levels, then SLICE id bytes
    constexpr unsigned ROWB = SLICE * 5;
    constexpr int PR = SLICE / 16;         // 16-byte pieces of an id row
    const int tid = threadIdx.x, nthreads = blockDim.x;
    if (*a.status != 0) return;
    const int D = a.depth;
    const unsigned stage0 = smem_u32(dsm), win0 = stage0 + a.stage_bytes;
    const unsigned rows_s = smem_u32(s_rows), bar0 = smem_u32(s_bar);
    if (tid < LEAN_K_MAX) s_rows[tid] = a.plan.rows[tid];
    for (int t = tid; t < 128; t += nthreads) s_cp[t] = 0;
    if (tid == 0) {
        // a stage completes on the record's bulk copy (one arrival carrying the byte count) plus one arrival
        // per thread once that thread's id-row pieces have landed
        for (int j = 0; j < D; ++j) mbar_init(bar0 + 8u * j, (unsigned)nthreads + 1u);
        mbar_init_fence();
    }
    __syncthreads();

    const int ll = (tid & 31) % LPV;                       // lane within the vertex
    const int group = (tid >> 5) * VPW + (tid & 31) / LPV; // vertex group of this lane
    const int ngroups = (nthreads >> 5) * VPW;
    const long long slice0 = (long long)blockIdx.x * SLICE;
    const unsigned win_lev_lane = win0 + (unsigned)(ll * CPT * 4);
    const unsigned id_delta = LEVB - (unsigned)(3 * ll * CPT);   // id bytes of a lane relative to its levels
    const unsigned rec_max = (unsigned)a.plan.rec_max;
    const bool two_pieces = a.plan.max_v * PR > nthreads;   // a thread fetches one id-row piece per chunk, or two
    const long long j0 = slice0 + (long long)(ll * CPT);
    const bool full = j0 + CPT <= a.P;        // all CPT candidates of this lane exist
    long long* const out_lane = a.lev + j0;
    const unsigned ldp8 = (unsigned)(a.ldp * 8);   // the host keeps ldp below 2^28
    unsigned k88;   // kept in a register (opaque to the compiler), so the selectors below can be immediates
    asm volatile("mov.u32 %0, 0x88888888;" : "=r"(k88));

    // copies of one chunk into a stage slot: d = its descriptor {offset/16, bytes, vertices, first index into
    // vlist}, v0/v1 = vertices of the id rows this thread fetches
    auto issue = [&](const uint4& d, unsigned v0, unsigned v1, unsigned slotb, unsigned bar) {
        if (d.y == 0) return;   // past the last chunk
        const long long ldp = a.ldp;
        const unsigned slice_bytes = (unsigned)((ldp - slice0) < SLICE ? (ldp - slice0) : SLICE);   // multiple of 16
        const uint8_t* part0 = a.part + slice0;
        const unsigned ldp32 = (unsigned)ldp;
        if (tid == 0) {
            mbar_expect_tx(bar, d.y);
            bulk_g2s(slotb, a.plan.blob + 16ll * d.x, d.y, bar);
        }
        {
            const int r = tid / PR, q = tid % PR;
            if (r < (int)d.z && (unsigned)(16 * q) < slice_bytes)
                cp_async16(slotb + rec_max + (unsigned)(r * SLICE + 16 * q), ptr_mad(part0 + 16 * q, v0, ldp32));
        }
        if (two_pieces) {
            const int p = tid + nthreads;
            const int r = p / PR, q = p % PR;
            if (r < (int)d.z && (unsigned)(16 * q) < slice_bytes)
                cp_async16(slotb + rec_max + (unsigned)(r * SLICE + 16 * q), ptr_mad(part0 + 16 * q, v1, ldp32));
        }
        cp_async_arrive_on(bar);
    };
    auto fetch_v = [&](const uint4& d, unsigned& v0, unsigned& v1) {
        const int r0 = tid / PR;
        v0 = r0 < (int)d.z ? (unsigned)__ldg(a.plan.vlist + d.w + r0) : 0u;
        v1 = 0;
        if (two_pieces) {
            const int r1 = (tid + nthreads) / PR;
            if (r1 < (int)d.z) v1 = (unsigned)__ldg(a.plan.vlist + d.w + r1);
        }
    };

    for (int j = 0; j < D; ++j) {   // chunks 0..D-1 (descriptors past the end are zero)
        const int4 di = __ldg(a.plan.desc + j);
        const uint4 d = make_uint4((unsigned)di.x, (unsigned)di.y, (unsigned)di.z, (unsigned)di.w);
        unsigned v0, v1;
        fetch_v(d, v0, v1);
        issue(d, v0, v1, stage0 + (unsigned)j * a.slot_stride, bar0 + 8u * j);
    }
    const int nc = a.plan.num_chunks;
    // Every wait on a stage is followed by a block-wide vote, so all threads agree whether it ran out (the records
    // hold block barriers that every thread must reach): before the loop for record 0, afterwards folded into the
    // barrier that ends a record.
    int slot = 0;
    unsigned par = 0;
    bool timed_out = nc > 0 && !mbar_wait(bar0, 0u, a.wait_limit);
    bool dead = __syncthreads_or(timed_out) != 0;
    for (int ci = 0; ci < nc && !dead; ++ci) {
        const unsigned slotb = stage0 + (unsigned)slot * a.slot_stride;
        const unsigned bar = bar0 + 8u * slot;
        unsigned vA0 = 0, vA1 = 0;
        {
            // the record of chunk ci names chunk ci+D: request the vertex ids of its id rows now, use them after the barrier
            fetch_v(lds128(slotb + 16u * (unsigned)D), vA0, vA1);
            const uint4 hdr = lds128(slotb);   // {chunks, byte offset of the edge area, vertices, -}
            const int nsub = (int)hdr.x;
            const unsigned vbase = slotb + LEAN_HDR_BYTES, ebase = slotb + hdr.y;
            const unsigned idrow = slotb + rec_max + (unsigned)(ll * CPT);
            const int vstride = a.plan.vstride;
            const unsigned estride = (unsigned)a.plan.estride;
            for (int sub = 0; sub < nsub; ++sub) {
            if (sub > 0) __syncthreads();   // the previous chunk of the record is in the window
            const uint2 sc = lds64(slotb + 16u + 16u * LEAN_DEPTH_MAX + 8u * (unsigned)sub);   // {first vertex, vertices}
            const int first = (int)sc.x, cnt = (int)sc.y;
            // rounds alternate direction: group g takes entries g, 2G-1-g, 2G+g, ... of the degree-sorted list
            for (int base = 0; base < cnt; base += 2 * ngroups) {
#pragma unroll 1
              for (int half = 0; half < 2; ++half) {
                const int il = half == 0 ? base + group : base + 2 * ngroups - 1 - group;
                if (il >= cnt) continue;
                const int i = first + il;
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
                unsigned ea = ebase + rec.z;
                const unsigned ee = ebase + rec.w;
                if (ea < ee) {
                    unsigned ns = lds32(ea);
                    bool more;
                    do {
                        const unsigned la = win_lev_lane + ns * ROWB;
                        const unsigned en = ea + estride;
                        more = en < ee;
                        if (more) ns = lds32(en);   // next edge's window slot, ahead of this edge's dependent loads
                        int lu[CPT];
                        ld_lev<CPT>(la, lu);
                        const unsigned pu = ld_ids<CPT>(la + id_delta);   // bytes 0x80 | device id
#pragma unroll
                        for (int c = 0; c < CPT; ++c) {
                            // selector 0x888(8|pu): byte 0 <- rows[pv][pu], bytes 1..3 <- 0 (sign of a byte below 0x80)
                            const unsigned sel = prmt(pu, k88, 0x4440u + (unsigned)c);
                            const unsigned off = prmt(rlo[c], rhi[c], sel);
                            const int w = (int)lds32_off4(ea + off);
                            best[c] = __viaddmax_s32(lu[c], w, best[c]);
                        }
                        ea = en;
                    } while (more);
                }
                int fin[CPT];
#pragma unroll
                for (int c = 0; c < CPT; ++c) fin[c] = best[c] + rt[c];
                if ((int)rec.x < 0) {   // sink (forward) / source (backward): enters the CP maximum; rare
#pragma unroll
                    for (int c = 0; c < CPT; ++c) atomicMax(&s_cp[ll * CPT + c], fin[c]);
                }
                // results: global memory (start time forward, bottom level backward) and the window
                long long* gout = ptr_mad(out_lane, rec.x & 0x7fffffffu, ldp8);
                if (full) {
                    if constexpr (CPT == 1) stg_cs(gout, FWD ? best[0] : fin[0]);
                    if constexpr (CPT >= 2) stg_cs_v2<0>(gout, FWD ? best[0] : fin[0], FWD ? best[1] : fin[1]);
                    if constexpr (CPT == 4) stg_cs_v2<16>(gout, FWD ? best[2] : fin[2], FWD ? best[3] : fin[3]);
                } else {
#pragma unroll
                    for (int c = 0; c < CPT; ++c)
                        if (j0 + c < a.P) stg_cs(gout + c, FWD ? best[c] : fin[c]);
                }
                const unsigned lo = win_lev_lane + rec.y * ROWB;
                st_lev<CPT>(lo, fin);
                st_ids<CPT>(lo + id_delta, (ids & 0x07070707u) | 0x80808080u);
              }
            }
            }
        }
        const uint4 dA = lds128(slotb + 16u * (unsigned)D);   // descriptor of record ci+D, before the slot is overwritten
        // wait for the next record, then one barrier: record ci is in the window, its stage slot is free again,
        // and the outcome of the wait is agreed on
        const int nslot = slot + 1 == D ? 0 : slot + 1;
        const unsigned npar = slot + 1 == D ? par ^ 1u : par;
        if (D > 1) {
            timed_out = ci + 1 < nc && !mbar_wait(bar0 + 8u * nslot, npar, a.wait_limit);
            dead = __syncthreads_or(timed_out) != 0;
            if (dead) break;
            issue(dA, vA0, vA1, slotb, bar);
        } else {   // a single stage: the next record can only be requested once this one is done with
            __syncthreads();
            issue(dA, vA0, vA1, slotb, bar);
            timed_out = ci + 1 < nc && !mbar_wait(bar0 + 8u * nslot, npar, a.wait_limit);
            dead = __syncthreads_or(timed_out) != 0;
            if (dead) break;
        }
        slot = nslot;
        par = npar;
    }
    if (dead) {
        if (timed_out) atomicCAS(a.status, 0, (int)TFPS_ERR_TIMEOUT);
        // copies already requested may still be landing in this block's shared memory: give them a bounded
        // time before the block (and its shared memory) goes away
#pragma unroll 1
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
        return;
    }
    __syncthreads();
    if (a.cp != nullptr)
        for (int t = tid; t < SLICE; t += nthreads)
            if (slice0 + t < a.P) a.cp[slice0 + t] = (long long)s_cp[t];
}

template <int CPT, int VPW, int MAXT>
cudaError_t lean_impl2(const LeanArgs& a, bool fwd, int warps, size_t smem, cudaStream_t st)
{
    constexpr int SLICE = 32 / VPW * CPT;
    const unsigned grid = (unsigned)((a.P + SLICE - 1) / SLICE);
    cudaError_t e;
    if (fwd) {
        e = cudaFuncSetAttribute(pass_lean_kernel<CPT, VPW, true, MAXT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        pass_lean_kernel<CPT, VPW, true, MAXT><<<grid, warps * 32, smem, st>>>(a);
    } else {
        e = cudaFuncSetAttribute(pass_lean_kernel<CPT, VPW, false, MAXT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        pass_lean_kernel<CPT, VPW, false, MAXT><<<grid, warps * 32, smem, st>>>(a);
    }
    count_launches(1);
    return cudaGetLastError();
}

template <int CPT, int VPW>
cudaError_t lean_impl(const LeanArgs& a, bool fwd, int warps, size_t smem, cudaStream_t st)
{
    if (warps <= 16) return lean_impl2<CPT, VPW, 512>(a, fwd, warps, smem, st);
    return lean_impl2<CPT, VPW, 1024>(a, fwd, warps, smem, st);
}

inline size_t up16(size_t x) { return (x + 15) & ~(size_t)15; }

}  // namespace

size_t lean_smem_bytes(const LeanPlan& plan, int slice, int warps, int depth, unsigned* slot_stride, unsigned* stage_bytes)
{
    const size_t slot = (size_t)plan.rec_max + up16((size_t)plan.max_v * (size_t)slice);
    size_t stage = (size_t)depth * slot;
    const size_t red = (size_t)warps * 128 * 4;   // CP reduction buffer after the last chunk (at most 4 candidates per lane)
    if (stage < red) stage = up16(red);
    if (slot_stride) *slot_stride = (unsigned)slot;
    if (stage_bytes) *stage_bytes = (unsigned)stage;
    return stage + (size_t)plan.R * (size_t)slice * (plan.wide ? 9 : 5);
}

// slice = candidates per block (16 ... 128), cpt = candidates per lane (4, 2 or 1): a vertex is served by slice / cpt
// lanes.  Four candidates per lane amortise a vertex' and an edge's bookkeeping best; fewer shorten the dependent
// chain of a level when the graph is deep and narrow and the batch too small to fill the machine anyway.
cudaError_t launch_pass_lean(const LeanArgs& a, bool fwd, int slice, int cpt, int warps, size_t smem, cudaStream_t st)
{
    if (a.plan.num_chunks <= 0) return cudaSuccess;
    const int lpv = slice / cpt;   // lanes per vertex
    if (cpt == 4) {
        if (lpv == 32) return lean_impl<4, 1>(a, fwd, warps, smem, st);
        if (lpv == 16) return lean_impl<4, 2>(a, fwd, warps, smem, st);
        if (lpv == 8) return lean_impl<4, 4>(a, fwd, warps, smem, st);
        if (lpv == 4) return lean_impl<4, 8>(a, fwd, warps, smem, st);
    } else if (cpt == 2) {
        if (lpv == 32) return lean_impl<2, 1>(a, fwd, warps, smem, st);
        if (lpv == 16) return lean_impl<2, 2>(a, fwd, warps, smem, st);
        if (lpv == 8) return lean_impl<2, 4>(a, fwd, warps, smem, st);
    } else if (cpt == 1) {
        if (lpv == 32) return lean_impl<1, 1>(a, fwd, warps, smem, st);
        if (lpv == 16) return lean_impl<1, 2>(a, fwd, warps, smem, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace tfps
