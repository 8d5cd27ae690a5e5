// Lean windowed candidate-sliced pass, wide form: 64-bit levels and up to 16 devices.
//
// Same structure as pass_lean_kernel (lean.cu): a block owns a slice of 8 to 128 candidates, walks the whole graph
// record by record and keeps the finish times (forward) or bottom levels (backward, Eq. 12) of the last R positions
// of its own candidates in shared memory, so that only one id read and one level write per vertex-candidate reach
// global memory.  Differences: levels, transfer times and the window are int64 (9 bytes per position and candidate,
// levels and ids in separate regions), the class of a link comes from a 16 x 16 byte table in shared memory (one
// byte load instead of a byte permute), and a vertex may be served by as few as two lanes (8 candidates per block),
// which is what lets a window of a few thousand positions fit beside the stage slots.
// Requirements (checked by the host): k <= 16, at most 30 distinct off-diagonal bandwidths, every vertex runtime
// below 2^31, the whole window resident.
#include "common.cuh"
#include "ptx.cuh"

namespace tfps {

namespace {

template <int BYTES> __device__ __forceinline__ void cp_async_piece(unsigned dst, const void* g)
{
    if constexpr (BYTES == 16) cp_async16(dst, g);
    else cp_async8_ca(dst, g);
}
template <int OFF> __device__ __forceinline__ void stg_cs_v2(long long* p, long long x, long long y)
{
    asm volatile("st.global.cs.v2.u64 [%0+%3], {%1, %2};" ::"l"(p), "l"(x), "l"(y), "n"(OFF) : "memory");
}
__device__ __forceinline__ void stg_cs(long long* p, long long x) { asm volatile("st.global.cs.u64 [%0], %1;" ::"l"(p), "l"(x) : "memory"); }
constexpr int CPT = 4;   // candidates per lane

// VPW vertices per warp: a vertex is handled by 32/VPW lanes with 4 candidates each, so a block owns
// SLICE = 128/VPW candidates (8 ... 128).
template <int VPW, bool FWD>
__global__ void __launch_bounds__(512, 1) pass_lean64_kernel(const __grid_constant__ LeanArgs a)
{
    extern __shared__ __align__(16) unsigned char dsm[];   // [stage slots][window levels][window ids]
    __shared__ __align__(16) unsigned long long s_rows[2 * LEAN64_K_MAX];   // byte [pv][pu] = 8 * class of the link
    __shared__ __align__(8) unsigned long long s_bar[LEAN_DEPTH_MAX];
    __shared__ long long s_cp[128];   // CP maxima of the block's candidates
    constexpr int LPV = 32 / VPW;            // lanes per vertex
    constexpr int SLICE = LPV * CPT;         // candidates of the block = bytes of an id row
    constexpr unsigned LROW = SLICE * 8;     // bytes of a window row of levels: candidates 0,1 of every lane, then 2,3
    constexpr unsigned LHALF = SLICE * 4;    // (16 bytes per lane and half, so each 16-byte access is conflict-free)
    constexpr unsigned IROW = SLICE;         // bytes of a window row of ids
    constexpr int PB = SLICE >= 16 ? 16 : 8; // bytes of an id-row piece
    constexpr int PR = SLICE / PB;           // pieces of an id row
    const int tid = threadIdx.x, nthreads = blockDim.x;
    if (*a.status != 0) return;
    const int D = a.depth;
    const unsigned stage0 = smem_u32(dsm), win_lev0 = stage0 + a.stage_bytes;
    const unsigned win_id0 = win_lev0 + (unsigned)a.plan.R * LROW;
    const unsigned rows_s = smem_u32(s_rows), bar0 = smem_u32(s_bar);
    if (tid < 2 * LEAN64_K_MAX) s_rows[tid] = a.plan.rows16[tid];
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
    const unsigned lev_lane = win_lev0 + (unsigned)(ll * 16);
    const unsigned id_lane = win_id0 + (unsigned)(ll * CPT);
    const unsigned rec_max = (unsigned)a.plan.rec_max;
    const bool two_pieces = a.plan.max_v * PR > nthreads;   // a thread fetches one id-row piece per record, or two
    const long long j0 = slice0 + (long long)(ll * CPT);
    const bool full = j0 + CPT <= a.P;        // all four candidates of this lane exist
    long long* const out_lane = a.lev + j0;
    const unsigned ldp8 = (unsigned)(a.ldp * 8);   // the host keeps ldp below 2^28

    // copies of one record into a stage slot: d = its descriptor {offset/16, bytes, vertices, first index into
    // vlist}, v0/v1 = vertices of the id rows this thread fetches
    auto issue = [&](const uint4& d, unsigned v0, unsigned v1, unsigned slotb, unsigned bar) {
        if (d.y == 0) return;   // past the last record
        const long long ldp = a.ldp;
        const unsigned slice_bytes = (unsigned)((ldp - slice0) < SLICE ? (ldp - slice0) : SLICE);
        const uint8_t* part0 = a.part + slice0;
        const unsigned ldp32 = (unsigned)ldp;
        if (tid == 0) {
            mbar_expect_tx(bar, d.y);
            bulk_g2s(slotb, a.plan.blob + 16ll * d.x, d.y, bar);
        }
        {
            const int r = tid / PR, q = tid % PR;
            if (r < (int)d.z && (unsigned)(PB * q) < slice_bytes)
                cp_async_piece<PB>(slotb + rec_max + (unsigned)(r * SLICE + PB * q), ptr_mad(part0 + PB * q, v0, ldp32));
        }
        if (two_pieces) {
            const int p = tid + nthreads;
            const int r = p / PR, q = p % PR;
            if (r < (int)d.z && (unsigned)(PB * q) < slice_bytes)
                cp_async_piece<PB>(slotb + rec_max + (unsigned)(r * SLICE + PB * q), ptr_mad(part0 + PB * q, v1, ldp32));
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

    for (int j = 0; j < D; ++j) {   // records 0..D-1 (descriptors past the end are zero)
        const int4 di = __ldg(a.plan.desc + j);
        const uint4 d = make_uint4((unsigned)di.x, (unsigned)di.y, (unsigned)di.z, (unsigned)di.w);
        unsigned v0, v1;
        fetch_v(d, v0, v1);
        issue(d, v0, v1, stage0 + (unsigned)j * a.slot_stride, bar0 + 8u * j);
    }
    const int nc = a.plan.num_chunks;
    // Every wait on a stage is followed by a block-wide vote, so all threads agree whether it ran out (the records
    // hold block barriers that every thread must reach).
    int slot = 0;
    unsigned par = 0;
    bool timed_out = nc > 0 && !mbar_wait(bar0, 0u, a.wait_limit);
    bool dead = __syncthreads_or(timed_out) != 0;
    for (int ci = 0; ci < nc && !dead; ++ci) {
        const unsigned slotb = stage0 + (unsigned)slot * a.slot_stride;
        const unsigned bar = bar0 + 8u * slot;
        unsigned vA0 = 0, vA1 = 0;
        // the record names record ci+D: request the vertex ids of its id rows now, use them after the barrier
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
                    const unsigned ids = lds32(idrow + (unsigned)(i * SLICE)) & 0x0f0f0f0fu;   // masked to the table size
                    unsigned rowaddr[CPT];
                    long long rt[CPT], best[CPT];
#pragma unroll
                    for (int c = 0; c < CPT; ++c) {
                        const unsigned pv16 = (c == 0 ? (ids << 4) : (ids >> (8 * c - 4))) & 0xf0u;   // 16 * own device id
                        rowaddr[c] = rows_s + pv16;
                        rt[c] = (long long)(int)lds32_off16(vr + (pv16 >> 2));
                        best[c] = 0;
                    }
                    unsigned ea = ebase + rec.z;
                    const unsigned ee = ebase + rec.w;
                    if (ea < ee) {
                        unsigned ns = lds32(ea);
                        bool more;
                        do {
                            const unsigned la = lev_lane + ns * LROW;
                            const unsigned ia = id_lane + ns * IROW;
                            const unsigned en = ea + estride;
                            more = en < ee;
                            if (more) ns = lds32(en);   // next edge's window slot, ahead of this edge's dependent loads
                            long long lu[CPT];
                            lds_2x64(la, lu[0], lu[1]);
                            lds_2x64(la + LHALF, lu[2], lu[3]);
                            const unsigned pu = lds32(ia);
#pragma unroll
                            for (int c = 0; c < CPT; ++c) {
                                const unsigned cls8 = lds_u8(rowaddr[c] + ((pu >> (8 * c)) & 0xfu));   // 8 * class of the link
                                const long long v = lu[c] + lds_s64_off8(ea + cls8);
                                best[c] = v > best[c] ? v : best[c];
                            }
                            ea = en;
                        } while (more);
                    }
                    long long fin[CPT];
#pragma unroll
                    for (int c = 0; c < CPT; ++c) fin[c] = best[c] + rt[c];
                    if ((int)rec.x < 0) {   // sink (forward) / source (backward): enters the CP maximum; rare
#pragma unroll
                        for (int c = 0; c < CPT; ++c) atomicMax(&s_cp[ll * CPT + c], fin[c]);
                    }
                    // results: global memory (start time forward, bottom level backward) and the window
                    long long* gout = ptr_mad(out_lane, rec.x & 0x7fffffffu, ldp8);
                    if (full) {
                        stg_cs_v2<0>(gout, FWD ? best[0] : fin[0], FWD ? best[1] : fin[1]);
                        stg_cs_v2<16>(gout, FWD ? best[2] : fin[2], FWD ? best[3] : fin[3]);
                    } else {
#pragma unroll
                        for (int c = 0; c < CPT; ++c)
                            if (j0 + c < a.P) stg_cs(gout + c, FWD ? best[c] : fin[c]);
                    }
                    const unsigned lo = lev_lane + rec.y * LROW;
                    sts_2x64(lo, fin[0], fin[1]);
                    sts_2x64(lo + LHALF, fin[2], fin[3]);
                    sts32(id_lane + rec.y * IROW, ids);
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
            if (slice0 + t < a.P) a.cp[slice0 + t] = s_cp[t];
}

template <int VPW>
cudaError_t lean64_impl(const LeanArgs& a, bool fwd, int warps, size_t smem, cudaStream_t st)
{
    constexpr int SLICE = 128 / VPW;
    const unsigned grid = (unsigned)((a.P + SLICE - 1) / SLICE);
    cudaError_t e;
    if (fwd) {
        e = cudaFuncSetAttribute(pass_lean64_kernel<VPW, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        pass_lean64_kernel<VPW, true><<<grid, warps * 32, smem, st>>>(a);
    } else {
        e = cudaFuncSetAttribute(pass_lean64_kernel<VPW, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        pass_lean64_kernel<VPW, false><<<grid, warps * 32, smem, st>>>(a);
    }
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace

// slice = candidates per block: 128, 64, 32, 16 or 8 (1, 2, 4, 8 or 16 vertices per warp); at most 16 warps
cudaError_t launch_pass_lean64(const LeanArgs& a, bool fwd, int slice, int warps, size_t smem, cudaStream_t st)
{
    if (a.plan.num_chunks <= 0) return cudaSuccess;
    if (slice == 128) return lean64_impl<1>(a, fwd, warps, smem, st);
    if (slice == 64) return lean64_impl<2>(a, fwd, warps, smem, st);
    if (slice == 32) return lean64_impl<4>(a, fwd, warps, smem, st);
    if (slice == 16) return lean64_impl<8>(a, fwd, warps, smem, st);
    return lean64_impl<16>(a, fwd, warps, smem, st);
}

}  // namespace tfps
