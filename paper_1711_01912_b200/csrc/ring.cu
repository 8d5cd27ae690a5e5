// Ring pass: candidate-sliced forward / backward longest-path pass for wide graphs whose edges reach far back.
//
// A block owns RING_SLICE = 8 candidates and walks the whole graph in processing order.  The finish times (forward:
// tlevel + runtime) or bottom levels (backward, Eq. 12) and the device ids of the last R vertices stay in a ring in
// shared memory, so a relaxation reads its neighbour from shared memory and only one id read and one level write per
// vertex and candidate reach global memory.  With eight candidates a ring row is 64 + 8 bytes, which lets a ring of a
// few thousand vertices fit (five layers of 512 vertices: 180 KB).
//
// Warp 0 is the producer: it copies the host-packed records (layout: common.cuh) into a ring of stage slots with one
// bulk copy each, and the id rows of the record's vertices with 8-byte asynchronous copies, both completing on the
// slot's "full" mbarrier; it refills a slot when every consumer warp has arrived on its "empty" mbarrier.  The other
// warps are consumers: a warp takes every W-th round of a step, eight lanes per item (one candidate per lane).
// Vertices with many edges come as wide rounds: the four items are quarters of the edge list and meet through two
// shuffle steps.  Between steps the consumers meet at a named barrier (a step reads what earlier steps wrote).
// Every wait is bounded: a consumer warp whose wait runs out stops computing but keeps the barriers and arrivals of
// the remaining records going, so nobody is left waiting, and the call reports TFPS_ERR_TIMEOUT.
#include "common.cuh"
#include "ptx.cuh"

namespace tfps {

namespace {

constexpr unsigned RING_BAR_STEP = 1;   // named barrier of the consumer warps

__device__ __forceinline__ void ring_bar_sync(unsigned threads)
{
    asm volatile("bar.sync %0, %1;" ::"n"(RING_BAR_STEP), "r"(threads) : "memory");
}
__device__ __forceinline__ void ring_stg_cs(long long* p, long long x)
{
    asm volatile("st.global.cs.u64 [%0], %1;" ::"l"(p), "l"(x) : "memory");
}
__device__ __forceinline__ void ring_stg_cs2(long long* p, long long x, long long y)
{
    asm volatile("st.global.cs.v2.u64 [%0], {%1, %2};" ::"l"(p), "l"(x), "l"(y) : "memory");
}
__device__ __forceinline__ long long ring_max(long long x, long long y) { return x > y ? x : y; }

template <bool FWD, int MAXT>
__global__ void __launch_bounds__(MAXT, 1) pass_ring_kernel(const __grid_constant__ RingArgs a)
{
    extern __shared__ __align__(16) unsigned char dsm[];   // [stage slots][ring levels][ring ids][cls][sc]
    __shared__ __align__(8) unsigned long long s_full[RING_DEPTH_MAX], s_empty[RING_DEPTH_MAX];
    __shared__ long long s_cp[RING_SLICE];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int W = (int)(blockDim.x >> 5) - 1;   // consumer warps
    __shared__ int s_status;
    if (tid == 0) s_status = *a.status;
    __syncthreads();
    if (s_status != 0) return;   // one reading for the whole block: every thread takes the same way
    const int D = a.depth;
    const unsigned slot_stride = (unsigned)(a.rec_max + 8 * a.max_v);
    unsigned char* const ring_lev_b = dsm + (size_t)D * slot_stride;
    unsigned char* const ring_id_b = ring_lev_b + (size_t)a.R * (RING_SLICE * 8);
    unsigned char* const cls_s = ring_id_b + (size_t)a.R * RING_SLICE;
    unsigned char* const sc_s = cls_s + a.kp * a.kp;
    const unsigned stage0 = smem_u32(dsm), full0 = smem_u32(s_full), empty0 = smem_u32(s_empty);
    for (int t = tid; t < a.kp * a.kp; t += blockDim.x) cls_s[t] = a.cls[t];
    if (tid < a.kp) sc_s[tid] = a.sc[tid];
    if (tid < RING_SLICE) s_cp[tid] = 0;
    if (tid == 0) {
        for (int j = 0; j < D; ++j) {
            mbar_init(full0 + 8u * j, 33u);          // the bulk copy's arrival and one per producer lane
            mbar_init(empty0 + 8u * j, (unsigned)W); // one per consumer warp
        }
        mbar_init_fence();
    }
    __syncthreads();
    const long long slice0 = (long long)blockIdx.x * RING_SLICE;
    const int nrec = a.num_records;
    bool timed_out = false;

    if (warp == 0) {
        // ---- producer ----
        const uint8_t* const part0 = a.part + slice0;
        const unsigned ldp32 = (unsigned)a.ldp;
        int slot = 0;
        unsigned par = 0;   // parity of the slot's previous "empty" phase
        for (int ci = 0; ci < nrec; ++ci) {
            const unsigned slotb = stage0 + (unsigned)slot * slot_stride;
            const unsigned bar = full0 + 8u * slot;
            int4 d;
            const unsigned idrow = slotb + (unsigned)a.rec_max;
            if (ci < D) {   // the first records are named by the descriptor array
                d = __ldg(a.desc + ci);
                const int nv = d.z & 0x7fffffff;
                for (int i = lane; i < nv; i += 32)
                    cp_async8_ca(idrow + 8u * i, ptr_mad(part0, (unsigned)__ldg(a.vlist + d.w + i), ldp32));
            } else {        // later ones by the record that held the slot before them
                bool ok = mbar_wait(empty0 + 8u * slot, par, a.wait_limit);
                ok = __all_sync(0xffffffffu, ok) != 0;
                if (!ok) { timed_out = true; break; }
                const unsigned char* const rec = dsm + (size_t)slot * slot_stride;
                d = *reinterpret_cast<const int4*>(rec + 16);
                const int* const vl = reinterpret_cast<const int*>(rec + reinterpret_cast<const int4*>(rec)->w);
                const int nv = d.z & 0x7fffffff;
                for (int i = lane; i < nv; i += 32) cp_async8_ca(idrow + 8u * i, ptr_mad(part0, (unsigned)vl[i], ldp32));
            }
            cp_async_arrive_on(bar);
            __syncwarp();   // every lane has taken what it needs from the old record before the new one lands on it
            if (lane == 0) {
                mbar_expect_tx(bar, (unsigned)d.y);
                bulk_g2s(slotb, a.blob + 16ll * d.x, (unsigned)d.y, bar);
            }
            if (++slot == D) { slot = 0; if (ci >= D) par ^= 1u; }
        }
    } else {
        // ---- consumers ----
        // lane = 2 * pair + half; a pair serves one item, a lane four candidates: 4 * half .. 4 * half + 3
        const int cw = warp - 1, half = lane & 1, pair = lane >> 1;
        const long long j0 = slice0 + 4 * half;
        const bool full = j0 + 4 <= a.P;
        long long* const out_lane = a.lev + j0;
        const unsigned ldp8 = (unsigned)(a.ldp * 8);   // the host keeps ldp below 2^28
        const unsigned kmask4 = ((unsigned)a.kp - 1u) * 0x01010101u, kp = (unsigned)a.kp;
        const unsigned eb = (unsigned)a.ebytes;
        // a ring row of levels: 16-byte columns {c0 c1 | c4 c5 | c2 c3 | c6 c7}, so that the two lanes of a pair read 32
        // contiguous bytes with each 16-byte load
        const unsigned char* const ring_lev = ring_lev_b + 16 * half;
        const unsigned char* const ring_id = ring_id_b + 4 * half;
        const unsigned cthreads = (unsigned)W * 32u;
        long long cpmax[4] = {0, 0, 0, 0};
        bool dead = false;
        int slot = 0;
        unsigned par = 0;
        int round0 = 0;   // rounds of the running step before this record
        bool newstep = true;   // the record opens a step (a live warp learns it from the record before)
        for (int ci = 0; ci < nrec; ++ci) {
            if (dead) newstep = __ldg(a.desc + ci).z < 0;
            if (newstep) {   // everything earlier is in the ring
                ring_bar_sync(cthreads);
                round0 = 0;
            }
            if (!dead) {
                bool ok = mbar_wait(full0 + 8u * slot, par, a.wait_limit);
                ok = __all_sync(0xffffffffu, ok) != 0;
                if (!ok) { dead = true; timed_out = true; }
            }
            if (!dead) {
                const unsigned char* const rec = dsm + (size_t)slot * slot_stride;
                const int4 hdr0 = *reinterpret_cast<const int4*>(rec);   // {rounds | next record opens a step << 31, runtime table, bytes of a runtime row, trailer}
                newstep = hdr0.x < 0;
                const int nrounds = hdr0.x & 0x7fffffff;
                const unsigned char* const ids = rec + a.rec_max + 4 * half;
                int r = cw - round0 % W;
                if (r < 0) r += W;
                for (; r < nrounds; r += W) {
                    const int4 it = *reinterpret_cast<const int4*>(rec + 32 + 256 * r + 16 * pair);
                    const unsigned kind = ((unsigned)it.x >> 27) & 3u;   // lane pairs per vertex: 1, 4 or 16 (the same for a whole round)
                    const unsigned idx = (unsigned)it.y >> 16, myslot = (unsigned)it.y & 0xffffu;
                    const unsigned pv4 = *reinterpret_cast<const unsigned*>(ids + 8u * idx) & kmask4;
                    const unsigned char* row[4];
                    long long best[4];
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        row[c] = cls_s + ((pv4 >> (8 * c)) & 0xffu) * kp;
                        best[c] = 0;
                    }
                    const unsigned char* ea = rec + it.z;
                    const unsigned char* const ee = rec + it.w;
                    if (ea < ee) {
                        unsigned ns = *reinterpret_cast<const unsigned*>(ea);
                        bool more;
                        do {
                            const unsigned char* const en = ea + eb;
                            more = en < ee;
                            const unsigned ns_now = ns;
                            if (more) ns = *reinterpret_cast<const unsigned*>(en);   // ahead of this edge's dependent loads
                            const longlong2 la = *reinterpret_cast<const longlong2*>(ring_lev + ns_now * 64u);
                            const longlong2 lb = *reinterpret_cast<const longlong2*>(ring_lev + ns_now * 64u + 32u);
                            const unsigned pu4 = *reinterpret_cast<const unsigned*>(ring_id + ns_now * 8u);
                            const long long lu[4] = {la.x, la.y, lb.x, lb.y};
#pragma unroll
                            for (int c = 0; c < 4; ++c) {
                                const unsigned c8 = row[c][(pu4 >> (8 * c)) & 0xffu];
                                const long long w = c8 ? *reinterpret_cast<const long long*>(ea + c8) : 0;
                                best[c] = ring_max(best[c], lu[c] + w);
                            }
                            ea = en;
                        } while (more);
                    }
                    if (kind >= 1) {   // quarters (or sixteenths) of one vertex' edges meet
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            best[c] = ring_max(best[c], __shfl_xor_sync(0xffffffffu, best[c], 2));
                            best[c] = ring_max(best[c], __shfl_xor_sync(0xffffffffu, best[c], 4));
                        }
                        if (kind >= 2) {
#pragma unroll
                            for (int c = 0; c < 4; ++c) {
                                best[c] = ring_max(best[c], __shfl_xor_sync(0xffffffffu, best[c], 8));
                                best[c] = ring_max(best[c], __shfl_xor_sync(0xffffffffu, best[c], 16));
                            }
                        }
                    }
                    if ((it.x & (3 << 29)) == 0) {   // neither padding nor a helper pair: this pair writes the vertex
                        const unsigned char* const rtrow = rec + hdr0.y + idx * (unsigned)hdr0.z;
                        long long fin[4];
#pragma unroll
                        for (int c = 0; c < 4; ++c)
                            fin[c] = best[c] + *reinterpret_cast<const int*>(rtrow + sc_s[(pv4 >> (8 * c)) & 0xffu]);
                        unsigned char* const wl = const_cast<unsigned char*>(ring_lev) + myslot * 64u;
                        *reinterpret_cast<longlong2*>(wl) = make_longlong2(fin[0], fin[1]);
                        *reinterpret_cast<longlong2*>(wl + 32) = make_longlong2(fin[2], fin[3]);
                        *reinterpret_cast<unsigned*>(const_cast<unsigned char*>(ring_id) + myslot * 8u) = pv4;
                        if (it.x < 0) {   // sink (forward) / source (backward)
#pragma unroll
                            for (int c = 0; c < 4; ++c) cpmax[c] = ring_max(cpmax[c], fin[c]);
                        }
                        long long* const gout = ptr_mad(out_lane, (unsigned)it.x & 0x03ffffffu, ldp8);
                        if (full) {
                            ring_stg_cs2(gout, FWD ? best[0] : fin[0], FWD ? best[1] : fin[1]);
                            ring_stg_cs2(gout + 2, FWD ? best[2] : fin[2], FWD ? best[3] : fin[3]);
                        } else {
#pragma unroll
                            for (int c = 0; c < 4; ++c)
                                if (j0 + c < a.P) ring_stg_cs(gout + c, FWD ? best[c] : fin[c]);
                        }
                    }
                }
                round0 += nrounds;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty0 + 8u * slot);
            if (++slot == D) { slot = 0; par ^= 1u; }
        }
        if (a.cp != nullptr && !dead) {
#pragma unroll
            for (int c = 0; c < 4; ++c) atomicMax(&s_cp[4 * half + c], cpmax[c]);
        }
    }
    if (timed_out) {
        atomicCAS(a.status, 0, (int)TFPS_ERR_TIMEOUT);
        // copies already requested may still be landing in this block's shared memory: give them a bounded time
#pragma unroll 1
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    }
    __syncthreads();
    if (a.cp != nullptr && tid < RING_SLICE && slice0 + tid < a.P && *a.status == 0) a.cp[slice0 + tid] = s_cp[tid];
}

}  // namespace

// dynamic shared memory of a block: stage slots, ring of levels and ids, class table, speed classes
size_t ring_smem_bytes(int R, int rec_max, int max_v, int depth, int kp)
{
    return (size_t)depth * (size_t)(rec_max + 8 * max_v) + (size_t)R * (RING_SLICE * 9) + (size_t)kp * kp + (size_t)kp;
}

// warps = consumer warps (the block has one more); at most 31
cudaError_t launch_pass_ring(const RingArgs& a, bool fwd, int warps, size_t smem, cudaStream_t st)
{
    if (a.num_records <= 0) return cudaSuccess;
    const unsigned grid = (unsigned)((a.P + RING_SLICE - 1) / RING_SLICE);
    if (warps > 31) warps = 31;
    const unsigned threads = (unsigned)(warps + 1) * 32u;
    cudaError_t e;
#define TFPS_RING_LAUNCH(F, M)                                                                                     \
    do {                                                                                                           \
        e = cudaFuncSetAttribute(pass_ring_kernel<F, M>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);  \
        if (e != cudaSuccess) return e;                                                                            \
        pass_ring_kernel<F, M><<<grid, threads, smem, st>>>(a);                                                    \
    } while (0)
    if (threads <= 544) { if (fwd) TFPS_RING_LAUNCH(true, 544); else TFPS_RING_LAUNCH(false, 544); }
    else { if (fwd) TFPS_RING_LAUNCH(true, 1024); else TFPS_RING_LAUNCH(false, 1024); }
#undef TFPS_RING_LAUNCH
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace tfps
