// Per-device compute load, memory load and id validation (the sum inside Eq. 7; the static reading of Eq. 2).
//
//   load[d][j]    = sum over vertices v with p_j(v) = d of rt(v, d) = ceil(c_v*S / s_d)
//   memload[d][j] = sum over the same vertices of mem_v
//
// rt(v, d) comes from a table filled once per tfps_devices_set (rt_rows_kernel), so the hot loop holds no
// division.  A thread owns C candidates and a private column of {load, memload} accumulators per device in
// shared memory (layout [device][c][thread]: no two threads touch the same word, every access is conflict-free),
// so a vertex-candidate costs one 16-byte read-modify-write plus the table lookup.  Ids are checked four at a
// time with byte-parallel arithmetic; an id >= k raises BAD_PARTITION and is counted modulo the padded table.
// Blocks split the vertices; partial sums are merged with 64-bit integer atomics (order independent).
#include "common.cuh"

namespace tfps {

namespace {

__global__ void rt_rows_kernel(int n, int k, int kp, const int* __restrict__ pos_of,
                               const unsigned long long* __restrict__ xvert, const DivConst* __restrict__ rt_div,
                               long long* __restrict__ rtv)
{
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (long long)n * kp) return;
    const int v = (int)(i / kp), d = (int)(i % kp);
    long long r = 0;
    if (d < k) {
        const unsigned long long X = xvert[pos_of[v]];   // runtime numerators are stored by level position
        if (X != NUM_ZERO) r = ceil_quot(X, rt_div[d]);
    }
    rtv[i] = r;
}

template <int C> __device__ __forceinline__ unsigned load_ids(const uint8_t* p)
{
    if constexpr (C == 1) return *p;
    else if constexpr (C == 2) return *reinterpret_cast<const unsigned short*>(p);
    else return *reinterpret_cast<const unsigned*>(p);
}

constexpr int LOADS_THREADS = 128;
constexpr int LOADS_TR = 16;   // rows per tile

__device__ __forceinline__ void cp_async16(void* dst, const void* g)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((unsigned)__cvta_generic_to_shared(dst)), "l"(g) : "memory");
}
__device__ __forceinline__ void cp_async8(void* dst, const void* g)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"((unsigned)__cvta_generic_to_shared(dst)), "l"(g) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait1() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }

// Rows are processed in tiles of LOADS_TR: while one tile is accumulated, the runtime rows and memory values of
// the next one are on their way into shared memory (cp.async) and its ids into registers, so neither the DRAM
// latency of the id stream nor the table lookup sits on the accumulators' dependent chain.
template <int C>   // candidates per thread: 1, 2 or 4
__global__ void __launch_bounds__(LOADS_THREADS)
loads2_kernel(int n, long long P, long long ldp, const uint8_t* __restrict__ part, const long long* __restrict__ rtv,
              const long long* __restrict__ mem, int k, int kp_shift, long long* load, long long* memload, int* status,
              int validate, int rows_per_block)
{
    extern __shared__ __align__(16) longlong2 acc[];   // [KP][C][threads] of {load, memload}, then the row tiles
    constexpr int TR = LOADS_TR;
    const int tid = threadIdx.x;
    const int KP = 1 << kp_shift;
    long long* rt_t = reinterpret_cast<long long*>(acc + KP * C * LOADS_THREADS);   // [2][TR][KP]
    long long* mem_t = rt_t + 2 * TR * KP;                                          // [2][TR]
    for (int i = 0; i < KP * C; ++i) acc[i * LOADS_THREADS + tid] = make_longlong2(0, 0);   // own columns only

    const long long j0 = ((long long)blockIdx.x * LOADS_THREADS + tid) * C;
    const long long rem = P - j0;
    const int nvalid = rem >= C ? C : (rem > 0 ? (int)rem : 0);
    const unsigned bytemask = nvalid >= 4 ? 0xffffffffu : ((1u << (8 * nvalid)) - 1u);
    const unsigned idmask = (unsigned)KP - 1u;
    const unsigned addk = (0x80u - (unsigned)k) * 0x01010101u;   // byte b < 128: b + (128 - k) sets bit 7 iff b >= k
    unsigned bad = 0;
    const int r0 = blockIdx.y * rows_per_block;   // a multiple of TR
    const int r1 = r0 + rows_per_block < n ? r0 + rows_per_block : n;
    const uint8_t* pcol = part + (nvalid > 0 ? j0 : 0);

    auto stage = [&](int t0, int buf) {   // rows t0 .. t0+TR-1 (those below r1) into tile `buf`
        for (int i = tid; i < TR * KP / 2; i += LOADS_THREADS)
            if (t0 + ((2 * i) >> kp_shift) < r1) cp_async16(rt_t + (buf * TR * KP + 2 * i), rtv + ((long long)t0 << kp_shift) + 2 * i);
        if (tid < TR && t0 + tid < r1) cp_async8(mem_t + (buf * TR + tid), mem + t0 + tid);
        cp_async_commit();
    };
    auto fetch_ids = [&](int t0, unsigned (&pk)[TR]) {
#pragma unroll
        for (int q = 0; q < TR; ++q)
            pk[q] = (nvalid > 0 && t0 + q < r1) ? (load_ids<C>(pcol + (long long)(t0 + q) * ldp) & bytemask) : 0u;
    };
    auto process = [&](int t0, int buf, const unsigned (&pk)[TR]) {
        const long long* rt_b = rt_t + buf * TR * KP;
        const long long* mem_b = mem_t + buf * TR;
#pragma unroll
        for (int q = 0; q < TR; ++q) {
            if (t0 + q < r1) {
                bad |= (pk[q] + addk) | pk[q];
                const long long mv = mem_b[q];
                // the C columns of one row are distinct words: read all, add, write all
                longlong2* a[C];
                longlong2 x[C];
                long long rt[C];
#pragma unroll
                for (int c = 0; c < C; ++c) {
                    const unsigned id = (pk[q] >> (8 * c)) & idmask;
                    rt[c] = rt_b[(q << kp_shift) + id];
                    a[c] = acc + ((id * C + c) * LOADS_THREADS + tid);
                    x[c] = *a[c];
                }
#pragma unroll
                for (int c = 0; c < C; ++c) {
                    x[c].x += rt[c];
                    x[c].y += mv;
                }
#pragma unroll
                for (int c = 0; c < C; ++c) *a[c] = x[c];
            }
        }
    };

    unsigned pkA[TR], pkB[TR];
    stage(r0, 0);
    fetch_ids(r0, pkA);
    for (int t0 = r0; t0 < r1; t0 += 2 * TR) {
        stage(t0 + TR, 1);
        fetch_ids(t0 + TR, pkB);
        cp_async_wait1();
        __syncthreads();
        process(t0, 0, pkA);
        __syncthreads();   // tile 0 is free again
        stage(t0 + 2 * TR, 0);
        fetch_ids(t0 + 2 * TR, pkA);
        cp_async_wait1();
        __syncthreads();
        process(t0 + TR, 1, pkB);
        __syncthreads();   // tile 1 is free again
    }
    if (validate && (bad & 0x80808080u)) atomicCAS(status, 0, (int)TFPS_ERR_BAD_PARTITION);
    for (int d = 0; d < k; ++d) {
#pragma unroll
        for (int c = 0; c < C; ++c) {
            if (c < nvalid) {
                const longlong2 x = acc[(d * C + c) * LOADS_THREADS + tid];
                if (load) atomicAdd(reinterpret_cast<unsigned long long*>(load + d * ldp + j0 + c), (unsigned long long)x.x);
                if (memload) atomicAdd(reinterpret_cast<unsigned long long*>(memload + d * ldp + j0 + c), (unsigned long long)x.y);
            }
        }
    }
}

template <int C>
cudaError_t loads2_impl(int n, long long P, long long ldp, const uint8_t* part, const long long* rtv, const long long* mem,
                        int k, int kp_shift, long long* load, long long* memload, int* status, bool validate, int sm_count,
                        int smem_optin, cudaStream_t st)
{
    const size_t smem = ((size_t)1 << kp_shift) * C * LOADS_THREADS * sizeof(longlong2) +
                        (size_t)2 * LOADS_TR * (((size_t)1 << kp_shift) + 1) * sizeof(long long);
    cudaError_t e = cudaFuncSetAttribute(loads2_kernel<C>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const long long gx = (P + LOADS_THREADS * C - 1) / (LOADS_THREADS * C);
    // several blocks per resident slot, so the last wave is short; every block still gets enough rows to pay for its merge
    int resident = (int)(((size_t)smem_optin + 1024) / (smem + 1024));
    if (resident < 1) resident = 1;
    int per_sm = resident * 8;
    if (const char* ov = getenv("TFPS_LOADS_BLOCKS_PER_SM")) { const int q = atoi(ov); if (q >= 1 && q <= 256) per_sm = q; }
    long long gy = ((long long)sm_count * per_sm + gx - 1) / gx;
    const long long gy_max = (n + 255) / 256;   // at least 256 rows per block
    if (gy > gy_max) gy = gy_max;
    if (gy < 1) gy = 1;
    if (gy > 65535) gy = 65535;
    int rows = (int)((n + gy - 1) / gy);
    rows = (rows + LOADS_TR - 1) / LOADS_TR * LOADS_TR;   // tiles start on 16-byte boundaries of the tables
    gy = (n + rows - 1) / rows;
    loads2_kernel<C><<<dim3((unsigned)gx, (unsigned)gy), LOADS_THREADS, smem, st>>>(n, P, ldp, part, rtv, mem, k, kp_shift, load,
                                                                                  memload, status, validate ? 1 : 0, rows);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_rt_rows(int n, int k, int kp, const int* pos_of, const unsigned long long* xvert, const DivConst* rt_div,
                           long long* rtv, cudaStream_t st)
{
    if (n <= 0) return cudaSuccess;
    const long long total = (long long)n * kp;
    rt_rows_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(n, k, kp, pos_of, xvert, rt_div, rtv);
    count_launches(1);
    return cudaGetLastError();
}

// kp = table width (power of two >= k, at most 32); part must be 4-byte aligned
cudaError_t launch_loads2(int n, long long P, long long ldp, const uint8_t* part, const long long* rtv, const long long* mem,
                          int k, int kp, long long* load, long long* memload, int* status, bool validate, int sm_count,
                          int smem_optin, cudaStream_t st)
{
    int kp_shift = 0;
    while ((1 << kp_shift) < kp) ++kp_shift;
    int c = kp <= 8 ? 4 : (kp <= 16 ? 2 : 1);   // 64 KB of accumulators per block at most
    if (const char* ov = getenv("TFPS_LOADS_CPT")) { const int q = atoi(ov); if ((q == 1 || q == 2 || q == 4) && q <= c) c = q; }
    if (c == 4) return loads2_impl<4>(n, P, ldp, part, rtv, mem, k, kp_shift, load, memload, status, validate, sm_count, smem_optin, st);
    if (c == 2) return loads2_impl<2>(n, P, ldp, part, rtv, mem, k, kp_shift, load, memload, status, validate, sm_count, smem_optin, st);
    return loads2_impl<1>(n, P, ldp, part, rtv, mem, k, kp_shift, load, memload, status, validate, sm_count, smem_optin, st);
}

}  // namespace tfps
