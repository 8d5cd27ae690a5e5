// Host runtime and C ABI of libtfps: graph handle, CSR validation, device
// tables (exact-division constants), topological structure, launch logic.
#include <algorithm>
#include <array>
#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <utility>

#include "common.cuh"

using namespace tfps;

namespace tfps {
static std::atomic<long long> g_launches{0};
void count_launches(long long n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
}  // namespace tfps

// Scratch of tfps_eval_cp_noalloc: one int64 level matrix, resident on every device that loads the library.
static __device__ __align__(256) unsigned char g_noalloc_scratch[TFPS_NOALLOC_SCRATCH_BYTES];

namespace {

std::mutex g_noalloc_mutex;
void* g_noalloc_ptr[128] = {};  // device address of g_noalloc_scratch, by device ordinal

// The array's name is only a host-side handle: the runtime is asked for its address on the current device, once
// per device.  Called from tfps_devices_set (set-up time), so that the evaluation call itself finds the address
// cached and touches neither the module loader nor an allocator.
cudaError_t noalloc_scratch_address(int device, void** out)
{
    if (device < 0 || device >= 128) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[device]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess) return e;
        g_noalloc_ptr[device] = p;
    }
    *out = g_noalloc_ptr[device];
    return cudaSuccess;
}

thread_local std::string g_last_error;

int fail(int code, const char* fmt, ...)
{
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    g_last_error = buf;
    return code;
}

int fail_cuda(cudaError_t e, const char* what)
{
    return fail(TFPS_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

#define CUDA_TRY(expr)                                              \
    do {                                                            \
        cudaError_t e__ = (expr);                                   \
        if (e__ != cudaSuccess) return fail_cuda(e__, #expr);       \
    } while (0)

#define TFPS_TRY(expr)                   \
    do {                                 \
        int rc__ = (expr);               \
        if (rc__ != TFPS_OK) return rc__; \
    } while (0)

struct DBuf {
    void* p = nullptr;
    size_t bytes = 0;
    DBuf() = default;
    DBuf(const DBuf&) = delete;
    DBuf& operator=(const DBuf&) = delete;
    ~DBuf() { release(); }
    void release() { if (p) cudaFree(p); p = nullptr; bytes = 0; }
    // (re)allocate exactly `b` bytes (at least 16 so that empty graphs still get a pointer)
    cudaError_t alloc(size_t b)
    {
        release();
        if (b < 16) b = 16;
        cudaError_t e = cudaMalloc(&p, b);
        if (e == cudaSuccess) bytes = b; else p = nullptr;
        return e;
    }
    cudaError_t reserve(size_t b) { return b <= bytes ? cudaSuccess : alloc(b); }
    template <typename T> T* as() const { return static_cast<T*>(p); }
};

typedef unsigned __int128 u128;
typedef __int128 i128;

DivConst make_div(unsigned long long d)
{
    unsigned sh = 0;
    while (((u128)1 << sh) < (u128)d) ++sh;  // ceil(log2 d)
    u128 num = (u128)1 << (62 + sh);
    u128 mul = (num + d - 1) / d;
    DivConst dc;
    dc.mul = (unsigned long long)mul;
    dc.sh = sh;
    dc.pad = 0;
    return dc;
}

constexpr long long LIMIT62 = (long long)1 << 62;

}  // namespace

struct tfps_graph {
    int device = 0;
    int sm_count = 1;
    long long n = 0, m = 0;
    // statistics of the inputs kept for the overflow bound
    long long max_c = 0, max_t = 0;
    u128 sum_c = 0, sum_t = 0;
    // graph (device)
    DBuf in_ptr, in_src, in_t, out_ptr, out_dst, out_t, c, mem;
    // topological structure
    bool topo_built = false;
    int num_levels = 0;
    std::vector<long long> h_level_ptr;
    DBuf level, order, level_ptr_d, sink_flag, sink_list;
    int sink_count = 0;
    DBuf f_eptr, f_nbr, f_t, b_eptr, b_nbr, b_t;
    // chunk tables of the candidate-sliced pass
    DBuf vertf, f_chunks, b_chunks;
    int f_num_chunks = 0, b_num_chunks = 0;
    bool f_all_staged = true, b_all_staged = true;
    int max_chunk_v = 1;
    // device tables
    bool dev_set = false;
    int k = 0;
    long long S = 0;
    DBuf rt_div, w_div, cap, xvert, xw_f, xnbr_f, xw_b;
    DBuf rtv;          // [n][rt_kp] runtime of every vertex on every device (loads kernel)
    int rt_kp = 0;     // table width: power of two >= k, or 0 when k is too large for the table
    DBuf pair_f, pair_b, cls_div, sel_f, sel_b;
    // level position of every vertex; longest edge in level positions
    DBuf pos_of;
    int maxspan = 0, smem_optin = 0;
    bool fits32 = false;  // every path length under any partition fits int32
    // host copies of the in-edge CSR for the worst-case path bound
    std::vector<long long> h_in_ptr, h_in_t;
    std::vector<int> h_in_src, h_c;
    int npass = 0, use_cls = 0, ncls_w = 0;
    // lean windowed pass: host-packed chunk records per direction (0 forward, 1 backward)
    struct Lean {
        bool ok = false;
        DBuf blob, desc, vlist;
        LeanPlan plan;
    } lean[2];
    // level-synchronous pass on vertex records (0 forward, 1 backward)
    struct LevRec {
        bool ok = false;
        bool by_id = false;    // steps follow the caller's vertex numbering
        DBuf blob, items, step_ptr, heavy, cls, flags, part_cnt, item_aux;
        std::vector<int> h_step_ptr;   // host copy: the chained variant launches step by step
        int heavy_count = 0;   // vertices evaluated in partial items (their rows start at zero)
        LevRecArgs args;
    } levrec[2];
    DBuf step_bar;             // barrier counters of the persistent record pass
    // ring pass: host-packed records per direction (0 forward, 1 backward)
    struct Ring {
        bool ok = false;
        DBuf blob, desc, vlist, cls, sc;
        RingArgs args;
        size_t smem = 0;
    } ring[2];
    bool id_topo = false;      // the caller's vertex numbering is a topological order ...
    int span_id = 0;           // ... whose longest edge spans this many vertices
    DBuf status;
    // placement constraints (tfps_constraints_set)
    DBuf cons_a, cons_b, cons_v, cons_d;
    // rank-driven partitioners: device speeds, devices from the fastest to the slowest, scratch
    DBuf speed_d, ord_d, bw_d, part_idx, part_flag, part_scr, rank_up, rank_down;
    DBuf sim_ready, sim_left, sim_list;   // scratch of the scheduling simulation
    long long msr_w[4] = {1, 1, 1, 5};     // MSR weights alpha, beta, gamma, delta (Section 5.1)
    int cons_pairs = 0, cons_dev = 0;
    // scratch owned by the handle
    DBuf scr_memload;
    DBuf st_part, st_lev, st_lev2, st_cp, st_load, st_mem, st_viol;
    // phase timing (TFPS_EVAL_PROFILE)
    cudaEvent_t ev[4] = {nullptr, nullptr, nullptr, nullptr};
    bool ev_valid = false;
    bool ran_fwd = false, ran_bwd = false;
    const char* last_kernel = "";
    // copy stream and per-chunk events of tfps_eval_batch_host (created on first use)
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t copy_ev[4] = {};
    // low-priority stream on which the loads kernel runs beside the lean passes (created by tfps_devices_set)
    cudaStream_t aux_stream = nullptr;
    cudaEvent_t aux_fork = nullptr, aux_join = nullptr;
    // second pass stream: the backward lean pass runs beside the forward one (both only read the ids)
    cudaStream_t pass2_stream = nullptr;
    cudaEvent_t pass2_join = nullptr;
    ~tfps_graph()
    {
        for (cudaEvent_t e : ev)
            if (e) cudaEventDestroy(e);
        for (cudaEvent_t e : copy_ev)
            if (e) cudaEventDestroy(e);
        if (copy_stream) cudaStreamDestroy(copy_stream);
        if (aux_fork) cudaEventDestroy(aux_fork);
        if (aux_join) cudaEventDestroy(aux_join);
        if (aux_stream) cudaStreamDestroy(aux_stream);
        if (pass2_join) cudaEventDestroy(pass2_join);
        if (pass2_stream) cudaStreamDestroy(pass2_stream);
    }
};

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

template <typename T>
int fetch(std::vector<T>& dst, const void* src, size_t count, int space, cudaStream_t st)
{
    dst.resize(count);
    if (count == 0) return TFPS_OK;
    if (space == TFPS_HOST) {
        memcpy(dst.data(), src, count * sizeof(T));
    } else {
        CUDA_TRY(cudaMemcpyAsync(dst.data(), src, count * sizeof(T), cudaMemcpyDeviceToHost, st));
        CUDA_TRY(cudaStreamSynchronize(st));
    }
    return TFPS_OK;
}

int fetch_wide(std::vector<long long>& dst, const void* src, size_t count, int dtype, int space, cudaStream_t st)
{
    if (dtype == TFPS_I64) return fetch(dst, src, count, space, st);
    std::vector<int> tmp;
    TFPS_TRY(fetch(tmp, src, count, space, st));
    dst.assign(tmp.begin(), tmp.end());
    return TFPS_OK;
}

int check_csr(const char* name, long long n, long long m, const std::vector<long long>& ptr, const std::vector<int>& idx)
{
    if (ptr[0] != 0) return fail(TFPS_ERR_BAD_CSR, "%s_ptr[0] != 0", name);
    for (long long v = 0; v < n; ++v)
        if (ptr[v + 1] < ptr[v]) return fail(TFPS_ERR_BAD_CSR, "%s_ptr decreases at %lld", name, v);
    if (ptr[n] != m) return fail(TFPS_ERR_BAD_CSR, "%s_ptr[n] = %lld, expected m = %lld", name, ptr[n], m);
    for (long long e = 0; e < m; ++e)
        if (idx[e] < 0 || idx[e] >= n) return fail(TFPS_ERR_BAD_CSR, "%s index %d out of range at edge %lld", name, idx[e], e);
    return TFPS_OK;
}

template <typename T>
int upload(DBuf& buf, const std::vector<T>& v, cudaStream_t st)
{
    CUDA_TRY(buf.alloc(v.size() * sizeof(T)));
    if (!v.empty()) CUDA_TRY(cudaMemcpyAsync(buf.p, v.data(), v.size() * sizeof(T), cudaMemcpyHostToDevice, st));
    return TFPS_OK;
}

int env_int(const char* name, int dflt);

int build_topo(tfps_graph* g, cudaStream_t st)
{
    if (g->topo_built) return TFPS_OK;
    const int n = (int)g->n;
    const int m = (int)g->m;
    if (n == 0) {
        g->num_levels = 0;
        g->h_level_ptr.assign(1, 0);
        g->topo_built = true;
        return TFPS_OK;
    }
    DBuf indeg, queue, level_cnt, result, keys;
    CUDA_TRY(indeg.alloc(sizeof(int) * (size_t)n));
    CUDA_TRY(queue.alloc(sizeof(int) * (size_t)n));
    CUDA_TRY(level_cnt.alloc(sizeof(int) * ((size_t)n + 2)));
    CUDA_TRY(result.alloc(sizeof(long long) * 2));
    CUDA_TRY(g->level.alloc(sizeof(int) * (size_t)n));
    CUDA_TRY(g->order.alloc(sizeof(int) * (size_t)n));
    CUDA_TRY(g->level_ptr_d.alloc(sizeof(long long) * ((size_t)n + 2)));
    CUDA_TRY(cudaMemsetAsync(level_cnt.p, 0, level_cnt.bytes, st));
    CUDA_TRY(cudaMemsetAsync(result.p, 0, result.bytes, st));
    CUDA_TRY(launch_kahn(n, g->in_ptr.as<long long>(), g->out_ptr.as<long long>(), g->out_dst.as<int>(),
                         indeg.as<int>(), g->level.as<int>(), queue.as<int>(), g->level_ptr_d.as<long long>(),
                         level_cnt.as<int>(), result.as<long long>(), g->sm_count, st));
    long long res[2] = {0, 0};
    CUDA_TRY(cudaMemcpyAsync(res, result.p, sizeof res, cudaMemcpyDeviceToHost, st));
    CUDA_TRY(cudaStreamSynchronize(st));
    if (res[1] != n) return fail(TFPS_ERR_CYCLE, "graph has a cycle: only %lld of %d vertices are reachable in topological order", res[1], n);
    g->num_levels = (int)res[0];
    g->h_level_ptr.resize((size_t)g->num_levels + 1);
    CUDA_TRY(cudaMemcpyAsync(g->h_level_ptr.data(), g->level_ptr_d.p, sizeof(long long) * g->h_level_ptr.size(),
                             cudaMemcpyDeviceToHost, st));

    int npad = 1024;
    while (npad < n) npad <<= 1;
    CUDA_TRY(keys.alloc(sizeof(unsigned long long) * (size_t)npad));
    CUDA_TRY(launch_sort_order(n, g->level.as<int>(), keys.as<unsigned long long>(), npad, g->order.as<int>(), st));

    CUDA_TRY(g->f_eptr.alloc(sizeof(int) * ((size_t)n + 1)));
    CUDA_TRY(g->b_eptr.alloc(sizeof(int) * ((size_t)n + 1)));
    CUDA_TRY(g->f_nbr.alloc(sizeof(int) * (size_t)m));
    CUDA_TRY(g->b_nbr.alloc(sizeof(int) * (size_t)m));
    CUDA_TRY(g->f_t.alloc(sizeof(long long) * (size_t)m));
    CUDA_TRY(g->b_t.alloc(sizeof(long long) * (size_t)m));
    CUDA_TRY(launch_build_adj(n, g->order.as<int>(), g->in_ptr.as<long long>(), g->in_src.as<int>(),
                              g->in_t.as<long long>(), g->f_eptr.as<int>(), g->f_nbr.as<int>(), g->f_t.as<long long>(), st));
    CUDA_TRY(launch_build_adj(n, g->order.as<int>(), g->out_ptr.as<long long>(), g->out_dst.as<int>(),
                              g->out_t.as<long long>(), g->b_eptr.as<int>(), g->b_nbr.as<int>(), g->b_t.as<long long>(), st));
    {
        DBuf span;
        CUDA_TRY(span.alloc(sizeof(int)));
        CUDA_TRY(cudaMemsetAsync(span.p, 0, sizeof(int), st));
        CUDA_TRY(g->pos_of.alloc(sizeof(int) * (size_t)n));
        CUDA_TRY(launch_positions(n, g->order.as<int>(), g->pos_of.as<int>(), g->f_nbr.as<int>(), g->f_eptr.as<int>(), span.as<int>(), st));
        CUDA_TRY(cudaMemcpyAsync(&g->maxspan, span.p, sizeof(int), cudaMemcpyDeviceToHost, st));
        CUDA_TRY(cudaStreamSynchronize(st));
    }
    CUDA_TRY(g->sink_flag.alloc((size_t)n));
    CUDA_TRY(launch_sink_flags(n, g->order.as<int>(), g->out_ptr.as<long long>(), g->sink_flag.as<uint8_t>(), st));
    std::vector<uint8_t> flags((size_t)n);
    CUDA_TRY(cudaMemcpyAsync(flags.data(), g->sink_flag.p, (size_t)n, cudaMemcpyDeviceToHost, st));
    CUDA_TRY(cudaStreamSynchronize(st));
    std::vector<int> sinks;
    for (int i = 0; i < n; ++i)
        if (flags[i]) sinks.push_back(i);
    g->sink_count = (int)sinks.size();
    TFPS_TRY(upload(g->sink_list, sinks, st));
    CUDA_TRY(g->vertf.alloc(sizeof(int) * (size_t)n));
    CUDA_TRY(launch_vertf(n, g->order.as<int>(), g->sink_flag.as<uint8_t>(), g->vertf.as<int>(), st));
    // chunk tables: runs of positions inside one level, bounded in vertices and edges
    for (int dir = 0; dir < 2; ++dir) {
        std::vector<int> eptr((size_t)n + 1);
        CUDA_TRY(cudaMemcpyAsync(eptr.data(), dir == 0 ? g->f_eptr.p : g->b_eptr.p, sizeof(int) * ((size_t)n + 1),
                                 cudaMemcpyDeviceToHost, st));
        CUDA_TRY(cudaStreamSynchronize(st));
        std::vector<int> chunks;
        for (int l = 0; l < g->num_levels; ++l) {
            int p = (int)g->h_level_ptr[l];
            const int pend = (int)g->h_level_ptr[l + 1];
            while (p < pend) {
                int q = p + 1;  // a chunk holds at least one vertex, however many edges it has
                while (q < pend && q - p < CHUNK_V && eptr[q + 1] - eptr[p] <= CHUNK_E) ++q;
                chunks.push_back(p);
                chunks.push_back(q - p);
                chunks.push_back(eptr[p]);
                chunks.push_back(eptr[q] - eptr[p]);
                if (eptr[q] - eptr[p] > CHUNK_E) (dir == 0 ? g->f_all_staged : g->b_all_staged) = false;
                g->max_chunk_v = std::max(g->max_chunk_v, q - p);
                p = q;
            }
        }
        (dir == 0 ? g->f_num_chunks : g->b_num_chunks) = (int)(chunks.size() / 4);
        TFPS_TRY(upload(dir == 0 ? g->f_chunks : g->b_chunks, chunks, st));
        CUDA_TRY(cudaStreamSynchronize(st));
    }
    CUDA_TRY(cudaStreamSynchronize(st));
    g->topo_built = true;
    return TFPS_OK;
}

DevTables make_tables(const tfps_graph* g)
{
    DevTables t;
    t.k = g->k;
    t.rt_div = g->rt_div.as<DivConst>();
    t.w_div = g->w_div.as<DivConst>();
    t.cap = g->cap.as<long long>();
    t.npass = g->npass;
    t.use_cls = g->use_cls;
    t.ncls_w = g->ncls_w;
    t.pair_f = g->pair_f.as<DivConst>();
    t.pair_b = g->pair_b.as<DivConst>();
    t.cls_div = g->cls_div.as<DivConst>();
    t.sel_f = g->sel_f.as<unsigned short>();
    t.sel_b = g->sel_b.as<unsigned short>();
    return t;
}

PassArgs make_args(const tfps_graph* g, bool fwd, long long P, long long ldp, const uint8_t* part, long long* lev,
                   long long* cp)
{
    PassArgs a;
    a.adj.vert = g->order.as<int>();
    a.adj.eptr = fwd ? g->f_eptr.as<int>() : g->b_eptr.as<int>();
    a.adj.nbr = fwd ? g->f_nbr.as<int>() : g->b_nbr.as<int>();
    a.adj.xw = fwd ? g->xw_f.as<unsigned long long>() : g->xw_b.as<unsigned long long>();
    a.adj.xnbr = fwd ? g->xnbr_f.as<unsigned long long>() : nullptr;
    a.adj.xvert = g->xvert.as<unsigned long long>();
    a.tab = make_tables(g);
    a.level_ptr = g->level_ptr_d.as<long long>();
    a.num_levels = g->num_levels;
    a.n = (int)g->n;
    a.P = P;
    a.ldp = ldp;
    a.part = part;
    a.lev = lev;
    a.cp = cp;
    a.status = g->status.as<int>();
    return a;
}

int env_int(const char* name, int dflt)
{
    const char* s = getenv(name);
    if (!s || !*s) return dflt;
    return atoi(s);
}

// Packs the chunk records of the lean windowed passes for both directions (layout: LeanPlan in common.cuh).
// Everything is computed on the host with plain integer division; `order` is the host copy of the level order.
// Narrow plan (pass_lean_kernel): every path fits int32 and k <= 8.  Wide plan (pass_lean64_kernel): k <= 16 and
// every vertex runtime below 2^31.  The plan walks the vertices either in level order or, when the caller's vertex
// numbering is itself a topological order whose edges are at least twice shorter, in that order (graphs built layer
// by layer, as data-flow graphs usually are): a shorter longest edge is a smaller window.
int build_lean(tfps_graph* g, int k, const int32_t* s, const int64_t* B, long long S, const std::vector<int>& order,
               cudaStream_t st)
{
    for (auto& L : g->lean) L.ok = false;
    const int n = (int)g->n, m = (int)g->m;
    if (n == 0 || env_int("TFPS_LEAN", 1) == 0) return TFPS_OK;
    std::vector<long long> wvals;   // distinct off-diagonal bandwidths; class c+1 <-> wvals[c], class 0 = same device
    auto cls_of = [&](long long x) {
        for (size_t i = 0; i < wvals.size(); ++i)
            if (wvals[i] == x) return (int)i;
        wvals.push_back(x);
        return (int)wvals.size() - 1;
    };
    long long s_min = INT64_MAX;
    for (int a = 0; a < k; ++a) {
        s_min = std::min<long long>(s_min, s[a]);
        for (int b = 0; b < k; ++b)
            if (a != b) cls_of(B[a * k + b]);
    }
    const int ncw = (int)wvals.size();
    if (ncw > LEAN_CLS_MAX) return TFPS_OK;
    const bool narrow_ok = g->fits32 && k <= LEAN_K_MAX && env_int("TFPS_LEAN_FORCE_WIDE", 0) == 0;
    const u128 rt_max = ((u128)g->max_c * (u128)S + (u128)s_min - 1) / (u128)s_min;
    const bool wide_ok = k <= LEAN64_K_MAX && rt_max < ((u128)1 << 31) && env_int("TFPS_LEAN64", 1) != 0;
    if (!narrow_ok && !wide_ok) return TFPS_OK;
    const bool wide = !narrow_ok;
    const int KP = wide ? 16 : (k <= 4 ? 4 : 8);
    const int vstride = 16 + 4 * KP, estride = wide ? 8 + 8 * (ncw + 1) : 4 * (ncw + 2);
    const int e_cap = std::max(64, std::min(1024, 24576 / estride));   // edges per record

    std::vector<int> pos_of((size_t)n);   // level position of a vertex
    for (int i = 0; i < n; ++i) pos_of[order[i]] = i;
    std::vector<int> eptr[2], nbr[2];     // level-ordered adjacency: [0] in-edges, [1] out-edges
    std::vector<long long> tt[2];
    for (int dir = 0; dir < 2; ++dir) {
        eptr[dir].resize((size_t)n + 1);
        nbr[dir].resize((size_t)m);
        tt[dir].resize((size_t)m);
        CUDA_TRY(cudaMemcpyAsync(eptr[dir].data(), dir == 0 ? g->f_eptr.p : g->b_eptr.p, sizeof(int) * ((size_t)n + 1),
                                 cudaMemcpyDeviceToHost, st));
        if (m > 0) {
            CUDA_TRY(cudaMemcpyAsync(nbr[dir].data(), dir == 0 ? g->f_nbr.p : g->b_nbr.p, sizeof(int) * (size_t)m,
                                     cudaMemcpyDeviceToHost, st));
            CUDA_TRY(cudaMemcpyAsync(tt[dir].data(), dir == 0 ? g->f_t.p : g->b_t.p, sizeof(long long) * (size_t)m,
                                     cudaMemcpyDeviceToHost, st));
        }
    }
    CUDA_TRY(cudaStreamSynchronize(st));
    auto ceil_div = [](long long a, long long S_, long long d) {
        if (a <= (LIMIT62 / S_)) return (a * S_ + d - 1) / d;   // 64-bit arithmetic suffices (d < 2^62)
        return (long long)(((u128)a * (u128)S_ + (u128)d - 1) / (u128)d);
    };

    // plan order: level order, or the caller's numbering when it is topological and its longest edge much shorter
    bool id_topo = true;
    int span_id = 0;
    for (int v = 0; v < n && id_topo; ++v)
        for (long long e = g->h_in_ptr[v]; e < g->h_in_ptr[v + 1]; ++e) {
            const int u = g->h_in_src[e];
            if (u >= v) { id_topo = false; break; }
            span_id = std::max(span_id, v - u);
        }
    bool use_id = id_topo && 2LL * (span_id + LEAN_CHUNK_V) <= (long long)g->maxspan + LEAN_CHUNK_V;
    const int forced_order = env_int("TFPS_LEAN_ORDER", 0);   // 1: level order, 2: caller's numbering (if topological)
    if (forced_order == 1) use_id = false;
    if (forced_order == 2) use_id = id_topo;
    const int span = use_id ? span_id : g->maxspan;
    // vertex at plan position q, plan position of vertex v, level position (index into eptr) of plan position q
    auto vert_at = [&](int q) { return use_id ? q : order[q]; };
    auto ppos = [&](int v) { return use_id ? v : pos_of[v]; };
    auto lpos = [&](int q) { return use_id ? pos_of[q] : q; };

    for (int dir = 0; dir < 2; ++dir) {
        tfps_graph::Lean& L = g->lean[dir];
        const std::vector<int>& ep = eptr[dir];
        auto deg = [&](int q) { const int a = lpos(q); return ep[a + 1] - ep[a]; };
        // chunks (first plan position, vertices) in processing order: mutually independent vertices, at most
        // LEAN_CHUNK_V of them and e_cap edges
        std::vector<int> ch_p0, ch_cnt;
        bool ok = true;
        int max_v = 1;
        if (!use_id) {   // runs of positions inside one level; a wide level is split evenly
            for (int li = 0; li < g->num_levels && ok; ++li) {
                const int l = dir == 0 ? li : g->num_levels - 1 - li;
                int p = (int)g->h_level_ptr[l];
                const int pend = (int)g->h_level_ptr[l + 1];
                const int width = pend - p;
                int target = width;
                if (width > LEAN_CHUNK_V) {
                    const int nch = (width + LEAN_CHUNK_V - 1) / LEAN_CHUNK_V;
                    target = std::min(LEAN_CHUNK_V, (((width + nch - 1) / nch) + 31) / 32 * 32);
                }
                while (p < pend) {
                    int q = p, edges = 0;
                    while (q < pend && q - p < target && edges + deg(q) <= e_cap) { edges += deg(q); ++q; }
                    if (q == p) { ok = false; break; }   // a vertex with more edges than a record can stage
                    ch_p0.push_back(p);
                    ch_cnt.push_back(q - p);
                    max_v = std::max(max_v, q - p);
                    p = q;
                }
            }
        } else {   // consecutive vertices none of which has a neighbour (of this direction) inside the run
            int lo = dir == 0 ? 0 : n - 1, cnt = 0, edges = 0;   // current run: forward [lo, lo+cnt), backward (lo-cnt, lo]
            auto close = [&]() {
                if (cnt == 0) return;
                ch_p0.push_back(dir == 0 ? lo : lo - cnt + 1);
                ch_cnt.push_back(cnt);
                max_v = std::max(max_v, cnt);
            };
            for (int step = 0; step < n && ok; ++step) {
                const int q = dir == 0 ? step : n - 1 - step;
                const int a = lpos(q), d = ep[a + 1] - ep[a];
                if (d > e_cap) { ok = false; break; }
                bool indep = true;   // every neighbour lies before the run (forward) / after it (backward)
                for (int e = ep[a]; e < ep[a + 1] && indep; ++e) {
                    const int x = ppos(nbr[dir][e]);
                    indep = dir == 0 ? x < lo : x > lo;
                }
                if (cnt > 0 && (!indep || cnt >= LEAN_CHUNK_V || edges + d > e_cap)) {
                    close();
                    cnt = 0;
                    edges = 0;
                }
                if (cnt == 0) lo = q;
                ++cnt;
                edges += d;
            }
            close();
        }
        if (!ok) continue;
        // records: consecutive chunks staged together (one wait and one copy issue per record, a block barrier
        // between its chunks), as many as fit LEAN_CHUNK_V vertices, e_cap edges and LEAN_SUB_MAX chunks
        const int nchunks = (int)ch_p0.size();
        auto chunk_edges = [&](int c) {
            int es = 0;
            for (int q = ch_p0[c]; q < ch_p0[c] + ch_cnt[c]; ++q) es += deg(q);
            return es;
        };
        std::vector<int> rec_c0, rec_nc;
        int max_rec_v = 1;
        for (int c = 0; c < nchunks;) {
            int q = c, vs = 0, es = 0;
            while (q < nchunks && q - c < LEAN_SUB_MAX) {
                const int ce = chunk_edges(q);
                if (q > c && (vs + ch_cnt[q] > LEAN_CHUNK_V || es + ce > e_cap)) break;
                vs += ch_cnt[q];
                es += ce;
                ++q;
            }
            rec_c0.push_back(c);
            rec_nc.push_back(q - c);
            max_rec_v = std::max(max_rec_v, vs);
            c = q;
        }
        // window rows: every position written while a record is processed must leave its readers' neighbours intact
        int R = span + max_rec_v;
        if (!wide) { R = 1; while (R < span + max_rec_v) R <<= 1; }
        {
            // a plan whose window cannot fit beside one stage slot at the narrowest block the library picks by itself is not
            // packed (narrower blocks of the wide kernel: only on request, TFPS_LEAN_SLICE)
            const int fs = env_int("TFPS_LEAN_SLICE", 0);
            const int slice_min = wide ? ((fs == 8 || fs == 16) ? fs : 32) : 16;
            if ((long long)R * slice_min * (wide ? 9 : 5) + 16 * 1024 > (long long)g->smem_optin) continue;
        }
        const int nc = (int)rec_c0.size();
        std::vector<int> desc((size_t)(nc + 2 * LEAN_DEPTH_MAX) * 4, 0), vlist((size_t)n);
        std::vector<unsigned char> blob;
        std::vector<int> idx, sorted((size_t)n);
        int rec_max = 16, vfirst = 0;
        // first the processing order and the descriptors (a record names the records that follow it) ...
        size_t total = 0;
        for (int r = 0; r < nc; ++r) {
            int cnt = 0, ne = 0;
            for (int c = rec_c0[r]; c < rec_c0[r] + rec_nc[r]; ++c) {
                const int p0 = ch_p0[c], cc = ch_cnt[c];
                idx.resize((size_t)cc);
                for (int i = 0; i < cc; ++i) idx[i] = p0 + i;
                // highest degree first: dealt to the vertex groups in alternating direction, every round sees similar degrees
                std::stable_sort(idx.begin(), idx.end(), [&](int x, int y) { return deg(x) > deg(y); });
                for (int i = 0; i < cc; ++i) { ne += deg(idx[i]); sorted[(size_t)vfirst + cnt + i] = idx[i]; }
                cnt += cc;
            }
            const size_t e_area = LEAN_HDR_BYTES + (size_t)cnt * vstride;
            const size_t bytes = (e_area + (size_t)ne * estride + 15) & ~(size_t)15;
            desc[4 * (size_t)r + 0] = (int)(total / 16);
            desc[4 * (size_t)r + 1] = (int)bytes;
            desc[4 * (size_t)r + 2] = cnt;
            desc[4 * (size_t)r + 3] = vfirst;
            vfirst += cnt;
            total += bytes;
            rec_max = std::max(rec_max, (int)bytes);
        }
        if (total / 16 >= ((size_t)1 << 31)) continue;
        // ... then the records
        blob.assign(total, 0);
        for (int r = 0; r < nc; ++r) {
            const int cnt = desc[4 * (size_t)r + 2];
            const size_t off = (size_t)desc[4 * (size_t)r] * 16;
            const int first = desc[4 * (size_t)r + 3];
            const size_t e_area = LEAN_HDR_BYTES + (size_t)cnt * vstride;
            int* hdr = reinterpret_cast<int*>(blob.data() + off);
            hdr[0] = rec_nc[r];
            hdr[1] = (int)e_area;
            hdr[2] = cnt;
            for (int d = 1; d <= LEAN_DEPTH_MAX; ++d)
                for (int q = 0; q < 4; ++q) hdr[4 * d + q] = desc[4 * (size_t)(r + d) + q];   // zero past the end
            int* sub = hdr + 4 + 4 * LEAN_DEPTH_MAX;   // per chunk {first vertex of the record, vertices}
            for (int j = 0, at = 0; j < rec_nc[r]; ++j) {
                sub[2 * j] = at;
                sub[2 * j + 1] = ch_cnt[rec_c0[r] + j];
                at += ch_cnt[rec_c0[r] + j];
            }
            int eb = 0;
            for (int i = 0; i < cnt; ++i) {
                const int p = sorted[(size_t)first + i], v = vert_at(p), a = lpos(p);
                int* vr = reinterpret_cast<int*>(blob.data() + off + LEAN_HDR_BYTES + (size_t)i * vstride);
                // the vertex enters the CP maximum: sinks forward, sources backward
                const bool flag = dir == 0 ? (eptr[1][a + 1] == eptr[1][a]) : (eptr[0][a + 1] == eptr[0][a]);
                vr[0] = v | (flag ? (int)0x80000000u : 0);
                vr[1] = p % R;
                vr[2] = eb;
                for (int d = 0; d < k; ++d) vr[4 + d] = (int)ceil_div(g->h_c[v], S, s[d]);
                for (int q = ep[a]; q < ep[a + 1]; ++q) {
                    unsigned char* er = blob.data() + off + e_area + (size_t)eb;
                    const int ns = ppos(nbr[dir][q]) % R;
                    memcpy(er, &ns, 4);
                    for (int w = 0; w < ncw; ++w) {
                        const long long val = ceil_div(tt[dir][q], S, wvals[w]);
                        if (wide) memcpy(er + 16 + 8 * w, &val, 8);                     // {slot, pad, W[0] = 0, W[1..]}
                        else { const int v32 = (int)val; memcpy(er + 8 + 4 * w, &v32, 4); }   // {slot, W[0] = 0, W[1..]}
                    }
                    eb += estride;
                }
                vr[3] = eb;
                vlist[(size_t)first + i] = v;
            }
        }
        if (blob.size() / 16 >= ((size_t)1 << 31)) continue;
        TFPS_TRY(upload(L.blob, blob, st));
        TFPS_TRY(upload(L.desc, desc, st));
        TFPS_TRY(upload(L.vlist, vlist, st));
        CUDA_TRY(cudaStreamSynchronize(st));
        L.plan.blob = L.blob.as<unsigned char>();
        L.plan.desc = L.desc.as<int4>();
        L.plan.vlist = L.vlist.as<int>();
        L.plan.num_chunks = nc;
        L.plan.vstride = vstride;
        L.plan.estride = estride;
        L.plan.R = R;
        L.plan.rec_max = rec_max;
        L.plan.max_v = max_rec_v;
        L.plan.max_sub = max_v;
        L.plan.wide = wide ? 1 : 0;
        // class of the link between a neighbour on device pu and a vertex on device pv (0 = same device), scaled to
        // the byte offset of its transfer time inside an edge record
        auto link = [&](int pu, int pv) {
            if (pv >= k || pu >= k || pu == pv) return 0;
            return cls_of(dir == 0 ? B[pu * k + pv] : B[pv * k + pu]) + 1;
        };
        for (int pv = 0; pv < LEAN_K_MAX; ++pv) {
            unsigned long long row = 0;
            for (int pu = 0; pu < LEAN_K_MAX; ++pu) row |= (unsigned long long)(4 * link(pu, pv)) << (8 * pu);
            L.plan.rows[pv] = row;
        }
        for (int pv = 0; pv < LEAN64_K_MAX; ++pv)
            for (int h = 0; h < 2; ++h) {
                unsigned long long row = 0;
                for (int b = 0; b < 8; ++b) row |= (unsigned long long)(8 * link(8 * h + b, pv)) << (8 * b);
                L.plan.rows16[2 * pv + h] = row;
            }
        L.ok = true;
    }
    return TFPS_OK;
}

// Packs the vertex records, work items and steps of the persistent record pass (layout: levrec.cu) for both
// directions.  Steps are the topological levels, or -- when the caller's vertex numbering is a topological order whose
// longest edge is at most half as long and which needs at most twice as many steps -- runs of consecutive vertices
// none of which depends on a vertex of the same run: the rows a step reads then lie within a short range of rows.
int build_levrec(tfps_graph* g, int k, const int32_t* s, const int64_t* B, long long S, const std::vector<int>& order,
                 cudaStream_t st)
{
    for (auto& L : g->levrec) L.ok = false;
    const int n = (int)g->n, m = (int)g->m;
    if (n == 0 || env_int("TFPS_LEVREC", 1) == 0) return TFPS_OK;
    std::vector<long long> wvals;
    auto cls_of = [&](long long x) {
        for (size_t i = 0; i < wvals.size(); ++i)
            if (wvals[i] == x) return (int)i;
        wvals.push_back(x);
        return (int)wvals.size() - 1;
    };
    long long s_min = INT64_MAX;
    for (int a = 0; a < k; ++a) {
        s_min = std::min<long long>(s_min, s[a]);
        for (int b = 0; b < k; ++b)
            if (a != b) cls_of(B[a * k + b]);
    }
    const int ncw = (int)wvals.size();
    const u128 rt_max = ((u128)g->max_c * (u128)S + (u128)s_min - 1) / (u128)s_min;
    if (ncw > 255 || rt_max >= ((u128)1 << 31)) return TFPS_OK;   // class indices are bytes, runtimes int32
    auto ceil_div = [](long long a, long long S_, long long d) {
        if (a <= (LIMIT62 / S_)) return (a * S_ + d - 1) / d;   // 64-bit arithmetic suffices (d < 2^62)
        return (long long)(((u128)a * (u128)S_ + (u128)d - 1) / (u128)d);
    };
    const int KP = k <= 16 ? 16 : 64;
    const int HDR = 16 + 4 * KP;
    // speed classes: the runtime of a vertex depends on its device only through the device's speed
    std::vector<long long> svals;
    std::vector<int> sc_of((size_t)k);
    for (int d = 0; d < k; ++d) {
        size_t i = 0;
        while (i < svals.size() && svals[i] != s[d]) ++i;
        if (i == svals.size()) svals.push_back(s[d]);
        sc_of[d] = (int)i;
    }
    const int ns = (int)svals.size();
    // forward edge costs: one value per (link class, speed class of the neighbour's device) when those are few
    // enough for a byte index, else transfer times per class plus the neighbour's runtimes per device (RTU form)
    const bool rtu = (ncw + 1) * ns > 255;
    std::vector<int> rtab((size_t)n * k);   // runtime of every vertex on every device
    for (int v = 0; v < n; ++v)
        for (int q = 0; q < k; ++q) rtab[(size_t)v * k + q] = (int)ceil_div(g->h_c[v], S, s[q]);
    std::vector<int> pos_of((size_t)n);
    for (int i = 0; i < n; ++i) pos_of[order[i]] = i;
    if (!g->step_bar.p) {
        CUDA_TRY(g->step_bar.alloc(128 * STEPREC_GROUPS_MAX));
    }
    for (int dir = 0; dir < 2; ++dir) {
        tfps_graph::LevRec& L = g->levrec[dir];
        std::vector<int> ep((size_t)n + 1), nb((size_t)m);
        std::vector<long long> tt((size_t)m);
        CUDA_TRY(cudaMemcpyAsync(ep.data(), dir == 0 ? g->f_eptr.p : g->b_eptr.p, sizeof(int) * ((size_t)n + 1), cudaMemcpyDeviceToHost, st));
        if (m > 0) {
            CUDA_TRY(cudaMemcpyAsync(nb.data(), dir == 0 ? g->f_nbr.p : g->b_nbr.p, sizeof(int) * (size_t)m, cudaMemcpyDeviceToHost, st));
            CUDA_TRY(cudaMemcpyAsync(tt.data(), dir == 0 ? g->f_t.p : g->b_t.p, sizeof(long long) * (size_t)m, cudaMemcpyDeviceToHost, st));
        }
        CUDA_TRY(cudaStreamSynchronize(st));
        const int ncomb = (dir == 0 && !rtu) ? (ncw + 1) * ns : ncw + 1;
        const int wbytes = 8 * ncomb;
        const int estride = (8 + wbytes + ((dir == 0 && rtu) ? 4 * KP : 0) + 15) & ~15;
        // a vertex with more than T edges becomes ceil(deg / T) partial items of at most T edges
        const int T = std::max(1, std::min(std::max(1, env_int("TFPS_TILE_SPLIT", 8)), 2048 / estride));
        // steps: lists of level positions in processing order
        std::vector<int> sp_level, sp_id, vs_id;   // step pointers; vertices (as level positions) of the caller-order steps
        for (int li = 0; li <= g->num_levels; ++li) sp_level.push_back((int)g->h_level_ptr[li]);
        bool use_id = false;
        if (g->id_topo && env_int("TFPS_STEP_ORDER", 0) != 1) {
            vs_id.resize((size_t)n);
            int lo = dir == 0 ? 0 : n - 1;   // first vertex of the running step
            sp_id.push_back(0);
            for (int stp = 0; stp < n; ++stp) {
                const int v = dir == 0 ? stp : n - 1 - stp;
                const int p = pos_of[v];
                bool indep = true;   // every neighbour lies before (forward) / after (backward) the running step
                for (int e = ep[p]; e < ep[p + 1] && indep; ++e) indep = dir == 0 ? nb[e] < lo : nb[e] > lo;
                if (!indep) { sp_id.push_back(stp); lo = v; }
                vs_id[(size_t)stp] = p;
            }
            sp_id.push_back(n);
            const bool shorter = 2LL * g->span_id <= (long long)g->maxspan && (long long)sp_id.size() - 1 <= 2LL * g->num_levels;
            use_id = shorter || env_int("TFPS_STEP_ORDER", 0) == 2;
        }
        const std::vector<int>& sp = use_id ? sp_id : sp_level;
        const int nsteps = (int)sp.size() - 1;
        std::vector<long long> roff((size_t)n + 1);
        size_t total = 0;   // in units of 16 bytes
        for (int p = 0; p < n; ++p) {
            roff[p] = (long long)total;
            total += ((size_t)HDR + (size_t)(ep[p + 1] - ep[p]) * estride) / 16;
        }
        roff[n] = (long long)total;
        if (total >= ((size_t)1 << 31)) continue;
        std::vector<int> items, step_ptr((size_t)nsteps + 1, 0), heavy, idx, aux;
        int item_edges = 0, max_items = 1;
        for (int sidx = 0; sidx < nsteps; ++sidx) {
            // forward: steps in ascending order; backward: level steps in descending order (caller-order steps are built descending)
            const int src = (dir == 1 && !use_id) ? nsteps - 1 - sidx : sidx;
            step_ptr[sidx] = (int)(items.size() / 8);
            idx.clear();
            for (int q = sp[src]; q < sp[src + 1]; ++q) idx.push_back(use_id ? vs_id[(size_t)q] : q);
            std::stable_sort(idx.begin(), idx.end(), [&](int x, int y) { return ep[x + 1] - ep[x] > ep[y + 1] - ep[y]; });
            auto push_item = [&](int p, bool partial, int e0, int e1) {   // descriptor, then the neighbours of its first four edges
                items.push_back(order[p] | (partial ? (int)0x80000000u : 0)); items.push_back((int)roff[p]); items.push_back(e0); items.push_back(e1);
                for (int q = 0; q < 4; ++q) items.push_back(e0 + q < e1 ? nb[(size_t)ep[p] + e0 + q] : 0);
                aux.push_back(partial ? (int)heavy.size() - 1 : 0);   // which of the cut vertices, and into how many items
                aux.push_back(partial ? (ep[p + 1] - ep[p] + T - 1) / T : 1);
            };
            for (int p : idx) {
                const int d = ep[p + 1] - ep[p];
                if (d > T) {
                    heavy.push_back(order[p]);
                    for (int e = 0; e < d; e += T) push_item(p, true, e, std::min(d, e + T));
                    item_edges = std::max(item_edges, T);
                } else {
                    push_item(p, false, 0, d);
                    item_edges = std::max(item_edges, d);
                }
            }
            max_items = std::max(max_items, (int)(items.size() / 8) - step_ptr[sidx]);
        }
        step_ptr[nsteps] = (int)(items.size() / 8);
        std::vector<unsigned char> blob(total * 16, 0);
        for (int p = 0; p < n; ++p) {
            unsigned char* r = blob.data() + (size_t)roff[p] * 16;
            const int v = order[p], d = ep[p + 1] - ep[p];
            int* hdr = reinterpret_cast<int*>(r);
            hdr[0] = v;
            hdr[1] = d;
            memcpy(hdr + 4, &rtab[(size_t)v * k], sizeof(int) * (size_t)k);
            for (int e = 0; e < d; ++e) {
                unsigned char* er = r + HDR + (size_t)e * estride;
                const int u = nb[(size_t)ep[p] + e];
                memcpy(er, &u, 4);
                // {neighbour, pad, V[ncomb]}: class 0 = same device (no transfer)
                for (int w = 0; w <= ncw; ++w) {
                    const long long tr = w == 0 ? 0 : ceil_div(tt[(size_t)ep[p] + e], S, wvals[(size_t)w - 1]);
                    if (dir == 0 && !rtu) {
                        for (int q = 0; q < ns; ++q) {
                            const long long val = tr + ceil_div(g->h_c[u], S, svals[(size_t)q]);   // + the neighbour's runtime
                            memcpy(er + 8 + 8 * (w * ns + q), &val, 8);
                        }
                    } else {
                        memcpy(er + 8 + 8 * w, &tr, 8);
                    }
                }
                if (dir == 0 && rtu) memcpy(er + 8 + wbytes, &rtab[(size_t)u * k], sizeof(int) * (size_t)k);
            }
        }
        // cost combination of a neighbour on device pu and a vertex on device pv (devices beyond k never occur: ids are
        // checked by the loads kernel; the table is zero there)
        std::vector<unsigned char> cls((size_t)KP * KP, 0);
        for (int pu = 0; pu < k; ++pu)
            for (int pv = 0; pv < k; ++pv) {
                const int lc = pu == pv ? 0 : cls_of(dir == 0 ? B[pu * k + pv] : B[pv * k + pu]) + 1;
                cls[(size_t)pu * KP + pv] = (unsigned char)((dir == 0 && !rtu) ? lc * ns + sc_of[pu] : lc);
            }
        TFPS_TRY(upload(L.blob, blob, st));
        TFPS_TRY(upload(L.items, items, st));
        TFPS_TRY(upload(L.step_ptr, step_ptr, st));
        TFPS_TRY(upload(L.heavy, heavy, st));
        TFPS_TRY(upload(L.cls, cls, st));
        TFPS_TRY(upload(L.item_aux, aux, st));
        CUDA_TRY(L.flags.alloc(sizeof(unsigned) * (size_t)std::max(1, n)));
        CUDA_TRY(L.part_cnt.alloc(sizeof(int) * 32 * std::max<size_t>(1, heavy.size())));
        CUDA_TRY(cudaStreamSynchronize(st));
        L.heavy_count = (int)heavy.size();
        L.h_step_ptr = step_ptr;
        L.by_id = use_id;
        L.args = LevRecArgs{};
        L.args.blob = L.blob.as<unsigned char>();
        L.args.items = L.items.as<int4>();
        L.args.step_ptr = L.step_ptr.as<int>();
        L.args.num_steps = nsteps;
        L.args.max_step_items = max_items;
        L.args.cls = L.cls.as<unsigned char>();
        L.args.bar = g->step_bar.as<unsigned>();
        L.args.kp = KP;
        L.args.estride = estride;
        L.args.wbytes = wbytes;
        L.args.rtu = (dir == 0 && rtu) ? 1 : 0;
        L.args.rec_max = HDR + item_edges * estride;
        L.args.flags = L.flags.as<unsigned>();
        L.args.part_cnt = L.part_cnt.as<int>();
        L.args.item_aux = L.item_aux.as<int2>();
        L.args.num_items = (int)(items.size() / 8);
        L.args.num_vertices = n;
        L.args.num_heavy = (int)heavy.size();
        L.ok = true;
    }
    return TFPS_OK;
}

// Packs the records of the ring pass (layout: common.cuh, kernel: ring.cu) for both directions.  Processing order and
// steps: the caller's vertex numbering cut into runs of mutually independent vertices when it is a topological order
// and its ring is shorter, else the topological levels.  The ring length R is the longest stretch, over the steps,
// from the oldest vertex a step reads to the last vertex it writes.
int build_ring(tfps_graph* g, int k, const int32_t* s, const int64_t* B, long long S, const std::vector<int>& order,
               cudaStream_t st)
{
    for (auto& L : g->ring) L.ok = false;
    const int n = (int)g->n, m = (int)g->m;
    if (n == 0 || env_int("TFPS_RING", 1) == 0) return TFPS_OK;
    std::vector<long long> wvals, svals;
    auto cls_of = [&](long long x) {
        for (size_t i = 0; i < wvals.size(); ++i)
            if (wvals[i] == x) return (int)i;
        wvals.push_back(x);
        return (int)wvals.size() - 1;
    };
    long long s_min = INT64_MAX;
    std::vector<int> sc_of((size_t)k);
    for (int a = 0; a < k; ++a) {
        s_min = std::min<long long>(s_min, s[a]);
        size_t i = 0;
        while (i < svals.size() && svals[i] != s[a]) ++i;
        if (i == svals.size()) svals.push_back(s[a]);
        sc_of[a] = (int)i;
        for (int b = 0; b < k; ++b)
            if (a != b) cls_of(B[a * k + b]);
    }
    const int ncw = (int)wvals.size(), nsc = (int)svals.size();
    const u128 rt_max = ((u128)g->max_c * (u128)S + (u128)s_min - 1) / (u128)s_min;
    if (ncw > RING_CLS_MAX || rt_max >= ((u128)1 << 31)) return TFPS_OK;
    auto ceil_div = [](long long a, long long S_, long long d) {
        if (a <= (LIMIT62 / S_)) return (a * S_ + d - 1) / d;
        return (long long)(((u128)a * (u128)S_ + (u128)d - 1) / (u128)d);
    };
    const int KP = k <= 16 ? 16 : 64;
    const int ebytes = 8 + 8 * ncw, rtrow = 4 * nsc;
    const int wide_min = std::max(1, env_int("TFPS_RING_WIDE", 6));      // more edges than this: four lane pairs per vertex
    const int wide2_min = std::max(wide_min, env_int("TFPS_RING_WIDE2", 24));   // more than this: all sixteen
    const int rec_v = std::max(4, std::min(1024, env_int("TFPS_RING_REC_V", 128)));
    const int rec_bytes = std::max(1024, env_int("TFPS_RING_REC_BYTES", 11000));
    std::vector<int> pos_of((size_t)n);
    for (int i = 0; i < n; ++i) pos_of[order[i]] = i;
    // both adjacencies by level position: the other direction's degrees tell sinks and sources
    std::vector<int> epd[2];
    for (int dir = 0; dir < 2; ++dir) {
        epd[dir].resize((size_t)n + 1);
        CUDA_TRY(cudaMemcpyAsync(epd[dir].data(), dir == 0 ? g->f_eptr.p : g->b_eptr.p, sizeof(int) * ((size_t)n + 1), cudaMemcpyDeviceToHost, st));
    }
    CUDA_TRY(cudaStreamSynchronize(st));
    for (int dir = 0; dir < 2; ++dir) {
        tfps_graph::Ring& L = g->ring[dir];
        const std::vector<int>& ep = epd[dir];
        const std::vector<int>& ep_other = epd[1 - dir];
        std::vector<int> nb((size_t)m);
        std::vector<long long> tt((size_t)m);
        if (m > 0) {
            CUDA_TRY(cudaMemcpyAsync(nb.data(), dir == 0 ? g->f_nbr.p : g->b_nbr.p, sizeof(int) * (size_t)m, cudaMemcpyDeviceToHost, st));
            CUDA_TRY(cudaMemcpyAsync(tt.data(), dir == 0 ? g->f_t.p : g->b_t.p, sizeof(long long) * (size_t)m, cudaMemcpyDeviceToHost, st));
        }
        CUDA_TRY(cudaStreamSynchronize(st));
        // candidate processing orders: seq = level positions in processing order, sp = step pointers into seq
        std::vector<int> seq_best, sp_best, qof_best;
        long long R_best = -1;
        for (int mode = 0; mode < 2; ++mode) {   // 0: topological levels, 1: the caller's numbering
            if (mode == 1 && (!g->id_topo || env_int("TFPS_STEP_ORDER", 0) == 1)) continue;
            std::vector<int> seq((size_t)n), sp;
            if (mode == 0) {
                for (int li = 0; li <= g->num_levels; ++li) sp.push_back((int)g->h_level_ptr[li]);
                if (dir == 0) for (int i = 0; i < n; ++i) seq[(size_t)i] = i;
                else {   // levels from the last to the first
                    std::vector<int> sp2;
                    int q = 0;
                    sp2.push_back(0);
                    for (int li = g->num_levels - 1; li >= 0; --li) {
                        for (int p = sp[(size_t)li]; p < sp[(size_t)li + 1]; ++p) seq[(size_t)q++] = p;
                        sp2.push_back(q);
                    }
                    sp.swap(sp2);
                }
            } else {
                int lo = dir == 0 ? 0 : n - 1;   // first vertex of the running step
                sp.push_back(0);
                for (int stp = 0; stp < n; ++stp) {
                    const int v = dir == 0 ? stp : n - 1 - stp;
                    const int p = pos_of[v];
                    bool indep = true;
                    for (int e = ep[p]; e < ep[p + 1] && indep; ++e) indep = dir == 0 ? nb[e] < lo : nb[e] > lo;
                    if (!indep) { sp.push_back(stp); lo = v; }
                    seq[(size_t)stp] = p;
                }
                sp.push_back(n);
            }
            std::vector<int> qof((size_t)n);   // processing index of every vertex
            for (int q = 0; q < n; ++q) qof[(size_t)order[seq[(size_t)q]]] = q;
            long long R = 1;
            for (size_t si = 0; si + 1 < sp.size(); ++si) {
                int oldest = sp[si];
                for (int q = sp[si]; q < sp[si + 1]; ++q) {
                    const int p = seq[(size_t)q];
                    for (int e = ep[p]; e < ep[p + 1]; ++e) oldest = std::min(oldest, qof[(size_t)nb[e]]);
                }
                R = std::max<long long>(R, (long long)sp[si + 1] - oldest);
            }
            if (R_best < 0 || R < R_best || env_int("TFPS_STEP_ORDER", 0) == 2) {
                R_best = R; seq_best.swap(seq); sp_best.swap(sp); qof_best.swap(qof);
            }
        }
        const std::vector<int>&seq = seq_best, &sp = sp_best, &qof = qof_best;
        const int R = (int)R_best;
        if (R_best > 65535) continue;
        // rounds step by step, records of consecutive rounds.  A round has 16 items (one per lane pair); a vertex takes
        // 1, 4 or 16 of them (kind 0, 1, 2) according to its degree, each with a share of its edges.
        struct Item { int p, e0, e1; bool helper, skip; };   // level position, edge range within the vertex
        struct Round { Item it[16]; int kind, cost; };
        std::vector<unsigned char> raw, blob;   // records without and with their trailers
        std::vector<int> desc, vlist, rec_raw, rec_nv, rec_vfirst, rec_first;
        std::vector<size_t> rec_base;
        int rec_max = 16, max_v = 2, nrecords = 0;
        std::vector<int> idx;
        std::vector<Round> rounds;
        bool fits = true;
        for (size_t si = 0; si + 1 < sp.size() && fits; ++si) {
            idx.assign(seq.begin() + sp[si], seq.begin() + sp[si + 1]);
            std::stable_sort(idx.begin(), idx.end(), [&](int x, int y) { return ep[x + 1] - ep[x] > ep[y + 1] - ep[y]; });
            rounds.clear();
            size_t i = 0;
            auto deg = [&](size_t q) { return ep[idx[q] + 1] - ep[idx[q]]; };
            for (int kind = 2; kind >= 0; --kind) {
                const int gsz = kind == 2 ? 16 : kind == 1 ? 4 : 1, per = 16 / gsz;   // pairs per vertex, vertices per round
                const int lower = kind == 2 ? wide2_min : kind == 1 ? wide_min : -1;  // degrees above this take this kind
                while (i < idx.size() && deg(i) > lower) {
                    Round r;
                    r.kind = kind;
                    r.cost = (deg(i) + gsz - 1) / gsz + 2 * kind;
                    for (int q = 0; q < per; ++q) {
                        const bool have = i < idx.size() && deg(i) > lower;
                        const int p = have ? idx[i] : idx[0], d = have ? ep[p + 1] - ep[p] : 0, share = (d + gsz - 1) / gsz;
                        for (int h = 0; h < gsz; ++h)
                            r.it[q * gsz + h] = Item{p, std::min(d, h * share), std::min(d, (h + 1) * share), h > 0, !have};
                        if (have) ++i;
                    }
                    rounds.push_back(r);
                }
            }
            // dearest rounds first (the warps take the rounds of a step in turn)
            std::vector<int> ro(rounds.size());
            for (size_t q = 0; q < ro.size(); ++q) ro[q] = (int)q;
            std::stable_sort(ro.begin(), ro.end(), [&](int x, int y) { return rounds[(size_t)x].cost > rounds[(size_t)y].cost; });
            size_t r0 = 0;
            bool first = true;
            while (r0 < ro.size()) {
                // rounds r0..r1-1 form a record: at most rec_v vertices and about rec_bytes bytes, at least one round
                size_t r1 = r0;
                int nv = 0, ne = 0;
                while (r1 < ro.size()) {
                    const Round& r = rounds[(size_t)ro[r1]];
                    int dv = 0, de = 0;
                    for (const Item& it : r.it) if (!it.skip && !it.helper) { ++dv; de += ep[it.p + 1] - ep[it.p]; }
                    const long long bytes = 32 + 256LL * (long long)(r1 - r0 + 1) + 4LL * rec_v +
                                            (((long long)(nv + dv) * rtrow + 7) & ~7LL) + (long long)(ne + de) * ebytes;
                    if (r1 > r0 && (nv + dv > rec_v || bytes > rec_bytes)) break;
                    nv += dv; ne += de; ++r1;
                }
                const int nr = (int)(r1 - r0);
                const int rtoff = 32 + 256 * nr, eoff = rtoff + ((nv * rtrow + 7) & ~7);
                const long long bytes_ll = (long long)eoff + (long long)ne * ebytes;   // without the trailer
                if (bytes_ll > 60000 || nv > 4096) { fits = false; break; }   // edge offsets and one stage slot stay far below 64 KB
                const int bytes = (int)bytes_ll;
                const size_t base = raw.size();
                raw.resize(base + (size_t)bytes, 0);
                unsigned char* rec = raw.data() + base;
                int hdr[4] = {nr, rtoff, rtrow, bytes};
                memcpy(rec, hdr, 16);
                const int vfirst = (int)vlist.size();
                int vi = 0, ecur = eoff;
                for (int rr = 0; rr < nr; ++rr) {
                    const Round& r = rounds[(size_t)ro[r0 + (size_t)rr]];
                    int my_eb = 0;
                    for (int q = 0; q < 16; ++q) {
                        const Item& it = r.it[q];
                        int out[4] = {0, 0, 0, 0};
                        if (it.skip) { out[0] = (1 << 29) | (r.kind << 27); }
                        else {
                            const int p = it.p, v = order[p], d = ep[p + 1] - ep[p];
                            if (!it.helper) {
                                // the vertex' runtimes, id row and edges enter the record once
                                for (int c = 0; c < nsc; ++c) {
                                    const int rtv = (int)ceil_div(g->h_c[v], S, svals[(size_t)c]);
                                    memcpy(rec + rtoff + vi * rtrow + 4 * c, &rtv, 4);
                                }
                                vlist.push_back(v);
                                for (int e = 0; e < d; ++e) {
                                    unsigned char* er = rec + ecur + e * ebytes;
                                    const int u = nb[(size_t)ep[p] + e];
                                    const int us = qof[(size_t)u] % R;
                                    memcpy(er, &us, 4);
                                    for (int w = 1; w <= ncw; ++w) {
                                        const long long tr = ceil_div(tt[(size_t)ep[p] + e], S, wvals[(size_t)w - 1]);
                                        memcpy(er + 8 * w, &tr, 8);
                                    }
                                }
                                my_eb = ecur;
                                ecur += d * ebytes;
                                ++vi;
                            }
                            const bool cpflag = ep_other[p + 1] == ep_other[p];   // forward: sink; backward: source
                            out[0] = v | (r.kind << 27) | (it.helper ? 1 << 30 : 0) | (cpflag ? (int)0x80000000u : 0);
                            out[1] = (qof[(size_t)v] % R) | ((vi - 1) << 16);
                            out[2] = my_eb + it.e0 * ebytes;
                            out[3] = my_eb + it.e1 * ebytes;
                        }
                        memcpy(rec + 32 + 256 * rr + 16 * q, out, 16);
                    }
                }
                rec_base.push_back(base); rec_raw.push_back(bytes); rec_nv.push_back(nv); rec_vfirst.push_back(vfirst);
                rec_first.push_back(first ? 1 : 0);
                first = false;
                max_v = std::max(max_v, (nv + 1) & ~1);
                ++nrecords;
                r0 = r1;
            }
        }
        if (!fits || raw.size() / 8 >= ((size_t)1 << 31)) continue;
        // Record i carries, as its trailer, the descriptor and the vertex list of record i + depth (the record that takes
        // over its stage slot).  Stage slots: as many as fit beside the ring, at least three.
        int depth = 0;
        size_t smem = 0;
        for (int d = RING_DEPTH_MAX; d >= 3 && depth == 0; --d) {
            int rmax = 16;
            for (int i = 0; i < nrecords; ++i)
                rmax = std::max(rmax, (rec_raw[(size_t)i] + (i + d < nrecords ? 4 * rec_nv[(size_t)i + d] : 0) + 15) & ~15);
            const size_t need = ring_smem_bytes(R, rmax, max_v, d, KP);
            if (need + 1024 <= (size_t)g->smem_optin) { depth = d; smem = need; rec_max = rmax; }
        }
        if (depth == 0) continue;
        std::vector<size_t> off((size_t)nrecords + 1, 0);
        for (int i = 0; i < nrecords; ++i)
            off[(size_t)i + 1] = off[(size_t)i] + (size_t)((rec_raw[(size_t)i] + (i + depth < nrecords ? 4 * rec_nv[(size_t)i + depth] : 0) + 15) & ~15);
        if (off[(size_t)nrecords] / 16 >= ((size_t)1 << 31)) continue;
        blob.assign(off[(size_t)nrecords], 0);
        desc.assign(4 * ((size_t)nrecords + 1), 0);   // one zero descriptor past the end
        for (int i = 0; i < nrecords; ++i) {
            desc[4 * (size_t)i] = (int)(off[(size_t)i] / 16);
            desc[4 * (size_t)i + 1] = (int)(off[(size_t)i + 1] - off[(size_t)i]);
            desc[4 * (size_t)i + 2] = rec_nv[(size_t)i] | (rec_first[(size_t)i] ? (int)0x80000000u : 0);
            desc[4 * (size_t)i + 3] = rec_vfirst[(size_t)i];
        }
        for (int i = 0; i < nrecords; ++i) {
            unsigned char* rec = blob.data() + off[(size_t)i];
            memcpy(rec, raw.data() + rec_base[(size_t)i], (size_t)rec_raw[(size_t)i]);
            if (i + 1 < nrecords && rec_first[(size_t)i + 1]) {   // the next record opens a step
                int nr;
                memcpy(&nr, rec, 4);
                nr |= (int)0x80000000u;
                memcpy(rec, &nr, 4);
            }
            if (i + depth < nrecords) {
                memcpy(rec + 16, &desc[4 * ((size_t)i + depth)], 16);
                memcpy(rec + rec_raw[(size_t)i], &vlist[(size_t)rec_vfirst[(size_t)i + depth]], 4 * (size_t)rec_nv[(size_t)i + depth]);
            }
        }
        raw.clear(); raw.shrink_to_fit();
        std::vector<unsigned char> cls((size_t)KP * KP, 0), scv((size_t)KP, 0);
        for (int pv = 0; pv < k; ++pv) {
            scv[(size_t)pv] = (unsigned char)(4 * sc_of[pv]);
            for (int pu = 0; pu < k; ++pu)   // forward: the edge runs from the neighbour to the vertex; backward the other way
                cls[(size_t)pv * KP + pu] = (unsigned char)(pu == pv ? 0 : 8 * (cls_of(dir == 0 ? B[pu * k + pv] : B[pv * k + pu]) + 1));
        }
        TFPS_TRY(upload(L.blob, blob, st));
        TFPS_TRY(upload(L.desc, desc, st));
        TFPS_TRY(upload(L.vlist, vlist, st));
        TFPS_TRY(upload(L.cls, cls, st));
        TFPS_TRY(upload(L.sc, scv, st));
        CUDA_TRY(cudaStreamSynchronize(st));
        L.args = RingArgs{};
        L.args.blob = L.blob.as<unsigned char>();
        L.args.desc = L.desc.as<int4>();
        L.args.vlist = L.vlist.as<int>();
        L.args.cls = L.cls.as<unsigned char>();
        L.args.sc = L.sc.as<unsigned char>();
        L.args.num_records = nrecords;
        L.args.kp = KP;
        L.args.R = R;
        L.args.rec_max = rec_max;
        L.args.max_v = max_v;
        L.args.ebytes = ebytes;
        L.args.depth = depth;
        L.smem = smem;
        L.ok = true;
    }
    return TFPS_OK;
}

}  // namespace

extern "C" {

const char* tfps_strerror(int status)
{
    switch (status) {
        case TFPS_OK: return "ok";
        case TFPS_ERR_INVALID_ARG: return "invalid argument";
        case TFPS_ERR_BAD_CSR: return "malformed CSR";
        case TFPS_ERR_CYCLE: return "graph has a cycle";
        case TFPS_ERR_BAD_DEVICES: return "bad device tables";
        case TFPS_ERR_BAD_PARTITION: return "partition id out of range";
        case TFPS_ERR_OVERFLOW: return "possible 64-bit overflow";
        case TFPS_ERR_WORKSPACE: return "workspace missing or too small";
        case TFPS_ERR_UNSUPPORTED: return "size beyond implementation limit";
        case TFPS_ERR_CUDA: return "CUDA runtime error";
        case TFPS_ERR_TIMEOUT: return "device-side wait timed out";
        case TFPS_ERR_STATE: return "call order violated";
        default: return "unknown status";
    }
}

const char* tfps_last_error(void) { return g_last_error.c_str(); }

int tfps_graph_create(tfps_graph** out, int64_t n, int64_t m,
                      const int64_t* in_ptr, const int32_t* in_src, const void* in_t,
                      const int64_t* out_ptr, const int32_t* out_dst, const void* out_t,
                      int t_dtype, const int32_t* c, const void* mem, int mem_dtype,
                      int ptr_space, void* stream)
{
    if (!out) return fail(TFPS_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    cudaStream_t st = (cudaStream_t)stream;
    if (n < 0 || m < 0) return fail(TFPS_ERR_INVALID_ARG, "negative size");
    if (n >= ((int64_t)1 << 26) || m >= ((int64_t)1 << 31) - 64)
        return fail(TFPS_ERR_UNSUPPORTED, "n must be below 2^26 and m below 2^31");
    if (!in_ptr || (n > 0 && !c) || (m > 0 && (!in_src || !in_t)))
        return fail(TFPS_ERR_INVALID_ARG, "in_ptr, in_src, in_t and c are required");
    const bool have_out = out_ptr || out_dst || out_t;
    if (have_out && (!out_ptr || (m > 0 && (!out_dst || !out_t))))
        return fail(TFPS_ERR_INVALID_ARG, "pass all of out_ptr, out_dst, out_t or none");
    if ((t_dtype != TFPS_I32 && t_dtype != TFPS_I64) || (mem && mem_dtype != TFPS_I32 && mem_dtype != TFPS_I64))
        return fail(TFPS_ERR_INVALID_ARG, "bad dtype selector");
    if (ptr_space != TFPS_HOST && ptr_space != TFPS_DEVICE) return fail(TFPS_ERR_INVALID_ARG, "bad ptr_space");

    std::vector<long long> h_in_ptr, h_out_ptr, h_in_t, h_out_t, h_mem;
    std::vector<int> h_in_src, h_out_dst, h_c;
    TFPS_TRY(fetch(h_in_ptr, in_ptr, (size_t)n + 1, ptr_space, st));
    TFPS_TRY(fetch(h_in_src, in_src, (size_t)m, ptr_space, st));
    TFPS_TRY(fetch_wide(h_in_t, in_t, (size_t)m, t_dtype, ptr_space, st));
    TFPS_TRY(fetch(h_c, c, (size_t)n, ptr_space, st));
    TFPS_TRY(check_csr("in", n, m, h_in_ptr, h_in_src));

    tfps_graph* g = new (std::nothrow) tfps_graph();
    if (!g) return fail(TFPS_ERR_INVALID_ARG, "out of host memory");
    struct Holder { tfps_graph* g; ~Holder() { delete g; } } holder{g};

    for (long long v = 0; v < n; ++v) {
        if (h_c[v] < 0) return fail(TFPS_ERR_BAD_CSR, "negative cost c[%lld]", v);
        g->sum_c += (u128)h_c[v];
        g->max_c = std::max<long long>(g->max_c, h_c[v]);
    }
    for (long long e = 0; e < m; ++e) {
        if (h_in_t[e] < 0) return fail(TFPS_ERR_BAD_CSR, "negative edge size at in-edge %lld", e);
        g->sum_t += (u128)h_in_t[e];
        g->max_t = std::max(g->max_t, h_in_t[e]);
    }
    for (long long v = 0; v < n; ++v)
        for (long long e = h_in_ptr[v]; e < h_in_ptr[v + 1]; ++e)
            if (h_in_src[e] == v) return fail(TFPS_ERR_CYCLE, "self loop at vertex %lld", v);
    g->id_topo = true;
    for (long long v = 0; v < n && g->id_topo; ++v)
        for (long long e = h_in_ptr[v]; e < h_in_ptr[v + 1]; ++e) {
            if (h_in_src[e] >= v) { g->id_topo = false; break; }
            g->span_id = std::max(g->span_id, (int)(v - h_in_src[e]));
        }

    // out-CSR by transposing the in-CSR (rows come out sorted by target, then by in-row order)
    std::vector<long long> t_ptr((size_t)n + 1, 0), t_t((size_t)m);
    std::vector<int> t_dst((size_t)m);
    for (long long e = 0; e < m; ++e) t_ptr[(size_t)h_in_src[e] + 1]++;
    for (long long v = 0; v < n; ++v) t_ptr[v + 1] += t_ptr[v];
    {
        std::vector<long long> fill(t_ptr.begin(), t_ptr.end() - 1);
        for (long long v = 0; v < n; ++v)
            for (long long e = h_in_ptr[v]; e < h_in_ptr[v + 1]; ++e) {
                long long o = fill[h_in_src[e]]++;
                t_dst[o] = (int)v;
                t_t[o] = h_in_t[e];
            }
    }
    if (have_out) {
        TFPS_TRY(fetch(h_out_ptr, out_ptr, (size_t)n + 1, ptr_space, st));
        TFPS_TRY(fetch(h_out_dst, out_dst, (size_t)m, ptr_space, st));
        TFPS_TRY(fetch_wide(h_out_t, out_t, (size_t)m, t_dtype, ptr_space, st));
        TFPS_TRY(check_csr("out", n, m, h_out_ptr, h_out_dst));
        // both directions must describe the same multiset of (u, v, t)
        std::vector<std::pair<int, long long>> ra, rb;
        for (long long v = 0; v < n; ++v) {
            if (h_out_ptr[v + 1] - h_out_ptr[v] != t_ptr[v + 1] - t_ptr[v])
                return fail(TFPS_ERR_BAD_CSR, "out-degree of vertex %lld disagrees with the in-edge lists", v);
            ra.clear(); rb.clear();
            for (long long e = h_out_ptr[v]; e < h_out_ptr[v + 1]; ++e) ra.emplace_back(h_out_dst[e], h_out_t[e]);
            for (long long e = t_ptr[v]; e < t_ptr[v + 1]; ++e) rb.emplace_back(t_dst[e], t_t[e]);
            std::sort(ra.begin(), ra.end());
            std::sort(rb.begin(), rb.end());
            if (ra != rb) return fail(TFPS_ERR_BAD_CSR, "out-edges of vertex %lld disagree with the in-edge lists", v);
        }
    } else {
        h_out_ptr.swap(t_ptr);
        h_out_dst.swap(t_dst);
        h_out_t.swap(t_t);
    }
    if (mem) {
        TFPS_TRY(fetch_wide(h_mem, mem, (size_t)n, mem_dtype, ptr_space, st));
        u128 tot = 0;
        for (long long v = 0; v < n; ++v) {
            if (h_mem[v] < 0) return fail(TFPS_ERR_BAD_CSR, "negative memory at vertex %lld", v);
            tot += (u128)h_mem[v];
        }
        if (tot >= (u128)LIMIT62) return fail(TFPS_ERR_OVERFLOW, "sum of vertex memory reaches 2^62");
    } else if (g->sum_t >= (u128)LIMIT62) {
        return fail(TFPS_ERR_OVERFLOW, "sum of edge sizes reaches 2^62");
    }

    CUDA_TRY(cudaGetDevice(&g->device));
    CUDA_TRY(cudaDeviceGetAttribute(&g->sm_count, cudaDevAttrMultiProcessorCount, g->device));
    CUDA_TRY(cudaDeviceGetAttribute(&g->smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, g->device));
    g->n = n;
    g->m = m;
    TFPS_TRY(upload(g->in_ptr, h_in_ptr, st));
    TFPS_TRY(upload(g->in_src, h_in_src, st));
    TFPS_TRY(upload(g->in_t, h_in_t, st));
    TFPS_TRY(upload(g->out_ptr, h_out_ptr, st));
    TFPS_TRY(upload(g->out_dst, h_out_dst, st));
    TFPS_TRY(upload(g->out_t, h_out_t, st));
    TFPS_TRY(upload(g->c, h_c, st));
    if (mem) {
        TFPS_TRY(upload(g->mem, h_mem, st));
    } else {
        CUDA_TRY(g->mem.alloc(sizeof(long long) * (size_t)n));
        CUDA_TRY(launch_default_mem((int)n, g->out_ptr.as<long long>(), g->out_t.as<long long>(), g->mem.as<long long>(), st));
    }
    CUDA_TRY(g->status.alloc(sizeof(int)));
    CUDA_TRY(cudaMemsetAsync(g->status.p, 0, sizeof(int), st));
    CUDA_TRY(cudaStreamSynchronize(st));  // host vectors go out of scope
    g->h_in_ptr.swap(h_in_ptr);
    g->h_in_src.swap(h_in_src);
    g->h_in_t.swap(h_in_t);
    g->h_c.swap(h_c);
    holder.g = nullptr;
    *out = g;
    return TFPS_OK;
}

int tfps_graph_destroy(tfps_graph* g)
{
    if (!g) return TFPS_OK;
    {
        DeviceGuard guard(g->device);
        delete g;
    }
    return TFPS_OK;
}

int tfps_graph_info(const tfps_graph* g, int64_t* n, int64_t* m, int32_t* num_levels, int32_t* k)
{
    if (!g) return fail(TFPS_ERR_INVALID_ARG, "graph is NULL");
    if (n) *n = g->n;
    if (m) *m = g->m;
    if (num_levels) *num_levels = g->topo_built ? g->num_levels : 0;
    if (k) *k = g->dev_set ? g->k : 0;
    return TFPS_OK;
}

int tfps_devices_set(tfps_graph* g, int k, const int32_t* s, const int64_t* C, const int64_t* B, int64_t scale)
{
    if (!g) return fail(TFPS_ERR_INVALID_ARG, "graph is NULL");
    if (k < 1 || k > TFPS_K_MAX) return fail(TFPS_ERR_BAD_DEVICES, "k = %d outside 1..%d", k, (int)TFPS_K_MAX);
    if (!s || !C || !B) return fail(TFPS_ERR_INVALID_ARG, "s, C and B are required");
    if (scale < 1) return fail(TFPS_ERR_BAD_DEVICES, "scale must be >= 1");
    long long s_min = INT64_MAX, b_min = INT64_MAX;
    for (int d = 0; d < k; ++d) {
        if (s[d] < 1) return fail(TFPS_ERR_BAD_DEVICES, "speed s[%d] = %d < 1", d, s[d]);
        if (C[d] < 0) return fail(TFPS_ERR_BAD_DEVICES, "capacity C[%d] < 0", d);
        s_min = std::min<long long>(s_min, s[d]);
        for (int e = 0; e < k; ++e) {
            if (d == e) continue;
            long long b = B[d * k + e];
            if (b < 1) return fail(TFPS_ERR_BAD_DEVICES, "bandwidth B[%d][%d] = %lld < 1", d, e, b);
            if (b >= LIMIT62) return fail(TFPS_ERR_BAD_DEVICES, "bandwidth B[%d][%d] too large", d, e);
            b_min = std::min(b_min, b);
        }
    }
    // numerators c*S and t*S must stay below 2^62; so must every path length and load
    if ((u128)g->max_c * (u128)scale >= (u128)LIMIT62 || (u128)g->max_t * (u128)scale >= (u128)LIMIT62)
        return fail(TFPS_ERR_OVERFLOW, "c*scale or t*scale reaches 2^62");
    u128 bound = g->sum_c * (u128)scale / (u128)s_min + (u128)g->n;
    if (k > 1) bound += g->sum_t * (u128)scale / (u128)b_min + (u128)g->m;
    if (bound >= (u128)LIMIT62) return fail(TFPS_ERR_OVERFLOW, "a path length or load could reach 2^62 ticks");

    DeviceGuard guard(g->device);
    if (!guard.ok) return fail(TFPS_ERR_CUDA, "cannot select the handle's device");
    cudaStream_t st = 0;
    TFPS_TRY(build_topo(g, st));

    std::vector<DivConst> rt((size_t)k), w((size_t)k * k);
    for (int d = 0; d < k; ++d) rt[d] = make_div((unsigned long long)s[d]);
    for (int a = 0; a < k; ++a)
        for (int b = 0; b < k; ++b) {
            if (a == b) { w[a * k + b] = DivConst{0ull, 0u, 0u}; continue; }
            w[a * k + b] = make_div((unsigned long long)B[a * k + b]);
        }
    std::vector<long long> cap(C, C + k);
    g->dev_set = false;
    // pair tables and value classes for the per-edge cost table
    g->npass = k <= TABLE_K_MAX ? (k * k + 31) / 32 : 0;
    g->use_cls = 0;
    g->ncls_w = 0;
    if (g->npass > 0) {
        const int ent = g->npass * 32;
        std::vector<DivConst> pf((size_t)ent), pb((size_t)ent), cls(32, DivConst{0ull, 0u, 0u});
        std::vector<unsigned short> sf((size_t)ent), sb((size_t)ent);
        std::vector<long long> wvals, svals;  // distinct off-diagonal bandwidths, distinct speeds
        auto cls_of = [](std::vector<long long>& vals, long long x) {
            for (size_t i = 0; i < vals.size(); ++i)
                if (vals[i] == x) return (int)i;
            vals.push_back(x);
            return (int)vals.size() - 1;
        };
        for (int a = 0; a < k; ++a)
            for (int b = 0; b < k; ++b)
                if (a != b) cls_of(wvals, B[a * k + b]);
        for (int d = 0; d < k; ++d) cls_of(svals, s[d]);
        const bool use_cls = wvals.size() + svals.size() <= 32;
        const int ncw = (int)wvals.size();
        for (int i = 0; i < ent; ++i) {
            const bool real = i < k * k;
            const int nb = real ? i / k : 0, vv = real ? i % k : 0;
            const bool diag = !real || nb == vv;
            pf[i] = diag ? DivConst{0ull, 0u, 0u} : make_div((unsigned long long)B[nb * k + vv]);
            pb[i] = diag ? DivConst{0ull, 0u, 0u} : make_div((unsigned long long)B[vv * k + nb]);
            pf[i].pad = (unsigned)nb | (diag ? 256u : 0u);
            pb[i].pad = (unsigned)vv | (diag ? 256u : 0u);
            if (use_cls) {
                const int cwf = diag ? 255 : cls_of(wvals, B[nb * k + vv]);
                const int cwb = diag ? 255 : cls_of(wvals, B[vv * k + nb]);
                sf[i] = (unsigned short)(cwf | ((ncw + cls_of(svals, s[nb])) << 8));
                sb[i] = (unsigned short)(cwb | ((ncw + cls_of(svals, s[vv])) << 8));
            } else {
                sf[i] = sb[i] = 255;
            }
        }
        if (use_cls) {
            for (int c = 0; c < ncw; ++c) cls[c] = make_div((unsigned long long)wvals[c]);
            for (size_t c = 0; c < svals.size(); ++c) cls[ncw + c] = make_div((unsigned long long)svals[c]);
        }
        g->use_cls = use_cls ? 1 : 0;
        g->ncls_w = ncw;
        TFPS_TRY(upload(g->pair_f, pf, st));
        TFPS_TRY(upload(g->pair_b, pb, st));
        TFPS_TRY(upload(g->cls_div, cls, st));
        TFPS_TRY(upload(g->sel_f, sf, st));
        TFPS_TRY(upload(g->sel_b, sb, st));

    }
    TFPS_TRY(upload(g->rt_div, rt, st));
    TFPS_TRY(upload(g->w_div, w, st));
    TFPS_TRY(upload(g->cap, cap, st));
    const int n = (int)g->n, m = (int)g->m;
    CUDA_TRY(g->xvert.reserve(sizeof(unsigned long long) * (size_t)n));
    CUDA_TRY(g->xw_f.reserve(sizeof(unsigned long long) * (size_t)m));
    CUDA_TRY(g->xnbr_f.reserve(sizeof(unsigned long long) * (size_t)m));
    CUDA_TRY(g->xw_b.reserve(sizeof(unsigned long long) * (size_t)m));
    if (n > 0)
        CUDA_TRY(launch_numerators(n, m, scale, g->order.as<int>(), g->c.as<int>(), g->f_nbr.as<int>(),
                                   g->f_t.as<long long>(), g->b_nbr.as<int>(), g->b_t.as<long long>(),
                                   g->xvert.as<unsigned long long>(), g->xw_f.as<unsigned long long>(),
                                   g->xnbr_f.as<unsigned long long>(), g->xw_b.as<unsigned long long>(), st));
    g->rt_kp = 0;
    if (n > 0 && k <= 32) {
        int kp = 2;   // at least two entries: rows of the table start on 16-byte boundaries
        while (kp < k) kp <<= 1;
        CUDA_TRY(g->rtv.reserve(sizeof(long long) * (size_t)n * kp));
        CUDA_TRY(launch_rt_rows(n, k, kp, g->pos_of.as<int>(), g->xvert.as<unsigned long long>(), g->rt_div.as<DivConst>(),
                                g->rtv.as<long long>(), st));
        g->rt_kp = kp;
    }
    g->fits32 = false;
    for (auto& L : g->lean) L.ok = false;
    if (n > 0) {
        // worst-case critical path: every vertex on the slowest device, every edge over the slowest link
        std::vector<int> order((size_t)n);
        CUDA_TRY(cudaMemcpyAsync(order.data(), g->order.p, sizeof(int) * (size_t)n, cudaMemcpyDeviceToHost, st));
        CUDA_TRY(cudaStreamSynchronize(st));
        std::vector<long long> fin((size_t)n);
        long long worst = 0;
        for (int i = 0; i < n; ++i) {
            const int v = order[i];
            long long start = 0;
            for (long long e = g->h_in_ptr[v]; e < g->h_in_ptr[v + 1]; ++e) {
                const long long w = k > 1 ? (long long)(((u128)g->h_in_t[e] * (u128)scale + (u128)b_min - 1) / (u128)b_min) : 0;
                start = std::max(start, fin[g->h_in_src[e]] + w);
            }
            fin[v] = start + (long long)(((u128)g->h_c[v] * (u128)scale + (u128)s_min - 1) / (u128)s_min);
            worst = std::max(worst, fin[v]);
        }
        g->fits32 = worst < (1LL << 31) - 1;
        TFPS_TRY(build_lean(g, k, s, B, scale, order, st));
        TFPS_TRY(build_levrec(g, k, s, B, scale, order, st));
        TFPS_TRY(build_ring(g, k, s, B, scale, order, st));
    }
    CUDA_TRY(cudaStreamSynchronize(st));
    if (!g->aux_stream) {
        int lo = 0, hi = 0;
        CUDA_TRY(cudaDeviceGetStreamPriorityRange(&lo, &hi));   // lo = least priority
        CUDA_TRY(cudaStreamCreateWithPriority(&g->aux_stream, cudaStreamNonBlocking, lo));
        CUDA_TRY(cudaEventCreateWithFlags(&g->aux_fork, cudaEventDisableTiming));
        CUDA_TRY(cudaEventCreateWithFlags(&g->aux_join, cudaEventDisableTiming));
        CUDA_TRY(cudaStreamCreateWithFlags(&g->pass2_stream, cudaStreamNonBlocking));
        CUDA_TRY(cudaEventCreateWithFlags(&g->pass2_join, cudaEventDisableTiming));
    }
    if (g->device >= 0 && g->device < 128) {
        void* scratch = nullptr;   // resolve the built-in scratch of tfps_eval_cp_noalloc now, not in the evaluation call
        CUDA_TRY(noalloc_scratch_address(g->device, &scratch));
    }
    g->k = k;
    g->S = scale;
    {
        std::vector<int> speed(s, s + k), ord((size_t)k);
        for (int d = 0; d < k; ++d) ord[d] = d;
        std::stable_sort(ord.begin(), ord.end(), [&](int a, int b) { return s[a] > s[b]; });   // equal speeds: lower index first
        TFPS_TRY(upload(g->speed_d, speed, st));
        TFPS_TRY(upload(g->ord_d, ord, st));
        std::vector<long long> bw(B, B + (size_t)k * k);
        for (int d = 0; d < k; ++d) bw[(size_t)d * k + d] = 1;   // the diagonal is never used as a divisor
        TFPS_TRY(upload(g->bw_d, bw, st));
        CUDA_TRY(cudaStreamSynchronize(st));
    }
    g->dev_set = true;
    return TFPS_OK;
}

int tfps_topo_levels(tfps_graph* g, int32_t* level, int32_t* order, int64_t* level_ptr, int64_t cap,
                     int32_t* num_levels, void* stream)
{
    if (!g) return fail(TFPS_ERR_INVALID_ARG, "graph is NULL");
    DeviceGuard guard(g->device);
    if (!guard.ok) return fail(TFPS_ERR_CUDA, "cannot select the handle's device");
    cudaStream_t st = (cudaStream_t)stream;
    TFPS_TRY(build_topo(g, st));
    if (num_levels) *num_levels = g->num_levels;
    if (level_ptr) {
        if (cap < (int64_t)g->num_levels + 1)
            return fail(TFPS_ERR_INVALID_ARG, "level_ptr has room for %lld entries, %d needed", (long long)cap, g->num_levels + 1);
        for (int l = 0; l <= g->num_levels; ++l) level_ptr[l] = g->h_level_ptr[l];
    }
    if (g->n > 0) {
        if (level) CUDA_TRY(cudaMemcpyAsync(level, g->level.p, sizeof(int) * (size_t)g->n, cudaMemcpyDeviceToDevice, st));
        if (order) CUDA_TRY(cudaMemcpyAsync(order, g->order.p, sizeof(int) * (size_t)g->n, cudaMemcpyDeviceToDevice, st));
    }
    CUDA_TRY(cudaStreamSynchronize(st));
    return TFPS_OK;
}

size_t tfps_eval_workspace_bytes(const tfps_graph* g, int64_t P, int64_t ldp, int flags)
{
    if (!g || P <= 0 || ldp < P) return 0;
    if (flags & TFPS_EVAL_SCRATCH_LEVELS) return sizeof(long long) * (size_t)g->n * (size_t)ldp;
    return 0;
}

int tfps_eval_batch(tfps_graph* g, int64_t P, int64_t ldp, const uint8_t* part, int64_t* tlevel, int64_t* blevel,
                    int64_t* cp, int64_t* load, int64_t* memload, uint64_t* viol, void* workspace,
                    size_t workspace_bytes, int flags, void* stream)
{
    if (!g) return fail(TFPS_ERR_INVALID_ARG, "graph is NULL");
    if (P < 0 || ldp < P || (ldp % 16) != 0) return fail(TFPS_ERR_INVALID_ARG, "need 0 <= P <= ldp and ldp %% 16 == 0");
    if ((flags & TFPS_EVAL_LEVEL_SYNC) && (flags & TFPS_EVAL_SLICED))
        return fail(TFPS_ERR_INVALID_ARG, "choose one kernel variant");
    if (!g->dev_set) return fail(TFPS_ERR_STATE, "tfps_devices_set has not been called");
    if (P == 0 || g->n == 0) return TFPS_OK;
    if (!part) return fail(TFPS_ERR_INVALID_ARG, "part is NULL");
    if (P > ((int64_t)1 << 31)) return fail(TFPS_ERR_UNSUPPORTED, "P above 2^31");
    {
        // the kernels read ids and read and write levels as 16-byte vectors: refuse anything else before any launch
        const void* ptrs[] = {part, tlevel, blevel, cp, load, memload, viol};
        const char* names[] = {"part", "tlevel", "blevel", "cp", "load", "memload", "viol"};
        for (int i = 0; i < 7; ++i)
            if (((uintptr_t)ptrs[i] & 15u) != 0)
                return fail(TFPS_ERR_INVALID_ARG, "%s must be 16-byte aligned", names[i]);
    }

    DeviceGuard guard(g->device);
    if (!guard.ok) return fail(TFPS_ERR_CUDA, "cannot select the handle's device");
    cudaStream_t st = (cudaStream_t)stream;
    TFPS_TRY(build_topo(g, st));

    const bool need_bwd = blevel != nullptr;
    const bool need_fwd = tlevel != nullptr || (cp != nullptr && !need_bwd);
    long long* fwd_lev = (long long*)tlevel;
    if (need_fwd && !tlevel) {
        const size_t need = sizeof(long long) * (size_t)g->n * (size_t)ldp;
        if (!workspace || workspace_bytes < need)
            return fail(TFPS_ERR_WORKSPACE, "workspace of %zu bytes needed for the level scratch, %zu given", need, workspace_bytes);
        if (((uintptr_t)workspace & 255u) != 0) return fail(TFPS_ERR_WORKSPACE, "workspace must be 256-byte aligned");
        fwd_lev = (long long*)workspace;
    }
    const bool validate = !(flags & TFPS_EVAL_NO_VALIDATE);
    const int n = (int)g->n;
    const int k = g->k;
    const DevTables tab = make_tables(g);
    int* status = g->status.as<int>();

    const bool profile = (flags & TFPS_EVAL_PROFILE) != 0;
    if (profile) {
        for (cudaEvent_t& e : g->ev)
            if (!e) CUDA_TRY(cudaEventCreate(&e));
        g->ev_valid = false;
        CUDA_TRY(cudaEventRecord(g->ev[0], st));
    }

    long long* ml = (long long*)memload;
    if (viol && !ml) {
        CUDA_TRY(g->scr_memload.reserve(sizeof(long long) * (size_t)k * (size_t)ldp));
        ml = g->scr_memload.as<long long>();
    }
    // loads, memory loads, violation flags and the id check, on stream `ls`
    auto run_loads = [&](cudaStream_t ls) -> int {
        if (load || ml) {
            if (load) CUDA_TRY(cudaMemset2DAsync(load, sizeof(long long) * (size_t)ldp, 0, sizeof(long long) * (size_t)P, (size_t)k, ls));
            if (ml) CUDA_TRY(cudaMemset2DAsync(ml, sizeof(long long) * (size_t)ldp, 0, sizeof(long long) * (size_t)P, (size_t)k, ls));
            if (g->rt_kp > 0 && ((uintptr_t)part & 3u) == 0 && env_int("TFPS_LOADS2", 1) != 0)
                CUDA_TRY(launch_loads2(n, P, ldp, part, g->rtv.as<long long>(), g->mem.as<long long>(), k, g->rt_kp,
                                       (long long*)load, ml, status, validate, g->sm_count, g->smem_optin, ls));
            else
                CUDA_TRY(launch_loads(n, P, ldp, part, g->order.as<int>(), g->xvert.as<unsigned long long>(), g->mem.as<long long>(),
                                      tab, (long long*)load, ml, status, validate, g->sm_count, ls));
            if (viol) CUDA_TRY(launch_viol(P, ldp, k, ml, tab.cap, (unsigned long long*)viol, status, ls));
        } else if (validate) {
            CUDA_TRY(launch_validate(n, P, ldp, part, k, status, g->sm_count, ls));
        }
        return TFPS_OK;
    };

    // kernel variant
    bool sliced;
    if (flags & TFPS_EVAL_SLICED) sliced = true;
    else if (flags & TFPS_EVAL_LEVEL_SYNC) sliced = false;
    else {
        // enough candidate slices to occupy the machine, or levels too narrow to be worth a launch each
        const long long avg_width = g->num_levels > 0 ? g->n / g->num_levels : g->n;
        sliced = (P >= 32LL * g->sm_count) || (avg_width * P < (1LL << 18));
    }
    // shape of the sliced kernel: candidates per lane and warps per block (overridable for tuning).
    // Wider lanes amortise the per-edge cost table over more candidates; keep enough slices to fill the SMs.
    const bool table = env_int("TFPS_SLICED_TABLE", 1) != 0;
    int cpt = env_int("TFPS_SLICED_CPT", 0);
    if (cpt != 1 && cpt != 2 && cpt != 4 && cpt != 8) {
        cpt = 1;
        if (table && g->npass > 0)
            for (int c = 4; c > 1; c >>= 1)
                if ((P + 32 * c - 1) / (32 * c) >= (3LL * g->sm_count) / 4) { cpt = c; break; }
    }
    int warps = env_int("TFPS_SLICED_WARPS", 0);
    if (warps < 1 || warps > 32) {
        const long long avg_width = g->num_levels > 0 ? g->n / g->num_levels : g->n;
        warps = 4;
        while (warps < 32 && warps < avg_width) warps <<= 1;
    }

    const int level_bytes = (g->fits32 && env_int("TFPS_LEVEL32", 1) != 0) ? 4 : 8;
    // Lean windowed pass (32-bit levels, whole window resident, host-packed records): block shape for one direction.
    struct LeanChoice { bool ok = false; int slice = 0, cpt = 4, warps = 0; size_t smem = 0; LeanArgs args; };
    auto pick_lean = [&](bool fwd) {
        LeanChoice ch;
        if (!(sliced && g->lean[0].ok && g->lean[1].ok && ((uintptr_t)part & 15u) == 0 && ldp < (1LL << 28) &&
              env_int("TFPS_LEAN", 1) != 0))
            return ch;
        const LeanPlan& lp = g->lean[fwd ? 0 : 1].plan;
        if (!lp.wide && level_bytes != 4) return ch;
        // the wide kernel can run blocks of 8 or 16 candidates, but a block that narrow is bound by the latency of a
        // record and measured slower than the level-synchronous kernels: only on request (TFPS_LEAN_SLICE)
        const int forced_slice = env_int("TFPS_LEAN_SLICE", 0);
        const int slice_min = lp.wide ? ((forced_slice == 8 || forced_slice == 16) ? forced_slice : 32) : 16;
        // candidates per block (slice): the widest that keeps the window in shared memory and leaves enough
        // blocks to occupy the machine; TFPS_LEAN_SLICE (or TFPS_SLICED_CPT = c for 32*c) forces one
        const int forced = env_int("TFPS_SLICED_CPT", 0);
        const long long want_slices = std::min<long long>((3LL * g->sm_count) / 4, (P + slice_min - 1) / slice_min);
        int d_want = env_int("TFPS_LEAN_DEPTH", 0);
        if (d_want < 1 || d_want > LEAN_DEPTH_MAX) d_want = 3;
        const int forced_warps = env_int("TFPS_SLICED_WARPS", 0);
        for (int slice = 128; slice >= slice_min && !ch.ok; slice >>= 1) {
            if (forced_slice == 8 || forced_slice == 16 || forced_slice == 32 || forced_slice == 64 || forced_slice == 128) {
                if (slice != std::max(forced_slice, slice_min)) continue;
            }
            else if (forced == 1 || forced == 2 || forced == 4) { if (slice != 32 * forced) continue; }
            else if ((P + slice - 1) / slice < want_slices && slice > slice_min) continue;
            // candidates per lane of the narrow kernel: 4; 2 where the levels are narrow and the slices small, so that a
            // level's dependent chain is shorter (config 4: 8.75 against 9.69 ms per step); TFPS_LEAN_CPT forces 1, 2 or 4
            int cpt = 4;
            if (!lp.wide) {
                if (lp.max_sub <= 32 && slice <= 32) cpt = 2;
                const int want_cpt = env_int("TFPS_LEAN_CPT", 0);
                if ((want_cpt == 1 && slice <= 32) || (want_cpt == 2 && slice <= 64) || want_cpt == 4) cpt = want_cpt;
            }
            const int vpw = 32 * cpt / slice, pr = std::max(1, slice / 16);
            // warps: one round of the vertex groups covers the widest chunk, up to 16 warps (512 threads with up to
            // 128 registers each measured faster than 1024 threads with 64: 2.95 against 3.21 ms on config 3)
            int w = 1;
            while (w < 16 && w * vpw < lp.max_sub) w <<= 1;
            const int wmax = lp.wide ? 16 : 32;   // the wide kernel is built for at most 512 threads
            if (forced_warps >= 1 && forced_warps <= wmax) w = forced_warps;
            while (w < wmax && lp.max_v * pr > 2 * w * 32) w <<= 1;   // a thread fetches at most two id-row pieces per record
            if (lp.max_v * pr > 2 * w * 32) continue;
            for (int d = d_want; d >= 1; --d) {
                unsigned slot_stride = 0, stage_bytes = 0;
                const size_t need = lean_smem_bytes(lp, slice, w, d, &slot_stride, &stage_bytes);
                if (need + 1024 <= (size_t)g->smem_optin) {
                    ch.ok = true; ch.slice = slice; ch.cpt = cpt; ch.warps = w; ch.smem = need;
                    ch.args.slot_stride = slot_stride;
                    ch.args.stage_bytes = stage_bytes;
                    ch.args.depth = d;
                    break;
                }
            }
        }
        if (ch.ok) {
            ch.args.part = part;
            ch.args.status = status;
            ch.args.P = P;
            ch.args.ldp = ldp;
            ch.args.plan = lp;
            ch.args.wait_limit = std::max(0, env_int("TFPS_WAIT_LIMIT", 1 << 20));
        }
        return ch;
    };
    LeanChoice lean_f, lean_b;
    if (need_fwd) lean_f = pick_lean(true);
    if (need_bwd) lean_b = pick_lean(false);
    // Automatic choice: a graph whose window does not fit (no lean pass) but whose levels are wide is better served
    // by the level-synchronous record pass than by a sliced kernel that reads its neighbours through L2.
    if (!(flags & (TFPS_EVAL_SLICED | TFPS_EVAL_LEVEL_SYNC)) && sliced && !((!need_fwd || lean_f.ok) && (!need_bwd || lean_b.ok)) &&
        g->levrec[0].ok && g->levrec[1].ok && env_int("TFPS_LEVREC", 1) != 0) {
        const long long avg_width = g->num_levels > 0 ? g->n / g->num_levels : g->n;
        // a level costs the record pass about 8 us however few candidates there are, a vertex costs a sliced kernel
        // without a resident window about 0.07 us: levels of more than a hundred vertices favour the record pass at
        // any P (1,590 levels of 660: 12.8 against 76.6 ms forward at P = 64), narrower ones only with enough candidates
        if (avg_width * P >= (1LL << 18) || avg_width >= 128) { sliced = false; lean_f.ok = false; lean_b.ok = false; }
    }
    // Ring pass: where no lean pass applies, the ring fits and there are enough blocks of eight candidates for the machine
    // (TFPS_RING = 2: whenever it fits; 0: never).
    const bool use_ring = !(flags & (TFPS_EVAL_SLICED | TFPS_EVAL_LEVEL_SYNC)) && env_int("TFPS_RING", 1) != 0 &&
                          !((!need_fwd || lean_f.ok) && (!need_bwd || lean_b.ok)) && g->ring[0].ok && g->ring[1].ok &&
                          ldp < (1LL << 28) && ((P + RING_SLICE - 1) / RING_SLICE >= g->sm_count || env_int("TFPS_RING", 1) == 2);
    if (use_ring) { lean_f.ok = false; lean_b.ok = false; }
    // The lean passes cannot leave their tables on a bad id (ids are masked), so the id check need not come first:
    // the loads kernel then runs on a low-priority stream beside them and fills the SMs the passes' last wave leaves idle.
    const bool overlap = (load || ml) && (need_fwd || need_bwd) && (!need_fwd || lean_f.ok) && (!need_bwd || lean_b.ok) &&
                         g->aux_stream && env_int("TFPS_OVERLAP_LOADS", 1) != 0;
    // Both lean passes only read the ids and write their own level matrix: the backward pass then runs on a second
    // stream beside the forward pass, so that the blocks of both fill the machine together (config 3: 2 x 256 blocks
    // are 3.5 waves of 148 instead of 2 x 2).  Not with phase timing, which brackets the passes on one stream.
    const bool overlap_passes = overlap && need_fwd && need_bwd && !profile && g->pass2_stream && env_int("TFPS_OVERLAP_PASSES", 1) != 0;
    if (!overlap) TFPS_TRY(run_loads(st));   // loads first: the same kernel checks the ids, and a bad id stops everything after it
    else {
        CUDA_TRY(cudaEventRecord(g->aux_fork, st));
        CUDA_TRY(cudaStreamWaitEvent(g->aux_stream, g->aux_fork, 0));
    }
    if (profile) CUDA_TRY(cudaEventRecord(g->ev[1], st));
    for (int pass = 0; pass < 2; ++pass) {
        const bool fwd = pass == 0;
        if (profile && !fwd) CUDA_TRY(cudaEventRecord(g->ev[2], st));
        if (fwd ? !need_fwd : !need_bwd) continue;
        long long* lev = fwd ? fwd_lev : (long long*)blevel;
        long long* cp_here = (cp && (fwd || !need_fwd)) ? (long long*)cp : nullptr;
        PassArgs a = make_args(g, fwd, P, ldp, part, lev, cp_here);
        g->last_kernel = sliced ? "pass_sliced_kernel" : "pass_level_kernel";
        {
            LeanChoice& ch = fwd ? lean_f : lean_b;
            if (ch.ok) {
                ch.args.lev = lev;
                ch.args.cp = cp_here;
                g->last_kernel = ch.args.plan.wide ? "pass_lean64_kernel" : "pass_lean_kernel";
                cudaStream_t ps = st;
                if (overlap_passes && !fwd) {
                    ps = g->pass2_stream;
                    CUDA_TRY(cudaStreamWaitEvent(ps, g->aux_fork, 0));
                }
                if (ch.args.plan.wide) CUDA_TRY(launch_pass_lean64(ch.args, fwd, ch.slice, ch.warps, ch.smem, ps));
                else CUDA_TRY(launch_pass_lean(ch.args, fwd, ch.slice, ch.cpt, ch.warps, ch.smem, ps));
                if (overlap_passes && !fwd) CUDA_TRY(cudaEventRecord(g->pass2_join, ps));
                if (overlap && (overlap_passes ? !fwd : fwd == need_fwd)) {
                    // the first pass is queued: now the loads, so that the pass gets the machine first
                    TFPS_TRY(run_loads(g->aux_stream));
                    CUDA_TRY(cudaEventRecord(g->aux_join, g->aux_stream));
                }
                continue;
            }
        }
        if (use_ring) {   // wide graph with a long window and enough candidates: blocks of eight candidates with a ring in shared memory
            tfps_graph::Ring& L = g->ring[fwd ? 0 : 1];
            RingArgs ra = L.args;
            ra.part = part;
            ra.lev = lev;
            ra.cp = cp_here;
            ra.status = status;
            ra.P = P;
            ra.ldp = ldp;
            ra.wait_limit = std::max(0, env_int("TFPS_WAIT_LIMIT", 1 << 20));
            g->last_kernel = "pass_ring_kernel";
            CUDA_TRY(launch_pass_ring(ra, fwd, std::max(1, std::min(31, env_int("TFPS_RING_WARPS", 16))), L.smem, st));
            continue;
        }
        if (sliced) {
            SlicedPlan plan;
            plan.vertf = g->vertf.as<int>();
            plan.chunks = fwd ? g->f_chunks.as<int>() : g->b_chunks.as<int>();
            plan.num_chunks = fwd ? g->f_num_chunks : g->b_num_chunks;
            plan.src_end = (int)g->h_level_ptr[1];
            CUDA_TRY(launch_pass_sliced(a, fwd, plan, cpt, warps, table, st));
        } else {
            {
                {
                    const int dirn = fwd ? 0 : 1;
                    const bool rec = g->levrec[dirn].ok && env_int("TFPS_LEVREC", 1) != 0;
                    if (rec) {   // vertex records (k <= 64): no divisions or per-edge tables in the kernel
                        tfps_graph::LevRec& L = g->levrec[dirn];
                        if (L.heavy_count > 0) CUDA_TRY(launch_zero_rows(L.heavy.as<int>(), L.heavy_count, P, ldp, lev, st));
                        LevRecArgs la = L.args;
                        la.part = part;
                        la.lev = lev;
                        la.status = status;
                        la.P = P;
                        la.ldp = ldp;
                        la.groups = std::max(1, std::min((int)STEPREC_GROUPS_MAX, env_int("TFPS_STEP_GROUPS", 2)));
                        la.tiles_per_group = std::max(1, env_int("TFPS_STEP_TILES", 8));
                        la.tiles_per_run = std::max(1, env_int("TFPS_STEP_RUN", 4));
                        la.blocks_per_sm = std::max(0, env_int("TFPS_STEP_BLOCKS", 0));
                        la.wait_limit = std::max(0, env_int("TFPS_WAIT_LIMIT", 1 << 20));
                        la.shape = env_int("TFPS_STEP_SHAPE", 0);
                        // One launch per step by default; the persistent form (one cooperative launch, barriers between
                        // the steps inside the kernel) measured slower at every batch width (config 5, forward pass: 14.4
                        // against 10.1 ms at P = 256, 18.9 against 16.0 at 1,024, 33.8 against 29.4 at 4,096) and is opt-in.
                        if (env_int("TFPS_STEP_FLOW", 0) == 1 && flow_applies(la)) {
                            g->last_kernel = "pass_flow_kernel";
                            CUDA_TRY(launch_pass_flow(la, fwd, g->sm_count, st));
                        } else if (env_int("TFPS_STEP_PERSISTENT", 0) == 1) {
                            g->last_kernel = "pass_steprec_kernel";
                            CUDA_TRY(launch_pass_steprec(la, fwd, g->sm_count, st));
                        } else {
                            g->last_kernel = "pass_stepchain_kernel";
                            CUDA_TRY(launch_pass_stepchain(la, fwd, L.h_step_ptr, st));
                        }
                    } else {   // runtimes beyond int32 or more than 255 distinct bandwidths: division per relaxation
                        CUDA_TRY(launch_pass_level_sync(a, fwd, g->h_level_ptr, st));
                    }
                }
            }
            if (cp_here) {
                CUDA_TRY(cudaMemsetAsync(cp_here, 0, sizeof(long long) * (size_t)P, st));
                if (fwd) CUDA_TRY(launch_cp_reduce(a, true, g->sink_list.as<int>(), g->sink_count, st));
                else CUDA_TRY(launch_cp_reduce(a, false, nullptr, (int)g->h_level_ptr[1], st));
            }
        }
    }
    if (overlap) CUDA_TRY(cudaStreamWaitEvent(st, g->aux_join, 0));
    if (overlap_passes) CUDA_TRY(cudaStreamWaitEvent(st, g->pass2_join, 0));
    if (profile) {
        CUDA_TRY(cudaEventRecord(g->ev[3], st));
        g->ev_valid = true;
        g->ran_fwd = need_fwd;
        g->ran_bwd = need_bwd;
    }
    return TFPS_OK;
}

int tfps_phase_times(tfps_graph* g, float ms[3])
{
    if (!g || !ms) return fail(TFPS_ERR_INVALID_ARG, "graph or ms is NULL");
    if (!g->ev_valid) return fail(TFPS_ERR_STATE, "no profiled tfps_eval_batch call to report");
    DeviceGuard guard(g->device);
    if (!guard.ok) return fail(TFPS_ERR_CUDA, "cannot select the handle's device");
    CUDA_TRY(cudaEventSynchronize(g->ev[3]));
    for (int i = 0; i < 3; ++i) CUDA_TRY(cudaEventElapsedTime(&ms[i], g->ev[i], g->ev[i + 1]));
    if (!g->ran_fwd) ms[1] = 0.f;
    if (!g->ran_bwd) ms[2] = 0.f;
    return TFPS_OK;
}

const char* tfps_last_pass_kernel(const tfps_graph* g) { return g ? g->last_kernel : ""; }

int64_t tfps_kernel_launches(void) { return (int64_t)tfps::g_launches.load(std::memory_order_relaxed); }


int tfps_eval_cp_noalloc(tfps_graph* g, int64_t P, int64_t ldp, const uint8_t* part, int64_t* cp, int flags,
                         void* stream)
{
    if (!g) return fail(TFPS_ERR_INVALID_ARG, "graph is NULL");
    if (P < 0 || ldp < P || (ldp % 16) != 0) return fail(TFPS_ERR_INVALID_ARG, "need 0 <= P <= ldp and ldp %% 16 == 0");
    if (!g->dev_set) return fail(TFPS_ERR_STATE, "tfps_devices_set has not been called");
    if (P == 0 || g->n == 0) return TFPS_OK;
    if (!part || !cp) return fail(TFPS_ERR_INVALID_ARG, "part and cp are required");
    const unsigned __int128 need = (unsigned __int128)g->n * (unsigned __int128)ldp * 8u;
    if (need > (unsigned __int128)TFPS_NOALLOC_SCRATCH_BYTES)
        return fail(TFPS_ERR_WORKSPACE, "n*ldp*8 = %llu bytes of level scratch needed, the built-in array holds %zu; "
                    "use tfps_eval_batch with a caller workspace", (unsigned long long)need, (size_t)TFPS_NOALLOC_SCRATCH_BYTES);
    if (g->device < 0 || g->device >= 128) return fail(TFPS_ERR_UNSUPPORTED, "device ordinal %d out of range", g->device);
    DeviceGuard guard(g->device);
    if (!guard.ok) return fail(TFPS_ERR_CUDA, "cannot select the handle's device");
    void* scratch = nullptr;
    CUDA_TRY(noalloc_scratch_address(g->device, &scratch));   // cached by tfps_devices_set on this device
    return tfps_eval_batch(g, P, ldp, part, nullptr, nullptr, cp, nullptr, nullptr, nullptr, scratch,
                           TFPS_NOALLOC_SCRATCH_BYTES, flags & ~TFPS_EVAL_PROFILE, stream);
}

int tfps_constraints_set(tfps_graph* g, int64_t npairs, const int32_t* pair_a, const int32_t* pair_b,
                         int64_t ndev, const int32_t* dc_vertex, const int32_t* dc_device)
{
    if (!g) return fail(TFPS_ERR_INVALID_ARG, "graph is NULL");
    if (npairs < 0 || ndev < 0 || npairs > INT32_MAX || ndev > INT32_MAX) return fail(TFPS_ERR_INVALID_ARG, "bad list length");
    if ((npairs > 0 && (!pair_a || !pair_b)) || (ndev > 0 && (!dc_vertex || !dc_device)))
        return fail(TFPS_ERR_INVALID_ARG, "a non-empty list needs both of its arrays");
    for (int64_t i = 0; i < npairs; ++i)
        if (pair_a[i] < 0 || pair_a[i] >= g->n || pair_b[i] < 0 || pair_b[i] >= g->n)
            return fail(TFPS_ERR_INVALID_ARG, "collocation pair %lld names a vertex outside 0..n-1", (long long)i);
    for (int64_t i = 0; i < ndev; ++i)
        if (dc_vertex[i] < 0 || dc_vertex[i] >= g->n || dc_device[i] < 0 || dc_device[i] >= (int)TFPS_K_MAX)
            return fail(TFPS_ERR_INVALID_ARG, "device constraint %lld names a vertex outside 0..n-1 or a device outside 0..%d",
                        (long long)i, (int)TFPS_K_MAX - 1);
    DeviceGuard guard(g->device);
    if (!guard.ok) return fail(TFPS_ERR_CUDA, "cannot select the handle's device");
    cudaStream_t st = 0;
    g->cons_pairs = g->cons_dev = 0;
    TFPS_TRY(upload(g->cons_a, std::vector<int>(pair_a, pair_a + npairs), st));
    TFPS_TRY(upload(g->cons_b, std::vector<int>(pair_b, pair_b + npairs), st));
    TFPS_TRY(upload(g->cons_v, std::vector<int>(dc_vertex, dc_vertex + ndev), st));
    TFPS_TRY(upload(g->cons_d, std::vector<int>(dc_device, dc_device + ndev), st));
    CUDA_TRY(cudaStreamSynchronize(st));
    g->cons_pairs = (int)npairs;
    g->cons_dev = (int)ndev;
    return TFPS_OK;
}

int tfps_eval_constraints(tfps_graph* g, int64_t P, int64_t ldp, const uint8_t* part, int32_t* coll_viol, int32_t* dev_viol,
                          void* stream)
{
    if (!g) return fail(TFPS_ERR_INVALID_ARG, "graph is NULL");
    if (P < 0 || ldp < P || (ldp % 16) != 0) return fail(TFPS_ERR_INVALID_ARG, "need 0 <= P <= ldp and ldp %% 16 == 0");
    if (P == 0 || g->n == 0 || (!coll_viol && !dev_viol)) return TFPS_OK;
    if (!part) return fail(TFPS_ERR_INVALID_ARG, "part is NULL");
    if (P > ((int64_t)1 << 31)) return fail(TFPS_ERR_UNSUPPORTED, "P above 2^31");
    if (((uintptr_t)part & 15u) != 0 || ((uintptr_t)coll_viol & 3u) != 0 || ((uintptr_t)dev_viol & 3u) != 0)
        return fail(TFPS_ERR_INVALID_ARG, "part must be 16-byte aligned, the outputs 4-byte aligned");
    DeviceGuard guard(g->device);
    if (!guard.ok) return fail(TFPS_ERR_CUDA, "cannot select the handle's device");
    CUDA_TRY(launch_constraints(P, ldp, part, g->cons_pairs, g->cons_a.as<int>(), g->cons_b.as<int>(), g->cons_dev,
                                g->cons_v.as<int>(), g->cons_d.as<int>(), coll_viol, dev_viol, g->status.as<int>(),
                                (cudaStream_t)stream));
    return TFPS_OK;
}

int tfps_critical_mask(int64_t n, int64_t P, int64_t ldp, const int64_t* tlevel, const int64_t* blevel, const int64_t* cp,
                       uint8_t* mask, void* stream)
{
    if (n < 0 || P < 0 || ldp < P || (ldp % 16) != 0) return fail(TFPS_ERR_INVALID_ARG, "need n >= 0, 0 <= P <= ldp and ldp %% 16 == 0");
    if (n == 0 || P == 0) return TFPS_OK;
    if (!tlevel || !blevel || !cp || !mask) return fail(TFPS_ERR_INVALID_ARG, "tlevel, blevel, cp and mask are required");
    if ((((uintptr_t)tlevel | (uintptr_t)blevel | (uintptr_t)mask | (uintptr_t)cp) & 15u) != 0)
        return fail(TFPS_ERR_INVALID_ARG, "tlevel, blevel, cp and mask must be 16-byte aligned");
    CUDA_TRY(launch_critical_mask(n, P, ldp, (const long long*)tlevel, (const long long*)blevel, (const long long*)cp, mask,
                                  (cudaStream_t)stream));
    return TFPS_OK;
}

int tfps_ranks(tfps_graph* g, int64_t* up, int64_t* down, int64_t* total, void* stream)
{
    if (!g) return fail(TFPS_ERR_INVALID_ARG, "graph is NULL");
    DeviceGuard guard(g->device);
    if (!guard.ok) return fail(TFPS_ERR_CUDA, "cannot select the handle's device");
    cudaStream_t st = (cudaStream_t)stream;
    TFPS_TRY(build_topo(g, st));
    if (g->n == 0) return TFPS_OK;
    // a rank is at most the sum of all costs, which tfps_graph_create has bounded; the total rank at most twice that
    if (g->sum_c >= (u128)(LIMIT62 / 2)) return fail(TFPS_ERR_OVERFLOW, "a total rank could reach 2^62");
    const size_t bytes = sizeof(long long) * (size_t)g->n;
    if (!up) { CUDA_TRY(g->rank_up.reserve(bytes)); up = g->rank_up.as<int64_t>(); }
    if (!down) { CUDA_TRY(g->rank_down.reserve(bytes)); down = g->rank_down.as<int64_t>(); }
    CUDA_TRY(launch_ranks((int)g->n, g->h_level_ptr, g->order.as<int>(), g->in_ptr.as<long long>(), g->in_src.as<int>(),
                          g->out_ptr.as<long long>(), g->out_dst.as<int>(), g->c.as<int>(), (long long*)up, (long long*)down,
                          (long long*)total, st));
    return TFPS_OK;
}

int tfps_critical_path(tfps_graph* g, const int64_t* down, int32_t* path, int64_t* len, void* stream)
{
    if (!g || !len) return fail(TFPS_ERR_INVALID_ARG, "graph and len are required");
    *len = 0;
    if (g->n == 0) return TFPS_OK;
    if (!down || !path) return fail(TFPS_ERR_INVALID_ARG, "down and path are required");
    DeviceGuard guard(g->device);
    if (!guard.ok) return fail(TFPS_ERR_CUDA, "cannot select the handle's device");
    cudaStream_t st = (cudaStream_t)stream;
    CUDA_TRY(g->part_scr.reserve(sizeof(long long) * 4));
    CUDA_TRY(launch_critical_path((int)g->n, g->in_ptr.as<long long>(), g->in_src.as<int>(), g->out_ptr.as<long long>(),
                                  (const long long*)down, path, g->part_scr.as<long long>(), st));
    long long h = 0;
    CUDA_TRY(cudaMemcpyAsync(&h, g->part_scr.as<long long>() + 2, sizeof(long long), cudaMemcpyDeviceToHost, st));
    CUDA_TRY(cudaStreamSynchronize(st));
    *len = h;
    return TFPS_OK;
}

int tfps_batch_split(tfps_graph* g, const int64_t* total, uint8_t* part, int64_t* unplaced, void* stream)
{
    if (!g || !unplaced) return fail(TFPS_ERR_INVALID_ARG, "graph and unplaced are required");
    *unplaced = 0;
    if (!g->dev_set) return fail(TFPS_ERR_STATE, "tfps_devices_set has not been called");
    if (g->n == 0) return TFPS_OK;
    if (!total || !part) return fail(TFPS_ERR_INVALID_ARG, "total and part are required");
    DeviceGuard guard(g->device);
    if (!guard.ok) return fail(TFPS_ERR_CUDA, "cannot select the handle's device");
    cudaStream_t st = (cudaStream_t)stream;
    int npad = 1;
    while (npad < g->n) npad <<= 1;
    CUDA_TRY(g->part_idx.reserve(sizeof(int) * (size_t)npad));
    CUDA_TRY(g->part_scr.reserve(sizeof(long long) * 4));
    long long* d_unplaced = g->part_scr.as<long long>() + 3;
    CUDA_TRY(launch_batch_split((int)g->n, npad, g->k, (const long long*)total, g->mem.as<long long>(), g->ord_d.as<int>(),
                                g->cap.as<long long>(), g->part_idx.as<int>(), part, d_unplaced, st));
    long long h = 0;
    CUDA_TRY(cudaMemcpyAsync(&h, d_unplaced, sizeof(long long), cudaMemcpyDeviceToHost, st));
    CUDA_TRY(cudaStreamSynchronize(st));
    *unplaced = h;
    return TFPS_OK;
}

int tfps_cp_partition(tfps_graph* g, const int32_t* path, int64_t len, uint8_t* part, int64_t* unplaced, void* stream)
{
    if (!g || !unplaced) return fail(TFPS_ERR_INVALID_ARG, "graph and unplaced are required");
    *unplaced = 0;
    if (!g->dev_set) return fail(TFPS_ERR_STATE, "tfps_devices_set has not been called");
    if (len < 0 || len > g->n) return fail(TFPS_ERR_INVALID_ARG, "need 0 <= len <= n");
    if (g->n == 0) return TFPS_OK;
    if (!part || (len > 0 && !path)) return fail(TFPS_ERR_INVALID_ARG, "part (and path when len > 0) are required");
    DeviceGuard guard(g->device);
    if (!guard.ok) return fail(TFPS_ERR_CUDA, "cannot select the handle's device");
    cudaStream_t st = (cudaStream_t)stream;
    CUDA_TRY(g->part_flag.reserve((size_t)g->n));
    CUDA_TRY(g->part_scr.reserve(sizeof(long long) * 4));
    long long* d_unplaced = g->part_scr.as<long long>() + 3;
    CUDA_TRY(launch_cp_partition((int)g->n, g->k, g->S, path, len, g->c.as<int>(), g->mem.as<long long>(),
                                 g->speed_d.as<int>(), g->ord_d.as<int>(), g->cap.as<long long>(),
                                 g->part_flag.as<uint8_t>(), part, d_unplaced, st));
    long long h = 0;
    CUDA_TRY(cudaMemcpyAsync(&h, d_unplaced, sizeof(long long), cudaMemcpyDeviceToHost, st));
    CUDA_TRY(cudaStreamSynchronize(st));
    *unplaced = h;
    return TFPS_OK;
}

int tfps_msr_weights_set(tfps_graph* g, int64_t alpha, int64_t beta, int64_t gamma, int64_t delta)
{
    if (!g) return fail(TFPS_ERR_INVALID_ARG, "graph is NULL");
    const int64_t w[4] = {alpha, beta, gamma, delta};
    for (int i = 0; i < 4; ++i)
        if (w[i] < 0 || w[i] > (1LL << 20)) return fail(TFPS_ERR_INVALID_ARG, "MSR weights must lie in 0 .. 2^20");
    for (int i = 0; i < 4; ++i) g->msr_w[i] = w[i];
    return TFPS_OK;
}

int tfps_simulate(tfps_graph* g, int64_t P, int64_t ldp, const uint8_t* part, int policy, const int64_t* prio,
                  int64_t* start, int64_t* makespan, void* stream)
{
    if (!g) return fail(TFPS_ERR_INVALID_ARG, "graph is NULL");
    if (P < 0 || ldp < P) return fail(TFPS_ERR_INVALID_ARG, "need 0 <= P <= ldp");
    if (policy != TFPS_SCHED_FIFO && policy != TFPS_SCHED_PCT && policy != TFPS_SCHED_MSR) return fail(TFPS_ERR_INVALID_ARG, "unknown scheduling policy %d", policy);
    if (!g->dev_set) return fail(TFPS_ERR_STATE, "tfps_devices_set has not been called");
    if (P == 0) return TFPS_OK;
    if (!makespan) return fail(TFPS_ERR_INVALID_ARG, "makespan is required");
    if (policy == TFPS_SCHED_PCT && !prio && g->n > 0) return fail(TFPS_ERR_INVALID_ARG, "the PCT policy needs the path computation times (blevel)");
    DeviceGuard guard(g->device);
    if (!guard.ok) return fail(TFPS_ERR_CUDA, "cannot select the handle's device");
    cudaStream_t st = (cudaStream_t)stream;
    if (g->n == 0) {   // nothing to execute: every schedule ends at 0
        CUDA_TRY(cudaMemsetAsync(makespan, 0, sizeof(int64_t) * (size_t)P, st));
        return TFPS_OK;
    }
    if (!part) return fail(TFPS_ERR_INVALID_ARG, "part is required");
    // one warp per candidate in flight; its scratch is 16 bytes per vertex, kept below 8 GB in all
    const int wpb = simulate_warps_per_block();
    long long warps = std::min<long long>((P + wpb - 1) / wpb * wpb, (long long)g->sm_count * 32);
    warps = std::min(warps, std::max<long long>(wpb, ((8LL << 30) / (16LL * g->n)) / wpb * wpb));
    const int blocks = (int)(warps / wpb);
    CUDA_TRY(g->sim_ready.reserve(sizeof(long long) * (size_t)warps * (size_t)g->n));
    CUDA_TRY(g->sim_left.reserve(sizeof(int) * (size_t)warps * (size_t)g->n));
    CUDA_TRY(g->sim_list.reserve(sizeof(int) * (size_t)warps * (size_t)g->n));
    CUDA_TRY(launch_simulate((int)g->n, g->k, P, ldp, g->S, part, g->in_ptr.as<long long>(), g->out_ptr.as<long long>(),
                             g->out_dst.as<int>(), g->out_t.as<long long>(), g->c.as<int>(), g->speed_d.as<int>(),
                             g->bw_d.as<long long>(), policy, (const long long*)prio, g->msr_w, (long long*)start,
                             (long long*)makespan, blocks, g->sim_ready.as<long long>(), g->sim_left.as<int>(), g->sim_list.as<int>(),
                             g->status.as<int>(), st));
    return TFPS_OK;
}

int tfps_get_status(tfps_graph* g, void* stream)
{
    if (!g) return fail(TFPS_ERR_INVALID_ARG, "graph is NULL");
    DeviceGuard guard(g->device);
    if (!guard.ok) return fail(TFPS_ERR_CUDA, "cannot select the handle's device");
    cudaStream_t st = (cudaStream_t)stream;
    int h = 0;
    CUDA_TRY(cudaMemcpyAsync(&h, g->status.p, sizeof(int), cudaMemcpyDeviceToHost, st));
    CUDA_TRY(cudaStreamSynchronize(st));
    if (h != 0) {
        CUDA_TRY(cudaMemsetAsync(g->status.p, 0, sizeof(int), st));
        CUDA_TRY(cudaStreamSynchronize(st));
        return fail(h, "device-side status: %s", tfps_strerror(h));
    }
    return TFPS_OK;
}

int tfps_eval_batch_host(tfps_graph* g, int64_t P, int64_t ldp, const uint8_t* part, int64_t* tlevel,
                         int64_t* blevel, int64_t* cp, int64_t* load, int64_t* memload, uint64_t* viol, int flags,
                         void* stream)
{
    if (!g) return fail(TFPS_ERR_INVALID_ARG, "graph is NULL");
    if (P < 0 || ldp < P || (ldp % 16) != 0) return fail(TFPS_ERR_INVALID_ARG, "need 0 <= P <= ldp and ldp %% 16 == 0");
    if (!g->dev_set) return fail(TFPS_ERR_STATE, "tfps_devices_set has not been called");
    if (P == 0 || g->n == 0) return TFPS_OK;
    if (!part) return fail(TFPS_ERR_INVALID_ARG, "part is NULL");
    DeviceGuard guard(g->device);
    if (!guard.ok) return fail(TFPS_ERR_CUDA, "cannot select the handle's device");
    cudaStream_t st = (cudaStream_t)stream;
    const int k = g->k;
    // Candidates are independent: the id matrix goes up in column chunks on a copy stream (two staging buffers) and
    // every chunk is evaluated as soon as it has landed, so the transfer of chunk c+1 overlaps the evaluation of
    // chunk c; results come back per chunk.  A chunk must still fill the GPU (one wave of blocks of the sliced kernel
    // is 64 candidates per SM) and rows shorter than 4 KiB copy far below the link rate, so chunks are as wide as the
    // scratch allows: the two level matrices of a chunk (int64 [n][width] each) are kept below 2 x 36 GB.
    int nchunks = P >= 128LL * g->sm_count * 3 / 4 ? 2 : 1;
    long long width = (P + nchunks - 1) / nchunks;
    const long long cap = std::max<long long>(128, ((36LL << 30) / (8LL * std::max<long long>(1, g->n))) / 128 * 128);
    width = std::min(width, cap);
    width = (width + 127) / 128 * 128;   // whole candidate slices per chunk
    if (width >= ldp) width = ldp;
    nchunks = (int)((P + width - 1) / width);
    const size_t ccells = (size_t)g->n * (size_t)width;
    const size_t kcells = (size_t)k * (size_t)width;
    CUDA_TRY(g->st_part.reserve(ccells * (nchunks > 1 ? 2 : 1)));
    CUDA_TRY(g->st_lev.reserve(ccells * 8));
    CUDA_TRY(g->st_lev2.reserve(ccells * 8));
    CUDA_TRY(g->st_cp.reserve((size_t)width * 8));
    if (load) CUDA_TRY(g->st_load.reserve(kcells * 8));
    if (memload || viol) CUDA_TRY(g->st_mem.reserve(kcells * 8));
    if (viol) CUDA_TRY(g->st_viol.reserve((size_t)width * 8));
    if (nchunks > 1) {
        if (!g->copy_stream) CUDA_TRY(cudaStreamCreateWithFlags(&g->copy_stream, cudaStreamNonBlocking));
        for (int c = 0; c < 4; ++c)
            if (!g->copy_ev[c]) CUDA_TRY(cudaEventCreateWithFlags(&g->copy_ev[c], cudaEventDisableTiming));
        // the staging buffers may still be in use by earlier work on the caller's stream
        CUDA_TRY(cudaEventRecord(g->copy_ev[2], st));
        CUDA_TRY(cudaStreamWaitEvent(g->copy_stream, g->copy_ev[2], 0));
    }
    for (int c = 0; c < nchunks; ++c) {
        const long long j0 = (long long)c * width;
        const long long w = std::min<long long>(width, P - j0);
        const long long wl = std::min<long long>(width, ldp - j0);   // bytes per row to copy: whole 16-byte pieces
        uint8_t* dpart = g->st_part.as<uint8_t>() + (size_t)(c & 1) * ccells;
        if (nchunks > 1) {
            // buffer c & 1 was last read by the evaluation of chunk c - 2
            if (c >= 2) CUDA_TRY(cudaStreamWaitEvent(g->copy_stream, g->copy_ev[3], 0));
            CUDA_TRY(cudaMemcpy2DAsync(dpart, (size_t)width, part + j0, (size_t)ldp, (size_t)wl, (size_t)g->n,
                                       cudaMemcpyHostToDevice, g->copy_stream));
            CUDA_TRY(cudaEventRecord(g->copy_ev[c & 1], g->copy_stream));
            CUDA_TRY(cudaStreamWaitEvent(st, g->copy_ev[c & 1], 0));
        } else {
            CUDA_TRY(cudaMemcpy2DAsync(dpart, (size_t)width, part, (size_t)ldp, (size_t)wl, (size_t)g->n, cudaMemcpyHostToDevice, st));
        }
        TFPS_TRY(tfps_eval_batch(g, w, width, dpart, g->st_lev.as<int64_t>(), g->st_lev2.as<int64_t>(), g->st_cp.as<int64_t>(),
                                 load ? g->st_load.as<int64_t>() : nullptr, (memload || viol) ? g->st_mem.as<int64_t>() : nullptr,
                                 viol ? g->st_viol.as<uint64_t>() : nullptr, nullptr, 0, flags, st));
        if (nchunks > 1 && c + 2 < nchunks) CUDA_TRY(cudaEventRecord(g->copy_ev[3], st));   // chunk c + 1 runs between: one event suffices
        // results of the chunk: strided copies into the caller's [.][ldp] arrays
        const size_t wb = (size_t)w * 8;
        if (tlevel) CUDA_TRY(cudaMemcpy2DAsync(tlevel + j0, (size_t)ldp * 8, g->st_lev.p, (size_t)width * 8, wb, (size_t)g->n, cudaMemcpyDeviceToHost, st));
        if (blevel) CUDA_TRY(cudaMemcpy2DAsync(blevel + j0, (size_t)ldp * 8, g->st_lev2.p, (size_t)width * 8, wb, (size_t)g->n, cudaMemcpyDeviceToHost, st));
        if (cp) CUDA_TRY(cudaMemcpyAsync(cp + j0, g->st_cp.p, wb, cudaMemcpyDeviceToHost, st));
        if (load) CUDA_TRY(cudaMemcpy2DAsync(load + j0, (size_t)ldp * 8, g->st_load.p, (size_t)width * 8, wb, (size_t)k, cudaMemcpyDeviceToHost, st));
        if (memload) CUDA_TRY(cudaMemcpy2DAsync(memload + j0, (size_t)ldp * 8, g->st_mem.p, (size_t)width * 8, wb, (size_t)k, cudaMemcpyDeviceToHost, st));
        if (viol) CUDA_TRY(cudaMemcpyAsync(viol + j0, g->st_viol.p, wb, cudaMemcpyDeviceToHost, st));
    }
    return tfps_get_status(g, stream);
}

int tfps_transpose_u8(const uint8_t* src, uint8_t* dst, int64_t P, int64_t n, int64_t ldp, void* stream)
{
    if (P < 0 || n < 0 || ldp < P) return fail(TFPS_ERR_INVALID_ARG, "need 0 <= P <= ldp, n >= 0");
    if (P == 0 || n == 0) return TFPS_OK;
    if (!src || !dst) return fail(TFPS_ERR_INVALID_ARG, "src and dst are required");
    if ((P + 63) / 64 > 65535) return fail(TFPS_ERR_UNSUPPORTED, "P above 64*65535");
    CUDA_TRY(launch_transpose_u8(src, dst, P, n, ldp, (cudaStream_t)stream));
    return TFPS_OK;
}

}  // extern "C"
