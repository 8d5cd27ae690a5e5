// Internal declarations shared by the translation units of libtfps.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <string>
#include <vector>

#include "tfps.h"

namespace tfps {

// ---------------------------------------------------------------------------
// Exact division by an invariant divisor d >= 1 for numerators x < 2^62:
//   floor(x / d) == umul64hi(mul, x << 2) >> sh
// with  sh = ceil(log2 d)  and  mul = ceil(2^(62+sh) / d)   (mul <= 2^63).
// Proof sketch: mul*d = 2^(62+sh) + e with 0 <= e < d <= 2^sh, so
// mul*x / 2^(62+sh) = x/d + x*e/(d*2^(62+sh)) and the excess is < 1/d, too
// small to carry the quotient over the next integer.
//
// A ceiling quotient of a positive numerator a is taken as 1 + floor((a-1)/d);
// the library stores numerators already in the form X = (a-1) << 2, with the
// reserved value NUM_ZERO standing for a == 0 (quotient 0).
// ---------------------------------------------------------------------------
struct DivConst {
    unsigned long long mul;
    unsigned int sh;
    unsigned int pad;
};
static_assert(sizeof(DivConst) == 16, "DivConst is loaded as one 16-byte word");

constexpr unsigned long long NUM_ZERO = ~0ull;

#ifdef __CUDACC__
// ceil(a/d) for the stored numerator X = (a-1)<<2 of a positive a
__device__ __forceinline__ long long ceil_quot(unsigned long long X, const DivConst& dc)
{
    return 1 + (long long)(__umul64hi(dc.mul, X) >> dc.sh);
}
#endif

// Device tables set by tfps_devices_set (global memory; kernels stage them in
// shared memory).  rt_div[d] divides by s_d, w_div[a*k+b] by B[a][b].
//
// Pair tables for the per-edge cost table of the sliced pass (k <= TABLE_K_MAX):
// entry i = nb*k + vv pairs the neighbour's device nb with the vertex's device
// vv.  pair_f[i] divides by B[nb][vv] (forward: edge neighbour -> vertex),
// pair_b[i] by B[vv][nb] (backward: edge vertex -> neighbour).  Both are padded
// to npass*32 entries; DivConst::pad holds  dev | diag << 8  where dev is the
// device whose speed enters the entry (nb forward, vv backward) and diag marks
// nb == vv or a padding entry (transfer cost 0).
//
// When the off-diagonal bandwidths and the speeds take at most 32 distinct
// values together ("classes"), cls_div[c] holds one divisor per class (transfer
// classes first, then ncls_w.. the speed classes) and sel_f/sel_b[i] = cw | cr << 8
// name the transfer class (255 = none) and the speed class lane of entry i.
constexpr int TABLE_K_MAX = 16;

struct DevTables {
    int k;
    const DivConst* rt_div;  // [k]
    const DivConst* w_div;   // [k*k]
    const long long* cap;    // [k]
    int npass;               // ceil(k*k/32) when k <= TABLE_K_MAX, else 0
    int use_cls;             // classes available
    int ncls_w;              // number of transfer classes
    const DivConst* pair_f;  // [npass*32]
    const DivConst* pair_b;  // [npass*32]
    const DivConst* cls_div; // [32]
    const unsigned short* sel_f;  // [npass*32]
    const unsigned short* sel_b;  // [npass*32]
};

// Level-ordered adjacency of one direction.  Position i runs over vertices
// sorted by (level, id); FWD lists in-edges, BWD out-edges.
struct LevelAdj {
    const int* vert;                 // [n]   vertex at position i
    const int* eptr;                 // [n+1] edge offsets by position
    const int* nbr;                  // [m]   neighbour vertex id
    const unsigned long long* xw;    // [m]   transfer numerator ((t*S-1)<<2 or NUM_ZERO)
    const unsigned long long* xnbr;  // [m]   neighbour's runtime numerator ((c*S-1)<<2 or NUM_ZERO)
    const unsigned long long* xvert; // [n]   own runtime numerator by position
};

struct PassArgs {
    LevelAdj adj;
    DevTables tab;
    const long long* level_ptr;  // [L+1] device copy
    int num_levels;
    int n;
    long long P, ldp;
    const uint8_t* part;
    long long* lev;       // [n][ldp] levels written by this pass
    long long* cp;        // [P] or NULL
    int* status;          // sticky status word
};

// Chunking of the candidate-sliced pass: a chunk is a run of positions inside one
// level with at most CHUNK_V vertices and CHUNK_E edges (a single vertex with more
// edges forms a chunk of its own and is read straight from global memory).
constexpr int CHUNK_V = 128;
constexpr int CHUNK_E = 320;

struct SlicedPlan {
    const int* vertf;    // [n] vertex id by position, bit 31 set for sinks
    const int* chunks;   // [num_chunks][4] = {first position, vertices, first edge, edges}
    int num_chunks;
    int src_end;         // positions below this are sources (level 0)
};

// Lean windowed pass (32-bit levels, k <= LEAN_K_MAX, whole window resident).  The host packs, per direction
// and in processing order, records of one or more consecutive chunks (a chunk = mutually independent vertices of
// one level; narrow levels share a record, so a deep narrow graph pays the staging once per several levels):
//   header  LEAN_HDR_BYTES: int4 {chunks, byte offset of the edge area, vertices, 0}, then the descriptors
//           {offset/16, bytes, vertices, first index into vlist} of the records 1..LEAN_DEPTH_MAX places later
//           (zero past the end), then per chunk {first vertex within the record, vertices}
//   vertex  [vstride bytes each]  {v | flag << 31, window slot, first edge byte, end edge byte, rt[KP]}
//           flag: sink (forward) / source (backward): the vertex enters the CP maximum;
//           rt[d] = ceil(c_v*S / s_d); edge bytes are relative to the edge area
//   edge    [estride bytes each]  {window slot of the neighbour, W[0] = 0, W[1..ncls]}
//           W[c] = ceil(t_e*S / b_c) for the c-th distinct off-diagonal bandwidth b_c
// rows[pv] holds, in byte pu, 4 * (class of the link between a neighbour on device pu and a vertex on device
// pv; 0 = same device), so one byte permute turns the neighbour's id into the offset of W inside the edge record.
// The window keeps finish times (forward) or bottom levels (backward), so an edge adds the transfer term only.
constexpr int LEAN_K_MAX = 8;
constexpr int LEAN_CLS_MAX = 30;     // 4 * (classes + 1) must stay below 0x80 (sign-replicating byte permute)
constexpr int LEAN_CHUNK_V = 128;
constexpr int LEAN_DEPTH_MAX = 4;
constexpr int LEAN_SUB_MAX = 16;      // chunks per record
constexpr int LEAN_HDR_BYTES = 16 + 16 * LEAN_DEPTH_MAX + 8 * LEAN_SUB_MAX;

struct LeanPlan {
    const unsigned char* blob;   // chunk records, 16-byte aligned each
    const int4* desc;            // [num_chunks + 2*LEAN_DEPTH_MAX] {offset/16, bytes, vertices, first index into vlist}; zero padded
    const int* vlist;            // [n] vertex ids in processing order
    int num_chunks;              // records
    int vstride, estride;
    int R;                       // window length in positions (power of two)
    int rec_max;                 // largest record, bytes (multiple of 16)
    int max_v;                   // most vertices in one record
    int max_sub;                 // most vertices in one chunk
    unsigned long long rows[LEAN_K_MAX];
    // wide plan (pass_lean64_kernel: int64 levels, k <= LEAN64_K_MAX): vertex records carry rt[16] (int32), edge
    // records {window slot, pad, W[0..ncls] as int64}; rows16[pv*2 + h] holds, in byte pu - 8h, 8 * class
    int wide;
    unsigned long long rows16[2 * 16];
};
constexpr int LEAN64_K_MAX = 16;

struct LeanArgs {
    const uint8_t* part;
    long long* lev;
    long long* cp;
    int* status;
    long long P, ldp;
    LeanPlan plan;
    int depth;                   // chunks in flight (stage slots)
    unsigned slot_stride;        // bytes of a stage slot: rec_max + max_v * (candidates per block)
    unsigned stage_bytes;        // bytes reserved for all stage slots (also the CP reduction buffer)
    int wait_limit;              // polls before a wait for a stage gives up (TFPS_ERR_TIMEOUT)
};

// Persistent step-synchronous pass on host-packed vertex records (levrec.cu).
struct LevRecArgs {
    const uint8_t* part;
    long long* lev;
    int* status;
    long long P, ldp;
    const unsigned char* blob;   // records, 16-byte aligned
    const int4* items;           // work items {vertex | partial << 31, record offset / 16, first edge within the record, end edge},
                                 // step by step in processing order
    const int* step_ptr;         // [num_steps + 1] first item of every step
    int num_steps;
    int max_step_items;          // most items in one step
    const unsigned char* cls;    // [kp * kp] byte [pu * kp + pv] = cost combination of a neighbour on pu and a vertex on pv
    unsigned* bar;               // one counter per phase, 128 bytes apart (zeroed by the launcher)
    int kp;                      // device table width: 16 or 64
    int estride;                 // bytes of an edge entry (multiple of 16)
    int wbytes;                  // bytes of the cost values of an edge entry: 8 * combinations
    int rtu;                     // forward records carry the neighbour's runtimes separately (too many combinations)
    int rec_max;                 // bytes of the largest item: header, runtimes and its edges
    int groups;                  // phases (column groups) of a walk
    int tiles_per_group;         // tiles of a phase
    int tiles_per_run;           // consecutive tiles of a phase a warp evaluates for one item
    int blocks_per_sm;           // 0: as many as fit
    int wait_limit;              // polls before a barrier wait gives up
    int shape;                   // block shape variant (tuning)
    // dataflow form (flow.cu)
    unsigned* flags;             // [num_vertices] ready bits of every vertex, one per candidate tile (zeroed by the launcher)
    int* part_cnt;               // [num_heavy][32] finished partial items per vertex cut into several and tile (zeroed by the launcher)
    const int2* item_aux;        // [num_items] partial items: {index of the vertex among the cut ones, number of its items}
    int num_items, num_vertices, num_heavy;
};
constexpr int STEPREC_GROUPS_MAX = 4;
cudaError_t launch_pass_steprec(const LevRecArgs& a, bool fwd, int sm_count, cudaStream_t st);
cudaError_t launch_pass_stepchain(const LevRecArgs& a, bool fwd, const std::vector<int>& step_ptr_host, cudaStream_t st);
bool flow_applies(const LevRecArgs& a);   // the dataflow form covers k <= 16, items of at most eight edges of at most 64 bytes, P <= 4096
cudaError_t launch_pass_flow(const LevRecArgs& a, bool fwd, int sm_count, cudaStream_t st);

// Ring pass (ring.cu): candidate-sliced pass for wide graphs whose window is long.  A block owns RING_SLICE
// candidates and keeps the finish times (forward) or bottom levels (backward) and the ids of the last R vertices in
// processing order in shared memory.  The host packs records (never across a step boundary; a step = vertices that do
// not depend on one another) in processing order:
//   header  16 bytes: int4 {rounds, byte offset of the runtime table, bytes of a runtime row, 0}
//   rounds  64 bytes each: four items int4 {v | skip << 29 | wide << 30 | cp << 31, ring slot | index within the
//           record << 16, first edge byte, end edge byte}; one warp takes a round, eight lanes an item; the four items
//           of a wide round are quarters of the edges of one vertex and meet through shuffles
//   runtime [4 * nsc bytes per vertex of the record]  rt[c] = ceil(c_v * S / speed of class c)
//   edge    [8 + 8 * ncls bytes each]  {ring slot of the neighbour, pad, W[1..ncls]}, W[c] = ceil(t_e * S / b_c)
// desc[i] = {offset / 16, bytes, vertices | new step << 31, first index into vlist}; vlist names the vertices whose id
// rows go with the record.  cls[pv * kp + pu] = 8 * class of the link between the neighbour's device pu and the
// vertex's device pv (0 = same device); sc[d] = 4 * speed class of device d.
constexpr int RING_SLICE = 8;
constexpr int RING_DEPTH_MAX = 8;
constexpr int RING_CLS_MAX = 30;
struct RingArgs {
    const uint8_t* part;
    long long* lev;
    long long* cp;
    int* status;
    long long P, ldp;
    const unsigned char* blob;
    const int4* desc;            // [num_records + 1], zero past the end
    const int* vlist;
    const unsigned char* cls;    // [kp * kp]
    const unsigned char* sc;     // [kp]
    int num_records;
    int kp;                      // 16 or 64
    int R;                       // ring length in vertices
    int rec_max;                 // bytes of the largest record (multiple of 16)
    int max_v;                   // most vertices in one record
    int ebytes;                  // bytes of an edge entry
    int depth;                   // stage slots
    int wait_limit;
};
size_t ring_smem_bytes(int R, int rec_max, int max_v, int depth, int kp);
cudaError_t launch_pass_ring(const RingArgs& a, bool fwd, int warps, size_t smem, cudaStream_t st);

size_t lean_smem_bytes(const LeanPlan& plan, int slice, int warps, int depth, unsigned* slot_stride, unsigned* stage_bytes);
cudaError_t launch_pass_lean(const LeanArgs& a, bool fwd, int slice, int cpt, int warps, size_t smem, cudaStream_t st);
cudaError_t launch_pass_lean64(const LeanArgs& a, bool fwd, int slice, int warps, size_t smem, cudaStream_t st);

// every kernel launch of the library goes through the wrappers below and is counted here
void count_launches(long long n);

// ---- launch wrappers (host side, implemented in the .cu files) -------------
cudaError_t launch_kahn(int n, const long long* in_ptr, const long long* out_ptr, const int* out_dst,
                        int* indeg, int* level, int* queue, long long* level_ptr_dev, int* level_cnt,
                        long long* result, int sm_count, cudaStream_t st);
cudaError_t launch_sort_order(int n, const int* level, unsigned long long* keys, int npad, int* order, cudaStream_t st);
cudaError_t launch_build_adj(int n, const int* order, const long long* ptr, const int* idx, const long long* t,
                             int* eptr, int* nbr, long long* tperm, cudaStream_t st);
cudaError_t launch_sink_flags(int n, const int* order, const long long* out_ptr, uint8_t* flag, cudaStream_t st);
cudaError_t launch_numerators(int n, int m, long long S, const int* order, const int* c,
                              const int* nbr_f, const long long* t_f, const int* nbr_b, const long long* t_b,
                              unsigned long long* xvert, unsigned long long* xw_f, unsigned long long* xnbr_f,
                              unsigned long long* xw_b, cudaStream_t st);
cudaError_t launch_default_mem(int n, const long long* out_ptr, const long long* out_t, long long* mem, cudaStream_t st);

int pick_cpt(long long P);
cudaError_t launch_pass_level_sync(const PassArgs& a, bool fwd, const std::vector<long long>& level_ptr_host, cudaStream_t st);
cudaError_t launch_zero_rows(const int* rows, int count, long long P, long long ldp, long long* lev, cudaStream_t st);
cudaError_t launch_pass_sliced(const PassArgs& a, bool fwd, const SlicedPlan& plan, int cpt, int warps, bool table,
                               cudaStream_t st);
cudaError_t launch_positions(int n, const int* order, int* pos_of, const int* nbr_f, const int* eptr_f, int* maxspan,
                             cudaStream_t st);
cudaError_t launch_vertf(int n, const int* order, const uint8_t* sink_flag, int* vertf, cudaStream_t st);
cudaError_t launch_cp_reduce(const PassArgs& a, bool from_tlevel, const int* list, int list_len, cudaStream_t st);
cudaError_t launch_loads(int n, long long P, long long ldp, const uint8_t* part, const int* vert,
                         const unsigned long long* xvert, const long long* mem, DevTables tab, long long* load,
                         long long* memload, int* status, bool validate, int sm_count, cudaStream_t st);
cudaError_t launch_rt_rows(int n, int k, int kp, const int* pos_of, const unsigned long long* xvert, const DivConst* rt_div,
                           long long* rtv, cudaStream_t st);
cudaError_t launch_loads2(int n, long long P, long long ldp, const uint8_t* part, const long long* rtv, const long long* mem,
                          int k, int kp, long long* load, long long* memload, int* status, bool validate, int sm_count,
                          int smem_optin, cudaStream_t st);
cudaError_t launch_validate(long long n, long long P, long long ldp, const uint8_t* part, int k, int* status,
                            int sm_count, cudaStream_t st);
cudaError_t launch_viol(long long P, long long ldp, int k, const long long* memload, const long long* cap,
                        unsigned long long* viol, const int* status, cudaStream_t st);
cudaError_t launch_constraints(long long P, long long ldp, const uint8_t* part, int npairs, const int* pair_a, const int* pair_b,
                               int ndev, const int* dc_v, const int* dc_d, int* coll_viol, int* dev_viol, const int* status,
                               cudaStream_t st);
cudaError_t launch_critical_mask(long long n, long long P, long long ldp, const long long* tlevel, const long long* blevel,
                                 const long long* cp, uint8_t* mask, cudaStream_t st);
// rank-driven partitioners (partition.cu)
cudaError_t launch_ranks(int n, const std::vector<long long>& level_ptr, const int* order, const long long* in_ptr,
                         const int* in_src, const long long* out_ptr, const int* out_dst, const int* c, long long* up,
                         long long* down, long long* total, cudaStream_t st);
cudaError_t launch_critical_path(int n, const long long* in_ptr, const int* in_src, const long long* out_ptr,
                                 const long long* down, int* path, long long* scratch, cudaStream_t st);
cudaError_t launch_batch_split(int n, int npad, int k, const long long* total, const long long* mem, const int* ord,
                               const long long* cap, int* idx, uint8_t* part, long long* unplaced, cudaStream_t st);
cudaError_t launch_cp_partition(int n, int k, long long S, const int* path, long long len, const int* c, const long long* mem,
                                const int* speed, const int* ord, const long long* cap, uint8_t* on_path, uint8_t* part,
                                long long* unplaced, cudaStream_t st);
// batched list-scheduling simulation (simulate.cu)
cudaError_t launch_simulate(int n, int k, long long P, long long ldp, long long S, const uint8_t* part,
                            const long long* in_ptr, const long long* out_ptr, const int* out_dst, const long long* out_t,
                            const int* c, const int* speed, const long long* B, int policy, const long long* prio,
                            const long long* msr_w, long long* start, long long* makespan, int blocks, long long* ready,
                            int* left, int* list, int* status, cudaStream_t st);
int simulate_warps_per_block();
cudaError_t launch_transpose_u8(const uint8_t* src, uint8_t* dst, long long P, long long n, long long ldp, cudaStream_t st);

}  // namespace tfps
