/*
 * TEST INFRASTRUCTURE -- NOT PART OF THE PRODUCT PATH.
 *
 * Plain, slow, single-threaded CPU oracle for critical-path evaluation of one
 * data-flow graph under one partition, written from the paper's definitions.
 * It shares no code, headers, tables or constants with the CUDA library; only
 * tests, the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * Model (Section 2): G=(V,E), vertex cost c_i, edge size t_i; device speed s,
 * capacity C, bandwidth matrix B.  Execution time of a vertex on its device is
 * c/s (Section 2, the c_1/s_1 example); the transfer time of an edge is 0 when
 * both end points sit on the same device, else tensor size over the transfer
 * rate between the two devices (Section 4.1, text before Eq. 12).
 *
 * Integer reading: time is counted in ticks, S ticks per paper time unit, and
 * every real quotient is rounded up once:
 *      rt(v)   = ceil(c_v * S / s_{p(v)})
 *      w(u->v) = 0 if p(u)==p(v), else ceil(t_uv * S / B[p(u)][p(v)])
 * with B indexed [device of the edge's source][device of its target].
 *
 * Parity pins (tests/test_oracle_*.py): hand-computed worked DAGs stored under
 * tests/golden/, brute-force enumeration of all paths on graphs of <= 12
 * vertices, single-device reduction against networkx/scipy longest path, the
 * unit-cost setting of the NP-completeness reduction (Lemma 1), exact-rational
 * error bound against the real-valued model, and the invariants listed there.
 * No function here is "parity unpinned".
 *
 * All arithmetic is int64; every product and sum is checked in __int128 and
 * reported as ORACLE_OVERFLOW instead of wrapping.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_BAD_ARG -1
#define ORACLE_CYCLE -2
#define ORACLE_OVERFLOW -3
#define ORACLE_BAD_PARTITION -4

typedef __int128 i128;

static int fits(i128 x) { return x >= 0 && x <= (i128)INT64_MAX; }

/* ceil(a*S/b) for a>=0, S>=1, b>=1 by plain integer division. */
static int ceil_scaled(int64_t a, int64_t S, int64_t b, int64_t *out)
{
    i128 num = (i128)a * (i128)S;
    i128 q = num / b;
    if (num % b != 0) q += 1;
    if (!fits(q)) return ORACLE_OVERFLOW;
    *out = (int64_t)q;
    return ORACLE_OK;
}

/*
 * Topological structure.  A vertex is schedulable once data on all incoming
 * edges is available (Section 2); Kahn's algorithm with a FIFO queue emits
 * vertices in such an order.  level(v) = 0 for sources, else 1 + the largest
 * level of a predecessor.  `order` lists vertices by level, ascending id
 * inside a level; level_ptr[l]..level_ptr[l+1] delimits level l.
 * level_ptr must have room for n+1 entries.  topo (may be NULL) receives the
 * raw Kahn order.
 */
int oracle_topo_levels(int64_t n, const int64_t *in_ptr, const int32_t *in_src,
                       const int64_t *out_ptr, const int32_t *out_dst,
                       int32_t *level, int32_t *order, int64_t *level_ptr,
                       int32_t *num_levels, int32_t *topo)
{
    if (n < 0) return ORACLE_BAD_ARG;
    int64_t *indeg = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n + 1));
    int32_t *queue = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n + 1));
    if (!indeg || !queue) { free(indeg); free(queue); return ORACLE_BAD_ARG; }
    int64_t head = 0, tail = 0;
    for (int64_t v = 0; v < n; ++v) {
        indeg[v] = in_ptr[v + 1] - in_ptr[v];
        if (indeg[v] == 0) queue[tail++] = (int32_t)v;
    }
    while (head < tail) {
        int32_t u = queue[head++];
        for (int64_t e = out_ptr[u]; e < out_ptr[u + 1]; ++e) {
            int32_t x = out_dst[e];
            if (--indeg[x] == 0) queue[tail++] = x;
        }
    }
    if (tail != n) { free(indeg); free(queue); return ORACLE_CYCLE; }
    int32_t L = 0;
    for (int64_t i = 0; i < n; ++i) {
        int32_t v = queue[i];
        int32_t lv = 0;
        for (int64_t e = in_ptr[v]; e < in_ptr[v + 1]; ++e) {
            int32_t cand = level[in_src[e]] + 1;
            if (cand > lv) lv = cand;
        }
        level[v] = lv;
        if (lv + 1 > L) L = lv + 1;
    }
    if (n == 0) L = 0;
    for (int32_t l = 0; l <= L; ++l) level_ptr[l] = 0;
    for (int64_t v = 0; v < n; ++v) level_ptr[level[v] + 1] += 1;
    for (int32_t l = 0; l < L; ++l) level_ptr[l + 1] += level_ptr[l];
    int64_t *fill = indeg; /* reuse */
    for (int32_t l = 0; l < L; ++l) fill[l] = level_ptr[l];
    for (int64_t v = 0; v < n; ++v) order[fill[level[v]]++] = (int32_t)v;
    if (topo) memcpy(topo, queue, sizeof(int32_t) * (size_t)n);
    *num_levels = L;
    free(indeg); free(queue);
    return ORACLE_OK;
}

/*
 * Default per-vertex memory: data leaving the source vertex of an edge
 * consumes memory of that vertex's device (Section 2), so mem_v = sum of the
 * sizes of v's outgoing edges.
 */
int oracle_default_mem(int64_t n, const int64_t *out_ptr, const int64_t *out_t, int64_t *mem)
{
    for (int64_t v = 0; v < n; ++v) {
        i128 acc = 0;
        for (int64_t e = out_ptr[v]; e < out_ptr[v + 1]; ++e) acc += out_t[e];
        if (!fits(acc)) return ORACLE_OVERFLOW;
        mem[v] = (int64_t)acc;
    }
    return ORACLE_OK;
}

/*
 * One candidate partition p (uint8 per vertex, element stride p_stride).
 * topo: any topological order of the graph (oracle_topo_levels gives one).
 *
 * tlevel(v): earliest start = max over in-edges (u->v) of
 *            tlevel(u) + rt(u) + w(u->v); 0 for sources.  This is the
 *            downward recursion of Eq. 6 carried out with execution times and
 *            transfer times and without the vertex's own term, i.e. the start
 *            time that the schedule function f returns (Section 2).
 * blevel(v): Eq. 12 (path computation time): rt(v) + max over out-edges
 *            (v->x) of ( blevel(x) + w(v->x) ); rt(v) for sinks.
 * cp:        start time of the artificial zero-cost sink joined to every sink
 *            by a zero-cost edge (Section 2, after Eq. 1) = max_v tlevel+rt.
 * load[d]:   sum of rt(v) over vertices on d (the sum inside Eq. 7).
 * memload[d]: sum of mem_v over vertices on d; Eq. 2 demands usage < C_d, so
 *            bit d of *viol is set iff memload[d] >= C[d].
 * Any of tlevel, blevel, load, memload, viol may be NULL.
 */
int oracle_eval_partition(int64_t n,
                          const int64_t *in_ptr, const int32_t *in_src, const int64_t *in_t,
                          const int64_t *out_ptr, const int32_t *out_dst, const int64_t *out_t,
                          const int32_t *c, const int64_t *mem,
                          int32_t k, const int32_t *s, const int64_t *C, const int64_t *B, int64_t S,
                          const int32_t *topo,
                          const uint8_t *p, int64_t p_stride,
                          int64_t *tlevel, int64_t *blevel, int64_t *cp,
                          int64_t *load, int64_t *memload, uint64_t *viol)
{
    if (n < 0 || k < 1 || k > 64 || S < 1) return ORACLE_BAD_ARG;
    int rc = ORACLE_OK;
    int64_t *rt = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n + 1));
    int64_t *tl = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n + 1));
    int64_t *bl = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n + 1));
    if (!rt || !tl || !bl) { rc = ORACLE_BAD_ARG; goto done; }

    for (int64_t v = 0; v < n; ++v) {
        int d = p[v * p_stride];
        if (d >= k) { rc = ORACLE_BAD_PARTITION; goto done; }
        if (c[v] < 0 || s[d] < 1) { rc = ORACLE_BAD_ARG; goto done; }
        rc = ceil_scaled(c[v], S, s[d], &rt[v]);
        if (rc) goto done;
    }

    /* forward: earliest start times */
    for (int64_t i = 0; i < n; ++i) {
        int32_t v = topo[i];
        int dv = p[v * p_stride];
        i128 best = 0;
        for (int64_t e = in_ptr[v]; e < in_ptr[v + 1]; ++e) {
            int32_t u = in_src[e];
            int du = p[u * p_stride];
            int64_t w = 0;
            if (du != dv) {
                if (in_t[e] < 0 || B[du * k + dv] < 1) { rc = ORACLE_BAD_ARG; goto done; }
                rc = ceil_scaled(in_t[e], S, B[du * k + dv], &w);
                if (rc) goto done;
            }
            i128 cand = (i128)tl[u] + rt[u] + w;
            if (cand > best) best = cand;
        }
        if (!fits(best)) { rc = ORACLE_OVERFLOW; goto done; }
        tl[v] = (int64_t)best;
    }

    /* backward: Eq. 12 */
    for (int64_t i = n - 1; i >= 0; --i) {
        int32_t v = topo[i];
        int dv = p[v * p_stride];
        i128 best = 0;
        for (int64_t e = out_ptr[v]; e < out_ptr[v + 1]; ++e) {
            int32_t x = out_dst[e];
            int dx = p[x * p_stride];
            int64_t w = 0;
            if (dx != dv) {
                if (out_t[e] < 0 || B[dv * k + dx] < 1) { rc = ORACLE_BAD_ARG; goto done; }
                rc = ceil_scaled(out_t[e], S, B[dv * k + dx], &w);
                if (rc) goto done;
            }
            i128 cand = (i128)bl[x] + w;
            if (cand > best) best = cand;
        }
        best += rt[v];
        if (!fits(best)) { rc = ORACLE_OVERFLOW; goto done; }
        bl[v] = (int64_t)best;
    }

    {
        i128 mx = 0;
        for (int64_t v = 0; v < n; ++v) {
            i128 f = (i128)tl[v] + rt[v];
            if (f > mx) mx = f;
        }
        if (!fits(mx)) { rc = ORACLE_OVERFLOW; goto done; }
        if (cp) *cp = (int64_t)mx;
    }

    {
        i128 ld[64], ml[64];
        for (int d = 0; d < k; ++d) { ld[d] = 0; ml[d] = 0; }
        for (int64_t v = 0; v < n; ++v) {
            int d = p[v * p_stride];
            ld[d] += rt[v];
            if (mem) {
                if (mem[v] < 0) { rc = ORACLE_BAD_ARG; goto done; }
                ml[d] += mem[v];
            }
        }
        uint64_t bits = 0;
        for (int d = 0; d < k; ++d) {
            if (!fits(ld[d]) || !fits(ml[d])) { rc = ORACLE_OVERFLOW; goto done; }
            if (load) load[d] = (int64_t)ld[d];
            if (memload) memload[d] = (int64_t)ml[d];
            if (mem && C && ml[d] >= (i128)C[d]) bits |= (uint64_t)1 << d;
        }
        if (viol) *viol = bits;
    }

    if (tlevel) memcpy(tlevel, tl, sizeof(int64_t) * (size_t)n);
    if (blevel) memcpy(blevel, bl, sizeof(int64_t) * (size_t)n);
done:
    free(rt); free(tl); free(bl);
    return rc;
}

/*
 * Placement constraints of one candidate partition p (uint8, byte stride pstride).
 *   collocation constraints (Section 2, Eq. 3): for every listed pair (a, b), p(a) = p(b) must hold;
 *   device constraints (Section 2, Eq. 4): for every listed pair (v, d), p(v) = d must hold.
 * Every listed pair is one requirement; *coll_viol and *dev_viol count the requirements that do not hold
 * (a vertex listed with two different devices therefore always violates at least one of them).
 * Pins: tests/test_oracle_constraints.py (a worked example, closed forms on the partition v mod k, invariants).
 */
int oracle_eval_constraints(int64_t n, const uint8_t *p, int64_t pstride,
                            int64_t npairs, const int32_t *pair_a, const int32_t *pair_b,
                            int64_t ndev, const int32_t *dc_v, const int32_t *dc_d,
                            int64_t *coll_viol, int64_t *dev_viol)
{
    int64_t cv = 0, dv = 0;
    if (n < 0 || npairs < 0 || ndev < 0 || !coll_viol || !dev_viol) return ORACLE_BAD_ARG;
    for (int64_t i = 0; i < npairs; ++i) {
        if (pair_a[i] < 0 || pair_a[i] >= n || pair_b[i] < 0 || pair_b[i] >= n) return ORACLE_BAD_ARG;
        if (p[(int64_t)pair_a[i] * pstride] != p[(int64_t)pair_b[i] * pstride]) ++cv;
    }
    for (int64_t i = 0; i < ndev; ++i) {
        if (dc_v[i] < 0 || dc_v[i] >= n || dc_d[i] < 0 || dc_d[i] > 255) return ORACLE_BAD_ARG;
        if ((int32_t)p[(int64_t)dc_v[i] * pstride] != dc_d[i]) ++dv;
    }
    *coll_viol = cv;
    *dev_viol = dv;
    return ORACLE_OK;
}

/*
 * Critical vertices of one evaluated candidate (Section 3.2: the critical path is the longest path from a source to
 * a sink): vertex v lies on a longest path exactly when the longest path into it plus the longest path out of it
 * spans the whole critical-path length, tlevel(v) + blevel(v) = CP (tlevel excludes v's own runtime, blevel includes
 * it, so a vertex is counted once).  mask[v] = 1 for those vertices, else 0; strides in elements.
 * Pins: tests/test_oracle_constraints.py (the critical sets of the worked DAGs, a chain, properties).
 */
int oracle_critical_mask(int64_t n, const int64_t *tlevel, int64_t tstride, const int64_t *blevel, int64_t bstride,
                         int64_t cp, uint8_t *mask, int64_t mstride)
{
    if (n < 0 || !tlevel || !blevel || !mask) return ORACLE_BAD_ARG;
    for (int64_t v = 0; v < n; ++v) {
        i128 total = (i128)tlevel[v * tstride] + (i128)blevel[v * bstride];
        if (!fits(total)) return ORACLE_OVERFLOW;
        mask[v * mstride] = (int64_t)total == cp ? 1 : 0;
    }
    return ORACLE_OK;
}

/*
 * Vertex ranks (Section 3.2, Eq. 5 and Eq. 6), independent of any partition:
 *      upRank(v)   = c_v + max over successors x of upRank(x)      (the maximum over no successor is 0: a sink has c_v)
 *      downRank(v) = c_v + max over predecessors u of downRank(u)  (a source has c_v)
 *      totalRank(v) = upRank(v) + downRank(v)                      (Section 3.2.1: "the sum of the upward rank and the
 *                                                                   downward rank"; c_v is in both terms, as printed)
 * topo: any topological order.  Any of up, down, total may be NULL.
 * Pins: tests/test_oracle_ranks.py (hand values on the worked DAGs, chain closed form, all source-to-sink paths
 * enumerated on small graphs, the single-device unit-speed evaluation of the same graph).
 */
int oracle_ranks(int64_t n, const int64_t *in_ptr, const int32_t *in_src, const int64_t *out_ptr, const int32_t *out_dst,
                 const int32_t *c, const int32_t *topo, int64_t *up, int64_t *down, int64_t *total)
{
    if (n < 0) return ORACLE_BAD_ARG;
    int64_t *u = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n + 1));
    int64_t *d = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n + 1));
    if (!u || !d) { free(u); free(d); return ORACLE_BAD_ARG; }
    int rc = ORACLE_OK;
    for (int64_t i = 0; i < n && rc == ORACLE_OK; ++i) {          /* Eq. 6, sources first */
        int32_t v = topo[i];
        i128 best = 0;
        for (int64_t e = in_ptr[v]; e < in_ptr[v + 1]; ++e)
            if ((i128)d[in_src[e]] > best) best = d[in_src[e]];
        best += c[v];
        if (!fits(best)) rc = ORACLE_OVERFLOW; else d[v] = (int64_t)best;
    }
    for (int64_t i = n - 1; i >= 0 && rc == ORACLE_OK; --i) {     /* Eq. 5, sinks first */
        int32_t v = topo[i];
        i128 best = 0;
        for (int64_t e = out_ptr[v]; e < out_ptr[v + 1]; ++e)
            if ((i128)u[out_dst[e]] > best) best = u[out_dst[e]];
        best += c[v];
        if (!fits(best)) rc = ORACLE_OVERFLOW; else u[v] = (int64_t)best;
    }
    for (int64_t v = 0; v < n && rc == ORACLE_OK; ++v) {
        i128 t = (i128)u[v] + (i128)d[v];
        if (!fits(t)) { rc = ORACLE_OVERFLOW; break; }
        if (up) up[v] = u[v];
        if (down) down[v] = d[v];
        if (total) total[v] = (int64_t)t;
    }
    free(u); free(d);
    return rc;
}

/* devices from the fastest to the slowest (equal speeds: lower index first) */
static void devices_by_speed(int32_t k, const int32_t *s, int32_t *ord)
{
    for (int32_t i = 0; i < k; ++i) ord[i] = i;
    for (int32_t i = 1; i < k; ++i) {          /* insertion sort, stable */
        int32_t x = ord[i], j = i;
        while (j > 0 && s[ord[j - 1]] < s[x]) { ord[j] = ord[j - 1]; --j; }
        ord[j] = x;
    }
}

static const int64_t *rank_keys;   /* keys of the sort below (the oracle is single-threaded) */
static int rank_order(const void *pa, const void *pb)
{
    int64_t a = *(const int64_t *)pa, b = *(const int64_t *)pb;
    if (rank_keys[a] != rank_keys[b]) return rank_keys[a] > rank_keys[b] ? -1 : 1;
    return a < b ? -1 : (a > b ? 1 : 0);
}

/*
 * Batch Split (Section 3.2.1): the vertices are taken in descending order of total rank (equal ranks: ascending
 * vertex id) and each is assigned, independently of the others, to the fastest feasible device.  Feasible = the
 * device's static memory use stays below its capacity with the vertex on it (Eq. 2: usage < C).  A vertex no device
 * can take goes to the fastest device and is counted in *unplaced (the paper does not say; the instance is then
 * infeasible).  part[v] receives the device.
 * Pins: tests/test_oracle_ranks.py (worked example, closed forms, capacity invariants).
 */
int oracle_batch_split(int64_t n, const int64_t *total, const int64_t *mem, int32_t k, const int32_t *s,
                       const int64_t *C, uint8_t *part, int64_t *unplaced)
{
    if (n < 0 || k < 1 || k > 64 || !unplaced) return ORACLE_BAD_ARG;
    int32_t ord[64];
    i128 used[64];
    devices_by_speed(k, s, ord);
    for (int32_t d = 0; d < k; ++d) used[d] = 0;
    int64_t *idx = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n + 1));
    if (!idx) return ORACLE_BAD_ARG;
    for (int64_t v = 0; v < n; ++v) idx[v] = v;
    rank_keys = total;
    qsort(idx, (size_t)n, sizeof(int64_t), rank_order);   /* descending total rank, ascending id */
    int64_t bad = 0;
    for (int64_t i = 0; i < n; ++i) {
        int64_t v = idx[i];
        int32_t chosen = -1;
        for (int32_t q = 0; q < k && chosen < 0; ++q) {
            int32_t d = ord[q];
            if (used[d] + (i128)mem[v] < (i128)C[d]) chosen = d;
        }
        if (chosen < 0) { chosen = ord[0]; ++bad; }
        used[chosen] += mem[v];
        part[v] = (uint8_t)chosen;
    }
    *unplaced = bad;
    free(idx);
    return ORACLE_OK;
}

/*
 * The critical path of the Critical Path strategy (Section 3.2.2, steps (1)-(4)): the sink with the largest downward
 * rank (equal ranks: the smallest id), then backwards along predecessors of largest downward rank (equal: smallest id)
 * until a source is reached.  path receives the vertices from the source to the sink, *len their number.
 * The summed cost of the path is the chosen sink's downward rank, whatever the tie rule.
 */
int oracle_critical_path(int64_t n, const int64_t *in_ptr, const int32_t *in_src, const int64_t *out_ptr,
                         const int64_t *down, int32_t *path, int64_t *len)
{
    if (n < 0 || !len) return ORACLE_BAD_ARG;
    *len = 0;
    if (n == 0) return ORACLE_OK;
    int64_t best = -1;
    for (int64_t v = 0; v < n; ++v)
        if (out_ptr[v + 1] == out_ptr[v] && (best < 0 || down[v] > down[best])) best = v;
    if (best < 0) return ORACLE_CYCLE;
    int64_t cnt = 0;
    for (int64_t v = best;;) {
        path[cnt++] = (int32_t)v;
        if (in_ptr[v + 1] == in_ptr[v]) break;
        int64_t u = -1;
        for (int64_t e = in_ptr[v]; e < in_ptr[v + 1]; ++e) {
            int64_t x = in_src[e];
            if (u < 0 || down[x] > down[u] || (down[x] == down[u] && x < u)) u = x;
        }
        v = u;
        if (cnt > n) return ORACLE_CYCLE;
    }
    for (int64_t i = 0; i < cnt / 2; ++i) { int32_t t = path[i]; path[i] = path[cnt - 1 - i]; path[cnt - 1 - i] = t; }
    *len = cnt;
    return ORACLE_OK;
}

/*
 * Critical Path partitioning (Section 3.2.2, Eq. 7).  The critical path goes to the fastest device that can hold all
 * of it (static memory below capacity, Eq. 2); if none can, it is divided among the fastest devices: the path is
 * walked from its source and every vertex goes to the fastest device that still has room for it.  Every other
 * vertex v, in ascending id, goes to the feasible device d that minimises (sum of the execution times of the vertices
 * already on d) + (execution time of v on d), execution time = ceil(c * S / s_d) ticks (equal sums: lower device
 * index).  A vertex no device can take is placed by the same rule over all devices and counted in *unplaced.
 */
int oracle_cp_partition(int64_t n, const int32_t *path, int64_t len, const int32_t *c, const int64_t *mem,
                        int32_t k, const int32_t *s, const int64_t *C, int64_t S, uint8_t *part, int64_t *unplaced)
{
    if (n < 0 || len < 0 || len > n || k < 1 || k > 64 || S < 1 || !unplaced) return ORACLE_BAD_ARG;
    int32_t ord[64];
    i128 used[64], load[64];
    devices_by_speed(k, s, ord);
    for (int32_t d = 0; d < k; ++d) { used[d] = 0; load[d] = 0; }
    uint8_t *on_path = (uint8_t *)calloc((size_t)(n + 1), 1);
    if (!on_path) return ORACLE_BAD_ARG;
    int64_t bad = 0;
    i128 path_mem = 0;
    for (int64_t i = 0; i < len; ++i) { on_path[path[i]] = 1; path_mem += mem[path[i]]; }
    int32_t whole = -1;
    for (int32_t q = 0; q < k && whole < 0; ++q)
        if (path_mem < (i128)C[ord[q]]) whole = ord[q];
    for (int64_t i = 0; i < len; ++i) {
        int64_t v = path[i];
        int32_t chosen = whole;
        for (int32_t q = 0; q < k && chosen < 0; ++q)
            if (used[ord[q]] + (i128)mem[v] < (i128)C[ord[q]]) chosen = ord[q];
        if (chosen < 0) { chosen = ord[0]; ++bad; }
        int64_t rt;
        if (ceil_scaled(c[v], S, s[chosen], &rt)) { free(on_path); return ORACLE_OVERFLOW; }
        used[chosen] += mem[v];
        load[chosen] += rt;
        part[v] = (uint8_t)chosen;
    }
    for (int64_t v = 0; v < n; ++v) {
        if (on_path[v]) continue;
        int32_t chosen = -1, any = -1;
        i128 best = 0, best_any = 0;
        for (int32_t d = 0; d < k; ++d) {
            int64_t rt;
            if (ceil_scaled(c[v], S, s[d], &rt)) { free(on_path); return ORACLE_OVERFLOW; }
            i128 sum = load[d] + rt;                                 /* Eq. 7 */
            if (any < 0 || sum < best_any) { any = d; best_any = sum; }
            if (used[d] + (i128)mem[v] < (i128)C[d] && (chosen < 0 || sum < best)) { chosen = d; best = sum; }
        }
        if (chosen < 0) { chosen = any; best = best_any; ++bad; }
        if (!fits(best)) { free(on_path); return ORACLE_OVERFLOW; }
        used[chosen] += mem[v];
        load[chosen] = best;
        part[v] = (uint8_t)chosen;
    }
    *unplaced = bad;
    free(on_path);
    return ORACLE_OK;
}

/*
 * List-scheduling simulation of one candidate partition (Section 4, criteria (1)-(6); the event-based simulation of
 * Section 5).  Every device executes the vertices assigned to it, one at a time and without interruption (criteria
 * 1-3, 5); a vertex is executable once every predecessor has finished and its tensor has arrived,
 *      ready(v) = max over in-edges (u->v) of finish(u) + w(u->v),   0 for a source           (criterion 4)
 * with the execution and transfer times of the evaluation (rt, w; transfers do not queue: the paper models none);
 * an idle device that has an executable vertex starts one at once, otherwise it stays idle (criterion 6).
 * Which one: policy 0 = FIFO (the vertex that became executable first; equal times: the smaller id),
 *            policy 1 = PCT (Section 4.1: the largest path computation time, Eq. 12, passed in as prio[]; equal: the
 *                       smaller id),
 *            policy 2 = MSR (Section 4.2, Eq. 13: the largest successor rank; equal: the smaller id).  The score of v is
 *                       the sum over its out-edges (v->x) of  alpha + beta [p(x) != p(v)] + gamma [x has one in-edge]
 *                       + delta [the device of x is idle and x has one in-edge], msr_w = {alpha, beta, gamma, delta};
 *                       "idle" is what held when the start step began: no execution on that device (the devices that
 *                       decide in this step are idle themselves).
 * Events are taken in time order; at one time T first every execution that ends at T is completed (and its
 * successors' ready times updated), then every idle device starts its best executable vertex; a vertex of zero
 * execution time ends at T as well, so the two steps repeat at T until nothing changes.
 * start[v] receives the start time of v (the schedule f of Section 2), *makespan the time the last vertex ends.
 * The per-device lists are plain arrays scanned linearly.
 */
int oracle_simulate(int64_t n,
                    const int64_t *in_ptr, const int64_t *out_ptr, const int32_t *out_dst, const int64_t *out_t,
                    const int32_t *c, int32_t k, const int32_t *s, const int64_t *B, int64_t S,
                    const uint8_t *p, int64_t p_stride, int32_t policy, const int64_t *prio, int64_t prio_stride,
                    const int64_t *msr_w, int64_t *start, int64_t *makespan)
{
    if (n < 0 || k < 1 || k > 64 || S < 1 || policy < 0 || policy > 2 || !makespan) return ORACLE_BAD_ARG;
    if (policy == 1 && !prio) return ORACLE_BAD_ARG;
    if (policy == 2 && !msr_w) return ORACLE_BAD_ARG;
    *makespan = 0;
    if (n == 0) return ORACLE_OK;
    int rc = ORACLE_OK;
    int64_t *rt = (int64_t *)malloc(sizeof(int64_t) * (size_t)n);
    int64_t *ready = (int64_t *)calloc((size_t)n, sizeof(int64_t));
    int64_t *left = (int64_t *)malloc(sizeof(int64_t) * (size_t)n);       /* predecessors not finished yet */
    int64_t *list = (int64_t *)malloc(sizeof(int64_t) * (size_t)n);       /* per device: vertices whose ready time is known */
    int64_t first[65], count[64], running[64], busy_until[64];
    int idle_then[64];
    int64_t *score = (int64_t *)calloc((size_t)n, sizeof(int64_t));       /* MSR score at the running start step */
    if (!rt || !ready || !left || !list || !score) { rc = ORACLE_BAD_ARG; goto done; }
    for (int32_t d = 0; d <= k; ++d) first[d] = 0;
    for (int64_t v = 0; v < n; ++v) {
        int32_t d = p[v * p_stride];
        if (d >= k) { rc = ORACLE_BAD_PARTITION; goto done; }
        if (ceil_scaled(c[v], S, s[d], &rt[v])) { rc = ORACLE_OVERFLOW; goto done; }
        first[d + 1] += 1;
        left[v] = in_ptr[v + 1] - in_ptr[v];
    }
    for (int32_t d = 0; d < k; ++d) { first[d + 1] += first[d]; count[d] = 0; running[d] = -1; busy_until[d] = 0; }
    for (int64_t v = 0; v < n; ++v)
        if (left[v] == 0) { int32_t d = p[v * p_stride]; list[first[d] + count[d]++] = v; }
    int64_t T = 0, done_cnt = 0, last = 0;
    while (done_cnt < n) {
        /* every idle device starts its best executable vertex */
        for (int32_t d = 0; d < k; ++d) idle_then[d] = running[d] < 0;
        for (int32_t d = 0; d < k; ++d) {
            if (running[d] >= 0) continue;
            int64_t best = -1, at = -1;
            for (int64_t i = 0; i < count[d]; ++i) {
                int64_t v = list[first[d] + i];
                if (ready[v] > T) continue;
                if (policy == 2) {                                   /* Eq. 13 */
                    i128 sc = 0;
                    for (int64_t e = out_ptr[v]; e < out_ptr[v + 1]; ++e) {
                        int64_t x = out_dst[e];
                        int32_t dx = p[x * p_stride];
                        int single = in_ptr[x + 1] - in_ptr[x] == 1;
                        sc += msr_w[0];
                        if (dx != d) sc += msr_w[1];
                        if (single) sc += msr_w[2];
                        if (single && idle_then[dx]) sc += msr_w[3];
                    }
                    if (!fits(sc)) { rc = ORACLE_OVERFLOW; goto done; }
                    score[v] = (int64_t)sc;
                }
                int better;
                if (best < 0) better = 1;
                else if (policy == 0) better = ready[v] < ready[best] || (ready[v] == ready[best] && v < best);
                else if (policy == 2) better = score[v] > score[best] || (score[v] == score[best] && v < best);
                else better = prio[v * prio_stride] > prio[best * prio_stride] ||
                              (prio[v * prio_stride] == prio[best * prio_stride] && v < best);
                if (better) { best = v; at = i; }
            }
            if (best < 0) continue;
            list[first[d] + at] = list[first[d] + --count[d]];
            i128 fin = (i128)T + (i128)rt[best];
            if (!fits(fin)) { rc = ORACLE_OVERFLOW; goto done; }
            running[d] = best;
            busy_until[d] = (int64_t)fin;
            if (start) start[best] = T;
        }
        /* the next time anything happens: an execution ends, or an idle device's earliest vertex becomes executable */
        int64_t next = -1;
        for (int32_t d = 0; d < k; ++d) {
            if (running[d] >= 0) {
                if (next < 0 || busy_until[d] < next) next = busy_until[d];
            } else {
                for (int64_t i = 0; i < count[d]; ++i) {
                    int64_t r = ready[list[first[d] + i]];
                    if (next < 0 || r < next) next = r;
                }
            }
        }
        if (next < 0) { rc = ORACLE_CYCLE; goto done; }   /* nothing runs and nothing is pending: not a DAG */
        T = next;
        /* executions that end at T */
        for (int32_t d = 0; d < k; ++d) {
            if (running[d] < 0 || busy_until[d] != T) continue;
            int64_t u = running[d];
            running[d] = -1;
            ++done_cnt;
            if (T > last) last = T;
            for (int64_t e = out_ptr[u]; e < out_ptr[u + 1]; ++e) {
                int64_t x = out_dst[e];
                int32_t dx = p[x * p_stride];
                int64_t w = 0;
                if (dx != d && ceil_scaled(out_t[e], S, B[(int64_t)d * k + dx], &w)) { rc = ORACLE_OVERFLOW; goto done; }
                i128 arr = (i128)T + (i128)w;
                if (!fits(arr)) { rc = ORACLE_OVERFLOW; goto done; }
                if ((int64_t)arr > ready[x]) ready[x] = (int64_t)arr;
                if (--left[x] == 0) list[first[dx] + count[dx]++] = x;
            }
        }
    }
    *makespan = last;
done:
    free(rt); free(ready); free(left); free(list); free(score);
    return rc;
}
