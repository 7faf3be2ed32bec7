// Shared pieces of the cooperative level-loop kernels (tensor-core bf16 and plain fp32): the description of a
// pass, the warps that prepare descriptions ahead of the arithmetic, and small copy helpers.
//
// The unit of work of those kernels is a pass: up to `et` child edges of a tile of `nt` nodes of one level.
// Nothing in a pass's description (node ids, child ids and positions, parent row of every edge) depends on h or c,
// so extra warps prepare the descriptions through a two-slot ring guarded by mbarriers; the chain of dependent
// index loads (perm -> child_ptr -> child_idx -> position) never sits between two passes of arithmetic.
#pragma once

#include "common.cuh"
#include "grid_sync.cuh"
#include "ptx_sm100.cuh"

namespace jdb {
namespace small {

constexpr int MAIN_WARPS = 16;     // gather, products, read-out, cell arithmetic
constexpr int META_WARPS = 4;      // pass descriptions
constexpr int MAIN_THREADS = MAIN_WARPS * 32;
constexpr int META_THREADS = META_WARPS * 32;
constexpr int STHREADS = MAIN_THREADS + META_THREADS;
constexpr int ET_MAX = 128;        // edges per pass, at most
constexpr int NT_MAX = 64;         // nodes per tile, at most

enum { BAR_MAIN = 1, BAR_META = 2 };
__device__ __forceinline__ void named_bar(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
// The same barrier carrying a vote: returns true in EVERY participating thread if any of them passed true.
// Whether to leave a loop is decided through this, never by each thread reading a flag that another role of the
// CTA may be writing at that moment: a split decision would leave some threads waiting at the next barrier.
__device__ __forceinline__ bool named_bar_any(int id, int threads, bool mine) {
    uint32_t any;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %3, 0;\n\t"
        "bar.red.or.pred p, %1, %2, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(any)
        : "r"(id), "r"(threads), "r"((uint32_t)mine)
        : "memory");
    return any != 0;
}

// What the arithmetic warps need to know about one pass; written by the description warps.
struct PassSlot {
    int ek_id[ET_MAX];      // child node id of every edge row (rows of h and c)
    int ek_pos[ET_MAX];     // its position in level order (rows of the bf16 copy of h), when positions are known
    int ep[ET_MAX];         // row of the parent inside the tile
    int nodes[NT_MAX];      // node ids of the tile's rows
    int prow[NT_MAX];       // their rows in the arrays kept by level order: position in level order minus the leaf count
    int eoff[NT_MAX + 1];   // prefix of the rows' child counts
    int pos0, m, ne, et0;   // first position and rows of the tile, its edges, first edge of this pass
};

// Shared-memory state of the ring (declared __shared__ by the kernel).
struct Ring {
    uint64_t bar_full[2], bar_empty[2];
    PassSlot slot[2];
    int t_ebeg[NT_MAX], t_wsum[2];  // description warps: first CSR edge of a row, per-warp child counts
};

// four consecutive fp32 of a row, with the row's tail guarded
__device__ __forceinline__ float4 load_row4(const float* row, int col, int H, int vec_ok) {
    if (vec_ok && col + 4 <= H) return __ldcg(reinterpret_cast<const float4*>(row + col));
    float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
    if (col < H) r.x = __ldcg(row + col);
    if (col + 1 < H) r.y = __ldcg(row + col + 1);
    if (col + 2 < H) r.z = __ldcg(row + col + 2);
    if (col + 3 < H) r.w = __ldcg(row + col + 3);
    return r;
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}

__device__ __forceinline__ void ring_init(Ring& R) {  // one thread, before the CTA-wide barrier
    for (int s = 0; s < 2; ++s) {
        ptx::mbar_init(ptx::smem_u32(&R.bar_full[s]), 1);
        ptx::mbar_init(ptx::smem_u32(&R.bar_empty[s]), 1);
    }
}

// Nodes per tile of a level: 32, or 64 where that is allowed (forests of low fan-out, so that a 64-node tile still
// fits one pass) and the level has more 32-node tiles than there are tile groups.
// nt_max < 32 selects the rule of the fp32 kernel, whose products are bound by shared-memory reads per CTA: spread
// a level over all tile groups, with tiles of 4 to 32 nodes.
__device__ __forceinline__ int tile_nodes(int level_nodes, int nt_max, int n_grp) {
    if (nt_max < 32) return min(32, max(4, (level_nodes + n_grp - 1) / n_grp));
    return (nt_max > 32 && level_nodes > n_grp * 32) ? 64 : 32;
}

struct DescribeArgs {
    const int32_t* child_ptr;
    const int32_t* child_idx;
    const int32_t* level_ptr;
    const int32_t* perm;
    const int32_t* inv;  // position of every node in level order (may be null: positions are then not filled in)
    int first_level, n_levels, grp, n_grp, active_grp, nt_max;
    int32_t* meta;       // debug checks: where the first offending index is recorded
    int n_nodes, n_edges, debug;
    // tree partition (G > 0): the nodes group `grp` has on a level are gperm[goff[level * G + grp] .. goff[level * G + grp + 1])
    // and the group takes all of their tiles itself; else a level's tiles are dealt out over the active groups
    const int32_t* gperm;
    const int32_t* goff;
    int G, n_leaves;
};

// Range of the nodes this group has on a level, and which array lists them.
__device__ __forceinline__ void group_level(const DescribeArgs& d, int level, int& lo, int& hi) {
    if (d.G > 0) {
        lo = d.goff[(long long)level * d.G + d.grp];
        hi = d.goff[(long long)level * d.G + d.grp + 1];
        if (d.debug && !(dbg_ok(d.meta, CHECK_LEVEL_PTR, lo, (long long)d.n_nodes + 1, level) &&
                         dbg_ok(d.meta, CHECK_LEVEL_PTR, hi, (long long)d.n_nodes + 1, level) &&
                         dbg_ok(d.meta, CHECK_LEVEL_PTR, hi - lo, (long long)d.n_nodes + 1, level)))
            lo = hi = 0;
    } else {
        checked_level(d.level_ptr, level, d.n_nodes, d.meta, d.debug, lo, hi);
    }
}

// The loop of the description warps (threads MAIN_THREADS .. STHREADS-1 of the CTA; tm = index among them).
// Walks the same (level, tile, pass) sequence as the arithmetic warps, up to two passes ahead of them.
// stage_tile(slot, m, tile_count, tm) is called once per tile after its first slot was filled in and may start
// asynchronous copies of per-tile data (they are awaited before the slot is published).
// Every wait is bounded; a wait that runs out raises *abort, which ends both loops.
template <class StageTile>
__device__ __forceinline__ void describe_passes(const DescribeArgs& d, Ring& R, int et, volatile int* abort, int tm,
                                                StageTile stage_tile) {
    const int lane = tm & 31;
    int k = 0;       // passes described so far
    int tcount = 0;  // tiles described so far
    bool alive = true;
    for (int level = d.first_level; level < d.n_levels && alive; ++level) {
        int lo, hi;
        group_level(d, level, lo, hi);
        const int nt = tile_nodes(hi - lo, d.nt_max, d.G > 0 ? 1 : d.n_grp);
        const int tiles = (hi - lo + nt - 1) / nt;
        const int32_t* order = d.G > 0 ? d.gperm : d.perm;
        for (int tile = d.G > 0 ? 0 : d.grp; tile < tiles && alive; tile += d.G > 0 ? 1 : d.active_grp, ++tcount) {
            const int pos0 = lo + tile * nt, m = min(nt, hi - pos0);
            // rows of the tile and the prefix of their child counts
            int v = -1, eb = 0, incl = 0, prow = 0;
            if (tm < NT_MAX) {
                if (tm < m) v = order[pos0 + tm];
                if (d.debug && tm < m && !dbg_ok(d.meta, CHECK_PERM, v, d.n_nodes, pos0 + tm)) v = -1;  // a row without a node: no edges, nothing stored
                int cnt = 0;
                if (v >= 0) { eb = d.child_ptr[v]; cnt = d.child_ptr[v + 1] - eb; }
                if (d.debug && !(dbg_ok(d.meta, CHECK_EDGE_PTR, eb, (long long)d.n_edges + 1, pos0 + tm) &&
                                 dbg_ok(d.meta, CHECK_EDGE_PTR, cnt, (long long)d.n_edges - eb + 1, pos0 + tm)))
                    eb = cnt = 0;
                // row of the node in the arrays kept by level order (the input projection's P, the bf16 copy of h)
                if (v >= 0) {
                    prow = pos0 + tm - d.n_leaves;
                    if (d.G > 0) {
                        prow = d.inv[v] - d.n_leaves;
                        if (d.debug && !dbg_ok(d.meta, CHECK_POSITION, prow, (long long)d.n_nodes - d.n_leaves, v)) { v = -1; eb = cnt = 0; prow = 0; }
                    }
                }
                incl = cnt;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int y = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += y;
                }
                if (lane == 31) R.t_wsum[tm >> 5] = incl;
            }
            named_bar(BAR_META, META_THREADS);
            if (tm >= 32 && tm < NT_MAX) incl += R.t_wsum[0];
            const int ne = R.t_wsum[0] + R.t_wsum[1];
            for (int et0 = 0; et0 < ne && alive; et0 += et, ++k) {
                const int s = k & 1;
                const bool got = ptx::mbar_wait_warp(ptx::smem_u32(&R.bar_empty[s]), (uint32_t)(((k >> 1) & 1) ^ 1), abort);
                if (!got) *abort = 1;
                if (named_bar_any(BAR_META, META_THREADS, !got || *abort != 0)) { alive = false; break; }  // one verdict for all four warps
                PassSlot& S = R.slot[s];
                if (tm < NT_MAX) {
                    S.nodes[tm] = v;
                    S.prow[tm] = prow;
                    S.eoff[tm + 1] = incl;
                    R.t_ebeg[tm] = eb;
                }
                if (tm == 0) {
                    S.eoff[0] = 0;
                    S.pos0 = pos0; S.m = m; S.ne = ne; S.et0 = et0;
                }
                named_bar(BAR_META, META_THREADS);  // nodes, prow, eoff and t_ebeg of this pass are in place
                if (et0 == 0) stage_tile(S, m, tcount, tm);
                if (tm < et) {
                    const int e = et0 + tm;
                    int pr = 0, kid = 0, kpos = 0;
                    if (e < ne) {
                        int lo_r = 0, hi_r = NT_MAX;  // row owning edge e: largest r with eoff[r] <= e
                        while (hi_r - lo_r > 1) {
                            const int mid = (lo_r + hi_r) >> 1;
                            if (S.eoff[mid] <= e) lo_r = mid; else hi_r = mid;
                        }
                        pr = lo_r;
                        kid = d.child_idx[R.t_ebeg[pr] + (e - S.eoff[pr])];
                        if (d.debug && !dbg_ok(d.meta, CHECK_CHILD, kid, d.n_nodes, R.t_ebeg[pr] + (e - S.eoff[pr]))) kid = 0;  // reported; row 0 stands in
                        if (d.inv) kpos = d.inv[kid];
                        if (d.debug && d.inv && !dbg_ok(d.meta, CHECK_POSITION, kpos, d.n_nodes, kid)) kpos = 0;
                    }
                    S.ek_id[tm] = kid;
                    S.ek_pos[tm] = kpos;
                    S.ep[tm] = pr;
                }
                cp_async_wait_all();
                named_bar(BAR_META, META_THREADS);
                if (tm == 0) ptx::mbar_arrive(ptx::smem_u32(&R.bar_full[s]));
            }
        }
    }
}

// Grid barrier among the arithmetic warps of the participating CTAs (all of them arrive; thread 0 waits).
// `target` = barriers passed so far + 1, times the number of participating CTAs, on the monotonically increasing
// counter meta[META_BARRIER].  Bounded by timeout_ns; on expiry the timeout word is raised (which releases every
// other waiter) and *abort is set.  Returns with all MAIN_THREADS threads synchronised, and the same verdict in all
// of them: false when the wait was given up here or *abort was seen raised by anybody.
// `counter` is meta[META_BARRIER] for a barrier over the whole grid, or the counter of one group of CTAs that walks its
// own trees (then `target` counts that group's CTAs only).
__device__ __forceinline__ bool main_grid_barrier(int32_t* meta, int32_t* counter, unsigned target, unsigned long long timeout_ns,
                                                  volatile int* abort, int tid) {
    named_bar(BAR_MAIN, MAIN_THREADS);  // every store of the arithmetic warps is ordered before the release below
    if (tid == 0) {
        asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(counter) : "memory");
        const unsigned long long t0 = global_ns();
        unsigned spins = 0;
        while (true) {
            int seen;
            asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
            if ((unsigned)seen >= target) break;
            if ((++spins & 15u) == 0) {
                if (atomicAdd(&meta[META_TIMEOUT], 0) != 0) { *abort = 1; break; }
                if (global_ns() - t0 > timeout_ns) {
                    atomicExch(&meta[META_TIMEOUT], 1);
                    *abort = 1;
                    break;
                }
            }
        }
    }
    return !named_bar_any(BAR_MAIN, MAIN_THREADS, *abort != 0);
}

}  // namespace small
}  // namespace jdb
