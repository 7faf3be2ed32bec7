// Partition of a forest by tree, for the cooperative level loop.
//
// No edge crosses trees (the per-sample graphs of Section 1 are independent), so a set of CTAs that owns whole trees
// can walk its trees through all their levels without ever waiting for the rest of the grid: the depth order of
// Section 4.2 has to hold inside a tree only.  This file assigns every tree to one of G groups, balanced on node
// count, and orders the nodes by (depth, group), so that the nodes a group has on a level are one contiguous range:
//
//   tree_parent    parent[] from the child lists
//   tree_root      root of every node (a bounded climb of at most n_levels steps) and the size of every tree
//   tree_place     every root takes an interval of the forest's node count as long as its tree (one atomic addition:
//                  the order of the trees is whatever order the roots arrive in, which balance does not care about)
//   tree_assign    group of a node = the G-quantile the midpoint of its tree's interval falls into; counts per (depth, group)
//   tree_offsets   running sum of those counts: goff[depth * G + group]
//   tree_scatter   gperm: node ids ordered by (depth, group); the order inside a range is arbitrary (nodes of one
//                  depth are independent, and a node's own arithmetic does not depend on its neighbours in a tile)
#include "common.cuh"

namespace jdb {
namespace {

constexpr int PT = 256;

__global__ void tree_parent_kernel(const int32_t* __restrict__ cp, const int32_t* __restrict__ ci, int N, int32_t* parent) {
    const int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= N) return;
    for (int e = cp[v]; e < cp[v + 1]; ++e) {
        const int k = ci[e];
        if (k >= 0 && k < N) parent[k] = v;
    }
}

__global__ void tree_root_kernel(const int32_t* __restrict__ parent, int N, const int32_t* __restrict__ meta, int32_t* root,
                                 int32_t* tsize) {
    const int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= N) return;
    const int limit = meta[META_N_LEVELS];   // a node is at most n_levels - 1 steps below its root
    int u = v;
    for (int it = 0; it < limit; ++it) {
        const int p = parent[u];
        if (p < 0) break;
        u = p;
    }
    root[v] = u;
    atomicAdd(&tsize[u], 1);
}

// exclusive running sum of `n` ints in place, one CTA of 1024 threads walking chunks of 1024
__global__ void __launch_bounds__(1024) scan_kernel(int32_t* data, long long n) {
    __shared__ int wsum[32];
    __shared__ int carry_s;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    for (long long base = 0; base < n; base += 1024) {
        const long long i = base + threadIdx.x;
        const int x = i < n ? data[i] : 0;
        int incl = x;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += y;
        }
        if (lane == 31) wsum[w] = incl;
        __syncthreads();
        if (w == 0) {
            int t = wsum[lane];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int y = __shfl_up_sync(0xffffffffu, t, o);
                if (lane >= o) t += y;
            }
            wsum[lane] = t;
        }
        __syncthreads();
        if (w > 0) incl += wsum[w - 1];
        const int carry = carry_s;
        if (i < n) data[i] = incl - x + carry;
        __syncthreads();
        if (threadIdx.x == 1023) carry_s = carry + incl;
        __syncthreads();
    }
}

__global__ void tree_place_kernel(const int32_t* __restrict__ parent, const int32_t* __restrict__ tsize, int N, int32_t* tstart,
                                  int32_t* running) {
    const int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= N || parent[v] >= 0) return;
    tstart[v] = atomicAdd(running, tsize[v]);
}

__global__ void tree_assign_kernel(const int32_t* __restrict__ root, const int32_t* __restrict__ tstart, const int32_t* __restrict__ tsize_copy,
                                   const int32_t* __restrict__ depth, int N, int G, long long table_entries, int32_t* grp, int32_t* cnt) {
    const int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= N) return;
    const int r = root[v];
    const long long mid = (long long)tstart[r] + (tsize_copy[r] >> 1);
    int g = (int)(mid * G / N);
    g = g < 0 ? 0 : (g >= G ? G - 1 : g);
    grp[v] = g;
    const long long key = (long long)depth[v] * G + g;
    if (key >= 0 && key < table_entries) atomicAdd(&cnt[key], 1);
}

__global__ void tree_scatter_kernel(const int32_t* __restrict__ grp, const int32_t* __restrict__ depth, int N, int G, long long table_entries,
                                    const int32_t* __restrict__ goff, int32_t* cursor, int32_t* gperm) {
    const int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= N) return;
    const long long key = (long long)depth[v] * G + grp[v];
    if (key < 0 || key >= table_entries) return;
    const int pos = goff[key] + atomicAdd(&cursor[key], 1);
    if (pos >= 0 && pos < N) gperm[pos] = v;
}

}  // namespace

size_t partition_ws_bytes(int32_t n_nodes) {
    const size_t n = (size_t)(n_nodes > 0 ? n_nodes : 1);
    // parent, root, tsize, tstart, grp, gperm; the (depth, group) table twice (offsets, cursors) and one spare entry;
    // one barrier counter per group
    return 6 * align_up(n * 4, 256) + 2 * align_up(((size_t)PARTITION_TABLE_MAX + 1) * 4, 256) + align_up(PARTITION_MAX_GROUPS * 4, 256);
}

jdb_status partition_enqueue(const ForwardArgs& fa, const int32_t* depth, int n_levels, int G, void* ws, Partition* out, cudaStream_t st) {
    const int N = fa.n_nodes;
    const size_t n = (size_t)N;
    if ((long long)n_levels * G > PARTITION_TABLE_MAX || G > PARTITION_MAX_GROUPS || G < 1) return JDB_ERR_UNSUPPORTED;
    char* p = (char*)ws;
    auto take = [&](size_t bytes) { char* q = p; p += align_up(bytes, 256); return q; };
    int32_t* parent = (int32_t*)take(n * 4);
    int32_t* root = (int32_t*)take(n * 4);
    int32_t* tsize = (int32_t*)take(n * 4);
    int32_t* tstart = (int32_t*)take(n * 4);
    int32_t* grp = (int32_t*)take(n * 4);
    int32_t* gperm = (int32_t*)take(n * 4);
    int32_t* goff = (int32_t*)take(((size_t)PARTITION_TABLE_MAX + 1) * 4);
    int32_t* cursor = (int32_t*)take(((size_t)PARTITION_TABLE_MAX + 1) * 4);
    int32_t* gbar = (int32_t*)take(PARTITION_MAX_GROUPS * 4);
    const long long entries = (long long)n_levels * G;
    JDB_CUDA_TRY(cudaMemsetAsync(parent, 0xFF, n * 4, st));
    JDB_CUDA_TRY(cudaMemsetAsync(tsize, 0, n * 4, st));
    JDB_CUDA_TRY(cudaMemsetAsync(goff, 0, ((size_t)entries + 1) * 4, st));
    JDB_CUDA_TRY(cudaMemsetAsync(cursor, 0, ((size_t)entries + 1) * 4, st));
    JDB_CUDA_TRY(cudaMemsetAsync(gbar, 0, (size_t)G * 4, st));
    const int blocks = ceil_div(N, PT);
    tree_parent_kernel<<<blocks, PT, 0, st>>>(fa.child_ptr, fa.child_idx, N, parent);
    tree_root_kernel<<<blocks, PT, 0, st>>>(parent, N, fa.meta, root, tsize);
    tree_place_kernel<<<blocks, PT, 0, st>>>(parent, tsize, N, tstart, cursor + entries);   // the spare table entry is the running total
    tree_assign_kernel<<<blocks, PT, 0, st>>>(root, tstart, tsize, depth, N, G, entries, grp, goff);
    scan_kernel<<<1, 1024, 0, st>>>(goff, entries + 1);
    tree_scatter_kernel<<<blocks, PT, 0, st>>>(grp, depth, N, G, entries, goff, cursor, gperm);
    JDB_CUDA_TRY(cudaGetLastError());
    out->gperm = gperm;
    out->goff = goff;
    out->gbar = gbar;
    out->G = G;
    return JDB_OK;
}

}  // namespace jdb
