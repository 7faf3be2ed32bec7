// Launch counts of Section 3 of the paper on the GPU: how many launches a batch of trees costs when cells are batched
// whole (cells merge only when depth and number of children agree) and when operators are batched (29 of a cell's 33
// operators merge across a whole depth, the 4 that depend on the number of children merge per (depth, number of
// children)).  Both batched counts follow from the number of distinct (depth, number of children) pairs, which one
// pass over the nodes counts with an open-addressing set of 64-bit keys in the caller's scratch:
//     cells batched     = pairs
//     operators batched = sum over depths (29 + 4 * kinds at that depth) = 29 * n_levels + 4 * pairs
#include "common.cuh"

namespace jdb {
namespace {

constexpr unsigned long long EMPTY_KEY = ~0ull;

__global__ void pair_count_kernel(const int32_t* __restrict__ child_ptr, const int32_t* __restrict__ depth, int N,
                                  unsigned long long* table, unsigned long long mask, unsigned long long* n_pairs) {
    const int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= N) return;
    const unsigned long long key = ((unsigned long long)(uint32_t)depth[v] << 32) | (uint32_t)(child_ptr[v + 1] - child_ptr[v]);
    unsigned long long h = key * 0x9E3779B97F4A7C15ull;
    h ^= h >> 29;
    // the table has at least twice as many places as there are nodes, so a free place is met long before the bound
    for (unsigned long long probe = 0; probe <= mask; ++probe) {
        const unsigned long long i = (h + probe) & mask;
        const unsigned long long seen = table[i];
        if (seen == key) return;
        if (seen == EMPTY_KEY) {
            const unsigned long long old = atomicCAS(&table[i], EMPTY_KEY, key);
            if (old == EMPTY_KEY) {
                atomicAdd(n_pairs, 1ull);
                return;
            }
            if (old == key) return;
        }
    }
}

unsigned long long table_places(int32_t n_nodes) {
    unsigned long long p = 1024;
    while (p < 2ull * (unsigned long long)(n_nodes > 0 ? n_nodes : 1)) p <<= 1;
    return p;
}

}  // namespace
}  // namespace jdb

using namespace jdb;

extern "C" {

size_t jdb_launch_counts_workspace_bytes(int32_t n_nodes) { return (size_t)(table_places(n_nodes) + 1) * sizeof(unsigned long long); }

jdb_status jdb_launch_counts(const jdb_forest* forest, const jdb_sched* sched, jdb_launch_stats* out, void* ws, size_t ws_bytes,
                             void* stream) {
    cudaStream_t st = (cudaStream_t)stream;
    if (!forest || !sched || !out || forest->n_nodes < 0) return JDB_ERR_INVALID_ARG;
    const int N = forest->n_nodes;
    *out = jdb_launch_stats{};
    if (N == 0) return JDB_OK;
    if (!forest->child_ptr || !sched->depth || !sched->meta || !ws || ((uintptr_t)ws & 7) != 0) return JDB_ERR_INVALID_ARG;
    if (ws_bytes < jdb_launch_counts_workspace_bytes(N)) return JDB_ERR_WORKSPACE;
    const unsigned long long places = table_places(N);
    unsigned long long* table = (unsigned long long*)ws;
    unsigned long long* n_pairs = table + places;
    JDB_CUDA_TRY(cudaMemsetAsync(table, 0xFF, places * sizeof(unsigned long long), st));
    JDB_CUDA_TRY(cudaMemsetAsync(n_pairs, 0, sizeof(unsigned long long), st));
    pair_count_kernel<<<ceil_div(N, 256), 256, 0, st>>>(forest->child_ptr, sched->depth, N, table, places - 1, n_pairs);
    JDB_CUDA_TRY(cudaGetLastError());
    unsigned long long pairs = 0;
    int32_t meta[JDB_META_INTS];
    JDB_CUDA_TRY(cudaMemcpyAsync(&pairs, n_pairs, sizeof(pairs), cudaMemcpyDeviceToHost, st));
    JDB_CUDA_TRY(cudaMemcpyAsync(meta, sched->meta, sizeof(meta), cudaMemcpyDeviceToHost, st));
    JDB_CUDA_TRY(cudaStreamSynchronize(st));
    if (meta[META_ERROR] != 0 || meta[META_UNFINISHED] != 0) return JDB_ERR_NOT_A_FOREST;
    out->cells_unbatched = N;
    out->cells_batched = (int64_t)pairs;
    out->ops_unbatched = 33LL * N;
    out->ops_batched = 29LL * meta[META_N_LEVELS] + 4LL * (int64_t)pairs;
    out->n_levels = meta[META_N_LEVELS];
    return JDB_OK;
}

}  // extern "C"
