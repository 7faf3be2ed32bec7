// Prefix sums over one int per element, in three steps: per-block totals, one CTA that turns the totals into block
// offsets, and a second pass of the caller's kernel that adds its block's offset; and what the fp32 kernels outside the
// tensor-core path build with them: the child edges of a forest numbered in the order of a node permutation ("edge
// slots": the children of perm[0], then of perm[1], ...), and the sum of the children's h per node.
#pragma once

#include "common.cuh"

namespace jdb {
namespace {

constexpr int SCAN_BLOCK = 1024;

// exclusive scan of one value per thread over a block of SCAN_BLOCK threads; returns the thread's offset, total in `total`
__device__ __forceinline__ int block_exclusive_scan(int v, int& total) {
    __shared__ int warp_sum[32];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += o;
    }
    if (lane == 31) warp_sum[w] = incl;
    __syncthreads();
    if (w == 0) {
        int s = warp_sum[lane];
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int o = __shfl_up_sync(0xffffffffu, s, d);
            if (lane >= d) s += o;
        }
        warp_sum[lane] = s;
    }
    __syncthreads();
    total = warp_sum[31];
    const int before = w > 0 ? warp_sum[w - 1] : 0;
    __syncthreads();
    return before + incl - v;
}

// one CTA turns the block sums into block offsets (in place)
__global__ void __launch_bounds__(SCAN_BLOCK) block_sums_scan_kernel(int* block_sum, int n_blocks) {
    __shared__ int carry;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (int b0 = 0; b0 < n_blocks; b0 += SCAN_BLOCK) {
        const int i = b0 + threadIdx.x;
        const int v = i < n_blocks ? block_sum[i] : 0;
        int total;
        const int off = block_exclusive_scan(v, total);
        const int base = carry;
        if (i < n_blocks) block_sum[i] = base + off;
        __syncthreads();
        if (threadIdx.x == 0) carry = base + total;
        __syncthreads();
    }
}

// ---- edge slots in the order of a node permutation -----------------------------------------------------------------

__device__ __forceinline__ int child_count(const int32_t* child_ptr, const int32_t* perm, int p, int n) {
    if (p >= n) return 0;
    const int j = perm[p];
    return child_ptr[j + 1] - child_ptr[j];
}

__global__ void __launch_bounds__(SCAN_BLOCK) slot_count_kernel(const int32_t* child_ptr, const int32_t* perm, int n, int* block_sum) {
    const int p = blockIdx.x * SCAN_BLOCK + threadIdx.x;
    int total;
    block_exclusive_scan(child_count(child_ptr, perm, p, n), total);
    if (threadIdx.x == 0) block_sum[blockIdx.x] = total;
}

// edge_ptr[p] = edge slots before position p; per slot: the child's node id and the parent's position
__global__ void __launch_bounds__(SCAN_BLOCK) slot_fill_kernel(const int32_t* child_ptr, const int32_t* child_idx, const int32_t* perm,
                                                               int n, int n_edges, const int* block_off, int* edge_ptr,
                                                               int* slot_child, int* slot_ppos) {
    const int p = blockIdx.x * SCAN_BLOCK + threadIdx.x;
    const int cnt = child_count(child_ptr, perm, p, n);
    int total;
    const int off = block_off[blockIdx.x] + block_exclusive_scan(cnt, total);
    if (p <= n) edge_ptr[p] = off;   // p == n: the total
    if (p < n && cnt > 0) {
        const int e0 = child_ptr[perm[p]];
        for (int k = 0; k < cnt; ++k) {
            if (off + k < n_edges) {
                slot_child[off + k] = child_idx[e0 + k];
                slot_ppos[off + k] = p;
            }
        }
    }
}

// lv[l] = level_ptr[l], lv[L + 1 + l] = edge slots before level l, l = 0 .. L
__global__ void level_table_kernel(const int32_t* level_ptr, const int* edge_ptr, int n_levels, int* lv) {
    const int l = blockIdx.x * blockDim.x + threadIdx.x;
    if (l <= n_levels) {
        lv[l] = level_ptr[l];
        lv[n_levels + 1 + l] = edge_ptr[level_ptr[l]];
    }
}

// HS[r] = sum of the children's h of the internal node at position n_leaves + r (child-list order)
__global__ void child_sum_f32_kernel(const int32_t* __restrict__ child_ptr, const int32_t* __restrict__ child_idx,
                                     const int32_t* __restrict__ perm, int n_leaves, int n_int, int H,
                                     const float* __restrict__ h, long long ldh, float* __restrict__ HS) {
    const int r = blockIdx.x * blockDim.y + threadIdx.y;
    if (r >= n_int) return;
    const int j = perm[n_leaves + r];
    const int e0 = child_ptr[j], e1 = child_ptr[j + 1];
    for (int col = threadIdx.x; col < H; col += blockDim.x) {
        float s = 0.0f;
        for (int e = e0; e < e1; ++e) s += h[(long long)child_idx[e] * ldh + col];
        HS[(long long)r * H + col] = s;
    }
}

}  // namespace
}  // namespace jdb
