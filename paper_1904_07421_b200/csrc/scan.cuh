// Prefix sums over one int per element, in three steps: per-block totals, one CTA that turns the totals into block
// offsets, and a second pass of the caller's kernel that adds its block's offset.
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

}  // namespace
}  // namespace jdb
