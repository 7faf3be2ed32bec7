// Relatedness head over pairs of root states (the scoring function of the paper's workload, Section 5, as defined by the
// Tree-LSTM model it cites): for a pair (h_L, h_R)
//     h_s = sig(W_x (h_L * h_R) + W_+ |h_L - h_R| + b_h),   p = softmax(W_p h_s + b_p),   y = sum_k k p_k.
// One CTA per group of four pairs (grid-stride): the pairs' feature vectors are built once in shared memory, one warp per
// hidden unit of the head takes the dot products of all four pairs from one coalesced read of the two weight rows, and
// the first four warps finish the K logits, the softmax and the expectation of one pair each.  fp32 throughout; sums run
// in a fixed order, so results are reproducible.
#include "common.cuh"

namespace jdb {
namespace {

constexpr int HEAD_THREADS = 256;
constexpr int HEAD_MAX_K = 32;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

constexpr int HEAD_PAIRS = 4;   // pairs per CTA pass: every weight row read serves four pairs

__global__ void __launch_bounds__(HEAD_THREADS) relatedness_kernel(const float* __restrict__ h, long long ldh, int n_nodes,
                                                                   const int32_t* __restrict__ left, const int32_t* __restrict__ right,
                                                                   int n_pairs, const float* __restrict__ Wx, const float* __restrict__ Wp,
                                                                   const float* __restrict__ bh, const float* __restrict__ Wq,
                                                                   const float* __restrict__ bq, int H, int Hs, int K,
                                                                   float* __restrict__ y, float* __restrict__ p, int32_t* bad) {
    extern __shared__ float sm[];
    float* fx = sm;                          // [HEAD_PAIRS][H]  h_L * h_R
    float* fp = fx + HEAD_PAIRS * H;         // [HEAD_PAIRS][H]  |h_L - h_R|
    float* hs = fp + HEAD_PAIRS * H;         // [HEAD_PAIRS][Hs]
    __shared__ int ok[HEAD_PAIRS];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = HEAD_THREADS / 32;
    const int n_groups = (n_pairs + HEAD_PAIRS - 1) / HEAD_PAIRS;
    for (int grp = blockIdx.x; grp < n_groups; grp += gridDim.x) {
        const int pair0 = grp * HEAD_PAIRS;
        for (int q = 0; q < HEAD_PAIRS; ++q) {
            const int pair = pair0 + q;
            int a = -1, b = -1;
            if (pair < n_pairs) { a = left[pair]; b = right[pair]; }
            const bool good = a >= 0 && a < n_nodes && b >= 0 && b < n_nodes;
            if (threadIdx.x == 0) {
                ok[q] = good;
                if (pair < n_pairs && !good) atomicExch(bad, 1);   // reported, the pair is skipped
            }
            for (int j = threadIdx.x; j < H; j += HEAD_THREADS) {
                const float u = good ? h[(long long)a * ldh + j] : 0.f, v = good ? h[(long long)b * ldh + j] : 0.f;
                fx[q * H + j] = u * v;
                fp[q * H + j] = fabsf(u - v);
            }
        }
        __syncthreads();
        for (int s = warp; s < Hs; s += n_warps) {
            const float* wx = Wx + (size_t)s * H;
            const float* wp = Wp + (size_t)s * H;
            float acc[HEAD_PAIRS];
#pragma unroll
            for (int q = 0; q < HEAD_PAIRS; ++q) acc[q] = 0.f;
            for (int j = lane; j < H; j += 32) {
                const float a = wx[j], b = wp[j];
#pragma unroll
                for (int q = 0; q < HEAD_PAIRS; ++q) acc[q] = fmaf(a, fx[q * H + j], fmaf(b, fp[q * H + j], acc[q]));
            }
#pragma unroll
            for (int q = 0; q < HEAD_PAIRS; ++q) {
                const float t = warp_sum(acc[q]);
                if (lane == 0) hs[q * Hs + s] = 1.f / (1.f + expf(-(t + bh[s])));
            }
        }
        __syncthreads();
        if (warp < HEAD_PAIRS && pair0 + warp < n_pairs && ok[warp]) {
            // warp q finishes pair q; lane k owns logit k (K <= 32)
            const int pair = pair0 + warp;
            float z = -INFINITY;
            if (lane < K) {
                float acc = bq[lane];
                for (int s = 0; s < Hs; ++s) acc = fmaf(Wq[(size_t)lane * Hs + s], hs[warp * Hs + s], acc);
                z = acc;
            }
            float m = z;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
            const float e = lane < K ? expf(z - m) : 0.f;
            const float tot = warp_sum(e);
            const float pk = e / tot;
            const float yk = warp_sum(pk * (float)(lane + 1));
            if (lane < K && p) p[(size_t)pair * K + lane] = pk;
            if (lane == 0) y[pair] = yk;
        }
        __syncthreads();
    }
}

}  // namespace
}  // namespace jdb

using namespace jdb;

extern "C" jdb_status jdb_relatedness_head(const float* h, int64_t ldh, int32_t n_nodes, const int32_t* left, const int32_t* right,
                                           int32_t n_pairs, const float* Wx, const float* Wp, const float* bh, const float* Wq,
                                           const float* bq, int32_t H, int32_t Hs, int32_t K, float* y, float* p, int32_t* bad_flag,
                                           void* stream) {
    if (n_pairs < 0 || n_nodes < 0 || H <= 0 || Hs <= 0 || K <= 0 || ldh < H) return JDB_ERR_INVALID_ARG;
    if (K > HEAD_MAX_K) return JDB_ERR_UNSUPPORTED;
    if (n_pairs == 0) return JDB_OK;
    if (!h || !left || !right || !Wx || !Wp || !bh || !Wq || !bq || !y || !bad_flag) return JDB_ERR_INVALID_ARG;
    const size_t smem = (size_t)HEAD_PAIRS * ((size_t)2 * H + Hs) * sizeof(float);
    if (smem > 48 * 1024) return JDB_ERR_UNSUPPORTED;
    DevInfo* di = dev_info();
    if (!di) return JDB_ERR_CUDA;
    const int n_groups = (n_pairs + HEAD_PAIRS - 1) / HEAD_PAIRS;
    const int grid = n_groups < di->n_sm * 8 ? n_groups : di->n_sm * 8;
    cudaStream_t st = (cudaStream_t)stream;
    JDB_CUDA_TRY(cudaMemsetAsync(bad_flag, 0, sizeof(int32_t), st));
    relatedness_kernel<<<grid, HEAD_THREADS, smem, st>>>(h, (long long)ldh, n_nodes, left, right, n_pairs, Wx, Wp, bh, Wq, bq, H, Hs, K,
                                                         y, p, bad_flag);
    JDB_CUDA_TRY(cudaGetLastError());
    return JDB_OK;
}
