// fp32 GEMM on the CUDA cores for the kernels that are not on the tensor-core path (the backward pass, the generic
// slot executor): C[m, n] (+)= sum_k A(m, k) B(k, n) with 128 x 128 x 16 tiles, 8 x 8 results per thread, 256 threads,
// two CTAs per SM.  Either operand is addressed by (row = m or n, k along the row) or by (row = k), with an optional
// row gather (a negative index reads as a row of zeros), the result rows can be scattered, a bias and one more row can
// be added, and the contraction can be split over CTAs whose partial sums are added atomically.
// Included by the translation units that launch it; everything lives in an unnamed namespace.
#pragma once

#include "common.cuh"

namespace jdb {
namespace {

constexpr int BM = 128, BN = 128, BK = 16, GEMM_THREADS = 256;
constexpr int LDS_ = BM + 4;   // row pitch of a staged tile (floats): keeps 16-byte alignment of the 4-wide reads

struct GemmArgs {
    const float* A;
    const float* B;
    float* C;
    long long lda, ldb, ldc;
    int M, N, K;
    const int* a_idx;     // row gather of A: along m (A_ROW_M) or along k
    const int* b_idx;     // row gather of B along k (B_ROW_K only)
    const int* c_idx;     // row scatter of C
    const float* bias;    // [N] added to every row (null = none)
    const float* add;     // rows added to the result: add[(add_idx[m] - add_off) * ldadd + n] (null = none)
    const int* add_idx;
    int add_off;
    long long ldadd;
    int beta;             // 1: C += result, 0: C = result
    int k_chunk;          // contraction range per blockIdx.z; more than one range: partial sums are added atomically
    int vec_a, vec_b;     // rows of A / B start on 16-byte boundaries and may be read four at a time
    int tn;               // tiles along n
};

__device__ __forceinline__ float sigmoidf_(float v) { return 1.0f / (1.0f + expf(-v)); }

// Eight elements of a tile for this thread.  ROW_MN: the matrix row is the tile's m (or n) index and k runs along it
// (thread: row t / 2, eight k from (t % 2) * 8); else the matrix row is k and m (or n) runs along it (thread: k = t / 16,
// eight m from (t % 16) * 8).
template <bool ROW_MN>
__device__ __forceinline__ void load_tile(const float* __restrict__ base, long long ld, const int* __restrict__ idx, int mn0,
                                          int MN, int k0, int kend, int vec, int t, float (&r)[8]) {
    int row, along0, along_end;
    bool row_ok;
    if (ROW_MN) {
        const int g = mn0 + (t >> 1);
        row_ok = g < MN;
        row = row_ok ? (idx ? idx[g] : g) : 0;
        if (row < 0) { row_ok = false; row = 0; }
        along0 = k0 + (t & 1) * 8;
        along_end = kend;
    } else {
        const int g = k0 + (t >> 4);
        row_ok = g < kend;
        row = row_ok ? (idx ? idx[g] : g) : 0;
        if (row < 0) { row_ok = false; row = 0; }
        along0 = mn0 + (t & 15) * 8;
        along_end = MN;
    }
    const float* p = base + (long long)row * ld + along0;
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        if (row_ok && vec && along0 + 4 * q + 4 <= along_end) {
            const float4 v = __ldg(reinterpret_cast<const float4*>(p + 4 * q));
            r[4 * q] = v.x; r[4 * q + 1] = v.y; r[4 * q + 2] = v.z; r[4 * q + 3] = v.w;
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) r[4 * q + i] = (row_ok && along0 + 4 * q + i < along_end) ? __ldg(p + 4 * q + i) : 0.0f;
        }
    }
}

template <bool ROW_MN>
__device__ __forceinline__ void store_tile(float (*S)[LDS_], int t, const float (&r)[8]) {
    if (ROW_MN) {
        const int mn = t >> 1, k = (t & 1) * 8;
#pragma unroll
        for (int i = 0; i < 8; ++i) S[k + i][mn] = r[i];
    } else {
        const int k = t >> 4, mn = (t & 15) * 8;
        *reinterpret_cast<float4*>(&S[k][mn]) = make_float4(r[0], r[1], r[2], r[3]);
        *reinterpret_cast<float4*>(&S[k][mn + 4]) = make_float4(r[4], r[5], r[6], r[7]);
    }
}

// C[m, n] (+)= sum_k A(m, k) B(k, n), fp32.  A(m, k) = A[row(m) * lda + k] (A_ROW_M) or A[row(k) * lda + m];
// B(k, n) = B[row(k) * ldb + n] (B_ROW_K) or B[n * ldb + k].
template <bool A_ROW_M, bool B_ROW_K>
__global__ void __launch_bounds__(GEMM_THREADS, 2) sgemm_kernel(GemmArgs g) {
    __shared__ __align__(16) float As[2][BK][LDS_];   // two buffers: the next tile is stored while this one is read,
    __shared__ __align__(16) float Bs[2][BK][LDS_];   // one barrier per K step
    const int t = threadIdx.x, ty = t >> 4, tx = t & 15;
    // tiles that share rows of A are neighbours in the grid: A reaches DRAM once, B (the smaller operand) stays in L2
    const int m0 = (blockIdx.x / g.tn) * BM, n0 = (blockIdx.x % g.tn) * BN;
    const int kbeg = blockIdx.z * g.k_chunk;
    const int kend = min(g.K, kbeg + g.k_chunk);
    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.0f;

    float ra[8], rb[8];
    if (kbeg < kend) {
        load_tile<A_ROW_M>(g.A, g.lda, g.a_idx, m0, g.M, kbeg, kend, g.vec_a, t, ra);
        load_tile<!B_ROW_K>(g.B, g.ldb, g.b_idx, n0, g.N, kbeg, kend, g.vec_b, t, rb);
        store_tile<A_ROW_M>(As[0], t, ra);
        store_tile<!B_ROW_K>(Bs[0], t, rb);
    }
    __syncthreads();
    int cur = 0;
    for (int k0 = kbeg; k0 < kend; k0 += BK) {
        const bool more = k0 + BK < kend;
        if (more) {   // the next tile's loads fly while this one is multiplied
            load_tile<A_ROW_M>(g.A, g.lda, g.a_idx, m0, g.M, k0 + BK, kend, g.vec_a, t, ra);
            load_tile<!B_ROW_K>(g.B, g.ldb, g.b_idx, n0, g.N, k0 + BK, kend, g.vec_b, t, rb);
        }
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            const float4 a0 = *reinterpret_cast<const float4*>(&As[cur][k][ty * 4]);
            const float4 a1 = *reinterpret_cast<const float4*>(&As[cur][k][64 + ty * 4]);
            const float4 b0 = *reinterpret_cast<const float4*>(&Bs[cur][k][tx * 4]);
            const float4 b1 = *reinterpret_cast<const float4*>(&Bs[cur][k][64 + tx * 4]);
            const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        if (more) {   // the other buffer was last read one step ago, before the barrier that ended that step
            store_tile<A_ROW_M>(As[cur ^ 1], t, ra);
            store_tile<!B_ROW_K>(Bs[cur ^ 1], t, rb);
        }
        __syncthreads();
        cur ^= 1;
    }
    if (kbeg >= kend && blockIdx.z > 0) return;

    const bool atomic = gridDim.z > 1;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int gm = m0 + (i < 4 ? ty * 4 + i : 64 + ty * 4 + (i - 4));
        if (gm >= g.M) continue;
        const long long crow = g.c_idx ? g.c_idx[gm] : gm;
        float* cp = g.C + crow * g.ldc;
        const float* ap = g.add ? g.add + (long long)(g.add_idx[gm] - g.add_off) * g.ldadd : nullptr;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int gn = n0 + (j < 4 ? tx * 4 + j : 64 + tx * 4 + (j - 4));
            if (gn >= g.N) continue;
            float v = acc[i][j];
            if (g.bias && blockIdx.z == 0) v += g.bias[gn];
            if (ap && blockIdx.z == 0) v += ap[gn];
            if (atomic) atomicAdd(cp + gn, v);
            else if (g.beta) cp[gn] += v;
            else cp[gn] = v;
        }
    }
}


bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

// min_steps: 0 = one CTA walks the whole contraction; else the contraction may be split over CTAs (partial sums added
// atomically) as long as every part keeps at least that many K steps, until the launch has two CTAs per SM.  A split
// result that is not accumulated (beta = 0) must be dense and is zeroed first.
template <bool A_ROW_M, bool B_ROW_K>
jdb_status gemm(GemmArgs g, int min_steps, int n_sm, cudaStream_t st) {
    if (g.M <= 0 || g.N <= 0) return JDB_OK;
    g.vec_a = aligned16(g.A) && g.lda % 4 == 0;
    g.vec_b = aligned16(g.B) && g.ldb % 4 == 0;
    const int tm = ceil_div(g.M, BM), tn = ceil_div(g.N, BN);
    const long long tiles = (long long)tm * tn;
    int splits = 1;
    if (min_steps > 0 && tiles < 2LL * n_sm) {
        // the number of parts that fills whole waves of two CTAs per SM best (fewest parts among equals)
        const long long most = (g.K + (long long)min_steps * BK - 1) / ((long long)min_steps * BK);
        double best = 0.0;
        for (long long sp = 1; sp <= most && sp <= 64; ++sp) {
            const long long ctas = tiles * sp, waves = (ctas + 2 * n_sm - 1) / (2 * n_sm);
            const double fill = (double)ctas / (double)(waves * 2 * n_sm);
            if (fill > best + 0.02) { best = fill; splits = (int)sp; }
        }
    }
    g.k_chunk = g.K <= 0 ? BK : ceil_div(ceil_div(g.K, splits), BK) * BK;
    splits = g.K <= 0 ? 1 : ceil_div(g.K, g.k_chunk);
    if (tiles > 0x7fffffffLL || splits > 65535) return JDB_ERR_UNSUPPORTED;
    g.tn = tn;
    if (splits > 1 && !g.beta) {
        if (g.c_idx || g.ldc != g.N) return JDB_ERR_UNSUPPORTED;
        JDB_CUDA_TRY(cudaMemsetAsync(g.C, 0, (size_t)g.M * g.N * sizeof(float), st));
    }
    sgemm_kernel<A_ROW_M, B_ROW_K><<<dim3((unsigned)tiles, 1, splits), GEMM_THREADS, 0, st>>>(g);
    JDB_CUDA_TRY(cudaGetLastError());
    return JDB_OK;
}


}  // namespace
}  // namespace jdb
