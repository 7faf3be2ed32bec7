// Backward pass of the batched Child-Sum Tree-LSTM over the depth table, levels in DESCENDING order (the training
// loop of Section 4.3 calls backward() inside the batching scope; Section 5 reports training next to inference).
//
// A node's gradient is complete once its one parent is done, so the sweep runs from the top level down.  Only the
// two products that hand a gradient to the children (through U_iou and U_f) depend on that order; everything else is
// one batch over the whole forest:
//   1. all pre-activations again (W x + b for every node, + U_iou h~ for internal nodes, U_f h_k for every edge):
//      every h is known after the forward pass, so these are three GEMMs over the whole forest, not per level;
//   2. per level, top down: the cell's pointwise derivative (dz of the four gates, dc handed to the children), then
//      dh_k += U_iou^T dz_iou(parent) + U_f^T dz_f(edge): two GEMMs over the level's nodes and edge slots;
//   3. the parameter gradients as four GEMMs whose contraction runs over all nodes or all edges (split over CTAs,
//      partial sums added atomically), the bias gradient as column sums, and dx = dz W.
// Everything is fp32 on the CUDA cores: one tiled GEMM kernel (128 x 128 x 16 tiles, 8 x 8 per thread) with row
// gathers on either operand, a row scatter on the result and an optional split of the contraction.
#include <vector>

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
        along0 = k0 + (t & 1) * 8;
        along_end = kend;
    } else {
        const int g = k0 + (t >> 4);
        row_ok = g < kend;
        row = row_ok ? (idx ? idx[g] : g) : 0;
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
    __shared__ __align__(16) float As[BK][LDS_];
    __shared__ __align__(16) float Bs[BK][LDS_];
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
    }
    for (int k0 = kbeg; k0 < kend; k0 += BK) {
        store_tile<A_ROW_M>(As, t, ra);
        store_tile<!B_ROW_K>(Bs, t, rb);
        __syncthreads();
        if (k0 + BK < kend) {   // the next tile's loads fly while this one is multiplied
            load_tile<A_ROW_M>(g.A, g.lda, g.a_idx, m0, g.M, k0 + BK, kend, g.vec_a, t, ra);
            load_tile<!B_ROW_K>(g.B, g.ldb, g.b_idx, n0, g.N, k0 + BK, kend, g.vec_b, t, rb);
        }
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            const float4 a0 = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
            const float4 a1 = *reinterpret_cast<const float4*>(&As[k][64 + ty * 4]);
            const float4 b0 = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
            const float4 b1 = *reinterpret_cast<const float4*>(&Bs[k][64 + tx * 4]);
            const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
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

// ---- tables: edge slots in level order ------------------------------------------------------------------------------

constexpr int SCAN_BLOCK = 1024;
constexpr int SWEEP_STEPS = 2;   // least K steps per part when a level's GEMM is split to fill the SMs

__device__ __forceinline__ int child_count(const int32_t* child_ptr, const int32_t* perm, int p, int n) {
    if (p >= n) return 0;
    const int j = perm[p];
    return child_ptr[j + 1] - child_ptr[j];
}

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

__global__ void __launch_bounds__(SCAN_BLOCK) slot_count_kernel(const int32_t* child_ptr, const int32_t* perm, int n, int* block_sum) {
    const int p = blockIdx.x * SCAN_BLOCK + threadIdx.x;
    int total;
    block_exclusive_scan(child_count(child_ptr, perm, p, n), total);
    if (threadIdx.x == 0) block_sum[blockIdx.x] = total;
}

// one CTA turns the block sums into block offsets (in place)
__global__ void __launch_bounds__(SCAN_BLOCK) slot_scan_kernel(int* block_sum, int n_blocks) {
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

// ---- pointwise kernels ----------------------------------------------------------------------------------------------

// dH = grad_h, dC = grad_c (or 0): the running gradients of every node's state
__global__ void init_grad_kernel(const float* __restrict__ gh, const float* __restrict__ gc, long long ldg, int n, int H,
                                 float* __restrict__ dH, float* __restrict__ dC) {
    const long long total = (long long)n * H;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const long long v = i / H;
        const int col = (int)(i - v * H);
        dH[i] = gh ? gh[v * ldg + col] : 0.0f;
        dC[i] = gc ? gc[v * ldg + col] : 0.0f;
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

// The cell's pointwise derivative for the nodes at positions [lo, hi).  Z rows (node order) hold the pre-activations
// (i, o, u, f blocks of H) on entry and dz on exit (the f block: the sum over the children); FE rows (edge slots) hold
// U_f h_k on entry and dz_f of the edge on exit; dC of every child receives its share.
__global__ void cell_backward_kernel(const int32_t* __restrict__ perm, const int* __restrict__ edge_ptr,
                                     const int* __restrict__ slot_child, int lo, int hi, int H, float* __restrict__ Z,
                                     float* __restrict__ FE, const float* __restrict__ c, long long ldh,
                                     const float* __restrict__ dH, float* __restrict__ dC) {
    const int p = lo + blockIdx.x * blockDim.y + threadIdx.y;
    if (p >= hi) return;
    const int j = perm[p];
    const int s0 = edge_ptr[p], s1 = edge_ptr[p + 1];
    float* z = Z + (long long)j * 4 * H;
    for (int col = threadIdx.x; col < H; col += blockDim.x) {
        const float i = sigmoidf_(z[col]), o = sigmoidf_(z[H + col]), u = tanhf(z[2 * H + col]);
        const float t = tanhf(c[(long long)j * ldh + col]);
        const float dh = dH[(long long)j * H + col];
        const float dcj = dC[(long long)j * H + col] + dh * o * (1.0f - t * t);
        z[col] = dcj * u * i * (1.0f - i);
        z[H + col] = dh * t * o * (1.0f - o);
        z[2 * H + col] = dcj * i * (1.0f - u * u);
        const float zf = z[3 * H + col];
        float sum = 0.0f;
        for (int s = s0; s < s1; ++s) {
            const int k = slot_child[s];
            const float f = sigmoidf_(zf + FE[(long long)s * H + col]);
            const float dzf = dcj * c[(long long)k * ldh + col] * f * (1.0f - f);
            dC[(long long)k * H + col] += dcj * f;   // a child has one parent: no other thread touches this element
            FE[(long long)s * H + col] = dzf;
            sum += dzf;
        }
        z[3 * H + col] = sum;
    }
}

// out[col] += sum over rows of Z[row, col]
__global__ void column_sum_kernel(const float* __restrict__ Z, int n, int cols, int rows_per_block, float* __restrict__ out) {
    const int col = blockIdx.x * blockDim.x + threadIdx.x;
    if (col >= cols) return;
    const int r0 = blockIdx.y * rows_per_block, r1 = min(n, r0 + rows_per_block);
    float s[4] = {0.0f, 0.0f, 0.0f, 0.0f};   // four loads in flight per thread
    int r = r0;
    for (; r + 4 <= r1; r += 4) {
#pragma unroll
        for (int q = 0; q < 4; ++q) s[q] += Z[(long long)(r + q) * cols + col];
    }
    for (; r < r1; ++r) s[0] += Z[(long long)r * cols + col];
    atomicAdd(out + col, (s[0] + s[1]) + (s[2] + s[3]));
}

// ---- host -----------------------------------------------------------------------------------------------------------

struct BwdWorkspace {
    float *Z, *HS, *FE, *DHS, *dH, *dC;
    int *edge_ptr, *slot_child, *slot_ppos, *block_sum, *lv;
    size_t total;
};

BwdWorkspace carve(void* ws, long long n, long long e, long long ni, int H) {
    BwdWorkspace w{};
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return (char*)ws + o; };
    w.Z = (float*)take((size_t)n * 4 * H * sizeof(float));
    w.HS = (float*)take((size_t)ni * H * sizeof(float));
    w.DHS = (float*)take((size_t)ni * H * sizeof(float));
    w.FE = (float*)take((size_t)e * H * sizeof(float));
    w.dH = (float*)take((size_t)n * H * sizeof(float));
    w.dC = (float*)take((size_t)n * H * sizeof(float));
    w.edge_ptr = (int*)take((size_t)(n + 1) * sizeof(int));
    w.slot_child = (int*)take((size_t)e * sizeof(int));
    w.slot_ppos = (int*)take((size_t)e * sizeof(int));
    w.block_sum = (int*)take((size_t)(n / SCAN_BLOCK + 2) * sizeof(int));
    w.lv = (int*)take((size_t)(2 * (n + 2)) * sizeof(int));
    w.total = off;
    return w;
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

size_t backward_ws_bytes(int32_t n_nodes, int32_t n_edges, int32_t n_internal_bound, int32_t H) {
    return carve(nullptr, n_nodes, n_edges, n_internal_bound, H).total;
}

}  // namespace jdb

using namespace jdb;

extern "C" {

size_t jdb_treelstm_backward_workspace_bytes(int32_t n_nodes, int32_t n_edges, int32_t n_internal_bound, int32_t H) {
    if (n_nodes < 0 || n_edges < 0 || n_internal_bound < 0 || H <= 0) return 0;
    return backward_ws_bytes(n_nodes, n_edges, n_internal_bound, H);
}

jdb_status jdb_treelstm_backward(const jdb_forest* forest, const jdb_sched* sched, const float* x, int64_t ldx,
                                 const float* W, const float* U, const float* b, int32_t D, int32_t H, const float* h,
                                 const float* c, int64_t ldh, const float* grad_h, const float* grad_c, int64_t ldg,
                                 float* dW, float* dU, float* db, float* dx, int64_t lddx, void* ws, size_t ws_bytes,
                                 void* stream) {
    cudaStream_t st = (cudaStream_t)stream;
    if (!forest || !sched || forest->n_nodes < 0 || forest->n_edges < 0 || D <= 0 || H <= 0) return JDB_ERR_INVALID_ARG;
    if (!W || !U || !b || !dW || !dU || !db) return JDB_ERR_INVALID_ARG;
    const int n = forest->n_nodes, ne = forest->n_edges;
    JDB_CUDA_TRY(cudaMemsetAsync(dW, 0, (size_t)4 * H * D * sizeof(float), st));   // zeroed here: also what an empty forest returns
    JDB_CUDA_TRY(cudaMemsetAsync(dU, 0, (size_t)4 * H * H * sizeof(float), st));
    JDB_CUDA_TRY(cudaMemsetAsync(db, 0, (size_t)4 * H * sizeof(float), st));
    if (n == 0) return JDB_OK;
    if (!forest->child_ptr || (ne > 0 && !forest->child_idx) || !x || !h || !c || !grad_h) return JDB_ERR_INVALID_ARG;
    if (!sched->level_ptr || !sched->perm) return JDB_ERR_INVALID_ARG;
    if (sched->n_levels < 1 || sched->n_leaves < 0 || sched->n_leaves > n) return JDB_ERR_INVALID_ARG;   // needs jdb_schedule
    if (ldx < D || ldh < H || ldg < H || (dx && lddx < D)) return JDB_ERR_INVALID_ARG;
    if (!ws || ((uintptr_t)ws & 255) != 0) return JDB_ERR_INVALID_ARG;
    const int L = sched->n_levels, nl = sched->n_leaves, ni = n - nl;
    if (ws_bytes < backward_ws_bytes(n, ne, ni, H)) return JDB_ERR_WORKSPACE;
    DevInfo* di = dev_info();
    if (!di) return JDB_ERR_CUDA;
    const int n_sm = di->n_sm;
    BwdWorkspace w = carve(ws, n, ne, ni, H);
    const int32_t* perm = sched->perm;

    // edge slots in level order and the level table on the host
    const int n_blocks = n / SCAN_BLOCK + 1;   // covers position n too (the total)
    slot_count_kernel<<<n_blocks, SCAN_BLOCK, 0, st>>>(forest->child_ptr, perm, n, w.block_sum);
    slot_scan_kernel<<<1, SCAN_BLOCK, 0, st>>>(w.block_sum, n_blocks);
    slot_fill_kernel<<<n_blocks, SCAN_BLOCK, 0, st>>>(forest->child_ptr, forest->child_idx, perm, n, ne, w.block_sum, w.edge_ptr,
                                                     w.slot_child, w.slot_ppos);
    level_table_kernel<<<ceil_div(L + 1, 256), 256, 0, st>>>(sched->level_ptr, w.edge_ptr, L, w.lv);
    JDB_CUDA_TRY(cudaGetLastError());
    std::vector<int> lv(2 * (size_t)(L + 1));
    JDB_CUDA_TRY(cudaMemcpyAsync(lv.data(), w.lv, lv.size() * sizeof(int), cudaMemcpyDeviceToHost, st));
    JDB_CUDA_TRY(cudaStreamSynchronize(st));
    const int* lp = lv.data();
    const int* eo = lv.data() + (L + 1);
    if (lp[0] != 0 || lp[L] != n || lp[1] != nl || eo[L] != ne) return JDB_ERR_INVALID_ARG;   // not this forest's schedule
    for (int l = 0; l < L; ++l)
        if (lp[l + 1] < lp[l] || eo[l + 1] < eo[l]) return JDB_ERR_INVALID_ARG;

    const int grid_pw = (int)((((long long)n * H + 255) / 256) < 8LL * n_sm ? (((long long)n * H + 255) / 256) : 8LL * n_sm);
    init_grad_kernel<<<grid_pw, 256, 0, st>>>(grad_h, grad_c, ldg, n, H, w.dH, w.dC);
    const dim3 pw_block(H >= 128 ? 128 : (H > 32 ? 64 : 32), H >= 128 ? 2 : (H > 32 ? 4 : 8));
    if (ni > 0)
        child_sum_f32_kernel<<<ceil_div(ni, pw_block.y), pw_block, 0, st>>>(forest->child_ptr, forest->child_idx, perm, nl, ni, H, h, ldh, w.HS);
    JDB_CUDA_TRY(cudaGetLastError());

    jdb_status s;
    const float* U_f = U + (size_t)3 * H * H;
    {   // Z = x W^T + b for every node
        GemmArgs g{};
        g.A = x; g.lda = ldx; g.B = W; g.ldb = D; g.C = w.Z; g.ldc = 4LL * H; g.M = n; g.N = 4 * H; g.K = D; g.bias = b;
        if ((s = gemm<true, false>(g, 0, n_sm, st)) != JDB_OK) return s;
    }
    if (ni > 0) {   // Z[internal, i o u] += h~ U_iou^T
        GemmArgs g{};
        g.A = w.HS; g.lda = H; g.B = U; g.ldb = H; g.C = w.Z; g.ldc = 4LL * H; g.M = ni; g.N = 3 * H; g.K = H;
        g.c_idx = perm + nl; g.beta = 1;
        if ((s = gemm<true, false>(g, 0, n_sm, st)) != JDB_OK) return s;
    }
    if (ne > 0) {   // FE[slot] = U_f h_child
        GemmArgs g{};
        g.A = h; g.lda = ldh; g.a_idx = w.slot_child; g.B = U_f; g.ldb = H; g.C = w.FE; g.ldc = H; g.M = ne; g.N = H; g.K = H;
        if ((s = gemm<true, false>(g, 0, n_sm, st)) != JDB_OK) return s;
    }

    for (int l = L - 1; l >= 0; --l) {
        const int lo = lp[l], hi = lp[l + 1], m = hi - lo;
        if (m <= 0) continue;
        cell_backward_kernel<<<ceil_div(m, pw_block.y), pw_block, 0, st>>>(perm, w.edge_ptr, w.slot_child, lo, hi, H, w.Z, w.FE, c, ldh, w.dH, w.dC);
        JDB_CUDA_TRY(cudaGetLastError());
        const int e0 = eo[l], e1 = eo[l + 1];
        if (l == 0 || e1 <= e0) continue;
        {   // DHS[r] = dz_iou(node at lo + r) U_iou: what every child of that node receives through the child sum
            GemmArgs g{};
            g.A = w.Z; g.lda = 4LL * H; g.a_idx = perm + lo; g.B = U; g.ldb = H; g.C = w.DHS; g.ldc = H; g.M = m; g.N = H; g.K = 3 * H;
            if ((s = gemm<true, true>(g, SWEEP_STEPS, n_sm, st)) != JDB_OK) return s;
        }
        {   // dH[child] += dz_f(slot) U_f + DHS[parent]
            GemmArgs g{};
            g.A = w.FE + (size_t)e0 * H; g.lda = H; g.B = U_f; g.ldb = H; g.C = w.dH; g.ldc = H; g.M = e1 - e0; g.N = H; g.K = H;
            g.c_idx = w.slot_child + e0; g.beta = 1; g.add = w.DHS; g.add_idx = w.slot_ppos + e0; g.add_off = lo; g.ldadd = H;
            if ((s = gemm<true, true>(g, SWEEP_STEPS, n_sm, st)) != JDB_OK) return s;
        }
    }

    {   // dW = dz^T x
        GemmArgs g{};
        g.A = w.Z; g.lda = 4LL * H; g.B = x; g.ldb = ldx; g.C = dW; g.ldc = D; g.M = 4 * H; g.N = D; g.K = n;
        if ((s = gemm<false, true>(g, 16, n_sm, st)) != JDB_OK) return s;
    }
    {
        // about 32 CTAs of 128 threads per SM, at least 32 rows each
        const int col_blocks = ceil_div(4 * H, 128);
        int rows_per_block = ceil_div(n, ceil_div(32 * n_sm, col_blocks));
        if (rows_per_block < 32) rows_per_block = 32;
        column_sum_kernel<<<dim3(ceil_div(4 * H, 128), ceil_div(n, rows_per_block)), 128, 0, st>>>(w.Z, n, 4 * H, rows_per_block, db);
        JDB_CUDA_TRY(cudaGetLastError());
    }
    if (ni > 0) {   // dU_iou = dz_iou^T h~ over the internal nodes
        GemmArgs g{};
        g.A = w.Z; g.lda = 4LL * H; g.a_idx = perm + nl; g.B = w.HS; g.ldb = H; g.C = dU; g.ldc = H; g.M = 3 * H; g.N = H; g.K = ni;
        if ((s = gemm<false, true>(g, 16, n_sm, st)) != JDB_OK) return s;
    }
    if (ne > 0) {   // dU_f = sum over edges dz_f h_child^T
        GemmArgs g{};
        g.A = w.FE; g.lda = H; g.B = h; g.ldb = ldh; g.b_idx = w.slot_child; g.C = dU + (size_t)3 * H * H; g.ldc = H; g.M = H; g.N = H; g.K = ne;
        if ((s = gemm<false, true>(g, 16, n_sm, st)) != JDB_OK) return s;
    }
    if (dx) {   // dx = dz W
        GemmArgs g{};
        g.A = w.Z; g.lda = 4LL * H; g.B = W; g.ldb = D; g.C = dx; g.ldc = lddx; g.M = n; g.N = D; g.K = 4 * H;
        if ((s = gemm<true, true>(g, lddx == D ? SWEEP_STEPS : 0, n_sm, st)) != JDB_OK) return s;
    }
    return JDB_OK;
}

}  // extern "C"
