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
#include "scan.cuh"
#include "sgemm.cuh"

namespace jdb {
namespace {

// ---- tables: edge slots in level order ------------------------------------------------------------------------------

constexpr int SWEEP_STEPS = 2;   // least K steps per part when a level's GEMM is split to fill the SMs

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
    block_sums_scan_kernel<<<1, SCAN_BLOCK, 0, st>>>(w.block_sum, n_blocks);
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
