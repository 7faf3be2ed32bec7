// The depth table for nodes of several kinds (Section 4.2: a node is filed under its depth and a key made of its type,
// settings and argument layout; nodes that share both share a slot), and the execution of such a table for two kinds
// of cell, one batched launch sequence per slot in depth order (Section 4.3).
//
//   jdb_batch_plan     node ids ordered by (depth, key, id) by a stable radix sort of depth * n_keys + key (8 bits per
//                      pass, from the identity order), then the slot boundaries by a scan over "differs from the
//                      previous position";
//   jdb_cells_forward  per slot: W x + b of the slot's rows, the recurrent products of its cell kind (Child-Sum: child
//                      sums and U_f h_k per edge; N-ary: one product per child position), the cell's pointwise part.
// fp32 on the CUDA cores (the GEMM of sgemm.cuh with row gathers); the tensor-core path of the Child-Sum forward is
// jdb_treelstm_forward.
#include <vector>

#include "common.cuh"
#include "scan.cuh"
#include "sgemm.cuh"

namespace jdb {
namespace {

// ---- plan ---------------------------------------------------------------------------------------------------------

constexpr int RS_BITS = 8, RS_BINS = 1 << RS_BITS, RS_TB = 256, RS_TILE = 2048;

__global__ void composite_key_kernel(const int32_t* __restrict__ depth, const int32_t* __restrict__ key, int n, int n_keys,
                                     int32_t* __restrict__ comp, int* __restrict__ bad) {
    const int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= n) return;
    int k = key[v];
    if (k < 0 || k >= n_keys) {
        *bad = 1;
        k = 0;
    }
    comp[v] = depth[v] * n_keys + k;
}

__device__ __forceinline__ int digit_of(const int32_t* comp, int v, int pass) { return (comp[v] >> (RS_BITS * pass)) & (RS_BINS - 1); }

// per-block digit counts, bin-major: hist[bin * n_blocks + block]
__global__ void __launch_bounds__(RS_TB) radix_hist_kernel(int pass, const int32_t* __restrict__ src, const int32_t* __restrict__ comp,
                                                           int n, int32_t* __restrict__ hist, int n_blocks) {
    __shared__ int bins[RS_BINS];
    bins[threadIdx.x] = 0;
    __syncthreads();
    const int base = blockIdx.x * RS_TILE;
    for (int r = 0; r < RS_TILE / RS_TB; ++r) {
        const int idx = base + r * RS_TB + threadIdx.x;
        if (idx < n) atomicAdd(&bins[digit_of(comp, src ? src[idx] : idx, pass)], 1);
    }
    __syncthreads();
    hist[(size_t)threadIdx.x * n_blocks + blockIdx.x] = bins[threadIdx.x];
}

// exclusive scan of the counts in place (one CTA)
__global__ void __launch_bounds__(SCAN_BLOCK) radix_scan_kernel(int32_t* hist, long long total) {
    __shared__ int carry;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (long long b0 = 0; b0 < total; b0 += SCAN_BLOCK) {
        const long long i = b0 + threadIdx.x;
        const int v = i < total ? hist[i] : 0;
        int sum;
        const int off = block_exclusive_scan(v, sum);
        const int base = carry;
        if (i < total) hist[i] = base + off;
        __syncthreads();
        if (threadIdx.x == 0) carry = base + sum;
        __syncthreads();
    }
}

// stable scatter: a warp owns 256 consecutive elements of the tile and walks them 32 at a time, so the rank of an
// element among those of its digit is (earlier warps) + (earlier rounds of this warp) + (earlier lanes of this round)
__global__ void __launch_bounds__(RS_TB) radix_scatter_kernel(int pass, const int32_t* __restrict__ src, const int32_t* __restrict__ comp,
                                                              int n, const int32_t* __restrict__ hist, int n_blocks,
                                                              int32_t* __restrict__ dst) {
    constexpr int W = RS_TB / 32, ROUNDS = RS_TILE / RS_TB;
    __shared__ uint16_t cnt[W][RS_BINS];
    for (int i = threadIdx.x; i < W * RS_BINS; i += RS_TB) (&cnt[0][0])[i] = 0;
    __syncthreads();
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int base = blockIdx.x * RS_TILE + w * (RS_TILE / W);
    int vals[ROUNDS], digs[ROUNDS];
    uint16_t rank[ROUNDS];
#pragma unroll
    for (int r = 0; r < ROUNDS; ++r) {
        const int idx = base + r * 32 + lane;
        const bool valid = idx < n;
        const int v = valid ? (src ? src[idx] : idx) : 0;
        const int dg = valid ? digit_of(comp, v, pass) : -1;
        const unsigned peers = __match_any_sync(0xffffffffu, dg);
        const int leader = __ffs(peers) - 1;
        int first = 0;
        if (valid && lane == leader) {
            first = cnt[w][dg];
            cnt[w][dg] = (uint16_t)(first + __popc(peers));
        }
        first = __shfl_sync(0xffffffffu, first, leader);
        vals[r] = v;
        digs[r] = dg;
        rank[r] = (uint16_t)(first + __popc(peers & ((1u << lane) - 1u)));
        __syncwarp();
    }
    __syncthreads();
    {   // counts of the earlier warps of this block, per digit
        const int bin = threadIdx.x;
        int run = 0;
#pragma unroll
        for (int ww = 0; ww < W; ++ww) {
            const int t = cnt[ww][bin];
            cnt[ww][bin] = (uint16_t)run;
            run += t;
        }
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < ROUNDS; ++r)
        if (digs[r] >= 0) dst[hist[(size_t)digs[r] * n_blocks + blockIdx.x] + cnt[w][digs[r]] + rank[r]] = vals[r];
}

__device__ __forceinline__ int starts_slot(const int32_t* comp, const int32_t* perm, int p, int n) {
    if (p >= n) return 0;
    return (p == 0 || comp[perm[p]] != comp[perm[p - 1]]) ? 1 : 0;
}

__global__ void __launch_bounds__(SCAN_BLOCK) slot_start_count_kernel(const int32_t* comp, const int32_t* perm, int n, int* block_sum) {
    int total;
    block_exclusive_scan(starts_slot(comp, perm, blockIdx.x * SCAN_BLOCK + threadIdx.x, n), total);
    if (threadIdx.x == 0) block_sum[blockIdx.x] = total;
}

// out[0] = number of slots; slot s: first position, depth, key; slot_ptr[n_slots] = n
__global__ void __launch_bounds__(SCAN_BLOCK) slot_start_fill_kernel(const int32_t* comp, const int32_t* perm, int n, int n_keys,
                                                                     const int* block_off, int32_t* slot_ptr, int32_t* slot_depth,
                                                                     int32_t* slot_key, int* out) {
    const int p = blockIdx.x * SCAN_BLOCK + threadIdx.x;
    const int flag = starts_slot(comp, perm, p, n);
    int total;
    const int s = block_off[blockIdx.x] + block_exclusive_scan(flag, total);
    if (flag) {
        const int cv = comp[perm[p]];
        slot_ptr[s] = p;
        slot_depth[s] = cv / n_keys;
        slot_key[s] = cv % n_keys;
    }
    if (p == n) {   // the thread just past the last node holds the total
        slot_ptr[s] = n;
        out[0] = s;
    }
}

// ---- execution ------------------------------------------------------------------------------------------------------

constexpr int SLOT_STEPS = 2;   // least K steps per part when a slot's product is split to fill the SMs

// kid[l * n + p] = child l of the node at plan position p, or -1; *bad = 1 if an N-ary node has more children than its arity
__global__ void child_positions_kernel(const int32_t* __restrict__ child_ptr, const int32_t* __restrict__ child_idx,
                                       const int32_t* __restrict__ perm, const int32_t* __restrict__ key, const int32_t* __restrict__ arity_of,
                                       int n, int n_keys, int amax, int32_t* __restrict__ kid, int* __restrict__ bad) {
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= n) return;
    const int j = perm[p];
    const int k = key[j];
    const int a = (k >= 0 && k < n_keys) ? arity_of[k] : 0;   // 0: a Child-Sum cell (any number of children)
    const int e0 = child_ptr[j], cnt = child_ptr[j + 1] - e0;
    if (a > 0 && cnt > a) *bad = 1;
    for (int l = 0; l < amax; ++l) kid[(size_t)l * n + p] = (a > 0 && l < cnt && l < a) ? child_idx[e0 + l] : -1;
}

// Rows that have a child in position l, compacted in plan order (most nodes of an N-ary cell have fewer children
// than the arity, and a product over a position should not pay for the rows that have no child there):
// cptr[p] = such rows before position p; ckid / cpos = the child's node id and the row's position.
__global__ void __launch_bounds__(SCAN_BLOCK) position_count_kernel(const int32_t* __restrict__ kid_l, int n, int* block_sum) {
    const int p = blockIdx.x * SCAN_BLOCK + threadIdx.x;
    int total;
    block_exclusive_scan((p < n && kid_l[p] >= 0) ? 1 : 0, total);
    if (threadIdx.x == 0) block_sum[blockIdx.x] = total;
}

__global__ void __launch_bounds__(SCAN_BLOCK) position_fill_kernel(const int32_t* __restrict__ kid_l, int n, const int* block_off,
                                                                   int32_t* __restrict__ cptr, int32_t* __restrict__ ckid,
                                                                   int32_t* __restrict__ cpos) {
    const int p = blockIdx.x * SCAN_BLOCK + threadIdx.x;
    const int flag = (p < n && kid_l[p] >= 0) ? 1 : 0;
    int total;
    const int off = block_off[blockIdx.x] + block_exclusive_scan(flag, total);
    if (p <= n) cptr[p] = off;
    if (flag) {
        ckid[off] = kid_l[p];
        cpos[off] = p;
    }
}

// tab[(s * amax + l) * 2 + {0, 1}] = first compacted row of slot s in position l, and one past its last
__global__ void position_table_kernel(const int32_t* __restrict__ slot_ptr, const int32_t* __restrict__ cptr, int n, int n_slots,
                                      int amax, int32_t* __restrict__ tab) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_slots * amax) return;
    const int s = i / amax, l = i % amax;
    tab[2 * i] = cptr[(size_t)l * (n + 1) + slot_ptr[s]];
    tab[2 * i + 1] = cptr[(size_t)l * (n + 1) + slot_ptr[s + 1]];
}

// Child-Sum cell, pointwise part, for the nodes at plan positions [lo, lo + m): Z rows (slot-local) hold W x + b
// (+ U_iou h~ in the i, o, u blocks), FE rows (edge slots of the plan order) hold U_f h_k
__global__ void childsum_pointwise_kernel(const int32_t* __restrict__ perm, const int* __restrict__ edge_ptr,
                                          const int* __restrict__ slot_child, int lo, int m, int H, const float* __restrict__ Z,
                                          const float* __restrict__ FE, float* __restrict__ h, float* __restrict__ c, long long ldh) {
    const int r = blockIdx.x * blockDim.y + threadIdx.y;
    if (r >= m) return;
    const int j = perm[lo + r];
    const int s0 = edge_ptr[lo + r], s1 = edge_ptr[lo + r + 1];
    const float* z = Z + (long long)r * 4 * H;
    for (int col = threadIdx.x; col < H; col += blockDim.x) {
        const float i = sigmoidf_(z[col]), o = sigmoidf_(z[H + col]), u = tanhf(z[2 * H + col]);
        float cc = i * u;
        for (int s = s0; s < s1; ++s)
            cc += sigmoidf_(z[3 * H + col] + FE[(long long)s * H + col]) * c[(long long)slot_child[s] * ldh + col];
        c[(long long)j * ldh + col] = cc;
        h[(long long)j * ldh + col] = o * tanhf(cc);
    }
}

// N-ary cell, pointwise part: G rows (by plan position, (3 + arity) H wide) hold sum_l U^l h_l (absent for a slot of leaves)
__global__ void nary_pointwise_kernel(const int32_t* __restrict__ perm, const int32_t* __restrict__ kid, int n, int lo, int m, int H,
                                      int arity, const float* __restrict__ Z, const float* __restrict__ G, float* __restrict__ h,
                                      float* __restrict__ c, long long ldh) {
    const int r = blockIdx.x * blockDim.y + threadIdx.y;
    if (r >= m) return;
    const int j = perm[lo + r];
    const float* z = Z + (long long)r * 4 * H;
    const float* g = G ? G + (long long)(lo + r) * (3 + arity) * H : nullptr;
    for (int col = threadIdx.x; col < H; col += blockDim.x) {
        const float i = sigmoidf_(z[col] + (g ? g[col] : 0.0f));
        const float o = sigmoidf_(z[H + col] + (g ? g[H + col] : 0.0f));
        const float u = tanhf(z[2 * H + col] + (g ? g[2 * H + col] : 0.0f));
        float cc = i * u;
        if (g) {
            for (int k = 0; k < arity; ++k) {
                const int ch = kid[(size_t)k * n + lo + r];
                if (ch >= 0) cc += sigmoidf_(z[3 * H + col] + g[(3 + k) * H + col]) * c[(long long)ch * ldh + col];
            }
        }
        c[(long long)j * ldh + col] = cc;
        h[(long long)j * ldh + col] = o * tanhf(cc);
    }
}

// The Child-Sum cell's pointwise part on the packed fp32 layout (columns interleaved by gate: hidden unit j, gate g at
// 4 j + g): Z rows hold W x + b, T rows (absent for leaves) h~ U^T of which the forget column is not used, FE rows U_f h_k.
__global__ void childsum_pointwise_il_kernel(const int32_t* __restrict__ perm, const int* __restrict__ edge_ptr,
                                             const int* __restrict__ slot_child, int lo, int m, int H, const float* __restrict__ Z,
                                             const float* __restrict__ T, const float* __restrict__ FE, float* __restrict__ h,
                                             float* __restrict__ c, long long ldh) {
    const int r = blockIdx.x * blockDim.y + threadIdx.y;
    if (r >= m) return;
    const int j = perm[lo + r];
    const int s0 = edge_ptr[lo + r], s1 = edge_ptr[lo + r + 1];
    const float4* z = reinterpret_cast<const float4*>(Z + (long long)r * 4 * H);
    const float4* t = T ? reinterpret_cast<const float4*>(T + (long long)r * 4 * H) : nullptr;
    for (int col = threadIdx.x; col < H; col += blockDim.x) {
        float4 g = z[col];
        if (t) {
            const float4 u = t[col];
            g.x += u.x; g.y += u.y; g.z += u.z;
        }
        float cc = sigmoidf_(g.x) * tanhf(g.z);
        for (int s = s0; s < s1; ++s)
            cc += sigmoidf_(g.w + FE[(long long)s * H + col]) * c[(long long)slot_child[s] * ldh + col];
        c[(long long)j * ldh + col] = cc;
        h[(long long)j * ldh + col] = sigmoidf_(g.y) * tanhf(cc);
    }
}

struct PlanWorkspace {
    int32_t *comp, *tmp0, *tmp1, *hist;
    int *block_sum, *flags;   // flags[0] slot count, flags[1] bad key
    size_t total;
};
PlanWorkspace carve_plan(void* ws, long long n) {
    PlanWorkspace w{};
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return (char*)ws + o; };
    const size_t n_blocks = (size_t)(n / RS_TILE + 1);
    w.comp = (int32_t*)take((size_t)(n + 1) * sizeof(int32_t));
    w.tmp0 = (int32_t*)take((size_t)(n + 1) * sizeof(int32_t));
    w.tmp1 = (int32_t*)take((size_t)(n + 1) * sizeof(int32_t));
    w.hist = (int32_t*)take(RS_BINS * n_blocks * sizeof(int32_t));
    w.block_sum = (int*)take((size_t)(n / SCAN_BLOCK + 2) * sizeof(int));
    w.flags = (int*)take(4 * sizeof(int));
    w.total = off;
    return w;
}

struct CellsWorkspace {
    float *Z, *G, *HS, *FE;
    int *edge_ptr, *slot_child, *slot_ppos, *block_sum, *flags;
    int32_t *kid, *arity_of, *table, *cptr, *ckid, *cpos;
    size_t total;
};
CellsWorkspace carve_cells(void* ws, long long n, long long e, int H, int amax, int n_keys) {
    CellsWorkspace w{};
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return (char*)ws + o; };
    w.Z = (float*)take((size_t)n * 4 * H * sizeof(float));
    w.G = (float*)take((size_t)n * (3 + (amax > 0 ? amax : 1)) * H * sizeof(float));
    w.HS = (float*)take((size_t)n * H * sizeof(float));
    w.FE = (float*)take((size_t)e * H * sizeof(float));
    w.edge_ptr = (int*)take((size_t)(n + 1) * sizeof(int));
    w.slot_child = (int*)take((size_t)e * sizeof(int));
    w.slot_ppos = (int*)take((size_t)e * sizeof(int));
    w.block_sum = (int*)take((size_t)(n / SCAN_BLOCK + 2) * sizeof(int));
    w.flags = (int*)take(4 * sizeof(int));
    w.kid = (int32_t*)take((size_t)(amax > 0 ? amax : 1) * n * sizeof(int32_t));
    w.arity_of = (int32_t*)take((size_t)(n_keys > 0 ? n_keys : 1) * sizeof(int32_t));
    w.table = (int32_t*)take((size_t)2 * (amax > 0 ? amax : 1) * (n + 1) * sizeof(int32_t));
    w.cptr = (int32_t*)take((size_t)(amax > 0 ? amax : 1) * (n + 1) * sizeof(int32_t));
    w.ckid = (int32_t*)take((size_t)(amax > 0 ? amax : 1) * n * sizeof(int32_t));
    w.cpos = (int32_t*)take((size_t)(amax > 0 ? amax : 1) * n * sizeof(int32_t));
    w.total = off;
    return w;
}

}  // namespace

// ---- fp32 forward of the Child-Sum cell for hidden sizes beyond the cooperative kernel (forward_simt.cu calls this) ----
struct F32Workspace {
    float *Z, *T, *HS, *FE;
    int *edge_ptr, *slot_child, *slot_ppos, *block_sum, *lv;
    size_t total;
};
static F32Workspace carve_f32(void* ws, long long n, long long ni, int H) {
    F32Workspace w{};
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return (char*)ws + o; };
    w.Z = (float*)take((size_t)n * 4 * H * sizeof(float));
    w.T = (float*)take((size_t)ni * 4 * H * sizeof(float));
    w.HS = (float*)take((size_t)ni * H * sizeof(float));
    w.FE = (float*)take((size_t)n * H * sizeof(float));      // a forest has fewer edges than nodes
    w.edge_ptr = (int*)take((size_t)(n + 1) * sizeof(int));
    w.slot_child = (int*)take((size_t)n * sizeof(int));
    w.slot_ppos = (int*)take((size_t)n * sizeof(int));
    w.block_sum = (int*)take((size_t)(n / SCAN_BLOCK + 2) * sizeof(int));
    w.lv = (int*)take((size_t)(2 * (n + 2)) * sizeof(int));
    w.total = off;
    return w;
}

size_t forward_f32_gemm_ws_bytes(int32_t n_nodes, int32_t n_internal_bound, int32_t H) {
    return carve_f32(nullptr, n_nodes > 0 ? n_nodes : 1, n_internal_bound > 0 ? n_internal_bound : 1, H).total;
}

// Level by level through the tiled fp32 GEMM: W x + b of the level's rows, h~ U^T, U_f h_k over the level's edge slots,
// then the pointwise part.  Needs the level table on the host: copies it back and synchronises `st` once.
jdb_status forward_f32_gemm_enqueue(const ForwardArgs& a, int n_levels, int n_internal_bound, void* ws, cudaStream_t st) {
    const int n = a.n_nodes, ne = a.n_edges, H = a.H, D = a.D, L = n_levels;
    if (n <= 0 || L <= 0) return JDB_OK;
    DevInfo* di = dev_info();
    if (!di) return JDB_ERR_CUDA;
    const int n_sm = di->n_sm;
    F32Workspace w = carve_f32(ws, n, n_internal_bound > 0 ? n_internal_bound : 1, H);
    const int32_t* perm = a.perm;
    const int sb = n / SCAN_BLOCK + 1;
    slot_count_kernel<<<sb, SCAN_BLOCK, 0, st>>>(a.child_ptr, perm, n, w.block_sum);
    block_sums_scan_kernel<<<1, SCAN_BLOCK, 0, st>>>(w.block_sum, sb);
    slot_fill_kernel<<<sb, SCAN_BLOCK, 0, st>>>(a.child_ptr, a.child_idx, perm, n, ne, w.block_sum, w.edge_ptr, w.slot_child, w.slot_ppos);
    level_table_kernel<<<ceil_div(L + 1, 256), 256, 0, st>>>(a.level_ptr, w.edge_ptr, L, w.lv);
    JDB_CUDA_TRY(cudaGetLastError());
    std::vector<int> lv(2 * (size_t)(L + 1));
    JDB_CUDA_TRY(cudaMemcpyAsync(lv.data(), w.lv, lv.size() * sizeof(int), cudaMemcpyDeviceToHost, st));
    JDB_CUDA_TRY(cudaStreamSynchronize(st));
    const int* lp = lv.data();
    const int* eo = lv.data() + (L + 1);
    if (lp[0] != 0 || lp[L] != n || eo[L] != ne || n - lp[1] > n_internal_bound) return JDB_ERR_INVALID_ARG;
    for (int l = 0; l < L; ++l)
        if (lp[l + 1] < lp[l] || eo[l + 1] < eo[l]) return JDB_ERR_INVALID_ARG;

    if (a.ev_begin) JDB_CUDA_TRY(cudaEventRecord(a.ev_begin, st));
    const dim3 pw_block(H >= 128 ? 128 : (H > 32 ? 64 : 32), H >= 128 ? 2 : (H > 32 ? 4 : 8));
    jdb_status r;
    for (int l = 0; l < L; ++l) {
        const int lo = lp[l], m = lp[l + 1] - lp[l];
        if (m <= 0) continue;
        {   // Z = x[rows] Wt + bias (columns interleaved by gate, as the packed weights are)
            GemmArgs g{};
            g.A = (const float*)a.x; g.lda = a.ldx; g.a_idx = perm + lo; g.B = a.Wt; g.ldb = 4LL * H; g.C = w.Z; g.ldc = 4LL * H;
            g.M = m; g.N = 4 * H; g.K = D; g.bias = a.bias;
            if ((r = gemm<true, true>(g, SLOT_STEPS, n_sm, st)) != JDB_OK) return r;
        }
        const int e0 = eo[l], e1 = eo[l + 1];
        if (l > 0) {
            child_sum_f32_kernel<<<ceil_div(m, pw_block.y), pw_block, 0, st>>>(a.child_ptr, a.child_idx, perm, lo, m, H, a.h, a.ldh, w.HS);
            GemmArgs g{};
            g.A = w.HS; g.lda = H; g.B = a.Ut; g.ldb = 4LL * H; g.C = w.T; g.ldc = 4LL * H; g.M = m; g.N = 4 * H; g.K = H;
            if ((r = gemm<true, true>(g, SLOT_STEPS, n_sm, st)) != JDB_OK) return r;
            if (e1 > e0) {
                GemmArgs f{};
                f.A = a.h; f.lda = a.ldh; f.a_idx = w.slot_child + e0; f.B = a.Uft; f.ldb = H; f.C = w.FE + (size_t)e0 * H; f.ldc = H;
                f.M = e1 - e0; f.N = H; f.K = H;
                if ((r = gemm<true, true>(f, SLOT_STEPS, n_sm, st)) != JDB_OK) return r;
            }
        }
        childsum_pointwise_il_kernel<<<ceil_div(m, pw_block.y), pw_block, 0, st>>>(perm, w.edge_ptr, w.slot_child, lo, m, H, w.Z,
                                                                                   l > 0 ? w.T : nullptr, w.FE, a.h, a.c, a.ldh);
        JDB_CUDA_TRY(cudaGetLastError());
        if (l == 0 && a.ev_xproj_done) JDB_CUDA_TRY(cudaEventRecord(a.ev_xproj_done, st));   // the leaves: projection only
    }
    if (a.ev_levels_done) JDB_CUDA_TRY(cudaEventRecord(a.ev_levels_done, st));
    return JDB_OK;
}

}  // namespace jdb

using namespace jdb;

extern "C" {

size_t jdb_batch_plan_workspace_bytes(int32_t n_nodes) {
    if (n_nodes < 0) return 0;
    return carve_plan(nullptr, n_nodes).total;
}

jdb_status jdb_batch_plan(const jdb_forest* forest, const jdb_sched* sched, const int32_t* key, int32_t n_keys, jdb_plan* out,
                          void* ws, size_t ws_bytes, void* stream) {
    cudaStream_t st = (cudaStream_t)stream;
    if (!forest || !sched || !out || forest->n_nodes < 0 || n_keys <= 0) return JDB_ERR_INVALID_ARG;
    const int n = forest->n_nodes;
    out->n_slots = 0;
    out->bad_key = 0;
    if (!out->slot_ptr) return JDB_ERR_INVALID_ARG;
    if (n == 0) {
        JDB_CUDA_TRY(cudaMemsetAsync(out->slot_ptr, 0, sizeof(int32_t), st));
        return JDB_OK;
    }
    if (!key || !sched->depth || !out->perm || !out->slot_depth || !out->slot_key) return JDB_ERR_INVALID_ARG;
    if (sched->n_levels < 1) return JDB_ERR_INVALID_ARG;   // the level count bounds the sort key: needs jdb_schedule
    if ((long long)sched->n_levels * n_keys > 0x7fffffffLL) return JDB_ERR_UNSUPPORTED;
    if (!ws || ((uintptr_t)ws & 255) != 0) return JDB_ERR_INVALID_ARG;
    if (ws_bytes < carve_plan(nullptr, n).total) return JDB_ERR_WORKSPACE;
    PlanWorkspace w = carve_plan(ws, n);
    JDB_CUDA_TRY(cudaMemsetAsync(w.flags, 0, 4 * sizeof(int), st));
    composite_key_kernel<<<ceil_div(n, 256), 256, 0, st>>>(sched->depth, key, n, n_keys, w.comp, w.flags + 1);
    int bits = 1;
    while (((long long)1 << bits) < (long long)sched->n_levels * n_keys) ++bits;
    const int passes = (bits + RS_BITS - 1) / RS_BITS;
    const int n_blocks = ceil_div(n, RS_TILE);
    const int32_t* src = nullptr;
    for (int pass = 0; pass < passes; ++pass) {
        int32_t* dst = pass == passes - 1 ? out->perm : (pass & 1 ? w.tmp1 : w.tmp0);
        radix_hist_kernel<<<n_blocks, RS_TB, 0, st>>>(pass, src, w.comp, n, w.hist, n_blocks);
        radix_scan_kernel<<<1, SCAN_BLOCK, 0, st>>>(w.hist, (long long)RS_BINS * n_blocks);
        radix_scatter_kernel<<<n_blocks, RS_TB, 0, st>>>(pass, src, w.comp, n, w.hist, n_blocks, dst);
        src = dst;
    }
    const int sb = n / SCAN_BLOCK + 1;   // covers position n, which holds the totals
    slot_start_count_kernel<<<sb, SCAN_BLOCK, 0, st>>>(w.comp, out->perm, n, w.block_sum);
    block_sums_scan_kernel<<<1, SCAN_BLOCK, 0, st>>>(w.block_sum, sb);
    slot_start_fill_kernel<<<sb, SCAN_BLOCK, 0, st>>>(w.comp, out->perm, n, n_keys, w.block_sum, out->slot_ptr, out->slot_depth,
                                                     out->slot_key, w.flags);
    JDB_CUDA_TRY(cudaGetLastError());
    int flags[2] = {0, 0};
    JDB_CUDA_TRY(cudaMemcpyAsync(flags, w.flags, sizeof(flags), cudaMemcpyDeviceToHost, st));
    JDB_CUDA_TRY(cudaStreamSynchronize(st));
    out->n_slots = flags[0];
    out->bad_key = flags[1];
    return flags[1] ? JDB_ERR_INVALID_ARG : JDB_OK;
}

size_t jdb_cells_forward_workspace_bytes(int32_t n_nodes, int32_t n_edges, int32_t H, int32_t max_arity, int32_t n_keys) {
    if (n_nodes < 0 || n_edges < 0 || H <= 0 || max_arity < 0 || n_keys <= 0) return 0;
    return carve_cells(nullptr, n_nodes, n_edges, H, max_arity, n_keys).total;
}

jdb_status jdb_cells_forward(const jdb_forest* forest, const jdb_plan* plan, const int32_t* key, const jdb_cell* cells,
                             int32_t n_keys, const float* x, int64_t ldx, int32_t D, int32_t H, float* h, float* c, int64_t ldh,
                             void* ws, size_t ws_bytes, void* stream) {
    cudaStream_t st = (cudaStream_t)stream;
    if (!forest || !plan || !cells || forest->n_nodes < 0 || forest->n_edges < 0 || n_keys <= 0 || D <= 0 || H <= 0) return JDB_ERR_INVALID_ARG;
    const int n = forest->n_nodes, ne = forest->n_edges;
    if (n == 0) return JDB_OK;
    if (!forest->child_ptr || (ne > 0 && !forest->child_idx) || !key || !x || !h || !c) return JDB_ERR_INVALID_ARG;
    if (!plan->perm || !plan->slot_ptr || !plan->slot_depth || !plan->slot_key || plan->n_slots < 1 || plan->n_slots > n) return JDB_ERR_INVALID_ARG;
    if (ldx < D || ldh < H) return JDB_ERR_INVALID_ARG;
    int amax = 0;
    std::vector<int32_t> arity(n_keys);
    for (int k = 0; k < n_keys; ++k) {
        const jdb_cell& cl = cells[k];
        if (!cl.W || !cl.U || !cl.b) return JDB_ERR_INVALID_ARG;
        if (cl.kind == JDB_CELL_CHILDSUM) arity[k] = 0;
        else if (cl.kind == JDB_CELL_NARY && cl.arity >= 1 && cl.arity <= 8) arity[k] = cl.arity;
        else return JDB_ERR_INVALID_ARG;
        if (arity[k] > amax) amax = arity[k];
    }
    if (!ws || ((uintptr_t)ws & 255) != 0) return JDB_ERR_INVALID_ARG;
    if (ws_bytes < carve_cells(nullptr, n, ne, H, amax, n_keys).total) return JDB_ERR_WORKSPACE;
    DevInfo* di = dev_info();
    if (!di) return JDB_ERR_CUDA;
    const int n_sm = di->n_sm;
    CellsWorkspace w = carve_cells(ws, n, ne, H, amax, n_keys);
    const int32_t* perm = plan->perm;
    const int S = plan->n_slots;

    // edge slots in plan order, the children by position, and the slot table on the host
    JDB_CUDA_TRY(cudaMemsetAsync(w.flags, 0, 4 * sizeof(int), st));
    JDB_CUDA_TRY(cudaMemcpyAsync(w.arity_of, arity.data(), (size_t)n_keys * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    const int sb = n / SCAN_BLOCK + 1;
    slot_count_kernel<<<sb, SCAN_BLOCK, 0, st>>>(forest->child_ptr, perm, n, w.block_sum);
    block_sums_scan_kernel<<<1, SCAN_BLOCK, 0, st>>>(w.block_sum, sb);
    slot_fill_kernel<<<sb, SCAN_BLOCK, 0, st>>>(forest->child_ptr, forest->child_idx, perm, n, ne, w.block_sum, w.edge_ptr, w.slot_child, w.slot_ppos);
    child_positions_kernel<<<ceil_div(n, 256), 256, 0, st>>>(forest->child_ptr, forest->child_idx, perm, key, w.arity_of, n, n_keys,
                                                           amax > 0 ? amax : 1, w.kid, w.flags);
    for (int l = 1; l < amax; ++l) {   // position 0 is held by every internal node: no list needed
        position_count_kernel<<<sb, SCAN_BLOCK, 0, st>>>(w.kid + (size_t)l * n, n, w.block_sum);
        block_sums_scan_kernel<<<1, SCAN_BLOCK, 0, st>>>(w.block_sum, sb);
        position_fill_kernel<<<sb, SCAN_BLOCK, 0, st>>>(w.kid + (size_t)l * n, n, w.block_sum, w.cptr + (size_t)l * (n + 1),
                                                       w.ckid + (size_t)l * n, w.cpos + (size_t)l * n);
    }
    if (amax > 1) position_table_kernel<<<ceil_div((long long)S * amax, 256), 256, 0, st>>>(plan->slot_ptr, w.cptr, n, S, amax, w.table);
    JDB_CUDA_TRY(cudaGetLastError());
    std::vector<int32_t> sp((size_t)S + 1), sd(S), sk(S), ep((size_t)n + 1), tab(amax > 1 ? (size_t)2 * S * amax : 0);
    if (amax > 1) JDB_CUDA_TRY(cudaMemcpyAsync(tab.data(), w.table, tab.size() * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    int bad = 0;
    JDB_CUDA_TRY(cudaMemcpyAsync(sp.data(), plan->slot_ptr, sp.size() * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    JDB_CUDA_TRY(cudaMemcpyAsync(sd.data(), plan->slot_depth, sd.size() * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    JDB_CUDA_TRY(cudaMemcpyAsync(sk.data(), plan->slot_key, sk.size() * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    JDB_CUDA_TRY(cudaMemcpyAsync(ep.data(), w.edge_ptr, ep.size() * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    JDB_CUDA_TRY(cudaMemcpyAsync(&bad, w.flags, sizeof(int), cudaMemcpyDeviceToHost, st));
    JDB_CUDA_TRY(cudaStreamSynchronize(st));
    if (bad) return JDB_ERR_INVALID_ARG;   // a node with more children than its cell's arity
    if (sp[0] != 0 || sp[S] != n || ep[n] != ne) return JDB_ERR_INVALID_ARG;
    for (int s = 0; s < S; ++s)
        if (sp[s + 1] <= sp[s] || sk[s] < 0 || sk[s] >= n_keys || sd[s] < 0) return JDB_ERR_INVALID_ARG;

    const dim3 pw_block(H >= 128 ? 128 : (H > 32 ? 64 : 32), H >= 128 ? 2 : (H > 32 ? 4 : 8));
    jdb_status r;
    for (int s = 0; s < S; ++s) {
        const int lo = sp[s], m = sp[s + 1] - sp[s];
        const jdb_cell& cl = cells[sk[s]];
        const bool leaves = sd[s] == 0;
        {   // Z = x[rows] W^T + b
            GemmArgs g{};
            g.A = x; g.lda = ldx; g.a_idx = perm + lo; g.B = cl.W; g.ldb = D; g.C = w.Z; g.ldc = 4LL * H; g.M = m; g.N = 4 * H; g.K = D; g.bias = cl.b;
            if ((r = gemm<true, false>(g, SLOT_STEPS, n_sm, st)) != JDB_OK) return r;
        }
        if (cl.kind == JDB_CELL_CHILDSUM) {
            const int e0 = ep[lo], e1 = ep[lo + m];
            if (!leaves) {
                child_sum_f32_kernel<<<ceil_div(m, pw_block.y), pw_block, 0, st>>>(forest->child_ptr, forest->child_idx, perm, lo, m, H, h, ldh, w.HS);
                GemmArgs g{};
                g.A = w.HS; g.lda = H; g.B = cl.U; g.ldb = H; g.C = w.Z; g.ldc = 4LL * H; g.M = m; g.N = 3 * H; g.K = H; g.beta = 1;
                if ((r = gemm<true, false>(g, SLOT_STEPS, n_sm, st)) != JDB_OK) return r;
                if (e1 > e0) {
                    GemmArgs f{};
                    f.A = h; f.lda = ldh; f.a_idx = w.slot_child + e0; f.B = cl.U + (size_t)3 * H * H; f.ldb = H; f.C = w.FE + (size_t)e0 * H; f.ldc = H;
                    f.M = e1 - e0; f.N = H; f.K = H;
                    if ((r = gemm<true, false>(f, SLOT_STEPS, n_sm, st)) != JDB_OK) return r;
                }
            }
            childsum_pointwise_kernel<<<ceil_div(m, pw_block.y), pw_block, 0, st>>>(perm, w.edge_ptr, w.slot_child, lo, m, H, w.Z, w.FE, h, c, ldh);
        } else {
            const int a = cl.arity;
            if (!leaves) {
                const long long ldg = (3LL + a) * H;
                for (int l = 0; l < a; ++l) {   // G (+)= h[child l] U^l T, over the rows that have a child l
                    GemmArgs g{};
                    g.A = h; g.lda = ldh; g.B = cl.U + (size_t)l * H; g.ldb = (long long)a * H; g.ldc = ldg; g.N = (3 + a) * H; g.K = H;
                    if (l == 0) {
                        g.a_idx = w.kid + lo; g.C = w.G + (size_t)lo * ldg; g.M = m;
                    } else {
                        const int c0 = tab[((size_t)s * amax + l) * 2], c1 = tab[((size_t)s * amax + l) * 2 + 1];
                        if (c1 <= c0) continue;
                        g.a_idx = w.ckid + (size_t)l * n + c0; g.c_idx = w.cpos + (size_t)l * n + c0; g.C = w.G; g.M = c1 - c0; g.beta = 1;
                    }
                    if ((r = gemm<true, false>(g, SLOT_STEPS, n_sm, st)) != JDB_OK) return r;
                }
            }
            nary_pointwise_kernel<<<ceil_div(m, pw_block.y), pw_block, 0, st>>>(perm, w.kid, n, lo, m, H, a, w.Z, leaves ? nullptr : w.G, h, c, ldh);
        }
        JDB_CUDA_TRY(cudaGetLastError());
    }
    return JDB_OK;
}

}  // extern "C"
