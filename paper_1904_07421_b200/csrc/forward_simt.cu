// Batched cell evaluation on the plain fp32 ALUs (FFMA): the path for JDB_FP32, whose 1e-4 bound rules the
// tensor cores out, and the reference-shaped fallback of the bf16 path for sizes the tensor-core kernels do
// not take.  One slot of the paper's table (Section 4.3) = one level = one batch, whatever the fan-out:
// the four child-count-dependent operators of the cell (gather, child-sum, per-child forget gate and the
// sum of f*c; Section 3) are loops inside the tile, not separate launches.
//
//   xproj_simt_kernel   Z = W x + b for every node, rows in level order.  Leaves finish here
//                       (c = sig(z_i) tanh(z_u), h = sig(z_o) tanh(c)); internal rows go to P.
//   level_kernel        one level: tiles of TM nodes; gather child h rows, child-sum, U products,
//                       per-child forget gates in chunks of TE edges, c/h update, scatter rows.
//   persistent_kernel   the same tiles inside one cooperative launch, levels separated by a bounded
//                       grid barrier (deep forests with tiny levels).
#include "common.cuh"
#include "grid_sync.cuh"

namespace jdb {

namespace {

constexpr int TM = 8;  // nodes per tile
constexpr int TE = 8;  // child edges per chunk of the forget-gate loop

__device__ __forceinline__ float sigmoid_acc(float t) { return 1.0f / (1.0f + expf(-t)); }
__device__ __forceinline__ float bf16r(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }

__device__ __forceinline__ float load_x(const void* x, int is_bf16, int64_t off) {
    if (is_bf16) return __bfloat162float(((const __nv_bfloat16*)x)[off]);
    return ((const float*)x)[off];
}

// Threads are (column j, K group): the K loop of a dot product is a chain of dependent loads from L2, so it is
// cut into `ks` pieces that run side by side and are summed through shared memory.
__global__ void __launch_bounds__(512) xproj_simt_kernel(ForwardArgs a, int jt, int ks) {
    extern __shared__ float sm[];
    float* xs = sm;                                               // [TM][D]
    float4* red = reinterpret_cast<float4*>(sm + ((TM * a.D + 3) & ~3));  // [ks-1][TM][jt]
    __shared__ int nodes[TM];
    const int N = a.n_nodes, D = a.D, H = a.H;
    const int n_leaves = a.meta[META_N_LEAVES];
    const int pos0 = blockIdx.x * TM;
    const int tx = threadIdx.x % jt, ky = threadIdx.x / jt;
    if (threadIdx.x < TM) {
        int v = (pos0 + threadIdx.x < N) ? a.perm[pos0 + threadIdx.x] : -1;
        if (a.debug && v != -1 && !dbg_ok(a.meta, CHECK_PERM, v, N, pos0 + threadIdx.x)) v = -1;
        nodes[threadIdx.x] = v;
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < TM * D; idx += blockDim.x) {
        int t = idx / D, d = idx - t * D;
        int v = nodes[t];
        float val = 0.f;
        if (v >= 0) {
            val = load_x(a.x, a.x_is_bf16, (int64_t)v * a.ldx + d);
            if (a.round_bf16 && !a.x_is_bf16) val = bf16r(val);
        }
        xs[idx] = val;
    }
    __syncthreads();
    const int j = blockIdx.y * jt + tx;
    const bool live = j < H;
    const float4* Wt4 = (const float4*)a.Wt;
    float4 acc[TM];
    const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
    const float4 b4 = (live && ky == 0) ? ((const float4*)a.bias)[j] : zero4;
#pragma unroll
    for (int t = 0; t < TM; ++t) acc[t] = b4;
    const int dchunk = (D + ks - 1) / ks, d0 = ky * dchunk, d1 = min(D, d0 + dchunk);
    if (live) {
#pragma unroll 8
        for (int d = d0; d < d1; ++d) {
            const float4 w4 = Wt4[(size_t)d * H + j];
#pragma unroll
            for (int t = 0; t < TM; ++t) {
                const float xv = xs[t * D + d];
                acc[t].x = fmaf(xv, w4.x, acc[t].x);
                acc[t].y = fmaf(xv, w4.y, acc[t].y);
                acc[t].z = fmaf(xv, w4.z, acc[t].z);
                acc[t].w = fmaf(xv, w4.w, acc[t].w);
            }
        }
    }
    if (ky > 0) {
#pragma unroll
        for (int t = 0; t < TM; ++t) red[((ky - 1) * TM + t) * jt + tx] = acc[t];
    }
    __syncthreads();
    if (ky > 0 || !live) return;
    for (int g = 0; g < ks - 1; ++g) {  // fixed order: the result does not depend on thread timing
#pragma unroll
        for (int t = 0; t < TM; ++t) {
            const float4 r = red[(g * TM + t) * jt + tx];
            acc[t].x += r.x; acc[t].y += r.y; acc[t].z += r.z; acc[t].w += r.w;
        }
    }
#pragma unroll
    for (int t = 0; t < TM; ++t) {
        const int v = nodes[t];
        if (v < 0) continue;
        const int pos = pos0 + t;
        if (pos < n_leaves) {
            const float cc = sigmoid_acc(acc[t].x) * tanhf(acc[t].z);
            a.c[(int64_t)v * a.ldh + j] = cc;
            a.h[(int64_t)v * a.ldh + j] = sigmoid_acc(acc[t].y) * tanhf(cc);
        } else {
            ((float4*)a.P)[(size_t)(pos - n_leaves) * H + j] = acc[t];
        }
    }
}

// One tile of m <= TM nodes of a level (perm positions pos0 .. pos0+m-1).
// Threads are (column j, K group) as in the projection kernel: jt columns, ks pieces of every K loop.
__device__ void level_tile(const ForwardArgs& a, int pos0, int m, int n_leaves, float* sm, int jt, int ks) {
    const int H = a.H, Hs = (H + 3) & ~3;
    float* hs = sm;                // [TM][Hs] child sums (GEMM operand)
    float* hk = hs + TM * Hs;      // [TE][Hs] child h rows of the current edge chunk
    float* cacc = hk + TE * Hs;    // [TM][Hs] running c
    float* pf = cacc + TM * Hs;    // [TM][Hs] forget pre-activation from the input projection
    float* og = pf + TM * Hs;      // [TM][Hs] output gate
    float* red = og + TM * Hs;     // [ks-1][TM][jt][4] partial sums of the K groups
    __shared__ int nodes[TM], ebeg[TM], eoff[TM + 1], ck_t[TE], ck_k[TE];
    const int tid = threadIdx.x, nt = blockDim.x;
    const int tx = tid % jt, ky = tid / jt;
    const int dchunk = (H + ks - 1) / ks, d0 = ky * dchunk, d1 = min(H, d0 + dchunk);

    if (tid < TM) {
        int v = tid < m ? a.perm[pos0 + tid] : -1;
        if (a.debug && v != -1 && !dbg_ok(a.meta, CHECK_PERM, v, a.n_nodes, pos0 + tid)) v = -1;
        nodes[tid] = v;
        int eb = v >= 0 ? a.child_ptr[v] : 0, cnt = v >= 0 ? a.child_ptr[v + 1] - eb : 0;
        if (a.debug && !(dbg_ok(a.meta, CHECK_EDGE_PTR, eb, (long long)a.n_edges + 1, pos0 + tid) &&
                         dbg_ok(a.meta, CHECK_EDGE_PTR, cnt, (long long)a.n_edges - eb + 1, pos0 + tid)))
            eb = cnt = 0;
        ebeg[tid] = eb;
        eoff[tid + 1] = cnt;
    }
    __syncthreads();
    if (tid == 0) {
        eoff[0] = 0;
        for (int t = 0; t < TM; ++t) eoff[t + 1] += eoff[t];
    }
    __syncthreads();

    // child-sum: thread owns column jj of row t; children added in CSR order
    for (int idx = tid; idx < TM * Hs; idx += nt) {
        const int t = idx / Hs, jj = idx - t * Hs;
        float s = 0.f;
        if (t < m && jj < H) {
            const int e0 = ebeg[t], e1 = e0 + (eoff[t + 1] - eoff[t]);
            for (int e = e0; e < e1; ++e) {
                const int k = a.child_idx[e];
                if (a.debug && !dbg_ok(a.meta, CHECK_CHILD, k, a.n_nodes, e)) continue;
                s += __ldcg(&a.h[(int64_t)k * a.ldh + jj]);
            }
            if (a.round_bf16) s = bf16r(s);
        }
        hs[idx] = s;
    }
    __syncthreads();

    // (i, o, u) = P + U_iou h~ ; keep i*u, o and the forget pre-activation
    const float4* Ut4 = (const float4*)a.Ut;
    for (int jb = 0; jb < H; jb += jt) {
        const int j = jb + tx;
        const bool live = j < H;
        float4 acc[TM];
#pragma unroll
        for (int t = 0; t < TM; ++t)
            acc[t] = (live && ky == 0 && t < m) ? __ldcg(&((const float4*)a.P)[(size_t)(pos0 + t - n_leaves) * H + j])
                                               : make_float4(0.f, 0.f, 0.f, 0.f);
        if (live) {
#pragma unroll 8
            for (int d = d0; d < d1; ++d) {
                const float4 u4 = Ut4[(size_t)d * H + j];
#pragma unroll
                for (int t = 0; t < TM; ++t) {
                    const float hv = hs[t * Hs + d];
                    acc[t].x = fmaf(hv, u4.x, acc[t].x);
                    acc[t].y = fmaf(hv, u4.y, acc[t].y);
                    acc[t].z = fmaf(hv, u4.z, acc[t].z);
                }
            }
        }
        if (ky > 0) {
#pragma unroll
            for (int t = 0; t < TM; ++t) reinterpret_cast<float4*>(red)[((ky - 1) * TM + t) * jt + tx] = acc[t];
        }
        __syncthreads();
        if (ky == 0 && live) {
            for (int g = 0; g < ks - 1; ++g) {
#pragma unroll
                for (int t = 0; t < TM; ++t) {
                    const float4 r = reinterpret_cast<const float4*>(red)[(g * TM + t) * jt + tx];
                    acc[t].x += r.x; acc[t].y += r.y; acc[t].z += r.z;
                }
            }
#pragma unroll
            for (int t = 0; t < TM; ++t) {
                cacc[t * Hs + j] = sigmoid_acc(acc[t].x) * tanhf(acc[t].z);
                og[t * Hs + j] = sigmoid_acc(acc[t].y);
                pf[t * Hs + j] = acc[t].w;
            }
        }
        __syncthreads();
    }

    // per-child forget gates, TE edges at a time, edges of the tile taken in (node, CSR) order
    const int ne = eoff[TM];
    for (int e0 = 0; e0 < ne; e0 += TE) {
        const int nc = min(TE, ne - e0);
        if (tid < TE) {
            int t = 0, k = -1;
            if (tid < nc) {
                const int e = e0 + tid;
                while (eoff[t + 1] <= e) ++t;
                k = a.child_idx[ebeg[t] + (e - eoff[t])];
                if (a.debug && !dbg_ok(a.meta, CHECK_CHILD, k, a.n_nodes, ebeg[t] + (e - eoff[t]))) k = -1;
            }
            ck_t[tid] = t;
            ck_k[tid] = k;
        }
        __syncthreads();
        for (int idx = tid; idx < TE * Hs; idx += nt) {
            const int ee = idx / Hs, jj = idx - ee * Hs;
            float val = 0.f;
            if (ee < nc && jj < H && ck_k[ee] >= 0) {
                val = __ldcg(&a.h[(int64_t)ck_k[ee] * a.ldh + jj]);
                if (a.round_bf16) val = bf16r(val);
            }
            hk[idx] = val;
        }
        __syncthreads();
        for (int jb = 0; jb < H; jb += jt) {
            const int j = jb + tx;
            const bool live = j < H;
            float dot[TE];
#pragma unroll
            for (int ee = 0; ee < TE; ++ee) dot[ee] = 0.f;
            if (live) {
#pragma unroll 8
                for (int d = d0; d < d1; ++d) {
                    const float uf = a.Uft[(size_t)d * H + j];
#pragma unroll
                    for (int ee = 0; ee < TE; ++ee) dot[ee] = fmaf(hk[ee * Hs + d], uf, dot[ee]);
                }
            }
            if (ky > 0) {
#pragma unroll
                for (int ee = 0; ee < TE; ++ee) red[((ky - 1) * TE + ee) * jt + tx] = dot[ee];
            }
            __syncthreads();
            if (ky == 0 && live) {
                for (int g = 0; g < ks - 1; ++g) {
#pragma unroll
                    for (int ee = 0; ee < TE; ++ee) dot[ee] += red[(g * TE + ee) * jt + tx];
                }
#pragma unroll
                for (int ee = 0; ee < TE; ++ee) {
                    if (ee < nc && ck_k[ee] >= 0) {
                        const int t = ck_t[ee];
                        const float f = sigmoid_acc(pf[t * Hs + j] + dot[ee]);
                        cacc[t * Hs + j] = fmaf(f, __ldcg(&a.c[(int64_t)ck_k[ee] * a.ldh + j]), cacc[t * Hs + j]);
                    }
                }
            }
            __syncthreads();
        }
    }

    // h = o * tanh(c); rows back to node order
    for (int idx = tid; idx < m * H; idx += nt) {
        const int t = idx / H, j = idx - t * H;
        if (nodes[t] < 0) continue;
        const int64_t row = (int64_t)nodes[t] * a.ldh;
        const float cc = cacc[t * Hs + j];
        a.c[row + j] = cc;
        a.h[row + j] = og[t * Hs + j] * tanhf(cc);
    }
    __syncthreads();
}

__global__ void __launch_bounds__(512) level_kernel(ForwardArgs a, int level, int jt, int ks) {
    extern __shared__ float sm[];
    const int n_levels = a.meta[META_N_LEVELS];
    if (level >= n_levels) return;
    const int n_leaves = a.level_ptr[1];
    int lo, hi;
    checked_level(a.level_ptr, level, a.n_nodes, a.meta, a.debug, lo, hi);
    const int tiles = (hi - lo + TM - 1) / TM;
    for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x)
        level_tile(a, lo + tile * TM, min(TM, hi - lo - tile * TM), n_leaves, sm, jt, ks);
}

__global__ void __launch_bounds__(512) persistent_kernel(ForwardArgs a, unsigned long long timeout_ns, int jt, int ks) {
    extern __shared__ float sm[];
    const int n_levels = a.meta[META_N_LEVELS];
    if (a.meta[META_ERROR] != 0 || a.meta[META_UNFINISHED] != 0) return;  // malformed forest: nothing to run
    const int n_leaves = n_levels > 0 ? a.level_ptr[1] : 0;
    for (int level = 1; level < n_levels; ++level) {
        int lo, hi;
        checked_level(a.level_ptr, level, a.n_nodes, a.meta, a.debug, lo, hi);
        const int tiles = (hi - lo + TM - 1) / TM;
        for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x)
            level_tile(a, lo + tile * TM, min(TM, hi - lo - tile * TM), n_leaves, sm, jt, ks);
        if (level + 1 < n_levels)
            if (!grid_barrier(a.meta, (unsigned)level * gridDim.x, timeout_ns)) return;
    }
}

int level_threads(int H) {
    int t = (H + 31) / 32 * 32;
    return t < 64 ? 64 : (t > 256 ? 256 : t);
}

}  // namespace

size_t forward_ws_bytes(int32_t n_nodes, int32_t n_internal_bound, int32_t D, int32_t H, int32_t precision) {
    (void)n_nodes; (void)D; (void)precision;
    size_t rows = (size_t)(n_internal_bound > 0 ? n_internal_bound : 1);
    return align_up(rows * (size_t)H * 4 * sizeof(float), 256);
}

jdb_status forward_enqueue(const ForwardArgs& a, int n_levels_host, int n_internal_bound, int mode,
                           uint64_t timeout_ns, cudaStream_t st) {
    const int N = a.n_nodes, H = a.H, D = a.D;
    int dev = 0, n_sm = 0, max_smem = 0;
    JDB_CUDA_TRY(cudaGetDevice(&dev));
    JDB_CUDA_TRY(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
    JDB_CUDA_TRY(cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));

    const int Hs = (H + 3) & ~3;
    // thread layout: jt columns x ks pieces of the K loops, at most 512 threads (128 registers each)
    const int lt_j = level_threads(H);
    int lks = 512 / lt_j;
    lks = lks < 1 ? 1 : (lks > 4 ? 4 : lks);
    const int xt_j = lt_j > 128 ? 128 : lt_j;
    const int xks = 4;
    const size_t x_smem = (size_t)((TM * D + 3) & ~3) * sizeof(float) + (size_t)(xks - 1) * TM * xt_j * sizeof(float4);
    const size_t l_smem = (size_t)(4 * TM + TE) * Hs * sizeof(float) + (size_t)(lks - 1) * TM * lt_j * sizeof(float4);
    if (x_smem > (size_t)max_smem || l_smem + 1024 > (size_t)max_smem) return JDB_ERR_UNSUPPORTED;
    JDB_CUDA_TRY(cudaFuncSetAttribute(xproj_simt_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)x_smem));
    JDB_CUDA_TRY(cudaFuncSetAttribute(level_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)l_smem));
    JDB_CUDA_TRY(cudaFuncSetAttribute(persistent_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)l_smem));

    dim3 xgrid(ceil_div(N, TM), ceil_div(H, xt_j));
    if (a.ev_begin) JDB_CUDA_TRY(cudaEventRecord(a.ev_begin, st));
    xproj_simt_kernel<<<xgrid, xt_j * xks, x_smem, st>>>(a, xt_j, xks);
    JDB_CUDA_TRY(cudaGetLastError());
    if (a.ev_xproj_done) JDB_CUDA_TRY(cudaEventRecord(a.ev_xproj_done, st));

    const int lt = lt_j * lks;
    const int max_tiles = ceil_div(n_internal_bound > 0 ? n_internal_bound : 1, TM);
    if (mode == JDB_MODE_PERSISTENT && !a.round_bf16 && small_levels_f32_supported(H)) {
        // fp32 with a small hidden size: hidden slices spread over the CTAs, weight slices resident in shared memory
        jdb_status s = small_levels_f32_enqueue(a, n_internal_bound, timeout_ns, st);
        if (s != JDB_OK) return s;
    } else if (mode == JDB_MODE_PERSISTENT) {
        int per_sm = 0;
        JDB_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, persistent_kernel, lt, l_smem));
        if (per_sm < 1) return JDB_ERR_UNSUPPORTED;
        int grid = n_sm * per_sm;
        if (grid > max_tiles) grid = max_tiles;
        ForwardArgs args = a;
        unsigned long long tmo = timeout_ns;
        int jt_arg = lt_j, ks_arg = lks;
        void* params[] = {&args, &tmo, &jt_arg, &ks_arg};
        JDB_CUDA_TRY(cudaLaunchCooperativeKernel((const void*)persistent_kernel, dim3(grid), dim3(lt), params, l_smem, st));
    } else {
        int grid = max_tiles < n_sm * 16 ? max_tiles : n_sm * 16;
        for (int level = 1; level < n_levels_host; ++level) level_kernel<<<grid, lt, l_smem, st>>>(a, level, lt_j, lks);
        JDB_CUDA_TRY(cudaGetLastError());
    }
    if (a.ev_levels_done) JDB_CUDA_TRY(cudaEventRecord(a.ev_levels_done, st));
    return JDB_OK;
}

}  // namespace jdb
