// C entry points of libjdb: argument checks, workspace carving, and the order of the launches.
#include <mutex>

#include "common.cuh"
#include "scan.cuh"

namespace jdb {
static thread_local int g_last_cuda_error = 0;
void set_last_cuda_error(cudaError_t e) { g_last_cuda_error = (int)e; }

DevInfo* dev_info() {
    static DevInfo table[64];
    static bool known[64] = {};
    static std::mutex mu;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!known[dev]) {
        DevInfo d{};
        if (cudaDeviceGetAttribute(&d.n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return nullptr;
        if (cudaDeviceGetAttribute(&d.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return nullptr;
        table[dev] = d;
        known[dev] = true;
    }
    return &table[dev];
}

namespace {

// ---- roots only: the rows of the nodes that no child list mentions, compacted in ascending id ----------------------
__global__ void mark_children_kernel(const int32_t* __restrict__ child_idx, int n_edges, int n, int* __restrict__ is_child) {
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= n_edges) return;
    const int c = child_idx[e];
    if (c >= 0 && c < n) is_child[c] = 1;
}
__global__ void __launch_bounds__(SCAN_BLOCK) root_count_kernel(const int* __restrict__ is_child, int n, int* block_sum) {
    const int v = blockIdx.x * SCAN_BLOCK + threadIdx.x;
    int total;
    block_exclusive_scan((v < n && !is_child[v]) ? 1 : 0, total);
    if (threadIdx.x == 0) block_sum[blockIdx.x] = total;
}
__global__ void __launch_bounds__(SCAN_BLOCK) root_list_kernel(const int* __restrict__ is_child, int n, const int* block_off, int n_roots,
                                                               int32_t* __restrict__ root_id) {
    const int v = blockIdx.x * SCAN_BLOCK + threadIdx.x;
    const int flag = (v < n && !is_child[v]) ? 1 : 0;
    int total;
    const int r = block_off[blockIdx.x] + block_exclusive_scan(flag, total);
    if (flag && r < n_roots) root_id[r] = v;
}
__global__ void root_rows_kernel(const int32_t* __restrict__ root_id, int n_roots, int H, const float* __restrict__ h,
                                 const float* __restrict__ c, long long ldh, float* __restrict__ hr, float* __restrict__ cr) {
    const int r = blockIdx.x * blockDim.y + threadIdx.y;
    if (r >= n_roots) return;
    const long long v = root_id[r];
    for (int col = threadIdx.x; col < H; col += blockDim.x) {
        hr[(long long)r * H + col] = h[v * ldh + col];
        cr[(long long)r * H + col] = c[v * ldh + col];
    }
}

jdb_status read_meta(const int32_t* meta_dev, int32_t* meta_host, cudaStream_t st) {
    JDB_CUDA_TRY(cudaMemcpyAsync(meta_host, meta_dev, JDB_META_INTS * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    JDB_CUDA_TRY(cudaStreamSynchronize(st));
    return JDB_OK;
}

// what the device recorded about the calls enqueued so far
jdb_status meta_status(const int32_t* meta) {
    if (meta[META_ERROR] != 0 || meta[META_UNFINISHED] != 0) return JDB_ERR_NOT_A_FOREST;
    if (meta[META_TIMEOUT] != 0) return JDB_ERR_TIMEOUT;
    if (meta[META_CHECK] != 0) return JDB_ERR_CHECK;
    return JDB_OK;
}

jdb_status check_forest_args(const jdb_forest* f) {
    if (!f || f->n_nodes < 0 || f->n_edges < 0) return JDB_ERR_INVALID_ARG;
    if (f->n_nodes > 0 && !f->child_ptr) return JDB_ERR_INVALID_ARG;
    if (f->n_edges > 0 && !f->child_idx) return JDB_ERR_INVALID_ARG;
    if (f->n_nodes == 0 && f->n_edges != 0) return JDB_ERR_NOT_A_FOREST;
    return JDB_OK;
}

jdb_status schedule_common(const jdb_forest* f, jdb_sched* out, void* ws, size_t ws_bytes, cudaStream_t st, bool sync) {
    jdb_status s = check_forest_args(f);
    if (s != JDB_OK) return s;
    if (!out || !out->level_ptr || !out->meta) return JDB_ERR_INVALID_ARG;
    if (f->n_nodes > 0 && (!out->depth || !out->perm)) return JDB_ERR_INVALID_ARG;
    if (f->n_nodes > SMALL_SCHED_MAX) {
        if (!ws || ((uintptr_t)ws & 255) != 0) return JDB_ERR_INVALID_ARG;
        if (ws_bytes < schedule_ws_bytes(f->n_nodes, f->n_edges)) return JDB_ERR_WORKSPACE;
    }
    out->n_levels = -1;
    out->n_leaves = -1;
    out->n_wide_levels = -1;
    s = schedule_enqueue(*f, *out, ws, ws_bytes, st);
    if (s != JDB_OK || !sync) return s;
    int32_t meta[JDB_META_INTS];
    s = read_meta(out->meta, meta, st);
    if (s != JDB_OK) return s;
    if (meta[META_ERROR] != 0 || meta[META_UNFINISHED] != 0) return JDB_ERR_NOT_A_FOREST;
    out->n_levels = meta[META_N_LEVELS];
    out->n_leaves = meta[META_N_LEAVES];
    out->n_wide_levels = meta[META_WIDE_LEVELS];
    return JDB_OK;
}

}  // namespace
}  // namespace jdb

using namespace jdb;

namespace jdb {
// Copies a request's arrays to `dev_ws`, enqueues analysis, forward and the copies back on `stream`; does not wait for them
// (except where the per-level launches need the level count: there the analysis synchronises).
jdb_status forward_host_enqueue(const int32_t* child_ptr, const int32_t* child_idx, int32_t n_nodes, int32_t n_edges,
                                const void* x, int32_t x_dtype, const void* packed, int32_t D, int32_t H, float* h, float* c,
                                const jdb_opts* opts, void* dev_ws, size_t dev_ws_bytes, int32_t** meta_out, void* stream) {
    cudaStream_t st = (cudaStream_t)stream;
    if (n_nodes < 0 || n_edges < 0 || !opts || D <= 0 || H <= 0) return JDB_ERR_INVALID_ARG;
    if (x_dtype != JDB_FP32 && x_dtype != JDB_BF16) return JDB_ERR_INVALID_ARG;
    *meta_out = nullptr;
    if (n_nodes == 0) return n_edges == 0 ? JDB_OK : JDB_ERR_NOT_A_FOREST;
    if (!child_ptr || (n_edges > 0 && !child_idx) || !x || !h || !c || !packed) return JDB_ERR_INVALID_ARG;
    if (!dev_ws || ((uintptr_t)dev_ws & 255) != 0) return JDB_ERR_INVALID_ARG;
    if (dev_ws_bytes < jdb_forward_host_workspace_bytes(n_nodes, n_edges, D, H, opts->precision, x_dtype))
        return JDB_ERR_WORKSPACE;
    const size_t n = (size_t)n_nodes, e = (size_t)(n_edges > 0 ? n_edges : 1), xb = x_dtype == JDB_BF16 ? 2 : 4;
    char* p = (char*)dev_ws;
    auto take = [&](size_t bytes) { char* q = p; p += align_up(bytes, 256); return q; };
    int32_t* d_cp = (int32_t*)take((n + 1) * 4);
    int32_t* d_ci = (int32_t*)take(e * 4);
    void* d_x = take(n * (size_t)D * xb);
    jdb_sched sch{};
    sch.depth = (int32_t*)take(n * 4);
    sch.perm = (int32_t*)take(n * 4);
    sch.level_ptr = (int32_t*)take((n + 2) * 4);
    sch.meta = (int32_t*)take(256);
    const size_t ldh = ((size_t)H + 3) / 4 * 4;  // device rows padded to 16 bytes: the kernels' vector paths apply
    float* d_h = (float*)take(n * ldh * 4);
    float* d_c = (float*)take(n * ldh * 4);
    size_t sws = schedule_ws_bytes(n_nodes, n_edges);
    void* d_sws = take(sws);
    size_t fws = jdb_forward_workspace_bytes(n_nodes, n_nodes, D, H, opts->precision);
    void* d_fws = take(fws);

    JDB_CUDA_TRY(cudaMemcpyAsync(d_cp, child_ptr, (n + 1) * 4, cudaMemcpyHostToDevice, st));
    if (n_edges > 0) JDB_CUDA_TRY(cudaMemcpyAsync(d_ci, child_idx, (size_t)n_edges * 4, cudaMemcpyHostToDevice, st));
    jdb_forest f{d_cp, d_ci, n_nodes, n_edges};
    // per-level launches (tensor-core path beyond the cooperative kernel's hidden sizes) need the level count on the
    // host: there the analysis synchronises, and the forward is sized by the real number of internal nodes.  The copy
    // of x follows the analysis, so that this wait covers the CSR and the analysis only.
    const bool per_level = opts->precision == JDB_BF16 && !small_levels_supported(H);
    jdb_status s = per_level ? jdb_schedule(&f, &sch, d_sws, sws, stream) : jdb_schedule_async(&f, &sch, d_sws, sws, stream);
    if (s != JDB_OK) return s;
    JDB_CUDA_TRY(cudaMemcpyAsync(d_x, x, n * (size_t)D * xb, cudaMemcpyHostToDevice, st));
    // enqueue the forward and the copies back before the one synchronisation
    jdb_opts o = *opts;
    o.mode = JDB_MODE_AUTO;
    o.flags = (o.flags | JDB_FLAG_NO_SYNC) & ~JDB_FLAG_ROOTS_ONLY;  // the status is read once, together with the results
    s = jdb_treelstm_forward(&f, &sch, d_x, x_dtype, D, packed, D, H, d_h, d_c, (int64_t)ldh, &o, d_fws, fws, stream);
    if (s != JDB_OK) return s;
    if (opts->flags & JDB_FLAG_ROOTS_ONLY) {
        int* is_child = (int*)take(n * 4);
        int32_t* root_id = (int32_t*)take(n * 4);
        int* block_sum = (int*)take((n / SCAN_BLOCK + 2) * 4);
        float* hr = (float*)take(n * (size_t)H * 4);
        float* cr = (float*)take(n * (size_t)H * 4);
        const int n_roots = n_nodes > n_edges ? n_nodes - n_edges : 0;   // every other node has exactly one parent edge
        const int sb = n_nodes / SCAN_BLOCK + 1;
        JDB_CUDA_TRY(cudaMemsetAsync(is_child, 0, n * 4, st));
        if (n_edges > 0) mark_children_kernel<<<ceil_div(n_edges, 256), 256, 0, st>>>(d_ci, n_edges, n_nodes, is_child);
        root_count_kernel<<<sb, SCAN_BLOCK, 0, st>>>(is_child, n_nodes, block_sum);
        block_sums_scan_kernel<<<1, SCAN_BLOCK, 0, st>>>(block_sum, sb);
        root_list_kernel<<<sb, SCAN_BLOCK, 0, st>>>(is_child, n_nodes, block_sum, n_roots, root_id);
        if (n_roots > 0) {
            const dim3 blk(H >= 128 ? 128 : 32, H >= 128 ? 2 : 8);
            root_rows_kernel<<<ceil_div(n_roots, blk.y), blk, 0, st>>>(root_id, n_roots, H, d_h, d_c, (long long)ldh, hr, cr);
            JDB_CUDA_TRY(cudaGetLastError());
            JDB_CUDA_TRY(cudaMemcpyAsync(h, hr, (size_t)n_roots * H * 4, cudaMemcpyDeviceToHost, st));
            JDB_CUDA_TRY(cudaMemcpyAsync(c, cr, (size_t)n_roots * H * 4, cudaMemcpyDeviceToHost, st));
        }
        JDB_CUDA_TRY(cudaGetLastError());
    } else if (ldh == (size_t)H) {
        JDB_CUDA_TRY(cudaMemcpyAsync(h, d_h, n * (size_t)H * 4, cudaMemcpyDeviceToHost, st));
        JDB_CUDA_TRY(cudaMemcpyAsync(c, d_c, n * (size_t)H * 4, cudaMemcpyDeviceToHost, st));
    } else {
        JDB_CUDA_TRY(cudaMemcpy2DAsync(h, (size_t)H * 4, d_h, ldh * 4, (size_t)H * 4, n, cudaMemcpyDeviceToHost, st));
        JDB_CUDA_TRY(cudaMemcpy2DAsync(c, (size_t)H * 4, d_c, ldh * 4, (size_t)H * 4, n, cudaMemcpyDeviceToHost, st));
    }
    *meta_out = sch.meta;
    return JDB_OK;
}

// the status words of a request enqueued by forward_host_enqueue, after its stream has drained
jdb_status forward_host_finish(const int32_t* meta_dev, int32_t* n_levels_out, void* stream) {
    if (n_levels_out) *n_levels_out = 0;
    if (!meta_dev) return JDB_OK;   // an empty forest: nothing was enqueued
    int32_t meta[JDB_META_INTS];
    jdb_status s = read_meta(meta_dev, meta, (cudaStream_t)stream);
    if (s != JDB_OK) return s;
    if (n_levels_out) *n_levels_out = meta[META_N_LEVELS];
    return meta_status(meta);
}

}  // namespace jdb

extern "C" {

const char* jdb_status_string(jdb_status s) {
    switch (s) {
        case JDB_OK: return "ok";
        case JDB_ERR_INVALID_ARG: return "invalid argument";
        case JDB_ERR_NOT_A_FOREST: return "input is not a forest (bad child id, node with two parents, cycle, or bad child_ptr)";
        case JDB_ERR_WORKSPACE: return "workspace or packed-weight buffer too small";
        case JDB_ERR_UNSUPPORTED: return "size not supported by the compiled kernels";
        case JDB_ERR_CUDA: return "CUDA runtime error";
        case JDB_ERR_TIMEOUT: return "device-side wait timed out";
        case JDB_ERR_CHECK: return "debug checks: a kernel met an index outside its array (access skipped; see jdb_debug_report)";
    }
    return "unknown status";
}

int jdb_last_cuda_error(void) { return g_last_cuda_error; }

size_t jdb_schedule_workspace_bytes(int32_t n_nodes, int32_t n_edges) { return schedule_ws_bytes(n_nodes, n_edges); }

jdb_status jdb_schedule(const jdb_forest* forest, jdb_sched* out, void* ws, size_t ws_bytes, void* stream) {
    return schedule_common(forest, out, ws, ws_bytes, (cudaStream_t)stream, true);
}

jdb_status jdb_schedule_async(const jdb_forest* forest, jdb_sched* out, void* ws, size_t ws_bytes, void* stream) {
    return schedule_common(forest, out, ws, ws_bytes, (cudaStream_t)stream, false);
}

size_t jdb_packed_weights_bytes(int32_t D, int32_t H, int32_t precision) {
    if (D <= 0 || H <= 0) return 0;
    size_t bytes = pack_layout(D, H, precision).total;
    if (precision == JDB_BF16) bytes += tc_pack_layout(D, H).total;  // tensor-core layout follows the plain one
    return bytes;
}

jdb_status jdb_pack_weights(const float* W, const float* U, const float* b, int32_t D, int32_t H, int32_t precision,
                            void* packed, size_t packed_bytes, void* stream) {
    if (!W || !U || !b || !packed || D <= 0 || H <= 0) return JDB_ERR_INVALID_ARG;
    if (precision != JDB_FP32 && precision != JDB_BF16) return JDB_ERR_INVALID_ARG;
    if (((uintptr_t)packed & 255) != 0) return JDB_ERR_INVALID_ARG;
    PackLayout L = pack_layout(D, H, precision);
    if (packed_bytes < jdb_packed_weights_bytes(D, H, precision)) return JDB_ERR_WORKSPACE;
    jdb_status s = pack_weights_enqueue(W, U, b, L, packed, (cudaStream_t)stream);
    if (s != JDB_OK || precision != JDB_BF16) return s;
    return tc_pack_weights_enqueue(W, U, b, D, H, (char*)packed + L.total, (cudaStream_t)stream);
}

size_t jdb_forward_workspace_bytes(int32_t n_nodes, int32_t n_internal_bound, int32_t D, int32_t H, int32_t precision) {
    size_t bytes = forward_ws_bytes(n_nodes, n_internal_bound, D, H, precision);
    // fp32 beyond the cooperative kernel's hidden sizes: the level-by-level GEMM path keeps its arrays behind the plain one's
    if (precision == JDB_FP32 && H > 0 && !small_levels_f32_supported(H))
        bytes = align_up(bytes, 256) + forward_f32_gemm_ws_bytes(n_nodes, n_internal_bound, H);
    if (precision == JDB_BF16) {
        size_t tc = forward_tc_ws_bytes(n_nodes, n_internal_bound, D, H);
        if (tc > bytes) bytes = tc;
    }
    return bytes;
}

jdb_status jdb_treelstm_forward(const jdb_forest* forest, const jdb_sched* sched, const void* x, int32_t x_dtype,
                                int64_t ldx, const void* packed, int32_t D, int32_t H, float* h, float* c, int64_t ldh,
                                const jdb_opts* opts, void* ws, size_t ws_bytes, void* stream) {
    cudaStream_t st = (cudaStream_t)stream;
    jdb_status s = check_forest_args(forest);
    if (s != JDB_OK) return s;
    if (!sched || !opts || !packed || D <= 0 || H <= 0) return JDB_ERR_INVALID_ARG;
    if (opts->precision != JDB_FP32 && opts->precision != JDB_BF16) return JDB_ERR_INVALID_ARG;
    if (x_dtype != JDB_FP32 && x_dtype != JDB_BF16) return JDB_ERR_INVALID_ARG;
    if (opts->precision == JDB_FP32 && x_dtype != JDB_FP32) return JDB_ERR_INVALID_ARG;
    if (opts->mode < JDB_MODE_AUTO || opts->mode > JDB_MODE_PERSISTENT) return JDB_ERR_INVALID_ARG;
    const int N = forest->n_nodes;
    if (N == 0) return JDB_OK;
    if (!x || !h || !c || !sched->level_ptr || !sched->perm || !sched->meta) return JDB_ERR_INVALID_ARG;
    if (ldx < D || ldh < H) return JDB_ERR_INVALID_ARG;
    if (((uintptr_t)packed & 255) != 0 || !ws || ((uintptr_t)ws & 255) != 0) return JDB_ERR_INVALID_ARG;
    const bool known = sched->n_levels >= 0 && sched->n_leaves >= 0;
    const int n_internal_bound = known ? N - sched->n_leaves : N;
    if (ws_bytes < jdb_forward_workspace_bytes(N, n_internal_bound, D, H, opts->precision)) return JDB_ERR_WORKSPACE;

    // which level loop runs:
    //   fp32: plain-ALU kernels, per-level launches or one cooperative launch;
    //   bf16: tensor-core kernels; H <= 192 has a one-launch cooperative level loop (persistent mode), any H has
    //         the per-level launches.  Per-level launches need the level count on the host.
    int mode = opts->mode;
    bool tc = opts->precision == JDB_BF16, tc_small = false;
    if (tc) {
        const bool small_ok = small_levels_supported(H);
        if (mode == JDB_MODE_AUTO) mode = small_ok ? JDB_MODE_PERSISTENT : JDB_MODE_PER_LEVEL;
        if (mode == JDB_MODE_PERSISTENT) {
            if (small_ok) tc_small = true;
            else tc = false;  // no tensor-core cooperative kernel for this H: the plain-ALU one serves
        }
    } else {
        if (!known) mode = JDB_MODE_PERSISTENT;  // the level count lives on the device only
        if (mode == JDB_MODE_AUTO)
            mode = (small_levels_f32_supported(H) || sched->n_levels > 6) ? JDB_MODE_PERSISTENT : JDB_MODE_PER_LEVEL;
    }
    int n_levels_host = known ? sched->n_levels : -1;
    if (tc && !tc_small && !known) {
        // per-level launches from a schedule made without synchronisation: fetch the level count now
        int32_t meta[JDB_META_INTS];
        s = read_meta(sched->meta, meta, st);
        if (s != JDB_OK) return s;
        if (meta[META_ERROR] != 0 || meta[META_UNFINISHED] != 0) return JDB_ERR_NOT_A_FOREST;
        n_levels_host = meta[META_N_LEVELS];
    }

    PackLayout L = pack_layout(D, H, opts->precision);
    const char* pk = (const char*)packed;
    ForwardArgs a{};
    a.child_ptr = forest->child_ptr;
    a.child_idx = forest->child_idx;
    a.level_ptr = sched->level_ptr;
    a.perm = sched->perm;
    a.meta = sched->meta;
    a.n_nodes = N;
    a.n_edges = forest->n_edges;
    a.x = x;
    a.x_is_bf16 = x_dtype == JDB_BF16;
    a.ldx = ldx;
    a.bias = (const float*)(pk + L.off_bias);
    a.Wt = (const float*)(pk + L.off_Wt);
    a.Ut = (const float*)(pk + L.off_Ut);
    a.Uft = (const float*)(pk + L.off_Uft);
    a.D = D;
    a.H = H;
    a.round_bf16 = opts->precision == JDB_BF16;
    a.P = (float*)ws;
    a.h = h;
    a.c = c;
    a.ldh = ldh;
    a.ev_begin = (cudaEvent_t)opts->ev_begin;
    a.ev_xproj_done = (cudaEvent_t)opts->ev_xproj_done;
    a.ev_levels_done = (cudaEvent_t)opts->ev_levels_done;
    a.trace = (unsigned long long*)opts->trace;
    a.trace_cap = opts->trace ? opts->trace_cap : 0;
    a.depth = sched->depth;
    a.tuning = opts->tuning;
    a.debug = (opts->flags & JDB_FLAG_DEBUG_CHECKS) ? 1 : 0;

    // what an earlier forward on this schedule may have left: the timeout word, the barrier counter, the debug record
    JDB_CUDA_TRY(cudaMemsetAsync(sched->meta + META_TIMEOUT, 0, 2 * sizeof(int32_t), st));
    if (a.debug) JDB_CUDA_TRY(cudaMemsetAsync(sched->meta + META_CHECK, 0, 4 * sizeof(int32_t), st));
    const uint64_t tmo = opts->barrier_timeout_ns ? opts->barrier_timeout_ns : 2000000000ull;
    // fp32 with a hidden size beyond the cooperative kernel, level count known, no special request: level by level through
    // the tiled GEMM (2.5 times the plain-ALU level loop at H = 512); it reads the level table back, so a caller that
    // forbids synchronisation, asks for a mode or for the index checks keeps the plain-ALU kernels
    const bool f32_gemm = !tc && opts->precision == JDB_FP32 && known && opts->mode == JDB_MODE_AUTO && !small_levels_f32_supported(H) &&
                          !a.debug && !(opts->flags & JDB_FLAG_NO_SYNC);
    if (tc)
        s = forward_tc_enqueue(a, pk + L.total, n_levels_host, n_internal_bound, ws, tc_small, tmo, st);
    else if (f32_gemm) {
        s = forward_f32_gemm_enqueue(a, n_levels_host, n_internal_bound,
                                     (char*)ws + align_up(forward_ws_bytes(N, n_internal_bound, D, H, opts->precision), 256), st);
        mode = JDB_MODE_PER_LEVEL;   // nothing cooperative ran: no status to wait for
    } else
        s = forward_enqueue(a, n_levels_host, n_internal_bound, mode, tmo, st);
    if (s != JDB_OK) return s;
    if (a.debug || (mode == JDB_MODE_PERSISTENT && !(opts->flags & JDB_FLAG_NO_SYNC))) {
        int32_t meta[JDB_META_INTS];
        s = read_meta(sched->meta, meta, st);
        if (s != JDB_OK) return s;
        return meta_status(meta);
    }
    return JDB_OK;
}

jdb_status jdb_debug_report(const jdb_sched* sched, int32_t out[4], void* stream) {
    if (!sched || !sched->meta || !out) return JDB_ERR_INVALID_ARG;
    int32_t meta[JDB_META_INTS];
    jdb_status s = read_meta(sched->meta, meta, (cudaStream_t)stream);
    if (s != JDB_OK) return s;
    for (int i = 0; i < 4; ++i) out[i] = meta[META_CHECK + i];
    return JDB_OK;
}

jdb_status jdb_sched_status(const jdb_sched* sched, int32_t* n_levels_out, int32_t* n_leaves_out, void* stream) {
    if (!sched || !sched->meta) return JDB_ERR_INVALID_ARG;
    int32_t meta[JDB_META_INTS];
    jdb_status s = read_meta(sched->meta, meta, (cudaStream_t)stream);
    if (s != JDB_OK) return s;
    if (n_levels_out) *n_levels_out = meta[META_N_LEVELS];
    if (n_leaves_out) *n_leaves_out = meta[META_N_LEAVES];
    return meta_status(meta);
}

size_t jdb_forward_host_workspace_bytes(int32_t n_nodes, int32_t n_edges, int32_t D, int32_t H, int32_t precision,
                                        int32_t x_dtype) {
    size_t n = (size_t)(n_nodes > 0 ? n_nodes : 1), e = (size_t)(n_edges > 0 ? n_edges : 1);
    size_t xb = x_dtype == JDB_BF16 ? 2 : 4;
    size_t bytes = 0;
    bytes += align_up((n + 1) * 4, 256) + align_up(e * 4, 256);            // CSR
    bytes += align_up(n * (size_t)D * xb, 256);                            // x
    bytes += 2 * align_up(n * 4, 256) + align_up((n + 2) * 4, 256) + 256;  // depth, perm, level_ptr, meta
    bytes += 2 * align_up(n * (((size_t)H + 3) / 4 * 4) * 4, 256);         // h, c (rows padded to 16 bytes)
    bytes += align_up(schedule_ws_bytes(n_nodes, n_edges), 256);
    bytes += jdb_forward_workspace_bytes(n_nodes, n_nodes, D, H, precision);
    // JDB_FLAG_ROOTS_ONLY: child marks, root ids, block sums, and the compacted rows (at most every node is a root)
    bytes += 2 * align_up(n * 4, 256) + align_up((n / SCAN_BLOCK + 2) * 4, 256) + 2 * align_up(n * (size_t)H * 4, 256);
    return bytes;
}

jdb_status jdb_treelstm_forward_host(const int32_t* child_ptr, const int32_t* child_idx, int32_t n_nodes,
                                     int32_t n_edges, const void* x, int32_t x_dtype, const void* packed, int32_t D,
                                     int32_t H, float* h, float* c, const jdb_opts* opts, void* dev_ws,
                                     size_t dev_ws_bytes, int32_t* n_levels_out, void* stream) {
    if (n_levels_out) *n_levels_out = 0;
    int32_t* meta_dev = nullptr;
    jdb_status s = forward_host_enqueue(child_ptr, child_idx, n_nodes, n_edges, x, x_dtype, packed, D, H, h, c, opts, dev_ws,
                                        dev_ws_bytes, &meta_dev, stream);
    if (s != JDB_OK) return s;
    return forward_host_finish(meta_dev, n_levels_out, stream);
}

}  // extern "C"
