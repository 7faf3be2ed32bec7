// Internal declarations shared by the translation units of libjdb.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/jdb.h"

namespace jdb {

// indices into jdb_sched.meta
enum {
    META_N_LEVELS = 0,
    META_ERROR = 1,      // bit flags below
    META_MAX_DEPTH = 2,
    META_N_LEAVES = 3,
    META_UNFINISHED = 4, // nodes whose children never all completed (cycle or earlier error)
    META_TIMEOUT = 5,    // set by a grid barrier that gave up
    META_BARRIER = 6,    // grid barrier arrival counter (persistent mode)
    META_WIDE_LEVELS = 7, // how many levels 1, 2, ... in a row hold at least WIDE_LEVEL_NODES nodes
    META_CHECK = 8,       // JDB_FLAG_DEBUG_CHECKS: which check failed first (0 = none), then value, bound, where
};
// A level this large keeps every SM busy with its own launches (gather + two GEMMs); smaller ones are cheaper
// inside the cooperative level loop, whose cost per level is one grid barrier.
constexpr int WIDE_LEVEL_NODES = 65536;
enum { ERR_BAD_PTR = 1, ERR_RANGE = 2, ERR_TWO_PARENTS = 4 };

void set_last_cuda_error(cudaError_t e);

#define JDB_CUDA_TRY(expr)                            \
    do {                                              \
        cudaError_t e__ = (expr);                     \
        if (e__ != cudaSuccess) {                     \
            ::jdb::set_last_cuda_error(e__);          \
            return JDB_ERR_CUDA;                      \
        }                                             \
    } while (0)

// Per-device facts looked up once (the calls are cheap but they sit on the launch path of microsecond-scale steps).
struct DevInfo {
    int n_sm;
    int max_smem_optin;
    unsigned attr_mask;   // which kernels already had their shared-memory attribute set on this device
    int small_per_sm;     // resident CTAs per SM of the cooperative small-H kernel (0 = not asked yet)
};
enum { ATTR_SMALL_SCHED = 1, ATTR_GEMM_TC = 2, ATTR_SMALL_LEVELS = 4, ATTR_SMALL_F32 = 8 };
DevInfo* dev_info();  // of the current device; nullptr if the runtime fails

// JDB_FLAG_DEBUG_CHECKS: true if 0 <= v < bound.  Otherwise the first offender of the call is recorded in meta
// (what, value, bound, where) and the caller skips the access.
enum { CHECK_PERM = 1, CHECK_CHILD = 2, CHECK_POSITION = 3, CHECK_SLOT = 4, CHECK_PARENT_ROW = 5, CHECK_LEVEL_PTR = 6,
       CHECK_EDGE_PTR = 7 };
#ifdef __CUDACC__
__device__ __forceinline__ bool dbg_ok(int32_t* meta, int what, long long v, long long bound, int where) {
    if (v >= 0 && v < bound) return true;
    if (atomicCAS(&meta[META_CHECK], 0, what) == 0) {
        meta[META_CHECK + 1] = (int32_t)(v < -2147483647LL ? -2147483647LL : (v > 2147483647LL ? 2147483647LL : v));
        meta[META_CHECK + 2] = (int32_t)(bound > 2147483647LL ? 2147483647LL : bound);
        meta[META_CHECK + 3] = where;
    }
    return false;
}
// Positions [lo, hi) of a level; with debug checks an inconsistent pair is recorded and the level made empty (every
// reader of the same pair takes the same decision).
__device__ __forceinline__ void checked_level(const int32_t* level_ptr, int level, int n_nodes, int32_t* meta, int debug,
                                              int& lo, int& hi) {
    lo = level_ptr[level];
    hi = level_ptr[level + 1];
    if (debug && !(dbg_ok(meta, CHECK_LEVEL_PTR, lo, (long long)n_nodes + 1, level) &&
                   dbg_ok(meta, CHECK_LEVEL_PTR, hi, (long long)n_nodes + 1, level) &&
                   dbg_ok(meta, CHECK_LEVEL_PTR, hi - lo, (long long)n_nodes + 1, level)))
        lo = hi = 0;
}
#endif

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
static inline int ceil_div(long long a, long long b) { return (int)((a + b - 1) / b); }

// ---- schedule.cu ------------------------------------------------------------------------------
constexpr int SORT_BITS = 11;
constexpr int SORT_BINS = 1 << SORT_BITS;
constexpr int SORT_TILE = 4096;       // elements per block in a sort pass
constexpr int SMALL_SCHED_MAX = 6144; // forests up to this many nodes are analysed by one CTA

size_t schedule_ws_bytes(int32_t n_nodes, int32_t n_edges);
jdb_status schedule_enqueue(const jdb_forest& f, const jdb_sched& s, void* ws, size_t ws_bytes, cudaStream_t st);

// ---- weights.cu -------------------------------------------------------------------------------
// Layout of the packed weight buffer (all offsets in bytes, 256-aligned).
struct PackLayout {
    int32_t D, H, precision;
    size_t off_bias;      // float  [H][4]        bias, gates interleaved (i,o,u,f) per hidden index
    size_t off_Wt;        // float  [D][H][4]     W transposed: Wt[d][j][g] = W[g*H + j][d]
    size_t off_Ut;        // float  [H][H][4]     U transposed: Ut[k][j][g] = U[g*H + j][k]
    size_t off_Uft;       // float  [H][H]        forget block alone: Uft[k][j] = U[3H + j][k]
    size_t total;
};
PackLayout pack_layout(int32_t D, int32_t H, int32_t precision);
jdb_status pack_weights_enqueue(const float* W, const float* U, const float* b, const PackLayout& L, void* packed,
                                cudaStream_t st);

// ---- forward_simt.cu --------------------------------------------------------------------------
struct ForwardArgs {
    const int32_t* child_ptr;
    const int32_t* child_idx;
    const int32_t* level_ptr;
    const int32_t* perm;
    int32_t* meta;
    int32_t n_nodes, n_edges;
    const void* x;
    int32_t x_is_bf16;
    int64_t ldx;
    const float* bias;  // packed
    const float* Wt;    // packed
    const float* Ut;    // packed
    const float* Uft;   // packed
    int32_t D, H;
    int32_t round_bf16; // 1: round GEMM operands h~ and h_k to bf16 (weights/x are already rounded)
    float* P;           // [n_internal_bound][H][4] pre-activations of internal nodes, row = perm pos - n_leaves
    float* h;
    float* c;
    int64_t ldh;
    cudaEvent_t ev_begin, ev_xproj_done, ev_levels_done;  // optional timing hooks (null = none)
    unsigned long long* trace;                             // optional level trace (null = none)
    long long trace_cap;
    const int32_t* depth;                                  // jdb_sched.depth (may be null)
    int32_t tuning;                                        // jdb_opts.tuning
    int32_t debug;                                         // 1: JDB_FLAG_DEBUG_CHECKS
};
size_t forward_ws_bytes(int32_t n_nodes, int32_t n_internal_bound, int32_t D, int32_t H, int32_t precision);
jdb_status forward_enqueue(const ForwardArgs& a, int n_levels_host, int n_internal_bound, int mode,
                           uint64_t timeout_ns, cudaStream_t st);

// ---- forward_tc.cu ----------------------------------------------------------------------------
struct TcPackLayout {
    int32_t Hp, Kd;       // H and D rounded up to 64
    size_t off_bias;      // float [Hp][4]
    size_t off_W;         // bf16  [4 Hp][Kd]   gates interleaved per 64-wide hidden slice (i,o,u,f)
    size_t off_Uiou;      // bf16  [3 Hp][Hp]   gates interleaved per 64-wide hidden slice (i,o,u)
    size_t off_Uf;        // bf16  [Hp][Hp]
    size_t total;
};
TcPackLayout tc_pack_layout(int32_t D, int32_t H);
jdb_status tc_pack_weights_enqueue(const float* W, const float* U, const float* b, int32_t D, int32_t H, void* packed_tc,
                                   cudaStream_t st);
size_t forward_tc_ws_bytes(int32_t n_nodes, int32_t n_internal_bound, int32_t D, int32_t H);
// use_small: run the level loop as the one cooperative launch of forward_small.cu (H <= 192; n_levels may be
// unknown on the host) instead of per-level launches (n_levels must be known)
jdb_status forward_tc_enqueue(const ForwardArgs& fa, const void* packed_tc, int n_levels, int n_internal_bound,
                              void* ws, bool use_small, uint64_t timeout_ns, cudaStream_t st);

// ---- batcher.cu ------------------------------------------------------------------------------
// fp32 forward through the tiled GEMM for hidden sizes the cooperative fp32 kernel does not hold; needs the level count
// on the host and synchronises once for the level table
size_t forward_f32_gemm_ws_bytes(int32_t n_nodes, int32_t n_internal_bound, int32_t H);
jdb_status forward_f32_gemm_enqueue(const ForwardArgs& a, int n_levels, int n_internal_bound, void* ws, cudaStream_t st);

// ---- api.cu ----------------------------------------------------------------------------------
// one request from host buffers: enqueue everything on `stream` (copies in, analysis, forward, copies back) without
// waiting, and read the recorded status once the stream has drained
jdb_status forward_host_enqueue(const int32_t* child_ptr, const int32_t* child_idx, int32_t n_nodes, int32_t n_edges,
                                const void* x, int32_t x_dtype, const void* packed, int32_t D, int32_t H, float* h, float* c,
                                const jdb_opts* opts, void* dev_ws, size_t dev_ws_bytes, int32_t** meta_out, void* stream);
jdb_status forward_host_finish(const int32_t* meta_dev, int32_t* n_levels_out, void* stream);

// ---- partition.cu -----------------------------------------------------------------------------
// Tree partition for the cooperative level loop: nodes ordered by (depth, group) and the offsets of every
// (depth, group) range; gbar holds one barrier counter per group (zeroed by partition_enqueue).
constexpr long long PARTITION_TABLE_MAX = 1 << 20;   // (depth, group) pairs the offset table can hold
constexpr int PARTITION_MAX_GROUPS = 1024;
struct Partition {
    const int32_t* gperm;  // [n_nodes]
    const int32_t* goff;   // [n_levels * G + 1]
    int32_t* gbar;         // [G]
    int32_t G;             // 0: no partition (levels are separated by grid-wide barriers)
};
size_t partition_ws_bytes(int32_t n_nodes);
jdb_status partition_enqueue(const ForwardArgs& fa, const int32_t* depth, int n_levels, int G, void* ws, Partition* out, cudaStream_t st);

// ---- forward_small.cu -------------------------------------------------------------------------
bool small_levels_supported(int32_t H);
// hb: bf16 copy of h, [n_nodes][Hp], rows in level order (leaf rows filled by the input projection);
// inv: position of every node in level order
// part: tree partition (G > 0: every group of CTAs walks its own trees, synchronising inside the group only), or G = 0
int small_levels_groups(int32_t H, int n_internal_bound);   // CTA groups the cooperative launch will have (0: unsupported)
jdb_status small_levels_enqueue(const ForwardArgs& fa, const void* packed_tc, const float* P, void* hb, const int32_t* inv,
                                int n_internal_bound, int first_level, uint64_t timeout_ns, const Partition& part, cudaStream_t st);

// ---- forward_small_f32.cu ---------------------------------------------------------------------
// the fp32 level loop as one cooperative launch with resident weight slices (H <= 192); reads fa.P as written by
// the fp32 input projection
bool small_levels_f32_supported(int32_t H);
jdb_status small_levels_f32_enqueue(const ForwardArgs& fa, int n_internal_bound, uint64_t timeout_ns, cudaStream_t st);

}  // namespace jdb
